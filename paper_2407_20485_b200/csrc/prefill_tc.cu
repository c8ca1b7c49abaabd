// Tensor-core prefill for 16-bit storage and d = 128 (sm_100a: TMA + tcgen05 + TMEM).
//
//   score pass (paper Eq. 5-6):  S_j = sum_{i>=j} alpha^(n-1-i) * exp(s_ij - lse_i)
//     One CTA owns 128 keys.  The logits are recomputed transposed, S^T = K_blk * Q_tile^T,
//     so that a key is a TMEM lane: the threads that own the lane sum its key's
//     probabilities over all query rows i >= j in a fixed order.  No atomics: the result
//     is deterministic.
//
// Warp roles per CTA (320 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM
// owner, warps 2-9 = epilogue.  A key is shared by two threads, one per 64-row half of the
// query tile (more warps per scheduler keep the special-function unit fed); each keeps its
// own running sum in row order and the two are added once at the end, in a fixed order.
#include <algorithm>
#include <mutex>
#include <type_traits>

#include "common.cuh"
#include "tc_sm100.cuh"

namespace a2sf {

A2SF_DEBUG_TRANSLATION_UNIT(prefill_tc)

// sticky device-side status: set when a bounded wait runs out
static __device__ int g_tc_status = 0;

namespace {

using namespace tc;

constexpr int kBlk = 128;                   // keys per CTA = TMEM lanes; query rows per tile
constexpr int kD = 128;
constexpr int kHalfBytes = kBlk * 64 * 2;   // one 64-column swizzled half of a tile: 16 KB
constexpr int kTileBytes = 2 * kHalfBytes;  // 32 KB
constexpr int kScoreStages = 2;
constexpr int kScoreThreads = 320;           // producer warp, MMA warp, 8 epilogue warps
constexpr int kScoreEpiThreads = 256;
// Ring of row-constant vectors written by the producer warp.  Slot x%ring is rewritten for tile x
// after the MMAs of tile x-2 have retired; those needed the accumulator that tile x-4 held, i.e.
// every epilogue thread had finished the arithmetic of tile x-5.  Any depth >= 5 is safe.
constexpr int kScoreCRing = 8;

struct ScoreArgs {
    const float *lse;     // [U][n]
    float *scores;        // [U][n]
    int n, H;
    int G;                // query heads per key/value head
    float sl2;            // scale * log2(e)
    float alpha;          // forgetting factor, or per unit:
    const float *alpha_vec;
    int skip_zero_rows;   // leave out query tiles whose forgetting weight underflows to exactly 0
    int window_rows;      // only the last window_rows query rows enter the sum (0 = all)
};

struct ScoreShared {
    uint64_t k_full, q_full[kScoreStages], q_empty[kScoreStages], acc_full[2], acc_empty[2];
    uint64_t c_ready[kScoreCRing];
    uint32_t tmem_base;
    int abort_flag;
    float cbuf[kScoreCRing][kBlk];   // row constants of the query tiles in flight
    float part[kBlk];           // upper-half partial sums, added to the lower half at the end
};

constexpr size_t kScoreSmemBytes = 1024 /*alignment slack*/ + kTileBytes * (1 + kScoreStages) +
                                   sizeof(ScoreShared);

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Two fp32 operations per instruction (sm_100 packed arithmetic on register pairs).
__device__ __forceinline__ uint64_t pack_f32x2(uint32_t lo, uint32_t hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}

// The issuing thread is the bottleneck of small-tile UMMA pipelines, so descriptors are built
// once per operand buffer and only advanced by a constant per K-step.
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t smem_addr)
{
    return make_sdesc_sw128(smem_addr, 16, 1024);
}

// 8 K-steps of 16 elements over a [128 x 128] K-major operand pair stored as two 64-column
// swizzled halves: step k starts (k/4) halves + (k%4)*32 bytes into the tile (16-byte units).
__device__ __forceinline__ void issue_qk_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                             uint32_t idesc)
{
#pragma unroll
    for (int k = 0; k < kD / 16; ++k) {
        const uint64_t off = (uint64_t)(((k >> 2) * kHalfBytes + (k & 3) * 32) >> 4);
        umma_ss(d_tmem, a_desc + off, b_desc + off, idesc, k > 0);
    }
}

// Sum of exp2(s*sl2 - c_i) over this thread's 64 query rows of the tile.  Masked: rows
// below `first_row` (relative to the strip) lie above the diagonal and contribute nothing.
template <bool Masked>
__device__ __forceinline__ float strip_sum(const uint32_t (&r)[2][32], const float *cb, float sl2,
                                           int first_row)
{
    float part[4] = {0.f, 0.f, 0.f, 0.f};           // four independent add chains
#pragma unroll
    for (int c = 0; c < 2; ++c) {
#pragma unroll
        for (int x = 0; x < 32; x += 4) {
            const float4 c4 = *reinterpret_cast<const float4 *>(cb + c * 32 + x);
            const float cc[4] = {c4.x, c4.y, c4.z, c4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float pw = ex2_approx(fmaf(__uint_as_float(r[c][x + e]), sl2, -cc[e]));
                if (Masked) pw = (c * 32 + x + e >= first_row) ? pw : 0.f;   // rows i >= j
                part[e] += pw;
            }
        }
    }
    return (part[0] + part[1]) + (part[2] + part[3]);
}

__global__ void __launch_bounds__(kScoreThreads, 2)
score_pass_tc(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
              ScoreArgs a, int ab_fmt)
{
    // once any CTA has given up on a wait, the rest of the grid drains without working
    __shared__ int s_skip;
    if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile int *>(&g_tc_status);
    __syncthreads();
    if (s_skip) return;

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                ~uintptr_t(1023));
    uint8_t *Ks = smem;
    uint8_t *Qs = smem + kTileBytes;
    ScoreShared *sh = reinterpret_cast<ScoreShared *>(smem + kTileBytes * (1 + kScoreStages));

    // CTAs of one unit are adjacent in the grid, so they run together and share the unit's
    // Q and K tiles through L2
    const int ntile_total = (a.n + kBlk - 1) / kBlk;
    const int u = blockIdx.x / ntile_total, kb = blockIdx.x % ntile_total;
    const int b = u / a.H, h = u % a.H;
    // Rows older than 127/(-log2 alpha) carry a weight below 2^-127: their flushed fp32
    // exponential is exactly 0, so leaving their tiles out changes no bit of the result.
    const float alpha = unit_alpha(a.alpha_vec, u, a.alpha);
    const float neg_log2_alpha = alpha > 0.f ? -log2f(alpha) : INFINITY;   // alpha = 0: only row n-1
    int t_first = kb;
    if (a.skip_zero_rows && neg_log2_alpha > 0.f) {
        const float span = ceilf(127.f / neg_log2_alpha);                  // first age with weight 0
        const int i_min = span >= (float)a.n ? 0 : min(a.n - 1, a.n - (int)span);
        t_first = max(kb, i_min / kBlk);
    }
    // truncated sum: rows before n - window_rows are left out (their constants become +inf)
    const int i_window = a.window_rows > 0 ? max(0, a.n - a.window_rows) : 0;
    t_first = max(t_first, i_window / kBlk);
    const int ntiles = ntile_total - t_first;          // query-row tiles t_first .. last
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &sh->abort_flag;

    if (threadIdx.x == 0) {
        mbar_init(&sh->k_full, 1);
        for (int s = 0; s < kScoreStages; ++s) { mbar_init(&sh->q_full[s], 1); mbar_init(&sh->q_empty[s], 1); }
        for (int x = 0; x < 2; ++x) {
            mbar_init(&sh->acc_full[x], 1);
            mbar_init(&sh->acc_empty[x], kScoreEpiThreads);
        }
        for (int x = 0; x < kScoreCRing; ++x) mbar_init(&sh->c_ready[x], 1);
        sh->abort_flag = 0;
        fence_mbar_init();
        // the K block and the first query tiles are requested here, before the tensor-memory
        // allocation and the CTA-wide barrier, so that their latency overlaps the set-up
        prefetch_tmap(&tmap_q);
        prefetch_tmap(&tmap_k);
        mbar_arrive_expect_tx(&sh->k_full, kTileBytes);
        tma_load_4d(Ks, &tmap_k, &sh->k_full, 0, kb * kBlk, h / a.G, b);
        tma_load_4d(Ks + kHalfBytes, &tmap_k, &sh->k_full, 64, kb * kBlk, h / a.G, b);
        for (int it = 0; it < kScoreStages && it < ntiles; ++it) {
            mbar_arrive_expect_tx(&sh->q_full[it], kTileBytes);
            uint8_t *dst = Qs + it * kTileBytes;
            tma_load_4d(dst, &tmap_q, &sh->q_full[it], 0, (t_first + it) * kBlk, h, b);
            tma_load_4d(dst + kHalfBytes, &tmap_q, &sh->q_full[it], 64, (t_first + it) * kBlk, h, b);
        }
    }
    if (warp == 1) {
        tmem_alloc(&sh->tmem_base, 256);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;

    if (warp == 0) {
        // ---- TMA producer; its 32 lanes also prepare the row constants ------------------
        //   c_i = lse_i*log2e + (n-1-i)*(-log2 alpha);  rows past n give +inf (weight 0).
        // They are written one tile ahead of the tensor core, so the epilogue warps never meet
        // at a barrier of their own and drift freely against each other.
        const float *lse = a.lse + (size_t)u * a.n;
        int issued = min(ntiles, kScoreStages);      // requested during set-up
        for (int it = 0; it < ntiles; ++it) {
            const int s = it % kScoreStages;
            const uint32_t ph = (it / kScoreStages) & 1;
            const int i0 = (t_first + it) * kBlk;
            // the constants' global loads are in flight while lane 0 waits for the stage
            float c4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int i = i0 + lane * 4 + e;
                const int age = a.n - 1 - i;
                c4[e] = (i < a.n && i >= i_window) ? fmaf(__ldg(lse + i), kLog2e, age == 0 ? 0.f : (float)age * neg_log2_alpha)
                                : INFINITY;
            }
            int ok = 1;
            if (lane == 0 && it >= kScoreStages) {
                ok = mbar_wait(&sh->q_empty[s], ph ^ 1, abort_flag) ? 1 : 0;
                if (ok) {
                    mbar_arrive_expect_tx(&sh->q_full[s], kTileBytes);
                    uint8_t *dst = Qs + s * kTileBytes;
                    tma_load_4d(dst, &tmap_q, &sh->q_full[s], 0, i0, h, b);
                    tma_load_4d(dst + kHalfBytes, &tmap_q, &sh->q_full[s], 64, i0, h, b);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            issued = max(issued, it + 1);
            if (A2SF_IN_RANGE(lane * 4 + 3, kBlk, kDbgScoreTc))
                *reinterpret_cast<float4 *>(&sh->cbuf[it % kScoreCRing][lane * 4]) =
                    make_float4(c4[0], c4[1], c4[2], c4[3]);
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->c_ready[it % kScoreCRing]);
        }
        if (lane == 0 && *abort_flag) {
            // give copies still in flight a bounded chance to land before the CTA exits
            int dummy = 0;
            for (int it = max(0, issued - kScoreStages); it < issued; ++it)
                mbar_wait(&sh->q_full[it % kScoreStages], (it / kScoreStages) & 1, &dummy);
            mbar_wait(&sh->k_full, 0, &dummy);
        }
    } else if (warp == 1) {
        // ---- MMA issuer -------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = make_idesc(ab_fmt, kBlk, kBlk, 0, 0);
            const uint64_t k_desc = kmajor_desc(smem_u32(Ks));
            uint64_t q_desc[kScoreStages];
            for (int s = 0; s < kScoreStages; ++s) q_desc[s] = kmajor_desc(smem_u32(Qs + s * kTileBytes));
            bool ok = mbar_wait(&sh->k_full, 0, abort_flag);
            for (int it = 0; ok && it < ntiles; ++it) {
                const int s = it % kScoreStages;
                const uint32_t ph = (it / kScoreStages) & 1;
                const int acc = it & 1;
                const uint32_t aph = (it >> 1) & 1;
                if (!mbar_wait(&sh->q_full[s], ph, abort_flag)) break;
                if (!mbar_wait(&sh->acc_empty[acc], aph ^ 1, abort_flag)) break;
                tc_fence_after_sync();
                issue_qk_mma(tmem_base + acc * kBlk, k_desc, q_desc[s], idesc);
                umma_commit(&sh->q_empty[s]);       // the stage is free once these MMAs retire
                umma_commit(&sh->acc_full[acc]);
            }
        }
    } else {
        // ---- epilogue: two threads per key (64 query rows of the tile each) -----------------
        const int quarter = warp & 3;               // TMEM lanes this warp may touch
        const int hsel = (warp - 2) >> 2;           // which half of the tile's query rows
        const int key_lane = quarter * 32 + lane;
        const int j = kb * kBlk + key_lane;
        // A failed wait poisons the CTA: later waits return at once and the loop keeps its
        // shape, so every thread still reaches the final barrier; the status word reports it.
        auto wait = [&](uint64_t *bar, uint32_t parity) -> bool {
            if (*abort_flag) return false;
            return mbar_wait(bar, parity, abort_flag);
        };
        float sum = 0.f;
        for (int it = 0; it < ntiles; ++it) {
            const int acc = it & 1;
            const uint32_t aph = (it >> 1) & 1;
            const int i0 = (t_first + it) * kBlk;
            wait(&sh->c_ready[it % kScoreCRing], (it / kScoreCRing) & 1);
            wait(&sh->acc_full[acc], aph);
            tc_fence_after_sync();
            const float *cb = sh->cbuf[it % kScoreCRing] + hsel * 64;
            const bool diag = (t_first + it == kb);
            // this thread's 64-row strip comes into registers with one wait, and the
            // accumulator buffer goes back to the tensor core before the arithmetic starts
            uint32_t r[2][32];
            const uint32_t t_addr = tmem_base + acc * kBlk + hsel * 64 + ((uint32_t)(quarter * 32) << 16);
            tmem_ld32(t_addr, r[0]);
            tmem_ld32(t_addr + 32, r[1]);
            tmem_wait_ld();
            tc_fence_before_sync();
            mbar_arrive(&sh->acc_empty[acc]);
            // only the diagonal tile needs the causal test; the others run the bare
            // multiply-add / exponential / add per logit
            if (diag) sum += strip_sum<true>(r, cb, a.sl2, j - (i0 + hsel * 64));
            else      sum += strip_sum<false>(r, cb, a.sl2, 0);
        }
        if (hsel == 1) sh->part[key_lane] = sum;
        named_barrier(1, kScoreEpiThreads);
        if (hsel == 0 && j < a.n && !*abort_flag && A2SF_IN_RANGE(key_lane, kBlk, kDbgScoreTc) &&
            A2SF_IN_RANGE((size_t)u * a.n + j, (size_t)gridDim.x / ntile_total * a.n, kDbgScoreTc))
            a.scores[(size_t)u * a.n + j] = sum + sh->part[key_lane];
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 256);
    }
    if (threadIdx.x == 0 && sh->abort_flag) g_tc_status = A2SF_ERR_TIMEOUT;
}


// ============================================================================================
// Attention pass (paper Eq. 3: causal softmax attention):  out_i = sum_j P_ij v_j,  lse_i.
//
// One CTA owns TWO adjacent 128-row query tiles ("streams" A and B) that share every K/V tile.
// The tensor core alternates between the streams,
//     S_A(0) S_B(0) | PV_A(0) S_A(1) | PV_B(0) S_B(1) | PV_A(1) S_A(2) | ...
// so that while one stream's rows are in the softmax warps the other stream's MMAs run.
//   S = Q K^T        -> TMEM, 128 fp32 columns per stream
//   softmax warps    : two threads per row.  The row's reference (what is subtracted before the
//                      exponential) moves lazily: a tile is first computed against the current
//                      one and redone, with the exact row maximum and a rescaled accumulator,
//                      only if its row sum shows that a probability may have left fp16's range.
//                      P, rounded
//                      to the storage type, is written back into the SAME tensor-memory columns
//                      the logits came from and is read from there as the A operand of the next
//                      MMA: shared-memory bandwidth is the scarce resource (two operands read
//                      from it at 128x128x16 per instruction already saturate it).  The row sum
//                      uses the unrounded values.
//   O += P V         -> TMEM, 128 fp32 columns per stream; V is consumed as an MN-major operand
//                      straight from its TMA tile
// Tensor memory: S/P_A | O_A | S/P_B | O_B = 512 columns.
// Warp roles (320 threads): warp 0 TMA producer, warp 1 MMA issuer / TMEM owner, warps 2-9
// softmax + epilogue: two threads per query row (64 logits each), all eight warps on one
// stream's tile at a time, the streams taken in turn.
// Measured on the longest CTA (63 stream tiles, 2393 clocks each against 1440 of tensor work,
// before the row-maximum pass became the exception): the softmax warps spent 65 % of their time
// in the exponential pass at ~12 clocks per logit per scheduler -- the special-function unit
// issues one warp instruction per 8 clocks and the other ~3.5 instructions per logit do not hide
// behind it -- and 8 % on the row maximum.  Every instruction per logit counts: dropping the
// maximum pass from the common path paid, while moving part of the exponentials to an FMA-pipe
// polynomial (+11 instructions each) or the fp16 packing to integer instructions made the
// pass slower, so neither is used.
// ============================================================================================
constexpr int kAttnThreads = 320;
constexpr int kKStages = 3;                  // K tiles in flight
constexpr int kVStages = 2;                  // V tiles in flight
constexpr float kRescaleThreshold = 8.0f;    // log2 units
constexpr float kOptimisticLimit = 32768.f;  // a row sum below this keeps every probability < 2^15

struct AttnArgs {
    void *out;            // [B][H][n][d], strides below
    float *lse;           // [U][n]
    int64_t st_b, st_h, st_t;
    int n, H;
    int G;                // query heads per key/value head
    float sl2;            // scale * log2(e)
    const int *v_flag;    // bf16 storage: 0 = the fp16 copy of V is exact, 1 = it is not
};

struct AttnShared {
    uint64_t q_full, k_full[kKStages], k_empty[kKStages], v_full[kVStages], v_empty[kVStages];
    uint64_t s_full[2], p_full[2], o_done[2];       // per stream
    uint32_t tmem_base;
    int abort_flag;
    float xch[2][2][kBlk];                          // [stream][column half][row]: row maxima / sums
};

// Q_A, Q_B, K ring, V ring.  The kernel has no static shared memory and declares the dynamic
// array 1024-byte aligned (the 128-byte swizzle pattern repeats every 1024 bytes), so no slack
// is added: the seven tiles leave 3 KB for the barriers and the exchange buffer.
constexpr size_t kAttnSmemBytes = kTileBytes * (2 + kKStages + kVStages) + sizeof(AttnShared);
static_assert(kAttnSmemBytes <= 227 * 1024, "attention pass shared memory");

template <typename T> __device__ __forceinline__ uint32_t pack2(float a, float b);
template <> __device__ __forceinline__ uint32_t pack2<__nv_bfloat16>(float a, float b)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&v);
}
template <> __device__ __forceinline__ uint32_t pack2<__half>(float a, float b)
{
    __half2 v = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&v);
}

// PvHalf (bf16 storage only): the P V product runs in fp16 -- P is rounded to fp16 (11
// significand bits, one term) and V comes from an fp16 copy made beforehand.  That form is valid
// only if the copy is exact; otherwise the plain bf16 form, which writes P as two bf16 terms,
// does the work (attn_pass_bf16_auto picks one of the two on the device).
template <typename T, bool PvHalf>
__device__ __forceinline__ void attn_body(const CUtensorMap *tmap_q, const CUtensorMap *tmap_k,
                                          const CUtensorMap *tmap_v, const AttnArgs &a)
{
    // once any CTA has given up on a wait, the rest of the grid drains without working
    extern __shared__ __align__(1024) uint8_t attn_smem[];
    {
        int skip = 0;
        if (threadIdx.x == 0) {
            skip = *reinterpret_cast<volatile int *>(&g_tc_status);
            if (smem_u32(attn_smem) & 1023u) {           // the swizzled tiles need this alignment
                g_tc_status = A2SF_ERR_CUDA;
                skip = 1;
            }
        }
        if (__syncthreads_or(skip)) return;
    }
    uint8_t *smem = attn_smem;
    uint8_t *Qs = smem;                                  // two tiles: stream A, stream B
    uint8_t *Ks = smem + 2 * kTileBytes;
    uint8_t *Vs = Ks + kKStages * kTileBytes;
    AttnShared *sh = reinterpret_cast<AttnShared *>(Vs + kVStages * kTileBytes);

    constexpr int ab_fmt = std::is_same<T, __nv_bfloat16>::value ? 1 : 0;
    using PT = typename std::conditional<PvHalf, __half, T>::type;      // element type of P and V
    constexpr int pv_fmt = std::is_same<PT, __nv_bfloat16>::value ? 1 : 0;
    // A bf16 probability keeps 8 significand bits; where the products p*v cancel, that
    // rounding alone exceeds the output tolerance.  For bf16 the probabilities are therefore
    // split into two bf16 terms (p = hi + lo, |lo| <= 2^-9 |hi|) and both are multiplied
    // with V.  fp16 keeps 11 bits and needs no second term.
    constexpr bool kSplitP = std::is_same<PT, __nv_bfloat16>::value;

    // CTAs of one unit are adjacent in the grid (longest rows first), so they run together
    // and share the unit's K and V tiles through L2
    const int T_total = (a.n + kBlk - 1) / kBlk;
    const int npairs = (T_total + 1) / 2;
    const int u = blockIdx.x / npairs;
    const int pair = npairs - 1 - blockIdx.x % npairs;
    const int rbA = 2 * pair, rbB = 2 * pair + 1;
    const bool hasB = rbB < T_total;
    const int ntA = rbA + 1;                            // key tiles 0 .. rbA
    const int ntB = hasB ? rbB + 1 : 0;
    const int nt = hasB ? ntB : ntA;
    const int b = u / a.H, h = u % a.H;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &sh->abort_flag;

    if (threadIdx.x == 0) {
        mbar_init(&sh->q_full, 1);
        for (int s = 0; s < kKStages; ++s) { mbar_init(&sh->k_full[s], 1); mbar_init(&sh->k_empty[s], 1); }
        for (int s = 0; s < kVStages; ++s) { mbar_init(&sh->v_full[s], 1); mbar_init(&sh->v_empty[s], 1); }
        for (int x = 0; x < 2; ++x) {
            mbar_init(&sh->s_full[x], 1);
            mbar_init(&sh->p_full[x], 2 * kBlk);
            mbar_init(&sh->o_done[x], 1);
        }
        sh->abort_flag = 0;
        fence_mbar_init();
        // The first tiles are requested here, before the tensor-memory allocation and the
        // CTA-wide barrier: their latency (about 5000 clocks until Q and K arrive) is the
        // longest item of a CTA's start-up.
        prefetch_tmap(tmap_q); prefetch_tmap(tmap_k); prefetch_tmap(tmap_v);
        mbar_arrive_expect_tx(&sh->q_full, hasB ? 2 * kTileBytes : kTileBytes);
        tma_load_4d(Qs, tmap_q, &sh->q_full, 0, rbA * kBlk, h, b);
        tma_load_4d(Qs + kHalfBytes, tmap_q, &sh->q_full, 64, rbA * kBlk, h, b);
        if (hasB) {
            tma_load_4d(Qs + kTileBytes, tmap_q, &sh->q_full, 0, rbB * kBlk, h, b);
            tma_load_4d(Qs + kTileBytes + kHalfBytes, tmap_q, &sh->q_full, 64, rbB * kBlk, h, b);
        }
        const int hk0 = h / a.G;
        mbar_arrive_expect_tx(&sh->k_full[0], kTileBytes);
        tma_load_4d(Ks, tmap_k, &sh->k_full[0], 0, 0, hk0, b);
        tma_load_4d(Ks + kHalfBytes, tmap_k, &sh->k_full[0], 64, 0, hk0, b);
        mbar_arrive_expect_tx(&sh->v_full[0], kTileBytes);
        tma_load_4d(Vs, tmap_v, &sh->v_full[0], 0, 0, hk0, b);
        tma_load_4d(Vs + kHalfBytes, tmap_v, &sh->v_full[0], 64, 0, hk0, b);
    }
    if (warp == 1) {
        tmem_alloc(&sh->tmem_base, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;

    // A failed wait poisons the CTA: every later wait returns at once, loops keep their shape,
    // and the status word reports the timeout.
    auto wait = [&](uint64_t *bar, uint32_t parity) -> bool {
        if (*abort_flag) return false;
        return mbar_wait(bar, parity, abort_flag);
    };

    if (warp == 0) {
        // ---- TMA producer -------------------------------------------------------------
        if (lane == 0) {
            // Q and the first K and V tiles were requested during set-up
            const int hk = h / a.G;                   // the K/V head this query head reads
            int k_issued = 1, v_issued = 1;
            for (int t = 1; t < nt; ++t) {
                const int ks = t % kKStages, vs = t % kVStages;
                if (!A2SF_IN_RANGE(t * kBlk, a.n, kDbgAttnTc)) break;      // a tile past the prompt is never requested
                if (!wait(&sh->k_empty[ks], ((t / kKStages) & 1) ^ 1)) break;
                mbar_arrive_expect_tx(&sh->k_full[ks], kTileBytes);
                tma_load_4d(Ks + ks * kTileBytes, tmap_k, &sh->k_full[ks], 0, t * kBlk, hk, b);
                tma_load_4d(Ks + ks * kTileBytes + kHalfBytes, tmap_k, &sh->k_full[ks], 64, t * kBlk, hk, b);
                k_issued = t + 1;
                if (!wait(&sh->v_empty[vs], ((t / kVStages) & 1) ^ 1)) break;
                mbar_arrive_expect_tx(&sh->v_full[vs], kTileBytes);
                tma_load_4d(Vs + vs * kTileBytes, tmap_v, &sh->v_full[vs], 0, t * kBlk, hk, b);
                tma_load_4d(Vs + vs * kTileBytes + kHalfBytes, tmap_v, &sh->v_full[vs], 64, t * kBlk, hk, b);
                v_issued = t + 1;
            }
            if (*abort_flag) {
                // bounded chance for copies in flight to land before the CTA exits
                int dummy = 0;
                for (int t = max(0, k_issued - kKStages); t < k_issued; ++t)
                    mbar_wait(&sh->k_full[t % kKStages], (t / kKStages) & 1, &dummy);
                for (int t = max(0, v_issued - kVStages); t < v_issued; ++t)
                    mbar_wait(&sh->v_full[t % kVStages], (t / kVStages) & 1, &dummy);
                mbar_wait(&sh->q_full, 0, &dummy);
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer -----------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc_qk = make_idesc(ab_fmt, kBlk, kBlk, 0, 0);
            const uint32_t idesc_pv = make_idesc(pv_fmt, kBlk, kD, 0, 1);     // V is MN-major
            uint64_t q_desc[2], k_desc[kKStages], v_desc[kVStages];
            for (int x = 0; x < 2; ++x) q_desc[x] = kmajor_desc(smem_u32(Qs + x * kTileBytes));
            for (int x = 0; x < kKStages; ++x) k_desc[x] = kmajor_desc(smem_u32(Ks + x * kTileBytes));
            // V as an MN-major operand: 64-wide d halves 16 KB apart, 8-key groups 1024 bytes apart
            for (int x = 0; x < kVStages; ++x)
                v_desc[x] = make_sdesc_sw128(smem_u32(Vs + x * kTileBytes), kHalfBytes, 1024);
            // S_X(t) = Q_X K_t^T into stream X's logits columns
            auto issue_s = [&](int X, int t) {
                issue_qk_mma(tmem_base + X * 2 * kBlk, q_desc[X], k_desc[t % kKStages], idesc_qk);
                umma_commit(&sh->s_full[X]);
            };
            // O_X += P_X(t) V_t with P read from stream X's logits columns
            auto issue_pv = [&](int X, int t) {
                const uint64_t vd = v_desc[t % kVStages];
                const uint32_t sp = tmem_base + X * 2 * kBlk, o = sp + kBlk;
                // 16 keys per step: 8 columns of packed P; two 8-key groups of V = 2048 bytes.
                // Keys 64h .. 64h+63 have their P at columns 64h .. 64h+31 (second term of the
                // two-term form at 64h+32 .. 64h+63): each softmax thread writes only over the
                // logits columns it has read itself.
#pragma unroll
                for (int k = 0; k < kBlk / 16; ++k)
                    umma_ts(o, sp + 64 * (k >> 2) + 8 * (k & 3), vd + (uint64_t)(k * 2048 >> 4), idesc_pv,
                            (t > 0) || (k > 0));
                if (kSplitP) {
#pragma unroll
                    for (int k = 0; k < kBlk / 16; ++k)
                        umma_ts(o, sp + 64 * (k >> 2) + 32 + 8 * (k & 3), vd + (uint64_t)(k * 2048 >> 4),
                                idesc_pv, 1);
                }
                umma_commit(&sh->o_done[X]);
            };
            wait(&sh->q_full, 0);
            wait(&sh->k_full[0], 0);
            tc_fence_after_sync();
            issue_s(0, 0);
            if (hasB) issue_s(1, 0);
            umma_commit(&sh->k_empty[0]);
            for (int t = 0; t < nt; ++t) {
                const bool nextA = t + 1 < ntA, nextB = t + 1 < ntB;
                wait(&sh->v_full[t % kVStages], (t / kVStages) & 1);
                if (nextA || nextB) wait(&sh->k_full[(t + 1) % kKStages], ((t + 1) / kKStages) & 1);
                if (t < ntA) {
                    wait(&sh->p_full[0], t & 1);
                    tc_fence_after_sync();
                    issue_pv(0, t);
                    if (nextA) issue_s(0, t + 1);
                }
                if (t < ntB) {
                    wait(&sh->p_full[1], t & 1);
                    tc_fence_after_sync();
                    issue_pv(1, t);
                    if (nextB) issue_s(1, t + 1);
                }
                umma_commit(&sh->v_empty[t % kVStages]);
                if (nextA || nextB) umma_commit(&sh->k_empty[(t + 1) % kKStages]);
            }
        }
    } else {
        // ---- softmax + epilogue: two threads per query row, the streams taken in turn --------
        // All eight warps work on one stream's tile at a time, each thread on 64 of its row's
        // 128 logits, so a tile spends half as long between its two MMAs as with one thread per
        // row; the other stream's MMAs fill that time.
        const int quarter = warp & 3;                      // TMEM lanes this warp may touch
        const int half = (warp - 2) >> 2;                  // columns 64*half .. 64*half+63
        const int r = quarter * 32 + lane;                 // row in the tile = TMEM lane
        const uint32_t lane_off = ((uint32_t)(quarter * 32) << 16) + half * 64;
        float m_used[2] = {0.f, 0.f}, l[2] = {0.f, 0.f};   // per stream; l covers this thread's columns
        auto do_tile = [&](auto Xc, int t, int ntX) {
            constexpr int X = decltype(Xc)::value;
            const uint32_t sp = tmem_base + X * 2 * kBlk + lane_off;   // own logits, then own P
            const uint32_t to = sp + kBlk;                             // own half of the accumulator
            wait(&sh->s_full[X], t & 1);
            tc_fence_after_sync();
            // the thread's 64 logits come into registers once and serve both passes
            uint32_t v[2][32];
            tmem_ld32(sp, v[0]);
            tmem_ld32(sp + 32, v[1]);
            tmem_wait_ld();
            if (t == ntX - 1) {
                // diagonal tile: a masked logit becomes -inf, whose exponential is exactly 0
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int x = 0; x < 32; ++x)
                        if (half * 64 + c * 32 + x > r) v[c][x] = 0xff800000u;
            }
            // Probabilities against the reference -neg_m, packed in pairs over the thread's own
            // logits columns (which are in registers by now); returns their sum.
            auto write_p = [&](float neg_m) -> float {
                // multiply-add and row sum on register pairs: one instruction per two logits
                const uint64_t sl2x2 = pack_f32x2(__float_as_uint(a.sl2), __float_as_uint(a.sl2));
                const uint64_t nmx2 = pack_f32x2(__float_as_uint(neg_m), __float_as_uint(neg_m));
                uint64_t rs2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t hi[16], lo[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        float x0, x1;
                        unpack_f32x2(fma_f32x2(pack_f32x2(v[c][2 * e], v[c][2 * e + 1]), sl2x2, nmx2), x0, x1);
                        const float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
                        rs2[e & 3] = add_f32x2(rs2[e & 3], pack_f32x2(__float_as_uint(p0), __float_as_uint(p1)));
                        hi[e] = pack2<PT>(p0, p1);
                        if (kSplitP)      // a bf16 is the upper half of an fp32
                            lo[e] = pack2<PT>(p0 - __uint_as_float(hi[e] << 16),
                                             p1 - __uint_as_float(hi[e] & 0xffff0000u));
                    }
                    tmem_st16(sp + c * 16, hi);
                    if (kSplitP) tmem_st16(sp + 32 + c * 16, lo);
                }
                float rs[8];
#pragma unroll
                for (int x = 0; x < 4; ++x) unpack_f32x2(rs2[x], rs[2 * x], rs[2 * x + 1]);
                return ((rs[0] + rs[1]) + (rs[2] + rs[3])) + ((rs[4] + rs[5]) + (rs[6] + rs[7]));
            };
            // Optimistic tile: keep the row's reference and look at the result.  The sum bounds
            // every probability, so a sum within kOptimisticLimit means that none has left
            // fp16's range; the row maximum is then never computed.  Both threads of a row (and
            // both warps of the quarter) take the same decision.
            float factor = 1.f, rowsum = 0.f;
            bool exact = (t == 0);
            if (!exact) {
                rowsum = write_p(-m_used[X]);
                const bool bad = !(rowsum <= kOptimisticLimit);          // also NaN
                sh->xch[X][half][r] = bad ? 1.f : 0.f;
                named_barrier(1 + quarter, 64);                // this quarter's two warps
                const bool pair_bad = bad || sh->xch[X][half ^ 1][r] != 0.f;
                exact = __any_sync(0xffffffffu, pair_bad);
                if (exact) named_barrier(1 + quarter, 64);     // flags read before the buffer is reused
            }
            if (exact) {
                // row maximum; the two threads of a row exchange theirs through shared memory
                float mx[2];
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    mx[c] = max3(__uint_as_float(v[c][0]), __uint_as_float(v[c][1]), __uint_as_float(v[c][2]));
#pragma unroll
                    for (int x = 3; x + 1 < 32; x += 2)
                        mx[c] = max3(mx[c], __uint_as_float(v[c][x]), __uint_as_float(v[c][x + 1]));
                    mx[c] = fmaxf(mx[c], __uint_as_float(v[c][31]));
                }
                const float own = fmaxf(mx[0], mx[1]);
                sh->xch[X][half][r] = own;
                named_barrier(1 + quarter, 64);
                const float smax = fmaxf(own, sh->xch[X][half ^ 1][r]);
                // The reference moves only on the first tile or when the row maximum exceeds it
                // by more than 2^8 (log2 domain); a row that overflowed the optimistic limit is
                // at least 2^9 above it.
                const float xmax = fmaf(smax, a.sl2, -m_used[X]);
                const bool grow = (t == 0) || (xmax > kRescaleThreshold);
                if (grow) {
                    m_used[X] += xmax;
                    factor = t == 0 ? 0.f : ex2_approx(-xmax);
                }
                if (t > 0 && __any_sync(0xffffffffu, grow)) {
                    // O_X holds tiles 0..t-1 once the previous P V product has retired
                    wait(&sh->o_done[X], (t - 1) & 1);
                    tc_fence_after_sync();
#pragma unroll 1
                    for (int c = 0; c < 2; ++c) {
                        uint32_t o[32];
                        tmem_ld32(to + c * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int x = 0; x < 32; ++x) o[x] = __float_as_uint(__uint_as_float(o[x]) * factor);
                        tmem_st32(to + c * 32, o);
                    }
                    tmem_wait_st();
                }
                rowsum = write_p(-m_used[X]);
            }
            tmem_wait_st();
            l[X] = fmaf(l[X], factor, rowsum);
            tc_fence_before_sync();
            mbar_arrive(&sh->p_full[X]);
        };
        for (int t = 0; t < nt; ++t) {
            if (t < ntA) do_tile(std::integral_constant<int, 0>{}, t, ntA);
            if (t < ntB) do_tile(std::integral_constant<int, 1>{}, t, ntB);
        }
        // ---- epilogue: each thread normalises and stores its 64 output columns ---------------
        auto finish = [&](auto Xc, int ntX, int rb) {
            constexpr int X = decltype(Xc)::value;
            if (ntX == 0) return;
            const uint32_t to = tmem_base + X * 2 * kBlk + kBlk + lane_off;
            const int i = rb * kBlk + r;
            named_barrier(1 + quarter, 64);                // the partner has read the last row maximum
            sh->xch[X][half][r] = l[X];
            named_barrier(1 + quarter, 64);
            const float lsum = l[X] + sh->xch[X][half ^ 1][r];
            const bool done = wait(&sh->o_done[X], (ntX - 1) & 1);
            tc_fence_after_sync();
            if (!done) return;
            const float inv = 1.f / lsum;
            T *orow = static_cast<T *>(a.out) + (int64_t)b * a.st_b + (int64_t)h * a.st_h +
                      (int64_t)i * a.st_t + half * 64;
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
                uint32_t o[32];
                tmem_ld32(to + c * 32, o);
                tmem_wait_ld();
                if (i < a.n && A2SF_IN_RANGE(half * 64 + c * 32 + 31, kD, kDbgAttnTc)) {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            w[e] = pack2<T>(__uint_as_float(o[q4 * 8 + 2 * e]) * inv,
                                            __uint_as_float(o[q4 * 8 + 2 * e + 1]) * inv);
                        *reinterpret_cast<uint4 *>(orow + c * 32 + q4 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            if (half == 0 && i < a.n && A2SF_IN_RANGE(u, gridDim.x / npairs, kDbgAttnTc))
                a.lse[(size_t)u * a.n + i] = (m_used[X] + log2f(lsum)) * 0.6931471805599453f;
        };
        finish(std::integral_constant<int, 0>{}, ntA, rbA);
        finish(std::integral_constant<int, 1>{}, ntB, rbB);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && sh->abort_flag) g_tc_status = A2SF_ERR_TIMEOUT;
}

template <typename T, bool PvHalf>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_pass_tc(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
             const __grid_constant__ CUtensorMap tmap_v, AttnArgs a)
{
    attn_body<T, PvHalf>(&tmap_q, &tmap_k, &tmap_v, a);
}

// bf16 storage with an fp16 copy of V in the workspace: one launch, and the flag written by the
// conversion kernel decides on the device which form of the P V product runs -- fp16 P with the
// fp16 copy when the copy is exact, two bf16 terms with the original V when it is not.
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_pass_bf16_auto(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_v_half,
                    AttnArgs a)
{
    const bool exact = *a.v_flag == 0;
    AttnArgs b = a;
    b.v_flag = nullptr;
    if (exact) attn_body<__nv_bfloat16, true>(&tmap_q, &tmap_k, &tmap_v_half, b);
    else       attn_body<__nv_bfloat16, false>(&tmap_q, &tmap_k, &tmap_v, b);
}

// fp16 copy of a bf16 V tensor, contiguous [U][n][d], for the PvHalf attention launch.  A bf16
// value converts exactly when its magnitude is within fp16's range (magnitudes below 2^-17 lose
// at most 2^-25 absolutely, which is immaterial); any value beyond 65504, infinite or NaN raises
// the flag, and the attention pass then multiplies in bf16.
__global__ void v_to_half_kernel(const __nv_bfloat16 *__restrict__ v, Strides st, int H, int n,
                                 size_t chunks, __half *__restrict__ dst, int *__restrict__ flag)
{
    constexpr int CH = kD / 8;                       // 16-byte chunks per row
    int bad = 0;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < chunks;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(idx % CH);
        const size_t row = idx / CH;
        const int t = (int)(row % n);
        const size_t u = row / n;
        const size_t b = u / H, h = u % H;
        const uint4 raw = ld_stream16(v + b * st.b + h * st.h + (size_t)t * st.t + c * 8);
        float f[8];
        Elem<__nv_bfloat16>::unpack(raw, f);
        uint4 o;
        __half2 *oh = reinterpret_cast<__half2 *>(&o);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            bad |= !(fabsf(f[2 * e]) <= 65504.f) | !(fabsf(f[2 * e + 1]) <= 65504.f);   // also NaN
            oh[e] = __floats2half2_rn(f[2 * e], f[2 * e + 1]);
        }
        if (A2SF_IN_RANGE(idx, chunks, kDbgVToHalf)) *reinterpret_cast<uint4 *>(dst + idx * 8) = o;
    }
    if (__any_sync(0xffffffffu, bad) && (threadIdx.x & 31) == 0) atomicOr(flag, 1);
}

// ---- host: tensor maps -----------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// [B][H][n][d] 16-bit tensor -> 4-D map (d, n, H, B), box 64 x 128 rows, 128-byte swizzle,
// out-of-range rows read as zero.
bool make_tile_map(CUtensorMap *map, int dtype, const void *base, const PrefillArgs &a, int heads,
                   const Strides &st)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)a.d, (cuuint64_t)a.n, (cuuint64_t)heads, (cuuint64_t)a.B};
    const cuuint64_t strides[3] = {(cuuint64_t)st.t * 2, (cuuint64_t)st.h * 2, (cuuint64_t)st.b * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)kBlk, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUtensorMapDataType dt =
        dtype == A2SF_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
    return fn(map, dt, 4, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool prefill_tc_supported(int dtype, const PrefillArgs &a)
{
    return (dtype == A2SF_BF16 || dtype == A2SF_F16) && a.d == kD &&
           (size_t)a.B * a.H * ((a.n + kBlk - 1) / kBlk) < 0x7fffffffull;
}

size_t prefill_tc_extra_bytes(int dtype, size_t units, int n, int d)
{
    if (dtype != A2SF_BF16 || d != kD) return 0;
    return 256 + ((units * (size_t)n * d * 2 + 255) / 256) * 256;      // flag word + fp16 copy of V
}

cudaError_t launch_prefill_pass1_tc(int dtype, const PrefillArgs &a, cudaStream_t s)
{
    CUtensorMap mq, mk, mv;
    const int Hkv = a.H / a.G;
    if (!make_tile_map(&mq, dtype, a.q, a, a.H, a.st) || !make_tile_map(&mk, dtype, a.k, a, Hkv, a.st_kv) ||
        !make_tile_map(&mv, dtype, a.v, a, Hkv, a.st_kv))
        return cudaErrorInvalidValue;
    static std::once_flag once[kMaxDevices];
    static cudaError_t attr_errs[kMaxDevices] = {};
    const int dev = current_device_index();
    std::call_once(once[dev], [dev] {
        const auto attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
        cudaError_t e = cudaFuncSetAttribute(attn_pass_tc<__nv_bfloat16, false>, attr, (int)kAttnSmemBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_pass_bf16_auto, attr, (int)kAttnSmemBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_pass_tc<__half, false>, attr, (int)kAttnSmemBytes);
        attr_errs[dev] = e;
    });
    if (attr_errs[dev] != cudaSuccess) return attr_errs[dev];
    AttnArgs aa;
    aa.out = a.out; aa.lse = a.lse;
    aa.st_b = a.st.b; aa.st_h = a.st.h; aa.st_t = a.st.t;
    aa.n = a.n; aa.H = a.H; aa.G = a.G;
    aa.sl2 = a.scale * kLog2e;
    aa.v_flag = nullptr;
    const int npairs = ((a.n + kBlk - 1) / kBlk + 1) / 2;
    const dim3 grid((unsigned)((size_t)a.B * a.H * npairs));
    if (dtype == A2SF_F16) {
        attn_pass_tc<__half, false><<<grid, kAttnThreads, kAttnSmemBytes, s>>>(mq, mk, mv, aa);
        count_launch();
        return cudaGetLastError();
    }
    if (!a.v_half || !a.v_flag) {       // no room for the fp16 copy: multiply in bf16
        attn_pass_tc<__nv_bfloat16, false><<<grid, kAttnThreads, kAttnSmemBytes, s>>>(mq, mk, mv, aa);
        count_launch();
        return cudaGetLastError();
    }
    // bf16: make the fp16 copy of V, then one launch that picks the form of the P V product on
    // the device from the flag the copy wrote (no host round trip)
    cudaError_t e = cudaMemsetAsync(a.v_flag, 0, sizeof(int), s);
    if (e != cudaSuccess) return e;
    const size_t chunks = (size_t)a.B * Hkv * a.n * (kD / 8);
    const unsigned cgrid = (unsigned)std::min<size_t>((chunks + 255) / 256, 148 * 16);
    v_to_half_kernel<<<cgrid, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(a.v), a.st_kv, Hkv, a.n, chunks,
                                           static_cast<__half *>(a.v_half), a.v_flag);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    const Strides contig{(int64_t)Hkv * a.n * kD, (int64_t)a.n * kD, (int64_t)kD};
    CUtensorMap mvh;
    if (!make_tile_map(&mvh, A2SF_F16, a.v_half, a, Hkv, contig)) return cudaErrorInvalidValue;
    aa.v_flag = a.v_flag;
    attn_pass_bf16_auto<<<grid, kAttnThreads, kAttnSmemBytes, s>>>(mq, mk, mv, mvh, aa);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_prefill_pass2_tc(int dtype, const PrefillArgs &a, cudaStream_t s)
{
    CUtensorMap mq, mk;
    if (!make_tile_map(&mq, dtype, a.q, a, a.H, a.st) ||
        !make_tile_map(&mk, dtype, a.k, a, a.H / a.G, a.st_kv))
        return cudaErrorInvalidValue;
    static std::once_flag once[kMaxDevices];
    static cudaError_t attr_errs[kMaxDevices] = {};
    const int dev = current_device_index();
    std::call_once(once[dev], [dev] {
        attr_errs[dev] = cudaFuncSetAttribute(score_pass_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kScoreSmemBytes);
    });
    if (attr_errs[dev] != cudaSuccess) return attr_errs[dev];
    ScoreArgs sa;
    sa.lse = a.lse; sa.scores = a.scores; sa.n = a.n; sa.H = a.H; sa.G = a.G;
    sa.sl2 = a.scale * kLog2e;
    sa.alpha = a.alpha;
    sa.alpha_vec = a.alpha_vec;
    sa.skip_zero_rows = a.skip_zero_rows;
    sa.window_rows = a.window_rows;
    const dim3 grid((unsigned)((size_t)a.B * a.H * ((a.n + kBlk - 1) / kBlk)));
    score_pass_tc<<<grid, kScoreThreads, kScoreSmemBytes, s>>>(mq, mk, sa, dtype == A2SF_BF16 ? 1 : 0);
    count_launch();
    return cudaGetLastError();
}

int *tc_status_word()
{
    static std::once_flag once[kMaxDevices];
    static int *ptr[kMaxDevices] = {};
    const int dev = current_device_index();
    std::call_once(once[dev], [dev] {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_tc_status) == cudaSuccess) ptr[dev] = static_cast<int *>(p);
    });
    return ptr[dev];
}

int read_and_clear_tc_status(cudaStream_t s)
{
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbolAsync(&v, g_tc_status, sizeof(int), 0, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return A2SF_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return A2SF_ERR_CUDA;
    if (v != 0 &&
        cudaMemcpyToSymbolAsync(g_tc_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return v;
}

}  // namespace a2sf
