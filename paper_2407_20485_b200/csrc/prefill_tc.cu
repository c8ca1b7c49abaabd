// Tensor-core prefill for 16-bit storage and d = 128 (sm_100a: TMA + tcgen05 + TMEM).
//
//   score pass (paper Eq. 5-6):  S_j = sum_{i>=j} alpha^(n-1-i) * exp(s_ij - lse_i)
//     One CTA owns 128 keys.  The logits are recomputed transposed, S^T = K_blk * Q_tile^T,
//     so that a key is a TMEM lane: the thread that owns the lane sums its key's
//     probabilities over all query rows i >= j in ascending order.  No cross-thread
//     reduction and no atomics: the result is deterministic.
//
// Warp roles per CTA (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and
// TMEM owner, warps 2-5 = epilogue (one TMEM lane quarter each).
#include <mutex>

#include "common.cuh"
#include "tc_sm100.cuh"

namespace a2sf {

// sticky device-side status: set when a bounded wait runs out
static __device__ int g_tc_status = 0;

namespace {

using namespace tc;

constexpr int kBlk = 128;                   // keys per CTA = TMEM lanes; query rows per tile
constexpr int kD = 128;
constexpr int kHalfBytes = kBlk * 64 * 2;   // one 64-column swizzled half of a tile: 16 KB
constexpr int kTileBytes = 2 * kHalfBytes;  // 32 KB
constexpr int kScoreStages = 2;
constexpr int kScoreThreads = 192;

struct ScoreArgs {
    const float *lse;     // [U][n]
    float *scores;        // [U][n]
    int n, H;
    float sl2;            // scale * log2(e)
    float neg_log2_alpha; // -log2(alpha); +inf for alpha = 0
};

struct ScoreShared {
    uint64_t k_full, q_full[kScoreStages], q_empty[kScoreStages], acc_full[2], acc_empty[2], c_full[2];
    uint32_t tmem_base;
    int abort_flag;
    float cbuf[2][kBlk];
};

constexpr size_t kScoreSmemBytes = 1024 /*alignment slack*/ + kTileBytes * (1 + kScoreStages) +
                                   sizeof(ScoreShared);

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 8 K-steps of 16 elements over a [128 x 128] K-major operand pair stored as two
// 64-column swizzled halves.
__device__ __forceinline__ void issue_qk_mma(uint32_t d_tmem, uint32_t a_addr, uint32_t b_addr,
                                             uint32_t idesc)
{
#pragma unroll
    for (int k = 0; k < kD / 16; ++k) {
        const uint32_t off = (k >> 2) * kHalfBytes + (k & 3) * 32;
        umma_ss(d_tmem, make_sdesc_sw128(a_addr + off, 16, 1024),
                make_sdesc_sw128(b_addr + off, 16, 1024), idesc, k > 0);
    }
}

__global__ void __launch_bounds__(kScoreThreads)
score_pass_tc(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
              ScoreArgs a, int ab_fmt)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                ~uintptr_t(1023));
    uint8_t *Ks = smem;
    uint8_t *Qs = smem + kTileBytes;
    ScoreShared *sh = reinterpret_cast<ScoreShared *>(smem + kTileBytes * (1 + kScoreStages));

    const int u = blockIdx.x, kb = blockIdx.y;
    const int b = u / a.H, h = u % a.H;
    const int ntile_total = (a.n + kBlk - 1) / kBlk;
    const int ntiles = ntile_total - kb;               // query-row tiles kb .. last
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &sh->abort_flag;

    if (threadIdx.x == 0) {
        mbar_init(&sh->k_full, 1);
        for (int s = 0; s < kScoreStages; ++s) { mbar_init(&sh->q_full[s], 1); mbar_init(&sh->q_empty[s], 1); }
        for (int x = 0; x < 2; ++x) {
            mbar_init(&sh->acc_full[x], 1);
            mbar_init(&sh->acc_empty[x], kBlk);
            mbar_init(&sh->c_full[x], kBlk);
        }
        sh->abort_flag = 0;
        fence_mbar_init();
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
        // ---- TMA producer ---------------------------------------------------------
        if (lane == 0) {
            prefetch_tmap(&tmap_q);
            prefetch_tmap(&tmap_k);
            mbar_arrive_expect_tx(&sh->k_full, kTileBytes);
            tma_load_4d(Ks, &tmap_k, &sh->k_full, 0, kb * kBlk, h, b);
            tma_load_4d(Ks + kHalfBytes, &tmap_k, &sh->k_full, 64, kb * kBlk, h, b);
            int issued = 0;
            for (int it = 0; it < ntiles; ++it) {
                const int s = it % kScoreStages;
                const uint32_t ph = (it / kScoreStages) & 1;
                if (!mbar_wait(&sh->q_empty[s], ph ^ 1, abort_flag)) break;
                mbar_arrive_expect_tx(&sh->q_full[s], kTileBytes);
                uint8_t *dst = Qs + s * kTileBytes;
                tma_load_4d(dst, &tmap_q, &sh->q_full[s], 0, (kb + it) * kBlk, h, b);
                tma_load_4d(dst + kHalfBytes, &tmap_q, &sh->q_full[s], 64, (kb + it) * kBlk, h, b);
                issued = it + 1;
            }
            if (*abort_flag) {
                // give copies still in flight a bounded chance to land before the CTA exits
                int dummy = 0;
                for (int it = max(0, issued - kScoreStages); it < issued; ++it)
                    mbar_wait(&sh->q_full[it % kScoreStages], (it / kScoreStages) & 1, &dummy);
                mbar_wait(&sh->k_full, 0, &dummy);
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer -------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = make_idesc(ab_fmt, kBlk, kBlk, 0, 0);
            const uint32_t k_addr = smem_u32(Ks);
            bool ok = mbar_wait(&sh->k_full, 0, abort_flag);
            for (int it = 0; ok && it < ntiles; ++it) {
                const int s = it % kScoreStages;
                const uint32_t ph = (it / kScoreStages) & 1;
                const int acc = it & 1;
                const uint32_t aph = (it >> 1) & 1;
                if (!mbar_wait(&sh->q_full[s], ph, abort_flag)) break;
                if (!mbar_wait(&sh->acc_empty[acc], aph ^ 1, abort_flag)) break;
                tc_fence_after_sync();
                issue_qk_mma(tmem_base + acc * kBlk, k_addr, smem_u32(Qs + s * kTileBytes), idesc);
                umma_commit(&sh->q_empty[s]);       // the stage is free once these MMAs retire
                umma_commit(&sh->acc_full[acc]);
            }
        }
    } else {
        // ---- epilogue: one thread per key --------------------------------------------
        const int quarter = warp & 3;               // TMEM lanes this warp may touch
        const int key_lane = quarter * 32 + lane;
        const int j = kb * kBlk + key_lane;
        const int et = threadIdx.x - 64;            // 0..127
        const float *lse = a.lse + (size_t)u * a.n;
        float sum = 0.f;
        for (int it = 0; it < ntiles; ++it) {
            const int acc = it & 1;
            const uint32_t aph = (it >> 1) & 1;
            const int i0 = (kb + it) * kBlk;
            {   // row constants c_i = lse_i*log2e + (n-1-i)*(-log2 alpha); rows past n give +inf
                const int i = i0 + et;
                float cv = INFINITY;
                if (i < a.n) {
                    const int age = a.n - 1 - i;
                    cv = fmaf(lse[i], kLog2e, age == 0 ? 0.f : (float)age * a.neg_log2_alpha);
                }
                sh->cbuf[it & 1][et] = cv;
            }
            mbar_arrive(&sh->c_full[acc]);       // release: the row constants are published
            if (!mbar_wait(&sh->c_full[acc], aph, abort_flag)) break;
            if (!mbar_wait(&sh->acc_full[acc], aph, abort_flag)) break;
            tc_fence_after_sync();
            const float *cb = sh->cbuf[it & 1];
            const bool diag = (it == 0);
#pragma unroll 1
            for (int c = 0; c < kBlk / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem_base + acc * kBlk + c * 32 + ((uint32_t)(quarter * 32) << 16), r);
                tmem_wait_ld();
#pragma unroll
                for (int x = 0; x < 32; ++x) {
                    float pw = ex2_approx(fmaf(__uint_as_float(r[x]), a.sl2, -cb[c * 32 + x]));
                    if (diag) pw = (i0 + c * 32 + x >= j) ? pw : 0.f;    // causal: rows i >= j
                    sum += pw;
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&sh->acc_empty[acc]);
        }
        if (j < a.n && !*abort_flag) a.scores[(size_t)u * a.n + j] = sum;
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 256);
    }
    if (threadIdx.x == 0 && sh->abort_flag) g_tc_status = A2SF_ERR_TIMEOUT;
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
bool make_tile_map(CUtensorMap *map, int dtype, const void *base, const PrefillArgs &a)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)a.d, (cuuint64_t)a.n, (cuuint64_t)a.H, (cuuint64_t)a.B};
    const cuuint64_t strides[3] = {(cuuint64_t)a.st.t * 2, (cuuint64_t)a.st.h * 2, (cuuint64_t)a.st.b * 2};
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
           (a.n + kBlk - 1) / kBlk <= 65535;
}

cudaError_t launch_prefill_pass2_tc(int dtype, const PrefillArgs &a, cudaStream_t s)
{
    CUtensorMap mq, mk;
    if (!make_tile_map(&mq, dtype, a.q, a) || !make_tile_map(&mk, dtype, a.k, a))
        return cudaErrorInvalidValue;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(score_pass_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)kScoreSmemBytes);
    });
    if (attr_err != cudaSuccess) return attr_err;
    ScoreArgs sa;
    sa.lse = a.lse; sa.scores = a.scores; sa.n = a.n; sa.H = a.H;
    sa.sl2 = a.scale * kLog2e;
    sa.neg_log2_alpha = a.alpha > 0.f ? -log2f(a.alpha) : INFINITY;
    dim3 grid(a.B * a.H, (a.n + kBlk - 1) / kBlk);
    score_pass_tc<<<grid, kScoreThreads, kScoreSmemBytes, s>>>(mq, mk, sa, dtype == A2SF_BF16 ? 1 : 0);
    count_launch();
    return cudaGetLastError();
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
