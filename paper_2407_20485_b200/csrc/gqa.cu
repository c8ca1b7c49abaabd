// Grouped query heads: G query heads share one K/V head and therefore one pruned cache.
// The paper scores tokens per head (Sec. 2.2) and leaves head grouping open (Limitation
// section); here a cached token's score gains, per step, the SUM of the group's attention
// probabilities, and one eviction serves the whole group.
//
//   group_sum_kernel       : prefill scores of the G query heads -> one score row per K/V head.
//   decode_step_group_kernel: the generation step for one K/V unit and its G queries.  K and V
//                            rows are read once; each lane keeps its 16-byte slice of all G
//                            queries in registers, so the extra heads cost arithmetic, not
//                            memory traffic.
#include <algorithm>

#include "common.cuh"

namespace a2sf {

A2SF_DEBUG_TRANSLATION_UNIT(gqa)
namespace {

constexpr int kGroupThreads = 256;
constexpr int kMaxGroup = 8;

__global__ void group_sum_kernel(const float *__restrict__ per_head, float *__restrict__ out, int G, int n,
                                 size_t total)
{
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const size_t u = idx / n, j = idx % n;
        float s = 0.f;
        for (int g = 0; g < G; ++g) s += per_head[(u * G + g) * (size_t)n + j];   // fixed order
        if (A2SF_IN_RANGE(idx, total, kDbgGroupSum)) out[idx] = s;
    }
}

// floats of shared memory per kernel instance, shared with the host-side size check
__host__ __device__ inline size_t group_wstride(int M) { return ((size_t)M + 1 + 3) & ~(size_t)3; }

__device__ __forceinline__ void cp_async4(void *smem_dst, const void *gmem_src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)),
                 "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// GMAX dot products, each spread over the LPR lanes of a row, are summed with a halving
// butterfly: at every step a lane passes on the half of its values that its partner keeps, so
// the whole reduction takes GMAX - 1 + log2(LPR / GMAX) shuffles instead of GMAX * log2(LPR).
// Afterwards every lane holds the total of query  sub / (LPR / GMAX).
template <int GMAX, int LPR>
__device__ __forceinline__ float group_reduce(float (&d)[GMAX], int sub)
{
    static_assert(GMAX <= LPR, "one lane per query at least");
    int nv = GMAX;
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) {
        if (nv > 1) {
            nv >>= 1;
            const bool upper = (sub & o) != 0;
#pragma unroll
            for (int i = 0; i < GMAX / 2; ++i) {
                if (i < nv) {
                    const float send = upper ? d[i] : d[i + nv];
                    const float keep = upper ? d[i + nv] : d[i];
                    d[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                }
            }
        } else {
            d[0] += __shfl_xor_sync(0xffffffffu, d[0], o);
        }
    }
    return d[0];
}

// GMAX: compile-time bound of the group size (2, 4 or 8): the per-lane query slices and
// accumulator rows are sized by it.  One CTA per K/V unit.  The kernel is a chain of dependent
// phases around little data, so every global word it needs is requested as early as it can be:
// the unit's scores and positions go to shared memory asynchronously at the start, K and V rows
// are loaded one batch of kUnroll row groups ahead of the arithmetic, and the first V batch is
// requested before the softmax.
template <typename T, int D, int GMAX>
__global__ void __launch_bounds__(kGroupThreads, 2)
decode_step_group_kernel(CacheView c, int G, float alpha, const T *__restrict__ q,
                         const T *__restrict__ k_new, const T *__restrict__ v_new, T *__restrict__ out,
                         int32_t *__restrict__ evicted)
{
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;              // lanes per row
    constexpr int RPW = 32 / LPR;             // rows per warp-wide load
    constexpr int NW = kGroupThreads / 32;
    constexpr int LPG = LPR / GMAX;           // lanes that end up with the same query's logit
    const int M = c.M;
    const int wstride = (int)group_wstride(M);

    extern __shared__ __align__(16) float gsm[];
    float *w = gsm;                                   // [G][wstride] logits, then probabilities
    float *part = w + (size_t)G * wstride;            // [NW][G][D] partial outputs
    float *s_old = part + (size_t)NW * G * D;         // [wstride] the unit's scores before the step
    int32_t *s_pos = reinterpret_cast<int32_t *>(s_old + wstride);   // [wstride] positions
    __shared__ float red_m[NW][GMAX], red_l[NW][GMAX];
    __shared__ unsigned long long red_key[NW];
    __shared__ int red_slot[NW];
    __shared__ int s_target;

    const int u = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, rsel = lane / LPR;
    const int cnt = min(c.count[u], M);
    const int p = c.len[u];
    T *Ku = reinterpret_cast<T *>(c.K) + (size_t)u * M * D;
    T *Vu = reinterpret_cast<T *>(c.V) + (size_t)u * M * D;
    float *Su = c.S + (size_t)u * M;
    int32_t *posu = c.pos + (size_t)u * M;
    const T *qu = q + (size_t)u * G * D;              // [G][D]
    const T *knu = k_new + (size_t)u * D, *vnu = v_new + (size_t)u * D;

    // scores and positions: thread tid stages, and later reads, slots tid, tid + 256, ...
    for (int s = tid; s < cnt; s += kGroupThreads) {
        cp_async4(s_old + s, Su + s);
        cp_async4(s_pos + s, posu + s);
    }

    // this lane's slice of every query (zero for the unused heads of the bound)
    float qf[GMAX][VEC];
#pragma unroll
    for (int g = 0; g < GMAX; ++g) {
        uint4 raw = make_uint4(0u, 0u, 0u, 0u);
        if (g < G) raw = *reinterpret_cast<const uint4 *>(qu + (size_t)g * D + sub * VEC);
        Elem<T>::unpack(raw, qf[g]);
    }

    constexpr int kUnroll = GMAX <= 4 ? 8 : 4;
    constexpr int kBatch = NW * RPW * kUnroll;        // rows per batch of the whole CTA
    // rows 0..cnt-1 are cached, row cnt is the new token's
    auto load_rows = [&](uint4(&raw)[kUnroll], int s0, const T *base, const T *fresh) {
#pragma unroll
        for (int x = 0; x < kUnroll; ++x) {
            const int s = s0 + x * NW * RPW + rsel;
            raw[x] = make_uint4(0u, 0u, 0u, 0u);
            if (s <= cnt && A2SF_IN_RANGE(s, c.M + 1, kDbgGroupSimt))
                raw[x] = *reinterpret_cast<const uint4 *>((s < cnt ? base + (size_t)s * D : fresh) + sub * VEC);
        }
    };

    // ---- (i) logits of the cached keys and of the new key, for every query of the group -----
    uint4 cur[kUnroll], nxt[kUnroll];
    load_rows(cur, warp * RPW, Ku, knu);
    for (int s0 = warp * RPW; s0 <= cnt; s0 += kBatch) {
        load_rows(nxt, s0 + kBatch, Ku, knu);         // nothing is loaded past row cnt
#pragma unroll
        for (int x = 0; x < kUnroll; ++x) {
            const int s = s0 + x * NW * RPW + rsel;
            float kf[VEC];
            Elem<T>::unpack(cur[x], kf);
            float dot[GMAX];
#pragma unroll
            for (int g = 0; g < GMAX; ++g) {
                dot[g] = 0.f;
#pragma unroll
                for (int e = 0; e < VEC; ++e) dot[g] = fmaf(qf[g][e], kf[e], dot[g]);
            }
            const float tot = group_reduce<GMAX, LPR>(dot, sub);
            const int g = sub / LPG;
            if (sub % LPG == 0 && g < G && s <= cnt && A2SF_IN_RANGE(s, wstride, kDbgGroupSimt)) w[g * wstride + s] = tot * c.scale;
        }
#pragma unroll
        for (int x = 0; x < kUnroll; ++x) cur[x] = nxt[x];
    }
    // the first values are on their way while the softmax runs
    load_rows(cur, warp * RPW, Vu, vnu);
    __syncthreads();

    // ---- (ii) one softmax per query, all threads on every query ----------------------------------
    float mg[GMAX], inv[GMAX];
#pragma unroll
    for (int g = 0; g < GMAX; ++g) {
        float m = -INFINITY;
        if (g < G)
            for (int s = tid; s <= cnt; s += kGroupThreads) m = fmaxf(m, w[g * wstride + s]);
        m = warp_max(m);
        if (lane == 0) red_m[warp][g] = m;
    }
    __syncthreads();
#pragma unroll
    for (int g = 0; g < GMAX; ++g) {
        float m = red_m[0][g];
#pragma unroll
        for (int x = 1; x < NW; ++x) m = fmaxf(m, red_m[x][g]);
        mg[g] = m;
        float l = 0.f;
        if (g < G)
            for (int s = tid; s <= cnt; s += kGroupThreads) {
                const float e = expf(w[g * wstride + s] - m);
                w[g * wstride + s] = e;
                l += e;
            }
        l = warp_sum(l);
        if (lane == 0) red_l[warp][g] = l;
    }
    __syncthreads();
#pragma unroll
    for (int g = 0; g < GMAX; ++g) {
        float l = red_l[0][g];
#pragma unroll
        for (int x = 1; x < NW; ++x) l += red_l[x][g];                  // fixed order
        inv[g] = 1.f / l;
        if (g < G)
            for (int s = tid; s <= cnt; s += kGroupThreads) w[g * wstride + s] *= inv[g];   // probabilities
    }
    (void)mg;
    __syncthreads();

    // ---- (iii) out_g = sum_slot a_g[slot] V[slot] + a_g[self] v_new -----------------------------
    float acc[GMAX][VEC];
#pragma unroll
    for (int g = 0; g < GMAX; ++g)
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[g][e] = 0.f;
    for (int s0 = warp * RPW; s0 <= cnt; s0 += kBatch) {
        load_rows(nxt, s0 + kBatch, Vu, vnu);
#pragma unroll
        for (int x = 0; x < kUnroll; ++x) {
            const int s = s0 + x * NW * RPW + rsel;
            if (s <= cnt) {
                float vf[VEC];
                Elem<T>::unpack(cur[x], vf);
#pragma unroll
                for (int g = 0; g < GMAX; ++g) {
                    if (g < G) {
                        const float a = w[g * wstride + s];
#pragma unroll
                        for (int e = 0; e < VEC; ++e) acc[g][e] = fmaf(a, vf[e], acc[g][e]);
                    }
                }
            }
        }
#pragma unroll
        for (int x = 0; x < kUnroll; ++x) cur[x] = nxt[x];
    }
#pragma unroll
    for (int g = 0; g < GMAX; ++g) {
        if (g < G) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                float v = acc[g][e];
#pragma unroll
                for (int o = LPR; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);   // over rsel
                if (rsel == 0) part[((size_t)warp * G + g) * D + sub * VEC + e] = v;
            }
        }
    }
    cp_async_wait_all();                       // this thread's staged scores and positions
    __syncthreads();
    for (int x = tid; x < G * D; x += kGroupThreads) {
        float o = 0.f;
#pragma unroll
        for (int wv = 0; wv < NW; ++wv) o += part[(size_t)wv * G * D + x];
        out[(size_t)u * G * D + x] = Elem<T>::from_float(o);
    }

    // ---- (iv) S <- alpha*S + sum_g a_g ; candidates for eviction ---------------------------------
    const bool full = cnt >= M;
    const int newest_evictable = p - c.R;
    unsigned long long best = ~0ull;
    int best_slot = -1;
    for (int s = tid; s < cnt; s += kGroupThreads) {
        float gain = 0.f;
        for (int g = 0; g < G; ++g) gain += w[g * wstride + s];
        const float sn = fmaf(alpha, s_old[s], gain);
        if (A2SF_IN_RANGE(s, c.M, kDbgGroupSimt)) Su[s] = sn;
        const int ps = s_pos[s];
        if (full && ps <= newest_evictable) {
            const unsigned long long key = ((unsigned long long)__float_as_uint(sn) << 32) | (unsigned)ps;
            if (key < best) { best = key; best_slot = s; }
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int os = __shfl_xor_sync(0xffffffffu, best_slot, o);
        if (ob < best) { best = ob; best_slot = os; }
    }
    if (lane == 0) { red_key[warp] = best; red_slot[warp] = best_slot; }
    __syncthreads();

    // ---- (v) eviction and in-place insert, (vi) length ------------------------------------------
    float s_new = 0.f;
    for (int g = 0; g < G; ++g) s_new += w[g * wstride + cnt];
    if (tid == 0) {
        int target = full ? -2 : cnt;
        if (full) {
            unsigned long long gb = red_key[0];
            int gs = red_slot[0];
            for (int x = 1; x < NW; ++x)
                if (red_key[x] < gb) { gb = red_key[x]; gs = red_slot[x]; }
            const unsigned long long self_key = ((unsigned long long)__float_as_uint(s_new) << 32) | (unsigned)p;
            if (gs >= 0 && (c.R > 0 || gb < self_key)) target = gs;
        }
        s_target = target;
    }
    __syncthreads();
    const int target = s_target;
    if (target >= 0) {
        if (!A2SF_IN_RANGE(target, c.M, kDbgGroupSimt)) {
        } else if (tid < LPR)
            *reinterpret_cast<uint4 *>(Ku + (size_t)target * D + tid * VEC) =
                *reinterpret_cast<const uint4 *>(knu + tid * VEC);
        else if (tid < 2 * LPR)
            *reinterpret_cast<uint4 *>(Vu + (size_t)target * D + (tid - LPR) * VEC) =
                *reinterpret_cast<const uint4 *>(vnu + (tid - LPR) * VEC);
    }
    if (tid == 0 && A2SF_IN_RANGE(u, c.U, kDbgGroupMma)) {
        if (target >= 0 && A2SF_IN_RANGE(target, c.M, kDbgGroupMma)) {
            Su[target] = s_new;
            posu[target] = p;
        }
        if (!full) c.count[u] = cnt + 1;
        c.len[u] = p + 1;
        evicted[u] = full ? target : -1;
    }
}

// ---- 16-bit storage: the group's products on the tensor cores -----------------------------------
// With G queries per K/V row the step is a skinny matrix product, [slots x d] . [d x G]: the
// CUDA-core form above spends ~18 instructions per cached element for G = 8 and is bound by them,
// not by memory.  Here a warp takes 16 slots at a time through mma.sync m16n8k16 (fp32
// accumulation), the 8 columns being the query heads (zero beyond G), with operands taken
// straight from 16-byte global loads:
//   logits  S[16 slots x 8] = K[16 x d] . Q^T: a sum over d does not depend on the order of its
//           terms, so lane (r, c) = (lane / 4, lane % 4) feeds the elements 32j + 8c .. + 7 of
//           its rows r and r + 8 (and of query r) as the instruction's k-columns 2c, 2c+1, 2c+8,
//           2c+9 of chunks 2j and 2j + 1: no shuffle, no shared-memory staging.
//   output  O^T[d x 8] = V^T[d x 16 slots] . P^T: lane (r, c) loads elements 16r .. 16r + 15
//           (d = 128) of slots 2c, 2c+1, 2c+8, 2c+9 and interleaves two rows with one byte
//           permute per register so that a slot pair sits in one register as the instruction
//           wants; row r / r + 8 of m-tile t is element E*r + t / E*r + E/2 + t (E = d / 8).
// Probabilities stay fp32 in shared memory for the scores; for the product they are rounded to
// fp16 (fp16 storage) or split into two bf16 terms hi + lo (bf16 storage, two products), the
// same precision argument as in the prefill's attention pass.
template <typename T> struct GroupMma;
template <> struct GroupMma<__half> {
    static constexpr int kTerms = 1;
    __device__ static void mma(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
    {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                     "{%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    // term 0: the pair rounded to fp16 (there is no second term)
    __device__ static uint32_t pack(float lo, float hi, int)
    {
        const __half2 h = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<const uint32_t *>(&h);
    }
};
template <> struct GroupMma<__nv_bfloat16> {
    static constexpr int kTerms = 2;
    __device__ static void mma(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
    {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                     "{%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    // term 0: the pair rounded to bf16; term 1: what that rounding left over, again in bf16
    __device__ static uint32_t pack(float lo, float hi, int term)
    {
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
        if (term == 1) h = __floats2bfloat162_rn(lo - __low2float(h), hi - __high2float(h));
        return *reinterpret_cast<const uint32_t *>(&h);
    }
};

constexpr int kMmaCols = 8;      // query-head columns of the instruction

__host__ __device__ inline size_t group_mma_smem_bytes(int M, int d)
{
    // probabilities [wstride][8], partial outputs [warps][8][d], staged scores and positions
    return ((size_t)(kMmaCols + 2) * group_wstride(M) + (size_t)(kGroupThreads / 32) * kMmaCols * d) * sizeof(float);
}

template <typename T, int D>
__global__ void __launch_bounds__(kGroupThreads, 2)
decode_step_group_mma_kernel(CacheView c, int G, float alpha, const T *__restrict__ q,
                             const T *__restrict__ k_new, const T *__restrict__ v_new, T *__restrict__ out,
                             int32_t *__restrict__ evicted)
{
    static_assert(sizeof(T) == 2 && (D == 64 || D == 128), "16-bit storage");
    constexpr int NW = kGroupThreads / 32;
    constexpr int KL = D / 32;                // 16-byte loads per K row and lane
    constexpr int E = D / 8;                  // V elements per slot and lane
    constexpr int VL = E / 8;                 // 16-byte loads per V row and lane
    constexpr int MT = D / 16;                // m-tiles of the output product
    using Mma = GroupMma<T>;
    const int M = c.M;
    const int wstride = (int)group_wstride(M);

    extern __shared__ __align__(16) float gsm[];
    float *w = gsm;                                   // [wstride][8] logits, then probabilities
    float *part = w + (size_t)kMmaCols * wstride;     // [NW][8][D] partial outputs
    float *s_old = part + (size_t)NW * kMmaCols * D;  // [wstride] the unit's scores before the step
    int32_t *s_pos = reinterpret_cast<int32_t *>(s_old + wstride);
    __shared__ float red_m[NW][kMmaCols], red_l[NW][kMmaCols], s_inv[kMmaCols];
    __shared__ unsigned long long red_key[NW];
    __shared__ int red_slot[NW];
    __shared__ int s_target;

    const int u = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r = lane >> 2, cq = lane & 3;
    const int cnt = min(c.count[u], M);
    const int p = c.len[u];
    T *Ku = reinterpret_cast<T *>(c.K) + (size_t)u * M * D;
    T *Vu = reinterpret_cast<T *>(c.V) + (size_t)u * M * D;
    float *Su = c.S + (size_t)u * M;
    int32_t *posu = c.pos + (size_t)u * M;
    const T *qu = q + (size_t)u * G * D;              // [G][D]
    const T *knu = k_new + (size_t)u * D, *vnu = v_new + (size_t)u * D;

    for (int s = tid; s < cnt; s += kGroupThreads) {
        cp_async4(s_old + s, Su + s);
        cp_async4(s_pos + s, posu + s);
    }

    // query r (zero beyond the group), the elements this lane pairs with its K slices
    uint4 qreg[KL];
#pragma unroll
    for (int j = 0; j < KL; ++j) {
        qreg[j] = make_uint4(0u, 0u, 0u, 0u);
        if (r < G) qreg[j] = *reinterpret_cast<const uint4 *>(qu + (size_t)r * D + 32 * j + 8 * cq);
    }

    const int ntile = (cnt + 1 + 15) >> 4;            // rows 0..cnt-1 cached, row cnt the new token
    auto row_ptr = [&](int s, const T *base, const T *fresh) { return s < cnt ? base + (size_t)s * D : fresh; };

    // ---- (i) logits ------------------------------------------------------------------------------
    auto load_k = [&](uint4(&buf)[2][KL], int tile) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int s = tile * 16 + r + 8 * h;
#pragma unroll
            for (int j = 0; j < KL; ++j) {
                buf[h][j] = make_uint4(0u, 0u, 0u, 0u);
                if (tile < ntile && s <= cnt && A2SF_IN_RANGE(s, c.M + 1, kDbgGroupMma))
                    buf[h][j] = *reinterpret_cast<const uint4 *>(row_ptr(s, Ku, knu) + 32 * j + 8 * cq);
            }
        }
    };
    {
        uint4 cur[2][KL], nxt[2][KL];
        load_k(cur, warp);
        float mx0 = -INFINITY, mx1 = -INFINITY;      // running maxima of query columns 2c, 2c + 1
        for (int tile = warp; tile < ntile; tile += NW) {
            load_k(nxt, tile + NW);
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int j = 0; j < KL; ++j) {
                const uint32_t a_even[4] = {cur[0][j].x, cur[1][j].x, cur[0][j].y, cur[1][j].y};
                const uint32_t a_odd[4] = {cur[0][j].z, cur[1][j].z, cur[0][j].w, cur[1][j].w};
                Mma::mma(acc, a_even, qreg[j].x, qreg[j].y);
                Mma::mma(acc, a_odd, qreg[j].z, qreg[j].w);
            }
            // acc: rows r, r + 8 of the tile, query columns 2c and 2c + 1
            const int s0 = tile * 16 + r;
            if (s0 <= cnt) {
                const float2 lg = make_float2(acc[0] * c.scale, acc[1] * c.scale);
                *reinterpret_cast<float2 *>(w + (size_t)s0 * kMmaCols + 2 * cq) = lg;
                mx0 = fmaxf(mx0, lg.x);
                mx1 = fmaxf(mx1, lg.y);
            }
            if (s0 + 8 <= cnt) {
                const float2 lg = make_float2(acc[2] * c.scale, acc[3] * c.scale);
                *reinterpret_cast<float2 *>(w + (size_t)(s0 + 8) * kMmaCols + 2 * cq) = lg;
                mx0 = fmaxf(mx0, lg.x);
                mx1 = fmaxf(mx1, lg.y);
            }
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int j = 0; j < KL; ++j) cur[h][j] = nxt[h][j];
        }
        // the warp's column maxima (over the lanes' rows r): no separate pass over the logits
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
        }
        if (lane < 4) {
            red_m[warp][2 * lane] = mx0;
            red_m[warp][2 * lane + 1] = mx1;
        }
    }

    // ---- (iii, loads) the first tile of values is on its way while the softmax runs ---------------
    auto load_v = [&](uint4(&buf)[4][VL], int tile) {
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const int s = tile * 16 + 2 * cq + (x & 1) + 8 * (x >> 1);
#pragma unroll
            for (int i = 0; i < VL; ++i) {
                buf[x][i] = make_uint4(0u, 0u, 0u, 0u);
                if (tile < ntile && s <= cnt && A2SF_IN_RANGE(s, c.M + 1, kDbgGroupMma))
                    buf[x][i] = *reinterpret_cast<const uint4 *>(row_ptr(s, Vu, vnu) + E * r + 8 * i);
            }
        }
    };
    uint4 vcur[4][VL], vnxt[4][VL];
    load_v(vcur, warp);
    __syncthreads();

    // ---- (ii) softmax per query column: thread = (row % 32, column) ------------------------------
    // The exponentials stay unnormalised: the output rows and the scores take the factor 1 / sum
    // at the end, so the logits are passed over once, between two barriers.
    {
        const int g = tid & 7;
        const int nrow = cnt + 1;
        float m = red_m[0][g];
#pragma unroll
        for (int x = 1; x < NW; ++x) m = fmaxf(m, red_m[x][g]);
        float l = 0.f;
#pragma unroll 4
        for (int s = tid >> 3; s < nrow; s += kGroupThreads / 8) {
            const float e = g < G ? expf(w[s * kMmaCols + g] - m) : 0.f;   // unused columns 0
            if (A2SF_IN_RANGE(s, c.M + 1, kDbgGroupMma)) w[s * kMmaCols + g] = e;
            l += e;
        }
        l += __shfl_xor_sync(0xffffffffu, l, 8);
        l += __shfl_xor_sync(0xffffffffu, l, 16);
        if (lane < 8) red_l[warp][lane] = l;
    }
    __syncthreads();
    if (tid < kMmaCols) {
        float l = red_l[0][tid];
#pragma unroll
        for (int x = 1; x < NW; ++x) l += red_l[x][tid];                // fixed order
        s_inv[tid] = tid < G ? 1.f / l : 0.f;     // read after the barrier that follows the products
    }

    // ---- (iii) out^T[d x 8] = sum over slots V^T . P^T ----------------------------------------------
    float oacc[MT][4];
#pragma unroll
    for (int t = 0; t < MT; ++t)
#pragma unroll
        for (int e = 0; e < 4; ++e) oacc[t][e] = 0.f;
    for (int tile = warp; tile < ntile; tile += NW) {
        load_v(vnxt, tile + NW);
        // P^T fragment: slots 2c, 2c+1 (b0) and 2c+8, 2c+9 (b1) of the tile, query r
        float pf[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const int s = tile * 16 + 2 * cq + (x & 1) + 8 * (x >> 1);
            pf[x] = s <= cnt ? w[(size_t)s * kMmaCols + r] : 0.f;
        }
#pragma unroll
        for (int term = 0; term < Mma::kTerms; ++term) {
            const uint32_t b0 = Mma::pack(pf[0], pf[1], term), b1 = Mma::pack(pf[2], pf[3], term);
#pragma unroll
            for (int t = 0; t < MT; ++t) {
                // element E*r + t (rows r) and E*r + E/2 + t (rows r + 8) of the four slots
                const uint32_t *v0 = reinterpret_cast<const uint32_t *>(vcur[0]);
                const uint32_t *v1 = reinterpret_cast<const uint32_t *>(vcur[1]);
                const uint32_t *v2 = reinterpret_cast<const uint32_t *>(vcur[2]);
                const uint32_t *v3 = reinterpret_cast<const uint32_t *>(vcur[3]);
                const int lo = t >> 1, hi = (E / 2 + t) >> 1;
                const uint32_t sel = (t & 1) ? 0x7632u : 0x5410u;
                const uint32_t a[4] = {__byte_perm(v0[lo], v1[lo], sel), __byte_perm(v0[hi], v1[hi], sel),
                                       __byte_perm(v2[lo], v3[lo], sel), __byte_perm(v2[hi], v3[hi], sel)};
                Mma::mma(oacc[t], a, b0, b1);
            }
        }
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int i = 0; i < VL; ++i) vcur[x][i] = vnxt[x][i];
    }
    // oacc[t]: (element E*r + t, queries 2c, 2c+1), (element E*r + E/2 + t, queries 2c, 2c+1)
    // Within its E elements of a row a lane's values are stored rotated by rot(r, c), so that the 32
    // lanes of one store hit 32 banks (unrotated, they would share two); the reader undoes it.
    {
        const int rot = 4 * (r / (32 / E)) + cq;
        float *pw = part + (size_t)warp * kMmaCols * D;
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            const int lo = E * r + ((t + rot) % E), hi = E * r + ((E / 2 + t + rot) % E);
            pw[(2 * cq) * D + lo] = oacc[t][0];
            pw[(2 * cq + 1) * D + lo] = oacc[t][1];
            pw[(2 * cq) * D + hi] = oacc[t][2];
            pw[(2 * cq + 1) * D + hi] = oacc[t][3];
        }
    }
    cp_async_wait_all();                       // this thread's staged scores and positions
    __syncthreads();
    for (int x = tid; x < G * D; x += kGroupThreads) {
        const int g = x / D, d = x % D, row = d / E;
        const int col = g * D + E * row + ((d % E + 4 * (row / (32 / E)) + (g >> 1)) % E);
        float o = 0.f;
#pragma unroll
        for (int wv = 0; wv < NW; ++wv) o += part[(size_t)wv * kMmaCols * D + col];
        out[(size_t)u * G * D + x] = Elem<T>::from_float(o * s_inv[g]);
    }

    // ---- (iv) S <- alpha*S + sum_g a_g ; candidates for eviction ---------------------------------
    const bool full = cnt >= M;
    const int newest_evictable = p - c.R;
    unsigned long long best = ~0ull;
    int best_slot = -1;
    for (int s = tid; s < cnt; s += kGroupThreads) {
        float gain = 0.f;
        for (int g = 0; g < G; ++g) gain += w[(size_t)s * kMmaCols + g] * s_inv[g];
        const float sn = fmaf(alpha, s_old[s], gain);
        if (A2SF_IN_RANGE(s, c.M, kDbgGroupSimt)) Su[s] = sn;
        const int ps = s_pos[s];
        if (full && ps <= newest_evictable) {
            const unsigned long long key = ((unsigned long long)__float_as_uint(sn) << 32) | (unsigned)ps;
            if (key < best) { best = key; best_slot = s; }
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int os = __shfl_xor_sync(0xffffffffu, best_slot, o);
        if (ob < best) { best = ob; best_slot = os; }
    }
    if (lane == 0) { red_key[warp] = best; red_slot[warp] = best_slot; }
    __syncthreads();

    // ---- (v) eviction and in-place insert, (vi) length ------------------------------------------
    float s_new = 0.f;
    for (int g = 0; g < G; ++g) s_new += w[(size_t)cnt * kMmaCols + g] * s_inv[g];
    if (tid == 0) {
        int target = full ? -2 : cnt;
        if (full) {
            unsigned long long gb = red_key[0];
            int gs = red_slot[0];
            for (int x = 1; x < NW; ++x)
                if (red_key[x] < gb) { gb = red_key[x]; gs = red_slot[x]; }
            const unsigned long long self_key = ((unsigned long long)__float_as_uint(s_new) << 32) | (unsigned)p;
            if (gs >= 0 && (c.R > 0 || gb < self_key)) target = gs;
        }
        s_target = target;
    }
    __syncthreads();
    const int target = s_target;
    if (target >= 0) {
        constexpr int LPR = D / 8;
        if (!A2SF_IN_RANGE(target, c.M, kDbgGroupMma)) {
        } else if (tid < LPR)
            *reinterpret_cast<uint4 *>(Ku + (size_t)target * D + tid * 8) =
                *reinterpret_cast<const uint4 *>(knu + tid * 8);
        else if (tid < 2 * LPR)
            *reinterpret_cast<uint4 *>(Vu + (size_t)target * D + (tid - LPR) * 8) =
                *reinterpret_cast<const uint4 *>(vnu + (tid - LPR) * 8);
    }
    if (tid == 0 && A2SF_IN_RANGE(u, c.U, kDbgGroupMma)) {
        if (target >= 0 && A2SF_IN_RANGE(target, c.M, kDbgGroupMma)) {
            Su[target] = s_new;
            posu[target] = p;
        }
        if (!full) c.count[u] = cnt + 1;
        c.len[u] = p + 1;
        evicted[u] = full ? target : -1;
    }
}

template <typename T, int D>
cudaError_t launch_group_mma(const CacheView &c, int G, float alpha, const void *q, const void *k_new,
                             const void *v_new, void *out, int32_t *evicted, cudaStream_t s)
{
    const size_t smem = group_mma_smem_bytes(c.M, D);
    auto kern = decode_step_group_mma_kernel<T, D>;
    if (cudaError_t e = allow_dynamic_smem<decode_step_group_mma_kernel<T, D>>(smem); e != cudaSuccess) return e;
    kern<<<c.U, kGroupThreads, smem, s>>>(c, G, alpha, static_cast<const T *>(q), static_cast<const T *>(k_new),
                                           static_cast<const T *>(v_new), static_cast<T *>(out), evicted);
    count_launch();
    return cudaGetLastError();
}

template <typename T, int D, int GMAX>
cudaError_t launch_group_n(const CacheView &c, int G, float alpha, const void *q, const void *k_new,
                           const void *v_new, void *out, int32_t *evicted, cudaStream_t s)
{
    const size_t smem = decode_group_smem_bytes(c.M, G, D);
    if (smem > 220 * 1024) return cudaErrorInvalidValue;
    auto kern = decode_step_group_kernel<T, D, GMAX>;
    if (cudaError_t e = allow_dynamic_smem<decode_step_group_kernel<T, D, GMAX>>(smem); e != cudaSuccess) return e;
    kern<<<c.U, kGroupThreads, smem, s>>>(c, G, alpha, static_cast<const T *>(q), static_cast<const T *>(k_new),
                                           static_cast<const T *>(v_new), static_cast<T *>(out), evicted);
    count_launch();
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch_group(const CacheView &c, int G, float alpha, const void *q, const void *k_new,
                         const void *v_new, void *out, int32_t *evicted, cudaStream_t s)
{
    // 16-bit storage takes the tensor-core form whenever its shared memory fits
    if constexpr (sizeof(T) == 2) {
        if (group_mma_smem_bytes(c.M, D) <= 220 * 1024)
            return launch_group_mma<T, D>(c, G, alpha, q, k_new, v_new, out, evicted, s);
    }
    if (G <= 2) return launch_group_n<T, D, 2>(c, G, alpha, q, k_new, v_new, out, evicted, s);
    if (G <= 4) return launch_group_n<T, D, 4>(c, G, alpha, q, k_new, v_new, out, evicted, s);
    return launch_group_n<T, D, 8>(c, G, alpha, q, k_new, v_new, out, evicted, s);
}

}  // namespace

cudaError_t launch_group_sum(const float *per_head, float *out, int G, int n, size_t units, cudaStream_t s)
{
    const size_t total = units * (size_t)n;
    const unsigned grid = (unsigned)std::min<size_t>((total + 255) / 256, 148 * 16);
    group_sum_kernel<<<grid, 256, 0, s>>>(per_head, out, G, n, total);
    count_launch();
    return cudaGetLastError();
}

size_t decode_group_smem_bytes(int M, int G, int d)
{
    // logits [G][wstride], partial outputs [warps][G][d], staged scores and positions [wstride] each
    return ((size_t)(G + 2) * group_wstride(M) + (size_t)(kGroupThreads / 32) * G * d) * sizeof(float);
}

cudaError_t launch_decode_step_group(const CacheView &c, int G, float alpha, const void *q, const void *k_new,
                                     const void *v_new, void *out, int32_t *evicted, cudaStream_t s)
{
    if (G < 1 || G > kMaxGroup) return cudaErrorInvalidValue;
#define A2SF_DISPATCH(T)                                                                  \
    (c.d == 64 ? launch_group<T, 64>(c, G, alpha, q, k_new, v_new, out, evicted, s)        \
               : launch_group<T, 128>(c, G, alpha, q, k_new, v_new, out, evicted, s))
    switch (c.dtype) {
    case A2SF_F32: return A2SF_DISPATCH(float);
    case A2SF_BF16: return A2SF_DISPATCH(__nv_bfloat16);
    default: return A2SF_DISPATCH(__half);
    }
#undef A2SF_DISPATCH
}

}  // namespace a2sf
