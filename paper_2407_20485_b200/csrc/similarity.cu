// Similarity with the ideal mask (paper Sec. 4.3, the mask figure and the similarity table).
//
// While the prompt streams through the pruning policy row by row, row i of the policy attends to
// the cached tokens and to itself.  The ideal row keeps the same number of tokens, budget + 1,
// but picks them by the size of their logits alone, from ALL tokens 0..i (nothing is ever
// removed for good).  The diagnostic is the cosine between the two probability rows.
//
//   ideal_stats_kernel   : one CTA per (row, unit): the row's logits, the (budget+1)-th largest
//                          under (logit, lower position first), and the sums the cosine needs.
//   similarity_row_kernel: one CTA per unit, before the step kernel handles row i: logits of the
//                          cached slots (the same arithmetic, so equal logits compare equal),
//                          cos_i = sum_kept a_j p_j / (|a| |p|).  With a = e^(w-m')/l' and
//                          p = e^(w-m)/Z both normalisers cancel:
//                          cos_i = sum_kept e^(w-m') e^(w-m) / sqrt(sum e^(2(w-m')) * sum_kept e^(2(w-m))).
#include <climits>

#include "common.cuh"

namespace a2sf {

A2SF_DEBUG_TRANSLATION_UNIT(similarity)
namespace {

constexpr int kSimThreads = 256;

// q . k_row in a fixed order; both kernels call this, so a logit has the same bits in both
template <typename T, int D>
__device__ __forceinline__ float row_dot(const float *qs, const T *krow)
{
    constexpr int VEC = Elem<T>::kVec;
    float acc = 0.f;
#pragma unroll
    for (int c = 0; c < D / VEC; ++c) {
        float f[VEC];
        Elem<T>::unpack(*reinterpret_cast<const uint4 *>(krow + c * VEC), f);
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc = fmaf(qs[c * VEC + e], f[e], acc);
    }
    return acc;
}

template <typename T, int D>
__device__ __forceinline__ void load_q(float *qs, const T *qrow)
{
    constexpr int VEC = Elem<T>::kVec;
    if (threadIdx.x < D / VEC) {
        float f[VEC];
        Elem<T>::unpack(*reinterpret_cast<const uint4 *>(qrow + threadIdx.x * VEC), f);
#pragma unroll
        for (int e = 0; e < VEC; ++e) qs[threadIdx.x * VEC + e] = f[e];
    }
}

// float bits -> unsigned key with the same order
__device__ __forceinline__ uint32_t ordered_bits(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
// larger logit first, then the lower position
__device__ __forceinline__ unsigned long long rank_key(float logit, int pos)
{
    return ((unsigned long long)ordered_bits(logit) << 32) | (unsigned long long)(0xffffffffu - (uint32_t)pos);
}

// deterministic block sum: per-warp shuffle tree, then warp 0 over the warp totals
__device__ float block_sum(float v, float *red)
{
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = threadIdx.x < kSimThreads / 32 ? red[threadIdx.x] : 0.f;
    t = warp_sum(t);
    if (threadIdx.x == 0) red[0] = t;
    __syncthreads();
    return red[0];
}
__device__ float block_max(float v, float *red)
{
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = threadIdx.x < kSimThreads / 32 ? red[threadIdx.x] : -INFINITY;
    t = warp_max(t);
    if (threadIdx.x == 0) red[0] = t;
    __syncthreads();
    return red[0];
}

struct IdealStats {      // five arrays [U][n] in the workspace
    float *thr;          // logit of the last kept token
    int32_t *thr_pos;    // among logits equal to thr: kept iff position <= thr_pos
    float *m, *n2;       // row maximum; sum over kept of e^(2(s-m))
};

template <typename T, int D>
__global__ void __launch_bounds__(kSimThreads)
ideal_stats_kernel(const T *__restrict__ q, const T *__restrict__ k, Strides st, int H, int n, int keep,
                   float scale, IdealStats out)
{
    extern __shared__ float sim_smem[];
    float *logit = sim_smem;                 // [n]
    float *qs = sim_smem + n;                // [D]
    float *red = qs + D;                     // [8]
    __shared__ int hist[256];
    __shared__ unsigned long long s_prefix;
    __shared__ int s_rank;

    const int i = blockIdx.x, u = blockIdx.y;
    const size_t base = (size_t)(u / H) * st.b + (size_t)(u % H) * st.h;
    load_q<T, D>(qs, q + base + (size_t)i * st.t);
    __syncthreads();
    float mx = -INFINITY;
    for (int j = threadIdx.x; j <= i; j += kSimThreads) {
        const float s = row_dot<T, D>(qs, k + base + (size_t)j * st.t) * scale;
        if (A2SF_IN_RANGE(j, n, kDbgIdealStats)) logit[j] = s;
        mx = fmaxf(mx, s);
    }
    const float m = block_max(mx, red);

    // the keep-th largest (logit, lower position) pair: radix select, 8 bits per pass
    unsigned long long thr_key = 0ull;       // keep >= i+1: every token stays
    if (keep < i + 1) {
        if (threadIdx.x == 0) { s_prefix = 0ull; s_rank = keep; }
        for (int pass = 7; pass >= 0; --pass) {
            hist[threadIdx.x] = 0;
            __syncthreads();
            const unsigned long long prefix = s_prefix;
            const unsigned long long hi_mask = pass == 7 ? 0ull : (~0ull << ((pass + 1) * 8));
            for (int j = threadIdx.x; j <= i; j += kSimThreads) {
                const unsigned long long key = rank_key(logit[j], j);
                if ((key & hi_mask) == prefix) atomicAdd(&hist[(int)((key >> (pass * 8)) & 0xff)], 1);
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                int rank = s_rank, b = 255;
                for (; b > 0; --b) {
                    if (hist[b] >= rank) break;
                    rank -= hist[b];
                }
                s_rank = rank;
                s_prefix = prefix | ((unsigned long long)b << (pass * 8));
            }
            __syncthreads();
        }
        thr_key = s_prefix;
    }
    float n2 = 0.f;
    for (int j = threadIdx.x; j <= i; j += kSimThreads) {
        const float s = logit[j];
        if (rank_key(s, j) >= thr_key) {
            const float e = exp2f((s - m) * kLog2e);
            n2 = fmaf(e, e, n2);
        }
    }
    n2 = block_sum(n2, red);
    if (threadIdx.x == 0) {
        const size_t o = (size_t)u * n + i;
        if (!A2SF_IN_RANGE(i, n, kDbgIdealStats)) return;
        out.thr[o] = keep < i + 1 ? from_ordered_bits((uint32_t)(thr_key >> 32)) : -INFINITY;
        out.thr_pos[o] = keep < i + 1 ? (int32_t)(0xffffffffu - (uint32_t)(thr_key & 0xffffffffu)) : INT_MAX;
        out.m[o] = m;
        out.n2[o] = n2;
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(kSimThreads)
similarity_row_kernel(CacheView c, const T *__restrict__ q, const T *__restrict__ k_new, int n, int i,
                      IdealStats ideal, float *__restrict__ cos_out)
{
    extern __shared__ float sim_smem[];
    float *w = sim_smem;                     // [M + 1]
    float *qs = sim_smem + c.M + 1;          // [D]
    float *red = qs + D;                     // [8]

    const int u = blockIdx.x;
    const size_t uo = io_offset(c, u);
    const int cnt = min(c.count[u], c.M);
    const T *Ku = reinterpret_cast<const T *>(c.K) + (size_t)u * c.M * D;
    const int32_t *posu = c.pos + (size_t)u * c.M;
    load_q<T, D>(qs, q + uo);
    __syncthreads();
    float mx = -INFINITY;
    for (int s = threadIdx.x; s <= cnt; s += kSimThreads) {
        const float v = row_dot<T, D>(qs, s < cnt ? Ku + (size_t)s * D : k_new + uo) * c.scale;
        if (A2SF_IN_RANGE(s, c.M + 1, kDbgSimilarityRow)) w[s] = v;
        mx = fmaxf(mx, v);
    }
    const float m_meth = block_max(mx, red);
    const size_t o = (size_t)u * n + i;
    const float thr = ideal.thr[o], m_id = ideal.m[o];
    const int thr_pos = ideal.thr_pos[o];
    float a2 = 0.f, dot = 0.f;
    for (int s = threadIdx.x; s <= cnt; s += kSimThreads) {
        const float v = w[s];
        const int pos = s < cnt ? posu[s] : i;
        const float e = exp2f((v - m_meth) * kLog2e);
        a2 = fmaf(e, e, a2);
        if (v > thr || (v == thr && pos <= thr_pos)) dot = fmaf(e, exp2f((v - m_id) * kLog2e), dot);
    }
    a2 = block_sum(a2, red);
    dot = block_sum(dot, red);
    if (threadIdx.x == 0 && A2SF_IN_RANGE(i, n, kDbgSimilarityRow)) cos_out[o] = dot / sqrtf(a2 * ideal.n2[o]);
}

template <typename T, int D>
cudaError_t run(const CacheView &view, float alpha, int H, int n, const void *q, const void *k,
                const void *v, Strides st, void *out, float *cos_out, int32_t *evicted, int32_t *ev_scratch,
                void *ws, cudaStream_t s)
{
    const size_t rows = (size_t)view.U * n;
    IdealStats is;
    is.thr = static_cast<float *>(ws);
    is.thr_pos = reinterpret_cast<int32_t *>(is.thr + rows);
    is.m = reinterpret_cast<float *>(is.thr_pos + rows);
    is.n2 = is.m + rows;
    const size_t smem_a = ((size_t)n + D + 8) * sizeof(float);
    const size_t smem_b = ((size_t)view.M + 1 + D + 8) * sizeof(float);
    auto ka = ideal_stats_kernel<T, D>;
    auto kb = similarity_row_kernel<T, D>;
    cudaError_t e;
    if (smem_a > 48 * 1024 &&
        (e = cudaFuncSetAttribute(ka, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_a)) != cudaSuccess)
        return e;
    if (smem_b > 48 * 1024 &&
        (e = cudaFuncSetAttribute(kb, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_b)) != cudaSuccess)
        return e;
    ka<<<dim3(n, view.U), kSimThreads, smem_a, s>>>(static_cast<const T *>(q), static_cast<const T *>(k), st,
                                                     H, n, view.M + 1, view.scale, is);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    CacheView c = view;
    c.io_st_b = st.b;
    c.io_st_h = st.h;
    for (int i = 0; i < n; ++i) {
        const size_t off = (size_t)i * (size_t)st.t;
        const T *qi = static_cast<const T *>(q) + off, *ki = static_cast<const T *>(k) + off;
        kb<<<view.U, kSimThreads, smem_b, s>>>(c, qi, ki, n, i, is, cos_out);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        int32_t *ev = evicted ? evicted + (size_t)i * view.U : ev_scratch;
        if ((e = launch_decode_step(c, alpha, nullptr, qi, ki, static_cast<const T *>(v) + off,
                                    static_cast<T *>(out) + off, ev, s)) != cudaSuccess)
            return e;
    }
    return cudaSuccess;
}

}  // namespace

size_t ideal_similarity_ws_bytes(size_t units, int n) { return units * (size_t)n * 4 * sizeof(float); }

cudaError_t launch_ideal_similarity(const CacheView &view, float alpha, int H, int n, const void *q,
                                    const void *k, const void *v, Strides st, void *out, float *cos_out,
                                    int32_t *evicted, int32_t *ev_scratch, void *ws, cudaStream_t s)
{
#define A2SF_DISPATCH(T)                                                                              \
    (view.d == 64 ? run<T, 64>(view, alpha, H, n, q, k, v, st, out, cos_out, evicted, ev_scratch, ws, s) \
                  : run<T, 128>(view, alpha, H, n, q, k, v, st, out, cos_out, evicted, ev_scratch, ws, s))
    switch (view.dtype) {
    case A2SF_F32: return A2SF_DISPATCH(float);
    case A2SF_BF16: return A2SF_DISPATCH(__nv_bfloat16);
    default: return A2SF_DISPATCH(__half);
    }
#undef A2SF_DISPATCH
}

}  // namespace a2sf
