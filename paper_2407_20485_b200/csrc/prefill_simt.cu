// CUDA-core (fp32 FMA) prefill kernels.  They serve the fp32 storage type, whose
// index-exactness bar is too tight for TF32 tensor-core products, and any shape the
// tensor-core path does not cover.
//
//   pass 1: causal flash attention with online softmax -> out, lse   (paper Eq. 3)
//   pass 2: S_j = sum_{i>=j} alpha^(n-1-i) exp(s_ij - lse_i)          (paper Eq. 5-6)
//           column-parallel: every key's sum runs over rows in ascending order in
//           one thread group, so the result is deterministic and uses no atomics.
#include "common.cuh"

namespace a2sf {

A2SF_DEBUG_TRANSLATION_UNIT(prefill_simt)

namespace {

constexpr int kRows = 32;       // query rows (pass 1) / keys (pass 2) per CTA, 4 threads each
constexpr int kTile = 32;       // streamed tile height
constexpr int kThreads = 128;

// cooperative load of kTile x D elements starting at row r0 into fp32 shared memory
template <typename T, int D>
__device__ __forceinline__ void load_tile(float *dst, const T *base, int64_t stride_t, int r0,
                                          int n)
{
    constexpr int VEC = Elem<T>::kVec;
    constexpr int CH = D / VEC;           // 16-byte chunks per row
    for (int idx = threadIdx.x; idx < kTile * CH; idx += kThreads) {
        const int r = idx / CH, ch = idx % CH;
        float f[VEC];
        if (r0 + r < n) {
            Elem<T>::unpack(*reinterpret_cast<const uint4 *>(base + (int64_t)(r0 + r) * stride_t +
                                                             ch * VEC), f);
        } else {
#pragma unroll
            for (int e = 0; e < VEC; ++e) f[e] = 0.f;
        }
#pragma unroll
        for (int e = 0; e < VEC; e += 4)
            *reinterpret_cast<float4 *>(dst + r * D + ch * VEC + e) =
                make_float4(f[e], f[e + 1], f[e + 2], f[e + 3]);
    }
}

// Thread (row, tq) owns the float4 chunks {tq*4 + 16*c}: the four threads of a row
// read four consecutive float4 of a shared row (conflict-free), rows broadcast.
template <int D>
__device__ __forceinline__ float dot_part(const float (&a)[D / 4], const float *row, int tq)
{
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < D / 16; ++c) {
        const float4 k4 = *reinterpret_cast<const float4 *>(row + c * 16 + tq * 4);
        s = fmaf(a[c * 4 + 0], k4.x, s);
        s = fmaf(a[c * 4 + 1], k4.y, s);
        s = fmaf(a[c * 4 + 2], k4.z, s);
        s = fmaf(a[c * 4 + 3], k4.w, s);
    }
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    return s;
}

template <typename T, int D>
__device__ __forceinline__ void load_own_row(float (&a)[D / 4], const T *row_ptr, int tq, bool valid)
{
#pragma unroll
    for (int c = 0; c < D / 16; ++c)
#pragma unroll
        for (int e = 0; e < 4; ++e)
            a[c * 4 + e] = valid ? Elem<T>::to_float(row_ptr[c * 16 + tq * 4 + e]) : 0.f;
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) prefill_pass1_simt(PrefillArgs a)
{
    __shared__ __align__(16) float Ks[kTile * D];
    __shared__ __align__(16) float Vs[kTile * D];

    const int nblk = (a.n + kRows - 1) / kRows;
    const int rb = nblk - 1 - blockIdx.y;            // longest rows first
    const int u = blockIdx.x;
    const int b = u / a.H, h = u % a.H;
    const int64_t base = (int64_t)b * a.st.b + (int64_t)h * a.st.h;
    const int64_t base_kv = (int64_t)b * a.st_kv.b + (int64_t)(h / a.G) * a.st_kv.h;   // shared K/V head
    const T *Q = static_cast<const T *>(a.q) + base;
    const T *K = static_cast<const T *>(a.k) + base_kv;
    const T *V = static_cast<const T *>(a.v) + base_kv;
    T *O = static_cast<T *>(a.out) + base;

    const int tq = threadIdx.x & 3;
    const int i = rb * kRows + (threadIdx.x >> 2);
    const bool valid = i < a.n;

    float qv[D / 4], o[D / 4];
    load_own_row<T, D>(qv, Q + (int64_t)i * a.st.t, tq, valid);
#pragma unroll
    for (int c = 0; c < D / 4; ++c) o[c] = 0.f;
    float m = -INFINITY, l = 0.f;

    const int last_row = min(a.n, (rb + 1) * kRows) - 1;
    for (int j0 = 0; j0 <= last_row; j0 += kTile) {
        __syncthreads();
        load_tile<T, D>(Ks, K, a.st_kv.t, j0, a.n);
        load_tile<T, D>(Vs, V, a.st_kv.t, j0, a.n);
        __syncthreads();
        float s[kTile];
        float tmax = -INFINITY;
#pragma unroll
        for (int jj = 0; jj < kTile; ++jj) {
            float t = dot_part<D>(qv, Ks + jj * D, tq) * a.scale;
            t = (j0 + jj <= i) ? t : -INFINITY;      // causal mask
            s[jj] = t;
            tmax = fmaxf(tmax, t);
        }
        if (tmax == -INFINITY) continue;             // whole tile masked for this row
        const float m_new = fmaxf(m, tmax);
        const float corr = expf(m - m_new);           // m = -inf -> 0
        l *= corr;
#pragma unroll
        for (int c = 0; c < D / 4; ++c) o[c] *= corr;
#pragma unroll
        for (int jj = 0; jj < kTile; ++jj) {
            const float pj = expf(s[jj] - m_new);    // masked -> 0
            l += pj;
#pragma unroll
            for (int c = 0; c < D / 16; ++c) {
                const float4 v4 = *reinterpret_cast<const float4 *>(Vs + jj * D + c * 16 + tq * 4);
                o[c * 4 + 0] = fmaf(pj, v4.x, o[c * 4 + 0]);
                o[c * 4 + 1] = fmaf(pj, v4.y, o[c * 4 + 1]);
                o[c * 4 + 2] = fmaf(pj, v4.z, o[c * 4 + 2]);
                o[c * 4 + 3] = fmaf(pj, v4.w, o[c * 4 + 3]);
            }
        }
        m = m_new;
    }
    if (valid && A2SF_IN_RANGE(i, a.n, kDbgPrefillSimt1)) {
        const float inv = 1.f / l;
        T *orow = O + (int64_t)i * a.st.t;
#pragma unroll
        for (int c = 0; c < D / 16; ++c)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                orow[c * 16 + tq * 4 + e] = Elem<T>::from_float(o[c * 4 + e] * inv);
        if (tq == 0) a.lse[(int64_t)u * a.n + i] = m + logf(l);
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) prefill_pass2_simt(PrefillArgs a)
{
    __shared__ __align__(16) float Qs[kTile * D];
    __shared__ float cs[kTile];                      // row constants, log2 domain

    const int kb = blockIdx.y;                       // key block 0 sees the most rows: first
    const int u = blockIdx.x;
    const int b = u / a.H, h = u % a.H;
    const int64_t base = (int64_t)b * a.st.b + (int64_t)h * a.st.h;
    const int64_t base_kv = (int64_t)b * a.st_kv.b + (int64_t)(h / a.G) * a.st_kv.h;
    const T *Q = static_cast<const T *>(a.q) + base;
    const T *K = static_cast<const T *>(a.k) + base_kv;
    const float *lse = a.lse + (int64_t)u * a.n;

    const int tq = threadIdx.x & 3;
    const int j = kb * kRows + (threadIdx.x >> 2);
    const bool valid = j < a.n;

    float kv[D / 4];
    load_own_row<T, D>(kv, K + (int64_t)j * a.st_kv.t, tq, valid);

    // weight alpha^(n-1-i) folded into the exponent: exp2(s*log2e - c_i),
    // c_i = lse_i*log2e - (n-1-i)*log2(alpha); alpha = 0 keeps only row n-1 (0^0 = 1).
    const float alpha = unit_alpha(a.alpha_vec, u, a.alpha);
    const float neg_log2_alpha = alpha > 0.f ? -log2f(alpha) : INFINITY;
    const float sl2 = a.scale * kLog2e;

    // rows whose weight is below 2^-152 contribute exactly 0 even with denormals
    int i_first = kb * kRows;
    if (a.skip_zero_rows && neg_log2_alpha > 0.f) {
        const float span = ceilf(152.f / neg_log2_alpha);
        const int i_min = span >= (float)a.n ? 0 : min(a.n - 1, a.n - (int)span);
        i_first = max(i_first, (i_min / kTile) * kTile);
    }
    // truncated sum: only the last window_rows query rows enter (the caller accepts the bound)
    const int i_window = a.window_rows > 0 ? max(0, a.n - a.window_rows) : 0;
    i_first = max(i_first, (i_window / kTile) * kTile);
    float acc = 0.f;
    for (int i0 = i_first; i0 < a.n; i0 += kTile) {
        __syncthreads();
        load_tile<T, D>(Qs, Q, a.st.t, i0, a.n);
        if (threadIdx.x < kTile) {
            const int i = i0 + threadIdx.x;
            float cv = INFINITY;                     // rows past n or before the window: nothing
            if (i < a.n && i >= i_window) {
                const int age = a.n - 1 - i;
                cv = lse[i] * kLog2e + (age == 0 ? 0.f : (float)age * neg_log2_alpha);
            }
            if (A2SF_IN_RANGE(threadIdx.x, kTile, kDbgPrefillSimt2)) cs[threadIdx.x] = cv;
        }
        __syncthreads();
#pragma unroll 8
        for (int ii = 0; ii < kTile; ++ii) {
            const float t = dot_part<D>(kv, Qs + ii * D, tq);
            const float pw = exp2f(fmaf(t, sl2, -cs[ii]));
            acc += (i0 + ii >= j) ? pw : 0.f;         // causal: rows i >= j only
        }
    }
    if (valid && tq == 0 && A2SF_IN_RANGE(j, a.n, kDbgPrefillSimt2)) a.scores[(int64_t)u * a.n + j] = acc;
}

template <typename T, int D>
cudaError_t launch1(const PrefillArgs &a, cudaStream_t s)
{
    dim3 grid(a.B * a.H, (a.n + kRows - 1) / kRows);
    prefill_pass1_simt<T, D><<<grid, kThreads, 0, s>>>(a);
    count_launch();
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch2(const PrefillArgs &a, cudaStream_t s)
{
    dim3 grid(a.B * a.H, (a.n + kRows - 1) / kRows);
    prefill_pass2_simt<T, D><<<grid, kThreads, 0, s>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

#define A2SF_DISPATCH(fn)                                                        \
    switch (dtype) {                                                             \
    case A2SF_F32: return a.d == 64 ? fn<float, 64>(a, s) : fn<float, 128>(a, s); \
    case A2SF_BF16:                                                              \
        return a.d == 64 ? fn<__nv_bfloat16, 64>(a, s) : fn<__nv_bfloat16, 128>(a, s); \
    default: return a.d == 64 ? fn<__half, 64>(a, s) : fn<__half, 128>(a, s);     \
    }

cudaError_t launch_prefill_pass1_simt(int dtype, const PrefillArgs &a, cudaStream_t s)
{
    A2SF_DISPATCH(launch1)
}

cudaError_t launch_prefill_pass2_simt(int dtype, const PrefillArgs &a, cudaStream_t s)
{
    A2SF_DISPATCH(launch2)
}

}  // namespace a2sf
