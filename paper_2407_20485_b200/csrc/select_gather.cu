// Kept-set selection (radix select on the fp32 score bits, ties resolved by
// position) and the gather that builds the slot-indexed cache.  Integer work:
// results are exact.  (Paper Sec. 3.1: low-score tokens leave the cache;
// Sec. 4.1: the budget is a recent window plus a selective part.)
#include "common.cuh"

namespace a2sf {

A2SF_DEBUG_TRANSLATION_UNIT(select_gather)

namespace {

constexpr int kSelThreads = 1024;

// exclusive block scan of one int per thread; returns the exclusive prefix and the total
__device__ __forceinline__ int block_excl_scan(int v, int *warp_tot, int &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int t = warp_tot[lane];
        int ti = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int x = __shfl_up_sync(0xffffffffu, ti, o);
            if (lane >= o) ti += x;
        }
        warp_tot[lane] = ti - t;          // exclusive offsets of the warps
        if (lane == 31) warp_tot[32] = ti;
    }
    __syncthreads();
    total = warp_tot[32];
    return warp_tot[warp] + incl - v;
}

// One CTA per unit.  Drops the `n - M` smallest candidates (positions < n - R)
// under (score, position) ascending; writes the survivors plus the recent window
// in ascending position order.
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float *__restrict__ scores, int32_t *__restrict__ kept, int n, int M, int R)
{
    __shared__ int hist[256];
    __shared__ int warp_tot[33];
    __shared__ unsigned s_prefix;
    __shared__ int s_rank;

    const int u = blockIdx.x;
    const unsigned *S = reinterpret_cast<const unsigned *>(scores + (size_t)u * n);
    int32_t *out = kept + (size_t)u * min(n, M);
    const int tid = threadIdx.x;

    if (n <= M) {
        for (int j = tid; j < n; j += kSelThreads)
            if (A2SF_IN_RANGE(j, min(n, M), kDbgSelect)) out[j] = j;
        return;
    }
    const int ncand = n - R;
    const int drop = n - M;               // 1 <= drop <= ncand

    // radix select: bit pattern of the drop-th smallest candidate score
    // (scores are >= 0, so the fp32 bit patterns order like the values)
    unsigned prefix = 0, mask = 0;
    int rank = drop;                      // 1-based rank inside the current bucket
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (int j = tid; j < ncand; j += kSelThreads) {
            const unsigned bits = A2SF_IN_RANGE(j, n, kDbgSelect) ? S[j] : 0u;
            if ((bits & mask) == prefix) atomicAdd(&hist[(bits >> shift) & 255u], 1);
        }
        __syncthreads();
        if (tid == 0) {
            int cum = 0, bkt = 0;
            for (; bkt < 255; ++bkt) {
                if (cum + hist[bkt] >= rank) break;
                cum += hist[bkt];
            }
            s_prefix = prefix | ((unsigned)bkt << shift);
            s_rank = rank - cum;
        }
        __syncthreads();
        prefix = s_prefix;
        rank = s_rank;
        mask |= 255u << shift;
        __syncthreads();
    }
    const unsigned thr = prefix;          // threshold score; `rank` equal-valued ones still go
    const int eq_drop = rank;

    int kept_base = 0, eq_base = 0;
    for (int j0 = 0; j0 < n; j0 += kSelThreads) {
        const int j = j0 + tid;
        unsigned bits = 0;
        bool cand = false;
        if (j < n && A2SF_IN_RANGE(j, n, kDbgSelect)) { bits = S[j]; cand = j < ncand; }
        const int is_eq = (cand && bits == thr) ? 1 : 0;
        int eq_total;
        const int eq_before = eq_base + block_excl_scan(is_eq, warp_tot, eq_total);
        bool keep = false;
        if (j < n) keep = !cand || bits > thr || (is_eq && eq_before >= eq_drop);
        int keep_total;
        const int kpos = kept_base + block_excl_scan(keep ? 1 : 0, warp_tot, keep_total);
        if (keep && kpos < M && A2SF_IN_RANGE(kpos, min(n, M), kDbgSelect)) out[kpos] = j;
        kept_base += keep_total;
        eq_base += eq_total;
    }
}

// One warp per (unit, slot): copy the kept token's K and V rows, score and position.
template <int ROW_BYTES>
__global__ void cache_load_kernel(CacheView c, int H, int n, const char *__restrict__ k,
                                  const char *__restrict__ v, Strides st_bytes,
                                  const float *__restrict__ scores,
                                  const int32_t *__restrict__ kept)
{
    const int warps_per_block = blockDim.x >> 5;
    const int slot = blockIdx.y * warps_per_block + (threadIdx.x >> 5);
    const int u = blockIdx.x;
    const int lane = threadIdx.x & 31;
    if (slot >= c.M || !A2SF_IN_RANGE(u, c.U, kDbgCacheLoad)) return;
    const int m = min(n, c.M);
    char *Kc = static_cast<char *>(c.K) + ((size_t)u * c.M + slot) * ROW_BYTES;
    char *Vc = static_cast<char *>(c.V) + ((size_t)u * c.M + slot) * ROW_BYTES;
    if (slot < m) {
        int j = kept[(size_t)u * m + slot];
        (void)A2SF_IN_RANGE(j, n, kDbgCacheLoad);      // debug build: a kept index outside the prompt is reported
        j = min(max(j, 0), n - 1);        // a corrupt index must not leave the tensor
        const int b = u / H, h = u % H;
        const int64_t off = b * st_bytes.b + h * st_bytes.h + (int64_t)j * st_bytes.t;
        for (int ch = lane; ch < ROW_BYTES / 16; ch += 32) {
            reinterpret_cast<uint4 *>(Kc)[ch] = *reinterpret_cast<const uint4 *>(k + off + ch * 16);
            reinterpret_cast<uint4 *>(Vc)[ch] = *reinterpret_cast<const uint4 *>(v + off + ch * 16);
        }
        if (lane == 0) {
            c.S[(size_t)u * c.M + slot] = scores[(size_t)u * n + j];
            c.pos[(size_t)u * c.M + slot] = j;
        }
    } else {
        for (int ch = lane; ch < ROW_BYTES / 16; ch += 32) {
            reinterpret_cast<uint4 *>(Kc)[ch] = make_uint4(0, 0, 0, 0);
            reinterpret_cast<uint4 *>(Vc)[ch] = make_uint4(0, 0, 0, 0);
        }
        if (lane == 0) {
            c.S[(size_t)u * c.M + slot] = 0.f;
            c.pos[(size_t)u * c.M + slot] = -1;
        }
    }
    if (slot == 0 && lane == 0) {
        c.count[u] = m;
        c.len[u] = n;
    }
}

}  // namespace

cudaError_t launch_select(const float *scores, int32_t *kept, int U, int n, int M, int R,
                          cudaStream_t s)
{
    select_kernel<<<U, kSelThreads, 0, s>>>(scores, kept, n, M, R);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_cache_load(const CacheView &c, int H, int n, const void *k, const void *v,
                              Strides st, const float *scores, const int32_t *kept,
                              cudaStream_t s)
{
    const int e = c.dtype == A2SF_F32 ? 4 : 2;
    const int row_bytes = c.d * e;
    Strides sb{st.b * e, st.h * e, st.t * e};
    const int wpb = 8;
    dim3 grid(c.U, (c.M + wpb - 1) / wpb);
    const char *kc = static_cast<const char *>(k), *vc = static_cast<const char *>(v);
    switch (row_bytes) {
    case 128: cache_load_kernel<128><<<grid, wpb * 32, 0, s>>>(c, H, n, kc, vc, sb, scores, kept); break;
    case 256: cache_load_kernel<256><<<grid, wpb * 32, 0, s>>>(c, H, n, kc, vc, sb, scores, kept); break;
    default: cache_load_kernel<512><<<grid, wpb * 32, 0, s>>>(c, H, n, kc, vc, sb, scores, kept); break;
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace a2sf
