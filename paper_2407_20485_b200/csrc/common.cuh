// Shared device/host helpers of liba2sf (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/a2sf.h"

namespace a2sf {

constexpr float kLog2e = 1.4426950408889634f;

// Strided view of a [B][H][n][d] tensor; strides in elements, d contiguous.
struct Strides {
    int64_t b, h, t;
};

// ---- element traits: 16-byte vector <-> fp32 --------------------------------
template <typename T> struct Elem;

template <> struct Elem<float> {
    static constexpr int kVec = 4;   // elements per 16 bytes
    __device__ static void unpack(const uint4 &r, float *f)
    {
        f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y);
        f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
    }
    __device__ static float to_float(float x) { return x; }
    __device__ static float from_float(float x) { return x; }
};

template <> struct Elem<__nv_bfloat16> {
    static constexpr int kVec = 8;
    __device__ static void unpack(const uint4 &r, float *f)
    {
        // a bf16 is the upper half of an fp32
        f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
        f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
        f[4] = __uint_as_float(r.z << 16); f[5] = __uint_as_float(r.z & 0xffff0000u);
        f[6] = __uint_as_float(r.w << 16); f[7] = __uint_as_float(r.w & 0xffff0000u);
    }
    __device__ static float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
    __device__ static __nv_bfloat16 from_float(float x) { return __float2bfloat16_rn(x); }
};

template <> struct Elem<__half> {
    static constexpr int kVec = 8;
    __device__ static void unpack(const uint4 &r, float *f)
    {
        const __half2 *h = reinterpret_cast<const __half2 *>(&r);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 t = __half22float2(h[i]);
            f[2 * i] = t.x; f[2 * i + 1] = t.y;
        }
    }
    __device__ static float to_float(__half x) { return __half2float(x); }
    __device__ static __half from_float(float x) { return __float2half_rn(x); }
};

// streaming 16-byte load that does not displace L1 lines; only for data that no thread writes
// while the kernel runs (the non-coherent path)
__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// the same for rows that the kernel itself may overwrite later in the launch (a cache row that
// the new token replaces): the ordinary coherent path, still without an L1 allocation
__device__ __forceinline__ uint4 ld_stream16_rw(const void *p)
{
    uint4 r;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p) : "memory");
    return r;
}

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ unsigned long long warp_min_u64(unsigned long long v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long t = __shfl_xor_sync(0xffffffffu, v, o);
        v = t < v ? t : v;
    }
    return v;
}

// ---- bounds-checked debug build (-DA2SF_DEBUG) -------------------------------------------
// In the debug library every slot, position, tile-row and ring-stage index that addresses
// global or shared memory passes through A2SF_IN_RANGE before it is used.  A violation is
// counted, the first one is recorded (kernel id, source line, index, bound) in a device word
// that a2sf_debug_violations reads, and the access is SKIPPED: nothing traps, the context stays
// usable.  In the release library the macro is the constant `true` and costs nothing.
enum DebugKernelId {
    kDbgSelect = 1, kDbgCacheLoad, kDbgDecodeStream, kDbgDecodeSplit, kDbgGroupMma, kDbgGroupSimt,
    kDbgGroupSum, kDbgPrefillSimt1, kDbgPrefillSimt2, kDbgAttnTc, kDbgScoreTc, kDbgVToHalf,
    kDbgIdealStats, kDbgSimilarityRow
};
#ifdef A2SF_DEBUG
// one record per translation unit (no relocatable device code): {violations, kernel << 32 | line,
// index, bound}
static __device__ unsigned long long g_dbg_record[4];
__device__ __forceinline__ bool dbg_in_range(long long idx, long long bound, int kernel_id, int line)
{
    if (idx >= 0 && idx < bound) return true;
    if (atomicAdd(&g_dbg_record[0], 1ull) == 0ull) {
        g_dbg_record[1] = ((unsigned long long)kernel_id << 32) | (unsigned)line;
        g_dbg_record[2] = (unsigned long long)idx;
        g_dbg_record[3] = (unsigned long long)bound;
    }
    return false;
}
#define A2SF_IN_RANGE(idx, bound, kernel_id) \
    (::a2sf::dbg_in_range((long long)(idx), (long long)(bound), (kernel_id), __LINE__))
// Host side: every translation unit with kernels registers a reader of its record.
typedef int (*DebugReader)(unsigned long long *out4, cudaStream_t s);
void register_debug_reader(DebugReader fn);
#define A2SF_DEBUG_TRANSLATION_UNIT(name)                                                              \
    namespace {                                                                                        \
    int dbg_read_##name(unsigned long long *out4, cudaStream_t s)                                      \
    {                                                                                                  \
        const unsigned long long zero[4] = {0, 0, 0, 0};                                               \
        if (cudaMemcpyFromSymbolAsync(out4, g_dbg_record, sizeof(zero), 0, cudaMemcpyDeviceToHost, s) != cudaSuccess ||  \
            cudaStreamSynchronize(s) != cudaSuccess)                                                   \
            return -1;                                                                                 \
        if (out4[0] != 0 &&                                                                            \
            (cudaMemcpyToSymbolAsync(g_dbg_record, zero, sizeof(zero), 0, cudaMemcpyHostToDevice, s) != cudaSuccess ||  \
             cudaStreamSynchronize(s) != cudaSuccess))                                                 \
            return -1;                                                                                 \
        return 0;                                                                                      \
    }                                                                                                  \
    struct DbgRegistrar_##name {                                                                       \
        DbgRegistrar_##name() { ::a2sf::register_debug_reader(&dbg_read_##name); }                     \
    } dbg_registrar_##name;                                                                            \
    }
#else
#define A2SF_IN_RANGE(idx, bound, kernel_id) (true)
#define A2SF_DEBUG_TRANSLATION_UNIT(name)
#endif

// ---- tracing: an NVTX range around each entry point of the C ABI ---------------------------
// (header-only NVTX: without a profiler attached a range costs one pointer test)
struct TraceRange {
    explicit TraceRange(const char *name);
    ~TraceRange();
    TraceRange(const TraceRange &) = delete;
    TraceRange &operator=(const TraceRange &) = delete;
};
#define A2SF_TRACE(name) ::a2sf::TraceRange a2sf_trace_range_(name)

// ---- host-side launch bookkeeping -------------------------------------------
void count_launch(int n = 1);

// Kernel attributes, symbol addresses and SM counts belong to a device: state that is set up
// once is kept per device, indexed by the current one.
constexpr int kMaxDevices = 64;
inline int current_device_index()
{
    int d = 0;
    if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= kMaxDevices) d = 0;
    return d;
}

// Number of SMs of the current device, looked up once per device.
inline int device_sm_count()
{
    static std::once_flag once[kMaxDevices];
    static int count[kMaxDevices] = {};
    const int dev = current_device_index();
    std::call_once(once[dev], [dev] {
        if (cudaDeviceGetAttribute(&count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) count[dev] = 0;
    });
    return count[dev];
}

// The dynamic shared-memory limit of a kernel is raised once per device and size, not per launch
// (the call is a driver round trip), under a lock.  The kernel is a template argument so that
// every kernel has its own record.
template <auto Kern>
cudaError_t allow_dynamic_smem(size_t smem)
{
    static std::mutex mu;
    static size_t granted[kMaxDevices] = {};
    if (smem <= 48 * 1024) return cudaSuccess;
    const int dev = current_device_index();
    std::lock_guard<std::mutex> lock(mu);
    if (smem > granted[dev]) {
        const cudaError_t e = cudaFuncSetAttribute(Kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        granted[dev] = smem;
    }
    return cudaSuccess;
}

// ---- host-side argument checks shared by every entry point (api.cu) ----------------------
int check_params(const a2sf_params *p);                                    // shape, policy, dtype, flags
int check_strides(const a2sf_params *p, int64_t sb, int64_t sh, int64_t st);   // element strides of q/k/v/out
float eff_scale(const a2sf_params *p);                                     // scale, or 1/sqrt(d) when 0

// ---- kernel launchers (one per translation unit) -----------------------------
struct PrefillArgs {
    const void *q, *k, *v;
    void *out;
    float *lse;        // [U][n]
    float *scores;     // [U][n]
    Strides st;        // of q and out
    Strides st_kv;     // of k and v ([B][H/G][n][d]); equal to st without head grouping
    int B, H, n, d;    // H = query heads
    int G;             // query heads per key/value head (1 = one K/V head per query head)
    float scale, alpha;
    const float *alpha_vec;   // per-unit forgetting factors [U] on the device, or nullptr (use alpha)
    int skip_zero_rows;       // scoring pass: leave out rows whose weight is exactly 0 in fp32
    int window_rows;          // scoring pass: only the last window_rows query rows (0 = all)
    void *v_half;             // bf16 tensor-core path: fp16 copy of V, contiguous [U][n][d] (workspace)
    int *v_flag;              // ... and the word that says the copy is not exact (workspace)
};

cudaError_t launch_prefill_pass1_simt(int dtype, const PrefillArgs &a, cudaStream_t s);
cudaError_t launch_prefill_pass2_simt(int dtype, const PrefillArgs &a, cudaStream_t s);

// tensor-core path (16-bit storage, d = 128)
bool prefill_tc_supported(int dtype, const PrefillArgs &a);
// extra workspace of the tensor-core attention pass (fp16 copy of V + flag; bf16 storage only)
size_t prefill_tc_extra_bytes(int dtype, size_t units, int n, int d);
cudaError_t launch_prefill_pass1_tc(int dtype, const PrefillArgs &a, cudaStream_t s);
cudaError_t launch_prefill_pass2_tc(int dtype, const PrefillArgs &a, cudaStream_t s);
int read_and_clear_tc_status(cudaStream_t s);
int *tc_status_word();       // device address of that status word on the current device (nullptr on failure)

cudaError_t launch_select(const float *scores, int32_t *kept, int U, int n, int M, int R,
                          cudaStream_t s);

struct CacheView {
    void *K, *V;          // [U][M][d]
    float *S;             // [U][M]
    int32_t *pos;         // [U][M]
    int32_t *count, *len; // [U]
    int32_t *sched;       // [2] unit-claim counter and finished-CTA counter of the decode kernel
    int U, M, R, d, dtype;
    float scale;
    // where unit u = b*io_H + h finds its row of the step's q, k_new, v_new and out (elements):
    // [B][H][d] contiguous for a generation step, a token's rows of a [B][H][n][d] tensor when
    // the prompt is streamed through the step kernel
    int io_H;
    long long io_st_b, io_st_h;
};

__host__ __device__ __forceinline__ size_t io_offset(const CacheView &c, int u)
{
    return (size_t)(u / c.io_H) * (size_t)c.io_st_b + (size_t)(u % c.io_H) * (size_t)c.io_st_h;
}

cudaError_t launch_cache_load(const CacheView &c, int H, int n, const void *k, const void *v,
                              Strides st, const float *scores, const int32_t *kept,
                              cudaStream_t s);

// alpha_vec: per-unit forgetting factors [U] on the device, or nullptr (use the scalar)
cudaError_t launch_decode_step(const CacheView &c, float alpha, const float *alpha_vec, const void *q,
                               const void *k_new, const void *v_new, void *out, int32_t *evicted,
                               cudaStream_t s);

// per-unit factors are clamped to [0, 1] on the device (they cannot be validated on the host)
__device__ __forceinline__ float unit_alpha(const float *alpha_vec, int u, float alpha)
{
    return alpha_vec ? fminf(fmaxf(alpha_vec[u], 0.f), 1.f) : alpha;
}

int read_and_clear_decode_status(cudaStream_t s);
int *decode_status_word();   // device address of that status word on the current device (nullptr on failure)
cudaError_t launch_wait_probe(int *status_word, long long limit_cycles, long long *report, cudaStream_t s);

// grouped query heads (G query heads per K/V head)
cudaError_t launch_group_sum(const float *per_head, float *out, int G, int n, size_t units, cudaStream_t s);
size_t decode_group_smem_bytes(int M, int G, int d);
cudaError_t launch_decode_step_group(const CacheView &c, int G, float alpha, const void *q, const void *k_new,
                                     const void *v_new, void *out, int32_t *evicted, cudaStream_t s);

// similarity with the ideal mask while the prompt streams through the step kernel
size_t ideal_similarity_ws_bytes(size_t units, int n);
cudaError_t launch_ideal_similarity(const CacheView &view, float alpha, int H, int n, const void *q,
                                    const void *k, const void *v, Strides st, void *out, float *cos_out,
                                    int32_t *evicted, int32_t *ev_scratch, void *ws, cudaStream_t s);

}  // namespace a2sf
