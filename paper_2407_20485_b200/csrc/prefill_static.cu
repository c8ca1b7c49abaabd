// Prefill for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a serving
// engine that has handed the whole device to its own pool allocator, in a plugin
// that is only given the tensors of one layer, or in a real-time loop where an
// allocation's implicit synchronisation is not acceptable.  a2sf_prefill needs a
// scratch row per (batch, head, token) for the log-sum-exp that the first pass
// writes and the scoring pass reads; here that scratch is a fixed array that lives
// in the library's own device image, so the caller passes inputs and outputs only.
#include <mutex>

#include "common.cuh"

namespace a2sf {

// 4 MiB of fp32 log-sum-exp rows: B*H*n <= 1,048,576 (e.g. 32 heads x 32768 tokens,
// or 256 heads x 4096).  Every GPU that loads the library holds it until exit.
constexpr size_t kStaticLseFloats = size_t(1) << 20;
static __device__ __align__(256) float g_static_lse[kStaticLseFloats];

namespace {

std::mutex g_mu;
float *g_lse_addr[kMaxDevices] = {};

// The array's name is only a host-side handle; the device address has to be asked
// for, once per device, with that device current.
int static_lse_address(float **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return A2SF_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_lse_addr[dev]) {
        float *ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_static_lse) != cudaSuccess || !ptr)
            return A2SF_ERR_CUDA;
        g_lse_addr[dev] = ptr;
    }
    *out = g_lse_addr[dev];
    return A2SF_OK;
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace
}  // namespace a2sf

using namespace a2sf;

extern "C" size_t a2sf_prefill_static_scratch_max_rows(void) { return kStaticLseFloats; }

extern "C" int a2sf_prefill_static_scratch(const a2sf_params *p, int32_t n, const void *q,
                                           const void *k, const void *v, int64_t stride_b,
                                           int64_t stride_h, int64_t stride_t, void *out,
                                           float *scores, int32_t *kept_idx, void *cuda_stream)
{
    A2SF_TRACE("a2sf_prefill_static_scratch");
    // the same checks, in the same order, as a2sf_prefill
    int rc = check_params(p);
    if (rc != A2SF_OK) return rc;
    if (n < 1 || !q || !k || !v || !out || !scores || !kept_idx) return A2SF_ERR_INVALID_ARG;
    if ((rc = check_strides(p, stride_b, stride_h, stride_t)) != A2SF_OK) return rc;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) ||
        (reinterpret_cast<uintptr_t>(scores) & 3) || (reinterpret_cast<uintptr_t>(kept_idx) & 3))
        return A2SF_ERR_INVALID_ARG;
    // the scratch is fixed: refuse what does not fit rather than overrun it
    if ((size_t)p->B * (size_t)p->H * (size_t)n > kStaticLseFloats) return A2SF_ERR_WORKSPACE;

    float *lse = nullptr;
    if ((rc = static_lse_address(&lse)) != A2SF_OK) return rc;

    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    PrefillArgs a;
    a.q = q; a.k = k; a.v = v; a.out = out;
    a.lse = lse;          // every row this call reads is written by its own first pass,
    a.scores = scores;    // so nothing has to be cleared between calls
    a.st = Strides{stride_b, stride_h, stride_t};
    a.st_kv = a.st; a.G = 1;
    a.B = p->B; a.H = p->H; a.n = n; a.d = p->d;
    a.scale = eff_scale(p);
    a.alpha = p->alpha;
    a.alpha_vec = nullptr;
    a.skip_zero_rows = (p->flags & A2SF_FLAG_SKIP_ZERO_WEIGHT_ROWS) ? 1 : 0;
    a.window_rows = p->score_window;
    // no workspace, hence no fp16 copy of V: 16-bit storage with d = 128 still runs on the tensor
    // cores (bf16 multiplies P as two bf16 terms with V as it is), everything else on CUDA cores
    a.v_half = nullptr;
    a.v_flag = nullptr;
    const bool tc = prefill_tc_supported(p->dtype, a);
    if ((tc ? launch_prefill_pass1_tc(p->dtype, a, s) : launch_prefill_pass1_simt(p->dtype, a, s)) != cudaSuccess)
        return A2SF_ERR_CUDA;
    if ((tc ? launch_prefill_pass2_tc(p->dtype, a, s) : launch_prefill_pass2_simt(p->dtype, a, s)) != cudaSuccess)
        return A2SF_ERR_CUDA;
    if (launch_select(scores, kept_idx, p->B * p->H, n, p->budget, p->recent, s) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return A2SF_OK;
}
