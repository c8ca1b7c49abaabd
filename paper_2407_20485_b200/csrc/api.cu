// Host side of the C ABI declared in include/a2sf.h: argument validation, the cache
// object, workspace carving and kernel dispatch.  No data is touched on the host.
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

namespace a2sf {

TraceRange::TraceRange(const char *name) { nvtxRangePushA(name); }
TraceRange::~TraceRange() { nvtxRangePop(); }

static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

#ifdef A2SF_DEBUG
namespace {
struct DebugReaders {
    DebugReader fn[32];
    int n;
};
DebugReaders &debug_readers()
{
    static DebugReaders r = {{}, 0};      // constructed on first use: registration runs during static initialisation
    return r;
}
}  // namespace
void register_debug_reader(DebugReader fn)
{
    DebugReaders &r = debug_readers();
    if (r.n < 32) r.fn[r.n++] = fn;
}
#endif

static inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }
static inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
static inline int elem_bytes(int dtype) { return dtype == A2SF_F32 ? 4 : 2; }

int check_params(const a2sf_params *p)
{
    if (!p) return A2SF_ERR_INVALID_ARG;
    if (p->B < 1 || p->H < 1 || p->budget < 1 || p->recent < 0 || p->recent > p->budget)
        return A2SF_ERR_INVALID_ARG;
    if (!(p->alpha >= 0.f && p->alpha <= 1.f)) return A2SF_ERR_INVALID_ARG;   // rejects NaN
    if (!(p->scale >= 0.f) || std::isinf(p->scale)) return A2SF_ERR_INVALID_ARG;
    if (p->dtype != A2SF_F32 && p->dtype != A2SF_BF16 && p->dtype != A2SF_F16)
        return A2SF_ERR_UNSUPPORTED;
    if (p->d != 64 && p->d != 128) return A2SF_ERR_UNSUPPORTED;
    if (p->budget > A2SF_MAX_BUDGET) return A2SF_ERR_UNSUPPORTED;
    if ((int64_t)p->B * p->H > 0x7fffffff) return A2SF_ERR_INVALID_ARG;
    if (p->flags & ~A2SF_FLAG_SKIP_ZERO_WEIGHT_ROWS) return A2SF_ERR_INVALID_ARG;
    if (p->score_window < 0) return A2SF_ERR_INVALID_ARG;
    return A2SF_OK;
}

float eff_scale(const a2sf_params *p)
{
    return p->scale > 0.f ? p->scale : 1.0f / std::sqrt((float)p->d);
}

int check_strides(const a2sf_params *p, int64_t sb, int64_t sh, int64_t st)
{
    const int vec = 16 / elem_bytes(p->dtype);
    if (st < p->d || sh < 1 || sb < 1) return A2SF_ERR_INVALID_ARG;
    if (st % vec || sh % vec || sb % vec) return A2SF_ERR_INVALID_ARG;
    return A2SF_OK;
}

// prefill workspace: the log-sum-exp rows when the caller does not keep them
static size_t prefill_ws_bytes(const a2sf_params *p, int n)
{
    return align_up((size_t)p->B * p->H * n * sizeof(float)) +
           prefill_tc_extra_bytes(p->dtype, (size_t)p->B * p->H, n, p->d);
}

static int run_scores_and_select(const a2sf_params *p, int n, PrefillArgs &a, int32_t *kept,
                                 cudaStream_t s)
{
    const cudaError_t e2 = prefill_tc_supported(p->dtype, a) ? launch_prefill_pass2_tc(p->dtype, a, s)
                                                             : launch_prefill_pass2_simt(p->dtype, a, s);
    if (e2 != cudaSuccess) return A2SF_ERR_CUDA;
    if (launch_select(a.scores, kept, p->B * p->H, n, p->budget, p->recent, s) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return A2SF_OK;
}

// Two side streams and the events that fork from / join into the caller's stream, for the
// chunked host-buffer prefill.  Built once per device, on first use, and kept for the life of
// the process (creating and destroying them on every call costs several driver round trips).
struct HostPipeline {
    cudaStream_t side[2] = {nullptr, nullptr};
    cudaEvent_t start = nullptr, done[2] = {nullptr, nullptr};
    bool ok = false;
    std::mutex mu;          // one chunked call at a time per device: the calls share the streams
};

static HostPipeline *host_pipeline()
{
    static std::once_flag once[kMaxDevices];
    static HostPipeline pipes[kMaxDevices];
    const int dev = current_device_index();
    std::call_once(once[dev], [dev] {
        HostPipeline &hp = pipes[dev];
        bool ok = cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess;
        for (int x = 0; ok && x < 2; ++x)
            ok = cudaStreamCreateWithFlags(&hp.side[x], cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.done[x], cudaEventDisableTiming) == cudaSuccess;
        hp.ok = ok;
    });
    return &pipes[dev];
}

}  // namespace a2sf

using namespace a2sf;

struct a2sf_cache {
    a2sf_params p;
    CacheView view;
    void *mem;
    size_t bytes;
    bool owns;
    // staging rows for the host-buffer step: q, k_new, v_new, out [U][d], evicted [U]
    void *st_q, *st_k, *st_v, *st_out;
    int32_t *st_ev;
};

extern "C" {

size_t a2sf_prefill_workspace_bytes(const a2sf_params *p, int32_t n)
{
    if (check_params(p) != A2SF_OK || n < 1) return 0;
    return prefill_ws_bytes(p, n);
}

size_t a2sf_rescore_workspace_bytes(const a2sf_params *p, int32_t n)
{
    (void)p; (void)n;
    return 0;
}

static int prefill_impl(const a2sf_params *p, int32_t n, const void *q, const void *k, const void *v,
                        int64_t stride_b, int64_t stride_h, int64_t stride_t, const float *alpha_vec,
                        void *out, float *scores, int32_t *kept_idx, float *lse_opt, void *workspace,
                        size_t workspace_bytes, void *cuda_stream)
{
    A2SF_TRACE("a2sf_prefill");
    int rc = check_params(p);
    if (rc != A2SF_OK) return rc;
    if (n < 1 || !q || !k || !v || !out || !scores || !kept_idx) return A2SF_ERR_INVALID_ARG;
    if ((rc = check_strides(p, stride_b, stride_h, stride_t)) != A2SF_OK) return rc;
    if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(out, 16) ||
        !aligned(scores, 4) || !aligned(kept_idx, 4))
        return A2SF_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256)) return A2SF_ERR_INVALID_ARG;
    if (workspace_bytes < prefill_ws_bytes(p, n)) return A2SF_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);

    PrefillArgs a;
    a.q = q; a.k = k; a.v = v; a.out = out;
    a.lse = lse_opt ? lse_opt : static_cast<float *>(workspace);
    a.scores = scores;
    a.st = Strides{stride_b, stride_h, stride_t};
    a.st_kv = a.st; a.G = 1;
    a.B = p->B; a.H = p->H; a.n = n; a.d = p->d;
    a.scale = eff_scale(p); a.alpha = p->alpha; a.alpha_vec = alpha_vec;
    a.skip_zero_rows = (p->flags & A2SF_FLAG_SKIP_ZERO_WEIGHT_ROWS) ? 1 : 0;
    a.window_rows = p->score_window;
    a.v_half = nullptr; a.v_flag = nullptr;
    if (prefill_tc_extra_bytes(p->dtype, (size_t)p->B * p->H, n, p->d) > 0) {
        char *extra = static_cast<char *>(workspace) + align_up((size_t)p->B * p->H * n * sizeof(float));
        a.v_flag = reinterpret_cast<int *>(extra);
        a.v_half = extra + 256;
    }
    const cudaError_t e1 = prefill_tc_supported(p->dtype, a) ? launch_prefill_pass1_tc(p->dtype, a, s)
                                                             : launch_prefill_pass1_simt(p->dtype, a, s);
    if (e1 != cudaSuccess) return A2SF_ERR_CUDA;
    return run_scores_and_select(p, n, a, kept_idx, s);
}

int a2sf_prefill(const a2sf_params *p, int32_t n, const void *q, const void *k, const void *v,
                 int64_t stride_b, int64_t stride_h, int64_t stride_t, void *out, float *scores,
                 int32_t *kept_idx, float *lse_opt, void *workspace, size_t workspace_bytes,
                 void *cuda_stream)
{
    return prefill_impl(p, n, q, k, v, stride_b, stride_h, stride_t, nullptr, out, scores, kept_idx,
                        lse_opt, workspace, workspace_bytes, cuda_stream);
}

// workspace of the grouped prefill: lse rows and per-query-head scores [B][H*G][n], then the
// tensor-core pass's own extra (the fp16 copy of the B*H K/V heads' V)
static size_t group_ws_bytes(const a2sf_params *p, int G, int n)
{
    const size_t rows = align_up((size_t)p->B * p->H * G * n * sizeof(float));
    return 2 * rows + prefill_tc_extra_bytes(p->dtype, (size_t)p->B * p->H, n, p->d);
}

size_t a2sf_prefill_group_workspace_bytes(const a2sf_params *p, int32_t group, int32_t n)
{
    if (check_params(p) != A2SF_OK || n < 1 || group < 1 || group > A2SF_MAX_GROUP) return 0;
    return group_ws_bytes(p, group, n);
}

int a2sf_prefill_group(const a2sf_params *p, int32_t group, int32_t n, const void *q, int64_t q_stride_b,
                       int64_t q_stride_h, int64_t q_stride_t, const void *k, const void *v,
                       int64_t kv_stride_b, int64_t kv_stride_h, int64_t kv_stride_t, void *out,
                       float *scores, int32_t *kept_idx, float *lse_opt, void *workspace,
                       size_t workspace_bytes, void *cuda_stream)
{
    A2SF_TRACE("a2sf_prefill_group");
    int rc = check_params(p);
    if (rc != A2SF_OK) return rc;
    if (group < 1 || group > A2SF_MAX_GROUP) return A2SF_ERR_UNSUPPORTED;
    if (p->score_window != 0 || p->flags != 0) return A2SF_ERR_UNSUPPORTED;
    if (n < 1 || !q || !k || !v || !out || !scores || !kept_idx) return A2SF_ERR_INVALID_ARG;
    if ((rc = check_strides(p, q_stride_b, q_stride_h, q_stride_t)) != A2SF_OK) return rc;
    if ((rc = check_strides(p, kv_stride_b, kv_stride_h, kv_stride_t)) != A2SF_OK) return rc;
    if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(out, 16) ||
        !aligned(scores, 4) || !aligned(kept_idx, 4))
        return A2SF_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256)) return A2SF_ERR_INVALID_ARG;
    if (workspace_bytes < group_ws_bytes(p, group, n)) return A2SF_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t rows = align_up((size_t)p->B * p->H * group * n * sizeof(float));
    char *ws = static_cast<char *>(workspace);

    PrefillArgs a;
    a.q = q; a.k = k; a.v = v; a.out = out;
    a.lse = lse_opt ? lse_opt : reinterpret_cast<float *>(ws);
    a.scores = reinterpret_cast<float *>(ws + rows);              // one row per QUERY head
    a.st = Strides{q_stride_b, q_stride_h, q_stride_t};
    a.st_kv = Strides{kv_stride_b, kv_stride_h, kv_stride_t};
    a.G = group;
    a.B = p->B; a.H = p->H * group; a.n = n; a.d = p->d;
    a.scale = eff_scale(p); a.alpha = p->alpha; a.alpha_vec = nullptr;
    a.skip_zero_rows = 0; a.window_rows = 0;
    a.v_half = nullptr; a.v_flag = nullptr;
    if (prefill_tc_extra_bytes(p->dtype, (size_t)p->B * p->H, n, p->d) > 0) {
        a.v_flag = reinterpret_cast<int *>(ws + 2 * rows);
        a.v_half = ws + 2 * rows + 256;
    }
    const bool tc = prefill_tc_supported(p->dtype, a);
    if ((tc ? launch_prefill_pass1_tc(p->dtype, a, s) : launch_prefill_pass1_simt(p->dtype, a, s)) != cudaSuccess)
        return A2SF_ERR_CUDA;
    if ((tc ? launch_prefill_pass2_tc(p->dtype, a, s) : launch_prefill_pass2_simt(p->dtype, a, s)) != cudaSuccess)
        return A2SF_ERR_CUDA;
    if (launch_group_sum(a.scores, scores, group, n, (size_t)p->B * p->H, s) != cudaSuccess)
        return A2SF_ERR_CUDA;
    if (launch_select(scores, kept_idx, p->B * p->H, n, p->budget, p->recent, s) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return A2SF_OK;
}

int a2sf_prefill_per_head(const a2sf_params *p, int32_t n, const void *q, const void *k, const void *v,
                          int64_t stride_b, int64_t stride_h, int64_t stride_t, const float *alphas,
                          void *out, float *scores, int32_t *kept_idx, float *lse_opt,
                          void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!alphas || !aligned(alphas, 4)) return A2SF_ERR_INVALID_ARG;
    return prefill_impl(p, n, q, k, v, stride_b, stride_h, stride_t, alphas, out, scores, kept_idx,
                        lse_opt, workspace, workspace_bytes, cuda_stream);
}

static int rescore_impl(const a2sf_params *p, int32_t n, const void *q, const void *k, int64_t stride_b,
                        int64_t stride_h, int64_t stride_t, const float *lse, const float *alpha_vec,
                        float *scores, int32_t *kept_idx, void *workspace, size_t workspace_bytes,
                        void *cuda_stream)
{
    A2SF_TRACE("a2sf_rescore");
    (void)workspace; (void)workspace_bytes;
    int rc = check_params(p);
    if (rc != A2SF_OK) return rc;
    if (n < 1 || !q || !k || !lse || !scores || !kept_idx) return A2SF_ERR_INVALID_ARG;
    if ((rc = check_strides(p, stride_b, stride_h, stride_t)) != A2SF_OK) return rc;
    if (!aligned(q, 16) || !aligned(k, 16)) return A2SF_ERR_INVALID_ARG;
    PrefillArgs a;
    a.q = q; a.k = k; a.v = nullptr; a.out = nullptr;
    a.lse = const_cast<float *>(lse);
    a.scores = scores;
    a.st = Strides{stride_b, stride_h, stride_t};
    a.st_kv = a.st; a.G = 1;
    a.B = p->B; a.H = p->H; a.n = n; a.d = p->d;
    a.scale = eff_scale(p); a.alpha = p->alpha; a.alpha_vec = alpha_vec;
    a.skip_zero_rows = (p->flags & A2SF_FLAG_SKIP_ZERO_WEIGHT_ROWS) ? 1 : 0;
    a.window_rows = p->score_window;
    a.v_half = nullptr; a.v_flag = nullptr;
    return run_scores_and_select(p, n, a, kept_idx, static_cast<cudaStream_t>(cuda_stream));
}

int a2sf_rescore(const a2sf_params *p, int32_t n, const void *q, const void *k, int64_t stride_b,
                 int64_t stride_h, int64_t stride_t, const float *lse, float *scores,
                 int32_t *kept_idx, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    return rescore_impl(p, n, q, k, stride_b, stride_h, stride_t, lse, nullptr, scores, kept_idx,
                        workspace, workspace_bytes, cuda_stream);
}

int a2sf_rescore_per_head(const a2sf_params *p, int32_t n, const void *q, const void *k,
                          int64_t stride_b, int64_t stride_h, int64_t stride_t, const float *lse,
                          const float *alphas, float *scores, int32_t *kept_idx, void *workspace,
                          size_t workspace_bytes, void *cuda_stream)
{
    if (!alphas || !aligned(alphas, 4)) return A2SF_ERR_INVALID_ARG;
    return rescore_impl(p, n, q, k, stride_b, stride_h, stride_t, lse, alphas, scores, kept_idx,
                        workspace, workspace_bytes, cuda_stream);
}

int a2sf_select(const a2sf_params *p, int32_t n, const float *scores, int32_t *kept_idx, void *cuda_stream)
{
    A2SF_TRACE("a2sf_select");
    int rc = check_params(p);
    if (rc != A2SF_OK) return rc;
    if (n < 1 || !scores || !kept_idx || !aligned(scores, 4) || !aligned(kept_idx, 4)) return A2SF_ERR_INVALID_ARG;
    if (launch_select(scores, kept_idx, p->B * p->H, n, p->budget, p->recent,
                      static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return A2SF_OK;
}

size_t a2sf_prefill_host_workspace_bytes(const a2sf_params *p, int32_t n)
{
    if (check_params(p) != A2SF_OK || n < 1) return 0;
    const size_t U = (size_t)p->B * p->H;
    const size_t tensor = align_up(U * n * p->d * elem_bytes(p->dtype));
    const size_t m = (size_t)(n < p->budget ? n : p->budget);
    return 4 * tensor + align_up(U * n * 4) + align_up(U * m * 4) + prefill_ws_bytes(p, n);
}

int a2sf_prefill_host(const a2sf_params *p, int32_t n, const void *q_host, const void *k_host,
                      const void *v_host, void *out_host, float *scores_host,
                      int32_t *kept_idx_host, void *workspace, size_t workspace_bytes,
                      void **dev_k, void **dev_v, float **dev_scores, int32_t **dev_kept,
                      void *cuda_stream)
{
    A2SF_TRACE("a2sf_prefill_host");
    int rc = check_params(p);
    if (rc != A2SF_OK) return rc;
    if (n < 1 || !q_host || !k_host || !v_host || !out_host || !scores_host || !kept_idx_host)
        return A2SF_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256)) return A2SF_ERR_INVALID_ARG;
    if (workspace_bytes < a2sf_prefill_host_workspace_bytes(p, n)) return A2SF_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t U = (size_t)p->B * p->H;
    const size_t tbytes = U * n * p->d * elem_bytes(p->dtype);
    const size_t tensor = align_up(tbytes);
    const size_t m = (size_t)(n < p->budget ? n : p->budget);
    char *base = static_cast<char *>(workspace);
    void *dq = base, *dk = base + tensor, *dv = base + 2 * tensor, *dout = base + 3 * tensor;
    float *dsc = reinterpret_cast<float *>(base + 4 * tensor);
    int32_t *dkept = reinterpret_cast<int32_t *>(base + 4 * tensor + align_up(U * n * 4));
    void *inner = base + 4 * tensor + align_up(U * n * 4) + align_up(U * m * 4);

    const int64_t st = p->d, sh = (int64_t)n * p->d, sb = (int64_t)p->H * n * p->d;
    // Batch rows are independent, so the call is pipelined over chunks of them on two internal
    // streams: while one chunk computes and its results travel back, the next chunk's inputs
    // are already on their way in (the two copy directions and the kernels overlap).
    const int chunks = p->B >= 2 ? (p->B < 8 ? p->B : 8) : 1;
    if (chunks == 1) {
        if (cudaMemcpyAsync(dq, q_host, tbytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
            cudaMemcpyAsync(dk, k_host, tbytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
            cudaMemcpyAsync(dv, v_host, tbytes, cudaMemcpyHostToDevice, s) != cudaSuccess)
            return A2SF_ERR_CUDA;
        rc = a2sf_prefill(p, n, dq, dk, dv, sb, sh, st, dout, dsc, dkept, nullptr, inner,
                          prefill_ws_bytes(p, n), cuda_stream);
        if (rc != A2SF_OK) return rc;
        if (cudaMemcpyAsync(out_host, dout, tbytes, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaMemcpyAsync(scores_host, dsc, U * n * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaMemcpyAsync(kept_idx_host, dkept, U * m * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return A2SF_ERR_CUDA;
        if (cudaStreamSynchronize(s) != cudaSuccess) return A2SF_ERR_CUDA;
    } else {
        HostPipeline *hp = host_pipeline();
        if (!hp->ok) return A2SF_ERR_CUDA;
        std::lock_guard<std::mutex> pipeline_lock(hp->mu);
        cudaStream_t *side = hp->side;
        cudaEvent_t start = hp->start, *done = hp->done;
        // work already queued on the caller's stream comes first
        bool ok = cudaEventRecord(start, s) == cudaSuccess;
        for (int x = 0; ok && x < 2; ++x) ok = cudaStreamWaitEvent(side[x], start, 0) == cudaSuccess;
        const size_t eb = elem_bytes(p->dtype);
        const int rows_per = (p->B + chunks - 1) / chunks;
        a2sf_params pc = *p;
        pc.B = rows_per;
        const size_t inner_half = align_up(prefill_ws_bytes(&pc, n));     // two of them fit: rows_per <= B/2 rounded up
        const bool two_inner = 2 * inner_half <= prefill_ws_bytes(p, n);
        int rc2 = A2SF_OK;
        for (int c = 0; ok && rc2 == A2SF_OK && c * rows_per < p->B; ++c) {
            const int b0 = c * rows_per, nb = (b0 + rows_per <= p->B) ? rows_per : p->B - b0;
            // without room for two inner workspaces the chunks' kernels share one stream
            cudaStream_t cs = side[two_inner ? (c & 1) : 0];
            const size_t ub = (size_t)b0 * p->H, un = (size_t)nb * p->H;
            const size_t off = ub * n * p->d * eb, len = un * n * p->d * eb;
            ok = cudaMemcpyAsync((char *)dq + off, (const char *)q_host + off, len, cudaMemcpyHostToDevice, cs) == cudaSuccess &&
                 cudaMemcpyAsync((char *)dk + off, (const char *)k_host + off, len, cudaMemcpyHostToDevice, cs) == cudaSuccess &&
                 cudaMemcpyAsync((char *)dv + off, (const char *)v_host + off, len, cudaMemcpyHostToDevice, cs) == cudaSuccess;
            if (!ok) break;
            pc.B = nb;
            rc2 = a2sf_prefill(&pc, n, (char *)dq + off, (char *)dk + off, (char *)dv + off, sb, sh, st,
                               (char *)dout + off, dsc + ub * n, dkept + ub * m, nullptr,
                               (char *)inner + ((two_inner && (c & 1)) ? inner_half : 0), inner_half, cs);
            if (rc2 != A2SF_OK) break;
            ok = cudaMemcpyAsync((char *)out_host + off, (char *)dout + off, len, cudaMemcpyDeviceToHost, cs) == cudaSuccess &&
                 cudaMemcpyAsync(scores_host + ub * n, dsc + ub * n, un * n * 4, cudaMemcpyDeviceToHost, cs) == cudaSuccess &&
                 cudaMemcpyAsync(kept_idx_host + ub * m, dkept + ub * m, un * m * 4, cudaMemcpyDeviceToHost, cs) == cudaSuccess;
        }
        // the caller's stream continues only after both side streams have drained
        for (int x = 0; x < 2; ++x)
            if (cudaEventRecord(done[x], side[x]) != cudaSuccess || cudaStreamWaitEvent(s, done[x], 0) != cudaSuccess)
                ok = false;
        const bool drained = cudaStreamSynchronize(s) == cudaSuccess;
        if (!ok)                                   // a failed fork or join: leave nothing running behind
            for (int x = 0; x < 2; ++x) cudaStreamSynchronize(side[x]);
        if (rc2 != A2SF_OK) return rc2;
        if (!ok || !drained) return A2SF_ERR_CUDA;
    }
    if (dev_k) *dev_k = dk;
    if (dev_v) *dev_v = dv;
    if (dev_scores) *dev_scores = dsc;
    if (dev_kept) *dev_kept = dkept;
    return A2SF_OK;
}

// ---- cache object --------------------------------------------------------------

struct CacheLayout {
    size_t K, V, S, pos, count, len, sched, st_q, st_k, st_v, st_out, st_ev, total;
};

static CacheLayout cache_layout(const a2sf_params *p)
{
    const size_t U = (size_t)p->B * p->H, M = p->budget, d = p->d, e = elem_bytes(p->dtype);
    CacheLayout L;
    size_t off = 0;
    L.K = off; off += align_up(U * M * d * e);
    L.V = off; off += align_up(U * M * d * e);
    L.S = off; off += align_up(U * M * 4);
    L.pos = off; off += align_up(U * M * 4);
    L.count = off; off += align_up(U * 4);
    L.len = off; off += align_up(U * 4);
    L.sched = off; off += align_up(2 * 4);
    L.st_q = off; off += align_up(U * d * e);
    L.st_k = off; off += align_up(U * d * e);
    L.st_v = off; off += align_up(U * d * e);
    L.st_out = off; off += align_up(U * d * e);
    L.st_ev = off; off += align_up(U * 4);
    L.total = off;
    return L;
}

size_t a2sf_cache_bytes(const a2sf_params *p)
{
    if (check_params(p) != A2SF_OK) return 0;
    return cache_layout(p).total;
}

int a2sf_cache_create(const a2sf_params *p, void *device_mem, size_t bytes, a2sf_cache **cache)
{
    int rc = check_params(p);
    if (rc != A2SF_OK) return rc;
    if (!cache) return A2SF_ERR_INVALID_ARG;
    *cache = nullptr;
    const CacheLayout L = cache_layout(p);
    a2sf_cache *c = new (std::nothrow) a2sf_cache;
    if (!c) return A2SF_ERR_CUDA;
    c->p = *p;
    c->owns = device_mem == nullptr;
    if (device_mem) {
        if (!aligned(device_mem, 256)) { delete c; return A2SF_ERR_INVALID_ARG; }
        if (bytes < L.total) { delete c; return A2SF_ERR_WORKSPACE; }
        c->mem = device_mem;
    } else if (cudaMalloc(&c->mem, L.total) != cudaSuccess) {
        delete c;
        return A2SF_ERR_CUDA;
    }
    c->bytes = L.total;
    char *b = static_cast<char *>(c->mem);
    c->view.K = b + L.K; c->view.V = b + L.V;
    c->view.S = reinterpret_cast<float *>(b + L.S);
    c->view.pos = reinterpret_cast<int32_t *>(b + L.pos);
    c->view.count = reinterpret_cast<int32_t *>(b + L.count);
    c->view.len = reinterpret_cast<int32_t *>(b + L.len);
    c->view.sched = reinterpret_cast<int32_t *>(b + L.sched);
    c->view.U = p->B * p->H; c->view.M = p->budget; c->view.R = p->recent;
    c->view.d = p->d; c->view.dtype = p->dtype; c->view.scale = eff_scale(p);
    c->view.io_H = p->H; c->view.io_st_b = (long long)p->H * p->d; c->view.io_st_h = p->d;
    c->st_q = b + L.st_q; c->st_k = b + L.st_k; c->st_v = b + L.st_v; c->st_out = b + L.st_out;
    c->st_ev = reinterpret_cast<int32_t *>(b + L.st_ev);
    // empty cache: zero scores and counters, positions -1
    if (cudaMemset(b + L.S, 0, L.st_q - L.S) != cudaSuccess ||
        cudaMemset(b + L.pos, 0xff, L.count - L.pos) != cudaSuccess ||
        cudaDeviceSynchronize() != cudaSuccess) {
        if (c->owns) cudaFree(c->mem);
        delete c;
        return A2SF_ERR_CUDA;
    }
    *cache = c;
    return A2SF_OK;
}

int a2sf_cache_destroy(a2sf_cache *cache)
{
    if (!cache) return A2SF_ERR_INVALID_ARG;
    int rc = A2SF_OK;
    if (cache->owns && cudaFree(cache->mem) != cudaSuccess) rc = A2SF_ERR_CUDA;
    delete cache;
    return rc;
}

int a2sf_cache_load(a2sf_cache *cache, int32_t n, const void *k, const void *v, int64_t stride_b,
                    int64_t stride_h, int64_t stride_t, const float *scores,
                    const int32_t *kept_idx, void *cuda_stream)
{
    A2SF_TRACE("a2sf_cache_load");
    if (!cache || n < 1 || !k || !v || !scores || !kept_idx) return A2SF_ERR_INVALID_ARG;
    int rc = check_strides(&cache->p, stride_b, stride_h, stride_t);
    if (rc != A2SF_OK) return rc;
    if (!aligned(k, 16) || !aligned(v, 16)) return A2SF_ERR_INVALID_ARG;
    if (launch_cache_load(cache->view, cache->p.H, n, k, v, Strides{stride_b, stride_h, stride_t},
                          scores, kept_idx, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return A2SF_OK;
}

int a2sf_decode_step(a2sf_cache *cache, float alpha, const void *q, const void *k_new,
                     const void *v_new, void *out, int32_t *evicted_slot, void *cuda_stream)
{
    A2SF_TRACE("a2sf_decode_step");
    if (!cache || !q || !k_new || !v_new || !out || !evicted_slot) return A2SF_ERR_INVALID_ARG;
    if (!(alpha >= 0.f && alpha <= 1.f)) return A2SF_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(k_new, 16) || !aligned(v_new, 16) || !aligned(out, 16))
        return A2SF_ERR_INVALID_ARG;
    if (launch_decode_step(cache->view, alpha, nullptr, q, k_new, v_new, out, evicted_slot,
                           static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return A2SF_OK;
}

double a2sf_score_window_bound(float alpha, int32_t n, int32_t score_window)
{
    if (score_window <= 0 || score_window >= n || !(alpha >= 0.f && alpha <= 1.f)) return 0.0;
    const double a = alpha;
    if (a >= 1.0) return (double)(n - score_window);
    return std::pow(a, (double)score_window) * (1.0 - std::pow(a, (double)(n - score_window))) / (1.0 - a);
}

int a2sf_cache_reset(a2sf_cache *cache, void *cuda_stream)
{
    if (!cache) return A2SF_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const CacheView &c = cache->view;
    const size_t U = c.U, M = c.M;
    if (cudaMemsetAsync(c.S, 0, U * M * 4, s) != cudaSuccess ||
        cudaMemsetAsync(c.pos, 0xff, U * M * 4, s) != cudaSuccess ||
        cudaMemsetAsync(c.count, 0, U * 4, s) != cudaSuccess ||
        cudaMemsetAsync(c.len, 0, U * 4, s) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return A2SF_OK;
}

int a2sf_decode_multi(a2sf_cache *cache, float alpha, int32_t steps, const void *q, const void *k_new,
                      const void *v_new, int64_t stride_b, int64_t stride_h, int64_t stride_t,
                      void *out, int32_t *evicted_opt, void *cuda_stream)
{
    A2SF_TRACE("a2sf_decode_multi");
    if (!cache || steps < 1 || !q || !k_new || !v_new || !out) return A2SF_ERR_INVALID_ARG;
    if (!(alpha >= 0.f && alpha <= 1.f)) return A2SF_ERR_INVALID_ARG;
    int rc = check_strides(&cache->p, stride_b, stride_h, stride_t);
    if (rc != A2SF_OK) return rc;
    if (!aligned(q, 16) || !aligned(k_new, 16) || !aligned(v_new, 16) || !aligned(out, 16))
        return A2SF_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    CacheView view = cache->view;
    view.io_st_b = stride_b;
    view.io_st_h = stride_h;
    const size_t eb = elem_bytes(cache->p.dtype), U = view.U;
    for (int32_t i = 0; i < steps; ++i) {
        const size_t off = (size_t)i * (size_t)stride_t * eb;
        int32_t *ev = evicted_opt ? evicted_opt + (size_t)i * U : cache->st_ev;
        if (launch_decode_step(view, alpha, nullptr, static_cast<const char *>(q) + off,
                               static_cast<const char *>(k_new) + off,
                               static_cast<const char *>(v_new) + off,
                               static_cast<char *>(out) + off, ev, s) != cudaSuccess)
            return A2SF_ERR_CUDA;
    }
    return A2SF_OK;
}

int a2sf_prefill_streaming(a2sf_cache *cache, float alpha, int32_t n, const void *q, const void *k,
                           const void *v, int64_t stride_b, int64_t stride_h, int64_t stride_t,
                           void *out, int32_t *evicted_opt, void *cuda_stream)
{
    A2SF_TRACE("a2sf_prefill_streaming");
    if (!cache || n < 1 || !q || !k || !v || !out) return A2SF_ERR_INVALID_ARG;
    if (!(alpha >= 0.f && alpha <= 1.f)) return A2SF_ERR_INVALID_ARG;
    int rc = check_strides(&cache->p, stride_b, stride_h, stride_t);
    if (rc != A2SF_OK) return rc;
    if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(out, 16))
        return A2SF_ERR_INVALID_ARG;
    rc = a2sf_cache_reset(cache, cuda_stream);
    if (rc != A2SF_OK) return rc;
    return a2sf_decode_multi(cache, alpha, n, q, k, v, stride_b, stride_h, stride_t, out, evicted_opt,
                             cuda_stream);
}

size_t a2sf_ideal_similarity_workspace_bytes(const a2sf_params *p, int32_t n)
{
    if (check_params(p) != A2SF_OK || n < 1 || n > A2SF_IDEAL_SIMILARITY_MAX_N) return 0;
    return align_up(ideal_similarity_ws_bytes((size_t)p->B * p->H, n));
}

int a2sf_ideal_similarity(a2sf_cache *cache, float alpha, int32_t n, const void *q, const void *k,
                          const void *v, int64_t stride_b, int64_t stride_h, int64_t stride_t,
                          void *out, float *cos_out, int32_t *evicted_opt, void *workspace,
                          size_t workspace_bytes, void *cuda_stream)
{
    A2SF_TRACE("a2sf_ideal_similarity");
    if (!cache || n < 1 || !q || !k || !v || !out || !cos_out) return A2SF_ERR_INVALID_ARG;
    if (n > A2SF_IDEAL_SIMILARITY_MAX_N) return A2SF_ERR_UNSUPPORTED;
    if (!(alpha >= 0.f && alpha <= 1.f)) return A2SF_ERR_INVALID_ARG;
    int rc = check_strides(&cache->p, stride_b, stride_h, stride_t);
    if (rc != A2SF_OK) return rc;
    if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(out, 16) || !aligned(cos_out, 4))
        return A2SF_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256)) return A2SF_ERR_INVALID_ARG;
    if (workspace_bytes < a2sf_ideal_similarity_workspace_bytes(&cache->p, n)) return A2SF_ERR_WORKSPACE;
    rc = a2sf_cache_reset(cache, cuda_stream);
    if (rc != A2SF_OK) return rc;
    if (launch_ideal_similarity(cache->view, alpha, cache->p.H, n, q, k, v,
                                Strides{stride_b, stride_h, stride_t}, out, cos_out, evicted_opt,
                                cache->st_ev, workspace, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return A2SF_OK;
}

int a2sf_decode_step_group(a2sf_cache *cache, int32_t group, float alpha, const void *q, const void *k_new,
                           const void *v_new, void *out, int32_t *evicted_slot, void *cuda_stream)
{
    A2SF_TRACE("a2sf_decode_step_group");
    if (!cache || !q || !k_new || !v_new || !out || !evicted_slot) return A2SF_ERR_INVALID_ARG;
    if (group < 1 || group > A2SF_MAX_GROUP) return A2SF_ERR_UNSUPPORTED;
    if (decode_group_smem_bytes(cache->view.M, group, cache->view.d) > 220 * 1024) return A2SF_ERR_UNSUPPORTED;
    if (!(alpha >= 0.f && alpha <= 1.f)) return A2SF_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(k_new, 16) || !aligned(v_new, 16) || !aligned(out, 16))
        return A2SF_ERR_INVALID_ARG;
    if (launch_decode_step_group(cache->view, group, alpha, q, k_new, v_new, out, evicted_slot,
                                 static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return A2SF_OK;
}

int a2sf_decode_step_per_head(a2sf_cache *cache, const float *alphas, const void *q,
                              const void *k_new, const void *v_new, void *out,
                              int32_t *evicted_slot, void *cuda_stream)
{
    A2SF_TRACE("a2sf_decode_step_per_head");
    if (!cache || !alphas || !q || !k_new || !v_new || !out || !evicted_slot)
        return A2SF_ERR_INVALID_ARG;
    if (!aligned(alphas, 4) || !aligned(q, 16) || !aligned(k_new, 16) || !aligned(v_new, 16) ||
        !aligned(out, 16))
        return A2SF_ERR_INVALID_ARG;
    if (launch_decode_step(cache->view, cache->p.alpha, alphas, q, k_new, v_new, out, evicted_slot,
                           static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return A2SF_OK;
}

// Device-side address of a pinned (page-locked, mapped) host buffer, or nullptr for anything
// else (pageable memory, device memory, misaligned rows).
static void *mapped_host_pointer(const void *host)
{
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
        cudaGetLastError();                       // older drivers report pageable memory as an error
        return nullptr;
    }
    if (at.type != cudaMemoryTypeHost || !at.devicePointer || !aligned(at.devicePointer, 16)) return nullptr;
    return at.devicePointer;
}

int a2sf_decode_step_host(a2sf_cache *cache, float alpha, const void *q_host,
                          const void *k_new_host, const void *v_new_host, void *out_host,
                          int32_t *evicted_slot_host, void *cuda_stream)
{
    A2SF_TRACE("a2sf_decode_step_host");
    if (!cache || !q_host || !k_new_host || !v_new_host || !out_host || !evicted_slot_host)
        return A2SF_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    // Pinned buffers are read and written by the step kernel itself, over the bus, while it
    // streams the cache from device memory: five copies and their latencies less per step
    // (about 1.3 KB per unit against the 270 KB of cache the same unit reads).
    {
        void *dq = mapped_host_pointer(q_host), *dk = mapped_host_pointer(k_new_host),
             *dv = mapped_host_pointer(v_new_host), *dout = mapped_host_pointer(out_host),
             *dev = mapped_host_pointer(evicted_slot_host);
        if (dq && dk && dv && dout && dev) {
            const int rc = a2sf_decode_step(cache, alpha, dq, dk, dv, dout, static_cast<int32_t *>(dev),
                                            cuda_stream);
            if (rc != A2SF_OK) return rc;
            return cudaStreamSynchronize(s) == cudaSuccess ? A2SF_OK : A2SF_ERR_CUDA;
        }
    }
    const size_t U = cache->view.U;
    const size_t row = U * cache->p.d * elem_bytes(cache->p.dtype);
    if (cudaMemcpyAsync(cache->st_q, q_host, row, cudaMemcpyHostToDevice, s) != cudaSuccess ||
        cudaMemcpyAsync(cache->st_k, k_new_host, row, cudaMemcpyHostToDevice, s) != cudaSuccess ||
        cudaMemcpyAsync(cache->st_v, v_new_host, row, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return A2SF_ERR_CUDA;
    int rc = a2sf_decode_step(cache, alpha, cache->st_q, cache->st_k, cache->st_v, cache->st_out,
                              cache->st_ev, cuda_stream);
    if (rc != A2SF_OK) return rc;
    if (cudaMemcpyAsync(out_host, cache->st_out, row, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemcpyAsync(evicted_slot_host, cache->st_ev, U * 4, cudaMemcpyDeviceToHost, s) !=
            cudaSuccess)
        return A2SF_ERR_CUDA;
    return cudaStreamSynchronize(s) == cudaSuccess ? A2SF_OK : A2SF_ERR_CUDA;
}

static int copy_part(void *dst, const void *src, size_t bytes, cudaStream_t s)
{
    if (!dst || !src) return A2SF_OK;
    return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, s) == cudaSuccess
               ? A2SF_OK : A2SF_ERR_CUDA;
}

int a2sf_cache_export(const a2sf_cache *cache, void *k, void *v, float *scores, int32_t *pos,
                      int32_t *count, int32_t *len, void *cuda_stream)
{
    A2SF_TRACE("a2sf_cache_export");
    if (!cache) return A2SF_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const CacheView &c = cache->view;
    const size_t U = c.U, M = c.M, rows = U * M * c.d * elem_bytes(c.dtype);
    int rc = copy_part(k, c.K, rows, s);
    if (rc == A2SF_OK) rc = copy_part(v, c.V, rows, s);
    if (rc == A2SF_OK) rc = copy_part(scores, c.S, U * M * 4, s);
    if (rc == A2SF_OK) rc = copy_part(pos, c.pos, U * M * 4, s);
    if (rc == A2SF_OK) rc = copy_part(count, c.count, U * 4, s);
    if (rc == A2SF_OK) rc = copy_part(len, c.len, U * 4, s);
    return rc;
}

int a2sf_cache_import(a2sf_cache *cache, const void *k, const void *v, const float *scores,
                      const int32_t *pos, const int32_t *count, const int32_t *len,
                      void *cuda_stream)
{
    A2SF_TRACE("a2sf_cache_import");
    if (!cache) return A2SF_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const CacheView &c = cache->view;
    const size_t U = c.U, M = c.M, rows = U * M * c.d * elem_bytes(c.dtype);
    int rc = copy_part(c.K, k, rows, s);
    if (rc == A2SF_OK) rc = copy_part(c.V, v, rows, s);
    if (rc == A2SF_OK) rc = copy_part(c.S, scores, U * M * 4, s);
    if (rc == A2SF_OK) rc = copy_part(c.pos, pos, U * M * 4, s);
    if (rc == A2SF_OK) rc = copy_part(c.count, count, U * 4, s);
    if (rc == A2SF_OK) rc = copy_part(c.len, len, U * 4, s);
    return rc;
}

int64_t a2sf_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int a2sf_last_device_status(void *cuda_stream)
{
    const int a = read_and_clear_tc_status(static_cast<cudaStream_t>(cuda_stream));
    const int b = read_and_clear_decode_status(static_cast<cudaStream_t>(cuda_stream));
    return a != A2SF_OK ? a : b;
}

int a2sf_selftest_bounded_wait(int32_t which, int64_t limit_cycles, int64_t *report, void *cuda_stream)
{
    if ((which != 0 && which != 1) || !report || !aligned(report, 8)) return A2SF_ERR_INVALID_ARG;
    if (limit_cycles < 1 || limit_cycles > A2SF_SELFTEST_MAX_WAIT_CYCLES) return A2SF_ERR_INVALID_ARG;
    int *word = which == 0 ? tc_status_word() : decode_status_word();
    if (!word) return A2SF_ERR_CUDA;
    static_assert(sizeof(long long) == sizeof(int64_t), "report words");
    if (launch_wait_probe(word, (long long)limit_cycles, reinterpret_cast<long long *>(report),
                          static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return A2SF_OK;
}

int a2sf_debug_build(void)
{
#ifdef A2SF_DEBUG
    return 1;
#else
    return 0;
#endif
}

int a2sf_debug_violations(int64_t *report, void *cuda_stream)
{
    if (!report) return A2SF_ERR_INVALID_ARG;
    report[0] = report[1] = report[2] = report[3] = 0;
#ifdef A2SF_DEBUG
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    DebugReaders &r = debug_readers();
    for (int i = 0; i < r.n; ++i) {
        unsigned long long rec[4] = {0, 0, 0, 0};
        if (r.fn[i](rec, s) != 0) return A2SF_ERR_CUDA;
        if (rec[0] != 0 && report[0] == 0) {
            report[1] = (int64_t)rec[1]; report[2] = (int64_t)rec[2]; report[3] = (int64_t)rec[3];
        }
        report[0] += (int64_t)rec[0];
    }
#else
    (void)cuda_stream;
#endif
    return A2SF_OK;
}

const char *a2sf_status_string(int status)
{
    switch (status) {
    case A2SF_OK: return "ok";
    case A2SF_ERR_INVALID_ARG: return "invalid argument";
    case A2SF_ERR_UNSUPPORTED: return "unsupported dtype or head size";
    case A2SF_ERR_CUDA: return "CUDA runtime error";
    case A2SF_ERR_TIMEOUT: return "device-side wait timed out";
    case A2SF_ERR_WORKSPACE: return "workspace too small";
    default: return "unknown status";
    }
}

}  // extern "C"
