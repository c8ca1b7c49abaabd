// Fused A2SF generation step (one kernel): attention over the pruned, slot-indexed
// cache + the new token, score recurrence S <- alpha*S + a (paper Eq. 5 written as a
// recurrence), argmin eviction under (S, position) over the non-recent slots
// (Sec. 3.1, Sec. 4.1) and the in-place write of the new K/V row.
//
// Memory-bound: every K and V row of the head is read exactly once with 16-byte
// loads, lanes laid across the row so a warp reads whole 512-byte spans.
#include <cooperative_groups.h>

#include "common.cuh"
#include "tc_sm100.cuh"

namespace a2sf {

namespace cg = cooperative_groups;

A2SF_DEBUG_TRANSLATION_UNIT(decode_step)

// sticky device-side status of the decode kernels (a bounded wait that ran out)
static __device__ int g_decode_status = 0;

namespace {

constexpr int kDecodeThreads = 256;
constexpr int kSplitMinBudget = 512;         // split-K only pays for long caches

template <int NT>
__device__ __forceinline__ float block_max(float v, float *red)
{
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) r = fmaxf(r, red[w]);
    return r;
}

template <int NT>
__device__ __forceinline__ float block_sum(float v, float *red)
{
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) r += red[w];   // fixed order: run-to-run identical
    return r;
}

// ============================================================================================
// Split-K variant for few units with large budgets (flash-decoding): a thread-block cluster of
// C CTAs shares one unit, each CTA owning a contiguous slice of its slots.  Every CTA computes
// the logits, the local maximum, the local exponential sum and the unnormalised partial output
// of its slice; the partials meet in distributed shared memory: every CTA stores its (max, sum)
// pair into all CTAs' inboxes and its partial output into rank 0's, one cluster barrier later
// each CTA forms the global softmax constants from its own inbox and rank 0 combines the
// outputs; every CTA then updates the scores of its own slots, stores its local eviction
// candidate into rank 0's inbox, arrives at the second barrier and is done; rank 0 alone waits
// there, picks the global (score, position) minimum and writes the new token in place.
// A peer's shared memory may be written only once that CTA runs: every thread arrives at a
// first barrier when the kernel starts and waits for it just before its first remote store,
// by which time it has long completed.
// With C = 1 this is the plain one-CTA-per-unit kernel.
// ============================================================================================
constexpr int kMaxSplit = 8;       // CTAs per unit at most
// What the CTAs of a cluster hand to each other, indexed by the sender's rank.  Every CTA
// receives all (max, sum) pairs; only rank 0's copy of the rest is ever written.
struct SplitInbox {
    float m[kMaxSplit], l[kMaxSplit];          // local maximum and sum of exp(logit - m)
    unsigned long long best[kMaxSplit];        // local (bits(S) << 32 | position) minimum over evictable slots
    int best_slot[kMaxSplit];
    float out[kMaxSplit][128];                 // unnormalised partial outputs (relative to m)
};

__device__ __forceinline__ void cluster_arrive()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait()
{
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <typename T, int D, int NT>
__global__ void __launch_bounds__(NT, 2)
decode_step_split_kernel(CacheView c, float alpha_all, const float *__restrict__ alpha_vec,
                         const T *__restrict__ q, const T *__restrict__ k_new,
                         const T *__restrict__ v_new, T *__restrict__ out, int32_t *__restrict__ evicted)
{
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;          // lanes per row
    constexpr int RPW = 32 / LPR;         // rows per warp-wide load
    constexpr int NW = NT / 32;
    static_assert(LPR <= 32 && 32 % LPR == 0 && D <= 128, "row must fit a warp");

    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    cluster_arrive();                            // "this CTA runs": waited for before the first remote store

    extern __shared__ float smem[];
    const int M = c.M;
    const int per_max = (M + C - 1) / C;
    float *w = smem;                             // [per_max+1] logits, then exp(logit - max)
    float *part = w + ((per_max + 1 + 3) & ~3);  // [NW][D] partial outputs
    float *red = part + NW * D;                  // [NW] reduction scratch
    __shared__ SplitInbox inbox;
    __shared__ unsigned long long red_key[NW];
    __shared__ int red_slot[NW];
    __shared__ int s_target;

    const int u = blockIdx.x / C;
    const size_t uo = io_offset(c, u);           // this unit's row of q, k_new, v_new, out
    const float alpha = unit_alpha(alpha_vec, u, alpha_all);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, rsel = lane / LPR;
    const int cnt = min(c.count[u], M);
    const int p = c.len[u];
    // this CTA's slice of the resident slots; rank 0 also owns the new token (local index nloc)
    const int per = (cnt + C - 1) / C;
    const int s0 = min(cnt, rank * per), s1 = min(cnt, s0 + per);
    const int nloc = s1 - s0;
    const int nsoft = nloc + (rank == 0 ? 1 : 0);

    T *Ku = reinterpret_cast<T *>(c.K) + (size_t)u * M * D;
    T *Vu = reinterpret_cast<T *>(c.V) + (size_t)u * M * D;
    float *Su = c.S + (size_t)u * M;
    int32_t *posu = c.pos + (size_t)u * M;

    float qf[VEC];
    Elem<T>::unpack(*reinterpret_cast<const uint4 *>(q + uo + sub * VEC), qf);

    // The step is a chain of dependent phases around little data per CTA, so every global word is
    // requested as early as it can be.  Rows move in batches of kBatchRows per CTA through two
    // register buffers: two batches are in flight at any time, the first two batches of V are
    // requested as soon as the last K batches have been consumed (they travel while the CTA sits
    // in the softmax reductions), and this thread's scores and positions are requested here.
    constexpr int kU = 8;                         // 16-byte loads per lane and batch
    constexpr int kBatchRows = NW * RPW * kU;
    constexpr int kPre = 2;                       // score/position words preloaded per thread
    float s_pre[kPre];
    int p_pre[kPre];
#pragma unroll
    for (int i = 0; i < kPre; ++i) {
        const int s = tid + i * NT;
        s_pre[i] = 0.f;
        p_pre[i] = 0;
        if (s < nloc) {
            s_pre[i] = Su[s0 + s];
            p_pre[i] = posu[s0 + s];
        }
    }
    const int nb = ((nloc + kBatchRows - 1) / kBatchRows + 1) & ~1;     // batches, padded to even
    auto load_batch = [&](uint4(&r)[kU], const T *base, int bidx) {
#pragma unroll
        for (int x = 0; x < kU; ++x) {
            const int row = ((bidx * kU + x) * NW + warp) * RPW + rsel;
            r[x] = make_uint4(0, 0, 0, 0);
            if (bidx < nb && row < nloc && A2SF_IN_RANGE(s0 + row, M, kDbgDecodeSplit))
                r[x] = ld_stream16_rw(base + (size_t)(s0 + row) * D + sub * VEC);
        }
    };
    // batch index b: K batch b for b < nb, V batch b - nb after that
    auto load_next = [&](uint4(&r)[kU], int b) {
        if (b < nb) load_batch(r, Ku, b);
        else load_batch(r, Vu, b - nb);
    };
    uint4 ra[kU], rb[kU];
    load_batch(ra, Ku, 0);
    load_batch(rb, Ku, 1);

    // ---- (i) logits of the slice, and (rank 0) of the new key ---------------------------------
    auto logits_of = [&](const uint4(&r)[kU], int bidx) {
#pragma unroll
        for (int x = 0; x < kU; ++x) {
            const int row = ((bidx * kU + x) * NW + warp) * RPW + rsel;
            float kf[VEC];
            Elem<T>::unpack(r[x], kf);
            float dot = 0.f;
#pragma unroll
            for (int e = 0; e < VEC; ++e) dot = fmaf(qf[e], kf[e], dot);
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
            if (sub == 0 && row < nloc && A2SF_IN_RANGE(row, per_max + 1, kDbgDecodeSplit)) w[row] = dot * c.scale;
        }
    };
    for (int b = 0; b < nb; b += 2) {
        logits_of(ra, b);
        load_next(ra, b + 2);
        logits_of(rb, b + 1);
        load_next(rb, b + 3);
    }
    if (warp == 0 && rank == 0) {
        float kf[VEC];
        Elem<T>::unpack(*reinterpret_cast<const uint4 *>(k_new + uo + sub * VEC), kf);
        float dot = 0.f;
#pragma unroll
        for (int e = 0; e < VEC; ++e) dot = fmaf(qf[e], kf[e], dot);
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        if (lane == 0 && A2SF_IN_RANGE(nloc, per_max + 1, kDbgDecodeSplit)) w[nloc] = dot * c.scale;
    }
    __syncthreads();

    // ---- (ii) local softmax statistics ----------------------------------------------------------
    float m_loc = -INFINITY;
    for (int s = tid; s < nsoft; s += NT) m_loc = fmaxf(m_loc, w[s]);
    m_loc = block_max<NT>(m_loc, red);
    float l_loc = 0.f;
    for (int s = tid; s < nsoft; s += NT) {
        const float e = expf(w[s] - m_loc);
        w[s] = e;
        l_loc += e;
    }
    l_loc = block_sum<NT>(l_loc, red);

    // ---- (iii) unnormalised partial output of the slice -----------------------------------------
    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
    auto accumulate = [&](const uint4(&r)[kU], int bidx) {
#pragma unroll
        for (int x = 0; x < kU; ++x) {
            const int row = ((bidx * kU + x) * NW + warp) * RPW + rsel;
            const float ws = row < nloc ? w[row] : 0.f;
            float vf[VEC];
            Elem<T>::unpack(r[x], vf);
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[e] = fmaf(ws, vf[e], acc[e]);
        }
    };
    // V batches 0 and 1 are already in ra and rb (nb is even)
    for (int b = 0; b < nb; b += 2) {
        accumulate(ra, b);
        load_batch(ra, Vu, b + 2);
        accumulate(rb, b + 1);
        load_batch(rb, Vu, b + 3);
    }
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1)
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
    if (rsel == 0)
#pragma unroll
        for (int e = 0; e < VEC; ++e) part[warp * D + sub * VEC + e] = acc[e];
    __syncthreads();
    cluster_wait();                              // every CTA of the cluster runs
    if (tid < D) {
        float o = 0.f;
#pragma unroll
        for (int x = 0; x < NW; ++x) o += part[x * D + tid];
        if (rank == 0) o = fmaf(w[nloc], Elem<T>::to_float(v_new[uo + tid]), o);
        cluster.map_shared_rank(&inbox, 0)->out[rank][tid] = o;
    }
    if (tid < C) {
        SplitInbox *peer = cluster.map_shared_rank(&inbox, tid);
        peer->m[rank] = m_loc;
        peer->l[rank] = l_loc;
    }
    cluster_arrive();
    cluster_wait();

    // ---- global softmax constants from the (max, sum) pairs, in rank order ------------------------
    float m = -INFINITY;
    for (int r2 = 0; r2 < C; ++r2) m = fmaxf(m, inbox.m[r2]);
    float l = 0.f;
    for (int r2 = 0; r2 < C; ++r2) l += inbox.l[r2] * expf(inbox.m[r2] - m);   // an empty slice has m = -inf, l = 0
    if (rank == 0 && tid < D) {
        float o = 0.f;
        for (int r2 = 0; r2 < C; ++r2) o = fmaf(inbox.out[r2][tid], expf(inbox.m[r2] - m), o);
        out[uo + tid] = Elem<T>::from_float(o / l);
    }

    // ---- (iv) S <- alpha*S + a for the slice ; local eviction candidate ---------------------------
    const bool full = cnt >= M;
    const int newest_evictable = p - c.R;     // candidates: position <= p - R
    const float rescale = expf(m_loc - m);
    unsigned long long best = ~0ull;
    int best_slot = -1;
    auto update = [&](int s, float s_before, int ps) {
        const float a = w[s] * rescale / l;
        const float sn = fmaf(alpha, s_before, a);
        if (A2SF_IN_RANGE(s0 + s, M, kDbgDecodeSplit)) Su[s0 + s] = sn;
        if (full && ps <= newest_evictable) {
            // scores are >= 0, so their bit patterns order like the values
            const unsigned long long key =
                ((unsigned long long)__float_as_uint(sn) << 32) | (unsigned)ps;
            if (key < best) { best = key; best_slot = s0 + s; }
        }
    };
#pragma unroll
    for (int i = 0; i < kPre; ++i)
        if (tid + i * NT < nloc) update(tid + i * NT, s_pre[i], p_pre[i]);
    for (int s = tid + kPre * NT; s < nloc; s += NT) update(s, Su[s0 + s], posu[s0 + s]);
    // positions are distinct, so the minimum key identifies its slot
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int os = __shfl_xor_sync(0xffffffffu, best_slot, o);
        if (ob < best) { best = ob; best_slot = os; }
    }
    if (lane == 0) { red_key[warp] = best; red_slot[warp] = best_slot; }
    __syncthreads();
    if (tid == 0) {
        unsigned long long gb = red_key[0];
        int gs = red_slot[0];
        for (int x = 1; x < NW; ++x)
            if (red_key[x] < gb) { gb = red_key[x]; gs = red_slot[x]; }
        SplitInbox *root = cluster.map_shared_rank(&inbox, 0);
        root->best[rank] = gb;
        root->best_slot[rank] = gs;
    }
    cluster_arrive();
    if (rank != 0) return;                       // nobody reads this CTA's shared memory
    cluster_wait();

    // ---- (v) rank 0 picks the global minimum and inserts the new token in place -------------------
    const float a_self = w[nloc] * rescale / l;
    if (tid == 0) {
        int target = full ? -2 : cnt;
        if (full) {
            unsigned long long gb = ~0ull;
            int gs = -1;
            for (int r2 = 0; r2 < C; ++r2)
                if (inbox.best[r2] < gb) { gb = inbox.best[r2]; gs = inbox.best_slot[r2]; }
            const unsigned long long self_key =
                ((unsigned long long)__float_as_uint(a_self) << 32) | (unsigned)p;
            if (gs >= 0 && (c.R > 0 || gb < self_key)) target = gs;
        }
        s_target = target;
    }
    __syncthreads();
    const int target = s_target;
    const bool target_ok = target >= 0 && A2SF_IN_RANGE(target, M, kDbgDecodeSplit);
    if (target_ok) {
        if (tid < LPR)
            *reinterpret_cast<uint4 *>(Ku + (size_t)target * D + tid * VEC) =
                *reinterpret_cast<const uint4 *>(k_new + uo + tid * VEC);
        else if (tid < 2 * LPR)
            *reinterpret_cast<uint4 *>(Vu + (size_t)target * D + (tid - LPR) * VEC) =
                *reinterpret_cast<const uint4 *>(v_new + uo + (tid - LPR) * VEC);
    }
    if (tid == 0 && A2SF_IN_RANGE(u, c.U, kDbgDecodeSplit)) {
        if (target_ok) {
            Su[target] = a_self;
            posu[target] = p;
        }
        if (!full) c.count[u] = cnt + 1;
        c.len[u] = p + 1;
        evicted[u] = full ? target : -1;
    }
}


// ============================================================================================
// Streaming variant: persistent CTAs, K/V rows brought into a shared-memory ring by bulk
// asynchronous copies that a producer warp keeps issuing across phase and unit boundaries,
// so HBM requests stay in flight while the consumer warps sit in the softmax reductions or
// in the eviction epilogue of the previous head.
// ============================================================================================
constexpr int kStreamConsumerWarps = 8;
constexpr int kStreamConsumers = kStreamConsumerWarps * 32;
constexpr int kStreamThreads = kStreamConsumers + 32;
constexpr int kChunkBytes = 16384;
constexpr int kMaxStreamStages = 12;
constexpr int kStreamCtasPerSm = 3;          // measured best on config 4 (2: 63.8 us, 3: 60.5 us, 4: 68.6 us)
constexpr int kPrefetchSlots = 2;            // score/position words each consumer thread preloads

// The cache is streamed once per step and never re-read before the next step, by which time
// the rest of the cache has passed through L2: marking the copies evict-first keeps them from
// displacing one another's lines in flight (measured on config 4: 61.0 -> 55.7 us per step).
__device__ __forceinline__ uint64_t evict_first_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar,
                                          uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1], %2, [%3], %4;"
        :
        : "r"(tc::smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(tc::smem_u32(bar)), "l"(policy)
        : "memory");
}

__device__ __forceinline__ void consumer_barrier()
{
    tc::named_barrier(1, kStreamConsumers);
}

// barrier over the consumer warps that also ORs a predicate: every thread gets the same answer
__device__ __forceinline__ bool consumer_any(bool pred)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred), "r"(kStreamConsumers)
        : "memory");
    return r != 0;
}

__device__ __forceinline__ float consumer_max(float v, float *red)
{
    v = warp_max(v);
    consumer_barrier();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    consumer_barrier();
    float r = red[0];
#pragma unroll
    for (int w = 1; w < kStreamConsumerWarps; ++w) r = fmaxf(r, red[w]);
    return r;
}

__device__ __forceinline__ float consumer_sum(float v, float *red)
{
    v = warp_sum(v);
    consumer_barrier();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    consumer_barrier();
    float r = red[0];
#pragma unroll
    for (int w = 1; w < kStreamConsumerWarps; ++w) r += red[w];   // fixed order
    return r;
}

constexpr int kUnitQueue = 4;                // units the producer may run ahead of the consumers

struct StreamShared {
    uint64_t full[kMaxStreamStages], empty[kMaxStreamStages];
    uint64_t uq_full[kUnitQueue], uq_empty[kUnitQueue];
    int unit_q[kUnitQueue];
    int cnt_q[kUnitQueue];
    unsigned long long red_key[kStreamConsumerWarps];
    float red[kStreamConsumerWarps];
    int target;
    int abort_flag;
    int unit_ok;        // 0 when a wait of the current unit ran out (one decision for all consumers)
};

template <typename T, int D>
__global__ void __launch_bounds__(kStreamThreads, 3)
decode_step_stream_kernel(CacheView c, float alpha_all, const float *__restrict__ alpha_vec,
                          const T *__restrict__ q,
                          const T *__restrict__ k_new, const T *__restrict__ v_new,
                          T *__restrict__ out, int32_t *__restrict__ evicted, int *status,
                          int kStreamStages)
{
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;                    // lanes per row
    constexpr int RPW = 32 / LPR;                   // rows per warp-wide 512-byte read
    constexpr int ROWB = D * (int)sizeof(T);
    constexpr int CR = kChunkBytes / ROWB;          // rows per chunk
    constexpr int NW = kStreamConsumerWarps;
    constexpr int LPC = CR / RPW / NW;              // warp-wide reads per warp and chunk
    static_assert(LPC == 4, "chunk geometry");

    extern __shared__ uint8_t smem_raw[];
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    const int M = c.M;
    float *w = reinterpret_cast<float *>(ring + kStreamStages * kChunkBytes);   // [M+1]
    float *part = w + ((M + 1 + 3) & ~3);                                       // [NW][D]
    StreamShared *sh = reinterpret_cast<StreamShared *>(part + NW * D);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    volatile int *abort_flag = &sh->abort_flag;

    if (tid == 0) {
        for (int s = 0; s < kStreamStages; ++s) { tc::mbar_init(&sh->full[s], 1); tc::mbar_init(&sh->empty[s], NW); }
        for (int x = 0; x < kUnitQueue; ++x) { tc::mbar_init(&sh->uq_full[x], 1); tc::mbar_init(&sh->uq_empty[x], NW); }
        sh->abort_flag = 0;
        tc::fence_mbar_init();
    }
    __syncthreads();

    // a wait that fails poisons the CTA: every later wait returns at once, control flow stays
    // uniform (all consumers still meet at their barriers) and the status word reports it
    auto wait = [&](uint64_t *bar, uint32_t parity) -> bool {
        if (*abort_flag) return false;
        return tc::mbar_wait(bar, parity, abort_flag);
    };

    if (warp == NW) {
        // ---- producer: one lane streams K then V of every unit this CTA claims -------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0, issued = 0;
            bool alive = true;
            const uint64_t policy = evict_first_policy();
            // Units are claimed from a device-wide counter, so a CTA that starts early or meets
            // short units simply takes more of them.  The claim for the NEXT unit and its row
            // count are requested before the current unit is streamed, so neither round trip
            // ever stalls the copy stream.
            // With no more units than CTAs the deal is static (unit = CTA index): the first
            // claim's round trip to the counter would sit at the head of a very short kernel.
            const bool static_deal = c.U <= (int)gridDim.x;
            int u_next = static_deal ? (int)blockIdx.x : atomicAdd(&c.sched[0], 1);
            if (u_next >= c.U) u_next = -1;
            int cnt_next = u_next >= 0 ? min(c.count[u_next], M) : 0;
            for (uint32_t n_unit = 0; alive; ++n_unit) {
                const int u = u_next, cnt = cnt_next;
                const int qi = n_unit % kUnitQueue;
                if (!wait(&sh->uq_empty[qi], ((n_unit / kUnitQueue) & 1) ^ 1)) { alive = false; break; }
                sh->unit_q[qi] = u;
                sh->cnt_q[qi] = cnt;
                tc::mbar_arrive(&sh->uq_full[qi]);
                if (u < 0) break;
                u_next = static_deal ? -1 : atomicAdd(&c.sched[0], 1);
                if (u_next >= c.U) u_next = -1;
                cnt_next = u_next >= 0 ? min(c.count[u_next], M) : 0;
                for (int pass = 0; alive && pass < 2; ++pass) {
                    const uint8_t *base = static_cast<const uint8_t *>(pass == 0 ? c.K : c.V) +
                                          (size_t)u * M * ROWB;
                    for (int r0 = 0; r0 < cnt; r0 += CR) {
                        if (!wait(&sh->empty[stage], phase ^ 1)) { alive = false; break; }
                        const uint32_t bytes = (uint32_t)min(CR, cnt - r0) * ROWB;
                        if (!A2SF_IN_RANGE(stage, kStreamStages, kDbgDecodeStream) ||
                            !A2SF_IN_RANGE(r0 + min(CR, cnt - r0) - 1, M, kDbgDecodeStream) ||
                            !A2SF_IN_RANGE(u, c.U, kDbgDecodeStream)) { alive = false; *abort_flag = 1; break; }
                        tc::mbar_arrive_expect_tx(&sh->full[stage], bytes);
                        bulk_load(ring + stage * kChunkBytes, base + (size_t)r0 * ROWB, bytes, &sh->full[stage], policy);
                        ++issued;
                        if (++stage == kStreamStages) { stage = 0; phase ^= 1; }
                    }
                }
            }
            if (!alive) {
                // bounded chance for copies already issued to land before the CTA exits
                int dummy = 0;
                const uint32_t back = issued < (uint32_t)kStreamStages ? issued : (uint32_t)kStreamStages;
                for (uint32_t x = 0; x < back; ++x) {
                    if (stage == 0) { stage = kStreamStages; phase ^= 1; }
                    --stage;
                    tc::mbar_wait(&sh->full[stage], phase, &dummy);
                }
            }
        }
    } else {
        // ---- consumers ---------------------------------------------------------------------
        const int sub = lane % LPR, rsel = lane / LPR;
        int stage = 0;
        uint32_t phase = 0;
        for (uint32_t n_unit = 0;; ++n_unit) {
            const int qi = n_unit % kUnitQueue;
            const bool got = wait(&sh->uq_full[qi], (n_unit / kUnitQueue) & 1);
            const int u = got ? sh->unit_q[qi] : -1;
            const int cnt = got ? sh->cnt_q[qi] : 0;
            if (consumer_any(!got) || u < 0 || !A2SF_IN_RANGE(u, c.U, kDbgDecodeStream)) break;   // uniform over the consumers
            if (lane == 0) tc::mbar_arrive(&sh->uq_empty[qi]);
            const int p = c.len[u];
            const float alpha = unit_alpha(alpha_vec, u, alpha_all);
            const size_t uo = io_offset(c, u);   // this unit's row of q, k_new, v_new, out
            T *Ku = reinterpret_cast<T *>(c.K) + (size_t)u * M * D;
            T *Vu = reinterpret_cast<T *>(c.V) + (size_t)u * M * D;
            float *Su = c.S + (size_t)u * M;
            int32_t *posu = c.pos + (size_t)u * M;

            // every global word this unit needs is requested up front, so its latency hides
            // behind the K and V phases instead of stalling the reductions and the epilogue
            float qf[VEC];
            Elem<T>::unpack(*reinterpret_cast<const uint4 *>(q + uo + sub * VEC), qf);
            const uint4 knew_raw = *reinterpret_cast<const uint4 *>(k_new + uo + sub * VEC);
            const float vnew_val = tid < D ? Elem<T>::to_float(v_new[uo + tid]) : 0.f;
            float s_pre[kPrefetchSlots];
            int pos_pre[kPrefetchSlots];
#pragma unroll
            for (int x = 0; x < kPrefetchSlots; ++x) {
                const int s_ = tid + x * kStreamConsumers;
                s_pre[x] = s_ < cnt ? Su[s_] : 0.f;
                pos_pre[x] = s_ < cnt ? posu[s_] : 0;
            }

            // (i) logits
            for (int r0 = 0; r0 < cnt; r0 += CR) {
                wait(&sh->full[stage], phase);
                const uint8_t *sbase = ring + stage * kChunkBytes;
                uint4 r[LPC];
#pragma unroll
                for (int x = 0; x < LPC; ++x) {
                    const int lrow = (x * NW + warp) * RPW + rsel;
                    r[x] = *reinterpret_cast<const uint4 *>(sbase + lrow * ROWB + sub * 16);
                }
#pragma unroll
                for (int x = 0; x < LPC; ++x) {
                    const int row = r0 + (x * NW + warp) * RPW + rsel;
                    float kf[VEC];
                    Elem<T>::unpack(r[x], kf);
                    float dot = 0.f;
#pragma unroll
                    for (int e = 0; e < VEC; ++e) dot = fmaf(qf[e], kf[e], dot);
#pragma unroll
                    for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                    if (sub == 0 && row < cnt && A2SF_IN_RANGE(row, M + 1, kDbgDecodeStream)) w[row] = dot * c.scale;
                }
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&sh->empty[stage]);
                if (++stage == kStreamStages) { stage = 0; phase ^= 1; }
            }
            if (warp == 0) {
                float kf[VEC];
                Elem<T>::unpack(knew_raw, kf);
                float dot = 0.f;
#pragma unroll
                for (int e = 0; e < VEC; ++e) dot = fmaf(qf[e], kf[e], dot);
#pragma unroll
                for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                if (lane == 0 && A2SF_IN_RANGE(cnt, M + 1, kDbgDecodeStream)) w[cnt] = dot * c.scale;
            }
            consumer_barrier();

            // (ii) softmax over resident + self
            float m = -INFINITY;
            for (int s_ = tid; s_ <= cnt; s_ += kStreamConsumers) m = fmaxf(m, w[s_]);
            m = consumer_max(m, sh->red);
            float l = 0.f;
            for (int s_ = tid; s_ <= cnt; s_ += kStreamConsumers) {
                const float e = expf(w[s_] - m);
                w[s_] = e;
                l += e;
            }
            l = consumer_sum(l, sh->red);
            const float e_self = w[cnt];

            // (iii) out
            float acc[VEC];
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
            for (int r0 = 0; r0 < cnt; r0 += CR) {
                wait(&sh->full[stage], phase);
                const uint8_t *sbase = ring + stage * kChunkBytes;
                uint4 r[LPC];
#pragma unroll
                for (int x = 0; x < LPC; ++x) {
                    const int lrow = (x * NW + warp) * RPW + rsel;
                    r[x] = *reinterpret_cast<const uint4 *>(sbase + lrow * ROWB + sub * 16);
                }
#pragma unroll
                for (int x = 0; x < LPC; ++x) {
                    const int row = r0 + (x * NW + warp) * RPW + rsel;
                    if (row < cnt) {                 // rows past the count hold stale bytes
                        const float ws = w[row];
                        float vf[VEC];
                        Elem<T>::unpack(r[x], vf);
#pragma unroll
                        for (int e = 0; e < VEC; ++e) acc[e] = fmaf(ws, vf[e], acc[e]);
                    }
                }
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&sh->empty[stage]);
                if (++stage == kStreamStages) { stage = 0; phase ^= 1; }
            }
#pragma unroll
            for (int o = LPR; o < 32; o <<= 1)
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
            if (rsel == 0)
#pragma unroll
                for (int e = 0; e < VEC; ++e) part[warp * D + sub * VEC + e] = acc[e];
            // All of this unit's waits lie behind.  If one of them ran out, its rows are not
            // trustworthy: the unit's cached state (scores, rows, counters) is then left as it
            // was.  One thread decides for all, so the state is never half updated.
            if (tid == 0) sh->unit_ok = !*abort_flag;
            consumer_barrier();
            const bool alive = sh->unit_ok != 0;
            if (tid < D) {
                float o = 0.f;
#pragma unroll
                for (int x = 0; x < NW; ++x) o += part[x * D + tid];
                o = fmaf(e_self, vnew_val, o);
                out[uo + tid] = Elem<T>::from_float(o / l);
            }

            // (iv) S <- alpha*S + a ; (v) argmin over the non-recent slots
            const bool full = cnt >= M;
            const int newest_evictable = p - c.R;
            unsigned long long best = ~0ull;
            int best_slot = -1;
            int x_pre = 0;
            for (int s_ = tid; s_ < cnt; s_ += kStreamConsumers, ++x_pre) {
                const float a = w[s_] / l;
                float s_old;
                int ps;
                if (x_pre == 0) { s_old = s_pre[0]; ps = pos_pre[0]; }
                else if (x_pre == 1) { s_old = s_pre[1]; ps = pos_pre[1]; }
                else { s_old = Su[s_]; ps = posu[s_]; }
                const float sn = fmaf(alpha, s_old, a);
                if (alive && A2SF_IN_RANGE(s_, M, kDbgDecodeStream)) Su[s_] = sn;
                if (full && ps <= newest_evictable) {
                    const unsigned long long key =
                        ((unsigned long long)__float_as_uint(sn) << 32) | (unsigned)ps;
                    if (key < best) { best = key; best_slot = s_; }
                }
            }
            const float a_self = e_self / l;
            const unsigned long long wbest = warp_min_u64(best);
            if (lane == 0) sh->red_key[warp] = wbest;
            if (tid == 0) sh->target = full ? -2 : cnt;
            consumer_barrier();
            unsigned long long gbest = sh->red_key[0];
#pragma unroll
            for (int x = 1; x < NW; ++x) gbest = sh->red_key[x] < gbest ? sh->red_key[x] : gbest;
            if (full && best_slot >= 0 && best == gbest) {
                const unsigned long long self_key =
                    ((unsigned long long)__float_as_uint(a_self) << 32) | (unsigned)p;
                if (c.R > 0 || gbest < self_key) sh->target = best_slot;
            }
            consumer_barrier();

            const int target = sh->target;
            if (target >= 0 && alive && A2SF_IN_RANGE(target, M, kDbgDecodeStream)) {
                if (tid < LPR)
                    *reinterpret_cast<uint4 *>(Ku + (size_t)target * D + tid * VEC) =
                        *reinterpret_cast<const uint4 *>(k_new + uo + tid * VEC);
                else if (tid < 2 * LPR)
                    *reinterpret_cast<uint4 *>(Vu + (size_t)target * D + (tid - LPR) * VEC) =
                        *reinterpret_cast<const uint4 *>(v_new + uo + (tid - LPR) * VEC);
            }
            if (tid == 0 && alive) {
                if (target >= 0 && A2SF_IN_RANGE(target, M, kDbgDecodeStream)) {
                    Su[target] = a_self;
                    posu[target] = p;
                }
                if (!full) c.count[u] = cnt + 1;
                c.len[u] = p + 1;
                evicted[u] = full ? target : -1;
            }
            consumer_barrier();      // w[], part[], target are reused by the next unit
        }
    }
    __syncthreads();
    if (tid == 0) {
        if (sh->abort_flag) *status = A2SF_ERR_TIMEOUT;
        // the last CTA to leave re-arms the claim counter for the next launch
        __threadfence();
        if (atomicAdd(&c.sched[1], 1) == (int)gridDim.x - 1) {
            c.sched[0] = 0;
            c.sched[1] = 0;
            __threadfence();
        }
    }
}

template <typename T, int D>
cudaError_t launch_split(const CacheView &c, int cluster_size, float alpha, const float *alpha_vec,
                         const void *q, const void *k_new, const void *v_new, void *out, int32_t *evicted,
                         cudaStream_t s)
{
    constexpr int NT = kDecodeThreads;
    const size_t per_max = ((size_t)c.M + cluster_size - 1) / cluster_size;
    const size_t smem = ((per_max + 1 + 3) & ~(size_t)3) * 4 + (size_t)(NT / 32) * D * 4 + (NT / 32) * 4;
    auto kern = decode_step_split_kernel<T, D, NT>;
    if (cudaError_t e = allow_dynamic_smem<decode_step_split_kernel<T, D, NT>>(smem); e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)c.U * cluster_size);
    cfg.blockDim = dim3(NT);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster_size;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, c, alpha, alpha_vec, static_cast<const T *>(q),
                                             static_cast<const T *>(k_new), static_cast<const T *>(v_new),
                                             static_cast<T *>(out), evicted);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch_stream(const CacheView &c, float alpha, const float *alpha_vec, const void *q,
                          const void *k_new, const void *v_new, void *out, int32_t *evicted, cudaStream_t s)
{
    const size_t fixed = 128 + (((size_t)c.M + 1 + 3) & ~(size_t)3) * 4 +
                         (size_t)kStreamConsumerWarps * D * 4 + sizeof(StreamShared);
    // several CTAs per SM so one CTA's reductions overlap the others' streaming; each ring
    // takes its share of the SM's shared memory
    constexpr int ctas_per_sm = kStreamCtasPerSm;
    const size_t per_cta = (227 * 1024) / ctas_per_sm - 1024;
    if (fixed + 3 * kChunkBytes > per_cta) return launch_split<T, D>(c, 1, alpha, alpha_vec, q, k_new, v_new, out, evicted, s);
    int stages = (int)((per_cta - fixed) / kChunkBytes);
    if (stages > kMaxStreamStages) stages = kMaxStreamStages;
    const size_t smem = fixed + (size_t)stages * kChunkBytes;
    auto kern = decode_step_stream_kernel<T, D>;
    const int num_sms = device_sm_count();
    if (num_sms <= 0) return cudaErrorUnknown;
    // Few units with long caches would leave most SMs idle: split each unit over a cluster.
    if (c.M >= kSplitMinBudget && c.U * 2 <= num_sms) {
        int cs = 2;
        while (cs < 8 && c.U * cs * 2 <= 2 * num_sms) cs *= 2;
        return launch_split<T, D>(c, cs, alpha, alpha_vec, q, k_new, v_new, out, evicted, s);
    }
    if (cudaError_t e = allow_dynamic_smem<decode_step_stream_kernel<T, D>>(smem); e != cudaSuccess) return e;
    int *status = decode_status_word();
    if (!status) return cudaErrorUnknown;
    const int grid = c.U < ctas_per_sm * num_sms ? c.U : ctas_per_sm * num_sms;
    kern<<<grid, kStreamThreads, smem, s>>>(c, alpha, alpha_vec, static_cast<const T *>(q),
                                            static_cast<const T *>(k_new), static_cast<const T *>(v_new),
                                            static_cast<T *>(out), evicted, status, stages);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_step(const CacheView &c, float alpha, const float *alpha_vec, const void *q,
                               const void *k_new, const void *v_new, void *out, int32_t *evicted,
                               cudaStream_t s)
{
#define A2SF_DISPATCH(T)                                                                     \
    (c.d == 64 ? launch_stream<T, 64>(c, alpha, alpha_vec, q, k_new, v_new, out, evicted, s)  \
               : launch_stream<T, 128>(c, alpha, alpha_vec, q, k_new, v_new, out, evicted, s))
    switch (c.dtype) {
    case A2SF_F32: return A2SF_DISPATCH(float);
    case A2SF_BF16: return A2SF_DISPATCH(__nv_bfloat16);
    default: return A2SF_DISPATCH(__half);
    }
#undef A2SF_DISPATCH
}

// device address of the status word, looked up once per device
int *decode_status_word()
{
    static std::once_flag once[kMaxDevices];
    static int *ptr[kMaxDevices] = {};
    const int dev = current_device_index();
    std::call_once(once[dev], [dev] {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_decode_status) == cudaSuccess) ptr[dev] = static_cast<int *>(p);
    });
    return ptr[dev];
}

int read_and_clear_decode_status(cudaStream_t s)
{
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbolAsync(&v, g_decode_status, sizeof(int), 0, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return A2SF_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return A2SF_ERR_CUDA;
    if (v != 0 &&
        cudaMemcpyToSymbolAsync(g_decode_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return A2SF_ERR_CUDA;
    return v;
}

}  // namespace a2sf
