// Pieces shared by the decode kernels: launch arguments, mbarrier / bulk-copy PTX wrappers, the
// division of the step line among CTAs, the producer warp, and the merge of partial softmax states.
//
// Execution shape (both kernels): a persistent grid of one CTA per SM.  The (sequence, KV head) units
// are cut into steps of two pages (32 tokens); the steps of all units form one line that is divided
// evenly among the CTAs, so a CTA owns a contiguous run of steps that may cross unit boundaries.
// Inside a CTA one producer warp streams pages into a shared-memory ring with bulk asynchronous copies
// that signal mbarriers; eight consumer warps each take whole steps and keep an online-softmax state
// (running max m in the log2 domain, running sum l, unnormalised output).  At the end of a unit's run
// the warps are merged by log-sum-exp; if several CTAs share the unit each writes a partial and the
// last to arrive (an atomic ticket, no waiting) merges them.
#pragma once

#include "spark_common.cuh"

namespace spark {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kDecodeThreads = kConsumerThreads + 32;
constexpr int kMaxSlots = 16;
constexpr int kStepTokens = 2 * kPageTokens;
constexpr unsigned kSpinLimit = 1u << 20;    // bounded mbarrier waits
constexpr unsigned kFull = 0xffffffffu;
constexpr int kRec = kHeadDim + 4;           // floats per head record: 128 outputs, running max, running sum, pad
constexpr float kLn2 = 0.6931471805599453f;

struct DecodeArgs {
    const void* q;
    const unsigned char* pages;
    const int32_t* block_table;
    int max_blocks;
    const int32_t* lens;
    const float* qnorm;
    float* out;
    float* lse;
    int B, Hq, Hkv;
    int64_t n_pool_pages;
    PageLayout L;
    float scale_log2e;
    int* status;
    int* tickets;
    float* partials;
    int nslots;
    int slot_stride;
};

// control block at the start of dynamic shared memory
constexpr int kCtrlBytes = 512;                                  // full[16], empty[16], flags
constexpr int kPrefixBytes = ((kMaxBatch + 1) * 4 + 15) / 16 * 16;

// ---- PTX helpers ----------------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p)
{
    return static_cast<unsigned>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Wait with an iteration limit.  On expiry (or if another thread already gave up) the CTA-wide abort
// flag is set, the status word records the timeout and the caller carries on without the data; the
// kernel then finishes structurally (same barriers) and returns.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity, volatile int* abort_flag, int* status)
{
    for (unsigned it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    record_error(status, SPARK_ERR_DEVICE_TIMEOUT);
    return false;
}
// Bulk copy global -> shared that signals `bar`; `policy` is an L2 eviction policy (pages are read once
// per step, so they are streamed evict-first and leave the L2 to the small tables and the partials).
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, unsigned bytes, uint64_t* bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void consumer_sync()
{
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}

__device__ __forceinline__ int steps_of(int len)
{
    return ((len + kPageTokens - 1) / kPageTokens + 1) >> 1;
}

__device__ __forceinline__ int clamp_len(int len, int max_tokens)
{
    return len < 0 ? 0 : (len > max_tokens ? max_tokens : len);
}

struct Segment {
    int b, h, i0, n, steps_b;
    int unit_start;          // global step index of the unit's first step
};

// Locate global step g (must be < total) and the run of steps it starts inside [g, c1).
__device__ __forceinline__ Segment locate(const int* prefix, int B, int Hkv, int g, int c1)
{
    int lo = 0, hi = B;                                   // first b' in (lo, hi] with Hkv*prefix[b'] > g
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (static_cast<int64_t>(Hkv) * prefix[mid] > g) hi = mid; else lo = mid;
    }
    Segment s;
    s.b = lo;
    s.steps_b = prefix[lo + 1] - prefix[lo];
    const int r = g - Hkv * prefix[lo];
    s.h = r / s.steps_b;
    s.i0 = r - s.h * s.steps_b;
    s.unit_start = Hkv * prefix[lo] + s.h * s.steps_b;
    const int left = s.steps_b - s.i0;
    s.n = (c1 - g < left) ? (c1 - g) : left;
    return s;
}

// How the step line is divided among the CTAs.
//   stream mode : CTA c owns steps [c*chunk, (c+1)*chunk) of the whole line; a CTA may cross unit
//                 boundaries (exact balance; used when sequences differ in length or units are many).
//   aligned mode: all units have the same number of steps and there are several CTAs per unit; unit u
//                 gets q or q+1 whole CTAs (the first `rem` units get q+1) and is split evenly among
//                 them, so no CTA crosses a unit boundary and every CTA publishes exactly once.
struct Plan {
    int total;        // steps on the line
    int chunk;        // stream mode: steps per CTA
    int aligned;      // 1: aligned mode
    int unit_steps;   // aligned mode: steps of every unit
    int q, rem;       // aligned mode: CTAs per unit
};

struct Ctrl {
    uint64_t* full;
    uint64_t* empty;
    volatile int* abort_flag;
    volatile int* last_flag;
    Plan* plan;
    int* prefix;
};

__device__ __forceinline__ Ctrl make_ctrl(unsigned char* smem)
{
    Ctrl c;
    c.full = reinterpret_cast<uint64_t*>(smem);
    c.empty = c.full + kMaxSlots;
    c.abort_flag = reinterpret_cast<volatile int*>(smem + 256);
    c.last_flag = reinterpret_cast<volatile int*>(smem + 260);
    c.plan = reinterpret_cast<Plan*>(smem + 272);
    c.prefix = reinterpret_cast<int*>(smem + kCtrlBytes);
    return c;
}

// Barrier init (thread 0) and the steps-per-sequence prefix (warp 0).  Ends with __syncthreads().
__device__ __forceinline__ void decode_prologue(const DecodeArgs& A, const Ctrl& C, int tid)
{
    const int warp = tid >> 5, lane = tid & 31;
    const int max_tokens = A.max_blocks * kPageTokens;
    if (tid == 0) {
        for (int s = 0; s < A.nslots; ++s) { mbar_init(&C.full[s], 1); mbar_init(&C.empty[s], 1); }
        *C.abort_flag = 0;
        *C.last_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 0) {
        int running = 0, smin = 0x7fffffff, smax = 0;
        for (int b0 = 0; b0 < A.B; b0 += 32) {
            const int b = b0 + lane;
            int st = 0;
            if (b < A.B) {
                const int len = A.lens[b];
                if (len < 0 || len > max_tokens) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
                st = steps_of(clamp_len(len, max_tokens));
                smin = min(smin, st);
                smax = max(smax, st);
            }
            int inc = st;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(kFull, inc, o);
                if (lane >= o) inc += n;
            }
            if (b < A.B) C.prefix[b + 1] = running + inc;
            running += __shfl_sync(kFull, inc, 31);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            smin = min(smin, __shfl_xor_sync(kFull, smin, o));
            smax = max(smax, __shfl_xor_sync(kFull, smax, o));
        }
        if (lane == 0) {
            C.prefix[0] = 0;
            Plan pl;
            const int nct = static_cast<int>(gridDim.x), units = A.B * A.Hkv;
            pl.total = A.Hkv * running;
            pl.chunk = (pl.total + nct - 1) / nct;
            pl.aligned = 0; pl.unit_steps = smax; pl.q = 0; pl.rem = 0;
            if (smin == smax && smax > 0 && units <= nct) {
                const int q = nct / units;
                const int makespan = (smax + q - 1) / q;
                if (q >= 2 && makespan * 25 <= pl.chunk * 26) {          // within 4 % of the even split
                    pl.aligned = 1; pl.q = q; pl.rem = nct - q * units;
                }
            }
            *C.plan = pl;
        }
    }
    __syncthreads();
}

// This CTA's run of steps [c0, c1) on the line.
__device__ __forceinline__ void cta_range(const Plan& pl, int cta, int& c0, int& c1)
{
    if (!pl.aligned) {
        c0 = min(pl.total, cta * pl.chunk);
        c1 = min(pl.total, c0 + pl.chunk);
        return;
    }
    const int big = pl.rem * (pl.q + 1);                   // CTAs that belong to units with q+1 CTAs
    int u, k, n;
    if (cta < big) { u = cta / (pl.q + 1); k = cta - u * (pl.q + 1); n = pl.q + 1; }
    else { u = pl.rem + (cta - big) / pl.q; k = (cta - big) - (u - pl.rem) * pl.q; n = pl.q; }
    const int per = (pl.unit_steps + n - 1) / n;
    c0 = u * pl.unit_steps + min(pl.unit_steps, k * per);
    c1 = u * pl.unit_steps + min(pl.unit_steps, (k + 1) * per);
}

// The CTAs that hold a part of the unit starting at step `unit_start` with `unit_steps` steps.
__device__ __forceinline__ void unit_parts(const Plan& pl, int unit_start, int unit_steps, int& first_cta, int& n_parts)
{
    if (!pl.aligned) {
        first_cta = unit_start / pl.chunk;
        n_parts = (unit_start + unit_steps - 1) / pl.chunk - first_cta + 1;
        return;
    }
    const int u = unit_start / pl.unit_steps;
    const int n = pl.q + (u < pl.rem ? 1 : 0);
    first_cta = u * pl.q + min(u, pl.rem);
    const int per = (pl.unit_steps + n - 1) / n;
    n_parts = (pl.unit_steps + per - 1) / per;             // trailing CTAs of the unit may be empty
}

// The producer warp: walks this CTA's steps [c0, c1) in order, looks the page ids up 32 steps at a
// time, and lane 0 issues one or two page copies per step into ring slot (ordinal % nslots) once the
// consumers have released it.
__device__ __forceinline__ void producer_loop(const DecodeArgs& A, const Ctrl& C, unsigned char* ring,
                                              int c0, int c1, int lane)
{
    const PageLayout L = A.L;
    const int NS = A.nslots, n_total = c1 - c0;
    const int max_tokens = A.max_blocks * kPageTokens;
    bool live = true;
    int issued = 0;
    const uint64_t policy = policy_evict_first();
    for (int n0 = 0; n0 < n_total; n0 += 32) {
        const int n = n0 + lane;
        int id0 = -1, id1 = -1;
        if (n < n_total) {
            const Segment s = locate(C.prefix, A.B, A.Hkv, c0 + n, c1);
            const int len = clamp_len(A.lens[s.b], max_tokens);
            const int nblk = (len + kPageTokens - 1) / kPageTokens;
            const int32_t* bt = A.block_table + (static_cast<int64_t>(s.b) * A.Hkv + s.h) * A.max_blocks;
            id0 = bt[2 * s.i0];
            if (2 * s.i0 + 1 < nblk) {
                id1 = bt[2 * s.i0 + 1];
                if (id1 < 0 || id1 >= A.n_pool_pages) { record_error(A.status, SPARK_ERR_DEVICE_BOUNDS); id1 = 0; }
            }
            if (id0 < 0 || id0 >= A.n_pool_pages) { record_error(A.status, SPARK_ERR_DEVICE_BOUNDS); id0 = 0; }
        }
        const int cnt = min(32, n_total - n0);
        for (int kk = 0; kk < cnt; ++kk) {
            const int p0 = __shfl_sync(kFull, id0, kk);
            const int p1 = __shfl_sync(kFull, id1, kk);
            if (lane == 0 && live) {
                const int nn = n0 + kk, slot = nn % NS, round = nn / NS;
                if (round > 0) live = mbar_wait(&C.empty[slot], (round - 1) & 1, C.abort_flag, A.status);
                if (live) {
                    unsigned char* dst = ring + static_cast<size_t>(slot) * A.slot_stride;
                    const unsigned bytes = L.page_bytes * (p1 >= 0 ? 2u : 1u);
                    mbar_expect_tx(&C.full[slot], bytes);
                    bulk_g2s(dst, A.pages + static_cast<int64_t>(p0) * L.page_bytes, L.page_bytes, &C.full[slot], policy);
                    if (p1 >= 0)
                        bulk_g2s(dst + L.page_bytes, A.pages + static_cast<int64_t>(p1) * L.page_bytes,
                                 L.page_bytes, &C.full[slot], policy);
                    ++issued;
                }
            }
        }
    }
    // after a give-up: let the copies already in flight land before the CTA may exit
    if (lane == 0 && !live) {
        for (int nn = max(0, issued - NS); nn < issued; ++nn) {
            uint64_t* bar = &C.full[nn % NS];
            const unsigned parity = (nn / NS) & 1;
            for (unsigned it = 0; it < kSpinLimit; ++it)
                if (mbar_try_wait(bar, parity)) break;
        }
    }
}

// zero-length sequences: out = 0, lse = -inf (consumer threads)
__device__ __forceinline__ void write_empty_sequences(const DecodeArgs& A, const int* prefix, int tid)
{
    for (int b = blockIdx.x; b < A.B; b += gridDim.x)
        if (prefix[b + 1] == prefix[b]) {
            for (int i = tid; i < A.Hq * kHeadDim; i += kConsumerThreads)
                A.out[static_cast<int64_t>(b) * A.Hq * kHeadDim + i] = 0.f;
            if (A.lse)
                for (int i = tid; i < A.Hq; i += kConsumerThreads)
                    A.lse[static_cast<int64_t>(b) * A.Hq + i] = -INFINITY;
        }
}

// Merge the per-warp states that the consumer warps have written to `merge`
// ([warp][G][kRec]: 128 unnormalised outputs, m, l) and publish the unit's result: directly when this
// CTA covers the whole unit, else as a partial followed by the last-arriver merge.  Called by all
// consumer threads after a consumer_sync(); ends with a consumer_sync().
template <int G>
__device__ __forceinline__ void merge_and_publish(const DecodeArgs& A, const Ctrl& C, const float* merge,
                                                  const Segment& sg, int tid)
{
    const int b = sg.b, h = sg.h;
    int first_cta, n_parts;
    unit_parts(*C.plan, sg.unit_start, sg.steps_b, first_cta, n_parts);
    const int unit = b * A.Hkv + h;
    float* part_out = A.partials + static_cast<int64_t>(blockIdx.x + unit) * G * kRec;
    for (int idx = tid; idx < G * kHeadDim; idx += kConsumerThreads) {
        const int gg = idx / kHeadDim, c = idx - gg * kHeadDim;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, merge[(w * G + gg) * kRec + kHeadDim]);
        float Ls = 0.f, O = 0.f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
            const float* r = merge + (w * G + gg) * kRec;
            const float f = exp2f(r[kHeadDim] - M);
            Ls = fmaf(r[kHeadDim + 1], f, Ls);
            O = fmaf(r[c], f, O);
        }
        if (n_parts == 1) {
            A.out[(static_cast<int64_t>(b) * A.Hq + h * G + gg) * kHeadDim + c] = O / Ls;
            if (c == 0 && A.lse)
                A.lse[static_cast<int64_t>(b) * A.Hq + h * G + gg] = (M + log2f(Ls)) * kLn2;
        } else {
            part_out[gg * kRec + c] = O;
            if (c == 0) { part_out[gg * kRec + kHeadDim] = M; part_out[gg * kRec + kHeadDim + 1] = Ls; }
        }
    }
    if (n_parts > 1) {
        // The barrier orders every consumer thread's partial stores before thread 0's gpu-scope
        // release; the last arriver's acquire (same atomic) plus the next barrier orders its reads
        // after all partials.
        consumer_sync();
        if (tid == 0) {
            int old;
            asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(A.tickets + unit) : "memory");
            *C.last_flag = (old == n_parts - 1) ? 1 : 0;
        }
        consumer_sync();
        if (*C.last_flag) {                              // last CTA of this unit: merge all partials
            constexpr int kBatch = 20;                   // loads of a batch are in flight together
            constexpr int64_t kStride = static_cast<int64_t>(G) * kRec;
            for (int idx = tid; idx < G * kHeadDim; idx += kConsumerThreads) {
                const int gg = idx / kHeadDim, c = idx - gg * kHeadDim;
                const float* r0 = A.partials + (static_cast<int64_t>(first_cta + unit) * G + gg) * kRec;
                float M = -INFINITY, Ls = 0.f, O = 0.f;
                for (int p0 = 0; p0 < n_parts; p0 += kBatch) {
                    float mv[kBatch], lv[kBatch], ov[kBatch];
#pragma unroll
                    for (int k = 0; k < kBatch; ++k) {
                        const bool in = p0 + k < n_parts;
                        const float* r = r0 + (p0 + k) * kStride;
                        mv[k] = in ? __ldcg(r + kHeadDim) : -INFINITY;
                        lv[k] = in ? __ldcg(r + kHeadDim + 1) : 0.f;
                        ov[k] = in ? __ldcg(r + c) : 0.f;
                    }
                    float Mn = M;
#pragma unroll
                    for (int k = 0; k < kBatch; ++k) Mn = fmaxf(Mn, mv[k]);
                    const float sc = exp2f(M - Mn);      // 0 for the first batch
                    Ls *= sc;
                    O *= sc;
#pragma unroll
                    for (int k = 0; k < kBatch; ++k) {
                        const float f = exp2f(mv[k] - Mn);
                        Ls = fmaf(lv[k], f, Ls);
                        O = fmaf(ov[k], f, O);
                    }
                    M = Mn;
                }
                A.out[(static_cast<int64_t>(b) * A.Hq + h * G + gg) * kHeadDim + c] = O / Ls;
                if (c == 0 && A.lse)
                    A.lse[static_cast<int64_t>(b) * A.Hq + h * G + gg] = (M + log2f(Ls)) * kLn2;
            }
            if (tid == 0) A.tickets[unit] = 0;          // ready for the next call
        }
    }
    consumer_sync();
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// per-dtype launchers (spark_decode.cu: fp32 storage, spark_decode_mma.cu: bf16 storage)
spark_status launch_decode_f32(int G, const DecodeArgs& A, int n_sms, int smem_optin, cudaStream_t stream);
spark_status launch_decode_bf16(int G, const DecodeArgs& A, int n_sms, int smem_optin, cudaStream_t stream);

}  // namespace spark
