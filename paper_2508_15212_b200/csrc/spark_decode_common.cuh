// Pieces shared by the decode kernels: launch arguments, mbarrier / bulk-copy PTX wrappers, the
// division of the step line among CTAs, the producer warp, and the merge of partial softmax states.
//
// Execution shape (both kernels): a persistent grid of one CTA per SM.  Every (sequence, KV head) unit
// is cut into steps of `pps` pages (16 or 32 tokens); the steps of all units form one line that is
// divided among the CTAs.  Inside a CTA one producer warp streams pages into a shared-memory ring with
// bulk asynchronous copies that signal mbarriers; NW consumer warps each take whole steps and keep an
// online-softmax state (running max m in the log2 domain, running sum l, unnormalised output).  At
// the end of a unit's run the warps are merged by log-sum-exp; if several CTAs share the unit each
// writes a partial and the last to arrive (an atomic ticket, no waiting) merges them.
#pragma once

#include "spark_common.cuh"

namespace spark {

constexpr int kMaxSlots = 32;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // every device-side wait gives up after one second
constexpr unsigned kClockEvery = 256;                        // polls between two looks at the clock
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
    int pps;                                 // pages per step (= per ring slot): 1 or 2
    int prefix_off;                          // shared-memory offset of the steps-per-sequence prefix ((B + 1) ints)
    int ring_off;                            // shared-memory offset of the ring (behind the prefix)
    int overlap;                             // launched as a programmatic dependent of the preceding kernel
    unsigned seed;                           // sampled recovery: seed of the per-entry draws
    const int* page_rows;                    // ragged pages: slot rows in use per pool page (else null: whole pages)
    int q_by_value;                          // host side only: q is a HOST pointer whose bytes travel as a launch parameter
};

// largest query (bytes) that may travel as a launch parameter (kernel parameters are limited to 32764 bytes)
constexpr int kMaxQueryByValueBytes = 24 * 1024;

// control block at the start of dynamic shared memory
constexpr int kCtrlBytes = 1024;                                 // full[32], empty[32], flags, plan
// the steps-per-sequence prefix sits between a kernel's fixed shared-memory areas and the ring and is as
// large as the batch needs, so small batches leave its room to the ring
inline int prefix_bytes(int batch) { return ((batch + 1) * 4 + 127) / 128 * 128; }

// Shared merge area for `nw` consumer warps and `g` heads: the warps' states ([warp][head][kRec] floats:
// 128 outputs, m, l and two spare words that the CTA-wide merge uses for the warp's weight and the head's
// (M, L)), reused by the final combine for the weights of up to kMaxCtas parts, the heads' (M, L) and one
// float4 per consumer thread.
__host__ __device__ constexpr int merge_state_floats(int nw, int g)
{
    return nw * g * kRec > kMaxCtas * g * 2 + nw * 32 * 4 ? nw * g * kRec : kMaxCtas * g * 2 + nw * 32 * 4;
}
__host__ __device__ constexpr int merge_bytes(int nw, int g) { return merge_state_floats(nw, g) * 4; }

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
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Expiry test of a polling loop: looks at the nanosecond clock every kClockEvery polls (the first look
// only records the start), so a wait is bounded by wall time, not by how fast the poll happens to spin.
struct WaitClock {
    unsigned it = 0;
    unsigned long long t0 = 0;
    __device__ __forceinline__ bool expired()
    {
        if ((++it & (kClockEvery - 1)) != 0) return false;
        const unsigned long long now = global_ns();
        if (t0 == 0) { t0 = now; return false; }
        return now - t0 > kWaitLimitNs;
    }
};
// Wait with a time limit.  On expiry (or if another thread already gave up) the CTA-wide abort
// flag is set, the status word records the timeout and the caller carries on without the data; the
// kernel then finishes structurally (same barriers) and returns.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity, volatile int* abort_flag, int* status)
{
    WaitClock wc;
    while (!wc.expired()) {
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
// Consumer side of a ring slot: wait until the data of revolution `round` has landed in `slot`.
// A parity wait alone cannot tell "revolution r has not been armed yet" from "revolution r is
// complete" (consumers of different revolutions of one slot are different warps), so the slot's
// revolution counter, written by the producer when it arms the barrier, is checked first.
__device__ __forceinline__ bool slot_wait(uint64_t* full, volatile int* seq, int slot, int round,
                                          volatile int* abort_flag, int* status)
{
    WaitClock wc;
    while (seq[slot] != round + 1) {
        if (wc.expired() || *abort_flag) {
            if (!*abort_flag) { *abort_flag = 1; record_error(status, SPARK_ERR_DEVICE_TIMEOUT); }
            return false;
        }
    }
    return mbar_wait(&full[slot], round & 1, abort_flag, status);
}
// Programmatic dependent launch (sm_90+).  launch_dependents: the kernel enqueued after this one may be
// scheduled as CTAs of this grid exit.  dependency_wait: returns once the kernel enqueued before this
// one has completed and its writes are visible (a no-op for an ordinary launch).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launch helper: ordinary launch, or with the programmatic-stream-serialization attribute.
template <typename Kernel, typename... More>
inline cudaError_t launch_decode_kernel(Kernel kernel, int grid, int threads, size_t smem, cudaStream_t stream,
                                        const DecodeArgs& A, const More&... more)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = A.overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, A, more...);
}

template <int NT> __device__ __forceinline__ void consumer_sync()
{
    asm volatile("bar.sync 1, %0;" ::"n"(NT) : "memory");
}

__device__ __forceinline__ int steps_of(int len, int pps)
{
    return ((len + kPageTokens - 1) / kPageTokens + pps - 1) / pps;
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
//   whole units : all units have the same number of steps and there are more units than CTAs; every CTA
//                 takes q or q+1 whole units (the first `rem` CTAs take q+1).  No unit is split, so
//                 there are no partials and no last-arriver merge; used when the uneven deal costs at
//                 most 25 % over the even split.
struct Plan {
    int total;        // steps on the line
    int chunk;        // stream mode: steps per CTA
    int aligned;      // 0: stream, 1: aligned mode, 2: whole units
    int unit_steps;   // aligned / whole units: steps of every unit
    int q, rem;       // aligned: CTAs per unit; whole units: units per CTA
};

struct Ctrl {
    uint64_t* full;
    uint64_t* empty;
    volatile int* abort_flag;
    volatile int* last_flag;
    volatile int* seq;        // [32] revolution + 1 for which each slot was last armed
    Plan* plan;
    int* prefix;
};

__device__ __forceinline__ Ctrl make_ctrl(unsigned char* smem, int prefix_off)
{
    Ctrl c;
    c.full = reinterpret_cast<uint64_t*>(smem);
    c.empty = c.full + kMaxSlots;
    c.abort_flag = reinterpret_cast<volatile int*>(smem + 512);
    c.last_flag = reinterpret_cast<volatile int*>(smem + 516);
    c.plan = reinterpret_cast<Plan*>(smem + 528);
    c.seq = reinterpret_cast<volatile int*>(smem + 640);
    c.prefix = reinterpret_cast<int*>(smem + prefix_off);
    return c;
}

// Start of the kernel.  The PRODUCER warp alone reads packed_lens, builds the steps-per-sequence prefix and
// the plan, initialises the ring barriers, and then arrives (without waiting) on hardware barrier 2; it
// goes straight on to its first page copies.  The consumer warps wait on barrier 2 for the plan.  So the
// chain from launch to the first bytes in flight is: packed_lens (one global round trip) -> plan -> page
// ids -> bulk copies, with no CTA-wide barrier in between.
//
// All threads first ask the L2 to fetch the block table (when there is one): the producer's page-id
// loads then find their lines on the way instead of starting a second cold DRAM round trip behind
// packed_lens.
constexpr int kPlanBarrier = 2;
constexpr int64_t kTablePrefetchMax = 8 << 20;             // bytes of block table asked for at most

__device__ __forceinline__ void prefetch_block_table(const DecodeArgs& A, int tid, int n_threads)
{
    if (!A.block_table) return;
    int64_t bytes = static_cast<int64_t>(A.B) * A.Hkv * A.max_blocks * 4;
    if (bytes > kTablePrefetchMax) bytes = kTablePrefetchMax;
    const char* base = reinterpret_cast<const char*>(A.block_table);
    for (int64_t o = (static_cast<int64_t>(blockIdx.x) * n_threads + tid) * 128; o < bytes;
         o += static_cast<int64_t>(gridDim.x) * n_threads * 128)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(base + o));
}

__device__ __forceinline__ void producer_prologue(const DecodeArgs& A, const Ctrl& C, int lane, int n_threads)
{
    const int max_tokens = A.max_blocks * kPageTokens;
    // packed_lens first: everything else of the prologue fits under this load's latency
    int first_len = 0;
    if (lane < A.B) first_len = A.lens[lane];
    if (lane < A.nslots) { mbar_init(&C.full[lane], 1); mbar_init(&C.empty[lane], 1); }
    C.seq[lane] = 0;
    if (lane == 0) { *C.abort_flag = 0; *C.last_flag = 0; }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    int running = 0, smin = 0x7fffffff, smax = 0;
    for (int b0 = 0; b0 < A.B; b0 += 32) {
        const int b = b0 + lane;
        int st = 0;
        if (b < A.B) {
            const int len = b0 == 0 ? first_len : A.lens[b];
            if (len < 0 || len > max_tokens) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
            st = steps_of(clamp_len(len, max_tokens), A.pps);
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
        } else if (smin == smax && smax > 0) {
            const int q = units / nct, rem = units - q * nct;
            const int makespan = (q + (rem ? 1 : 0)) * smax;
            if (makespan * 4 <= pl.chunk * 5) {                      // within 25 % of the even split
                pl.aligned = 2; pl.q = q; pl.rem = rem;
            }
        }
        *C.plan = pl;
    }
    __syncwarp();
    asm volatile("bar.arrive %0, %1;" ::"n"(kPlanBarrier), "r"(n_threads) : "memory");
}

// consumer side of the prologue: returns once the plan, the prefix and the ring barriers are in place
__device__ __forceinline__ void consumer_wait_plan(int n_threads)
{
    asm volatile("bar.sync %0, %1;" ::"n"(kPlanBarrier), "r"(n_threads) : "memory");
}

// This CTA's run of steps [c0, c1) on the line.
__device__ __forceinline__ void cta_range(const Plan& pl, int cta, int& c0, int& c1)
{
    if (!pl.aligned) {
        c0 = min(pl.total, cta * pl.chunk);
        c1 = min(pl.total, c0 + pl.chunk);
        return;
    }
    if (pl.aligned == 2) {                                  // whole units: the first `rem` CTAs take q + 1
        const int first = cta * pl.q + min(cta, pl.rem);
        c0 = first * pl.unit_steps;
        c1 = c0 + (pl.q + (cta < pl.rem ? 1 : 0)) * pl.unit_steps;
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
    if (pl.aligned == 2) {
        const int u2 = unit_start / pl.unit_steps, big = pl.rem * (pl.q + 1);
        first_cta = u2 < big ? u2 / (pl.q + 1) : pl.rem + (u2 - big) / pl.q;
        n_parts = 1;
        return;
    }
    const int u = unit_start / pl.unit_steps;
    const int n = pl.q + (u < pl.rem ? 1 : 0);
    first_cta = u * pl.q + min(u, pl.rem);
    const int per = (pl.unit_steps + n - 1) / n;
    n_parts = (pl.unit_steps + per - 1) / per;             // trailing CTAs of the unit may be empty
}

// The producer warp.  Lane i owns ring slot i: it handles this CTA's steps i, i + nslots, i + 2 nslots,
// ... in order.  Per revolution of the ring every lane looks up the page ids of its step (block-table
// loads of the next revolution are issued before the current one is polled, so their latency hides
// behind the wait), then the warp polls: a lane whose slot has been released by the consumers arms
// the slot's barrier and issues its page copies at once.  Polling is bounded; on expiry the CTA-wide
// abort flag is set and the lanes wait (bounded) for their own copies in flight before returning.
// bytes of page `id` to bring in: everything, or (ragged pages) up to the last slot row in use
__device__ __forceinline__ unsigned page_copy_bytes(const DecodeArgs& A, int id)
{
    if (!A.page_rows) return static_cast<unsigned>(A.L.page_bytes);
    int rows = A.page_rows[id];
    rows = rows < 0 ? 0 : (rows > A.L.keep ? A.L.keep : rows);
    return static_cast<unsigned>(A.L.vals_off + rows * kPageTokens * A.L.esize);
}

__device__ __forceinline__ void producer_page_ids(const DecodeArgs& A, const Ctrl& C, int g, int c1, bool active,
                                                  int& id0, int& id1, unsigned& n0, unsigned& n1)
{
    id0 = -1; id1 = -1; n0 = 0; n1 = 0;
    if (!active) return;
    const Segment s = locate(C.prefix, A.B, A.Hkv, g, c1);
    const int64_t row = (static_cast<int64_t>(s.b) * A.Hkv + s.h) * A.max_blocks;
    const int32_t* bt = A.block_table ? A.block_table + row : nullptr;       // no table: pages of a unit are consecutive
    id0 = bt ? bt[A.pps * s.i0] : static_cast<int>(row + A.pps * s.i0);
    if (A.pps == 2) {                                       // second page of the step, if the sequence has one
        const int len = clamp_len(A.lens[s.b], A.max_blocks * kPageTokens);
        if (2 * s.i0 + 1 < (len + kPageTokens - 1) / kPageTokens) {
            id1 = bt ? bt[2 * s.i0 + 1] : static_cast<int>(row + 2 * s.i0 + 1);
            if (id1 < 0 || id1 >= A.n_pool_pages) { record_error(A.status, SPARK_ERR_DEVICE_BOUNDS); id1 = 0; }
            n1 = page_copy_bytes(A, id1);
        }
    }
    if (id0 < 0 || id0 >= A.n_pool_pages) { record_error(A.status, SPARK_ERR_DEVICE_BOUNDS); id0 = 0; }
    n0 = page_copy_bytes(A, id0);
}

__device__ __forceinline__ void producer_loop(const DecodeArgs& A, const Ctrl& C, unsigned char* ring,
                                              int c0, int c1, int lane)
{
    const PageLayout L = A.L;
    const int NS = A.nslots, n_total = c1 - c0;
    const uint64_t policy = policy_evict_first();
    const bool owner = lane < NS;
    unsigned char* dst = ring + static_cast<size_t>(lane) * A.slot_stride;
    uint64_t* full = &C.full[owner ? lane : 0];
    uint64_t* empty = &C.empty[owner ? lane : 0];
    bool live = true;
    int last_round = -1;                                   // last revolution in which this lane issued
    int id0, id1;
    unsigned n0, n1;                                       // bytes to copy of the two pages
    producer_page_ids(A, C, c0 + lane, c1, owner && lane < n_total, id0, id1, n0, n1);
    for (int round = 0; round * NS < n_total; ++round) {
        const int n = round * NS + lane;
        bool pending = owner && n < n_total;
        const int cur0 = id0, cur1 = id1;
        const unsigned b0 = n0, b1 = n1;
        // next revolution's ids: the lookup waits for its block-table loads, so it runs before the poll
        // (hidden behind the wait for free slots) except in the first revolution, where every slot is
        // free and the copies go out first
        if (round > 0) producer_page_ids(A, C, c0 + n + NS, c1, owner && n + NS < n_total, id0, id1, n0, n1);
        WaitClock wc;
        while (__any_sync(kFull, pending)) {
            if (pending && (round == 0 || mbar_try_wait(empty, (round - 1) & 1))) {
                C.seq[lane] = round + 1;
                mbar_expect_tx(full, b0 + (cur1 >= 0 ? b1 : 0u));
                bulk_g2s(dst, A.pages + static_cast<int64_t>(cur0) * L.page_bytes, b0, full, policy);
                if (cur1 >= 0)
                    bulk_g2s(dst + L.page_bytes, A.pages + static_cast<int64_t>(cur1) * L.page_bytes, b1, full, policy);
                last_round = round;
                pending = false;
            }
            if (wc.expired() || *C.abort_flag) { live = false; break; }
        }
        if (!live) break;
        if (round == 0) producer_page_ids(A, C, c0 + n + NS, c1, owner && n + NS < n_total, id0, id1, n0, n1);
    }
    if (!live) {
        if (lane == 0) { *C.abort_flag = 1; record_error(A.status, SPARK_ERR_DEVICE_TIMEOUT); }
        if (last_round >= 0) {                             // let this lane's copy in flight land
            WaitClock wc;
            while (!wc.expired())
                if (mbar_try_wait(full, last_round & 1)) break;
        }
    }
}

// zero-length sequences: out = 0, lse = -inf (consumer threads)
template <int NT>
__device__ __forceinline__ void write_empty_sequences(const DecodeArgs& A, const int* prefix, int tid)
{
    for (int b = blockIdx.x; b < A.B; b += gridDim.x)
        if (prefix[b + 1] == prefix[b]) {
            for (int i = tid; i < A.Hq * kHeadDim; i += NT)
                A.out[static_cast<int64_t>(b) * A.Hq * kHeadDim + i] = 0.f;
            if (A.lse)
                for (int i = tid; i < A.Hq; i += NT)
                    A.lse[static_cast<int64_t>(b) * A.Hq + i] = -INFINITY;
        }
}

// Merge the per-warp states that the NW consumer warps have written to `merge`
// ([warp][G][kRec]: 128 unnormalised outputs, m, l) and publish the unit's result: directly when this
// CTA covers the whole unit, else as a partial followed by the last-arriver merge.  Called by all
// consumer threads after a consumer_sync(); ends with a consumer_sync().
//
// Both merges are laid out so that no thread walks a chain of dependent shared-memory loads: the
// log-sum-exp weights of the parts are computed once, by one warp per head with warp reductions, and the
// weighted sums then read independent operands.
template <int G, int NW>
__device__ __forceinline__ void merge_and_publish(const DecodeArgs& A, const Ctrl& C, float* merge,
                                                  const Segment& sg, int tid)
{
    constexpr int NT = NW * 32;
    static_assert(G <= NW && NW <= 32, "one warp per head computes the weights of up to 32 warps");
    const int b = sg.b, h = sg.h;
    const int warp = tid >> 5, lane = tid & 31;
    int first_cta, n_parts;
    unit_parts(*C.plan, sg.unit_start, sg.steps_b, first_cta, n_parts);
    const int unit = b * A.Hkv + h;
    static_assert(NW >= 2, "the heads' (M, L) live in the spare words of the first two warps' records");
    constexpr int kWt = kHeadDim + 2, kMl = kHeadDim + 3;     // spare words of a record
    // ---- weights of the warps: warp g serves head g, lane w holds warp w's (m, l) ----
    if (warp < G) {
        const float m = lane < NW ? merge[(lane * G + warp) * kRec + kHeadDim] : -INFINITY;
        const float l = lane < NW ? merge[(lane * G + warp) * kRec + kHeadDim + 1] : 0.f;
        float M = m;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFull, M, o));
        const float wt = (m == -INFINITY) ? 0.f : exp2f(m - M);
        float Ls = l * wt;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) Ls += __shfl_xor_sync(kFull, Ls, o);
        if (lane < NW) merge[(lane * G + warp) * kRec + kWt] = wt;
        if (lane == 0) { merge[warp * kRec + kMl] = M; merge[(G + warp) * kRec + kMl] = Ls; }
    }
    consumer_sync<NT>();
    // ---- weighted sums: a thread owns two channels of one head ----
    float* part_out = A.partials + static_cast<int64_t>(blockIdx.x + unit) * G * kRec;
    for (int idx = tid; idx < G * (kHeadDim / 2); idx += NT) {
        const int gg = idx / (kHeadDim / 2), c2 = idx - gg * (kHeadDim / 2);
        float2 v[NW];
#pragma unroll
        for (int w = 0; w < NW; ++w) v[w] = *reinterpret_cast<const float2*>(merge + (w * G + gg) * kRec + 2 * c2);
        float2 O = make_float2(0.f, 0.f);
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float f = merge[(w * G + gg) * kRec + kWt];
            O.x = fmaf(v[w].x, f, O.x);
            O.y = fmaf(v[w].y, f, O.y);
        }
        const float M = merge[gg * kRec + kMl], Ls = merge[(G + gg) * kRec + kMl];
        if (n_parts == 1) {
            const float inv = 1.0f / Ls;
            *reinterpret_cast<float2*>(A.out + (static_cast<int64_t>(b) * A.Hq + h * G + gg) * kHeadDim + 2 * c2) =
                make_float2(O.x * inv, O.y * inv);
            if (c2 == 0 && A.lse)
                A.lse[static_cast<int64_t>(b) * A.Hq + h * G + gg] = (M + log2f(Ls)) * kLn2;
        } else {
            *reinterpret_cast<float2*>(part_out + gg * kRec + 2 * c2) = O;
            if (c2 == 0) *reinterpret_cast<float2*>(part_out + gg * kRec + kHeadDim) = make_float2(M, Ls);
        }
    }
    if (n_parts > 1) {
        // The barrier orders every consumer thread's partial stores before thread 0's gpu-scope
        // release; the last arriver's acquire (same atomic) plus the next barrier orders its reads
        // after all partials.
        consumer_sync<NT>();
        if (tid == 0) {
            int old;
            asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(A.tickets + unit) : "memory");
            *C.last_flag = (old == n_parts - 1) ? 1 : 0;
        }
        consumer_sync<NT>();
        if (*C.last_flag) {
            // Last CTA of this unit: merge all partials.  Every load is issued before the first use:
            // thread (ph, g, c4) fetches channels 4*c4..4*c4+3 of head g for parts ph, ph+PH, ...;
            // meanwhile warp g turns the (m, l) pairs of head g into weights (lane = part) and the
            // head's (M, L).  After one barrier the weights are known, and the weighted sums are
            // reduced over ph through shared memory.
            constexpr int TPG = G * 32;                  // threads per part group
            constexpr int PH = NT / TPG;                 // part groups
            constexpr int kBatch = 8;
            constexpr int kMlRegs = kMaxCtas / 32;       // (m, l) pairs a lane may hold
            constexpr int64_t kStride = static_cast<int64_t>(G) * kRec;
            float* pw = merge;                           // [n_parts][G] weights, n_parts <= kMaxCtas
            float* pML = merge + kMaxCtas * G;           // [G][2]
            float4* red = reinterpret_cast<float4*>(merge + kMaxCtas * G * 2);
            const float* base = A.partials + static_cast<int64_t>(first_cta + unit) * G * kRec;
            const int ph = tid / TPG, rem = tid - ph * TPG, gg = rem >> 5, c4 = rem & 31;
            const bool worker = ph < PH;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int p0 = 0; p0 < n_parts; p0 += kBatch * PH) {
                float4 o4[kBatch];
#pragma unroll
                for (int k = 0; k < kBatch; ++k) {
                    const int p = p0 + k * PH + ph;
                    o4[k] = (worker && p < n_parts)
                                ? *reinterpret_cast<const float4*>(base + p * kStride + gg * kRec + 4 * c4)
                                : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                if (p0 == 0) {
                    if (warp < G) {
                        float2 ml[kMlRegs];
#pragma unroll
                        for (int k = 0; k < kMlRegs; ++k) {
                            const int p = k * 32 + lane;
                            ml[k] = p < n_parts ? *reinterpret_cast<const float2*>(base + p * kStride + warp * kRec + kHeadDim)
                                                : make_float2(-INFINITY, 0.f);
                        }
                        float M = -INFINITY;
#pragma unroll
                        for (int k = 0; k < kMlRegs; ++k) M = fmaxf(M, ml[k].x);
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFull, M, o));
                        float Ls = 0.f;
#pragma unroll
                        for (int k = 0; k < kMlRegs; ++k) {
                            const int p = k * 32 + lane;
                            const float wt = (ml[k].x == -INFINITY) ? 0.f : exp2f(ml[k].x - M);
                            Ls = fmaf(ml[k].y, wt, Ls);
                            if (p < n_parts) pw[p * G + warp] = wt;
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) Ls += __shfl_xor_sync(kFull, Ls, o);
                        if (lane == 0) { pML[2 * warp] = M; pML[2 * warp + 1] = Ls; }
                    }
                    consumer_sync<NT>();
                }
#pragma unroll
                for (int k = 0; k < kBatch; ++k) {
                    const int p = p0 + k * PH + ph;
                    if (worker && p < n_parts) {
                        const float f = pw[p * G + gg];
                        acc.x = fmaf(o4[k].x, f, acc.x); acc.y = fmaf(o4[k].y, f, acc.y);
                        acc.z = fmaf(o4[k].z, f, acc.z); acc.w = fmaf(o4[k].w, f, acc.w);
                    }
                }
            }
            if (PH > 1) {
                if (worker && ph > 0) red[tid] = acc;
                consumer_sync<NT>();
                if (ph == 0)
#pragma unroll
                    for (int k = 1; k < PH; ++k) {
                        const float4 v = red[k * TPG + tid];
                        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                    }
            }
            if (ph == 0) {
                const float M = pML[2 * gg], Ls = pML[2 * gg + 1];
                const float inv = 1.0f / Ls;
                *reinterpret_cast<float4*>(A.out + (static_cast<int64_t>(b) * A.Hq + h * G + gg) * kHeadDim + 4 * c4) =
                    make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
                if (c4 == 0 && A.lse)
                    A.lse[static_cast<int64_t>(b) * A.Hq + h * G + gg] = (M + log2f(Ls)) * kLn2;
            }
            if (tid == 0) A.tickets[unit] = 0;          // ready for the next call
        }
    }
    consumer_sync<NT>();
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Device properties the launchers need, looked up once per device and then served from a table
// (spark_decode.cu); `dev` is the current device.
struct DeviceInfo { int n_sms; int smem_optin; };
bool device_info(int* dev, DeviceInfo* info);

// Raises a kernel's dynamic shared-memory limit to the device maximum, once per device and kernel.
constexpr int kMaxDevices = 64;
template <typename Kernel> inline bool allow_max_smem(Kernel kernel, int dev, int smem_optin, unsigned char (&done)[kMaxDevices])
{
    if (dev < 0 || dev >= kMaxDevices) return false;
    if (done[dev]) return true;                           // a racing first call only repeats the same setting
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess) return false;
    done[dev] = 1;
    return true;
}

// per-dtype launchers (spark_decode.cu: fp32 storage, spark_decode_mma.cu: bf16 storage)
spark_status launch_decode_f32(int G, const DecodeArgs& A, int dev, const DeviceInfo& info, cudaStream_t stream);
spark_status launch_decode_bf16(int G, const DecodeArgs& A, int dev, const DeviceInfo& info, cudaStream_t stream);
spark_status launch_decode_bf16_sampled(int G, const DecodeArgs& A, int dev, const DeviceInfo& info, cudaStream_t stream);

}  // namespace spark
