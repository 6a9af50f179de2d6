// Decode attention over the packed SparK cache (Sec. "Channel Recovery", degenerate distribution, then
// the softmax attention of Sec. "Preliminaries").
//
// With a[j] = max(|q-bar_j|, eps) the reconstructed key is K~[t][j] = K[t][j] on kept channels and
// mu[t] / a[j] on pruned ones, so for one query head
//     q . K~[t] = sum_{j kept} q[j] * (K[t][j] - mu[t] / a[j])  +  mu[t] * sum_j q[j] / a[j].
// The kernel evaluates that form: only kept entries are touched and the second sum is one constant
// per (sequence, query head).
//
// Execution shape: a persistent grid of one CTA per SM.  The (sequence, KV head) units are cut into
// steps of two pages (32 tokens); the steps of all units form one line that is divided evenly among
// the CTAs, so a CTA owns a contiguous run of steps that may cross unit boundaries.  Inside a CTA one
// producer warp streams pages into a shared-memory ring with bulk asynchronous copies that signal
// mbarriers; eight consumer warps each take whole steps (lane = token for the scores, lane = four
// channels for P.V) and keep an online-softmax state.  At the end of a unit's run the warps are
// merged by log-sum-exp; if several CTAs share the unit each writes a partial and the last to arrive
// (an atomic ticket, no waiting) merges them.  All G query heads of a KV head are served from one
// read of its pages.
#include "spark_common.cuh"

namespace spark {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kDecodeThreads = kConsumerThreads + 32;
constexpr int kMaxSlots = 16;
constexpr int kStepTokens = 2 * kPageTokens;
constexpr unsigned kSpinLimit = 1u << 20;       // bounded mbarrier waits
constexpr unsigned kFull = 0xffffffffu;
constexpr int kRec = kHeadDim + 4;           // floats per (head) record: 128 accumulators, running max, running sum, pad

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

// ---- shared-memory carve-up ---------------------------------------------------------------------
template <int G> struct Smem {
    static constexpr int GP = ((G + 1 + 3) / 4) * 4;     // floats per table entry: G scaled queries + 1/a
    static constexpr int GPP = ((G + 3) / 4) * 4;        // floats per probability entry
    static constexpr int kCtrl = 0;                       // full[16], empty[16], flags
    static constexpr int kPrefix = 512;
    static constexpr int kQtab = kPrefix + ((kMaxBatch + 1) * 4 + 15) / 16 * 16;
    static constexpr int kQsum = kQtab + kHeadDim * GP * 4;
    static constexpr int kPscr = kQsum + 32;
    static constexpr int kMerge = kPscr + kConsumerWarps * 32 * GPP * 4;
    static constexpr int kRing = (kMerge + kConsumerWarps * G * kRec * 4 + 127) / 128 * 128;
};

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
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, unsigned bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void consumer_sync()
{
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}

__device__ __forceinline__ int steps_of(int len)
{
    return ((len + kPageTokens - 1) / kPageTokens + 1) >> 1;
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

template <typename E, int G>
__global__ void __launch_bounds__(kDecodeThreads, 1) decode_kernel(const DecodeArgs A)
{
    using S = Smem<G>;
    constexpr int GP = S::GP, GPP = S::GPP;
    constexpr bool kBf16 = (sizeof(E) == 2);
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + S::kCtrl);
    uint64_t* empty = full + kMaxSlots;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + S::kCtrl + 256);
    volatile int* last_flag = reinterpret_cast<volatile int*>(smem + S::kCtrl + 260);
    int* prefix = reinterpret_cast<int*>(smem + S::kPrefix);
    float* qtab = reinterpret_cast<float*>(smem + S::kQtab);
    float* qsum = reinterpret_cast<float*>(smem + S::kQsum);
    float* pscr_all = reinterpret_cast<float*>(smem + S::kPscr);
    float* merge = reinterpret_cast<float*>(smem + S::kMerge);
    unsigned char* ring = smem + S::kRing;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const PageLayout L = A.L;
    const int NS = A.nslots;
    const int max_tokens = A.max_blocks * kPageTokens;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        *abort_flag = 0;
        *last_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // steps-per-sequence prefix (warp 0, 32 sequences per round)
    if (warp == 0) {
        int running = 0;
        for (int b0 = 0; b0 < A.B; b0 += 32) {
            const int b = b0 + lane;
            int st = 0;
            if (b < A.B) {
                int len = A.lens[b];
                if (len < 0 || len > max_tokens) {
                    record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
                    len = len < 0 ? 0 : max_tokens;
                }
                st = steps_of(len);
            }
            int inc = st;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(kFull, inc, o);
                if (lane >= o) inc += n;
            }
            if (b < A.B) prefix[b + 1] = running + inc;
            running += __shfl_sync(kFull, inc, 31);
        }
        if (lane == 0) prefix[0] = 0;
    }
    __syncthreads();

    const int total = A.Hkv * prefix[A.B];
    const int nct = static_cast<int>(gridDim.x);
    const int chunk = (total + nct - 1) / nct;
    const int c0 = min(total, static_cast<int>(blockIdx.x) * chunk);
    const int c1 = min(total, c0 + chunk);
    const int n_total = c1 - c0;

    // ================================ producer warp ================================
    if (warp == kConsumerWarps) {
        bool live = true;
        int issued = 0;
        for (int n0 = 0; n0 < n_total; n0 += 32) {
            const int n = n0 + lane;
            int id0 = -1, id1 = -1;
            if (n < n_total) {
                const Segment s = locate(prefix, A.B, A.Hkv, c0 + n, c1);
                int len = A.lens[s.b];
                len = len < 0 ? 0 : (len > max_tokens ? max_tokens : len);
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
                    if (round > 0) live = mbar_wait(&empty[slot], (round - 1) & 1, abort_flag, A.status);
                    if (live) {
                        unsigned char* dst = ring + static_cast<size_t>(slot) * A.slot_stride;
                        const unsigned bytes = L.page_bytes * (p1 >= 0 ? 2u : 1u);
                        mbar_expect_tx(&full[slot], bytes);
                        bulk_g2s(dst, A.pages + static_cast<int64_t>(p0) * L.page_bytes, L.page_bytes, &full[slot]);
                        if (p1 >= 0)
                            bulk_g2s(dst + L.page_bytes, A.pages + static_cast<int64_t>(p1) * L.page_bytes,
                                     L.page_bytes, &full[slot]);
                        ++issued;
                    }
                }
            }
        }
        // after a give-up: let the copies already in flight land before the CTA may exit
        if (lane == 0 && !live) {
            for (int nn = max(0, issued - NS); nn < issued; ++nn) {
                uint64_t* bar = &full[nn % NS];
                const unsigned parity = (nn / NS) & 1;
                for (unsigned it = 0; it < kSpinLimit; ++it)
                    if (mbar_try_wait(bar, parity)) break;
            }
        }
        return;
    }

    // ================================ consumer warps ================================
    // zero-length sequences: out = 0, lse = -inf
    for (int b = blockIdx.x; b < A.B; b += nct)
        if (prefix[b + 1] == prefix[b]) {
            for (int i = tid; i < A.Hq * kHeadDim; i += kConsumerThreads)
                A.out[static_cast<int64_t>(b) * A.Hq * kHeadDim + i] = 0.f;
            if (A.lse)
                for (int i = tid; i < A.Hq; i += kConsumerThreads)
                    A.lse[static_cast<int64_t>(b) * A.Hq + i] = -INFINITY;
        }

    float* pscr = pscr_all + warp * 32 * GPP;
    int base = 0;                                          // ordinal (within this CTA) of the segment's first step
    for (int g = c0; g < c1;) {
        const Segment sg = locate(prefix, A.B, A.Hkv, g, c1);
        const int b = sg.b, h = sg.h;
        int len = A.lens[b];
        len = len < 0 ? 0 : (len > max_tokens ? max_tokens : len);

        // ---- per-unit table: entry j = { q_0[j]*c, ..., q_{G-1}[j]*c, 1/a[j] },  c = scale*log2(e)
        for (int idx = tid; idx < kHeadDim * GP; idx += kConsumerThreads) {
            const int j = idx / GP, e = idx - j * GP;
            float val = 0.f;
            if (e < G)
                val = Elem<E>::load(A.q, (static_cast<int64_t>(b) * A.Hq + h * G + e) * kHeadDim + j) * A.scale_log2e;
            else if (e == G)
                val = 1.0f / A.qnorm[(static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim + j];
            qtab[idx] = val;
        }
        consumer_sync();
        if (warp < G) {                                    // Qsum[g] = sum_j q_g[j]*c / a[j]
            double part = 0.0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float* e = qtab + (lane * 4 + i) * GP;
                part += static_cast<double>(e[warp]) * static_cast<double>(e[G]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(kFull, part, o);
            if (lane == 0) qsum[warp] = static_cast<float>(part);
        }
        consumer_sync();

        float m_run[G], l_run[G], acc[G][4];
#pragma unroll
        for (int gg = 0; gg < G; ++gg) {
            m_run[gg] = -INFINITY;
            l_run[gg] = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[gg][c] = 0.f;
        }

        // first ordinal >= base that this warp owns
        int n = base + ((warp - base) % kConsumerWarps + kConsumerWarps) % kConsumerWarps;
        for (; n < base + sg.n; n += kConsumerWarps) {
            const int i = sg.i0 + (n - base);
            const int slot = n % NS;
            const bool ok = mbar_wait(&full[slot], (n / NS) & 1, abort_flag, A.status);
            const unsigned char* sbase = ring + static_cast<size_t>(slot) * A.slot_stride;
            const int n_valid = min(kStepTokens, len - i * kStepTokens);
            if (ok) {
                // ---------------- scores: lane = token ----------------
                float s[G];
                const bool valid = lane < n_valid;
                if (valid) {
                    const unsigned char* page = sbase + (lane >> 4) * L.page_bytes;
                    const int p = lane & 15;
                    const uint4 mk = *reinterpret_cast<const uint4*>(page + L.mask_off + p * 16);
                    const float mu = *reinterpret_cast<const float*>(page + L.mu_off + p * 4);
                    const unsigned words[4] = {mk.x, mk.y, mk.z, mk.w};
                    const unsigned char* vp = page + p * 4;
                    float a[G];
#pragma unroll
                    for (int gg = 0; gg < G; ++gg) a[gg] = 0.f;
                    int slot_i = 0;
#pragma unroll
                    for (int wi = 0; wi < 4; ++wi) {
                        unsigned w = words[wi];
                        const float* tb = qtab + wi * 32 * GP;
                        while (w) {
                            const int bp = __ffs(w) - 1;
                            w &= w - 1;
                            const float* e = tb + bp * GP;
                            float kv;
                            if (kBf16)
                                kv = bf16_bits_to_float(*reinterpret_cast<const unsigned short*>(
                                    vp + (slot_i >> 1) * 64 + (slot_i & 1) * 2));
                            else
                                kv = *reinterpret_cast<const float*>(vp + slot_i * 64);
                            ++slot_i;
                            float tv[GP];
#pragma unroll
                            for (int c4 = 0; c4 < GP / 4; ++c4) {
                                const float4 f = reinterpret_cast<const float4*>(e)[c4];
                                tv[4 * c4] = f.x; tv[4 * c4 + 1] = f.y; tv[4 * c4 + 2] = f.z; tv[4 * c4 + 3] = f.w;
                            }
                            const float x = fmaf(-mu, tv[G], kv);
#pragma unroll
                            for (int gg = 0; gg < G; ++gg) a[gg] = fmaf(tv[gg], x, a[gg]);
                        }
                    }
#pragma unroll
                    for (int gg = 0; gg < G; ++gg) s[gg] = fmaf(mu, qsum[gg], a[gg]);
                } else {
#pragma unroll
                    for (int gg = 0; gg < G; ++gg) s[gg] = -INFINITY;
                }
                // ---------------- online softmax ----------------
                float alpha[G];
#pragma unroll
                for (int gg = 0; gg < G; ++gg) {
                    float mt = s[gg];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, o));
                    const float m_new = fmaxf(m_run[gg], mt);
                    alpha[gg] = exp2f(m_run[gg] - m_new);         // 0 on the first step (m_run = -inf)
                    const float pg = exp2f(s[gg] - m_new);        // 0 for invalid lanes
                    l_run[gg] = fmaf(l_run[gg], alpha[gg], pg);
                    m_run[gg] = m_new;
                    pscr[lane * GPP + gg] = pg;
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[gg][c] *= alpha[gg];
                }
                __syncwarp();
                // ---------------- P.V: lane = channels 4*lane .. 4*lane+3 ----------------
                for (int t = 0; t < n_valid; ++t) {
                    const unsigned char* vrow = sbase + (t >> 4) * L.page_bytes + L.v_off +
                                                (t & 15) * (kHeadDim * static_cast<int>(sizeof(E)));
                    float vv[4];
                    if (kBf16) {
                        const uint2 r = *reinterpret_cast<const uint2*>(vrow + lane * 8);
                        vv[0] = __uint_as_float(r.x << 16); vv[1] = __uint_as_float(r.x & 0xffff0000u);
                        vv[2] = __uint_as_float(r.y << 16); vv[3] = __uint_as_float(r.y & 0xffff0000u);
                    } else {
                        const float4 r = *reinterpret_cast<const float4*>(vrow + lane * 16);
                        vv[0] = r.x; vv[1] = r.y; vv[2] = r.z; vv[3] = r.w;
                    }
                    float pv[GPP];
#pragma unroll
                    for (int c4 = 0; c4 < GPP / 4; ++c4) {
                        const float4 f = reinterpret_cast<const float4*>(pscr + t * GPP)[c4];
                        pv[4 * c4] = f.x; pv[4 * c4 + 1] = f.y; pv[4 * c4 + 2] = f.z; pv[4 * c4 + 3] = f.w;
                    }
#pragma unroll
                    for (int gg = 0; gg < G; ++gg)
#pragma unroll
                        for (int c = 0; c < 4; ++c) acc[gg][c] = fmaf(pv[gg], vv[c], acc[gg][c]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[slot]);
        }

        // ---------------- merge the warps of this CTA ----------------
        float* mine = merge + warp * G * kRec;
#pragma unroll
        for (int gg = 0; gg < G; ++gg) {
            float lsum = l_run[gg];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(kFull, lsum, o);
            *reinterpret_cast<float4*>(mine + gg * kRec + lane * 4) =
                make_float4(acc[gg][0], acc[gg][1], acc[gg][2], acc[gg][3]);
            if (lane == 0) {
                mine[gg * kRec + kHeadDim] = m_run[gg];
                mine[gg * kRec + kHeadDim + 1] = lsum;
            }
        }
        consumer_sync();

        const int unit_end = sg.unit_start + sg.steps_b;
        const int first_cta = sg.unit_start / chunk, last_cta = (unit_end - 1) / chunk;
        const int n_parts = last_cta - first_cta + 1;
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
                    A.lse[static_cast<int64_t>(b) * A.Hq + h * G + gg] = (M + log2f(Ls)) * 0.6931471805599453f;
            } else {
                part_out[gg * kRec + c] = O;
                if (c == 0) { part_out[gg * kRec + kHeadDim] = M; part_out[gg * kRec + kHeadDim + 1] = Ls; }
            }
        }
        if (n_parts > 1) {
            __threadfence();
            consumer_sync();
            if (tid == 0) {
                const int old = atomicAdd(&A.tickets[unit], 1);
                *last_flag = (old == n_parts - 1) ? 1 : 0;
            }
            consumer_sync();
            if (*last_flag) {                              // last CTA of this unit: merge all partials
                __threadfence();
                for (int idx = tid; idx < G * kHeadDim; idx += kConsumerThreads) {
                    const int gg = idx / kHeadDim, c = idx - gg * kHeadDim;
                    float M = -INFINITY;
                    for (int pc = first_cta; pc <= last_cta; ++pc)
                        M = fmaxf(M, __ldcg(A.partials + (static_cast<int64_t>(pc + unit) * G + gg) * kRec + kHeadDim));
                    float Ls = 0.f, O = 0.f;
                    for (int pc = first_cta; pc <= last_cta; ++pc) {
                        const float* r = A.partials + (static_cast<int64_t>(pc + unit) * G + gg) * kRec;
                        const float f = exp2f(__ldcg(r + kHeadDim) - M);
                        Ls = fmaf(__ldcg(r + kHeadDim + 1), f, Ls);
                        O = fmaf(__ldcg(r + c), f, O);
                    }
                    A.out[(static_cast<int64_t>(b) * A.Hq + h * G + gg) * kHeadDim + c] = O / Ls;
                    if (c == 0 && A.lse)
                        A.lse[static_cast<int64_t>(b) * A.Hq + h * G + gg] = (M + log2f(Ls)) * 0.6931471805599453f;
                }
                if (tid == 0) A.tickets[unit] = 0;        // ready for the next call
            }
        }
        consumer_sync();
        g += sg.n;
        base += sg.n;
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

size_t decode_workspace_bytes(const spark_params& p)
{
    const int G = p.n_q_heads / p.n_kv_heads;
    const size_t units = static_cast<size_t>(p.batch) * p.n_kv_heads;
    size_t bytes = kWorkspaceHeader;
    bytes += align_up(units * sizeof(int), 256);
    bytes += (kMaxCtas + units) * G * kRec * sizeof(float);
    return align_up(bytes, 256);
}

template <typename E, int G>
static spark_status launch_one(const DecodeArgs& A0, int n_sms, int smem_optin, cudaStream_t stream)
{
    DecodeArgs A = A0;
    using S = Smem<G>;
    A.slot_stride = static_cast<int>(align_up(2 * static_cast<size_t>(A.L.page_bytes), 128));
    int ns = (smem_optin - S::kRing) / A.slot_stride;
    if (ns > kMaxSlots) ns = kMaxSlots;
    if (ns < 2) return SPARK_ERR_UNSUPPORTED;
    A.nslots = ns;
    const size_t smem = S::kRing + static_cast<size_t>(ns) * A.slot_stride;
    if (cudaFuncSetAttribute(decode_kernel<E, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(smem)) != cudaSuccess)
        return SPARK_ERR_CUDA;
    const int grid = n_sms < kMaxCtas ? n_sms : kMaxCtas;
    decode_kernel<E, G><<<grid, kDecodeThreads, smem, stream>>>(A);
    return cudaGetLastError() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

template <typename E>
static spark_status launch_g(int G, const DecodeArgs& A, int n_sms, int smem_optin, cudaStream_t stream)
{
    switch (G) {
        case 1: return launch_one<E, 1>(A, n_sms, smem_optin, stream);
        case 2: return launch_one<E, 2>(A, n_sms, smem_optin, stream);
        case 3: return launch_one<E, 3>(A, n_sms, smem_optin, stream);
        case 4: return launch_one<E, 4>(A, n_sms, smem_optin, stream);
        case 5: return launch_one<E, 5>(A, n_sms, smem_optin, stream);
        case 6: return launch_one<E, 6>(A, n_sms, smem_optin, stream);
        case 7: return launch_one<E, 7>(A, n_sms, smem_optin, stream);
        case 8: return launch_one<E, 8>(A, n_sms, smem_optin, stream);
        default: return SPARK_ERR_UNSUPPORTED;
    }
}

spark_status launch_decode(const spark_params& p, const void* q, const void* pages,
                           const int32_t* block_table, int32_t max_blocks, const int32_t* packed_lens,
                           const float* qnorm, float* out, float* lse, void* workspace,
                           size_t workspace_bytes, cudaStream_t stream, int* launches)
{
    (void)workspace_bytes;
    int dev = 0, n_sms = 0, smem_optin = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
        return SPARK_ERR_CUDA;
    const int G = p.n_q_heads / p.n_kv_heads;
    const size_t units = static_cast<size_t>(p.batch) * p.n_kv_heads;
    DecodeArgs A;
    A.q = q; A.pages = static_cast<const unsigned char*>(pages); A.block_table = block_table;
    A.max_blocks = max_blocks; A.lens = packed_lens; A.qnorm = qnorm; A.out = out; A.lse = lse;
    A.B = p.batch; A.Hq = p.n_q_heads; A.Hkv = p.n_kv_heads; A.n_pool_pages = p.n_pool_pages;
    A.L = make_layout(p.dtype, p.keep);
    const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / sqrtf(static_cast<float>(p.head_dim));
    A.scale_log2e = scale * 1.4426950408889634f;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    A.status = reinterpret_cast<int*>(ws);
    A.tickets = reinterpret_cast<int*>(ws + kWorkspaceHeader);
    A.partials = reinterpret_cast<float*>(ws + kWorkspaceHeader + align_up(units * sizeof(int), 256));
    A.nslots = 0; A.slot_stride = 0;
    spark_status st = (p.dtype == SPARK_BF16)
                          ? launch_g<__nv_bfloat16>(G, A, n_sms, smem_optin, stream)
                          : launch_g<float>(G, A, n_sms, smem_optin, stream);
    if (st == SPARK_OK) ++*launches;
    return st;
}

}  // namespace spark
