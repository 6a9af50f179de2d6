// Decode attention over the packed SparK cache on the CUDA cores: fp32 storage with the degenerate recovery
// distribution, and either storage type with a SAMPLED recovery distribution (Sec. "Channel Recovery":
// Gaussian / Exponential; then the softmax attention of Sec. "Preliminaries"); also the dispatch of
// spark_decode_attn to the kernels.
//
// With a[j] = max(|q-bar_j|, eps) the reconstructed key is K~[t][j] = K[t][j] on kept channels and
// mu[t] / a[j] on pruned ones, so for one query head
//     q . K~[t] = sum_{j kept} q[j] * (K[t][j] - mu[t] / a[j])  +  mu[t] * sum_j q[j] / a[j].
// This kernel evaluates that form on the CUDA cores: a lane owns a token for the scores (it walks the set
// bits of the token's mask and gathers the query entries from a shared table) and four channels for
// P.V.  fp32 caches are the small high-precision configuration (the bf16 tensor-core kernel carries the
// bandwidth-bound workloads), so with the degenerate rule the table and the score sums are double: a
// score then carries one rounding (to fp32, before the exponential) instead of the ~1e-6 relative error
// of an fp32 sum over up to 128 cancelling terms, which at large logits was most of the output error.
//
// Sampled recovery (template parameter R = 1 Gaussian, 2 Exponential): every pruned entry of a token is a
// draw w~ from the distribution built on the token's all-channel statistics (mean, population deviation;
// App. "Caching Pruned Channel Statistics", stored per token in the page), and the recovered key is
// w~ / a[j].  The draw is a pure function of (seed, unit, token, channel) -- the splitmix64 mixer of a
// 64-bit counter, two 24-bit uniforms, Box-Muller or inversion -- so the recovered keys never change while
// the cache lives.  The algebraic folding of the degenerate rule does not apply: the lane walks all 128
// channels of its token, which makes this the method's slow variant (the paper's ablation also ranks it
// below the degenerate rule).
#include <type_traits>

#include "spark_decode_common.cuh"

namespace spark {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kDecodeThreads = kConsumerThreads + 32;     // + producer warp
constexpr int kStepTokens = 2 * kPageTokens;              // a lane per token: two pages per step

// one sampled saliency: Gaussian N(mu, sigma^2) by Box-Muller (R = 1) or Exponential with mean mu by
// inversion (R = 2), from the counter (unit, t, j)
// the 64 mixed bits of the counter (unit, t, j)
__device__ __forceinline__ unsigned long long draw_bits(unsigned seed, unsigned long long unit_t, int j)
{
    unsigned long long z = unit_t ^ static_cast<unsigned long long>(j);
    z += static_cast<unsigned long long>(seed) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

template <int R>
__device__ __forceinline__ float sample_saliency(unsigned seed, unsigned long long unit_t, int j, float mu, float sigma)
{
    const unsigned long long z = draw_bits(seed, unit_t, j);
    // (x + 0.5) / 2^24 with x < 2^24: the sum needs 25 bits, so it is formed in double and rounded once
    const float u1 = static_cast<float>((static_cast<double>(z >> 40) + 0.5) * (1.0 / 16777216.0));
    if (R == 2) return -mu * logf(u1);
    const float u2 = static_cast<float>((static_cast<double>((z >> 16) & 0xFFFFFFull) + 0.5) * (1.0 / 16777216.0));
    return fmaf(sigma * sqrtf(-2.0f * logf(u1)), cospif(2.0f * u2), mu);
}

// the same draw evaluated in double: fp32 storage, where the output is held to the fp32 bar
template <int R>
__device__ __forceinline__ double sample_saliency_f64(unsigned seed, unsigned long long unit_t, int j, float mu, float sigma)
{
    const unsigned long long z = draw_bits(seed, unit_t, j);
    const double u1 = (static_cast<double>(z >> 40) + 0.5) * (1.0 / 16777216.0);
    if (R == 2) return -static_cast<double>(mu) * log(u1);
    const double u2 = (static_cast<double>((z >> 16) & 0xFFFFFFull) + 0.5) * (1.0 / 16777216.0);
    return fma(static_cast<double>(sigma) * sqrt(-2.0 * log(u1)), cospi(2.0 * u2), static_cast<double>(mu));
}

template <typename E> __device__ __forceinline__ float load_query(const void* q, int64_t i);
template <> __device__ __forceinline__ float load_query<float>(const void* q, int64_t i) { return static_cast<const float*>(q)[i]; }
template <> __device__ __forceinline__ float load_query<__nv_bfloat16>(const void* q, int64_t i)
{
    return bf16_bits_to_float(static_cast<const unsigned short*>(q)[i]);
}

template <int G> struct SmemF32 {
    static constexpr int GP = ((G + 1 + 3) / 4) * 4;     // floats per table entry: G scaled queries + 1/a
    static constexpr int GPD = ((G + 1 + 1) / 2) * 2;    // doubles per table entry (degenerate rule: double table)
    static constexpr int GPP = ((G + 3) / 4) * 4;        // floats per probability entry
    static constexpr int kQtab = kCtrlBytes;
    static constexpr int kQsum = kQtab + kHeadDim * GPD * 8;     // sized for the double table (>= the float one)
    static constexpr int kPscr = kQsum + 64;             // Qsum: [8] double
    static constexpr int kMerge = kPscr + kConsumerWarps * 32 * GPP * 4;
    static constexpr int kFixed = (kMerge + merge_bytes(kConsumerWarps, G) + 127) / 128 * 128;   // prefix and ring start here
};

template <int G, typename E, int R>
__global__ void __launch_bounds__(kDecodeThreads, 1) decode_scalar_kernel(const DecodeArgs A)
{
    constexpr bool kBf16 = (sizeof(E) == 2);
    static_assert(!(kBf16 && R == 0), "bf16 storage with the degenerate rule runs on the tensor-core kernel");
    using S = SmemF32<G>;
    // table element: double with the degenerate rule (fp32 storage, the high-precision configuration), else float
    constexpr bool kDbl = (R == 0);
    using TabT = typename std::conditional<kDbl, double, float>::type;
    constexpr int GP = kDbl ? S::GPD : S::GP, GPP = S::GPP;
    extern __shared__ __align__(128) unsigned char smem[];
    const Ctrl C = make_ctrl(smem, A.prefix_off);
    TabT* qtab = reinterpret_cast<TabT*>(smem + S::kQtab);
    double* qsum = reinterpret_cast<double*>(smem + S::kQsum);
    float* pscr_all = reinterpret_cast<float*>(smem + S::kPscr);
    float* merge = reinterpret_cast<float*>(smem + S::kMerge);
    unsigned char* ring = smem + A.ring_off;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const PageLayout L = A.L;
    const int NS = A.nslots;
    const int max_tokens = A.max_blocks * kPageTokens;

    prefetch_block_table(A, tid, kDecodeThreads);
    if (tid == 0) pdl_launch_dependents();
    if (warp == kConsumerWarps) {
        producer_prologue(A, C, lane, kDecodeThreads);
        int p0, p1;
        cta_range(*C.plan, static_cast<int>(blockIdx.x), p0, p1);
        producer_loop(A, C, ring, p0, p1, lane);
        return;
    }
    consumer_wait_plan(kDecodeThreads);
    const int* prefix = C.prefix;
    int c0, c1;
    cta_range(*C.plan, static_cast<int>(blockIdx.x), c0, c1);
    pdl_dependency_wait();                                 // q, qnorm, out and the workspace from here on
    write_empty_sequences<kConsumerThreads>(A, prefix, tid);

    float* pscr = pscr_all + warp * 32 * GPP;
    int base = 0;                                          // ordinal (within this CTA) of the segment's first step
    for (int g = c0; g < c1;) {
        const Segment sg = locate(prefix, A.B, A.Hkv, g, c1);
        const int b = sg.b, h = sg.h;
        const int len = clamp_len(A.lens[b], max_tokens);

        // ---- per-unit table: entry j = { q_0[j]*c, ..., q_{G-1}[j]*c, 1/a[j] },  c = scale*log2(e)
        for (int idx = tid; idx < kHeadDim * GP; idx += kConsumerThreads) {
            const int j = idx / GP, e = idx - j * GP;
            TabT val = 0;
            if (e < G)
                val = static_cast<TabT>(load_query<E>(A.q, (static_cast<int64_t>(b) * A.Hq + h * G + e) * kHeadDim + j)) *
                      static_cast<TabT>(A.scale_log2e);
            else if (e == G)
                val = static_cast<TabT>(1) / static_cast<TabT>(A.qnorm[(static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim + j]);
            qtab[idx] = val;
        }
        consumer_sync<kConsumerThreads>();
        if (warp < G) {                                    // Qsum[g] = sum_j q_g[j]*c / a[j]
            double part = 0.0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const TabT* e = qtab + (lane * 4 + i) * GP;
                part += static_cast<double>(e[warp]) * static_cast<double>(e[G]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(kFull, part, o);
            if (lane == 0) qsum[warp] = part;
        }
        consumer_sync<kConsumerThreads>();

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
            const bool ok = slot_wait(C.full, C.seq, slot, n / NS, C.abort_flag, A.status);
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
                    const unsigned words[4] = {mk.x, mk.y, mk.z, mk.w};
                    // kept slot s of token p (see val_offset): fp32 rows hold token p at element p, bf16 rows at
                    // element (p & 7) * 2 + (p >> 3); rows are 16 elements apart
                    const unsigned char* vp = page + L.vals_off + (kBf16 ? ((p & 7) * 2 + (p >> 3)) * 2 : p * 4);
                    constexpr int kRowBytes = kPageTokens * static_cast<int>(sizeof(E));
                    // sampled rules: fp32 storage sums the score in double as well (bf16 storage: fp32 is ample)
                    using AccT = typename std::conditional<kBf16, float, double>::type;
                    AccT a[G];
#pragma unroll
                    for (int gg = 0; gg < G; ++gg) a[gg] = 0;
                    if constexpr (R == 0) {
                        // fp32 storage is the high-precision configuration: the score of a token is summed in
                        // double from a double table (products of two fp32 numbers are exact there), so that the
                        // error of the step is that of the exponentials and of the fp32 value sums alone
                        const double mu_d = static_cast<double>(*reinterpret_cast<const float*>(page + L.mu_off + p * 4));
                        double ad[G];
#pragma unroll
                        for (int gg = 0; gg < G; ++gg) ad[gg] = 0.0;
#pragma unroll
                        for (int wi = 0; wi < 4; ++wi) {
                            unsigned w = words[wi];
                            const double* tb = qtab + wi * 32 * GP;
                            while (w) {
                                const int bp = __ffs(w) - 1;
                                w &= w - 1;
                                const double* e = tb + bp * GP;
                                const float kv = *reinterpret_cast<const float*>(vp);
                                vp += kRowBytes;
                                double tv[GP];
#pragma unroll
                                for (int c2 = 0; c2 < GP / 2; ++c2) {
                                    const double2 f = reinterpret_cast<const double2*>(e)[c2];
                                    tv[2 * c2] = f.x; tv[2 * c2 + 1] = f.y;
                                }
                                const double x = fma(-mu_d, tv[G], static_cast<double>(kv));
#pragma unroll
                                for (int gg = 0; gg < G; ++gg) ad[gg] = fma(tv[gg], x, ad[gg]);
                            }
                        }
#pragma unroll
                        for (int gg = 0; gg < G; ++gg) s[gg] = static_cast<float>(fma(mu_d, qsum[gg], ad[gg]));
                    } else {
                        // sampled recovery: every channel contributes, kept ones their stored value, pruned
                        // ones a draw divided by a[j]
                        const float mean = *reinterpret_cast<const float*>(page + L.stats_off + p * 4);
                        const float dev = *reinterpret_cast<const float*>(page + L.stats_off + (kPageTokens + p) * 4);
                        const unsigned long long unit_t =
                            (static_cast<unsigned long long>(b * A.Hkv + h) << 40) ^
                            (static_cast<unsigned long long>(i * kStepTokens + lane) << 8);
#pragma unroll 1
                        for (int wi = 0; wi < 4; ++wi) {
                            const unsigned w = words[wi];
#pragma unroll 4
                            for (int bp = 0; bp < 32; ++bp) {
                                const int j = wi * 32 + bp;
                                const float* e = qtab + j * GP;
                                float tv[GP];
#pragma unroll
                                for (int c4 = 0; c4 < GP / 4; ++c4) {
                                    const float4 f = reinterpret_cast<const float4*>(e)[c4];
                                    tv[4 * c4] = f.x; tv[4 * c4 + 1] = f.y; tv[4 * c4 + 2] = f.z; tv[4 * c4 + 3] = f.w;
                                }
                                AccT x;
                                if ((w >> bp) & 1u) {
                                    x = kBf16 ? bf16_bits_to_float(*reinterpret_cast<const unsigned short*>(vp))
                                              : *reinterpret_cast<const float*>(vp);
                                    vp += kRowBytes;
                                } else if constexpr (kBf16) {
                                    x = sample_saliency<R>(A.seed, unit_t, j, mean, dev) * tv[G];
                                } else {
                                    x = sample_saliency_f64<R>(A.seed, unit_t, j, mean, dev) * static_cast<double>(tv[G]);
                                }
#pragma unroll
                                for (int gg = 0; gg < G; ++gg)
                                    a[gg] = fma(static_cast<AccT>(tv[gg]), x, a[gg]);
                            }
                        }
#pragma unroll
                        for (int gg = 0; gg < G; ++gg) s[gg] = static_cast<float>(a[gg]);
                    }
                } else {
#pragma unroll
                    for (int gg = 0; gg < G; ++gg) s[gg] = -INFINITY;
                }
                // ---------------- online softmax ----------------
#pragma unroll
                for (int gg = 0; gg < G; ++gg) {
                    float mt = s[gg];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, o));
                    const float m_new = fmaxf(m_run[gg], mt);
                    const float alpha = exp2f(m_run[gg] - m_new);   // 0 on the first step (m_run = -inf)
                    const float pg = exp2f(s[gg] - m_new);          // 0 for invalid lanes
                    l_run[gg] = fmaf(l_run[gg], alpha, pg);
                    m_run[gg] = m_new;
                    pscr[lane * GPP + gg] = pg;
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[gg][c] *= alpha;
                }
                __syncwarp();
                // ---------------- P.V: lane = channels 4*lane .. 4*lane+3 ----------------
                for (int t = 0; t < n_valid; ++t) {
                    const unsigned char* pg = sbase + (t >> 4) * L.page_bytes;
                    float vv[4];
                    if (!kBf16 && L.keep_v < kHeadDim) {   // pruned values (fp32 pages): this lane's nibble of the value mask
                        const int p = t & 15, wi = lane >> 3, sh = 4 * (lane & 7);
                        const uint4 vm = *reinterpret_cast<const uint4*>(pg + L.vmask_off + p * 16);
                        const unsigned word = wi == 0 ? vm.x : (wi == 1 ? vm.y : (wi == 2 ? vm.z : vm.w));
                        int slot = __popc(word & ((1u << sh) - 1u)) + (wi > 0 ? __popc(vm.x) : 0) +
                                   (wi > 1 ? __popc(vm.y) : 0) + (wi > 2 ? __popc(vm.z) : 0);
                        const unsigned nib = (word >> sh) & 0xfu;
                        const float* vb = reinterpret_cast<const float*>(pg + L.v_off) + p;    // slot s at vb[16 s]
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const bool on = (nib >> c) & 1u;
                            vv[c] = on ? vb[kPageTokens * slot] : 0.f;
                            slot += on ? 1 : 0;
                        }
                    } else if (kBf16) {                    // 16-byte chunks of a bf16 value row are stored swizzled
                        const uint2 r = *reinterpret_cast<const uint2*>(
                            pg + L.v_off + v_chunk_offset(2, t & 15, lane >> 1) + (lane & 1) * 8);
                        vv[0] = __uint_as_float(r.x << 16); vv[1] = __uint_as_float(r.x & 0xffff0000u);
                        vv[2] = __uint_as_float(r.y << 16); vv[3] = __uint_as_float(r.y & 0xffff0000u);
                    } else {
                        const float4 r = *reinterpret_cast<const float4*>(pg + L.v_off + (t & 15) * (kHeadDim * 4) + lane * 16);
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
            if (lane == 0) mbar_arrive(&C.empty[slot]);
        }

        // ---------------- hand the warp states to the merge ----------------
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
        consumer_sync<kConsumerThreads>();
        merge_and_publish<G, kConsumerWarps>(A, C, merge, sg, tid);
        g += sg.n;
        base += sg.n;
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
bool device_info(int* dev, DeviceInfo* info)
{
    static DeviceInfo table[kMaxDevices];
    static unsigned char known[kMaxDevices] = {};
    if (cudaGetDevice(dev) != cudaSuccess || *dev < 0 || *dev >= kMaxDevices) return false;
    if (!known[*dev]) {                                   // a racing first call writes the same values
        DeviceInfo d;
        if (cudaDeviceGetAttribute(&d.n_sms, cudaDevAttrMultiProcessorCount, *dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, *dev) != cudaSuccess)
            return false;
        table[*dev] = d;
        known[*dev] = 1;
    }
    *info = table[*dev];
    return true;
}

size_t decode_workspace_bytes(const spark_params& p)
{
    const int G = p.n_q_heads / p.n_kv_heads;
    const size_t units = static_cast<size_t>(p.batch) * p.n_kv_heads;
    size_t bytes = kWorkspaceHeader;
    bytes += align_up(units * sizeof(int), 256);
    bytes += (kMaxCtas + units) * G * kRec * sizeof(float);
    return align_up(bytes, 256);
}

template <int G, typename E, int R>
static spark_status launch_scalar(const DecodeArgs& A0, int dev, const DeviceInfo& info, cudaStream_t stream)
{
    static unsigned char smem_raised[kMaxDevices] = {};
    const int n_sms = info.n_sms, smem_optin = info.smem_optin;
    DecodeArgs A = A0;
    using S = SmemF32<G>;
    A.pps = 2;
    A.slot_stride = static_cast<int>(align_up(2 * static_cast<size_t>(A.L.page_bytes), 128));
    A.prefix_off = S::kFixed;
    A.ring_off = S::kFixed + prefix_bytes(A.B);
    int ns = (smem_optin - A.ring_off) / A.slot_stride;
    if (ns > kMaxSlots) ns = kMaxSlots;
    if (ns < 2) return SPARK_ERR_UNSUPPORTED;
    A.nslots = ns;
    const size_t smem = A.ring_off + static_cast<size_t>(ns) * A.slot_stride;
    if (!allow_max_smem(decode_scalar_kernel<G, E, R>, dev, smem_optin, smem_raised)) return SPARK_ERR_CUDA;
    const int grid = n_sms < kMaxCtas ? n_sms : kMaxCtas;
    return launch_decode_kernel(decode_scalar_kernel<G, E, R>, grid, kDecodeThreads, smem, stream, A) == cudaSuccess
               ? SPARK_OK : SPARK_ERR_CUDA;
}

template <typename E, int R>
static spark_status launch_scalar_g(int G, const DecodeArgs& A, int dev, const DeviceInfo& info, cudaStream_t stream)
{
    switch (G) {
        case 1: return launch_scalar<1, E, R>(A, dev, info, stream);
        case 2: return launch_scalar<2, E, R>(A, dev, info, stream);
        case 3: return launch_scalar<3, E, R>(A, dev, info, stream);
        case 4: return launch_scalar<4, E, R>(A, dev, info, stream);
        case 5: return launch_scalar<5, E, R>(A, dev, info, stream);
        case 6: return launch_scalar<6, E, R>(A, dev, info, stream);
        case 7: return launch_scalar<7, E, R>(A, dev, info, stream);
        case 8: return launch_scalar<8, E, R>(A, dev, info, stream);
        default: return SPARK_ERR_UNSUPPORTED;
    }
}

spark_status launch_decode_f32(int G, const DecodeArgs& A, int dev, const DeviceInfo& info, cudaStream_t stream)
{
    switch (A.L.recovery) {
        case SPARK_RECOVER_GAUSSIAN: return launch_scalar_g<float, 1>(G, A, dev, info, stream);
        case SPARK_RECOVER_EXPONENTIAL: return launch_scalar_g<float, 2>(G, A, dev, info, stream);
        default: return launch_scalar_g<float, 0>(G, A, dev, info, stream);
    }
}

// bf16 storage with a sampled recovery distribution (the degenerate rule runs on the tensor-core kernel)
spark_status launch_decode_bf16_sampled(int G, const DecodeArgs& A, int dev, const DeviceInfo& info, cudaStream_t stream)
{
    return A.L.recovery == SPARK_RECOVER_GAUSSIAN ? launch_scalar_g<__nv_bfloat16, 1>(G, A, dev, info, stream)
                                                  : launch_scalar_g<__nv_bfloat16, 2>(G, A, dev, info, stream);
}

size_t query_by_value_limit() { return kMaxQueryByValueBytes; }

spark_status launch_decode(const spark_params& p, const void* q, const void* pages,
                           const int32_t* block_table, int32_t max_blocks, const int32_t* packed_lens,
                           const float* qnorm, float* out, float* lse, void* workspace,
                           size_t workspace_bytes, cudaStream_t stream, int* launches, bool q_by_value)
{
    (void)workspace_bytes;
    int dev = 0;
    DeviceInfo info;
    if (!device_info(&dev, &info)) return SPARK_ERR_CUDA;
    const int G = p.n_q_heads / p.n_kv_heads;
    const size_t units = static_cast<size_t>(p.batch) * p.n_kv_heads;
    DecodeArgs A;
    A.q = q; A.pages = static_cast<const unsigned char*>(pages); A.block_table = block_table;
    A.max_blocks = max_blocks; A.lens = packed_lens; A.qnorm = qnorm; A.out = out; A.lse = lse;
    A.B = p.batch; A.Hq = p.n_q_heads; A.Hkv = p.n_kv_heads; A.n_pool_pages = p.n_pool_pages;
    A.L = make_layout(p);
    const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / sqrtf(static_cast<float>(p.head_dim));
    A.scale_log2e = scale * 1.4426950408889634f;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    A.status = reinterpret_cast<int*>(ws);
    A.tickets = reinterpret_cast<int*>(ws + kWorkspaceHeader);
    A.partials = reinterpret_cast<float*>(ws + kWorkspaceHeader + align_up(units * sizeof(int), 256));
    A.nslots = 0; A.slot_stride = 0; A.pps = 1; A.prefix_off = 0; A.ring_off = 0;
    A.overlap = (p.flags & SPARK_FLAG_OVERLAP_PREVIOUS) ? 1 : 0;
    A.seed = p.seed;
    A.q_by_value = q_by_value ? 1 : 0;
    A.page_rows = A.L.ragged ? reinterpret_cast<const int*>(A.pages + rows_offset(p.n_pool_pages, A.L.page_bytes)) : nullptr;
    if (q_by_value && (p.dtype != SPARK_BF16 || p.recovery != SPARK_RECOVER_DEGENERATE)) return SPARK_ERR_UNSUPPORTED;
    const spark_status st = (p.dtype != SPARK_BF16) ? launch_decode_f32(G, A, dev, info, stream)
                            : (p.recovery != SPARK_RECOVER_DEGENERATE) ? launch_decode_bf16_sampled(G, A, dev, info, stream)
                                                                       : launch_decode_bf16(G, A, dev, info, stream);
    if (st == SPARK_OK) ++*launches;
    return st;
}

}  // namespace spark
