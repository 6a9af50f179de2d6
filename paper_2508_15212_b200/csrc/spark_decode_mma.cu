// Decode attention over the packed SparK cache, bf16 storage (Sec. "Channel Recovery", degenerate
// distribution, then the softmax attention of Sec. "Preliminaries").
//
// For one query head, with a[j] = max(|q-bar_j|, eps) and q'[j] = q[j] / a[j]:
//     q . K~[t] = sum_{j kept} q[j] K[t][j]  +  mu[t] * ( sum_j q'[j]  -  sum_{j kept} q'[j] ).
// Both kept-channel sums are contractions over the 128 channels of [heads x channels] by
// [channels x tokens], so they run on the tensor cores (mma.sync m16n8k16, bf16 in, fp32 out):
//   - first operand rows: the G query heads (bf16, exact) for the first sum; q' split into a bf16 high
//     and low part (rows r and r+8) for the second;
//   - second operand: the token's kept values expanded to dense form for the first sum, and the
//     token's mask as 0/1 for the second.  The expansion happens in registers: the four lanes that
//     hold a token's column each own one 32-bit mask word, walk its eight nibbles, and pull the next
//     kept value from shared memory for every set bit.  The channel order inside a k-step is a fixed
//     permutation (lane c, step s  <->  channels 32c+4s .. 32c+4s+3) applied to both operands.
// P.V is the third contraction: probabilities (bf16 high and low parts in rows r and r+8, so the
// product keeps ~16 mantissa bits) by value rows fetched with transposing matrix loads; the value rows
// are stored chunk-swizzled in the page so those loads are conflict free.  Softmax statistics and all
// accumulators are fp32.
#include "spark_decode_common.cuh"

namespace spark {

template <int G> struct SmemBf16 {
    static constexpr int kTab = kCtrlBytes + kPrefixBytes;                       // q, q' high, q' low: 3 x [G][128] bf16
    static constexpr int kQsum = kTab + 3 * G * kHeadDim * 2;                    // [8] float
    static constexpr int kMerge = kQsum + 32;
    static constexpr int kRing = (kMerge + kConsumerWarps * G * kRec * 4 + 127) / 128 * 128;
};

__device__ __forceinline__ void mma_bf16(float (&d)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                         unsigned b0, unsigned b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4_trans(unsigned (&r)[4], unsigned smem_addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_addr));
}

__device__ __forceinline__ unsigned lds_u32(unsigned addr)
{
    unsigned v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ float2 lds_f32x2(unsigned addr)
{
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds_u32x4(unsigned addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ unsigned pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const unsigned*>(&v);
}

__device__ __forceinline__ float bf16_round(float x)
{
    return __bfloat162float(__float2bfloat16_rn(x));
}

// One mask nibble (bits b0m..b3m of word w) -> the second-operand registers of a k-step:
//   k0,k1 : the nibble's kept values in dense positions (zero where pruned); `addr` is the shared
//           address of the token's next unread kept value (rows of 32 bytes) and advances per set bit;
//   m0,m1 : the nibble as 0/1 in bf16 (1.0 = 0x3F80).
// Predicated loads, no branches.
__device__ __forceinline__ void expand_nibble(unsigned w, unsigned b0m, unsigned b1m, unsigned b2m, unsigned b3m,
                                              unsigned& addr, unsigned& k0, unsigned& k1, unsigned& m0, unsigned& m1)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p0, p1, p2, p3;\n\t"
        ".reg .b32 t0, t1, t2, t3;\n\t"
        ".reg .b16 h0, h1, h2, h3;\n\t"
        "and.b32 t0, %5, %6;\n\t"
        "and.b32 t1, %5, %7;\n\t"
        "and.b32 t2, %5, %8;\n\t"
        "and.b32 t3, %5, %9;\n\t"
        "setp.ne.u32 p0, t0, 0;\n\t"
        "setp.ne.u32 p1, t1, 0;\n\t"
        "setp.ne.u32 p2, t2, 0;\n\t"
        "setp.ne.u32 p3, t3, 0;\n\t"
        "mov.b16 h0, 0;\n\t"
        "mov.b16 h1, 0;\n\t"
        "mov.b16 h2, 0;\n\t"
        "mov.b16 h3, 0;\n\t"
        "@p0 ld.shared.u16 h0, [%4];\n\t"
        "@p0 add.u32 %4, %4, 32;\n\t"
        "@p1 ld.shared.u16 h1, [%4];\n\t"
        "@p1 add.u32 %4, %4, 32;\n\t"
        "@p2 ld.shared.u16 h2, [%4];\n\t"
        "@p2 add.u32 %4, %4, 32;\n\t"
        "@p3 ld.shared.u16 h3, [%4];\n\t"
        "@p3 add.u32 %4, %4, 32;\n\t"
        "mov.b32 %0, {h0, h1};\n\t"
        "mov.b32 %1, {h2, h3};\n\t"
        "selp.b32 %2, 0x3F80, 0, p0;\n\t"
        "selp.b32 %3, 0x3F80, 0, p2;\n\t"
        "@p1 or.b32 %2, %2, 0x3F800000;\n\t"
        "@p3 or.b32 %3, %3, 0x3F800000;\n\t"
        "}"
        : "=&r"(k0), "=&r"(k1), "=&r"(m0), "=&r"(m1), "+r"(addr)
        : "r"(w), "r"(b0m), "r"(b1m), "r"(b2m), "r"(b3m));
}

template <int G>
__global__ void __launch_bounds__(kDecodeThreads, 1) decode_bf16_kernel(const DecodeArgs A)
{
    using S = SmemBf16<G>;
    extern __shared__ __align__(128) unsigned char smem[];
    const Ctrl C = make_ctrl(smem);
    unsigned char* tab = smem + S::kTab;
    float* qsum_s = reinterpret_cast<float*>(smem + S::kQsum);
    float* merge = reinterpret_cast<float*>(smem + S::kMerge);
    unsigned char* ring = smem + S::kRing;
    const unsigned ring_u = smem_u32(ring);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const PageLayout L = A.L;
    const int NS = A.nslots;
    const int max_tokens = A.max_blocks * kPageTokens;

    decode_prologue(A, C, tid);
    const int* prefix = C.prefix;
    int c0, c1;
    cta_range(*C.plan, static_cast<int>(blockIdx.x), c0, c1);

#ifdef SPARK_CTA_TIMING
    unsigned long long t_start = 0, t_first = 0, t_probe[12];
    int n_probe = 0;
    for (int i = 0; i < 12; ++i) t_probe[i] = 0;
#define SPARK_PROBE() do { if (tid == 0 && n_probe < 12) { asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_probe[n_probe])); ++n_probe; } } while (0)
    if (tid == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_start));
#else
#define SPARK_PROBE() do { } while (0)
#endif
    if (warp == kConsumerWarps) {
        producer_loop(A, C, ring, c0, c1, lane);
        return;
    }
    write_empty_sequences(A, prefix, tid);

    const int c = lane & 3, r = lane >> 2;                 // quad lane / fragment row (= token column)
    const bool row_ok = r < G;
    int base = 0;
    for (int g = c0; g < c1;) {
        const Segment sg = locate(prefix, A.B, A.Hkv, g, c1);
        const int b = sg.b, h = sg.h;
        const int len = clamp_len(A.lens[b], max_tokens);

        // ---- per-unit tables, built once per CTA: warp `hd` prepares query head hd ----
        //   tab[0][hd][j] = q[j] (bf16 as stored), tab[1] / tab[2] = bf16 high / low part of q[j] / a[j],
        //   qsum_s[hd]    = sum over all 128 channels of the 16-bit q' (so kept terms cancel exactly).
        if (warp < G) {
            const uint2 qr = *reinterpret_cast<const uint2*>(
                static_cast<const unsigned short*>(A.q) +
                (static_cast<int64_t>(b) * A.Hq + h * G + warp) * kHeadDim + 4 * lane);
            const float4 a4 = *reinterpret_cast<const float4*>(
                A.qnorm + (static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim + 4 * lane);
            const float qf[4] = {__uint_as_float(qr.x << 16), __uint_as_float(qr.x & 0xffff0000u),
                                 __uint_as_float(qr.y << 16), __uint_as_float(qr.y & 0xffff0000u)};
            const float av[4] = {a4.x, a4.y, a4.z, a4.w};
            float hi[4], lo[4];
            double part = 0.0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float qp = qf[e] / av[e];
                hi[e] = bf16_round(qp);
                lo[e] = bf16_round(qp - hi[e]);
                part += static_cast<double>(hi[e]) + static_cast<double>(lo[e]);
            }
            unsigned char* row = tab + warp * (kHeadDim * 2) + lane * 8;
            *reinterpret_cast<uint2*>(row) = qr;
            *reinterpret_cast<uint2*>(row + G * kHeadDim * 2) = make_uint2(pack_bf16(hi[0], hi[1]), pack_bf16(hi[2], hi[3]));
            *reinterpret_cast<uint2*>(row + 2 * G * kHeadDim * 2) = make_uint2(pack_bf16(lo[0], lo[1]), pack_bf16(lo[2], lo[3]));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(kFull, part, o);
            if (lane == 0) qsum_s[warp] = static_cast<float>(part);
        }
        consumer_sync();
        // first-operand fragments of this thread: Aq[2s], Aq[2s+1] = q[row r][32c+4s .. +3], same for q' parts
        unsigned Aq[16], Ahi[16], Alo[16];
        float qsum = 0.f;
        if (row_ok) {
            const unsigned t0 = smem_u32(tab) + r * (kHeadDim * 2) + c * 64;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 u = lds_u32x4(t0 + i * 16);
                const uint4 v = lds_u32x4(t0 + G * kHeadDim * 2 + i * 16);
                const uint4 x = lds_u32x4(t0 + 2 * G * kHeadDim * 2 + i * 16);
                Aq[4 * i] = u.x; Aq[4 * i + 1] = u.y; Aq[4 * i + 2] = u.z; Aq[4 * i + 3] = u.w;
                Ahi[4 * i] = v.x; Ahi[4 * i + 1] = v.y; Ahi[4 * i + 2] = v.z; Ahi[4 * i + 3] = v.w;
                Alo[4 * i] = x.x; Alo[4 * i + 1] = x.y; Alo[4 * i + 2] = x.z; Alo[4 * i + 3] = x.w;
            }
            qsum = qsum_s[r];
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) { Aq[i] = 0; Ahi[i] = 0; Alo[i] = 0; }
        }
        SPARK_PROBE();      // setup done

        float m_run = -INFINITY, l_run = 0.f;
        float o[16][4];
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) { o[nt][0] = 0.f; o[nt][1] = 0.f; o[nt][2] = 0.f; o[nt][3] = 0.f; }

        int n = base + ((warp - base) % kConsumerWarps + kConsumerWarps) % kConsumerWarps;
        for (; n < base + sg.n; n += kConsumerWarps) {
            const int i = sg.i0 + (n - base);
            const int slot = n % NS;
            const bool ok = mbar_wait(&C.full[slot], (n / NS) & 1, C.abort_flag, A.status);
            const unsigned sbase = ring_u + static_cast<unsigned>(slot) * A.slot_stride;
            const int n_valid = min(kStepTokens, len - i * kStepTokens);
#ifdef SPARK_CTA_TIMING
            if (tid == 0 && t_first == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_first));
#endif
            if (ok) {
#pragma unroll 1
                for (int pg = 0; pg < 2; ++pg) {
                    if (pg * kPageTokens >= n_valid) break;                    // warp-uniform
                    const unsigned page = sbase + pg * L.page_bytes;
                    // ---------------- scores of the page's 16 tokens ----------------
                    float accA[2][4], accB[2][4];
                    unsigned vaddr[2], w[2];
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) { accA[j][e] = 0.f; accB[j][e] = 0.f; }
                        const int tok = 8 * j + r;
                        w[j] = lds_u32(page + L.mask_off + tok * 16 + c * 4);
                        const int cnt = __popc(w[j]);
                        int x = cnt;
                        int t = __shfl_up_sync(kFull, x, 1, 4);
                        if (c >= 1) x += t;
                        t = __shfl_up_sync(kFull, x, 2, 4);
                        if (c >= 2) x += t;
                        vaddr[j] = page + tok * 2 + (x - cnt) * 32;
                    }
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            unsigned k0, k1, m0, m1;
                            expand_nibble(w[j], 1u << (4 * ks), 2u << (4 * ks), 4u << (4 * ks), 8u << (4 * ks),
                                          vaddr[j], k0, k1, m0, m1);
                            mma_bf16(accA[j], Aq[2 * ks], 0u, Aq[2 * ks + 1], 0u, k0, k1);
                            mma_bf16(accB[j], Ahi[2 * ks], Alo[2 * ks], Ahi[2 * ks + 1], Alo[2 * ks + 1], m0, m1);
                        }
                    }
                    // ---------------- online softmax over the 16 tokens ----------------
                    float s[2][2];
                    float mt = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const float2 mu = lds_f32x2(page + L.mu_off + (8 * j + 2 * c) * 4);
                        const float muv[2] = {mu.x, mu.y};
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int tok = pg * kPageTokens + 8 * j + 2 * c + e;
                            const float rec = qsum - accB[j][e] - accB[j][2 + e];
                            const float sv = A.scale_log2e * fmaf(muv[e], rec, accA[j][e]);
                            s[j][e] = (tok < n_valid) ? sv : -INFINITY;
                            mt = fmaxf(mt, s[j][e]);
                        }
                    }
                    mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 1));
                    mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 2));
                    const float m_new = fmaxf(m_run, mt);
                    const float alpha = exp2f(m_run - m_new);
                    m_run = m_new;
                    float hi[2][2], lo[2][2], psum = 0.f;
#pragma unroll
                    for (int j = 0; j < 2; ++j)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const float p = row_ok ? exp2f(s[j][e] - m_new) : 0.f;
                            psum += p;
                            hi[j][e] = bf16_round(p);
                            lo[j][e] = p - hi[j][e];
                        }
                    l_run = fmaf(l_run, alpha, psum);
                    const unsigned P0 = pack_bf16(hi[0][0], hi[0][1]), P1 = pack_bf16(lo[0][0], lo[0][1]);
                    const unsigned P2 = pack_bf16(hi[1][0], hi[1][1]), P3 = pack_bf16(lo[1][0], lo[1][1]);
                    if (__any_sync(kFull, alpha != 1.0f)) {
#pragma unroll
                        for (int nt = 0; nt < 16; ++nt) {
                            o[nt][0] *= alpha; o[nt][1] *= alpha; o[nt][2] *= alpha; o[nt][3] *= alpha;
                        }
                    }
                    // ---------------- P.V ----------------
                    const int mi = lane >> 3, rr = lane & 7;
                    const unsigned vrow = page + L.v_off + (((mi & 1) << 3) + rr) * (kHeadDim * 2);
#pragma unroll
                    for (int cb = 0; cb < 8; ++cb) {
                        unsigned vb[4];
                        ldmatrix_x4_trans(vb, vrow + (((2 * cb + (mi >> 1)) ^ rr) << 4));
                        mma_bf16(o[2 * cb], P0, P1, P2, P3, vb[0], vb[1]);
                        mma_bf16(o[2 * cb + 1], P0, P1, P2, P3, vb[2], vb[3]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&C.empty[slot]);
        }
        SPARK_PROBE();      // steps done (warp 0)

        // ---------------- hand the warp state to the merge ----------------
        {
            float lsum = l_run;
            lsum += __shfl_xor_sync(kFull, lsum, 1);
            lsum += __shfl_xor_sync(kFull, lsum, 2);
            if (row_ok) {
                float* mine = merge + (warp * G + r) * kRec;
#pragma unroll
                for (int nt = 0; nt < 16; ++nt)
                    *reinterpret_cast<float2*>(mine + 8 * nt + 2 * c) =
                        make_float2(o[nt][0] + o[nt][2], o[nt][1] + o[nt][3]);
                if (c == 0) { mine[kHeadDim] = m_run; mine[kHeadDim + 1] = lsum; }
            }
        }
        consumer_sync();
        SPARK_PROBE();      // all warps done
        merge_and_publish<G>(A, C, merge, sg, tid);
        SPARK_PROBE();      // published
        g += sg.n;
        base += sg.n;
    }
#ifdef SPARK_CTA_TIMING
    if (tid == 0) {
        unsigned long long t_end;
        unsigned smid;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_end));
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        unsigned long long* rec = reinterpret_cast<unsigned long long*>(
            A.partials + static_cast<int64_t>(kMaxCtas + A.B * A.Hkv - 1 - blockIdx.x) * G * kRec);
        rec[0] = t_start; rec[1] = t_first; rec[2] = t_end; rec[3] = smid;
        for (int i = 0; i < 12; ++i) rec[4 + i] = t_probe[i];
    }
#endif
}

template <int G>
static spark_status launch_bf16(const DecodeArgs& A0, int n_sms, int smem_optin, cudaStream_t stream)
{
    DecodeArgs A = A0;
    using S = SmemBf16<G>;
    A.slot_stride = static_cast<int>(align_up(2 * static_cast<size_t>(A.L.page_bytes), 128));
    int ns = (smem_optin - S::kRing) / A.slot_stride;
    if (ns > kMaxSlots) ns = kMaxSlots;
    if (ns < 2) return SPARK_ERR_UNSUPPORTED;
    A.nslots = ns;
    const size_t smem = S::kRing + static_cast<size_t>(ns) * A.slot_stride;
    if (cudaFuncSetAttribute(decode_bf16_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(smem)) != cudaSuccess)
        return SPARK_ERR_CUDA;
    const int grid = n_sms < kMaxCtas ? n_sms : kMaxCtas;
    decode_bf16_kernel<G><<<grid, kDecodeThreads, smem, stream>>>(A);
    return cudaGetLastError() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

spark_status launch_decode_bf16(int G, const DecodeArgs& A, int n_sms, int smem_optin, cudaStream_t stream)
{
    switch (G) {
        case 1: return launch_bf16<1>(A, n_sms, smem_optin, stream);
        case 2: return launch_bf16<2>(A, n_sms, smem_optin, stream);
        case 3: return launch_bf16<3>(A, n_sms, smem_optin, stream);
        case 4: return launch_bf16<4>(A, n_sms, smem_optin, stream);
        case 5: return launch_bf16<5>(A, n_sms, smem_optin, stream);
        case 6: return launch_bf16<6>(A, n_sms, smem_optin, stream);
        case 7: return launch_bf16<7>(A, n_sms, smem_optin, stream);
        case 8: return launch_bf16<8>(A, n_sms, smem_optin, stream);
        default: return SPARK_ERR_UNSUPPORTED;
    }
}

}  // namespace spark
