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
    static constexpr int kLut = kCtrlBytes + kPrefixBytes;                       // 16 x uint2
    static constexpr int kMerge = kLut + 128;
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

__device__ __forceinline__ void ldmatrix_x4_trans(unsigned (&r)[4], const void* smem_row)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_u32(smem_row)));
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

// Expand the kept values of one mask nibble into the two second-operand registers of a k-step.
// `vptr` points at the token's next unread kept value (rows of 32 bytes) and advances per set bit.
__device__ __forceinline__ void expand_nibble(unsigned nb, const unsigned char*& vptr, unsigned& b0, unsigned& b1)
{
    unsigned v0 = 0, v1 = 0, v2 = 0, v3 = 0;
    if (nb & 1u) { v0 = *reinterpret_cast<const unsigned short*>(vptr); vptr += 32; }
    if (nb & 2u) { v1 = *reinterpret_cast<const unsigned short*>(vptr); vptr += 32; }
    if (nb & 4u) { v2 = *reinterpret_cast<const unsigned short*>(vptr); vptr += 32; }
    if (nb & 8u) { v3 = *reinterpret_cast<const unsigned short*>(vptr); vptr += 32; }
    b0 = v0 | (v1 << 16);
    b1 = v2 | (v3 << 16);
}

template <int G>
__global__ void __launch_bounds__(kDecodeThreads, 1) decode_bf16_kernel(const DecodeArgs A)
{
    using S = SmemBf16<G>;
    extern __shared__ __align__(128) unsigned char smem[];
    const Ctrl C = make_ctrl(smem);
    uint2* lut = reinterpret_cast<uint2*>(smem + S::kLut);
    float* merge = reinterpret_cast<float*>(smem + S::kMerge);
    unsigned char* ring = smem + S::kRing;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const PageLayout L = A.L;
    const int NS = A.nslots;
    const int max_tokens = A.max_blocks * kPageTokens;

    if (tid < 16) {                                        // nibble -> 0/1 pattern in bf16 (1.0 = 0x3F80)
        const unsigned x = ((tid & 1) ? 0x3F80u : 0u) | ((tid & 2) ? 0x3F800000u : 0u);
        const unsigned y = ((tid & 4) ? 0x3F80u : 0u) | ((tid & 8) ? 0x3F800000u : 0u);
        lut[tid] = make_uint2(x, y);
    }
    decode_prologue(A, C, tid);
    const int* prefix = C.prefix;
    const int total = A.Hkv * prefix[A.B];
    const int nct = static_cast<int>(gridDim.x);
    const int chunk = (total + nct - 1) / nct;
    const int c0 = min(total, static_cast<int>(blockIdx.x) * chunk);
    const int c1 = min(total, c0 + chunk);

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

        // ---- first-operand fragments of this unit (every warp keeps its own copy in registers) ----
        // Aq[2s], Aq[2s+1]: q[row][32c+4s .. +3];  Ahi/Alo: bf16 high / low part of q / a.
        unsigned Aq[16], Ahi[16], Alo[16];
        float qsum = 0.f;
        {
            double part = 0.0;
            if (row_ok) {
                const uint4* qs = reinterpret_cast<const uint4*>(
                    static_cast<const unsigned short*>(A.q) +
                    (static_cast<int64_t>(b) * A.Hq + h * G + r) * kHeadDim + 32 * c);
                const float4* an = reinterpret_cast<const float4*>(
                    A.qnorm + (static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim + 32 * c);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 u = qs[i];
                    Aq[4 * i] = u.x; Aq[4 * i + 1] = u.y; Aq[4 * i + 2] = u.z; Aq[4 * i + 3] = u.w;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 a4 = an[i];
                    const float av[4] = {a4.x, a4.y, a4.z, a4.w};
                    float hi[4], lo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const unsigned wq = Aq[2 * i + (e >> 1)];
                        const float qf = __uint_as_float((e & 1) ? (wq & 0xffff0000u) : (wq << 16));
                        const float qp = qf / av[e];
                        hi[e] = bf16_round(qp);
                        lo[e] = bf16_round(qp - hi[e]);
                        part += static_cast<double>(hi[e]) + static_cast<double>(lo[e]);
                    }
                    Ahi[2 * i] = pack_bf16(hi[0], hi[1]); Ahi[2 * i + 1] = pack_bf16(hi[2], hi[3]);
                    Alo[2 * i] = pack_bf16(lo[0], lo[1]); Alo[2 * i + 1] = pack_bf16(lo[2], lo[3]);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) { Aq[i] = 0; Ahi[i] = 0; Alo[i] = 0; }
            }
            part += __shfl_xor_sync(kFull, part, 1);
            part += __shfl_xor_sync(kFull, part, 2);
            qsum = static_cast<float>(part);              // sum over all 128 channels of the 16-bit q'
        }

        float m_run = -INFINITY, l_run = 0.f;
        float o[16][4];
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) { o[nt][0] = 0.f; o[nt][1] = 0.f; o[nt][2] = 0.f; o[nt][3] = 0.f; }

        int n = base + ((warp - base) % kConsumerWarps + kConsumerWarps) % kConsumerWarps;
        for (; n < base + sg.n; n += kConsumerWarps) {
            const int i = sg.i0 + (n - base);
            const int slot = n % NS;
            const bool ok = mbar_wait(&C.full[slot], (n / NS) & 1, C.abort_flag, A.status);
            const unsigned char* sbase = ring + static_cast<size_t>(slot) * A.slot_stride;
            const int n_valid = min(kStepTokens, len - i * kStepTokens);
            if (ok) {
#pragma unroll 1
                for (int pg = 0; pg < 2; ++pg) {
                    if (pg * kPageTokens >= n_valid) break;                    // warp-uniform
                    const unsigned char* page = sbase + pg * L.page_bytes;
                    // ---------------- scores of the page's 16 tokens ----------------
                    float accA[2][4], accB[2][4];
                    const unsigned char* vptr[2];
                    unsigned w[2];
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) { accA[j][e] = 0.f; accB[j][e] = 0.f; }
                        const int tok = 8 * j + r;
                        w[j] = *reinterpret_cast<const unsigned*>(page + L.mask_off + tok * 16 + c * 4);
                        const int cnt = __popc(w[j]);
                        int x = cnt;
                        int t = __shfl_up_sync(kFull, x, 1, 4);
                        if (c >= 1) x += t;
                        t = __shfl_up_sync(kFull, x, 2, 4);
                        if (c >= 2) x += t;
                        vptr[j] = page + tok * 2 + (x - cnt) * 32;
                    }
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            const unsigned nb = (w[j] >> (4 * ks)) & 15u;
                            unsigned b0, b1;
                            expand_nibble(nb, vptr[j], b0, b1);
                            const uint2 mk = lut[nb];
                            mma_bf16(accA[j], Aq[2 * ks], 0u, Aq[2 * ks + 1], 0u, b0, b1);
                            mma_bf16(accB[j], Ahi[2 * ks], Alo[2 * ks], Ahi[2 * ks + 1], Alo[2 * ks + 1], mk.x, mk.y);
                        }
                    }
                    // ---------------- online softmax over the 16 tokens ----------------
                    float s[2][2];
                    float mt = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const float2 mu = *reinterpret_cast<const float2*>(page + L.mu_off + (8 * j + 2 * c) * 4);
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
                    const unsigned char* vrow = page + L.v_off + (((mi & 1) << 3) + rr) * (kHeadDim * 2);
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
        merge_and_publish<G>(A, C, merge, sg, chunk, tid);
        g += sg.n;
        base += sg.n;
    }
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
