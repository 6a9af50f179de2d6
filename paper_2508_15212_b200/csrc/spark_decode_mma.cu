// Decode attention over the packed SparK cache, bf16 storage (Sec. "Channel Recovery", degenerate
// distribution, then the softmax attention of Sec. "Preliminaries").
//
// For one query head, with a[j] = max(|q-bar_j|, eps) and q'[j] = q[j] / a[j]:
//     q . K~[t] = sum_{j kept} q[j] K[t][j]  +  mu[t] * ( sum_j q'[j]  -  sum_{j kept} q'[j] ).
// Both kept-channel sums are contractions over the 128 channels, [tokens x channels] by
// [channels x heads], so they run on the tensor cores (mma.sync m16n8k16, bf16 in, fp32 out) with the
// 16 tokens of a page as the rows:
//   - first operand: the tokens' kept values expanded to dense form (first sum) and the tokens' masks
//     as 0/1 (second sum).  The expansion happens in registers: the four lanes that hold a token row
//     each own one 32-bit mask word, walk its eight nibbles, and pull the next kept value from shared
//     memory for every set bit (predicated loads).  The channel order inside a k-step is a fixed
//     permutation (lane c, step s  <->  channels 32c+4s .. 32c+4s+3) applied to both operands;
//   - second operand (constant per unit, kept in registers): the G query heads as stored (bf16) for
//     the first sum, and q' split into a bf16 high and low part for the second.  With G <= 4 the high
//     and low parts share one 8-column operand (columns 0-3 / 4-7); otherwise they are two operands.
// P.V is the third contraction, [channels x tokens] by [tokens x heads]: value rows come in through
// transposing matrix loads (the rows are stored chunk-swizzled in the page, so these are conflict
// free) and the probabilities, split in bf16 high and low parts so the product keeps ~16 mantissa
// bits, are moved from the score layout to the operand layout with a warp matrix transpose.
// Softmax statistics and all accumulators are fp32.
//
// With value-channel pruning (App. "Pruning Value Cache Channels") a page carries kept value entries and
// a second mask instead of dense value rows; the warp first expands them (same nibble walk, zeros where
// pruned) into a 4 KB tile of its own in shared memory, in the chunk-swizzled row layout of a dense
// page, and the third contraction reads that tile.
#include <cstring>

#include "spark_decode_common.cuh"

namespace spark {

constexpr int kNW = 15;                       // consumer warps (+ 1 producer warp = 16 warps, 4 per scheduler)
constexpr int kNT = kNW * 32;
constexpr int kThreads = kNT + 32;
constexpr float kSlack = 8.f;                 // log2 units a score may exceed the running reference maximum

constexpr int kVTileBytes = kPageTokens * kHeadDim * 2;                          // dense value rows of one page

// Shared-memory map (fixed part; the steps prefix and the ring follow at offsets chosen by the launcher).
template <int G, bool kPV> struct SmemBf16 {
    static constexpr int kTab = kCtrlBytes;                                      // q, q' high, q' low: 3 x [G][128] bf16
    static constexpr int kQsum = kTab + 3 * G * kHeadDim * 2;                    // [8] float
    static constexpr int kMerge = kQsum + 32;
    static constexpr int kVTile = (kMerge + merge_bytes(kNW, G) + 127) / 128 * 128;   // per-warp tiles (pruned values)
    static constexpr int kFixed = kVTile + (kPV ? kNW * kVTileBytes : 0);        // prefix and ring start here
};

__device__ __forceinline__ void mma_bf16(float (&d)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                         unsigned b0, unsigned b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4_trans(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3, unsigned smem_addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(smem_addr));
}

// 8x8 b16 transpose across the warp: lane (r, c) gives row r, columns 2c..2c+1 and receives
// rows 2c..2c+1 of column r.
__device__ __forceinline__ unsigned movmatrix_trans(unsigned x)
{
    unsigned y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}

__device__ __forceinline__ unsigned lds_u32(unsigned addr)
{
    unsigned v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ float lds_f32(unsigned addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds_u32x4(unsigned addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
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

// One mask nibble (bits b0m..b3m of word w) -> the first-operand registers of a k-step for one token:
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

// The value-side nibble: kept value entries in dense positions, zero where pruned (see expand_nibble).
__device__ __forceinline__ void expand_nibble_v(unsigned w, unsigned b0m, unsigned b1m, unsigned b2m, unsigned b3m,
                                                unsigned& addr, unsigned& k0, unsigned& k1)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p0, p1, p2, p3;\n\t"
        ".reg .b32 t0, t1, t2, t3;\n\t"
        ".reg .b16 h0, h1, h2, h3;\n\t"
        "and.b32 t0, %3, %4;\n\t"
        "and.b32 t1, %3, %5;\n\t"
        "and.b32 t2, %3, %6;\n\t"
        "and.b32 t3, %3, %7;\n\t"
        "setp.ne.u32 p0, t0, 0;\n\t"
        "setp.ne.u32 p1, t1, 0;\n\t"
        "setp.ne.u32 p2, t2, 0;\n\t"
        "setp.ne.u32 p3, t3, 0;\n\t"
        "mov.b16 h0, 0;\n\t"
        "mov.b16 h1, 0;\n\t"
        "mov.b16 h2, 0;\n\t"
        "mov.b16 h3, 0;\n\t"
        "@p0 ld.shared.u16 h0, [%2];\n\t"
        "@p0 add.u32 %2, %2, 32;\n\t"
        "@p1 ld.shared.u16 h1, [%2];\n\t"
        "@p1 add.u32 %2, %2, 32;\n\t"
        "@p2 ld.shared.u16 h2, [%2];\n\t"
        "@p2 add.u32 %2, %2, 32;\n\t"
        "@p3 ld.shared.u16 h3, [%2];\n\t"
        "@p3 add.u32 %2, %2, 32;\n\t"
        "mov.b32 %0, {h0, h1};\n\t"
        "mov.b32 %1, {h2, h3};\n\t"
        "}"
        : "=&r"(k0), "=&r"(k1), "+r"(addr)
        : "r"(w), "r"(b0m), "r"(b1m), "r"(b2m), "r"(b3m));
}

// Tables of one query head of a unit (one warp; lane l owns channels 4l .. 4l+3):
//   tab[0][hd][j] = q[j] (bf16 as stored), tab[1] / tab[2] = bf16 high / low part of q[j] / a[j],
//   qsum[hd]      = sum over all 128 channels of the 16-bit q' (so kept terms cancel exactly).
template <int G>
__device__ __forceinline__ void write_head_tables(unsigned char* tab, float* qsum, int hd, int lane, uint2 qr, float4 a4)
{
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
    unsigned char* row = tab + hd * (kHeadDim * 2) + lane * 8;
    *reinterpret_cast<uint2*>(row) = qr;
    *reinterpret_cast<uint2*>(row + G * kHeadDim * 2) = make_uint2(pack_bf16(hi[0], hi[1]), pack_bf16(hi[2], hi[3]));
    *reinterpret_cast<uint2*>(row + 2 * G * kHeadDim * 2) = make_uint2(pack_bf16(lo[0], lo[1]), pack_bf16(lo[2], lo[3]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(kFull, part, o);
    if (lane == 0) qsum[hd] = static_cast<float>(part);
}

__device__ __forceinline__ void sts_u32x4(unsigned addr, unsigned a, unsigned b, unsigned c, unsigned d)
{
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// The whole step; `q_src` is where the query rows are read from (global memory, or the launch's own
// parameter block when the query travels with the launch).
template <int G, bool kPV>
__device__ __forceinline__ void decode_bf16_body(const DecodeArgs& A, const void* q_src)
{
    using S = SmemBf16<G, kPV>;
    constexpr bool kShared8 = (G <= 4);        // q' high and low parts share one 8-column operand
    extern __shared__ __align__(128) unsigned char smem[];
    const Ctrl C = make_ctrl(smem, A.prefix_off);
    unsigned char* tab = smem + S::kTab;
    float* qsum_s = reinterpret_cast<float*>(smem + S::kQsum);
    float* merge = reinterpret_cast<float*>(smem + S::kMerge);
    unsigned char* ring = smem + A.ring_off;
    const unsigned ring_u = smem_u32(ring);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const PageLayout L = A.L;
    const int NS = A.nslots;
    const int max_tokens = A.max_blocks * kPageTokens;

    prefetch_block_table(A, tid, kThreads);
    if (tid == 0) pdl_launch_dependents();
    if (warp == kNW) {
        producer_prologue(A, C, lane, kThreads);
        int p0, p1;
        cta_range(*C.plan, static_cast<int>(blockIdx.x), p0, p1);
        producer_loop(A, C, ring, p0, p1, lane);
        return;
    }
    consumer_wait_plan(kThreads);
    const int* prefix = C.prefix;
    int c0, c1;
    cta_range(*C.plan, static_cast<int>(blockIdx.x), c0, c1);
    pdl_dependency_wait();                                 // q, qnorm, out and the workspace from here on
    write_empty_sequences<kNT>(A, prefix, tid);

    const int c = lane & 3, r = lane >> 2;                 // quad lane / fragment row
    int base = 0;
    for (int g = c0; g < c1;) {
        const Segment sg = locate(prefix, A.B, A.Hkv, g, c1);
        const int b = sg.b, h = sg.h;
        const int len = clamp_len(A.lens[b], max_tokens);

        // ---- per-unit tables, built once per CTA: warp `hd` prepares query head hd ----
        if (warp < G) {
            const uint2 qr = *reinterpret_cast<const uint2*>(
                static_cast<const unsigned short*>(q_src) +
                (static_cast<int64_t>(b) * A.Hq + h * G + warp) * kHeadDim + 4 * lane);
            const float4 a4 = *reinterpret_cast<const float4*>(
                A.qnorm + (static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim + 4 * lane);
            write_head_tables<G>(tab, qsum_s, warp, lane, qr, a4);
        }
        consumer_sync<kNT>();
        // second-operand fragments (column r of each operand, channels 32c .. 32c+31):
        //   Bq[2s], Bq[2s+1] = q[head r][32c+4s .. +3];  Bp / Bpl likewise from the q' parts.
        unsigned Bq[16], Bp[16], Bpl[kShared8 ? 1 : 16];
        {
            const unsigned t0 = smem_u32(tab) + c * 64;
            const unsigned plane = G * kHeadDim * 2;
            const int pr = kShared8 ? (r & 3) : r;                     // head of column r in the q' operand
            const unsigned pofs = kShared8 ? ((r < 4) ? plane : 2 * plane) : plane;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 u = make_uint4(0, 0, 0, 0), v = make_uint4(0, 0, 0, 0), x = make_uint4(0, 0, 0, 0);
                if (r < G) u = lds_u32x4(t0 + r * (kHeadDim * 2) + i * 16);
                if (pr < G) v = lds_u32x4(t0 + pofs + pr * (kHeadDim * 2) + i * 16);
                if (!kShared8 && r < G) x = lds_u32x4(t0 + 2 * plane + r * (kHeadDim * 2) + i * 16);
                Bq[4 * i] = u.x; Bq[4 * i + 1] = u.y; Bq[4 * i + 2] = u.z; Bq[4 * i + 3] = u.w;
                Bp[4 * i] = v.x; Bp[4 * i + 1] = v.y; Bp[4 * i + 2] = v.z; Bp[4 * i + 3] = v.w;
                if (!kShared8) { Bpl[4 * i] = x.x; Bpl[4 * i + 1] = x.y; Bpl[4 * i + 2] = x.z; Bpl[4 * i + 3] = x.w; }
            }
        }
        // this thread's two heads in the score layout (columns 2c, 2c+1)
        bool hv[2];
        float qsum[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            hv[e] = (2 * c + e < G) && (!kShared8 || c < 2);
            qsum[e] = hv[e] ? qsum_s[2 * c + e] : 0.f;
        }

        float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
        float thr[2] = {hv[0] ? -INFINITY : INFINITY, hv[1] ? -INFINITY : INFINITY};
        float o[8][4];
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) { o[mt][0] = 0.f; o[mt][1] = 0.f; o[mt][2] = 0.f; o[mt][3] = 0.f; }

        int n = base + ((warp - base) % kNW + kNW) % kNW;
        int slot = n % NS, round = n / NS;                 // ring position of step n, kept incrementally
        for (; n < base + sg.n; n += kNW, slot += kNW) {
            while (slot >= NS) { slot -= NS; ++round; }
            const int i = sg.i0 + (n - base);
            const bool ok = slot_wait(C.full, C.seq, slot, round, C.abort_flag, A.status);
            const unsigned page = ring_u + static_cast<unsigned>(slot) * A.slot_stride;
            const int n_valid = min(kPageTokens, len - i * kPageTokens);
            if (ok) {
                // ---------------- scores of the page's 16 tokens (rows r and r+8) ----------------
                float d1[4] = {0.f, 0.f, 0.f, 0.f}, d2[4] = {0.f, 0.f, 0.f, 0.f}, d3[4] = {0.f, 0.f, 0.f, 0.f};
                unsigned vaddr[2], vaddr_hi[2], w[2];
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int tok = 8 * j + r;
                    w[j] = lds_u32(page + L.mask_off + tok * 16 + c * 4);
                    const int cnt = __popc(w[j]);
                    int x = cnt;
                    int t = __shfl_up_sync(kFull, x, 1, 4);
                    if (c >= 1) x += t;
                    t = __shfl_up_sync(kFull, x, 2, 4);
                    if (c >= 2) x += t;
                    vaddr[j] = page + L.vals_off + (r * 2 + j) * 2 + (x - cnt) * 32;      // see val_offset: token r + 8j
                    vaddr_hi[j] = vaddr[j] + __popc(w[j] & 0xffffu) * 32;    // upper half of the word walks on its own
                }
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    unsigned k0[2], k1[2], m0[2], m1[2];
#pragma unroll
                    for (int j = 0; j < 2; ++j)
                        expand_nibble(w[j], 1u << (4 * ks), 2u << (4 * ks), 4u << (4 * ks), 8u << (4 * ks),
                                      ks < 4 ? vaddr[j] : vaddr_hi[j], k0[j], k1[j], m0[j], m1[j]);
                    mma_bf16(d1, k0[0], k0[1], k1[0], k1[1], Bq[2 * ks], Bq[2 * ks + 1]);
                    mma_bf16(d2, m0[0], m0[1], m1[0], m1[1], Bp[2 * ks], Bp[2 * ks + 1]);
                    if (!kShared8) mma_bf16(d3, m0[0], m0[1], m1[0], m1[1], Bpl[2 * ks], Bpl[2 * ks + 1]);
                }
                // kept q' sums of this thread's heads: high part + low part
                float rk[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float other = kShared8 ? __shfl_xor_sync(kFull, d2[e], 2) : d3[e];
                    rk[e] = d2[e] + other;
                }
                // ---------------- online softmax over the 16 tokens ----------------
                // The reference maximum m_run of a head moves only when a score of the page exceeds it
                // by more than kSlack (log2 units), so most pages skip the warp-wide maximum and the
                // rescaling; probabilities then lie in (0, 2^kSlack], which fp32 sums and the bf16
                // high/low split carry without loss.  thr = m_run + kSlack (+inf for unused columns).
                const float mu[2] = {lds_f32(page + L.mu_off + r * 4), lds_f32(page + L.mu_off + (r + 8) * 4)};
                float s[2][2];
#pragma unroll
                for (int e = 0; e < 2; ++e)
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const float sv = A.scale_log2e * fmaf(mu[j], qsum[e] - rk[2 * j + e], d1[2 * j + e]);
                        s[j][e] = (r + 8 * j < n_valid) ? sv : -INFINITY;
                    }
                const float over = fmaxf(fmaxf(s[0][0], s[1][0]) - thr[0], fmaxf(s[0][1], s[1][1]) - thr[1]);
                if (__any_sync(kFull, over > 0.f)) {
                    float alpha[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        float mt = fmaxf(s[0][e], s[1][e]);
                        mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 4));
                        mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 8));
                        mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 16));
                        const float m_new = fmaxf(m_run[e], mt);
                        alpha[e] = hv[e] ? ex2(m_run[e] - m_new) : 1.f;
                        l_run[e] *= alpha[e];
                        m_run[e] = m_new;
                        thr[e] = hv[e] ? m_new + kSlack : INFINITY;
                    }
                    float a0 = alpha[0], a1 = alpha[1];      // columns 2c, 2c+1 of every output tile
                    if (kShared8) {
                        const float y0 = __shfl_xor_sync(kFull, a0, 2), y1 = __shfl_xor_sync(kFull, a1, 2);
                        if (c >= 2) { a0 = y0; a1 = y1; }
                    }
#pragma unroll
                    for (int mt = 0; mt < 8; ++mt) {
                        o[mt][0] *= a0; o[mt][1] *= a1; o[mt][2] *= a0; o[mt][3] *= a1;
                    }
                }
                float ph[2][2], pl[2][2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float p0 = hv[e] ? ex2(s[0][e] - m_run[e]) : 0.f;
                    const float p1 = hv[e] ? ex2(s[1][e] - m_run[e]) : 0.f;
                    l_run[e] += p0 + p1;
                    ph[0][e] = bf16_round(p0); pl[0][e] = p0 - ph[0][e];
                    ph[1][e] = bf16_round(p1); pl[1][e] = p1 - ph[1][e];
                }
                // probabilities: score layout (row = token, cols = heads) -> operand layout (k = token, n = col)
                unsigned pb0, pb1, pc0 = 0, pc1 = 0;
                {
                    const unsigned h0 = pack_bf16(ph[0][0], ph[0][1]), h1 = pack_bf16(ph[1][0], ph[1][1]);
                    const unsigned l0 = pack_bf16(pl[0][0], pl[0][1]), l1 = pack_bf16(pl[1][0], pl[1][1]);
                    if (kShared8) {                      // columns 4-7 carry the low parts of heads 0-3
                        const unsigned x0 = __shfl_xor_sync(kFull, l0, 2), x1 = __shfl_xor_sync(kFull, l1, 2);
                        pb0 = movmatrix_trans(c < 2 ? h0 : x0);
                        pb1 = movmatrix_trans(c < 2 ? h1 : x1);
                    } else {
                        pb0 = movmatrix_trans(h0); pb1 = movmatrix_trans(h1);
                        pc0 = movmatrix_trans(l0); pc1 = movmatrix_trans(l1);
                    }
                }
                // ---------------- P.V: out^T[channel][col] += V^T[channel][token] P^T[token][col] ----------------
                unsigned vbase = page + L.v_off;
                if (kPV) {
                    // lane (r, c) expands mask word c of tokens r and r + 8: channels 32c + 8u .. + 7 of a
                    // token are 16-byte chunk k = 4c + u, stored at chunk index k ^ r ^ ((k >> 3) << 1) of the
                    // token's row (the extra term keeps the four lanes of a row on different banks)
                    vbase = smem_u32(smem + S::kVTile) + warp * kVTileBytes;
                    unsigned vw[2], va[2];
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        vw[j] = lds_u32(page + L.vmask_off + (8 * j + r) * 16 + c * 4);
                        const int cnt = __popc(vw[j]);
                        int x = cnt;
                        int t = __shfl_up_sync(kFull, x, 1, 4);
                        if (c >= 1) x += t;
                        t = __shfl_up_sync(kFull, x, 2, 4);
                        if (c >= 2) x += t;
                        va[j] = page + L.v_off + (r * 2 + j) * 2 + (x - cnt) * 32;
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u)
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            unsigned e0, e1, e2, e3;
                            expand_nibble_v(vw[j], 1u << (8 * u), 2u << (8 * u), 4u << (8 * u), 8u << (8 * u), va[j], e0, e1);
                            expand_nibble_v(vw[j], 16u << (8 * u), 32u << (8 * u), 64u << (8 * u), 128u << (8 * u), va[j], e2, e3);
                            sts_u32x4(vbase + (8 * j + r) * (kHeadDim * 2) + (((4 * c + u) ^ r ^ (c & 2)) << 4), e0, e1, e2, e3);
                        }
                    __syncwarp();
                }
                const int mi = lane >> 3, rr = lane & 7;
                const unsigned vrow = vbase + (((mi >> 1) << 3) + rr) * (kHeadDim * 2);
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) {
                    unsigned a0, a1, a2, a3;
                    ldmatrix_x4_trans(a0, a1, a2, a3, vrow + (((2 * mt + (mi & 1)) ^ rr ^ (kPV ? ((mt >> 2) << 1) : 0)) << 4));
                    mma_bf16(o[mt], a0, a1, a2, a3, pb0, pb1);
                    if (!kShared8) mma_bf16(o[mt], a0, a1, a2, a3, pc0, pc1);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&C.empty[slot]);
        }

        // ---------------- hand the warp state to the merge ----------------
        {
            float lsum[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                lsum[e] = l_run[e];
                lsum[e] += __shfl_xor_sync(kFull, lsum[e], 4);
                lsum[e] += __shfl_xor_sync(kFull, lsum[e], 8);
                lsum[e] += __shfl_xor_sync(kFull, lsum[e], 16);
            }
#pragma unroll
            for (int mt = 0; mt < 8; ++mt)
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    float v = o[mt][q4];
                    if (kShared8) v += __shfl_xor_sync(kFull, v, 2);       // high-part column + low-part column
                    const int e = q4 & 1;
                    if (hv[e]) merge[(warp * G + 2 * c + e) * kRec + 16 * mt + r + ((q4 >> 1) << 3)] = v;
                }
#pragma unroll
            for (int e = 0; e < 2; ++e)
                if (hv[e] && r == 0) {
                    merge[(warp * G + 2 * c + e) * kRec + kHeadDim] = m_run[e];
                    merge[(warp * G + 2 * c + e) * kRec + kHeadDim + 1] = lsum[e];
                }
        }
        consumer_sync<kNT>();
        merge_and_publish<G, kNW>(A, C, merge, sg, tid);
        g += sg.n;
        base += sg.n;
    }
}

template <int G, bool kPV>
__global__ void __launch_bounds__(kThreads, 1) decode_bf16_kernel(const DecodeArgs A)
{
    decode_bf16_body<G, kPV>(A, A.q);
}

// The query as a kernel parameter: the launch itself carries the bytes to the GPU (no copy before the step,
// no reads over the bus inside it).  Two sizes, so that a small query does not pay for a large parameter block.
template <int kBytes> struct QueryBlob { uint4 v[kBytes / 16]; };
constexpr int kBlobSmall = 8 * 1024, kBlobLarge = 24 * 1024;
static_assert(kBlobLarge == kMaxQueryByValueBytes, "the launcher's limit is the large blob");

template <int G, int kBytes>
__global__ void __launch_bounds__(kThreads, 1) decode_bf16_qv_kernel(const __grid_constant__ DecodeArgs A,
                                                                     const __grid_constant__ QueryBlob<kBytes> Q)
{
    decode_bf16_body<G, false>(A, &Q);
}

template <int G, int kBytes>
static spark_status launch_bf16_qv(const DecodeArgs& A, int dev, int smem_optin, int grid, size_t smem, size_t q_bytes,
                                   cudaStream_t stream)
{
    static unsigned char smem_raised[kMaxDevices] = {};
    if (!allow_max_smem(decode_bf16_qv_kernel<G, kBytes>, dev, smem_optin, smem_raised)) return SPARK_ERR_CUDA;
    QueryBlob<kBytes> blob;                                 // A.q is a host pointer here; the bytes are taken now
    memcpy(&blob, A.q, q_bytes);
    return launch_decode_kernel(decode_bf16_qv_kernel<G, kBytes>, grid, kThreads, smem, stream, A, blob) == cudaSuccess
               ? SPARK_OK : SPARK_ERR_CUDA;
}

template <int G, bool kPV>
static spark_status launch_bf16(const DecodeArgs& A0, int dev, const DeviceInfo& info, cudaStream_t stream)
{
    static unsigned char smem_raised[kMaxDevices] = {};
    const int n_sms = info.n_sms, smem_optin = info.smem_optin;
    DecodeArgs A = A0;
    using S = SmemBf16<G, kPV>;
    A.pps = 1;
    A.slot_stride = static_cast<int>(align_up(static_cast<size_t>(A.L.page_bytes), 128));
    A.prefix_off = S::kFixed;
    A.ring_off = S::kFixed + prefix_bytes(A.B);
    int ns = (smem_optin - A.ring_off) / A.slot_stride;
    if (ns > kMaxSlots) ns = kMaxSlots;
    if (ns < 2) return SPARK_ERR_UNSUPPORTED;
    A.nslots = ns;
    const size_t smem = A.ring_off + static_cast<size_t>(ns) * A.slot_stride;
    const int grid = n_sms < kMaxCtas ? n_sms : kMaxCtas;
    if (A.q_by_value) {
        const size_t q_bytes = static_cast<size_t>(A.B) * A.Hq * kHeadDim * 2;
        if (kPV || q_bytes > static_cast<size_t>(kBlobLarge)) return SPARK_ERR_UNSUPPORTED;
        if (q_bytes <= static_cast<size_t>(kBlobSmall))
            return launch_bf16_qv<G, kBlobSmall>(A, dev, smem_optin, grid, smem, q_bytes, stream);
        return launch_bf16_qv<G, kBlobLarge>(A, dev, smem_optin, grid, smem, q_bytes, stream);
    }
    if (!allow_max_smem(decode_bf16_kernel<G, kPV>, dev, smem_optin, smem_raised)) return SPARK_ERR_CUDA;
    return launch_decode_kernel(decode_bf16_kernel<G, kPV>, grid, kThreads, smem, stream, A) == cudaSuccess
               ? SPARK_OK : SPARK_ERR_CUDA;
}

spark_status launch_decode_bf16(int G, const DecodeArgs& A, int dev, const DeviceInfo& info, cudaStream_t stream)
{
    const bool pv = A.L.keep_v < kHeadDim;                  // value rows are pruned: expand them per page
    switch (G) {
        case 1: return pv ? launch_bf16<1, true>(A, dev, info, stream) : launch_bf16<1, false>(A, dev, info, stream);
        case 2: return pv ? launch_bf16<2, true>(A, dev, info, stream) : launch_bf16<2, false>(A, dev, info, stream);
        case 3: return pv ? launch_bf16<3, true>(A, dev, info, stream) : launch_bf16<3, false>(A, dev, info, stream);
        case 4: return pv ? launch_bf16<4, true>(A, dev, info, stream) : launch_bf16<4, false>(A, dev, info, stream);
        case 5: return pv ? launch_bf16<5, true>(A, dev, info, stream) : launch_bf16<5, false>(A, dev, info, stream);
        case 6: return pv ? launch_bf16<6, true>(A, dev, info, stream) : launch_bf16<6, false>(A, dev, info, stream);
        case 7: return pv ? launch_bf16<7, true>(A, dev, info, stream) : launch_bf16<7, false>(A, dev, info, stream);
        case 8: return pv ? launch_bf16<8, true>(A, dev, info, stream) : launch_bf16<8, false>(A, dev, info, stream);
        default: return SPARK_ERR_UNSUPPORTED;
    }
}

}  // namespace spark
