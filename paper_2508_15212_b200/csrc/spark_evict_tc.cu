// Eviction votes on the 5th-generation tensor cores (tcgen05 + tensor memory), bf16 storage.
//
// The window-attention scores of the eviction pre-step are the one dense contraction of the method:
// per KV head, [G*W window-query rows x 128 channels] by [128 channels x S keys].  This file computes
// the same two passes as the CUDA-core kernels of spark_evict.cu with tcgen05.mma:
//   pass 1   D[row][token]  = Q . K^T   (M = 128 query rows, N = 128 keys per tile): a thread owns a
//            query row of the accumulator in tensor memory and keeps the row's running softmax max and
//            sum over all the tiles of its CTA -- no cross-thread reduction;
//   pass 2   D[token][row]  = K . Q^T   (M = 128 keys, N = padded row count <= 256): a thread owns a key
//            and adds up its probabilities over the query rows in a fixed order -- the votes are
//            reproducible and need no atomics.
// Operands are staged in shared memory by ordinary loads in the canonical K-major 128-byte-swizzled
// layout that the matrix descriptors name (row r of a 64-channel block at r*128 bytes, its 16-byte
// chunks XOR-ed with r & 7; 8-row groups 1024 bytes apart).  One thread issues the MMAs; completion
// arrives on an mbarrier through tcgen05.commit; every wait is bounded.
#include "spark_common.cuh"

namespace spark {

constexpr int kTcTile = 128;            // keys per tile
constexpr int kTcThreads = 128;
constexpr unsigned kTcSpin = 1u << 22;

struct EvictTcArgs {
    const void* q_win;
    const void* k;
    int64_t sb, sh, st;
    const int32_t* seq_lens;
    int Hq, Hkv, W, budget;
    int S_max, tiles_per_cta, parts;     // parts = CTAs per unit
    float* partial;      // [units][R][parts][2]   (pass 1 out)
    const float* rowstat;// [units][R][2]          (pass 2 in)
    float* votes;        // [units][S_max]
    int* status;
};

__device__ __forceinline__ unsigned tc_smem_u32(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }

// K-major, 128-byte swizzle: start address, stride between 8-row groups = 1024 bytes, descriptor version 1.
__device__ __forceinline__ uint64_t tc_desc(unsigned smem_addr)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);            // bits [0,14)  start address >> 4
    d |= static_cast<uint64_t>(1) << 16;                                 // bits [16,30) leading byte offset (unused for swizzled K-major)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;                         // bits [32,46) stride byte offset >> 4
    d |= static_cast<uint64_t>(1) << 46;                                 // bits [46,48) descriptor version
    d |= static_cast<uint64_t>(2) << 61;                                 // bits [61,64) layout: 128-byte swizzle
    return d;
}

// kind::f16 instruction descriptor: D = f32, A = B = bf16, both K-major, shape M x N x 16.
__device__ __forceinline__ unsigned tc_idesc(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<unsigned>(N >> 3) << 17) | (static_cast<unsigned>(M >> 4) << 24);
}

__device__ __forceinline__ void tc_mma(unsigned d_tmem, uint64_t a_desc, uint64_t b_desc, unsigned idesc, unsigned accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ float tc_ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void tc_ld32(unsigned taddr, float (&v)[32])
{
    unsigned r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// 128 consecutive columns of this thread's tensor-memory lane: two 64-column loads and one wait in a single
// statement, so nothing reads the registers before the wait.
__device__ __forceinline__ void tc_ld128(unsigned taddr, float (&v)[128])
{
    unsigned r[128];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%128];\n\t"
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%64,%65,%66,%67,%68,%69,%70,%71,%72,%73,%74,%75,%76,%77,%78,%79,%80,%81,%82,%83,%84,%85,%86,%87,%88,%89,%90,%91,%92,%93,%94,%95,%96,%97,%98,%99,%100,%101,%102,%103,%104,%105,%106,%107,%108,%109,%110,%111,%112,%113,%114,%115,%116,%117,%118,%119,%120,%121,%122,%123,%124,%125,%126,%127}, [%129];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63]), "=r"(r[64]), "=r"(r[65]), "=r"(r[66]), "=r"(r[67]), "=r"(r[68]), "=r"(r[69]), "=r"(r[70]), "=r"(r[71]), "=r"(r[72]), "=r"(r[73]), "=r"(r[74]), "=r"(r[75]), "=r"(r[76]), "=r"(r[77]), "=r"(r[78]), "=r"(r[79]), "=r"(r[80]), "=r"(r[81]), "=r"(r[82]), "=r"(r[83]), "=r"(r[84]), "=r"(r[85]), "=r"(r[86]), "=r"(r[87]), "=r"(r[88]), "=r"(r[89]), "=r"(r[90]), "=r"(r[91]), "=r"(r[92]), "=r"(r[93]), "=r"(r[94]), "=r"(r[95]), "=r"(r[96]), "=r"(r[97]), "=r"(r[98]), "=r"(r[99]), "=r"(r[100]), "=r"(r[101]), "=r"(r[102]), "=r"(r[103]), "=r"(r[104]), "=r"(r[105]), "=r"(r[106]), "=r"(r[107]), "=r"(r[108]), "=r"(r[109]), "=r"(r[110]), "=r"(r[111]), "=r"(r[112]), "=r"(r[113]), "=r"(r[114]), "=r"(r[115]), "=r"(r[116]), "=r"(r[117]), "=r"(r[118]), "=r"(r[119]), "=r"(r[120]), "=r"(r[121]), "=r"(r[122]), "=r"(r[123]), "=r"(r[124]), "=r"(r[125]), "=r"(r[126]), "=r"(r[127])
        : "r"(taddr), "r"(taddr + 64u)
        : "memory");
#pragma unroll
    for (int i = 0; i < 128; ++i) v[i] = __uint_as_float(r[i]);
}

// Copy `rows` rows of 128 bf16 channels (row i at src + i*stride elements; rows >= valid are zero) into
// the two 64-channel swizzled blocks at dst (block 0 at dst, block 1 at dst + rows_alloc*128 bytes).
__device__ __forceinline__ void tc_stage_rows(unsigned char* dst, int rows_alloc, const unsigned short* src, int64_t stride,
                                              int valid, int tid)
{
    for (int i = tid; i < rows_alloc * 16; i += kTcThreads) {
        const int r = i >> 4, ch16 = i & 15;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (r < valid) v = *reinterpret_cast<const uint4*>(src + static_cast<int64_t>(r) * stride + ch16 * 8);
        const int kb = ch16 >> 3, c8 = ch16 & 7;
        *reinterpret_cast<uint4*>(dst + static_cast<size_t>(kb) * rows_alloc * 128 + r * 128 + ((c8 ^ (r & 7)) << 4)) = v;
    }
}

// The same copy for a key tile with 16-byte asynchronous copies (rows >= valid are zero-filled): the
// caller commits the group and waits for it one tile later, so the load of tile i+1 runs under the MMAs
// and the epilogue of tile i.
__device__ __forceinline__ void tc_stage_rows_async(unsigned dst_u, int rows_alloc, const unsigned short* src, int64_t stride,
                                                    int valid, int tid)
{
    for (int i = tid; i < rows_alloc * 16; i += kTcThreads) {
        const int r = i >> 4, ch16 = i & 15;
        const int kb = ch16 >> 3, c8 = ch16 & 7;
        const bool live = r < valid;
        const unsigned short* g = src + static_cast<int64_t>(live ? r : 0) * stride + ch16 * 8;
        const unsigned d = dst_u + static_cast<unsigned>(kb) * rows_alloc * 128u + r * 128u + ((c8 ^ (r & 7)) << 4);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(g), "r"(live ? 16 : 0) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

template <int PASS>
__global__ void __launch_bounds__(kTcThreads, 2) evict_scores_tc_kernel(EvictTcArgs A)
{
    extern __shared__ __align__(1024) unsigned char tc_smem[];
    __shared__ __align__(8) uint64_t mma_bar;
    __shared__ unsigned tmem_base_s;
    __shared__ __align__(16) float row_c[256];              // pass 2: log2-domain softmax offset of each query row

    const int part = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int S = min(A.seq_lens[b], A.S_max);
    if (S <= A.budget) return;
    const int G = A.Hq / A.Hkv, R = G * A.W, P = S - A.W;
    const int Rpad = (R + 127) / 128 * 128;                   // staged query rows (1 or 2 blocks of 128)
    const int Rn = (R + 15) / 16 * 16;                        // pass 2: N of the MMA
    const int unit = b * A.Hkv + h;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int tile0 = part * A.tiles_per_cta;
    const int n_tiles_total = (S + kTcTile - 1) / kTcTile;
    const int tile1 = min(n_tiles_total, tile0 + A.tiles_per_cta);
    // scores are kept in the log2 domain: 2^(s * log2 e) = e^s, one ex2 per probability
    const float scale = rsqrtf(static_cast<float>(kHeadDim)) * 1.4426950408889634f;

    // operand tiles start on a 1024-byte boundary (the swizzle atom); the launch reserves the slack
    unsigned char* q_s = tc_smem + ((1024u - (tc_smem_u32(tc_smem) & 1023u)) & 1023u);   // [2][Rpad][128 B]
    unsigned char* k_s = q_s + static_cast<size_t>(Rpad) * 256;                            // 2 buffers of [2][128][128 B]
    const int n_cols = (PASS == 1) ? Rpad : (Rn <= 128 ? 128 : 256);   // tensor-memory columns (power of two >= 32)

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(&tmem_base_s)), "r"(n_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tc_smem_u32(&mma_bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // query rows of the group: row = g*W + w  ->  q_win[b][h*G+g][w][:]  (contiguous over (g, w))
    tc_stage_rows(q_s, Rpad, static_cast<const unsigned short*>(A.q_win) + (static_cast<int64_t>(b) * A.Hq + h * G) * A.W * kHeadDim,
                  kHeadDim, R, tid);
    if (PASS == 2)                                         // p = 2^(s - c), c = row max + log2(row sum); padding rows give 0
        for (int r = tid; r < 256; r += kTcThreads)
            row_c[r] = (r < R) ? A.rowstat[(static_cast<int64_t>(unit) * R + r) * 2] +
                                     log2f(A.rowstat[(static_cast<int64_t>(unit) * R + r) * 2 + 1])
                               : INFINITY;
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem = tmem_base_s;
    const unsigned q_u = tc_smem_u32(q_s), k_u0 = tc_smem_u32(k_s);
    const unsigned short* k_unit = static_cast<const unsigned short*>(A.k) + static_cast<int64_t>(b) * A.sb +
                                   static_cast<int64_t>(h) * A.sh;
    if (tile0 < tile1)                                     // first key tile in flight
        tc_stage_rows_async(k_u0, kTcTile, k_unit + static_cast<int64_t>(tile0) * kTcTile * A.st, A.st,
                            min(kTcTile, S - tile0 * kTcTile), tid);

    float run_m[2] = {-INFINITY, -INFINITY}, run_l[2] = {0.f, 0.f};       // pass 1: rows tid and 128 + tid
    unsigned phase = 0;
    bool dead = false;

    for (int tile = tile0; tile < tile1; ++tile) {
        const int t0 = tile * kTcTile;
        const unsigned k_u = k_u0 + static_cast<unsigned>((tile - tile0) & 1) * (kTcTile * 256u);
        asm volatile("cp.async.wait_group 0;" ::: "memory");             // this tile's keys have landed
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // generic-proxy writes -> tensor-core reads
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (tile + 1 < tile1)                                            // next tile into the other buffer
            tc_stage_rows_async(k_u0 + static_cast<unsigned>((tile + 1 - tile0) & 1) * (kTcTile * 256u), kTcTile,
                                k_unit + static_cast<int64_t>(t0 + kTcTile) * A.st, A.st,
                                min(kTcTile, S - (t0 + kTcTile)), tid);
        if (tid == 0 && !dead) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (PASS == 1) {
                const unsigned idesc = tc_idesc(128, kTcTile);
                for (int mb = 0; mb < Rpad / 128; ++mb)
#pragma unroll
                    for (int k16 = 0; k16 < 8; ++k16) {
                        const unsigned koff = (k16 >> 2) * 128u * 128u + (k16 & 3) * 32u;     // 64-channel block, 32 B per k-step
                        tc_mma(tmem + mb * 128, tc_desc(q_u + (k16 >> 2) * (Rpad * 128u) + mb * (128u * 128u) + (k16 & 3) * 32u),
                               tc_desc(k_u + koff), idesc, k16 > 0);
                    }
            } else {
                const unsigned idesc = tc_idesc(128, Rn);
#pragma unroll
                for (int k16 = 0; k16 < 8; ++k16)
                    tc_mma(tmem, tc_desc(k_u + (k16 >> 2) * 128u * 128u + (k16 & 3) * 32u),
                           tc_desc(q_u + (k16 >> 2) * (Rpad * 128u) + (k16 & 3) * 32u), idesc, k16 > 0);
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(tc_smem_u32(&mma_bar)) : "memory");
        }
        // wait for the MMAs of this tile (bounded).  The verdict is made CTA-uniform by the barrier below, so
        // that the warp-collective tensor-memory loads of the epilogue are never executed divergently and,
        // once a wait has run out, no thread issues further MMAs or reads the accumulator.
        {
            unsigned ok = dead ? 1u : 0u;
            for (unsigned it = 0; it < kTcSpin && !ok; ++it)
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(ok) : "r"(tc_smem_u32(&mma_bar)), "r"(phase) : "memory");
            const bool timed_out = __syncthreads_or(!ok) != 0;
            if (timed_out && !dead) {
                dead = true;
                if (tid == 0) record_error(A.status, SPARK_ERR_DEVICE_TIMEOUT);
                // give the MMAs that were issued one more bounded chance to retire before the accumulator is freed
                for (unsigned it = 0; it < kTcSpin && !ok; ++it)
                    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                                 : "=r"(ok) : "r"(tc_smem_u32(&mma_bar)), "r"(phase) : "memory");
            }
        }
        phase ^= 1u;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned lane_addr = tmem + (static_cast<unsigned>(warp * 32) << 16);
        if (!dead) {
            if (PASS == 1) {
                for (int mb = 0; mb < Rpad / 128; ++mb) {
                    const int row = mb * 128 + tid;
                    const bool row_ok = row < R;
                    const int last = P + (row_ok ? row % A.W : 0);
                    float m = run_m[mb], l = run_l[mb];
                    float v[kTcTile];
                    tc_ld128(lane_addr + mb * 128, v);
                    if (t0 + kTcTile <= P + 1) {               // every key of the tile is visible to every window row
                        if (row_ok) {
                            float c4[4] = {v[0], v[1], v[2], v[3]};
#pragma unroll
                            for (int i = 4; i < kTcTile; ++i) c4[i & 3] = fmaxf(c4[i & 3], v[i]);
                            const float mn = fmaxf(m, fmaxf(fmaxf(c4[0], c4[1]), fmaxf(c4[2], c4[3])) * scale);
                            float add[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                            for (int i = 0; i < kTcTile; ++i) add[i & 3] += tc_ex2(fmaf(v[i], scale, -mn));
                            l = l * tc_ex2(m - mn) + ((add[0] + add[1]) + (add[2] + add[3]));
                            m = mn;
                        }
                    } else {
                        float cm = -INFINITY;
#pragma unroll
                        for (int i = 0; i < kTcTile; ++i) {
                            const int t = t0 + i;
                            v[i] = (row_ok && t <= last && t < S) ? v[i] * scale : -INFINITY;
                            cm = fmaxf(cm, v[i]);
                        }
                        if (cm > -INFINITY) {
                            const float mn = fmaxf(m, cm);
                            float add[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                            for (int i = 0; i < kTcTile; ++i) add[i & 3] += tc_ex2(v[i] - mn);    // 2^(-inf) = 0 for masked keys
                            l = l * tc_ex2(m - mn) + ((add[0] + add[1]) + (add[2] + add[3]));
                            m = mn;
                        }
                    }
                    run_m[mb] = m; run_l[mb] = l;
                }
            } else {
                const int t = t0 + tid;
                float vote = 0.f;
#pragma unroll 1
                for (int c0 = 0; c0 < Rn; c0 += 128) {
                    float v[128];
                    tc_ld128(lane_addr + c0, v);
                    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int i = 0; i < 128; i += 4) {
                        const float4 c = *reinterpret_cast<const float4*>(row_c + c0 + i);     // same address for all threads
                        acc[0] += tc_ex2(fmaf(v[i], scale, -c.x));
                        acc[1] += tc_ex2(fmaf(v[i + 1], scale, -c.y));
                        acc[2] += tc_ex2(fmaf(v[i + 2], scale, -c.z));
                        acc[3] += tc_ex2(fmaf(v[i + 3], scale, -c.w));
                    }
                    vote += (acc[0] + acc[1]) + (acc[2] + acc[3]);
                }
                if (t < S) A.votes[static_cast<int64_t>(unit) * A.S_max + t] = (t < P) ? vote : 0.f;
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();                                       // accumulator and key tile are free again
    }
    if (PASS == 1)
        for (int mb = 0; mb < Rpad / 128; ++mb) {
            const int row = mb * 128 + tid;
            if (row < R) {
                float* dst = A.partial + ((static_cast<int64_t>(unit) * R + row) * A.parts + part) * 2;
                dst[0] = (tile1 > tile0 && !dead) ? run_m[mb] : -INFINITY;
                dst[1] = (tile1 > tile0 && !dead) ? run_l[mb] : 0.f;
            }
        }
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(n_cols) : "memory");
}

// merge the per-CTA partials of pass 1 into the rows' softmax normalisers
__global__ void evict_rowstats_tc_kernel(EvictTcArgs A, float* rowstat)
{
    const int h = blockIdx.x, b = blockIdx.y;
    const int S = min(A.seq_lens[b], A.S_max);
    if (S <= A.budget) return;
    const int G = A.Hq / A.Hkv, R = G * A.W;
    const int unit = b * A.Hkv + h;
    for (int row = threadIdx.x; row < R; row += blockDim.x) {
        const float* src = A.partial + (static_cast<int64_t>(unit) * R + row) * A.parts * 2;
        float M = -INFINITY, L = 0.f;
        for (int p = 0; p < A.parts; ++p) {
            const float m = src[2 * p], l = src[2 * p + 1];
            if (m == -INFINITY) continue;
            const float Mn = fmaxf(M, m);
            L = L * exp2f(M - Mn) + l * exp2f(m - Mn);
            M = Mn;
        }
        rowstat[(static_cast<int64_t>(unit) * R + row) * 2] = M;
        rowstat[(static_cast<int64_t>(unit) * R + row) * 2 + 1] = L;
    }
}

bool evict_tc_supported(const spark_params& p)
{
    const int R = (p.n_q_heads / p.n_kv_heads) * p.window;
    return p.dtype == SPARK_BF16 && R <= 256;
}

// Tensor-core votes: same workspace regions as the CUDA-core path (partial, rowstat, votes).
spark_status launch_evict_votes_tc(const spark_params& p, const void* q_win, const void* k, int64_t sb, int64_t sh,
                                   int64_t st, const int32_t* seq_lens, int32_t max_seq_tokens, float* partial,
                                   float* rowstat, float* votes, int* status, cudaStream_t stream, int* launches)
{
    const int R = (p.n_q_heads / p.n_kv_heads) * p.window;
    const int Rpad = (R + 127) / 128 * 128;
    EvictTcArgs A;
    A.q_win = q_win; A.k = k; A.sb = sb; A.sh = sh; A.st = st; A.seq_lens = seq_lens;
    A.Hq = p.n_q_heads; A.Hkv = p.n_kv_heads; A.W = p.window; A.budget = p.token_budget; A.S_max = max_seq_tokens;
    const int n_tiles = (max_seq_tokens + kTcTile - 1) / kTcTile;
    // Two CTAs are resident per SM; a CTA pays a fixed start-up (tensor-memory allocation, the query
    // block, the first key tile), so the tiles are cut into about one wave of CTAs, at least 8 tiles each.
    int dev = 0, n_sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return SPARK_ERR_CUDA;
    const int64_t units = static_cast<int64_t>(p.batch) * p.n_kv_heads;
    const int64_t wave = 2 * static_cast<int64_t>(n_sms);
    int64_t per = (static_cast<int64_t>(n_tiles) * units + wave - 1) / wave;
    if (per < 8) per = 8;
    if (per > n_tiles) per = n_tiles > 0 ? n_tiles : 1;
    A.tiles_per_cta = static_cast<int>(per);
    A.parts = (n_tiles + A.tiles_per_cta - 1) / A.tiles_per_cta;
    A.partial = partial; A.rowstat = rowstat; A.votes = votes; A.status = status;
    const size_t smem = static_cast<size_t>(Rpad) * 256 + 2 * kTcTile * 256 + 1024;     // queries, two key buffers, alignment slack
    if (cudaFuncSetAttribute(evict_scores_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess ||
        cudaFuncSetAttribute(evict_scores_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
        return SPARK_ERR_CUDA;
    const dim3 grid(A.parts, p.n_kv_heads, p.batch), ugrid(p.n_kv_heads, p.batch);
    evict_scores_tc_kernel<1><<<grid, kTcThreads, smem, stream>>>(A);
    evict_rowstats_tc_kernel<<<ugrid, 256, 0, stream>>>(A, rowstat);
    evict_scores_tc_kernel<2><<<grid, kTcThreads, smem, stream>>>(A);
    *launches += 3;
    return cudaGetLastError() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

}  // namespace spark
