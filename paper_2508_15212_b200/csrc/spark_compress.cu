// Prefill-side kernels: window-mean query norm, per-token top-T channel selection + page packing,
// and the inverse (pages -> logical arrays).
//
// Method (paper sections): the mean window query replaces per-token queries (Sec. "SparK"); the
// saliency of channel j of token t is w = |q-bar_j| * |K[t][j]| (Sec. "Problem Formulation"); the T
// channels of largest w are kept (Eq. (cal)); the mean saliency of the pruned channels is cached per
// token (App. "Caching Pruned Channel Statistics").  With value-channel pruning (App. "Pruning Value
// Cache Channels") the same per-token selection runs on |V[t][j]| and the page stores the kept values and a
// second mask instead of the dense value row.
#include "spark_common.cuh"

namespace spark {

constexpr unsigned kFullMask = 0xffffffffu;

// ------------------------------------------------------------------------------------------------
// a[b][h][j] = max(|mean over the G*W window queries of the group|, eps).
// One thread per channel; the sum runs in double over (g outer, w inner), so the rounded mean does
// not depend on launch shape.  Thread 0 of the first head also publishes packed_lens when there is
// no eviction step.
// ------------------------------------------------------------------------------------------------
template <typename E>
__global__ void __launch_bounds__(kHeadDim)
window_qnorm_kernel(const void* __restrict__ q_win, int Hq, int Hkv, int W, float eps,
                    float* __restrict__ qnorm, const int32_t* __restrict__ seq_lens,
                    int32_t* __restrict__ packed_lens, int max_seq_tokens, int* status)
{
    const int h = blockIdx.x, b = blockIdx.y, j = threadIdx.x;
    const int G = Hq / Hkv;
    // the group's G*W window rows are consecutive in memory, (g outer, w inner)
    const int64_t base = ((static_cast<int64_t>(b) * Hq + h * G) * W) * kHeadDim + j;
    const int rows = G * W;
    double acc = 0.0;
    int r = 0;
    for (; r + 32 <= rows; r += 32) {                      // thirty-two loads in flight, summed in order
        float x[32];
#pragma unroll
        for (int u = 0; u < 32; ++u) x[u] = Elem<E>::load(q_win, base + static_cast<int64_t>(r + u) * kHeadDim);
#pragma unroll
        for (int u = 0; u < 32; ++u) acc += static_cast<double>(x[u]);
    }
    for (; r < rows; ++r)
        acc += static_cast<double>(Elem<E>::load(q_win, base + static_cast<int64_t>(r) * kHeadDim));
    const float m = static_cast<float>(acc / static_cast<double>(G * W));
    qnorm[(static_cast<int64_t>(b) * Hkv + h) * kHeadDim + j] = fmaxf(fabsf(m), eps);
    if (packed_lens && h == 0 && j == 0) {
        int len = seq_lens[b];
        if (len < 0 || len > max_seq_tokens) {
            record_error(status, SPARK_ERR_DEVICE_BOUNDS);
            len = len < 0 ? 0 : max_seq_tokens;
        }
        packed_lens[b] = len;
    }
}

// ------------------------------------------------------------------------------------------------
// One token of one KV head, one warp: saliency, exact top-T selection, and the token's entries of a
// page image at `image` (kept values in slot order, mask words, mu).  A lane owns channels
// 4*lane .. 4*lane+3: `kf` are its key values, `raw` their stored bit patterns, `a` its qnorm entries.
//
// Selection is exact: the saliency is one __fmul_rn, its bit pattern (non-negative float) is an
// order-preserving 31-bit key, the T-th largest key is found by a bitwise radix descent with warp
// reductions, and keys equal to it are admitted in ascending channel order until T channels are kept.
//
// The same routine prunes a value row (a = 1, so the key is |V[t][j]| itself): `vals_off` / `mask_off`
// select the section that receives the kept entries and the mask, and mu is written only when
// `mu_off` >= 0 (`inv_pruned` = 1 / (D - T), or 0 when nothing is pruned: the mean is taken as a product
// in double, which rounds to the same float as the quotient except on a rounding boundary of the double).
// ------------------------------------------------------------------------------------------------
// How the kept key channels of a token are chosen, and which statistics the page stores.
struct SelectArgs {
    int select;                   // spark_select
    float top_p;                  // SPARK_SELECT_TOP_P
    unsigned rank_keep[4];        // SPARK_SELECT_GROUPS: bit r set <=> the channel of saliency rank r is kept
    int recovery;                 // spark_recovery: a sampled distribution needs the all-channel statistics
};

// Exact top-T of the warp's 128 keys: kept[i] for the lane's four channels (see pack_token).
__device__ __forceinline__ void select_top_t(const unsigned (&key)[4], int T, int lane, bool (&kept)[4])
{
    const unsigned lt = (1u << lane) - 1u;
    // T-th largest key by radix descent over the bits in which the 128 keys differ.  The descent
    // stops as soon as a candidate threshold has exactly T keys at or above it (then those are the
    // kept set and no tie can straddle the boundary); otherwise it ends with the exact T-th largest
    // key and equal keys are admitted in ascending channel order.
    const unsigned k_or = __reduce_or_sync(kFullMask, key[0] | key[1] | key[2] | key[3]);
    const unsigned k_and = __reduce_and_sync(kFullMask, key[0] & key[1] & key[2] & key[3]);
    const unsigned diff = k_or ^ k_and;
    const int top = diff ? (31 - __clz(diff)) : -1;              // highest bit in which keys differ
    unsigned thr = (top >= 0) ? (k_and & ~((2u << top) - 1u)) : k_and;   // common leading bits
    bool exact = false;
    for (int bit = top; bit >= 0; --bit) {
        const unsigned cand = thr | (1u << bit);
        const int mine = (key[0] >= cand) + (key[1] >= cand) + (key[2] >= cand) + (key[3] >= cand);
        const int cnt = __reduce_add_sync(kFullMask, mine);
        if (cnt >= T) thr = cand;
        if (cnt == T) { exact = true; break; }
    }
    if (exact) {
#pragma unroll
        for (int i = 0; i < 4; ++i) kept[i] = key[i] >= thr;
    } else {
        unsigned eqb[4];
        int c_gt = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            c_gt += __popc(__ballot_sync(kFullMask, key[i] > thr));
            eqb[i] = __ballot_sync(kFullMask, key[i] == thr);
        }
        const int need_eq = T - c_gt;
        int rank = 0;                                        // equal keys on lower channels
#pragma unroll
        for (int i = 0; i < 4; ++i) rank += __popc(eqb[i] & lt);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const bool eq = key[i] == thr;
            kept[i] = key[i] > thr || (eq && rank < need_eq);
            rank += eq ? 1 : 0;
        }
    }
}

// The ratio-free selection rules (Sec. "Ablation Studies", adaptive variants) need every channel's saliency
// RANK, so the warp sorts its 128 keys: a bitonic network over (saliency bits, 127 - channel), descending,
// four consecutive ranks per lane.  SparK-p then keeps the shortest rank prefix whose saliencies (summed in
// double, most salient first) reach top_p of the token's total, at least one and at most `cap` channels;
// SparK-g keeps the ranks listed in rank_keep.  Returns kept[i] for the lane's four CHANNELS and the count.
__device__ __forceinline__ int select_by_rank(const unsigned (&key)[4], int lane, const SelectArgs& sel, int cap,
                                              bool (&kept)[4])
{
    unsigned long long K[4];
#pragma unroll
    for (int e = 0; e < 4; ++e)
        K[e] = (static_cast<unsigned long long>(key[e]) << 7) | static_cast<unsigned>(127 - (4 * lane + e));
#pragma unroll
    for (int size = 2; size <= 128; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            if (stride >= 4) {
                const bool lower = ((4 * lane) & stride) == 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const unsigned long long other = __shfl_xor_sync(kFullMask, K[e], stride >> 2);
                    const bool down = ((4 * lane + e) & size) == 0;     // this block ends up descending
                    const bool take_max = (lower == down);
                    K[e] = take_max ? (K[e] > other ? K[e] : other) : (K[e] < other ? K[e] : other);
                }
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if ((e & stride) == 0) {
                        const bool down = ((4 * lane + e) & size) == 0;
                        const unsigned long long x = K[e], y = K[e ^ stride];
                        const unsigned long long hi = x > y ? x : y, lo = x > y ? y : x;
                        K[e] = down ? hi : lo;
                        K[e ^ stride] = down ? lo : hi;
                    }
            }
        }
    }
    unsigned rk[4] = {sel.rank_keep[0], sel.rank_keep[1], sel.rank_keep[2], sel.rank_keep[3]};
    if (sel.select == SPARK_SELECT_TOP_P) {
        double c[4];
        double run = 0.0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            run += static_cast<double>(__uint_as_float(static_cast<unsigned>(K[e] >> 7)));
            c[e] = run;
        }
        double incl = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(kFullMask, incl, o);
            if (lane >= o) incl += up;
        }
        const double total = __shfl_sync(kFullMask, incl, 31);
        const double need = static_cast<double>(sel.top_p) * total;
        const double before = incl - run;
        int below = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) below += (before + c[e] < need) ? 1 : 0;
        int n = __reduce_add_sync(kFullMask, below) + 1;       // first rank whose running sum reaches `need`
        n = n > kHeadDim ? kHeadDim : n;
        n = n > cap ? cap : n;
#pragma unroll
        for (int wi = 0; wi < 4; ++wi)
            rk[wi] = n >= 32 * (wi + 1) ? 0xffffffffu : (n > 32 * wi ? ((1u << (n - 32 * wi)) - 1u) : 0u);
    }
    unsigned m[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int r = 4 * lane + e;
        if ((rk[r >> 5] >> (r & 31)) & 1u) {
            const int j = 127 - static_cast<int>(K[e] & 127u);
#pragma unroll
            for (int wi = 0; wi < 4; ++wi)
                if ((j >> 5) == wi) m[wi] |= 1u << (j & 31);
        }
    }
    int n_kept = 0;
#pragma unroll
    for (int wi = 0; wi < 4; ++wi) {
        m[wi] = __reduce_or_sync(kFullMask, m[wi]);
        n_kept += __popc(m[wi]);
    }
    unsigned mine = m[0];
#pragma unroll
    for (int wi = 1; wi < 4; ++wi)
        if ((lane >> 3) == wi) mine = m[wi];
#pragma unroll
    for (int i = 0; i < 4; ++i) kept[i] = (mine >> (4 * (lane & 7) + i)) & 1u;
    return n_kept;
}

template <bool kBf16, bool kRank>
__device__ __forceinline__ int pack_token(unsigned char* image, int vals_off, int mask_off, int mu_off,
                                           int p, int T, int lane,
                                           const float (&a)[4], const float (&kf)[4], const unsigned (&raw)[4],
                                           double inv_pruned = 0.0, const SelectArgs* sel = nullptr, int stats_off = -1)
{
    const unsigned lt = (1u << lane) - 1u;
    float w[4];
    unsigned key[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        w[i] = __fmul_rn(a[i], fabsf(kf[i]));                 // the one rounding that decides selection
        key[i] = __float_as_uint(w[i]);
    }
    bool kept[4];
    int n_kept = T;
    if (kRank) n_kept = select_by_rank(key, lane, *sel, T, kept);     // a ratio-free rule (keys only)
    else select_top_t(key, T, lane, kept);
    // slot of each kept channel = kept channels below it
    int slot = 0;
    unsigned nib = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        slot += __popc(__ballot_sync(kFullMask, kept[i]) & lt);
        nib |= kept[i] ? (1u << i) : 0u;
    }
    double pruned = 0.0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (kept[i]) {
            unsigned char* dst = image + vals_off + val_offset(kBf16 ? 2 : 4, p, slot);
            if (kBf16) *reinterpret_cast<unsigned short*>(dst) = static_cast<unsigned short>(raw[i]);
            else *reinterpret_cast<unsigned*>(dst) = raw[i];
            ++slot;
        } else {
            pruned += static_cast<double>(w[i]);
        }
    }
    unsigned word = nib << (4 * (lane & 7));
    word |= __shfl_xor_sync(kFullMask, word, 1);
    word |= __shfl_xor_sync(kFullMask, word, 2);
    word |= __shfl_xor_sync(kFullMask, word, 4);
    if ((lane & 7) == 0)
        reinterpret_cast<unsigned*>(image + mask_off)[p * kMaskWords + (lane >> 3)] = word;
    if (mu_off < 0) return n_kept;                            // warp-uniform
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) pruned += __shfl_xor_sync(kFullMask, pruned, o);
    if (lane == 0) {
        float mu;
        if (kRank)
            mu = n_kept < kHeadDim ? static_cast<float>(pruned / static_cast<double>(kHeadDim - n_kept)) : 0.f;
        else
            mu = static_cast<float>(pruned * inv_pruned);
        reinterpret_cast<float*>(image + mu_off)[p] = mu;
    }
    if (stats_off < 0) return n_kept;                         // warp-uniform
    // all-channel mean and population deviation of the token's saliencies (sampled recovery)
    double s1 = (static_cast<double>(w[0]) + static_cast<double>(w[1])) + (static_cast<double>(w[2]) + static_cast<double>(w[3]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s1 += __shfl_xor_sync(kFullMask, s1, o);
    const double mean = s1 / static_cast<double>(kHeadDim);
    double s2 = 0.0;
#pragma unroll
    for (int i = 0; i < 4; ++i) { const double d = static_cast<double>(w[i]) - mean; s2 += d * d; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s2 += __shfl_xor_sync(kFullMask, s2, o);
    if (lane == 0) {
        reinterpret_cast<float*>(image + stats_off)[p] = static_cast<float>(mean);
        reinterpret_cast<float*>(image + stats_off)[kPageTokens + p] = static_cast<float>(sqrt(s2 / static_cast<double>(kHeadDim)));
    }
    return n_kept;
}

// Key entries and value entries of one token row into the page image.  A lane owns channels 4*lane ..
// 4*lane+3; `row` is the element offset of its first channel in k and v.  `inv_pruned` = 1 / (D - T)
// (0 when T = D), computed once on the host.
template <bool kBf16, bool kRank>
__device__ __forceinline__ int pack_token_kv(unsigned char* image, const PageLayout& L, int p, int lane,
                                              const float (&a)[4], const void* k, const void* v, int64_t row,
                                              double inv_pruned, const SelectArgs& sel)
{
    unsigned kraw[4], vraw[4];
    float kf[4];
    if (kBf16) {
        const uint2 kk = *reinterpret_cast<const uint2*>(static_cast<const unsigned short*>(k) + row);
        const uint2 vv = *reinterpret_cast<const uint2*>(static_cast<const unsigned short*>(v) + row);
        kraw[0] = kk.x & 0xffffu; kraw[1] = kk.x >> 16; kraw[2] = kk.y & 0xffffu; kraw[3] = kk.y >> 16;
#pragma unroll
        for (int i = 0; i < 4; ++i) kf[i] = __uint_as_float(kraw[i] << 16);
        if (L.keep_v < kHeadDim) {
            vraw[0] = vv.x & 0xffffu; vraw[1] = vv.x >> 16; vraw[2] = vv.y & 0xffffu; vraw[3] = vv.y >> 16;
        } else {
            *reinterpret_cast<uint2*>(image + L.v_off + v_chunk_offset(2, p, lane >> 1) + (lane & 1) * 8) = vv;
        }
    } else {
        const uint4 kk = *reinterpret_cast<const uint4*>(static_cast<const float*>(k) + row);
        const uint4 vv = *reinterpret_cast<const uint4*>(static_cast<const float*>(v) + row);
        kraw[0] = kk.x; kraw[1] = kk.y; kraw[2] = kk.z; kraw[3] = kk.w;
#pragma unroll
        for (int i = 0; i < 4; ++i) kf[i] = __uint_as_float(kraw[i]);
        if (L.keep_v < kHeadDim) { vraw[0] = vv.x; vraw[1] = vv.y; vraw[2] = vv.z; vraw[3] = vv.w; }
        else *reinterpret_cast<uint4*>(image + L.v_off + v_chunk_offset(4, p, lane)) = vv;
    }
    if (L.keep_v < kHeadDim) {                             // value-channel pruning: same selection on |V|
        float vf[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) vf[i] = __uint_as_float(kBf16 ? vraw[i] << 16 : vraw[i]);
        const float one[4] = {1.f, 1.f, 1.f, 1.f};
        pack_token<kBf16, false>(image, L.v_off, L.vmask_off, -1, p, L.keep_v, lane, one, vf, vraw);
    }
    return pack_token<kBf16, kRank>(image, L.vals_off, L.mask_off, L.mu_off, p, L.keep, lane, a, kf, kraw, inv_pruned, &sel,
                             L.recovery != SPARK_RECOVER_DEGENERATE ? L.stats_off : -1);
}

// ------------------------------------------------------------------------------------------------
// One CTA builds one page (16 tokens of one KV head) in shared memory and writes it out with
// coalesced 16-byte stores.  One warp per token, two rounds; a lane owns channels 4*lane .. 4*lane+3.
//
// Selection is exact: the saliency is one __fmul_rn, its bit pattern (non-negative float) is an
// order-preserving 31-bit key, the T-th largest key is found by a bitwise radix descent with warp
// ballots, and keys equal to it are admitted in ascending channel order until T channels are kept.
// ------------------------------------------------------------------------------------------------
struct CompressArgs {
    const void* k;
    const void* v;
    int64_t sb, sh, st;
    const int32_t* lens;          // tokens per sequence AFTER eviction (packed lens)
    const int32_t* gather;        // optional [B][Hkv][gather_stride] source token positions
    int gather_stride;
    const float* qnorm;
    unsigned char* pages;
    const int32_t* block_table;
    int max_blocks;
    int Hkv;
    int keep;
    int64_t n_pool_pages;
    PageLayout L;
    double inv_pruned;            // 1 / (D - T), 0 when T = D
    SelectArgs sel;
    int* status;
};

template <typename E, bool kRank>
__global__ void __launch_bounds__(256) compress_pages_kernel(CompressArgs A)
{
    extern __shared__ __align__(16) unsigned char image[];
    const int blk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int len = A.lens[b];
    if (blk * kPageTokens >= len) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const PageLayout L = A.L;
    constexpr bool kBf16 = (sizeof(E) == 2);

    __shared__ int rows_used;
    if (threadIdx.x == 0) rows_used = 0;
    for (int i = threadIdx.x; i < L.page_bytes / 16; i += blockDim.x)
        reinterpret_cast<uint4*>(image)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();

    const float4 a4 = reinterpret_cast<const float4*>(
        A.qnorm + (static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim)[lane];
    const float a[4] = {a4.x, a4.y, a4.z, a4.w};
    for (int p = warp; p < kPageTokens; p += 8) {
        const int t = blk * kPageTokens + p;
        if (t >= len) continue;                                   // warp-uniform
        const int src_t = A.gather
            ? A.gather[(static_cast<int64_t>(b) * A.Hkv + h) * A.gather_stride + t] : t;
        const int64_t row = static_cast<int64_t>(b) * A.sb + static_cast<int64_t>(h) * A.sh +
                            static_cast<int64_t>(src_t) * A.st + lane * 4;
        const int n_kept = pack_token_kv<kBf16, kRank>(image, L, p, lane, a, A.k, A.v, row, A.inv_pruned, A.sel);
        if (kRank && L.ragged && lane == 0) atomicMax(&rows_used, n_kept);
    }
    __syncthreads();

    const int64_t entry = (static_cast<int64_t>(b) * A.Hkv + h) * A.max_blocks + blk;
    const int64_t page_id = A.block_table ? A.block_table[entry] : entry;     // no table: contiguous cache
    if (page_id < 0 || page_id >= A.n_pool_pages) {
        if (threadIdx.x == 0) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
        return;
    }
    uint4* dst = reinterpret_cast<uint4*>(A.pages + page_id * L.page_bytes);
    for (int i = threadIdx.x; i < L.page_bytes / 16; i += blockDim.x)
        dst[i] = reinterpret_cast<const uint4*>(image)[i];
    if (kRank && L.ragged && threadIdx.x == 0)
        reinterpret_cast<int*>(A.pages + rows_offset(A.n_pool_pages, L.page_bytes))[page_id] = rows_used;
}

// ------------------------------------------------------------------------------------------------
// Fixed-T pages, four tokens per warp.  Most of what the selection costs per token is warp-wide
// bookkeeping (reductions, votes, loop control) that serves one token when a warp owns one token.  Here a
// token belongs to EIGHT lanes (16 channels per lane), a warp carries four tokens through the same
// instructions, and the radix descent compares two keys per instruction while it works on the keys' upper
// 16 bits (the bf16 image of a non-negative float orders like the float): `set.ge.u32.bf16x2` yields a
// 0xFFFF / 0 half-word mask per key, eight such masks are folded into one word with one logic op each and
// counted with one population count.  Below bit 16 the descent continues on the full keys.  The result is
// the same exact top-T set, with ties to the lower channel, as select_top_t.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int group8_sum(int v)              // (a masked hardware reduction measured slower)
{
    v += __shfl_xor_sync(kFullMask, v, 1);
    v += __shfl_xor_sync(kFullMask, v, 2);
    v += __shfl_xor_sync(kFullMask, v, 4);
    return v;
}
__device__ __forceinline__ double group8_sum(double v)
{
    v += __shfl_xor_sync(kFullMask, v, 1);
    v += __shfl_xor_sync(kFullMask, v, 2);
    v += __shfl_xor_sync(kFullMask, v, 4);
    return v;
}
__device__ __forceinline__ int group8_exclusive(int v, int l8)      // sum over the lower lanes of the group
{
    int x = v;
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
        const int y = __shfl_up_sync(kFullMask, x, o, 8);
        if (l8 >= o) x += y;
    }
    return x - v;
}
// per half: 1.0 (bf16) where a >= b, else 0 -- on the half-precision pipe, so that counting the keys at or
// above a candidate costs the integer pipe nothing
__device__ __forceinline__ __nv_bfloat162 ge_one_bf16x2(unsigned a, unsigned b)
{
    return __hge2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
}

// kept bits (bit i <=> the lane's channel i) of the exact top-T among the 128 keys of the lane's group
__device__ __forceinline__ unsigned select_top_t16(const unsigned (&key)[16], int T, int l8)
{
    unsigned hk[8];                                              // upper halves of the keys, two per word
#pragma unroll
    for (int i = 0; i < 8; ++i) hk[i] = (key[2 * i] >> 16) | (key[2 * i + 1] & 0xffff0000u);
    // bits in which the group's keys differ: from the upper halves, and from the full keys only when the
    // upper halves all agree
    unsigned o = hk[0], n = hk[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) { o |= hk[i]; n &= hk[i]; }
    o |= o << 16; n &= n << 16;                                  // fold the two keys of a word into the upper half
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) {
        o |= __shfl_xor_sync(kFullMask, o, d);
        n &= __shfl_xor_sync(kFullMask, n, d);
    }
    o &= 0xffff0000u; n &= 0xffff0000u;
    if (__any_sync(kFullMask, o == n)) {                         // rare: some group's keys share their upper halves
        unsigned o2 = key[0], n2 = key[0];
#pragma unroll
        for (int i = 1; i < 16; ++i) { o2 |= key[i]; n2 &= key[i]; }
#pragma unroll
        for (int d = 1; d < 8; d <<= 1) {
            o2 |= __shfl_xor_sync(kFullMask, o2, d);
            n2 &= __shfl_xor_sync(kFullMask, n2, d);
        }
        o = o2; n = n2;
    } else {
        o |= 0xffffu;                                            // lower halves: treated as differing everywhere
    }
    const unsigned diff = o ^ n;
    const int top = diff ? (31 - __clz(diff)) : -1;              // highest bit in which the group's keys differ
    unsigned thr = (top >= 0) ? (n & ~((2u << top) - 1u)) : n;   // common leading bits
    bool done = top < 0, exact = false;
    const int start = __reduce_max_sync(kFullMask, top);
    int bit = start;
    for (; bit >= 16; --bit) {
        if (__all_sync(kFullMask, done)) break;
        const bool act = !done && bit <= top;
        const unsigned cand = thr | (1u << bit);
        const unsigned c2 = (cand >> 16) * 0x00010001u;
        __nv_bfloat162 g[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) g[i] = ge_one_bf16x2(hk[i], c2);
        const __nv_bfloat162 acc = __hadd2(__hadd2(__hadd2(g[0], g[1]), __hadd2(g[2], g[3])),
                                           __hadd2(__hadd2(g[4], g[5]), __hadd2(g[6], g[7])));   // counts <= 8: exact in bf16
        const int cnt = group8_sum(static_cast<int>(__low2float(acc) + __high2float(acc)));
        if (act && cnt >= T) thr = cand;
        if (act && cnt == T) { exact = true; done = true; }
    }
    for (bit = bit > 15 ? 15 : bit; bit >= 0; --bit) {
        if (__all_sync(kFullMask, done)) break;
        const bool act = !done && bit <= top;
        const unsigned cand = thr | (1u << bit);
        int mine = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) mine += (key[i] >= cand) ? 1 : 0;
        const int cnt = group8_sum(mine);
        if (act && cnt >= T) thr = cand;
        if (act && cnt == T) { exact = true; done = true; }
    }
    unsigned kept = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) kept |= (key[i] >= thr) ? (1u << i) : 0u;
    if (__any_sync(kFullMask, !exact)) {
        // not an exact split: thr is the T-th largest key and the keys equal to it are admitted in ascending
        // channel order (lanes ascending, channels inside a lane ascending) until T channels are kept
        int n_gt = 0, n_eq = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            n_gt += (key[i] > thr) ? 1 : 0;
            n_eq += (key[i] == thr) ? 1 : 0;
        }
        const int need_eq = T - group8_sum(n_gt);
        int rank = group8_exclusive(n_eq, l8);
        if (!exact) {
            kept = 0;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const bool eq = key[i] == thr;
                if (key[i] > thr || (eq && rank < need_eq)) kept |= 1u << i;
                rank += eq ? 1 : 0;
            }
        }
    }
    return kept;
}

// One token of one KV head handled by the eight lanes of a group: saliency, selection, and the token's
// entries of the page image.  The lane owns channels 16*l8 .. 16*l8+15; `raw` holds their stored bit patterns
// (two bf16 per word, or one fp32 per word).  Same outputs as pack_token.
template <bool kBf16>
__device__ __forceinline__ void pack_token16(unsigned char* image, int vals_off, int mask_off, int mu_off,
                                             int stats_off, int p, int T, int l8, bool live,
                                             const float* __restrict__ a, const unsigned* raw, double inv_pruned)
{
    unsigned key[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float kf = kBf16 ? __uint_as_float((i & 1) ? (raw[i >> 1] & 0xffff0000u) : (raw[i >> 1] << 16))
                               : __uint_as_float(raw[i]);
        key[i] = __float_as_uint(__fmul_rn(a ? a[i] : 1.f, fabsf(kf)));     // the one rounding that decides selection
    }
    const unsigned kept = select_top_t16(key, T, l8);
    const int slot0 = group8_exclusive(__popc(kept), l8);
    double pruned = 0.0, s1 = 0.0;
    if (live) {
        unsigned char* dst = image + vals_off + val_offset(kBf16 ? 2 : 4, p, slot0);
        constexpr int kRow = kPageTokens * (kBf16 ? 2 : 4);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            if ((kept >> i) & 1u) {
                if (kBf16) *reinterpret_cast<unsigned short*>(dst) =
                               static_cast<unsigned short>((i & 1) ? (raw[i >> 1] >> 16) : (raw[i >> 1] & 0xffffu));
                else *reinterpret_cast<unsigned*>(dst) = raw[i];
                dst += kRow;
            } else {
                pruned += static_cast<double>(__uint_as_float(key[i]));
            }
        }
    }
    const unsigned other = __shfl_xor_sync(kFullMask, kept, 1);
    if (live && (l8 & 1) == 0)
        reinterpret_cast<unsigned*>(image + mask_off)[p * kMaskWords + (l8 >> 1)] = kept | (other << 16);
    if (mu_off < 0) return;                                   // warp-uniform
    pruned = group8_sum(pruned);
    if (live && l8 == 0) reinterpret_cast<float*>(image + mu_off)[p] = static_cast<float>(pruned * inv_pruned);
    if (stats_off < 0) return;                                // warp-uniform
#pragma unroll
    for (int i = 0; i < 16; ++i) s1 += static_cast<double>(__uint_as_float(key[i]));
    const double mean = group8_sum(s1) / static_cast<double>(kHeadDim);
    double s2 = 0.0;
#pragma unroll
    for (int i = 0; i < 16; ++i) { const double d = static_cast<double>(__uint_as_float(key[i])) - mean; s2 += d * d; }
    s2 = group8_sum(s2);
    if (live && l8 == 0) {
        reinterpret_cast<float*>(image + stats_off)[p] = static_cast<float>(mean);
        reinterpret_cast<float*>(image + stats_off)[kPageTokens + p] = static_cast<float>(sqrt(s2 / static_cast<double>(kHeadDim)));
    }
}

template <typename E>
__global__ void __launch_bounds__(128, 8) compress_pages4_kernel(CompressArgs A)
{
    extern __shared__ __align__(16) unsigned char image[];
    constexpr bool kBf16 = (sizeof(E) == 2);
    constexpr int kWords = kBf16 ? 8 : 16;                     // 32-bit words of a lane's 16 channels
    const int blk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int len = A.lens[b];
    if (blk * kPageTokens >= len) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, l8 = lane & 7;
    const int p = warp * 4 + (lane >> 3);                      // this group's token of the page
    const PageLayout L = A.L;

    for (int i = threadIdx.x; i < L.page_bytes / 16; i += blockDim.x)
        reinterpret_cast<uint4*>(image)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();

    float a[16];
    {
        const float4* src = reinterpret_cast<const float4*>(A.qnorm + (static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim) + 4 * l8;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 f = src[i];
            a[4 * i] = f.x; a[4 * i + 1] = f.y; a[4 * i + 2] = f.z; a[4 * i + 3] = f.w;
        }
    }
    const int t = blk * kPageTokens + p;
    const bool live = t < len;
    unsigned kraw[kWords], vraw[kWords];
#pragma unroll
    for (int i = 0; i < kWords; ++i) { kraw[i] = 0u; vraw[i] = 0u; }
    if (live) {
        const int src_t = A.gather ? A.gather[(static_cast<int64_t>(b) * A.Hkv + h) * A.gather_stride + t] : t;
        const int64_t row = static_cast<int64_t>(b) * A.sb + static_cast<int64_t>(h) * A.sh +
                            static_cast<int64_t>(src_t) * A.st + l8 * 16;
        const uint4* ks = reinterpret_cast<const uint4*>(static_cast<const E*>(A.k) + row);
        const uint4* vs = reinterpret_cast<const uint4*>(static_cast<const E*>(A.v) + row);
#pragma unroll
        for (int i = 0; i < kWords / 4; ++i) {
            const uint4 kk = ks[i], vv = vs[i];
            kraw[4 * i] = kk.x; kraw[4 * i + 1] = kk.y; kraw[4 * i + 2] = kk.z; kraw[4 * i + 3] = kk.w;
            vraw[4 * i] = vv.x; vraw[4 * i + 1] = vv.y; vraw[4 * i + 2] = vv.z; vraw[4 * i + 3] = vv.w;
        }
        if (L.keep_v >= kHeadDim) {                        // dense value row: the lane's 16-byte chunks
#pragma unroll
            for (int i = 0; i < kWords / 4; ++i)
                *reinterpret_cast<uint4*>(image + L.v_off + v_chunk_offset(kBf16 ? 2 : 4, p, (kWords / 4) * l8 + i)) =
                    make_uint4(vraw[4 * i], vraw[4 * i + 1], vraw[4 * i + 2], vraw[4 * i + 3]);
        }
    }
    if (L.keep_v < kHeadDim)                               // value-channel pruning: same selection on |V|
        pack_token16<kBf16>(image, L.v_off, L.vmask_off, -1, -1, p, L.keep_v, l8, live, nullptr, vraw, 0.0);
    pack_token16<kBf16>(image, L.vals_off, L.mask_off, L.mu_off,
                        L.recovery != SPARK_RECOVER_DEGENERATE ? L.stats_off : -1, p, L.keep, l8, live, a, kraw,
                        A.inv_pruned);
    __syncthreads();

    const int64_t entry = (static_cast<int64_t>(b) * A.Hkv + h) * A.max_blocks + blk;
    const int64_t page_id = A.block_table ? A.block_table[entry] : entry;     // no table: contiguous cache
    if (page_id < 0 || page_id >= A.n_pool_pages) {
        if (threadIdx.x == 0) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
        return;
    }
    uint4* dst = reinterpret_cast<uint4*>(A.pages + page_id * L.page_bytes);
    for (int i = threadIdx.x; i < L.page_bytes / 16; i += blockDim.x)
        dst[i] = reinterpret_cast<const uint4*>(image)[i];
}

// ------------------------------------------------------------------------------------------------
// Decode-time append: one new token per sequence is pruned with the sequence's prefill statistics
// (qnorm) and written into the next token slot of its last page (a fresh page is zeroed first).
// One warp per (sequence, KV head).  With more than 32 KV heads: a CTA per warp, and a second
// one-thread-per-sequence kernel advances packed_lens; otherwise one launch does both (below).
// ------------------------------------------------------------------------------------------------
struct AppendArgs {
    const void* k_new;
    const void* v_new;
    unsigned char* pages;
    const int32_t* block_table;
    int max_blocks;
    int B, Hkv, keep;
    int64_t n_pool_pages;
    PageLayout L;
    const float* qnorm;
    int32_t* packed_lens;
    double inv_pruned;            // 1 / (D - T), 0 when T = D
    SelectArgs sel;
    int* status;
};

template <typename E, bool kRank>
__global__ void __launch_bounds__(32) append_token_kernel(AppendArgs A)
{
    constexpr bool kBf16 = (sizeof(E) == 2);
    const int h = blockIdx.x, b = blockIdx.y, lane = threadIdx.x;
    const PageLayout L = A.L;
    const int t = A.packed_lens[b];
    const int blk = t / kPageTokens, p = t - blk * kPageTokens;
    if (t < 0 || blk >= A.max_blocks) {                       // no room: recorded, nothing written
        if (lane == 0) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
        return;
    }
    const int64_t entry = (static_cast<int64_t>(b) * A.Hkv + h) * A.max_blocks + blk;
    const int64_t page_id = A.block_table ? A.block_table[entry] : entry;
    if (page_id < 0 || page_id >= A.n_pool_pages) {
        if (lane == 0) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
        return;
    }
    unsigned char* page = A.pages + page_id * L.page_bytes;
    int* rows = L.ragged ? reinterpret_cast<int*>(A.pages + rows_offset(A.n_pool_pages, L.page_bytes)) + page_id : nullptr;
    if (p == 0) {                                             // first token of a page: clear it
        for (int i = lane; i < L.page_bytes / 16; i += 32) reinterpret_cast<uint4*>(page)[i] = make_uint4(0, 0, 0, 0);
        if (rows && lane == 0) *rows = 0;
        __syncwarp();
    }
    const float4 a4 = reinterpret_cast<const float4*>(A.qnorm + (static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim)[lane];
    const float a[4] = {a4.x, a4.y, a4.z, a4.w};
    const int64_t row = (static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim + lane * 4;
    const int n_kept = pack_token_kv<kBf16, kRank>(page, L, p, lane, a, A.k_new, A.v_new, row, A.inv_pruned, A.sel);
    if (rows && lane == 0) atomicMax(rows, n_kept);
}

// The same for up to 32 KV heads in ONE launch: a CTA per sequence, a warp per KV head.  Every warp reads the
// sequence's length before the first barrier and thread 0 advances it after the second, so no warp can see
// the advanced length.
template <typename E, bool kRank>
__global__ void __launch_bounds__(1024) append_token_cta_kernel(AppendArgs A)
{
    constexpr bool kBf16 = (sizeof(E) == 2);
    const int b = blockIdx.x, h = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const PageLayout L = A.L;
    const int t = A.packed_lens[b];
    __syncthreads();
    const int blk = t / kPageTokens, p = t - blk * kPageTokens;
    const bool room = t >= 0 && blk < A.max_blocks;
    if (!room) {                                               // no room: recorded, nothing written
        if (threadIdx.x == 0) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
    } else {
        const int64_t entry = (static_cast<int64_t>(b) * A.Hkv + h) * A.max_blocks + blk;
        const int64_t page_id = A.block_table ? A.block_table[entry] : entry;
        if (page_id < 0 || page_id >= A.n_pool_pages) {
            if (lane == 0) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
        } else {
            unsigned char* page = A.pages + page_id * L.page_bytes;
            int* rows = L.ragged ? reinterpret_cast<int*>(A.pages + rows_offset(A.n_pool_pages, L.page_bytes)) + page_id : nullptr;
            if (p == 0) {                                      // first token of a page: clear it
                for (int i = lane; i < L.page_bytes / 16; i += 32) reinterpret_cast<uint4*>(page)[i] = make_uint4(0, 0, 0, 0);
                if (rows && lane == 0) *rows = 0;
                __syncwarp();
            }
            const float4 a4 = reinterpret_cast<const float4*>(A.qnorm + (static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim)[lane];
            const float a[4] = {a4.x, a4.y, a4.z, a4.w};
            const int64_t row = (static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim + lane * 4;
            const int n_kept = pack_token_kv<kBf16, kRank>(page, L, p, lane, a, A.k_new, A.v_new, row, A.inv_pruned, A.sel);
            if (rows && lane == 0) atomicMax(rows, n_kept);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && room) A.packed_lens[b] = t + 1;
}

__global__ void append_advance_kernel(AppendArgs A)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= A.B) return;
    const int t = A.packed_lens[b];
    if (t >= 0 && t / kPageTokens < A.max_blocks) A.packed_lens[b] = t + 1;
}

// Block append: n_new tokens per sequence at once (the keys a caller has kept dense for a while and now hands
// over for pruning).  Three launches: fresh pages are zeroed, every (sequence, head, new token) gets a warp that
// prunes it exactly like append_token_kernel, packed_lens advances by the tokens that found room.
struct AppendBlockArgs {
    AppendArgs a;
    int n_new;
};

__global__ void __launch_bounds__(32) append_block_clear_kernel(AppendBlockArgs B_)
{
    const AppendArgs& A = B_.a;
    const int h = blockIdx.x, b = blockIdx.y, lane = threadIdx.x;
    const int t0 = A.packed_lens[b];
    if (t0 < 0) return;
    const int blk = (t0 + kPageTokens - 1) / kPageTokens + static_cast<int>(blockIdx.z);   // pages that start at or after t0
    if (static_cast<int64_t>(blk) * kPageTokens >= static_cast<int64_t>(t0) + B_.n_new || blk >= A.max_blocks) return;
    const int64_t entry = (static_cast<int64_t>(b) * A.Hkv + h) * A.max_blocks + blk;
    const int64_t page_id = A.block_table ? A.block_table[entry] : entry;
    if (page_id < 0 || page_id >= A.n_pool_pages) {
        if (lane == 0) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
        return;
    }
    uint4* page = reinterpret_cast<uint4*>(A.pages + page_id * A.L.page_bytes);
    for (int i = lane; i < A.L.page_bytes / 16; i += 32) page[i] = make_uint4(0, 0, 0, 0);
    if (A.L.ragged && lane == 0)
        reinterpret_cast<int*>(A.pages + rows_offset(A.n_pool_pages, A.L.page_bytes))[page_id] = 0;
}

template <typename E, bool kRank>
__global__ void __launch_bounds__(32) append_block_token_kernel(AppendBlockArgs B_)
{
    constexpr bool kBf16 = (sizeof(E) == 2);
    const AppendArgs& A = B_.a;
    const int h = blockIdx.x, b = blockIdx.y, tok = blockIdx.z, lane = threadIdx.x;
    const PageLayout L = A.L;
    const int t0 = A.packed_lens[b];
    const int64_t t = static_cast<int64_t>(t0) + tok;
    const int64_t blk = t / kPageTokens;
    const int p = static_cast<int>(t - blk * kPageTokens);
    if (t0 < 0 || blk >= A.max_blocks) {                      // no room: recorded, nothing written
        if (lane == 0) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
        return;
    }
    const int64_t entry = (static_cast<int64_t>(b) * A.Hkv + h) * A.max_blocks + blk;
    const int64_t page_id = A.block_table ? A.block_table[entry] : entry;
    if (page_id < 0 || page_id >= A.n_pool_pages) {
        if (lane == 0) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
        return;
    }
    unsigned char* page = A.pages + page_id * L.page_bytes;
    const float4 a4 = reinterpret_cast<const float4*>(A.qnorm + (static_cast<int64_t>(b) * A.Hkv + h) * kHeadDim)[lane];
    const float a[4] = {a4.x, a4.y, a4.z, a4.w};
    const int64_t row = ((static_cast<int64_t>(b) * A.Hkv + h) * B_.n_new + tok) * kHeadDim + lane * 4;
    const int n_kept = pack_token_kv<kBf16, kRank>(page, L, p, lane, a, A.k_new, A.v_new, row, A.inv_pruned, A.sel);
    if (L.ragged && lane == 0)
        atomicMax(reinterpret_cast<int*>(A.pages + rows_offset(A.n_pool_pages, L.page_bytes)) + page_id, n_kept);
}

__global__ void append_block_advance_kernel(AppendBlockArgs B_)
{
    const AppendArgs& A = B_.a;
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= A.B) return;
    const int t = A.packed_lens[b];
    if (t < 0) return;
    const int64_t room = static_cast<int64_t>(A.max_blocks) * kPageTokens;
    const int64_t want = static_cast<int64_t>(t) + B_.n_new;
    A.packed_lens[b] = static_cast<int>(want < room ? want : (t > room ? t : room));
}

// selection arguments of a parameter block (the rank mask of SparK-g is laid out on the host)
static SelectArgs make_select(const spark_params& p)
{
    SelectArgs s;
    s.select = p.select; s.top_p = p.top_p; s.recovery = p.recovery;
    s.rank_keep[0] = s.rank_keep[1] = s.rank_keep[2] = s.rank_keep[3] = 0u;
    if (p.select == SPARK_SELECT_GROUPS) {
        int start = 0;
        for (int i = 0; i < p.n_groups; ++i) {
            const int size = kHeadDim / p.n_groups + (i < kHeadDim % p.n_groups ? 1 : 0);
            const int kp = group_keep(size, 1, &p.group_prune[i]);          // floor((1 - prune) * size)
            for (int r = start; r < start + kp; ++r) s.rank_keep[r >> 5] |= 1u << (r & 31);
            start += size;
        }
    }
    return s;
}

spark_status launch_append(const spark_params& p, const void* k_new, const void* v_new, void* pages,
                           const int32_t* block_table, int32_t max_blocks, const float* qnorm,
                           int32_t* packed_lens, void* workspace, cudaStream_t stream, int* launches)
{
    AppendArgs A;
    A.k_new = k_new; A.v_new = v_new; A.pages = static_cast<unsigned char*>(pages); A.block_table = block_table;
    A.max_blocks = max_blocks; A.B = p.batch; A.Hkv = p.n_kv_heads; A.keep = p.keep; A.n_pool_pages = p.n_pool_pages;
    A.L = make_layout(p); A.qnorm = qnorm; A.packed_lens = packed_lens;
    A.inv_pruned = p.keep < kHeadDim ? 1.0 / static_cast<double>(kHeadDim - p.keep) : 0.0;
    A.sel = make_select(p);
    A.status = static_cast<int*>(workspace);
    const bool rank = p.select != SPARK_SELECT_FIXED;
    if (p.n_kv_heads <= 32) {                                  // one launch: a CTA per sequence, a warp per KV head
        const int threads = p.n_kv_heads * 32;
        if (p.dtype == SPARK_BF16) {
            if (rank) append_token_cta_kernel<__nv_bfloat16, true><<<p.batch, threads, 0, stream>>>(A);
            else append_token_cta_kernel<__nv_bfloat16, false><<<p.batch, threads, 0, stream>>>(A);
        } else {
            if (rank) append_token_cta_kernel<float, true><<<p.batch, threads, 0, stream>>>(A);
            else append_token_cta_kernel<float, false><<<p.batch, threads, 0, stream>>>(A);
        }
        *launches += 1;
        return cudaGetLastError() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
    }
    const dim3 grid(p.n_kv_heads, p.batch);
    if (p.dtype == SPARK_BF16) {
        if (rank) append_token_kernel<__nv_bfloat16, true><<<grid, 32, 0, stream>>>(A);
        else append_token_kernel<__nv_bfloat16, false><<<grid, 32, 0, stream>>>(A);
    } else {
        if (rank) append_token_kernel<float, true><<<grid, 32, 0, stream>>>(A);
        else append_token_kernel<float, false><<<grid, 32, 0, stream>>>(A);
    }
    append_advance_kernel<<<(p.batch + 127) / 128, 128, 0, stream>>>(A);
    *launches += 2;
    return cudaGetLastError() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

spark_status launch_append_block(const spark_params& p, const void* k_new, const void* v_new, int32_t n_new,
                                 void* pages, const int32_t* block_table, int32_t max_blocks, const float* qnorm,
                                 int32_t* packed_lens, void* workspace, cudaStream_t stream, int* launches)
{
    if (n_new == 0) return SPARK_OK;
    AppendBlockArgs Bk;
    AppendArgs& A = Bk.a;
    A.k_new = k_new; A.v_new = v_new; A.pages = static_cast<unsigned char*>(pages); A.block_table = block_table;
    A.max_blocks = max_blocks; A.B = p.batch; A.Hkv = p.n_kv_heads; A.keep = p.keep; A.n_pool_pages = p.n_pool_pages;
    A.L = make_layout(p); A.qnorm = qnorm; A.packed_lens = packed_lens;
    A.inv_pruned = p.keep < kHeadDim ? 1.0 / static_cast<double>(kHeadDim - p.keep) : 0.0;
    A.sel = make_select(p);
    A.status = static_cast<int*>(workspace);
    Bk.n_new = n_new;
    const int fresh = (n_new + kPageTokens - 1) / kPageTokens + 1;       // pages that can start inside the new tokens
    append_block_clear_kernel<<<dim3(p.n_kv_heads, p.batch, fresh), 32, 0, stream>>>(Bk);
    const dim3 grid(p.n_kv_heads, p.batch, n_new);
    const bool rank = p.select != SPARK_SELECT_FIXED;
    if (p.dtype == SPARK_BF16) {
        if (rank) append_block_token_kernel<__nv_bfloat16, true><<<grid, 32, 0, stream>>>(Bk);
        else append_block_token_kernel<__nv_bfloat16, false><<<grid, 32, 0, stream>>>(Bk);
    } else {
        if (rank) append_block_token_kernel<float, true><<<grid, 32, 0, stream>>>(Bk);
        else append_block_token_kernel<float, false><<<grid, 32, 0, stream>>>(Bk);
    }
    append_block_advance_kernel<<<(p.batch + 127) / 128, 128, 0, stream>>>(Bk);
    *launches += 3;
    return cudaGetLastError() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------
// Two partial attention results over disjoint token sets -> the result over their union (the log-sum-exp
// merge that split decoding uses, exposed for callers that hold a sequence in more than one cache).
// One warp per (sequence, query head) row; lane l owns channels 4l .. 4l+3.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) merge_attn_kernel(int rows, const float* __restrict__ out_a, const float* __restrict__ lse_a,
                                                         const float* __restrict__ out_b, const float* __restrict__ lse_b,
                                                         float* __restrict__ out, float* __restrict__ lse)
{
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= rows) return;
    const float la = lse_a[row], lb = lse_b[row];
    const float m = fmaxf(la, lb);
    float wa = 0.f, wb = 0.f, l = -INFINITY;
    if (m > -INFINITY) {                                       // at least one side saw tokens
        const float ea = expf(la - m), eb = expf(lb - m);
        const float inv = 1.0f / (ea + eb);
        wa = ea * inv; wb = eb * inv;
        l = m + logf(ea + eb);
    }
    const float4 a = reinterpret_cast<const float4*>(out_a + static_cast<int64_t>(row) * kHeadDim)[lane];
    const float4 b = reinterpret_cast<const float4*>(out_b + static_cast<int64_t>(row) * kHeadDim)[lane];
    reinterpret_cast<float4*>(out + static_cast<int64_t>(row) * kHeadDim)[lane] =
        make_float4(fmaf(wa, a.x, wb * b.x), fmaf(wa, a.y, wb * b.y), fmaf(wa, a.z, wb * b.z), fmaf(wa, a.w, wb * b.w));
    if (lane == 0 && lse) lse[row] = l;
}

spark_status launch_merge_attn(int rows, const float* out_a, const float* lse_a, const float* out_b, const float* lse_b,
                               float* out, float* lse, cudaStream_t stream)
{
    if (rows == 0) return SPARK_OK;
    merge_attn_kernel<<<(rows + 3) / 4, 128, 0, stream>>>(rows, out_a, lse_a, out_b, lse_b, out, lse);
    return cudaGetLastError() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------
// pages -> logical arrays
// ------------------------------------------------------------------------------------------------
struct UnpackArgs {
    const unsigned char* pages;
    const int32_t* block_table;
    int max_blocks;
    const int32_t* lens;
    int max_tokens;
    int Hkv;
    int64_t n_pool_pages;
    PageLayout L;
    uint32_t* mask;
    float* mu;
    void* vals;
    void* v;
    uint32_t* vmask;
    float* mu_all;
    float* sigma_all;
};

__global__ void __launch_bounds__(128) unpack_pages_kernel(UnpackArgs A)
{
    const int blk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const PageLayout L = A.L;
    const int T = L.keep;
    int len = A.lens[b];
    len = len < 0 ? 0 : (len > A.max_tokens ? A.max_tokens : len);
    const int64_t unit = static_cast<int64_t>(b) * A.Hkv + h;
    const unsigned char* page = nullptr;
    if (blk * kPageTokens < len) {
        const int64_t id = A.block_table ? A.block_table[unit * A.max_blocks + blk] : unit * A.max_blocks + blk;
        if (id >= 0 && id < A.n_pool_pages) page = A.pages + id * L.page_bytes;
    }
    const int t0 = blk * kPageTokens;
    const int64_t row0 = unit * A.max_tokens + t0;
    if (A.mask)
        for (int i = threadIdx.x; i < kPageTokens * kMaskWords; i += blockDim.x) {
            const int p = i / kMaskWords;
            if (t0 + p >= A.max_tokens) continue;
            A.mask[(row0 + p) * kMaskWords + (i % kMaskWords)] =
                (page && t0 + p < len) ? reinterpret_cast<const unsigned*>(page + L.mask_off)[i] : 0u;
        }
    if (A.mu)
        for (int p = threadIdx.x; p < kPageTokens; p += blockDim.x) {
            if (t0 + p >= A.max_tokens) continue;
            A.mu[row0 + p] = (page && t0 + p < len) ? reinterpret_cast<const float*>(page + L.mu_off)[p] : 0.f;
        }
    if (A.mu_all || A.sigma_all)                                  // only called for layouts that carry the section
        for (int p = threadIdx.x; p < kPageTokens; p += blockDim.x) {
            if (t0 + p >= A.max_tokens) continue;
            const bool live = page && t0 + p < len;
            const float* st = reinterpret_cast<const float*>(page + L.stats_off);
            if (A.mu_all) A.mu_all[row0 + p] = live ? st[p] : 0.f;
            if (A.sigma_all) A.sigma_all[row0 + p] = live ? st[kPageTokens + p] : 0.f;
        }
    if (A.vals)
        for (int i = threadIdx.x; i < kPageTokens * T; i += blockDim.x) {
            const int p = i / T, s = i % T;
            if (t0 + p >= A.max_tokens) continue;
            const bool live = page && t0 + p < len;
            const int64_t o = (row0 + p) * T + s;
            if (L.esize == 2)
                static_cast<unsigned short*>(A.vals)[o] =
                    live ? *reinterpret_cast<const unsigned short*>(page + L.vals_off + val_offset(2, p, s)) : 0;
            else
                static_cast<unsigned*>(A.vals)[o] =
                    live ? *reinterpret_cast<const unsigned*>(page + L.vals_off + val_offset(4, p, s)) : 0u;
        }
    if (A.vmask)                                                  // all ones for dense value rows
        for (int i = threadIdx.x; i < kPageTokens * kMaskWords; i += blockDim.x) {
            const int p = i / kMaskWords;
            if (t0 + p >= A.max_tokens) continue;
            const bool live = page && t0 + p < len;
            A.vmask[(row0 + p) * kMaskWords + (i % kMaskWords)] =
                !live ? 0u : (L.keep_v < kHeadDim ? reinterpret_cast<const unsigned*>(page + L.vmask_off)[i] : 0xffffffffu);
        }
    if (A.v)                                                      // pruned value entries read back as zero
        for (int i = threadIdx.x; i < kPageTokens * kHeadDim; i += blockDim.x) {
            const int p = i / kHeadDim, j = i % kHeadDim;
            if (t0 + p >= A.max_tokens) continue;
            const bool live = page && t0 + p < len;
            const int64_t o = (row0 + p) * kHeadDim + j;
            const unsigned char* src = nullptr;
            if (live && L.keep_v < kHeadDim) {
                const unsigned* vm = reinterpret_cast<const unsigned*>(page + L.vmask_off) + p * kMaskWords;
                if ((vm[j >> 5] >> (j & 31)) & 1u) {
                    int slot = __popc(vm[j >> 5] & ((1u << (j & 31)) - 1u));
                    for (int w = 0; w < (j >> 5); ++w) slot += __popc(vm[w]);
                    src = page + L.v_off + val_offset(L.esize, p, slot);
                }
            } else if (live) {
                src = L.esize == 2 ? page + L.v_off + v_chunk_offset(2, p, j >> 3) + (j & 7) * 2
                                   : page + L.v_off + v_chunk_offset(4, p, j >> 2) + (j & 3) * 4;
            }
            if (L.esize == 2) static_cast<unsigned short*>(A.v)[o] = src ? *reinterpret_cast<const unsigned short*>(src) : 0;
            else static_cast<unsigned*>(A.v)[o] = src ? *reinterpret_cast<const unsigned*>(src) : 0u;
        }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
size_t compress_workspace_bytes(const spark_params& p, int64_t max_seq_tokens)
{
    return kWorkspaceHeader + evict_workspace_bytes(p, max_seq_tokens);
}

spark_status launch_compress(const spark_params& p, const void* q_win, const void* k, const void* v,
                             int64_t sb, int64_t sh, int64_t st, const int32_t* seq_lens,
                             int32_t max_seq_tokens, void* pages, const int32_t* block_table,
                             int32_t max_blocks, float* qnorm, int32_t* packed_lens, int32_t* kept_tokens,
                             void* workspace, size_t workspace_bytes, cudaStream_t stream, int* launches)
{
    (void)workspace_bytes;
    int* status = static_cast<int*>(workspace);
    const bool evict = p.token_budget > 0;
    if (evict) {            // writes kept_tokens and packed_lens
        const spark_status st_e = launch_evict(p, q_win, k, sb, sh, st, seq_lens, max_seq_tokens, packed_lens,
                                               kept_tokens, workspace, stream, launches);
        if (st_e != SPARK_OK) return st_e;
    }
    const float eps = p.qnorm_eps > 0.f ? p.qnorm_eps : 1e-12f;
    const dim3 qgrid(p.n_kv_heads, p.batch);
    if (p.dtype == SPARK_BF16)
        window_qnorm_kernel<__nv_bfloat16><<<qgrid, kHeadDim, 0, stream>>>(
            q_win, p.n_q_heads, p.n_kv_heads, p.window, eps, qnorm, seq_lens, evict ? nullptr : packed_lens, max_seq_tokens, status);
    else
        window_qnorm_kernel<float><<<qgrid, kHeadDim, 0, stream>>>(
            q_win, p.n_q_heads, p.n_kv_heads, p.window, eps, qnorm, seq_lens, evict ? nullptr : packed_lens, max_seq_tokens, status);
    ++*launches;
    if (cudaGetLastError() != cudaSuccess) return SPARK_ERR_CUDA;

    const int max_packed = (evict && p.token_budget < max_seq_tokens) ? p.token_budget : max_seq_tokens;
    const int n_blocks = (max_packed + kPageTokens - 1) / kPageTokens;
    if (n_blocks == 0) return SPARK_OK;
    CompressArgs A;
    A.k = k; A.v = v; A.sb = sb; A.sh = sh; A.st = st;
    A.lens = packed_lens; A.gather = evict ? kept_tokens : nullptr; A.gather_stride = evict ? p.token_budget : 0;
    A.qnorm = qnorm; A.pages = static_cast<unsigned char*>(pages);
    A.block_table = block_table; A.max_blocks = max_blocks; A.Hkv = p.n_kv_heads; A.keep = p.keep;
    A.n_pool_pages = p.n_pool_pages; A.L = make_layout(p); A.status = status;
    A.inv_pruned = p.keep < kHeadDim ? 1.0 / static_cast<double>(kHeadDim - p.keep) : 0.0;
    A.sel = make_select(p);
    const dim3 grid(n_blocks, p.n_kv_heads, p.batch);
    const bool rank = p.select != SPARK_SELECT_FIXED;      // a ratio-free rule: the kernels with the rank sort
    if (p.dtype == SPARK_BF16) {
        if (rank) compress_pages_kernel<__nv_bfloat16, true><<<grid, 256, A.L.page_bytes, stream>>>(A);
        else compress_pages4_kernel<__nv_bfloat16><<<grid, 128, A.L.page_bytes, stream>>>(A);
    } else {
        if (rank) compress_pages_kernel<float, true><<<grid, 256, A.L.page_bytes, stream>>>(A);
        else compress_pages4_kernel<float><<<grid, 128, A.L.page_bytes, stream>>>(A);
    }
    ++*launches;
    if (cudaGetLastError() != cudaSuccess) return SPARK_ERR_CUDA;
    return SPARK_OK;
}

spark_status launch_unpack(const spark_params& p, const void* pages, const int32_t* block_table,
                           int32_t max_blocks, const int32_t* packed_lens, int32_t max_tokens,
                           uint32_t* mask, float* mu, void* vals, void* v, uint32_t* vmask, float* mu_all,
                           float* sigma_all, cudaStream_t stream)
{
    const int n_blocks = (max_tokens + kPageTokens - 1) / kPageTokens;
    if (n_blocks == 0) return SPARK_OK;
    UnpackArgs A;
    A.pages = static_cast<const unsigned char*>(pages); A.block_table = block_table;
    A.max_blocks = max_blocks; A.lens = packed_lens; A.max_tokens = max_tokens; A.Hkv = p.n_kv_heads;
    A.n_pool_pages = p.n_pool_pages; A.L = make_layout(p);
    A.mask = mask; A.mu = mu; A.vals = vals; A.v = v; A.vmask = vmask; A.mu_all = mu_all; A.sigma_all = sigma_all;
    unpack_pages_kernel<<<dim3(n_blocks, p.n_kv_heads, p.batch), 128, 0, stream>>>(A);
    if (cudaGetLastError() != cudaSuccess) return SPARK_ERR_CUDA;
    return SPARK_OK;
}

}  // namespace spark
