// Token eviction pre-step of spark_compress (token_budget > 0).
//
// The paper applies channel pruning on top of a token-eviction method and only cites that method's
// settings (App. "Implementation": observation window 32, max-pool kernel 7).  The rule implemented here
// is the benchmark's: for every KV head, the window queries of its G query heads attend (causally inside
// the window) to all earlier keys; the softmax probabilities of the prefix tokens are summed over the
// G*W query rows ("votes"), max-pooled over `pool` neighbours, and the (budget - W) prefix tokens with
// the largest pooled vote (ties: lower position) are kept together with the W window tokens, in
// original order.  Sequences no longer than the budget are kept whole.
//
// Kernels (fp32 CUDA-core arithmetic; this step is preparation, not the timed decode step):
//   evict_scores_kernel<pass 1>  per 128-token tile and query row: max and sum of exp of the scores
//   evict_rowstats_kernel        merge the tile partials into the row's softmax normaliser
//   evict_scores_kernel<pass 2>  recompute the tile's scores, accumulate the column sums = votes
//   evict_pool_kernel            pooled max of the votes, as order-preserving integer keys
//   evict_hist_kernel<0..3>      radix select of the k-th largest key, one byte per pass, all SMs
//   evict_count / compact        ordered compaction of the kept positions into kept_tokens
// Column sums are accumulated inside one CTA in a fixed order, so the votes are reproducible.
#include "spark_common.cuh"

namespace spark {

constexpr int kEvTile = 128;          // tokens per CTA tile
constexpr int kEvRows = 64;           // query rows per pass over the tile
constexpr int kEvThreads = 256;
constexpr int kEvStride = kHeadDim + 1;   // padded row length in shared memory (floats)

struct EvictArgs {
    const void* q_win;
    const void* k;
    int64_t sb, sh, st;
    const int32_t* seq_lens;
    int Hq, Hkv, W, budget, pool;
    int S_max, n_tiles;
    float* partial;      // [units][R][n_tiles][2]
    float* rowstat;      // [units][R][2]
    float* votes;        // [units][S_max]
    unsigned* pooled;    // [units][S_max] pooled votes as order-preserving keys
    int* hist;           // [units][4][256] radix-select histograms, one per pass
    int* counts;         // [units][n_chunks][2] keys above / equal to the threshold per 4096-token chunk
    int n_chunks;
    int32_t* kept;       // [units][budget]
    int32_t* packed_lens;
    int* status;
};

template <typename E, int PASS>
__global__ void __launch_bounds__(kEvThreads) evict_scores_kernel(EvictArgs A)
{
    extern __shared__ __align__(16) float ev_smem[];
    float* Ks = ev_smem;                                   // [128][129]
    float* Qs = Ks + kEvTile * kEvStride;                  // [64][129]
    float* colsum = Qs + kEvRows * kEvStride;              // [128]
    const int tile = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int S = min(A.seq_lens[b], A.S_max);
    if (S <= A.budget) return;                             // kept whole
    const int t0 = tile * kEvTile;
    if (t0 >= S) return;
    const int G = A.Hq / A.Hkv, R = G * A.W, P = S - A.W;
    const int unit = b * A.Hkv + h;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const float scale = rsqrtf(static_cast<float>(kHeadDim));

    for (int i = tid; i < kEvTile * kHeadDim; i += kEvThreads) {
        const int tt = i / kHeadDim, j = i - tt * kHeadDim;
        const int t = t0 + tt;
        Ks[tt * kEvStride + j] = (t < S)
            ? Elem<E>::load(A.k, static_cast<int64_t>(b) * A.sb + static_cast<int64_t>(h) * A.sh +
                                     static_cast<int64_t>(t) * A.st + j)
            : 0.f;
    }
    if (PASS == 2 && tid < kEvTile) colsum[tid] = 0.f;

    for (int r0 = 0; r0 < R; r0 += kEvRows) {
        __syncthreads();
        for (int i = tid; i < kEvRows * kHeadDim; i += kEvThreads) {
            const int rr = i / kHeadDim, j = i - rr * kHeadDim;
            const int row = r0 + rr;
            float v = 0.f;
            if (row < R) {
                const int g = row / A.W, w = row - g * A.W;
                v = Elem<E>::load(A.q_win, ((static_cast<int64_t>(b) * A.Hq + h * G + g) * A.W + w) * kHeadDim + j);
            }
            Qs[rr * kEvStride + j] = v;
        }
        __syncthreads();
        float acc[4][8];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
        for (int kk = 0; kk < kHeadDim; ++kk) {
            float a[4], bb[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = Qs[(ty * 4 + i) * kEvStride + kk];
#pragma unroll
            for (int j = 0; j < 8; ++j) bb[j] = Ks[(tx + 16 * j) * kEvStride + kk];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
        }
        // thread (ty, tx): rows r0 + 4 ty + i, tokens t0 + tx + 16 j
        float cs[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) cs[j] = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = r0 + ty * 4 + i;
            const bool row_ok = row < R;
            const int w = row_ok ? (row % A.W) : 0;
            const int last = P + w;                        // causal: this query sees tokens <= last
            if (PASS == 1) {
                float m = -INFINITY;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int t = t0 + tx + 16 * j;
                    acc[i][j] = (row_ok && t <= last && t < S) ? acc[i][j] * scale : -INFINITY;
                    m = fmaxf(m, acc[i][j]);
                }
#pragma unroll
                for (int o = 1; o < 16; o <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                float l = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) l += (acc[i][j] == -INFINITY) ? 0.f : expf(acc[i][j] - m);
#pragma unroll
                for (int o = 1; o < 16; o <<= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
                if (row_ok && tx == 0) {
                    float* dst = A.partial + ((static_cast<int64_t>(unit) * R + row) * A.n_tiles + tile) * 2;
                    dst[0] = m;
                    dst[1] = l;
                }
            } else {
                float M = 0.f, invL = 0.f;
                if (row_ok) {
                    const float* rs = A.rowstat + (static_cast<int64_t>(unit) * R + row) * 2;
                    M = rs[0];
                    invL = 1.0f / rs[1];
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int t = t0 + tx + 16 * j;
                    if (row_ok && t < P) cs[j] += expf(acc[i][j] * scale - M) * invL;
                }
            }
        }
        if (PASS == 2) {
            // fixed-order accumulation of the column sums: row groups take turns
            for (int turn = 0; turn < 16; ++turn) {
                if (ty == turn)
#pragma unroll
                    for (int j = 0; j < 8; ++j) colsum[tx + 16 * j] += cs[j];
                __syncthreads();
            }
        }
    }
    if (PASS == 2) {
        __syncthreads();
        if (tid < kEvTile && t0 + tid < S)
            A.votes[static_cast<int64_t>(unit) * A.S_max + t0 + tid] = colsum[tid];
    }
}

__global__ void evict_rowstats_kernel(EvictArgs A)
{
    const int h = blockIdx.x, b = blockIdx.y;
    const int S = min(A.seq_lens[b], A.S_max);
    if (S <= A.budget) return;
    const int G = A.Hq / A.Hkv, R = G * A.W;
    const int unit = b * A.Hkv + h;
    const int tiles = (S + kEvTile - 1) / kEvTile;
    for (int row = threadIdx.x; row < R; row += blockDim.x) {
        const float* src = A.partial + (static_cast<int64_t>(unit) * R + row) * A.n_tiles * 2;
        float M = -INFINITY, L = 0.f;
        for (int t = 0; t < tiles; ++t) {
            const float m = src[2 * t], l = src[2 * t + 1];
            if (m == -INFINITY) continue;
            const float Mn = fmaxf(M, m);
            L = L * expf(M - Mn) + l * expf(m - Mn);
            M = Mn;
        }
        A.rowstat[(static_cast<int64_t>(unit) * R + row) * 2] = M;
        A.rowstat[(static_cast<int64_t>(unit) * R + row) * 2 + 1] = L;
    }
}

// pooled[t] = max of the votes within (pool-1)/2 positions of t (clamped to the prefix), stored as the
// float's bit pattern: votes are >= 0, so unsigned comparison of the patterns is the order of the values.
__global__ void __launch_bounds__(256) evict_pool_kernel(EvictArgs A)
{
    const int h = blockIdx.y, b = blockIdx.z;
    const int S = min(A.seq_lens[b], A.S_max);
    if (S <= A.budget) return;
    const int P = S - A.W, half = (A.pool - 1) / 2;
    if (blockIdx.x == 0)                                   // fresh histograms for this call's radix select
        for (int i = threadIdx.x; i < 1024; i += blockDim.x) A.hist[static_cast<int64_t>(b * A.Hkv + h) * 1024 + i] = 0;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= P) return;
    const int64_t base = static_cast<int64_t>(b * A.Hkv + h) * A.S_max;
    float m = A.votes[base + t];
    for (int u = t - half; u <= t + half; ++u)
        if (u >= 0 && u < P) m = fmaxf(m, A.votes[base + u]);
    A.pooled[base + t] = __float_as_uint(m);
}

// ------------------------------------------------------------------------------------------------
// Exact top-k of the pooled votes and ordered compaction, spread over the whole GPU.
//
// The k-th largest key of a unit is found by a radix select, 8 bits per pass: every CTA histograms its
// 4096-token chunk into shared memory and adds the non-empty bins to the unit's histogram of that pass
// (integer atomics: the result does not depend on arrival order).  The choice made by each finished pass
// (the byte of the threshold, the rank left inside that bin) is recomputed from the stored histograms by
// whoever needs it, so there is no separate "pick" launch.  After four passes the threshold key and the
// number of equal keys to admit (lowest positions first) are known; a counting kernel gives every chunk
// its base position and the compaction kernel writes the kept positions in order.
// ------------------------------------------------------------------------------------------------
constexpr int kSelChunk = 4096;
constexpr int kSelThreads = 256;
constexpr int kSelPerThread = kSelChunk / kSelThreads;

struct SelState { unsigned prefix, mask; int need; };

// Replays the first `passes` picks from the unit's histograms ([4][256]).  One full warp.
__device__ __forceinline__ SelState select_state(const int* hist, int passes, int k, int lane)
{
    SelState s;
    s.prefix = 0u; s.mask = 0u; s.need = k;
    for (int p = 0; p < passes; ++p) {
        const int* hp = hist + p * 256;
        const int shift = 24 - 8 * p;
        int loc[8], sum = 0;                              // lane l: bins 255 - 8l, 254 - 8l, ... (descending)
#pragma unroll
        for (int i = 0; i < 8; ++i) { loc[i] = hp[255 - 8 * lane - i]; sum += loc[i]; }
        int inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int n = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += n; }
        const unsigned cross = __ballot_sync(0xffffffffu, inc >= s.need);
        const int src = cross ? __ffs(cross) - 1 : 31;   // lane whose bins contain the need-th largest key
        int bin = 0, left = 0;
        if (lane == src) {
            int need = s.need - (inc - sum), i = 0;
            for (; i < 7; ++i) { if (loc[i] >= need) break; need -= loc[i]; }
            bin = 255 - 8 * lane - i;
            left = need;
        }
        bin = __shfl_sync(0xffffffffu, bin, src);
        left = __shfl_sync(0xffffffffu, left, src);
        s.need = left;                                    // rank inside the chosen bin
        s.prefix |= static_cast<unsigned>(bin) << shift;
        s.mask |= 255u << shift;
    }
    return s;
}

template <int PASS>
__global__ void __launch_bounds__(kSelThreads) evict_hist_kernel(EvictArgs A)
{
    __shared__ int sh[256];
    __shared__ SelState st;
    const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int S = min(A.seq_lens[b], A.S_max);
    if (S <= A.budget) return;
    const int P = S - A.W, k = A.budget - A.W, t0 = chunk * kSelChunk;
    if (t0 >= P) return;
    const int unit = b * A.Hkv + h, tid = threadIdx.x, lane = tid & 31;
    int* hist = A.hist + static_cast<int64_t>(unit) * 1024;
    sh[tid] = 0;
    if (tid < 32) {
        const SelState s = select_state(hist, PASS, k, lane);
        if (lane == 0) st = s;
    }
    __syncthreads();
    const unsigned prefix = st.prefix, mask = st.mask;
    constexpr int shift = 24 - 8 * PASS;
    const unsigned* pooled = A.pooled + static_cast<int64_t>(unit) * A.S_max;
#pragma unroll 4
    for (int i = 0; i < kSelPerThread; ++i) {              // whole warps iterate together (votes below)
        const int t = t0 + i * kSelThreads + tid;
        const unsigned key = t < P ? pooled[t] : 0u;
        const bool in = t < P && (key & mask) == prefix;
        const unsigned bin = (key >> shift) & 255u;
        // lanes that hit the same bin add once: keys of neighbouring tokens mostly share their top bytes
        const unsigned active = __ballot_sync(0xffffffffu, in);
        if (in) {
            const unsigned peers = __match_any_sync(active, bin);
            if (lane == __ffs(peers) - 1) atomicAdd(&sh[bin], __popc(peers));
        }
    }
    __syncthreads();
    if (sh[tid]) atomicAdd(&hist[PASS * 256 + tid], sh[tid]);
}

// counts[unit][chunk] = (keys above the threshold, keys equal to it) in the chunk
__global__ void __launch_bounds__(kSelThreads) evict_count_kernel(EvictArgs A)
{
    __shared__ SelState st;
    __shared__ int red[2][kSelThreads / 32];
    const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int S = min(A.seq_lens[b], A.S_max);
    if (S <= A.budget) return;
    const int P = S - A.W, k = A.budget - A.W, t0 = chunk * kSelChunk;
    if (t0 >= P) return;
    const int unit = b * A.Hkv + h, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid < 32) {
        const SelState s = select_state(A.hist + static_cast<int64_t>(unit) * 1024, 4, k, lane);
        if (lane == 0) st = s;
    }
    __syncthreads();
    const unsigned thr = st.prefix;
    const unsigned* pooled = A.pooled + static_cast<int64_t>(unit) * A.S_max;
    int gt = 0, eq = 0;
#pragma unroll 4
    for (int i = 0; i < kSelPerThread; ++i) {
        const int t = t0 + i * kSelThreads + tid;
        if (t < P) { const unsigned key = pooled[t]; gt += key > thr; eq += key == thr; }
    }
    gt = __reduce_add_sync(0xffffffffu, gt);
    eq = __reduce_add_sync(0xffffffffu, eq);
    if (lane == 0) { red[0][warp] = gt; red[1][warp] = eq; }
    __syncthreads();
    if (tid == 0) {
        int g = 0, e = 0;
        for (int w = 0; w < kSelThreads / 32; ++w) { g += red[0][w]; e += red[1][w]; }
        int* c = A.counts + (static_cast<int64_t>(unit) * A.n_chunks + chunk) * 2;
        c[0] = g; c[1] = e;
    }
}

// Ordered compaction: thread i of the chunk's CTA owns 16 consecutive tokens.  Also publishes packed_lens
// and handles sequences that are kept whole.
__global__ void __launch_bounds__(kSelThreads) evict_compact_kernel(EvictArgs A)
{
    __shared__ SelState st;
    __shared__ int s_base_kept, s_base_eq;
    __shared__ int scan_eq[kSelThreads / 32], scan_keep[kSelThreads / 32];
    const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int S = A.seq_lens[b];
    if (S < 0 || S > A.S_max) {
        if (chunk == 0 && tid == 0) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
        S = S < 0 ? 0 : A.S_max;
    }
    const int unit = b * A.Hkv + h;
    int32_t* kept = A.kept + static_cast<int64_t>(unit) * A.budget;
    if (chunk == 0 && h == 0 && tid == 0) A.packed_lens[b] = S < A.budget ? S : A.budget;
    if (S <= A.budget) {                                  // kept whole
        for (int t = chunk * kSelChunk + tid; t < min(A.budget, (chunk + 1) * kSelChunk); t += kSelThreads)
            kept[t] = t < S ? t : -1;
        if (chunk == 0)                                   // budget beyond the chunked range (short max_seq_tokens)
            for (int t = A.n_chunks * kSelChunk + tid; t < A.budget; t += kSelThreads) kept[t] = t < S ? t : -1;
        return;
    }
    const int P = S - A.W, k = A.budget - A.W, t0 = chunk * kSelChunk;
    if (chunk == 0)
        for (int w = tid; w < A.W; w += kSelThreads) kept[k + w] = P + w;
    if (t0 >= P) return;
    if (tid < 32) {
        const SelState s = select_state(A.hist + static_cast<int64_t>(unit) * 1024, 4, k, lane);
        if (lane == 0) {
            st = s;
            // position of this chunk's first kept token and number of equal keys before the chunk
            const int* c = A.counts + static_cast<int64_t>(unit) * A.n_chunks * 2;
            int base_kept = 0, base_eq = 0;
            for (int cc = 0; cc < chunk; ++cc) {
                const int take = min(c[2 * cc + 1], max(0, s.need - base_eq));
                base_kept += c[2 * cc] + take;
                base_eq += c[2 * cc + 1];
            }
            s_base_kept = base_kept; s_base_eq = base_eq;
        }
    }
    __syncthreads();
    const unsigned thr = st.prefix;
    const int need_eq = st.need;
    const unsigned* pooled = A.pooled + static_cast<int64_t>(unit) * A.S_max;
    const int tb = t0 + tid * kSelPerThread;
    unsigned key[kSelPerThread];
    int eq_cnt = 0;
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i) {
        key[i] = (tb + i < P) ? pooled[tb + i] : 0u;
        eq_cnt += (tb + i < P && key[i] == thr) ? 1 : 0;
    }
    // exclusive scan of eq_cnt over the CTA's threads (threads are in position order)
    int v = eq_cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int n = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += n; }
    if (lane == 31) scan_eq[warp] = v;
    __syncthreads();
    int eq_rank = s_base_eq + v - eq_cnt;
    for (int w = 0; w < warp; ++w) eq_rank += scan_eq[w];
    unsigned keep_bits = 0u;
    int keep_cnt = 0;
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i) {
        const bool live = tb + i < P;
        const bool eq = live && key[i] == thr;
        const bool keep = live && (key[i] > thr || (eq && eq_rank < need_eq));
        eq_rank += eq ? 1 : 0;
        keep_bits |= keep ? (1u << i) : 0u;
        keep_cnt += keep ? 1 : 0;
    }
    int u = keep_cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int n = __shfl_up_sync(0xffffffffu, u, o); if (lane >= o) u += n; }
    if (lane == 31) scan_keep[warp] = u;
    __syncthreads();
    int pos = s_base_kept + u - keep_cnt;
    for (int w = 0; w < warp; ++w) pos += scan_keep[w];
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i)
        if ((keep_bits >> i) & 1u) {
            if (pos < k) kept[pos] = tb + i;
            ++pos;
        }
    // the thread that owns the last prefix token sees the total
    if (tb <= P - 1 && P - 1 < tb + kSelPerThread && pos != k) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
}

bool evict_tc_supported(const spark_params& p);
spark_status launch_evict_votes_tc(const spark_params& p, const void* q_win, const void* k, int64_t sb, int64_t sh,
                                   int64_t st, const int32_t* seq_lens, int32_t max_seq_tokens, float* partial,
                                   float* rowstat, float* votes, int* status, cudaStream_t stream, int* launches);

size_t evict_workspace_bytes(const spark_params& p, int64_t max_seq_tokens)
{
    if (p.token_budget <= 0) return 0;
    const size_t units = static_cast<size_t>(p.batch) * p.n_kv_heads;
    const size_t R = static_cast<size_t>(p.n_q_heads / p.n_kv_heads) * p.window;
    const size_t tiles = (max_seq_tokens + kEvTile - 1) / kEvTile;
    size_t bytes = units * R * tiles * 2 * sizeof(float);
    bytes += units * R * 2 * sizeof(float);
    bytes += 2 * units * static_cast<size_t>(max_seq_tokens) * sizeof(float);      // votes, pooled keys
    const size_t chunks = (max_seq_tokens + kSelChunk - 1) / kSelChunk;
    bytes += units * (1024 + 2 * (chunks ? chunks : 1)) * sizeof(int);             // select histograms, chunk counts
    return (bytes + 255) / 256 * 256;
}

spark_status launch_evict(const spark_params& p, const void* q_win, const void* k, int64_t sb, int64_t sh,
                          int64_t st, const int32_t* seq_lens, int32_t max_seq_tokens, int32_t* packed_lens,
                          int32_t* kept_tokens, void* workspace, cudaStream_t stream, int* launches)
{
    const size_t units = static_cast<size_t>(p.batch) * p.n_kv_heads;
    const size_t R = static_cast<size_t>(p.n_q_heads / p.n_kv_heads) * p.window;
    EvictArgs A;
    A.q_win = q_win; A.k = k; A.sb = sb; A.sh = sh; A.st = st; A.seq_lens = seq_lens;
    A.Hq = p.n_q_heads; A.Hkv = p.n_kv_heads; A.W = p.window; A.budget = p.token_budget; A.pool = p.pool_kernel;
    A.S_max = max_seq_tokens; A.n_tiles = (max_seq_tokens + kEvTile - 1) / kEvTile;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    A.status = reinterpret_cast<int*>(ws);
    A.partial = reinterpret_cast<float*>(ws + kWorkspaceHeader);
    A.rowstat = A.partial + units * R * A.n_tiles * 2;
    A.votes = A.rowstat + units * R * 2;
    A.pooled = reinterpret_cast<unsigned*>(A.votes + units * static_cast<size_t>(max_seq_tokens));
    A.hist = reinterpret_cast<int*>(A.pooled + units * static_cast<size_t>(max_seq_tokens));
    A.counts = A.hist + units * 1024;
    A.n_chunks = (max_seq_tokens + kSelChunk - 1) / kSelChunk;
    if (A.n_chunks < 1) A.n_chunks = 1;
    A.kept = kept_tokens; A.packed_lens = packed_lens;
    const size_t smem = (static_cast<size_t>(kEvTile + kEvRows) * kEvStride + kEvTile) * sizeof(float);
    const dim3 grid(A.n_tiles, p.n_kv_heads, p.batch), ugrid(p.n_kv_heads, p.batch);
    const bool bf16 = p.dtype == SPARK_BF16;
    if (A.n_tiles > 0 && max_seq_tokens > p.token_budget && evict_tc_supported(p)) {
        const spark_status st_tc = launch_evict_votes_tc(p, q_win, k, sb, sh, st, seq_lens, max_seq_tokens, A.partial,
                                                         A.rowstat, A.votes, A.status, stream, launches);
        if (st_tc != SPARK_OK) return st_tc;
    } else if (A.n_tiles > 0 && max_seq_tokens > p.token_budget) {
        cudaError_t e1 = bf16 ? cudaFuncSetAttribute(evict_scores_kernel<__nv_bfloat16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem))
                              : cudaFuncSetAttribute(evict_scores_kernel<float, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        cudaError_t e2 = bf16 ? cudaFuncSetAttribute(evict_scores_kernel<__nv_bfloat16, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem))
                              : cudaFuncSetAttribute(evict_scores_kernel<float, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e1 != cudaSuccess || e2 != cudaSuccess) return SPARK_ERR_CUDA;
        if (bf16) evict_scores_kernel<__nv_bfloat16, 1><<<grid, kEvThreads, smem, stream>>>(A);
        else evict_scores_kernel<float, 1><<<grid, kEvThreads, smem, stream>>>(A);
        evict_rowstats_kernel<<<ugrid, 256, 0, stream>>>(A);
        if (bf16) evict_scores_kernel<__nv_bfloat16, 2><<<grid, kEvThreads, smem, stream>>>(A);
        else evict_scores_kernel<float, 2><<<grid, kEvThreads, smem, stream>>>(A);
        *launches += 3;
    }
    const dim3 sgrid(A.n_chunks, p.n_kv_heads, p.batch);
    if (max_seq_tokens > p.token_budget) {
        evict_pool_kernel<<<dim3((max_seq_tokens + 255) / 256, p.n_kv_heads, p.batch), 256, 0, stream>>>(A);
        evict_hist_kernel<0><<<sgrid, kSelThreads, 0, stream>>>(A);
        evict_hist_kernel<1><<<sgrid, kSelThreads, 0, stream>>>(A);
        evict_hist_kernel<2><<<sgrid, kSelThreads, 0, stream>>>(A);
        evict_hist_kernel<3><<<sgrid, kSelThreads, 0, stream>>>(A);
        evict_count_kernel<<<sgrid, kSelThreads, 0, stream>>>(A);
        *launches += 6;
    }
    evict_compact_kernel<<<sgrid, kSelThreads, 0, stream>>>(A);
    ++*launches;
    return cudaGetLastError() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

}  // namespace spark
