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
//   evict_select_kernel          pooled max, exact top-k by radix select on the float bit pattern,
//                                ordered compaction into kept_tokens
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
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= P) return;
    const int64_t base = static_cast<int64_t>(b * A.Hkv + h) * A.S_max;
    float m = A.votes[base + t];
    for (int u = t - half; u <= t + half; ++u)
        if (u >= 0 && u < P) m = fmaxf(m, A.votes[base + u]);
    A.pooled[base + t] = __float_as_uint(m);
}

// One CTA per unit: exact top-k of the pooled votes, ordered compaction.
__global__ void __launch_bounds__(1024) evict_select_kernel(EvictArgs A)
{
    __shared__ int hist[256];
    __shared__ int scan[32];
    __shared__ unsigned s_prefix, s_mask;
    __shared__ int s_need, s_base_kept, s_base_eq;
    const int h = blockIdx.x, b = blockIdx.y;
    int S = A.seq_lens[b];
    if (S < 0 || S > A.S_max) {
        if (threadIdx.x == 0) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
        S = S < 0 ? 0 : A.S_max;
    }
    const int unit = b * A.Hkv + h;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t* kept = A.kept + static_cast<int64_t>(unit) * A.budget;
    if (h == 0 && tid == 0) A.packed_lens[b] = S < A.budget ? (S < 0 ? 0 : S) : A.budget;
    if (S <= A.budget) {
        for (int t = tid; t < A.budget; t += blockDim.x) kept[t] = t < S ? t : -1;
        return;
    }
    const int P = S - A.W, k = A.budget - A.W;
    const unsigned* pooled = A.pooled + static_cast<int64_t>(unit) * A.S_max;
    auto pooled_key = [&](int t) -> unsigned { return pooled[t]; };
    // radix select of the k-th largest key, 8 bits per pass
    if (tid == 0) { s_prefix = 0; s_mask = 0; s_need = k; }
    __syncthreads();
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        const unsigned prefix = s_prefix, mask = s_mask;
        for (int t0 = 0; t0 < P; t0 += blockDim.x) {        // all lanes iterate together (warp votes below)
            const int t = t0 + tid;
            const unsigned key = t < P ? pooled_key(t) : 0u;
            const bool in = t < P && (key & mask) == prefix;
            const unsigned bin = (key >> shift) & 255u;
            // lanes that hit the same bin add once: keys of neighbouring tokens mostly share their top bytes
            const unsigned active = __ballot_sync(0xffffffffu, in);
            if (in) {
                const unsigned peers = __match_any_sync(active, bin);
                if (lane == __ffs(peers) - 1) atomicAdd(&hist[bin], __popc(peers));
            }
        }
        __syncthreads();
        if (tid == 0) {
            int need = s_need, bin = 255;
            for (; bin > 0; --bin) {
                if (hist[bin] >= need) break;
                need -= hist[bin];
            }
            s_need = need;                                  // rank inside the chosen bin
            s_prefix = prefix | (static_cast<unsigned>(bin) << shift);
            s_mask = mask | (255u << shift);
        }
        __syncthreads();
    }
    const unsigned thr = s_prefix;                          // k-th largest key; s_need of the keys equal to it are kept
    const int need_eq = s_need;
    if (tid == 0) { s_base_kept = 0; s_base_eq = 0; }
    __syncthreads();
    for (int c0 = 0; c0 < P; c0 += blockDim.x) {
        const int t = c0 + tid;
        const unsigned key = t < P ? pooled_key(t) : 0u;
        const int eq = (t < P && key == thr) ? 1 : 0;
        // exclusive scan of eq over the block
        int v = eq;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int n = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += n; }
        if (lane == 31) scan[warp] = v;
        __syncthreads();
        if (warp == 0) {
            int s = scan[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int n = __shfl_up_sync(0xffffffffu, s, o); if (lane >= o) s += n; }
            scan[lane] = s;
        }
        __syncthreads();
        const int eq_rank = s_base_eq + (warp ? scan[warp - 1] : 0) + v - eq;
        const int eq_total = scan[31];
        const int keep = (t < P && (key > thr || (eq && eq_rank < need_eq))) ? 1 : 0;
        __syncthreads();
        int u = keep;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int n = __shfl_up_sync(0xffffffffu, u, o); if (lane >= o) u += n; }
        if (lane == 31) scan[warp] = u;
        __syncthreads();
        if (warp == 0) {
            int s = scan[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int n = __shfl_up_sync(0xffffffffu, s, o); if (lane >= o) s += n; }
            scan[lane] = s;
        }
        __syncthreads();
        const int pos = s_base_kept + (warp ? scan[warp - 1] : 0) + u - keep;
        if (keep && pos < k) kept[pos] = t;
        const int kept_total = scan[31];
        __syncthreads();
        if (tid == 0) { s_base_kept += kept_total; s_base_eq += eq_total; }
        __syncthreads();
    }
    for (int w = tid; w < A.W; w += blockDim.x) kept[k + w] = P + w;
    if (tid == 0 && s_base_kept != k) record_error(A.status, SPARK_ERR_DEVICE_BOUNDS);
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
    if (max_seq_tokens > p.token_budget) {
        evict_pool_kernel<<<dim3((max_seq_tokens + 255) / 256, p.n_kv_heads, p.batch), 256, 0, stream>>>(A);
        ++*launches;
    }
    evict_select_kernel<<<ugrid, 1024, 0, stream>>>(A);
    ++*launches;
    return cudaGetLastError() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

}  // namespace spark
