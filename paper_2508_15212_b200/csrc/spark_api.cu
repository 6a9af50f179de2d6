// C ABI of the SparK library: argument checks, sizes, and dispatch to the kernel launchers.
#include <math.h>

#include "spark_common.cuh"

using namespace spark;

static thread_local int g_last_launches = 0;

static inline bool misaligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }
constexpr int32_t kMaxBlocksArg = INT32_MAX / kPageTokens;      // 16 * max_blocks must fit an int

// A NULL block table means a contiguous cache: unit (b, h) owns pages [u * max_blocks, (u + 1) * max_blocks),
// u = b * n_kv_heads + h.  The pool must hold them all.
static inline bool contiguous_pool_too_small(const spark_params* p, const void* block_table, int32_t max_blocks)
{
    return !block_table && static_cast<int64_t>(p->batch) * p->n_kv_heads * max_blocks > p->n_pool_pages;
}

spark_status spark::check_params(const spark_params* p)
{
    if (!p) return SPARK_ERR_NULL;
    if (p->head_dim != kHeadDim || p->page_tokens != kPageTokens) return SPARK_ERR_UNSUPPORTED;
    if (p->dtype != SPARK_F32 && p->dtype != SPARK_BF16) return SPARK_ERR_UNSUPPORTED;
    if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1) return SPARK_ERR_BAD_SHAPE;
    if (p->n_q_heads % p->n_kv_heads) return SPARK_ERR_BAD_SHAPE;
    if (p->n_q_heads / p->n_kv_heads > kMaxGroup) return SPARK_ERR_UNSUPPORTED;
    if (p->batch > kMaxBatch) return SPARK_ERR_UNSUPPORTED;
    if (p->keep < 1 || p->keep > p->head_dim) return SPARK_ERR_BAD_SHAPE;
    if (p->n_pool_pages < 1) return SPARK_ERR_BAD_SHAPE;
    if (p->token_budget < 0) return SPARK_ERR_BAD_SHAPE;
    if (!(p->qnorm_eps >= 0.f) || !(p->softmax_scale >= 0.f)) return SPARK_ERR_BAD_SHAPE;
    if (p->flags & ~(SPARK_FLAG_OVERLAP_PREVIOUS | SPARK_FLAG_HOST_MAPPED)) return SPARK_ERR_BAD_SHAPE;
    if (p->keep_v < 0 || p->keep_v > p->head_dim) return SPARK_ERR_BAD_SHAPE;
    if (p->select < SPARK_SELECT_FIXED || p->select > SPARK_SELECT_GROUPS) return SPARK_ERR_BAD_SHAPE;
    if (p->select == SPARK_SELECT_TOP_P && (!(p->top_p > 0.f) || !(p->top_p <= 1.f))) return SPARK_ERR_BAD_SHAPE;
    if (p->select == SPARK_SELECT_GROUPS) {
        const int need = group_keep(p->head_dim, p->n_groups, p->group_prune);
        if (need < 0 || need > p->keep) return SPARK_ERR_BAD_SHAPE;
    }
    if (p->recovery < SPARK_RECOVER_DEGENERATE || p->recovery > SPARK_RECOVER_EXPONENTIAL) return SPARK_ERR_BAD_SHAPE;
    if (p->recovery != SPARK_RECOVER_DEGENERATE && value_keep(p->keep_v) < kHeadDim) return SPARK_ERR_UNSUPPORTED;
    return SPARK_OK;
}

int spark::group_keep(int head_dim, int n_groups, const float* prune)
{
    if (head_dim < 1 || n_groups < 1 || n_groups > 8 || n_groups > head_dim || !prune) return -1;
    int total = 0;
    for (int i = 0; i < n_groups; ++i) {
        if (!(prune[i] >= 0.f) || !(prune[i] <= 1.f)) return -1;
        const int size = head_dim / n_groups + (i < head_dim % n_groups ? 1 : 0);
        // the small offset absorbs binary representation error of ratios whose product is an integer
        int kp = static_cast<int>(floor((1.0 - static_cast<double>(prune[i])) * size + 1e-9));
        total += kp < 0 ? 0 : (kp > size ? size : kp);
    }
    return total;
}

extern "C" {

int32_t spark_version(void) { return 100; }

int32_t spark_last_launch_count(void) { return g_last_launches; }

int32_t spark_keep_count(int32_t head_dim, double ratio)
{
    if (!(ratio >= 0.0) || !(ratio < 1.0) || head_dim < 1) return -1;
    // the small offset absorbs binary representation error of ratios whose product is an integer
    return static_cast<int32_t>(floor((1.0 - ratio) * head_dim + 1e-9));
}

int32_t spark_group_keep(int32_t head_dim, int32_t n_groups, const float* group_prune)
{
    return group_keep(head_dim, n_groups, group_prune);
}

size_t spark_page_bytes(const spark_params* p)
{
    if (!p || p->head_dim != kHeadDim || p->page_tokens != kPageTokens) return 0;
    if (p->dtype != SPARK_F32 && p->dtype != SPARK_BF16) return 0;
    if (p->keep < 1 || p->keep > kHeadDim) return 0;
    if (p->keep_v < 0 || p->keep_v > kHeadDim) return 0;
    if (p->recovery < SPARK_RECOVER_DEGENERATE || p->recovery > SPARK_RECOVER_EXPONENTIAL) return 0;
    return static_cast<size_t>(make_layout(*p).page_bytes);
}

size_t spark_pool_bytes(const spark_params* p)
{
    const size_t page = spark_page_bytes(p);
    if (!page || p->n_pool_pages < 1) return 0;
    const PageLayout L = make_layout(*p);
    if (!L.ragged) return page * static_cast<size_t>(p->n_pool_pages);
    return static_cast<size_t>(rows_offset(p->n_pool_pages, L.page_bytes)) + static_cast<size_t>(p->n_pool_pages) * sizeof(int32_t);
}

size_t spark_algorithmic_bytes_per_token(const spark_params* p)
{
    if (!p || p->keep < 1 || p->keep > p->head_dim || p->keep_v < 0 || p->keep_v > p->head_dim) return 0;
    const size_t e = (p->dtype == SPARK_BF16) ? 2 : 4;
    const int tv = value_keep(p->keep_v);
    const size_t stats = (p->recovery != SPARK_RECOVER_DEGENERATE) ? 8 : 0;       // all-channel mean and deviation
    return e * p->keep + 16 + 4 + stats + (tv < kHeadDim ? e * tv + 16 : e * p->head_dim);
}

spark_status spark_workspace_bytes(const spark_params* p, int64_t max_seq_tokens,
                                   size_t* compress_bytes, size_t* decode_bytes)
{
    spark_status st = check_params(p);
    if (st != SPARK_OK) return st;
    if (max_seq_tokens < 0) return SPARK_ERR_BAD_SHAPE;
    if (compress_bytes) *compress_bytes = compress_workspace_bytes(*p, max_seq_tokens);
    if (decode_bytes) *decode_bytes = decode_workspace_bytes(*p);
    return SPARK_OK;
}

spark_status spark_workspace_init(void* workspace, size_t workspace_bytes, spark_stream_t stream)
{
    if (!workspace) return SPARK_ERR_NULL;
    if (workspace_bytes < kWorkspaceHeader || (reinterpret_cast<uintptr_t>(workspace) & 255))
        return SPARK_ERR_WORKSPACE;
    if (cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return SPARK_ERR_CUDA;
    return SPARK_OK;
}

spark_status spark_compress(const spark_params* p, const void* q_win, const void* k, const void* v,
                            int64_t stride_b, int64_t stride_h, int64_t stride_t,
                            const int32_t* seq_lens, int32_t max_seq_tokens, void* pages,
                            const int32_t* block_table, int32_t max_blocks, float* qnorm,
                            int32_t* packed_lens, int32_t* kept_tokens, void* workspace,
                            size_t workspace_bytes, spark_stream_t stream)
{
    spark_status st = check_params(p);
    if (st != SPARK_OK) return st;
    if (!q_win || !k || !v || !seq_lens || !pages || !qnorm || !packed_lens || !workspace)
        return SPARK_ERR_NULL;
    if (p->window < 1 || max_seq_tokens < 0 || max_blocks < 0 || max_blocks > kMaxBlocksArg) return SPARK_ERR_BAD_SHAPE;
    if (stride_t < p->head_dim || stride_b < 0 || stride_h < 0) return SPARK_ERR_BAD_SHAPE;
    if (misaligned(pages, 16) || misaligned(qnorm, 16)) return SPARK_ERR_BAD_SHAPE;
    if (contiguous_pool_too_small(p, block_table, max_blocks)) return SPARK_ERR_BAD_SHAPE;
    // vector loads of K/V rows need 16-byte aligned rows
    const int e = (p->dtype == SPARK_BF16) ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(k) & 15) || (reinterpret_cast<uintptr_t>(v) & 15) ||
        ((stride_b * e) & 15) || ((stride_h * e) & 15) || ((stride_t * e) & 15))
        return SPARK_ERR_BAD_SHAPE;
    if (p->token_budget > 0) {
        if (p->token_budget < p->window || p->pool_kernel < 1 || !(p->pool_kernel & 1))
            return SPARK_ERR_BAD_SHAPE;
        if (!kept_tokens) return SPARK_ERR_NULL;
    }
    const int64_t max_packed = (p->token_budget > 0 && p->token_budget < max_seq_tokens)
                                   ? p->token_budget : max_seq_tokens;
    if ((max_packed + kPageTokens - 1) / kPageTokens > max_blocks) return SPARK_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) ||
        workspace_bytes < compress_workspace_bytes(*p, max_seq_tokens))
        return SPARK_ERR_WORKSPACE;
    int launches = 0;
    st = launch_compress(*p, q_win, k, v, stride_b, stride_h, stride_t, seq_lens, max_seq_tokens, pages,
                         block_table, max_blocks, qnorm, packed_lens, kept_tokens, workspace,
                         workspace_bytes, static_cast<cudaStream_t>(stream), &launches);
    if (st == SPARK_OK) g_last_launches = launches;
    return st;
}

spark_status spark_append(const spark_params* p, const void* k_new, const void* v_new, void* pages,
                          const int32_t* block_table, int32_t max_blocks, const float* qnorm,
                          int32_t* packed_lens, void* workspace, size_t workspace_bytes, spark_stream_t stream)
{
    spark_status st = check_params(p);
    if (st != SPARK_OK) return st;
    if (!k_new || !v_new || !pages || !qnorm || !packed_lens || !workspace) return SPARK_ERR_NULL;
    if (max_blocks < 1 || max_blocks > kMaxBlocksArg) return SPARK_ERR_BAD_SHAPE;
    if (contiguous_pool_too_small(p, block_table, max_blocks)) return SPARK_ERR_BAD_SHAPE;
    if (misaligned(pages, 16) || misaligned(k_new, 16) || misaligned(v_new, 16) || misaligned(qnorm, 16))
        return SPARK_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < kWorkspaceHeader) return SPARK_ERR_WORKSPACE;
    int launches = 0;
    st = launch_append(*p, k_new, v_new, pages, block_table, max_blocks, qnorm, packed_lens, workspace,
                       static_cast<cudaStream_t>(stream), &launches);
    if (st == SPARK_OK) g_last_launches = launches;
    return st;
}

spark_status spark_append_block(const spark_params* p, const void* k_new, const void* v_new, int32_t n_new,
                                void* pages, const int32_t* block_table, int32_t max_blocks, const float* qnorm,
                                int32_t* packed_lens, void* workspace, size_t workspace_bytes, spark_stream_t stream)
{
    spark_status st = check_params(p);
    if (st != SPARK_OK) return st;
    if (!k_new || !v_new || !pages || !qnorm || !packed_lens || !workspace) return SPARK_ERR_NULL;
    if (max_blocks < 1 || max_blocks > kMaxBlocksArg || n_new < 0 || n_new > 65535) return SPARK_ERR_BAD_SHAPE;
    if (contiguous_pool_too_small(p, block_table, max_blocks)) return SPARK_ERR_BAD_SHAPE;
    if (misaligned(pages, 16) || misaligned(k_new, 16) || misaligned(v_new, 16) || misaligned(qnorm, 16))
        return SPARK_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < kWorkspaceHeader) return SPARK_ERR_WORKSPACE;
    int launches = 0;
    st = launch_append_block(*p, k_new, v_new, n_new, pages, block_table, max_blocks, qnorm, packed_lens, workspace,
                             static_cast<cudaStream_t>(stream), &launches);
    if (st == SPARK_OK) g_last_launches = launches;
    return st;
}

spark_status spark_merge_attn(int32_t batch, int32_t n_q_heads, int32_t head_dim, const float* out_a,
                              const float* lse_a, const float* out_b, const float* lse_b, float* out, float* lse,
                              spark_stream_t stream)
{
    if (!out_a || !lse_a || !out_b || !lse_b || !out) return SPARK_ERR_NULL;
    if (head_dim != kHeadDim) return SPARK_ERR_UNSUPPORTED;
    if (batch < 0 || n_q_heads < 0 || static_cast<int64_t>(batch) * n_q_heads > INT32_MAX) return SPARK_ERR_BAD_SHAPE;
    if (misaligned(out_a, 16) || misaligned(out_b, 16) || misaligned(out, 16)) return SPARK_ERR_BAD_SHAPE;
    return launch_merge_attn(batch * n_q_heads, out_a, lse_a, out_b, lse_b, out, lse, static_cast<cudaStream_t>(stream));
}

// spark_decode_attn proper; q_by_value: q is a host pointer whose bytes go into the launch (see launch_decode)
static spark_status decode_attn(const spark_params* p, const void* q, const void* pages,
                                const int32_t* block_table, int32_t max_blocks,
                                const int32_t* packed_lens, const float* qnorm, float* out, float* lse,
                                void* workspace, size_t workspace_bytes, spark_stream_t stream, bool q_by_value)
{
    spark_status st = check_params(p);
    if (st != SPARK_OK) return st;
    if (!q || !pages || !packed_lens || !qnorm || !out || !workspace) return SPARK_ERR_NULL;
    if (max_blocks < 0 || max_blocks > kMaxBlocksArg) return SPARK_ERR_BAD_SHAPE;
    if (contiguous_pool_too_small(p, block_table, max_blocks)) return SPARK_ERR_BAD_SHAPE;
    // the kernels read q and qnorm and write out with 16-byte vector accesses
    if (misaligned(pages, 16) || misaligned(q, 16) || misaligned(qnorm, 16) || misaligned(out, 16) ||
        misaligned(lse, 4))
        return SPARK_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < decode_workspace_bytes(*p))
        return SPARK_ERR_WORKSPACE;
    int launches = 0;
    st = launch_decode(*p, q, pages, block_table, max_blocks, packed_lens, qnorm, out, lse, workspace,
                       workspace_bytes, static_cast<cudaStream_t>(stream), &launches, q_by_value);
    if (st == SPARK_OK) g_last_launches = launches;
    return st;
}

spark_status spark_decode_attn(const spark_params* p, const void* q, const void* pages,
                               const int32_t* block_table, int32_t max_blocks,
                               const int32_t* packed_lens, const float* qnorm, float* out, float* lse,
                               void* workspace, size_t workspace_bytes, spark_stream_t stream)
{
    return decode_attn(p, q, pages, block_table, max_blocks, packed_lens, qnorm, out, lse, workspace, workspace_bytes,
                       stream, false);
}

spark_status spark_decode_attn_host(const spark_params* p, const void* q_host, void* q_dev, const void* pages,
                                    const int32_t* block_table, int32_t max_blocks,
                                    const int32_t* packed_lens, const float* qnorm, float* out_dev,
                                    float* out_host, float* lse_dev, float* lse_host, void* workspace,
                                    size_t workspace_bytes, spark_stream_t stream)
{
    spark_status st = check_params(p);
    if (st != SPARK_OK) return st;
    if (!q_host || !out_host) return SPARK_ERR_NULL;
    if (p->flags & SPARK_FLAG_HOST_MAPPED) {
        // The kernel writes the result (posted stores) straight into the page-locked host buffers.  The query
        // travels inside the launch when it is small enough (read here, during the call); otherwise the kernel
        // reads it over the bus during the step.
        const size_t q_bytes = static_cast<size_t>(p->batch) * p->n_q_heads * p->head_dim * 2;
        const bool by_value = p->dtype == SPARK_BF16 && p->recovery == SPARK_RECOVER_DEGENERATE &&
                              value_keep(p->keep_v) == kHeadDim && q_bytes <= query_by_value_limit();
        void *dq = nullptr, *dout = nullptr, *dlse = nullptr;
        if ((!by_value && cudaHostGetDevicePointer(&dq, const_cast<void*>(q_host), 0) != cudaSuccess) ||
            cudaHostGetDevicePointer(&dout, out_host, 0) != cudaSuccess ||
            (lse_host && cudaHostGetDevicePointer(&dlse, lse_host, 0) != cudaSuccess)) {
            cudaGetLastError();                            // clear the sticky-free error of the failed lookup
            return SPARK_ERR_BAD_SHAPE;
        }
        return decode_attn(p, by_value ? q_host : dq, pages, block_table, max_blocks, packed_lens, qnorm,
                           static_cast<float*>(dout), static_cast<float*>(dlse), workspace, workspace_bytes, stream,
                           by_value);
    }
    if (!q_dev || !out_dev) return SPARK_ERR_NULL;
    if ((lse_dev == nullptr) != (lse_host == nullptr)) return SPARK_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t e = (p->dtype == SPARK_BF16) ? 2 : 4;
    const size_t nq = static_cast<size_t>(p->batch) * p->n_q_heads * p->head_dim;
    if (cudaMemcpyAsync(q_dev, q_host, nq * e, cudaMemcpyHostToDevice, s) != cudaSuccess) return SPARK_ERR_CUDA;
    st = spark_decode_attn(p, q_dev, pages, block_table, max_blocks, packed_lens, qnorm, out_dev, lse_dev,
                           workspace, workspace_bytes, stream);
    if (st != SPARK_OK) return st;
    if (cudaMemcpyAsync(out_host, out_dev, nq * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return SPARK_ERR_CUDA;
    if (lse_dev && cudaMemcpyAsync(lse_host, lse_dev, static_cast<size_t>(p->batch) * p->n_q_heads * sizeof(float),
                                   cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return SPARK_ERR_CUDA;
    return SPARK_OK;
}

spark_status spark_unpack_pages(const spark_params* p, const void* pages, const int32_t* block_table,
                                int32_t max_blocks, const int32_t* packed_lens, int32_t max_tokens,
                                uint32_t* mask, float* mu, void* vals, void* v, spark_stream_t stream)
{
    spark_status st = check_params(p);
    if (st != SPARK_OK) return st;
    if (!pages || !packed_lens) return SPARK_ERR_NULL;
    if (contiguous_pool_too_small(p, block_table, max_blocks)) return SPARK_ERR_BAD_SHAPE;
    if (max_tokens < 0 || max_blocks < 0 || max_blocks > kMaxBlocksArg) return SPARK_ERR_BAD_SHAPE;
    if ((static_cast<int64_t>(max_tokens) + kPageTokens - 1) / kPageTokens > max_blocks)
        return SPARK_ERR_BAD_SHAPE;
    return launch_unpack(*p, pages, block_table, max_blocks, packed_lens, max_tokens, mask, mu, vals, v, nullptr,
                         nullptr, nullptr, static_cast<cudaStream_t>(stream));
}

spark_status spark_unpack_stats(const spark_params* p, const void* pages, const int32_t* block_table,
                                int32_t max_blocks, const int32_t* packed_lens, int32_t max_tokens,
                                float* mu_all, float* sigma_all, spark_stream_t stream)
{
    spark_status st = check_params(p);
    if (st != SPARK_OK) return st;
    if (!pages || !packed_lens) return SPARK_ERR_NULL;
    if (p->recovery == SPARK_RECOVER_DEGENERATE) return SPARK_ERR_UNSUPPORTED;
    if (contiguous_pool_too_small(p, block_table, max_blocks)) return SPARK_ERR_BAD_SHAPE;
    if (max_tokens < 0 || max_blocks < 0 || max_blocks > kMaxBlocksArg) return SPARK_ERR_BAD_SHAPE;
    if ((static_cast<int64_t>(max_tokens) + kPageTokens - 1) / kPageTokens > max_blocks)
        return SPARK_ERR_BAD_SHAPE;
    return launch_unpack(*p, pages, block_table, max_blocks, packed_lens, max_tokens, nullptr, nullptr, nullptr,
                         nullptr, nullptr, mu_all, sigma_all, static_cast<cudaStream_t>(stream));
}

spark_status spark_unpack_value_masks(const spark_params* p, const void* pages, const int32_t* block_table,
                                      int32_t max_blocks, const int32_t* packed_lens, int32_t max_tokens,
                                      uint32_t* vmask, spark_stream_t stream)
{
    spark_status st = check_params(p);
    if (st != SPARK_OK) return st;
    if (!pages || !packed_lens || !vmask) return SPARK_ERR_NULL;
    if (contiguous_pool_too_small(p, block_table, max_blocks)) return SPARK_ERR_BAD_SHAPE;
    if (max_tokens < 0 || max_blocks < 0) return SPARK_ERR_BAD_SHAPE;
    if ((static_cast<int64_t>(max_tokens) + kPageTokens - 1) / kPageTokens > max_blocks)
        return SPARK_ERR_BAD_SHAPE;
    return launch_unpack(*p, pages, block_table, max_blocks, packed_lens, max_tokens, nullptr, nullptr, nullptr,
                         nullptr, vmask, nullptr, nullptr, static_cast<cudaStream_t>(stream));
}

spark_status spark_read_status(const void* workspace, spark_stream_t stream)
{
    if (!workspace) return SPARK_ERR_NULL;
    int code = 0;
    if (cudaMemcpyAsync(&code, workspace, sizeof(int), cudaMemcpyDeviceToHost,
                        static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return SPARK_ERR_CUDA;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return SPARK_ERR_CUDA;
    return static_cast<spark_status>(code);
}

}  // extern "C"
