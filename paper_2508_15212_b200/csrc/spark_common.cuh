// Shared declarations of the SparK CUDA library: page layout, status word, small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/spark.h"

namespace spark {

constexpr int kHeadDim = 128;        // D
constexpr int kPageTokens = 16;      // P
constexpr int kMaskWords = 4;        // 128-bit channel mask per token
constexpr int kMaxGroup = 8;         // G = Hq / Hkv
constexpr int kMaxBatch = 1024;      // sequences per call (decode keeps a per-sequence prefix in shared memory)
constexpr int kMaxCtas = 256;        // upper bound of the persistent decode grid (sizes the partial-result slots)
constexpr int kWorkspaceHeader = 256;

// Byte layout of one page (16 tokens of one KV head).  Private to the library.
//
//   vals : T rows of 16 elements.  Row s holds kept slot s of every token; slot s of a token is its
//          s-th kept channel in ascending channel order.  Rows are 32 bytes (bf16) or 64 bytes (fp32), so
//          the section is exactly T elements per token.  In fp32 rows token p sits at element p; in bf16
//          rows at element (p & 7) * 2 + (p >> 3), so the eight tokens that one half of a matrix
//          fragment reads together fall into eight different 4-byte banks.
//   mask : [16][4] uint32, bit (j % 32) of word (j / 32) set <=> channel j kept
//   mu   : [16] float, mean saliency of the pruned channels
//   stats: (sampled recovery only) [16] float mean and [16] float population deviation of ALL the token's saliencies
//   v    : dense values (keep_v == 128): [16][128] elements, the value rows.  In bf16 pages the 16-byte
//          chunks of row p are stored at chunk index (c ^ (p & 7)), which makes the transposing matrix
//          loads of the decode kernel free of bank conflicts; fp32 pages store rows plainly.
//          pruned values (keep_v < 128): T_v rows of 16 elements laid out exactly like `vals` (slot s of
//          a token = its s-th kept value channel), followed by
//   vmask: [16][4] uint32 (pruned values only), bit (j % 32) of word (j / 32) set <=> value channel j kept
struct PageLayout {
    int vals_off;    // start of the kept key values (0, or behind everything else when `ragged`)
    int ragged;      // SparK-p pages: the slot rows come last and a per-page row count says how many are in use
    int esize;       // bytes per element (2 bf16, 4 fp32)
    int keep;        // T
    int keep_v;      // T_v (128: dense value rows)
    int mask_off;
    int mu_off;
    int stats_off;   // [16] float all-channel mean, [16] float population deviation (sampled recovery only)
    int recovery;    // spark_recovery
    int v_off;
    int vmask_off;   // meaningful when keep_v < 128
    int page_bytes;
};

// spark_params.keep_v -> T_v (0 and 128 both mean dense value rows)
__host__ __device__ inline int value_keep(int keep_v) { return (keep_v <= 0 || keep_v >= kHeadDim) ? kHeadDim : keep_v; }

// With SparK-p the number of kept channels varies per token, so a page's slot rows are only used up to the
// largest count among its 16 tokens.  Such pages are laid out with the slot rows LAST, and a row count per
// pool page (int32, in a side array behind the pages of the pool) tells the decode step how many bytes of the
// page to copy: mask | mu | (stats) | values | the first `rows` slot rows.
__host__ __device__ inline PageLayout make_layout(int dtype, int keep, int keep_v, int recovery, int ragged = 0)
{
    PageLayout L;
    L.esize = (dtype == SPARK_BF16) ? 2 : 4;
    L.keep = keep;
    L.keep_v = value_keep(keep_v);
    L.ragged = ragged;
    L.vals_off = 0;
    L.mask_off = ragged ? 0 : keep * kPageTokens * L.esize;
    L.mu_off = L.mask_off + kPageTokens * 16;
    L.stats_off = L.mu_off + kPageTokens * 4;
    L.recovery = recovery;
    L.v_off = L.stats_off + (recovery != SPARK_RECOVER_DEGENERATE ? 2 * kPageTokens * 4 : 0);
    L.vmask_off = L.v_off + L.keep_v * kPageTokens * L.esize;
    L.page_bytes = L.vmask_off + (L.keep_v < kHeadDim ? kPageTokens * 16 : 0);
    if (ragged) {
        L.vals_off = L.page_bytes;
        L.page_bytes += keep * kPageTokens * L.esize;
    }
    return L;
}

// the per-page row counts of a ragged pool: an int32 per pool page behind the pages (256-byte aligned)
__host__ __device__ inline int64_t rows_offset(int64_t n_pool_pages, int page_bytes)
{
    return (n_pool_pages * page_bytes + 255) / 256 * 256;
}

// byte offset of kept slot s of token p inside the vals section
__host__ __device__ inline int val_offset(int esize, int p, int s)
{
    return esize == 2 ? (s * kPageTokens + ((p & 7) * 2 + (p >> 3))) * 2 : (s * kPageTokens + p) * 4;
}

// byte offset (inside the v section) of the 16-byte chunk c of token p's value row
__host__ __device__ inline int v_chunk_offset(int esize, int p, int c)
{
    return esize == 2 ? (p * (kHeadDim * 2) + ((c ^ (p & 7)) << 4)) : (p * (kHeadDim * 4) + (c << 4));
}

// Workspace header: word 0 is the status word (first error wins).
__device__ inline void record_error(int* status, int code)
{
    atomicCAS(status, 0, code);
}

__device__ __forceinline__ float bf16_bits_to_float(unsigned short h)
{
    return __uint_as_float(static_cast<unsigned>(h) << 16);
}

template <typename E> struct Elem;
template <> struct Elem<float> {
    static constexpr int dtype = SPARK_F32;
    __device__ static float load(const void* p, int64_t i) { return static_cast<const float*>(p)[i]; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int dtype = SPARK_BF16;
    __device__ static float load(const void* p, int64_t i)
    {
        return bf16_bits_to_float(static_cast<const unsigned short*>(p)[i]);
    }
};

// host-side validation of a parameter block (spark_api.cu)
spark_status check_params(const spark_params* p);

// ---- host-side launchers implemented in the .cu files -------------------------------------------
spark_status launch_compress(const spark_params& p, const void* q_win, const void* k, const void* v,
                             int64_t sb, int64_t sh, int64_t st, const int32_t* seq_lens,
                             int32_t max_seq_tokens, void* pages, const int32_t* block_table,
                             int32_t max_blocks, float* qnorm, int32_t* packed_lens, int32_t* kept_tokens,
                             void* workspace, size_t workspace_bytes, cudaStream_t stream, int* launches);

spark_status launch_unpack(const spark_params& p, const void* pages, const int32_t* block_table,
                           int32_t max_blocks, const int32_t* packed_lens, int32_t max_tokens,
                           uint32_t* mask, float* mu, void* vals, void* v, uint32_t* vmask, float* mu_all,
                           float* sigma_all, cudaStream_t stream);
inline PageLayout make_layout(const spark_params& p)
{
    return make_layout(p.dtype, p.keep, p.keep_v, p.recovery, p.select == SPARK_SELECT_TOP_P ? 1 : 0);
}
int group_keep(int head_dim, int n_groups, const float* prune);

spark_status launch_decode(const spark_params& p, const void* q, const void* pages,
                           const int32_t* block_table, int32_t max_blocks, const int32_t* packed_lens,
                           const float* qnorm, float* out, float* lse, void* workspace,
                           size_t workspace_bytes, cudaStream_t stream, int* launches, bool q_by_value = false);
// q_by_value: q is a HOST pointer and its bytes travel as a launch parameter (bf16 storage, degenerate recovery,
// dense value rows, at most query_by_value_limit() bytes; anything else is refused)
size_t query_by_value_limit();

spark_status launch_append(const spark_params& p, const void* k_new, const void* v_new, void* pages,
                           const int32_t* block_table, int32_t max_blocks, const float* qnorm,
                           int32_t* packed_lens, void* workspace, cudaStream_t stream, int* launches);

spark_status launch_append_block(const spark_params& p, const void* k_new, const void* v_new, int32_t n_new,
                                 void* pages, const int32_t* block_table, int32_t max_blocks, const float* qnorm,
                                 int32_t* packed_lens, void* workspace, cudaStream_t stream, int* launches);
spark_status launch_merge_attn(int rows, const float* out_a, const float* lse_a, const float* out_b, const float* lse_b,
                               float* out, float* lse, cudaStream_t stream);

size_t decode_workspace_bytes(const spark_params& p);
size_t evict_workspace_bytes(const spark_params& p, int64_t max_seq_tokens);
spark_status launch_evict(const spark_params& p, const void* q_win, const void* k, int64_t sb, int64_t sh,
                          int64_t st, const int32_t* seq_lens, int32_t max_seq_tokens, int32_t* packed_lens,
                          int32_t* kept_tokens, void* workspace, cudaStream_t stream, int* launches);
size_t compress_workspace_bytes(const spark_params& p, int64_t max_seq_tokens);

}  // namespace spark
