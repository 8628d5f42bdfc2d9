// Host-side declarations shared by the C-ABI front end and the kernel launchers.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "rpx.h"

namespace rpx {

// Encodes a tiled bf16 tensor map with 128-byte swizzle (inner box extent must be 64 elements).
// dims/strides innermost first; strides_bytes has rank-1 entries (the innermost is contiguous).
// cuTensorMapEncodeTiled is looked up through the runtime, so libcuda is not a link dependency.
rpx_status_t encode_tmap_bf16(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                              const uint64_t* strides_bytes, const uint32_t* box);

int sm_count();                 // multiprocessors of the current device (cached per device)
int sm_budget();                // process-wide cap on persistent grids; 0 = none
void set_sm_budget(int sms);
int lm_head_pairing();          // process-wide: 1 = the LM head runs its CTA-pair (cta_group::2) kernel
void set_lm_head_pairing(int on);
rpx_status_t check_arch();      // RPX_OK on compute capability 10.x

// f32 -> bf16 (round to nearest even) of `rows` rows of `cols` contiguous elements.
rpx_status_t launch_cast_f32_bf16(const float* src, int64_t src_row_stride, __nv_bfloat16_raw* dst, int64_t rows,
                                  int64_t cols, cudaStream_t stream);

struct AttnArgs {
    int32_t num_q_heads, num_kv_heads, head_dim;
    float softmax_scale;
    const void *q, *k, *v;             // bf16
    int64_t q_tok_stride, k_tok_stride, v_tok_stride;
    const int32_t* cu_seqlens;         // query/self-key packing
    const int32_t* prefix_lens;        // NULL for the prefix pass
    int32_t batch;
    int64_t total_tokens;
    int32_t max_q_len, max_prefix_len;
    const rpx_kv_cache_t* cache;       // prefix pass: written (nullable); suffix pass: read
    bool append_cache = false;         // chunked prefill: read the earlier chunks AND append this one
    uint32_t* item_counter = nullptr;  // 4 bytes of workspace: the kernel's work-item counter (zeroed by the launcher)
    void* split_ws = nullptr;          // suffix pass only: room for split-KV partials (attn_split_workspace bytes), or NULL
    void* out;                         // bf16 (launch_attention) or float32 (launch_attention_f32)
    float* lse;
    int32_t* device_status;
    cudaStream_t stream;
};
rpx_status_t launch_attention(const AttnArgs& a);
// RPX_F32: q, k, v are float32 (strides in elements), out is float32; the cache stays bf16.
rpx_status_t launch_attention_f32(const AttnArgs& a);
// Split-KV workspace of a suffix pass over `tokens` query tokens: arrival counters, (max, sum) pairs and fp32
// partial rows for up to 4 ranges; 0 when the pass is too large to ever be split.
size_t attn_split_workspace(int64_t tokens, int32_t num_q_heads, int32_t head_dim);

struct LogprobArgs {
    const void* hidden;   // bf16 [n][hidden_row_stride]
    int64_t hidden_row_stride;
    const void* w;        // bf16 [vocab][hidden_dim]
    const int32_t* target_ids;
    int64_t n_tokens;
    int32_t hidden_dim, vocab;
    float* logprobs;
    float* lse;
    float* entropy;       // nullable
    void* shard_stats;    // nullable float4 [n_tokens]: emit the merged record instead of final outputs
    int32_t target_offset;  // first vocabulary column of `w` (vocabulary-parallel shards), else 0
    void* partials;       // float4 [logprob_num_chunks(vocab, tiles_per_chunk)][n_tokens]
    int32_t tiles_per_chunk;  // vocabulary tiles (256 columns) one work item sweeps
    int32_t* device_status;
    cudaStream_t stream;
};
int32_t logprob_tiles_per_chunk(int64_t n_tokens, int32_t vocab);  // the default policy
int32_t logprob_num_chunks(int32_t vocab, int32_t tiles_per_chunk);
rpx_status_t launch_token_logprobs(const LogprobArgs& a);
rpx_status_t launch_logprob_merge(const void* shard_stats, int32_t n_shards, const int32_t* target_ids, int64_t n_tokens,
                                  int32_t vocab_total, float* logprobs, float* lse, float* entropy, int32_t* status,
                                  cudaStream_t stream);

struct LogprobBwdArgs {
    const void* hidden;        // bf16 [n][hidden_row_stride]
    int64_t hidden_row_stride;
    const void* w;             // bf16 [vocab][hidden_dim]
    const int32_t* target_ids;
    const float* lse;          // [n], from the forward call
    const float* upstream;     // [n], dL / d logprob
    int64_t n_tokens;
    int32_t hidden_dim, vocab;
    void* dhidden;             // bf16 [n][hidden_dim], nullable
    float* dw = nullptr;       // fp32 [vocab][hidden_dim], nullable
    bool accumulate_dw = false;  // add dW to what the buffer holds
    void* dlogits;             // workspace: bf16 [logprob_backward_block_rows(n)][vocab rounded up to 64]
    int32_t* device_status;
    cudaStream_t stream;
};
int64_t logprob_backward_block_rows(int64_t n_tokens);
size_t logprob_backward_workspace(int64_t n_tokens, int32_t vocab);
rpx_status_t launch_token_logprobs_backward(const LogprobBwdArgs& a);

struct AttnBwdArgs {
    int32_t num_q_heads, num_kv_heads, head_dim;
    float softmax_scale;
    const void *q, *k, *v;      // bf16, packed whole sequences
    int64_t q_tok_stride, k_tok_stride, v_tok_stride;
    const void *out, *dout;     // bf16 [tokens][H_q][d], contiguous
    const float* lse;           // [tokens][H_q]
    const int32_t* cu_seqlens;
    const int32_t *q_begin, *q_end;  // nullable: the query rows of every sequence that take part
    int32_t batch;
    int64_t total_tokens;
    int32_t max_seqlen;
    float *dq, *dk, *dv;        // fp32
    bool accumulate;            // add dK / dV to what the buffers hold
    float* dvec;                // workspace: fp32 [tokens][H_q]
    int32_t* device_status;
    cudaStream_t stream;
};
rpx_status_t launch_attention_backward(const AttnBwdArgs& a);

rpx_status_t launch_bounded_wait_selftest(long long limit_cycles, int32_t* status, cudaStream_t stream);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace rpx
