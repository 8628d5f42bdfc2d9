// C-ABI front end: host-side validation, workspace carving, the fp32 -> bf16 pre-pass, and
// dispatch to the sm_100a kernels.  Nothing here allocates device memory or synchronises.
#include <cuda_bf16.h>

#include "rpx_internal.h"

namespace {

using namespace rpx;

constexpr size_t kWsAlign = 256;

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
// Workspaces are carved in 256-byte pieces that the kernels access with vector loads and stores of up to 32 bytes.
bool aligned_ws(const void* p) { return (reinterpret_cast<uintptr_t>(p) & (kWsAlign - 1)) == 0; }

rpx_status_t check_attn_desc(const rpx_attn_desc_t* d) {
    if (d == nullptr) return RPX_ERR_NULL;
    if (d->dtype != RPX_BF16 && d->dtype != RPX_F32) return RPX_ERR_DTYPE;
    if (d->head_dim != 64 && d->head_dim != 128) return RPX_ERR_SHAPE;
    if (d->num_q_heads <= 0 || d->num_kv_heads <= 0 || d->num_q_heads % d->num_kv_heads != 0) return RPX_ERR_SHAPE;
    return RPX_OK;
}

// Layout: [work-item counter, kWsAlign bytes][suffix passes small enough to be split over the cached prefix:
// split-KV partials].  The RPX_F32 path keeps nothing there, but asks for the counter's piece all the same so that a
// caller's workspace handling does not depend on the element type.
size_t attn_workspace(const rpx_attn_desc_t* d, int64_t tokens, bool is_suffix) {
    if (d == nullptr || tokens <= 0) return 0;
    if (d->dtype == RPX_F32) return kWsAlign;
    return kWsAlign + (is_suffix ? attn_split_workspace(tokens, d->num_q_heads, d->head_dim) : 0);
}

rpx_status_t check_cache(const rpx_kv_cache_t* c, int32_t batch) {
    if (c->k_cache == nullptr || c->v_cache == nullptr || c->block_table == nullptr) return RPX_ERR_NULL;
    if (c->block_size != 16 || c->num_blocks <= 0 || c->num_blocks > INT32_MAX) return RPX_ERR_SHAPE;
    if (batch > 0 && c->block_table_stride <= 0) return RPX_ERR_SHAPE;
    if (!aligned16(c->k_cache) || !aligned16(c->v_cache)) return RPX_ERR_ALIGN;
    return RPX_OK;
}

// Shared body of the two attention entry points.  prefix_lens == NULL selects the prefix pass.
rpx_status_t run_attention(const rpx_attn_desc_t* desc, const void* q, const void* k, const void* v,
                           int64_t q_tok_stride, int64_t k_tok_stride, int64_t v_tok_stride, const int32_t* cu_seqlens,
                           const int32_t* prefix_lens, bool is_suffix, bool append_cache, int32_t batch, int64_t total_tokens,
                           int32_t max_q_len, int32_t max_prefix_len, const rpx_kv_cache_t* cache, void* out, float* lse,
                           void* workspace, size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
    if (rpx_status_t rc = check_attn_desc(desc)) return rc;
    if (batch < 0 || total_tokens < 0 || max_q_len < 0 || max_prefix_len < 0) return RPX_ERR_SHAPE;
    if (total_tokens >= INT32_MAX) return RPX_ERR_SHAPE;
    if (is_suffix) {
        if (cache == nullptr) return RPX_ERR_NULL;
        if (batch > 0 && prefix_lens == nullptr) return RPX_ERR_NULL;
    }
    if (cache != nullptr)
        if (rpx_status_t rc = check_cache(cache, batch)) return rc;
    if (batch == 0 || total_tokens == 0 || max_q_len == 0) return RPX_OK;
    if (q == nullptr || k == nullptr || v == nullptr || out == nullptr || cu_seqlens == nullptr) return RPX_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return RPX_ERR_ALIGN;
    const int64_t q_row = static_cast<int64_t>(desc->num_q_heads) * desc->head_dim;
    const int64_t kv_row = static_cast<int64_t>(desc->num_kv_heads) * desc->head_dim;
    if (q_tok_stride < q_row || k_tok_stride < kv_row || v_tok_stride < kv_row) return RPX_ERR_SHAPE;
    if (q_tok_stride % 8 || k_tok_stride % 8 || v_tok_stride % 8) return RPX_ERR_ALIGN;
    const size_t need = attn_workspace(desc, total_tokens, is_suffix);
    if (need > 0 && (workspace == nullptr || workspace_bytes < need)) return RPX_ERR_WORKSPACE;
    if (need > 0 && !aligned_ws(workspace)) return RPX_ERR_ALIGN;
    if (rpx_status_t rc = check_arch()) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    AttnArgs a;
    a.num_q_heads = desc->num_q_heads;
    a.num_kv_heads = desc->num_kv_heads;
    a.head_dim = desc->head_dim;
    a.softmax_scale = desc->softmax_scale;
    a.q = q;
    a.k = k;
    a.v = v;
    a.q_tok_stride = q_tok_stride;
    a.k_tok_stride = k_tok_stride;
    a.v_tok_stride = v_tok_stride;
    a.cu_seqlens = cu_seqlens;
    a.prefix_lens = is_suffix ? prefix_lens : nullptr;
    a.batch = batch;
    a.total_tokens = total_tokens;
    a.max_q_len = max_q_len;
    a.max_prefix_len = max_prefix_len;
    a.cache = cache;
    a.item_counter = static_cast<uint32_t*>(workspace);
    if (is_suffix && desc->dtype != RPX_F32 && attn_split_workspace(total_tokens, desc->num_q_heads, desc->head_dim) > 0)
        a.split_ws = static_cast<uint8_t*>(workspace) + kWsAlign;
    a.append_cache = is_suffix && append_cache;
    a.out = out;
    a.lse = lse;
    a.device_status = device_status;
    a.stream = stream;
    // fp32 tensors take the fp32 CUDA-core path; out is then float32 and 16-byte alignment is all the tensors need
    if (desc->dtype == RPX_F32) return launch_attention_f32(a);
    return launch_attention(a);
}

}  // namespace

extern "C" {

rpx_status_t rpx_prefix_attn(const rpx_attn_desc_t* desc, const void* q, const void* k, const void* v,
                             int64_t q_tok_stride, int64_t k_tok_stride, int64_t v_tok_stride,
                             const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens, int32_t max_seqlen,
                             const rpx_kv_cache_t* cache, void* out, float* lse, void* workspace,
                             size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
    return run_attention(desc, q, k, v, q_tok_stride, k_tok_stride, v_tok_stride, cu_seqlens, nullptr, false, false, batch,
                         total_tokens, max_seqlen, 0, cache, out, lse, workspace, workspace_bytes, device_status,
                         cuda_stream);
}

rpx_status_t rpx_suffix_attn(const rpx_attn_desc_t* desc, const void* q, const void* k, const void* v,
                             int64_t q_tok_stride, int64_t k_tok_stride, int64_t v_tok_stride,
                             const int32_t* cu_seqlens_suffix, const int32_t* prefix_lens, int32_t batch,
                             int64_t total_suffix_tokens, int32_t max_suffix_len, int32_t max_prefix_len,
                             const rpx_kv_cache_t* cache, void* out, float* lse, void* workspace,
                             size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
    return run_attention(desc, q, k, v, q_tok_stride, k_tok_stride, v_tok_stride, cu_seqlens_suffix, prefix_lens, true,
                         false, batch, total_suffix_tokens, max_suffix_len, max_prefix_len, cache, out, lse, workspace,
                         workspace_bytes, device_status, cuda_stream);
}

size_t rpx_prefix_attn_workspace_bytes(const rpx_attn_desc_t* desc, int64_t total_tokens) {
    return attn_workspace(desc, total_tokens, false);
}

rpx_status_t rpx_chunk_attn(const rpx_attn_desc_t* desc, const void* q, const void* k, const void* v,
                            int64_t q_tok_stride, int64_t k_tok_stride, int64_t v_tok_stride, const int32_t* cu_seqlens_chunk,
                            const int32_t* cached_lens, int32_t batch, int64_t total_chunk_tokens, int32_t max_chunk_len,
                            int32_t max_cached_len, const rpx_kv_cache_t* cache, void* out, float* lse, void* workspace,
                            size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
    return run_attention(desc, q, k, v, q_tok_stride, k_tok_stride, v_tok_stride, cu_seqlens_chunk, cached_lens, true,
                         true, batch, total_chunk_tokens, max_chunk_len, max_cached_len, cache, out, lse, workspace,
                         workspace_bytes, device_status, cuda_stream);
}

size_t rpx_suffix_attn_workspace_bytes(const rpx_attn_desc_t* desc, int64_t total_suffix_tokens) {
    return attn_workspace(desc, total_suffix_tokens, true);
}

size_t rpx_token_logprobs_workspace_bytes(int64_t n_tokens, int32_t hidden_dim, int32_t vocab, rpx_dtype_t dtype) {
    if (n_tokens <= 0 || hidden_dim <= 0 || vocab <= 0) return 0;
    size_t bytes = align_up(static_cast<size_t>(logprob_num_chunks(vocab, logprob_tiles_per_chunk(n_tokens, vocab))) * n_tokens * sizeof(float4), kWsAlign);
    if (dtype == RPX_F32) {
        bytes += align_up(static_cast<size_t>(n_tokens) * hidden_dim * 2, kWsAlign);
        bytes += align_up(static_cast<size_t>(vocab) * hidden_dim * 2, kWsAlign);
    }
    return bytes;
}

}  // extern "C"

namespace {

// Shared body of the LM-head entry points.  shard_stats != NULL selects the vocabulary-shard form
// (W holds columns vocab_begin .. vocab_begin + vocab - 1; the merged record per row is the output).
rpx_status_t run_token_logprobs(const void* hidden, int64_t hidden_row_stride, const void* w_vocab,
                                const int32_t* target_ids, int64_t n_tokens, int32_t hidden_dim, int32_t vocab,
                                int32_t vocab_begin, rpx_dtype_t dtype, float* logprobs, float* lse, float* entropy,
                                float* shard_stats, void* workspace, size_t workspace_bytes, int32_t* device_status,
                                void* cuda_stream) {
    if (dtype != RPX_BF16 && dtype != RPX_F32) return RPX_ERR_DTYPE;
    if (n_tokens < 0 || n_tokens >= INT32_MAX || hidden_dim <= 0 || vocab <= 0) return RPX_ERR_SHAPE;
    if (hidden_dim % 8 != 0) return RPX_ERR_SHAPE;
    if (n_tokens == 0) return RPX_OK;
    if (hidden == nullptr || w_vocab == nullptr || target_ids == nullptr) return RPX_ERR_NULL;
    if (logprobs == nullptr && shard_stats == nullptr) return RPX_ERR_NULL;
    if (vocab_begin < 0) return RPX_ERR_SHAPE;
    if (hidden_row_stride < hidden_dim) return RPX_ERR_SHAPE;
    if (hidden_row_stride % 8 != 0) return RPX_ERR_ALIGN;
    if (!aligned16(hidden) || !aligned16(w_vocab) || !aligned16(shard_stats)) return RPX_ERR_ALIGN;
    const size_t need = rpx_token_logprobs_workspace_bytes(n_tokens, hidden_dim, vocab, dtype);
    if (workspace == nullptr || workspace_bytes < need) return RPX_ERR_WORKSPACE;
    if (!aligned_ws(workspace)) return RPX_ERR_ALIGN;
    if (rpx_status_t rc = check_arch()) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    uint8_t* ws = static_cast<uint8_t*>(workspace);
    LogprobArgs a;
    a.partials = ws;
    a.tiles_per_chunk = logprob_tiles_per_chunk(n_tokens, vocab);
    ws += align_up(static_cast<size_t>(logprob_num_chunks(vocab, a.tiles_per_chunk)) * n_tokens * sizeof(float4), kWsAlign);
    a.hidden = hidden;
    a.hidden_row_stride = hidden_row_stride;
    a.w = w_vocab;
    if (dtype == RPX_F32) {
        auto* hh = reinterpret_cast<__nv_bfloat16_raw*>(ws);
        ws += align_up(static_cast<size_t>(n_tokens) * hidden_dim * 2, kWsAlign);
        auto* wh = reinterpret_cast<__nv_bfloat16_raw*>(ws);
        if (rpx_status_t rc = launch_cast_f32_bf16(static_cast<const float*>(hidden), hidden_row_stride, hh, n_tokens, hidden_dim, stream)) return rc;
        if (rpx_status_t rc = launch_cast_f32_bf16(static_cast<const float*>(w_vocab), hidden_dim, wh, vocab, hidden_dim, stream)) return rc;
        a.hidden = hh;
        a.hidden_row_stride = hidden_dim;
        a.w = wh;
    }
    a.target_ids = target_ids;
    a.n_tokens = n_tokens;
    a.hidden_dim = hidden_dim;
    a.vocab = vocab;
    a.logprobs = logprobs;
    a.lse = lse;
    a.entropy = entropy;
    a.shard_stats = shard_stats;
    a.target_offset = vocab_begin;
    a.device_status = device_status;
    a.stream = stream;
    return launch_token_logprobs(a);
}

}  // namespace

extern "C" {

rpx_status_t rpx_token_logprobs_entropy(const void* hidden, int64_t hidden_row_stride, const void* w_vocab,
                                        const int32_t* target_ids, int64_t n_tokens, int32_t hidden_dim, int32_t vocab,
                                        rpx_dtype_t dtype, float* logprobs, float* lse, float* entropy, void* workspace,
                                        size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
    return run_token_logprobs(hidden, hidden_row_stride, w_vocab, target_ids, n_tokens, hidden_dim, vocab, 0, dtype,
                              logprobs, lse, entropy, nullptr, workspace, workspace_bytes, device_status, cuda_stream);
}

rpx_status_t rpx_token_logprobs_shard(const void* hidden, int64_t hidden_row_stride, const void* w_shard,
                                      const int32_t* target_ids, int64_t n_tokens, int32_t hidden_dim,
                                      int32_t vocab_local, int32_t vocab_begin, rpx_dtype_t dtype, float* shard_stats,
                                      void* workspace, size_t workspace_bytes, int32_t* device_status,
                                      void* cuda_stream) {
    if (n_tokens > 0 && shard_stats == nullptr) return RPX_ERR_NULL;
    return run_token_logprobs(hidden, hidden_row_stride, w_shard, target_ids, n_tokens, hidden_dim, vocab_local,
                              vocab_begin, dtype, nullptr, nullptr, nullptr, shard_stats, workspace, workspace_bytes,
                              device_status, cuda_stream);
}

rpx_status_t rpx_token_logprobs_merge(const float* shard_stats, int32_t n_shards, const int32_t* target_ids,
                                      int64_t n_tokens, int32_t vocab_total, float* logprobs, float* lse, float* entropy,
                                      int32_t* device_status, void* cuda_stream) {
    if (n_shards <= 0 || n_tokens < 0 || n_tokens >= INT32_MAX || vocab_total <= 0) return RPX_ERR_SHAPE;
    if (n_tokens == 0) return RPX_OK;
    if (shard_stats == nullptr || target_ids == nullptr || logprobs == nullptr) return RPX_ERR_NULL;
    if (!aligned16(shard_stats)) return RPX_ERR_ALIGN;
    if (rpx_status_t rc = check_arch()) return rc;
    return launch_logprob_merge(shard_stats, n_shards, target_ids, n_tokens, vocab_total, logprobs, lse, entropy,
                                device_status, static_cast<cudaStream_t>(cuda_stream));
}

rpx_status_t rpx_token_logprobs(const void* hidden, int64_t hidden_row_stride, const void* w_vocab,
                                const int32_t* target_ids, int64_t n_tokens, int32_t hidden_dim, int32_t vocab,
                                rpx_dtype_t dtype, float* logprobs, float* lse, void* workspace, size_t workspace_bytes,
                                int32_t* device_status, void* cuda_stream) {
    return rpx_token_logprobs_entropy(hidden, hidden_row_stride, w_vocab, target_ids, n_tokens, hidden_dim, vocab, dtype,
                                      logprobs, lse, nullptr, workspace, workspace_bytes, device_status, cuda_stream);
}

size_t rpx_token_logprobs_backward_workspace_bytes(int64_t n_tokens, int32_t hidden_dim, int32_t vocab, rpx_dtype_t dtype) {
    if (n_tokens <= 0 || hidden_dim <= 0 || vocab <= 0 || dtype != RPX_BF16) return 0;
    return align_up(logprob_backward_workspace(n_tokens, vocab), kWsAlign);
}

rpx_status_t rpx_token_logprobs_backward_full(const void* hidden, int64_t hidden_row_stride, const void* w_vocab,
                                              const int32_t* target_ids, const float* lse, const float* upstream,
                                              int64_t n_tokens, int32_t hidden_dim, int32_t vocab, rpx_dtype_t dtype,
                                              void* dhidden, float* dw, int32_t accumulate_dw, void* workspace,
                                              size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
    if (dtype != RPX_BF16 && dtype != RPX_F32) return RPX_ERR_DTYPE;
    if (dtype != RPX_BF16) return RPX_ERR_DTYPE;  // the backward pass takes bf16 tensors only
    if (n_tokens < 0 || n_tokens >= INT32_MAX || hidden_dim <= 0 || vocab <= 0) return RPX_ERR_SHAPE;
    if (hidden_dim % 8 != 0) return RPX_ERR_SHAPE;
    if (n_tokens == 0) return RPX_OK;
    if (hidden == nullptr || w_vocab == nullptr || target_ids == nullptr || lse == nullptr || upstream == nullptr ||
        (dhidden == nullptr && dw == nullptr))
        return RPX_ERR_NULL;
    if (hidden_row_stride < hidden_dim) return RPX_ERR_SHAPE;
    if (hidden_row_stride % 8 != 0) return RPX_ERR_ALIGN;
    if (!aligned16(hidden) || !aligned16(w_vocab) || !aligned16(dhidden) || !aligned16(dw)) return RPX_ERR_ALIGN;
    const size_t need = rpx_token_logprobs_backward_workspace_bytes(n_tokens, hidden_dim, vocab, dtype);
    if (workspace == nullptr || workspace_bytes < need) return RPX_ERR_WORKSPACE;
    if (!aligned_ws(workspace)) return RPX_ERR_ALIGN;
    if (rpx_status_t rc = check_arch()) return rc;
    LogprobBwdArgs a;
    a.hidden = hidden;
    a.hidden_row_stride = hidden_row_stride;
    a.w = w_vocab;
    a.target_ids = target_ids;
    a.lse = lse;
    a.upstream = upstream;
    a.n_tokens = n_tokens;
    a.hidden_dim = hidden_dim;
    a.vocab = vocab;
    a.dhidden = dhidden;
    a.dw = dw;
    a.accumulate_dw = accumulate_dw != 0;
    a.dlogits = workspace;
    a.device_status = device_status;
    a.stream = static_cast<cudaStream_t>(cuda_stream);
    return launch_token_logprobs_backward(a);
}

rpx_status_t rpx_token_logprobs_backward(const void* hidden, int64_t hidden_row_stride, const void* w_vocab,
                                         const int32_t* target_ids, const float* lse, const float* upstream,
                                         int64_t n_tokens, int32_t hidden_dim, int32_t vocab, rpx_dtype_t dtype,
                                         void* dhidden, void* workspace, size_t workspace_bytes, int32_t* device_status,
                                         void* cuda_stream) {
    if (dtype == RPX_BF16 && n_tokens > 0 && hidden_dim > 0 && vocab > 0 && hidden_dim % 8 == 0 && dhidden == nullptr)
        return RPX_ERR_NULL;
    return rpx_token_logprobs_backward_full(hidden, hidden_row_stride, w_vocab, target_ids, lse, upstream, n_tokens,
                                            hidden_dim, vocab, dtype, dhidden, nullptr, 0, workspace, workspace_bytes,
                                            device_status, cuda_stream);
}

size_t rpx_attn_backward_workspace_bytes(const rpx_attn_desc_t* desc, int64_t total_tokens) {
    if (desc == nullptr || total_tokens <= 0 || desc->num_q_heads <= 0) return 0;
    return align_up(static_cast<size_t>(total_tokens) * desc->num_q_heads * sizeof(float), kWsAlign);
}

rpx_status_t rpx_attn_backward(const rpx_attn_desc_t* desc, const void* q, const void* k, const void* v,
                               int64_t q_tok_stride, int64_t k_tok_stride, int64_t v_tok_stride, const void* out,
                               const void* dout, const float* lse, const int32_t* cu_seqlens, const int32_t* q_begin,
                               const int32_t* q_end, int32_t batch, int64_t total_tokens, int32_t max_seqlen, float* dq,
                               float* dk, float* dv, int32_t accumulate_dkv, void* workspace, size_t workspace_bytes,
                               int32_t* device_status, void* cuda_stream) {
    if (rpx_status_t rc = check_attn_desc(desc)) return rc;
    if (desc->dtype != RPX_BF16) return RPX_ERR_DTYPE;  // the backward pass takes bf16 tensors only
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0 || total_tokens >= INT32_MAX) return RPX_ERR_SHAPE;
    if (batch == 0 || total_tokens == 0 || max_seqlen == 0) return RPX_OK;
    if (q == nullptr || k == nullptr || v == nullptr || out == nullptr || dout == nullptr || lse == nullptr ||
        cu_seqlens == nullptr || dq == nullptr || dk == nullptr || dv == nullptr)
        return RPX_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(dout) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv))
        return RPX_ERR_ALIGN;
    const int64_t q_row = static_cast<int64_t>(desc->num_q_heads) * desc->head_dim;
    const int64_t kv_row = static_cast<int64_t>(desc->num_kv_heads) * desc->head_dim;
    if (q_tok_stride < q_row || k_tok_stride < kv_row || v_tok_stride < kv_row) return RPX_ERR_SHAPE;
    if (q_tok_stride % 8 || k_tok_stride % 8 || v_tok_stride % 8) return RPX_ERR_ALIGN;
    const size_t need = rpx_attn_backward_workspace_bytes(desc, total_tokens);
    if (workspace == nullptr || workspace_bytes < need) return RPX_ERR_WORKSPACE;
    if (!aligned_ws(workspace)) return RPX_ERR_ALIGN;
    if (rpx_status_t rc = check_arch()) return rc;
    AttnBwdArgs a;
    a.num_q_heads = desc->num_q_heads;
    a.num_kv_heads = desc->num_kv_heads;
    a.head_dim = desc->head_dim;
    a.softmax_scale = desc->softmax_scale;
    a.q = q;
    a.k = k;
    a.v = v;
    a.q_tok_stride = q_tok_stride;
    a.k_tok_stride = k_tok_stride;
    a.v_tok_stride = v_tok_stride;
    a.out = out;
    a.dout = dout;
    a.lse = lse;
    a.cu_seqlens = cu_seqlens;
    a.q_begin = q_begin;
    a.q_end = q_end;
    a.batch = batch;
    a.total_tokens = total_tokens;
    a.max_seqlen = max_seqlen;
    a.dq = dq;
    a.dk = dk;
    a.dv = dv;
    a.accumulate = accumulate_dkv != 0;
    a.dvec = static_cast<float*>(workspace);
    a.device_status = device_status;
    a.stream = static_cast<cudaStream_t>(cuda_stream);
    return launch_attention_backward(a);
}

rpx_status_t rpx_selftest_bounded_wait(int64_t limit_cycles, int32_t* device_status, void* cuda_stream) {
    if (device_status == nullptr) return RPX_ERR_NULL;
    if (limit_cycles <= 0 || limit_cycles > 2000000000ll) return RPX_ERR_SHAPE;
    if (rpx_status_t rc = check_arch()) return rc;
    return launch_bounded_wait_selftest(limit_cycles, device_status, static_cast<cudaStream_t>(cuda_stream));
}

const char* rpx_status_string(rpx_status_t status) {
    switch (status) {
        case RPX_OK: return "ok";
        case RPX_ERR_NULL: return "a required pointer is NULL";
        case RPX_ERR_SHAPE: return "unsupported or inconsistent sizes";
        case RPX_ERR_DTYPE: return "unknown element type";
        case RPX_ERR_ALIGN: return "pointer or stride alignment";
        case RPX_ERR_WORKSPACE: return "workspace missing or too small";
        case RPX_ERR_ARCH: return "device is not compute capability 10.x (sm_100a kernels only)";
        case RPX_ERR_CUDA: return "a CUDA call failed";
        case RPX_ERR_DEVICE_DATA: return "out-of-range id in device data";
        case RPX_ERR_TIMEOUT: return "a bounded kernel-side wait expired";
        default: return "unknown status";
    }
}

rpx_status_t rpx_set_sm_budget(int32_t sms) {
    if (sms < 0) return RPX_ERR_SHAPE;
    rpx::set_sm_budget(sms);
    return RPX_OK;
}

int32_t rpx_get_sm_budget(void) { return rpx::sm_budget(); }

rpx_status_t rpx_set_lm_head_pairing(int32_t on) {
    rpx::set_lm_head_pairing(on);
    return RPX_OK;
}

int32_t rpx_get_lm_head_pairing(void) { return rpx::lm_head_pairing(); }

int32_t rpx_version(void) { return 100; }

}  // extern "C"
