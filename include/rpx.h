/*
 * rpx — prefix/suffix scoring kernels for NVIDIA B200 (sm_100a), C ABI.
 *
 * The operations follow the paper's statement of the problem (Section 2.3 "Observation and
 * Opportunity"; Section 3.1 Phases 1-2; Table 4, rows "Boundary prefix KV" and "Prefix
 * logprobs"): every model invocation of an RL iteration is split at the first response position
 * into a response-independent PREFIX (the prompt: visual + text tokens) and a response SUFFIX.
 * The prefix pass produces boundary KV state and prefix log-probabilities before the responses
 * exist; the suffix pass consumes the responses together with the retained boundary KV; prefix
 * and suffix log-probabilities together are the full-sequence values.
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers unless marked "host".  Descriptor structs
 *     (rpx_attn_desc_t, rpx_kv_cache_t) are read on the HOST during the call.
 *   - The caller owns every buffer (inputs, outputs, cache pool, block table, workspace, status
 *     word) and must keep it alive until `cuda_stream` has executed the enqueued work.  The
 *     library allocates no device memory, keeps no state between calls (but see
 *     rpx_set_sm_budget) and never synchronises: a call only enqueues kernels, and small
 *     asynchronous memsets of its workspace, on `cuda_stream` (a cudaStream_t passed as void*,
 *     NULL = the legacy default stream) of the current device.
 *   - A workspace belongs to one call at a time: the kernels keep their work-item counters and
 *     partial results there, so two calls that may overlap on the GPU (different streams) need
 *     different workspaces.  Calls on one stream may share one.
 *   - Packed layouts: a [tokens][heads][head_dim] tensor has head_dim contiguous, heads
 *     contiguous (stride head_dim) and a caller-given token stride in ELEMENTS.  Sequence s owns
 *     tokens cu_seqlens[s] .. cu_seqlens[s+1]-1 (int32, device, batch+1 entries, cu_seqlens[0]=0).
 *   - Query head h reads KV head h / (num_q_heads / num_kv_heads).
 *   - Element types: RPX_BF16 tensors are bfloat16.  RPX_F32 tensors are float32 and exist for checking the
 *     method against an unrounded reference, not for throughput: the attention calls then run an fp32 CUDA-core
 *     kernel (q, the call's own k, v and every product stay fp32; out is float32), and the LM-head calls round
 *     hidden and w_vocab to bf16 (nearest-even) in a pre-pass into the workspace before the tensor-core kernel.
 *     The KV cache is always bf16: an RPX_F32 prefix pass stores K and V rounded to nearest-even, and a later
 *     suffix or chunk pass reads those rounded values, as the bf16 path does.
 *   - Host-checkable problems (NULL pointer, head counts, head_dim, block size, alignment,
 *     strides, workspace size, device architecture) return a negative status BEFORE any launch.
 *     Problems only visible on the device (a kernel-side wait that ran out, an out-of-range
 *     target id or block id, sequence offsets that run backwards or past the end of the packed
 *     tensors, a sequence with more pages than a row of the block table) are written to *device_status (nullable, device int32, zeroed by the
 *     caller): the first error code wins; the caller reads it after its own synchronisation.
 *     Every kernel-side wait is bounded: on expiry the kernel records RPX_ERR_TIMEOUT, drains and
 *     returns; outputs of that call are then undefined.
 *   - Alignment: every tensor pointer 16-byte aligned; token/row strides multiples of 8 elements;
 *     every workspace pointer 256-byte aligned (RPX_ERR_ALIGN otherwise, before any launch).
 *   - Zero-length sequences, batch == 0 and n_tokens == 0 are legal no-ops.
 */
#ifndef RPX_H_
#define RPX_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define RPX_API __attribute__((visibility("default")))
#else
#define RPX_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t rpx_status_t;
enum {
    RPX_OK = 0,
    RPX_ERR_NULL = -1,        /* a required pointer is NULL                                  */
    RPX_ERR_SHAPE = -2,       /* unsupported or inconsistent sizes                           */
    RPX_ERR_DTYPE = -3,       /* unknown element type                                        */
    RPX_ERR_ALIGN = -4,       /* pointer or stride alignment                                 */
    RPX_ERR_WORKSPACE = -5,   /* workspace NULL or smaller than *_workspace_bytes            */
    RPX_ERR_ARCH = -6,        /* current device is not compute capability 10.x               */
    RPX_ERR_CUDA = -7,        /* a CUDA runtime/driver call failed                           */
    RPX_ERR_DEVICE_DATA = -8, /* (device_status) out-of-range id found in device data        */
    RPX_ERR_TIMEOUT = -9      /* (device_status) a bounded kernel-side wait expired          */
};

typedef enum { RPX_BF16 = 0, RPX_F32 = 1 } rpx_dtype_t;

/* Attention problem shape.  head_dim is 64 or 128; num_q_heads % num_kv_heads == 0.
 * softmax_scale <= 0 selects 1/sqrt(head_dim).  No bias, soft-cap, window or dropout. */
typedef struct {
    int32_t num_q_heads;
    int32_t num_kv_heads;
    int32_t head_dim;
    float softmax_scale;
    rpx_dtype_t dtype; /* element type of q, k, v and out */
} rpx_attn_desc_t;

/* Paged boundary-KV cache (Table 4, "Boundary prefix KV": produced by the prefix pass, kept in
 * HBM by the caller, consumed by the suffix pass).
 *   k_cache, v_cache : bf16 [num_blocks][num_kv_heads][block_size][head_dim], 16-byte aligned
 *   block_table      : device int32 [batch][block_table_stride]; prefix position t of sequence s
 *                      lives in slot  block_table[s][t / block_size] * block_size + t % block_size
 *   block_size       : must be 16 */
typedef struct {
    void* k_cache;
    void* v_cache;
    int64_t num_blocks;
    int32_t block_size;
    const int32_t* block_table;
    int32_t block_table_stride;
} rpx_kv_cache_t;

/*
 * Prefix attention + boundary-KV write (Section 3.1, Phase 1: the prompt is prefilled before any
 * response exists, which leaves behind the KV state at the prompt/response boundary).  For every
 * sequence s, query head h and prompt position i:
 *     out[i,h,:] = sum_{j<=i} softmax_j(scale * q[i,h,:].k[j,g,:]) * v[j,g,:],   g = h / group
 * and, when `cache` is non-NULL, K and V of every prompt token are stored (as bf16) at the
 * token's slot of the paged cache; slots no token maps to are not touched.
 *   q [total_tokens][num_q_heads][head_dim], k, v [total_tokens][num_kv_heads][head_dim]
 *   out [total_tokens][num_q_heads][head_dim] contiguous, element type desc->dtype
 *   lse (nullable) float32 [total_tokens][num_q_heads]: ln sum_j exp(scale * q.k_j)
 *   max_seqlen: an upper bound on the longest sequence (sizes the grid).  A sequence longer than
 *   the bound rounded up to 256 gets RPX_ERR_DEVICE_DATA in *device_status (its rows beyond the
 *   bound are not computed); the same holds for max_suffix_len / max_chunk_len below.
 */
RPX_API rpx_status_t rpx_prefix_attn(const rpx_attn_desc_t* desc, const void* q, const void* k, const void* v,
                             int64_t q_tok_stride, int64_t k_tok_stride, int64_t v_tok_stride,
                             const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens,
                             int32_t max_seqlen, const rpx_kv_cache_t* cache, void* out, float* lse,
                             void* workspace, size_t workspace_bytes, int32_t* device_status,
                             void* cuda_stream);

/*
 * Suffix attention over the retained boundary (Section 3.1, Phase 2: the suffix pass takes the
 * responses together with the boundary state kept from Phase 1; Section 2.3: the prompt is not
 * computed a second time).  Response position r of sequence s (global
 * position prefix_lens[s] + r) attends to all prefix_lens[s] cached keys and to response keys
 * 0..r; the result equals rows prefix_lens[s].. of one-pass attention over the whole sequence.
 *   q, k, v: response tokens only, packed by cu_seqlens_suffix; prefix_lens device int32 [batch]
 *   cache: required, read-only here (response K/V are NOT appended; they have no later reader)
 *   workspace: rpx_suffix_attn_workspace_bytes includes, for passes of up to 113 664 (token, head) rows,
 *   room for split-KV partials: when the batch is a few long items, the cached prefix of each is cut
 *   into ranges worked on by different SMs and merged by the last to finish (same result up to fp32
 *   rounding of the merge, identical from run to run).
 *   max_suffix_len / max_prefix_len: upper bounds (grid sizing only).
 */
RPX_API rpx_status_t rpx_suffix_attn(const rpx_attn_desc_t* desc, const void* q, const void* k, const void* v,
                             int64_t q_tok_stride, int64_t k_tok_stride, int64_t v_tok_stride,
                             const int32_t* cu_seqlens_suffix, const int32_t* prefix_lens, int32_t batch,
                             int64_t total_suffix_tokens, int32_t max_suffix_len, int32_t max_prefix_len,
                             const rpx_kv_cache_t* cache, void* out, float* lse, void* workspace,
                             size_t workspace_bytes, int32_t* device_status, void* cuda_stream);

/*
 * Chunked prefill of the prefix (an extension: the paper prefills each prompt in one pass and only
 * fixes a per-prompt token budget, Section 4.1).  One call handles the next chunk of every prompt:
 * chunk position i of sequence s (global position cached_lens[s] + i) attends to the cached_lens[s]
 * keys already in the cache and to chunk keys 0..i, exactly as rpx_suffix_attn does, AND the
 * chunk's K and V are appended to the cache at global positions cached_lens[s] + i, exactly as
 * rpx_prefix_attn stores them.  After the last chunk the cache and the concatenated outputs equal
 * those of one rpx_prefix_attn call over the whole prompts.
 *   cached_lens device int32 [batch]: tokens already cached; each must be a multiple of the
 *   block size (chunks start on a page edge) — otherwise nothing is stored for that sequence and
 *   RPX_ERR_DEVICE_DATA appears in *device_status (its attention rows are still computed).
 *   The block table must cover cached_lens[s] + chunk length.  A sequence whose chunk is empty
 *   (cu_seqlens_chunk[s] == cu_seqlens_chunk[s+1]) is skipped whatever its cached_lens.
 *   Other arguments as rpx_suffix_attn; workspace as rpx_suffix_attn_workspace_bytes.
 */
RPX_API rpx_status_t rpx_chunk_attn(const rpx_attn_desc_t* desc, const void* q, const void* k, const void* v,
                            int64_t q_tok_stride, int64_t k_tok_stride, int64_t v_tok_stride,
                            const int32_t* cu_seqlens_chunk, const int32_t* cached_lens, int32_t batch,
                            int64_t total_chunk_tokens, int32_t max_chunk_len, int32_t max_cached_len,
                            const rpx_kv_cache_t* cache, void* out, float* lse, void* workspace,
                            size_t workspace_bytes, int32_t* device_status, void* cuda_stream);

/*
 * Fused LM-head log-probabilities (Section 3.1: Phase 1 yields the log-probabilities of the prefix
 * positions, Phase 2 those of the suffix; Table 4, row on prefix log-probabilities).  For every row n:
 *     z_v = hidden[n,:] . w_vocab[v,:]          (never stored)
 *     logprobs[n] = z_{target_ids[n]} - ln sum_v exp(z_v)
 *   hidden [n_tokens][hidden_dim] with row stride in elements; w_vocab [vocab][hidden_dim]
 *   row-major contiguous; target_ids device int32 [n_tokens]; hidden_dim % 8 == 0.
 *   logprobs float32 [n_tokens]; lse (nullable) float32 [n_tokens].
 * A target outside [0, vocab) gives NaN for that row and RPX_ERR_DEVICE_DATA in *device_status.
 * The kernel is position-agnostic: which (hidden row, next token) pairs form the prefix call and
 * which the suffix call is the caller's choice.
 */
RPX_API rpx_status_t rpx_token_logprobs(const void* hidden, int64_t hidden_row_stride, const void* w_vocab,
                                const int32_t* target_ids, int64_t n_tokens, int32_t hidden_dim,
                                int32_t vocab, rpx_dtype_t dtype, float* logprobs, float* lse,
                                void* workspace, size_t workspace_bytes, int32_t* device_status,
                                void* cuda_stream);

/*
 * rpx_token_logprobs with one more output from the same pass (an extension; the paper only needs
 * the log-probs): entropy[n] = - sum_v p_v ln p_v of the next-token distribution p = softmax(z[n,:]),
 * float32 [n_tokens], nullable.  It costs one more multiply-add per logit in the epilogue and no
 * extra memory traffic; every other argument, the workspace size and the error behaviour are those
 * of rpx_token_logprobs (which is this call with entropy == NULL).
 */
RPX_API rpx_status_t rpx_token_logprobs_entropy(const void* hidden, int64_t hidden_row_stride, const void* w_vocab,
                                                const int32_t* target_ids, int64_t n_tokens, int32_t hidden_dim,
                                                int32_t vocab, rpx_dtype_t dtype, float* logprobs, float* lse,
                                                float* entropy, void* workspace, size_t workspace_bytes,
                                                int32_t* device_status, void* cuda_stream);

/*
 * Vocabulary-parallel LM head (an extension; it is how a tensor-parallel reference model, such as
 * the paper's TP=8 one, lays out its LM head).  Each rank holds the rows vocab_begin ..
 * vocab_begin + vocab_local - 1 of W_vocab and calls rpx_token_logprobs_shard on the full hidden
 * rows; the call leaves one 16-byte record per row in shard_stats (float [n_tokens][4], 16-byte
 * aligned): (running max in log2 units, sum of 2^(x - max), target logit if the target lies in
 * this shard else 0, sum of 2^(x - max) * logit).  The ranks exchange their records (one
 * all-gather of 16 bytes per row and rank) and every rank calls rpx_token_logprobs_merge on the
 * gathered array float [n_shards][n_tokens][4]; the result equals rpx_token_logprobs(_entropy) on
 * the whole vocabulary up to fp32 summation order.  target_ids hold GLOBAL vocabulary ids in both
 * calls; workspace as rpx_token_logprobs_workspace_bytes(n_tokens, hidden_dim, vocab_local, dtype).
 */
RPX_API rpx_status_t rpx_token_logprobs_shard(const void* hidden, int64_t hidden_row_stride, const void* w_shard,
                                              const int32_t* target_ids, int64_t n_tokens, int32_t hidden_dim,
                                              int32_t vocab_local, int32_t vocab_begin, rpx_dtype_t dtype,
                                              float* shard_stats, void* workspace, size_t workspace_bytes,
                                              int32_t* device_status, void* cuda_stream);
RPX_API rpx_status_t rpx_token_logprobs_merge(const float* shard_stats, int32_t n_shards, const int32_t* target_ids,
                                              int64_t n_tokens, int32_t vocab_total, float* logprobs, float* lse,
                                              float* entropy, int32_t* device_status, void* cuda_stream);

/*
 * Backward of rpx_token_logprobs with respect to the hidden states (Section 3.2, the autograd contract of the
 * training actor: its suffix and prefix passes are differentiated, and the gradient reaches the prefix through
 * the retained boundary; Table 4, the row on the training actor's boundary KV, which stays attached).  The LM head is
 * where that gradient starts.  With p = softmax(z[n,:]), z = hidden . w_vocab^T, and the caller's upstream gradient
 * g[n] = dL / d logprobs[n]:
 *     dL/dz[n,v]   = g[n] * ([v == target_ids[n]] - p_v)           (recomputed from lse, one block of rows at a time)
 *     dhidden[n,:] = sum_v dL/dz[n,v] * w_vocab[v,:]
 *   hidden, w_vocab, target_ids: as in the forward call; bf16 only (RPX_F32 returns RPX_ERR_DTYPE)
 *   lse      device float32 [n_tokens]: the forward call's lse output for the same rows
 *   upstream device float32 [n_tokens]
 *   dhidden  bf16 [n_tokens][hidden_dim] contiguous, 16-byte aligned
 *   workspace: rpx_token_logprobs_backward_workspace_bytes; it holds dL/dz of one block of at most 9472 rows as
 *   bf16 (9472 x 152064 x 2 bytes = 2.9 GB for the 152064-column vocabulary), never of the whole batch.
 * A target outside [0, vocab) contributes no one-hot term and sets RPX_ERR_DEVICE_DATA in *device_status.
 *
 * rpx_token_logprobs_backward_full also produces the weight gradient from the same block-wise dL/dz:
 *     dw[v,:] = sum_n dL/dz[n,v] * hidden[n,:]
 *   dhidden  as above, or NULL to skip it
 *   dw       device float32 [vocab][hidden_dim] contiguous, 16-byte aligned, or NULL to skip it (at least one of the
 *            two must be given); accumulate_dw == 0: written, != 0: the call's gradient is ADDED to what dw holds
 *            (gradient accumulation over micro-batches)
 * The contraction runs over the rows, so both operands are read as MN-major tiles straight from the row-major dL/dz
 * block and hidden tensor.  rpx_token_logprobs_backward is the same call with dw == NULL.
 */
RPX_API rpx_status_t rpx_token_logprobs_backward(const void* hidden, int64_t hidden_row_stride, const void* w_vocab,
                                                 const int32_t* target_ids, const float* lse, const float* upstream,
                                                 int64_t n_tokens, int32_t hidden_dim, int32_t vocab, rpx_dtype_t dtype,
                                                 void* dhidden, void* workspace, size_t workspace_bytes,
                                                 int32_t* device_status, void* cuda_stream);
RPX_API rpx_status_t rpx_token_logprobs_backward_full(const void* hidden, int64_t hidden_row_stride, const void* w_vocab,
                                                      const int32_t* target_ids, const float* lse, const float* upstream,
                                                      int64_t n_tokens, int32_t hidden_dim, int32_t vocab,
                                                      rpx_dtype_t dtype, void* dhidden, float* dw, int32_t accumulate_dw,
                                                      void* workspace, size_t workspace_bytes, int32_t* device_status,
                                                      void* cuda_stream);
RPX_API size_t rpx_token_logprobs_backward_workspace_bytes(int64_t n_tokens, int32_t hidden_dim, int32_t vocab,
                                                           rpx_dtype_t dtype);

/*
 * Backward of causal GQA attention over packed whole sequences (Section 3.2: the training actor differentiates both
 * its suffix pass and its prefix pass, and the suffix pass's gradient reaches the prompt through the prefix K/V it
 * attended to; Table 4, the row on the boundary KV that stays attached).  A sequence is prompt followed by response;
 * with P the softmax weights of query row (i, h) over the keys j <= i of its sequence (recomputed from lse), g the KV
 * head of h, dP_ij = dout[i,h,:] . v[j,g,:], D_i = sum_c dout[i,h,c] * out[i,h,c] and dS_ij = P_ij (dP_ij - D_i):
 *     dv[j,g,:] = sum_{h in g} sum_{i >= j} P_ij  dout[i,h,:]
 *     dk[j,g,:] = scale * sum_{h in g} sum_{i >= j} dS_ij q[i,h,:]
 *     dq[i,h,:] = scale * sum_{j <= i} dS_ij k[j,g,:]
 *   q, k, v, strides, cu_seqlens, batch, total_tokens, max_seqlen: as in rpx_prefix_attn; bf16 only (RPX_F32
 *       returns RPX_ERR_DTYPE)
 *   out, dout  device bf16 [total_tokens][num_q_heads][head_dim] contiguous: the forward output and its gradient
 *   lse        device float32 [total_tokens][num_q_heads]: the forward pass's lse (natural log)
 *   q_begin, q_end   nullable device int32 [batch]: only the query rows q_begin[s] <= i < q_end[s] of sequence s take
 *       part (clamped to the sequence; NULL = 0 and the sequence length).  Rows outside get dq = 0 and add nothing
 *       to dk, dv.  With q_begin = prompt length the call is the suffix pass's backward (the gradient of the
 *       response rows with respect to their own K/V and to the prompt's K/V); with q_end = prompt length it is
 *       the prefix pass's.
 *   dq         device float32 [total_tokens][num_q_heads][head_dim], written (rows outside the range: 0)
 *   dk, dv     device float32 [total_tokens][num_kv_heads][head_dim]; accumulate_dkv == 0: written;
 *       != 0: the call's dk, dv are ADDED to what the buffers hold, so that the suffix pass's call followed by the
 *       prefix pass's call leaves the same sums as one call over all rows
 *   workspace: rpx_attn_backward_workspace_bytes (D, 4 bytes per token and query head), 256-byte aligned
 * P and dS are rounded to bf16 before they enter the tensor-core products, as P is in the forward pass.
 * cu_seqlens that leave the packed tensors are not followed and set RPX_ERR_DEVICE_DATA in *device_status; so does a
 * sequence longer than max_seqlen rounded up to 128 (its rows beyond the bound take no part).
 */
RPX_API rpx_status_t rpx_attn_backward(const rpx_attn_desc_t* desc, const void* q, const void* k, const void* v,
                                       int64_t q_tok_stride, int64_t k_tok_stride, int64_t v_tok_stride, const void* out,
                                       const void* dout, const float* lse, const int32_t* cu_seqlens,
                                       const int32_t* q_begin, const int32_t* q_end, int32_t batch, int64_t total_tokens,
                                       int32_t max_seqlen, float* dq, float* dk, float* dv, int32_t accumulate_dkv,
                                       void* workspace, size_t workspace_bytes, int32_t* device_status,
                                       void* cuda_stream);
RPX_API size_t rpx_attn_backward_workspace_bytes(const rpx_attn_desc_t* desc, int64_t total_tokens);

/*
 * Allocation-free variant of rpx_token_logprobs (the paper has no counterpart: this entry point
 * exists for deployment, not for the method).  It is meant for callers that cannot give the
 * library a workspace because they cannot allocate one: a scoring hook that runs inside an
 * engine which has already handed every free byte of HBM to its KV pool (the co-located
 * rollout/training setting), or a section of a serving loop where calling the device allocator is
 * off limits because cudaMalloc may fail there or stall the whole device while it runs.
 *
 * The per-(vocab chunk, row) partial records that rpx_token_logprobs keeps in the caller's
 * workspace live here in a fixed array of RPX_STATIC_SCRATCH_BYTES inside the library image;
 * every GPU that loads the library holds that array until the process exits.  Inputs and outputs
 * are still the caller's.  bf16 inputs only; the result equals that of rpx_token_logprobs up to the order in
 * which fp32 partial sums are merged (this entry point always cuts the vocabulary into 16-tile chunks, the
 * workspace variant into 2 to 16 tiles depending on the row count).
 *   - Limit: ceil(ceil(vocab / 256) / 16) * n_tokens * 16 bytes must not exceed
 *     RPX_STATIC_SCRATCH_BYTES (vocab 152064 => at most 13797 rows per call); larger problems
 *     return RPX_ERR_WORKSPACE before any launch — split the rows over several calls.
 *   - The first call on each device looks up the array's device address (one host-side runtime
 *     query, no allocation).  Make that first call before starting any stream capture.
 *   - Every call on a device shares the one array, which keeps the previous call's contents.
 *     Nothing in it has to start at zero (each call overwrites every record it later reads), but
 *     two calls that overlap on the GPU (different streams, or different threads) race on it:
 *     issue them on one stream or serialise them yourself.
 *   - No cudaMalloc, cudaFree or allocating library routine is called.
 */
#define RPX_STATIC_SCRATCH_BYTES (8u << 20)
RPX_API rpx_status_t rpx_token_logprobs_static(const void* hidden, int64_t hidden_row_stride, const void* w_vocab,
                                               const int32_t* target_ids, int64_t n_tokens, int32_t hidden_dim,
                                               int32_t vocab, float* logprobs, float* lse, int32_t* device_status,
                                               void* cuda_stream);

/* Workspace sizes in bytes for the calls above (pure host arithmetic; 0 is possible). */
RPX_API size_t rpx_prefix_attn_workspace_bytes(const rpx_attn_desc_t* desc, int64_t total_tokens);
RPX_API size_t rpx_suffix_attn_workspace_bytes(const rpx_attn_desc_t* desc, int64_t total_suffix_tokens);
RPX_API size_t rpx_token_logprobs_workspace_bytes(int64_t n_tokens, int32_t hidden_dim, int32_t vocab,
                                          rpx_dtype_t dtype);

/*
 * Self-test of the bounded kernel-side wait every kernel of this library relies on (no counterpart
 * in the paper).  Enqueues a one-CTA kernel in which one thread waits, for at most `limit_cycles`
 * SM cycles (1 .. 2e9), on a barrier that nothing ever signals; the wait must give up, the kernel
 * must return, and RPX_ERR_TIMEOUT must appear in *device_status (device int32, zeroed by the
 * caller).  The CUDA context stays usable: nothing traps, faults or spins without a limit.
 */
RPX_API rpx_status_t rpx_selftest_bounded_wait(int64_t limit_cycles, int32_t* device_status, void* cuda_stream);

/*
 * SM budget for co-running (Section 3.1, Eq. 1).  The overlap model charges the decode side a
 * slowdown Delta_D for sharing the GPU with prefix work; how large it is depends on how much of
 * the GPU the prefix kernels leave free.  The LM-head and attention kernels are persistent (one
 * CTA per SM, all shared memory of the SM), so left alone they leave nothing.  rpx_set_sm_budget(n)
 * caps their grids at n CTAs for every later call of this process (all devices, all streams);
 * 0 removes the cap, n < 0 returns RPX_ERR_SHAPE and changes nothing.  Results do not depend on
 * the budget bit for bit.  Host-only state: no CUDA call, no allocation, nothing set on the GPU.
 */
RPX_API rpx_status_t rpx_set_sm_budget(int32_t sms);
RPX_API int32_t rpx_get_sm_budget(void);

/*
 * Which LM-head kernel later calls of this process use (rpx_token_logprobs, _entropy, _shard, _static): 0 = one
 * CTA per 128 x 256 tile, != 0 = CTA pairs (a cluster of two CTAs per 256 x 256 tile, tcgen05 cta_group::2: each
 * CTA loads its own 128 rows of hidden states and half of the W tile, the even CTA issues the MMAs for both).
 * Results equal each other up to the order of fp32 partial sums (the partial records of a row do not depend on
 * which kernel produced them; the split of the vocabulary into chunks is the same).  Host-only state.
 */
RPX_API rpx_status_t rpx_set_lm_head_pairing(int32_t on);
RPX_API int32_t rpx_get_lm_head_pairing(void);

/* Static string for a status code; never NULL. */
RPX_API const char* rpx_status_string(rpx_status_t status);

/* Library version: major * 10000 + minor * 100 + patch. */
RPX_API int32_t rpx_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RPX_H_ */
