// RPX_F32 attention: fp32 arithmetic end to end on the CUDA cores.
//
// The fp32 element type exists for checking the method against an unrounded reference, not for throughput: a
// bf16 tensor-core pass over rounded copies of q, k, v cannot hold 1e-2 against fp32 inputs (the rounding of
// K moves the scores, that of V the output).  So this path keeps q, the self K/V and every product in fp32 and only
// the paged cache - which is bf16 by contract - carries rounded values, exactly as the bf16 path writes them.
//
// One warp per (query row, query head).  Its lanes split head_dim (lane l owns the columns l, l + 32, ...), so every
// K and V row is read with coalesced 128-byte requests; a score is a warp-wide sum, the softmax is the usual online
// one in log2 units.  Keys come first from the paged cache (the cached prefix of a suffix or chunk pass, through the
// block table), then from the call's own k, v up to the row itself.  The warp of the first query head of a KV group
// also stores its token's K and V in the cache when the pass writes one.
#include <math_constants.h>

#include "rpx_internal.h"

namespace rpx {

namespace {

constexpr int kPage = 16;
constexpr int kRowsPerCta = 4;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct Params {
    const float *q, *k, *v;
    int64_t q_tok_stride, k_tok_stride, v_tok_stride;
    const int32_t* cu_seqlens;
    const int32_t* prefix_lens;  // nullable
    int32_t batch, num_q_heads, num_kv_heads, group;
    int64_t total_tokens;
    int32_t row_bound;           // query rows per sequence the grid covers
    __nv_bfloat16* k_cache;      // nullable: [num_blocks][H_kv][16][d]
    __nv_bfloat16* v_cache;
    const int32_t* block_table;
    int32_t block_table_stride;
    int32_t num_blocks;
    int32_t write_cache;         // store this call's K/V behind the cached prefix
    float scale_log2;
    float* out;                  // [tokens][H_q][d]
    float* lse;                  // nullable
    int32_t* status;
};

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
}

template <int D>
__global__ void __launch_bounds__(kRowsPerCta * 32) attn_f32_kernel(const Params p) {
    constexpr int U = D / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int32_t seq = blockIdx.y, head = blockIdx.z;
    const int32_t i = blockIdx.x * kRowsPerCta + warp;  // query row within the sequence
    const int32_t kv_head = head / p.group;
    const int32_t tok0 = __ldg(p.cu_seqlens + seq);
    const int32_t len_q = __ldg(p.cu_seqlens + seq + 1) - tok0;
    const int32_t len_p = p.prefix_lens != nullptr ? __ldg(p.prefix_lens + seq) : 0;
    // the same checks as the tensor-core path: offsets that leave the packed tensors, more pages than a row of the
    // block table, a sequence longer than the caller's bound, an append that does not start on a page edge
    const int64_t table_tokens = static_cast<int64_t>(len_p) + (p.write_cache != 0 ? len_q : 0);
    bool bad = tok0 < 0 || len_q < 0 || static_cast<int64_t>(tok0) + len_q > p.total_tokens || len_p < 0 ||
               (p.block_table != nullptr && (table_tokens + kPage - 1) / kPage > p.block_table_stride);
    bool flag = bad || (!bad && len_q > p.row_bound);
    const bool write = p.write_cache != 0 && !bad && (len_p % kPage) == 0;
    if (p.write_cache != 0 && !bad && (len_p % kPage) != 0) flag = true;
    if (bad || i >= len_q) {
        if (flag && threadIdx.x == 0 && blockIdx.x == 0 && head == 0 && p.status != nullptr)
            atomicCAS(p.status, 0, RPX_ERR_DEVICE_DATA);
        return;
    }
    if (flag && threadIdx.x == 0 && blockIdx.x == 0 && head == 0 && p.status != nullptr)
        atomicCAS(p.status, 0, RPX_ERR_DEVICE_DATA);

    const int64_t tok = static_cast<int64_t>(tok0) + i;
    float qv[U], acc[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        qv[u] = __ldg(p.q + tok * p.q_tok_stride + static_cast<int64_t>(head) * D + u * 32 + lane) * p.scale_log2;
        acc[u] = 0.f;
    }
    float m = -CUDART_INF_F, l = 0.f;
    auto step = [&](const float (&kr)[U], const float (&vr)[U]) {
        float s = 0.f;
#pragma unroll
        for (int u = 0; u < U; ++u) s = fmaf(qv[u], kr[u], s);
        s = warp_sum(s);
        const float m_new = fmaxf(m, s);
        const float corr = exp2f(m - m_new), pj = exp2f(s - m_new);
        l = fmaf(l, corr, pj);
#pragma unroll
        for (int u = 0; u < U; ++u) acc[u] = fmaf(acc[u], corr, pj * vr[u]);
        m = m_new;
    };
    // ---- the cached prefix (bf16, paged)
    bool bad_block = false;
    for (int32_t j = 0; j < len_p; ++j) {
        const int32_t block = __ldg(p.block_table + static_cast<int64_t>(seq) * p.block_table_stride + j / kPage);
        if (block < 0 || block >= p.num_blocks) {
            bad_block = true;
            continue;
        }
        const int64_t row = ((static_cast<int64_t>(block) * p.num_kv_heads + kv_head) * kPage + j % kPage) * D;
        float kr[U], vr[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            kr[u] = __bfloat162float(p.k_cache[row + u * 32 + lane]);
            vr[u] = __bfloat162float(p.v_cache[row + u * 32 + lane]);
        }
        step(kr, vr);
    }
    // ---- the call's own keys, causal
    for (int32_t j = 0; j <= i; ++j) {
        const int64_t t = static_cast<int64_t>(tok0) + j;
        float kr[U], vr[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            kr[u] = __ldg(p.k + t * p.k_tok_stride + static_cast<int64_t>(kv_head) * D + u * 32 + lane);
            vr[u] = __ldg(p.v + t * p.v_tok_stride + static_cast<int64_t>(kv_head) * D + u * 32 + lane);
        }
        step(kr, vr);
    }
    const float inv = 1.f / l;
#pragma unroll
    for (int u = 0; u < U; ++u) p.out[(tok * p.num_q_heads + head) * D + u * 32 + lane] = acc[u] * inv;
    if (p.lse != nullptr && lane == 0) p.lse[tok * p.num_q_heads + head] = (m + log2f(l)) * kLn2;
    // ---- this token's K, V into the cache (once per KV head)
    if (write && head % p.group == 0) {
        const int32_t pos = len_p + i;
        const int32_t block = __ldg(p.block_table + static_cast<int64_t>(seq) * p.block_table_stride + pos / kPage);
        if (block < 0 || block >= p.num_blocks) {
            bad_block = true;
        } else {
            const int64_t row = ((static_cast<int64_t>(block) * p.num_kv_heads + kv_head) * kPage + pos % kPage) * D;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                p.k_cache[row + u * 32 + lane] =
                    __float2bfloat16_rn(__ldg(p.k + tok * p.k_tok_stride + static_cast<int64_t>(kv_head) * D + u * 32 + lane));
                p.v_cache[row + u * 32 + lane] =
                    __float2bfloat16_rn(__ldg(p.v + tok * p.v_tok_stride + static_cast<int64_t>(kv_head) * D + u * 32 + lane));
            }
        }
    }
    if (bad_block && lane == 0 && p.status != nullptr) atomicCAS(p.status, 0, RPX_ERR_DEVICE_DATA);
}

}  // namespace

rpx_status_t launch_attention_f32(const AttnArgs& a) {
    if (a.batch == 0 || a.total_tokens == 0 || a.max_q_len == 0) return RPX_OK;
    Params p;
    p.q = static_cast<const float*>(a.q);
    p.k = static_cast<const float*>(a.k);
    p.v = static_cast<const float*>(a.v);
    p.q_tok_stride = a.q_tok_stride;
    p.k_tok_stride = a.k_tok_stride;
    p.v_tok_stride = a.v_tok_stride;
    p.cu_seqlens = a.cu_seqlens;
    p.prefix_lens = a.prefix_lens;
    p.batch = a.batch;
    p.num_q_heads = a.num_q_heads;
    p.num_kv_heads = a.num_kv_heads;
    p.group = a.num_q_heads / a.num_kv_heads;
    p.total_tokens = a.total_tokens;
    p.row_bound = (a.max_q_len + 255) / 256 * 256;  // the bf16 path's bound: whole pairs of 128-row tiles
    p.k_cache = a.cache != nullptr ? static_cast<__nv_bfloat16*>(a.cache->k_cache) : nullptr;
    p.v_cache = a.cache != nullptr ? static_cast<__nv_bfloat16*>(a.cache->v_cache) : nullptr;
    p.block_table = a.cache != nullptr ? a.cache->block_table : nullptr;
    p.block_table_stride = a.cache != nullptr ? a.cache->block_table_stride : 0;
    p.num_blocks = a.cache != nullptr ? static_cast<int32_t>(a.cache->num_blocks) : 0;
    // the prefix pass writes its tokens from position 0; chunked prefill appends behind the cached chunks
    p.write_cache = a.cache != nullptr && (a.prefix_lens == nullptr || a.append_cache) ? 1 : 0;
    const float scale = a.softmax_scale > 0.f ? a.softmax_scale : 1.0f / sqrtf(static_cast<float>(a.head_dim));
    p.scale_log2 = scale * kLog2e;
    p.out = static_cast<float*>(a.out);
    p.lse = a.lse;
    p.status = a.device_status;
    if (a.batch > 65535 || a.num_q_heads > 65535) return RPX_ERR_SHAPE;
    const dim3 grid((p.row_bound + kRowsPerCta - 1) / kRowsPerCta, a.batch, a.num_q_heads);
    if (a.head_dim == 128)
        attn_f32_kernel<128><<<grid, kRowsPerCta * 32, 0, a.stream>>>(p);
    else if (a.head_dim == 64)
        attn_f32_kernel<64><<<grid, kRowsPerCta * 32, 0, a.stream>>>(p);
    else
        return RPX_ERR_SHAPE;
    return cudaGetLastError() == cudaSuccess ? RPX_OK : RPX_ERR_CUDA;
}

}  // namespace rpx
