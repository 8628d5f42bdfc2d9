// Backward of the fused LM-head log-probabilities for sm_100a: the gradient with respect to the hidden states.
//
//   dL/dz[n,v]   = g[n] * ([v == target[n]] - exp(z[n,v] - lse[n])),   z = hidden . W_vocab^T  (recomputed, never kept
//                                                                      beyond one block of rows)
//   dhidden[n,:] = sum_v dL/dz[n,v] * W_vocab[v,:]
//
// The rows are taken in blocks (74 row tiles of 128 rows = half a wave of CTAs on each of two output-column tiles).
// Per block two persistent kernels run back to back on the caller's stream:
//   dlogits kernel   the forward kernel's GEMM (hidden x W^T, TMA ring, two TMEM accumulators) with another epilogue:
//                    instead of folding a tile into (max, sum) it turns it into dL/dz with the saved lse and the
//                    upstream gradient and stores it as bf16 into the workspace, [block rows][vocab].
//   dhidden kernel   dlogits x W: the contraction now runs over the vocabulary, so W_vocab [V][H] is the B operand
//                    with its contiguous dimension (H) as N: an MN-major operand taken straight from the row-major
//                    weight, exactly as V is taken in the attention kernel; never transposed, never copied.
// CTAs resident together cover (block row tiles) x (4 output-column tiles) and walk the vocabulary in step, so
// every dlogits and W tile is pulled from HBM once per wave and shared through L2.
//   dW kernel        (optional) dlogits^T x hidden: the contraction runs over the block's rows, so BOTH operands are
//                    MN-major - dlogits [rows][vocab] with the vocabulary as M, hidden [rows][H] with H as N - again
//                    straight from their row-major tensors; 128 vocabulary rows x 256 columns of W's gradient per
//                    tile, written (first block) or added (later blocks) as fp32.
//
// Warp roles as in the forward kernel (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2..5 = epilogue (warp w reads TMEM lanes 32*(w%4) .. +31).
#include <math_constants.h>

#include "rpx_internal.h"
#include "rpx_ptx.cuh"

namespace rpx {

namespace {

constexpr int kBM = 128, kBN = 256, kBK = 64, kStages = 4;
constexpr int kABytes = kBM * kBK * 2, kBBytes = kBN * kBK * 2;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kBlockRowTiles = 74;       // row tiles per block: 74 x (H / 256) items is a whole number of 148-CTA rounds for even H / 256
constexpr int kTilesPerChunk = 8;        // vocabulary tiles one dlogits work item sweeps

struct Ctl {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t drain_flag;
    uint32_t data_error;
};
constexpr size_t kSmemBytes = 1024 + static_cast<size_t>(kStages) * (kABytes + kBBytes) + sizeof(Ctl);

struct Params {
    int64_t n_rows;        // rows of this block
    int32_t vocab;
    int32_t hidden_dim;
    int32_t k_blocks;      // dlogits: ceil(hidden_dim / 64); dhidden: ceil(vocab / 64)
    int32_t n_row_tiles;
    int32_t n_col_tiles;   // dlogits: vocabulary tiles; dhidden: output-column tiles (of hidden_dim)
    int32_t n_chunks;      // dlogits: chunks of kTilesPerChunk vocabulary tiles; dhidden: == n_col_tiles
    int32_t group_width;   // column chunks / tiles in flight side by side
    int32_t total_items;
    const int32_t* target_ids;  // this block's rows
    const float* lse;
    const float* upstream;
    __nv_bfloat16* dlogits;     // [n_rows][dlogits_stride]
    int64_t dlogits_stride;
    __nv_bfloat16* dhidden;     // [n_rows][dhidden_stride]
    int64_t dhidden_stride;
    float* dw;                  // dW kernel: [vocab][hidden_dim]
    int32_t dw_add;             // add to what dw holds (every block after the first, or the caller's request)
    int32_t* status;
};

struct Item {
    int32_t m_tile, chunk;
};

// chunk groups of `group_width` x all row tiles x chunk: the resident CTAs cover many row tiles times a few column
// chunks, so operand tiles are shared through L2 (the forward kernel's order)
__device__ __forceinline__ Item decode_item(const Params& p, int32_t idx) {
    const int32_t per_group = p.n_row_tiles * p.group_width;
    const int32_t cg = idx / per_group;
    const int32_t rem = idx - cg * per_group;
    const int32_t first = cg * p.group_width;
    const int32_t width = min(p.group_width, p.n_chunks - first);
    Item it;
    it.m_tile = rem / width;
    it.chunk = first + rem % width;
    return it;
}

// Four K=16 steps of D (+)= A[smem, K-major] * B[smem, MN-major]: A advances 32 bytes (2 units of 16 bytes) per
// step inside its 128-byte swizzled rows, B advances 16 rows of 128 bytes (128 units).
__device__ __forceinline__ void umma_ss_k64_bmn(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                uint32_t accumulate_first) {
    asm volatile(
        "{\n"
        ".reg .pred pf, pt;\n"
        ".reg .b64 da, db;\n"
        "setp.ne.b32 pf, %4, 0;\n"
        "setp.eq.b32 pt, %4, %4;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pf;\n"
        "add.s64 da, %1, 2;\n"
        "add.s64 db, %2, 128;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, pt;\n"
        "add.s64 da, %1, 4;\n"
        "add.s64 db, %2, 256;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, pt;\n"
        "add.s64 da, %1, 6;\n"
        "add.s64 db, %2, 384;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, pt;\n"
        "}\n" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate_first)
        : "memory");
}

// Four K=16 steps of D (+)= A[smem, MN-major] * B[smem, MN-major]: both advance 16 rows of 128 bytes (128 units).
__device__ __forceinline__ void umma_ss_k64_amn_bmn(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                    uint32_t accumulate_first) {
    asm volatile(
        "{\n"
        ".reg .pred pf, pt;\n"
        ".reg .b64 da, db;\n"
        "setp.ne.b32 pf, %4, 0;\n"
        "setp.eq.b32 pt, %4, %4;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pf;\n"
        "add.s64 da, %1, 128;\n"
        "add.s64 db, %2, 128;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, pt;\n"
        "add.s64 da, %1, 256;\n"
        "add.s64 db, %2, 256;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, pt;\n"
        "add.s64 da, %1, 384;\n"
        "add.s64 db, %2, 384;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, pt;\n"
        "}\n" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate_first)
        : "memory");
}

// kMode 0: the dlogits kernel (A = hidden, B = W K-major over hidden_dim, epilogue = dL/dz to the workspace)
// kMode 1: the dhidden kernel (A = dlogits, B = W MN-major over the vocabulary, epilogue = bf16 tile out)
// kMode 2: the dW kernel      (A = dlogits MN-major with the vocabulary as M, B = hidden MN-major, contraction over
//                              the block's rows, epilogue = fp32 tile of W's gradient, written or added)
template <int kMode>
__global__ void __launch_bounds__(kThreads, 1)
lm_head_bwd_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* smem_a = smem;
    uint8_t* smem_b = smem + kStages * kABytes;
    Ctl* ctl = reinterpret_cast<Ctl*>(smem + kStages * (kABytes + kBBytes));
    volatile uint32_t* abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    constexpr bool kDhidden = kMode == 1, kDw = kMode == 2;
    const int32_t tiles_per_item = kMode == 0 ? kTilesPerChunk : 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&ctl->tmem_full[a], 1);
            mbar_init(&ctl->tmem_empty[a], 128);
        }
        mbar_init(&ctl->drain, 1);
        ctl->abort_flag = 0;
        ctl->drain_flag = 0;
        ctl->data_error = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc(&ctl->tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (one thread)
        if (elect_one()) {
            uint32_t it = 0;
            bool ok = true;
            for (int32_t idx = blockIdx.x; ok && idx < p.total_items; idx += gridDim.x) {
                const Item item = decode_item(p, idx);
                const int32_t t0 = item.chunk * tiles_per_item, t1 = min(t0 + tiles_per_item, p.n_col_tiles);
                for (int32_t t = t0; ok && t < t1; ++t) {
                    for (int32_t kb = 0; kb < p.k_blocks; ++kb, ++it) {
                        const uint32_t stage = it % kStages, phase = (it / kStages) & 1u;
                        if (!mbar_wait(&ctl->empty[stage], phase ^ 1u, abort_flag)) {
                            ok = false;
                            break;
                        }
                        mbar_arrive_expect_tx(&ctl->full[stage], kABytes + kBBytes);
                        if (kDw) {
                            // dlogits [rows][vocab] as {vocab, rows}: two boxes of 64 vocabulary columns x 64 rows
                            for (int i = 0; i < kBM / 64; ++i)
                                tma_load_2d(smem_a + stage * kABytes + i * (kBK * 128), &tmap_a, &ctl->full[stage],
                                            item.m_tile * kBM + i * 64, kb * kBK);
                        } else {
                            tma_load_2d(smem_a + stage * kABytes, &tmap_a, &ctl->full[stage], kb * kBK, item.m_tile * kBM);
                        }
                        if (kDhidden || kDw) {
                            // W [V][H] as {H, V} (dW: hidden [rows][H] as {H, rows}): four boxes of 64 output columns x
                            // 64 rows of the contraction
                            for (int i = 0; i < kBN / 64; ++i)
                                tma_load_2d(smem_b + stage * kBBytes + i * (kBK * 128), &tmap_b, &ctl->full[stage],
                                            t * kBN + i * 64, kb * kBK);
                        } else {
                            tma_load_2d(smem_b + stage * kBBytes, &tmap_b, &ctl->full[stage], kb * kBK, t * kBN);
                        }
                    }
                }
            }
            if (!ok) {
                // abort: let the copies already in flight land before the CTA's smem goes away
                const uint32_t first = it > kStages ? it - kStages : 0u;
                for (uint32_t j = first; j < it; ++j)
                    mbar_wait(&ctl->full[j % kStages], (j / kStages) & 1u, &ctl->drain_flag, kDrainLimitCycles);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (one thread)
        if (elect_one()) {
            constexpr uint32_t idesc = make_idesc_bf16(kBM, kBN, kDw, kDhidden || kDw);
            // MN-major operands: 64-element blocks of M (or N) lie kBK rows of 128 bytes apart
            const uint64_t a_desc0 = make_smem_desc_sw128(smem_u32(smem_a), kDw ? kBK * 128 : 16, 1024);
            const uint64_t b_desc0 = make_smem_desc_sw128(smem_u32(smem_b), (kDhidden || kDw) ? kBK * 128 : 16, 1024);
            uint32_t it = 0, tile_count = 0;
            bool ok = true;
            for (int32_t idx = blockIdx.x; ok && idx < p.total_items; idx += gridDim.x) {
                const Item item = decode_item(p, idx);
                const int32_t t0 = item.chunk * tiles_per_item, t1 = min(t0 + tiles_per_item, p.n_col_tiles);
                for (int32_t t = t0; ok && t < t1; ++t, ++tile_count) {
                    const uint32_t acc = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
                    if (!mbar_wait(&ctl->tmem_empty[acc], acc_phase ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + acc * kBN;
                    for (int32_t kb = 0; kb < p.k_blocks; ++kb, ++it) {
                        const uint32_t stage = it % kStages, phase = (it / kStages) & 1u;
                        if (!mbar_wait(&ctl->full[stage], phase, abort_flag)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        const uint64_t ad = a_desc0 + static_cast<uint64_t>(stage * (kABytes >> 4));
                        const uint64_t bd = b_desc0 + static_cast<uint64_t>(stage * (kBBytes >> 4));
                        if (kDw) umma_ss_k64_amn_bmn(d_tmem, ad, bd, idesc, kb != 0 ? 1u : 0u);
                        else if (kDhidden) umma_ss_k64_bmn(d_tmem, ad, bd, idesc, kb != 0 ? 1u : 0u);
                        else umma_ss_k64(d_tmem, ad, bd, idesc, kb != 0 ? 1u : 0u);
                        umma_commit(&ctl->empty[stage]);
                    }
                    if (ok) umma_commit(&ctl->tmem_full[acc]);
                }
            }
            if (!ok) {
                umma_commit(&ctl->drain);
                mbar_wait(&ctl->drain, 0, &ctl->drain_flag, kDrainLimitCycles);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue (128 threads, thread = row)
        const uint32_t quarter = warp & 3;
        const int32_t row_in_tile = quarter * 32 + lane;
        const uint32_t lane_addr = (quarter * 32u) << 16;
        uint32_t tile_count = 0;
        bool ok = true;
        for (int32_t idx = blockIdx.x; ok && idx < p.total_items; idx += gridDim.x) {
            const Item item = decode_item(p, idx);
            const int64_t row = static_cast<int64_t>(item.m_tile) * kBM + row_in_tile;
            const bool valid = kDw ? row < p.vocab : row < p.n_rows;  // dW: the tile's rows are vocabulary rows
            int32_t target = -1;
            float lse2 = 0.f, g = 0.f;
            if (kMode == 0 && valid) {
                target = __ldg(p.target_ids + row);
                if (target < 0 || target >= p.vocab) {
                    ctl->data_error = 1;  // no one-hot term for such a row (its log-prob is NaN in the forward pass)
                    target = -1;
                }
                lse2 = __ldg(p.lse + row) * kLog2e;
                g = __ldg(p.upstream + row);
            }
            const int32_t t0 = item.chunk * tiles_per_item, t1 = min(t0 + tiles_per_item, p.n_col_tiles);
            for (int32_t t = t0; ok && t < t1; ++t, ++tile_count) {
                const uint32_t acc = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
                if (!mbar_wait(&ctl->tmem_full[acc], acc_phase, abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const int32_t n0 = t * kBN;
                const int32_t n_cols = kMode == 0 ? p.vocab : p.hidden_dim;
                __nv_bfloat16* dst_row = kDhidden ? p.dhidden + row * p.dhidden_stride : p.dlogits + row * p.dlogits_stride;
#pragma unroll 1
                for (int c = 0; c < kBN / 32; ++c) {
                    const int32_t col0 = n0 + c * 32;
                    if (col0 >= n_cols) break;
                    uint32_t r[32];
                    tmem_ld32(tmem_base + acc * kBN + c * 32 + lane_addr, r);
                    tmem_ld_wait();
                    if (kDw) {
                        // fp32 tile of W's gradient; hidden_dim is a multiple of 8, so whole groups of 4 columns
                        if (valid) {
                            float* dst = p.dw + row * p.hidden_dim + col0;
#pragma unroll
                            for (int i = 0; i < 32; i += 4) {
                                if (col0 + i < n_cols) {
                                    float4 v = make_float4(__uint_as_float(r[i]), __uint_as_float(r[i + 1]),
                                                           __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
                                    float4* q4 = reinterpret_cast<float4*>(dst + i);
                                    if (p.dw_add != 0) {
                                        const float4 old = *q4;
                                        v.x += old.x;
                                        v.y += old.y;
                                        v.z += old.z;
                                        v.w += old.w;
                                    }
                                    *q4 = v;
                                }
                            }
                        }
                        continue;
                    }
                    uint32_t w[16];
                    if (kDhidden) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) w[i] = pack_bf16x2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                    } else {
                        // dL/dz = g * (onehot - p), p = 2^(z * log2 e - lse * log2 e)
                        float d[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) d[i] = -g * fast_exp2(fmaf(__uint_as_float(r[i]), kLog2e, -lse2));
                        const uint32_t tl = static_cast<uint32_t>(target - col0);
                        if (tl < 32u) {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (tl == static_cast<uint32_t>(i)) d[i] += g;
                        }
#pragma unroll
                        for (int i = 0; i < 16; ++i) w[i] = pack_bf16x2(d[2 * i], d[2 * i + 1]);
                    }
                    if (valid) {
                        __nv_bfloat16* dst = dst_row + col0;
                        if (col0 + 32 <= n_cols && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0u) {
                            st_global_v8(dst, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
                            st_global_v8(dst + 16, w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]);
                        } else {
                            // the ragged last columns (the column count is a multiple of 8 for dhidden, anything for the vocabulary)
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                if (col0 + 2 * i < n_cols) dst[2 * i] = __ushort_as_bfloat16(static_cast<unsigned short>(w[i] & 0xffffu));
                                if (col0 + 2 * i + 1 < n_cols) dst[2 * i + 1] = __ushort_as_bfloat16(static_cast<unsigned short>(w[i] >> 16));
                            }
                        }
                    }
                }
                tc_fence_before_sync();
                mbar_arrive(&ctl->tmem_empty[acc]);
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && p.status != nullptr) {
        if (ctl->abort_flag != 0u) atomicCAS(p.status, 0, RPX_ERR_TIMEOUT);
        else if (ctl->data_error != 0u) atomicCAS(p.status, 0, RPX_ERR_DEVICE_DATA);
    }
}

int64_t dlogits_stride_of(int32_t vocab) { return (static_cast<int64_t>(vocab) + 63) / 64 * 64; }

}  // namespace

int64_t logprob_backward_block_rows(int64_t n_tokens) {
    const int64_t cap = static_cast<int64_t>(kBlockRowTiles) * kBM;
    return n_tokens < cap ? n_tokens : cap;
}

size_t logprob_backward_workspace(int64_t n_tokens, int32_t vocab) {
    if (n_tokens <= 0 || vocab <= 0) return 0;
    return static_cast<size_t>(logprob_backward_block_rows(n_tokens)) * static_cast<size_t>(dlogits_stride_of(vocab)) * 2;
}

rpx_status_t launch_token_logprobs_backward(const LogprobBwdArgs& a) {
    if (a.n_tokens == 0) return RPX_OK;
    int sms = sm_count();
    if (sms <= 0) return RPX_ERR_CUDA;
    if (const int budget = sm_budget(); budget > 0 && budget < sms) sms = budget;  // leave the rest to a co-runner
    if (cudaFuncSetAttribute(lm_head_bwd_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(kSmemBytes)) != cudaSuccess ||
        cudaFuncSetAttribute(lm_head_bwd_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(kSmemBytes)) != cudaSuccess ||
        cudaFuncSetAttribute(lm_head_bwd_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(kSmemBytes)) != cudaSuccess)
        return RPX_ERR_CUDA;
    const int64_t block_rows = logprob_backward_block_rows(a.n_tokens);
    const int64_t dl_stride = dlogits_stride_of(a.vocab);
    auto* dlogits = static_cast<__nv_bfloat16*>(a.dlogits);
    auto* hidden = static_cast<const __nv_bfloat16*>(a.hidden);
    auto* dhidden = static_cast<__nv_bfloat16*>(a.dhidden);

    CUtensorMap tmap_w_k, tmap_w_mn;
    {   // W as the K-major B operand of hidden x W^T: {hidden_dim, vocab}, box 64 x 256
        const uint64_t dims[2] = {static_cast<uint64_t>(a.hidden_dim), static_cast<uint64_t>(a.vocab)};
        const uint64_t strides[1] = {static_cast<uint64_t>(a.hidden_dim) * 2};
        const uint32_t box_k[2] = {kBK, kBN};
        if (rpx_status_t rc = encode_tmap_bf16(&tmap_w_k, a.w, 2, dims, strides, box_k)) return rc;
        // and as the MN-major B operand of dlogits x W: the same view, box 64 output columns x 64 vocabulary rows
        const uint32_t box_mn[2] = {64, kBK};
        if (rpx_status_t rc = encode_tmap_bf16(&tmap_w_mn, a.w, 2, dims, strides, box_mn)) return rc;
    }
    for (int64_t r0 = 0; r0 < a.n_tokens; r0 += block_rows) {
        const int64_t rows = a.n_tokens - r0 < block_rows ? a.n_tokens - r0 : block_rows;
        CUtensorMap tmap_h, tmap_dl, tmap_h_mn, tmap_dl_mn;
        {
            const uint64_t dims[2] = {static_cast<uint64_t>(a.hidden_dim), static_cast<uint64_t>(rows)};
            const uint64_t strides[1] = {static_cast<uint64_t>(a.hidden_row_stride) * 2};
            const uint32_t box[2] = {kBK, kBM};
            if (rpx_status_t rc = encode_tmap_bf16(&tmap_h, hidden + r0 * a.hidden_row_stride, 2, dims, strides, box)) return rc;
        }
        {
            const uint64_t dims[2] = {static_cast<uint64_t>(a.vocab), static_cast<uint64_t>(rows)};
            const uint64_t strides[1] = {static_cast<uint64_t>(dl_stride) * 2};
            const uint32_t box[2] = {kBK, kBM};
            if (rpx_status_t rc = encode_tmap_bf16(&tmap_dl, dlogits, 2, dims, strides, box)) return rc;
        }
        if (a.dw != nullptr) {
            // the dW kernel's views: boxes of 64 contiguous elements (vocabulary columns of dlogits, columns of hidden)
            // x 64 rows of the block; rows beyond the block read as zero
            const uint32_t box[2] = {64, kBK};
            const uint64_t hdims[2] = {static_cast<uint64_t>(a.hidden_dim), static_cast<uint64_t>(rows)};
            const uint64_t hstrides[1] = {static_cast<uint64_t>(a.hidden_row_stride) * 2};
            if (rpx_status_t rc = encode_tmap_bf16(&tmap_h_mn, hidden + r0 * a.hidden_row_stride, 2, hdims, hstrides, box)) return rc;
            const uint64_t ddims[2] = {static_cast<uint64_t>(a.vocab), static_cast<uint64_t>(rows)};
            const uint64_t dstrides[1] = {static_cast<uint64_t>(dl_stride) * 2};
            if (rpx_status_t rc = encode_tmap_bf16(&tmap_dl_mn, dlogits, 2, ddims, dstrides, box)) return rc;
        }
        Params p;
        p.dw = a.dw;
        p.dw_add = (a.accumulate_dw || r0 > 0) ? 1 : 0;
        p.n_rows = rows;
        p.vocab = a.vocab;
        p.hidden_dim = a.hidden_dim;
        p.n_row_tiles = static_cast<int32_t>((rows + kBM - 1) / kBM);
        p.target_ids = a.target_ids + r0;
        p.lse = a.lse + r0;
        p.upstream = a.upstream + r0;
        p.dlogits = dlogits;
        p.dlogits_stride = dl_stride;
        p.dhidden = dhidden + r0 * a.hidden_dim;
        p.dhidden_stride = a.hidden_dim;
        p.status = a.device_status;
        // ---- dL/dz of the block
        p.k_blocks = (a.hidden_dim + kBK - 1) / kBK;
        p.n_col_tiles = (a.vocab + kBN - 1) / kBN;
        p.n_chunks = (p.n_col_tiles + kTilesPerChunk - 1) / kTilesPerChunk;
        int64_t total = static_cast<int64_t>(p.n_row_tiles) * p.n_chunks;
        if (total > INT32_MAX) return RPX_ERR_SHAPE;
        p.total_items = static_cast<int32_t>(total);
        int grid = static_cast<int>(total < sms ? total : sms);
        p.group_width = grid % 4 == 0 ? 4 : (grid % 2 == 0 ? 2 : 1);
        lm_head_bwd_kernel<0><<<grid, kThreads, kSmemBytes, a.stream>>>(tmap_h, tmap_w_k, p);
        if (cudaGetLastError() != cudaSuccess) return RPX_ERR_CUDA;
        // ---- dhidden of the block
        if (a.dhidden != nullptr) {
            p.k_blocks = (a.vocab + kBK - 1) / kBK;
            p.n_col_tiles = (a.hidden_dim + kBN - 1) / kBN;
            p.n_chunks = p.n_col_tiles;
            total = static_cast<int64_t>(p.n_row_tiles) * p.n_chunks;
            p.total_items = static_cast<int32_t>(total);
            grid = static_cast<int>(total < sms ? total : sms);
            p.group_width = p.n_col_tiles % 4 == 0 ? 4 : (p.n_col_tiles % 2 == 0 ? 2 : 1);
            lm_head_bwd_kernel<1><<<grid, kThreads, kSmemBytes, a.stream>>>(tmap_dl, tmap_w_mn, p);
            if (cudaGetLastError() != cudaSuccess) return RPX_ERR_CUDA;
        }
        // ---- this block's share of dW: the work list runs over (128 vocabulary rows) x (256 columns of hidden_dim),
        // all column tiles of a vocabulary tile side by side, so a dlogits slice is pulled from HBM once
        if (a.dw != nullptr) {
            p.k_blocks = static_cast<int32_t>((rows + kBK - 1) / kBK);
            p.n_row_tiles = (a.vocab + kBM - 1) / kBM;
            p.n_col_tiles = (a.hidden_dim + kBN - 1) / kBN;
            p.n_chunks = p.n_col_tiles;
            total = static_cast<int64_t>(p.n_row_tiles) * p.n_chunks;
            if (total > INT32_MAX) return RPX_ERR_SHAPE;
            p.total_items = static_cast<int32_t>(total);
            grid = static_cast<int>(total < sms ? total : sms);
            p.group_width = p.n_col_tiles <= 20 ? p.n_col_tiles : 16;
            lm_head_bwd_kernel<2><<<grid, kThreads, kSmemBytes, a.stream>>>(tmap_dl_mn, tmap_h_mn, p);
            if (cudaGetLastError() != cudaSuccess) return RPX_ERR_CUDA;
        }
    }
    return RPX_OK;
}

}  // namespace rpx
