// Fused LM-head log-probabilities for sm_100a.
//
//   logprob[n] = z[n, target[n]] - ln sum_v exp(z[n, v]),   z = hidden . W_vocab^T  (never stored)
//
// One persistent CTA per SM.  A work item is (row tile of 128 rows, chunk of 16 (4 for small, 8 for very
// large row counts) vocab tiles of 256 columns): the CTA sweeps the chunk tile by tile; each tile is a TMA-fed tcgen05
// GEMM over the hidden dimension into one of two 128x256 fp32 TMEM accumulators, and while the
// tensor core fills one accumulator the four epilogue warps fold the other into a running
// (max, sum-exp, target-logit) per row.  One partial per (chunk, row) goes to the workspace; a
// small second kernel merges the partials.  Items are ordered so that the CTAs resident at any
// moment cover a few vocab chunks times many row tiles: every W tile is pulled from HBM once per
// wave and shared through L2, and the wave's hidden rows stay L2-resident across the chunk.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2..5 = epilogue (warp w reads TMEM lanes 32*(w%4) .. +31).
#include <math_constants.h>

#include <mutex>

#include "rpx_internal.h"
#include "rpx_ptx.cuh"

namespace rpx {

namespace {

constexpr int kBM = 128, kBN = 256, kBK = 64, kStages = 4;
constexpr int kTilesPerChunkLarge = 16;  // many row tiles: long items, few partial records
constexpr int kTilesPerChunkSmall = 4;   // few row tiles: short items, so the last wave is short too
constexpr int kTilesPerChunkHuge = 8;    // very many row tiles: there are enough items per CTA that halving
                                         // them costs nothing and evens out the last wave (measured +1 %)
constexpr int kSmallRowTiles = 64;
constexpr int kHugeRowTiles = 192;
constexpr int kABytes = kBM * kBK * 2, kBBytes = kBN * kBK * 2;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct Ctl {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t drain_flag;
};
constexpr size_t kSmemBytes = 1024 + static_cast<size_t>(kStages) * (kABytes + kBBytes) + sizeof(Ctl);

struct Params {
    int64_t n_rows;
    int32_t vocab;
    int32_t k_blocks;      // ceil(hidden_dim / 64)
    int32_t n_row_tiles;
    int32_t n_vocab_tiles;
    int32_t n_chunks;
    int32_t tiles_per_chunk;
    int32_t group_width;   // vocab chunks in flight side by side
    int32_t total_items;
    const int32_t* target_ids;
    int32_t target_offset; // first vocabulary column of this W (0 unless W is one shard of the vocabulary)
    float4* partials;      // [n_chunks][n_rows]: (max in log2 units, sum of 2^(x-max), target logit,
                           //                      sum of 2^(x-max) * z  -- for the entropy)
    int32_t* status;
};

struct Item {
    int32_t m_tile, chunk, tile_begin, tile_end;
};

__device__ __forceinline__ Item decode_item(const Params& p, int32_t idx) {
    const int32_t per_group = p.n_row_tiles * p.group_width;
    const int32_t cg = idx / per_group;
    const int32_t rem = idx - cg * per_group;
    const int32_t first = cg * p.group_width;
    const int32_t width = min(p.group_width, p.n_chunks - first);
    Item it;
    it.m_tile = rem / width;
    it.chunk = first + rem % width;
    it.tile_begin = it.chunk * p.tiles_per_chunk;
    it.tile_end = min(it.tile_begin + p.tiles_per_chunk, p.n_vocab_tiles);
    return it;
}

__global__ void __launch_bounds__(kThreads, 1)
lm_head_partial_kernel(const __grid_constant__ CUtensorMap tmap_hidden, const __grid_constant__ CUtensorMap tmap_w,
                       const Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* smem_a = smem;
    uint8_t* smem_b = smem + kStages * kABytes;
    Ctl* ctl = reinterpret_cast<Ctl*>(smem + kStages * (kABytes + kBBytes));
    volatile uint32_t* abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

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
        fence_barrier_init();
        tma_prefetch_desc(&tmap_hidden);
        tma_prefetch_desc(&tmap_w);
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
                for (int32_t t = item.tile_begin; ok && t < item.tile_end; ++t) {
                    for (int32_t kb = 0; kb < p.k_blocks; ++kb, ++it) {
                        const uint32_t stage = it % kStages, phase = (it / kStages) & 1u;
                        if (!mbar_wait(&ctl->empty[stage], phase ^ 1u, abort_flag)) {
                            ok = false;
                            break;
                        }
                        mbar_arrive_expect_tx(&ctl->full[stage], kABytes + kBBytes);
                        tma_load_2d(smem_a + stage * kABytes, &tmap_hidden, &ctl->full[stage], kb * kBK,
                                    item.m_tile * kBM);
                        tma_load_2d(smem_b + stage * kBBytes, &tmap_w, &ctl->full[stage], kb * kBK, t * kBN);
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
            constexpr uint32_t idesc = make_idesc_bf16(kBM, kBN, false, false);
            const uint64_t a_desc0 = make_smem_desc_sw128(smem_u32(smem_a), 16, 1024);
            const uint64_t b_desc0 = make_smem_desc_sw128(smem_u32(smem_b), 16, 1024);
            uint32_t it = 0, tile_count = 0;
            bool ok = true;
            for (int32_t idx = blockIdx.x; ok && idx < p.total_items; idx += gridDim.x) {
                const Item item = decode_item(p, idx);
                for (int32_t t = item.tile_begin; ok && t < item.tile_end; ++t, ++tile_count) {
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
                        umma_ss_k64(d_tmem, a_desc0 + static_cast<uint64_t>(stage * (kABytes >> 4)),
                                    b_desc0 + static_cast<uint64_t>(stage * (kBBytes >> 4)), idesc, kb != 0 ? 1u : 0u);
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
        // ------------------------------------------------------------ epilogue (128 threads)
        const uint32_t quarter = warp & 3;
        const int32_t row_in_tile = quarter * 32 + lane;
        const uint32_t lane_addr = (quarter * 32u) << 16;
        uint32_t tile_count = 0;
        bool ok = true;
        for (int32_t idx = blockIdx.x; ok && idx < p.total_items; idx += gridDim.x) {
            const Item item = decode_item(p, idx);
            const int64_t row = static_cast<int64_t>(item.m_tile) * kBM + row_in_tile;
            const bool valid = row < p.n_rows;
            const int32_t target = valid ? __ldg(p.target_ids + row) - p.target_offset : -1;
            float run_max = -CUDART_INF_F, run_sum = 0.f, target_logit = 0.f, run_wsum = 0.f;
            for (int32_t t = item.tile_begin; ok && t < item.tile_end; ++t, ++tile_count) {
                const uint32_t acc = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
                if (!mbar_wait(&ctl->tmem_full[acc], acc_phase, abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const int32_t n0 = t * kBN;
#pragma unroll 1
                for (int c = 0; c < kBN / 32; ++c) {
                    const int32_t col0 = n0 + c * 32;
                    if (col0 >= p.vocab) break;
                    uint32_t r[32];
                    tmem_ld32(tmem_base + acc * kBN + c * 32 + lane_addr, r);
                    tmem_ld_wait();
                    float x[32];
                    float cmax = -CUDART_INF_F;
                    if (col0 + 32 <= p.vocab) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            x[i] = __uint_as_float(r[i]) * kLog2e;
                            cmax = fmaxf(cmax, x[i]);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            x[i] = (col0 + i < p.vocab) ? __uint_as_float(r[i]) * kLog2e : -CUDART_INF_F;
                            cmax = fmaxf(cmax, x[i]);
                        }
                    }
                    const uint32_t tl = static_cast<uint32_t>(target - col0);
                    if (tl < 32u) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (tl == static_cast<uint32_t>(i)) target_logit = __uint_as_float(r[i]);
                    }
                    const float new_max = fmaxf(run_max, cmax);
                    const float shrink = fast_exp2(run_max - new_max);
                    run_sum *= shrink;
                    run_wsum *= shrink;
                    float part = 0.f, wpart = 0.f;  // sum of weights, and of weight * logit (entropy)
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float e = fast_exp2(x[i] - new_max);  // 0 for masked columns (x = -inf)
                        part += e;
                        wpart = fmaf(e, __uint_as_float(r[i]), wpart);
                    }
                    run_sum += part;
                    run_wsum += wpart;
                    run_max = new_max;
                }
                tc_fence_before_sync();
                mbar_arrive(&ctl->tmem_empty[acc]);
            }
            if (ok && valid)
                p.partials[static_cast<int64_t>(item.chunk) * p.n_rows + row] =
                    make_float4(run_max, run_sum, target_logit, run_wsum);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && ctl->abort_flag != 0u && p.status != nullptr) atomicCAS(p.status, 0, RPX_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------------------------
// CTA-pair variant (cta_group::2): a cluster of two CTAs computes a 256-row x 256-column tile.  Each CTA loads its own
// 128 rows of hidden states and HALF of the W tile (128 of the 256 vocabulary rows), so a stage is 32 KB instead of
// 48 KB per CTA: a third less L2 -> SM and shared-memory traffic per flop, and six stages in the same shared memory.
// The even CTA issues the MMAs for both (M = 256); each CTA's four epilogue warps read their own 128 TMEM lanes.
//   full[s]       lives in the even CTA: its producer arms it with the bytes of BOTH CTAs' loads, and both CTAs'
//                 TMA loads complete on it
//   empty[s], tmem_full[a]   live in each CTA; the even CTA's issuer signals both copies with one multicast commit
//   tmem_empty[a] lives in the even CTA: one arrival per epilogue warp of either CTA (the odd CTA's arrive remotely)
constexpr int kPairStages = 6;
constexpr int kPairBBytes = 128 * kBK * 2;
constexpr int kPairStageBytes = kABytes + kPairBBytes;

struct PairCtl {
    uint64_t full[kPairStages];
    uint64_t empty[kPairStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t drain_flag;
};
constexpr size_t kPairSmemBytes = 1024 + static_cast<size_t>(kPairStages) * kPairStageBytes + sizeof(PairCtl);

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
lm_head_partial_pair_kernel(const __grid_constant__ CUtensorMap tmap_hidden, const __grid_constant__ CUtensorMap tmap_w,
                            const Params p) {
    extern __shared__ uint8_t smem_raw[];
    // both CTAs of a pair must use the same offsets: the dynamic window starts at the same shared-memory address in
    // every CTA of a launch, so rounding it up gives the same result in both
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* smem_a = smem;
    uint8_t* smem_b = smem + kPairStages * kABytes;
    PairCtl* ctl = reinterpret_cast<PairCtl*>(smem + kPairStages * kPairStageBytes);
    volatile uint32_t* abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // 0 = the CTA that issues the MMAs
    const int32_t pair = static_cast<int32_t>(blockIdx.x >> 1), n_pairs = static_cast<int32_t>(gridDim.x >> 1);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&ctl->tmem_full[a], 1);
            mbar_init(&ctl->tmem_empty[a], 8);  // four epilogue warps in each CTA
        }
        mbar_init(&ctl->drain, 1);
        ctl->abort_flag = 0;
        ctl->drain_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmap_hidden);
        tma_prefetch_desc(&tmap_w);
    }
    if (warp == 1) {
        tmem_alloc_pair(&ctl->tmem_base, kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers exist before anything is sent to them
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (one thread in each CTA)
        if (elect_one()) {
            uint32_t it = 0;
            bool ok = true;
            for (int32_t idx = pair; ok && idx < p.total_items; idx += n_pairs) {
                const Item item = decode_item(p, idx);  // m_tile counts 256-row tiles here
                for (int32_t t = item.tile_begin; ok && t < item.tile_end; ++t) {
                    for (int32_t kb = 0; kb < p.k_blocks; ++kb, ++it) {
                        const uint32_t stage = it % kPairStages, phase = (it / kPairStages) & 1u;
                        if (!mbar_wait(&ctl->empty[stage], phase ^ 1u, abort_flag)) {
                            ok = false;
                            break;
                        }
                        if (rank == 0) mbar_arrive_expect_tx(&ctl->full[stage], 2 * kPairStageBytes);
                        const uint32_t full0 = mapa_u32(smem_u32(&ctl->full[stage]), 0);
                        tma_load_2d_pair(smem_a + stage * kABytes, &tmap_hidden, full0, kb * kBK,
                                         (item.m_tile * 2 + static_cast<int32_t>(rank)) * kBM);
                        tma_load_2d_pair(smem_b + stage * kPairBBytes, &tmap_w, full0, kb * kBK,
                                         t * kBN + static_cast<int32_t>(rank) * (kBN / 2));
                    }
                }
            }
            if (!ok && rank == 0) {
                const uint32_t first = it > kPairStages ? it - kPairStages : 0u;
                for (uint32_t j = first; j < it; ++j)
                    mbar_wait(&ctl->full[j % kPairStages], (j / kPairStages) & 1u, &ctl->drain_flag, kDrainLimitCycles);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (one thread of the even CTA)
        if (rank == 0 && elect_one()) {
            constexpr uint32_t idesc = make_idesc_bf16(2 * kBM, kBN, false, false);
            const uint64_t a_desc0 = make_smem_desc_sw128(smem_u32(smem_a), 16, 1024);
            const uint64_t b_desc0 = make_smem_desc_sw128(smem_u32(smem_b), 16, 1024);
            uint32_t it = 0, tile_count = 0;
            bool ok = true;
            for (int32_t idx = pair; ok && idx < p.total_items; idx += n_pairs) {
                const Item item = decode_item(p, idx);
                for (int32_t t = item.tile_begin; ok && t < item.tile_end; ++t, ++tile_count) {
                    const uint32_t acc = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
                    if (!mbar_wait(&ctl->tmem_empty[acc], acc_phase ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + acc * kBN;
                    for (int32_t kb = 0; kb < p.k_blocks; ++kb, ++it) {
                        const uint32_t stage = it % kPairStages, phase = (it / kPairStages) & 1u;
                        if (!mbar_wait(&ctl->full[stage], phase, abort_flag)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        umma_pair_ss_k64(d_tmem, a_desc0 + static_cast<uint64_t>(stage * (kABytes >> 4)),
                                         b_desc0 + static_cast<uint64_t>(stage * (kPairBBytes >> 4)), idesc, kb != 0 ? 1u : 0u);
                        umma_commit_pair(&ctl->empty[stage], 3);  // the stage is free in both CTAs
                    }
                    if (ok) umma_commit_pair(&ctl->tmem_full[acc], 3);
                }
            }
            if (!ok) {
                umma_commit(&ctl->drain);
                mbar_wait(&ctl->drain, 0, &ctl->drain_flag, kDrainLimitCycles);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue (128 threads in each CTA)
        const uint32_t quarter = warp & 3;
        const int32_t row_in_tile = quarter * 32 + lane;
        const uint32_t lane_addr = (quarter * 32u) << 16;
        uint32_t tile_count = 0;
        bool ok = true;
        for (int32_t idx = pair; ok && idx < p.total_items; idx += n_pairs) {
            const Item item = decode_item(p, idx);
            const int64_t row = (static_cast<int64_t>(item.m_tile) * 2 + rank) * kBM + row_in_tile;
            const bool valid = row < p.n_rows;
            const int32_t target = valid ? __ldg(p.target_ids + row) - p.target_offset : -1;
            float run_max = -CUDART_INF_F, run_sum = 0.f, target_logit = 0.f, run_wsum = 0.f;
            for (int32_t t = item.tile_begin; ok && t < item.tile_end; ++t, ++tile_count) {
                const uint32_t acc = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
                if (!mbar_wait(&ctl->tmem_full[acc], acc_phase, abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const int32_t n0 = t * kBN;
#pragma unroll 1
                for (int c = 0; c < kBN / 32; ++c) {
                    const int32_t col0 = n0 + c * 32;
                    if (col0 >= p.vocab) break;
                    uint32_t r[32];
                    tmem_ld32(tmem_base + acc * kBN + c * 32 + lane_addr, r);
                    tmem_ld_wait();
                    float x[32];
                    float cmax = -CUDART_INF_F;
                    if (col0 + 32 <= p.vocab) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            x[i] = __uint_as_float(r[i]) * kLog2e;
                            cmax = fmaxf(cmax, x[i]);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            x[i] = (col0 + i < p.vocab) ? __uint_as_float(r[i]) * kLog2e : -CUDART_INF_F;
                            cmax = fmaxf(cmax, x[i]);
                        }
                    }
                    const uint32_t tl = static_cast<uint32_t>(target - col0);
                    if (tl < 32u) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (tl == static_cast<uint32_t>(i)) target_logit = __uint_as_float(r[i]);
                    }
                    const float new_max = fmaxf(run_max, cmax);
                    const float shrink = fast_exp2(run_max - new_max);
                    run_sum *= shrink;
                    run_wsum *= shrink;
                    float part = 0.f, wpart = 0.f;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float e = fast_exp2(x[i] - new_max);
                        part += e;
                        wpart = fmaf(e, __uint_as_float(r[i]), wpart);
                    }
                    run_sum += part;
                    run_wsum += wpart;
                    run_max = new_max;
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(mapa_u32(smem_u32(&ctl->tmem_empty[acc]), 0));
            }
            if (ok && valid)
                p.partials[static_cast<int64_t>(item.chunk) * p.n_rows + row] =
                    make_float4(run_max, run_sum, target_logit, run_wsum);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();  // neither CTA leaves, or frees TMEM, while the other may still signal or read
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && ctl->abort_flag != 0u && p.status != nullptr) atomicCAS(p.status, 0, RPX_ERR_TIMEOUT);
}

__global__ void lm_head_combine_kernel(const float4* __restrict__ partials, int32_t n_chunks, int64_t n_rows,
                                       const int32_t* __restrict__ target_ids, int32_t vocab,
                                       float* __restrict__ logprobs, float* __restrict__ lse,
                                       float* __restrict__ entropy, float4* __restrict__ stats_out, int32_t* status) {
    const int64_t row = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
    if (row >= n_rows) return;
    float gmax = -CUDART_INF_F;
    for (int32_t c = 0; c < n_chunks; ++c) gmax = fmaxf(gmax, partials[static_cast<int64_t>(c) * n_rows + row].x);
    float sum = 0.f, zt = 0.f, wsum = 0.f;
    for (int32_t c = 0; c < n_chunks; ++c) {
        const float4 v = partials[static_cast<int64_t>(c) * n_rows + row];
        const float f = exp2f(v.x - gmax);
        sum += v.y * f;
        wsum += v.w * f;
        zt += v.z;
    }
    if (stats_out != nullptr) {  // one vocabulary shard: hand the merged record on, another launch finishes
        stats_out[row] = make_float4(gmax, sum, zt, wsum);
        return;
    }
    const float l = (gmax + log2f(sum)) * kLn2;
    const int32_t t = target_ids[row];
    float lp;
    if (t < 0 || t >= vocab) {
        lp = CUDART_NAN_F;
        if (status != nullptr) atomicCAS(status, 0, RPX_ERR_DEVICE_DATA);
    } else {
        lp = zt - l;
    }
    logprobs[row] = lp;
    if (lse != nullptr) lse[row] = l;
    // H = -sum_v p_v ln p_v = lse - E_p[z]
    if (entropy != nullptr) entropy[row] = l - wsum / sum;
}

}  // namespace

int32_t logprob_tiles_per_chunk(int64_t n_tokens, int32_t vocab) {
    const int64_t row_tiles = (n_tokens + kBM - 1) / kBM;
    if (row_tiles <= kSmallRowTiles) {
        // Few row tiles mean few work items per CTA, so the last, partly filled round of items weighs in:
        // take the chunk length (2..8 tiles) that needs the fewest tile-times on the part's 148 SMs, the
        // longer one on a tie (fewer partial records).  This is pure arithmetic on the sizes, so that the
        // workspace size can be computed without a device; on another SM count it is merely not tuned.
        const int64_t vocab_tiles = (static_cast<int64_t>(vocab) + kBN - 1) / kBN;
        int32_t best = kTilesPerChunkSmall;
        int64_t best_cost = INT64_MAX;
        for (int32_t tpc = 8; tpc >= 2; --tpc) {
            const int64_t items = row_tiles * ((vocab_tiles + tpc - 1) / tpc);
            const int64_t cost = ((items + 147) / 148) * tpc;
            if (cost < best_cost) {
                best_cost = cost;
                best = tpc;
            }
        }
        return best;
    }
    return row_tiles >= kHugeRowTiles ? kTilesPerChunkHuge : kTilesPerChunkLarge;
}

int32_t logprob_num_chunks(int32_t vocab, int32_t tiles_per_chunk) {
    const int32_t tiles = (vocab + kBN - 1) / kBN;
    return (tiles + tiles_per_chunk - 1) / tiles_per_chunk;
}

rpx_status_t launch_token_logprobs(const LogprobArgs& a) {
    if (a.n_tokens == 0) return RPX_OK;
    CUtensorMap tmap_h, tmap_w;
    {
        const uint64_t dims[2] = {static_cast<uint64_t>(a.hidden_dim), static_cast<uint64_t>(a.n_tokens)};
        const uint64_t strides[1] = {static_cast<uint64_t>(a.hidden_row_stride) * 2};
        const uint32_t box[2] = {kBK, kBM};
        if (rpx_status_t rc = encode_tmap_bf16(&tmap_h, a.hidden, 2, dims, strides, box)) return rc;
    }
    {
        const uint64_t dims[2] = {static_cast<uint64_t>(a.hidden_dim), static_cast<uint64_t>(a.vocab)};
        const uint64_t strides[1] = {static_cast<uint64_t>(a.hidden_dim) * 2};
        const uint32_t box[2] = {kBK, kBN};
        if (rpx_status_t rc = encode_tmap_bf16(&tmap_w, a.w, 2, dims, strides, box)) return rc;
    }
    Params p;
    p.n_rows = a.n_tokens;
    p.vocab = a.vocab;
    p.k_blocks = (a.hidden_dim + kBK - 1) / kBK;
    p.n_row_tiles = static_cast<int32_t>((a.n_tokens + kBM - 1) / kBM);
    p.n_vocab_tiles = (a.vocab + kBN - 1) / kBN;
    p.tiles_per_chunk = a.tiles_per_chunk;
    p.n_chunks = logprob_num_chunks(a.vocab, a.tiles_per_chunk);
    const int64_t total = static_cast<int64_t>(p.n_row_tiles) * p.n_chunks;
    if (total > INT32_MAX) return RPX_ERR_SHAPE;
    p.total_items = static_cast<int32_t>(total);
    int sms = sm_count();
    if (sms <= 0) return RPX_ERR_CUDA;
    if (const int budget = sm_budget(); budget > 0 && budget < sms) sms = budget;  // leave the rest to a co-runner
    const int grid = static_cast<int>(total < sms ? total : sms);
    // vocab chunks swept side by side by the resident CTAs: 4 keeps (grid / 4) row tiles of hidden states
    // L2-resident while each W tile is shared by that many CTAs (2 and 8 measured 3 % slower at 256 row
    // tiles); with few row tiles 2 is 3 % faster
    p.group_width = (grid % 4 == 0 && p.n_row_tiles > kSmallRowTiles) ? 4 : (grid % 2 == 0 ? 2 : 1);
    p.target_ids = a.target_ids;
    p.target_offset = a.target_offset;
    p.partials = static_cast<float4*>(a.partials);
    p.status = a.device_status;

    if (lm_head_pairing() != 0 && sms >= 2) {
        // CTA pairs: the work list runs over 256-row tiles, the W map hands out half tiles of 128 vocabulary rows
        CUtensorMap tmap_w_half;
        const uint64_t dims[2] = {static_cast<uint64_t>(a.hidden_dim), static_cast<uint64_t>(a.vocab)};
        const uint64_t strides[1] = {static_cast<uint64_t>(a.hidden_dim) * 2};
        const uint32_t box[2] = {kBK, kBN / 2};
        if (rpx_status_t rc = encode_tmap_bf16(&tmap_w_half, a.w, 2, dims, strides, box)) return rc;
        p.n_row_tiles = (p.n_row_tiles + 1) / 2;
        const int64_t total_pairs = static_cast<int64_t>(p.n_row_tiles) * p.n_chunks;
        p.total_items = static_cast<int32_t>(total_pairs);
        const int pairs = static_cast<int>(total_pairs < sms / 2 ? total_pairs : sms / 2);
        p.group_width = (pairs % 4 == 0 && p.n_row_tiles > kSmallRowTiles / 2) ? 4 : (pairs % 2 == 0 ? 2 : 1);
        if (cudaFuncSetAttribute(lm_head_partial_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(kPairSmemBytes)) != cudaSuccess)
            return RPX_ERR_CUDA;
        lm_head_partial_pair_kernel<<<2 * pairs, kThreads, kPairSmemBytes, a.stream>>>(tmap_h, tmap_w_half, p);
        if (cudaGetLastError() != cudaSuccess) return RPX_ERR_CUDA;
    } else {
        if (cudaFuncSetAttribute(lm_head_partial_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(kSmemBytes)) != cudaSuccess)  // per device, cheap: set every time
            return RPX_ERR_CUDA;
        lm_head_partial_kernel<<<grid, kThreads, kSmemBytes, a.stream>>>(tmap_h, tmap_w, p);
        if (cudaGetLastError() != cudaSuccess) return RPX_ERR_CUDA;
    }
    const int cthreads = 256;
    const unsigned cblocks = static_cast<unsigned>((a.n_tokens + cthreads - 1) / cthreads);
    lm_head_combine_kernel<<<cblocks, cthreads, 0, a.stream>>>(p.partials, p.n_chunks, a.n_tokens, a.target_ids,
                                                               a.vocab, a.logprobs, a.lse, a.entropy,
                                                               static_cast<float4*>(a.shard_stats), a.device_status);
    return cudaGetLastError() == cudaSuccess ? RPX_OK : RPX_ERR_CUDA;
}

rpx_status_t launch_logprob_merge(const void* shard_stats, int32_t n_shards, const int32_t* target_ids, int64_t n_tokens,
                                  int32_t vocab_total, float* logprobs, float* lse, float* entropy, int32_t* status,
                                  cudaStream_t stream) {
    if (n_tokens == 0) return RPX_OK;
    const int cthreads = 256;
    const unsigned cblocks = static_cast<unsigned>((n_tokens + cthreads - 1) / cthreads);
    lm_head_combine_kernel<<<cblocks, cthreads, 0, stream>>>(static_cast<const float4*>(shard_stats), n_shards, n_tokens,
                                                             target_ids, vocab_total, logprobs, lse, entropy, nullptr, status);
    return cudaGetLastError() == cudaSuccess ? RPX_OK : RPX_ERR_CUDA;
}

}  // namespace rpx

// ---------------------------------------------------------------------------------------------
// Allocation-free variant.  The partial (max, sum, target-logit) records normally live in the
// caller's workspace; here they live in a fixed array inside the library image, so a caller that
// has no device memory left to hand over (or must not touch the allocator) can still score.
// ---------------------------------------------------------------------------------------------
namespace rpx {
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[RPX_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};

// Device address of g_static_scratch on the CURRENT device.  In host code the array's name is only
// a handle for the runtime, not a device address; the address has to be asked for, per device.
rpx_status_t static_scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RPX_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return RPX_ERR_CUDA;
        g_static_ptr[dev] = ptr;
    }
    *out = g_static_ptr[dev];
    return RPX_OK;
}

}  // namespace
}  // namespace rpx

extern "C" RPX_API rpx_status_t rpx_token_logprobs_static(const void* hidden, int64_t hidden_row_stride,
                                                          const void* w_vocab, const int32_t* target_ids,
                                                          int64_t n_tokens, int32_t hidden_dim, int32_t vocab,
                                                          float* logprobs, float* lse, int32_t* device_status,
                                                          void* cuda_stream) {
    using namespace rpx;
    if (n_tokens < 0 || n_tokens >= INT32_MAX || hidden_dim <= 0 || vocab <= 0 || hidden_dim % 8 != 0)
        return RPX_ERR_SHAPE;
    if (n_tokens == 0) return RPX_OK;
    if (hidden == nullptr || w_vocab == nullptr || target_ids == nullptr || logprobs == nullptr) return RPX_ERR_NULL;
    if (hidden_row_stride < hidden_dim) return RPX_ERR_SHAPE;
    if (hidden_row_stride % 8 != 0) return RPX_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(hidden) & 15u) != 0 || (reinterpret_cast<uintptr_t>(w_vocab) & 15u) != 0)
        return RPX_ERR_ALIGN;
    // one 16-byte record per (vocab chunk, row) must fit in the built-in array
    const size_t need = static_cast<size_t>(logprob_num_chunks(vocab, kTilesPerChunkLarge)) * static_cast<size_t>(n_tokens) * sizeof(float4);
    if (need > static_cast<size_t>(RPX_STATIC_SCRATCH_BYTES)) return RPX_ERR_WORKSPACE;
    if (rpx_status_t rc = check_arch()) return rc;
    void* scratch = nullptr;
    if (rpx_status_t rc = static_scratch_for_current_device(&scratch)) return rc;

    LogprobArgs a;
    a.hidden = hidden;
    a.hidden_row_stride = hidden_row_stride;
    a.w = w_vocab;
    a.target_ids = target_ids;
    a.n_tokens = n_tokens;
    a.hidden_dim = hidden_dim;
    a.vocab = vocab;
    a.logprobs = logprobs;
    a.lse = lse;
    a.entropy = nullptr;
    a.shard_stats = nullptr;
    a.target_offset = 0;
    a.partials = scratch;
    a.tiles_per_chunk = kTilesPerChunkLarge;  // the documented size limit assumes 16-tile chunks
    a.device_status = device_status;
    a.stream = static_cast<cudaStream_t>(cuda_stream);
    return launch_token_logprobs(a);
}
