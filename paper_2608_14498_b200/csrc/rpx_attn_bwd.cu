// Backward of varlen causal GQA attention for sm_100a (gradients through the prefix/suffix boundary).
//
// With P_ij the softmax weights of query row (i,h) over keys j <= i (recomputed from the forward pass's LSE),
// g = h / (H_q / H_kv), dP_ij = dO[i,h,:] . V[j,g,:], D_i = sum_c dO[i,h,c] O[i,h,c] (= sum_j P_ij dP_ij) and
// dS_ij = P_ij (dP_ij - D_i):
//     dV[j,g,:] = sum_{h in g} sum_{i >= j} P_ij  dO[i,h,:]
//     dK[j,g,:] = scale * sum_{h in g} sum_{i >= j} dS_ij Q[i,h,:]
//     dQ[i,h,:] = scale * sum_{j <= i} dS_ij K[j,g,:]
// A key of the prompt receives terms from prompt queries and from response queries alike.  The query rows that take
// part can be restricted per sequence ([q_begin, q_end)), and dK / dV can be added to what the buffers hold, so the
// split schedule - the suffix pass's gradients first, the prefix pass's on top - is two calls of the same kernels.
//
// One kernel template serves both directions, because they are the same computation with the roles of the operands
// exchanged.  An item keeps one OUTER pair of 128-row tiles (X1, X2) in shared memory and walks INNER pairs (Y1, Y2):
//     T1 = X1 Y1^T,  T2 = X2 Y2^T          (two SS MMAs into TMEM, 128 x 128 fp32 each)
//     element-wise: P = 2^(T1 * scale * log2 e - lse * log2 e), dS = P (T2 - D), masked; bf16 back into TMEM
//     accumulate: A_a += P Y2, A_b += dS Y1  (TS MMAs: the TMEM tile is the A operand, Y straight from its
//                                             [rows][d] tile as an MN-major B operand)
//   kDq = false: (X1, X2, Y1, Y2) = (K_j, V_j, Q_i, dO_i): T1 = S^T, T2 = dP^T with keys as TMEM lanes, A_a = dV_j,
//                A_b = dK_j; the inner loop runs over the query heads of the KV head and the query tiles i >= j.
//   kDq = true : (X1, X2, Y1, Y2) = (Q_i, dO_i, K_j, V_j): T1 = S, T2 = dP with queries as lanes, A_b = dQ_i (A_a is
//                not needed); the inner loop runs over the key tiles j <= i.
// Because the transposed scores are computed directly (K Q^T instead of Q K^T), P^T and dS^T are born with keys as
// TMEM lanes, which is what makes them usable as A operands for dV and dK without a trip through shared memory.
//
// Warp roles (320 threads): warp 0 = TMA producer (it also copies the inner tile's lse and D vectors), warp 1 =
// TMEM owner + tcgen05 issuer, warps 2..9 = element-wise + epilogue (thread = outer row = TMEM lane; two warps per
// lane quarter, each taking half of the columns).
// TMEM holds the two accumulators (2 x d columns) and ONE T1/T2 pair (256 columns), so to overlap tensor-core and
// element-wise work an inner tile is processed as two halves of 64 inner rows: while the warps turn half a into
// P / dS, the tensor core computes T of half b, then accumulates half a, then computes the next step's half a, ...
// Masking costs nothing off the diagonal: rows of the inner query tile that do not take part get -lse = -inf (P = 0,
// dS = 0) in the vector the producer prepares, and outer rows that do not exist only pollute their own accumulator
// lanes, which are never stored; only the diagonal tile applies the causal predicate per element.
#include <math_constants.h>

#include "rpx_internal.h"
#include "rpx_ptx.cuh"

namespace rpx {

namespace {

constexpr int kTile = 128;
constexpr int kStages = 4;   // half inner tiles (64 rows of Y1 and of Y2) in flight: two steps of data, released a half at a time (a fifth stage measured no faster)
constexpr int kThreads = 320;
constexpr int kHalf = 64;    // inner rows per half step
constexpr uint32_t kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;

struct Ctl {
    uint64_t outer_full;          // producer -> issuer: X1, X2 are in shared memory
    uint64_t outer_empty;         // issuer -> producer: the item's last T MMAs have finished
    uint64_t in_full[kStages];
    uint64_t in_empty[kStages];
    uint64_t t_full[2];           // issuer -> element-wise warps: T1, T2 of a half step are in TMEM
    uint64_t e_ready[2];          // element-wise warps -> issuer: P / dS of the half step are in TMEM
    uint64_t acc_done;            // issuer -> element-wise warps: the item's last accumulate MMAs have finished
    uint64_t acc_free;            // element-wise warps -> issuer: the accumulators have been read out
    uint64_t drain;
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t drain_flag;
    uint32_t data_error;
    float vec[kStages][2][kHalf]; // kDq = false: (-lse * log2 e or -inf, -D) of the stage's 64 inner query rows
};

template <int D>
struct Layout {
    static constexpr int kHalves = D / 64;
    static constexpr int kHalfBytes = kTile * 128;
    static constexpr int kTileBytes = kHalves * kHalfBytes;
    static constexpr int kOuterOff = 0;                                  // X1, X2
    static constexpr int kInnerOff = 2 * kTileBytes;                     // kStages x (Y1 half, Y2 half)
    static constexpr int kBlockBytes = kHalf * 128;                      // one [64 rows][64 bf16] swizzled block of a half
    static constexpr int kHalfTileBytes = kHalves * kBlockBytes;         // 64 rows of one inner tile
    static constexpr int kStageBytes = 2 * kHalfTileBytes;
    static constexpr int kCtlOff = kInnerOff + kStages * kStageBytes;
    static constexpr size_t kSmemBytes = kCtlOff + sizeof(Ctl);
};

struct Params {
    const int32_t* cu_seqlens;
    const int32_t* q_begin;   // nullable: first query row of every sequence that takes part
    const int32_t* q_end;     // nullable: one past the last
    int32_t batch, num_q_heads, num_kv_heads, group;
    int32_t n_tiles;          // 128-row tiles per sequence the work list covers
    int32_t n_items;
    int64_t total_tokens;
    const float* lse;         // [tokens][H_q], natural log
    const float* dvec;        // [tokens][H_q]: D = rowsum(dO * O)
    float scale, scale_log2;
    float* dq;                // [tokens][H_q][D]
    float* dk;                // [tokens][H_kv][D]
    float* dv;
    int32_t accumulate;       // add dK / dV to what the buffers hold
    int32_t* status;
};

struct Item {
    int32_t seq, head, tile, tok0, len, qb, qe;
    int32_t in_lo, in_hi, n_heads;  // inner tiles in_lo .. in_hi (inclusive) for each of n_heads heads
    bool active, bad;
};

// Four K=16 steps of D (+)= A[tmem] * B[smem, MN-major] over 64 inner rows.  The A operand of steps 0, 1 sits in
// columns 0..15 and that of steps 2, 3 in columns 32..47 (each warp group leaves its 16 packed columns at the start of
// the 32 it has read); B advances 16 rows of 128 bytes (128 units) per step.
__device__ __forceinline__ void umma_ts_k64_split(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc,
                                                  uint32_t accumulate_first) {
    asm volatile(
        "{\n"
        ".reg .pred pf, pt;\n"
        ".reg .b64 db;\n"
        ".reg .b32 ta;\n"
        "setp.ne.b32 pf, %4, 0;\n"
        "setp.eq.b32 pt, %4, %4;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, pf;\n" RPX_UMMA_TS_STEP(8, 128) RPX_UMMA_TS_STEP(32, 256)
            RPX_UMMA_TS_STEP(40, 384) "}\n" ::"r"(tmem_d),
        "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate_first)
        : "memory");
}

// Items are ordered longest first; the CTAs take them in serpentine order (0 .. G-1, then G-1 .. 0, ...), which
// evens out the inner steps per CTA far better than a plain stride when the item lengths fall linearly.
__device__ __forceinline__ int32_t item_of_round(int32_t rnd) {
    const int32_t g = static_cast<int32_t>(gridDim.x), b = static_cast<int32_t>(blockIdx.x);
    return rnd * g + ((rnd & 1) ? g - 1 - b : b);
}

// Eight K=16 steps of D = A * B: A's two 64-element K blocks lie 16 KiB (1024 units) apart (a 128-row tile), B's
// 8 KiB (512 units) apart (a 64-row half tile).
__device__ __forceinline__ void umma_ss_k128_half_b(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc) {
#define RPX_UMMA_SS_STEP_AB(aoff, boff)                                        \
    "add.s64 da, %1, " #aoff ";\n"                                             \
    "add.s64 db, %2, " #boff ";\n"                                             \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, pt;\n"
    asm volatile(
        "{\n"
        ".reg .pred pf, pt;\n"
        ".reg .b64 da, db;\n"
        "setp.ne.b32 pf, %3, %3;\n"
        "setp.eq.b32 pt, %3, %3;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pf;\n" RPX_UMMA_SS_STEP_AB(2, 2) RPX_UMMA_SS_STEP_AB(4, 4)
            RPX_UMMA_SS_STEP_AB(6, 6) RPX_UMMA_SS_STEP_AB(1024, 512) RPX_UMMA_SS_STEP_AB(1026, 514)
                RPX_UMMA_SS_STEP_AB(1028, 516) RPX_UMMA_SS_STEP_AB(1030, 518) "}\n" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc)
        : "memory");
#undef RPX_UMMA_SS_STEP_AB
}

template <bool kDq>
__device__ __forceinline__ Item decode_item(const Params& p, int32_t idx) {
    Item it;
    const int32_t heads = kDq ? p.num_q_heads : p.num_kv_heads;
    const int32_t per_tile = p.batch * heads;
    // dkdv: early key tiles have the most query tiles behind them, dq: late query tiles the most keys: longest first
    const int32_t t = idx / per_tile;
    it.tile = kDq ? p.n_tiles - 1 - t : t;
    const int32_t rem = idx % per_tile;
    it.seq = rem / heads;
    it.head = rem % heads;
    it.tok0 = __ldg(p.cu_seqlens + it.seq);
    it.len = __ldg(p.cu_seqlens + it.seq + 1) - it.tok0;
    bool bad = it.tok0 < 0 || it.len < 0 || static_cast<int64_t>(it.tok0) + it.len > p.total_tokens;
    it.qb = p.q_begin != nullptr ? __ldg(p.q_begin + it.seq) : 0;
    it.qe = p.q_end != nullptr ? __ldg(p.q_end + it.seq) : it.len;
    it.bad = bad;
    if (bad) it.len = 0;
    it.qb = max(0, it.qb);
    it.qe = min(it.len, it.qe);
    it.active = !bad && it.tile * kTile < it.len && it.qb < it.qe;
    if (kDq) {
        // outer = query tile: it must hold rows of the range; inner = key tiles 0 .. tile
        it.active = it.active && it.tile * kTile < it.qe && (it.tile + 1) * kTile > it.qb;
        it.in_lo = 0;
        it.in_hi = it.tile;
        it.n_heads = 1;
    } else {
        // outer = key tile; inner = query tiles that hold rows >= the tile's first key and inside the range
        it.in_lo = max(it.tile, it.qb / kTile);
        it.in_hi = (it.qe - 1) / kTile;
        it.n_heads = p.group;
        it.active = it.active && it.in_lo <= it.in_hi;
    }
    if (!it.active) it.n_heads = 0;
    return it;
}

template <int D, bool kDq>
__global__ void __launch_bounds__(kThreads, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmap_x1, const __grid_constant__ CUtensorMap tmap_x2,
                const __grid_constant__ CUtensorMap tmap_y1, const __grid_constant__ CUtensorMap tmap_y2, const Params p) {
    // x1, x2: the outer tiles' tensors (K, V for dK/dV; Q, dO for dQ), boxes of 128 rows; y1, y2: the inner tiles'
    // (Q, dO; K, V), boxes of 64 rows
    using L = Layout<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    if ((smem_u32(smem) & 1023u) != 0u) {
        if (threadIdx.x == 0 && p.status != nullptr) atomicCAS(p.status, 0, RPX_ERR_CUDA);
        return;
    }
    Ctl* ctl = reinterpret_cast<Ctl*>(smem + L::kCtlOff);
    volatile uint32_t* abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(&ctl->outer_full, 1);
        mbar_init(&ctl->outer_empty, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&ctl->in_full[s], 1);
            mbar_init(&ctl->in_empty[s], 1);
        }
        for (int h = 0; h < 2; ++h) {
            mbar_init(&ctl->t_full[h], 1);
            mbar_init(&ctl->e_ready[h], 8);
        }
        mbar_init(&ctl->acc_done, 1);
        mbar_init(&ctl->acc_free, 8);
        mbar_init(&ctl->drain, 1);
        ctl->abort_flag = 0;
        ctl->drain_flag = 0;
        ctl->data_error = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(&ctl->tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl->tmem_base;
    // TMEM columns: T1 at 0, T2 at 128, accumulator a at 256, accumulator b at 256 + D
    const CUtensorMap *map_x1 = &tmap_x1, *map_x2 = &tmap_x2, *map_y1 = &tmap_y1, *map_y2 = &tmap_y2;

    if (warp == 0) {
        // =========================================================== producer warp
        bool ok = true;
        uint32_t n_items = 0, n_in = 0;
        for (int32_t rnd = 0, idx = blockIdx.x; ok && idx < p.n_items; idx = item_of_round(++rnd)) {
            const Item it = decode_item<kDq>(p, idx);
            // offsets that leave the packed tensors are reported, not followed; so is a sequence longer than the caller's
            // bound, whose rows beyond it the work list never reaches
            if (it.bad || it.len > p.n_tiles * kTile) ctl->data_error = 1u;
            if (!it.active) continue;
            const int32_t kv_head = kDq ? it.head / p.group : it.head;
            if (n_items > 0 && !mbar_wait(&ctl->outer_empty, (n_items - 1) & 1u, abort_flag)) {
                ok = false;
                break;
            }
            if (lane == 0) {
                mbar_arrive_expect_tx(&ctl->outer_full, 2 * L::kTileBytes);
                for (int hf = 0; hf < L::kHalves; ++hf) {
                    // x1/x2 head coordinate: K, V by KV head; Q, dO by query head
                    tma_load_3d(smem + L::kOuterOff + hf * L::kHalfBytes, map_x1, &ctl->outer_full, hf * 64,
                                kDq ? it.head : kv_head, it.tok0 + it.tile * kTile);
                    tma_load_3d(smem + L::kOuterOff + L::kTileBytes + hf * L::kHalfBytes, map_x2, &ctl->outer_full, hf * 64,
                                kDq ? it.head : kv_head, it.tok0 + it.tile * kTile);
                }
            }
            for (int32_t hh = 0; ok && hh < it.n_heads; ++hh) {
                const int32_t qh = kDq ? it.head : it.head * p.group + hh;  // the query head of this inner run
                for (int32_t in2 = 2 * it.in_lo; ok && in2 <= 2 * it.in_hi + 1; ++in2, ++n_in) {
                    const int32_t in = in2 >> 1, h = in2 & 1;  // n_in counts half tiles here
                    const uint32_t stage = n_in % kStages, phase = (n_in / kStages) & 1u;
                    if (!mbar_wait(&ctl->in_empty[stage], phase ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    uint8_t* y1 = smem + L::kInnerOff + stage * L::kStageBytes;
                    uint8_t* y2 = y1 + L::kHalfTileBytes;
                    if (!kDq) {
                        // -lse (in log2 units) and -D of the inner query tile, for the element-wise warps
                        for (int32_t r = lane; r < kHalf; r += 32) {
                            const int32_t qr = in * kTile + h * kHalf + r;
                            float l2 = -CUDART_INF_F, dd = 0.f;  // a row that takes no part: P = 2^(-inf) = 0, dS = 0
                            if (qr >= it.qb && qr < it.qe) {
                                const int64_t rh = static_cast<int64_t>(it.tok0 + qr) * p.num_q_heads + qh;
                                l2 = -__ldg(p.lse + rh) * kLog2e;
                                dd = -__ldg(p.dvec + rh);
                            }
                            ctl->vec[stage][0][r] = l2;
                            ctl->vec[stage][1][r] = dd;
                        }
                        __syncwarp();
                    }
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&ctl->in_full[stage], L::kStageBytes);
                        for (int hf = 0; hf < L::kHalves; ++hf) {
                            tma_load_3d(y1 + hf * L::kBlockBytes, map_y1, &ctl->in_full[stage], hf * 64, kDq ? kv_head : qh,
                                        it.tok0 + in * kTile + h * kHalf);
                            tma_load_3d(y2 + hf * L::kBlockBytes, map_y2, &ctl->in_full[stage], hf * 64, kDq ? kv_head : qh,
                                        it.tok0 + in * kTile + h * kHalf);
                        }
                    }
                    __syncwarp();
                }
            }
            ++n_items;
        }
        if (!ok) {
            const uint32_t first = n_in > kStages ? n_in - kStages : 0u;
            for (uint32_t i = first; i < n_in; ++i)
                mbar_wait(&ctl->in_full[i % kStages], (i / kStages) & 1u, &ctl->drain_flag, kDrainLimitCycles);
            if (n_items > 0) mbar_wait(&ctl->outer_full, (n_items - 1) & 1u, &ctl->drain_flag, kDrainLimitCycles);
        }
    } else if (warp == 1) {
        // =========================================================== tcgen05 issuer (one thread)
        if (elect_one()) {
            constexpr uint32_t idesc_t = make_idesc_bf16(kTile, kHalf, false, false);
            constexpr uint32_t idesc_acc = make_idesc_bf16(kTile, D, false, true);
            const uint32_t outer_addr = smem_u32(smem + L::kOuterOff);
            const uint32_t inner_addr = smem_u32(smem + L::kInnerOff);
            const uint64_t x1_desc = make_smem_desc_sw128(outer_addr, 16, 1024);
            const uint64_t x2_desc = make_smem_desc_sw128(outer_addr + L::kTileBytes, 16, 1024);
            // T1 = X1 Y1^T and T2 = X2 Y2^T for the inner rows 64 h .. 64 h + 63 of the pair in `stage`
            auto issue_t = [&](uint32_t stage, int h) {
                const uint32_t y1_addr = inner_addr + stage * L::kStageBytes;
                const uint64_t y1_k = make_smem_desc_sw128(y1_addr, 16, 1024);
                const uint64_t y2_k = make_smem_desc_sw128(y1_addr + L::kHalfTileBytes, 16, 1024);
                if (D == 128) {
                    umma_ss_k128_half_b(tmem_base + h * kHalf, x1_desc, y1_k, idesc_t);
                    umma_ss_k128_half_b(tmem_base + kTile + h * kHalf, x2_desc, y2_k, idesc_t);
                } else {
                    umma_ss_k64_overwrite(tmem_base + h * kHalf, x1_desc, y1_k, idesc_t);
                    umma_ss_k64_overwrite(tmem_base + kTile + h * kHalf, x2_desc, y2_k, idesc_t);
                }
                umma_commit(&ctl->t_full[h]);
            };
            bool ok = true;
            uint32_t n_items = 0, n_in = 0;
            for (int32_t rnd = 0, idx = blockIdx.x; ok && idx < p.n_items; idx = item_of_round(++rnd)) {
                const Item it = decode_item<kDq>(p, idx);
                if (!it.active) continue;
                ok = mbar_wait(&ctl->outer_full, n_items & 1u, abort_flag);
                // the accumulators still hold the previous item's result until its epilogue has read them
                if (ok && n_items > 0) ok = mbar_wait(&ctl->acc_free, (n_items - 1) & 1u, abort_flag);
                const int32_t steps = it.n_heads * (it.in_hi - it.in_lo + 1);
                // n_in counts steps; the half tile (step n, half h) is the ring's entry 2 n + h
                for (int h = 0; ok && h < 2; ++h) {
                    const uint32_t e = 2 * n_in + h;
                    ok = mbar_wait(&ctl->in_full[e % kStages], (e / kStages) & 1u, abort_flag);
                    if (ok) {
                        tc_fence_after_sync();
                        issue_t(e % kStages, h);
                    }
                }
                if (ok && steps == 1) umma_commit(&ctl->outer_empty);
                for (int32_t s = 0; ok && s < steps; ++s, ++n_in) {
                    for (int h = 0; ok && h < 2; ++h) {
                        const uint32_t stage = (2 * n_in + h) % kStages;
                        const uint32_t y1_addr = inner_addr + stage * L::kStageBytes;
                        const uint64_t y1_mn = make_smem_desc_sw128(y1_addr, L::kBlockBytes, 1024);              // MN-major
                        const uint64_t y2_mn = make_smem_desc_sw128(y1_addr + L::kHalfTileBytes, L::kBlockBytes, 1024);
                        if (!mbar_wait(&ctl->e_ready[h], n_in & 1u, abort_flag)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        // accumulate over the 64 inner rows of the half: a += P Y2 (dV; not for dQ), b += dS Y1 (dK or dQ)
                        const uint32_t acc = (s != 0 || h != 0) ? 1u : 0u;
                        if (!kDq)
                            umma_ts_k64_split(tmem_base + 2 * kTile, tmem_base + h * kHalf, y2_mn, idesc_acc, acc);
                        umma_ts_k64_split(tmem_base + 2 * kTile + D, tmem_base + kTile + h * kHalf, y1_mn, idesc_acc, acc);
                        umma_commit(&ctl->in_empty[stage]);
                        if (s + 1 < steps) {
                            // the next step's T of this half, in order behind the accumulate MMAs that read P / dS from
                            // the same columns
                            const uint32_t ne = 2 * (n_in + 1) + h, nstage = ne % kStages;
                            if (!mbar_wait(&ctl->in_full[nstage], (ne / kStages) & 1u, abort_flag)) {
                                ok = false;
                                break;
                            }
                            tc_fence_after_sync();
                            issue_t(nstage, h);
                            if (h == 1 && s + 2 == steps) umma_commit(&ctl->outer_empty);
                        }
                    }
                }
                if (ok) umma_commit(&ctl->acc_done);
                ++n_items;
            }
            if (!ok) {
                umma_commit(&ctl->drain);
                mbar_wait(&ctl->drain, 0, &ctl->drain_flag, kDrainLimitCycles);
            }
        }
        __syncwarp();
    } else {
        // =========================================================== element-wise + epilogue warps (thread = outer row)
        const uint32_t quarter = warp & 3;
        const uint32_t grp = (warp - 2) >> 2;  // which 32 of a half's 64 columns
        const int32_t r = quarter * 32 + lane;
        const uint32_t lane_addr = (quarter * 32u) << 16;
        const uint32_t t1 = tmem_base + lane_addr, t2 = tmem_base + kTile + lane_addr;
        const uint64_t sl2 = f2_pack(p.scale_log2, p.scale_log2);
        bool ok = true;
        uint32_t n_items = 0, n_in = 0;
        for (int32_t rnd = 0, idx = blockIdx.x; ok && idx < p.n_items; idx = item_of_round(++rnd)) {
            const Item it = decode_item<kDq>(p, idx);
            if (!it.active) continue;
            const int32_t outer_row = it.tile * kTile + r;  // key position (dK/dV) or query position (dQ)
            // rows of the outer tile that do not exist or take no part pollute only their own accumulator lanes, which
            // are not stored
            const bool row_ok = kDq ? (outer_row >= it.qb && outer_row < it.qe) : outer_row < it.len;
            uint64_t nl2_row = 0, nd_row = 0;
            if (kDq && row_ok) {
                const int64_t rh = static_cast<int64_t>(it.tok0 + outer_row) * p.num_q_heads + it.head;
                const float l2 = -__ldg(p.lse + rh) * kLog2e, nd = -__ldg(p.dvec + rh);
                nl2_row = f2_pack(l2, l2);
                nd_row = f2_pack(nd, nd);
            }
            const int32_t n_inner = it.in_hi - it.in_lo + 1;
            const int32_t steps = it.n_heads * n_inner;
            for (int32_t s = 0; ok && s < steps; ++s, ++n_in) {
                const int32_t in = it.in_lo + s % n_inner;
                const bool diagonal = in == it.tile;
                for (int h = 0; h < 2; ++h) {
                    const uint32_t e = 2 * n_in + h, stage = e % kStages;
                    // the producer's lse / D vectors of this stage are visible once the stage's barrier has completed
                    if (!kDq && !mbar_wait(&ctl->in_full[stage], (e / kStages) & 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    if (!mbar_wait(&ctl->t_full[h], n_in & 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t col = h * kHalf + grp * 32;  // this thread's 32 inner rows of the step
                    uint32_t a[32], b[32];
                    tmem_ld32(t1 + col, a);
                    tmem_ld32(t2 + col, b);
                    tmem_ld_wait();
                    uint32_t pw[16], dw[16];
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        uint64_t nl2, nd;
                        if (kDq) {
                            nl2 = nl2_row;
                            nd = nd_row;
                        } else {
                            const float2 lv = *reinterpret_cast<const float2*>(&ctl->vec[stage][0][grp * 32 + i]);
                            const float2 dv2 = *reinterpret_cast<const float2*>(&ctl->vec[stage][1][grp * 32 + i]);
                            nl2 = f2_pack(lv.x, lv.y);
                            nd = f2_pack(dv2.x, dv2.y);
                        }
                        // P = 2^(T1 * scale * log2 e - lse * log2 e), dS = P (T2 - D), two elements per instruction
                        float x0, x1;
                        f2_unpack(f2_fma(f2_pack(__uint_as_float(a[i]), __uint_as_float(a[i + 1])), sl2, nl2), x0, x1);
                        if (diagonal) {  // causal: the key position must not exceed the query position
                            const int32_t inner_pos = in * kTile + col + i;
                            const bool v0 = kDq ? inner_pos <= outer_row : inner_pos >= outer_row;
                            const bool v1 = kDq ? inner_pos + 1 <= outer_row : inner_pos + 1 >= outer_row;
                            x0 = v0 ? x0 : -CUDART_INF_F;
                            x1 = v1 ? x1 : -CUDART_INF_F;
                        }
                        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                        float d0, d1;
                        f2_unpack(f2_add(f2_pack(__uint_as_float(b[i]), __uint_as_float(b[i + 1])), nd), d0, d1);
                        pw[i >> 1] = pack_bf16x2(p0, p1);
                        dw[i >> 1] = pack_bf16x2(p0 * d0, p1 * d1);
                    }
                    // P over the first 16 of the 32 columns this thread has read from T1, dS likewise in T2
                    if (!kDq) tmem_st16(t1 + col, pw);
                    tmem_st16(t2 + col, dw);
                    tmem_st_wait();
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->e_ready[h]);
                }
            }
            if (!ok) break;
            // ---- epilogue: the accumulators -> global (fp32), dK and dQ times the softmax scale
            ok = mbar_wait(&ctl->acc_done, n_items & 1u, abort_flag);
            ++n_items;
            if (!ok) break;
            tc_fence_after_sync();
            const int32_t out_heads = kDq ? p.num_q_heads : p.num_kv_heads;
            const int64_t out_off = (static_cast<int64_t>(it.tok0 + outer_row) * out_heads + it.head) * D;
            // dK/dV: one warp group per accumulator; dQ: the groups split the columns of the one accumulator
            const uint32_t acc_col = kDq ? 2 * kTile + D + grp * (D / 2) : 2 * kTile + grp * D;
            float* dst = (kDq ? p.dq + grp * (D / 2) : (grp == 0 ? p.dv : p.dk)) + out_off;
            const float mul = (kDq || grp == 1) ? p.scale : 1.f;
            const bool add = !kDq && p.accumulate != 0;
            constexpr int kChunks = (kDq ? D / 2 : D) / 32;
#pragma unroll 1
            for (int c = 0; c < kChunks; ++c) {
                uint32_t a[32];
                tmem_ld32(tmem_base + acc_col + c * 32 + lane_addr, a);
                tmem_ld_wait();
                if (row_ok) {
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        float4 v = make_float4(__uint_as_float(a[i]) * mul, __uint_as_float(a[i + 1]) * mul,
                                               __uint_as_float(a[i + 2]) * mul, __uint_as_float(a[i + 3]) * mul);
                        float4* q4 = reinterpret_cast<float4*>(dst + c * 32 + i);
                        if (add) {
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
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->acc_free);
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

// D[token, head] = sum_c dO[token, head, c] * O[token, head, c]; one warp per (token, head)
__global__ void attn_bwd_dvec_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout,
                                     int64_t rows, int32_t head_dim, float* __restrict__ dvec) {
    const int64_t row = (blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    float acc = 0.f;
    for (int c = lane * 2; c < head_dim; c += 64) {
        const __nv_bfloat162 o = *reinterpret_cast<const __nv_bfloat162*>(out + row * head_dim + c);
        const __nv_bfloat162 g = *reinterpret_cast<const __nv_bfloat162*>(dout + row * head_dim + c);
        acc = fmaf(__bfloat162float(o.x), __bfloat162float(g.x), acc);
        acc = fmaf(__bfloat162float(o.y), __bfloat162float(g.y), acc);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) dvec[row] = acc;
}

// rows of dK / dV no key tile's item writes (sequences outside every range): cleared when not accumulating
__global__ void attn_bwd_zero_kernel(float* __restrict__ a, float* __restrict__ b, int64_t n) {
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        a[i] = 0.f;
        if (b != nullptr) b[i] = 0.f;
    }
}

template <int D>
rpx_status_t launch_d(const AttnBwdArgs& a) {
    using L = Layout<D>;
    // every tensor twice: boxes of 128 rows where it is the outer tile, of 64 rows where it is streamed as inner halves
    CUtensorMap tq[2], tk[2], tv[2], tdo[2];
    const uint64_t tokens = static_cast<uint64_t>(a.total_tokens);
    for (int m = 0; m < 2; ++m) {
        const uint32_t box[3] = {64, 1, m == 0 ? static_cast<uint32_t>(kTile) : static_cast<uint32_t>(kHalf)};
        {
            const uint64_t dims[3] = {D, static_cast<uint64_t>(a.num_q_heads), tokens};
            const uint64_t qs[2] = {D * 2ull, static_cast<uint64_t>(a.q_tok_stride) * 2};
            const uint64_t os[2] = {D * 2ull, static_cast<uint64_t>(a.num_q_heads) * D * 2ull};
            if (rpx_status_t rc = encode_tmap_bf16(&tq[m], a.q, 3, dims, qs, box)) return rc;
            if (rpx_status_t rc = encode_tmap_bf16(&tdo[m], a.dout, 3, dims, os, box)) return rc;
        }
        {
            const uint64_t dims[3] = {D, static_cast<uint64_t>(a.num_kv_heads), tokens};
            const uint64_t ks[2] = {D * 2ull, static_cast<uint64_t>(a.k_tok_stride) * 2};
            const uint64_t vs[2] = {D * 2ull, static_cast<uint64_t>(a.v_tok_stride) * 2};
            if (rpx_status_t rc = encode_tmap_bf16(&tk[m], a.k, 3, dims, ks, box)) return rc;
            if (rpx_status_t rc = encode_tmap_bf16(&tv[m], a.v, 3, dims, vs, box)) return rc;
        }
    }
    int sms = sm_count();
    if (sms <= 0) return RPX_ERR_CUDA;
    if (const int budget = sm_budget(); budget > 0 && budget < sms) sms = budget;
    // ---- D = rowsum(dO * O)
    const int64_t rows = a.total_tokens * a.num_q_heads;
    {
        const int threads = 256;
        const int64_t blocks = (rows * 32 + threads - 1) / threads;
        attn_bwd_dvec_kernel<<<static_cast<unsigned>(blocks), threads, 0, a.stream>>>(
            static_cast<const __nv_bfloat16*>(a.out), static_cast<const __nv_bfloat16*>(a.dout), rows, D, a.dvec);
        if (cudaGetLastError() != cudaSuccess) return RPX_ERR_CUDA;
    }
    const int64_t n_q = a.total_tokens * a.num_q_heads * D, n_kv = a.total_tokens * a.num_kv_heads * D;
    attn_bwd_zero_kernel<<<sms * 4, 256, 0, a.stream>>>(a.dq, nullptr, n_q);
    if (!a.accumulate) attn_bwd_zero_kernel<<<sms * 4, 256, 0, a.stream>>>(a.dk, a.dv, n_kv);
    if (cudaGetLastError() != cudaSuccess) return RPX_ERR_CUDA;

    Params p;
    p.cu_seqlens = a.cu_seqlens;
    p.q_begin = a.q_begin;
    p.q_end = a.q_end;
    p.batch = a.batch;
    p.num_q_heads = a.num_q_heads;
    p.num_kv_heads = a.num_kv_heads;
    p.group = a.num_q_heads / a.num_kv_heads;
    p.n_tiles = (a.max_seqlen + kTile - 1) / kTile;
    p.total_tokens = a.total_tokens;
    p.lse = a.lse;
    p.dvec = a.dvec;
    p.scale = a.softmax_scale > 0.f ? a.softmax_scale : 1.0f / sqrtf(static_cast<float>(D));
    p.scale_log2 = p.scale * kLog2e;
    p.dq = a.dq;
    p.dk = a.dk;
    p.dv = a.dv;
    p.accumulate = a.accumulate ? 1 : 0;
    p.status = a.device_status;
    if (cudaFuncSetAttribute(attn_bwd_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(L::kSmemBytes)) != cudaSuccess ||
        cudaFuncSetAttribute(attn_bwd_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(L::kSmemBytes)) != cudaSuccess)
        return RPX_ERR_CUDA;
    {
        const int64_t items = static_cast<int64_t>(p.n_tiles) * a.batch * a.num_kv_heads;
        if (items > INT32_MAX) return RPX_ERR_SHAPE;
        p.n_items = static_cast<int32_t>(items);
        const unsigned grid = static_cast<unsigned>(items < sms ? items : sms);
        attn_bwd_kernel<D, false><<<grid, kThreads, L::kSmemBytes, a.stream>>>(tk[0], tv[0], tq[1], tdo[1], p);
        if (cudaGetLastError() != cudaSuccess) return RPX_ERR_CUDA;
    }
    {
        const int64_t items = static_cast<int64_t>(p.n_tiles) * a.batch * a.num_q_heads;
        if (items > INT32_MAX) return RPX_ERR_SHAPE;
        p.n_items = static_cast<int32_t>(items);
        const unsigned grid = static_cast<unsigned>(items < sms ? items : sms);
        attn_bwd_kernel<D, true><<<grid, kThreads, L::kSmemBytes, a.stream>>>(tq[0], tdo[0], tk[1], tv[1], p);
        if (cudaGetLastError() != cudaSuccess) return RPX_ERR_CUDA;
    }
    return RPX_OK;
}

}  // namespace

rpx_status_t launch_attention_backward(const AttnBwdArgs& a) {
    if (a.total_tokens == 0 || a.batch == 0 || a.max_seqlen == 0) return RPX_OK;
    if (a.head_dim == 128) return launch_d<128>(a);
    if (a.head_dim == 64) return launch_d<64>(a);
    return RPX_ERR_SHAPE;
}

}  // namespace rpx
