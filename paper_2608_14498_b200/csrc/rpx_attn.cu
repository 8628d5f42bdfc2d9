// Varlen causal GQA flash attention for sm_100a, shared by the prefix pass (which also writes the
// paged boundary-KV cache) and the suffix pass (which reads it back through the block table).
//
// A work item is two adjacent 128-row query tiles of one (sequence, query head); the kernel is
// persistent (one CTA per SM) and its CTAs draw items, longest first, from a device counter.  For an
// item the CTA walks the key tiles (128 keys) that those rows may see: first the cached prefix tiles (suffix pass only,
// unmasked except the last partial one), then the self tiles up to each query tile's diagonal.
//   warps 0-3 : softmax of query tile 0: thread = one row = one TMEM lane, all 128 scores of the
//               row in registers (two threads per row were tried: the extra exchange of the row
//               maximum cost more than the shorter dependency chains gained)
//   warps 4-7 : softmax of query tile 1
//   warp  8   : TMA producer (Q once; K/V through a 4-slot ring; paged tiles = one TMA box per
//               16-token page); it also stores the diagonal K/V tiles into the paged cache
//   warp  9   : TMEM owner and tcgen05 issuer:  S_t = Q_t K^T  (smem x smem -> TMEM),
//               O_t += P_t V  (P_t = bf16 probabilities written back into the first 64 columns
//               of S_t's TMEM region and consumed as the TMEM A operand; V straight from its
//               [keys][d] tile as an MN-major B operand)
//   warps 10-11: fill the producer's and the issuer's warp group: after setup that group hands most of its registers
//               to the two softmax warp groups (setmaxnreg), whose step keeps 128 scores and their exponentials live
// The two query tiles alternate on the tensor core in the order PV_0(j) QK_0(j+1) PV_1(j)
// QK_1(j+1): while the softmax warps of one tile work on S_t, the tensor core runs the other
// tile's two MMAs; issuing PV_t(j) before QK_t(j+1) also orders the read of P_t before the
// overwrite of S_t.  Scores are kept in log2 units; O is rescaled lazily (only when a row's
// running max grows by more than 2^8).
#include <math_constants.h>

#include <type_traits>

#include "rpx_internal.h"
#include "rpx_ptx.cuh"

namespace rpx {

namespace {

constexpr int kTileQ = 128, kTileK = 128, kPage = 16;
constexpr int kSlots = 4;  // K/V tiles in flight (two key steps); a fifth slot measured no faster
constexpr int kMaxSplits = 4;  // ranges an item's cached prefix may be cut into
constexpr int kItemRing = 4;  // work-item ids the producer may hand out ahead of the slowest warp
constexpr int kChunks = kTileK / 32;  // 32-column TMEM loads per row and step
constexpr int kWarpsPerTile = 4;
constexpr int kProducerWarp = 2 * kWarpsPerTile, kMmaWarp = kProducerWarp + 1;
// Three warp groups of four: the eight softmax warps, then the producer, the issuer and two warps that only take part
// in the register hand-over (setmaxnreg works on whole warp groups).
constexpr int kThreads = 32 * 12;
// Registers per thread after the hand-over (256 softmax threads, 128 others; the SM has 65536).  The prefix pass's
// branch-free softmax step wants as many as it can get (208 + 80); in passes over cached tiles the producer's paged
// loads set the pace and it must not be squeezed (184 + 128): measured, the other way round loses 3 - 7 % each.
template <bool kFastSteps> struct Regs {
    static constexpr int kSoftmax = kFastSteps ? 208 : 184, kOther = kFastSteps ? 80 : 128;
};
constexpr uint32_t kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;
#ifndef RPX_POLY_PAIRS_OF_4
#define RPX_POLY_PAIRS_OF_4 1
#endif
constexpr int kPolyPairsOf4 = RPX_POLY_PAIRS_OF_4;  // of every 4 element pairs, how many take the polynomial exp2

struct Ctl {
    uint64_t q_full;
    uint64_t kv_full[kSlots];
    uint64_t kv_empty[kSlots];
    uint64_t s_full[2];   // tensor core -> softmax: S_t(j) is in TMEM (and PV_t(j-1) has finished)
    uint64_t p_ready[2];  // softmax -> tensor core: P_t(j) is in TMEM, O_t rescaled if needed
    uint64_t o_done[2];   // tensor core -> softmax: the last PV_t of the work item has finished
    uint64_t o_free[2];   // softmax -> tensor core: O_t of the finished item has been read out of TMEM
    uint64_t q_empty;     // tensor core -> producer: the item's last Q K^T has finished, Q may be overwritten
    uint64_t item_full[kItemRing];   // producer -> everyone: item_id[k] holds the next work item
    uint64_t item_empty[kItemRing];  // everyone -> producer: item_id[k] has been read
    int4 item_rec[kItemRing];        // (item number or -1, first token, query length, cached prefix length)
    uint64_t drain;
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t drain_flag;
    uint32_t data_error;
};

template <int D>
struct Layout {
    static constexpr int kHalves = D / 64;               // 64-element (128-byte) column blocks
    static constexpr int kHalfBytes = kTileK * 128;      // one [128 rows][64 bf16] swizzled block
    static constexpr int kQBytes = kHalves * kHalfBytes; // one query tile
    static constexpr int kKvBytes = kHalves * kHalfBytes;
    static constexpr int kQOff = 0;
    static constexpr int kKvOff = 2 * kQBytes;
    static constexpr int kCtlOff = kKvOff + kSlots * kKvBytes;
    static constexpr size_t kSmemBytes = kCtlOff + sizeof(Ctl);  // the dynamic window is declared 1024-aligned
};

struct Params {
    const int32_t* cu_seqlens;
    const int32_t* prefix_lens;   // NULL: no cached prefix (prefix pass)
    const int32_t* block_table;
    int32_t block_table_stride;
    int64_t num_blocks;
    __nv_bfloat16* k_cache;       // used by the ragged-page paths
    __nv_bfloat16* v_cache;
    int32_t write_cache;          // store this call's K/V into the cache (prefix pass, chunked prefill)
    int32_t batch, num_q_heads, num_kv_heads, group;
    int32_t n_pairs;              // query tile pairs per sequence the work list covers
    // Row packing (suffix pass): a query tile holds tile_tokens = 128 / group consecutive tokens times the `group`
    // query heads of ONE KV head (row = token * group + head within the group), so a cached K/V tile is fetched once
    // per KV head instead of once per query head and a short response fills its tile.  pack == 0: a tile is 128
    // tokens of one query head.
    int32_t pack;
    int32_t tile_tokens;          // query tokens per tile: 128, or 128 / group when packed
    int32_t item_heads;           // heads the work list runs over: num_q_heads, or num_kv_heads when packed
    int32_t n_items;              // n_pairs * batch * num_q_heads
    uint32_t* next_item;          // device counter, zero before the launch: work items are handed out in order
    // Split-KV (suffix passes with few, long items): the cached prefix of an item is cut into n_splits
    // ranges taken by different CTAs; each writes an un-normalised partial, the last to arrive merges.
    int32_t n_splits;             // 1 = off
    float* part_o;                // [n_splits][tokens][H_q][D] fp32
    float2* part_ml;              // [n_splits][tokens][H_q]: (row maximum in log2 units, row sum)
    uint32_t* split_cnt;          // [tokens][H_q], zero before the launch: arrivals per 32-row group
    int64_t total_tokens;
    float scale_log2;
    float inv_scale_log2;
    void* out;                    // bf16 [tokens][H_q][D] (fp32 tensors take the CUDA-core kernel)
    float* lse;
    int32_t* status;
};

// byte offset of 16-byte chunk `cc` (0..D/8-1) of row `r` inside a swizzled [128][D] tile
__device__ __forceinline__ uint32_t swz_off(int r, int cc) {
    return static_cast<uint32_t>((cc >> 3) * (kTileK * 128) + r * 128 + (((cc & 7) ^ (r & 7)) << 4));
}

// One work item = two adjacent 128-row query tiles of one (sequence, query head).  Items are numbered
// so that late query tiles (most keys, longest work) come first; CTAs take them in that order from a
// device counter, so the longest items start first and the short ones fill the tail.
struct Item {
    int32_t pair, seq, head, kv_head, tok0, len_q, q0, len_p, n_prefix_tiles, n_tile0, n_kv;
    int32_t pt0;      // first cached tile this item walks (n_prefix_tiles counts the tiles of its range)
    int32_t x1;       // extra key steps of query tile 1 over tile 0 (0 or 1)
    int32_t split, s_eff;  // which range of the cached prefix, out of how many (1 = the whole item)
    bool active, active1;
};

// The lengths come from device memory once per item (the producer's lane 0 reads them, a tile ahead of
// everyone else, and passes them on through shared memory); the rest is arithmetic on the item number.
// Offsets that do not describe a range inside the packed tensors (a negative length, an end beyond total_tokens, a
// negative cached length, more pages than a row of the block table holds) are reported and the item is handed on
// empty, so nothing is read or written through them.
__device__ __forceinline__ int4 fetch_item(const Params& p, int32_t idx, uint32_t* data_error) {
    const int32_t seq = ((idx / p.n_splits) % (p.batch * p.item_heads)) / p.item_heads;
    const int32_t tok0 = __ldg(p.cu_seqlens + seq);
    int32_t len_q = __ldg(p.cu_seqlens + seq + 1) - tok0;
    int32_t len_p = p.prefix_lens != nullptr ? __ldg(p.prefix_lens + seq) : 0;
    // pages the block table must hold for this sequence: its cached prefix, plus its own tokens where they are stored
    const int64_t table_tokens = static_cast<int64_t>(len_p) + (p.write_cache != 0 ? len_q : 0);
    if (tok0 < 0 || len_q < 0 || static_cast<int64_t>(tok0) + len_q > p.total_tokens || len_p < 0 ||
        (p.block_table != nullptr && (table_tokens + kPage - 1) / kPage > p.block_table_stride)) {
        *data_error = 1;
        len_q = 0;
        len_p = 0;
    }
    return make_int4(idx, tok0, len_q, len_p);
}

__device__ __forceinline__ int4 read_item_rec(const int4* rec) {
    const volatile int32_t* w = reinterpret_cast<const volatile int32_t*>(rec);
    return make_int4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ Item decode_item(const Params& p, int4 rec) {
    Item it;
    const int32_t idx = rec.x / p.n_splits;  // the item's (pair, sequence, head); its splits are numbered consecutively
    it.split = rec.x % p.n_splits;
    const int32_t per_pair = p.batch * p.item_heads;
    it.pair = p.n_pairs - 1 - idx / per_pair;
    const int32_t rem = idx % per_pair;
    it.seq = rem / p.item_heads;
    it.head = rem % p.item_heads;  // packed: the KV head whose query heads share the tile
    it.kv_head = p.pack != 0 ? it.head : it.head / p.group;
    it.tok0 = rec.y;
    it.len_q = rec.z;
    it.q0 = it.pair * 2 * p.tile_tokens;
    it.active = it.q0 < it.len_q;
    it.len_p = it.active ? rec.w : 0;
    it.active1 = it.q0 + p.tile_tokens < it.len_q;
    const int32_t n_pt = (it.len_p + kTileK - 1) / kTileK;  // cached tiles of the whole prefix
    it.s_eff = max(1, min(p.n_splits, n_pt));                // a prefix shorter than n_splits tiles is cut in fewer
    if (it.split >= it.s_eff) it.active = false;
    it.pt0 = n_pt * min(it.split, it.s_eff) / it.s_eff;
    it.n_prefix_tiles = n_pt * min(it.split + 1, it.s_eff) / it.s_eff - it.pt0;
    // self key tiles each query tile walks: up to the tile that holds its last token (the last range of a split
    // item takes them, the others none)
    const int32_t last = it.split == it.s_eff - 1 ? 1 : 0;
    const int32_t self0 = (min(it.len_q, it.q0 + p.tile_tokens) + kTileK - 1) / kTileK;
    const int32_t self1 = it.active1 ? (min(it.len_q, it.q0 + 2 * p.tile_tokens) + kTileK - 1) / kTileK : self0;
    // key steps of query tile t: n_tile0 + t * x1.  (Scalars, not arrays: a small array indexed at
    // run time lives in local memory, and with nearly all L1 carved out as shared memory every such
    // load stalls the in-order warp for hundreds of cycles.)
    it.n_tile0 = it.n_prefix_tiles + last * self0;
    it.x1 = last * (self1 - self0);  // 0 or 1: a tile spans at most 128 tokens
    it.n_kv = it.n_tile0 + it.x1;
    return it;
}

// kFastSteps: also instantiate the branch-free form of the softmax step (see there); the launcher picks it for the
// prefix pass.
template <int D, bool kFastSteps>
__global__ void __launch_bounds__(kThreads, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
            const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_kc,
            const __grid_constant__ CUtensorMap tmap_vc, const Params p) {
    using L = Layout<D>;
    // Rows that see only a handful of keys (the first rows of a sequence with little or no cached
    // prefix) get no averaging over keys, so the 2^-9 rounding of each bf16 probability shows up in
    // O at full size (up to 2^-9 * |v|) and, stacked on the bf16 rounding of O itself, can pass 1e-2.
    // A query tile that holds such rows has at most two key steps (n_tile0 + t <= 2: the first CTA
    // of a sequence with at most one tile of cached prefix).  For it the probabilities are kept as
    // two bf16 terms, P = P_hi + P_lo, with P_lo in the unused upper half of S_t's columns and a
    // second PV MMA: exact to 2^-17 at the cost of at most four extra MMA groups per sequence and head.
    //
    // The CTA is persistent: it takes work items until the list is empty.  The producer warp draws the
    // item numbers from the device counter and hands them to the other warps through a small ring, so
    // it can fetch the next item's Q and first K tiles while the softmax warps still write the current
    // item's output; barrier parities run on counters that carry over from item to item.

    extern __shared__ __align__(1024) uint8_t smem[];
    if ((smem_u32(smem) & 1023u) != 0u) {  // swizzled tiles need 1024-byte alignment; never expected
        if (threadIdx.x == 0 && p.status != nullptr) atomicCAS(p.status, 0, RPX_ERR_CUDA);
        return;
    }
    Ctl* ctl = reinterpret_cast<Ctl*>(smem + L::kCtlOff);
    volatile uint32_t* abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(&ctl->q_full, 1);
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(&ctl->kv_full[s], 1);
            mbar_init(&ctl->kv_empty[s], 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(&ctl->s_full[t], 1);
            mbar_init(&ctl->p_ready[t], kWarpsPerTile);  // one arrival per softmax warp
            mbar_init(&ctl->o_done[t], 1);
        }
        for (int t = 0; t < 2; ++t) mbar_init(&ctl->o_free[t], kWarpsPerTile);
        mbar_init(&ctl->q_empty, 1);
        for (int k = 0; k < kItemRing; ++k) {
            mbar_init(&ctl->item_full[k], 1);
            mbar_init(&ctl->item_empty[k], 2 * kWarpsPerTile + 1);  // every softmax warp and the issuer
        }
        mbar_init(&ctl->drain, 1);
        ctl->abort_flag = 0;
        ctl->drain_flag = 0;
        ctl->data_error = 0;
        fence_barrier_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(&ctl->tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl->tmem_base;
    // TMEM columns: S_t at 128 t (P_t aliases its first 64), O_t at 256 + 128 t
    // The kernel starts with 168 registers per thread (65536 / 384); the producer / issuer warp group gives most of
    // its share to the two softmax warp groups, whose step keeps 128 scores and their exponentials in flight.
    // (each role states its new count at the top of its own branch, which is where the compiler looks for it)

    if (warp == kProducerWarp) {
        // =========================================================== producer warp
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(Regs<kFastSteps>::kOther));
        bool ok = true;
        if (lane == 0) {
            tma_prefetch_desc(&tmap_q);
            tma_prefetch_desc(&tmap_k);
            tma_prefetch_desc(&tmap_v);
        }
        uint32_t n_loaded = 0;  // K/V tiles loaded so far (ring position)
        uint32_t n_fetched = 0; // work items drawn so far (item ring position)
        uint32_t n_active = 0;  // of those, items with any rows (parity of the Q barriers)
        for (;;) {
            // ---- draw the next work item and hand its number to the other warps
            const uint32_t ring = n_fetched % kItemRing;
            if (!mbar_wait(&ctl->item_empty[ring], ((n_fetched / kItemRing) & 1u) ^ 1u, abort_flag)) {
                ok = false;
                break;
            }
            int4 rec = make_int4(-1, 0, 0, 0);
            if (lane == 0) {
                const int32_t idx = static_cast<int32_t>(atomicAdd(p.next_item, 1u));
                if (idx < p.n_items) rec = fetch_item(p, idx, &ctl->data_error);
                ctl->item_rec[ring] = rec;
                mbar_arrive(&ctl->item_full[ring]);
            }
            rec.x = __shfl_sync(0xffffffffu, rec.x, 0);
            rec.y = __shfl_sync(0xffffffffu, rec.y, 0);
            rec.z = __shfl_sync(0xffffffffu, rec.z, 0);
            rec.w = __shfl_sync(0xffffffffu, rec.w, 0);
            ++n_fetched;
            if (rec.x < 0) break;
            const Item it = decode_item(p, rec);
            // A sequence longer than the caller's bound would leave rows the work list never reaches: report it.
            if (it.pair == 0 && it.head == 0 && lane == 0 && it.len_q > p.n_pairs * 2 * p.tile_tokens) ctl->data_error = 1;
            if (!it.active) continue;
            const int32_t pair = it.pair, seq = it.seq, head = it.head, kv_head = it.kv_head, tok0 = it.tok0;
            const int32_t len_q = it.len_q, q0 = it.q0, len_p = it.len_p, n_prefix_tiles = it.n_prefix_tiles;
            const int32_t n_tile0 = it.n_tile0, n_kv = it.n_kv, pt0 = it.pt0, x1 = it.x1;
            const bool active1 = it.active1;
            (void)pair; (void)seq; (void)head; (void)kv_head; (void)tok0; (void)len_q; (void)q0; (void)len_p;
            (void)n_prefix_tiles; (void)n_tile0; (void)n_kv; (void)active1; (void)pt0; (void)x1;
            // ---- Q of this item, once the previous item's last Q K^T has let go of the buffer
            if (n_active > 0 && !mbar_wait(&ctl->q_empty, (n_active - 1) & 1u, abort_flag)) {
                ok = false;
                break;
            }
            if (lane == 0) {
                // packed: one box of tile_tokens tokens x group heads lands as consecutive 128-byte rows (token-major)
                const int32_t rows = p.pack != 0 ? p.tile_tokens * p.group : kTileQ;
                mbar_arrive_expect_tx(&ctl->q_full, (active1 ? 2 : 1) * L::kHalves * rows * 128);
                for (int t = 0; t < (active1 ? 2 : 1); ++t)
                    for (int hf = 0; hf < L::kHalves; ++hf)
                        tma_load_3d(smem + L::kQOff + t * L::kQBytes + hf * L::kHalfBytes, &tmap_q, &ctl->q_full, hf * 64,
                                    p.pack != 0 ? kv_head * p.group : head, tok0 + q0 + t * p.tile_tokens);
            }
        // Appending behind a cached prefix (chunked prefill) needs the chunk to start on a page edge:
        // pages are written whole or from their first row.  Anything else is reported, not written.
        const bool page_aligned = (len_p % kPage) == 0;
        if (p.write_cache != 0 && !page_aligned && lane == 0) ctl->data_error = 1;
        const bool owns_cache_write = p.write_cache != 0 && p.pack == 0 && page_aligned && (head % p.group) == 0;
        const int32_t write_page0 = len_p / kPage;  // first page of this call's own tokens
        // Block id of page `lane` of cached tile jt (lanes 0..7; 0 where the prefix has no such page).
        // Read one tile ahead, so the table's global-memory latency is off the ring's critical path.
        auto read_block_ids = [&](int32_t jt) -> int32_t {
            int32_t b = 0;
            const int32_t page = jt * (kTileK / kPage) + lane;
            if (lane < kTileK / kPage && page < (len_p + kPage - 1) / kPage)
                b = __ldg(p.block_table + static_cast<int64_t>(seq) * p.block_table_stride + page);
            return b;
        };
        int32_t blk_next = n_prefix_tiles > 0 ? read_block_ids(pt0) : 0;
        for (int32_t j = 0; ok && j < n_kv; ++j) {
            const bool from_cache = j < n_prefix_tiles;
            const int32_t jt = from_cache ? pt0 + j : j - n_prefix_tiles;  // tile index inside its key source
            uint32_t slot_k = 0, slot_v = 0;
            int32_t blk = blk_next;  // this tile's pages (cached tiles only)
            if (from_cache) {
                if (blk < 0 || blk >= p.num_blocks) {
                    ctl->data_error = 1;
                    blk = 0;
                }
                if (j + 1 < n_prefix_tiles) blk_next = read_block_ids(pt0 + j + 1);
            }
            for (int which = 0; which < 2; ++which, ++n_loaded) {  // 0 = K, 1 = V
                const uint32_t slot = n_loaded % kSlots, phase = (n_loaded / kSlots) & 1u;
                if (which == 0) slot_k = slot; else slot_v = slot;
                if (!mbar_wait(&ctl->kv_empty[slot], phase ^ 1u, abort_flag)) {
                    ok = false;
                    break;
                }
                uint8_t* dst = smem + L::kKvOff + slot * L::kKvBytes;
                if (!from_cache) {
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&ctl->kv_full[slot], L::kKvBytes);
                        for (int hf = 0; hf < L::kHalves; ++hf)
                            tma_load_3d(dst + hf * L::kHalfBytes, which == 0 ? &tmap_k : &tmap_v, &ctl->kv_full[slot],
                                        hf * 64, kv_head, tok0 + jt * kTileK);
                    }
                } else {
                    // paged tile: whole 16-token pages by TMA; the ragged last page and the rows past
                    // the prefix end by plain 16-byte copies / zero fill (a masked P of 0 must never
                    // meet a non-finite stale V row)
                    const int32_t rows_valid = min(kTileK, len_p - jt * kTileK);
                    const int32_t full_pages = rows_valid / kPage;
                    if (full_pages < kTileK / kPage) {
                        const int32_t blk_r = __shfl_sync(0xffffffffu, blk, full_pages);
                        const __nv_bfloat16* src_pool = which == 0 ? p.k_cache : p.v_cache;
                        const uint4* src = reinterpret_cast<const uint4*>(
                            src_pool + (static_cast<int64_t>(blk_r) * p.num_kv_heads + kv_head) * kPage * D);
                        const int32_t first_row = full_pages * kPage;
                        const int32_t n_chunks = (kTileK - first_row) * (D / 8);
                        for (int32_t i = lane; i < n_chunks; i += 32) {
                            const int32_t r = first_row + i / (D / 8), cc = i % (D / 8);
                            uint4 val = make_uint4(0u, 0u, 0u, 0u);
                            if (r < rows_valid) val = __ldg(src + (r - first_row) * (D / 8) + cc);
                            *reinterpret_cast<uint4*>(dst + swz_off(r, cc)) = val;
                        }
                        fence_proxy_async_smem();
                    }
                    if (lane == 0) {
                        if (full_pages > 0) mbar_arrive_expect_tx(&ctl->kv_full[slot], full_pages * kPage * D * 2);
                        else mbar_arrive(&ctl->kv_full[slot]);
                    }
                    __syncwarp();  // the byte count is armed before any copy can complete
                    if (lane < full_pages) {  // lane pg fetches page pg (it holds that page's block id)
                        for (int hf = 0; hf < L::kHalves; ++hf)
                            tma_load_4d(dst + hf * L::kHalfBytes + lane * (kPage * 128), which == 0 ? &tmap_kc : &tmap_vc,
                                        &ctl->kv_full[slot], hf * 64, 0, kv_head, blk);
                    }
                }
                __syncwarp();
            }
            // ---- boundary-KV write: the two diagonal key tiles of this pair, one writer per KV head
            if (ok && owns_cache_write && !from_cache && jt >= 2 * pair) {
                for (int which = 0; which < 2 && ok; ++which) {
                    const uint32_t idx = n_loaded - 2 + which;
                    const uint32_t slot = which == 0 ? slot_k : slot_v;
                    if (!mbar_wait(&ctl->kv_full[slot], (idx / kSlots) & 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint8_t* src = smem + L::kKvOff + slot * L::kKvBytes;
                    __nv_bfloat16* pool = which == 0 ? p.k_cache : p.v_cache;
                    const int32_t rows_valid = min(kTileK, len_q - jt * kTileK);
                    const int32_t n_pages = (rows_valid + kPage - 1) / kPage;
                    int32_t blk = 0;
                    if (lane < n_pages) {
                        blk = p.block_table[static_cast<int64_t>(seq) * p.block_table_stride + write_page0 +
                                            jt * (kTileK / kPage) + lane];
                        if (blk < 0 || blk >= p.num_blocks) {
                            ctl->data_error = 1;
                            blk = -1;
                        }
                    }
                    for (int32_t pg = 0; pg < n_pages; ++pg) {
                        const int32_t b = __shfl_sync(0xffffffffu, blk, pg);
                        if (b < 0) continue;
                        const int32_t rows = min(kPage, rows_valid - pg * kPage);
                        if (rows == kPage) {
                            if (lane == 0)
                                for (int hf = 0; hf < L::kHalves; ++hf)
                                    tma_store_4d(which == 0 ? &tmap_kc : &tmap_vc, src + hf * L::kHalfBytes + pg * (kPage * 128),
                                                 hf * 64, 0, kv_head, b);
                        } else {
                            uint4* dstp = reinterpret_cast<uint4*>(
                                pool + (static_cast<int64_t>(b) * p.num_kv_heads + kv_head) * kPage * D);
                            for (int32_t i = lane; i < rows * (D / 8); i += 32) {
                                const int32_t r = pg * kPage + i / (D / 8), cc = i % (D / 8);
                                dstp[i] = *reinterpret_cast<const uint4*>(src + swz_off(r, cc));
                            }
                        }
                    }
                    if (lane == 0) {
                        tma_store_commit();
                        tma_store_wait_read();
                    }
                    __syncwarp();
                }
            }
        }
            ++n_active;
            if (!ok) break;
        }
        if (lane == 0) tma_store_wait_all();
        if (!ok) {
            // abort: give copies already in flight a moment to land before smem is released
            const uint32_t first = n_loaded > kSlots ? n_loaded - kSlots : 0u;
            for (uint32_t i = first; i < n_loaded; ++i)
                mbar_wait(&ctl->kv_full[i % kSlots], (i / kSlots) & 1u, &ctl->drain_flag, kDrainLimitCycles);
            if (n_active > 0) mbar_wait(&ctl->q_full, (n_active - 1) & 1u, &ctl->drain_flag, kDrainLimitCycles);
        }
    } else if (warp == kMmaWarp) {
        // =========================================================== tcgen05 issuer (one thread)
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(Regs<kFastSteps>::kOther));
        if (elect_one()) {
            constexpr uint32_t idesc_qk = make_idesc_bf16(kTileQ, kTileK, false, false);
            constexpr uint32_t idesc_pv = make_idesc_bf16(kTileQ, D, false, true);
            const uint32_t q_addr = smem_u32(smem + L::kQOff);
            const uint32_t kv_addr = smem_u32(smem + L::kKvOff);
            bool ok = true;

            // descriptors: everything but the start address is constant, so keep bases and add offsets
            const uint64_t q_desc0 = make_smem_desc_sw128(q_addr, 16, 1024);
            const uint64_t k_desc0 = make_smem_desc_sw128(kv_addr, 16, 1024);             // K tile: K-major
            const uint64_t v_desc0 = make_smem_desc_sw128(kv_addr, L::kHalfBytes, 1024);  // V tile: MN-major
            uint32_t n_seen = 0;              // work items read from the item ring
            uint32_t n_active = 0;            // items with rows so far = items in which tile 0 took part
            uint32_t items1 = 0;              // items in which tile 1 took part
            uint32_t cnt0 = 0, cnt1 = 0;      // key steps tile 0 / tile 1 have been through (barrier parity)
            uint32_t kv_base = 0;             // K/V tiles consumed before this item
            for (;;) {
            const uint32_t ring = n_seen % kItemRing;
            if (!mbar_wait(&ctl->item_full[ring], (n_seen / kItemRing) & 1u, abort_flag)) {
                ok = false;
                break;
            }
            const int4 rec = read_item_rec(&ctl->item_rec[ring]);
            mbar_arrive(&ctl->item_empty[ring]);
            ++n_seen;
            if (rec.x < 0) break;
            const Item it = decode_item(p, rec);
            if (!it.active) continue;
            const int32_t pair = it.pair, seq = it.seq, head = it.head, kv_head = it.kv_head, tok0 = it.tok0;
            const int32_t len_q = it.len_q, q0 = it.q0, len_p = it.len_p, n_prefix_tiles = it.n_prefix_tiles;
            const int32_t n_tile0 = it.n_tile0, n_kv = it.n_kv, pt0 = it.pt0, x1 = it.x1;
            const bool active1 = it.active1;
            (void)pair; (void)seq; (void)head; (void)kv_head; (void)tok0; (void)len_q; (void)q0; (void)len_p;
            (void)n_prefix_tiles; (void)n_tile0; (void)n_kv; (void)active1; (void)pt0; (void)x1;
            auto issue_qk = [&](int t, uint32_t k_slot) {
                const uint64_t kd = k_desc0 + static_cast<uint64_t>(k_slot * (L::kKvBytes >> 4));
                const uint64_t qd = q_desc0 + static_cast<uint64_t>(t * (L::kQBytes >> 4));
                if (D == 128) umma_ss_k128_overwrite(tmem_base + t * 128, qd, kd, idesc_qk);
                else umma_ss_k64_overwrite(tmem_base + t * 128, qd, kd, idesc_qk);
                umma_commit(&ctl->s_full[t]);
            };
            auto issue_pv = [&](int t, uint32_t v_slot, bool accumulate) {
                // 16 keys of P = 8 TMEM columns of packed bf16 pairs; 16 keys of V = 2 KiB of rows
                const uint64_t vd = v_desc0 + static_cast<uint64_t>(v_slot * (L::kKvBytes >> 4));
                umma_ts_k128(tmem_base + 256 + t * 128, tmem_base + t * 128, vd, idesc_pv, accumulate ? 1u : 0u);
                if (it.s_eff == 1 && n_tile0 + t * x1 <= 2)  // + P_lo V, P_lo in columns 64..127 of S_t
                    umma_ts_k128(tmem_base + 256 + t * 128, tmem_base + t * 128 + 64, vd, idesc_pv, 1u);
            };

            ok = mbar_wait(&ctl->q_full, n_active & 1u, abort_flag);
            const uint32_t k0_slot = kv_base % kSlots;  // K_0 is the item's first load
            if (ok) ok = mbar_wait(&ctl->kv_full[k0_slot], (kv_base / kSlots) & 1u, abort_flag);
            if (ok) {
                tc_fence_after_sync();
                issue_qk(0, k0_slot);
                if (active1) issue_qk(1, k0_slot);
                umma_commit(&ctl->kv_empty[k0_slot]);
                if (n_kv == 1) umma_commit(&ctl->q_empty);  // no further Q K^T in this item
            }
            for (int32_t j = 0; ok && j < n_kv; ++j) {
                const uint32_t v_idx = kv_base + 2 * j + 1, kn_idx = kv_base + 2 * j + 2;
                const uint32_t v_slot = v_idx % kSlots, kn_slot = kn_idx % kSlots;
                // V_j and K_{j+1} were asked for a step ago: make sure of them BEFORE waiting for the probabilities, so
                // that the tensor core starts the moment the softmax warps arrive
                const bool have_kn = j + 1 < n_kv;
                if (!mbar_wait(&ctl->kv_full[v_slot], (v_idx / kSlots) & 1u, abort_flag) ||
                    (have_kn && !mbar_wait(&ctl->kv_full[kn_slot], (kn_idx / kSlots) & 1u, abort_flag))) {
                    ok = false;
                    break;
                }
                for (int t = 0; t < 2 && ok; ++t) {
                    if ((t == 1 && !active1) || j >= n_tile0 + t * x1) continue;
                    if (!mbar_wait(&ctl->p_ready[t], ((t ? cnt1 : cnt0) + j) & 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    if (j == 0) {
                        // the first PV of an item overwrites O_t: the previous item's output must have left TMEM
                        const uint32_t before = t ? items1 : n_active;
                        if (before > 0 && !mbar_wait(&ctl->o_free[t], (before - 1) & 1u, abort_flag)) {
                            ok = false;
                            break;
                        }
                    }
                    tc_fence_after_sync();
                    issue_pv(t, v_slot, j != 0);
                    if (j + 1 < n_tile0 + t * x1) {
                        issue_qk(t, kn_slot);  // in order behind PV_t(j): P_t is read before S_t is rewritten
                    } else {
                        umma_commit(&ctl->o_done[t]);
                    }
                }
                if (!ok) break;
                umma_commit(&ctl->kv_empty[v_slot]);
                if (have_kn) umma_commit(&ctl->kv_empty[kn_slot]);
                if (j == n_kv - 2) umma_commit(&ctl->q_empty);  // the item's last Q K^T went out in this step
            }
            if (!ok) break;
            kv_base += 2u * static_cast<uint32_t>(n_kv);
            cnt0 += static_cast<uint32_t>(n_tile0);
            if (active1) {
                cnt1 += static_cast<uint32_t>(n_tile0 + x1);
                ++items1;
            }
            ++n_active;
            }
            if (!ok) {
                umma_commit(&ctl->drain);
                mbar_wait(&ctl->drain, 0, &ctl->drain_flag, kDrainLimitCycles);
            }
        }
        __syncwarp();
    } else if (warp > kMmaWarp) {
        // warps 10 and 11: nothing to do between the register hand-over and the teardown
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(Regs<kFastSteps>::kOther));
    } else {
        // =========================================================== softmax warps
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(Regs<kFastSteps>::kSoftmax));
        const int t = warp / kWarpsPerTile;
        uint32_t n_seen = 0;  // work items read from the item ring
        uint32_t cnt = 0;     // key steps this tile has been through (barrier parity)
        uint32_t items_t = 0; // items this tile took part in
        bool ok = true;
        while (ok) {
            const uint32_t ring = n_seen % kItemRing;
            if (!mbar_wait(&ctl->item_full[ring], (n_seen / kItemRing) & 1u, abort_flag)) break;
            const int4 rec = read_item_rec(&ctl->item_rec[ring]);
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->item_empty[ring]);
            ++n_seen;
            if (rec.x < 0) break;
            const Item it = decode_item(p, rec);
            if (!it.active || (t == 1 && !it.active1)) continue;
            const int32_t pair = it.pair, seq = it.seq, head = it.head, kv_head = it.kv_head, tok0 = it.tok0;
            const int32_t len_q = it.len_q, q0 = it.q0, len_p = it.len_p, n_prefix_tiles = it.n_prefix_tiles;
            const int32_t n_tile0 = it.n_tile0, n_kv = it.n_kv, pt0 = it.pt0, x1 = it.x1;
            const bool active1 = it.active1;
            (void)pair; (void)seq; (void)head; (void)kv_head; (void)tok0; (void)len_q; (void)q0; (void)len_p;
            (void)n_prefix_tiles; (void)n_tile0; (void)n_kv; (void)active1; (void)pt0; (void)x1;
            const uint32_t quarter = warp & 3;
            const int32_t row = quarter * 32 + lane;
            // which query token and head this thread's row is: unpacked, row = token of the item's head; packed,
            // row = token * group + head within the KV head's group (rows beyond tile_tokens * group are padding)
            int32_t q_local, row_head;  // position among this call's query tokens; query head
            bool row_in_tile = true;
            if (p.pack != 0) {
                const int32_t tok = row / p.group;
                q_local = q0 + t * p.tile_tokens + tok;
                row_head = kv_head * p.group + (row - tok * p.group);
                row_in_tile = tok < p.tile_tokens;
            } else {
                q_local = q0 + t * kTileQ + row;
                row_head = head;
            }
            const uint32_t lane_addr = (quarter * 32u) << 16;
            const int32_t my_tiles = n_tile0 + t * x1;
            const uint32_t my_s = tmem_base + t * 128 + lane_addr;        // this thread's lane of S_t / P_t
            const uint32_t my_o = tmem_base + 256 + t * 128 + lane_addr;  // and of O_t
            float run_max = -CUDART_INF_F, run_sum = 0.f;
            // The whole step loop is instantiated twice, so the common (kSplit = false) instance is
            // scheduled and register-allocated exactly as if the two-term variant did not exist.
            auto run_steps = [&](auto split_tag) {
              constexpr bool kSplit = decltype(split_tag)::value;
              for (int32_t j = 0; j < my_tiles; ++j) {
                if (!mbar_wait(&ctl->s_full[t], (cnt + j) & 1u, abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                // ---- the row's 128 scores
                uint32_t sc[kChunks][32];
#pragma unroll
                for (int c = 0; c < kChunks; ++c) tmem_ld32(my_s + c * 32, sc[c]);
                tmem_ld_wait();
                // ---- how many leading keys of this tile the row may see
                int32_t n_vis;
                if (j < n_prefix_tiles) {
                    n_vis = min(kTileK, len_p - (pt0 + j) * kTileK);
                } else {
                    const int32_t jt = j - n_prefix_tiles;
                    n_vis = min(kTileK, max(0, q_local - jt * kTileK + 1));
                }
                // The step's arithmetic exists twice: the general form masks the scores a row may not see and skips
                // whole chunks nobody in the warp sees; the fast form, for tiles every row of the warp sees completely
                // (the self tiles left of the diagonal), has neither test, so the unrolled step is one basic block the
                // compiler can schedule across.  Only the prefix pass's instance of the kernel has it: passes over cached
                // tiles run at the pace of the producer's page-sized loads, and there the second copy of the step
                // measured 2 - 7 % slower.
                float alpha = 1.f;
                bool rescale = false;
                auto body = [&](auto fast_tag) {
                constexpr bool kFast = decltype(fast_tag)::value;
                if (!kFast && n_vis < kTileK) {
#pragma unroll
                    for (int c = 0; c < kChunks; ++c)
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (c * 32 + i >= n_vis) sc[c][i] = 0xff800000u;  // -inf
                }
                // keys no row of this warp may see (the upper right of a diagonal tile, the tail of the last
                // prefix tile) need no exponentials: their 32-column chunks get P = 0 directly
                const int32_t n_vis_warp = kFast ? kTileK : __reduce_max_sync(0xffffffffu, n_vis);
                // eight independent chains of three-input maxima (the maximum runs on the half-rate ALU pipe,
                // so halving its instruction count is worth more than it looks)
                float mx[8];
                auto score = [&](int e) { return __uint_as_float(sc[e >> 5][e & 31]); };
#pragma unroll
                for (int u = 0; u < 8; ++u) mx[u] = fmaxf(score(u), score(8 + u));
#pragma unroll
                for (int e = 16; e < kTileK; e += 16)
#pragma unroll
                    for (int u = 0; u < 8; ++u) mx[u] = fmax3(mx[u], score(e + u), score(e + 8 + u));
                float cmax = fmax3(fmax3(mx[0], mx[1], mx[2]), fmax3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7]));
                cmax *= p.scale_log2;  // scale > 0, so max commutes with the scaling
                // The running maximum is kept integer-valued (rounded up): any upper bound serves the softmax, and
                // an integer maximum can be folded exactly into the rounding constant of the polynomial exp2 below.
                const bool grow = cmax > run_max + kRescaleThreshold;
                const float new_max = grow ? ceilf(cmax) : run_max;
                alpha = grow ? fast_exp2(run_max - new_max) : 1.f;
                rescale = j > 0 && __any_sync(0xffffffffu, grow);
                run_sum *= alpha;
                run_max = new_max;
                // ---- P = 2^(x - max) as packed bf16 pairs over the first 64 columns of S_t
                const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2);
                const uint64_t neg_max2 = f2_pack(-run_max, -run_max);
                const uint64_t magic_max2 = f2_pack(12582912.f - run_max, 12582912.f - run_max);
                const float min_score = (run_max - 125.f) * p.inv_scale_log2;
                uint64_t part2[4] = {0ull, 0ull, 0ull, 0ull};  // four packed accumulators = eight chains
                // kSplit also writes the second bf16 term of each probability (what the first term's
                // rounding dropped) to columns 64..127, four words at a time to keep it in registers.
                {
#pragma unroll
                    for (int c = 0; c < kChunks; ++c) {
                        uint32_t packed[16];
                        uint32_t lo[4];
                        if (!kFast && c * 32 >= n_vis_warp) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) packed[i] = 0u;
                            tmem_st16(my_s + c * 16, packed);
                            if constexpr (kSplit) tmem_st16(my_s + 64 + c * 16, packed);
                            continue;
                        }
#pragma unroll
                        for (int i = 0; i < 32; i += 2) {
                            float e0, e1;
                            if (((i / 2) % 4) < kPolyPairsOf4) {  // compile-time per unrolled pair
                                // exp2 on the FMA pipe, with the scaling folded in: s * scale + (1.5 * 2^23 - max)
                                // rounds x = s * scale - max to the integer n in its low mantissa bits (the
                                // maximum is an integer, so the constant is exact); f = x - n by a second FMA;
                                // 2^f by a cubic; 2^n goes into the exponent field.  Scores are clamped so that
                                // x >= -125 (masked ones are -inf): the result is then at most 2^-125.
                                const uint64_t sp = f2_pack(fmaxf(__uint_as_float(sc[c][i]), min_score),
                                                            fmaxf(__uint_as_float(sc[c][i + 1]), min_score));
                                const uint64_t shifted = f2_fma(sp, scale2, magic_max2);
                                const uint64_t f = f2_fma(sp, scale2, f2_sub(magic_max2, shifted));
                                uint64_t pf = f2_fma(f2_pack(0.05500858f, 0.05500858f), f, f2_pack(0.24221037f, 0.24221037f));
                                pf = f2_fma(pf, f, f2_pack(0.6932829f, 0.6932829f));
                                pf = f2_fma(pf, f, f2_pack(1.0f, 1.0f));
                                float p0, p1, s0, s1;
                                f2_unpack(pf, p0, p1);
                                f2_unpack(shifted, s0, s1);
                                e0 = __uint_as_float(__float_as_uint(p0) + (__float_as_uint(s0) << 23));
                                e1 = __uint_as_float(__float_as_uint(p1) + (__float_as_uint(s1) << 23));
                            } else {
                                const uint64_t x = f2_fma(
                                    f2_pack(__uint_as_float(sc[c][i]), __uint_as_float(sc[c][i + 1])), scale2, neg_max2);
                                float x0, x1;
                                f2_unpack(x, x0, x1);
                                e0 = fast_exp2(x0);
                                e1 = fast_exp2(x1);
                            }
                            part2[(i / 2) % 4] = f2_add(part2[(i / 2) % 4], f2_pack(e0, e1));
                            const uint32_t hi = pack_bf16x2(e0, e1);
                            packed[i >> 1] = hi;
                            if constexpr (kSplit) {
                                lo[(i >> 1) & 3] = pack_bf16x2(e0 - __uint_as_float(hi << 16),
                                                               e1 - __uint_as_float(hi & 0xffff0000u));
                                if (((i >> 1) & 3) == 3) tmem_st4(my_s + 64 + c * 16 + (i >> 1) - 3, lo);
                            }
                        }
                        tmem_st16(my_s + c * 16, packed);
                    }
                }
                {
                    float a0, a1;
                    f2_unpack(f2_add(f2_add(part2[0], part2[1]), f2_add(part2[2], part2[3])), a0, a1);
                    run_sum += a0 + a1;
                }
                };
                if (kFastSteps && !kSplit && __all_sync(0xffffffffu, n_vis == kTileK)) body(std::true_type{});
                else body(std::false_type{});
                // S_t(j) was committed behind PV_t(j-1), so O_t is quiescent until this warp's arrival
                // below.  Done here,
                // after the scores are dead, so the 32 staging registers do not force spills.
                if (rescale) {
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t r[32];
                        const uint32_t addr = my_o + c * 32;
                        tmem_ld32(addr, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                        tmem_st32(addr, r);
                    }
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->p_ready[t]);
              }
            };
            if (it.s_eff == 1 && my_tiles <= 2)
                run_steps(std::true_type{});
            else
                run_steps(std::false_type{});
            // ---- epilogue: O / l -> global, LSE
            cnt += static_cast<uint32_t>(my_tiles);
            if (ok) ok = mbar_wait(&ctl->o_done[t], items_t & 1u, abort_flag);
            ++items_t;
            if (ok) {
                tc_fence_after_sync();
                const bool row_valid = row_in_tile && q_local < len_q;
                float inv = 1.f / run_sum;
                const int64_t out_row = (static_cast<int64_t>(tok0 + q_local) * p.num_q_heads + row_head) * D;
                // two chunks of 32 columns in flight: the next chunk's TMEM load runs under this chunk's stores
                uint32_t ra[32], rb[32];
                // A warp's store instruction touches 32 rows, so its cost is the number of 32-byte sectors
                // it writes: 32-byte stores (one full sector per row and instruction) halve the count
                // against 16-byte ones.  They need the output base on a 32-byte boundary.
                const bool wide = (reinterpret_cast<uintptr_t>(p.out) & 31u) == 0u;
                auto store_chunk = [&](const uint32_t (&r)[32], int c) {
                    if (!row_valid) return;
                    {
                        __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.out) + out_row + c * 32;
                        uint32_t w[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            w[i] = pack_bf16x2(__uint_as_float(r[2 * i]) * inv, __uint_as_float(r[2 * i + 1]) * inv);
                        if (wide) {
                            st_global_v8(dst, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
                            st_global_v8(dst + 16, w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]);
                        } else {
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                reinterpret_cast<uint4*>(dst)[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
                        }
                    }
                };
                if (it.s_eff > 1) {
                    // ---- one range of a split item: the un-normalised row and its (maximum, sum) go to the
                    // workspace; whichever of the s_eff CTAs arrives last for these 32 rows merges them
                    const int64_t rh = static_cast<int64_t>(tok0 + q_local) * p.num_q_heads + row_head;
                    const int64_t per_split = p.total_tokens * p.num_q_heads;
                    float* po = p.part_o + (static_cast<int64_t>(it.split) * per_split + rh) * D;
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        tmem_ld32(my_o + c * 32, ra);
                        tmem_ld_wait();
                        if (c == D / 32 - 1) {  // O_t is out of TMEM
                            tc_fence_before_sync();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&ctl->o_free[t]);
                        }
                        if (row_valid) {
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                st_global_v8(po + c * 32 + 8 * i, ra[8 * i], ra[8 * i + 1], ra[8 * i + 2], ra[8 * i + 3],
                                             ra[8 * i + 4], ra[8 * i + 5], ra[8 * i + 6], ra[8 * i + 7]);
                        }
                    }
                    // rows are ordered by token, so when lane 0's row is beyond the sequence the whole warp's are
                    const bool warp_valid = __shfl_sync(0xffffffffu, row_valid ? 1 : 0, 0) != 0;
                    if (row_valid) p.part_ml[static_cast<int64_t>(it.split) * per_split + rh] = make_float2(run_max, run_sum);
                    uint32_t arrived = 0;
                    const int64_t rh_lane0 = __shfl_sync(0xffffffffu, rh, 0);  // the 32-row group's arrival counter
                    if (warp_valid) {
                        __threadfence();
                        __syncwarp();
                        if (lane == 0) arrived = atomicAdd(p.split_cnt + rh_lane0, 1u);
                        arrived = __shfl_sync(0xffffffffu, arrived, 0);
                    }
                    if (warp_valid && arrived == static_cast<uint32_t>(it.s_eff - 1)) {
                        __threadfence();
                        float f[kMaxSplits];
                        float top = -CUDART_INF_F, total = 0.f;
                        if (row_valid) {
#pragma unroll
                            for (int sp = 0; sp < kMaxSplits; ++sp)
                                if (sp < it.s_eff)
                                    top = fmaxf(top, __ldcg(p.part_ml + static_cast<int64_t>(sp) * per_split + rh).x);
                            total = 0.f;
#pragma unroll
                            for (int sp = 0; sp < kMaxSplits; ++sp) {
                                if (sp < it.s_eff) {
                                    const float2 ml = __ldcg(p.part_ml + static_cast<int64_t>(sp) * per_split + rh);
                                    f[sp] = fast_exp2(ml.x - top);
                                    total = fmaf(f[sp], ml.y, total);
                                } else {
                                    f[sp] = 0.f;
                                }
                            }
                            inv = 1.f / total;
#pragma unroll 1
                            for (int c = 0; c < D / 32; ++c) {
#pragma unroll
                                for (int i = 0; i < 32; ++i) ra[i] = 0u;
#pragma unroll
                                for (int sp = 0; sp < kMaxSplits; ++sp) {
                                    if (sp < it.s_eff) {
                                        const float4* src = reinterpret_cast<const float4*>(
                                            p.part_o + (static_cast<int64_t>(sp) * per_split + rh) * D + c * 32);
#pragma unroll
                                        for (int i = 0; i < 8; ++i) {
                                            const float4 v = __ldcg(src + i);
                                            ra[4 * i] = __float_as_uint(fmaf(f[sp], v.x, __uint_as_float(ra[4 * i])));
                                            ra[4 * i + 1] = __float_as_uint(fmaf(f[sp], v.y, __uint_as_float(ra[4 * i + 1])));
                                            ra[4 * i + 2] = __float_as_uint(fmaf(f[sp], v.z, __uint_as_float(ra[4 * i + 2])));
                                            ra[4 * i + 3] = __float_as_uint(fmaf(f[sp], v.w, __uint_as_float(ra[4 * i + 3])));
                                        }
                                    }
                                }
                                store_chunk(ra, c);
                            }
                            if (p.lse != nullptr) p.lse[rh] = (top + log2f(total)) * kLn2;
                        }
                    }
                } else {
                tmem_ld32(my_o, ra);
#pragma unroll
                for (int c = 0; c < D / 32; c += 2) {
                    tmem_ld32(my_o + (c + 1) * 32, rb);
                    tmem_ld_wait();  // both loads: ra and rb are in registers
                    if (c + 2 >= D / 32) {  // O_t is out of TMEM: the next item's first PV may overwrite it
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&ctl->o_free[t]);
                    } else {
                        store_chunk(ra, c);
                        tmem_ld32(my_o + (c + 2) * 32, ra);
                        store_chunk(rb, c + 1);
                        continue;
                    }
                    store_chunk(ra, c);
                    store_chunk(rb, c + 1);
                }
                if (row_valid && p.lse != nullptr)
                    p.lse[static_cast<int64_t>(tok0 + q_local) * p.num_q_heads + row_head] = (run_max + log2f(run_sum)) * kLn2;
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && p.status != nullptr) {
        if (ctl->abort_flag != 0u) atomicCAS(p.status, 0, RPX_ERR_TIMEOUT);
        else if (ctl->data_error != 0u) atomicCAS(p.status, 0, RPX_ERR_DEVICE_DATA);
    }
}

template <int D>
rpx_status_t launch_attention_d(const AttnArgs& a) {
    using L = Layout<D>;
    CUtensorMap tq, tk, tv, tkc, tvc;
    const uint64_t tokens = static_cast<uint64_t>(a.total_tokens);
    // Row packing: in the suffix pass the query heads of one KV head share a tile (see Params::pack).  Not for passes
    // that store K/V (one writer per KV head is chosen among the per-head items) and pointless without grouping.
    const int32_t group = a.num_q_heads / a.num_kv_heads;
    const bool pack = a.prefix_lens != nullptr && !(a.cache != nullptr && a.append_cache) && group >= 2 && group <= kTileQ;
    const int32_t tile_tokens = pack ? kTileQ / group : kTileQ;
    {
        const uint64_t dims[3] = {D, static_cast<uint64_t>(a.num_q_heads), tokens};
        const uint64_t strides[2] = {D * 2ull, static_cast<uint64_t>(a.q_tok_stride) * 2};
        const uint32_t box[3] = {64, pack ? static_cast<uint32_t>(group) : 1u, static_cast<uint32_t>(tile_tokens)};
        if (rpx_status_t rc = encode_tmap_bf16(&tq, a.q, 3, dims, strides, box)) return rc;
    }
    {
        const uint64_t dims[3] = {D, static_cast<uint64_t>(a.num_kv_heads), tokens};
        const uint64_t ks[2] = {D * 2ull, static_cast<uint64_t>(a.k_tok_stride) * 2};
        const uint64_t vs[2] = {D * 2ull, static_cast<uint64_t>(a.v_tok_stride) * 2};
        const uint32_t box[3] = {64, 1, kTileK};
        if (rpx_status_t rc = encode_tmap_bf16(&tk, a.k, 3, dims, ks, box)) return rc;
        if (rpx_status_t rc = encode_tmap_bf16(&tv, a.v, 3, dims, vs, box)) return rc;
    }
    if (a.cache != nullptr) {
        const uint64_t dims[4] = {D, kPage, static_cast<uint64_t>(a.num_kv_heads), static_cast<uint64_t>(a.cache->num_blocks)};
        const uint64_t strides[3] = {D * 2ull, kPage * D * 2ull, static_cast<uint64_t>(a.num_kv_heads) * kPage * D * 2ull};
        const uint32_t box[4] = {64, kPage, 1, 1};
        if (rpx_status_t rc = encode_tmap_bf16(&tkc, a.cache->k_cache, 4, dims, strides, box)) return rc;
        if (rpx_status_t rc = encode_tmap_bf16(&tvc, a.cache->v_cache, 4, dims, strides, box)) return rc;
    } else {
        tkc = tk;  // never dereferenced without a cache
        tvc = tv;
    }
    Params p;
    p.cu_seqlens = a.cu_seqlens;
    p.prefix_lens = a.prefix_lens;
    p.block_table = a.cache ? a.cache->block_table : nullptr;
    p.block_table_stride = a.cache ? a.cache->block_table_stride : 0;
    p.num_blocks = a.cache ? a.cache->num_blocks : 0;
    p.k_cache = a.cache ? static_cast<__nv_bfloat16*>(a.cache->k_cache) : nullptr;
    p.v_cache = a.cache ? static_cast<__nv_bfloat16*>(a.cache->v_cache) : nullptr;
    p.write_cache = (a.cache != nullptr && (a.prefix_lens == nullptr || a.append_cache)) ? 1 : 0;
    p.batch = a.batch;
    p.num_q_heads = a.num_q_heads;
    p.num_kv_heads = a.num_kv_heads;
    p.group = group;
    p.pack = pack ? 1 : 0;
    p.tile_tokens = tile_tokens;
    p.item_heads = pack ? a.num_kv_heads : a.num_q_heads;
    p.n_pairs = (a.max_q_len + 2 * tile_tokens - 1) / (2 * tile_tokens);
    const float scale = a.softmax_scale > 0.f ? a.softmax_scale : 1.0f / sqrtf(static_cast<float>(D));
    p.scale_log2 = scale * kLog2e;
    p.inv_scale_log2 = 1.0f / p.scale_log2;
    p.out = a.out;
    p.lse = a.lse;
    p.status = a.device_status;
    const int64_t n_base = static_cast<int64_t>(p.n_pairs) * a.batch * p.item_heads;
    if (n_base <= 0) return RPX_OK;
    int sms_all = sm_count();
    if (sms_all <= 0) return RPX_ERR_CUDA;
    if (const int budget = sm_budget(); budget > 0 && budget < sms_all) sms_all = budget;
    // ---- split-KV: a suffix pass with few, long items leaves most SMs idle in its last round of items.
    // Cutting the cached prefix of every item into S ranges gives S times as many, shorter items; taken when
    // the estimated number of key steps on the busiest SM drops by more than 15 %.
    p.n_splits = 1;
    p.part_o = nullptr;
    p.part_ml = nullptr;
    p.split_cnt = nullptr;
    p.total_tokens = a.total_tokens;
    if (a.prefix_lens != nullptr && p.write_cache == 0 && a.split_ws != nullptr &&
        attn_split_workspace(a.total_tokens, a.num_q_heads, D) > 0) {
        const int64_t prefix_steps = (a.max_prefix_len + kTileK - 1) / kTileK;
        const int64_t self_steps = (static_cast<int64_t>(a.max_q_len) + kTileK - 1) / kTileK;
        // rounds of items x (key steps + about four steps' worth of fixed cost per item); with three ranges on C2's
        // suffix pass (224 items of 35 steps) the merge and the fixed costs ate the gain: 0.219 against 0.156 ms
        auto cost = [&](int64_t S) { return ((n_base * S + sms_all - 1) / sms_all) * (prefix_steps / S + 4) + self_steps; };
        int best = 1;
        for (int S = 2; S <= kMaxSplits; ++S)
            if (prefix_steps / S >= 4 && cost(S) < cost(best)) best = S;
        if (best > 1 && cost(best) * 100 < cost(1) * 85) {
            p.n_splits = best;
            const size_t rows = static_cast<size_t>(a.total_tokens) * a.num_q_heads;
            uint8_t* ws = static_cast<uint8_t*>(a.split_ws);
            p.split_cnt = reinterpret_cast<uint32_t*>(ws);
            ws += (rows * sizeof(uint32_t) + 255) / 256 * 256;
            p.part_ml = reinterpret_cast<float2*>(ws);
            ws += (kMaxSplits * rows * sizeof(float2) + 255) / 256 * 256;
            p.part_o = reinterpret_cast<float*>(ws);
            if (cudaMemsetAsync(p.split_cnt, 0, rows * sizeof(uint32_t), a.stream) != cudaSuccess) return RPX_ERR_CUDA;
        }
    }
    const int64_t n_items = n_base * p.n_splits;
    if (n_items > INT32_MAX - 65536) return RPX_ERR_SHAPE;  // the counter runs past n_items by one draw per CTA
    if (a.item_counter == nullptr) return RPX_ERR_WORKSPACE;
    p.n_items = static_cast<int32_t>(n_items);
    p.next_item = a.item_counter;
    const int sms = sms_all;  // SM count, or the caller's SM budget: the rest is left to a co-runner
    const int64_t grid = n_items < sms ? n_items : sms;  // persistent: one CTA per SM
    if (cudaMemsetAsync(a.item_counter, 0, sizeof(uint32_t), a.stream) != cudaSuccess) return RPX_ERR_CUDA;
    // the prefix pass (no cached tiles) runs the instance with the branch-free softmax step
    auto* kernel = a.prefix_lens == nullptr ? attn_kernel<D, true> : attn_kernel<D, false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(L::kSmemBytes)) !=
        cudaSuccess)
        return RPX_ERR_CUDA;
    kernel<<<static_cast<unsigned>(grid), kThreads, L::kSmemBytes, a.stream>>>(tq, tk, tv, tkc, tvc, p);
    return cudaGetLastError() == cudaSuccess ? RPX_OK : RPX_ERR_CUDA;
}

}  // namespace

size_t attn_split_workspace(int64_t tokens, int32_t num_q_heads, int32_t head_dim) {
    // worth splitting only while the items (256 rows each) do not fill the SMs a few times over anyway
    const int64_t rows = tokens * num_q_heads;
    if (tokens <= 0 || rows > 3 * 148 * 2 * kTileQ) return 0;
    const size_t r = static_cast<size_t>(rows);
    return (r * sizeof(uint32_t) + 255) / 256 * 256 + (kMaxSplits * r * sizeof(float2) + 255) / 256 * 256 +
           (kMaxSplits * r * head_dim * sizeof(float) + 255) / 256 * 256;
}

rpx_status_t launch_attention(const AttnArgs& a) {
    if (a.total_tokens == 0 || a.batch == 0 || a.max_q_len == 0) return RPX_OK;
    if (a.head_dim == 128) return launch_attention_d<128>(a);
    if (a.head_dim == 64) return launch_attention_d<64>(a);
    return RPX_ERR_SHAPE;
}

}  // namespace rpx
