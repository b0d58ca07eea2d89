// Internal declarations shared by the translation units of libvorta.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "vorta.h"

namespace vorta {

// How an attention work item addresses its rows.
enum : int32_t {
    MODE_LINEAR = 0,   // full head: 128 consecutive tokens of the original tensors per block
    MODE_TILES = 1,    // sliding head: one 3D (sub-)tile of the original tensors per block
    MODE_COMPACT = 2   // core-set head: 128 consecutive rows of the gathered tensors per block
};

constexpr int kBlockM = 128;       // query rows per M-block (one MMA M)
constexpr int kMaxBoxes = 8;       // a sliding tile is cut into at most this many TMA boxes of <= 128 tokens
constexpr int kMaxMasks = 1 + 8 * kMaxBoxes;  // column-mask classes of the sliding branch (0 = none):
                                              // which axes the grid cuts the tile on x which box of the tile
constexpr int kBoxShapes = 8;      // KV box shapes of the sliding branch: bit 2 / 1 / 0 = cut by the grid on T / H / W
constexpr int kAttnThreads = 320;  // tcgen05 kernel: 2 control warps + 2 x 4 softmax warps
constexpr int kBucketTabStride = 34;  // per bucket shape class: token count, centre, 32 token offsets

// Plain geometry, passed to kernels by value.
struct Geometry {
    int32_t B, heads;
    int32_t T, H, W, L, d;
    int32_t tile[3], nt[3], n_tiles;      // sliding tiles (T, H, W order)
    int32_t half[3], restricted[3];       // floor(w/2); 0 when the window covers the axis
    int32_t bucket[3], nb[3], n_buckets;  // core-set buckets
    int32_t Lc;
    int32_t Lt;                           // text tokens after the video tokens of every head (joint sequence)
    int32_t Ltot, Lct;                    // rows per head of Q, K, V, O (L + Lt) and of the compact tensors (Lc + Lt)
    int32_t text_blocks;                  // KV blocks of bn_tile text keys a sliding item appends: ceil(Lt / bn_tile)
    double ratio;
    // sliding branch blocking: one block = a TMA box of box[0] x box[1] x box[2] tokens
    // (T, H, W order); a tile is nbox[0] x nbox[1] x nbox[2] boxes, numbered bx = (bt * nbox[1] + bh) * nbox[2] + bw
    int32_t box[3], nbox[3], box_rows, bn_tile, boxes_per_tile, max_kv_per_tile;
};

// One KV block of a sliding-tile query: origin of its box and its column-mask class.  In the lists of
// packed items (two query tiles in one 128-row block, see WorkItem::flags) the two top bits of mask_id
// say which of the two tiles has the block in its window: 0 both, 1 only the first, 2 only the second.
struct KvEntry {
    int16_t w0, h0, t0;
    uint16_t mask_id;
};
constexpr uint32_t kMaskIdBits = 0x1fffu;
// kEntryPaired (per-tile lists only): the block is TWO boxes, this one and the same box of the next tile along W, each
// the 64-row part inside the grid of a box the grid cuts on T only (the last, short T tile): 64 + 64 real keys that
// fill a whole 128-key block, fetched by two loads into the halves of one ring slot.  Its class is 0 (a whole block).
constexpr uint32_t kEntryPaired = 0x2000u;
constexpr int kVisShift = 14;
constexpr int32_t kItemPacked = 1;      // WorkItem::flags
constexpr int32_t kItemSameWindow = 2;  // with kItemPacked: both tiles have the item's own window (see WorkItem)

// One unit of work of the attention kernel: up to two 128-row query blocks that
// walk the same sequence of KV blocks.
struct WorkItem {
    int32_t mode;
    int32_t slice;        // 5th tensor-map coordinate: b*heads + head, or the compact problem id
    int32_t n_mblk;       // 1 or 2
    int32_t kv_count;     // number of KV blocks
    int32_t kv_begin;     // MODE_TILES: first entry in the KV list
    int32_t kv_len;       // linear modes: number of keys (L or Lc)
    int32_t q_org[2][3];  // per M-block: (w0, h0, t0) of the box, or (row0, 0, 0)
    int32_t out_slice;    // slice of the output tensor the rows are written to (non-compact modes)
    int32_t kv_fast;      // the first kv_fast blocks are 128 real keys each: no column needs masking
    int32_t kv_text;      // MODE_TILES: blocks [kv_count - kv_text, kv_count) are bn_tile-key blocks of text tokens
    // kItemPacked (MODE_TILES, tiles of at most 64 tokens, n_mblk = 1): the one query block holds TWO tiles
    // that are neighbours along W, q_org[0] in rows [0, 64) and q_org[1] in rows [64, 128); the KV blocks are
    // the union of the two windows, listed in AttnParams::kv_pairs from kv_begin on.
    // kItemPacked | kItemSameWindow: the two tiles are lone, short boxes (at most 64 rows, e.g. the one valid frame of
    // the last T tile) of tiles with the SAME window: the keys are the first tile's list in AttnParams::kv_list, every
    // block is seen by both, and each box is fetched through AttnMaps::q_lone (a 64-row box).
    int32_t flags;
};
static_assert(sizeof(WorkItem) == 64, "WorkItem must stay 64 bytes");

// the KV list an item's kv_begin counts in
__host__ __device__ inline bool item_uses_pair_list(int32_t flags)
{
    return (flags & kItemPacked) && !(flags & kItemSameWindow);
}

// Tensor maps of one attention launch (all 5-D: d, W|rows, H, T, slice).
struct AttnMaps {
    CUtensorMap q[3], k[3], v[3];  // indexed by mode
    CUtensorMap kt, vt;            // text rows [L, L + Lt) of K and V in boxes of bn_tile rows (sliding items)
    CUtensorMap k_half[3];         // pair kernel: K of the linear modes in boxes of 64 rows
    // Sliding branch, KV boxes the grid cuts: one map per shape whose box is just the part inside the
    // grid (index = which axes are cut; 0 is unused, the whole box goes through k/v[MODE_TILES]), so a
    // cut box arrives as a short run of real keys instead of a 128-row box with holes.
    CUtensorMap k_cut[kBoxShapes], v_cut[kBoxShapes];
    CUtensorMap q_lone;            // Q of the sliding branch in boxes of the lone short box (kItemSameWindow)
};

struct AttnParams {
    Geometry g;
    float scale_log2;              // softmax scale * log2(e)
    const WorkItem *items;
    const int32_t *cta_begin;      // [grid] first item of each CTA
    const int32_t *cta_count;      // [grid]
    const KvEntry *kv_list;
    const KvEntry *kv_pairs;       // KV lists of the packed items
    const uint32_t *colmasks;      // [kMaxMasks][4]
    uint8_t cls_shape[kMaxMasks + 7];  // column-mask class -> box shape (0: whole box, or no short map for it)
    int16_t shape_rows[kBoxShapes];    // keys in a box of each shape (all of them real)
    int32_t lone_rows;                 // rows of a q_lone box (kItemSameWindow items)
    __nv_bfloat16 *O;              // [B*heads, L + Lt, d]
    __nv_bfloat16 *Oc;             // [n_compact, Lc + Lt, d]
    const __nv_bfloat16 *Q, *K, *V;     // originals (SIMT kernel)
    const __nv_bfloat16 *Qc, *Kc, *Vc;  // gathered (SIMT kernel)
    int32_t *status;               // device word: 0 or the code of an expired wait
#ifdef VORTA_TRACE
    long long *trace;              // [4 roles][8 blocks][8 events] cycle stamps of CTA 0 (debug builds)
#endif
};

// ---- launchers (each returns cudaGetLastError of its launch) ----------------------
cudaError_t launch_block_mask(const Geometry &g, uint8_t *bm, KvEntry *kv_list, int32_t *kv_count,
                              int32_t pair_t, cudaStream_t s);
cudaError_t launch_select(const Geometry &g, const __nv_bfloat16 *X, int32_t dx, int32_t n_prob,
                          const int32_t *prob_slice, const int32_t *seg_start, const int32_t *bucket_tab,
                          int32_t *core_idx, int32_t *src_slot, cudaStream_t s);
cudaError_t launch_gather(const Geometry &g, int32_t n_prob, const int32_t *prob_slice,
                          const int32_t *core_idx, const __nv_bfloat16 *Q, const __nv_bfloat16 *K,
                          const __nv_bfloat16 *V, __nv_bfloat16 *Qc, __nv_bfloat16 *Kc,
                          __nv_bfloat16 *Vc, cudaStream_t s);
cudaError_t launch_merge(const Geometry &g, int32_t n_prob, const int32_t *prob_slice, const int32_t *seg_start,
                         const int32_t *bucket_tab, const int32_t *src_slot, const __nv_bfloat16 *Q,
                         const __nv_bfloat16 *K, const __nv_bfloat16 *V, __nv_bfloat16 *Qc, __nv_bfloat16 *Kc,
                         __nv_bfloat16 *Vc, cudaStream_t s);
cudaError_t launch_scatter(const Geometry &g, int32_t n_prob, const int32_t *prob_slice,
                           const int32_t *src_slot, const __nv_bfloat16 *Oc, __nv_bfloat16 *O,
                           cudaStream_t s);
cudaError_t launch_mix_combine(const Geometry &g, const float *gates, const __nv_bfloat16 *branches,
                               __nv_bfloat16 *O, cudaStream_t s);
cudaError_t launch_router(const float *T, const float *WR, int32_t d_model, int32_t heads, float *gates,
                          uint8_t *routes, cudaStream_t s);
cudaError_t launch_attention_simt(const AttnParams &p, int32_t n_items, cudaStream_t s);
cudaError_t launch_attention_sm100(const AttnParams &p, const AttnMaps &maps, int32_t grid,
                                   cudaStream_t s);
cudaError_t attention_sm100_prepare();  // opt in to the kernel's dynamic shared memory
cudaError_t launch_attention_sm100_pair(const AttnParams &p, const AttnMaps &maps, int32_t grid,
                                        cudaStream_t s);  // p's work lists are indexed by CTA pair
cudaError_t attention_sm100_pair_prepare();

// Row r of an M-/KV-block -> token id; false if the row lies outside the grid/sequence.
__host__ __device__ inline bool block_row_token(const Geometry &g, int32_t mode, const int32_t org[3],
                                                int32_t len, int32_t r, int32_t *token)
{
    if (mode == MODE_TILES) {
        if (r >= g.box_rows) return false;
        int32_t lw = r % g.box[2];
        int32_t lh = (r / g.box[2]) % g.box[1];
        int32_t lt = r / (g.box[2] * g.box[1]);
        int32_t w = org[0] + lw, h = org[1] + lh, t = org[2] + lt;
        if (w >= g.W || h >= g.H || t >= g.T) return false;
        *token = (t * g.H + h) * g.W + w;
        return true;
    }
    int32_t i = org[0] + r;
    if (i >= len) return false;
    *token = i;
    return true;
}

}  // namespace vorta
