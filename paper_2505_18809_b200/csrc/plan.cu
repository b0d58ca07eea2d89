// Host side of libvorta: argument checking, geometry, work lists, tensor maps and
// the C entry points declared in vorta.h.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <functional>
#include <mutex>
#include <new>
#include <queue>
#include <unordered_map>

#include "vorta_internal.h"

using namespace vorta;

struct vorta_plan {
    Geometry g{};
    float scale = 0.f;
    bool host_only = false;
    bool pool_merge = false;  // merge the pruned tokens into their centre (mean) before attending
    int device = 0;
    int sm_count = 0;
    std::vector<uint8_t> routes;
    std::vector<int32_t> seg_start;   // per bucket: first slot of its core_idx segment
    std::vector<int32_t> kv_count;    // per query tile (read back from the device), then the leading unmasked ones
    std::vector<int32_t> core_heads;  // heads routed to core-set, ascending
    // device tables
    uint8_t *d_bm = nullptr;
    KvEntry *d_kv_list = nullptr;
    int32_t *d_kv_count = nullptr;
    uint32_t *d_colmasks = nullptr;
    // Packed query blocks (tiles of at most 64 tokens in one box): tiles 2k and 2k+1 of a row of tiles along
    // W share one 128-row query block; their KV list is the union of the two windows.  Per pair
    // ((tile_T * nt_H + tile_H) * (nt_W / 2) + k): first entry, entries, and key columns issued.
    KvEntry *d_kv_pairs = nullptr;
    std::vector<int32_t> pair_begin, pair_count;
    std::vector<int64_t> pair_keys;
    bool pack_tiles = false;
    int32_t lone_t = 0;  // frames of the lone short box of the last T tile (0: that tile has no such box); see build_list
    // KV boxes the grid cuts (sliding branch): column-mask class -> box shape, and per shape the extents
    // (T, H, W) and the number of keys of the part of the box that lies inside the grid
    uint8_t cls_shape[kMaxMasks + 7] = {};
    int16_t shape_rows[kBoxShapes] = {};
    int32_t shape_ext[kBoxShapes][3] = {};
    int32_t *d_seg_start = nullptr;
    int32_t *d_bucket_tab = nullptr;  // [8 shape classes][kBucketTabStride]
    // the ordered work of one attention launch: `routed` follows the current routes,
    // `mixture` runs every head through all three branches (built on first use)
    struct WorkList {
        WorkItem *d_items = nullptr;
        int32_t *d_cta_begin = nullptr, *d_cta_count = nullptr;
        int32_t n_items = 0;
        int32_t n_linear = 0;  // items over consecutive rows (full and core-set heads); the others are sliding tiles
        double linear_share = 0.0;  // their share of the attention work of the list
        int64_t items_cap = 0;
        double flops_issued = 0.0;
        bool built = false;
    };
    WorkList routed, mixture;  // `routed` is a copy of the active cache entry's list (the entry owns the buffers)
    // Work lists by route vector.  The router picks routes per timestep (Section 3.3) and a sampler
    // revisits few distinct vectors, so the lists of the last few are kept, each with device buffers of
    // its own: switching back to a known vector touches nothing on the device, and building a new one
    // never writes to buffers a kernel in flight may be reading (an entry is reused only after the last
    // call that used it has finished).
    struct RouteEntry {
        std::vector<uint8_t> routes;
        WorkList wl;
        std::vector<int32_t> core_heads;
        int32_t *d_core_slice = nullptr, *d_core_xslice = nullptr;
        cudaEvent_t used = nullptr;  // recorded after the last call that ran this entry's lists
        bool used_valid = false;
        uint64_t stamp = 0;          // activation order, for least-recently-used replacement
    };
    static constexpr int kRouteCache = 4;
    mutable std::vector<RouteEntry> cache;
    int cur = -1;
    uint64_t activations = 0;
    bool host_call_made = false;  // ev_out has been recorded: the groups' lists may be in use until it completes
    // The host-buffer entry point works through the heads in groups, so that the copies
    // of one group run under the kernels of another: each group has its own work list
    // and core-set problem tables, built with the routes.
    struct HostChunk {
        WorkList wl;
        std::vector<int32_t> heads;
        int32_t n_core = 0;
        int32_t *d_core_slice = nullptr, *d_core_xslice = nullptr;
        cudaEvent_t ev_in = nullptr, ev_done = nullptr;
    };
    mutable std::vector<HostChunk> chunks;
    mutable bool chunks_stale = true;  // the groups are rebuilt by the first host-buffer call after a route change
    cudaStream_t s_in = nullptr, s_out = nullptr;  // copy-in and copy-out streams of that entry point
    cudaStream_t s_alt = nullptr;                  // second kernel queue: odd groups run here, even ones on the caller's stream
    cudaEvent_t ev_start = nullptr, ev_out = nullptr;
    int32_t *d_core_slice = nullptr;  // [B * n_core]: compact problem -> b*heads + head
    int32_t *d_core_xslice = nullptr; // same for a shared X with one head
    int32_t *d_status = nullptr;
    double sliding_pairs = 0.0;  // sum over listed tile pairs of valid-token products
    int32_t kernel = VORTA_KERNEL_AUTO;
    // profiling: a ring of event sets, one per call, so that several calls can be
    // enqueued before their stage times are read
    static constexpr int kProfSlots = 64;
    mutable cudaEvent_t ev[kProfSlots][6] = {};  // 0..4 around the four stages; 5 between the two attention launches
    mutable bool ev_valid[kProfSlots][6] = {};
    mutable int64_t prof_calls = 0;  // calls recorded so far
    bool profiling = false;
    mutable int32_t last_launches = 0;
    // set when a route change failed half-way (an allocation or a copy): counts, routes and device
    // lists may then disagree, so nothing is launched until a later vorta_plan_set_routes succeeds
    bool broken = false;
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
        return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
    return fn;
}

// 5-D bf16 map (d, n1, n2, n3, slices) over a contiguous [slices, n3, n2, n1, d]
// tensor with a (64, b1, b2, b3, 1) box and the 128-byte swizzle.
// slice_rows: rows of d elements between consecutive slices (>= n1*n2*n3; the map may cover only the
// leading or, with an offset base, the trailing rows of a slice).
bool make_map(CUtensorMap *m, const void *base, int32_t d, int64_t n1, int64_t n2, int64_t n3,
              int64_t slices, int32_t b1, int32_t b2, int32_t b3, int64_t slice_rows = 0)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[5] = {(cuuint64_t)d, (cuuint64_t)n1, (cuuint64_t)n2, (cuuint64_t)n3,
                          (cuuint64_t)slices};
    cuuint64_t row = (cuuint64_t)d * 2;
    cuuint64_t strides[4] = {row, row * n1, row * n1 * n2, row * (slice_rows ? slice_rows : n1 * n2 * n3)};
    cuuint32_t box[5] = {64, (cuuint32_t)b1, (cuuint32_t)b2, (cuuint32_t)b3, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(base), dims, strides,
                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Cut a tile into equal boxes of at most 128 tokens (one MMA block of rows or keys): the fewest
// boxes, at most kMaxBoxes; among equals the split that cuts T before H before W (long rows along
// W keep the TMA boxes contiguous).  false if the tile has no such split.
bool choose_boxes(const int32_t tile[3], int32_t nbox[3])
{
    int32_t best = kMaxBoxes + 1;
    for (int32_t n2 = 1; n2 <= kMaxBoxes; ++n2) {
        if (tile[2] % n2) continue;
        for (int32_t n1 = 1; n1 * n2 <= kMaxBoxes; ++n1) {
            if (tile[1] % n1) continue;
            for (int32_t n0 = 1; n0 * n1 * n2 <= kMaxBoxes; ++n0) {
                if (tile[0] % n0) continue;
                const int64_t rows = (int64_t)(tile[0] / n0) * (tile[1] / n1) * (tile[2] / n2);
                const int32_t boxes = n0 * n1 * n2;
                // strict <: with n2 outermost and n0 innermost the first split found of a given
                // size is the one with the fewest cuts along W, then along H
                if (rows <= kBlockM && boxes < best) {
                    best = boxes;
                    nbox[0] = n0; nbox[1] = n1; nbox[2] = n2;
                }
            }
        }
    }
    return best <= kMaxBoxes;
}

int64_t keep_count(int64_t n, double r)
{
    int64_t k = (int64_t)std::floor(r * (double)n + 0.5);
    return k < 1 ? 1 : k;
}

inline int64_t align_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// Workspace layout for n_prob = B * n_core compact problems.
struct Workspace {
    int64_t core_idx, src_slot, Qc, Kc, Vc, Oc, total;
};
Workspace workspace_layout(const Geometry &g, int64_t n_prob)
{
    Workspace w{};
    int64_t off = 0;
    w.core_idx = off; off = align_up(off + n_prob * g.Lc * 4, 256);
    w.src_slot = off; off = align_up(off + n_prob * g.L * 4, 256);
    int64_t rows = align_up(n_prob * (int64_t)g.Lct * g.d * 2, 256);
    w.Qc = off; off += rows;
    w.Kc = off; off += rows;
    w.Vc = off; off += rows;
    w.Oc = off; off += rows;
    w.total = n_prob ? off : 0;
    return w;
}

int64_t tensor_bytes(const Geometry &g) { return (int64_t)g.B * g.heads * g.Ltot * g.d * 2; }

// Bytes of the three branch outputs and of the all-heads core-set scratch of a mixture call.
int64_t mixture_workspace_bytes(const Geometry &g)
{
    return workspace_layout(g, (int64_t)g.B * g.heads).total + align_up(3 * tensor_bytes(g), 256);
}

void free_device(vorta_plan *p)
{
    cudaFree(p->d_bm); cudaFree(p->d_kv_list); cudaFree(p->d_kv_count); cudaFree(p->d_colmasks);
    cudaFree(p->d_kv_pairs);
    cudaFree(p->d_seg_start); cudaFree(p->d_bucket_tab);
    cudaFree(p->mixture.d_items); cudaFree(p->mixture.d_cta_begin); cudaFree(p->mixture.d_cta_count);
    for (auto &e : p->cache) {
        cudaFree(e.wl.d_items); cudaFree(e.wl.d_cta_begin); cudaFree(e.wl.d_cta_count);
        cudaFree(e.d_core_slice); cudaFree(e.d_core_xslice);
        if (e.used) cudaEventDestroy(e.used);
    }
    p->cache.clear();
    for (auto &c : p->chunks) {
        cudaFree(c.wl.d_items); cudaFree(c.wl.d_cta_begin); cudaFree(c.wl.d_cta_count);
        cudaFree(c.d_core_slice); cudaFree(c.d_core_xslice);
        if (c.ev_in) cudaEventDestroy(c.ev_in);
        if (c.ev_done) cudaEventDestroy(c.ev_done);
    }
    p->chunks.clear();
    if (p->s_in) cudaStreamDestroy(p->s_in);
    if (p->s_out) cudaStreamDestroy(p->s_out);
    if (p->s_alt) cudaStreamDestroy(p->s_alt);
    if (p->ev_start) cudaEventDestroy(p->ev_start);
    if (p->ev_out) cudaEventDestroy(p->ev_out);
    cudaFree(p->d_status);
    for (auto &set : p->ev)
        for (auto &e : set)
            if (e) cudaEventDestroy(e);
}

// valid tokens of tile `id` on axis a
inline int32_t tile_valid(const Geometry &g, int a, int32_t id)
{
    const int32_t dim[3] = {g.T, g.H, g.W};
    return std::min(g.tile[a], dim[a] - id * g.tile[a]);
}

// sum over (query tile, key tile in its window) of valid(q) * valid(k); separable per axis
double sliding_valid_pairs(const Geometry &g)
{
    double total = 1.0;
    for (int a = 0; a < 3; ++a) {
        double s = 0.0;
        for (int32_t q = 0; q < g.nt[a]; ++q) {
            int32_t lo = 0, hi = g.nt[a] - 1;
            if (g.restricted[a]) {
                int32_t c = std::min(std::max(q, g.half[a]), g.nt[a] - 1 - g.half[a]);
                lo = c - g.half[a];
                hi = c + g.half[a];
            }
            double keys = 0.0;
            for (int32_t k = lo; k <= hi; ++k) keys += tile_valid(g, a, k);
            s += (double)tile_valid(g, a, q) * keys;
        }
        total *= s;
    }
    return total;
}

// Key columns the tensor-core kernel issues for the window of query tile qt: whole boxes count
// bn_tile columns, a box the grid cuts counts the keys of its part inside the grid, rounded up to the
// MMA granularity of 16 (classes without a short map keep the whole box).
int64_t tile_issued_keys(const vorta_plan *p, int32_t qt)
{
    const Geometry &g = p->g;
    const int32_t dim[3] = {g.T, g.H, g.W};
    const int32_t q[3] = {qt / (g.nt[2] * g.nt[1]), (qt / g.nt[2]) % g.nt[1], qt % g.nt[2]};
    int32_t lo[3], hi[3];
    for (int a = 0; a < 3; ++a) {
        lo[a] = 0;
        hi[a] = g.nt[a] - 1;
        if (g.restricted[a]) {
            const int32_t c = std::min(std::max(q[a], g.half[a]), g.nt[a] - 1 - g.half[a]);
            lo[a] = c - g.half[a];
            hi[a] = c + g.half[a];
        }
    }
    int64_t keys = 0;
    for (int32_t kt = lo[0]; kt <= hi[0]; ++kt)
        for (int32_t kh = lo[1]; kh <= hi[1]; ++kh)
            for (int32_t kw = lo[2]; kw <= hi[2]; ++kw) {
                const int32_t k[3] = {kt, kh, kw};
                int32_t code = 0;
                for (int a = 0; a < 3; ++a)
                    if (dim[a] - k[a] * g.tile[a] < g.tile[a]) code |= 4 >> a;
                for (int32_t bx = 0; bx < g.boxes_per_tile; ++bx) {
                    const int32_t b[3] = {bx / (g.nbox[1] * g.nbox[2]), (bx / g.nbox[2]) % g.nbox[1], bx % g.nbox[2]};
                    bool inside = true;
                    for (int a = 0; a < 3; ++a) inside = inside && k[a] * g.tile[a] + b[a] * g.box[a] < dim[a];
                    if (!inside) continue;
                    const int32_t shape = code ? p->cls_shape[1 + code * g.boxes_per_tile + bx] : 0;
                    if (!shape) { keys += g.bn_tile; continue; }
                    const int32_t n = (p->shape_rows[shape] + 15) / 16 * 16;
                    keys += (g.bn_tile > 64 && n < 32) ? 32 : n;  // two sub-blocks per block: at least 16 columns each
                }
            }
    return keys;
}

// host -> device on the plan's copy stream (the caller waits for that stream before the data are used)
cudaError_t upload(vorta_plan *p, void *dst, const void *src, size_t bytes)
{
    return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, p->s_in);
}

// window of query tile index q on axis a: key tiles [lo, hi]
inline void tile_window(const Geometry &g, int a, int32_t q, int32_t &lo, int32_t &hi)
{
    lo = 0;
    hi = g.nt[a] - 1;
    if (g.restricted[a]) {
        const int32_t c = std::min(std::max(q, g.half[a]), g.nt[a] - 1 - g.half[a]);
        lo = c - g.half[a];
        hi = c + g.half[a];
    }
}

// KV lists of the packed query blocks (see vorta_plan::d_kv_pairs): the blocks both tiles have in their
// windows first (a row's first block must hold a key for it), then those only one of them has, marked.
int build_pair_lists(vorta_plan *p)
{
    const Geometry &g = p->g;
    p->pack_tiles = g.boxes_per_tile == 1 && g.box_rows <= 64 && g.nt[2] >= 2;
    if (!p->pack_tiles) return VORTA_OK;
    const int32_t dim[3] = {g.T, g.H, g.W};
    const int32_t per_row = g.nt[2] / 2;
    std::vector<KvEntry> all;
    for (int32_t qt = 0; qt < g.nt[0]; ++qt)
        for (int32_t qh = 0; qh < g.nt[1]; ++qh)
            for (int32_t k = 0; k < per_row; ++k) {
                int32_t lo[3], hi[3], loB, hiB;
                tile_window(g, 0, qt, lo[0], hi[0]);
                tile_window(g, 1, qh, lo[1], hi[1]);
                tile_window(g, 2, 2 * k, lo[2], hi[2]);
                tile_window(g, 2, 2 * k + 1, loB, hiB);
                p->pair_begin.push_back((int32_t)all.size());
                int64_t keys = 0;
                for (int pass = 0; pass < 2; ++pass)
                    for (int32_t kt = lo[0]; kt <= hi[0]; ++kt)
                        for (int32_t kh = lo[1]; kh <= hi[1]; ++kh)
                            for (int32_t kw = std::min(lo[2], loB); kw <= std::max(hi[2], hiB); ++kw) {
                                const bool inA = kw >= lo[2] && kw <= hi[2], inB = kw >= loB && kw <= hiB;
                                const uint32_t vis = inA && inB ? 0u : (inA ? 1u : 2u);
                                if ((vis == 0) != (pass == 0)) continue;
                                const int32_t kk[3] = {kt, kh, kw};
                                int32_t code = 0;
                                for (int a = 0; a < 3; ++a)
                                    if (dim[a] - kk[a] * g.tile[a] < g.tile[a]) code |= 4 >> a;
                                const bool whole = code == 0 && g.box_rows == g.bn_tile;
                                const uint32_t id = whole ? 0u : (uint32_t)(1 + code);  // one box per tile
                                KvEntry e;
                                e.w0 = (int16_t)(kw * g.tile[2]);
                                e.h0 = (int16_t)(kh * g.tile[1]);
                                e.t0 = (int16_t)(kt * g.tile[0]);
                                e.mask_id = (uint16_t)(id | (vis << kVisShift));
                                all.push_back(e);
                                const int32_t shape = p->cls_shape[id];
                                keys += shape ? (p->shape_rows[shape] + 15) / 16 * 16 : g.bn_tile;
                            }
                // The first block of a list must hold a key for every row of the query block.  Two windows with
                // no tile in common (a window of one tile along W) give no such block: the pair is not packed.
                bool shared = false;
                for (size_t i = (size_t)p->pair_begin.back(); i < all.size(); ++i) shared = shared || (all[i].mask_id >> kVisShift) == 0;
                if (!shared) all.resize((size_t)p->pair_begin.back());
                p->pair_count.push_back((int32_t)all.size() - p->pair_begin.back());
                p->pair_keys.push_back(keys);
            }
    if (all.empty()) { p->pack_tiles = false; return VORTA_OK; }  // no pair can be packed
    if (cudaMalloc(&p->d_kv_pairs, sizeof(KvEntry) * all.size()) != cudaSuccess ||
        cudaMemcpy(p->d_kv_pairs, all.data(), sizeof(KvEntry) * all.size(), cudaMemcpyHostToDevice) != cudaSuccess)
        return VORTA_ERR_CUDA;
    return VORTA_OK;
}

// Build the ordered work list of one attention launch and upload it.  `branches[h]` is a
// bit set of the branches head h runs (bit r = route r); a head with several branches
// writes branch r to output slice r * B * heads + (b * heads + h).  Core-set problems are
// numbered b * n_core + k over the heads that have the core-set bit, in ascending order.
int build_list(vorta_plan *p, vorta_plan::WorkList &wl, const std::vector<uint8_t> &branches, bool by_branch)
{
    const Geometry &g = p->g;
    std::vector<int32_t> core_heads;
    for (int32_t h = 0; h < g.heads; ++h)
        if (branches[h] & (1u << VORTA_ROUTE_CORESET)) core_heads.push_back(h);
    const int32_t n_core = (int32_t)core_heads.size();
    const int32_t BH = g.B * g.heads;
    std::vector<WorkItem> items;
    std::vector<double> cost;
    std::vector<int64_t> item_keys;    // key columns issued per query block of the item
    std::vector<int64_t> issued_keys;  // per query tile (sliding branch)
    bool any_sliding = false;
    for (int32_t h = 0; h < g.heads; ++h) any_sliding = any_sliding || (branches[h] & (1u << VORTA_ROUTE_SLIDING));
    if (any_sliding) {
        issued_keys.resize(g.n_tiles);
        for (int32_t qt = 0; qt < g.n_tiles; ++qt) issued_keys[qt] = tile_issued_keys(p, qt);
    }
    // query rows [q0, q1) of a sequence of `len` keys, two 128-row blocks per item
    auto linear_items = [&](int32_t mode, int32_t slice, int32_t out_slice, int32_t len, int32_t q0, int32_t q1) {
        int32_t nblk = (q1 - q0 + kBlockM - 1) / kBlockM;
        int32_t kv = (len + kBlockM - 1) / kBlockM;
        for (int32_t b0 = 0; b0 < nblk; b0 += 2) {
            WorkItem w{};
            w.mode = mode; w.slice = slice; w.out_slice = out_slice; w.kv_count = kv; w.kv_len = len;
            w.kv_fast = len % kBlockM ? kv - 1 : kv;
            w.n_mblk = std::min(2, nblk - b0);
            for (int m = 0; m < w.n_mblk; ++m) w.q_org[m][0] = q0 + (b0 + m) * kBlockM;
            items.push_back(w);
            item_keys.push_back((int64_t)kv * kBlockM);
            cost.push_back((double)w.n_mblk * kv + 2.0);
        }
    };
    for (int32_t b = 0; b < g.B; ++b) {
        for (int32_t h = 0; h < g.heads; ++h) {
            const int32_t slice = b * g.heads + h;
            if (branches[h] & (1u << VORTA_ROUTE_FULL))
                linear_items(MODE_LINEAR, slice, by_branch ? VORTA_ROUTE_FULL * BH + slice : slice, g.Ltot, 0, g.Ltot);
            if (branches[h] & (1u << VORTA_ROUTE_SLIDING)) {
                std::unordered_map<int64_t, size_t> lone;  // window centre -> item holding one lone box so far
                for (int32_t qt = 0; qt < g.n_tiles; ++qt) {
                    int32_t q[3] = {qt / (g.nt[2] * g.nt[1]), (qt / g.nt[2]) % g.nt[1], qt % g.nt[2]};
                    const int32_t pi = (q[0] * g.nt[1] + q[1]) * (g.nt[2] / 2) + q[2] / 2;
                    if (p->pack_tiles && q[2] < (g.nt[2] & ~1) && p->pair_count[pi] > 0) {
                        // tiles of at most 64 tokens: this tile and its right-hand neighbour in one query block
                        if (q[2] & 1) continue;  // taken with the tile before it
                        WorkItem w{};
                        w.mode = MODE_TILES; w.slice = slice;
                        w.out_slice = by_branch ? VORTA_ROUTE_SLIDING * BH + slice : slice;
                        w.flags = kItemPacked;
                        w.kv_text = g.text_blocks;
                        w.kv_count = p->pair_count[pi] + w.kv_text;
                        w.kv_fast = 0;
                        w.kv_begin = p->pair_begin[pi];
                        w.n_mblk = 1;
                        for (int t = 0; t < 2; ++t) {
                            w.q_org[t][0] = (q[2] + t) * g.tile[2];
                            w.q_org[t][1] = q[1] * g.tile[1];
                            w.q_org[t][2] = q[0] * g.tile[0];
                        }
                        items.push_back(w);
                        item_keys.push_back(p->pair_keys[pi] + (int64_t)w.kv_text * g.bn_tile);
                        cost.push_back((double)item_keys.back() / 128.0 + 2.0);
                        continue;
                    }
                    // the boxes of the tile that start inside the grid, two per item
                    int32_t org[kMaxBoxes][3], nb = 0;
                    for (int32_t bx = 0; bx < g.boxes_per_tile; ++bx) {
                        const int32_t bb[3] = {bx / (g.nbox[1] * g.nbox[2]), (bx / g.nbox[2]) % g.nbox[1], bx % g.nbox[2]};
                        const int32_t o3[3] = {q[0] * g.tile[0] + bb[0] * g.box[0], q[1] * g.tile[1] + bb[1] * g.box[1],
                                               q[2] * g.tile[2] + bb[2] * g.box[2]};
                        if (o3[0] >= g.T || o3[1] >= g.H || o3[2] >= g.W) continue;
                        org[nb][0] = o3[2]; org[nb][1] = o3[1]; org[nb][2] = o3[0];  // (w0, h0, t0)
                        ++nb;
                    }
                    for (int32_t b0 = 0; b0 < nb; b0 += 2) {
                        WorkItem w{};
                        w.mode = MODE_TILES; w.slice = slice;
                        w.out_slice = by_branch ? VORTA_ROUTE_SLIDING * BH + slice : slice;
                        // the boxes of the window, then every text key in blocks of bn_tile
                        w.kv_text = g.text_blocks;
                        w.kv_count = p->kv_count[qt] + w.kv_text;
                        w.kv_fast = g.bn_tile == kBlockM ? p->kv_count[g.n_tiles + qt] : 0;
                        w.kv_begin = qt * g.max_kv_per_tile;
                        w.kv_len = 0;
                        w.n_mblk = std::min(2, nb - b0);
                        for (int m = 0; m < w.n_mblk; ++m)
                            for (int a = 0; a < 3; ++a) w.q_org[m][a] = org[b0 + m][a];
                        if (w.n_mblk == 1) {
                            // A lone box (the one box of a tile the grid cuts down to one, e.g. the last, one-frame
                            // T tile of the 720p grids) would run with one of the two softmax groups idle.  Tiles
                            // whose windows have the same centre tile on every axis (neighbours at a border of the
                            // tile grid) have the SAME key list: two lone boxes of such tiles share an item.
                            int64_t key = 0;
                            for (int a = 0; a < 3; ++a) {
                                const int32_t c = g.restricted[a] ? std::min(std::max(q[a], g.half[a]), g.nt[a] - 1 - g.half[a]) : 0;
                                key = key * 65536 + c;
                            }
                            // (a lone box of at most 64 rows: two of those even fit ONE query block, rows 0-63 and
                            // 64-127; short boxes only pair with short boxes)
                            const bool shorty = p->lone_t > 0 && nb == 1 && q[0] == g.nt[0] - 1;
                            key = key * 2 + (shorty ? 1 : 0);
                            auto it = lone.find(key);
                            if (it != lone.end()) {
                                WorkItem &first = items[it->second];
                                for (int a = 0; a < 3; ++a) first.q_org[1][a] = w.q_org[0][a];
                                if (shorty) {
                                    first.flags = kItemPacked | kItemSameWindow;
                                    cost[it->second] = 1.3 * (double)item_keys[it->second] / 128.0 + 2.0;
                                } else {
                                    first.n_mblk = 2;
                                    cost[it->second] = 2.0 * (double)item_keys[it->second] / 128.0 + 2.0;
                                }
                                lone.erase(it);
                                continue;
                            }
                            lone[key] = items.size();
                        }
                        items.push_back(w);
                        item_keys.push_back(issued_keys[qt] + (int64_t)w.kv_text * g.bn_tile);
                        cost.push_back((double)w.n_mblk * (double)item_keys.back() / 128.0 + 2.0);
                    }
                }
                // the text queries of a sliding head see every key: linear items over rows [L, L + Lt)
                if (g.Lt > 0)
                    linear_items(MODE_LINEAR, slice, by_branch ? VORTA_ROUTE_SLIDING * BH + slice : slice, g.Ltot,
                                 g.L, g.Ltot);
            }
            if (branches[h] & (1u << VORTA_ROUTE_CORESET)) {
                int32_t k = (int32_t)(std::find(core_heads.begin(), core_heads.end(), h) - core_heads.begin());
                linear_items(MODE_COMPACT, b * n_core + k, 0, g.Lct, 0, g.Lct);
            }
        }
    }
    // issued tensor-core work: per query block of 128 rows a QK^T and a PV over the item's key columns
    double issued = 0.0;
    for (size_t i = 0; i < items.size(); ++i) issued += (double)items[i].n_mblk * 4.0 * kBlockM * (double)item_keys[i] * g.d;

    // Longest-processing-time assignment of items to the persistent CTAs.  Three lists share the
    // device arrays: every item over the CTAs (the single-CTA kernel alone); and, for the hybrid
    // mode, the items over consecutive rows over the CTA PAIRS (pair kernel) followed by the sliding
    // items over the CTAs (single-CTA kernel beside it).  Items: [0, n) | [n, n + n_linear) |
    // [n + n_linear, 2n); begin/count: [0, grid) | [grid, grid + grid/2) | [grid + grid/2, 2 grid + grid/2).
    const int32_t grid = p->sm_count, n_pairs = grid / 2;
    std::vector<int32_t> order(items.size());
    for (size_t i = 0; i < order.size(); ++i) order[i] = (int32_t)i;
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return cost[a] > cost[b]; });
    std::vector<WorkItem> sorted;
    sorted.reserve(2 * items.size());
    const int32_t n_bins = 2 * grid + n_pairs;
    std::vector<int32_t> begin(n_bins), count(n_bins);
    // which: 0 every item, 1 the linear ones, 2 the sliding ones
    auto assign = [&](int32_t bins, int32_t first_bin, int which) {
        typedef std::pair<double, int32_t> Load;
        std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
        for (int32_t c = 0; c < bins; ++c) heap.push(Load(0.0, c));
        std::vector<std::vector<int32_t>> per_bin(bins);
        for (int32_t i : order) {
            const bool tiles = items[i].mode == MODE_TILES;
            if ((which == 1 && tiles) || (which == 2 && !tiles)) continue;
            Load l = heap.top();
            heap.pop();
            per_bin[l.second].push_back(i);
            heap.push(Load(l.first + cost[i], l.second));
        }
        const size_t base = sorted.size();
        for (int32_t c = 0; c < bins; ++c) {
            begin[first_bin + c] = (int32_t)(sorted.size() - base);
            count[first_bin + c] = (int32_t)per_bin[c].size();
            for (int32_t i : per_bin[c]) sorted.push_back(items[i]);
        }
        return (int32_t)(sorted.size() - base);
    };
    assign(grid, 0, 0);
    const int32_t n_linear = assign(n_pairs, grid, 1);
    assign(grid, grid + n_pairs, 2);
    double cost_all = 0.0, cost_linear = 0.0;
    for (size_t i = 0; i < items.size(); ++i) {
        cost_all += cost[i];
        if (items[i].mode != MODE_TILES) cost_linear += cost[i];
    }
    const double linear_share = cost_all > 0.0 ? cost_linear / cost_all : 0.0;
    wl.built = false;  // until the new lists are on the device

    if (!wl.d_cta_begin &&
        (cudaMalloc(&wl.d_cta_begin, sizeof(int32_t) * n_bins) != cudaSuccess ||
         cudaMalloc(&wl.d_cta_count, sizeof(int32_t) * n_bins) != cudaSuccess))
        return VORTA_ERR_CUDA;
    if ((int64_t)sorted.size() > wl.items_cap) {
        cudaFree(wl.d_items);
        wl.d_items = nullptr;
        wl.items_cap = (int64_t)sorted.size();
        if (cudaMalloc(&wl.d_items, sizeof(WorkItem) * std::max<size_t>(sorted.size(), 1)) != cudaSuccess)
            return VORTA_ERR_CUDA;
    }
    // Copies on the plan's own (non-blocking) copy stream, and a wait for just these copies: a plain
    // cudaMemcpy would queue behind everything in the legacy default stream, i.e. behind the attention
    // kernels of the step still running.  The destinations are not in use (see RouteEntry).
    if (!sorted.empty() && upload(p, wl.d_items, sorted.data(), sizeof(WorkItem) * sorted.size()) != cudaSuccess)
        return VORTA_ERR_CUDA;
    if (upload(p, wl.d_cta_begin, begin.data(), sizeof(int32_t) * n_bins) != cudaSuccess ||
        upload(p, wl.d_cta_count, count.data(), sizeof(int32_t) * n_bins) != cudaSuccess ||
        cudaStreamSynchronize(p->s_in) != cudaSuccess)
        return VORTA_ERR_CUDA;
    // the counts follow the device lists: set only now that every allocation and copy has succeeded
    wl.n_items = (int32_t)items.size();
    wl.n_linear = n_linear;
    wl.linear_share = linear_share;
    wl.flops_issued = issued;
    wl.built = true;
    return VORTA_OK;
}

// Groups of heads for the host-buffer entry point.  Heads are taken in descending order of
// attention work and cut into at most kHostChunks groups: the expensive groups run first, so
// the kernels always have a group to work on while the copy engine brings in the cheap ones.
// The first group's copy in and the last group's copy out are the only transfers nothing
// overlaps, so the first groups are small (1, then 2 heads) and so is the last (1 head); the
// heads between are split evenly.
constexpr int kHostChunks = 12;  // measured: 8 and 16 groups are 2 % slower end to end at hunyuan-720p

std::vector<int32_t> host_chunk_sizes(int32_t heads)
{
    std::vector<int32_t> sizes;
    if (heads < 2 * kHostChunks) {  // few heads: equal groups
        const int32_t n = std::min<int32_t>(kHostChunks, heads), per = (heads + n - 1) / n;
        for (int32_t left = heads; left > 0; left -= per) sizes.push_back(std::min(per, left));
        return sizes;
    }
    sizes = {1, 2};
    const int32_t mid = heads - 4, n_mid = kHostChunks - 3;
    for (int32_t i = 0; i < n_mid; ++i) sizes.push_back(mid / n_mid + (i < mid % n_mid ? 1 : 0));
    sizes.push_back(1);
    return sizes;
}

int build_host_chunks(vorta_plan *p)
{
    const Geometry &g = p->g;
    // the groups' lists and tables are rewritten in place: the last host-buffer call must be through with them
    if (p->host_call_made && cudaEventSynchronize(p->ev_out) != cudaSuccess) return VORTA_ERR_CUDA;
    std::vector<double> cost(g.heads);
    for (int32_t h = 0; h < g.heads; ++h) {
        const uint8_t r = p->routes[h];
        cost[h] = r == VORTA_ROUTE_FULL ? (double)g.Ltot * g.Ltot
                  : r == VORTA_ROUTE_SLIDING ? p->sliding_pairs + (double)g.L * g.Lt + (double)g.Lt * g.Ltot
                                             : (double)g.Lct * g.Lct;
    }
    std::vector<int32_t> order(g.heads);
    for (int32_t h = 0; h < g.heads; ++h) order[h] = h;
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return cost[a] > cost[b]; });
    const std::vector<int32_t> sizes = host_chunk_sizes(g.heads);
    const int32_t per = *std::max_element(sizes.begin(), sizes.end());
    const size_t want = sizes.size();
    while (p->chunks.size() < want) {
        p->chunks.emplace_back();
        vorta_plan::HostChunk &c = p->chunks.back();
        if (cudaEventCreateWithFlags(&c.ev_in, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c.ev_done, cudaEventDisableTiming) != cudaSuccess ||
            cudaMalloc(&c.d_core_slice, sizeof(int32_t) * g.B * per) != cudaSuccess ||
            cudaMalloc(&c.d_core_xslice, sizeof(int32_t) * g.B * per) != cudaSuccess)
            return VORTA_ERR_CUDA;
    }
    size_t first = 0;
    for (size_t ci = 0; ci < want; first += (size_t)sizes[ci], ++ci) {
        vorta_plan::HostChunk &c = p->chunks[ci];
        c.heads.assign(order.begin() + first, order.begin() + first + sizes[ci]);
        std::sort(c.heads.begin(), c.heads.end());
        std::vector<uint8_t> branches(g.heads, 0);
        std::vector<int32_t> core;
        for (int32_t h : c.heads) {
            branches[h] = (uint8_t)(1u << p->routes[h]);
            if (p->routes[h] == VORTA_ROUTE_CORESET) core.push_back(h);
        }
        int rc = build_list(p, c.wl, branches, false);
        if (rc != VORTA_OK) return rc;
        c.n_core = (int32_t)core.size();
        std::vector<int32_t> cs((size_t)g.B * std::max(c.n_core, 1)), cx(cs.size());
        for (int32_t b = 0; b < g.B; ++b)
            for (int32_t k = 0; k < c.n_core; ++k) {
                cs[(size_t)b * c.n_core + k] = b * g.heads + core[k];
                cx[(size_t)b * c.n_core + k] = b;
            }
        if (c.n_core &&
            (upload(p, c.d_core_slice, cs.data(), sizeof(int32_t) * g.B * c.n_core) != cudaSuccess ||
             upload(p, c.d_core_xslice, cx.data(), sizeof(int32_t) * g.B * c.n_core) != cudaSuccess ||
             cudaStreamSynchronize(p->s_in) != cudaSuccess))
            return VORTA_ERR_CUDA;
    }
    return VORTA_OK;
}

// Make the work list of the current routes the active one: a list kept from an earlier use of the same
// route vector, or a new one built into the least recently used entry.
int build_work(vorta_plan *p)
{
    const Geometry &g = p->g;
    std::vector<int32_t> core_heads;
    for (int32_t h = 0; h < g.heads; ++h)
        if (p->routes[h] == VORTA_ROUTE_CORESET) core_heads.push_back(h);
    if (p->host_only) {
        p->core_heads = core_heads;
        return VORTA_OK;
    }
    int hit = -1;
    for (size_t i = 0; i < p->cache.size(); ++i)
        if (p->cache[i].routes == p->routes) hit = (int)i;
    if (hit < 0) {
        if ((int)p->cache.size() < vorta_plan::kRouteCache) {
            p->cache.emplace_back();
            hit = (int)p->cache.size() - 1;
            vorta_plan::RouteEntry &e = p->cache[hit];
            if (cudaEventCreateWithFlags(&e.used, cudaEventDisableTiming) != cudaSuccess ||
                cudaMalloc(&e.d_core_slice, sizeof(int32_t) * (size_t)g.B * g.heads) != cudaSuccess ||
                cudaMalloc(&e.d_core_xslice, sizeof(int32_t) * (size_t)g.B * g.heads) != cudaSuccess)
                return VORTA_ERR_CUDA;
        } else {
            hit = 0;
            for (size_t i = 1; i < p->cache.size(); ++i)
                if (p->cache[i].stamp < p->cache[hit].stamp) hit = (int)i;
            // its buffers are about to be overwritten: the last call that used them must be done
            if (p->cache[hit].used_valid && cudaEventSynchronize(p->cache[hit].used) != cudaSuccess) return VORTA_ERR_CUDA;
        }
        vorta_plan::RouteEntry &e = p->cache[hit];
        e.routes.clear();  // not a valid entry until everything below has succeeded
        e.used_valid = false;
        std::vector<uint8_t> branches(g.heads);
        for (int32_t h = 0; h < g.heads; ++h) branches[h] = (uint8_t)(1u << p->routes[h]);
        int rc = build_list(p, e.wl, branches, false);
        if (rc != VORTA_OK) return rc;
        const int32_t n_core = (int32_t)core_heads.size();
        std::vector<int32_t> core_slice((size_t)g.B * std::max(n_core, 1)), core_x(core_slice.size());
        for (int32_t b = 0; b < g.B; ++b)
            for (int32_t k = 0; k < n_core; ++k) {
                core_slice[(size_t)b * n_core + k] = b * g.heads + core_heads[k];
                core_x[(size_t)b * n_core + k] = b;
            }
        if (n_core &&
            (upload(p, e.d_core_slice, core_slice.data(), sizeof(int32_t) * g.B * n_core) != cudaSuccess ||
             upload(p, e.d_core_xslice, core_x.data(), sizeof(int32_t) * g.B * n_core) != cudaSuccess ||
             cudaStreamSynchronize(p->s_in) != cudaSuccess))
            return VORTA_ERR_CUDA;
        e.core_heads = core_heads;
        e.routes = p->routes;
    }
    vorta_plan::RouteEntry &e = p->cache[hit];
    e.stamp = ++p->activations;
    p->cur = hit;
    p->routed = e.wl;
    p->core_heads = e.core_heads;
    p->d_core_slice = e.d_core_slice;
    p->d_core_xslice = e.d_core_xslice;
    p->chunks_stale = true;
    return VORTA_OK;
}

// Order between the two kinds of persistent attention kernel on one device.  A cluster kernel (CTA
// pairs) and the single-CTA kernel must not share the GPU: side by side, the single-CTA kernel's
// bounded waits have expired.  Calls from different plans or streams could still mix them, so every
// launch of one kind first makes its stream wait for the last launch of the other kind on that
// device, and records itself afterwards.  Kernels of the same kind may overlap freely.
struct KernelOrder {
    std::mutex m;
    cudaEvent_t last[2] = {nullptr, nullptr};  // 0: pair kernel, 1: single-CTA kernel
    bool recorded[2] = {false, false};
};
KernelOrder *kernel_order(int device)
{
    static KernelOrder table[64];
    return device >= 0 && device < 64 ? &table[device] : nullptr;
}
// before a launch of `kind` on stream s
cudaError_t order_before(int device, int kind, cudaStream_t s)
{
    KernelOrder *o = kernel_order(device);
    if (!o) return cudaSuccess;
    std::lock_guard<std::mutex> lock(o->m);
    const int other = kind ^ 1;
    return o->recorded[other] ? cudaStreamWaitEvent(s, o->last[other], 0) : cudaSuccess;
}
// after it
cudaError_t order_after(int device, int kind, cudaStream_t s)
{
    KernelOrder *o = kernel_order(device);
    if (!o) return cudaSuccess;
    std::lock_guard<std::mutex> lock(o->m);
    if (!o->last[kind]) {
        cudaError_t e = cudaEventCreateWithFlags(&o->last[kind], cudaEventDisableTiming);
        if (e != cudaSuccess) return e;
    }
    cudaError_t e = cudaEventRecord(o->last[kind], s);
    if (e == cudaSuccess) o->recorded[kind] = true;
    return e;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        changed = ok && prev != dev;
    }
    ~DeviceGuard() { if (changed) cudaSetDevice(prev); }
    bool changed = false;
};

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

// the pair kernel is built for d = 128 and needs the SMs in pairs
static bool pair_supported(const vorta_plan *p) { return p->g.d == 128 && (p->sm_count & 1) == 0 && p->sm_count >= 2; }

// The kernel a call over `wl` runs: VORTA_KERNEL_AUTO takes the pair kernel (with the single-CTA
// kernel for the sliding heads) where the full and core-set heads hold at least 60 % of the work:
// measured on a B200, the split is 4 to 6 % faster at shares of 0.9 and above and 1 to 2 % slower at
// 0.53 and below (two launches, two tails).
static int32_t resolve_kernel(const vorta_plan *p, const vorta_plan::WorkList &wl)
{
    if (p->kernel != VORTA_KERNEL_AUTO) return p->kernel;
    return pair_supported(p) && wl.linear_share >= 0.6 ? VORTA_KERNEL_PAIR : VORTA_KERNEL_TCGEN05;
}

#ifdef VORTA_TRACE
static long long *g_vorta_trace = nullptr;
extern "C" __attribute__((visibility("default"))) int vorta_debug_trace(long long *out_host)
{
    if (!g_vorta_trace) return 1;
    cudaDeviceSynchronize();
    return cudaMemcpy(out_host, g_vorta_trace, 4 * 8 * 8 * sizeof(long long), cudaMemcpyDeviceToHost) != cudaSuccess;
}
#endif

// ------------------------------------------------------------------------------------
extern "C" {

const char *vorta_status_string(int s)
{
    switch (s) {
    case VORTA_OK: return "ok";
    case VORTA_ERR_INVALID_ARG: return "invalid argument";
    case VORTA_ERR_UNSUPPORTED: return "unsupported configuration";
    case VORTA_ERR_ALIGNMENT: return "misaligned pointer";
    case VORTA_ERR_WORKSPACE: return "workspace missing or too small";
    case VORTA_ERR_CUDA: return "CUDA call failed";
    case VORTA_ERR_TIMEOUT: return "bounded device-side wait expired";
    case VORTA_ERR_INTERNAL: return "internal self-check failed";
    default: return "unknown status";
    }
}

int vorta_plan_create(const vorta_plan_desc *desc, vorta_plan **out)
{
    if (!desc || !out) return VORTA_ERR_INVALID_ARG;
    *out = nullptr;
    const vorta_plan_desc &D = *desc;
    if (!D.routes || D.B < 1 || D.heads < 1 || D.T < 1 || D.H < 1 || D.W < 1) return VORTA_ERR_INVALID_ARG;
    if (D.T > 32767 || D.H > 32767 || D.W > 32767) return VORTA_ERR_INVALID_ARG;
    int64_t L64 = (int64_t)D.T * D.H * D.W;
    if (D.text_tokens < 0 || L64 + D.text_tokens >= (int64_t)1 << 31) return VORTA_ERR_INVALID_ARG;
    if ((int64_t)D.B * D.heads > 65535) return VORTA_ERR_INVALID_ARG;
    if (!(D.coreset_ratio > 0.f) || !(D.coreset_ratio <= 1.f)) return VORTA_ERR_INVALID_ARG;
    if (!(D.softmax_scale >= 0.f) || !std::isfinite(D.softmax_scale)) return VORTA_ERR_INVALID_ARG;
    if (D.flags & ~(VORTA_PLAN_HOST_ONLY | VORTA_PLAN_POOL_MERGE)) return VORTA_ERR_INVALID_ARG;
    int32_t bucket[3] = {D.bucket[0], D.bucket[1], D.bucket[2]};
    if (bucket[0] == 0 && bucket[1] == 0 && bucket[2] == 0) { bucket[0] = 2; bucket[1] = 3; bucket[2] = 2; }
    for (int a = 0; a < 3; ++a)
        if (D.tile[a] < 1 || D.window[a] < 1 || bucket[a] < 1) return VORTA_ERR_INVALID_ARG;
    for (int32_t h = 0; h < D.heads; ++h)
        if (D.routes[h] > VORTA_ROUTE_CORESET) return VORTA_ERR_INVALID_ARG;
    if (D.d != 64 && D.d != 128) return VORTA_ERR_UNSUPPORTED;
    if (D.tile[0] > 256 || D.tile[1] > 256 || D.tile[2] > 256) return VORTA_ERR_UNSUPPORTED;
    int32_t nbox[3];
    if (!choose_boxes(D.tile, nbox)) return VORTA_ERR_UNSUPPORTED;
    if ((int64_t)bucket[0] * bucket[1] * bucket[2] > 32) return VORTA_ERR_UNSUPPORTED;

    vorta_plan *p = new (std::nothrow) vorta_plan();
    if (!p) return VORTA_ERR_INTERNAL;
    Geometry &g = p->g;
    g.B = D.B; g.heads = D.heads; g.T = D.T; g.H = D.H; g.W = D.W; g.L = (int32_t)L64; g.d = D.d;
    const int32_t dim[3] = {D.T, D.H, D.W};
    g.n_tiles = 1; g.n_buckets = 1;
    for (int a = 0; a < 3; ++a) {
        g.tile[a] = D.tile[a];
        g.nt[a] = (dim[a] + D.tile[a] - 1) / D.tile[a];
        g.half[a] = D.window[a] / 2;
        g.restricted[a] = g.nt[a] > 2 * g.half[a] + 1;
        g.bucket[a] = bucket[a];
        g.nb[a] = (dim[a] + bucket[a] - 1) / bucket[a];
        g.n_tiles *= g.nt[a];
        g.n_buckets *= g.nb[a];
    }
    g.ratio = (double)D.coreset_ratio;
    p->scale = D.softmax_scale > 0.f ? D.softmax_scale : 1.0f / std::sqrt((float)D.d);
    p->host_only = (D.flags & VORTA_PLAN_HOST_ONLY) != 0;
    p->pool_merge = (D.flags & VORTA_PLAN_POOL_MERGE) != 0;
    p->routes.assign(D.routes, D.routes + D.heads);

    // core-set segments: prefix sum of keep(n) over the buckets in raster order
    p->seg_start.resize(g.n_buckets);
    int64_t Lc = 0;
    for (int32_t b = 0; b < g.n_buckets; ++b) {
        int32_t id[3] = {b / (g.nb[2] * g.nb[1]), (b / g.nb[2]) % g.nb[1], b % g.nb[2]};
        int64_t n = 1;
        for (int a = 0; a < 3; ++a) n *= std::min(g.bucket[a], dim[a] - g.bucket[a] * id[a]);
        p->seg_start[b] = (int32_t)Lc;
        Lc += keep_count(n, g.ratio);
    }
    g.Lc = (int32_t)Lc;
    g.Lt = D.text_tokens;
    g.Ltot = g.L + g.Lt;
    g.Lct = g.Lc + g.Lt;

    // sliding branch blocking: equal boxes of at most 128 tokens
    g.boxes_per_tile = nbox[0] * nbox[1] * nbox[2];
    for (int a = 0; a < 3; ++a) {
        g.nbox[a] = nbox[a];
        g.box[a] = g.tile[a] / nbox[a];
    }
    g.box_rows = g.box[0] * g.box[1] * g.box[2];
    g.bn_tile = (g.box_rows + 15) / 16 * 16;
    int32_t kv_tiles = 1;
    for (int a = 0; a < 3; ++a) kv_tiles *= std::min(g.nt[a], 2 * g.half[a] + 1);
    g.max_kv_per_tile = kv_tiles * g.boxes_per_tile;
    g.text_blocks = (g.Lt + g.bn_tile - 1) / g.bn_tile;
    p->sliding_pairs = sliding_valid_pairs(g);
    {
        // The last T tile may hold a single box with fewer frames than a box has: if those frames are at most 64 rows,
        // two such boxes (of tiles with the same window) fit one 128-row query block.
        const int32_t rem = g.T - (g.nt[0] - 1) * g.tile[0];
        if (g.boxes_per_tile > 1 && rem < g.box[0] && rem * g.box[1] * g.box[2] <= 64) p->lone_t = rem;
    }

    if (p->host_only) {
        int rc = build_work(p);
        if (rc != VORTA_OK) { delete p; return rc; }
        *out = p;
        return VORTA_OK;
    }

    // ---- device side ----
    int dev = D.device;
    if (dev < 0 && cudaGetDevice(&dev) != cudaSuccess) { delete p; return VORTA_ERR_CUDA; }
    p->device = dev;
    DeviceGuard guard(dev);
    cudaDeviceProp prop;
    if (!guard.ok || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { delete p; return VORTA_ERR_CUDA; }
    if (prop.major != 10) { delete p; return VORTA_ERR_UNSUPPORTED; }
    p->sm_count = prop.multiProcessorCount;

    // column masks of the sliding branch: class -> valid columns of a KV box.  Class
    // 1 + (4 pt + 2 ph + pw) * boxes_per_tile + bx: box bx of a tile the grid cuts on the axes flagged.
    std::vector<uint32_t> masks((size_t)kMaxMasks * 4, 0u);
    for (int32_t code = 0; code < 8; ++code) {
        const int32_t part[3] = {(code >> 2) & 1, (code >> 1) & 1, code & 1};
        for (int32_t bx = 0; bx < g.boxes_per_tile; ++bx) {
            const int32_t b[3] = {bx / (g.nbox[1] * g.nbox[2]), (bx / g.nbox[2]) % g.nbox[1], bx % g.nbox[2]};
            int32_t valid[3];
            for (int a = 0; a < 3; ++a) {
                const int32_t extent = part[a] ? dim[a] - (g.nt[a] - 1) * g.tile[a] : g.tile[a];
                valid[a] = std::min(std::max(extent - b[a] * g.box[a], 0), g.box[a]);
            }
            const int32_t id = 1 + code * g.boxes_per_tile + bx;
            // the shape of the part inside the grid: which axes cut THIS box (a box of a cut tile may
            // still be whole, or lie outside altogether: such boxes are never listed)
            int32_t shape = 0;
            for (int a = 0; a < 3; ++a)
                if (valid[a] > 0 && valid[a] < g.box[a]) shape |= 4 >> a;
            if (valid[0] > 0 && valid[1] > 0 && valid[2] > 0 && shape) {
                p->cls_shape[id] = (uint8_t)shape;
                p->shape_rows[shape] = (int16_t)(valid[0] * valid[1] * valid[2]);
                for (int a = 0; a < 3; ++a) p->shape_ext[shape][a] = valid[a];
            }
            for (int32_t r = 0; r < g.box_rows; ++r) {
                int32_t lw = r % g.box[2], lh = (r / g.box[2]) % g.box[1], lt = r / (g.box[2] * g.box[1]);
                if (lw < valid[2] && lh < valid[1] && lt < valid[0]) masks[(size_t)id * 4 + r / 32] |= 1u << (r % 32);
            }
        }
    }

    // bucket shape classes (bit 2: cut on T, bit 1: on H, bit 0: on W): token count, centre,
    // and the token offset of every local index from the bucket's first token
    std::vector<int32_t> btab((size_t)8 * kBucketTabStride, 0);
    for (int32_t cls = 0; cls < 8; ++cls) {
        int32_t e[3];
        for (int a = 0; a < 3; ++a) {
            bool cut = (cls >> (2 - a)) & 1;
            int32_t rem = dim[a] - (g.nb[a] - 1) * g.bucket[a];
            e[a] = cut ? rem : g.bucket[a];
        }
        int32_t n = e[0] * e[1] * e[2];
        if (n > 32) continue;  // only used for buckets of at most 32 tokens
        int32_t *t = &btab[(size_t)cls * kBucketTabStride];
        t[0] = n;
        t[1] = ((e[0] / 2) * e[1] + (e[1] / 2)) * e[2] + (e[2] / 2);
        for (int32_t l = 0; l < n; ++l) {
            int32_t lw = l % e[2], lh = (l / e[2]) % e[1], lt = l / (e[2] * e[1]);
            t[2 + l] = (lt * g.H + lh) * g.W + lw;
        }
    }

    bool ok = true;
    int64_t nt2 = (int64_t)g.n_tiles * g.n_tiles;
    ok = ok && cudaMalloc(&p->d_bm, (size_t)nt2) == cudaSuccess;
    ok = ok && cudaMalloc(&p->d_kv_list, sizeof(KvEntry) * (size_t)g.n_tiles * g.max_kv_per_tile) == cudaSuccess;
    ok = ok && cudaMalloc(&p->d_kv_count, sizeof(int32_t) * 2 * g.n_tiles) == cudaSuccess;
    ok = ok && cudaMalloc(&p->d_colmasks, sizeof(uint32_t) * masks.size()) == cudaSuccess;
    ok = ok && cudaMalloc(&p->d_seg_start, sizeof(int32_t) * g.n_buckets) == cudaSuccess;
    ok = ok && cudaMalloc(&p->d_bucket_tab, sizeof(int32_t) * btab.size()) == cudaSuccess;
    ok = ok && cudaMemcpy(p->d_bucket_tab, btab.data(), sizeof(int32_t) * btab.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMalloc(&p->d_status, sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMemset(p->d_status, 0, sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMemcpy(p->d_colmasks, masks.data(), sizeof(uint32_t) * masks.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(p->d_seg_start, p->seg_start.data(), sizeof(int32_t) * g.n_buckets, cudaMemcpyHostToDevice) == cudaSuccess;
    for (auto &set : p->ev)
        for (auto &e : set) ok = ok && cudaEventCreate(&e) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&p->s_in, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&p->s_out, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&p->s_alt, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&p->ev_start, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&p->ev_out, cudaEventDisableTiming) == cudaSuccess;
    // the mask builder runs once per shape; its per-tile counts come back for the work list
    // short T boxes of exactly 64 keys pair up into whole 128-key blocks (see kv_list_kernel)
    const int32_t pair_t = (g.bn_tile == kBlockM && p->shape_rows[4] == 64 && g.nbox[1] == 1 && g.nbox[2] == 1) ? 1 : 0;
    ok = ok && launch_block_mask(g, p->d_bm, p->d_kv_list, p->d_kv_count, pair_t, nullptr) == cudaSuccess;
    p->kv_count.resize(2 * (size_t)g.n_tiles);
    ok = ok && cudaMemcpy(p->kv_count.data(), p->d_kv_count, sizeof(int32_t) * 2 * g.n_tiles, cudaMemcpyDeviceToHost) == cudaSuccess;
    ok = ok && attention_sm100_prepare() == cudaSuccess;
    ok = ok && attention_sm100_pair_prepare() == cudaSuccess;
    if (!ok) { cudaGetLastError(); free_device(p); delete p; return VORTA_ERR_CUDA; }
    // self-check: the lists must hold exactly the blocks the window arithmetic predicts
    for (int32_t qt = 0; qt < g.n_tiles; ++qt)
        if (p->kv_count[qt] < 1 || p->kv_count[qt] > g.max_kv_per_tile) { free_device(p); delete p; return VORTA_ERR_INTERNAL; }
    int rc = build_pair_lists(p);
    if (rc == VORTA_OK) rc = build_work(p);
    if (rc != VORTA_OK) { free_device(p); delete p; return rc; }
    *out = p;
    return VORTA_OK;
}

int vorta_plan_set_routes(vorta_plan *p, const uint8_t *routes, int32_t n)
{
    if (!p || !routes || n != p->g.heads) return VORTA_ERR_INVALID_ARG;
    for (int32_t h = 0; h < n; ++h)
        if (routes[h] > VORTA_ROUTE_CORESET) return VORTA_ERR_INVALID_ARG;
    p->routes.assign(routes, routes + n);
    if (p->host_only) return build_work(p);
    DeviceGuard guard(p->device);
    p->broken = true;
    if (!guard.ok) return VORTA_ERR_CUDA;
    int rc = build_work(p);  // no device-wide wait: see RouteEntry
    p->broken = rc != VORTA_OK;
    return rc;
}

int vorta_plan_destroy(vorta_plan *p)
{
    if (!p) return VORTA_ERR_INVALID_ARG;
    if (!p->host_only) {
        DeviceGuard guard(p->device);
        cudaDeviceSynchronize();
        free_device(p);
    }
    delete p;
    return VORTA_OK;
}

int vorta_plan_info(const vorta_plan *p, vorta_plan_info_t *o)
{
    if (!p || !o) return VORTA_ERR_INVALID_ARG;
    const Geometry &g = p->g;
    std::memset(o, 0, sizeof(*o));
    o->L = g.L; o->Lc = g.Lc;
    for (int a = 0; a < 3; ++a) o->tiles_per_axis[a] = g.nt[a];
    o->n_tiles = g.n_tiles; o->n_buckets = g.n_buckets;
    o->kv_tiles_per_q_tile = g.max_kv_per_tile / g.boxes_per_tile;
    for (uint8_t r : p->routes) {
        if (r == VORTA_ROUTE_FULL) ++o->n_full;
        else if (r == VORTA_ROUTE_SLIDING) ++o->n_sliding;
        else ++o->n_coreset;
    }
    o->workspace_bytes = workspace_layout(g, (int64_t)g.B * o->n_coreset).total;
    o->workspace_bytes_max = workspace_layout(g, (int64_t)g.B * g.heads).total;
    // four tensors, then one core-set workspace per group of heads (their sizes add up to the layer's,
    // plus alignment padding per group)
    o->host_call_scratch_bytes = 4 * align_up(tensor_bytes(g), 256) + o->workspace_bytes + kHostChunks * 8 * 256;
    o->mixture_workspace_bytes = mixture_workspace_bytes(g);
    o->text_tokens = g.Lt;
    o->flops_full_head = 4.0 * g.d * (double)g.Ltot * (double)g.Ltot;
    o->flops_sliding_head = 4.0 * g.d * (p->sliding_pairs + (double)g.L * g.Lt + (double)g.Lt * g.Ltot);
    o->flops_coreset_head = 4.0 * g.d * (double)g.Lct * (double)g.Lct;
    o->flops_layer = g.B * (o->n_full * o->flops_full_head + o->n_sliding * o->flops_sliding_head +
                            o->n_coreset * o->flops_coreset_head);
    o->flops_issued_layer = p->host_only ? 0.0 : p->routed.flops_issued;
    o->n_work_items = p->host_only ? 0 : p->routed.n_items;
    o->select_bytes_head = (int64_t)g.L * g.d * 2 + ((int64_t)g.Lc + g.L) * 4;
    o->gather_bytes_head = 3 * 2 * (int64_t)g.Lct * g.d * 2;
    o->scatter_bytes_head = ((int64_t)g.Lct + g.Ltot) * g.d * 2;
    return VORTA_OK;
}

int vorta_plan_device(const vorta_plan *p, int32_t *device)
{
    if (!p || !device) return VORTA_ERR_INVALID_ARG;
    *device = p->host_only ? -1 : p->device;
    return VORTA_OK;
}

int vorta_shard_heads(const vorta_plan *p, int32_t n_ranks, int32_t *rank_of_head, double *rank_flops)
{
    if (!p || !rank_of_head || n_ranks < 1) return VORTA_ERR_INVALID_ARG;
    const Geometry &g = p->g;
    vorta_plan_info_t info;
    int rc = vorta_plan_info(p, &info);
    if (rc != VORTA_OK) return rc;
    std::vector<double> cost(g.heads);
    for (int32_t h = 0; h < g.heads; ++h)
        cost[h] = p->routes[h] == VORTA_ROUTE_FULL ? info.flops_full_head
                  : p->routes[h] == VORTA_ROUTE_SLIDING ? info.flops_sliding_head : info.flops_coreset_head;
    std::vector<int32_t> order(g.heads);
    for (int32_t h = 0; h < g.heads; ++h) order[h] = h;
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return cost[a] > cost[b]; });
    std::vector<double> load((size_t)n_ranks, 0.0);
    for (int32_t h : order) {
        int32_t best = 0;
        for (int32_t r = 1; r < n_ranks; ++r)
            if (load[r] < load[best]) best = r;
        rank_of_head[h] = best;
        load[best] += cost[h];
    }
    if (rank_flops)
        for (int32_t r = 0; r < n_ranks; ++r) rank_flops[r] = load[r];
    return VORTA_OK;
}

int vorta_plan_block_mask(const vorta_plan *p, uint8_t *out_host)
{
    if (!p || !out_host) return VORTA_ERR_INVALID_ARG;
    if (p->host_only) return VORTA_ERR_UNSUPPORTED;
    DeviceGuard guard(p->device);
    if (!guard.ok) return VORTA_ERR_CUDA;
    size_t n = (size_t)p->g.n_tiles * p->g.n_tiles;
    return cudaMemcpy(out_host, p->d_bm, n, cudaMemcpyDeviceToHost) == cudaSuccess ? VORTA_OK : VORTA_ERR_CUDA;
}

int vorta_plan_set_kernel(vorta_plan *p, int32_t kernel)
{
    if (!p || kernel < VORTA_KERNEL_TCGEN05 || kernel > VORTA_KERNEL_AUTO) return VORTA_ERR_INVALID_ARG;
    if (kernel == VORTA_KERNEL_PAIR && !pair_supported(p)) return VORTA_ERR_UNSUPPORTED;
    p->kernel = kernel;
    return VORTA_OK;
}

int32_t vorta_plan_kernel_in_use(const vorta_plan *p)
{
    if (!p || p->host_only) return -1;
    return resolve_kernel(p, p->routed);
}

int vorta_plan_set_profiling(vorta_plan *p, int32_t on)
{
    if (!p) return VORTA_ERR_INVALID_ARG;
    p->profiling = on != 0;
    return VORTA_OK;
}

int vorta_plan_stage_ms_at(const vorta_plan *p, int32_t calls_back, float ms[4])
{
    if (!p || !ms || calls_back < 0 || calls_back >= vorta_plan::kProfSlots) return VORTA_ERR_INVALID_ARG;
    if (p->host_only) return VORTA_ERR_UNSUPPORTED;
    if (calls_back >= p->prof_calls) return VORTA_ERR_INVALID_ARG;
    const int slot = (int)((p->prof_calls - 1 - calls_back) % vorta_plan::kProfSlots);
    for (int i = 0; i < 4; ++i) {
        ms[i] = 0.f;
        if (p->ev_valid[slot][i] && p->ev_valid[slot][i + 1] &&
            cudaEventElapsedTime(&ms[i], p->ev[slot][i], p->ev[slot][i + 1]) != cudaSuccess) {
            cudaGetLastError();
            return VORTA_ERR_CUDA;
        }
    }
    return VORTA_OK;
}

int vorta_plan_stage_ms(const vorta_plan *p, float ms[4]) { return vorta_plan_stage_ms_at(p, 0, ms); }

int vorta_plan_attention_ms_at(const vorta_plan *p, int32_t calls_back, float ms[2])
{
    if (!p || !ms || calls_back < 0 || calls_back >= vorta_plan::kProfSlots) return VORTA_ERR_INVALID_ARG;
    if (p->host_only) return VORTA_ERR_UNSUPPORTED;
    if (calls_back >= p->prof_calls) return VORTA_ERR_INVALID_ARG;
    const int slot = (int)((p->prof_calls - 1 - calls_back) % vorta_plan::kProfSlots);
    ms[0] = ms[1] = 0.f;
    if (!p->ev_valid[slot][2] || !p->ev_valid[slot][3]) return VORTA_OK;
    cudaError_t e;
    if (p->ev_valid[slot][5]) {
        e = cudaEventElapsedTime(&ms[0], p->ev[slot][2], p->ev[slot][5]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms[1], p->ev[slot][5], p->ev[slot][3]);
    } else {
        e = cudaEventElapsedTime(&ms[0], p->ev[slot][2], p->ev[slot][3]);
    }
    if (e != cudaSuccess) {
        cudaGetLastError();
        return VORTA_ERR_CUDA;
    }
    return VORTA_OK;
}

int vorta_plan_last_launches(const vorta_plan *p, int32_t *n)
{
    if (!p || !n) return VORTA_ERR_INVALID_ARG;
    *n = p->last_launches;
    return VORTA_OK;
}

int vorta_coreset_select(const vorta_plan *p, const void *X, int32_t Hx, int32_t dx, int32_t *core_idx,
                         int32_t *src_slot, void *stream)
{
    if (!p || !X || !core_idx || !src_slot || Hx < 1 || dx < 8 || (dx % 8) != 0) return VORTA_ERR_INVALID_ARG;
    if (p->host_only) return VORTA_ERR_UNSUPPORTED;
    if (!aligned(X, 16) || !aligned(core_idx, 4) || !aligned(src_slot, 4)) return VORTA_ERR_ALIGNMENT;
    DeviceGuard guard(p->device);
    if (!guard.ok) return VORTA_ERR_CUDA;
    cudaError_t e = launch_select(p->g, static_cast<const __nv_bfloat16 *>(X), dx, p->g.B * Hx, nullptr,
                                  p->d_seg_start, p->d_bucket_tab, core_idx, src_slot, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? VORTA_OK : VORTA_ERR_CUDA;
}

// One layer over a work list: select, gather, attention, scatter.  `o_attn` is the tensor
// the attention kernel writes full and sliding rows to (indexed by the items' output
// slices), `o_scatter` the [B*heads, L, d] tensor the core-set rows are scattered into.
// core_slice == nullptr means the identity (every head is a core-set problem).
static int run_layer(const vorta_plan *p, const vorta_plan::WorkList &wl, int32_t n_core, const int32_t *core_slice,
                     const int32_t *core_xslice, const __nv_bfloat16 *q, const __nv_bfloat16 *k,
                     const __nv_bfloat16 *v, __nv_bfloat16 *o_attn, __nv_bfloat16 *o_scatter, const void *X,
                     int32_t Hx, void *workspace, cudaStream_t s, bool profile)
{
    const Geometry &g = p->g;
    const int32_t n_prob = g.B * n_core;
    Workspace ws = workspace_layout(g, n_prob);
    char *wsb = static_cast<char *>(workspace);
    int32_t *core_idx = n_prob ? reinterpret_cast<int32_t *>(wsb + ws.core_idx) : nullptr;
    int32_t *src_slot = n_prob ? reinterpret_cast<int32_t *>(wsb + ws.src_slot) : nullptr;
    __nv_bfloat16 *Qc = n_prob ? reinterpret_cast<__nv_bfloat16 *>(wsb + ws.Qc) : nullptr;
    __nv_bfloat16 *Kc = n_prob ? reinterpret_cast<__nv_bfloat16 *>(wsb + ws.Kc) : nullptr;
    __nv_bfloat16 *Vc = n_prob ? reinterpret_cast<__nv_bfloat16 *>(wsb + ws.Vc) : nullptr;
    __nv_bfloat16 *Oc = n_prob ? reinterpret_cast<__nv_bfloat16 *>(wsb + ws.Oc) : nullptr;

    AttnParams prm{};
    prm.g = g;
    prm.scale_log2 = p->scale * 1.4426950408889634f;
    prm.items = wl.d_items; prm.cta_begin = wl.d_cta_begin; prm.cta_count = wl.d_cta_count;
    prm.kv_list = p->d_kv_list; prm.kv_pairs = p->d_kv_pairs; prm.colmasks = p->d_colmasks;
    std::memcpy(prm.cls_shape, p->cls_shape, sizeof(prm.cls_shape));
    std::memcpy(prm.shape_rows, p->shape_rows, sizeof(prm.shape_rows));
    prm.lone_rows = p->lone_t * g.box[1] * g.box[2];
    prm.O = o_attn; prm.Oc = Oc; prm.Q = q; prm.K = k; prm.V = v; prm.Qc = Qc; prm.Kc = Kc; prm.Vc = Vc;
    prm.status = p->d_status;
#ifdef VORTA_TRACE
    {
        static long long *d_trace = nullptr;
        if (!d_trace) cudaMalloc(&d_trace, 4 * 8 * 8 * sizeof(long long));
        cudaMemsetAsync(d_trace, 0, 4 * 8 * 8 * sizeof(long long), s);
        prm.trace = d_trace;
        g_vorta_trace = d_trace;
    }
#endif

    AttnMaps maps;
    std::memset(&maps, 0, sizeof(maps));
    // Hybrid mode: the items over consecutive rows (full and core-set heads) go to the pair kernel,
    // the sliding items to the single-CTA kernel, each with its own lists behind the common ones.
    const int32_t kernel = resolve_kernel(p, wl);
    const bool pair = kernel == VORTA_KERNEL_PAIR;
    AttnParams prm_pair = prm, prm_tiles = prm;
    if (pair) {
        const int32_t n_pairs = p->sm_count / 2;
        prm_pair.items = wl.d_items + wl.n_items;
        prm_pair.cta_begin = wl.d_cta_begin + p->sm_count;
        prm_pair.cta_count = wl.d_cta_count + p->sm_count;
        prm_tiles.items = wl.d_items + wl.n_items + wl.n_linear;
        prm_tiles.cta_begin = wl.d_cta_begin + p->sm_count + n_pairs;
        prm_tiles.cta_count = wl.d_cta_count + p->sm_count + n_pairs;
    }
    if (kernel == VORTA_KERNEL_TCGEN05 || pair) {
        const int64_t BH = (int64_t)g.B * g.heads;
        bool ok = true;
        const void *src[3] = {q, k, v};
        CUtensorMap *dst[3] = {maps.q, maps.k, maps.v};
        for (int t = 0; t < 3 && ok; ++t) {
            ok = ok && make_map(&dst[t][MODE_LINEAR], src[t], g.d, g.Ltot, 1, 1, BH, kBlockM, 1, 1);
            // the video rows of a head as a T x H x W grid; heads are L + Lt rows apart
            ok = ok && make_map(&dst[t][MODE_TILES], src[t], g.d, g.W, g.H, g.T, BH, g.box[2], g.box[1], g.box[0],
                                g.Ltot);
        }
        // the short boxes of the KV tiles the grid cuts (shapes that do not occur alias the whole box)
        for (int sh = 0; sh < kBoxShapes && ok; ++sh) {
            if (p->shape_rows[sh] > 0) {
                const int32_t *e = p->shape_ext[sh];
                ok = ok && make_map(&maps.k_cut[sh], k, g.d, g.W, g.H, g.T, BH, e[2], e[1], e[0], g.Ltot);
                ok = ok && make_map(&maps.v_cut[sh], v, g.d, g.W, g.H, g.T, BH, e[2], e[1], e[0], g.Ltot);
            } else {
                maps.k_cut[sh] = maps.k[MODE_TILES];
                maps.v_cut[sh] = maps.v[MODE_TILES];
            }
        }
        if (p->lone_t > 0)
            ok = ok && make_map(&maps.q_lone, q, g.d, g.W, g.H, g.T, BH, g.box[2], g.box[1], p->lone_t, g.Ltot);
        else
            maps.q_lone = maps.q[MODE_TILES];
        if (g.Lt > 0) {
            // the text rows of K and V: Lt rows starting L rows into every head, in boxes of bn_tile rows
            const __nv_bfloat16 *kt = k + (int64_t)g.L * g.d, *vt = v + (int64_t)g.L * g.d;
            ok = ok && make_map(&maps.kt, kt, g.d, g.Lt, 1, 1, BH, g.bn_tile, 1, 1, g.Ltot);
            ok = ok && make_map(&maps.vt, vt, g.d, g.Lt, 1, 1, BH, g.bn_tile, 1, 1, g.Ltot);
        } else {
            maps.kt = maps.k[MODE_LINEAR];
            maps.vt = maps.v[MODE_LINEAR];
        }
        const void *csrc[3] = {Qc, Kc, Vc};
        for (int t = 0; t < 3 && ok; ++t) {
            if (n_prob) ok = ok && make_map(&dst[t][MODE_COMPACT], csrc[t], g.d, g.Lct, 1, 1, n_prob, kBlockM, 1, 1);
            else dst[t][MODE_COMPACT] = dst[t][MODE_LINEAR];
        }
        if (pair) {
            // K in boxes of 64 rows: the first or second half of a block's keys for each CTA of a pair
            ok = ok && make_map(&maps.k_half[MODE_LINEAR], k, g.d, g.Ltot, 1, 1, BH, kBlockM / 2, 1, 1);
            maps.k_half[MODE_TILES] = maps.k_half[MODE_LINEAR];  // unused: sliding items run in the other kernel
            if (n_prob) ok = ok && make_map(&maps.k_half[MODE_COMPACT], Kc, g.d, g.Lct, 1, 1, n_prob, kBlockM / 2, 1, 1);
            else maps.k_half[MODE_COMPACT] = maps.k_half[MODE_LINEAR];
        }
        if (!ok) return VORTA_ERR_CUDA;
    }

    int32_t launches = 0;
    const bool prof = profile && p->profiling;
    const int pslot = (int)(p->prof_calls % vorta_plan::kProfSlots);
    if (prof) {
        for (auto &f : p->ev_valid[pslot]) f = false;
        ++p->prof_calls;
    }
    auto mark = [&](int i) {
        if (prof && cudaEventRecord(p->ev[pslot][i], s) == cudaSuccess) p->ev_valid[pslot][i] = true;
    };
    cudaError_t e = cudaSuccess;
    mark(0);
    if (n_prob) {
        const __nv_bfloat16 *xs = X ? static_cast<const __nv_bfloat16 *>(X) : k;
        const int32_t *xslice = (X && Hx == 1) ? core_xslice : core_slice;
        e = launch_select(g, xs, g.d, n_prob, xslice, p->d_seg_start, p->d_bucket_tab, core_idx, src_slot, s);
        if (e != cudaSuccess) return VORTA_ERR_CUDA;
        ++launches;
    }
    mark(1);
    if (n_prob) {
        e = launch_gather(g, n_prob, core_slice, core_idx, q, k, v, Qc, Kc, Vc, s);
        if (e != cudaSuccess) return VORTA_ERR_CUDA;
        ++launches;
        if (p->pool_merge) {
            e = launch_merge(g, n_prob, core_slice, p->d_seg_start, p->d_bucket_tab, src_slot, q, k, v, Qc, Kc, Vc, s);
            if (e != cudaSuccess) return VORTA_ERR_CUDA;
            ++launches;
        }
    }
    mark(2);
    if (wl.n_items > 0) {
        if (pair) {
            // One after the other on the caller's stream.  (Run side by side on two queues, so that the
            // second kernel's CTAs fill the SMs the first one's tail leaves, the single-CTA kernel's
            // bounded waits expired at hunyuan-720p: CTAs of a cluster kernel and of a plain kernel
            // are not mixed on the GPU here.)
            if (wl.n_linear > 0) {
                if (order_before(p->device, 0, s) != cudaSuccess) return VORTA_ERR_CUDA;
                e = launch_attention_sm100_pair(prm_pair, maps, p->sm_count, s);
                if (e != cudaSuccess || order_after(p->device, 0, s) != cudaSuccess) return VORTA_ERR_CUDA;
                ++launches;
            }
            if (wl.n_linear > 0 && wl.n_items - wl.n_linear > 0) mark(5);
            if (wl.n_items - wl.n_linear > 0) {
                if (order_before(p->device, 1, s) != cudaSuccess) return VORTA_ERR_CUDA;
                e = launch_attention_sm100(prm_tiles, maps, p->sm_count, s);
                if (e != cudaSuccess || order_after(p->device, 1, s) != cudaSuccess) return VORTA_ERR_CUDA;
                ++launches;
            }
        } else if (kernel == VORTA_KERNEL_TCGEN05) {
            if (order_before(p->device, 1, s) != cudaSuccess) return VORTA_ERR_CUDA;
            e = launch_attention_sm100(prm, maps, p->sm_count, s);
            if (e != cudaSuccess || order_after(p->device, 1, s) != cudaSuccess) return VORTA_ERR_CUDA;
            ++launches;
        } else {
            e = launch_attention_simt(prm, wl.n_items, s);
            if (e != cudaSuccess) return VORTA_ERR_CUDA;
            ++launches;
        }
    }
    mark(3);
    if (n_prob) {
        e = launch_scatter(g, n_prob, core_slice, src_slot, Oc, o_scatter, s);
        if (e != cudaSuccess) return VORTA_ERR_CUDA;
        ++launches;
    }
    mark(4);
    p->last_launches = launches;
    return VORTA_OK;
}

int vorta_routed_attention(const vorta_plan *p, const void *Q, const void *K, const void *V, void *O,
                           const void *X, int32_t Hx, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!p || !Q || !K || !V || !O) return VORTA_ERR_INVALID_ARG;
    if (p->host_only) return VORTA_ERR_UNSUPPORTED;
    if (p->broken) return VORTA_ERR_INTERNAL;
    const Geometry &g = p->g;
    if (X && Hx != 1 && Hx != g.heads) return VORTA_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || (X && !aligned(X, 16)))
        return VORTA_ERR_ALIGNMENT;
    const int32_t n_core = (int32_t)p->core_heads.size();
    if (n_core > 0) {
        if (!workspace || (int64_t)workspace_bytes < workspace_layout(g, (int64_t)g.B * n_core).total)
            return VORTA_ERR_WORKSPACE;
        if (!aligned(workspace, 256)) return VORTA_ERR_ALIGNMENT;
    }
    DeviceGuard guard(p->device);
    if (!guard.ok) return VORTA_ERR_CUDA;
    __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(O);
    int rc = run_layer(p, p->routed, n_core, p->d_core_slice, p->d_core_xslice, static_cast<const __nv_bfloat16 *>(Q),
                       static_cast<const __nv_bfloat16 *>(K), static_cast<const __nv_bfloat16 *>(V), o, o, X, Hx,
                       workspace, static_cast<cudaStream_t>(stream), true);
    // this route vector's lists are in use until here on the stream
    if (p->cur >= 0) {
        vorta_plan::RouteEntry &e = p->cache[p->cur];
        if (cudaEventRecord(e.used, static_cast<cudaStream_t>(stream)) == cudaSuccess) e.used_valid = true;
        else if (rc == VORTA_OK) rc = VORTA_ERR_CUDA;
    }
    return rc;
}

int vorta_soft_mixture(vorta_plan *p, const void *Q, const void *K, const void *V, const float *gates, void *O,
                       void *workspace, size_t workspace_bytes, void *stream)
{
    if (!p || !Q || !K || !V || !O || !gates) return VORTA_ERR_INVALID_ARG;
    if (p->host_only) return VORTA_ERR_UNSUPPORTED;
    const Geometry &g = p->g;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(gates, 4))
        return VORTA_ERR_ALIGNMENT;
    if (!workspace || (int64_t)workspace_bytes < mixture_workspace_bytes(g)) return VORTA_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return VORTA_ERR_ALIGNMENT;
    DeviceGuard guard(p->device);
    if (!guard.ok) return VORTA_ERR_CUDA;
    if (!p->mixture.built) {
        std::vector<uint8_t> all(g.heads, (uint8_t)7);  // every head runs all three branches
        int rc = build_list(p, p->mixture, all, true);
        if (rc != VORTA_OK) return rc;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the three branch outputs [3, B*heads, L, d] sit back to back after the core-set scratch
    char *wsb = static_cast<char *>(workspace);
    char *branches = wsb + workspace_layout(g, (int64_t)g.B * g.heads).total;
    __nv_bfloat16 *br = reinterpret_cast<__nv_bfloat16 *>(branches);
    __nv_bfloat16 *br_core = reinterpret_cast<__nv_bfloat16 *>(branches + VORTA_ROUTE_CORESET * tensor_bytes(g));
    int rc = run_layer(p, p->mixture, g.heads, nullptr, nullptr, static_cast<const __nv_bfloat16 *>(Q),
                       static_cast<const __nv_bfloat16 *>(K), static_cast<const __nv_bfloat16 *>(V), br, br_core,
                       nullptr, 0, workspace, s, false);
    if (rc != VORTA_OK) return rc;
    if (launch_mix_combine(g, gates, br, static_cast<__nv_bfloat16 *>(O), s) != cudaSuccess) return VORTA_ERR_CUDA;
    p->last_launches += 1;
    return VORTA_OK;
}

int vorta_router_gates(const float *T, const float *WR, int32_t d_model, int32_t heads, float *gates,
                       uint8_t *routes, void *stream)
{
    if (!T || !WR || !gates || !routes || d_model < 1 || heads < 1) return VORTA_ERR_INVALID_ARG;
    if (!aligned(T, 4) || !aligned(WR, 4) || !aligned(gates, 4)) return VORTA_ERR_ALIGNMENT;
    return launch_router(T, WR, d_model, heads, gates, routes, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? VORTA_OK
               : VORTA_ERR_CUDA;
}

int vorta_routed_attention_host(const vorta_plan *p, const void *Qh, const void *Kh, const void *Vh, void *Oh,
                                void *scratch, size_t scratch_bytes, void *stream)
{
    if (!p || !Qh || !Kh || !Vh || !Oh || !scratch) return VORTA_ERR_INVALID_ARG;
    if (p->host_only) return VORTA_ERR_UNSUPPORTED;
    if (p->broken) return VORTA_ERR_INTERNAL;
    vorta_plan_info_t info;
    vorta_plan_info(p, &info);
    if ((int64_t)scratch_bytes < info.host_call_scratch_bytes) return VORTA_ERR_WORKSPACE;
    if (!aligned(scratch, 256)) return VORTA_ERR_ALIGNMENT;
    DeviceGuard guard(p->device);
    if (!guard.ok) return VORTA_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const Geometry &g = p->g;
    if (p->chunks_stale) {
        // first call since the routes were set: build the groups' work lists (small device
        // allocations and synchronous copies; later calls only enqueue)
        int rc = build_host_chunks(const_cast<vorta_plan *>(p));
        if (rc != VORTA_OK) {
            const_cast<vorta_plan *>(p)->broken = true;  // the groups' lists are half built
            return rc;
        }
        p->chunks_stale = false;
    }
    const int64_t tb = tensor_bytes(g), tba = align_up(tb, 256);
    char *base = static_cast<char *>(scratch);
    char *dq = base, *dk = base + tba, *dv = base + 2 * tba, *dO = base + 3 * tba;
    void *ws = base + 4 * tba;
    const char *hq = static_cast<const char *>(Qh), *hk = static_cast<const char *>(Kh),
               *hv = static_cast<const char *>(Vh);
    char *ho = static_cast<char *>(Oh);
    const int64_t hb = (int64_t)g.Ltot * g.d * (int64_t)sizeof(__nv_bfloat16);  // one head of one tensor

    // Four queues: copies in (own stream), kernels (the caller's stream for even groups, a second
    // stream for odd ones), copies out (own stream).  Group c's kernels wait for its copies in; its
    // copy out waits for its kernels.  Consecutive groups sit in different kernel queues and use
    // different slices of the core-set workspace, so the persistent CTAs of the next group move
    // into the SMs the tail of the current one leaves.  Everything starts after the work already
    // in the caller's stream and the caller's stream ends up waiting for the last copy out (which
    // waited for every group's kernels), so the call as a whole behaves as one operation enqueued
    // on `stream`.
    if (cudaEventRecord(p->ev_start, s) != cudaSuccess || cudaStreamWaitEvent(p->s_in, p->ev_start, 0) != cudaSuccess ||
        cudaStreamWaitEvent(p->s_out, p->ev_start, 0) != cudaSuccess ||
        cudaStreamWaitEvent(p->s_alt, p->ev_start, 0) != cudaSuccess)
        return VORTA_ERR_CUDA;
    int64_t ws_off = 0;
    int32_t ci = 0;
    // Which attention kernels the previous group launched.  The pair kernel (clusters) and the single-CTA
    // kernel are never left to share the GPU (run side by side they made the latter's bounded waits expire):
    // where consecutive groups would mix them, the later group's queue waits for the earlier group's kernels.
    bool prev_pair = false, prev_single = false;
    const vorta_plan::HostChunk *prev = nullptr;
    for (const vorta_plan::HostChunk &c : p->chunks) {
        cudaStream_t sk = (ci++ & 1) ? p->s_alt : s;
        const int32_t kernel = resolve_kernel(p, c.wl);
        const bool use_pair = kernel == VORTA_KERNEL_PAIR && c.wl.n_linear > 0;
        const bool use_single = kernel == VORTA_KERNEL_TCGEN05 ? c.wl.n_items > 0
                                                               : (kernel == VORTA_KERNEL_PAIR && c.wl.n_items > c.wl.n_linear);
        if (prev && ((prev_pair && use_single) || (prev_single && use_pair)) &&
            cudaStreamWaitEvent(sk, prev->ev_done, 0) != cudaSuccess)
            return VORTA_ERR_CUDA;
        prev_pair = use_pair;
        prev_single = use_single;
        prev = &c;
        for (int32_t b = 0; b < g.B; ++b)
            for (int32_t h : c.heads) {
                const int64_t off = ((int64_t)b * g.heads + h) * hb;
                if (cudaMemcpyAsync(dq + off, hq + off, hb, cudaMemcpyHostToDevice, p->s_in) != cudaSuccess ||
                    cudaMemcpyAsync(dk + off, hk + off, hb, cudaMemcpyHostToDevice, p->s_in) != cudaSuccess ||
                    cudaMemcpyAsync(dv + off, hv + off, hb, cudaMemcpyHostToDevice, p->s_in) != cudaSuccess)
                    return VORTA_ERR_CUDA;
            }
        if (cudaEventRecord(c.ev_in, p->s_in) != cudaSuccess || cudaStreamWaitEvent(sk, c.ev_in, 0) != cudaSuccess)
            return VORTA_ERR_CUDA;
        __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(dO);
        void *ws_c = c.n_core ? static_cast<char *>(ws) + ws_off : nullptr;
        ws_off += align_up(workspace_layout(g, (int64_t)g.B * c.n_core).total, 256);
        int rc = run_layer(p, c.wl, c.n_core, c.d_core_slice, c.d_core_xslice, reinterpret_cast<const __nv_bfloat16 *>(dq),
                           reinterpret_cast<const __nv_bfloat16 *>(dk), reinterpret_cast<const __nv_bfloat16 *>(dv), o, o,
                           nullptr, 0, ws_c, sk, false);
        if (rc != VORTA_OK) return rc;
        if (cudaEventRecord(c.ev_done, sk) != cudaSuccess || cudaStreamWaitEvent(p->s_out, c.ev_done, 0) != cudaSuccess)
            return VORTA_ERR_CUDA;
        for (int32_t b = 0; b < g.B; ++b)
            for (int32_t h : c.heads) {
                const int64_t off = ((int64_t)b * g.heads + h) * hb;
                if (cudaMemcpyAsync(ho + off, dO + off, hb, cudaMemcpyDeviceToHost, p->s_out) != cudaSuccess)
                    return VORTA_ERR_CUDA;
            }
    }
    if (cudaEventRecord(p->ev_out, p->s_out) != cudaSuccess || cudaStreamWaitEvent(s, p->ev_out, 0) != cudaSuccess)
        return VORTA_ERR_CUDA;
    const_cast<vorta_plan *>(p)->host_call_made = true;
    return VORTA_OK;
}

int vorta_device_status(const vorta_plan *p, void *stream, int32_t *code_out)
{
    if (!p || !code_out) return VORTA_ERR_INVALID_ARG;
    if (p->host_only) return VORTA_ERR_UNSUPPORTED;
    DeviceGuard guard(p->device);
    if (!guard.ok) return VORTA_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(s) != cudaSuccess) return VORTA_ERR_CUDA;
    int32_t code = 0;
    if (cudaMemcpy(&code, p->d_status, sizeof(code), cudaMemcpyDeviceToHost) != cudaSuccess) return VORTA_ERR_CUDA;
    *code_out = code;
    if (code != 0) {
        cudaMemset(p->d_status, 0, sizeof(int32_t));
        return VORTA_ERR_TIMEOUT;
    }
    return VORTA_OK;
}

}  // extern "C"
