// Memory-bound kernels of the routed-attention layer: the block-sparse sliding-tile
// mask builder, bucketed core-set selection, the gather (pool) of the kept rows
// and the scatter (unpool) of the attention output.
#include <algorithm>

#include "vorta_internal.h"

namespace vorta {

// ---------------------------------------------------------------------------------
// Sliding tile mask between tiles (Appendix A.1, Algorithm 1).
// ---------------------------------------------------------------------------------

__device__ __forceinline__ void tile_triple(const Geometry &g, int32_t id, int32_t q[3])
{
    q[2] = id % g.nt[2];
    q[1] = (id / g.nt[2]) % g.nt[1];
    q[0] = id / (g.nt[2] * g.nt[1]);
}

// One thread per (query tile, key tile): move the query tile to its window-centre
// tile, then test the per-axis tile distance against floor(w/2).
__global__ void block_mask_kernel(Geometry g, uint8_t *__restrict__ bm)
{
    int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int64_t total = (int64_t)g.n_tiles * g.n_tiles;
    if (idx >= total) return;
    int32_t q[3], k[3];
    tile_triple(g, (int32_t)(idx / g.n_tiles), q);
    tile_triple(g, (int32_t)(idx % g.n_tiles), k);
    bool m = true;
#pragma unroll
    for (int a = 0; a < 3; ++a) {
        if (!g.restricted[a]) continue;
        int32_t c = min(max(q[a], g.half[a]), g.nt[a] - 1 - g.half[a]);
        m = m && (abs(c - k[a]) <= g.half[a]);
    }
    bm[idx] = m ? 1 : 0;
}

// One thread per query tile: turn its mask row into the list of KV blocks the
// attention kernel walks (key tiles ascending; a tile of more than 128 tokens
// gives several boxes; boxes that lie wholly outside the grid are dropped).
// pair_t: a box the grid cuts on T only down to exactly 64 rows (the one valid frame of the last
// T tile of the 720p grids) is listed together with the same box of the next window tile along W
// as ONE block of 64 + 64 real keys (kEntryPaired): a whole block as far as the MMAs and the
// softmax are concerned.
__global__ void kv_list_kernel(Geometry g, const uint8_t *__restrict__ bm, KvEntry *__restrict__ list,
                               int32_t *__restrict__ count, int32_t pair_t)
{
    int32_t qt = blockIdx.x * blockDim.x + threadIdx.x;
    if (qt >= g.n_tiles) return;
    KvEntry *out = list + (int64_t)qt * g.max_kv_per_tile;
    // the query tile's window along W: tiles [lo_w, hi_w]
    int32_t lo_w = 0, hi_w = g.nt[2] - 1;
    if (g.restricted[2]) {
        const int32_t c = min(max(qt % g.nt[2], g.half[2]), g.nt[2] - 1 - g.half[2]);
        lo_w = c - g.half[2];
        hi_w = c + g.half[2];
    }
    // the last tile along W does not pair if the grid cuts it
    const int32_t hi_pair = (g.W - hi_w * g.tile[2] < g.tile[2]) ? hi_w - 1 : hi_w;
    // Two passes: the boxes that lie wholly inside the grid (mask class 0) and the paired short boxes
    // first, the other cut ones after them, so that the attention kernel can run the leading blocks
    // without any masking.  count[n_tiles + qt] is the number of those leading blocks.
    int32_t n = 0, n_whole = 0;
    for (int pass = 0; pass < 2; ++pass) {
        for (int32_t kt = 0; kt < g.n_tiles; ++kt) {
            if (!bm[(int64_t)qt * g.n_tiles + kt]) continue;
            int32_t k[3];
            tile_triple(g, kt, k);
            int32_t t0 = k[0] * g.tile[0], h0 = k[1] * g.tile[1], w0 = k[2] * g.tile[2];
            int32_t pt = (g.T - t0 < g.tile[0]), ph = (g.H - h0 < g.tile[1]), pw = (g.W - w0 < g.tile[2]);
            bool whole = !pt && !ph && !pw && g.box_rows == g.bn_tile;
            for (int32_t bx = 0; bx < g.boxes_per_tile; ++bx) {
                // box bx of the tile; boxes that start outside the grid are dropped
                int32_t tb = t0 + (bx / (g.nbox[1] * g.nbox[2])) * g.box[0];
                int32_t hb = h0 + ((bx / g.nbox[2]) % g.nbox[1]) * g.box[1];
                int32_t wb = w0 + (bx % g.nbox[2]) * g.box[2];
                if (tb >= g.T || hb >= g.H || wb >= g.W) continue;
                // a short T box that pairs with its neighbour in the window: position r in the run of
                // pairable tiles [lo_w, hi_pair] of this row of tiles
                const int32_t vt = min(g.box[0], g.T - tb);
                const bool shorty = pair_t && pt && !ph && !pw && vt < g.box[0] && vt * g.box[1] * g.box[2] == 64 &&
                                    g.nbox[1] == 1 && g.nbox[2] == 1 && k[2] <= hi_pair;
                const int32_t r = k[2] - lo_w;
                const bool first_of_pair = shorty && (r % 2 == 0) && k[2] + 1 <= hi_pair;
                const bool second_of_pair = shorty && (r % 2 == 1);
                if (second_of_pair) continue;  // listed with the tile before it
                const bool lead = whole || first_of_pair;
                if (lead != (pass == 0)) continue;
                if (n < g.max_kv_per_tile) {
                    KvEntry e;
                    e.w0 = (int16_t)wb;
                    e.h0 = (int16_t)hb;
                    e.t0 = (int16_t)tb;
                    e.mask_id = whole ? 0 : (first_of_pair ? (uint16_t)kEntryPaired
                                                           : (uint16_t)(1 + ((pt * 2 + ph) * 2 + pw) * g.boxes_per_tile + bx));
                    out[n] = e;
                }
                ++n;
            }
        }
        if (pass == 0) n_whole = n;
    }
    count[qt] = n;
    count[g.n_tiles + qt] = n_whole;
}

cudaError_t launch_block_mask(const Geometry &g, uint8_t *bm, KvEntry *kv_list, int32_t *kv_count,
                              int32_t pair_t, cudaStream_t s)
{
    int64_t total = (int64_t)g.n_tiles * g.n_tiles;
    block_mask_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(g, bm);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    kv_list_kernel<<<(g.n_tiles + 127) / 128, 128, 0, s>>>(g, bm, kv_list, kv_count, pair_t);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------
// Bucketed core-set selection (Section 3.2; Appendix A.1).
// One warp per (problem, bucket).  Eight lanes share a token: each lane takes
// every eighth 16-byte chunk of the row, products and sums are fp64 (a bf16 x bf16
// product is exact there), and three shuffle steps finish the row.  Four tokens
// are scored per pass.
// ---------------------------------------------------------------------------------

__device__ __forceinline__ double shfl_xor_f64(double v, int m)
{
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_xor_sync(0xffffffffu, lo, m);
    hi = __shfl_xor_sync(0xffffffffu, hi, m);
    return __hiloint2double(hi, lo);
}

__device__ __forceinline__ double shfl_f64(double v, int src)
{
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_sync(0xffffffffu, lo, src);
    hi = __shfl_sync(0xffffffffu, hi, src);
    return __hiloint2double(hi, lo);
}

__device__ __forceinline__ void bf16x8_to_f64(const uint4 &u, double out[8])
{
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        out[2 * i] = (double)__uint_as_float(w[i] << 16);
        out[2 * i + 1] = (double)__uint_as_float(w[i] & 0xffff0000u);
    }
}

__global__ void __launch_bounds__(256)
coreset_select_kernel(Geometry g, const __nv_bfloat16 *__restrict__ X, int32_t dx, int32_t n_prob,
                      const int32_t *__restrict__ prob_slice, const int32_t *__restrict__ seg_start,
                      int32_t *__restrict__ core_idx, int32_t *__restrict__ src_slot)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (warp >= (int64_t)n_prob * g.n_buckets) return;
    const int32_t p = (int32_t)(warp / g.n_buckets);
    const int32_t bkt = (int32_t)(warp % g.n_buckets);
    const int32_t slice = prob_slice ? prob_slice[p] : p;
    const __nv_bfloat16 *Xs = X + (int64_t)slice * g.Ltot * dx;  // video rows of the slice

    // the bucket: id, extents cut by the grid, token count, centre
    int32_t id[3] = {bkt / (g.nb[2] * g.nb[1]), (bkt / g.nb[2]) % g.nb[1], bkt % g.nb[2]};
    const int32_t dim[3] = {g.T, g.H, g.W};
    int32_t e[3];
#pragma unroll
    for (int a = 0; a < 3; ++a) e[a] = min(g.bucket[a], dim[a] - g.bucket[a] * id[a]);
    const int32_t n = e[0] * e[1] * e[2];
    const int32_t centre = ((e[0] / 2) * e[1] + (e[1] / 2)) * e[2] + (e[2] / 2);
    auto token_of = [&](int32_t l) -> int32_t {
        int32_t lw = l % e[2], lh = (l / e[2]) % e[1], lt = l / (e[2] * e[1]);
        return ((id[0] * g.bucket[0] + lt) * g.H + (id[1] * g.bucket[1] + lh)) * g.W +
               (id[2] * g.bucket[2] + lw);
    };

    const int sub = lane >> 3, sl = lane & 7;
    const int32_t chunks = dx >> 3;
    const uint4 *xc = reinterpret_cast<const uint4 *>(Xs + (int64_t)token_of(centre) * dx);

    double my_score = 0.0;  // lane l ends up with the score of local token l
    double ncsq = 0.0;
    for (int32_t pass = 0; pass * 4 < n; ++pass) {
        const int32_t l = pass * 4 + sub;
        const bool active = l < n;
        double dot = 0.0, njsq = 0.0, csq = 0.0;
        if (active) {
            const uint4 *xj = reinterpret_cast<const uint4 *>(Xs + (int64_t)token_of(l) * dx);
            for (int32_t c = sl; c < chunks; c += 8) {
                double a[8], b[8];
                bf16x8_to_f64(__ldg(xc + c), a);
                bf16x8_to_f64(__ldg(xj + c), b);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    dot = fma(a[i], b[i], dot);
                    njsq = fma(b[i], b[i], njsq);
                    csq = fma(a[i], a[i], csq);
                }
            }
        }
#pragma unroll
        for (int m = 4; m >= 1; m >>= 1) {
            dot += shfl_xor_f64(dot, m);
            njsq += shfl_xor_f64(njsq, m);
            csq += shfl_xor_f64(csq, m);
        }
        if (pass == 0) ncsq = shfl_f64(csq, 0);  // token 0 always exists
        double nc = sqrt(ncsq), nj = sqrt(njsq);
        double score = (nc == 0.0 || nj == 0.0) ? 0.0 : dot / (nc * nj);
        double got = shfl_f64(score, (lane & 3) * 8);
        if ((lane >> 2) == pass) my_score = got;
    }

    // keep(n) = max(1, floor(r n + 1/2)); the k = n - keep most similar tokens go
    int32_t keep = (int32_t)floor(g.ratio * (double)n + 0.5);
    keep = max(keep, 1);
    const int32_t k = n - keep;
    const bool is_tok = lane < n, is_centre = lane == centre;
    int32_t rank = 0;
    for (int32_t m = 0; m < n; ++m) {
        double sm = shfl_f64(my_score, m);
        if (m != centre && (sm > my_score || (sm == my_score && m < lane))) ++rank;
    }
    const bool kept = is_tok && (is_centre || rank >= k);
    const uint32_t kept_others = __ballot_sync(0xffffffffu, kept && !is_centre);
    if (!is_tok) return;
    const int32_t seg = seg_start[bkt];
    const int32_t tok = token_of(lane);
    int32_t slot = seg;  // the centre's slot: pruned tokens receive its output
    if (kept && !is_centre) slot = seg + 1 + __popc(kept_others & ((1u << lane) - 1u));
    if (kept) core_idx[(int64_t)p * g.Lc + slot] = tok;
    src_slot[(int64_t)p * g.L + tok] = slot;
}

__device__ __forceinline__ void bf16x8_to_f32(const uint4 &u, float out[8])
{
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        out[2 * i] = __uint_as_float(w[i] << 16);
        out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// ---------------------------------------------------------------------------------
// The same selection for the common case dx = 128 and buckets of at most 12 tokens (the
// paper's (2, 3, 2)), with ONE THREAD PER TOKEN.  A block of 256 threads takes 21 buckets
// (12 slots per bucket): thread 12 b + l is local token l of the block's bucket b.
//
// The block first brings the rows of its 252 tokens into shared memory with coalesced
// 16-byte asynchronous copies, sixteen consecutive threads per row.  (A thread reading
// its own row straight from global memory makes every load instruction touch 32 cache
// lines, and the L1 pipeline, not HBM, sets the pace: measured 0.103 ms per layer at 7 heads
// of 118 800 tokens; staged: 0.078 ms.)  Every thread then reads its own row and its
// bucket's centre row from shared memory (rows 272 bytes apart: conflict-free 16-byte
// reads) and keeps fp32 sums of <centre, row> and <row, row>, taken with the
// mixed-precision fma on the bf16 halves as they are; the centre's own <row, row> is the
// centre norm, shared through shared memory.  A warp per bucket with eight lanes per row
// (the first version of this kernel) needed about 850 warp instructions per bucket and
// was bound by instruction issue at 0.088 ms.
//
// Scores are first taken in fp32 (products of bf16 values are exact there; the sums of 128
// terms are not): each cosine is then within 2.5e-5 of its true value.  Only the SET of
// pruned tokens matters, i.e. the order of the k-th and (k+1)-th largest scores, so the
// fp32 ranking is accepted when those two are at least 2^-13 apart.  Otherwise -- near-ties,
// exact ties, rows whose squared norm, or whose product of squared norms with the centre's,
// leaves the range fp32 handles -- the bucket is scored again in fp64 with the formula of
// the general kernel, the sums running over the channels in ascending order like the plain
// definition of the cosine, and ranked on those scores.
// ---------------------------------------------------------------------------------
constexpr int kRowsThreads = 256, kRowsSlots = 12, kRowsBuckets = kRowsThreads / kRowsSlots;
constexpr int kRowsPitch = 272;  // bytes between staged rows: 256 of data, 16 of padding

__global__ void __launch_bounds__(kRowsThreads)
coreset_select_rows_kernel(Geometry g, const __nv_bfloat16 *__restrict__ X, const int32_t *__restrict__ prob_slice,
                           const int32_t *__restrict__ seg_start, const int32_t *__restrict__ bucket_tab,
                           int32_t *__restrict__ core_idx, int32_t *__restrict__ src_slot)
{
    constexpr int32_t dx = 128;
    constexpr float kGuard = 1.220703125e-4f;  // 2^-13
    __shared__ int32_t tab[8 * kBucketTabStride];
    __shared__ int32_t keep_tab[8];
    __shared__ float sc32[kRowsThreads], csq_s[kRowsBuckets], lo_s[kRowsBuckets], hi_s[kRowsBuckets];
    __shared__ double sc64[kRowsThreads], csq64_s[kRowsBuckets];
    __shared__ int32_t doubt_s[kRowsBuckets];
    __shared__ uint8_t kept_s[kRowsThreads];
    __shared__ int32_t tok_s[kRowsThreads];
    extern __shared__ __align__(16) unsigned char rows_smem[];  // [252][kRowsPitch]
    for (int i = threadIdx.x; i < 8 * kBucketTabStride; i += blockDim.x) tab[i] = bucket_tab[i];
    if (threadIdx.x < kRowsBuckets) doubt_s[threadIdx.x] = 0;
    __syncthreads();
    if (threadIdx.x < 8) {
        const int32_t n = tab[threadIdx.x * kBucketTabStride];
        keep_tab[threadIdx.x] = max((int32_t)floor(g.ratio * (double)n + 0.5), 1);
    }

    const int32_t t = threadIdx.x, b = t / kRowsSlots, l = t - b * kRowsSlots;
    const int32_t bkt = blockIdx.x * kRowsBuckets + b;
    const bool has_bucket = b < kRowsBuckets && bkt < g.n_buckets;
    const int32_t p = blockIdx.y;
    const int32_t slice = prob_slice ? prob_slice[p] : p;
    const __nv_bfloat16 *Xs = X + (int64_t)slice * g.Ltot * dx;  // video rows of the slice
    int32_t n = 0, centre = 0, cls = 0, origin = 0, seg = 0;
    if (has_bucket) {
        const int32_t bt = bkt / (g.nb[2] * g.nb[1]), bhw = bkt - bt * (g.nb[2] * g.nb[1]);
        const int32_t bh = bhw / g.nb[2], bw = bhw - bh * g.nb[2];
        cls = ((g.T - bt * g.bucket[0] < g.bucket[0]) ? 4 : 0) | ((g.H - bh * g.bucket[1] < g.bucket[1]) ? 2 : 0) |
              ((g.W - bw * g.bucket[2] < g.bucket[2]) ? 1 : 0);
        origin = (bt * g.bucket[0] * g.H + bh * g.bucket[1]) * g.W + bw * g.bucket[2];
        n = tab[cls * kBucketTabStride];
        centre = tab[cls * kBucketTabStride + 1];
        seg = seg_start[bkt];  // needed at the end: in flight under the scoring
    }
    const bool is_tok = has_bucket && l < n, is_centre = is_tok && l == centre;
    const int32_t tok = is_tok ? origin + tab[cls * kBucketTabStride + 2 + l] : 0;
    // stage the rows: slot s of the block (= thread s's token) at rows_smem + s * kRowsPitch
    tok_s[t] = is_tok ? tok : -1;
    __syncthreads();
    {
        const uint32_t base = static_cast<uint32_t>(__cvta_generic_to_shared(rows_smem));
#pragma unroll 4
        for (int32_t idx = t; idx < kRowsBuckets * kRowsSlots * 16; idx += kRowsThreads) {
            const int32_t slot = idx >> 4, chunk = idx & 15, tk = tok_s[slot];
            if (tk >= 0)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(base + slot * kRowsPitch + chunk * 16),
                             "l"(reinterpret_cast<const unsigned char *>(Xs + (int64_t)tk * dx) + chunk * 16)
                             : "memory");
        }
        asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const uint4 *row = reinterpret_cast<const uint4 *>(rows_smem + (size_t)t * kRowsPitch);
    const uint4 *cen = reinterpret_cast<const uint4 *>(rows_smem + (size_t)(b < kRowsBuckets ? b * kRowsSlots + centre : 0) * kRowsPitch);

    // ---- fp32 sums over the 128 channels
    float dot = 0.f, nsq = 0.f;
    if (is_tok) {
        // four partial sums each (independent chains; the order of an fp32 sum is free here: what the
        // ranking may rest on is decided by the guard band)
        float d4[4] = {0.f, 0.f, 0.f, 0.f}, n4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int i = 0; i < 16; ++i) {
            // the mixed-precision fma takes the bf16 halves of the words as they are (exact products,
            // fp32 sums): no unpacking
            const uint4 cu = cen[i], ru = row[i];
            const uint32_t cw[4] = {cu.x, cu.y, cu.z, cu.w}, rw[4] = {ru.x, ru.y, ru.z, ru.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                unsigned short a0, a1, r0, r1;
                asm("mov.b32 {%0, %1}, %2;" : "=h"(a0), "=h"(a1) : "r"(cw[e]));
                asm("mov.b32 {%0, %1}, %2;" : "=h"(r0), "=h"(r1) : "r"(rw[e]));
                asm("fma.rn.f32.bf16 %0, %1, %2, %0;" : "+f"(d4[e]) : "h"(a0), "h"(r0));
                asm("fma.rn.f32.bf16 %0, %1, %2, %0;" : "+f"(n4[e]) : "h"(r0), "h"(r0));
                asm("fma.rn.f32.bf16 %0, %1, %2, %0;" : "+f"(d4[e]) : "h"(a1), "h"(r1));
                asm("fma.rn.f32.bf16 %0, %1, %2, %0;" : "+f"(n4[e]) : "h"(r1), "h"(r1));
            }
        }
        dot = (d4[0] + d4[1]) + (d4[2] + d4[3]);
        nsq = (n4[0] + n4[1]) + (n4[2] + n4[3]);
    }
    if (is_centre) csq_s[b] = nsq;
    __syncthreads();

    // fp32 score; a bucket with a norm (or a product of norms) outside the range fp32 handles is doubtful
    float my32 = 0.f;
    if (is_tok && !is_centre) {
        const float csq = csq_s[b], prod = csq * nsq;
        if (!(csq > 1e-30f && csq < 1e30f && nsq > 1e-30f && nsq < 1e30f && prod > 1e-30f && prod < 1e30f)) doubt_s[b] = 1;
        my32 = dot * rsqrtf(prod);
    }
    sc32[t] = my32;
    const int32_t keep = keep_tab[cls], k = n - keep;
    __syncthreads();
    // rank among the bucket's other tokens: most similar first, equal scores by ascending index
    int32_t rank = 0;
    if (is_tok && !is_centre) {
        for (int32_t m = 0; m < n; ++m) {
            const float sm = sc32[b * kRowsSlots + m];
            if (m != centre && (sm > my32 || (sm == my32 && m < l))) ++rank;
        }
        // last pruned (rank k-1) and first surviving (rank k) token of the bucket
        if (k > 0 && k < n - 1) {
            if (rank == k - 1) lo_s[b] = my32;
            if (rank == k) hi_s[b] = my32;
        }
    }
    __syncthreads();
    const bool need64 = has_bucket && (doubt_s[b] != 0 || (k > 0 && k < n - 1 && !(lo_s[b] - hi_s[b] >= kGuard)));

    // ---- fp64 scores and ranks for the buckets the guard band does not clear
    double ddot = 0.0, dnsq = 0.0;
    if (is_tok && need64) {
        for (int i = 0; i < 16; ++i) {
            double a[8], r[8];
            bf16x8_to_f64(cen[i], a);
            bf16x8_to_f64(row[i], r);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                ddot = fma(a[e], r[e], ddot);
                dnsq = fma(r[e], r[e], dnsq);
            }
        }
        if (is_centre) csq64_s[b] = dnsq;
    }
    __syncthreads();
    double my64 = 0.0;
    if (is_tok && need64 && !is_centre) {
        const double nc = sqrt(csq64_s[b]), nj = sqrt(dnsq);
        my64 = (nc == 0.0 || nj == 0.0) ? 0.0 : ddot / (nc * nj);
    }
    sc64[t] = my64;
    __syncthreads();
    if (is_tok && need64 && !is_centre) {
        rank = 0;
        for (int32_t m = 0; m < n; ++m) {
            const double sm = sc64[b * kRowsSlots + m];
            if (m != centre && (sm > my64 || (sm == my64 && m < l))) ++rank;
        }
    }

    // ---- the bucket's segment of the index list: centre first, then the other kept tokens ascending
    const bool kept = is_tok && (is_centre || rank >= k);
    kept_s[t] = kept && !is_centre;
    __syncthreads();
    if (!is_tok) return;
    int32_t slot = seg;  // the centre's slot: pruned tokens receive its output
    if (kept && !is_centre) {
        int32_t before = 0;
        for (int32_t m = 0; m < l; ++m) before += kept_s[b * kRowsSlots + m];
        slot = seg + 1 + before;
    }
    if (kept) core_idx[(int64_t)p * g.Lc + slot] = tok;
    src_slot[(int64_t)p * g.L + tok] = slot;
}
cudaError_t launch_select(const Geometry &g, const __nv_bfloat16 *X, int32_t dx, int32_t n_prob,
                          const int32_t *prob_slice, const int32_t *seg_start, const int32_t *bucket_tab,
                          int32_t *core_idx, int32_t *src_slot, cudaStream_t s)
{
    int64_t warps = (int64_t)n_prob * g.n_buckets;
    if (warps == 0) return cudaSuccess;
    if (dx == 128 && g.bucket[0] * g.bucket[1] * g.bucket[2] <= 12 && n_prob <= 65535) {
        constexpr int kSmem = kRowsBuckets * kRowsSlots * kRowsPitch;
        // more than 48 KB of dynamic shared memory has to be asked for, once per device
        static bool attr_set[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return cudaGetLastError();
        if (dev < 0 || dev >= 64 || !attr_set[dev]) {
            cudaError_t ea = cudaFuncSetAttribute(coreset_select_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
            if (ea != cudaSuccess) return ea;
            if (dev >= 0 && dev < 64) attr_set[dev] = true;
        }
        dim3 grid((unsigned)((g.n_buckets + kRowsBuckets - 1) / kRowsBuckets), (unsigned)n_prob);
        coreset_select_rows_kernel<<<grid, kRowsThreads, kSmem, s>>>(g, X, prob_slice, seg_start, bucket_tab, core_idx, src_slot);
    } else {
        int64_t blocks = (warps + 7) / 8;
        coreset_select_kernel<<<(unsigned)blocks, 256, 0, s>>>(g, X, dx, n_prob, prob_slice, seg_start,
                                                               core_idx, src_slot);
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------
// pool: gather the kept rows of Q, K, V into compact [n_prob, Lc, d] tensors.
// 16 bytes per thread; blockIdx.y picks the tensor.
// ---------------------------------------------------------------------------------
// One problem per blockIdx.y, the tensor per blockIdx.z.  A thread owns one 16-byte chunk of a row and
// walks the rows in steps of the grid, four rows at a time (four index loads, then four row loads in
// flight); rows and chunks come from shifts (d / 8 chunks per row is 8 or 16), never from a division.
constexpr int kCopyUnroll = 4;

__global__ void __launch_bounds__(256)
gather_rows_kernel(Geometry g, const int32_t *__restrict__ prob_slice, const int32_t *__restrict__ core_idx,
                   const uint4 *__restrict__ Q, const uint4 *__restrict__ K, const uint4 *__restrict__ V,
                   uint4 *__restrict__ Qc, uint4 *__restrict__ Kc, uint4 *__restrict__ Vc)
{
    const int32_t cpr = g.d >> 3, sh = g.d == 128 ? 4 : 3;  // 16-byte chunks per row
    const int32_t c = (int32_t)threadIdx.x & (cpr - 1), rows_per_block = 256 >> sh;
    const int32_t p = blockIdx.y;
    const int32_t slice = prob_slice ? prob_slice[p] : p;
    const uint4 *src = (blockIdx.z == 0 ? Q : (blockIdx.z == 1 ? K : V)) + (int64_t)slice * g.Ltot * cpr;
    uint4 *dst = (blockIdx.z == 0 ? Qc : (blockIdx.z == 1 ? Kc : Vc)) + (int64_t)p * g.Lct * cpr;
    const int32_t *idx = core_idx + (int64_t)p * g.Lc;
    const int32_t step = (int32_t)gridDim.x * rows_per_block;
    // compact row r of a problem: kept video token core_idx[r] for r < Lc, text token r - Lc after that
    for (int32_t r0 = (int32_t)blockIdx.x * rows_per_block + ((int32_t)threadIdx.x >> sh); r0 < g.Lct; r0 += kCopyUnroll * step) {
        int32_t tok[kCopyUnroll];
        uint4 v[kCopyUnroll];
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u) {
            const int32_t r = r0 + u * step;
            tok[u] = r < g.Lc ? __ldg(idx + r) : g.L + (r - g.Lc);
        }
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u)
            if (r0 + u * step < g.Lct) v[u] = __ldg(src + (int64_t)tok[u] * cpr + c);
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u)
            if (r0 + u * step < g.Lct) dst[(int64_t)(r0 + u * step) * cpr + c] = v[u];
    }
}

// blocks along x for `rows` rows of one problem: enough to fill the GPU a few times over, no more
static unsigned copy_blocks(int64_t rows, int32_t d, int64_t n_launch_y)
{
    const int64_t rows_per_block = 256 / (d >> 3);
    int64_t want = (rows + rows_per_block * kCopyUnroll - 1) / (rows_per_block * kCopyUnroll);
    const int64_t cap = std::max<int64_t>(1, (148 * 16 + n_launch_y - 1) / n_launch_y);
    return (unsigned)std::max<int64_t>(1, std::min(want, cap));
}

cudaError_t launch_gather(const Geometry &g, int32_t n_prob, const int32_t *prob_slice,
                          const int32_t *core_idx, const __nv_bfloat16 *Q, const __nv_bfloat16 *K,
                          const __nv_bfloat16 *V, __nv_bfloat16 *Qc, __nv_bfloat16 *Kc,
                          __nv_bfloat16 *Vc, cudaStream_t s)
{
    if (n_prob == 0) return cudaSuccess;
    gather_rows_kernel<<<dim3(copy_blocks(g.Lct, g.d, (int64_t)n_prob * 3), (unsigned)n_prob, 3), 256, 0, s>>>(
        g, prob_slice, core_idx, reinterpret_cast<const uint4 *>(Q),
        reinterpret_cast<const uint4 *>(K), reinterpret_cast<const uint4 *>(V),
        reinterpret_cast<uint4 *>(Qc), reinterpret_cast<uint4 *>(Kc), reinterpret_cast<uint4 *>(Vc));
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------
// Optional merge (Section 3.2: the pruned tokens' information is merged into the centre;
// read here as the plain mean): after the gather, the centre's compact rows of Q, K and V
// become the mean over the centre and the tokens pruned from its bucket.  One warp per
// (problem, bucket); a lane owns one 16-byte chunk of one of the three rows; fp32 sums,
// one rounding to bf16.
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
merge_centres_kernel(Geometry g, const int32_t *__restrict__ prob_slice, const int32_t *__restrict__ seg_start,
                     const int32_t *__restrict__ bucket_tab, const int32_t *__restrict__ src_slot,
                     const uint4 *__restrict__ Q, const uint4 *__restrict__ K, const uint4 *__restrict__ V,
                     uint4 *__restrict__ Qc, uint4 *__restrict__ Kc, uint4 *__restrict__ Vc)
{
    __shared__ int32_t tab[8 * kBucketTabStride];
    for (int i = threadIdx.x; i < 8 * kBucketTabStride; i += blockDim.x) tab[i] = bucket_tab[i];
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int32_t bkt = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (bkt >= g.n_buckets) return;
    const int32_t p = blockIdx.y;
    const int32_t slice = prob_slice ? prob_slice[p] : p;
    const int32_t bt = bkt / (g.nb[2] * g.nb[1]), bhw = bkt - bt * (g.nb[2] * g.nb[1]);
    const int32_t bh = bhw / g.nb[2], bw = bhw - bh * g.nb[2];
    const int32_t cls = ((g.T - bt * g.bucket[0] < g.bucket[0]) ? 4 : 0) | ((g.H - bh * g.bucket[1] < g.bucket[1]) ? 2 : 0) |
                        ((g.W - bw * g.bucket[2] < g.bucket[2]) ? 1 : 0);
    const int32_t *t = tab + cls * kBucketTabStride;
    const int32_t n = t[0], centre = t[1];
    const int32_t origin = (bt * g.bucket[0] * g.H + bh * g.bucket[1]) * g.W + bw * g.bucket[2];
    const int32_t seg = seg_start[bkt];
    const int32_t my_tok = lane < n ? origin + t[2 + lane] : 0;
    const bool mine = lane < n && (lane == centre || src_slot[(int64_t)p * g.L + my_tok] == seg);
    uint32_t members = __ballot_sync(0xffffffffu, mine);  // the centre and the tokens pruned into it
    const int32_t count = __popc(members);
    if (count <= 1) return;  // warp-uniform
    const int32_t cpr = g.d >> 3;
    const float inv = 1.f / (float)count;
    for (int32_t idx = lane; idx < 3 * cpr; idx += 32) {
        const int32_t which = idx / cpr, c = idx - which * cpr;
        const uint4 *src = which == 0 ? Q : (which == 1 ? K : V);
        uint4 *dst = which == 0 ? Qc : (which == 1 ? Kc : Vc);
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (uint32_t m = members; m; m &= m - 1) {
            const int32_t l = __ffs(m) - 1;
            const int32_t tok = origin + t[2 + l];
            const uint4 u = __ldg(src + ((int64_t)slice * g.Ltot + tok) * cpr + c);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                acc[2 * i] += __uint_as_float(w[i] << 16);
                acc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
            }
        }
        uint32_t r[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 v = __floats2bfloat162_rn(acc[2 * i] * inv, acc[2 * i + 1] * inv);
            r[i] = *reinterpret_cast<uint32_t *>(&v);
        }
        dst[((int64_t)p * g.Lct + seg) * cpr + c] = make_uint4(r[0], r[1], r[2], r[3]);
    }
}

cudaError_t launch_merge(const Geometry &g, int32_t n_prob, const int32_t *prob_slice, const int32_t *seg_start,
                         const int32_t *bucket_tab, const int32_t *src_slot, const __nv_bfloat16 *Q,
                         const __nv_bfloat16 *K, const __nv_bfloat16 *V, __nv_bfloat16 *Qc, __nv_bfloat16 *Kc,
                         __nv_bfloat16 *Vc, cudaStream_t s)
{
    if (n_prob == 0) return cudaSuccess;
    dim3 grid((unsigned)((g.n_buckets + 7) / 8), (unsigned)n_prob);
    merge_centres_kernel<<<grid, 256, 0, s>>>(g, prob_slice, seg_start, bucket_tab, src_slot,
                                              reinterpret_cast<const uint4 *>(Q), reinterpret_cast<const uint4 *>(K),
                                              reinterpret_cast<const uint4 *>(V), reinterpret_cast<uint4 *>(Qc),
                                              reinterpret_cast<uint4 *>(Kc), reinterpret_cast<uint4 *>(Vc));
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------
// unpool: every token of a core-set head receives the output row of its slot
// (its own row if kept, its bucket centre's row if pruned).
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
scatter_rows_kernel(Geometry g, const int32_t *__restrict__ prob_slice, const int32_t *__restrict__ src_slot,
                    const uint4 *__restrict__ Oc, uint4 *__restrict__ O)
{
    const int32_t cpr = g.d >> 3, sh = g.d == 128 ? 4 : 3;
    const int32_t c = (int32_t)threadIdx.x & (cpr - 1), rows_per_block = 256 >> sh;
    const int32_t p = blockIdx.y;
    const int32_t slice = prob_slice ? prob_slice[p] : p;
    const uint4 *src = Oc + (int64_t)p * g.Lct * cpr;
    uint4 *dst = O + (int64_t)slice * g.Ltot * cpr;
    const int32_t *slots = src_slot + (int64_t)p * g.L;
    const int32_t step = (int32_t)gridDim.x * rows_per_block;
    // a video token takes the row of its slot, a text token its own compact row
    for (int32_t t0 = (int32_t)blockIdx.x * rows_per_block + ((int32_t)threadIdx.x >> sh); t0 < g.Ltot; t0 += kCopyUnroll * step) {
        int32_t slot[kCopyUnroll];
        uint4 v[kCopyUnroll];
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u) {
            const int32_t tok = t0 + u * step;
            slot[u] = tok < g.L ? __ldg(slots + tok) : g.Lc + (tok - g.L);
        }
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u)
            if (t0 + u * step < g.Ltot) v[u] = __ldg(src + (int64_t)slot[u] * cpr + c);
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u)
            if (t0 + u * step < g.Ltot) dst[(int64_t)(t0 + u * step) * cpr + c] = v[u];
    }
}

cudaError_t launch_scatter(const Geometry &g, int32_t n_prob, const int32_t *prob_slice,
                           const int32_t *src_slot, const __nv_bfloat16 *Oc, __nv_bfloat16 *O,
                           cudaStream_t s)
{
    if (n_prob == 0) return cudaSuccess;
    scatter_rows_kernel<<<dim3(copy_blocks(g.Ltot, g.d, n_prob), (unsigned)n_prob), 256, 0, s>>>(
        g, prob_slice, src_slot, reinterpret_cast<const uint4 *>(Oc), reinterpret_cast<uint4 *>(O));
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------
// Router (Section 3.3, Eq. 3-4): gates = softmax(T W_R) per head, and the branch the
// inference rule picks: sliding if its gate is strictly the largest, core-set if its
// gate is strictly the largest, full otherwise (so every tie goes to full).  One warp
// per head; fp64 accumulation of fp32 inputs; the rule is evaluated on the logits,
// which order exactly like the gates.
// ---------------------------------------------------------------------------------
__global__ void router_kernel(const float *__restrict__ T, const float *__restrict__ WR, int32_t d_model,
                              int32_t heads, float *__restrict__ gates, uint8_t *__restrict__ routes)
{
    const int lane = threadIdx.x & 31;
    const int32_t h = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (h >= heads) return;
    const float *W = WR + (int64_t)h * d_model * 3;
    double l[3] = {0.0, 0.0, 0.0};
    for (int32_t c = lane; c < d_model; c += 32) {
        const double t = (double)T[c];
#pragma unroll
        for (int r = 0; r < 3; ++r) l[r] = fma(t, (double)W[c * 3 + r], l[r]);
    }
#pragma unroll
    for (int r = 0; r < 3; ++r)
        for (int m = 16; m >= 1; m >>= 1) l[r] += shfl_xor_f64(l[r], m);
    if (lane != 0) return;
    const double mx = fmax(l[0], fmax(l[1], l[2]));
    const double e0 = exp(l[0] - mx), e1 = exp(l[1] - mx), e2 = exp(l[2] - mx), z = e0 + e1 + e2;
    gates[h * 3 + 0] = (float)(e0 / z);
    gates[h * 3 + 1] = (float)(e1 / z);
    gates[h * 3 + 2] = (float)(e2 / z);
    uint8_t route = VORTA_ROUTE_FULL;
    if (l[1] > l[0] && l[1] > l[2]) route = VORTA_ROUTE_SLIDING;
    else if (l[2] > l[0] && l[2] > l[1]) route = VORTA_ROUTE_CORESET;
    routes[h] = route;
}

cudaError_t launch_router(const float *T, const float *WR, int32_t d_model, int32_t heads, float *gates,
                          uint8_t *routes, cudaStream_t s)
{
    router_kernel<<<(heads * 32 + 127) / 128, 128, 0, s>>>(T, WR, d_model, heads, gates, routes);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------
// Soft mixture (Section 3.3, Eq. 5): O = a1 * full + a2 * sliding + a3 * core-set per head,
// from the three branch outputs [3, B*heads, L, d]; fp32 arithmetic, bf16 result.
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
mix_combine_kernel(Geometry g, const float *__restrict__ gates, const uint4 *__restrict__ branches,
                   uint4 *__restrict__ O)
{
    const int32_t cpr = g.d >> 3;
    const int64_t per_slice = (int64_t)g.Ltot * cpr, total = (int64_t)g.B * g.heads * per_slice;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t h = (int32_t)((i / per_slice) % g.heads);
        const float a0 = __ldg(gates + h * 3), a1 = __ldg(gates + h * 3 + 1), a2 = __ldg(gates + h * 3 + 2);
        const uint4 x = __ldg(branches + i), y = __ldg(branches + total + i), z = __ldg(branches + 2 * total + i);
        const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w}, zs[4] = {z.x, z.y, z.z, z.w};
        uint32_t r[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float lo = a0 * __uint_as_float(xs[k] << 16) + a1 * __uint_as_float(ys[k] << 16) +
                             a2 * __uint_as_float(zs[k] << 16);
            const float hi = a0 * __uint_as_float(xs[k] & 0xffff0000u) + a1 * __uint_as_float(ys[k] & 0xffff0000u) +
                             a2 * __uint_as_float(zs[k] & 0xffff0000u);
            __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
            r[k] = *reinterpret_cast<uint32_t *>(&v);
        }
        O[i] = make_uint4(r[0], r[1], r[2], r[3]);
    }
}

cudaError_t launch_mix_combine(const Geometry &g, const float *gates, const __nv_bfloat16 *branches,
                               __nv_bfloat16 *O, cudaStream_t s)
{
    int64_t total = (int64_t)g.B * g.heads * g.Ltot * (g.d >> 3);
    unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    mix_combine_kernel<<<blocks, 256, 0, s>>>(g, gates, reinterpret_cast<const uint4 *>(branches),
                                              reinterpret_cast<uint4 *>(O));
    return cudaGetLastError();
}

}  // namespace vorta
