// Memory-bound kernels of the routed-attention layer: the block-sparse sliding-tile
// mask builder, bucketed core-set selection, the gather (pool) of the kept rows
// and the scatter (unpool) of the attention output.
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
__global__ void kv_list_kernel(Geometry g, const uint8_t *__restrict__ bm, KvEntry *__restrict__ list,
                               int32_t *__restrict__ count)
{
    int32_t qt = blockIdx.x * blockDim.x + threadIdx.x;
    if (qt >= g.n_tiles) return;
    KvEntry *out = list + (int64_t)qt * g.max_kv_per_tile;
    // Two passes: the boxes that lie wholly inside the grid (mask class 0) first, the cut
    // ones after them, so that the attention kernel can run the leading blocks without
    // any masking.  count[n_tiles + qt] is the number of leading whole boxes.
    int32_t n = 0, n_whole = 0;
    for (int pass = 0; pass < 2; ++pass) {
        for (int32_t kt = 0; kt < g.n_tiles; ++kt) {
            if (!bm[(int64_t)qt * g.n_tiles + kt]) continue;
            int32_t k[3];
            tile_triple(g, kt, k);
            int32_t t0 = k[0] * g.tile[0], h0 = k[1] * g.tile[1], w0 = k[2] * g.tile[2];
            int32_t pt = (g.T - t0 < g.tile[0]), ph = (g.H - h0 < g.tile[1]), pw = (g.W - w0 < g.tile[2]);
            bool whole = !pt && !ph && !pw && g.box_rows == g.bn_tile;
            if (whole != (pass == 0)) continue;
            for (int32_t bx = 0; bx < g.boxes_per_tile; ++bx) {
                // box bx of the tile; boxes that start outside the grid are dropped
                int32_t tb = t0 + (bx / (g.nbox[1] * g.nbox[2])) * g.box[0];
                int32_t hb = h0 + ((bx / g.nbox[2]) % g.nbox[1]) * g.box[1];
                int32_t wb = w0 + (bx % g.nbox[2]) * g.box[2];
                if (tb >= g.T || hb >= g.H || wb >= g.W) continue;
                if (n < g.max_kv_per_tile) {
                    KvEntry e;
                    e.w0 = (int16_t)wb;
                    e.h0 = (int16_t)hb;
                    e.t0 = (int16_t)tb;
                    e.mask_id = whole ? 0 : (uint16_t)(1 + ((pt * 2 + ph) * 2 + pw) * g.boxes_per_tile + bx);
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
                              cudaStream_t s)
{
    int64_t total = (int64_t)g.n_tiles * g.n_tiles;
    block_mask_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(g, bm);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    kv_list_kernel<<<(g.n_tiles + 127) / 128, 128, 0, s>>>(g, bm, kv_list, kv_count);
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

// The same selection for the common case dx = 128 and buckets of at most 12 tokens
// (the paper's (2, 3, 2)).  Every lane first issues the loads of all its chunks -- its
// share of the centre row and of the three token rows it helps to score -- so that a
// warp has the whole bucket in flight before any arithmetic.
//
// Scores are first taken in fp32 (products of bf16 values are exact there; the sums of
// 128 terms are not): each cosine is then within 2.5e-5 of its true value.  Only the SET
// of pruned tokens matters, i.e. the order of the k-th and (k+1)-th largest scores, so
// the fp32 ranking is accepted when those two are at least 2^-13 apart.  Otherwise --
// near-ties, exact ties, rows with a vanishing or non-finite squared norm in fp32 -- the
// bucket is scored again in fp64 with the formula of the general kernel, from the same
// registers, and ranked on those scores.  The results are those of the general kernel.
__device__ __forceinline__ void bf16x8_to_f32(const uint4 &u, float out[8])
{
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        out[2 * i] = __uint_as_float(w[i] << 16);
        out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

__global__ void __launch_bounds__(256, 4)
coreset_select_d128_kernel(Geometry g, const __nv_bfloat16 *__restrict__ X, const int32_t *__restrict__ prob_slice,
                           const int32_t *__restrict__ seg_start, const int32_t *__restrict__ bucket_tab,
                           int32_t *__restrict__ core_idx, int32_t *__restrict__ src_slot)
{
    constexpr int32_t dx = 128, kPasses = 3;
    constexpr float kGuard = 1.220703125e-4f;  // 2^-13
    // bucket shape classes (which axes the grid cuts): token count, centre, token offsets
    __shared__ int32_t tab[8 * kBucketTabStride];
    for (int i = threadIdx.x; i < 8 * kBucketTabStride; i += blockDim.x) tab[i] = bucket_tab[i];
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int32_t bkt = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (bkt >= g.n_buckets) return;
    const int32_t p = blockIdx.y;
    const int32_t slice = prob_slice ? prob_slice[p] : p;
    const __nv_bfloat16 *Xs = X + (int64_t)slice * g.Ltot * dx;  // video rows of the slice

    const int32_t bt = bkt / (g.nb[2] * g.nb[1]), bhw = bkt - bt * (g.nb[2] * g.nb[1]);
    const int32_t bh = bhw / g.nb[2], bw = bhw - bh * g.nb[2];
    const int32_t cls = ((g.T - bt * g.bucket[0] < g.bucket[0]) ? 4 : 0) | ((g.H - bh * g.bucket[1] < g.bucket[1]) ? 2 : 0) |
                        ((g.W - bw * g.bucket[2] < g.bucket[2]) ? 1 : 0);
    const int32_t *t = tab + cls * kBucketTabStride;
    const int32_t n = t[0], centre = t[1];
    const int32_t origin = (bt * g.bucket[0] * g.H + bh * g.bucket[1]) * g.W + bw * g.bucket[2];
    auto token_of = [&](int32_t l) -> int32_t { return origin + t[2 + l]; };

    const int sub = lane >> 3, sl = lane & 7;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    const uint4 *xc = reinterpret_cast<const uint4 *>(Xs + (int64_t)token_of(centre) * dx);
    const uint4 c0 = __ldg(xc + sl), c1 = __ldg(xc + sl + 8);
    uint4 r[kPasses][2];
#pragma unroll
    for (int pass = 0; pass < kPasses; ++pass) {
        const int32_t l = pass * 4 + sub;
        r[pass][0] = zero;
        r[pass][1] = zero;
        if (l < n) {
            const uint4 *xj = reinterpret_cast<const uint4 *>(Xs + (int64_t)token_of(l) * dx);
            r[pass][0] = __ldg(xj + sl);
            r[pass][1] = __ldg(xj + sl + 8);
        }
    }

    int32_t keep = (int32_t)floor(g.ratio * (double)n + 0.5);
    keep = max(keep, 1);
    const int32_t k = n - keep;
    const bool is_tok = lane < n, is_centre = lane == centre;

    // ---- fp32 scores and ranks
    float my32 = 0.f;
    bool doubtful = false;
    {
        float csq = 0.f;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float a[8];
            bf16x8_to_f32(h ? c1 : c0, a);
#pragma unroll
            for (int i = 0; i < 8; ++i) csq = fmaf(a[i], a[i], csq);
        }
#pragma unroll
        for (int m = 4; m >= 1; m >>= 1) csq += __shfl_xor_sync(0xffffffffu, csq, m);
        doubtful = !(csq > 1e-30f && csq < 1e30f);
#pragma unroll
        for (int pass = 0; pass < kPasses; ++pass) {
            if (pass * 4 >= n) break;  // warp-uniform
            float dot = 0.f, njsq = 0.f;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float a[8], b[8];
                bf16x8_to_f32(h ? c1 : c0, a);
                bf16x8_to_f32(r[pass][h], b);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    dot = fmaf(a[i], b[i], dot);
                    njsq = fmaf(b[i], b[i], njsq);
                }
            }
#pragma unroll
            for (int m = 4; m >= 1; m >>= 1) {
                dot += __shfl_xor_sync(0xffffffffu, dot, m);
                njsq += __shfl_xor_sync(0xffffffffu, njsq, m);
            }
            // the product of the two squared norms must itself be an ordinary fp32 number: two small
            // norms (or two large ones) each pass the range test and still underflow (overflow) together,
            // and the infinite or zero score that follows would slip through the guard band
            const float nsq = csq * njsq;
            if (pass * 4 + sub < n && !(njsq > 1e-30f && njsq < 1e30f && nsq > 1e-30f && nsq < 1e30f)) doubtful = true;
            const float score = dot * rsqrtf(nsq);
            const float got = __shfl_sync(0xffffffffu, score, (lane & 3) * 8);
            if ((lane >> 2) == pass) my32 = got;
        }
    }
    int32_t rank = 0;
    for (int32_t m = 0; m < n; ++m) {
        const float sm = __shfl_sync(0xffffffffu, my32, m);
        if (m != centre && (sm > my32 || (sm == my32 && m < lane))) ++rank;
    }
    bool need64 = __any_sync(0xffffffffu, doubtful);
    if (!need64 && k > 0 && k < n - 1) {
        // last pruned (rank k-1) against first surviving (rank k) token
        const uint32_t b_lo = __ballot_sync(0xffffffffu, is_tok && !is_centre && rank == k - 1);
        const uint32_t b_hi = __ballot_sync(0xffffffffu, is_tok && !is_centre && rank == k);
        const float s_lo = __shfl_sync(0xffffffffu, my32, __ffs(b_lo) - 1);
        const float s_hi = __shfl_sync(0xffffffffu, my32, __ffs(b_hi) - 1);
        need64 = !(s_lo - s_hi >= kGuard);
    }

    // ---- fp64 scores and ranks for the buckets the guard band does not clear
    if (need64) {
        // (the summation order differs from the general kernel's only in grouping by chunk)
        double csq = 0.0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            double a[8];
            bf16x8_to_f64(h ? c1 : c0, a);
#pragma unroll
            for (int i = 0; i < 8; ++i) csq = fma(a[i], a[i], csq);
        }
#pragma unroll
        for (int m = 4; m >= 1; m >>= 1) csq += shfl_xor_f64(csq, m);
        const double nc = sqrt(csq);
        double my64 = 0.0;
#pragma unroll 1
        for (int pass = 0; pass < kPasses; ++pass) {
            if (pass * 4 >= n) break;
            double dot = 0.0, njsq = 0.0;
            const uint4 rp0 = pass == 0 ? r[0][0] : (pass == 1 ? r[1][0] : r[2][0]);
            const uint4 rp1 = pass == 0 ? r[0][1] : (pass == 1 ? r[1][1] : r[2][1]);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                double a[8], b[8];
                bf16x8_to_f64(h ? c1 : c0, a);
                bf16x8_to_f64(h ? rp1 : rp0, b);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    dot = fma(a[i], b[i], dot);
                    njsq = fma(b[i], b[i], njsq);
                }
            }
#pragma unroll
            for (int m = 4; m >= 1; m >>= 1) {
                dot += shfl_xor_f64(dot, m);
                njsq += shfl_xor_f64(njsq, m);
            }
            const double nj = sqrt(njsq);
            const double score = (nc == 0.0 || nj == 0.0) ? 0.0 : dot / (nc * nj);
            const double got = shfl_f64(score, (lane & 3) * 8);
            if ((lane >> 2) == pass) my64 = got;
        }
        rank = 0;
        for (int32_t m = 0; m < n; ++m) {
            const double sm = shfl_f64(my64, m);
            if (m != centre && (sm > my64 || (sm == my64 && m < lane))) ++rank;
        }
    }

    const bool kept = is_tok && (is_centre || rank >= k);
    const uint32_t kept_others = __ballot_sync(0xffffffffu, kept && !is_centre);
    if (!is_tok) return;
    const int32_t seg = seg_start[bkt];
    const int32_t tok = token_of(lane);
    int32_t slot = seg;
    if (kept && !is_centre) slot = seg + 1 + __popc(kept_others & ((1u << lane) - 1u));
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
        dim3 grid((unsigned)((g.n_buckets + 7) / 8), (unsigned)n_prob);
        coreset_select_d128_kernel<<<grid, 256, 0, s>>>(g, X, prob_slice, seg_start, bucket_tab, core_idx, src_slot);
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
__global__ void __launch_bounds__(256)
gather_rows_kernel(Geometry g, int32_t n_prob, const int32_t *__restrict__ prob_slice,
                   const int32_t *__restrict__ core_idx, const uint4 *__restrict__ Q,
                   const uint4 *__restrict__ K, const uint4 *__restrict__ V, uint4 *__restrict__ Qc,
                   uint4 *__restrict__ Kc, uint4 *__restrict__ Vc)
{
    const int32_t cpr = g.d >> 3;  // 16-byte chunks per row
    // compact row r of a problem: kept video token core_idx[r] for r < Lc, text token r - Lc after that
    const int64_t total = (int64_t)n_prob * g.Lct * cpr;
    const uint4 *src = blockIdx.y == 0 ? Q : (blockIdx.y == 1 ? K : V);
    uint4 *dst = blockIdx.y == 0 ? Qc : (blockIdx.y == 1 ? Kc : Vc);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        int64_t row = i / cpr;
        int32_t c = (int32_t)(i % cpr);
        int32_t p = (int32_t)(row / g.Lct);
        int32_t r = (int32_t)(row % g.Lct);
        int32_t tok = r < g.Lc ? __ldg(core_idx + (int64_t)p * g.Lc + r) : g.L + (r - g.Lc);
        const int32_t slice = prob_slice ? prob_slice[p] : p;
        dst[i] = __ldg(src + ((int64_t)slice * g.Ltot + tok) * cpr + c);
    }
}

cudaError_t launch_gather(const Geometry &g, int32_t n_prob, const int32_t *prob_slice,
                          const int32_t *core_idx, const __nv_bfloat16 *Q, const __nv_bfloat16 *K,
                          const __nv_bfloat16 *V, __nv_bfloat16 *Qc, __nv_bfloat16 *Kc,
                          __nv_bfloat16 *Vc, cudaStream_t s)
{
    if (n_prob == 0) return cudaSuccess;
    int64_t total = (int64_t)n_prob * g.Lct * (g.d >> 3);
    unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    gather_rows_kernel<<<dim3(blocks, 3), 256, 0, s>>>(
        g, n_prob, prob_slice, core_idx, reinterpret_cast<const uint4 *>(Q),
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
scatter_rows_kernel(Geometry g, int32_t n_prob, const int32_t *__restrict__ prob_slice,
                    const int32_t *__restrict__ src_slot, const uint4 *__restrict__ Oc,
                    uint4 *__restrict__ O)
{
    const int32_t cpr = g.d >> 3;
    // a video token takes the row of its slot, a text token its own compact row
    const int64_t total = (int64_t)n_prob * g.Ltot * cpr;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        int64_t row = i / cpr;
        int32_t c = (int32_t)(i % cpr);
        int32_t p = (int32_t)(row / g.Ltot);
        int32_t tok = (int32_t)(row % g.Ltot);
        int32_t slot = tok < g.L ? __ldg(src_slot + (int64_t)p * g.L + tok) : g.Lc + (tok - g.L);
        const int32_t slice = prob_slice ? prob_slice[p] : p;
        O[((int64_t)slice * g.Ltot + tok) * cpr + c] = __ldg(Oc + ((int64_t)p * g.Lct + slot) * cpr + c);
    }
}

cudaError_t launch_scatter(const Geometry &g, int32_t n_prob, const int32_t *prob_slice,
                           const int32_t *src_slot, const __nv_bfloat16 *Oc, __nv_bfloat16 *O,
                           cudaStream_t s)
{
    if (n_prob == 0) return cudaSuccess;
    int64_t total = (int64_t)n_prob * g.Ltot * (g.d >> 3);
    unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    scatter_rows_kernel<<<blocks, 256, 0, s>>>(g, n_prob, prob_slice, src_slot,
                                               reinterpret_cast<const uint4 *>(Oc),
                                               reinterpret_cast<uint4 *>(O));
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
