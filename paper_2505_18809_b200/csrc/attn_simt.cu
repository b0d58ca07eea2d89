// A slow CUDA-core attention kernel over the same work items, KV lists and column
// masks as the tensor-core kernel.  It exists to tell apart faults in the work
// lists from faults in the tcgen05 pipeline; it is never the default.
#include "vorta_internal.h"

namespace vorta {

namespace {

constexpr int kKvChunk = 32;  // keys staged in shared memory at a time

template <int D>
__global__ void __launch_bounds__(256)
attention_simt_kernel(AttnParams p)
{
    __shared__ __align__(16) __nv_bfloat16 sK[kKvChunk][D];
    __shared__ __align__(16) __nv_bfloat16 sV[kKvChunk][D];
    __shared__ int32_t sTok[kKvChunk];  // token (row) id of each staged key, -1 = masked

    const Geometry &g = p.g;
    const WorkItem w = p.items[blockIdx.x];
    const int mblk = threadIdx.x >> 7, r = threadIdx.x & 127;
    const bool compact = w.mode == MODE_COMPACT;
    const __nv_bfloat16 *Q = compact ? p.Qc : p.Q, *K = compact ? p.Kc : p.K, *V = compact ? p.Vc : p.V;
    __nv_bfloat16 *O = compact ? p.Oc : p.O;
    const int64_t rows = compact ? g.Lct : g.Ltot;
    const int64_t base = (int64_t)w.slice * rows * D;
    const float scale = p.scale_log2 * 0.6931471805599453f;

    int32_t qtok = 0;
    // packed item: rows 0-63 of the one query block are the first tile's, rows 64-127 the second's
    const bool packed = (w.flags & kItemPacked) != 0;
    const uint32_t my_vis = packed ? 1u + (uint32_t)(r >> 6) : 0u;
    const bool q_valid = mblk < w.n_mblk &&
                         block_row_token(g, w.mode, w.q_org[packed ? (r >> 6) : mblk], w.kv_len, packed ? (r & 63) : r, &qtok);
    __nv_bfloat162 q[D / 2];  // packed: the row and its accumulator must both fit in registers
    float acc[D];
#pragma unroll
    for (int c = 0; c < D / 2; ++c) {
        q[c] = q_valid ? *reinterpret_cast<const __nv_bfloat162 *>(Q + base + (int64_t)qtok * D + 2 * c)
                       : __floats2bfloat162_rn(0.f, 0.f);
        acc[2 * c] = 0.f;
        acc[2 * c + 1] = 0.f;
    }
    float m = -INFINITY, l = 0.f;

    const int32_t bn = w.mode == MODE_TILES ? g.bn_tile : kBlockM;
    for (int32_t j = 0; j < w.kv_count; ++j) {
        int32_t org[3];
        uint32_t mask[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};
        // the last kv_text blocks of a sliding item are runs of bn_tile text tokens (rows L + ...)
        const bool text = w.mode == MODE_TILES && j >= w.kv_count - w.kv_text;
        int32_t kv_mode = w.mode, kv_len = w.kv_len;
        uint32_t vis = 0;  // packed items: which of the two tiles sees the block (0: both)
        bool paired = false;  // the block is two 64-row boxes: this one and the same box one tile further along W
        if (text) {
            kv_mode = MODE_LINEAR;
            kv_len = g.Ltot;
            org[0] = g.L + (j - (w.kv_count - w.kv_text)) * g.bn_tile; org[1] = 0; org[2] = 0;
        } else if (w.mode == MODE_TILES) {
            KvEntry e = (item_uses_pair_list(w.flags) ? p.kv_pairs : p.kv_list)[w.kv_begin + j];
            org[0] = e.w0; org[1] = e.h0; org[2] = e.t0;
            vis = e.mask_id >> kVisShift;
            paired = (e.mask_id & kEntryPaired) != 0;
            const uint32_t id = e.mask_id & kMaskIdBits;
            if (id)
                for (int i = 0; i < 4; ++i) mask[i] = p.colmasks[id * 4 + i];
        } else {
            org[0] = j * kBlockM; org[1] = 0; org[2] = 0;
        }
        for (int32_t c0 = 0; c0 < bn; c0 += kKvChunk) {
            __syncthreads();
            if (threadIdx.x < kKvChunk) {
                int32_t n = c0 + threadIdx.x, tok = -1, t;
                int32_t o2[3] = {org[0], org[1], org[2]}, nn = n;
                if (paired && n >= 64) {
                    o2[0] += g.tile[2];
                    nn = n - 64;
                }
                if (n < bn && (!paired || nn < 64) && ((mask[n >> 5] >> (n & 31)) & 1u) &&
                    block_row_token(g, kv_mode, o2, kv_len, nn, &t))
                    tok = t;
                sTok[threadIdx.x] = tok;
            }
            __syncthreads();
            for (int i = threadIdx.x; i < kKvChunk * (D / 8); i += blockDim.x) {
                int n = i / (D / 8), c = i % (D / 8);
                int32_t tok = sTok[n];
                uint4 kk = make_uint4(0, 0, 0, 0), vv = kk;
                if (tok >= 0) {
                    kk = *reinterpret_cast<const uint4 *>(K + base + (int64_t)tok * D + c * 8);
                    vv = *reinterpret_cast<const uint4 *>(V + base + (int64_t)tok * D + c * 8);
                }
                *reinterpret_cast<uint4 *>(&sK[n][c * 8]) = kk;
                *reinterpret_cast<uint4 *>(&sV[n][c * 8]) = vv;
            }
            __syncthreads();
            if (!q_valid || (vis && vis != my_vis)) continue;
            for (int n = 0; n < kKvChunk; ++n) {
                if (sTok[n] < 0) continue;
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < D / 2; ++c) {
                    float2 qq = __bfloat1622float2(q[c]);
                    float2 kk = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&sK[n][2 * c]));
                    s = fmaf(qq.x, kk.x, s);
                    s = fmaf(qq.y, kk.y, s);
                }
                s *= scale;
                if (s > m) {
                    float a = __expf(m - s);
                    l *= a;
#pragma unroll
                    for (int c = 0; c < D; ++c) acc[c] *= a;
                    m = s;
                }
                float pj = __expf(s - m);
                l += pj;
#pragma unroll
                for (int c = 0; c < D; ++c) acc[c] = fmaf(pj, __bfloat162float(sV[n][c]), acc[c]);
            }
        }
    }
    if (q_valid) {
        float inv = 1.f / l;
        __nv_bfloat16 *o = O + (int64_t)(compact ? w.slice : w.out_slice) * rows * D + (int64_t)qtok * D;
#pragma unroll
        for (int c = 0; c < D; c += 2)
            *reinterpret_cast<__nv_bfloat162 *>(o + c) = __floats2bfloat162_rn(acc[c] * inv, acc[c + 1] * inv);
    }
}

}  // namespace

cudaError_t launch_attention_simt(const AttnParams &p, int32_t n_items, cudaStream_t s)
{
    if (p.g.d == 128)
        attention_simt_kernel<128><<<n_items, 256, 0, s>>>(p);
    else
        attention_simt_kernel<64><<<n_items, 256, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace vorta
