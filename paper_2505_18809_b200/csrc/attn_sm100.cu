// Persistent route-dispatching attention kernel for sm_100a.
//
// One CTA per SM walks its share of the work items.  An item is up to two
// 128-row query blocks (tiles 0 and 1) that share one sequence of KV blocks:
//   full head      128 consecutive tokens per block, all KV blocks of the head;
//   sliding head   one 3D (sub-)tile per block, the KV boxes of the tiles in its
//                  window (Algorithm 1), fetched by 5-D TMA boxes straight from
//                  the row-major [T, H, W, d] layout;
//   core-set head  like a full head, over the gathered rows.
//
// Warp roles (320 threads; every role is compiled for the launch bound's 168 registers,
// three warps on an SM sub-partition's 16 K registers; no setmaxnreg):
//   warp 0        TMA producer: Q once per item, then K_j, V_j into a 4-slot ring
//   warp 1        TMEM allocation; MMA issuer: S = Q K^T and O += P V as tcgen05.mma,
//                 accumulators in TMEM
//   warps 2-5     softmax of tile 0 (one thread per query row = one TMEM lane; a warp
//                 reaches the 32 lanes of TMEM quadrant warp % 4)
//   warps 6-9     softmax of tile 1
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512).  A KV block of up
// to 128 keys is worked through as sub-blocks of up to 64 keys, and the S region of a
// tile is two 64-column buffers that successive sub-blocks alternate between: while
// the softmax threads turn S(u) into P(u) (bf16, written over the first half of the
// same buffer) the scores S(u+1) already wait in the other buffer, and the MMA warp
// issues O += P(u) V(u) followed by S(u+2) = Q K(u+2)^T into the buffer P(u) leaves.
// The softmax threads therefore never wait for the tensor pipe in steady state, and
// the tensor pipe always has the other tile's MMAs queued.  Softmax is the usual
// online form in the log2 domain with a lazy accumulator rescale (only when the row
// maximum grew by more than 2^8), done by the softmax threads themselves once the
// PV MMAs issued so far have completed.
//
// Every wait is bounded: a wait that sees no progress for about two seconds
// records a code in the status word, raises the CTA's abort flag and every role
// leaves its loop; the CTA then gives outstanding copies time to land, frees its
// TMEM and returns.
#include <type_traits>

#include "sm100_common.cuh"

namespace vorta {

namespace {

using namespace sm100;

constexpr int kStages = 4;                // KV ring slots (K and V blocks alternate)
constexpr uint32_t kHalfBytes = 16384;    // 128 rows x 64 bf16: one swizzled half tile
constexpr uint32_t kTileBytes = 32768;    // two halves (d = 128)
constexpr uint32_t kSmemQ = 0;
constexpr uint32_t kSmemKV = 2 * kTileBytes;
constexpr uint32_t kSmemBars = kSmemKV + kStages * kTileBytes;
constexpr uint32_t kCtlBytes = 2048;  // control block: barriers, flags, the column-mask classes
constexpr uint32_t kSmemTotal = kSmemBars + kCtlBytes;
constexpr uint32_t kSmemAlloc = kSmemTotal + 1024;  // slack to align the base to 1024 B

// barrier indices
enum {
    BAR_Q_FULL = 0,
    BAR_Q_EMPTY = 1,
    BAR_KV_FULL = 2,               // +slot
    BAR_KV_EMPTY = 2 + kStages,    // +slot
    BAR_S_FULL = 2 + 2 * kStages,  // +2 * tile + buffer: S(u) written (and every MMA issued before it done)
    BAR_P_READY = BAR_S_FULL + 4,  // +2 * tile + buffer: P(u) written over S(u)
    BAR_O_FREE = BAR_P_READY + 4,  // +tile: the epilogue has read O out of TMEM
    BAR_MMA_DRAINED = BAR_O_FREE + 2,
    BAR_COUNT
};

struct Ctl {
    static constexpr int32_t kStatusBase = 0;  // added to the code of an expired wait in the status word
    uint64_t bars[BAR_COUNT];
    uint32_t tmem_base;
    volatile int32_t abort;
    uint32_t colmasks[kMaxMasks * 4];  // copy of the plan's column-mask classes
};
static_assert(sizeof(Ctl) <= kCtlBytes, "control block outgrew its reservation");
static_assert(kMaxMasks * 4 <= kAttnThreads, "one thread copies one word of the column masks");

// Optional cycle trace of one CTA (compiled in only with -DVORTA_TRACE; a debugging aid).
#ifdef VORTA_TRACE
#define VORTA_TRACE_J0 16
#define VORTA_TRACE_NJ 8
#define TRACE(role, j, ev)                                                                      \
    do {                                                                                         \
        if (p.trace && blockIdx.x == 0 && it == 0 && (j) >= VORTA_TRACE_J0 &&                    \
            (j) < VORTA_TRACE_J0 + VORTA_TRACE_NJ)                                               \
            p.trace[(((role) * VORTA_TRACE_NJ) + ((j) - VORTA_TRACE_J0)) * 8 + (ev)] = clock64(); \
    } while (0)
#else
#define TRACE(role, j, ev) do { } while (0)
#endif

// ------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int32_t c0,
                                            int32_t c1, int32_t c2, int32_t c3, int32_t c4)
{
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
        : "memory");
}

// The MMA warp stays converged: every lane runs the (warp-uniform) descriptor
// arithmetic, and `leader` (1 in lane 0, 0 elsewhere) guards the instruction itself.
__device__ __forceinline__ void tc_commit(uint32_t bar, uint32_t leader)
{
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(bar), "r"(leader)
        : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate, uint32_t leader)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(leader)
        : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate, uint32_t leader)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(leader)
        : "memory");
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128.  (A and B must have the same
// 16-bit format: an fp16 P against a bf16 V is rejected by the hardware.)
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, uint32_t b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// Coordinates of block `j` of the item's KV sequence and its column-mask class.  text: the
// block is a run of bn_tile text tokens (the last kv_text blocks of a sliding item), fetched
// through the text-row tensor maps.
__device__ __forceinline__ void kv_block_coords(const AttnParams &p, const WorkItem &w, int32_t j, int32_t &c1,
                                                int32_t &c2, int32_t &c3, uint32_t &mask_id, bool &text, bool &paired)
{
    paired = false;
    text = w.mode == MODE_TILES && j >= w.kv_count - w.kv_text;
    if (text) {
        c1 = (j - (w.kv_count - w.kv_text)) * p.g.bn_tile; c2 = 0; c3 = 0; mask_id = 0;
    } else if (w.mode == MODE_TILES) {
        const KvEntry e = (item_uses_pair_list(w.flags) ? p.kv_pairs : p.kv_list)[w.kv_begin + j];
        c1 = e.w0; c2 = e.h0; c3 = e.t0; mask_id = e.mask_id & kMaskIdBits;
        paired = (e.mask_id & kEntryPaired) != 0;
    } else {
        c1 = j * kBlockM; c2 = 0; c3 = 0; mask_id = 0;
    }
}

// A KV block of n keys (a multiple of 16, at most 128) of an item worked through as `spb` sub-blocks
// per block: the widths of the two sub-blocks.  With two sub-blocks per block both get at least 16
// columns (a block of 16 keys gets a second sub-block of 16 columns that are no keys).
__host__ __device__ __forceinline__ void split_block(int32_t n, int32_t spb, int32_t &w0, int32_t &w1)
{
    if (spb == 1) { w0 = n; w1 = 0; }
    else if (n > 64) { w0 = 64; w1 = n - 64; }
    else if (n >= 32) { w0 = ((n >> 1) + 15) & ~15; w1 = n - w0; }
    else { w0 = 16; w1 = 16; }
}

// write the packed P words of a sub-block of `width` keys to the first width/2 columns at t_p
__device__ __forceinline__ void store_p(uint32_t t_p, int32_t width, uint32_t (&s)[64])
{
    if (width == 64) {
        uint32_t(&all)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
        ptx::tcgen05_st_32x32b(t_p, all);
    } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t(&chunk)[8] = *reinterpret_cast<uint32_t(*)[8]>(&s[8 * c]);
            if (c * 16 < width) ptx::tcgen05_st_32x32b(t_p + c * 8, chunk);
        }
    }
    tc_wait_st();
}

// ------------------------------------------------------------------ roles
template <int D>
__device__ __forceinline__ void producer_role(const AttnParams &p, const AttnMaps &maps, Ctl *ctl, uint32_t smem_base,
                                              int32_t begin, int32_t count, int lane)
{
    constexpr int kHalves = D / 64;
    const uint32_t bars = smem_u32(ctl->bars);
    uint32_t kv_it = 0;
    for (int32_t it = 0; it < count; ++it) {
        const WorkItem w = p.items[begin + it];
        const uint32_t rows = w.mode == MODE_TILES ? (uint32_t)p.g.box_rows : (uint32_t)kBlockM;
        const uint32_t half_bytes = rows * 128u;
        if (!mbar_wait(bars + 8 * BAR_Q_EMPTY, (it & 1) ^ 1, ctl, p.status, 101)) return;
        if (lane == 0) {
            if (w.flags & kItemPacked) {
                // two tiles of at most 64 tokens in one query block: the second one 64 rows further down
                // (lone short boxes of larger tiles come through a map whose box is 64 rows at most)
                const bool lone = (w.flags & kItemSameWindow) != 0;
                const CUtensorMap *qmap = lone ? &maps.q_lone : &maps.q[w.mode];
                mbar_expect_tx(bars + 8 * BAR_Q_FULL, (lone ? (uint32_t)p.lone_rows * 128u : half_bytes) * kHalves * 2);
                for (int t = 0; t < 2; ++t)
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(smem_base + kSmemQ + h * kHalfBytes + t * (kHalfBytes / 2), qmap,
                                    bars + 8 * BAR_Q_FULL, h * 64, w.q_org[t][0], w.q_org[t][1], w.q_org[t][2], w.slice);
            } else {
                mbar_expect_tx(bars + 8 * BAR_Q_FULL, half_bytes * kHalves * w.n_mblk);
                for (int m = 0; m < w.n_mblk; ++m)
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(smem_base + kSmemQ + m * kTileBytes + h * kHalfBytes, &maps.q[w.mode],
                                    bars + 8 * BAR_Q_FULL, h * 64, w.q_org[m][0], w.q_org[m][1], w.q_org[m][2], w.slice);
            }
        }
        for (int32_t j = 0; j < w.kv_count; ++j) {
            int32_t c1, c2, c3;
            uint32_t mask_id;
            bool text, paired;
            kv_block_coords(p, w, j, c1, c2, c3, mask_id, text, paired);
            // a box the grid cuts is fetched as its part inside the grid: a short run of real keys
            const uint32_t shape = (!text && w.mode == MODE_TILES) ? p.cls_shape[mask_id] : 0u;
            const uint32_t kv_bytes = (text ? (uint32_t)p.g.bn_tile * 128u
                                            : (shape ? (uint32_t)p.shape_rows[shape] * 128u : half_bytes)) * kHalves;
#pragma unroll
            for (int kv = 0; kv < 2; ++kv) {
                const uint32_t slot = kv_it % kStages;
                if (!mbar_wait(bars + 8 * (BAR_KV_EMPTY + slot), ((kv_it / kStages) & 1) ^ 1, ctl, p.status, 102)) return;
                if (lane == 0) {
                    const uint32_t full = bars + 8 * (BAR_KV_FULL + slot);
                    mbar_expect_tx(full, kv_bytes);
                    const CUtensorMap *map = text ? (kv == 0 ? &maps.kt : &maps.vt)
                                             : shape ? (kv == 0 ? &maps.k_cut[shape] : &maps.v_cut[shape])
                                                     : (kv == 0 ? &maps.k[w.mode] : &maps.v[w.mode]);
                    if (paired) {
                        // two 64-row boxes (the short T box of this tile and of the next one along W) fill the slot
                        const CUtensorMap *cut = kv == 0 ? &maps.k_cut[4] : &maps.v_cut[4];
                        for (int t = 0; t < 2; ++t)
                            for (int h = 0; h < kHalves; ++h)
                                tma_load_5d(smem_base + kSmemKV + slot * kTileBytes + h * kHalfBytes + t * (kHalfBytes / 2), cut,
                                            full, h * 64, c1 + t * p.g.tile[2], c2, c3, w.slice);
                    } else {
                        for (int h = 0; h < kHalves; ++h)
                            tma_load_5d(smem_base + kSmemKV + slot * kTileBytes + h * kHalfBytes, map, full, h * 64, c1,
                                        c2, c3, w.slice);
                    }
                }
                ++kv_it;
            }
        }
        __syncwarp();
    }
}

template <int D>
__device__ __forceinline__ void mma_role(const AttnParams &p, Ctl *ctl, uint32_t smem_base, uint32_t tmem,
                                         int32_t begin, int32_t count)
{
    const uint32_t bars = smem_u32(ctl->bars);
    const uint32_t leader = elect_one();
    tmem = uniform_u32(tmem);
    begin = (int32_t)uniform_u32((uint32_t)begin);
    count = (int32_t)uniform_u32((uint32_t)count);
    uint32_t kv_base = 0;  // ring position of the item's first K block (K_j at +2j, V_j at +2j+1)
    uint32_t p_par = 0, o_par = 0;  // phase parities: bit 2m+b of P_READY[m][b], bit m of O_FREE[m]

    // Descriptors of tile 0 / slot 0; the others differ by a multiple of the tile pitch
    // in the (16-byte granular) address field, so one 64-bit add moves between them.
    const uint64_t q_desc0 = smem_desc(smem_base + kSmemQ, 16, 1024);
    const uint64_t k_desc0 = smem_desc(smem_base + kSmemKV, 16, 1024);          // K-major
    const uint64_t v_desc0 = smem_desc(smem_base + kSmemKV, kHalfBytes, 1024);  // MN-major
    constexpr uint64_t kTileStep = kTileBytes >> 4;
    const uint32_t idesc_pv = instr_desc((uint32_t)D, 1);

    auto wait_kv = [&](uint32_t pos, int32_t code) {
        return mbar_wait_uniform(bars + 8 * (BAR_KV_FULL + pos % kStages), (pos / kStages) & 1, ctl, p.status, code);
    };
    auto free_kv = [&](uint32_t pos) { tc_commit(bars + 8 * (BAR_KV_EMPTY + pos % kStages), leader); };
    // S_m[buffer b] = Q_m K^T over sub-block h of the K block at ring position pos (16 channels per MMA)
    // (koff: where the sub-block starts in its K or V block, in 16-byte units: 8 per key)
    auto issue_qk = [&](int m, uint32_t pos, int b, uint32_t koff, uint32_t idesc) {
        const uint64_t qa = q_desc0 + (uint64_t)m * kTileStep;
        const uint64_t kb = k_desc0 + (uint64_t)(pos % kStages) * kTileStep + (uint64_t)koff;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t off = (uint64_t)(((kk / 4) * kHalfBytes + (kk % 4) * 32) >> 4);
            mma_ss(tmem + m * 128 + b * 64, qa + off, kb + off, idesc, kk > 0 ? 1u : 0u, leader);
        }
    };
    // O_m (+)= P_m[buffer b] V over sub-block h of the V block at pos (16 keys per MMA)
    auto issue_pv = [&](int m, uint32_t pos, int b, uint32_t koff, int ksteps, bool first) {
        const uint64_t vb = v_desc0 + (uint64_t)(pos % kStages) * kTileStep + (uint64_t)koff;
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (i < ksteps)
                mma_ts(tmem + 256 + m * 128, tmem + m * 128 + b * 64 + i * 8, vb + (uint64_t)(i * (2048 >> 4)), idesc_pv,
                       (!first || i > 0) ? 1u : 0u, leader);
    };

    for (int32_t it = 0; it < count; ++it) {
        const WorkItem *w = p.items + begin + it;
        const int32_t bn = uniform_u32((uint32_t)w->mode) == MODE_TILES ? p.g.bn_tile : kBlockM;
        const int32_t n = (int32_t)uniform_u32((uint32_t)w->kv_count);
        const int32_t nm = (int32_t)uniform_u32((uint32_t)w->n_mblk);
        const int32_t spb = bn > 64 ? 2 : 1;  // sub-blocks per KV block
        const int32_t n_sub = n * spb;
        int32_t width0, width1;
        split_block(bn, spb, width0, width1);
        // Sub-block widths of block j.  The boxes a sliding item lists after its kv_fast whole ones may be
        // short (the part of a cut box inside the grid): their key count comes from the box's class.
        const bool tiles = uniform_u32((uint32_t)w->mode) == MODE_TILES;
        const int32_t first_cut = tiles ? (int32_t)uniform_u32((uint32_t)w->kv_fast) : n;
        const int32_t n_boxes = n - (tiles ? (int32_t)uniform_u32((uint32_t)w->kv_text) : 0);
        const KvEntry *entries = (item_uses_pair_list((int32_t)uniform_u32((uint32_t)w->flags)) ? p.kv_pairs : p.kv_list) +
                                 (tiles ? (int32_t)uniform_u32((uint32_t)w->kv_begin) : 0);
        // The classes of 32 consecutive blocks are fetched with one load (lane l holds block tab_first + l)
        // and handed round by shuffle: a load per block would put a trip to global memory on this warp's
        // path every time a cut box comes up.
        int32_t tab_first = -1;
        uint32_t tab_shape = 0;
        auto block_widths = [&](int32_t j, int32_t &w0, int32_t &w1) {
            w0 = width0;
            w1 = width1;
            if (j >= first_cut && j < n_boxes) {
                if (tab_first < 0 || j < tab_first || j >= tab_first + 32) {
                    tab_first = j;
                    const int32_t mine = j + (int32_t)(threadIdx.x & 31);
                    tab_shape = mine < n_boxes ? (uint32_t)p.cls_shape[entries[mine].mask_id & kMaskIdBits] : 0u;
                }
                const uint32_t shape = uniform_u32(__shfl_sync(0xffffffffu, tab_shape, j - tab_first));
                if (shape) {
                    split_block((int32_t)uniform_u32((uint32_t)((p.shape_rows[shape] + 15) & ~15)), spb, w0, w1);
                    w0 = (int32_t)uniform_u32((uint32_t)w0);
                    w1 = (int32_t)uniform_u32((uint32_t)w1);
                }
            }
        };
        const uint32_t idesc_qk0 = instr_desc((uint32_t)width0, 0), idesc_qk1 = instr_desc((uint32_t)max(width1, 16), 0);
        int32_t kj = -1, kw0 = 0, kw1 = 0, vj = -1, vw0 = 0, vw1 = 0;  // widths of the K / V block in hand

        if (!mbar_wait_uniform(bars + 8 * BAR_Q_FULL, it & 1, ctl, p.status, 201)) return;
        // the first two score sub-blocks of both tiles
        for (int32_t u = 0; u < min(n_sub, 2); ++u) {
            const int32_t j = u / spb, h = u - j * spb;
            if (j != kj) { block_widths(j, kw0, kw1); kj = j; }
            if (h == 0 && !wait_kv(kv_base + 2 * j, 202)) return;
            tc_fence_after();
            const uint32_t idesc = instr_desc((uint32_t)(h ? kw1 : kw0), 0);
            for (int m = 0; m < nm; ++m) {
                issue_qk(m, kv_base + 2 * j, u & 1, h ? (uint32_t)kw0 * 8u : 0u, idesc);
                tc_commit(bars + 8 * (BAR_S_FULL + 2 * m + (u & 1)), leader);
            }
            if (h == spb - 1) free_kv(kv_base + 2 * j);
        }
        if (n_sub <= 2) tc_commit(bars + 8 * BAR_Q_EMPTY, leader);

        for (int32_t u = 0; u < n_sub; ++u) {
            const int32_t jv = u / spb, h = u - jv * spb, b = u & 1;
            const int32_t u2 = u + 2, jk = u2 / spb, h2 = u2 - jk * spb;
            const bool has2 = u2 < n_sub;
            const uint32_t pos_v = kv_base + 2 * jv + 1, pos_k = kv_base + 2 * jk;
            // blocks before the item's first cut box (all of them, for most items) keep the item's constants
            uint32_t idesc_k = h2 ? idesc_qk1 : idesc_qk0, koff_k = h2 ? (uint32_t)width0 * 8u : 0u;
            uint32_t koff_v = h ? (uint32_t)width0 * 8u : 0u;
            int32_t ksteps_v = (h ? width1 : width0) >> 4;
            if (max(jv, has2 ? jk : 0) >= first_cut) {
                if (jv != vj) { block_widths(jv, vw0, vw1); vj = jv; }
                if (has2 && jk != kj) { block_widths(jk, kw0, kw1); kj = jk; }
                idesc_k = instr_desc((uint32_t)(h2 ? kw1 : kw0), 0);
                koff_k = h2 ? (uint32_t)kw0 * 8u : 0u;
                koff_v = h ? (uint32_t)vw0 * 8u : 0u;
                ksteps_v = (h ? vw1 : vw0) >> 4;
            }
            if (h == 0 && !wait_kv(pos_v, 203)) return;
            if (has2 && h2 == 0 && !wait_kv(pos_k, 206)) return;
            for (int m = 0; m < nm; ++m) {
                if (!mbar_wait_uniform(bars + 8 * (BAR_P_READY + 2 * m + b), (p_par >> (2 * m + b)) & 1, ctl, p.status, 204)) return;
                p_par ^= 1u << (2 * m + b);
                if (u == 0) {
                    // the previous item's epilogue must have read O_m out of TMEM
                    if (!mbar_wait_uniform(bars + 8 * (BAR_O_FREE + m), ((o_par >> m) & 1) ^ 1, ctl, p.status, 205)) return;
                    o_par ^= 1u << m;
                }
                tc_fence_after();
                if (leader) TRACE(m, u, 0);
                issue_pv(m, pos_v, b, koff_v, ksteps_v, u == 0);
                if (has2) issue_qk(m, pos_k, b, koff_k, idesc_k);
                // S(u+2) is ready; and, for the lazy rescale and the epilogue: PV(u) is done
                tc_commit(bars + 8 * (BAR_S_FULL + 2 * m + b), leader);
                if (leader) TRACE(m, u, 1);
            }
            if (h == spb - 1) free_kv(pos_v);
            if (has2 && h2 == spb - 1) free_kv(pos_k);
            if (has2 && u2 == n_sub - 1) tc_commit(bars + 8 * BAR_Q_EMPTY, leader);
        }
        kv_base += 2 * (uint32_t)n;
    }
    // every commit issued above must have landed before the CTA's barriers go away
    tc_commit(bars + 8 * BAR_MMA_DRAINED, leader);
    mbar_wait_uniform(bars + 8 * BAR_MMA_DRAINED, 0, ctl, p.status, 207);
}

template <int D>
__device__ __forceinline__ void softmax_role(const AttnParams &p, Ctl *ctl, uint32_t tmem, int32_t begin,
                                             int32_t count, int m, int row, int warp_q)
{
    const uint32_t bars = smem_u32(ctl->bars);
    const int lane = row & 31;
    const uint32_t lane_base = (uint32_t)(warp_q * 32) << 16;
    const uint32_t t_s = tmem + lane_base + m * 128;        // scores, later P (two 64-column buffers)
    const uint32_t t_o = tmem + lane_base + 256 + m * 128;  // output accumulator
    const float scale = p.scale_log2;
    uint32_t s_par = 0;  // bit b: parity of the next phase of S_FULL[m][b] this thread will consume

    for (int32_t it = 0; it < count; ++it) {
        const WorkItem *wp = p.items + begin + it;
        if (m >= wp->n_mblk) continue;
        const int32_t w_mode = wp->mode, w_kv_len = wp->kv_len, w_kv_count = wp->kv_count;
        const bool packed = (wp->flags & kItemPacked) != 0;
        const KvEntry *kv_entries = (item_uses_pair_list(wp->flags) ? p.kv_pairs : p.kv_list) + wp->kv_begin;
        // packed item: this row belongs to the first (rows 0-63) or the second tile; a block that only the
        // other tile has in its window holds no key for it (visibility code in the entry's top bits)
        const uint32_t my_vis = packed ? 1u + (uint32_t)(row >> 6) : 0u;
        const bool has_text = w_mode == MODE_TILES && wp->kv_text > 0;
        const int32_t n_boxes = has_text ? w_kv_count - wp->kv_text : w_kv_count;  // the rest: text-token blocks
        const int32_t bn = w_mode == MODE_TILES ? p.g.bn_tile : kBlockM;
        const int32_t sh = bn > 64 ? 1 : 0;  // log2 of the sub-blocks per KV block
        const int32_t n_sub = w_kv_count << sh;
        int32_t width0, width1;
        split_block(bn, 1 << sh, width0, width1);
        // columns of a short block: every block of a sliding head whose tile has fewer than 128
        // tokens, else the last block of the sequence
        const int32_t tail_valid = w_mode == MODE_TILES ? bn : w_kv_len - (w_kv_count - 1) * kBlockM;
        const bool tail_partial = tail_valid < kBlockM;
        float row_max = -INFINITY, row_sum = 0.f;

        // wait for S(u) and read this thread's row of it (all 64 columns, or `width` of them)
        auto load_sub = [&](auto full, int32_t u, int32_t width, uint32_t(&s)[64]) -> bool {
            const int32_t b = u & 1;
            if (!mbar_wait(bars + 8 * (BAR_S_FULL + 2 * m + b), (s_par >> b) & 1, ctl, p.status, 301 + m)) return false;
            s_par ^= 1u << b;
            tc_fence_after();
            if (decltype(full)::value || width > 32) {
                ptx::tcgen05_ld_32x32b(s, t_s + b * 64);  // one 64-column load
            } else {
                uint32_t(&chunk)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
                ptx::tcgen05_ld_32x32b(chunk, t_s + b * 64);
            }
            tc_wait_ld();
            return true;
        };
        // Sub-block u of the generic path: its width in columns, how many of its leading columns are
        // keys (64 and more: all that the registers hold), and the class whose column mask applies
        // instead (0: none).  id: mask class of the sub-block's KV block (0 for whole boxes and for the
        // linear modes), fetched ahead by the caller.
        //   text-token block      the last one is cut at Lt;
        //   box the grid cuts     fetched as its part inside the grid, a short run of real keys
        //                         (classes without such a map keep the whole box and a column mask);
        //   tile under 128 tokens / last block of a sequence: a prefix of the block.
        auto sub_dims = [&](auto with_text, int32_t u, uint32_t raw_id, int32_t &width, int32_t &valid, uint32_t &mask_id) {
            const int32_t j = u >> sh, h = u & sh;
            const uint32_t id = raw_id & kMaskIdBits, vis = raw_id >> kVisShift;
            width = h ? width1 : width0;
            valid = 64;
            mask_id = 0;
            if (decltype(with_text)::value && j >= n_boxes) {
                valid = min(p.g.Lt - (j - n_boxes) * bn, bn) - 64 * h;
            } else if (id) {
                const uint32_t shape = p.cls_shape[id];
                if (shape) {
                    const int32_t rows = p.shape_rows[shape];
                    int32_t w0, w1;
                    split_block((rows + 15) & ~15, 1 << sh, w0, w1);
                    width = h ? w1 : w0;
                    valid = rows - (h ? w0 : 0);
                } else {
                    mask_id = id;
                }
            } else if (tail_partial && (w_mode == MODE_TILES || j == w_kv_count - 1)) {
                valid = tail_valid - 64 * h;
            }
            if (!mask_id) valid = min(valid, width);  // columns past the width were never loaded
            if (vis && vis != my_vis) {                // the other tile's block
                valid = 0;
                mask_id = 0;
            }
        };
        // strike the columns that are not keys
        auto apply_mask = [&](int32_t u, int32_t valid, uint32_t mask_id, uint32_t(&s)[64]) {
            uint32_t m0, m1;
            if (mask_id) {
                m0 = ctl->colmasks[mask_id * 4 + 2 * (u & sh)];
                m1 = ctl->colmasks[mask_id * 4 + 2 * (u & sh) + 1];
            } else if (valid < 64) {
                const int32_t v0 = min(max(valid, 0), 32), v1 = min(max(valid - 32, 0), 32);
                m0 = v0 == 32 ? 0xffffffffu : ((1u << v0) - 1u);
                m1 = v1 == 32 ? 0xffffffffu : ((1u << v1) - 1u);
            } else {
                return;
            }
#pragma unroll
            for (int c = 0; c < 64; ++c)
                if (!(((c < 32 ? m0 : m1) >> (c & 31)) & 1u)) s[c] = 0xff800000u;  // -inf: not a key
        };
        int32_t cur_width = 64;  // width of the sub-block whose scores s holds (generic path)
        // One sub-block: s holds the scores of u and row_max covers them.  Writes P(u), then
        // reads S(u+1) and moves row_max over it.  full: u and u+1 are both whole 64-key
        // sub-blocks of unmasked blocks, so nothing about widths or masks is looked at.
        // with_text: the item ends in blocks of text tokens (looked at only then)
        auto step = [&](auto full, auto with_text, int32_t u, uint32_t(&s)[64]) -> bool {
            constexpr bool kFull = decltype(full)::value;
            constexpr bool kText = decltype(with_text)::value;
            const int32_t b = u & 1;
            const bool has_next = kFull || u + 1 < n_sub;
            // mask class of the next sub-block's KV block, in flight under the exponentials
            const uint32_t next_id =
                (!kFull && has_next && w_mode == MODE_TILES && (!kText || ((u + 1) >> sh) < n_boxes))
                    ? kv_entries[(u + 1) >> sh].mask_id : 0u;
            if (row == 0) TRACE(2 + m, u, 0);
            // P = exp2(S * scale - max) as packed bf16 over the first half of the buffer
            float2 sum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
            if (kFull) exp_block(s, scale, -row_max, sum);
            else exp_block<false>(s, scale, -row_max, sum, cur_width);
            if (row == 0) TRACE(2 + m, u, 1);
            store_p(t_s + b * 64, kFull ? 64 : cur_width, s);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bars + 8 * (BAR_P_READY + 2 * m + b));
            if (row == 0) TRACE(2 + m, u, 2);
            row_sum += (sum[0].x + sum[0].y) + (sum[1].x + sum[1].y);
            if (has_next) {
                int32_t width = 64, valid = 64;
                uint32_t mask_id = 0;
                if (!kFull) sub_dims(with_text, u + 1, next_id, width, valid, mask_id);
                if (!load_sub(full, u + 1, width, s)) return false;
                if (row == 0) TRACE(2 + m, u, 3);
                if (!kFull) {
                    apply_mask(u + 1, valid, mask_id, s);
                    cur_width = width;
                }
                const float m_new = fmaxf(row_max, row_max64(s) * scale);
                if (__any_sync(0xffffffffu, m_new - row_max > kRescaleThreshold)) {
                    // Lazy rescale: O and the row sum move to the new maximum only when it grew by
                    // more than the threshold; until then P may reach 2^threshold.  O may be touched
                    // once PV(u) has completed: the commit that follows it is the next phase of
                    // this buffer's barrier (looked at here, consumed at sub-block u+2 or in the tail).
                    if (!mbar_wait(bars + 8 * (BAR_S_FULL + 2 * m + b), (s_par >> b) & 1, ctl, p.status, 321 + m)) return false;
                    tc_fence_after();
                    const float a = ex2(row_max - m_new);
                    row_sum *= a;
                    row_max = m_new;
                    rescale_o<D>(t_o, a);
                }
                if (row == 0) TRACE(2 + m, u, 4);
            }
            return true;
        };

        uint32_t s[64];
        {
            int32_t valid;
            uint32_t mask_id;
            sub_dims(std::true_type{}, 0, (w_mode == MODE_TILES && n_boxes > 0) ? kv_entries[0].mask_id : 0u, cur_width, valid,
                     mask_id);
            if (!load_sub(std::false_type{}, 0, cur_width, s)) return;
            apply_mask(0, valid, mask_id, s);
        }
        row_max = row_max64(s) * scale;
        // the leading unmasked blocks, then whatever is cut, short or last
        const int32_t n_full = min(2 * wp->kv_fast, n_sub) - 1;  // steps whose u and u+1 are both whole
        int32_t u = 0;
        for (; u < n_full; ++u)
            if (!step(std::true_type{}, std::false_type{}, u, s)) return;
        if (has_text) {
            for (; u < n_sub; ++u)
                if (!step(std::false_type{}, std::true_type{}, u, s)) return;
        } else {
            for (; u < n_sub; ++u)
                if (!step(std::false_type{}, std::false_type{}, u, s)) return;
        }

        // the commits that follow the last two PV MMAs: O is complete
        for (int32_t u = max(n_sub - 2, 0); u < n_sub; ++u) {
            if (!mbar_wait(bars + 8 * (BAR_S_FULL + 2 * m + (u & 1)), (s_par >> (u & 1)) & 1, ctl, p.status, 311 + m)) return;
            s_par ^= 1u << (u & 1);
        }
        tc_fence_after();
        // epilogue: O / row_sum -> bf16 -> global memory
        int32_t token = 0;
        const int qi = packed ? (row >> 6) : m;
        const int32_t q_org[3] = {wp->q_org[qi][0], wp->q_org[qi][1], wp->q_org[qi][2]};
        const bool valid = block_row_token(p.g, w_mode, q_org, w_kv_len, packed ? (row & 63) : row, &token);
        const int64_t rows = w_mode == MODE_COMPACT ? p.g.Lct : p.g.Ltot;
        __nv_bfloat16 *out = (w_mode == MODE_COMPACT ? p.Oc + (int64_t)wp->slice * rows * D : p.O + (int64_t)wp->out_slice * rows * D) +
                             (int64_t)token * D;
        const float inv = 1.f / row_sum;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            ptx::tcgen05_ld_32x32b(o, t_o + c * 32);
            tc_wait_ld();
            if (valid) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 v;
                    v.x = pack_bf16(__uint_as_float(o[8 * i + 0]) * inv, __uint_as_float(o[8 * i + 1]) * inv);
                    v.y = pack_bf16(__uint_as_float(o[8 * i + 2]) * inv, __uint_as_float(o[8 * i + 3]) * inv);
                    v.z = pack_bf16(__uint_as_float(o[8 * i + 4]) * inv, __uint_as_float(o[8 * i + 5]) * inv);
                    v.w = pack_bf16(__uint_as_float(o[8 * i + 6]) * inv, __uint_as_float(o[8 * i + 7]) * inv);
                    *reinterpret_cast<uint4 *>(out + c * 32 + i * 8) = v;
                }
            }
        }
        tc_fence_before();
        mbar_arrive(bars + 8 * (BAR_O_FREE + m));
    }
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_sm100_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ AttnMaps maps)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t smem_base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (smem_base - raw);
    Ctl *ctl = reinterpret_cast<Ctl *>(smem + kSmemBars);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // zero the operand tiles once: rows a TMA box never writes must read as 0
    for (uint32_t i = threadIdx.x; i < kSmemBars / 16; i += blockDim.x)
        reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) {
        const uint32_t bars = smem_u32(ctl->bars);
        for (int i = 0; i < BAR_COUNT; ++i) {
            // P_READY: one arrival per softmax warp; O_FREE: one per softmax thread
            mbar_init(bars + 8 * i, i >= BAR_O_FREE && i < BAR_O_FREE + 2 ? 128 : (i >= BAR_P_READY && i < BAR_O_FREE ? 4 : 1));
        }
        ctl->abort = 0;
        ctl->tmem_base = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < kMaxMasks * 4) ctl->colmasks[threadIdx.x] = p.colmasks[threadIdx.x];
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&ctl->tmem_base))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    const int32_t begin = p.cta_begin[blockIdx.x], count = p.cta_count[blockIdx.x];
    if (warp == 0) {
        producer_role<D>(p, maps, ctl, smem_base, begin, count, lane);
    } else if (warp == 1) {
        mma_role<D>(p, ctl, smem_base, tmem, begin, count);
    } else {
        const int m = (warp - 2) >> 2;
        softmax_role<D>(p, ctl, tmem, begin, count, m, (warp & 3) * 32 + lane, warp & 3);
    }

    if (ctl->abort) {
        // give copies and MMAs still in flight time to land before the CTA goes away
        for (int i = 0; i < 2000 && ctl->abort; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

}  // namespace

cudaError_t attention_sm100_prepare()
{
    cudaError_t e = cudaFuncSetAttribute(attention_sm100_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kSmemAlloc);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(attention_sm100_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)kSmemAlloc);
}

cudaError_t launch_attention_sm100(const AttnParams &p, const AttnMaps &maps, int32_t grid, cudaStream_t s)
{
    if (p.g.d == 128)
        attention_sm100_kernel<128><<<grid, kAttnThreads, kSmemAlloc, s>>>(p, maps);
    else
        attention_sm100_kernel<64><<<grid, kAttnThreads, kSmemAlloc, s>>>(p, maps);
    return cudaGetLastError();
}

}  // namespace vorta
