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
// Warp roles (384 threads):
//   warp 0        TMA producer: Q once per item, then K_j, V_j into a 4-slot ring
//   warp 1        MMA issuer: S = Q K^T and O += P V as tcgen05.mma, accumulators in TMEM
//   warp 2        TMEM allocation
//   warps 4-7     softmax of tile 0 (one thread per query row = one TMEM lane)
//   warps 8-11    softmax of tile 1
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P (bf16) is
// written over the first half of its S.  Softmax is the usual online form in the
// log2 domain with a lazy accumulator rescale (only when the row maximum grew by
// more than 2^8), done by the softmax threads themselves between two PV MMAs.
//
// Every wait is bounded: a wait that sees no progress for about two seconds
// records a code in the status word, raises the CTA's abort flag and every role
// leaves its loop; the CTA then gives outstanding copies time to land, frees its
// TMEM and returns.
#include <cuda/ptx>

#include "vorta_internal.h"

namespace vorta {

namespace {

namespace ptx = cuda::ptx;

constexpr int kStages = 4;                // KV ring slots (K and V blocks alternate)
constexpr uint32_t kHalfBytes = 16384;    // 128 rows x 64 bf16: one swizzled half tile
constexpr uint32_t kTileBytes = 32768;    // two halves (d = 128)
constexpr uint32_t kSmemQ = 0;
constexpr uint32_t kSmemKV = 2 * kTileBytes;
constexpr uint32_t kSmemBars = kSmemKV + kStages * kTileBytes;
constexpr uint32_t kSmemTotal = kSmemBars + 512;
constexpr uint32_t kSmemAlloc = kSmemTotal + 1024;  // slack to align the base to 1024 B
constexpr float kRescaleThreshold = 8.0f;           // log2 units
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

// barrier indices
enum {
    BAR_Q_FULL = 0,
    BAR_Q_EMPTY = 1,
    BAR_KV_FULL = 2,               // +slot
    BAR_KV_EMPTY = 2 + kStages,    // +slot
    BAR_S_FULL = 2 + 2 * kStages,  // +tile
    BAR_P_FULL = BAR_S_FULL + 2,
    BAR_PV_DONE = BAR_P_FULL + 2,
    BAR_O_FREE = BAR_PV_DONE + 2,
    BAR_MMA_DRAINED = BAR_O_FREE + 2,
    BAR_COUNT
};

struct Ctl {
    uint64_t bars[BAR_COUNT];
    uint32_t tmem_base;
    volatile int32_t abort;
};
static_assert(sizeof(Ctl) <= 512, "control block outgrew its reservation");

// ------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(bar),
                 "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait on a phase of an mbarrier.  Returns false if the CTA is aborting.
__device__ __forceinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, Ctl *ctl, int32_t *status, int32_t code)
{
    const unsigned long long t0 = global_ns();
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 0) {
            if (ctl->abort) return false;
            if (global_ns() - t0 > kWaitLimitNs) {
                ctl->abort = code;
                atomicCAS(status, 0, code);
                return false;
            }
        }
    }
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, Ctl *ctl, int32_t *status, int32_t code)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, ctl, status, code);
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int32_t c0,
                                            int32_t c1, int32_t c2, int32_t c3, int32_t c4)
{
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1.
// lbo/sbo in bytes: for a K-major operand sbo is the pitch of 8-row groups; for an
// MN-major operand lbo is the pitch of 64-element column blocks and sbo the pitch
// of 8-row (K) groups.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;  // version
    d |= (uint64_t)2 << 61;  // SWIZZLE_128B
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128.
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, uint32_t b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

template <int REGS>
__device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS)); }
template <int REGS>
__device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS)); }

// Coordinates of block `j` of the item's KV sequence and its column mask.
struct KvBlock {
    int32_t c1, c2, c3;
    uint32_t mask[4];
    bool whole;  // all 128 columns valid
};

__device__ __forceinline__ void kv_block_coords(const AttnParams &p, const WorkItem &w, int32_t j, int32_t &c1,
                                                int32_t &c2, int32_t &c3, uint32_t &mask_id)
{
    if (w.mode == MODE_TILES) {
        const KvEntry e = p.kv_list[w.kv_begin + j];
        c1 = e.w0; c2 = e.h0; c3 = e.t0; mask_id = e.mask_id;
    } else {
        c1 = j * kBlockM; c2 = 0; c3 = 0; mask_id = 0;
    }
}

// 64 score columns of this thread's row (only the chunks below `cols` are read)
__device__ __forceinline__ void load_scores(uint32_t (&s)[64], uint32_t taddr, int32_t cols)
{
    uint32_t(&lo)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
    uint32_t(&hi)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[32]);
    ptx::tcgen05_ld_32x32b(lo, taddr);
    if (cols > 32) ptx::tcgen05_ld_32x32b(hi, taddr + 32);
    tc_wait_ld();
}

// columns whose mask bit is 0 are not keys: their score becomes -inf
__device__ __forceinline__ void mask_scores(uint32_t (&s)[64], uint32_t m0, uint32_t m1)
{
#pragma unroll
    for (int c = 0; c < 32; ++c) {
        if (!((m0 >> c) & 1u)) s[c] = 0xff800000u;
        if (!((m1 >> c) & 1u)) s[32 + c] = 0xff800000u;
    }
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
            mbar_expect_tx(bars + 8 * BAR_Q_FULL, half_bytes * kHalves * w.n_mblk);
            for (int m = 0; m < w.n_mblk; ++m)
                for (int h = 0; h < kHalves; ++h)
                    tma_load_5d(smem_base + kSmemQ + m * kTileBytes + h * kHalfBytes, &maps.q[w.mode],
                                bars + 8 * BAR_Q_FULL, h * 64, w.q_org[m][0], w.q_org[m][1], w.q_org[m][2], w.slice);
        }
        for (int32_t j = 0; j < w.kv_count; ++j) {
            int32_t c1, c2, c3;
            uint32_t mask_id;
            kv_block_coords(p, w, j, c1, c2, c3, mask_id);
#pragma unroll
            for (int kv = 0; kv < 2; ++kv) {
                const uint32_t slot = kv_it % kStages;
                if (!mbar_wait(bars + 8 * (BAR_KV_EMPTY + slot), ((kv_it / kStages) & 1) ^ 1, ctl, p.status, 102)) return;
                if (lane == 0) {
                    const uint32_t full = bars + 8 * (BAR_KV_FULL + slot);
                    mbar_expect_tx(full, half_bytes * kHalves);
                    const CUtensorMap *map = kv == 0 ? &maps.k[w.mode] : &maps.v[w.mode];
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(smem_base + kSmemKV + slot * kTileBytes + h * kHalfBytes, map, full, h * 64, c1,
                                    c2, c3, w.slice);
                }
                ++kv_it;
            }
        }
        __syncwarp();
    }
}

template <int D>
__device__ __forceinline__ void mma_role(const AttnParams &p, Ctl *ctl, uint32_t smem_base, uint32_t tmem,
                                         int32_t begin, int32_t count, int lane)
{
    const uint32_t bars = smem_u32(ctl->bars);
    uint32_t kv_it = 0;
    uint32_t p_cnt[2] = {0, 0}, o_uses[2] = {0, 0};

    // S_m = Q_m K^T over the K block in `slot`
    auto issue_qk = [&](int m, uint32_t slot, uint32_t idesc) {
        const uint32_t qa = smem_base + kSmemQ + m * kTileBytes;
        const uint32_t kb = smem_base + kSmemKV + slot * kTileBytes;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = (kk / 4) * kHalfBytes + (kk % 4) * 32;
            mma_ss(tmem + m * 128, smem_desc(qa + off, 16, 1024), smem_desc(kb + off, 16, 1024), idesc, kk > 0);
        }
    };
    // O_m (+)= P_m V over the V block in `slot`; P is packed bf16 in S_m's columns
    auto issue_pv = [&](int m, uint32_t slot, uint32_t idesc, int32_t bn, bool first) {
        const uint32_t vb = smem_base + kSmemKV + slot * kTileBytes;
        for (int kk = 0; kk < bn / 16; ++kk)
            mma_ts(tmem + 256 + m * 128, tmem + m * 128 + kk * 8, smem_desc(vb + kk * 2048, kHalfBytes, 1024), idesc,
                   (!first || kk > 0) ? 1u : 0u);
    };

    for (int32_t it = 0; it < count; ++it) {
        const WorkItem w = p.items[begin + it];
        const int32_t bn = w.mode == MODE_TILES ? p.g.bn_tile : kBlockM;
        const int32_t n = w.kv_count, nm = w.n_mblk;
        const uint32_t idesc_qk = instr_desc((uint32_t)bn, 0), idesc_pv = instr_desc((uint32_t)D, 1);

        if (!mbar_wait(bars + 8 * BAR_Q_FULL, it & 1, ctl, p.status, 201)) return;
        // block 0: both score tiles
        uint32_t slot_k = kv_it % kStages;
        if (!mbar_wait(bars + 8 * (BAR_KV_FULL + slot_k), (kv_it / kStages) & 1, ctl, p.status, 202)) return;
        ++kv_it;
        tc_fence_after();
        if (lane == 0) {
            for (int m = 0; m < nm; ++m) {
                issue_qk(m, slot_k, idesc_qk);
                tc_commit(bars + 8 * (BAR_S_FULL + m));
            }
            tc_commit(bars + 8 * (BAR_KV_EMPTY + slot_k));
            if (n == 1) tc_commit(bars + 8 * BAR_Q_EMPTY);
        }
        __syncwarp();
        for (int32_t j = 0; j < n; ++j) {
            const uint32_t slot_v = kv_it % kStages;
            if (!mbar_wait(bars + 8 * (BAR_KV_FULL + slot_v), (kv_it / kStages) & 1, ctl, p.status, 203)) return;
            ++kv_it;
            const bool has_next = j + 1 < n;
            slot_k = kv_it % kStages;
            for (int m = 0; m < nm; ++m) {
                if (!mbar_wait(bars + 8 * (BAR_P_FULL + m), p_cnt[m] & 1, ctl, p.status, 204)) return;
                ++p_cnt[m];
                if (j == 0) {
                    // the previous item's epilogue must have read O_m out of TMEM
                    if (!mbar_wait(bars + 8 * (BAR_O_FREE + m), (o_uses[m] & 1) ^ 1, ctl, p.status, 205)) return;
                    ++o_uses[m];
                }
                if (has_next && m == 0) {
                    if (!mbar_wait(bars + 8 * (BAR_KV_FULL + slot_k), (kv_it / kStages) & 1, ctl, p.status, 206)) return;
                }
                tc_fence_after();
                if (lane == 0) {
                    issue_pv(m, slot_v, idesc_pv, bn, j == 0);
                    if (!has_next) tc_commit(bars + 8 * (BAR_PV_DONE + m));
                    if (has_next) {
                        issue_qk(m, slot_k, idesc_qk);
                        tc_commit(bars + 8 * (BAR_S_FULL + m));
                    }
                }
                __syncwarp();
            }
            if (lane == 0) {
                tc_commit(bars + 8 * (BAR_KV_EMPTY + slot_v));
                if (has_next) {
                    tc_commit(bars + 8 * (BAR_KV_EMPTY + slot_k));
                    if (j + 2 == n) tc_commit(bars + 8 * BAR_Q_EMPTY);
                }
            }
            if (has_next) ++kv_it;
            __syncwarp();
        }
    }
    // every commit issued above must have landed before the CTA's barriers go away
    if (lane == 0) tc_commit(bars + 8 * BAR_MMA_DRAINED);
    __syncwarp();
    mbar_wait(bars + 8 * BAR_MMA_DRAINED, 0, ctl, p.status, 207);
}

template <int D>
__device__ __forceinline__ void softmax_role(const AttnParams &p, Ctl *ctl, uint32_t tmem, int32_t begin,
                                             int32_t count, int m, int row, int warp_q)
{
    const uint32_t bars = smem_u32(ctl->bars);
    const uint32_t lane_base = (uint32_t)(warp_q * 32) << 16;
    const uint32_t t_s = tmem + lane_base + m * 128;        // scores, later P
    const uint32_t t_o = tmem + lane_base + 256 + m * 128;  // output accumulator
    const float scale = p.scale_log2;
    uint32_t s_cnt = 0, part = 0;

    for (int32_t it = 0; it < count; ++it) {
        const WorkItem w = p.items[begin + it];
        if (m >= w.n_mblk) continue;
        const int32_t bn = w.mode == MODE_TILES ? p.g.bn_tile : kBlockM;
        float row_max = -INFINITY, row_sum = 0.f;

        for (int32_t j = 0; j < w.kv_count; ++j) {
            // which columns of this block are real keys
            uint32_t mask[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};
            bool whole = true;
            if (w.mode == MODE_TILES) {
                const uint32_t mask_id = p.kv_list[w.kv_begin + j].mask_id;
                if (mask_id) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) mask[i] = __ldg(p.colmasks + mask_id * 4 + i);
                    whole = false;
                } else if (bn < kBlockM) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        int32_t v = min(max(bn - 32 * i, 0), 32);
                        mask[i] = v == 32 ? 0xffffffffu : ((1u << v) - 1u);
                    }
                    whole = false;
                }
            } else {
                const int32_t valid = w.kv_len - j * kBlockM;
                if (valid < kBlockM) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        int32_t v = min(max(valid - 32 * i, 0), 32);
                        mask[i] = v == 32 ? 0xffffffffu : ((1u << v) - 1u);
                    }
                    whole = false;
                }
            }

            if (!mbar_wait(bars + 8 * (BAR_S_FULL + m), s_cnt & 1, ctl, p.status, 301 + m)) return;
            ++s_cnt;
            tc_fence_after();

            // pass 1: the row maximum, 64 columns at a time
            float mx = -INFINITY;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (h * 64 >= bn) break;
                uint32_t s[64];
                load_scores(s, t_s + h * 64, bn - h * 64);
                if (!whole) mask_scores(s, mask[2 * h], mask[2 * h + 1]);
#pragma unroll
                for (int c = 0; c < 64; ++c) mx = fmaxf(mx, __uint_as_float(s[c]));
            }
            const float m_new = fmaxf(row_max, mx * scale);
            if (j == 0) {
                row_max = m_new;
            } else if (__any_sync(0xffffffffu, m_new - row_max > kRescaleThreshold)) {
                // the previous PV of this tile has completed (it was issued before the QK
                // whose completion we just waited for), so O may be rescaled in place
                const float a = ex2(row_max - m_new);
                row_sum *= a;
                row_max = m_new;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    ptx::tcgen05_ld_32x32b(o, t_o + c * 32);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * a);
                    ptx::tcgen05_st_32x32b(t_o + c * 32, o);
                }
            }
            // pass 2: P = exp2(S * scale - max) as packed bf16 over the first bn/2 columns of S.
            // Half h reads columns [64h, 64h + 64) and writes [32h, 32h + 32): never ahead of a read.
            const float neg_max = -row_max;
            float sum = 0.f;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (h * 64 >= bn) break;
                uint32_t s[64];
                load_scores(s, t_s + h * 64, bn - h * 64);
                if (!whole) mask_scores(s, mask[2 * h], mask[2 * h + 1]);
#pragma unroll
                for (int c = 0; c < 64; c += 2) {
                    const float p0 = ex2(fmaf(__uint_as_float(s[c]), scale, neg_max));
                    const float p1 = ex2(fmaf(__uint_as_float(s[c + 1]), scale, neg_max));
                    // the row sum takes the rounded values the PV MMA will really use, so
                    // that O / sum stays a true weighted mean of V rows
                    const uint32_t pk = pack_bf16(p0, p1);
                    sum += __uint_as_float(pk << 16) + __uint_as_float(pk & 0xffff0000u);
                    s[c >> 1] = pk;
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t(&chunk)[8] = *reinterpret_cast<uint32_t(*)[8]>(&s[8 * c]);
                    if (h * 64 + c * 16 < bn) ptx::tcgen05_st_32x32b(t_s + h * 32 + c * 8, chunk);
                }
            }
            row_sum += sum;
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bars + 8 * (BAR_P_FULL + m));
        }

        // epilogue: O / row_sum -> bf16 -> global memory
        if (!mbar_wait(bars + 8 * (BAR_PV_DONE + m), part & 1, ctl, p.status, 311 + m)) return;
        ++part;
        tc_fence_after();
        int32_t token = 0;
        const bool valid = block_row_token(p.g, w.mode, w.q_org[m], w.kv_len, row, &token);
        const int64_t rows = w.mode == MODE_COMPACT ? p.g.Lc : p.g.L;
        __nv_bfloat16 *out = (w.mode == MODE_COMPACT ? p.Oc : p.O) + ((int64_t)w.slice * rows + token) * D;
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
            const bool many = (i >= BAR_P_FULL && i < BAR_P_FULL + 2) || (i >= BAR_O_FREE && i < BAR_O_FREE + 2);
            mbar_init(bars + 8 * i, many ? 128 : 1);
        }
        ctl->abort = 0;
        ctl->tmem_base = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&ctl->tmem_base))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    const int32_t begin = p.cta_begin[blockIdx.x], count = p.cta_count[blockIdx.x];
    if (warp < 4) {
        reg_dec<64>();
        if (warp == 0) producer_role<D>(p, maps, ctl, smem_base, begin, count, lane);
        else if (warp == 1) mma_role<D>(p, ctl, smem_base, tmem, begin, count, lane);
    } else {
        reg_inc<216>();
        const int m = (warp - 4) >> 2;
        softmax_role<D>(p, ctl, tmem, begin, count, m, (warp & 3) * 32 + lane, warp & 3);
    }

    if (ctl->abort) {
        // give copies and MMAs still in flight time to land before the CTA goes away
        for (int i = 0; i < 2000 && ctl->abort; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
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
