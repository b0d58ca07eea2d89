// CTA-pair attention kernel for sm_100a: the heads whose items are runs of consecutive rows
// (full heads, and core-set heads over their gathered rows), d = 128.
//
// Two CTAs of a cluster (an SM pair) walk the work items of the pair together.  An item
// is up to two 128-row query tiles sharing one sequence of 128-key KV blocks; CTA r of the
// pair owns tile r.  The MMAs are pair MMAs (tcgen05.mma.cta_group::2, M = 256) issued by
// the even CTA: each CTA holds its own 128 query rows (Q in shared memory, S, P and O in its
// tensor memory) and HALF of every K/V block, which the tensor cores of both SMs read:
//   S = Q K^T   B operand K [keys x d], keys split:   CTA r holds keys [64 r, 64 r + 64)
//   O += P V    B operand V [d x keys], d split:      CTA r holds channels [64 r, 64 r + 64)
// so a K/V block is fetched from L2 once per 256 query rows although a CTA works on 128.
//
// With one tile per CTA the 512 tensor-memory columns hold THREE score buffers of 128
// columns and O.  Block number n (running over all items of the pair) uses buffer n % 3;
// P (bf16) is written over the first half of the buffer.  The MMA warp keeps Q K^T two to
// three blocks ahead of the softmax (S of block j+3 is issued right after O += P V of
// block j), so neither the ~500 cycles a tcgen05.commit takes to reach a waiting thread
// nor another group's block delays a softmax thread.
//
// Warp roles (448 threads per CTA, 128 registers each):
//   warp 0        TMA producer of this CTA's Q tile and K/V halves (4-slot ring of 32 KB: the K
//                 half of block i and the V half of block i-3, which the MMA warp needs together)
//   warp 1        tensor-memory allocation; in the even CTA the MMA issuer of the pair
//   warps 2-13    softmax: three groups of four warps, one thread per query row; group k
//                 owns score buffer k, i.e. the KV blocks whose running number is k modulo
//                 3.  The groups work a third of a period apart: while one computes
//                 exponentials the others load scores and settle the reference, so the
//                 exponential unit and the issue slots stay busy.  A thread reads its row of
//                 a block 64 columns at a time and the second half twice (once for the
//                 maximum, once for the exponentials): tensor-memory loads are cheap, and 64
//                 live scores instead of 128 are what lets twelve softmax warps fit.
// All groups accumulate into the same O, so they share one reference maximum per row
// (log2 domain): the thread of block n reads the reference of block n-1 from shared
// memory, raises it only if its own row maximum exceeds it by more than 2^8 (then it
// rescales O once the PV MMAs issued so far have completed, before handing over its P),
// and publishes the reference of block n.  Each thread sums the P it produced; the three
// partial sums of a row are brought to the final reference and added in the epilogue.
//
// Barriers that collect arrivals from both CTAs (operand loads landed, P written, O read)
// live in the even CTA; the odd CTA arrives on them through the cluster's shared-memory
// window.  A commit of the pair's MMAs arrives on the barrier at the same offset in both
// CTAs.  Every load is a plain copy into the issuing CTA's own shared memory.
//
// Every wait is bounded: a wait that sees no progress for about two seconds records a
// code in the status word (1000 + the code, to tell it from the single-CTA kernel's),
// raises the CTA's abort flag and every role of the CTA leaves its loop (the peer's waits
// then run out the same way); the CTAs meet at a cluster barrier, free their tensor
// memory, meet again and return.
#include <type_traits>

#include "sm100_common.cuh"

namespace vorta {

namespace {

using namespace sm100;

constexpr int D = 128;                   // head dimension this kernel is built for
constexpr int kStages = 4;               // ring slots: the K half of one block and the V half of another
constexpr int kSBufs = 3;                // score buffers in tensor memory
constexpr uint32_t kSlabBytes = 16384;   // 128 rows x 64 bf16: one swizzled slab of Q or of a V half
constexpr uint32_t kKSlabBytes = 8192;   // 64 rows x 64 bf16: one slab of a K half
constexpr uint32_t kQBytes = 2 * kSlabBytes;
constexpr uint32_t kHalfBytes = 16384;   // a K half (two 8 KB slabs) or a V half (one slab)
constexpr uint32_t kSlotBytes = 2 * kHalfBytes;  // K half at +0, V half at +kHalfBytes
constexpr uint32_t kSmemQ = 0;
constexpr uint32_t kSmemKV = kQBytes;
constexpr uint32_t kSmemCtl = kSmemKV + kStages * kSlotBytes;
constexpr int kGroups = 3;                // softmax groups: group k owns score buffer k
constexpr int kSoftmaxWarps = 4 * kGroups;
constexpr int kPairThreads = 64 + 32 * kSoftmaxWarps;

// barrier indices ("even": only the even CTA's copy is used, both CTAs arrive on it)
enum {
    BAR_Q_FULL = 0,                          // even: both Q tiles landed
    BAR_Q_EMPTY = 1,                         // the last Q K^T of the item has read Q
    BAR_KV_FULL = 2,                         // +slot, even: both halves landed
    BAR_KV_EMPTY = BAR_KV_FULL + kStages,    // +slot: the MMAs reading the slot are done
    BAR_S_FULL = BAR_KV_EMPTY + kStages,     // +buffer: S of a block written
    BAR_PV_DONE = BAR_S_FULL + kSBufs,       // +buffer: O += P V of a block done
    BAR_P_READY = BAR_PV_DONE + kSBufs,      // +buffer, even: P of a block written over S by both CTAs
    BAR_REF = BAR_P_READY + kSBufs,          // +group: reference maxima of a block published
    BAR_STAGGER = BAR_REF + kGroups,         // +0 / +1: the group of the item's first / second block is halfway into it
    BAR_EPI = BAR_STAGGER + 2,               // partial row sums of an item published
    BAR_O_FREE = BAR_EPI + 1,                // even: both epilogues have read O out of tensor memory
    BAR_MMA_DRAINED = BAR_O_FREE + 1,
    BAR_COUNT
};

struct Ctl {
    static constexpr int32_t kStatusBase = 1000;  // this kernel's wait codes in the status word: 1xxx
    uint64_t bars[BAR_COUNT];
    uint32_t tmem_base;
    volatile int32_t abort;
    float ref[4][kBlockM];             // reference maximum of block n at [n % 4][row]
    float part_sum[kGroups][kBlockM];  // [group][row]: partial row sums at the final reference
};
constexpr uint32_t kSmemTotal = kSmemCtl + ((sizeof(Ctl) + 127) / 128) * 128;
constexpr uint32_t kSmemAlloc = kSmemTotal + 1024;  // slack to align the base to 1024 B
static_assert(kSmemAlloc <= 232448, "shared memory budget of an sm_100 CTA");
// A group's consecutive blocks use the same score buffer, so it asks for a buffer's scores one phase
// after the other.  (A group hopping between buffers could ask for a buffer's next scores before its
// previous ones were produced, and a parity wait two phases ahead passes at once.)
static_assert(kSBufs == kGroups, "the parity waits on BAR_S_FULL rely on one score buffer per softmax group");

// Optional cycle trace of CTA pair 0 (compiled in only with -DVORTA_TRACE; a debugging aid):
// role 0 the MMA warp, 1 / 2 the first warp of softmax group 0 / 1 in the even CTA, 3 group 0 in the odd CTA.
#ifdef VORTA_TRACE
#define VORTA_TRACE_J0 40
#define VORTA_TRACE_NJ 8
#define TRACE(role, g, ev)                                                                          \
    do {                                                                                             \
        if (p.trace && (blockIdx.x >> 1) == 0 && (g) >= VORTA_TRACE_J0 && (g) < VORTA_TRACE_J0 + VORTA_TRACE_NJ) \
            p.trace[(((role) * VORTA_TRACE_NJ) + ((g) - VORTA_TRACE_J0)) * 8 + (ev)] = clock64();   \
    } while (0)
#else
#define TRACE(role, g, ev) do { } while (0)
#endif

// ------------------------------------------------------------------ PTX helpers
// address, in the cluster's shared-memory window, of this CTA's `addr` in CTA `rank`
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.relaxed.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr),
                 "r"(bytes)
                 : "memory");
}

// (Barriers that also take arrivals from the peer CTA are waited on like the others: the data behind
// those arrivals is in tensor memory or was written by TMA.)

// Tiled bulk load into this CTA's shared memory whose bytes are counted on a barrier of
// the even CTA (`bar` is an address in the cluster window); the data go to this CTA only.
__device__ __forceinline__ void tma_load_5d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar, int32_t c0,
                                                 int32_t c1, int32_t c2, int32_t c3, int32_t c4)
{
    asm volatile(
        "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// The MMA warp stays converged: every lane runs the (warp-uniform) descriptor arithmetic,
// and `leader` (1 in one lane, 0 elsewhere) guards the instruction itself.
// Commit of the pair's MMAs issued so far: one arrival on the barrier at this offset in both CTAs.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, uint32_t leader)
{
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %2;\n\t}"
        ::"r"(bar), "r"(leader), "h"((uint16_t)3)
        : "memory");
}

// D[tmem] (+)= A[smem] * B[smem], M = 256 over the pair
__device__ __forceinline__ void mma_pair_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate, uint32_t leader)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(leader)
        : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem], M = 256 over the pair
__device__ __forceinline__ void mma_pair_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate, uint32_t leader)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(leader)
        : "memory");
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = 256 (128 rows in each CTA), N = n over the pair.
__device__ __forceinline__ uint32_t instr_desc_pair(uint32_t n, uint32_t b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major << 16) | ((n >> 3) << 17) | ((256u >> 4) << 24);
}

// write the 32 packed P words of 64 keys held in s[0 .. 32) to t_p (the caller waits for the stores)
__device__ __forceinline__ void store_p(uint32_t t_p, uint32_t (&s)[64])
{
    uint32_t(&all)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
    ptx::tcgen05_st_32x32b(t_p, all);
}

// The K/V load sequence of an item with n KV blocks, in the order the MMA warp consumes it: step i
// carries K_i (if i < n) and V_{i-3} (if 3 <= i < n + 3), so that what block j needs after its own K,
// namely V_j, and what follows it in the tensor pipe, K_{j+3}, arrive together in one ring slot behind
// one barrier.  Steps that carry nothing (i in [n, 3) of an item shorter than three blocks) are skipped
// by both sides.
__device__ __forceinline__ bool step_has_k(int32_t i, int32_t n) { return i < n; }
__device__ __forceinline__ bool step_has_v(int32_t i, int32_t n) { return i >= kSBufs && i < n + kSBufs; }

// ------------------------------------------------------------------ roles
// Loads of CTA `rank`: its Q tile, and of every KV block its half of K (keys) and of V (channels).
__device__ __forceinline__ void producer_role(const AttnParams &p, const AttnMaps &maps, Ctl *ctl, uint32_t smem_base,
                                              int32_t begin, int32_t count, int lane, uint32_t rank)
{
    const uint32_t bars = smem_u32(ctl->bars);
    const uint32_t even_bars = map_to_rank(bars, 0);
    uint32_t kv_it = 0;
    for (int32_t it = 0; it < count; ++it) {
        const WorkItem w = p.items[begin + it];
        if (!mbar_wait(bars + 8 * BAR_Q_EMPTY, (it & 1) ^ 1, ctl, p.status, 101)) return;
        if (lane == 0) {
            if ((int32_t)rank < w.n_mblk) {
                mbar_expect_tx_cluster(even_bars + 8 * BAR_Q_FULL, kQBytes);
                for (int h = 0; h < 2; ++h)
                    tma_load_5d_pair(smem_base + kSmemQ + h * kSlabBytes, &maps.q[w.mode], even_bars + 8 * BAR_Q_FULL,
                                     h * 64, w.q_org[rank][0], 0, 0, w.slice);
            } else {
                mbar_arrive_cluster(even_bars + 8 * BAR_Q_FULL);  // no second tile: nothing to load
            }
        }
        for (int32_t i = 0; i < w.kv_count + kSBufs; ++i) {
            const bool has_k = step_has_k(i, w.kv_count), has_v = step_has_v(i, w.kv_count);
            if (!has_k && !has_v) continue;
            const uint32_t slot = kv_it % kStages;
            if (!mbar_wait(bars + 8 * (BAR_KV_EMPTY + slot), ((kv_it / kStages) & 1) ^ 1, ctl, p.status, 102)) return;
            if (lane == 0) {
                const uint32_t full = even_bars + 8 * (BAR_KV_FULL + slot);
                const uint32_t dst = smem_base + kSmemKV + slot * kSlotBytes;
                // rows past the end of the sequence arrive as zeros and count like the others
                mbar_expect_tx_cluster(full, (has_k ? kHalfBytes : 0u) + (has_v ? kHalfBytes : 0u));
                if (has_k) {
                    // keys [64 rank, 64 rank + 64) of block i, all channels
                    for (int h = 0; h < 2; ++h)
                        tma_load_5d_pair(dst + h * kKSlabBytes, &maps.k_half[w.mode], full, h * 64,
                                         i * kBlockM + (int32_t)rank * (kBlockM / 2), 0, 0, w.slice);
                }
                if (has_v) {
                    // the 128 keys of block i - 3, channels [64 rank, 64 rank + 64)
                    tma_load_5d_pair(dst + kHalfBytes, &maps.v[w.mode], full, (int32_t)rank * 64, (i - kSBufs) * kBlockM,
                                     0, 0, w.slice);
                }
            }
            ++kv_it;
        }
        __syncwarp();
    }
}

// Even CTA only: the pair's MMAs.
__device__ __forceinline__ void mma_role(const AttnParams &p, Ctl *ctl, uint32_t smem_base, uint32_t tmem,
                                         int32_t begin, int32_t count)
{
    const uint32_t bars = smem_u32(ctl->bars);
    const uint32_t leader = elect_one();
    tmem = uniform_u32(tmem);
    begin = (int32_t)uniform_u32((uint32_t)begin);
    count = (int32_t)uniform_u32((uint32_t)count);
    uint32_t kv_it = 0;  // steps of the K/V load sequence consumed so far
    uint32_t g0 = 0;     // KV blocks of the items before this one

    // Descriptors of slot 0; the others differ by a multiple of the slot pitch in the
    // (16-byte granular) address field, so one 64-bit add moves between them.
    const uint64_t q_desc = smem_desc(smem_base + kSmemQ, 16, 1024);
    const uint64_t k_desc0 = smem_desc(smem_base + kSmemKV, 16, 1024);          // K-major, 64-row slabs
    const uint64_t v_desc0 = smem_desc(smem_base + kSmemKV + kHalfBytes, kSlabBytes, 1024);  // MN-major, one 64-channel slab
    constexpr uint64_t kSlotStep = kSlotBytes >> 4;
    const uint32_t idesc_pv = instr_desc_pair((uint32_t)D, 1), idesc_qk = instr_desc_pair((uint32_t)kBlockM, 0);
    const uint32_t t_o = tmem + kSBufs * 128;

    // next step of the load sequence: wait for both CTAs' halves of it, return the ring slot
    auto next_kv = [&](uint32_t &slot, int32_t code) {
        slot = kv_it % kStages;
        const bool ok = mbar_wait_uniform(bars + 8 * (BAR_KV_FULL + slot), (kv_it / kStages) & 1, ctl, p.status, code);
        ++kv_it;
        return ok;
    };
    auto free_kv = [&](uint32_t slot) { tc_commit_pair(bars + 8 * (BAR_KV_EMPTY + slot), leader); };
    // S[buf] = Q K^T over the K half-blocks in `slot` (16 channels per MMA)
    auto issue_qk = [&](uint32_t buf, uint32_t slot) {
        const uint64_t kb = k_desc0 + (uint64_t)slot * kSlotStep;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t qoff = (uint64_t)(((kk / 4) * kSlabBytes + (kk % 4) * 32) >> 4);
            const uint64_t koff = (uint64_t)(((kk / 4) * kKSlabBytes + (kk % 4) * 32) >> 4);
            mma_pair_ss(tmem + buf * 128, q_desc + qoff, kb + koff, idesc_qk, kk > 0 ? 1u : 0u, leader);
        }
    };
    // O (+)= P[buf] V over the V half-blocks in `slot`; P is packed bf16 in the first 64 columns of
    // S[buf] (16 keys per MMA)
    auto issue_pv = [&](uint32_t buf, uint32_t slot, bool first) {
        const uint64_t vb = v_desc0 + (uint64_t)slot * kSlotStep;
#pragma unroll
        for (int kk = 0; kk < kBlockM / 16; ++kk)
            mma_pair_ts(t_o, tmem + buf * 128 + kk * 8, vb + (uint64_t)(kk * (2048 >> 4)), idesc_pv,
                        (!first || kk > 0) ? 1u : 0u, leader);
    };

    for (int32_t it = 0; it < count; ++it) {
        const WorkItem *w = p.items + begin + it;
        const int32_t n = (int32_t)uniform_u32((uint32_t)w->kv_count);

        if (!mbar_wait_uniform(bars + 8 * BAR_Q_FULL, it & 1, ctl, p.status, 201)) return;
        // scores of the first blocks, one per buffer (steps 0 .. 2 carry K only)
        for (int32_t j = 0; j < min(n, kSBufs); ++j) {
            uint32_t slot;
            if (!next_kv(slot, 202)) return;
            tc_fence_after();
            const uint32_t buf = (g0 + j) % kSBufs;
            issue_qk(buf, slot);
            tc_commit_pair(bars + 8 * (BAR_S_FULL + buf), leader);
            free_kv(slot);
        }
        if (n <= kSBufs) tc_commit_pair(bars + 8 * BAR_Q_EMPTY, leader);

        for (int32_t j = 0; j < n; ++j) {
            const uint32_t g = g0 + (uint32_t)j, buf = g % kSBufs, par = (g / kSBufs) & 1;
            // step j + 3: V_j and, if the item has it, K_{j+3}
            uint32_t slot;
            if (!next_kv(slot, 203)) return;
            if (leader) TRACE(0, g, 0);
            if (!mbar_wait_uniform(bars + 8 * (BAR_P_READY + buf), par, ctl, p.status, 204)) return;
            if (j == 0) {
                // the previous item's epilogues must have read O out of tensor memory
                if (!mbar_wait_uniform(bars + 8 * BAR_O_FREE, (it & 1) ^ 1, ctl, p.status, 205)) return;
            }
            tc_fence_after();
            if (leader) TRACE(0, g, 1);
            issue_pv(buf, slot, j == 0);
            tc_commit_pair(bars + 8 * (BAR_PV_DONE + buf), leader);
            if (leader) TRACE(0, g, 3);
            if (j + kSBufs < n) {
                // the buffer P(j) leaves takes the scores of block j+3
                issue_qk(buf, slot);
                tc_commit_pair(bars + 8 * (BAR_S_FULL + buf), leader);
                if (j + kSBufs == n - 1) tc_commit_pair(bars + 8 * BAR_Q_EMPTY, leader);
            }
            free_kv(slot);
            if (leader) TRACE(0, g, 5);
        }
        g0 += (uint32_t)n;
    }
}

// What a softmax thread carries from block to block of an item.
struct RowState {
    float known;   // reference the partial sum is relative to (-inf before the first block)
    float sum;     // this thread's partial row sum
};

// Arrival on a barrier of the even CTA: local there, through the cluster window from the odd CTA.
// The data the arrival announces sits in tensor memory (written, waited for, fenced), so the remote
// form carries no memory ordering of its own.
__device__ __forceinline__ void arrive_even(uint32_t bars, uint32_t even_bars, uint32_t rank, int bar)
{
    if (rank == 0)
        mbar_arrive(bars + 8 * bar);
    else
        mbar_arrive_cluster(even_bars + 8 * bar);
}

// One KV block of one softmax thread (query row `row`, TMEM quadrant row / 32) whose group owns the
// block: running number g in the pair, number jb in the item.  kFull: all 128 columns are real keys,
// so nothing about widths or masks is looked at.  The two variants are separate functions so that the
// mask logic of the cut, short and last blocks costs the common one no registers.
template <bool kFull>
__device__ __forceinline__ bool softmax_block(const AttnParams &p, Ctl *ctl, const WorkItem *wp, uint32_t t_row, uint32_t g,
                                              int32_t jb, int grp, int row, uint32_t rank, RowState &st)
{
    const uint32_t bars = smem_u32(ctl->bars);
    const uint32_t even_bars = map_to_rank(bars, 0);
    const int lane = row & 31;
    const uint32_t buf = g % kSBufs, par = (g / kSBufs) & 1;
    const uint32_t t_s = t_row + buf * 128;
    const uint32_t t_o = t_row + kSBufs * 128;
    const float scale = p.scale_log2;
    const int trole = rank == 0 ? (grp < 2 ? 1 + grp : -1) : (grp == 0 ? 3 : -1);
    const bool tr = row == 0 && trole >= 0;
    if (tr) TRACE(trole, g, 0);
    if (!mbar_wait(bars + 8 * (BAR_S_FULL + buf), par, ctl, p.status, 301 + grp)) return false;
    tc_fence_after();
    if (tr) TRACE(trole, g, 1);
    // which columns are keys: all but in the last block of a sequence whose length is no multiple of 128
    uint32_t m[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};
    if (!kFull && jb == wp->kv_count - 1) {
        const int32_t valid = wp->kv_len - jb * kBlockM;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int32_t v = min(max(valid - 32 * i, 0), 32);
            m[i] = v == 32 ? 0xffffffffu : ((1u << v) - 1u);
        }
    }
    // this thread's row of S, 64 columns at a time: half h is keys [64 h, 64 h + 64)
    uint32_t s[64];
    auto load_half = [&](int h) {
        ptx::tcgen05_ld_32x32b(s, t_s + h * 64);  // one 64-column load (two 32-column ones: 1.2 % slower)
        tc_wait_ld();
        if (!kFull && (m[2 * h] & m[2 * h + 1]) != 0xffffffffu) {
#pragma unroll
            for (int c = 0; c < 64; ++c)
                if (!((m[2 * h + (c >> 5)] >> (c & 31)) & 1u)) s[c] = 0xff800000u;  // -inf: not a key
        }
    };
    // The row maximum needs all 128 scores before the first exponential; holding them all would
    // leave the thread no registers, so the second half is read twice (tensor-memory loads are
    // cheap): maximum of half 1, then half 0, which stays in registers for its exponentials.
    load_half(1);
    const float mx = row_max64(s);
    load_half(0);
    if (tr) TRACE(trole, g, 2);
    const float mine = fmaxf(mx, row_max64(s)) * scale;
    // the reference: that of the previous block unless this block's maximum is far above it
    float prev = -INFINITY;
    if (jb > 0) {
        if (!mbar_wait(bars + 8 * (BAR_REF + (g - 1) % kGroups), ((g - 1) / kGroups) & 1, ctl, p.status, 351 + grp)) return false;
        prev = ctl->ref[(g - 1) & 3][row];
    }
    if (tr) TRACE(trole, g, 3);
    const bool raise = jb > 0 && mine > prev + kRescaleThreshold;
    const float cur = (jb == 0 || raise) ? mine : prev;
    ctl->ref[g & 3][row] = cur;
    __syncwarp();
    if (lane == 0) mbar_arrive(bars + 8 * (BAR_REF + g % kGroups));
    if (__any_sync(0xffffffffu, raise)) {
        // O moves to the new reference.  It may be touched once PV of block jb-1 has completed
        // (PV of this block cannot be issued before this thread's P arrives).
        const uint32_t gb = g - 1;
        if (!mbar_wait(bars + 8 * (BAR_PV_DONE + gb % kSBufs), (gb / kSBufs) & 1, ctl, p.status, 321 + grp)) return false;
        tc_fence_after();
        rescale_o<D>(t_o, raise ? ex2(prev - cur) : 1.f);
        tc_wait_st();
    }
    float my_sum = st.sum;
    if (st.known != cur) {
        my_sum *= ex2(st.known - cur);  // known = -inf only while the sum is 0
        st.known = cur;
    }
    // P = exp2(S * scale - reference) as packed bf16 over the first half of the buffer
    float2 sum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
    exp_block(s, scale, -cur, sum);
    store_p(t_s, s);
    if (jb < 2) {
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + 8 * (BAR_STAGGER + jb));  // halfway: the next block's group may start
    }
    if (tr) TRACE(trole, g, 4);
    // P of keys [0, 64) went to columns [0, 32): the scores of the other keys are still in place
    load_half(1);
    exp_block(s, scale, -cur, sum);
    store_p(t_s + 32, s);
    tc_wait_st();  // both halves of P are in tensor memory
    tc_fence_before();
    __syncwarp();
    if (lane == 0) arrive_even(bars, even_bars, rank, BAR_P_READY + buf);
    if (tr) TRACE(trole, g, 5);
    st.sum = my_sum + ((sum[0].x + sum[0].y) + (sum[1].x + sum[1].y));
    return true;
}

__device__ __noinline__ bool softmax_block_generic(const AttnParams &p, Ctl *ctl, const WorkItem *wp, uint32_t t_row,
                                                   uint32_t g, int32_t jb, int grp, int row, uint32_t rank, RowState &st)
{
    return softmax_block<false>(p, ctl, wp, t_row, g, jb, grp, row, rank, st);
}

__device__ __noinline__ bool softmax_block_full(const AttnParams &p, Ctl *ctl, const WorkItem *wp, uint32_t t_row,
                                                    uint32_t g, int32_t jb, int grp, int row, uint32_t rank, RowState &st)
{
    return softmax_block<true>(p, ctl, wp, t_row, g, jb, grp, row, rank, st);
}

// The thread of query row `row` in group `grp` (blocks whose running number is grp modulo 3).
// A CTA without a tile in an item only keeps the barrier phases of the pair moving.
__device__ __forceinline__ void softmax_role(const AttnParams &p, Ctl *ctl, uint32_t tmem, int32_t begin, int32_t count,
                                             int grp, int quad, int lane, uint32_t rank)
{
    const uint32_t bars = smem_u32(ctl->bars);
    const uint32_t even_bars = map_to_rank(bars, 0);
    const int row = quad * 32 + lane;
    const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16);
    const uint32_t t_o = t_row + kSBufs * 128;
    uint32_t g0 = 0;  // KV blocks of the items before this one

    for (int32_t it = 0; it < count; ++it) {
        const WorkItem *wp = p.items + begin + it;
        const int32_t w_mode = wp->mode, w_kv_len = wp->kv_len, n = wp->kv_count;
        const uint32_t gl = g0 + (uint32_t)n - 1;  // the item's last block
        // this group's blocks of the item: those whose running number is grp modulo 3
        int32_t j = (int32_t)(((uint32_t)grp + kGroups - g0 % kGroups) % kGroups);
        const bool dry = (int32_t)rank >= wp->n_mblk;  // no tile of this CTA in the item

        // The groups work a third of a block period apart, so that one computes exponentials while
        // another loads scores and settles the reference, and the scores of a group's next block are
        // complete when it asks for them.  Started together they stay together (each then waits for
        // scores that depend on the others' hand-overs), so the group of the item's second (third)
        // block holds back until the group of the first (second) is halfway through its exponentials.
        if (j > 0 && !mbar_wait(bars + 8 * (BAR_STAGGER + j - 1), it & 1, ctl, p.status, 331)) return;
        if (j < 2 && (dry || j >= n)) {
            __syncwarp();
            if (lane == 0) mbar_arrive(bars + 8 * (BAR_STAGGER + j));
        }

        if (dry) {
            // follow the score buffers and hand over nothing
            for (; j < n; j += kGroups) {
                const uint32_t g = g0 + (uint32_t)j, buf = g % kSBufs, par = (g / kSBufs) & 1;
                if (!mbar_wait(bars + 8 * (BAR_S_FULL + buf), par, ctl, p.status, 391 + grp)) return;
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bars + 8 * (BAR_REF + g % kGroups));  // keeps the phase of this barrier in step with g
                    arrive_even(bars, even_bars, rank, BAR_P_READY + buf);
                }
            }
            if (!mbar_wait(bars + 8 * (BAR_PV_DONE + gl % kSBufs), (gl / kSBufs) & 1, ctl, p.status, 393 + grp)) return;
            __syncwarp();
            if (lane == 0) mbar_arrive(bars + 8 * BAR_EPI);  // one phase per item here too
            if (!mbar_wait(bars + 8 * BAR_EPI, it & 1, ctl, p.status, 395 + grp)) return;
            if (lane == 0) arrive_even(bars, even_bars, rank, BAR_O_FREE);
            g0 += (uint32_t)n;
            continue;
        }

        // this group's blocks: the leading unmasked ones, then whatever is cut, short or last
        RowState st = {-INFINITY, 0.f};
        const int32_t n_full = min(wp->kv_fast, n);
        for (; j < n_full; j += kGroups)
            if (!softmax_block_full(p, ctl, wp, t_row, g0 + (uint32_t)j, j, grp, row, rank, st)) return;
        for (; j < n; j += kGroups)
            if (!softmax_block_generic(p, ctl, wp, t_row, g0 + (uint32_t)j, j, grp, row, rank, st)) return;

        // epilogue: all PV MMAs done; partial sums at the final reference; O / sum -> bf16 -> global memory
        if (!mbar_wait(bars + 8 * (BAR_PV_DONE + gl % kSBufs), (gl / kSBufs) & 1, ctl, p.status, 311 + grp)) return;
        if (!mbar_wait(bars + 8 * (BAR_REF + gl % kGroups), (gl / kGroups) & 1, ctl, p.status, 371 + grp)) return;
        tc_fence_after();
        const float fin = ctl->ref[gl & 3][row];
        ctl->part_sum[grp][row] = st.known == -INFINITY ? 0.f : st.sum * ex2(st.known - fin);
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + 8 * BAR_EPI);
        if (!mbar_wait(bars + 8 * BAR_EPI, it & 1, ctl, p.status, 381 + grp)) return;
        const float total = ctl->part_sum[0][row] + ctl->part_sum[1][row] + ctl->part_sum[2][row];
        int32_t token = 0;
        const int32_t q_org[3] = {wp->q_org[rank][0], wp->q_org[rank][1], wp->q_org[rank][2]};
        const bool valid = block_row_token(p.g, w_mode, q_org, w_kv_len, row, &token);
        const int64_t rows = w_mode == MODE_COMPACT ? p.g.Lct : p.g.Ltot;
        // the threads of a row in groups 0 and 1 write half of the channels each
        constexpr int kShare = D / 2;
        __nv_bfloat16 *out = (w_mode == MODE_COMPACT ? p.Oc + (int64_t)wp->slice * rows * D : p.O + (int64_t)wp->out_slice * rows * D) +
                             (int64_t)token * D + grp * kShare;
        const float inv = 1.f / total;
#pragma unroll
        for (int c = 0; c < kShare / 32; ++c) {
            if (grp >= 2) break;
            uint32_t o[32];
            ptx::tcgen05_ld_32x32b(o, t_o + grp * kShare + c * 32);
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
        __syncwarp();
        if (lane == 0) arrive_even(bars, even_bars, rank, BAR_O_FREE);
        g0 += (uint32_t)n;
    }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
attention_sm100_pair_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ AttnMaps maps)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t smem_base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (smem_base - raw);
    Ctl *ctl = reinterpret_cast<Ctl *>(smem + kSmemCtl);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = blockIdx.x & 1u;  // rank in the cluster (clusters are consecutive CTA pairs)

    // zero the operand tiles once: rows a TMA box never writes must read as 0
    for (uint32_t i = threadIdx.x; i < kSmemCtl / 16; i += blockDim.x)
        reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) {
        const uint32_t bars = smem_u32(ctl->bars);
        for (int i = 0; i < BAR_COUNT; ++i) {
            uint32_t n = 1;  // one commit of the pair's MMAs
            if (i == BAR_Q_FULL || (i >= BAR_KV_FULL && i < BAR_KV_FULL + kStages)) n = 2;  // one producer per CTA
            if (i >= BAR_P_READY && i < BAR_P_READY + kSBufs) n = 8;  // four warps of a group in each CTA
            if (i >= BAR_REF && i < BAR_EPI) n = 4;               // four warps of a group
            if (i == BAR_EPI) n = kSoftmaxWarps;
            if (i == BAR_O_FREE) n = 2 * kSoftmaxWarps;
            mbar_init(bars + 8 * i, n);
        }
        ctl->abort = 0;
        ctl->tmem_base = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&ctl->tmem_base))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync_all();  // both CTAs' barriers are initialised before either arrives on the other's
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    const int32_t pair = (int32_t)(blockIdx.x >> 1);
    const int32_t begin = p.cta_begin[pair], count = p.cta_count[pair];
    if (warp == 0) {
        producer_role(p, maps, ctl, smem_base, begin, count, lane, rank);
    } else if (warp == 1) {
        const uint32_t bars = smem_u32(ctl->bars);
        if (rank == 0) {
            mma_role(p, ctl, smem_base, tmem, begin, count);
            // every MMA and commit issued above must have landed before either CTA goes away
            tc_commit_pair(bars + 8 * BAR_MMA_DRAINED, elect_one());
        }
        mbar_wait_uniform(bars + 8 * BAR_MMA_DRAINED, 0, ctl, p.status, 207);
    } else {
        softmax_role(p, ctl, tmem, begin, count, (warp - 2) >> 2, warp & 3, lane, rank);
    }

    if (ctl->abort) {
        // give copies and MMAs still in flight time to land before the CTAs go away
        for (int i = 0; i < 2000 && ctl->abort; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncwarp();
    cluster_sync_all();  // the peer may still arrive on this CTA's barriers or read its operands
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
    // Neither CTA leaves before both have released the pair's tensor memory: a CTA of another
    // kernel may start on an SM the moment its CTA exits, and must not meet a release still to come.
    __syncwarp();
    cluster_sync_all();
}

}  // namespace

cudaError_t attention_sm100_pair_prepare()
{
    return cudaFuncSetAttribute(attention_sm100_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)kSmemAlloc);
}

// grid: CTAs (two per pair).  The work lists of `p` are indexed by pair.
cudaError_t launch_attention_sm100_pair(const AttnParams &p, const AttnMaps &maps, int32_t grid, cudaStream_t s)
{
    attention_sm100_pair_kernel<<<grid, kPairThreads, kSmemAlloc, s>>>(p, maps);
    return cudaGetLastError();
}

}  // namespace vorta
