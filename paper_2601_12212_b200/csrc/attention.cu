// Tree-masked verification attention (Section 3.2, "Verification Phase": all tree
// tokens are scored by the target in one pass; Appendix D: the attention mask
// follows the tree).
//
// Split-KV flash-decode on the 5th-generation tensor cores.  The query rows of one
// KV head (tree token x the Hq/Hkv heads sharing it) are packed into 128-row tiles,
// so that Q K^T and P V are dense contractions: tcgen05.mma with the fp32
// accumulators (S and O) in tensor memory.  K/V tiles of 64 keys are staged by TMA
// (cp.async.bulk.tensor, one elected thread) into 128-byte-swizzled shared memory
// through mbarrier rings (four stages each for K and V), Q tiles likewise (prefetched for the next item).
//
// A CTA runs two symmetric lanes.  A lane is an MMA-issuing warp, a softmax warpgroup
// (one TMEM lane = one query row per thread) and a quarter of tensor memory (two S/P
// buffers and one O accumulator).  The softmax warpgroup scales, applies the ancestor
// bitmask (from registers, only on tiles that reach past the prefix), keeps the online
// softmax state and writes P back into the tensor-memory columns S came from, from
// where it is the A operand of P V.  P is kept as two bf16 terms (p = hi + lo): one
// bf16 rounding of the weights alone would cost up to 2^-9 per weight, about 1 % of an
// output row's rms in the worst element.
//
// A work item is (sequence, KV head, group of row tiles, range of key tiles).  With more
// than 128 rows in the group, lane x takes row tile x over all key tiles ("row mode");
// otherwise both lanes take the one row tile and alternate key tiles ("key mode") and
// merge their two results inside the CTA (a lane reads the other's accumulator straight
// from tensor memory).  The work list depends only on the step parameters, which are the
// same for every layer of a step: a one-CTA kernel derives it once from the
// device-resident parameters and leaves it in the workspace as a table (one 32-byte
// descriptor per item), so nothing about a launch depends on (TT, d, k, L) and a CTA
// learns its work from one load.  Items whose group has a single split write O directly;
// all others write normalised partials that a second, small kernel combines.
//
// Every wait (mbarrier) is bounded: when it runs out the CTA raises
// RESPS_STATUS_WAIT_TIMEOUT, stops issuing work, drains its copies in flight, frees
// its tensor memory and returns.  Every barrier is used so that a waiter can never
// fall two phases behind (a parity wait would then never return).
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cmath>
#include <mutex>
#include <new>
#include <unordered_map>

#include "common.cuh"

namespace resps {
namespace {

constexpr int kBM = 128;           // rows per row tile (one TMEM lane each)
constexpr int kBN = 64;            // keys per tile
// Ring depths.  Both must be even: in key mode the lanes take alternate tiles and a lane waits for
// (and looks ahead at) the "full" barriers of its own tiles only, so the previous use of a stage
// must have been its own too -- with an odd depth it would be the other lane's, which this lane has
// not seen complete, and a parity wait cannot tell "not yet" from "one phase on".
constexpr int kStagesK = 4;
constexpr int kStagesV = 4;
static_assert(kStagesK % 2 == 0 && kStagesV % 2 == 0, "ring depths must be even (key mode)");
constexpr int kRowTiles = 2;       // row tiles per item
constexpr int kSoftmaxThreads = 256;
constexpr int kProducerWarp = 8;   // K and Q tiles
constexpr int kMmaWarp0 = 9;       // lane x is issued by warp kMmaWarp0 + x
constexpr int kVProducerWarp = 11; // V tiles
constexpr int kAttnThreads = 384;
constexpr int kRegsSoftmax = 216;  // setmaxnreg: 256 x 216 + 128 x 72 = 384 x 168 <= 64 K registers
constexpr int kRegsIssue = 72;
constexpr int kSyncThreads = 320;  // softmax warps + the MMA warps meet at the end of an item
constexpr int kMaxBatchSmem = 256;
constexpr int kTmemCols = 512;
constexpr int kCombineThreads = 256;
constexpr int kMaxRounds = 4;      // rounds of items the work list may plan for (long sequences only)
constexpr uint32_t kWaitLimitCycles = kWaitTest ? 2000000u : 0x70000000u;  // bounded waits give up after ~1 s of SM clocks
constexpr float kRescaleSlack = 8.0f;  // O is rescaled only when the running max grows by > 2^8
constexpr unsigned kFull = 0xFFFFFFFFu;

// What the work list keeps per sequence (the combine kernels walk rows, not items) ...
struct PlanSeq {
    int n, L, mp, nfull, kt, s_row, s_key, item0;
};
// ... and per item: everything a CTA needs to start.
struct PlanItem {
    int b_g;          // sequence | KV head << 16
    int pair_splits;  // group index within the head | splits of the group << 16
    int sp, first_item, t_begin, t_end;
    int n, L;         // the sequence's tree size and prefix length
};
static_assert(sizeof(PlanSeq) == 32 && sizeof(PlanItem) == 32, "two 16-byte loads each");

struct AttnArgs {
    const resps_step* steps;
    const int32_t* n_nodes;
    int batch;
    const __nv_bfloat16* q;
    __nv_bfloat16* o;
    float* lse;
    int64_t capacity;
    const uint64_t* mask;
    float scale_log2;
    int Hq, Hkv, max_tt;
    // Partials of split groups.  O is stored normalised (O / l, a convex combination of V rows) as
    // fp16 times a per-row power of two that only differs from 1 when a value would leave the fp16
    // range: half the bytes of fp32, and 11 significant bits per element (2^-11, against the 2^-9
    // of the final bf16 rounding).
    uint4* part_o;    // [items][2 row tiles][D/8][128 rows]  eight fp16 each
    float4* part_ml;  // [items][2 row tiles][128 rows]   (running max m, running sum l, l * row scale, -)
    int max_items;
    int sched_grid;   // CTAs of the attention grid (the work list is balanced for it)
    int min_tiles;    // smallest key-tile count worth a split of its own
    int single_units; // single row tiles while no sequence has more than this many (row tiles)^2 x key tiles
    int rounds;       // 0: the work list chooses its number of rounds; 1..kMaxRounds: as told (tests)
    int stagger;      // cycles lane 1 starts behind lane 0 in row mode
    int q_by_tma;     // 1: Q tiles come by TMA (128 % (Hq/Hkv) == 0), 0: by plain loads
    int plan_after_wait;  // 1: the work list was written by the kernel just before this one
    int test_drop;        // test build only: 1 = the CTA's first V copy is left out
    int32_t* status;
    // The work list, written by attention_plan_kernel.
    int4* plan_head;             // (items, rows per group, -, -)
    PlanSeq* plan_seq;       // [batch + 1]; entry [batch].item0 = items
    PlanItem* plan_item;  // [max_items]
};

// ---------------------------------------------------------------------------- work list
// A group is (sequence, KV head, pair of row tiles).  A pair with more than 128 rows runs in row
// mode and costs two units per key tile; the last pair of a head may have at most 128 rows, runs
// in key mode and costs one.  Every group is cut into splits of at most T units, with the smallest
// T for which the items fit one round of the grid (found by a short search; steps of 1/16), so
// that the CTAs finish together whatever the mix of tree sizes and prefix lengths.
// Groups are single row tiles instead, all in key mode, while no sequence has many row tiles per KV
// head over a long prefix: items of half the size fill the grid where row-mode items (at least two key
// tiles for each of two row tiles) cannot, and the two halves of a CTA merge into one partial; the
// price is that K and V pass through L2 once per row tile instead of once per pair.  Measured
// crossovers (per-call time, both groupings forced): 2 row tiles per KV head (8B shape, 60 nodes) --
// single tiles ahead up to a prefix of 24 000, level at 32 000; 6 row tiles (70B shape, 96 nodes) --
// ahead up to 3 000, 1.5 % behind from 4 000; ragged batch of 8 with up to 3 row tiles and prefixes up
// to 8 000 -- ahead by 3 %.  All of them sit near (row tiles)^2 x key tiles = 2000 for the largest
// sequence, which is the rule (`single_units`).  On the 8B-shaped workload with the prefix growing from
// 1024 to 3010 this gives 480 us per step, against 510 already at 1837 with the first rule (at most two
// units of work per CTA).
struct Sched {
    int group_rows;             // rows of a group: 256 (pairs of row tiles) or 128 (single tiles)
    int n[kMaxBatchSmem];       // tree nodes (0 = sequence skipped)
    int L[kMaxBatchSmem];
    int mp[kMaxBatchSmem];      // row-tile pairs
    int nfull[kMaxBatchSmem];   // pairs in row mode (mp or mp - 1)
    int kt[kMaxBatchSmem];      // key tiles
    int s_row[kMaxBatchSmem];   // splits of a row-mode group
    int s_key[kMaxBatchSmem];   // splits of the key-mode group
    int item0[kMaxBatchSmem + 1];
};

__device__ __forceinline__ int ceil_div(int a, int b) {  // a >= 0, b > 0: the unsigned division is the shorter one
    return static_cast<int>((static_cast<unsigned>(a) + static_cast<unsigned>(b) - 1u) / static_cast<unsigned>(b));
}

// Runs in the first warp (one lane per sequence, eight rounds for the largest batch); the block
// meets once at the end.  This sits at the head of the kernel's critical path (nothing can be
// fetched before the CTA knows its item), hence the care for the length of the dependent chain.
__device__ __forceinline__ void build_sched(const AttnArgs& a, Sched& sc, int tid) {
    if (tid < 32) {
        const int G = a.Hq / a.Hkv;
        const int nblk = (a.batch + 31) >> 5;
        const int mt = max(a.min_tiles, 1);
        // ---- pass 1: sizes, and the cost in row-tile x key-tile units (the same for both groupings:
        // a row-mode pair costs two units per key tile, a single tile one) ----------------------------
        unsigned cost = 0;   // saturates: it only seeds the search below
        unsigned cost2 = 0;  // largest (row tiles)^2 x key tiles of a sequence: decides the grouping
#pragma unroll 1
        for (int i = 0; i < nblk; ++i) {
            const int b = i * 32 + tid;
            if (b < a.batch) {
                int n = min(max(a.n_nodes[b], 0), a.max_tt);
                const int L = max(a.steps[b].prefix_len, 0);
                if (static_cast<int64_t>(L) + n > a.capacity) {
                    atomicOr(a.status, RESPS_STATUS_KV_OVERFLOW);
                    n = 0;
                }
                const int tiles = (n * G + kBM - 1) / kBM;
                const int kt = (n > 0) ? (L + n + kBN - 1) / kBN : 0;
                sc.n[b] = n, sc.L[b] = L, sc.kt[b] = kt;
                cost += min(static_cast<unsigned>(a.Hkv * tiles) * static_cast<unsigned>(kt), 1u << 23);
                cost2 = max(cost2, min(static_cast<unsigned>(tiles * tiles) * static_cast<unsigned>(kt), 1u << 26));
            }
        }
        cost = __reduce_add_sync(0xFFFFFFFFu, min(cost, 1u << 26));
        cost2 = __reduce_max_sync(0xFFFFFFFFu, cost2);
        // a small call is cut into single row tiles (see above)
        const bool single = cost2 <= static_cast<unsigned>(a.single_units);
        const int group_rows = single ? kBM : kRowTiles * kBM;
        if (tid == 0) sc.group_rows = group_rows;
#pragma unroll 1
        for (int i = 0; i < nblk; ++i) {
            const int b = i * 32 + tid;
            if (b < a.batch) {
                const int M = sc.n[b] * G;
                const int mp = (M + group_rows - 1) / group_rows;
                sc.mp[b] = mp;
                sc.nfull[b] = single ? 0 : ((mp > 0 && M - (mp - 1) * group_rows <= kBM) ? mp - 1 : mp);
            }
        }
        // the lane's first sequence stays in registers (its only one up to 32 sequences)
        int kt0 = 0, nfull0 = 0, nkey0 = 0;
        if (tid < a.batch) kt0 = sc.kt[tid], nfull0 = sc.nfull[tid], nkey0 = sc.mp[tid] - nfull0;
        // Smallest T (in steps of T/16) for which the items fit `rounds` rounds of the grid.  One round
        // is the rule.  With long sequences and few groups it can leave CTAs idle (40 groups of 3 splits
        // are 120 items for 148 CTAs); two to four rounds of shorter items then fill the grid better.
        // An item more costs a CTA about kItemUnits units (its epilogue and the start of the next), so
        // more rounds are only looked at when items are long, where the time of this search does not
        // matter either.
        constexpr int kItemUnits = 8;
        const int forced = min(a.rounds, kMaxRounds);
        int T = 1, best = 0x7FFFFFFF;
#pragma unroll 1
        for (int rounds = max(forced, 1); rounds <= (forced > 0 ? forced : kMaxRounds); ++rounds) {
            int Tr = max(ceil_div(static_cast<int>(cost), rounds * a.sched_grid), 1);
#pragma unroll 1
            for (int tries = 0; tries < 24; ++tries) {
                const int t_row = max((Tr + 1) >> 1, mt), t_key = max(Tr, mt);
                unsigned cnt = a.Hkv * (nfull0 * ceil_div(kt0, t_row) + nkey0 * ceil_div(kt0, t_key));
#pragma unroll 1
                for (int i = 1; i < nblk; ++i) {
                    const int b = i * 32 + tid;
                    if (b < a.batch)
                        cnt += a.Hkv * (sc.nfull[b] * ceil_div(sc.kt[b], t_row) +
                                        (sc.mp[b] - sc.nfull[b]) * ceil_div(sc.kt[b], t_key));
                }
                cnt = __reduce_add_sync(0xFFFFFFFFu, min(cnt, 1u << 20));
                if (cnt <= static_cast<unsigned>(rounds * a.sched_grid)) break;
                Tr += max(1, Tr >> 4);
            }
            if (rounds * (Tr + kItemUnits) < best) best = rounds * (Tr + kItemUnits), T = Tr;
            if (forced == 0 && Tr < 8 * kItemUnits) break;  // short items: no further rounds
        }
        const int s_row0 = ceil_div(kt0, max((T + 1) >> 1, mt)), s_key0 = ceil_div(kt0, max(T, mt));
        const int t_row = max((T + 1) >> 1, mt), t_key = max(T, mt);
        int base = 0;
#pragma unroll 1
        for (int i = 0; i < nblk; ++i) {
            const int b = i * 32 + tid;
            int mine = 0, s_row = s_row0, s_key = s_key0;
            if (i > 0 && b < a.batch) s_row = ceil_div(sc.kt[b], t_row), s_key = ceil_div(sc.kt[b], t_key);
            if (b < a.batch) mine = a.Hkv * (sc.nfull[b] * s_row + (sc.mp[b] - sc.nfull[b]) * s_key);
            int incl = mine;  // inclusive prefix sum over the lanes
            if (a.batch > 1) {
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const int v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                    if (tid >= d) incl += v;
                }
            }
            if (b < a.batch) sc.s_row[b] = s_row, sc.s_key[b] = s_key, sc.item0[b] = base + incl - mine;
            base += __shfl_sync(0xFFFFFFFFu, incl, a.batch > 1 ? 31 : 0);
        }
        if (tid == 0) sc.item0[a.batch] = base;
    }
    __syncthreads();
}

struct Item {
    int b, g, pair, sp, splits, first_item;
    int n, L, M, row_base, nmt, t_begin, t_end;
    int tok0;  // first token of the group's rows
};

__device__ __forceinline__ PlanItem plan_entry(const Sched& sc, int item) {
    PlanItem p;
    int b = 0;
    while (item >= sc.item0[b + 1]) ++b;
    const int nfull = sc.nfull[b], s_row = sc.s_row[b], s_key = sc.s_key[b];
    const int row_items = nfull * s_row;
    const int per_head = row_items + (sc.mp[b] - nfull) * s_key;
    const int local = item - sc.item0[b];
    const int g = static_cast<int>(static_cast<unsigned>(local) / static_cast<unsigned>(per_head));
    const int rem = local - g * per_head;
    int pair, splits;
    if (rem < row_items) {
        pair = static_cast<int>(static_cast<unsigned>(rem) / static_cast<unsigned>(s_row));
        p.sp = rem - pair * s_row;
        splits = s_row;
    } else {
        pair = nfull + static_cast<int>(static_cast<unsigned>(rem - row_items) / static_cast<unsigned>(s_key));
        p.sp = rem - row_items - (pair - nfull) * s_key;
        splits = s_key;
    }
    p.b_g = static_cast<int>(static_cast<unsigned>(b) | (static_cast<unsigned>(g) << 16));
    p.pair_splits = static_cast<int>(static_cast<unsigned>(pair) | (static_cast<unsigned>(splits) << 16));
    p.first_item = item - p.sp;
    // kt <= 2^15 (cache capacity is checked on the host), so the products fit 32 bits
    const unsigned kt = static_cast<unsigned>(sc.kt[b]), sp = static_cast<unsigned>(p.sp);
    p.t_begin = static_cast<int>(kt * sp / static_cast<unsigned>(splits));
    p.t_end = static_cast<int>(kt * (sp + 1u) / static_cast<unsigned>(splits));
    p.n = sc.n[b], p.L = sc.L[b];
    return p;
}

// The work list of one call: the per-sequence figures and one descriptor per item, written to the
// workspace.  One CTA; it runs once per step (the list is the same for every layer).
__global__ void __launch_bounds__(256) attention_plan_kernel(const AttnArgs a) {
    __shared__ Sched sc;
    pdl_wait();  // the step parameters and node counts are complete
    pdl_launch_dependents();
    build_sched(a, sc, threadIdx.x);  // ends with __syncthreads()
    const int total = min(sc.item0[a.batch], a.max_items);
    if (threadIdx.x == 0) *a.plan_head = make_int4(total, sc.group_rows, 0, 0);
    for (int b = threadIdx.x; b <= a.batch; b += blockDim.x) {
        PlanSeq q = {};
        q.item0 = sc.item0[b];
        if (b < a.batch)
            q.n = sc.n[b], q.L = sc.L[b], q.mp = sc.mp[b], q.nfull = sc.nfull[b], q.kt = sc.kt[b],
            q.s_row = sc.s_row[b], q.s_key = sc.s_key[b];
        a.plan_seq[b] = q;
    }
    for (int item = threadIdx.x; item < total; item += blockDim.x) a.plan_item[item] = plan_entry(sc, item);
}

// A CTA's view of one entry of the work list.
__device__ __forceinline__ Item load_item(const AttnArgs& a, int item, int group_rows, int G) {
    const int4* src = reinterpret_cast<const int4*>(a.plan_item + item);
    const int4 lo = __ldcg(src), hi = __ldcg(src + 1);
    Item it;
    it.b = lo.x & 0xFFFF, it.g = static_cast<int>(static_cast<unsigned>(lo.x) >> 16);
    it.pair = lo.y & 0xFFFF, it.splits = static_cast<int>(static_cast<unsigned>(lo.y) >> 16);
    it.sp = lo.z, it.first_item = lo.w;
    it.t_begin = hi.x, it.t_end = hi.y, it.n = hi.z, it.L = hi.w;
    it.M = it.n * G;
    it.row_base = it.pair * group_rows;
    it.nmt = (group_rows > kBM && it.M - it.row_base > kBM) ? 2 : 1;
    it.tok0 = (it.row_base == 0) ? 0 : it.row_base / G;
    return it;
}

// ---------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
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
// Bounded wait: false when this wait ran out (about a second of SM clocks) or another thread of
// the CTA has given up.  Kept to a few instructions, because it is inlined at every wait and the
// kernel's code has to stay small (see the note on code size at the kernel); the caller records
// the failure in its `alive` flag, and the status word is written once, at the end of the kernel.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try(bar, parity)) return true;  // the common case does not even read the clock
    const uint32_t t0 = static_cast<uint32_t>(clock());
    uint32_t spins = 0;
    while (!mbar_try(bar, parity)) {
        // the 32-bit cycle counter wraps after two seconds; it is read far more often than that
        if ((++spins & 255u) == 0u && (*abort_flag || static_cast<uint32_t>(clock()) - t0 > kWaitLimitCycles))
            return false;
    }
    return true;
}
// For the tear-down: a copy this thread issued must have landed before the CTA gives up its shared
// memory, whatever else went wrong, so this wait looks at nothing but its own barrier and clock.
__device__ __forceinline__ bool drain_wait(uint32_t bar, uint32_t parity) {
    const uint32_t t0 = static_cast<uint32_t>(clock());
    uint32_t spins = 0;
    while (!mbar_try(bar, parity))
        if ((++spins & 255u) == 0u && static_cast<uint32_t>(clock()) - t0 > kWaitLimitCycles) return false;
    return true;
}
// Same, with a warp-uniform answer (the callers go on to warp-collective TMEM instructions).
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    const bool ok = mbar_wait(bar, parity, abort_flag);
    return __all_sync(0xFFFFFFFFu, ok);
}
// One lane of a converged warp.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "elect.sync _|P, 0xFFFFFFFF;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// TMA: one box of a 5-D view into shared memory.  The last dimension of every view is the
// 64-element column panel, so that one copy brings all panels of a tile, each in its own
// 128-byte-swizzled block (the innermost coordinate is always 0).
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2, int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4, %5, %6}], [%7];" ::"r"(dst),
        "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
        : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(lbo_bytes >> 4) << 16;
    d |= static_cast<uint64_t>(sbo_bytes >> 4) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, A K-major.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) |
           (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(kBM >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                     uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// A operand from tensor memory (lane = row, two bf16 per 32-bit column).
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}

#define RESPS_R8(a, o) "%" #a "0" #o
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
          "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
          "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
          "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
#undef RESPS_R8
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]),
        "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]),
        "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Packed fp32 pairs (one instruction for two lanes of arithmetic) and the 3-input maximum.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ unsigned long long sub2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("sub.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// ---------------------------------------------------------------------------- shared memory map
template <int D>
struct Smem {
    static constexpr int kPanels = D / 64;                   // 64-element (128-byte) column panels
    static constexpr int kQPanel = kBM * 128;                // one panel of a Q row tile
    static constexpr int kQTile = kPanels * kQPanel;
    static constexpr int kKVPanel = kBN * 128;
    static constexpr int kKVTile = kPanels * kKVPanel;
    static constexpr int kOffQ = 0;
    static constexpr int kOffK = kOffQ + kRowTiles * kQTile;
    static constexpr int kOffV = kOffK + kStagesK * kKVTile;
    static constexpr int kOffBar = kOffV + kStagesV * kKVTile;
    static constexpr int kNumBars = 2 * (kStagesK + kStagesV) + 1 + kRowTiles * 5 + 3;
    static constexpr int kOffMisc = kOffBar + 8 * 32;
    static constexpr int kOffMerge = kOffMisc + 64;          // (max, sum) of every row of both lanes
    static constexpr int kUsed = kOffMerge + kRowTiles * kBM * 8 + 1024;  // + slack to align the base to 1024
    // Never less than 120 KB, more than half of an SM's shared memory: one CTA per SM, so the
    // 512-column TMEM allocation can never wait for a neighbour.
    static constexpr int kBytes = kUsed > 120 * 1024 ? kUsed : 120 * 1024;
    static_assert(kNumBars <= 32, "barrier area");
    static_assert(2 * kBytes > 228 * 1024, "two CTAs must not fit on one SM");
};

// barrier indices
__device__ __forceinline__ constexpr int bar_kfull(int s) { return s; }
__device__ __forceinline__ constexpr int bar_vfull(int s) { return kStagesK + s; }
// K and V stages are released separately: a K tile is dead once its Q K^T has completed, long
// before the P V of the same tile, and the next K can be on its way meanwhile.
__device__ __forceinline__ constexpr int bar_kempty(int s) { return kStagesK + kStagesV + s; }
__device__ __forceinline__ constexpr int bar_vempty(int s) { return 2 * kStagesK + kStagesV + s; }
constexpr int kBar0 = 2 * (kStagesK + kStagesV);  // first barrier after the ring's
__device__ __forceinline__ constexpr int bar_qfull() { return kBar0; }
// Lane m's S and P share a TMEM buffer (its j-th tile uses buffer j & 1) and each buffer has its own pair of
// barriers: a buffer's next phase cannot complete before the other side has observed the
// current one (QK(j+2) is issued after PV(j), which is issued after pfull(j) was seen), so a
// parity wait never falls two phases behind.  One pfull barrier for both buffers would: the
// softmax warps can finish tile j+1 while the MMA thread still waits for V(j).
__device__ __forceinline__ constexpr int bar_sfull(int m, int buf) { return kBar0 + 1 + m * 5 + buf; }
__device__ __forceinline__ constexpr int bar_pfull(int m, int buf) { return kBar0 + 1 + m * 5 + 2 + buf; }
__device__ __forceinline__ constexpr int bar_pvdone(int m) { return kBar0 + 1 + m * 5 + 4; }
__device__ __forceinline__ constexpr int bar_item() { return kBar0 + 1 + kRowTiles * 5; }
__device__ __forceinline__ constexpr int bar_qempty() { return kBar0 + 2 + kRowTiles * 5; }
// key mode: both softmax warpgroups have their partial result (and its PV completions) behind them
__device__ __forceinline__ constexpr int bar_merge() { return kBar0 + 3 + kRowTiles * 5; }

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
tree_attention_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap map_k,
                      const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_q) {
    using S = Smem<D>;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = a.Hq / a.Hkv;
    const uint32_t bars = base + S::kOffBar;
    auto bar = [&](int i) { return bars + 8u * i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + S::kOffMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + S::kOffMisc + 8);

    // The work list was written once for the whole step.  From the second layer on it is at least
    // two kernels old: this kernel can only have started after its predecessor had started, which
    // can only have started after every CTA of the kernel before that one had passed its own
    // dependency wait, i.e. after the kernel that wrote the list had completed and flushed.  (Every
    // kernel of the library signals its dependents only after its own wait, or never.)  So the
    // list is read before the wait, under the tail of the preceding kernel; only when the list was
    // written by the kernel immediately before this one does the read have to follow the wait.
    // Every thread reads the CTA's first item for itself: no role waits for another.
    int4 head = make_int4(0, 0, 0, 0);
    Item first_it = {};
    auto read_plan = [&]() {
        head = __ldcg(a.plan_head);
        if (static_cast<int>(blockIdx.x) < head.x) first_it = load_item(a, blockIdx.x, head.y, G);
    };
    if (!a.plan_after_wait) read_plan();

    // ---- one-time set-up ---------------------------------------------------------------
    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kStagesK; ++s) {
            mbar_init(bar(bar_kfull(s)), 1);
            mbar_init(bar(bar_kempty(s)), 2);  // one arrival per lane (two from the owner in key mode)
        }
        for (int s = 0; s < kStagesV; ++s) {
            mbar_init(bar(bar_vfull(s)), 1);
            mbar_init(bar(bar_vempty(s)), 2);
        }
        mbar_init(bar(bar_qfull()), a.q_by_tma ? 1 : kSoftmaxThreads);
        mbar_init(bar(bar_qempty()), 2);
        for (int m = 0; m < kRowTiles; ++m) {
            for (int bf = 0; bf < 2; ++bf) {
                mbar_init(bar(bar_sfull(m, bf)), 1);
                mbar_init(bar(bar_pfull(m, bf)), kBM);
            }
            mbar_init(bar(bar_pvdone(m)), 1);
        }
        mbar_init(bar(bar_item()), kSyncThreads);
        mbar_init(bar(bar_merge()), kSoftmaxThreads);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         base + S::kOffMisc),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (warp == kProducerWarp && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
    }
    // Everything above touches no global memory, so under programmatic dependent launch it
    // overlaps the tail of the preceding kernel.
    pdl_wait();
    pdl_launch_dependents();
    if (a.plan_after_wait) read_plan();
    tc_fence_before();
    __syncthreads();  // barriers and the TMEM address are visible
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int total_items = head.x, group_rows = head.y;
    // The list must still describe the step parameters it is used with (the caller changes them only
    // through the library, or asks for a new list): one thread compares its item's sequence.
    bool stale = false;
    if (tid == 0 && static_cast<int>(blockIdx.x) < total_items) {
        const int n_live = min(max(a.n_nodes[first_it.b], 0), a.max_tt), L_live = max(a.steps[first_it.b].prefix_len, 0);
        stale = (n_live != first_it.n) || (L_live != first_it.L);
    }
    // The producers issue the first copies of the CTA's first item at once.
    const bool early = (warp == kProducerWarp || warp == kVProducerWarp) && lane == 0 &&
                       static_cast<int>(blockIdx.x) < total_items;
    if (early) {
        const Item& it = first_it;
        if (warp == kProducerWarp) {
            mbar_expect_tx(bar(bar_kfull(0)), S::kKVTile);
            tma_load_5d(base + S::kOffK, &map_k, bar(bar_kfull(0)), 0, it.t_begin * kBN, it.g, it.b, 0);
            if (a.q_by_tma) {
                mbar_expect_tx(bar(bar_qfull()), it.nmt * S::kQTile);
                for (int m = 0; m < it.nmt; ++m)
                    tma_load_5d(base + S::kOffQ + m * S::kQTile, &map_q, bar(bar_qfull()), 0, 0, it.g,
                                it.b * a.max_tt + it.tok0 + m * (kBM / G), 0);
            }
        } else if (!(kWaitTest && (a.test_drop & 1))) {
            mbar_expect_tx(bar(bar_vfull(0)), S::kKVTile);
            tma_load_5d(base + S::kOffV, &map_v, bar(bar_vfull(0)), 0, it.t_begin * kBN, it.g, it.b, 0);
        }
    }
    auto get_item = [&](int item, int local) {  // local = how many items this CTA has started before
        return local == 0 ? first_it : load_item(a, item, group_rows, G);
    };

    // Running use counts of the barrier families.  Every role walks the same items and tiles in
    // the same order, so each keeps its own copy.
    uint32_t kt_run = 0;     // K/V ring uses (all tiles of all items)
    uint32_t jx = 0;         // tiles this lane has taken (S/P buffers, PV completions)
    uint32_t items_run = 0;
    uint32_t merges_run = 0;  // key-mode items (uses of the merge barrier)
    bool alive = true;

    // Registers follow the roles: the softmax warpgroups hold a tile of S, a tile of P and a row of
    // O; the warpgroup of the producers and MMA issuers needs few (384 x 168 at launch).
    if (warp >= kProducerWarp) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsIssue));
    if (warp == kProducerWarp) {
        // ================================ TMA producer: K tiles and Q =======================
        if (lane == 0) {
            int li = 0;
            for (int item = blockIdx.x; item < total_items && alive; item += gridDim.x, ++li) {
                const Item it = get_item(item, li);
                for (int t = it.t_begin; t < it.t_end; ++t, ++kt_run) {
                    const int s = kt_run % kStagesK;
                    if (kt_run > 0) {  // the CTA's very first tile went out during the set-up
                        // the first use of a stage finds it free
                        if (kt_run >= kStagesK &&
                            !mbar_wait(bar(bar_kempty(s)), ((kt_run / kStagesK) & 1u) ^ 1u, abort_flag)) {
                            alive = false;
                            break;
                        }
                        mbar_expect_tx(bar(bar_kfull(s)), S::kKVTile);
                        tma_load_5d(base + S::kOffK + s * S::kKVTile, &map_k, bar(bar_kfull(s)), 0, t * kBN, it.g,
                                    it.b, 0);
                    }
                    if (t == it.t_begin && a.q_by_tma) {
                        // Q follows the first K tile: K and Q are what the first MMA needs.  The Q
                        // tiles of the previous item are free once its last QK^T has completed.
                        if (items_run > 0) {
                            if (!mbar_wait(bar(bar_qempty()), (items_run & 1u) ^ 1u, abort_flag)) {
                                alive = false;
                                break;
                            }
                            mbar_expect_tx(bar(bar_qfull()), it.nmt * S::kQTile);
                            for (int m = 0; m < it.nmt; ++m)
                                tma_load_5d(base + S::kOffQ + m * S::kQTile, &map_q, bar(bar_qfull()), 0, 0, it.g,
                                            it.b * a.max_tt + it.tok0 + m * (kBM / G), 0);
                        }
                        ++items_run;
                    }
                }
            }
            // Drain: every copy this thread issued has landed before the CTA may exit (each one is
            // waited for, also after an earlier wait has run out).
            bool landed = !(a.q_by_tma && items_run > 0) || drain_wait(bar(bar_qfull()), (items_run - 1u) & 1u);
            const uint32_t issued = kt_run;
            for (uint32_t u = (issued > kStagesK ? issued - kStagesK : 0u); u < issued; ++u)
                landed = drain_wait(bar(bar_kfull(u % kStagesK)), (u / kStagesK) & 1u) && landed;
            alive = alive && landed;
        }
    } else if (warp == kVProducerWarp) {
        // ================================ TMA producer: V tiles =============================
        if (lane == 0) {
            int li = 0;
            for (int item = blockIdx.x; item < total_items && alive; item += gridDim.x, ++li) {
                const Item it = get_item(item, li);
                for (int t = it.t_begin; t < it.t_end; ++t, ++kt_run) {
                    const int s = kt_run % kStagesV;
                    if (kt_run == 0) continue;  // went out during the set-up
                    if (kt_run >= kStagesV &&
                        !mbar_wait(bar(bar_vempty(s)), ((kt_run / kStagesV) & 1u) ^ 1u, abort_flag)) {
                        alive = false;
                        break;
                    }
                    mbar_expect_tx(bar(bar_vfull(s)), S::kKVTile);
                    tma_load_5d(base + S::kOffV + s * S::kKVTile, &map_v, bar(bar_vfull(s)), 0, t * kBN, it.g, it.b,
                                0);
                }
            }
            const uint32_t issued = kt_run;
            bool landed = true;
            for (uint32_t u = (issued > kStagesV ? issued - kStagesV : 0u); u < issued; ++u)
                landed = drain_wait(bar(bar_vfull(u % kStagesV)), (u / kStagesV) & 1u) && landed;
            alive = alive && landed;
        }
    } else if (warp == kMmaWarp0 || warp == kMmaWarp0 + 1) {
        // ================================ MMA issuer of lane x ============================
        // The whole warp walks the loop and waits (so that every value stays warp-uniform);
        // one elected lane issues.  The MMAs of one thread execute in issue order: QK of this
        // lane's tile j+1 is issued before PV of tile j, so the tensor pipe has S(j+1) to work on
        // while the softmax warps turn S(j) into P(j), and QK(j+2) cannot overwrite the TMEM
        // buffer j & 1 before PV(j) has read P(j) from it.
        const int x = warp - kMmaWarp0;
        constexpr uint32_t kIdescQK = instr_desc(kBN, false);
        constexpr uint32_t kIdescPV = instr_desc(D, true);
        // Descriptors differ only in the (16-byte granular) start address, the low 14 bits.
        const uint64_t qdesc0 = smem_desc(base + S::kOffQ, 16, 1024);
        const uint64_t kdesc0 = smem_desc(base + S::kOffK, 16, 1024);
        const uint64_t vdesc0 = smem_desc(base + S::kOffV, S::kKVPanel, 1024);
        const uint32_t o_t = tmem + x * 256 + 128;
        uint32_t k_seen = 0xFFFFFFFFu;  // ring use whose K tile this warp has already seen arrive
        for (int item = blockIdx.x; item < total_items && alive; item += gridDim.x, ++items_run) {
            const Item it = get_item(item, static_cast<int>(items_run));
            const bool row_mode = it.nmt == 2;
            const uint64_t qdesc = qdesc0 + static_cast<uint64_t>((row_mode ? x : 0) * (S::kQTile >> 4));
            alive = warp_wait(bar(bar_qfull()), items_run & 1u, abort_flag);
            tc_fence_after();
            if (row_mode && x == 1) {
                // Lane 1 starts half a tile period behind lane 0: the lanes' bursts of MMAs (P V of one
                // tile, Q K^T of the tile after next) then take turns on the tensor pipe instead of
                // queueing behind each other, which is what decides when a lane gets its next S.
                const long long t_go = clock64() + a.stagger;
                while (clock64() < t_go) {}
            }
            bool have_prev = false, first_pv = true;
            uint32_t prev_kt = 0, prev_j = 0;
            // In key mode a tile belongs to one lane alone: its owner releases the stage for both.
            const int releases = row_mode ? 1 : 2;
            // P V of this lane's previous tile.  While it waits for P it looks (without blocking) at
            // the K tile of the lane's next Q K^T, whose wait would otherwise sit between P V and the
            // next Q K^T: the chain that decides when the softmax warps get their next S.
            auto issue_pv = [&](uint32_t next_use) {
                const int s = prev_kt % kStagesV;
                if (!warp_wait(bar(bar_vfull(s)), (prev_kt / kStagesV) & 1u, abort_flag)) return false;
                if (next_use != 0xFFFFFFFFu &&
                    __all_sync(kFull, mbar_try(bar(bar_kfull(next_use % kStagesK)), (next_use / kStagesK) & 1u)))
                    k_seen = next_use;
                if (!warp_wait(bar(bar_pfull(x, prev_j & 1u)), (prev_j >> 1) & 1u, abort_flag)) return false;
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t vdesc = vdesc0 + static_cast<uint64_t>(s * (S::kKVTile >> 4));
                    // P of keys 32h .. 32h+31: hi in columns 32h .. 32h+15, lo in 32h+16 .. 32h+31
                    const uint32_t p_t = tmem + x * 256 + (prev_j & 1u) * kBN;
#pragma unroll
                    for (int kk = 0; kk < kBN / 16; ++kk) {
                        const uint32_t a_t = p_t + (kk >> 1) * 32 + (kk & 1) * 8;
                        umma_ts(o_t, a_t, vdesc + kk * (2048 >> 4), kIdescPV, (first_pv && kk == 0) ? 0u : 1u);
                        umma_ts(o_t, a_t + 16, vdesc + kk * (2048 >> 4), kIdescPV, 1u);
                    }
                    umma_commit(bar(bar_pvdone(x)));
                    for (int rls = 0; rls < releases; ++rls) umma_commit(bar(bar_vempty(s)));
                }
                __syncwarp();
                first_pv = false;
                return true;
            };
            const int t_step = row_mode ? 1 : 2;  // distance to this lane's next tile
            for (int t = it.t_begin; t < it.t_end && alive; ++t, ++kt_run) {
                const int s = kt_run % kStagesK;
                const bool own = row_mode || (((t - it.t_begin) & 1) == x);
                if (own) {
                    if (k_seen != kt_run)
                        alive = warp_wait(bar(bar_kfull(s)), (kt_run / kStagesK) & 1u, abort_flag);
                    if (!alive) break;
                    tc_fence_after();
                    if (elect_one()) {
                        const uint64_t kdesc = kdesc0 + static_cast<uint64_t>(s * (S::kKVTile >> 4));
                        const uint32_t s_t = tmem + x * 256 + (jx & 1u) * kBN;
#pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks)
                            umma(s_t, qdesc + ((ks >> 2) * (S::kQPanel >> 4) + (ks & 3) * 2),
                                 kdesc + ((ks >> 2) * (S::kKVPanel >> 4) + (ks & 3) * 2), kIdescQK, ks > 0 ? 1u : 0u);
                        umma_commit(bar(bar_sfull(x, jx & 1u)));
                        for (int rls = 0; rls < releases; ++rls) umma_commit(bar(bar_kempty(s)));
                    }
                    __syncwarp();
                    if (have_prev)
                        alive = issue_pv(t + t_step < it.t_end ? kt_run + static_cast<uint32_t>(t_step) : 0xFFFFFFFFu);
                    have_prev = true, prev_kt = kt_run, prev_j = jx;
                    ++jx;
                }
                // Q is free for the next item once the last QK^T of both lanes has completed
                if (t + 1 == it.t_end && elect_one()) umma_commit(bar(bar_qempty()));
                __syncwarp();
            }
            if (alive && have_prev) alive = issue_pv(0xFFFFFFFFu);
            tc_fence_before();
            if (!alive) break;
            // end of item: the softmax warps have read O and S, Q and P may be overwritten
            mbar_arrive(bar(bar_item()));
            alive = warp_wait(bar(bar_item()), items_run & 1u, abort_flag);
        }
    }
    } else {
        // ================================ softmax warpgroup of lane x =====================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        const int x = warp >> 2;
        const int r = (warp & 3) * 32 + lane;          // row inside the tile = TMEM lane
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t o_t = tmem + lane_sel + x * 256 + 128;
        constexpr int kChunks = D / 8;                 // 16-byte pieces of a row
        for (int item = blockIdx.x; item < total_items && alive; item += gridDim.x, ++items_run) {
            const Item it = get_item(item, static_cast<int>(items_run));
            const bool row_mode = it.nmt == 2;
            // ---- Q tiles -> shared memory in the swizzled K-major layout (only when the group
            // size does not allow the TMA view) ---------------------------------------------
            if (!a.q_by_tma) {
                // (a plain loop: this path serves group sizes that do not divide 128 and is not
                // worth its unrolled form's code size)
                const int total = it.nmt * kBM * kChunks;
#pragma unroll 1
                for (int i = tid; i < total; i += kSoftmaxThreads) {
                    const int row = i / kChunks, c = i % kChunks;
                    const int Rq = it.row_base + row;
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (Rq < it.M) {
                        const int t = Rq / G, h = it.g * G + Rq % G;
                        v = __ldg(reinterpret_cast<const uint4*>(
                            a.q + ((static_cast<int64_t>(it.b) * a.max_tt + t) * a.Hq + h) * D + c * 8));
                    }
                    const int m = row / kBM, rr = row % kBM;
                    unsigned char* dst = base_ptr + S::kOffQ + m * S::kQTile + (c >> 3) * S::kQPanel + rr * 128 +
                                         (((c & 7) ^ (rr & 7)) << 4);
                    *reinterpret_cast<uint4*>(dst) = v;
                }
                fence_proxy_async();
                mbar_arrive(bar(bar_qfull()));
            }

            const int R = it.row_base + (row_mode ? x * kBM : 0) + r;
            const bool row_ok = R < it.M;
            unsigned long long mlo = 0ull, mhi = 0ull;
            if (row_ok) {
                const int t = R / G;
                mlo = a.mask[(static_cast<int64_t>(it.b) * a.max_tt + t) * 2 + 0];
                mhi = a.mask[(static_cast<int64_t>(it.b) * a.max_tt + t) * 2 + 1];
                // only nodes of this tree can be visible
                if (it.n < 64) {
                    mlo &= (1ull << it.n) - 1ull;
                    mhi = 0ull;
                } else if (it.n < 128) {
                    mhi &= (1ull << (it.n - 64)) - 1ull;
                }
            }
            float m_ref = -INFINITY, l_run = 0.f;
            const int kv_len = it.L + it.n;
            // PV completions of this lane seen so far.  pvdone completes once per tile and a parity
            // wait must never fall two phases behind, so PV(j-1) is observed before P(j) is handed
            // over (PV(j) cannot be issued earlier): by then it has usually completed.
            uint32_t pv_seen = jx;
            bool first = true;
            // A wait on a barrier costs a few hundred cycles even when its phase completed long ago,
            // and this loop is the longest dependent chain of the kernel.  So the two things a tile
            // has to wait for are looked at early, without blocking, and the answers are used later:
            // PV(j-1) before the exponentials, S(j+1) between their halves.  When S(j+1) is there its
            // load is issued before P(j) is handed over, and the next round starts with the data.
            uint32_t sr[2][32];
            bool s_loaded = false;
            const int t_step = row_mode ? 1 : 2;  // distance to this lane's next tile

            for (int t = it.t_begin; t < it.t_end; ++t, ++kt_run) {
                if (!(row_mode || (((t - it.t_begin) & 1) == x))) continue;
                const uint32_t buf = jx & 1u;
                if (!s_loaded) {
                    if (!warp_wait(bar(bar_sfull(x, buf)), (jx >> 1) & 1u, abort_flag)) {
                        alive = false;
                        break;
                    }
                    tc_fence_after();
                    tmem_ld32(tmem + lane_sel + x * 256 + buf * kBN, sr[0]);
                    tmem_ld32(tmem + lane_sel + x * 256 + buf * kBN + 32, sr[1]);
                }
                tmem_wait_ld();

                // ---- ancestor mask (tiles that reach past the prefix only), row maximum -------
                const int j0 = t * kBN;
                float tmax = -INFINITY;
                if (j0 + kBN > it.L) {
                    const int off = j0 - it.L;  // tile start relative to the first tree slot
                    unsigned long long allowed;
                    if (off >= 64)
                        allowed = mhi >> (off - 64);
                    else if (off > 0)
                        allowed = (mlo >> off) | (mhi << (64 - off));
                    else if (off == 0)
                        allowed = mlo;
                    else  // -64 < off < 0: the first -off keys are prefix
                        allowed = (mlo << (-off)) | ((1ull << (-off)) - 1ull);
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            float s = __uint_as_float(sr[h][c]);
                            if (!((allowed >> (h * 32 + c)) & 1ull)) s = -INFINITY;
                            sr[h][c] = __float_as_uint(s);
                            tmax = fmaxf(tmax, s);
                        }
                } else {
                    float t4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // four independent chains
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int c = 0; c < 32; c += 2)
                            t4[(c >> 1) & 3] = max3(t4[(c >> 1) & 3], __uint_as_float(sr[h][c]), __uint_as_float(sr[h][c + 1]));
                    tmax = fmaxf(fmaxf(t4[0], t4[1]), fmaxf(t4[2], t4[3]));
                }
                tmax *= a.scale_log2;  // the scale is positive: max(scale * s) = scale * max(s)
                const float m_new = fmaxf(m_ref, tmax);
                // Lazy rescale: O and l keep the old reference maximum while the true one
                // grew by less than 2^kRescaleSlack (fp32 accumulators have the head-room).
                const bool need = !first && (m_new > m_ref + kRescaleSlack);
                if (first) m_ref = m_new;
                if (__any_sync(kFull, need)) {
                    // O may only be touched once PV of the previous tile has completed
                    while (pv_seen < jx) {
                        if (!warp_wait(bar(bar_pvdone(x)), pv_seen & 1u, abort_flag)) alive = false;
                        ++pv_seen;
                    }
                    if (!alive) break;
                    const float corr = need ? ex2_approx(m_ref - m_new) : 1.f;
                    if (need) m_ref = m_new;
                    l_run *= corr;
                    tc_fence_after();
#pragma unroll 1
                    for (int c0 = 0; c0 < D; c0 += 32) {
                        uint32_t orr[32];
                        tmem_ld32(o_t + c0, orr);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) orr[c] = __float_as_uint(__uint_as_float(orr[c]) * corr);
                        tmem_st32(o_t + c0, orr);
                    }
                    tmem_wait_st();
                }
                const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                // PV(j-1): asked now, answered after the exponentials (pv_seen is jx or jx - 1 here)
                const bool pv_probe = (pv_seen == jx) || mbar_try(bar(bar_pvdone(x)), pv_seen & 1u);
                const bool has_next = t + t_step < it.t_end;
                bool s_probe = false;

                // ---- stale V rows of the sequence's last tile must not reach the MMA (in row mode
                // both lanes clear them: each lane's PV is ordered behind its own warpgroup only) ----
                const bool clear_v = j0 + kBN > kv_len;
                if (clear_v) {
                    const int s = kt_run % kStagesV;
                    if (!warp_wait(bar(bar_vfull(s)), (kt_run / kStagesV) & 1u, abort_flag)) {
                        alive = false;
                        break;
                    }
                    const int valid = kv_len - j0;
                    unsigned char* vt = base_ptr + S::kOffV + s * S::kKVTile;
                    for (int i = r; i < (kBN - valid) * 8 * S::kPanels; i += kBM) {
                        const int row = valid + i / (8 * S::kPanels), cc = i % (8 * S::kPanels);
                        *reinterpret_cast<uint4*>(vt + (cc >> 3) * S::kKVPanel + row * 128 + ((cc & 7) << 4)) =
                            make_uint4(0u, 0u, 0u, 0u);
                    }
                }

                // ---- P = exp2(scale * S - m) as bf16 hi + lo, back into the columns S came from.
                // hi is p truncated to bf16, so p - hi is exact and lo = bf16(p - hi) leaves an
                // error of 2^-16 p.  Packed fp32 pairs halve the instruction count.  Each half of the
                // tile (32 keys) becomes 16 columns of hi and 16 of lo in place of its own 32 columns
                // of S, stored as soon as it is ready so that the store overlaps the other half.
                {
                    const unsigned long long sc2 = pack2(a.scale_log2, a.scale_log2);
                    const unsigned long long nm2 = pack2(-m_use, -m_use);
                    unsigned long long psum2 = pack2(0.f, 0.f);
                    const uint32_t p_t = tmem + lane_sel + x * 256 + buf * kBN;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (h == 1 && has_next)
                            s_probe = mbar_try(bar(bar_sfull(x, buf ^ 1u)), ((jx + 1u) >> 1) & 1u);
                        uint32_t w[32];
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            float x0, x1;
                            unpack2(fma2(pack2(__uint_as_float(sr[h][2 * c]), __uint_as_float(sr[h][2 * c + 1])), sc2, nm2),
                                    x0, x1);
                            const float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
                            const unsigned long long p2 = pack2(p0, p1);
                            psum2 = add2(psum2, p2);
                            const uint32_t b0 = __float_as_uint(p0), b1 = __float_as_uint(p1);
                            w[c] = __byte_perm(b0, b1, 0x7632);
                            float l0, l1;
                            unpack2(sub2(p2, pack2(__uint_as_float(b0 & 0xFFFF0000u), __uint_as_float(b1 & 0xFFFF0000u))),
                                    l0, l1);
                            w[16 + c] = pack_bf16(l0, l1);
                        }
                        tmem_st32(p_t + h * 32, w);
                    }
                    float ps0, ps1;
                    unpack2(psum2, ps0, ps1);
                    l_run += ps0 + ps1;
                }
                // S of this lane's next tile, if it has arrived (sr is free now)
                s_loaded = false;
                if (has_next) {
                    if (!__all_sync(kFull, s_probe))
                        s_probe = mbar_try(bar(bar_sfull(x, buf ^ 1u)), ((jx + 1u) >> 1) & 1u);
                    if (__all_sync(kFull, s_probe)) {
                        tc_fence_after();
                        tmem_ld32(tmem + lane_sel + x * 256 + (buf ^ 1u) * kBN, sr[0]);
                        tmem_ld32(tmem + lane_sel + x * 256 + (buf ^ 1u) * kBN + 32, sr[1]);
                        s_loaded = true;
                    }
                }
                tmem_wait_st();
                if (clear_v) fence_proxy_async();
                if (pv_seen < jx) {
                    if (!__all_sync(kFull, pv_probe) &&
                        !warp_wait(bar(bar_pvdone(x)), pv_seen & 1u, abort_flag))
                        alive = false;
                    ++pv_seen;
                }
                if (!alive) break;
                tc_fence_before();
                mbar_arrive(bar(bar_pfull(x, buf)));
                ++jx;
                first = false;
            }
            if (!alive) break;

            // ---- epilogue --------------------------------------------------------------
            // Row mode: the lane owns its rows and all their columns.  Key mode: the two lanes hold
            // partial results over different keys for the same rows; they exchange (max, sum) through
            // shared memory and each merges one half of the columns, reading the other lane's
            // accumulator straight from tensor memory (same TMEM lanes, other columns).
            const bool direct = it.splits == 1;  // the group's only item: the result is final
            const int nt_oth = row_mode ? 0 : ((it.t_end - it.t_begin + (x ? 1 : 0)) >> 1);  // the other lane's tiles
            while (pv_seen < jx) {
                if (!warp_wait(bar(bar_pvdone(x)), pv_seen & 1u, abort_flag)) alive = false;
                ++pv_seen;
            }
            if (!alive) break;
            const bool use_self = !first, use_oth = nt_oth > 0;
            float m_tot = (l_run > 0.f) ? m_ref : -INFINITY, l_tot = l_run, w_self = 1.f, w_oth = 0.f;
            int c_begin = 0, c_end = D / 32;  // 32-column pieces of the row this thread writes
            if (!row_mode) {
                float2* xch = reinterpret_cast<float2*>(base_ptr + S::kOffMerge);
                xch[x * kBM + r] = make_float2(m_tot, l_run);
                tc_fence_before();
                mbar_arrive(bar(bar_merge()));
                alive = warp_wait(bar(bar_merge()), merges_run & 1u, abort_flag);
                ++merges_run;
                if (!alive) break;
                const float2 oth = xch[(x ^ 1) * kBM + r];
                const float m_self = m_tot;
                m_tot = fmaxf(m_self, oth.x);
                w_self = (m_self == -INFINITY) ? 0.f : ex2_approx(m_self - m_tot);
                w_oth = (oth.x == -INFINITY) ? 0.f : ex2_approx(oth.x - m_tot);
                l_tot = l_run * w_self + oth.y * w_oth;
                c_begin = x * (D / 64), c_end = c_begin + D / 64;
            }
            tc_fence_after();
            {
                const int t = R / G, h = it.g * G + R % G;
                const float inv = (l_tot > 0.f) ? 1.f / l_tot : 0.f;
                __nv_bfloat16* dst = a.o + ((static_cast<int64_t>(it.b) * a.max_tt + t) * a.Hq + h) * D;
                const int64_t slot = static_cast<int64_t>(item) * kRowTiles + (row_mode ? x : 0);
                uint4* po = a.part_o + slot * (D / 8) * kBM + r;
                const uint32_t oth_t = tmem + lane_sel + (x ^ 1) * 256 + 128;
                if (row_ok && direct && a.lse && (row_mode || x == 0))
                    a.lse[(static_cast<int64_t>(it.b) * a.max_tt + t) * a.Hq + h] =
                        (m_tot + log2f(l_tot)) * 0.6931471805599453f;
                // The row leaves tensor memory in 32-column pieces (plain loops: the stores, not
                // the loads, bound this part, and it runs once per item, so small code wins).
                // Partials assume a scale of 1 and keep the largest magnitude; when a row of the
                // warp would leave the fp16 range, a second pass writes such rows again with
                // their scale (a scale per half of the columns: the halves may come from
                // different lanes).
                float am[4] = {0.f, 0.f, 0.f, 0.f};
                float scale = 1.f;  // O = Ohat * l * scale
                uint32_t r0[32], r1[32];
#pragma unroll 1
                for (int pass = 0; pass < 2; ++pass) {
                    const float mul = (pass == 0) ? inv : inv / scale;
                    const bool store = row_ok && (pass == 0 || scale != 1.f);
                    // Two loads from tensor memory are in flight together: in key mode a piece of this
                    // lane's O and the same piece of the other lane's, in row mode two pieces of its own.
                    // (The loads are warp-wide and their conditions warp-uniform.)
                    const int c_step = row_mode ? 2 : 1;
#pragma unroll 1
                    for (int c0 = c_begin; c0 < c_end; c0 += c_step) {
                        const bool second = row_mode && c0 + 1 < c_end;
                        if (use_self) tmem_ld32(o_t + c0 * 32, r0);
                        if (use_oth) tmem_ld32(oth_t + c0 * 32, r1);
                        if (second) tmem_ld32(o_t + (c0 + 1) * 32, r1);
                        tmem_wait_ld();
#pragma unroll
                        for (int h2 = 0; h2 < 2; ++h2) {
                            if (h2 == 1 && !second) break;
                            const int c = c0 + h2;
                            if (store) {
#pragma unroll
                                for (int q4 = 0; q4 < 4; ++q4) {
                                    float g8[8];
#pragma unroll
                                    for (int e = 0; e < 8; ++e) {
                                        float v;
                                        if (h2 == 1) {
                                            v = __uint_as_float(r1[q4 * 8 + e]);
                                        } else {
                                            v = use_self ? __uint_as_float(r0[q4 * 8 + e]) * w_self : 0.f;
                                            if (use_oth) v = fmaf(__uint_as_float(r1[q4 * 8 + e]), w_oth, v);
                                        }
                                        g8[e] = v;
                                    }
                                    uint4 v;
                                    if (direct) {
                                        v.x = pack_bf16(g8[0] * mul, g8[1] * mul), v.y = pack_bf16(g8[2] * mul, g8[3] * mul);
                                        v.z = pack_bf16(g8[4] * mul, g8[5] * mul), v.w = pack_bf16(g8[6] * mul, g8[7] * mul);
                                        *reinterpret_cast<uint4*>(dst + (c * 4 + q4) * 8) = v;
                                    } else {
                                        am[q4] = max3(am[q4], fabsf(g8[0]), fabsf(g8[1]));
                                        am[q4] = max3(am[q4], fabsf(g8[2]), fabsf(g8[3]));
                                        am[q4] = max3(am[q4], fabsf(g8[4]), fabsf(g8[5]));
                                        am[q4] = max3(am[q4], fabsf(g8[6]), fabsf(g8[7]));
                                        v.x = pack_half2(g8[0] * mul, g8[1] * mul), v.y = pack_half2(g8[2] * mul, g8[3] * mul);
                                        v.z = pack_half2(g8[4] * mul, g8[5] * mul), v.w = pack_half2(g8[6] * mul, g8[7] * mul);
                                        __stcg(po + (c * 4 + q4) * kBM, v);
                                    }
                                }
                            }
                        }
                    }
                    if (direct || pass == 1) break;
                    // scale: 1 unless |O / l| would exceed 2^14 (fp16 holds up to 65504)
                    if (row_ok) {
                        const float nmax = fmaxf(fmaxf(am[0], am[1]), fmaxf(am[2], am[3])) * inv;
                        if (nmax > 16384.f) scale = exp2f(ceilf(log2f(nmax)) - 14.f);
                    }
                    // (the loads from tensor memory are warp-wide: the whole warp goes round again)
                    if (!__any_sync(kFull, scale != 1.f)) break;
                }
                if (row_ok && !direct) {
                    float* ml = reinterpret_cast<float*>(a.part_ml + slot * kBM + r);
                    if (row_mode) {
                        __stcg(a.part_ml + slot * kBM + r, make_float4(m_tot, l_tot, l_tot * scale, l_tot * scale));
                    } else if (x == 0) {
                        __stcg(reinterpret_cast<float2*>(ml), make_float2(m_tot, l_tot));
                        __stcg(ml + 2, l_tot * scale);
                    } else {
                        __stcg(ml + 3, l_tot * scale);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bar(bar_item()));
            alive = warp_wait(bar(bar_item()), items_run & 1u, abort_flag);
        }
    }

    // ---- tear-down: every role arrives here, whatever happened ------------------------------
    if (!alive) {
        *abort_flag = 1;
        atomicOr(a.status, RESPS_STATUS_WAIT_TIMEOUT);
    }
    if (stale) atomicOr(a.status, RESPS_STATUS_STALE_PLAN);
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp0) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// The per-sequence part of the work list, from the workspace into shared memory (the list is at
// least two kernels old when a combine kernel starts: see the note at the attention kernel).
__device__ __forceinline__ void load_sched(const AttnArgs& a, Sched& sc, int tid, int nthreads) {
    for (int b = tid; b <= a.batch; b += nthreads) {
        const int4* src = reinterpret_cast<const int4*>(a.plan_seq + b);
        const int4 lo = __ldcg(src), hi = __ldcg(src + 1);
        sc.item0[b] = hi.w;
        if (b < a.batch)
            sc.n[b] = lo.x, sc.L[b] = lo.y, sc.mp[b] = lo.z, sc.nfull[b] = lo.w, sc.kt[b] = hi.x, sc.s_row[b] = hi.y,
            sc.s_key[b] = hi.z;
    }
    if (tid == 0) sc.group_rows = __ldcg(a.plan_head).y;
    __syncthreads();
}

// Combines the partials of every (sequence, KV head, group of row tiles) that did not write O
// directly: O = sum_p w_p O_p / sum_p w_p l_p with w_p = 2^(m_p - max m).  A group has one partial
// per split and row tile (in key mode the two lanes of a CTA have merged theirs already).
//
// The kernel is two dependent round trips to L2 (partials in, O out) behind a dependency wait, so
// what counts is how many memory requests an SM has to issue: with plain loads a warp-load is four
// 128-byte requests, an SM can only keep so many in flight, and 100 requests per warp made the
// kernel several round trips long.  Here a CTA takes one row tile x two 8-column pieces and lets
// the copy engine fetch its share of every partial (one bulk copy per partial and column piece,
// one for the (max, sum, scales) of the rows) into shared memory: a few dozen requests per CTA, all
// in flight at once.
constexpr int kCombChunk = 8;   // partials fetched together
constexpr int kCombPieces = 2;  // 8-column pieces per CTA
constexpr int kCombSlotBytes = (kCombPieces + 1) * kBM * 16;  // per partial: the pieces, then (max, sum, scales)

template <int D>
__global__ void __launch_bounds__(kCombineThreads) attention_combine_kernel(const AttnArgs a) {
    constexpr int kPieces = D / 8;                    // 16-byte pieces of a row
    constexpr int kCtasPerTile = kPieces / kCombPieces;
    static_assert(kCombineThreads == kCombPieces * kBM, "thread = (row, piece)");
    extern __shared__ __align__(128) unsigned char comb_smem[];  // [kCombChunk][kCombSlotBytes]
    __shared__ Sched sc;
    __shared__ __align__(8) unsigned long long s_bar;
    pdl_launch_dependents();
    // The work list is fetched and the CTA's share located before the wait for the attention
    // kernel: all of this runs while that kernel drains.  A CTA without work leaves at once.
    load_sched(a, sc, threadIdx.x, kCombineThreads);  // ends with __syncthreads()
    const int tid = threadIdx.x;
    const int G = a.Hq / a.Hkv;
    const int group_rows = sc.group_rows;
    int blk = blockIdx.x, b = 0, tiles = 0;
    for (; b < a.batch; ++b) {
        tiles = ceil_div(sc.n[b] * G, kBM);
        if (blk < a.Hkv * tiles * kCtasPerTile) break;
        blk -= a.Hkv * tiles * kCtasPerTile;
    }
    if (b == a.batch) return;
    const int M = sc.n[b] * G;
    const int g = blk / (tiles * kCtasPerTile);
    const int tile = (blk - g * tiles * kCtasPerTile) / kCtasPerTile;
    const int c8_0 = (blk % kCtasPerTile) * kCombPieces;
    const int R0 = tile * kBM;
    const int nfull = sc.nfull[b], s_row = sc.s_row[b], s_key = sc.s_key[b];
    const int pair = R0 / group_rows;
    const bool key_mode = pair >= nfull;
    const int splits = key_mode ? s_key : s_row;
    if (splits <= 1) return;  // the group wrote O directly
    const int row_items = nfull * s_row;
    const int64_t item_first = sc.item0[b] + static_cast<int64_t>(g) * (row_items + (sc.mp[b] - nfull) * s_key) +
                               (key_mode ? row_items + (pair - nfull) * s_key : pair * s_row);
    const int mt = (R0 % group_rows) / kBM;  // row tile inside the group (a key-mode group is one tile)
    const int nv = min(kBM, M - R0);         // valid rows of the tile
    const uint32_t bar = smem_u32(&s_bar);
    if (tid == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int r = tid % kBM, cc = tid / kBM;
    pdl_wait();  // the attention kernel has finished and its partials are visible

    float Mx = -INFINITY, den = 0.f;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    bool ok = true;
    uint32_t phase = 0;
#pragma unroll 1
    for (int p0 = 0; p0 < splits; p0 += kCombChunk, phase ^= 1u) {
        const int np = min(kCombChunk, splits - p0);
        // one copy per thread, so that they are issued side by side: a partial's column pieces and
        // its (max, sum, scales), each nv x 16 contiguous bytes
        if (tid == 0) mbar_expect_tx(bar, static_cast<uint32_t>(np * (kCombPieces + 1) * nv * 16));
        if (tid < np * (kCombPieces + 1)) {
            const int u = tid / (kCombPieces + 1), c = tid % (kCombPieces + 1);
            const int64_t slot = (item_first + p0 + u) * kRowTiles + mt;
            const uint32_t dst = smem_u32(comb_smem + u * kCombSlotBytes + c * kBM * 16);
            const void* src = (c < kCombPieces) ? static_cast<const void*>(a.part_o + (slot * kPieces + c8_0 + c) * kBM)
                                                : static_cast<const void*>(a.part_ml + slot * kBM);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                         "l"(src), "r"(nv * 16), "r"(bar)
                         : "memory");
        }
        {
            // bounded: on expiry the status word is flagged and the CTA leaves without a result
            const uint32_t t0 = static_cast<uint32_t>(clock());
            uint32_t spins = 0;
            while (ok && !mbar_try(bar, phase))
                if ((++spins & 255u) == 0u && static_cast<uint32_t>(clock()) - t0 > kWaitLimitCycles) ok = false;
        }
        if (!__syncthreads_and(ok)) {
            if (tid == 0) atomicOr(a.status, RESPS_STATUS_WAIT_TIMEOUT);
            return;
        }
        if (r < nv) {
            float mx = Mx;
            for (int u = 0; u < np; ++u)
                mx = fmaxf(mx, reinterpret_cast<const float4*>(comb_smem + u * kCombSlotBytes + kCombPieces * kBM * 16)[r].x);
            if (mx != -INFINITY) {
                const float corr = ex2_approx(Mx - mx);  // 0 on the first chunk
                den *= corr;
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] *= corr;
                Mx = mx;
#pragma unroll 2
                for (int u = 0; u < np; ++u) {
                    const unsigned char* sl = comb_smem + u * kCombSlotBytes;
                    const float4 ml = reinterpret_cast<const float4*>(sl + kCombPieces * kBM * 16)[r];
                    if (ml.x == -INFINITY) continue;  // an empty partial holds no O
                    const float w = ex2_approx(ml.x - Mx);
                    den += ml.y * w;
                    const float wo = (c8_0 + cc < kPieces / 2 ? ml.z : ml.w) * w;  // O_p = Ohat * l * scale of this half
                    const uint4 v = reinterpret_cast<const uint4*>(sl + cc * kBM * 16)[r];
                    const uint32_t hw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&hw[e]));
                        acc[2 * e] += f.x * wo, acc[2 * e + 1] += f.y * wo;
                    }
                }
            }
        }
        if (p0 + kCombChunk < splits) __syncthreads();  // the next chunk overwrites the staging area
    }
    if (r >= nv) return;
    const float inv = 1.f / den;
    const int R = R0 + r;
    const int t = R / G, h = g * G + (R - t * G);
    __nv_bfloat16* dst = a.o + ((static_cast<int64_t>(b) * a.max_tt + t) * a.Hq + h) * D + (c8_0 + cc) * 8;
    uint4 out;
    out.x = pack_bf16(acc[0] * inv, acc[1] * inv);
    out.y = pack_bf16(acc[2] * inv, acc[3] * inv);
    out.z = pack_bf16(acc[4] * inv, acc[5] * inv);
    out.w = pack_bf16(acc[6] * inv, acc[7] * inv);
    *reinterpret_cast<uint4*>(dst) = out;
    if (a.lse && c8_0 + cc == 0)
        a.lse[(static_cast<int64_t>(b) * a.max_tt + t) * a.Hq + h] = (Mx + log2f(den)) * 0.6931471805599453f;
}

// The same with plain loads, one thread per (row, 8 columns) over a flat index space: its first
// data arrives sooner than through the copy engine, which wins when there is little to combine (a
// single sequence with at most two row tiles per KV head: 12.0 against 13.3 us per call on the
// 8B-shaped workload); with more rows the copy-engine form is ahead (26.4 against 28.1 us on the
// 70B-shaped one).
template <int D>
__global__ void __launch_bounds__(kCombineThreads) attention_combine_small_kernel(const AttnArgs a) {
    __shared__ Sched sc;
    pdl_launch_dependents();
    // The work list is fetched, and the thread's first piece of work located, before the wait
    // for the attention kernel: all of this runs while that kernel drains, in one round trip to
    // memory (the list carries the tree sizes it was planned for, which the attention kernel has
    // checked against the live ones).
    load_sched(a, sc, threadIdx.x, kCombineThreads);  // ends with __syncthreads()
    // A CTA past the last row of the largest tree has nothing to do and leaves: it may have started
    // only after the attention kernel ended, and whatever it does until it exits delays the next
    // kernel in the stream.
    {
        bool mine = false;
        for (int b = 0; b < a.batch; ++b)
            mine = mine || static_cast<long long>(blockIdx.x) * kCombineThreads < 1ll * sc.n[b] * a.Hq * (D / 8);
        if (!mine) return;
    }
    const unsigned G = static_cast<unsigned>(a.Hq / a.Hkv);
    const unsigned stride = gridDim.x * kCombineThreads;
    const unsigned group_rows = static_cast<unsigned>(sc.group_rows);
    // Work: (sequence, KV head, 8 columns, row) over the valid rows of groups that wrote partials;
    // consecutive threads take consecutive rows.  Every count fits 32 bits (at most 2^11 rows per
    // KV head, 2^4 column pieces, 2^7 heads).
    int b = 0;
    unsigned idx = blockIdx.x * kCombineThreads + threadIdx.x;
    bool waited = false;
    for (;;) {
        // ---- the next piece of work of this thread ------------------------------------------
        bool have = false;
        unsigned g = 0, c8 = 0, R = 0, M = 0;
        int splits = 0, n_parts = 0;
        bool key_mode = false;
        int64_t item_first = 0;
        for (; b < a.batch; ++b, idx = blockIdx.x * kCombineThreads + threadIdx.x) {
            const int nfull = sc.nfull[b], mp_b = sc.mp[b], s_row = sc.s_row[b], s_key_b = sc.s_key[b];
            if (sc.n[b] == 0 || ((s_row <= 1 || nfull == 0) && (s_key_b <= 1 || nfull == mp_b)))
                continue;  // every group wrote O directly
            M = static_cast<unsigned>(sc.n[b]) * G;
            const unsigned per_head = M * (D / 8);
            for (; idx < a.Hkv * per_head; idx += stride) {
                g = idx / per_head;
                const unsigned rem = idx - g * per_head;
                c8 = rem / M;
                R = rem - c8 * M;
                const int pair = static_cast<int>(R / group_rows);
                key_mode = pair >= nfull;
                splits = key_mode ? s_key_b : s_row;
                if (splits <= 1) continue;
                const int row_items = nfull * s_row;
                item_first = sc.item0[b] + static_cast<int64_t>(g) * (row_items + (mp_b - nfull) * s_key_b) +
                             (key_mode ? row_items + (pair - nfull) * s_key_b : pair * s_row);
                n_parts = splits;
                have = true;
                break;
            }
            if (have) break;
        }
        if (!waited) {
            pdl_wait();  // the attention kernel has finished and its partials are visible
            waited = true;
        }
        if (!have) break;

        // ---- O = sum_p w_p O_p / sum_p w_p l_p, w_p = 2^(m_p - max m): one pass over the partials,
        // ten at a time so that their loads are in flight together ---------------------------------
        const unsigned row2 = R % group_rows;
        const unsigned mt = row2 / kBM, r = row2 % kBM;  // (a key-mode group is one row tile: mt = 0)
        constexpr int kBatch = 10;
        float Mx = -INFINITY, den = 0.f;
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
        for (int p0 = 0; p0 < n_parts; p0 += kBatch) {
            float4 ml[kBatch];
            uint4 v[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int p = min(p0 + u, n_parts - 1);
                const int64_t slot = (item_first + p) * kRowTiles + mt;
                ml[u] = a.part_ml[slot * kBM + r];  // shared by the 16 column pieces of a row: through L1
                v[u] = __ldcg(a.part_o + (slot * (D / 8) + c8) * kBM + r);
            }
            float mx = Mx;
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                if (p0 + u < n_parts) mx = fmaxf(mx, ml[u].x);
            if (mx == -INFINITY) continue;
            const float corr = ex2_approx(Mx - mx);  // 0 on the first batch
            den *= corr;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] *= corr;
            Mx = mx;
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                if (p0 + u >= n_parts || ml[u].x == -INFINITY) continue;  // an empty partial holds no O
                const float w = ex2_approx(ml[u].x - Mx);
                den += ml[u].y * w;
                const float wo = (c8 < D / 16 ? ml[u].z : ml[u].w) * w;  // O_p = Ohat * l * scale of this half of the row
                const uint32_t hw[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&hw[e]));
                    acc[2 * e] += f.x * wo, acc[2 * e + 1] += f.y * wo;
                }
            }
        }
        const float inv = 1.f / den;
        const unsigned t = R / G, h = g * G + (R - t * G);
        __nv_bfloat16* dst = a.o + ((static_cast<int64_t>(b) * a.max_tt + t) * a.Hq + h) * D + c8 * 8;
        uint4 out;
        out.x = pack_bf16(acc[0] * inv, acc[1] * inv);
        out.y = pack_bf16(acc[2] * inv, acc[3] * inv);
        out.z = pack_bf16(acc[4] * inv, acc[5] * inv);
        out.w = pack_bf16(acc[6] * inv, acc[7] * inv);
        *reinterpret_cast<uint4*>(dst) = out;
        if (a.lse && c8 == 0)
            a.lse[(static_cast<int64_t>(b) * a.max_tt + t) * a.Hq + h] = (Mx + log2f(den)) * 0.6931471805599453f;
        idx += stride;
    }
}

// The same for batches of several sequences.  The kernel is a chain of two dependent memory round
// trips (partials in, O out) behind a
// dependency wait, so it is laid out for latency: one flat index space over all sequences (no
// pass per sequence), a piece of work = (row, 8 columns, one of 1, 2 or 4 shares of the partials)
// so that a thread has at most four partials (eight loads) to fetch and they are all in flight
// at once, the shares merged by shuffles, and few enough registers for four CTAs per SM, so
// that even the largest trees are one resident round.
constexpr int kCombineBatch = 4;  // partials a thread fetches at once

template <int D>
__global__ void __launch_bounds__(kCombineThreads, 4) attention_combine_flat_kernel(const AttnArgs a) {
    __shared__ Sched sc;
    __shared__ unsigned s_work0[kMaxBatchSmem + 1];  // first flat index of a sequence
    __shared__ unsigned char s_shares[kMaxBatchSmem];
    pdl_launch_dependents();
    // The work list is fetched, and the thread's first piece of work located, before the wait
    // for the attention kernel: all of this runs while that kernel drains, in one round trip to
    // memory (the list carries the tree sizes it was planned for, which the attention kernel has
    // checked against the live ones).
    load_sched(a, sc, threadIdx.x, kCombineThreads);  // ends with __syncthreads()
    // A CTA past the last piece of work that the trees at hand could need (four shares each) has
    // nothing to do and leaves: it may have started only after the attention kernel ended, and
    // whatever it does until it exits delays the next kernel in the stream.
    {
        unsigned long long bound = 0;
        for (int b = 0; b < a.batch; ++b) bound += 4ull * sc.n[b] * a.Hq * (D / 8) + 4;
        if (static_cast<unsigned long long>(blockIdx.x) * kCombineThreads >= bound) return;
    }
    const unsigned G = static_cast<unsigned>(a.Hq / a.Hkv);
    const unsigned group_rows = static_cast<unsigned>(sc.group_rows);
    if (threadIdx.x < 32) {
        // shares per piece of work and flat offsets (every sequence's range is a multiple of 4,
        // so that the shares of a piece sit in adjacent, aligned lanes)
        unsigned base = 0;
        for (int b0 = 0; b0 < a.batch; b0 += 32) {
            const int b = b0 + threadIdx.x;
            unsigned mine = 0;
            if (b < a.batch && sc.n[b] > 0) {
                const int nfull = sc.nfull[b], nkey = sc.mp[b] - nfull;
                const int parts = max(nfull > 0 && sc.s_row[b] > 1 ? sc.s_row[b] : 0, nkey > 0 && sc.s_key[b] > 1 ? sc.s_key[b] : 0);
                const unsigned shares = parts <= kCombineBatch ? 1u : parts <= 2 * kCombineBatch ? 2u : 4u;
                s_shares[b] = static_cast<unsigned char>(shares);
                if (parts > 0) mine = (static_cast<unsigned>(sc.n[b]) * a.Hq * (D / 8) * shares + 3u) & ~3u;
            }
            unsigned incl = mine;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const unsigned v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                if (threadIdx.x >= d) incl += v;
            }
            if (b < a.batch) s_work0[b] = base + incl - mine;
            base += __shfl_sync(0xFFFFFFFFu, incl, 31);
        }
        if (threadIdx.x == 0) s_work0[a.batch] = base;
    }
    __syncthreads();
    const unsigned total = s_work0[a.batch];
    const unsigned stride = gridDim.x * kCombineThreads;
    bool waited = false;
    // every lane of a warp goes round the same number of times (the merge is by shuffles)
    for (unsigned w0 = blockIdx.x * kCombineThreads + (threadIdx.x & ~31u); w0 < total || !waited; w0 += stride) {
        const unsigned w = w0 + (threadIdx.x & 31u);
        // ---- this thread's piece of work ------------------------------------------------------
        bool have = false;
        int b = 0, n_parts = 0, splits = 0;
        unsigned g = 0, c8 = 0, R = 0, share = 0, shares = 1;
        bool key_mode = false;
        int64_t item_first = 0;
        if (w < total) {
            int lo = 0, hi = a.batch;  // last sequence whose range starts at or before w
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (s_work0[mid] <= w) lo = mid; else hi = mid;
            }
            b = lo;
            shares = s_shares[b];
            const unsigned local = w - s_work0[b];
            const unsigned piece = local / shares;
            share = local - piece * shares;
            const unsigned M = static_cast<unsigned>(sc.n[b]) * G;
            const unsigned per_head = M * (D / 8);
            if (piece < a.Hkv * per_head) {  // (the range is padded to a multiple of 4)
                g = piece / per_head;
                const unsigned rem = piece - g * per_head;
                c8 = rem / M;
                R = rem - c8 * M;
                const int nfull = sc.nfull[b], s_row = sc.s_row[b], s_key_b = sc.s_key[b];
                const int pair = static_cast<int>(R / group_rows);
                key_mode = pair >= nfull;
                splits = key_mode ? s_key_b : s_row;
                if (splits > 1) {  // otherwise the group wrote O directly
                    const int row_items = nfull * s_row;
                    item_first = sc.item0[b] + static_cast<int64_t>(g) * (row_items + (sc.mp[b] - nfull) * s_key_b) +
                                 (key_mode ? row_items + (pair - nfull) * s_key_b : pair * s_row);
                    n_parts = splits;
                    have = true;
                }
            }
        }
        if (!waited) {
            pdl_wait();  // the attention kernel has finished and its partials are visible
            waited = true;
        }
        if (!__any_sync(0xFFFFFFFFu, have)) continue;

        // ---- this share's partials: p = share, share + shares, ... ------------------------------
        const unsigned row2 = R % group_rows;
        const unsigned mt = row2 / kBM, r = row2 % kBM;
        float Mx = -INFINITY, den = 0.f;
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (have) {
#pragma unroll 1
            for (int p0 = static_cast<int>(share); p0 < n_parts; p0 += kCombineBatch * static_cast<int>(shares)) {
                float4 ml[kCombineBatch];
                uint4 v[kCombineBatch];
#pragma unroll
                for (int u = 0; u < kCombineBatch; ++u) {
                    const int p = min(p0 + u * static_cast<int>(shares), n_parts - 1);
                    const int64_t slot = (item_first + p) * kRowTiles + mt;
                    ml[u] = a.part_ml[slot * kBM + r];  // shared by the 16 column pieces of a row: through L1
                    v[u] = __ldcg(a.part_o + (slot * (D / 8) + c8) * kBM + r);
                }
                float mx = Mx;
#pragma unroll
                for (int u = 0; u < kCombineBatch; ++u)
                    if (p0 + u * static_cast<int>(shares) < n_parts) mx = fmaxf(mx, ml[u].x);
                if (mx == -INFINITY) continue;
                const float corr = ex2_approx(Mx - mx);  // 0 on the first batch
                den *= corr;
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] *= corr;
                Mx = mx;
#pragma unroll
                for (int u = 0; u < kCombineBatch; ++u) {
                    if (p0 + u * static_cast<int>(shares) >= n_parts || ml[u].x == -INFINITY) continue;  // an empty partial holds no O
                    const float wgt = ex2_approx(ml[u].x - Mx);
                    den += ml[u].y * wgt;
                    const float wo = (c8 < D / 16 ? ml[u].z : ml[u].w) * wgt;  // O_p = Ohat * l * scale of this half of the row
                    const uint32_t hw[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&hw[e]));
                        acc[2 * e] += f.x * wo, acc[2 * e + 1] += f.y * wo;
                    }
                }
            }
        }
        // ---- the shares of a piece sit in adjacent lanes: merge them (every lane takes part) ----
#pragma unroll
        for (unsigned d = 1; d < 4; d <<= 1) {
            const float Mo = __shfl_xor_sync(0xFFFFFFFFu, Mx, d);
            const float Mn = fmaxf(Mx, Mo);
            const float sc_self = (Mx == -INFINITY) ? 0.f : ex2_approx(Mx - Mn);
            const bool on = d < shares;
            float dn = den * sc_self;
            float ac[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) ac[e] = acc[e] * sc_self;
            const float dno = __shfl_xor_sync(0xFFFFFFFFu, dn, d);
            if (on) den = dn + dno, Mx = Mn;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float o = __shfl_xor_sync(0xFFFFFFFFu, ac[e], d);
                if (on) acc[e] = ac[e] + o;
            }
        }
        if (have && share == 0) {
            const float inv = 1.f / den;
            const unsigned t = R / G, h = g * G + (R - t * G);
            __nv_bfloat16* dst = a.o + ((static_cast<int64_t>(b) * a.max_tt + t) * a.Hq + h) * D + c8 * 8;
            uint4 out;
            out.x = pack_bf16(acc[0] * inv, acc[1] * inv);
            out.y = pack_bf16(acc[2] * inv, acc[3] * inv);
            out.z = pack_bf16(acc[4] * inv, acc[5] * inv);
            out.w = pack_bf16(acc[6] * inv, acc[7] * inv);
            *reinterpret_cast<uint4*>(dst) = out;
            if (a.lse && c8 == 0)
                a.lse[(static_cast<int64_t>(b) * a.max_tt + t) * a.Hq + h] = (Mx + log2f(den)) * 0.6931471805599453f;
        }
    }
}

// cuTensorMapEncodeTiled, resolved at run time so that the library has no link-time
// dependency on the driver (it must load on a machine without one).
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// (element, slot, head, sequence, panel) view of a bf16 cache; a box is 64 slots of all panels.
bool make_kv_map(CUtensorMap* map, const void* basep, int D, int64_t capacity, int Hkv, int batch,
                 int64_t s_tok, int64_t s_head, int64_t s_seq) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    // a dimension of extent 1 never uses its stride; give it a valid one
    if (s_head <= 0) s_head = capacity * s_tok;
    if (s_seq <= 0) s_seq = s_head * Hkv;
    const cuuint32_t panels = static_cast<cuuint32_t>(D / 64);
    const cuuint64_t dims[5] = {64, static_cast<cuuint64_t>(capacity), static_cast<cuuint64_t>(Hkv),
                                static_cast<cuuint64_t>(batch), panels};
    const cuuint64_t strides[4] = {static_cast<cuuint64_t>(s_tok) * 2, static_cast<cuuint64_t>(s_head) * 2,
                                   static_cast<cuuint64_t>(s_seq) * 2, 128};
    const cuuint32_t box[5] = {64, static_cast<cuuint32_t>(kBN), 1, 1, panels};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(basep), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// (element, head in group, KV head, token of any sequence, panel) view of Q [batch][max_tt][Hq][D]:
// a box of 64 elements x G heads x 128/G tokens x all panels is one 128-row tile in (token, head)
// row order.  The sequences are folded into the token dimension (they are contiguous), so rows
// past a sequence's max_tt read the next sequence's; such rows are never valid.
bool make_q_map(CUtensorMap* map, const void* basep, int D, int G, int Hkv, int max_tt, int batch) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t Hq = static_cast<cuuint64_t>(G) * Hkv;
    const cuuint32_t panels = static_cast<cuuint32_t>(D / 64);
    const cuuint64_t dims[5] = {64, static_cast<cuuint64_t>(G), static_cast<cuuint64_t>(Hkv),
                                static_cast<cuuint64_t>(max_tt) * batch, panels};
    const cuuint64_t strides[4] = {static_cast<cuuint64_t>(D) * 2, static_cast<cuuint64_t>(G) * D * 2, Hq * D * 2, 128};
    const cuuint32_t box[5] = {64, static_cast<cuuint32_t>(G), 1, static_cast<cuuint32_t>(kBM / G), panels};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(basep), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor maps are kept per context, keyed by everything that goes into them: a decode loop calls
// with the same few buffers over and over, and encoding a map is a driver call.
struct MapKey {
    const void* base;
    int64_t a, b, c, d;  // K/V: token, head, sequence strides and capacity; Q: G, max_tt, 0, 0
    int hkv, batch, kind;  // kind 0: K/V cache, 1: Q
    bool operator==(const MapKey& o) const {
        return base == o.base && a == o.a && b == o.b && c == o.c && d == o.d && hkv == o.hkv && batch == o.batch &&
               kind == o.kind;
    }
};
struct MapKeyHash {
    size_t operator()(const MapKey& k) const {
        uint64_t h = reinterpret_cast<uintptr_t>(k.base) * 0x9E3779B97F4A7C15ull;
        h ^= (static_cast<uint64_t>(k.a) * 31 + k.b) * 0xBF58476D1CE4E5B9ull + k.c + k.d * 7 + k.batch * 131 + k.kind +
             k.hkv * 8191;
        return static_cast<size_t>(h ^ (h >> 29));
    }
};
struct HostState {
    std::mutex mu;
    std::unordered_map<MapKey, CUtensorMap, MapKeyHash> maps;
    // The work list in the workspace was made for these arguments ...
    bool plan_valid = false;
    const resps_step* plan_steps = nullptr;
    const int32_t* plan_n_nodes = nullptr;
    int plan_batch = 0;
    int64_t plan_capacity = 0;
    cudaStream_t plan_stream = nullptr;
    // ... and this many kernels of the library have been enqueued behind the one that wrote it.
    int plan_age = 0;
};
constexpr size_t kMaxCachedMaps = 4096;

HostState* host_state(const resps_ctx* ctx) { return static_cast<HostState*>(ctx->attn_host); }

const CUtensorMap* cached_map(HostState* hs, const MapKey& key, int D) {
    auto it = hs->maps.find(key);
    if (it != hs->maps.end()) return &it->second;
    CUtensorMap m;
    const bool ok = key.kind == 0 ? make_kv_map(&m, key.base, D, key.d, key.hkv, key.batch, key.a, key.b, key.c)
                                  : make_q_map(&m, key.base, D, static_cast<int>(key.a), key.hkv,
                                               static_cast<int>(key.b), key.batch);
    if (!ok) return nullptr;
    if (hs->maps.size() >= kMaxCachedMaps) hs->maps.clear();
    return &hs->maps.emplace(key, m).first->second;
}

template <int D>
cudaError_t launch_for_dim(const resps_ctx* ctx, const AttnArgs& a, const CUtensorMap& mk, const CUtensorMap& mv,
                           const CUtensorMap& mq, cudaStream_t st) {
    cudaError_t e = launch_pdl(tree_attention_kernel<D>, dim3(ctx->ws.attn_grid), dim3(kAttnThreads), Smem<D>::kBytes, st, a, mk,
                               mv, mq);
    if (e != cudaSuccess) return e;
    // One resident round of CTAs at most, and no more than the largest trees could use.  A single
    // sequence (or two) is served best by few, register-heavy threads that all start under the
    // attention kernel's tail; a batch by the flat index space and four CTAs per SM.
    const long long pieces = 1ll * a.max_tt * a.Hq * (D / 8);
    if (a.batch > 2) {
        const long long most = (4ll * a.batch * (pieces + 1) + kCombineThreads - 1) / kCombineThreads;
        const int grid = static_cast<int>(std::min<long long>(ctx->ws.attn_combine_flat_grid, std::max<long long>(most, 1)));
        return launch_pdl(attention_combine_flat_kernel<D>, dim3(grid), dim3(kCombineThreads), 0, st, a);
    }
    const int G = a.Hq / a.Hkv;
    if (a.max_tt * G <= kRowTiles * kBM) {
        const long long few = (a.batch * pieces + kCombineThreads - 1) / kCombineThreads;
        return launch_pdl(attention_combine_small_kernel<D>, dim3(static_cast<unsigned>(std::max<long long>(few, 1))),
                          dim3(kCombineThreads), 0, st, a);
    }
    // one CTA per (row tile, pair of column pieces) of the largest trees (CTAs past the trees at hand leave at once)
    const long long most = 1ll * a.batch * a.Hkv * ((a.max_tt * G + kBM - 1) / kBM) * (D / 8 / kCombPieces);
    return launch_pdl(attention_combine_kernel<D>, dim3(static_cast<unsigned>(std::max<long long>(most, 1))),
                      dim3(kCombineThreads), kCombChunk * kCombSlotBytes, st, a);
}

}  // namespace

cudaError_t attention_setup(resps_ctx* ctx) {
    ctx->attn_host = new (std::nothrow) HostState();
    if (!ctx->attn_host) return cudaErrorMemoryAllocation;
    cudaError_t e = cudaFuncSetAttribute(tree_attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         Smem<128>::kBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(tree_attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<64>::kBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attention_combine_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kCombChunk * kCombSlotBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attention_combine_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kCombChunk * kCombSlotBytes);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = (ctx->shape.head_dim == 128)
            ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, attention_combine_flat_kernel<128>, kCombineThreads, 0)
            : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, attention_combine_flat_kernel<64>, kCombineThreads, 0);
    if (e != cudaSuccess) return e;
    ctx->ws.attn_combine_flat_grid = ctx->sm_count * std::max(per_sm, 1);
    return cudaSuccess;
}

void attention_teardown(resps_ctx* ctx) {
    delete host_state(ctx);
    ctx->attn_host = nullptr;
}

// The step parameters or node counts behind `steps` may have changed (or the scheduling knobs
// have): the next attention call derives its work list anew.
void attention_plan_invalidate(resps_ctx* ctx, const void* steps_or_null) {
    HostState* hs = host_state(ctx);
    if (!hs) return;
    std::lock_guard<std::mutex> lock(hs->mu);
    if (steps_or_null == nullptr || steps_or_null == hs->plan_steps || steps_or_null == hs->plan_n_nodes)
        hs->plan_valid = false;
}

cudaError_t launch_tree_attention(const resps_ctx* ctx, const resps_step* d_steps,
                                  const int32_t* d_n_nodes, int batch, const __nv_bfloat16* q,
                                  __nv_bfloat16* o, float* lse, const __nv_bfloat16* k_cache,
                                  const __nv_bfloat16* v_cache, int64_t stride_seq,
                                  int64_t stride_head, int64_t stride_tok, int64_t capacity,
                                  const uint64_t* mask, float scale, cudaStream_t st) {
    AttnArgs a;
    a.steps = d_steps, a.n_nodes = d_n_nodes, a.batch = batch;
    a.q = q, a.o = o, a.lse = lse;
    a.capacity = capacity;
    a.mask = mask;
    a.scale_log2 = scale * 1.4426950408889634f;
    a.Hq = ctx->shape.n_q_heads, a.Hkv = ctx->shape.n_kv_heads, a.max_tt = ctx->shape.max_tt;
    a.part_o = reinterpret_cast<uint4*>(ctx->ws.attn_part_o), a.part_ml = ctx->ws.attn_part_ml;
    a.max_items = ctx->ws.attn_max_items, a.sched_grid = ctx->ws.attn_grid;
    a.min_tiles = ctx->ws.attn_min_tiles, a.status = ctx->ws.status;
    a.single_units = ctx->ws.attn_single;
    a.rounds = ctx->ws.attn_rounds;
    a.stagger = ctx->ws.attn_stagger;
    a.plan_head = reinterpret_cast<int4*>(ctx->ws.attn_plan);
    a.plan_seq = reinterpret_cast<PlanSeq*>(ctx->ws.attn_plan + 16);
    a.plan_item = reinterpret_cast<PlanItem*>(ctx->ws.attn_plan + 16 + sizeof(PlanSeq) * (ctx->shape.max_batch + 1));
    const int D = ctx->shape.head_dim;
    const int G = a.Hq / a.Hkv;
    a.q_by_tma = (G <= kBM && kBM % G == 0) ? 1 : 0;
    HostState* hs = host_state(ctx);
    std::lock_guard<std::mutex> lock(hs->mu);
    MapKey kk = {k_cache, stride_tok, stride_head, stride_seq, capacity, a.Hkv, batch, 0};
    MapKey kv = kk;
    kv.base = v_cache;
    const CUtensorMap* mk = cached_map(hs, kk, D);
    const CUtensorMap* mv = cached_map(hs, kv, D);
    if (!mk || !mv) return cudaErrorInvalidValue;
    const CUtensorMap* mq = mk;  // unused by the kernel unless Q comes by TMA
    if (a.q_by_tma) {
        MapKey kq = {q, G, a.max_tt, 0, 0, a.Hkv, batch, 1};
        mq = cached_map(hs, kq, D);
        if (!mq) return cudaErrorInvalidValue;
    }
    // The work list: made by the first call after anything that may have changed the step, reused
    // by the calls for the other layers.
    const bool reuse = hs->plan_valid && hs->plan_steps == d_steps && hs->plan_n_nodes == d_n_nodes &&
                       hs->plan_batch == batch && hs->plan_capacity == capacity && hs->plan_stream == st;
    if (!reuse) {
        cudaError_t e = launch_pdl(attention_plan_kernel, dim3(1), dim3(256), 0, st, a);
        if (e != cudaSuccess) return e;
        hs->plan_valid = true, hs->plan_steps = d_steps, hs->plan_n_nodes = d_n_nodes, hs->plan_batch = batch;
        hs->plan_capacity = capacity, hs->plan_stream = st, hs->plan_age = 0;
    }
    a.plan_after_wait = hs->plan_age == 0 ? 1 : 0;
    a.test_drop = ctx->ws.test_drop;
    cudaError_t e = D == 128 ? launch_for_dim<128>(ctx, a, *mk, *mv, *mq, st) : launch_for_dim<64>(ctx, a, *mk, *mv, *mq, st);
    hs->plan_age += 2;
    return e;
}

int attention_item_rows() { return kRowTiles * kBM; }
int attention_max_rounds() { return kMaxRounds; }
int attention_max_batch() { return kMaxBatchSmem; }
size_t attention_plan_bytes(int max_batch, int max_items) {
    return 16 + sizeof(PlanSeq) * (max_batch + 1) + sizeof(PlanItem) * static_cast<size_t>(max_items);
}

}  // namespace resps
