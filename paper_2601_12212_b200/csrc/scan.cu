// Vocabulary scans: fused top-k + log-sum-exp over draft rows (tree expansion,
// Section 3.2 "Draft Tree Expansion") and arg-max over target rows (greedy
// verification, Section 3.1).  Both are single-pass, HBM-bound streaming
// kernels: every logit is read exactly once with 128-bit coalesced loads.
//
// A row is cut into `splits` chunks, one CTA each.  A CTA reduces its chunk to a
// partial result in the context workspace; the last CTA of a row to arrive
// (atomic arrival counter, self-resetting) merges the partials and writes the
// row's final result, so no second launch is needed.
#include <cmath>
#include <mutex>

#include "common.cuh"

namespace resps {
namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr float kLog2e = 1.4426950408889634f;

struct ScanArgs {
    const resps_step* steps;
    const float* logits;
    int64_t ld_b, ld_level, ld_row;
    int n_levels, n_slots;
    int vocab, max_tt, max_k, max_rows;
    int chunk, splits;
    int slices, cps;  // streaming kernel: slices per row, chunks per slice (partials keep the stride `splits`)
    int test_drop;    // test build only: 2 = the second chunk copy of every slice is left out
    int only_level;   // -1: the rows of all levels; j >= 0: only level j's rows (blockIdx.y = slot)
    unsigned long long* part_key;
    float2* part_ms;
    unsigned int* counter;
    float* row_val;
    int32_t* row_id;
    double* row_lse;
    int32_t* status;
};

// Running (max, sum) of 2^(y - max) with y = x*log2(e).
struct LseAcc {
    float m2 = -INFINITY;
    float s = 0.f;
    __device__ __forceinline__ void merge(float om, float os) {
        const float M = fmaxf(m2, om);
        if (M == -INFINITY) return;
        s = s * ex2_approx(m2 - M) + os * ex2_approx(om - M);
        m2 = M;
    }
};

// rank-by-counting selection: the `k` largest of n keys in shared memory, written in order.
template <typename Out>
__device__ __forceinline__ void select_top_by_rank(const unsigned long long* keys, int n, int k, Out out) {
    for (int c = threadIdx.x; c < n; c += kScanThreads) {  // callers run it with kScanThreads threads
        const unsigned long long mine = keys[c];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (keys[j] > mine) || (keys[j] == mine && j < c);
        if (rank < k) out(rank, mine);
    }
}

constexpr int kScanPerThread = 32;                              // logits a thread keeps in registers
constexpr int kScanChunkMax = kScanThreads * kScanPerThread;    // 8192 per CTA
constexpr int kQuads = kScanThreads / 4;                        // units of 4 threads = 128 logits
constexpr int kQuadElems = 4 * kScanPerThread;

__device__ __forceinline__ float max3f(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// One CTA reduces one chunk (<= 8192 logits, all held in registers) of one row.
//  1. every quad of threads (128 logits) finds its best logit; the k-th best of the 64 quad
//     maxima, tau, is a lower bound for the chunk's k-th best logit;
//  2. every logit that ranks at or before tau is a candidate: they belong to the k quads whose
//     maximum does, so there are between k and 128 k of them (about 2 k for random data);
//  3. the candidates are ranked by counting and the k best written out.
// Keys are (ordered value, ~id) pairs, unique, so that "larger key" is exactly the method's order
// (value descending, token id ascending).  The log-sum-exp partial is a per-thread
// (max, sum 2^(y - max)) reduced over the CTA.
template <bool VEC>
__global__ void __launch_bounds__(kScanThreads, 4) row_scan_kernel(const ScanArgs a) {
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    extern __shared__ unsigned long long s_keys[];  // max(128 max_k, splits max_k) keys
    __shared__ unsigned long long s_quad[kQuads];
    __shared__ unsigned long long s_tau;
    __shared__ int s_count;
    __shared__ float2 s_ms[kScanThreads / 32];
    __shared__ bool s_last;
    const int b = blockIdx.z, ry = blockIdx.y, sp = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const StepDims sd = clamp_step(a.steps[b], a.n_levels, a.n_slots, a.max_tt, a.max_k, a.vocab);
    const int k = sd.k;
    const int rows = 1 + (sd.d - 1) * k;
    if (a.only_level >= 0 && ry >= (a.only_level == 0 ? 1 : k)) return;
    const int r = (a.only_level < 0) ? ry : (a.only_level == 0 ? 0 : 1 + (a.only_level - 1) * k + ry);
    if (r >= rows) return;
    if (sd.clamped && r == 0 && sp == 0 && tid == 0) atomicOr(a.status, RESPS_STATUS_STEP_CLAMPED);
    const int level = (r == 0) ? 0 : 1 + (r - 1) / k;
    const int slot = (r == 0) ? 0 : (r - 1) % k;
    const float* row = a.logits + b * a.ld_b + level * a.ld_level + slot * a.ld_row;
    const int begin = sp * a.chunk;
    const int end = min(a.vocab, begin + a.chunk);

    // ---- the chunk into registers: 8 independent 128-bit loads per thread ------------------
    float v[kScanPerThread];
#pragma unroll
    for (int u = 0; u < kScanPerThread / 4; ++u) {
        const int e0 = begin + (u * kScanThreads + tid) * 4;
        v[4 * u] = v[4 * u + 1] = v[4 * u + 2] = v[4 * u + 3] = -INFINITY;
        if (VEC) {
            if (e0 < end) {  // vocab and chunk are multiples of 4 on this path
                const float4 x = __ldcs(reinterpret_cast<const float4*>(row + e0));
                v[4 * u] = x.x, v[4 * u + 1] = x.y, v[4 * u + 2] = x.z, v[4 * u + 3] = x.w;
            }
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (e0 + c < end) v[4 * u + c] = __ldcs(row + e0 + c);
        }
    }
    if (tid == 0) s_count = 0;
    // position i of a thread is logit begin + ((i / 4) * 256 + tid) * 4 + i % 4: ids ascend with i
    auto elem_id = [&](int i) { return begin + ((i >> 2) * kScanThreads + tid) * 4 + (i & 3); };

    // ---- thread maximum and its first position ---------------------------------------------
    float tmax = v[0];
#pragma unroll
    for (int i = 1; i + 1 < kScanPerThread; i += 2) tmax = max3f(tmax, v[i], v[i + 1]);
    tmax = fmaxf(tmax, v[kScanPerThread - 1]);
    int tpos = 0;
#pragma unroll
    for (int i = kScanPerThread - 1; i >= 0; --i)
        if (v[i] == tmax) tpos = i;
    const bool has_any = elem_id(0) < end;  // a thread's positions are valid up to some i: 0 is valid or none
    const unsigned long long my_key = has_any ? pack_val_id(tmax, elem_id(tpos)) : 0ull;

    // ---- log-sum-exp partial (-inf padding adds 2^-inf = 0) ----------------------------------
    LseAcc acc;
    if (has_any) {
        acc.m2 = tmax * kLog2e;
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int i = 0; i < kScanPerThread; i += 2) {
            s0 += ex2_approx(fmaf(v[i], kLog2e, -acc.m2));
            s1 += ex2_approx(fmaf(v[i + 1], kLog2e, -acc.m2));
        }
        acc.s = s0 + s1;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(kFull, acc.m2, o);
        const float os = __shfl_xor_sync(kFull, acc.s, o);
        acc.merge(om, os);
    }
    if (lane == 0) s_ms[warp] = make_float2(acc.m2, acc.s);

    // ---- tau: the k-th best of the 64 quad maxima (0 = fewer than k non-empty quads) -----------
    unsigned long long quad_key = my_key;
    {
        unsigned long long o = __shfl_xor_sync(kFull, quad_key, 1);
        quad_key = o > quad_key ? o : quad_key;
        o = __shfl_xor_sync(kFull, quad_key, 2);
        quad_key = o > quad_key ? o : quad_key;
    }
    if ((lane & 3) == 0) s_quad[tid >> 2] = quad_key;
    __syncthreads();
    if (tid < kQuads) {
        const unsigned long long mine = s_quad[tid];
        int rank = 0;
#pragma unroll 8
        for (int j = 0; j < kQuads; ++j) {
            const unsigned long long o = s_quad[j];
            rank += (o > mine) || (o == mine && j < tid);  // equal keys are both 0 (empty)
        }
        if (rank == min(k, kQuads) - 1) s_tau = mine;
    }
    __syncthreads();
    // with k > 64 quads every non-empty quad qualifies; k <= RESPS_MAX_K = 32 keeps this exact
    const unsigned long long tau = s_tau;

    // ---- candidates: every logit at or before tau ------------------------------------------------
    if (quad_key >= tau && has_any) {  // only the k quads whose maximum qualifies can hold any
        const float tau_v = (tau == 0ull) ? -INFINITY : key_val(tau);
#pragma unroll
        for (int i = 0; i < kScanPerThread; ++i) {
            if (v[i] >= tau_v && elem_id(i) < end) {
                const unsigned long long key = pack_val_id(v[i], elem_id(i));
                if (key >= tau) s_keys[atomicAdd(&s_count, 1)] = key;
            }
        }
    }
    __syncthreads();
    const int n_cand = s_count;  // <= 128 k
    const int64_t prow = static_cast<int64_t>(b) * a.max_rows + r;
    unsigned long long* part = a.part_key + (prow * a.splits + sp) * a.max_k;
    select_top_by_rank(s_keys, n_cand, k, [&](int rank, unsigned long long key) { part[rank] = key; });
    if (tid >= n_cand && tid < k) part[tid] = 0ull;  // fewer than k logits in the chunk
    if (tid == 0) {
        LseAcc t;
        for (int w = 0; w < kScanThreads / 32; ++w) t.merge(s_ms[w].x, s_ms[w].y);
        a.part_ms[prow * a.splits + sp] = make_float2(t.m2, t.s);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(a.counter + prow, 1u) == static_cast<unsigned>(a.splits - 1));
    __syncthreads();
    if (!s_last) return;

    // ---- last CTA of the row: merge the partial lists and the partial sums ----
    __threadfence();
    const unsigned long long* parts = a.part_key + prow * a.splits * a.max_k;
    for (int i = tid; i < a.splits * k; i += kScanThreads)
        s_keys[i] = __ldcg(parts + (i / k) * a.max_k + (i % k));
    float2 my_ms = make_float2(-INFINITY, 0.f);
    if (tid < a.splits) my_ms = __ldcg(a.part_ms + prow * a.splits + tid);  // splits <= 128 < threads
    __syncthreads();
    float* oval = a.row_val + prow * a.max_k;
    int32_t* oid = a.row_id + prow * a.max_k;
    select_top_by_rank(s_keys, a.splits * k, k, [&](int rank, unsigned long long key) {
        oval[rank] = key_val(key);
        oid[rank] = key_id(key);
    });
    if (warp < 4) {  // partial sums: weights in fp32 (relative error 2^-22), accumulation in fp64
        float M = my_ms.x;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFull, M, o));
        if (lane == 0) s_ms[warp] = make_float2(M, 0.f);
    }
    __syncthreads();
    if (warp < 4) {
        const float M = fmaxf(fmaxf(s_ms[0].x, s_ms[1].x), fmaxf(s_ms[2].x, s_ms[3].x));
        double sum = (my_ms.y > 0.f) ? static_cast<double>(my_ms.y) * static_cast<double>(ex2_approx(my_ms.x - M)) : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(kFull, sum, o);
        if (lane == 0) s_quad[warp] = __double_as_longlong(sum);
    }
    __syncthreads();
    if (tid == 0) {
        const float M = fmaxf(fmaxf(s_ms[0].x, s_ms[1].x), fmaxf(s_ms[2].x, s_ms[3].x));
        const double sum = __longlong_as_double(s_quad[0]) + __longlong_as_double(s_quad[1]) +
                           __longlong_as_double(s_quad[2]) + __longlong_as_double(s_quad[3]);
        a.row_lse[prow] = (static_cast<double>(M) + log2(sum)) * 0.6931471805599453094;
        a.counter[prow] = 0u;
    }
}

// ---------------------------------------------------------------------------------------
// Streaming variant (16-byte aligned rows): a CTA walks a slice of several chunks of one row.
// One thread issues bulk copies (cp.async.bulk, global -> shared, completion on an mbarrier)
// three chunks ahead, so the loads of the next chunks run under the arithmetic of the current
// one.  The first chunk establishes the threshold tau as above; afterwards tau is the k-th best
// logit seen so far, a chunk contributes only the (few) logits at or above it, and the list is
// cut back to its k best when it has grown.  The log-sum-exp state stays in registers across
// chunks.  A chunk whose hits would not fit the list (adversarial order) re-derives a threshold
// of its own from its quad maxima, which bounds its candidates by 128 k.
// ---------------------------------------------------------------------------------------
constexpr int kStreamStages = 3;
constexpr long long kScanWaitLimitCycles = kWaitTest ? 2000000ll : 4000000000ll;

__device__ __forceinline__ uint32_t scan_smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ bool scan_mbar_try(uint32_t bar, uint32_t parity) {
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
// Bounded: on expiry the status word is flagged and the caller goes on (its results are then
// meaningless, but every counter protocol still completes).
__device__ __forceinline__ void scan_mbar_wait(uint32_t bar, uint32_t parity, int32_t* status) {
    if (scan_mbar_try(bar, parity)) return;
    const long long t0 = clock64();
    unsigned spins = 0;
    while (!scan_mbar_try(bar, parity)) {
        if ((++spins & 63u) == 0u && clock64() - t0 > kScanWaitLimitCycles) {
            if (status) atomicOr(status, RESPS_STATUS_WAIT_TIMEOUT);
            return;
        }
    }
}

constexpr int kStreamThreads = kScanThreads + 32;  // eight consumer warps + the copy-issuing warp

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ bool consumer_any(bool pred) {  // barrier over the consumers, OR of pred
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, 256, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"(pred ? 1u : 0u)
        : "memory");
    return out != 0;
}

__global__ void __launch_bounds__(kStreamThreads, 2) row_scan_stream_kernel(const ScanArgs a) {
    extern __shared__ __align__(128) unsigned char s_raw[];
    float* s_stage = reinterpret_cast<float*>(s_raw);                                    // [3][8192]
    unsigned long long* s_keys =
        reinterpret_cast<unsigned long long*>(s_raw + kStreamStages * kScanChunkMax * sizeof(float));  // list
    __shared__ __align__(8) unsigned long long s_bar[2 * kStreamStages];  // full[3], empty[3]
    __shared__ unsigned long long s_quad[kQuads];
    __shared__ unsigned long long s_top[RESPS_MAX_K];
    __shared__ unsigned long long s_tau;
    __shared__ int s_count;
    __shared__ float2 s_ms[kScanThreads / 32];
    __shared__ bool s_last;
    const int b = blockIdx.z, ry = blockIdx.y, sl = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t bar0 = scan_smem_u32(s_bar);
    auto full_bar = [&](int st) { return bar0 + 8u * st; };
    auto empty_bar = [&](int st) { return bar0 + 8u * (kStreamStages + st); };
    // the barriers are set up under the tail of the preceding kernel: nothing here touches global memory
    if (tid == 0) {
        for (int st = 0; st < kStreamStages; ++st) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(full_bar(st)) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty_bar(st)), "r"(kScanThreads) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        s_count = 0;
        s_tau = 0ull;
    }
    __syncthreads();
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    const StepDims sd = clamp_step(a.steps[b], a.n_levels, a.n_slots, a.max_tt, a.max_k, a.vocab);
    const int k = sd.k;
    const int rows = 1 + (sd.d - 1) * k;
    if (a.only_level >= 0 && ry >= (a.only_level == 0 ? 1 : k)) return;
    const int r = (a.only_level < 0) ? ry : (a.only_level == 0 ? 0 : 1 + (a.only_level - 1) * k + ry);
    if (r >= rows) return;
    if (sd.clamped && r == 0 && sl == 0 && tid == 0) atomicOr(a.status, RESPS_STATUS_STEP_CLAMPED);
    const int level = (r == 0) ? 0 : 1 + (r - 1) / k;
    const int slot = (r == 0) ? 0 : (r - 1) % k;
    const float* row = a.logits + b * a.ld_b + level * a.ld_level + slot * a.ld_row;
    const int c_begin = sl * a.cps;
    const int c_end = min(a.splits, c_begin + a.cps);  // chunks [c_begin, c_end) of this row
    const int list_cap = (kQuadElems + 1) * a.max_k;

    if (warp == kScanThreads / 32) {
        // ---- copy-issuing warp: a stage is refilled as soon as every consumer has read it ----------
        if (lane == 0) {
            for (int c = c_begin; c < c_end; ++c) {
                const int u = c - c_begin, st = u % kStreamStages;
                scan_mbar_wait(empty_bar(st), ((u / kStreamStages) & 1u) ^ 1u, a.status);
                const int e0 = c * kScanChunkMax;
                const uint32_t bytes = static_cast<uint32_t>(min(a.vocab - e0, kScanChunkMax)) * 4u;
                if (kWaitTest && (a.test_drop & 2) && u == 1) continue;
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full_bar(st)), "r"(bytes)
                             : "memory");
                asm volatile(
                    "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                        scan_smem_u32(s_stage + st * kScanChunkMax)),
                    "l"(row + e0), "r"(bytes), "r"(full_bar(st))
                    : "memory");
            }
        }
        return;  // the consumers wait for every copy that was issued
    }

    int list_n = 0;                // entries of the candidate list (same in every thread)
    LseAcc acc;                    // this thread's running (max, sum) over all its logits
    unsigned long long tau = 0ull; // k-th best so far (0 = none yet: everything qualifies)
    float tau_v = -INFINITY;

    for (int c = c_begin; c < c_end; ++c) {
        const int u0 = c - c_begin, st = u0 % kStreamStages;
        const int begin = c * kScanChunkMax;
        const int end = min(a.vocab, begin + kScanChunkMax);
        scan_mbar_wait(full_bar(st), (u0 / kStreamStages) & 1u, a.status);
        float v[kScanPerThread];
#pragma unroll
        for (int u = 0; u < kScanPerThread / 4; ++u) {
            const int off = (u * kScanThreads + tid) * 4;
            v[4 * u] = v[4 * u + 1] = v[4 * u + 2] = v[4 * u + 3] = -INFINITY;
            if (begin + off < end) {  // the vocabulary is a multiple of 4 on this path
                const float4 x = *reinterpret_cast<const float4*>(s_stage + st * kScanChunkMax + off);
                v[4 * u] = x.x, v[4 * u + 1] = x.y, v[4 * u + 2] = x.z, v[4 * u + 3] = x.w;
            }
        }
        auto release_stage = [&]() {
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar(st)) : "memory");
        };
        auto elem_id = [&](int i) { return begin + ((i >> 2) * kScanThreads + tid) * 4 + (i & 3); };
        const bool has_any = elem_id(0) < end;

        // ---- thread maximum, log-sum-exp update ---------------------------------------------------
        float tmax = v[0];
#pragma unroll
        for (int i = 1; i + 1 < kScanPerThread; i += 2) tmax = max3f(tmax, v[i], v[i + 1]);
        tmax = fmaxf(tmax, v[kScanPerThread - 1]);
        if (has_any) {
            const float m_new = fmaxf(acc.m2, tmax * kLog2e);
            float s0 = acc.s * ex2_approx(acc.m2 - m_new), s1 = 0.f;  // 0 * 2^-inf = 0 on the first chunk
#pragma unroll
            for (int i = 0; i < kScanPerThread; i += 2) {
                s0 += ex2_approx(fmaf(v[i], kLog2e, -m_new));
                s1 += ex2_approx(fmaf(v[i + 1], kLog2e, -m_new));
            }
            acc.m2 = m_new, acc.s = s0 + s1;
        }
        const bool first = (c == c_begin);
        // One barrier per chunk in the common case: does any thread hold a logit at or above tau?
        // (branch-free bit mask; the few hits are then re-read from the stage by index)
        uint32_t hits = 0u;
        if (!first) {
            if (tmax >= tau_v) {  // only a thread whose best logit qualifies has anything to mark
#pragma unroll
                for (int i = 0; i < kScanPerThread; ++i) hits |= (v[i] >= tau_v) ? (1u << i) : 0u;
            }
            if (!consumer_any(hits != 0u)) {
                release_stage();
                continue;
            }
        }

        // Threads that hold such logits append them to the list.  Should the list overflow
        // (adversarial order: every logit beats the threshold), the appended entries are dropped
        // and the chunk takes the bounded path below.
        bool slow = first;
        if (!first) {
            const float* stage = s_stage + st * kScanChunkMax;
            while (hits) {
                const int i = __ffs(hits) - 1;
                hits &= hits - 1u;
                const int e = elem_id(i);
                if (e < end) {
                    const unsigned long long key = pack_val_id(stage[e - begin], e);
                    if (key >= tau) {
                        const int at = atomicAdd(&s_count, 1);
                        if (at < list_cap) s_keys[at] = key;
                    }
                }
            }
            consumer_sync();
            slow = s_count > list_cap;  // fixed until the next barrier
        }
        release_stage();
        if (slow) {
            // the chunk's own threshold from its quad maxima (see row_scan_kernel); the list is cut
            // to its k best first so that the chunk's at most 128 k candidates fit behind them
            if (!first) {  // the first list_n entries are the list as it was before this chunk
                for (int cidx = tid; cidx < list_n; cidx += kScanThreads) {
                    const unsigned long long mine = s_keys[cidx];
                    int rank = 0;
                    for (int j = 0; j < list_n; ++j) rank += (s_keys[j] > mine) ? 1 : 0;
                    if (rank < k) s_top[rank] = mine;
                }
                consumer_sync();
                const int nk = min(list_n, k);
                if (tid < nk) s_keys[tid] = s_top[tid];
                if (tid == 0) s_count = nk;
                consumer_sync();
            }
            int tpos = 0;
#pragma unroll
            for (int i = kScanPerThread - 1; i >= 0; --i)
                if (v[i] == tmax) tpos = i;
            const unsigned long long my_key = has_any ? pack_val_id(tmax, elem_id(tpos)) : 0ull;
            unsigned long long quad_key = my_key;
            {
                unsigned long long o = __shfl_xor_sync(kFull, quad_key, 1);
                quad_key = o > quad_key ? o : quad_key;
                o = __shfl_xor_sync(kFull, quad_key, 2);
                quad_key = o > quad_key ? o : quad_key;
            }
            if ((lane & 3) == 0) s_quad[tid >> 2] = quad_key;
            consumer_sync();
            if (tid < kQuads) {
                const unsigned long long mine = s_quad[tid];
                int rank = 0;
#pragma unroll 8
                for (int j = 0; j < kQuads; ++j) {
                    const unsigned long long o = s_quad[j];
                    rank += (o > mine) || (o == mine && j < tid);
                }
                if (rank == min(k, kQuads) - 1) s_tau = mine;
            }
            consumer_sync();
            const unsigned long long tau_c = s_tau > tau ? s_tau : tau;  // never below the running one
            if (quad_key >= tau_c && has_any) {
                const float tv = (tau_c == 0ull) ? -INFINITY : key_val(tau_c);
#pragma unroll
                for (int i = 0; i < kScanPerThread; ++i)
                    if (v[i] >= tv && elem_id(i) < end) {
                        const unsigned long long key = pack_val_id(v[i], elem_id(i));
                        if (key >= tau_c) s_keys[atomicAdd(&s_count, 1)] = key;
                    }
            }
        }
        consumer_sync();
        // ---- tighten: tau = k-th best of the list; cut the list back when it has grown ----------
        const int n_list = s_count;
        list_n = n_list;
        if (slow || n_list > 8 * k) {
            for (int cidx = tid; cidx < n_list; cidx += kScanThreads) {
                const unsigned long long mine = s_keys[cidx];
                int rank = 0;
                for (int j = 0; j < n_list; ++j) rank += (s_keys[j] > mine) ? 1 : 0;
                if (rank < k) s_top[rank] = mine;
            }
            consumer_sync();
            const int nk = min(n_list, k);
            if (tid < nk) s_keys[tid] = s_top[tid];
            if (tid == 0) {
                s_count = nk;
                s_tau = (n_list >= k) ? s_top[k - 1] : 0ull;
            }
            consumer_sync();
            tau = s_tau;
            tau_v = (tau == 0ull) ? -INFINITY : key_val(tau);
            list_n = nk;
        }
    }

    // ---- the slice's k best and its log-sum-exp partial ------------------------------------------
    consumer_sync();
    const int n_cand = s_count;
    const int64_t prow = static_cast<int64_t>(b) * a.max_rows + r;
    unsigned long long* part = a.part_key + (prow * a.splits + sl) * a.max_k;
    select_top_by_rank(s_keys, n_cand, k, [&](int rank, unsigned long long key) { part[rank] = key; });
    if (tid >= n_cand && tid < k) part[tid] = 0ull;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(kFull, acc.m2, o);
        const float os = __shfl_xor_sync(kFull, acc.s, o);
        acc.merge(om, os);
    }
    if (lane == 0) s_ms[warp] = make_float2(acc.m2, acc.s);
    consumer_sync();
    if (tid == 0) {
        LseAcc t;
        for (int w = 0; w < kScanThreads / 32; ++w) t.merge(s_ms[w].x, s_ms[w].y);
        a.part_ms[prow * a.splits + sl] = make_float2(t.m2, t.s);
    }
    __threadfence();
    consumer_sync();
    if (tid == 0) s_last = (atomicAdd(a.counter + prow, 1u) == static_cast<unsigned>(a.slices - 1));
    consumer_sync();
    if (!s_last) return;

    // ---- last CTA of the row: merge the slices ---------------------------------------------------
    __threadfence();
    const unsigned long long* parts = a.part_key + prow * a.splits * a.max_k;
    for (int i = tid; i < a.slices * k; i += kScanThreads) s_keys[i] = __ldcg(parts + (i / k) * a.max_k + (i % k));
    float2 my_ms = make_float2(-INFINITY, 0.f);
    if (tid < a.slices) my_ms = __ldcg(a.part_ms + prow * a.splits + tid);
    consumer_sync();
    float* oval = a.row_val + prow * a.max_k;
    int32_t* oid = a.row_id + prow * a.max_k;
    select_top_by_rank(s_keys, a.slices * k, k, [&](int rank, unsigned long long key) {
        oval[rank] = key_val(key);
        oid[rank] = key_id(key);
    });
    if (warp < 4) {
        float M = my_ms.x;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFull, M, o));
        if (lane == 0) s_ms[warp] = make_float2(M, 0.f);
    }
    consumer_sync();
    if (warp < 4) {
        const float M = fmaxf(fmaxf(s_ms[0].x, s_ms[1].x), fmaxf(s_ms[2].x, s_ms[3].x));
        double sum = (my_ms.y > 0.f) ? static_cast<double>(my_ms.y) * static_cast<double>(ex2_approx(my_ms.x - M)) : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(kFull, sum, o);
        if (lane == 0) s_quad[warp] = __double_as_longlong(sum);
    }
    consumer_sync();
    if (tid == 0) {
        const float M = fmaxf(fmaxf(s_ms[0].x, s_ms[1].x), fmaxf(s_ms[2].x, s_ms[3].x));
        const double sum = __longlong_as_double(s_quad[0]) + __longlong_as_double(s_quad[1]) +
                           __longlong_as_double(s_quad[2]) + __longlong_as_double(s_quad[3]);
        a.row_lse[prow] = (static_cast<double>(M) + log2(sum)) * 0.6931471805599453094;
        a.counter[prow] = 0u;
    }
}

struct ArgmaxArgs {
    const int32_t* n_nodes;
    const float* logits;
    int64_t ld_b, ld_row;
    int vocab, max_tt, chunk, splits;
    int slices, cps;  // streaming kernel: slices per row, chunks per slice (partials keep the stride `splits`)
    unsigned long long* part;
    unsigned int* counter;
    unsigned int* seq_counter;  // streaming kernel: CTAs of a sequence that have delivered their slice
    int32_t* out;
    unsigned long long* key_out;  // optional [batch][max_tt]: the packed (value, id) of every row's arg-max
    int32_t* status;            // streaming kernel: where a wait that ran out is flagged (may be null)
};

// Streaming arg-max (16-byte aligned rows): like the streaming scan, a CTA walks a slice of several
// 8192-logit chunks of one row behind a copy-issuing warp (cp.async.bulk three chunks ahead), a thread
// keeps 32 logits of the chunk in registers and its best (ordered value, ~id) key across chunks.  The
// last CTA of a sequence to deliver its slice merges the slices of all rows and goes on to the
// acceptance walk (Section 3.2, "Acceptance Criterion" at temperature 0) when the caller asked for
// it, so that arg-max and walk are one kernel.
__global__ void __launch_bounds__(kStreamThreads, 2) row_argmax_stream_kernel(const ArgmaxArgs a, const AcceptArgs w,
                                                                               const int do_walk) {
    extern __shared__ __align__(128) unsigned char s_raw[];
    float* s_stage = reinterpret_cast<float*>(s_raw);  // [3][8192]
    __shared__ __align__(8) unsigned long long s_bar[2 * kStreamStages];  // full[3], empty[3]
    __shared__ unsigned long long s_k[kScanThreads / 32];
    __shared__ int s_flag;
    __shared__ int s_tgt[RESPS_MAX_TT];
    __shared__ int s_next[RESPS_MAX_DEPTH];
    const int b = blockIdx.z, r = blockIdx.y, sl = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t bar0 = scan_smem_u32(s_bar);
    auto full_bar = [&](int st) { return bar0 + 8u * st; };
    auto empty_bar = [&](int st) { return bar0 + 8u * (kStreamStages + st); };
    // the barriers are set up under the tail of the preceding kernel: nothing here touches global memory
    if (tid == 0) {
        for (int st = 0; st < kStreamStages; ++st) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(full_bar(st)) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty_bar(st)), "r"(kScanThreads) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    const int n = min(max(a.n_nodes[b], 0), a.max_tt);
    if (r >= n) return;
    const float* row = a.logits + b * a.ld_b + r * a.ld_row;
    const int c_begin = sl * a.cps;
    const int c_end = min(a.splits, c_begin + a.cps);  // chunks [c_begin, c_end) of this row

    if (warp == kScanThreads / 32) {
        // ---- copy-issuing warp: a stage is refilled as soon as every consumer has read it ----------
        if (lane == 0) {
            for (int c = c_begin; c < c_end; ++c) {
                const int u = c - c_begin, st = u % kStreamStages;
                scan_mbar_wait(empty_bar(st), ((u / kStreamStages) & 1u) ^ 1u, a.status);
                const int e0 = c * kScanChunkMax;
                const uint32_t bytes = static_cast<uint32_t>(min(a.vocab - e0, kScanChunkMax)) * 4u;
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full_bar(st)), "r"(bytes)
                             : "memory");
                asm volatile(
                    "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                        scan_smem_u32(s_stage + st * kScanChunkMax)),
                    "l"(row + e0), "r"(bytes), "r"(full_bar(st))
                    : "memory");
            }
        }
        return;  // the consumers wait for every copy that was issued
    }

    unsigned long long best = 0ull;  // 0 = nothing yet (every real key has a non-zero value part)
    for (int c = c_begin; c < c_end; ++c) {
        const int u0 = c - c_begin, st = u0 % kStreamStages;
        const int begin = c * kScanChunkMax;
        const int end = min(a.vocab, begin + kScanChunkMax);
        scan_mbar_wait(full_bar(st), (u0 / kStreamStages) & 1u, a.status);
        float v[kScanPerThread];
#pragma unroll
        for (int u = 0; u < kScanPerThread / 4; ++u) {
            const int off = (u * kScanThreads + tid) * 4;
            v[4 * u] = v[4 * u + 1] = v[4 * u + 2] = v[4 * u + 3] = -INFINITY;
            if (begin + off < end) {  // the vocabulary is a multiple of 4 on this path
                const float4 x = *reinterpret_cast<const float4*>(s_stage + st * kScanChunkMax + off);
                v[4 * u] = x.x, v[4 * u + 1] = x.y, v[4 * u + 2] = x.z, v[4 * u + 3] = x.w;
            }
        }
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar(st)) : "memory");
        // position i of a thread is logit begin + ((i / 4) * 256 + tid) * 4 + i % 4: ids ascend with i
        if (begin + tid * 4 < end) {
            float tmax = v[0];
#pragma unroll
            for (int i = 1; i + 1 < kScanPerThread; i += 2) tmax = max3f(tmax, v[i], v[i + 1]);
            tmax = fmaxf(tmax, v[kScanPerThread - 1]);
            int tpos = 0;
#pragma unroll
            for (int i = kScanPerThread - 1; i >= 0; --i)
                if (v[i] == tmax) tpos = i;
            const unsigned long long key = pack_val_id(tmax, begin + ((tpos >> 2) * kScanThreads + tid) * 4 + (tpos & 3));
            best = key > best ? key : best;  // an equal value later in the row has a higher id: a smaller key
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(kFull, best, o);
        best = (other > best) ? other : best;
    }
    if (lane == 0) s_k[warp] = best;
    consumer_sync();
    const int64_t prow = static_cast<int64_t>(b) * a.max_tt + r;
    const int64_t ob = static_cast<int64_t>(b) * a.max_tt;
    // ---- a row in one slice and no walk: the CTA's result is the row's -------------------------------
    if (a.slices == 1 && !do_walk) {
        if (tid == 0) {
            for (int wq = 1; wq < kScanThreads / 32; ++wq) best = (s_k[wq] > best) ? s_k[wq] : best;
            a.out[prow] = key_id(best);
            if (a.key_out) a.key_out[prow] = best;
        }
        return;
    }
    // ---- otherwise the last CTA of the whole sequence to arrive merges the slices of every row (one
    // counter per sequence: one fence and one atomic on every CTA's way out) and, when asked, goes
    // on to the acceptance walk with the targets already in shared memory ---------------------------
    if (tid == 0) {
        for (int wq = 1; wq < kScanThreads / 32; ++wq) best = (s_k[wq] > best) ? s_k[wq] : best;
        a.part[prow * a.splits + sl] = best;
        __threadfence();
        const unsigned arrivals = static_cast<unsigned>(n) * static_cast<unsigned>(a.slices);
        const int last = (atomicAdd(a.seq_counter + b, 1u) == arrivals - 1u);
        if (last) a.seq_counter[b] = 0u;
        s_flag = last;
    }
    consumer_sync();
    if (!s_flag) return;
    __threadfence();
    for (int t = tid; t < n; t += kScanThreads) {
        unsigned long long top = 0ull;
        for (int i = 0; i < a.slices; ++i) {
            const unsigned long long p = __ldcg(a.part + (ob + t) * a.splits + i);
            top = (p > top) ? p : top;
        }
        a.out[ob + t] = key_id(top);
        if (a.key_out) a.key_out[ob + t] = top;
        if (t < RESPS_MAX_TT) s_tgt[t] = key_id(top);
    }
    if (!do_walk) return;
    // (the walk's first barrier orders s_tgt; Section 3.2, "Acceptance Criterion" at temperature 0)
    accept_walk_device(w, b, tid, s_tgt, s_next, true, [] { consumer_sync(); });
}

template <bool VEC>
__global__ void __launch_bounds__(kScanThreads, 4) row_argmax_kernel(const ArgmaxArgs a) {
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    const int b = blockIdx.z, r = blockIdx.y, sp = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = min(max(a.n_nodes[b], 0), a.max_tt);
    if (r >= n) return;
    const float* row = a.logits + b * a.ld_b + r * a.ld_row;
    const int begin = sp * a.chunk;
    const int end = min(a.vocab, begin + a.chunk);

    float best = -INFINITY;
    int best_id = 0x7FFFFFFF;
    constexpr int kUnroll = 8;
    for (int base = begin; base < end; base += kScanThreads * 4 * kUnroll) {
        float v[kUnroll][4];
        int nv[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int e0 = base + (u * kScanThreads + tid) * 4;
            nv[u] = max(0, min(4, end - e0));
            if (VEC) {
                if (nv[u] > 0) {
                    const float4 x = __ldcs(reinterpret_cast<const float4*>(row + e0));
                    v[u][0] = x.x, v[u][1] = x.y, v[u][2] = x.z, v[u][3] = x.w;
                }
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (c < nv[u]) v[u][c] = __ldcs(row + e0 + c);
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int e0 = base + (u * kScanThreads + tid) * 4;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (c < nv[u] && (v[u][c] > best || best_id == 0x7FFFFFFF)) {
                    best = v[u][c];
                    best_id = e0 + c;
                }
        }
    }
    unsigned long long key = (best_id == 0x7FFFFFFF) ? 0ull : pack_val_id(best, best_id);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(kFull, key, o);
        key = (other > key) ? other : key;
    }
    __shared__ unsigned long long s_k[kScanThreads / 32];
    __shared__ bool s_last;
    if (lane == 0) s_k[warp] = key;
    __syncthreads();
    const int64_t prow = static_cast<int64_t>(b) * a.max_tt + r;
    if (tid == 0) {
        for (int w = 1; w < kScanThreads / 32; ++w) key = (s_k[w] > key) ? s_k[w] : key;
        if (a.splits == 1) {
            a.out[prow] = key_id(key);
            if (a.key_out) a.key_out[prow] = key;
            s_last = false;
        } else {
            a.part[prow * a.splits + sp] = key;
            __threadfence();
            s_last = (atomicAdd(a.counter + prow, 1u) == static_cast<unsigned>(a.splits - 1));
        }
    }
    __syncthreads();
    if (!s_last || warp != 0) return;
    __threadfence();
    unsigned long long m = 0ull;
    for (int i = lane; i < a.splits; i += 32) {
        const unsigned long long p = __ldcg(a.part + prow * a.splits + i);
        m = (p > m) ? p : m;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(kFull, m, o);
        m = (other > m) ? other : m;
    }
    if (lane == 0) {
        a.out[prow] = key_id(m);
        if (a.key_out) a.key_out[prow] = m;
        a.counter[prow] = 0u;
    }
}

// ---------------------------------------------------------------------------------------
// Vocabulary sharded over several GPUs: every rank scans its own columns of every row with the
// kernels above (its context is created with its shard's width), the ranks exchange what they
// found -- k (value, id) pairs and one log-sum-exp per draft row, one (value, id) per target row --
// and every rank merges the shards' results with these two kernels.  Ids become global by the
// shard's first column; the order (value descending, id ascending) is the method's.
// ---------------------------------------------------------------------------------------
struct ShardMergeArgs {
    const resps_step* steps;
    int n_levels, n_slots, vocab, max_tt, max_k, max_rows, n_shards, batch;
    const float* all_val;      // [n_shards][batch][max_rows][max_k]
    const int32_t* all_id;
    const double* all_lse;     // [n_shards][batch][max_rows]
    const int32_t* shard_offset;  // [n_shards]
    float* row_val;
    int32_t* row_id;
    double* row_lse;
};

__global__ void __launch_bounds__(128) shard_merge_rows_kernel(const ShardMergeArgs a) {
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    __shared__ unsigned long long s_keys[16 * RESPS_MAX_K];
    const int b = blockIdx.y, r = blockIdx.x, tid = threadIdx.x;
    const StepDims sd = clamp_step(a.steps[b], a.n_levels, a.n_slots, a.max_tt, a.max_k, a.vocab);
    const int k = sd.k;
    if (r >= 1 + (sd.d - 1) * k) return;
    const int64_t prow = static_cast<int64_t>(b) * a.max_rows + r;
    const int n = a.n_shards * k;
    for (int i = tid; i < n; i += blockDim.x) {
        const int p = i / k, q = i - p * k;
        const int64_t src = (static_cast<int64_t>(p) * a.batch * a.max_rows + prow) * a.max_k + q;
        s_keys[i] = pack_val_id(a.all_val[src], a.all_id[src] + a.shard_offset[p]);
    }
    __syncthreads();
    for (int c = tid; c < n; c += blockDim.x) {
        const unsigned long long mine = s_keys[c];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (s_keys[j] > mine) || (s_keys[j] == mine && j < c);
        if (rank < k) {
            a.row_val[prow * a.max_k + rank] = key_val(mine);
            a.row_id[prow * a.max_k + rank] = key_id(mine);
        }
    }
    if (tid == 0) {  // log of the sum over the shards of exp(shard's log-sum-exp), fp64
        double m = -INFINITY;
        for (int p = 0; p < a.n_shards; ++p) m = fmax(m, a.all_lse[static_cast<int64_t>(p) * a.batch * a.max_rows + prow]);
        double sum = 0.0;
        for (int p = 0; p < a.n_shards; ++p) sum += exp(a.all_lse[static_cast<int64_t>(p) * a.batch * a.max_rows + prow] - m);
        a.row_lse[prow] = m + log(sum);
    }
}

struct ShardArgmaxArgs {
    const int32_t* n_nodes;
    int max_tt, n_shards, batch;
    const unsigned long long* all_key;  // [n_shards][batch][max_tt] packed (value, local id)
    const int32_t* shard_offset;
    int32_t* out;
};

__global__ void __launch_bounds__(RESPS_MAX_TT) shard_merge_argmax_kernel(const ShardArgmaxArgs a) {
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    const int b = blockIdx.x, i = threadIdx.x;
    const int n = min(max(a.n_nodes[b], 0), a.max_tt);
    if (i >= n) return;
    unsigned long long best = 0ull;
    for (int p = 0; p < a.n_shards; ++p) {
        const unsigned long long key = a.all_key[(static_cast<int64_t>(p) * a.batch + b) * a.max_tt + i];
        const unsigned long long global = pack_val_id(key_val(key), key_id(key) + a.shard_offset[p]);
        best = global > best ? global : best;
    }
    a.out[static_cast<int64_t>(b) * a.max_tt + i] = key_id(best);
}

inline bool vec_ok(const void* p, int64_t s0, int64_t s1, int64_t s2, int vocab, int chunk) {
    return (reinterpret_cast<uintptr_t>(p) % 16 == 0) && s0 % 4 == 0 && s1 % 4 == 0 && s2 % 4 == 0 &&
           vocab % 4 == 0 && chunk % 4 == 0;
}

}  // namespace

int scan_chunk_max() { return kScanChunkMax; }

static size_t stream_smem_bytes(int max_k, int slices) {
    return kStreamStages * kScanChunkMax * sizeof(float) +
           sizeof(unsigned long long) * max((kQuadElems + 1) * max_k, slices * max_k);
}

cudaError_t scan_setup(resps_ctx* ctx) {
    cudaError_t e = cudaFuncSetAttribute(row_argmax_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kStreamStages * kScanChunkMax * sizeof(float)));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(row_scan_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                static_cast<int>(stream_smem_bytes(ctx->shape.max_k, 128)));
}

cudaError_t launch_row_scan(const resps_ctx* ctx, const resps_step* d_steps, int batch,
                            const float* logits, int64_t ld_b, int64_t ld_level, int64_t ld_row,
                            int n_levels, int n_slots, int only_level, cudaStream_t st) {
    const Workspace& w = ctx->ws;
    ScanArgs a;
    a.steps = d_steps;
    a.logits = logits;
    a.ld_b = ld_b, a.ld_level = ld_level, a.ld_row = ld_row;
    a.n_levels = n_levels, a.n_slots = n_slots;
    a.vocab = ctx->shape.vocab, a.max_tt = ctx->shape.max_tt, a.max_k = ctx->shape.max_k;
    a.max_rows = w.max_rows, a.chunk = w.scan_chunk, a.splits = w.scan_splits;
    a.part_key = w.part_key, a.part_ms = w.part_ms, a.counter = w.row_counter;
    a.row_val = w.row_val, a.row_id = w.row_id, a.row_lse = w.row_lse, a.status = w.status;
    const int k_ext = min(n_slots, ctx->shape.max_k);
    a.only_level = only_level;
    const int rows = (only_level >= 0) ? (only_level == 0 ? 1 : k_ext) : ((n_levels > 1) ? 1 + (n_levels - 1) * k_ext : 1);
    a.slices = w.scan_splits, a.cps = 1;
    a.test_drop = w.test_drop;
    const size_t smem = sizeof(unsigned long long) * ctx->shape.max_k * max(kQuadElems, w.scan_splits);
    if (vec_ok(logits, ld_b, ld_level, ld_row, a.vocab, a.chunk) && w.scan_chunk == kScanChunkMax) {
        // Slices per row: two CTAs fit an SM, and a slice's first chunk costs about three later ones (the
        // threshold has to be found), so a row is cut only as far as all CTAs still run at once; with
        // more rows than that, one slice per row (measured at 712 rows: 108 us in one slice, 119 in two).
        int want = max(1, 2 * ctx->sm_count / max(rows * batch, 1));
        if (w.scan_slices_hint > 0) want = w.scan_slices_hint;
        const int slices0 = max(1, min(w.scan_splits, want));
        a.cps = (w.scan_splits + slices0 - 1) / slices0;
        a.slices = (w.scan_splits + a.cps - 1) / a.cps;
        dim3 grid(a.slices, rows, batch);
        return launch_pdl(row_scan_stream_kernel, grid, dim3(kStreamThreads), stream_smem_bytes(ctx->shape.max_k, a.slices), st, a);
    } else {
        dim3 grid(w.scan_splits, rows, batch);
        return launch_pdl(row_scan_kernel<false>, grid, dim3(kScanThreads), smem, st, a);
    }
    return cudaGetLastError();
}

cudaError_t launch_row_argmax(const resps_ctx* ctx, const int32_t* d_n_nodes, int batch,
                              const float* logits, int64_t ld_b, int64_t ld_row, int32_t* argmax_out,
                              const AcceptArgs* walk, bool* walked, cudaStream_t st, unsigned long long* key_out) {
    const Workspace& w = ctx->ws;
    ArgmaxArgs a;
    a.n_nodes = d_n_nodes;
    a.logits = logits;
    a.ld_b = ld_b, a.ld_row = ld_row;
    a.vocab = ctx->shape.vocab, a.max_tt = ctx->shape.max_tt;
    a.chunk = w.scan_chunk, a.splits = w.scan_splits;
    a.slices = w.scan_splits, a.cps = 1;
    a.part = w.amax_part, a.counter = w.amax_counter, a.seq_counter = w.amax_seq_counter, a.out = argmax_out;
    a.key_out = key_out;
    a.status = w.status;
    if (walked) *walked = false;
    if (vec_ok(logits, ld_b, ld_row, 0, a.vocab, a.chunk) && w.scan_chunk == kScanChunkMax) {
        // Slices per row as in the scan: a row is cut only as far as all CTAs still run at once.
        const int want = max(1, 2 * ctx->sm_count / max(ctx->shape.max_tt * batch, 1));
        const int slices0 = max(1, min(w.scan_splits, want));
        a.cps = (w.scan_splits + slices0 - 1) / slices0;
        a.slices = (w.scan_splits + a.cps - 1) / a.cps;
        AcceptArgs wa = {};
        if (walk) wa = *walk;
        if (walked) *walked = walk != nullptr;
        dim3 grid(a.slices, ctx->shape.max_tt, batch);
        return launch_pdl(row_argmax_stream_kernel, grid, dim3(kStreamThreads),
                          kStreamStages * kScanChunkMax * sizeof(float), st, a, wa, walk ? 1 : 0);
    }
    dim3 grid(w.scan_splits, ctx->shape.max_tt, batch);
    if (vec_ok(logits, ld_b, ld_row, 0, a.vocab, a.chunk))
        return launch_pdl(row_argmax_kernel<true>, grid, dim3(kScanThreads), 0, st, a);
    else
        return launch_pdl(row_argmax_kernel<false>, grid, dim3(kScanThreads), 0, st, a);
    return cudaGetLastError();
}

cudaError_t launch_shard_merge_rows(const resps_ctx* ctx, const resps_step* d_steps, int batch, int n_levels, int n_slots,
                                    int n_shards, const float* all_val, const int32_t* all_id, const double* all_lse,
                                    const int32_t* shard_offset, cudaStream_t st) {
    const Workspace& w = ctx->ws;
    ShardMergeArgs a;
    a.steps = d_steps, a.n_levels = n_levels, a.n_slots = n_slots;
    a.vocab = ctx->shape.vocab, a.max_tt = ctx->shape.max_tt, a.max_k = ctx->shape.max_k, a.max_rows = w.max_rows;
    a.n_shards = n_shards, a.batch = batch;
    a.all_val = all_val, a.all_id = all_id, a.all_lse = all_lse, a.shard_offset = shard_offset;
    a.row_val = w.row_val, a.row_id = w.row_id, a.row_lse = w.row_lse;
    const int k_ext = min(n_slots, ctx->shape.max_k);
    const int rows = (n_levels > 1) ? 1 + (n_levels - 1) * k_ext : 1;
    return launch_pdl(shard_merge_rows_kernel, dim3(rows, batch), dim3(128), 0, st, a);
}

cudaError_t launch_shard_merge_argmax(const resps_ctx* ctx, const int32_t* d_n_nodes, int batch, int n_shards,
                                      const unsigned long long* all_key, const int32_t* shard_offset, int32_t* out,
                                      cudaStream_t st) {
    ShardArgmaxArgs a;
    a.n_nodes = d_n_nodes, a.max_tt = ctx->shape.max_tt, a.n_shards = n_shards, a.batch = batch;
    a.all_key = all_key, a.shard_offset = shard_offset, a.out = out;
    return launch_pdl(shard_merge_argmax_kernel, dim3(batch), dim3(RESPS_MAX_TT), 0, st, a);
}

// ---------------------------------------------------------------------------------------
// Arg-max without a context and without any allocation (see resps_target_argmax_static in
// resps.h).  The split partials and arrival counters of row_argmax_kernel live in a
// file-scope device array instead of a context's cudaMalloc'ed workspace.
// ---------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxRows = RESPS_STATIC_MAX_ROWS;  // batch * max_tt
constexpr int kStaticMaxSplits = 64;
constexpr size_t kStaticPartBytes = sizeof(unsigned long long) * kStaticMaxRows * kStaticMaxSplits;
constexpr size_t kStaticCounterBytes = sizeof(unsigned int) * kStaticMaxRows;

// [rows][splits] packed (value, id) partials, then [rows] arrival counters: 516 KB per GPU.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticPartBytes + kStaticCounterBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
unsigned char* g_static_ptr[kMaxDevices] = {};  // device address of g_static_scratch, per device

// In host code the array's name only stands for the symbol; its device address has to be asked
// for, once per device, with that device current.
int static_scratch_address(unsigned char** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RESPS_ERR_NO_DEVICE;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return RESPS_ERR_CUDA;
        g_static_ptr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_static_ptr[dev];
    return RESPS_OK;
}

}  // namespace
}  // namespace resps

extern "C" int resps_target_argmax_static(const int32_t* d_n_nodes, int batch, int max_tt, int vocab,
                                          const float* d_target_logits, int64_t ld_b, int64_t ld_row,
                                          int32_t* d_target_argmax, resps_stream stream) {
    using namespace resps;
    if (!d_n_nodes || !d_target_logits || !d_target_argmax) return RESPS_ERR_INVALID_ARG;
    if (batch < 1 || max_tt < 1 || vocab < 1 || ld_row < vocab || ld_b < 0) return RESPS_ERR_INVALID_ARG;
    if (max_tt > RESPS_MAX_TT) return RESPS_ERR_UNSUPPORTED_SHAPE;
    if (static_cast<int64_t>(batch) * max_tt > kStaticMaxRows) return RESPS_ERR_CAPACITY;
    int chunk = 8192;
    if ((vocab + chunk - 1) / chunk > kStaticMaxSplits)
        chunk = ((vocab + kStaticMaxSplits - 1) / kStaticMaxSplits + 1023) / 1024 * 1024;
    const int splits = (vocab + chunk - 1) / chunk;
    unsigned char* scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != RESPS_OK) return rc;
    ArgmaxArgs a;
    a.n_nodes = d_n_nodes;
    a.logits = d_target_logits;
    a.ld_b = ld_b, a.ld_row = ld_row;
    a.vocab = vocab, a.max_tt = max_tt, a.chunk = chunk, a.splits = splits;
    a.slices = splits, a.cps = 1, a.seq_counter = nullptr, a.status = nullptr, a.key_out = nullptr;
    a.part = reinterpret_cast<unsigned long long*>(scratch);
    a.counter = reinterpret_cast<unsigned int*>(scratch + kStaticPartBytes);
    a.out = d_target_argmax;
    // The array keeps whatever the last call left: the counters must start at zero.
    if (cudaMemsetAsync(a.counter, 0, sizeof(unsigned int) * batch * max_tt, stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    dim3 grid(splits, max_tt, batch);
    if (vec_ok(d_target_logits, ld_b, ld_row, 0, vocab, chunk))
        row_argmax_kernel<true><<<grid, kScanThreads, 0, stream>>>(a);
    else
        row_argmax_kernel<false><<<grid, kScanThreads, 0, stream>>>(a);
    return cudaGetLastError() == cudaSuccess ? RESPS_OK : RESPS_ERR_CUDA;
}
