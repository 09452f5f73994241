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
    unsigned long long* part_key;
    float2* part_ms;
    unsigned int* counter;
    float* row_val;
    int32_t* row_id;
    double* row_lse;
    int32_t* status;
};

// Insert `nk` into the warp's descending list (one entry per lane).
__device__ __forceinline__ void warp_insert(unsigned long long& mine, unsigned long long nk, int lane) {
    const unsigned ahead = __ballot_sync(kFull, mine > nk);
    const int pos = __popc(ahead);
    const unsigned long long up = __shfl_up_sync(kFull, mine, 1);
    if (lane == pos)
        mine = nk;
    else if (lane > pos)
        mine = up;
}

struct WarpTopK {
    unsigned long long mine = 0ull;  // this lane's list entry (0 = empty, ranks last)
    unsigned long long kth = 0ull;   // entry k-1, warp-uniform
    float thr = -INFINITY;       // its value: nothing below it can enter the top k

    // Offer up to four consecutive elements per lane; `nvalid` of them exist.
    __device__ __forceinline__ void offer4(const float (&v)[4], int id0, int nvalid, int k, int lane) {
        bool hit = false;
#pragma unroll
        for (int c = 0; c < 4; ++c) hit |= (c < nvalid) && (v[c] >= thr);
        if (!__any_sync(kFull, hit)) return;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            unsigned pending = __ballot_sync(kFull, (c < nvalid) && (v[c] >= thr));
            const unsigned long long cand = pack_val_id(v[c], id0 + c);
            while (pending) {
                const int src = __ffs(pending) - 1;
                pending &= pending - 1;
                const unsigned long long nk = __shfl_sync(kFull, cand, src);
                if (nk > kth) {
                    warp_insert(mine, nk, lane);
                    kth = __shfl_sync(kFull, mine, k - 1);
                    thr = (kth == 0ull) ? -INFINITY : key_val(kth);
                }
            }
        }
    }
};

// Running (max, sum) of 2^(y - max) with y = x*log2(e).
struct LseAcc {
    float m2 = -INFINITY;
    float s = 0.f;
    __device__ __forceinline__ void add4(const float (&v)[4], int nvalid) {
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (c < nvalid) mx = fmaxf(mx, v[c] * kLog2e);
        if (mx > m2) {
            s *= ex2_approx(m2 - mx);
            m2 = mx;
        }
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (c < nvalid) s += ex2_approx(fmaf(v[c], kLog2e, -m2));
    }
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
    for (int c = threadIdx.x; c < n; c += blockDim.x) {
        const unsigned long long mine = keys[c];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (keys[j] > mine) || (keys[j] == mine && j < c);
        if (rank < k) out(rank, mine);
    }
}

template <bool VEC>
__global__ void __launch_bounds__(kScanThreads, 4) row_scan_kernel(const ScanArgs a) {
    const int b = blockIdx.z, r = blockIdx.y, sp = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const StepDims sd = clamp_step(a.steps[b], a.n_levels, a.n_slots, a.max_tt, a.max_k, a.vocab);
    const int k = sd.k;
    const int rows = 1 + (sd.d - 1) * k;
    if (r >= rows) return;
    if (sd.clamped && r == 0 && sp == 0 && tid == 0) atomicOr(a.status, RESPS_STATUS_STEP_CLAMPED);
    const int level = (r == 0) ? 0 : 1 + (r - 1) / k;
    const int slot = (r == 0) ? 0 : (r - 1) % k;
    const float* row = a.logits + b * a.ld_b + level * a.ld_level + slot * a.ld_row;
    const int begin = sp * a.chunk;
    const int end = min(a.vocab, begin + a.chunk);

    WarpTopK top;
    LseAcc acc;
    constexpr int kUnroll = 4;
    for (int base = begin; base < end; base += kScanThreads * 4 * kUnroll) {
        float v[kUnroll][4];
        int nv[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int e0 = base + (u * kScanThreads + tid) * 4;
            nv[u] = max(0, min(4, end - e0));
            if (VEC) {
                if (nv[u] > 0) {  // vocab and chunk are multiples of 4 on this path
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
            if (nv[u] > 0) acc.add4(v[u], nv[u]);
            top.offer4(v[u], e0, nv[u], k, lane);
        }
    }

    // ---- CTA reduction -------------------------------------------------------
    __shared__ unsigned long long s_keys[64 * RESPS_MAX_K];  // 8 warp lists, later `splits` partial lists
    __shared__ float2 s_ms[kScanThreads / 32];
    __shared__ bool s_last;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(kFull, acc.m2, o);
        const float os = __shfl_xor_sync(kFull, acc.s, o);
        acc.merge(om, os);
    }
    if (lane < k) s_keys[warp * k + lane] = top.mine;
    if (lane == 0) s_ms[warp] = make_float2(acc.m2, acc.s);
    __syncthreads();
    const int64_t prow = static_cast<int64_t>(b) * a.max_rows + r;
    unsigned long long* part = a.part_key + (prow * a.splits + sp) * a.max_k;
    select_top_by_rank(s_keys, (kScanThreads / 32) * k, k,
                       [&](int rank, unsigned long long key) { part[rank] = key; });
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
    __syncthreads();
    float* oval = a.row_val + prow * a.max_k;
    int32_t* oid = a.row_id + prow * a.max_k;
    select_top_by_rank(s_keys, a.splits * k, k, [&](int rank, unsigned long long key) {
        oval[rank] = key_val(key);
        oid[rank] = key_id(key);
    });
    if (tid == 0) {
        const float2* ms = a.part_ms + prow * a.splits;
        double M = -INFINITY;
        for (int i = 0; i < a.splits; ++i) M = fmax(M, static_cast<double>(__ldcg(&ms[i].x)));
        double sum = 0.0;
        for (int i = 0; i < a.splits; ++i) {
            const float2 p = __ldcg(ms + i);
            if (p.y > 0.f) sum += static_cast<double>(p.y) * exp2(static_cast<double>(p.x) - M);
        }
        a.row_lse[prow] = (M + log2(sum)) * 0.6931471805599453094;
        a.counter[prow] = 0u;
    }
}

struct ArgmaxArgs {
    const int32_t* n_nodes;
    const float* logits;
    int64_t ld_b, ld_row;
    int vocab, max_tt, chunk, splits;
    unsigned long long* part;
    unsigned int* counter;
    int32_t* out;
};

template <bool VEC>
__global__ void __launch_bounds__(kScanThreads, 4) row_argmax_kernel(const ArgmaxArgs a) {
    const int b = blockIdx.z, r = blockIdx.y, sp = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = min(max(a.n_nodes[b], 0), a.max_tt);
    if (r >= n) return;
    const float* row = a.logits + b * a.ld_b + r * a.ld_row;
    const int begin = sp * a.chunk;
    const int end = min(a.vocab, begin + a.chunk);

    float best = -INFINITY;
    int best_id = 0x7FFFFFFF;
    constexpr int kUnroll = 4;
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
        a.counter[prow] = 0u;
    }
}

inline bool vec_ok(const void* p, int64_t s0, int64_t s1, int64_t s2, int vocab, int chunk) {
    return (reinterpret_cast<uintptr_t>(p) % 16 == 0) && s0 % 4 == 0 && s1 % 4 == 0 && s2 % 4 == 0 &&
           vocab % 4 == 0 && chunk % 4 == 0;
}

}  // namespace

cudaError_t launch_row_scan(const resps_ctx* ctx, const resps_step* d_steps, int batch,
                            const float* logits, int64_t ld_b, int64_t ld_level, int64_t ld_row,
                            int n_levels, int n_slots, cudaStream_t st) {
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
    const int rows = (n_levels > 1) ? 1 + (n_levels - 1) * k_ext : 1;
    dim3 grid(w.scan_splits, rows, batch);
    if (vec_ok(logits, ld_b, ld_level, ld_row, a.vocab, a.chunk))
        row_scan_kernel<true><<<grid, kScanThreads, 0, st>>>(a);
    else
        row_scan_kernel<false><<<grid, kScanThreads, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_row_argmax(const resps_ctx* ctx, const int32_t* d_n_nodes, int batch,
                              const float* logits, int64_t ld_b, int64_t ld_row, int32_t* argmax_out,
                              cudaStream_t st) {
    const Workspace& w = ctx->ws;
    ArgmaxArgs a;
    a.n_nodes = d_n_nodes;
    a.logits = logits;
    a.ld_b = ld_b, a.ld_row = ld_row;
    a.vocab = ctx->shape.vocab, a.max_tt = ctx->shape.max_tt;
    a.chunk = w.scan_chunk, a.splits = w.scan_splits;
    a.part = w.amax_part, a.counter = w.amax_counter, a.out = argmax_out;
    dim3 grid(w.scan_splits, ctx->shape.max_tt, batch);
    if (vec_ok(logits, ld_b, ld_row, 0, a.vocab, a.chunk))
        row_argmax_kernel<true><<<grid, kScanThreads, 0, st>>>(a);
    else
        row_argmax_kernel<false><<<grid, kScanThreads, 0, st>>>(a);
    return cudaGetLastError();
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
