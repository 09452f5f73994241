// Tree-masked verification attention (Section 3.2, "Verification Phase": all tree
// tokens are scored by the target in one pass; Appendix D: the attention mask
// follows the tree).  Split-KV flash-decode: the query rows of one KV head
// (tree token x the Hq/Hkv heads sharing it) are packed into 64-row tiles so that
// QK^T and PV are dense tensor-core contractions; K/V tiles of 64 keys stream
// through a double-buffered shared-memory pipeline; the ancestor bitmask is applied
// from registers only on tiles that reach past the prefix.
//
// Work list: every (sequence, KV head, row tile, key split) is an item; a persistent
// grid walks the items.  The list is derived inside the kernel from the device-resident
// step parameters, so nothing about the launch depends on (TT, d, k, L).  Items of one
// (sequence, head, row tile) group write un-normalised partials; the group's last
// arriving CTA combines them.
#include <cmath>

#include "common.cuh"

namespace resps {
namespace {

constexpr int kAttnThreads = 128;
constexpr int kBM = 64;  // query rows per item
constexpr int kBN = 64;  // keys per tile
constexpr int kMaxBatchSmem = 256;
constexpr unsigned kFull = 0xFFFFFFFFu;

struct AttnArgs {
    const resps_step* steps;
    const int32_t* n_nodes;
    int batch;
    const __nv_bfloat16* q;
    __nv_bfloat16* o;
    float* lse;
    const __nv_bfloat16* kc;
    const __nv_bfloat16* vc;
    int64_t s_seq, s_head, s_tok, capacity;
    const uint64_t* mask;
    float scale_log2;
    int Hq, Hkv, max_tt;
    float* part_o;
    float2* part_ml;
    unsigned int* counter;
    int max_items;
    int32_t* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N));
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Byte offset of 16-byte piece `chunk` of row `row` in a [rows][D] bf16 tile whose pieces
// are XOR-swizzled by the row so that 8 consecutive rows hit 8 different bank groups.
template <int D>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
    return static_cast<uint32_t>(row * (D * 2) + ((chunk ^ (row & 7)) << 4));
}

struct Sched {
    int n[kMaxBatchSmem];       // tree nodes (0 = sequence skipped)
    int L[kMaxBatchSmem];
    int mt[kMaxBatchSmem];      // row tiles
    int kt[kMaxBatchSmem];      // key tiles
    int splits[kMaxBatchSmem];
    int item0[kMaxBatchSmem + 1];
    int group0[kMaxBatchSmem + 1];
};

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 2) tree_attention_kernel(const AttnArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ Sched sc;
    __shared__ bool s_last;
    constexpr int kTileBytes = kBN * D * 2;
    constexpr int kChunks = D / 8;  // 16-byte pieces per row
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = a.Hq / a.Hkv;
    unsigned char* sK[2] = {smem, smem + kTileBytes};
    unsigned char* sV[2] = {smem + 2 * kTileBytes, smem + 3 * kTileBytes};

    // ---- work list from the device-resident step parameters ------------------------
    for (int b = tid; b < a.batch; b += kAttnThreads) {
        int n = min(max(a.n_nodes[b], 0), a.max_tt);
        const int L = max(a.steps[b].prefix_len, 0);
        if (static_cast<int64_t>(L) + n > a.capacity) {
            atomicOr(a.status, RESPS_STATUS_KV_OVERFLOW);
            n = 0;
        }
        sc.n[b] = n;
        sc.L[b] = L;
        sc.mt[b] = (n * G + kBM - 1) / kBM;
        sc.kt[b] = (n > 0) ? (L + n + kBN - 1) / kBN : 0;
    }
    __syncthreads();
    if (tid == 0) {
        long long total_tiles = 0;
        for (int b = 0; b < a.batch; ++b) total_tiles += 1ll * a.Hkv * sc.mt[b] * sc.kt[b];
        const int tps = max(1, static_cast<int>((total_tiles + gridDim.x - 1) / gridDim.x));
        int items = 0, groups = 0;
        for (int b = 0; b < a.batch; ++b) {
            sc.item0[b] = items;
            sc.group0[b] = groups;
            sc.splits[b] = (sc.kt[b] + tps - 1) / tps;
            items += a.Hkv * sc.mt[b] * sc.splits[b];
            groups += a.Hkv * sc.mt[b];
        }
        sc.item0[a.batch] = items;
        sc.group0[a.batch] = groups;
    }
    __syncthreads();
    const int total_items = min(sc.item0[a.batch], a.max_items);

    for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
        int b = 0;
        while (item >= sc.item0[b + 1]) ++b;
        const int n = sc.n[b], L = sc.L[b], splits = sc.splits[b];
        const int local = item - sc.item0[b];
        const int sp = local % splits;
        const int grp_local = local / splits;  // = g * mt + mtile
        const int mtile = grp_local % sc.mt[b];
        const int g = grp_local / sc.mt[b];
        const int group = sc.group0[b] + grp_local;
        const int kv_len = L + n;
        const int M = n * G;
        const int t_begin = static_cast<int>(1ll * sc.kt[b] * sp / splits);
        const int t_end = static_cast<int>(1ll * sc.kt[b] * (sp + 1) / splits);
        const int row_base = mtile * kBM;

        const __nv_bfloat16* kbase = a.kc + b * a.s_seq + g * a.s_head;
        const __nv_bfloat16* vbase = a.vc + b * a.s_seq + g * a.s_head;
        auto issue_tile = [&](int stage, int t) {
            const int j0 = t * kBN;
            const uint32_t dk = smem_u32(sK[stage]), dv = smem_u32(sV[stage]);
            for (int i = tid; i < kBN * kChunks; i += kAttnThreads) {
                const int r = i / kChunks, c = i % kChunks;
                const int j = j0 + r;
                const bool ok = j < kv_len;
                const int64_t off = static_cast<int64_t>(ok ? j : 0) * a.s_tok + c * 8;
                cp_async16(dk + tile_off<D>(r, c), kbase + off, ok);
                cp_async16(dv + tile_off<D>(r, c), vbase + off, ok);
            }
        };

        // prologue: first K/V tile into stage 0, the Q tile into the (still free) V stage 1
        issue_tile(0, t_begin);
        {
            const uint32_t dq = smem_u32(sV[1]);
            for (int i = tid; i < kBM * kChunks; i += kAttnThreads) {
                const int r = i / kChunks, c = i % kChunks;
                const int R = row_base + r;
                const bool ok = R < M;
                const int t = ok ? R / G : 0, h = g * G + (ok ? R % G : 0);
                const __nv_bfloat16* src =
                    a.q + ((static_cast<int64_t>(b) * a.max_tt + t) * a.Hq + h) * D + c * 8;
                cp_async16(dq + tile_off<D>(r, c), src, ok);
            }
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();
        uint32_t qf[D / 16][4];
        {
            const uint32_t dq = smem_u32(sV[1]);
            const int mi = lane >> 3, r8 = lane & 7;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const int row = warp * 16 + r8 + (mi & 1) * 8;
                const int chunk = ks * 2 + (mi >> 1);
                ldsm_x4(dq + tile_off<D>(row, chunk), qf[ks]);
            }
        }
        __syncthreads();

        // rows of this thread: r_lo = warp*16 + lane/4 and r_lo + 8
        const int r_lo = row_base + warp * 16 + (lane >> 2);
        unsigned long long mlo[2], mhi[2];
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
            const int R = r_lo + h2 * 8;
            const int t = R / G;
            const bool ok = R < M;
            mlo[h2] = ok ? a.mask[(static_cast<int64_t>(b) * a.max_tt + t) * 2 + 0] : 0ull;
            mhi[h2] = ok ? a.mask[(static_cast<int64_t>(b) * a.max_tt + t) * 2 + 1] : 0ull;
        }

        float oacc[D / 8][4];
#pragma unroll
        for (int i = 0; i < D / 8; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
        float row_m[2] = {-INFINITY, -INFINITY}, row_l[2] = {0.f, 0.f};

        for (int t = t_begin; t < t_end; ++t) {
            const int stage = (t - t_begin) & 1;
            if (t + 1 < t_end) {
                issue_tile(stage ^ 1, t + 1);
                cp_async_commit();
                cp_async_wait<1>();
            } else {
                cp_async_wait<0>();
            }
            __syncthreads();

            // ---- S = Q K^T ---------------------------------------------------------
            float sacc[kBN / 8][4];
#pragma unroll
            for (int i = 0; i < kBN / 8; ++i) sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
            const uint32_t dk = smem_u32(sK[stage]), dv = smem_u32(sV[stage]);
            {
                const int mi = lane >> 3, r8 = lane & 7;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
                    for (int np = 0; np < kBN / 16; ++np) {
                        uint32_t bf[4];
                        const int key = np * 16 + r8 + (mi >> 1) * 8;
                        const int chunk = ks * 2 + (mi & 1);
                        ldsm_x4(dk + tile_off<D>(key, chunk), bf);
                        mma_bf16(sacc[np * 2], qf[ks], bf[0], bf[1]);
                        mma_bf16(sacc[np * 2 + 1], qf[ks], bf[2], bf[3]);
                    }
                }
            }

            // ---- scale, mask, online softmax -----------------------------------------
            const int j0 = t * kBN;
            const bool need_mask = (j0 + kBN > L);
            float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int nt = 0; nt < kBN / 8; ++nt) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int h2 = e >> 1;
                    float s = sacc[nt][e] * a.scale_log2;
                    if (need_mask) {
                        const int j = j0 + nt * 8 + (lane & 3) * 2 + (e & 1);
                        const int i = j - L;
                        bool ok = true;
                        if (i >= 0) {
                            const unsigned long long w = (i < 64) ? mlo[h2] : mhi[h2];
                            ok = (i < n) && ((w >> (i & 63)) & 1ull);
                        }
                        if (!ok) s = -INFINITY;
                    }
                    sacc[nt][e] = s;
                    tmax[h2] = fmaxf(tmax[h2], s);
                }
            }
            float corr[2], m_use[2];
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
                tmax[h2] = fmaxf(tmax[h2], __shfl_xor_sync(kFull, tmax[h2], 1));
                tmax[h2] = fmaxf(tmax[h2], __shfl_xor_sync(kFull, tmax[h2], 2));
                const float m_new = fmaxf(row_m[h2], tmax[h2]);
                m_use[h2] = (m_new == -INFINITY) ? 0.f : m_new;
                corr[h2] = ex2_approx(row_m[h2] - m_use[h2]);
                row_m[h2] = m_new;
            }
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                oacc[i][0] *= corr[0], oacc[i][1] *= corr[0];
                oacc[i][2] *= corr[1], oacc[i][3] *= corr[1];
            }

            // ---- P = exp2(S - m), O += P V -----------------------------------------------
            // P is fed to the tensor cores as bf16 hi + bf16 lo (two products per V tile):
            // a single bf16 rounding of P alone would cost ~0.4 % per weight, which shows up
            // as ~1 % of a row's rms in the worst element; the split keeps it near fp32.
            float psum[2] = {0.f, 0.f};
            {
                const int mi = lane >> 3, r8 = lane & 7;
#pragma unroll
                for (int kk = 0; kk < kBN / 16; ++kk) {
                    uint32_t phi[4], plo[4];
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const int nt = kk * 2 + half;
                        const float p0 = ex2_approx(sacc[nt][0] - m_use[0]);
                        const float p1 = ex2_approx(sacc[nt][1] - m_use[0]);
                        const float p2 = ex2_approx(sacc[nt][2] - m_use[1]);
                        const float p3 = ex2_approx(sacc[nt][3] - m_use[1]);
                        psum[0] += p0 + p1;
                        psum[1] += p2 + p3;
                        const __nv_bfloat162 h01 = __floats2bfloat162_rn(p0, p1);
                        const __nv_bfloat162 h23 = __floats2bfloat162_rn(p2, p3);
                        phi[half * 2 + 0] = *reinterpret_cast<const uint32_t*>(&h01);
                        phi[half * 2 + 1] = *reinterpret_cast<const uint32_t*>(&h23);
                        plo[half * 2 + 0] = pack_bf16(p0 - __low2float(h01), p1 - __high2float(h01));
                        plo[half * 2 + 1] = pack_bf16(p2 - __low2float(h23), p3 - __high2float(h23));
                    }
#pragma unroll
                    for (int dp = 0; dp < D / 16; ++dp) {
                        uint32_t bf[4];
                        const int key = kk * 16 + r8 + (mi & 1) * 8;
                        const int chunk = dp * 2 + (mi >> 1);
                        ldsm_x4_t(dv + tile_off<D>(key, chunk), bf);
                        mma_bf16(oacc[dp * 2], phi, bf[0], bf[1]);
                        mma_bf16(oacc[dp * 2 + 1], phi, bf[2], bf[3]);
                        mma_bf16(oacc[dp * 2], plo, bf[0], bf[1]);
                        mma_bf16(oacc[dp * 2 + 1], plo, bf[2], bf[3]);
                    }
                }
            }
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) row_l[h2] = row_l[h2] * corr[h2] + psum[h2];
            __syncthreads();  // the stage is free for the load issued next iteration
        }

        // ---- row sums across the 4 lanes of a row --------------------------------------
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
            row_l[h2] += __shfl_xor_sync(kFull, row_l[h2], 1);
            row_l[h2] += __shfl_xor_sync(kFull, row_l[h2], 2);
        }

        if (splits == 1) {
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
                const int R = r_lo + h2 * 8;
                if (R >= M) continue;
                const int t = R / G, h = g * G + R % G;
                const float inv = 1.f / row_l[h2];
                __nv_bfloat16* dst = a.o + ((static_cast<int64_t>(b) * a.max_tt + t) * a.Hq + h) * D;
#pragma unroll
                for (int i = 0; i < D / 8; ++i) {
                    const uint32_t v = pack_bf16(oacc[i][h2 * 2] * inv, oacc[i][h2 * 2 + 1] * inv);
                    *reinterpret_cast<uint32_t*>(dst + i * 8 + (lane & 3) * 2) = v;
                }
                if (a.lse && (lane & 3) == 0)
                    a.lse[(static_cast<int64_t>(b) * a.max_tt + t) * a.Hq + h] =
                        (row_m[h2] + log2f(row_l[h2])) * 0.6931471805599453f;
            }
            continue;
        }

        // ---- partial result, then the group's last CTA combines ------------------------
        float* po = a.part_o + static_cast<int64_t>(item) * kBM * D;
        float2* pml = a.part_ml + static_cast<int64_t>(item) * kBM;
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
            const int r = warp * 16 + (lane >> 2) + h2 * 8;
#pragma unroll
            for (int i = 0; i < D / 8; ++i)
                __stcg(reinterpret_cast<float2*>(po + r * D + i * 8 + (lane & 3) * 2),
                       make_float2(oacc[i][h2 * 2], oacc[i][h2 * 2 + 1]));
            if ((lane & 3) == 0) __stcg(pml + r, make_float2(row_m[h2], row_l[h2]));
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) s_last = (atomicAdd(a.counter + group, 1u) == static_cast<unsigned>(splits - 1));
        __syncthreads();
        if (s_last) {
            __threadfence();
            const int item_first = item - sp;
            const int rows_here = min(kBM, M - row_base);
            // thread -> (row, 4 consecutive columns)
            for (int idx = tid; idx < rows_here * (D / 4); idx += kAttnThreads) {
                const int r = idx / (D / 4), c4 = idx % (D / 4);
                float Mx = -INFINITY;
                for (int s2 = 0; s2 < splits; ++s2)
                    Mx = fmaxf(Mx, __ldcg(&a.part_ml[static_cast<int64_t>(item_first + s2) * kBM + r].x));
                float den = 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int s2 = 0; s2 < splits; ++s2) {
                    const float2 ml = __ldcg(&a.part_ml[static_cast<int64_t>(item_first + s2) * kBM + r]);
                    const float w = ex2_approx(ml.x - Mx);
                    den += ml.y * w;
                    const float4 v = __ldcg(reinterpret_cast<const float4*>(
                        a.part_o + (static_cast<int64_t>(item_first + s2) * kBM + r) * D + c4 * 4));
                    acc.x += v.x * w, acc.y += v.y * w, acc.z += v.z * w, acc.w += v.w * w;
                }
                const float inv = 1.f / den;
                const int R = row_base + r;
                const int t = R / G, h = g * G + R % G;
                __nv_bfloat16* dst =
                    a.o + ((static_cast<int64_t>(b) * a.max_tt + t) * a.Hq + h) * D + c4 * 4;
                uint2 out;
                out.x = pack_bf16(acc.x * inv, acc.y * inv);
                out.y = pack_bf16(acc.z * inv, acc.w * inv);
                *reinterpret_cast<uint2*>(dst) = out;
                if (a.lse && c4 == 0)
                    a.lse[(static_cast<int64_t>(b) * a.max_tt + t) * a.Hq + h] =
                        (Mx + log2f(den)) * 0.6931471805599453f;
            }
            if (tid == 0) a.counter[group] = 0u;
        }
        __syncthreads();
    }
}

}  // namespace

cudaError_t attention_setup(resps_ctx*) {
    cudaError_t e = cudaFuncSetAttribute(tree_attention_kernel<128>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, 4 * kBN * 128 * 2);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(tree_attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                4 * kBN * 64 * 2);
}

cudaError_t launch_tree_attention(const resps_ctx* ctx, const resps_step* d_steps,
                                  const int32_t* d_n_nodes, int batch, const __nv_bfloat16* q,
                                  __nv_bfloat16* o, float* lse, const __nv_bfloat16* k_cache,
                                  const __nv_bfloat16* v_cache, int64_t stride_seq,
                                  int64_t stride_head, int64_t stride_tok, int64_t capacity,
                                  const uint64_t* mask, float scale, cudaStream_t st) {
    AttnArgs a;
    a.steps = d_steps, a.n_nodes = d_n_nodes, a.batch = batch;
    a.q = q, a.o = o, a.lse = lse, a.kc = k_cache, a.vc = v_cache;
    a.s_seq = stride_seq, a.s_head = stride_head, a.s_tok = stride_tok, a.capacity = capacity;
    a.mask = mask;
    a.scale_log2 = scale * 1.4426950408889634f;
    a.Hq = ctx->shape.n_q_heads, a.Hkv = ctx->shape.n_kv_heads, a.max_tt = ctx->shape.max_tt;
    a.part_o = ctx->ws.attn_part_o, a.part_ml = ctx->ws.attn_part_ml, a.counter = ctx->ws.attn_counter;
    a.max_items = ctx->ws.attn_max_items, a.status = ctx->ws.status;
    const int D = ctx->shape.head_dim;
    const size_t smem = 4 * kBN * D * 2;
    if (D == 128)
        tree_attention_kernel<128><<<ctx->ws.attn_grid, kAttnThreads, smem, st>>>(a);
    else
        tree_attention_kernel<64><<<ctx->ws.attn_grid, kAttnThreads, smem, st>>>(a);
    return cudaGetLastError();
}

int attention_tile_rows() { return kBM; }
int attention_max_batch() { return kMaxBatchSmem; }

}  // namespace resps
