// Controller glue (Algorithm 1: action caching over a cache interval of N steps; Eq. 3 / Eq. 5: the
// reward, tokens per second, averaged over the interval; Eq. 4: the state is the concatenation of three
// hidden layers of the target model, read in place; Appendix A: the policy is a [128, 128] network over
// the filtered action grid).  One kernel per decoding step: it books the reward of the step that has
// just finished and, when the interval is over, asks the policy and writes the new (TT, d, k) into the
// device-resident step parameters, where the kernels of the step read them.
//
// The policy's first layer is a matrix-vector product over the 3 x 4096 state (6 MB of fp32 weights):
// a CTA per hidden unit and sequence, each thread a strided share of the features in 16-byte loads that
// are all in flight together, fp32 accumulation.  The last CTA of a sequence to arrive runs the two
// small layers (two threads per output, half a row each), picks the action and updates the state;
// sequences whose cached action is still valid skip the product altogether.
#include <cmath>

#include "common.cuh"

namespace resps {
namespace {

constexpr int kCtlThreads = 256;
constexpr int kMaxHidden = 256;
constexpr int kMaxActions = 1024;
constexpr unsigned kFull = 0xFFFFFFFFu;

struct ControllerArgs {
    resps_policy pol;
    const __nv_bfloat16* hidden[3];  // three layers' hidden states, [batch][features / 3] each
    int64_t ld_hidden;
    int batch, interval;
    float temperature;
    const double* uniform;       // [batch] or null (temperature 0)
    const int32_t* accept_len;   // [batch] of the finished step, or null
    const float* elapsed_s;      // [batch] seconds of the finished step, or null
    resps_controller_state* state;
    resps_step* steps;
    float* reward_avg;           // [batch]: written when an interval closes (else left alone)
    float* logits_out;           // [batch][n_actions] or null
    int32_t* action_out;         // [batch] or null
    float* h1;                   // workspace [batch][hidden]
    unsigned int* counter;       // workspace [batch]
};

__device__ __forceinline__ float block_sum(float v, float* s_red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = 0.f;
    for (int w = 0; w < kCtlThreads / 32; ++w) r += s_red[w];
    return r;
}

__device__ __forceinline__ bool aligned_to(const void* p, unsigned bytes) {
    return (reinterpret_cast<unsigned long long>(p) & (bytes - 1u)) == 0ull;
}

// out(o) = bias[o] + sum_i W[o][i] * s_in[i] for o < n_out, by the whole CTA: two threads per output, each
// half a row in 16-byte loads that are all in flight together (rows of 16-byte aligned fp32, n_in a
// multiple of 8; one thread per output and scalar loads otherwise).
template <typename Out>
__device__ __forceinline__ void dense_layer(const float* W, const float* bias, const float* s_in, int n_out, int n_in,
                                            Out out) {
    const int tid = threadIdx.x;
    if ((n_in & 7) == 0 && aligned_to(W, 16)) {
        const int half = tid & 1, quads = n_in >> 3;  // float4 per half row
        for (int o0 = 0; o0 < n_out; o0 += kCtlThreads / 2) {
            const int o = o0 + (tid >> 1);
            float acc = 0.f;
            if (o < n_out) {
                const float4* w4 = reinterpret_cast<const float4*>(W + static_cast<int64_t>(o) * n_in) + half * quads;
                const float* x = s_in + half * quads * 4;
#pragma unroll 8
                for (int i = 0; i < quads; ++i) {
                    const float4 w = __ldg(w4 + i);
                    acc = fmaf(w.x, x[4 * i], fmaf(w.y, x[4 * i + 1], fmaf(w.z, x[4 * i + 2], fmaf(w.w, x[4 * i + 3], acc))));
                }
            }
            acc += __shfl_xor_sync(kFull, acc, 1);
            if (o < n_out && half == 0) out(o, acc + bias[o]);
        }
    } else {
        for (int o = tid; o < n_out; o += kCtlThreads) {
            const float* w = W + static_cast<int64_t>(o) * n_in;
            float acc = bias[o];
            for (int i = 0; i < n_in; ++i) acc = fmaf(__ldg(w + i), s_in[i], acc);
            out(o, acc);
        }
    }
}

__global__ void __launch_bounds__(kCtlThreads) controller_kernel(const ControllerArgs a) {
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    __shared__ float s_red[kCtlThreads / 32];
    __shared__ float s_h1[kMaxHidden], s_h2[kMaxHidden];
    __shared__ float s_logit[kMaxActions];
    __shared__ double s_term[kMaxActions];
    __shared__ double s_mx;
    __shared__ unsigned long long s_key[kCtlThreads / 32];
    __shared__ int s_last;
    const int b = blockIdx.y, unit = blockIdx.x, tid = threadIdx.x;
    const resps_controller_state st = a.state[b];
    const bool ask = (st.cache_step == 0) || (st.action < 0);
    const int H = a.pol.hidden, F = a.pol.n_features, A = a.pol.n_actions;
    if (!ask) {
        // ---- the cached action stays: book the finished step's reward, advance the cache step ----------
        // (by the last CTA of the sequence to come by, when every other one has read the state)
        if (tid == 0 && atomicAdd(a.counter + b, 1u) == static_cast<unsigned>(H - 1)) {
            a.counter[b] = 0u;
            resps_controller_state n = st;
            if (a.accept_len) {
                n.reward_sum += static_cast<float>(a.accept_len[b] + 1) / a.elapsed_s[b];
                n.reward_steps += 1;
            }
            n.cache_step += 1;
            if (n.cache_step >= a.interval) n.cache_step = 0;
            a.state[b] = n;
            if (a.action_out) a.action_out[b] = n.action;
        }
        return;
    }
    // ---- first layer: hidden unit `unit` of sequence b -------------------------------------------------
    {
        const int per_layer = F / 3;
        const float* w = a.pol.w1 + static_cast<int64_t>(unit) * F;
        float acc = 0.f;
        const bool vec = (per_layer & 3) == 0 && (a.ld_hidden & 3) == 0 && aligned_to(a.pol.w1, 16) &&
                         aligned_to(a.hidden[0], 8) && aligned_to(a.hidden[1], 8) && aligned_to(a.hidden[2], 8);
        if (vec) {
            // four weights (16 bytes) and four features (8 bytes) per load, the loads of a thread independent
            // of one another: the 6 MB of weights stream in one or two round trips
#pragma unroll
            for (int layer = 0; layer < 3; ++layer) {
                const float4* w4 = reinterpret_cast<const float4*>(w + layer * per_layer);
                const uint2* h2 = reinterpret_cast<const uint2*>(a.hidden[layer] + b * a.ld_hidden);
#pragma unroll 4
                for (int i = tid; i < (per_layer >> 2); i += kCtlThreads) {
                    const float4 x = __ldg(w4 + i);
                    const uint2 h = __ldg(h2 + i);
                    acc = fmaf(x.x, __uint_as_float(h.x << 16), acc);
                    acc = fmaf(x.y, __uint_as_float(h.x & 0xFFFF0000u), acc);
                    acc = fmaf(x.z, __uint_as_float(h.y << 16), acc);
                    acc = fmaf(x.w, __uint_as_float(h.y & 0xFFFF0000u), acc);
                }
            }
        } else {
            for (int i = tid; i < F; i += kCtlThreads) {
                const int layer = i / per_layer, e = i - layer * per_layer;
                acc = fmaf(__ldg(w + i), __bfloat162float(a.hidden[layer][b * a.ld_hidden + e]), acc);
            }
        }
        acc = block_sum(acc, s_red);
        if (tid == 0) {
            a.h1[b * H + unit] = tanhf(acc + a.pol.b1[unit]);
            __threadfence();
            s_last = (atomicAdd(a.counter + b, 1u) == static_cast<unsigned>(H - 1));
        }
        __syncthreads();
        if (!s_last) return;
    }
    // ---- the last CTA of the sequence: second layer, action logits, the choice ---------------------------
    __threadfence();
    for (int i = tid; i < H; i += kCtlThreads) s_h1[i] = __ldcg(a.h1 + b * H + i);
    __syncthreads();
    dense_layer(a.pol.w2, a.pol.b2, s_h1, H, H, [&](int o, float v) { s_h2[o] = tanhf(v); });
    __syncthreads();
    dense_layer(a.pol.w3, a.pol.b3, s_h2, A, H, [&](int o, float v) {
        s_logit[o] = v;
        if (a.logits_out) a.logits_out[static_cast<int64_t>(b) * A + o] = v;
    });
    __syncthreads();
    const bool draw = a.temperature > 0.f;
    if (draw) {
        // softmax(logits / T) in fp64: the maximum by one thread, the exponentials by all, the sums below in
        // action order by one thread again (a few hundred terms)
        if (tid == 0) {
            double mx = -INFINITY;
            for (int o = 0; o < A; ++o) mx = fmax(mx, static_cast<double>(s_logit[o]) / a.temperature);
            s_mx = mx;
        }
        __syncthreads();
        for (int o = tid; o < A; o += kCtlThreads) s_term[o] = exp(static_cast<double>(s_logit[o]) / a.temperature - s_mx);
        __syncthreads();
    }
    if (!draw) {
        // arg-max over the actions, ties -> lowest index: (ordered value, ~index) keys, largest wins
        unsigned long long best = 0ull;
        for (int o = tid; o < A; o += kCtlThreads) {
            const unsigned u = __float_as_uint(s_logit[o]);
            const unsigned ord = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
            const unsigned long long key = (static_cast<unsigned long long>(ord) << 32) | (0xFFFFFFFFu - static_cast<unsigned>(o));
            best = key > best ? key : best;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const unsigned long long other = __shfl_xor_sync(kFull, best, off);
            best = other > best ? other : best;
        }
        if ((tid & 31) == 0) s_key[tid >> 5] = best;
        __syncthreads();
    }
    if (tid == 0) {
        int action = 0;
        if (!draw) {
            unsigned long long best = s_key[0];
            for (int wq = 1; wq < kCtlThreads / 32; ++wq) best = s_key[wq] > best ? s_key[wq] : best;
            action = static_cast<int>(0xFFFFFFFFu - static_cast<unsigned>(best & 0xFFFFFFFFull));
        } else {
            // inverse CDF in action order
            double total = 0.0;
            for (int o = 0; o < A; ++o) total += s_term[o];
            const double target = a.uniform[b] * total;
            double run = 0.0;
            action = A - 1;
            for (int o = 0; o < A; ++o) {
                run += s_term[o];
                if (run > target) {
                    action = o;
                    break;
                }
            }
        }
        resps_controller_state n = st;
        if (a.accept_len) {
            n.reward_sum += static_cast<float>(a.accept_len[b] + 1) / a.elapsed_s[b];
            n.reward_steps += 1;
        }
        if (n.reward_steps > 0) a.reward_avg[b] = n.reward_sum / static_cast<float>(n.reward_steps);  // Eq. 5
        n.reward_sum = 0.f, n.reward_steps = 0;
        n.action = action;
        n.cache_step = 1;
        if (n.cache_step >= a.interval) n.cache_step = 0;
        a.state[b] = n;
        resps_step s = a.steps[b];
        s.tt = a.pol.actions[3 * action + 0], s.d = a.pol.actions[3 * action + 1], s.k = a.pol.actions[3 * action + 2];
        a.steps[b] = s;
        if (a.action_out) a.action_out[b] = action;
        a.counter[b] = 0u;
    }
}

}  // namespace

int controller_max_hidden() { return kMaxHidden; }
int controller_max_actions() { return kMaxActions; }

cudaError_t launch_controller(const resps_ctx* ctx, const resps_policy* pol, const void* h, const void* m, const void* l,
                              int64_t ld_hidden, int batch, int interval, float temperature, const double* uniform,
                              const int32_t* accept_len, const float* elapsed_s, resps_controller_state* state,
                              resps_step* steps, float* reward_avg, float* logits_out, int32_t* action_out,
                              cudaStream_t st) {
    ControllerArgs a;
    a.pol = *pol;
    a.hidden[0] = static_cast<const __nv_bfloat16*>(h);
    a.hidden[1] = static_cast<const __nv_bfloat16*>(m);
    a.hidden[2] = static_cast<const __nv_bfloat16*>(l);
    a.ld_hidden = ld_hidden, a.batch = batch, a.interval = interval, a.temperature = temperature;
    a.uniform = uniform, a.accept_len = accept_len, a.elapsed_s = elapsed_s;
    a.state = state, a.steps = steps, a.reward_avg = reward_avg, a.logits_out = logits_out, a.action_out = action_out;
    a.h1 = ctx->ws.ctl_h1, a.counter = ctx->ws.ctl_counter;
    return launch_pdl(controller_kernel, dim3(pol->hidden, batch), dim3(kCtlThreads), 0, st, a);
}

}  // namespace resps
