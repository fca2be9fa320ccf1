// Adaptive block length (Section 3.1 "Adaptive Block Length"; Section 4: tau = 0.8): after every draft a small router
// decides, per sequence, whether the small model goes on drafting or the drafts made so far are verified.
//
// Features of one draft, from the small model's distribution q = softmax(logits) for it: the entropy of q (nats), the
// k largest probabilities in descending order (lowest id first on ties), and the small model's embedding rows of those
// k tokens.  Router: hidden = relu(W1 x + b1), s = sigmoid(w2 . hidden + b2) = predicted probability that the large
// model disagrees; drafting continues while 1 - s >= tau and fewer than gamma_max drafts exist.
//
// All sums run in a fixed order (strided per thread, then over the warps in order), fp32.
// Dynamic shared memory: (1 + k + k * d) floats for the feature vector.
#pragma once
#include <math.h>
#include <limits.h>
#include "common.cuh"
#include "misc_kernels.cuh"
#include "tc_common.cuh"

namespace tandem {

constexpr int RT_THREADS = 1024;   // one CTA reads a whole row of logits and the router's weights: many loads in flight
constexpr int RT_WARPS = RT_THREADS / 32;
constexpr int RT_MAX_K = 8;

struct RouterArgs {
    const float* w1;    // [hidden][1 + k + k * d]
    const float* b1;    // [hidden]
    const float* w2;    // [hidden]
    float b2, tau;
    int k, hidden;
};

__device__ __forceinline__ float rt_block_sum(float v, float* red) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = 0.f;
#pragma unroll
    for (int w = 0; w < RT_WARPS; ++w) r += red[w];
    return r;
}
__device__ __forceinline__ float rt_block_max(float v, float* red) {
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
#pragma unroll
    for (int w = 1; w < RT_WARPS; ++w) r = fmaxf(r, red[w]);
    return r;
}

// Start of an adaptive iteration: every live sequence drafts, nobody has a draft yet.  grid: 1; block: 256.
__global__ void __launch_bounds__(256) adaptive_begin_kernel(LoopState st, int batch) {
    pdl_wait();
    pdl_launch_dependents();
    __shared__ int s_live;
    if (threadIdx.x == 0) s_live = 0;
    __syncthreads();
    for (int b = threadIdx.x; b < batch; b += 256) {
        const int live = st.done[b] ? 0 : 1;
        st.drafting[b] = live;
        st.block_len[b] = 0;
        if (live) atomicAdd(&s_live, 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) { st.counters[7] = s_live; st.counters[9] = 0; }
}

// After draft step s (0-based): the router's decision for every sequence that is still drafting.  The last CTA to
// finish publishes (router ticket, sequences still drafting) to the host.
// logits: [batch][V] of this step; emb: the small model's embedding table [V][d].  grid: batch; block: RT_THREADS.
template <typename T>
__global__ void __launch_bounds__(RT_THREADS) router_kernel(LoopState st, int batch, const float* __restrict__ logits, int V, int s,
                                                            int gamma_max, const T* __restrict__ emb, int d, RouterArgs r) {
    extern __shared__ float s_x[];            // the feature vector, 1 + k + k * d floats
    __shared__ float red[RT_WARPS];
    __shared__ float s_bv[RT_WARPS];
    __shared__ int s_bi[RT_WARPS];
    __shared__ float s_prob[RT_MAX_K];
    __shared__ int s_top[RT_MAX_K];
    __shared__ float s_hid[RT_WARPS];
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (st.drafting[b]) {   // (uniform over the block)
        const float* row = logits + (size_t)b * V;
        // pass 1: the row maximum and this thread's k largest logits (value descending, lower id first on ties);
        // the row is read 16 bytes at a time, several loads in flight (one CTA reads the whole row: latency counts)
        float tv[RT_MAX_K];
        int ti[RT_MAX_K];
#pragma unroll
        for (int j = 0; j < RT_MAX_K; ++j) { tv[j] = -INFINITY; ti[j] = INT_MAX; }
        float m = -INFINITY;
        auto offer = [&](float v, int i) {
            m = fmaxf(m, v);
            if (v > tv[RT_MAX_K - 1] || (v == tv[RT_MAX_K - 1] && i < ti[RT_MAX_K - 1])) {   // rare once the list has warmed up
                tv[RT_MAX_K - 1] = v; ti[RT_MAX_K - 1] = i;
#pragma unroll
                for (int j = RT_MAX_K - 1; j > 0; --j) {
                    if (tv[j] > tv[j - 1] || (tv[j] == tv[j - 1] && ti[j] < ti[j - 1])) {
                        const float fv = tv[j]; tv[j] = tv[j - 1]; tv[j - 1] = fv;
                        const int fi = ti[j]; ti[j] = ti[j - 1]; ti[j - 1] = fi;
                    }
                }
            }
        };
        const bool vec = (V & 3) == 0 && (reinterpret_cast<uintptr_t>(row) & 15) == 0;
        const int V4 = vec ? V >> 2 : 0;
#pragma unroll 4
        for (int i4 = tid; i4 < V4; i4 += RT_THREADS) {
            const float4 x = __ldcg(reinterpret_cast<const float4*>(row) + i4);
            offer(x.x, 4 * i4); offer(x.y, 4 * i4 + 1); offer(x.z, 4 * i4 + 2); offer(x.w, 4 * i4 + 3);
        }
        for (int i = 4 * V4 + tid; i < V; i += RT_THREADS) offer(__ldcg(row + i), i);
        m = rt_block_max(m, red);
        // pass 2: normaliser and sum of e * (l - m)
        float z = 0.f, s1 = 0.f;
#pragma unroll 4
        for (int i4 = tid; i4 < V4; i4 += RT_THREADS) {
            const float4 x = __ldcg(reinterpret_cast<const float4*>(row) + i4);
            const float t0 = x.x - m, t1 = x.y - m, t2 = x.z - m, t3 = x.w - m;
            const float e0 = expf(t0), e1 = expf(t1), e2 = expf(t2), e3 = expf(t3);
            z += (e0 + e1) + (e2 + e3);
            s1 = fmaf(e0, t0, s1); s1 = fmaf(e1, t1, s1); s1 = fmaf(e2, t2, s1); s1 = fmaf(e3, t3, s1);
        }
        for (int i = 4 * V4 + tid; i < V; i += RT_THREADS) {
            const float t = __ldcg(row + i) - m, e = expf(t);
            z += e;
            s1 = fmaf(e, t, s1);
        }
        z = rt_block_sum(z, red);
        s1 = rt_block_sum(s1, red);
        const float entropy = logf(z) - s1 / z;          // -sum q log q with q = e / z
        // the k most probable tokens of the row: k rounds, each thread offering the best entry of its list not taken yet
        int head = 0;
        for (int j = 0; j < r.k; ++j) {
            float bv = -INFINITY;
            int bi = INT_MAX;
#pragma unroll
            for (int jj = 0; jj < RT_MAX_K; ++jj) if (jj == head) { bv = tv[jj]; bi = ti[jj]; }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            __syncthreads();
            if (lane == 0) { s_bv[warp] = bv; s_bi[warp] = bi; }
            __syncthreads();
            if (tid == 0) {
                for (int w = 1; w < RT_WARPS; ++w)
                    if (s_bv[w] > bv || (s_bv[w] == bv && s_bi[w] < bi)) { bv = s_bv[w]; bi = s_bi[w]; }
                s_top[j] = bi == INT_MAX ? 0 : bi;
                s_prob[j] = expf(bv - m) / z;
            }
            __syncthreads();
            if (head < RT_MAX_K) {   // the owner of the winner moves on to its next entry
                bool mine = false;
#pragma unroll
                for (int jj = 0; jj < RT_MAX_K; ++jj) if (jj == head && ti[jj] == s_top[j]) mine = true;
                if (mine) ++head;
            }
        }
        // the feature vector into shared memory, then the hidden units: warp w takes units w, w + 32, ...; lanes
        // stride over the features (the weight row is read coalesced, eight loads in flight per lane)
        const int F = 1 + r.k + r.k * d;
        for (int f = tid; f < F; f += RT_THREADS) {
            float x;
            if (f == 0) x = entropy;
            else if (f <= r.k) x = s_prob[f - 1];
            else { const int j = (f - 1 - r.k) / d, e = (f - 1 - r.k) - j * d; x = to_float(emb[(size_t)s_top[j] * d + e]); }
            s_x[f] = x;
        }
        __syncthreads();
        float acc = 0.f;                                  // this warp's share of w2 . relu(hidden)
        for (int u = warp; u < r.hidden; u += RT_WARPS) {
            const float* wr = r.w1 + (size_t)u * F;
            float dot = 0.f;
#pragma unroll 8
            for (int f = lane; f < F; f += 32) dot = fmaf(__ldg(wr + f), s_x[f], dot);
            dot = warp_sum(dot) + __ldg(r.b1 + u);
            acc = fmaf(__ldg(r.w2 + u), fmaxf(dot, 0.f), acc);
        }
        __syncthreads();
        if (lane == 0) s_hid[warp] = acc;
        __syncthreads();
        if (tid == 0) {
            float pre = r.b2;
            for (int w = 0; w < RT_WARPS; ++w) pre += s_hid[w];
            const float disagree = 1.0f / (1.0f + expf(-pre));
            const float conf = 1.0f - disagree;
            st.block_len[b] = s + 1;
            st.confidence[b * st.gamma_limit + s] = conf;
            if (!(conf >= r.tau) || s + 1 >= gamma_max) {
                st.drafting[b] = 0;
                atomicSub(st.counters + 7, 1);
            }
        }
    }
    // the last CTA of the launch publishes to the host: data first, then the ticket it polls on
    if (tid == 0) {
        __threadfence();
        const int t = atomicAdd(st.counters + 9, 1);
        if (t == batch - 1) {
            st.counters[9] = 0;
            __threadfence();
            const int ticket = st.counters[8] + 1;
            st.counters[8] = ticket;
            st.host_flags[6] = atomicAdd(st.counters + 7, 0);
            __threadfence_system();
            st.host_flags[5] = ticket;
        }
    }
}

}  // namespace tandem
