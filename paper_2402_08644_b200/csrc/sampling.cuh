// Sampled Tandem + SPEED (Section 3.1 builds on the SPEED / speculative-decoding framework): drafts are drawn from
// the small model's distribution q = softmax(logits_S / T_S); draft r is kept with probability min(1, p(d_r) / q(d_r)),
// p = softmax(logits_L / T_L); at the first rejection the token is redrawn from the positive part of p - q; if every
// draft is kept, one more token is drawn from the large model's next distribution.
//
// Every draw uses one uniform variate from a counter-based generator keyed by (seed, sequence, iteration, slot):
// slots 0..gamma-1 draw the drafts, 16 + r tests draft r, 48 redraws.  A draw from weights w with variate u returns
// the first index whose running sum exceeds u * sum(w).  The running sums are fp32: thread t of the block owns the
// contiguous segment [t * seg, (t + 1) * seg) and adds it front to back, the segments' sums are scanned in thread
// order, and the thread whose segment contains the target walks it again in the same order.
#pragma once
#include <math.h>
#include "common.cuh"
#include "misc_kernels.cuh"
#include "tc_common.cuh"

namespace tandem {

constexpr int SMP_THREADS = 256;
constexpr int SMP_SLOT_ACCEPT = 16;
constexpr int SMP_SLOT_REDRAW = 48;

__device__ __forceinline__ float uniform_variate(unsigned long long seed, int seq, int iteration, int slot) {
    const unsigned long long x = splitmix64(splitmix64(splitmix64(splitmix64(seed) ^ (unsigned long long)seq) ^ (unsigned long long)iteration) ^
                                            (unsigned long long)slot);
    return (float)(x >> 40) * (1.0f / 16777216.0f);   // 24 bits: exact in fp32
}

// Block-wide reductions over SMP_THREADS threads; `red` holds 8 floats.  Every thread gets the result.
__device__ __forceinline__ float smp_block_max(float v, float* red) {
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
#pragma unroll
    for (int w = 1; w < SMP_THREADS / 32; ++w) r = fmaxf(r, red[w]);
    return r;
}

// Maximum of row[0..V).
__device__ __forceinline__ float smp_row_max(const float* row, int V, float* red) {
    float m = -INFINITY;
    for (int i = threadIdx.x; i < V; i += SMP_THREADS) m = fmaxf(m, __ldcg(row + i));
    return smp_block_max(m, red);
}

// Inverse-CDF draw from the non-negative weights w(i), i in [0, V), with variate u in [0, 1).
// scan: SMP_THREADS floats of shared memory; s_pick: one int.  Every thread returns the drawn index.
// Also returns the total of the weights through *total_out (nullable).
template <typename W>
__device__ __forceinline__ int smp_draw(W w, int V, float u, float* scan, int* s_pick, float* total_out) {
    const int tid = threadIdx.x;
    const int seg = (V + SMP_THREADS - 1) / SMP_THREADS;
    const int i0 = min(V, tid * seg), i1 = min(V, i0 + seg);
    float local = 0.f;
    int last_pos = -1;
    for (int i = i0; i < i1; ++i) {
        const float x = w(i);
        local += x;
        if (x > 0.f) last_pos = i;
    }
    __syncthreads();
    scan[tid] = local;
    if (tid == 0) *s_pick = -1;
    __syncthreads();
    if (tid == 0) {   // inclusive scan of the segments' sums in thread order (256 additions, one thread: a fixed order)
        float run = 0.f;
        for (int t = 0; t < SMP_THREADS; ++t) { run += scan[t]; scan[t] = run; }
    }
    __syncthreads();
    const float total = scan[SMP_THREADS - 1];
    const float target = u * total;
    const float incl = scan[tid], excl = tid > 0 ? scan[tid - 1] : 0.f;
    if (incl > target && excl <= target) {   // exactly one segment contains the target
        float run = excl;
        int pick = -1;
        for (int i = i0; i < i1; ++i) {
            run += w(i);
            if (run > target) { pick = i; break; }
        }
        if (pick < 0) pick = last_pos;       // rounding: the segment's own walk fell just short
        *s_pick = pick;
    }
    __syncthreads();
    if (*s_pick < 0) {   // rounding left no index beyond the target: the last index with a positive weight
        __syncthreads();
        atomicMax(s_pick, last_pos);
        __syncthreads();
    }
    if (total_out) *total_out = total;
    return max(*s_pick, 0);   // (all weights zero: index 0)
}

// Draft s of every live sequence, drawn from softmax(logits / temp).  logits: [batch][V] of draft step s.
// grid: batch; block: SMP_THREADS.
__global__ void __launch_bounds__(SMP_THREADS) sample_draft_kernel(LoopState st, const float* __restrict__ logits, int V, int s,
                                                                   float temp, unsigned long long seed) {
    __shared__ float red[8], scan[SMP_THREADS];
    __shared__ int s_pick;
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x;
    const float* row = logits + (size_t)b * V;
    const float m = smp_row_max(row, V, red);
    const float inv_t = 1.0f / temp;
    const float u = uniform_variate(seed, b, st.counters[0], s);
    const int tok = smp_draw([&](int i) { return expf((__ldcg(row + i) - m) * inv_t); }, V, u, scan, &s_pick, nullptr);
    if (threadIdx.x == 0) st.drafts[b * st.gamma_limit + s] = tok;
}

// Accept / redraw decisions of one iteration, one CTA per sequence: writes accept_len[b] and, at index accept_len of
// the sequence's target array, the token that follows the kept drafts.  The bookkeeping (emit, advance n, publish)
// is done by verify_kernel in mode 4, which takes these decisions as given.
// logits_large: [batch][gamma+1][V]; logits_small: [gamma][batch][V].  grid: batch; block: SMP_THREADS.
__global__ void __launch_bounds__(SMP_THREADS) sample_verify_kernel(LoopState st, int batch, int gamma, const float* __restrict__ logits_large,
                                                                    const float* __restrict__ logits_small, int V, float temp_large,
                                                                    float temp_small, unsigned long long seed) {
    __shared__ float red[8], scan[SMP_THREADS];
    __shared__ int s_pick;
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x;
    if (st.done[b]) return;
    const int iteration = st.counters[0];
    const float inv_tl = 1.0f / temp_large, inv_ts = 1.0f / temp_small;
    const int* d = st.drafts + b * st.gamma_limit;
    int a = 0;
    float mL = 0.f, mS = 0.f, zL = 1.f, zS = 1.f;
    const float* lrow = logits_large + (size_t)b * (gamma + 1) * V;
    const float* srow = nullptr;
    for (; a < gamma; ++a) {
        lrow = logits_large + ((size_t)b * (gamma + 1) + a) * V;
        srow = logits_small + ((size_t)a * batch + b) * V;
        mL = smp_row_max(lrow, V, red);
        mS = smp_row_max(srow, V, red);
        // the two normalisers, each summed in the draw's own order (segments front to back, then in thread order)
        smp_draw([&](int i) { return expf((__ldcg(lrow + i) - mL) * inv_tl); }, V, 0.f, scan, &s_pick, &zL);
        smp_draw([&](int i) { return expf((__ldcg(srow + i) - mS) * inv_ts); }, V, 0.f, scan, &s_pick, &zS);
        const int tok = d[a];
        const float pL = expf((__ldcg(lrow + tok) - mL) * inv_tl) / zL;
        const float pS = expf((__ldcg(srow + tok) - mS) * inv_ts) / zS;
        const float ratio = pS > 0.f ? fminf(1.0f, pL / pS) : 1.0f;
        const float u = uniform_variate(seed, b, iteration, SMP_SLOT_ACCEPT + a);
        if (!(u < ratio)) break;   // rejected: redraw below from this position's distributions
    }
    const float u = uniform_variate(seed, b, iteration, SMP_SLOT_REDRAW);
    int tok;
    if (a < gamma) {
        const float* lr = lrow;
        const float* sr = srow;
        const float cl = 1.0f / zL, cs = 1.0f / zS;
        tok = smp_draw([&](int i) {
            return fmaxf(expf((__ldcg(lr + i) - mL) * inv_tl) * cl - expf((__ldcg(sr + i) - mS) * inv_ts) * cs, 0.f);
        }, V, u, scan, &s_pick, nullptr);
    } else {
        const float* lr = logits_large + ((size_t)b * (gamma + 1) + gamma) * V;
        const float m = smp_row_max(lr, V, red);
        tok = smp_draw([&](int i) { return expf((__ldcg(lr + i) - m) * inv_tl); }, V, u, scan, &s_pick, nullptr);
    }
    if (threadIdx.x == 0) {
        st.accept_len[b] = a;
        st.targets[b * (st.gamma_limit + 1) + a] = tok;
    }
}

}  // namespace tandem
