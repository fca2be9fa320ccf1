// Sampled Tandem + SPEED (Section 3.1 builds on the SPEED / speculative-decoding framework): drafts are drawn from
// the small model's distribution q = softmax(logits_S / T_S); draft r is kept with probability min(1, p(d_r) / q(d_r)),
// p = softmax(logits_L / T_L); at the first rejection the token is redrawn from the positive part of p - q; if every
// draft is kept, one more token is drawn from the large model's next distribution.
//
// Every draw uses one uniform variate from a counter-based generator keyed by (seed, sequence, iteration, slot):
// slots 0..gamma-1 draw the drafts, 16 + r tests draft r, 48 redraws.  A draw from weights w with variate u returns
// the first index whose running sum exceeds u * sum(w).  The running sums are fp32: each warp of the block owns a
// contiguous range of the row, the ranges' sums are scanned in warp order, and the warp whose range contains the
// target walks it again 32 weights at a time.
#pragma once
#include <math.h>
#include "common.cuh"
#include "misc_kernels.cuh"
#include "tc_common.cuh"

namespace tandem {

constexpr int SMP_THREADS = 1024;   // one CTA walks a whole row of logits several times: many loads in flight
constexpr int SMP_WARPS = SMP_THREADS / 32;
constexpr int SMP_SLOT_ACCEPT = 16;
constexpr int SMP_SLOT_REDRAW = 48;

__device__ __forceinline__ float uniform_variate(unsigned long long seed, int seq, int iteration, int slot) {
    const unsigned long long x = splitmix64(splitmix64(splitmix64(splitmix64(seed) ^ (unsigned long long)seq) ^ (unsigned long long)iteration) ^
                                            (unsigned long long)slot);
    return (float)(x >> 40) * (1.0f / 16777216.0f);   // 24 bits: exact in fp32
}

// Block-wide reductions over SMP_THREADS threads; `red` holds SMP_WARPS floats.  Every thread gets the result.
__device__ __forceinline__ float smp_block_max(float v, float* red) {
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
#pragma unroll
    for (int w = 1; w < SMP_WARPS; ++w) r = fmaxf(r, red[w]);
    return r;
}

// Maximum of row[0..V).
__device__ __forceinline__ float smp_row_max(const float* row, int V, float* red) {
    float m = -INFINITY;
    const bool vec = (V & 3) == 0 && (reinterpret_cast<uintptr_t>(row) & 15) == 0;   // 16 bytes at a time, several loads in flight
    const int V4 = vec ? V >> 2 : 0;
#pragma unroll 4
    for (int i4 = threadIdx.x; i4 < V4; i4 += SMP_THREADS) {
        const float4 x = __ldcg(reinterpret_cast<const float4*>(row) + i4);
        m = fmaxf(fmaxf(m, fmaxf(x.x, x.y)), fmaxf(x.z, x.w));
    }
    for (int i = 4 * V4 + threadIdx.x; i < V; i += SMP_THREADS) m = fmaxf(m, __ldcg(row + i));
    return smp_block_max(m, red);
}

// Inverse-CDF draw from the non-negative weights w(i), i in [0, V), with variate u in [0, 1).
// Warp j of the block owns the contiguous range [j * chunk, (j + 1) * chunk).  Pass A: every warp sums its range
// (lanes stride over it, coalesced), the warps' sums are scanned in warp order.  Pass B: the warp whose range
// contains the target u * total walks it again, 32 consecutive weights at a time with a warp-wide running sum, and
// takes the first index whose running sum exceeds the target.
// wsum: SMP_WARPS floats of shared memory; s_pick: one int.  Every thread returns the drawn index; *total_out
// (nullable) receives the total of the weights.
template <typename W>
__device__ __forceinline__ int smp_draw(W w, int V, float u, float* wsum, int* s_pick, float* total_out) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int chunk = (((V + SMP_WARPS - 1) / SMP_WARPS) + 31) & ~31;
    const int i0 = min(V, warp * chunk), i1 = min(V, i0 + chunk);
    float local = 0.f;
    int last_pos = -1;
    for (int i = i0 + lane; i < i1; i += 32) {
        const float x = w(i);
        local += x;
        if (x > 0.f) last_pos = i;
    }
    local = warp_sum(local);
    __syncthreads();
    if (lane == 0) wsum[warp] = local;
    if (tid == 0) *s_pick = -1;
    __syncthreads();
    if (tid == 0) {   // inclusive scan of the warps' sums in warp order
        float run = 0.f;
        for (int t = 0; t < SMP_WARPS; ++t) { run += wsum[t]; wsum[t] = run; }
    }
    __syncthreads();
    const float total = wsum[SMP_WARPS - 1];
    const float target = u * total;
    const float incl = wsum[warp], excl = warp > 0 ? wsum[warp - 1] : 0.f;
    if (incl > target && excl <= target) {   // exactly one warp's range contains the target (warp-uniform condition)
        float run = excl;
        int pick = -1;
        for (int base = i0; base < i1 && pick < 0; base += 32) {
            const int i = base + lane;
            float p = i < i1 ? w(i) : 0.f;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {   // inclusive running sum over the 32 lanes
                const float q = __shfl_up_sync(0xffffffffu, p, o);
                if (lane >= o) p += q;
            }
            const unsigned hit = __ballot_sync(0xffffffffu, run + p > target);
            if (hit) pick = base + __ffs(hit) - 1;
            run += __shfl_sync(0xffffffffu, p, 31);
        }
        if (pick < 0) {   // rounding: the second walk fell just short of the target: the range's last positive weight
            int lp = last_pos;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lp = max(lp, __shfl_xor_sync(0xffffffffu, lp, o));
            pick = lp;
        }
        if (lane == 0) *s_pick = pick;
    }
    __syncthreads();
    if (*s_pick < 0) {   // rounding left no range beyond the target: the last index with a positive weight
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
    __shared__ float red[SMP_WARPS], scan[SMP_WARPS];
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
    __shared__ float red[SMP_WARPS], scan[SMP_WARPS];
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
