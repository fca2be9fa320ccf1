// Row set-up, embedding, LayerNorm, casts, arg-max, and the verify / accept / rollback kernel.
#pragma once
#include <math.h>
#include <limits.h>
#include "common.cuh"
#include "tc_common.cuh"

namespace tandem {

// Device-resident loop state (all int32 arrays live in the caller's arena).
struct LoopState {
    int* n;            // [B] committed tokens per sequence (prompt included); position n-1 is pending
    int* pending;      // [B] the pending token c[n-1]
    int* drafts;       // [B][gamma_limit]   d_1..d_gamma of the current iteration
    int* targets;      // [B][gamma_limit+1] the large model's arg-max per block row
    int* accept_len;   // [B]
    int* emitted;      // [B] tokens written to out_ids since the generate call began
    int* done;         // [B]
    int* out_ids;      // [B][out_cap]
    int* counters;     // [0] iteration index since prefill (advances while sequences are live), [1] live sequences,
                       // [2] error flags, [3] max_b n_b, [4] sum_b n_b, [5] live iterations of the current call,
                       // [6] verify kernels executed since the context was created (the host's ticket),
                       // [7] sequences still drafting (adaptive block length), [8] router launches since the prompt pass,
                       // [9] CTAs of the running router launch that have finished
    volatile int* host_flags;   // mapped pinned host memory: [0] ticket, [1] live, [2] n_max, [3] n_sum, [4] iterations,
                                // [5] router ticket, [6] sequences still drafting
    int* block_len;    // [B] adaptive block length: drafts made in the current iteration
    int* drafting;     // [B] adaptive block length: 1 while the router lets the sequence go on drafting
    float* confidence; // [B][gamma_limit] the router's 1 - s for every draft of the current iteration
    unsigned long long* hist;   // [gamma_limit+1] accept-length histogram of live sequences
    int out_cap;
    int gamma_limit;
};

// Decode rows: sequence b contributes rows r0 .. r0+nq-1 of its block (row 0 = pending token, row r = draft r).
// Row m = b*nq + (r - r0):  token, sequence, absolute position n_b - 1 + r.
__global__ void setup_rows_kernel(LoopState st, int batch, int r0, int nq, int* row_tok, int* row_seq, int* row_pos) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= batch * nq) return;
    const int b = m / nq, r = r0 + (m - b * nq);
    row_tok[m] = (r == 0) ? st.pending[b] : st.drafts[b * st.gamma_limit + r - 1];
    row_seq[m] = b;
    row_pos[m] = st.n[b] - 1 + r;
}

// x^(0) = Emb(t) + Pos(index)  (Eq. 1); fp32 residual stream.  grid: rows; block: 128.
template <typename T>
__global__ void embed_kernel(const int* __restrict__ row_tok, const int* __restrict__ row_pos, const T* __restrict__ emb,
                             const T* __restrict__ pos, float* __restrict__ h, int d) {
    const int m = blockIdx.x;
    const T* er = emb + (size_t)row_tok[m] * d;
    const T* pr = pos + (size_t)row_pos[m] * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) h[(size_t)m * d + i] = to_float(er[i]) + to_float(pr[i]);
}

// Arg-max of one row from the per-tile (value, index) pairs an output-head GEMM left behind; lowest index
// on ties.  Warp-wide; every lane returns the result.
__device__ __forceinline__ int argmax_from_tiles(const float* val, const int* idx, int n_tiles) {
    const int lane = threadIdx.x & 31;
    float bv = -INFINITY;
    int bi = INT_MAX;
    for (int t0 = lane; t0 < n_tiles; t0 += 256) {   // eight loads in flight per lane
        float v[8];
        int ix[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int t = t0 + 32 * u;
            v[u] = t < n_tiles ? __ldcg(val + t) : -INFINITY;
            ix[u] = t < n_tiles ? __ldcg(idx + t) : INT_MAX;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (v[u] > bv || (v[u] == bv && ix[u] < bi)) { bv = v[u]; bi = ix[u]; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    return bi == INT_MAX ? 0 : bi;
}

// Start of a pass over decode rows: row set-up and x^(0) = Emb(t) + Pos(index) in one kernel (Eq. 1).
// Row m = b*nq + (r - r0) carries block row r of sequence b (row 0 = pending token, row r = draft r).
// The token of block row fin_r is not known yet as an id: it is the arg-max of the small model's last
// output-head GEMM, finished here from its per-tile results and recorded as draft fin_r.  grid: rows; block: 128.
template <typename T>
__global__ void __launch_bounds__(128) step_begin_kernel(LoopState st, int r0, int nq, int fin_r, const float* amax_val,
                                                         const int* amax_idx, int amax_stride, int n_tiles, int* row_tok,
                                                         int* row_seq, int* row_pos, const T* __restrict__ emb,
                                                         const T* __restrict__ pos, float* __restrict__ h, int d, float* snap) {
    __shared__ int s_tok, s_pos;
    pdl_wait();
    pdl_launch_dependents();
    const int m = blockIdx.x;
    const int b = m / nq, r = r0 + (m - b * nq);
    if (threadIdx.x < 32) {
        int tok;
        if (r == 0) tok = st.pending[b];
        else if (r == fin_r) tok = argmax_from_tiles(amax_val + (size_t)b * amax_stride, amax_idx + (size_t)b * amax_stride, n_tiles);
        else tok = st.drafts[b * st.gamma_limit + r - 1];
        if (threadIdx.x == 0) {
            if (r == fin_r && r > 0) st.drafts[b * st.gamma_limit + r - 1] = tok;
            const int p = st.n[b] - 1 + r;
            s_tok = tok; s_pos = p;
            row_tok[m] = tok; row_seq[m] = b; row_pos[m] = p;
        }
    }
    __syncthreads();
    const T* er = emb + (size_t)s_tok * d;
    const T* pr = pos + (size_t)s_pos * d;
    for (int i = threadIdx.x; i < d; i += 128) {
        const float v = to_float(er[i]) + to_float(pr[i]);
        h[(size_t)m * d + i] = v;
        if (snap) snap[(size_t)m * d + i] = v;   // copy for the FF_Tandem projection of x^(0)
    }
}

__device__ __forceinline__ float block_sum_128(float v, float* red) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    return red[0] + red[1] + red[2] + red[3];
}

// LayerNorm of fp32 rows (biased variance, eps 1e-5), output in the storage type.  grid: rows; block: 128.
template <typename T>
__global__ void __launch_bounds__(128) layernorm_kernel(const float* __restrict__ x, const float* __restrict__ gain,
                                                        const float* __restrict__ bias, T* __restrict__ out, int d) {
    __shared__ float red[4];
    const float* xr = x + (size_t)blockIdx.x * d;
    float s = 0.f;
    for (int i = threadIdx.x; i < d; i += 128) s += xr[i];
    const float mu = block_sum_128(s, red) / d;
    float v = 0.f;
    for (int i = threadIdx.x; i < d; i += 128) { const float c = xr[i] - mu; v = fmaf(c, c, v); }
    const float rstd = 1.0f / sqrtf(block_sum_128(v, red) / d + 1e-5f);
    for (int i = threadIdx.x; i < d; i += 128)
        out[(size_t)blockIdx.x * d + i] = from_float<T>((xr[i] - mu) * rstd * gain[i] + bias[i]);
}

// Four normalised values to the output row: fp32 as they are, bf16 rounded.
__device__ __forceinline__ void ln_store4(float* orow, int k4, float y0, float y1, float y2, float y3) {
    reinterpret_cast<float4*>(orow)[k4] = make_float4(y0, y1, y2, y3);
}
__device__ __forceinline__ void ln_store4(bf16* orow, int k4, float y0, float y1, float y2, float y3) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(y0, y1), hi = __floats2bfloat162_rn(y2, y3);
    reinterpret_cast<uint2*>(orow)[k4] = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
}
// value plane + remainder plane (x = bf16(x) + bf16(x - bf16(x))), for a GEMM that loads its token rows by TMA
__device__ __forceinline__ void ln_store4_split(bf16* vrow, bf16* rrow, int k4, float y0, float y1, float y2, float y3) {
    const __nv_bfloat162 a = __floats2bfloat162_rn(y0, y1), b = __floats2bfloat162_rn(y2, y3);
    const __nv_bfloat162 ra = __floats2bfloat162_rn(y0 - __low2float(a), y1 - __high2float(a));
    const __nv_bfloat162 rb = __floats2bfloat162_rn(y2 - __low2float(b), y3 - __high2float(b));
    reinterpret_cast<uint2*>(vrow)[k4] = make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b));
    reinterpret_cast<uint2*>(rrow)[k4] = make_uint2(*reinterpret_cast<const uint32_t*>(&ra), *reinterpret_cast<const uint32_t*>(&rb));
}
__device__ __forceinline__ void ln_store4(float* orow, bf16*, int k4, float y0, float y1, float y2, float y3) { ln_store4(orow, k4, y0, y1, y2, y3); }
__device__ __forceinline__ void ln_store4(bf16* orow, bf16* rrow, int k4, float y0, float y1, float y2, float y3) {
    if (rrow) ln_store4_split(orow, rrow, k4, y0, y1, y2, y3);
    else ln_store4(orow, k4, y0, y1, y2, y3);
}

// Decode-path LayerNorm of fp32 rows ahead of the tensor-core GEMMs (fp32 out; bf16 out for the stand-alone
// projection above 64 rows): the row sits in registers between the passes (up to 4096 elements), loads and stores
// are 16 bytes wide.  grid: rows; block: 128; d % 4 == 0.
template <typename TO>
__global__ void __launch_bounds__(128) layernorm_rows_kernel(const float* __restrict__ x, const float* __restrict__ gain,
                                                             const float* __restrict__ bias, TO* __restrict__ out, int d,
                                                             bf16* out_lo = nullptr) {
    __shared__ float red[4];
    const int d4 = d >> 2;
    const float4* xr = reinterpret_cast<const float4*>(x + (size_t)blockIdx.x * d);
    TO* orow = out + (size_t)blockIdx.x * d;
    bf16* rrow = out_lo ? out_lo + (size_t)blockIdx.x * d : nullptr;   // TO = bf16 only: the remainder plane's row
    if (d4 <= 8 * 128) {
        // gains and biases are parameters: fetched while the kernel that writes x is still running
        float4 gq[8], bq[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int k4 = threadIdx.x + 128 * u;
            gq[u] = k4 < d4 ? __ldg(reinterpret_cast<const float4*>(gain) + k4) : make_float4(0.f, 0.f, 0.f, 0.f);
            bq[u] = k4 < d4 ? __ldg(reinterpret_cast<const float4*>(bias) + k4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        pdl_wait();
        pdl_launch_dependents();
        float4 t[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) t[u] = (threadIdx.x + 128 * u < d4) ? __ldcg(xr + threadIdx.x + 128 * u) : make_float4(0.f, 0.f, 0.f, 0.f);
        float s = 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) s += (t[u].x + t[u].y) + (t[u].z + t[u].w);
        const float mu = block_sum_128(s, red) / d;
        float q = 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (threadIdx.x + 128 * u < d4) {
                const float d0 = t[u].x - mu, d1 = t[u].y - mu, d2 = t[u].z - mu, d3 = t[u].w - mu;
                q = fmaf(d0, d0, q); q = fmaf(d1, d1, q); q = fmaf(d2, d2, q); q = fmaf(d3, d3, q);
            }
        }
        const float rs = 1.0f / sqrtf(block_sum_128(q, red) / d + 1e-5f);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int k4 = threadIdx.x + 128 * u;
            if (k4 < d4) {
                const float4 g = gq[u], b = bq[u];
                ln_store4(orow, rrow, k4, (t[u].x - mu) * rs * g.x + b.x, (t[u].y - mu) * rs * g.y + b.y,
                          (t[u].z - mu) * rs * g.z + b.z, (t[u].w - mu) * rs * g.w + b.w);
            }
        }
    } else {
        pdl_wait();
        pdl_launch_dependents();
        float s = 0.f;
        for (int k4 = threadIdx.x; k4 < d4; k4 += 128) { const float4 t = __ldcg(xr + k4); s += (t.x + t.y) + (t.z + t.w); }
        const float mu = block_sum_128(s, red) / d;
        float q = 0.f;
        for (int k4 = threadIdx.x; k4 < d4; k4 += 128) {
            const float4 t = __ldcg(xr + k4);
            const float d0 = t.x - mu, d1 = t.y - mu, d2 = t.z - mu, d3 = t.w - mu;
            q = fmaf(d0, d0, q); q = fmaf(d1, d1, q); q = fmaf(d2, d2, q); q = fmaf(d3, d3, q);
        }
        const float rs = 1.0f / sqrtf(block_sum_128(q, red) / d + 1e-5f);
        for (int k4 = threadIdx.x; k4 < d4; k4 += 128) {
            const float4 t = __ldcg(xr + k4);
            const float4 g = __ldg(reinterpret_cast<const float4*>(gain) + k4), b = __ldg(reinterpret_cast<const float4*>(bias) + k4);
            ln_store4(orow, rrow, k4, (t.x - mu) * rs * g.x + b.x, (t.y - mu) * rs * g.y + b.y, (t.z - mu) * rs * g.z + b.z,
                      (t.w - mu) * rs * g.w + b.w);
        }
    }
}

template <typename T>
__global__ void cast_rows_kernel(const float* __restrict__ x, T* __restrict__ out, size_t n) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = from_float<T>(x[i]);
}

// Arg-max of fp32 rows, lowest index on ties.  grid: rows; block: 256.
// Row m belongs to sequence m / nq; the result goes to dst[(m / nq) * seq_stride + m % nq + off].
__global__ void __launch_bounds__(256) argmax_rows_kernel(const float* __restrict__ logits, int V, int* dst, int nq, int seq_stride, int off) {
    __shared__ float sv[8];
    __shared__ int si[8];
    const float* lr = logits + (size_t)blockIdx.x * V;
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int i = threadIdx.x; i < V; i += 256) {
        const float v = lr[i];
        if (v > best || (v == best && i < bi)) { best = v; bi = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
    }
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = best; si[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w)
            if (sv[w] > best || (sv[w] == best && si[w] < bi)) { best = sv[w]; bi = si[w]; }
        const int m = blockIdx.x;
        dst[(size_t)(m / nq) * seq_stride + (m % nq) + off] = bi;
    }
}

// Verify / accept / rollback (Section 3.1), one thread per sequence, one CTA.
//   a = longest prefix of drafts equal to the large model's tokens (or forced);
//   the sequence gains d_1..d_a and g_{a+1}; n advances; g_{a+1} becomes pending.
// Rolling the caches back is the update of n: positions >= n-1 are rewritten by the next iteration.
// When amax_val is given, the large model's arg-max per block row is first finished from the per-tile results of
// its output-head GEMM.
// mode 3 is the round of stand-alone Tandem without the free token (Section 3 "Inference", "Representation
// Generation Only"; Figure 3): the large model has read gamma rows and predicted nothing, all gamma tokens of the
// small model are kept and the last one becomes pending.  The last draft is then not a block row, so nobody has
// turned it into a token id yet: when fin_val is given it is finished here from the small head's per-tile results.
// mode 4 is sampled SPEED: sample_verify_kernel has already written each sequence's accept length and, at that index
// of its targets, the token drawn after the kept drafts; this kernel only does the bookkeeping.
// block_len (nullable): per-sequence number of drafts of this iteration when the router chose it.
// block: 256.
__global__ void __launch_bounds__(256) verify_kernel(LoopState st, int batch, int gamma, int mode, unsigned long long seed,
                                                     int max_new, const float* amax_val, const int* amax_idx, int amax_stride,
                                                     int n_tiles, const float* fin_val, const int* fin_idx, const int* block_len) {
    pdl_wait();
    pdl_launch_dependents();
    if (mode == 3) {
        if (fin_val != nullptr && gamma > 0) {
            for (int b = threadIdx.x >> 5; b < batch; b += 8) {
                const int tok = argmax_from_tiles(fin_val + (size_t)b * amax_stride, fin_idx + (size_t)b * amax_stride, n_tiles);
                if ((threadIdx.x & 31) == 0) st.drafts[b * st.gamma_limit + gamma - 1] = tok;
            }
        }
        __syncthreads();
    } else if (amax_val != nullptr && mode != 4) {   // (mode 4: the sampled decisions are already in place)
        const int rows = batch * (gamma + 1);
        for (int m = threadIdx.x >> 5; m < rows; m += 8) {
            const int tok = argmax_from_tiles(amax_val + (size_t)m * amax_stride, amax_idx + (size_t)m * amax_stride, n_tiles);
            if ((threadIdx.x & 31) == 0) st.targets[(m / (gamma + 1)) * (st.gamma_limit + 1) + m % (gamma + 1)] = tok;
        }
        __syncthreads();
    }
    const int b = threadIdx.x;
    const int iteration = st.counters[0];
    const int live_before = st.counters[1];
    __syncthreads();
    if (b < batch && !st.done[b]) {
        const int* d = st.drafts + b * st.gamma_limit;
        const int* g = st.targets + b * (st.gamma_limit + 1);
        int a = 0;
        if (mode == 1 || mode == 3) a = gamma;
        else if (mode == 4) a = min(max(st.accept_len[b], 0), gamma);   // sampled SPEED: decided by sample_verify_kernel, with g[a] the token it drew
        else if (mode == 2) a = (int)(splitmix64(splitmix64(splitmix64(seed) ^ (unsigned long long)b) ^ (unsigned long long)iteration) % (unsigned long long)(gamma + 1));
        else {   // adaptive block length: only the drafts the sequence really made count (later rows are dead)
            const int gamma_b = block_len ? min(block_len[b], gamma) : gamma;
            while (a < gamma_b && d[a] == g[a]) ++a;
        }
        st.accept_len[b] = a;
        atomicAdd(st.hist + a, 1ull);
        const int em = st.emitted[b];
        const int room = max_new - em;
        const int take = min(mode == 3 ? a : a + 1, room);
        int last = st.pending[b];
        for (int i = 0; i < take; ++i) {
            last = (i < a) ? d[i] : g[a];
            if (em + i < st.out_cap) st.out_ids[(size_t)b * st.out_cap + em + i] = last;
        }
        st.emitted[b] = em + take;
        st.n[b] += take;
        st.pending[b] = last;
        if (em + take >= max_new) { st.done[b] = 1; atomicSub(st.counters + 1, 1); }
    }
    __syncthreads();
    if (b == 0) {
        if (live_before > 0) { st.counters[0] = iteration + 1; st.counters[5] += 1; }
        int n_max = 0, n_sum = 0;
        for (int i = 0; i < batch; ++i) { n_max = max(n_max, st.n[i]); n_sum += st.n[i]; }
        st.counters[3] = n_max;
        st.counters[4] = n_sum;
        const int ticket = st.counters[6] + 1;
        st.counters[6] = ticket;
        // publish to the host: data first, then the ticket it polls on
        st.host_flags[1] = st.counters[1];
        st.host_flags[2] = n_max;
        st.host_flags[3] = n_sum;
        st.host_flags[4] = st.counters[5];
        __threadfence_system();
        st.host_flags[0] = ticket;
    }
}

// Teacher-forced Tandem forward (Eq. 2 over a given sequence): the next gamma tokens of every sequence become the
// "drafts" of the round, so that draft step s reads the true token of its position.  forced: [batch][stride] token
// ids; positions at or beyond forced_len[b] read as token 0 (rows past a sequence's end are computed and ignored).
// grid: 1; block: 256.
__global__ void __launch_bounds__(256) forced_fill_kernel(LoopState st, int batch, int gamma, const int* __restrict__ forced,
                                                          const int* __restrict__ forced_len, int stride) {
    pdl_wait();
    pdl_launch_dependents();
    for (int i = threadIdx.x; i < batch * gamma; i += 256) {
        const int b = i / gamma, r = i - b * gamma;
        const int p = st.n[b] + r;                       // position of the token that draft r + 1 stands for
        st.drafts[b * st.gamma_limit + r] = p < forced_len[b] ? forced[(size_t)b * stride + p] : 0;
    }
}

// Scores of a teacher-forced round: for draft step s of sequence b, at position p = n_b - 1 + s, the negative
// log-likelihood of the true token at p + 1 under softmax(logits) and the arg-max (lowest id on ties).
// logits: [gamma][batch][V].  grid: (gamma, batch); block: 256.
__global__ void __launch_bounds__(256) score_rows_kernel(LoopState st, int batch, const float* __restrict__ logits, int V,
                                                         const int* __restrict__ forced, const int* __restrict__ forced_len, int stride,
                                                         float* __restrict__ nll, int* __restrict__ top1) {
    __shared__ float sv[8], ss[8];
    __shared__ int si[8];
    pdl_wait();
    pdl_launch_dependents();
    const int s = blockIdx.x, b = blockIdx.y;
    const int p = st.n[b] - 1 + s;
    if (p + 1 >= forced_len[b]) return;                  // no true next token: nothing to score
    const float* row = logits + ((size_t)s * batch + b) * V;
    float best = -INFINITY;
    int bi = INT_MAX;
    for (int i = threadIdx.x; i < V; i += 256) {
        const float v = __ldcg(row + i);
        if (v > best || (v == best && i < bi)) { best = v; bi = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
    }
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = best; si[threadIdx.x >> 5] = bi; }
    __syncthreads();
    for (int w = 0; w < 8; ++w)
        if (sv[w] > best || (sv[w] == best && si[w] < bi)) { best = sv[w]; bi = si[w]; }
    float z = 0.f;
    for (int i = threadIdx.x; i < V; i += 256) z += expf(__ldcg(row + i) - best);
    z = warp_sum(z);
    if ((threadIdx.x & 31) == 0) ss[threadIdx.x >> 5] = z;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
        for (int w = 0; w < 8; ++w) tot += ss[w];
        const int truth = forced[(size_t)b * stride + p + 1];
        nll[(size_t)b * stride + p] = best + logf(tot) - __ldcg(row + truth);
        top1[(size_t)b * stride + p] = bi;
    }
}

// Test hook: gathers K or V of one (layer, sequence) from [H][t_max][dh] into fp32 [n][H*dh].
template <typename T>
__global__ void gather_kv_kernel(const T* __restrict__ cache_seq, float* __restrict__ dst, int n, int n_heads, int d_head, int t_max) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int d = n_heads * d_head;
    if (i >= (size_t)n * d) return;
    const int t = (int)(i / d), c = (int)(i - (size_t)t * d);
    const int h = c / d_head, el = c - h * d_head;
    dst[i] = to_float(cache_seq[((size_t)h * t_max + t) * d_head + el]);
}

}  // namespace tandem
