// Attention over a KV cache laid out [seq][head][position][d_head].
//
// One kernel serves three uses (Eq. 1 and Eq. 2, second line):
//   * the small model's decode step: one query per (sequence, head) over the mixed context; positions
//     the large model has processed hold large-derived keys/values, later ones the small model's own,
//     in one contiguous cache, so the boundary needs no special handling here;
//   * the large model's block pass: gamma+1 queries per sequence share one sweep over the cache, each
//     limited to its own position (causal inside the block);
//   * the prompt pass (LOOP = true): a group of consecutive queries sweeps all chunks up to its last position.
//
// The context is cut into chunks of ATT_CH positions anchored at absolute position 0.  In split mode one
// CTA handles one chunk and writes (max, sum, weighted values) per query; the CTA of a (group, head)
// that finishes last combines the chunks in position order.  A query's arithmetic never depends on how many other queries ride along,
// so a block pass and single-token passes produce identical bits.
#pragma once
#include <limits.h>
#include <math.h>
#include "common.cuh"
#include "tc_common.cuh"

namespace tandem {

constexpr int ATT_CH = 128;       // positions per chunk
constexpr int ATT_NQ = 16;        // most queries per CTA (gamma limit + 1)
constexpr int ATT_THREADS = 128;

struct AttnArgs {
    const void* q; int ldq;              // T [M][ldq]; head h at columns h*DH..
    const void* kcache; const void* vcache;   // [seq][head][t_max][DH]
    const void* k2; const void* v2;            // optional second segment [seq][head][t_max2][DH] holding
    int split, t_max2;                         //   positions >= split (used when k2 != nullptr)
    void* out; int ldo;                  // T [M][ldo]
    const int* row_seq; const int* row_pos;
    const int* grp_row0; const int* grp_cnt;   // nullable: then group g = rows g*nq .. g*nq+nq-1
    int nq;
    int n_heads, t_max;
    float* part_ml;                      // split mode: [M][H][n_chunks_max][2]
    float* part_acc;                     //             [M][H][n_chunks_max][DH]
    int n_chunks_max;
    float scale;
    int* merge_counters;                 // split mode: [groups][H], zero between launches
};

template <typename T, int DH>
constexpr size_t attn_smem_bytes() {
    return (size_t)2 * ATT_CH * (DH + VecN<T>::N) * sizeof(T) + (size_t)ATT_NQ * DH * sizeof(float) +
           (size_t)ATT_NQ * ATT_CH * sizeof(float) + (size_t)2 * ATT_NQ * sizeof(float);
}

// grid: (chunks, heads, groups) in split mode; (1, heads, groups) in loop mode.
template <typename T, int DH, bool LOOP>
__global__ void __launch_bounds__(ATT_THREADS) attn_kernel(AttnArgs a) {
    constexpr int VN = VecN<T>::N;
    constexpr int LD = DH + VN;                 // padded row: keeps 16-byte alignment, spreads banks
    constexpr int VPR = DH / VN;                // 16-byte vectors per row
    constexpr int QS = ATT_THREADS / DH;        // query stride of the value phase
    constexpr int QPT = (ATT_NQ + QS - 1) / QS; // queries per thread in the value phase
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int s_last;
    pdl_launch_dependents();   // the next kernel may start fetching its weights
    pdl_wait();                // queries and keys/values come from earlier kernels
    T* ks = reinterpret_cast<T*>(smem_raw);
    T* vs = ks + ATT_CH * LD;
    float* qs = reinterpret_cast<float*>(vs + ATT_CH * LD);
    float* ss = qs + ATT_NQ * DH;
    float* cm = ss + ATT_NQ * ATT_CH;
    float* cl = cm + ATT_NQ;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = blockIdx.z, h = blockIdx.y;
    const int row0 = a.grp_row0 ? a.grp_row0[g] : g * a.nq;
    const int cnt = a.grp_cnt ? a.grp_cnt[g] : a.nq;
    if (cnt <= 0) return;
    const int b = a.row_seq[row0];
    const int pos_first = a.row_pos[row0];
    const int pos_last = pos_first + cnt - 1;
    const int c_begin = LOOP ? 0 : blockIdx.x;
    const int c_end = LOOP ? pos_last / ATT_CH + 1 : blockIdx.x + 1;
    if (c_begin * ATT_CH > pos_last) return;

    const T* qg = static_cast<const T*>(a.q);
    for (int i = tid; i < cnt * DH; i += ATT_THREADS) {
        const int qi = i / DH, el = i - qi * DH;
        qs[qi * DH + el] = to_float(qg[(size_t)(row0 + qi) * a.ldq + h * DH + el]);
    }

    const int e = tid % DH, qsub = tid / DH;
    float racc[QPT], rm[QPT], rl[QPT];
#pragma unroll
    for (int i = 0; i < QPT; ++i) { racc[i] = 0.f; rm[i] = -INFINITY; rl[i] = 0.f; }

    const size_t head_base = ((size_t)b * a.n_heads + h) * a.t_max;
    const size_t head_base2 = ((size_t)b * a.n_heads + h) * a.t_max2;
    const int split = a.k2 ? a.split : INT_MAX;
    for (int c = c_begin; c < c_end; ++c) {
        const int t0 = c * ATT_CH;
        const int nt = min(ATT_CH, pos_last + 1 - t0);
        __syncthreads();   // previous chunk fully consumed (and qs written, first time round)
        for (int i = tid; i < nt * VPR; i += ATT_THREADS) {
            const int t = i / VPR, v = i - t * VPR;
            const int ta = t0 + t;
            const T* kg;
            const T* vg;
            if (ta < split) {
                kg = static_cast<const T*>(a.kcache) + (head_base + ta) * DH;
                vg = static_cast<const T*>(a.vcache) + (head_base + ta) * DH;
            } else {
                kg = static_cast<const T*>(a.k2) + (head_base2 + (ta - split)) * DH;
                vg = static_cast<const T*>(a.v2) + (head_base2 + (ta - split)) * DH;
            }
            cp_async16(ks + t * LD + v * VN, kg + v * VN);
            cp_async16(vs + t * LD + v * VN, vg + v * VN);
        }
        cp_async_commit();
        cp_async_wait_all();
        __syncthreads();

        // scores: thread t owns key t0+t for every query
        for (int t = tid; t < nt; t += ATT_THREADS) {
            float dot[ATT_NQ];
#pragma unroll
            for (int qi = 0; qi < ATT_NQ; ++qi) dot[qi] = 0.f;
#pragma unroll 2
            for (int v = 0; v < VPR; ++v) {
                float kv[VN];
                load_vec(ks + t * LD + v * VN, kv);
#pragma unroll
                for (int qi = 0; qi < ATT_NQ; ++qi) {
                    if (qi < cnt) {
#pragma unroll
                        for (int i = 0; i < VN; ++i) dot[qi] = fmaf(qs[qi * DH + v * VN + i], kv[i], dot[qi]);
                    }
                }
            }
#pragma unroll
            for (int qi = 0; qi < ATT_NQ; ++qi)
                if (qi < cnt) ss[qi * ATT_CH + t] = (t0 + t <= pos_first + qi) ? dot[qi] * a.scale : -INFINITY;
        }
        __syncthreads();

        // per query: chunk max, exponentials, chunk sum
        for (int qi = warp; qi < cnt; qi += ATT_THREADS / 32) {
            float m = -INFINITY;
            for (int t = lane; t < nt; t += 32) m = fmaxf(m, ss[qi * ATT_CH + t]);
            m = warp_max(m);
            float l = 0.f;
            if (m > -INFINITY) {
                for (int t = lane; t < nt; t += 32) {
                    const float p = expf(ss[qi * ATT_CH + t] - m);
                    ss[qi * ATT_CH + t] = p;
                    l += p;
                }
                l = warp_sum(l);
            }
            if (lane == 0) { cm[qi] = m; cl[qi] = l; }
        }
        __syncthreads();

        // weighted values: thread owns element e for queries qsub, qsub+QS, ...
#pragma unroll
        for (int i = 0; i < QPT; ++i) {
            const int qi = qsub + i * QS;
            if (qi < cnt && cm[qi] > -INFINITY) {
                float o = 0.f;
                for (int t = 0; t < nt; ++t) o = fmaf(ss[qi * ATT_CH + t], to_float(vs[t * LD + e]), o);
                if (LOOP) {
                    const float m_new = fmaxf(rm[i], cm[qi]);
                    const float f_old = expf(rm[i] - m_new), f_new = expf(cm[qi] - m_new);
                    racc[i] = racc[i] * f_old + o * f_new;
                    rl[i] = rl[i] * f_old + cl[qi] * f_new;
                    rm[i] = m_new;
                } else {
                    const size_t p = ((size_t)(row0 + qi) * a.n_heads + h) * a.n_chunks_max + c;
                    a.part_acc[p * DH + e] = o;
                    if (e == 0) { a.part_ml[p * 2] = cm[qi]; a.part_ml[p * 2 + 1] = cl[qi]; }
                }
            }
        }
    }
    T* og = static_cast<T*>(a.out);
    if (LOOP) {
#pragma unroll
        for (int i = 0; i < QPT; ++i) {
            const int qi = qsub + i * QS;
            if (qi < cnt) og[(size_t)(row0 + qi) * a.ldo + h * DH + e] = from_float<T>(racc[i] / rl[i]);
        }
    } else {
        // The CTA that finishes last for this (group, head) merges every query's chunks in position order.
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int active = min((int)gridDim.x, pos_last / ATT_CH + 1);   // CTAs that got this far
            int* counter = a.merge_counters + (size_t)g * a.n_heads + h;
            const int t = atomicAdd(counter, 1);
            s_last = (t == active - 1);
            if (t == active - 1) *counter = 0;   // ready for the next launch
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
#pragma unroll
        for (int i = 0; i < QPT; ++i) {
            const int qi = qsub + i * QS;
            if (qi >= cnt) continue;
            const int nc = (pos_first + qi) / ATT_CH + 1;
            const size_t base = ((size_t)(row0 + qi) * a.n_heads + h) * a.n_chunks_max;
            float mx = -INFINITY;
#pragma unroll 8
            for (int c = 0; c < nc; ++c) mx = fmaxf(mx, __ldcg(a.part_ml + (base + c) * 2));
            float l = 0.f, o = 0.f;
#pragma unroll 4
            for (int c = 0; c < nc; ++c) {
                const float2 ml = __ldcg(reinterpret_cast<const float2*>(a.part_ml + (base + c) * 2));
                const float pa = __ldcg(a.part_acc + (base + c) * DH + e);
                const float f = expf(ml.x - mx);
                l = fmaf(ml.y, f, l);
                o = fmaf(pa, f, o);
            }
            og[(size_t)(row0 + qi) * a.ldo + h * DH + e] = from_float<T>(o / l);
        }
    }
}

}  // namespace tandem
