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
    TC_PROBE_INIT(LOOP ? 201 : 200);
    pdl_wait();                // queries and keys/values come from earlier kernels
    pdl_launch_dependents();   // the next kernel may start fetching its weights
    if (threadIdx.x == 0) TC_PROBE(1);
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
        if (threadIdx.x == 0) TC_PROBE(2);

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

        if (threadIdx.x == 0) TC_PROBE(3);
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

        if (threadIdx.x == 0) TC_PROBE(4);
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
        if (threadIdx.x == 0) TC_PROBE(5);
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) TC_PROBE(6);
        if (tid == 0) {
            const int active = min((int)gridDim.x, pos_last / ATT_CH + 1);   // CTAs that got this far
            int* counter = a.merge_counters + (size_t)g * a.n_heads + h;
            const int t = atomicAdd(counter, 1);
            s_last = (t == active - 1);
            if (t == active - 1) *counter = 0;   // ready for the next launch
        }
        __syncthreads();
        if (threadIdx.x == 0) TC_PROBE(7);
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
        if (threadIdx.x == 0) TC_PROBE(8);
    }
}

// ---------------------------------------------------------------------------------------------------
// Decode attention, bf16, built for short dependent chains and for streaming: a cluster of CL CTAs (1, 2, 4 or 8,
// fixed per launch configuration) serves one (sequence, head).  CTA `rank` takes the 128-position chunks rank, rank + CL, ... (anchored at
// absolute position 0); inside a chunk warp w owns positions 16w .. 16w+15.  Every warp runs on its own: it
// fetches its rows through a private cp.async ring, keeps an online-softmax state per query in registers and
// never waits for another warp until the end, where the CTA folds its warps' states in warp order, sends the
// result to the CTA that finishes the query (remote shared-memory stores), and that CTA merges the CL
// states in rank order.  No global scratch, no second kernel.  DH / 8 lanes share a key (16 bytes each); a
// query's arithmetic does not depend on the other queries.  The probabilities use the fast exponential
// (2^x hardware approximation), well inside the bf16 tolerance.
// ---------------------------------------------------------------------------------------------------
constexpr int ATD_THREADS = 256;
constexpr int ATD_WARPS = ATD_THREADS / 32;
constexpr int ATD_CLUSTER = 8;                                      // largest cluster; launches use 1, 2, 4 or 8
constexpr int ATD_SLOTS = ATT_NQ;                                   // inbox states per CTA: cluster size x queries it finishes <= 16
constexpr int ATD_WROWS = ATT_CH / ATD_WARPS;                       // positions of a chunk per warp (16)

template <int DH> struct AtdCfg {
    static constexpr int TPK = DH / 8;               // lanes per key
    static constexpr int KPW = 32 / TPK;             // keys per warp pass
    static constexpr int PPW = ATD_WROWS / KPW;      // passes per chunk
    static constexpr int STAGES = DH <= 64 ? 3 : 2;
    static constexpr int TILE_ELEMS = ATD_WROWS * DH;   // a warp's keys (or values) of one chunk
    static constexpr int STAGE_ELEMS = 2 * TILE_ELEMS;
    static constexpr int UNITS = ATD_WROWS * TPK / 32;  // 16-byte units per lane per tile
};
template <int DH, int QG>
constexpr size_t attn_decode_smem_bytes() {
    return (size_t)ATD_WARPS * AtdCfg<DH>::STAGES * AtdCfg<DH>::STAGE_ELEMS * sizeof(bf16) +
           sizeof(float) * ((size_t)ATT_NQ * DH + (size_t)ATD_WARPS * QG * (DH + 2) + (size_t)ATD_SLOTS * (DH + 2));
}

// grid: (CL, heads, sequences) with the CL CTAs along x forming one cluster, CL in {1, 2, 4, 8}; block: ATD_THREADS.
template <int DH, int QG>
__global__ void __launch_bounds__(ATD_THREADS) attn_decode_kernel(AttnArgs a) {
    using C = AtdCfg<DH>;
    constexpr int NW = ATD_WARPS;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    bf16* ring_all = reinterpret_cast<bf16*>(smem_raw);
    float* qs = reinterpret_cast<float*>(ring_all + (size_t)NW * C::STAGES * C::STAGE_ELEMS);   // [ATT_NQ][DH]
    float* wst = qs + ATT_NQ * DH;                 // [NW][QG][DH + 2] the warps' states of the current query group
    float* inbox = wst + NW * QG * (DH + 2);       // [CL][QPC][DH + 2] states sent by the cluster's CTAs
    TC_PROBE_INIT(210);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = blockIdx.x, h = blockIdx.y, g = blockIdx.z;
    const int CL = gridDim.x;                      // cluster size
    const int QPC = (ATT_NQ + CL - 1) / CL;        // queries a CTA finishes at most
    const int part = lane % C::TPK, kslot = lane / C::TPK;
    bf16* ring = ring_all + (size_t)warp * C::STAGES * C::STAGE_ELEMS;
    pdl_wait();   // queries and the newest keys/values come from earlier kernels
    pdl_launch_dependents();
    if (tid == 0) TC_PROBE(1);
    const int cnt = a.nq, row0 = g * a.nq;
    const bf16* qg = static_cast<const bf16*>(a.q);
    for (int i = tid; i < cnt * DH; i += ATD_THREADS) {
        const int qi = i / DH, el = i - qi * DH;
        qs[i] = to_float(qg[(size_t)(row0 + qi) * a.ldq + h * DH + el]);
    }
    const int b = a.row_seq[row0];
    const int pos_first = a.row_pos[row0];
    const int pos_last = pos_first + cnt - 1;
    const int n_chunks = pos_last / ATT_CH + 1;
    const int n_mine = rank < n_chunks ? (n_chunks - rank + CL - 1) / CL : 0;
    const size_t head_base = ((size_t)b * a.n_heads + h) * a.t_max;
    const size_t head_base2 = ((size_t)b * a.n_heads + h) * a.t_max2;
    const int split = a.k2 ? a.split : INT_MAX;

    // this warp's rows of its CTA's it-th chunk into stage it % STAGES
    auto issue = [&](int it) {
        const int t0 = (rank + it * CL) * ATT_CH + warp * ATD_WROWS;
        bf16* ks = ring + (size_t)(it % C::STAGES) * C::STAGE_ELEMS;
        bf16* vs = ks + C::TILE_ELEMS;
#pragma unroll
        for (int u = 0; u < C::UNITS; ++u) {
            const int idx = lane + 32 * u;
            const int t = idx / C::TPK, v = idx - t * C::TPK;
            const int ta = t0 + t;
            if (ta <= pos_last) {
                const bf16 *kg, *vg;
                if (ta < split) {
                    kg = static_cast<const bf16*>(a.kcache) + (head_base + ta) * DH;
                    vg = static_cast<const bf16*>(a.vcache) + (head_base + ta) * DH;
                } else {
                    kg = static_cast<const bf16*>(a.k2) + (head_base2 + (ta - split)) * DH;
                    vg = static_cast<const bf16*>(a.v2) + (head_base2 + (ta - split)) * DH;
                }
                cp_async16(ks + idx * 8, kg + v * 8);
                cp_async16(vs + idx * 8, vg + v * 8);
            } else {   // past the last query: zeros, so that a zero weight times them stays zero
                *reinterpret_cast<uint4*>(ks + idx * 8) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4*>(vs + idx * 8) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
    };
    __syncthreads();   // qs written
    if (tid == 0) TC_PROBE(2);

    for (int q0 = 0; q0 < cnt; q0 += QG) {
#pragma unroll
        for (int it = 0; it < C::STAGES - 1; ++it) {
            if (it < n_mine) issue(it);
            cp_async_commit();
        }
        float qreg[QG][8];
#pragma unroll
        for (int qi = 0; qi < QG; ++qi)
#pragma unroll
            for (int j = 0; j < 8; ++j) qreg[qi][j] = (q0 + qi < cnt) ? qs[(q0 + qi) * DH + part * 8 + j] : 0.f;
        float m[QG], l[QG], acc[QG][8];
#pragma unroll
        for (int qi = 0; qi < QG; ++qi) {
            m[qi] = -INFINITY; l[qi] = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[qi][j] = 0.f;
        }
        for (int it = 0; it < n_mine; ++it) {
            if (it + C::STAGES - 1 < n_mine) issue(it + C::STAGES - 1);
            cp_async_commit();
            asm volatile("cp.async.wait_group %0;" ::"n"(C::STAGES - 1) : "memory");
            __syncwarp();
            if (tid == 0 && it == 0 && q0 == 0) TC_PROBE(3);
            const int t0 = (rank + it * CL) * ATT_CH + warp * ATD_WROWS;
            const bf16* ks = ring + (size_t)(it % C::STAGES) * C::STAGE_ELEMS;
            const bf16* vs = ks + C::TILE_ELEMS;
            if constexpr (QG == 4) {
                // Four queries: the DH/8 lanes of a key split the four dot products among themselves while they add
                // them up (a reduce-scatter with the same pairing, hence the same bits, as the one-query butterfly):
                // the lane whose low position bits are (b0, b1) ends up with query 2*b0 + b1 and does that query's
                // softmax step; probabilities and rescale factors are then handed round within the key's lanes.
                const bool b0 = (part & 1) != 0, b1 = (part & 2) != 0;
                const int qsel = (b0 ? 2 : 0) + (b1 ? 1 : 0);
                const int key_lane0 = lane & ~(C::TPK - 1);
                const bool q_live = q0 + qsel < cnt;
                const int q_pos = pos_first + q0 + qsel;
                float sp[C::PPW];
                float mcm = -INFINITY;
#pragma unroll
                for (int p = 0; p < C::PPW; ++p) {
                    const int key = p * C::KPW + kslot;
                    float kf[8];
                    load_vec(ks + key * DH + part * 8, kf);
                    float d[4];
#pragma unroll
                    for (int qi = 0; qi < 4; ++qi) {
                        d[qi] = 0.f;
#pragma unroll
                        for (int j = 0; j < 8; ++j) d[qi] = fmaf(qreg[qi][j], kf[j], d[qi]);
                    }
                    const float r0 = __shfl_xor_sync(0xffffffffu, b0 ? d[0] : d[2], 1);
                    const float r1 = __shfl_xor_sync(0xffffffffu, b0 ? d[1] : d[3], 1);
                    const float e0 = (b0 ? d[2] : d[0]) + r0, e1 = (b0 ? d[3] : d[1]) + r1;
                    const float r2 = __shfl_xor_sync(0xffffffffu, b1 ? e0 : e1, 2);
                    float dq = (b1 ? e1 : e0) + r2;
#pragma unroll
                    for (int o = 4; o < C::TPK; o <<= 1) dq += __shfl_xor_sync(0xffffffffu, dq, o);
                    sp[p] = (q_live && t0 + key <= q_pos) ? dq * a.scale : -INFINITY;
                    mcm = fmaxf(mcm, sp[p]);
                }
#pragma unroll
                for (int o = C::TPK; o < 32; o <<= 1) mcm = fmaxf(mcm, __shfl_xor_sync(0xffffffffu, mcm, o));
                const float mn = fmaxf(m[0], mcm);
                const float fm = m[0] > -INFINITY ? __expf(m[0] - mn) : 0.f;
                m[0] = mn;
                float ls = 0.f;
#pragma unroll
                for (int p = 0; p < C::PPW; ++p) {
                    sp[p] = mn > -INFINITY ? __expf(sp[p] - mn) : 0.f;
                    ls += sp[p];
                }
                l[0] = l[0] * fm + ls;   // this lane's keys only; the key slots are added up at the end
#pragma unroll
                for (int qi = 0; qi < 4; ++qi) {
                    const float fq = __shfl_sync(0xffffffffu, fm, key_lane0 | ((qi >> 1) | ((qi & 1) << 1)));
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[qi][j] *= fq;
                }
#pragma unroll
                for (int p = 0; p < C::PPW; ++p) {
                    const int key = p * C::KPW + kslot;
                    float vf[8];
                    load_vec(vs + key * DH + part * 8, vf);
#pragma unroll
                    for (int qi = 0; qi < 4; ++qi) {
                        const float pq = __shfl_sync(0xffffffffu, sp[p], key_lane0 | ((qi >> 1) | ((qi & 1) << 1)));
#pragma unroll
                        for (int j = 0; j < 8; ++j) acc[qi][j] = fmaf(pq, vf[j], acc[qi][j]);
                    }
                }
            } else {
            float sc[QG][C::PPW], mc[QG];
#pragma unroll
            for (int qi = 0; qi < QG; ++qi) mc[qi] = -INFINITY;
#pragma unroll
            for (int p = 0; p < C::PPW; ++p) {
                const int key = p * C::KPW + kslot;
                float kf[8];
                load_vec(ks + key * DH + part * 8, kf);
#pragma unroll
                for (int qi = 0; qi < QG; ++qi) {
                    float d = 0.f;
#pragma unroll
                    for (int j = 0; j < 8; ++j) d = fmaf(qreg[qi][j], kf[j], d);
#pragma unroll
                    for (int o = 1; o < C::TPK; o <<= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
                    const bool live = (q0 + qi < cnt) && (t0 + key <= pos_first + q0 + qi);
                    sc[qi][p] = live ? d * a.scale : -INFINITY;
                    mc[qi] = fmaxf(mc[qi], sc[qi][p]);
                }
            }
#pragma unroll
            for (int qi = 0; qi < QG; ++qi) {
#pragma unroll
                for (int o = C::TPK; o < 32; o <<= 1) mc[qi] = fmaxf(mc[qi], __shfl_xor_sync(0xffffffffu, mc[qi], o));
                const float mn = fmaxf(m[qi], mc[qi]);
                const float f = m[qi] > -INFINITY ? __expf(m[qi] - mn) : 0.f;
                m[qi] = mn;
                float ls = 0.f;
#pragma unroll
                for (int p = 0; p < C::PPW; ++p) {
                    const float pr = mn > -INFINITY ? __expf(sc[qi][p] - mn) : 0.f;
                    sc[qi][p] = pr;
                    ls += pr;
                }
                l[qi] = l[qi] * f + ls;   // this lane's keys only; the key slots are added up at the end
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[qi][j] *= f;
            }
#pragma unroll
            for (int p = 0; p < C::PPW; ++p) {
                const int key = p * C::KPW + kslot;
                float vf[8];
                load_vec(vs + key * DH + part * 8, vf);
#pragma unroll
                for (int qi = 0; qi < QG; ++qi)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[qi][j] = fmaf(sc[qi][p], vf[j], acc[qi][j]);
            }
            }
            __syncwarp();   // the stage may be refilled by this warp's next issue
            if (tid == 0 && it == 0 && q0 == 0) TC_PROBE(8);
        }
        // the warp's state: add up its key slots (lanes that share `part`), lanes 0 .. TPK-1 publish it
        if constexpr (QG == 4) {   // each lane carries the running maximum and sum of one query only
#pragma unroll
            for (int o = C::TPK; o < 32; o <<= 1) l[0] += __shfl_xor_sync(0xffffffffu, l[0], o);
            if (lane < 4) {        // lane = position bits (b0, b1) of key slot 0: query 2*b0 + b1
                float* st = wst + (size_t)(warp * QG + (((lane & 1) << 1) | (lane >> 1))) * (DH + 2);
                st[DH] = m[0]; st[DH + 1] = l[0];
            }
        }
#pragma unroll
        for (int qi = 0; qi < QG; ++qi) {
#pragma unroll
            for (int o = C::TPK; o < 32; o <<= 1) {
                if (QG != 4) l[qi] += __shfl_xor_sync(0xffffffffu, l[qi], o);
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[qi][j] += __shfl_xor_sync(0xffffffffu, acc[qi][j], o);
            }
            if (lane < C::TPK) {
                float* st = wst + (size_t)(warp * QG + qi) * (DH + 2);
#pragma unroll
                for (int j = 0; j < 8; ++j) st[lane * 8 + j] = acc[qi][j];
                if (QG != 4 && lane == 0) { st[DH] = m[qi]; st[DH + 1] = l[qi]; }
            }
        }
        __syncthreads();
        if (tid == 0 && q0 == 0) TC_PROBE(4);
        // fold the warps' states in warp order and send the CTA's state of query qi to CTA qi % 8
        for (int i = tid; i < QG * (DH + 2); i += ATD_THREADS) {
            const int qi = i / (DH + 2), e = i - qi * (DH + 2);
            const int qa = q0 + qi;
            if (qa < cnt) {
                float mx = -INFINITY;
#pragma unroll
                for (int w = 0; w < NW; ++w) mx = fmaxf(mx, wst[(size_t)(w * QG + qi) * (DH + 2) + DH]);
                float val;
                if (e == DH) {
                    val = mx;
                } else {
                    val = 0.f;
#pragma unroll
                    for (int w = 0; w < NW; ++w) {
                        const float* st = wst + (size_t)(w * QG + qi) * (DH + 2);
                        const float f = st[DH] > -INFINITY ? __expf(st[DH] - mx) : 0.f;
                        val = fmaf(e < DH ? st[e] : st[DH + 1], f, val);
                    }
                }
                float* slot = inbox + ((size_t)rank * QPC + qa / CL) * (DH + 2) + e;
                if (CL > 1) st_dsmem_f32(smem_u32(slot), qa % CL, val);
                else *slot = val;
            }
        }
        __syncthreads();   // wst is rewritten by the next query group
    }
    if (CL > 1) cluster_sync_all(); else __syncthreads();
    if (tid == 0) TC_PROBE(5);
    for (int u = 0; u < QPC; ++u) {
        const int qi = rank + u * CL;
        if (qi < cnt && tid < DH) {
            float mx = -INFINITY;
            for (int r = 0; r < CL; ++r) mx = fmaxf(mx, inbox[((size_t)r * QPC + u) * (DH + 2) + DH]);
            float l = 0.f, o = 0.f;
            for (int r = 0; r < CL; ++r) {
                const float* st = inbox + ((size_t)r * QPC + u) * (DH + 2);
                const float f = st[DH] > -INFINITY ? __expf(st[DH] - mx) : 0.f;
                l = fmaf(st[DH + 1], f, l);
                o = fmaf(st[tid], f, o);
            }
            static_cast<bf16*>(a.out)[(size_t)(row0 + qi) * a.ldo + h * DH + tid] = __float2bfloat16_rn(o / l);
        }
    }
    if (tid == 0) TC_PROBE(6);
}

}  // namespace tandem
