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
    void* out; int ldo;                  // T [M][ldo]; float when out_f32 is set (attn_decode_kernel only)
    int out_f32;
    const int* row_seq; const int* row_pos;
    const int* grp_row0; const int* grp_cnt;   // nullable: then group g = rows g*nq .. g*nq+nq-1
    int nq;
    int n_heads, t_max;
    int n_kv_heads;                      // key/value heads of the caches; 0 = n_heads.  Query head h reads kv head h / (n_heads / n_kv_heads)
    int* err_flag;                       // attn_decode_kernel: where a bounded wait that ran out records its code (nullable)
    void* out_lo;                        // attn_decode_kernel, optional: `out` is then the bf16 plane of the values and this the bf16
                                         // plane of the remainders (fp32 result = value + remainder), both [M][ldo]
    int heads_per_cta;                   // attn_decode_kernel: query heads of one key/value head served by one CTA (their rows share
                                         // the 16-row tile: heads_per_cta * nq <= 16); 0 = 1.  grid.y = n_heads / heads_per_cta
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
    pdl_wait();                // queries and keys/values come from earlier kernels
    pdl_launch_dependents();   // the next kernel may start fetching its weights
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

    const int n_kv = a.n_kv_heads > 0 ? a.n_kv_heads : a.n_heads;
    const int kvh = h / (a.n_heads / n_kv);            // grouped-query attention: several query heads share one key/value head
    const size_t head_base = ((size_t)b * n_kv + kvh) * a.t_max;
    const size_t head_base2 = ((size_t)b * n_kv + kvh) * a.t_max2;
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

// ---------------------------------------------------------------------------------------------------
// Decode attention, bf16, built for short dependent chains and for streaming: a cluster of CL CTAs (1, 2, 4 or 8,
// fixed per launch configuration) serves one (sequence, head).  CTA `rank` takes the 128-position chunks rank,
// rank + CL, ... (anchored at absolute position 0); inside a chunk warp w owns positions 16w .. 16w+15.  Every warp
// runs on its own: it fetches its rows through a private cp.async ring, keeps the online-softmax state of all the
// block's queries (up to 16) in registers and never waits for another warp until the end, where the CTA folds its
// warps' states in warp order, sends the result to the CTA that finishes the query (remote shared-memory stores),
// and that CTA merges the CL states in rank order.  No global scratch, no second kernel.
//
// The two small products of a 16-position tile, S = Q K^T (16 query rows x 16 keys) and O += P V, run on the tensor
// cores as warp-level m16n8k16 MMAs: with scalar FMAs and shuffles a block of gamma+1 queries is bound by
// instruction issue at well under half of the memory bandwidth.  The query rows are the MMA's A rows (absent rows
// are zero), K and V fragments come straight from the ring with ldmatrix (V transposed on the way), the softmax
// works on the accumulator fragments (a row's 16 scores sit in the four lanes of a quad), and each probability
// enters the second product as two bf16 numbers (value and remainder).  An output row depends on its own query row
// only, so a block pass and a one-row pass give the same bits.  The probabilities use the fast exponential
// (2^x hardware approximation), well inside the bf16 tolerance.
// ---------------------------------------------------------------------------------------------------
constexpr int ATD_THREADS = 256;
constexpr int ATD_WARPS = ATD_THREADS / 32;
constexpr int ATD_ERR_EXCHANGE = 5;                                 // error code: the wait for the cluster's states gave up
constexpr int ATD_CLUSTER = 8;                                      // largest cluster; launches use 1, 2, 4 or 8
constexpr int ATD_SLOTS = ATT_NQ;                                   // inbox states per CTA: cluster size x queries it finishes <= 16
constexpr int ATD_WROWS = ATT_CH / ATD_WARPS;                       // positions of a chunk per warp (16)
static_assert(ATD_WROWS == 16 && ATT_NQ == 16, "one m16n8k16 tile per warp and chunk");

template <int DH> struct AtdCfg {
    static constexpr int TPK = DH / 8;               // 16-byte units per key
    static constexpr int STAGES = DH <= 64 ? 3 : 2;
    static constexpr int TILE_ELEMS = ATD_WROWS * DH;   // a warp's keys (or values) of one chunk
    static constexpr int STAGE_ELEMS = 2 * TILE_ELEMS;
    static constexpr int UNITS = ATD_WROWS * TPK / 32;  // 16-byte units per lane per tile
    static constexpr int KSTEPS = DH / 16;           // MMAs along the head dimension for S
    static constexpr int NTILES = DH / 8;            // 8-wide output tiles of O
};
template <int DH>
constexpr size_t attn_decode_smem_bytes() {
    // the warps' rings (reused for the warps' final states) + the inbox of states sent by the cluster's CTAs
    return (size_t)ATD_WARPS * AtdCfg<DH>::STAGES * AtdCfg<DH>::STAGE_ELEMS * sizeof(bf16) + sizeof(float) * (size_t)ATD_SLOTS * (DH + 2);
}
static_assert((size_t)ATD_WARPS * ATT_NQ * (128 + 2) * sizeof(float) <= (size_t)ATD_WARPS * AtdCfg<128>::STAGES * AtdCfg<128>::STAGE_ELEMS * sizeof(bf16) &&
              (size_t)ATD_WARPS * ATT_NQ * (32 + 2) * sizeof(float) <= (size_t)ATD_WARPS * AtdCfg<32>::STAGES * AtdCfg<32>::STAGE_ELEMS * sizeof(bf16),
              "the warps' states fit in the ring");

// Where the 16-byte unit u of ring row r lives within the row: XOR-swizzled so that the eight row addresses of
// one ldmatrix fall into different banks (rows are DH * 2 bytes apart).
template <int DH>
__device__ __forceinline__ int atd_swz(int r, int u) { return u ^ (DH >= 64 ? (r & 7) : ((r >> 1) & 3)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t atd_pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&p);
}

// grid: (CL, heads, sequences) with the CL CTAs along x forming one cluster, CL in {1, 2, 4, 8}; block: ATD_THREADS.
template <int DH>
__global__ void __launch_bounds__(ATD_THREADS) attn_decode_kernel(AttnArgs a) {
    using C = AtdCfg<DH>;
    constexpr int NW = ATD_WARPS;
    constexpr int SW = DH + 2;                     // a state: DH output sums, the running maximum, the running sum
    extern __shared__ __align__(128) unsigned char smem_raw[];
    bf16* ring_all = reinterpret_cast<bf16*>(smem_raw);
    float* wst = reinterpret_cast<float*>(smem_raw);                                            // [NW][16][SW], after the main loop
    float* inbox = reinterpret_cast<float*>(ring_all + (size_t)NW * C::STAGES * C::STAGE_ELEMS);   // [CL][QPC][SW]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = blockIdx.x, g = blockIdx.z;
    // Grouped-query attention: the tile's 16 rows hold the block's queries of `gpc` query heads that share one
    // key/value head (row = head * nq + block row), so their keys and values are streamed once for all of them.
    const int gpc = a.heads_per_cta > 0 ? a.heads_per_cta : 1;
    const int h = blockIdx.y * gpc;                // first query head of this CTA
    const int CL = gridDim.x;                      // cluster size
    const int QPC = (ATT_NQ + CL - 1) / CL;        // queries a CTA finishes at most
    __shared__ __align__(8) uint64_t s_inbox_bar;  // counts the bytes of the states sent to this CTA by the cluster's CTAs
    if (CL > 1 && tid == 0) { mbar_init(smem_u32(&s_inbox_bar), 1); mbar_init_fence(); }
    if (CL > 1) cluster_arrive_relaxed();          // opening handshake: waited for just before the first remote store
    bf16* ring = ring_all + (size_t)warp * C::STAGES * C::STAGE_ELEMS;
    const uint32_t ring_s = smem_u32(ring);
    // The row arrays were written at the start of the pass, at least two kernels back in the stream, so they may be
    // read before the wait below: a kernel lets its successor start only after its own wait has returned, that is
    // after its predecessor has finished, hence everything older than the immediate predecessor is complete.
    const int nq = a.nq, cnt = gpc * nq, row0 = g * nq;   // cnt: rows of the tile in use
    const int b = __ldcg(a.row_seq + row0);          // from L2: nothing an earlier kernel on this SM may have cached
    const int pos_first = __ldcg(a.row_pos + row0);
    const int pos_last = pos_first + nq - 1;
    const int n_chunks = pos_last / ATT_CH + 1;
    const int n_mine = rank < n_chunks ? (n_chunks - rank + CL - 1) / CL : 0;
    const int n_kv = a.n_kv_heads > 0 ? a.n_kv_heads : a.n_heads;
    const int kvh = h / (a.n_heads / n_kv);            // grouped-query attention: several query heads share one key/value head
    const size_t head_base = ((size_t)b * n_kv + kvh) * a.t_max;
    const size_t head_base2 = ((size_t)b * n_kv + kvh) * a.t_max2;
    const int split = a.k2 ? a.split : INT_MAX;

    // this warp's rows of its CTA's it-th chunk into stage it % STAGES.  Lane L moves unit L % TPK of rows
    // L / TPK + (32 / TPK) * u; a tile that lies wholly in one cache and before the last query (all but a
    // boundary tile or two) takes the short way: one base address, constant steps.
    constexpr int RSTEP = 32 / C::TPK;             // rows between a lane's consecutive units
    const int i_row = lane / C::TPK, i_unit = lane - i_row * C::TPK;
    auto issue = [&](int it) {
        const int t0 = (rank + it * CL) * ATT_CH + warp * ATD_WROWS;
        bf16* ks = ring + (size_t)(it % C::STAGES) * C::STAGE_ELEMS;
        bf16* vs = ks + C::TILE_ELEMS;
        const bool first = t0 + ATD_WROWS <= split, second = t0 >= split;
        if (t0 + ATD_WROWS - 1 <= pos_last && (first || second)) {
            const size_t src = first ? (head_base + t0 + i_row) * DH : (head_base2 + (t0 - split) + i_row) * DH;
            const bf16* kg = static_cast<const bf16*>(first ? a.kcache : a.k2) + src + i_unit * 8;
            const bf16* vg = static_cast<const bf16*>(first ? a.vcache : a.v2) + src + i_unit * 8;
#pragma unroll
            for (int u = 0; u < C::UNITS; ++u) {
                const int t = i_row + RSTEP * u;
                const int dst = t * DH + atd_swz<DH>(t, i_unit) * 8;
                cp_async16(ks + dst, kg + (size_t)u * RSTEP * DH);
                cp_async16(vs + dst, vg + (size_t)u * RSTEP * DH);
            }
            return;
        }
#pragma unroll
        for (int u = 0; u < C::UNITS; ++u) {
            const int t = i_row + RSTEP * u, v = i_unit;
            const int ta = t0 + t;
            const int dst = t * DH + atd_swz<DH>(t, v) * 8;
            if (ta <= pos_last) {
                const bf16 *kg, *vg;
                if (ta < split) {
                    kg = static_cast<const bf16*>(a.kcache) + (head_base + ta) * DH;
                    vg = static_cast<const bf16*>(a.vcache) + (head_base + ta) * DH;
                } else {
                    kg = static_cast<const bf16*>(a.k2) + (head_base2 + (ta - split)) * DH;
                    vg = static_cast<const bf16*>(a.v2) + (head_base2 + (ta - split)) * DH;
                }
                cp_async16(ks + dst, kg + v * 8);
                cp_async16(vs + dst, vg + v * 8);
            } else {   // past the last query: zeros, so that a zero weight times them stays zero
                *reinterpret_cast<uint4*>(ks + dst) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4*>(vs + dst) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
    };
    // Tiles that end before the block's first position hold committed keys and values from earlier iterations (or
    // earlier steps of this one): they are fetched before the wait; what the predecessor may have written, after it.
    int pre = 0;
#pragma unroll
    for (int it = 0; it < C::STAGES - 1; ++it) {
        if (it == pre && it < n_mine && (rank + it * CL) * ATT_CH + (warp + 1) * ATD_WROWS <= pos_first) {
            issue(it);
            cp_async_commit();
            ++pre;
        }
    }
    pdl_wait();   // queries and the newest keys/values come from the kernel before this one
#pragma unroll
    for (int it = 0; it < C::STAGES - 1; ++it) {
        if (it >= pre) {
            if (it < n_mine) issue(it);
            cp_async_commit();
        }
    }

    // The queries as A fragments: this lane holds rows lane/4 and lane/4 + 8, columns 2*(lane%4) (+1) (+8) of each
    // 16-wide step along the head dimension.
    const int row_lo = lane >> 2, row_hi = row_lo + 8, kc = 2 * (lane & 3);
    // tile row -> (query head within the CTA, block row); rows beyond cnt are absent (zero queries, never stored)
    const int hq_lo = row_lo < cnt ? row_lo / nq : 0, hq_hi = row_hi < cnt ? row_hi / nq : 0;
    const int i_lo = row_lo < cnt ? row_lo - hq_lo * nq : 0, i_hi = row_hi < cnt ? row_hi - hq_hi * nq : 0;
    uint32_t qf[C::KSTEPS][4];
    {
        const bf16* qg = static_cast<const bf16*>(a.q) + h * DH + kc;
        const bf16* q_lo = qg + (size_t)(row0 + i_lo) * a.ldq + hq_lo * DH;
        const bf16* q_hi = qg + (size_t)(row0 + i_hi) * a.ldq + hq_hi * DH;
#pragma unroll
        for (int ks = 0; ks < C::KSTEPS; ++ks) {
            qf[ks][0] = row_lo < cnt ? *reinterpret_cast<const uint32_t*>(q_lo + ks * 16) : 0u;
            qf[ks][1] = row_hi < cnt ? *reinterpret_cast<const uint32_t*>(q_hi + ks * 16) : 0u;
            qf[ks][2] = row_lo < cnt ? *reinterpret_cast<const uint32_t*>(q_lo + ks * 16 + 8) : 0u;
            qf[ks][3] = row_hi < cnt ? *reinterpret_cast<const uint32_t*>(q_hi + ks * 16 + 8) : 0u;
        }
    }
    float o[C::NTILES][4];
#pragma unroll
    for (int nt = 0; nt < C::NTILES; ++nt) { o[nt][0] = 0.f; o[nt][1] = 0.f; o[nt][2] = 0.f; o[nt][3] = 0.f; }
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;   // l: this lane's keys only until the end
    const bool has_hi = cnt > 8;

    // ldmatrix row addresses of this lane (matrix lane/8, row lane%8), relative to the K (or V) tile of a stage
    const int lm_m = lane >> 3, lm_r = lane & 7;
    const int lm_sw = DH >= 64 ? lm_r : (lm_r >> 1);
    const uint32_t k_row = (uint32_t)(lm_r * DH * 2);                           // K: key = 8 * nt + row, unit = 4 * kp + matrix
    const uint32_t v_row = (uint32_t)((((lm_m & 1) << 3) + lm_r) * DH * 2);     // V: key = 8 * (matrix & 1) + row, unit = 2 * np + matrix / 2

    for (int it = 0; it < n_mine; ++it) {
        if (it + C::STAGES - 1 < n_mine) issue(it + C::STAGES - 1);
        cp_async_commit();
        asm volatile("cp.async.wait_group %0;" ::"n"(C::STAGES - 1) : "memory");
        __syncwarp();
        const int t0 = (rank + it * CL) * ATT_CH + warp * ATD_WROWS;
        const uint32_t ks_s = ring_s + (uint32_t)((it % C::STAGES) * C::STAGE_ELEMS * 2);
        const uint32_t vs_s = ks_s + (uint32_t)(C::TILE_ELEMS * 2);

        // S = Q K^T for the tile's 16 keys: two 8-key halves
        float sc[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            sc[nt][0] = 0.f; sc[nt][1] = 0.f; sc[nt][2] = 0.f; sc[nt][3] = 0.f;
#pragma unroll
            for (int kp = 0; kp < C::KSTEPS / 2; ++kp) {
                uint32_t kf[4];
                ldmatrix_x4(ks_s + (uint32_t)(nt * 8 * DH * 2) + k_row + (uint32_t)((((kp * 4 + lm_m) ^ lm_sw)) << 4), kf);
                mma_bf16_16816(sc[nt], qf[2 * kp], kf[0], kf[1]);
                mma_bf16_16816(sc[nt], qf[2 * kp + 1], kf[2], kf[3]);
            }
        }
        // scale, causal mask, running maxima (a row's scores sit in the four lanes of a quad).  Rows 8-15 are
        // skipped when the block has at most eight queries: their state stays (-inf, 0, 0) and is never read.
        float mc_lo = -INFINITY, mc_hi = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int ta = t0 + nt * 8 + kc + e;
                sc[nt][e] = (row_lo < cnt && ta <= pos_first + i_lo) ? sc[nt][e] * a.scale : -INFINITY;
                mc_lo = fmaxf(mc_lo, sc[nt][e]);
                if (has_hi) {
                    sc[nt][2 + e] = (row_hi < cnt && ta <= pos_first + i_hi) ? sc[nt][2 + e] * a.scale : -INFINITY;
                    mc_hi = fmaxf(mc_hi, sc[nt][2 + e]);
                }
            }
        }
        mc_lo = fmaxf(mc_lo, __shfl_xor_sync(0xffffffffu, mc_lo, 1));
        mc_lo = fmaxf(mc_lo, __shfl_xor_sync(0xffffffffu, mc_lo, 2));
        const float mn_lo = fmaxf(m_lo, mc_lo);
        const float f_lo = m_lo > -INFINITY ? __expf(m_lo - mn_lo) : 0.f;
        m_lo = mn_lo;
        float mn_hi = -INFINITY, f_hi = 1.f;
        if (has_hi) {
            mc_hi = fmaxf(mc_hi, __shfl_xor_sync(0xffffffffu, mc_hi, 1));
            mc_hi = fmaxf(mc_hi, __shfl_xor_sync(0xffffffffu, mc_hi, 2));
            mn_hi = fmaxf(m_hi, mc_hi);
            f_hi = m_hi > -INFINITY ? __expf(m_hi - mn_hi) : 0.f;
            m_hi = mn_hi;
        }
        // probabilities as the sum of two bf16 numbers (the rounded value and the rounded remainder): the second
        // product then sees them to about 16 significant bits instead of 8, at the price of a second MMA
        uint32_t pf[4], pr[4];
        float ls_lo = 0.f, ls_hi = 0.f;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const float p0 = mn_lo > -INFINITY ? __expf(sc[nt][0] - mn_lo) : 0.f, p1 = mn_lo > -INFINITY ? __expf(sc[nt][1] - mn_lo) : 0.f;
            ls_lo += p0 + p1;
            const __nv_bfloat162 h_lo = __floats2bfloat162_rn(p0, p1);
            pf[2 * nt] = *reinterpret_cast<const uint32_t*>(&h_lo);       // keys 8 nt + kc (+1): A columns of the same numbers
            pr[2 * nt] = atd_pack_bf16x2(p0 - __low2float(h_lo), p1 - __high2float(h_lo));
            pf[2 * nt + 1] = 0u; pr[2 * nt + 1] = 0u;
            if (has_hi) {
                const float p2 = mn_hi > -INFINITY ? __expf(sc[nt][2] - mn_hi) : 0.f, p3 = mn_hi > -INFINITY ? __expf(sc[nt][3] - mn_hi) : 0.f;
                ls_hi += p2 + p3;
                const __nv_bfloat162 h_hi = __floats2bfloat162_rn(p2, p3);
                pf[2 * nt + 1] = *reinterpret_cast<const uint32_t*>(&h_hi);
                pr[2 * nt + 1] = atd_pack_bf16x2(p2 - __low2float(h_hi), p3 - __high2float(h_hi));
            }
        }
        l_lo = l_lo * f_lo + ls_lo;
        l_hi = l_hi * f_hi + ls_hi;
        // O = O * f + P V; the rescaling is skipped while no row of the warp has a new maximum (a factor of exactly 1)
        const bool rescale = __any_sync(0xffffffffu, f_lo != 1.f || f_hi != 1.f);
#pragma unroll
        for (int np = 0; np < C::NTILES / 2; ++np) {
            uint32_t vf[4];
            ldmatrix_x4_trans(vs_s + v_row + (uint32_t)((((2 * np + (lm_m >> 1)) ^ lm_sw)) << 4), vf);
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                float (&acc)[4] = o[2 * np + hh];
                if (rescale) { acc[0] *= f_lo; acc[1] *= f_lo; acc[2] *= f_hi; acc[3] *= f_hi; }
                mma_bf16_16816(acc, pf, vf[2 * hh], vf[2 * hh + 1]);
                mma_bf16_16816(acc, pr, vf[2 * hh], vf[2 * hh + 1]);
            }
        }
        __syncwarp();   // the stage may be refilled by this warp's next issue
    }
    pdl_launch_dependents();   // the successor starts behind the merge, not behind this kernel's loads (measured: a little faster)
    // a row's sum: add the quad's lanes
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();   // every warp is done with its ring: the warps' states go where the rings were
    {
        float* st_lo = wst + (size_t)(warp * ATT_NQ + row_lo) * SW;
        float* st_hi = wst + (size_t)(warp * ATT_NQ + row_hi) * SW;
        if (row_lo < cnt) {
#pragma unroll
            for (int nt = 0; nt < C::NTILES; ++nt) *reinterpret_cast<float2*>(st_lo + nt * 8 + kc) = make_float2(o[nt][0], o[nt][1]);
            if ((lane & 3) == 0) { st_lo[DH] = m_lo; st_lo[DH + 1] = l_lo; }
        }
        if (row_hi < cnt) {
#pragma unroll
            for (int nt = 0; nt < C::NTILES; ++nt) *reinterpret_cast<float2*>(st_hi + nt * 8 + kc) = make_float2(o[nt][2], o[nt][3]);
            if ((lane & 3) == 0) { st_hi[DH] = m_hi; st_hi[DH + 1] = l_hi; }
        }
    }
    __syncthreads();
    // fold the warps' states in warp order and send the CTA's state of query qa to CTA qa % CL
    if (CL > 1) cluster_wait();   // closes the opening handshake: every CTA of the cluster is running
    // One thread per (query, output element); the thread of element 0 also folds the query's running sum and sends its
    // maximum (with 4 queries of 64 elements that is one pass over the block's 256 threads).
    for (int i = tid; i < cnt * DH; i += ATD_THREADS) {
        const int qa = i / DH, e = i - qa * DH;
        float mx = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) mx = fmaxf(mx, wst[(size_t)(w * ATT_NQ + qa) * SW + DH]);
        float val = 0.f, lsum = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float* st = wst + (size_t)(w * ATT_NQ + qa) * SW;
            const float f = st[DH] > -INFINITY ? __expf(st[DH] - mx) : 0.f;
            val = fmaf(st[e], f, val);
            if (e == 0) lsum = fmaf(st[DH + 1], f, lsum);
        }
        float* slot = inbox + ((size_t)rank * QPC + qa / CL) * SW;
        if (CL > 1) {   // counted on the receiver's barrier
            st_async_dsmem_f32(smem_u32(slot + e), smem_u32(&s_inbox_bar), qa % CL, val);
            if (e == 0) {
                st_async_dsmem_f32(smem_u32(slot + DH), smem_u32(&s_inbox_bar), qa % CL, mx);
                st_async_dsmem_f32(smem_u32(slot + DH + 1), smem_u32(&s_inbox_bar), qa % CL, lsum);
            }
        } else {
            slot[e] = val;
            if (e == 0) { slot[DH] = mx; slot[DH + 1] = lsum; }
        }
    }
    if (CL > 1) {
        // This CTA finishes queries rank, rank + CL, ...: it waits (bounded) until every CTA's state of each of them
        // has arrived.  No cluster-wide barrier: a CTA without queries of its own leaves right after sending.
        const int n_fin = rank < cnt ? (cnt - rank + CL - 1) / CL : 0;
        if (n_fin > 0) {
            if (tid == 0) mbar_arrive_expect_tx(smem_u32(&s_inbox_bar), (uint32_t)(CL * n_fin * SW * 4));
            if (!mbar_wait(smem_u32(&s_inbox_bar), 0) && a.err_flag) atomicExch(a.err_flag, ATD_ERR_EXCHANGE);
        }
    } else {
        __syncthreads();
    }
    for (int u = 0; u < QPC; ++u) {
        const int qi = rank + u * CL;
        if (qi < cnt && tid < DH) {
            // the CTAs' states in rank order; all loads and exponentials first, then the two sums (same order as a plain loop)
            float mr[ATD_CLUSTER], lr[ATD_CLUSTER], orr[ATD_CLUSTER];
            float mx = -INFINITY;
#pragma unroll
            for (int r = 0; r < ATD_CLUSTER; ++r) {
                const float* st = inbox + ((size_t)r * QPC + u) * SW;
                mr[r] = r < CL ? st[DH] : -INFINITY;
                lr[r] = r < CL ? st[DH + 1] : 0.f;
                orr[r] = r < CL ? st[tid] : 0.f;
                mx = fmaxf(mx, mr[r]);
            }
            float l = 0.f, ov = 0.f;
#pragma unroll
            for (int r = 0; r < ATD_CLUSTER; ++r) {
                if (r < CL) {
                    const float f = mr[r] > -INFINITY ? __expf(mr[r] - mx) : 0.f;
                    l = fmaf(lr[r], f, l);
                    ov = fmaf(orr[r], f, ov);
                }
            }
            const int hq = qi / nq;                  // tile row qi = query head hq of this CTA, block row qi - hq * nq
            const size_t oi = (size_t)(row0 + qi - hq * nq) * a.ldo + (h + hq) * DH + tid;
            const float res = ov / l;
            if (a.out_lo) {
                const bf16 hi = __float2bfloat16_rn(res);
                static_cast<bf16*>(a.out)[oi] = hi;
                static_cast<bf16*>(a.out_lo)[oi] = __float2bfloat16_rn(res - __bfloat162float(hi));
            } else if (a.out_f32) static_cast<float*>(a.out)[oi] = res;
            else static_cast<bf16*>(a.out)[oi] = __float2bfloat16_rn(res);
        }
    }
}

}  // namespace tandem
