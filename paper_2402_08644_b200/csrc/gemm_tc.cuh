// bf16 GEMMs  y[m][n] = sum_k x[m][k] * W[n][k]  on the tcgen05 tensor cores, fp32 accumulation in TMEM.
//
//  gemm_tc_decode_kernel   few rows (<= 64): the weight matrix is the MMA's A operand (128 output features
//                          per tile on the TMEM lanes), the token rows are the B operand (16..64 columns).
//                          The job is streaming W once from HBM: every CTA owns one (tile, K-slice) unit so
//                          that all SMs pull weights, tiles arrive by TMA through a ring of stages, and the
//                          K-slices of a tile sit in one thread-block cluster: each CTA sends its partial
//                          sums to the CTA that finishes those token rows (remote shared-memory stores), which
//                          adds them in slice order.
//                          The token rows are written into the B stages by the CTA's own threads, which is
//                          where the LayerNorm of the residual stream is fused.  Activations arrive in fp32 and
//                          enter the product as the sum of two bf16 numbers (the rounded value and the rounded
//                          remainder, about 16 significant bits): the B tile holds the NB value rows followed
//                          by the NB remainder rows, one MMA of N = 2 NB covers both (the weight tile is read
//                          from shared memory once), and the epilogue adds the two accumulator columns of a
//                          token row.  The kernel streams weights, so the wider B operand costs no bandwidth.
//                          The weight loads are issued before the kernel waits for its predecessor in the
//                          stream (programmatic dependent launch), so they overlap its run; a kernel lets its
//                          own successor start once the predecessor is done, which keeps one kernel's worth of
//                          prefetch in flight (deeper chains of waiting kernels cost more than they hide).
//  gemm_tc_tiled_kernel    many rows (prompt pass): 128 x 256 output tiles, both operands by TMA; persistent CTAs with two
//                          accumulators in TMEM, so that a tile's epilogue runs under the next tile's MMAs.
//
// An output element's reduction order depends on (N, K) only, never on the number of rows, so a block
// pass and a one-row pass give identical bits.
#pragma once
#include <limits.h>
#include "common.cuh"
#include "gemm_simt.cuh"
#include "tc_common.cuh"

namespace tandem {

// How the token rows become the B operand: PRO_BF16: bf16 rows as they are (remainder rows zero); PRO_LN: fp32 rows,
// LayerNorm, then value + remainder; PRO_F32: fp32 rows as value + remainder; PRO_TMA: the producer of the rows has
// already written them as two bf16 planes (values, remainders), and TMA brings them into the B stages beside the
// weights (no registers, no rounds, nothing for warps 0-3 to do before the epilogue).
enum { PRO_BF16 = 0, PRO_LN = 1, PRO_F32 = 2, PRO_TMA = 3 };
constexpr int EPI_ARGMAX = 6;                       // fp32 store plus the (max, index) of each row within the tile
enum { TC_ERR_SLOT = 1, TC_ERR_OPERANDS = 2, TC_ERR_ACCUM = 3, TC_ERR_EXCHANGE = 4 };   // which bounded wait gave up

struct TcDecodeArgs {
    const void* x;          // PRO_BF16: bf16 [rows][ldx];  PRO_LN / PRO_F32: float [rows][ldx];  PRO_TMA: unused (tensor map)
    int ldx;
    int x_row0, x_plane_rows;   // PRO_TMA: first token row of this launch; rows between the value and the remainder plane
    int release_early;          // PRO_TMA: the successor is released right after the wait on the predecessor (a small matrix:
                                // a chain of dependent steps, nothing to protect) instead of after the last token-row loads
    const float* ln_g;      // PRO_LN: LayerNorm gain / bias [K]
    const float* ln_b;
    int rows, K, N;         // N = output features over all segments
    int seg_rows0, tiles0;  // output features and tiles of the first weight segment (one tensor map per segment)
    int seg_rows;           // output features of every further segment
    int tiles_per_seg;      // ceil(seg_rows / 128)
    int splits;             // K-slices per tile: 1, 2, 4 or 8 = the cluster size; grid = tiles * splits
    int stream_weights;     // 1: weights are read once per pass and should not stay in L2
    int* err_flag;          // nullable
    unsigned poll_limit;    // polls before a wait on an mbarrier gives up; 0 = MBAR_POLL_LIMIT
    int withhold_weights;   // test hook for the give-up path: the TMA thread issues no loads, so the wait for
                            // operands must run out (nothing is in flight when the kernel leaves)
    float* amax_val;        // EPI_ARGMAX: [rows][amax_stride] best value per tile
    int* amax_idx;          //             and its output feature
    int amax_stride;
    EpiArgs e;
};

constexpr int TCD_THREADS = 192;   // warps 0-3: B operand + epilogue; warp 4: TMA; warp 5: TMEM + MMA issue
template <int NB> struct TcdCfg {
    static constexpr int NB2 = 2 * NB;              // B-operand rows = accumulator columns: values, then remainders
    static constexpr int STAGES = NB <= 16 ? 5 : 3;   // two CTAs fit on an SM up to NB = 48 (at most 113 KB each with the static part)
    static constexpr int A_BYTES = 128 * 128;       // 128 weight rows x 64 bf16
    static constexpr int B_BYTES = NB2 * 128;       // 2 NB rows x 64 bf16
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int INBOX_BYTES = NB * 128 * 4;   // the K-slices' partial sums for the token rows this CTA finishes
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + INBOX_BYTES + 1024;   // + slack to align the ring to 1024
    static constexpr int TMEM_COLS = NB2 <= 32 ? 32 : (NB2 <= 64 ? 64 : 128);
};
static_assert(TcdCfg<16>::SMEM_BYTES + 3072 <= 113 * 1024 && TcdCfg<32>::SMEM_BYTES + 3072 <= 113 * 1024 &&
              TcdCfg<48>::SMEM_BYTES + 3072 <= 113 * 1024, "two CTAs per SM: a kernel and its prefetching successor");

// x = hi + lo with hi = bf16(x), lo = bf16(x - hi): the pair carries x to about 16 significant bits.
__device__ __forceinline__ void split_bf16x2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
    const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - __low2float(h), x1 - __high2float(h));
    hi = *reinterpret_cast<const uint32_t*>(&h);
    lo = *reinterpret_cast<const uint32_t*>(&l);
}

__device__ __forceinline__ void tc_report(int* err_flag, int code) {
    if (err_flag) atomicExch(err_flag, code);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&p);
}
__device__ __forceinline__ float4 ln_apply(float4 x, float mu, float rs, float4 g, float4 b) {
    return make_float4((x.x - mu) * rs * g.x + b.x, (x.y - mu) * rs * g.y + b.y, (x.z - mu) * rs * g.z + b.z, (x.w - mu) * rs * g.w + b.w);
}

// Where column c of weight segment `seg` goes for EPI_QKV / EPI_KV: the query buffer (row stride ldo) or a cache.
// The address of (row j, column c) is base + row term + col, with the row term j * ldo or the cache row offset.
struct ScatterCol { bf16* base; long long col; bool is_q; };
template <int EPI>
__device__ __forceinline__ ScatterCol scatter_col(const EpiArgs& e, int seg, int c) {
    ScatterCol sc;
    int s = seg;
    if (EPI == EPI_QKV && s == 0) { sc.base = static_cast<bf16*>(e.out); sc.col = c; sc.is_q = true; return sc; }
    if (EPI == EPI_QKV) s -= 1;
    const int h = c / e.d_head, el = c - h * e.d_head;
    sc.base = static_cast<bf16*>(s == 0 ? e.kcache : e.vcache);
    sc.col = (long long)h * e.t_max * e.d_head + el;
    sc.is_q = false;
    return sc;
}

// grid: tiles * splits CTAs in clusters of `splits` (the K-slices of one tile); dynamic smem TcdCfg<NB>::SMEM_BYTES.
template <int NB, int PRO, int EPI>
__global__ void __launch_bounds__(TCD_THREADS)
gemm_tc_decode_kernel(const TcDecodeArgs a, const __grid_constant__ CUtensorMap tm0, const __grid_constant__ CUtensorMap tm1,
                      const __grid_constant__ CUtensorMap tm2, const __grid_constant__ CUtensorMap tmx) {
    using C = TcdCfg<NB>;
    extern __shared__ __align__(1024) unsigned char smem_dyn[];
    __shared__ __align__(8) uint64_t s_full[C::STAGES];
    __shared__ __align__(8) uint64_t s_empty[C::STAGES];
    __shared__ __align__(8) uint64_t s_accum;
    __shared__ __align__(8) uint64_t s_inbox;   // counts the bytes of the K-slices' partial sums sent to this CTA
    __shared__ uint32_t s_tmem;
    __shared__ float s_mu[NB], s_rstd[NB];
    __shared__ float s_av[4][NB];
    __shared__ int s_ai[4][NB];
    __shared__ long long s_rowoff[NB];   // EPI_QKV / EPI_KV: the row-dependent part of an output's cache index

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t ring0 = (smem_u32(smem_dyn) + 1023u) & ~1023u;          // shared-space address of stage 0
    unsigned char* ring = smem_dyn + (ring0 - smem_u32(smem_dyn));         // the same place as a generic pointer

    const int S = a.splits;
    const uint32_t poll_limit = a.poll_limit ? a.poll_limit : MBAR_POLL_LIMIT;
    const int unit = blockIdx.x;
    const int tile = unit / S, sp = unit - tile * S;                       // sp = this CTA's rank in its cluster
    const int seg = tile < a.tiles0 ? 0 : 1 + (tile - a.tiles0) / a.tiles_per_seg;
    const int n_local0 = (seg == 0 ? tile : tile - a.tiles0 - (seg - 1) * a.tiles_per_seg) * 128;
    const int seg_rows = seg == 0 ? a.seg_rows0 : a.seg_rows;               // output features of this tile's segment
    const int seg_base = seg == 0 ? 0 : a.seg_rows0 + (seg - 1) * a.seg_rows;   // and its first output feature
    const int KB = (a.K + 63) >> 6;
    const int kb_base = KB / S, kb_rem = KB - kb_base * S;
    const int kb0 = sp * kb_base + min(sp, kb_rem);
    const int nkb = kb_base + (sp < kb_rem ? 1 : 0);
    const int K4 = a.K >> 2;
    // LayerNorm rows short enough to sit in registers (8 float4 per lane) and a K-slice that fits the ring
    // without reuse: the B operand is then written straight from the registers that gave the statistics.
    const bool ln_regs = PRO == PRO_LN && K4 <= 256 && nkb <= C::STAGES;
    // Token rows whose outputs this CTA finishes: all of them without split-K, else a contiguous share of ceil(rows / S).
    const int rpc = S == 1 ? a.rows : (a.rows + S - 1) / S;
    const int j_first = S == 1 ? 0 : sp * rpc;
    const int j_count = max(0, min(rpc, a.rows - j_first));
    float hres[EPI == EPI_RESID ? NB : 1];   // EPI_RESID: the residual values this thread's outputs are added to
    int my_seq = 0, my_pos = 0;              // EPI_QKV / EPI_KV, threads below a.rows: this token row's sequence and position

    if (warp == 5) {
        if (lane == 0) {
            for (int s = 0; s < C::STAGES; ++s) {
                mbar_init(smem_u32(&s_full[s]), PRO == PRO_TMA ? 2 : 5);   // the TMA thread's arrive + one per B-operand warp (PRO_TMA: its second arrive)
                mbar_init(smem_u32(&s_empty[s]), 1);   // the MMA thread's commit
            }
            mbar_init(smem_u32(&s_accum), 1);
            mbar_init(smem_u32(&s_inbox), 1);
            mbar_init_fence();
        }
        __syncwarp();
        tmem_alloc(smem_u32(&s_tmem), C::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = s_tmem;
    if (S > 1) cluster_arrive_relaxed();   // opening handshake: waited for just before the first remote store

    if (warp == 4) {
        // ---- weight tiles: independent of every earlier kernel, so no wait on the predecessor here ----
        if (PRO == PRO_TMA && lane == 0 && !a.withhold_weights) {
            // Weights of the first ring-ful before the wait on the predecessor, then the wait, then their token rows
            // (two planes, 16-row boxes), then weights and rows together as stages come free.
            const CUtensorMap* tm = seg == 0 ? &tm0 : (seg == 1 ? &tm1 : &tm2);
            tma_prefetch_desc(tm);
            tma_prefetch_desc(&tmx);
            const uint64_t pol = l2_policy_evict_first();
            auto load_a = [&](int i, int st) {
                const uint32_t bar = smem_u32(&s_full[st]);
                mbar_arrive_expect_tx(bar, C::A_BYTES);
                if (a.stream_weights) tma_load_2d(ring0 + st * C::STAGE_BYTES, tm, (kb0 + i) * 64, n_local0, bar, pol);
                else tma_load_2d_nohint(ring0 + st * C::STAGE_BYTES, tm, (kb0 + i) * 64, n_local0, bar);
            };
            auto load_b = [&](int i, int st) {
                const uint32_t bar = smem_u32(&s_full[st]);
                const uint32_t dst = ring0 + st * C::STAGE_BYTES + C::A_BYTES;
                mbar_arrive_expect_tx(bar, C::B_BYTES);
#pragma unroll
                for (int r16 = 0; r16 < NB; r16 += 16) {
                    tma_load_2d_nohint(dst + r16 * 128, &tmx, (kb0 + i) * 64, a.x_row0 + r16, bar);                          // values
                    tma_load_2d_nohint(dst + (NB + r16) * 128, &tmx, (kb0 + i) * 64, a.x_plane_rows + a.x_row0 + r16, bar);   // remainders
                }
            };
            const int n_pre = min(nkb, C::STAGES);
            for (int i = 0; i < n_pre; ++i) load_a(i, i);
            pdl_wait();
            for (int i = 0; i < n_pre; ++i) load_b(i, i);
            for (int i = n_pre; i < nkb; ++i) {
                const int st = i % C::STAGES;
                if (!mbar_wait(smem_u32(&s_empty[st]), ((i / C::STAGES) - 1) & 1, poll_limit)) {
                    tc_report(a.err_flag, TC_ERR_SLOT);
                    break;
                }
                load_a(i, st);
                load_b(i, st);
            }
            pdl_launch_dependents();   // the last token rows are on their way: the successor may start (see the note at the epilogue)
        } else if (lane == 0 && !a.withhold_weights) {
            const CUtensorMap* tm = seg == 0 ? &tm0 : (seg == 1 ? &tm1 : &tm2);
            tma_prefetch_desc(tm);
            const uint64_t pol = l2_policy_evict_first();
            for (int i = 0; i < nkb; ++i) {
                const int st = i % C::STAGES;
                if (i >= C::STAGES && !mbar_wait(smem_u32(&s_empty[st]), ((i / C::STAGES) - 1) & 1, poll_limit)) {
                    tc_report(a.err_flag, TC_ERR_SLOT);
                    break;
                }
                const uint32_t bar = smem_u32(&s_full[st]);
                mbar_arrive_expect_tx(bar, C::A_BYTES);
                if (a.stream_weights) tma_load_2d(ring0 + st * C::STAGE_BYTES, tm, (kb0 + i) * 64, n_local0, bar, pol);
                else tma_load_2d_nohint(ring0 + st * C::STAGE_BYTES, tm, (kb0 + i) * 64, n_local0, bar);
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        // ---- MMA issue: one thread ----
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, C::NB2);
            for (int i = 0; i < nkb; ++i) {
                const int st = i % C::STAGES;
                if (!mbar_wait(smem_u32(&s_full[st]), (i / C::STAGES) & 1, poll_limit)) {
                    tc_report(a.err_flag, TC_ERR_OPERANDS);
                    break;
                }
                tc_fence_after_sync();
                const uint64_t da = umma_desc_k_sw128(ring0 + st * C::STAGE_BYTES);
                const uint64_t db = umma_desc_k_sw128(ring0 + st * C::STAGE_BYTES + C::A_BYTES);
#pragma unroll
                for (int k = 0; k < 4; ++k)   // 4 x 16 elements of K per stage
                    umma_bf16(tmem, da + 2 * k, db + 2 * k, idesc, (i | k) != 0 ? 1u : 0u);
                umma_commit(smem_u32(&s_empty[st]));
            }
            umma_commit(smem_u32(&s_accum));
        }
        __syncwarp();
        // TMEM goes back as soon as the epilogue warps have read the accumulator (they arrive on barrier 2 right after
        // their loads), not at the end of the kernel: nothing is left to do for this warp after that.
        asm volatile("bar.sync 2, 160;" ::: "memory");
        tc_fence_after_sync();
        tmem_dealloc(tmem, C::TMEM_COLS);
    } else {
    // ---- warps 0-3: token rows into the B stages (then the epilogue) ----
    float4 gq[C::STAGES], bq[C::STAGES];   // register path: gain / bias of this lane's slot in each of the CTA's K-blocks
    if (ln_regs) {
#pragma unroll
        for (int i = 0; i < C::STAGES; ++i) {
            const int k4 = ((kb0 + i) >> 1) * 32 + lane;
            const bool mine = i < nkb && ((kb0 + i) & 1) == (lane >> 4) && k4 < K4;
            gq[i] = mine ? __ldg(reinterpret_cast<const float4*>(a.ln_g) + k4) : make_float4(0.f, 0.f, 0.f, 0.f);
            bq[i] = mine ? __ldg(reinterpret_cast<const float4*>(a.ln_b) + k4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
    pdl_wait();   // x, and everything the epilogue touches, comes from earlier kernels; gains and biases are parameters
    if (EPI == EPI_QKV || EPI == EPI_KV) {
        // cache index of (row j, head h, element el) = ((seq_j * H + h) * t_max + pos_j) * d_head + el: the row part once
        // per row.  Only the epilogue needs it: the two loads are in flight while the B operand is produced, and the
        // barrier that publishes the offsets sits after that.
        if (tid < a.rows) { my_seq = a.e.row_seq[tid]; my_pos = a.e.row_pos[tid]; }   // first used ahead of the epilogue
    }
    if (EPI == EPI_RESID) {
        // the residual-stream values this thread will add to: fetched now, off the critical path
        const float* hp = static_cast<const float*>(a.e.out);
        const int nl = n_local0 + tid;
#pragma unroll
        for (int s = 0; s < NB; ++s) {
            if (s >= j_count) break;   // (every loop over rows leaves at the last row: the unrolled rest is never fetched)
            hres[s] = nl < seg_rows ? __ldcg(hp + (size_t)(j_first + s) * a.e.ldo + seg_base + nl) : 0.f;
        }
    }
    if (ln_regs) {
        // short LayerNorm rows: one pass over x.  Lane L holds the row's float4 number L + 32u in
        // t[u], i.e. K-block 2u + (L >= 16), 16-byte chunk (L & 15) / 2, half L & 1.
        // A warp's rows are fetched one row ahead, so the loads of its rows overlap.
        float4 tn[8];
        if (warp < a.rows) {
            const float4* xr = reinterpret_cast<const float4*>(static_cast<const float*>(a.x) + (size_t)warp * a.ldx);
#pragma unroll
            for (int u = 0; u < 8; ++u) tn[u] = (lane + 32 * u < K4) ? __ldcg(xr + lane + 32 * u) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        pdl_launch_dependents();   // (a K-slice that fits the ring: see the note at the epilogue)
        for (int r = warp; r < a.rows; r += 4) {
            float4 t[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) t[u] = tn[u];
            if (r + 4 < a.rows) {
                const float4* xr = reinterpret_cast<const float4*>(static_cast<const float*>(a.x) + (size_t)(r + 4) * a.ldx);
#pragma unroll
                for (int u = 0; u < 8; ++u) tn[u] = (lane + 32 * u < K4) ? __ldcg(xr + lane + 32 * u) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            float s = 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u) s += (t[u].x + t[u].y) + (t[u].z + t[u].w);
            const float mu = warp_sum(s) / (float)a.K;
            float q = 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (lane + 32 * u < K4) {
                    const float d0 = t[u].x - mu, d1 = t[u].y - mu, d2 = t[u].z - mu, d3 = t[u].w - mu;
                    q = fmaf(d0, d0, q); q = fmaf(d1, d1, q); q = fmaf(d2, d2, q); q = fmaf(d3, d3, q);
                }
            }
            const float rs = 1.0f / sqrtf(warp_sum(q) / (float)a.K + 1e-5f);
#pragma unroll
            for (int i = 0; i < C::STAGES; ++i) {
                const int kb = kb0 + i;
                if (i >= nkb) break;
                if ((kb & 1) == (lane >> 4)) {
                    const int u = kb >> 1;
                    float4 xv = t[0];
#pragma unroll
                    for (int uu = 1; uu < 8; ++uu) if (u == uu) xv = t[uu];
                    uint2 val = make_uint2(0u, 0u), rem = make_uint2(0u, 0u);   // beyond K the weights are zero-filled; so is x
                    if (u * 32 + lane < K4) {
                        const float4 y = ln_apply(xv, mu, rs, gq[i], bq[i]);
                        split_bf16x2(y.x, y.y, val.x, rem.x);
                        split_bf16x2(y.z, y.w, val.y, rem.y);
                    }
                    const int c = (lane & 15) >> 1;
                    unsigned char* bt = ring + i * C::STAGE_BYTES + C::A_BYTES + r * 128 + ((c ^ (r & 7)) << 4) + ((lane & 1) << 3);
                    *reinterpret_cast<uint2*>(bt) = val;
                    *reinterpret_cast<uint2*>(bt + NB * 128) = rem;   // NB is a multiple of 8: the same swizzle phase
                }
            }
        }
        // rows >= a.rows of the B tiles stay as they are: a column of the product depends on its own row only
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0)
            for (int i = 0; i < nkb; ++i) mbar_arrive(smem_u32(&s_full[i]));
    } else if (PRO != PRO_TMA) {
        // general case: statistics (LayerNorm), then the K-blocks a ring's worth at a time
        if (PRO == PRO_LN) {
            for (int r = warp; r < a.rows; r += 4) {   // one warp per row, fixed lane-strided order
                const float4* xr = reinterpret_cast<const float4*>(static_cast<const float*>(a.x) + (size_t)r * a.ldx);
                float mu, var;
                if (K4 <= 256) {   // the same arithmetic as the register path above
                    float4 t[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) t[u] = (lane + 32 * u < K4) ? __ldcg(xr + lane + 32 * u) : make_float4(0.f, 0.f, 0.f, 0.f);
                    float s = 0.f;
#pragma unroll
                    for (int u = 0; u < 8; ++u) s += (t[u].x + t[u].y) + (t[u].z + t[u].w);
                    mu = warp_sum(s) / (float)a.K;
                    float q = 0.f;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (lane + 32 * u < K4) {
                            const float d0 = t[u].x - mu, d1 = t[u].y - mu, d2 = t[u].z - mu, d3 = t[u].w - mu;
                            q = fmaf(d0, d0, q); q = fmaf(d1, d1, q); q = fmaf(d2, d2, q); q = fmaf(d3, d3, q);
                        }
                    }
                    var = warp_sum(q) / (float)a.K;
                } else {
                    float s = 0.f;
#pragma unroll 8
                    for (int k4 = lane; k4 < K4; k4 += 32) { const float4 t = __ldcg(xr + k4); s += (t.x + t.y) + (t.z + t.w); }
                    mu = warp_sum(s) / (float)a.K;
                    float q = 0.f;
#pragma unroll 8
                    for (int k4 = lane; k4 < K4; k4 += 32) {
                        const float4 t = __ldcg(xr + k4);
                        const float d0 = t.x - mu, d1 = t.y - mu, d2 = t.z - mu, d3 = t.w - mu;
                        q = fmaf(d0, d0, q); q = fmaf(d1, d1, q); q = fmaf(d2, d2, q); q = fmaf(d3, d3, q);
                    }
                    var = warp_sum(q) / (float)a.K;
                }
                if (lane == 0) { s_mu[r] = mu; s_rstd[r] = 1.0f / sqrtf(var + 1e-5f); }
            }
            bar_sync(1, 128);
        }
        constexpr int CPT = NB * 8 / 128;   // 8-element chunks of the NB token rows of one K-block per thread
        for (int i0 = 0; i0 < nkb; i0 += C::STAGES) {
            // a ring's worth of K-blocks at a time: all loads first, so their latencies overlap
            uint4 raw[PRO == PRO_BF16 ? C::STAGES : 1][CPT];
            float4 raw32[PRO == PRO_BF16 ? 1 : C::STAGES][CPT][2];
#pragma unroll
            for (int g = 0; g < C::STAGES; ++g)
#pragma unroll
                for (int ch = 0; ch < CPT; ++ch) {
                    const int idx = tid + ch * 128, r = idx >> 3, c = idx & 7;
                    const int k = (kb0 + i0 + g) * 64 + c * 8;
                    const bool live = i0 + g < nkb && r < a.rows && k < a.K;
                    if (PRO == PRO_BF16) {
                        raw[g][ch] = live ? __ldcg(reinterpret_cast<const uint4*>(static_cast<const bf16*>(a.x) + (size_t)r * a.ldx + k))
                                          : make_uint4(0u, 0u, 0u, 0u);
                    } else {
                        const float4* xp = reinterpret_cast<const float4*>(static_cast<const float*>(a.x) + (size_t)r * a.ldx + k);
                        raw32[g][ch][0] = live ? __ldcg(xp) : make_float4(0.f, 0.f, 0.f, 0.f);
                        raw32[g][ch][1] = live ? __ldcg(xp + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
            if (nkb <= C::STAGES) pdl_launch_dependents();   // (a K-slice that fits the ring: see the note at the epilogue)
            bool dead = false;
#pragma unroll
            for (int g = 0; g < C::STAGES; ++g) {
                const int i = i0 + g;
                if (i >= nkb || dead) break;
                const int st = g;   // i0 is a multiple of STAGES
                if (i >= C::STAGES && !mbar_wait(smem_u32(&s_empty[st]), ((i / C::STAGES) - 1) & 1, poll_limit)) {
                    tc_report(a.err_flag, TC_ERR_SLOT);
                    dead = true;
                    break;
                }
                unsigned char* bt = ring + st * C::STAGE_BYTES + C::A_BYTES;
#pragma unroll
                for (int ch = 0; ch < CPT; ++ch) {
                    const int idx = tid + ch * 128, r = idx >> 3, c = idx & 7;
                    uint4 val = make_uint4(0u, 0u, 0u, 0u), rem = make_uint4(0u, 0u, 0u, 0u);
                    if (PRO == PRO_BF16) {
                        val = raw[g][ch];
                    } else {
                        const int k = (kb0 + i) * 64 + c * 8;
                        if (r < a.rows && k < a.K) {
                            float4 u0 = raw32[g][ch][0], u1 = raw32[g][ch][1];
                            if (PRO == PRO_LN) {
                                const float mu = s_mu[r], rs = s_rstd[r];
                                u0 = ln_apply(u0, mu, rs, __ldg(reinterpret_cast<const float4*>(a.ln_g + k)), __ldg(reinterpret_cast<const float4*>(a.ln_b + k)));
                                u1 = ln_apply(u1, mu, rs, __ldg(reinterpret_cast<const float4*>(a.ln_g + k) + 1), __ldg(reinterpret_cast<const float4*>(a.ln_b + k) + 1));
                            }
                            split_bf16x2(u0.x, u0.y, val.x, rem.x); split_bf16x2(u0.z, u0.w, val.y, rem.y);
                            split_bf16x2(u1.x, u1.y, val.z, rem.z); split_bf16x2(u1.z, u1.w, val.w, rem.w);
                        }
                    }
                    // 128-byte swizzle: the 16-byte chunk index is XORed with the row index modulo 8
                    unsigned char* dst = bt + r * 128 + ((c ^ (r & 7)) << 4);
                    *reinterpret_cast<uint4*>(dst) = val;
                    *reinterpret_cast<uint4*>(dst + NB * 128) = rem;   // the remainder row of token row r (same swizzle phase)
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&s_full[st]));
            }
        }
    }
    }

    // ---- epilogue: warps 0-3 own TMEM lanes 32 * warp .. +31 = output features of the tile ----
    float v[NB];
    const int tl = warp * 32 + lane;
    if (warp < 4) {
        // The successor may start (set up, fetch its first weight tiles) once this kernel's token-row loads are out of
        // its way: right after they have been issued when the K-slice fits the ring (one round of loads; see above),
        // else here, after the last round has been written.  Letting it start right after the wait measured 2-3 %
        // slower per iteration (its CTAs' set-up and loads compete with the row loads); later than here (after the
        // accumulator is ready, or after the exchange) slower again (the successor's head start shrinks).
        // (PRO_TMA with a K-slice longer than the ring and a matrix large enough to be a stream: the TMA thread does it, after
        // its last loads; otherwise there is nothing of this kernel's in the successor's way, and it is released at once)
        if (PRO != PRO_TMA || nkb <= C::STAGES || a.release_early) pdl_launch_dependents();
        if (EPI == EPI_QKV || EPI == EPI_KV) {
            if (tid < a.rows) s_rowoff[tid] = ((long long)my_seq * a.e.n_heads * a.e.t_max + my_pos) * a.e.d_head;
            bar_sync(1, 128);
        }
        if (!mbar_wait(smem_u32(&s_accum), 0, poll_limit)) tc_report(a.err_flag, TC_ERR_ACCUM);
        tc_fence_after_sync();
#pragma unroll
        for (int c0 = 0; c0 < NB; c0 += 16) {
            if (c0 >= a.rows) break;                  // columns of absent token rows are never read
            float t[16], u[16];
            tmem_ld16(tmem + (static_cast<uint32_t>(warp * 32) << 16) + c0, t);        // x's values times W
            tmem_ld16(tmem + (static_cast<uint32_t>(warp * 32) << 16) + NB + c0, u);   // x's remainders times W
#pragma unroll
            for (int i = 0; i < 16; ++i) v[c0 + i] = t[i] + u[i];
        }
        tc_fence_before_sync();
        asm volatile("bar.arrive 2, 160;" ::: "memory");   // the accumulator has been read: warp 5 may free the TMEM columns
    }
    const int n_local = n_local0 + tl;                 // warps 0-3: this thread's output feature
    const bool valid = n_local < seg_rows;
    const int n = seg_base + n_local;
    if (EPI == EPI_ARGMAX) {                            // whole tiles only (S == 1)
        if (warp < 4) {
            float* out = static_cast<float*>(a.e.out);
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                if (j >= a.rows) break;
                {
                    float bv = valid ? v[j] : -INFINITY;
                    int bi = valid ? n : INT_MAX;
                    if (valid) out[(size_t)j * a.e.ldo + n] = v[j];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
                    }
                    if (lane == 0) { s_av[warp][j] = bv; s_ai[warp][j] = bi; }
                }
            }
            bar_sync(1, 128);
            if (tid < a.rows) {
                float bv = s_av[0][tid];
                int bi = s_ai[0][tid];
                for (int w = 1; w < 4; ++w)
                    if (s_av[w][tid] > bv || (s_av[w][tid] == bv && s_ai[w][tid] < bi)) { bv = s_av[w][tid]; bi = s_ai[w][tid]; }
                a.amax_val[(size_t)tid * a.amax_stride + tile] = bv;
                a.amax_idx[(size_t)tid * a.amax_stride + tile] = bi;
            }
        }
    } else {
        if (S > 1) {
            // The cluster's CTAs hold the K-slices of one tile, and CTA r finishes token rows [r * rpc, (r + 1) * rpc).
            // Every CTA sends each row's partial sums to the inbox of the CTA that finishes it, with stores that count
            // their bytes on the receiver's inbox barrier; a CTA that finishes rows waits until S x rows x 128 floats
            // have arrived and sums its inbox in slice order.  No cluster-wide barrier: a CTA without rows of its own
            // leaves right after sending, the others once everything addressed to them has arrived (nothing is
            // written into a CTA's shared memory after that).
            const uint32_t inbox0 = ring0 + C::STAGES * C::STAGE_BYTES;           // [S][rpc][128] fp32
            cluster_wait();   // closes the opening handshake: every CTA of the cluster is running
            if (warp < 4) {
                const uint32_t ibar = smem_u32(&s_inbox);
                if (tid == 0 && j_count > 0) mbar_arrive_expect_tx(ibar, (uint32_t)(S * j_count * 128 * 4));
                int dst = 0, jj = 0;
#pragma unroll
                for (int j = 0; j < NB; ++j) {
                    if (j >= a.rows) break;
                    st_async_dsmem_f32(inbox0 + ((sp * rpc + jj) * 128 + tl) * 4, ibar, dst, v[j]);
                    if (++jj == rpc) { jj = 0; ++dst; }
                }
                if (j_count > 0 && !mbar_wait(ibar, 0, poll_limit)) tc_report(a.err_flag, TC_ERR_EXCHANGE);
            }
            if (warp < 4) {
                const float* inbox = reinterpret_cast<const float*>(ring + C::STAGES * C::STAGE_BYTES);
#pragma unroll
                for (int s = 0; s < NB / 2; ++s) {
                    if (s >= j_count) break;
                    float acc = 0.f;
#pragma unroll
                    for (int ss = 0; ss < 8; ++ss) if (ss < S) acc += inbox[((ss * rpc + s) * 128) + tl];   // slice order
                    v[s] = acc;
                }
            }
        }
        // v[s] is now the finished product of token row j_first + s and this thread's feature
        if (warp < 4) {
            ScatterCol sc;
            if (EPI == EPI_QKV || EPI == EPI_KV) sc = scatter_col<EPI>(a.e, seg, n_local);
#pragma unroll
            for (int s = 0; s < NB; ++s) {
                if (s >= j_count) break;
                {
                    const int j = j_first + s;
                    float hv = v[s];
                    if (EPI == EPI_RESID) hv += hres[s];
                    if (valid) {
                        if (EPI == EPI_RESID || EPI == EPI_STORE_F32) {
                            static_cast<float*>(a.e.out)[(size_t)j * a.e.ldo + n] = hv;
                            if (EPI == EPI_RESID && a.e.snap) static_cast<float*>(a.e.snap)[(size_t)j * a.e.snap_ld + n] = hv;
                        } else if (EPI == EPI_GELU) {   // activations between the decode kernels stay fp32, or value + remainder planes
                            const float gv = gelu_bf16_out(hv);
                            if (a.e.out_lo) {
                                const bf16 hi = __float2bfloat16_rn(gv);
                                static_cast<bf16*>(a.e.out)[(size_t)j * a.e.ldo + n] = hi;
                                static_cast<bf16*>(a.e.out_lo)[(size_t)j * a.e.ldo + n] = __float2bfloat16_rn(gv - __bfloat162float(hi));
                            } else {
                                static_cast<float*>(a.e.out)[(size_t)j * a.e.ldo + n] = gv;
                            }
                        } else if (EPI == EPI_QKV || EPI == EPI_KV) {
                            sc.base[(sc.is_q ? (long long)j * a.e.ldo : s_rowoff[j]) + sc.col] = __float2bfloat16_rn(hv);
                        } else {
                            epilogue<bf16, EPI>(a.e, j, n, hv);
                        }
                    }
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// Many rows: 128 x 256 output tiles, A = token rows, B = weight rows, both by TMA.
// ---------------------------------------------------------------------------------------------------

struct TcTiledArgs {
    int M, K, N;
    int seg_rows0, tiles0;   // first segment: output features, tiles of BN
    int seg_rows, tiles_per_seg;
    int tiles_n, tiles_m;    // BN-wide feature tiles over all segments, 128-row tiles
    int* err_flag;
    EpiArgs e;
};

constexpr int TCT_THREADS = 192;
constexpr int TCT_TILE_BYTES = 128 * 128;          // one TMA box: 128 rows x 64 bf16
// BN = output features per tile: 256 when that still fills the GPU (each token-row tile read from shared memory then
// feeds twice the MMA work of a square tile), else 128.
template <int BN> struct TctCfg {
    static constexpr int STAGES = BN == 256 ? 4 : 6;
    static constexpr int STAGE_BYTES = (1 + BN / 128) * TCT_TILE_BYTES;   // token rows, then the weight rows (one box per 128)
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024;
    static constexpr int TMEM_COLS = 2 * BN;   // two accumulators
};

// Sixteen consecutive output features of one row.  n_local0 is a multiple of 16.
template <int EPI>
__device__ __forceinline__ void epilogue16(const EpiArgs& e, int m, int seg, int seg_base, int seg_rows, int n_local0, const float (&v)[16]) {
    const int n0 = seg_base + n_local0;
    if (n_local0 + 16 > seg_rows || (e.ldo & 7) || (seg_rows & 7)) {
        for (int i = 0; i < 16; ++i)
            if (n_local0 + i < seg_rows) epilogue<bf16, EPI>(e, m, n0 + i, v[i]);
        return;
    }
    if (EPI == EPI_STORE_F32 || EPI == EPI_RESID) {
        float4* p = reinterpret_cast<float4*>(static_cast<float*>(e.out) + (size_t)m * e.ldo + n0);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float4 t = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            if (EPI == EPI_RESID) { const float4 o = p[i]; t.x += o.x; t.y += o.y; t.z += o.z; t.w += o.w; }
            p[i] = t;
        }
        return;
    }
    uint4 lo, hi;
    if (EPI == EPI_GELU) {
        lo.x = pack_bf16x2(gelu_bf16_out(v[0]), gelu_bf16_out(v[1])); lo.y = pack_bf16x2(gelu_bf16_out(v[2]), gelu_bf16_out(v[3]));
        lo.z = pack_bf16x2(gelu_bf16_out(v[4]), gelu_bf16_out(v[5])); lo.w = pack_bf16x2(gelu_bf16_out(v[6]), gelu_bf16_out(v[7]));
        hi.x = pack_bf16x2(gelu_bf16_out(v[8]), gelu_bf16_out(v[9])); hi.y = pack_bf16x2(gelu_bf16_out(v[10]), gelu_bf16_out(v[11]));
        hi.z = pack_bf16x2(gelu_bf16_out(v[12]), gelu_bf16_out(v[13])); hi.w = pack_bf16x2(gelu_bf16_out(v[14]), gelu_bf16_out(v[15]));
    } else {
        lo.x = pack_bf16x2(v[0], v[1]); lo.y = pack_bf16x2(v[2], v[3]); lo.z = pack_bf16x2(v[4], v[5]); lo.w = pack_bf16x2(v[6], v[7]);
        hi.x = pack_bf16x2(v[8], v[9]); hi.y = pack_bf16x2(v[10], v[11]); hi.z = pack_bf16x2(v[12], v[13]); hi.w = pack_bf16x2(v[14], v[15]);
    }
    bf16* dst;
    if (EPI == EPI_STORE || EPI == EPI_GELU) {
        dst = static_cast<bf16*>(e.out) + (size_t)m * e.ldo + n0;
    } else {   // EPI_QKV / EPI_KV: the query goes to its buffer, keys and values straight into the cache
        int s = seg;
        if (EPI == EPI_QKV && s == 0) {
            dst = static_cast<bf16*>(e.out) + (size_t)m * e.ldo + n_local0;
        } else {
            if (EPI == EPI_QKV) s -= 1;
            const int h = n_local0 / e.d_head, el = n_local0 - h * e.d_head;
            const size_t idx = (((size_t)e.row_seq[m] * e.n_heads + h) * e.t_max + e.row_pos[m]) * e.d_head + el;
            dst = static_cast<bf16*>(s == 0 ? e.kcache : e.vcache) + idx;
        }
    }
    reinterpret_cast<uint4*>(dst)[0] = lo;
    reinterpret_cast<uint4*>(dst)[1] = hi;
}

// Persistent: grid = min(tiles, SMs) CTAs, CTA b takes output tiles b, b + grid, ... (tile = (row tile, BN-wide feature
// tile), feature tiles fastest).  The TMA ring runs on across tile boundaries, and two accumulators in TMEM alternate,
// so that the epilogue of one tile (TMEM -> registers -> global) overlaps the MMAs of the next.
// dynamic smem TctCfg<BN>::SMEM_BYTES.
template <int EPI, int BN>
__global__ void __launch_bounds__(TCT_THREADS)
gemm_tc_tiled_kernel(const TcTiledArgs a, const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tm0,
                     const __grid_constant__ CUtensorMap tm1, const __grid_constant__ CUtensorMap tm2) {
    using C = TctCfg<BN>;
    extern __shared__ __align__(1024) unsigned char smem_dyn[];
    __shared__ __align__(8) uint64_t s_full[C::STAGES];
    __shared__ __align__(8) uint64_t s_empty[C::STAGES];
    __shared__ __align__(8) uint64_t s_acc_full[2], s_acc_free[2];
    __shared__ uint32_t s_tmem;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t ring0 = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const int KB = (a.K + 63) >> 6;
    const int total = a.tiles_n * a.tiles_m;
    // feature tile -> (segment, first feature within it)
    auto seg_of = [&](int tile_n, int& n_local0) {
        const int seg = tile_n < a.tiles0 ? 0 : 1 + (tile_n - a.tiles0) / a.tiles_per_seg;
        n_local0 = (seg == 0 ? tile_n : tile_n - a.tiles0 - (seg - 1) * a.tiles_per_seg) * BN;
        return seg;
    };

    if (warp == 5) {
        if (lane == 0) {
            for (int s = 0; s < C::STAGES; ++s) { mbar_init(smem_u32(&s_full[s]), 1); mbar_init(smem_u32(&s_empty[s]), 1); }
            for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&s_acc_full[s]), 1); mbar_init(smem_u32(&s_acc_free[s]), 4); }   // free: one arrive per epilogue warp
            mbar_init_fence();
        }
        __syncwarp();
        tmem_alloc(smem_u32(&s_tmem), C::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = s_tmem;

    if (warp == 4) {
        if (lane == 0) {
            tma_prefetch_desc(&tmx);
            tma_prefetch_desc(&tm0);
            long long g = 0;   // k-blocks issued by this CTA over all of its tiles: ring position
            bool ok = true;
            for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
                int n_local0;
                const int seg = seg_of(t % a.tiles_n, n_local0);
                const int m0 = (t / a.tiles_n) * 128;
                const CUtensorMap* tw = seg == 0 ? &tm0 : (seg == 1 ? &tm1 : &tm2);
                for (int i = 0; i < KB; ++i, ++g) {
                    const int st = (int)(g % C::STAGES);
                    if (g >= C::STAGES && !mbar_wait(smem_u32(&s_empty[st]), (uint32_t)((g / C::STAGES) - 1) & 1)) {
                        tc_report(a.err_flag, TC_ERR_SLOT);
                        ok = false;
                        break;
                    }
                    const uint32_t bar = smem_u32(&s_full[st]);
                    mbar_arrive_expect_tx(bar, C::STAGE_BYTES);
                    tma_load_2d_nohint(ring0 + st * C::STAGE_BYTES, &tmx, i * 64, m0, bar);
#pragma unroll
                    for (int hb = 0; hb < BN / 128; ++hb)   // rows past the segment's end arrive as zeros
                        tma_load_2d_nohint(ring0 + st * C::STAGE_BYTES + (1 + hb) * TCT_TILE_BYTES, tw, i * 64, n_local0 + hb * 128, bar);
                }
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, BN);
            long long g = 0;
            bool ok = true;
            int it = 0;
            for (int t = blockIdx.x; t < total && ok; t += gridDim.x, ++it) {
                const int buf = it & 1;
                // the accumulator's previous tile (two tiles back) must have been read out
                if (it >= 2 && !mbar_wait(smem_u32(&s_acc_free[buf]), (uint32_t)((it >> 1) - 1) & 1)) {
                    tc_report(a.err_flag, TC_ERR_ACCUM);
                    break;
                }
                tc_fence_after_sync();
                for (int i = 0; i < KB; ++i, ++g) {
                    const int st = (int)(g % C::STAGES);
                    if (!mbar_wait(smem_u32(&s_full[st]), (uint32_t)(g / C::STAGES) & 1)) {
                        tc_report(a.err_flag, TC_ERR_OPERANDS);
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint64_t da = umma_desc_k_sw128(ring0 + st * C::STAGE_BYTES);
                    const uint64_t db = umma_desc_k_sw128(ring0 + st * C::STAGE_BYTES + TCT_TILE_BYTES);
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_bf16(tmem + buf * BN, da + 2 * k, db + 2 * k, idesc, (i | k) != 0 ? 1u : 0u);
                    umma_commit(smem_u32(&s_empty[st]));
                }
                umma_commit(smem_u32(&s_acc_full[buf]));   // (also after a failed wait: the epilogue warps must not be left waiting)
            }
        }
        __syncwarp();
    } else {
        int it = 0;
        for (int t = blockIdx.x; t < total; t += gridDim.x, ++it) {
            const int buf = it & 1;
            int n_local0;
            const int seg = seg_of(t % a.tiles_n, n_local0);
            const int seg_rows = seg == 0 ? a.seg_rows0 : a.seg_rows;
            const int seg_base = seg == 0 ? 0 : a.seg_rows0 + (seg - 1) * a.seg_rows;
            if (!mbar_wait(smem_u32(&s_acc_full[buf]), (uint32_t)(it >> 1) & 1)) { tc_report(a.err_flag, TC_ERR_ACCUM); break; }
            tc_fence_after_sync();
            const int m = (t / a.tiles_n) * 128 + warp * 32 + lane;   // output row = TMEM lane
            const uint32_t acc = tmem + (static_cast<uint32_t>(warp * 32) << 16) + buf * BN;
            if (EPI == EPI_RESID && n_local0 + BN <= seg_rows && (a.e.ldo & 3) == 0 && (seg_base & 3) == 0) {
                // residual add on whole tiles: the old values of 64 columns are fetched together (sixteen 16-byte loads in
                // flight) before the accumulator is read, instead of one exposed round trip per 16 columns
                float* prow = static_cast<float*>(a.e.out) + (size_t)min(m, a.M - 1) * a.e.ldo + seg_base + n_local0;
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 64) {
                    float4 old[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) old[j] = __ldcg(reinterpret_cast<const float4*>(prow + c0) + j);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float v[16];
                        tmem_ld16(acc + c0 + 16 * q, v);   // warp-wide: every lane takes part
                        if (m < a.M) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float4 o = old[4 * q + i];
                                reinterpret_cast<float4*>(prow + c0 + 16 * q)[i] =
                                    make_float4(v[4 * i] + o.x, v[4 * i + 1] + o.y, v[4 * i + 2] + o.z, v[4 * i + 3] + o.w);
                            }
                        }
                    }
                }
            } else {
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 16) {
                    float v[16];
                    tmem_ld16(acc + c0, v);   // warp-wide: every lane takes part
                    if (m < a.M && n_local0 + c0 < seg_rows) epilogue16<EPI>(a.e, m, seg, seg_base, seg_rows, n_local0 + c0, v);
                }
            }
            tc_fence_before_sync();   // this warp's TMEM reads are done: the accumulator may be overwritten
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_acc_free[buf]));
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) tmem_dealloc(tmem, C::TMEM_COLS);
}

}  // namespace tandem
