// Causal prompt attention (Eq. 1 over the prompt) on the tcgen05 tensor cores, bf16, head size 64 or 128.
//
// One CTA serves one (head, tile of up to 128 consecutive queries of one sequence); two such CTAs share an SM, so
// that one's tensor work runs while the other's softmax does.  The context is swept in chunks of 64 keys anchored
// at position 0, up to the tile's last query:
//     S  = Q K^T        M = 128 queries on the TMEM lanes, N = 64 keys, K = head size; two S buffers in TMEM
//     P  = softmax step thread i owns query i: reads its row of S from TMEM once, masks keys after its position,
//                       writes bf16 probabilities into a swizzled A tile (one 128-byte row)
//     O += P V          M = 128 queries, N = head size, K = 64 keys, accumulated in TMEM over all chunks; V is used as
//                       it lies in the cache ([key][element], i.e. MN-major for the B operand)
// The running maximum is lazy: probabilities are taken relative to a reference m that moves only when a chunk's
// maximum exceeds it by more than ATC_LAZY (so they stay below e^ATC_LAZY); only then is O, in TMEM, rescaled
// (tcgen05.ld, multiply, tcgen05.st) - rare after the first chunks.  The row sum adds the fp32 probabilities (their
// bf16 roundings, which the tensor core multiplies with V, differ from them by 2^-9 each with random signs).
// Warp 4 streams K (two stages) and V (one stage) by TMA, warp 5 allocates TMEM and issues the MMAs (S of chunk c+1
// goes out before the probabilities of chunk c are awaited), warps 0-3 do the softmax and the epilogue.  Every wait is
// bounded.
#pragma once
#include "common.cuh"
#include "gemm_tc.cuh"
#include "tc_common.cuh"

namespace tandem {

struct AttnTcArgs {
    void* out; int ldo;                   // bf16 [M][ldo]; head h at columns h*DH..
    const int* row_seq; const int* row_pos;
    const int* grp_row0; const int* grp_cnt;
    int n_heads, t_max;
    int n_kv_heads;                       // key/value heads of the cache (<= n_heads, divides it)
    float scale;
    int* err_flag;
};

constexpr int ATC_THREADS = 192;
constexpr int ATC_Q = 128;                // queries per tile
constexpr int ATC_KC = 64;                // keys per chunk
constexpr int ATC_SUB = 128 * 128;        // bytes of one 128-row x 64-element bf16 sub-tile (queries, probabilities)
constexpr int ATC_KSUB = ATC_KC * 128;    // bytes of one 64-key x 64-element sub-tile (keys, values)
constexpr float ATC_LAZY = 5.0f;          // how far a chunk's maximum may exceed the reference before O is rescaled
template <int DH> struct AtcCfg {
    static constexpr int NSUB = DH / 64;                       // 64-element sub-tiles along the head dimension
    static constexpr int Q_BYTES = NSUB * ATC_SUB;
    static constexpr int K_BYTES = NSUB * ATC_KSUB;            // keys (or values) of one chunk
    static constexpr int P_BYTES = ATC_SUB;                    // 128 queries x 64 keys bf16
    static constexpr int SMEM_BYTES = Q_BYTES + 3 * K_BYTES + P_BYTES + 1024;   // two key stages, one value stage
    static constexpr int TMEM_COLS = 256;                      // S of even / odd chunks: columns 0..63 / 64..127; O: 128..128+DH-1
};
static_assert(AtcCfg<128>::SMEM_BYTES + 2048 <= 113 * 1024, "two CTAs per SM");

// Instruction descriptor: bf16 A (K-major) and B, fp32 accumulation; b_mn = 1 when B is MN-major.
__host__ __device__ constexpr uint32_t umma_idesc_bf16_b(int M, int N, int b_mn) {
    return umma_idesc_bf16(M, N) | (static_cast<uint32_t>(b_mn) << 16);
}
// Shared-memory descriptor of an MN-major bf16 operand with the 128-byte swizzle: rows of 64 MN-elements (128 bytes),
// one row per K index, 8-row groups 1024 bytes apart; further 64-element MN blocks `mn_block_bytes` apart.
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr, uint32_t mn_block_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((mn_block_bytes >> 4) & 0x3FFFu) << 16;   // leading-dimension offset: next MN block
    d |= static_cast<uint64_t>(1024 >> 4) << 32;                          // stride offset: next group of 8 K rows
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}
// 16 consecutive fp32 columns of this thread's TMEM lane, written back (the counterpart of tmem_ld16).
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
          "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
          "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
          "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 64 consecutive fp32 columns of this thread's TMEM lane in one load (load and wait in one statement: the registers
// are not read before the load has landed).
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, float (&v)[64]) {
    uint32_t r[64];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%64];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
              "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
              "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
              "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]),
              "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]),
              "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]),
              "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]),
              "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}
// 2^x by the hardware approximation (relative error about 2^-22; 2^-inf = 0), one instruction.
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// grid: (heads, groups); dynamic smem AtcCfg<DH>::SMEM_BYTES.
// tmq: queries [M][d_model] (box 64 x 128); tmk / tmv: one layer's cache seen as [(seq, kv head, position)][DH] (box 64 x 64).
template <int DH>
__global__ void __launch_bounds__(ATC_THREADS, 2)
attn_prefill_tc_kernel(const AttnTcArgs a, const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                       const __grid_constant__ CUtensorMap tmv) {
    using C = AtcCfg<DH>;
    extern __shared__ __align__(1024) unsigned char smem_dyn[];
    __shared__ __align__(8) uint64_t s_qfull, s_kfull[2], s_kfree[2], s_vfull, s_vfree, s_sfull[2], s_pready, s_ofull;
    __shared__ uint32_t s_tmem;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t base0 = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* base = smem_dyn + (base0 - smem_u32(smem_dyn));
    const uint32_t q0 = base0, k0 = q0 + C::Q_BYTES, v0 = k0 + 2 * C::K_BYTES, p0 = v0 + C::K_BYTES;
    unsigned char* pg = base + C::Q_BYTES + 3 * C::K_BYTES;

    const int h = blockIdx.x, g = blockIdx.y;
    const int row0 = a.grp_row0[g], cnt = a.grp_cnt[g];
    if (cnt <= 0) return;
    const int b = a.row_seq[row0];
    const int pos_first = a.row_pos[row0];
    const int pos_last = pos_first + cnt - 1;
    const int n_chunks = pos_last / ATC_KC + 1;
    const int kv_row0 = (b * a.n_kv_heads + h / (a.n_heads / a.n_kv_heads)) * a.t_max;   // row of position 0 of this head's key/value head in the cache's 2-D view

    if (warp == 5) {
        if (lane == 0) {
            mbar_init(smem_u32(&s_qfull), 1);
            for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&s_kfull[s]), 1); mbar_init(smem_u32(&s_kfree[s]), 1); mbar_init(smem_u32(&s_sfull[s]), 1); }
            mbar_init(smem_u32(&s_vfull), 1);
            mbar_init(smem_u32(&s_vfree), 1);
            mbar_init(smem_u32(&s_pready), 4);   // one arrive per softmax warp
            mbar_init(smem_u32(&s_ofull), 1);
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
        // ---- TMA: Q once; K of chunk c+1 as soon as its stage is free (S of chunk c-1 done), V of chunk c+1 once P V of chunk c is done ----
        if (lane == 0) {
            tma_prefetch_desc(&tmq); tma_prefetch_desc(&tmk); tma_prefetch_desc(&tmv);
            mbar_arrive_expect_tx(smem_u32(&s_qfull), C::Q_BYTES);
            for (int sb = 0; sb < C::NSUB; ++sb) tma_load_2d_nohint(q0 + sb * ATC_SUB, &tmq, h * DH + sb * 64, row0, smem_u32(&s_qfull));
            auto load_k = [&](int c) {
                const uint32_t bar = smem_u32(&s_kfull[c & 1]);
                mbar_arrive_expect_tx(bar, C::K_BYTES);
                for (int sb = 0; sb < C::NSUB; ++sb) tma_load_2d_nohint(k0 + (c & 1) * C::K_BYTES + sb * ATC_KSUB, &tmk, sb * 64, kv_row0 + c * ATC_KC, bar);
            };
            auto load_v = [&](int c) {
                const uint32_t bar = smem_u32(&s_vfull);
                mbar_arrive_expect_tx(bar, C::K_BYTES);
                for (int sb = 0; sb < C::NSUB; ++sb) tma_load_2d_nohint(v0 + sb * ATC_KSUB, &tmv, sb * 64, kv_row0 + c * ATC_KC, bar);
            };
            load_k(0);
            load_v(0);
            for (int c = 0; c + 1 < n_chunks; ++c) {
                if (c + 1 >= 2 && !mbar_wait(smem_u32(&s_kfree[(c + 1) & 1]), (((c + 1) >> 1) - 1) & 1)) { tc_report(a.err_flag, TC_ERR_SLOT); break; }
                load_k(c + 1);
                if (!mbar_wait(smem_u32(&s_vfree), c & 1)) { tc_report(a.err_flag, TC_ERR_SLOT); break; }
                load_v(c + 1);
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        // ---- MMA issue: one thread ----
        if (lane == 0) {
            constexpr uint32_t idesc_s = umma_idesc_bf16_b(128, ATC_KC, 0);
            constexpr uint32_t idesc_o = umma_idesc_bf16_b(128, DH, 1);
            bool ok = mbar_wait(smem_u32(&s_qfull), 0);
            if (!ok) tc_report(a.err_flag, TC_ERR_OPERANDS);
            // S = Q K^T of chunk c into S buffer c & 1: both K-major, 16 elements of the head dimension per instruction
            auto issue_s = [&](int c) -> bool {
                const int st = c & 1;
                if (!mbar_wait(smem_u32(&s_kfull[st]), (c >> 1) & 1)) { tc_report(a.err_flag, TC_ERR_OPERANDS); return false; }
                tc_fence_after_sync();
                const uint32_t kaddr = k0 + st * C::K_BYTES;
#pragma unroll
                for (int sb = 0; sb < C::NSUB; ++sb)
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_bf16(tmem + st * ATC_KC, umma_desc_k_sw128(q0 + sb * ATC_SUB) + 2 * k, umma_desc_k_sw128(kaddr + sb * ATC_KSUB) + 2 * k,
                                  idesc_s, (sb | k) != 0 ? 1u : 0u);
                umma_commit(smem_u32(&s_sfull[st]));
                umma_commit(smem_u32(&s_kfree[st]));   // the key stage may be refilled
                return true;
            };
            ok = ok && issue_s(0);
            for (int c = 0; c < n_chunks && ok; ++c) {
                // the next chunk's scores are computed while the softmax warps work on this one (its S buffer was
                // released with the probabilities of chunk c - 1)
                if (c + 1 < n_chunks && !issue_s(c + 1)) break;
                if (!mbar_wait(smem_u32(&s_pready), c & 1)) { tc_report(a.err_flag, TC_ERR_ACCUM); break; }
                if (!mbar_wait(smem_u32(&s_vfull), c & 1)) { tc_report(a.err_flag, TC_ERR_OPERANDS); break; }
                tc_fence_after_sync();
                // O += P V: P K-major (one 64-key sub-tile), V MN-major; 16 keys per instruction
#pragma unroll
                for (int ks = 0; ks < ATC_KC / 16; ++ks)
                    umma_bf16(tmem + 128, umma_desc_k_sw128(p0) + 2 * ks, umma_desc_mn_sw128(v0 + ks * 2048, ATC_KSUB), idesc_o,
                              (c | ks) != 0 ? 1u : 0u);
                umma_commit(smem_u32(&s_vfree));    // V of this chunk may be overwritten
                umma_commit(smem_u32(&s_ofull));    // O holds chunks 0..c; the P tile may be rewritten
            }
        }
        __syncwarp();
    } else {
        // ---- softmax warps: thread = query = TMEM lane ----
        const int qi = warp * 32 + lane;
        const int qpos = pos_first + qi;                 // (rows past cnt compute on whatever the tile holds; never stored)
        const uint32_t lane_addr = tmem + (static_cast<uint32_t>(warp * 32) << 16);
        // Everything runs in the base-2 domain: with sc2 = scale * log2(e), a probability is 2^(s * sc2 - m) (one
        // multiply-add and one ex2 per element); m is the reference maximum in that domain.
        const float sc2 = a.scale * 1.4426950408889634f;
        constexpr float LAZY2 = ATC_LAZY * 1.4426950408889634f;
        float m = -INFINITY, l = 0.f;                    // reference maximum of the exponentials, running sum
        bool ok = true;
        for (int c = 0; c < n_chunks && ok; ++c) {
            if (!mbar_wait(smem_u32(&s_sfull[c & 1]), (c >> 1) & 1)) { tc_report(a.err_flag, TC_ERR_ACCUM); ok = false; break; }
            tc_fence_after_sync();
            const uint32_t s_addr = lane_addr + (c & 1) * ATC_KC;
            // this row of S, raw; keys after the query's position become -inf (every chunk but the tile's last ones lies
            // wholly before its first query and needs no mask)
            const bool full = c * ATC_KC + ATC_KC - 1 <= pos_first;
            float t[ATC_KC];
            tmem_ld64(s_addr, t);                        // the whole row in one load
            float mr = -INFINITY;
            if (full) {
#pragma unroll
                for (int i = 0; i < ATC_KC; ++i) mr = fmaxf(mr, t[i]);
            } else {
#pragma unroll
                for (int i = 0; i < ATC_KC; ++i) {
                    t[i] = (c * ATC_KC + i <= qpos) ? t[i] : -INFINITY;
                    mr = fmaxf(mr, t[i]);
                }
            }
            const float mc = mr * sc2;                   // the chunk's maximum in the base-2 domain (the scale is positive)
            tc_fence_before_sync();      // the TMEM reads of S are done before the MMA after next may overwrite the buffer
            // P V of the previous chunk must be complete before the P tile is rewritten or O is touched
            if (c > 0) {
                if (!mbar_wait(smem_u32(&s_ofull), (c - 1) & 1)) { tc_report(a.err_flag, TC_ERR_ACCUM); ok = false; break; }
                tc_fence_after_sync();
            }
            // lazy reference: it moves only when this chunk's maximum exceeds it by more than the margin
            const bool move = mc > m + LAZY2;            // (first chunk: m = -inf, every row with a visible key moves)
            if (c > 0 && __any_sync(0xffffffffu, move)) {
                const float f = (move && m > -INFINITY) ? ex2_approx(m - mc) : 1.0f;   // rows that keep their reference: exactly 1
#pragma unroll
                for (int e0 = 0; e0 < DH; e0 += 16) {
                    float o[16];
                    tmem_ld16(lane_addr + 128 + e0, o);
#pragma unroll
                    for (int i = 0; i < 16; ++i) o[i] *= f;
                    tmem_st16(lane_addr + 128 + e0, o);
                }
                tmem_wait_st();
                l *= f;
            }
            if (move) m = mc;
            // probabilities relative to the reference (2^(-inf) = 0 for masked keys), their sum, and one 128-byte row
            // of the bf16 P tile
            unsigned char* prow = pg + qi * 128;
            const float nm = -m;
            float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
            for (int c0 = 0; c0 < ATC_KC; c0 += 8) {
                uint32_t pk[4];
#pragma unroll
                for (int i = 0; i < 8; i += 2) {
                    const float p0v = ex2_approx(fmaf(t[c0 + i], sc2, nm));
                    const float p1v = ex2_approx(fmaf(t[c0 + i + 1], sc2, nm));
                    ls0 += p0v; ls1 += p1v;
                    pk[i >> 1] = pack_bf16x2(p0v, p1v);
                }
                *reinterpret_cast<uint4*>(prow + ((((c0 >> 3)) ^ (qi & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            const float ls = ls0 + ls1;
            l += ls;
            tc_fence_before_sync();      // the rescaled O is in TMEM before the next P V accumulates onto it
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_pready));
        }
        if (ok) {   // all chunks accumulated
            if (!mbar_wait(smem_u32(&s_ofull), (n_chunks - 1) & 1)) { tc_report(a.err_flag, TC_ERR_ACCUM); ok = false; }
            tc_fence_after_sync();
            const float inv = 1.0f / l;
            bf16* dst = static_cast<bf16*>(a.out) + (size_t)(row0 + qi) * a.ldo + h * DH;
#pragma unroll
            for (int e0 = 0; e0 < DH; e0 += 16) {
                float o[16];
                tmem_ld16(lane_addr + 128 + e0, o);   // warp-wide: every lane takes part
                if (ok && qi < cnt) {
                    uint4 lo, hi;
                    lo.x = pack_bf16x2(o[0] * inv, o[1] * inv); lo.y = pack_bf16x2(o[2] * inv, o[3] * inv);
                    lo.z = pack_bf16x2(o[4] * inv, o[5] * inv); lo.w = pack_bf16x2(o[6] * inv, o[7] * inv);
                    hi.x = pack_bf16x2(o[8] * inv, o[9] * inv); hi.y = pack_bf16x2(o[10] * inv, o[11] * inv);
                    hi.z = pack_bf16x2(o[12] * inv, o[13] * inv); hi.w = pack_bf16x2(o[14] * inv, o[15] * inv);
                    *reinterpret_cast<uint4*>(dst + e0) = lo;
                    *reinterpret_cast<uint4*>(dst + e0 + 8) = hi;
                }
            }
            tc_fence_before_sync();
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) tmem_dealloc(tmem, C::TMEM_COLS);
}

}  // namespace tandem
