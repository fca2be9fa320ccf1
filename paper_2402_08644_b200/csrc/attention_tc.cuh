// Causal prompt attention (Eq. 1 over the prompt) on the tcgen05 tensor cores, bf16, head size 64 or 128.
//
// One CTA serves one (head, tile of up to 128 consecutive queries of one sequence).  The context is swept in
// chunks of 128 keys anchored at position 0, up to the tile's last query:
//     S  = Q K^T        one MMA group, M = 128 queries on the TMEM lanes, N = 128 keys, K = head size
//     P  = softmax step thread i owns query i: reads its row of S from TMEM, masks keys after its position,
//                       keeps the running maximum and sum, writes bf16 probabilities into a swizzled A tile
//     PV = P V          M = 128 queries, N = head size, K = 128 keys; V is used as it lies in the cache
//                       ([key][element], i.e. MN-major for the B operand)
//     O  = O * f + PV   in the thread's registers (f rescales to the new maximum)
// Warp 4 streams K and V chunks by TMA through a two-stage ring, warp 5 allocates TMEM and issues the MMAs,
// warps 0-3 do the softmax and the epilogue.  The tensor work hides behind the softmax: S of chunk c+1 (a second S
// buffer in TMEM) is computed while the softmax warps work on chunk c, and PV of chunk c while they take the maximum
// of chunk c+1; they add PV of chunk c only then.  Every wait is bounded.
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
constexpr int ATC_SUB = 128 * 128;        // bytes of one 128-row x 64-element bf16 sub-tile
template <int DH> struct AtcCfg {
    static constexpr int NSUB = DH / 64;                       // 64-element sub-tiles along the head dimension
    static constexpr int Q_BYTES = NSUB * ATC_SUB;
    static constexpr int KV_BYTES = 2 * NSUB * ATC_SUB;        // K and V of one chunk
    static constexpr int P_BYTES = 2 * ATC_SUB;                // 128 queries x 128 keys bf16
    static constexpr int SMEM_BYTES = Q_BYTES + 2 * KV_BYTES + P_BYTES + 1024;
    static constexpr int TMEM_COLS = 512;                      // S of even chunks: columns 0..127, PV: 128..128+DH-1, S of odd chunks: 256..383
};

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

// grid: (heads, groups); dynamic smem AtcCfg<DH>::SMEM_BYTES.
// tmq: queries [M][d_model] (box 64 x 128); tmk / tmv: one layer's cache seen as [(seq, head, position)][DH] (box 64 x 128).
template <int DH>
__global__ void __launch_bounds__(ATC_THREADS)
attn_prefill_tc_kernel(const AttnTcArgs a, const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                       const __grid_constant__ CUtensorMap tmv) {
    using C = AtcCfg<DH>;
    extern __shared__ __align__(1024) unsigned char smem_dyn[];
    __shared__ __align__(8) uint64_t s_qfull, s_kvfull[2], s_kvfree[2], s_sfull[2], s_pready, s_ofull;
    __shared__ uint32_t s_tmem;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t base0 = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* base = smem_dyn + (base0 - smem_u32(smem_dyn));
    const uint32_t q0 = base0, kv0 = base0 + C::Q_BYTES, p0 = kv0 + 2 * C::KV_BYTES;
    unsigned char* pg = base + C::Q_BYTES + 2 * C::KV_BYTES;

    const int h = blockIdx.x, g = blockIdx.y;
    const int row0 = a.grp_row0[g], cnt = a.grp_cnt[g];
    if (cnt <= 0) return;
    const int b = a.row_seq[row0];
    const int pos_first = a.row_pos[row0];
    const int pos_last = pos_first + cnt - 1;
    const int n_chunks = pos_last / 128 + 1;
    const int kv_row0 = (b * a.n_kv_heads + h / (a.n_heads / a.n_kv_heads)) * a.t_max;     // row of position 0 of this head's key/value head in the cache's 2-D view

    if (warp == 5) {
        if (lane == 0) {
            mbar_init(smem_u32(&s_qfull), 1);
            for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&s_kvfull[s]), 1); mbar_init(smem_u32(&s_kvfree[s]), 1); }
            mbar_init(smem_u32(&s_sfull[0]), 1);
            mbar_init(smem_u32(&s_sfull[1]), 1);
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
        if (lane == 0) {
            tma_prefetch_desc(&tmq); tma_prefetch_desc(&tmk); tma_prefetch_desc(&tmv);
            mbar_arrive_expect_tx(smem_u32(&s_qfull), C::Q_BYTES);
            for (int sb = 0; sb < C::NSUB; ++sb) tma_load_2d_nohint(q0 + sb * ATC_SUB, &tmq, h * DH + sb * 64, row0, smem_u32(&s_qfull));
            for (int c = 0; c < n_chunks; ++c) {
                const int st = c & 1;
                if (c >= 2 && !mbar_wait(smem_u32(&s_kvfree[st]), ((c >> 1) - 1) & 1)) { tc_report(a.err_flag, TC_ERR_SLOT); break; }
                const uint32_t bar = smem_u32(&s_kvfull[st]);
                mbar_arrive_expect_tx(bar, C::KV_BYTES);
                const uint32_t kdst = kv0 + st * C::KV_BYTES, vdst = kdst + C::NSUB * ATC_SUB;
                for (int sb = 0; sb < C::NSUB; ++sb) {
                    tma_load_2d_nohint(kdst + sb * ATC_SUB, &tmk, sb * 64, kv_row0 + c * 128, bar);
                    tma_load_2d_nohint(vdst + sb * ATC_SUB, &tmv, sb * 64, kv_row0 + c * 128, bar);
                }
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t idesc_s = umma_idesc_bf16_b(128, 128, 0);
            constexpr uint32_t idesc_o = umma_idesc_bf16_b(128, DH, 1);
            bool ok = mbar_wait(smem_u32(&s_qfull), 0);
            if (!ok) tc_report(a.err_flag, TC_ERR_OPERANDS);
            // S = Q K^T of chunk c into the S buffer c & 1: both K-major, 16 elements of the head dimension per instruction
            auto issue_s = [&](int c) -> bool {
                const int st = c & 1;
                if (!mbar_wait(smem_u32(&s_kvfull[st]), (c >> 1) & 1)) { tc_report(a.err_flag, TC_ERR_OPERANDS); return false; }
                tc_fence_after_sync();
                const uint32_t kaddr = kv0 + st * C::KV_BYTES;
#pragma unroll
                for (int sb = 0; sb < C::NSUB; ++sb)
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_bf16(tmem + st * 256, umma_desc_k_sw128(q0 + sb * ATC_SUB) + 2 * k, umma_desc_k_sw128(kaddr + sb * ATC_SUB) + 2 * k, idesc_s,
                                  (sb | k) != 0 ? 1u : 0u);
                umma_commit(smem_u32(&s_sfull[st]));
                return true;
            };
            ok = ok && issue_s(0);
            for (int c = 0; c < n_chunks && ok; ++c) {
                const int st = c & 1;
                // the next chunk's scores are computed while the softmax warps work on this one (its S buffer was
                // released with the probabilities of chunk c - 1)
                if (c + 1 < n_chunks && !issue_s(c + 1)) break;
                if (!mbar_wait(smem_u32(&s_pready), c & 1)) { tc_report(a.err_flag, TC_ERR_ACCUM); break; }
                tc_fence_after_sync();
                const uint32_t vaddr = kv0 + st * C::KV_BYTES + C::NSUB * ATC_SUB;
                // PV = P V: P K-major (two 64-key sub-tiles), V MN-major; 16 keys per instruction
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t dp = umma_desc_k_sw128(p0 + (ks >> 2) * ATC_SUB) + 2 * (ks & 3);
                    const uint64_t dv = umma_desc_mn_sw128(vaddr + ks * 2048, ATC_SUB);
                    umma_bf16(tmem + 128, dp, dv, idesc_o, ks != 0 ? 1u : 0u);
                }
                umma_commit(smem_u32(&s_kvfree[st]));   // K, V of this stage may be overwritten
                umma_commit(smem_u32(&s_ofull));        // PV is complete; the P tile may be rewritten
            }
        }
        __syncwarp();
    } else {
        const int qi = warp * 32 + lane;                 // this thread's query = TMEM lane
        const int qpos = pos_first + qi;                 // (rows past cnt compute on whatever the tile holds; never stored)
        const uint32_t lane_addr = tmem + (static_cast<uint32_t>(warp * 32) << 16);
        float o[DH];
#pragma unroll
        for (int e = 0; e < DH; ++e) o[e] = 0.f;
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        for (int c = 0; c < n_chunks && ok; ++c) {
            if (!mbar_wait(smem_u32(&s_sfull[c & 1]), (c >> 1) & 1)) { tc_report(a.err_flag, TC_ERR_ACCUM); ok = false; break; }
            tc_fence_after_sync();
            const uint32_t s_addr = lane_addr + (c & 1) * 256;
            // pass 1: the row's maximum over this chunk (every chunk but the tile's last one or two lies wholly before
            // the tile's first query: no key of it is masked for any row)
            const bool full = c * 128 + 127 <= pos_first;
            float mc = -INFINITY;
#pragma unroll 1
            for (int c0 = 0; c0 < 128; c0 += 16) {
                float t[16];
                tmem_ld16(s_addr + c0, t);
                if (full) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) mc = fmaxf(mc, t[i] * a.scale);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (c * 128 + c0 + i <= qpos) mc = fmaxf(mc, t[i] * a.scale);
                }
            }
            const float mn = fmaxf(m, mc);
            const float f = m > -INFINITY ? __expf(m - mn) : 0.f;
            m = mn;
            // O += PV of the previous chunk (it ran during pass 1; it is on the scale of the previous maximum, like o),
            // which also frees the P tile
            if (c > 0) {
                if (!mbar_wait(smem_u32(&s_ofull), (c - 1) & 1)) { tc_report(a.err_flag, TC_ERR_ACCUM); ok = false; break; }
                tc_fence_after_sync();
#pragma unroll
                for (int e0 = 0; e0 < DH; e0 += 16) {
                    float t[16];
                    tmem_ld16(lane_addr + 128 + e0, t);
#pragma unroll
                    for (int i = 0; i < 16; ++i) o[e0 + i] += t[i];
                }
            }
            // pass 2: probabilities, row sum, bf16 P tile (row qi: 128 keys = two sub-tiles of 64, 128-byte swizzle)
            float ls = 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < 128; c0 += 16) {
                float t[16];
                tmem_ld16(s_addr + c0, t);
                uint32_t pk[8];
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    const float p0v = (full || (c * 128 + c0 + i <= qpos && mn > -INFINITY)) ? __expf(t[i] * a.scale - mn) : 0.f;
                    const float p1v = (full || (c * 128 + c0 + i + 1 <= qpos && mn > -INFINITY)) ? __expf(t[i + 1] * a.scale - mn) : 0.f;
                    const __nv_bfloat162 pb = __floats2bfloat162_rn(p0v, p1v);
                    // the sum uses the rounded values, the same ones the tensor core multiplies with V
                    ls += __bfloat162float(pb.x) + __bfloat162float(pb.y);
                    pk[i >> 1] = *reinterpret_cast<const uint32_t*>(&pb);
                }
                const int sub = c0 >> 6, ch = (c0 & 63) >> 3;   // 16 keys = two 16-byte chunks
                unsigned char* prow = pg + sub * ATC_SUB + qi * 128;
                *reinterpret_cast<uint4*>(prow + (((ch) ^ (qi & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                *reinterpret_cast<uint4*>(prow + (((ch + 1) ^ (qi & 7)) << 4)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
            }
            l = l * f + ls;
            if (f != 1.f) {   // a factor of exactly 1 (no new maximum) changes nothing
#pragma unroll
                for (int e = 0; e < DH; ++e) o[e] *= f;
            }
            tc_fence_before_sync();      // the TMEM reads of S are done before the next chunk's MMA may overwrite it
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_pready));
        }
        if (ok) {   // the last chunk's PV
            if (!mbar_wait(smem_u32(&s_ofull), (n_chunks - 1) & 1)) { tc_report(a.err_flag, TC_ERR_ACCUM); ok = false; }
            tc_fence_after_sync();
            if (ok) {
#pragma unroll
                for (int e0 = 0; e0 < DH; e0 += 16) {
                    float t[16];
                    tmem_ld16(lane_addr + 128 + e0, t);
#pragma unroll
                    for (int i = 0; i < 16; ++i) o[e0 + i] += t[i];
                }
            }
            tc_fence_before_sync();
        }
        if (ok && qi < cnt) {
            const float inv = 1.0f / l;
            bf16* dst = static_cast<bf16*>(a.out) + (size_t)(row0 + qi) * a.ldo + h * DH;
#pragma unroll
            for (int e = 0; e < DH; e += 8) {
                uint4 v;
                v.x = pack_bf16x2(o[e] * inv, o[e + 1] * inv); v.y = pack_bf16x2(o[e + 2] * inv, o[e + 3] * inv);
                v.z = pack_bf16x2(o[e + 4] * inv, o[e + 5] * inv); v.w = pack_bf16x2(o[e + 6] * inv, o[e + 7] * inv);
                *reinterpret_cast<uint4*>(dst + e) = v;
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) tmem_dealloc(tmem, C::TMEM_COLS);
}

}  // namespace tandem
