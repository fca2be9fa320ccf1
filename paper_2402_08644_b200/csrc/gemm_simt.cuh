// SIMT GEMMs  y[m][n] = sum_k x[m][k] * W[n][k]  (weights [out][in]) with fused epilogues.
//
//  gemm_smallm_kernel  decode path (few rows): one warp per group of output columns streams the weight
//                      rows once with 16-byte loads; the rows of x sit in shared memory.  HBM-bound.
//                      Each output element is reduced in an order that depends only on K, never on the
//                      number of rows, so a block pass and a one-row pass give identical bits.
//  gemm_tiled_kernel   prompt path (many rows), classic shared-memory tiling.
//
// Both are the exact-arithmetic (fp32 FMA) paths of the fp32 test mode.
#pragma once
#include "common.cuh"

namespace tandem {

enum { EPI_STORE = 0, EPI_STORE_F32 = 1, EPI_GELU = 2, EPI_RESID = 3, EPI_QKV = 4, EPI_KV = 5 };

struct EpiArgs {
    void* out;            // EPI_STORE/GELU: T [M][ldo] (GELU on the tensor-core decode path: float);  STORE_F32/RESID: float [M][ldo];  QKV: q as T [M][ldo]
    int ldo;
    void* kcache;         // QKV / KV: this layer's keys   [B][H][t_max][d_head] (T)
    void* vcache;         //           this layer's values
    const int* row_seq;   // [M] sequence of each row
    const int* row_pos;   // [M] absolute position of each row
    int n_heads, d_head, t_max;   // n_heads: key/value heads of the cache
    int seg0;             // QKV / KV: columns of the first segment (QKV: the queries, d_model; KV: the keys)
    int seg;              //           columns of every further segment (keys / values: kv heads * d_head)
    void* out_lo;         // EPI_GELU on the tensor-core decode path, optional: `out` is then the bf16 plane of the values and this
                          // the bf16 plane of the remainders (x = value + remainder), both [M][ldo], for a consumer that loads them by TMA
    void* snap;           // EPI_RESID on the tensor-core decode path: optional fp32 copy of the new values [M][snap_ld]
    int snap_ld;
};

struct WSegs {            // up to three weight matrices stacked along N: [seg_rows0][K], then [seg_rows][K] each
    const void* w[3];
    int seg_rows0;
    int seg_rows;
};

template <typename T>
__device__ __forceinline__ const T* weight_row(const WSegs& ws, int n, int K) {
    if (n < ws.seg_rows0) return static_cast<const T*>(ws.w[0]) + (size_t)n * K;
    const int r = n - ws.seg_rows0, s = r / ws.seg_rows;
    return static_cast<const T*>(ws.w[1 + s]) + (size_t)(r - s * ws.seg_rows) * K;
}

template <typename T, int EPI>
__device__ __forceinline__ void epilogue(const EpiArgs& e, int m, int n, float v) {
    if (EPI == EPI_STORE) {
        static_cast<T*>(e.out)[(size_t)m * e.ldo + n] = from_float<T>(v);
    } else if (EPI == EPI_STORE_F32) {
        static_cast<float*>(e.out)[(size_t)m * e.ldo + n] = v;
    } else if (EPI == EPI_GELU) {
        static_cast<T*>(e.out)[(size_t)m * e.ldo + n] = from_float<T>(sizeof(T) == 2 ? gelu_bf16_out(v) : gelu_exact(v));
    } else if (EPI == EPI_RESID) {
        float* p = static_cast<float*>(e.out) + (size_t)m * e.ldo + n;
        *p = *p + v;
    } else {
        int s = 0, c = n;
        if (n >= e.seg0) { s = 1 + (n - e.seg0) / e.seg; c = (n - e.seg0) - (s - 1) * e.seg; }
        if (EPI == EPI_QKV) {
            if (s == 0) {
                static_cast<T*>(e.out)[(size_t)m * e.ldo + c] = from_float<T>(v);
                return;
            }
            s -= 1;
        }
        const int h = c / e.d_head, el = c - h * e.d_head;
        const size_t idx = (((size_t)e.row_seq[m] * e.n_heads + h) * e.t_max + e.row_pos[m]) * e.d_head + el;
        T* base = static_cast<T*>(s == 0 ? e.kcache : e.vcache);
        base[idx] = from_float<T>(v);
    }
}

constexpr int GS_THREADS = 256;
constexpr int GS_WARPS = GS_THREADS / 32;
constexpr int GS_COLS = 4;       // output columns per warp
constexpr int GS_KC = 2048;      // K elements of x staged in shared memory at a time

// grid: (ceil(N / (GS_WARPS*GS_COLS)), ceil(M / MT)); dynamic smem: MT * GS_KC * sizeof(T)
template <typename T, int MT, int EPI>
__global__ void __launch_bounds__(GS_THREADS)
gemm_smallm_kernel(const T* __restrict__ x, int ldx, int M, int K, WSegs ws, int N, EpiArgs e) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* xs = reinterpret_cast<T*>(smem_raw);
    constexpr int VN = VecN<T>::N;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = (blockIdx.x * GS_WARPS + warp) * GS_COLS;
    const int m0 = blockIdx.y * MT;

    const T* wrow[GS_COLS];
#pragma unroll
    for (int c = 0; c < GS_COLS; ++c) wrow[c] = (n0 + c < N) ? weight_row<T>(ws, n0 + c, K) : nullptr;

    float acc[MT][GS_COLS];
#pragma unroll
    for (int r = 0; r < MT; ++r)
#pragma unroll
        for (int c = 0; c < GS_COLS; ++c) acc[r][c] = 0.f;

    for (int k0 = 0; k0 < K; k0 += GS_KC) {
        const int kc = min(GS_KC, K - k0);
        const int vec_per_row = kc / VN;
        __syncthreads();
        for (int i = threadIdx.x; i < MT * vec_per_row; i += GS_THREADS) {
            const int r = i / vec_per_row, v = i - r * vec_per_row;
            uint4 val = make_uint4(0u, 0u, 0u, 0u);
            if (m0 + r < M) val = *reinterpret_cast<const uint4*>(x + (size_t)(m0 + r) * ldx + k0 + v * VN);
            *reinterpret_cast<uint4*>(xs + r * GS_KC + v * VN) = val;
        }
        __syncthreads();
#pragma unroll 2
        for (int kk = lane * VN; kk < kc; kk += 32 * VN) {
            float wv[GS_COLS][VN];
#pragma unroll
            for (int c = 0; c < GS_COLS; ++c) {
                uint4 raw = make_uint4(0u, 0u, 0u, 0u);
                if (wrow[c] != nullptr) raw = ldg_stream(wrow[c] + k0 + kk);
                widen(raw, wv[c]);
            }
#pragma unroll
            for (int r = 0; r < MT; ++r) {
                float xv[VN];
                load_vec(xs + r * GS_KC + kk, xv);
#pragma unroll
                for (int c = 0; c < GS_COLS; ++c)
#pragma unroll
                    for (int i = 0; i < VN; ++i) acc[r][c] = fmaf(xv[i], wv[c][i], acc[r][c]);
            }
        }
    }
#pragma unroll
    for (int r = 0; r < MT; ++r)
#pragma unroll
        for (int c = 0; c < GS_COLS; ++c) {
            const float v = warp_sum(acc[r][c]);
            if (lane == 0 && m0 + r < M && n0 + c < N) epilogue<T, EPI>(e, m0 + r, n0 + c, v);
        }
}

// Shared-memory tiled GEMM for many rows.  64x64 output tile, 16-deep K slices, 4x4 outputs per thread.
constexpr int GT_BM = 64, GT_BN = 64, GT_BK = 16, GT_THREADS = 256;

template <typename T, int EPI>
__global__ void __launch_bounds__(GT_THREADS)
gemm_tiled_kernel(const T* __restrict__ x, int ldx, int M, int K, WSegs ws, int N, EpiArgs e) {
    __shared__ float xs[GT_BK][GT_BM + 4];
    __shared__ float wsm[GT_BK][GT_BN + 4];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * GT_BM, n0 = blockIdx.x * GT_BN;
    // loader mapping: 64 rows x 16 k; each thread moves 4 consecutive k of one row
    const int lrow = tid >> 2, lk = (tid & 3) * 4;
    const T* xrow = (m0 + lrow < M) ? x + (size_t)(m0 + lrow) * ldx : nullptr;
    const T* wrow = (n0 + lrow < N) ? weight_row<T>(ws, n0 + lrow, K) : nullptr;

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < K; k0 += GT_BK) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int k = k0 + lk + i;
            xs[lk + i][lrow] = (xrow != nullptr && k < K) ? to_float(xrow[k]) : 0.f;
            wsm[lk + i][lrow] = (wrow != nullptr && k < K) ? to_float(wrow[k]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < GT_BK; ++k) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = xs[k][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = wsm[k][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
            if (m < M && n < N) epilogue<T, EPI>(e, m, n, acc[i][j]);
        }
}

}  // namespace tandem
