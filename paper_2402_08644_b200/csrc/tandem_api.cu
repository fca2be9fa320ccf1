// Host side of the C boundary: context, arena layout, pass scheduling, and the exported entry points.
#include <cuda_runtime.h>
#include <limits.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <time.h>

#include <algorithm>
#include <atomic>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/tandem.h"
#include "attention.cuh"
#include "attention_tc.cuh"
#include "common.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "misc_kernels.cuh"
#include "router.cuh"
#include "sampling.cuh"

using namespace tandem;

namespace {

thread_local char g_cuda_err[256] = "";

#define CK(call)                                                                                  \
    do {                                                                                          \
        cudaError_t err__ = (call);                                                               \
        if (err__ != cudaSuccess) {                                                               \
            snprintf(g_cuda_err, sizeof(g_cuda_err), "%s at %s:%d", cudaGetErrorString(err__), __FILE__, __LINE__); \
            return TANDEM_ERR_CUDA;                                                               \
        }                                                                                         \
    } while (0)
#define TRY(expr)                             \
    do {                                      \
        tandem_status st__ = (expr);          \
        if (st__ != TANDEM_OK) return st__;   \
    } while (0)

size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }
int cdiv(int a, int b) { return (a + b - 1) / b; }

struct Layout {   // byte offsets into the arena
    size_t kv_large, kv_small;
    size_t st_n, st_pending, st_drafts, st_targets, st_accept, st_emitted, st_done, st_out, st_counters, st_hist;
    size_t st_block_len, st_drafting, st_confidence;
    size_t forced_ids, forced_len, forced_nll, forced_top;   // teacher-forced forward: given tokens [B][T], lengths [B], scores [B][T]
    size_t row_tok, row_seq, row_pos, grp_row0, grp_cnt;
    size_t attn_counters;   // inside the zero-filled state block
    size_t h_large, h_small, a, q, o, f, xb, t1, yhat, a_s, logits_large, logits_small, part_ml, part_acc, dbg;
    size_t amax_val_large, amax_idx_large, amax_val_small, amax_idx_small;
    size_t a32, o32, f32;                           // fp32 activations between the bf16 decode kernels: LayerNorm / attention / GELU outputs
    size_t proj_snap, proj_yhat, proj_a, proj_t1;   // per small layer: the decode projection's own buffers (it runs beside the large pass)
    size_t total;
    int max_rows, dec_rows, max_groups, n_chunks_max, vocab_tiles;
    size_t kv_large_layer, kv_small_layer;   // elements per (layer, k-or-v)
};

struct Model {
    tandem_dims d;
    int kv_heads, d_kv;     // key/value heads and the width of a position's keys (kv_heads * d_head)
    int wbase;
    size_t kv_off;          // arena offset of this model's KV cache
    size_t kv_layer_elems;  // elements per (layer, K or V): B * kv_heads * T * dh
};

}  // namespace

enum { PC_GEMM_SMALLM = 0, PC_GEMM_TILED, PC_ATTN_SPLIT, PC_ATTN_MERGE, PC_ATTN_PROMPT, PC_LAYERNORM, PC_ROWS, PC_ARGMAX,
       PC_VERIFY, PC_GEMM_TC_DECODE, PC_GEMM_TC_TILED, PC_COUNT };

struct Prof {   // optional per-launch timing with CUDA events (measurement hook)
    bool on = false;
    std::vector<cudaEvent_t> ev;
    std::vector<int> cls;
    std::vector<double> bytes;
    size_t used = 0;   // events used (two per launch)
};

struct tandem_ctx {
    Prof prof;
    tandem_config cfg;
    std::vector<int32_t> layer_map;
    std::vector<const void*> w;
    Layout lay;
    Model large, small;
    int tbase;          // first FF_Tandem weight index
    int hidden;
    unsigned char* arena;
    cudaStream_t stream;
    size_t esz;         // storage element size
    // host trackers
    int batch;          // sequences of the current prefill (0 = none)
    int n_ub;           // upper bound on max_b n_b (exact after every synchronising call)
    long long n_sum;    // sum_b n_b at the last synchronisation (accounting only)
    int32_t* pinned;    // staging for prefill row arrays and small read-backs
    size_t pinned_ints;
    int64_t launches = 0;
    int last_gamma = 0;
    LoopState st{};
    // CUDA graphs of one iteration, keyed by everything baked into the captured launches
    struct GraphEntry {
        int kind, gamma, mode, max_new, batch, chunks;
        uint64_t seed;
        bool warm;
        cudaGraphExec_t exec;
        int64_t kernels;
    };
    std::vector<GraphEntry> graphs;
    cudaStream_t cap_stream = nullptr;   // capture happens here (the caller's stream may be the legacy default stream)
    bool use_graphs = true;
    int chunks_launch = 1;               // attention grid size along the context for the current iteration
    int32_t* hflags = nullptr;           // mapped pinned host memory the verify kernel publishes to
    int64_t ticket = 0;                  // verify kernels enqueued since creation
    // tensor-core path (bf16 only)
    bool tc = false;                     // weights have tensor maps; GEMMs run on tcgen05
    bool use_pdl = true;                 // programmatic dependent launch between the decode kernels
    int n_sms = 0;                       // multiprocessors of the context's device: split-K decode GEMMs aim for about one CTA each
    std::vector<CUtensorMap> wmap;       // one per weight pointer (matrices only), box 128 rows x 64 columns
    // Decode activations as two bf16 planes (values, then remainders, dec_rows rows each) that the consuming GEMM loads by
    // TMA: maps of the LayerNorm / attention / GELU buffers, [buffer 0..2][0 large, 1 small], 16-row boxes.
    CUtensorMap xmap[3][2];
    bool xmap_ok = false;
    std::vector<char> wmap_ok;
    std::vector<CUtensorMap> kmap, vmap; // the large model's key / value cache of each layer as [(seq, head, position)][d_head]
    cudaStream_t side = nullptr;         // the decode-time FF_Tandem projections run here, beside the large model's later layers
    std::vector<cudaEvent_t> ev_fork;    // one per small layer
    cudaEvent_t ev_join = nullptr;
    bool next_launch_plain = false;      // the next launch follows a cross-stream wait: no programmatic dependency on a kernel
    bool setup_failed = false;           // a launch helper could not encode a tensor map: reported by the enclosing call
    bool tc_prompt_attn = false;         // prompt attention on the tensor cores (head size 64 or 128)
    int prompt_group = ATT_NQ;           // queries per attention group of the prompt pass
    float temp_large = 1.0f, temp_small = 1.0f;   // sampled SPEED (accept mode 4): temperatures of the two models
    RouterArgs router{};                 // adaptive block length: the router's weights (caller-owned, DEVICE) and threshold
    bool has_router = false;
    int64_t router_ticket = 0;           // router launches since the prompt pass
    double prompt_sq_sum = 0.0;          // sum over the sequences of the current prompt pass of (rows)^2 (accounting of the attention's work)
};

namespace {
// Brackets one launch with two events when profiling is on.
struct ProfScope {
    tandem_ctx& c;
    bool active;
    ProfScope(tandem_ctx& ctx, int cls, double bytes) : c(ctx), active(false) {
        Prof& p = c.prof;
        if (p.on && p.used + 2 <= p.ev.size()) {
            active = true;
            p.cls.push_back(cls);
            p.bytes.push_back(bytes);
            cudaEventRecord(p.ev[p.used], c.stream);
        }
    }
    ~ProfScope() {
        if (active) { cudaEventRecord(c.prof.ev[c.prof.used + 1], c.stream); c.prof.used += 2; }
    }
};
}  // namespace

namespace {

int dims_ok(const tandem_dims& d) {
    if (d.n_layers < 1 || d.d_model < 8 || d.n_heads < 1 || d.d_ff < 8 || d.vocab < 1 || d.max_pos < 1) return 0;
    if (d.d_model % d.n_heads) return 0;
    const int dh = d.d_model / d.n_heads;
    if (dh != 32 && dh != 64 && dh != 128) return 0;
    if (d.d_model % 8 || d.d_ff % 8) return 0;
    if (d.n_kv_heads < 0 || (d.n_kv_heads > 0 && d.n_heads % d.n_kv_heads)) return 0;
    return 1;
}
int kv_heads_of(const tandem_dims& d) { return d.n_kv_heads > 0 ? d.n_kv_heads : d.n_heads; }
int d_kv_of(const tandem_dims& d) { return kv_heads_of(d) * (d.d_model / d.n_heads); }

tandem_status validate(const tandem_config* c) {
    if (!c || !c->layer_map) return TANDEM_ERR_INVALID_ARG;
    if (c->dtype != TANDEM_DTYPE_FP32 && c->dtype != TANDEM_DTYPE_BF16) return TANDEM_ERR_INVALID_ARG;
    if (c->ff_tandem_kind != TANDEM_FF_LINEAR && c->ff_tandem_kind != TANDEM_FF_MLP) return TANDEM_ERR_INVALID_ARG;
    if (c->max_batch < 1 || c->max_seq < 2 || c->gamma_max < 0 || c->gamma_max > TANDEM_GAMMA_LIMIT) return TANDEM_ERR_INVALID_ARG;
    if (c->max_prefill_rows < 0 || c->ff_tandem_hidden < 0 || c->device < 0) return TANDEM_ERR_INVALID_ARG;
    if (!dims_ok(c->large) || !dims_ok(c->small)) return TANDEM_ERR_SHAPE;
    if (c->large.vocab != c->small.vocab) return TANDEM_ERR_SHAPE;
    if (c->ff_tandem_hidden % 8) return TANDEM_ERR_SHAPE;
    if ((long long)c->max_batch * (c->gamma_max + 1) > 256) return TANDEM_ERR_SHAPE;
    for (int j = 0; j < c->small.n_layers; ++j)
        if (c->layer_map[j] < 0 || c->layer_map[j] > c->large.n_layers) return TANDEM_ERR_INVALID_ARG;
    return TANDEM_OK;
}

Layout make_layout(const tandem_config& c) {
    Layout L;
    memset(&L, 0, sizeof(L));
    const size_t esz = c.dtype == TANDEM_DTYPE_BF16 ? 2 : 4;
    const size_t B = c.max_batch, T = c.max_seq, GL = TANDEM_GAMMA_LIMIT;
    const int hidden = c.ff_tandem_hidden > 0 ? c.ff_tandem_hidden : c.small.d_model;
    L.dec_rows = c.max_batch * (c.gamma_max + 1);
    const long long pre = c.max_prefill_rows > 0 ? c.max_prefill_rows : (long long)c.max_batch * c.max_seq;
    L.max_rows = (int)std::max<long long>(pre, L.dec_rows);
    L.max_groups = L.max_rows / ATT_NQ + c.max_batch + 1;
    L.n_chunks_max = cdiv(c.max_seq, ATT_CH);
    const size_t dmax = std::max(std::max(c.large.d_model, c.small.d_model), hidden);
    const size_t fmax = std::max(c.large.d_ff, c.small.d_ff);
    const size_t hmax = std::max(c.large.n_heads, c.small.n_heads);
    const size_t R = L.max_rows, RD = L.dec_rows, V = c.large.vocab;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    L.kv_large_layer = B * T * d_kv_of(c.large);
    L.kv_small_layer = B * T * d_kv_of(c.small);
    L.kv_large = take((size_t)c.large.n_layers * 2 * L.kv_large_layer * esz);
    L.kv_small = take((size_t)c.small.n_layers * 2 * L.kv_small_layer * esz);
    L.st_n = take(B * 4); L.st_pending = take(B * 4); L.st_drafts = take(B * GL * 4);
    L.st_targets = take(B * (GL + 1) * 4); L.st_accept = take(B * 4); L.st_emitted = take(B * 4);
    L.st_done = take(B * 4); L.st_out = take(B * T * 4); L.st_counters = take(16 * 4); L.st_hist = take((GL + 1) * 8);
    L.st_block_len = take(B * 4); L.st_drafting = take(B * 4); L.st_confidence = take(B * GL * 4);
    L.row_tok = take(R * 4); L.row_seq = take(R * 4); L.row_pos = take(R * 4);
    L.grp_row0 = take((size_t)L.max_groups * 4); L.grp_cnt = take((size_t)L.max_groups * 4);
    L.attn_counters = take(B * hmax * 4);
    L.h_large = take(R * c.large.d_model * 4);
    L.h_small = take(B * c.small.d_model * 4);
    L.a = take(R * dmax * esz); L.q = take(R * dmax * esz); L.o = take(R * dmax * esz);
    L.f = take(R * fmax * esz);
    L.xb = take(R * c.large.d_model * esz); L.t1 = take(R * hidden * esz);
    L.yhat = take(R * c.small.d_model * 4); L.a_s = take(R * c.small.d_model * esz);
    L.logits_large = take(RD * V * 4);
    L.logits_small = take((size_t)std::max(1, c.gamma_max) * B * V * 4);
    L.part_ml = take(RD * hmax * L.n_chunks_max * 2 * 4);
    L.part_acc = take(RD * dmax * L.n_chunks_max * 4);
    L.dbg = take(T * dmax * 4);
    L.forced_ids = take(B * T * 4); L.forced_len = take(B * 4); L.forced_nll = take(B * T * 4); L.forced_top = take(B * T * 4);
    L.vocab_tiles = cdiv(c.large.vocab, 128);
    L.amax_val_large = take(RD * L.vocab_tiles * 4); L.amax_idx_large = take(RD * L.vocab_tiles * 4);
    L.amax_val_small = take(B * L.vocab_tiles * 4); L.amax_idx_small = take(B * L.vocab_tiles * 4);
    const size_t nS = c.small.n_layers;
    L.a32 = take(RD * dmax * 4); L.o32 = take(RD * dmax * 4); L.f32 = take(RD * fmax * 4);
    L.proj_snap = take(nS * RD * c.large.d_model * 4);
    L.proj_yhat = take(nS * RD * c.small.d_model * 4);
    L.proj_a = take(nS * RD * c.small.d_model * 4);
    L.proj_t1 = take(nS * RD * hidden * 4);
    L.total = off;
    return L;
}

int n_weight_ptrs(const tandem_config& c) {
    const int per_t = c.ff_tandem_kind == TANDEM_FF_LINEAR ? 1 : 2;
    return (5 + 10 * c.large.n_layers) + (5 + 10 * c.small.n_layers) + per_t * c.small.n_layers;
}

enum { W_LN1G = 0, W_LN1B, W_WQ, W_WK, W_WV, W_WO, W_LN2G, W_LN2B, W_W1, W_W2 };
inline const void* w_emb(const tandem_ctx& c, const Model& m) { return c.w[m.wbase]; }
inline const void* w_pos(const tandem_ctx& c, const Model& m) { return c.w[m.wbase + 1]; }
inline const void* w_layer(const tandem_ctx& c, const Model& m, int l, int k) { return c.w[m.wbase + 2 + 10 * l + k]; }
inline const void* w_tail(const tandem_ctx& c, const Model& m, int k) { return c.w[m.wbase + 2 + 10 * m.d.n_layers + k]; }

inline int wi_layer(const Model& m, int l, int k) { return m.wbase + 2 + 10 * l + k; }
inline int wi_tail(const Model& m, int k) { return m.wbase + 2 + 10 * m.d.n_layers + k; }
inline int wi_tandem(const tandem_ctx& c, int j, int k) { return c.tbase + (c.cfg.ff_tandem_kind == TANDEM_FF_LINEAR ? j : 2 * j + k); }

// A linear map given by the indices of up to three weight matrices stacked along the output features.
// (the first matrix has seg_rows0 rows, the others seg_rows each: queries next to narrower keys / values)
struct Lin { int i0, i1, i2, seg_rows0, seg_rows, K; };
inline Lin lin1(int i0, int rows, int K) { Lin l = {i0, -1, -1, rows, rows, K}; return l; }
inline Lin lin3(int i0, int i1, int i2, int rows0, int rows, int K) { Lin l = {i0, i1, i2, rows0, rows, K}; return l; }
inline int lin_n(const Lin& l) { return l.seg_rows0 + ((l.i1 >= 0) + (l.i2 >= 0)) * l.seg_rows; }

template <typename P> P* at(tandem_ctx& c, size_t off) { return reinterpret_cast<P*>(c.arena + off); }

constexpr int MAX_DEVICES = 64;
int cur_dev() {   // opt-in shared-memory sizes are per device
    int d = 0;
    cudaGetDevice(&d);
    return (d >= 0 && d < MAX_DEVICES) ? d : 0;
}

// ---------------------------------------------------------------------------------------------------
// launch helpers
// ---------------------------------------------------------------------------------------------------

// Opt-in dynamic shared memory of a kernel, requested once per device (`done`: one bit per device, one word per
// kernel instantiation).  The attribute call is idempotent, so two threads racing to be first is harmless.
template <typename K>
void ensure_dyn_smem(K kernel, size_t bytes, std::atomic<unsigned long long>& done) {
    const unsigned long long bit = 1ull << cur_dev();
    if (done.load(std::memory_order_acquire) & bit) return;
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    done.fetch_or(bit, std::memory_order_release);
}

// Multiprocessors of the current device (asked once per device).
int sm_count() {
    static std::atomic<int> cache[MAX_DEVICES];
    const int dev = cur_dev();
    int n = cache[dev].load(std::memory_order_relaxed);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 1;
    cache[dev].store(n, std::memory_order_relaxed);
    return n;
}

template <typename T, int MT, int EPI>
void launch_smallm(tandem_ctx& c, const T* x, int ldx, int M, int K, const WSegs& ws, int N, const EpiArgs& e) {
    static std::atomic<unsigned long long> attr_done{0};
    const size_t smem = (size_t)MT * GS_KC * sizeof(T);
    ensure_dyn_smem(gemm_smallm_kernel<T, MT, EPI>, smem, attr_done);
    dim3 grid(cdiv(N, GS_WARPS * GS_COLS), cdiv(M, MT));
    ProfScope ps(c, PC_GEMM_SMALLM, ((double)N * K + (double)M * K + (double)M * N) * sizeof(T));
    gemm_smallm_kernel<T, MT, EPI><<<grid, GS_THREADS, smem, c.stream>>>(x, ldx, M, K, ws, N, e);
    c.launches++;
}

// ---------------------------------------------------------------------------------------------------
// tensor-core GEMMs: tensor maps and launches
// ---------------------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (the library does not link libcuda).
EncodeTiledFn tmap_encoder() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
        return q == cudaDriverEntryPointSuccess ? reinterpret_cast<EncodeTiledFn>(p) : nullptr;
    }();
    return fn;
}

// bf16 matrix [rows][cols] with leading dimension ld (elements), tiles of box_rows (128 by default) rows x 64 columns,
// 128-byte swizzle.  base 16-byte aligned, ld a multiple of 8.
bool make_tmap_bf16(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows = 128) {
    EncodeTiledFn enc = tmap_encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct TcW {              // up to three weight matrices stacked along the output features
    CUtensorMap tm[3];
    int n_segs, seg_rows0, seg_rows, K;   // rows of the first segment, rows of every further one
};
inline int tcw_n(const TcW& w) { return w.seg_rows0 + (w.n_segs - 1) * w.seg_rows; }
struct TcScratch {
    int* err;                  // where a bounded wait that ran out records its code (nullable)
    unsigned poll_limit = 0;   // 0: the kernels' default
    int withhold_weights = 0;  // test hook, see TcDecodeArgs
};

TcW tcw3(const tandem_ctx& c, int i0, int i1, int i2, int seg_rows0, int seg_rows, int K) {
    TcW w;
    w.tm[0] = c.wmap[i0];
    w.tm[1] = c.wmap[i1 >= 0 ? i1 : i0];
    w.tm[2] = c.wmap[i2 >= 0 ? i2 : i0];
    w.n_segs = 1 + (i1 >= 0) + (i2 >= 0);
    w.seg_rows0 = seg_rows0; w.seg_rows = seg_rows; w.K = K;
    return w;
}
TcW tcw(const tandem_ctx& c, int i0, int i1, int i2, int seg_rows, int K) { return tcw3(c, i0, i1, i2, seg_rows, seg_rows, K); }

TcScratch tc_scratch(tandem_ctx& c) {
    TcScratch s;
    s.err = c.st.counters ? c.st.counters + 2 : nullptr;
    return s;
}

template <typename... KArgs, typename... Args>
void launch_ex(tandem_ctx& c, bool pdl, int cluster, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, Args&&... args) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = c.stream;
    cudaLaunchAttribute attr[2];
    int n = 0;
    const bool plain = c.next_launch_plain;
    c.next_launch_plain = false;
    if (pdl && c.use_pdl && !plain) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (cluster > 1) {   // consecutive blocks along x form a thread-block cluster
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)cluster; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
    c.launches++;
}

template <int NB, int PRO, int EPI>
void launch_tc_decode_nb(tandem_ctx& c, const TcDecodeArgs& a, const TcW& w, int units, const CUtensorMap* xmap) {
    using C = TcdCfg<NB>;
    static std::atomic<unsigned long long> attr_done{0};
    ensure_dyn_smem(gemm_tc_decode_kernel<NB, PRO, EPI>, C::SMEM_BYTES, attr_done);
    launch_ex(c, true, a.splits, gemm_tc_decode_kernel<NB, PRO, EPI>, dim3(units), dim3(TCD_THREADS), (size_t)C::SMEM_BYTES, a, w.tm[0], w.tm[1], w.tm[2],
              xmap ? *xmap : w.tm[0]);
}

// y = prologue(x) W^T for few rows on the tensor cores, streaming W once per group of up to 64 rows (one group in
// every benchmark configuration; more rows than that re-read the weights per group, with unchanged arithmetic).
template <int PRO, int EPI>
void launch_tc_decode(tandem_ctx& c, const TcScratch& sc, const void* x, int ldx, const void* ln_g, const void* ln_b, int rows,
                      const TcW& w, bool stream_weights, const EpiArgs& e, float* amax_val = nullptr, int* amax_idx = nullptr,
                      int amax_stride = 0, const CUtensorMap* xmap = nullptr, int x_plane_rows = 0) {
    if (rows <= 0) return;
    TcDecodeArgs a;
    memset(&a, 0, sizeof(a));
    a.ldx = ldx; a.ln_g = static_cast<const float*>(ln_g); a.ln_b = static_cast<const float*>(ln_b);
    a.K = w.K; a.N = tcw_n(w); a.seg_rows0 = w.seg_rows0; a.tiles0 = cdiv(w.seg_rows0, 128);
    a.seg_rows = w.seg_rows; a.tiles_per_seg = cdiv(w.seg_rows, 128);
    const int tiles = a.tiles0 + (w.n_segs - 1) * a.tiles_per_seg, KB = cdiv(w.K, 64);
    // K-slices per tile = cluster size: the smallest power of two that puts tiles * S CTAs at or above one per
    // multiprocessor, at most 8 and at most one per 64-element K-block.  The head GEMM keeps whole tiles.
    int S = 1;
    if (EPI != EPI_ARGMAX)
        while (S < 8 && 2 * S <= KB && tiles * S < c.n_sms) S *= 2;
    a.splits = S;
    a.stream_weights = stream_weights ? 1 : 0;
    a.err_flag = sc.err;
    a.poll_limit = sc.poll_limit;
    a.withhold_weights = sc.withhold_weights;
    a.amax_stride = amax_stride;
    const size_t xsz = PRO == PRO_BF16 ? 2 : 4;
    const size_t osz = EPI == EPI_STORE ? 2 : 4;       // EPI_QKV: the query buffer is bf16 too (below)
    const int units = tiles * S;
    for (int r0 = 0; r0 < rows; r0 += 64) {
        const int nr = std::min(64, rows - r0);
        a.rows = nr;
        a.x_row0 = r0; a.x_plane_rows = x_plane_rows;
        a.release_early = (size_t)a.N * (size_t)w.K * 2 <= ((size_t)16 << 20) ? 1 : 0;
        a.x = static_cast<const unsigned char*>(x) + (size_t)r0 * ldx * xsz;
        a.amax_val = amax_val ? amax_val + (size_t)r0 * amax_stride : nullptr;
        a.amax_idx = amax_idx ? amax_idx + (size_t)r0 * amax_stride : nullptr;
        a.e = e;
        if (e.out) a.e.out = static_cast<unsigned char*>(e.out) + (size_t)r0 * e.ldo * ((EPI == EPI_QKV || e.out_lo) ? 2 : osz);
        if (e.out_lo) a.e.out_lo = static_cast<unsigned char*>(e.out_lo) + (size_t)r0 * e.ldo * 2;   // (value / remainder planes are bf16)
        if (e.row_seq) { a.e.row_seq = e.row_seq + r0; a.e.row_pos = e.row_pos + r0; }
        if (e.snap) a.e.snap = static_cast<float*>(e.snap) + (size_t)r0 * e.snap_ld;
        ProfScope ps(c, PC_GEMM_TC_DECODE, 2.0 * a.N * w.K + (double)nr * w.K * xsz + (double)nr * a.N * (EPI == EPI_QKV || EPI == EPI_KV || EPI == EPI_STORE ? 2.0 : 4.0));
        if (nr <= 16) launch_tc_decode_nb<16, PRO, EPI>(c, a, w, units, xmap);
        else if (nr <= 32) launch_tc_decode_nb<32, PRO, EPI>(c, a, w, units, xmap);
        else if (nr <= 48) launch_tc_decode_nb<48, PRO, EPI>(c, a, w, units, xmap);
        else launch_tc_decode_nb<64, PRO, EPI>(c, a, w, units, xmap);
    }
}

// y = x W^T for many rows on the tensor cores; x bf16 [M][ldx].
template <int EPI, int BN>
void launch_tc_tiled_bn(tandem_ctx& c, TcTiledArgs& a, const CUtensorMap& tmx, const TcW& w, int M) {
    using C = TctCfg<BN>;
    static std::atomic<unsigned long long> attr_done{0};
    ensure_dyn_smem(gemm_tc_tiled_kernel<EPI, BN>, C::SMEM_BYTES, attr_done);
    a.tiles0 = cdiv(w.seg_rows0, BN);
    a.tiles_per_seg = cdiv(w.seg_rows, BN);
    a.tiles_n = a.tiles0 + (w.n_segs - 1) * a.tiles_per_seg;
    a.tiles_m = cdiv(M, 128);
    launch_ex(c, false, 1, gemm_tc_tiled_kernel<EPI, BN>, dim3(std::min(a.tiles_n * a.tiles_m, std::max(1, c.n_sms))), dim3(TCT_THREADS), (size_t)C::SMEM_BYTES,
              a, tmx, w.tm[0], w.tm[1], w.tm[2]);
}

template <int EPI>
tandem_status launch_tc_tiled(tandem_ctx& c, const bf16* x, int ldx, int M, const TcW& w, const EpiArgs& e, int* err) {
    if (M <= 0) return TANDEM_OK;
    CUtensorMap tmx;
    if (!make_tmap_bf16(&tmx, x, (uint64_t)M, (uint64_t)w.K, (uint64_t)ldx)) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled failed for an activation buffer");
        return TANDEM_ERR_CUDA;
    }
    TcTiledArgs a;
    memset(&a, 0, sizeof(a));
    a.M = M; a.K = w.K; a.N = tcw_n(w); a.seg_rows0 = w.seg_rows0; a.seg_rows = w.seg_rows;
    a.err_flag = err; a.e = e;
    ProfScope ps(c, PC_GEMM_TC_TILED, 2.0 * M * (double)a.N * w.K);   // flops
    // 256-wide tiles when they still give every SM a tile, else square ones
    if ((long long)(cdiv(w.seg_rows0, 256) + (w.n_segs - 1) * cdiv(w.seg_rows, 256)) * cdiv(M, 128) >= c.n_sms) launch_tc_tiled_bn<EPI, 256>(c, a, tmx, w, M);
    else launch_tc_tiled_bn<EPI, 128>(c, a, tmx, w, M);
    return TANDEM_OK;
}

WSegs segs_of(const tandem_ctx& c, const Lin& l) {
    WSegs s;
    s.w[0] = c.w[l.i0];
    s.w[1] = l.i1 >= 0 ? c.w[l.i1] : nullptr;
    s.w[2] = l.i2 >= 0 ? c.w[l.i2] : nullptr;
    s.seg_rows0 = l.seg_rows0;
    s.seg_rows = l.seg_rows;
    return s;
}

// y = x W^T with a fused epilogue.  decode: few rows, streaming kernel; otherwise the prompt-pass kernels
// (tensor cores for bf16 when the context has tensor maps).
template <typename T, int EPI>
void launch_gemm(tandem_ctx& c, bool decode, const T* x, int ldx, int M, const Lin& l, const EpiArgs& e) {
    if (M <= 0) return;
    const WSegs ws = segs_of(c, l);
    const int N = lin_n(l), K = l.K;
    if (decode) {
        if (M <= 1) launch_smallm<T, 1, EPI>(c, x, ldx, M, K, ws, N, e);
        else if (M <= 2) launch_smallm<T, 2, EPI>(c, x, ldx, M, K, ws, N, e);
        else if (M <= 4) launch_smallm<T, 4, EPI>(c, x, ldx, M, K, ws, N, e);
        else launch_smallm<T, 8, EPI>(c, x, ldx, M, K, ws, N, e);
    } else if (sizeof(T) == 2 && c.tc) {
        if (launch_tc_tiled<EPI>(c, reinterpret_cast<const bf16*>(x), ldx, M, tcw3(c, l.i0, l.i1, l.i2, l.seg_rows0, l.seg_rows, l.K), e,
                                 c.st.counters + 2) != TANDEM_OK)
            c.setup_failed = true;
    } else {
        dim3 grid(cdiv(N, GT_BN), cdiv(M, GT_BM));
        ProfScope ps(c, PC_GEMM_TILED, 2.0 * M * (double)N * K);   // flops, not bytes: this one is compute-bound
        gemm_tiled_kernel<T, EPI><<<grid, GT_THREADS, 0, c.stream>>>(x, ldx, M, K, ws, N, e);
        c.launches++;
    }
}

template <typename T, int DH>
void launch_attn_dh(tandem_ctx& c, const AttnArgs& a, int groups, bool loop, int n_chunks, double kv_bytes) {
    static std::atomic<unsigned long long> attr_done_split{0}, attr_done_loop{0};
    ensure_dyn_smem(attn_kernel<T, DH, false>, attn_smem_bytes<T, DH>(), attr_done_split);
    ensure_dyn_smem(attn_kernel<T, DH, true>, attn_smem_bytes<T, DH>(), attr_done_loop);
    if (loop) {
        ProfScope ps(c, PC_ATTN_PROMPT, kv_bytes);
        launch_ex(c, false, 1, attn_kernel<T, DH, true>, dim3(1, a.n_heads, groups), dim3(ATT_THREADS), attn_smem_bytes<T, DH>(), a);
    } else {
        ProfScope ps(c, PC_ATTN_SPLIT, kv_bytes);
        launch_ex(c, true, 1, attn_kernel<T, DH, false>, dim3(n_chunks, a.n_heads, groups), dim3(ATT_THREADS), attn_smem_bytes<T, DH>(), a);
    }
}

template <typename T>
void launch_attn(tandem_ctx& c, int d_head, const AttnArgs& a, int groups, bool loop, int n_chunks, double kv_bytes) {
    if (d_head == 32) launch_attn_dh<T, 32>(c, a, groups, loop, n_chunks, kv_bytes);
    else if (d_head == 64) launch_attn_dh<T, 64>(c, a, groups, loop, n_chunks, kv_bytes);
    else launch_attn_dh<T, 128>(c, a, groups, loop, n_chunks, kv_bytes);
}

// bf16 decode attention: one cluster of `cl` CTAs per (sequence, head); no scratch.
template <int DH>
void launch_attn_decode_dq(tandem_ctx& c, const AttnArgs& a, int groups, int cl, double kv_bytes) {
    static std::atomic<unsigned long long> attr_done{0};
    ensure_dyn_smem(attn_decode_kernel<DH>, attn_decode_smem_bytes<DH>(), attr_done);
    ProfScope ps(c, PC_ATTN_SPLIT, kv_bytes);
    launch_ex(c, true, cl, attn_decode_kernel<DH>, dim3(cl, a.n_heads / std::max(1, a.heads_per_cta), groups), dim3(ATD_THREADS),
              attn_decode_smem_bytes<DH>(), a);
}
// Cluster size: the largest of 1, 2, 4, 8 that keeps the launch within one wave of resident CTAs (two per SM,
// one for 128-wide heads).  It depends on the number of sequences and heads only, so every pass of a run
// (block or one-row) cuts the context the same way.  (Sizes in between, which would fill the wave better, measured
// 3 % slower per iteration at batch 8: a cluster of three merges more states than its extra CTAs save.)
int attn_cluster_size(int n_sms, int groups, int n_heads, int d_head) {
    const long long slots = (long long)n_sms * (d_head == 128 ? 1 : 2);
    int cl = 1;
    while (cl < ATD_CLUSTER && (long long)groups * n_heads * cl * 2 <= slots) cl *= 2;
    return cl;
}
void launch_attn_decode(tandem_ctx& c, int d_head, const AttnArgs& a0, int groups, double kv_bytes) {
    AttnArgs a = a0;
    // Grouped-query attention: the query heads of one key/value head ride in one CTA as far as the 16-row tile has
    // room (heads * queries per block <= 16; a power of two that divides the group).  The cluster size is taken
    // from the key/value heads, which do not depend on the number of queries: a block pass and a one-row pass cut
    // the context the same way.
    const int n_kv = a.n_kv_heads > 0 ? a.n_kv_heads : a.n_heads;
    const int group = a.n_heads / n_kv;
    int gpc = 1;
    while (gpc * 2 <= group && group % (gpc * 2) == 0 && gpc * 2 * a.nq <= ATT_NQ) gpc *= 2;
    a.heads_per_cta = gpc;
    const int cl = attn_cluster_size(c.n_sms, groups, n_kv, d_head);
    if (d_head == 32) launch_attn_decode_dq<32>(c, a, groups, cl, kv_bytes);
    else if (d_head == 64) launch_attn_decode_dq<64>(c, a, groups, cl, kv_bytes);
    else launch_attn_decode_dq<128>(c, a, groups, cl, kv_bytes);
}

template <typename T>
void launch_layernorm(tandem_ctx& c, int M, const float* x, const void* gain, const void* bias, T* out, int d) {
    ProfScope ps(c, PC_LAYERNORM, (double)M * d * (4.0 + sizeof(T)));
    layernorm_kernel<T><<<M, 128, 0, c.stream>>>(x, static_cast<const float*>(gain), static_cast<const float*>(bias), out, d);
    c.launches++;
}

// Describes the rows of one pass.
struct Rows {
    int M;            // rows
    int groups;       // attention groups
    int nq;           // rows per group when group arrays are not used (decode)
    bool decode;      // decode kernels (split attention, streaming GEMM) or prompt kernels
    int n_chunks;     // split attention grid size along the context
    double kv_positions;   // context positions read by one attention launch, summed over sequences (accounting only)
};

template <typename T>
T* kv_ptr(tandem_ctx& c, const Model& m, int layer, int which) {
    return at<T>(c, m.kv_off) + ((size_t)layer * 2 + which) * m.kv_layer_elems;
}

EpiArgs epi_plain(void* out, int ldo) {
    EpiArgs e; memset(&e, 0, sizeof(e)); e.out = out; e.ldo = ldo; return e;
}

template <typename T>
EpiArgs epi_cache(tandem_ctx& c, const Model& m, int layer, void* q_out) {
    EpiArgs e; memset(&e, 0, sizeof(e));
    e.out = q_out; e.ldo = m.d.d_model;
    e.kcache = kv_ptr<T>(c, m, layer, 0); e.vcache = kv_ptr<T>(c, m, layer, 1);
    e.row_seq = at<int>(c, c.lay.row_seq); e.row_pos = at<int>(c, c.lay.row_pos);
    e.n_heads = m.kv_heads; e.d_head = m.d.d_model / m.d.n_heads; e.t_max = c.cfg.max_seq;
    e.seg0 = q_out ? m.d.d_model : m.d_kv; e.seg = m.d_kv;   // with queries: [d_model | d_kv | d_kv]; keys / values alone: [d_kv | d_kv]
    return e;
}

// Prompt attention of the large model's layer l on the tensor cores; groups of up to 128 queries.
template <int DH>
void launch_attn_prompt_tc_dh(tandem_ctx& c, const AttnTcArgs& a, const CUtensorMap& tmq, int l, int groups) {
    static std::atomic<unsigned long long> attr_done{0};
    ensure_dyn_smem(attn_prefill_tc_kernel<DH>, AtcCfg<DH>::SMEM_BYTES, attr_done);
    launch_ex(c, false, 1, attn_prefill_tc_kernel<DH>, dim3(a.n_heads, groups), dim3(ATC_THREADS), (size_t)AtcCfg<DH>::SMEM_BYTES, a, tmq,
              c.kmap[l], c.vmap[l]);
}
void launch_attn_prompt_tc(tandem_ctx& c, int l, const bf16* q, bf16* o, const Rows& r) {
    const int d = c.large.d.d_model, H = c.large.d.n_heads, dh = d / H;
    CUtensorMap tmq;
    if (!make_tmap_bf16(&tmq, q, (uint64_t)r.M, (uint64_t)d, (uint64_t)d)) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled failed for the query buffer");
        c.setup_failed = true;
        return;
    }
    AttnTcArgs a;
    memset(&a, 0, sizeof(a));
    a.out = o; a.ldo = d; a.row_seq = at<int>(c, c.lay.row_seq); a.row_pos = at<int>(c, c.lay.row_pos);
    a.grp_row0 = at<int>(c, c.lay.grp_row0); a.grp_cnt = at<int>(c, c.lay.grp_cnt);
    a.n_heads = H; a.n_kv_heads = c.large.kv_heads; a.t_max = c.cfg.max_seq; a.scale = 1.0f / sqrtf((float)dh); a.err_flag = c.st.counters + 2;
    // causal attention: Q K^T and P V over the lower triangle, 2 * d_head * T^2 flops per head and sequence
    ProfScope ps(c, PC_ATTN_PROMPT, 2.0 * dh * H * c.prompt_sq_sum);
    if (dh == 64) launch_attn_prompt_tc_dh<64>(c, a, tmq, l, r.groups);
    else launch_attn_prompt_tc_dh<128>(c, a, tmq, l, r.groups);
}

template <typename T>
void attention(tandem_ctx& c, const Model& m, int l, const T* q, T* o, const Rows& r) {
    const int d = m.d.d_model, H = m.d.n_heads, dh = d / H;
    AttnArgs aa; memset(&aa, 0, sizeof(aa));
    aa.q = q; aa.ldq = d; aa.kcache = kv_ptr<T>(c, m, l, 0); aa.vcache = kv_ptr<T>(c, m, l, 1);
    aa.out = o; aa.ldo = d; aa.row_seq = at<int>(c, c.lay.row_seq); aa.row_pos = at<int>(c, c.lay.row_pos);
    if (!r.decode) { aa.grp_row0 = at<int>(c, c.lay.grp_row0); aa.grp_cnt = at<int>(c, c.lay.grp_cnt); }
    aa.nq = r.nq; aa.n_heads = H; aa.n_kv_heads = m.kv_heads; aa.t_max = c.cfg.max_seq;
    aa.part_ml = at<float>(c, c.lay.part_ml); aa.part_acc = at<float>(c, c.lay.part_acc);
    aa.n_chunks_max = c.lay.n_chunks_max; aa.scale = 1.0f / sqrtf((float)dh);
    aa.merge_counters = at<int>(c, c.lay.attn_counters);
    if (!r.decode && sizeof(T) == 2 && c.tc_prompt_attn && &m == &c.large) {
        launch_attn_prompt_tc(c, l, reinterpret_cast<const bf16*>(q), reinterpret_cast<bf16*>(o), r);
        return;
    }
    launch_attn<T>(c, dh, aa, r.groups, !r.decode, r.n_chunks, r.kv_positions * 2.0 * d * sizeof(T));
}

// bf16 decode / block attention over the cache of layer l: bf16 queries, fp32 output rows.
void attention_decode(tandem_ctx& c, const Model& m, int l, const bf16* q, float* o, const Rows& r, bf16* o_lo = nullptr) {
    const int d = m.d.d_model, H = m.d.n_heads, dh = d / H;
    AttnArgs aa; memset(&aa, 0, sizeof(aa));
    aa.q = q; aa.ldq = d; aa.kcache = kv_ptr<bf16>(c, m, l, 0); aa.vcache = kv_ptr<bf16>(c, m, l, 1);
    aa.out = o; aa.ldo = d; aa.out_f32 = 1; aa.row_seq = at<int>(c, c.lay.row_seq); aa.row_pos = at<int>(c, c.lay.row_pos);
    aa.nq = r.nq; aa.n_heads = H; aa.n_kv_heads = m.kv_heads; aa.t_max = c.cfg.max_seq; aa.scale = 1.0f / sqrtf((float)dh);
    aa.err_flag = tc_scratch(c).err;
    aa.out_lo = o_lo;   // non-null: o is the bf16 value plane, o_lo the remainder plane
    launch_attn_decode(c, dh, aa, r.groups, r.kv_positions * 2.0 * d * 2.0);
}

// Eq. 2, first line, for small layer j, then that layer's LayerNorm and key/value maps: writes the
// small model's large-derived keys/values for the rows' positions.
template <typename T>
void project_layer(tandem_ctx& c, int j, const Rows& r) {
    const int dL = c.large.d.d_model, dS = c.small.d.d_model;
    T* xb = at<T>(c, c.lay.xb);
    float* yhat = at<float>(c, c.lay.yhat);
    T* a_s = at<T>(c, c.lay.a_s);
    if (c.cfg.ff_tandem_kind == TANDEM_FF_LINEAR) {
        launch_gemm<T, EPI_STORE_F32>(c, r.decode, xb, dL, r.M, lin1(wi_tandem(c, j, 0), dS, dL), epi_plain(yhat, dS));
    } else {
        T* t1 = at<T>(c, c.lay.t1);
        launch_gemm<T, EPI_GELU>(c, r.decode, xb, dL, r.M, lin1(wi_tandem(c, j, 0), c.hidden, dL), epi_plain(t1, c.hidden));
        launch_gemm<T, EPI_STORE_F32>(c, r.decode, t1, c.hidden, r.M, lin1(wi_tandem(c, j, 1), dS, c.hidden), epi_plain(yhat, dS));
    }
    launch_layernorm<T>(c, r.M, yhat, w_layer(c, c.small, j, W_LN1G), w_layer(c, c.small, j, W_LN1B), a_s, dS);
    launch_gemm<T, EPI_KV>(c, r.decode, a_s, dS, r.M, lin3(wi_layer(c.small, j, W_WK), wi_layer(c.small, j, W_WV), -1, c.small.d_kv, c.small.d_kv, dS),
                           epi_cache<T>(c, c.small, j, nullptr));
}

template <typename T>
void project_after(tandem_ctx& c, int n_large_layers_done, const Rows& r) {
    bool any = false;
    for (int j = 0; j < c.small.d.n_layers; ++j) any |= (c.layer_map[j] == n_large_layers_done);
    if (!any) return;
    const size_t n = (size_t)r.M * c.large.d.d_model;
    {
        ProfScope ps(c, PC_ROWS, (double)n * (4.0 + sizeof(T)));
        cast_rows_kernel<T><<<(unsigned)((n + 255) / 256), 256, 0, c.stream>>>(at<float>(c, c.lay.h_large), at<T>(c, c.lay.xb), n);
        c.launches++;
    }
    for (int j = 0; j < c.small.d.n_layers; ++j)
        if (c.layer_map[j] == n_large_layers_done) project_layer<T>(c, j, r);
}

// One decoder layer (Eq. 1; the same form serves the small model's layers in Eq. 2) on residual stream h.
template <typename T>
void decoder_layer(tandem_ctx& c, const Model& m, int l, float* h, const Rows& r) {
    const int d = m.d.d_model, dff = m.d.d_ff;
    T* a = at<T>(c, c.lay.a);
    T* q = at<T>(c, c.lay.q);
    T* o = at<T>(c, c.lay.o);
    T* f = at<T>(c, c.lay.f);
    launch_layernorm<T>(c, r.M, h, w_layer(c, m, l, W_LN1G), w_layer(c, m, l, W_LN1B), a, d);
    launch_gemm<T, EPI_QKV>(c, r.decode, a, d, r.M, lin3(wi_layer(m, l, W_WQ), wi_layer(m, l, W_WK), wi_layer(m, l, W_WV), d, m.d_kv, d),
                            epi_cache<T>(c, m, l, q));
    attention<T>(c, m, l, q, o, r);
    launch_gemm<T, EPI_RESID>(c, r.decode, o, d, r.M, lin1(wi_layer(m, l, W_WO), d, d), epi_plain(h, d));
    launch_layernorm<T>(c, r.M, h, w_layer(c, m, l, W_LN2G), w_layer(c, m, l, W_LN2B), a, d);
    launch_gemm<T, EPI_GELU>(c, r.decode, a, d, r.M, lin1(wi_layer(m, l, W_W1), dff, d), epi_plain(f, dff));
    launch_gemm<T, EPI_RESID>(c, r.decode, f, dff, r.M, lin1(wi_layer(m, l, W_W2), d, dff), epi_plain(h, d));
}

// Final LayerNorm, output head, arg-max.  dst[(m / nq) * seq_stride + m % nq + off].
template <typename T>
void head_argmax(tandem_ctx& c, const Model& m, float* h, const Rows& r, float* logits, int* dst, int seq_stride, int off) {
    const int d = m.d.d_model, V = m.d.vocab;
    T* a = at<T>(c, c.lay.a);
    launch_layernorm<T>(c, r.M, h, w_tail(c, m, 0), w_tail(c, m, 1), a, d);
    launch_gemm<T, EPI_STORE_F32>(c, r.decode, a, d, r.M, lin1(wi_tail(m, 2), V, d), epi_plain(logits, V));
    ProfScope ps(c, PC_ARGMAX, (double)r.M * V * 4.0);
    argmax_rows_kernel<<<r.M, 256, 0, c.stream>>>(logits, V, dst, r.nq, seq_stride, off);
    c.launches++;
}

// The large model over the current rows (block mode in decode, whole prompt otherwise).
template <typename T>
void large_pass(tandem_ctx& c, const Rows& r, bool project, bool head) {
    float* h = at<float>(c, c.lay.h_large);
    {
        ProfScope ps(c, PC_ROWS, (double)r.M * c.large.d.d_model * (4.0 + 2 * sizeof(T)));
        embed_kernel<T><<<r.M, 128, 0, c.stream>>>(at<int>(c, c.lay.row_tok), at<int>(c, c.lay.row_pos), (const T*)w_emb(c, c.large),
                                                   (const T*)w_pos(c, c.large), h, c.large.d.d_model);
        c.launches++;
    }
    if (project) project_after<T>(c, 0, r);
    for (int l = 0; l < c.large.d.n_layers; ++l) {
        decoder_layer<T>(c, c.large, l, h, r);
        if (project) project_after<T>(c, l + 1, r);
    }
    if (head)
        head_argmax<T>(c, c.large, h, r, at<float>(c, c.lay.logits_large), c.st.targets, TANDEM_GAMMA_LIMIT + 1, 0);
}

Rows decode_rows(tandem_ctx& c, int r_last, int nq) {
    Rows r;
    r.M = c.batch * nq; r.groups = c.batch; r.nq = nq; r.decode = true;
    r.n_chunks = c.chunks_launch;
    r.kv_positions = (double)c.n_sum + (double)c.batch * r_last;
    return r;
}

void setup_rows(tandem_ctx& c, int r0, int nq) {
    const int M = c.batch * nq;
    ProfScope ps(c, PC_ROWS, (double)M * 12.0);
    setup_rows_kernel<<<cdiv(M, 128), 128, 0, c.stream>>>(c.st, c.batch, r0, nq, at<int>(c, c.lay.row_tok), at<int>(c, c.lay.row_seq), at<int>(c, c.lay.row_pos));
    c.launches++;
}

// Draft step s: one token per sequence through the small model over the mixed context (Eq. 2, lines 2-3).
// dst: where the step's arg-max goes (default: draft s of the loop state; a teacher-forced round keeps its given
// drafts and sends the arg-max to the unused target array).
template <typename T>
void small_step(tandem_ctx& c, int s, bool keep_drafts = false) {
    setup_rows(c, s, 1);
    Rows r = decode_rows(c, s, 1);
    float* y = at<float>(c, c.lay.h_small);
    {
        ProfScope ps(c, PC_ROWS, (double)r.M * c.small.d.d_model * (4.0 + 2 * sizeof(T)));
        embed_kernel<T><<<r.M, 128, 0, c.stream>>>(at<int>(c, c.lay.row_tok), at<int>(c, c.lay.row_pos), (const T*)w_emb(c, c.small),
                                                   (const T*)w_pos(c, c.small), y, c.small.d.d_model);
        c.launches++;
    }
    for (int j = 0; j < c.small.d.n_layers; ++j) decoder_layer<T>(c, c.small, j, y, r);
    float* logits = at<float>(c, c.lay.logits_small) + (size_t)s * c.batch * c.small.d.vocab;
    if (keep_drafts) head_argmax<T>(c, c.small, y, r, logits, c.st.targets, TANDEM_GAMMA_LIMIT + 1, s);
    else head_argmax<T>(c, c.small, y, r, logits, c.st.drafts, TANDEM_GAMMA_LIMIT, s);
}

// Teacher-forced round (accept mode 5): the given tokens become the round's drafts; after the draft steps their
// logits are scored against the given next tokens.
void launch_forced_fill(tandem_ctx& c, int gamma) {
    ProfScope ps(c, PC_ROWS, (double)c.batch * gamma * 8.0);
    launch_ex(c, true, 1, forced_fill_kernel, dim3(1), dim3(256), 0, c.st, c.batch, gamma, (const int*)at<int>(c, c.lay.forced_ids),
              (const int*)at<int>(c, c.lay.forced_len), (int)c.cfg.max_seq);
}
void launch_score_rows(tandem_ctx& c, int gamma) {
    ProfScope ps(c, PC_ARGMAX, (double)c.batch * gamma * c.small.d.vocab * 8.0);
    launch_ex(c, true, 1, score_rows_kernel, dim3(gamma, c.batch), dim3(256), 0, c.st, c.batch, (const float*)at<float>(c, c.lay.logits_small),
              (int)c.small.d.vocab, (const int*)at<int>(c, c.lay.forced_ids), (const int*)at<int>(c, c.lay.forced_len), (int)c.cfg.max_seq,
              at<float>(c, c.lay.forced_nll), at<int>(c, c.lay.forced_top));
}

void launch_verify(tandem_ctx& c, int gamma, int mode, uint64_t seed, int max_new, bool from_tiles, bool adaptive = false) {
    ProfScope ps(c, PC_VERIFY, (double)c.batch * (2 * gamma + 8) * 4.0);
    launch_ex(c, true, 1, verify_kernel, dim3(1), dim3(256), 0, c.st, c.batch, gamma, mode, (unsigned long long)seed, max_new,
              from_tiles ? (const float*)at<float>(c, c.lay.amax_val_large) : (const float*)nullptr,
              from_tiles ? (const int*)at<int>(c, c.lay.amax_idx_large) : (const int*)nullptr, c.lay.vocab_tiles, c.lay.vocab_tiles,
              from_tiles ? (const float*)at<float>(c, c.lay.amax_val_small) : (const float*)nullptr,
              from_tiles ? (const int*)at<int>(c, c.lay.amax_idx_small) : (const int*)nullptr,
              adaptive ? (const int*)c.st.block_len : (const int*)nullptr);
}

// Adaptive block length: the router's decision after draft step s, for every sequence that is still drafting.
void launch_router(tandem_ctx& c, int s, int gamma_max) {
    const float* logits = at<float>(c, c.lay.logits_small) + (size_t)s * c.batch * c.small.d.vocab;
    ProfScope ps(c, PC_ARGMAX, (double)c.batch * c.small.d.vocab * 8.0);
    const size_t feat_bytes = sizeof(float) * (size_t)(1 + c.router.k + c.router.k * c.small.d.d_model);   // <= 48 KB, checked by tandem_set_router
    if (c.cfg.dtype == TANDEM_DTYPE_BF16)
        launch_ex(c, true, 1, router_kernel<bf16>, dim3(c.batch), dim3(RT_THREADS), feat_bytes, c.st, c.batch, logits, (int)c.small.d.vocab, s, gamma_max,
                  (const bf16*)w_emb(c, c.small), (int)c.small.d.d_model, c.router);
    else
        launch_ex(c, true, 1, router_kernel<float>, dim3(c.batch), dim3(RT_THREADS), feat_bytes, c.st, c.batch, logits, (int)c.small.d.vocab, s, gamma_max,
                  (const float*)w_emb(c, c.small), (int)c.small.d.d_model, c.router);
}
void launch_adaptive_begin(tandem_ctx& c) {
    ProfScope ps(c, PC_ROWS, (double)c.batch * 8.0);
    launch_ex(c, true, 1, adaptive_begin_kernel, dim3(1), dim3(256), 0, c.st, c.batch);
}

// Sampled SPEED: draft s of every sequence drawn from the small model's logits of step s.
void launch_sample_draft(tandem_ctx& c, int s, uint64_t seed) {
    const float* logits = at<float>(c, c.lay.logits_small) + (size_t)s * c.batch * c.small.d.vocab;
    ProfScope ps(c, PC_ARGMAX, (double)c.batch * c.small.d.vocab * 8.0);
    launch_ex(c, true, 1, sample_draft_kernel, dim3(c.batch), dim3(SMP_THREADS), 0, c.st, logits, (int)c.small.d.vocab, s, c.temp_small,
              (unsigned long long)seed);
}
// Sampled SPEED: accept / redraw decisions of the iteration, ahead of the verify kernel's bookkeeping.
void launch_sample_verify(tandem_ctx& c, int gamma, uint64_t seed) {
    ProfScope ps(c, PC_ARGMAX, (double)c.batch * (2 * gamma + 1) * c.large.d.vocab * 8.0);
    launch_ex(c, true, 1, sample_verify_kernel, dim3(c.batch), dim3(SMP_THREADS), 0, c.st, c.batch, gamma,
              (const float*)at<float>(c, c.lay.logits_large), (const float*)at<float>(c, c.lay.logits_small), (int)c.large.d.vocab,
              c.temp_large, c.temp_small, (unsigned long long)seed);
}

template <typename T>
void iteration(tandem_ctx& c, int gamma, int mode, uint64_t seed, int max_new) {
    if (mode == 5) launch_forced_fill(c, gamma);
    for (int s = 0; s < gamma; ++s) {
        small_step<T>(c, s, mode == 5);
        if (mode == 4) launch_sample_draft(c, s, seed);   // replaces the arg-max draft of this step
    }
    if (mode == 5) launch_score_rows(c, gamma);
    if (mode == 3 || mode == 5) {   // stand-alone Tandem without the free token: gamma rows, no output head
        setup_rows(c, 0, gamma);
        large_pass<T>(c, decode_rows(c, gamma - 1, gamma), true, false);
    } else {
        setup_rows(c, 0, gamma + 1);
        large_pass<T>(c, decode_rows(c, gamma, gamma + 1), true, true);
    }
    if (mode == 4) launch_sample_verify(c, gamma, seed);
    launch_verify(c, gamma, mode == 5 ? 3 : mode, seed, max_new, false);
    c.last_gamma = gamma;
}

template <typename T>
void greedy_iteration(tandem_ctx& c, int max_new) {
    setup_rows(c, 0, 1);
    large_pass<T>(c, decode_rows(c, 0, 1), false, true);
    launch_verify(c, 0, 0, 0ull, max_new, false);
    c.last_gamma = 0;
}

// ---------------------------------------------------------------------------------------------------
// bf16 decode on the tensor cores: five kernels per decoder layer, chained by programmatic dependent launch
// ---------------------------------------------------------------------------------------------------

// Row set-up + embedding for block rows r0 .. r0+nq-1 of every sequence; fin_r: block row whose token is the
// arg-max the small model's last head GEMM left as per-tile results (-1: none).
void tc_begin(tandem_ctx& c, const Model& m, float* h, int r0, int nq, int fin_r, float* snap = nullptr) {
    ProfScope ps(c, PC_ROWS, (double)c.batch * nq * m.d.d_model * 8.0);
    launch_ex(c, true, 1, step_begin_kernel<bf16>, dim3(c.batch * nq), dim3(128), 0, c.st, r0, nq, fin_r,
              (const float*)at<float>(c, c.lay.amax_val_small), (const int*)at<int>(c, c.lay.amax_idx_small), c.lay.vocab_tiles,
              c.lay.vocab_tiles, at<int>(c, c.lay.row_tok), at<int>(c, c.lay.row_seq), at<int>(c, c.lay.row_pos),
              (const bf16*)w_emb(c, m), (const bf16*)w_pos(c, m), h, m.d.d_model, snap);
}

// The decode activations' value / remainder planes (see tandem_ctx::xmap): buffer 0 = LayerNorm output, 1 = attention
// output, 2 = GELU output; K = the row length in use (the model's width, or its FFN width for buffer 2).
struct XPlanes { bf16* hi; bf16* lo; const CUtensorMap* map; };
XPlanes x_planes(tandem_ctx& c, int buf, const Model& m) {
    const size_t off = buf == 0 ? c.lay.a32 : (buf == 1 ? c.lay.o32 : c.lay.f32);
    const size_t K = buf == 2 ? m.d.d_ff : m.d.d_model;
    XPlanes p;
    p.hi = reinterpret_cast<bf16*>(c.arena + off);
    p.lo = p.hi + (size_t)c.lay.dec_rows * K;
    p.map = &c.xmap[buf][&m == &c.large ? 0 : 1];
    return p;
}

// Whether LayerNorm is fused into the GEMM's operand load.  Fused, every CTA of the GEMM normalises the rows it
// needs itself: right for a couple of sequences and short rows, wasteful beyond (eight sequences of 768 elements
// already measured 2 % slower per iteration than the LayerNorm kernel).  The choice depends on the batch
// and the model only, never on the number of rows, so a block pass and a one-row pass take the same route.
bool tc_fused_prologue(const tandem_ctx& c, int K) { return c.batch <= 2 && K <= 1024; }

// y = LayerNorm(h) W^T with the given epilogue; h fp32 [rows][K].  ln_out: where the normalised rows go when the
// LayerNorm runs as its own kernel (default: the pass's activation buffer).
template <int EPI>
void tc_ln_gemm(tandem_ctx& c, const float* h, const void* ln_g, const void* ln_b, int rows, const TcW& w, bool stream_w,
                const EpiArgs& e, float* amax_val = nullptr, int* amax_idx = nullptr, int amax_stride = 0, float* ln_out = nullptr) {
    const TcScratch sc = tc_scratch(c);
    if (tc_fused_prologue(c, w.K)) {
        launch_tc_decode<PRO_LN, EPI>(c, sc, h, w.K, ln_g, ln_b, rows, w, stream_w, e, amax_val, amax_idx, amax_stride);
        return;
    }
    const Model* hm = h == reinterpret_cast<const float*>(c.arena + c.lay.h_large) ? &c.large :
                      (h == reinterpret_cast<const float*>(c.arena + c.lay.h_small) ? &c.small : nullptr);
    if (!ln_out && c.xmap_ok && hm && hm->d.d_model == w.K) {
        // the LayerNorm kernel leaves value and remainder planes, the GEMM loads them by TMA beside its weights
        const XPlanes xp = x_planes(c, 0, *hm);
        {
            ProfScope ps(c, PC_LAYERNORM, (double)rows * w.K * 8.0);
            launch_ex(c, true, 1, layernorm_rows_kernel<bf16>, dim3(rows), dim3(128), 0, h, static_cast<const float*>(ln_g),
                      static_cast<const float*>(ln_b), xp.hi, w.K, xp.lo);
        }
        launch_tc_decode<PRO_TMA, EPI>(c, sc, xp.hi, w.K, nullptr, nullptr, rows, w, stream_w, e, amax_val, amax_idx, amax_stride, xp.map,
                                       c.lay.dec_rows);
        return;
    }
    float* a = ln_out ? ln_out : at<float>(c, c.lay.a32);
    {
        ProfScope ps(c, PC_LAYERNORM, (double)rows * w.K * 8.0);
        launch_ex(c, true, 1, layernorm_rows_kernel<float>, dim3(rows), dim3(128), 0, h, static_cast<const float*>(ln_g),
                  static_cast<const float*>(ln_b), a, w.K, (bf16*)nullptr);
    }
    launch_tc_decode<PRO_F32, EPI>(c, sc, a, w.K, nullptr, nullptr, rows, w, stream_w, e, amax_val, amax_idx, amax_stride);
}

// One decoder layer of a decode pass.  Between the kernels the activations are fp32 (attention and GELU outputs,
// normalised rows); only the queries and the cached keys / values are bf16.
void tc_decoder_layer(tandem_ctx& c, const Model& m, int l, float* h, const Rows& r, bool stream_w, float* snap = nullptr) {
    const int d = m.d.d_model, dff = m.d.d_ff;
    bf16* q = at<bf16>(c, c.lay.q);
    float* o = at<float>(c, c.lay.o32);
    float* f = at<float>(c, c.lay.f32);
    const TcScratch sc = tc_scratch(c);
    tc_ln_gemm<EPI_QKV>(c, h, w_layer(c, m, l, W_LN1G), w_layer(c, m, l, W_LN1B), r.M,
                        tcw3(c, wi_layer(m, l, W_WQ), wi_layer(m, l, W_WK), wi_layer(m, l, W_WV), d, m.d_kv, d), stream_w, epi_cache<bf16>(c, m, l, q));
    EpiArgs e2 = epi_plain(h, d);
    e2.snap = snap; e2.snap_ld = d;   // copy of x^(l+1) when an FF_Tandem projection reads it
    if (c.xmap_ok) {
        // attention and GELU outputs as value / remainder planes that the next GEMM loads by TMA
        const XPlanes xo = x_planes(c, 1, m), xf = x_planes(c, 2, m);
        attention_decode(c, m, l, q, reinterpret_cast<float*>(xo.hi), r, xo.lo);
        launch_tc_decode<PRO_TMA, EPI_RESID>(c, sc, xo.hi, d, nullptr, nullptr, r.M, tcw(c, wi_layer(m, l, W_WO), -1, -1, d, d), stream_w,
                                             epi_plain(h, d), nullptr, nullptr, 0, xo.map, c.lay.dec_rows);
        EpiArgs e1 = epi_plain(xf.hi, dff);
        e1.out_lo = xf.lo;
        tc_ln_gemm<EPI_GELU>(c, h, w_layer(c, m, l, W_LN2G), w_layer(c, m, l, W_LN2B), r.M, tcw(c, wi_layer(m, l, W_W1), -1, -1, dff, d),
                             stream_w, e1);
        launch_tc_decode<PRO_TMA, EPI_RESID>(c, sc, xf.hi, dff, nullptr, nullptr, r.M, tcw(c, wi_layer(m, l, W_W2), -1, -1, d, dff), stream_w, e2,
                                             nullptr, nullptr, 0, xf.map, c.lay.dec_rows);
        return;
    }
    attention_decode(c, m, l, q, o, r);
    launch_tc_decode<PRO_F32, EPI_RESID>(c, sc, o, d, nullptr, nullptr, r.M, tcw(c, wi_layer(m, l, W_WO), -1, -1, d, d), stream_w,
                                         epi_plain(h, d));
    tc_ln_gemm<EPI_GELU>(c, h, w_layer(c, m, l, W_LN2G), w_layer(c, m, l, W_LN2B), r.M, tcw(c, wi_layer(m, l, W_W1), -1, -1, dff, d),
                         stream_w, epi_plain(f, dff));
    launch_tc_decode<PRO_F32, EPI_RESID>(c, sc, f, dff, nullptr, nullptr, r.M, tcw(c, wi_layer(m, l, W_W2), -1, -1, d, dff), stream_w, e2);
}

// Final LayerNorm + output head; leaves fp32 logits and the per-tile (max, index) pairs that the next kernel
// (the next pass's row set-up, or the verify kernel) turns into token ids.
void tc_head(tandem_ctx& c, const Model& m, float* h, const Rows& r, float* logits, size_t amax_val_off, size_t amax_idx_off, bool stream_w) {
    tc_ln_gemm<EPI_ARGMAX>(c, h, w_tail(c, m, 0), w_tail(c, m, 1), r.M, tcw(c, wi_tail(m, 2), -1, -1, m.d.vocab, m.d.d_model), stream_w,
                           epi_plain(logits, m.d.vocab), at<float>(c, amax_val_off), at<int>(c, amax_idx_off), c.lay.vocab_tiles);
}

// sampled: the previous draft was drawn by sample_draft_kernel (it is in the loop state already), not left as per-tile
// arg-max results.
void tc_small_step(tandem_ctx& c, int s, bool sampled) {
    float* y = at<float>(c, c.lay.h_small);
    tc_begin(c, c.small, y, s, 1, (s > 0 && !sampled) ? s : -1);
    const Rows r = decode_rows(c, s, 1);
    for (int j = 0; j < c.small.d.n_layers; ++j) tc_decoder_layer(c, c.small, j, y, r, false);
    float* logits = at<float>(c, c.lay.logits_small) + (size_t)s * c.batch * c.small.d.vocab;
    tc_head(c, c.small, y, r, logits, c.lay.amax_val_small, c.lay.amax_idx_small, false);
}

// FF_Tandem of the block's rows after n large layers (Eq. 2, first line) for every small layer fed from there, then
// that layer's LayerNorm and key/value maps with the cache write as the GEMM epilogue.  It runs on the side stream,
// from the copy `snap` of x^(l(j)) that the producing kernel left: it depends on nothing the large model does
// afterwards (and nothing in the iteration depends on it before the next draft), so it runs beside the large model's
// later layers instead of in their chain.
void tc_project_forked(tandem_ctx& c, int n_large_layers_done, int slot, const Rows& r) {
    const int dL = c.large.d.d_model, dS = c.small.d.d_model;
    const TcScratch sc = tc_scratch(c);
    const size_t RD = (size_t)c.lay.dec_rows;
    const float* snap = at<float>(c, c.lay.proj_snap) + (size_t)slot * RD * dL;
    cudaStream_t main_stream = c.stream;
    cudaEventRecord(c.ev_fork[slot], main_stream);
    cudaStreamWaitEvent(c.side, c.ev_fork[slot], 0);
    c.stream = c.side;
    c.next_launch_plain = true;   // first kernel after a cross-stream wait
    for (int j = 0; j < c.small.d.n_layers; ++j) {
        if (c.layer_map[j] != n_large_layers_done) continue;
        float* yhat = at<float>(c, c.lay.proj_yhat) + (size_t)j * RD * dS;
        float* a_j = at<float>(c, c.lay.proj_a) + (size_t)j * RD * dS;
        if (c.cfg.ff_tandem_kind == TANDEM_FF_LINEAR) {
            launch_tc_decode<PRO_F32, EPI_STORE_F32>(c, sc, snap, dL, nullptr, nullptr, r.M, tcw(c, wi_tandem(c, j, 0), -1, -1, dS, dL), true,
                                                     epi_plain(yhat, dS));
        } else {
            float* t1 = at<float>(c, c.lay.proj_t1) + (size_t)j * RD * c.hidden;
            launch_tc_decode<PRO_F32, EPI_GELU>(c, sc, snap, dL, nullptr, nullptr, r.M, tcw(c, wi_tandem(c, j, 0), -1, -1, c.hidden, dL), true,
                                                epi_plain(t1, c.hidden));
            launch_tc_decode<PRO_F32, EPI_STORE_F32>(c, sc, t1, c.hidden, nullptr, nullptr, r.M, tcw(c, wi_tandem(c, j, 1), -1, -1, dS, c.hidden),
                                                     true, epi_plain(yhat, dS));
        }
        tc_ln_gemm<EPI_KV>(c, yhat, w_layer(c, c.small, j, W_LN1G), w_layer(c, c.small, j, W_LN1B), r.M,
                           tcw(c, wi_layer(c.small, j, W_WK), wi_layer(c.small, j, W_WV), -1, c.small.d_kv, dS), true, epi_cache<bf16>(c, c.small, j, nullptr),
                           nullptr, nullptr, 0, a_j);
    }
    c.stream = main_stream;
}

// Slot of the projection buffers for the residual stream after `n` large layers: the first small layer fed from there, or -1.
int project_slot(const tandem_ctx& c, int n) {
    for (int j = 0; j < c.small.d.n_layers; ++j)
        if (c.layer_map[j] == n) return j;
    return -1;
}

// The large model over nq block rows per sequence (row 0 = pending token, row r = draft r); fin_r: block row whose
// token the small model's last head GEMM left as per-tile results (-1: none); head: final LayerNorm + output head.
void tc_large_block(tandem_ctx& c, int nq, int fin_r, bool project, bool head) {
    float* h = at<float>(c, c.lay.h_large);
    const size_t snap_elems = (size_t)c.lay.dec_rows * c.large.d.d_model;
    auto snap_of = [&](int n) -> float* {
        const int slot = project ? project_slot(c, n) : -1;
        return slot >= 0 ? at<float>(c, c.lay.proj_snap) + (size_t)slot * snap_elems : nullptr;
    };
    bool any_fork = false;
    tc_begin(c, c.large, h, 0, nq, fin_r, snap_of(0));
    const Rows r = decode_rows(c, nq - 1, nq);
    if (project && project_slot(c, 0) >= 0) { tc_project_forked(c, 0, project_slot(c, 0), r); any_fork = true; }
    for (int l = 0; l < c.large.d.n_layers; ++l) {
        tc_decoder_layer(c, c.large, l, h, r, true, snap_of(l + 1));
        if (project && project_slot(c, l + 1) >= 0) { tc_project_forked(c, l + 1, project_slot(c, l + 1), r); any_fork = true; }
    }
    if (head) tc_head(c, c.large, h, r, at<float>(c, c.lay.logits_large), c.lay.amax_val_large, c.lay.amax_idx_large, true);
    if (any_fork) {   // the projections join the main stream before the verify kernel
        cudaEventRecord(c.ev_join, c.side);
        cudaStreamWaitEvent(c.stream, c.ev_join, 0);
        c.next_launch_plain = true;
    }
}

void tc_iteration(tandem_ctx& c, int gamma, int mode, uint64_t seed, int max_new) {
    const bool sampled = mode == 4, forced = mode == 5;
    if (forced) launch_forced_fill(c, gamma);
    for (int s = 0; s < gamma; ++s) {
        tc_small_step(c, s, sampled || forced);   // (both find their drafts in the loop state, not in per-tile arg-max results)
        if (sampled) launch_sample_draft(c, s, seed);
    }
    if (forced) {   // teacher-forced round: score the logits, then a representation-only block whose drafts are the given tokens
        launch_score_rows(c, gamma);
        tc_large_block(c, gamma, -1, true, false);
        launch_verify(c, gamma, 3, seed, max_new, false);
        c.last_gamma = gamma;
        return;
    }
    if (mode == 3) tc_large_block(c, gamma, -1, true, false);   // gamma rows, no head: the last draft is finished by the verify kernel
    else tc_large_block(c, gamma + 1, (gamma > 0 && !sampled) ? gamma : -1, true, true);
    if (sampled) launch_sample_verify(c, gamma, seed);
    launch_verify(c, gamma, mode, seed, max_new, true);
    c.last_gamma = gamma;
}

void tc_greedy_iteration(tandem_ctx& c, int max_new) {
    tc_large_block(c, 1, -1, false, true);
    launch_verify(c, 0, 0, 0ull, max_new, true);
    c.last_gamma = 0;
}

tandem_status check_launch() {
    CK(cudaGetLastError());
    return TANDEM_OK;
}
// The same for a context: also reports a launch helper that had to skip its launch.
tandem_status check_launch(tandem_ctx& c) {
    if (c.setup_failed) { c.setup_failed = false; return TANDEM_ERR_CUDA; }
    return check_launch();
}

// kind 0: draft + verify (gamma drafts, accept mode);  1: plain greedy M_L;
// kind 3: one draft step of the adaptive block length (gamma = step index, mode = gamma_max) followed by the router;
// kind 4: the verify half of an adaptive iteration (gamma = longest block of the batch).
void enqueue_iteration(tandem_ctx& c, int kind, int gamma, int mode, uint64_t seed, int max_new) {
    const bool bf = c.cfg.dtype == TANDEM_DTYPE_BF16;   // one bf16 path: the tensor-core kernels (a bf16 context always has tensor maps)
    if (kind == 3) {
        if (gamma == 0) launch_adaptive_begin(c);
        if (bf) tc_small_step(c, gamma, false); else small_step<float>(c, gamma);
        launch_router(c, gamma, mode);
        return;
    }
    if (kind == 4) {
        if (bf) {
            tc_large_block(c, gamma + 1, gamma, true, true);
        } else {
            setup_rows(c, 0, gamma + 1);
            large_pass<float>(c, decode_rows(c, gamma, gamma + 1), true, true);
        }
        launch_verify(c, gamma, TANDEM_ACCEPT_NATURAL, 0ull, max_new, bf, true);
        c.last_gamma = gamma;
        return;
    }
    if (bf) {
        if (kind == 0) tc_iteration(c, gamma, mode, seed, max_new); else tc_greedy_iteration(c, max_new);
        return;
    }
    if (kind == 0) iteration<float>(c, gamma, mode, seed, max_new);
    else greedy_iteration<float>(c, max_new);
}

// Enqueues one iteration on the context's stream: eagerly the first time a launch shape is seen (and whenever
// per-launch profiling is on), as a CUDA graph afterwards.  kind 0 = draft + verify, 1 = plain greedy M_L.
tandem_status launch_iteration(tandem_ctx& c, int kind, int gamma, int mode, uint64_t seed, int max_new) {
    const int need = (c.n_ub - 1 + gamma) / ATT_CH + 1;
    c.chunks_launch = std::min(c.lay.n_chunks_max, (need + 3) / 4 * 4);
    if (c.cfg.dtype == TANDEM_DTYPE_BF16)
        c.chunks_launch = 1;   // the cluster attention's grid does not depend on the context length: one graph serves all
    if (kind == 3) c.router_ticket++; else c.ticket++;   // what the host will wait for: the router's or the verify kernel's publication
    if (kind != 3) c.last_gamma = kind == 1 ? 0 : gamma;   // (set here, not while enqueueing: a replayed graph enqueues nothing on the host)
    if (c.prof.on || !c.use_graphs) {
        enqueue_iteration(c, kind, gamma, mode, seed, max_new);
        return check_launch();
    }
    tandem_ctx::GraphEntry* g = nullptr;
    for (auto& e : c.graphs)
        if (e.kind == kind && e.gamma == gamma && e.mode == mode && e.max_new == max_new && e.batch == c.batch &&
            e.chunks == c.chunks_launch && e.seed == seed) { g = &e; break; }
    if (!g) {
        c.graphs.push_back({kind, gamma, mode, max_new, c.batch, c.chunks_launch, seed, false, nullptr, 0});
        g = &c.graphs.back();
    }
    if (!g->warm) {   // first use: run eagerly (sets kernel attributes, surfaces launch errors outside a capture)
        g->warm = true;
        enqueue_iteration(c, kind, gamma, mode, seed, max_new);
        return check_launch();
    }
    if (!g->exec) {
        cudaStream_t user = c.stream;
        const int64_t l0 = c.launches;
        CK(cudaStreamBeginCapture(c.cap_stream, cudaStreamCaptureModeThreadLocal));
        c.stream = c.cap_stream;
        enqueue_iteration(c, kind, gamma, mode, seed, max_new);
        c.stream = user;
        cudaGraph_t graph = nullptr;
        cudaError_t e = cudaStreamEndCapture(c.cap_stream, &graph);
        g->kernels = c.launches - l0;
        c.launches = l0;
        if (e == cudaSuccess) e = cudaGraphInstantiate(&g->exec, graph, 0);
        if (graph) cudaGraphDestroy(graph);
        if (e != cudaSuccess) {
            g->exec = nullptr;
            snprintf(g_cuda_err, sizeof(g_cuda_err), "%s while capturing an iteration", cudaGetErrorString(e));
            return TANDEM_ERR_CUDA;
        }
    }
    CK(cudaGraphLaunch(g->exec, c.stream));
    c.launches += g->kernels;
    return TANDEM_OK;
}

// Waits (bounded) until the kernel that publishes into slot `slot` of the host flags (0: verify kernel, 5: router)
// has reached the given ticket.
tandem_status wait_ticket(tandem_ctx& c, int64_t ticket, int slot = 0) {
    volatile int32_t* hf = c.hflags + slot;
    struct timespec t0, t1;
    clock_gettime(CLOCK_MONOTONIC, &t0);
    for (unsigned spin = 0; (int64_t)hf[0] < ticket; ++spin) {
        if ((spin & 1023) == 1023) {
            if (cudaStreamQuery(c.stream) != cudaErrorNotReady && (int64_t)hf[0] < ticket) {
                // the stream drained (or failed) without publishing: report instead of spinning forever
                cudaError_t e = cudaStreamSynchronize(c.stream);
                if ((int64_t)hf[0] >= ticket) break;
                snprintf(g_cuda_err, sizeof(g_cuda_err), "%s while waiting for an iteration", cudaGetErrorString(e));
                return e == cudaSuccess ? TANDEM_ERR_TIMEOUT : TANDEM_ERR_CUDA;
            }
            clock_gettime(CLOCK_MONOTONIC, &t1);
            if (t1.tv_sec - t0.tv_sec > 60) return TANDEM_ERR_TIMEOUT;
        }
    }
    __sync_synchronize();
    return TANDEM_OK;
}

tandem_status begin_call(tandem_ctx* c) {
    if (!c) return TANDEM_ERR_INVALID_ARG;
    CK(cudaSetDevice(c->cfg.device));
    return TANDEM_OK;
}

__global__ void reset_call_kernel(LoopState st, int batch) {
    const int b = threadIdx.x;
    if (b < batch) { st.emitted[b] = 0; st.done[b] = 0; }
    if (b == 0) { st.counters[1] = batch; st.counters[5] = 0; }
}

}  // namespace
// =====================================================================================================
// exported entry points
// =====================================================================================================

extern "C" const char* tandem_status_string(tandem_status s) {
    switch (s) {
        case TANDEM_OK: return "ok";
        case TANDEM_ERR_INVALID_ARG: return "invalid argument";
        case TANDEM_ERR_SHAPE: return "unsupported shape";
        case TANDEM_ERR_ARENA_TOO_SMALL: return "arena too small";
        case TANDEM_ERR_CAPACITY: return "capacity exceeded";
        case TANDEM_ERR_STATE: return "call out of order";
        case TANDEM_ERR_CUDA: return "CUDA error";
        case TANDEM_ERR_TIMEOUT: return "device wait timed out";
        case TANDEM_ERR_UNIMPLEMENTED: return "not implemented";
    }
    return "unknown status";
}

extern "C" const char* tandem_last_cuda_error(void) { return g_cuda_err; }

extern "C" tandem_status tandem_query_arena(const tandem_config* cfg, size_t* bytes) {
    if (!bytes) return TANDEM_ERR_INVALID_ARG;
    TRY(validate(cfg));
    *bytes = make_layout(*cfg).total;
    return TANDEM_OK;
}

namespace {
void release_side(tandem_ctx& c) {
    for (cudaEvent_t ev : c.ev_fork) cudaEventDestroy(ev);
    c.ev_fork.clear();
    if (c.ev_join) { cudaEventDestroy(c.ev_join); c.ev_join = nullptr; }
    if (c.side) { cudaStreamDestroy(c.side); c.side = nullptr; }
}
}  // namespace

extern "C" tandem_status tandem_create(const tandem_config* cfg, const tandem_weights* weights, void* arena,
                                       size_t arena_bytes, tandem_ctx** out) {
    if (!out || !weights || !weights->ptrs || !arena) return TANDEM_ERR_INVALID_ARG;
    TRY(validate(cfg));
    if (weights->n_ptrs != n_weight_ptrs(*cfg)) return TANDEM_ERR_INVALID_ARG;
    for (int i = 0; i < weights->n_ptrs; ++i)
        if (!weights->ptrs[i] || ((uintptr_t)weights->ptrs[i] & 15)) return TANDEM_ERR_INVALID_ARG;
    if ((uintptr_t)arena & 255) return TANDEM_ERR_INVALID_ARG;
    Layout lay = make_layout(*cfg);
    if (arena_bytes < lay.total) return TANDEM_ERR_ARENA_TOO_SMALL;
    CK(cudaSetDevice(cfg->device));

    tandem_ctx* c = new (std::nothrow) tandem_ctx();
    if (!c) return TANDEM_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->layer_map.assign(cfg->layer_map, cfg->layer_map + cfg->small.n_layers);
    c->cfg.layer_map = c->layer_map.data();
    c->w.assign(weights->ptrs, weights->ptrs + weights->n_ptrs);
    c->lay = lay;
    c->arena = static_cast<unsigned char*>(arena);
    c->stream = static_cast<cudaStream_t>(cfg->stream);
    c->esz = cfg->dtype == TANDEM_DTYPE_BF16 ? 2 : 4;
    c->hidden = cfg->ff_tandem_hidden > 0 ? cfg->ff_tandem_hidden : cfg->small.d_model;
    c->large.kv_heads = kv_heads_of(cfg->large); c->large.d_kv = d_kv_of(cfg->large);
    c->small.kv_heads = kv_heads_of(cfg->small); c->small.d_kv = d_kv_of(cfg->small);
    c->large.d = cfg->large; c->large.wbase = 0; c->large.kv_off = lay.kv_large; c->large.kv_layer_elems = lay.kv_large_layer;
    c->small.d = cfg->small; c->small.wbase = 5 + 10 * cfg->large.n_layers; c->small.kv_off = lay.kv_small; c->small.kv_layer_elems = lay.kv_small_layer;
    c->tbase = c->small.wbase + 5 + 10 * cfg->small.n_layers;
    c->batch = 0; c->n_ub = 0; c->launches = 0; c->last_gamma = 0;
    c->pinned_ints = (size_t)3 * lay.max_rows + 2 * lay.max_groups + 4 * cfg->max_batch + 64;
    c->pinned = nullptr;
    LoopState& st = c->st;
    st.n = at<int>(*c, lay.st_n); st.pending = at<int>(*c, lay.st_pending); st.drafts = at<int>(*c, lay.st_drafts);
    st.targets = at<int>(*c, lay.st_targets); st.accept_len = at<int>(*c, lay.st_accept); st.emitted = at<int>(*c, lay.st_emitted);
    st.done = at<int>(*c, lay.st_done); st.out_ids = at<int>(*c, lay.st_out); st.counters = at<int>(*c, lay.st_counters);
    st.hist = at<unsigned long long>(*c, lay.st_hist);
    st.block_len = at<int>(*c, lay.st_block_len); st.drafting = at<int>(*c, lay.st_drafting);
    st.confidence = at<float>(*c, lay.st_confidence);
    st.out_cap = cfg->max_seq; st.gamma_limit = TANDEM_GAMMA_LIMIT;
    cudaError_t e = cudaMallocHost(reinterpret_cast<void**>(&c->pinned), c->pinned_ints * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaHostAlloc(reinterpret_cast<void**>(&c->hflags), 16 * sizeof(int32_t), cudaHostAllocMapped);
    if (e == cudaSuccess) {
        memset(c->hflags, 0, 16 * sizeof(int32_t));
        int* dptr = nullptr;
        e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&dptr), c->hflags, 0);
        st.host_flags = dptr;
    }
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming);
    for (int j = 0; j < cfg->small.n_layers && e == cudaSuccess; ++j) {
        cudaEvent_t ev = nullptr;
        e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
        if (e == cudaSuccess) c->ev_fork.push_back(ev);
    }
    // Two diagnostic switches, read here once (see tandem.h): launch every kernel eagerly instead of replaying a
    // graph, and plain stream order instead of programmatic dependent launch.  Neither changes any result.
    c->use_graphs = getenv("TANDEM_NO_GRAPH") == nullptr;
    c->use_pdl = getenv("TANDEM_NO_PDL") == nullptr;
    c->n_sms = sm_count();
    if (e == cudaSuccess && cfg->dtype == TANDEM_DTYPE_BF16) {
        // one tensor map per weight matrix: [out_features][in_features], 128 x 64 tiles
        c->wmap.resize(c->w.size());
        c->wmap_ok.assign(c->w.size(), 0);
        bool ok = tmap_encoder() != nullptr;
        auto add = [&](int idx, int rows, int cols) {
            if (ok && make_tmap_bf16(&c->wmap[idx], c->w[idx], (uint64_t)rows, (uint64_t)cols, (uint64_t)cols)) c->wmap_ok[idx] = 1;
            else ok = false;
        };
        for (const Model* m : {&c->large, &c->small}) {
            const int d = m->d.d_model, dff = m->d.d_ff;
            for (int l = 0; l < m->d.n_layers; ++l) {
                add(wi_layer(*m, l, W_WQ), d, d); add(wi_layer(*m, l, W_WK), m->d_kv, d); add(wi_layer(*m, l, W_WV), m->d_kv, d);
                add(wi_layer(*m, l, W_WO), d, d); add(wi_layer(*m, l, W_W1), dff, d); add(wi_layer(*m, l, W_W2), d, dff);
            }
            add(wi_tail(*m, 2), m->d.vocab, d);
        }
        for (int j = 0; j < cfg->small.n_layers; ++j) {
            if (cfg->ff_tandem_kind == TANDEM_FF_LINEAR) add(wi_tandem(*c, j, 0), cfg->small.d_model, cfg->large.d_model);
            else { add(wi_tandem(*c, j, 0), c->hidden, cfg->large.d_model); add(wi_tandem(*c, j, 1), cfg->small.d_model, c->hidden); }
        }
        if (!ok) {
            snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled unavailable or failed for a weight matrix");
            if (c->pinned) cudaFreeHost(c->pinned);
            if (c->hflags) cudaFreeHost(c->hflags);
            if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
            release_side(*c);
            delete c;
            return TANDEM_ERR_CUDA;
        }
        c->tc = true;
        {
            bool okx = true;
            const uint64_t RDx = (uint64_t)lay.dec_rows;
            for (int buf = 0; buf < 3 && okx; ++buf)
                for (int mi = 0; mi < 2 && okx; ++mi) {
                    const Model& mm = mi == 0 ? c->large : c->small;
                    const uint64_t K = buf == 2 ? mm.d.d_ff : mm.d.d_model;
                    const size_t off = buf == 0 ? lay.a32 : (buf == 1 ? lay.o32 : lay.f32);
                    okx = K % 8 == 0 && make_tmap_bf16(&c->xmap[buf][mi], c->arena + off, 2 * RDx, K, K, 16);
                }
            c->xmap_ok = okx;
        }
        const int dhL = cfg->large.d_model / cfg->large.n_heads;
        if (dhL == 64 || dhL == 128) {
            c->kmap.resize(cfg->large.n_layers);
            c->vmap.resize(cfg->large.n_layers);
            bool okm = true;
            const uint64_t kv_rows = (uint64_t)cfg->max_batch * c->large.kv_heads * cfg->max_seq;
            for (int l = 0; l < cfg->large.n_layers && okm; ++l)
                okm = make_tmap_bf16(&c->kmap[l], kv_ptr<bf16>(*c, c->large, l, 0), kv_rows, (uint64_t)dhL, (uint64_t)dhL, ATC_KC) &&
                      make_tmap_bf16(&c->vmap[l], kv_ptr<bf16>(*c, c->large, l, 1), kv_rows, (uint64_t)dhL, (uint64_t)dhL, ATC_KC);
            if (okm) { c->tc_prompt_attn = true; c->prompt_group = ATC_Q; }
        }
    }
    if (e == cudaSuccess) e = cudaMemsetAsync(c->arena + lay.st_n, 0, lay.h_large - lay.st_n, c->stream);
    // positions nobody has written yet are read (and masked, or weighted by zero) by chunked attention: keep them finite
    if (e == cudaSuccess) e = cudaMemsetAsync(c->arena + lay.kv_large, 0, lay.st_n - lay.kv_large, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "%s in tandem_create", cudaGetErrorString(e));
        if (c->pinned) cudaFreeHost(c->pinned);
        if (c->hflags) cudaFreeHost(c->hflags);
        if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
            release_side(*c);
        delete c;
        return TANDEM_ERR_CUDA;
    }
    *out = c;
    return TANDEM_OK;
}

extern "C" tandem_status tandem_destroy(tandem_ctx* c) {
    if (!c) return TANDEM_ERR_INVALID_ARG;
    cudaSetDevice(c->cfg.device);
    cudaError_t e = cudaStreamSynchronize(c->stream);
    if (c->pinned) cudaFreeHost(c->pinned);
    for (cudaEvent_t ev : c->prof.ev) cudaEventDestroy(ev);
    for (auto& g : c->graphs) if (g.exec) cudaGraphExecDestroy(g.exec);
    if (c->hflags) cudaFreeHost(c->hflags);
    if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
    release_side(*c);
    delete c;
    if (e != cudaSuccess) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "%s in tandem_destroy", cudaGetErrorString(e));
        return TANDEM_ERR_CUDA;
    }
    return TANDEM_OK;
}

namespace {

// Prompt pass for n_queries prompts, each the start of `samples` sequences (query q owns sequences q * samples ..
// q * samples + samples - 1).  The large model reads each prompt once, into the first sequence of its query; the
// other sequences of the query get copies of the keys / values it produced (both caches) and the same pending token.
tandem_status prefill_impl(tandem_ctx* c, int n_queries, int samples, const int32_t* prompt_ids, const int32_t* prompt_lens) {
    if (!prompt_ids || !prompt_lens || n_queries < 1 || samples < 1) return TANDEM_ERR_INVALID_ARG;
    const long long batch_ll = (long long)n_queries * samples;
    if (batch_ll > c->cfg.max_batch) return TANDEM_ERR_CAPACITY;
    const int batch = (int)batch_ll;
    const int pos_cap = std::min(c->cfg.max_seq, std::min(c->cfg.large.max_pos, c->cfg.small.max_pos));
    long long rows = 0, total = 0, total_ids = 0;
    int n_max = 0;
    for (int q = 0; q < n_queries; ++q) {
        if (prompt_lens[q] < 1) return TANDEM_ERR_INVALID_ARG;
        if (prompt_lens[q] > pos_cap) return TANDEM_ERR_CAPACITY;
        rows += prompt_lens[q] - 1;
        total += (long long)prompt_lens[q] * samples;
        total_ids += prompt_lens[q];
        n_max = std::max(n_max, prompt_lens[q]);
    }
    if (rows > c->lay.max_rows) return TANDEM_ERR_CAPACITY;
    for (long long i = 0; i < total_ids; ++i)
        if (prompt_ids[i] < 0 || prompt_ids[i] >= c->cfg.large.vocab) return TANDEM_ERR_INVALID_ARG;

    CK(cudaStreamSynchronize(c->stream));   // staging buffer free again; no verify kernel in flight
    c->ticket = 0;                          // the device-side tickets are cleared with the rest of the loop state below
    c->router_ticket = 0;
    c->hflags[0] = 0;
    c->hflags[5] = 0;
    const int M = (int)rows;
    int32_t* p_tok = c->pinned;
    int32_t* p_seq = p_tok + c->lay.max_rows;
    int32_t* p_pos = p_seq + c->lay.max_rows;
    int32_t* p_g0 = p_pos + c->lay.max_rows;
    int32_t* p_gc = p_g0 + c->lay.max_groups;
    int32_t* p_n = p_gc + c->lay.max_groups;
    int32_t* p_pend = p_n + c->cfg.max_batch;
    int m = 0, groups = 0;
    long long off = 0;
    for (int q = 0; q < n_queries; ++q) {
        const int len = prompt_lens[q];
        for (int p = 0; p < len - 1; ++p) {
            if (p % c->prompt_group == 0) { p_g0[groups] = m; p_gc[groups] = std::min(c->prompt_group, len - 1 - p); ++groups; }
            p_tok[m] = prompt_ids[off + p]; p_seq[m] = q * samples; p_pos[m] = p; ++m;
        }
        for (int j = 0; j < samples; ++j) {
            p_n[q * samples + j] = len;
            p_pend[q * samples + j] = prompt_ids[off + len - 1];
        }
        off += len;
    }
    cudaStream_t s = c->stream;
    if (M > 0) {
        CK(cudaMemcpyAsync(c->arena + c->lay.row_tok, p_tok, (size_t)M * 4, cudaMemcpyHostToDevice, s));
        CK(cudaMemcpyAsync(c->arena + c->lay.row_seq, p_seq, (size_t)M * 4, cudaMemcpyHostToDevice, s));
        CK(cudaMemcpyAsync(c->arena + c->lay.row_pos, p_pos, (size_t)M * 4, cudaMemcpyHostToDevice, s));
        CK(cudaMemcpyAsync(c->arena + c->lay.grp_row0, p_g0, (size_t)groups * 4, cudaMemcpyHostToDevice, s));
        CK(cudaMemcpyAsync(c->arena + c->lay.grp_cnt, p_gc, (size_t)groups * 4, cudaMemcpyHostToDevice, s));
    }
    CK(cudaMemsetAsync(c->arena + c->lay.st_n, 0, c->lay.row_tok - c->lay.st_n, s));
    CK(cudaMemcpyAsync(c->st.n, p_n, (size_t)batch * 4, cudaMemcpyHostToDevice, s));
    CK(cudaMemcpyAsync(c->st.pending, p_pend, (size_t)batch * 4, cudaMemcpyHostToDevice, s));
    c->batch = batch;
    c->n_ub = n_max;
    c->n_sum = total;
    c->prompt_sq_sum = 0.0;
    for (int q = 0; q < n_queries; ++q) c->prompt_sq_sum += (double)(prompt_lens[q] - 1) * (prompt_lens[q] - 1);
    if (M > 0) {
        Rows r; r.M = M; r.groups = groups; r.nq = 0; r.decode = false; r.n_chunks = 0; r.kv_positions = (double)rows;
        if (c->cfg.dtype == TANDEM_DTYPE_BF16) large_pass<bf16>(*c, r, true, false);
        else large_pass<float>(*c, r, true, false);
    }
    TRY(check_launch(*c));
    if (samples > 1) {
        // the prompt's keys / values, per (model, layer, K or V, key/value head): positions 0 .. len - 2 of sequence
        // q * samples go to the query's other sequences (one strided copy per destination)
        for (const Model* mdl : {&c->large, &c->small}) {
            const int dh = mdl->d.d_model / mdl->d.n_heads;
            const size_t pitch = (size_t)c->cfg.max_seq * dh * c->esz;            // one head's positions
            const size_t seq_bytes = pitch * mdl->kv_heads;
            for (int l = 0; l < mdl->d.n_layers; ++l)
                for (int which = 0; which < 2; ++which) {
                    unsigned char* base = c->arena + mdl->kv_off + ((size_t)l * 2 + which) * mdl->kv_layer_elems * c->esz;
                    for (int q = 0; q < n_queries; ++q) {
                        const size_t width = (size_t)(prompt_lens[q] - 1) * dh * c->esz;
                        if (width == 0) continue;
                        const unsigned char* src = base + (size_t)q * samples * seq_bytes;
                        for (int j = 1; j < samples; ++j)
                            CK(cudaMemcpy2DAsync(base + ((size_t)q * samples + j) * seq_bytes, pitch, src, pitch, width, mdl->kv_heads,
                                                 cudaMemcpyDeviceToDevice, s));
                    }
                }
        }
    }
    return TANDEM_OK;
}

}  // namespace

extern "C" tandem_status tandem_prefill(tandem_ctx* c, int32_t batch, const int32_t* prompt_ids, const int32_t* prompt_lens) {
    TRY(begin_call(c));
    return prefill_impl(c, batch, 1, prompt_ids, prompt_lens);
}

extern "C" tandem_status tandem_prefill_samples(tandem_ctx* c, int32_t n_queries, int32_t num_samples, const int32_t* prompt_ids,
                                                const int32_t* prompt_lens) {
    TRY(begin_call(c));
    return prefill_impl(c, n_queries, num_samples, prompt_ids, prompt_lens);
}

namespace {

tandem_status capacity_for(tandem_ctx* c, int extra_tokens, int gamma) {
    const int pos_cap = std::min(c->cfg.max_seq, std::min(c->cfg.large.max_pos, c->cfg.small.max_pos));
    // rows of the last iteration reach position (n_ub + extra - 1) + gamma
    if ((long long)c->n_ub + extra_tokens + gamma > pos_cap) return TANDEM_ERR_CAPACITY;
    return TANDEM_OK;
}

}  // namespace

extern "C" tandem_status tandem_block_step(tandem_ctx* c, int32_t gamma, int32_t accept_mode, uint64_t mode_seed,
                                           tandem_step_result* result) {
    TRY(begin_call(c));
    if (gamma < 0 || gamma > c->cfg.gamma_max || accept_mode < 0 || accept_mode > 4) return TANDEM_ERR_INVALID_ARG;
    if (accept_mode == TANDEM_ACCEPT_REPRESENTATION_ONLY && gamma < 1) return TANDEM_ERR_INVALID_ARG;
    if (c->batch == 0) return TANDEM_ERR_STATE;
    TRY(capacity_for(c, 0, gamma));
    reset_call_kernel<<<1, 256, 0, c->stream>>>(c->st, c->batch);
    c->launches++;
    TRY(launch_iteration(*c, 0, gamma, accept_mode, mode_seed, INT_MAX));
    c->n_ub += gamma + 1;
    c->n_sum += (long long)c->batch * (gamma + 1);
    if (result) {
        int32_t* cnt = c->pinned;   // staging is idle outside prefill
        CK(cudaMemcpyAsync(cnt, c->st.counters, 5 * 4, cudaMemcpyDeviceToHost, c->stream));
        const int B = c->batch, GL = TANDEM_GAMMA_LIMIT;
        // everything lands in private buffers first: the caller's arrays are written only once the iteration is known to be good
        std::vector<int32_t> d((size_t)B * GL), t((size_t)B * (GL + 1)), acc((size_t)B), ncm((size_t)B);
        if (result->drafts) CK(cudaMemcpyAsync(d.data(), c->st.drafts, d.size() * 4, cudaMemcpyDeviceToHost, c->stream));
        if (result->targets) CK(cudaMemcpyAsync(t.data(), c->st.targets, t.size() * 4, cudaMemcpyDeviceToHost, c->stream));
        if (result->accept_len) CK(cudaMemcpyAsync(acc.data(), c->st.accept_len, (size_t)B * 4, cudaMemcpyDeviceToHost, c->stream));
        if (result->n_committed) CK(cudaMemcpyAsync(ncm.data(), c->st.n, (size_t)B * 4, cudaMemcpyDeviceToHost, c->stream));
        CK(cudaStreamSynchronize(c->stream));
        c->n_ub = cnt[3];
        c->n_sum = cnt[4];
        if (cnt[2] != 0) {
            snprintf(g_cuda_err, sizeof(g_cuda_err), "device-side wait expired (code %d)", cnt[2]);
            CK(cudaMemsetAsync(c->st.counters + 2, 0, 4, c->stream));
            return TANDEM_ERR_TIMEOUT;
        }
        for (int b = 0; b < B; ++b) {
            if (result->drafts) for (int i = 0; i < gamma; ++i) result->drafts[b * gamma + i] = d[(size_t)b * GL + i];
            if (result->targets) for (int i = 0; i <= gamma; ++i)   // no predictions of the large model in a representation-only round
                result->targets[b * (gamma + 1) + i] = accept_mode == TANDEM_ACCEPT_REPRESENTATION_ONLY ? -1 : t[(size_t)b * (GL + 1) + i];
            if (result->accept_len) result->accept_len[b] = acc[b];
            if (result->n_committed) result->n_committed[b] = ncm[b];
        }
    }
    return TANDEM_OK;
}

namespace {

// lead_large_step: the call starts with one round of the large model alone over the pending token (a block of one
// row with projection and output head), which gives the first new token (Figure 2, left).
tandem_status run_generate(tandem_ctx* c, bool speculative, int gamma, int max_new, int mode, uint64_t seed,
                           int32_t* out_ids, int32_t* out_lens, tandem_stats* stats, bool lead_large_step = false) {
    if (!out_ids || max_new < 1) return TANDEM_ERR_INVALID_ARG;
    if (c->batch == 0) return TANDEM_ERR_STATE;
    if (max_new > c->cfg.max_seq) return TANDEM_ERR_CAPACITY;
    TRY(capacity_for(c, max_new, gamma));
    const int B = c->batch;
    const int64_t launches0 = c->launches;
    reset_call_kernel<<<1, 256, 0, c->stream>>>(c->st, B);
    c->launches++;
    CK(cudaMemsetAsync(c->st.hist, 0, (TANDEM_GAMMA_LIMIT + 1) * 8, c->stream));
    // Iterations are enqueued ahead of the host's knowledge of their outcome.  None can be the last one before
    // ceil(max_new / (gamma + 1)); after that at most DEPTH iterations are in flight beyond the last one whose
    // result the host has seen (surplus iterations find every sequence frozen and change nothing).
    const int DEPTH = 3;
    const int kind = speculative ? 0 : 1;
    const int64_t ticket0 = c->ticket;
    const int per_iter = (mode == TANDEM_ACCEPT_REPRESENTATION_ONLY || mode == 5) ? gamma : gamma + 1;   // most tokens one iteration can emit
    const int lead = lead_large_step ? 1 : 0;
    const int min_iters = lead + (max_new - lead + per_iter - 1) / per_iter;
    const int n_known0 = c->n_ub;
    int64_t enq = 0, seen = 0;   // iterations of this call enqueued / observed
    int n_known = n_known0;      // max_b n_b after the last observed iteration
    bool finished = false;
    while (!finished) {
        if (enq >= min_iters && enq - seen >= DEPTH) {
            TRY(wait_ticket(*c, ticket0 + enq - DEPTH + 1));
        }
        // take whatever has been published so far
        const int64_t pub = (int64_t)((volatile int32_t*)c->hflags)[0] - ticket0;
        if (pub > seen) {
            __sync_synchronize();
            seen = std::min<int64_t>(pub, enq);
            n_known = c->hflags[2];
            c->n_sum = c->hflags[3];
            if (seen >= min_iters && c->hflags[1] <= 0) finished = true;
        }
        if (finished) break;
        if (enq > (int64_t)max_new + DEPTH + 1) return TANDEM_ERR_STATE;   // every live iteration emits a token
        c->n_ub = std::min<long long>((long long)n_known + (enq - seen) * (gamma + 1), (long long)n_known0 + max_new);
        if (lead && enq == 0) TRY(launch_iteration(*c, 0, 0, TANDEM_ACCEPT_NATURAL, 0ull, max_new));
        else TRY(launch_iteration(*c, kind, gamma, mode, seed, max_new));
        ++enq;
    }
    int32_t* cnt = c->pinned;   // staging is idle outside prefill
    CK(cudaMemcpyAsync(cnt, c->st.counters, 8 * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    c->n_ub = cnt[3];
    c->n_sum = cnt[4];
    if (cnt[2] != 0) {   // a bounded device-side wait gave up somewhere in this call
        snprintf(g_cuda_err, sizeof(g_cuda_err), "device-side wait expired (code %d)", cnt[2]);
        CK(cudaMemsetAsync(c->st.counters + 2, 0, 4, c->stream));
        return TANDEM_ERR_TIMEOUT;
    }
    const int64_t iters = cnt[5];
    TRY(check_launch());
    CK(cudaMemcpy2DAsync(out_ids, (size_t)max_new * 4, c->st.out_ids, (size_t)c->st.out_cap * 4, (size_t)max_new * 4, B,
                         cudaMemcpyDeviceToHost, c->stream));
    std::vector<unsigned long long> hist(TANDEM_GAMMA_LIMIT + 1);
    CK(cudaMemcpyAsync(hist.data(), c->st.hist, hist.size() * 8, cudaMemcpyDeviceToHost, c->stream));
    if (out_lens) CK(cudaMemcpyAsync(out_lens, c->st.emitted, (size_t)B * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (stats) {
        memset(stats, 0, sizeof(*stats));
        stats->iterations = iters;
        stats->large_runs = iters;
        stats->small_runs = speculative ? std::max<int64_t>(0, iters - lead) * gamma : 0;
        stats->emitted = (int64_t)B * max_new;
        for (int i = 0; i <= TANDEM_GAMMA_LIMIT; ++i) stats->accept_hist[i] = (int64_t)hist[i];
        stats->kernel_launches = c->launches - launches0;
    }
    return TANDEM_OK;
}

}  // namespace

namespace {

// One adaptive iteration, synchronous: draft steps until the router has stopped every sequence (the host reads the
// count the router publishes after each step) or gamma_max drafts exist, then one verify pass over the longest block.
tandem_status adaptive_iteration(tandem_ctx* c, int gamma_max, int max_new, int* block_max) {
    int s = 0;
    for (; s < gamma_max; ++s) {
        TRY(launch_iteration(*c, 3, s, gamma_max, 0ull, max_new));
        TRY(wait_ticket(*c, c->router_ticket, 5));
        if (c->hflags[6] <= 0) { ++s; break; }
    }
    *block_max = s;
    TRY(launch_iteration(*c, 4, s, 0, 0ull, max_new));
    TRY(wait_ticket(*c, c->ticket, 0));
    c->n_ub = c->hflags[2];
    c->n_sum = c->hflags[3];
    return TANDEM_OK;
}

tandem_status check_error_word(tandem_ctx* c) {
    int32_t* cnt = c->pinned;   // staging is idle outside prefill
    CK(cudaMemcpyAsync(cnt, c->st.counters, 8 * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (cnt[2] != 0) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "device-side wait expired (code %d)", cnt[2]);
        CK(cudaMemsetAsync(c->st.counters + 2, 0, 4, c->stream));
        return TANDEM_ERR_TIMEOUT;
    }
    return TANDEM_OK;
}

}  // namespace

extern "C" tandem_status tandem_set_router(tandem_ctx* c, int32_t top_k, int32_t hidden, const void* w1, const void* b1, const void* w2,
                                           float b2, float tau) {
    TRY(begin_call(c));
    if (!w1 || !b1 || !w2 || top_k < 1 || top_k > RT_MAX_K || hidden < 1 || top_k > c->cfg.small.vocab) return TANDEM_ERR_INVALID_ARG;
    if (((uintptr_t)w1 | (uintptr_t)b1 | (uintptr_t)w2) & 3) return TANDEM_ERR_INVALID_ARG;
    if (sizeof(float) * (size_t)(1 + top_k + (size_t)top_k * c->cfg.small.d_model) > 48 * 1024) return TANDEM_ERR_SHAPE;   // the feature vector sits in shared memory
    CK(cudaStreamSynchronize(c->stream));
    for (auto& g : c->graphs)   // the router's arguments are baked into the captured draft steps
        if (g.kind == 3 && g.exec) { cudaGraphExecDestroy(g.exec); g.exec = nullptr; }
    c->router.w1 = static_cast<const float*>(w1); c->router.b1 = static_cast<const float*>(b1); c->router.w2 = static_cast<const float*>(w2);
    c->router.b2 = b2; c->router.tau = tau; c->router.k = top_k; c->router.hidden = hidden;
    c->has_router = true;
    return TANDEM_OK;
}

extern "C" tandem_status tandem_adaptive_step(tandem_ctx* c, int32_t gamma_max, tandem_step_result* result, int32_t* block_len,
                                              float* confidence) {
    TRY(begin_call(c));
    if (gamma_max < 1 || gamma_max > c->cfg.gamma_max) return TANDEM_ERR_INVALID_ARG;
    if (c->batch == 0 || !c->has_router) return TANDEM_ERR_STATE;
    TRY(capacity_for(c, 0, gamma_max));
    reset_call_kernel<<<1, 256, 0, c->stream>>>(c->st, c->batch);
    c->launches++;
    int block_max = 0;
    TRY(adaptive_iteration(c, gamma_max, INT_MAX, &block_max));
    TRY(check_error_word(c));
    const int B = c->batch, GL = TANDEM_GAMMA_LIMIT;
    std::vector<int32_t> d((size_t)B * GL), t((size_t)B * (GL + 1)), acc((size_t)B), ncm((size_t)B), bl((size_t)B);
    std::vector<float> cf((size_t)B * GL);
    CK(cudaMemcpyAsync(d.data(), c->st.drafts, d.size() * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(t.data(), c->st.targets, t.size() * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(acc.data(), c->st.accept_len, (size_t)B * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(ncm.data(), c->st.n, (size_t)B * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(bl.data(), c->st.block_len, (size_t)B * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(cf.data(), c->st.confidence, cf.size() * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    for (int b = 0; b < B; ++b) {
        for (int i = 0; i < gamma_max; ++i) {   // entries beyond a sequence's own block length are -1 / 0
            const bool own = i < bl[b];
            if (result && result->drafts) result->drafts[b * gamma_max + i] = own ? d[(size_t)b * GL + i] : -1;
            if (confidence) confidence[b * gamma_max + i] = own ? cf[(size_t)b * GL + i] : 0.f;
        }
        if (result && result->targets) for (int i = 0; i <= gamma_max; ++i)
            result->targets[b * (gamma_max + 1) + i] = i <= bl[b] ? t[(size_t)b * (GL + 1) + i] : -1;
        if (result && result->accept_len) result->accept_len[b] = acc[b];
        if (result && result->n_committed) result->n_committed[b] = ncm[b];
        if (block_len) block_len[b] = bl[b];
    }
    return TANDEM_OK;
}

extern "C" tandem_status tandem_adaptive_generate(tandem_ctx* c, int32_t gamma_max, int32_t max_new, int32_t* out_ids, int32_t* out_lens,
                                                  tandem_stats* stats) {
    TRY(begin_call(c));
    if (gamma_max < 1 || gamma_max > c->cfg.gamma_max || !out_ids || max_new < 1) return TANDEM_ERR_INVALID_ARG;
    if (c->batch == 0 || !c->has_router) return TANDEM_ERR_STATE;
    if (max_new > c->cfg.max_seq) return TANDEM_ERR_CAPACITY;
    TRY(capacity_for(c, max_new, gamma_max));
    const int B = c->batch;
    const int64_t launches0 = c->launches;
    reset_call_kernel<<<1, 256, 0, c->stream>>>(c->st, B);
    c->launches++;
    CK(cudaMemsetAsync(c->st.hist, 0, (TANDEM_GAMMA_LIMIT + 1) * 8, c->stream));
    int64_t iters = 0, small_runs = 0;
    for (;;) {
        if (iters > max_new) return TANDEM_ERR_STATE;   // every live iteration emits a token
        int block_max = 0;
        TRY(adaptive_iteration(c, gamma_max, max_new, &block_max));
        ++iters;
        small_runs += block_max;
        if (c->hflags[1] <= 0) break;
    }
    TRY(check_error_word(c));
    CK(cudaMemcpy2DAsync(out_ids, (size_t)max_new * 4, c->st.out_ids, (size_t)c->st.out_cap * 4, (size_t)max_new * 4, B,
                         cudaMemcpyDeviceToHost, c->stream));
    std::vector<unsigned long long> hist(TANDEM_GAMMA_LIMIT + 1);
    CK(cudaMemcpyAsync(hist.data(), c->st.hist, hist.size() * 8, cudaMemcpyDeviceToHost, c->stream));
    if (out_lens) CK(cudaMemcpyAsync(out_lens, c->st.emitted, (size_t)B * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (stats) {
        memset(stats, 0, sizeof(*stats));
        stats->iterations = iters;
        stats->large_runs = iters;
        stats->small_runs = small_runs;
        stats->emitted = (int64_t)B * max_new;
        for (int i = 0; i <= TANDEM_GAMMA_LIMIT; ++i) stats->accept_hist[i] = (int64_t)hist[i];
        stats->kernel_launches = c->launches - launches0;
    }
    return TANDEM_OK;
}

extern "C" tandem_status tandem_speculative_generate(tandem_ctx* c, int32_t gamma, int32_t max_new_tokens, int32_t accept_mode,
                                                     uint64_t mode_seed, int32_t* out_ids, int32_t* out_lens, tandem_stats* stats) {
    TRY(begin_call(c));
    if (gamma < 0 || gamma > c->cfg.gamma_max || accept_mode < 0 || accept_mode > 4) return TANDEM_ERR_INVALID_ARG;
    if (accept_mode == TANDEM_ACCEPT_REPRESENTATION_ONLY && gamma < 1) return TANDEM_ERR_INVALID_ARG;
    return run_generate(c, true, gamma, max_new_tokens, accept_mode, mode_seed, out_ids, out_lens, stats);
}

extern "C" tandem_status tandem_teacher_forced_forward(tandem_ctx* c, int32_t gamma, int32_t batch, const int32_t* ids, const int32_t* lens,
                                                       float* nll, int32_t* top1) {
    TRY(begin_call(c));
    if (!ids || !lens || !nll || batch < 1 || gamma < 1 || gamma > c->cfg.gamma_max) return TANDEM_ERR_INVALID_ARG;
    if (batch > c->cfg.max_batch) return TANDEM_ERR_CAPACITY;
    int max_len = 0;
    long long total = 0;
    for (int b = 0; b < batch; ++b) {
        if (lens[b] < 2) return TANDEM_ERR_INVALID_ARG;
        max_len = std::max(max_len, lens[b]);
        total += lens[b];
    }
    const int pos_cap = std::min(c->cfg.max_seq, std::min(c->cfg.large.max_pos, c->cfg.small.max_pos));
    if ((long long)max_len + gamma > pos_cap) return TANDEM_ERR_CAPACITY;
    for (long long i = 0; i < total; ++i)
        if (ids[i] < 0 || ids[i] >= c->cfg.large.vocab) return TANDEM_ERR_INVALID_ARG;
    // an empty prompt pass: the first token of every sequence is its pending token
    std::vector<int32_t> first((size_t)batch), ones((size_t)batch, 1), padded((size_t)batch * c->cfg.max_seq, 0);
    long long off = 0;
    for (int b = 0; b < batch; ++b) {
        first[b] = ids[off];
        memcpy(padded.data() + (size_t)b * c->cfg.max_seq, ids + off, (size_t)lens[b] * 4);
        off += lens[b];
    }
    TRY(prefill_impl(c, batch, 1, first.data(), ones.data()));
    CK(cudaMemcpyAsync(c->arena + c->lay.forced_ids, padded.data(), padded.size() * 4, cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(c->arena + c->lay.forced_len, lens, (size_t)batch * 4, cudaMemcpyHostToDevice, c->stream));
    CK(cudaStreamSynchronize(c->stream));   // the host arrays above go out of scope
    std::vector<int32_t> scratch_ids((size_t)batch * (max_len - 1));
    TRY(run_generate(c, true, gamma, max_len - 1, 5, 0ull, scratch_ids.data(), nullptr, nullptr));
    std::vector<float> h_nll((size_t)batch * c->cfg.max_seq);
    std::vector<int32_t> h_top((size_t)batch * c->cfg.max_seq);
    CK(cudaMemcpyAsync(h_nll.data(), c->arena + c->lay.forced_nll, h_nll.size() * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(h_top.data(), c->arena + c->lay.forced_top, h_top.size() * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    long long o = 0;
    for (int b = 0; b < batch; ++b)
        for (int p = 0; p + 1 < lens[b]; ++p, ++o) {
            nll[o] = h_nll[(size_t)b * c->cfg.max_seq + p];
            if (top1) top1[o] = h_top[(size_t)b * c->cfg.max_seq + p];
        }
    return TANDEM_OK;
}

extern "C" tandem_status tandem_set_sampling(tandem_ctx* c, float temp_large, float temp_small) {
    TRY(begin_call(c));
    if (!(temp_large > 0.f) || !(temp_small > 0.f)) return TANDEM_ERR_INVALID_ARG;
    if (temp_large == c->temp_large && temp_small == c->temp_small) return TANDEM_OK;
    // the temperatures are kernel arguments baked into the captured iterations: drop the sampled ones
    CK(cudaStreamSynchronize(c->stream));
    for (auto& g : c->graphs)
        if (g.mode == TANDEM_ACCEPT_SAMPLE && g.exec) { cudaGraphExecDestroy(g.exec); g.exec = nullptr; }
    c->temp_large = temp_large;
    c->temp_small = temp_small;
    return TANDEM_OK;
}

extern "C" tandem_status tandem_standalone_generate(tandem_ctx* c, int32_t gamma, int32_t variant, int32_t max_new_tokens,
                                                    int32_t* out_ids, int32_t* out_lens, tandem_stats* stats) {
    TRY(begin_call(c));
    if (gamma < 1 || gamma > c->cfg.gamma_max) return TANDEM_ERR_INVALID_ARG;
    switch (variant) {
        case TANDEM_STANDALONE_FREE_TOKEN:
            return run_generate(c, true, gamma, max_new_tokens, TANDEM_ACCEPT_ALL, 0ull, out_ids, out_lens, stats);
        case TANDEM_STANDALONE_REPRESENTATION_ONLY:
            return run_generate(c, true, gamma, max_new_tokens, TANDEM_ACCEPT_REPRESENTATION_ONLY, 0ull, out_ids, out_lens, stats);
        case TANDEM_STANDALONE_FREE_TOKEN_FULL_PROMPT:
            return run_generate(c, true, gamma, max_new_tokens, TANDEM_ACCEPT_ALL, 0ull, out_ids, out_lens, stats, true);
        default: return TANDEM_ERR_INVALID_ARG;
    }
}

extern "C" tandem_status tandem_large_greedy_generate(tandem_ctx* c, int32_t max_new_tokens, int32_t* out_ids, int32_t* out_lens,
                                                      tandem_stats* stats) {
    TRY(begin_call(c));
    return run_generate(c, false, 0, max_new_tokens, 0, 0ull, out_ids, out_lens, stats);
}

extern "C" int64_t tandem_launch_count(tandem_ctx* c) { return c ? c->launches : -1; }

extern "C" const char* tandem_profile_class_name(int32_t cls) {
    static const char* names[PC_COUNT] = {"gemm_smallm", "gemm_tiled", "attn_split", "attn_merge", "attn_prompt",
                                          "layernorm", "rows", "argmax", "verify", "gemm_tc_decode", "gemm_tc_tiled"};
    return (cls >= 0 && cls < PC_COUNT) ? names[cls] : nullptr;
}

extern "C" tandem_status tandem_profile_enable(tandem_ctx* c, int32_t max_launches) {
    TRY(begin_call(c));
    if (max_launches < 0) return TANDEM_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(c->stream));
    Prof& p = c->prof;
    p.on = max_launches > 0;
    p.used = 0;
    p.cls.clear();
    p.bytes.clear();
    while (p.ev.size() < (size_t)2 * max_launches) {
        cudaEvent_t e;
        CK(cudaEventCreate(&e));
        p.ev.push_back(e);
    }
    return TANDEM_OK;
}

extern "C" tandem_status tandem_profile_read(tandem_ctx* c, int32_t n_classes, double* ms, int64_t* launches, double* work) {
    TRY(begin_call(c));
    if (!ms || !launches || !work || n_classes < 1) return TANDEM_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(c->stream));
    for (int i = 0; i < n_classes; ++i) { ms[i] = 0; launches[i] = 0; work[i] = 0; }
    Prof& p = c->prof;
    for (size_t i = 0; i + 1 < p.used; i += 2) {
        const int cls = p.cls[i / 2];
        if (cls >= n_classes) continue;
        float t = 0.f;
        CK(cudaEventElapsedTime(&t, p.ev[i], p.ev[i + 1]));
        ms[cls] += t;
        launches[cls] += 1;
        work[cls] += p.bytes[i / 2];
    }
    p.used = 0;
    p.cls.clear();
    p.bytes.clear();
    return TANDEM_OK;
}

extern "C" tandem_status tandem_debug_expire_wait(tandem_ctx* c) {
    TRY(begin_call(c));
    if (c->cfg.dtype != TANDEM_DTYPE_BF16) return TANDEM_ERR_UNIMPLEMENTED;
    // One CTA of the decode GEMM over the first 128 x 64 corner of the large model's first query matrix, with the
    // weight loads withheld and a poll limit of 1024: the MMA thread's wait for operands runs out, the kernel
    // records the code in the context's error word and leaves through its normal tear-down.  The (meaningless)
    // product goes to the debug scratch area.
    TcScratch sc = tc_scratch(*c);
    sc.poll_limit = 1024;
    sc.withhold_weights = 1;
    const int d = c->large.d.d_model;
    TcW w = tcw(*c, wi_layer(c->large, 0, W_WQ), -1, -1, std::min(128, d), 64);
    c->next_launch_plain = true;
    launch_tc_decode<PRO_F32, EPI_STORE_F32>(*c, sc, at<float>(*c, c->lay.h_large), d, nullptr, nullptr, 1, w, false,
                                             epi_plain(at<float>(*c, c->lay.dbg), 128));
    return check_launch(*c);
}

extern "C" tandem_status tandem_debug_read(tandem_ctx* c, int32_t what, int32_t layer, int32_t seq, void* host_dst, size_t bytes) {
    TRY(begin_call(c));
    if (!host_dst) return TANDEM_ERR_INVALID_ARG;
    if (c->batch == 0) return TANDEM_ERR_STATE;
    const int B = c->batch, g = c->last_gamma, V = c->cfg.large.vocab;
    CK(cudaStreamSynchronize(c->stream));
    if (what == 0 || what == 1 || what == 2) {
        size_t n;
        const void* src;
        if (what == 0) { n = (size_t)B * (g + 1) * V; src = c->arena + c->lay.logits_large; }
        else if (what == 1) { n = (size_t)g * B * V; src = c->arena + c->lay.logits_small; }
        else { n = (size_t)B * (g + 1) * c->cfg.large.d_model; src = c->arena + c->lay.h_large; }
        if (bytes != n * 4) return TANDEM_ERR_INVALID_ARG;
        if (n) CK(cudaMemcpy(host_dst, src, bytes, cudaMemcpyDeviceToHost));
        return TANDEM_OK;
    }
    if (what >= 3 && what <= 6) {
        const Model& m = (what <= 4) ? c->large : c->small;
        if (layer < 0 || layer >= m.d.n_layers || seq < 0 || seq >= B) return TANDEM_ERR_INVALID_ARG;
        int n_b = 0;
        CK(cudaMemcpy(&n_b, c->st.n + seq, 4, cudaMemcpyDeviceToHost));
        const int n = n_b - 1, H = m.kv_heads, dh = m.d.d_model / m.d.n_heads, d = m.d_kv;
        if (bytes != (size_t)n * d * 4) return TANDEM_ERR_INVALID_ARG;
        if (n == 0) return TANDEM_OK;
        const int which = (what == 3 || what == 5) ? 0 : 1;
        float* dbg = at<float>(*c, c->lay.dbg);
        const size_t total = (size_t)n * d;
        const size_t seq_off = (size_t)seq * H * c->cfg.max_seq * dh;
        if (c->cfg.dtype == TANDEM_DTYPE_BF16)
            gather_kv_kernel<bf16><<<(unsigned)((total + 255) / 256), 256, 0, c->stream>>>(kv_ptr<bf16>(*c, m, layer, which) + seq_off, dbg, n, H, dh, c->cfg.max_seq);
        else
            gather_kv_kernel<float><<<(unsigned)((total + 255) / 256), 256, 0, c->stream>>>(kv_ptr<float>(*c, m, layer, which) + seq_off, dbg, n, H, dh, c->cfg.max_seq);
        TRY(check_launch());
        CK(cudaMemcpyAsync(host_dst, dbg, bytes, cudaMemcpyDeviceToHost, c->stream));
        CK(cudaStreamSynchronize(c->stream));
        return TANDEM_OK;
    }
    if (what == 7) {
        if (bytes != (size_t)B * 4) return TANDEM_ERR_INVALID_ARG;
        CK(cudaMemcpy(host_dst, c->st.n, bytes, cudaMemcpyDeviceToHost));
        return TANDEM_OK;
    }
    return TANDEM_ERR_INVALID_ARG;
}

// ---------------------------------------------------------------------------------------------------
// stand-alone kernels
// ---------------------------------------------------------------------------------------------------

namespace {
struct AttnScratch { size_t rows, total; };
// The kernel reads each row's sequence and position from two int arrays; that is all the work space it needs.
AttnScratch attn_scratch_layout(int batch) {
    AttnScratch s;
    s.rows = 0;
    s.total = align_up((size_t)batch * 2 * 4);
    return s;
}
__global__ void iota_rows_kernel(int* row_seq, int* row_pos, int n, int pos) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) { row_seq[i] = i; row_pos[i] = pos; }
}
}  // namespace

extern "C" size_t tandem_decode_attention_scratch_bytes(int32_t batch, int32_t n_heads, int32_t d_head, int32_t derived_len, int32_t own_len) {
    if (batch < 1 || n_heads < 1 || d_head < 1 || derived_len < 0 || own_len < 0 || derived_len + own_len < 1) return 0;
    return attn_scratch_layout(batch).total;
}

extern "C" tandem_status tandem_decode_attention(const void* q, const void* k_derived, const void* v_derived, const void* k_own,
                                                 const void* v_own, void* out, void* scratch, size_t scratch_bytes, int32_t batch,
                                                 int32_t n_heads, int32_t d_head, int32_t derived_len, int32_t own_len, void* stream) {
    if (!q || !out || !scratch) return TANDEM_ERR_INVALID_ARG;
    if (batch < 1 || n_heads < 1 || derived_len < 0 || own_len < 0 || derived_len + own_len < 1) return TANDEM_ERR_INVALID_ARG;
    if ((derived_len > 0 && (!k_derived || !v_derived)) || (own_len > 0 && (!k_own || !v_own))) return TANDEM_ERR_INVALID_ARG;
    if (d_head != 32 && d_head != 64 && d_head != 128) return TANDEM_ERR_SHAPE;
    if ((long long)batch * n_heads > 65535 * 16) return TANDEM_ERR_SHAPE;
    if (((uintptr_t)q | (uintptr_t)k_derived | (uintptr_t)v_derived | (uintptr_t)k_own | (uintptr_t)v_own | (uintptr_t)out | (uintptr_t)scratch) & 15)
        return TANDEM_ERR_INVALID_ARG;
    const AttnScratch sl = attn_scratch_layout(batch);
    if (scratch_bytes < sl.total) return TANDEM_ERR_ARENA_TOO_SMALL;
    if (batch > 65535) return TANDEM_ERR_SHAPE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned char* sc = static_cast<unsigned char*>(scratch);
    int* row_seq = reinterpret_cast<int*>(sc + sl.rows);
    int* row_pos = row_seq + batch;
    iota_rows_kernel<<<cdiv(batch, 256), 256, 0, s>>>(row_seq, row_pos, batch, derived_len + own_len - 1);
    AttnArgs a; memset(&a, 0, sizeof(a));
    a.q = q; a.ldq = n_heads * d_head; a.kcache = k_derived; a.vcache = v_derived; a.k2 = k_own; a.v2 = v_own;
    a.split = derived_len; a.t_max = derived_len; a.t_max2 = own_len;
    a.out = out; a.ldo = n_heads * d_head; a.row_seq = row_seq; a.row_pos = row_pos; a.nq = 1; a.n_heads = n_heads;
    a.scale = 1.0f / sqrtf((float)d_head);
    tandem_ctx tmp;   // only the stream, the launch counter and the launch options are used by the launch helpers
    tmp.stream = s;
    tmp.use_pdl = false;
    tmp.n_sms = sm_count();
    launch_attn_decode(tmp, d_head, a, batch, 0.0);
    return check_launch();
}

// ---------------------------------------------------------------------------------------------------
// Decode attention for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------------------------

// The per-row index arrays of tandem_decode_attention_static live here instead of in a caller-provided buffer.  Every GPU that loads this library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_attn_scratch[TANDEM_STATIC_SCRATCH_BYTES];

namespace {
// In host code the array's name is only a handle for the runtime, not a device address: the address
// a kernel may use comes from cudaGetSymbolAddress, asked once per device with that device current.
void* g_static_scratch_addr[MAX_DEVICES] = {};
std::mutex g_static_scratch_mutex;

tandem_status static_scratch_for_current_device(void** out) {
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return TANDEM_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_addr[dev]) {
        void* p = nullptr;
        CK(cudaGetSymbolAddress(&p, g_static_attn_scratch));
        g_static_scratch_addr[dev] = p;
    }
    *out = g_static_scratch_addr[dev];
    return TANDEM_OK;
}
}  // namespace

extern "C" tandem_status tandem_decode_attention_static(const void* q, const void* k_derived, const void* v_derived,
                                                        const void* k_own, const void* v_own, void* out, int32_t batch,
                                                        int32_t n_heads, int32_t d_head, int32_t derived_len, int32_t own_len,
                                                        void* stream) {
    if (batch < 1 || n_heads < 1 || d_head < 1 || derived_len < 0 || own_len < 0 || derived_len + own_len < 1)
        return TANDEM_ERR_INVALID_ARG;
    const size_t need = attn_scratch_layout(batch).total;
    if (need > (size_t)TANDEM_STATIC_SCRATCH_BYTES) {
        snprintf(g_cuda_err, sizeof(g_cuda_err),
                 "tandem_decode_attention_static: this batch needs %zu bytes of work space, the built-in buffer holds %d; "
                 "use tandem_decode_attention with your own scratch", need, TANDEM_STATIC_SCRATCH_BYTES);
        return TANDEM_ERR_CAPACITY;
    }
    void* scratch = nullptr;
    TRY(static_scratch_for_current_device(&scratch));
    return tandem_decode_attention(q, k_derived, v_derived, k_own, v_own, out, scratch, (size_t)TANDEM_STATIC_SCRATCH_BYTES, batch,
                                   n_heads, d_head, derived_len, own_len, stream);
}

// ---------------------------------------------------------------------------------------------------
// Stand-alone GEMM entry points: their bounded waits report into one word per device
// ---------------------------------------------------------------------------------------------------

static __device__ int g_standalone_err;

namespace {
int* g_standalone_err_addr[MAX_DEVICES] = {};
std::mutex g_standalone_err_mutex;

// Device address of the current device's error word (looked up once per device); null if the lookup fails, in
// which case the kernels run without reporting.
int* standalone_err_word() {
    const int dev = cur_dev();
    std::lock_guard<std::mutex> lock(g_standalone_err_mutex);
    if (!g_standalone_err_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_standalone_err) == cudaSuccess) g_standalone_err_addr[dev] = static_cast<int*>(p);
    }
    return g_standalone_err_addr[dev];
}

struct ProjScratch { size_t yhat, a_s, rows, total; };
ProjScratch proj_scratch_layout(int rows, int d_small) {
    ProjScratch p;
    size_t off = 0;
    p.yhat = off; off = align_up(off + (size_t)rows * d_small * 4);
    p.a_s = off; off = align_up(off + (size_t)rows * d_small * 4);
    p.rows = off; off = align_up(off + (size_t)rows * 8);
    p.total = off;
    return p;
}
}  // namespace

extern "C" tandem_status tandem_standalone_check(void* stream) {
    int* word = standalone_err_word();
    if (!word) return TANDEM_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int code = 0;
    CK(cudaMemcpyAsync(&code, word, sizeof(int), cudaMemcpyDeviceToHost, s));
    CK(cudaStreamSynchronize(s));
    if (code == 0) return TANDEM_OK;
    snprintf(g_cuda_err, sizeof(g_cuda_err), "device-side wait expired (code %d)", code);
    CK(cudaMemsetAsync(word, 0, sizeof(int), s));
    return TANDEM_ERR_TIMEOUT;
}

extern "C" size_t tandem_ff_tandem_project_scratch_bytes(int32_t rows, int32_t d_small) {
    if (rows < 1 || rows > 256 || d_small < 8) return 0;
    return proj_scratch_layout(rows, d_small).total;
}

extern "C" tandem_status tandem_ff_tandem_project(const void* x, const void* w_t, const void* ln_g, const void* ln_b, const void* wk,
                                                  const void* wv, void* k_out, void* v_out, void* scratch, size_t scratch_bytes,
                                                  int32_t rows, int32_t d_large, int32_t d_small, void* stream) {
    if (!x || !w_t || !ln_g || !ln_b || !wk || !wv || !k_out || !v_out || !scratch) return TANDEM_ERR_INVALID_ARG;
    if (rows < 1 || rows > 256 || d_large < 8 || d_small < 8) return TANDEM_ERR_INVALID_ARG;
    if (d_large % 8 || d_small % 8) return TANDEM_ERR_SHAPE;
    const ProjScratch pl = proj_scratch_layout(rows, d_small);
    if (scratch_bytes < pl.total) return TANDEM_ERR_ARENA_TOO_SMALL;
    if (((uintptr_t)x | (uintptr_t)w_t | (uintptr_t)wk | (uintptr_t)wv | (uintptr_t)k_out | (uintptr_t)v_out | (uintptr_t)scratch |
         (uintptr_t)ln_g | (uintptr_t)ln_b) & 15)
        return TANDEM_ERR_INVALID_ARG;
    tandem_ctx tmp;   // only the stream, the launch counter and the launch options are used by the launch helpers
    tmp.stream = static_cast<cudaStream_t>(stream);
    tmp.use_pdl = false;
    tmp.n_sms = sm_count();
    unsigned char* sc = static_cast<unsigned char*>(scratch);
    float* yhat = reinterpret_cast<float*>(sc + pl.yhat);
    float* a_s = reinterpret_cast<float*>(sc + pl.a_s);
    int* row_seq = reinterpret_cast<int*>(sc + pl.rows);
    int* row_pos = row_seq + rows;
    TcW wt, wkv;
    if (!make_tmap_bf16(&wt.tm[0], w_t, (uint64_t)d_small, (uint64_t)d_large, (uint64_t)d_large) ||
        !make_tmap_bf16(&wkv.tm[0], wk, (uint64_t)d_small, (uint64_t)d_small, (uint64_t)d_small) ||
        !make_tmap_bf16(&wkv.tm[1], wv, (uint64_t)d_small, (uint64_t)d_small, (uint64_t)d_small)) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled unavailable or failed");
        return TANDEM_ERR_CUDA;
    }
    wt.tm[1] = wt.tm[2] = wt.tm[0]; wt.n_segs = 1; wt.seg_rows0 = wt.seg_rows = d_small; wt.K = d_large;
    wkv.tm[2] = wkv.tm[0]; wkv.n_segs = 2; wkv.seg_rows0 = wkv.seg_rows = d_small; wkv.K = d_small;
    iota_rows_kernel<<<cdiv(rows, 256), 256, 0, tmp.stream>>>(row_seq, row_pos, rows, 0);
    EpiArgs e; memset(&e, 0, sizeof(e));
    e.kcache = k_out; e.vcache = v_out; e.row_seq = row_seq; e.row_pos = row_pos; e.n_heads = 1; e.d_head = d_small; e.t_max = 1; e.seg0 = e.seg = d_small;
    // weights streamed once per GEMM and group of 64 rows; for a few short rows the LayerNorm is fused into the
    // second GEMM's operand load
    TcScratch ts; ts.err = standalone_err_word();
    launch_tc_decode<PRO_BF16, EPI_STORE_F32>(tmp, ts, x, d_large, nullptr, nullptr, rows, wt, true, epi_plain(yhat, d_small));
    if (rows <= 8 && d_small <= 1024) {
        launch_tc_decode<PRO_LN, EPI_KV>(tmp, ts, yhat, d_small, ln_g, ln_b, rows, wkv, true, e);
    } else {
        launch_ex(tmp, false, 1, layernorm_rows_kernel<float>, dim3(rows), dim3(128), 0, (const float*)yhat, static_cast<const float*>(ln_g),
                  static_cast<const float*>(ln_b), a_s, (int)d_small, (bf16*)nullptr);
        launch_tc_decode<PRO_F32, EPI_KV>(tmp, ts, a_s, d_small, nullptr, nullptr, rows, wkv, true, e);
    }
    return check_launch();
}

extern "C" tandem_status tandem_block_linear(const void* x, const void* w, void* y, int32_t rows, int32_t in_features,
                                             int32_t out_features, void* stream) {
    if (!x || !w || !y) return TANDEM_ERR_INVALID_ARG;
    if (rows < 1 || rows > 64 || in_features < 8 || out_features < 1) return TANDEM_ERR_INVALID_ARG;
    if (in_features % 8) return TANDEM_ERR_SHAPE;
    if (((uintptr_t)x | (uintptr_t)w | (uintptr_t)y) & 15) return TANDEM_ERR_INVALID_ARG;
    tandem_ctx tmp;   // only the stream, the launch counter and the launch options are used by the launch helpers
    tmp.stream = static_cast<cudaStream_t>(stream);
    tmp.use_pdl = false;
    tmp.n_sms = sm_count();
    TcW tw;
    if (!make_tmap_bf16(&tw.tm[0], w, (uint64_t)out_features, (uint64_t)in_features, (uint64_t)in_features)) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled unavailable or failed");
        return TANDEM_ERR_CUDA;
    }
    tw.tm[1] = tw.tm[2] = tw.tm[0]; tw.n_segs = 1; tw.seg_rows0 = tw.seg_rows = out_features; tw.K = in_features;
    TcScratch ts; ts.err = standalone_err_word();
    launch_tc_decode<PRO_BF16, EPI_STORE>(tmp, ts, x, in_features, nullptr, nullptr, rows, tw, true, epi_plain(y, out_features));
    return check_launch();
}
