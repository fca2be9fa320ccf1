"""ctypes binding of libtandem_b200.so: the same entry points as include/tandem.h, argument marshalling only.

PyTorch is used here for device memory (weights, the arena) and streams; every step of the path runs in
the library's CUDA kernels.  There is no CPU or eager fallback: if the shared library is missing, or no
CUDA device is present, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

from . import synth

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libtandem_b200.so")
_lib = None

GAMMA_LIMIT = 15
ACCEPT_NATURAL, ACCEPT_ALL, ACCEPT_HASH, ACCEPT_REPRESENTATION_ONLY, ACCEPT_SAMPLE = 0, 1, 2, 3, 4
STANDALONE_FREE_TOKEN, STANDALONE_REPRESENTATION_ONLY, STANDALONE_FREE_TOKEN_FULL_PROMPT = 0, 1, 2
STATUS_NAMES = ["OK", "INVALID_ARG", "SHAPE", "ARENA_TOO_SMALL", "CAPACITY", "STATE", "CUDA", "TIMEOUT", "UNIMPLEMENTED"]
(READ_LARGE_LOGITS, READ_SMALL_LOGITS, READ_LARGE_HIDDEN, READ_LARGE_K, READ_LARGE_V, READ_SMALL_K, READ_SMALL_V,
 READ_COMMITTED) = range(8)

EXPORTS = ["tandem_query_arena", "tandem_create", "tandem_destroy", "tandem_prefill", "tandem_block_step",
           "tandem_speculative_generate", "tandem_large_greedy_generate", "tandem_debug_read",
           "tandem_decode_attention_scratch_bytes", "tandem_decode_attention", "tandem_ff_tandem_project",
           "tandem_ff_tandem_project_scratch_bytes", "tandem_block_linear",
           "tandem_status_string", "tandem_last_cuda_error", "tandem_profile_enable", "tandem_profile_read",
           "tandem_profile_class_name", "tandem_launch_count", "tandem_decode_attention_static",
           "tandem_debug_expire_wait", "tandem_standalone_check", "tandem_standalone_generate",
           "tandem_set_sampling", "tandem_prefill_samples", "tandem_set_router", "tandem_adaptive_step",
           "tandem_adaptive_generate", "tandem_teacher_forced_forward"]


class TandemError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        detail = ""
        if status == 6 and _lib is not None:
            detail = ": " + _lib.tandem_last_cuda_error().decode()
        super().__init__(f"{where} failed with TANDEM_ERR_{name}{detail}")


class Dims(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "d_ff", "vocab", "max_pos", "n_kv_heads")]


class Config(C.Structure):
    _fields_ = [("large", Dims), ("small", Dims), ("ff_tandem_kind", C.c_int32), ("ff_tandem_hidden", C.c_int32),
                ("layer_map", C.POINTER(C.c_int32)), ("dtype", C.c_int32), ("max_batch", C.c_int32),
                ("max_seq", C.c_int32), ("gamma_max", C.c_int32), ("max_prefill_rows", C.c_int32),
                ("device", C.c_int32), ("stream", C.c_void_p)]


class Weights(C.Structure):
    _fields_ = [("ptrs", C.POINTER(C.c_void_p)), ("n_ptrs", C.c_int32)]


class StepResult(C.Structure):
    _fields_ = [(n, C.POINTER(C.c_int32)) for n in ("drafts", "targets", "accept_len", "n_committed")]


class Stats(C.Structure):
    _fields_ = [("iterations", C.c_int64), ("large_runs", C.c_int64), ("small_runs", C.c_int64), ("emitted", C.c_int64),
                ("accept_hist", C.c_int64 * (GAMMA_LIMIT + 1)), ("kernel_launches", C.c_int64)]


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads the shared library (once) and declares the signatures of include/tandem.h."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it first (python -m paper_2402_08644_b200.build); "
                           "there is no fallback path")
    lib = C.CDLL(_LIB_PATH)
    i32, u64, vp, sz = C.c_int32, C.c_uint64, C.c_void_p, C.c_size_t
    pi32 = C.POINTER(C.c_int32)
    lib.tandem_query_arena.argtypes = [C.POINTER(Config), C.POINTER(sz)]
    lib.tandem_create.argtypes = [C.POINTER(Config), C.POINTER(Weights), vp, sz, C.POINTER(vp)]
    lib.tandem_destroy.argtypes = [vp]
    lib.tandem_prefill.argtypes = [vp, i32, pi32, pi32]
    lib.tandem_prefill_samples.argtypes = [vp, i32, i32, pi32, pi32]
    lib.tandem_block_step.argtypes = [vp, i32, i32, u64, C.POINTER(StepResult)]
    lib.tandem_speculative_generate.argtypes = [vp, i32, i32, i32, u64, pi32, pi32, C.POINTER(Stats)]
    lib.tandem_large_greedy_generate.argtypes = [vp, i32, pi32, pi32, C.POINTER(Stats)]
    lib.tandem_standalone_generate.argtypes = [vp, i32, i32, i32, pi32, pi32, C.POINTER(Stats)]
    lib.tandem_set_sampling.argtypes = [vp, C.c_float, C.c_float]
    lib.tandem_teacher_forced_forward.argtypes = [vp, i32, i32, pi32, pi32, C.POINTER(C.c_float), pi32]
    lib.tandem_set_router.argtypes = [vp, i32, i32, vp, vp, vp, C.c_float, C.c_float]
    lib.tandem_adaptive_step.argtypes = [vp, i32, C.POINTER(StepResult), pi32, C.POINTER(C.c_float)]
    lib.tandem_adaptive_generate.argtypes = [vp, i32, i32, pi32, pi32, C.POINTER(Stats)]
    lib.tandem_debug_read.argtypes = [vp, i32, i32, i32, vp, sz]
    lib.tandem_decode_attention_scratch_bytes.argtypes = [i32] * 5
    lib.tandem_decode_attention_scratch_bytes.restype = sz
    lib.tandem_decode_attention.argtypes = [vp] * 7 + [sz] + [i32] * 5 + [vp]
    lib.tandem_ff_tandem_project.argtypes = [vp] * 9 + [sz] + [i32] * 3 + [vp]
    lib.tandem_block_linear.argtypes = [vp] * 3 + [i32] * 3 + [vp]
    lib.tandem_ff_tandem_project_scratch_bytes.argtypes = [i32] * 2
    lib.tandem_ff_tandem_project_scratch_bytes.restype = sz
    lib.tandem_decode_attention_static.argtypes = [vp] * 6 + [i32] * 5 + [vp]
    lib.tandem_debug_expire_wait.argtypes = [vp]
    lib.tandem_standalone_check.argtypes = [vp]
    lib.tandem_profile_enable.argtypes = [vp, i32]
    lib.tandem_profile_read.argtypes = [vp, i32, C.POINTER(C.c_double), C.POINTER(C.c_int64), C.POINTER(C.c_double)]
    lib.tandem_profile_class_name.argtypes = [i32]
    lib.tandem_launch_count.argtypes = [vp]
    lib.tandem_launch_count.restype = C.c_int64
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name.endswith("_string") or name.endswith("_cuda_error") or name.endswith("_class_name"):
            fn.restype = C.c_char_p
        elif name not in ("tandem_decode_attention_scratch_bytes", "tandem_ff_tandem_project_scratch_bytes", "tandem_block_linear",
                          "tandem_launch_count"):
            fn.restype = C.c_int
    lib.tandem_status_string.argtypes = [C.c_int]
    lib.tandem_last_cuda_error.argtypes = []
    _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != 0:
        raise TandemError(status, where)


def _dims(d: synth.ModelDims) -> Dims:
    return Dims(d.n_layers, d.d_model, d.n_heads, d.d_ff, d.vocab, d.max_pos, d.n_kv_heads)


def make_config(shape: synth.TandemShape, max_batch: int, max_seq: int, gamma_max: int, device: int = 0,
                stream: int = 0, max_prefill_rows: int = 0):
    """Returns (Config, keep-alive objects)."""
    lm = (C.c_int32 * len(shape.layer_map))(*shape.layer_map)
    cfg = Config(_dims(shape.large), _dims(shape.small), shape.ff_tandem_kind, shape.ff_tandem_hidden, lm, shape.dtype,
                 max_batch, max_seq, gamma_max, max_prefill_rows, device, C.c_void_p(stream or None))
    return cfg, lm


def tandem_query_arena(cfg: Config) -> int:
    out = C.c_size_t(0)
    _check(load_library().tandem_query_arena(C.byref(cfg), C.byref(out)), "tandem_query_arena")
    return out.value


def upload_weights(shape: synth.TandemShape, weights: Dict[str, np.ndarray], device) -> Dict[str, "torch.Tensor"]:
    """Host arrays (float32 values) -> device tensors in the context's storage type; LayerNorm
    parameters stay fp32.  For bf16 shapes the host values are already bf16-representable."""
    import torch
    store = torch.bfloat16 if shape.dtype == synth.DTYPE_BF16 else torch.float32
    out = {}
    for name in synth.weight_names(shape):
        t = torch.from_numpy(np.ascontiguousarray(weights[name], dtype=np.float32))
        out[name] = t.to(device=device, dtype=torch.float32 if synth.is_norm_param(name) else store).contiguous()
    return out


class Tandem:
    """One context: owns the device weights and the arena (as torch tensors) and wraps the C calls."""

    def __init__(self, shape: synth.TandemShape, weights, max_batch: int, max_seq: int, gamma_max: int,
                 device: int = 0, max_prefill_rows: int = 0, stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2402_08644_b200 needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        self.shape, self.max_batch, self.max_seq, self.gamma_max = shape, max_batch, max_seq, gamma_max
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        first = next(iter(weights.values()))
        self.weights = weights if hasattr(first, "data_ptr") else upload_weights(shape, weights, self.device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self.cfg, self._lm = make_config(shape, max_batch, max_seq, gamma_max, device, self.stream.cuda_stream,
                                         max_prefill_rows)
        self.arena_bytes = tandem_query_arena(self.cfg)
        self.arena = torch.empty(self.arena_bytes, dtype=torch.uint8, device=self.device)
        names = synth.weight_names(shape)
        self._ptrs = (C.c_void_p * len(names))(*[self.weights[n].data_ptr() for n in names])
        w = Weights(self._ptrs, len(names))
        ctx = C.c_void_p()
        torch.cuda.synchronize(self.device)
        _check(self.lib.tandem_create(C.byref(self.cfg), C.byref(w), C.c_void_p(self.arena.data_ptr()),
                                      self.arena_bytes, C.byref(ctx)), "tandem_create")
        self.ctx = ctx
        self.batch = 0

    def close(self) -> None:
        if getattr(self, "ctx", None):
            _check(self.lib.tandem_destroy(self.ctx), "tandem_destroy")
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def tandem_prefill(self, prompts: Sequence[Sequence[int]]) -> None:
        lens = np.asarray([len(p) for p in prompts], dtype=np.int32)
        ids = np.ascontiguousarray(np.concatenate([np.asarray(p, dtype=np.int32) for p in prompts]))
        _check(self.lib.tandem_prefill(self.ctx, len(prompts), ids.ctypes.data_as(C.POINTER(C.c_int32)),
                                       lens.ctypes.data_as(C.POINTER(C.c_int32))), "tandem_prefill")
        self.batch = len(prompts)

    def tandem_prefill_samples(self, prompts: Sequence[Sequence[int]], num_samples: int) -> None:
        lens = np.asarray([len(p) for p in prompts], dtype=np.int32)
        ids = np.ascontiguousarray(np.concatenate([np.asarray(p, dtype=np.int32) for p in prompts]))
        _check(self.lib.tandem_prefill_samples(self.ctx, len(prompts), num_samples, ids.ctypes.data_as(C.POINTER(C.c_int32)),
                                               lens.ctypes.data_as(C.POINTER(C.c_int32))), "tandem_prefill_samples")
        self.batch = len(prompts) * num_samples

    def tandem_block_step(self, gamma: int, accept_mode: int = 0, mode_seed: int = 0, want_result: bool = True):
        if not want_result:
            _check(self.lib.tandem_block_step(self.ctx, gamma, accept_mode, mode_seed, None), "tandem_block_step")
            return None
        B = self.batch
        d = np.zeros((B, gamma), np.int32)
        t = np.zeros((B, gamma + 1), np.int32)
        a = np.zeros(B, np.int32)
        n = np.zeros(B, np.int32)
        p = lambda x: x.ctypes.data_as(C.POINTER(C.c_int32))
        res = StepResult(p(d), p(t), p(a), p(n))
        _check(self.lib.tandem_block_step(self.ctx, gamma, accept_mode, mode_seed, C.byref(res)), "tandem_block_step")
        return {"drafts": d, "targets": t, "accept_len": a, "n_committed": n}

    @staticmethod
    def _stats(s: Stats, gamma: int) -> dict:
        return {"iterations": s.iterations, "large_runs": s.large_runs, "small_runs": s.small_runs, "emitted": s.emitted,
                "accept_hist": [int(v) for v in s.accept_hist][: gamma + 1], "kernel_launches": s.kernel_launches}

    def tandem_speculative_generate(self, gamma: int, max_new: int, accept_mode: int = 0, mode_seed: int = 0):
        out = np.zeros((self.batch, max_new), np.int32)
        lens = np.zeros(self.batch, np.int32)
        st = Stats()
        p = lambda x: x.ctypes.data_as(C.POINTER(C.c_int32))
        _check(self.lib.tandem_speculative_generate(self.ctx, gamma, max_new, accept_mode, mode_seed, p(out), p(lens),
                                                    C.byref(st)), "tandem_speculative_generate")
        return out, lens, self._stats(st, gamma)

    def tandem_teacher_forced_forward(self, sequences: Sequence[Sequence[int]], gamma: int):
        """Returns ([nll per sequence], [top1 per sequence]): arrays of len(seq) - 1 entries each."""
        lens = np.asarray([len(p) for p in sequences], dtype=np.int32)
        ids = np.ascontiguousarray(np.concatenate([np.asarray(p, dtype=np.int32) for p in sequences]))
        n = int((lens - 1).sum())
        nll = np.zeros(n, np.float32); top = np.zeros(n, np.int32)
        p = lambda x: x.ctypes.data_as(C.POINTER(C.c_int32))
        _check(self.lib.tandem_teacher_forced_forward(self.ctx, gamma, len(sequences), p(ids), p(lens),
                                                      nll.ctypes.data_as(C.POINTER(C.c_float)), p(top)), "tandem_teacher_forced_forward")
        self.batch = len(sequences)
        cuts = np.cumsum(lens - 1)[:-1]
        return np.split(nll, cuts), np.split(top, cuts)

    def tandem_set_sampling(self, temp_large: float, temp_small: float) -> None:
        _check(self.lib.tandem_set_sampling(self.ctx, temp_large, temp_small), "tandem_set_sampling")

    def tandem_set_router(self, router: Dict[str, np.ndarray], tau: float) -> None:
        """router: {"k", "w1" [hidden][F], "b1", "w2", "b2"} as made by synth.make_router; kept on the device here."""
        import torch
        self._router = {n: torch.from_numpy(np.ascontiguousarray(router[n], dtype=np.float32)).to(self.device) for n in ("w1", "b1", "w2")}
        _check(self.lib.tandem_set_router(self.ctx, int(router["k"]), int(router["w1"].shape[0]), C.c_void_p(self._router["w1"].data_ptr()),
                                          C.c_void_p(self._router["b1"].data_ptr()), C.c_void_p(self._router["w2"].data_ptr()),
                                          float(router["b2"]), float(tau)), "tandem_set_router")

    def tandem_adaptive_step(self, gamma_max: int):
        B = self.batch
        d = np.zeros((B, gamma_max), np.int32); t = np.zeros((B, gamma_max + 1), np.int32)
        a = np.zeros(B, np.int32); n = np.zeros(B, np.int32); bl = np.zeros(B, np.int32)
        cf = np.zeros((B, gamma_max), np.float32)
        p = lambda x: x.ctypes.data_as(C.POINTER(C.c_int32))
        res = StepResult(p(d), p(t), p(a), p(n))
        _check(self.lib.tandem_adaptive_step(self.ctx, gamma_max, C.byref(res), p(bl), cf.ctypes.data_as(C.POINTER(C.c_float))),
               "tandem_adaptive_step")
        return {"drafts": d, "targets": t, "accept_len": a, "n_committed": n, "block_len": bl, "confidence": cf}

    def tandem_adaptive_generate(self, gamma_max: int, max_new: int):
        out = np.zeros((self.batch, max_new), np.int32)
        lens = np.zeros(self.batch, np.int32)
        st = Stats()
        p = lambda x: x.ctypes.data_as(C.POINTER(C.c_int32))
        _check(self.lib.tandem_adaptive_generate(self.ctx, gamma_max, max_new, p(out), p(lens), C.byref(st)), "tandem_adaptive_generate")
        return out, lens, self._stats(st, gamma_max)

    def tandem_standalone_generate(self, gamma: int, variant: int, max_new: int):
        out = np.zeros((self.batch, max_new), np.int32)
        lens = np.zeros(self.batch, np.int32)
        st = Stats()
        p = lambda x: x.ctypes.data_as(C.POINTER(C.c_int32))
        _check(self.lib.tandem_standalone_generate(self.ctx, gamma, variant, max_new, p(out), p(lens), C.byref(st)),
               "tandem_standalone_generate")
        return out, lens, self._stats(st, gamma)

    def tandem_large_greedy_generate(self, max_new: int):
        out = np.zeros((self.batch, max_new), np.int32)
        lens = np.zeros(self.batch, np.int32)
        st = Stats()
        p = lambda x: x.ctypes.data_as(C.POINTER(C.c_int32))
        _check(self.lib.tandem_large_greedy_generate(self.ctx, max_new, p(out), p(lens), C.byref(st)),
               "tandem_large_greedy_generate")
        return out, lens, self._stats(st, 0)

    def tandem_debug_expire_wait(self) -> None:
        _check(self.lib.tandem_debug_expire_wait(self.ctx), "tandem_debug_expire_wait")

    def tandem_launch_count(self) -> int:
        return int(self.lib.tandem_launch_count(self.ctx))

    def tandem_profile_enable(self, max_launches: int) -> None:
        _check(self.lib.tandem_profile_enable(self.ctx, max_launches), "tandem_profile_enable")

    def tandem_profile_read(self) -> dict:
        """{class name: {"ms": total, "launches": n, "work": bytes or flops}} for the recorded launches."""
        names = []
        while self.lib.tandem_profile_class_name(len(names)) is not None:
            names.append(self.lib.tandem_profile_class_name(len(names)).decode())
        n = len(names)
        ms, cnt, work = (C.c_double * n)(), (C.c_int64 * n)(), (C.c_double * n)()
        _check(self.lib.tandem_profile_read(self.ctx, n, ms, cnt, work), "tandem_profile_read")
        return {names[i]: {"ms": ms[i], "launches": int(cnt[i]), "work": work[i]} for i in range(n)}

    def tandem_debug_read(self, what: int, gamma: int = 0, layer: int = 0, seq: int = 0) -> np.ndarray:
        B, V = self.batch, self.shape.large.vocab
        if what == READ_LARGE_LOGITS:
            out = np.zeros((B, gamma + 1, V), np.float32)
        elif what == READ_SMALL_LOGITS:
            out = np.zeros((gamma, B, V), np.float32)
        elif what == READ_LARGE_HIDDEN:
            out = np.zeros((B, gamma + 1, self.shape.large.d_model), np.float32)
        elif what == READ_COMMITTED:
            out = np.zeros(B, np.int32)
        else:
            n = int(self.tandem_debug_read(READ_COMMITTED)[seq]) - 1
            d = self.shape.large.d_kv if what in (READ_LARGE_K, READ_LARGE_V) else self.shape.small.d_kv
            out = np.zeros((n, d), np.float32)
        _check(self.lib.tandem_debug_read(self.ctx, what, layer, seq, out.ctypes.data_as(C.c_void_p), out.nbytes),
               "tandem_debug_read")
        return out


def tandem_decode_attention(q, k_derived, v_derived, k_own, v_own, out=None, scratch=None):
    """bf16 device tensors: q [B][H][dh]; k/v_derived [B][H][Td][dh]; k/v_own [B][H][To][dh].  Returns out."""
    import torch
    lib = load_library()
    B, H, dh = q.shape
    Td, To = k_derived.shape[2], k_own.shape[2]
    need = lib.tandem_decode_attention_scratch_bytes(B, H, dh, Td, To)
    if scratch is None:
        scratch = torch.empty(need, dtype=torch.uint8, device=q.device)
    if out is None:
        out = torch.empty_like(q)
    ptr = lambda t: C.c_void_p(t.data_ptr() if t.numel() else None)
    _check(lib.tandem_decode_attention(ptr(q), ptr(k_derived), ptr(v_derived), ptr(k_own), ptr(v_own), ptr(out),
                                       ptr(scratch), scratch.numel(), B, H, dh, Td, To,
                                       C.c_void_p(torch.cuda.current_stream(q.device).cuda_stream or None)),
           "tandem_decode_attention")
    return out


STATIC_SCRATCH_BYTES = 64 * 1024


def tandem_decode_attention_static(q, k_derived, v_derived, k_own, v_own, out):
    """tandem_decode_attention without a scratch argument, for callers that may not allocate device memory:
    the kernel's work space (8 bytes per sequence) is a buffer built into the library (at most STATIC_SCRATCH_BYTES
    are needed, else TandemError with status CAPACITY).  `out` is required, so this wrapper allocates nothing either.  Calls
    share that buffer: keep them on one stream.  Make the first call on a device outside any stream capture."""
    import torch
    lib = load_library()
    B, H, dh = q.shape
    Td, To = k_derived.shape[2], k_own.shape[2]
    ptr = lambda t: C.c_void_p(t.data_ptr() if t.numel() else None)
    _check(lib.tandem_decode_attention_static(ptr(q), ptr(k_derived), ptr(v_derived), ptr(k_own), ptr(v_own), ptr(out),
                                              B, H, dh, Td, To,
                                              C.c_void_p(torch.cuda.current_stream(q.device).cuda_stream or None)),
           "tandem_decode_attention_static")
    return out


def tandem_ff_tandem_project(x, w_t, ln_g, ln_b, wk, wv, scratch=None):
    """x [rows][d_L] bf16, w_t [d_S][d_L], ln_* [d_S] fp32, wk/wv [d_S][d_S] -> (k, v) [rows][d_S] bf16."""
    import torch
    lib = load_library()
    rows, d_l = x.shape
    d_s = w_t.shape[0]
    k = torch.empty(rows, d_s, dtype=torch.bfloat16, device=x.device)
    v = torch.empty_like(k)
    if scratch is None:
        scratch = torch.empty(lib.tandem_ff_tandem_project_scratch_bytes(rows, d_s), dtype=torch.uint8, device=x.device)
    ptr = lambda t: C.c_void_p(t.data_ptr())
    _check(lib.tandem_ff_tandem_project(ptr(x), ptr(w_t), ptr(ln_g), ptr(ln_b), ptr(wk), ptr(wv), ptr(k), ptr(v),
                                        ptr(scratch), scratch.numel(), rows, d_l, d_s,
                                        C.c_void_p(torch.cuda.current_stream(x.device).cuda_stream or None)),
           "tandem_ff_tandem_project")
    return k, v


def tandem_block_linear(x, w, y=None):
    """x [rows][K] bf16, w [N][K] bf16 -> y [rows][N] bf16 (rows <= 64)."""
    import torch
    lib = load_library()
    rows, k = x.shape
    n = w.shape[0]
    if y is None:
        y = torch.empty(rows, n, dtype=torch.bfloat16, device=x.device)
    _check(lib.tandem_block_linear(C.c_void_p(x.data_ptr()), C.c_void_p(w.data_ptr()), C.c_void_p(y.data_ptr()), rows, k, n,
                                   C.c_void_p(torch.cuda.current_stream(x.device).cuda_stream or None)),
           "tandem_block_linear")
    return y


def tandem_standalone_check(device=None) -> None:
    """Waits for the current stream; raises TandemError(TIMEOUT) if a bounded device-side wait ran out in a
    stand-alone GEMM call since the last check."""
    import torch
    lib = load_library()
    _check(lib.tandem_standalone_check(C.c_void_p(torch.cuda.current_stream(device).cuda_stream or None)),
           "tandem_standalone_check")
