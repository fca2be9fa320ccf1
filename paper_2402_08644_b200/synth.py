"""Seeded synthetic inputs for Tandem + SPEED: model shapes, random-init weights, random prompts.

This module holds no arithmetic of the method.  It only produces the arrays that both the CUDA path
and the CPU checker consume: weight tensors drawn from N(0, std^2), LayerNorm gains of one and
biases of zero, and prompts of i.i.d. uniform token ids.  The fixed-length random prompts stand in
for the paper's CNN/DailyMail, Reddit Posts and LM1B prompts (Section 4.2), and the random-init
weights for its PaLM2 checkpoints (Section 4, "Further Training Details"), none of which are
available here.

Weight layout convention (shared by every consumer): every matrix is stored row-major as
[out_features][in_features], so a linear map is  y = x @ W.T .  Embedding and position tables are
[rows][d_model]; the output head is [vocab][d_model].
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Sequence

import numpy as np

FF_TANDEM_LINEAR = 0  # a single projection d_large -> d_small (the paper's choice, Section 3)
FF_TANDEM_MLP = 1     # two layers with a GELU between them

DTYPE_FP32 = 0
DTYPE_BF16 = 1


@dataclass(frozen=True)
class ModelDims:
    n_layers: int
    d_model: int
    n_heads: int
    d_ff: int
    vocab: int
    max_pos: int
    n_kv_heads: int = 0     # key/value heads (multi-query / grouped-query attention); 0 = n_heads (multi-head)

    @property
    def d_head(self) -> int:
        return self.d_model // self.n_heads

    @property
    def kv_heads(self) -> int:
        return self.n_kv_heads if self.n_kv_heads > 0 else self.n_heads

    @property
    def d_kv(self) -> int:
        """Width of a position's keys (or values): kv_heads * d_head."""
        return self.kv_heads * self.d_head


@dataclass(frozen=True)
class TandemShape:
    large: ModelDims
    small: ModelDims
    ff_tandem_kind: int = FF_TANDEM_LINEAR
    ff_tandem_hidden: int = 0           # MLP only; 0 means d_small
    layer_map: Sequence[int] = field(default_factory=tuple)  # [small.n_layers], values in [0, large.n_layers]
    dtype: int = DTYPE_BF16

    @property
    def hidden(self) -> int:
        return self.ff_tandem_hidden if self.ff_tandem_hidden > 0 else self.small.d_model


def default_layer_map(n_small: int, n_large: int) -> tuple:
    """Evenly spaced assignment: small layer j (0-based) reads the large residual stream after
    floor((j+1) * L_L / L_S) large layers (0 would mean the embedding output)."""
    return tuple(((j + 1) * n_large) // n_small for j in range(n_small))


def make_shape(large: ModelDims, small: ModelDims, kind: int = FF_TANDEM_LINEAR, hidden: int = 0,
               layer_map: Sequence[int] | None = None, dtype: int = DTYPE_BF16) -> TandemShape:
    if layer_map is None:
        layer_map = default_layer_map(small.n_layers, large.n_layers)
    return TandemShape(large, small, kind, hidden, tuple(int(v) for v in layer_map), dtype)


def named_config(name: str, max_pos: int | None = None) -> TandemShape:
    """The model pairs of the benchmark configurations.  `max_pos` sizes the position tables."""
    if name == "tiny":      # fp32 test configuration
        mp = max_pos or 128
        return make_shape(ModelDims(4, 256, 4, 1024, 512, mp), ModelDims(2, 128, 4, 512, 512, mp),
                          FF_TANDEM_MLP, 128, dtype=DTYPE_FP32)
    if name == "small":
        mp = max_pos or 1024
        return make_shape(ModelDims(12, 1024, 16, 4096, 32000, mp), ModelDims(4, 512, 8, 2048, 32000, mp))
    if name == "medium":
        mp = max_pos or 2560
        return make_shape(ModelDims(24, 2048, 16, 8192, 32000, mp), ModelDims(8, 768, 12, 3072, 32000, mp))
    if name == "large":
        mp = max_pos or 8960
        return make_shape(ModelDims(32, 4096, 32, 11008, 32000, mp), ModelDims(12, 1024, 16, 4096, 32000, mp))
    raise KeyError(name)


def with_dtype(shape: TandemShape, dtype: int) -> TandemShape:
    return replace(shape, dtype=dtype)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def weight_names(shape: TandemShape) -> List[str]:
    """The fixed order in which weight pointers cross the C boundary."""
    names: List[str] = []
    for tag, dims in (("L", shape.large), ("S", shape.small)):
        names += [f"{tag}.emb", f"{tag}.pos"]
        for l in range(dims.n_layers):
            p = f"{tag}.{l}."
            names += [p + s for s in ("ln1_g", "ln1_b", "wq", "wk", "wv", "wo", "ln2_g", "ln2_b", "w1", "w2")]
        names += [f"{tag}.lnf_g", f"{tag}.lnf_b", f"{tag}.w_out"]
    for j in range(shape.small.n_layers):
        if shape.ff_tandem_kind == FF_TANDEM_LINEAR:
            names.append(f"T.{j}.w_t")
        else:
            names += [f"T.{j}.w_t1", f"T.{j}.w_t2"]
    return names


def weight_shape(shape: TandemShape, name: str) -> tuple:
    parts = name.split(".")
    if parts[0] == "T":
        dl, ds, hid = shape.large.d_model, shape.small.d_model, shape.hidden
        return {"w_t": (ds, dl), "w_t1": (hid, dl), "w_t2": (ds, hid)}[parts[2]]
    dims = shape.large if parts[0] == "L" else shape.small
    d, f, v = dims.d_model, dims.d_ff, dims.vocab
    leaf = parts[-1]
    table = {"emb": (v, d), "pos": (dims.max_pos, d), "w_out": (v, d),
             "wq": (d, d), "wk": (dims.d_kv, d), "wv": (dims.d_kv, d), "wo": (d, d), "w1": (f, d), "w2": (d, f)}
    if leaf in table:
        return table[leaf]
    return (d,)   # LayerNorm gain / bias


def is_norm_param(name: str) -> bool:
    leaf = name.split(".")[-1]
    return leaf.startswith("ln")


def make_weights(shape: TandemShape, seed: int, std: float = 0.02) -> Dict[str, np.ndarray]:
    """Random-init weights: matrices and tables ~ N(0, std^2); LayerNorm gain 1, bias 0.

    One Philox stream per tensor keyed by (seed, tensor index), so a tensor's values do not depend
    on the others.  For bf16 shapes the values are rounded to bfloat16 once here, so that every
    consumer sees exactly the same numbers.  Arrays are float32.
    """
    out: Dict[str, np.ndarray] = {}
    for t, name in enumerate(weight_names(shape)):
        shp = weight_shape(shape, name)
        if is_norm_param(name):
            fill = 1.0 if name.endswith("_g") else 0.0
            out[name] = np.full(shp, fill, dtype=np.float32)
            continue
        gen = np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, t]))
        w = gen.standard_normal(shp, dtype=np.float32) * np.float32(std)
        if shape.dtype == DTYPE_BF16:
            w = round_to_bf16(w)
        out[name] = w
    return out


def perturb_norm_params(weights: Dict[str, np.ndarray], seed: int, scale: float = 0.1) -> None:
    """In place: give LayerNorm gains and biases non-trivial values (tests only, so that a kernel
    that ignores them cannot pass)."""
    for t, name in enumerate(sorted(weights)):
        if is_norm_param(name):
            gen = np.random.Generator(np.random.Philox(key=[(seed + 7919) & 0xFFFFFFFFFFFFFFFF, t]))
            noise = gen.standard_normal(weights[name].shape, dtype=np.float32) * np.float32(scale)
            weights[name] = (weights[name] + noise).astype(np.float32)


def make_prompts(batch: int, lengths, vocab: int, seed: int) -> List[np.ndarray]:
    """`batch` independent prompts of i.i.d. uniform token ids; `lengths` is an int or a list."""
    if isinstance(lengths, int):
        lengths = [lengths] * batch
    gen = np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, 0xFEED]))
    return [gen.integers(0, vocab, size=int(n), dtype=np.int64).astype(np.int32) for n in lengths]


def self_tandem_shape(dims: ModelDims, dtype: int = DTYPE_FP32) -> TandemShape:
    """A pair whose small model has the large model's shape and reads layer j's input from the
    large residual stream after j layers (tests only; see `make_self_tandem_weights`)."""
    return make_shape(dims, dims, FF_TANDEM_LINEAR, 0, tuple(range(dims.n_layers)), dtype)


def make_self_tandem_weights(shape: TandemShape, seed: int, std: float = 0.02) -> Dict[str, np.ndarray]:
    """Weights for `self_tandem_shape`: the small model is a copy of the large one and every
    FF_Tandem is the identity matrix."""
    w = make_weights(shape, seed, std)
    for name in list(w):
        if name.startswith("S."):
            w[name] = w["L." + name[2:]].copy()
        elif name.startswith("T."):
            w[name] = np.eye(shape.small.d_model, shape.large.d_model, dtype=np.float32)
    return w


def device_weights(shape: TandemShape, seed: int, device) -> Dict[str, "torch.Tensor"]:
    """Random-init weights of the same distribution drawn directly on a CUDA device as torch tensors (bf16
    matrices, fp32 LayerNorm parameters), for shapes too large to draw on the host in reasonable time.  No CPU
    checker run can use them: they serve timing and GPU-internal invariants only."""
    import torch
    g = torch.Generator(device=device).manual_seed(seed)
    out = {}
    for name in weight_names(shape):
        shp = weight_shape(shape, name)
        if is_norm_param(name):
            out[name] = torch.full(shp, 1.0 if name.endswith("_g") else 0.0, dtype=torch.float32, device=device)
        else:
            out[name] = (torch.randn(shp, generator=g, device=device, dtype=torch.float32) * 0.02).to(torch.bfloat16)
    return out


def make_router(shape: TandemShape, k: int, hidden: int, seed: int) -> Dict[str, np.ndarray]:
    """Random-init weights of the adaptive-block-length router (a stand-in for the trained router of Section 3.1):
    w1 [hidden][1 + k + k * d_small] ~ N(0, 1 / fan_in), b1 [hidden] ~ N(0, 0.1^2), w2 [hidden] ~ N(0, 1 / hidden),
    b2 scalar 0.  float32."""
    f = 1 + k + k * shape.small.d_model
    gen = np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, 0xA6]))
    return {"k": k, "w1": (gen.standard_normal((hidden, f), dtype=np.float32) / np.float32(np.sqrt(f))).astype(np.float32),
            "b1": (gen.standard_normal(hidden, dtype=np.float32) * np.float32(0.1)).astype(np.float32),
            "w2": (gen.standard_normal(hidden, dtype=np.float32) / np.float32(np.sqrt(hidden))).astype(np.float32),
            "b2": np.float32(0.0)}
