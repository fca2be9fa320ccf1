"""Small shapes and helpers shared by the tests (no method arithmetic here)."""
import numpy as np

from paper_2402_08644_b200 import synth


def toy_shape(kind=synth.FF_TANDEM_LINEAR, layer_map=None, dtype=synth.DTYPE_FP32, max_pos=64,
              large=(3, 32, 4, 64), small=(2, 16, 2, 48), vocab=50, hidden=0):
    L = synth.ModelDims(large[0], large[1], large[2], large[3], vocab, max_pos)
    S = synth.ModelDims(small[0], small[1], small[2], small[3], vocab, max_pos)
    return synth.make_shape(L, S, kind, hidden, layer_map, dtype)


def toy_weights(shape, seed=1, std=0.35, perturb=True):
    """Larger std than the benchmark's 0.02 so that attention is far from uniform and logits are
    well separated; LayerNorm gains/biases perturbed so they cannot be ignored."""
    w = synth.make_weights(shape, seed, std)
    if perturb:
        synth.perturb_norm_params(w, seed)
    return w
