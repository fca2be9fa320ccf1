"""Pins for the checker's elementary pieces: closed forms, textbook special cases and library routines.

Each test is chosen so that one plausible mistake (a dropped term, a wrong sign, a transposed operand,
a wrong axis) makes it fail."""
import math

import numpy as np
import pytest
import torch

from oracle import tandem_oracle as O
from paper_2402_08644_b200 import synth
from helpers import toy_shape, toy_weights


def test_softmax_rows_sum_to_one_and_shift_invariant():
    rng = np.random.default_rng(0)
    s = rng.normal(size=(7, 33)) * 5
    p = O.softmax(s)
    assert np.allclose(p.sum(-1), 1.0, atol=1e-14)
    assert np.allclose(O.softmax(s + 123.0), p, atol=1e-13)
    # closed form for two logits: sigmoid of the difference
    assert np.isclose(O.softmax(np.array([0.3, -1.1]))[0], 1 / (1 + math.exp(-1.4)))


def test_gelu_closed_forms():
    assert O.gelu(np.array(0.0)) == 0.0
    assert np.isclose(O.gelu(np.array(1.0)), 0.8413447460685429, atol=1e-15)   # Phi(1)
    x = np.linspace(-6, 6, 101)
    assert np.allclose(O.gelu(x) - O.gelu(-x), x, atol=1e-14)                  # odd part is x/2 * 2
    assert np.isclose(O.gelu(np.array(12.0)), 12.0)
    assert abs(O.gelu(np.array(-12.0))) < 1e-12
    t = torch.tensor(x, dtype=torch.float64)
    assert np.allclose(O.gelu(x), torch.nn.functional.gelu(t).numpy(), atol=1e-14)


def test_layer_norm_special_cases_and_library():
    rng = np.random.default_rng(1)
    g, b = rng.normal(size=16), rng.normal(size=16)
    const = np.full((3, 16), 4.25)
    assert np.allclose(O.layer_norm(const, g, b), np.broadcast_to(b, (3, 16)), atol=1e-12)
    x = rng.normal(size=(5, 16)) * 3 + 1
    ref = torch.nn.functional.layer_norm(torch.tensor(x), (16,), torch.tensor(g), torch.tensor(b), eps=1e-5)
    assert np.allclose(O.layer_norm(x, g, b), ref.numpy(), atol=1e-13)
    # unit gain, zero bias: rows have zero mean and (almost) unit biased variance
    y = O.layer_norm(x, np.ones(16), np.zeros(16))
    assert np.allclose(y.mean(-1), 0, atol=1e-13)
    assert np.allclose((y ** 2).mean(-1), x.var(-1) / (x.var(-1) + 1e-5), atol=1e-12)


def test_attend_uniform_keys_is_mean_of_values():
    rng = np.random.default_rng(2)
    q = rng.normal(size=12)
    K = np.tile(rng.normal(size=12), (9, 1))
    V = rng.normal(size=(9, 12))
    assert np.allclose(O.attend(q, K, V, 3), V.mean(0), atol=1e-13)


def test_attend_single_key_returns_its_value_and_matches_library():
    rng = np.random.default_rng(3)
    q = rng.normal(size=16)
    K, V = rng.normal(size=(1, 16)), rng.normal(size=(1, 16))
    assert np.allclose(O.attend(q, K, V, 4), V[0])
    n, H, dh = 11, 4, 4
    K, V = rng.normal(size=(n, 16)), rng.normal(size=(n, 16))
    tq = torch.tensor(q).view(1, H, 1, dh)
    tk = torch.tensor(K).view(n, H, dh).permute(1, 0, 2).unsqueeze(0)
    tv = torch.tensor(V).view(n, H, dh).permute(1, 0, 2).unsqueeze(0)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).reshape(16).numpy()
    assert np.allclose(O.attend(q, K, V, H), ref, atol=1e-13)


def test_argmax_ties_go_to_lowest_id_in_float32():
    assert O.argmax_decision(np.array([0.1, 0.7, 0.7, 0.2])) == 1
    # two values that differ only below float32 resolution tie after rounding
    assert O.argmax_decision(np.array([0.0, 1.0, 1.0 + 1e-12])) == 1
    assert O.argmax_decision(np.array([0.0, 1.0, 1.0 + 1e-6])) == 2


def _torch_decoder_logits(shape, w, ids):
    """The same decoder assembled from torch.nn building blocks (pre-LN TransformerEncoderLayer with a
    causal mask, exact GELU, biases zeroed) in float64."""
    d = shape.large
    layers = []
    for l in range(d.n_layers):
        lay = torch.nn.TransformerEncoderLayer(d.d_model, d.n_heads, d.d_ff, dropout=0.0, activation="gelu",
                                               batch_first=True, norm_first=True, dtype=torch.float64)
        g = lambda k: torch.tensor(w[f"L.{l}.{k}"], dtype=torch.float64)
        with torch.no_grad():
            lay.self_attn.in_proj_weight.copy_(torch.cat([g("wq"), g("wk"), g("wv")], 0))
            lay.self_attn.in_proj_bias.zero_()
            lay.self_attn.out_proj.weight.copy_(g("wo"))
            lay.self_attn.out_proj.bias.zero_()
            lay.linear1.weight.copy_(g("w1")); lay.linear1.bias.zero_()
            lay.linear2.weight.copy_(g("w2")); lay.linear2.bias.zero_()
            lay.norm1.weight.copy_(g("ln1_g")); lay.norm1.bias.copy_(g("ln1_b"))
            lay.norm2.weight.copy_(g("ln2_g")); lay.norm2.bias.copy_(g("ln2_b"))
        lay.eval()
        layers.append(lay)
    S = len(ids)
    t = lambda k: torch.tensor(w[k], dtype=torch.float64)
    h = (t("L.emb")[torch.tensor(ids)] + t("L.pos")[:S]).unsqueeze(0)
    mask = torch.triu(torch.full((S, S), float("-inf"), dtype=torch.float64), diagonal=1)
    reps = [h[0].numpy().copy()]
    with torch.no_grad():
        for lay in layers:
            h = lay(h, src_mask=mask)
            reps.append(h[0].numpy().copy())
        out = torch.nn.functional.layer_norm(h[0], (d.d_model,), t("L.lnf_g"), t("L.lnf_b"), eps=1e-5)
        logits = out @ t("L.w_out").T
    return reps, logits.numpy()


def test_decoder_full_forward_matches_torch_transformer_layers():
    shape = toy_shape()
    w = toy_weights(shape, seed=5)
    ids = synth.make_prompts(1, 13, shape.large.vocab, seed=3)[0]
    dec = O.Decoder(w, "L", shape.large.n_layers, shape.large.n_heads)
    reps, logits = O.decoder_full_forward(dec, ids)
    ref_reps, ref_logits = _torch_decoder_logits(shape, w, [int(i) for i in ids])
    for a, b in zip(reps, ref_reps):
        assert np.allclose(a, b, atol=1e-10, rtol=1e-10)
    assert np.allclose(logits, ref_logits, atol=1e-10, rtol=1e-10)
    assert np.abs(logits).max() > 0.5   # the comparison is not vacuous


def test_splitmix64_matches_published_sequence_head():
    # First outputs of the public-domain splitmix64 generator started from state 0 (Vigna's
    # reference values, widely reproduced): next() adds the golden-ratio increment, then mixes.
    assert O.splitmix64(0) == 0xE220A8397B1DCDAF
    assert O.splitmix64(0x9E3779B97F4A7C15) == 0x6E789E6AA1B965F4
    for g in (1, 3, 7):
        vals = {O.hashed_accept_length(11, 0, it, g) for it in range(200)}
        assert vals == set(range(g + 1))


def _projection(kind, d_large, d_small, hidden, seed):
    rng = np.random.default_rng(seed)
    if kind == synth.FF_TANDEM_LINEAR:
        w = {"T.0.w_t": rng.normal(size=(d_small, d_large))}
    else:
        w = {"T.0.w_t1": rng.normal(size=(hidden, d_large)), "T.0.w_t2": rng.normal(size=(d_small, hidden))}
    return O.TandemProjection(w, 1, kind), w


def test_ff_tandem_mlp_matches_a_library_two_layer_module():
    """Eq. 2, first line, with the two-layer FF_Tandem: Linear -> GELU -> Linear without biases, built
    separately from torch modules.  Non-square widths so that a transposed matrix cannot pass."""
    proj, w = _projection(synth.FF_TANDEM_MLP, d_large=24, d_small=10, hidden=17, seed=5)
    lin1 = torch.nn.Linear(24, 17, bias=False, dtype=torch.float64)
    lin2 = torch.nn.Linear(17, 10, bias=False, dtype=torch.float64)
    with torch.no_grad():
        lin1.weight.copy_(torch.tensor(w["T.0.w_t1"]))
        lin2.weight.copy_(torch.tensor(w["T.0.w_t2"]))
    module = torch.nn.Sequential(lin1, torch.nn.GELU(), lin2)
    x = np.random.default_rng(6).normal(size=(9, 24)) * 2
    with torch.no_grad():
        want = module(torch.tensor(x)).numpy()
    assert np.allclose(proj(0, x), want, atol=1e-12)
    assert np.allclose(proj(0, x[3]), want[3], atol=1e-12)      # a single row, as the cached path calls it


def test_ff_tandem_mlp_hand_cases():
    """First map = identity: the projection is GELU(x) W_T2^T, so dropping the GELU, applying it after the
    second map, or swapping the two matrices all give something else.  Closed-form values at x = 1 and x = 0."""
    d = 6
    rng = np.random.default_rng(7)
    w2 = rng.normal(size=(4, d))
    proj = O.TandemProjection({"T.0.w_t1": np.eye(d), "T.0.w_t2": w2}, 1, synth.FF_TANDEM_MLP)
    x = rng.normal(size=(5, d)) * 2
    phi = 0.5 * (1 + np.vectorize(math.erf)(x / math.sqrt(2)))
    want = (x * phi) @ w2.T
    assert np.allclose(proj(0, x), want, atol=1e-13)
    assert not np.allclose(proj(0, x), x @ w2.T, atol=1e-3)                   # GELU dropped
    assert np.allclose(proj(0, np.zeros(d)), 0.0)
    ones = proj(0, np.ones(d))
    assert np.allclose(ones, 0.8413447460685429 * w2.sum(axis=1), atol=1e-13)     # Phi(1) * row sums
    # second map = identity instead: GELU applies to the first map's output, not to x
    w1 = rng.normal(size=(d, d))
    proj2 = O.TandemProjection({"T.0.w_t1": w1, "T.0.w_t2": np.eye(d)}, 1, synth.FF_TANDEM_MLP)
    h = x @ w1.T
    assert np.allclose(proj2(0, x), h * 0.5 * (1 + np.vectorize(math.erf)(h / math.sqrt(2))), atol=1e-13)


def test_ff_tandem_linear_is_one_matrix_product():
    proj, w = _projection(synth.FF_TANDEM_LINEAR, d_large=24, d_small=10, hidden=0, seed=8)
    x = np.random.default_rng(9).normal(size=(4, 24))
    want = torch.nn.functional.linear(torch.tensor(x), torch.tensor(w["T.0.w_t"])).numpy()
    assert np.allclose(proj(0, x), want, atol=1e-13)


@pytest.mark.parametrize("n_heads,n_kv_heads", [(8, 1), (8, 2), (6, 3), (4, 4)])
def test_attend_grouped_query_matches_library(n_heads, n_kv_heads):
    """Multi-query / grouped-query attention against torch's scaled_dot_product_attention with enable_gqa, and
    against multi-head attention over keys/values repeated per group (the definition)."""
    rng = np.random.default_rng(n_heads * 10 + n_kv_heads)
    dh, n = 5, 11
    q = rng.normal(size=n_heads * dh)
    K = rng.normal(size=(n, n_kv_heads * dh))
    V = rng.normal(size=(n, n_kv_heads * dh))
    got = O.attend(q, K, V, n_heads, n_kv_heads)
    tq = torch.tensor(q).reshape(1, n_heads, 1, dh)
    tk = torch.tensor(K).reshape(n, n_kv_heads, dh).permute(1, 0, 2).unsqueeze(0)
    tv = torch.tensor(V).reshape(n, n_kv_heads, dh).permute(1, 0, 2).unsqueeze(0)
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, enable_gqa=True).reshape(-1).numpy()
    assert np.allclose(got, want, atol=1e-12)
    rep = n_heads // n_kv_heads
    K_full = K.reshape(n, n_kv_heads, dh).repeat(rep, axis=1).reshape(n, n_heads * dh)
    V_full = V.reshape(n, n_kv_heads, dh).repeat(rep, axis=1).reshape(n, n_heads * dh)
    assert np.allclose(got, O.attend(q, K_full, V_full, n_heads), atol=1e-13)
    if 1 < n_kv_heads < n_heads:  # the grouping matters: a rotated head-to-group map gives something else
        assert not np.allclose(got, O.attend(q, np.roll(K_full, dh, axis=1), np.roll(V_full, dh, axis=1), n_heads), atol=1e-3)
