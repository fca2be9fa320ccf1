"""Pins for the sampled SPEED rule of the checker (draft from the small model's distribution, keep with
probability min(1, p/q), redraw from the positive part of p - q): closed forms and exact identities."""
import numpy as np
import pytest

from oracle import tandem_oracle as O
from paper_2402_08644_b200 import synth
from helpers import toy_shape, toy_weights


def test_uniform_variates_are_24_bit_fractions_keyed_by_every_argument():
    u = O.uniform_variate(5, 2, 9, 1)
    assert 0.0 <= u < 1.0 and float(np.float32(u)) == u and (u * (1 << 24)) == int(u * (1 << 24))
    # the definition written out with the published mixing function's first outputs for state 0
    x = O.splitmix64(O.splitmix64(O.splitmix64(O.splitmix64(0)) ^ 0) ^ 0)
    assert O.uniform_variate(0, 0, 0, 0) == (x >> 40) / 2.0 ** 24
    keys = {O.uniform_variate(*k) for k in ((5, 2, 9, 1), (6, 2, 9, 1), (5, 3, 9, 1), (5, 2, 10, 1), (5, 2, 9, 2))}
    assert len(keys) == 5
    us = np.array([O.uniform_variate(1, 0, i, 0) for i in range(4000)])
    assert abs(us.mean() - 0.5) < 0.02 and abs((us < 0.25).mean() - 0.25) < 0.03


def test_draw_index_is_the_inverse_cdf():
    w = np.array([0.0, 2.0, 0.0, 1.0, 5.0, 0.0])
    assert O.draw_index(w, 0.0) == 1 and O.draw_index(w, 0.2499) == 1 and O.draw_index(w, 0.25) == 3
    assert O.draw_index(w, 0.3749) == 3 and O.draw_index(w, 0.375) == 4 and O.draw_index(w, 0.999999) == 4
    # a regular grid of N variates hits index i exactly round(N * p_i) times (up to one per boundary)
    rng = np.random.default_rng(0)
    p = rng.random(17); p /= p.sum()
    N = 20000
    counts = np.bincount([O.draw_index(p, (i + 0.5) / N) for i in range(N)], minlength=17)
    assert np.abs(counts - N * p).max() <= 1.0
    # library routine: searchsorted on the cumulative sum
    for u in rng.random(200):
        assert O.draw_index(p, u) == int(np.searchsorted(np.cumsum(p), u * np.cumsum(p)[-1], side="right"))


def test_rejection_rule_reproduces_the_target_distribution_exactly():
    """P(token t is emitted at a position) = q(t) min(1, p(t)/q(t)) + P(reject) * residual(t) must equal p(t):
    the identity that makes sampled SPEED distribute like the large model (Section 3.1: quality matching the
    verifier)."""
    rng = np.random.default_rng(3)
    for _ in range(5):
        p = O.temperature_softmax(rng.normal(size=23) * 2, 0.7)
        q = O.temperature_softmax(rng.normal(size=23) * 2, 1.0)
        keep = np.array([q[t] * O.accept_probability(p, q, t) for t in range(23)])
        res = O.residual_weights(p, q)
        emitted = keep + (1.0 - keep.sum()) * res / res.sum()
        assert np.allclose(emitted, p, atol=1e-14)
        assert np.isclose(1.0 - keep.sum(), 0.5 * np.abs(p - q).sum(), atol=1e-14)    # P(reject) = total variation distance
    # identical distributions: every draft is kept
    assert all(O.accept_probability(p, p, t) == 1.0 for t in range(23))


def test_temperature_softmax_limits():
    lg = np.array([0.3, 2.0, -1.0, 1.9])
    assert np.allclose(O.temperature_softmax(lg, 1.0), O.softmax(lg))
    assert O.temperature_softmax(lg, 1e-3).argmax() == 1 and O.temperature_softmax(lg, 1e-3)[1] > 1 - 1e-12
    assert np.allclose(O.temperature_softmax(lg, 1e6), 0.25, atol=1e-5)
    assert np.isclose(O.temperature_softmax(np.array([0.0, np.log(3.0)]), 0.5)[1], 0.9)     # 3^2 / (1 + 3^2)


def test_cold_sampling_is_greedy_speed_and_self_tandem_keeps_every_draft():
    shape = toy_shape()
    w = toy_weights(shape, seed=8)
    prompt = [int(t) for t in synth.make_prompts(1, [6], shape.large.vocab, 3)[0]]
    greedy, acc_g = O.TandemOracle(shape, w).generate(prompt, 3, 10)
    cold, acc_c = O.TandemOracle(shape, w).generate_sampling(prompt, 3, 10, 1e-4, 1e-4, seed=5)
    assert cold == greedy == O.plain_greedy(shape, w, prompt, 10) and acc_c == acc_g
    dims = synth.ModelDims(2, 32, 4, 64, 50, 64)
    st = synth.self_tandem_shape(dims)
    ws = synth.make_self_tandem_weights(st, seed=6, std=0.35)
    o = O.TandemOracle(st, ws)
    o.prefill(prompt)
    for _ in range(3):
        r = o.step_sampling(4, 0.8, 0.8, seed=11)
        assert r["accept_len"] == 4 and all(abs(x - 1.0) < 1e-9 for x in r["ratios"])
        assert r["emitted"] == r["drafts"] + [r["final"]] and o.large_cache.length() == len(o.tokens) - 1


def test_sampled_steps_follow_the_rule_and_forced_choices_are_replayed():
    shape = toy_shape()
    w = toy_weights(shape, seed=9)
    prompt = [int(t) for t in synth.make_prompts(1, [5], shape.large.vocab, 4)[0]]
    a, b = O.TandemOracle(shape, w), O.TandemOracle(shape, w)
    a.prefill(prompt); b.prefill(prompt)
    seen = set()
    for it in range(8):
        r = a.step_sampling(3, 0.9, 1.0, seed=21, seq=2)
        k = r["accept_len"]
        seen.add(k)
        assert all(r["tests"][i] < r["ratios"][i] for i in range(k)) and (k == 3 or r["tests"][k] >= r["ratios"][k])
        assert r["final"] == O.draw_index(r["final_weights"], r["u_final"])
        if k < 3:
            assert r["final_weights"][r["drafts"][k]] == 0.0 or r["p"][k][r["drafts"][k]] > r["q"][k][r["drafts"][k]]
        f = b.step_sampling(3, 0.9, 1.0, seed=21, seq=2, forced={"drafts": r["drafts"], "accept_len": k, "final": r["final"]})
        assert f["own_drafts"] == r["drafts"] and f["own_accept_len"] == k and f["own_final"] == r["final"]
        assert a.tokens == b.tokens and a.large_cache.length() == b.large_cache.length() == len(a.tokens) - 1
    assert len(seen) >= 2          # the run exercised more than one accept length
