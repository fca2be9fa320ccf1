"""Pins for the adaptive block length of the checker: the router's features and perceptron against closed forms
and library routines, and the loop's invariants (exactness for any router, fixed-length limits)."""
import numpy as np
import pytest
import torch

from oracle import tandem_oracle as O
from paper_2402_08644_b200 import synth
from helpers import toy_shape, toy_weights


def _router(shape, tau, seed=3, k=3, hidden=8):
    r = synth.make_router(shape, k, hidden, seed)
    return O.Router(r["k"], r["w1"], r["b1"], r["w2"], r["b2"], tau)


def test_router_features_closed_forms_and_library():
    rng = np.random.default_rng(0)
    emb = rng.normal(size=(7, 4))
    r = O.Router(2, np.zeros((3, 1 + 2 + 8)), np.zeros(3), np.zeros(3), 0.0, 0.5)
    x = r.features(np.zeros(7), emb)                     # uniform distribution
    assert np.isclose(x[0], np.log(7.0)) and np.allclose(x[1:3], 1 / 7)
    assert np.allclose(x[3:7], emb[0]) and np.allclose(x[7:11], emb[1])       # ties: lowest ids first
    lg = np.array([0.1, 3.0, -1.0, 2.5, 0.0, 2.5, -4.0])
    x = r.features(lg, emb)
    q = torch.softmax(torch.tensor(lg), 0)
    assert np.isclose(x[0], torch.distributions.Categorical(probs=q).entropy().item(), atol=1e-12)
    tv, ti = torch.topk(q, 2)
    assert np.allclose(x[1:3], tv.numpy()) and ti.tolist() == [1, 3]          # 2.5 twice: id 3 before id 5
    assert np.allclose(x[3:7], emb[1]) and np.allclose(x[7:11], emb[3])
    peaked = r.features(np.array([50.0, 0, 0, 0, 0, 0, 0]), emb)
    assert peaked[0] < 1e-15 * 50 + 1e-12 and np.isclose(peaked[1], 1.0)


def test_router_perceptron_matches_a_library_module_and_hand_case():
    rng = np.random.default_rng(1)
    k, d, hidden, V = 3, 5, 6, 11
    emb = rng.normal(size=(V, d))
    w1, b1, w2, b2 = rng.normal(size=(hidden, 1 + k + k * d)), rng.normal(size=hidden), rng.normal(size=hidden), 0.3
    r = O.Router(k, w1, b1, w2, b2, 0.8)
    lg = rng.normal(size=V) * 2
    lin1 = torch.nn.Linear(1 + k + k * d, hidden, dtype=torch.float64)
    lin2 = torch.nn.Linear(hidden, 1, dtype=torch.float64)
    with torch.no_grad():
        lin1.weight.copy_(torch.tensor(w1)); lin1.bias.copy_(torch.tensor(b1))
        lin2.weight.copy_(torch.tensor(w2)[None]); lin2.bias.fill_(b2)
        want = torch.sigmoid(lin2(torch.relu(lin1(torch.tensor(r.features(lg, emb)))))).item()
    assert np.isclose(r.disagreement(lg, emb), want, atol=1e-13)
    go_on, conf = r.keep_drafting(lg, emb)
    assert np.isclose(conf, 1 - want) and go_on == (1 - want >= 0.8)
    # zero weights: s = sigmoid(b2); a large negative b2 means "never disagrees"
    z = O.Router(k, np.zeros_like(w1), np.zeros(hidden), np.zeros(hidden), 0.0, 0.5)
    assert z.disagreement(lg, emb) == 0.5 and z.keep_drafting(lg, emb)[0]
    # relu, not identity: negative pre-activations contribute nothing
    neg = O.Router(k, np.zeros_like(w1), -np.ones(hidden), np.ones(hidden), 0.0, 0.5)
    assert neg.disagreement(lg, emb) == 0.5


def test_adaptive_loop_is_exact_for_any_router_and_has_the_fixed_length_limits():
    shape = toy_shape()
    w = toy_weights(shape, seed=5)
    prompt = [int(t) for t in synth.make_prompts(1, [6], shape.large.vocab, 3)[0]]
    greedy = O.plain_greedy(shape, w, prompt, 12)
    always = _router(shape, tau=-1.0)       # confidence always >= tau: drafts gamma_max tokens every time
    never = _router(shape, tau=2.0)         # never: one draft per iteration
    t_a, len_a = O.TandemOracle(shape, w).generate_adaptive(prompt, 4, 12, always)
    t_n, len_n = O.TandemOracle(shape, w).generate_adaptive(prompt, 4, 12, never)
    fixed4, acc4 = O.TandemOracle(shape, w).generate(prompt, 4, 12)
    fixed1, acc1 = O.TandemOracle(shape, w).generate(prompt, 1, 12)
    assert t_a == t_n == greedy == fixed4 == fixed1
    assert set(len_a) == {4} and set(len_n) == {1} and len(len_a) == len(acc4) and len(len_n) == len(acc1)
    # a router in between: pick tau as the median confidence it shows, so that both outcomes occur
    probe = O.TandemOracle(shape, w)
    probe.prefill(prompt)
    confs = [c for _ in range(4) for c in probe.step_adaptive(4, always)["confidences"]]
    mixed = _router(shape, tau=float(np.median(confs)))
    o = O.TandemOracle(shape, w)
    toks, lens = o.generate_adaptive(prompt, 4, 12, mixed)
    assert toks == greedy and len(set(lens)) >= 2 and all(1 <= n <= 4 for n in lens)
    assert o.n_small_runs == sum(lens) and o.n_large_runs == len(lens)       # the run counts of Table 6


def test_adaptive_step_records_and_forced_replay():
    shape = toy_shape()
    w = toy_weights(shape, seed=6)
    prompt = [int(t) for t in synth.make_prompts(1, [5], shape.large.vocab, 4)[0]]
    probe = O.TandemOracle(shape, w)
    probe.prefill(prompt)
    always = _router(shape, tau=-1.0)
    confs = [c for _ in range(3) for c in probe.step_adaptive(5, always)["confidences"]]
    router = _router(shape, tau=float(np.median(confs)))
    a, b = O.TandemOracle(shape, w), O.TandemOracle(shape, w)
    a.prefill(prompt); b.prefill(prompt)
    for _ in range(5):
        r = a.step_adaptive(5, router)
        n = r["block_len"]
        assert all(c >= router.tau for c in r["confidences"][: n - 1]) and (n == 5 or r["confidences"][n - 1] < router.tau)
        assert len(r["targets"]) == n + 1 and r["accept_len"] <= n
        f = b.step_adaptive(5, router, forced_len=n, forced_drafts=r["drafts"])
        assert f["own_block_len"] == n and f["own_drafts"] == r["drafts"] and a.tokens == b.tokens
