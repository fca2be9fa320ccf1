"""Pins for the checker's algorithmic paths: what the paper and the mathematics fix.

I1  greedy Tandem + SPEED emits exactly plain greedy decoding of the large model (abstract, Section 3.1)
I2  one block pass over gamma+1 tokens equals gamma+1 single-token passes (Section 3 "Inference")
I3  with no large-processed positions the small model is a plain decoder (Section 1: gamma -> infinity)
I4  gamma = 0 is a plain greedy step of the large model (Section 1: gamma = 0)
I5  self-tandem (small == large, identity FF_Tandem, l(j) = j): Eq. 2 collapses to Eq. 1 for ANY boundary
I6  cached mixed-context path equals brute-force recomputation of Eq. 2
plus the schedule of Figures 2 and 3, hand-made accept cases, forced modes and run counts.
"""
import os

import numpy as np
import torch
import pytest

from oracle import tandem_oracle as O
from paper_2402_08644_b200 import synth
from helpers import toy_shape, toy_weights

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _prompt(shape, n, seed=0):
    return [int(t) for t in synth.make_prompts(1, n, shape.large.vocab, seed)[0]]


@pytest.mark.parametrize("gamma", [1, 2, 3, 4, 5, 8])
@pytest.mark.parametrize("kind", [synth.FF_TANDEM_LINEAR, synth.FF_TANDEM_MLP])
def test_I1_speed_equals_plain_greedy(gamma, kind):
    shape = toy_shape(kind=kind, hidden=24 if kind else 0)
    w = toy_weights(shape, seed=gamma)
    prompt = _prompt(shape, 6, seed=gamma)
    want = O.plain_greedy(shape, w, prompt, 12)
    got, accepts = O.TandemOracle(shape, w).generate(prompt, gamma, 12)
    assert got == want
    assert all(0 <= a <= gamma for a in accepts)


def test_I1_holds_for_a_garbage_small_model_and_a_one_token_prompt():
    shape = toy_shape()
    w = toy_weights(shape, seed=3)
    for k in w:
        if k.startswith("S.") and not synth.is_norm_param(k):
            w[k] = w[k] * 40.0          # nonsense drafts
    for P in (1, 2, 9):
        prompt = _prompt(shape, P, seed=P)
        assert O.TandemOracle(shape, w).generate(prompt, 3, 10)[0] == O.plain_greedy(shape, w, prompt, 10)
    assert O.plain_greedy_cached(shape, w, _prompt(shape, 5), 9) == O.plain_greedy(shape, w, _prompt(shape, 5), 9)


def test_I2_block_pass_equals_single_token_passes_and_full_forward():
    shape = toy_shape()
    w = toy_weights(shape, seed=7)
    dec = O.Decoder(w, "L", shape.large.n_layers, shape.large.n_heads)
    ids = _prompt(shape, 11)
    c1, c2 = O.KVCache(dec.n_layers), O.KVCache(dec.n_layers)
    O.large_block_pass(dec, c1, ids[:6], 0)
    O.large_block_pass(dec, c2, ids[:6], 0)
    reps_b, logits_b = O.large_block_pass(dec, c1, ids[6:], 6)
    rows = [O.large_block_pass(dec, c2, [t], 6 + r) for r, t in enumerate(ids[6:])]
    for r, (reps_s, logits_s) in enumerate(rows):
        assert np.allclose(logits_b[r], logits_s[0], atol=1e-10)
        for l in range(dec.n_layers + 1):
            assert np.allclose(reps_b[l][r], reps_s[l][0], atol=1e-10)
    for l in range(dec.n_layers):
        assert np.allclose(np.stack(c1.k[l]), np.stack(c2.k[l]), atol=1e-10)
        assert np.allclose(np.stack(c1.v[l]), np.stack(c2.v[l]), atol=1e-10)
    full_reps, full_logits = O.decoder_full_forward(dec, ids)
    assert np.allclose(full_logits[6:], logits_b, atol=1e-10)
    assert np.allclose(full_reps[2][6:], reps_b[2], atol=1e-10)
    assert np.abs(full_logits).max() > 0.5


def test_I3_no_large_context_means_plain_small_decoder():
    shape = toy_shape()
    w = toy_weights(shape, seed=9)
    ids = _prompt(shape, 7)
    o = O.TandemOracle(shape, w)
    o.prefill(ids[:1])                         # one-token prompt: the large model has seen nothing
    _, logits = o.draft(6, forced=ids[1:7])
    small = O.Decoder(w, "S", shape.small.n_layers, shape.small.n_heads)
    _, want = O.decoder_full_forward(small, ids[:6])
    assert np.allclose(np.stack(logits), want, atol=1e-10)


def test_I4_gamma_zero_is_a_plain_large_step():
    shape = toy_shape()
    w = toy_weights(shape, seed=2)
    prompt = _prompt(shape, 5)
    got, accepts = O.TandemOracle(shape, w).generate(prompt, 0, 7)
    assert got == O.plain_greedy(shape, w, prompt, 7)
    assert accepts == [0] * 7


@pytest.mark.parametrize("gamma", [1, 3, 4])
def test_I5_self_tandem_accepts_everything(gamma):
    dims = synth.ModelDims(3, 32, 4, 64, 50, 64)
    shape = synth.self_tandem_shape(dims)
    w = synth.make_self_tandem_weights(shape, seed=4, std=0.35)
    synth.perturb_norm_params(w, 4)
    for k in list(w):                          # keep the copy exact after perturbing the norms
        if k.startswith("S."):
            w[k] = w["L." + k[2:]].copy()
    prompt = _prompt(shape, 5)
    o = O.TandemOracle(shape, w)
    o.prefill(prompt)
    for it in range(4):
        res = o.step(gamma)
        assert res["accept_len"] == gamma
        assert res["drafts"] == res["targets"][:gamma]
        for s in range(gamma):                 # the small model's logits are the large model's
            assert np.allclose(res["small_logits"][s], res["large_logits"][s], atol=1e-9)
    assert o.tokens[5:] == O.plain_greedy(shape, w, prompt, 4 * (gamma + 1))


@pytest.mark.parametrize("kind", [synth.FF_TANDEM_LINEAR, synth.FF_TANDEM_MLP])
def test_I6_cached_mixed_context_equals_brute_force_eq2(kind):
    shape = toy_shape(kind=kind, hidden=20 if kind else 0, layer_map=(1, 3))
    w = toy_weights(shape, seed=11)
    prompt = _prompt(shape, 6)
    o = O.TandemOracle(shape, w)
    o.prefill(prompt)
    large = O.Decoder(w, "L", shape.large.n_layers, shape.large.n_heads)
    small = O.Decoder(w, "S", shape.small.n_layers, shape.small.n_heads)
    proj = O.TandemProjection(w, shape.small.n_layers, kind)
    for it in range(4):
        n = len(o.tokens)
        drafts, s_logits = o.draft(3)
        seq = o.tokens + drafts[:-1]                      # inputs of the three draft steps
        reps, _ = O.decoder_full_forward(large, o.tokens[: n - 1])
        want = O.tandem_small_full_forward(small, proj, shape.layer_map, reps, n - 1, seq)
        assert np.allclose(np.stack(s_logits), want, atol=1e-10)
        targets, l_logits, xs = o.verify(drafts)
        a = (it * 2) % 4                                  # 0, 2, 0, 2 ... plus 3 below: ragged rollback
        if it == 3:
            a = 3
        o.commit(a, drafts, targets, xs)
        # provenance: every derived key equals a from-scratch projection of the large model's reps
        reps_now, _ = O.decoder_full_forward(large, o.tokens[:-1])
        for j in range(small.n_layers):
            p = small.layers[j]
            ctx = O.layer_norm(proj(j, reps_now[shape.layer_map[j]]), p["ln1_g"], p["ln1_b"])
            assert np.allclose(np.stack(o.derived.k[j]), ctx @ p["wk"].T, atol=1e-10)
            assert np.allclose(np.stack(o.derived.v[j]), ctx @ p["wv"].T, atol=1e-10)
        assert o.large_cache.length() == len(o.tokens) - 1 and o.own.length() == 0


def test_brute_force_eq2_is_sensitive_to_the_boundary():
    """The mixed context matters: moving the boundary changes the small model's logits (so the
    equalities above are not satisfied by a path that ignores the large model)."""
    shape = toy_shape()
    w = toy_weights(shape, seed=13)
    ids = _prompt(shape, 8)
    large = O.Decoder(w, "L", shape.large.n_layers, shape.large.n_heads)
    small = O.Decoder(w, "S", shape.small.n_layers, shape.small.n_heads)
    proj = O.TandemProjection(w, shape.small.n_layers, 0)
    reps, _ = O.decoder_full_forward(large, ids)
    a = O.tandem_small_full_forward(small, proj, shape.layer_map, reps, 6, ids)[-1]
    b = O.tandem_small_full_forward(small, proj, shape.layer_map, reps, 3, ids)[-1]
    assert np.abs(a - b).max() > 1e-3


def test_accept_all_equals_standalone_tandem_with_free_token():
    for kind, gamma in ((synth.FF_TANDEM_LINEAR, 2), (synth.FF_TANDEM_MLP, 3)):
        shape = toy_shape(kind=kind, hidden=12 if kind else 0)
        w = toy_weights(shape, seed=21 + gamma)
        prompt = _prompt(shape, 5, seed=gamma)
        got, accepts = O.TandemOracle(shape, w).generate(prompt, gamma, 11, mode=O.ACCEPT_ALL)
        assert got == O.standalone_tandem_free_token(shape, w, prompt, gamma, 11)
        assert accepts == [gamma] * len(accepts)
        assert got != O.plain_greedy(shape, w, prompt, 11)     # it is a different decoder


def _read_schedule(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                m, a, b = line.split()
                rows.append((m, list(range(int(a), int(b) + 1))))
    return rows


def test_schedule_matches_figures_2_and_3():
    shape = toy_shape()
    w = toy_weights(shape, seed=1)
    fig2 = _read_schedule("fig2_schedule_gamma2.txt")
    o = O.TandemOracle(shape, w)
    o.prefill(_prompt(shape, 9))
    for _ in range(3):
        o.step(2, mode=O.ACCEPT_ALL)
    assert o.schedule == fig2
    fig3 = _read_schedule("fig3_prompt_schedule_gamma2.txt")
    o = O.TandemOracle(shape, w)
    o.prefill(_prompt(shape, 8))
    o.draft(2)
    assert o.schedule == fig3


def test_accept_length_hand_cases():
    A = O.TandemOracle.accept_length
    assert A([5, 6, 7], [5, 6, 7, 9]) == 3          # all verified: i = gamma + 1
    assert A([5, 6, 7], [4, 6, 7, 9]) == 0          # first draft wrong, later matches do not count
    assert A([5, 6, 7], [5, 1, 7, 9]) == 1
    assert A([5, 6, 7], [5, 6, 1, 9]) == 2
    assert A([], [3]) == 0
    assert A([5, 6, 7], [0, 0, 0, 0], mode=O.ACCEPT_ALL) == 3
    a = A([5, 6, 7], [0, 0, 0, 0], mode=O.ACCEPT_HASH, mode_seed=5, seq=2, iteration=9)
    assert a == O.hashed_accept_length(5, 2, 9, 3) and 0 <= a <= 3


def test_commit_emits_prefix_plus_correction_and_rolls_back():
    shape = toy_shape()
    w = toy_weights(shape, seed=17)
    o = O.TandemOracle(shape, w)
    o.prefill(_prompt(shape, 4))
    drafts, _ = o.draft(3)
    targets, _, reps = o.verify(drafts)
    assert o.large_cache.length() == 3 + 4
    emitted = o.commit(1, drafts, targets, reps)
    assert emitted == [drafts[0], targets[1]]
    assert len(o.tokens) == 6 and o.large_cache.length() == 5 and o.derived.length() == 5


def test_hash_mode_still_emits_valid_lengths_and_counts_runs():
    shape = toy_shape()
    w = toy_weights(shape, seed=19)
    prompts = [list(p) for p in synth.make_prompts(3, [4, 7, 2], shape.large.vocab, 5)]
    toks, accs, runs = O.generate_batch(shape, w, prompts, 3, 10, mode=O.ACCEPT_HASH, mode_seed=77)
    assert [len(t) for t in toks] == [10, 10, 10]
    assert accs[0] != accs[1]                      # the hash depends on the sequence index
    for a, (nl, ns) in zip(accs, runs):
        assert nl == len(a) and ns == 3 * len(a)   # one large run and gamma small runs per iteration
        assert sum(x + 1 for x in a) >= 10 > sum(x + 1 for x in a[:-1])


# ------------------------------------------------------------------------------------------------
# Stand-alone Tandem variants (Section 3 "Inference"; Figures 2 and 3)
# ------------------------------------------------------------------------------------------------

def test_representation_only_cached_equals_brute_force_figure3():
    for kind, gamma, new in ((synth.FF_TANDEM_LINEAR, 2, 9), (synth.FF_TANDEM_MLP, 3, 8), (synth.FF_TANDEM_LINEAR, 1, 4)):
        shape = toy_shape(kind=kind, hidden=12 if kind else 0)
        w = toy_weights(shape, seed=40 + gamma)
        prompt = _prompt(shape, 5, seed=gamma)
        got = O.TandemOracle(shape, w).generate_representation_only(prompt, gamma, new)
        assert got == O.standalone_tandem_representation_only(shape, w, prompt, gamma, new)
        assert len(got) == new
    # it is neither the large model's greedy decoding nor the free-token variant
    assert got != O.plain_greedy(shape, w, prompt, new)


def test_representation_only_schedule_matches_figure3_for_three_blocks():
    shape = toy_shape()
    w = toy_weights(shape, seed=1)
    o = O.TandemOracle(shape, w)
    o.prefill(_prompt(shape, 8))
    for _ in range(3):
        o.step_representation_only(2)
    assert o.schedule == _read_schedule("fig3_schedule_three_blocks_gamma2.txt")
    assert (o.n_large_runs, o.n_small_runs) == (3, 6)
    assert o.large_cache.length() == o.derived.length() == len(o.tokens) - 1 and o.own.length() == 0


def _derived_boundaries(schedule):
    """For every small-model run: (its position, number of positions the large model had read before it)."""
    seen, out = 0, []
    for model, positions in schedule:
        if model == "L":
            seen = max(seen, positions[-1] + 1)
        else:
            out.append((positions[0], seen))
    return out


def test_both_variants_agree_on_which_positions_are_large_derived():
    """Whenever the small model runs at position p inside a block that starts at position s, the large model has
    read exactly positions 0..s-1 — with and without the free token (the training bullets of Section 3)."""
    shape = toy_shape()
    w = toy_weights(shape, seed=3)
    for gamma in (1, 2, 4):
        a, b = O.TandemOracle(shape, w), O.TandemOracle(shape, w)
        a.prefill(_prompt(shape, 6)); b.prefill(_prompt(shape, 6))
        for _ in range(3):
            a.step_representation_only(gamma)
            b.step(gamma, mode=O.ACCEPT_ALL)
        for sched, per_round in ((a.schedule, gamma), (b.schedule, gamma + 1)):
            runs = _derived_boundaries(sched)
            assert len(runs) == 3 * gamma
            for i, (pos, seen) in enumerate(runs):
                block_start = 5 + (i // gamma) * per_round
                assert seen == block_start and block_start <= pos < block_start + gamma


def test_self_tandem_representation_only_is_plain_greedy():
    """Small = large, identity FF_Tandem, l(j) = j: Eq. 2 is Eq. 1 for any boundary, so the small model's tokens are
    the large model's greedy tokens although the large model never predicts anything."""
    dims = synth.ModelDims(2, 32, 4, 64, 50, 64)
    shape = synth.self_tandem_shape(dims)
    w = synth.make_self_tandem_weights(shape, seed=6, std=0.35)
    prompt = _prompt(shape, 4, seed=9)
    got = O.TandemOracle(shape, w).generate_representation_only(prompt, 3, 10)
    assert got == O.plain_greedy(shape, w, prompt, 10)


def test_full_prompt_free_token_variant_matches_brute_force_and_figure2():
    shape = toy_shape(kind=synth.FF_TANDEM_MLP, hidden=12)
    w = toy_weights(shape, seed=23)
    prompt = _prompt(shape, 8, seed=2)
    o = O.TandemOracle(shape, w)
    got = o.generate_free_token_full_prompt(prompt, 2, 9)
    assert got == O.standalone_tandem_free_token_full_prompt(shape, w, prompt, 2, 9)
    assert got[0] == O.plain_greedy(shape, w, prompt, 1)[0]          # the first token is the large model's own
    # Figure 2's schedule: the golden file describes it from the 9-token prompt (query + free token) onwards
    fig2 = _read_schedule("fig2_schedule_gamma2.txt")
    assert o.schedule[: len(fig2)] == fig2
    # reading the whole prompt at once equals the Figure-3 prompt pass followed by a one-row large step
    a, b = O.TandemOracle(shape, w), O.TandemOracle(shape, w)
    first = a.prefill_all_tokens(prompt)
    b.prefill(prompt)
    assert b.step(0)["emitted"] == [first] and a.tokens == b.tokens
    for layer in range(shape.small.n_layers):
        assert np.allclose(np.stack(a.derived.k[layer]), np.stack(b.derived.k[layer]), atol=1e-10)


def test_grouped_query_models_keep_every_invariant():
    """Multi-query large model and grouped-query small model (Section 3): SPEED == plain greedy, block == single
    passes, cached == brute force, and keys/values have the narrower width."""
    L = synth.ModelDims(3, 32, 4, 64, 50, 64, n_kv_heads=1)
    S = synth.ModelDims(2, 24, 6, 48, 50, 64, n_kv_heads=2)
    shape = synth.make_shape(L, S, synth.FF_TANDEM_LINEAR, 0, (1, 3), synth.DTYPE_FP32)
    w = toy_weights(shape, seed=12)
    assert w["L.0.wk"].shape == (8, 32) and w["S.1.wv"].shape == (8, 24) and w["L.0.wq"].shape == (32, 32)
    prompt = _prompt(shape, 6, seed=4)
    o = O.TandemOracle(shape, w)
    got, accepts = o.generate(prompt, 3, 9)
    assert got == O.plain_greedy(shape, w, prompt, 9)
    assert o.large_cache.k[0][0].shape == (8,) and o.derived.k[0][0].shape == (8,)
    assert O.TandemOracle(shape, w).generate(prompt, 2, 7, mode=O.ACCEPT_ALL)[0] == O.standalone_tandem_free_token(shape, w, prompt, 2, 7)
    assert O.TandemOracle(shape, w).generate_representation_only(prompt, 2, 6) == \
        O.standalone_tandem_representation_only(shape, w, prompt, 2, 6)


# ------------------------------------------------------------------------------------------------
# Teacher-forced Tandem forward (Eq. 2 over a given sequence)
# ------------------------------------------------------------------------------------------------

def test_teacher_forced_forward_limits_and_cached_path():
    shape = toy_shape(kind=synth.FF_TANDEM_MLP, hidden=12)
    w = toy_weights(shape, seed=31)
    ids = _prompt(shape, 11, seed=6)
    small = O.Decoder(w, "S", shape.small.n_layers, shape.small.n_heads)
    # one block over the whole sequence: no large-derived context, a plain decoder (Eq. 1 with the small model's weights)
    assert np.allclose(O.teacher_forced_tandem_logits(shape, w, ids, 64), O.decoder_full_forward(small, ids)[1], atol=1e-10)
    for gamma in (1, 2, 3, 4):
        brute = O.teacher_forced_tandem_logits(shape, w, ids, gamma)
        cached = O.TandemOracle(shape, w).teacher_forced_logits(ids, gamma)
        assert brute.shape == (11, shape.small.vocab) and np.allclose(brute, cached, atol=1e-9)
        # positions of the first block see no large model at all
        assert np.allclose(brute[:gamma], O.decoder_full_forward(small, ids[:gamma])[1], atol=1e-10)
    assert np.abs(O.teacher_forced_tandem_logits(shape, w, ids, 2) - O.teacher_forced_tandem_logits(shape, w, ids, 3)).max() > 1e-3
    # self-tandem: Eq. 2 is Eq. 1 of the large model for any block length
    dims = synth.ModelDims(2, 32, 4, 64, 50, 64)
    st = synth.self_tandem_shape(dims)
    ws = synth.make_self_tandem_weights(st, seed=6, std=0.35)
    large = O.Decoder(ws, "L", 2, 4)
    assert np.allclose(O.teacher_forced_tandem_logits(st, ws, ids, 3), O.decoder_full_forward(large, ids)[1], atol=1e-9)


def test_next_token_scores_against_library_cross_entropy():
    rng = np.random.default_rng(2)
    logits = rng.normal(size=(6, 9)) * 3
    ids = [3, 1, 4, 1, 5, 8]
    nll, top = O.next_token_scores(logits, ids)
    want = torch.nn.functional.cross_entropy(torch.tensor(logits[:5]), torch.tensor(ids[1:]), reduction="none").numpy()
    assert np.allclose(nll, want, atol=1e-12) and top.tolist() == logits[:5].argmax(1).tolist()
    assert np.isclose(O.next_token_scores(np.zeros((2, 7)), [0, 3])[0][0], np.log(7.0))
