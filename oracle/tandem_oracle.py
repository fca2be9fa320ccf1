"""CPU checker for greedy Tandem + SPEED decoding (Tandem Transformers, arXiv 2402.08644).

THIS IS TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  It is a plain, slow, fp64 numpy restatement of the
paper's equations, used by the tests, by the smoke check and by the benchmark's CPU-baseline leg to
decide whether the CUDA library computes the right thing.  It shares no code with the CUDA path and
must never be imported by it.

What it computes, in the paper's notation (x = large-model representations, y = small-model
representations, y_hat = projected large representations, gamma = block length):

  * Eq. 1 (Section 3, "Standard (Decoder) Transformer"): causal decoder, both as a brute-force
    whole-sequence forward (no cache) and as an incremental pass over a key/value cache.
  * Eq. 2 (Section 3, "Tandem Transformer"): y_hat = FF_Tandem(x^(l(j))); small layer j attends the
    projected large representations for positions the large model has processed and its own
    representations for the rest.  Brute force and cached.
  * Section 3, "Inference", Figures 2 and 3: prompt handling (large model reads the prompt without
    its last token), block-mode large pass, the free token.
  * Section 3.1: draft gamma tokens, verify the block, first mismatch, take the large model's token
    there, continue with the large model's representations of all previous tokens.

Readings taken where the paper is silent or inconsistent:
  R1  Boundary.  Eq. 2 prints k = floor(i/gamma)*gamma, which would let a token at a multiple of gamma
      attend the large model's representation of itself.  The training bullets of Section 3 and
      Figure 3 say that the current block, including the query token, uses the small model's own
      keys/values.  Here the boundary is simply the number of positions the large model has processed;
      a query always sees its own key/value.  Inside SPEED the boundary is ragged (Section 3.1: "all
      the previous tokens").
  R2  x^(l) is the residual stream after l large layers; l = 0 is the embedding output.
  R3  y_hat replaces y as the *layer input* at that position: K = LN1_S(y_hat) Wk^T, V likewise.
  R17 Multi-query / grouped-query attention ("whether the attention is multi-head or multi-query", Section 3):
      n_kv_heads key/value heads of the same head size; query head h reads key/value head
      h // (n_heads / n_kv_heads); W_k and W_v map d_model to n_kv_heads * d_head.  Either model, independently.
  R18 Sampling inside SPEED (Section 3.1 builds on the SPEED / speculative-decoding framework and its
      experiments use sampled responses, num-samples 1 and 4).  The rule of that framework: draft d_r is drawn
      from the small model's distribution q_r = softmax(logits_S / T_S); it is kept with probability
      min(1, p_r(d_r) / q_r(d_r)), p_r = softmax(logits_L / T_L); at the first rejection the token is redrawn
      from the normalised positive part of p_r - q_r; if all gamma drafts are kept, one more token is drawn from
      p_{gamma+1}.  Every draw uses one uniform variate from a counter-based generator keyed by
      (seed, sequence, iteration, slot): slots 0..gamma-1 draw the drafts, 16+r tests draft r, 48 redraws.
      A draw from weights w with variate u returns the first index whose running sum exceeds u * sum(w).
  R19 Adaptive block length (Section 3.1 "Adaptive Block Length", Section 4: tau = 0.8).  After every draft the
      router looks at the small model's distribution q = softmax(logits_S) for that draft: features
      [entropy of q (nats), the k largest probabilities in descending order (lowest id first on ties), the small
      model's embedding rows of those k tokens], a two-layer perceptron hidden = relu(W1 x + b1),
      s = sigmoid(w2 . hidden + b2) = predicted probability that the large model disagrees (what the paper trains
      it to predict).  The small model goes on drafting while 1 - s >= tau and fewer than gamma_max drafts exist;
      otherwise the drafts made so far (at least one) are verified as a block of that length.  k, the hidden width
      and the weights are inputs (the paper gives none); decisions are per sequence.
  R20 Teacher-forced Tandem forward (Eq. 2 over a whole given sequence, as in training and in the accuracy /
      cross-entropy evaluation of Section 4.1): blocks of gamma positions anchored at position 0; the token at
      position i is the small model's input at i, its context holds the projected large representations of
      positions below the block's start floor(i / gamma) * gamma and the small model's own representations from
      there to i (R1); its logits predict the token at i + 1.  Per position: the negative log-likelihood of the
      true next token (natural log) and the arg-max.
  R4  Pre-LayerNorm blocks (gain and bias, eps 1e-5, biased variance), exact-erf GELU, no linear
      biases, learned absolute position embeddings, untied output head.
  R6  FF_Tandem MLP variant: hidden width given by the shape, GELU, no biases.
  R7  The large model reads prompt[0..P-2]; prompt[P-1] is the pending token the small model starts from.
  R8  "Deemed incorrect" = the draft differs from the arg-max of the large model's logits (greedy).
  R9  Arg-max ties go to the lowest token id.  The decision is taken on logits rounded to float32,
      the precision in which the CUDA path holds its logits.
  R10 The verify pass has gamma+1 rows (pending token + gamma drafts) and can emit up to gamma+1 tokens.
  R11 Accept lengths are per sequence; sequences are independent.
  R12 A sequence stops after exactly max_new tokens; surplus tokens of the last iteration are dropped.
  R13 accept_mode 1 keeps all gamma drafts whatever the comparison says (equal to stand-alone Tandem
      with the free token, Figure 2); accept_mode 2 takes a pseudo-random accept length from a
      counter-based hash (test only).
  R16 Stand-alone Tandem (Section 3, "Inference", the two configurations; Figures 2 and 3).
      "Representation Generation Only": per round the small model appends gamma tokens starting from the
      pending token, then the large model reads the pending token and the first gamma-1 new tokens as one
      block of gamma rows, without an output head; the last new token becomes pending (Figure 3, right).
      "Representation Generation + Token Prediction" for the prompt too (Figure 2, left): the large model
      reads all P prompt tokens and its prediction is the first response token, which becomes pending.
      A response that is not a whole number of blocks long drops the surplus of the last round (as R12).

Pins: every function here is pinned by tests/test_oracle_*.py (library decoder layer, both FF_Tandem
branches against library modules and closed forms, brute force vs cache, the stand-alone variants against
brute-force loops, Figure 3's schedule and the self-tandem collapse, SPEED == plain greedy, self-tandem, block == single-token passes, schedule fixtures from
Figures 2 and 3, hand-made accept cases).  The absolute logit values of a random-init *Tandem* pair
have no value printed in the paper to compare with: for those, parity unpinned beyond the invariants.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
from scipy.special import erf

LN_EPS = 1e-5

ACCEPT_NATURAL = 0
ACCEPT_ALL = 1
ACCEPT_HASH = 2


# ----------------------------------------------------------------------------------------------
# Elementary pieces (Eq. 1's Atn and FF, written out)
# ----------------------------------------------------------------------------------------------

def layer_norm(x: np.ndarray, gain: np.ndarray, bias: np.ndarray) -> np.ndarray:
    """LayerNorm over the last axis: (x - mean) / sqrt(var + eps) * gain + bias, biased variance."""
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + LN_EPS) * gain + bias


def gelu(x: np.ndarray) -> np.ndarray:
    """Exact GELU: x * Phi(x)."""
    return 0.5 * x * (1.0 + erf(x / math.sqrt(2.0)))


def softmax(s: np.ndarray) -> np.ndarray:
    """Softmax over the last axis."""
    e = np.exp(s - s.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def attend(q: np.ndarray, K: np.ndarray, V: np.ndarray, n_heads: int, n_kv_heads: Optional[int] = None) -> np.ndarray:
    """Multi-head attention of ONE query q[d] over a context K[n][d_kv], V[n][d_kv]: per head,
    softmax(q_h . k_g / sqrt(d_h)) weighted sum of v_g; heads concatenated.  With fewer key/value heads than
    query heads (multi-query / grouped-query attention, which Section 3 allows for either model), query head h
    reads key/value head g = h // (n_heads / n_kv_heads); by default g = h and d_kv = d."""
    d = q.shape[0]
    dh = d // n_heads
    kv = n_heads if n_kv_heads is None else n_kv_heads
    group = n_heads // kv
    out = np.empty(d, dtype=q.dtype)
    for h in range(n_heads):
        sl = slice(h * dh, (h + 1) * dh)
        g = h // group
        sg = slice(g * dh, (g + 1) * dh)
        scores = K[:, sg] @ q[sl] / math.sqrt(dh)
        out[sl] = softmax(scores) @ V[:, sg]
    return out


def argmax_decision(logits: np.ndarray) -> int:
    """Greedy token: arg-max of the float32-rounded logits, lowest id on ties (R9)."""
    return int(np.argmax(logits.astype(np.float32)))


def splitmix64(x: int) -> int:
    """One round of the public splitmix64 mixing function on a 64-bit counter."""
    m = 0xFFFFFFFFFFFFFFFF
    x = (x + 0x9E3779B97F4A7C15) & m
    z = x
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & m
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & m
    return z ^ (z >> 31)


def hashed_accept_length(mode_seed: int, seq: int, iteration: int, gamma: int) -> int:
    """accept_mode 2 (R13): a = mix(mix(mix(seed) ^ seq) ^ iteration) mod (gamma + 1)."""
    return splitmix64(splitmix64(splitmix64(mode_seed) ^ seq) ^ iteration) % (gamma + 1)


# ----------------------------------------------------------------------------------------------
# Sampling (R18)
# ----------------------------------------------------------------------------------------------

SLOT_ACCEPT = 16      # slot of the variate that tests draft r: SLOT_ACCEPT + r
SLOT_REDRAW = 48      # slot of the variate that redraws (or draws the extra token)


def uniform_variate(seed: int, seq: int, iteration: int, slot: int) -> float:
    """Counter-based uniform in [0, 1) with 24 bits: the top 24 bits of
    mix(mix(mix(mix(seed) ^ seq) ^ iteration) ^ slot), exactly representable in float32 and float64."""
    x = splitmix64(splitmix64(splitmix64(splitmix64(seed) ^ seq) ^ iteration) ^ slot)
    return (x >> 40) / float(1 << 24)


def temperature_softmax(logits: np.ndarray, temperature: float) -> np.ndarray:
    """softmax(logits / T) over the last axis."""
    return softmax(np.asarray(logits, dtype=np.float64) / temperature)


def draw_index(weights: np.ndarray, u: float) -> int:
    """Inverse-CDF draw from non-negative (unnormalised) weights: the first index whose running sum exceeds
    u * sum(weights); the last index with a positive weight if rounding leaves none."""
    c = np.cumsum(weights)
    target = u * c[-1]
    for i in range(len(c)):
        if c[i] > target:
            return i
    return int(np.nonzero(weights > 0)[0][-1])


def accept_probability(p: np.ndarray, q: np.ndarray, token: int) -> float:
    """Probability of keeping a draft drawn from q when the target distribution is p: min(1, p / q)."""
    return min(1.0, p[token] / q[token]) if q[token] > 0 else 1.0


def residual_weights(p: np.ndarray, q: np.ndarray) -> np.ndarray:
    """Unnormalised distribution of the redrawn token after a rejection: the positive part of p - q."""
    return np.maximum(p - q, 0.0)


# ----------------------------------------------------------------------------------------------
# Router of the adaptive block length (R19)
# ----------------------------------------------------------------------------------------------

class Router:
    """Two-layer perceptron on [entropy, top-k probabilities, top-k embedding rows] (R19)."""

    def __init__(self, k: int, w1: np.ndarray, b1: np.ndarray, w2: np.ndarray, b2: float, tau: float, dtype=np.float64):
        self.k, self.tau = int(k), float(tau)
        self.w1, self.b1 = np.asarray(w1, dtype=dtype), np.asarray(b1, dtype=dtype)
        self.w2, self.b2 = np.asarray(w2, dtype=dtype), float(b2)

    def features(self, logits: np.ndarray, emb: np.ndarray) -> np.ndarray:
        q = softmax(np.asarray(logits, dtype=np.float64))
        nz = q[q > 0]
        entropy = -(nz * np.log(nz)).sum()
        top = np.argsort(-q, kind="stable")[: self.k]          # descending probability, lowest id first on ties
        return np.concatenate([[entropy], q[top]] + [emb[t] for t in top])

    def disagreement(self, logits: np.ndarray, emb: np.ndarray) -> float:
        x = self.features(logits, emb)
        hidden = np.maximum(self.w1 @ x + self.b1, 0.0)
        return float(1.0 / (1.0 + np.exp(-(self.w2 @ hidden + self.b2))))

    def keep_drafting(self, logits: np.ndarray, emb: np.ndarray) -> Tuple[bool, float]:
        """(whether the small model may go on, the confidence 1 - s compared with tau)."""
        conf = 1.0 - self.disagreement(logits, emb)
        return conf >= self.tau, conf


# ----------------------------------------------------------------------------------------------
# Weights
# ----------------------------------------------------------------------------------------------

class Decoder:
    """Weights of one decoder (prefix 'L' or 'S' in the weight dict), cast to the compute dtype."""

    def __init__(self, weights: Dict[str, np.ndarray], prefix: str, n_layers: int, n_heads: int,
                 dtype=np.float64, n_kv_heads: Optional[int] = None):
        g = lambda name: np.asarray(weights[f"{prefix}.{name}"], dtype=dtype)
        self.n_layers, self.n_heads = n_layers, n_heads
        self.n_kv_heads = n_heads if not n_kv_heads else n_kv_heads
        self.emb, self.pos = g("emb"), g("pos")
        self.layers = []
        for l in range(n_layers):
            self.layers.append({k: g(f"{l}.{k}") for k in
                                ("ln1_g", "ln1_b", "wq", "wk", "wv", "wo", "ln2_g", "ln2_b", "w1", "w2")})
        self.lnf_g, self.lnf_b, self.w_out = g("lnf_g"), g("lnf_b"), g("w_out")

    def embed(self, token: int, index: int) -> np.ndarray:
        """x^(0) = Emb(t) + Pos(index)   (Eq. 1, R4)."""
        return self.emb[token] + self.pos[index]

    def feed_forward(self, l: int, h: np.ndarray) -> np.ndarray:
        """h + GELU(LN2(h) W1^T) W2^T   (the FF of Eq. 1, R4)."""
        p = self.layers[l]
        return h + gelu(layer_norm(h, p["ln2_g"], p["ln2_b"]) @ p["w1"].T) @ p["w2"].T

    def logits(self, h: np.ndarray) -> np.ndarray:
        return layer_norm(h, self.lnf_g, self.lnf_b) @ self.w_out.T


class TandemProjection:
    """FF_Tandem^(j) for every small layer j (Eq. 2, first line)."""

    def __init__(self, weights: Dict[str, np.ndarray], n_small_layers: int, kind: int, dtype=np.float64):
        self.kind = kind
        self.w = []
        for j in range(n_small_layers):
            if kind == 0:
                self.w.append((np.asarray(weights[f"T.{j}.w_t"], dtype=dtype),))
            else:
                self.w.append((np.asarray(weights[f"T.{j}.w_t1"], dtype=dtype),
                               np.asarray(weights[f"T.{j}.w_t2"], dtype=dtype)))

    def __call__(self, j: int, x: np.ndarray) -> np.ndarray:
        if self.kind == 0:
            return x @ self.w[j][0].T
        return gelu(x @ self.w[j][0].T) @ self.w[j][1].T


# ----------------------------------------------------------------------------------------------
# Brute force: whole-sequence forwards with no cache (the plain definitions)
# ----------------------------------------------------------------------------------------------

def decoder_full_forward(dec: Decoder, ids: Sequence[int]) -> Tuple[List[np.ndarray], np.ndarray]:
    """Eq. 1 over a whole sequence, recomputing everything.  Returns ([x^(0), ..., x^(L)], logits),
    each x^(l) of shape [S][d], logits [S][V]."""
    S = len(ids)
    h = np.stack([dec.embed(int(t), i) for i, t in enumerate(ids)]) if S else np.zeros((0, dec.emb.shape[1]))
    reps = [h]
    for l in range(dec.n_layers):
        p = dec.layers[l]
        a = layer_norm(h, p["ln1_g"], p["ln1_b"])
        q, k, v = a @ p["wq"].T, a @ p["wk"].T, a @ p["wv"].T
        o = np.stack([attend(q[i], k[: i + 1], v[: i + 1], dec.n_heads, dec.n_kv_heads) for i in range(S)]) if S else h
        h = h + o @ p["wo"].T
        h = dec.feed_forward(l, h)
        reps.append(h)
    return reps, dec.logits(h)


def tandem_small_full_forward(small: Decoder, proj: TandemProjection, layer_map: Sequence[int],
                              large_reps: List[np.ndarray], boundary: int, ids: Sequence[int]) -> np.ndarray:
    """Eq. 2 by brute force for positions boundary .. len(ids)-1 (the ones the small model runs on).

    `large_reps[l]` holds x^(l) for at least the first `boundary` positions.  For small layer j the
    context representation at position p is y_hat_p = FF_Tandem^(j)(x_p^(l(j))) if p < boundary, else
    the small model's own y_p^(j) (R1); keys and values are LN1_S(context) Wk^T / Wv^T (R3).
    Returns the small model's logits for positions boundary .. len(ids)-1."""
    S = len(ids)
    own = list(range(boundary, S))
    y = np.stack([small.embed(int(ids[p]), p) for p in own])
    for j in range(small.n_layers):
        p_ = small.layers[j]
        if boundary > 0:
            ctx = np.concatenate([proj(j, large_reps[layer_map[j]][:boundary]), y], axis=0)
        else:
            ctx = y
        a_ctx = layer_norm(ctx, p_["ln1_g"], p_["ln1_b"])
        k, v = a_ctx @ p_["wk"].T, a_ctx @ p_["wv"].T
        q = layer_norm(y, p_["ln1_g"], p_["ln1_b"]) @ p_["wq"].T
        o = np.stack([attend(q[r], k[: p + 1], v[: p + 1], small.n_heads, small.n_kv_heads) for r, p in enumerate(own)])
        y = y + o @ p_["wo"].T
        y = small.feed_forward(j, y)
    return small.logits(y)


# ----------------------------------------------------------------------------------------------
# Incremental passes over key/value caches
# ----------------------------------------------------------------------------------------------

class KVCache:
    """Per layer, keys and values by absolute position.  `truncate` implements rollback."""

    def __init__(self, n_layers: int):
        self.k: List[List[np.ndarray]] = [[] for _ in range(n_layers)]
        self.v: List[List[np.ndarray]] = [[] for _ in range(n_layers)]

    def length(self, layer: int = 0) -> int:
        return len(self.k[layer])

    def append(self, layer: int, k: np.ndarray, v: np.ndarray) -> None:
        self.k[layer].append(k)
        self.v[layer].append(v)

    def truncate(self, n: int) -> None:
        for l in range(len(self.k)):
            del self.k[l][n:]
            del self.v[l][n:]


def large_block_pass(dec: Decoder, cache: KVCache, tokens: Sequence[int], start: int
                     ) -> Tuple[List[np.ndarray], np.ndarray]:
    """Block mode (Section 3, "Inference"; Section 3.1): the large model processes `tokens` at
    positions start, start+1, ... together.  Row r attends cache positions 0 .. start+r (causal
    inside the block).  Appends the rows' keys/values to the cache.
    Returns ([x^(0), ..., x^(L)] each [rows][d], logits [rows][V])."""
    assert cache.length() == start
    R = len(tokens)
    h = np.stack([dec.embed(int(t), start + r) for r, t in enumerate(tokens)])
    reps = [h]
    for l in range(dec.n_layers):
        p = dec.layers[l]
        a = layer_norm(h, p["ln1_g"], p["ln1_b"])
        q, k, v = a @ p["wq"].T, a @ p["wk"].T, a @ p["wv"].T
        for r in range(R):
            cache.append(l, k[r], v[r])
        K, V = np.stack(cache.k[l]), np.stack(cache.v[l])
        o = np.stack([attend(q[r], K[: start + r + 1], V[: start + r + 1], dec.n_heads, dec.n_kv_heads) for r in range(R)])
        h = h + o @ p["wo"].T
        h = dec.feed_forward(l, h)
        reps.append(h)
    return reps, dec.logits(h)


class TandemOracle:
    """Greedy Tandem + SPEED for ONE sequence, step by step (Section 3.1)."""

    def __init__(self, shape, weights: Dict[str, np.ndarray], dtype=np.float64):
        self.shape = shape
        self.large = Decoder(weights, "L", shape.large.n_layers, shape.large.n_heads, dtype, shape.large.kv_heads)
        self.small = Decoder(weights, "S", shape.small.n_layers, shape.small.n_heads, dtype, shape.small.kv_heads)
        self.proj = TandemProjection(weights, shape.small.n_layers, shape.ff_tandem_kind, dtype)
        self.layer_map = list(shape.layer_map)
        self.tokens: List[int] = []           # committed tokens c[0..n-1]; c[n-1] is pending
        self.large_cache = KVCache(shape.large.n_layers)
        self.derived = KVCache(shape.small.n_layers)   # large-derived region of the small model's K/V
        self.own = KVCache(shape.small.n_layers)       # the small model's own K/V for the current block
        self.n_large_runs = 0
        self.n_small_runs = 0
        self.iteration = 0
        self.schedule: List[Tuple[str, List[int]]] = []   # (model, positions) per run, for Figures 2/3

    # --- Eq. 2, first line, then the small layer's key/value maps (R3) --------------------------
    def _project_rows(self, reps: List[np.ndarray], rows: range) -> None:
        for j in range(self.small.n_layers):
            p = self.small.layers[j]
            for r in rows:
                y_hat = self.proj(j, reps[self.layer_map[j]][r])
                a = layer_norm(y_hat, p["ln1_g"], p["ln1_b"])
                self.derived.append(j, a @ p["wk"].T, a @ p["wv"].T)

    # --- prompt (Section 3 "Inference"; Figure 3; R7) --------------------------------------------
    def prefill(self, prompt: Sequence[int]) -> None:
        assert len(prompt) >= 1
        self.tokens = [int(t) for t in prompt]
        m = len(prompt) - 1
        if m > 0:
            reps, _ = large_block_pass(self.large, self.large_cache, self.tokens[:m], 0)
            self._project_rows(reps, range(m))
            self.schedule.append(("L", list(range(m))))

    def prefill_all_tokens(self, prompt: Sequence[int]) -> int:
        """Figure 2, left (R16): the large model reads the whole prompt; its prediction for the next position is
        the first response token, which is appended and becomes the pending token.  Returns that token."""
        assert len(prompt) >= 1
        self.tokens = [int(t) for t in prompt]
        P = len(prompt)
        reps, logits = large_block_pass(self.large, self.large_cache, self.tokens, 0)
        self._project_rows(reps, range(P))
        self.n_large_runs += 1
        self.schedule.append(("L", list(range(P))))
        first = argmax_decision(logits[P - 1])
        self.tokens.append(first)
        return first

    def step_representation_only(self, gamma: int, forced: Optional[Sequence[int]] = None) -> dict:
        """One round of stand-alone Tandem without the free token (Figure 3, R16): gamma small-model steps from the
        pending token; all gamma tokens are kept; the large model then reads the pending token and the first
        gamma-1 new tokens as one block (no output head) and those rows are projected for the small model."""
        assert gamma >= 1
        n = len(self.tokens)
        drafts, s_logits = self.draft(gamma, forced)
        kept = [int(t) for t in (forced if forced is not None else drafts)]
        rows = [self.tokens[-1]] + kept[:-1]
        reps, _ = large_block_pass(self.large, self.large_cache, rows, n - 1)
        self.n_large_runs += 1
        self.schedule.append(("L", list(range(n - 1, n - 1 + gamma))))
        self.tokens += kept
        self._project_rows(reps, range(gamma))
        self.own.truncate(0)
        self.iteration += 1
        return {"drafts": drafts, "emitted": kept, "small_logits": s_logits, "n_committed": len(self.tokens), "reps": reps}

    def teacher_forced_logits(self, ids: Sequence[int], gamma: int) -> np.ndarray:
        """The same logits as `teacher_forced_tandem_logits` through the caches: the first token is the pending
        token of an empty prompt pass, then representation-only rounds fed the given tokens (R20)."""
        seq = [int(t) for t in ids]
        self.prefill(seq[:1])
        out = []
        while len(out) < len(seq):
            g = min(gamma, len(seq) - len(out))
            nxt = seq[len(out) + 1: len(out) + 1 + g]
            forced = nxt + [0] * (g - len(nxt))          # the token after the last position does not exist: any id, never used
            out += self.step_representation_only(g, forced=forced)["small_logits"]
        return np.stack(out)

    def generate_representation_only(self, prompt: Sequence[int], gamma: int, max_new: int) -> List[int]:
        self.prefill(prompt)
        P = len(prompt)
        while len(self.tokens) - P < max_new:
            self.step_representation_only(gamma)
        return self.tokens[P:P + max_new]

    def generate_free_token_full_prompt(self, prompt: Sequence[int], gamma: int, max_new: int) -> List[int]:
        """Figure 2 as drawn: the first response token comes from the large model reading the whole prompt, then
        rounds of gamma small-model tokens followed by one large-model token (accept-all rounds)."""
        self.prefill_all_tokens(prompt)
        P = len(prompt)
        while len(self.tokens) - P < max_new:
            self.step(gamma, ACCEPT_ALL)
        return self.tokens[P:P + max_new]

    # --- one token through the small model over the mixed context (Eq. 2, lines 2-3) --------------
    def _small_step(self, token: int, index: int) -> np.ndarray:
        sm = self.small
        y = sm.embed(token, index)
        for j in range(sm.n_layers):
            p = sm.layers[j]
            a = layer_norm(y, p["ln1_g"], p["ln1_b"])
            self.own.append(j, a @ p["wk"].T, a @ p["wv"].T)
            K = np.stack(self.derived.k[j] + self.own.k[j])
            V = np.stack(self.derived.v[j] + self.own.v[j])
            assert K.shape[0] == index + 1
            y = y + attend(a @ p["wq"].T, K, V, sm.n_heads, sm.n_kv_heads) @ p["wo"].T
            y = sm.feed_forward(j, y)
        self.n_small_runs += 1
        self.schedule.append(("S", [index]))
        return sm.logits(y)

    def draft(self, gamma: int, forced: Optional[Sequence[int]] = None) -> Tuple[List[int], List[np.ndarray]]:
        """gamma autoregressive small-model steps starting from the pending token (Section 3.1).
        Returns (own arg-max drafts, logits per step).  If `forced` is given, step s+1 is fed
        forced[s] instead of its own arg-max (teacher forcing, used by replay tests)."""
        n = len(self.tokens)
        assert self.derived.length() == n - 1 and self.own.length() == 0
        u = self.tokens[-1]
        drafts, all_logits = [], []
        for s in range(gamma):
            lg = self._small_step(u, n - 1 + s)
            d = argmax_decision(lg)
            drafts.append(d)
            all_logits.append(lg)
            u = int(forced[s]) if forced is not None else d
        return drafts, all_logits

    def verify(self, drafts: Sequence[int]) -> Tuple[List[int], np.ndarray, List[np.ndarray]]:
        """The large model processes the pending token and the drafts as one block (R10).
        Returns (targets g[0..gamma], logits [gamma+1][V], reps)."""
        n = len(self.tokens)
        rows = [self.tokens[-1]] + [int(d) for d in drafts]
        reps, logits = large_block_pass(self.large, self.large_cache, rows, n - 1)
        self.n_large_runs += 1
        self.schedule.append(("L", list(range(n - 1, n - 1 + len(rows)))))
        return [argmax_decision(logits[r]) for r in range(len(rows))], logits, reps

    @staticmethod
    def accept_length(drafts: Sequence[int], targets: Sequence[int], mode: int = ACCEPT_NATURAL,
                      mode_seed: int = 0, seq: int = 0, iteration: int = 0) -> int:
        """Number of drafts kept: the length of the longest prefix on which draft r equals the large
        model's token for the same position (Section 3.1, R8); or gamma (mode 1); or hashed (mode 2)."""
        gamma = len(drafts)
        if mode == ACCEPT_ALL:
            return gamma
        if mode == ACCEPT_HASH:
            return hashed_accept_length(mode_seed, seq, iteration, gamma)
        a = 0
        while a < gamma and int(drafts[a]) == int(targets[a]):
            a += 1
        return a

    def commit(self, a: int, drafts: Sequence[int], targets: Sequence[int], reps: List[np.ndarray]) -> List[int]:
        """Keep drafts[0..a-1], then the large model's token for the next position; roll the large
        cache back to the kept rows; project the kept rows for the small model; drop the small
        model's own keys/values (Section 3.1)."""
        n = len(self.tokens)
        emitted = [int(d) for d in drafts[:a]] + [int(targets[a])]
        self.tokens += emitted
        self.large_cache.truncate(n + a)            # rows 0..a stay: positions n-1 .. n-1+a
        self._project_rows(reps, range(a + 1))
        self.own.truncate(0)
        self.iteration += 1
        return emitted

    def step_sampling(self, gamma: int, temp_large: float, temp_small: float, seed: int, seq: int = 0,
                      forced: Optional[dict] = None) -> dict:
        """One sampled Tandem + SPEED iteration (R18).  Returns the drafts, the accept length, the token emitted
        after the kept drafts, and the distributions / variates behind every decision.  With `forced`
        ({"drafts", "accept_len", "final"}: another implementation's choices) those choices are followed instead
        of this function's own, so that the caller can check each of them against the returned records."""
        n = len(self.tokens)
        it = self.iteration
        assert self.derived.length() == n - 1 and self.own.length() == 0
        u_in = self.tokens[-1]
        drafts, own_drafts, q_list, s_logits = [], [], [], []
        for s_ in range(gamma):
            lg = self._small_step(u_in, n - 1 + s_)
            q = temperature_softmax(lg, temp_small)
            d = draw_index(q, uniform_variate(seed, seq, it, s_))
            own_drafts.append(d)
            u_in = int(forced["drafts"][s_]) if forced is not None else d
            drafts.append(u_in)
            q_list.append(q)
            s_logits.append(lg)
        rows = [self.tokens[-1]] + drafts
        reps, l_logits = large_block_pass(self.large, self.large_cache, rows, n - 1)
        self.n_large_runs += 1
        p_list = [temperature_softmax(l_logits[r], temp_large) for r in range(gamma + 1)]
        ratios = [accept_probability(p_list[r], q_list[r], drafts[r]) for r in range(gamma)]
        tests = [uniform_variate(seed, seq, it, SLOT_ACCEPT + r) for r in range(gamma)]
        own_a = 0
        while own_a < gamma and tests[own_a] < ratios[own_a]:
            own_a += 1
        a = int(forced["accept_len"]) if forced is not None else own_a
        final_w = residual_weights(p_list[a], q_list[a]) if a < gamma else p_list[gamma]
        u_final = uniform_variate(seed, seq, it, SLOT_REDRAW)
        own_final = draw_index(final_w, u_final)
        final = int(forced["final"]) if forced is not None else own_final
        emitted = drafts[:a] + [final]
        self.tokens += emitted
        self.large_cache.truncate(n + a)
        self._project_rows(reps, range(a + 1))
        self.own.truncate(0)
        self.iteration += 1
        return {"drafts": drafts, "own_drafts": own_drafts, "accept_len": a, "own_accept_len": own_a, "final": final,
                "own_final": own_final, "emitted": emitted, "q": q_list, "p": p_list, "ratios": ratios, "tests": tests,
                "final_weights": final_w, "u_final": u_final, "small_logits": s_logits, "large_logits": l_logits,
                "n_committed": len(self.tokens)}

    def generate_sampling(self, prompt: Sequence[int], gamma: int, max_new: int, temp_large: float, temp_small: float,
                          seed: int, seq: int = 0) -> Tuple[List[int], List[int]]:
        self.prefill(prompt)
        P = len(prompt)
        accepts = []
        while len(self.tokens) - P < max_new:
            accepts.append(self.step_sampling(gamma, temp_large, temp_small, seed, seq)["accept_len"])
        return self.tokens[P:P + max_new], accepts

    def step_adaptive(self, gamma_max: int, router: "Router", forced_len: Optional[int] = None,
                      forced_drafts: Optional[Sequence[int]] = None) -> dict:
        """One greedy Tandem + SPEED iteration whose block length the router chooses (R19): draft, ask the router,
        stop at its first "verify now" or at gamma_max, then verify exactly the drafts made.  With `forced_len` /
        `forced_drafts` (another implementation's block length and draft ids) those are followed; the router's
        confidences are returned either way so that the caller can check each decision."""
        n = len(self.tokens)
        assert self.derived.length() == n - 1 and self.own.length() == 0 and gamma_max >= 1
        u = self.tokens[-1]
        drafts, own_drafts, s_logits, confs = [], [], [], []
        own_len = None
        s_ = 0
        while True:
            lg = self._small_step(u, n - 1 + s_)
            d = argmax_decision(lg)
            own_drafts.append(d)
            u = int(forced_drafts[s_]) if forced_drafts is not None else d
            drafts.append(u)
            s_logits.append(lg)
            go_on, conf = router.keep_drafting(lg, self.small.emb)
            confs.append(conf)
            s_ += 1
            if own_len is None and (not go_on or s_ == gamma_max):
                own_len = s_
            if (forced_len is None and own_len is not None) or (forced_len is not None and s_ == forced_len):
                break
        targets, l_logits, reps = self.verify(drafts)
        a = self.accept_length(drafts, targets)
        emitted = self.commit(a, drafts, targets, reps)
        return {"drafts": drafts, "own_drafts": own_drafts, "block_len": len(drafts), "own_block_len": own_len,
                "confidences": confs, "targets": targets, "accept_len": a, "emitted": emitted, "small_logits": s_logits,
                "large_logits": l_logits, "n_committed": len(self.tokens)}

    def generate_adaptive(self, prompt: Sequence[int], gamma_max: int, max_new: int, router: "Router") -> Tuple[List[int], List[int]]:
        """Full response with the adaptive block length; returns (tokens, block length of every iteration)."""
        self.prefill(prompt)
        P = len(prompt)
        lens = []
        while len(self.tokens) - P < max_new:
            lens.append(self.step_adaptive(gamma_max, router)["block_len"])
        return self.tokens[P:P + max_new], lens

    def step(self, gamma: int, mode: int = ACCEPT_NATURAL, mode_seed: int = 0, seq: int = 0) -> dict:
        drafts, s_logits = self.draft(gamma)
        targets, l_logits, reps = self.verify(drafts)
        a = self.accept_length(drafts, targets, mode, mode_seed, seq, self.iteration)
        emitted = self.commit(a, drafts, targets, reps)
        return {"drafts": drafts, "targets": targets, "accept_len": a, "emitted": emitted,
                "small_logits": s_logits, "large_logits": l_logits, "n_committed": len(self.tokens)}

    def generate(self, prompt: Sequence[int], gamma: int, max_new: int, mode: int = ACCEPT_NATURAL,
                 mode_seed: int = 0, seq: int = 0) -> Tuple[List[int], List[int]]:
        """Full response (R12).  Returns (max_new tokens, accept length of every iteration)."""
        self.prefill(prompt)
        P = len(prompt)
        accepts = []
        while len(self.tokens) - P < max_new:
            accepts.append(self.step(gamma, mode, mode_seed, seq)["accept_len"])
        return self.tokens[P:P + max_new], accepts


# ----------------------------------------------------------------------------------------------
# Independent reference loops used as pins
# ----------------------------------------------------------------------------------------------

def plain_greedy(shape, weights: Dict[str, np.ndarray], prompt: Sequence[int], max_new: int,
                 dtype=np.float64) -> List[int]:
    """Greedy decoding of the large model alone by full recompute: tok[t] = argmax M_L(prompt ++ tok[<t]).
    This is the definition that SPEED's output must equal (abstract; Section 3.1)."""
    dec = Decoder(weights, "L", shape.large.n_layers, shape.large.n_heads, dtype, shape.large.kv_heads)
    seq = [int(t) for t in prompt]
    for _ in range(max_new):
        _, logits = decoder_full_forward(dec, seq)
        seq.append(argmax_decision(logits[-1]))
    return seq[len(prompt):]


def plain_greedy_cached(shape, weights: Dict[str, np.ndarray], prompt: Sequence[int], max_new: int,
                        dtype=np.float64) -> List[int]:
    """The same tokens with a key/value cache and one-row block passes (used where full recompute
    is too slow; pinned against `plain_greedy` on small cases)."""
    dec = Decoder(weights, "L", shape.large.n_layers, shape.large.n_heads, dtype, shape.large.kv_heads)
    cache = KVCache(dec.n_layers)
    seq = [int(t) for t in prompt]
    if len(seq) > 1:
        large_block_pass(dec, cache, seq[:-1], 0)
    out = []
    for _ in range(max_new):
        _, logits = large_block_pass(dec, cache, [seq[-1]], len(seq) - 1)
        seq.append(argmax_decision(logits[0]))
        out.append(seq[-1])
    return out


def standalone_tandem_free_token(shape, weights: Dict[str, np.ndarray], prompt: Sequence[int], gamma: int,
                                 max_new: int, dtype=np.float64) -> List[int]:
    """Stand-alone Tandem decoding with the free token, written directly from Figure 2 and the
    "Representation Generation + Token Prediction" variant of Section 3, by brute force (no cache,
    no accept logic).  The prompt itself is read as in Figure 3 (R7).

    Each round: the small model, reading the large model's representations of everything but the
    last token, appends gamma tokens one at a time; then the large model reads the whole sequence
    and appends its own prediction of the next token."""
    large = Decoder(weights, "L", shape.large.n_layers, shape.large.n_heads, dtype, shape.large.kv_heads)
    small = Decoder(weights, "S", shape.small.n_layers, shape.small.n_heads, dtype, shape.small.kv_heads)
    proj = TandemProjection(weights, shape.small.n_layers, shape.ff_tandem_kind, dtype)
    seq = [int(t) for t in prompt]
    P = len(seq)
    while len(seq) - P < max_new:
        boundary = len(seq) - 1
        reps, _ = decoder_full_forward(large, seq[:boundary])
        for _ in range(gamma):
            lg = tandem_small_full_forward(small, proj, shape.layer_map, reps, boundary, seq)
            seq.append(argmax_decision(lg[-1]))
        _, logits = decoder_full_forward(large, seq)
        seq.append(argmax_decision(logits[-1]))
    return seq[P:P + max_new]


def standalone_tandem_representation_only(shape, weights: Dict[str, np.ndarray], prompt: Sequence[int], gamma: int,
                                          max_new: int, dtype=np.float64) -> List[int]:
    """Stand-alone Tandem decoding without the free token, written directly from Figure 3 and the
    "Representation Generation Only" variant of Section 3, by brute force (no cache).

    Each round: the large model's representations of everything but the last token are recomputed from
    scratch; the small model, attending them, appends gamma tokens one at a time.  The large model never
    predicts a token."""
    large = Decoder(weights, "L", shape.large.n_layers, shape.large.n_heads, dtype, shape.large.kv_heads)
    small = Decoder(weights, "S", shape.small.n_layers, shape.small.n_heads, dtype, shape.small.kv_heads)
    proj = TandemProjection(weights, shape.small.n_layers, shape.ff_tandem_kind, dtype)
    seq = [int(t) for t in prompt]
    P = len(seq)
    while len(seq) - P < max_new:
        boundary = len(seq) - 1
        reps, _ = decoder_full_forward(large, seq[:boundary])
        for _ in range(gamma):
            lg = tandem_small_full_forward(small, proj, shape.layer_map, reps, boundary, seq)
            seq.append(argmax_decision(lg[-1]))
    return seq[P:P + max_new]


def standalone_tandem_free_token_full_prompt(shape, weights: Dict[str, np.ndarray], prompt: Sequence[int], gamma: int,
                                             max_new: int, dtype=np.float64) -> List[int]:
    """Figure 2 as drawn, by brute force: the large model reads the whole sequence and appends its prediction;
    the small model, attending the large model's representations of everything before that token, appends
    gamma tokens; repeat."""
    large = Decoder(weights, "L", shape.large.n_layers, shape.large.n_heads, dtype, shape.large.kv_heads)
    small = Decoder(weights, "S", shape.small.n_layers, shape.small.n_heads, dtype, shape.small.kv_heads)
    proj = TandemProjection(weights, shape.small.n_layers, shape.ff_tandem_kind, dtype)
    seq = [int(t) for t in prompt]
    P = len(seq)
    while len(seq) - P < max_new:
        reps, logits = decoder_full_forward(large, seq)
        boundary = len(seq)
        seq.append(argmax_decision(logits[-1]))
        for _ in range(gamma):
            lg = tandem_small_full_forward(small, proj, shape.layer_map, reps, boundary, seq)
            seq.append(argmax_decision(lg[-1]))
    return seq[P:P + max_new]


def teacher_forced_tandem_logits(shape, weights: Dict[str, np.ndarray], ids: Sequence[int], gamma: int,
                                 dtype=np.float64) -> np.ndarray:
    """Eq. 2 over a whole given sequence by brute force (R20): for every block, the large model's representations of
    everything before the block are recomputed from scratch and the small model reads the block on top of them.
    Returns the small model's logits for positions 0 .. len(ids) - 1, shape [S][V]."""
    large = Decoder(weights, "L", shape.large.n_layers, shape.large.n_heads, dtype, shape.large.kv_heads)
    small = Decoder(weights, "S", shape.small.n_layers, shape.small.n_heads, dtype, shape.small.kv_heads)
    proj = TandemProjection(weights, shape.small.n_layers, shape.ff_tandem_kind, dtype)
    seq = [int(t) for t in ids]
    out = []
    for start in range(0, len(seq), gamma):
        end = min(len(seq), start + gamma)
        reps, _ = decoder_full_forward(large, seq[:start])
        out.append(tandem_small_full_forward(small, proj, shape.layer_map, reps, start, seq[:end]))
    return np.concatenate(out, axis=0)


def next_token_scores(logits: np.ndarray, ids: Sequence[int]) -> Tuple[np.ndarray, np.ndarray]:
    """For positions 0 .. S-2: (negative log-likelihood of the true next token under softmax(logits), arg-max)."""
    S = len(ids)
    nll = np.empty(S - 1)
    top = np.empty(S - 1, dtype=np.int64)
    for i in range(S - 1):
        row = np.asarray(logits[i], dtype=np.float64)
        m = row.max()
        nll[i] = m + math.log(np.exp(row - m).sum()) - row[int(ids[i + 1])]
        top[i] = argmax_decision(logits[i])
    return nll, top


def generate_batch(shape, weights: Dict[str, np.ndarray], prompts: Sequence[Sequence[int]], gamma: int,
                   max_new: int, mode: int = ACCEPT_NATURAL, mode_seed: int = 0, dtype=np.float64):
    """Independent sequences (R11).  Returns (tokens per sequence, accept lengths per sequence,
    (large runs, small runs) per sequence)."""
    toks, accs, runs = [], [], []
    for b, p in enumerate(prompts):
        o = TandemOracle(shape, weights, dtype)
        t, a = o.generate(p, gamma, max_new, mode, mode_seed, b)
        toks.append(t)
        accs.append(a)
        runs.append((o.n_large_runs, o.n_small_runs))
    return toks, accs, runs
