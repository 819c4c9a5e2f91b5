"""CPU oracle for SkipDecode's batched skip-decode forward pass.  TEST INFRASTRUCTURE.

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
import this module.  It shares no code with the CUDA library and never calls it.

Everything is plain PyTorch CPU arithmetic in `dtype` (float64 unless the caller
asks for float32); weights may be stored in bf16 or fp32 and are widened at use,
so a bf16 configuration is evaluated on exactly the bf16-rounded weight values.

What it computes (paper sections in brackets):

* `schedule`            per-position layer budget, linear decay from max to min
                        over the generated positions, all layers for the prompt
                        [Section 2.3, the token_idx equation and Figure 3].
* `active_layers`       which layers run at a position: the bottom `warmup`
                        layers plus the top (n - warmup) layers; the layers in
                        between are bypassed [Section 2.4].
* `forward_sequence`    THE DEFINITION.  A whole sequence, layer by layer; a layer
                        that is not active at a position leaves that position's
                        hidden state untouched and produces no key/value there;
                        active positions attend causally to the keys/values of
                        that same layer.  Monotone budgets make every key/value
                        that is needed exist [Sections 2.1, 2.2, 2.4].
* `CachedDecoder`       the same numbers produced the way generation runs:
                        prompt first with all layers, then one column of the
                        batch per step, reusing cached keys/values untouched
                        [Sections 2.1-2.3].
* `full_forward`        an ordinary pre-LayerNorm OPT-style decoder with no notion
                        of skipping: the 1x base model of Section 3.1.
* `forward_ragged`      rows of different prompt lengths in one batch, aligned at the
                        right: each row alone, budgets taken by slot [Sections 2.1, 5].
* `sample_top_p`        the paper's token selection: temperature softmax, nucleus of
                        mass top_p, inverse-CDF draw from a caller-supplied uniform
                        number [Section 3.2: beam 1, top-p 0.7, temperature 0.3].

Model (OPT-style, the family the paper evaluates in Section 3): learned absolute
positions added to token embeddings; per layer  u = LN1(h);  q = (Wq u + bq)/sqrt(hd),
k = Wk u + bk, v = Wv u + bv;  a = concat_heads softmax_j<=i(q.k_j) v_j;
r = h + Wo a + bo;  h' = r + W2 relu(W1 LN2(r) + b1) + b2;  logits = E LN_f(h_L) with
the head tied to the token embedding E.  LayerNorm uses the biased variance and
eps 1e-5.

Pins (tests/test_oracle_*.py): schedule against the figure's printed function,
Table 2's budgets, exact rational arithmetic and the prose invariants;
`full_forward` against the Hugging Face OPT implementation with the same weights;
`forward_sequence` and `CachedDecoder` against each other, against `full_forward`
for a full budget, against closed forms (bias-only model, zero-query attention =
running mean of values, LayerNorm of a hand-computed vector) and against a
scalar pure-Python evaluation on a toy model; `nucleus` / `sample_top_p` against an
exhaustive search over all subsets of a small vocabulary, the Hugging Face
temperature and top-p logits warpers, exact frequencies under equally spaced
uniforms, and the argmax limits.
Parity unpinned: absolute logit values with trained OPT weights and any output
quality figure of the paper (no trained weights or datasets are available).
"""
from __future__ import annotations

import math
from fractions import Fraction

import torch

LN_EPS = 1e-5


# --------------------------------------------------------------------------- schedule

def schedule(max_layers: int, min_layers: int, warmup: int, gen_len: int, n_layers: int,
             closed_interval: bool = True):
    """Layer budget for the gen_len generated positions [Section 2.3].

    The paper's line is (1 - t) * max + t * min.  With `closed_interval` (the
    reading used throughout) t = g / (gen_len - 1), so the first generated
    position gets exactly max and the last exactly min, as the prose and the
    plotted function of Figure 3 say; the literal equation divides by gen_len
    instead and is kept only as the alternative (`closed_interval=False`).
    The real value is rounded to the nearest integer, halves up, in exact
    rational arithmetic.  Returns (n_active, top_begin): at generated index g the
    active layers are [0, warmup) and [top_begin[g], n_layers) [Section 2.4].
    """
    if not (0 <= warmup < min_layers <= max_layers <= n_layers and gen_len >= 1):
        raise ValueError("need 0 <= warmup < min <= max <= n_layers and gen_len >= 1")
    n_active, top_begin = [], []
    for g in range(gen_len):
        if gen_len == 1:
            t = Fraction(0)
        elif closed_interval:
            t = Fraction(g, gen_len - 1)
        else:
            t = Fraction(g, gen_len)
        line = (1 - t) * max_layers + t * min_layers
        n = math.floor(line + Fraction(1, 2))
        n_active.append(n)
        top_begin.append(n_layers - (n - warmup))
    return n_active, top_begin


def schedule_power(max_layers: int, min_layers: int, warmup: int, gen_len: int, n_layers: int, alpha: int):
    """Power-law decay, which Section 2.3 names as another possible budget function:
    min + (max - min) * (1 - t)^alpha with t = g / (gen_len - 1) (reading: integer exponent,
    same closed interval and rounding as the linear schedule; alpha = 1 is that schedule)."""
    if not (0 <= warmup < min_layers <= max_layers <= n_layers and gen_len >= 1 and alpha >= 1):
        raise ValueError("bad schedule arguments")
    n_active, top_begin = [], []
    for g in range(gen_len):
        t = Fraction(0) if gen_len == 1 else Fraction(g, gen_len - 1)
        n = math.floor(min_layers + (max_layers - min_layers) * (1 - t) ** alpha + Fraction(1, 2))
        n_active.append(n)
        top_begin.append(n_layers - (n - warmup))
    return n_active, top_begin


def active_layers(n_layers: int, n: int, warmup: int):
    """Indices of the layers that run when the budget is n [Section 2.4]."""
    return list(range(warmup)) + list(range(n_layers - (n - warmup), n_layers))


def active_matrix(n_layers: int, prompt_len: int, n_active, warmup: int) -> torch.Tensor:
    """bool [prompt_len + len(n_active), n_layers]; prompt rows are all True."""
    S = prompt_len + len(n_active)
    act = torch.zeros(S, n_layers, dtype=torch.bool)
    act[:prompt_len, :] = True
    for g, n in enumerate(n_active):
        act[prompt_len + g, active_layers(n_layers, n, warmup)] = True
    return act


# --------------------------------------------------------------------------- pieces

def layer_norm(x: torch.Tensor, gamma: torch.Tensor, beta: torch.Tensor) -> torch.Tensor:
    mean = x.mean(dim=-1, keepdim=True)
    var = ((x - mean) ** 2).mean(dim=-1, keepdim=True)
    return (x - mean) / torch.sqrt(var + LN_EPS) * gamma + beta


def _w(t: torch.Tensor, dtype) -> torch.Tensor:
    return t.to(dtype)


def _split_heads(x: torch.Tensor, n_heads: int) -> torch.Tensor:
    # [..., S, d] -> [..., H, S, hd]
    *lead, S, d = x.shape
    return x.reshape(*lead, S, n_heads, d // n_heads).transpose(-3, -2)


def _merge_heads(x: torch.Tensor) -> torch.Tensor:
    # [..., H, S, hd] -> [..., S, H*hd]
    x = x.transpose(-3, -2)
    *lead, S, H, hd = x.shape
    return x.reshape(*lead, S, H * hd)


def _qkv(u: torch.Tensor, lw: dict, n_heads: int, dtype):
    d = u.shape[-1]
    qkv = u @ _w(lw["w_qkv"], dtype).T + _w(lw["b_qkv"], dtype)
    q, k, v = qkv[..., :d], qkv[..., d:2 * d], qkv[..., 2 * d:]
    q = q / math.sqrt(d // n_heads)
    return q, k, v


def _ffn(r: torch.Tensor, lw: dict, dtype) -> torch.Tensor:
    u2 = layer_norm(r, _w(lw["ln2_g"], dtype), _w(lw["ln2_b"], dtype))
    y = torch.relu(u2 @ _w(lw["w_fc1"], dtype).T + _w(lw["b_fc1"], dtype))
    return r + y @ _w(lw["w_fc2"], dtype).T + _w(lw["b_fc2"], dtype)


def _embed(weights: dict, tokens: torch.Tensor, positions: torch.Tensor, dtype) -> torch.Tensor:
    return _w(weights["tok_emb"][tokens.long()], dtype) + _w(weights["pos_emb"][positions.long()], dtype)


def _head(weights: dict, h: torch.Tensor, dtype) -> torch.Tensor:
    z = layer_norm(h, _w(weights["lnf_g"], dtype), _w(weights["lnf_b"], dtype))
    return z @ _w(weights["tok_emb"], dtype).T


def _causal_layer(h: torch.Tensor, lw: dict, n_heads: int, dtype) -> torch.Tensor:
    """One decoder layer over positions 0..S-1 of every row, causal attention."""
    S = h.shape[-2]
    u = layer_norm(h, _w(lw["ln1_g"], dtype), _w(lw["ln1_b"], dtype))
    q, k, v = _qkv(u, lw, n_heads, dtype)
    qh, kh, vh = (_split_heads(t, n_heads) for t in (q, k, v))
    scores = qh @ kh.transpose(-1, -2)                       # [B,H,S,S]
    future = torch.triu(torch.ones(S, S, dtype=torch.bool), diagonal=1)
    scores = scores.masked_fill(future, float("-inf"))
    a = _merge_heads(torch.softmax(scores, dim=-1) @ vh)
    r = h + a @ _w(lw["w_o"], dtype).T + _w(lw["b_o"], dtype)
    return _ffn(r, lw, dtype)


# --------------------------------------------------------------------------- definition

def forward_sequence(weights: dict, n_heads: int, tokens: torch.Tensor, active: torch.Tensor,
                     dtype=torch.float64, return_hidden: bool = False, logits_from: int = 0):
    """Logits at every position of tokens[B,S] under per-position layer sets.

    active[i, l] says whether layer l runs at position i.  A layer that does not
    run at a position is the identity there and contributes no key/value
    [Section 2.4]; the positions where a layer runs must form a prefix 0..m-1
    (monotone budgets, Section 2.2), otherwise a needed key would not exist and
    the call raises.  Logits are returned for positions logits_from..S-1 only.
    """
    B, S = tokens.shape
    L = len(weights["layers"])
    assert active.shape == (S, L)
    h = _embed(weights, tokens, torch.arange(S).expand(B, S), dtype)        # [B,S,d]
    for l in range(L):
        m = int(active[:, l].sum())
        if not bool(active[:m, l].all()):
            raise ValueError(f"layer {l}: active positions are not a prefix (budget not monotone)")
        if m == 0:
            continue
        h = torch.cat([_causal_layer(h[:, :m], weights["layers"][l], n_heads, dtype), h[:, m:]], dim=1)
    logits = _head(weights, h[:, logits_from:], dtype)
    return (logits, h) if return_hidden else logits


def forward_ragged(weights: dict, n_heads: int, tokens: torch.Tensor, pad, active: torch.Tensor,
                   dtype=torch.float64, logits_from: int = 0) -> torch.Tensor:
    """Left-padded batch: row b's sequence occupies slots pad[b]..S-1 of tokens[b].

    Batching puts every row's token of one step into the same slot, and the layer
    budget belongs to the slot (all tokens of a batch at one position share it,
    Section 2.1); rows of different prompt lengths are aligned at the right, so a
    shorter row starts later (the limitation discussed in Section 5: rows can only
    share a batch at matching positions).  Padding must be invisible: row b is the
    sequence tokens[b, pad[b]:] on its own, its first real token at position 0,
    with slot s using the layer set active[s].  Each row is therefore evaluated
    alone by `forward_sequence`.  Returns logits [B, S - logits_from, V]; entries
    of slots that hold padding are NaN.
    """
    B, S = tokens.shape
    out = None
    for b in range(B):
        p = int(pad[b])
        if not 0 <= p < S:
            raise ValueError("a row needs at least one real token")
        lg = forward_sequence(weights, n_heads, tokens[b:b + 1, p:], active[p:], dtype,
                              logits_from=max(logits_from - p, 0))[0]
        if out is None:
            out = torch.full((B, S - logits_from, lg.shape[-1]), float("nan"), dtype=lg.dtype)
        out[b, S - logits_from - lg.shape[0]:] = lg
    return out


def full_forward(weights: dict, n_heads: int, tokens: torch.Tensor, dtype=torch.float64) -> torch.Tensor:
    """Ordinary decoder forward over tokens[B,S]: every layer at every position."""
    B, S = tokens.shape
    h = _embed(weights, tokens, torch.arange(S).expand(B, S), dtype)
    for lw in weights["layers"]:
        h = _causal_layer(h, lw, n_heads, dtype)
    return _head(weights, h, dtype)


# --------------------------------------------------------------------------- generation order

class CachedDecoder:
    """Prompt with all layers, then one position per step with cached keys/values.

    Mirrors the library's call order: `set_schedule`, `prefill`, then
    `decode_step(ids, P)`, `decode_step(ids, P + 1)`, ...  Cached entries are
    appended only in the layers that run and are never rewritten [Section 2.2].
    """

    def __init__(self, weights: dict, n_heads: int, dtype=torch.float64):
        self.w, self.H, self.dtype = weights, n_heads, dtype
        self.L = len(weights["layers"])
        self.n_active = self.top_begin = None
        self.warmup = 0
        self.P = None
        self.k = self.v = None
        self.layer_steps = 0

    def set_table(self, n_active, warmup):
        """Installs an arbitrary non-increasing budget table."""
        if any(b > a for a, b in zip(n_active, n_active[1:])) or any(not (warmup < n <= self.L) for n in n_active):
            raise ValueError("budget table must be non-increasing with warmup < n <= n_layers")
        self.n_active = list(n_active)
        self.top_begin = [self.L - (n - warmup) for n in n_active]
        self.warmup = warmup
        return self.n_active, self.top_begin

    def set_schedule(self, max_layers, min_layers, warmup, gen_len):
        self.n_active, self.top_begin = schedule(max_layers, min_layers, warmup, gen_len, self.L)
        self.warmup = warmup
        return self.n_active, self.top_begin

    def _step(self, ids: torch.Tensor, pos: int, layers) -> torch.Tensor:
        B = ids.shape[0]
        h = _embed(self.w, ids.reshape(B, 1), torch.full((B, 1), pos), self.dtype)      # [B,1,d]
        for l in layers:
            lw = self.w["layers"][l]
            u = layer_norm(h, _w(lw["ln1_g"], self.dtype), _w(lw["ln1_b"], self.dtype))
            q, k, v = _qkv(u, lw, self.H, self.dtype)
            have = 0 if self.k[l] is None else self.k[l].shape[-2]
            if have != pos:     # a skipped position would leave a hole: budgets must be monotone
                raise RuntimeError(f"layer {l} holds {have} cached positions at position {pos}")
            kh, vh = _split_heads(k, self.H), _split_heads(v, self.H)
            self.k[l] = kh if self.k[l] is None else torch.cat([self.k[l], kh], dim=-2)
            self.v[l] = vh if self.v[l] is None else torch.cat([self.v[l], vh], dim=-2)
            p = torch.softmax(_split_heads(q, self.H) @ self.k[l].transpose(-1, -2), dim=-1)   # [B,H,1,T]
            a = _merge_heads(p @ self.v[l])
            r = h + a @ _w(lw["w_o"], self.dtype).T + _w(lw["b_o"], self.dtype)
            h = _ffn(r, lw, self.dtype)
        return _head(self.w, h, self.dtype)[:, 0]

    def prefill_stepwise(self, tokens: torch.Tensor) -> torch.Tensor:
        """Prompt one position at a time through every layer (slow, tiny inputs)."""
        B, P = tokens.shape
        self.k, self.v = [None] * self.L, [None] * self.L
        for i in range(P):
            logits = self._step(tokens[:, i], i, range(self.L))
        self.P = P
        return logits

    def prefill(self, tokens: torch.Tensor) -> torch.Tensor:
        """Prompt in one batched causal pass per layer; fills the cache for all
        layers and returns the logits of the last prompt position [Section 2.3]."""
        B, P = tokens.shape
        self.k, self.v = [None] * self.L, [None] * self.L
        h = _embed(self.w, tokens, torch.arange(P).expand(B, P), self.dtype)
        future = torch.triu(torch.ones(P, P, dtype=torch.bool), diagonal=1)
        for l, lw in enumerate(self.w["layers"]):
            u = layer_norm(h, _w(lw["ln1_g"], self.dtype), _w(lw["ln1_b"], self.dtype))
            q, k, v = _qkv(u, lw, self.H, self.dtype)
            self.k[l], self.v[l] = _split_heads(k, self.H), _split_heads(v, self.H)
            s = (_split_heads(q, self.H) @ self.k[l].transpose(-1, -2)).masked_fill(future, float("-inf"))
            a = _merge_heads(torch.softmax(s, dim=-1) @ self.v[l])
            r = h + a @ _w(lw["w_o"], self.dtype).T + _w(lw["b_o"], self.dtype)
            h = _ffn(r, lw, self.dtype)
        self.P = P
        return _head(self.w, h[:, -1:], self.dtype)[:, 0]

    def decode_step(self, ids: torch.Tensor, position: int) -> torch.Tensor:
        g = position - self.P
        if self.n_active is None or not (0 <= g < len(self.n_active)):
            raise RuntimeError("position outside the installed schedule")
        layers = active_layers(self.L, self.n_active[g], self.warmup)
        self.layer_steps += len(layers)
        return self._step(ids, position, layers)


def greedy(logits: torch.Tensor) -> torch.Tensor:
    """Lowest index attaining the maximum of each row."""
    return torch.argmax(logits, dim=-1).to(torch.int32)


# --------------------------------------------------------------------------- sampling

def nucleus(logits_row: torch.Tensor, temperature: float, top_p: float):
    """Temperature softmax and its nucleus for ONE row of logits.

    The paper's generation settings are a beam of 1, top-p 0.7 and temperature 0.3
    (Section 3.2, Datasets).  Top-p ("nucleus") sampling keeps the smallest set of
    most probable tokens whose probabilities add up to at least top_p and samples
    from that set in proportion to the probabilities.

    Returns (order, probs, k): token ids sorted by decreasing probability (equal
    probabilities: lower id first), their float64 probabilities in that order, and
    the size k >= 1 of the nucleus, the first k entries of `order`.
    """
    x = logits_row.to(torch.float64) / float(temperature)
    probs = torch.softmax(x, dim=0)
    order = torch.sort(probs, descending=True, stable=True).indices
    sorted_probs = probs[order]
    cum = torch.cumsum(sorted_probs, dim=0)
    reached = torch.nonzero(cum >= top_p)
    k = int(reached[0]) + 1 if reached.numel() else int(probs.numel())
    return order, sorted_probs, k


def sample_top_p(logits: torch.Tensor, uniforms: torch.Tensor, temperature: float, top_p: float) -> torch.Tensor:
    """One token per row by inverse-CDF sampling inside the nucleus.

    `uniforms[b]` in [0, 1) is the random number of row b, supplied by the caller.
    With the nucleus in decreasing-probability order and M its total probability,
    the token chosen is the first whose running sum reaches uniforms[b] * M (the
    last token of the nucleus if rounding leaves the target unreached).
    """
    out = torch.empty(logits.shape[0], dtype=torch.int32)
    for b in range(logits.shape[0]):
        order, sorted_probs, k = nucleus(logits[b], temperature, top_p)
        cum = torch.cumsum(sorted_probs[:k], dim=0)
        target = float(uniforms[b]) * float(cum[-1])
        hit = torch.nonzero(cum > target)
        j = int(hit[0]) if hit.numel() else k - 1
        out[b] = int(order[j])
    return out
