"""Pins for the oracle's forward pass.

The ordinary forward is pinned to an independent library implementation of the
same architecture (Hugging Face OPT) and to a scalar pure-Python evaluation;
the skip semantics are pinned by closed forms and by the agreement of the
definition (whole sequence, layer by layer) with cached position-by-position
generation.  The last test plants mistakes in the oracle and checks the pins
notice them.
"""
import math

import pytest
import torch

from oracle import skipdecode_oracle as O
from paper_2307_02628_b200 import synth

F64 = torch.float64


def toy_shape(L=3, d=32, H=4, f=48, V=61, maxpos=40):
    return synth.ModelShape("toy", L, d, H, f, V, maxpos, "fp32")


def toy_weights(shape, seed=7, std=0.3):
    w = synth.make_weights(shape, seed=seed, std=std, random_ln=True, threads=1)
    return w


def hf_logits(shape, w, tokens, attention_mask=None):
    from transformers import OPTConfig, OPTForCausalLM
    cfg = OPTConfig(vocab_size=shape.vocab, hidden_size=shape.d_model, num_hidden_layers=shape.n_layers,
                    ffn_dim=shape.d_ffn, num_attention_heads=shape.n_heads,
                    max_position_embeddings=shape.max_pos, word_embed_proj_dim=shape.d_model,
                    do_layer_norm_before=True, dropout=0.0, attention_dropout=0.0,
                    activation_function="relu", layer_norm_elementwise_affine=True,
                    enable_bias=True, tie_word_embeddings=True)
    m = OPTForCausalLM(cfg).double().eval()
    d = shape.d_model
    sd = {}
    dec = "model.decoder."
    sd[dec + "embed_tokens.weight"] = w["tok_emb"]
    pos = torch.zeros(shape.max_pos + 2, d)
    pos[2:] = w["pos_emb"]                       # the library offsets learned positions by 2
    sd[dec + "embed_positions.weight"] = pos
    sd[dec + "final_layer_norm.weight"] = w["lnf_g"]
    sd[dec + "final_layer_norm.bias"] = w["lnf_b"]
    for l, lw in enumerate(w["layers"]):
        p = f"{dec}layers.{l}."
        for i, nm in enumerate("qkv"):
            sd[p + f"self_attn.{nm}_proj.weight"] = lw["w_qkv"][i * d:(i + 1) * d]
            sd[p + f"self_attn.{nm}_proj.bias"] = lw["b_qkv"][i * d:(i + 1) * d]
        sd[p + "self_attn.out_proj.weight"] = lw["w_o"]
        sd[p + "self_attn.out_proj.bias"] = lw["b_o"]
        sd[p + "self_attn_layer_norm.weight"] = lw["ln1_g"]
        sd[p + "self_attn_layer_norm.bias"] = lw["ln1_b"]
        sd[p + "fc1.weight"] = lw["w_fc1"]
        sd[p + "fc1.bias"] = lw["b_fc1"]
        sd[p + "fc2.weight"] = lw["w_fc2"]
        sd[p + "fc2.bias"] = lw["b_fc2"]
        sd[p + "final_layer_norm.weight"] = lw["ln2_g"]
        sd[p + "final_layer_norm.bias"] = lw["ln2_b"]
    sd["lm_head.weight"] = w["tok_emb"]
    missing, unexpected = m.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not unexpected and all("lm_head" in k for k in missing), (missing, unexpected)
    with torch.no_grad():
        if attention_mask is not None:
            return m(tokens.long(), attention_mask=attention_mask.long()).logits
        return m(tokens.long()).logits


def hf_gap(shape=None, seed=7):
    shape = shape or toy_shape()
    w = toy_weights(shape, seed)
    tokens = synth.make_tokens(shape.vocab, 3, 11, seed=5)
    ref = hf_logits(shape, w, tokens)
    got = O.full_forward(w, shape.n_heads, tokens, F64)
    return float((ref - got).abs().max()), float(ref.abs().max())


def test_full_forward_matches_library_opt():
    gap, scale = hf_gap()
    assert scale > 0.5                      # the comparison is not between zeros
    assert gap < 1e-9, gap


# ---------------------------------------------------------------- scalar brute force

def scalar_forward(shape, w, toks, active):
    """Logits at the last position of one row, with Python floats and index loops."""
    L, d, H, f, V = shape.n_layers, shape.d_model, shape.n_heads, shape.d_ffn, shape.vocab
    hd = d // H
    A = lambda t: t.double().tolist()

    def ln(x, g, b):
        mu = sum(x) / len(x)
        var = sum((xi - mu) ** 2 for xi in x) / len(x)
        return [(xi - mu) / math.sqrt(var + 1e-5) * gi + bi for xi, gi, bi in zip(x, g, b)]

    def lin(Wm, bv, x):      # y[o] = sum_i W[o][i] x[i] + b[o]
        return [sum(Wm[o][i] * x[i] for i in range(len(x))) + bv[o] for o in range(len(Wm))]

    S = len(toks)
    te, pe = A(w["tok_emb"]), A(w["pos_emb"])
    h = [[te[toks[i]][c] + pe[i][c] for c in range(d)] for i in range(S)]
    for l in range(L):
        lw = {k: A(v) for k, v in w["layers"][l].items()}
        ks, vs = {}, {}
        newh = [row[:] for row in h]
        for i in range(S):
            if not active[i][l]:
                continue
            u = ln(h[i], lw["ln1_g"], lw["ln1_b"])
            qkv = lin(lw["w_qkv"], lw["b_qkv"], u)
            q, ks[i], vs[i] = [x / math.sqrt(hd) for x in qkv[:d]], qkv[d:2 * d], qkv[2 * d:]
            a = [0.0] * d
            for hh in range(H):
                sl = range(hh * hd, (hh + 1) * hd)
                sc = [sum(q[c] * ks[j][c] for c in sl) for j in range(i + 1)]
                mx = max(sc)
                e = [math.exp(s - mx) for s in sc]
                z = sum(e)
                for c in sl:
                    a[c] = sum(e[j] / z * vs[j][c] for j in range(i + 1))
            o = lin(lw["w_o"], lw["b_o"], a)
            r = [h[i][c] + o[c] for c in range(d)]
            y = [max(0.0, t) for t in lin(lw["w_fc1"], lw["b_fc1"], ln(r, lw["ln2_g"], lw["ln2_b"]))]
            z2 = lin(lw["w_fc2"], lw["b_fc2"], y)
            newh[i] = [r[c] + z2[c] for c in range(d)]
        h = newh
    zf = ln(h[S - 1], A(w["lnf_g"]), A(w["lnf_b"]))
    return [sum(te[v][c] * zf[c] for c in range(d)) for v in range(V)]


def test_definition_matches_scalar_brute_force_with_skips():
    shape = toy_shape(L=3, d=8, H=2, f=12, V=9, maxpos=8)
    w = toy_weights(shape, seed=11, std=0.5)
    toks = [3, 8, 0, 5, 1]
    # prompt of 2 (all layers), then budgets 3, 2 (warm-up 1 => layers {0, 2}), 2
    act = O.active_matrix(3, 2, [3, 2, 2], 1)
    assert act.tolist()[3] == [True, False, True]
    ref = scalar_forward(shape, w, toks, act.tolist())
    got = O.forward_sequence(w, shape.n_heads, torch.tensor([toks]), act, F64)[0, -1]
    assert max(abs(a - b) for a, b in zip(ref, got.tolist())) < 1e-10
    # and the skipping changes the answer (the comparison is not vacuous)
    full = O.full_forward(w, shape.n_heads, torch.tensor([toks]), F64)[0, -1]
    assert float((full - got).abs().max()) > 1e-3


# ---------------------------------------------------------------- closed forms

def test_layer_norm_hand_computed():
    x = torch.tensor([[1.0, 2.0, 3.0, 4.0]], dtype=F64)
    y = O.layer_norm(x, torch.ones(4, dtype=F64), torch.zeros(4, dtype=F64))[0].tolist()
    s = 1.0 / math.sqrt(1.25 + 1e-5)           # mean 2.5, biased variance 1.25
    assert y == pytest.approx([-1.5 * s, -0.5 * s, 0.5 * s, 1.5 * s], abs=1e-14)
    y2 = O.layer_norm(x, torch.tensor([2.0, 2, 2, 2], dtype=F64), torch.tensor([1.0, 1, 1, 1], dtype=F64))[0]
    assert y2.tolist() == pytest.approx([1 - 3 * s, 1 - s, 1 + s, 1 + 3 * s], abs=1e-14)


def _zero_matrices(w):
    for lw in w["layers"]:
        for k in ("w_qkv", "w_o", "w_fc1", "w_fc2"):
            lw[k] = torch.zeros_like(lw[k])


def test_bias_only_model_counts_exactly_the_active_layers():
    # With every matrix zero a layer adds b_o + b_fc2 to the residual wherever it runs
    # and nothing elsewhere, so the final hidden state spells out the active set.
    shape = toy_shape(L=6, d=16, H=2, f=24, V=23, maxpos=32)
    w = toy_weights(shape, seed=3)
    _zero_matrices(w)
    P, G, warm = 4, 9, 1
    n, top = O.schedule(5, 2, warm, G, shape.n_layers)
    act = O.active_matrix(shape.n_layers, P, n, warm)
    toks = synth.make_tokens(shape.vocab, 2, P + G, seed=9)
    _, h = O.forward_sequence(w, shape.n_heads, toks, act, F64, return_hidden=True)
    for b in range(2):
        for i in range(P + G):
            layers = range(shape.n_layers) if i < P else O.active_layers(shape.n_layers, n[i - P], warm)
            want = w["tok_emb"][toks[b, i].item()].double() + w["pos_emb"][i].double()
            for l in layers:
                want = want + w["layers"][l]["b_o"].double() + w["layers"][l]["b_fc2"].double()
            assert torch.allclose(h[b, i], want, atol=1e-12)


def test_zero_query_attention_is_running_mean_of_values():
    # One layer, zero query projection => uniform causal attention; W_o = I, FFN off:
    # h'_i = h_i + mean_{j<=i} v_j with v_j = LN1(h_j) (W_v = I, b_v = 0).
    shape = toy_shape(L=1, d=8, H=2, f=8, V=13, maxpos=16)
    w = toy_weights(shape, seed=5, std=1.0)
    lw = w["layers"][0]
    d = shape.d_model
    lw["w_qkv"] = torch.cat([torch.zeros(d, d), torch.randn(d, d), torch.eye(d)])
    lw["b_qkv"] = torch.zeros(3 * d)
    lw["w_o"], lw["b_o"] = torch.eye(d), torch.zeros(d)
    lw["w_fc2"], lw["b_fc2"] = torch.zeros_like(lw["w_fc2"]), torch.zeros(d)
    lw["ln1_g"], lw["ln1_b"] = torch.ones(d), torch.zeros(d)
    toks = synth.make_tokens(shape.vocab, 1, 7, seed=2)
    _, h = O.forward_sequence(w, shape.n_heads, toks, torch.ones(7, 1, dtype=torch.bool), F64, return_hidden=True)
    h0 = w["tok_emb"][toks[0].long()].double() + w["pos_emb"][:7].double()
    v = (h0 - h0.mean(-1, keepdim=True)) / h0.std(-1, unbiased=False, keepdim=True).pow(2).add(1e-5).sqrt()
    for i in range(7):
        assert torch.allclose(h[0, i], h0[i] + v[: i + 1].mean(0), atol=1e-12)


def test_single_key_attention_returns_the_value():
    # At position 0 the softmax has one term, so the attention output is v_0 exactly.
    shape = toy_shape(L=1, d=8, H=2, f=8, V=13, maxpos=16)
    w = toy_weights(shape, seed=6, std=1.0)
    lw = w["layers"][0]
    d = shape.d_model
    lw["w_o"], lw["b_o"] = torch.eye(d), torch.zeros(d)
    lw["w_fc2"], lw["b_fc2"] = torch.zeros_like(lw["w_fc2"]), torch.zeros(d)
    toks = torch.tensor([[4]], dtype=torch.int32)
    _, h = O.forward_sequence(w, shape.n_heads, toks, torch.ones(1, 1, dtype=torch.bool), F64, return_hidden=True)
    h0 = (w["tok_emb"][4] + w["pos_emb"][0]).double()
    u = O.layer_norm(h0, lw["ln1_g"].double(), lw["ln1_b"].double())
    v0 = lw["w_qkv"][2 * d:].double() @ u + lw["b_qkv"][2 * d:].double()
    assert torch.allclose(h[0, 0], h0 + v0, atol=1e-12)


# ---------------------------------------------------------------- formulations agree

@pytest.mark.parametrize("mx,mn,warm,P,G,B", [(3, 3, 0, 5, 6, 2), (3, 1, 0, 4, 7, 3), (3, 2, 1, 1, 5, 1), (3, 2, 1, 6, 1, 2)])
def test_cached_generation_equals_definition(mx, mn, warm, P, G, B):
    shape = toy_shape()
    w = toy_weights(shape)
    prompts = synth.make_tokens(shape.vocab, B, P, seed=1)
    dec = O.CachedDecoder(w, shape.n_heads, F64)
    n, top = dec.set_schedule(mx, mn, warm, G)
    logits = [dec.prefill(prompts)]
    toks = [prompts]
    for g in range(G):
        ids = O.greedy(logits[-1])
        toks.append(ids.reshape(B, 1))
        logits.append(dec.decode_step(ids, P + g))
    seq = torch.cat(toks, dim=1)
    act = O.active_matrix(shape.n_layers, P, n, warm)
    ref = O.forward_sequence(w, shape.n_heads, seq, act, F64)
    for g in range(G + 1):
        assert torch.allclose(logits[g], ref[:, P - 1 + g], atol=1e-10, rtol=0), g
    assert dec.layer_steps == sum(n)
    if mx == mn == shape.n_layers:          # a full budget is ordinary decoding (the 1x base model)
        assert torch.allclose(ref, O.full_forward(w, shape.n_heads, seq, F64), atol=1e-12, rtol=0)


def test_prefill_batched_equals_stepwise():
    shape = toy_shape()
    w = toy_weights(shape)
    prompts = synth.make_tokens(shape.vocab, 2, 9, seed=4)
    a, b = O.CachedDecoder(w, shape.n_heads, F64), O.CachedDecoder(w, shape.n_heads, F64)
    la, lb = a.prefill(prompts), b.prefill_stepwise(prompts)
    assert torch.allclose(la, lb, atol=1e-11, rtol=0)
    for l in range(shape.n_layers):
        assert torch.allclose(a.k[l], b.k[l], atol=1e-11) and torch.allclose(a.v[l], b.v[l], atol=1e-11)


def test_rows_are_independent():
    shape = toy_shape()
    w = toy_weights(shape)
    toks = synth.make_tokens(shape.vocab, 4, 8, seed=8)
    act = O.active_matrix(shape.n_layers, 3, [3, 2, 2, 1, 1], 0)
    full = O.forward_sequence(w, shape.n_heads, toks, act, F64)
    perm = torch.tensor([2, 0, 3, 1])
    assert torch.allclose(O.forward_sequence(w, shape.n_heads, toks[perm], act, F64), full[perm], atol=1e-12)
    assert torch.allclose(O.forward_sequence(w, shape.n_heads, toks[1:2], act, F64), full[1:2], atol=1e-12)


def test_non_monotone_budget_is_rejected():
    shape = toy_shape()
    w = toy_weights(shape)
    act = torch.ones(4, 3, dtype=torch.bool)
    act[1, 0] = False                       # position 1 skips layer 0 but position 2 runs it
    with pytest.raises(ValueError):
        O.forward_sequence(w, shape.n_heads, synth.make_tokens(shape.vocab, 1, 4, seed=1), act, F64)
    dec = O.CachedDecoder(w, shape.n_heads, F64)
    dec.prefill(synth.make_tokens(shape.vocab, 1, 4, seed=1))
    dec.n_active, dec.warmup = [1, 2], 0    # budget grows: layer 1 has a hole at position 4
    dec.decode_step(torch.tensor([1]), 4)
    with pytest.raises(RuntimeError):
        dec.decode_step(torch.tensor([1]), 5)


def test_fp32_mode_is_close_to_fp64():
    shape = toy_shape()
    w = toy_weights(shape, std=0.05)
    toks = synth.make_tokens(shape.vocab, 2, 10, seed=8)
    act = O.active_matrix(shape.n_layers, 4, [3, 3, 2, 2, 1, 1], 0)
    a = O.forward_sequence(w, shape.n_heads, toks, act, torch.float64)
    b = O.forward_sequence(w, shape.n_heads, toks, act, torch.float32)
    assert float((a - b.double()).abs().max()) < 1e-5


# ---------------------------------------------------------------- the pins bite

@pytest.mark.parametrize("mistake", ["unbiased_variance", "no_query_scale", "transposed_out_proj",
                                     "dropped_fc2_bias", "wrong_residual", "non_causal"])
def test_planted_mistakes_are_caught(monkeypatch, mistake):
    if mistake == "unbiased_variance":
        def ln(x, g, b):
            return (x - x.mean(-1, keepdim=True)) / torch.sqrt(x.var(-1, unbiased=True, keepdim=True) + 1e-5) * g + b
        monkeypatch.setattr(O, "layer_norm", ln)
    elif mistake == "no_query_scale":
        orig = O._qkv
        def qkv(u, lw, H, dt):
            q, k, v = orig(u, lw, H, dt)
            return q * math.sqrt(u.shape[-1] // H), k, v
        monkeypatch.setattr(O, "_qkv", qkv)
    elif mistake == "transposed_out_proj":
        orig = O._w
        marks = {}
        def wfn(t, dt):
            return orig(t, dt).T if (t.dim() == 2 and t.shape[0] == t.shape[1] and marks.get("on")) else orig(t, dt)
        marks["on"] = True
        monkeypatch.setattr(O, "_w", wfn)
    elif mistake == "dropped_fc2_bias":
        def ffn(r, lw, dt):
            u2 = O.layer_norm(r, lw["ln2_g"].to(dt), lw["ln2_b"].to(dt))
            return r + torch.relu(u2 @ lw["w_fc1"].to(dt).T + lw["b_fc1"].to(dt)) @ lw["w_fc2"].to(dt).T
        monkeypatch.setattr(O, "_ffn", ffn)
    elif mistake == "wrong_residual":
        def ffn(r, lw, dt):
            u2 = O.layer_norm(r, lw["ln2_g"].to(dt), lw["ln2_b"].to(dt))
            y = torch.relu(u2 @ lw["w_fc1"].to(dt).T + lw["b_fc1"].to(dt))
            return u2 + y @ lw["w_fc2"].to(dt).T + lw["b_fc2"].to(dt)
        monkeypatch.setattr(O, "_ffn", ffn)
    elif mistake == "non_causal":
        monkeypatch.setattr(torch, "triu", lambda x, diagonal=0: torch.zeros_like(x))
    gap, _ = hf_gap()
    assert gap > 1e-4, (mistake, gap)


# ---------------------------------------------------------------- ragged (left-padded) batches

def test_ragged_rows_match_library_opt_with_a_left_padded_mask():
    # the library model given a left-padded batch and its attention mask (positions counted from each
    # row's first real token) against the oracle's rows-on-their-own evaluation, full budget
    shape = toy_shape()
    w = toy_weights(shape)
    S, pad = 13, [0, 4, 9, 12]
    tokens = synth.make_tokens(shape.vocab, len(pad), S, seed=9)
    mask = torch.ones(len(pad), S, dtype=torch.long)
    for b, p in enumerate(pad):
        mask[b, :p] = 0
    ref = hf_logits(shape, w, tokens, attention_mask=mask)
    active = torch.ones(S, shape.n_layers, dtype=torch.bool)
    got = O.forward_ragged(w, shape.n_heads, tokens, pad, active, F64)
    for b, p in enumerate(pad):
        assert torch.isnan(got[b, :p]).all()
        assert float((got[b, p:] - ref[b, p:]).abs().max()) < 1e-9
    # and the pad tokens' identities are irrelevant
    other = tokens.clone()
    other[2, :9] = (other[2, :9] + 7) % shape.vocab
    again = O.forward_ragged(w, shape.n_heads, other, pad, active, F64)
    assert torch.equal(again[2, 9:], got[2, 9:])


def test_ragged_budget_goes_by_slot_not_by_row_position():
    # a row that starts late takes the layer set of the slot it sits in: with pad 0 the ragged evaluation
    # is the plain one, and a padded row equals the plain evaluation of its tokens under the shifted table
    shape = toy_shape(L=4)
    w = toy_weights(shape, seed=3)
    P, G = 6, 7
    n, _ = O.schedule(4, 1, 0, G, 4)
    active = O.active_matrix(4, P, n, 0)
    tokens = synth.make_tokens(shape.vocab, 2, P + G, seed=2)
    rag = O.forward_ragged(w, shape.n_heads, tokens, [0, 3], active, F64)
    plain = O.forward_sequence(w, shape.n_heads, tokens, active, F64)
    assert torch.equal(rag[0], plain[0])
    alone = O.forward_sequence(w, shape.n_heads, tokens[1:2, 3:], active[3:], F64)[0]
    assert torch.equal(rag[1, 3:], alone)
    # the shifted row really differs from running it with the unshifted table
    unshifted = O.forward_sequence(w, shape.n_heads, tokens[1:2, 3:], active[:P + G - 3], F64)[0]
    assert float((unshifted - alone).abs().max()) > 1e-6


def test_greedy_takes_the_lowest_index_of_the_maximum():
    # the decoding rule of the five configurations: argmax, exact ties to the lowest token id
    assert O.greedy(torch.tensor([[1.0, 3.0, 3.0, 2.0]])).tolist() == [1]
    assert O.greedy(torch.zeros(2, 9)).tolist() == [0, 0]                       # every entry ties
    assert O.greedy(torch.tensor([[5.0, 1.0, 5.0], [0.0, 1.0, 2.0], [2.0, 1.0, 0.0]])).tolist() == [0, 2, 0]
    x = torch.full((1, 50272), -1.0, dtype=torch.float64)
    x[0, 50271] = x[0, 777] = 4.0
    assert O.greedy(x).tolist() == [777]
    x[0, 50271] = 4.0 + 1e-12                                                   # no longer a tie
    assert O.greedy(x).tolist() == [50271]
    assert O.greedy(torch.tensor([[-float("inf"), -3.0, -3.0]])).tolist() == [1]
    assert O.greedy(x).dtype == torch.int32
    # against a scan written out by hand
    g = torch.Generator().manual_seed(3)
    r = torch.randint(0, 4, (6, 40), generator=g).double()                      # many exact ties
    want = [min(range(40), key=lambda i: (-float(row[i]), i)) for row in r]
    assert O.greedy(r).tolist() == want
