"""Parity of the device token selection (temperature + top-p, Section 3.2's settings) with the oracle.

Both sides receive the same fp32 logits and the same uniform numbers.  A draw is an integer
decided by floating point: the device weighs tokens with a single-precision exponential and
2^-40 fixed-point sums, the oracle in float64, so a target that falls within rounding of a
boundary may pick the neighbouring token.  The bar: the same token on >= 99 % of the rows, and
every other row's token inside the oracle's nucleus at a rank next to the oracle's.
"""
import pytest
import torch

import harness
from oracle import skipdecode_oracle as O
from paper_2307_02628_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _draw(dec, logits, uniforms, temperature, top_p):
    got = dec.sample_top_p(logits.to(dec.device), uniforms.to(dec.device), temperature, top_p)
    dec.synchronize()          # the library's stream, not torch's current one
    return got.cpu()


def _compare(dec, logits, uniforms, temperature, top_p):
    got = _draw(dec, logits, uniforms, temperature, top_p)
    ref = O.sample_top_p(logits, uniforms.double(), temperature, top_p)
    same = int((got == ref).sum())
    for b in torch.nonzero(got != ref).flatten().tolist():
        order, _, k = O.nucleus(logits[b], temperature, top_p)
        rank = {int(t): i for i, t in enumerate(order[:k].tolist())}
        assert int(got[b]) in rank, (b, int(got[b]))
        assert abs(rank[int(got[b])] - rank[int(ref[b])]) <= 1, (b, int(got[b]), int(ref[b]))
    assert same >= 0.99 * len(ref), (same, len(ref))
    return same, len(ref)


@pytest.fixture(scope="module")
def dec_full_vocab():
    wl = synth.CONFIGS["c2"]
    dec = harness.make_decoder(wl, synth.make_weights(wl.shape, seed=0))
    yield dec, wl
    dec.close()


@pytest.mark.parametrize("scale,step", [(0.6, 0.0), (3.0, 0.0), (1.0, 0.25), (0.05, 0.0)])
@pytest.mark.parametrize("temperature,top_p", [(0.3, 0.7), (1.0, 0.9), (1.0, 1.0), (0.7, 0.05)])
def test_sampling_full_vocabulary(dec_full_vocab, scale, step, temperature, top_p):
    dec, wl = dec_full_vocab
    B = 64
    logits = synth.make_logits(B, wl.shape.vocab, seed=17, scale=scale, step=step)
    u = synth.make_uniforms(B, seed=23)
    same, n = _compare(dec, logits, u, temperature, top_p)
    print(f"scale {scale} step {step} T {temperature} p {top_p}: {same}/{n} identical")


def test_sampling_edges(dec_full_vocab):
    dec, wl = dec_full_vocab
    V = wl.shape.vocab
    logits = synth.make_logits(8, V, seed=5, scale=1.0)
    # u = 0 is the most probable token; u just below 1 the last token of the nucleus
    zero = torch.zeros(8)
    got = _draw(dec, logits, zero, 0.3, 0.7)
    assert torch.equal(got, O.greedy(logits))
    _compare(dec, logits, torch.full((8,), 0.99999994), 0.3, 0.7)
    # one row, and a row where every logit is the same value: tokens come in id order
    flat = torch.zeros(1, V)
    for u in (0.0, 0.3, 0.999):
        got = _draw(dec, flat, torch.tensor([u]), 1.0, 1.0)
        assert int(got) == int(O.sample_top_p(flat, torch.tensor([u], dtype=torch.float32).double(), 1.0, 1.0))
    # a maximum that dwarfs the rest is always chosen; -inf entries are never chosen
    spike = synth.make_logits(4, V, seed=6, scale=1.0)
    spike[:, 123] = 80.0
    spike[:, 7] = float("-inf")
    got = _draw(dec, spike, synth.make_uniforms(4, 1), 1.0, 1.0)
    assert got.tolist() == [123] * 4
    # invalid settings are rejected on the host
    for t, p in ((0.0, 0.7), (-1.0, 0.7), (0.3, 0.0), (0.3, 1.5), (float("nan"), 0.7)):
        with pytest.raises(binding.SdError):
            dec.sample_top_p(logits.to(dec.device), zero.to(dec.device), t, p)
    assert dec.status() == 0


def test_sampling_small_vocabulary_and_generation():
    # vocabulary smaller than the block; then a sampled generation whose every step is checked
    wl = synth.CONFIGS["c1"]
    w = synth.make_weights(wl.shape, seed=0)
    dec = harness.make_decoder(wl, w)
    logits = synth.make_logits(wl.batch, wl.shape.vocab, seed=9, scale=2.0)
    _compare(dec, logits, synth.make_uniforms(wl.batch, 3), 0.3, 0.7)
    ref = O.CachedDecoder(w, wl.shape.n_heads)
    ref.set_schedule(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len)
    prompts = synth.make_prompts(wl)
    dec.schedule(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len)
    lg = dec.prefill(prompts)
    lr = ref.prefill(prompts)
    agree = 0
    for g in range(wl.gen_len):
        u = synth.make_uniforms(wl.batch, 100 + g)
        ids = dec.sample_top_p(lg, u.to(dec.device), 0.3, 0.7)
        dec.synchronize()
        ids_ref = O.sample_top_p(lr, u.double(), 0.3, 0.7)
        agree += int((ids.cpu() == ids_ref).sum())
        # both sides continue from the oracle's choice, so every step is an independent comparison
        lg = dec.decode_step(ids_ref.to(dec.device), wl.prompt_len + g)
        lr = ref.decode_step(ids_ref, wl.prompt_len + g)
    dec.close()
    assert agree >= 0.99 * wl.batch * wl.gen_len, agree


def test_sampling_vocabulary_too_large_for_shared_memory():
    # above 52 224 entries the row is not staged in shared memory and every pass reads it from global memory
    shape = synth.ModelShape("toy-big-vocab", 1, 64, 1, 128, 60001, 16, "bf16")
    wl = synth.Workload(shape, 6, 4, 2, 1, 1, 0)
    dec = harness.make_decoder(wl, synth.make_weights(shape, seed=1))
    for scale, step, temperature, top_p in ((1.0, 0.0, 0.3, 0.7), (2.0, 0.5, 1.0, 0.95), (0.2, 0.0, 0.3, 1.0)):
        logits = synth.make_logits(6, shape.vocab, seed=31, scale=scale, step=step)
        same, n = _compare(dec, logits, synth.make_uniforms(6, seed=32), temperature, top_p)
        assert same == n
    dec.close()
