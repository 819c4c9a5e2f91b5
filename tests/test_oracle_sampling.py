"""Pins for the oracle's top-p sampling (Section 3.2: beam 1, top-p 0.7, temperature 0.3)."""
import itertools
import math

import pytest
import torch

from oracle import skipdecode_oracle as orc


def _rows(n, vocab, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(n, vocab, generator=g) * scale


def test_nucleus_is_the_smallest_set_by_exhaustive_search():
    # every subset of a 7-token vocabulary: the nucleus must have the minimum size among the subsets whose
    # probability reaches top_p, and the largest probability among the subsets of that size
    for seed, top_p, temp in itertools.product(range(6), (0.3, 0.7, 0.95), (0.3, 1.0)):
        row = _rows(1, 7, seed, 2.0)[0]
        e = [math.exp(float(v) / temp) for v in row]
        z = sum(e)
        p = [v / z for v in e]
        best = None
        for size in range(1, 8):
            reach = [(sum(p[i] for i in s), s) for s in itertools.combinations(range(7), size)
                     if sum(p[i] for i in s) >= top_p]
            if reach:
                best = max(reach)
                break
        order, sorted_probs, k = orc.nucleus(row, temp, top_p)
        assert k == len(best[1])
        assert sorted(order[:k].tolist()) == sorted(best[1])
        assert abs(float(sorted_probs[:k].sum()) - best[0]) < 1e-12


def test_nucleus_matches_the_library_warpers():
    tr = pytest.importorskip("transformers")
    from transformers.generation.logits_process import TemperatureLogitsWarper, TopPLogitsWarper
    rows = _rows(8, 500, 11, 3.0)
    for temp, top_p in ((0.3, 0.7), (1.0, 0.9), (0.7, 0.5)):
        warped = TopPLogitsWarper(top_p=top_p)(None, TemperatureLogitsWarper(temp)(None, rows.clone()))
        for b in range(rows.shape[0]):
            kept = set(torch.nonzero(torch.isfinite(warped[b])).flatten().tolist())
            order, _, k = orc.nucleus(rows[b], temp, top_p)
            assert set(order[:k].tolist()) == kept


def test_equally_spaced_uniforms_reproduce_the_renormalised_distribution():
    n = 20000
    u = (torch.arange(n, dtype=torch.float64) + 0.5) / n
    for temp, top_p in ((0.3, 0.7), (1.0, 1.0), (1.0, 0.6)):
        row = _rows(1, 40, 5, 1.5)[0]
        picks = orc.sample_top_p(row.expand(n, -1), u, temp, top_p)
        counts = torch.bincount(picks.long(), minlength=40).double()
        p = torch.softmax(row.double() / temp, 0)
        order, _, k = orc.nucleus(row, temp, top_p)
        inside = torch.zeros(40, dtype=torch.bool)
        inside[order[:k]] = True
        assert counts[~inside].sum() == 0
        expect = torch.where(inside, p, torch.zeros_like(p))
        expect = expect / expect.sum() * n
        assert float((counts - expect).abs().max()) <= 1.0 + 1e-9
        # the chosen token's rank never decreases as the random number grows
        rank = torch.empty(40, dtype=torch.long)
        rank[order] = torch.arange(40)
        r = rank[picks.long()]
        assert bool((r[1:] >= r[:-1]).all())


def test_limits_reduce_to_argmax():
    rows = _rows(16, 300, 3, 2.0)
    u = torch.rand(16, generator=torch.Generator().manual_seed(1), dtype=torch.float64)
    top = orc.greedy(rows)
    # a nucleus no larger than the most probable token's own mass is that token alone
    pmax = torch.softmax(rows.double(), 1).max(1).values.min()
    assert torch.equal(orc.sample_top_p(rows, u, 1.0, float(pmax) * 0.999), top)
    # a vanishing temperature concentrates all mass on the maximum
    assert torch.equal(orc.sample_top_p(rows, u, 1e-3, 0.7), top)
    # u = 0 always selects the most probable token
    assert torch.equal(orc.sample_top_p(rows, torch.zeros(16), 0.3, 0.7), top)


def test_ties_take_the_lower_token_first():
    row = torch.tensor([0.0, 1.0, 1.0, 1.0, -2.0])
    order, _, k = orc.nucleus(row, 1.0, 0.5)
    assert order[:3].tolist() == [1, 2, 3] and k == 2
    assert int(orc.sample_top_p(row[None], torch.tensor([0.49]), 1.0, 0.5)) == 1
    assert int(orc.sample_top_p(row[None], torch.tensor([0.51]), 1.0, 0.5)) == 2
