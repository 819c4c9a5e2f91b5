"""Shared helpers of the parity tests: run the CUDA library and the CPU oracle on the
same seeded inputs and compare them."""
from __future__ import annotations

import torch

from oracle import skipdecode_oracle as O
from paper_2307_02628_b200 import synth

TOL = {"fp32": 1e-4, "bf16": 3e-2}     # max-abs logit error allowed per storage type
# Two GPU runs of the same products in bf16 storage that add their fp32 partial sums in a different order
# (atomic adds in arrival order, another K split, another attention split) differ in the last bits of those
# sums; where such a sum is then rounded into the bf16 cache or an fp16 operand, a value near a rounding
# boundary can land on either side, which moves a logit by up to a few 1e-3 at the tested sizes (2.1e-3 seen).
REORDER_TOL = 5e-3


def make_decoder(wl: synth.Workload, weights, full_capacity=False, **kw):
    from paper_2307_02628_b200 import binding
    return binding.Decoder(wl.shape, weights, wl.batch, wl.prompt_len, wl.gen_len,
                           plan=(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len),
                           full_capacity=full_capacity, **kw)


def gpu_run_forced(dec, wl: synth.Workload, prompts, forced, rows=None, table=None):
    """Prefill + gen_len decode steps feeding forced[:, g] at step g.
    Returns fp32 CPU logits [len(rows), gen_len + 1, vocab] (index 0 = prefill)."""
    B, G = wl.batch, wl.gen_len
    rows = list(range(B)) if rows is None else rows
    ridx = torch.tensor(rows, device=dec.device)
    out = torch.empty(len(rows), G + 1, wl.shape.vocab, dtype=torch.float32)
    with torch.cuda.stream(dec.stream):
        if table is None:
            dec.schedule(wl.max_layers, wl.min_layers, wl.warmup, G)
        else:
            dec.schedule_custom(table, wl.warmup)       # caller-supplied budget per generated position
        logits = dec.prefill(prompts)
        out[:, 0] = logits[ridx].cpu()
        forced_d = forced.to(dec.device)
        buf = torch.empty(B, wl.shape.vocab, dtype=torch.float32, device=dec.device)
        for g in range(G):
            dec.decode_step(forced_d[:, g].contiguous(), wl.prompt_len + g, buf)
            out[:, g + 1] = buf[ridx].cpu()
    assert dec.status() == 0
    return out


def oracle_run_forced(wl: synth.Workload, weights, prompts, forced, rows=None, dtype=torch.float64, table=None):
    """The definition on the same token sequences: logits [len(rows), gen_len + 1, vocab]."""
    rows = list(range(wl.batch)) if rows is None else rows
    n = table if table is not None else O.schedule(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len, wl.shape.n_layers)[0]
    act = O.active_matrix(wl.shape.n_layers, wl.prompt_len, n, wl.warmup)
    seq = torch.cat([prompts, forced], dim=1)[rows]
    # the token fed at the last step produces logits for a position nobody consumes; keep it anyway
    return O.forward_sequence(weights, wl.shape.n_heads, seq, act, dtype, logits_from=wl.prompt_len - 1)


def oracle_greedy(wl: synth.Workload, weights, prompts, dtype=torch.float64):
    """Greedy generation by the cached oracle: (logits [B, G+1, V], tokens fed [B, G])."""
    dec = O.CachedDecoder(weights, wl.shape.n_heads, dtype)
    dec.set_schedule(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len)
    logits = [dec.prefill(prompts)]
    fed = []
    for g in range(wl.gen_len):
        ids = O.greedy(logits[-1])
        fed.append(ids)
        logits.append(dec.decode_step(ids, wl.prompt_len + g))
    return torch.stack(logits, dim=1), torch.stack(fed, dim=1)


def compare(gpu_logits, ref_logits, tol):
    """Returns (max abs error, strict argmax agreement, agreement counting near-ties)."""
    ref = ref_logits.to(torch.float64)
    got = gpu_logits.to(torch.float64)
    err = float((got - ref).abs().max())
    a, b = got.argmax(-1), ref.argmax(-1)
    strict = float((a == b).double().mean())
    # a differing choice is a near-tie when the oracle scores it within 2*tol of its own maximum
    chosen = ref.gather(-1, a.unsqueeze(-1)).squeeze(-1)
    near = ((a == b) | (chosen >= ref.max(-1).values - 2 * tol)).double().mean()
    return err, strict, float(near)
