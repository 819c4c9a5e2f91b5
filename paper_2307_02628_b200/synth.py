"""Seeded synthetic inputs: model shapes, random-init weights, prompts, forced tokens.

This module holds no arithmetic of the method.  It only draws numbers: the
tests hand the same tensors to the CPU oracle and to the CUDA library.

Workloads.  The paper evaluates OPT-1.3B (24 layers) and OPT-6.7B (32 layers)
on E2E, Reddit-TLDR and CNN-DM (Section 3, dataset paragraph: prompts up to
60 / 512 / 1024 tokens, sequences up to 160 / 1024 / 2048).  Neither the data
nor trained weights are used here; the five configurations below stand in for
them by shape, with uniform-random token ids and N(0, 0.02) random weights.
Every kernel on the decode path has data-independent control flow, so values
do not change its cost.

Recipe.  Each tensor owns a torch CPU generator seeded from (seed, tensor
name), so tensors can be drawn in any order or in parallel and stay
bit-identical.  Matrices, embeddings and biases are N(0, std); LayerNorm gains
are 1 and offsets 0 unless `random_ln` is set.  For a bf16 configuration the
fp32 draw is rounded once to bf16 (nearest-even) and those bytes go to both
sides.
"""
from __future__ import annotations

import hashlib
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace

import torch

from .shapes import ModelShape, storage_dtype  # noqa: F401  (re-exported)


@dataclass(frozen=True)
class Workload:
    """One configuration: model shape + batch, prompt, generation and schedule."""
    shape: ModelShape
    batch: int
    prompt_len: int
    gen_len: int
    max_layers: int
    min_layers: int
    warmup: int = 0

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


TINY = ModelShape("tiny-fp32", 4, 256, 4, 1024, 1024, 128, "fp32")
OPT_125M = ModelShape("opt-125m", 12, 768, 12, 3072, 50272, 2048, "bf16")
OPT_1B3 = ModelShape("opt-1.3b", 24, 2048, 32, 8192, 50272, 2048, "bf16")
OPT_6B7 = ModelShape("opt-6.7b", 32, 4096, 32, 16384, 50272, 2048, "bf16")

CONFIGS = {
    "c1": Workload(TINY, 4, 32, 32, 4, 2),
    "c2": Workload(OPT_125M, 8, 128, 128, 12, 4),
    "c3": Workload(OPT_1B3, 32, 512, 256, 24, 8),
    "c4": Workload(OPT_6B7, 64, 1024, 512, 32, 8),
    "c5": Workload(OPT_6B7, 256, 256, 1024, 32, 4),
    # profiler case: config 4's kernels (same d, heads, batch, prompt, hence the same attention and GEMM
    # launches) on a 2-layer model, so that a counter capture holds a few GB instead of 60
    "c4-2layer": Workload(ModelShape("opt-6.7b-2layer", 2, 4096, 32, 16384, 50272, 2048, "bf16"), 64, 1024, 16, 2, 2),
    # the same for config 5's launches (batch 256: the tensor-bound GEMM regime)
    "c5-2layer": Workload(ModelShape("opt-6.7b-2layer", 2, 4096, 32, 16384, 50272, 2048, "bf16"), 256, 256, 16, 2, 2),
}


# Table 2's presets (base layers -> {target speed-up: (warm-up, min, max)}) at the sequence envelopes of
# the paper's three datasets (Section 3.2: prompt / total length 60/160, 512/1024, 1024/2048), batch 64:
# "t2-6.7b-3x-reddit" and so on.  Same synthetic tokens and weights as the five configurations above.
TABLE2 = {"6.7b": (OPT_6B7, {2: (1, 11, 22), 3: (1, 8, 14), 4: (1, 6, 10), 5: (1, 5, 8)}),
          "1.3b": (OPT_1B3, {2: (1, 8, 16), 3: (1, 6, 10), 4: (1, 5, 7), 5: (1, 4, 6)})}
ENVELOPES = {"e2e": (60, 100), "reddit": (512, 512), "cnndm": (1024, 1024)}
for _model, (_shape, _rows) in TABLE2.items():
    for _k, (_w, _mn, _mx) in _rows.items():
        for _ds, (_p, _g) in ENVELOPES.items():
            CONFIGS[f"t2-{_model}-{_k}x-{_ds}"] = Workload(_shape, 64, _p, _g, _mx, _mn, _w)


def _seed_for(seed: int, name: str) -> int:
    h = hashlib.sha256(f"{seed}:{name}".encode()).digest()
    return int.from_bytes(h[:8], "little") & 0x7FFFFFFFFFFFFFFF


def _normal(seed: int, name: str, shape, std: float, dtype: torch.dtype) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(_seed_for(seed, name))
    t = torch.empty(shape, dtype=torch.float32)
    t.normal_(0.0, std, generator=g)
    return t.to(dtype)


def make_weights(shape: ModelShape, seed: int = 0, std: float = 0.02,
                 random_ln: bool = False, threads: int = 8) -> dict:
    """Random-init weights as CPU tensors in the configuration's storage type.

    Layout (row-major [out, in], as a linear layer stores it):
      tok_emb [V,d], pos_emb [max_pos,d], lnf_g [d], lnf_b [d],
      layers[l]: ln1_g, ln1_b [d]; w_qkv [3d,d] (rows ordered q,k,v), b_qkv [3d];
                 w_o [d,d], b_o [d]; ln2_g, ln2_b [d]; w_fc1 [f,d], b_fc1 [f];
                 w_fc2 [d,f], b_fc2 [d].
    The LM head is tied to tok_emb.
    """
    dt = storage_dtype(shape)
    d, f, V = shape.d_model, shape.d_ffn, shape.vocab
    jobs = {("tok_emb",): ((V, d), "n"), ("pos_emb",): ((shape.max_pos, d), "n"),
            ("lnf_g",): ((d,), "g"), ("lnf_b",): ((d,), "b")}
    for l in range(shape.n_layers):
        for nm, shp, kind in (("ln1_g", (d,), "g"), ("ln1_b", (d,), "b"),
                              ("w_qkv", (3 * d, d), "n"), ("b_qkv", (3 * d,), "n"),
                              ("w_o", (d, d), "n"), ("b_o", (d,), "n"),
                              ("ln2_g", (d,), "g"), ("ln2_b", (d,), "b"),
                              ("w_fc1", (f, d), "n"), ("b_fc1", (f,), "n"),
                              ("w_fc2", (d, f), "n"), ("b_fc2", (d,), "n")):
            jobs[("layers", l, nm)] = (shp, kind)

    def draw(item):
        key, (shp, kind) = item
        name = ".".join(str(k) for k in key)
        if kind == "n":
            return key, _normal(seed, name, shp, std, dt)
        if kind == "g":
            if random_ln:
                return key, (1.0 + _normal(seed, name, shp, 0.1, torch.float32)).to(dt)
            return key, torch.ones(shp, dtype=dt)
        if random_ln:
            return key, _normal(seed, name, shp, 0.1, dt)
        return key, torch.zeros(shp, dtype=dt)

    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        drawn = list(ex.map(draw, jobs.items()))
    w: dict = {"layers": [dict() for _ in range(shape.n_layers)]}
    for key, t in drawn:
        if key[0] == "layers":
            w["layers"][key[1]][key[2]] = t
        else:
            w[key[0]] = t
    return w


def make_tokens(vocab: int, batch: int, length: int, seed: int) -> torch.Tensor:
    """Uniform-random token ids, int32 [batch, length]."""
    g = torch.Generator(device="cpu")
    g.manual_seed(_seed_for(seed, f"tokens:{batch}x{length}"))
    return torch.randint(0, vocab, (batch, length), generator=g, dtype=torch.int64).to(torch.int32)


def make_prompts(wl: Workload, seed: int = 1) -> torch.Tensor:
    return make_tokens(wl.shape.vocab, wl.batch, wl.prompt_len, seed)


def make_forced_tokens(wl: Workload, seed: int = 3) -> torch.Tensor:
    """Token ids fed at the gen_len decode steps when a run is teacher-forced
    with random ids rather than with greedy choices: int32 [batch, gen_len]."""
    return make_tokens(wl.shape.vocab, wl.batch, wl.gen_len, seed)


def sample_rows(batch: int, count: int, seed: int = 2) -> list:
    """First, last and seeded-random batch rows, `count` of them, sorted."""
    if count <= 1 or batch == 1:
        return [0]
    rows = {0, batch - 1}
    g = torch.Generator(device="cpu")
    g.manual_seed(_seed_for(seed, f"rows:{batch}"))
    perm = torch.randperm(batch, generator=g).tolist()
    for r in perm:
        if len(rows) >= min(count, batch):
            break
        rows.add(r)
    return sorted(rows)


def make_logits(batch: int, vocab: int, seed: int, scale: float = 1.0, step: float = 0.0) -> torch.Tensor:
    """Stand-in logits for the token-selection tests: N(0, scale) fp32 [batch, vocab]; with
    step > 0 they are rounded to multiples of `step`, which makes many of them equal."""
    t = _normal(seed, f"logits:{batch}x{vocab}", (batch, vocab), scale, torch.float32)
    if step > 0:
        t = torch.round(t / step) * step
    return t


def make_uniforms(batch: int, seed: int) -> torch.Tensor:
    """The random numbers of one sampling step: fp32 [batch] in [0, 1)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(_seed_for(seed, f"uniforms:{batch}"))
    return torch.rand(batch, generator=g, dtype=torch.float32)
