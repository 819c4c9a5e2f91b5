"""CPU-only checks of the library's host logic: exports, integer schedule, cache plan."""
import os
import re

import pytest

from oracle import skipdecode_oracle as O
from paper_2307_02628_b200 import binding, synth


def test_library_exports_every_declared_symbol(repo_root):
    hdr = open(os.path.join(repo_root, "include", "skipdecode.h")).read()
    declared = set(re.findall(r"\b(sd_[a-z_]+)\s*\(", hdr))
    assert declared == set(binding.EXPORTS)
    L = binding.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_binding_constants_are_the_headers(repo_root):
    # the ctypes binding restates the header's enumerators: option numbers, error codes, kernel classes
    hdr = open(os.path.join(repo_root, "include", "skipdecode.h")).read()
    enums = {name: int(value, 0) for name, value in re.findall(r"\b(SD_[A-Z0-9_]+)\s*=\s*(-?(?:0x[0-9a-fA-F]+|\d+))", hdr)}
    checked = 0
    for name, value in enums.items():
        if hasattr(binding, name):
            assert getattr(binding, name) == value, name
            checked += 1
    assert checked >= 15
    for name in ("SD_OPT_GRAPHS", "SD_OPT_ATTN_CHUNK", "SD_OPT_GEMM", "SD_OPT_TIMING", "SD_OPT_PDL", "SD_OPT_PREFILL_ATTN",
                 "SD_OPT_GEMM_PERSISTENT", "SD_OPT_GEMM_SPLITK", "SD_OPT_DETERMINISTIC", "SD_OPT_TEST_WAIT_EXPIRY",
                 "SD_OPT_ATTN_STAGED"):
        assert name in enums and hasattr(binding, name), name
    classes = [n for n in enums if n.startswith("SD_K_") and n != "SD_K_COUNT"]
    assert enums["SD_K_COUNT"] == len(classes) == len(binding.KERNEL_CLASSES)


SCHEDULES = [(4, 4, 2, 0, 32), (12, 12, 4, 0, 128), (24, 24, 8, 0, 256), (32, 32, 8, 0, 512), (32, 32, 4, 0, 1024),
             (32, 22, 11, 1, 1024), (32, 14, 8, 1, 512), (32, 10, 6, 1, 100), (32, 8, 5, 1, 1024),
             (24, 16, 8, 1, 512), (24, 10, 6, 1, 100), (24, 7, 5, 1, 37), (24, 6, 4, 1, 3),
             (7, 7, 7, 0, 5), (9, 8, 2, 1, 1), (9, 8, 2, 1, 2), (40, 39, 3, 2, 2047)]


@pytest.mark.parametrize("L,mx,mn,w,G", SCHEDULES)
def test_schedule_is_bit_exact_with_the_oracle(L, mx, mn, w, G):
    n, top = binding.schedule_compute(L, mx, mn, w, G)
    n_ref, top_ref = O.schedule(mx, mn, w, G, L)
    assert n == n_ref and top == top_ref


@pytest.mark.parametrize("args", [(4, 5, 2, 0, 8), (8, 4, 5, 0, 8), (8, 4, 2, 2, 8), (8, 4, 2, 0, 0), (8, 4, 2, -1, 8)])
def test_schedule_rejects_bad_arguments(args):
    with pytest.raises(binding.SdError) as e:
        binding.schedule_compute(*args)
    assert e.value.code == binding.SD_ERR_ARG


def test_table2_presets_are_the_papers_rows():
    # every preset workload carries the (warm-up, min, max) of its row of Table 2 and the schedule's mean
    # layer count is the row's midpoint, the figure the target speed-up is computed from
    import os
    rows = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "table2_budgets.txt")):
        if line.strip() and not line.startswith("#"):
            base, speed, avg, warm, mn, mx = line.split()
            rows[(int(base), int(speed))] = (int(warm), int(mn), int(mx))
    assert len(rows) == 8
    seen = 0
    for name, wl in synth.CONFIGS.items():
        if not name.startswith("t2-"):
            continue
        _, model, speed, ds = name.split("-")
        assert (wl.warmup, wl.min_layers, wl.max_layers) == rows[(wl.shape.n_layers, int(speed[0]))]
        assert (wl.prompt_len, wl.gen_len) == synth.ENVELOPES[ds] and wl.prompt_len + wl.gen_len <= wl.shape.max_pos
        n, top = binding.schedule_compute(wl.shape.n_layers, wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len)
        assert abs(sum(n) / len(n) - (wl.max_layers + wl.min_layers) / 2) <= 0.5 / len(n) + 1e-9 or wl.gen_len % 2 == 0
        assert n[0] == wl.max_layers and n[-1] == wl.min_layers
        seen += 1
    assert seen == 24


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4", "c5"])
def test_cache_plan_matches_the_active_sets(name):
    wl = synth.CONFIGS[name]
    cfg = binding.make_config(wl.shape, wl.batch, wl.prompt_len, wl.gen_len)
    plan = binding.SdPlan(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len, 0)
    cap = binding.layer_capacity(cfg, plan)
    n, _ = O.schedule(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len, wl.shape.n_layers)
    act = O.active_matrix(wl.shape.n_layers, wl.prompt_len, n, wl.warmup)
    assert cap == [int(c) for c in act.sum(0)]          # positions at which each layer ever runs
    full = binding.layer_capacity(cfg, binding.SdPlan(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len, 1))
    assert full == [wl.prompt_len + wl.gen_len] * wl.shape.n_layers
    e = 4 if wl.shape.dtype == "fp32" else 2
    kv = 2 * sum(cap) * wl.batch * wl.shape.d_model * e
    total = binding.arena_bytes(cfg, plan)
    s = wl.shape
    packed = 0                                          # bf16 mode keeps a tile-packed copy of every weight matrix
    if s.dtype == "bf16":
        packed = 2 * (s.n_layers * (4 * s.d_model ** 2 + 2 * s.d_model * s.d_ffn) + (s.vocab + 255) // 256 * 256 * s.d_model)
    assert kv + packed <= total <= kv + packed + (2 << 30)   # the rest (activations, partials) is bounded


def test_config_validation():
    shape = synth.TINY
    plan = binding.SdPlan(4, 2, 0, 8, 0)
    for bad in (dict(n_heads=3), dict(d_model=250), dict(max_prompt=100, max_gen=100), dict(dtype=2), dict(max_batch=0)):
        cfg = binding.make_config(shape, 2, 8, 8)
        for k, v in bad.items():
            setattr(cfg, k, v)
        with pytest.raises(binding.SdError):
            binding.arena_bytes(cfg, plan)
    cfg = binding.make_config(shape, 2, 8, 8)
    with pytest.raises(binding.SdError):
        binding.arena_bytes(cfg, binding.SdPlan(4, 2, 0, 9, 0))     # plan longer than max_gen
    assert binding.lib().sd_strerror(binding.SD_ERR_POSITION).decode().startswith("position")


@pytest.mark.parametrize("L,mx,mn,w,G,alpha", [(32, 32, 8, 0, 512, 1), (32, 32, 8, 0, 512, 2), (32, 22, 11, 1, 1024, 3),
                                                 (24, 16, 8, 1, 2047, 4), (12, 12, 4, 0, 1, 2), (12, 12, 4, 0, 2, 8)])
def test_power_law_schedule_is_bit_exact_with_the_oracle(L, mx, mn, w, G, alpha):
    assert binding.schedule_power_compute(L, mx, mn, w, G, alpha) == tuple(O.schedule_power(mx, mn, w, G, L, alpha))


def test_power_law_schedule_rejects_what_its_integers_cannot_hold():
    # (G-1)^8 * 2 (max - min) passes 2^124 near G = 2^15: refused instead of wrapping around
    with pytest.raises(binding.SdError) as e:
        binding.schedule_power_compute(32, 32, 4, 0, 65536, 8)
    assert e.value.code == binding.SD_ERR_ARG
    # well inside the limit the table is still the oracle's
    assert binding.schedule_power_compute(32, 32, 4, 0, 4097, 8) == tuple(O.schedule_power(32, 4, 0, 4097, 32, 8))
    assert binding.schedule_power_compute(32, 32, 4, 0, 65536, 4) == tuple(O.schedule_power(32, 4, 0, 65536, 32, 4))


def test_bf16_weights_are_fp16_values_inside_the_fp16_range():
    # What the packed weight copies rely on: a bf16 has 8 significant bits, an fp16 has 11, so every bf16 whose
    # magnitude lies in [2^-14, 65504] is an fp16 value exactly; below that it lands on the fp16 subnormal grid
    # (spacing 2^-24, error at most 2^-25); above it the conversion has to clip.  All 65 536 bit patterns.
    import torch
    bits = torch.arange(65536, dtype=torch.int32).to(torch.int16)
    v = bits.view(torch.bfloat16).to(torch.float64)
    finite = torch.isfinite(v)
    mag = v.abs()
    normal = finite & (mag >= 2.0 ** -14) & (mag <= 65504.0)
    as_f16 = v.to(torch.float16).to(torch.float64)
    assert int(normal.sum()) == 2 * 30 * 128                # 30 binades, 128 mantissas, two signs
    assert torch.equal(as_f16[normal], v[normal])
    small = finite & (mag < 2.0 ** -14)
    assert float((as_f16[small] - v[small]).abs().max()) <= 2.0 ** -25
    big = finite & (mag > 65504.0)
    assert bool(torch.isinf(as_f16[big]).all())              # a plain conversion overflows: the pack kernel saturates instead
    # the largest bf16 below the limit is exactly representable, the next one is not
    assert float(v[normal].abs().max()) == 65280.0
