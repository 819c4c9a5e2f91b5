"""The decode-attention kernel that stages K and V through shared memory (bf16 storage).

The library gives a decode step's attention to that kernel only when the launch has at least 12 (row, head)
pairs per SM and the handle is configured for at least 1024 positions, so the cases here are small models with
many rows and heads, run with SD_OPT_ATTN_STAGED = 2 (no length condition) and with 0 (the register-only
kernel); both must match the CPU oracle, and each other up to summation order.  One case is configured for
1024 positions and runs on the default setting."""
import pytest
import torch

import harness
import test_gpu_ragged as ragged
from paper_2307_02628_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _pairs_needed():
    return 12 * torch.cuda.get_device_properties(0).multi_processor_count


@pytest.mark.parametrize("hd,heads,B", [(32, 32, 64), (64, 16, 120), (128, 16, 112)])
@pytest.mark.parametrize("chunk", [0, 32])
def test_staged_kernel_matches_the_oracle_and_the_register_kernel(hd, heads, B, chunk):
    # chunk 32: several splits per (row, head), merged by the block that arrives last; the last split is ragged
    if B * heads < _pairs_needed():
        pytest.skip("this GPU has more SMs than the case was sized for")
    shape = synth.ModelShape(f"staged-hd{hd}", 2, hd * heads, heads, 1024, 640, 128, "bf16")
    wl = synth.Workload(shape, B, 70, 5, 2, 1, 0)
    w = synth.make_weights(shape, seed=21, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    rows = synth.sample_rows(B, 6)
    ref = harness.oracle_run_forced(wl, w, prompts, forced, rows=rows)
    runs = {}
    for staged in (2, 0):
        dec = harness.make_decoder(wl, w)
        dec.set_option(binding.SD_OPT_ATTN_STAGED, staged)
        dec.set_option(binding.SD_OPT_ATTN_CHUNK, chunk)
        runs[staged] = harness.gpu_run_forced(dec, wl, prompts, forced, rows=rows)
        dec.close()
        err, strict, near = harness.compare(runs[staged], ref, harness.TOL["bf16"])
        print(f"hd={hd} chunk={chunk} staged={staged}: max|err|={err:.3e} argmax strict={strict:.4f} near={near:.4f}")
        assert err <= harness.TOL["bf16"] and near >= 0.99
    assert float((runs[2] - runs[0]).abs().max()) <= harness.REORDER_TOL


def test_staged_kernel_with_left_padding_and_retired_rows():
    # 64 rows x 32 heads; paddings from none to all but one prompt slot; four rows stop after step 2 (60 x 32 pairs
    # is still a staged launch)
    B, heads = 64, 32
    if (B - 4) * heads < _pairs_needed():
        pytest.skip("this GPU has more SMs than the case was sized for")
    shape = synth.ModelShape("staged-ragged", 2, 1024, heads, 1024, 640, 128, "bf16")
    g = torch.Generator().manual_seed(5)
    pad = torch.randint(0, 70, (B,), generator=g).tolist()
    pad[0], pad[1], pad[2] = 0, 69, 33
    keep = [r for r in range(B) if r not in (3, 17, 40, 63)]
    err = ragged._run(shape, B, 70, 5, 2, 1, 0, pad=pad, retire={2: keep}, seed=22, options={binding.SD_OPT_ATTN_STAGED: 2})
    print("staged, ragged: max|err| =", err)
    assert err <= harness.TOL["bf16"]


def test_default_setting_on_a_handle_configured_for_1024_positions():
    # prompt 1000 + 24 generated positions: the default rule (many pairs and at least 1024 positions) picks the staged
    # kernel by itself; rows of 1001..1024 keys are 32 stages each, the last one ragged
    B, heads = 64, 32
    if B * heads < _pairs_needed():
        pytest.skip("this GPU has more SMs than the case was sized for")
    shape = synth.ModelShape("staged-long", 2, 1024, heads, 1024, 640, 1024, "bf16")
    wl = synth.Workload(shape, B, 1000, 24, 2, 1, 0)
    w = synth.make_weights(shape, seed=23, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    rows = [0, 63]
    ref = harness.oracle_run_forced(wl, w, prompts, forced, rows=rows)
    runs = {}
    for staged in (1, 0):
        dec = harness.make_decoder(wl, w)
        dec.set_option(binding.SD_OPT_ATTN_STAGED, staged)
        runs[staged] = harness.gpu_run_forced(dec, wl, prompts, forced, rows=rows)
        dec.close()
        err, strict, near = harness.compare(runs[staged], ref, harness.TOL["bf16"])
        print(f"1024 positions staged={staged}: max|err|={err:.3e} argmax strict={strict:.4f} near={near:.4f}")
        assert err <= harness.TOL["bf16"] and near >= 0.99
    assert float((runs[1] - runs[0]).abs().max()) <= harness.REORDER_TOL

