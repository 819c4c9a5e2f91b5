"""sd_decode_step_static: the decode step for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits: inside a host application
that owns all device memory, or in a serving loop that must not allocate after start-up.  For them the library offers one entry point whose only scratch
(the split-KV attention partials) sits in an array inside the library image.  This test
calls it through the C ABI on two consecutive decode steps and checks each against
sd_decode_step on the same inputs (the two run the same kernels, so they may differ only by the
order in which split sums arrive: 5e-3 in bf16 storage, 1e-5 in fp32) and against the CPU oracle
with the tolerance of the other parity tests.

It is collected last on purpose: if it fails, a run that stops at the first failure has
already exercised everything else.  It builds all of its own state, so it passes alone
in a fresh process as well as after the other tests.
"""
import pytest
import torch

import harness
from paper_2307_02628_b200 import binding, synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,shape", [
    ("fp32", synth.TINY),
    ("bf16", synth.ModelShape("static-bf16", 3, 256, 4, 512, 1000, 256, "bf16")),
])
def test_static_scratch_step_matches_regular_step_twice_in_a_row(name, shape):
    wl = synth.Workload(shape, 4, 70, 6, shape.n_layers, shape.n_layers - 1, 0)
    w = synth.make_weights(shape, seed=12)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    dec = harness.make_decoder(wl, w)
    dec.set_option(binding.SD_OPT_ATTN_CHUNK, 32)          # several splits per (row, head): the scratch is really used
    tol = harness.TOL[name]
    same = {"fp32": 1e-5, "bf16": harness.REORDER_TOL}[name]               # one GPU path against the other
    ref = harness.oracle_run_forced(wl, w, prompts, forced)    # [B, 1 + gen_len, vocab], index 0 = prompt pass
    with torch.cuda.stream(dec.stream):
        dec.schedule(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len)
        dec.prefill(prompts)
        f = forced.to(dec.device)
        regular = [dec.decode_step(f[:, g].contiguous(), wl.prompt_len + g).clone() for g in range(2)]
        dec.rewind()
        out = torch.empty_like(regular[0])                  # allocated before the calls under test
        ids = [f[:, g].contiguous() for g in range(2)]
        torch.cuda.synchronize()
        for g in range(2):                                  # two calls in a row share the static array
            dec.decode_step_static(ids[g], wl.prompt_len + g, out)
            dec.synchronize()
            err = float((out - regular[g]).abs().max())
            assert err <= same, (g, err)
            err_oracle = float((out.cpu().double() - ref[:, g + 1].double()).abs().max())
            assert err_oracle <= tol, (g, err_oracle)
            assert float(regular[g].abs().max()) > 0.05     # not a comparison of zeros
        # the two entry points may be mixed inside one sequence
        third = dec.decode_step(f[:, 2].contiguous(), wl.prompt_len + 2)
        dec.rewind()
        for g in range(2):
            dec.decode_step_static(ids[g], wl.prompt_len + g, out)
        again = dec.decode_step_static(f[:, 2].contiguous(), wl.prompt_len + 2)
        dec.synchronize()
        assert float((again - third).abs().max()) <= same
        assert float((again.cpu().double() - ref[:, 3].double()).abs().max()) <= tol
    assert dec.status() == 0
    dec.close()


def test_static_scratch_rejects_steps_beyond_its_size():
    # 64 rows x 32 heads x 48 splits of 32 keys x (128 + 2) floats = 51 MB > the 16 MiB array
    shape = synth.ModelShape("static-big", 1, 4096, 32, 64, 64, 2048, "bf16")
    wl = synth.Workload(shape, 64, 1520, 2, 1, 1, 0)
    need = 64 * 32 * 48 * 130 * 4
    assert need > 16 << 20
    w = synth.make_weights(shape, seed=1)
    dec = harness.make_decoder(wl, w)
    dec.set_option(binding.SD_OPT_ATTN_CHUNK, 32)
    with torch.cuda.stream(dec.stream):
        dec.schedule(1, 1, 0, 2)
        dec.prefill(synth.make_prompts(wl))
        ids = synth.make_forced_tokens(wl)[:, 0].contiguous()
        with pytest.raises(binding.SdError) as e:
            dec.decode_step_static(ids, wl.prompt_len)
        assert e.value.code == binding.SD_ERR_CAPACITY
        dec.decode_step(ids, wl.prompt_len)                 # nothing was enqueued or advanced by the failed call
    assert dec.status() == 0
    dec.close()
