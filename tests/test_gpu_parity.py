"""Parity of the CUDA library (through the C ABI) with the CPU oracle.

Tolerances: max-abs logit error 1e-4 for the fp32 configuration and 3e-2 for the
bf16 ones, over every compared row, step and vocabulary entry; schedule and layer
indices bit-exact; greedy argmax agreeing on >= 99 % of (row, step) pairs, where a
differing choice whose oracle logit lies within 2*tol of the oracle's maximum is
counted as a near-tie (reported, and allowed for at most 1 % more).
Runs are teacher-forced: both sides consume the same token ids at every step, so
each step is an independent comparison.
"""
import pytest
import torch

import harness
from oracle import skipdecode_oracle as O
from paper_2307_02628_b200 import synth

pytestmark = pytest.mark.gpu


def _check(gpu, ref, dtype_name, what):
    tol = harness.TOL[dtype_name]
    err, strict, near = harness.compare(gpu, ref, tol)
    print(f"{what}: max|err|={err:.3e} argmax strict={strict:.4f} with near-ties={near:.4f}")
    assert err <= tol, (what, err)
    assert near >= 0.99 and strict >= 0.98, (what, strict, near)
    return err, strict


def test_schedule_through_handle_is_bit_exact():
    wl = synth.CONFIGS["c1"]
    w = synth.make_weights(wl.shape, seed=0)
    dec = harness.make_decoder(wl, w)
    for mx, mn, warm, G in [(4, 2, 0, 32), (4, 2, 1, 17), (3, 3, 0, 1), (4, 4, 0, 32)]:
        if mx == mn == 4 or warm:      # needs more cache than the plan (4, 2, 0, 32) reserved
            continue
        assert dec.schedule(mx, mn, warm, G) == O.schedule(mx, mn, warm, G, wl.shape.n_layers)
    dec.close()
    dec = harness.make_decoder(wl, w, full_capacity=True)
    for mx, mn, warm, G in [(4, 2, 0, 32), (4, 2, 1, 17), (3, 3, 0, 1), (4, 4, 0, 32)]:
        assert dec.schedule(mx, mn, warm, G) == O.schedule(mx, mn, warm, G, wl.shape.n_layers)
    dec.close()


@pytest.mark.parametrize("graphs", [1, 0])
def test_config1_fp32_greedy_teacher_forced(graphs):
    from paper_2307_02628_b200 import binding
    wl = synth.CONFIGS["c1"]
    w = synth.make_weights(wl.shape, seed=0)
    prompts = synth.make_prompts(wl)
    ref, fed = harness.oracle_greedy(wl, w, prompts)
    dec = harness.make_decoder(wl, w)
    dec.set_option(binding.SD_OPT_GRAPHS, graphs)
    gpu = harness.gpu_run_forced(dec, wl, prompts, fed)
    steps, layer_steps = dec.stats()
    assert steps == wl.gen_len and layer_steps == 96          # sum of the 4 -> 2 budget over 32 positions
    dec.close()
    _check(gpu, ref, "fp32", f"c1 graphs={graphs}")
    # the definition (whole sequence, layer by layer) gives the same numbers as cached generation
    ref2 = harness.oracle_run_forced(wl, w, prompts, fed)
    assert float((ref2 - ref).abs().max()) < 1e-9


def test_config1_free_running_greedy_matches_oracle_tokens():
    wl = synth.CONFIGS["c1"]
    w = synth.make_weights(wl.shape, seed=0)
    prompts = synth.make_prompts(wl)
    ref, fed = harness.oracle_greedy(wl, w, prompts)
    dec = harness.make_decoder(wl, w)
    with torch.cuda.stream(dec.stream):
        dec.schedule(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len)
        logits = dec.prefill(prompts)
        toks = []
        for g in range(wl.gen_len):
            ids = dec.greedy(logits)
            toks.append(ids.clone())
            logits = dec.decode_step(ids, wl.prompt_len + g)
        got = torch.stack(toks, dim=1).cpu()
    dec.close()
    # fp32 against fp64: a flip needs a top-2 gap below ~1e-5, so free-running tokens agree
    assert float((got == fed).double().mean()) >= 0.99


@pytest.mark.parametrize("warm,mx,mn,B,P,G", [(1, 4, 2, 3, 7, 9), (0, 3, 1, 1, 1, 5), (1, 4, 3, 5, 33, 1), (0, 4, 4, 2, 31, 34)])
def test_fp32_odd_sizes_and_warmup(warm, mx, mn, B, P, G):
    wl = synth.Workload(synth.TINY, B, P, G, mx, mn, warm)
    w = synth.make_weights(wl.shape, seed=4, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    ref = harness.oracle_run_forced(wl, w, prompts, forced)
    dec = harness.make_decoder(wl, w)
    gpu = harness.gpu_run_forced(dec, wl, prompts, forced)
    dec.close()
    _check(gpu, ref, "fp32", f"tiny warm={warm} {mx}->{mn} B{B} P{P} G{G}")


@pytest.mark.parametrize("hd,dtype", [(32, "fp32"), (128, "fp32"), (32, "bf16"), (64, "bf16"), (128, "bf16")])
def test_head_dims_and_storage_types(hd, dtype):
    shape = synth.ModelShape(f"toy-{hd}-{dtype}", 3, 4 * hd if hd < 128 else 256, 4 if hd < 128 else 2, 384, 777, 96, dtype)
    wl = synth.Workload(shape, 3, 37, 40, 3, 1, 0)
    w = synth.make_weights(shape, seed=5, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    ref = harness.oracle_run_forced(wl, w, prompts, forced)
    dec = harness.make_decoder(wl, w)
    gpu = harness.gpu_run_forced(dec, wl, prompts, forced)
    dec.close()
    _check(gpu, ref, dtype, f"toy hd={hd} {dtype}")


@pytest.mark.parametrize("hd,P", [(64, 64), (64, 65), (64, 200), (128, 129), (128, 255)])
def test_prompt_attention_tiles(hd, P):
    # the prompt pass's tensor-core attention: several 64-key tiles, a ragged last tile, both head sizes;
    # the decode steps that follow read what every prompt position wrote in every layer
    from paper_2307_02628_b200 import binding
    shape = synth.ModelShape(f"toy-prompt-{hd}", 3, 256, 256 // hd, 384, 777, 320, "bf16")
    wl = synth.Workload(shape, 3, P, 12, 3, 2, 0)
    w = synth.make_weights(shape, seed=8, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    ref = harness.oracle_run_forced(wl, w, prompts, forced)
    runs = {}
    for tiles in (1, 0):
        dec = harness.make_decoder(wl, w)
        dec.set_option(binding.SD_OPT_PREFILL_ATTN, tiles)
        runs[tiles] = harness.gpu_run_forced(dec, wl, prompts, forced)
        dec.close()
        _check(runs[tiles], ref, "bf16", f"prompt attention hd={hd} P={P} tiles={tiles}")
    assert float((runs[1] - runs[0]).abs().max()) <= 1e-2


@pytest.mark.parametrize("chunk", [32, 64, 96])
def test_attention_split_sizes_agree(chunk):
    from paper_2307_02628_b200 import binding
    wl = synth.Workload(synth.TINY, 2, 50, 40, 4, 2, 0)
    w = synth.make_weights(wl.shape, seed=6)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    ref = harness.oracle_run_forced(wl, w, prompts, forced)
    dec = harness.make_decoder(wl, w)
    dec.set_option(binding.SD_OPT_ATTN_CHUNK, chunk)
    gpu = harness.gpu_run_forced(dec, wl, prompts, forced)
    dec.close()
    _check(gpu, ref, "fp32", f"chunk={chunk}")


def test_config2_bf16_greedy_teacher_forced():
    wl = synth.CONFIGS["c2"]
    w = synth.make_weights(wl.shape, seed=0)
    prompts = synth.make_prompts(wl)
    ref, fed = harness.oracle_greedy(wl, w, prompts)
    dec = harness.make_decoder(wl, w)
    gpu = harness.gpu_run_forced(dec, wl, prompts, fed)
    assert dec.stats() == (128, 1024)
    dec.close()
    _check(gpu, ref, "bf16", "c2")


def test_full_budget_equals_ordinary_decoding():
    wl = synth.Workload(synth.TINY, 2, 16, 12, 4, 4, 0)
    w = synth.make_weights(wl.shape, seed=2)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    seq = torch.cat([prompts, forced], dim=1)
    ref = O.full_forward(w, wl.shape.n_heads, seq)[:, wl.prompt_len - 1:]
    dec = harness.make_decoder(wl, w)
    gpu = harness.gpu_run_forced(dec, wl, prompts, forced)
    dec.close()
    _check(gpu, ref, "fp32", "full budget")


def test_host_buffer_step_and_greedy_kernel():
    wl = synth.CONFIGS["c1"]
    w = synth.make_weights(wl.shape, seed=0)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    dec = harness.make_decoder(wl, w)
    a = harness.gpu_run_forced(dec, wl, prompts, forced)
    with torch.cuda.stream(dec.stream):
        dec.schedule(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len)
        dec.prefill(prompts)
        h_logits = torch.empty(wl.batch, wl.shape.vocab, dtype=torch.float32).pin_memory()
        for g in range(wl.gen_len):
            dec.decode_step_host(forced[:, g].contiguous(), wl.prompt_len + g, h_logits)
            assert torch.equal(h_logits, a[:, g + 1])            # same kernels, same order: bit-identical
        d = a[:, 5].to(dec.device)
        d[1, 7] = d[1, 900] = d[1].max() + 1.0                   # an exact tie: the lowest index wins
        nxt = dec.greedy(d).cpu()
    assert nxt.tolist() == [int(t) for t in O.greedy(d.cpu())] and nxt[1] == 7
    dec.close()


def test_errors_are_reported_not_fatal():
    from paper_2307_02628_b200 import binding
    wl = synth.CONFIGS["c1"]
    w = synth.make_weights(wl.shape, seed=0)
    dec = harness.make_decoder(wl, w)
    prompts = synth.make_prompts(wl)
    ids = prompts[:, 0].contiguous()
    with torch.cuda.stream(dec.stream):
        with pytest.raises(binding.SdError) as e:
            dec.prefill(prompts)
        assert e.value.code == binding.SD_ERR_STATE                  # no schedule yet
        with pytest.raises(binding.SdError) as e:
            dec.schedule(4, 4, 0, 32)
        assert e.value.code == binding.SD_ERR_CAPACITY               # needs more cache than planned
        dec.schedule(4, 2, 0, 32)
        with pytest.raises(binding.SdError) as e:
            dec.decode_step(ids, 32)
        assert e.value.code == binding.SD_ERR_STATE                  # no prefill yet
        with pytest.raises(binding.SdError) as e:
            dec.prefill(torch.zeros(5, 32, dtype=torch.int32))
        assert e.value.code == binding.SD_ERR_CAPACITY               # batch beyond max_batch
        dec.prefill(prompts)
        with pytest.raises(binding.SdError) as e:
            dec.decode_step(ids, 33)
        assert e.value.code == binding.SD_ERR_POSITION               # out of order
        dec.decode_step(ids, 32)
        assert dec.status() == 0
        bad = ids.clone()
        bad[2] = wl.shape.vocab + 5
        dec.decode_step(bad, 33)                                     # flagged on the device, clamped, no fault
        assert dec.status() == 1
    dec.close()


@pytest.mark.parametrize("B,P", [(3, 37), (20, 9), (70, 5), (130, 3)])
def test_tensor_core_and_cuda_core_gemm_paths_agree(B, P):
    """bf16 products on the tcgen05 path against the same products on CUDA cores: every
    token-tile width (16..256), ragged feature tiles (vocab 777, d_ffn 384) and split K."""
    from paper_2307_02628_b200 import binding
    shape = synth.ModelShape("toy-gemm", 2, 256, 4, 384, 777, 64, "bf16")
    wl = synth.Workload(shape, B, P, 6, 2, 1, 0)
    w = synth.make_weights(shape, seed=8, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    ref = harness.oracle_run_forced(wl, w, prompts, forced)
    outs = []
    for mode in (1, 2):             # CUDA cores, tcgen05 kernels
        dec = harness.make_decoder(wl, w)
        dec.set_option(binding.SD_OPT_GEMM, mode)
        outs.append(harness.gpu_run_forced(dec, wl, prompts, forced))
        dec.close()
        _check(outs[-1], ref, "bf16", f"gemm mode {mode} B{B} P{P}")
    # a different summation order flips some bf16 roundings of the activations: ulp-scale differences
    assert float((outs[0] - outs[1]).abs().max()) < 1e-2


def test_launch_modes_compute_the_same_function():
    """CUDA graphs and programmatic dependent launch only change how kernels are enqueued."""
    from paper_2307_02628_b200 import binding
    runs = {}
    for shape in (synth.TINY, synth.ModelShape("modes-bf16", 3, 256, 2, 512, 640, 160, "bf16")):
        wl = synth.Workload(shape, 5, 40, 24, 3, 2, 1)
        w = synth.make_weights(shape, seed=9)
        prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
        ref = harness.oracle_run_forced(wl, w, prompts, forced)
        for graphs in (1, 0):
            for pdl in (0x1ff, 0):
                dec = harness.make_decoder(wl, w)
                dec.set_option(binding.SD_OPT_GRAPHS, graphs)
                dec.set_option(binding.SD_OPT_PDL, pdl)
                out = harness.gpu_run_forced(dec, wl, prompts, forced)
                dec.close()
                _check(out, ref, shape.dtype, f"{shape.name} graphs={graphs} pdl={pdl}")
                runs[(shape.name, graphs, pdl)] = out
        if shape.dtype == "fp32":            # no atomics on this path: bit-identical in every mode
            base = runs[(shape.name, 1, 0x1ff)]
            for key, out in runs.items():
                if key[0] == shape.name:
                    assert torch.equal(out, base), key


@pytest.mark.parametrize("B,P", [(32, 128), (40, 100)])
def test_persistent_gemm_in_the_prompt_pass(B, P):
    # enough 128-token tiles per product (more than SMs) for the persistent kernel to take the QKV, out-proj,
    # fc1 and fc2 products of the prompt pass; the second case ends in a partial token tile
    from paper_2307_02628_b200 import binding
    shape = synth.ModelShape("persist-bf16", 2, 768, 6, 1024, 640, 160, "bf16")
    wl = synth.Workload(shape, B, P, 4, 2, 1, 0)
    w = synth.make_weights(shape, seed=14, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    rows = synth.sample_rows(B, 6)
    ref = harness.oracle_run_forced(wl, w, prompts, forced, rows=rows)
    runs = {}
    for persistent in (1, 0):
        dec = harness.make_decoder(wl, w)
        dec.set_option(binding.SD_OPT_GEMM_PERSISTENT, persistent)
        runs[persistent] = harness.gpu_run_forced(dec, wl, prompts, forced, rows=rows)
        dec.close()
        err, strict, near = harness.compare(runs[persistent], ref, harness.TOL["bf16"])
        print(f"persistent={persistent} B={B} P={P}: max|err|={err:.3e} argmax strict={strict:.4f} near={near:.4f}")
        assert err <= harness.TOL["bf16"] and near >= 0.99
    assert float((runs[1] - runs[0]).abs().max()) <= harness.REORDER_TOL     # same products; the residual adds arrive in another order


def test_persistent_gemm_with_96_token_tiles():
    # 2400 prompt tokens and 8 to 24 weight tiles per product: 96-token tiles take fewer rounds per block than
    # 128-token tiles, so the QKV, out-proj, fc1 and fc2 products of the prompt pass run on them (25 token tiles,
    # none ragged); at 160 rows per decode step so does the LM head (100 weight tiles, second token tile ragged)
    from paper_2307_02628_b200 import binding
    shape = synth.ModelShape("persist96-bf16", 2, 1024, 8, 1024, 12800, 32, "bf16")
    wl = synth.Workload(shape, 160, 15, 3, 2, 1, 0)
    w = synth.make_weights(shape, seed=16, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    rows = synth.sample_rows(wl.batch, 6)
    ref = harness.oracle_run_forced(wl, w, prompts, forced, rows=rows)
    runs = {}
    for mode in (1, 2, 0):
        dec = harness.make_decoder(wl, w)
        dec.set_option(binding.SD_OPT_GEMM_PERSISTENT, mode)
        runs[mode] = harness.gpu_run_forced(dec, wl, prompts, forced, rows=rows)
        dec.close()
        err, strict, near = harness.compare(runs[mode], ref, harness.TOL["bf16"])
        print(f"persistent={mode}: max|err|={err:.3e} argmax strict={strict:.4f} near={near:.4f}")
        assert err <= harness.TOL["bf16"] and near >= 0.99
    assert float((runs[1] - runs[2]).abs().max()) <= harness.REORDER_TOL
    assert float((runs[1] - runs[0]).abs().max()) <= harness.REORDER_TOL


@pytest.mark.parametrize("d,heads,B", [(1024, 8, 20), (1024, 8, 64), (1536, 12, 33), (1536, 12, 100)])
def test_split_k_under_nonlinear_epilogues(d, heads, B):
    # few output tiles and 16 or 24 k-blocks: the QKV (cache-writing), fc1 (ReLU) and LM-head (store) products of
    # a decode step split K in two or three, park their partial tiles and let the last block finish the tile;
    # token tiles of 32, 64 and 128
    from paper_2307_02628_b200 import binding
    shape = synth.ModelShape("splitk-bf16", 2, d, heads, 2048, 640, 64, "bf16")
    wl = synth.Workload(shape, B, 9, 5, 2, 1, 0)
    w = synth.make_weights(shape, seed=15, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    rows = synth.sample_rows(B, 6)
    ref = harness.oracle_run_forced(wl, w, prompts, forced, rows=rows)
    runs = {}
    for splitk in (8, 0):
        for graphs in (1, 0):
            dec = harness.make_decoder(wl, w)
            dec.set_option(binding.SD_OPT_GEMM_SPLITK, splitk)
            dec.set_option(binding.SD_OPT_GRAPHS, graphs)
            runs[splitk, graphs] = harness.gpu_run_forced(dec, wl, prompts, forced, rows=rows)
            dec.close()
            err, strict, near = harness.compare(runs[splitk, graphs], ref, harness.TOL["bf16"])
            print(f"splitk={splitk} graphs={graphs} d={d} B={B}: max|err|={err:.3e} argmax strict={strict:.4f} near={near:.4f}")
            assert err <= harness.TOL["bf16"] and near >= 0.99
    assert float((runs[8, 1] - runs[0, 1]).abs().max()) <= harness.REORDER_TOL     # same products, partial sums added in another order
    assert float((runs[8, 1] - runs[8, 0]).abs().max()) <= harness.REORDER_TOL


@pytest.mark.parametrize("alpha", [2, 3])
def test_power_law_budget_table(alpha):
    """A caller-supplied budget table (power-law decay with warm-up 1) through sd_schedule_custom."""
    from paper_2307_02628_b200 import binding
    shape = synth.ModelShape("toy-power", 6, 256, 4, 512, 999, 96, "bf16")
    wl = synth.Workload(shape, 3, 21, 40, 6, 2, 1)
    table, top = O.schedule_power(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len, shape.n_layers, alpha)
    assert binding.schedule_power_compute(shape.n_layers, 6, 2, 1, 40, alpha) == (table, top)
    w = synth.make_weights(shape, seed=13, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    ref = harness.oracle_run_forced(wl, w, prompts, forced, table=table)
    dec = harness.make_decoder(wl, w)                       # cache plan: the linear 6 -> 2 schedule, which dominates
    gpu = harness.gpu_run_forced(dec, wl, prompts, forced, table=table)
    assert dec.stats() == (wl.gen_len, sum(table))
    with pytest.raises(binding.SdError) as e:
        dec.schedule_custom([2, 3] + [2] * 38, 1)           # a budget that grows is refused
    assert e.value.code == binding.SD_ERR_ARG
    dec.close()
    _check(gpu, ref, "bf16", f"power law alpha={alpha}")


@pytest.mark.parametrize("dtype,max_prompt,P,B", [("fp32", 100, 64, 64), ("bf16", 100, 64, 64), ("bf16", 90, 17, 50)])
def test_prompt_shorter_than_the_configured_maximum(dtype, max_prompt, P, B):
    """A handle built for prompts of up to max_prompt tokens given a shorter one: the prompt pass takes as many
    whole batch rows per pass as the activation buffers were sized for (here several passes), and the decode
    steps that follow read what every pass wrote."""
    from paper_2307_02628_b200 import binding
    shape = synth.ModelShape(f"short-prompt-{dtype}", 2, 256, 4, 512, 640, 128, dtype)
    wl = synth.Workload(shape, B, P, 4, 2, 1, 0)
    w = synth.make_weights(shape, seed=17, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    rows = synth.sample_rows(B, 8)
    ref = harness.oracle_run_forced(wl, w, prompts, forced, rows=rows)
    dec = binding.Decoder(shape, w, B, max_prompt, wl.gen_len, plan=(2, 1, 0, wl.gen_len))
    gpu = harness.gpu_run_forced(dec, wl, prompts, forced, rows=rows)
    with torch.cuda.stream(dec.stream):
        with pytest.raises(binding.SdError) as e:
            dec.prefill(torch.zeros(B, max_prompt + 1, dtype=torch.int32))
        assert e.value.code == binding.SD_ERR_CAPACITY
    dec.close()
    _check(gpu, ref, dtype, f"max_prompt={max_prompt} P={P} B={B} {dtype}")


@pytest.mark.parametrize("B", [5, 40])
def test_deterministic_option_gives_the_same_bits_every_run(B):
    """bf16 storage splits K of the out-projection and fc2 over several blocks.  By default their partial sums reach
    the residual stream by atomic adds (arrival order); with SD_OPT_DETERMINISTIC they are added in split order."""
    from paper_2307_02628_b200 import binding
    shape = synth.ModelShape("det-bf16", 3, 1024, 8, 2048, 640, 96, "bf16")      # 16 and 32 k-blocks: K is split 4 ways
    wl = synth.Workload(shape, B, 19, 8, 3, 2, 0)
    w = synth.make_weights(shape, seed=23, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    ref = harness.oracle_run_forced(wl, w, prompts, forced)
    runs = []
    for det, graphs in ((1, 1), (1, 1), (1, 0), (0, 1)):
        dec = harness.make_decoder(wl, w)
        dec.set_option(binding.SD_OPT_DETERMINISTIC, det)
        dec.set_option(binding.SD_OPT_GRAPHS, graphs)
        runs.append(harness.gpu_run_forced(dec, wl, prompts, forced))
        dec.close()
        _check(runs[-1], ref, "bf16", f"deterministic={det} graphs={graphs} B={B}")
    assert torch.equal(runs[0], runs[1]) and torch.equal(runs[0], runs[2])
    assert float((runs[0] - runs[3]).abs().max()) <= harness.REORDER_TOL


def test_expired_device_wait_is_reported_and_the_handle_stays_usable():
    """The bounded waits inside the tensor-core kernels: a product whose accumulator never completes (test hook) gives
    up after about a millisecond, sets the status word, and leaves nothing in flight; sd_status reports it, and after
    the next sd_prefill the handle computes correct results again."""
    from paper_2307_02628_b200 import binding
    shape = synth.ModelShape("expiry-bf16", 2, 256, 2, 512, 640, 96, "bf16")
    wl = synth.Workload(shape, 6, 17, 4, 2, 1, 0)
    w = synth.make_weights(shape, seed=24)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    ref = harness.oracle_run_forced(wl, w, prompts, forced)
    dec = harness.make_decoder(wl, w)
    good = harness.gpu_run_forced(dec, wl, prompts, forced)
    with torch.cuda.stream(dec.stream):
        dec.rewind()
        dec.set_option(binding.SD_OPT_TEST_WAIT_EXPIRY, 1)
        dec.decode_step(forced[:, 0].contiguous(), wl.prompt_len)       # its first product gives up its wait
        code = binding.lib().sd_status(dec.h, None)
        assert code == binding.SD_ERR_DEVICE
        assert dec.status() & 2                                         # STATUS_WAIT_EXPIRED
    again = harness.gpu_run_forced(dec, wl, prompts, forced)            # schedule + prefill (clears the word) + all steps
    dec.close()
    err, strict, near = harness.compare(again, ref, harness.TOL["bf16"])
    print(f"after an expired wait: max|err|={err:.3e} argmax strict={strict:.4f} with near-ties={near:.4f}")
    assert err <= harness.TOL["bf16"] and near >= 0.99              # 30 (row, step) pairs: one near-tie moves `strict` by 3 %
    assert float((again - good).abs().max()) <= harness.REORDER_TOL


def test_weight_beyond_the_fp16_range_is_reported_at_create():
    # bf16 storage multiplies fp16 copies of the weights: a weight above 65504 is clipped in the copy and bit 8 of the
    # status word says so right after sd_create; weights inside the range leave the word at zero
    from paper_2307_02628_b200 import binding
    shape = synth.ModelShape("range-bf16", 1, 256, 4, 512, 640, 64, "bf16")
    wl = synth.Workload(shape, 2, 8, 2, 1, 1, 0)
    w = synth.make_weights(shape, seed=3)
    dec = harness.make_decoder(wl, w)
    assert dec.status() == 0
    dec.close()
    w["layers"][0]["w_fc1"][5, 7] = 1.0e5
    dec = harness.make_decoder(wl, w)
    assert dec.status() == 8
    dec.close()

