"""Ragged batches on the device: prompts of different lengths aligned at the right (left padding),
and rows that stop generating while the others go on.  The oracle evaluates every row alone."""
import pytest
import torch

import harness
from oracle import skipdecode_oracle as O
from paper_2307_02628_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _run(shape, B, P, G, mx, mn, warm, pad, retire, graphs=1, tiles=1, seed=12, options=None):
    """retire: {step g: rows that generate from step g on}.  Returns the worst logit error."""
    wl = synth.Workload(shape, B, P, G, mx, mn, warm)
    w = synth.make_weights(shape, seed=seed, random_ln=True)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    n, _ = O.schedule(mx, mn, warm, G, shape.n_layers)
    active = O.active_matrix(shape.n_layers, P, n, warm)
    ref = O.forward_ragged(w, shape.n_heads, torch.cat([prompts, forced], 1), pad, active, logits_from=P - 1)
    dec = harness.make_decoder(wl, w)
    dec.set_option(binding.SD_OPT_GRAPHS, graphs)
    dec.set_option(binding.SD_OPT_PREFILL_ATTN, tiles)
    for opt, value in (options or {}).items():
        dec.set_option(opt, value)
    worst = 0.0
    agree = total = 0
    with torch.cuda.stream(dec.stream):
        dec.schedule(mx, mn, warm, G)
        dec.set_padding(pad)
        lg = dec.prefill(prompts).cpu()
        worst = max(worst, float((lg.double() - ref[:, 0]).abs().max()))
        rows = list(range(B))
        for g in range(G):
            if g in retire:
                rows = retire[g]
                dec.set_rows(rows)
            out = dec.decode_step(forced[rows, g].contiguous(), P + g).cpu()
            assert out.shape[0] == len(rows)
            r = ref[rows, g + 1]
            worst = max(worst, float((out.double() - r).abs().max()))
            agree += int((out.argmax(-1) == r.argmax(-1)).sum())
            total += len(rows)
    assert dec.status() == 0
    dec.close()
    assert agree >= 0.98 * total
    return worst


@pytest.mark.parametrize("graphs", [1, 0])
def test_left_padding_and_retiring_rows_bf16(graphs):
    shape = synth.ModelShape("toy-ragged-64", 3, 256, 4, 384, 777, 160, "bf16")
    err = _run(shape, 5, 70, 12, 3, 1, 0, pad=[0, 3, 17, 64, 69], retire={4: [0, 2, 4], 8: [2]}, graphs=graphs)
    print("ragged bf16 hd=64: max|err| =", err)
    assert err <= harness.TOL["bf16"]


@pytest.mark.parametrize("tiles", [1, 0])
def test_padding_longer_than_a_key_tile(tiles):
    # head size 128; paddings that cover whole 64-key tiles, end inside one, and leave a single real token
    shape = synth.ModelShape("toy-ragged-128", 3, 256, 2, 384, 777, 200, "bf16")
    err = _run(shape, 4, 130, 6, 3, 2, 1, pad=[0, 70, 128, 129], retire={3: [1, 3]}, tiles=tiles)
    print(f"ragged bf16 hd=128 tiles={tiles}: max|err| =", err)
    assert err <= harness.TOL["bf16"]


def test_left_padding_fp32_path():
    err = _run(synth.TINY, 3, 20, 9, 4, 2, 0, pad=[0, 5, 19], retire={2: [1, 2], 6: [1]})
    print("ragged fp32: max|err| =", err)
    assert err <= harness.TOL["fp32"]


def test_padding_content_is_invisible_and_errors():
    shape = synth.ModelShape("toy-ragged-64", 3, 256, 4, 384, 777, 160, "bf16")
    wl = synth.Workload(shape, 2, 40, 4, 3, 2, 0)
    w = synth.make_weights(shape, seed=12)
    prompts = synth.make_prompts(wl)
    dec = harness.make_decoder(wl, w)
    with torch.cuda.stream(dec.stream):
        dec.schedule(3, 2, 0, 4)
        with pytest.raises(binding.SdError):
            dec.set_rows([0])                           # nothing prefilled yet
        dec.set_padding([0, 30])
        with pytest.raises(binding.SdError):
            dec.prefill(prompts[:, :30].contiguous())   # no real token left in row 1
        for bad in ([0, -1], [0, 40], [0, 1, 2]):
            with pytest.raises(binding.SdError):
                dec.set_padding(bad)
        dec.set_padding([0, 25])
        a = dec.prefill(prompts).cpu()
        other = prompts.clone()
        other[1, :25] = (other[1, :25] + 11) % shape.vocab
        b = dec.prefill(other).cpu()
        assert torch.equal(a, b)                        # bit-identical: the padding slots are never read by the row
        for bad in ([1, 0], [0, 0], [2], []):
            with pytest.raises(binding.SdError):
                dec.set_rows(bad)
        dec.set_rows([1])
        one = dec.decode_step(torch.tensor([5], dtype=torch.int32), 40).cpu()
        dec.set_rows(None)
        dec.rewind()
        both = dec.decode_step(torch.tensor([9, 5], dtype=torch.int32), 40).cpu()
        assert float((both[1] - one[0]).abs().max()) <= 1e-3   # the same row, alone or in company (other GEMM tiling)
        dec.set_padding(None)
        with pytest.raises(binding.SdError):
            dec.decode_step(torch.tensor([9, 5], dtype=torch.int32), 41)   # padding changed: prefill first
    dec.close()


def test_host_buffer_and_static_scratch_steps_follow_the_row_list():
    # the other two step entry points take and return exactly the generating rows as well
    shape = synth.ModelShape("toy-ragged-64", 3, 256, 4, 384, 777, 160, "bf16")
    wl = synth.Workload(shape, 5, 40, 4, 3, 2, 0)
    w = synth.make_weights(shape, seed=12)
    prompts, forced = synth.make_prompts(wl), synth.make_forced_tokens(wl)
    rows = [1, 3, 4]
    dec = harness.make_decoder(wl, w)
    with torch.cuda.stream(dec.stream):
        dec.schedule(3, 2, 0, 4)
        dec.set_padding([0, 7, 0, 39, 12])
        dec.prefill(prompts)
        dec.set_rows(rows)
        ids = forced[rows, 0].contiguous()
        regular = dec.decode_step(ids, 40).cpu()
        dec.rewind()
        static = dec.decode_step_static(ids.to(dec.device), 40).cpu()
        dec.rewind()
        host = torch.empty(len(rows), shape.vocab, dtype=torch.float32).pin_memory()
        dec.decode_step_host(ids, 40, host)
    assert dec.status() == 0
    dec.close()
    assert regular.shape == (3, shape.vocab)
    assert float((static - regular).abs().max()) <= 1e-3 and float((host - regular).abs().max()) <= 1e-3
    assert float(regular.abs().max()) > 0.05
