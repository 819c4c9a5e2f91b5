"""Benchmark: skip-decode tokens/s of an OPT-shaped decoder on B200, with its roofline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c4] [--impl ours|reference]

One "step" is one pass of the whole decode path over one batch: gen_len calls of
sd_decode_step (every position of the budget schedule, the greedy pick between
them) starting from the prompt's cache.  The prompt is processed once, untimed.
`value` = batch * gen_len * N / seconds per step, timed on the device with the
inputs resident in HBM; `e2e` is the same loop through sd_decode_step_host with
pinned HOST buffers (token ids in, logits out, every step).

With N > 1 (torchrun) every rank runs an independent replica of the workload on
its own GPU: the path has no exchange step, so no collective is in the timed
region; the barrier and the max over ranks use NCCL.

--impl reference times the CPU oracle as it stands on the host cores, on a bounded
sample of the same workload (a few batch rows, a few decode steps per "step").
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2307_02628_b200 import synth  # noqa: E402

METRIC = "decode tokens/s at OPT-6.7B shape bs64 (% roofline); speedup vs full-layer"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# --------------------------------------------------------------------------- byte model

def layer_weight_bytes(shape: synth.ModelShape) -> int:
    d, f = shape.d_model, shape.d_ffn
    e = 4 if shape.dtype == "fp32" else 2
    return (4 * d * d + 2 * d * f + 9 * d + f) * e


def step_bytes(wl: synth.Workload, n_active) -> float:
    """Algorithmic bytes of one pass: per decode step n (W_layer + K,V read) + LM head + logits."""
    s = wl.shape
    e = 4 if s.dtype == "fp32" else 2
    total = 0.0
    for g, n in enumerate(n_active):
        T = wl.prompt_len + g + 1
        total += n * (layer_weight_bytes(s) + 2.0 * T * s.d_model * wl.batch * e)
        total += s.vocab * s.d_model * e + wl.batch * s.vocab * 4
    return total


# --------------------------------------------------------------------------- ncu traffic of the dominant kernel

# DRAM bytes (read + write) per algorithmic byte of attn_partial_kernel, from an ncu --set full
# capture at config 4's launch shape (1.0825 GB moved for 1.07688 GB of K and V at T = 1027; the
# traffic is proportional to T; a summary of the capture is kept under profiles/).  Valid only for the kernel source it was
# taken on: the hash below is checked and `traffic` is null once the kernel text has changed.
ATTN_TRAFFIC_RATIO = 1.0057
ATTN_KERNEL_SHA256 = "31a94a145b5ed8ac87c0b55544c26e415ec060262f217260c54eeee81869bd3d"
# attn_stream_kernel (the staged kernel, which takes the launches of at least 12 (row, head) pairs per SM): DRAM bytes
# beyond K and V per launch, from ncu --set full captures at two launch shapes, keyed by (d_model, heads, batch).
# Config 4's shape at T = 1027: 1.077985 GB read + 4.18 MB written for 1.076888 GB of K and V; config 5's at T = 259:
# 1.090583 GB + 5.55 MB for 1.086324 GB.  The surplus is q, the output rows and the sectors at the ends of the
# streams, none of which grows with T, so it is added per launch rather than as a factor.  Valid for the kernel source
# the captures were taken on (hash of attn_stream.cuh).
ATTN_STREAM_EXTRA_BYTES = {(4096, 32, 64): 5.27e6, (4096, 32, 256): 9.81e6}
ATTN_STREAM_SHA256 = "a2197a93fa28a4e060c0c5f931e3017c1017dc356643d126225f2708029b22c9"


def attention_kernel_hash() -> str:
    import hashlib
    src = open(os.path.join(ROOT, "paper_2307_02628_b200", "csrc", "kernels.cuh")).read()
    i = src.index("template <typename T, int HD, int UNROLL>")
    j = src.index("// Host side: launch with the programmatic")
    return hashlib.sha256(src[i:j].encode()).hexdigest()


def staged_kernel_hash() -> str:
    import hashlib
    return hashlib.sha256(open(os.path.join(ROOT, "paper_2307_02628_b200", "csrc", "attn_stream.cuh")).read().encode()).hexdigest()


def uses_staged_attention(wl, args) -> bool:
    """The library's rule (skipdecode.cu, attn_staged): bf16 storage, at least 12 (row, head) pairs per SM, and a
    handle configured for at least 1024 positions (option value 2 drops the last condition)."""
    sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    if wl.shape.dtype != "bf16" or args.attn_staged == 0 or wl.batch * wl.shape.n_heads < 12 * sms:
        return False
    return args.attn_staged == 2 or wl.prompt_len + wl.gen_len >= 1024


# --------------------------------------------------------------------------- ranks

def max_over_ranks(value: float, dist, device) -> float:
    """Every rank times its own replica; the job's time is the slowest rank's."""
    if dist is None:
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(world: int, batch: int, steps: int, ms: float) -> float:
    """Whole-job throughput of `world` independent replicas advancing in lock-step."""
    return world * batch * steps / (ms / 1e3)


# --------------------------------------------------------------------------- clocks

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        self.rows, self.proc = [], None
        try:
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.cmd = ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "200"]
        except Exception:
            self.cmd = None

    def start(self):
        if not self.cmd:
            return
        try:
            self.proc = subprocess.Popen(self.cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self.thread.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for nm, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            except Exception:
                continue
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------- CPU oracle leg

def oracle_sample(wl: synth.Workload, weights, rows: int, steps_per_call: int, calls: int, warm_calls: int):
    """Times the oracle's cached decode steps on `rows` batch rows: returns (tokens/s, seconds per call)."""
    from oracle import skipdecode_oracle as O
    prompts = synth.make_prompts(wl)[:rows]
    dec = O.CachedDecoder(weights, wl.shape.n_heads, torch.float32)
    dec.set_schedule(wl.max_layers, wl.min_layers, wl.warmup, wl.gen_len)
    logits = dec.prefill(prompts)
    pos = wl.prompt_len
    times = []
    for c in range(warm_calls + calls):
        t0 = time.perf_counter()
        for _ in range(steps_per_call):
            if pos - wl.prompt_len >= wl.gen_len:
                break
            ids = O.greedy(logits)
            logits = dec.decode_step(ids, pos)
            pos += 1
        dt = time.perf_counter() - t0
        if c >= warm_calls:
            times.append(dt)
    sec = sum(times) / max(1, len(times))
    return rows * steps_per_call / sec, sec


def reference_arm(args, wl, rank):
    if rank != 0:
        return
    cores = torch.get_num_threads()
    weights = synth.make_weights(wl.shape, seed=0, threads=cores)
    rows, spc = args.ref_rows, args.ref_steps
    tps, sec = oracle_sample(wl, weights, rows, spc, args.steps, args.warmup)
    sample = f"{rows} batch row(s), {spc} decode step(s) per timed step from position {wl.prompt_len}, fp32, after an untimed prompt pass"
    line = {"impl": "reference", "metric": METRIC, "value": tps, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": bench_config(wl, args),
            "cpu_baseline": {"value": tps, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": tps, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def bench_config(wl, args):
    s = wl.shape
    return {"workload": f"{args.config}: {s.name} L{s.n_layers} d{s.d_model} H{s.n_heads} f{s.d_ffn} V{s.vocab} {s.dtype}, "
                        f"batch {wl.batch}, prompt {wl.prompt_len}, gen {wl.gen_len}, linear budget {wl.max_layers}->{wl.min_layers} top layers, warm-up {wl.warmup}",
            "global_batch": wl.batch * args.gpus, "l2": "inputs larger than L2 (KV cache and weights are GBs)",
            "tokens": ("greedy on device" if args.select == "greedy" else "top-p 0.7, temperature 0.3 on device, seeded uniforms")
                      + " (value); forced ids from host (e2e)"}


# --------------------------------------------------------------------------- GPU arm

def measure_workload(name, wl, weights, args, device, dist, world, steps, warmup, e2e_steps, profile_every, full_steps):
    """Times one workload on this rank's GPU.  Returns a dict of raw results (times are the max over ranks)."""
    from paper_2307_02628_b200 import binding
    s, B, P, G = wl.shape, wl.batch, wl.prompt_len, wl.gen_len
    free, _total = torch.cuda.mem_get_info(device)
    wbytes = sum(t.numel() * t.element_size() for t in [weights["tok_emb"], weights["pos_emb"]] +
                 [t for lw in weights["layers"] for t in lw.values()])
    cfg = binding.make_config(s, B, P, G)
    need_full = binding.arena_bytes(cfg, binding.SdPlan(wl.max_layers, wl.min_layers, wl.warmup, G, 1))
    full_ok = full_steps > 0 and need_full + wbytes + (4 << 30) < free
    dec = binding.Decoder(s, weights, B, P, G, plan=(wl.max_layers, wl.min_layers, wl.warmup, G),
                          full_capacity=full_ok, device=str(device))
    stream = dec.stream
    if args.no_graphs:
        dec.set_option(binding.SD_OPT_GRAPHS, 0)
    if args.gemm_mode:
        dec.set_option(binding.SD_OPT_GEMM, args.gemm_mode)
    if args.no_persistent:
        dec.set_option(binding.SD_OPT_GEMM_PERSISTENT, 0)
    elif args.persistent_tiles is not None:
        dec.set_option(binding.SD_OPT_GEMM_PERSISTENT, args.persistent_tiles)
    if args.splitk is not None:
        dec.set_option(binding.SD_OPT_GEMM_SPLITK, args.splitk)
    if args.pdl is not None:
        dec.set_option(binding.SD_OPT_PDL, args.pdl)
    if args.deterministic:
        dec.set_option(binding.SD_OPT_DETERMINISTIC, 1)
    if args.attn_staged is not None:
        dec.set_option(binding.SD_OPT_ATTN_STAGED, args.attn_staged)
    if args.attn_chunk:
        dec.set_option(binding.SD_OPT_ATTN_CHUNK, args.attn_chunk)
    prompts = synth.make_prompts(wl).to(device)
    forced = synth.make_forced_tokens(wl)
    logits0 = torch.empty(B, s.vocab, dtype=torch.float32, device=device)
    logits = torch.empty(B, s.vocab, dtype=torch.float32, device=device)
    ids = torch.empty(B, dtype=torch.int32, device=device)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(device)

    G_run = G if args.max_gen_steps <= 0 else min(G, args.max_gen_steps)   # < G only for profiler runs

    # the paper's own token selection (Section 3.2) instead of greedy: one seeded uniform per (step, row)
    uniforms = None
    if args.select == "top-p":
        uniforms = torch.stack([synth.make_uniforms(B, seed=1000 + g) for g in range(G + 1)]).to(device)

    def choose(d, lg, g):
        if uniforms is None:
            d.greedy(lg, ids)
        else:
            d.sample_top_p(lg, uniforms[g], 0.3, 0.7, ids)

    def one_pass(nsteps=None, d=None):
        d = d or dec
        d.rewind()
        choose(d, logits0, 0)
        for g in range(G_run if nsteps is None else nsteps):
            d.decode_step(ids, P + g, logits)
            choose(d, logits, g + 1)

    def timed(fn, reps):
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        barrier()
        return max_over_ranks(a.elapsed_time(b), dist, device) / reps

    with torch.cuda.stream(stream):
        n_active, _ = dec.schedule(wl.max_layers, wl.min_layers, wl.warmup, G)
        tp0 = time.perf_counter()
        dec.prefill(prompts, logits0)
        stream.synchronize()
        t_prefill = time.perf_counter() - tp0

        for _ in range(warmup):
            one_pass()
        clocks = ClockSampler(device)
        clocks.start()
        l0 = dec.launch_count()
        ms_step = timed(one_pass, steps)
        launches = dec.launch_count() - l0
        clock_info = clocks.stop()
        assert dec.status() == 0, "device status word set"

        # end to end: host ids in, logits out, every step, through sd_decode_step_host
        e2e_s = float("nan")
        if e2e_steps > 0:
            h_ids = forced.t().contiguous().pin_memory()            # [G, B]
            h_logits = torch.empty(B, s.vocab, dtype=torch.float32).pin_memory()

            def e2e_pass():
                dec.rewind()
                for g in range(G_run):
                    dec.decode_step_host(h_ids[g], P + g, h_logits)

            e2e_pass()
            barrier()
            te = time.perf_counter()
            for _ in range(e2e_steps):
                e2e_pass()
            barrier()
            e2e_s = (time.perf_counter() - te) / e2e_steps
        e2e_s = max_over_ranks(e2e_s, dist, device)

        # dominant kernel (decode attention): device time per launch on sampled steps
        dec.rewind()
        dec.kernel_times_reset()
        dec.greedy(logits0, ids)
        attn_bytes = 0.0
        e = 4 if s.dtype == "fp32" else 2
        for g in range(G_run if profile_every > 0 else 0):
            sampled = (g % profile_every == 0)
            dec.set_option(binding.SD_OPT_TIMING, 1 if sampled else 0)
            dec.decode_step(ids, P + g, logits)
            dec.greedy(logits, ids)
            if sampled:
                attn_bytes += n_active[g] * 2.0 * (P + g + 1) * s.d_model * B * e
        dec.set_option(binding.SD_OPT_TIMING, 0)
        kt = dec.kernel_times()

        full = None
        if full_ok:
            dec.schedule(s.n_layers, s.n_layers, 0, G)
            one_pass()
            ms_full = timed(one_pass, full_steps)
            full = {"ms_per_step": ms_full, "tokens_per_s": world * B * G_run / (ms_full / 1e3),
                    "speedup_skip_over_full": ms_full / ms_step,
                    "byte_model_bound": step_bytes(wl, [s.n_layers] * G_run) / step_bytes(wl, n_active[:G_run])}
        elif full_steps > 0 and G_run == G:
            # The all-layers cache for the whole generation does not fit beside the weights (config 5:
            # 172 GB): compare over the longest prefix of positions whose full cache does fit, skip and
            # full-layer both timed on exactly those positions.
            free_now, _ = torch.cuda.mem_get_info(device)
            mine = dec.arena_bytes
            Gp = 0
            for cand in range(G - G % 64, 0, -64):
                need = binding.arena_bytes(binding.make_config(s, B, P, cand), binding.SdPlan(s.n_layers, s.n_layers, 0, cand, 1))
                if need + (4 << 30) < free_now + mine:     # this decoder is released first; the next one uploads the weights again
                    Gp = cand
                    break
            if Gp:
                one_pass(Gp)
                ms_skip_p = timed(lambda: one_pass(Gp), full_steps)
                dec.close()
                torch.cuda.empty_cache()
                dec2 = binding.Decoder(s, weights, B, P, Gp, plan=(s.n_layers, s.n_layers, 0, Gp), full_capacity=True,
                                       device=str(device), stream=stream)
                dec2.schedule(s.n_layers, s.n_layers, 0, Gp)
                dec2.prefill(prompts, logits0)
                one_pass(Gp, dec2)
                ms_full_p = timed(lambda: one_pass(Gp, dec2), full_steps)
                assert dec2.status() == 0
                dec2.close()
                full = {"prefix_steps": Gp, "ms_full": ms_full_p, "ms_skip_same_steps": ms_skip_p,
                        "speedup_skip_over_full": ms_full_p / ms_skip_p,
                        "byte_model_bound": step_bytes(wl, [s.n_layers] * Gp) / step_bytes(wl, n_active[:Gp]),
                        "note": f"all-layers cache for all {G} steps does not fit; both timed on the first {Gp} positions"}
    dec.close()
    torch.cuda.empty_cache()
    return {"name": name, "wl": wl, "G_run": G_run, "n_active": n_active, "ms_step": ms_step, "launches": launches,
            "staged": uses_staged_attention(wl, args),
            "clocks": clock_info, "e2e_s": e2e_s, "attn_bytes": attn_bytes, "kt": kt, "full": full, "prefill_s": t_prefill}


def roofline_entry(r, peak, peak_kind):
    """The dominant kernel's roofline object from a measure_workload result."""
    wl = r["wl"]
    s = wl.shape
    attn_ms, attn_n = r["kt"]["attention"]
    achieved = r["attn_bytes"] / (attn_ms / 1e3) / 1e9 if attn_ms > 0 else None
    traffic = source = None
    if r["staged"]:
        kernel = "attn_stream_kernel (split-KV decode attention, K and V staged through shared memory by bulk copies)"
        extra = ATTN_STREAM_EXTRA_BYTES.get((s.d_model, s.n_heads, wl.batch))
        if attn_n and extra is not None and staged_kernel_hash() == ATTN_STREAM_SHA256:
            traffic = r["attn_bytes"] / attn_n + extra
            source = "K and V bytes of a launch + the surplus an ncu capture of this kernel source measured at this launch shape on a 2-layer case"
    else:
        kernel = "attn_partial_kernel (split-KV decode attention)"
        if attn_n and s.dtype == "bf16" and attention_kernel_hash() == ATTN_KERNEL_SHA256:
            traffic = ATTN_TRAFFIC_RATIO * r["attn_bytes"] / attn_n
            source = "ncu capture of this kernel source on a 2-layer case of config 4's launch shape, scaled by the keys read"
    return {"kernel": kernel, "bound": "hbm", "achieved": achieved,
            "peak": peak, "unit": "GB/s", "frac": (achieved / peak) if achieved else None, "peak_kind": peak_kind,
            "traffic": traffic, "traffic_source": source,
            "launches_timed": int(attn_n),
            "algorithmic_bytes_per_launch": r["attn_bytes"] / attn_n if attn_n else None}


def gpu_arm(args, wl, rank, world):
    local = int(os.environ.get("LOCAL_RANK", 0))
    device = torch.device(f"cuda:{local}")
    torch.cuda.set_device(device)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist_.init_process_group("nccl", device_id=device)
        dist = dist_
    s, B = wl.shape, wl.batch
    t0 = time.perf_counter()
    weights = synth.make_weights(s, seed=0, threads=torch.get_num_threads())
    t_weights = time.perf_counter() - t0

    r = measure_workload(args.config, wl, weights, args, device, dist, world, args.steps, args.warmup, args.e2e_steps,
                         args.profile_every, 0 if args.no_full_layer else max(1, min(2, args.steps)))
    peak, peak_kind = measured_peaks()
    G_run, n_active, ms_step = r["G_run"], r["n_active"], r["ms_step"]
    value = job_tokens_per_s(world, B, G_run, ms_step)
    total_bytes = step_bytes(wl, n_active[:G_run])
    kt = r["kt"]
    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if s.dtype == "bf16" else "f32", "data": "synthetic", "config": bench_config(wl, args),
        "clocks": r["clocks"], "gpu_launches": int(r["launches"]),
        "e2e": {"value": world * B * G_run / r["e2e_s"], "unit": "tokens/s", "h2d_bytes_per_step": G_run * B * 4,
                "d2h_bytes_per_step": G_run * B * s.vocab * 4},
        "roofline": roofline_entry(r, peak, peak_kind),
        "step_roofline": {"algorithmic_bytes_per_step": total_bytes, "achieved_gbs": total_bytes / (ms_step / 1e3) / 1e9,
                          "frac_of_measured_hbm": total_bytes / (ms_step / 1e3) / 1e9 / peak,
                          "frac_of_8tbs": total_bytes / (ms_step / 1e3) / 1e9 / 8000.0},
        "kernel_time_ms": {k: v[0] for k, v in kt.items()}, "kernel_launches_timed": {k: v[1] for k, v in kt.items()},
        "full_layer": r["full"], "prefill_s": r["prefill_s"], "weights_s": t_weights,
        "mean_active_layers": sum(n_active) / len(n_active),
    }
    if G_run != wl.gen_len:
        line["partial_pass"] = f"first {G_run} of {wl.gen_len} decode steps per pass: a profiler run, not a benchmark value"

    # The other configurations that are large enough to time (the 1.3B shape and the batch-256 case), in short:
    # one warm-up pass and two timed passes each, same kernels, same clock rules.  Config 5 shares config 4's weights.
    if args.config == "c4" and world == 1 and not args.no_other_configs and args.max_gen_steps <= 0:
        others = {}
        for name in ("c3", "c5"):
            wl2 = synth.CONFIGS[name]
            w2 = weights if wl2.shape == s else synth.make_weights(wl2.shape, seed=0, threads=torch.get_num_threads())
            r2 = measure_workload(name, wl2, w2, args, device, dist, world, 2, 1, 0, args.profile_every, 1)
            b2 = step_bytes(wl2, r2["n_active"])
            rf = roofline_entry(r2, peak, peak_kind)
            others[name] = {"workload": bench_config(wl2, args)["workload"].replace(args.config + ":", name + ":", 1),
                            "value": job_tokens_per_s(world, wl2.batch, wl2.gen_len, r2["ms_step"]), "unit": "tokens/s",
                            "ms_per_step": r2["ms_step"], "steps": 2, "warmup": 1, "clocks": r2["clocks"],
                            "step_roofline_frac_of_measured_hbm": b2 / (r2["ms_step"] / 1e3) / 1e9 / peak,
                            "attention_gbs": rf["achieved"], "attention_frac": rf["frac"], "full_layer": r2["full"],
                            "prefill_s": r2["prefill_s"]}
            del w2
        line["other_configs"] = others

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cores = torch.get_num_threads()
        tps, sec = oracle_sample(wl, weights, args.ref_rows, args.ref_steps, 2, 1)
        line["cpu_baseline"] = {"value": tps, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                                "sample": f"{args.ref_rows} batch row(s), 2 timed calls of {args.ref_steps} decode step(s) from position {wl.prompt_len}, fp32, after an untimed prompt pass"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c4", choices=sorted(synth.CONFIGS))
    ap.add_argument("--e2e-steps", type=int, default=1)
    ap.add_argument("--profile-every", type=int, default=8)
    ap.add_argument("--max-gen-steps", type=int, default=0,
                    help="run only the first N decode steps of each pass (for short profiler captures)")
    ap.add_argument("--no-graphs", action="store_true", help="plain launches instead of CUDA graph replay (profiler runs)")
    ap.add_argument("--gemm-mode", type=int, default=0, help="SD_OPT_GEMM (0 automatic, 1 CUDA cores)")
    ap.add_argument("--select", default="greedy", choices=["greedy", "top-p"],
                    help="token selection in the timed generation loop (the five configurations are greedy)")
    ap.add_argument("--no-persistent", action="store_true", help="SD_OPT_GEMM_PERSISTENT = 0")
    ap.add_argument("--persistent-tiles", type=int, default=None, help="SD_OPT_GEMM_PERSISTENT: 1 = 96- or 128-token tiles (default), 2 = 128 only")
    ap.add_argument("--splitk", type=int, default=None, help="SD_OPT_GEMM_SPLITK (most splits of K under a non-linear epilogue; 0 = off)")
    ap.add_argument("--attn-chunk", type=int, default=0, help="SD_OPT_ATTN_CHUNK (0 automatic)")
    ap.add_argument("--pdl", type=int, default=None, help="SD_OPT_PDL mask of kernel classes (0 = off)")
    ap.add_argument("--deterministic", action="store_true", help="SD_OPT_DETERMINISTIC = 1")
    ap.add_argument("--attn-staged", type=int, default=None, help="SD_OPT_ATTN_STAGED: 0 = register-only decode attention everywhere, 2 = staged whatever the sequence length")
    ap.add_argument("--no-full-layer", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true", help="with the default workload (c4): do not also time c3 and c5")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ref-rows", type=int, default=1)
    ap.add_argument("--ref-steps", type=int, default=1)
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    wl = synth.CONFIGS[args.config]
    if args.impl == "reference":
        reference_arm(args, wl, rank)
        return
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torchrun for N > 1")
    gpu_arm(args, wl, rank, world)


if __name__ == "__main__":
    main()
