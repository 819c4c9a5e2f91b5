"""Thin ctypes binding of include/skipdecode.h: argument marshalling only.

Every step of the path runs in the CUDA library; torch is used here for device
memory, streams and nothing else.  Opening the library fails loudly when it has
not been built (`python -m paper_2307_02628_b200.build`); there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from .shapes import ModelShape, storage_dtype

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libskipdecode.so")
_lib = None

SD_OK, SD_ERR_ARG, SD_ERR_STATE, SD_ERR_POSITION, SD_ERR_CAPACITY, SD_ERR_CUDA, SD_ERR_DEVICE = 0, -1, -2, -3, -4, -5, -6
SD_OPT_GRAPHS, SD_OPT_ATTN_CHUNK, SD_OPT_GEMM, SD_OPT_TIMING, SD_OPT_PDL, SD_OPT_PREFILL_ATTN, SD_OPT_GEMM_PERSISTENT, SD_OPT_GEMM_SPLITK, SD_OPT_DETERMINISTIC, SD_OPT_TEST_WAIT_EXPIRY, SD_OPT_ATTN_STAGED = 1, 2, 3, 4, 5, 8, 10, 11, 12, 13, 14
KERNEL_CLASSES = ("embed", "layernorm", "gemm_qkv", "kv_append", "attention", "lm_head", "gemm_out", "gemm_fc1", "gemm_fc2")

EXPORTS = ("sd_arena_bytes", "sd_create", "sd_schedule", "sd_schedule_compute", "sd_schedule_power_compute",
           "sd_schedule_custom", "sd_layer_capacity",
           "sd_prefill", "sd_decode_step", "sd_decode_step_static", "sd_rewind", "sd_launch_count", "sd_decode_step_host", "sd_greedy", "sd_sample_top_p", "sd_set_padding", "sd_set_rows", "sd_status", "sd_stats",
           "sd_set_option", "sd_kernel_time", "sd_kernel_time_reset", "sd_strerror", "sd_destroy")


class SdConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "d_ffn", "vocab", "max_pos",
                                          "max_batch", "max_prompt", "max_gen", "dtype")] + [("ln_eps", C.c_float)]


_PP = C.POINTER(C.c_void_p)
_LAYER_FIELDS = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o", "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2")


class SdWeights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("pos_emb", C.c_void_p)] + [(n, _PP) for n in _LAYER_FIELDS] + \
               [("lnf_g", C.c_void_p), ("lnf_b", C.c_void_p), ("lm_head", C.c_void_p)]


class SdPlan(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("max_layers", "min_layers", "warmup", "gen_len", "full_capacity")]


class SdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().sd_strerror(code).decode() if _lib is not None else str(code)
        super().__init__(f"{where}: {msg} ({code})")


def lib() -> C.CDLL:
    """Opens libskipdecode.so (built in-tree) and declares the prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2307_02628_b200.build`; "
                           "there is no fallback path")
    L = C.CDLL(_LIB_PATH)
    vp, i32p = C.c_void_p, C.POINTER(C.c_int32)
    L.sd_arena_bytes.argtypes = [C.POINTER(SdConfig), C.POINTER(SdPlan), C.POINTER(C.c_size_t)]
    L.sd_create.argtypes = [C.POINTER(SdConfig), C.POINTER(SdWeights), C.POINTER(SdPlan), vp, C.c_size_t, vp, C.POINTER(vp)]
    L.sd_schedule.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, i32p, i32p]
    L.sd_schedule_compute.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, i32p, i32p]
    L.sd_schedule_power_compute.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, i32p, i32p]
    L.sd_schedule_custom.argtypes = [vp, i32p, C.c_int, C.c_int, i32p]
    L.sd_layer_capacity.argtypes = [C.POINTER(SdConfig), C.POINTER(SdPlan), i32p]
    L.sd_prefill.argtypes = [vp, vp, C.c_int, C.c_int, vp]
    L.sd_decode_step.argtypes = [vp, vp, C.c_int, vp]
    L.sd_decode_step_static.argtypes = [vp, vp, C.c_int, vp]
    L.sd_rewind.argtypes = [vp]
    L.sd_launch_count.argtypes = [vp, C.POINTER(C.c_int64)]
    L.sd_decode_step_host.argtypes = [vp, vp, C.c_int, vp]
    L.sd_greedy.argtypes = [vp, vp, C.c_int, vp]
    L.sd_set_padding.argtypes = [vp, vp, C.c_int]
    L.sd_set_rows.argtypes = [vp, vp, C.c_int]
    L.sd_sample_top_p.argtypes = [vp, vp, C.c_int, C.c_float, C.c_float, vp, vp]
    L.sd_status.argtypes = [vp, i32p]
    L.sd_stats.argtypes = [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    L.sd_set_option.argtypes = [vp, C.c_int, C.c_int]
    L.sd_kernel_time.argtypes = [vp, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    L.sd_kernel_time_reset.argtypes = [vp]
    L.sd_strerror.argtypes = [C.c_int]
    L.sd_strerror.restype = C.c_char_p
    L.sd_destroy.argtypes = [vp]
    L.sd_destroy.restype = None
    for name in EXPORTS:
        if name not in ("sd_strerror", "sd_destroy"):
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _check(code: int, where: str):
    if code != SD_OK:
        raise SdError(code, where)


def make_config(shape: ModelShape, max_batch: int, max_prompt: int, max_gen: int) -> SdConfig:
    return SdConfig(shape.n_layers, shape.d_model, shape.n_heads, shape.d_ffn, shape.vocab, shape.max_pos,
                    max_batch, max_prompt, max_gen, 0 if shape.dtype == "fp32" else 1, 1e-5)


def schedule_compute(n_layers: int, max_layers: int, min_layers: int, warmup: int, gen_len: int):
    """The library's integer schedule, host only: (n_active, top_begin) as lists."""
    n = (C.c_int32 * max(gen_len, 1))()
    t = (C.c_int32 * max(gen_len, 1))()
    _check(lib().sd_schedule_compute(n_layers, max_layers, min_layers, warmup, gen_len, n, t), "sd_schedule_compute")
    return list(n)[:gen_len], list(t)[:gen_len]


def schedule_power_compute(n_layers: int, max_layers: int, min_layers: int, warmup: int, gen_len: int, alpha: int):
    """Power-law budget table, host only: (n_active, top_begin) as lists."""
    n = (C.c_int32 * max(gen_len, 1))()
    t = (C.c_int32 * max(gen_len, 1))()
    _check(lib().sd_schedule_power_compute(n_layers, max_layers, min_layers, warmup, gen_len, alpha, n, t),
           "sd_schedule_power_compute")
    return list(n)[:gen_len], list(t)[:gen_len]


def layer_capacity(cfg: SdConfig, plan: SdPlan):
    cap = (C.c_int32 * cfg.n_layers)()
    _check(lib().sd_layer_capacity(C.byref(cfg), C.byref(plan), cap), "sd_layer_capacity")
    return list(cap)


def arena_bytes(cfg: SdConfig, plan: SdPlan) -> int:
    need = C.c_size_t(0)
    _check(lib().sd_arena_bytes(C.byref(cfg), C.byref(plan), C.byref(need)), "sd_arena_bytes")
    return need.value


class Decoder:
    """A handle of the CUDA library plus the device buffers it was given.

    weights: a dict {tok_emb, pos_emb, lnf_g, lnf_b, [lm_head], layers: [{ln1_g, ..., b_fc2}]} (CPU or CUDA tensors in the
    configuration's storage type); they are moved to `device` and kept alive here.
    plan: (max_layers, min_layers, warmup, gen_len) the KV caches are sized for.
    """

    def __init__(self, shape: ModelShape, weights: dict, max_batch: int, max_prompt: int, max_gen: int,
                 plan=None, full_capacity: bool = False, device: str = "cuda:0", stream=None):
        L = lib()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the decode path has no CPU fallback")
        self.shape, self.device = shape, torch.device(device)
        self.cfg = make_config(shape, max_batch, max_prompt, max_gen)
        mx, mn, w, G = plan if plan is not None else (shape.n_layers, shape.n_layers, 0, max_gen)
        self.plan = SdPlan(mx, mn, w, G, 1 if full_capacity else 0)
        self.arena_bytes = arena_bytes(self.cfg, self.plan)
        torch.cuda.set_device(self.device)
        self.stream = stream if stream is not None else torch.cuda.Stream(device=self.device)
        dt = storage_dtype(shape)
        self._keep = []

        def dev(t):
            t = t.to(device=self.device, dtype=dt).contiguous()
            self._keep.append(t)
            return t.data_ptr()

        n = shape.n_layers
        self._arrs = {nm: (C.c_void_p * n)(*[dev(weights["layers"][l][nm]) for l in range(n)]) for nm in _LAYER_FIELDS}
        head = weights.get("lm_head")
        self.w = SdWeights(dev(weights["tok_emb"]), dev(weights["pos_emb"]),
                           *[C.cast(self._arrs[nm], _PP) for nm in _LAYER_FIELDS],
                           dev(weights["lnf_g"]), dev(weights["lnf_b"]), dev(head) if head is not None else None)
        self.arena = torch.empty(self.arena_bytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.arena.data_ptr() + 255) // 256 * 256
        self.h = C.c_void_p()
        torch.cuda.synchronize(self.device)
        _check(L.sd_create(C.byref(self.cfg), C.byref(self.w), C.byref(self.plan), base, self.arena_bytes,
                           self.stream.cuda_stream, C.byref(self.h)), "sd_create")
        self.B = self.P = None
        self._keep_io = None

    # -- the four calls ---------------------------------------------------------------
    def schedule(self, max_layers: int, min_layers: int, warmup: int, gen_len: int):
        n = (C.c_int32 * max(gen_len, 1))()
        t = (C.c_int32 * max(gen_len, 1))()
        _check(lib().sd_schedule(self.h, max_layers, min_layers, warmup, gen_len, n, t), "sd_schedule")
        return list(n)[:gen_len], list(t)[:gen_len]

    def schedule_custom(self, n_active, warmup: int):
        G = len(n_active)
        n = (C.c_int32 * G)(*n_active)
        t = (C.c_int32 * G)()
        _check(lib().sd_schedule_custom(self.h, n, warmup, G, t), "sd_schedule_custom")
        return list(t)

    def prefill(self, tokens: torch.Tensor, logits: torch.Tensor | None = None) -> torch.Tensor:
        B, P = tokens.shape
        tokens = self._dev_i32(tokens)
        if logits is None:
            logits = torch.empty(B, self.shape.vocab, dtype=torch.float32, device=self.device)
        self._order()
        _check(lib().sd_prefill(self.h, tokens.data_ptr(), B, P, logits.data_ptr()), "sd_prefill")
        self._keep_io = (tokens, logits)
        self.B, self.P = B, P
        self._n_rows = None
        return logits

    def decode_step(self, ids: torch.Tensor, position: int, logits: torch.Tensor | None = None) -> torch.Tensor:
        ids = self._dev_i32(ids)
        n = getattr(self, "_n_rows", None) or self.B
        if n is not None:              # before a prefill the library itself reports the state error
            assert ids.numel() == n, f"{ids.numel()} token ids for {n} generating rows"
        if logits is None:
            logits = torch.empty(ids.shape[0], self.shape.vocab, dtype=torch.float32, device=self.device)
        self._order()
        _check(lib().sd_decode_step(self.h, ids.data_ptr(), position, logits.data_ptr()), "sd_decode_step")
        self._keep_io = (ids, logits)
        return logits

    def decode_step_static(self, ids: torch.Tensor, position: int, logits: torch.Tensor | None = None) -> torch.Tensor:
        """sd_decode_step_static: the same step with the attention partials in the library's
        own static device array, for callers that may not allocate (the tensors passed here
        must already exist: this wrapper allocates `logits` only when it is not given)."""
        ids = self._dev_i32(ids)
        if logits is None:
            logits = torch.empty(ids.shape[0], self.shape.vocab, dtype=torch.float32, device=self.device)
        self._order()
        _check(lib().sd_decode_step_static(self.h, ids.data_ptr(), position, logits.data_ptr()), "sd_decode_step_static")
        self._keep_io = (ids, logits)
        return logits

    def decode_step_host(self, ids: torch.Tensor, position: int, logits: torch.Tensor) -> torch.Tensor:
        """ids, logits: CPU tensors (int32 [B], fp32 [B, vocab]); returns after the copy back."""
        assert ids.device.type == "cpu" and logits.device.type == "cpu" and ids.dtype == torch.int32
        assert logits.dtype == torch.float32 and logits.is_contiguous() and ids.is_contiguous()
        _check(lib().sd_decode_step_host(self.h, ids.data_ptr(), position, logits.data_ptr()), "sd_decode_step_host")
        return logits

    def rewind(self):
        _check(lib().sd_rewind(self.h), "sd_rewind")

    def launch_count(self) -> int:
        v = C.c_int64(0)
        _check(lib().sd_launch_count(self.h, C.byref(v)), "sd_launch_count")
        return v.value

    # -- helpers ----------------------------------------------------------------------
    def greedy(self, logits: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
        B = logits.shape[0]
        if out is None:
            out = torch.empty(B, dtype=torch.int32, device=self.device)
        _check(lib().sd_greedy(self.h, logits.data_ptr(), B, out.data_ptr()), "sd_greedy")
        return out

    def set_padding(self, pad=None):
        """Left-padding slots per row (host list), or None to remove; call before prefill."""
        if pad is None:
            _check(lib().sd_set_padding(self.h, None, 0), "sd_set_padding")
            return
        arr = (C.c_int32 * len(pad))(*[int(p) for p in pad])
        _check(lib().sd_set_padding(self.h, arr, len(pad)), "sd_set_padding")

    def set_rows(self, rows=None):
        """Rows that still generate (host list, increasing), or None for all; call after prefill."""
        if rows is None:
            _check(lib().sd_set_rows(self.h, None, 0), "sd_set_rows")
            self._n_rows = None
            return
        arr = (C.c_int32 * len(rows))(*[int(r) for r in rows])
        _check(lib().sd_set_rows(self.h, arr, len(rows)), "sd_set_rows")
        self._n_rows = len(rows)

    def sample_top_p(self, logits: torch.Tensor, uniforms: torch.Tensor, temperature: float = 0.3,
                     top_p: float = 0.7, out: torch.Tensor | None = None) -> torch.Tensor:
        B = logits.shape[0]
        if out is None:
            out = torch.empty(B, dtype=torch.int32, device=self.device)
        assert uniforms.dtype == torch.float32 and uniforms.is_cuda and uniforms.numel() == B
        self._order()
        _check(lib().sd_sample_top_p(self.h, logits.data_ptr(), B, temperature, top_p, uniforms.data_ptr(),
                                     out.data_ptr()), "sd_sample_top_p")
        return out

    def status(self) -> int:
        v = C.c_int32(0)
        code = lib().sd_status(self.h, C.byref(v))
        if code not in (SD_OK, SD_ERR_DEVICE):
            raise SdError(code, "sd_status")
        return v.value

    def stats(self):
        a, b = C.c_int64(0), C.c_int64(0)
        _check(lib().sd_stats(self.h, C.byref(a), C.byref(b)), "sd_stats")
        return a.value, b.value

    def set_option(self, option: int, value: int):
        _check(lib().sd_set_option(self.h, option, value), "sd_set_option")

    def kernel_times(self) -> dict:
        out = {}
        for i, name in enumerate(KERNEL_CLASSES):
            ms, n = C.c_double(0), C.c_int64(0)
            _check(lib().sd_kernel_time(self.h, i, C.byref(ms), C.byref(n)), "sd_kernel_time")
            out[name] = (ms.value, n.value)
        return out

    def kernel_times_reset(self):
        _check(lib().sd_kernel_time_reset(self.h), "sd_kernel_time_reset")

    def synchronize(self):
        self.stream.synchronize()

    def close(self):
        if getattr(self, "h", None) is not None and self.h.value:
            self.stream.synchronize()
            lib().sd_destroy(self.h)
            self.h = C.c_void_p()
        self.arena = None
        self._keep = []

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _dev_i32(self, t: torch.Tensor) -> torch.Tensor:
        return t.to(device=self.device, dtype=torch.int32).contiguous()

    def _order(self):
        # buffers produced on torch's current stream must be complete before the library's stream reads them
        cur = torch.cuda.current_stream(self.device)
        if cur != self.stream:
            self.stream.wait_stream(cur)
