"""Thin ctypes layer over the C ABI of libmcce.so (see include/mcce.h).

Argument marshalling only: torch supplies device memory and streams, every step of the method runs in
the library's CUDA kernels.  There is no CPU fallback; a missing library or device is an error.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MCCE_LIB in the environment points at another build of the library (e.g. to compare two versions)
LIB_PATH = os.environ.get("MCCE_LIB") or os.path.join(_HERE, "libmcce.so")

F32, BF16 = 0, 1
DELTA_RUNNING, DELTA_FIXED = 0, 1
FFN_AUTO, FFN_SIMT, FFN_TENSOR = 0, 1, 2
RERANK_CACHE_PRIOR, RERANK_MAX_RANK, RERANK_CUMSUM = 0, 1, 2
ROUTE_AUTO, ROUTE_TWO_KERNELS, ROUTE_FUSED = 0, 1, 2
ROUTER_FP32_PIPE, ROUTER_GEMM_TAIL, ROUTER_RESIDENT_TAIL, ROUTER_FUSED = 0, 1, 2, 3

EXPORTS = [
    "mcce_workspace_bytes", "mcce_create", "mcce_destroy", "mcce_set_router", "mcce_set_experts", "mcce_reset",
    "mcce_route_step", "mcce_moe_forward", "mcce_decode_step_host", "mcce_decode_step_chained", "mcce_pipeline_submit_host", "mcce_pipeline_submit", "mcce_pipeline_wait", "mcce_cache_stats", "mcce_calibrate_delta", "mcce_get_cache_state",
    "mcce_get_grouping", "mcce_lifetime_stats", "mcce_set_miss_trace", "mcce_belady_replay", "mcce_profile", "mcce_profile_read", "mcce_uses_tensor_path", "mcce_router_kernel_kind", "mcce_selftest_wait_timeout", "mcce_route_trace_static",
    "mcce_route_trace_static_limit", "mcce_gen_normal", "mcce_gen_hidden_step", "mcce_gen_philox_words", "mcce_strerror",
    "mcce_last_cuda_error",
]


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "n_experts", "top_k", "top_j", "n_shared", "d_model", "d_ff",
                                         "cache_capacity", "n_streams")] + [
        ("lam", C.c_float), ("delta_mode", C.c_int32), ("renorm", C.c_int32), ("hidden_dtype", C.c_int32),
        ("weight_dtype", C.c_int32), ("ffn_impl", C.c_int32), ("device", C.c_int32),
        ("rerank_mode", C.c_int32), ("max_rank", C.c_int32), ("cum_threshold", C.c_float),
        ("track_lifetime", C.c_int32), ("route_impl", C.c_int32), ("deterministic", C.c_int32),
        ("checked", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("steps", "selections", "misses", "cold_misses")]

    def as_tuple(self):
        return (self.steps, self.selections, self.misses, self.cold_misses)


class McceError(RuntimeError):
    pass


_lib = None


def load():
    """Loads libmcce.so; raises if it has not been built (python -m paper_2412_00099_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise McceError("libmcce.so is missing: build it with `python -m paper_2412_00099_b200.build`")
        lib = C.CDLL(LIB_PATH)
        vp, i32, u32, u64, f32 = C.c_void_p, C.c_int32, C.c_uint32, C.c_uint64, C.c_float
        lib.mcce_workspace_bytes.restype = C.c_size_t
        lib.mcce_workspace_bytes.argtypes = [C.POINTER(Config)]
        lib.mcce_create.argtypes = [C.POINTER(Config), vp, C.c_size_t, C.POINTER(vp)]
        lib.mcce_destroy.argtypes = [vp]
        lib.mcce_set_router.argtypes = [vp, vp, vp]
        lib.mcce_set_experts.argtypes = [vp] * 7
        lib.mcce_reset.argtypes = [vp, vp, C.c_int, vp, C.c_int64]
        lib.mcce_route_step.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
        lib.mcce_moe_forward.argtypes = [vp] * 6
        lib.mcce_decode_step_host.argtypes = [vp] * 5
        lib.mcce_decode_step_chained.argtypes = [vp] * 5
        lib.mcce_pipeline_submit_host.argtypes = [vp] * 5
        lib.mcce_pipeline_submit.argtypes = [vp] * 6
        lib.mcce_pipeline_wait.argtypes = [vp]
        lib.mcce_cache_stats.argtypes = [vp, C.POINTER(Stats), C.POINTER(Stats)]
        lib.mcce_calibrate_delta.argtypes = [vp, vp]
        lib.mcce_get_cache_state.argtypes = [vp, vp, vp, vp, C.POINTER(C.c_int64)]
        lib.mcce_get_grouping.argtypes = [vp, vp, vp]
        lib.mcce_lifetime_stats.argtypes = [vp, vp, vp]
        lib.mcce_set_miss_trace.argtypes = [vp, vp, C.c_int64]
        lib.mcce_belady_replay.argtypes = [vp, i32, i32, i32, i32, i32, vp, i32, vp, vp, vp]
        lib.mcce_uses_tensor_path.argtypes = [vp]
        lib.mcce_router_kernel_kind.argtypes = [vp, i32]
        lib.mcce_selftest_wait_timeout.argtypes = [vp, C.c_uint64]
        lib.mcce_route_trace_static_limit.restype = C.c_size_t
        lib.mcce_route_trace_static.argtypes = [C.POINTER(Config), i32, vp, vp, vp, vp, vp, vp, C.POINTER(Stats), vp]
        lib.mcce_profile.argtypes = [vp, C.c_int]
        lib.mcce_profile_read.argtypes = [vp, vp, vp, C.c_int]
        lib.mcce_gen_normal.argtypes = [vp, i32, u64, u64, u32, u32, u32, f32, vp]
        lib.mcce_gen_hidden_step.argtypes = [vp, vp, i32, u64, u32, u32, f32, f32, f32, vp]
        lib.mcce_gen_philox_words.argtypes = [vp, u64, u64, u32, u32, u32, vp]
        lib.mcce_strerror.restype = C.c_char_p
        lib.mcce_strerror.argtypes = [C.c_int]
        lib.mcce_last_cuda_error.argtypes = [vp]
        _lib = lib
    return _lib


def _check(rc: int, ctx=None):
    if rc != 0:
        msg = load().mcce_strerror(rc).decode()
        if rc == -4 and ctx is not None:
            msg += " [cudaError %d]" % load().mcce_last_cuda_error(ctx)
        raise McceError("mcce error %d: %s" % (rc, msg))


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous()
        return C.c_void_p(t.data_ptr())
    assert t.flags.c_contiguous
    return C.c_void_p(t.ctypes.data)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _tdtype(code):
    return torch.bfloat16 if code == BF16 else torch.float32


class Engine:
    """One mcce context: the cache state of every (stream, layer) plus borrowed weights."""

    def __init__(self, *, L, E, K, J, n_shared, d, I, C_cap, S, lam, delta_mode=DELTA_RUNNING, renorm=1, dtype=BF16,
                 ffn_impl=FFN_AUTO, device=0, rerank_mode=RERANK_CACHE_PRIOR, max_rank=0, cum_threshold=0.0,
                 track_lifetime=False, route_impl=ROUTE_AUTO, deterministic=False, checked=False):
        if not torch.cuda.is_available():
            raise McceError("no CUDA device: this library has no CPU path")
        self.lib = load()
        self.cfg = Config(L, E, K, J, n_shared, d, I, C_cap, S, lam, delta_mode, renorm, dtype, dtype, ffn_impl,
                          device, rerank_mode, max_rank, cum_threshold, int(track_lifetime), route_impl,
                          int(deterministic), int(checked))
        self.device = torch.device("cuda", device)
        nbytes = self.lib.mcce_workspace_bytes(C.byref(self.cfg))
        if nbytes == 0:
            raise McceError("invalid configuration")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self.ctx = C.c_void_p()
        _check(self.lib.mcce_create(C.byref(self.cfg), C.c_void_p(base), nbytes, C.byref(self.ctx)))
        self._keep = []
        self.L, self.E, self.K, self.S, self.d, self.I, self.Ccap = L, E, K, S, d, I, C_cap
        self.dtype = dtype

    def close(self):
        if self.ctx:
            torch.cuda.synchronize(self.device)
            self.lib.mcce_destroy(self.ctx)
            self.ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- weights ------------------------------------------------------------------------------------
    def set_router(self, Wr: torch.Tensor, fixed_delta: torch.Tensor | None = None):
        assert Wr.dtype == torch.float32 and tuple(Wr.shape) == (self.L, self.E, self.d)
        self._keep += [Wr, fixed_delta]
        _check(self.lib.mcce_set_router(self.ctx, _ptr(Wr), _ptr(fixed_delta)), self.ctx)

    def set_experts(self, Wg, Wu, Wd, shWg=None, shWu=None, shWd=None):
        for t in (Wg, Wu, Wd, shWg, shWu, shWd):
            assert t is None or t.dtype == _tdtype(self.dtype)
        self._keep += [Wg, Wu, Wd, shWg, shWu, shWd]
        _check(self.lib.mcce_set_experts(self.ctx, *[_ptr(t) for t in (Wg, Wu, Wd, shWg, shWu, shWd)]), self.ctx)

    def reset(self, init_order: np.ndarray | None = None, keep_delta_stats=False, delta_sum=None, delta_count=0):
        if init_order is not None:
            init_order = np.ascontiguousarray(init_order, np.int32)
            assert init_order.shape == (self.L, self.S, self.Ccap)
        if delta_sum is not None:
            delta_sum = np.ascontiguousarray(delta_sum, np.float32)
        _check(self.lib.mcce_reset(self.ctx, _ptr(init_order), int(keep_delta_stats), _ptr(delta_sum),
                                   int(delta_count)), self.ctx)

    # -- the hot path ---------------------------------------------------------------------------------
    def route_step(self, hidden=None, logits=None, n_steps=1, want_logits=False, out=None):
        """hidden [n_steps,L,S,d] or logits [n_steps,L,S,E] (device tensors).  Returns sel_idx
        [n_steps,L,S,K] int32 and sel_w fp32 (and the logits used, if asked)."""
        shape = (n_steps, self.L, self.S, self.K)
        if out is None:
            sel = torch.empty(shape, dtype=torch.int32, device=self.device)
            w = torch.empty(shape, dtype=torch.float32, device=self.device)
        else:
            sel, w = out
        zo = torch.empty((n_steps, self.L, self.S, self.E), dtype=torch.float32,
                         device=self.device) if want_logits else None
        if hidden is not None:
            assert hidden.dtype == _tdtype(self.dtype) and hidden.numel() == n_steps * self.L * self.S * self.d
        if logits is not None:
            assert logits.dtype == torch.float32 and logits.numel() == n_steps * self.L * self.S * self.E
        _check(self.lib.mcce_route_step(self.ctx, n_steps, _ptr(hidden), _ptr(logits), _ptr(sel), _ptr(w), _ptr(zo),
                                        _stream()), self.ctx)
        return (sel, w, zo) if want_logits else (sel, w)

    def moe_forward(self, hidden, sel_idx, sel_w, out=None):
        """hidden [L,S,d], sel_idx [L,S,K] int32, sel_w [L,S,K] fp32 -> y [L,S,d] fp32."""
        assert hidden.dtype == _tdtype(self.dtype) and hidden.numel() == self.L * self.S * self.d
        assert sel_idx.dtype == torch.int32 and sel_w.dtype == torch.float32
        y = out if out is not None else torch.empty((self.L, self.S, self.d), dtype=torch.float32, device=self.device)
        _check(self.lib.mcce_moe_forward(self.ctx, _ptr(hidden), _ptr(sel_idx), _ptr(sel_w), _ptr(y), _stream()),
               self.ctx)
        return y

    def decode_step_host(self, hidden_host: torch.Tensor, y_host: torch.Tensor, sel_host: torch.Tensor | None = None):
        """One whole step from (pinned) host tensors; copies in and out inside the call."""
        assert not hidden_host.is_cuda and not y_host.is_cuda
        _check(self.lib.mcce_decode_step_host(self.ctx, _ptr(hidden_host), _ptr(y_host), _ptr(sel_host), _stream()),
               self.ctx)

    def decode_step_chained(self, x0: torch.Tensor, want_sel=False):
        """One token with the layers chained through a residual stream: x0 [S,d] -> x_L [S,d] (and sel [L,S,K])."""
        assert x0.dtype == _tdtype(self.dtype) and x0.numel() == self.S * self.d
        x_out = torch.empty_like(x0)
        sel = torch.empty((self.L, self.S, self.K), dtype=torch.int32, device=self.device) if want_sel else None
        _check(self.lib.mcce_decode_step_chained(self.ctx, _ptr(x0), _ptr(x_out), _ptr(sel), _stream()), self.ctx)
        return (x_out, sel) if want_sel else x_out

    def pipeline_submit_host(self, hidden_host, y_host, sel_host=None):
        """Asynchronous variant of decode_step_host: copies overlap the compute of neighbouring steps; call
        pipeline_wait() before reading y_host."""
        assert not hidden_host.is_cuda and not y_host.is_cuda
        _check(self.lib.mcce_pipeline_submit_host(self.ctx, _ptr(hidden_host), _ptr(y_host), _ptr(sel_host),
                                                  _stream()), self.ctx)

    def pipeline_submit(self, hidden, y, sel=None, hidden_ready=None):
        """The same with device tensors: hidden [L,S,d] must be complete (or `hidden_ready`, a torch.cuda.Event,
        marks it); y [L,S,d] fp32 and sel [L,S,K] int32 are complete in the current stream's order.  Alternate
        between two y tensors from call to call."""
        assert hidden.is_cuda and y.is_cuda and y.dtype == torch.float32 and hidden.dtype == _tdtype(self.dtype)
        ev = C.c_void_p(hidden_ready.cuda_event) if hidden_ready is not None else None
        _check(self.lib.mcce_pipeline_submit(self.ctx, _ptr(hidden), _ptr(y), _ptr(sel), ev, _stream()), self.ctx)

    def pipeline_wait(self):
        _check(self.lib.mcce_pipeline_wait(self.ctx), self.ctx)

    # -- state ------------------------------------------------------------------------------------------
    def cache_stats(self):
        total = Stats()
        per = (Stats * self.L)()
        _check(self.lib.mcce_cache_stats(self.ctx, C.byref(total), per), self.ctx)
        return total.as_tuple(), [p.as_tuple() for p in per]

    def cache_state(self):
        order = np.empty((self.L, self.S, self.Ccap), np.int32)
        ever = np.empty((self.L, self.S, self.E), np.uint8)
        dsum = np.empty((self.L, self.S), np.float32)
        cnt = C.c_int64()
        _check(self.lib.mcce_get_cache_state(self.ctx, _ptr(order), _ptr(ever), _ptr(dsum), C.byref(cnt)), self.ctx)
        return order, ever, dsum, cnt.value

    KERNELS = ("route", "group", "gather", "ffn_up", "ffn_down", "combine", "route_gemm")

    def uses_tensor_path(self) -> bool:
        return self.lib.mcce_uses_tensor_path(self.ctx) == 1

    def router_kernel_kind(self, n_tokens: int = 1) -> int:
        """ROUTER_FP32_PIPE / ROUTER_GEMM_TAIL / ROUTER_RESIDENT_TAIL / ROUTER_FUSED for a launch of n_tokens."""
        kind = self.lib.mcce_router_kernel_kind(self.ctx, n_tokens)
        if kind < 0:
            _check(kind, self.ctx)
        return kind

    def profile(self, enable: bool):
        _check(self.lib.mcce_profile(self.ctx, int(enable)), self.ctx)

    def profile_read(self, reset=True):
        """{kernel: (total ms, launches)} from the CUDA events recorded around each launch."""
        ms = np.zeros(len(self.KERNELS), np.float64)
        n = np.zeros(len(self.KERNELS), np.int64)
        _check(self.lib.mcce_profile_read(self.ctx, _ptr(ms), _ptr(n), int(reset)), self.ctx)
        return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(self.KERNELS)}

    def record_misses(self, n_tokens: int) -> torch.Tensor:
        """Allocates and registers a miss-trace buffer [n_tokens, L, S] (uint32 bit masks, viewed as int32):
        bit k of entry (t, l, s) is set iff the k-th selected expert of that token missed the cache."""
        self._trace = torch.zeros((n_tokens, self.L, self.S), dtype=torch.int32, device=self.device)
        _check(self.lib.mcce_set_miss_trace(self.ctx, _ptr(self._trace), n_tokens), self.ctx)
        return self._trace

    def lifetimes(self):
        """(evictions, mean, standard deviation) of cache lifetimes in tokens, and the raw per-layer sums."""
        total = np.zeros(3, np.int64)
        per = np.zeros((self.L, 3), np.int64)
        _check(self.lib.mcce_lifetime_stats(self.ctx, _ptr(total), _ptr(per)), self.ctx)
        n, s1, s2 = (int(x) for x in total)
        mean = s1 / n if n else 0.0
        sd = max(0.0, s2 / n - mean * mean) ** 0.5 if n else 0.0
        return (n, mean, sd), per

    def calibrated_delta(self) -> np.ndarray:
        """Per-layer logit range from the running statistics gathered so far (mcce_calibrate_delta): the
        constants for a context in DELTA_FIXED mode, i.e. the "estimate over a calibration set" variant of
        the paper's appendix on logit-range estimation."""
        delta = np.empty(self.L, np.float32)
        _check(self.lib.mcce_calibrate_delta(self.ctx, _ptr(delta)), self.ctx)
        return delta

    def grouping(self):
        offsets = np.empty((self.L, self.E + 1), np.int32)
        perm = np.empty((self.L, self.S * self.K), np.int32)
        _check(self.lib.mcce_get_grouping(self.ctx, _ptr(offsets), _ptr(perm)), self.ctx)
        return offsets, perm


def engine_for(wl, **kw) -> Engine:
    """Engine with the shapes of a synth.Workload."""
    args = dict(L=wl.L, E=wl.E, K=wl.K, J=wl.J, n_shared=wl.n_shared, d=wl.d, I=wl.I, C_cap=wl.C, S=wl.S, lam=wl.lam,
                dtype=BF16 if wl.bf16 else F32)
    args.update(kw)
    return Engine(**args)


# -- generators ----------------------------------------------------------------------------------------
def gen_normal(out: torch.Tensor, seed: int, tensor_id: int, t: int = 0, std: float = 1.0, start: int = 0):
    """Fills `out` (fp32 or bf16, contiguous) with elements [start, start+numel) of the seeded tensor."""
    code = BF16 if out.dtype == torch.bfloat16 else F32
    assert out.dtype in (torch.float32, torch.bfloat16)
    _check(load().mcce_gen_normal(_ptr(out), code, start, out.numel(), seed, tensor_id, t, float(np.float32(std)),
                                  _stream()))
    return out


def gen_hidden_step(state: torch.Tensor, x_out: torch.Tensor, seed: int, t: int, rho: float, topic_offset: bool):
    code = BF16 if x_out.dtype == torch.bfloat16 else F32
    c = float(np.float32(np.sqrt(1.0 - float(rho) ** 2)))
    off = float(np.float32(np.sqrt(0.5))) if topic_offset else 0.0
    assert state.dtype == torch.float32 and state.numel() == x_out.numel()
    _check(load().mcce_gen_hidden_step(_ptr(state), _ptr(x_out), code, state.numel(), seed, t,
                                       float(np.float32(rho)), c, off, _stream()))
    return x_out


def gen_philox_words(n_blocks: int, seed: int, tensor_id: int, t: int, start_block: int = 0, device="cuda"):
    out = torch.empty((n_blocks, 4), dtype=torch.int32, device=device)
    _check(load().mcce_gen_philox_words(_ptr(out), start_block, n_blocks, seed, tensor_id, t, _stream()))
    return out


def route_trace_static(*, L, E, K, J, C_cap, S, lam, logits=None, hidden=None, Wr=None, fixed_delta=None,
                       delta_mode=DELTA_RUNNING, renorm=1, want_totals=True):
    """Routing over a whole trace from empty caches through the entry point that allocates nothing inside
    the library (its cache state lives in a fixed array of the library image).  Output tensors are the
    caller's; here they are torch tensors for convenience.  Returns sel_idx, sel_w[, totals]."""
    src = logits if logits is not None else hidden
    n_steps = src.shape[0]
    d = hidden.shape[-1] if hidden is not None else 8
    dtype = BF16 if (hidden is not None and hidden.dtype == torch.bfloat16) else F32
    cfg = Config(L, E, K, J, 0, d, 8, C_cap, S, lam, delta_mode, renorm, dtype, dtype, 0, src.device.index or 0)
    sel = torch.empty((n_steps, L, S, K), dtype=torch.int32, device=src.device)
    w = torch.empty((n_steps, L, S, K), dtype=torch.float32, device=src.device)
    totals = Stats()
    with torch.cuda.device(src.device):
        _check(load().mcce_route_trace_static(C.byref(cfg), n_steps, _ptr(hidden), _ptr(Wr), _ptr(logits),
                                              _ptr(fixed_delta), _ptr(sel), _ptr(w),
                                              C.byref(totals) if want_totals else None, _stream()))
    return (sel, w, totals.as_tuple()) if want_totals else (sel, w)


def belady_replay(sel_trace: torch.Tensor, n_experts: int, capacities) -> torch.Tensor:
    """Misses of Belady's optimal eviction on a selection trace [T,L,S,K] (int32, device), for each capacity:
    int64 tensor [n_capacities, L, S]."""
    assert sel_trace.dtype == torch.int32 and sel_trace.dim() == 4
    T, L, S, K = sel_trace.shape
    caps = torch.tensor(list(capacities), dtype=torch.int32, device=sel_trace.device)
    assert int(caps.min()) >= K, "Belady with a cache smaller than the K experts of one token is undefined"
    scratch = torch.empty_like(sel_trace)
    out = torch.empty((len(caps), L, S), dtype=torch.int64, device=sel_trace.device)
    with torch.cuda.device(sel_trace.device):
        _check(load().mcce_belady_replay(_ptr(sel_trace.contiguous()), T, L, S, n_experts, K, _ptr(caps), len(caps),
                                         _ptr(scratch), _ptr(out), _stream()))
    return out
