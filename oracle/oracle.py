"""ctypes front end of the CPU oracle (``mcce_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg, never by the product package.  It adds no arithmetic of its own; every number
comes from the C file, which follows the paper formula by formula.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mcce_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc.  No fused multiply-add, no fast-math: each fp32 operation of
    the routing decision is one IEEE round-to-nearest operation."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
             "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_layers", "n_experts", "top_k", "top_j", "n_shared", "d_model", "d_ff",
                 "cache_capacity", "n_streams")] + [
        ("lam", C.c_float), ("delta_mode", C.c_int32), ("renorm", C.c_int32), ("dtype", C.c_int32),
        ("rerank_mode", C.c_int32), ("max_rank", C.c_int32), ("cum_threshold", C.c_float)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_belady_misses.restype = C.c_int64
        _lib.orc_lru_misses.restype = C.c_int64
        _lib.orc_cumsum_threshold.restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


@dataclass
class OracleConfig:
    n_layers: int
    n_experts: int
    top_k: int
    top_j: int
    n_shared: int
    d_model: int
    d_ff: int
    cache_capacity: int
    n_streams: int
    lam: float
    delta_mode: int = 0
    renorm: int = 1
    dtype: int = 1  # 0 fp32, 1 bf16 (uint16 storage)
    rerank_mode: int = 0  # 0 Cache-Prior, 1 Max-Rank, 2 Cumsum-Threshold
    max_rank: int = 0
    cum_threshold: float = 0.0

    def c(self) -> _Cfg:
        return _Cfg(self.n_layers, self.n_experts, self.top_k, self.top_j, self.n_shared,
                    self.d_model, self.d_ff, self.cache_capacity, self.n_streams, self.lam,
                    self.delta_mode, self.renorm, self.dtype, self.rerank_mode, self.max_rank,
                    self.cum_threshold)


def _split(n: int, parts: int):
    parts = max(1, min(parts, n))
    edges = [n * i // parts for i in range(parts + 1)]
    return [(edges[i], edges[i + 1]) for i in range(parts) if edges[i + 1] > edges[i]]


class Oracle:
    """Routing state of every (layer, stream) plus the calls that advance it by one token."""

    def __init__(self, cfg: OracleConfig, fixed_delta=None, threads: int = 1):
        self.cfg = cfg
        L, S, E = cfg.n_layers, cfg.n_streams, cfg.n_experts
        assert E <= 1024 and 1 <= cfg.top_k <= E and 0 <= cfg.top_j <= cfg.top_k
        self.stamp = np.zeros((L, S, E), np.int64)
        self.ever = np.zeros((L, S, E), np.uint8)
        self.sum_range = np.zeros((L, S), np.float32)
        self.count = np.zeros((L, S), np.int64)
        self.tok = np.zeros((L, S), np.int64)
        self.counters = np.zeros((L, S, 4), np.int64)
        self.load_tok = np.zeros((L, S, E), np.int64)
        self.life = np.zeros((L, S, 3), np.int64)
        self.last_miss_mask = np.zeros((L, S), np.uint32)   # of the latest token: bit k = slot k missed
        self.fixed_delta = None if fixed_delta is None else np.ascontiguousarray(fixed_delta, np.float32)
        self.threads = threads
        self._pool = ThreadPoolExecutor(threads) if threads > 1 else None

    # -- helpers ---------------------------------------------------------------------------
    def _par(self, fn):
        S = self.cfg.n_streams
        if self._pool is None:
            fn(0, S)
        else:
            list(self._pool.map(lambda r: fn(*r), _split(S, self.threads)))

    def snapshot(self):
        return tuple(a.copy() for a in (self.stamp, self.ever, self.sum_range, self.count, self.tok,
                                        self.counters, self.load_tok, self.life))

    def restore(self, snap):
        for dst, src in zip((self.stamp, self.ever, self.sum_range, self.count, self.tok,
                             self.counters, self.load_tok, self.life), snap):
            dst[...] = src

    def reset(self, init_order=None, keep_delta_stats: bool = False):
        cfg = self.cfg
        self.stamp[...] = 0
        self.ever[...] = 0
        self.tok[...] = 0
        self.counters[...] = 0
        self.load_tok[...] = 0
        self.life[...] = 0
        if not keep_delta_stats:
            self.sum_range[...] = 0
            self.count[...] = 0
        if init_order is not None:
            init_order = np.ascontiguousarray(init_order, np.int32)
            for l in range(cfg.n_layers):
                for s in range(cfg.n_streams):
                    lib().orc_import_order(_p(init_order[l, s]), cfg.n_experts, cfg.cache_capacity,
                                           _p(self.stamp[l, s]), _p(self.ever[l, s]))

    # -- the method -------------------------------------------------------------------------
    def logits(self, Wr: np.ndarray, hidden: np.ndarray) -> np.ndarray:
        """z = W_r x for every (layer, stream); hidden is fp32 or bf16-as-uint16 [L,S,d]."""
        cfg = self.cfg
        assert Wr.dtype == np.float32 and Wr.flags.c_contiguous and hidden.flags.c_contiguous
        assert hidden.dtype == (np.uint16 if cfg.dtype else np.float32)
        z = np.empty((cfg.n_layers, cfg.n_streams, cfg.n_experts), np.float32)
        cc = cfg.c()
        self._par(lambda a, b: lib().orc_router_logits_slab(C.byref(cc), _p(Wr), _p(hidden), _p(z), a, b))
        return z

    def route(self, z: np.ndarray, want_margin: bool = False):
        """Advance every (layer, stream) by one token given its logits z [L,S,E] (fp32).
        Returns sel [L,S,K] int32 (rank order of z'), w [L,S,K] fp32, and optionally margins and
        the Delta used."""
        cfg = self.cfg
        z = np.ascontiguousarray(z, np.float32)
        L, S, K = cfg.n_layers, cfg.n_streams, cfg.top_k
        sel = np.empty((L, S, K), np.int32)
        w = np.empty((L, S, K), np.float32)
        margin = np.empty((L, S), np.float32) if want_margin else None
        delta = np.empty((L, S), np.float32) if want_margin else None
        cc = cfg.c()
        self._par(lambda a, b: lib().orc_route_slab(
            C.byref(cc), _p(z), _p(self.fixed_delta), _p(self.stamp), _p(self.ever),
            _p(self.sum_range), _p(self.count), _p(self.tok), _p(self.counters), _p(sel), _p(w),
            _p(margin), _p(delta), _p(self.load_tok), _p(self.life), _p(self.last_miss_mask), a, b))
        if want_margin:
            return sel, w, margin, delta
        return sel, w

    def ffn(self, hidden, sel, w, Wg, Wu, Wd, shWg=None, shWu=None, shWd=None) -> np.ndarray:
        """y = sum_k w_k E_sel_k(x) + sum_shared E_sh(x) for every (layer, stream)."""
        cfg = self.cfg
        y = np.empty((cfg.n_layers, cfg.n_streams, cfg.d_model), np.float32)
        sel = np.ascontiguousarray(sel, np.int32)
        w = np.ascontiguousarray(w, np.float32)
        for a in (hidden, Wg, Wu, Wd, shWg, shWu, shWd):
            assert a is None or a.flags.c_contiguous
        cc = cfg.c()
        self._par(lambda a, b: lib().orc_ffn_slab(
            C.byref(cc), _p(hidden), _p(sel), _p(w), _p(Wg), _p(Wu), _p(Wd), _p(shWg), _p(shWu),
            _p(shWd), _p(y), a, b))
        return y

    # -- state export -----------------------------------------------------------------------
    def order(self) -> np.ndarray:
        """Resident experts of every (layer, stream), most recently used first, -1 padded [L,S,C]."""
        cfg = self.cfg
        out = np.empty((cfg.n_layers, cfg.n_streams, cfg.cache_capacity), np.int32)
        for l in range(cfg.n_layers):
            for s in range(cfg.n_streams):
                lib().orc_export_order(_p(self.stamp[l, s]), cfg.n_experts, cfg.cache_capacity,
                                       _p(out[l, s]))
        return out

    def lifetimes(self):
        """(evictions, mean, standard deviation) of the cache lifetimes of evicted experts, in tokens."""
        n, s1, s2 = (int(x) for x in self.life.sum(axis=(0, 1)))
        if n == 0:
            return 0, 0.0, 0.0
        mean = s1 / n
        return n, mean, max(0.0, s2 / n - mean * mean) ** 0.5

    def stats(self):
        """{steps, selections, misses, cold_misses} summed over everything, and per layer [L,4]."""
        per_layer = self.counters.sum(axis=1)
        return per_layer.sum(axis=0), per_layer


# -- stateless pieces -----------------------------------------------------------------------------
def expert_ffn(x, Wg, Wu, Wd, dtype: int) -> np.ndarray:
    """One expert on one token, double precision output [d]."""
    I, d = Wg.shape
    o = np.empty(d, np.float64)
    lib().orc_expert_ffn(_p(np.ascontiguousarray(x)), _p(np.ascontiguousarray(Wg)),
                         _p(np.ascontiguousarray(Wu)), _p(np.ascontiguousarray(Wd)), d, I, dtype, _p(o))
    return o


def promote(subset, all_):
    subset = np.ascontiguousarray(subset, np.int32)
    all_ = np.ascontiguousarray(all_, np.int32)
    out = np.empty(len(all_), np.int32)
    lib().orc_promote(_p(subset), len(subset), _p(all_), len(all_), _p(out))
    return out.tolist()


def max_rank(r, in_cache, M: int, J: int):
    r = np.ascontiguousarray(r, np.int32)
    in_cache = np.ascontiguousarray(in_cache, np.uint8)
    out = np.empty(len(r), np.int32)
    lib().orc_max_rank(_p(r), len(r), _p(in_cache), M, J, _p(out))
    return out.tolist()


def cumsum_threshold(r, w, in_cache, p: float, J: int):
    r = np.ascontiguousarray(r, np.int32)
    w = np.ascontiguousarray(w, np.float32)
    in_cache = np.ascontiguousarray(in_cache, np.uint8)
    out = np.empty(len(r), np.int32)
    M = lib().orc_cumsum_threshold(_p(r), len(r), _p(w), _p(in_cache), C.c_float(p), J, _p(out))
    return M, out.tolist()


def belady_misses(trace, E: int, Ccap: int) -> int:
    trace = np.ascontiguousarray(trace, np.int32)
    T, K = trace.shape
    return int(lib().orc_belady_misses(_p(trace), T, K, E, Ccap))


def lru_misses(trace, E: int, Ccap: int) -> int:
    trace = np.ascontiguousarray(trace, np.int32)
    T, K = trace.shape
    return int(lib().orc_lru_misses(_p(trace), T, K, E, Ccap))
