"""Seeded synthetic inputs: the five model-shaped workloads and the counter-based generator.

This module holds no arithmetic of the routing / caching / FFN method.  It only produces inputs
(hidden-state traces, router and expert weights), and is the one piece that both the CUDA library's
users and the CPU checker draw from.

Generator definition (the CUDA generator kernels implement the same definition independently):

* Integers: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3",
  SC'11).  key = (seed, 0); counter = (block_lo, block_hi, t, tensor_id) where block = flat element
  index // 4.  One call yields four uint32, hence four normal variates (elements 4*block .. +3).
* Normals: Box-Muller on two 24-bit uniforms, with ln, sin and cos evaluated by short series that
  use only +, -, *, / and sqrt in a fixed order and no fused multiply-add.  Every such operation is
  correctly rounded by IEEE-754, so the CPU (numpy float32) and the GPU produce identical bits.
* `synth_host.c` is the same definition in plain C for the host (compiled on first use; the numpy code below is
  the fallback and the reference it is tested against).
* AR(1) hidden states: h_0 = n_0, h_t = rho*h_{t-1} + sqrt(1-rho^2)*n_t (fp32, mul, mul, add);
  emitted x_t = h_t + topic_offset, rounded to bf16 (ties to even) for the bf16 workloads.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace

import numpy as np

# tensor ids (fourth counter word)
T_ROUTER, T_WG, T_WU, T_WD, T_SH_WG, T_SH_WU, T_SH_WD, T_NOISE, T_OFFSET, T_LOGITS, T_MISC = range(1, 12)

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0: int, k1: int):
    """Ten rounds of Philox-4x32 on arrays of counters (uint64 arrays holding 32-bit values)."""
    c0 = np.asarray(c0, np.uint64)
    c1 = np.asarray(c1, np.uint64) + np.zeros_like(c0)
    c2 = np.asarray(c2, np.uint64) + np.zeros_like(c0)
    c3 = np.asarray(c3, np.uint64) + np.zeros_like(c0)
    k0 &= 0xFFFFFFFF
    k1 &= 0xFFFFFFFF
    for _ in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK
        c0, c1, c2, c3 = hi1 ^ c1 ^ np.uint64(k0), lo1, hi0 ^ c3 ^ np.uint64(k1), lo0
        k0 = (k0 + _W0) & 0xFFFFFFFF
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return c0, c1, c2, c3


_F = np.float32
_LN2 = _F(0.6931471805599453)
_SQRT2 = _F(1.4142135623730951)
_QPI_SCALED = _F(0.7853981633974483 / 2097152.0)  # (pi/4) * 2^-21


def _box_muller(xa, xb):
    """Two standard normals from two uint32 words, exact-operation float32 arithmetic."""
    # radius: r = sqrt(-2 ln u1), u1 = (k+1) 2^-24 in (0, 1]
    n = (xa >> np.uint64(8)) + np.uint64(1)                      # 1 .. 2^24
    mant, ex = np.frexp(n.astype(np.float64))                    # n = mant * 2^ex, mant in [0.5,1)
    e = ex.astype(np.int64) - 1                                  # index of the top bit
    m = (mant * 2.0).astype(np.float32)                          # exact (n has <= 25 bits), [1,2)
    big = m > _SQRT2
    m = np.where(big, m * _F(0.5), m)
    e = np.where(big, e + 1, e)
    s = (m - _F(1.0)) / (m + _F(1.0))
    s2 = s * s
    poly = _F(2.0 / 11.0)
    for coef in (2.0 / 9.0, 2.0 / 7.0, 2.0 / 5.0, 2.0 / 3.0, 2.0):
        poly = poly * s2 + _F(coef)
    ln_u = poly * s + (e - 24).astype(np.float32) * _LN2
    r = np.sqrt(_F(-2.0) * ln_u)
    # angle: theta = 2 pi k2 2^-24, reduced to an octant
    k2 = xb >> np.uint64(8)
    octant = (k2 >> np.uint64(21)).astype(np.int64)
    f = k2 & np.uint64((1 << 21) - 1)
    odd = (octant & 1) == 1
    f = np.where(odd, np.uint64(1 << 21) - f, f)
    a = f.astype(np.float32) * _QPI_SCALED
    a2 = a * a
    ps = _F(1.0 / 362880.0)
    for coef in (-1.0 / 5040.0, 1.0 / 120.0, -1.0 / 6.0, 1.0):
        ps = ps * a2 + _F(coef)
    sin_a = ps * a
    pc = _F(-1.0 / 3628800.0)
    for coef in (1.0 / 40320.0, -1.0 / 720.0, 1.0 / 24.0, -0.5, 1.0):
        pc = pc * a2 + _F(coef)
    cos_a = pc
    swap = ((octant + 1) >> 1) & 1 == 1           # octants 1,2,5,6: cos <- sin, sin <- cos
    cx = np.where(swap, sin_a, cos_a)
    sx = np.where(swap, cos_a, sin_a)
    neg_c = ((octant + 2) >> 2) & 1 == 1          # octants 2..5
    neg_s = octant >= 4
    cx = np.where(neg_c, -cx, cx)
    sx = np.where(neg_s, -sx, sx)
    return r * cx, r * sx


_CHUNK = 1 << 20     # elements per work item when a large draw is split over host threads

# ---- the same definition compiled from synth_host.c (identical bits, much faster); numpy is the fallback ------
_HERE = os.path.dirname(os.path.abspath(__file__))
_HOST_SRC = os.path.join(_HERE, "synth_host.c")
_HOST_LIB = os.path.join(_HERE, "libsynth_host.so")
_host = None


def build_host(force: bool = False):
    """Compiles synth_host.c with gcc (no fused multiply-add, no fast-math); returns the library path or None."""
    try:
        if force or not os.path.exists(_HOST_LIB) or os.path.getmtime(_HOST_LIB) < os.path.getmtime(_HOST_SRC):
            subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
                                   "-o", _HOST_LIB, _HOST_SRC, "-lm"], stderr=subprocess.DEVNULL)
        return _HOST_LIB
    except (OSError, subprocess.CalledProcessError):
        return None


def _host_lib():
    global _host
    if _host is None:
        path = None if os.environ.get("MCCE_SYNTH_NUMPY") else build_host()
        _host = False
        if path:
            try:
                lib = ctypes.CDLL(path)
                lib.synth_fill.argtypes = [ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint64,
                                           ctypes.c_uint64, ctypes.c_float, ctypes.c_int, ctypes.c_void_p]
                lib.synth_fill.restype = None
                lib.synth_hidden_step.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64,
                                                  ctypes.c_float, ctypes.c_float, ctypes.c_int, ctypes.c_int,
                                                  ctypes.c_void_p]
                lib.synth_hidden_step.restype = None
                _host = lib
            except OSError:
                _host = False
    return _host or None


def _fill(seed, tensor_id, t, start, count, std, bf16):
    """std * normals of elements [start, start+count), fp32 or bf16 bits, over all host threads."""
    lib = _host_lib()
    out = np.empty(count, np.uint16 if bf16 else np.float32)
    if lib is None:
        x = _normal_numpy(seed, tensor_id, t, start, count) * _F(std)
        return to_bf16_bits(x) if bf16 else x
    pieces = [(o, min(_CHUNK, count - o)) for o in range(0, count, _CHUNK)]

    def fill(piece):
        o, n = piece
        lib.synth_fill(seed & 0xFFFFFFFF, tensor_id, t, start + o, n, float(_F(std)), int(bool(bf16)),
                       out[o:o + n].ctypes.data)

    if len(pieces) > 1:
        with ThreadPoolExecutor(os.cpu_count() or 1) as ex:
            list(ex.map(fill, pieces))
    else:
        for piece in pieces:
            fill(piece)
    return out


def normal(seed: int, tensor_id: int, t: int, start: int, count: int) -> np.ndarray:
    """Standard normals for flat elements [start, start+count) of tensor `tensor_id` at step t (fp32)."""
    return _fill(seed, tensor_id, t, start, count, 1.0, False)


def _normal_numpy(seed: int, tensor_id: int, t: int, start: int, count: int) -> np.ndarray:
    """The definition in numpy (what synth_host.c and the CUDA generator reproduce bit for bit)."""
    if count > 2 * _CHUNK and start % 4 == 0:
        out = np.empty(count, np.float32)
        pieces = [(o, min(_CHUNK, count - o)) for o in range(0, count, _CHUNK)]

        def fill(piece):
            o, n = piece
            out[o:o + n] = _normal_numpy(seed, tensor_id, t, start + o, n)

        with ThreadPoolExecutor(os.cpu_count() or 1) as ex:
            list(ex.map(fill, pieces))
        return out
    b0, b1 = start // 4, (start + count + 3) // 4
    blocks = np.arange(b0, b1, dtype=np.uint64)
    x0, x1, x2, x3 = philox4x32_10(blocks & _MASK, blocks >> np.uint64(32), t, tensor_id, seed, 0)
    n0, n1 = _box_muller(x0, x1)
    n2, n3 = _box_muller(x2, x3)
    out = np.stack([n0, n1, n2, n3], axis=1).reshape(-1)
    off = start - 4 * b0
    return np.ascontiguousarray(out[off:off + count])


def uint32_stream(seed: int, tensor_id: int, t: int, start_block: int, n_blocks: int) -> np.ndarray:
    """The raw Philox words [n_blocks, 4] (for checking a second implementation bit by bit)."""
    blocks = np.arange(start_block, start_block + n_blocks, dtype=np.uint64)
    x = philox4x32_10(blocks & _MASK, blocks >> np.uint64(32), t, tensor_id, seed, 0)
    return np.stack(x, axis=1).astype(np.uint32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    return ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def scaled_normal(seed, tensor_id, t, start, count, std: float, bf16: bool) -> np.ndarray:
    """std * n (one fp32 multiplication), as fp32 or as bf16 bit patterns."""
    return _fill(seed, tensor_id, t, start, count, std, bf16)


# ---------------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    """Shapes and input recipe of one synthetic workload (model-shaped; no trained weights)."""
    name: str
    L: int
    E: int
    K: int
    J: int
    n_shared: int
    d: int
    I: int
    C: int
    S: int
    T: int
    bf16: bool
    rho: float
    topic_offset: bool
    weight_std: float
    seed: int
    lam: float = 0.5

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)

    # -- weights ------------------------------------------------------------------------------
    def router(self, layers=None) -> np.ndarray:
        """W_r [L,E,d] fp32."""
        n = self.L * self.E * self.d
        return scaled_normal(self.seed, T_ROUTER, 0, 0, n, self.weight_std, False).reshape(self.L, self.E, self.d)

    def expert_matrix(self, tensor_id: int, l: int, e: int) -> np.ndarray:
        """One expert matrix ([I,d] for gate/up, [d,I] for down) of layer l; shared experts use the
        T_SH_* ids with e < n_shared."""
        per = self.I * self.d
        n_e = self.n_shared if tensor_id in (T_SH_WG, T_SH_WU, T_SH_WD) else self.E
        start = (l * n_e + e) * per
        x = scaled_normal(self.seed, tensor_id, 0, start, per, self.weight_std, self.bf16)
        return x.reshape((self.d, self.I) if tensor_id in (T_WD, T_SH_WD) else (self.I, self.d))

    def expert_tensor(self, tensor_id: int) -> np.ndarray:
        """All experts of all layers ([L,E,I,d] / [L,E,d,I]); only for workloads small enough."""
        n_e = self.n_shared if tensor_id in (T_SH_WG, T_SH_WU, T_SH_WD) else self.E
        n = self.L * n_e * self.I * self.d
        x = scaled_normal(self.seed, tensor_id, 0, 0, n, self.weight_std, self.bf16)
        tail = (self.d, self.I) if tensor_id in (T_WD, T_SH_WD) else (self.I, self.d)
        return x.reshape((self.L, n_e) + tail)

    # -- hidden states -----------------------------------------------------------------------
    def hidden_trace(self, T: int, rows=None):
        """Iterator over t of x_t [L,S,d] (or the given list of (l,s) rows -> [n_rows,d]):
        fp32 arrays, or bf16 bit patterns (uint16) for the bf16 workloads."""
        L, S, d = self.L, self.S, self.d
        rho = _F(self.rho)
        c = _F(np.sqrt(1.0 - float(self.rho) ** 2))

        def draw(tid, t):
            if rows is None:
                return normal(self.seed, tid, t, 0, L * S * d).reshape(L, S, d)
            return np.stack([normal(self.seed, tid, t, (l * S + s) * d, d) for l, s in rows])

        off = draw(T_OFFSET, 0) * _F(np.sqrt(0.5)) if self.topic_offset else None
        lib = _host_lib()
        if lib is not None:
            # the same recurrence through synth_host.c, in place and over all host threads
            h = None
            for t in range(T):
                n = np.ascontiguousarray(draw(T_NOISE, t))
                if h is None:
                    h = np.empty_like(n)
                out = np.empty(n.shape, np.uint16 if self.bf16 else np.float32)
                flat_h, flat_n, flat_o = h.reshape(-1), n.reshape(-1), out.reshape(-1)
                flat_off = None if off is None else np.ascontiguousarray(off).reshape(-1)
                pieces = [(o, min(_CHUNK, flat_n.size - o)) for o in range(0, flat_n.size, _CHUNK)]

                def step(piece, t=t, flat_h=flat_h, flat_n=flat_n, flat_o=flat_o, flat_off=flat_off):
                    o, m = piece
                    lib.synth_hidden_step(flat_h[o:].ctypes.data, flat_n[o:].ctypes.data,
                                          None if flat_off is None else flat_off[o:].ctypes.data, m, float(rho),
                                          float(c), int(t == 0), int(self.bf16), flat_o[o:].ctypes.data)

                if len(pieces) > 1:
                    with ThreadPoolExecutor(os.cpu_count() or 1) as ex:
                        list(ex.map(step, pieces))
                else:
                    step(pieces[0])
                yield out
            return
        h = None
        for t in range(T):
            n = draw(T_NOISE, t)
            h = n if t == 0 else rho * h + c * n
            x = h + off if off is not None else h
            yield to_bf16_bits(x).reshape(x.shape) if self.bf16 else x


# The five workloads.  J follows the paper's setting (1 for the coarse-grained models, 2 for the
# fine-grained ones); the headline promotion strength is 0.5.
TINY = Workload("tiny", L=1, E=8, K=2, J=1, n_shared=0, d=64, I=128, C=4, S=4, T=256, bf16=False,
                rho=0.9, topic_offset=False, weight_std=1.0 / 8.0, seed=0)
QWEN = Workload("qwen1.5-moe-a2.7b-shaped", L=24, E=60, K=4, J=2, n_shared=4, d=2048, I=1408, C=30,
                S=256, T=1024, bf16=True, rho=0.8, topic_offset=True, weight_std=0.02, seed=1)
OLMOE = Workload("olmoe-shaped", L=16, E=64, K=8, J=2, n_shared=0, d=2048, I=1024, C=32, S=512,
                 T=1024, bf16=True, rho=0.8, topic_offset=True, weight_std=0.02, seed=2)
DEEPSEEK = Workload("deepseek-v2-lite-shaped", L=26, E=64, K=6, J=2, n_shared=2, d=2048, I=1408,
                    C=24, S=256, T=2048, bf16=True, rho=0.7, topic_offset=True, weight_std=0.02, seed=3)
MIXTRAL = Workload("mixtral-8x7b-shaped", L=32, E=8, K=2, J=1, n_shared=0, d=4096, I=14336, C=4,
                   S=64, T=2048, bf16=True, rho=0.9, topic_offset=False, weight_std=0.02, seed=4)

WORKLOADS = {w.name: w for w in (TINY, QWEN, OLMOE, DEEPSEEK, MIXTRAL)}
ALIASES = {"tiny": TINY, "qwen": QWEN, "olmoe": OLMOE, "deepseek": DEEPSEEK, "mixtral": MIXTRAL}
