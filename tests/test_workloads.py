"""The synthetic workloads carry the shapes the paper states for its models, and the seeded generator has the
statistics the input recipe promises (CPU only)."""
import os

import numpy as np

from paper_2412_00099_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_model_shapes.txt")


def test_workload_shapes_match_table_1():
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, shared, experts, top_k, params = line.split()
        wl = synth.ALIASES[name]
        assert (wl.n_shared, wl.E, wl.K) == (int(shared), int(experts), int(top_k))
        per_expert = 3 * wl.d * wl.I / 1e6                  # gate, up and down projections of a SwiGLU expert
        assert abs(per_expert - float(params)) / float(params) < 0.01
    # guaranteed top-J as in the paper's implementation details: 1 for the coarse models, 2 for the granular ones
    assert synth.MIXTRAL.J == 1 and synth.QWEN.J == 2 and synth.DEEPSEEK.J == 2


def test_hidden_trace_statistics():
    wl = synth.QWEN.with_(L=1, S=6, d=512)
    xs = np.stack([synth.bf16_bits_to_f32(x) for x in wl.hidden_trace(400)])          # [T, 1, S, d]
    off = xs.mean(axis=0)                                                              # topic offset per element
    h = xs - off
    assert abs(off.var() - 0.5) < 0.06 and abs(h.var() - 1.0) < 0.05                   # N(0, 0.5 I) offset, unit AR(1)
    lag1 = (h[1:] * h[:-1]).mean() / h.var()
    assert abs(lag1 - wl.rho) < 0.03                                                   # AR(1) coefficient
    nooff = synth.MIXTRAL.with_(L=1, S=2, d=256)
    ys = np.stack([synth.bf16_bits_to_f32(x) for x in nooff.hidden_trace(300)])
    assert abs(ys.mean()) < 0.05


def test_weights_have_the_stated_spread():
    w = synth.bf16_bits_to_f32(synth.QWEN.expert_matrix(synth.T_WG, 3, 7))
    assert abs(w.std() - 0.02) < 2e-4 and abs(w.mean()) < 2e-4
    r = synth.TINY.router()
    assert abs(r.var() - 1.0 / synth.TINY.d) < 0.15 / synth.TINY.d * 8               # N(0, 1/d), 512 samples


def test_compiled_host_generator_equals_the_numpy_definition(monkeypatch):
    """synth_host.c against the numpy code it restates: normals (ragged starts, beyond 2^32 blocks), scaled bf16
    weights and the AR(1) trace, bit for bit."""
    assert synth.build_host() is not None, "gcc could not build synth_host.c"
    synth._host = None
    cases = [(1, 2, 0, 0, 1000), (5, 3, 7, 4096 + 3, 100_003), (9, 8, 13, (1 << 34) + 8, 5000), (0, 11, 2, 1, 7),
             (3, 8, 1, 0, 2_500_000)]
    fast = [(synth.normal(*c), synth.scaled_normal(*c, 0.02, True)) for c in cases]
    wls = (synth.TINY.with_(S=5, L=2), synth.QWEN.with_(L=2, S=7, d=64), synth.MIXTRAL.with_(L=1, S=3, d=128))
    fast_traces = [list(w.hidden_trace(5)) + list(w.hidden_trace(5, rows=[(0, 1), (w.L - 1, 2)])) for w in wls]
    assert synth._host_lib() is not None
    monkeypatch.setenv("MCCE_SYNTH_NUMPY", "1")
    synth._host = None
    try:
        assert synth._host_lib() is None
        for c, (n, b) in zip(cases, fast):
            assert np.array_equal(n.view(np.uint32), synth.normal(*c).view(np.uint32))
            assert np.array_equal(b, synth.scaled_normal(*c, 0.02, True))
        for w, tr in zip(wls, fast_traces):
            slow = list(w.hidden_trace(5)) + list(w.hidden_trace(5, rows=[(0, 1), (w.L - 1, 2)]))
            for a, b in zip(tr, slow):
                assert a.dtype == b.dtype and a.shape == b.shape and np.array_equal(a.view(np.uint8), b.view(np.uint8))
    finally:
        synth._host = None
