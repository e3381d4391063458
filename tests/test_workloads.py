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
