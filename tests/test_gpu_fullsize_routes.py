"""Routing parity at full size over ALL (layer, stream) pairs, for every configuration the workloads list:
each model-shaped workload with each of its cache capacities and each promotion strength of the sweep.

Inputs (router, hidden states of every pair) come from the host generator and are uploaded, so both sides see
the same bits.  The library routes one token per launch from hidden states, as the benchmark does; the oracle
follows every pair in the follow-mode protocol of helpers.check_route_follow: its own fp64 logits must lie
within the logit tolerance of the library's; advanced on the library's logits it must reproduce every
selection, weight, cache state and counter; and where its decision on its OWN logits differs, the deciding gap
must be a near tie (< 1e-4).  Near-tie counts are printed per configuration.  One more case per workload feeds
eight tokens per launch (the batched launch configuration: cache state stays in registers across the tokens,
and the logits come from one GEMM launch or from the single cooperative kernel).

No expert weights are needed, so every case fits in a few hundred MB."""
import os

import numpy as np
import pytest
import torch

from paper_2412_00099_b200 import synth

pytestmark = pytest.mark.gpu

T_TOKENS = 16
SWEEP = [(synth.QWEN, (15, 30, 45)), (synth.OLMOE, (16, 32)), (synth.DEEPSEEK, (24,)), (synth.MIXTRAL, (4,))]
LAMBDAS = (0.0, 0.5, 1.0)

_inputs = {}


def inputs_of(wl):
    """Router, hidden states of T_TOKENS tokens of every pair (host generator) and the oracle's own logits for
    them; shared by all (C, lambda) cases of a workload.  Only one workload is kept at a time."""
    from oracle import oracle as orc
    if wl.name not in _inputs:
        _inputs.clear()
        Wr = wl.router()
        xs = list(wl.hidden_trace(T_TOKENS))
        o = orc.Oracle(orc.OracleConfig(wl.L, wl.E, wl.K, wl.J, 0, wl.d, 8, wl.C, wl.S, 0.0, 0, 1, 1),
                       threads=os.cpu_count() or 1)
        z_own = [o.logits(Wr, x) for x in xs]
        _inputs[wl.name] = (Wr, xs, z_own)
    return _inputs[wl.name]


def route_engine(wl, **kw):
    from paper_2412_00099_b200 import binding as mb
    import helpers as H
    # the expert buffers of the context are not used: smallest intermediate size, no shared experts
    eng = mb.engine_for(wl, n_shared=0, I=8, ffn_impl=mb.FFN_SIMT, **kw)
    eng.set_router(H.to_dev(inputs_of(wl)[0]))
    return eng


# tokens per launch: 1 as in the benchmark's decode step; one more case per workload feeds 8 tokens per launch
CASES = []
for _wl, _caps in SWEEP:
    CASES += [(_wl, C, lam, 1) for C in _caps for lam in LAMBDAS] + [(_wl, _wl.C, 0.5, 8)]


@pytest.mark.parametrize("base,C,lam,n", CASES,
                         ids=["%s-C%d-lam%g-%dtok" % (w.name, C, lam, n) for w, C, lam, n in CASES])
def test_every_pair_follows_the_oracle(base, C, lam, n):
    from oracle import oracle as orc
    import helpers as H
    wl = base.with_(C=C, lam=lam)
    Wr, xs, z_own = inputs_of(wl)
    eng = route_engine(wl)
    o = orc.Oracle(orc.OracleConfig(wl.L, wl.E, wl.K, wl.J, 0, wl.d, 8, wl.C, wl.S, wl.lam, 0, 1, 1),
                   threads=os.cpu_count() or 1)
    near, worst = 0, 0.0
    for t0 in range(0, T_TOKENS, n):
        xd = torch.stack([H.to_dev(x) for x in xs[t0:t0 + n]])
        sel_n, w_n, zg_n = (a.cpu().numpy() for a in eng.route_step(hidden=xd, n_steps=n, want_logits=True))
        for i in range(n):
            t, sel, w, zg = t0 + i, sel_n[i], w_n[i], zg_n[i]
            dz = np.abs(zg - z_own[t]) / np.maximum(1.0, np.abs(z_own[t]))
            worst = max(worst, float(dz.max()))
            assert dz.max() <= H.LOGIT_RTOL
            snap = o.snapshot()
            sel_own, _, margin_own, _ = o.route(z_own[t], want_margin=True)
            o.restore(snap)
            osel, ow = o.route(zg)
            assert np.array_equal(sel, osel), "selection differs at token %d" % t
            assert np.allclose(w, ow, rtol=1e-5, atol=1e-7)
            differs = np.any(sel_own != osel, axis=-1)
            if differs.any():
                assert (margin_own[differs] < H.NEAR_TIE).all(), "unexplained routing difference at token %d" % t
                near += int(differs.sum())
    H.assert_state_equal(eng, o)                  # recency lists, ever-resident bits, Delta sums, counters
    total, _ = eng.cache_stats()
    print("%s C=%d lambda=%g, %d token(s) per launch (kernel kind %d): %d steps (all %d pairs x %d tokens), "
          "%d near ties, max logit err %.2e, miss rate %.4f"
          % (wl.name, C, lam, n, eng.router_kernel_kind(n), total[0], wl.L * wl.S, T_TOKENS, near, worst,
             total[2] / total[1]))
    eng.close()
