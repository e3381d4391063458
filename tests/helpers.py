"""Shared pieces of the GPU parity tests: build the same seeded inputs for the CUDA library and for
the CPU oracle, and the two comparison protocols (identical logits -> bit-exact; hidden states ->
follow mode with near-tie accounting)."""
from __future__ import annotations

import numpy as np
import torch

from oracle import oracle as orc
from paper_2412_00099_b200 import synth

NEAR_TIE = 1e-4          # a routing difference is only acceptable if an outcome-deciding gap is below this
LOGIT_RTOL = 1e-5        # |z_gpu - z_oracle| <= LOGIT_RTOL * max(1, |z_oracle|)
FFN_ATOL, FFN_RTOL = 2e-3, 1e-2


def oracle_for(wl, threads=4, **kw):
    args = dict(n_layers=wl.L, n_experts=wl.E, top_k=wl.K, top_j=wl.J, n_shared=wl.n_shared, d_model=wl.d,
                d_ff=wl.I, cache_capacity=wl.C, n_streams=wl.S, lam=wl.lam, delta_mode=0, renorm=1,
                dtype=1 if wl.bf16 else 0)
    fixed = kw.pop("fixed_delta", None)
    args.update(kw)
    return orc.Oracle(orc.OracleConfig(**args), fixed_delta=fixed, threads=threads)


def to_dev(a: np.ndarray, bf16: bool = False) -> torch.Tensor:
    """numpy -> cuda tensor; uint16 arrays are bf16 bit patterns."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def assert_state_equal(eng, o):
    order, ever, dsum, cnt = eng.cache_state()
    assert np.array_equal(order, o.order())
    assert np.array_equal(ever, o.ever)
    if o.cfg.delta_mode == 0:
        assert np.array_equal(dsum.view(np.uint32), o.sum_range.view(np.uint32))
        assert cnt == int(o.count.flat[0])
    total, per_layer = eng.cache_stats()
    ot, opl = o.stats()
    assert list(total) == ot.tolist()
    assert [list(p) for p in per_layer] == opl.tolist()
    if eng.cfg.track_lifetime:
        assert eng.lifetimes()[1].tolist() == o.life.sum(axis=1).tolist()


def check_route_exact(eng, o, z_all: np.ndarray, chunk: int = 1, check_every: int = 8):
    """Feed identical fp32 logits [T,L,S,E] to both; indices, weights, states and counters must agree
    (indices, states, counters, Delta sums: bit for bit; weights: rel 1e-5)."""
    T = z_all.shape[0]
    zd = to_dev(z_all)
    t = 0
    while t < T:
        n = min(chunk, T - t)
        sel, w = eng.route_step(logits=zd[t:t + n], n_steps=n)
        sel, w = sel.cpu().numpy(), w.cpu().numpy()
        for i in range(n):
            osel, ow = o.route(z_all[t + i])
            assert np.array_equal(sel[i], osel), "selection differs at token %d" % (t + i)
            assert np.allclose(w[i], ow, rtol=1e-5, atol=1e-7)
        t += n
        if (t // chunk) % check_every == 0 or t >= T:
            assert_state_equal(eng, o)


def check_route_follow(eng, o, Wr: np.ndarray, hidden_iter, bf16: bool):
    """From hidden states.  The oracle forms its own logits; the library's logits must be within
    LOGIT_RTOL of them.  The state machine is then advanced on the library's logits (so both sides
    stay aligned) and must reproduce the library's selection exactly; wherever the oracle's decision
    on its OWN logits differs, the deciding gap must be a near tie.  Returns (steps, near_ties)."""
    near, steps = 0, 0
    max_dz = 0.0
    for x in hidden_iter:
        xd = to_dev(x)
        sel, w, zg = eng.route_step(hidden=xd[None], n_steps=1, want_logits=True)
        sel, w, zg = sel.cpu().numpy()[0], w.cpu().numpy()[0], zg.cpu().numpy()[0]
        z_own = o.logits(Wr, x)
        dz = np.abs(zg - z_own) / np.maximum(1.0, np.abs(z_own))
        max_dz = max(max_dz, float(dz.max()))
        assert dz.max() <= LOGIT_RTOL, "router logits off by %g" % dz.max()
        snap = o.snapshot()
        sel_own, _, margin_own, _ = o.route(z_own, want_margin=True)
        o.restore(snap)
        osel, ow = o.route(zg)
        assert np.array_equal(sel, osel)
        assert np.allclose(w, ow, rtol=1e-5, atol=1e-7)
        differs = np.any(sel_own != osel, axis=-1)
        if differs.any():
            assert (margin_own[differs] < NEAR_TIE).all(), "unexplained routing difference"
            near += int(differs.sum())
        steps += sel.shape[0] * sel.shape[1]
    assert_state_equal(eng, o)
    return steps, near, max_dz


def ffn_close(y_gpu: np.ndarray, y_ref: np.ndarray):
    err = np.abs(y_gpu - y_ref)
    bound = FFN_ATOL + FFN_RTOL * np.abs(y_ref)
    assert (err <= bound).all(), "FFN mismatch: max abs %g, worst ratio %g" % (err.max(), (err / bound).max())
    return float(err.max()), float((err / np.maximum(np.abs(y_ref), 1e-6)).max())


def small_workload(base, **kw):
    return base.with_(**kw)


def weights_for(wl):
    """All expert tensors of a (small) workload on the CPU: dict name -> array."""
    out = {"Wg": wl.expert_tensor(synth.T_WG), "Wu": wl.expert_tensor(synth.T_WU), "Wd": wl.expert_tensor(synth.T_WD)}
    if wl.n_shared:
        out.update(shWg=wl.expert_tensor(synth.T_SH_WG), shWu=wl.expert_tensor(synth.T_SH_WU),
                   shWd=wl.expert_tensor(synth.T_SH_WD))
    else:
        out.update(shWg=None, shWu=None, shWd=None)
    return out
