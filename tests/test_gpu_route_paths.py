"""The kernels behind mcce_route_step, each against the oracle: the routing tail with a group of lanes per
stream and the warp-per-stream tail on identical logits (bit-exact), the router-resident tensor-core GEMM
followed by the tail, and the single cooperative kernel that runs both (logits within tolerance, every
decision reproduced by the oracle on the library's own logits, near ties counted)."""
import numpy as np
import pytest
import torch

from paper_2412_00099_b200 import binding as mb
from paper_2412_00099_b200 import synth
from tests import helpers as H
from tests.test_gpu_parity import ROUTE_CASES, ar1_logits

pytestmark = pytest.mark.gpu


GROUP_CASES = [c for c in ROUTE_CASES if c[0] <= 64] + [
    # E,  K, J, C,  lam, delta_mode, renorm, quant
    (64, 16, 3, 40, 0.5, 0, 1, None),      # two selections per lane of an eight-lane group
    (64, 12, 2, 10, 0.8, 0, 0, 0.25),      # C < K, K not a multiple of 4, no renormalisation, ties
    (16, 16, 2, 8, 0.5, 0, 1, None),       # K = E with two lanes per stream
    (8, 8, 1, 3, 0.7, 1, 1, 0.5),          # K = E with one lane per stream, fixed Delta
    (24, 7, 7, 24, 0.3, 0, 1, None),       # four lanes per stream, the last lane empty
    (57, 9, 0, 57, 1.0, 0, 1, 0.125),      # odd expert count: scalar loads of the logits
]


@pytest.mark.parametrize("E,K,J,C,lam,dm,renorm,quant", GROUP_CASES)
@pytest.mark.parametrize("chunk", [1, 5])
def test_group_tail_from_logits_is_bit_exact(E, K, J, C, lam, dm, renorm, quant, chunk):
    """Without lifetime tracking and with at most 64 experts the group-of-lanes tail runs (one to eight lanes
    per stream); several streams share a warp, the last warp of a layer is partly idle (S = 19)."""
    L, S, T = 3, 19, 40
    wl = synth.TINY.with_(L=L, E=E, K=K, J=J, C=C, S=S, lam=lam, d=64, I=64)
    fixed = np.linspace(2.0, 4.0, L).astype(np.float32) if dm else None
    eng = mb.engine_for(wl, delta_mode=dm, renorm=renorm, track_lifetime=False)
    if dm:
        eng.set_router(torch.zeros((L, E, 64), device="cuda"), H.to_dev(fixed))
    o = H.oracle_for(wl, delta_mode=dm, renorm=renorm, fixed_delta=fixed)
    z = ar1_logits(E * 77 + K, T, L, S, E, quant=quant)
    H.check_route_exact(eng, o, z, chunk=chunk, check_every=2)
    eng.close()


def test_group_tail_and_warp_tail_agree_bit_for_bit():
    """Same logits through both tails (lifetime tracking selects the warp-per-stream kernel): identical
    selections, cache states and counters; handing the state from one kernel to the other in mid-trace works."""
    wl = synth.QWEN.with_(L=2, S=70, d=64, I=64, C=15)
    z = H.to_dev(ar1_logits(5, 36, wl.L, wl.S, wl.E, quant=0.125))
    a, b = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT), mb.engine_for(wl, ffn_impl=mb.FFN_SIMT, track_lifetime=True)
    sa, wa = a.route_step(logits=z, n_steps=36)
    sb, wb = b.route_step(logits=z, n_steps=36)
    assert torch.equal(sa, sb)
    assert torch.allclose(wa, wb, rtol=1e-6, atol=0)
    assert list(a.cache_stats()[0]) == list(b.cache_stats()[0])
    for x, y in zip(a.cache_state()[:3], b.cache_state()[:3]):
        assert np.array_equal(x, y)
    a.close()
    b.close()


def follow_chunked(eng, o, Wr, xs, chunk, kind):
    """check_route_follow with `chunk` tokens per launch (a list: the lengths of successive launches)."""
    T = xs.shape[0]
    xd = torch.from_numpy(xs.view(np.int16)).cuda().view(torch.bfloat16)
    near, max_dz, t, i = 0, 0.0, 0, 0
    while t < T:
        n = min(chunk[i % len(chunk)] if isinstance(chunk, (list, tuple)) else chunk, T - t)
        i += 1
        if kind is not None:
            assert eng.router_kernel_kind(n) == kind
        sel, w, zg = (a.cpu().numpy() for a in eng.route_step(hidden=xd[t:t + n], n_steps=n, want_logits=True))
        for i in range(n):
            z_own = o.logits(Wr, xs[t + i])
            dz = np.abs(zg[i] - z_own) / np.maximum(1.0, np.abs(z_own))
            max_dz = max(max_dz, float(dz.max()))
            assert dz.max() <= H.LOGIT_RTOL, "router logits off by %g" % dz.max()
            snap = o.snapshot()
            sel_own, _, margin_own, _ = o.route(z_own, want_margin=True)
            o.restore(snap)
            osel, ow = o.route(zg[i])
            assert np.array_equal(sel[i], osel), "selection differs at token %d" % (t + i)
            assert np.allclose(w[i], ow, rtol=1e-5, atol=1e-7)
            differs = np.any(sel_own != osel, axis=-1)
            if differs.any():
                assert (margin_own[differs] < H.NEAR_TIE).all(), "unexplained routing difference"
                near += int(differs.sum())
        t += n
    H.assert_state_equal(eng, o)
    return near, max_dz


FUSED_CASES = [
    # enough layers for the K parts of all layers to fill the device; S spans two stream tiles with a ragged tail
    (synth.QWEN, dict(L=20, S=200, d=512, C=15), 8),
    (synth.OLMOE, dict(L=19, S=130, d=512), 5),
    (synth.MIXTRAL, dict(L=32, S=64, d=1024), 8),
    (synth.QWEN, dict(L=24, S=97, d=448, E=36, K=3, C=9), 4),     # experts not a multiple of 8, one ragged tile
]


@pytest.mark.parametrize("base,kw,chunk", FUSED_CASES)
def test_fused_route_kernel_from_hidden_states(base, kw, chunk):
    wl = base.with_(**kw)
    Wr = wl.router()
    xs = np.stack(list(wl.hidden_trace(2 * chunk + 1)))
    eng, o = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT, route_impl=mb.ROUTE_FUSED), H.oracle_for(wl)
    eng.set_router(H.to_dev(Wr))
    assert eng.router_kernel_kind(chunk) == mb.ROUTER_FUSED
    # two fused launches of several tokens, then one of a single token
    near, dz = follow_chunked(eng, o, Wr, xs[:2 * chunk], chunk, mb.ROUTER_FUSED)
    near2, dz2 = follow_chunked(eng, o, Wr, xs[2 * chunk:], 1, mb.ROUTER_FUSED)
    print("%s fused: %d near ties, max logit err %.2e" % (wl.name, near + near2, max(dz, dz2)))
    eng.close()


@pytest.mark.parametrize("base,kw", [
    (synth.QWEN, dict(L=3, S=300, d=512, C=30)),        # three stream tiles, the last one ragged
    (synth.DEEPSEEK, dict(L=2, S=128, d=2048)),
    (synth.QWEN, dict(L=2, S=40, d=256, E=80, K=4)),    # the most experts the router-resident GEMM takes
    (synth.QWEN, dict(L=24, S=97, d=448, E=37, K=3, C=9)),   # experts not a multiple of 4: no fused kernel either
])
def test_router_resident_gemm_then_tail(base, kw):
    wl = base.with_(**kw)
    Wr = wl.router()
    xs = np.stack(list(wl.hidden_trace(10)))
    eng, o = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT, route_impl=mb.ROUTE_FUSED), H.oracle_for(wl)
    eng.set_router(H.to_dev(Wr))
    assert eng.router_kernel_kind(8) == mb.ROUTER_RESIDENT_TAIL     # no fused kernel for this shape, even if asked
    near, dz = follow_chunked(eng, o, Wr, xs[:8], 8, mb.ROUTER_RESIDENT_TAIL)
    near2, dz2 = follow_chunked(eng, o, Wr, xs[8:], 1, mb.ROUTER_RESIDENT_TAIL)
    print("%s resident: %d near ties, max logit err %.2e" % (wl.name, near + near2, max(dz, dz2)))
    eng.close()


def test_fused_launches_of_varying_length_and_a_reset_in_between():
    """The fused kernel accumulates a launch's logits in an array that it leaves at zero, and its two sets of
    ready counters alternate from launch to launch: launches of different lengths (some of them two-kernel
    launches of one or two tokens in between) must not see anything of each other, nor must a reset."""
    wl = synth.QWEN.with_(L=20, S=200, d=512, C=15)
    Wr = wl.router()
    xs = np.stack(list(wl.hidden_trace(41)))
    eng, o = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT), H.oracle_for(wl)
    eng.set_router(H.to_dev(Wr))
    assert eng.router_kernel_kind(8) == mb.ROUTER_FUSED and eng.router_kernel_kind(2) == mb.ROUTER_RESIDENT_TAIL
    near, dz = follow_chunked(eng, o, Wr, xs[:33], [8, 3, 1, 8, 5, 2, 6], None)
    eng.reset()
    o = H.oracle_for(wl)
    near2, dz2 = follow_chunked(eng, o, Wr, xs[33:], [5, 3], mb.ROUTER_FUSED)
    print("varying launches: %d near ties, max logit err %.2e" % (near + near2, max(dz, dz2)))
    eng.close()


def test_fused_kernel_and_two_kernel_path_leave_the_same_state():
    """The same trace once in launches of eight tokens (fused) and once token by token (two kernels): the
    logits agree to rounding of the differently split reduction, selections and cache state are identical."""
    wl = synth.QWEN.with_(L=20, S=160, d=512, C=15)
    Wr = H.to_dev(wl.router())
    xs = np.stack(list(wl.hidden_trace(16)))
    x = torch.from_numpy(xs.view(np.int16)).cuda().view(torch.bfloat16)
    a = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT, route_impl=mb.ROUTE_FUSED)
    b = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT, route_impl=mb.ROUTE_TWO_KERNELS)
    a.set_router(Wr)
    b.set_router(Wr)
    assert a.router_kernel_kind(16) == mb.ROUTER_FUSED and b.router_kernel_kind(1) == mb.ROUTER_RESIDENT_TAIL
    sa, wa, za = a.route_step(hidden=x, n_steps=16, want_logits=True)
    outs = [b.route_step(hidden=x[t:t + 1], want_logits=True) for t in range(16)]
    zb = torch.cat([o[2] for o in outs])
    assert torch.allclose(za, zb, rtol=0, atol=3e-6)
    same = torch.equal(sa, torch.cat([o[0] for o in outs]))
    if not same:   # only a near tie may separate the two
        diff = (sa != torch.cat([o[0] for o in outs])).any(dim=-1)
        top = torch.sort(za, dim=-1, descending=True).values
        assert (top[..., :-1] - top[..., 1:]).min(dim=-1).values[diff].max().item() < H.NEAR_TIE
    else:
        assert a.cache_stats()[0] == b.cache_stats()[0]
        assert np.array_equal(a.cache_state()[0], b.cache_state()[0])
    a.close()
    b.close()


def test_automatic_choice_of_the_routing_kernels():
    """MCCE_ROUTE_AUTO: the fused kernel from three tokens per launch where the configuration has one, the two
    kernels otherwise."""
    for base, kw, n, want in ((synth.MIXTRAL, dict(L=32, S=64, d=1024), 8, mb.ROUTER_FUSED),
                              (synth.MIXTRAL, dict(L=32, S=64, d=1024), 1, mb.ROUTER_RESIDENT_TAIL),
                              (synth.QWEN, dict(L=24, S=64, d=512), 8, mb.ROUTER_FUSED),
                              (synth.OLMOE, dict(L=16, S=512, d=512), 8, mb.ROUTER_FUSED),
                              (synth.OLMOE, dict(L=16, S=512, d=512), 2, mb.ROUTER_RESIDENT_TAIL),
                              (synth.QWEN, dict(L=2, S=16, d=256, E=100), 8, mb.ROUTER_GEMM_TAIL),
                              (synth.TINY, dict(), 8, mb.ROUTER_FP32_PIPE)):
        wl = base.with_(**kw)
        eng = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT)
        eng.set_router(H.to_dev(wl.router()))
        assert eng.router_kernel_kind(n) == want, (wl.name, n)
        eng.close()
    # the fused kernel adds the parts of a logit in order of arrival: not in the deterministic or the checked mode
    wl = synth.QWEN.with_(L=24, S=64, d=512)
    for kw in (dict(deterministic=1), dict(checked=1)):
        eng = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT, route_impl=mb.ROUTE_FUSED, **kw)
        eng.set_router(H.to_dev(wl.router()))
        assert eng.router_kernel_kind(8) == mb.ROUTER_RESIDENT_TAIL, kw
        eng.close()
