"""The allocation-free routing entry point (`mcce_route_trace_static`).

Some users of this library cannot allocate device memory at the point where they need routing
decisions -- their framework's memory pool already owns the GPU, or they sit in a callback that must
not enter the allocator -- so this entry point keeps the cache state it needs in a fixed array inside
the library instead of a workspace.  Here it is called through the C ABI and compared with the ordinary
context-based entry point (`mcce_route_step` on a fresh context) on the same inputs, twice in a row:
the second call must not see anything the first one left in the shared array.  It is also compared with
the CPU oracle directly: bit for bit on given logits, in follow mode from hidden states.

This file sorts last on purpose, so that a run that stops at the first failure has run all other tests.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2412_00099_b200 import synth

pytestmark = pytest.mark.gpu


def _logits(seed, T, L, S, E):
    n = synth.normal(seed, synth.T_LOGITS, 0, 0, T * L * S * E).reshape(T, L, S, E)
    z = np.empty_like(n)
    h = n[0]
    for t in range(T):
        h = n[t] if t == 0 else np.float32(0.8) * h + np.float32(0.6) * n[t]
        z[t] = np.float32(1.5) * h
    return z


@pytest.mark.parametrize("L,S,E,K,J,Ccap,lam", [(3, 21, 60, 4, 2, 30, 0.5), (2, 9, 130, 7, 1, 5, 1.0)])
def test_static_routing_matches_context_routing_twice(L, S, E, K, J, Ccap, lam):
    from paper_2412_00099_b200 import binding as mb
    T = 40
    traces = [torch.from_numpy(_logits(100 + i, T, L, S, E)).cuda() for i in range(2)]
    for z in traces:                      # two calls in a row on different inputs, then compare each
        sel, w, totals = mb.route_trace_static(L=L, E=E, K=K, J=J, C_cap=Ccap, S=S, lam=lam, logits=z)
        eng = mb.Engine(L=L, E=E, K=K, J=J, n_shared=0, d=64, I=64, C_cap=Ccap, S=S, lam=lam, dtype=mb.F32)
        rsel, rw = eng.route_step(logits=z, n_steps=T)
        rtot, _ = eng.cache_stats()
        assert torch.equal(sel, rsel)                      # expert indices: bit for bit
        assert torch.allclose(w, rw, rtol=1e-5, atol=1e-7)  # weights: the routing tests' tolerance
        assert tuple(totals) == tuple(rtot)
        eng.close()
        # and against the oracle on the same logits: indices and Eq. 4 counters bit for bit
        from oracle import oracle as orc
        o = orc.Oracle(orc.OracleConfig(L, E, K, J, 0, 8, 8, Ccap, S, lam, 0, 1, 0), threads=4)
        zh, sel_h, w_h = z.cpu().numpy(), sel.cpu().numpy(), w.cpu().numpy()
        for t in range(T):
            osel, ow = o.route(zh[t])
            assert np.array_equal(sel_h[t], osel), "token %d" % t
            assert np.allclose(w_h[t], ow, rtol=1e-5, atol=1e-7)
        assert tuple(totals) == tuple(o.stats()[0].tolist())


def test_static_routing_from_hidden_states_and_without_totals():
    """From bf16 hidden states this entry point forms the logits on the fp32 pipe, a context on the tensor cores:
    the two may differ in the last bits, so selections are compared with the oracle in follow mode (its own fp64
    logits; a difference needs a deciding gap below 1e-4) and with the context wherever the step is no near tie."""
    from oracle import oracle as orc
    from paper_2412_00099_b200 import binding as mb
    import helpers as H
    wl = synth.QWEN.with_(L=2, S=12, d=256)
    T = 6
    Wr_h = wl.router()
    Wr = torch.from_numpy(Wr_h).cuda()
    xs = np.stack(list(wl.hidden_trace(T)))
    x = torch.from_numpy(xs.view(np.int16)).cuda().view(torch.bfloat16)
    for _ in range(2):
        sel, w = mb.route_trace_static(L=wl.L, E=wl.E, K=wl.K, J=wl.J, C_cap=wl.C, S=wl.S, lam=wl.lam, hidden=x,
                                       Wr=Wr, want_totals=False)
        eng = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT)
        eng.set_router(Wr)
        rsel, rw = eng.route_step(hidden=x, n_steps=T)
        eng.close()
        o = H.oracle_for(wl)
        sel_h, rsel_h = sel.cpu().numpy(), rsel.cpu().numpy()
        diverged = np.zeros((wl.L, wl.S), bool)          # after a near-tie difference the cache states differ
        for t in range(T):
            osel, _, margin, _ = o.route(o.logits(Wr_h, xs[t]), want_margin=True)
            for got in (sel_h[t], rsel_h[t]):
                differs = np.any(got != osel, axis=-1) & ~diverged
                assert (margin[differs] < H.NEAR_TIE).all(), "unexplained routing difference at token %d" % t
                diverged |= differs
        assert diverged.sum() <= 2
        ok = ~diverged
        assert np.array_equal(sel_h[:, ok], rsel_h[:, ok])
        assert torch.allclose(w[:, torch.from_numpy(ok).cuda()], rw[:, torch.from_numpy(ok).cuda()], rtol=1e-5, atol=1e-6)


def test_static_routing_rejects_unaligned_logits():
    from paper_2412_00099_b200 import binding as mb
    L, S, E, K = 1, 4, 8, 2
    buf = torch.zeros(1 + 3 * L * S * E, device="cuda")
    with pytest.raises(mb.McceError, match="invalid argument"):
        mb.route_trace_static(L=L, E=E, K=K, J=1, C_cap=4, S=S, lam=0.5, logits=buf[1:].view(3, L, S, E))


def test_static_routing_refuses_what_does_not_fit():
    from paper_2412_00099_b200 import binding as mb
    lib = mb.load()
    assert lib.mcce_route_trace_static_limit() == 4 << 20
    L, S, E, K = 64, 1024, 256, 4           # 64 MiB of cache state: far beyond the fixed array
    cfg = mb.Config(L, E, K, 1, 0, 8, 8, 16, S, 0.5, 0, 1, 0, 0, 0, 0)
    z = torch.zeros(8, device="cuda")       # never touched: the call must fail before any launch
    sel = torch.zeros(8, dtype=torch.int32, device="cuda")
    w = torch.zeros(8, device="cuda")
    rc = lib.mcce_route_trace_static(C.byref(cfg), 1, None, None, C.c_void_p(z.data_ptr()), None,
                                     C.c_void_p(sel.data_ptr()), C.c_void_p(w.data_ptr()), None, None)
    assert rc == -6 and b"fixed 4 MiB array" in lib.mcce_strerror(rc)
    with pytest.raises(mb.McceError):
        mb.route_trace_static(L=L, E=E, K=K, J=1, C_cap=16, S=S, lam=0.5,
                              logits=torch.zeros((1, 1, 1, 1), device="cuda"))
