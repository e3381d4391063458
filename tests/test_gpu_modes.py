"""The deterministic and the checked mode of a context, and what the library does with inputs it cannot use:
an expert id outside [0, E) handed to mcce_moe_forward, non-finite logits, misaligned logit buffers.  Everything
goes through the C ABI; every input here is turned into an error code by a host-side check or by a range check
in the kernel that reads it."""
import numpy as np
import pytest
import torch

from paper_2412_00099_b200 import synth
from test_gpu_parity import ROUTE_CASES, TC_CASES, ar1_logits, run_forward_case

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2412_00099_b200 import binding as mb
    import helpers as H


def forward_setup(wl, **kw):
    W = H.weights_for(wl)
    eng = mb.engine_for(wl, **kw)
    eng.set_router(H.to_dev(wl.router()))
    eng.set_experts(**{k: (None if v is None else H.to_dev(v)) for k, v in W.items()})
    return eng, W


# ---- deterministic mode ------------------------------------------------------------------------------------
@pytest.mark.parametrize("base,kw", [
    (synth.QWEN, dict(L=2, S=72, E=20, K=4, C=10, d=512, I=640, n_shared=2)),
    (synth.OLMOE, dict(L=2, S=150, E=16, K=8, C=8, d=384, I=256)),
])
def test_deterministic_mode_repeats_bit_for_bit_and_matches_the_oracle(base, kw):
    """Slot-order combine on the tensor-core path: repeated runs give identical bits (the atomic combine need
    not), a second context gives the same bits, and the result is within the FFN tolerance of the oracle."""
    wl = base.with_(**kw)
    eng, W = forward_setup(wl, ffn_impl=mb.FFN_TENSOR, deterministic=True)
    eng2, _ = forward_setup(wl, ffn_impl=mb.FFN_TENSOR, deterministic=True)
    assert eng.uses_tensor_path()
    o = H.oracle_for(wl)
    for x in wl.hidden_trace(3):
        xd = H.to_dev(x)
        sel, w, zg = eng.route_step(hidden=xd[None], want_logits=True)
        eng2.route_step(hidden=xd[None])
        ys = [eng.moe_forward(xd, sel[0], w[0]).clone() for _ in range(4)] + [eng2.moe_forward(xd, sel[0], w[0])]
        for y in ys[1:]:
            assert torch.equal(ys[0], y)
        osel, ow = o.route(zg[0].cpu().numpy())
        y_ref = o.ffn(x, osel, ow, W["Wg"], W["Wu"], W["Wd"], W["shWg"], W["shWu"], W["shWd"])
        H.ffn_close(ys[0].cpu().numpy(), y_ref)


def test_deterministic_tensor_path_equals_slot_order_sum_of_the_atomic_path_terms():
    """The deterministic and the atomic combine add the same K + n_shared terms; only the order differs."""
    wl = synth.QWEN.with_(L=2, S=40, E=12, K=4, C=6, d=256, I=384, n_shared=1)
    det, _ = forward_setup(wl, ffn_impl=mb.FFN_TENSOR, deterministic=True)
    fast, _ = forward_setup(wl, ffn_impl=mb.FFN_TENSOR)
    x = H.to_dev(next(iter(wl.hidden_trace(1))))
    sel, w = det.route_step(hidden=x[None])
    a, b = det.moe_forward(x, sel[0], w[0]), fast.moe_forward(x, sel[0], w[0])
    assert torch.allclose(a, b, rtol=1e-5, atol=1e-6)


# ---- checked mode: the suite's valid inputs raise nothing ------------------------------------------------------
@pytest.mark.parametrize("E,K,J,C,lam,dm,renorm,quant", ROUTE_CASES[3:10])
def test_checked_mode_is_silent_on_valid_routing(E, K, J, C, lam, dm, renorm, quant):
    L, S, T = 2, 19, 24
    wl = synth.TINY.with_(L=L, E=E, K=K, J=J, C=C, S=S, lam=lam, d=64, I=64)
    fixed = np.linspace(2.0, 4.0, L).astype(np.float32) if dm else None
    eng = mb.engine_for(wl, delta_mode=dm, renorm=renorm, checked=True)
    if dm:
        eng.set_router(torch.zeros((L, E, 64), device="cuda"), H.to_dev(fixed))
    o = H.oracle_for(wl, delta_mode=dm, renorm=renorm, fixed_delta=fixed)
    H.check_route_exact(eng, o, ar1_logits(E * 131 + K, T, L, S, E, quant=quant), chunk=5, check_every=1)
    eng.close()


@pytest.mark.parametrize("base,kw", TC_CASES[:3])
def test_checked_mode_is_silent_on_valid_forward(base, kw, monkeypatch):
    """route (tensor-core logits) + group + experts with every check switched on; cache_stats must return OK."""
    real = mb.engine_for
    monkeypatch.setattr(mb, "engine_for", lambda wl, **k: real(wl, checked=True, **k))
    run_forward_case(base.with_(**kw), 3, mb.FFN_TENSOR)


def test_checked_mode_covers_the_batched_and_chained_paths():
    wl = synth.QWEN.with_(L=3, S=40, E=16, K=4, C=8, d=256, I=256, n_shared=1)
    eng, _ = forward_setup(wl, checked=True)
    xs = np.stack(list(wl.hidden_trace(8)))
    x = torch.from_numpy(xs.view(np.int16)).cuda().view(torch.bfloat16)
    eng.route_step(hidden=x, n_steps=8)                      # several tokens per launch
    eng.decode_step_chained(x[0, 0])                         # layer after layer
    eng.cache_stats()                                        # raises on any recorded violation


# ---- inputs the library cannot use ----------------------------------------------------------------------------
@pytest.mark.parametrize("ffn_impl,bad", [("tensor", -1), ("tensor", 12), ("simt", -1), ("simt", 1 << 30)])
def test_expert_id_out_of_range_is_skipped_and_reported(ffn_impl, bad):
    """A sel_idx entry outside [0, E) (padding, an uninitialised buffer): the pair contributes nothing, every other
    output is as if its weight were zero, and mcce_cache_stats reports MCCE_EINDEX until the next reset."""
    wl = synth.QWEN.with_(L=2, S=24, E=12, K=4, C=6, d=256, I=384, n_shared=1)
    impl = mb.FFN_TENSOR if ffn_impl == "tensor" else mb.FFN_SIMT
    eng, W = forward_setup(wl, ffn_impl=impl)
    x = next(iter(wl.hidden_trace(1)))
    xd = H.to_dev(x)
    sel, w = eng.route_step(hidden=xd[None])
    sel_bad = sel[0].clone()
    sel_bad[0, 3, 1] = bad
    sel_bad[1, 20, 0] = bad
    y = eng.moe_forward(xd, sel_bad, w[0]).cpu().numpy()
    with pytest.raises(mb.McceError, match="expert id outside"):
        eng.cache_stats()
    # the oracle on the valid selection with the two pairs' weights set to zero
    w_ref = w[0].cpu().numpy().copy()
    w_ref[0, 3, 1] = 0.0
    w_ref[1, 20, 0] = 0.0
    o = H.oracle_for(wl)
    y_ref = o.ffn(x, sel[0].cpu().numpy(), w_ref, W["Wg"], W["Wu"], W["Wd"], W["shWg"], W["shWu"], W["shWd"])
    H.ffn_close(y, y_ref)
    eng.reset()
    eng.cache_stats()                                        # the report is cleared by a reset
    y2 = eng.moe_forward(xd, sel[0], w[0]).cpu().numpy()      # and the context still works
    H.ffn_close(y2, o.ffn(x, sel[0].cpu().numpy(), w[0].cpu().numpy(), W["Wg"], W["Wu"], W["Wd"], W["shWg"],
                          W["shWu"], W["shWd"]))


def test_non_finite_logits_are_reported_in_checked_mode():
    wl = synth.TINY.with_(L=2, S=5, E=16, K=2, C=4)
    z = ar1_logits(3, 4, wl.L, wl.S, wl.E)
    z[2, 1, 3, 7] = np.nan
    z[3, 0, 0, 0] = np.inf
    quiet, loud = mb.engine_for(wl), mb.engine_for(wl, checked=True)
    for eng in (quiet, loud):
        sel, _ = eng.route_step(logits=H.to_dev(z), n_steps=4)
        assert int(sel.min()) >= 0 and int(sel.max()) < wl.E      # indices stay in range whatever the logits are
    quiet.cache_stats()
    with pytest.raises(mb.McceError, match="NaN or infinite"):
        loud.cache_stats()
    # fp32 hidden states: the route kernel forms the logits itself and checks them on the way
    eng = mb.engine_for(wl, checked=True)
    eng.set_router(H.to_dev(wl.router()))
    x = next(iter(wl.hidden_trace(1))).copy()
    x[1, 2, 5] = np.inf
    eng.route_step(hidden=H.to_dev(x)[None])
    with pytest.raises(mb.McceError, match="NaN or infinite"):
        eng.cache_stats()


def test_misaligned_logit_buffers_are_rejected():
    """Rows of logits are accessed four floats at a time when E is a multiple of 4: a buffer that is only
    4-byte aligned is refused on the host (a view one float into a tensor), nothing is launched."""
    wl = synth.TINY.with_(L=1, S=4, E=8, K=2, C=4)
    eng = mb.engine_for(wl)
    buf = torch.zeros(1 + wl.L * wl.S * wl.E, device="cuda")
    lib = mb.load()
    import ctypes as C
    sel = torch.zeros((1, wl.L, wl.S, wl.K), dtype=torch.int32, device="cuda")
    w = torch.zeros((1, wl.L, wl.S, wl.K), device="cuda")
    args = lambda zin, zout: (eng.ctx, 1, None, C.c_void_p(zin), C.c_void_p(sel.data_ptr()), C.c_void_p(w.data_ptr()),
                              C.c_void_p(zout) if zout else None, None)
    assert lib.mcce_route_step(*args(buf.data_ptr() + 4, 0)) == -1
    assert lib.mcce_route_step(*args(buf.data_ptr(), buf.data_ptr() + 4)) == -1
    assert lib.mcce_route_step(*args(buf.data_ptr(), 0)) == 0
    assert eng.cache_stats()[0][0] == wl.L * wl.S


def test_calibration_needs_routed_tokens():
    eng = mb.engine_for(synth.TINY)
    with pytest.raises(mb.McceError):
        eng.calibrated_delta()
