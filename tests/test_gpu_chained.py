"""Sequential-layer decode mode (layers chained through a residual stream).

What can be stated exactly: the chained entry point equals the composition of single-layer steps -- the same
kernels launched layer by layer through the public per-layer calls -- bit for bit wherever the combine is
deterministic (the fp32-pipe expert path, and the tensor-core path of a context in deterministic mode); and for
fp32 workloads it follows an independent oracle chain, layer after layer.  With bf16 states the input of layer
l+1 is a rounding of a sum whose last bits differ between the two sides: there the oracle checks every layer
step from the library's own input of that layer, and a free-running oracle chain is followed with the measured
logit difference between the two chains added to the near-tie allowance."""
import numpy as np
import pytest
import torch

from paper_2412_00099_b200 import synth

pytestmark = pytest.mark.gpu


def build(wl, ffn_impl, **kw):
    from paper_2412_00099_b200 import binding as mb
    import helpers as H
    Wr, W = wl.router(), H.weights_for(wl)
    full = mb.engine_for(wl, ffn_impl=ffn_impl, **kw)
    full.set_router(H.to_dev(Wr))
    Wd = {k: (None if v is None else H.to_dev(v)) for k, v in W.items()}
    full.set_experts(**Wd)
    singles = []
    for l in range(wl.L):
        e = mb.engine_for(wl.with_(L=1), ffn_impl=ffn_impl, **kw)
        e.set_router(H.to_dev(Wr[l:l + 1]))
        e.set_experts(**{k: (None if v is None else v[l:l + 1].contiguous()) for k, v in Wd.items()})
        singles.append(e)
    return full, singles, Wr, W


def first_inputs(wl, T):
    import helpers as H
    return [H.to_dev(x)[0] for x in wl.with_(L=1).hidden_trace(T)]          # [S,d] per token


@pytest.mark.parametrize("wl", [synth.TINY.with_(L=3, S=6), synth.QWEN.with_(L=3, S=20, E=12, K=4, C=6, d=256, I=256,
                                                                          n_shared=1)])
def test_chained_equals_layer_by_layer_composition(wl):
    from paper_2412_00099_b200 import binding as mb
    full, singles, _, _ = build(wl, mb.FFN_SIMT)
    for x0 in first_inputs(wl, 6):
        x_c, sel_c = full.decode_step_chained(x0, want_sel=True)
        x = x0
        for l, e in enumerate(singles):
            sel, w = e.route_step(hidden=x[None, None])
            y = e.moe_forward(x[None], sel[0], w[0])[0]
            assert torch.equal(sel[0, 0], sel_c[l])
            x = (x.float() + y).to(x.dtype)
        assert torch.equal(x, x_c)
    tot = full.cache_stats()[0]
    assert tot[2] == sum(e.cache_stats()[0][2] for e in singles) and tot[0] == 6 * wl.L * wl.S


def test_chained_tensor_path_tracks_the_composition():
    from paper_2412_00099_b200 import binding as mb
    wl = synth.QWEN.with_(L=4, S=40, E=16, K=4, C=8, d=256, I=384, n_shared=1)
    full, singles, _, _ = build(wl, mb.FFN_TENSOR)
    agree, total = 0, 0
    for x0 in first_inputs(wl, 4):
        x_c, sel_c = full.decode_step_chained(x0, want_sel=True)
        x = x0
        for l, e in enumerate(singles):
            sel, w = e.route_step(hidden=x[None, None])
            y = e.moe_forward(x[None], sel[0], w[0])[0]
            if l == 0:
                assert torch.equal(sel[0, 0], sel_c[0])                       # same input, same kernels
            agree += int((sel[0, 0] == sel_c[l]).all(dim=-1).sum())
            total += wl.S
            x = (x.float() + y).to(x.dtype)
        close = torch.isclose(x.float(), x_c.float(), rtol=2e-2, atol=2e-2).float().mean().item()
        assert close > 0.995 and torch.isfinite(x_c.float()).all()
    assert agree >= 0.97 * total          # atomically summed outputs: the last bit of a state may differ
    print("chained tensor path: %d of %d (layer, stream) selections identical to the composition" % (agree, total))


def test_chained_tensor_path_equals_the_composition_in_deterministic_mode():
    """With the slot-order combine the tensor-core path repeats bit for bit, so the chained call and the layer-by-
    layer composition agree exactly: residual stream, selections of every layer, counters."""
    from paper_2412_00099_b200 import binding as mb
    wl = synth.QWEN.with_(L=4, S=40, E=16, K=4, C=8, d=256, I=384, n_shared=1)
    full, singles, _, _ = build(wl, mb.FFN_TENSOR, deterministic=True)
    assert full.uses_tensor_path()
    for x0 in first_inputs(wl, 4):
        x_c, sel_c = full.decode_step_chained(x0, want_sel=True)
        x = x0
        for l, e in enumerate(singles):
            sel, w = e.route_step(hidden=x[None, None])
            y = e.moe_forward(x[None], sel[0], w[0])[0]
            assert torch.equal(sel[0, 0], sel_c[l])
            x = (x.float() + y).to(x.dtype)
        assert torch.equal(x, x_c)
    assert full.cache_stats()[0][2] == sum(e.cache_stats()[0][2] for e in singles)


def test_chained_bf16_against_the_oracle_layer_by_layer_and_as_a_chain():
    """bf16 states on the tensor-core paths (deterministic combine), L = 4.
    (1) Layer by layer: the oracle is given the library's own input x_l of every layer (obtained from the
        single-layer composition, which the test above shows to be bit-identical to the chained call): its logits
        must be within the logit tolerance, its selection equal except behind a near tie (< 1e-4; it then adopts
        the library's choice), its FFN output within the FFN tolerance, and x_{l+1} = bf16(x_l + y_l) within one
        bf16 rounding step of the library's.
    (2) Free-running: a second oracle chain feeds its own bf16-rounded x + y forward.  Its logits differ from
        chain (1)'s by a measured amount dz (the states differ by rounding flips), so a selection difference
        needs a deciding gap below 1e-4 + 2 dz; streams that have diverged are counted and left out; for the
        others the final residual stream agrees within the accumulated FFN tolerance."""
    from paper_2412_00099_b200 import binding as mb
    import helpers as H
    wl = synth.QWEN.with_(L=4, S=40, E=16, K=4, C=8, d=256, I=384, n_shared=1)
    full, singles, Wr, W = build(wl, mb.FFN_TENSOR, deterministic=True)
    wl1 = wl.with_(L=1)
    forced = [H.oracle_for(wl1) for _ in range(wl.L)]        # (1): fed the library's x_l
    free = [H.oracle_for(wl1) for _ in range(wl.L)]          # (2): fed its own chain
    Wl = [{k: (None if v is None else np.ascontiguousarray(v[l:l + 1])) for k, v in W.items()} for l in range(wl.L)]
    names = ("Wg", "Wu", "Wd", "shWg", "shWu", "shWd")
    f32 = synth.bf16_bits_to_f32

    def bits_of(t):
        return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)

    diverged = np.zeros(wl.S, bool)
    near_forced = 0
    for x0 in first_inputs(wl, 6):
        x_c, sel_c = full.decode_step_chained(x0, want_sel=True)
        sel_c = sel_c.cpu().numpy()
        x_lib = x0                                           # library's residual stream, layer by layer
        x_free = bits_of(x0)
        for l in range(wl.L):
            xb = bits_of(x_lib)
            sel, w, zg = singles[l].route_step(hidden=x_lib[None, None], want_logits=True)
            y = singles[l].moe_forward(x_lib[None], sel[0], w[0])[0]
            assert torch.equal(sel[0, 0], torch.from_numpy(sel_c[l]).cuda())
            # ---- (1) the oracle on the library's input of this layer ----
            o = forced[l]
            z_own = o.logits(Wr[l:l + 1], xb[None])
            zg_h = zg[0].cpu().numpy()
            assert (np.abs(zg_h - z_own) <= H.LOGIT_RTOL * np.maximum(1.0, np.abs(z_own))).all()
            snap = o.snapshot()
            sel_own, _, margin, _ = o.route(z_own, want_margin=True)
            o.restore(snap)
            osel, ow = o.route(zg_h)
            assert np.array_equal(osel[0], sel_c[l])
            differs = np.any(sel_own[0] != osel[0], axis=-1)
            assert (margin[0][differs] < H.NEAR_TIE).all()
            near_forced += int(differs.sum())
            y_ref = o.ffn(xb[None], osel, ow, *[Wl[l][k] for k in names])[0]
            H.ffn_close(y.cpu().numpy(), y_ref)
            x_next_ref = f32(synth.to_bf16_bits(f32(xb) + y_ref))
            x_next = (x_lib.float() + y).to(x_lib.dtype)
            step = np.maximum(np.abs(x_next_ref), 1e-3) * 2.0 ** -7          # one bf16 step at that magnitude
            assert (np.abs(x_next.float().cpu().numpy() - x_next_ref) <= H.FFN_ATOL + H.FFN_RTOL * np.abs(y_ref) + step).all()
            # ---- (2) the free-running oracle chain ----
            of = free[l]
            z_free = of.logits(Wr[l:l + 1], x_free[None])
            dz = np.abs(z_free[0] - z_own[0]).max(axis=-1)                     # per stream
            sel_f, w_f, margin_f, _ = of.route(z_free, want_margin=True)
            same = (sel_f[0] == sel_c[l]).all(axis=-1)
            assert (same | diverged | (margin_f[0] < H.NEAR_TIE + 2 * dz)).all(), "unexplained divergence, layer %d" % l
            diverged |= ~same
            y_free = of.ffn(x_free[None], sel_f, w_f, *[Wl[l][k] for k in names])[0]
            x_free = synth.to_bf16_bits(f32(x_free) + y_free)
            x_lib = x_next
        assert torch.equal(x_lib, x_c)                        # composition == chained call
        ok = ~diverged
        got, ref = x_c.float().cpu().numpy()[ok], f32(x_free)[ok]
        # every layer adds an FFN output within tolerance and a bf16 rounding of the running sum
        bound = wl.L * (H.FFN_ATOL + 2.0 ** -7 * np.maximum(np.abs(ref), 1.0)) + H.FFN_RTOL * np.abs(ref)
        assert (np.abs(got - ref) <= bound).all()
    assert diverged.sum() <= wl.S // 8
    print("bf16 chain: %d near ties against the layer-wise oracle, %d of %d streams diverged from the free chain"
          % (near_forced, int(diverged.sum()), wl.S))


def test_chained_follows_an_oracle_chain_fp32():
    """fp32 states: the oracle's own chain (per-layer oracles, x + y in fp32) against the library's."""
    from oracle import oracle as orc
    from paper_2412_00099_b200 import binding as mb
    import helpers as H
    wl = synth.TINY.with_(L=3, S=5)
    full, _, Wr, W = build(wl, mb.FFN_SIMT)
    oracles = [H.oracle_for(wl.with_(L=1)) for _ in range(wl.L)]
    diverged = np.zeros(wl.S, bool)
    for x0 in first_inputs(wl, 12):
        x_c, sel_c = full.decode_step_chained(x0, want_sel=True)
        sel_c = sel_c.cpu().numpy()
        x = x0.cpu().numpy()
        for l, o in enumerate(oracles):
            z = o.logits(Wr[l:l + 1], x[None])
            sel, w, margin, _ = o.route(z, want_margin=True)
            same = (sel[0] == sel_c[l]).all(axis=-1)
            assert (same | diverged | (margin[0] < H.NEAR_TIE)).all()      # a difference needs a near tie
            diverged |= ~same
            y = o.ffn(x[None], sel, w, *[None if W[k] is None else W[k][l:l + 1] for k in
                                         ("Wg", "Wu", "Wd", "shWg", "shWu", "shWd")])
            x = (x + y[0]).astype(np.float32)
        ok = ~diverged
        assert np.allclose(x_c.cpu().numpy()[ok], x[ok], rtol=1e-4, atol=1e-5)
    assert diverged.sum() <= 1
