"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded
inputs.  Integer results (expert indices, cache states, counters, grouping) bit for bit; floating point
within the stated tolerances."""
import numpy as np
import pytest
import torch

from paper_2412_00099_b200 import synth

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2412_00099_b200 import binding as mb
    import helpers as H


def ar1_logits(seed, T, L, S, E, rho=0.8, scale=1.5, quant=None):
    """Synthetic router logits with temporal locality, drawn from the seeded generator."""
    n = synth.normal(seed, synth.T_LOGITS, 0, 0, T * L * S * E).reshape(T, L, S, E)
    z = np.empty_like(n)
    h = n[0]
    for t in range(T):
        h = n[t] if t == 0 else np.float32(rho) * h + np.float32(np.sqrt(1 - rho * rho)) * n[t]
        z[t] = np.float32(scale) * h
    if quant:
        z = (np.round(z / quant) * quant).astype(np.float32)   # exact ties, to exercise tie-breaking
    return z


# ---- generator -------------------------------------------------------------------------------------
def test_generator_matches_host_definition_bit_for_bit():
    words = mb.gen_philox_words(1000, seed=5, tensor_id=3, t=7, start_block=(1 << 32) - 500).cpu().numpy()
    assert np.array_equal(words.view(np.uint32), synth.uint32_stream(5, 3, 7, (1 << 32) - 500, 1000))
    for dtype in (torch.float32, torch.bfloat16):
        out = torch.empty(100_003, dtype=dtype, device="cuda")
        mb.gen_normal(out, seed=9, tensor_id=synth.T_WG, t=0, std=0.02, start=4096)
        ref = synth.scaled_normal(9, synth.T_WG, 0, 4096, 100_003, 0.02, dtype == torch.bfloat16)
        got = out.view(torch.int16).cpu().numpy().view(np.uint16) if dtype == torch.bfloat16 else out.cpu().numpy()
        assert np.array_equal(got.view(ref.dtype), ref)
    big = torch.empty(4_000_000, dtype=torch.float32, device="cuda")
    mb.gen_normal(big, seed=1, tensor_id=synth.T_NOISE, t=3)
    assert abs(big.mean().item()) < 2e-3 and abs(big.std().item() - 1) < 2e-3


@pytest.mark.parametrize("wl", [synth.TINY, synth.QWEN.with_(L=2, S=3, d=64)])
def test_hidden_trace_matches_host_definition(wl):
    state = torch.empty(wl.L * wl.S * wl.d, dtype=torch.float32, device="cuda")
    x = torch.empty((wl.L, wl.S, wl.d), dtype=torch.bfloat16 if wl.bf16 else torch.float32, device="cuda")
    for t, ref in enumerate(wl.hidden_trace(12)):
        mb.gen_hidden_step(state, x, wl.seed, t, wl.rho, wl.topic_offset)
        got = x.view(torch.int16).cpu().numpy().view(np.uint16) if wl.bf16 else x.cpu().numpy()
        assert np.array_equal(got, ref)


# ---- routing from identical logits: bit-exact ---------------------------------------------------------
ROUTE_CASES = [
    # E,  K, J, C,  lam, delta_mode, renorm, quant
    (8, 2, 1, 4, 0.5, 0, 1, None),
    (8, 2, 1, 4, 0.0, 0, 1, None),
    (8, 2, 1, 4, 1.0, 0, 0, 0.25),
    (60, 4, 2, 30, 0.5, 0, 1, None),
    (60, 4, 2, 15, 1.0, 1, 1, 0.125),
    (64, 8, 2, 32, 0.5, 0, 1, 0.25),
    (64, 6, 0, 24, 0.7, 0, 1, None),
    (64, 6, 6, 24, 0.7, 0, 1, None),       # J = K
    (33, 5, 1, 3, 0.9, 0, 1, None),        # C < K, E not a multiple of 32
    (16, 2, 1, 1, 0.6, 0, 1, None),        # cache of one
    (20, 3, 1, 20, 0.5, 0, 1, None),       # C = E
    (12, 3, 1, 50, 0.5, 0, 1, None),       # C > E
    (130, 7, 2, 40, 0.4, 0, 1, 0.5),       # five lanes-slots per lane, many ties
    (256, 16, 3, 100, 0.3, 0, 1, None),    # maximum sizes
    (1, 1, 0, 1, 0.5, 0, 1, None),         # degenerate: one expert
    (5, 5, 2, 2, 2.5, 0, 1, None),         # K = E, lambda > 1
]


@pytest.mark.parametrize("E,K,J,C,lam,dm,renorm,quant", ROUTE_CASES)
@pytest.mark.parametrize("chunk", [1, 7])
def test_route_from_logits_is_bit_exact(E, K, J, C, lam, dm, renorm, quant, chunk):
    L, S, T = 3, 19, 48          # S not a multiple of the CTA's stream block
    wl = synth.TINY.with_(L=L, E=E, K=K, J=J, C=C, S=S, lam=lam, d=64, I=64)
    fixed = np.linspace(2.0, 4.0, L).astype(np.float32) if dm else None
    eng = mb.engine_for(wl, delta_mode=dm, renorm=renorm, track_lifetime=True)
    if dm:
        eng.set_router(torch.zeros((L, E, 64), device="cuda"), H.to_dev(fixed))
    o = H.oracle_for(wl, delta_mode=dm, renorm=renorm, fixed_delta=fixed)
    z = ar1_logits(E * 131 + K, T, L, S, E, quant=quant)
    H.check_route_exact(eng, o, z, chunk=chunk, check_every=3)
    eng.close()


RERANK_CASES = [
    # mode, E, K, J, C, M, p
    (1, 8, 2, 1, 4, 0, 0.0),      # Max-Rank with M = 0: nothing promoted
    (1, 8, 2, 1, 4, 4, 0.0),
    (1, 60, 4, 2, 30, 12, 0.0),
    (1, 64, 8, 0, 16, 64, 0.0),   # M = E, J = 0: every cached expert first
    (1, 130, 7, 2, 40, 33, 0.0),
    (2, 8, 2, 1, 4, 0, 0.6),      # Cumsum-Threshold
    (2, 60, 4, 2, 30, 0, 0.5),
    (2, 64, 6, 2, 24, 0, 0.9),
    (2, 33, 5, 1, 3, 0, 1.5),     # p > 1: the whole ranking
    (2, 16, 2, 1, 8, 0, 0.0),     # p = 0: plain top-K
]


@pytest.mark.parametrize("mode,E,K,J,C,M,p", RERANK_CASES)
def test_baseline_rerankers_match_the_oracle(mode, E, K, J, C, M, p):
    """Algorithms 1 and 2 as routing modes, identical logits on both sides.  Indices, cache states and
    counters bit for bit; for the cumulative threshold a step whose partial sum lies within 1e-6 of p
    may legitimately resolve either way (the probabilities are floating point), which ends the comparison."""
    L, S, T = 2, 11, 40
    wl = synth.TINY.with_(L=L, E=E, K=K, J=J, C=C, S=S, d=64, I=64)
    eng = mb.engine_for(wl, rerank_mode=mode, max_rank=M, cum_threshold=p, track_lifetime=True)
    o = H.oracle_for(wl, rerank_mode=mode, max_rank=M, cum_threshold=p)
    z = ar1_logits(E * 7 + mode, T, L, S, E, quant=0.25 if mode == 1 else None)
    zd = H.to_dev(z)
    for t in range(T):
        sel, w = eng.route_step(logits=zd[t:t + 1])
        osel, ow, margin, _ = o.route(z[t], want_margin=True)
        same = np.array_equal(sel[0].cpu().numpy(), osel)
        if not same and mode == 2:
            bad = np.any(sel[0].cpu().numpy() != osel, axis=-1)
            assert (margin[bad] < 1e-6).all(), "unexplained difference in the cumulative threshold"
            print("near-threshold step at token %d: comparison ends" % t)
            return
        assert same
        assert np.allclose(w[0].cpu().numpy(), ow, rtol=1e-5, atol=1e-7)
    H.assert_state_equal(eng, o)


def test_cumsum_threshold_reached_exactly_on_gpu():
    """Four equal logits: probabilities of exactly 1/4; p = 1/2 stops after two ranks (see the oracle pin)."""
    for p, want in ((0.5, 0), (0.51, 2)):
        eng = mb.Engine(L=1, E=4, K=1, J=0, n_shared=0, d=64, I=64, C_cap=2, S=1, lam=0.5, dtype=mb.F32,
                        rerank_mode=mb.RERANK_CUMSUM, cum_threshold=p)
        eng.reset(init_order=np.array([[[2, -1]]], np.int32))
        sel, _ = eng.route_step(logits=torch.zeros((1, 1, 1, 4), device="cuda"))
        assert sel.flatten().tolist() == [want]


def test_miss_trace_matches_the_oracle():
    """Per-token miss bits, through both routing front ends (given logits; hidden states via the GEMM)."""
    wl = synth.QWEN.with_(L=2, S=19, d=128, C=9)
    T = 20
    eng, o = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT), H.oracle_for(wl)
    trace = eng.record_misses(T - 4)                         # shorter than the run: the tail is not recorded
    z = ar1_logits(77, T, wl.L, wl.S, wl.E)
    eng.route_step(logits=H.to_dev(z[:12]), n_steps=12)
    for t in range(12, T):
        eng.route_step(logits=H.to_dev(z[t:t + 1]))
    want = np.zeros((T, wl.L, wl.S), np.uint32)
    for t in range(T):
        o.route(z[t])
        want[t] = o.last_miss_mask
    got = trace.cpu().numpy().view(np.uint32)
    assert np.array_equal(got, want[:T - 4])
    assert sum(bin(int(v)).count("1") for v in want.ravel()) == eng.cache_stats()[0][2]
    # from hidden states (tensor-core logits): follow the library's logits, compare the bits
    eng2, o2 = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT), H.oracle_for(wl)
    eng2.set_router(H.to_dev(wl.router()))
    tr2 = eng2.record_misses(6)
    for t, x in enumerate(wl.hidden_trace(6)):
        _, _, zg = eng2.route_step(hidden=H.to_dev(x)[None], want_logits=True)
        o2.route(zg[0].cpu().numpy())
        assert np.array_equal(tr2[t].cpu().numpy().view(np.uint32), o2.last_miss_mask)


def test_calibrated_delta_feeds_fixed_mode():
    """Logit range estimated on a warm-up trace (running mode), then used as per-layer constants."""
    wl = synth.QWEN.with_(L=3, S=16, d=128, lam=0.5)
    Wr = wl.router()
    xs = list(wl.hidden_trace(24))
    warm, o_warm = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT), H.oracle_for(wl)
    warm.set_router(H.to_dev(Wr))
    for x in xs[:12]:
        sel, w, z = warm.route_step(hidden=H.to_dev(x)[None], want_logits=True)
        o_warm.route(z[0].cpu().numpy())
    delta = warm.calibrated_delta()
    ref = (o_warm.sum_range.astype(np.float64).mean(axis=1) / o_warm.count[0, 0]).astype(np.float32)
    assert np.array_equal(delta, ref) and (delta > 0).all()
    eng = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT, delta_mode=mb.DELTA_FIXED)
    eng.set_router(H.to_dev(Wr), H.to_dev(delta))
    o = H.oracle_for(wl, delta_mode=1, fixed_delta=delta)
    H.check_route_follow(eng, o, Wr, iter(xs[12:]), wl.bf16)


def test_route_initial_state_and_resume():
    wl = synth.TINY.with_(L=2, E=24, K=3, J=1, C=7, S=5, lam=0.5)
    rng = np.random.default_rng(0)
    init = np.full((wl.L, wl.S, wl.C), -1, np.int32)
    for l in range(wl.L):
        for s in range(wl.S):
            n = int(rng.integers(0, wl.C + 1))
            init[l, s, :n] = rng.choice(wl.E, n, replace=False)
    z = ar1_logits(3, 40, wl.L, wl.S, wl.E)
    eng, o = mb.engine_for(wl), H.oracle_for(wl)
    eng.reset(init_order=init)
    o.reset(init_order=init)
    H.check_route_exact(eng, o, z[:20], chunk=4, check_every=1)
    # export, rebuild a second engine from the exported state, continue: must stay identical
    order, ever, dsum, cnt = eng.cache_state()
    eng2 = mb.engine_for(wl)
    eng2.reset(init_order=order, delta_sum=dsum, delta_count=cnt)
    s1, w1 = eng.route_step(logits=H.to_dev(z[20:]), n_steps=20)
    s2, w2 = eng2.route_step(logits=H.to_dev(z[20:]), n_steps=20)
    assert torch.equal(s1, s2) and torch.equal(w1, w2)
    assert np.array_equal(eng.cache_state()[0], eng2.cache_state()[0])
    # and the first engine still tracks the oracle (the second lost only the 'ever' bits / counters)
    for i in range(20):
        osel, _ = o.route(z[20 + i])
        assert np.array_equal(s1[i].cpu().numpy(), osel)
    H.assert_state_equal(eng, o)


def test_full_cache_only_cold_misses_on_gpu():
    wl = synth.TINY.with_(L=2, E=16, K=4, J=1, C=16, S=9, lam=0.5)
    eng = mb.engine_for(wl)
    z = ar1_logits(11, 64, wl.L, wl.S, wl.E)
    sel, _ = eng.route_step(logits=H.to_dev(z), n_steps=64)
    total, _ = eng.cache_stats()
    sel = sel.cpu().numpy()
    distinct = sum(len(np.unique(sel[:, l, s])) for l in range(wl.L) for s in range(wl.S))
    assert total[2] == total[3] == distinct and total[1] == 64 * wl.L * wl.S * wl.K


# ---- routing from hidden states: follow mode -----------------------------------------------------------
@pytest.mark.parametrize("lam", [0.0, 0.5, 1.0])
def test_tiny_workload_end_to_end_routing(lam):
    wl = synth.TINY.with_(lam=lam)
    Wr = wl.router()
    eng, o = mb.engine_for(wl), H.oracle_for(wl)
    eng.set_router(H.to_dev(Wr))
    steps, near, dz = H.check_route_follow(eng, o, Wr, wl.hidden_trace(wl.T), wl.bf16)
    assert steps == wl.T * wl.S * wl.L
    print("tiny lam=%.1f: %d steps, %d near ties, max logit err %.2e" % (lam, steps, near, dz))


@pytest.mark.parametrize("base,kw", [
    (synth.QWEN, dict(L=2, S=21, T=24)),
    (synth.OLMOE, dict(L=2, S=16, T=16)),
    (synth.DEEPSEEK, dict(L=1, S=10, T=16)),
    (synth.MIXTRAL, dict(L=2, S=9, T=16)),
    (synth.QWEN, dict(L=1, S=8, T=8, d=8200)),        # hidden size beyond one shared-memory chunk
])
def test_model_shaped_routing_from_hidden_states(base, kw):
    kw = dict(kw)
    T = kw.pop("T")
    wl = base.with_(**kw)
    Wr = wl.router()
    eng, o = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT), H.oracle_for(wl)
    eng.set_router(H.to_dev(Wr))
    steps, near, dz = H.check_route_follow(eng, o, Wr, wl.hidden_trace(T), wl.bf16)
    print("%s: %d steps, %d near ties, max logit err %.2e" % (wl.name, steps, near, dz))


def test_many_tokens_per_launch_from_hidden_states():
    """n_steps beyond one logits-buffer chunk in a single call against one call per token: the cache
    recurrence must be the same however the tokens are batched into launches."""
    wl = synth.QWEN.with_(L=2, S=40, d=512)
    Wr = H.to_dev(wl.router())
    xs = np.stack(list(wl.hidden_trace(21)))
    x = torch.from_numpy(xs.view(np.int16)).cuda().view(torch.bfloat16)
    a, b = mb.engine_for(wl, ffn_impl=mb.FFN_SIMT), mb.engine_for(wl, ffn_impl=mb.FFN_SIMT)
    a.set_router(Wr)
    b.set_router(Wr)
    sa, wa, za = a.route_step(hidden=x, n_steps=21, want_logits=True)
    outs = [b.route_step(hidden=x[t:t + 1], want_logits=True) for t in range(21)]
    zb = torch.cat([o[2] for o in outs])
    assert torch.allclose(za, zb, rtol=0, atol=2e-6)       # the reduction may be split differently
    assert torch.equal(sa, torch.cat([o[0] for o in outs]))
    assert a.cache_stats()[0] == b.cache_stats()[0]
    assert np.array_equal(a.cache_state()[0], b.cache_state()[0])


# ---- grouping -------------------------------------------------------------------------------------------
@pytest.mark.parametrize("L,S,E,K", [(1, 4, 8, 2), (3, 256, 60, 4), (2, 512, 64, 8), (2, 37, 200, 5), (1, 1, 1, 1)])
def test_grouping_is_the_stable_counting_sort(L, S, E, K):
    wl = synth.TINY.with_(L=L, S=S, E=E, K=K, J=0, C=max(1, E // 2), d=64, I=64)
    eng = mb.engine_for(wl)
    W = {k: (None if v is None else H.to_dev(v)) for k, v in H.weights_for(wl).items()}
    eng.set_experts(**W)
    rng = np.random.default_rng(L * 1000 + S)
    sel = np.stack([[rng.choice(E, K, replace=False) for _ in range(S)] for _ in range(L)]).astype(np.int32)
    if E > 4:
        sel[0, :, 0] = 1            # one very full bucket ...
        sel[0][sel[0] == 3] = 0     # ... and one empty
    x = torch.zeros((L, S, 64), device="cuda")
    eng.moe_forward(x, H.to_dev(sel), torch.ones((L, S, K), device="cuda"))
    offsets, perm = eng.grouping()
    for l in range(L):
        flat = sel[l].reshape(-1)
        assert np.array_equal(offsets[l], np.concatenate([[0], np.cumsum(np.bincount(flat, minlength=E))]))
        assert np.array_equal(perm[l], np.argsort(flat, kind="stable"))


# ---- expert FFN ---------------------------------------------------------------------------------------
def run_forward_case(wl, T, ffn_impl):
    Wr = wl.router()
    W = H.weights_for(wl)
    eng, o = mb.engine_for(wl, ffn_impl=ffn_impl), H.oracle_for(wl)
    eng.set_router(H.to_dev(Wr))
    eng.set_experts(**{k: (None if v is None else H.to_dev(v)) for k, v in W.items()})
    worst = (0.0, 0.0)
    for x in wl.hidden_trace(T):
        xd = H.to_dev(x)
        sel, w, zg = eng.route_step(hidden=xd[None], want_logits=True)
        y = eng.moe_forward(xd, sel[0], w[0]).cpu().numpy()
        osel, ow = o.route(zg[0].cpu().numpy())
        assert np.array_equal(sel[0].cpu().numpy(), osel)
        # the oracle's FFN runs on the oracle's own selection and weights
        y_ref = o.ffn(x, osel, ow, W["Wg"], W["Wu"], W["Wd"], W["shWg"], W["shWu"], W["shWd"])
        e = H.ffn_close(y, y_ref)
        worst = (max(worst[0], e[0]), max(worst[1], e[1]))
    assert eng.cache_stats()[0] == tuple(o.stats()[0].tolist())
    return worst


def test_tiny_workload_forward_fp32():
    worst = run_forward_case(synth.TINY.with_(T=32), 32, mb.FFN_SIMT)
    print("tiny fp32 forward: max abs err %.2e" % worst[0])


@pytest.mark.parametrize("base,kw", [
    (synth.QWEN, dict(L=2, S=24, E=12, K=4, C=6, d=256, I=384, n_shared=2)),
    (synth.MIXTRAL, dict(L=1, S=5, E=8, K=2, C=4, d=512, I=1032)),
    (synth.OLMOE, dict(L=1, S=40, E=16, K=8, C=8, d=128, I=72)),
])
def test_model_shaped_forward_simt_bf16(base, kw):
    worst = run_forward_case(base.with_(**kw), 3, mb.FFN_SIMT)
    print("%s simt forward: max abs err %.2e" % (base.name, worst[0]))


TC_CASES = [
    (synth.QWEN, dict(L=2, S=24, E=12, K=4, C=6, d=256, I=384, n_shared=2)),      # small groups, empty groups
    (synth.QWEN, dict(L=1, S=300, E=4, K=2, C=2, d=128, I=128, n_shared=1)),      # > 128 tokens per expert: chunks
    (synth.OLMOE, dict(L=2, S=77, E=16, K=8, C=8, d=384, I=256)),                 # ragged token counts
    (synth.MIXTRAL, dict(L=1, S=19, E=8, K=2, C=4, d=1024, I=2048)),              # long reductions, many stages
    (synth.DEEPSEEK, dict(L=3, S=33, E=64, K=6, C=24, d=256, I=128, n_shared=2)),  # many experts, most nearly empty
]


@pytest.mark.parametrize("base,kw", TC_CASES)
def test_model_shaped_forward_tensor_core_bf16(base, kw):
    wl = base.with_(**kw)
    eng = mb.engine_for(wl, ffn_impl=mb.FFN_TENSOR)
    assert eng.uses_tensor_path()
    eng.close()
    worst = run_forward_case(wl, 3, mb.FFN_TENSOR)
    print("%s tensor-core forward: max abs err %.2e" % (base.name, worst[0]))


@pytest.mark.parametrize("skew", [False, True])
def test_tensor_core_path_agrees_with_simt_path(skew):
    """Same inputs through both expert-FFN implementations of the library (a consistency check on top of
    the oracle comparisons above).  With skew every stream selects expert 0 as well, so that one group is
    several times larger than the token tile the launch was sized for and takes several passes."""
    wl = synth.QWEN.with_(L=2, S=72, E=20, K=4, C=10, d=512, I=640, n_shared=1)
    W = {k: (None if v is None else H.to_dev(v)) for k, v in H.weights_for(wl).items()}
    x = H.to_dev(next(iter(wl.hidden_trace(1))))
    rng = np.random.default_rng(1)
    sel = np.stack([[rng.choice(np.arange(1, wl.E), wl.K, replace=False) for _ in range(wl.S)]
                    for _ in range(wl.L)]).astype(np.int32)
    if skew:
        sel[..., 0] = 0
    sel = H.to_dev(sel)
    w = torch.rand((wl.L, wl.S, wl.K), device="cuda")
    ys = []
    for impl in (mb.FFN_SIMT, mb.FFN_TENSOR):
        eng = mb.engine_for(wl, ffn_impl=impl)
        eng.set_experts(**W)
        ys.append(eng.moe_forward(x, sel, w).cpu().numpy())
        eng.cache_stats()
    H.ffn_close(ys[1], ys[0])


@pytest.mark.parametrize("seed", range(10))
def test_random_configurations_end_to_end(seed):
    """Seeded random shapes and routing parameters (C < K, C >= E, J = 0, J = K, E not a multiple of 32, with
    and without shared experts, ragged stream counts) through route + forward on the tensor-core paths."""
    rng = np.random.default_rng(1000 + seed)
    E = int(rng.integers(2, 97))
    K = int(rng.integers(1, min(E, 8) + 1))
    J = int(rng.integers(0, K + 1))
    C = int(rng.choice([1, max(1, K - 1), K, max(K, E // 2), E, E + 3]))
    wl = synth.QWEN.with_(L=int(rng.integers(1, 4)), S=int(rng.integers(1, 150)), E=E, K=K, J=J, C=C,
                          d=128 * int(rng.integers(1, 5)), I=128 * int(rng.integers(1, 6)),
                          n_shared=int(rng.integers(0, 3)), lam=float(rng.choice([0.0, 0.3, 0.5, 1.0, 2.0])),
                          seed=100 + seed)
    worst = run_forward_case(wl, 2, mb.FFN_TENSOR)
    print("random config %d: L=%d S=%d E=%d K=%d J=%d C=%d d=%d I=%d sh=%d lam=%.1f -> max abs err %.2e" % (
        seed, wl.L, wl.S, E, K, J, C, wl.d, wl.I, wl.n_shared, wl.lam, worst[0]))


def test_decode_step_from_host_buffers():
    wl = synth.QWEN.with_(L=2, S=16, E=12, K=4, C=6, d=256, I=256, n_shared=1)
    Wr, W = wl.router(), H.weights_for(wl)
    eng, ref = mb.engine_for(wl), mb.engine_for(wl)
    for e in (eng, ref):
        e.set_router(H.to_dev(Wr))
        e.set_experts(**{k: (None if v is None else H.to_dev(v)) for k, v in W.items()})
    xh = torch.empty((wl.L, wl.S, wl.d), dtype=torch.bfloat16).pin_memory()
    yh = torch.empty((wl.L, wl.S, wl.d), dtype=torch.float32).pin_memory()
    sh = torch.empty((wl.L, wl.S, wl.K), dtype=torch.int32).pin_memory()
    for x in wl.hidden_trace(4):
        xh.copy_(torch.from_numpy(x.view(np.int16)).view(torch.bfloat16))
        eng.decode_step_host(xh, yh, sh)
        xd = xh.cuda()
        sel, w = ref.route_step(hidden=xd[None])
        y = ref.moe_forward(xd, sel[0], w[0])
        assert torch.equal(sh, sel[0].cpu())
        # y is summed with fp32 atomics on the tensor path: same terms, order not fixed
        assert torch.allclose(yh, y.cpu(), rtol=1e-5, atol=1e-6)


@pytest.mark.parametrize("E,K,S,T", [(8, 2, 5, 60), (60, 4, 7, 80), (130, 7, 3, 50), (16, 1, 4, 100)])
def test_belady_replay_matches_the_oracle(E, K, S, T):
    """Optimal-eviction miss counts on the trace the route kernel produces at lambda = 0, for several cache
    sizes at once, against the oracle's farthest-next-use replay (itself pinned by exhaustive search)."""
    from oracle import oracle as orc
    L = 2
    wl = synth.TINY.with_(L=L, E=E, K=K, J=0, C=max(K, E // 2), S=S, lam=0.0, d=64, I=64)
    eng = mb.engine_for(wl)
    z = ar1_logits(E + K, T, L, S, E, rho=0.6)
    sel, _ = eng.route_step(logits=H.to_dev(z), n_steps=T)
    caps = sorted({K, K + 1, max(K, E // 4), max(K, E // 2), E})
    got = mb.belady_replay(sel, E, caps).cpu().numpy()
    tr = sel.cpu().numpy()
    lru_total, _ = eng.cache_stats()
    for ci, c in enumerate(caps):
        for l in range(L):
            for s in range(S):
                assert got[ci, l, s] == orc.belady_misses(tr[:, l, s], E, c)
    # lossless bound: at the engine's capacity Belady cannot do worse than the LRU run that made the trace
    assert got[caps.index(wl.C)].sum() <= lru_total[2]
    assert (np.diff(got.sum(axis=(1, 2))) <= 0).all()            # more cache, never more misses


def test_bounded_wait_gives_up_and_the_context_survives():
    """A wait that can never be satisfied ends after its limit with an error status instead of hanging;
    afterwards the same context routes correctly."""
    wl = synth.TINY.with_(L=1, S=4)
    eng = mb.engine_for(wl)
    assert eng.lib.mcce_selftest_wait_timeout(eng.ctx, 1_000_000) == 0          # 1 ms limit
    with pytest.raises(mb.McceError, match="bounded wait"):
        eng.cache_stats()
    eng.reset()                                                                  # clears the error word
    z = ar1_logits(5, 4, wl.L, wl.S, wl.E)
    H.check_route_exact(eng, H.oracle_for(wl), z)


def test_pipelined_host_steps_match_synchronous_ones():
    wl = synth.QWEN.with_(L=2, S=16, E=12, K=4, C=6, d=256, I=256, n_shared=1)
    Wr, W = wl.router(), H.weights_for(wl)
    a, b = mb.engine_for(wl), mb.engine_for(wl)
    for e in (a, b):
        e.set_router(H.to_dev(Wr))
        e.set_experts(**{k: (None if v is None else H.to_dev(v)) for k, v in W.items()})
    T = 7
    xs = torch.stack([torch.from_numpy(x.view(np.int16)).view(torch.bfloat16) for x in wl.hidden_trace(T)]).pin_memory()
    y_sync = torch.empty((T, wl.L, wl.S, wl.d), dtype=torch.float32).pin_memory()
    s_sync = torch.empty((T, wl.L, wl.S, wl.K), dtype=torch.int32).pin_memory()
    y_pipe, s_pipe = torch.zeros_like(y_sync).pin_memory(), torch.zeros_like(s_sync).pin_memory()
    for t in range(T):
        a.decode_step_host(xs[t], y_sync[t], s_sync[t])
        b.pipeline_submit_host(xs[t], y_pipe[t], s_pipe[t])
    b.pipeline_wait()
    assert torch.equal(s_sync, s_pipe)
    assert torch.allclose(y_sync, y_pipe, rtol=1e-5, atol=1e-6)
    assert a.cache_stats()[0] == b.cache_stats()[0]


@pytest.mark.parametrize("deterministic", [False, True])
def test_pipelined_device_steps_match_step_by_step_calls(deterministic):
    """mcce_pipeline_submit (routing + grouping of step t+1 on an internal stream while the experts of step t run)
    against one mcce_route_step + mcce_moe_forward per token: same selections, cache state and counters; y bit
    for bit in deterministic mode, else equal up to the order of the atomic adds."""
    wl = synth.QWEN.with_(L=3, S=40, E=16, K=4, C=8, d=256, I=384, n_shared=1)
    Wr, W = wl.router(), H.weights_for(wl)
    a, b = mb.engine_for(wl, deterministic=deterministic), mb.engine_for(wl, deterministic=deterministic)
    for e in (a, b):
        e.set_router(H.to_dev(Wr))
        e.set_experts(**{k: (None if v is None else H.to_dev(v)) for k, v in W.items()})
    T = 9
    xs = torch.stack([H.to_dev(x) for x in wl.hidden_trace(T)])
    torch.cuda.synchronize()
    ys = torch.zeros((T, wl.L, wl.S, wl.d), dtype=torch.float32, device="cuda")
    sels = torch.zeros((T, wl.L, wl.S, wl.K), dtype=torch.int32, device="cuda")
    for t in range(T):
        b.pipeline_submit(xs[t], ys[t], sels[t])
    b.pipeline_wait()
    for t in range(T):
        sel, w = a.route_step(hidden=xs[t:t + 1])
        y = a.moe_forward(xs[t], sel[0], w[0])
        assert torch.equal(sel[0], sels[t]), "token %d" % t
        if deterministic:
            assert torch.equal(y, ys[t])
        else:
            assert torch.allclose(y, ys[t], rtol=1e-5, atol=1e-6)
    assert a.cache_stats()[0] == b.cache_stats()[0]
    assert np.array_equal(a.cache_state()[0], b.cache_state()[0])
    # the context goes on with the ordinary calls afterwards
    sel_a, _ = a.route_step(hidden=xs[:1])
    sel_b, _ = b.route_step(hidden=xs[:1])
    assert torch.equal(sel_a, sel_b)


# ---- argument checking: errors come back as codes, nothing is launched ------------------------------------
def test_bad_arguments_are_rejected():
    with pytest.raises(mb.McceError):
        mb.Engine(L=1, E=300, K=2, J=1, n_shared=0, d=64, I=64, C_cap=4, S=4, lam=0.5)      # E too large
    with pytest.raises(mb.McceError):
        mb.Engine(L=1, E=8, K=2, J=3, n_shared=0, d=64, I=64, C_cap=4, S=4, lam=0.5)        # J > K
    with pytest.raises(mb.McceError):
        mb.Engine(L=1, E=8, K=2, J=1, n_shared=0, d=64, I=64, C_cap=4, S=4, lam=float("nan"))
    eng = mb.engine_for(synth.TINY)
    x = torch.zeros((1, 4, 64), device="cuda")
    with pytest.raises(mb.McceError):
        eng.route_step(hidden=x[None])                                                       # router not set
    with pytest.raises(mb.McceError):
        eng.moe_forward(x, torch.zeros((1, 4, 2), dtype=torch.int32, device="cuda"),
                        torch.zeros((1, 4, 2), device="cuda"))                               # experts not set
    lib = mb.load()
    assert lib.mcce_route_step(eng.ctx, 1, None, None, None, None, None, None) == -1
    assert lib.mcce_workspace_bytes(None) == 0
