"""Pins for the CPU oracle: every check here compares the oracle with something that is NOT the
oracle's own formula retyped -- an identity the paper states, a value it prints, a closed form, a
library routine on a special case, or exhaustive search on a tiny input."""
import itertools
import os
from collections import OrderedDict

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2412_00099_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def make(E=8, K=2, J=1, C=4, S=3, L=2, lam=0.5, delta_mode=0, renorm=1, d=16, I=8, dtype=0, n_shared=0,
         fixed_delta=None):
    cfg = orc.OracleConfig(L, E, K, J, n_shared, d, I, C, S, lam, delta_mode, renorm, dtype)
    return orc.Oracle(cfg, fixed_delta=fixed_delta)


def ar1_logits(rng, T, L, S, E, rho=0.8):
    z = np.empty((T, L, S, E), np.float32)
    h = rng.standard_normal((L, S, E))
    for t in range(T):
        h = rho * h + np.sqrt(1 - rho * rho) * rng.standard_normal((L, S, E))
        z[t] = (1.5 * h).astype(np.float32)
    return z


def plain_topk(z, K):
    """Reference selection: stable sort by value descending, ties to the lower index."""
    idx = np.lexsort((np.arange(z.shape[-1]), -z.astype(np.float64)))
    return idx[:K]


# ---- P1 / P2: the two reductions to the original routing ------------------------------------------
@pytest.mark.parametrize("J", [0, 1, 2, 3])
def test_lambda_zero_is_plain_topk(J):
    """lambda = 0 reproduces the original routing (Eq. 7 and the sentence after it)."""
    rng = np.random.default_rng(J)
    o = make(E=11, K=3, J=J, C=4, lam=0.0)
    for z in ar1_logits(rng, 40, 2, 3, 11):
        sel, _ = o.route(z)
        for l in range(2):
            for s in range(3):
                assert sel[l, s].tolist() == plain_topk(z[l, s], 3).tolist()


@pytest.mark.parametrize("lam", [0.0, 0.3, 1.0, 5.0])
def test_J_equals_K_is_plain_topk(lam):
    """With J = K the guaranteed top-J experts fill the selection: routing cannot change as a set."""
    rng = np.random.default_rng(7)
    o = make(E=9, K=3, J=3, C=4, lam=lam)
    for z in ar1_logits(rng, 40, 2, 3, 9):
        sel, _ = o.route(z)
        for l in range(2):
            for s in range(3):
                assert sorted(sel[l, s].tolist()) == sorted(plain_topk(z[l, s], 3).tolist())


# ---- P3: C >= E leaves only compulsory misses -----------------------------------------------------
@pytest.mark.parametrize("C", [8, 12])
def test_full_cache_only_cold_misses(C):
    rng = np.random.default_rng(3)
    o = make(E=8, K=2, J=1, C=C, lam=0.4)
    seen = [[set() for _ in range(3)] for _ in range(2)]
    for z in ar1_logits(rng, 60, 2, 3, 8):
        sel, _ = o.route(z)
        for l in range(2):
            for s in range(3):
                seen[l][s].update(sel[l, s].tolist())
    total, per_layer = o.stats()
    distinct = sum(len(x) for row in seen for x in row)
    assert total[2] == total[3] == distinct          # misses == cold misses == distinct experts
    assert total[0] == 60 * 6 and total[1] == 60 * 6 * 2


# ---- P4: saturation -- a bias larger than the logit range is the list promote operator -----------
def py_promote(subset, all_):
    return list(subset) + [x for x in all_ if x not in subset]


@pytest.mark.parametrize("J", [0, 1, 2])
def test_saturated_bias_equals_list_promote(J):
    rng = np.random.default_rng(11 + J)
    E, K, C = 10, 3, 5
    o = make(E=E, K=K, J=J, C=C, lam=2.0, L=1, S=2)   # lambda*Delta_avg >= 2*mean range ...
    zs = ar1_logits(rng, 50, 1, 2, E)
    for t, z in enumerate(zs):
        resident_before = (o.stamp != 0).copy()
        sel, _, margin, delta = o.route(z, want_margin=True)
        for s in range(2):
            zz = z[0, s]
            if 2.0 * delta[0, s] <= zz.max() - zz.min():
                continue                                  # ... but only tokens where it saturates count
            r = plain_topk(zz, E).tolist()
            m_tilde = set(np.flatnonzero(resident_before[0, s]).tolist()) | set(r[:J])
            expect = py_promote([e for e in r if e in m_tilde], r)[:K]
            assert sel[0, s].tolist() == expect
            assert orc.promote([e for e in r if e in m_tilde], r)[:K] == expect


# ---- P5: the appendix's worked example ------------------------------------------------------------
def _golden():
    out = {}
    for line in open(os.path.join(GOLDEN, "max_rank_example.txt")):
        if line.startswith("#") or "=" not in line:
            continue
        k, v = line.split("=")
        out[k.strip()] = [int(x) for x in v.split()]
    return out


def test_worked_max_rank_example():
    g = _golden()
    r = g["r"]
    in_cache = np.zeros(7, np.uint8)
    in_cache[g["cache"]] = 1
    M, K, J = g["M"][0], g["K"][0], g["J"][0]
    step1 = orc.promote([e for e in r[:M] if in_cache[e]], r)
    assert step1 == g["after_promote_cache"]
    assert orc.promote(r[:J], step1) == g["after_promote_topj"]
    assert orc.max_rank(r, in_cache, M, J) == g["after_promote_topj"]
    assert orc.max_rank(r, in_cache, M, J)[:K] == g["selected"]


def test_cumsum_threshold_picks_smallest_M():
    """Algorithm 2: M is the first rank count whose probability mass reaches p, then Algorithm 1."""
    w = np.array([0.0, 0.4, 0.3, 0.15, 0.1, 0.04, 0.01], np.float32)  # experts 1..6
    r = [1, 2, 3, 4, 5, 6]
    in_cache = np.zeros(7, np.uint8)
    in_cache[[3, 4, 6]] = 1
    M, out = orc.cumsum_threshold(r, w, in_cache, 0.8, 1)
    assert M == 3 and out == [1, 3, 2, 4, 5, 6]        # 0.4+0.3 < 0.8 <= 0.4+0.3+0.15
    M, out = orc.cumsum_threshold(r, w, in_cache, 0.9, 1)
    assert M == 4 and out == [1, 3, 4, 2, 5, 6]
    M, out = orc.cumsum_threshold(r, w, in_cache, 0.3, 0)
    assert M == 1 and out == r                          # peaky router: nothing may be promoted
    # "until the threshold is reached": a partial sum that equals p exactly stops the walk
    w2 = np.array([0.0, 0.5, 0.25, 0.125, 0.0625, 0.03125, 0.03125], np.float32)
    M, out = orc.cumsum_threshold(r, w2, in_cache, 0.75, 0)
    assert M == 2 and out == r
    M, out = orc.cumsum_threshold(r, w2, in_cache, 0.875, 0)
    assert M == 3 and out == [3, 1, 2, 4, 5, 6]


def test_cumsum_mode_reaches_the_threshold_exactly():
    """Four equal logits give probabilities of exactly 1/4: with p = 1/2 the walk stops after two ranks, so
    the cached expert at rank 3 is outside the window and the router's top-1 stays selected."""
    cfg = orc.OracleConfig(1, 4, 1, 0, 0, 16, 8, 2, 1, 0.5, 0, 1, 0, 2, 0, 0.5)
    o = orc.Oracle(cfg)
    o.reset(init_order=np.array([[[2, -1]]], np.int32))
    sel, _ = o.route(np.zeros((1, 1, 4), np.float32))
    assert sel[0, 0].tolist() == [0]
    cfg.cum_threshold = 0.51                    # now three ranks are needed and the cached expert wins
    o = orc.Oracle(cfg)
    o.reset(init_order=np.array([[[2, -1]]], np.int32))
    sel, _ = o.route(np.zeros((1, 1, 4), np.float32))
    assert sel[0, 0].tolist() == [2]


# ---- hand-computed instances of Eq. 7 / Eq. 8 / Eq. 4 / the in-token LRU order --------------------
def test_eq7_hand_examples():
    """z = [3,2,1,0], expert 3 cached, K=1, J=0, Delta fixed to the range 3:
    lambda=0.5 -> z'_3 = 1.5 (not enough), lambda=1.0 -> 3.0 ties with expert 0 (lower index wins),
    lambda=1.1 -> 3.3 (expert 3 selected, a hit)."""
    z = np.array([[[3, 2, 1, 0]]], np.float32)
    for lam, want, misses in [(0.5, 0, 1), (1.0, 0, 1), (1.1, 3, 0)]:
        o = make(E=4, K=1, J=0, C=2, L=1, S=1, lam=lam, delta_mode=1, fixed_delta=[3.0])
        o.reset(init_order=np.array([[[3, -1]]], np.int32))
        sel, w = o.route(z)
        assert sel[0, 0, 0] == want
        assert o.stats()[0][2] == misses
        assert w[0, 0, 0] == pytest.approx(1.0)         # weight renormalised over one expert


def test_eq7_top_j_is_always_selected_and_weights_ignore_bias():
    """Top-J of the router stays selected however strong the bias; weights come from z, not z'."""
    z = np.array([[[5.0, 0.1, 0.0, -0.1, -0.2, -0.3]]], np.float32)
    o = make(E=6, K=2, J=1, C=3, L=1, S=1, lam=1.0, delta_mode=1, fixed_delta=[100.0])
    o.reset(init_order=np.array([[[4, 5, -1]]], np.int32))
    sel, w = o.route(z)
    assert sel[0, 0].tolist() == [0, 4]                  # top-1 kept, then best cached expert
    p = torch.softmax(torch.tensor([5.0, -0.2], dtype=torch.float64), 0).numpy()
    assert np.allclose(w[0, 0], p, rtol=1e-6)


def test_eq8_running_mean():
    """Ranges 1 then 3 -> Delta_avg 1 then 2 (cumulative mean that includes the current token)."""
    o = make(E=3, K=1, J=0, C=1, L=1, S=1, lam=0.0)
    _, _, _, d1 = o.route(np.array([[[0, 0.5, 1]]], np.float32), want_margin=True)
    _, _, _, d2 = o.route(np.array([[[-1, 0, 2]]], np.float32), want_margin=True)
    assert d1[0, 0] == 1.0 and d2[0, 0] == 2.0


def test_in_token_order_higher_weight_is_evicted_first():
    """K=2 into a cache of one: the expert with the higher router weight goes first, the lower stays."""
    o = make(E=4, K=2, J=0, C=1, L=1, S=1, lam=0.0)
    o.route(np.array([[[0.0, 2.0, 1.0, -1.0]]], np.float32))      # selects 1 (w high) and 2 (w low)
    assert o.order()[0, 0].tolist() == [2]
    # both were misses; next token selects 2 (hit, it stayed) and 0 (miss)
    o.route(np.array([[[1.0, -2.0, 2.0, -1.0]]], np.float32))
    assert o.stats()[0][2] == 3
    o2 = make(E=4, K=2, J=0, C=3, L=1, S=1, lam=0.0)
    o2.route(np.array([[[0.0, 2.0, 1.0, -1.0]]], np.float32))
    assert o2.order()[0, 0].tolist() == [2, 1, -1]                 # most recent first


def test_hits_counted_against_pre_token_cache():
    """Eq. 4 intersects with the cache before the token: an expert inserted by this token is a miss
    even though it is resident afterwards."""
    o = make(E=4, K=2, J=0, C=2, L=1, S=1, lam=0.0)
    o.route(np.array([[[3, 2, 0, 0]]], np.float32))   # 0,1 -> 2 misses
    o.route(np.array([[[3, 0, 2, 0]]], np.float32))   # 0 hit, 2 miss
    o.route(np.array([[[0, 3, 2, 0]]], np.float32))   # 1 was evicted by 2 -> miss, 2 hit
    total, _ = o.stats()
    assert total.tolist() == [3, 6, 4, 3]


# ---- P6: order preservation inside the promoted set and its complement ----------------------------
def test_rerank_preserves_relative_orders_and_keeps_top_j():
    rng = np.random.default_rng(5)
    E, K, J, C = 12, 4, 2, 5
    o = make(E=E, K=K, J=J, C=C, lam=0.6, L=1, S=4)
    for z in ar1_logits(rng, 80, 1, 4, E):
        resident = (o.stamp != 0).copy()
        sel, _ = o.route(z)
        for s in range(4):
            r = plain_topk(z[0, s], E).tolist()
            assert set(r[:J]) <= set(sel[0, s].tolist())
            m_tilde = set(np.flatnonzero(resident[0, s]).tolist()) | set(r[:J])
            inside = [e for e in sel[0, s] if e in m_tilde]
            outside = [e for e in sel[0, s] if e not in m_tilde]
            # each group is a prefix of the router's own ranking restricted to that group
            assert inside == [e for e in r if e in m_tilde][:len(inside)]
            assert outside == [e for e in r if e not in m_tilde][:len(outside)]


# ---- P7: weights ------------------------------------------------------------------------------------
@pytest.mark.parametrize("renorm", [0, 1])
def test_weights_are_softmax_of_unmodified_logits(renorm):
    rng = np.random.default_rng(9)
    E, K = 10, 3
    o = make(E=E, K=K, J=1, C=4, lam=0.8, renorm=renorm)
    for z in ar1_logits(rng, 30, 2, 3, E):
        sel, w = o.route(z)
        zt = torch.tensor(z, dtype=torch.float64)
        full = torch.softmax(zt, -1)
        picked = torch.gather(full, -1, torch.tensor(sel, dtype=torch.int64))
        if renorm:
            picked = picked / picked.sum(-1, keepdim=True)
            assert np.allclose(w.sum(-1), 1.0, atol=1e-6)
        assert np.allclose(w, picked.numpy(), rtol=1e-6, atol=1e-9)


# ---- P8 / P9: LRU against two independent re-implementations ---------------------------------------
def test_lru_matches_list_lru_and_invariants():
    rng = np.random.default_rng(13)
    for (E, K, J, C, lam) in [(8, 2, 1, 4, 0.5), (8, 3, 0, 2, 0.0), (6, 2, 2, 1, 1.0), (9, 4, 1, 9, 0.7),
                              (5, 5, 0, 3, 0.3)]:
        o = make(E=E, K=K, J=J, C=C, lam=lam, L=1, S=2)
        lists = [[], []]                                   # front = least recently used
        touched = [set(), set()]
        for z in ar1_logits(rng, 60, 1, 2, E):
            sel, _ = o.route(z)
            for s in range(2):
                order = sorted(sel[0, s].tolist(), key=lambda e: (-float(z[0, s, e]), e))
                for e in order:                            # highest weight first = oldest
                    if e in lists[s]:
                        lists[s].remove(e)
                    lists[s].append(e)
                while len(lists[s]) > C:
                    lists[s].pop(0)
                touched[s].update(order)
                got = [e for e in o.order()[0, s].tolist() if e >= 0]
                assert got == lists[s][::-1]
                assert len(got) == min(C, len(touched[s]))
                st = o.stamp[0, s]
                assert len(set(st[st != 0].tolist())) == (st != 0).sum()   # strict total order
        total, _ = o.stats()
        assert total[1] == total[0] * K and 0 <= total[2] <= total[1]


def test_k1_is_textbook_lru():
    rng = np.random.default_rng(17)
    E, C = 7, 3
    o = make(E=E, K=1, J=0, C=C, lam=0.0, L=1, S=1)
    od, misses = OrderedDict(), 0
    for z in ar1_logits(rng, 200, 1, 1, E, rho=0.5):
        sel, _ = o.route(z)
        e = int(sel[0, 0, 0])
        if e in od:
            od.move_to_end(e)
        else:
            misses += 1
            od[e] = True
            if len(od) > C:
                od.popitem(last=False)
        assert [x for x in o.order()[0, 0].tolist() if x >= 0] == list(od.keys())[::-1]
    assert o.stats()[0][2] == misses


# ---- P10 / P11: Belady ---------------------------------------------------------------------------
def brute_force_min_misses(trace, E, C):
    """Exhaustive search over every demand-fetch eviction policy (experts of the current token are
    pinned)."""
    T = len(trace)
    best = [10 ** 9]

    def rec(t, cache, misses):
        if misses >= best[0]:
            return
        if t == T:
            best[0] = misses
            return
        req = set(trace[t])
        misses += len(req - cache)
        cache = cache | req
        over = len(cache) - C
        if over <= 0:
            rec(t + 1, cache, misses)
            return
        for victims in itertools.combinations(sorted(cache - req), over):
            rec(t + 1, cache - set(victims), misses)

    rec(0, frozenset(), 0)
    return best[0]


def test_belady_equals_exhaustive_search_and_bounds_lru():
    rng = np.random.default_rng(19)
    for trial in range(25):
        E = int(rng.integers(4, 8))
        K = int(rng.integers(1, 3))
        C = int(rng.integers(K, 5))
        T = int(rng.integers(4, 11))
        trace = np.stack([rng.choice(E, K, replace=False) for _ in range(T)]).astype(np.int32)
        b = orc.belady_misses(trace, E, C)
        assert b == brute_force_min_misses([tuple(x) for x in trace.tolist()], E, C)
        assert b <= orc.lru_misses(trace, E, C)


def test_cache_prior_may_beat_belady_on_the_original_trace():
    """Lossless policies are bounded by Belady on the router's own trace; the lossy reranking is not.
    Nothing is asserted about how often -- only that the bound orders LRU correctly and that the
    comparison is well defined."""
    rng = np.random.default_rng(23)
    E, K, C, T = 8, 2, 4, 200
    zs = ar1_logits(rng, T, 1, 1, E, rho=0.6)
    base = make(E=E, K=K, J=1, C=C, lam=0.0, L=1, S=1)
    trace = np.stack([base.route(z)[0][0, 0] for z in zs])
    # touch order inside a token for the plain LRU helper: higher weight first
    ordered = np.stack([sorted(tr.tolist(), key=lambda e: (-float(z[0, 0, e]), e)) for tr, z in zip(trace, zs)])
    lru = orc.lru_misses(ordered.astype(np.int32), E, C)
    assert lru == base.stats()[0][2]
    bel = orc.belady_misses(trace.astype(np.int32), E, C)
    assert bel <= lru
    prior = make(E=E, K=K, J=1, C=C, lam=1.0, L=1, S=1)
    for z in zs:
        prior.route(z)
    assert prior.stats()[0][2] <= lru        # direction of the paper's claim on a local trace


# ---- P12: direction of the miss-rate curve on the Tiny workload -----------------------------------
def test_miss_rate_falls_with_lambda_on_tiny():
    """Direction of the paper's trade-off curve on a trace with temporal locality: the miss rate falls
    as lambda grows, and with J > 0 it flattens out at the floor the guaranteed top-J experts impose."""
    wl = synth.TINY
    Wr = wl.router()
    xs = list(wl.hidden_trace(wl.T))
    for J in (0, 1):
        rates = []
        for lam in (0.0, 0.5, 1.0):
            o = orc.Oracle(orc.OracleConfig(wl.L, wl.E, wl.K, J, 0, wl.d, wl.I, wl.C, wl.S, lam, 0, 1, 0))
            for x in xs:
                o.route(o.logits(Wr, x))
            total, _ = o.stats()
            rates.append(total[2] / total[1])
        assert rates[0] > 1.5 * rates[1] and rates[0] > 1.5 * rates[2] > 0
        if J == 0:
            assert rates[1] > rates[2]
        else:
            assert abs(rates[1] - rates[2]) < 0.1 * rates[1]      # plateau


# ---- P13: library special cases -----------------------------------------------------------------
def test_lambda_zero_matches_torch_topk_softmax():
    rng = np.random.default_rng(29)
    E, K = 16, 4
    o = make(E=E, K=K, J=1, C=8, lam=0.0, renorm=0, L=1, S=5)
    for z in ar1_logits(rng, 20, 1, 5, E):
        sel, w = o.route(z)
        pv, pi = torch.topk(torch.softmax(torch.tensor(z, dtype=torch.float64), -1), K, dim=-1)
        assert np.array_equal(sel, pi.numpy())
        assert np.allclose(w, pv.numpy(), rtol=1e-6)


def test_router_logits_match_float64_matmul():
    rng = np.random.default_rng(31)
    L, S, E, d = 2, 3, 5, 24
    Wr = rng.standard_normal((L, E, d)).astype(np.float32)
    x = rng.standard_normal((L, S, d)).astype(np.float32)
    o = make(E=E, K=2, J=0, C=2, L=L, S=S, d=d)
    ref = np.einsum("led,lsd->lse", Wr.astype(np.float64), x.astype(np.float64))
    assert np.allclose(o.logits(Wr, x), ref, rtol=1e-6, atol=1e-6)
    # bf16 hidden
    xb = synth.to_bf16_bits(x).reshape(x.shape)
    ob = make(E=E, K=2, J=0, C=2, L=L, S=S, d=d, dtype=1)
    refb = np.einsum("led,lsd->lse", Wr.astype(np.float64), synth.bf16_bits_to_f32(xb).astype(np.float64))
    assert np.allclose(ob.logits(Wr, xb), refb, rtol=1e-6, atol=1e-6)


def torch_swiglu(x, Wg, Wu, Wd, round_h):
    g, u = Wg @ x, Wu @ x
    h = torch.nn.functional.silu(g) * u
    if round_h:
        h = h.to(torch.bfloat16).to(torch.float64)
    return Wd @ h


@pytest.mark.parametrize("dtype", [0, 1])
def test_ffn_matches_float64_torch_swiglu(dtype):
    rng = np.random.default_rng(37)
    L, S, E, K, nsh, d, I = 2, 3, 4, 2, 1, 24, 40         # I != d catches a transposed operand
    mk = lambda *sh: (rng.standard_normal(sh) * 0.3).astype(np.float32)
    x, Wg, Wu, Wd = mk(L, S, d), mk(L, E, I, d), mk(L, E, I, d), mk(L, E, d, I)
    sg, su, sd = mk(L, nsh, I, d), mk(L, nsh, I, d), mk(L, nsh, d, I)
    sel = np.stack([[rng.choice(E, K, replace=False) for _ in range(S)] for _ in range(L)]).astype(np.int32)
    w = rng.random((L, S, K)).astype(np.float32)
    arrs = [x, Wg, Wu, Wd, sg, su, sd]
    if dtype:
        bits = [synth.to_bf16_bits(a).reshape(a.shape) for a in arrs]
        vals = [synth.bf16_bits_to_f32(b) for b in bits]
    else:
        bits, vals = arrs, arrs
    o = make(E=E, K=K, J=1, C=2, L=L, S=S, d=d, I=I, dtype=dtype, n_shared=nsh)
    y = o.ffn(bits[0], sel, w, *bits[1:])
    tx, tg, tu, td, tsg, tsu, tsd = [torch.tensor(v, dtype=torch.float64) for v in vals]
    for l in range(L):
        for s in range(S):
            ref = sum(float(w[l, s, k]) * torch_swiglu(tx[l, s], tg[l, sel[l, s, k]], tu[l, sel[l, s, k]],
                                                       td[l, sel[l, s, k]], dtype) for k in range(K))
            ref = ref + torch_swiglu(tx[l, s], tsg[l, 0], tsu[l, 0], tsd[l, 0], dtype)
            assert np.allclose(y[l, s], ref.numpy(), rtol=1e-5, atol=1e-6)


def test_single_expert_moe_is_a_dense_ffn():
    rng = np.random.default_rng(41)
    d, I = 12, 20
    x = rng.standard_normal((1, 1, d)).astype(np.float32)
    Wg, Wu = [rng.standard_normal((1, 1, I, d)).astype(np.float32) for _ in range(2)]
    Wd = rng.standard_normal((1, 1, d, I)).astype(np.float32)
    o = make(E=1, K=1, J=0, C=1, L=1, S=1, d=d, I=I, lam=0.5)
    Wr = rng.standard_normal((1, 1, d)).astype(np.float32)
    sel, w = o.route(o.logits(Wr, x))
    assert sel.item() == 0 and w.item() == pytest.approx(1.0)
    y = o.ffn(x, sel, w, Wg, Wu, Wd)
    ref = torch_swiglu(*[torch.tensor(a, dtype=torch.float64) for a in (x[0, 0], Wg[0, 0], Wu[0, 0], Wd[0, 0])], 0)
    assert np.allclose(y[0, 0], ref.numpy(), rtol=1e-5, atol=1e-6)


def test_bf16_rounding_matches_torch():
    """The rounding of h, isolated: with x = 1, W_g = b >= 40 (silu(b) == b in double), W_u = a and
    W_d = 1 the expert returns round_bf16(a*b); a*b has up to 16 significant bits, so ties occur."""
    rng = np.random.default_rng(43)
    a = synth.bf16_bits_to_f32(synth.to_bf16_bits((rng.standard_normal(400) * 3).astype(np.float32)))
    b = synth.bf16_bits_to_f32(synth.to_bf16_bits(rng.uniform(40, 100, 400).astype(np.float32)))
    a[:3], b[:3] = [1.5, -1.5, 1.25], [40.25, 40.25, 40.5]         # 60.375, -60.375 (ties), 50.625
    one = synth.to_bf16_bits(np.array([1.0], np.float32))
    for ai, bi in zip(a, b):
        got = orc.expert_ffn(one, synth.to_bf16_bits(np.array([[bi]], np.float32)),
                             synth.to_bf16_bits(np.array([[ai]], np.float32)), one.reshape(1, 1), 1)[0]
        want = torch.tensor(float(ai) * float(bi), dtype=torch.float32).to(torch.bfloat16).double().item()
        assert got == want
    assert orc.expert_ffn(one, synth.to_bf16_bits(np.array([[40.25]], np.float32)),
                          synth.to_bf16_bits(np.array([[1.5]], np.float32)), one.reshape(1, 1), 1)[0] == 60.5


# ---- P14: determinism and resume --------------------------------------------------------------------
def test_deterministic_and_resumable():
    rng = np.random.default_rng(47)
    zs = ar1_logits(rng, 40, 2, 3, 8)
    a, b = make(), make()
    outs_a = [a.route(z) for z in zs]
    outs_b = []
    for t, z in enumerate(zs):
        if t == 17:                                      # resume from an exported snapshot
            snap = b.snapshot()
            b = make()
            b.restore(snap)
        outs_b.append(b.route(z))
    for (s1, w1), (s2, w2) in zip(outs_a, outs_b):
        assert np.array_equal(s1, s2) and np.array_equal(w1.view(np.uint32), w2.view(np.uint32))
    assert np.array_equal(a.stamp, b.stamp) and np.array_equal(a.counters, b.counters)


def test_initial_cache_state_is_older_than_any_touch():
    o = make(E=6, K=1, J=0, C=3, L=1, S=1, lam=0.0)
    o.reset(init_order=np.array([[[4, 2, 5]]], np.int32))      # 4 most recent, 5 least
    assert o.order()[0, 0].tolist() == [4, 2, 5]
    o.route(np.array([[[9, 0, 0, 0, 0, 0]]], np.float32))       # miss on 0 evicts 5
    assert o.order()[0, 0].tolist() == [0, 4, 2]
    o.route(np.array([[[0, 0, 9, 0, 0, 0]]], np.float32))       # hit on 2
    assert o.order()[0, 0].tolist() == [2, 0, 4]
    assert o.stats()[0].tolist() == [2, 2, 1, 1]


# ---- the two baseline rerankers as routing modes (Algorithms 1 and 2) -------------------------------
def make_mode(mode, E, K, J, C, M=0, p=0.0, lam=0.5, L=1, S=3):
    cfg = orc.OracleConfig(L, E, K, J, 0, 16, 8, C, S, lam, 0, 1, 0, mode, M, p)
    return orc.Oracle(cfg)


def py_max_rank_select(z, resident, M, J, K):
    r = plain_topk(z, len(z)).tolist()
    step1 = py_promote([e for e in r[:M] if resident[e]], r)
    return py_promote(r[:J], step1)[:K]


@pytest.mark.parametrize("M", [0, 2, 4, 9])
@pytest.mark.parametrize("J", [0, 1, 2])
def test_max_rank_mode_follows_algorithm_1(M, J):
    rng = np.random.default_rng(100 + 10 * M + J)
    E, K, C = 9, 3, 4
    o = make_mode(1, E, K, J, C, M=M)
    for z in ar1_logits(rng, 60, 1, 3, E):
        resident = (o.stamp != 0).copy()
        sel, _ = o.route(z)
        for s in range(3):
            assert sel[0, s].tolist() == py_max_rank_select(z[0, s], resident[0, s], M, J, K)
            if M == 0:
                assert sel[0, s].tolist() == plain_topk(z[0, s], K).tolist()     # nothing may be promoted


@pytest.mark.parametrize("J", [0, 1, 2])
def test_max_rank_over_all_ranks_is_the_saturated_cache_prior(J):
    """Two independent routes through the oracle: Eq. 7 with a bias beyond the logit range, and the list
    operator with M = N.  Same trace, same cache evolution, same selections."""
    rng = np.random.default_rng(7 + J)
    E, K, C = 10, 3, 5
    a = make_mode(0, E, K, J, C, lam=50.0)
    b = make_mode(1, E, K, J, C, M=E)
    for z in ar1_logits(rng, 80, 1, 3, E):
        sa, wa = a.route(z)
        sb, wb = b.route(z)
        assert np.array_equal(sa, sb) and np.array_equal(wa, wb)
    assert np.array_equal(a.stamp, b.stamp) and np.array_equal(a.counters, b.counters)


@pytest.mark.parametrize("p", [0.0, 0.3, 0.6, 0.9, 1.5])
def test_cumsum_mode_follows_algorithm_2(p):
    rng = np.random.default_rng(int(p * 10) + 200)
    E, K, J, C = 8, 2, 1, 4
    o = make_mode(2, E, K, J, C, p=p)
    for z in ar1_logits(rng, 60, 1, 3, E):
        resident = (o.stamp != 0).copy()
        sel, _, margin, _ = o.route(z, want_margin=True)
        for s in range(3):
            zz = z[0, s]
            w = torch.softmax(torch.tensor(zz, dtype=torch.float64), 0).numpy()
            r = plain_topk(zz, E).tolist()
            cum = np.cumsum(w[r])
            M = int(np.searchsorted(cum, p, side="left")) + 1 if p > 0 else 0
            M = min(M, E)
            if margin[0, s] < 1e-6:
                continue                      # threshold within rounding of a partial sum: either M is right
            assert sel[0, s].tolist() == py_max_rank_select(zz, resident[0, s], M, J, K)
    if p == 0.0:
        assert o.stats()[0][2] == make_and_run_plain(E, K, J, C, int(p * 10) + 200)


def make_and_run_plain(E, K, J, C, seed):
    rng = np.random.default_rng(seed)
    o = make_mode(0, E, K, J, C, lam=0.0)
    for z in ar1_logits(rng, 60, 1, 3, E):
        o.route(z)
    return o.stats()[0][2]


# ---- cache lifetimes (the statistic of the paper's Table 2) -------------------------------------------
def test_lifetimes_match_brute_force_over_resident_sets():
    """Lifetime of a residency = number of tokens from the token that loaded the expert to the token
    that evicted it; recomputed here from the exported resident set after every token."""
    rng = np.random.default_rng(53)
    for (E, K, J, C, lam) in [(8, 2, 1, 4, 0.0), (8, 2, 1, 4, 0.7), (10, 3, 0, 2, 0.3), (6, 2, 1, 1, 0.5)]:
        o = make(E=E, K=K, J=J, C=C, lam=lam, L=1, S=2)
        loaded = [dict(), dict()]
        lives = []
        for t, z in enumerate(ar1_logits(rng, 120, 1, 2, E, rho=0.6)):
            sel, _ = o.route(z)
            after = o.order()
            for s in range(2):
                now = set(e for e in after[0, s].tolist() if e >= 0)
                for e in sel[0, s].tolist():                 # every selected expert is (re)loaded if absent
                    loaded[s].setdefault(e, t)
                for e in list(loaded[s]):
                    if e not in now:                          # evicted during this token
                        lives.append(t - loaded[s].pop(e))
        n, mean, sd = o.lifetimes()
        assert n == len(lives)
        assert mean == pytest.approx(np.mean(lives)) and sd == pytest.approx(np.std(lives))


def test_lifetimes_grow_with_lambda_on_tiny():
    """Direction of Table 2: experts stay resident longer under cache-aware routing."""
    wl = synth.TINY
    Wr = wl.router()
    xs = list(wl.hidden_trace(wl.T))
    means = []
    for lam in (0.0, 0.5):
        o = orc.Oracle(orc.OracleConfig(wl.L, wl.E, wl.K, 0, 0, wl.d, wl.I, wl.C, wl.S, lam, 0, 1, 0))
        for x in xs:
            o.route(o.logits(Wr, x))
        means.append(o.lifetimes()[1])
    assert means[1] > 1.5 * means[0]


def test_miss_trace_matches_resident_sets():
    """Per-token miss bits (slot k of the selection missed) against the resident set exported before the token."""
    rng = np.random.default_rng(59)
    E, K, C = 9, 3, 4
    o = make(E=E, K=K, J=1, C=C, lam=0.4, L=1, S=2)
    total = 0
    for z in ar1_logits(rng, 80, 1, 2, E, rho=0.6):
        before = [set(e for e in row.tolist() if e >= 0) for row in o.order()[0]]
        sel, _ = o.route(z)
        for s in range(2):
            want = sum(1 << k for k in range(K) if int(sel[0, s, k]) not in before[s])
            assert int(o.last_miss_mask[0, s]) == want
            total += bin(want).count("1")
    assert total == o.stats()[0][2]


def test_near_tie_margin_hand_instances():
    """The near-tie report (the smallest gap that decided an outcome of the step) on instances worked by hand,
    one per kind of gap: K-th against (K+1)-th promoted logit (Eq. 7), the top-J boundary of the unmodified
    logits (Sec. 3.3), neighbours in the in-token eviction order (Sec. 4.2), and the distance of the cumulative
    probability from the threshold (Algorithm 2).  All values are dyadic, so the expected gaps are exact."""
    def one(z, E, K, J, C, lam, cached=(), fixed=1.0, mode=0, p=0.0):
        cfg = orc.OracleConfig(1, E, K, J, 0, 16, 8, C, 1, lam, 1, 1, 0, mode, 0, p)
        o = orc.Oracle(cfg, fixed_delta=np.array([fixed], np.float32))
        if cached:
            init = np.full((1, 1, C), -1, np.int32)
            init[0, 0, :len(cached)] = cached
            o.reset(init_order=init)
        sel, _, margin, _ = o.route(np.array(z, np.float32).reshape(1, 1, E), want_margin=True)
        return sel[0, 0].tolist(), float(margin[0, 0])

    # (a) expert 3 is cached and gets the bias 1.0: z' = [2, 1.5, 1.25, 1.75]; the second and third largest
    #     promoted logits are 1.75 and 1.5 -> 0.25 (the selected pair's own logits, 2 and 0.75, lie 1.25 apart)
    assert one([2.0, 1.5, 1.25, 0.75], 4, 2, 0, 2, 1.0, cached=(3,)) == ([0, 3], 0.25)
    # (b) J = 1: the router's first and second choice lie 0.0625 apart; expert 2 is cached and promoted by 4 to
    #     4.5, far from everything else (K boundary 4.5 - 1.9375, in-token order 2.0 - 0.5)
    assert one([2.0, 1.9375, 0.5, 0.25], 4, 2, 1, 2, 1.0, cached=(2,), fixed=4.0) == ([0, 2], 0.0625)
    # (c) nothing cached, J = 0: the two selected experts lie 0.03125 apart (which of them is evicted first),
    #     the K boundary 0.96875
    assert one([1.0, 0.96875, 0.0, -1.0], 4, 2, 0, 2, 0.5) == ([0, 1], 0.03125)
    # (d) Algorithm 2: probabilities 4/7, 2/7, 1/7; p = 0.7 is passed by the second rank (6/7), and lies
    #     0.7 - 4/7 = 0.128571 above the first partial sum; neighbouring logits are ln 2 apart
    ln2 = float(np.log(2.0))
    sel, m = one([2 * ln2, ln2, 0.0], 3, 1, 0, 2, 0.5, mode=2, p=0.7)
    assert sel == [0] and abs(m - (0.7 - 4.0 / 7.0)) < 1e-6
    # ... and with p = 0.5 the first rank alone passes it, 4/7 - 0.5 = 0.0714 beyond
    sel, m = one([2 * ln2, ln2, 0.0], 3, 1, 0, 2, 0.5, mode=2, p=0.5)
    assert abs(m - (4.0 / 7.0 - 0.5)) < 1e-6
