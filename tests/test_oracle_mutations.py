"""Do the pins actually bite?  Each case plants one plausible mistake (a wrong sign, a dropped term, a
swapped index, an off-by-one) in a COPY of the oracle's C source, builds it, and runs the pins against
the mutated library: at least one pin must fail.  CPU only; the committed oracle is never touched."""
import ctypes as C
import os
import subprocess

import pytest

from oracle import oracle as orc
import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(orc.__file__), "mcce_oracle.c")

MUTATIONS = [
    ("promotion subtracts the bias", "zp[e] = mask[e] ? z[e] + bias : z[e];", "zp[e] = mask[e] ? z[e] - bias : z[e];"),
    ("bias ignores the logit range", "const float bias = c->lambda * delta;", "const float bias = c->lambda;"),
    ("bias applied to the uncached experts", "zp[e] = mask[e] ? z[e] + bias : z[e];",
     "zp[e] = mask[e] ? z[e] : z[e] + bias;"),
    ("top-J experts not added to the mask", "for (int j = 0; j < J; ++j) mask[topj[j]] = 1;", ";"),
    ("weights taken from the promoted logits", "w[k] = (float)(exp((double)z[sel[k]] - (double)zmax)",
     "w[k] = (float)(exp((double)zp[sel[k]] - (double)zmax)"),
    ("renormalisation denominators swapped", "(c->renorm ? denom_sel : denom_all)", "(c->renorm ? denom_all : denom_sel)"),
    ("hits counted as misses", "if (stamp[sel[k]] == 0) ++miss;", "if (stamp[sel[k]] != 0) ++miss;"),
    ("miss trace marks the hits", "if (stamp[sel[k]] == 0) miss_mask |= 1u << k;", "if (stamp[sel[k]] != 0) miss_mask |= 1u << k;"),
    ("miss trace indexed by expert instead of slot", "if (stamp[sel[k]] == 0) miss_mask |= 1u << k;",
     "if (stamp[sel[k]] == 0) miss_mask |= 1u << (sel[k] & 31);"),
    ("in-token order reversed", "stamp[e] = (int64_t)E + tok * K + r + 1;", "stamp[e] = (int64_t)E + tok * K + (K - 1 - r) + 1;"),
    ("evicts the most recent expert", "if (victim < 0 || stamp[e] < stamp[victim]) victim = e;\n        }\n        if (resident <= C) break;\n        stamp[victim] = 0;\n        if (life_all)",
     "if (victim < 0 || stamp[e] > stamp[victim]) victim = e;\n        }\n        if (resident <= C) break;\n        stamp[victim] = 0;\n        if (life_all)"),
    ("capacity off by one", "if (resident <= C) break;\n        stamp[victim] = 0;\n        if (life_all)",
     "if (resident <= C + 1) break;\n        stamp[victim] = 0;\n        if (life_all)"),
    ("ties broken towards the higher index", "return va > vb || (va == vb && ia < ib);", "return va > vb || (va == vb && ia > ib);"),
    ("ascending instead of descending sort", "return va > vb || (va == vb && ia < ib);", "return va < vb || (va == vb && ia < ib);"),
    ("running mean excludes the current token", "delta = sum_range_all[p] / (float)count_all[p];",
     "delta = (sum_range_all[p] - range) / (float)(count_all[p] > 1 ? count_all[p] - 1 : 1);"),
    ("range taken as max + min", "const float range = zmax - zmin;", "const float range = zmax + zmin;"),
    ("silu with the wrong sign in the exponent", "const double silu = g / (1.0 + exp(-g));", "const double silu = g / (1.0 + exp(g));"),
    ("gate and up swapped", "h[i] = dtype ? round_to_bf16(silu * u) : silu * u;", "h[i] = dtype ? round_to_bf16(u / (1.0 + exp(-u)) * g) : u / (1.0 + exp(-u)) * g;"),
    ("down projection transposed", "acc += load_elem(Wd, (size_t)j * I + i, dtype) * h[i];", "acc += load_elem(Wd, (size_t)i * d + j, dtype) * h[i];"),
    ("intermediate not rounded to bf16", "h[i] = dtype ? round_to_bf16(silu * u) : silu * u;", "h[i] = silu * u;"),
    ("bf16 rounding truncates", "double q = nearbyint(ldexp(m, 8));", "double q = trunc(ldexp(m, 8));"),
    ("shared experts dropped", "for (int j = 0; j < d; ++j) acc[j] += o[j];", ";"),
    ("expert weights ignored in the combine", "acc[j] += (double)w[p * K + k] * o[j];", "acc[j] += o[j];"),
    ("router row index transposed", "acc += (double)Wr[(size_t)e * d + j] * xj;", "acc += (double)Wr[(size_t)j * E + e] * xj;"),
    ("promote keeps the subset in place", "for (int i = 0; i < n_subset; ++i) out[n++] = subset[i];\n  for (int i = 0; i < n_all; ++i) {",
     "for (int i = 0; i < 0; ++i) out[n++] = subset[i];\n  for (int i = 0; i < n_all; ++i) {\n    if (n_subset >= 0) { out[n++] = all[i]; continue; }"),
    ("max-rank window off by one", "for (int i = 0; i < M && i < n; ++i)", "for (int i = 0; i <= M && i < n; ++i)"),
    ("cumulative threshold strict", "if (mass[i] >= p) M = i, reached = 1;", "if (mass[i] > p) M = i, reached = 1;"),
    ("cumulative mass skips the first rank", "mass[i + 1] = mass[i] + w_by_rank[i];",
     "mass[i + 1] = mass[i] + w_by_rank[i < n - 1 ? i + 1 : i];"),
    ("near-tie margin ignores the K / K+1 gap of the promoted logits",
     "if (K < E && c->rerank_mode == 0) m = fminf(m, zp[rank[K - 1]] - zp[rank[K]]);", ";"),
    ("near-tie margin takes the K / K+1 gap from the unmodified logits",
     "if (K < E && c->rerank_mode == 0) m = fminf(m, zp[rank[K - 1]] - zp[rank[K]]);",
     "if (K < E && c->rerank_mode == 0) m = fminf(m, z[rank[K - 1]] - z[rank[K]]);"),
    ("near-tie margin ignores the top-J boundary", "m = fminf(m, z[tj[J - 1]] - z[tj[J]]);", ";"),
    ("near-tie margin ignores the in-token order", "for (int r = 0; r + 1 < K; ++r) m = fminf(m, zsel[order[r]] - zsel[order[r + 1]]);", ";"),
    ("near-tie margin ignores the distance to the cumulative threshold", "m = fminf(m, cum_margin);", ";"),
    ("threshold distance one-sided", "fminf(mass[M] - p, p - mass[M - 1])", "(mass[M] - p)"),
    ("Belady evicts the nearest next use", "if (next > victim_next) {", "if (victim_next < 0 || next < victim_next) {"),
    ("lifetime counted from the first token", "const int64_t life = tok - load_tok_all[p * E + victim];", "const int64_t life = tok;"),
]


def run_pins():
    """A broad, fast subset of the pins; returns the names of those that fail."""
    calls = [(pins.test_lambda_zero_is_plain_topk, (1,)), (pins.test_J_equals_K_is_plain_topk, (1.0,)),
             (pins.test_full_cache_only_cold_misses, (8,)), (pins.test_saturated_bias_equals_list_promote, (1,)),
             (pins.test_worked_max_rank_example, ()), (pins.test_cumsum_threshold_picks_smallest_M, ()),
             (pins.test_eq7_hand_examples, ()), (pins.test_eq7_top_j_is_always_selected_and_weights_ignore_bias, ()),
             (pins.test_eq8_running_mean, ()), (pins.test_in_token_order_higher_weight_is_evicted_first, ()),
             (pins.test_hits_counted_against_pre_token_cache, ()),
             (pins.test_rerank_preserves_relative_orders_and_keeps_top_j, ()),
             (pins.test_weights_are_softmax_of_unmodified_logits, (0,)),
             (pins.test_weights_are_softmax_of_unmodified_logits, (1,)),
             (pins.test_lru_matches_list_lru_and_invariants, ()), (pins.test_k1_is_textbook_lru, ()),
             (pins.test_belady_equals_exhaustive_search_and_bounds_lru, ()),
             (pins.test_lambda_zero_matches_torch_topk_softmax, ()), (pins.test_router_logits_match_float64_matmul, ()),
             (pins.test_ffn_matches_float64_torch_swiglu, (0,)), (pins.test_ffn_matches_float64_torch_swiglu, (1,)),
             (pins.test_bf16_rounding_matches_torch, ()), (pins.test_initial_cache_state_is_older_than_any_touch, ()),
             (pins.test_max_rank_mode_follows_algorithm_1, (4, 1)), (pins.test_cumsum_mode_follows_algorithm_2, (0.6,)),
             (pins.test_max_rank_over_all_ranks_is_the_saturated_cache_prior, (1,)),
             (pins.test_lifetimes_match_brute_force_over_resident_sets, ()),
             (pins.test_cumsum_mode_reaches_the_threshold_exactly, ()),
             (pins.test_miss_trace_matches_resident_sets, ()),
             (pins.test_near_tie_margin_hand_instances, ())]
    failed = []
    for fn, args in calls:
        try:
            fn(*args)
        except Exception:            # assertion, or a crash of the mutated arithmetic
            failed.append(fn.__name__)
    return failed


def test_unmutated_oracle_passes_the_subset():
    assert run_pins() == []


@pytest.mark.parametrize("what,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(what, old, new, tmp_path):
    src = open(SRC).read()
    assert src.count(old) >= 1, "mutation site not found: the oracle changed, update this case"
    mutated = tmp_path / "mutated.c"
    mutated.write_text(src.replace(old, new, 1))
    lib_path = tmp_path / "libmutated.so"
    subprocess.check_call(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-w", "-o", str(lib_path),
                           str(mutated), "-lm"])
    good = orc.lib()
    bad = C.CDLL(str(lib_path))
    bad.orc_belady_misses.restype = C.c_int64
    bad.orc_lru_misses.restype = C.c_int64
    bad.orc_cumsum_threshold.restype = C.c_int
    orc._lib = bad
    try:
        failed = run_pins()
    finally:
        orc._lib = good
    assert failed, "no pin noticed: " + what
