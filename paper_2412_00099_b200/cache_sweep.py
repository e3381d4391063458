"""Miss rate against cache size for LRU with the original routing, Belady's optimal eviction on the same
trace, and Cache-Prior routing with an LRU cache (the comparison of the paper's cache-size ablation), on one
of the synthetic workloads.  Routing only (no expert FFN); everything runs in the library's kernels.

    python -m paper_2412_00099_b200.cache_sweep --workload qwen --tokens 256
"""
from __future__ import annotations

import argparse

import torch

from . import binding as mb
from . import synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="qwen", choices=sorted(synth.ALIASES))
    ap.add_argument("--tokens", type=int, default=256)
    ap.add_argument("--lams", type=float, nargs="*", default=[0.25, 0.5, 1.0])
    args = ap.parse_args()
    wl = synth.ALIASES[args.workload]
    dev = torch.device("cuda")
    T = args.tokens
    dt = torch.bfloat16 if wl.bf16 else torch.float32
    Wr = mb.gen_normal(torch.empty((wl.L, wl.E, wl.d), dtype=torch.float32, device=dev), wl.seed, synth.T_ROUTER,
                       std=wl.weight_std)
    hidden = torch.empty((T, wl.L, wl.S, wl.d), dtype=dt, device=dev)
    state = torch.empty(wl.L * wl.S * wl.d, dtype=torch.float32, device=dev)
    for t in range(T):
        mb.gen_hidden_step(state, hidden[t], wl.seed, t, wl.rho, wl.topic_offset)
    caps = sorted({c for c in (wl.K, wl.E // 8, wl.E // 4, wl.E // 2, 3 * wl.E // 4, wl.E) if c >= wl.K})

    def run(C, lam):
        eng = mb.engine_for(wl.with_(C=C, lam=lam), ffn_impl=mb.FFN_SIMT)
        eng.set_router(Wr)
        sel, _ = eng.route_step(hidden=hidden, n_steps=T)
        total, _ = eng.cache_stats()
        eng.close()
        return sel, total[2] / total[1]

    sel0, _ = run(caps[0], 0.0)                       # the original routing does not depend on the cache
    belady = mb.belady_replay(sel0, wl.E, caps).sum(dim=(1, 2)).cpu().numpy() / (T * wl.L * wl.S * wl.K)
    print("%s, %d tokens x %d streams x %d layers, K = %d, J = %d" % (wl.name, T, wl.S, wl.L, wl.K, wl.J))
    print("| cache size | LRU, original routing | Belady (optimal eviction), original routing | "
          + " | ".join("Cache-Prior λ=%g + LRU" % l for l in args.lams) + " |")
    print("|---|---|---|" + "---|" * len(args.lams))
    for ci, C in enumerate(caps):
        lru = run(C, 0.0)[1]
        prior = [run(C, lam)[1] for lam in args.lams]
        print("| %d / %d | %.2f %% | %.2f %% | " % (C, wl.E, 100 * lru, 100 * belady[ci])
              + " | ".join("%.2f %%" % (100 * p) for p in prior) + " |")


if __name__ == "__main__":
    main()
