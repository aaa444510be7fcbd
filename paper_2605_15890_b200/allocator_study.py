"""Allocator comparison of Sec. VI (the setting of the paper's Fig. 2) on synthetic straggler
probabilities: mean objective F(r) of problem (b-SP1) for Algorithm 1, the exact DP, the greedy
and the continuous-relaxation heuristics and the concave-envelope upper bound, for residual
budgets Z_res = n, 2n, .., 5n at n = 10 and 50 workers, averaged over seeds, with and without the
error-balance factor of Sec. V-B. All allocators are the library's host routines.

    python -m paper_2605_15890_b200.allocator_study [--seeds 50] [--dim 512] [--markdown]
"""
import argparse

import numpy as np

from . import binding as B


def shifted_exponential_probs(n, seed, psi_range=(0.1, 2.0), tau_th=1.1):
    """Sec. V-A / VI: p_i = exp(-psi_i (tau_th - 1)), psi_i uniform on psi_range."""
    rng = np.random.default_rng(np.random.SeedSequence([int(seed), 21]))
    psi = rng.uniform(psi_range[0], psi_range[1], n)
    return np.exp(-psi * (tau_th - 1.0))


def study(ns=(10, 50), multiples=(1, 2, 3, 4, 5), seeds=50, dim=512.0, b_max=0, with_eta=False):
    rows = []
    for n in ns:
        for mult in multiples:
            z_tot = 2 * n + mult * n
            acc = {"alg1": 0.0, "dp": 0.0, "greedy": 0.0, "relaxation": 0.0, "bound": 0.0}
            worst = 1.0
            for seed in range(seeds):
                p = shifted_exponential_probs(n, seed)
                eta = B.agc_eta_balance(p, z_tot, dim) if with_eta else 1.0
                f_dp = B.agc_bit_allocate_dp(p, z_tot, b_max=b_max, phi_dim=dim, eta=eta)[1]
                f_a = B.agc_bit_allocate(p, z_tot, b_max=b_max, phi_dim=dim, eta=eta)[1]
                acc["dp"] += f_dp
                acc["alg1"] += f_a
                acc["greedy"] += B.agc_bit_allocate_heuristic(B.AGC_ALLOC_GREEDY, p, z_tot, b_max=b_max, phi_dim=dim, eta=eta)[1]
                acc["relaxation"] += B.agc_bit_allocate_heuristic(B.AGC_ALLOC_RELAXATION, p, z_tot, b_max=b_max, phi_dim=dim,
                                                                  eta=eta)[1]
                acc["bound"] += B.agc_allocation_upper_bound(p, z_tot, b_max=b_max, phi_dim=dim, eta=eta)
                worst = min(worst, f_a / f_dp)
            row = {"n": n, "z_res": mult * n, "eta": bool(with_eta), "alg1_min_ratio": worst}
            row.update({k: v / seeds for k, v in acc.items()})
            rows.append(row)
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--seeds", type=int, default=50)
    ap.add_argument("--dim", type=float, default=512.0)
    ap.add_argument("--markdown", action="store_true")
    args = ap.parse_args()
    sep = " | " if args.markdown else "  "
    head = ["n", "Z_res", "eta", "Alg. 1", "DP", "greedy", "relaxation", "bound", "min Alg.1/DP"]
    print(("| " if args.markdown else "") + sep.join(head) + (" |" if args.markdown else ""))
    if args.markdown:
        print("|" + "---|" * len(head))
    for with_eta in (False, True):
        for r in study(seeds=args.seeds, dim=args.dim, with_eta=with_eta):
            cells = [str(r["n"]), str(r["z_res"]), "balanced" if r["eta"] else "1", f"{r['alg1']:.4f}", f"{r['dp']:.4f}",
                     f"{r['greedy']:.4f}", f"{r['relaxation']:.4f}", f"{r['bound']:.4f}", f"{r['alg1_min_ratio']:.4f}"]
            print(("| " if args.markdown else "") + sep.join(cells) + (" |" if args.markdown else ""))


if __name__ == "__main__":
    main()
