"""Re-derives the numbers in hand_cases.json from their closed forms.

Uses only Python's math module: neither the oracle nor the CUDA path is involved.
Run `python tests/golden/make_golden.py` to print the values and compare them with
the stored file (it does not rewrite the file).
"""
import json
import os
from math import exp, log, pi, sqrt

ln2, ln3 = log(2.0), log(3.0)
dy8 = [1 / 2, 1 / 4, 1 / 8, 1 / 16, 1 / 32, 1 / 64, 1 / 128, 1 / 128]
s_half = sum(sqrt(x) for x in dy8)
s_sq = sum(x * x for x in dy8)
h = 0.2 * 2.25 ** (-0.2)
norm = 3.0 * h * sqrt(2.0 * pi)
VALUES = {
    "entropy_dyadic": {"H": 1.75 * ln2},
    "entropy_of_softmax_log1234": {"lse": log(10.0),
                                   "H": log(10.0) - (0.2 * ln2 + 0.3 * ln3 + 0.4 * log(4.0))},
    "kl_ce_dyadic_vs_uniform": {"CE": 2.0 * ln2, "KL": 0.25 * ln2},
    "jsd_half_vs_onehot": {"JSD": 1.5 * ln2 - 0.75 * ln3,
                           "d": sqrt((1.5 * ln2 - 0.75 * ln3) / ln2)},
    "jsd_dyadic_vs_uniform": {"JSD": 0.5 * log(4.0 / 3.0) + 0.25 * log(2.0 / 3.0)},
    "jsd_disjoint": {"JSD": ln2, "d": 1.0},
    "kde_three_point": {"std": 0.2, "h_silverman": h, "h_scott": 0.2 * 3.0 ** (-0.2),
                        "f_0.4": (1.0 + 2.0 * exp(-0.5 * (0.2 / h) ** 2)) / norm,
                        "f_0.2": (1.0 + exp(-0.5 * (0.2 / h) ** 2) + exp(-0.5 * (0.4 / h) ** 2)) / norm},
    "warp_dyadic_v8": {"t2_p0": sqrt(0.5) / s_half, "t2_p7": sqrt(1 / 128) / s_half,
                       "thalf_p0": 0.25 / s_sq, "thalf_p1": (1 / 16) / s_sq,
                       "topk3_H": log(7.0) - (10.0 / 7.0) * ln2, "topk3_lse": log(7.0 / 8.0),
                       "topp08_margin": 0.05,
                       "topp074_H": ln3 - (2.0 / 3.0) * ln2, "topp074_lse": log(0.75)},
}

if __name__ == "__main__":
    here = os.path.dirname(os.path.abspath(__file__))
    stored = {c["name"]: c["expect"] for c in json.load(open(os.path.join(here, "hand_cases.json")))["cases"]}
    worst = 0.0
    for name, vals in VALUES.items():
        for k, v in vals.items():
            diff = abs(stored[name][k] - v)
            worst = max(worst, diff)
            print(f"{name:32s} {k:12s} {v!r:24} stored {stored[name][k]!r} diff {diff:.2e}")
    print("worst difference", worst)
