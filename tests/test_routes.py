"""Route-table helper: the oracle against the weights, budgets, coverage and
sparsity the paper prints, and the library's host function against the oracle."""
import os

import numpy as np

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import binding

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "contribution_weights.txt")


def load():
    w, budgets = {}, {}
    for line in open(GOLDEN):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "budget":
            budgets[f[1]] = (int(f[2]), int(f[3]), float(f[4]), float(f[5]), float(f[6]))
        else:
            w.setdefault((f[0], f[1]), {})[int(f[2])] = float(f[3])
    return w, budgets


def arrays(w, model):
    lay, grp = w[(model, "layer")], w[(model, "group")]
    return np.array([lay[i + 1] for i in range(len(lay))]), np.array([grp[i + 1] for i in range(len(grp))])


def test_oracle_reproduces_the_printed_budgets():
    w, budgets = load()
    for model, n_layers in (("Ql", 36), ("Qs", 28)):
        sl, sg = arrays(w, model)
        assert len(sl) == n_layers and len(sg) == 8
        kl, kg, ccl, ccg, rho = budgets[model]
        omega, keep_l, keep_g, cl, cg = orc.routes_from_contributions(sl, sg, kl, kg)
        # the kept units are the table's first K rows (the file lists units in rank order)
        rank_l = list(w[(model, "layer")].keys()); rank_g = list(w[(model, "group")].keys())
        assert sorted(i + 1 for i in keep_l) == sorted(rank_l[:kl])
        assert sorted(i + 1 for i in keep_g) == sorted(rank_g[:kg])
        assert abs(100 * cl - ccl) < 0.15 and abs(100 * cg - ccg) < 0.15       # printed weights are rounded to 0.01
        assert int(omega.sum()) == kl * kg
        assert round(100 * orc.structural_sparsity(kl, kg, n_layers, 8), 1) == rho
        assert round(100 * (1 - omega.mean()), 1) == rho
    # zero-weight units appear in the table in increasing index order: ties go to the lower index
    sl, sg = arrays(w, "Ql")
    _, keep_all, _, _, _ = orc.routes_from_contributions(sl, sg, 36, 8)
    assert [i + 1 for i in keep_all[-7:]] == [1, 2, 4, 6, 7, 26, 29]


def test_library_matches_oracle_including_ties_and_negative_scores():
    rng = np.random.default_rng(0)
    for trial in range(50):
        nl, ng = int(rng.integers(1, 40)), int(rng.integers(1, 9))
        sl = np.round(rng.normal(0.2, 1.0, nl), 1)       # coarse rounding: many ties, many negatives
        sg = np.round(rng.normal(0.5, 1.0, ng), 1)
        kl, kg = int(rng.integers(0, nl + 1)), int(rng.integers(0, ng + 1))
        omega, ccl, ccg, rho = binding.build_routes(sl, sg, kl, kg)
        want, _, _, wl_, wg_ = orc.routes_from_contributions(sl, sg, kl, kg)
        assert np.array_equal(omega, want)
        assert abs(ccl - wl_) < 1e-12 and abs(ccg - wg_) < 1e-12
        assert abs(rho - orc.structural_sparsity(kl, kg, nl, ng)) < 1e-15
