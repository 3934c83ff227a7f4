"""The oracle against hand-worked trajectories derived from Eq. 2 (tests/golden/)."""
import numpy as np
import pytest

from oracle import OracleDaSGD
from tests.golden_io import load

CASES = ["w1_xi_blend.txt", "w2_momentum.txt", "w3_d_equals_tau.txt", "w4_delta_merge.txt",
         "w1_stacked_p8.txt", "w5_momentum_averaging.txt"]


@pytest.mark.parametrize("name", CASES)
def test_golden_trajectory(name):
    cfg, W0, G, exp_w, exp_m, exp_mean = load(name)
    o = OracleDaSGD(cfg["K"], cfg["P"], cfg["tau"], cfg["d"], cfg["xi"], cfg["momentum"],
                    cfg["weight_decay"], merge_mode=cfg["merge_mode"], average_momentum=bool(cfg.get("average_momentum")))
    o.set_state(W0)
    exp_mean_m = cfg.get("expect_mean_m", {})
    seen_w = seen_m = seen_mean = 0
    for t in range(G.shape[0]):
        o.step(G[t], cfg["lr"])
        u = t + 1
        w, m = o.w, o.m
        for k in range(cfg["K"]):
            if (u, k) in exp_w:
                np.testing.assert_array_equal(w[k], np.array(exp_w[(u, k)], np.float32), err_msg=f"w u={u} k={k}")
                seen_w += 1
            if (u, k) in exp_m:
                np.testing.assert_array_equal(m[k], np.array(exp_m[(u, k)], np.float32), err_msg=f"m u={u} k={k}")
                seen_m += 1
        if u in exp_mean:
            # the snapshot taken at u is the newest pending one
            s, _, mean = o.pending(o.n_pending - 1)
            assert s == u
            np.testing.assert_array_equal(mean, np.array(exp_mean[u], np.float32), err_msg=f"mean s={u}")
            seen_mean += 1
        if u in exp_mean_m:
            _, mean_m = o.pending_momentum(o.n_pending - 1)
            np.testing.assert_array_equal(mean_m, np.array(exp_mean_m[u], np.float32), err_msg=f"mean of m s={u}")
            seen_mean += 1
    assert seen_w == len(exp_w) and seen_m == len(exp_m) and seen_mean == len(exp_mean) + len(exp_mean_m)
