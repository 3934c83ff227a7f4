"""Reader for the hand-worked trajectory fixtures under tests/golden/."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def load(name):
    cfg, w0, g, exp_w, exp_m, exp_mean = {}, {}, {}, {}, {}, {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].split()
            if not line:
                continue
            key, rest = line[0], line[1:]
            if key in ("K", "P", "tau", "d", "merge_mode", "average_momentum"):
                cfg[key] = int(rest[0])
            elif key in ("xi", "lr", "momentum", "weight_decay"):
                cfg[key] = float(rest[0])
            elif key == "w0":
                w0[int(rest[0])] = [float(v) for v in rest[1:]]
            elif key == "g":
                g[(int(rest[0]), int(rest[1]))] = [float(v) for v in rest[2:]]
            elif key == "expect_w":
                exp_w[(int(rest[0]), int(rest[1]))] = [float(v) for v in rest[2:]]
            elif key == "expect_m":
                exp_m[(int(rest[0]), int(rest[1]))] = [float(v) for v in rest[2:]]
            elif key == "expect_mean_m":     # mean of the momentum buffers of the snapshot taken at that step
                cfg.setdefault("expect_mean_m", {})[int(rest[0])] = [float(v) for v in rest[1:]]
            elif key == "expect_mean":
                exp_mean[int(rest[0])] = [float(v) for v in rest[1:]]
            else:
                raise ValueError(f"{name}: unknown key {key}")
    K, P = cfg["K"], cfg["P"]
    T = 1 + max(t for t, _ in g)
    W0 = np.array([w0[k] for k in range(K)], np.float32)
    G = np.array([[g[(t, k)] for k in range(K)] for t in range(T)], np.float32)
    assert W0.shape == (K, P) and G.shape == (T, K, P)
    return cfg, W0, G, exp_w, exp_m, exp_mean
