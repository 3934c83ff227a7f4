"""The delay guideline (Eq. 3, Sections III-D, VI-C, VI-D) against the paper's own Table II."""
import os
import random

import pytest

import oracle
from paper_2006_00441_b200 import binding as B

HERE = os.path.dirname(os.path.abspath(__file__))


def table2():
    rows = []
    for line in open(os.path.join(HERE, "golden", "table2_delay.txt")):
        line = line.split("#")[0].split()
        if line:
            rows.append((line[0], line[1], float(line[2]), float(line[3]), float(line[4]), int(line[5]), int(line[6])))
    assert len(rows) == 14
    return rows


@pytest.mark.parametrize("row", table2(), ids=lambda r: f"{r[0]}-{r[1]}")
def test_oracle_reproduces_table2(row):
    _, _, t_p, t_c_tree, _, d, tau = row
    assert oracle.delay_guideline(t_c_tree, t_p) == (d, tau)


@pytest.mark.parametrize("row", table2(), ids=lambda r: f"{r[0]}-{r[1]}")
def test_library_reproduces_table2(row):
    _, _, t_p, t_c_tree, _, d, tau = row
    assert B.dasgd_delay_guideline(t_c_tree, t_p) == (d, tau)


def test_library_equals_oracle_and_satisfies_the_inequality():
    r = random.Random(0)
    cases = [(0.0, 1.0), (1.0, 1.0), (0.999999, 1.0), (2.0, 1.0), (7.0, 0.5), (1e-9, 3.0), (123456.7, 0.01)]
    cases += [(r.uniform(0, 50), r.uniform(0.01, 10)) for _ in range(500)]
    for t_c, t_p in cases:
        d, tau = B.dasgd_delay_guideline(t_c, t_p)
        assert (d, tau) == oracle.delay_guideline(t_c, t_p)
        assert d >= 1 and tau == d + 1
        assert t_c < d * t_p and (d == 1 or not t_c < (d - 1) * t_p)   # smallest d that hides the averaging


def test_from_system_parameters():
    # t_c = m*n_p/BW, t_p = B_l*FLOP/FLOPS (Eq. 3): 256 workers, 25.5M parameters ...
    d, tau = oracle.delay_from_system(m=256, n_p=25.5e6, BW=2.5e9, B_l=64, FLOP=8e9, FLOPS=6e12)
    t_c, t_p = 256 * 25.5e6 / 2.5e9, 64 * 8e9 / 6e12
    assert (d, tau) == oracle.delay_guideline(t_c, t_p)


def test_bad_arguments():
    with pytest.raises(B.DasgdError):
        B.dasgd_delay_guideline(1.0, 0.0)
    with pytest.raises(B.DasgdError):
        B.dasgd_delay_guideline(-1.0, 1.0)
    with pytest.raises(oracle.OracleError):
        oracle.delay_guideline(1.0, 0.0)


@pytest.mark.gpu
def test_advise_delay_from_measured_kernels():
    import torch
    K, P = 8, 1 << 20
    gpu = B.DaSGD(K, P, 2, 1, 0.25, 0.9, flags=B.DASGD_FLAG_TIMING)
    g = torch.zeros(K, P, device="cuda")
    with pytest.raises(B.DasgdError):
        gpu.advise_delay()                       # nothing timed yet
    for _ in range(12):
        gpu.step(g, 0.1)
    d, tau, t_c, t_p = gpu.advise_delay()
    assert t_c > 0 and t_p > 0 and tau == d + 1
    assert (d, tau) == oracle.delay_guideline(t_c, t_p)
    # a long forward/backward makes one step of delay enough
    assert gpu.advise_delay(extra_tp_ms=1000.0)[0] == 1
