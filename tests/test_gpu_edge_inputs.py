"""Inputs outside the comfortable range: weights of magnitude 1e3, denormal gradients, and gradients that
hold NaN and +/-Inf.  Plain arithmetic on both sides (nothing here can fault): non-finite values must appear
at exactly the same elements with the same kind (NaN, +Inf, -Inf), finite ones must agree within tolerance."""
import numpy as np
import pytest
import torch

from paper_2006_00441_b200 import inputs
from tests.harness import TOL_RUN, TOL_STEP, make_pair, padded_grad, to_oracle_grad

pytestmark = pytest.mark.gpu
FUSE_SNAP, FUSE_MERGE, ROTATE, INLINE, LANES, FUSE_D1 = 0x2, 0x4, 0x8, 0x10, 0x100, 0x80
SCHEDS = [(0, 0), (ROTATE | FUSE_MERGE | LANES | 0x400, 3), (ROTATE | FUSE_MERGE | FUSE_D1, 0), (FUSE_SNAP | FUSE_MERGE, 0), (INLINE, 0)]


@pytest.fixture(scope="module")
def B():
    from paper_2006_00441_b200 import binding
    return binding


def assert_same_kind_and_close(gpu, cpu, tol, what):
    gpu, cpu = np.asarray(gpu, np.float64), np.asarray(cpu, np.float64)
    assert gpu.shape == cpu.shape
    assert np.array_equal(np.isnan(gpu), np.isnan(cpu)), f"{what}: NaN at different elements"
    assert np.array_equal(np.isposinf(gpu), np.isposinf(cpu)), f"{what}: +Inf at different elements"
    assert np.array_equal(np.isneginf(gpu), np.isneginf(cpu)), f"{what}: -Inf at different elements"
    f = np.isfinite(cpu)
    err = np.abs(gpu[f] - cpu[f]) / (1.0 + np.abs(cpu[f]))
    assert err.size == 0 or err.max() <= tol, f"{what}: max scaled error {err.max():.3e} > {tol:.1e}"


def state(gpu):
    gpu.sync()
    P = gpu.P
    return gpu.w[:, :P].cpu().numpy(), (gpu.m[:, :P].cpu().numpy() if gpu.m is not None else None)


@pytest.mark.parametrize("flags,n_chunks", SCHEDS)
@pytest.mark.parametrize("K,dtype", [(4, 0), (33, 0), (3, 1)])
def test_large_weights(B, flags, n_chunks, K, dtype):
    """|w| ~ 1e3: the mean's float32 pairwise sum against the oracle's double sum, at the relative tolerance."""
    P, tau, d = 2 * 4096 + 45, 2, 1
    ld = (P + 7) // 8 * 8
    gd = torch.bfloat16 if dtype else torch.float32
    r = np.random.default_rng(K)
    w0 = (r.standard_normal((K, P)) * 1e3).astype(np.float32)
    gpu, cpu = make_pair(B, K, P, tau, d, 0.25, 0.9, 1e-4, dtype=dtype, flags=flags, ld=ld, w0=w0, n_chunks=n_chunks)
    for t in range(40):
        g = padded_grad(inputs.grad_block(300, t, K, P, 30.0, dtype=gd), ld)
        gpu.step(g, 0.1); cpu.step(to_oracle_grad(g, P), 0.1)
        if t == 0:
            w, m = state(gpu)
            assert_same_kind_and_close(w, cpu.w, TOL_STEP, "w after one step")
    w, m = state(gpu)
    assert np.abs(cpu.w).max() > 500
    assert_same_kind_and_close(w, cpu.w, TOL_RUN, "w"); assert_same_kind_and_close(m, cpu.m, TOL_RUN, "m")
    for i in range(cpu.n_pending):
        assert_same_kind_and_close(gpu.pending_mean(i).cpu().numpy(), cpu.pending(i)[2], TOL_RUN, f"mean {i}")


@pytest.mark.parametrize("flags,n_chunks", SCHEDS)
def test_denormal_gradients_and_weights(B, flags, n_chunks):
    """Gradients and weights around 1e-40 (float32 denormals): nothing is flushed to zero on either side."""
    K, P, tau, d = 4, 4096 + 29, 1, 1
    ld = (P + 7) // 8 * 8
    r = np.random.default_rng(11)
    w0 = (r.standard_normal((K, P)) * 1e-39).astype(np.float32)
    gpu, cpu = make_pair(B, K, P, tau, d, 0.5, 0.5, 0.0, flags=flags, ld=ld, w0=w0, n_chunks=n_chunks)
    ULP = 1.4012984643e-45                                 # spacing of float32 denormals
    for t in range(12):
        g = (r.standard_normal((K, P)) * 1e-40).astype(np.float32)
        assert (np.abs(g) < 1.2e-38).all() and (g != 0).any()
        gd = padded_grad(torch.from_numpy(g), ld)
        gpu.step(gd, 0.5); cpu.step(g, 0.5)
        if t == 0:     # one step from identical states: every stored value within two roundings of the oracle's
            w, m = state(gpu)
            assert np.abs(w.astype(np.float64) - cpu.w).max() <= 2 * ULP
            assert np.abs(m.astype(np.float64) - cpu.m).max() <= 2 * ULP
    w, m = state(gpu)
    assert (cpu.w != 0).mean() > 0.9                       # the run did not collapse to zeros
    # Absolute agreement to a few denormal spacings (1e-6*(1+|cpu|) would accept anything here).  Down there
    # every store rounds to a multiple of ULP, so twelve free-running steps may drift by a couple of dozen.
    assert np.abs(w.astype(np.float64) - cpu.w).max() <= 32 * ULP
    assert np.abs(m.astype(np.float64) - cpu.m).max() <= 32 * ULP


@pytest.mark.parametrize("flags,n_chunks", SCHEDS)
@pytest.mark.parametrize("dtype,mode,wd", [(0, 0, 1e-3), (0, 0, 0.0), (1, 0, 0.0), (0, 1, 1e-3)])
def test_nan_and_inf_gradients_propagate_identically(B, flags, n_chunks, dtype, mode, wd):
    if flags & INLINE and mode == 1:
        pytest.skip("the inline-mean schedule has no delta merge")
    K, P, tau, d = 5, 3 * 4096 + 17, 2, 1
    ld = (P + 7) // 8 * 8
    gd = torch.bfloat16 if dtype else torch.float32
    w0 = inputs.shared_start(5, P, 0.05).numpy()
    gpu, cpu = make_pair(B, K, P, tau, d, 0.25, 0.9, wd, dtype=dtype, merge_mode=mode, flags=flags, ld=ld, w0=w0, n_chunks=n_chunks)
    bad = {1: [(0, 3, np.nan), (2, 4096 + 5, np.inf), (4, P - 1, -np.inf)],
           4: [(1, 7, np.inf), (3, 7, -np.inf), (0, 2 * 4096, np.nan)],        # +Inf and -Inf in one column: the mean is NaN
           7: [(2, 4096 + 5, -np.inf)]}                                        # the opposite infinity where one already sits
    for t in range(14):
        g = inputs.grad_block(301, t, K, P, 0.05, dtype=gd)
        for k, p, v in bad.get(t, ()):
            g[k, p] = v
        g = padded_grad(g, ld)
        gpu.step(g, 0.1); cpu.step(to_oracle_grad(g, P), 0.1)
    w, m = state(gpu)
    assert np.isnan(cpu.w).any() and np.isfinite(cpu.w).mean() > 0.99
    assert_same_kind_and_close(w, cpu.w, TOL_RUN, "w"); assert_same_kind_and_close(m, cpu.m, TOL_RUN, "m")
    for i in range(cpu.n_pending):
        assert_same_kind_and_close(gpu.pending_mean(i).cpu().numpy(), cpu.pending(i)[2], TOL_RUN, f"mean {i}")
