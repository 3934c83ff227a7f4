"""Momentum averaging (the variant in which the momentum buffers are snapshotted, averaged and blended like the
weights) through the C ABI against the CPU oracle, across schedules of dasgd_step and the explicit calls."""
import numpy as np
import pytest
import torch

from oracle import OracleDaSGD
from paper_2006_00441_b200 import inputs
from tests.harness import TOL_RUN, TOL_STEP, assert_close, bf16_bits, padded_grad, state_of, to_oracle_grad

pytestmark = pytest.mark.gpu

FUSE_SNAP, FUSE_MERGE, ROTATE, INLINE, FUSE_D1, LANES, GRAPH = 0x2, 0x4, 0x8, 0x10, 0x80, 0x100, 0x200
SCHEDS = [(0, 0), (FUSE_SNAP | FUSE_MERGE, 0), (ROTATE, 0), (ROTATE | FUSE_MERGE, 0), (ROTATE | FUSE_MERGE | FUSE_D1, 0),
          (ROTATE | FUSE_MERGE, 3), (ROTATE | FUSE_MERGE | LANES, 2), (ROTATE | FUSE_MERGE | LANES | GRAPH, 3),
          (ROTATE | FUSE_MERGE | LANES | 0x400, 3)]
SCHEDULES = [(1, 1), (2, 1), (1, 2), (2, 2), (3, 2), (2, 3), (3, 0), (1, 0)]


@pytest.fixture(scope="module")
def B():
    from paper_2006_00441_b200 import binding
    return binding


def pair(B, K, P, tau, d, xi, mu, wd, dtype, mode, flags, ld, n_chunks, w0):
    gpu = B.DaSGD(K, P, tau, d, xi, mu, wd, dtype=dtype, merge_mode=mode, flags=flags, ld=ld, n_chunks=n_chunks,
                  average_momentum=True)
    cpu = OracleDaSGD(K, P, tau, d, xi, mu, wd, dtype=dtype, merge_mode=mode, average_momentum=True)
    gpu.set_state(torch.from_numpy(w0)); cpu.set_state(w0)
    return gpu, cpu


@pytest.mark.parametrize("tau,d", SCHEDULES)
@pytest.mark.parametrize("K,dtype,mode", [(4, 0, 0), (3, 1, 0), (5, 0, 1), (2, 1, 1)])
def test_free_running_against_the_oracle_and_bit_identical_across_schedules(B, tau, d, K, dtype, mode):
    P, T = 2 * 4096 + 77, 60
    ld = (P + 7) // 8 * 8
    w0 = inputs.shared_start(80, P, 0.02).numpy()
    gd = torch.bfloat16 if dtype else torch.float32
    G = [padded_grad(inputs.grad_block(81, t, K, P, 0.0316, dtype=gd), ld) for t in range(T)]
    first = None
    for flags, n_chunks in SCHEDS:
        if n_chunks and d < 1:
            continue
        gpu, cpu = pair(B, K, P, tau, d, 0.25, 0.9, 1e-4, dtype, mode, flags, ld, n_chunks, w0)
        for t in range(T):
            gpu.step(G[t], 0.1)
            if first is None:
                cpu.step(to_oracle_grad(G[t], P), 0.1)
        w, m = state_of(gpu)
        if first is None:
            assert gpu.n_pending == cpu.n_pending
            assert_close(w, cpu.w, TOL_RUN, "w"); assert_close(m, cpu.m, TOL_RUN, "m")
            moved = OracleDaSGD(K, P, tau, d, 0.25, 0.9, 1e-4, dtype=dtype, merge_mode=mode)   # the run without the variant
            moved.set_state(w0)
            for t in range(T):
                moved.step(to_oracle_grad(G[t], P), 0.1)
            assert np.abs(moved.m - cpu.m).max() > 1e-4         # the variant does change the buffers
            for i in range(cpu.n_pending):
                _, mean_m = cpu.pending_momentum(i)
                assert_close(gpu.pending_momentum_mean(i).cpu().numpy(), mean_m, TOL_RUN, f"pending mean of m {i}")
            first = (w, m)
        else:
            np.testing.assert_array_equal(w, first[0], err_msg=str((flags, n_chunks)))
            np.testing.assert_array_equal(m, first[1], err_msg=str((flags, n_chunks)))
        if dtype:
            np.testing.assert_array_equal(bf16_bits(gpu.w_lp[:, :P]), bf16_bits(gpu.w[:, :P].to(torch.bfloat16)))
        gpu.close()


@pytest.mark.parametrize("P", [5, 1000, 4096 + 3, 3 * 4096 + 1029])
@pytest.mark.parametrize("mode,xi", [(0, 0.25), (0, 0.0), (0, 1.0), (1, 0.25)])
def test_explicit_calls_teacher_forced(B, P, mode, xi):
    """snapshot / average / local steps / merge spelled out, the GPU restarted from the oracle's state before every
    operation that is compared at the one-step tolerance."""
    K, tau, d = 3, 4, 2
    ld = P if P % 8 == 0 or P < 8 else (P + 7) // 8 * 8
    r = np.random.default_rng(82)
    w0 = r.standard_normal((K, P)).astype(np.float32)
    m0 = r.standard_normal((K, P)).astype(np.float32)
    gpu = B.DaSGD(K, P, tau, d, xi, 0.9, 0.0, merge_mode=mode, ld=ld, average_momentum=True)
    cpu = OracleDaSGD(K, P, tau, d, xi, 0.9, 0.0, merge_mode=mode, average_momentum=True)
    gpu.set_state(torch.from_numpy(w0), torch.from_numpy(m0)); cpu.set_state(w0, m0)
    gpu.snapshot(); gpu.average_async()
    cpu.snapshot(); cpu.average()
    snap_m, mean_m = cpu.pending_momentum(0)
    gpu.sync()
    assert_close(gpu.pending_momentum_mean(0).cpu().numpy(), mean_m, TOL_STEP, "mean of m")
    for t in range(d):
        g = padded_grad(inputs.grad_block(83, t, K, P, 0.3), ld)
        gpu.local_step(g, 0.1); cpu.local_step(to_oracle_grad(g, P), 0.1)
    gpu.set_state(torch.from_numpy(cpu.w), torch.from_numpy(cpu.m))    # teacher forcing: merge from the oracle's state
    gpu.merge(); cpu.merge()
    w, m = state_of(gpu)
    assert_close(w, cpu.w, TOL_STEP, "w after merge"); assert_close(m, cpu.m, TOL_STEP, "m after merge")
    if xi == 1.0 and mode == 0:
        np.testing.assert_array_equal(m, cpu.m)


def test_refused_combinations(B):
    with pytest.raises(B.DasgdError) as e:
        B.DaSGD(2, 64, 1, 1, 0.5, 0.0, average_momentum=True)
    assert e.value.status == B.DASGD_ERR_INVALID_ARG
    with pytest.raises(B.DasgdError) as e:
        B.DaSGD(2, 64, 1, 1, 0.5, 0.9, flags=INLINE, average_momentum=True)
    assert e.value.status == B.DASGD_ERR_UNSUPPORTED
    gpu = B.DaSGD(2, 64, 1, 1, 0.5, 0.9, average_momentum=True)
    with pytest.raises(B.DasgdError) as e:
        gpu.set_shard(4, exchange=lambda *a: None)
    assert e.value.status == B.DASGD_ERR_UNSUPPORTED
    g = torch.zeros(2, 64, device="cuda")
    gpu.step(g, 0.1)
    with pytest.raises(B.DasgdError) as e:       # only before first use
        B.dasgd_set_momentum_averaging(gpu.ctx, gpu.m_snap.data_ptr(), gpu.m_mean.data_ptr())
    assert e.value.status == B.DASGD_ERR_BAD_STATE
