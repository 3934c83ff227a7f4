"""The extremes of the worker axis and of the launch geometry: one worker, the largest number of workers the
library accepts, and a K x P too large for one grid, which must be refused before anything is launched."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2006_00441_b200 import inputs
from tests.harness import TOL_RUN, assert_close, make_pair, padded_grad, state_of, to_oracle_grad

pytestmark = pytest.mark.gpu
FUSE_MERGE, ROTATE, INLINE, LANES = 0x4, 0x8, 0x10, 0x100


@pytest.fixture(scope="module")
def B():
    from paper_2006_00441_b200 import binding
    return binding


@pytest.mark.parametrize("flags,n_chunks", [(0, 0), (ROTATE | FUSE_MERGE, 0), (INLINE, 0)])
@pytest.mark.parametrize("dtype", [0, 1])
def test_largest_number_of_workers(B, flags, n_chunks, dtype):
    """K = 65535 (the limit: the scalar kernels put the worker index in gridDim.y).  Thirteen columns, so that
    both the vector path and the one-column ragged end run; the mean adds 65535 terms per column."""
    K, P, tau, d, T = 65535, 13, 2, 1, 6
    ld = 16
    w0 = inputs.shared_start(90, P, 0.02).numpy()
    gpu, cpu = make_pair(B, K, P, tau, d, 0.25, 0.9, 1e-4, dtype=dtype, flags=flags, ld=ld, w0=w0, n_chunks=n_chunks)
    gd = torch.bfloat16 if dtype else torch.float32
    r = np.random.default_rng(91)      # the seeded generator of the other tests walks the rows one by one: too slow here
    for t in range(T):
        g = padded_grad(torch.from_numpy((0.0316 * r.standard_normal((K, P))).astype(np.float32)).to(gd), ld)
        gpu.step(g, 0.1); cpu.step(to_oracle_grad(g, P), 0.1)
    w, m = state_of(gpu)
    assert_close(w, cpu.w, TOL_RUN, "w"); assert_close(m, cpu.m, TOL_RUN, "m")
    for i in range(cpu.n_pending):
        assert_close(gpu.pending_mean(i).cpu().numpy(), cpu.pending(i)[2], TOL_RUN, "pending mean")
    with pytest.raises(B.DasgdError) as e:
        B.DaSGD(K + 1, P, tau, d, 0.25)
    assert e.value.status == B.DASGD_ERR_INVALID_ARG


@pytest.mark.parametrize("tau,d", [(1, 1), (2, 0), (1, 2)])
def test_a_single_worker_is_its_own_mean(B, tau, d):
    """K = 1: the mean of one worker is that worker's snapshot, so the merge blends the weights with their own
    earlier value."""
    K, P, T = 1, 4096 + 9, 10
    ld = (P + 7) // 8 * 8
    w0 = inputs.shared_start(92, P, 0.02).numpy()
    for flags, n_chunks in [(0, 0), (ROTATE | FUSE_MERGE | LANES, 2), (INLINE, 0)]:
        if n_chunks and d < 1:
            continue
        gpu, cpu = make_pair(B, K, P, tau, d, 0.25, 0.9, 0.0, flags=flags, ld=ld, w0=w0, n_chunks=n_chunks)
        for t in range(T):
            g = padded_grad(inputs.grad_block(93, t, K, P, 0.0316), ld)
            gpu.step(g, 0.1); cpu.step(to_oracle_grad(g, P), 0.1)
        w, m = state_of(gpu)
        assert_close(w, cpu.w, TOL_RUN, "w"); assert_close(m, cpu.m, TOL_RUN, "m")
        for i in range(cpu.n_pending):
            s, snap, mean = cpu.pending(i)
            np.testing.assert_array_equal(mean, snap[0])
            assert_close(gpu.pending_mean(i).cpu().numpy(), mean, TOL_RUN, "pending mean")


def test_a_grid_beyond_the_launch_limit_is_refused_before_any_launch(B):
    """K * ceil(P / 4096) must fit the x dimension of one grid (2^31 - 1 thread blocks).  A configuration beyond
    that is accepted by dasgd_init (which cannot know how much memory stands behind the pointers) and refused by
    the first call that would launch, with DASGD_ERR_UNSUPPORTED and without touching the GPU: the buffers given
    here are far smaller than the claimed shape, so a launch would be out of bounds, and the launch counter must
    stay at zero."""
    K, P = 65535, 4096 * 40000          # 65535 * 40000 tiles = 2.6e9 > 2^31 - 1
    small = torch.zeros(1 << 16, device="cuda")
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    cfg = B.dasgd_config()
    cfg.K, cfg.tau, cfg.d, cfg.dtype, cfg.merge_mode, cfg.n_slots, cfg.flags, cfg.device = K, 1, 1, 0, 0, 1, 0, 0
    cfg.P, cfg.ld, cfg.xi, cfg.momentum, cfg.weight_decay = P, P, 0.25, 0.0, 0.0
    cfg.w = cfg.snap = cfg.mean = small.data_ptr()
    cfg.main_stream, cfg.side_stream = main.cuda_stream, side.cuda_stream
    ctx = B.dasgd_init(cfg)
    try:
        with pytest.raises(B.DasgdError) as e:
            B.dasgd_local_step(ctx, small.data_ptr(), 0.1)
        assert e.value.status == B.DASGD_ERR_UNSUPPORTED and "too large" in str(e.value)
        with pytest.raises(B.DasgdError) as e:
            B.dasgd_step(ctx, small.data_ptr(), 0.1)
        assert e.value.status == B.DASGD_ERR_UNSUPPORTED
        with pytest.raises(B.DasgdError) as e:
            B.dasgd_snapshot(ctx)
        assert e.value.status == B.DASGD_ERR_UNSUPPORTED
        assert B.dasgd_get_launches(ctx) == 0
    finally:
        B.dasgd_destroy(ctx)
    torch.cuda.synchronize()
