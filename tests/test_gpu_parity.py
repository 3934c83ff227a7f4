"""libdasgd (through its C ABI) against the CPU oracle, element by element, on seeded inputs.

Tolerances (float32 path): per teacher-forced step |gpu-cpu| <= 1e-6*(1+|cpu|); after a free-running
run of 100 steps <= 1e-4*(1+|cpu|).  bf16 mode compares the float32 masters with the same bounds and
the bfloat16 copy bit for bit against the cast of the GPU's own master.
"""
import numpy as np
import pytest
import torch

from paper_2006_00441_b200 import inputs
from tests.harness import TOL_RUN, TOL_STEP, assert_close, bf16_bits, make_pair, padded_grad, state_of, to_oracle_grad

pytestmark = pytest.mark.gpu

FUSE_SNAP, FUSE_MERGE, ROTATE, INLINE = 0x2, 0x4, 0x8, 0x10
NESTEROV, DECOUPLED = 0x20, 0x40
FUSE_D1, LANES, GRAPH, SIDES = 0x80, 0x100, 0x200, 0x400
# schedules of dasgd_step: (flags, n_chunks).  The chunked pipeline applies to every d >= 1.
SCHEDS = [(0, 0), (FUSE_SNAP, 0), (FUSE_MERGE, 0), (FUSE_SNAP | FUSE_MERGE, 0), (ROTATE, 0), (ROTATE | FUSE_MERGE, 0),
          (ROTATE | FUSE_MERGE, 3), (ROTATE | FUSE_MERGE, 2), (ROTATE | FUSE_MERGE | LANES, 3), (ROTATE | FUSE_MERGE | LANES | GRAPH, 3), (ROTATE | FUSE_MERGE | GRAPH, 2),
          (ROTATE | FUSE_MERGE | LANES | SIDES, 3), (ROTATE | FUSE_MERGE | SIDES, 2),
          (ROTATE | FUSE_MERGE | FUSE_D1, 0), (FUSE_MERGE | FUSE_D1, 0),
          (INLINE, 0)]
# f32 vector tile = 256 threads * 4 units * 4 elements = 4096 elements; bf16 tile = 256*2*8 = 4096
SIZES = [1, 3, 4, 7, 8, 1000, 4096, 3 * 4096 + 1029]


@pytest.fixture(scope="module")
def B():
    from paper_2006_00441_b200 import binding
    return binding


def grads(seed, t, K, P, std, dtype, ld):
    g = inputs.grad_block(seed, t, K, P, std, dtype=dtype)
    return padded_grad(g, ld)


# ------------------------------------------------------------------ teacher-forced, one op at a time

@pytest.mark.parametrize("P", SIZES)
@pytest.mark.parametrize("K,dtype,mom,wd", [(3, 0, 0.9, 1e-2), (1, 0, 0.0, 0.0), (8, 0, 0.0, 1e-3), (4, 1, 0.9, 0.0),
                                            (5, 1, 0.0, 1e-2), (33, 0, 0.5, 0.0)])
def test_local_step_teacher_forced(B, P, K, dtype, mom, wd):
    ld = P if P % 8 == 0 or P < 8 else (P + 7) // 8 * 8
    w0 = inputs.shared_start(1, P, 0.5).numpy()
    gpu, cpu = make_pair(B, K, P, 4, 1, 0.25, mom, wd, dtype=dtype, ld=ld, w0=w0)
    gd = torch.bfloat16 if dtype else torch.float32
    for t in range(4):
        # teacher forcing: the GPU starts every step from the oracle's state
        gpu.set_state(torch.from_numpy(cpu.w), torch.from_numpy(cpu.m) if mom else None)
        g = grads(3, t, K, P, 0.3, gd, ld)
        gpu.local_step(g, 0.1)
        cpu.local_step(to_oracle_grad(g, P), 0.1)
        w, m = state_of(gpu)
        assert_close(w, cpu.w, TOL_STEP, f"w t={t}")
        if mom:
            assert_close(m, cpu.m, TOL_STEP, f"m t={t}")
        if dtype:
            np.testing.assert_array_equal(bf16_bits(gpu.w_lp[:, :P]), bf16_bits(gpu.w[:, :P].to(torch.bfloat16)))
        if ld > P:  # padding columns are never touched
            assert float(gpu.w[:, P:].abs().max()) == 0.0


@pytest.mark.parametrize("P", SIZES)
@pytest.mark.parametrize("K,dtype,mode", [(2, 0, 0), (3, 0, 0), (8, 0, 1), (32, 0, 0), (33, 0, 0), (4, 1, 0), (3, 1, 1)])
def test_snapshot_mean_merge_teacher_forced(B, P, K, dtype, mode):
    ld = P if P % 8 == 0 or P < 8 else (P + 7) // 8 * 8
    r = np.random.default_rng(P * 131 + K)
    W = r.standard_normal((K, P)).astype(np.float32)
    gpu, cpu = make_pair(B, K, P, 2, 1, 0.25, 0.0, 0.0, dtype=dtype, merge_mode=mode, ld=ld, w0=W)
    gd = torch.bfloat16 if dtype else torch.float32
    gpu.snapshot(); gpu.average_async()
    cpu.snapshot(); cpu.average()
    gpu.sync()
    s, snap, mean = cpu.pending(0)
    _, snap_ptr, _ = B.dasgd_get_pending(gpu.ctx, 0)
    assert snap_ptr == gpu.snap[0].data_ptr()
    np.testing.assert_array_equal(gpu.snap[0, :, :P].cpu().numpy(), snap)           # a copy is exact
    assert_close(gpu.pending_mean(0).cpu().numpy(), mean, TOL_STEP, "mean")
    # teacher forcing: hand the oracle's mean to the GPU before the merge
    gpu.mean[0, :P] = torch.from_numpy(mean).cuda()
    torch.cuda.synchronize()
    g = grads(5, 0, K, P, 0.3, gd, ld)
    gpu.local_step(g, 0.1); cpu.local_step(to_oracle_grad(g, P), 0.1)
    gpu.set_state(torch.from_numpy(cpu.w))
    gpu.merge(); cpu.merge()
    w, _ = state_of(gpu)
    assert_close(w, cpu.w, TOL_STEP, "merged w")
    if dtype:
        np.testing.assert_array_equal(bf16_bits(gpu.w_lp[:, :P]), bf16_bits(gpu.w[:, :P].to(torch.bfloat16)))
    assert gpu.n_pending == 0 and cpu.n_pending == 0


@pytest.mark.parametrize("variant", [NESTEROV, DECOUPLED, NESTEROV | DECOUPLED])
@pytest.mark.parametrize("sched", [0, ROTATE | FUSE_MERGE, INLINE])
@pytest.mark.parametrize("dtype,P", [(0, 4096 + 7), (1, 2 * 4096 + 9), (0, 5)])
def test_local_step_variants(B, variant, sched, dtype, P):
    """Nesterov momentum and decoupled weight decay: one teacher-forced step at 1e-6, then 60 free steps."""
    K, ld = 3, (P + 7) // 8 * 8
    gd = torch.bfloat16 if dtype else torch.float32
    w0 = inputs.shared_start(50, P, 0.5).numpy()
    gpu, cpu = make_pair(B, K, P, 2, 2, 0.25, 0.9, 0.05, dtype=dtype, flags=variant | sched, ld=ld, w0=w0)
    g = grads(51, 0, K, P, 0.3, gd, ld)
    gpu.local_step(g, 0.1); cpu.local_step(to_oracle_grad(g, P), 0.1)
    w, m = state_of(gpu)
    assert_close(w, cpu.w, TOL_STEP, "w after one step"); assert_close(m, cpu.m, TOL_STEP, "m after one step")
    gpu2, cpu2 = make_pair(B, K, P, 2, 2, 0.25, 0.9, 0.05, dtype=dtype, flags=variant | sched, ld=ld, w0=w0)
    for t in range(60):
        g = grads(52, t, K, P, 0.1, gd, ld)
        gpu2.step(g, 0.05); cpu2.step(to_oracle_grad(g, P), 0.05)
    w, m = state_of(gpu2)
    assert_close(w, cpu2.w, TOL_RUN, "w"); assert_close(m, cpu2.m, TOL_RUN, "m")
    plain, _ = make_pair(B, K, P, 2, 2, 0.25, 0.9, 0.05, dtype=dtype, flags=sched, ld=ld, w0=w0)
    for t in range(60):
        plain.step(grads(52, t, K, P, 0.1, gd, ld), 0.05)
    wp, _ = state_of(plain)
    assert np.abs(wp - w).max() > 1e-4            # the variants really change the trajectory


def test_nesterov_needs_momentum(B):
    with pytest.raises(B.DasgdError) as e:
        B.DaSGD(2, 64, 2, 1, 0.25, 0.0, flags=NESTEROV)
    assert e.value.status == B.DASGD_ERR_INVALID_ARG


# ------------------------------------------------------------------ free-running schedules

SCHEDULES = [(1, 1), (2, 1), (4, 1), (1, 2), (2, 2), (4, 2), (2, 3), (3, 0), (1, 0)]


@pytest.mark.parametrize("tau,d", SCHEDULES)
@pytest.mark.parametrize("flags,n_chunks", SCHEDS)
@pytest.mark.parametrize("K,dtype,mode", [(4, 0, 0), (3, 1, 0), (8, 0, 1)])
def test_free_running_100_steps(B, tau, d, flags, n_chunks, K, dtype, mode):
    if flags & INLINE and mode == 1:
        pytest.skip("the inline-mean schedule has no delta merge")
    if n_chunks and d < 1:
        pytest.skip("chunks need d >= 1")
    P, T = 2 * 4096 + 77, 100
    ld = (P + 7) // 8 * 8
    w0 = inputs.shared_start(2, P, 0.02).numpy()
    gpu, cpu = make_pair(B, K, P, tau, d, 0.25, 0.9, 1e-4, dtype=dtype, merge_mode=mode, flags=flags, ld=ld, w0=w0,
                         n_chunks=n_chunks)
    gd = torch.bfloat16 if dtype else torch.float32
    for t in range(T):
        g = grads(7, t, K, P, 0.0316, gd, ld)
        gpu.step(g, 0.1)
        cpu.step(to_oracle_grad(g, P), 0.1)
        assert gpu.n_pending == cpu.n_pending
    w, m = state_of(gpu)
    assert gpu.t == cpu.t == T
    assert_close(w, cpu.w, TOL_RUN, "w after 100 steps")
    assert_close(m, cpu.m, TOL_RUN, "m after 100 steps")
    if dtype:
        np.testing.assert_array_equal(bf16_bits(gpu.w_lp[:, :P]), bf16_bits(gpu.w[:, :P].to(torch.bfloat16)))
    for i in range(cpu.n_pending):
        _, _, mean = cpu.pending(i)
        assert_close(gpu.pending_mean(i).cpu().numpy(), mean, TOL_RUN, f"pending mean {i}")


@pytest.mark.parametrize("tau,d", SCHEDULES)
@pytest.mark.parametrize("dtype,mode", [(0, 0), (1, 0), (0, 1)])
def test_fused_schedules_are_bit_identical_to_unfused(B, tau, d, dtype, mode):
    K, P, T = 4, 2 * 4096 + 13, 25
    ld = (P + 7) // 8 * 8
    w0 = inputs.shared_start(4, P, 0.02)
    gd = torch.bfloat16 if dtype else torch.float32
    outs = {}
    for flags, n_chunks in SCHEDS:
        if (flags & INLINE and mode != 0) or (n_chunks and d < 1):
            continue
        gpu = B.DaSGD(K, P, tau, d, 0.25, 0.9, 1e-4, dtype=dtype, merge_mode=mode, flags=flags, ld=ld, n_chunks=n_chunks)
        gpu.set_state(w0)
        for t in range(T):
            gpu.step(grads(9, t, K, P, 0.0316, gd, ld), 0.1)
        gpu.sync()
        outs[(flags, n_chunks)] = (gpu.w[:, :P].clone(), gpu.m[:, :P].clone(), gpu.launches)   # payload columns only
    w_ref, m_ref, n_ref = outs[(0, 0)]
    for key, (w, m, _) in outs.items():
        assert torch.equal(w, w_ref) and torch.equal(m, m_ref), key
    if d >= 1:
        assert outs[(FUSE_SNAP, 0)][2] < n_ref   # the fused snapshot removes launches
        assert outs[(ROTATE, 0)][2] < n_ref      # so does the rotating snapshot
    if d == 1:                                   # and folding the d = 1 merge into the step kernel removes the merge kernels
        assert outs[(ROTATE | FUSE_MERGE | FUSE_D1, 0)][2] < outs[(ROTATE | FUSE_MERGE, 0)][2]


def test_unaligned_rows_and_gradient_pointer_take_the_scalar_path(B):
    K, P, T = 3, 1001, 12
    w0 = inputs.shared_start(5, P, 0.1).numpy()
    gpu, cpu = make_pair(B, K, P, 2, 1, 0.25, 0.9, 1e-3, ld=P, w0=w0)       # ld = 1001: rows not 16-byte aligned
    for t in range(T):
        g = grads(11, t, K, P, 0.1, torch.float32, P)
        gpu.step(g, 0.05); cpu.step(to_oracle_grad(g, P), 0.05)
    w, m = state_of(gpu)
    assert_close(w, cpu.w, TOL_RUN); assert_close(m, cpu.m, TOL_RUN)
    # aligned rows, misaligned gradient base pointer
    P = 1024
    gpu, cpu = make_pair(B, K, P, 2, 1, 0.25, 0.9, 0.0, w0=np.zeros(P, np.float32))
    buf = torch.zeros(K * P + 1, device="cuda")
    g = buf[1:].view(K, P)
    g.copy_(inputs.grad_block(12, 0, K, P, 0.1))
    gpu.step(g, 0.05); cpu.step(to_oracle_grad(g, P), 0.05)
    w, _ = state_of(gpu)
    assert_close(w, cpu.w, TOL_STEP)


# ------------------------------------------------------------------ explicit call sequence and misuse

@pytest.mark.parametrize("flags", [0, ROTATE])
def test_explicit_calls_equal_step(B, flags):
    K, P, tau, d, T = 4, 5000, 2, 1, 9
    w0 = inputs.shared_start(6, P, 0.1)
    a = B.DaSGD(K, P, tau, d, 0.25, 0.9, flags=flags)
    b = B.DaSGD(K, P, tau, d, 0.25, 0.9, flags=flags)
    a.set_state(w0); b.set_state(w0)
    for t in range(T):
        g = grads(13, t, K, P, 0.1, torch.float32, P)
        a.step(g, 0.1)
        b.local_step(g, 0.1)
        u = t + 1
        if u - d >= tau and (u - d) % tau == 0:
            b.merge()
        if u % tau == 0:
            b.snapshot(); b.average_async()
    a.sync(); b.sync()
    assert torch.equal(a.w, b.w) and torch.equal(a.m, b.m)


@pytest.mark.parametrize("mode", [0, 1])
def test_chunked_pipeline_mixes_with_the_explicit_calls(B, mode):
    """A context with n_chunks > 1: snapshots taken by dasgd_step (one event per column range) may be merged by
    dasgd_merge, and snapshots taken by the explicit calls (one event) may be merged by dasgd_step."""
    K, P, tau, d, T = 3, 3 * 4096 + 50, 2, 1, 12
    ld = (P + 7) // 8 * 8
    w0 = inputs.shared_start(60, P, 0.1).numpy()
    gpu, cpu = make_pair(B, K, P, tau, d, 0.25, 0.9, 1e-3, merge_mode=mode, flags=ROTATE | FUSE_MERGE | LANES, ld=ld, w0=w0, n_chunks=3)
    for t in range(T):
        g = grads(61, t, K, P, 0.05, torch.float32, ld)
        u = t + 1
        if t % 4 < 2:      # the library's scheduler
            gpu.step(g, 0.1)
        else:              # the same iteration spelled out with the explicit calls
            gpu.local_step(g, 0.1)
            if u - d >= tau and (u - d) % tau == 0:
                gpu.merge()
            if u % tau == 0:
                gpu.snapshot(); gpu.average_async()
        cpu.step(to_oracle_grad(g, P), 0.1)
        assert gpu.n_pending == cpu.n_pending
    w, m = state_of(gpu)
    assert_close(w, cpu.w, TOL_RUN, "w"); assert_close(m, cpu.m, TOL_RUN, "m")


@pytest.mark.parametrize("K,dtype,mode,tau,d", [(3, 0, 0, 1, 1), (2, 1, 0, 1, 2), (5, 0, 1, 2, 2), (4, 1, 1, 1, 1)])
def test_whole_array_merging_launch_with_several_tile_groups(B, K, dtype, mode, tau, d):
    """A merge folded into one launch over the whole array walks the rows in groups of 512 tiles of 4096 columns.
    Here: one full group, a ragged second group (300 tiles and a partial one) and a scalar tail."""
    P, T = (512 + 300) * 4096 + 1000 + 13, 8
    ld = (P + 7) // 8 * 8
    w0 = inputs.shared_start(95, P, 0.02).numpy()
    gpu, cpu = make_pair(B, K, P, tau, d, 0.25, 0.9, 1e-4, dtype=dtype, merge_mode=mode,
                         flags=ROTATE | FUSE_MERGE | FUSE_D1, ld=ld, w0=w0)
    gd = torch.bfloat16 if dtype else torch.float32
    ring = [grads(96, t, K, P, 0.0316, gd, ld) for t in range(2)]
    for t in range(T):
        gpu.step(ring[t % 2], 0.1)
        cpu.step(to_oracle_grad(ring[t % 2], P), 0.1)
    w, m = state_of(gpu)
    assert_close(w, cpu.w, TOL_RUN, "w"); assert_close(m, cpu.m, TOL_RUN, "m")
    if dtype:
        np.testing.assert_array_equal(bf16_bits(gpu.w_lp[:, :P]), bf16_bits(gpu.w[:, :P].to(torch.bfloat16)))


def test_chunks_need_rotation_fused_merge_and_a_delay(B):
    for kw in (dict(flags=ROTATE), dict(flags=FUSE_MERGE), dict(flags=ROTATE | FUSE_MERGE, d=0), dict(flags=ROTATE | FUSE_MERGE, n_chunks=1025)):
        args = dict(K=2, P=64, tau=2, d=1, xi=0.25, n_chunks=4)
        args.update(kw)
        with pytest.raises(B.DasgdError) as e:
            B.DaSGD(**args)
        assert e.value.status == B.DASGD_ERR_INVALID_ARG and "n_chunks" in str(e.value)


def test_pending_slot_of_the_inline_schedule_reports_no_snapshot_array(B):
    K, P = 2, 5000
    a = B.DaSGD(K, P, 2, 1, 0.25, flags=INLINE, snapshot_arrays=False)
    g = torch.zeros(K, P, device="cuda")
    a.step(g, 0.1); a.step(g, 0.1); a.sync()
    assert a.n_pending == 1
    s, snap, mean = B.dasgd_get_pending(a.ctx, 0)
    assert s == 2 and snap is None and mean == a.mean[0].data_ptr()


def test_init_rejects_buffers_that_are_not_on_the_device(B):
    e0 = B.DaSGD(2, 64, 2, 1, 0.25)
    cfg = B.dasgd_config.from_buffer_copy(e0.cfg)
    host = torch.zeros(2 * 64).pin_memory()
    cfg.w = host.data_ptr()
    with pytest.raises(B.DasgdError) as e:
        B.dasgd_init(cfg)
    assert e.value.status == B.DASGD_ERR_INVALID_ARG and "device memory" in str(e.value)


def test_refresh_lp_is_the_oracles_rounding(B):
    """With equal float32 masters the library's bfloat16 copy equals the oracle's bit for bit."""
    K, P = 3, 4096 + 21
    r = np.random.default_rng(5)
    W = (r.standard_normal((K, P)) * np.exp(r.uniform(-8, 8, (K, P)))).astype(np.float32)
    W[0, :4] = [1.00390625, 1.01171875, -1.00390625, 3.0e-39]    # ties to even, and a denormal
    gpu, cpu = make_pair(B, K, P, 2, 1, 0.25, 0.9, 0.0, dtype=1, ld=(P + 7) // 8 * 8, w0=W)
    np.testing.assert_array_equal(bf16_bits(gpu.w_lp[:, :P]), cpu.w_lp)
    g = grads(70, 0, K, P, 0.1, torch.bfloat16, gpu.ld)
    gpu.set_state(torch.from_numpy(cpu.w))
    gpu.local_step(g, 0.1); cpu.local_step(to_oracle_grad(g, P), 0.1)
    gpu.set_state(torch.from_numpy(cpu.w))          # teacher-force the masters, then compare the copies
    np.testing.assert_array_equal(bf16_bits(gpu.w_lp[:, :P]), cpu.w_lp)
    f32 = B.DaSGD(2, 64, 2, 1, 0.25)
    with pytest.raises(B.DasgdError) as e:
        B.dasgd_refresh_lp(f32.ctx)
    assert e.value.status == B.DASGD_ERR_BAD_STATE


def test_inline_mean_needs_no_snapshot_arrays_and_refuses_delta(B):
    K, P = 4, 5000
    with pytest.raises(B.DasgdError) as e:
        B.DaSGD(K, P, 2, 1, 0.25, merge_mode=1, flags=INLINE)
    assert e.value.status == B.DASGD_ERR_INVALID_ARG
    a = B.DaSGD(K, P, 2, 1, 0.25, 0.9, flags=INLINE, snapshot_arrays=False)
    b = B.DaSGD(K, P, 2, 1, 0.25, 0.9)
    assert a.snap is None
    w0 = inputs.shared_start(21, P, 0.1)
    a.set_state(w0); b.set_state(w0)
    for t in range(11):
        g = grads(22, t, K, P, 0.1, torch.float32, P)
        a.step(g, 0.1); b.step(g, 0.1)
    a.sync(); b.sync()
    assert torch.equal(a.w, b.w) and torch.equal(a.m, b.m)
    assert a.launches == 11                       # one kernel per iteration
    with pytest.raises(B.DasgdError) as e:
        a.snapshot()                               # the explicit calls need snapshot arrays
    assert e.value.status in (B.DASGD_ERR_BAD_STATE, B.DASGD_ERR_NO_SLOT)


def test_misuse_returns_status_codes(B):
    gpu = B.DaSGD(2, 64, 2, 1, 0.25)
    with pytest.raises(B.DasgdError) as e:
        gpu.merge()
    assert e.value.status == B.DASGD_ERR_BAD_STATE
    with pytest.raises(B.DasgdError) as e:
        gpu.average_async()
    assert e.value.status == B.DASGD_ERR_BAD_STATE
    gpu.snapshot()
    with pytest.raises(B.DasgdError) as e:
        gpu.snapshot()
    assert e.value.status == B.DASGD_ERR_NO_SLOT
    with pytest.raises(B.DasgdError) as e:
        gpu.merge()                      # snapshot exists but was never averaged
    assert e.value.status == B.DASGD_ERR_BAD_STATE
    gpu.average_async(); gpu.merge(); gpu.sync()
    with pytest.raises(B.DasgdError) as e:
        gpu.step_host(torch.zeros(2, 64), 0.1)
    assert e.value.status == B.DASGD_ERR_BAD_STATE
    # the context is still usable afterwards
    gpu.step(torch.zeros(2, 64, device="cuda"), 0.1); gpu.sync()
    assert gpu.t == 1


@pytest.mark.parametrize("flags", [0, ROTATE | FUSE_MERGE, INLINE])
@pytest.mark.parametrize("n_stage", [1, 2])
def test_step_host_matches_step(B, n_stage, flags):
    K, P, T = 4, 4096 + 8, 9
    w0 = inputs.shared_start(8, P, 0.1)
    a = B.DaSGD(K, P, 2, 1, 0.25, 0.9, host_staging=n_stage, flags=flags)
    b = B.DaSGD(K, P, 2, 1, 0.25, 0.9)
    a.set_state(w0); b.set_state(w0)
    probe = torch.empty(256, dtype=torch.float32).pin_memory()
    hosts = [inputs.grad_block(14, t, K, P, 0.1).pin_memory() for t in range(T)]
    for t in range(T):
        a.step_host(hosts[t], 0.1, probe)
        b.step(hosts[t].cuda(), 0.1)
    a.sync(); b.sync()
    assert torch.equal(a.w, b.w)
    assert torch.equal(probe, a.w[0, :256].cpu())


def test_timing_reports_hidden_fraction(B):
    K, P = 8, 1 << 20
    gpu = B.DaSGD(K, P, 2, 1, 0.25, 0.9, flags=B.DASGD_FLAG_TIMING)
    g = torch.zeros(K, P, device="cuda")
    for _ in range(20):
        gpu.step(g, 0.1)
    n, ms_avg, ms_stall = gpu.timing()
    assert n == 10                     # snapshots (and means) at t = 2, 4, .., 20
    assert ms_avg > 0 and ms_stall >= 0
    kt = gpu.kernel_timing()
    assert kt["local_step"][0] == 20 and kt["snapshot"][0] == 10 and kt["mean"][0] == 10
    assert kt["merge"][0] == 9 and kt["stall"][0] == 9   # merges at t = 3, 5, .., 19; the last mean stays pending
    assert all(v[1] > 0 for k, v in kt.items() if k != "stall")
    gpu.reset_timing()
    assert gpu.kernel_timing()["local_step"] == (0, 0.0)


def test_stall_accounting_sees_a_mean_that_blocks_and_one_that_does_not(B):
    """d = 1 with the merge folded into an unchunked step kernel and back-to-back steps: the kernel of step s+1
    cannot start before the mean of step s is complete, and the main stream has nothing else to do meanwhile,
    so practically all of the mean's time is stall.  The chunked pipeline gives each range's mean a window."""
    K, P = 8, 1 << 21
    g = torch.zeros(K, P, device="cuda")
    fracs = {}
    for name, flags, n_chunks in (("blocking", ROTATE | FUSE_MERGE | FUSE_D1, 0), ("pipelined", ROTATE | FUSE_MERGE, 8)):
        gpu = B.DaSGD(K, P, 1, 1, 0.25, 0.9, flags=flags | B.DASGD_FLAG_TIMING, n_chunks=n_chunks, order_after_current=False)
        for _ in range(5):
            gpu.step(g, 0.1)
        gpu.reset_timing()
        for _ in range(30):
            gpu.step(g, 0.1)
        n, ms_avg, ms_stall = gpu.timing()
        kt = gpu.kernel_timing()
        assert n == 30 * max(1, n_chunks) and kt["stall"][0] == n and ms_avg > 0
        fracs[name] = ms_stall / ms_avg
    assert fracs["blocking"] > 0.5
    assert fracs["pipelined"] < fracs["blocking"]


def test_sync_gives_up_after_its_timeout_and_the_context_survives(B):
    """Failure detection on the host: dasgd_sync polls with a deadline.  Nothing on the GPU is made to
    hang: the queue is simply longer than a 1 ms deadline."""
    K, P = 8, 8_000_000
    gpu = B.DaSGD(K, P, 1, 1, 0.25, 0.9, sync_timeout_ms=1, order_after_current=False)
    g = torch.zeros(K, P, device="cuda")
    torch.cuda.synchronize()
    for _ in range(60):                       # tens of milliseconds of queued kernels
        gpu.step(g, 0.1)
    with pytest.raises(B.DasgdError) as e:
        gpu.sync()
    assert e.value.status == B.DASGD_ERR_TIMEOUT
    torch.cuda.synchronize()                  # the work itself completes normally
    gpu.sync()                                # and the context is still usable
    gpu.step(g, 0.1)
    torch.cuda.synchronize()
    assert gpu.t == 61


@pytest.mark.parametrize("tau,d,flags,mode", [(1, 1, ROTATE, 0), (1, 2, ROTATE | FUSE_MERGE, 0), (2, 3, 0, 1), (2, 1, FUSE_SNAP, 0),
                                              (1, 2, ROTATE, 1), (2, 1, INLINE, 0)])
def test_checkpoint_resume_continues_bit_for_bit(B, tau, d, flags, mode):
    K, P, ld, T1, T2 = 3, 4096 + 40, 4096 + 40, 7, 6

    def run(e, a, b):
        for t in range(a, b):
            e.step(grads(31, t, K, P, 0.05, torch.float32, ld), 0.1)

    ref = B.DaSGD(K, P, tau, d, 0.25, 0.9, 1e-3, merge_mode=mode, flags=flags)
    ref.set_state(inputs.shared_start(30, P, 0.1))
    run(ref, 0, T1)
    sd = ref.state_dict()
    run(ref, T1, T1 + T2)
    ref.sync()
    new = B.DaSGD(K, P, tau, d, 0.25, 0.9, 1e-3, merge_mode=mode, flags=flags)
    new.load_state_dict(sd)
    snaps = list(range(tau, T1 + 1, tau))
    assert new.t == T1 and new.n_pending == len([s for s in snaps if s + d > T1])
    run(new, T1, T1 + T2)
    new.sync()
    assert new.t == ref.t
    assert torch.equal(new.w[:, :P], ref.w[:, :P]) and torch.equal(new.m[:, :P], ref.m[:, :P])
    with pytest.raises(B.DasgdError):
        new.load_state_dict(sd)                   # only a fresh context may import
    other = B.DaSGD(K, P, tau + 1, d, 0.25, 0.9, 1e-3, merge_mode=mode, flags=flags, n_slots=new.n_slots)
    with pytest.raises(B.DasgdError):
        other.load_state_dict(sd)                 # different configuration


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("flags,mode", [(0, 0), (ROTATE, 0), (ROTATE, 1), (0, 1)])
def test_random_call_sequences_match_the_oracle(B, seed, flags, mode):
    """Scheduler fuzz: random but valid orders of the four explicit calls (several snapshots in flight,
    means started late, merges in bursts), the same order on the library and on the oracle."""
    import random
    rnd = random.Random(seed * 7 + flags + mode)
    K, P, n_slots = rnd.choice([2, 3, 5]), rnd.choice([1000, 4096 + 9, 2 * 4096]), 3
    ld = (P + 7) // 8 * 8
    gpu, cpu = make_pair(B, K, P, 1, n_slots, 0.25, 0.9, 1e-3, merge_mode=mode, flags=flags, ld=ld, n_slots=n_slots,
                         w0=inputs.shared_start(40 + seed, P, 0.1).numpy())
    snapped = averaged = 0          # snapshots without a mean yet / with a mean, oldest first overall
    for i in range(60):
        choices = ["step"]
        if snapped + averaged < n_slots:
            choices.append("snapshot")
        if snapped:
            choices.append("average")
        if averaged and snapped + averaged > 0:
            choices.append("merge")
        op = rnd.choice(choices)
        if op == "step":
            g = grads(41 + seed, i, K, P, 0.05, torch.float32, ld)
            gpu.local_step(g, 0.1); cpu.local_step(to_oracle_grad(g, P), 0.1)
        elif op == "snapshot":
            gpu.snapshot(); cpu.snapshot(); snapped += 1
        elif op == "average":
            gpu.average_async(); cpu.average(); snapped -= 1; averaged += 1
        else:
            # the oldest pending snapshot must be the one that has its mean: true because means are
            # started oldest first and merged oldest first
            gpu.merge(); cpu.merge(); averaged -= 1
        assert gpu.n_pending == cpu.n_pending == snapped + averaged
    w, m = state_of(gpu)
    assert_close(w, cpu.w, TOL_RUN, "w"); assert_close(m, cpu.m, TOL_RUN, "m")
    for j in range(averaged):
        _, _, mean = cpu.pending(j)
        assert_close(gpu.pending_mean(j).cpu().numpy(), mean, TOL_RUN, f"mean {j}")


@pytest.mark.parametrize("seed", range(40))
def test_random_configurations_match_the_oracle(B, seed):
    """Random draws over every knob of dasgd_step (sizes, schedule, hyper-parameters, dtype, merge form,
    fusion flags, extra slots), 40 steps each."""
    import random
    rnd = random.Random(1000 + seed)
    K = rnd.choice([1, 2, 3, 4, 7, 8, 9, 16, 31])
    P = rnd.choice([1, 5, 8, 63, 1000, 4095, 4096, 4097, 9000, 3 * 4096 + 5])
    tau, d = rnd.choice([1, 2, 3, 5]), rnd.choice([0, 1, 1, 2, 3, 4])
    xi = rnd.choice([0.0, 0.25, 0.5, 0.9, 1.0])
    mom, wd = rnd.choice([0.0, 0.5, 0.9]), rnd.choice([0.0, 1e-4, 1e-2])
    dtype, mode = rnd.choice([0, 0, 1]), rnd.choice([0, 0, 1])
    flags = rnd.choice([0, FUSE_SNAP, FUSE_MERGE, FUSE_SNAP | FUSE_MERGE, ROTATE, ROTATE | FUSE_MERGE] + ([INLINE] if mode == 0 else []))
    ld = rnd.choice([P, (P + 7) // 8 * 8, (P + 7) // 8 * 8 + 8])
    n_slots = max(1, -(-d // tau)) + rnd.choice([0, 0, 1])
    gd = torch.bfloat16 if dtype else torch.float32
    gpu, cpu = make_pair(B, K, P, tau, d, xi, mom, wd, dtype=dtype, merge_mode=mode, flags=flags, ld=ld, n_slots=n_slots,
                         w0=inputs.shared_start(seed, P, 0.05).numpy())
    lr = rnd.choice([0.01, 0.1])
    for t in range(40):
        g = grads(2000 + seed, t, K, P, 0.05, gd, ld)
        gpu.step(g, lr); cpu.step(to_oracle_grad(g, P), lr)
        assert gpu.n_pending == cpu.n_pending
    w, m = state_of(gpu)
    what = f"K={K} P={P} ld={ld} tau={tau} d={d} xi={xi} mom={mom} wd={wd} dtype={dtype} mode={mode} flags={flags} slots={n_slots}"
    assert_close(w, cpu.w, TOL_RUN, what)
    if mom:
        assert_close(m, cpu.m, TOL_RUN, what)
    if dtype:
        np.testing.assert_array_equal(bf16_bits(gpu.w_lp[:, :P]), bf16_bits(gpu.w[:, :P].to(torch.bfloat16)))
