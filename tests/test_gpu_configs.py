"""The five benchmark configurations at full size, in the launch configuration bench.py times
(rotating snapshots, merge folded into the step kernel: chunked pipeline with two lanes when d = 1),
checked against the CPU oracle.

Every operation of the path is independent across the parameter index p, so the oracle runs on a
sample of columns -- at least one from EVERY 4096-column tile of the vector kernels, the first and last
tile of each row in full, plus random ones -- with gradients regenerated on the host by the same
counter-based generator; the GPU works on the full arrays.  Configuration 2 is also compared on every one of
its K*P elements.
"""
import numpy as np
import pytest
import torch

from oracle import OracleDaSGD
from paper_2006_00441_b200 import inputs
from tests.harness import TOL_RUN, TOL_STEP, assert_close, bf16_bits, to_oracle_grad

pytestmark = pytest.mark.gpu
FUSED = 0x4 | 0x8 | 0x100 | 0x400   # snapshots by array rotation; merge folded into the step kernel; two lanes and two side streams when chunked
def chunks_for(K, P, d):
    """The benchmark's policy for the number of column ranges."""
    import bench
    return bench.auto_chunks(K, P) if d >= 1 and P >= 2 * 4096 else 0


@pytest.fixture(scope="module")
def B():
    from paper_2006_00441_b200 import binding
    return binding


def sample_columns(P, n_random=6000, edge=4096 + 24, seed=0, tile=4096):
    """First and last `edge` columns, one column at a random offset inside every tile, and random ones."""
    r = np.random.default_rng(seed)
    parts = [np.arange(min(edge, P)), np.arange(max(0, P - edge), P), r.integers(0, P, size=n_random)]
    starts = np.arange(0, P, tile, dtype=np.int64)
    parts.append(np.minimum(starts + r.integers(0, tile, size=starts.size), P - 1))
    return np.unique(np.concatenate(parts).astype(np.int64))


def test_sample_columns_touch_every_tile():
    for P in (25_600_000, 335_000_000, 4 * 4096 * 4096, 9000):
        idx = sample_columns(P, seed=P % 97)
        assert np.array_equal(np.unique(idx // 4096), np.arange((P + 4095) // 4096))
        assert idx[0] == 0 and idx[-1] == P - 1


def run_sampled(B, K, P, tau, d, xi, mom, wd, lr, T, g_std, dtype=0, ring=4, seed=0, checkpoints=(100,), flags=FUSED):
    """Full-size GPU run against the oracle on sampled columns.  Gradients: a ring of `ring` blocks."""
    gd = torch.bfloat16 if dtype else torch.float32
    idx = sample_columns(P, seed=seed)
    gpu = B.DaSGD(K, P, tau, d, xi, mom, wd, dtype=dtype, flags=flags, order_after_current=False,
                  n_chunks=chunks_for(K, P, d) if flags & 0x4 and flags & 0x8 else 0)
    gpu.set_state(inputs.shared_start(seed, P, 0.02, device="cuda"))
    cpu = OracleDaSGD(K, len(idx), tau, d, xi, mom, wd, dtype=dtype)
    cpu.set_state(inputs.shared_start(seed, P, 0.02, p_index=idx).numpy())
    dev_ring = [inputs.grad_block(seed, r, K, P, g_std, dtype=gd, device="cuda") for r in range(ring)]
    host_ring = [to_oracle_grad(inputs.grad_block(seed, r, K, P, g_std, dtype=gd, p_index=idx), len(idx))
                 for r in range(ring)]
    torch.cuda.synchronize()
    tidx = torch.from_numpy(idx).cuda()
    for t in range(T):
        gpu.step(dev_ring[t % ring], lr)
        cpu.step(host_ring[t % ring], lr)
        if (t + 1) in checkpoints or t + 1 == T:
            gpu.sync()
            assert_close(gpu.w[:, tidx].cpu().numpy(), cpu.w, TOL_RUN, f"w after {t + 1} steps")
            if mom:
                assert_close(gpu.m[:, tidx].cpu().numpy(), cpu.m, TOL_RUN, f"m after {t + 1} steps")
            if dtype:
                np.testing.assert_array_equal(bf16_bits(gpu.w_lp[:, tidx]), bf16_bits(gpu.w[:, tidx].to(torch.bfloat16)))
    assert gpu.t == cpu.t == T and gpu.n_pending == cpu.n_pending
    for i in range(cpu.n_pending):
        _, _, mean = cpu.pending(i)
        assert_close(gpu.pending_mean(i)[tidx].cpu().numpy(), mean, TOL_RUN, f"pending mean {i}")
    gpu.close()
    del dev_ring
    torch.cuda.empty_cache()


# ---------------------------------------------------------------- config 1: linear regression

def test_config1_linear_regression(B):
    K, P, batch, lr, tau, d, xi, T = 4, 1024, 32, 0.01, 4, 1, 0.25, 100
    prob = inputs.LinearRegression(0, K, P, batch, noise_var=0.01, dtype=torch.float64)   # oracle side: float64
    X = [[prob.batch_xy(t, k) for k in range(K)] for t in range(T)]

    def grad_gpu(t, w):  # the GPU side does its own forward/backward in float32 on the device
        out = torch.empty(K, P, device="cuda")
        for k in range(K):
            Xk, yk = X[t][k][0].cuda(), X[t][k][1].cuda()
            out[k] = Xk.T @ (Xk @ w[k] - yk) / batch
        return out

    # free-running: each side computes gradients from its own weights
    gpu = B.DaSGD(K, P, tau, d, xi, flags=FUSED)
    cpu = OracleDaSGD(K, P, tau, d, xi)
    losses = []
    for t in range(T):
        gpu.sync()
        gpu.step(grad_gpu(t, gpu.w), lr)
        cpu.step(prob.grad(t, torch.from_numpy(cpu.w)).numpy(), lr)
        if t % 10 == 0:
            losses.append(prob.loss(t, torch.from_numpy(cpu.w)))
    gpu.sync()
    assert_close(gpu.w.cpu().numpy(), cpu.w, TOL_RUN, "free-running, 100 steps")
    assert losses[-1] < 0.6 * losses[0]   # the run actually optimises

    # teacher-forced: the GPU starts every step from the oracle's state and gets the oracle's gradient
    gpu2 = B.DaSGD(K, P, tau, d, xi)
    cpu2 = OracleDaSGD(K, P, tau, d, xi)
    for t in range(T):
        g = prob.grad(t, torch.from_numpy(cpu2.w))
        gpu2.set_state(torch.from_numpy(cpu2.w))
        u = t + 1
        gpu2.local_step(g.cuda(), lr); cpu2.local_step(g.numpy(), lr)
        gpu2.sync()
        assert_close(gpu2.w.cpu().numpy(), cpu2.w, TOL_STEP, f"local step {t}")
        if u - d >= tau and (u - d) % tau == 0:
            _, _, mean = cpu2.pending(0)
            gpu2.pending_mean(0).copy_(torch.from_numpy(mean))     # teacher-force the mean as well
            torch.cuda.synchronize()
            gpu2.merge(); cpu2.merge(); gpu2.sync()
            assert_close(gpu2.w.cpu().numpy(), cpu2.w, TOL_STEP, f"merge at {u}")
        if u % tau == 0:
            gpu2.snapshot(); gpu2.average_async(); cpu2.snapshot(); cpu2.average(); gpu2.sync()
            _, _, mean = cpu2.pending(cpu2.n_pending - 1)
            assert_close(gpu2.pending_mean(gpu2.n_pending - 1).cpu().numpy(), mean, TOL_STEP, f"mean at {u}")


# ---------------------------------------------------------------- config 2: ResNet-50-sized

def test_config2_resnet50_sized_200_steps(B):
    run_sampled(B, K=8, P=25_600_000, tau=1, d=1, xi=0.25, mom=0.9, wd=1e-4, lr=0.1, T=200, g_std=1e-3 ** 0.5,
                checkpoints=(1, 2, 100))


def test_config2_every_element_20_steps(B):
    """All K*P = 204.8M elements against the OpenMP build of the oracle (the same source as the plain build),
    in the launch configuration the benchmark times.  The gradients are the seeded generator's, made once on
    the device and copied to the host, so both sides read the same numbers."""
    K, P, tau, d, xi, mom, wd, lr, T = 8, 25_600_000, 1, 1, 0.25, 0.9, 1e-4, 0.1, 20
    ring = 3
    gpu = B.DaSGD(K, P, tau, d, xi, mom, wd, flags=FUSED, n_chunks=chunks_for(K, P, d), order_after_current=False)
    w0 = inputs.shared_start(7, P, 0.02, device="cuda")
    gpu.set_state(w0)
    cpu = OracleDaSGD(K, P, tau, d, xi, mom, wd, omp=True)
    cpu.set_state(w0.cpu().numpy())
    dev_ring = [inputs.grad_block(7, r, K, P, 1e-3 ** 0.5, device="cuda") for r in range(ring)]
    host_ring = [g.cpu().numpy() for g in dev_ring]
    torch.cuda.synchronize()
    for t in range(T):
        gpu.step(dev_ring[t % ring], lr)
        cpu.step(host_ring[t % ring], lr)
        if t + 1 in (1, 2, T):
            gpu.sync()
            tol = TOL_STEP if t == 0 else TOL_RUN      # the first step starts from identical states
            assert_close(gpu.w.cpu().numpy(), cpu.w, tol, f"all elements of w after {t + 1} steps")
            assert_close(gpu.m.cpu().numpy(), cpu.m, tol, f"all elements of m after {t + 1} steps")
    assert gpu.n_pending == cpu.n_pending == 1
    assert_close(gpu.pending_mean(0).cpu().numpy(), cpu.pending(0)[2], TOL_RUN, "pending mean, all elements")
    gpu.close()


def test_config2_inline_mean_schedule(B):
    run_sampled(B, K=8, P=25_600_000, tau=1, d=1, xi=0.25, mom=0.9, wd=1e-4, lr=0.1, T=100, g_std=1e-3 ** 0.5,
                flags=0x10)


@pytest.mark.parametrize("K,tau,d", [(32, 1, 2), (2, 4, 1), (16, 2, 2)])
def test_config4_points_inline_mean_schedule(B, K, tau, d):
    run_sampled(B, K=K, P=25_600_000, tau=tau, d=d, xi=0.25, mom=0.9, wd=0.0, lr=0.1, T=100, g_std=1e-3 ** 0.5,
                ring=2, seed=K + tau + d, flags=0x10)


# ---------------------------------------------------------------- config 3: BERT-large-sized, bf16

def test_config3_bert_large_sized_bf16_50_steps(B):
    run_sampled(B, K=4, P=335_000_000, tau=2, d=1, xi=0.25, mom=0.9, wd=0.0, lr=1e-3, T=50, g_std=1e-2,
                dtype=1, ring=2, checkpoints=(1, 3, 25))


def test_config3_inline_mean_schedule(B):
    run_sampled(B, K=4, P=335_000_000, tau=2, d=1, xi=0.25, mom=0.9, wd=0.0, lr=1e-3, T=50, g_std=1e-2,
                dtype=1, ring=2, flags=0x10)


# ---------------------------------------------------------------- config 4: the sweep

@pytest.mark.parametrize("d", [1, 2])
@pytest.mark.parametrize("tau", [1, 2, 4])
@pytest.mark.parametrize("K", [2, 4, 8, 16, 32])
def test_config4_sweep(B, K, tau, d):
    run_sampled(B, K=K, P=25_600_000, tau=tau, d=d, xi=0.25, mom=0.9, wd=0.0, lr=0.1, T=100, g_std=1e-3 ** 0.5,
                ring=2 if K >= 16 else 4, seed=K * 10 + tau * 3 + d)


# ---------------------------------------------------------------- config 5: K replicas of an MLP, end to end

def test_config5_mlp_reduced_size_whole_loop_against_oracle(B):
    """Hidden size 256: both sides run their own forward/backward (GPU: bf16 matmuls on the device;
    oracle side: the same workload in bf16 on the host) from their own weights, 100 steps."""
    K, H, T, lr, tau, d, xi = 8, 256, 100, 1e-3, 1, 1, 0.25
    net_gpu = inputs.TeacherMLP(3, K, H, device="cuda", dtype=torch.bfloat16)
    net_cpu = inputs.TeacherMLP(3, K, H, device="cpu", dtype=torch.bfloat16)
    P = net_gpu.P
    gpu = B.DaSGD(K, P, tau, d, xi, 0.9, 0.0, dtype=1, flags=FUSED)
    cpu = OracleDaSGD(K, P, tau, d, xi, 0.9, 0.0, dtype=1)
    w0 = net_cpu.student_init()
    gpu.set_state(w0); cpu.set_state(w0.numpy())
    g_gpu = torch.zeros(K, P, dtype=torch.bfloat16, device="cuda")
    g_cpu = torch.zeros(K, P, dtype=torch.bfloat16)
    first = last = None
    for t in range(T):
        gpu.sync()
        loss = net_gpu.forward_backward(t, gpu.w_lp, g_gpu)
        gpu.step(g_gpu, lr)
        w_lp_cpu = torch.from_numpy(cpu.w_lp.view(np.int16)).view(torch.bfloat16)
        net_cpu.forward_backward(t, w_lp_cpu, g_cpu)
        cpu.step(to_oracle_grad(g_cpu, P), lr)
        first = float(loss.mean()) if first is None else first
        last = float(loss.mean())
    gpu.sync()
    assert_close(gpu.w.cpu().numpy(), cpu.w, TOL_RUN, "masters after 100 steps")
    assert last < first


def test_config5_mlp_full_size_500_steps(B):
    """Hidden size 4096, batch 256 per worker, 500 steps on the GPU (forward/backward: bf16 batched
    matmuls).  A host forward/backward at this size is out of reach, so the oracle is fed the gradient
    columns the workload produced on the device: this checks the update / snapshot / mean / merge path
    (teacher-forced on the gradients), not the matmuls."""
    K, H, T, lr, tau, d, xi = 8, 4096, 500, 1e-3, 1, 1, 0.25
    net = inputs.TeacherMLP(4, K, H, device="cuda", dtype=torch.bfloat16)
    P = net.P
    idx = sample_columns(P, n_random=3000, seed=5)
    tidx = torch.from_numpy(idx).cuda()
    gpu = B.DaSGD(K, P, tau, d, xi, 0.9, 0.0, dtype=1, flags=FUSED | 0x80)   # forward/backward is the mean's window
    cpu = OracleDaSGD(K, len(idx), tau, d, xi, 0.9, 0.0, dtype=1)
    w0 = net.student_init()
    gpu.set_state(w0); cpu.set_state(w0[tidx].cpu().numpy())
    g = torch.zeros(K, P, dtype=torch.bfloat16, device="cuda")
    losses = []
    for t in range(T):
        gpu.sync()
        loss = net.forward_backward(t, gpu.w_lp, g)
        gpu.step(g, lr)
        cpu.step(to_oracle_grad(g[:, tidx], len(idx)), lr)
        if t % 50 == 0 or t == T - 1:
            losses.append(float(loss.mean()))
        if t + 1 in (1, 100, T):
            gpu.sync()
            assert_close(gpu.w[:, tidx].cpu().numpy(), cpu.w, TOL_RUN, f"masters after {t + 1} steps")
    assert losses[-1] < losses[0]
