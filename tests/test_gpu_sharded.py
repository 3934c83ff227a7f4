"""The sharded worker axis on the GPU (each context holds some of the K workers; the partial sums are
exchanged; one division by K where the merge reads the total), checked against the UNSHARDED CPU oracle.

Two set-ups, neither of which needs more than one GPU:
  * a one-rank NCCL communicator: the library's own exchange (ncclAllReduce on the side stream) runs for
    real, with nothing to add;
  * two contexts on one GPU, each holding half of the workers, whose exchange is done by the test itself
    between iterations (the callback only notes where the sums are; the test adds them once both contexts
    have been given the iteration and have drained).  Nothing on the GPU waits for anything else.
"""
import numpy as np
import pytest
import torch

from oracle import OracleDaSGD
from paper_2006_00441_b200 import inputs
from tests.harness import TOL_RUN, TOL_STEP, assert_close, padded_grad, to_oracle_grad

pytestmark = pytest.mark.gpu
ROTATE, FUSE_MERGE, FUSE_SNAP, LANES, FUSE_D1 = 0x8, 0x4, 0x2, 0x100, 0x80


@pytest.fixture(scope="module")
def B():
    from paper_2006_00441_b200 import binding
    return binding


@pytest.fixture(scope="module")
def comm(B):
    c = B.dasgd_nccl_comm_init(B.dasgd_nccl_unique_id(), 1, 0, 0)
    yield c
    torch.cuda.synchronize()
    B.dasgd_nccl_comm_destroy(c)


def grads(seed, t, K, P, std, dtype, ld):
    return padded_grad(inputs.grad_block(seed, t, K, P, std, dtype=dtype), ld)


@pytest.mark.parametrize("tau,d", [(1, 1), (2, 1), (1, 2), (3, 0), (2, 3)])
@pytest.mark.parametrize("K,dtype,mode,flags,n_chunks", [
    (4, 0, 0, 0, 0), (1, 0, 0, ROTATE | FUSE_MERGE, 0), (3, 1, 0, ROTATE | FUSE_MERGE | LANES, 3), (8, 0, 1, ROTATE | FUSE_MERGE, 2),
    (1, 1, 0, ROTATE | FUSE_MERGE | LANES, 3), (5, 0, 0, FUSE_SNAP | FUSE_MERGE | FUSE_D1, 0)])
def test_one_rank_nccl_exchange_matches_the_oracle(B, comm, tau, d, K, dtype, mode, flags, n_chunks):
    if n_chunks and d < 1:
        pytest.skip("chunks need d >= 1")
    P, T = 2 * 4096 + 77, 40
    ld = (P + 7) // 8 * 8
    gd = torch.bfloat16 if dtype else torch.float32
    r = np.random.default_rng(K * 7 + tau)
    w0 = (r.standard_normal((K, P)) * 0.05).astype(np.float32)
    gpu = B.DaSGD(K, P, tau, d, 0.25, 0.9, 1e-4, dtype=dtype, merge_mode=mode, flags=flags, ld=ld, n_chunks=n_chunks)
    gpu.set_shard(K, nccl_comm=comm)
    cpu = OracleDaSGD(K, P, tau, d, 0.25, 0.9, 1e-4, dtype=dtype, merge_mode=mode)
    gpu.set_state(torch.from_numpy(w0)); cpu.set_state(w0)
    for t in range(T):
        g = grads(90, t, K, P, 0.03, gd, ld)
        gpu.step(g, 0.1); cpu.step(to_oracle_grad(g, P), 0.1)
        assert gpu.n_pending == cpu.n_pending
    gpu.sync()
    assert_close(gpu.w[:, :P].cpu().numpy(), cpu.w, TOL_RUN, "w")
    assert_close(gpu.m[:, :P].cpu().numpy(), cpu.m, TOL_RUN, "m")
    for i in range(cpu.n_pending):          # the slot holds the SUM over all workers
        assert_close(gpu.pending_mean(i).cpu().numpy() / K, cpu.pending(i)[2], TOL_RUN, f"pending sum {i} / K")
    gpu.close()


def test_one_rank_nccl_teacher_forced_mean_and_merge(B, comm):
    """One operation at a time at the per-step tolerance: the sum, then the merge that divides it by K."""
    K, P = 6, 4096 + 13
    r = np.random.default_rng(3)
    W = r.standard_normal((K, P)).astype(np.float32)
    gpu = B.DaSGD(K, P, 2, 1, 0.25, ld=P + 3)
    gpu.set_shard(K, nccl_comm=comm)
    cpu = OracleDaSGD(K, P, 2, 1, 0.25)
    gpu.set_state(torch.from_numpy(W)); cpu.set_state(W)
    gpu.snapshot(); gpu.average_async(); cpu.snapshot(); cpu.average(); gpu.sync()
    assert_close(gpu.pending_mean(0).cpu().numpy() / K, cpu.pending(0)[2], TOL_STEP, "sum / K")
    W2 = r.standard_normal((K, P)).astype(np.float32)
    gpu.set_state(torch.from_numpy(W2)); cpu.set_state(W2)
    gpu.merge(); cpu.merge(); gpu.sync()
    assert_close(gpu.w[:, :P].cpu().numpy(), cpu.w, TOL_STEP, "merged w")


class Deferred:
    """Exchange callback of one emulated shard: remembers (send, recv, count) of every call."""

    def __init__(self):
        self.calls = []

    def __call__(self, send, recv, count, stream):
        self.calls.append((send, recv, count))


def view_of(eng, ptr, count):
    """The float32 elements [ptr, ptr + 4*count) as a view into whichever tensor of `eng` holds them."""
    for t in (eng.mean, eng.snap, eng._w0):
        if t is None:
            continue
        base, n = t.data_ptr(), t.numel()
        if base <= ptr and ptr + 4 * count <= base + 4 * n:
            off = (ptr - base) // 4
            return t.view(-1)[off:off + count]
    raise AssertionError("exchange pointer outside the context's arrays")


@pytest.mark.parametrize("tau,d", [(1, 1), (2, 1), (1, 2), (2, 2)])
@pytest.mark.parametrize("split,dtype,mode,flags,n_chunks", [
    ((4, 4), 0, 0, ROTATE | FUSE_MERGE | LANES, 3), ((3, 5), 0, 0, 0, 0), ((1, 1), 0, 0, ROTATE | FUSE_MERGE, 2),
    ((1, 3), 1, 0, ROTATE | FUSE_MERGE, 0), ((2, 2), 0, 1, ROTATE | FUSE_MERGE | LANES, 3)])
def test_two_shards_on_one_gpu_reproduce_the_unsharded_oracle(B, tau, d, split, dtype, mode, flags, n_chunks):
    K, P, T = sum(split), 3 * 4096 + 40, 30
    ld = (P + 7) // 8 * 8
    gd = torch.bfloat16 if dtype else torch.float32
    r = np.random.default_rng(K * 13 + tau * 3 + d)
    w0 = (r.standard_normal((K, P)) * 0.05).astype(np.float32)
    cpu = OracleDaSGD(K, P, tau, d, 0.25, 0.9, 1e-4, dtype=dtype, merge_mode=mode)
    cpu.set_state(w0)
    starts = np.cumsum((0,) + split)
    shards = []
    for a, b in zip(starts[:-1], starts[1:]):
        e = B.DaSGD(int(b - a), P, tau, d, 0.25, 0.9, 1e-4, dtype=dtype, merge_mode=mode, flags=flags, ld=ld, n_chunks=n_chunks)
        x = Deferred()
        e.set_shard(K, exchange=x)
        e.set_state(torch.from_numpy(w0[a:b]))
        shards.append((int(a), int(b), e, x))
    for t in range(T):
        g = grads(91, t, K, P, 0.03, gd, ld)
        for a, b, e, x in shards:
            e.step(g[a:b].contiguous(), 0.1)
        cpu.step(to_oracle_grad(g, P), 0.1)
        for _, _, e, _ in shards:
            e.sync()
        # the all-reduce, done here: every shard made the same calls in the same order
        n_calls = len(shards[0][3].calls)
        assert all(len(x.calls) == n_calls for _, _, _, x in shards)
        for i in range(n_calls):
            parts = [view_of(e, x.calls[i][0], x.calls[i][2]) for _, _, e, x in shards]
            total = parts[0].clone()
            for p_ in parts[1:]:
                total += p_
            for _, _, e, x in shards:
                view_of(e, x.calls[i][1], x.calls[i][2]).copy_(total)
        for _, _, _, x in shards:
            x.calls.clear()
        torch.cuda.synchronize()
    for a, b, e, _ in shards:
        assert e.n_pending == cpu.n_pending
        assert_close(e.w[:, :P].cpu().numpy(), cpu.w[a:b], TOL_RUN, f"w rows {a}:{b}")
        assert_close(e.m[:, :P].cpu().numpy(), cpu.m[a:b], TOL_RUN, f"m rows {a}:{b}")
        e.close()


def test_shard_misuse(B, comm):
    e = B.DaSGD(4, 64, 2, 1, 0.25)
    with pytest.raises(B.DasgdError) as err:
        e.set_shard(3, nccl_comm=comm)                  # fewer workers in total than here
    assert err.value.status == B.DASGD_ERR_INVALID_ARG
    e.step(torch.zeros(4, 64, device="cuda"), 0.1)
    with pytest.raises(B.DasgdError) as err:
        e.set_shard(8, nccl_comm=comm)                  # only a fresh context can be made a shard
    assert err.value.status == B.DASGD_ERR_BAD_STATE
    inline = B.DaSGD(4, 64, 2, 1, 0.25, flags=0x10)
    with pytest.raises(B.DasgdError) as err:
        inline.set_shard(8, nccl_comm=comm)
    assert err.value.status == B.DASGD_ERR_UNSUPPORTED
