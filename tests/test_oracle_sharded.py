"""Pins for the oracle's sharded worker axis: a partitioned run (each shard holds some of the workers, the
partial sums are added across shards, one division by the total) reproduces the unsharded oracle.

The two-rank case runs as two processes that exchange their partial sums through a gloo all-reduce, the
way the ranks of a sharded GPU job exchange theirs; it pins the partition arithmetic without a GPU."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import OracleDaSGD, OracleError

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TOL = 1e-6


def workload(K, P, T, seed):
    r = np.random.default_rng(seed)
    w0 = (r.standard_normal((K, P)) * 0.1).astype(np.float32)      # distinct starts: the mean is not trivial
    G = (r.standard_normal((T, K, P)) * 0.05).astype(np.float32)
    return w0, G


def run_unsharded(K, P, tau, d, xi, w0, G, lr, mode=0):
    o = OracleDaSGD(K, P, tau, d, xi, 0.9, 1e-3, merge_mode=mode)
    o.set_state(w0)
    out = []
    for t in range(G.shape[0]):
        o.step(G[t], lr)
        out.append(o.w.copy())
    return out, o


@pytest.mark.parametrize("tau,d", [(1, 1), (2, 1), (1, 2), (3, 0), (2, 2)])
@pytest.mark.parametrize("split", [(4, 4), (3, 5), (1, 7), (2, 2, 4), (1,) * 8])
def test_shards_in_one_process_reproduce_the_unsharded_oracle(tau, d, split):
    K, P, T, lr, xi = 8, 257, 14, 0.1, 0.25
    w0, G = workload(K, P, T, 10 * tau + d)
    ref, oref = run_unsharded(K, P, tau, d, xi, w0, G, lr)
    starts = np.cumsum((0,) + split)
    shards = []
    for a, b in zip(starts[:-1], starts[1:]):
        o = OracleDaSGD(int(b - a), P, tau, d, xi, 0.9, 1e-3)
        o.set_shard(K)
        o.set_state(w0[a:b])
        shards.append((a, b, o))
    same = total = 0
    for t in range(T):
        # lock-step: every shard takes its local step and merge, then all exchange their sums
        sums = []
        for a, b, o in shards:
            o.local_step(G[t][a:b], lr)
            u = o.t
            if d > 0 and u - d >= tau and (u - d) % tau == 0:
                o.merge()
            if u % tau == 0:
                o.snapshot()
                sums.append(o.partial_sum())
        if sums:
            tot = np.sum(sums, axis=0)
            for a, b, o in shards:
                o.set_mean_from_sum(tot)
                if d == 0:
                    o.merge()
        for a, b, o in shards:
            got, want = o.w.astype(np.float64), ref[t][a:b].astype(np.float64)
            assert (np.abs(got - want) <= TOL * (1 + np.abs(want))).all(), (t, a, b)
            same += int((o.w == ref[t][a:b]).sum()); total += got.size
    assert same >= 0.999 * total            # the two-level sum almost never changes the rounded mean
    for a, b, o in shards:
        assert o.n_pending == oref.n_pending


def test_one_shard_holding_every_worker_is_the_unsharded_oracle_bit_for_bit():
    K, P, T = 5, 100, 9
    w0, G = workload(K, P, T, 3)
    ref, _ = run_unsharded(K, P, 2, 1, 0.25, w0, G, 0.1)
    o = OracleDaSGD(K, P, 2, 1, 0.25, 0.9, 1e-3)
    o.set_shard(K)
    o.set_state(w0)
    for t in range(T):
        o.sharded_step(G[t], 0.1, lambda s: s)
        np.testing.assert_array_equal(o.w, ref[t])


def test_mean_divides_by_the_total_number_of_workers():
    """Two shards of one worker each whose snapshots are 1.0 and 3.0: the mean is 2.0 (not 1.0 or 3.0, which a
    division by the shard's own size would give, and not 4.0)."""
    shards = [OracleDaSGD(1, 4, 1, 1, 0.0) for _ in range(2)]
    for o, v in zip(shards, (1.0, 3.0)):
        o.set_shard(2)
        o.set_state(np.full((1, 4), v, np.float32))
        o.snapshot()
    tot = shards[0].partial_sum() + shards[1].partial_sum()
    np.testing.assert_array_equal(tot, np.full(4, 4.0))
    for o in shards:
        o.set_mean_from_sum(tot)
        o.merge()                      # xi = 0: the weights become the mean
        np.testing.assert_array_equal(o.w, np.full((1, 4), 2.0, np.float32))


def test_explicit_calls_on_shards_with_two_snapshots_in_flight():
    """Two snapshots pending without a mean: the partial sum (and the mean set from the total) belong to the OLDER one."""
    K, P = 4, 31
    w0, G = workload(K, P, 3, 77)
    ref = OracleDaSGD(K, P, 1, 2, 0.5)
    ref.set_state(w0)
    shards = [OracleDaSGD(2, P, 1, 2, 0.5) for _ in range(2)]
    for i, o in enumerate(shards):
        o.set_shard(K)
        o.set_state(w0[2 * i:2 * i + 2])
    for t in range(2):                     # two steps, a snapshot after each, no mean yet
        ref.local_step(G[t], 0.1); ref.snapshot()
        for i, o in enumerate(shards):
            o.local_step(G[t][2 * i:2 * i + 2], 0.1); o.snapshot()
    for _ in range(2):                     # now the means, oldest first
        ref.average()
        tot = shards[0].partial_sum() + shards[1].partial_sum()
        for o in shards:
            o.set_mean_from_sum(tot)
    for j in range(2):
        _, _, mean = ref.pending(j)
        for o in shards:
            np.testing.assert_allclose(o.pending(j)[2], mean, rtol=0, atol=1e-7)
    ref.merge()
    for i, o in enumerate(shards):
        o.merge()
        np.testing.assert_allclose(o.w, ref.w[2 * i:2 * i + 2], rtol=0, atol=1e-7)


def test_a_shard_cannot_average_alone():
    o = OracleDaSGD(2, 4, 1, 1, 0.25)
    o.set_shard(4)
    o.snapshot()
    with pytest.raises(OracleError):
        o.average()
    with pytest.raises(OracleError):
        OracleDaSGD(4, 4, 1, 1, 0.25).set_shard(2)      # fewer workers in total than in the shard


# ---------------------------------------------------------------- two ranks, gloo

def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, cases, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    dist.init_process_group("gloo", rank=rank, world_size=world)

    def exchange(s):
        t = torch.from_numpy(s.copy())
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return t.numpy()

    worst = 0.0
    for tau, d in cases:
        K, P, T, lr, xi = 8, 513, 12, 0.1, 0.25
        w0, G = workload(K, P, T, 100 + 10 * tau + d)
        ref, _ = run_unsharded(K, P, tau, d, xi, w0, G, lr)
        a, b = rank * K // world, (rank + 1) * K // world
        o = OracleDaSGD(b - a, P, tau, d, xi, 0.9, 1e-3)
        o.set_shard(K)
        o.set_state(w0[a:b])
        for t in range(T):
            o.sharded_step(G[t][a:b], lr, exchange)
            got, want = o.w.astype(np.float64), ref[t][a:b].astype(np.float64)
            worst = max(worst, float((np.abs(got - want) / (1 + np.abs(want))).max()))
    out[rank] = worst
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_with_an_all_reduce_reproduce_the_unsharded_oracle():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank, args=(world, port, [(1, 1), (2, 1), (1, 2)], out), nprocs=world, join=True)
        res = dict(out)
    assert sorted(res) == [0, 1]
    assert max(res.values()) <= TOL
