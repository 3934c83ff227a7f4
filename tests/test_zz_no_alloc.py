"""dasgd_average_merge_noalloc: the entry point for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits -- in a serving loop whose memory pool
is frozen once warm, as a plug-in that is handed a fixed arena, or beside another runtime that owns
the device allocator.  For them the library
carries its own 4 MiB mean vector.  The test drives the new call through the C ABI twice in a row (the
built-in vector keeps the first call's contents, which must not leak into the second) and checks each
result against the ordinary snapshot / average / merge entry points, which use caller-provided buffers, and
against the CPU oracle run with a delay of 0 (snapshot, mean and blend in one go).
This file sorts last on purpose: a run that stops at the first failure has then run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from tests.harness import TOL_STEP, assert_close


def test_noalloc_rejects_sizes_beyond_its_built_in_vector():
    from paper_2006_00441_b200 import binding as B
    with pytest.raises(B.DasgdError) as e:
        B.dasgd_average_merge_noalloc(0x1000, 4, B.DASGD_NOALLOC_MAX_P + 1, 0, 0.25, 0, None)
    assert e.value.status == B.DASGD_ERR_UNSUPPORTED and "DASGD_NOALLOC_MAX_P" in str(e.value)
    with pytest.raises(B.DasgdError) as e:
        B.dasgd_average_merge_noalloc(None, 4, 16, 0, 0.25, 0, None)
    assert e.value.status == B.DASGD_ERR_INVALID_ARG


@pytest.mark.gpu
@pytest.mark.parametrize("K,P,ld,xi", [(8, 300_001, 300_008, 0.25), (3, 1_048_576, 1_048_576, 0.25), (5, 7, 7, 0.25),
                                       (1, 4099, 4104, 0.5), (4, 70_000, 70_000, 0.0), (4, 70_000, 70_000, 1.0)])
def test_noalloc_matches_the_buffered_entry_points_twice_in_a_row(K, P, ld, xi):
    from oracle import OracleDaSGD
    from paper_2006_00441_b200 import binding as B
    gen = torch.Generator(device="cpu").manual_seed(K * 1000 + P % 997)
    stream = torch.cuda.Stream()
    for call in range(2):
        # different data and a different scale on the second call: stale contents of the built-in
        # vector would show up as a wrong mean
        W = (torch.randn(K, P, generator=gen) * (1.0 + 3.0 * call) + call).float()
        ref = B.DaSGD(K, P, tau=1, d=0, xi=xi, ld=ld)
        ref.set_state(W)
        ref.snapshot(); ref.average_async(); ref.merge(); ref.sync()
        want = ref.w[:, :P].cpu().numpy()
        ref.close()

        w = torch.zeros(K, ld, device="cuda")
        w[:, :P] = W.cuda()
        torch.cuda.synchronize()
        B.dasgd_average_merge_noalloc(w.data_ptr(), K, P, ld, xi, 0, stream.cuda_stream)
        stream.synchronize()
        got = w[:, :P].cpu().numpy()
        assert_close(got, want, TOL_STEP, f"call {call}")
        exact = xi * W.double() + (1 - xi) * W.double().mean(0, keepdim=True)
        assert_close(got, exact.numpy(), TOL_STEP, f"call {call} vs definition")
        cpu = OracleDaSGD(K, P, 1, 0, xi)
        cpu.set_state(W.numpy())
        cpu.snapshot(); cpu.average(); cpu.merge()
        assert_close(got, cpu.w, TOL_STEP, f"call {call} vs the oracle")
        if ld > P:
            assert float(w[:, P:].abs().max()) == 0.0
