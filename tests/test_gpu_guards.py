"""Out-of-bounds check without a sanitizer: every device array handed to the library is carved out of
one allocation with sentinel-filled guard zones before and after it; after a run that exercises every
kernel (vector bodies, scalar tails, both dtypes, copy and rotate snapshots, fused merge) the guards and
the row padding must be untouched.  The same for the column-range pipeline (two lanes, two side streams), the
inline-mean schedule and the arrays of the momentum-averaging variant."""
import ctypes

import pytest
import torch

from paper_2006_00441_b200 import inputs

pytestmark = pytest.mark.gpu
GUARD = 4096          # bytes on each side of every array
SENTINEL = 0x5A


class Arena:
    def __init__(self, nbytes):
        self.buf = torch.full((nbytes,), SENTINEL, dtype=torch.uint8, device="cuda")
        self.off = 0
        self.payloads = []

    def carve(self, nbytes):
        start = (self.off + GUARD + 255) // 256 * 256
        self.payloads.append((start, nbytes))
        self.off = start + nbytes
        assert self.off + GUARD <= self.buf.numel()
        return self.buf[start:start + nbytes]

    def guards_intact(self):
        mask = torch.ones(self.buf.numel(), dtype=torch.bool, device="cuda")
        for start, n in self.payloads:
            mask[start:start + n] = False
        return bool((self.buf[mask] == SENTINEL).all())


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("flags,n_chunks,avg_m", [(0, 0, False), (0x2 | 0x4, 0, False), (0x8 | 0x4, 0, False), (0x10, 0, False),
                                                 (0x8 | 0x4 | 0x100 | 0x400, 3, False), (0x8 | 0x4 | 0x100 | 0x400, 2, True),
                                                 (0, 0, True)])
@pytest.mark.parametrize("P,ld", [(4096 * 2 + 13, 4096 * 2 + 16), (1001, 1001), (7, 8)])
def test_guard_zones_and_padding_survive(dtype, flags, n_chunks, avg_m, P, ld):
    from paper_2006_00441_b200 import binding as B
    K, tau, d, n_slots, T = 3, 1, 2, 2, 9
    gsz = 2 if dtype else 4
    arena = Arena(64 * 1024 + (K * ld * 4) * (2 + 2 * n_slots) + 2 * n_slots * ld * 4 + K * ld * (2 + gsz) + 24 * GUARD)
    def f32(n): return arena.carve(n * 4).view(torch.float32)
    w, m = f32(K * ld), f32(K * ld)
    snap, mean = f32(n_slots * K * ld), f32(n_slots * ld)
    m_snap, m_mean = (f32(n_slots * K * ld), f32(n_slots * ld)) if avg_m else (None, None)
    w_lp = arena.carve(K * ld * 2).view(torch.bfloat16) if dtype else None
    g = arena.carve(K * ld * gsz).view(torch.bfloat16 if dtype else torch.float32)
    PAD = 123.0
    for t in (w, m, snap, mean, g) + ((w_lp,) if dtype else ()) + ((m_snap, m_mean) if avg_m else ()):
        t.fill_(PAD)
    w.view(K, ld)[:, :P] = inputs.shared_start(1, P, 0.1).cuda()
    m.view(K, ld)[:, :P] = 0
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    cfg = B.dasgd_config()
    cfg.K, cfg.tau, cfg.d, cfg.dtype, cfg.merge_mode, cfg.n_slots, cfg.flags = K, tau, d, dtype, 0, n_slots, flags
    cfg.device, cfg.P, cfg.ld, cfg.xi, cfg.momentum, cfg.weight_decay = 0, P, ld, 0.25, 0.9, 1e-3
    cfg.w, cfg.m, cfg.snap, cfg.mean = w.data_ptr(), m.data_ptr(), snap.data_ptr(), mean.data_ptr()
    cfg.w_lp = w_lp.data_ptr() if dtype else None
    cfg.main_stream, cfg.side_stream = main.cuda_stream, side.cuda_stream
    cfg.n_chunks = n_chunks
    torch.cuda.synchronize()
    ctx = B.dasgd_init(cfg)
    if avg_m:
        B.dasgd_set_momentum_averaging(ctx, m_snap.data_ptr(), m_mean.data_ptr())
    gd = torch.bfloat16 if dtype else torch.float32
    for t in range(T):
        g.view(K, ld)[:, :P] = inputs.grad_block(2, t, K, P, 0.1, dtype=gd).cuda()
        torch.cuda.synchronize()
        B.dasgd_step(ctx, g.data_ptr(), 0.05)
        B.dasgd_sync(ctx)
    B.dasgd_destroy(ctx)
    assert arena.guards_intact()
    if ld > P:   # padding columns of every [K][ld] array keep their fill value
        for t in (w, m, g) + ((w_lp,) if dtype else ()):
            assert bool((t.view(K, ld)[:, P:].float() == PAD).all())
        assert bool((snap.view(n_slots, K, ld)[:, :, P:] == PAD).all())
        assert bool((mean.view(n_slots, ld)[:, P:] == PAD).all())
        if avg_m:
            assert bool((m_snap.view(n_slots, K, ld)[:, :, P:] == PAD).all())
            assert bool((m_mean.view(n_slots, ld)[:, P:] == PAD).all())
    assert torch.isfinite(w.view(K, ld)[:, :P]).all()
