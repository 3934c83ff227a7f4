"""Shared helpers of the GPU parity tests: drive libdasgd and the CPU oracle on the same inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import OracleDaSGD

TOL_STEP = 1e-6   # per element, one teacher-forced step:   |gpu - cpu| <= TOL_STEP * (1 + |cpu|)
TOL_RUN = 1e-4    # per element, after a free-running run:  |gpu - cpu| <= TOL_RUN  * (1 + |cpu|)


def assert_close(gpu, cpu, tol, what=""):
    gpu = np.asarray(gpu, dtype=np.float64)
    cpu = np.asarray(cpu, dtype=np.float64)
    assert gpu.shape == cpu.shape, f"{what}: shape {gpu.shape} vs {cpu.shape}"
    if gpu.size == 0:
        return
    err = np.abs(gpu - cpu) / (1.0 + np.abs(cpu))
    worst = float(err.max())
    assert np.isfinite(gpu).all(), f"{what}: non-finite GPU values"
    assert worst <= tol, f"{what}: max scaled error {worst:.3e} > {tol:.1e} at {np.unravel_index(err.argmax(), err.shape)}"


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def to_oracle_grad(g: torch.Tensor, P: int) -> np.ndarray:
    """[K, ld] device gradients -> the [K, P] host array the oracle wants (float32 or bf16 bits)."""
    g = g[:, :P].detach().cpu().contiguous()
    if g.dtype == torch.bfloat16:
        return g.view(torch.int16).numpy().view(np.uint16)
    return g.numpy()


def make_pair(B, K, P, tau, d, xi, momentum=0.0, weight_decay=0.0, dtype=0, merge_mode=0, flags=0,
              ld=None, n_slots=None, w0=None, n_chunks=0):
    """A libdasgd instance and an oracle with the same configuration and start point."""
    gpu = B.DaSGD(K, P, tau, d, xi, momentum, weight_decay, dtype=dtype, merge_mode=merge_mode, flags=flags,
                  ld=ld, n_slots=n_slots, n_chunks=n_chunks)
    cpu = OracleDaSGD(K, P, tau, d, xi, momentum, weight_decay, dtype=dtype, merge_mode=merge_mode,
                      nesterov=bool(flags & 0x20), decoupled_wd=bool(flags & 0x40))
    if w0 is not None:
        w0 = np.asarray(w0, np.float32)
        gpu.set_state(torch.from_numpy(w0))
        cpu.set_state(w0)
    return gpu, cpu


def padded_grad(g_kp: torch.Tensor, ld: int) -> torch.Tensor:
    """[K, P] -> contiguous [K, ld] CUDA tensor (padding filled with a sentinel that must never leak)."""
    K, P = g_kp.shape
    out = torch.full((K, ld), 7.0, dtype=g_kp.dtype, device="cuda")
    out[:, :P] = g_kp.to("cuda")
    return out


def state_of(gpu):
    gpu.sync()
    w = gpu.w[:, :gpu.P].cpu().numpy()
    m = gpu.m[:, :gpu.P].cpu().numpy() if gpu.m is not None else None
    return w, m
