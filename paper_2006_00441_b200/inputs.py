"""Seeded synthetic inputs for DaSGD workloads (gradients, start points, a
linear-regression problem).

This module holds none of the method's arithmetic: it only turns
``(seed, stream, counter)`` into numbers.  Everything is a pure function of its
arguments, written with integer torch ops whose results do not depend on the
device, so the same call on ``cpu`` and on ``cuda`` returns bit-identical
tensors.  That lets a host-side checker regenerate any slice of a workload that
was generated on the device, without copying it back.

Generator.  A 32-bit counter hash (two xor-shift/multiply rounds, constants
chosen here; all intermediates stay below 2**63 so int64 never overflows) is
evaluated four times per element; its eight 16-bit halves are summed.  The
centred sum (an Irwin-Hall variate, n = 8, excess kurtosis -0.15) converts to
float32 exactly and is scaled by ONE float32 multiply, so there is a single
rounding and it is the same on every IEEE-754 device.
"""
from __future__ import annotations

import math

import torch

_M32 = 0xFFFFFFFF
# odd multipliers below 2**31: (value < 2**32) * (mult < 2**31) < 2**63
_C1 = 0x2C9277B5
_C2 = 0x5F356495
_C3 = 0x3C6EF35F
_GOLD = 0x1E3779B9

# variance of the sum of eight independent uniforms on {0..65535}
_IH_N = 8
_IH_VAR = _IH_N * (65536.0**2 - 1.0) / 12.0
_IH_MEAN_X2 = _IH_N * 65535  # twice the mean, kept integer


def _mix(x: torch.Tensor) -> torch.Tensor:
    """One avalanche pass over int64 values in [0, 2**32)."""
    x = x ^ (x >> 15)
    x = (x * _C1) & _M32
    x = x ^ (x >> 13)
    x = (x * _C2) & _M32
    x = x ^ (x >> 16)
    return x


def _mix_int(x: int) -> int:
    x &= _M32
    x ^= x >> 15
    x = (x * _C1) & _M32
    x ^= x >> 13
    x = (x * _C2) & _M32
    x ^= x >> 16
    return x


def _key(seed: int, stream: int) -> int:
    return _mix_int(_mix_int(seed & _M32) ^ ((stream * _C3) & _M32) ^ _GOLD)


def hash_u32(seed: int, stream: int, counter: torch.Tensor, lane: int = 0) -> torch.Tensor:
    """32-bit hash of a 64-bit ``counter`` tensor (int64, non-negative)."""
    lo = counter & _M32
    hi = (counter >> 32) & _M32
    k = _key(seed, stream)
    h = _mix(hi ^ k)
    h = _mix(lo ^ h ^ ((lane * _GOLD) & _M32))
    return _mix((h + k) & _M32)


def irwin_hall_i32(seed: int, stream: int, counter: torch.Tensor) -> torch.Tensor:
    """Twice the centred sum of eight 16-bit uniforms (an even/odd-exact integer)."""
    acc = torch.zeros_like(counter)
    for lane in range(_IH_N // 2):
        h = hash_u32(seed, stream, counter, lane)
        acc = acc + (h & 0xFFFF) + (h >> 16)
    return 2 * acc - _IH_MEAN_X2


def normal_f32(seed: int, stream: int, counter: torch.Tensor, std: float) -> torch.Tensor:
    """Approximately N(0, std**2) float32 values, one per counter."""
    z = irwin_hall_i32(seed, stream, counter).to(torch.float32)  # |z| < 2**21: exact
    scale = torch.tensor(std / (2.0 * math.sqrt(_IH_VAR)), dtype=torch.float32,
                         device=counter.device)
    return z * scale


def _p_index(P: int, p_index, device) -> torch.Tensor:
    if p_index is None:
        return torch.arange(P, dtype=torch.int64, device=device)
    return torch.as_tensor(p_index, dtype=torch.int64, device=device)


def shared_start(seed: int, P: int, std: float, p_index=None, device="cpu",
                 stream: int = 1) -> torch.Tensor:
    """The common starting point ``w_0[p]`` (all replicas begin there)."""
    return normal_f32(seed, stream, _p_index(P, p_index, device), std)


def grad_block(seed: int, t: int, K: int, P: int, std: float, p_index=None,
               device="cpu", dtype=torch.float32, stream: int = 2,
               out: torch.Tensor | None = None, chunk: int = 1 << 24) -> torch.Tensor:
    """Synthetic gradients for step ``t``: ``g[k][j]`` for ``j`` over ``p_index``.

    The counter of element (t, k, p) is ``(t*K + k)*P + p`` whatever slice is
    asked for, so a slice equals the same columns of the full block.
    ``chunk`` bounds temporary memory.
    """
    p = _p_index(P, p_index, device)
    n = p.numel()
    if out is None:
        out = torch.empty((K, n), dtype=dtype, device=device)
    for k in range(K):
        base = (t * K + k) * P
        for a in range(0, n, chunk):
            b = min(n, a + chunk)
            out[k, a:b] = normal_f32(seed, stream, p[a:b] + base, std).to(dtype)
    return out


class LinearRegression:
    """Noisy linear-regression batches: ``y = X w* + eps`` per (step, worker).

    ``w* ~ N(0,1)``, ``X ~ N(0,1)`` of shape [batch, P], ``eps ~ N(0, noise_var)``.
    ``grad`` is the gradient of ``(1/2B)·||X w - y||^2`` — the model's
    forward/backward pass, which belongs to the workload, not to the optimiser.
    """

    def __init__(self, seed: int, K: int, P: int, batch: int, noise_var: float = 0.01,
                 device="cpu", dtype=torch.float32):
        self.seed, self.K, self.P, self.batch = seed, K, P, batch
        self.noise_std = math.sqrt(noise_var)
        self.device, self.dtype = device, dtype
        self.w_star = normal_f32(seed, 10, torch.arange(P, dtype=torch.int64, device=device), 1.0)

    def batch_xy(self, t: int, k: int):
        B, P = self.batch, self.P
        c = torch.arange(B * P, dtype=torch.int64, device=self.device) + (t * self.K + k) * B * P
        X = normal_f32(self.seed, 11, c, 1.0).reshape(B, P)
        e = normal_f32(self.seed, 12,
                       torch.arange(B, dtype=torch.int64, device=self.device) + (t * self.K + k) * B,
                       self.noise_std)
        # y is formed in float64 and rounded once so both devices agree bit for bit
        y = (X.double() @ self.w_star.double() + e.double()).to(torch.float32)
        return X, y

    def grad(self, t: int, w: torch.Tensor) -> torch.Tensor:
        """``g[k] = Xᵀ(X w[k] - y)/B`` for all K workers; computed in ``self.dtype``."""
        out = torch.empty((self.K, self.P), dtype=torch.float32, device=self.device)
        for k in range(self.K):
            X, y = self.batch_xy(t, k)
            Xc, yc, wk = X.to(self.dtype), y.to(self.dtype), w[k].to(self.dtype)
            out[k] = ((Xc.T @ (Xc @ wk - yc)) / self.batch).to(torch.float32)
        return out

    def loss(self, t: int, w: torch.Tensor) -> float:
        tot = 0.0
        for k in range(self.K):
            X, y = self.batch_xy(t, k)
            r = X.double() @ w[k].double() - y.double()
            tot += float((r * r).mean()) * 0.5
        return tot / self.K


class TeacherMLP:
    """Regression against a fixed random teacher: K replicas of a bias-free ``layers``-deep MLP
    (``hidden -> hidden``, ReLU between layers) whose weights live as rows of a ``[K, P]`` array,
    ``P = layers * hidden**2`` (layer ``l`` of replica ``k`` is ``w[k, l*H*H:(l+1)*H*H].view(H, H)``).

    ``forward_backward`` is the workload's forward/backward pass (batched matmuls, i.e. the GEMM
    library of the device the tensors live on); it returns the loss per replica and writes the
    weight gradients, in the layout of the parameters, into ``g_out``.
    """

    def __init__(self, seed: int, K: int, hidden: int, layers: int = 4, batch: int = 256,
                 device="cpu", dtype=torch.float32):
        self.seed, self.K, self.H, self.L, self.B = seed, K, hidden, layers, batch
        self.P = layers * hidden * hidden
        self.device, self.dtype = torch.device(device), dtype
        idx = torch.arange(self.P, dtype=torch.int64, device=self.device)
        self.teacher = normal_f32(seed, 7, idx, (1.0 / hidden) ** 0.5).to(dtype).view(layers, hidden, hidden)

    def student_init(self) -> torch.Tensor:
        """Shared start of all replicas, N(0, 2/H), float32 [P]."""
        idx = torch.arange(self.P, dtype=torch.int64, device=self.device)
        return normal_f32(self.seed, 8, idx, (2.0 / self.H) ** 0.5)

    def precompute_batches(self, n: int) -> None:
        """Keep ``n`` input batches and their teacher outputs resident; step ``t`` then uses batch
        ``t % n`` and the forward/backward pass does no input generation and no teacher pass."""
        self._ring = [(x, self._teacher_out(x)) for x in (self.batch_x(t) for t in range(n))]

    def batch_x(self, t: int) -> torch.Tensor:
        n = self.K * self.B * self.H
        c = torch.arange(n, dtype=torch.int64, device=self.device) + t * n
        return normal_f32(self.seed, 9, c, 1.0).to(self.dtype).view(self.K, self.B, self.H)

    def _teacher_out(self, x):
        h = x
        for l in range(self.L):
            h = h @ self.teacher[l].T
            if l + 1 < self.L:
                h = torch.relu(h)
        return h

    def forward_backward(self, t: int, w: torch.Tensor, g_out: torch.Tensor) -> torch.Tensor:
        """``w``, ``g_out``: ``[K, >=P]`` tensors of ``self.dtype`` (only the first P columns are used)."""
        K, H, L = self.K, self.H, self.L
        W = w[:, :self.P].unflatten(1, (L, H, H))          # view, replica stride kept
        G = g_out[:, :self.P].unflatten(1, (L, H, H))
        ring = getattr(self, "_ring", None)
        if ring:
            x, y = ring[t % len(ring)]
        else:
            x = self.batch_x(t)
            y = self._teacher_out(x)
        acts = [x]
        for l in range(L):
            z = torch.bmm(acts[-1], W[:, l].transpose(1, 2))
            acts.append(torch.relu(z) if l + 1 < L else z)
        diff = (acts[-1] - y).float()
        loss = 0.5 * (diff * diff).mean(dim=(1, 2))
        delta = (diff / (self.B * H)).to(self.dtype)        # d loss / d output
        for l in reversed(range(L)):
            G[:, l] = torch.bmm(delta.transpose(1, 2), acts[l])
            if l > 0:
                delta = torch.bmm(delta, W[:, l]) * (acts[l] > 0).to(self.dtype)
        return loss
