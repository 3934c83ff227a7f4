"""The seeded input generators: determinism, slice consistency, distribution."""
import numpy as np
import pytest
import torch

from paper_2006_00441_b200 import inputs


def test_normal_moments_and_independence():
    c = torch.arange(1 << 20, dtype=torch.int64)
    z = inputs.normal_f32(0, 2, c, 1.0).double().numpy()
    assert abs(z.mean()) < 4e-3
    assert abs(z.std() - 1.0) < 4e-3
    kurt = ((z - z.mean()) ** 4).mean() / z.var() ** 2 - 3.0
    assert abs(kurt + 0.15) < 0.03          # Irwin-Hall, n = 8
    assert abs(np.corrcoef(z[:-1], z[1:])[0, 1]) < 4e-3
    z2 = inputs.normal_f32(1, 2, c, 1.0).double().numpy()
    z3 = inputs.normal_f32(0, 3, c, 1.0).double().numpy()
    assert abs(np.corrcoef(z, z2)[0, 1]) < 4e-3 and abs(np.corrcoef(z, z3)[0, 1]) < 4e-3


def test_counter_above_32_bits_changes_values():
    c = torch.arange(1000, dtype=torch.int64)
    a = inputs.normal_f32(0, 2, c, 1.0)
    b = inputs.normal_f32(0, 2, c + (1 << 32), 1.0)
    assert (a != b).float().mean() > 0.99


def test_grad_block_slice_equals_columns_of_full_block():
    K, P = 3, 1000
    full = inputs.grad_block(7, 5, K, P, 0.03)
    idx = [0, 1, 17, 500, 999]
    part = inputs.grad_block(7, 5, K, P, 0.03, p_index=idx)
    assert torch.equal(full[:, idx], part)
    other_t = inputs.grad_block(7, 6, K, P, 0.03)
    assert not torch.equal(full, other_t)
    assert abs(float(full.std()) - 0.03) < 2e-3
    chunked = inputs.grad_block(7, 5, K, P, 0.03, chunk=64)
    assert torch.equal(full, chunked)


def test_bf16_grad_block_is_cast_of_f32():
    a = inputs.grad_block(0, 0, 2, 64, 0.01)
    b = inputs.grad_block(0, 0, 2, 64, 0.01, dtype=torch.bfloat16)
    assert torch.equal(a.to(torch.bfloat16), b)


def test_linear_regression_gradient_is_the_loss_gradient():
    prob = inputs.LinearRegression(0, K=2, P=16, batch=8, dtype=torch.float64)
    w = torch.randn(2, 16, dtype=torch.float64, requires_grad=True)
    g = prob.grad(3, w.detach())
    tot = 0.0
    for k in range(2):
        X, y = prob.batch_xy(3, k)
        r = X.double() @ w[k] - y.double()
        tot = tot + 0.5 * (r * r).mean()
    tot.backward()
    assert torch.allclose(w.grad.float(), g, rtol=1e-5, atol=1e-6)


@pytest.mark.gpu
def test_generators_are_bit_identical_on_cpu_and_gpu():
    K, P = 4, 100_003
    for dt in (torch.float32, torch.bfloat16):
        a = inputs.grad_block(3, 9, K, P, 0.0316, dtype=dt)
        b = inputs.grad_block(3, 9, K, P, 0.0316, dtype=dt, device="cuda")
        assert torch.equal(a, b.cpu())
    assert torch.equal(inputs.shared_start(3, P, 0.02), inputs.shared_start(3, P, 0.02, device="cuda").cpu())
