"""Pins for the CPU oracle that do not come from the oracle itself.

Each test checks the oracle against something the paper or plain mathematics
fixes: the minibatch-SGD and Local-SGD special cases, the averaged-model
recursion (Section III-C-1), the deviation contraction used in the theorem's
proof, a literal evaluation of the matrix form of the update rule in exact
rational arithmetic, closed forms, torch.optim.SGD and torch's bfloat16 cast.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import BF16_MASTER_F32, MERGE_DELTA, OracleDaSGD


def rng_grads(T, K, P, seed=0, scale=1.0):
    r = np.random.default_rng(seed)
    return (r.standard_normal((T, K, P)) * scale).astype(np.float32)


def run(o, G, lr, record_every_step=True):
    out = []
    for t in range(G.shape[0]):
        o.step(G[t], lr)
        out.append(o.w.astype(np.float64))
    return out


# ---------------------------------------------------------------- special cases

def test_minibatch_sgd_equivalence():
    """Eq. 1: d=0, tau=1, xi=0, shared start => every replica takes the SGD step on the mean gradient."""
    K, P, lr = 4, 33, 0.1
    G = rng_grads(3, K, P, 1)
    w0 = np.random.default_rng(2).standard_normal(P).astype(np.float32)
    o = OracleDaSGD(K, P, tau=1, d=0, xi=0.0)
    o.set_state(w0)
    ref = w0.astype(np.float64)
    for t in range(3):
        o.step(G[t], lr)
        ref = ref - np.float64(np.float32(lr)) * G[t].astype(np.float64).mean(axis=0)
        for k in range(K):
            np.testing.assert_allclose(o.w[k], ref, rtol=0, atol=3e-7)


def test_local_sgd_special_case():
    """Section II-C-3: d=0, xi=0 => after every tau-th step all replicas equal the mean of the stepped replicas."""
    K, P, tau, lr = 3, 17, 4, 0.05
    G = rng_grads(12, K, P, 3)
    o = OracleDaSGD(K, P, tau=tau, d=0, xi=0.0)
    o.set_state(np.zeros(P, np.float32))
    indep = np.zeros((K, P))
    for t in range(12):
        o.step(G[t], lr)
        indep = indep - np.float64(np.float32(lr)) * G[t]
        if (t + 1) % tau == 0:
            indep[:] = indep.mean(axis=0)
            assert np.ptp(o.w, axis=0).max() == 0.0
        np.testing.assert_allclose(o.w, indep, rtol=0, atol=1e-6)


@pytest.mark.parametrize("tau,d", [(1, 1), (2, 1), (4, 2), (1, 2), (3, 0)])
def test_xi_one_is_independent_sgd_and_matches_torch(tau, d):
    """xi=1 makes the merge a no-op: K independent runs.  The momentum / weight-decay
    local step must then agree with torch.optim.SGD (the usual form of the paper's platform)."""
    K, P, T, lr, mu, wd = 3, 29, 15, 0.1, 0.9, 0.01
    G = rng_grads(T, K, P, 4)
    w0 = np.random.default_rng(5).standard_normal((K, P)).astype(np.float32)
    o = OracleDaSGD(K, P, tau, d, xi=1.0, momentum=mu, weight_decay=wd)
    o.set_state(w0)
    p = torch.tensor(w0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=float(np.float32(lr)), momentum=float(np.float32(mu)),
                          weight_decay=float(np.float32(wd)))
    for t in range(T):
        o.step(G[t], lr)
        p.grad = torch.tensor(G[t], dtype=torch.float64)
        opt.step()
        np.testing.assert_allclose(o.w, p.detach().numpy(), rtol=2e-6, atol=2e-6)
    buf = opt.state[p]["momentum_buffer"].numpy()
    np.testing.assert_allclose(o.m, buf, rtol=2e-6, atol=2e-6)


def test_identical_replicas_stay_identical_and_mean_is_identity():
    K, P, T = 5, 11, 9
    g1 = rng_grads(T, 1, P, 6)
    G = np.repeat(g1, K, axis=1)
    o = OracleDaSGD(K, P, tau=2, d=1, xi=0.25, momentum=0.9, weight_decay=1e-2)
    o.set_state(np.random.default_rng(7).standard_normal(P).astype(np.float32))
    for t in range(T):
        o.step(G[t], 0.1)
        w = o.w
        assert np.ptp(w, axis=0).max() == 0.0
        if o.n_pending:
            s, snap, mean = o.pending(o.n_pending - 1)
            np.testing.assert_array_equal(mean, snap[0])  # averaging equal values is exact


# -------------------------------------------- averaged-model recursion (Sec. III-C-1)

@pytest.mark.parametrize("K,tau,d,xi", [(2, 2, 1, 0.25), (4, 4, 1, 0.25), (8, 4, 2, 0.25), (3, 3, 2, 0.5),
                                        (4, 1, 1, 0.25), (5, 2, 2, 0.75), (4, 3, 3, 0.0), (4, 4, 3, 0.0)])
def test_mean_recursion(K, tau, d, xi):
    """mu_{a+tau} = mu_a - eta*[sum_{i<tau-d} gbar_{a+i} + xi*sum_{tau-d<=i<tau} gbar_{a+i}] at merge times
    a = s+d, and the first period mu_{tau+d} = mu_0 - eta*[sum_{u<tau} gbar_u + xi*sum_{tau<=u<tau+d} gbar_u]."""
    P, T, lr = 13, 5 * tau + d + 1, 0.125
    G = rng_grads(T, K, P, 8)
    gbar = G.astype(np.float64).mean(axis=1)
    w0 = np.random.default_rng(9).standard_normal(P).astype(np.float32)
    o = OracleDaSGD(K, P, tau, d, xi)
    o.set_state(w0)
    mus = [w0.astype(np.float64)] + [w.mean(axis=0) for w in run(o, G, lr)]
    xi_ = float(np.float32(xi))
    pred = mus[0] - lr * (gbar[:tau].sum(0) + xi_ * gbar[tau:tau + d].sum(0))
    np.testing.assert_allclose(mus[tau + d], pred, rtol=0, atol=2e-6)
    a = tau + d
    checked = 0
    while a + tau <= T:
        pred = mus[a] - lr * (gbar[a:a + tau - d].sum(0) + xi_ * gbar[a + tau - d:a + tau].sum(0))
        np.testing.assert_allclose(mus[a + tau], pred, rtol=0, atol=2e-6)
        a += tau
        checked += 1
    assert checked >= 3


def test_mean_frozen_when_xi_zero_and_d_equals_tau():
    """Consequence of the recursion: xi=0 and d=tau => the mean stops moving after the first period."""
    K, P, tau = 4, 7, 2
    G = rng_grads(12, K, P, 10)
    o = OracleDaSGD(K, P, tau, tau, xi=0.0)
    o.set_state(np.zeros(P, np.float32))
    mus = [w.mean(axis=0) for w in run(o, G, 0.1)]
    for a in range(2 * tau, 12, tau):
        np.testing.assert_allclose(mus[a + tau - 1], mus[a - 1], rtol=0, atol=1e-6)


@pytest.mark.parametrize("tau,d", [(4, 1), (3, 2), (1, 2), (2, 3)])
def test_mean_does_plain_sgd_between_merges(tau, d):
    K, P, T, lr = 4, 9, 14, 0.1
    G = rng_grads(T, K, P, 11)
    o = OracleDaSGD(K, P, tau, d, 0.25)
    o.set_state(np.zeros(P, np.float32))
    prev = np.zeros(P)
    for t in range(T):
        o.step(G[t], lr)
        u = t + 1
        mu = o.w.astype(np.float64).mean(axis=0)
        merged = d > 0 and u - d >= tau and (u - d) % tau == 0
        if not merged:
            np.testing.assert_allclose(mu, prev - np.float64(np.float32(lr)) * G[t].astype(np.float64).mean(0),
                                       rtol=0, atol=1e-6)
        prev = mu


@pytest.mark.parametrize("xi", [0.0, 0.25, 0.5, 1.0])
def test_deviation_contracts_by_xi_at_each_merge(xi):
    """Proof of the theorem: X(J-I) right after a merge = xi * (stepped state)(J-I)."""
    K, P, tau, d, lr = 4, 10, 3, 1, 0.1
    G = rng_grads(13, K, P, 12)
    o = OracleDaSGD(K, P, tau, d, xi)
    o.set_state(np.zeros(P, np.float32))
    n = 0
    for t in range(13):
        u = t + 1
        before = o.w.astype(np.float64)
        o.step(G[t], lr)
        if u - d >= tau and (u - d) % tau == 0:
            y = before - np.float64(np.float32(lr)) * G[t]
            dev_y = y - y.mean(0)
            w = o.w.astype(np.float64)
            np.testing.assert_allclose(w - w.mean(0), xi * dev_y, rtol=0, atol=1e-6)
            n += 1
    assert n == 4


def test_delta_merge_keeps_mean_on_plain_sgd():
    """merge_mode 1 (not in the paper): w + (mean - snap) leaves the replica mean equal to the stepped mean."""
    K, P, tau, d, lr = 4, 6, 2, 1, 0.1
    G = rng_grads(9, K, P, 13)
    o = OracleDaSGD(K, P, tau, d, 0.25, merge_mode=MERGE_DELTA)
    o.set_state(np.zeros(P, np.float32))
    mu = np.zeros(P)
    for t in range(9):
        o.step(G[t], lr)
        mu = mu - np.float64(np.float32(lr)) * G[t].astype(np.float64).mean(0)
        np.testing.assert_allclose(o.w.astype(np.float64).mean(0), mu, rtol=0, atol=1e-6)


def test_p_slicing_commutes():
    K, P, T = 3, 40, 11
    G = rng_grads(T, K, P, 14)
    w0 = np.random.default_rng(15).standard_normal(P).astype(np.float32)
    idx = np.array([0, 3, 4, 17, 39])
    full = OracleDaSGD(K, P, 2, 1, 0.25, 0.9, 1e-3)
    part = OracleDaSGD(K, len(idx), 2, 1, 0.25, 0.9, 1e-3)
    full.set_state(w0)
    part.set_state(w0[idx])
    for t in range(T):
        full.step(G[t], 0.1)
        part.step(np.ascontiguousarray(G[t][:, idx]), 0.1)
    np.testing.assert_array_equal(full.w[:, idx], part.w)
    np.testing.assert_array_equal(full.m[:, idx], part.m)


# --------------------------- literal matrix form, exact rationals, full history

def brute_force_history(W0, G, tau, d, xi, lr):
    """X_{u} from the matrix form of the update rule (Appendix, "Matrix Representation"),
    keeping every iterate: a merge at u reads the iterate of u-d from history and
    right-multiplies it by J = 11^T/M.  Exact arithmetic (Fractions)."""
    K, P = W0.shape
    xi, lr = Fraction(xi), Fraction(lr)
    X = [[[Fraction(float(W0[k, p])) for p in range(P)] for k in range(K)]]
    for t in range(G.shape[0]):
        u = t + 1
        Y = [[X[t][k][p] - lr * Fraction(float(G[t, k, p])) for p in range(P)] for k in range(K)]
        if d > 0 and u - d >= tau and (u - d) % tau == 0:
            old = X[u - d]
            mean = [sum(old[k][p] for k in range(K)) / K for p in range(P)]
            Y = [[xi * Y[k][p] + (1 - xi) * mean[p] for p in range(P)] for k in range(K)]
        X.append(Y)
    return X


@pytest.mark.parametrize("K,tau,d,xi", [(2, 2, 1, 0.25), (4, 3, 1, 0.5), (2, 4, 3, 0.25), (4, 3, 2, 0.75),
                                        (3, 2, 1, 0.25), (2, 1, 1, 0.5), (2, 1, 2, 0.25), (4, 2, 3, 0.5)])
def test_against_exact_history_form(K, tau, d, xi):
    P, T, lr = 8, 9, 0.5
    r = np.random.default_rng(16)
    G = r.integers(-4, 5, size=(T, K, P)).astype(np.float32)
    W0 = np.repeat(r.integers(-2, 3, size=(1, P)).astype(np.float32), K, axis=0)
    X = brute_force_history(W0, G, tau, d, xi, lr)
    o = OracleDaSGD(K, P, tau, d, xi)
    o.set_state(W0)
    for t in range(T):
        o.step(G[t], lr)
        want = np.array([[float(v) for v in row] for row in X[t + 1]])
        if K in (2, 4):  # every value is a short dyadic rational: the oracle must be exact
            np.testing.assert_array_equal(o.w.astype(np.float64), want)
        else:
            np.testing.assert_allclose(o.w, want, rtol=0, atol=2e-6)


# ------------------------------------------------------------------ closed forms

def test_momentum_closed_form_constant_gradient():
    """m_t = g(1-mu^t)/(1-mu);  w_T = w_0 - eta*g*sum_t (1-mu^t)/(1-mu)."""
    mu, lr, g, T = 0.5, 0.25, 3.0, 10
    o = OracleDaSGD(1, 1, tau=4, d=1, xi=1.0, momentum=mu)  # xi=1: the merge is a no-op
    o.set_state(np.array([[2.0]], np.float32))
    for _ in range(T):
        o.step(np.array([[g]], np.float32), lr)
    m_T = g * (1 - mu**T) / (1 - mu)
    w_T = 2.0 - lr * g * sum((1 - mu**t) / (1 - mu) for t in range(1, T + 1))
    assert o.m[0, 0] == np.float32(m_T)
    assert o.w[0, 0] == np.float32(w_T)


def test_weight_decay_closed_form_zero_gradient():
    """With g = 0 and no momentum, coupled L2 decay gives w_T = w_0 (1 - eta*lambda)^T."""
    lr, wd, T = 0.5, 0.25, 6
    o = OracleDaSGD(2, 3, tau=2, d=1, xi=1.0, weight_decay=wd)  # xi=1: the merge is a no-op
    o.set_state(np.full((2, 3), 8.0, np.float32))
    for _ in range(T):
        o.step(np.zeros((2, 3), np.float32), lr)
    assert np.all(o.w == np.float32(8.0 * (1 - lr * wd) ** T))


# ------------------------------------------------------------------ variants of the local step

def _torch_sgd_run(w0, G, lr, mu, wd, nesterov=False, scale_weights_by=None):
    p = torch.tensor(w0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=float(np.float32(lr)), momentum=float(np.float32(mu)),
                          weight_decay=float(np.float32(wd)), nesterov=nesterov)
    for t in range(G.shape[0]):
        if scale_weights_by is not None:
            with torch.no_grad():
                p.mul_(scale_weights_by)
        p.grad = torch.tensor(G[t], dtype=torch.float64)
        opt.step()
    return p.detach().numpy()


def test_nesterov_matches_torch():
    K, P, T, lr, mu, wd = 2, 23, 12, 0.1, 0.9, 0.01
    G = rng_grads(T, K, P, 30)
    w0 = np.random.default_rng(31).standard_normal((K, P)).astype(np.float32)
    o = OracleDaSGD(K, P, 3, 1, xi=1.0, momentum=mu, weight_decay=wd, nesterov=True)
    o.set_state(w0)
    for t in range(T):
        o.step(G[t], lr)
    np.testing.assert_allclose(o.w, _torch_sgd_run(w0, G, lr, mu, wd, nesterov=True), rtol=3e-6, atol=3e-6)
    plain = OracleDaSGD(K, P, 3, 1, xi=1.0, momentum=mu, weight_decay=wd)
    plain.set_state(w0)
    for t in range(T):
        plain.step(G[t], lr)
    assert np.abs(plain.w - o.w).max() > 1e-3          # the variant is not a no-op


@pytest.mark.parametrize("mu,nesterov", [(0.9, False), (0.0, False), (0.5, True)])
def test_decoupled_weight_decay_matches_scaled_weights_then_torch(mu, nesterov):
    """w <- w - eta*lambda*w - eta*dir  ==  scale the weights by (1 - eta*lambda), then an SGD step without decay."""
    K, P, T, lr, wd = 2, 19, 10, 0.1, 0.05
    G = rng_grads(T, K, P, 32)
    w0 = np.random.default_rng(33).standard_normal((K, P)).astype(np.float32)
    o = OracleDaSGD(K, P, 2, 1, xi=1.0, momentum=mu, weight_decay=wd, decoupled_wd=True, nesterov=nesterov)
    o.set_state(w0)
    for t in range(T):
        o.step(G[t], lr)
    scale = 1.0 - float(np.float32(lr)) * float(np.float32(wd))
    want = _torch_sgd_run(w0, G, lr, mu, 0.0, nesterov=nesterov, scale_weights_by=scale)
    np.testing.assert_allclose(o.w, want, rtol=3e-6, atol=3e-6)


def test_decoupled_weight_decay_closed_form_with_momentum():
    """Zero gradients: decoupled decay shrinks w by (1 - eta*lambda) per step whatever the momentum
    (the coupled form would not, because the decay term accumulates in the momentum buffer)."""
    lr, wd, T = 0.5, 0.25, 6
    o = OracleDaSGD(1, 2, 2, 1, xi=1.0, momentum=0.9, weight_decay=wd, decoupled_wd=True)
    o.set_state(np.full((1, 2), 8.0, np.float32))
    for _ in range(T):
        o.step(np.zeros((1, 2), np.float32), lr)
    assert np.all(o.w == np.float32(8.0 * (1 - lr * wd) ** T))
    assert np.all(o.m == 0.0)
    with pytest.raises(Exception):
        OracleDaSGD(1, 2, 2, 1, xi=1.0, momentum=0.0, nesterov=True)


# ------------------------------------------------------------------ bf16 mode

def test_bf16_rounding_matches_torch_cast():
    vals = np.array([1.0, 1.00390625, 1.0078125, 1.01171875, -1.00390625, 3.1415927, 1e-30, -2.5e38,
                     0.0, 65504.0, 1.0 + 2**-8 + 2**-20, 1.0 + 2**-8 - 2**-20], np.float32)
    r = np.random.default_rng(17).standard_normal(5000).astype(np.float32)
    w = np.concatenate([vals, r])[None, :]
    o = OracleDaSGD(1, w.shape[1], 1, 1, 1.0, dtype=BF16_MASTER_F32)
    o.set_state(w)
    want = torch.tensor(w).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(o.w_lp, want)


def test_bf16_mode_master_equals_f32_run_on_widened_gradients():
    """bf16 gradients widen exactly, so the fp32 master must equal an fp32-mode run fed the widened values,
    and the low-precision copy must be the cast of the master after steps and merges alike."""
    K, P, T = 4, 50, 7
    g32 = rng_grads(T, K, P, 18, 0.01)
    g16 = torch.tensor(g32).to(torch.bfloat16)
    gw = g16.to(torch.float32).numpy()
    gb = g16.view(torch.int16).numpy().view(np.uint16)
    w0 = (np.random.default_rng(19).standard_normal(P) * 0.02).astype(np.float32)
    a = OracleDaSGD(K, P, 2, 1, 0.25, 0.9, 0.0, dtype=BF16_MASTER_F32)
    b = OracleDaSGD(K, P, 2, 1, 0.25, 0.9, 0.0)
    a.set_state(w0)
    b.set_state(w0)
    for t in range(T):
        a.step(gb[t], 1e-3)
        b.step(gw[t], 1e-3)
        np.testing.assert_array_equal(a.w, b.w)
        want = torch.tensor(a.w).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        np.testing.assert_array_equal(a.w_lp, want)


# ------------------------------------------------------------------ schedule bookkeeping

@pytest.mark.parametrize("tau,d", [(1, 1), (1, 2), (2, 3), (4, 1), (2, 2), (3, 0)])
def test_pending_queue_depth_and_explicit_calls_match_step(tau, d):
    """The explicit call sequence (local_step, merge, snapshot, average) reproduces step()."""
    K, P, T = 2, 5, 13
    G = rng_grads(T, K, P, 20)
    a = OracleDaSGD(K, P, tau, d, 0.25, 0.5)
    b = OracleDaSGD(K, P, tau, d, 0.25, 0.5)
    for t in range(T):
        a.step(G[t], 0.1)
        b.local_step(G[t], 0.1)
        u = t + 1
        if d > 0 and u - d >= tau and (u - d) % tau == 0:
            b.merge()
        if u % tau == 0:
            b.snapshot()
            b.average()
            if d == 0:
                b.merge()
        np.testing.assert_array_equal(a.w, b.w)
        assert a.n_pending == b.n_pending <= max(1, -(-d // tau))


# ---------------------------------------------------------------- momentum averaging (a variant, not in the paper)

def _independent_period(w, m, G, lr, mu):
    """tau plain momentum-SGD steps of every worker from the state (w, m): a run with xi = 1 (no merge acts)."""
    K, P = w.shape
    o = OracleDaSGD(K, P, tau=G.shape[0] + 1, d=1, xi=1.0, momentum=mu)
    o.set_state(w, m)
    for t in range(G.shape[0]):
        o.step(G[t], lr)
    return o.w.astype(np.float64), o.m.astype(np.float64)


@pytest.mark.parametrize("xi", [0.0, 0.25, 1.0])
def test_momentum_averaging_without_delay_blends_both_halves_of_the_state(xi):
    """d = 0: right after a merge, w_k = xi*w_k' + (1-xi)*mean(w') and m_k = xi*m_k' + (1-xi)*mean(m'), where the
    primed state is what tau independent momentum-SGD steps give (taken from runs in which no merge acts).
    xi = 0: every worker then holds the same weights and the same buffer; any xi: the worker-mean of the buffers
    is untouched by the merge."""
    K, P, tau, lr, mu = 3, 19, 3, 0.1, 0.8
    G = rng_grads(3 * tau, K, P, 40)
    w = np.random.default_rng(41).standard_normal((K, P)).astype(np.float32)
    m = np.zeros((K, P), np.float32)
    o = OracleDaSGD(K, P, tau=tau, d=0, xi=xi, momentum=mu, average_momentum=True)
    o.set_state(w)
    for period in range(3):
        Gp = G[period * tau:(period + 1) * tau]
        for t in range(tau):
            o.step(Gp[t], lr)
        wp, mp = _independent_period(w, m, Gp, lr, mu)
        xi64 = np.float64(np.float32(xi))
        w_want = xi64 * wp + (1 - xi64) * wp.mean(axis=0)
        m_want = xi64 * mp + (1 - xi64) * mp.mean(axis=0)
        np.testing.assert_allclose(o.w, w_want, rtol=0, atol=2e-6)
        np.testing.assert_allclose(o.m, m_want, rtol=0, atol=2e-6)
        np.testing.assert_allclose(o.m.astype(np.float64).mean(axis=0), mp.mean(axis=0), rtol=0, atol=2e-6)
        if xi == 0.0:
            assert np.ptp(o.w, axis=0).max() == 0.0 and np.ptp(o.m, axis=0).max() == 0.0
        w, m = o.w, o.m


@pytest.mark.parametrize("tau,d", [(1, 1), (2, 1), (3, 2), (2, 2), (1, 2)])
def test_momentum_averaging_is_a_no_op_at_xi_one(tau, d):
    K, P, T = 3, 23, 12
    G = rng_grads(T, K, P, 42)
    w0 = np.random.default_rng(43).standard_normal((K, P)).astype(np.float32)
    a = OracleDaSGD(K, P, tau, d, xi=1.0, momentum=0.9, weight_decay=0.01, average_momentum=True)
    b = OracleDaSGD(K, P, tau, d, xi=1.0, momentum=0.9, weight_decay=0.01)
    a.set_state(w0); b.set_state(w0)
    for t in range(T):
        a.step(G[t], 0.1); b.step(G[t], 0.1)
    np.testing.assert_array_equal(a.w, b.w)
    np.testing.assert_array_equal(a.m, b.m)


@pytest.mark.parametrize("tau,d,xi", [(2, 1, 0.25), (3, 2, 0.5), (2, 2, 0.0), (1, 2, 0.25)])
def test_momentum_averaging_uses_the_stale_mean_of_the_buffers(tau, d, xi):
    """Zero gradients, no decay: a buffer only decays, m(t) = mu^t m(0), so the first merge (at step tau+d, of the
    snapshot taken at step tau) must give m_k = xi*mu^(tau+d)*m_k(0) + (1-xi)*mu^tau*mean(m(0)): the mean is the
    one of d steps ago, not the current one."""
    K, P, mu = 4, 9, 0.5
    r = np.random.default_rng(44)
    m0 = r.standard_normal((K, P)).astype(np.float32)
    o = OracleDaSGD(K, P, tau, d, xi=xi, momentum=mu, average_momentum=True)
    o.set_state(r.standard_normal((K, P)).astype(np.float32), m0)
    Z = np.zeros((K, P), np.float32)
    for t in range(tau + d):                   # no merge lands before step tau + d
        np.testing.assert_allclose(o.m, mu ** t * m0.astype(np.float64), rtol=0, atol=1e-6)
        o.step(Z, 0.1)
    xi64 = np.float64(np.float32(xi))
    want = xi64 * mu ** (tau + d) * m0.astype(np.float64) + (1 - xi64) * mu ** tau * m0.astype(np.float64).mean(axis=0)
    np.testing.assert_allclose(o.m, want, rtol=0, atol=1e-6)


@pytest.mark.parametrize("tau,d", [(2, 1), (1, 1), (3, 2), (1, 2)])
def test_momentum_averaging_delta_form_keeps_the_mean_buffer_on_its_plain_recursion(tau, d):
    """merge_mode 1: m_k <- m_k + (mean(m^) - m^_k) adds corrections that sum to zero over the workers, so the
    worker-mean of the buffers obeys mean_m <- mu*mean_m + mean(g) at every step, merges or not."""
    K, P, T, mu = 4, 13, 14, 0.7
    G = rng_grads(T, K, P, 45)
    o = OracleDaSGD(K, P, tau, d, xi=0.25, momentum=mu, merge_mode=MERGE_DELTA, average_momentum=True)
    o.set_state(np.random.default_rng(46).standard_normal((K, P)).astype(np.float32))
    mean_m = np.zeros(P)
    moved = False
    plain = OracleDaSGD(K, P, tau, d, xi=0.25, momentum=mu, merge_mode=MERGE_DELTA)
    plain.set_state(o.w)
    for t in range(T):
        o.step(G[t], 0.05); plain.step(G[t], 0.05)
        mean_m = np.float64(np.float32(mu)) * mean_m + G[t].astype(np.float64).mean(axis=0)
        np.testing.assert_allclose(o.m.astype(np.float64).mean(axis=0), mean_m, rtol=0, atol=5e-6)
        moved = moved or np.abs(o.m - plain.m).max() > 1e-3
    assert moved      # the buffers themselves do differ from the run without momentum averaging


def test_momentum_averaging_identical_workers():
    """Identical workers with identical gradients stay identical; with d = 0 the merge is then the identity and the
    run is plain momentum SGD (torch.optim.SGD)."""
    K, P, T, lr, mu = 3, 11, 10, 0.1, 0.9
    g1 = rng_grads(T, 1, P, 47)
    G = np.repeat(g1, K, axis=1)
    w0 = np.random.default_rng(48).standard_normal(P).astype(np.float32)
    for tau, d in [(2, 1), (1, 2), (2, 0)]:
        o = OracleDaSGD(K, P, tau, d, xi=0.25, momentum=mu, average_momentum=True)
        o.set_state(w0)
        p = torch.tensor(w0, dtype=torch.float64, requires_grad=True)
        opt = torch.optim.SGD([p], lr=float(np.float32(lr)), momentum=float(np.float32(mu)))
        for t in range(T):
            o.step(G[t], lr)
            p.grad = torch.tensor(g1[t, 0], dtype=torch.float64)
            opt.step()
            assert np.ptp(o.w, axis=0).max() == 0.0 and np.ptp(o.m, axis=0).max() == 0.0
            if d == 0:
                np.testing.assert_allclose(o.w[0], p.detach().numpy(), rtol=2e-6, atol=2e-6)


def test_momentum_averaging_needs_momentum_and_an_unsharded_worker_axis():
    from oracle import OracleError
    with pytest.raises(OracleError):
        OracleDaSGD(2, 4, 1, 1, 0.5, momentum=0.0, average_momentum=True)
    o = OracleDaSGD(2, 4, 1, 1, 0.5, momentum=0.9, average_momentum=True)
    with pytest.raises(OracleError):
        o.set_shard(4)


def test_momentum_averaging_delta_form_without_delay_equalises_the_buffers():
    """merge_mode 1 with d = 0: the snapshot is the current state, so m_k + (mean(m) - m_k) = mean(m) for every
    worker (and likewise for the weights): the sign of the correction matters here."""
    K, P, tau = 3, 7, 2
    G = rng_grads(6, K, P, 49)
    o = OracleDaSGD(K, P, tau, 0, xi=0.25, momentum=0.6, merge_mode=MERGE_DELTA, average_momentum=True)
    o.set_state(np.random.default_rng(50).standard_normal((K, P)).astype(np.float32))
    for t in range(6):
        before_m = o.m.astype(np.float64)
        o.step(G[t], 0.1)
        if (t + 1) % tau == 0:
            stepped = np.float64(np.float32(0.6)) * before_m + G[t]
            np.testing.assert_allclose(o.m, np.broadcast_to(stepped.mean(axis=0), (K, P)), rtol=0, atol=2e-6)
            np.testing.assert_allclose(np.ptp(o.w.astype(np.float64), axis=0), 0, atol=1e-6)


def test_momentum_averaging_mean_is_that_of_the_snapshot_not_of_later_buffers():
    """Explicit calls with a local step between the snapshot and its averaging: the mean must be the one of the
    buffers as they were at the snapshot."""
    K, P = 3, 5
    G = rng_grads(3, K, P, 51)
    o = OracleDaSGD(K, P, 4, 2, xi=0.5, momentum=0.9, average_momentum=True)
    o.set_state(np.zeros(P, np.float32))
    o.local_step(G[0], 0.1)
    o.snapshot()
    m_at_snapshot = o.m.astype(np.float64)
    o.local_step(G[1], 0.1)
    o.average()
    snap_m, mean_m = o.pending_momentum(0)
    np.testing.assert_array_equal(snap_m, m_at_snapshot.astype(np.float32))
    np.testing.assert_allclose(mean_m, m_at_snapshot.mean(axis=0), rtol=0, atol=1e-6)
    assert np.abs(o.m.astype(np.float64).mean(axis=0) - mean_m).max() > 1e-3
