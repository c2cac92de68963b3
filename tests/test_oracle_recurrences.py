"""Pins for the oracle's recurrences, Eq. (parle_y)-(parle_x) of Section 3:
exact closed forms on a quadratic loss, the proximal limit of Section 2.3,
reduction to plain SGD and to Entropy-SGD (Eq. lesgd), exactness of the mean
(Section 3.1), replica symmetry, and planted-mistake checks."""
import math
from fractions import Fraction as Fr

import numpy as np
import pytest

from oracle import parle_oracle as po
import synth_inputs as si


# ---- closed form on f(y) = 1/2 lam y^2 (per coordinate), exact rationals ----
def closed_form_q(lam, eta_p, alpha, gamma, L):
    """z_L = q x and y_L = yL x after L inner steps started at y_0 = z_0 = x.

    Derivation: with m = 1 - eta'(lam + 1/gamma) and s = 1/(1 + gamma lam),
    y_j = (s + (1-s) m^j) x; summing the geometric series of the exponential
    average gives q."""
    m = 1 - eta_p * (lam + 1 / gamma)
    s = 1 / (1 + gamma * lam)
    yL = s + (1 - s) * m ** L
    q = alpha ** L + s * (1 - alpha ** L) + (1 - s) * (1 - alpha) * m * (m ** L - alpha ** L) / (m - alpha)
    return q, yL


CASES = [
    dict(lam=Fr(7, 10), eta=Fr(1, 10), eta_p=Fr(1, 10), alpha=Fr(3, 4), gamma=Fr(1), rho=Fr(1), L=5),
    dict(lam=Fr(13, 10), eta=Fr(1, 4), eta_p=Fr(1, 20), alpha=Fr(3, 4), gamma=Fr(3), rho=Fr(1, 2), L=25),
    dict(lam=Fr(1, 20), eta=Fr(1), eta_p=Fr(3, 10), alpha=Fr(1, 2), gamma=Fr(1, 4), rho=Fr(5), L=7),
]


@pytest.mark.parametrize("c", CASES)
def test_quadratic_closed_form_one_round(c):
    q, yL = closed_form_q(c["lam"], c["eta_p"], c["alpha"], c["gamma"], c["L"])
    hp = po.Hyper(float(c["eta"]), float(c["eta_p"]), float(c["alpha"]), float(c["gamma"]), float(c["rho"]))
    x0 = np.array([[1.5], [-0.25], [3.0]])
    xbar0 = np.array([0.4])                       # deliberately NOT the mean: tests the xbar term
    out = po.parle_round(x0, xbar0, po.quadratic_grad_fn([float(c["lam"])]), c["L"], hp)
    np.testing.assert_allclose(out["y"], float(yL) * x0, rtol=1e-13)
    np.testing.assert_allclose(out["z"], float(q) * x0, rtol=1e-13)
    ce = float(1 - c["eta"] * (1 - q) - c["eta"] / c["rho"])
    want_x = ce * x0 + float(c["eta"] / c["rho"]) * xbar0
    np.testing.assert_allclose(out["x"], want_x, rtol=1e-13)
    np.testing.assert_allclose(out["xbar"], want_x.mean(axis=0), rtol=1e-13)


def test_quadratic_closed_form_three_rounds_mean_contracts():
    # when xbar is the replica mean, one round maps xbar -> (1 - eta(1-q)) xbar
    c = CASES[0]
    q, _ = closed_form_q(c["lam"], c["eta_p"], c["alpha"], c["gamma"], c["L"])
    assert abs(float(q) - 0.853199426325) < 1e-12      # value worked out by hand for this case
    hp = po.Hyper(0.1, 0.1, 0.75, 1.0, 1.0)
    x = np.array([[1.0, -2.0], [0.5, 4.0], [-3.0, 0.25], [2.0, 2.0]])
    xbar = x.mean(axis=0)
    fn = po.quadratic_grad_fn([0.7, 0.7])
    f = float(1 - c["eta"] * (1 - q))
    for r in range(3):
        out = po.parle_round(x, xbar, fn, 5, hp)
        np.testing.assert_allclose(out["xbar"], f * xbar, rtol=1e-13)
        x, xbar = out["x"], out["xbar"]


def test_inner_loop_converges_to_the_proximal_point():
    # Section 2.3: y descends f(y) + |y-x|^2/(2 gamma); for f = 1/2 y^T A y the
    # minimiser is (I + gamma A)^{-1} x.  Dense symmetric A, many steps.
    rng = np.random.default_rng(4)
    Q, _ = np.linalg.qr(rng.normal(size=(6, 6)))
    A = Q @ np.diag([0.1, 0.5, 1.0, 1.5, 2.0, 3.0]) @ Q.T
    gamma = 0.8
    hp = po.Hyper(0.1, 0.05, 0.75, gamma, 1.0)
    x = rng.normal(size=(1, 6))
    out = po.parle_round(x, x[0], lambda a, l, y: (0.0, A @ y), 4000, hp)
    want = np.linalg.solve(np.eye(6) + gamma * A, x[0])
    np.testing.assert_allclose(out["y"][0], want, rtol=1e-12)
    # and the local-entropy gradient estimate (x - <y>)/gamma tends to A (I + gamma A)^{-1} x
    np.testing.assert_allclose((x[0] - out["z"][0]) / gamma, A @ want, rtol=1e-9)


def test_couplings_off_L1_is_plain_sgd():
    cfg = si.C1
    dims = cfg.dims
    X, c = si.round_batches(cfg.scaled(L=1), 0)
    x0 = np.stack([po.pack(si.init_replica(cfg, a)) for a in range(cfg.n)])
    hp = po.Hyper(eta=1.0, eta_prime=0.1, alpha=0.0, gamma=math.inf, rho=math.inf)
    out = po.parle_round(x0, x0.mean(axis=0), po.mlp_grad_fn(dims, X, c), 1, hp)
    for a in range(cfg.n):
        _, g = po.mlp_loss_grad(x0[a], dims, X[0, a], c[0, a])
        sgd = x0[a] - 0.1 * g                      # the one-line SGD step
        np.testing.assert_allclose(out["x"][a], sgd, rtol=0, atol=1e-15)
    # general alpha, eta: step size eta (1 - alpha) eta'
    hp = po.Hyper(eta=0.5, eta_prime=0.2, alpha=0.75, gamma=math.inf, rho=math.inf)
    out = po.parle_round(x0, x0.mean(axis=0), po.mlp_grad_fn(dims, X, c), 1, hp)
    for a in range(cfg.n):
        _, g = po.mlp_loss_grad(x0[a], dims, X[0, a], c[0, a])
        np.testing.assert_allclose(out["x"][a], x0[a] - 0.5 * 0.25 * 0.2 * g, rtol=0, atol=1e-15)


def test_single_replica_no_elastic_term_is_entropy_sgd():
    """n = 1 and 1/rho = 0 must reproduce Eq. (lesgd), coded here on its own
    with a running index k as the paper writes it."""
    cfg = si.C1.scaled(n=1, L=4)
    dims = cfg.dims
    eta, eta_p, alpha, gamma = 0.3, 0.1, 0.75, 2.0
    x = po.pack(si.init_replica(cfg, 0))
    xs_oracle = x[None].copy()
    xbar = x.copy()
    hp = po.Hyper(eta, eta_p, alpha, gamma, math.inf)
    batches = [si.round_batches(cfg, r) for r in range(3)]
    for r in range(3):
        X, c = batches[r]
        out = po.parle_round(xs_oracle, xbar, po.mlp_grad_fn(dims, X, c), cfg.L, hp)
        xs_oracle, xbar = out["x"], out["xbar"]
    # literal Eq. (lesgd)
    xk = x.copy(); yk = x.copy(); zk = x.copy()
    for k in range(3 * cfg.L):
        r, l = divmod(k, cfg.L)
        if l == 0:
            yk = xk.copy(); zk = xk.copy()
        X, c = batches[r]
        _, g = po.mlp_loss_grad(yk, dims, X[l, 0], c[l, 0])
        yk = yk - eta_p * (g + (yk - xk) / gamma)
        zk = alpha * zk + (1 - alpha) * yk
        if (k + 1) % cfg.L == 0:
            xk = xk - eta * (xk - zk)
    np.testing.assert_allclose(xs_oracle[0], xk, rtol=0, atol=1e-15)
    np.testing.assert_allclose(xbar, xk, rtol=0, atol=1e-15)      # n = 1: mean is the replica


def test_mean_is_exact_and_permutation_invariant():
    rng = np.random.default_rng(9)
    xs = rng.normal(size=(16, 257)) * np.logspace(-3, 3, 257)
    m = po.replica_mean(xs)
    want = np.array([math.fsum(xs[:, j]) / 16 for j in range(257)])   # exactly rounded sum
    scale = np.abs(xs).sum(axis=0) / 16           # error bound is relative to sum |x^a|, not to the sum
    assert np.all(np.abs(m - want) <= 1e-15 * scale)
    assert np.all(np.abs(po.replica_mean(xs[::-1]) - m) <= 1e-15 * scale)
    assert np.array_equal(po.replica_mean(np.tile(xs[:1], (2, 1))), xs[0])    # (v + v)/2 is exact
    np.testing.assert_allclose(po.replica_mean(np.tile(xs[:1], (8, 1))), xs[0], rtol=1e-15)


def test_after_a_round_xbar_is_the_mean_of_the_new_replicas():
    cfg = si.C1
    X, c = si.round_batches(cfg, 0)
    x0 = np.stack([po.pack(si.init_replica(cfg, a)) for a in range(cfg.n)])
    hp = po.Hyper(cfg.eta, cfg.eta_prime, cfg.alpha, cfg.gamma, cfg.rho)
    out = po.parle_round(x0, x0.mean(axis=0), po.mlp_grad_fn(cfg.dims, X, c), cfg.L, hp)
    want = np.array([math.fsum(out["x"][:, j]) / cfg.n for j in range(x0.shape[1])])
    assert np.all(np.abs(out["xbar"] - want) <= 1e-15 * np.abs(out["x"]).mean(axis=0) + 1e-300)
    # the simultaneous ("Jacobi") reading lags by one round instead
    outj = po.parle_round(x0, x0.mean(axis=0), po.mlp_grad_fn(cfg.dims, X, c), cfg.L, hp, jacobi_mean=True)
    np.testing.assert_allclose(outj["xbar"], x0.mean(axis=0), rtol=1e-15, atol=1e-18)
    np.testing.assert_array_equal(outj["x"], out["x"])


def test_identical_replicas_with_shared_batches_stay_identical():
    cfg = si.C1
    X, c = si.round_batches(cfg, 0, shared=True)
    one = po.pack(si.init_replica(cfg, 0))
    x = np.tile(one, (cfg.n, 1)); xbar = one.copy()
    hp = po.Hyper(cfg.eta, cfg.eta_prime, cfg.alpha, cfg.gamma, cfg.rho)
    for r in range(2):
        out = po.parle_round(x, xbar, po.mlp_grad_fn(cfg.dims, X, c), cfg.L, hp)
        x, xbar = out["x"], out["xbar"]
        for a in range(1, cfg.n):
            assert np.array_equal(x[a], x[0])
        # n = 3: (3v)/3 may differ from v by one rounding
        np.testing.assert_allclose(xbar, x[0], rtol=4e-16, atol=0)
    # elastic term vanished: same result as a single uncoupled replica
    hp1 = po.Hyper(cfg.eta, cfg.eta_prime, cfg.alpha, cfg.gamma, math.inf)
    x1 = one[None].copy(); xb1 = one.copy()
    for r in range(2):
        o1 = po.parle_round(x1, xb1, po.mlp_grad_fn(cfg.dims, X[:, :1], c[:, :1]), cfg.L, hp1)
        x1, xb1 = o1["x"], o1["xbar"]
    np.testing.assert_allclose(x[0], x1[0], rtol=1e-14, atol=1e-16)


def test_reading_flags_change_what_they_should():
    c = CASES[1]
    hp = po.Hyper(float(c["eta"]), float(c["eta_p"]), float(c["alpha"]), float(c["gamma"]), float(c["rho"]))
    x0 = np.array([[1.0], [2.0]]); xbar = np.array([1.5])
    fn = po.quadratic_grad_fn([float(c["lam"])])
    base = po.parle_round(x0, xbar, fn, 5, hp)
    q, _ = closed_form_q(c["lam"], c["eta_p"], c["alpha"], c["gamma"], 5)
    # coefficient eta/gamma on (x - z) instead of eta
    alt = po.parle_round(x0, xbar, fn, 5, hp, unscaled_lr=True)
    ce = float(1 - c["eta"] / c["gamma"] * (1 - q) - c["eta"] / c["rho"])
    np.testing.assert_allclose(alt["x"], ce * x0 + float(c["eta"] / c["rho"]) * xbar, rtol=1e-13)
    assert not np.allclose(alt["x"], base["x"])
    # z carried across rounds
    pers = po.parle_round(x0, xbar, fn, 5, hp, z_prev=np.zeros_like(x0), z_persist=True)
    a5 = float(c["alpha"]) ** 5
    np.testing.assert_allclose(pers["z"], base["z"] - a5 * x0, rtol=1e-13)


# ---- planted mistakes: each plausible slip must break a closed-form pin ----
@pytest.mark.parametrize("mutant", ["y_sign", "z_uses_old_y", "drop_elastic", "gamma_for_rho", "alpha_swapped"])
def test_planted_mistakes_break_the_closed_form(monkeypatch, mutant):
    c = CASES[1]
    hp = po.Hyper(float(c["eta"]), float(c["eta_p"]), float(c["alpha"]), float(c["gamma"]), float(c["rho"]))
    if mutant == "y_sign":
        monkeypatch.setattr(po, "inner_step", lambda y, z, x, g, h: (
            y - h.eta_prime * (g - h.inv_gamma * (y - x)),
            h.alpha * z + (1 - h.alpha) * (y - h.eta_prime * (g - h.inv_gamma * (y - x)))))
    elif mutant == "z_uses_old_y":
        monkeypatch.setattr(po, "inner_step", lambda y, z, x, g, h: (
            y - h.eta_prime * (g + h.inv_gamma * (y - x)), h.alpha * z + (1 - h.alpha) * y))
    elif mutant == "alpha_swapped":
        monkeypatch.setattr(po, "inner_step", lambda y, z, x, g, h: (
            y - h.eta_prime * (g + h.inv_gamma * (y - x)),
            (1 - h.alpha) * z + h.alpha * (y - h.eta_prime * (g + h.inv_gamma * (y - x)))))
    elif mutant == "drop_elastic":
        monkeypatch.setattr(po, "outer_step", lambda x, z, xb, h, u=False: x - h.eta * (x - z))
    elif mutant == "gamma_for_rho":
        monkeypatch.setattr(po, "outer_step", lambda x, z, xb, h, u=False: x - h.eta * (x - z) - h.eta * h.inv_gamma * (x - xb))
    with pytest.raises(AssertionError):
        test_quadratic_closed_form_one_round(c)


def test_scoping_schedule_closed_form_and_clipping():
    # Section 3.1: gamma_0 = 100, rho_0 = 1, clipped at 1 and 0.1
    B, L = 50, 25
    g, r = po.scoping(100.0, 1.0, B, 0, L)
    assert (g, r) == (100.0, 1.0)
    assert po.scoping(100.0, 1.0, B, L - 1, L) == (100.0, 1.0)          # constant inside a round
    g, r = po.scoping(100.0, 1.0, B, 7 * L + 3, L)
    assert abs(g - 100 * 0.99 ** 7) < 1e-12 and abs(r - 0.99 ** 7) < 1e-14
    # gamma hits its floor after ln(100)/-ln(0.99) = 458.2 rounds, rho after ln(10)/-ln(0.99) = 229.1
    assert po.scoping(100.0, 1.0, B, 458 * L, L)[0] > 1.0 and po.scoping(100.0, 1.0, B, 459 * L, L)[0] == 1.0
    assert po.scoping(100.0, 1.0, B, 229 * L, L)[1] > 0.1 and po.scoping(100.0, 1.0, B, 230 * L, L)[1] == 0.1
    seq = [po.scoping(100.0, 1.0, B, k * L, L) for k in range(600)]
    assert all(a[0] >= b[0] and a[1] >= b[1] for a, b in zip(seq, seq[1:]))
    # exact rational check of one value
    assert abs(po.scoping(3.0, 2.0, 2, 3, 1)[0] - float(Fr(3) * Fr(3, 4) ** 3)) < 1e-15


def test_momentum_round_matches_torch_nesterov_sgd():
    """The momentum form is pinned to an independent implementation: torch.optim.SGD(nesterov=True)
    stepping on the inner objective f(y) + |y - x|^2 / (2 gamma) (Section 2.3) and on the outer
    objective |x - z|^2 / 2 + |x - xbar|^2 / (2 rho), whose gradients are the directions of Eq. (parle)."""
    import torch
    rng = np.random.default_rng(12)
    d, n, L, mu = 7, 2, 6, 0.9
    A = rng.normal(size=(d, d)); A = A @ A.T / d
    hp = po.Hyper(eta=0.3, eta_prime=0.05, alpha=0.75, gamma=2.0, rho=0.5)
    x = rng.normal(size=(n, d)); xbar = x.mean(axis=0) + 0.1; vx = np.zeros((n, d))
    At = torch.tensor(A)
    tx = [torch.tensor(x[a].copy(), requires_grad=True) for a in range(n)]
    opt_x = [torch.optim.SGD([t], lr=hp.eta, momentum=mu, nesterov=True) for t in tx]
    txbar = torch.tensor(xbar.copy())
    for rnd in range(3):
        out = po.parle_round_momentum(x, xbar, vx, lambda a, l, y: (0.0, A @ y), L, hp, mu)
        for a in range(n):
            xa = tx[a].detach().clone()
            y = xa.clone().requires_grad_(True)
            z = xa.clone()
            opt_y = torch.optim.SGD([y], lr=hp.eta_prime, momentum=mu, nesterov=True)   # fresh buffer every round
            for l in range(L):
                opt_y.zero_grad()
                (0.5 * y @ At @ y + ((y - xa) ** 2).sum() / (2 * hp.gamma)).backward()
                opt_y.step()
                z = hp.alpha * z + (1 - hp.alpha) * y.detach()
            np.testing.assert_allclose(out["y"][a], y.detach().numpy(), rtol=1e-12, atol=1e-14)
            np.testing.assert_allclose(out["z"][a], z.numpy(), rtol=1e-12, atol=1e-14)
            opt_x[a].zero_grad()
            (0.5 * ((tx[a] - z) ** 2).sum() + ((tx[a] - txbar) ** 2).sum() / (2 * hp.rho)).backward()
            opt_x[a].step()                                                            # buffer persists across rounds
            np.testing.assert_allclose(out["x"][a], tx[a].detach().numpy(), rtol=1e-12, atol=1e-14)
        x, xbar, vx = out["x"], out["xbar"], out["vx"]
        txbar = torch.stack([t.detach() for t in tx]).mean(dim=0)
        np.testing.assert_allclose(xbar, txbar.numpy(), rtol=1e-13)


def test_zero_momentum_is_the_plain_round():
    cfg = si.C1
    X, c = si.round_batches(cfg, 0)
    x0 = np.stack([po.pack(si.init_replica(cfg, a)) for a in range(cfg.n)])
    hp = po.Hyper(cfg.eta, cfg.eta_prime, cfg.alpha, 2.0, 0.5)
    fn = po.mlp_grad_fn(cfg.dims, X, c)
    a = po.parle_round(x0, x0.mean(axis=0), fn, cfg.L, hp)
    b = po.parle_round_momentum(x0, x0.mean(axis=0), np.zeros_like(x0), fn, cfg.L, hp, 0.0)
    for k in ("x", "xbar", "y", "z"):
        np.testing.assert_allclose(b[k], a[k], rtol=1e-14, atol=1e-16)
