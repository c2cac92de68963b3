"""GPU parity of the streaming kernels (Eq. parle_y, parle_z, parle_xa,
parle_x) against the fp64 oracle, through the C ABI, on flat parameter
vectors: the quadratic-loss closed-form setting and the update-sweep shapes."""
import math

import numpy as np
import pytest
import torch

import paper_1707_00424_b200 as pb
import synth_inputs as si
from oracle import parle_oracle as po
from _util import rel_l2

pytestmark = pytest.mark.gpu
TOL = 1e-4          # fp32 state vs fp64 oracle, relative L2 (the paper-level bound for fp32 configs)
DEV = "cuda:0"


def _flat(n, d, **hyper):
    m = pb.Parle(n, (d,), 0, **hyper).alloc(DEV)
    return m


def _load(m, x, xbar):
    m.x.zero_(); m.xbar.zero_()
    m.x[:, :x.shape[1]].copy_(torch.from_numpy(x))
    m.xbar[:xbar.shape[0]].copy_(torch.from_numpy(xbar))


@pytest.mark.parametrize("n,d", [(1, 100), (3, 1000003), (16, 4097), (8, 32)])
def test_quadratic_rounds_match_oracle(n, d):
    hp = dict(eta=0.25, eta_prime=0.05, alpha=0.75, gamma=3.0, rho=0.5)
    L = 7
    lam = si.quadratic_spectrum(3, d)
    x0, _, _, _ = si.sweep_state(5, n, d)
    xbar0 = x0.astype(np.float64).mean(axis=0).astype(np.float32)
    m = _flat(n, d, **hp)
    _load(m, x0, xbar0)
    lam_dev = torch.zeros(m.stride, device=DEV); lam_dev[:d] = torch.from_numpy(lam.astype(np.float32))
    xo, xb = x0.astype(np.float64), xbar0.astype(np.float64)
    lam32 = lam.astype(np.float32).astype(np.float64)
    for rnd in range(3):
        m.round_begin()
        for l in range(L):
            cur = m.x if l == 0 else m.y              # y == x on the first step of a round
            g = cur * lam_dev                         # deterministic gradient of 1/2 y^T diag(lam) y
            m.inner_update(g)
        y_gpu, z_gpu = m.y.cpu().numpy()[:, :d], m.z.cpu().numpy()[:, :d]
        m.outer_step()
        torch.cuda.synchronize()
        out = po.parle_round(xo, xb, po.quadratic_grad_fn(lam32), L, po.Hyper(**hp))
        xo, xb = out["x"], out["xbar"]
        assert rel_l2(y_gpu, out["y"]) < TOL and rel_l2(z_gpu, out["z"]) < TOL
        assert rel_l2(m.x.cpu().numpy()[:, :d], xo) < TOL
        assert rel_l2(m.xbar.cpu().numpy()[:d], xb) < TOL
        # elementwise too (no reduction hides a misplaced element)
        np.testing.assert_allclose(m.x.cpu().numpy()[:, :d], xo, rtol=2e-5, atol=2e-6)
    assert m.status() == 0
    # padding stayed zero
    assert torch.all(m.x[:, d:] == 0) and torch.all(m.xbar[d:] == 0)


def test_sweep_shape_single_calls_match_oracle_elementwise():
    n, d = 3, 1 << 20
    x, y, z, g = si.sweep_state(11, n, d)
    hp = po.Hyper(eta=0.1, eta_prime=0.1, alpha=0.75, gamma=1.0, rho=1.0)
    m = _flat(n, d)
    xbar = x.astype(np.float64).mean(axis=0).astype(np.float32)
    _load(m, x, xbar)
    gd = torch.from_numpy(g).to(DEV)
    # first step of a round (reset folded in): y0 = z0 = x
    m.round_begin(); m.inner_update(gd)
    y1, z1 = po.inner_step(x.astype(np.float64), x.astype(np.float64), x.astype(np.float64), g.astype(np.float64), hp)
    np.testing.assert_allclose(m.y.cpu().numpy(), y1, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(m.z.cpu().numpy(), z1, rtol=1e-6, atol=1e-7)
    # steady-state step from arbitrary y, z
    m.y.copy_(torch.from_numpy(y)); m.z.copy_(torch.from_numpy(z))
    m.inner_update(gd)
    y2, z2 = po.inner_step(y.astype(np.float64), z.astype(np.float64), x.astype(np.float64), g.astype(np.float64), hp)
    np.testing.assert_allclose(m.y.cpu().numpy(), y2, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(m.z.cpu().numpy(), z2, rtol=1e-6, atol=1e-7)
    # outer step + mean
    m.outer_step(); torch.cuda.synchronize()
    xn = np.stack([po.outer_step(x[a].astype(np.float64), z2[a], xbar.astype(np.float64), hp) for a in range(n)])
    np.testing.assert_allclose(m.x.cpu().numpy(), xn, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(m.xbar.cpu().numpy(), po.replica_mean(xn), rtol=1e-6, atol=2e-7)
    # stand-alone mean after writing x directly
    m.x.copy_(torch.from_numpy(y)); m.mean(); torch.cuda.synchronize()
    np.testing.assert_allclose(m.xbar.cpu().numpy(), po.replica_mean(y.astype(np.float64)), rtol=1e-6, atol=2e-7)


def test_mean_invariants_and_determinism():
    n, d = 8, 70001
    x, y, z, g = si.sweep_state(2, n, d)
    m = _flat(n, d)
    _load(m, np.tile(x[:1], (n, 1)), np.zeros(d, np.float32))
    m.mean(); torch.cuda.synchronize()
    # identical replicas: the mean is the replica up to the roundings of the running sum (3v, 5v, ...)
    assert torch.allclose(m.xbar[:d], m.x[0, :d], rtol=3e-7, atol=0)
    m2 = _flat(2, d)
    _load(m2, np.tile(x[:1], (2, 1)), np.zeros(d, np.float32))
    m2.mean(); torch.cuda.synchronize()
    assert torch.equal(m2.xbar[:d], m2.x[0, :d])              # (v + v)/2 is exact
    runs = []
    for _ in range(2):
        _load(m, x, x.mean(axis=0))
        gd = torch.from_numpy(g).to(DEV)
        gp = torch.zeros_like(m.x); gp[:, :d] = gd
        m.round_begin(); m.inner_update(gp); m.inner_update(gp); m.outer_step(); torch.cuda.synchronize()
        runs.append((m.x.clone(), m.xbar.clone(), m.y.clone(), m.z.clone()))
    for a, b in zip(*runs):
        assert torch.equal(a, b)                              # bit-identical: no atomics, fixed order


def test_buffers_outside_the_state_are_untouched():
    n, d = 3, 5000
    m = pb.Parle(n, (d,), 0)
    S, pad = m.stride, 256
    bufs = [torch.full((n * S + 2 * pad,), 7.5, device=DEV) for _ in range(4)]
    xb = torch.full((S + 2 * pad,), 7.5, device=DEV)
    ws = torch.empty(m.workspace_bytes, dtype=torch.uint8, device=DEV)
    views = [b[pad:pad + n * S].view(n, S) for b in bufs]
    for v in views:
        v.normal_()
    m.bind(views[0], views[1], views[2], views[3], xb[pad:pad + S], ws)
    m.round_begin(); m.inner_update(views[3]); m.inner_update(views[3]); m.outer_step(); m.mean()
    torch.cuda.synchronize()
    for b in bufs + [xb]:
        assert torch.all(b[:pad] == 7.5) and torch.all(b[-pad:] == 7.5)


def test_couplings_off_and_state_errors_and_nan_flag():
    n, d = 2, 64
    m = _flat(n, d, gamma=math.inf, rho=math.inf, eta=1.0, alpha=0.0, eta_prime=0.5)
    x, _, _, g = si.sweep_state(4, n, d)
    _load(m, x, np.zeros(d, np.float32))
    with pytest.raises(pb.ParleError) as e:
        m.inner_update(m.grad)                                 # no round open
    assert e.value.code == -5
    m.round_begin()
    with pytest.raises(pb.ParleError) as e:
        m.outer_step()                                         # round without an inner step
    assert e.value.code == -5
    gp = torch.zeros_like(m.x); gp[:, :d] = torch.from_numpy(g).to(DEV)
    m.inner_update(gp); m.outer_step(); torch.cuda.synchronize()
    # both couplings off, L = 1, alpha = 0, eta = 1: exactly one SGD step of size eta'
    np.testing.assert_allclose(m.x.cpu().numpy()[:, :d], x - 0.5 * g, rtol=1e-6, atol=1e-7)
    assert m.status() == 0
    gp[0, 3] = float("nan")
    m.round_begin(); m.inner_update(gp); torch.cuda.synchronize()
    assert m.status() & pb.FLAG_NONFINITE
    m.clear_status(); assert m.status() == 0


def test_bind_rejects_misaligned_and_small_buffers():
    m = pb.Parle(2, (100,), 0)
    S = m.stride
    big = torch.zeros(2 * S + 64, device=DEV)
    ok = lambda: torch.zeros(2, S, device=DEV)
    ws = torch.empty(max(m.workspace_bytes, 1024), dtype=torch.uint8, device=DEV)
    with pytest.raises(pb.ParleError) as e:
        m.bind(big[1:1 + 2 * S].view(2, S), ok(), ok(), ok(), torch.zeros(S, device=DEV), ws)
    assert e.value.code == -3
    with pytest.raises(pb.ParleError) as e:
        m.bind(ok(), ok(), ok(), ok(), torch.zeros(S, device=DEV), ws[:16])
    assert e.value.code == -6


def test_momentum_rounds_on_a_quadratic_match_oracle():
    """Nesterov momentum on the y and x^a steps (Remark, Section 3.1) through parle_inner_update /
    parle_outer_step on flat vectors, three rounds (vy restarts every round, vx carries over)."""
    n, d, L, mu = 3, 4099, 5, 0.9
    hp = dict(eta=0.2, eta_prime=0.05, alpha=0.75, gamma=2.0, rho=0.5)
    lam = si.quadratic_spectrum(9, d)
    x0, _, _, _ = si.sweep_state(6, n, d)
    m = _flat(n, d, **hp)
    xbar0 = x0.astype(np.float64).mean(axis=0).astype(np.float32)
    _load(m, x0, xbar0)
    with pytest.raises(pb.ParleError) as e:
        m._check(pb.lib().parle_set_momentum(m._h, 0.5), "parle_set_momentum")       # no buffers bound yet
    assert e.value.code == -2
    m.set_momentum(mu)
    m.vy.fill_(123.0)                                  # stale y-momentum must not survive the round start
    lam_dev = torch.zeros(m.stride, device=DEV); lam_dev[:d] = torch.from_numpy(lam.astype(np.float32))
    lam32 = lam.astype(np.float32).astype(np.float64)
    xo, xb, vx = x0.astype(np.float64), xbar0.astype(np.float64), np.zeros((n, d))
    for rnd in range(3):
        m.round_begin()
        for l in range(L):
            m.inner_update((m.x if l == 0 else m.y) * lam_dev)
        y_gpu = m.y.cpu().numpy()[:, :d]
        m.outer_step(); torch.cuda.synchronize()
        out = po.parle_round_momentum(xo, xb, vx, po.quadratic_grad_fn(lam32), L, po.Hyper(**hp), mu)
        xo, xb, vx = out["x"], out["xbar"], out["vx"]
        assert rel_l2(y_gpu, out["y"]) < TOL
        assert rel_l2(m.x.cpu().numpy()[:, :d], xo) < TOL and rel_l2(m.xbar.cpu().numpy()[:d], xb) < TOL
        assert rel_l2(m.vx.cpu().numpy()[:, :d], vx) < TOL
    assert m.status() == 0
    assert torch.all(m.x[:, d:] == 0) and torch.all(m.vx[:, d:] == 0)
    m.set_momentum(0.0)                                # back to the plain steps
    m.round_begin(); m.inner_update(m.x * lam_dev); m.outer_step(); torch.cuda.synchronize()
    out = po.parle_round(xo, xb, po.quadratic_grad_fn(lam32), 1, po.Hyper(**hp))
    assert rel_l2(m.x.cpu().numpy()[:, :d], out["x"]) < TOL
