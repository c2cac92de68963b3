"""Pins for the oracle's minibatch gradient (average cross-entropy of a ReLU
MLP, Section 1.1 / Section 2.1): finite differences, an independent autograd
library, and closed-form special cases."""
import math

import numpy as np
import pytest
import torch

from oracle import parle_oracle as po


def _rand_problem(dims, B, seed):
    rng = np.random.default_rng(seed)
    vec = rng.normal(size=po.param_count(dims)) * 0.7
    X = rng.normal(size=(B, dims[0]))
    c = rng.integers(0, dims[-1], size=B)
    return vec, X, c


@pytest.mark.parametrize("dims,B", [((5, 4, 3), 3), ((6, 5, 4, 3), 4), ((4, 3), 5)])
def test_gradient_matches_central_differences(dims, B):
    vec, X, c = _rand_problem(dims, B, seed=11)
    _, g = po.mlp_loss_grad(vec, dims, X, c)
    h = 1e-6
    for i in range(vec.size):
        e = np.zeros_like(vec); e[i] = h
        fp, _ = po.mlp_loss_grad(vec + e, dims, X, c)
        fm, _ = po.mlp_loss_grad(vec - e, dims, X, c)
        fd = (fp - fm) / (2 * h)
        assert abs(fd - g[i]) <= 1e-6 * max(1.0, abs(g[i])), (i, fd, g[i])


def test_gradient_matches_torch_autograd():
    dims, B = (7, 6, 5, 4), 9
    vec, X, c = _rand_problem(dims, B, seed=5)
    loss, g = po.mlp_loss_grad(vec, dims, X, c)
    # independent route: torch's own linear / relu / cross_entropy + autograd
    params, o = [], 0
    for l in range(len(dims) - 1):
        W = torch.tensor(vec[o:o + dims[l + 1] * dims[l]].reshape(dims[l + 1], dims[l]),
                         dtype=torch.float64, requires_grad=True); o += dims[l + 1] * dims[l]
        b = torch.tensor(vec[o:o + dims[l + 1]], dtype=torch.float64, requires_grad=True); o += dims[l + 1]
        params.append((W, b))
    h = torch.tensor(X, dtype=torch.float64)
    for l, (W, b) in enumerate(params):
        h = torch.nn.functional.linear(h, W, b)
        if l + 1 < len(params):
            h = torch.relu(h)
    tl = torch.nn.functional.cross_entropy(h, torch.tensor(c, dtype=torch.long))
    tl.backward()
    tg = np.concatenate([np.concatenate([W.grad.numpy().ravel(), b.grad.numpy().ravel()]) for W, b in params])
    assert abs(loss - tl.item()) < 1e-13
    np.testing.assert_allclose(g, tg, rtol=1e-12, atol=1e-14)


def test_zero_network_loss_is_log_C_and_bias_gradient_closed_form():
    dims, B = (5, 4, 6), 8
    rng = np.random.default_rng(0)
    X = rng.normal(size=(B, dims[0]))
    c = rng.integers(0, dims[-1], size=B)
    vec = np.zeros(po.param_count(dims))
    loss, g = po.mlp_loss_grad(vec, dims, X, c)
    assert abs(loss - math.log(dims[-1])) < 1e-14
    layers = po.unpack(g, dims)
    # uniform softmax: d loss / d b_last[j] = 1/C - (count of label j)/B
    want = 1.0 / dims[-1] - np.bincount(c, minlength=dims[-1]) / B
    np.testing.assert_allclose(layers[-1][1], want, atol=1e-15)
    # all hidden activations are 0 and ReLU'(0)=0: nothing flows below
    assert np.all(layers[0][0] == 0) and np.all(layers[0][1] == 0)
    assert np.all(layers[-1][0] == 0)


def test_dlogits_rows_sum_to_zero_and_scale_with_batch():
    rng = np.random.default_rng(3)
    logits = rng.normal(size=(6, 5)) * 4
    c = rng.integers(0, 5, size=6)
    loss, d = po.softmax_ce(logits, c)
    np.testing.assert_allclose(d.sum(axis=1), 0.0, atol=1e-16)
    # shifting a row of logits by a constant changes nothing (softmax invariance)
    loss2, d2 = po.softmax_ce(logits + 1000.0, c)
    assert abs(loss - loss2) < 1e-10
    np.testing.assert_allclose(d, d2, atol=1e-13)
    # single-row case against the definition -log p_c
    l1, d1 = po.softmax_ce(logits[:1], c[:1])
    p = np.exp(logits[0]) / np.exp(logits[0]).sum()
    assert abs(l1 + math.log(p[c[0]])) < 1e-13
    want = p.copy(); want[c[0]] -= 1
    np.testing.assert_allclose(d1[0], want, atol=1e-15)


def test_linear_softmax_gradient_matches_textbook_formula():
    # one affine layer: dW = (P - Y)^T X / B, db = mean(P - Y)
    dims, B = (4, 3), 7
    vec, X, c = _rand_problem(dims, B, seed=2)
    (W, b), = po.unpack(vec, dims)
    logits = X @ W.T + b
    P = np.exp(logits); P /= P.sum(axis=1, keepdims=True)
    Y = np.eye(3)[c]
    _, g = po.mlp_loss_grad(vec, dims, X, c)
    (dW, db), = po.unpack(g, dims)
    np.testing.assert_allclose(dW, (P - Y).T @ X / B, atol=1e-15)
    np.testing.assert_allclose(db, (P - Y).mean(axis=0), atol=1e-15)


def test_planted_mistakes_are_caught_by_finite_differences(monkeypatch):
    """A transposed product or a dropped ReLU mask must break the FD pin."""
    dims, B = (5, 4, 3), 3
    vec, X, c = _rand_problem(dims, B, seed=11)

    def fd_ok():
        _, g = po.mlp_loss_grad(vec, dims, X, c)
        h = 1e-6
        for i in range(vec.size):
            e = np.zeros_like(vec); e[i] = h
            fd = (po.mlp_loss_grad(vec + e, dims, X, c)[0] - po.mlp_loss_grad(vec - e, dims, X, c)[0]) / (2 * h)
            if abs(fd - g[i]) > 1e-6 * max(1.0, abs(g[i])):
                return False
        return True

    assert fd_ok()
    real = po.softmax_ce
    monkeypatch.setattr(po, "softmax_ce", lambda lg, lb: (real(lg, lb)[0], real(lg, lb)[1] * lg.shape[0]))
    assert not fd_ok()          # forgot the 1/B
    monkeypatch.setattr(po, "softmax_ce", real)
    # dropping the ReLU mask in the backward pass == treating hidden units as linear there
    orig = po.mlp_forward

    def fwd_no_mask(layers, X_):
        logits, acts = orig(layers, X_)
        return logits, [a + (a == 0) * 1e-300 for a in acts]   # every unit looks active
    monkeypatch.setattr(po, "mlp_forward", fwd_no_mask)
    assert not fd_ok()


def test_bf16_rounding_helper_and_rounded_mode():
    # exact cases of round-to-nearest-even at 8 significant bits
    vals = np.array([1.0, 1.00390625, 1.001953125, 1.005859375, -3.1415926, 0.0, 65504.0])
    want = np.array([1.0, 1.0, 1.0, 1.0078125, -3.140625, 0.0, 65536.0])
    np.testing.assert_array_equal(po.round_to_bf16(vals), want)
    # against torch's own bfloat16 conversion
    r = np.random.default_rng(0).normal(size=1000) * 10.0 ** np.random.default_rng(1).integers(-5, 5, 1000)
    t = torch.tensor(r, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(po.round_to_bf16(r), t)
    # identity "rounding" reproduces the exact gradient; bf16 rounding stays close
    dims, B = (16, 12, 5), 8
    vec, X, c = _rand_problem(dims, B, seed=8)
    l0, g0 = po.mlp_loss_grad(vec, dims, X, c)
    l1, g1 = po.mlp_loss_grad(vec, dims, X, c, operand_rounding=lambda a: np.asarray(a, np.float64))
    assert abs(l0 - l1) < 1e-14 and np.allclose(g0, g1, rtol=1e-13, atol=1e-15)
    l2, g2 = po.mlp_loss_grad(vec, dims, X, c, operand_rounding=po.round_to_bf16)
    assert 0 < np.linalg.norm(g2 - g0) / np.linalg.norm(g0) < 0.05


def _wd_fd_ok(vec, dims, X, c, lam):
    _, g = po.mlp_loss_grad(vec, dims, X, c, weight_decay=lam)
    h = 1e-6
    for i in range(vec.size):
        e = np.zeros_like(vec); e[i] = h
        fd = (po.mlp_loss_grad(vec + e, dims, X, c, weight_decay=lam)[0]
              - po.mlp_loss_grad(vec - e, dims, X, c, weight_decay=lam)[0]) / (2 * h)
        if abs(fd - g[i]) > 1e-6 * max(1.0, abs(g[i])):
            return False
    return True


def test_weight_decay_term_of_f():
    """Section 1.1 lets f carry a regulariser besides the average loss and names weight decay as the example.  The
    reading taken is f(y) = data term + (lambda/2) |y|^2 over every parameter: the loss grows by exactly that amount,
    the gradient by lambda y, central differences of the regularised loss give the regularised gradient, and the
    regulariser's own second derivative is lambda."""
    dims, B, lam = (5, 4, 3), 3, 0.37
    vec, X, c = _rand_problem(dims, B, seed=21)
    l0, g0 = po.mlp_loss_grad(vec, dims, X, c)
    l1, g1 = po.mlp_loss_grad(vec, dims, X, c, weight_decay=lam)
    assert abs((l1 - l0) - 0.5 * lam * sum(v * v for v in vec.tolist())) < 1e-13     # the sum written out in Python
    np.testing.assert_allclose(g1 - g0, lam * vec, rtol=1e-13, atol=1e-15)
    assert _wd_fd_ok(vec, dims, X, c, lam)
    # second derivative of the regulariser alone, by differencing the gradient: lambda on the diagonal
    e = np.zeros_like(vec); e[7] = 1e-5
    gp = po.mlp_loss_grad(vec + e, dims, X, c, weight_decay=lam)[1] - po.mlp_loss_grad(vec + e, dims, X, c)[1]
    gm = po.mlp_loss_grad(vec - e, dims, X, c, weight_decay=lam)[1] - po.mlp_loss_grad(vec - e, dims, X, c)[1]
    np.testing.assert_allclose((gp - gm)[7] / 2e-5, lam, rtol=1e-9)


def test_planted_weight_decay_mistakes_are_caught(monkeypatch):
    """A dropped 1/2 in the regulariser's loss, a flipped sign of its gradient, or decay applied to the weights but
    not the biases each break the pin above."""
    dims, B, lam = (5, 4, 3), 3, 0.37
    vec, X, c = _rand_problem(dims, B, seed=21)
    assert _wd_fd_ok(vec, dims, X, c, lam)
    real = po.mlp_loss_grad

    def no_half(v, d, X_, c_, weight_decay=0.0, operand_rounding=None):
        loss, g = real(v, d, X_, c_, weight_decay, operand_rounding)
        return loss + 0.5 * weight_decay * float(np.dot(v, v)), g
    monkeypatch.setattr(po, "mlp_loss_grad", no_half)
    assert not _wd_fd_ok(vec, dims, X, c, lam)

    def wrong_sign(v, d, X_, c_, weight_decay=0.0, operand_rounding=None):
        loss, g = real(v, d, X_, c_, weight_decay, operand_rounding)
        return loss, g - 2.0 * weight_decay * np.asarray(v)
    monkeypatch.setattr(po, "mlp_loss_grad", wrong_sign)
    assert not _wd_fd_ok(vec, dims, X, c, lam)

    def weights_only(v, d, X_, c_, weight_decay=0.0, operand_rounding=None):
        loss, g = real(v, d, X_, c_, weight_decay, operand_rounding)
        g = g.copy()
        o = 0
        for l in range(len(d) - 1):
            o += d[l + 1] * d[l]
            g[o:o + d[l + 1]] -= weight_decay * np.asarray(v)[o:o + d[l + 1]]
            o += d[l + 1]
        return loss, g
    monkeypatch.setattr(po, "mlp_loss_grad", weights_only)
    assert not _wd_fd_ok(vec, dims, X, c, lam)
