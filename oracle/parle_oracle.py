"""fp64 CPU oracle for one Parle round (arXiv 1707.00424, Section 3).

TEST INFRASTRUCTURE.  This file is the slow, plain reference that the CUDA
library is checked against.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may use it; the product never routes through it.
It shares no code with the CUDA path and imports nothing from it.

Everything is float64 numpy.  ``numpy.matmul`` is the only library primitive
used as a step (the dense products of the forward and backward passes); there
is no tiling, fusion or reordering beyond what the equations state.

What each function follows:

* ``mlp_forward`` / ``softmax_ce`` / ``mlp_loss_grad`` -- the minibatch
  gradient of the average cross-entropy loss f (Section 1.1; Section 2.1 for
  the minibatch estimate), textbook backpropagation through a ReLU MLP.
* ``inner_step``  -- Eq. (parle_y) then Eq. (parle_z) (identical to
  Eqs. (lesgd_y), (lesgd_z) of Section 2.1).
* ``outer_step``  -- Eq. (parle_xa).
* ``replica_mean`` -- Eq. (parle_x) with eta'' = rho/n (Section 3.1), which
  turns the reference update into the plain replica mean.
* ``inner_step_momentum`` / ``outer_step_momentum`` / ``parle_round_momentum`` -- the same
  recurrences with Nesterov momentum (Remark, Section 3.1).
* ``scoping`` -- Eq. (scoping), the schedule of gamma and rho (Section 3.1).
* ``parle_round`` -- the loop of Section 3: reset y^a (and z^a) to x^a, L
  inner steps, the outer step, the mean.

Readings of points the paper leaves open (each switchable for experiments):
  z is reset to x^a together with y at the start of a round (z_persist=False);
  the outer step uses the coefficient eta on (x^a - z^a) exactly as printed in
  Eq. (parle_xa), with no 1/gamma (unscaled_lr=False), see the Remark on
  scoping; x-bar seen by the outer step is the mean left by the previous round
  and the new mean is taken over the *updated* x^a (jacobi_mean=False);
  one round = reset, L inner steps, outer step; the loss is the mean over the
  replica's own minibatch with no regulariser (weight_decay=0); ReLU'(0)=0;
  gamma or rho = +inf means the coupling is off (1/gamma or 1/rho = 0).

Parity pins live in tests/test_oracle_*.py: finite differences and autograd
for the gradient, closed forms on a quadratic loss for the recurrences,
reduction to plain SGD and to Entropy-SGD, exactness of the mean, symmetry.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, List, Sequence, Tuple

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# Parameter packing used by the oracle: dense [W_1 | b_1 | W_2 | b_2 | ...],
# W_l stored row-major as [d_l, d_{l-1}].  (No padding; the CUDA library's
# padded layout is mapped onto this one by the tests.)
# --------------------------------------------------------------------------

def param_count(dims: Sequence[int]) -> int:
    return sum(dims[l + 1] * dims[l] + dims[l + 1] for l in range(len(dims) - 1))


def pack(layers: Sequence[Tuple[np.ndarray, np.ndarray]]) -> np.ndarray:
    return np.concatenate([np.concatenate([np.asarray(W, F64).ravel(), np.asarray(b, F64).ravel()])
                           for W, b in layers])


def unpack(vec: np.ndarray, dims: Sequence[int]) -> List[Tuple[np.ndarray, np.ndarray]]:
    out, o = [], 0
    for l in range(len(dims) - 1):
        d_in, d_out = dims[l], dims[l + 1]
        W = vec[o:o + d_out * d_in].reshape(d_out, d_in); o += d_out * d_in
        b = vec[o:o + d_out]; o += d_out
        out.append((W, b))
    assert o == vec.size
    return out


# --------------------------------------------------------------------------
# Minibatch loss and gradient of the network  (Section 1.1: f is the average
# cross-entropy loss; Section 2.1: evaluated on a minibatch)
# --------------------------------------------------------------------------

def mlp_forward(layers, X):
    """h_0 = X; h_l = max(0, h_{l-1} W_l^T + b_l) for hidden layers; the last
    layer is affine (logits).  Returns (logits, [h_0, ..., h_{last-1}])."""
    h = np.asarray(X, F64)
    acts = [h]
    for l, (W, b) in enumerate(layers):
        pre = np.matmul(h, W.T) + b
        if l + 1 < len(layers):
            h = np.maximum(pre, 0.0)
            acts.append(h)
        else:
            return pre, acts
    raise ValueError("empty network")


def softmax_ce(logits, labels):
    """Mean over the batch of CE_i = logsumexp(logits_i) - logits_i[c_i], and
    its gradient w.r.t. the logits, (softmax - onehot)/B."""
    B = logits.shape[0]
    m = logits.max(axis=1, keepdims=True)
    e = np.exp(logits - m)
    s = e.sum(axis=1, keepdims=True)
    lse = (m + np.log(s))[:, 0]
    rows = np.arange(B)
    loss = float(np.mean(lse - logits[rows, labels]))
    d = e / s
    d[rows, labels] -= 1.0
    return loss, d / B


def round_to_bf16(a):
    """Round fp64 values to the nearest bfloat16 (ties to even), returned as fp64.
    Diagnostic only: used to imitate a mixed-precision implementation's operand
    rounding so that a kernel bug can be told apart from rounding."""
    f = np.asarray(a, np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(F64).reshape(np.shape(a))


def mlp_loss_grad(vec, dims, X, labels, weight_decay: float = 0.0, operand_rounding=None):
    """Loss f(vec) on the minibatch and its gradient in the oracle's packing.

    operand_rounding (diagnostic, default None = exact fp64): a function applied
    to every operand of every dense product (weights, layer inputs, hidden
    activations, back-propagated deltas) before it is used, as a bf16-operand
    implementation would; sums stay in fp64."""
    q = operand_rounding
    layers = unpack(np.asarray(vec, F64), dims)
    if q is not None:
        return _mlp_loss_grad_rounded(layers, X, np.asarray(labels), q)
    logits, acts = mlp_forward(layers, X)
    loss, delta = softmax_ce(logits, np.asarray(labels))
    grads = [None] * len(layers)
    for l in range(len(layers) - 1, -1, -1):
        W, _ = layers[l]
        dW = np.matmul(delta.T, acts[l])          # [d_l, d_{l-1}]
        db = delta.sum(axis=0)
        grads[l] = (dW, db)
        if l > 0:
            delta = np.matmul(delta, W) * (acts[l] > 0.0)   # ReLU'(0) = 0
    g = pack(grads)
    if weight_decay:
        loss += 0.5 * weight_decay * float(np.dot(vec, vec))
        g = g + weight_decay * vec
    return loss, g


def _mlp_loss_grad_rounded(layers, X, labels, q):
    """Same forward/backward with every product operand passed through q."""
    Wq = [q(W) for W, _ in layers]
    h = q(np.asarray(X, F64))
    acts = [h]
    for l, (_, b) in enumerate(layers):
        pre = np.matmul(h, Wq[l].T) + b
        if l + 1 < len(layers):
            h = q(np.maximum(pre, 0.0))
            acts.append(h)
    loss, delta = softmax_ce(pre, labels)
    delta = q(delta)
    grads = [None] * len(layers)
    for l in range(len(layers) - 1, -1, -1):
        grads[l] = (np.matmul(delta.T, acts[l]), delta.sum(axis=0))
        if l > 0:
            delta = q(np.matmul(delta, Wq[l]) * (acts[l] > 0.0))
    return loss, pack(grads)


# --------------------------------------------------------------------------
# The recurrences of Eq. (parle)
# --------------------------------------------------------------------------

@dataclass
class Hyper:
    eta: float
    eta_prime: float
    alpha: float
    gamma: float = 1.0
    rho: float = 1.0

    @property
    def inv_gamma(self) -> float:
        return 0.0 if np.isinf(self.gamma) else 1.0 / self.gamma

    @property
    def inv_rho(self) -> float:
        return 0.0 if np.isinf(self.rho) else 1.0 / self.rho


def inner_step(y, z, x, g, hp: Hyper):
    """Eq. (parle_y): y <- y - eta' [ g + (y - x)/gamma ]  (g, y old values);
    Eq. (parle_z): z <- alpha z + (1 - alpha) y_new."""
    y_new = y - hp.eta_prime * (g + hp.inv_gamma * (y - x))
    z_new = hp.alpha * z + (1.0 - hp.alpha) * y_new
    return y_new, z_new


def outer_step(x, z, xbar, hp: Hyper, unscaled_lr: bool = False):
    """Eq. (parle_xa): x^a <- x^a - eta (x^a - z^a) - (eta/rho)(x^a - xbar)."""
    c = hp.eta * (hp.inv_gamma if unscaled_lr else 1.0)
    return x - c * (x - z) - hp.eta * hp.inv_rho * (x - xbar)


def replica_mean(xs):
    """Eq. (parle_x) with eta'' = rho/n: xbar <- (1/n) sum_a x^a.  xs: [n, P]."""
    xs = np.asarray(xs, F64)
    acc = np.zeros(xs.shape[1:], F64)
    for a in range(xs.shape[0]):
        acc = acc + xs[a]
    return acc / xs.shape[0]


def inner_step_momentum(y, z, v, x, g, hp: Hyper, mu: float):
    """Eq. (parle_y) with Nesterov momentum mu (Remark in Section 3.1; the paper does not print the form,
    the reading taken is the usual one of SGD with Nesterov momentum): with the descent direction
    d = g + (y - x)/gamma,   v <- mu v + d,   y <- y - eta' (d + mu v);   then Eq. (parle_z)."""
    d = g + hp.inv_gamma * (y - x)
    v_new = mu * v + d
    y_new = y - hp.eta_prime * (d + mu * v_new)
    z_new = hp.alpha * z + (1.0 - hp.alpha) * y_new
    return y_new, z_new, v_new


def outer_step_momentum(x, z, xbar, vx, hp: Hyper, mu: float):
    """Eq. (parle_xa) with Nesterov momentum: d = (x - z) + (x - xbar)/rho, vx <- mu vx + d,
    x <- x - eta (d + mu vx)."""
    d = (x - z) + hp.inv_rho * (x - xbar)
    vx_new = mu * vx + d
    return x - hp.eta * (d + mu * vx_new), vx_new


def parle_round_momentum(x, xbar, vx, grad_fn, L: int, hp: Hyper, mu: float):
    """One round with Nesterov momentum on the y and x^a updates (none on xbar, as in the paper's Remark).
    The y-momentum starts from zero in every round (it belongs to the trajectory that is reset); the
    x^a-momentum vx [n, P] carries over between rounds."""
    x = np.array(x, F64); xbar = np.array(xbar, F64); vx = np.array(vx, F64)
    n = x.shape[0]
    y, z, v = x.copy(), x.copy(), np.zeros_like(x)
    losses = np.zeros((L, n), F64)
    for l in range(L):
        for a in range(n):
            losses[l, a], g = grad_fn(a, l, y[a])
            y[a], z[a], v[a] = inner_step_momentum(y[a], z[a], v[a], x[a], g, hp, mu)
    x_new, vx_new = np.empty_like(x), np.empty_like(vx)
    for a in range(n):
        x_new[a], vx_new[a] = outer_step_momentum(x[a], z[a], xbar, vx[a], hp, mu)
    return {"x": x_new, "xbar": replica_mean(x_new), "vx": vx_new, "y": y, "z": z, "loss": losses}


def scoping(gamma0: float, rho0: float, batches: int, k: int, L: int,
            gamma_floor: float = 1.0, rho_floor: float = 0.1):
    """Eq. (scoping), Section 3.1: gamma_k = gamma_0 (1 - 1/(2B))^floor(k/L), rho_k likewise, B = number
    of minibatches in the dataset; gamma clipped at gamma_floor (paper: 1), rho at rho_floor (paper: 0.1)."""
    rounds_done = k // L
    factor = 1.0
    for _ in range(rounds_done):                  # the power written out as repeated multiplication
        factor *= 1.0 - 1.0 / (2.0 * batches)
    return max(gamma0 * factor, gamma_floor), max(rho0 * factor, rho_floor)


GradFn = Callable[[int, int, np.ndarray], Tuple[float, np.ndarray]]


def parle_round(x, xbar, grad_fn: GradFn, L: int, hp: Hyper, *,
                z_prev=None, z_persist: bool = False, unscaled_lr: bool = False,
                jacobi_mean: bool = False):
    """One Parle round over n replicas.

    x [n, P] and xbar [P] are the state entering the round.  grad_fn(a, l, y)
    returns (loss, gradient of f at y) for replica a at inner step l.
    Returns a dict with the new x, xbar and the y, z at the end of the inner
    loop, plus the per-step losses [L, n].
    """
    x = np.array(x, F64)
    xbar = np.array(xbar, F64)
    n = x.shape[0]
    y = x.copy()                                   # reset y^a <- x^a  (Section 3)
    z = np.array(z_prev, F64) if (z_persist and z_prev is not None) else x.copy()
    losses = np.zeros((L, n), F64)
    for l in range(L):
        for a in range(n):
            loss, g = grad_fn(a, l, y[a])
            losses[l, a] = loss
            y[a], z[a] = inner_step(y[a], z[a], x[a], g, hp)
    x_old = x
    x_new = np.empty_like(x)
    for a in range(n):
        x_new[a] = outer_step(x[a], z[a], xbar, hp, unscaled_lr)
    xbar_new = replica_mean(x_old if jacobi_mean else x_new)
    return {"x": x_new, "xbar": xbar_new, "y": y, "z": z, "loss": losses}


def mlp_grad_fn(dims, X, labels, weight_decay: float = 0.0) -> GradFn:
    """grad_fn for parle_round from X [L, n, B, d_0] and labels [L, n, B]."""
    def fn(a, l, yv):
        return mlp_loss_grad(yv, dims, X[l, a], labels[l, a], weight_decay)
    return fn


def quadratic_grad_fn(lam) -> GradFn:
    """f(y) = 1/2 y^T diag(lam) y, deterministic gradient lam * y."""
    lam = np.asarray(lam, F64)

    def fn(a, l, yv):
        return 0.5 * float(np.dot(lam * yv, yv)), lam * yv
    return fn
