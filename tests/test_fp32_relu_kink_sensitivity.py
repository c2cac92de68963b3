"""Why the MNIST-shaped fp32 workload (784-1024-1024-10, U[0,1] inputs, eta' = 0.1) gets a wider bound on the inner
iterates y^a, z^a than the 1e-4 every other fp32 case is held to -- shown on the CPU, with the oracle alone.

The minibatch gradient (Section 2.1) of a ReLU network is discontinuous where a pre-activation crosses zero.  In
round 0 of replica 1 the fp64 trajectory of Eq. (parle_y) passes, at inner step 16, within 6e-8 of such a kink
(one unit of the second hidden layer for one sample; the pre-activations there are sums of ~1000 terms of size
~0.05, so every fp32 evaluation of that sum has an error of about that size and lands on either side).  Taking
the other side changes that step's gradient by 3e-3 of its norm, and the remaining steps enlarge the difference
(with all-positive inputs the loss has a Hessian eigenvalue near 2/eta', the inner loop runs at the edge of
stability): y^a ends 3.5e-4 away, z^a 1.8e-4, x^a 1.8e-5, the round's displacement of x^a 2e-2.  Both outcomes
are correct roundings of the same iteration, so no fp32 implementation can be held to 1e-4 on y^a and z^a there;
x^a and xbar stay inside 1e-4.

The same is then seen with a plain float32 numpy transcription of the oracle's steps (which side it lands on
depends on the BLAS's summation order, so only the upper bounds are asserted for it)."""
import numpy as np

import synth_inputs as si
from oracle import parle_oracle as po
from _util import rel_l2

CFG, REPLICA, STEP, LAYER, SAMPLE, UNIT = si.C2, 1, 16, 1, 56, 534


def _problem():
    cfg = CFG
    mb = [si.minibatch(cfg, REPLICA, 0, l) for l in range(cfg.L)]
    X = np.stack([m[0] for m in mb])[:, None]          # [L, 1, B, d_0]
    c = np.stack([m[1] for m in mb])[:, None]
    x0 = po.pack(si.init_replica(cfg, REPLICA))[None]
    hp = po.Hyper(cfg.eta, cfg.eta_prime, cfg.alpha, cfg.gamma, cfg.rho)
    return cfg, X, c, x0, hp


def test_one_relu_unit_at_the_kink_moves_y_by_more_than_1e_4():
    cfg, X, c, x0, hp = _problem()
    base = po.mlp_grad_fn(cfg.dims, X, c)
    seen = {}

    def watching(a, l, y):
        if l == STEP:
            layers = po.unpack(y, cfg.dims)
            h = X[l, 0].astype(np.float64)
            for k in range(LAYER + 1):
                pre = h @ layers[k][0].T + layers[k][1]
                h = np.maximum(pre, 0.0)
            seen["pre"] = pre[SAMPLE, UNIT]
            seen["scale"] = float(np.sqrt(np.mean(pre ** 2)))
        return base(a, l, y)

    ref = po.parle_round(x0, x0[0], watching, cfg.L, hp)
    assert abs(seen["pre"]) < 1e-7 and seen["scale"] > 0.1, seen      # far inside fp32 rounding of that sum

    d = cfg.dims
    bias_of_unit = d[0] * d[1] + d[1] + d[1] * d[2] + UNIT            # b_2[UNIT] in the oracle's packing

    def other_side(a, l, y):
        if l == STEP:                                                  # evaluate the gradient just across the kink
            y = y.copy()
            y[bias_of_unit] -= 2.1 * seen["pre"]
        return base(a, l, y)

    alt = po.parle_round(x0, x0[0], other_side, cfg.L, hp)
    ey, ez = rel_l2(alt["y"][0], ref["y"][0]), rel_l2(alt["z"][0], ref["z"][0])
    ex = rel_l2(alt["x"][0], ref["x"][0])
    disp = rel_l2(alt["x"][0] - x0[0], ref["x"][0] - x0[0])
    print(f"other side of the kink: y {ey:.2e} z {ez:.2e} x {ex:.2e} displacement {disp:.2e}")
    assert 1e-4 < ey < 1e-3 and 1e-4 < ez < 1e-3                      # beyond 1e-4, inside the 1e-3 the GPU test allows
    assert ex < 1e-4                                                  # the stated bound on the parameters holds
    assert 5e-3 < disp < 5e-2                                         # hence the displacement bound of that test


def test_float32_transcription_of_the_round_stays_inside_the_widened_bounds():
    cfg, X, c, x0, hp = _problem()
    ref = po.parle_round(x0, x0[0], po.mlp_grad_fn(cfg.dims, X, c), cfg.L, hp)
    f = np.float32
    d = cfg.dims
    x = x0[0].astype(f); y = x.copy(); z = x.copy()
    for l in range(cfg.L):
        layers, o = [], 0
        for k in range(len(d) - 1):
            W = y[o:o + d[k + 1] * d[k]].reshape(d[k + 1], d[k]); o += d[k + 1] * d[k]
            b = y[o:o + d[k + 1]]; o += d[k + 1]
            layers.append((W, b))
        h = X[l, 0].astype(f); acts = [h]
        for k, (W, b) in enumerate(layers):
            pre = h @ W.T + b
            if k + 1 < len(layers):
                h = np.maximum(pre, f(0)); acts.append(h)
        e = np.exp(pre - pre.max(axis=1, keepdims=True))
        delta = e / e.sum(axis=1, keepdims=True)
        delta[np.arange(cfg.batch), c[l, 0]] -= f(1)
        delta = delta / f(cfg.batch)
        parts = [None] * len(layers)
        for k in range(len(layers) - 1, -1, -1):
            parts[k] = np.concatenate([(delta.T @ acts[k]).ravel(), delta.sum(axis=0)])
            if k > 0:
                delta = (delta @ layers[k][0]) * (acts[k] > 0)
        g = np.concatenate(parts).astype(f)
        y = y - f(hp.eta_prime) * (g + f(hp.inv_gamma) * (y - x))
        z = f(hp.alpha) * z + (f(1) - f(hp.alpha)) * y
    xn = x - f(hp.eta) * (x - z) - f(hp.eta * hp.inv_rho) * (x - x)   # xbar = x^a for a single replica
    ey, ez, ex = rel_l2(y, ref["y"][0]), rel_l2(z, ref["z"][0]), rel_l2(xn, ref["x"][0])
    print(f"float32 numpy round: y {ey:.2e} z {ez:.2e} x {ex:.2e}")
    assert ey < 1e-3 and ez < 1e-3 and ex < 1e-4
