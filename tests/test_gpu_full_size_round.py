"""The largest workload at its full size, in the configuration the benchmark times: sixteen replicas of the
243 M-parameter network, batch 256, L = 25, the round replayed from a CUDA graph, Eq. (parle_z) applied two steps
at a time, y of the weights kept as two 16-bit planes, the update fused into the weight-gradient kernel.

A full fp64 round of this size is far beyond what the host can do in a test, so the check has two legs:

* the same round from the same start in the literal configuration (one launch per kernel, separate weight-gradient
  and update kernels, z and fp32 y read and written at every inner step): y^a must come out bit for bit the same,
  z^a, x^a and xbar to rounding.  That literal configuration is what the smaller tests hold against the oracle.
* Eq. (parle_xa) and Eq. (parle_x) against the oracle, element by element on slices of all sixteen replicas, from
  the state the GPU holds before and after the outer step (they are element-wise, so slices cost the host nothing).

The slices cover the start of the state, the element at global offset 2^31 (inside replica 8), the middle of a
hidden layer of the last replica and the end of the last replica (last layer, biases, padding)."""
import numpy as np
import pytest
import torch

import paper_1707_00424_b200 as pb
import synth_inputs as si
from oracle import parle_oracle as po

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _draw_replicas(m, cfg):
    gen = torch.Generator(device=DEV).manual_seed(cfg.seed % (1 << 31))
    m.x.zero_()
    for a in range(cfg.n):
        for l in range(cfg.n_layers):
            w_off, _ = m.layer_offset(l)
            m.x[a, w_off:w_off + cfg.dims[l] * cfg.dims[l + 1]].normal_(0.0, cfg.dims[l] ** -0.5, generator=gen)
    m.mean()


def test_c5_full_size_round_in_the_timed_configuration():
    cfg = si.C5
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 100 * (1 << 30):
        pytest.skip("needs 100 GiB of free device memory")
    assert cfg.n == 16 and cfg.L == 25 and cfg.batch == 256
    X, c = si.round_batches(cfg, 0, pool=4)             # four distinct minibatches per replica, cycled (as the benchmark does)
    Xd, cd = torch.from_numpy(X).to(DEV), torch.from_numpy(c).to(DEV)
    m = pb.Parle(cfg.n, cfg.dims, cfg.batch, cfg.gemm_dtype, gamma=cfg.gamma, rho=cfg.rho, alpha=cfg.alpha,
                 eta=cfg.eta, eta_prime=cfg.eta_prime).alloc(DEV)
    S = m.stride
    assert cfg.n * S > (1 << 31)
    a31, e31 = divmod(1 << 31, S)                        # replica and coordinate of global element 2^31
    w2, _ = m.layer_offset(2)
    mid = w2 + (cfg.dims[2] * cfg.dims[3]) // 2
    W = 1 << 17
    spots = [(0, 0), (a31, max(0, e31 - W // 2)), (cfg.n - 1, mid), (cfg.n - 1, S - W), (5, S - W)]
    take = lambda t: [t[a, lo:lo + W].clone() for a, lo in spots]
    cols = [lo for _, lo in spots]
    take_all = lambda t: [t[..., lo:lo + W].cpu().numpy().astype(np.float64) for lo in cols]   # all replicas (or xbar)

    results = []
    for timed in (True, False):
        _draw_replicas(m, cfg)
        m.set_round_graphs(timed); m.set_paired_z_update(timed); m.set_split_y(timed); m.set_fused_update(timed)
        x_old, xbar_old = take_all(m.x), take_all(m.xbar)
        loss = torch.zeros(cfg.L, cfg.n, device=DEV)
        m.round(cfg.L, Xd, cd, loss)
        torch.cuda.synchronize()
        assert m.status() == 0
        results.append(dict(y=take(m.y), z=take(m.z), x=take(m.x), xbar=[m.xbar[lo:lo + W].clone() for lo in cols], loss=loss.cpu().numpy()))
        if timed:
            # Eq. (parle_xa), Eq. (parle_x) on slices of every replica, from the z the inner steps left
            hp = po.Hyper(eta=cfg.eta, eta_prime=cfg.eta_prime, alpha=cfg.alpha, gamma=cfg.gamma, rho=cfg.rho)
            z_all, x_new, xbar_new = take_all(m.z), take_all(m.x), take_all(m.xbar)
            for k in range(len(cols)):
                want = np.stack([po.outer_step(x_old[k][a], z_all[k][a], xbar_old[k], hp) for a in range(cfg.n)])
                np.testing.assert_allclose(x_new[k], want, rtol=1e-6, atol=1e-7)
                np.testing.assert_allclose(xbar_new[k], po.replica_mean(want), rtol=1e-6, atol=1e-7)
    del m, Xd, cd
    torch.cuda.empty_cache()                             # hand the 75 GB back before the next test asks how much is free
    fast, plain = results
    # losses: finite, near log(C) at the start (random weights), the same in both configurations up to summation order
    assert np.isfinite(fast["loss"]).all() and abs(float(fast["loss"][0].mean()) - np.log(cfg.dims[-1])) < 1.5
    np.testing.assert_allclose(fast["loss"], plain["loss"], rtol=1e-5)
    for k in range(len(spots)):
        assert torch.equal(fast["y"][k], plain["y"][k]), ("y", spots[k])
        for name in ("z", "x", "xbar"):
            got, want = fast[name][k].double(), plain[name][k].double()
            scale = float(want.abs().max())
            assert float((got - want).abs().max()) <= 2e-6 * scale + 1e-9, (name, spots[k])
    # the slices are not trivially equal: y moved away from x, and differs between replicas
    assert float((fast["y"][2] - fast["x"][2]).abs().max()) > 0
    assert not torch.equal(fast["y"][3], fast["y"][4])
