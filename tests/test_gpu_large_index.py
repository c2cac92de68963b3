"""Parity where element offsets pass 2^31: the update sweep's largest vectors and the 243 M-parameter network
with nine or more replicas address their state with offsets that no longer fit 32 bits.  Flat vectors against the
oracle on slices (Eq. parle_y, parle_z, parle_xa, parle_x); the network's fused weight-gradient + update kernel
against the separate kernels on the last replica, with sampled weight-gradient entries recomputed in fp64.

State is drawn on the device with seeded torch generators (the host generator would need minutes for 2.4e9
values); the slices handed to the oracle are copied out before the kernels run."""
import numpy as np
import pytest
import torch

import paper_1707_00424_b200 as pb
import synth_inputs as si
from oracle import parle_oracle as po

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PAD = 1024           # canary elements on both sides of every state buffer


def _need(gib):
    free, _ = torch.cuda.mem_get_info()
    if free < gib * (1 << 30):
        pytest.skip(f"needs {gib} GiB of free device memory")


def _guarded(n, stride):
    raw = torch.full((n * stride + 2 * PAD,), 7.5, device=DEV)
    return raw, raw[PAD:PAD + n * stride].view(n, stride)


def test_flat_vectors_past_2_to_31_elements_match_oracle_on_slices():
    n, d = 9, (1 << 28) + 4128            # element 2^31 lies inside replica 7; replica 8 lies wholly beyond it
    _need(48)
    hp = dict(eta=0.25, eta_prime=0.05, alpha=0.75, gamma=3.0, rho=0.5)
    m = pb.Parle(n, (d,), 0, **hp)
    S = m.stride
    assert S == d and n * S > (1 << 31) and 7 * S < (1 << 31) < 8 * S
    raws, views = zip(*[_guarded(n, S) for _ in range(4)])
    x, y, z, g = views
    xbar_raw, xbar = _guarded(1, S)
    xbar = xbar[0]
    ws = torch.empty(max(m.workspace_bytes, 1024), dtype=torch.uint8, device=DEV)
    gen = torch.Generator(device=DEV).manual_seed(2031)
    for a in range(n):
        x[a].normal_(generator=gen); g[a].normal_(0.0, 0.1, generator=gen)
    xbar.normal_(generator=gen)                                   # any xbar: the outer step takes it as given
    m.bind(x, y, z, g, xbar, ws)
    cross = (1 << 31) - 7 * S                                     # coordinate of replica 7 that sits at element 2^31
    slices = [(0, 1 << 20), (cross - (1 << 19), cross + (1 << 19)), (S - (1 << 20), S)]
    take = lambda t: [t[..., lo:hi].cpu().numpy().astype(np.float64) for lo, hi in slices]
    x0, g0, xb0 = take(x), take(g), take(xbar)
    H = po.Hyper(**hp)

    # first inner step of a round (reset folded in), a later step, the outer step with its mean
    m.round_begin(); m.inner_update(g); torch.cuda.synchronize()
    y1, z1 = take(y), take(z)
    g.mul_(-0.5)
    g1 = take(g)
    m.inner_update(g); torch.cuda.synchronize()
    y2, z2 = take(y), take(z)
    m.outer_step(); torch.cuda.synchronize()
    x1, xb1 = take(x), take(xbar)
    assert m.status() == 0
    for k in range(len(slices)):
        wy1, wz1 = po.inner_step(x0[k], x0[k], x0[k], g0[k], H)
        np.testing.assert_allclose(y1[k], wy1, rtol=1e-6, atol=5e-7)
        np.testing.assert_allclose(z1[k], wz1, rtol=1e-6, atol=5e-7)
        wy2, wz2 = po.inner_step(wy1, wz1, x0[k], g1[k], H)
        np.testing.assert_allclose(y2[k], wy2, rtol=1e-6, atol=5e-7)
        np.testing.assert_allclose(z2[k], wz2, rtol=1e-6, atol=5e-7)
        wx = np.stack([po.outer_step(x0[k][a], wz2[a], xb0[k], H) for a in range(n)])
        np.testing.assert_allclose(x1[k], wx, rtol=1e-6, atol=1e-6)
        np.testing.assert_allclose(xb1[k], po.replica_mean(wx), rtol=1e-6, atol=1e-6)
    # the stand-alone mean after writing x directly
    for a in range(n):
        x[a].normal_(generator=gen)
    xs = take(x)
    m.mean(); torch.cuda.synchronize()
    for k, got in enumerate(take(xbar)):
        np.testing.assert_allclose(got, po.replica_mean(xs[k]), rtol=1e-6, atol=5e-7)
    # nothing outside the state was written
    for raw in list(raws) + [xbar_raw]:
        assert torch.all(raw[:PAD] == 7.5) and torch.all(raw[-PAD:] == 7.5)


def test_network_past_2_to_31_elements_fused_equals_separate_update_bf16():
    """The 243 M-parameter shape with ten replicas: element 2^31 falls inside replica 8, replica 9 lies wholly beyond it.
    Two inner steps (the first of a round and a later one): the fused kernel's y, z (last two replicas) and bf16 operand
    copy (last replica) equal, bit for bit, what the weight-gradient product + separate update kernel give; sampled
    entries of that replica's weight gradient are recomputed in fp64 from the operands the GPU used."""
    cfg = si.C5.scaled(name="C5x10", n=10, L=2)
    _need(70)
    last = cfg.n - 1
    X, c = si.round_batches(cfg, 0)
    Xd, cd = torch.from_numpy(X).to(DEV), torch.from_numpy(c).to(DEV)
    rng = np.random.default_rng(9)
    keep = []
    for fused in (False, True):
        m = pb.Parle(cfg.n, cfg.dims, cfg.batch, cfg.gemm_dtype).alloc(DEV)
        assert last * m.stride > (1 << 31) > (last - 1) * m.stride
        m.set_fused_update(fused)
        gen = torch.Generator(device=DEV).manual_seed(77)
        for a in range(cfg.n):
            for l in range(cfg.n_layers):
                w_off, _ = m.layer_offset(l)
                m.x[a, w_off:w_off + cfg.dims[l] * cfg.dims[l + 1]].normal_(0.0, cfg.dims[l] ** -0.5, generator=gen)
        m.mean(); m.round_begin()
        m.inner_step(Xd[0], cd[0]); torch.cuda.synchronize()
        assert m.status() == 0
        if not fused:
            f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
            H = [po.round_to_bf16(X[0, last].astype(np.float64))] + \
                [f64(m.debug_buffer(m.DBG_ACT, l)[last]) for l in range(cfg.n_layers - 1)]
            for l in range(cfg.n_layers):
                din, dout = cfg.dims[l], cfg.dims[l + 1]
                dH = f64(m.debug_buffer(m.DBG_DACT, l)[last])
                w_off, _ = m.layer_offset(l)
                j = rng.integers(0, dout, 64); k = rng.integers(0, din, 64)
                got = m.grad[last, w_off:w_off + dout * din].view(dout, din)[torch.from_numpy(j).to(DEV), torch.from_numpy(k).to(DEV)]
                want = np.einsum("bs,bs->s", dH[:, j], H[l][:, k])
                assert np.allclose(got.cpu().numpy(), want, rtol=1e-4, atol=1e-9), ("dW", l)
        m.inner_step(Xd[1], cd[1]); torch.cuda.synchronize()
        assert m.status() == 0
        keep.append((m.y[last].clone(), m.z[last].clone(), m.debug_buffer(m.DBG_OPERAND_COPY)[last].clone(),
                     m.y[last - 1].clone(), m.z[last - 1].clone(), m.y[0, :1 << 20].clone()))
        del m
        torch.cuda.empty_cache()
    for a, b in zip(*keep):
        assert torch.equal(a, b)
    assert torch.isfinite(keep[0][0]).all() and float(keep[0][0].abs().max()) > 0
