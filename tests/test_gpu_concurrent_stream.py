"""The library's kernels with other work resident on the same SMs.  In the library's own order of launches nothing runs
beside the fused weight-gradient + update kernel, so its hand-offs between warps are never under pressure in the other
tests; a caller's second stream can put CTAs next to it.  Here a kernel that keeps the load/store units busy (16-byte loads
512 bytes apart) runs on a second stream during the inner steps (Section 3.1: Eq. parle_y, parle_z in the epilogue of the
weight-gradient product), and y, z and the bf16 operand copy must equal, bit for bit, what the separate kernels give on a
quiet device.  With a stage of the state ring handed back to its loader before the stores that use its values, this
comparison failed in every run (32-96 weights per launch took the x, y or z of a later tile)."""
import pytest
import torch

import paper_1707_00424_b200 as pb
import synth_inputs as si

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _steps(cfg, fused, busy, Xd, cd):
    m = pb.Parle(cfg.n, cfg.dims, cfg.batch, cfg.gemm_dtype).alloc(DEV)
    m.set_fused_update(fused)
    gen = torch.Generator(device=DEV).manual_seed(77)
    for a in range(cfg.n):
        for l in range(cfg.n_layers):
            w_off, _ = m.layer_offset(l)
            m.x[a, w_off:w_off + cfg.dims[l] * cfg.dims[l + 1]].normal_(0.0, cfg.dims[l] ** -0.5, generator=gen)
    m.mean(); m.round_begin()
    torch.cuda.synchronize()
    for s in range(cfg.L):
        if busy is not None:
            busy.launch(times=24)
        m.inner_step(Xd[s], cd[s])
    torch.cuda.synchronize()
    assert m.status() == 0
    out = (m.y.clone(), m.z.clone(), m.debug_buffer(m.DBG_OPERAND_COPY).clone())
    del m
    torch.cuda.empty_cache()
    return out


def test_fused_update_is_exact_with_a_busy_second_stream_bf16():
    pytest.importorskip("cuda.bindings")
    from _busy_kernel import BusyKernel
    free, _ = torch.cuda.mem_get_info()
    if free < 8 << 30:
        pytest.skip("needs 8 GiB of free device memory")
    cfg = si.C5.scaled(name="C5-two-layers", n=3, dims=(4096, 8192, 1000), L=3)
    X, c = si.round_batches(cfg, 0)
    Xd, cd = torch.from_numpy(X).to(DEV), torch.from_numpy(c).to(DEV)
    want = _steps(cfg, False, None, Xd, cd)
    busy = BusyKernel(DEV)
    try:
        for rep in range(3):
            got = _steps(cfg, True, busy, Xd, cd)
            for name, a, b in zip(("y", "z", "operand copy"), want, got):
                assert torch.equal(a, b), (rep, name, int((a != b).sum()))
    finally:
        busy.close()


@pytest.mark.parametrize("name", ["C3", "C5/2", "C2"])
def test_rounds_are_reproducible_with_a_busy_second_stream(name):
    """Whole rounds (graph replay: chained two-CTA GEMMs, loss, fused update with paired z and two-plane y; for the fp32
    workload the three-product tf32 kernels and the separate update) give the same bits with and without the second stream's
    kernel resident: no hand-off between warps of any kernel depends on how fast its neighbours run."""
    pytest.importorskip("cuda.bindings")
    from _busy_kernel import BusyKernel
    free, _ = torch.cuda.mem_get_info()
    if free < 16 << 30:
        pytest.skip("needs 16 GiB of free device memory")
    if name == "C3":
        cfg = si.C3.scaled(name="C3x3", n=3, L=6)
    elif name == "C5/2":
        cfg = si.C5.scaled(name="C5/2", n=3, dims=(2048, 4096, 4096, 4096, 1000), L=5)
    else:
        cfg = si.C2.scaled(name="C2x4", n=4, L=6)
    X, c = si.round_batches(cfg, 0)
    Xd, cd = torch.from_numpy(X).to(DEV), torch.from_numpy(c).to(DEV)

    def rounds(busy):
        m = pb.Parle(cfg.n, cfg.dims, cfg.batch, cfg.gemm_dtype, eta=cfg.eta, eta_prime=cfg.eta_prime, alpha=cfg.alpha,
                     gamma=cfg.gamma, rho=cfg.rho).alloc(DEV)
        gen = torch.Generator(device=DEV).manual_seed(3)
        for a in range(cfg.n):
            for l in range(cfg.n_layers):
                w_off, _ = m.layer_offset(l)
                m.x[a, w_off:w_off + cfg.dims[l] * cfg.dims[l + 1]].normal_(0.0, cfg.dims[l] ** -0.5, generator=gen)
        m.mean()
        m.set_round_graphs(True)
        loss = torch.zeros(cfg.L, cfg.n, device=DEV)
        torch.cuda.synchronize()
        for r in range(3):
            if busy is not None:
                busy.launch(times=32)
            m.round(cfg.L, Xd, cd, loss)
        torch.cuda.synchronize()
        assert m.status() == 0
        out = (m.x.clone(), m.xbar.clone(), m.y.clone(), m.z.clone(), loss.clone())
        del m
        torch.cuda.empty_cache()
        return out

    want = rounds(None)
    busy = BusyKernel(DEV)
    try:
        for rep in range(2):
            got = rounds(busy)
            for nm, a, b in zip(("x", "xbar", "y", "z", "loss"), want, got):
                assert torch.equal(a, b), (rep, nm, int((a != b).sum()))
    finally:
        busy.close()
