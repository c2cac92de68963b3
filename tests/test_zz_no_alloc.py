"""The allocation-free loss entry point against the regular inner step.

Some users of this library cannot allocate device memory or pass a workspace
(they live inside someone else's fixed memory pool); parle_softmax_ce_static
keeps its scratch in a fixed array inside the library instead.  It must give
what parle_inner_step gives for the same logits: here the logits, dlogits and
losses of a regular inner step are read back and the new entry point is run on
those logits, twice in a row with different data (the array is shared between
calls and keeps old contents, so the second call checks that nothing stale
leaks through)."""
import gc

import numpy as np
import pytest
import torch

import paper_1707_00424_b200 as pb
import synth_inputs as si
from oracle import parle_oracle as po
from _util import to_padded

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inner_step_outputs(cfg, step):
    m = pb.Parle(cfg.n, cfg.dims, cfg.batch, cfg.gemm_dtype).alloc(DEV)
    x0 = np.stack([po.pack(si.init_replica(cfg, a)) for a in range(cfg.n)])
    m.x.copy_(torch.from_numpy(to_padded(m, x0)))
    X, c = si.round_batches(cfg, 0)
    loss = torch.zeros(cfg.n, device=DEV)
    labels = torch.from_numpy(c[step]).to(DEV)
    m.round_begin()
    m.inner_step(torch.from_numpy(X[step]).to(DEV), labels, loss)
    torch.cuda.synchronize()
    logits = m.debug_buffer(m.DBG_LOGITS).clone()
    dlogits = m.debug_buffer(m.DBG_DACT, cfg.n_layers - 1).clone()
    return logits, labels, dlogits, loss.clone()


def test_static_loss_matches_inner_step_twice_in_a_row():
    big = si.C1.scaled(n=4, dims=(48, 40, 100), batch=72)      # more rows first, fewer second
    cases = [(big, 0), (si.C1, 1)]
    for cfg, step in cases:
        logits, labels, want_d, want_loss = _inner_step_outputs(cfg, step)
        C = cfg.dims[-1]
        got_d = torch.full_like(want_d.contiguous(), float("nan"))
        got_loss = torch.full((cfg.n,), float("nan"), device=DEV)
        flags = torch.full((1,), -1, dtype=torch.int32, device=DEV)
        logits = logits.contiguous()
        gc.collect(); torch.cuda.synchronize()               # drop the finished model's tensors first
        before = torch.cuda.memory_allocated()
        pb.softmax_ce_static(logits, labels, cfg.n, cfg.batch, C, got_d, got_loss, flags)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before       # torch's allocator was not touched
        # same kernels, same inputs: equal to rounding (the tolerance of the fp32 element-wise tests)
        np.testing.assert_allclose(got_d.cpu().numpy(), want_d.cpu().numpy(), rtol=1e-6, atol=1e-7)
        np.testing.assert_allclose(got_loss.cpu().numpy(), want_loss.cpu().numpy(), rtol=1e-6, atol=1e-7)
        assert flags.item() == 0
        # and against the oracle's softmax cross-entropy on the same logits, replica by replica
        lg = logits.cpu().numpy().astype(np.float64).reshape(cfg.n, cfg.batch, C)
        lab = labels.cpu().numpy().reshape(cfg.n, cfg.batch)
        gd = got_d.cpu().numpy().reshape(cfg.n, cfg.batch, -1)[:, :, :C]
        for a in range(cfg.n):
            want_l, want_dl = po.softmax_ce(lg[a], lab[a])
            np.testing.assert_allclose(gd[a], want_dl, rtol=1e-5, atol=1e-7)
            assert abs(got_loss[a].item() - want_l) <= 1e-5 * max(1.0, abs(want_l))


def test_static_loss_flags_bad_labels_and_then_clears():
    n, B, C = 2, 8, 5
    logits = torch.randn(n * B, C, device=DEV)
    labels = torch.randint(0, C, (n * B,), dtype=torch.int32, device=DEV)
    d, loss = torch.empty_like(logits), torch.empty(n, device=DEV)
    flags = torch.zeros(1, dtype=torch.int32, device=DEV)
    bad = labels.clone(); bad[3] = C
    pb.softmax_ce_static(logits, bad, n, B, C, d, loss, flags); torch.cuda.synchronize()
    assert flags.item() != 0
    pb.softmax_ce_static(logits, labels, n, B, C, d, loss, flags); torch.cuda.synchronize()
    assert flags.item() == 0                                  # slots are cleared at every call
    want = torch.nn.functional.cross_entropy(logits.view(n, B, C).transpose(1, 2), labels.view(n, B).long(), reduction="none").mean(dim=1)
    assert torch.allclose(loss, want, rtol=1e-5, atol=1e-6)


def test_static_loss_rejects_sizes_beyond_its_capacity():
    t = torch.zeros(8, device=DEV)
    lab = torch.zeros(8, dtype=torch.int32, device=DEV)
    with pytest.raises(pb.ParleError) as e:
        pb.softmax_ce_static(t, lab, pb.STATIC_LOSS_MAX_ROWS // 4 + 1, 4, 1, t, t)
    assert e.value.code == -8 and "capacity" in str(e.value)
    with pytest.raises(pb.ParleError) as e:
        pb.softmax_ce_static(t, lab, 0, 4, 2, t, t)
    assert e.value.code == -1
