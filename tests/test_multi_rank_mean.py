"""Two ranks on CPU (gloo): replicas sharded across ranks, one exchange per round -- the average
of the per-rank means -- must reproduce the single-process round over all replicas (Section 3:
the only coupling between replicas is Eq. parle_x)."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import synth_inputs as si
from oracle import parle_oracle as po


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, rounds, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_1707_00424_b200.parallel import allreduce_mean_
    cfg = si.C1.scaled(n=4)
    per = cfg.n // world
    mine = range(rank * per, (rank + 1) * per)
    hp = po.Hyper(cfg.eta, cfg.eta_prime, cfg.alpha, cfg.gamma, cfg.rho)
    x = np.stack([po.pack(si.init_replica(cfg, a)) for a in mine])
    xbar = torch.from_numpy(x.mean(axis=0)); allreduce_mean_(xbar)
    for r in range(rounds):
        X, c = si.round_batches(cfg, r)
        out = po.parle_round(x, xbar.numpy(), po.mlp_grad_fn(cfg.dims, X[:, list(mine)], c[:, list(mine)]), cfg.L, hp)
        x = out["x"]
        xbar = torch.from_numpy(out["xbar"].copy())      # mean of this rank's replicas
        allreduce_mean_(xbar)                            # the one exchange of the round
    np.save(os.path.join(out_dir, f"x{rank}.npy"), x)
    np.save(os.path.join(out_dir, f"xbar{rank}.npy"), xbar.numpy())
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_process_round(tmp_path):
    world, rounds = 2, 2
    mp.spawn(_worker, args=(world, _free_port(), rounds, str(tmp_path)), nprocs=world, join=True)
    cfg = si.C1.scaled(n=4)
    hp = po.Hyper(cfg.eta, cfg.eta_prime, cfg.alpha, cfg.gamma, cfg.rho)
    x = np.stack([po.pack(si.init_replica(cfg, a)) for a in range(cfg.n)])
    xbar = x.mean(axis=0)
    for r in range(rounds):
        X, c = si.round_batches(cfg, r)
        out = po.parle_round(x, xbar, po.mlp_grad_fn(cfg.dims, X, c), cfg.L, hp)
        x, xbar = out["x"], out["xbar"]
    got_x = np.concatenate([np.load(tmp_path / f"x{r}.npy") for r in range(world)])
    np.testing.assert_allclose(got_x, x, rtol=1e-13, atol=1e-15)
    for r in range(world):
        np.testing.assert_allclose(np.load(tmp_path / f"xbar{r}.npy"), xbar, rtol=1e-13, atol=1e-15)


def test_allreduce_mean_is_identity_without_a_group():
    from paper_1707_00424_b200.parallel import allreduce_mean_
    t = torch.arange(4.0)
    assert torch.equal(allreduce_mean_(t.clone()), t)
