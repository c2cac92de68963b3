"""The seeded generator: reproducible, addressable per tensor, right moments."""
import numpy as np

import synth_inputs as si


def test_streams_are_reproducible_and_distinct():
    a = si.normal_f32(si.stream_key(1, 2, 3), (1000,))
    b = si.normal_f32(si.stream_key(1, 2, 3), (1000,))
    c = si.normal_f32(si.stream_key(1, 2, 4), (1000,))
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    # a prefix of a longer draw is the same stream
    assert np.array_equal(si.normal_f32(si.stream_key(1, 2, 3), (500,)), a[:500])


def test_moments():
    z = si.normal01(si.stream_key(7, 0), 400_000)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01
    assert abs((z ** 3).mean()) < 0.03 and abs((z ** 4).mean() - 3) < 0.1
    u = si.uniform01(si.stream_key(7, 1), 400_000)
    assert 0 < u.min() and u.max() < 1 and abs(u.mean() - 0.5) < 0.005 and abs(u.var() - 1 / 12) < 0.002


def test_init_and_batches_follow_the_config():
    cfg = si.C1
    layers = si.init_replica(cfg, 1)
    assert [W.shape for W, _ in layers] == [(32, 64), (10, 32)]
    assert all(np.all(b == 0) for _, b in layers)
    assert abs(layers[0][0].std() - 64 ** -0.5) < 0.01
    assert not np.array_equal(layers[0][0], si.init_replica(cfg, 0)[0][0])
    X, c = si.round_batches(cfg, 0)
    assert X.shape == (5, 3, 16, 64) and c.shape == (5, 3, 16) and c.dtype == np.int32
    assert 0 <= c.min() and c.max() < 10 and len(np.unique(c)) > 3
    Xs, cs = si.round_batches(cfg, 0, shared=True)
    assert np.array_equal(Xs[:, 0], Xs[:, 2]) and np.array_equal(Xs[:, 0], X[:, 0])
    assert sum(cfg.dims[l + 1] * (cfg.dims[l] + 1) for l in range(2)) == cfg.n_params == 2410


def test_mnist_shaped_teacher_uses_all_classes():
    cfg = si.C2.scaled(batch=64, L=1, n=2)
    X, c = si.round_batches(cfg, 0)
    assert X.min() >= 0 and X.max() <= 1
    assert len(np.unique(c)) >= 5


def test_split_dataset_gives_each_replica_its_own_shard():
    cfg = si.C1.scaled(n=3, L=4)
    D = 90
    X, c, idx = si.dataset_round_batches(cfg, 0, D, split=True)
    for a in range(cfg.n):
        lo, hi = si.shard_bounds(D, cfg.n, a)
        assert (lo, hi) == (30 * a, 30 * a + 30)
        assert idx[:, a].min() >= lo and idx[:, a].max() < hi
    Xf, cf, idxf = si.dataset_round_batches(cfg, 0, D, split=False)
    assert idxf[:, 0].max() >= 30 and idxf.min() >= 0 and idxf.max() < D      # full data: replica 0 leaves shard 0
    # a sample is the same whoever draws it, and so is its label
    k = int(idx[0, 1, 0])
    assert np.array_equal(X[0, 1, 0], si.dataset_sample(cfg, k))
    where = np.argwhere(idxf == k)
    for l, a, i in where[:3]:
        assert np.array_equal(Xf[l, a, i], X[0, 1, 0]) and cf[l, a, i] == c[0, 1, 0]
