"""Test helpers: move parameters between the oracle's dense packing and the
library's padded [n, stride] layout (offsets come from parle_layer_offset),
and the relative-L2 parity metric."""
import numpy as np


def offsets(model):
    return [model.layer_offset(l) for l in range(len(model.dims) - 1)]


def to_padded(model, dense):
    """dense [n, P] (oracle packing) -> [n, stride] float32 with zero padding."""
    dense = np.asarray(dense)
    out = np.zeros((dense.shape[0], model.stride), dtype=np.float32)
    o = 0
    for l, (w_off, b_off) in enumerate(offsets(model)):
        nw = model.dims[l + 1] * model.dims[l]
        nb = model.dims[l + 1]
        out[:, w_off:w_off + nw] = dense[:, o:o + nw]; o += nw
        out[:, b_off:b_off + nb] = dense[:, o:o + nb]; o += nb
    assert o == dense.shape[1]
    return out


def to_dense(model, padded):
    """[n, stride] (or [stride]) -> [n, P] float64 in the oracle's packing."""
    padded = np.asarray(padded, dtype=np.float64)
    single = padded.ndim == 1
    if single:
        padded = padded[None]
    parts = []
    for l, (w_off, b_off) in enumerate(offsets(model)):
        nw = model.dims[l + 1] * model.dims[l]
        nb = model.dims[l + 1]
        parts += [padded[:, w_off:w_off + nw], padded[:, b_off:b_off + nb]]
    out = np.concatenate(parts, axis=1)
    return out[0] if single else out


def padding_mask(model):
    m = np.ones(model.stride, dtype=bool)
    for l, (w_off, b_off) in enumerate(offsets(model)):
        m[w_off:w_off + model.dims[l + 1] * model.dims[l]] = False
        m[b_off:b_off + model.dims[l + 1]] = False
    return m


def rel_l2(got, want):
    got = np.asarray(got, np.float64); want = np.asarray(want, np.float64)
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))


def bf16_weight(a):
    """The library's bf16 copy of a weight, as fp64: the fp32 value rounded to the nearest bf16 with ties away from
    zero (upper half of the fp32 word + 0x8000).  Activations use ties-to-even (the oracle's round_to_bf16); the two
    differ on exact ties only."""
    u = np.asarray(a, np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x8000) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(a))
