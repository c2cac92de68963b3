"""The C-ABI library builds, loads without a GPU and exports every symbol the
header declares; host-side argument checking and layout planning."""
import ctypes
import math
import os
import re

import pytest

import paper_1707_00424_b200 as pb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "parle.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(parle_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    L = pb.lib()
    names = declared_symbols()
    assert "parle_init" in names and "parle_inner_step" in names and "parle_outer_step" in names and "parle_mean" in names
    for name in names:
        assert hasattr(L, name), name


def test_layout_matches_the_documented_packing():
    m = pb.Parle(3, (64, 32, 10), 16)
    assert m.param_count == 64 * 32 + 32 + 32 * 10 + 10 == 2410
    assert m.layer_offset(0) == (0, 2048) and m.layer_offset(1) == (2080, 2400)
    assert m.stride == 2432 and m.stride % 32 == 0
    m = pb.Parle(2, (37, 19, 7), 5)
    (w0, b0), (w1, b1) = m.layer_offset(0), m.layer_offset(1)
    assert w0 == 0 and b0 == 704 and w1 == 736 and b1 == 896 and m.stride == 928
    for o in (w0, b0, w1, b1):
        assert o % 32 == 0
    flat = pb.Parle(3, (1000003,), 0)
    assert flat.param_count == 1000003 and flat.stride == 1000032
    big = pb.Parle(16, (4096, 8192, 8192, 8192, 8192, 1000), 256, pb.GEMM_BF16)
    assert big.param_count == 243106792
    assert big.workspace_bytes > 16 * big.stride * 2


@pytest.mark.parametrize("kw", [
    dict(n=0), dict(n=65), dict(alpha=1.0), dict(alpha=-0.1), dict(gamma=0.0), dict(rho=-1.0),
    dict(eta=0.0), dict(eta_prime=-1.0), dict(dims=(4, 0, 3)), dict(batch=0), dict(gemm_dtype=7),
    dict(gamma=float("nan")),
])
def test_init_rejects_bad_arguments(kw):
    args = dict(n=2, dims=(8, 8, 4), batch=8, gemm_dtype=0)
    hyper = dict(gamma=1.0, rho=1.0, alpha=0.75, eta=0.1, eta_prime=0.1)
    for k, v in kw.items():
        (args if k in args else hyper)[k] = v
    with pytest.raises(pb.ParleError) as e:
        pb.Parle(args["n"], args["dims"], args["batch"], args["gemm_dtype"], **hyper)
    assert e.value.code == -1


def test_bf16_path_rejects_shapes_it_cannot_take_and_infinite_coupling_is_allowed():
    with pytest.raises(pb.ParleError) as e:
        pb.Parle(2, (10, 16, 4), 8, pb.GEMM_BF16)
    assert e.value.code == -7
    with pytest.raises(pb.ParleError):
        pb.Parle(2, (16, 16, 4), 12, pb.GEMM_BF16)
    pb.Parle(2, (16, 16, 5), 8, pb.GEMM_BF16)            # the last width is free
    m = pb.Parle(2, (8, 4), 4, gamma=math.inf, rho=math.inf)
    m.set_coupling(math.inf, 2.0)
    with pytest.raises(pb.ParleError):
        m.set_coupling(0.0, 1.0)


def test_calls_before_bind_fail_cleanly():
    m = pb.Parle(2, (8, 4), 4)
    for call in (m.round_begin, m.outer_step, m.mean):
        with pytest.raises(pb.ParleError) as e:
            call()
        assert e.value.code == -2
    assert m.status() == 0 and m.launch_count == 0
    L = pb.lib()
    assert L.parle_strerror(-5) == b"call out of order"
    assert L.parle_param_count(None) == 0
    assert L.parle_round_begin(None) == -1


def test_scoping_schedule_host_function():
    # Eq. (scoping) with the paper's constants; values worked out by hand
    assert pb.scoping(100.0, 1.0, 50, 0) == (100.0, 1.0)
    g, r = pb.scoping(100.0, 1.0, 50, 7)
    assert abs(g - 100 * 0.99 ** 7) < 1e-10 and abs(r - 0.99 ** 7) < 1e-12
    assert pb.scoping(100.0, 1.0, 50, 459) == (1.0, 0.1)
    assert pb.scoping(100.0, 1.0, 50, 458)[0] > 1.0 and pb.scoping(100.0, 1.0, 50, 230)[1] == 0.1
    with pytest.raises(pb.ParleError):
        pb.scoping(100.0, 1.0, 0, 1)
    m = pb.Parle(2, (8, 4), 4)
    m.set_weight_decay(1e-3)
    with pytest.raises(pb.ParleError):
        m.set_weight_decay(-1.0)


def test_path_switches_check_their_arguments_without_a_gpu():
    m = pb.Parle(2, (256, 256, 8), 64)                   # fp32: the tensor-core path exists for it, but nothing is bound yet
    assert not m.fp32_tensor_cores_active
    for mode in (0, 1, 2):
        m.set_fp32_tensor_cores(mode)
    with pytest.raises(pb.ParleError) as e:
        m.set_fp32_tensor_cores(3)
    assert e.value.code == -1
    with pytest.raises(pb.ParleError):
        pb.Parle(2, (64, 64, 8), 64, pb.GEMM_BF16).set_fp32_tensor_cores(1)     # a bf16 context has no such switch
    m.set_paired_z_update(False); m.set_paired_z_update(True)
    # the workspace of an fp32 context whose shapes allow the tensor-core path holds the hi/lo operand pairs too
    odd = pb.Parle(2, (254, 256, 8), 64)                 # 254 is not a multiple of 4: FMA pipes only
    assert m.workspace_bytes > odd.workspace_bytes + 2 * 2 * m.stride * 4
