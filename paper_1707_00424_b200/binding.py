"""ctypes binding of libparle.so: argument marshalling only.

PyTorch appears here for device memory and streams alone; there is no CPU or
PyTorch fallback -- if the CUDA library cannot be loaded every call fails.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Optional, Sequence

GEMM_FP32, GEMM_BF16 = 0, 1
FLAG_NONFINITE, FLAG_WAIT_LIMIT, FLAG_BAD_LABEL = 1, 2, 4

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB: Optional[C.CDLL] = None


class ParleError(RuntimeError):
    def __init__(self, code: int, what: str, cuda: int = 0):
        self.code = code
        msg = f"{what}: {lib().parle_strerror(code).decode()} ({code})"
        if cuda:
            msg += f" [CUDA error {cuda}]"
        super().__init__(msg)


class _Model(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("dims", C.POINTER(C.c_int)), ("batch", C.c_int), ("gemm_dtype", C.c_int)]


class _Buffers(C.Structure):
    _fields_ = [("x", C.c_void_p), ("y", C.c_void_p), ("z", C.c_void_p), ("grad", C.c_void_p),
                ("xbar", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


def library_path() -> str:
    return os.path.join(_HERE, "libparle.so")


def lib() -> C.CDLL:
    """Load the CUDA library (building it first if the sources are newer)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        from .build import build
        build()
    L = C.CDLL(path)
    vp, ci, cd, sz = C.c_void_p, C.c_int, C.c_double, C.c_size_t
    sig = {
        "parle_init": (ci, [C.POINTER(vp), ci, C.POINTER(_Model), cd, cd, cd, cd, cd]),
        "parle_destroy": (None, [vp]),
        "parle_param_count": (sz, [vp]),
        "parle_stride": (sz, [vp]),
        "parle_workspace_bytes": (sz, [vp]),
        "parle_layer_offset": (ci, [vp, ci, C.POINTER(sz), C.POINTER(sz)]),
        "parle_bind": (ci, [vp, C.POINTER(_Buffers), vp]),
        "parle_round_begin": (ci, [vp]),
        "parle_inner_step": (ci, [vp, vp, vp, vp]),
        "parle_inner_step_host": (ci, [vp, vp, vp, vp]),
        "parle_inner_update": (ci, [vp, vp]),
        "parle_outer_step": (ci, [vp]),
        "parle_mean": (ci, [vp]),
        "parle_round": (ci, [vp, ci, vp, vp, vp]),
        "parle_round_host": (ci, [vp, ci, vp, vp, vp]),
        "parle_set_round_graphs": (ci, [vp, ci]),
        "parle_round_graph_count": (ci, [vp]),
        "parle_set_coupling": (ci, [vp, cd, cd]),
        "parle_set_lr": (ci, [vp, cd, cd]),
        "parle_set_fused_update": (ci, [vp, ci]),
        "parle_set_fp32_tensor_cores": (ci, [vp, ci]),
        "parle_set_paired_z_update": (ci, [vp, ci]),
        "parle_set_split_y": (ci, [vp, ci]),
        "parle_fp32_tensor_cores_active": (ci, [vp]),
        "parle_set_weight_decay": (ci, [vp, cd]),
        "parle_set_wide_tile_threshold": (ci, [vp, ci]),
        "parle_set_pair_gemm": (ci, [vp, ci]),
        "parle_set_fused_loss": (ci, [vp, ci]),
        "parle_bind_momentum": (ci, [vp, vp, vp]),
        "parle_set_momentum": (ci, [vp, cd]),
        "parle_scoping": (ci, [cd, cd, C.c_longlong, C.c_longlong, cd, cd, C.POINTER(cd), C.POINTER(cd)]),
        "parle_status": (ci, [vp, C.POINTER(ci)]),
        "parle_clear_status": (ci, [vp]),
        "parle_profile_enable": (ci, [vp, ci]),
        "parle_profile_read": (ci, [vp, ci, C.POINTER(cd), C.POINTER(C.c_longlong), C.POINTER(C.c_longlong)]),
        "parle_profile_class_count": (ci, []),
        "parle_profile_class_name": (C.c_char_p, [ci]),
        "parle_debug_buffer": (ci, [vp, ci, ci, C.POINTER(sz), C.POINTER(sz)]),
        "parle_softmax_ce_static": (ci, [vp, vp, ci, ci, ci, vp, vp, vp, vp]),
        "parle_launch_count": (C.c_longlong, [vp]),
        "parle_last_cuda_error": (ci, [vp]),
        "parle_strerror": (C.c_char_p, [ci]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    _LIB = L
    return L


def _ptr(t) -> int:
    """Device (or host) address of a torch tensor / raw int / None."""
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    return t.data_ptr()


STATIC_LOSS_MAX_ROWS = 65536


def softmax_ce_static(logits, labels, n: int, B: int, C_: int, dlogits, loss, flags=None, stream=None):
    """Allocation-free loss step (parle_softmax_ce_static): for callers that cannot give the
    library a workspace.  All arguments are caller-owned device tensors; nothing is allocated."""
    import torch
    if stream is None:
        stream = torch.cuda.current_stream(logits.device)
    with torch.cuda.device(logits.device):
        rc = lib().parle_softmax_ce_static(_ptr(logits), _ptr(labels), n, B, C_, _ptr(dlogits), _ptr(loss),
                                           _ptr(flags), C.c_void_p(stream.cuda_stream))
    if rc != 0:
        raise ParleError(rc, "parle_softmax_ce_static")


def scoping(gamma0: float, rho0: float, minibatches_per_epoch: int, round_index: int,
            gamma_floor: float = 1.0, rho_floor: float = 0.1):
    """(gamma, rho) of a round by Eq. (scoping) (parle_scoping)."""
    g, r = C.c_double(), C.c_double()
    rc = lib().parle_scoping(gamma0, rho0, minibatches_per_epoch, round_index, gamma_floor, rho_floor,
                             C.byref(g), C.byref(r))
    if rc != 0:
        raise ParleError(rc, "parle_scoping")
    return g.value, r.value


class Parle:
    """One context = n replicas of one MLP with the scalars of Eq. (parle).

    Mirrors the C entry points one to one (same names without the prefix).
    `alloc()` makes the caller-owned state with torch and binds it.
    """

    def __init__(self, n: int, dims: Sequence[int], batch: int = 0, gemm_dtype: int = GEMM_FP32, *,
                 gamma: float = 1.0, rho: float = 1.0, alpha: float = 0.75, eta: float = 0.1,
                 eta_prime: float = 0.1):
        self._L = lib()
        self.n, self.dims, self.batch, self.gemm_dtype = n, tuple(int(d) for d in dims), batch, gemm_dtype
        arr = (C.c_int * len(self.dims))(*self.dims)
        model = _Model(len(self.dims) - 1, arr, batch, gemm_dtype)
        h = C.c_void_p()
        rc = self._L.parle_init(C.byref(h), n, C.byref(model), gamma, rho, alpha, eta, eta_prime)
        if rc != 0:
            raise ParleError(rc, "parle_init")
        self._h = h
        self.param_count = self._L.parle_param_count(h)
        self.stride = self._L.parle_stride(h)
        self.workspace_bytes = self._L.parle_workspace_bytes(h)
        self.x = self.y = self.z = self.grad = self.xbar = self.workspace = None

    # -- life cycle -------------------------------------------------------
    def close(self):
        if getattr(self, "_h", None):
            self._L.parle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, what: str):
        if rc != 0:
            raise ParleError(rc, what, self._L.parle_last_cuda_error(self._h))

    # -- layout -----------------------------------------------------------
    def layer_offset(self, layer: int):
        w, b = C.c_size_t(), C.c_size_t()
        self._check(self._L.parle_layer_offset(self._h, layer, C.byref(w), C.byref(b)), "parle_layer_offset")
        return w.value, b.value

    # -- memory -----------------------------------------------------------
    def alloc(self, device="cuda:0", stream=None):
        """Allocate x, y, z, grad, xbar and the workspace with torch and bind them."""
        import torch
        dev = torch.device(device)
        with torch.cuda.device(dev):
            mk = lambda *s: torch.zeros(*s, dtype=torch.float32, device=dev)
            self.x, self.y, self.z, self.grad = (mk(self.n, self.stride) for _ in range(4))
            self.xbar = mk(self.stride)
            self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=dev)
            self.bind(self.x, self.y, self.z, self.grad, self.xbar, self.workspace, stream)
        return self

    def bind(self, x, y, z, grad, xbar, workspace, stream=None):
        import torch
        if stream is None:
            stream = torch.cuda.current_stream(x.device)
        self._stream = stream
        b = _Buffers(_ptr(x), _ptr(y), _ptr(z), _ptr(grad), _ptr(xbar), _ptr(workspace),
                     workspace.numel() * workspace.element_size())
        sp = stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream or 0)
        with torch.cuda.device(x.device):
            self._check(self._L.parle_bind(self._h, C.byref(b), C.c_void_p(sp)), "parle_bind")
        self.x, self.y, self.z, self.grad, self.xbar, self.workspace = x, y, z, grad, xbar, workspace
        self._momentum_bound = False          # parle_bind detaches the momentum buffers

    # -- the round --------------------------------------------------------
    def round_begin(self):
        self._check(self._L.parle_round_begin(self._h), "parle_round_begin")

    def inner_step(self, inputs, labels, loss_out=None):
        self._check(self._L.parle_inner_step(self._h, _ptr(inputs), _ptr(labels), _ptr(loss_out)), "parle_inner_step")

    def inner_step_host(self, inputs_host, labels_host, loss_out_host=None):
        self._check(self._L.parle_inner_step_host(self._h, _ptr(inputs_host), _ptr(labels_host), _ptr(loss_out_host)),
                    "parle_inner_step_host")

    def inner_update(self, grad):
        self._check(self._L.parle_inner_update(self._h, _ptr(grad)), "parle_inner_update")

    def outer_step(self):
        self._check(self._L.parle_outer_step(self._h), "parle_outer_step")

    def mean(self):
        self._check(self._L.parle_mean(self._h), "parle_mean")

    def round(self, L: int, inputs, labels, loss_out=None):
        self._check(self._L.parle_round(self._h, L, _ptr(inputs), _ptr(labels), _ptr(loss_out)), "parle_round")

    def round_host(self, L: int, inputs_host, labels_host, loss_out_host=None):
        self._check(self._L.parle_round_host(self._h, L, _ptr(inputs_host), _ptr(labels_host), _ptr(loss_out_host)),
                    "parle_round_host")

    def set_round_graphs(self, on: bool):
        self._check(self._L.parle_set_round_graphs(self._h, 1 if on else 0), "parle_set_round_graphs")

    @property
    def round_graph_count(self) -> int:
        return self._L.parle_round_graph_count(self._h)

    def set_coupling(self, gamma: float, rho: float):
        self._check(self._L.parle_set_coupling(self._h, gamma, rho), "parle_set_coupling")

    def set_lr(self, eta: float, eta_prime: float):
        self._check(self._L.parle_set_lr(self._h, eta, eta_prime), "parle_set_lr")

    def set_momentum(self, mu: float, vy=None, vx=None):
        """Nesterov momentum on the y and x^a steps; allocates (zeroed) vy, vx with torch when not given."""
        import torch
        if mu > 0 and not getattr(self, "_momentum_bound", False):
            have = getattr(self, "vy", None) is not None
            self.vy = vy if vy is not None else (self.vy if have else torch.zeros_like(self.x))
            self.vx = vx if vx is not None else (self.vx if have else torch.zeros_like(self.x))
            self._check(self._L.parle_bind_momentum(self._h, _ptr(self.vy), _ptr(self.vx)), "parle_bind_momentum")
            self._momentum_bound = True
        self._check(self._L.parle_set_momentum(self._h, mu), "parle_set_momentum")

    def set_wide_tile_threshold(self, tiles_per_sm: int):
        self._check(self._L.parle_set_wide_tile_threshold(self._h, tiles_per_sm), "parle_set_wide_tile_threshold")

    def set_fused_loss(self, on: bool):
        """bf16 path, at most 128 classes: softmax cross-entropy backward in the last forward GEMM's epilogue (default on)."""
        self._check(self._L.parle_set_fused_loss(self._h, 1 if on else 0), "parle_set_fused_loss")

    def set_pair_gemm(self, mode: int):
        """bf16 path: hidden-layer forward / data-gradient products on pairs of SMs: 0 never, 1 one launch per layer,
        2 (default) consecutive layers chained in one launch where that pays, 3 always chained."""
        self._check(self._L.parle_set_pair_gemm(self._h, int(mode)), "parle_set_pair_gemm")

    def set_weight_decay(self, lam: float):
        self._check(self._L.parle_set_weight_decay(self._h, lam), "parle_set_weight_decay")

    def set_fused_update(self, on: bool):
        self._check(self._L.parle_set_fused_update(self._h, 1 if on else 0), "parle_set_fused_update")

    def set_paired_z_update(self, on: bool):
        """Whole rounds on the fused bf16 path: update z every other inner step with the two-step form of Eq. (parle_z)."""
        self._check(self._L.parle_set_paired_z_update(self._h, 1 if on else 0), "parle_set_paired_z_update")

    def set_split_y(self, on: bool):
        """Whole rounds on the fused bf16 path: keep y of the weights as bf16 operand copy + lower-half plane between steps."""
        self._check(self._L.parle_set_split_y(self._h, 1 if on else 0), "parle_set_split_y")

    def set_fp32_tensor_cores(self, mode: int):
        """0: FMA pipes, 1: tensor cores (3 x tf32) for wide layers, 2: tensor cores whenever the shapes allow."""
        self._check(self._L.parle_set_fp32_tensor_cores(self._h, mode), "parle_set_fp32_tensor_cores")

    @property
    def fp32_tensor_cores_active(self) -> bool:
        return bool(self._L.parle_fp32_tensor_cores_active(self._h))

    def status(self) -> int:
        f = C.c_int()
        self._check(self._L.parle_status(self._h, C.byref(f)), "parle_status")
        return f.value

    def clear_status(self):
        self._check(self._L.parle_clear_status(self._h), "parle_clear_status")

    DBG_ACT, DBG_ACT_T, DBG_DACT, DBG_DACT_T, DBG_LOGITS, DBG_OPERAND_COPY = range(6)
    DBG_T3_PARAMS, DBG_T3_INPUT_T, DBG_T3_ACT_T, DBG_T3_DACT_T = 6, 8, 10, 12      # hi; + 1 = lo

    def debug_buffer(self, kind: int, layer: int = 0):
        """View (torch, no copy) of an intermediate of the last inner step inside the workspace."""
        import torch
        off, nbytes = C.c_size_t(), C.c_size_t()
        self._check(self._L.parle_debug_buffer(self._h, kind, layer, C.byref(off), C.byref(nbytes)), "parle_debug_buffer")
        raw = self.workspace[off.value:off.value + nbytes.value]
        n, B = self.n, self.batch
        bf = self.gemm_dtype == GEMM_BF16
        d = self.dims[layer + 1]
        if kind == self.DBG_LOGITS:
            return raw.view(torch.float32).view(n, B, self.dims[-1])
        if kind >= self.DBG_T3_PARAMS:
            t = raw.view(torch.float32)
            if kind - (kind & 1) == self.DBG_T3_PARAMS:
                return t.view(n, -1)
            return t.view(n, self.dims[0] if kind - (kind & 1) == self.DBG_T3_INPUT_T else d, B)
        if kind == self.DBG_OPERAND_COPY:
            return raw.view(torch.bfloat16).view(n, -1)
        if kind in (self.DBG_ACT_T, self.DBG_DACT_T):
            return raw.view(torch.bfloat16).view(n, d, B)
        t = raw.view(torch.bfloat16 if bf else torch.float32)
        return t.view(n, B, -1)[:, :, :d]

    def profile_enable(self, on: bool = True):
        self._check(self._L.parle_profile_enable(self._h, 1 if on else 0), "parle_profile_enable")

    def profile_read(self):
        """Synchronises the stream; returns {class name: (total ms, launches)} and the dropped count."""
        k = self._L.parle_profile_class_count()
        ms, cnt, drop = (C.c_double * k)(), (C.c_longlong * k)(), C.c_longlong()
        self._check(self._L.parle_profile_read(self._h, k, ms, cnt, C.byref(drop)), "parle_profile_read")
        out = {self._L.parle_profile_class_name(i).decode(): (ms[i], cnt[i]) for i in range(k) if cnt[i]}
        return out, drop.value

    @property
    def launch_count(self) -> int:
        return self._L.parle_launch_count(self._h)
