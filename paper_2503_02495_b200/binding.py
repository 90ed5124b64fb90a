"""ctypes binding of libuoe.so: argument marshalling only.

Every function here has the name and argument order of its C entry point (include/uoe.h), takes
torch CUDA tensors, allocates the outputs and the workspace with torch, passes raw pointers and the
current CUDA stream, and raises UoeError on a non-zero status.  No arithmetic of the method lives
in Python.  If the shared library is missing, importing this module fails: there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libuoe.so")

UOE_ROW_ALIGN = 128
UOE_F32, UOE_BF16 = 0, 1
ACTS = {"gelu_erf": 0, "gelu_tanh": 1, "silu": 2, "identity": 3}
UOE_FLAG_RESIDUAL, UOE_FLAG_GATE, UOE_FLAG_CAUSAL, UOE_FLAG_DYNAMIC_C, UOE_FLAG_GENERAL_PATH = 1, 2, 4, 8, 16
UOE_OP_ROUTE, UOE_OP_MLP_FWD, UOE_OP_MLP_BWD, UOE_OP_SMHA_FWD, UOE_OP_SMHA_BWD = 0, 1, 2, 3, 4
UOE_OP_BALANCE_BWD = 5


class UoeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class _Routing(ctypes.Structure):
    _fields_ = [(f, ctypes.c_void_p) for f in ("expert_idx", "patch_idx", "gate", "p_samp", "p_patch", "expert_offsets")]


class _Problem(ctypes.Structure):
    _fields_ = [(f, ctypes.c_int32) for f in
                ("B", "L", "L_valid", "d", "n", "k", "m", "c", "d_e", "H", "d_h", "dtype", "act")] + \
               [("flags", ctypes.c_uint32), ("d_rope", ctypes.c_int32)]


@dataclass
class Problem:
    """Mirror of the C struct uoe_problem."""
    B: int
    L: int
    L_valid: int
    d: int
    n: int
    k: int
    m: int
    c: int
    d_e: int = 0
    H: int = 0
    d_h: int = 0
    dtype: str = "bf16"
    act: str = "silu"
    residual: bool = True
    gate: bool = True
    causal: bool = False
    dynamic_c: bool = False
    d_rope: int = 0
    general_path: bool = False      # UOE_FLAG_GENERAL_PATH: no single-mode shortcuts (same results)

    def c_struct(self) -> _Problem:
        flags = (UOE_FLAG_RESIDUAL if self.residual else 0) | (UOE_FLAG_GATE if self.gate else 0) | \
                (UOE_FLAG_CAUSAL if self.causal else 0) | (UOE_FLAG_DYNAMIC_C if self.dynamic_c else 0) | \
                (UOE_FLAG_GENERAL_PATH if self.general_path else 0)
        return _Problem(self.B, self.L, self.L_valid, self.d, self.n, self.k, self.m, self.c, self.d_e, self.H,
                        self.d_h, UOE_BF16 if self.dtype == "bf16" else UOE_F32, ACTS[self.act], flags, self.d_rope)

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def l_p(self) -> int:
        return self.L // self.m

    @property
    def l_a(self) -> int:
        return self.c * self.l_p


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python paper_2503_02495_b200/build.py` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, sz, i32p, f32p = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p
    pp = ctypes.POINTER(_Problem)
    lib.uoe_max_routed_rows.restype = ctypes.c_int64
    lib.uoe_max_routed_rows.argtypes = [pp]
    lib.uoe_workspace_bytes.restype = sz
    lib.uoe_workspace_bytes.argtypes = [pp, ctypes.c_int]
    lib.uoe_route.restype = ctypes.c_int
    lib.uoe_route.argtypes = [pp, vp, vp, i32p, i32p, f32p, f32p, f32p, i32p, vp, sz, vp]
    lib.uoe_route_static.restype = ctypes.c_int
    lib.uoe_route_static.argtypes = [pp, vp, vp, i32p, i32p, f32p, f32p, f32p, i32p, vp]
    lib.uoe_mlp_forward.restype = ctypes.c_int
    lib.uoe_mlp_forward.argtypes = [pp, vp, vp, vp, vp, vp, i32p, i32p, f32p, i32p, vp, vp, vp, sz, vp]
    lib.uoe_mlp_backward.restype = ctypes.c_int
    lib.uoe_mlp_backward.argtypes = [pp, vp, vp, vp, vp, i32p, i32p, f32p, i32p, f32p, f32p, vp, vp, vp, f32p, f32p,
                                     f32p, vp, sz, vp]
    lib.uoe_smha_forward.restype = ctypes.c_int
    lib.uoe_smha_forward.argtypes = [pp, vp, vp, vp, vp, vp, i32p, i32p, f32p, i32p, vp, f32p, vp, sz, vp]
    lib.uoe_smha_backward.restype = ctypes.c_int
    lib.uoe_smha_backward.argtypes = [pp, vp, vp, vp, vp, vp, vp, i32p, i32p, f32p, i32p, f32p, f32p, vp, vp, f32p, f32p,
                                      f32p, f32p, f32p, vp, sz, vp]
    lib.uoe_route_balance.restype = ctypes.c_int
    lib.uoe_route_balance.argtypes = [pp, f32p, ctypes.c_float, f32p, i32p, i32p, vp]
    lib.uoe_route_balance_backward.restype = ctypes.c_int
    lib.uoe_route_balance_backward.argtypes = [pp, vp, vp, f32p, ctypes.c_float, f32p, vp, f32p, vp, sz, vp]
    lib.uoe_block_workspace_bytes.restype = sz
    lib.uoe_block_workspace_bytes.argtypes = [pp, pp]
    lib.uoe_block_forward.restype = ctypes.c_int
    lib.uoe_block_forward.argtypes = [pp, pp] + [vp] * 9 + [ctypes.POINTER(_Routing)] * 2 + [vp, vp, vp, f32p, vp, sz, vp]
    lib.uoe_status_string.restype = ctypes.c_char_p
    lib.uoe_status_string.argtypes = [ctypes.c_int]
    lib.uoe_workspace_init.restype = ctypes.c_int
    lib.uoe_workspace_init.argtypes = [vp, sz, vp]
    lib.uoe_read_device_status.restype = ctypes.c_int
    lib.uoe_read_device_status.argtypes = [vp, vp]
    lib.uoe_launch_count.restype = ctypes.c_int64
    lib.uoe_launch_count.argtypes = []
    lib.uoe_tensor_map_encodings.restype = ctypes.c_int64
    lib.uoe_tensor_map_encodings.argtypes = []
    lib.uoe_profile_enable.restype = None
    lib.uoe_profile_enable.argtypes = [ctypes.c_int]
    lib.uoe_profile_count.restype = ctypes.c_int
    lib.uoe_profile_count.argtypes = []
    lib.uoe_profile_get.restype = ctypes.c_int
    lib.uoe_profile_get.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_float)]
    return lib


_lib = _load()


def status_string(status: int) -> str:
    return _lib.uoe_status_string(int(status)).decode()


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(st: int, where: str):
    if st != 0:
        raise UoeError(st, where)


def _contig(t, dtype=None):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    if dtype is not None:
        assert t.dtype == dtype, f"expected {dtype}, got {t.dtype}"
    return t


def uoe_max_routed_rows(prob: Problem) -> int:
    return int(_lib.uoe_max_routed_rows(ctypes.byref(prob.c_struct())))


def uoe_workspace_bytes(prob: Problem, op: int) -> int:
    return int(_lib.uoe_workspace_bytes(ctypes.byref(prob.c_struct()), op))


def uoe_launch_count() -> int:
    return int(_lib.uoe_launch_count())


def uoe_tensor_map_encodings() -> int:
    return int(_lib.uoe_tensor_map_encodings())


def uoe_profile_enable(on: bool) -> None:
    _lib.uoe_profile_enable(1 if on else 0)


def uoe_profile_records():
    """[(label, milliseconds)] of every launch recorded since uoe_profile_enable(True)."""
    out = []
    for i in range(_lib.uoe_profile_count()):
        name, ms = ctypes.c_char_p(), ctypes.c_float()
        _check(_lib.uoe_profile_get(i, ctypes.byref(name), ctypes.byref(ms)), "uoe_profile_get")
        out.append((name.value.decode(), float(ms.value)))
    return out


def alloc_workspace(prob: Problem, op: int, device="cuda") -> torch.Tensor:
    nbytes = uoe_workspace_bytes(prob, op)
    if nbytes == 0:
        raise UoeError(1, "uoe_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    with torch.cuda.device(ws.device):
        _check(_lib.uoe_workspace_init(_ptr(ws), nbytes, _stream()), "uoe_workspace_init")
    return ws


def uoe_read_device_status(ws: torch.Tensor) -> int:
    return int(_lib.uoe_read_device_status(_ptr(ws), _stream()))


@dataclass
class Routing:
    expert_idx: torch.Tensor      # [B,k] int32
    patch_idx: torch.Tensor       # [B,k,c] int32
    gate: torch.Tensor            # [B,k,c] float32
    p_samp: torch.Tensor          # [B,n] float32
    p_patch: torch.Tensor         # [B,n,m] float32
    expert_offsets: torch.Tensor  # [n+1] int32


def alloc_routing(prob: Problem, device="cuda") -> Routing:
    i32, f32 = torch.int32, torch.float32
    return Routing(torch.empty(prob.B, prob.k, dtype=i32, device=device),
                   torch.empty(prob.B, prob.k, prob.c, dtype=i32, device=device),
                   torch.empty(prob.B, prob.k, prob.c, dtype=f32, device=device),
                   torch.empty(prob.B, prob.n, dtype=f32, device=device),
                   torch.empty(prob.B, prob.n, prob.m, dtype=f32, device=device),
                   torch.empty(prob.n + 1, dtype=i32, device=device))


def uoe_route(prob: Problem, x, W_r, out: Routing | None = None, ws=None, check: bool = True) -> Routing:
    _contig(x, prob.torch_dtype)
    _contig(W_r, prob.torch_dtype)
    r = out if out is not None else alloc_routing(prob, x.device)
    ws = ws if ws is not None else alloc_workspace(prob, UOE_OP_ROUTE, x.device)
    st = _lib.uoe_route(ctypes.byref(prob.c_struct()), _ptr(x), _ptr(W_r), _ptr(r.expert_idx), _ptr(r.patch_idx),
                        _ptr(r.gate), _ptr(r.p_samp), _ptr(r.p_patch), _ptr(r.expert_offsets), _ptr(ws), ws.numel(),
                        _stream())
    _check(st, "uoe_route")
    if check:
        _check(uoe_read_device_status(ws), "uoe_route (device)")
    return r


UOE_ROUTE_STATIC_SCRATCH_BYTES = 2 << 20


def uoe_route_static(prob: Problem, x, W_r, out: Routing | None = None) -> Routing:
    """uoe_route for callers that cannot supply a workspace: the scratch is a fixed array inside the
    library (limit UOE_ROUTE_STATIC_SCRATCH_BYTES).  Only the output tensors are created here, and only
    when `out` is not given; the C call itself allocates nothing.  Calls on one device must not overlap."""
    _contig(x, prob.torch_dtype)
    _contig(W_r, prob.torch_dtype)
    r = out if out is not None else alloc_routing(prob, x.device)
    st = _lib.uoe_route_static(ctypes.byref(prob.c_struct()), _ptr(x), _ptr(W_r), _ptr(r.expert_idx),
                               _ptr(r.patch_idx), _ptr(r.gate), _ptr(r.p_samp), _ptr(r.p_patch),
                               _ptr(r.expert_offsets), _stream())
    _check(st, "uoe_route_static")
    return r


def uoe_mlp_forward(prob: Problem, x, W1, W2, r: Routing, b1=None, b2=None, y=None, saved_h=None, ws=None,
                    check: bool = True):
    for t in (x, W1, W2, b1, b2):
        _contig(t, prob.torch_dtype)
    y = y if y is not None else torch.empty_like(x)
    ws = ws if ws is not None else alloc_workspace(prob, UOE_OP_MLP_FWD, x.device)
    st = _lib.uoe_mlp_forward(ctypes.byref(prob.c_struct()), _ptr(x), _ptr(W1), _ptr(W2), _ptr(b1), _ptr(b2),
                              _ptr(r.expert_idx), _ptr(r.patch_idx), _ptr(r.gate), _ptr(r.expert_offsets),
                              _ptr(y), _ptr(saved_h), _ptr(ws), ws.numel(), _stream())
    _check(st, "uoe_mlp_forward")
    if check:
        _check(uoe_read_device_status(ws), "uoe_mlp_forward (device)")
    return y


def alloc_saved_h(prob: Problem, device="cuda") -> torch.Tensor:
    return torch.empty(uoe_max_routed_rows(prob), prob.d_e, dtype=prob.torch_dtype, device=device)


def uoe_mlp_backward(prob: Problem, x, W1, W2, W_r, r: Routing, saved_h, dy, dx=None, dW1=None, dW2=None,
                     dW_r=None, ws=None, check: bool = True):
    for t in (x, W1, W2, W_r, saved_h, dy):
        _contig(t, prob.torch_dtype)
    f32 = torch.float32
    dx = dx if dx is not None else torch.empty_like(x)
    dW1 = dW1 if dW1 is not None else torch.empty(W1.shape, dtype=f32, device=x.device)
    dW2 = dW2 if dW2 is not None else torch.empty(W2.shape, dtype=f32, device=x.device)
    dW_r = dW_r if dW_r is not None else torch.empty(W_r.shape, dtype=f32, device=x.device)
    ws = ws if ws is not None else alloc_workspace(prob, UOE_OP_MLP_BWD, x.device)
    st = _lib.uoe_mlp_backward(ctypes.byref(prob.c_struct()), _ptr(x), _ptr(W1), _ptr(W2), _ptr(W_r),
                               _ptr(r.expert_idx), _ptr(r.patch_idx), _ptr(r.gate), _ptr(r.expert_offsets),
                               _ptr(r.p_samp), _ptr(r.p_patch), _ptr(saved_h), _ptr(dy), _ptr(dx), _ptr(dW1),
                               _ptr(dW2), _ptr(dW_r), _ptr(ws), ws.numel(), _stream())
    _check(st, "uoe_mlp_backward")
    if check:
        _check(uoe_read_device_status(ws), "uoe_mlp_backward (device)")
    return dx, dW1, dW2, dW_r


def uoe_smha_forward(prob: Problem, x, Wq, Wk, Wv, Wo, r: Routing, y=None, lse=None, ws=None, check: bool = True):
    for t in (x, Wq, Wk, Wv, Wo):
        _contig(t, prob.torch_dtype)
    y = y if y is not None else torch.empty_like(x)
    ws = ws if ws is not None else alloc_workspace(prob, UOE_OP_SMHA_FWD, x.device)
    st = _lib.uoe_smha_forward(ctypes.byref(prob.c_struct()), _ptr(x), _ptr(Wq), _ptr(Wk), _ptr(Wv), _ptr(Wo),
                               _ptr(r.expert_idx), _ptr(r.patch_idx), _ptr(r.gate), _ptr(r.expert_offsets),
                               _ptr(y), _ptr(lse), _ptr(ws), ws.numel(), _stream())
    _check(st, "uoe_smha_forward")
    if check:
        _check(uoe_read_device_status(ws), "uoe_smha_forward (device)")
    return y


def uoe_smha_backward(prob: Problem, x, Wq, Wk, Wv, Wo, W_r, r: Routing, dy, dx=None, dWq=None, dWk=None, dWv=None,
                      dWo=None, dW_r=None, ws=None, check: bool = True):
    for t in (x, Wq, Wk, Wv, Wo, W_r, dy):
        _contig(t, prob.torch_dtype)
    f32 = torch.float32
    new = lambda like: torch.empty(like.shape, dtype=f32, device=x.device)
    dx = dx if dx is not None else torch.empty_like(x)
    dWq = dWq if dWq is not None else new(Wq)
    dWk = dWk if dWk is not None else new(Wk)
    dWv = dWv if dWv is not None else new(Wv)
    dWo = dWo if dWo is not None else new(Wo)
    dW_r = dW_r if dW_r is not None else new(W_r)
    ws = ws if ws is not None else alloc_workspace(prob, UOE_OP_SMHA_BWD, x.device)
    st = _lib.uoe_smha_backward(ctypes.byref(prob.c_struct()), _ptr(x), _ptr(Wq), _ptr(Wk), _ptr(Wv), _ptr(Wo), _ptr(W_r),
                                _ptr(r.expert_idx), _ptr(r.patch_idx), _ptr(r.gate), _ptr(r.expert_offsets),
                                _ptr(r.p_samp), _ptr(r.p_patch), _ptr(dy), _ptr(dx), _ptr(dWq), _ptr(dWk), _ptr(dWv),
                                _ptr(dWo), _ptr(dW_r), _ptr(ws), ws.numel(), _stream())
    _check(st, "uoe_smha_backward")
    if check:
        _check(uoe_read_device_status(ws), "uoe_smha_backward (device)")
    return dx, dWq, dWk, dWv, dWo, dW_r


def uoe_route_balance(prob: Problem, p_patch, alpha: float = 1.0):
    """(lb_loss [B] float32, expert_count [B,n] int32, c_dyn [B] int32) for the patch gate written by uoe_route."""
    _contig(p_patch, torch.float32)
    dev = p_patch.device
    lb = torch.empty(prob.B, dtype=torch.float32, device=dev)
    cnt = torch.empty(prob.B, prob.n, dtype=torch.int32, device=dev)
    cd = torch.empty(prob.B, dtype=torch.int32, device=dev)
    st = _lib.uoe_route_balance(ctypes.byref(prob.c_struct()), _ptr(p_patch), ctypes.c_float(alpha), _ptr(lb), _ptr(cnt),
                                _ptr(cd), _stream())
    _check(st, "uoe_route_balance")
    return lb, cnt, cd


def uoe_route_balance_backward(prob: Problem, x, W_r, p_patch, alpha: float, dloss, ws=None):
    """(dx [B,L,d], dW_r [d,n] float32): gradient of sum(dloss * lb_loss) with respect to x and W_r."""
    _contig(x, prob.torch_dtype)
    _contig(W_r, prob.torch_dtype)
    _contig(p_patch, torch.float32)
    _contig(dloss, torch.float32)
    dx = torch.empty_like(x)
    dW_r = torch.empty(W_r.shape, dtype=torch.float32, device=x.device)
    ws = ws if ws is not None else alloc_workspace(prob, UOE_OP_BALANCE_BWD, x.device)
    st = _lib.uoe_route_balance_backward(ctypes.byref(prob.c_struct()), _ptr(x), _ptr(W_r), _ptr(p_patch),
                                         ctypes.c_float(alpha), _ptr(dloss), _ptr(dx), _ptr(dW_r), _ptr(ws), ws.numel(),
                                         _stream())
    _check(st, "uoe_route_balance_backward")
    return dx, dW_r


def uoe_block_workspace_bytes(att: Problem | None, mlp: Problem | None) -> int:
    pa = ctypes.byref(att.c_struct()) if att is not None else None
    pm = ctypes.byref(mlp.c_struct()) if mlp is not None else None
    return int(_lib.uoe_block_workspace_bytes(pa, pm))


def alloc_block_workspace(att: Problem | None, mlp: Problem | None, device="cuda") -> torch.Tensor:
    nbytes = uoe_block_workspace_bytes(att, mlp)
    if nbytes == 0:
        raise UoeError(1, "uoe_block_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    with torch.cuda.device(ws.device):
        _check(_lib.uoe_workspace_init(_ptr(ws), nbytes, _stream()), "uoe_workspace_init")
    return ws


def _routing_struct(r: Routing | None):
    if r is None:
        return None
    return ctypes.byref(_Routing(*(t.data_ptr() for t in (r.expert_idx, r.patch_idx, r.gate, r.p_samp, r.p_patch,
                                                          r.expert_offsets))))


def uoe_block_forward(att: Problem | None, mlp: Problem | None, x, weights: dict, r_att: Routing | None = None,
                      r_mlp: Routing | None = None, u=None, y=None, saved_h=None, lse=None, ws=None, check: bool = True):
    """One UoE block (SMHA half, then UoME half; either may be None) through the single C entry point.
    `weights` holds Wr_att, Wq, Wk, Wv, Wo and / or Wr_mlp, W1, W2.  Returns y (and fills u, r_att, r_mlp when given)."""
    p0 = att or mlp
    _contig(x, p0.torch_dtype)
    g = lambda name: _contig(weights.get(name), p0.torch_dtype)
    y = y if y is not None else torch.empty_like(x)
    if att is not None and mlp is not None and u is None:
        u = torch.empty_like(x)
    ws = ws if ws is not None else alloc_block_workspace(att, mlp, x.device)
    pa = ctypes.byref(att.c_struct()) if att is not None else None
    pm = ctypes.byref(mlp.c_struct()) if mlp is not None else None
    st = _lib.uoe_block_forward(pa, pm, _ptr(x), _ptr(g("Wr_att")), _ptr(g("Wq")), _ptr(g("Wk")), _ptr(g("Wv")),
                                _ptr(g("Wo")), _ptr(g("Wr_mlp")), _ptr(g("W1")), _ptr(g("W2")), _routing_struct(r_att),
                                _routing_struct(r_mlp), _ptr(u), _ptr(y), _ptr(saved_h), _ptr(lse), _ptr(ws), ws.numel(),
                                _stream())
    _check(st, "uoe_block_forward")
    if check:
        _check(uoe_read_device_status(ws), "uoe_block_forward (device)")
    return y
