"""Host-side checks that need no GPU: the shared library loads, exports every symbol the header
declares, and its launch-free entry points validate their arguments."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def uoe():
    import __graft_entry__ as ge
    ge.build()
    import paper_2503_02495_b200 as mod
    return mod


def test_library_exports_every_declared_symbol(uoe):
    header = open(os.path.join(ROOT, "include", "uoe.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(uoe_[a-z_0-9]+)\s*\(", header))
    assert {"uoe_route", "uoe_mlp_forward", "uoe_mlp_backward", "uoe_smha_forward", "uoe_workspace_bytes",
            "uoe_max_routed_rows", "uoe_status_string", "uoe_read_device_status", "uoe_workspace_init", "uoe_launch_count", "uoe_tensor_map_encodings",
            "uoe_profile_enable", "uoe_profile_count", "uoe_profile_get"} <= names
    lib = ctypes.CDLL(uoe.LIB_PATH)
    for nm in names:
        assert hasattr(lib, nm), nm


def test_sizes_and_validation(uoe):
    p = uoe.Problem(B=2, L=256, L_valid=256, d=256, n=4, k=2, m=8, c=4, d_e=256, dtype="f32", act="gelu_erf")
    assert uoe.uoe_max_routed_rows(p) % uoe.UOE_ROW_ALIGN == 0
    assert uoe.uoe_max_routed_rows(p) >= 2 * 2 * 4 * 32
    assert uoe.uoe_workspace_bytes(p, uoe.UOE_OP_ROUTE) > 0
    assert uoe.uoe_workspace_bytes(p, uoe.UOE_OP_MLP_FWD) >= uoe.uoe_max_routed_rows(p) * (256 + 256 + 256) * 4
    bad = uoe.Problem(B=2, L=250, L_valid=250, d=256, n=4, k=2, m=8, c=4, d_e=256)      # L % m != 0
    assert uoe.uoe_workspace_bytes(bad, uoe.UOE_OP_ROUTE) == 0
    bad = uoe.Problem(B=2, L=256, L_valid=256, d=256, n=4, k=5, m=8, c=4, d_e=256)      # k > n
    assert uoe.uoe_max_routed_rows(bad) == 0
    bad = uoe.Problem(B=2, L=256, L_valid=300, d=256, n=4, k=2, m=8, c=4, d_e=256)      # L_valid > L
    assert uoe.uoe_max_routed_rows(bad) == 0
    assert uoe.status_string(0) == "ok" and "workspace" in uoe.status_string(3)


def test_null_arguments_are_rejected_before_any_launch(uoe):
    lib = ctypes.CDLL(uoe.LIB_PATH)
    p = uoe.Problem(B=2, L=256, L_valid=256, d=256, n=4, k=2, m=8, c=4, d_e=256, dtype="f32").c_struct()
    lib.uoe_route.restype = ctypes.c_int
    st = lib.uoe_route(ctypes.byref(p), *([None] * 9), ctypes.c_size_t(0), None)
    assert st == 1
    lib.uoe_mlp_forward.restype = ctypes.c_int
    st = lib.uoe_mlp_forward(ctypes.byref(p), *([None] * 12), ctypes.c_size_t(0), None)
    assert st == 1
    st = lib.uoe_route(None, *([None] * 9), ctypes.c_size_t(0), None)
    assert st == 1


def test_every_entry_point_validates_on_the_host(uoe):
    """Null pointers, bad problems and unsupported shapes are answered with a status code before anything is launched,
    so these calls are safe without a GPU."""
    lib = ctypes.CDLL(uoe.LIB_PATH)
    for name in ("uoe_mlp_backward", "uoe_smha_forward", "uoe_smha_backward", "uoe_route_static", "uoe_route_balance",
                 "uoe_workspace_init", "uoe_read_device_status"):
        getattr(lib, name).restype = ctypes.c_int
    att = uoe.Problem(B=2, L=256, L_valid=256, d=256, n=4, k=2, m=8, c=4, H=4, d_h=64).c_struct()
    mlp = uoe.Problem(B=2, L=256, L_valid=256, d=256, n=4, k=2, m=8, c=4, d_e=256).c_struct()
    sz0 = ctypes.c_size_t(0)
    assert lib.uoe_mlp_backward(ctypes.byref(mlp), *([None] * 17), sz0, None) == 1
    assert lib.uoe_smha_forward(ctypes.byref(att), *([None] * 12), sz0, None) == 1
    assert lib.uoe_smha_backward(ctypes.byref(att), *([None] * 20), sz0, None) == 1
    assert lib.uoe_route_static(ctypes.byref(mlp), *([None] * 8), None) == 1
    assert lib.uoe_route_balance(ctypes.byref(mlp), None, ctypes.c_float(1.0), None, None, None, None) == 1
    lib.uoe_route_balance_backward.restype = ctypes.c_int
    assert lib.uoe_route_balance_backward(ctypes.byref(mlp), None, None, None, ctypes.c_float(1.0), None, None, None, None,
                                          sz0, None) == 1
    assert lib.uoe_workspace_init(None, sz0, None) == 1
    assert lib.uoe_read_device_status(None, None) == 1
    # a problem that is itself invalid is refused whatever the pointers are
    odd_rope = uoe.Problem(B=2, L=256, L_valid=256, d=256, n=4, k=2, m=8, c=4, H=4, d_h=64, d_rope=3)
    assert uoe.uoe_workspace_bytes(odd_rope, uoe.UOE_OP_SMHA_FWD) == 0
    big_rope = uoe.Problem(B=2, L=256, L_valid=256, d=256, n=4, k=2, m=8, c=4, H=4, d_h=64, d_rope=66)
    assert uoe.uoe_workspace_bytes(big_rope, uoe.UOE_OP_SMHA_FWD) == 0
    ok_rope = uoe.Problem(B=2, L=256, L_valid=256, d=256, n=4, k=2, m=8, c=4, H=4, d_h=64, d_rope=32)
    assert uoe.uoe_workspace_bytes(ok_rope, uoe.UOE_OP_SMHA_FWD) > 0
    assert uoe.uoe_workspace_bytes(ok_rope, uoe.UOE_OP_SMHA_BWD) > uoe.uoe_workspace_bytes(ok_rope, uoe.UOE_OP_SMHA_FWD)
    # the router's tickets live in a fixed control block: more samples than it holds is "unsupported", not a fault
    huge = uoe.Problem(B=300000, L=64, L_valid=64, d=64, n=4, k=2, m=8, c=4, d_e=64).c_struct()
    dummy = ctypes.c_void_p(4096)        # non-null, 16-byte aligned, never dereferenced: validation fails first
    lib.uoe_route.restype = ctypes.c_int
    st = lib.uoe_route(ctypes.byref(huge), dummy, dummy, dummy, dummy, dummy, dummy, dummy, dummy, dummy,
                       ctypes.c_size_t(1 << 40), None)
    assert st == 2
