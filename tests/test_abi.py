"""Host-side checks of the C ABI: the library loads, exports every symbol the
public header declares, and rejects bad arguments before touching a device.
No compute is launched here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER_DIR = os.path.join(ROOT, "include")


def _declared_functions():
    names = []
    for fn in sorted(os.listdir(HEADER_DIR)):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(HEADER_DIR, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(ec_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_header_declares_the_three_operations():
    names = _declared_functions()
    for must in ("ec_kv_refresh", "ec_attend", "ec_entropy_gate"):
        assert must in names


def test_library_loads_and_exports_every_declared_symbol():
    import paper_2603_18489_b200 as ec

    raw = ctypes.CDLL(ec.LIB_PATH)
    for name in _declared_functions():
        assert hasattr(raw, name), f"{name} is declared in include/ but not exported"
    assert ec.version() >= 100
    assert ec.status_string(0) == "EC_OK"
    assert "workspace" in ec.status_string(5).lower()


def test_workspace_queries_are_pure_host_functions():
    import paper_2603_18489_b200 as ec

    d = ec.make_desc(1, 768, 32, 32, 128, ec.EC_BF16)
    assert ec.ec_attend_workspace_bytes(d, 34) > 0
    assert ec.ec_attend_workspace_bytes(d, 768) > 0
    assert ec.ec_attend_workspace_bytes(d, 769) == 0      # more active rows than positions
    bad = ec.make_desc(1, 768, 32, 5, 128, ec.EC_BF16)    # 32 % 5 != 0
    assert ec.ec_attend_workspace_bytes(bad, 34) == 0
    assert ec.ec_entropy_gate_workspace_bytes(32, 126464) > 0
    assert ec.ec_entropy_gate_workspace_bytes(0, 126464) == 0


def test_argument_validation_returns_status_codes():
    import paper_2603_18489_b200 as ec

    L = ec.lib
    d = ec.make_desc(1, 64, 4, 4, 64, ec.EC_F32)
    fake = ctypes.c_void_p(0x1000)   # aligned, never dereferenced: every call below fails validation first
    odd = ctypes.c_void_p(0x1004)
    null = None
    # refresh
    assert L.ec_kv_refresh(None, fake, fake, fake, fake, null, 64, null) == 1
    assert L.ec_kv_refresh(ctypes.byref(d), null, fake, fake, fake, null, 64, null) == 1
    assert L.ec_kv_refresh(ctypes.byref(d), odd, fake, fake, fake, null, 64, null) == 4
    assert L.ec_kv_refresh(ctypes.byref(d), fake, fake, fake, fake, null, 10, null) == 2  # identity needs n == L
    assert L.ec_kv_refresh(ctypes.byref(d), fake, fake, fake, fake, fake, 65, null) == 2
    assert L.ec_kv_refresh(ctypes.byref(d), fake, fake, fake, fake, fake, 0, null) == 0   # no-op
    for field, val, code in (("dtype", 7, 3), ("head_dim", 48, 6), ("n_kv_heads", 3, 2), ("batch", 0, 2)):
        b = ec.make_desc(1, 64, 4, 4, 64, ec.EC_F32)
        setattr(b, field, val)
        assert L.ec_kv_refresh(ctypes.byref(b), fake, fake, fake, fake, null, 64, null) == code
    # attend
    assert L.ec_attend(ctypes.byref(d), null, fake, fake, fake, fake, null, 64, fake, fake, 1 << 20, null, null) == 1
    assert L.ec_attend(ctypes.byref(d), fake, fake, null, fake, fake, null, 64, fake, fake, 1 << 20, null, null) == 1
    assert L.ec_attend(ctypes.byref(d), fake, fake, fake, fake, fake, null, 64, fake, null, 0, null, null) == 5
    assert L.ec_attend(ctypes.byref(d), fake, fake, fake, fake, fake, null, 64, odd, fake, 1 << 20, null, null) == 4
    assert L.ec_attend(ctypes.byref(d), fake, fake, fake, fake, fake, null, 0, fake, null, 0, null, null) == 0
    # gate
    g = L.ec_entropy_gate
    ws = 1 << 24
    assert g(null, 1, 32, 1024, 1024, 32, fake, 1.5, null, null, null, fake, fake, fake, ws, null) == 1
    assert g(fake, 5, 32, 1024, 1024, 32, fake, 1.5, null, null, null, fake, fake, fake, ws, null) == 3
    assert g(fake, 1, 32, 1024, 1000, 32, fake, 1.5, null, null, null, fake, fake, fake, ws, null) == 2  # stride < V
    assert g(fake, 1, 32, 1024, 1024, 5, fake, 1.5, null, null, null, fake, fake, fake, ws, null) == 2   # 32 % 5
    assert g(fake, 1, 32, 1027, 1027, 32, fake, 1.5, null, null, null, fake, fake, fake, ws, null) == 4  # row not 16B
    assert g(fake, 1, 32, 1024, 1024, 32, fake, 1.5, null, null, null, fake, fake, fake, 8, null) == 5
    assert g(fake, 1, 32, 1 << 20, 1 << 20, 32, fake, 1.5, null, null, null, fake, fake, fake, ws, null) == 6
    assert g(fake, 1, 32, 1024, 1024, 32, fake, float("nan"), null, null, null, fake, fake, fake, ws, null) == 2
    assert g(fake, 1, 0, 1024, 1024, 32, fake, 1.5, null, null, null, fake, fake, fake, ws, null) == 0


def test_binding_refuses_host_tensors():
    import torch
    import paper_2603_18489_b200 as ec

    d = ec.make_desc(1, 8, 1, 1, 64, ec.EC_F32)
    x = torch.zeros(1, 8, 1, 64)
    with pytest.raises(ValueError):
        ec.ec_kv_refresh(d, x, x, x, x, None)


def test_descriptor_flags_are_validated_and_mirror_the_header():
    """ec_attn_desc.flags: the one defined bit is accepted, unknown bits make every entry point that takes the
    descriptor refuse it (host side, nothing launched); the Python mirror has the C struct's size."""
    import paper_2603_18489_b200 as ec

    text = open(os.path.join(HEADER_DIR, "entropycache.h")).read()
    assert re.search(r"#define\s+EC_ATTN_CACHE_SETTLED\s+1u", text) and ec.EC_ATTN_CACHE_SETTLED == 1
    assert ctypes.sizeof(ec.ec_attn_desc) == 32     # seven 4-byte fields and the flags word
    ok = ec.make_desc(1, 768, 32, 32, 128, ec.EC_BF16, flags=ec.EC_ATTN_CACHE_SETTLED)
    bad = ec.make_desc(1, 768, 32, 32, 128, ec.EC_BF16, flags=2)
    assert ec.ec_attend_workspace_bytes(ok, 34) > 0 and ec.ec_attend_kernel_name(ok, 34) != ""
    assert ec.ec_attend_workspace_bytes(bad, 34) == 0 and ec.ec_attend_kernel_name(bad, 34) == ""
    st = ec.lib.ec_attend(ctypes.byref(bad), None, None, None, None, None, None, 34, None, None, 0, None, None)
    assert st == 6                                  # EC_ERR_UNSUPPORTED, before any pointer is looked at
