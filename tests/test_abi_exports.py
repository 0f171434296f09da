"""The C-ABI library builds, loads and exports every function include/moehub.h declares; the host-side
argument checks answer without a GPU.  No compute call is made here."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2605_05888_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return B.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "moehub.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moe_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), f"{n} declared in moehub.h but not exported"
    assert sorted(B.EXPORTS) == names, "binding.EXPORTS and the header disagree"


def header_config_fields():
    """(name, ctypes type) of every field of moe_config_t, parsed from the header."""
    text = open(os.path.join(ROOT, "include", "moehub.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} moe_config_t;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    ctype = {"int32_t": ctypes.c_int32, "int64_t": ctypes.c_int64, "uint64_t": ctypes.c_uint64}
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if not decl:
            continue
        ty, names = decl.split(None, 1)
        for name in names.split(","):
            name = name.strip()
            m = re.fullmatch(r"(\w+)\[(\d+)\]", name)
            fields.append((m.group(1), ctype[ty] * int(m.group(2))) if m else (name, ctype[ty]))
    return fields


def test_config_struct_matches_header():
    """Same fields, same order, same types: the binding's ctypes structure mirrors the C struct."""
    want = header_config_fields()
    got = [(n, t) for n, t in B.MoeConfig._fields_]
    assert [n for n, _ in got] == [n for n, _ in want]
    for (n, t_got), (_, t_want) in zip(got, want):
        assert ctypes.sizeof(t_got) == ctypes.sizeof(t_want), n

    class Mirror(ctypes.Structure):
        _fields_ = want
    assert ctypes.sizeof(B.MoeConfig) == ctypes.sizeof(Mirror)
    for n, _ in want:
        assert getattr(B.MoeConfig, n).offset == getattr(Mirror, n).offset, n


def test_host_side_checks_without_gpu(lib):
    ok = B.make_config(4096, 4096, 8, 8, 2, 14336, B.DTYPE_BF16)
    assert B.moe_pool_tiles(ok) == 4096 * 2 // 128 + 8
    assert B.moe_workspace_bytes(ok) > 2 * 72 * 128 * 4096 * 2
    static = B.make_config(300, 128, 8, 2, 2, 64, B.DTYPE_BF16, dispatch_mode=B.DISPATCH_ATOMIC_STATIC)
    assert B.moe_pool_tiles(static) == 8 * 3            # capacity defaults to T rounded up to 128
    for bad, code in [(B.make_config(16, 100, 8, 2, 2, 64, B.DTYPE_BF16), -2),      # H*2 not multiple of 16
                      (B.make_config(16, 128, 8, 3, 2, 64, B.DTYPE_BF16), -1),      # E % R
                      (B.make_config(16, 128, 8, 2, 9, 64, B.DTYPE_BF16), -1),      # K > E
                      (B.make_config(16, 128, 512, 2, 2, 64, B.DTYPE_BF16), -3),    # E > 256
                      (B.make_config(16, 128, 8, 2, 2, 64, 7), -1)]:                # dtype
        with pytest.raises(B.MoeError) as ei:
            B.moe_workspace_bytes(bad)
        assert ei.value.code == code
    assert B.strerror(0) == "ok" and "overflow" in B.strerror(-5)
    h = ctypes.c_void_p()
    assert lib.moe_plan_create(ctypes.byref(ok), None, 0, ctypes.byref(h)) == -1   # null workspace
    assert lib.moe_route(None, None, None, None, None, None, None) == -1
