"""CPU checks of the boundary: the C-ABI library builds/loads and exports every symbol include/l2a.h
declares; host-only entry points behave (no GPU work is launched here)."""
import ctypes
import os
import re

import pytest

from paper_2603_17484_b200 import build as l2a_build
from paper_2603_17484_b200 import l2a

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    l2a_build.build_lib()
    return l2a.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "l2a.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(l2a_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"l2a_route_compact", "l2a_forward", "l2a_backward"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/l2a.h but not exported"
    assert set(names) == set(l2a.EXPORTS)


def test_version_and_status_strings(lib):
    assert "sm_100a" in l2a.version()
    assert l2a.status_string(0) == "ok"
    for code in (-1, -2, -3, -4, -5):
        assert l2a.status_string(code) not in ("ok", "unknown status")


def test_workspace_sizes_and_validation(lib):
    p = l2a.params(1, 131072, 131072, 32, 8, 128, 4096)
    r, f, b = l2a.l2a_workspace_bytes(p)
    assert r >= 256 and r % 256 == 0
    assert f >= 131072 * 32 * 128 * 2            # room for the compact query buffer, worst case
    assert b >= 256
    bad = l2a.params(1, 128, 64, 2, 1, 128, 4)   # Lq + offset > Lk with offset forced to 0
    bad.q_pos_offset = 0
    with pytest.raises(l2a.L2AError):
        l2a.l2a_workspace_bytes(bad)
    with pytest.raises(l2a.L2AError):
        l2a.l2a_workspace_bytes(l2a.params(1, 128, 128, 3, 2, 128, 4))
    with pytest.raises(l2a.L2AError) as e:
        l2a.l2a_workspace_bytes(l2a.params(1, 128, 128, 2, 1, 80, 4))
    assert e.value.code == -2


def test_params_struct_layout_matches_header():
    # ten 32-bit fields, four {batch, token} stride pairs of 64-bit integers, the packed-sequence table pointer
    assert ctypes.sizeof(l2a.L2AParams) == 40 + 4 * 2 * 8 + 8
    assert l2a.L2AParams.q_stride.offset == 40 and l2a.L2AParams.o_stride.offset == 88
    assert l2a.L2AParams.seq_bounds.offset == 104


def test_stride_arguments_are_validated_on_the_host():
    ok = dict(B=2, Lq=256, Lk=256, Hq=4, Hkv=2, D=128, window=16)
    row = 4 * 128
    l2a.l2a_workspace_bytes(l2a.params(**ok, q_stride=(256 * 2 * row, 2 * row)))          # a slice of a wider buffer
    for bad in ((0, row + 4),            # not a multiple of 8 elements
                (0, row - 8),            # rows overlap
                (255 * row, row),        # batches overlap
                (-8, row)):
        with pytest.raises(l2a.L2AError) as e:
            l2a.l2a_workspace_bytes(l2a.params(**ok, q_stride=bad))
        assert e.value.code == -1


def test_flag_and_router_constants_match_the_header():
    """The binding's constants are the header's #defines (same names without the L2A_ prefix)."""
    text = open(os.path.join(ROOT, "include", "l2a.h")).read()
    defines = {m.group(1): int(m.group(2)) for m in re.finditer(r"#define\s+L2A_((?:FLAG|ROUTER)_[A-Z0-9_]+)\s+(\d+)u?", text)}
    assert len([k for k in defines if k.startswith("FLAG_")]) >= 6 and "ROUTER_MASK_U8" in defines
    for name, value in defines.items():
        assert getattr(l2a, name) == value, name
    flags = [v for k, v in defines.items() if k.startswith("FLAG_")]
    assert len(set(flags)) == len(flags) and all(v & (v - 1) == 0 for v in flags)   # distinct single bits


def test_packed_sequence_table_is_validated_on_the_host():
    """l2a_params.seq_bounds needs one token axis (B = 1), Lq = Lk, no position offset and an 8-byte aligned table;
    the check runs before anything is launched (the pointer is never dereferenced on the host)."""
    class Fake:                      # stands in for a device tensor: only its address is marshalled
        def __init__(self, addr): self.addr = addr
        def data_ptr(self): return self.addr
    ok = dict(B=1, Lq=512, Lk=512, Hq=4, Hkv=2, D=128, window=16)
    l2a.l2a_workspace_bytes(l2a.params(**ok, seq_bounds=Fake(0x10000)))
    for bad in (dict(ok, B=2), dict(ok, Lk=1024), dict(ok, Lk=1024, q_pos_offset=0)):
        with pytest.raises(l2a.L2AError) as e:
            l2a.l2a_workspace_bytes(l2a.params(**bad, seq_bounds=Fake(0x10000)))
        assert e.value.code == -1
    with pytest.raises(l2a.L2AError):
        l2a.l2a_workspace_bytes(l2a.params(**ok, seq_bounds=Fake(0x10004)))
