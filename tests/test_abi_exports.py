"""The C-ABI library loads and exports every entry point that include/mop_moe.h declares (no
compute calls: this runs without a GPU), and the host-side argument checks answer with codes."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__
    __graft_entry__.build()
    from paper_2607_01844_b200 import binding
    return binding.lib()


def declared_symbols():
    text = (ROOT / "include" / "mop_moe.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mop_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"mop_moe_route", "mop_moe_permute", "mop_moe_expert_ffn_fwd", "mop_moe_expert_ffn_bwd",
            "mop_moe_combine", "mop_create", "mop_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in mop_moe.h but not exported"


def test_shape_struct_matches_header():
    from paper_2607_01844_b200 import binding
    text = (ROOT / "include" / "mop_moe.h").read_text()
    body = re.search(r"typedef struct \{(.*?)\} mop_moe_shape;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = [f.strip() for decl in re.findall(r"int32_t([^;]*);", body) for f in decl.split(",")]
    assert fields == [n for n, _ in binding.MopShape._fields_]


def test_argument_checks_need_no_device(lib):
    from paper_2607_01844_b200.binding import MopShape
    ok = MopShape(256, 256, 8, 2, 512, 0, 0, 0, 0, 0, 0)
    assert lib.mop_workspace_bytes(ctypes.byref(ok)) > 0
    for bad in (MopShape(256, 256, 8, 9, 512, 0, 0, 0, 0, 0, 0),     # k > E
                MopShape(256, 252, 8, 2, 512, 0, 0, 0, 0, 0, 0),     # d not a multiple of 8
                MopShape(256, 256, 8, 2, 512, 0, 1, 0, 0, 0, 0),     # post-score bias with softmax
                MopShape(256, 256, 8, 2, 512, 3, 0, 0, 0, 0, 0)):    # bad enum
        assert lib.mop_workspace_bytes(ctypes.byref(bad)) == 0
    assert lib.mop_status_string(7) == b"device-side wait ran out"
    assert lib.mop_moe_combine(None, None, None, None, None) == 1
    assert lib.mop_launch_count(None) == 0
