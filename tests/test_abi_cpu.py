"""Host-side checks of the C ABI that need no GPU: the library builds, loads,
exports every symbol the header declares, and rejects bad problem statements
before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2402_04902_b200 import binding as l4q
from paper_2402_04902_b200 import build as l4q_build
from paper_2402_04902_b200.synth import CONFIG1, CONFIG2

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    l4q_build.build()
    return l4q.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "l4q.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(l4q_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found in include/l4q.h"
    assert declared == set(l4q.EXPORTED_SYMBOLS)
    for name in declared:
        assert hasattr(lib, name), name


def test_desc_struct_layout_matches_header():
    # int64 x3, int32, float, int32 x3, uint32, float -> 56 bytes, 8-byte aligned
    assert ctypes.sizeof(l4q.L4QDesc) == 56
    assert l4q.L4QDesc.rank.offset == 24 and l4q.L4QDesc.grad_scale.offset == 48


def test_status_strings(lib):
    assert l4q.status_string(0) == "ok"
    assert "timed out" in l4q.status_string(5)
    assert l4q.status_string(99) == "unknown status"


def test_workspace_query_and_rejections(lib):
    d = l4q.make_desc(CONFIG2)
    assert l4q.l4q_workspace_bytes(d, l4q.L4Q_OP_FWD) >= CONFIG2.d_in * CONFIG2.d_out * 2
    # optional scratch of the export: one split-operand block of 16 KiB per 128-wide panel of A and of B at rank 16
    assert l4q.l4q_workspace_bytes(d, l4q.L4Q_OP_PACK) == (CONFIG2.d_in // 128 + CONFIG2.d_out // 128) * 16384
    assert l4q.l4q_workspace_bytes(l4q.make_desc(CONFIG2.with_(io_dtype="f32")), l4q.L4Q_OP_PACK) == 0
    bad = l4q.make_desc(CONFIG2.with_(group_size=100))        # d_in % group_size != 0
    assert l4q.l4q_workspace_bytes(bad, l4q.L4Q_OP_FWD) == 0


@pytest.mark.parametrize("mutation,expected", [
    (dict(tokens=0), 1), (dict(rank=0), 1), (dict(group_size=96), 2), (dict(bits=9), 2), (dict(bits=1), 2),
    (dict(group_size=4, d_in=256), 2),
    (dict(rank=129), 2), (dict(rank=256), 2),       # above L4Q_MAX_RANK
])
def test_bad_desc_is_an_error_code_not_a_crash(lib, mutation, expected):
    d = l4q.make_desc(CONFIG1.with_(**mutation))
    st = lib.l4q_linear_fwd(ctypes.byref(d), None, None, None, None, None, None, None, None, 0, None)
    assert st == expected


@pytest.mark.parametrize("rank", [64, 128])
def test_ranks_up_to_the_limit_get_a_workspace_size(lib, rank):
    """Ranks the header admits pass the descriptor check in both modes (the plain-ALU weight-tile kernel serves ranks
    above 64; its shared-memory need of rank x 320 floats fits at the limit), and the first rank above it does not."""
    for dt in ("bf16", "f32"):
        d = l4q.make_desc(CONFIG1.with_(rank=rank, io_dtype=dt))
        assert l4q.l4q_workspace_bytes(d, l4q.L4Q_OP_FWD) > 0
        assert l4q.l4q_workspace_bytes(d, l4q.L4Q_OP_BWD) >= l4q.l4q_workspace_bytes(d, l4q.L4Q_OP_FWD)
    assert l4q.L4Q_MAX_RANK == 128 and l4q.L4Q_MAX_RANK * 320 * 4 <= 227 * 1024
    d = l4q.make_desc(CONFIG1.with_(rank=l4q.L4Q_MAX_RANK + 1))
    assert l4q.l4q_workspace_bytes(d, l4q.L4Q_OP_FWD) == 0


def test_null_pointers_rejected_before_any_launch(lib):
    d = l4q.make_desc(CONFIG1)
    n0 = l4q.l4q_launch_count()
    assert lib.l4q_linear_fwd(ctypes.byref(d), None, None, None, None, None, None, None, None, 0, None) == 1
    assert lib.l4q_linear_bwd(ctypes.byref(d), *([None] * 12), None, 0, None) == 1
    assert lib.l4q_pack_int(ctypes.byref(d), *([None] * 8), None, 0, None) == 1
    assert lib.l4q_linear_fwd(None, *([None] * 7), None, 0, None) == 1
    assert l4q.l4q_launch_count() == n0
