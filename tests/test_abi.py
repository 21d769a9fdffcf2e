"""Boundary checks that need no GPU: the shared library loads, exports every symbol the header
declares, sizes workspaces sensibly and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

import paper_2506_22694_b200 as vt
from paper_2506_22694_b200 import build as vt_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    vt_build.build()
    return vt.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "vocabtrim.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"#ifdef VT_STAMPS.*?#endif", "", text, flags=re.S)       # instrumented builds only
    return sorted(set(re.findall(r"\b(vt_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = _declared_symbols()
    assert set(vt.EXPORTS) <= set(names)
    assert {"vt_build_vocab", "vt_trim_head", "vt_draft_head", "vt_histogram", "vt_select_topk"} <= set(names)
    for n in names:
        assert hasattr(lib, n), "missing export " + n


def test_status_strings(lib):
    assert vt.status_str(0) == "ok"
    assert "workspace" in vt.status_str(3)
    assert vt.status_str(99) == "unknown status"


def test_workspace_bytes(lib):
    V = 128256
    hist = vt.workspace_bytes(vt.VT_OP_HISTOGRAM, 10**9, V)
    sel = vt.workspace_bytes(vt.VT_OP_SELECT_TOPK, 0, V, 32768)
    both = vt.workspace_bytes(vt.VT_OP_BUILD_VOCAB, 10**9, V, 32768)
    assert hist >= 256 + 4 * V and sel >= 256 + 16 * V
    assert both >= 256 + 4 * V + max(hist, sel) - 256
    assert vt.workspace_bytes(vt.VT_OP_HISTOGRAM, 100, 4096) == 256          # bins fit in shared memory
    assert vt.workspace_bytes(vt.VT_OP_SELECT_TOPK, 0, 100, 101) == 0         # K > V
    assert vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, 32768, 4096, 10, 10) > 256
    assert vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, 32768, 4097, 10, 10) == 0   # d % 8 != 0
    assert vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, 32768, 4096, 10, 65) == 0   # topk > 64
    assert vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, 4, 64, 1, 5) == 0           # topk > K
    host = vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD_HOST, 0, 0, 32768, 4096, 10, 10)
    assert host >= vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, 32768, 4096, 10, 10) + 10 * 32768 * 4
    assert vt.workspace_bytes(12345) == 0
    # largest vocabulary the histogram takes: its lookup table (8 bytes per 32 ids) may use 160 KB
    assert vt.workspace_bytes(vt.VT_OP_HISTOGRAM, 100, 655_360) > 256
    assert vt.workspace_bytes(vt.VT_OP_HISTOGRAM, 100, 655_361) == 0
    assert vt.workspace_bytes(vt.VT_OP_BUILD_VOCAB, 100, 655_361, 10) == 0


def test_argument_errors_return_before_any_cuda_call(lib):
    null = ctypes.c_void_p(0)
    fake = ctypes.c_void_p(0x1000)            # never dereferenced: the calls must fail first
    # null pointers / bad sizes -> VT_ERR_INVALID_ARG (1)
    assert lib.vt_histogram(null, 10, 100, fake, 0, fake, 1 << 20, null) == 1
    assert lib.vt_histogram(fake, -1, 100, fake, 0, fake, 1 << 20, null) == 1
    assert lib.vt_select_topk(fake, 100, 0, fake, fake, fake, 1 << 20, null) == 1
    assert lib.vt_select_topk(fake, 100, 101, fake, fake, fake, 1 << 20, null) == 1
    assert lib.vt_build_vocab(fake, 10, 100, 200, fake, fake, fake, 1 << 20, null) == 1
    assert lib.vt_trim_head(fake, fake, fake, 100, 10, 12, null, null) == 1           # d % 8
    assert lib.vt_trim_head(null, fake, fake, 100, 10, 16, null, null) == 1
    head = [fake, fake, null, 1, 1024, 256, fake, 4, null, fake, fake]
    assert lib.vt_draft_head(*head, null, 0, null) == 3                                # no workspace
    assert lib.vt_draft_head(*head, fake, 16, null) == 3                               # too small
    bad = list(head)
    bad[7] = 0                                                                         # topk = 0
    assert lib.vt_draft_head(*bad, fake, 1 << 20, null) == 1
    bad = list(head)
    bad[5] = 250                                                                       # d % 8
    assert lib.vt_draft_head(*bad, fake, 1 << 20, null) == 1
    # misaligned workspace -> VT_ERR_WORKSPACE
    assert lib.vt_histogram(fake, 10, 100, fake, 0, ctypes.c_void_p(0x1010), 1 << 20, null) == 3
    assert lib.vt_workspace_init(null, 1024, null) == 3


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(vt, "_lib", None)
    monkeypatch.setattr(vt, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libvocabtrim.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        vt.lib()


def test_mbsu_host_calculator_matches_a_table_cell_of_the_paper():
    """Table 1, independent drafter (314M parameters, block size 4, 3.21e9-parameter target):
    block efficiency 3.846 is printed with a memory-bound speed-up of 2.765."""
    import math
    import paper_2506_22694_b200 as vt
    assert abs(vt.vt_mbsu(3.846, 314.0e6, 3212.7e6, 4) - 2.765) < 2.5e-3
    assert vt.vt_mbsu(5.0, 0.0, 1.0, 4) == 5.0
    assert math.isnan(vt.vt_mbsu(1.0, 1.0, 0.0, 4)) and math.isnan(vt.vt_mbsu(-1.0, 1.0, 1.0, 4))
