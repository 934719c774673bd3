"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the header
declares, sizes workspaces, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2601_13143_b200 import build as fbuild
from paper_2601_13143_b200 import fastav

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fbuild.build()
    return fastav.library()


def _params(**over):
    base = dict(batch=2, total_tokens=300, max_seqlen=200, total_q=8, max_qlen=4, total_keep=150, max_keep=100,
                num_q_heads=8, num_kv_heads=2, head_dim=64, hidden=512, softmax_scale=0.0, flags=3)
    base.update(over)
    return fastav.make_params(**base)


def test_header_symbols_are_exported(lib):
    with open(os.path.join(ROOT, "include", "fastav.h")) as f:
        header = f.read()
    declared = set(re.findall(r"\b(fastav_[a-z_]+)\s*\(", header))
    assert declared == set(fastav.EXPORTS), declared ^ set(fastav.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.fastav_version() == int(re.search(r"#define FASTAV_VERSION (\d+)", header).group(1))


def test_params_struct_layout_matches_header():
    # 11 int32, padding to 8, 10 int64, float, uint32
    assert ctypes.sizeof(fastav.fastav_params) == 136
    assert fastav.fastav_params.q_stride_tok.offset == 48
    assert fastav.fastav_params.softmax_scale.offset == 128


def test_status_strings(lib):
    for code in (0, -1, -2, -3, -4, -5):
        assert fastav.fastav_status_string(code) not in ("", "unknown status")
    assert fastav.fastav_status_string(-99) == "unknown status"


def test_workspace_size_grows_with_shapes(lib):
    small = fastav.fastav_workspace_bytes(_params())
    big = fastav.fastav_workspace_bytes(_params(total_tokens=3000, max_seqlen=2000, total_keep=1500, max_keep=1000))
    assert 0 < small < big and small % 256 == 0 and big % 256 == 0


@pytest.mark.parametrize("over,status", [
    (dict(batch=0), fastav.FASTAV_ERR_INVALID_ARG),
    (dict(num_q_heads=7), fastav.FASTAV_ERR_INVALID_ARG),
    (dict(total_keep=301), fastav.FASTAV_ERR_INVALID_ARG),
    (dict(max_seqlen=301), fastav.FASTAV_ERR_INVALID_ARG),
    (dict(head_dim=96), fastav.FASTAV_ERR_UNSUPPORTED),
    (dict(hidden=508), fastav.FASTAV_ERR_UNSUPPORTED),
])
def test_bad_shapes_are_rejected(lib, over, status):
    with pytest.raises(fastav.FastavError) as e:
        fastav.fastav_workspace_bytes(_params(**over))
    assert e.value.status == status


def test_null_and_workspace_errors_enqueue_nothing(lib):
    p = _params()
    null = ctypes.c_void_p(None)
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: validation fails first
    rc = lib.fastav_score(ctypes.byref(p), null, fake, fake, fake, fake, null, fake, fake, ctypes.c_size_t(1 << 30), null, null)
    assert rc == fastav.FASTAV_ERR_INVALID_ARG            # q missing
    rc = lib.fastav_score(ctypes.byref(p), fake, fake, fake, fake, fake, null, fake, fake, ctypes.c_size_t(16), null, null)
    assert rc == fastav.FASTAV_ERR_WORKSPACE              # too small
    rc = lib.fastav_score(ctypes.byref(p), fake, fake, fake, fake, fake, null, fake, ctypes.c_void_p(0x1010), ctypes.c_size_t(1 << 30), null, null)
    assert rc == fastav.FASTAV_ERR_WORKSPACE              # not 256-byte aligned
    rc = lib.fastav_score(ctypes.byref(p), ctypes.c_void_p(0x1008), fake, fake, fake, fake, null, fake, fake, ctypes.c_size_t(1 << 30), null, null)
    assert rc == fastav.FASTAV_ERR_UNSUPPORTED            # q not 16-byte aligned
    p_bad = _params()
    p_bad.k_stride_head = 60                               # shorter than a row
    rc = lib.fastav_score(ctypes.byref(p_bad), fake, fake, fake, fake, fake, null, fake, fake, ctypes.c_size_t(1 << 30), null, null)
    assert rc == fastav.FASTAV_ERR_INVALID_ARG
    p_bad.k_stride_head = 68                               # rows no longer 16-byte aligned
    rc = lib.fastav_score(ctypes.byref(p_bad), fake, fake, fake, fake, fake, null, fake, fake, ctypes.c_size_t(1 << 30), null, null)
    assert rc == fastav.FASTAV_ERR_UNSUPPORTED


def test_compact_rejects_unpaired_and_overlapping_buffers(lib):
    p = _params()
    null = ctypes.c_void_p(None)
    fake = ctypes.c_void_p(0x100000)
    far = ctypes.c_void_p(0x40000000)
    rc = lib.fastav_compact(ctypes.byref(p), fake, fake, fake, fake, null, null, null, null, null, null, null, null, null)
    assert rc == fastav.FASTAV_ERR_INVALID_ARG            # hidden_in without hidden_out
    rc = lib.fastav_compact(ctypes.byref(p), fake, fake, fake, fake, ctypes.c_void_p(0x100000 + 512), null, null, null, null, null, null, null, null)
    assert rc == fastav.FASTAV_ERR_INVALID_ARG            # output inside the input
    rc = lib.fastav_compact(ctypes.byref(p), null, fake, fake, fake, far, null, null, null, null, null, null, null, null)
    assert rc == fastav.FASTAV_ERR_INVALID_ARG            # keep_idx missing


def test_missing_library_is_a_loud_error(monkeypatch, tmp_path):
    monkeypatch.setenv("FASTAV_LIBRARY", str(tmp_path / "nope.so"))
    monkeypatch.setattr(fastav, "_lib", None)
    with pytest.raises(OSError):
        fastav.library()
