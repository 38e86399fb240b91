"""Host-only checks of the C-ABI library: it loads without a GPU, exports every symbol the
header declares, and its pure-host entry points behave."""
import ctypes as C
import os
import re

import pytest

from paper_2609_33184_b200 import binding as ssb
from paper_2609_33184_b200 import build as ssbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ssbuild.build()
    return ssb.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "specstream.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ss_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"ss_verify_begin", "ss_verify_chunk", "ss_verify_local", "ss_verify_finalize",
            "ss_commit_gather", "ss_stream_round"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(ssb.EXPORTS) == names


def test_struct_layout_matches(lib):
    assert lib.ss_sizeof_stream_desc() == C.sizeof(ssb.ss_stream_desc)


def test_workspace_bytes_and_config_validation(lib):
    cfg = ssb.ss_config(16, 32, 8, 128, 8, 8, 2048, 0, 0, 0)
    n = lib.ss_workspace_bytes(C.byref(cfg))
    assert n > 0 and n % 256 == 0
    bigger = ssb.ss_config(16, 32, 8, 128, 16, 8, 2048, 0, 0, 0)
    assert lib.ss_workspace_bytes(C.byref(bigger)) > n
    for bad in (ssb.ss_config(16, 30, 8, 128, 8, 8, 2048, 0, 0, 0),     # H_q % H_kv
                ssb.ss_config(16, 32, 8, 96, 8, 8, 2048, 0, 0, 0),      # head dim
                ssb.ss_config(0, 32, 8, 128, 8, 8, 2048, 0, 0, 0),
                ssb.ss_config(16, 32, 8, 128, 8, 8, 2048, 1000, 0, 0)):
        assert lib.ss_workspace_bytes(C.byref(bad)) == 0


def test_strerror(lib):
    seen = {lib.ss_strerror(i).decode() for i in range(10)}
    assert len(seen) == 10 and "ok" in seen


def test_null_arguments_are_rejected_without_a_device(lib):
    assert lib.ss_create(None, None, None, 0) == ssb.SS_ERR_ARG
    assert lib.ss_destroy(None) == ssb.SS_ERR_ARG
    t = ssb.ss_tensor(None, 0, 0, 0)
    assert lib.ss_verify_begin(None, t, 1, 1, 1.0, None) == ssb.SS_ERR_ARG
    assert lib.ss_verify_chunk(None, t, t, 1, None, None) == ssb.SS_ERR_ARG
    assert lib.ss_verify_finalize(None, None, None, None) == ssb.SS_ERR_ARG
    assert lib.ss_verify_abort(None) == ssb.SS_ERR_ARG
    assert lib.ss_stream_round(None, None, None) == ssb.SS_ERR_ARG
