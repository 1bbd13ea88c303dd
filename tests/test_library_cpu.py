"""Host-side checks that need no GPU: the C-ABI library builds, loads and exports what fc.h declares."""
import ctypes as C

import pytest

import paper_2602_10825_b200 as fc
from paper_2602_10825_b200 import build as fc_build


@pytest.fixture(scope="module")
def built():
    fc_build.build()
    return fc.lib()


def test_every_declared_symbol_is_exported(built):
    declared = fc.declared_symbols()
    for must in ("fc_create", "fc_destroy", "fc_chunk_decide", "fc_chunk_attention", "fc_kv_score",
                 "fc_kv_select_compact", "fc_chunk_decide_workspace_bytes", "fc_chunk_attention_workspace_bytes",
                 "fc_kv_score_workspace_bytes", "fc_kv_select_compact_workspace_bytes", "fc_status_string",
                 "fc_last_cuda_error", "fc_sm_count"):
        assert must in declared
    assert fc.exported_symbols() == declared


def test_status_strings_and_host_only_queries(built):
    assert built.fc_status_string(0) == b"ok"
    assert b"workspace" in built.fc_status_string(-4)
    assert built.fc_chunk_decide_workspace_bytes(C.c_int64(1 << 20), 4) >= 16 * ((1 << 20) // 4096)
    assert built.fc_kv_select_compact_workspace_bytes(8, 1000) > 0
    # a NULL descriptor is rejected by the size query, not dereferenced
    assert built.fc_kv_score_workspace_bytes(None) == 0


def test_create_without_a_device_fails_cleanly(built):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(fc.FcError):
        fc.Context(0)
