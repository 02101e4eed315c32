"""The C-ABI library: it loads, exports every symbol include/toktier.h declares, rejects malformed
vocabularies on the host, and its class table equals the oracle's on all 1,114,112 code points."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tt():
    from paper_2607_29678_b200 import build
    build.build()
    import paper_2607_29678_b200 as m
    return m


def test_exports_every_declared_symbol(tt):
    header = open(os.path.join(ROOT, "include", "toktier.h")).read()
    declared = set(re.findall(r"\b(tt_[a-z_]+)\s*\(", header))
    assert declared == set(tt.EXPORTS), declared ^ set(tt.EXPORTS)
    lib = ctypes.CDLL(tt.LIB_PATH)
    for name in declared:
        assert getattr(lib, name) is not None


def test_strerror(tt):
    assert tt.strerror(0) == "ok"
    assert "UTF-8" in tt.strerror(tt.TT_ERR_INVALID_UTF8)


def test_class_table_equals_oracle_everywhere(tt):
    gpu = tt.class_table()
    # kernel codes: 0 other, 1 mark, 2 whitespace, 3 number, 4 lower, 5 upper/title, 6 caseless
    to_oracle = np.array([oracle.K_O, oracle.K_M, oracle.K_W, oracle.K_N, oracle.K_LL, oracle.K_LU, oracle.K_LB], dtype=np.uint8)
    assert gpu.max() <= 6
    assert np.array_equal(to_oracle[gpu], oracle.class_table())


def test_vocab_validation_without_a_device(tt):
    """Malformed merge tables are rejected before any CUDA call is made."""
    ok_map = np.arange(256, dtype=np.int32)

    def load(merges, byte_map=ok_map, pattern=0):
        h = ctypes.c_void_p()
        m = np.ascontiguousarray(merges, dtype=np.int32).reshape(-1, 3)
        return tt.lib().tt_vocab_load(m.ctypes.data, m.shape[0], byte_map.ctypes.data, pattern, ctypes.byref(h))

    assert load([[97, 98, 256], [97, 98, 257]]) == tt.TT_ERR_BAD_VOCAB          # duplicate pair
    assert load([[97, 300, 256]]) == tt.TT_ERR_BAD_VOCAB                        # forward reference
    assert load([[97, 98, 97]]) == tt.TT_ERR_BAD_VOCAB                          # result collides with a base id
    assert load([[97, 98, 256], [256, 99, 256]]) == tt.TT_ERR_BAD_VOCAB         # result reused
    assert load([[97, 98, -5]]) == tt.TT_ERR_BAD_VOCAB
    dup_map = ok_map.copy(); dup_map[5] = 6
    assert load([[97, 98, 256]], byte_map=dup_map) == tt.TT_ERR_BAD_VOCAB       # byte map not injective
    assert load([[97, 98, 256]], pattern=7) == tt.TT_ERR_ARG
    # a well-formed table passes validation; without a device the upload then fails with TT_ERR_CUDA
    assert load([[97, 98, 256]]) in (tt.TT_OK, tt.TT_ERR_CUDA)
