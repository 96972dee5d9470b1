"""Host-only checks of the C-ABI library: it builds, loads without a GPU, exports every
symbol the header declares, and validates arguments before touching any device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "hsa.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2609_34606_b200 import build
    return C.CDLL(build.build())


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hsa_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert {"hsa_create", "hsa_append_kv", "hsa_select_blocks", "hsa_forward", "hsa_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    from paper_2609_34606_b200 import hsa
    assert sorted(hsa.EXPORTS) == names
    for n in names:
        assert callable(getattr(hsa, n)), n


def test_query_sizes_and_config_validation():
    from paper_2609_34606_b200 import hsa
    cfg = hsa.hsa_config(12, 128, 64, 732, 4680, 64, 1, 0, 0.0, 0)
    s = hsa.hsa_query_sizes(cfg)
    assert s.k_pool == s.v_pool == 732 * 12 * 64 * 128 * 2
    assert s.state >= 12 * 128 * 128 * 4 * 2 + 12 * 732 * 128 * 4
    big = hsa.hsa_query_sizes(hsa.hsa_config(12, 128, 64, 732, 4680, 64, 1, 0, 0.0, hsa.HSA_CFG_CAUSAL))
    assert big.workspace >= s.workspace + 4680 * 12 * 128 * 4
    for bad in [dict(head_dim=96), dict(page_tokens=32), dict(num_heads=0), dict(max_pages=0),
                dict(lin_mode=2), dict(gate_act=3), dict(max_topk=0), dict(feature_map=2)]:
        kw = dict(num_heads=12, head_dim=128, page_tokens=64, max_pages=8, max_q_tokens=128, max_topk=4,
                  lin_mode=1, gate_act=0, softmax_scale=0.0, flags=0, lin_rank=0, lin_seg_tokens=0,
                  split_blocks=0, feature_map=0)
        kw.update(bad)
        with pytest.raises(hsa.HSAError) as e:
            hsa.hsa_query_sizes(hsa.hsa_config(*kw.values()))
        assert e.value.code == hsa.HSA_ERR_INVALID_ARG


def test_null_and_bad_arguments_rejected_on_host(lib):
    from paper_2609_34606_b200 import hsa
    assert hsa._lib.hsa_create(None, None, None, None) == hsa.HSA_ERR_INVALID_ARG
    h = C.c_void_p()
    cfg = hsa.hsa_config(2, 64, 64, 4, 128, 4, 1, 0, 0.0, 0)
    bufs = hsa.hsa_buffers(None, None, None, None)
    assert hsa._lib.hsa_create(C.byref(h), C.byref(cfg), C.byref(bufs), None) == hsa.HSA_ERR_INVALID_ARG
    # misaligned buffers and a page order that is not a permutation are rejected before any CUDA call
    bufs = hsa.hsa_buffers(0x1000 + 8, 0x2000, 0x3000, 0x4000)
    assert hsa._lib.hsa_create(C.byref(h), C.byref(cfg), C.byref(bufs), None) == hsa.HSA_ERR_INVALID_ARG
    bufs = hsa.hsa_buffers(0x1000, 0x2000, 0x3000, 0x4000)
    order = (C.c_int32 * 4)(0, 1, 1, 3)
    assert hsa._lib.hsa_create(C.byref(h), C.byref(cfg), C.byref(bufs), order) == hsa.HSA_ERR_INVALID_ARG
    assert h.value is None
    assert hsa._lib.hsa_append_kv(None, None, None, 1, 8, 8, None) == hsa.HSA_ERR_INVALID_ARG
    assert hsa._lib.hsa_destroy(None) == hsa.HSA_ERR_INVALID_ARG
    assert hsa.hsa_status_string(0) == "ok"
    assert "unsupported" in hsa.hsa_status_string(hsa.HSA_ERR_UNSUPPORTED)


def test_product_does_not_import_oracle():
    pkg = os.path.join(ROOT, "paper_2609_34606_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|oracle/|hsa_oracle", src, re.M), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            src = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2609_34606_b200" not in src and "libhsa" not in src, f
