"""Host-side checks that need no GPU: the shared library loads, exports every symbol the
header declares, and validates arguments before touching CUDA."""

import ctypes
import os
import re

import numpy as np
import pytest

import paper_2312_01712_b200 as lib
from paper_2312_01712_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    libbuild.build()
    return lib.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ivfpq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ivfpq_[a-z_]+)\s*\(", text)))


def test_header_and_binding_agree_on_exports(L):
    names = declared_functions()
    assert len(names) >= 12
    assert sorted(lib.EXPORTS) == names
    for n in names:
        assert hasattr(L, n), f"{n} is declared in ivfpq.h but not exported"
        assert callable(getattr(lib, n, None)) or n in ("ivfpq_index_derived_bytes", "ivfpq_error_string",
                                                        "ivfpq_search_host_workspace_bytes"), n


def test_error_strings(L):
    seen = set()
    for code in (0, -1, -2, -3, -4, -5):
        s = L.ivfpq_error_string(code).decode()
        assert s and s not in seen
        seen.add(s)
    assert "unknown" in L.ivfpq_error_string(-99).decode()


def make_desc(**kw):
    off = np.array(kw.pop("offsets", [0, 40, 40, 100]), np.int64)
    base = dict(d=8, nlist=len(off) - 1, nsub=4, dsub=2, ksub=256, metric=0, ntotal=int(off[-1]))
    base.update(kw)
    desc = lib.ivfpq_index_desc_t(base["d"], base["nlist"], base["nsub"], base["dsub"], base["ksub"],
                                  base["metric"], base["ntotal"], 0, 0, off.ctypes.data, 0, 0)
    desc._keep = off
    return desc


def test_derived_bytes_and_description_validation(L):
    good = make_desc()
    n = L.ivfpq_index_derived_bytes(ctypes.byref(good))
    # 2 + 0 + 2 blocks of 32 points x 1 word x 4 bytes, plus two list tables, 256-byte granules
    assert n >= 4 * 32 * 4 + 2 * 4 * 8 and n % 256 == 0
    assert L.ivfpq_index_derived_bytes(None) == 0
    for bad in (dict(d=9), dict(ksub=257), dict(nsub=0), dict(metric=2), dict(ntotal=99),
                dict(offsets=[0, 50, 40, 100]), dict(offsets=[1, 40, 100]), dict(nsub=65, dsub=1, d=65),
                dict(nsub=1, dsub=17, d=17)):
        assert L.ivfpq_index_derived_bytes(ctypes.byref(make_desc(**bad))) == 0, bad


def test_load_rejects_bad_arguments_before_any_cuda_call(L):
    out = ctypes.c_void_p()
    good = make_desc()
    assert L.ivfpq_index_load(ctypes.byref(good), None, 0, None, None) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_index_load(None, None, 0, None, ctypes.byref(out)) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    # null device arrays
    assert L.ivfpq_index_load(ctypes.byref(good), None, 0, None, ctypes.byref(out)) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_index_load(ctypes.byref(make_desc(ksub=300)), None, 0, None, ctypes.byref(out)) == \
        lib.IVFPQ_ERR_UNSUPPORTED
    assert out.value is None
    assert L.ivfpq_index_free(None) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_search_workspace_bytes(None, 10, 1, 1) == 0
    assert L.ivfpq_search_dense(None, None, 1, 1, 1, None, None, None, 0, None) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_search_sparse(None, None, 1, 1, None, 1, None, None, None, 0, None) == \
        lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_sync_status(None, None, None) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_index_set_option(None, lib.IVFPQ_OPT_NSPLIT, 1) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_last_launch_count(None) == 0
    assert L.ivfpq_probe_static(None, None, 1, 1, None, None, None) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_query_thresholds(None, None, 1, None, None, None) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_query_thresholds_knn(None, None, 1, 1, 1, None, None, None, 0, None) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_static_status is not None
    assert L.ivfpq_entry_stats(None, None, None, 1, None, 1, None, None, None, None) == lib.IVFPQ_ERR_INVALID_ARGUMENT


def test_binding_refuses_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    from test_oracle_pins import hand_index
    with pytest.raises(RuntimeError, match="no CUDA device"):
        lib.ivfpq_index_load(hand_index())


def test_index_file_roundtrip(tmp_path, wl_small):
    from ivfpq_inputs import load_index, save_index
    p = str(tmp_path / "idx.bin")
    save_index(wl_small.index, p)
    back = load_index(p)
    for f in ("coarse_centroids", "codebooks", "list_offsets", "codes", "ids"):
        assert np.array_equal(getattr(back, f), getattr(wl_small.index, f))
    assert (back.d, back.nlist, back.nsub, back.dsub, back.ksub, back.ntotal) == \
        (wl_small.index.d, wl_small.index.nlist, wl_small.index.nsub, wl_small.index.dsub,
         wl_small.index.ksub, wl_small.index.ntotal)
    raw = open(p, "rb").read()
    open(p, "wb").write(raw[:-5])
    with pytest.raises(ValueError):
        load_index(p)
    open(p, "wb").write(b"\0" * 4 + raw[4:])
    with pytest.raises(ValueError):
        load_index(p)
