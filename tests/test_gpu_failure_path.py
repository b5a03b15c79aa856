"""A device-side failure path, exercised without faulting anything.

The tensor-core filtering kernel waits on mbarriers with a poll limit; a wait that runs out raises
the status flag, the warp roles leave their loops, the tensor memory is released and the kernel
returns.  The test-only option IVFPQ_OPT_TEST_FAULT makes one producer leave out its last tile
load (nothing is issued, so nothing is left in flight) and shortens the limit: the wait for that
tile runs out.  Checked here: the search call itself still returns, ivfpq_sync_status reports
IVFPQ_ERR_DEVICE_FLAG, the context stays usable, and with the option off again the same handle
gives the oracle's answers."""

import numpy as np
import pytest
import torch

import oracle
import paper_2312_01712_b200 as lib
from parity import assert_topk_parity

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_and_the_handle_recovers(wl_small):
    wl = wl_small
    h = lib.ivfpq_index_load(wl.index)
    try:
        q = torch.from_numpy(wl.queries).cuda()
        o = oracle.search(wl.index, wl.queries, 5, 20, dense=True)
        d, i = lib.ivfpq_search_dense(h, q, 5, 20)
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        assert_topk_parity(d.cpu().numpy(), i.cpu().numpy(), o["dist"], o["ids"])

        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_TEST_FAULT, 1)
        lib.ivfpq_search_dense(h, q, 5, 20)            # returns: the kernels give up and finish
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_ERR_DEVICE_FLAG
        assert "flag" in lib.error_string(lib.IVFPQ_ERR_DEVICE_FLAG)
        lib.ivfpq_search_dense(h, q, 5, 20)            # the flag is raised again, every time
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_ERR_DEVICE_FLAG

        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_TEST_FAULT, 0)
        torch.cuda.synchronize()                        # the context is intact
        for _ in range(2):                              # tensor memory was released: the kernel can allocate it again
            d, i = lib.ivfpq_search_dense(h, q, 5, 20)
            assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
            assert_topk_parity(d.cpu().numpy(), i.cpu().numpy(), o["dist"], o["ids"])
    finally:
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_TEST_FAULT, 0)
        lib.ivfpq_index_free(h)


def test_fault_option_is_refused_where_it_has_no_effect():
    from ivfpq_inputs import lossless_toy_index
    idx, _ = lossless_toy_index(seed=3, n=200, nlist=8, nsub=3, dsub=3, ksub=16)    # d = 9: not served by the tensor-core kernel
    h = lib.ivfpq_index_load(idx)
    try:
        with pytest.raises(lib.IvfpqError) as e:
            lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_TEST_FAULT, 1)
        assert e.value.code == lib.IVFPQ_ERR_UNSUPPORTED
    finally:
        lib.ivfpq_index_free(h)
