"""The workspace-free filtering entry point, `ivfpq_probe_static`.

Some users of this library cannot hand it a workspace: they run after all device memory has been
given to a pool of their own, or inside a host application that forbids cudaMalloc because of the
device-wide synchronisation it implies.  For them the library keeps the [queries][nlist] distance
tile of the filtering stage in an array compiled into it.  These tests call that entry point
through the C ABI and compare it with the ordinary one (`ivfpq_debug_probes`, which takes a
caller's workspace): the probe lists and their distances must be identical bit for bit, on two
calls in a row of different shapes, because the second call finds the first call's leftovers in
the shared array.

The file name sorts last on purpose: a run that stops at the first failure has then already been
through every other test.
"""

import numpy as np
import pytest
import torch

import paper_2312_01712_b200 as lib
from ivfpq_inputs import lossless_toy_index

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_static_scratch_probes_equal_workspace_probes_twice(wl_small):
    h = lib.ivfpq_index_load(wl_small.index)
    try:
        q = dev(wl_small.queries)
        # first call: the whole batch; second call: fewer queries, another nprobe, stale tile below it
        for nq, nprobe in ((q.shape[0], 7), (40, 3), (q.shape[0], wl_small.index.nlist)):
            qs = q[:nq].contiguous()
            ref_ids, ref_d = lib.ivfpq_debug_probes(h, qs, nprobe)
            out = (torch.full((nq, nprobe), -7, dtype=torch.int32, device="cuda"),
                   torch.full((nq, nprobe), -1.0, dtype=torch.float32, device="cuda"))
            ids, d = lib.ivfpq_probe_static(h, qs, nprobe, out=out)
            # the call has no workspace whose status word could be read: its own status entry point
            assert lib.ivfpq_static_status() == lib.IVFPQ_OK
            assert torch.equal(ids, ref_ids)
            assert torch.equal(d.view(torch.int32), ref_d.view(torch.int32))
            # with the outputs supplied, further calls leave the device's free memory where it was
            free0 = torch.cuda.mem_get_info()[0]
            for _ in range(3):
                lib.ivfpq_probe_static(h, qs, nprobe, out=out)
                assert lib.ivfpq_static_status() == lib.IVFPQ_OK
            assert torch.cuda.mem_get_info()[0] == free0
            assert torch.equal(out[0], ref_ids)
    finally:
        lib.ivfpq_index_free(h)


def test_static_scratch_chunks_a_batch_larger_than_the_array():
    # nlist 4096 -> 511 queries fit the 8 MiB array at once; 1300 queries take three chunks
    idx, base = lossless_toy_index(seed=5, n=6000, nlist=4096, nsub=4, dsub=2, ksub=16, spread=4.0)
    h = lib.ivfpq_index_load(idx)
    try:
        rng = np.random.default_rng(3)
        q = dev((base[rng.integers(0, 6000, 1300)] + rng.standard_normal((1300, idx.d))).astype(np.float32))
        ref_ids, ref_d = lib.ivfpq_debug_probes(h, q, 9)
        for _ in range(2):
            ids, d = lib.ivfpq_probe_static(h, q, 9)
            assert torch.equal(ids, ref_ids) and torch.equal(d.view(torch.int32), ref_d.view(torch.int32))
    finally:
        lib.ivfpq_index_free(h)


def test_static_scratch_rejects_an_index_beyond_its_limit():
    nlist = lib.IVFPQ_STATIC_MAX_NLIST + 1
    idx, base = lossless_toy_index(seed=6, n=nlist + 50, nlist=nlist, nsub=2, dsub=2, ksub=8)
    h = lib.ivfpq_index_load(idx)
    try:
        q = dev(base[:4])
        with pytest.raises(lib.IvfpqError) as e:
            lib.ivfpq_probe_static(h, q, 2)
        assert e.value.code == lib.IVFPQ_ERR_STATIC_LIMIT
        assert "scratch" in str(e.value)
        # the ordinary entry point still serves it
        ids, _ = lib.ivfpq_debug_probes(h, q, 2)
        assert ids.shape == (4, 2)
    finally:
        lib.ivfpq_index_free(h)
