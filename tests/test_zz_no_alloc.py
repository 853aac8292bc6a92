"""gva_decode_static: the decode entry point for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is not an option (a serving loop with a frozen
memory pool, a plug-in that receives tensors but no allocator), so they cannot hand gva_decode a
workspace.  gva_decode_static keeps the split-KV partial results in a fixed array inside the
library instead.  This test calls it through the C ABI twice in a row -- the second call finds
the array filled with the first call's partials -- and checks both results against gva_decode
with a caller workspace, within the tight gate the other parity tests use.  It lives in a file
that pytest collects last so that a failure here cannot hide any other test's result.
"""
import numpy as np
import pytest
import torch

from paper_2609_13285_b200 import binding as gb
from paper_2609_13285_b200 import harness
from paper_2609_13285_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from tests import gpu_util
    gpu_util.ensure_built()


def test_static_scratch_decode_matches_workspace_decode_twice():
    from tests import gpu_util as U
    # two different batches back to back: the second call must not be disturbed by what the first left
    cases = [wl.make_case("noalloc0", wl.SHAPE_A, [3000, 129, 0, 64, 4097], page_size=64, cache_dtype="bf16", seed=301,
                          poison_unused=True),
             wl.make_case("noalloc1", wl.SHAPE_A, [70, 2500, 1], page_size=64, cache_dtype="bf16", seed=302)]
    for num_splits in (0, 3):
        for case in cases:
            dc = harness.upload(case)
            try:
                dc.absorb()
                ref_out, ref_lse = dc.decode(num_splits=num_splits)
                ref_out, ref_lse = ref_out.clone(), ref_lse.clone()
                o_ref, _ = U.oracle_for_gpu_q(case, dc.q_abs)
                r = ref_out.cpu().numpy().astype(np.float64)
                live = case.seq_lens > 0
                for _rep in range(2):                 # two calls in a row on the same scratch
                    dc.out.fill_(float("nan"))
                    dc.lse.fill_(float("nan"))
                    torch.cuda.synchronize()
                    free_before = torch.cuda.mem_get_info()[0]          # cudaMemGetInfo: free device bytes, driver's view
                    gb.gva_decode_static(dc.handle, dc.cache, dc.q_abs, dc.seq_lens, dc.out, dc.lse, case.B,
                                         dc.max_seq_len, num_splits, dc.status)
                    torch.cuda.synchronize()
                    # the call allocated nothing: not a byte of device memory less than before it
                    assert torch.cuda.mem_get_info()[0] == free_before
                    assert int(dc.status.item()) == 0
                    a = dc.out.cpu().numpy().astype(np.float64)
                    assert np.isfinite(a).all()
                    assert np.max(np.abs(a - r)) <= U.TOL_TIGHT_MAXABS
                    assert np.allclose(dc.lse.cpu().numpy()[live], ref_lse.cpu().numpy()[live], atol=1e-5)
                    assert np.max(np.abs(a - o_ref)) <= U.TOL_TIGHT_MAXABS      # and against the oracle directly
            finally:
                dc.close()


def test_static_scratch_rejects_requests_beyond_its_size():
    case = wl.make_case("noalloc_big", wl.SHAPE_A, [64], page_size=64, cache_dtype="bf16", seed=303)
    dc = harness.upload(case)
    try:
        dc.absorb()
        B_big, splits = 4096, 16                      # 4096 * 16 partial records: far beyond 16 MiB
        assert gb.gva_decode_workspace_bytes(dc.handle, B_big, 64, splits) > gb.GVA_STATIC_SCRATCH_BYTES
        rc = gb.gva_decode_static(dc.handle, dc.cache, dc.q_abs, dc.seq_lens, dc.out, dc.lse, B_big, 64, splits,
                                  dc.status, check=False)
        assert rc == gb.GVA_ERR_STATIC_LIMIT
        assert "built-in scratch" in gb.status_string(rc)
    finally:
        dc.close()


def test_static_scratch_holds_the_five_benchmark_workloads():
    # at automatic splits every one of the five workloads of the benchmark needs less than the built-in array
    # (the header says so; this keeps the statement true when the partition or the record layout changes)
    shapes = {"cfg0": (wl.SHAPE_A, gb.GVA_F32, 1, 128), "cfg1": (wl.SHAPE_A, gb.GVA_BF16, 8, 4096),
              "cfg2": (wl.SHAPE_A, gb.GVA_BF16, 32, 32768), "cfg3": (wl.SHAPE_B, gb.GVA_BF16, 64, 16384),
              "cfg4": (wl.SHAPE_A, gb.GVA_BF16, 128, 8193)}
    for name, (s, dtype, B, T) in shapes.items():
        h = gb.gva_create(H=s.H, G=s.G, d_v=s.d_v, d_c=s.d_c, d_r=s.d_r, page_size=64, cache_dtype=dtype)
        try:
            need = gb.gva_decode_workspace_bytes(h, B, T, 0)
            assert 0 < need <= gb.GVA_STATIC_SCRATCH_BYTES, (name, need)
        finally:
            gb.gva_destroy(h)
