"""Matched GQA decode (the two-stream baseline the cache-size comparison refers to) against its oracle."""
import numpy as np
import pytest
import torch

from oracle import gva_oracle as orc
from paper_2609_13285_b200 import binding as gb
from paper_2609_13285_b200 import harness
from paper_2609_13285_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from tests import gpu_util
    gpu_util.ensure_built()


@pytest.mark.parametrize("kernel", [gb.GVA_KERNEL_FMA, gb.GVA_KERNEL_MMA])
@pytest.mark.parametrize("H,G,d_h", [(16, 4, 64), (32, 8, 128)])
@pytest.mark.parametrize("num_splits", [0, 3])
def test_gqa_decode_matches_oracle(kernel, H, G, d_h, num_splits):
    from tests import gpu_util as U
    g = wl.gqa_case("gqa", H, G, d_h, [0, 1, 63, 64, 65, 700, 2049], page_size=64, seed=401)
    dc = harness.upload_gqa(g, kernel=kernel)
    try:
        out, lse = dc.decode(num_splits=num_splits)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        ref, ref_lse = orc.gqa_decode(g["k_pool"], g["v_pool"], g["block_table"], g["seq_lens"], g["q"])
        o = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all()
        assert np.max(np.abs(o - ref)) <= U.TOL_TIGHT_MAXABS
        live = g["seq_lens"] > 0
        assert np.max(np.abs(lse.cpu().numpy()[live] - ref_lse[live])) <= 1e-4
        assert np.all(o[~live] == 0)
    finally:
        dc.close()


def test_gqa_f32_cache():
    g = wl.gqa_case("gqa32", 16, 4, 64, [5, 130, 1000], page_size=64, cache_dtype="f32", seed=402)
    dc = harness.upload_gqa(g)
    try:
        out, _ = dc.decode()
        torch.cuda.synchronize()
        ref, _ = orc.gqa_decode(g["k_pool"], g["v_pool"], g["block_table"], g["seq_lens"], g["q"])
        assert np.max(np.abs(out.cpu().numpy() - ref)) <= 1e-5
    finally:
        dc.close()


@pytest.mark.parametrize("H,G,d_h", [(16, 4, 64), (32, 8, 128)])
@pytest.mark.parametrize("num_splits", [0, 3])
def test_gqa_decode_over_the_8_bit_cache(H, G, d_h, num_splits):
    # keys and values as e4m3 codes: the decode widens them exactly, so the f32-level gate of the 16-bit cache stays
    from tests import gpu_util as U
    g = wl.gqa_case("gqa8", H, G, d_h, [0, 1, 63, 64, 65, 700, 2049, 5000], page_size=64, cache_dtype="fp8", seed=403)
    dc = harness.upload_gqa(g)
    try:
        out, lse = dc.decode(num_splits=num_splits)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        ref, ref_lse = orc.gqa_decode(g["k_pool"], g["v_pool"], g["block_table"], g["seq_lens"], g["q"])
        o = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all()
        assert np.max(np.abs(o - ref)) <= U.TOL_TIGHT_MAXABS
        live = g["seq_lens"] > 0
        assert np.max(np.abs(lse.cpu().numpy()[live] - ref_lse[live])) <= 1e-4
        assert np.all(o[~live] == 0)
    finally:
        dc.close()
