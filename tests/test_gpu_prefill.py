"""GPU parity of the prefill / chunked-prefill path (gva_absorb_query -> gva_append_chunk -> gva_prefill, through the
C ABI) against the fp64 oracle, which forms the keys explicitly (K_h = V_g M_h) and applies a plain causal softmax.

Tolerance: the kernel feeds the tensor cores bf16 operands -- the absorbed query and the softmax weights are each
rounded once to bf16 (relative error <= 2^-9), products are exact and accumulate in f32.  For unit-variance data a
score moves by about sqrt(d_v) * 2^-9 / sqrt(3) * scale ~ 1e-3 and a weight by 2^-9 relative, so outputs move by a few
1e-3 at most; the contract for a bf16 cache (max-abs <= 2e-2) is asserted, with rel-L2 <= 5e-3 as the tighter gate."""
import numpy as np
import pytest
import torch

from oracle import gva_oracle as orc
from paper_2609_13285_b200 import binding as gb
from paper_2609_13285_b200 import harness
from paper_2609_13285_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_MAXABS = 2e-2
TOL_REL_L2 = 5e-3
TOL_LSE = 2e-2


@pytest.fixture(scope="module", autouse=True)
def _built():
    from tests import gpu_util
    gpu_util.ensure_built()


def rel_l2(a, ref):
    return float(np.linalg.norm((a - ref).ravel()) / max(np.linalg.norm(ref.ravel()), 1e-30))


def run_prefill(pc, append=False):
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        if append:
            pd.append()
        out, lse = pd.prefill()
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0, f"device status {int(pd.status.item()):#x}"
        n = pc.n_q
        return out[:n].cpu().numpy().astype(np.float64), lse[:n].cpu().numpy().astype(np.float64), pd.dc.pools_to_host()
    finally:
        pd.close()


def check(pc):
    out, lse, _ = run_prefill(pc)
    ref_out, ref_lse = orc.prefill_case(pc)
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    err = float(np.max(np.abs(out - ref_out))) if out.size else 0.0
    assert err <= TOL_MAXABS, f"max-abs {err:.3e}"
    assert rel_l2(out, ref_out) <= TOL_REL_L2, f"rel-L2 {rel_l2(out, ref_out):.3e}"
    assert np.max(np.abs(lse - ref_lse)) <= TOL_LSE
    return err


@pytest.mark.parametrize("ctx,q", [
    ([0], [1]),                                   # one token sees itself
    ([0], [64]),                                  # exactly one tile, two query blocks
    ([0], [65]),                                  # ragged: one token into the second tile
    ([0, 5, 100, 64, 0, 1000], [70, 33, 1, 128, 200, 37]),
    ([0, 0, 7], [0, 300, 0]),                     # sequences without new tokens
])
def test_prefill_matches_oracle_shape_a(ctx, q):
    pc = wl.make_prefill_case("pf", wl.SHAPE_A, ctx, q, page_size=64, seed=501, poison_unused=True)
    check(pc)


def test_prefill_matches_oracle_shape_b():
    pc = wl.make_prefill_case("pfb", wl.SHAPE_B, [0, 130, 31], [150, 40, 97], page_size=64, seed=502, poison_unused=True)
    check(pc)


def test_prefill_contiguous_cache_and_large_pages():
    pc = wl.make_prefill_case("pfc", wl.SHAPE_A, [10, 200], [190, 100], page_size=128, paged=False, seed=503)
    check(pc)


def test_prefill_row_equals_decode_kernel_row():
    # the last row of a chunk is one decode step over the whole sequence: compare with gva_decode on the same cache
    pc = wl.make_prefill_case("pfd", wl.SHAPE_A, [300, 0], [100, 257], page_size=64, seed=504)
    out, lse, _ = run_prefill(pc)
    ref_out, _ = orc.prefill_case(pc)
    c = pc.cache
    last = pc.cu_q[1:] - 1
    c.q_c[:] = pc.q_c[last]; c.q_r[:] = pc.q_r[last]; c.q_pos[:] = pc.q_pos[last]
    dc = harness.upload(c)
    try:
        dc.absorb()
        o, _ = dc.decode()
        torch.cuda.synchronize()
        o = o.cpu().numpy().astype(np.float64)
    finally:
        dc.close()
    assert np.max(np.abs(o - ref_out[last])) <= 2e-5            # the decode kernel keeps f32 operands
    assert np.max(np.abs(o - out[last])) <= TOL_MAXABS


def test_chunked_prefill_equals_whole_prefill():
    whole = wl.make_prefill_case("w", wl.SHAPE_A, [0, 0], [333, 150], page_size=64, seed=505)
    out_w, lse_w, _ = run_prefill(whole)
    cut = np.array([100, 149])
    part = wl.make_prefill_case("p", wl.SHAPE_A, cut, np.array([333, 150]) - cut, page_size=64, seed=505)
    assert np.array_equal(part.cache.v_pool, whole.cache.v_pool)
    rows = np.concatenate([np.arange(whole.cu_q[b] + cut[b], whole.cu_q[b + 1]) for b in range(2)])
    part.q_c[:] = whole.q_c[rows]; part.q_r[:] = whole.q_r[rows]
    out_p, lse_p, _ = run_prefill(part)
    # same rows, same tiles, different row-to-block assignment: equal up to the bf16 rounding of the weights
    assert np.max(np.abs(out_p - out_w[rows])) <= 5e-3
    assert np.max(np.abs(lse_p - lse_w[rows])) <= 1e-3


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_append_chunk_is_bit_exact(dtype):
    pc = wl.make_prefill_case("ap", wl.SHAPE_A, [0, 63, 64, 500], [130, 2, 0, 77], page_size=64, cache_dtype=dtype, seed=506)
    c = pc.cache
    v_ref, k_ref = c.v_pool.copy(), c.kr_pool.copy()
    assert orc.append_chunk(v_ref, k_ref, c.block_table, pc.v_new, pc.kr_new, pc.cu_q, pc.ctx_lens) == 0
    pd = harness.upload_prefill(pc)
    try:
        pd.append()
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        v, k = pd.dc.pools_to_host()
    finally:
        pd.close()
    assert np.array_equal(v.view(np.uint8), v_ref.view(np.uint8)) and np.array_equal(k.view(np.uint8), k_ref.view(np.uint8))


@pytest.mark.parametrize("dtype", ["bf16", "f32", "fp8"])
def test_append_chunk_from_rows_that_are_only_4_byte_aligned(dtype):
    # the copy loop takes four elements per thread when the new rows are 16-byte aligned and one otherwise: same bits
    pc = wl.make_prefill_case("apu", wl.SHAPE_A, [5, 63, 500], [67, 2, 77], page_size=64, cache_dtype=dtype, seed=531)
    c = pc.cache
    v_ref, k_ref = c.v_pool.copy(), c.kr_pool.copy()
    assert orc.append_chunk(v_ref, k_ref, c.block_table, pc.v_new, pc.kr_new, pc.cu_q, pc.ctx_lens) == 0
    pd = harness.upload_prefill(pc)
    try:
        buf = torch.empty(pd.v_new.numel() + 1, dtype=torch.float32, device=pd.v_new.device)
        shifted = buf[1:].view(pd.v_new.shape)
        shifted.copy_(pd.v_new)
        assert shifted.data_ptr() % 16 == 4
        pd.v_new = shifted
        pd.append()
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        v, k = pd.dc.pools_to_host()
    finally:
        pd.close()
    assert np.array_equal(v.view(np.uint8), v_ref.view(np.uint8)) and np.array_equal(k.view(np.uint8), k_ref.view(np.uint8))


def test_append_then_prefill_follows_algorithm_order():
    # the chunk's own rows come from the append, not from the generator
    pc = wl.make_prefill_case("apf", wl.SHAPE_A, [40, 0], [90, 129], page_size=64, seed=507)
    c = pc.cache
    out, lse, (v, k) = run_prefill(pc, append=True)
    assert orc.append_chunk(c.v_pool, c.kr_pool, c.block_table, pc.v_new, pc.kr_new, pc.cu_q, pc.ctx_lens) == 0
    assert np.array_equal(v, c.v_pool) and np.array_equal(k, c.kr_pool)
    ref_out, ref_lse = orc.prefill_case(pc)
    assert np.max(np.abs(out - ref_out)) <= TOL_MAXABS and rel_l2(out, ref_out) <= TOL_REL_L2


def test_prefill_rejects_what_it_does_not_support():
    for kw in (dict(cache_dtype=gb.GVA_F32), dict(page_size=32)):
        args = dict(H=16, G=4, d_v=64, d_c=64, d_r=16, page_size=64)
        args.update(kw)
        h = gb.gva_create(**args)
        try:
            t = torch.zeros(4096, dtype=torch.float32, device="cuda")
            i = torch.zeros(16, dtype=torch.int32, device="cuda")
            cache = gb.make_cache(t, t, None, 4, 4)
            assert gb.gva_prefill(h, cache, t, i, i, t, None, 1, 8, check=False) == gb.GVA_ERR_UNSUPPORTED
        finally:
            gb.gva_destroy(h)


def test_prefill_reports_bad_page_and_long_sequence():
    pc = wl.make_prefill_case("bad", wl.SHAPE_A, [0, 0], [100, 40], page_size=64, seed=508)
    pc.cache.block_table[0, 1] = pc.cache.num_pages + 5
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        pd.prefill()
        torch.cuda.synchronize()
        st = int(pd.status.item())
        assert st & 0xff == gb.GVA_ERR_BAD_PAGE and st >> 8 == 0
        out = pd.out.cpu().numpy()
        ref, _ = orc.prefill_case(wl.make_prefill_case("bad", wl.SHAPE_A, [0, 0], [100, 40], page_size=64, seed=508))
        assert np.max(np.abs(out[100:140] - ref[100:140])) <= TOL_MAXABS     # the other sequence is unaffected
        pd.status.zero_()
        pd.dc.block_table.copy_(torch.from_numpy(wl.make_prefill_case("bad", wl.SHAPE_A, [0, 0], [100, 40], page_size=64,
                                                                      seed=508).cache.block_table).to(pd.dc.block_table.device))
        pd.ctx_lens[1] = 10_000                                               # beyond its block table
        pd.prefill()
        torch.cuda.synchronize()
        st = int(pd.status.item())
        assert st & 0xff == gb.GVA_ERR_SEQ_LEN and st >> 8 == 1
    finally:
        pd.close()


@pytest.mark.parametrize("shape", [wl.SHAPE_A, wl.SHAPE_B])
def test_absorb_many_rows_matches_oracle_and_the_small_batch_kernel(shape):
    # prefill absorbs one row per new token: above 512 rows a tensor-core kernel takes over (f16 hi/lo operands); it must
    # give the oracle's values within the same bound, the same rotated slice bit for bit (fp64 rotation, one rounding),
    # and agree with the decode-batch kernel to f32 rounding level
    n = 1000 + 37
    pc = wl.make_prefill_case("abs", shape, [3], [n], page_size=64, seed=509)
    pd = harness.upload_prefill(pc)
    try:
        q = pd.absorb().cpu().numpy()
        ref = orc.absorb(pc.q_c, pc.q_r, pc.cache.M, pc.q_pos)
        assert np.max(np.abs(q.astype(np.float64) - ref)) <= 1e-5
        assert np.array_equal(q[..., shape.d_v:], ref[..., shape.d_v:].astype(np.float32))      # fp64 rotation, one rounding
        small = torch.empty_like(pd.q_abs)
        for lo in range(0, n, 100):
            hi = min(n, lo + 100)
            gb.gva_absorb_query(pd.handle, pd.q_c[lo:hi], pd.q_r[lo:hi], pd.dc.M, pd.q_pos[lo:hi], small[lo:hi], hi - lo)
        torch.cuda.synchronize()
        sm = small.cpu().numpy()
        assert np.array_equal(sm[..., shape.d_v:].view(np.uint32), q[..., shape.d_v:].view(np.uint32))
        assert np.max(np.abs(sm.astype(np.float64) - q.astype(np.float64))) <= 2e-5      # each is within 1e-5 of the oracle
    finally:
        pd.close()


# ------------------------------------------------------------------ multi-token decode with split-KV
@pytest.mark.parametrize("num_splits", [0, 1, 2, 7, 64])
def test_decode_multi_matches_oracle_and_prefill(num_splits):
    # a few new tokens per sequence over a long cached context: the oracle's chunked-prefill rows, computed by several
    # thread blocks per query block and merged; more splits than some sequences have tiles; a sequence without new tokens
    ctx = [5000, 130, 64, 0, 2047, 700]
    q = [4, 1, 8, 3, 33, 0]
    pc = wl.make_prefill_case("multi", wl.SHAPE_A, ctx, q, page_size=64, seed=510, poison_unused=True)
    ref_out, ref_lse = orc.prefill_case(pc)
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        out, lse = pd.decode_multi(num_splits=num_splits)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all() and np.isfinite(l).all()
        assert np.max(np.abs(o - ref_out)) <= TOL_MAXABS and rel_l2(o, ref_out) <= TOL_REL_L2
        assert np.max(np.abs(l - ref_lse)) <= TOL_LSE
        pd.out.fill_(float("nan"))
        o1, _ = pd.prefill()
        torch.cuda.synchronize()
        assert np.max(np.abs(o1[:pc.n_q].cpu().numpy() - o)) <= 5e-3
    finally:
        pd.close()


def test_decode_multi_wide_shape_and_workspace_check():
    pc = wl.make_prefill_case("multi-b", wl.SHAPE_B, [1500, 90], [5, 2], page_size=64, seed=511)
    ref_out, _ = orc.prefill_case(pc)
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        out, _ = pd.decode_multi(num_splits=0)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out[:pc.n_q].cpu().numpy().astype(np.float64)
        assert np.max(np.abs(o - ref_out)) <= TOL_MAXABS and rel_l2(o, ref_out) <= TOL_REL_L2
        small = torch.empty(256, dtype=torch.uint8, device="cuda")
        rc = gb.gva_decode_multi(pd.handle, pd.dc.cache, pd.q_abs, pd.cu_q, pd.ctx_lens, pd.out, pd.lse, small, 2, pc.n_q, 5, 1505, 4,
                                 check=False)
        assert rc == gb.GVA_ERR_WORKSPACE
    finally:
        pd.close()


# ------------------------------------------------------------------ q_len new tokens on the split-KV decode kernel
@pytest.mark.parametrize("q_len", [2, 3, 4])
@pytest.mark.parametrize("shape", [wl.SHAPE_A, wl.SHAPE_B, wl.SHAPE_C])
@pytest.mark.parametrize("num_splits", [0, 1, 5])
def test_decode_tokens_matches_oracle(q_len, shape, num_splits):
    # exactly q_len new tokens per sequence over contexts around tile and page boundaries (a context of 0 too: the first
    # new token then sees only itself), poisoned unused slots; the oracle is the chunked-prefill oracle
    ctx = [0, 1, 61, 62, 63, 64, 65, 127, 128, 700, 2047, 5000]
    pc = wl.make_prefill_case("tok", shape, ctx, [q_len] * len(ctx), page_size=64, seed=520 + q_len, poison_unused=True)
    ref_out, ref_lse = orc.prefill_case(pc)
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        out, lse = pd.decode_tokens(q_len, num_splits=num_splits)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all() and np.isfinite(l).all()
        assert np.max(np.abs(o - ref_out)) <= TOL_MAXABS, np.max(np.abs(o - ref_out))
        assert rel_l2(o, ref_out) <= TOL_REL_L2
        assert np.max(np.abs(l - ref_lse)) <= TOL_LSE
    finally:
        pd.close()


def test_decode_tokens_unsupported_and_page_size_32():
    pc = wl.make_prefill_case("tok32", wl.SHAPE_A, [300, 31], [2, 2], page_size=32, seed=530)
    ref_out, _ = orc.prefill_case(pc)
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        out, _ = pd.decode_tokens(2)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        assert np.max(np.abs(out[:pc.n_q].cpu().numpy().astype(np.float64) - ref_out)) <= TOL_MAXABS
        ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
        # more than eight new tokens, and five to eight with pages that are not a multiple of 64 tokens, are not built
        rc = gb.gva_decode_tokens(pd.handle, pd.dc.cache, pd.q_abs, pd.dc.seq_lens, pd.out, pd.lse, ws, 2, 9, 302, 0, check=False)
        assert rc == gb.GVA_ERR_UNSUPPORTED
        ws = torch.empty(gb.gva_decode_tokens_workspace_bytes(pd.handle, 2, 5, 302, 0), dtype=torch.uint8, device="cuda")
        rc = gb.gva_decode_tokens(pd.handle, pd.dc.cache, pd.q_abs, pd.dc.seq_lens, pd.out, pd.lse, ws, 2, 5, 302, 0, check=False)
        assert rc == gb.GVA_ERR_UNSUPPORTED
    finally:
        pd.close()


@pytest.mark.parametrize("shape", [wl.SHAPE_A0, wl.SHAPE_B0])
def test_prefill_and_decode_multi_value_only_cache(shape):
    # the cache without a positional slice (d_r = 0): keys are the reconstructed content keys alone, scale 1/sqrt(d_c)
    pc = wl.make_prefill_case("pf0", shape, [0, 70, 1000], [130, 33, 5], page_size=64, seed=540, poison_unused=True)
    check(pc)
    ref_out, _ = orc.prefill_case(pc)
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        out, _ = pd.decode_multi(num_splits=3)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out[:pc.n_q].cpu().numpy().astype(np.float64)
        assert np.max(np.abs(o - ref_out)) <= TOL_MAXABS and rel_l2(o, ref_out) <= TOL_REL_L2
    finally:
        pd.close()


def test_prefill_and_decode_multi_rope_width_24():
    # d_r = 24: 48-byte positional-key rows, which enter the score product as 32 dims of which the last 8 are zero on both sides
    pc = wl.make_prefill_case("pf24", wl.SHAPE_C, [0, 70, 1000, 63], [130, 33, 5, 64], page_size=64, seed=541, poison_unused=True)
    check(pc)
    ref_out, ref_lse = orc.prefill_case(pc)
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        for splits in (1, 3):
            out, lse = pd.decode_multi(num_splits=splits)
            torch.cuda.synchronize()
            assert int(pd.status.item()) == 0
            o = out[:pc.n_q].cpu().numpy().astype(np.float64)
            assert np.max(np.abs(o - ref_out)) <= TOL_MAXABS and rel_l2(o, ref_out) <= TOL_REL_L2
            assert np.max(np.abs(lse[:pc.n_q].cpu().numpy() - ref_lse)) <= TOL_LSE
    finally:
        pd.close()
    # peaked scores keep the contract there too (the query enters as hi + lo in all 32 positional columns)
    pk = wl.make_prefill_case("pf24p", wl.SHAPE_C, [300], [100], page_size=64, seed=542, q_gain=6.0)
    check(pk)


def test_append_then_decode_tokens_follows_algorithm_order():
    # Algorithm 1 for three new tokens at once: absorb, append all three, then attend; the new tokens' own rows come
    # from the append (bit-exact against the oracle's), each new token sees its predecessors and itself
    q_len = 3
    pc = wl.make_prefill_case("atok", wl.SHAPE_A, [63, 640, 0, 4095], [q_len] * 4, page_size=64, seed=541)
    c = pc.cache
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        pd.append()
        out, lse = pd.decode_tokens(q_len)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        v, k = pd.dc.pools_to_host()
        o = out[:pc.n_q].cpu().numpy().astype(np.float64)
    finally:
        pd.close()
    assert orc.append_chunk(c.v_pool, c.kr_pool, c.block_table, pc.v_new, pc.kr_new, pc.cu_q, pc.ctx_lens) == 0
    assert np.array_equal(v, c.v_pool) and np.array_equal(k, c.kr_pool)
    ref_out, _ = orc.prefill_case(pc)
    assert np.max(np.abs(o - ref_out)) <= TOL_MAXABS and rel_l2(o, ref_out) <= TOL_REL_L2


@pytest.mark.parametrize("q_gain", [0.0, 6.0, 30.0])
def test_prefill_and_decode_tokens_flat_and_peaked_scores(q_gain):
    # zero queries give uniform weights (the running mean of the value rows); large queries give sharply peaked
    # weights whose maximum jumps from tile to tile, so the reference of a row moves and O is rescaled again and again.
    # The kernels take the score product with the query as two bf16 numbers (hi + lo), so the size of the scores does
    # not enter the error: the contract holds at every gain (what is left is the bf16 rounding of the softmax weights,
    # about 2^-9 of the largest value component).
    pc = wl.make_prefill_case("peak", wl.SHAPE_A, [0, 900], [300, 4], page_size=64, seed=550, q_gain=q_gain)
    ref_out, ref_lse = orc.prefill_case(pc)
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        out, lse = pd.prefill()
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all() and np.isfinite(l).all()
        assert np.max(np.abs(o - ref_out)) <= TOL_MAXABS and np.max(np.abs(l - ref_lse)) <= TOL_LSE
        pd.out.fill_(float("nan")); pd.lse.fill_(float("nan"))
        out2, lse2 = pd.decode_multi(num_splits=4)
        torch.cuda.synchronize()
        o2 = out2[:pc.n_q].cpu().numpy().astype(np.float64); l2 = lse2[:pc.n_q].cpu().numpy().astype(np.float64)
        assert np.max(np.abs(o2 - ref_out)) <= TOL_MAXABS and np.max(np.abs(l2 - ref_lse)) <= TOL_LSE
    finally:
        pd.close()
    # the same on the split-KV decode kernel (gva_decode_tokens: every sequence with the same number of new tokens)
    for shape, q_len in ((wl.SHAPE_A, 4), (wl.SHAPE_A, 2), (wl.SHAPE_B, 3)):
        pc = wl.make_prefill_case("peakt", shape, [900, 64, 0], [q_len] * 3, page_size=64, seed=551 + q_len, q_gain=q_gain)
        ref_out, ref_lse = orc.prefill_case(pc)
        pd = harness.upload_prefill(pc)
        try:
            pd.absorb()
            out, lse = pd.decode_tokens(q_len)
            torch.cuda.synchronize()
            assert int(pd.status.item()) == 0
            o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
            assert np.max(np.abs(o - ref_out)) <= TOL_MAXABS and np.max(np.abs(l - ref_lse)) <= TOL_LSE, (shape, q_len)
        finally:
            pd.close()


@pytest.mark.parametrize("it", range(16))
def test_random_cases_through_every_multi_token_entry_point(it):
    # seeded random batches (shape, batch, contexts, chunk lengths, page size, paged or contiguous, poisoned slots) through
    # gva_prefill, gva_decode_multi (given and automatic split counts) and gva_decode_tokens, against the oracle
    rng = np.random.default_rng(7000 + it)
    shape = wl.SHAPE_A if it % 3 else wl.SHAPE_B
    B = int(rng.integers(1, 7))
    ctx = rng.integers(0, 1500, size=B)
    mode = it % 4
    if mode == 3:
        q = np.full(B, int(rng.integers(2, 5)))
    else:
        q = rng.integers(0, 200, size=B)
        if q.sum() == 0:
            q[0] = 5
    pc = wl.make_prefill_case("rnd", shape, ctx, q, page_size=64 if it % 5 else 128, seed=9000 + it, poison_unused=True,
                              paged=bool(it % 2))
    ref, ref_l = orc.prefill_case(pc)
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        if mode == 0:
            out, lse = pd.prefill()
        elif mode == 1:
            out, lse = pd.decode_multi(num_splits=int(rng.integers(1, 9)))
        elif mode == 2:
            out, lse = pd.decode_multi(num_splits=0)
        else:
            out, lse = pd.decode_tokens(int(q[0]), num_splits=int(rng.integers(0, 4)))
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all() and np.isfinite(l).all()
        assert np.max(np.abs(o - ref)) <= TOL_MAXABS and np.max(np.abs(l - ref_l)) <= TOL_LSE
    finally:
        pd.close()


@pytest.mark.parametrize("block", range(6))
def test_random_sweep_over_shapes_cache_types_and_score_scales(block):
    # ten seeded random cases per block: the five head shapes, bf16 and 8-bit caches, queries at 1, 6 and 30 times the unit
    # scale (scaled scores up to +-100, single rows dominating), through gva_prefill, gva_decode_multi, gva_decode_tokens
    # and gva_decode_tokens_ragged; one contract for all: |out - oracle| <= 2e-2, |lse - oracle| <= 2e-2
    rng = np.random.default_rng(4321 + block)
    shapes = [wl.SHAPE_A, wl.SHAPE_B, wl.SHAPE_C, wl.SHAPE_A0, wl.SHAPE_B0]
    for it in range(10):
        shape = shapes[int(rng.integers(0, len(shapes)))]
        dt = "fp8" if (rng.random() < 0.4 and shape.d_r != 24) else "bf16"
        B = int(rng.integers(1, 9))
        ctx = rng.integers(0, 2500, size=B)
        mode = int(rng.integers(0, 5))
        gain = float(rng.choice([1.0, 1.0, 6.0, 30.0]))
        maxq = 8 if (dt == "bf16" and shape.d_v == 64) else 4
        if dt == "fp8" and shape.d_r == 0 and mode >= 3:
            mode = 1                                   # the 8-bit multi-token kernel needs a positional slice
        if mode == 3:
            q = np.full(B, int(rng.integers(2, maxq + 1)))
        elif mode == 4:
            q = rng.integers(0, maxq + 1, size=B)
            q[int(rng.integers(0, B))] = maxq
        else:
            q = rng.integers(0, 260, size=B)
            if q.sum() == 0:
                q[0] = 5
        pc = wl.make_prefill_case("sweep", shape, ctx, q, page_size=64 if rng.random() < 0.8 else 128, cache_dtype=dt,
                                  seed=19000 + 100 * block + it, poison_unused=True, paged=bool(rng.integers(0, 2)), q_gain=gain)
        ref, ref_l = orc.prefill_case(pc)
        pd = harness.upload_prefill(pc)
        try:
            pd.absorb()
            pd.out.fill_(float("nan"))
            if mode == 0:
                out, lse = pd.prefill()
            elif mode == 1:
                out, lse = pd.decode_multi(num_splits=int(rng.integers(0, 9)))
            elif mode == 2:
                out, lse = pd.decode_multi(num_splits=0)
            elif mode == 3:
                out, lse = pd.decode_tokens(int(q[0]), num_splits=int(rng.integers(0, 4)))
            else:
                out, lse = pd.decode_tokens_ragged(num_splits=int(rng.integers(0, 3)))
            torch.cuda.synchronize()
            what = (block, it, mode, shape, dt, gain, q.tolist())
            assert int(pd.status.item()) == 0, what
            o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
            assert np.isfinite(o).all() and np.isfinite(l).all(), what
            assert np.max(np.abs(o - ref)) <= TOL_MAXABS and np.max(np.abs(l - ref_l)) <= TOL_LSE, what
        finally:
            pd.close()


@pytest.mark.parametrize("q_len", [5, 6, 7, 8])
@pytest.mark.parametrize("shape_name", ["A", "A0", "C"])
def test_decode_tokens_five_to_eight_new_tokens(q_len, shape_name):
    # five to eight new tokens per sequence on the split-KV decode kernel (two consumer warps per value group share each
    # tile's columns), over ragged contexts with poisoned slots, given and automatic split counts, flat and peaked scores
    shape = {"A": wl.SHAPE_A, "A0": wl.SHAPE_A0, "C": wl.SHAPE_C}[shape_name]
    for gain, splits in ((1.0, 0), (6.0, 3)):
        pc = wl.make_prefill_case("tok8", shape, [4095 - q_len, 0, 63, 700, 64 - q_len], [q_len] * 5, page_size=64, seed=560 + q_len,
                                  q_gain=gain, poison_unused=True)
        ref_out, ref_lse = orc.prefill_case(pc)
        pd = harness.upload_prefill(pc)
        try:
            pd.absorb()
            out, lse = pd.decode_tokens(q_len, num_splits=splits)
            torch.cuda.synchronize()
            assert int(pd.status.item()) == 0
            o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
            assert np.isfinite(o).all() and np.isfinite(l).all()
            assert np.max(np.abs(o - ref_out)) <= TOL_MAXABS and rel_l2(o, ref_out) <= TOL_REL_L2
            assert np.max(np.abs(l - ref_lse)) <= TOL_LSE
        finally:
            pd.close()


@pytest.mark.parametrize("case_no", range(6))
def test_decode_tokens_with_a_count_per_sequence(case_no):
    # gva_decode_tokens_ragged: every sequence its own number of new tokens (none .. eight), against the chunked-prefill
    # oracle; rows of sequences without new tokens do not exist, rows past the last one must stay untouched
    rng = np.random.default_rng(8100 + case_no)
    B = int(rng.integers(1, 9))
    max_q = [8, 4, 2, 8, 3, 1][case_no]
    q = rng.integers(0, max_q + 1, size=B)
    q[int(rng.integers(0, B))] = max_q
    ctx = rng.integers(0, 3000, size=B)
    shape = wl.SHAPE_A if case_no != 4 else wl.SHAPE_B          # (the wide-head shape goes up to four new tokens)
    pc = wl.make_prefill_case("rag", shape, ctx, q, page_size=64, seed=8200 + case_no, poison_unused=True, paged=bool(case_no % 2))
    ref_out, ref_lse = orc.prefill_case(pc)
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        pd.out.fill_(float("nan")); pd.lse.fill_(float("nan"))
        out, lse = pd.decode_tokens_ragged(num_splits=0 if case_no % 3 else 2)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all() and np.isfinite(l).all()
        assert np.max(np.abs(o - ref_out)) <= TOL_MAXABS and np.max(np.abs(l - ref_lse)) <= TOL_LSE
        assert torch.isnan(out[pc.n_q:]).all()
    finally:
        pd.close()


def test_value_only_cache_multi_token_and_host_step():
    # the cache without a positional slice through gva_decode_tokens (2 and 4 new tokens) and through the host-buffer step
    for q_len in (2, 4):
        pc = wl.make_prefill_case("vo-tok", wl.SHAPE_A0, [900, 0, 63], [q_len] * 3, page_size=64, seed=570 + q_len)
        ref_out, _ = orc.prefill_case(pc)
        pd = harness.upload_prefill(pc)
        try:
            pd.absorb()
            out, _ = pd.decode_tokens(q_len)
            torch.cuda.synchronize()
            assert int(pd.status.item()) == 0
            assert np.max(np.abs(out[:pc.n_q].cpu().numpy().astype(np.float64) - ref_out)) <= TOL_MAXABS
        finally:
            pd.close()
    lens = np.array([300, 64, 1], dtype=np.int32)
    case = wl.make_case("vo-host", wl.SHAPE_A0, lens, page_size=64, cache_dtype="bf16", seed=575, q_pos=lens - 1, append_pos=lens - 1)
    dc = harness.upload(case)
    try:
        want, _ = dc.step()
        torch.cuda.synchronize()
        want = want.clone()
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        h_out = torch.empty(want.shape, dtype=torch.float32).pin_memory()
        scratch = torch.empty(gb.gva_step_scratch_bytes(dc.handle, case.B, int(lens.max()), 0), dtype=torch.uint8, device="cuda")
        gb.gva_decode_step_host(dc.handle, dc.cache, dc.M, pin(case.q_c), None, pin(case.v_new), None, pin(case.append_pos),
                                pin(lens), h_out, scratch, case.B, int(lens.max()), 0, dc.status)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        assert torch.equal(h_out, want.cpu())
    finally:
        dc.close()
