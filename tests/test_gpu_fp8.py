"""GPU parity over the 8-bit (e4m3) cache: the CUDA library against the fp64 oracle, which reads the same stored codes
exactly (every e4m3 value is an f16 value), so the tight f32-arithmetic gates apply unchanged."""
import numpy as np
import pytest
import torch

from oracle import gva_oracle as orc
from paper_2609_13285_b200 import binding as gb
from paper_2609_13285_b200 import harness
from paper_2609_13285_b200 import workloads as wl

pytestmark = pytest.mark.gpu

EDGE_LENS = [0, 1, 31, 32, 33, 63, 64, 65, 127, 128, 129, 640, 641, 1000]


@pytest.fixture(scope="module", autouse=True)
def _built():
    from tests import gpu_util
    gpu_util.ensure_built()


def U():
    from tests import gpu_util
    return gpu_util


SHAPES = [wl.SHAPE_A, wl.SHAPE_B, wl.SHAPE_A0, wl.SHAPE_B0]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("num_splits", [0, 1, 5, 40])
def test_ragged_edge_lengths_poisoned(shape, num_splits):
    # lengths around tile and page boundaries, an empty sequence, more splits than tiles; every slot no live token
    # occupies holds the NaN code and unused block-table entries are -1
    case = wl.make_case("edge8", shape, EDGE_LENS, page_size=64, cache_dtype="fp8", seed=801, poison_unused=True,
                        extra_pages=2)
    U().check_decode(case, gb.GVA_KERNEL_AUTO, num_splits=num_splits)


def test_eight_groups_of_narrow_heads():
    # d_v = 64 with G = 8 (nine-warp blocks, two per SM instead of four): ragged, poisoned, balanced and split
    shape = wl.HeadShape(H=32, G=8, d_v=64, d_c=64, d_r=16)
    for num_splits in (0, 3):
        case = wl.make_case("g8", shape, [5, 64, 700, 2049, 0, 333], page_size=64, cache_dtype="fp8", seed=813,
                            poison_unused=True)
        U().check_decode(case, gb.GVA_KERNEL_AUTO, num_splits=num_splits)


@pytest.mark.parametrize("shape", [wl.SHAPE_A, wl.SHAPE_B])
@pytest.mark.parametrize("num_splits", [0, 2, 7])
def test_long_batch_all_split_counts(shape, num_splits):
    case = wl.make_case("long8", shape, [4096] * 8, page_size=64, cache_dtype="fp8", paged=False, seed=802)
    dc = harness.upload(case)
    try:
        U().check_decode(case, gb.GVA_KERNEL_AUTO, num_splits=num_splits, dc=dc)
        assert gb.gva_last_kernel(dc.handle) == gb.GVA_KERNEL_MMA
    finally:
        dc.close()


@pytest.mark.parametrize("shape", [wl.SHAPE_A, wl.SHAPE_B])
def test_every_value_dim_and_token_slot_lands_where_it_should(shape):
    # one-hot probes: a cache whose only non-zero element is (token t, group g, dim d) and a flat score row give
    # out[h, d'] = value / T at d' = d for the heads of group g and zero elsewhere -- catches any permutation of dims,
    # tokens or heads on the way through the byte fragments
    T = 128
    case = wl.make_case("onehot8", shape, [T] * 6, page_size=64, cache_dtype="fp8", seed=803, q_gain=0.0)
    one = int(wl.f32_to_e4m3_bits(np.array([1.0], dtype=np.float32))[0])
    case.v_pool[:] = 0
    case.kr_pool[:] = 0
    probes = [(0, 0, 0), (1, 1, 17), (77, 2, 34), (127, 3, 63), (64, 0, 49), (15, 3, 6)]
    if shape.d_v == 128:
        probes = [(0, 0, 0), (1, 5, 17 + 64), (77, 2, 34), (127, 7, 127), (33, 4, 49 + 64), (47, 3, 6 + 64)]
    for b, (t, g, d) in enumerate(probes):
        page = int(case.block_table[b, t // 64])
        case.v_pool[page, g, t % 64, d] = one
    dc = harness.upload(case)
    try:
        dc.absorb()
        out, _ = dc.decode()
        torch.cuda.synchronize()
        o = out.cpu().numpy()
        s = case.shape
        for b, (t, g, d) in enumerate(probes):
            want = np.zeros((s.H, s.d_v), dtype=np.float32)
            want[g * 4:(g + 1) * 4, d] = 1.0 / T
            assert np.allclose(o[b], want, atol=1e-7), (b, t, g, d)
    finally:
        dc.close()


@pytest.mark.parametrize("s", [wl.SHAPE_A, wl.SHAPE_B])
def test_score_side_sees_every_dim_in_place(s):
    # scores pick the token: a query far along one dim and a cache whose token t carries a large value at that dim only
    # must put (nearly) all weight on t -- one probe per 16-dim chunk and byte lane, the positional slice included
    T = 64
    dims = [0, 1, 2, 3, 5, 18, 35, 52, 63, 64, 67, 70, 79]        # >= d_v: the positional slice
    if s.d_v == 128:
        dims = [0, 3, 18, 63, 64, 77, 100, 127, 128, 131, 141, 146, 159]
    case = wl.make_case("score8", s, [T] * len(dims), page_size=64, cache_dtype="fp8", seed=804, q_gain=0.0)
    big = int(wl.f32_to_e4m3_bits(np.array([16.0], dtype=np.float32))[0])
    one = int(wl.f32_to_e4m3_bits(np.array([1.0], dtype=np.float32))[0])
    case.v_pool[:] = 0
    case.kr_pool[:] = 0
    for b, d in enumerate(dims):
        t = (7 * b + 3) % T
        page = int(case.block_table[b, 0])
        if d < s.d_v:
            case.v_pool[page, :, t, d] = big
        else:
            case.kr_pool[page, t, d - s.d_v] = big
        case.v_pool[page, :, t, (d + 9) % s.d_v] = one      # marks the token in the output (beside the score dim)
    dc = harness.upload(case)
    try:
        q = np.zeros((len(dims), s.H, s.d_v + s.d_r), dtype=np.float32)
        for b, d in enumerate(dims):
            q[b, :, d] = 40.0
        dc.q_abs.copy_(torch.from_numpy(q))
        out, _ = dc.decode()
        torch.cuda.synchronize()
        o = out.cpu().numpy().astype(np.float64)
        ref, _ = orc.decode_case(case, q.astype(np.float64))
        assert np.max(np.abs(o - ref)) <= 2e-5
        for b, d in enumerate(dims):
            assert abs(o[b, 0, (d + 9) % s.d_v] - 1.0) < 1e-3
    finally:
        dc.close()


def test_peaked_and_flat_scores():
    case = wl.make_case("peak8", wl.SHAPE_A, [500, 2049, 64], page_size=64, cache_dtype="fp8", seed=805, q_gain=30.0)
    U().check_decode(case, gb.GVA_KERNEL_AUTO, tight=False)
    case = wl.make_case("flat8", wl.SHAPE_A, [500, 2049, 64], page_size=64, cache_dtype="fp8", seed=806, q_gain=0.0)
    U().check_decode(case, gb.GVA_KERNEL_AUTO)


def test_page_sizes_and_contiguous():
    for P, paged in ((128, True), (256, False), (64, False)):
        case = wl.make_case("ps8", wl.SHAPE_A, [777, 3], page_size=P, cache_dtype="fp8", paged=paged, seed=807 + P,
                            poison_unused=True)
        U().check_decode(case, gb.GVA_KERNEL_AUTO)


@pytest.mark.parametrize("shape", SHAPES)
def test_append_is_bit_exact_and_saturates(shape):
    lens = [1, 64, 65, 300, 129, 4000, 8193]
    case = wl.make_case("append8", shape, lens, page_size=64, cache_dtype="fp8", seed=808, extra_pages=3)
    # values beyond the largest finite code, ties between codes, subnormals and zeros of both signs
    case.v_new[0, 0, :8] = [1e6, -1e6, 448.0, 464.0, 1.0625, 1.1875, 2.0 ** -10, -0.0]
    case.v_new[1, 1, :4] = [3 * 2.0 ** -10, 2.0 ** -6 - 2.0 ** -10, -449.0, 0.0]
    dc = harness.upload(case)
    try:
        dc.append()
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        v_gpu, k_gpu = dc.pools_to_host()
        assert orc.append_case(case) == 0                  # oracle applies the same append to the host copy
        assert np.array_equal(v_gpu, case.v_pool)
        assert np.array_equal(k_gpu, case.kr_pool)
    finally:
        dc.close()


def test_append_chunk_is_bit_exact():
    pc = wl.make_prefill_case("ap8", wl.SHAPE_A, [0, 63, 64, 500], [130, 2, 0, 77], page_size=64, cache_dtype="fp8", seed=812)
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
    assert np.array_equal(v, v_ref) and np.array_equal(k, k_ref)


@pytest.mark.parametrize("shape", SHAPES)
def test_fused_step_is_bitwise_the_three_calls_and_matches_the_oracle(shape):
    lens = np.array([1, 64, 65, 1001, 4096, 130], dtype=np.int32)
    mk = lambda: wl.make_case("fstep8", shape, lens, page_size=64, cache_dtype="fp8", seed=809,
                              q_pos=lens - 1, append_pos=lens - 1)
    case = mk()
    a, b = harness.upload(mk()), harness.upload(mk())
    try:
        a.absorb(); a.append(); a.decode()
        b.step()
        torch.cuda.synchronize()
        assert int(a.status.item()) == 0 and int(b.status.item()) == 0
        assert torch.equal(a.q_abs, b.q_abs)
        assert torch.equal(a.v_pool, b.v_pool) and torch.equal(a.kr_pool, b.kr_pool)
        assert torch.equal(a.out, b.out) and torch.equal(a.lse, b.lse)
        assert orc.append_case(case) == 0                      # oracle: append, then attend, with its own fp64 query
        ref_out, _ = orc.decode_case(case)
        assert np.max(np.abs(b.out.cpu().numpy().astype(np.float64) - ref_out)) <= 5e-5
    finally:
        a.close(); b.close()


def test_static_entry_point_and_host_step():
    case = wl.make_case("host8", wl.SHAPE_A, [200, 64, 1300], page_size=64, cache_dtype="fp8", seed=810,
                        q_pos=np.array([199, 63, 1299]), append_pos=np.array([199, 63, 1299]))
    dc = harness.upload(case)
    try:
        dc.step()
        torch.cuda.synchronize()
        want = dc.out.clone()
        dc.out.fill_(float("nan"))
        gb.gva_decode_static(dc.handle, dc.cache, dc.q_abs, dc.seq_lens, dc.out, dc.lse, case.B, dc.max_seq_len, 0, dc.status)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        assert torch.equal(dc.out, want)
    finally:
        dc.close()


def test_what_the_8_bit_cache_does_not_cover():
    for kw in (dict(H=16, G=4, d_v=64, d_c=64, d_r=24, page_size=64),
               dict(H=16, G=4, d_v=64, d_c=64, d_r=16, page_size=32),
               dict(H=16, G=4, d_v=64, d_c=64, d_r=16, page_size=64, kernel=gb.GVA_KERNEL_FMA)):
        with pytest.raises(gb.GvaError) as e:
            gb.gva_create(cache_dtype=gb.GVA_E4M3, **kw)
        assert e.value.status == gb.GVA_ERR_UNSUPPORTED


@pytest.mark.parametrize("shape", [wl.SHAPE_A, wl.SHAPE_B, wl.SHAPE_A0])
def test_prefill_and_decode_multi_over_the_8_bit_cache(shape):
    # the tcgen05 kernel over e4m3 tiles: the producer warp widens them to f16 in shared memory, queries (hi + lo) and
    # weights are f16; ragged chunks over contexts around tile boundaries, poisoned unused slots, flat and peaked scores
    for gain in (1.0, 6.0):
        pc = wl.make_prefill_case("pf8", shape, [0, 70, 1000, 63, 5], [130, 33, 5, 64, 300], page_size=64, cache_dtype="fp8",
                                  seed=811, poison_unused=True, q_gain=gain)
        ref_out, ref_lse = orc.prefill_case(pc)
        pd = harness.upload_prefill(pc)
        try:
            pd.absorb()
            for call in (pd.prefill, lambda: pd.decode_multi(num_splits=0), lambda: pd.decode_multi(num_splits=3)):
                pd.out.fill_(float("nan"))
                out, lse = call()
                torch.cuda.synchronize()
                assert int(pd.status.item()) == 0
                o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
                assert np.isfinite(o).all() and np.isfinite(l).all()
                assert np.max(np.abs(o - ref_out)) <= 2e-2, np.max(np.abs(o - ref_out))
                assert U().rel_l2(o, ref_out) <= 1e-2
                assert np.max(np.abs(l - ref_lse)) <= 2e-2
        finally:
            pd.close()


def test_prefill_bench_size_over_the_8_bit_cache_sampled_rows():
    # the prefill benchmark's shape (8 prompts of 8192 tokens) over e4m3 codes, same launch: sampled query rows one by one
    # against the decode oracle over the row's prefix, finiteness for the rest
    pc = wl.make_prefill_case("prefill8", wl.SHAPE_A, [0] * 8, [8192] * 8, page_size=64, cache_dtype="fp8", seed=wl.MASTER_SEED + 7100)
    c, s = pc.cache, pc.cache.shape
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        out, lse = pd.prefill()
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out.cpu().numpy().astype(np.float64)
        l = lse.cpu().numpy().astype(np.float64)
        q_abs = pd.q_abs.cpu().numpy().astype(np.float64)
    finally:
        pd.close()
    assert np.isfinite(o).all() and np.isfinite(l).all()
    T = int(pc.q_lens[0])
    rng = np.random.default_rng(9)
    for b in (0, c.B - 1):
        for t in sorted(set([0, 1, 63, 64, 65, 127, 128, 4095, 4096, T - 33, T - 1] + rng.integers(0, T, size=5).tolist())):
            n = int(pc.cu_q[b]) + t
            lens = np.zeros(c.B, dtype=np.int32); lens[b] = t + 1
            qa = np.zeros((c.B, s.H, s.d_v + s.d_r)); qa[b] = q_abs[n]
            ref_o, ref_l = orc.decode(c.v_pool, c.kr_pool, c.block_table, lens, qa, s.H, d_c=s.d_c)
            assert np.max(np.abs(o[n] - ref_o[b])) <= 2e-2, (b, t)
            assert np.max(np.abs(l[n] - ref_l[b])) <= 2e-2, (b, t)


def test_full_size_long_context_sampled():
    # bench.py's 8-bit workload (the long-context paged configuration with one byte per cache element), same launch:
    # the oracle evaluates a sample of sequences; the Gaussian-tilting statistic covers the rest
    case = wl.make_case("cfg2-fp8", wl.SHAPE_A, [32768] * 32, page_size=64, cache_dtype="fp8", paged=True,
                        seed=wl.MASTER_SEED + 2000)
    dc = harness.upload(case)
    try:
        dc.absorb()
        out, lse = dc.decode(num_splits=0)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        o = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all()
        sample = [0, 17, 31]
        lens = np.zeros_like(case.seq_lens)
        lens[sample] = case.seq_lens[sample]
        ref, _ = U().oracle_for_gpu_q(case, dc.q_abs, seq_lens=lens)
        assert np.max(np.abs(o[sample] - ref[sample])) <= U().TOL_TIGHT_MAXABS
        s = case.shape
        q = dc.q_abs.cpu().numpy().astype(np.float64)
        target = q[..., :s.d_v] / np.sqrt(s.d_c + s.d_r)
        assert np.max(np.abs(o - target)) < 0.25      # e4m3 rounding of N(0, 1) rows adds ~0.1 % variance only
    finally:
        dc.close()


def test_full_size_ragged_wide_heads_sampled():
    # bench.py's cfg3-fp8 workload (64 ragged sequences, H=32, d_v=128, one byte per cache element), same launch: the
    # shortest, a median and the longest sequence against the oracle; finiteness for the rest
    seed = wl.MASTER_SEED + 3000
    case = wl.make_case("cfg3-fp8", wl.SHAPE_B, wl.config3_seq_lens(seed), page_size=64, cache_dtype="fp8", paged=True,
                        seed=seed, poison_unused=True)
    order = np.argsort(case.seq_lens)
    sample = [int(order[0]), int(order[len(order) // 2]), int(order[-1])]
    dc = harness.upload(case)
    try:
        dc.absorb()
        out, lse = dc.decode(num_splits=0)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        o = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all()
        lens = np.zeros_like(case.seq_lens)
        lens[sample] = case.seq_lens[sample]
        ref, _ = U().oracle_for_gpu_q(case, dc.q_abs, seq_lens=lens)
        assert np.max(np.abs(o[sample] - ref[sample])) <= U().TOL_TIGHT_MAXABS
    finally:
        dc.close()


@pytest.mark.parametrize("q_len", [2, 3, 4])
@pytest.mark.parametrize("shape", [wl.SHAPE_A, wl.SHAPE_B])
@pytest.mark.parametrize("num_splits", [0, 3])
def test_decode_tokens_matches_oracle(q_len, shape, num_splits):
    # exactly q_len new tokens per sequence over contexts around tile and page boundaries (a context of 0 too: the first
    # new token then sees only itself), poisoned unused slots; the oracle is the chunked-prefill oracle over the same
    # codes.  Queries and weights enter the MMAs as single f16 values (relative 2^-12): tolerances of the 16-bit
    # multi-token kernels
    ctx = [0, 1, 61, 62, 63, 64, 65, 127, 128, 700, 2047, 5000]
    pc = wl.make_prefill_case("tok8", shape, ctx, [q_len] * len(ctx), page_size=64, cache_dtype="fp8", seed=820 + q_len,
                              poison_unused=True)
    ref_out, ref_lse = orc.prefill_case(pc)
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        out, lse = pd.decode_tokens(q_len, num_splits=num_splits)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all() and np.isfinite(l).all()
        assert np.max(np.abs(o - ref_out)) <= 5e-3, np.max(np.abs(o - ref_out))
        assert U().rel_l2(o, ref_out) <= 2e-3
        assert np.max(np.abs(l - ref_lse)) <= 5e-3
    finally:
        pd.close()


def test_decode_tokens_sharply_peaked_scores():
    # queries 30 times the unit scale: scaled scores reach +-100 and single rows dominate; the 8-bit multi-token kernel takes the
    # queries as two f16 numbers each (hi + lo), so outputs and lse stay far inside the contract
    for q_len in (2, 4):
        pc = wl.make_prefill_case("tok8p", wl.SHAPE_A, [700, 63, 2047, 0], [q_len] * 4, page_size=64, cache_dtype="fp8", seed=870 + q_len,
                                  poison_unused=True, q_gain=30.0)
        ref_out, ref_lse = orc.prefill_case(pc)
        pd = harness.upload_prefill(pc)
        try:
            pd.absorb()
            out, lse = pd.decode_tokens(q_len)
            torch.cuda.synchronize()
            assert int(pd.status.item()) == 0
            o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
            assert np.max(np.abs(o - ref_out)) <= 5e-3, np.max(np.abs(o - ref_out))
            assert np.max(np.abs(l - ref_lse)) <= 5e-3
        finally:
            pd.close()


@pytest.mark.parametrize("case_no", range(4))
def test_decode_tokens_with_a_count_per_sequence(case_no):
    # gva_decode_tokens_ragged over the 8-bit cache: every sequence its own number of new tokens (none .. four)
    rng = np.random.default_rng(8300 + case_no)
    B = int(rng.integers(1, 9))
    max_q = [4, 2, 3, 4][case_no]
    q = rng.integers(0, max_q + 1, size=B)
    q[int(rng.integers(0, B))] = max_q
    ctx = rng.integers(0, 3000, size=B)
    shape = wl.SHAPE_A if case_no != 3 else wl.SHAPE_B
    pc = wl.make_prefill_case("rag8", shape, ctx, q, page_size=64, cache_dtype="fp8", seed=8400 + case_no, poison_unused=True,
                              paged=bool(case_no % 2))
    ref_out, ref_lse = orc.prefill_case(pc)
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        pd.out.fill_(float("nan")); pd.lse.fill_(float("nan"))
        out, lse = pd.decode_tokens_ragged(num_splits=0 if case_no % 2 else 2)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out[:pc.n_q].cpu().numpy().astype(np.float64); l = lse[:pc.n_q].cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all() and np.isfinite(l).all()
        assert np.max(np.abs(o - ref_out)) <= 5e-3 and np.max(np.abs(l - ref_lse)) <= 5e-3
        assert torch.isnan(out[pc.n_q:]).all()
    finally:
        pd.close()


def test_append_then_decode_tokens_follows_algorithm_order():
    # Algorithm 1 for three new tokens at once over the 8-bit cache: absorb, append all three (bit-exact codes), attend
    q_len = 3
    pc = wl.make_prefill_case("atok8", wl.SHAPE_A, [63, 640, 0, 4095], [q_len] * 4, page_size=64, cache_dtype="fp8", seed=841)
    c = pc.cache
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        pd.append()
        out, _ = pd.decode_tokens(q_len)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        v, k = pd.dc.pools_to_host()
        assert orc.append_chunk(c.v_pool, c.kr_pool, c.block_table, pc.v_new, pc.kr_new, pc.cu_q, pc.ctx_lens) == 0
        assert np.array_equal(v, c.v_pool) and np.array_equal(k, c.kr_pool)
        ref_out, _ = orc.prefill_case(pc)
        assert np.max(np.abs(out[:pc.n_q].cpu().numpy().astype(np.float64) - ref_out)) <= 5e-3
    finally:
        pd.close()
