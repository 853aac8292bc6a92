"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle on the same seeded inputs."""
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


def U():
    from tests import gpu_util
    return gpu_util


KERNELS_BF16 = [gb.GVA_KERNEL_FMA, gb.GVA_KERNEL_MMA]


def _mma_or_skip(kernel):
    if kernel == gb.GVA_KERNEL_MMA:
        try:
            h = gb.gva_create(H=16, G=4, d_v=64, d_c=64, d_r=16, page_size=64, kernel=gb.GVA_KERNEL_MMA)
            gb.gva_destroy(h)
        except gb.GvaError as e:
            if e.status == gb.GVA_ERR_UNSUPPORTED:
                pytest.skip("tensor-core kernel not built")
            raise


# ------------------------------------------------------------------ absorb
@pytest.mark.parametrize("shape,B", [(wl.SHAPE_A, 1), (wl.SHAPE_A, 19), (wl.SHAPE_B, 9), (wl.SHAPE_C, 11)])
def test_absorb_matches_oracle(shape, B):
    lens = np.arange(B) * 37 + 5
    case = wl.make_case("absorb", shape, lens, page_size=64, cache_dtype="bf16", seed=101,
                        q_pos=(np.arange(B) * 911 + 3) % 20000)
    dc = harness.upload(case)
    try:
        q = dc.absorb().cpu().numpy().astype(np.float64)
        ref = orc.absorb_case(case)
        assert np.max(np.abs(q - ref)) <= U().TOL_QABS
        # rotated slice: fp64 rotation rounded once to f32
        assert np.array_equal(q[..., shape.d_v:].astype(np.float32), ref[..., shape.d_v:].astype(np.float32))
    finally:
        dc.close()


# ------------------------------------------------------------------ append (bit exact)
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("shape", [wl.SHAPE_A, wl.SHAPE_B, wl.SHAPE_C, wl.SHAPE_A0])
def test_append_is_bit_exact_and_touches_nothing_else(dtype, shape):
    lens = [1, 64, 65, 300, 129, 4000, 8193]
    case = wl.make_case("append", shape, lens, page_size=64, cache_dtype=dtype, seed=102, extra_pages=3)
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


def test_append_contiguous_and_bad_positions():
    case = wl.make_case("append_c", wl.SHAPE_A, [100, 128, 7], page_size=64, cache_dtype="bf16", paged=False, seed=103)
    dc = harness.upload(case)
    try:
        dc.append()
        torch.cuda.synchronize()
        v_gpu, k_gpu = dc.pools_to_host()
        orc.append_case(case)
        assert np.array_equal(v_gpu, case.v_pool) and np.array_equal(k_gpu, case.kr_pool)
        # position beyond the block table: reported, nothing written
        before_v = dc.v_pool.clone()
        dc.append_pos.copy_(torch.tensor([5, 64 * case.max_pages_per_seq, 3], dtype=torch.int32))
        dc.append()
        torch.cuda.synchronize()
        st = int(dc.status.item())
        assert st & 0xFF == gb.GVA_ERR_SEQ_LEN and st >> 8 == 1
        changed = (before_v != dc.v_pool).view(case.num_pages, 4, 64, 64).any(dim=(1, 3)).nonzero().tolist()
        assert sorted(map(tuple, changed)) == [(0, 5), (2 * case.max_pages_per_seq, 3)]
    finally:
        dc.close()


def test_append_reports_bad_page():
    case = wl.make_case("append_bad", wl.SHAPE_A, [10, 10], page_size=64, cache_dtype="bf16", seed=104)
    case.block_table[1, 0] = case.num_pages + 5
    dc = harness.upload(case)
    try:
        before = dc.v_pool.clone()
        dc.append()
        torch.cuda.synchronize()
        st = int(dc.status.item())
        assert st & 0xFF == gb.GVA_ERR_BAD_PAGE and st >> 8 == 1
        p0 = int(case.block_table[0, 0])
        diff = (before != dc.v_pool).view(case.num_pages, -1).any(dim=1).nonzero().flatten().tolist()
        assert diff == [p0]
    finally:
        dc.close()


# ------------------------------------------------------------------ decode: the named small configs
def test_config0_f32_contiguous():
    err = U().check_decode(wl.config0(), gb.GVA_KERNEL_FMA)
    assert err <= 1e-5


@pytest.mark.parametrize("kernel", KERNELS_BF16)
@pytest.mark.parametrize("num_splits", [0, 1, 2, 7, 16])
def test_config1_bf16_all_split_counts(kernel, num_splits):
    _mma_or_skip(kernel)
    case = wl.config1()
    dc = harness.upload(case, kernel=kernel)
    try:
        U().check_decode(case, kernel, num_splits=num_splits, dc=dc)
        n = gb.gva_last_num_splits(dc.handle)
        assert n == (case.B * num_splits if num_splits else n) and n >= 1
        assert gb.gva_last_kernel(dc.handle) == kernel
    finally:
        dc.close()


# ------------------------------------------------------------------ decode: edge cases
EDGE_LENS = [0, 1, 31, 32, 33, 63, 64, 65, 127, 128, 129, 640, 641, 1000]


@pytest.mark.parametrize("kernel", KERNELS_BF16)
@pytest.mark.parametrize("shape", [wl.SHAPE_A, wl.SHAPE_B, wl.SHAPE_C, wl.SHAPE_A0, wl.SHAPE_B0])
@pytest.mark.parametrize("num_splits", [0, 1, 5, 40])
def test_ragged_edge_lengths_poisoned(kernel, shape, num_splits):
    # lengths around tile and page boundaries, an empty sequence, more splits than tiles;
    # every slot no live token occupies holds NaN and unused block-table entries are -1
    _mma_or_skip(kernel)
    case = wl.make_case("edge", shape, EDGE_LENS, page_size=64, cache_dtype="bf16", seed=201, poison_unused=True,
                        extra_pages=2)
    U().check_decode(case, kernel, num_splits=num_splits)


@pytest.mark.parametrize("shape", [wl.SHAPE_A, wl.SHAPE_B, wl.SHAPE_C, wl.SHAPE_A0, wl.SHAPE_B0])
@pytest.mark.parametrize("num_splits", [0, 3])
def test_ragged_edge_lengths_f32(shape, num_splits):
    case = wl.make_case("edge32", shape, EDGE_LENS, page_size=64, cache_dtype="f32", seed=202, poison_unused=True)
    U().check_decode(case, gb.GVA_KERNEL_FMA, num_splits=num_splits)


@pytest.mark.parametrize("kernel", KERNELS_BF16)
def test_single_sequence_and_page_sizes(kernel):
    _mma_or_skip(kernel)
    for P, paged in ((32, True), (128, True), (256, False), (64, False)):
        case = wl.make_case("ps", wl.SHAPE_A, [777], page_size=P, cache_dtype="bf16", paged=paged, seed=203 + P,
                            poison_unused=True)
        U().check_decode(case, kernel)


@pytest.mark.parametrize("kernel", KERNELS_BF16)
def test_peaked_and_flat_scores(kernel):
    _mma_or_skip(kernel)
    # queries x30: near one-hot rows (max subtraction); zero queries: all scores equal
    case = wl.make_case("peak", wl.SHAPE_A, [500, 2049, 64], page_size=64, cache_dtype="bf16", seed=204, q_gain=30.0)
    U().check_decode(case, kernel, tight=False)
    case = wl.make_case("flat", wl.SHAPE_A, [500, 2049, 64], page_size=64, cache_dtype="bf16", seed=205, q_gain=0.0)
    U().check_decode(case, kernel)


@pytest.mark.parametrize("kernel", KERNELS_BF16)
def test_shared_prefix_pages(kernel):
    _mma_or_skip(kernel)
    case = wl.make_case("prefix", wl.SHAPE_A, [300, 300, 200], page_size=64, cache_dtype="bf16", seed=206)
    case.block_table[1, :2] = case.block_table[0, :2]        # two sequences read the same physical prefix
    U().check_decode(case, kernel)


@pytest.mark.parametrize("kernel", KERNELS_BF16)
def test_bitwise_reproducible(kernel):
    _mma_or_skip(kernel)
    case = wl.make_case("repro", wl.SHAPE_A, [3000, 1234, 64, 5000], page_size=64, cache_dtype="bf16", seed=207)
    dc = harness.upload(case, kernel=kernel)
    try:
        dc.absorb()
        for ns in (0, 6):
            a = dc.decode(num_splits=ns)[0].clone()
            b = dc.decode(num_splits=ns)[0].clone()
            torch.cuda.synchronize()
            assert torch.equal(a, b)
    finally:
        dc.close()


@pytest.mark.parametrize("kernel", KERNELS_BF16)
def test_bad_page_and_bad_length_are_reported_not_read(kernel):
    _mma_or_skip(kernel)
    case = wl.make_case("bad", wl.SHAPE_A, [200, 200, 200], page_size=64, cache_dtype="bf16", seed=208)
    good = U().oracle_for_gpu_q
    dc = harness.upload(case, kernel=kernel)
    try:
        dc.absorb()
        bt = dc.block_table.clone()
        dc.block_table[1, 1] = -7
        dc.decode()
        torch.cuda.synchronize()
        st = int(dc.status.item())
        assert st & 0xFF == gb.GVA_ERR_BAD_PAGE and st >> 8 == 1
        ref, _ = good(case, dc.q_abs)
        o = dc.out.cpu().numpy()
        assert np.max(np.abs(o[[0, 2]] - ref[[0, 2]])) <= U().TOL_TIGHT_MAXABS      # other sequences unaffected
        assert np.isfinite(o).all()
        dc.block_table.copy_(bt)
        dc.status.zero_()
        lens = dc.seq_lens.clone()
        lens[2] = case.max_pages_per_seq * 64 + 1
        dc.decode(seq_lens=lens)
        torch.cuda.synchronize()
        st = int(dc.status.item())
        assert st & 0xFF == gb.GVA_ERR_SEQ_LEN and st >> 8 == 2
        o = dc.out.cpu().numpy()
        assert np.all(o[2] == 0) and np.max(np.abs(o[:2] - ref[:2])) <= U().TOL_TIGHT_MAXABS
    finally:
        dc.close()


def test_host_side_argument_errors():
    case = wl.make_case("args", wl.SHAPE_A, [100], page_size=64, cache_dtype="bf16", seed=209)
    dc = harness.upload(case)
    try:
        dc.absorb()
        ws = dc.ensure_workspace(0)
        rc = gb.gva_decode(dc.handle, dc.cache, dc.q_abs, dc.seq_lens, dc.out, dc.lse, ws, 1, 100, 0, dc.status,
                           workspace_bytes=128, check=False)
        assert rc == gb.GVA_ERR_WORKSPACE
        rc = gb.gva_decode(dc.handle, dc.cache, None, dc.seq_lens, dc.out, dc.lse, ws, 1, 100, 0, dc.status, check=False)
        assert rc == gb.GVA_ERR_INVALID_ARG
        rc = gb.gva_decode(dc.handle, dc.cache, dc.q_abs, dc.seq_lens, dc.out, dc.lse, ws, 1, 100, -1, dc.status, check=False)
        assert rc == gb.GVA_ERR_INVALID_ARG
        assert gb.gva_decode_workspace_bytes(dc.handle, 1, 100, 0) > 0
        assert gb.gva_decode_workspace_bytes(dc.handle, 4, 100, 8) >= 4 * 8 * 16 * 66 * 4
        # lse is optional
        gb.gva_decode(dc.handle, dc.cache, dc.q_abs, dc.seq_lens, dc.out, None, ws, 1, 100, 0, dc.status)
        torch.cuda.synchronize()
    finally:
        dc.close()


# ------------------------------------------------------------------ end to end: absorb -> append -> decode
@pytest.mark.parametrize("kernel", KERNELS_BF16)
def test_full_step_follows_algorithm_order(kernel):
    _mma_or_skip(kernel)
    T = 1000
    lens = np.full(6, T + 1, dtype=np.int32)
    case = wl.make_case("step", wl.SHAPE_A, lens, page_size=64, cache_dtype="bf16", seed=210,
                        q_pos=np.full(6, T), append_pos=np.full(6, T))
    dc = harness.upload(case, kernel=kernel)
    try:
        dc.absorb()
        dc.append()
        out, lse = dc.decode()
        torch.cuda.synchronize()
        assert orc.append_case(case) == 0                      # oracle: append, then attend over T+1 tokens
        ref_out, ref_lse = orc.decode_case(case)               # with its own fp64 absorbed query
        o = out.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(o - ref_out)) <= 5e-5
    finally:
        dc.close()


# ------------------------------------------------------------------ fused step entry point
@pytest.mark.parametrize("kernel", KERNELS_BF16)
@pytest.mark.parametrize("shape", [wl.SHAPE_A, wl.SHAPE_B, wl.SHAPE_C, wl.SHAPE_A0])
def test_fused_step_is_bitwise_the_three_calls(kernel, shape):
    _mma_or_skip(kernel)
    lens = np.array([1, 64, 65, 1001, 4096, 130], dtype=np.int32)
    mk = lambda: wl.make_case("fstep", shape, lens, page_size=64, cache_dtype="bf16", seed=211,
                              q_pos=lens - 1, append_pos=lens - 1)
    a, b = harness.upload(mk(), kernel=kernel), harness.upload(mk(), kernel=kernel)
    try:
        a.absorb(); a.append(); a.decode()
        b.step()
        torch.cuda.synchronize()
        assert int(a.status.item()) == 0 and int(b.status.item()) == 0
        assert torch.equal(a.q_abs, b.q_abs)
        assert torch.equal(a.v_pool, b.v_pool) and torch.equal(a.kr_pool, b.kr_pool)
        assert torch.equal(a.out, b.out) and torch.equal(a.lse, b.lse)
    finally:
        a.close(); b.close()


@pytest.mark.parametrize("shape,dtype", [(wl.SHAPE_A, "bf16"), (wl.SHAPE_B, "bf16"), (wl.SHAPE_C, "bf16"), (wl.SHAPE_A, "fp8")])
def test_fused_step_of_a_large_batch_is_bitwise_the_three_calls(shape, dtype):
    # Batches whose front grid would exceed one block per SM take the folded front kernel (appends inside the absorb
    # blocks, 16 sequences per absorb item for the 64-wide shape): same bits as the three separate calls.
    rng = np.random.default_rng(77)
    lens = rng.integers(1, 400, size=300).astype(np.int32)
    mk = lambda: wl.make_case("fstep-big", shape, lens, page_size=64, cache_dtype=dtype, seed=212,
                              q_pos=lens - 1, append_pos=lens - 1)
    a, b = harness.upload(mk()), harness.upload(mk())
    try:
        a.absorb(); a.append(); a.decode()
        b.step()
        torch.cuda.synchronize()
        assert int(a.status.item()) == 0 and int(b.status.item()) == 0
        assert torch.equal(a.q_abs, b.q_abs)
        assert torch.equal(a.v_pool, b.v_pool) and torch.equal(a.kr_pool, b.kr_pool)
        assert torch.equal(a.out, b.out) and torch.equal(a.lse, b.lse)
    finally:
        a.close(); b.close()


@pytest.mark.parametrize("kernel", KERNELS_BF16)
def test_fused_steps_back_to_back_generate_tokens(kernel):
    # 24 decode steps in a row with no host synchronisation in between: every step appends one token that the
    # same step's query must already see (the decode kernel starts early, behind the fused front kernel)
    _mma_or_skip(kernel)
    T0, n_steps, B = 120, 24, 5
    lens0 = np.array([T0, T0 + 7, 63, 64, 1], dtype=np.int32)
    case = wl.make_case("gen", wl.SHAPE_A, lens0 + n_steps, page_size=64, cache_dtype="bf16", seed=212)
    rng = np.random.default_rng(5)
    v_steps = rng.standard_normal((n_steps, B, 4, 64)).astype(np.float32) * 3.0
    k_steps = rng.standard_normal((n_steps, B, 16)).astype(np.float32)
    qc_steps = rng.standard_normal((n_steps, B, 16, 64)).astype(np.float32)
    dc = harness.upload(case, kernel=kernel)
    try:
        dv, dk, dq = (torch.from_numpy(x).cuda() for x in (v_steps, k_steps, qc_steps))
        outs = []
        for s in range(n_steps):
            pos = torch.from_numpy(lens0 + s).cuda()
            dc.append_pos.copy_(pos); dc.q_pos.copy_(pos); dc.seq_lens.copy_(pos + 1)
            dc.v_new.copy_(dv[s]); dc.kr_new.copy_(dk[s]); dc.q_c.copy_(dq[s])
            ws = dc.ensure_workspace(0)
            gb.gva_decode_step(dc.handle, dc.cache, dc.M, dc.q_c, dc.q_r, dc.v_new, dc.kr_new, dc.append_pos, dc.seq_lens,
                               dc.q_abs, dc.out, dc.lse, ws, B, int(lens0.max()) + n_steps, 0, dc.status)
            outs.append(dc.out.clone())
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        for s in range(n_steps):                                   # oracle replays the same generation
            pos = (lens0 + s).astype(np.int32)
            case.append_pos[:] = pos; case.q_pos[:] = pos
            case.v_new[:] = v_steps[s]; case.kr_new[:] = k_steps[s]; case.q_c[:] = qc_steps[s]
            assert orc.append_case(case) == 0
            ref, _ = orc.decode_case(case, seq_lens=pos + 1)
            # end to end against the oracle's own fp64 absorbed query; rows here reach |v| ~ 10
            assert np.max(np.abs(outs[s].cpu().numpy() - ref)) <= 2e-5 * max(1.0, float(np.max(np.abs(ref)))), s
        v_gpu, k_gpu = dc.pools_to_host()
        assert np.array_equal(v_gpu, case.v_pool) and np.array_equal(k_gpu, case.kr_pool)
    finally:
        dc.close()


@pytest.mark.parametrize("pinned", [True, False])
def test_host_buffer_step_matches_device_step(pinned):
    # gva_decode_step_host with pinned buffers (read and written in place by the kernels) and with pageable
    # buffers (staged copies) must both equal the device-buffer step
    lens = np.array([700, 64, 1, 2049], dtype=np.int32)
    mk = lambda: wl.make_case("hstep", wl.SHAPE_A, lens, page_size=64, cache_dtype="bf16", seed=213,
                              q_pos=lens - 1, append_pos=lens - 1)
    a, b = harness.upload(mk()), harness.upload(mk())
    try:
        a.step()
        case = b.case
        mkh = (lambda x: torch.from_numpy(np.ascontiguousarray(x)).pin_memory()) if pinned else \
            (lambda x: torch.from_numpy(np.ascontiguousarray(x)))
        h = [mkh(x) for x in (case.q_c, case.q_r, case.v_new, case.kr_new, case.append_pos, case.seq_lens)]
        out_h = torch.full((case.B, 16, 64), float("nan"))
        if pinned:
            out_h = out_h.pin_memory()
        scratch = torch.empty(gb.gva_step_scratch_bytes(b.handle, case.B, int(lens.max()), 0), dtype=torch.uint8,
                              device="cuda")
        for _ in range(2):
            gb.gva_decode_step_host(b.handle, b.cache, b.M, h[0], h[1], h[2], h[3], h[4], h[5], out_h, scratch, case.B,
                                    int(lens.max()), 0, b.status)
            torch.cuda.synchronize()
        assert int(b.status.item()) == 0
        assert torch.equal(out_h, a.out.cpu())
        assert torch.equal(a.v_pool, b.v_pool) and torch.equal(a.kr_pool, b.kr_pool)
        # the same call with its arguments marshalled once
        call = gb.prepare_decode_step_host(b.handle, b.cache, b.M, h[0], h[1], h[2], h[3], h[4], h[5], out_h, scratch, case.B,
                                           int(lens.max()), 0, b.status)
        out_h.fill_(float("nan"))
        for _ in range(2):
            assert call() == 0
            torch.cuda.synchronize()
        assert int(b.status.item()) == 0
        assert torch.equal(out_h, a.out.cpu())
    finally:
        a.close(); b.close()


def test_prepared_calls_equal_direct_calls():
    # binding.prepare_call marshals the arguments once; the enqueued work is the same call
    lens = np.array([700, 64, 1, 2049, 0], dtype=np.int32)
    pos = np.maximum(lens - 1, 0)
    mk = lambda: wl.make_case("prep", wl.SHAPE_A, lens, page_size=64, cache_dtype="bf16", seed=219, q_pos=pos, append_pos=pos)
    a, b = harness.upload(mk()), harness.upload(mk())
    try:
        B, L = a.case.B, int(lens.max())
        a.absorb(); a.decode()
        ws = b.ensure_workspace(0)
        nbytes = ws.numel() * ws.element_size()
        absorb = gb.prepare_call("gva_absorb_query", b.handle, b.q_c, b.q_r, b.M, b.q_pos, b.q_abs, B)
        decode = gb.prepare_call("gva_decode", b.handle, b.cache, b.q_abs, b.seq_lens, b.out, b.lse, ws, nbytes, B, L, 0, b.status)
        for _ in range(2):
            assert absorb() == 0 and decode() == 0
        torch.cuda.synchronize()
        assert int(b.status.item()) == 0
        assert torch.equal(a.out, b.out) and torch.equal(a.lse, b.lse) and torch.equal(a.q_abs, b.q_abs)
        with pytest.raises(TypeError):
            gb.prepare_call("gva_decode", b.handle, b.cache)
        bad = gb.prepare_call("gva_decode", b.handle, b.cache, b.q_abs, b.seq_lens, b.out, b.lse, ws, 16, B, L, 0, b.status)
        with pytest.raises(gb.GvaError):
            bad()                                  # a workspace of 16 bytes: the status comes back as it does from a direct call
    finally:
        a.close(); b.close()


@pytest.mark.parametrize("kernel", KERNELS_BF16)
def test_odd_page_size_many_short_sequences_and_one_long(kernel):
    _mma_or_skip(kernel)
    # 96-token pages (a multiple of 32 but not of 64), 300 short ragged sequences, and one sequence long
    # enough that every block of the grid holds a piece of it
    rng = np.random.default_rng(9)
    case = wl.make_case("p96", wl.SHAPE_A, rng.integers(0, 200, size=300), page_size=96, cache_dtype="bf16", seed=214,
                        poison_unused=True)
    U().check_decode(case, kernel)
    case = wl.make_case("long1", wl.SHAPE_A, [150_001], page_size=64, cache_dtype="bf16", seed=215, poison_unused=True)
    U().check_decode(case, kernel)
    case = wl.make_case("long1b", wl.SHAPE_B, [70_003, 5], page_size=64, cache_dtype="bf16", seed=216, poison_unused=True)
    U().check_decode(case, kernel)


@pytest.mark.parametrize("kernel", KERNELS_BF16)
def test_workspace_and_outputs_stay_inside_their_bounds(kernel):
    # guard bands around the workspace, the outputs and the absorbed queries must survive every kind of call
    _mma_or_skip(kernel)
    lens = np.array([5000, 64, 0, 1, 777], dtype=np.int32)
    case = wl.make_case("canary", wl.SHAPE_A, lens, page_size=64, cache_dtype="bf16", seed=217,
                        q_pos=np.maximum(lens - 1, 0), append_pos=np.maximum(lens - 1, 0))
    dc = harness.upload(case, kernel=kernel)
    try:
        B, guard = case.B, 4096
        def banded(nbytes):
            buf = torch.full((nbytes + 2 * guard,), 0x5A, dtype=torch.uint8, device="cuda")
            return buf, buf[guard:guard + nbytes]
        checks = []
        for ns in (0, 3):
            need = gb.gva_decode_workspace_bytes(dc.handle, B, int(lens.max()), ns)
            ws_full, ws = banded(need)
            out_full, out_b = banded(B * 16 * 64 * 4)
            lse_full, lse_b = banded(B * 16 * 4)
            qa_full, qa_b = banded(B * 16 * 80 * 4)
            out, lse, q_abs = out_b.view(torch.float32), lse_b.view(torch.float32), qa_b.view(torch.float32)
            gb.gva_absorb_query(dc.handle, dc.q_c, dc.q_r, dc.M, dc.q_pos, q_abs, B)
            gb.gva_decode(dc.handle, dc.cache, q_abs, dc.seq_lens, out, lse, ws, B, int(lens.max()), ns, dc.status,
                          workspace_bytes=need)
            gb.gva_decode_step(dc.handle, dc.cache, dc.M, dc.q_c, dc.q_r, dc.v_new, dc.kr_new, dc.append_pos, dc.seq_lens,
                               q_abs, out, lse, ws, B, int(lens.max()), ns, dc.status)
            torch.cuda.synchronize()
            for full, n in ((ws_full, need), (out_full, out.numel() * 4), (lse_full, lse.numel() * 4),
                            (qa_full, q_abs.numel() * 4)):
                checks.append(bool((full[:guard] == 0x5A).all()) and bool((full[guard + n:] == 0x5A).all()))
            assert torch.isfinite(out).all()
        assert all(checks)
        assert int(dc.status.item()) == 0
    finally:
        dc.close()


def test_value_only_cache_long_context():
    # the cache without a positional slice (Section 3.4): a paged long-context case on both kernels
    case = wl.make_case("vo-long", wl.SHAPE_A0, [20000, 8191, 4097, 333], page_size=64, cache_dtype="bf16", seed=231)
    for kernel in KERNELS_BF16:
        _mma_or_skip(kernel)
        U().check_decode(case, kernel)


def test_two_handles_take_turns_on_one_workspace():
    # The merge kernel may pick up the workspace header before the decode kernel has finished, recognising it by a stamp
    # of (handle, call number).  Two handles whose call numbers run in lockstep share one workspace here, with batches
    # whose sequences split into different runs of records: a header left by the other handle must never be taken.
    _mma_or_skip(gb.GVA_KERNEL_MMA)
    a = wl.make_case("turn-a", wl.SHAPE_A, [9000, 300, 5000, 64, 12000, 1], page_size=64, cache_dtype="bf16", seed=241)
    b = wl.make_case("turn-b", wl.SHAPE_A, [128, 15000, 2, 7000, 900, 4000], page_size=64, cache_dtype="bf16", seed=242)
    da, db = harness.upload(a, kernel=gb.GVA_KERNEL_MMA), harness.upload(b, kernel=gb.GVA_KERNEL_MMA)
    try:
        ws = da.ensure_workspace(0)
        if db.ensure_workspace(0).numel() > ws.numel():
            ws = db.workspace
        da.workspace = db.workspace = ws
        da.absorb()
        db.absorb()
        torch.cuda.synchronize()
        ref = {id(da): U().oracle_for_gpu_q(a, da.q_abs)[0], id(db): U().oracle_for_gpu_q(b, db.q_abs)[0]}
        outs = []
        for turn in range(8):                       # back to back, no synchronisation in between
            for d in (da, db):
                d.decode()
                outs.append((d, d.out.clone()))
        torch.cuda.synchronize()
        assert int(da.status.item()) == 0 and int(db.status.item()) == 0
        for d, o in outs:
            assert np.max(np.abs(o.cpu().numpy().astype(np.float64) - ref[id(d)])) <= U().TOL_TIGHT_MAXABS
    finally:
        da.close()
        db.close()


def test_one_captured_decode_call_replayed_with_changing_lengths():
    # A single gva_decode call captured in a CUDA graph and replayed: every replay carries the same call number, so
    # nothing in the device-side scheduling state (tail tickets, the workspace header's stamp) may depend on the number
    # changing from call to call.  The lengths change between replays (in place, on the device), so that the runs of
    # records per sequence differ from one replay to the next.
    _mma_or_skip(gb.GVA_KERNEL_MMA)
    # (long enough for the balanced partition to hand out tail units dynamically: at least eight tiles per thread block)
    lens0 = np.array([32768, 30000, 31000, 29000, 32000, 28000, 32768, 30001], dtype=np.int32)
    case = wl.make_case("graph", wl.SHAPE_A, lens0, page_size=64, cache_dtype="bf16", seed=251)
    dc = harness.upload(case, kernel=gb.GVA_KERNEL_MMA)
    try:
        dc.absorb()
        ws = dc.ensure_workspace(0)
        L = int(lens0.max())
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):              # (the binding launches on torch's current stream)
            dc.decode()                            # warm-up outside the capture: attributes, tensor maps, sync region
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            gb.gva_decode(dc.handle, dc.cache, dc.q_abs, dc.seq_lens, dc.out, dc.lse, ws, case.B, L, 0, dc.status)
        torch.cuda.synchronize()
        for lens in (lens0, lens0 - np.array([977, 0, 5000, 8999, 1, 699, 64, 12345], dtype=np.int32), lens0 - 7000, lens0):
            dc.seq_lens.copy_(torch.from_numpy(lens.astype(np.int32)))
            dc.out.fill_(float("nan"))
            torch.cuda.synchronize()
            g.replay()
            g.replay()                              # twice back to back: the second finds what the first left behind
            torch.cuda.synchronize()
            assert int(dc.status.item()) == 0
            ref, _ = U().oracle_for_gpu_q(case, dc.q_abs, seq_lens=lens.astype(np.int32))
            o = dc.out.cpu().numpy().astype(np.float64)
            assert np.max(np.abs(o - ref)) <= U().TOL_TIGHT_MAXABS, lens
    finally:
        dc.close()


def test_one_captured_fused_step_replayed():
    # the same for gva_decode_step: a step is idempotent when it is replayed with the same inputs (the appended row is written
    # again with the same values), so three replays must leave exactly what one direct call leaves
    _mma_or_skip(gb.GVA_KERNEL_MMA)
    lens = np.array([32768, 30000, 31000, 29000, 32000, 28000, 32768, 30001], dtype=np.int32)
    mk = lambda: wl.make_case("graph-step", wl.SHAPE_A, lens, page_size=64, cache_dtype="bf16", seed=252,
                              q_pos=lens - 1, append_pos=lens - 1)
    a, b = harness.upload(mk(), kernel=gb.GVA_KERNEL_MMA), harness.upload(mk(), kernel=gb.GVA_KERNEL_MMA)
    try:
        a.step()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            b.step()                                # warm-up outside the capture
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            b.step()
        b.out.fill_(float("nan"))
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        assert int(a.status.item()) == 0 and int(b.status.item()) == 0
        assert torch.equal(a.out, b.out) and torch.equal(a.lse, b.lse)
        assert torch.equal(a.v_pool, b.v_pool) and torch.equal(a.kr_pool, b.kr_pool)
    finally:
        a.close(); b.close()
