"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.  The decode workloads are
compared with the oracle on every sequence of the batch (and, for the 24-layer workload, on every layer), through the
three separate calls and through the fused step; the prefill and multi-token workloads on sampled rows."""
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


def _whole_batch_check(case, kernel):
    """absorb -> decode and the fused step on every sequence of the batch, against the oracle fed the GPU's own
    absorbed queries (tight gates), plus the Gaussian-tilting statistic on the long sequences."""
    from tests import gpu_util as U
    dc = harness.upload(case, kernel=kernel)
    try:
        dc.absorb()
        out, lse = dc.decode(num_splits=0)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        o = out.cpu().numpy().astype(np.float64)
        l = lse.cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all()
        ref, ref_lse = U.oracle_for_gpu_q(case, dc.q_abs)
        err = np.max(np.abs(o - ref))
        assert err <= U.TOL_TIGHT_MAXABS, err
        assert U.rel_l2(o, ref) <= U.TOL_TIGHT_REL_L2
        assert np.max(np.abs(l - ref_lse)) <= 1e-4 * max(1.0, np.max(np.abs(ref_lse)))
        # every sequence: the softmax-weighted mean of N(0, I) rows sits near q~ / sqrt(d_qk)
        s = case.shape
        q = dc.q_abs.cpu().numpy().astype(np.float64)
        target = q[..., :s.d_v] / np.sqrt(s.d_c + s.d_r)
        long_enough = np.asarray(case.seq_lens) >= 4096
        assert np.max(np.abs(o[long_enough] - target[long_enough])) < 0.2
        n_blocks = gb.gva_last_num_splits(dc.handle)
        # the call bench.py times: the fused step (append position = last attended token; the appended row differs
        # from the generated one, so the oracle appends too before it attends)
        from oracle import gva_oracle as orc
        out1 = out.clone()
        out2, _ = dc.step()
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        v_gpu, k_gpu = dc.pools_to_host()
        assert orc.append_case(case) == 0
        assert np.array_equal(v_gpu, case.v_pool) and np.array_equal(k_gpu, case.kr_pool)       # bit-exact append, whole pool
        ref2, _ = U.oracle_for_gpu_q(case, dc.q_abs)
        o2 = out2.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(o2 - ref2)) <= U.TOL_TIGHT_MAXABS
        assert not torch.equal(out1, out2)                  # (the step really attended the newly appended rows)
        return n_blocks
    finally:
        dc.close()


def _mma_built():
    try:
        h = gb.gva_create(H=16, G=4, d_v=64, d_c=64, d_r=16, page_size=64, kernel=gb.GVA_KERNEL_MMA)
        gb.gva_destroy(h)
        return True
    except gb.GvaError:
        return False


def _auto_kernel():
    return gb.GVA_KERNEL_AUTO


def test_config2_long_context_paged_whole_batch():
    case = wl.config2()
    case.append_pos[:] = case.seq_lens - 1          # the step appends at the last attended position (Algorithm 1's order)
    case.q_pos[:] = case.seq_lens - 1
    _whole_batch_check(case, _auto_kernel())


def test_config3_ragged_wide_heads_whole_batch():
    case = wl.config3(poison=True)
    case.append_pos[:] = case.seq_lens - 1
    case.q_pos[:] = case.seq_lens - 1
    _whole_batch_check(case, _auto_kernel())


def test_config4_every_layer_whole_batch():
    # the 24-layer step, one layer on the host at a time: bit-exact append on every layer (whole pool), every
    # sequence's output against the oracle end to end (the oracle's own fp64 absorbed query), first through the three
    # separate calls, then through the fused step, whose outputs must equal the three calls' bit for bit
    from oracle import gva_oracle as orc
    for layer in range(wl.CONFIG4_LAYERS):
        case = wl.config4_layer(layer)
        dc = harness.upload(case, kernel=_auto_kernel())
        try:
            dc.absorb()
            dc.append()
            out, lse = dc.decode()
            torch.cuda.synchronize()
            assert int(dc.status.item()) == 0, layer
            v_gpu, k_gpu = dc.pools_to_host()
            assert orc.append_case(case) == 0
            assert np.array_equal(v_gpu, case.v_pool) and np.array_equal(k_gpu, case.kr_pool), layer   # bit-exact append
            ref, ref_lse = orc.decode_case(case)                # oracle's own fp64 absorbed query: end to end
            o = out.cpu().numpy().astype(np.float64)
            assert np.max(np.abs(o - ref)) <= 5e-5, layer
            assert np.max(np.abs(lse.cpu().numpy().astype(np.float64) - ref_lse)) <= 1e-4 * max(1.0, np.max(np.abs(ref_lse))), layer
            q1, o1, l1 = dc.q_abs.clone(), out.clone(), lse.clone()
            dc.q_abs.fill_(float("nan")); dc.out.fill_(float("nan")); dc.lse.fill_(float("nan"))
            out2, lse2 = dc.step()                              # appends the same rows again: the pools must not change
            torch.cuda.synchronize()
            assert int(dc.status.item()) == 0, layer
            assert torch.equal(dc.q_abs, q1) and torch.equal(out2, o1) and torch.equal(lse2, l1), layer
            v2, k2 = dc.pools_to_host()
            assert np.array_equal(v2, case.v_pool) and np.array_equal(k2, case.kr_pool), layer
        finally:
            dc.close()
        del case


@pytest.mark.parametrize("shape_name", ["A", "B"])
def test_prefill_bench_size_sampled_rows(shape_name):
    # bench.py's prefill workload, same launch: a sample of query rows (first / last rows, tile and block edges, random
    # ones) is checked one by one against the decode oracle over the row's prefix (a prefill row IS one decode step over
    # its prefix -- pinned in the CPU tests); every other row is covered by finiteness and the Gaussian-tilting statistic
    from oracle import gva_oracle as orc
    pc = wl.prefill_bench_case() if shape_name == "A" else wl.prefill_bench_case_b()
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
    rng = np.random.default_rng(7)
    for b in (0, c.B - 1):
        toks = sorted(set([0, 1, 31, 32, 63, 64, 65, 127, 128, 4095, 4096, T - 33, T - 32, T - 2, T - 1] +
                          rng.integers(0, T, size=6).tolist()))
        for t in toks:
            n = int(pc.cu_q[b]) + t
            lens = np.zeros(c.B, dtype=np.int32); lens[b] = t + 1
            qa = np.zeros((c.B, s.H, s.d_v + s.d_r)); qa[b] = q_abs[n]
            ref_o, ref_l = orc.decode(c.v_pool, c.kr_pool, c.block_table, lens, qa, s.H, d_c=s.d_c)
            assert np.max(np.abs(o[n] - ref_o[b])) <= 2e-2, (b, t)
            assert np.max(np.abs(l[n] - ref_l[b])) <= 2e-2, (b, t)
    # rows with a long prefix: the softmax-weighted mean of N(0, I) rows sits near q~ / sqrt(d_qk)
    target = q_abs[..., :s.d_v] / np.sqrt(s.d_c + s.d_r)
    # (tens of millions of components here, so the bound is on a high quantile and the maximum only has to stay sane)
    far = pc.q_pos >= 4096
    dev = np.abs(o[far] - target[far])
    assert np.quantile(dev, 0.9999) < 0.2 and dev.max() < 1.0


def test_decode_multi_bench_size_sampled_rows():
    # bench.py's multi-token decode workload (cfg2 shapes, 4 new tokens per sequence over 32764 cached), same launch:
    # every new token of a sample of sequences against the decode oracle over its prefix; finiteness for the rest
    from oracle import gva_oracle as orc
    B, T, q_len = 32, 32768, 4
    pc = wl.make_prefill_case("multi", wl.SHAPE_A, [T - q_len] * B, [q_len] * B, page_size=64, seed=wl.MASTER_SEED + 7300)
    c, s = pc.cache, pc.cache.shape
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        out, lse = pd.decode_multi(num_splits=0)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out.cpu().numpy().astype(np.float64)
        l = lse.cpu().numpy().astype(np.float64)
        q_abs = pd.q_abs.cpu().numpy().astype(np.float64)
    finally:
        pd.close()
    assert np.isfinite(o).all() and np.isfinite(l).all()
    for b in (0, 13, B - 1):
        for i in range(q_len):
            n = int(pc.cu_q[b]) + i
            lens = np.zeros(c.B, dtype=np.int32); lens[b] = T - q_len + i + 1
            qa = np.zeros((c.B, s.H, s.d_v + s.d_r)); qa[b] = q_abs[n]
            ref_o, ref_l = orc.decode(c.v_pool, c.kr_pool, c.block_table, lens, qa, s.H, d_c=s.d_c)
            assert np.max(np.abs(o[n] - ref_o[b])) <= 2e-2, (b, i)
            assert np.max(np.abs(l[n] - ref_l[b])) <= 2e-2, (b, i)


@pytest.mark.parametrize("q_len", [2, 4])
def test_decode_tokens_bench_size_sampled_rows(q_len):
    # bench.py's gva_decode_tokens workload (cfg2 shapes), same launch: every new token of a sample of sequences against
    # the decode oracle over its prefix; finiteness for the rest
    from oracle import gva_oracle as orc
    B, T = 32, 32768
    pc = wl.make_prefill_case("multi", wl.SHAPE_A, [T - q_len] * B, [q_len] * B, page_size=64, seed=wl.MASTER_SEED + 7300)
    c, s = pc.cache, pc.cache.shape
    pd = harness.upload_prefill(pc)
    try:
        pd.absorb()
        out, lse = pd.decode_tokens(q_len)
        torch.cuda.synchronize()
        assert int(pd.status.item()) == 0
        o = out.cpu().numpy().astype(np.float64)
        l = lse.cpu().numpy().astype(np.float64)
        q_abs = pd.q_abs.cpu().numpy().astype(np.float64)
    finally:
        pd.close()
    assert np.isfinite(o).all() and np.isfinite(l).all()
    for b in (0, 17, B - 1):
        for i in range(q_len):
            n = int(pc.cu_q[b]) + i
            lens = np.zeros(c.B, dtype=np.int32); lens[b] = T - q_len + i + 1
            qa = np.zeros((c.B, s.H, s.d_v + s.d_r)); qa[b] = q_abs[n]
            ref_o, ref_l = orc.decode(c.v_pool, c.kr_pool, c.block_table, lens, qa, s.H, d_c=s.d_c)
            assert np.max(np.abs(o[n] - ref_o[b])) <= 2e-2, (b, i)
            assert np.max(np.abs(l[n] - ref_l[b])) <= 2e-2, (b, i)
