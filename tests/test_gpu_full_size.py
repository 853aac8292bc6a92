"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the oracle
evaluates a sample of sequences one by one; Gaussian-tilting statistics cover the rest."""
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


def _sampled_check(case, kernel, sample):
    from tests import gpu_util as U
    dc = harness.upload(case, kernel=kernel)
    try:
        dc.absorb()
        out, lse = dc.decode(num_splits=0)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        o = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all()
        lens = np.zeros_like(case.seq_lens)
        lens[sample] = case.seq_lens[sample]
        ref, ref_lse = U.oracle_for_gpu_q(case, dc.q_abs, seq_lens=lens)
        err = np.max(np.abs(o[sample] - ref[sample]))
        assert err <= U.TOL_TIGHT_MAXABS, err
        assert U.rel_l2(o[sample], ref[sample]) <= U.TOL_TIGHT_REL_L2
        # every sequence: the softmax-weighted mean of N(0, I) rows sits near q~ / sqrt(d_qk)
        s = case.shape
        q = dc.q_abs.cpu().numpy().astype(np.float64)
        target = q[..., :s.d_v] / np.sqrt(s.d_c + s.d_r)
        long_enough = np.asarray(case.seq_lens) >= 4096
        assert np.max(np.abs(o[long_enough] - target[long_enough])) < 0.2
        return gb.gva_last_num_splits(dc.handle)
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


def test_config2_long_context_paged_sampled():
    _sampled_check(wl.config2(), _auto_kernel(), [0, 17, 31])


def test_config3_ragged_wide_heads_sampled():
    case = wl.config3(poison=True)
    order = np.argsort(case.seq_lens)
    _sampled_check(case, _auto_kernel(), [int(order[0]), int(order[len(order) // 2]), int(order[-1])])


def test_config4_two_layers_full_batch():
    from oracle import gva_oracle as orc
    from tests import gpu_util as U
    for layer in (0, 23):
        case = wl.config4_layer(layer)
        dc = harness.upload(case, kernel=_auto_kernel())
        try:
            dc.absorb()
            dc.append()
            out, _ = dc.decode()
            torch.cuda.synchronize()
            assert int(dc.status.item()) == 0
            v_gpu, k_gpu = dc.pools_to_host()
            assert orc.append_case(case) == 0
            assert np.array_equal(v_gpu, case.v_pool) and np.array_equal(k_gpu, case.kr_pool)   # bit-exact append
            sample = [0, 64, 127]
            lens = np.zeros_like(case.seq_lens)
            lens[sample] = case.seq_lens[sample]
            ref, _ = orc.decode_case(case, seq_lens=lens)       # oracle's own fp64 absorbed query: end to end
            o = out.cpu().numpy().astype(np.float64)
            assert np.max(np.abs(o[sample] - ref[sample])) <= 5e-5
        finally:
            dc.close()


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
