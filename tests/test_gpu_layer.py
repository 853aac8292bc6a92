"""The projections around the attention (input projection with folded maps + fused append, output projection,
whole layer step) against the fp64 oracle."""
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


def _setup(shape, lens, d_model, dtype="bf16", seed=501):
    lens = np.asarray(lens, dtype=np.int32)
    case = wl.make_case("layer", shape, lens, page_size=64, cache_dtype=dtype, seed=seed, q_pos=lens - 1,
                        append_pos=lens - 1)
    lw = wl.layer_weights(shape, d_model, case.B, seed=seed + 1)
    dc = harness.upload(case)
    W_in = gb.gva_pack_input_weights(dc.handle, lw["W_q_nope"], lw["W_q_rope"], lw["W_v"], lw["W_r"], case.M, d_model)
    W_o = gb.gva_pack_bf16(lw["W_o"])
    return case, lw, dc, W_in, W_o


def _dev16(a):
    return torch.from_numpy(a.view(np.int16)).cuda()


@pytest.mark.parametrize("shape", [wl.SHAPE_A, wl.SHAPE_B, wl.SHAPE_C, wl.SHAPE_A0])
def test_packed_weights_are_the_fp64_fold_rounded_once(shape):
    case, lw, dc, W_in, W_o = _setup(shape, [5, 70], d_model=64)
    try:
        ref = orc.pack_input_weights(lw["W_q_nope"], lw["W_q_rope"], lw["W_v"], lw["W_r"], case.M)
        assert W_in.shape == ref.shape == (64, gb.gva_input_width(dc.handle))
        assert np.array_equal(W_in, orc.bf16_round(ref))
        assert np.array_equal(W_o, orc.bf16_round(lw["W_o"]))
    finally:
        dc.close()


@pytest.mark.parametrize("shape,B", [(wl.SHAPE_A, 3), (wl.SHAPE_A, 37), (wl.SHAPE_B, 20), (wl.SHAPE_C, 130), (wl.SHAPE_A0, 37),
                                     (wl.SHAPE_B0, 5)])
@pytest.mark.parametrize("dtype", ["bf16", "f32", "fp8"])
def test_project_in_queries_and_append(shape, B, dtype):
    if dtype == "fp8" and shape.d_r not in (16, 32):
        pytest.skip("the 8-bit cache is built for the caches with a 16- or 32-wide positional slice")
    rng = np.random.default_rng(B)
    lens = rng.integers(1, 600, size=B)
    d_model = 256
    case, lw, dc, W_in, W_o = _setup(shape, lens, d_model, dtype)
    try:
        x = torch.from_numpy(lw["x"]).cuda()
        v0, k0 = dc.pools_to_host()
        v0, k0 = v0.copy(), k0.copy()
        gb.gva_project_in(dc.handle, dc.cache, x, _dev16(W_in), d_model, dc.append_pos, dc.q_abs, B, dc.status)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        Wd = wl.bf16_bits_to_f32(W_in).astype(np.float64)           # the weights the GPU sees
        q_t, q_r, v_new, kr_new = orc.project_in(lw["x"], Wd, shape.H, shape.G, shape.d_v, shape.d_r)
        q_ref = np.concatenate([q_t, np.stack([orc.rope(q_r[b], int(case.append_pos[b])) for b in range(B)])], axis=2)
        q = dc.q_abs.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(q - q_ref)) <= 1e-5 * max(1.0, np.max(np.abs(q_ref)))
        # append: exactly the new rows change; their values are the oracle's within one rounding of the cache type
        v1, k1 = dc.pools_to_host()
        P = case.page_size
        touched_v = np.zeros(v1.shape[:3], dtype=bool); touched_k = np.zeros(k1.shape[:2], dtype=bool)
        to64 = wl.pool_to_f64
        ulp = {"bf16": 2.0 ** -8, "f32": 2.0 ** -23, "fp8": 2.0 ** -4}[dtype]      # half a unit in the last place, relative
        tiny = 2.0 ** -10 if dtype == "fp8" else 0.0                                # ... and below the smallest normal, absolute
        for b in range(B):
            t = int(case.append_pos[b]); page, slot = case.page_of(b, t // P), t % P
            touched_v[page, :, slot] = True; touched_k[page, slot] = True
            got_v = to64(v1[page, :, slot]); ref_v = v_new[b]
            # one rounding to the cache type of an f32-accumulated product (error ~1e-6 for unit-scale values)
            assert np.all(np.abs(got_v - ref_v) <= np.abs(ref_v) * ulp + tiny + 1e-5)
            got_k = to64(k1[page, slot]); ref_k = orc.rope(kr_new[b], t)
            assert np.all(np.abs(got_k - ref_k) <= np.abs(ref_k) * ulp + tiny + 1e-5)
        assert np.array_equal(v1[~touched_v], v0[~touched_v]) and np.array_equal(k1[~touched_k], k0[~touched_k])
    finally:
        dc.close()


@pytest.mark.parametrize("shape,B,dtype", [(wl.SHAPE_A, 37, "bf16"), (wl.SHAPE_B, 9, "bf16"), (wl.SHAPE_C, 130, "bf16"),
                                           (wl.SHAPE_A, 37, "fp8"), (wl.SHAPE_B, 9, "fp8")])
def test_project_in_appends_the_rows_gva_append_cache_would_write(shape, B, dtype):
    # The fused append rounds its f32 products exactly as gva_append_cache rounds f32 inputs.  The products themselves are read
    # back from an f32 cache written at position 0 (a rotation by the identity, stored without rounding); appending them with
    # gva_append_cache at the real positions must then give the same bf16 pools, bit for bit, as the fused kernel wrote.
    lens = np.random.default_rng(B).integers(1, 600, size=B)
    d_model = 256
    case32, lw, dc32, W_in, _ = _setup(shape, lens, d_model, "f32")
    try:
        x = torch.from_numpy(lw["x"]).cuda()
        zero = torch.zeros(B, dtype=torch.int32, device="cuda")
        gb.gva_project_in(dc32.handle, dc32.cache, x, _dev16(W_in), d_model, zero, dc32.q_abs, B, dc32.status)
        torch.cuda.synchronize()
        assert int(dc32.status.item()) == 0
        v32, k32 = dc32.pools_to_host()
        pages = [case32.page_of(b, 0) for b in range(B)]
        c_v = np.stack([v32[pg, :, 0] for pg in pages]).astype(np.float32)           # [B][G][d_v]
        c_k = np.stack([k32[pg, 0] for pg in pages]).astype(np.float32)              # [B][d_r]
    finally:
        dc32.close()
    case, lw2, dc, W_in2, _ = _setup(shape, lens, d_model, dtype)
    try:
        assert np.array_equal(W_in, W_in2) and np.array_equal(lw["x"], lw2["x"])
        v_b, k_b = dc.v_pool.clone(), dc.kr_pool.clone()
        gb.gva_project_in(dc.handle, dc.cache, x, _dev16(W_in), d_model, dc.append_pos, dc.q_abs, B, dc.status)
        other = gb.make_cache(v_b, k_b, dc.block_table, case.num_pages, case.max_pages_per_seq)
        gb.gva_append_cache(dc.handle, other, torch.from_numpy(c_v).cuda(), torch.from_numpy(c_k).cuda(), dc.append_pos, B, dc.status)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        assert torch.equal(dc.v_pool.view(torch.uint8), v_b.view(torch.uint8))
        assert torch.equal(dc.kr_pool.view(torch.uint8), k_b.view(torch.uint8))
    finally:
        dc.close()


@pytest.mark.parametrize("B", [1, 33, 200])
def test_project_out(B):
    case, lw, dc, W_in, W_o = _setup(wl.SHAPE_A, [4] * B, d_model=512)
    try:
        rng = np.random.default_rng(7)
        attn = rng.standard_normal((B, 16 * 64)).astype(np.float32)
        y = torch.empty((B, 512), dtype=torch.float32, device="cuda")
        gb.gva_project_out(dc.handle, torch.from_numpy(attn).cuda(), _dev16(W_o), 512, y, B)
        torch.cuda.synchronize()
        ref = orc.matmul(attn, wl.bf16_bits_to_f32(W_o).astype(np.float64))
        assert np.max(np.abs(y.cpu().numpy() - ref)) <= 1e-5 * max(1.0, np.max(np.abs(ref)))
    finally:
        dc.close()


@pytest.mark.parametrize("shape,dtype", [(wl.SHAPE_A, "bf16"), (wl.SHAPE_B, "bf16"), (wl.SHAPE_C, "bf16"), (wl.SHAPE_A0, "bf16"),
                                         (wl.SHAPE_B0, "bf16"), (wl.SHAPE_A, "fp8"), (wl.SHAPE_B, "fp8"), (wl.SHAPE_A, "f32")])
def test_whole_layer_step_from_the_hidden_state(shape, dtype):
    lens = np.array([1, 64, 65, 700, 2049, 130], dtype=np.int32)
    d_model = 1024
    case, lw, dc, W_in, W_o = _setup(shape, lens, d_model, dtype)
    try:
        B = case.B
        x = torch.from_numpy(lw["x"]).cuda()
        attn = torch.empty((B, shape.H, shape.d_v), dtype=torch.float32, device="cuda")
        y = torch.empty((B, d_model), dtype=torch.float32, device="cuda")
        ws = dc.ensure_workspace(0)
        gb.gva_layer_step(dc.handle, dc.cache, x, _dev16(W_in), _dev16(W_o), d_model, dc.append_pos, dc.seq_lens, dc.q_abs,
                          attn, y, ws, B, int(lens.max()), 0, dc.status)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0
        # oracle: same bf16 weights, its own fp64 arithmetic end to end; then attention over the cache the GPU wrote
        # (appended rows are rounded from an f32 product on the GPU and from fp64 in the oracle: they may differ by
        # one unit in the last place, so the attention check reads the GPU's cache)
        Wd = wl.bf16_bits_to_f32(W_in).astype(np.float64); Wo = wl.bf16_bits_to_f32(W_o).astype(np.float64)
        v_gpu, k_gpu = dc.pools_to_host()
        q_gpu = dc.q_abs.cpu().numpy().astype(np.float64)
        out_ref, _ = orc.decode(v_gpu, k_gpu, case.block_table, case.seq_lens, q_gpu, shape.H,
                                scale=1.0 / np.sqrt(float(shape.d_c + shape.d_r)))
        a = attn.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(a - out_ref)) <= 2e-5
        y_ref = orc.matmul(a.reshape(B, -1), Wo)
        assert np.max(np.abs(y.cpu().numpy() - y_ref)) <= 1e-5 * max(1.0, np.max(np.abs(y_ref)))
        # and end to end against the oracle's own layer step (its own append): loose only by the cache rounding
        y_e2e, out_e2e, _ = orc.layer_step(lw["x"], Wd, Wo, case.v_pool, case.kr_pool, case.block_table, case.append_pos,
                                           case.seq_lens, shape.H, shape.G, shape.d_c)
        assert np.max(np.abs(a - out_e2e)) <= 2e-2
        assert np.max(np.abs(y.cpu().numpy() - y_e2e)) <= 2e-2
    finally:
        dc.close()
