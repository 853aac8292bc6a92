"""Pins for the fp64 oracle: every check here compares the oracle with something other than itself --
identities the paper states, closed forms, library routines, or a brute-force second path.
CPU only."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import gva_oracle as orc
from oracle import naive
from paper_2609_13285_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_kv(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def _rows(name):
    return [line.split() for line in open(os.path.join(GOLDEN, name)) if line.strip() and not line.startswith("#")]


def small_case(**kw):
    args = dict(page_size=16, cache_dtype="f32", paged=True, seed=7)
    args.update(kw)
    return wl.make_case("small", wl.HeadShape(H=8, G=2, d_v=16, d_c=12, d_r=8), [37, 5, 16, 1], **args)


# ---------------------------------------------------------------- P2: RoPE (Section 3.2 / 3.3)
def test_rope_closed_form_d2():
    # d_r = 2: theta_0 = base^0 = 1, so the rotation angle is the position itself
    for p in (0, 1, 2, 7, 100):
        y = orc.rope(np.array([1.0, 0.0]), p)
        assert np.allclose(y, [math.cos(p), math.sin(p)], atol=1e-15)
        y = orc.rope(np.array([0.0, 1.0]), p)
        assert np.allclose(y, [-math.sin(p), math.cos(p)], atol=1e-15)


def test_rope_frequencies_closed_form():
    # d_r = 4, base 10000: second pair rotates by p * 10000^(-1/2) = p / 100
    y = orc.rope(np.array([0.0, 0.0, 1.0, 0.0]), 50)
    assert np.allclose(y, [0, 0, math.cos(0.5), math.sin(0.5)], atol=1e-15)
    y = orc.rope(np.array([2.0, 0.0, 0.0, 0.0]), 3, base=100.0)
    assert np.allclose(y, [2 * math.cos(3), 2 * math.sin(3), 0, 0], atol=1e-15)


def test_rope_identity_norm_composition():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 16))
    assert np.array_equal(orc.rope(x, 0), x)
    for p, q in ((3, 11), (1000, 24)):
        y = orc.rope(x, p)
        assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-14)
        assert np.allclose(orc.rope(y, q), orc.rope(x, p + q), atol=1e-12)


def test_rope_relative_position_invariance():
    # R_{j-t} = R_t^T R_j: the positional score depends on j - t only
    rng = np.random.default_rng(1)
    a, b = rng.standard_normal(16), rng.standard_normal(16)
    ref = float(orc.rope(a, 40) @ orc.rope(b, 33))
    for shift in (1, 7, 500, 8000):
        assert abs(float(orc.rope(a, 40 + shift) @ orc.rope(b, 33 + shift)) - ref) < 1e-10
    assert abs(float(orc.rope(a, 41) @ orc.rope(b, 33)) - ref) > 1e-3   # and it does depend on j - t


def test_rope_matches_naive():
    rng = np.random.default_rng(2)
    x = rng.standard_normal(32)
    assert np.allclose(orc.rope(x, 12345), naive.rope(list(x), 12345), atol=1e-13)


# ---------------------------------------------------------------- P1: absorption identity (Eq. absorb)
def test_absorption_identity_explicit_keys():
    c = small_case()
    s = c.shape
    q_abs = orc.absorb_case(c)
    V = wl.pool_to_f64(c.v_pool)
    for b in range(c.B):
        for h in range(s.H):
            g = h // (s.H // s.G)
            for t in range(int(c.seq_lens[b])):
                v = V[c.page_of(b, t // c.page_size), g, t % c.page_size]
                k = v @ c.M[h].astype(np.float64)                      # K_h = V_g(h) M_h   (d_c wide)
                lhs = float(c.q_c[b, h].astype(np.float64) @ k)       # q k^T
                rhs = float(q_abs[b, h, :s.d_v] @ v)                  # q~ v^T
                assert abs(lhs - rhs) <= 1e-12 * max(1.0, abs(lhs))


def test_absorb_orientation_rectangular():
    # d_v != d_c makes a transposed M a shape error or a different number
    c = small_case()
    s = c.shape
    q_abs = orc.absorb_case(c)
    ref = np.einsum("bhj,hij->bhi", c.q_c.astype(np.float64), c.M.astype(np.float64))
    assert np.allclose(q_abs[..., :s.d_v], ref, atol=1e-13)
    for b in range(c.B):
        assert np.allclose(q_abs[b, :, s.d_v:], orc.rope(c.q_r[b], int(c.q_pos[b])), atol=1e-14)


# ---------------------------------------------------------------- P3: full-key SDPA equivalence (library routine)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_full_key_sdpa_equivalence(dtype):
    c = small_case(cache_dtype=dtype)
    s = c.shape
    out, lse = orc.decode_case(c)
    V = torch.from_numpy(wl.pool_to_f64(c.v_pool))
    KR = torch.from_numpy(wl.pool_to_f64(c.kr_pool))
    M = torch.from_numpy(c.M.astype(np.float64))
    for b in range(c.B):
        L = int(c.seq_lens[b])
        pages = [c.page_of(b, t // c.page_size) for t in range(L)]
        slots = [t % c.page_size for t in range(L)]
        qr = torch.from_numpy(orc.rope(c.q_r[b], int(c.q_pos[b])))
        q_full = torch.cat([torch.from_numpy(c.q_c[b].astype(np.float64)), qr], dim=-1)      # [H, d_c+d_r]
        keys, vals = [], []
        for h in range(s.H):
            g = h // (s.H // s.G)
            Vg = V[pages, g, slots]                                                            # [L, d_v]
            keys.append(torch.cat([Vg @ M[h], KR[pages, slots]], dim=-1))                      # [V M_h | k^rope]
            vals.append(Vg)
        K, Vv = torch.stack(keys), torch.stack(vals)
        ref = torch.nn.functional.scaled_dot_product_attention(
            q_full[None, :, None, :], K[None], Vv[None], scale=1.0 / math.sqrt(s.d_c + s.d_r))[0, :, 0]
        assert np.allclose(out[b], ref.numpy(), atol=1e-12)
        logits = torch.einsum("hd,hld->hl", q_full, K) / math.sqrt(s.d_c + s.d_r)
        assert np.allclose(lse[b], torch.logsumexp(logits, dim=-1).numpy(), atol=1e-12)


# ---------------------------------------------------------------- P4: special cases that are textbook attention
def test_shared_kv_limit_is_plain_attention():
    # M_h = I and a silent positional channel: keys are the values themselves (the shared-KV design)
    c = small_case()
    s = wl.HeadShape(H=4, G=4, d_v=8, d_c=8, d_r=4)
    c = wl.make_case("skv", s, [9, 3], page_size=4, cache_dtype="f32", paged=True, seed=3)
    c.M[:] = np.eye(8, dtype=np.float32)
    c.q_r[:] = 0
    out, _ = orc.decode_case(c)
    V = wl.pool_to_f64(c.v_pool)
    for b in range(c.B):
        L = int(c.seq_lens[b])
        for h in range(s.H):                                       # G = H: independent heads
            Vh = np.stack([V[c.page_of(b, t // 4), h, t % 4] for t in range(L)])
            sc = (Vh @ c.q_c[b, h].astype(np.float64)) / math.sqrt(s.d_c + s.d_r)
            p = np.exp(sc - sc.max()); p /= p.sum()
            assert np.allclose(out[b, h], p @ Vh, atol=1e-13)


def test_group_map_is_contiguous_blocks():
    # one group with a distinctive value: only heads h with h // (H/G) == that group see it
    s = wl.HeadShape(H=8, G=4, d_v=4, d_c=4, d_r=2)
    c = wl.make_case("gmap", s, [6], page_size=2, cache_dtype="f32", paged=False, seed=4)
    c.v_pool[:] = 0
    c.v_pool[:, 2] = 1.0                                           # group 2 rows are all ones
    out, _ = orc.decode_case(c)
    for h in range(8):
        expect = 1.0 if h // 2 == 2 else 0.0
        assert np.allclose(out[0, h], expect, atol=1e-14)


def test_single_group_is_mqa_like():
    s = wl.HeadShape(H=4, G=1, d_v=4, d_c=4, d_r=2)
    c = wl.make_case("mqa", s, [5], page_size=8, cache_dtype="f32", paged=False, seed=5)
    c.q_c[0, :] = c.q_c[0, 0]
    c.q_r[0, :] = c.q_r[0, 0]
    c.M[:] = c.M[0]
    out, _ = orc.decode_case(c)
    for h in range(1, 4):
        assert np.allclose(out[0, h], out[0, 0], atol=1e-15)


# ---------------------------------------------------------------- P5: softmax invariants
def test_softmax_rows_sum_to_one_and_hull():
    c = small_case(cache_dtype="bf16")
    s = c.shape
    q_abs = orc.absorb_case(c)
    out, lse = orc.decode_case(c, q_abs)
    V = wl.pool_to_f64(c.v_pool)
    scale = 1.0 / math.sqrt(s.d_c + s.d_r)
    for b in range(c.B):
        L = int(c.seq_lens[b])
        for h in (0, 3, 7):
            p = orc.decode_weights(c.v_pool, c.kr_pool, c.block_table, c.seq_lens, q_abs, s.H, b, h, scale)
            assert abs(p.sum() - 1.0) < 1e-15 * max(L, 8)
            assert (p >= 0).all()
            g = h // (s.H // s.G)
            rows = np.stack([V[c.page_of(b, t // c.page_size), g, t % c.page_size] for t in range(L)])
            assert (out[b, h] <= rows.max(0) + 1e-12).all() and (out[b, h] >= rows.min(0) - 1e-12).all()
            assert np.allclose(out[b, h], p @ rows, atol=1e-13)


def test_zero_query_gives_mean_and_log_count():
    c = small_case()
    s = c.shape
    q_abs = np.zeros((c.B, s.H, s.d_v + s.d_r))
    out, lse = orc.decode_case(c, q_abs)
    V = wl.pool_to_f64(c.v_pool)
    for b in range(c.B):
        L = int(c.seq_lens[b])
        rows = np.stack([V[c.page_of(b, t // c.page_size), 1, t % c.page_size] for t in range(L)])
        assert np.allclose(out[b, s.H - 1], rows.mean(0), atol=1e-14)
        assert np.allclose(lse[b], math.log(L), atol=1e-14)


def test_dominant_score_selects_row_and_constant_shift():
    s = wl.HeadShape(H=2, G=1, d_v=4, d_c=4, d_r=2)
    c = wl.make_case("dom", s, [8], page_size=8, cache_dtype="f32", paged=False, seed=6)
    q_abs = np.zeros((1, 2, 6))
    # make row 5 twice as long as the longest other row: with q along it, Cauchy-Schwarz bounds every other
    # score by half of row 5's, so the gap is guaranteed rather than hoped for
    norms = np.linalg.norm(wl.pool_to_f64(c.v_pool)[0, 0, :8], axis=1)
    c.v_pool[0, 0, 5] *= np.float32(2.0 * np.delete(norms, 5).max() / norms[5])
    v5 = wl.pool_to_f64(c.v_pool)[0, 0, 5]
    q_abs[0, 0, :4] = 400.0 * v5 / np.linalg.norm(v5)          # hugely aligned with token 5
    out, _ = orc.decode_case(c, q_abs)
    scores = (wl.pool_to_f64(c.v_pool)[0, 0, :8] @ q_abs[0, 0, :4]) / math.sqrt(s.d_c + s.d_r)
    assert np.argmax(scores) == 5 and np.sort(scores)[-1] - np.sort(scores)[-2] > 40     # exp(-40) ~ 4e-18
    assert np.allclose(out[0, 0], v5, atol=1e-12)
    # the other head of the group has a zero query and must still see the mean of the (changed) rows
    assert np.allclose(out[0, 1], wl.pool_to_f64(c.v_pool)[0, 0, :8].mean(0), atol=1e-13)
    # adding a constant to every score (via a constant k_r channel) leaves out unchanged, shifts lse
    c.kr_pool[:] = 0
    c.kr_pool[..., 0] = 1.0
    qa = orc.absorb_case(c)
    o1, l1 = orc.decode_case(c, qa)
    qb = qa.copy(); qb[..., s.d_v] += 3.0
    o2, l2 = orc.decode_case(c, qb)
    assert np.allclose(o1, o2, atol=1e-13)
    assert np.allclose(l2 - l1, 3.0 / math.sqrt(s.d_c + s.d_r), atol=1e-13)


def test_flat_softmax_caption_case():
    n, sigma, w, tol = map(float, _rows("flat_softmax_caption.txt")[0])
    n = int(n)
    s = wl.HeadShape(H=1, G=1, d_v=64, d_c=64, d_r=2)
    c = wl.make_case("flat", s, [n], page_size=16, cache_dtype="f32", paged=False, seed=8)
    c.M[0] = np.eye(64, dtype=np.float32)
    c.v_pool *= np.float32(sigma)                                  # keys = values, sigma_K = sigma
    c.kr_pool[:] = 0
    q_abs = orc.absorb(c.q_c * np.float32(sigma), c.q_r * 0, c.M, c.q_pos)
    p = orc.decode_weights(c.v_pool, c.kr_pool, None, c.seq_lens, q_abs, 1, 0, 0, 1 / math.sqrt(64.0),
                           max_pages_per_seq=c.max_pages_per_seq)
    assert np.all(np.abs(p - w) < tol)


# ---------------------------------------------------------------- P6: split / paging invariance
def test_lse_recombination_of_arbitrary_partitions():
    c = small_case(cache_dtype="bf16")
    s = c.shape
    q_abs = orc.absorb_case(c)
    out, lse = orc.decode_case(c, q_abs)
    V = wl.pool_to_f64(c.v_pool); KR = wl.pool_to_f64(c.kr_pool)
    b = 0
    L = int(c.seq_lens[b])
    cuts = [0, 1, 9, 10, 30, L]
    scale = 1 / math.sqrt(s.d_c + s.d_r)
    for h in range(s.H):
        g = h // (s.H // s.G)
        parts = []
        for lo, hi in zip(cuts[:-1], cuts[1:]):
            rows = np.stack([V[c.page_of(b, t // 16), g, t % 16] for t in range(lo, hi)])
            kr = np.stack([KR[c.page_of(b, t // 16), t % 16] for t in range(lo, hi)])
            sc = (rows @ q_abs[b, h, :s.d_v] + kr @ q_abs[b, h, s.d_v:]) * scale
            m = sc.max(); e = np.exp(sc - m)
            parts.append((m, e.sum(), e @ rows))
        mstar = max(p[0] for p in parts)
        Lsum = sum(p[1] * math.exp(p[0] - mstar) for p in parts)
        o = sum(p[2] * math.exp(p[0] - mstar) for p in parts) / Lsum
        assert np.allclose(o, out[b, h], atol=1e-13)
        assert abs(mstar + math.log(Lsum) - lse[b, h]) < 1e-13


def test_page_permutation_and_contiguous_equivalence():
    c = small_case(paged=False)
    out0, lse0 = orc.decode_case(c)
    perm = np.random.default_rng(9).permutation(c.num_pages)
    inv = np.argsort(perm)
    bt = np.array([[inv[b * c.max_pages_per_seq + j] for j in range(c.max_pages_per_seq)] for b in range(c.B)],
                  dtype=np.int32)
    v2, k2 = np.ascontiguousarray(c.v_pool[perm]), np.ascontiguousarray(c.kr_pool[perm])
    out1, lse1 = orc.decode(v2, k2, bt, c.seq_lens, orc.absorb_case(c), c.shape.H,
                            scale=1 / math.sqrt(c.shape.d_c + c.shape.d_r))
    assert np.array_equal(out0, out1) and np.array_equal(lse0, lse1)


# ---------------------------------------------------------------- P11: brute force and hand-computed numbers
def test_hand_computed_two_token_case():
    g = _read_kv("closed_form_two_tokens.txt")
    M = np.array([[[0.0, 5.0], [1.0, 0.0]]])
    q_abs = orc.absorb(np.array([[[1.0, 0.0]]]), np.zeros((1, 1, 2)), M, [2])
    assert q_abs[0, 0, 0] == g["q_tilde_0"] and q_abs[0, 0, 1] == g["q_tilde_1"]
    v_pool = np.zeros((1, 1, 2, 2), dtype=np.float32)
    v_pool[0, 0, 1, 1] = np.float32(2 * math.log(3))
    kr_pool = np.ones((1, 2, 2), dtype=np.float32)
    out, lse = orc.decode(v_pool, kr_pool, None, [2], q_abs, 1, scale=0.5, max_pages_per_seq=1)
    p = orc.decode_weights(v_pool, kr_pool, None, [2], q_abs, 1, 0, 0, 0.5, max_pages_per_seq=1)
    assert np.allclose(p, [g["p_0"], g["p_1"]], atol=1e-7)               # v is stored in f32
    assert np.allclose(out[0, 0], [g["out_0"], g["out_1"]], atol=1e-6)
    assert abs(lse[0, 0] - g["lse"]) < 1e-7


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_brute_force_tiny_paged_ragged(dtype):
    s = wl.HeadShape(H=4, G=2, d_v=4, d_c=4, d_r=2)
    c = wl.make_case("tiny", s, [0, 1, 3, 5], page_size=2, cache_dtype=dtype, paged=True, seed=11,
                     poison_unused=True)
    out, lse = orc.decode_case(c)
    V = wl.pool_to_f64(c.v_pool).tolist(); KR = wl.pool_to_f64(c.kr_pool).tolist()
    Vt, Kt = naive.gather_tokens(V, KR, c.block_table.tolist(), c.seq_lens.tolist(), 2, c.max_pages_per_seq)
    o2, l2 = naive.decode_step(c.q_c.astype(np.float64).tolist(), c.q_r.astype(np.float64).tolist(),
                               c.M.astype(np.float64).tolist(), c.q_pos.tolist(), Vt, Kt, 4, 2, 4)
    assert np.isfinite(out).all()
    assert np.allclose(out, np.array(o2), atol=1e-13)
    assert np.allclose(lse[1:], np.array(l2)[1:], atol=1e-13)
    assert np.all(out[0] == 0) and np.all(np.isneginf(lse[0]))          # empty sequence


def test_naive_explicit_key_path_agrees():
    # naive path with explicit K = V M (never absorbed) against the C oracle's absorbed path
    s = wl.HeadShape(H=2, G=1, d_v=3, d_c=5, d_r=2)
    c = wl.make_case("expl", s, [4], page_size=4, cache_dtype="f32", paged=False, seed=12)
    out, _ = orc.decode_case(c)
    V = wl.pool_to_f64(c.v_pool)[0, 0]; KR = wl.pool_to_f64(c.kr_pool)[0]
    for h in range(2):
        qr = naive.rope(c.q_r[0, h].astype(np.float64).tolist(), int(c.q_pos[0]))
        sc = []
        for t in range(4):
            k = naive.reconstruct_key(V[t].tolist(), c.M[h].astype(np.float64).tolist())
            sc.append((sum(a * b for a, b in zip(c.q_c[0, h].astype(np.float64), k)) +
                       sum(a * b for a, b in zip(qr, KR[t]))) / math.sqrt(5 + 2))
        p = naive.softmax(sc)
        o = [sum(p[t] * V[t][i] for t in range(4)) for i in range(3)]
        assert np.allclose(out[0, h], o, atol=1e-14)


# ---------------------------------------------------------------- P7 / P8: statistics on the synthetic distribution
def test_gaussian_tilting_limit():
    # V rows ~ N(0, I): softmax-weighted mean tends to q~ / sqrt(d_qk) as T grows
    s = wl.SHAPE_A
    c = wl.make_case("tilt", s, [16384], page_size=64, cache_dtype="bf16", paged=True, seed=13)
    q_abs = orc.absorb_case(c)
    out, _ = orc.decode_case(c, q_abs)
    target = q_abs[0, :, :s.d_v] / math.sqrt(s.d_c + s.d_r)
    assert np.max(np.abs(out[0] - target)) < 0.08
    assert np.corrcoef(out[0].ravel(), target.ravel())[0, 1] > 0.9


def test_variance_rules_of_the_generator():
    c = wl.make_case("var", wl.SHAPE_A, [2048], page_size=64, cache_dtype="bf16", paged=True, seed=14)
    V = wl.pool_to_f64(c.v_pool)
    K = V[:, 0].reshape(-1, 64) @ c.M[0].astype(np.float64)              # reconstructed keys, head 0
    assert abs(K.std() - 1.0) < 0.05                                     # Var(K) ~ d_in sigma_V^2 Var(M) = 1
    logits = (K @ c.q_c[0, 0].astype(np.float64)) / 8.0                  # q k^T / sqrt(d_h)
    assert abs(logits.var() / (c.q_c[0, 0].astype(np.float64) ** 2).mean() - 1.0) < 0.15


# ---------------------------------------------------------------- P10: cache byte accounting
def test_cache_ratio_formula_and_bytes():
    for G, d_h, d_r, ratio, pct in _rows("cache_ratio.txt"):
        G, d_h, d_r, ratio, pct = int(G), int(d_h), int(d_r), float(ratio), float(pct)
        T = 1000
        n_gva = T * G * d_h + T * d_r
        n_gqa = 2 * T * G * d_h
        assert n_gva / n_gqa == ratio == 0.5 + d_r / (2 * G * d_h)
        assert round(100 * (1 - ratio)) == pct
    c = wl.make_case("bytes", wl.SHAPE_A, [100, 7], page_size=64, cache_dtype="bf16", seed=1)
    assert c.cache_bytes() == 107 * 272 * 2
    assert c.algorithmic_bytes() == 107 * 544 + 2 * 16 * 80 * 4 + 2 * 16 * 64 * 4
    assert wl.SHAPE_B.row_elems * 2 == 2112


# ---------------------------------------------------------------- P12: append
def test_bf16_rounding_against_library_cast():
    rng = np.random.default_rng(15)
    x = np.concatenate([rng.standard_normal(4000), rng.standard_normal(500) * 1e-30, rng.standard_normal(500) * 1e30,
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38, 3.4e38, 1e-40, -1e-45]])
    for v in x:
        f = np.float32(v)
        got = orc.bf16_from_double(float(f))
        ref = torch.tensor([f], dtype=torch.float32).bfloat16().view(torch.int16).item() & 0xFFFF
        assert got == ref, (v, hex(got), hex(ref))
    # a double that float rounding would push onto a bf16 tie: direct rounding must not double-round
    x = 1.0 + 2.0 ** -8 + 2.0 ** -30       # just above the tie between 1.0 and 1.0078125 -> rounds up
    assert orc.bf16_from_double(x) == 0x3F81
    assert orc.bf16_from_double(1.0 + 2.0 ** -8) == 0x3F80     # exact tie -> even
    assert orc.bf16_from_double(1.0 + 3 * 2.0 ** -8) == 0x3F82  # exact tie -> even (up)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_append_touches_exactly_the_new_rows(dtype):
    c = small_case(cache_dtype=dtype)
    s = c.shape
    v0, k0 = c.v_pool.copy(), c.kr_pool.copy()
    assert orc.append_case(c) == 0
    changed_v = np.zeros(c.v_pool.shape[:3], dtype=bool)
    changed_k = np.zeros(c.kr_pool.shape[:2], dtype=bool)
    for b in range(c.B):
        t = int(c.append_pos[b])
        page, slot = c.page_of(b, t // c.page_size), t % c.page_size
        changed_v[page, :, slot] = True
        changed_k[page, slot] = True
        rot = orc.rope(c.kr_new[b], t)
        if dtype == "bf16":
            ref_v = torch.from_numpy(c.v_new[b]).bfloat16().view(torch.int16).numpy().view(np.uint16)
            assert np.array_equal(c.v_pool[page, :, slot], ref_v)
            got = wl.bf16_bits_to_f32(c.kr_pool[page, slot]).astype(np.float64)
            assert np.all(np.abs(got - rot) <= np.abs(rot) * 2.0 ** -8 + 1e-40)
        else:
            assert np.array_equal(c.v_pool[page, :, slot], c.v_new[b])
            assert np.array_equal(c.kr_pool[page, slot], rot.astype(np.float32))
    assert np.array_equal(c.v_pool[~changed_v], v0[~changed_v])
    assert np.array_equal(c.kr_pool[~changed_k], k0[~changed_k])


def test_append_then_decode_follows_algorithm_order():
    # the appended token is attended by its own query (cache is extended before attention)
    s = wl.HeadShape(H=2, G=1, d_v=4, d_c=4, d_r=2)
    c = wl.make_case("order", s, [3], page_size=4, cache_dtype="f32", paged=False, seed=16,
                     q_pos=[2], append_pos=[2])
    c.v_new[:] = 50.0
    orc.append_case(c)
    q_abs = np.zeros((1, 2, 6)); q_abs[..., :4] = 5.0                    # strongly prefers the new, large row
    out, _ = orc.decode_case(c, q_abs)
    assert np.allclose(out, 50.0, atol=1e-6)


def test_append_reports_bad_page():
    c = small_case()
    c.block_table[1, 0] = c.num_pages + 3
    assert orc.append_case(c) == 2


@pytest.mark.parametrize("bad", [-1, -64, "first_beyond", "far_beyond"])
def test_append_refuses_positions_outside_the_block_table(bad):
    # a position that is negative or at/after max_pages * P has no block-table entry: the sequence is reported
    # (1 + b), nothing of it or of later sequences is written, and earlier sequences are written as usual
    c = small_case()
    cap = c.max_pages_per_seq * c.page_size
    t_bad = {"first_beyond": cap, "far_beyond": cap + 5 * c.page_size + 3}.get(bad, bad)
    good = small_case()
    assert orc.append_case(good) == 0
    v0, k0 = c.v_pool.copy(), c.kr_pool.copy()
    c.append_pos[1] = t_bad
    assert orc.append_case(c) == 2
    t0 = int(c.append_pos[0])
    page, slot = c.page_of(0, t0 // c.page_size), t0 % c.page_size
    mask_v = np.zeros(c.v_pool.shape[:3], dtype=bool); mask_v[page, :, slot] = True
    mask_k = np.zeros(c.kr_pool.shape[:2], dtype=bool); mask_k[page, slot] = True
    assert np.array_equal(c.v_pool[mask_v], good.v_pool[mask_v]) and np.array_equal(c.kr_pool[mask_k], good.kr_pool[mask_k])
    assert np.array_equal(c.v_pool[~mask_v], v0[~mask_v]) and np.array_equal(c.kr_pool[~mask_k], k0[~mask_k])
    # the chunked form takes the same decision (context length such that the chunk's first token is the bad position)
    pc = small_prefill("bf16", paged=True, seed=36)
    pcap = pc.cache.max_pages_per_seq * pc.cache.page_size
    ctx = np.array(pc.ctx_lens, dtype=np.int32)
    ctx[0] = {"first_beyond": pcap, "far_beyond": pcap + 5 * pc.cache.page_size + 3}.get(bad, bad)
    v1, k1 = pc.cache.v_pool.copy(), pc.cache.kr_pool.copy()
    q0 = int(pc.cu_q[1] - pc.cu_q[0])
    assert q0 > 0
    assert orc.append_chunk(v1, k1, pc.cache.block_table, pc.v_new, pc.kr_new, pc.cu_q, ctx) == 1
    assert np.array_equal(v1, pc.cache.v_pool) and np.array_equal(k1, pc.cache.kr_pool)


# ---------------------------------------------------------------- GQA companion
def test_gqa_oracle_against_sdpa():
    g = wl.gqa_case("gqa", H=8, G=2, d_h=16, seq_lens=[33, 7], page_size=8, cache_dtype="bf16", seed=17)
    out, lse = orc.gqa_decode(g["k_pool"], g["v_pool"], g["block_table"], g["seq_lens"], g["q"])
    K = torch.from_numpy(wl.pool_to_f64(g["k_pool"])); V = torch.from_numpy(wl.pool_to_f64(g["v_pool"]))
    for b in range(2):
        L = int(g["seq_lens"][b])
        pages = [int(g["block_table"][b, t // 8]) for t in range(L)]
        slots = [t % 8 for t in range(L)]
        Kb = K[pages, :, slots].permute(1, 0, 2).repeat_interleave(4, dim=0)   # [H, L, d]
        Vb = V[pages, :, slots].permute(1, 0, 2).repeat_interleave(4, dim=0)
        q = torch.from_numpy(g["q"][b].astype(np.float64))
        ref = torch.nn.functional.scaled_dot_product_attention(q[None, :, None], Kb[None], Vb[None])[0, :, 0]
        assert np.allclose(out[b], ref.numpy(), atol=1e-12)


def test_c_oracle_thread_count_is_positive():
    assert orc.num_threads() >= 1


# ---------------------------------------------------------------- projections around the attention
def _tiny_layer(seed=31):
    s = wl.HeadShape(H=4, G=2, d_v=4, d_c=6, d_r=2)
    lw = wl.layer_weights(s, d_model=10, B=3, seed=seed)
    rng = np.random.default_rng(seed)
    M = (rng.standard_normal((s.H, s.d_v, s.d_c)) / 2).astype(np.float32)
    return s, lw, M


def test_matmul_against_library_routine():
    rng = np.random.default_rng(30)
    x, W = rng.standard_normal((5, 17)), rng.standard_normal((17, 9))
    assert np.allclose(orc.matmul(x, W), x @ W, atol=1e-13)


def test_weight_absorption_is_associativity():
    # (x W_Q^nope) M^T == x (W_Q^nope M^T): the folded projection gives the absorbed query directly
    s, lw, M = _tiny_layer()
    x = lw["x"].astype(np.float64)
    W_abs = orc.fold_maps(lw["W_q_nope"], M)
    for h in range(s.H):
        q_nope = x @ lw["W_q_nope"][:, h, :].astype(np.float64)               # Algorithm 1: q = x W_Q
        two_step = q_nope @ M[h].astype(np.float64).T                           # then q~ = q^nope M_h^T
        assert np.allclose(x @ W_abs[:, h, :], two_step, atol=1e-13)
    ref = np.einsum("mhj,hij->mhi", lw["W_q_nope"].astype(np.float64), M.astype(np.float64))
    assert np.allclose(W_abs, ref, atol=1e-14)


def test_packed_projection_layout():
    s, lw, M = _tiny_layer()
    W_in = orc.pack_input_weights(lw["W_q_nope"], lw["W_q_rope"], lw["W_v"], lw["W_r"], M)
    assert W_in.shape == (10, s.H * (s.d_v + s.d_r) + s.G * s.d_v + s.d_r)
    q_t, q_r, v, kr = orc.project_in(lw["x"], W_in, s.H, s.G, s.d_v, s.d_r)
    x = lw["x"].astype(np.float64)
    assert np.allclose(q_r, np.einsum("bm,mhr->bhr", x, lw["W_q_rope"].astype(np.float64)), atol=1e-13)
    assert np.allclose(v, np.einsum("bm,mgd->bgd", x, lw["W_v"].astype(np.float64)), atol=1e-13)
    assert np.allclose(kr, x @ lw["W_r"].astype(np.float64), atol=1e-13)
    assert np.allclose(q_t, np.einsum("bm,mhj,hij->bhi", x, lw["W_q_nope"].astype(np.float64), M.astype(np.float64)),
                       atol=1e-13)


def test_layer_step_against_algorithm_line_by_line():
    # the oracle's layer step (folded weights, absorbed scores, paged cache) against the naive path that follows
    # Algorithm 1 from the hidden state with explicit keys K = V M, for each sequence separately
    s, lw, M = _tiny_layer()
    T = [3, 0, 5]                                        # tokens already cached per sequence
    case = wl.make_case("layer", s, [t + 1 for t in T], page_size=2, cache_dtype="f32", paged=True, seed=32,
                        q_pos=T, append_pos=T)
    V0 = wl.pool_to_f64(case.v_pool).tolist(); K0 = wl.pool_to_f64(case.kr_pool).tolist()
    Vt, Kt = naive.gather_tokens(V0, K0, case.block_table.tolist(), T, 2, case.max_pages_per_seq)
    W_in = orc.pack_input_weights(lw["W_q_nope"], lw["W_q_rope"], lw["W_v"], lw["W_r"], M)
    y, out, _ = orc.layer_step(lw["x"], W_in, lw["W_o"], case.v_pool, case.kr_pool, case.block_table, T,
                               [t + 1 for t in T], s.H, s.G, s.d_c)
    W_Q = np.concatenate([lw["W_q_rope"], lw["W_q_nope"]], axis=2).astype(np.float64).tolist()   # [m][h][rope | nope]
    for b in range(3):
        V_cache = [[Vt[b][t][g] for t in range(T[b])] for g in range(s.G)]
        KR_cache = [Kt[b][t] for t in range(T[b])]
        y_ref, outs = naive.layer_decode_step(lw["x"][b].astype(np.float64).tolist(), W_Q,
                                              lw["W_v"].astype(np.float64).tolist(), lw["W_r"].astype(np.float64).tolist(),
                                              lw["W_o"].astype(np.float64).tolist(), M.astype(np.float64).tolist(), T[b],
                                              V_cache, KR_cache, s.H, s.G, s.d_c, s.d_r)
        # the cache is f32 in this case: the appended row is rounded to f32 before it is attended
        assert np.allclose(out[b], np.array(outs), atol=1e-6)
        assert np.allclose(y[b], np.array(y_ref), atol=1e-6)


def test_bf16_round_matches_library_cast():
    rng = np.random.default_rng(33)
    a = rng.standard_normal(300).astype(np.float32)
    ref = torch.from_numpy(a).bfloat16().view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.bf16_round(a), ref)


# ---------------------------------------------------------------- prefill / chunked prefill (causal, explicit keys)
def small_prefill(cache_dtype="bf16", paged=True, seed=31):
    s = wl.HeadShape(H=4, G=2, d_v=8, d_c=6, d_r=4)
    return wl.make_prefill_case("pf", s, [0, 5, 3, 9], [7, 4, 0, 1], page_size=4, cache_dtype=cache_dtype, paged=paged,
                                seed=seed, poison_unused=True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_prefill_causal_sdpa_equivalence(dtype):
    # library routine with an explicit boolean causal mask over explicitly formed full keys [V M_h | k^rope]
    pc = small_prefill(dtype)
    c, s = pc.cache, pc.cache.shape
    out, lse = orc.prefill_case(pc)
    V = torch.from_numpy(wl.pool_to_f64(c.v_pool)); KR = torch.from_numpy(wl.pool_to_f64(c.kr_pool))
    M = torch.from_numpy(c.M.astype(np.float64))
    for b in range(c.B):
        n, ctx = int(pc.q_lens[b]), int(pc.ctx_lens[b])
        if n == 0:
            continue
        L = ctx + n
        pages = [c.page_of(b, t // c.page_size) for t in range(L)]; slots = [t % c.page_size for t in range(L)]
        rows = slice(int(pc.cu_q[b]), int(pc.cu_q[b + 1]))
        q_rot = np.stack([orc.rope(pc.q_r[int(pc.cu_q[b]) + i], ctx + i) for i in range(n)])            # [n, H, d_r]
        q_full = torch.cat([torch.from_numpy(pc.q_c[rows].astype(np.float64)), torch.from_numpy(q_rot)], dim=-1)
        mask = torch.arange(L)[None, :] <= (ctx + torch.arange(n))[:, None]                              # [n, L]
        for h in range(s.H):
            Vg = V[pages, h // (s.H // s.G), slots]
            K = torch.cat([Vg @ M[h], KR[pages, slots]], dim=-1)
            ref = torch.nn.functional.scaled_dot_product_attention(
                q_full[None, None, :, h], K[None, None], Vg[None, None], attn_mask=mask[None, None],
                scale=1.0 / math.sqrt(s.d_c + s.d_r))[0, 0]
            assert np.allclose(out[rows, h], ref.numpy(), atol=1e-12)
            logits = (q_full[:, h] @ K.T) / math.sqrt(s.d_c + s.d_r)
            ref_lse = torch.logsumexp(logits.masked_fill(~mask, -math.inf), dim=-1)
            assert np.allclose(lse[rows, h], ref_lse.numpy(), atol=1e-12)


def test_prefill_row_equals_decode_of_its_prefix():
    # each query row is one decode step over the first t+1 tokens (Algorithm 1 applied token by token); the decode
    # oracle uses the absorbed form, the prefill oracle explicit keys, so this is also the absorption identity
    pc = small_prefill("bf16", paged=True, seed=32)
    c, s = pc.cache, pc.cache.shape
    out, lse = orc.prefill_case(pc)
    q_abs = orc.absorb(pc.q_c, pc.q_r, c.M, pc.q_pos)
    for n in range(pc.n_q):
        b = int(pc.q_seq[n])
        lens = np.zeros(c.B, dtype=np.int32); lens[b] = pc.q_pos[n] + 1
        qa = np.zeros((c.B, s.H, s.d_v + s.d_r)); qa[b] = q_abs[n]
        o, l = orc.decode(c.v_pool, c.kr_pool, c.block_table, lens, qa, s.H, d_c=s.d_c)
        assert np.allclose(out[n], o[b], atol=1e-13) and np.allclose(lse[n], l[b], atol=1e-13)


def test_prefill_brute_force_and_closed_forms():
    pc = small_prefill("f32", paged=True, seed=33)
    c, s = pc.cache, pc.cache.shape
    out, lse = orc.prefill_case(pc)
    V = wl.pool_to_f64(c.v_pool).tolist(); KR = wl.pool_to_f64(c.kr_pool).tolist()
    Vt, Kt = naive.gather_tokens(V, KR, c.block_table.tolist(), c.seq_lens.tolist(), c.page_size, c.max_pages_per_seq)
    for b in range(c.B):
        rows = slice(int(pc.cu_q[b]), int(pc.cu_q[b + 1]))
        o2 = naive.prefill_sequence(pc.q_c[rows].astype(np.float64).tolist(), pc.q_r[rows].astype(np.float64).tolist(),
                                    c.M.astype(np.float64).tolist(), int(pc.ctx_lens[b]), Vt[b], Kt[b], s.H, s.G)
        if pc.q_lens[b]:
            assert np.allclose(out[rows], np.array(o2), atol=1e-13)
    # the first token of a prompt with no context sees only itself: o = its own value row, lse = its own score
    first = int(pc.cu_q[0])
    Vd = wl.pool_to_f64(c.v_pool)
    for h in range(s.H):
        g = h // (s.H // s.G)
        assert np.allclose(out[first, h], Vd[c.page_of(0, 0), g, 0], atol=1e-15)
    # zero queries: uniform weights over the visible prefix -> running mean of the value rows, lse = log(t + 1)
    pz = small_prefill("f32", paged=False, seed=34)
    pz.q_c[:] = 0; pz.q_r[:] = 0
    oz, lz = orc.prefill_case(pz)
    cz = pz.cache
    Vz = wl.pool_to_f64(cz.v_pool)
    for n in range(pz.n_q):
        b, t = int(pz.q_seq[n]), int(pz.q_pos[n])
        rowsV = np.stack([Vz[cz.page_of(b, j // cz.page_size), :, j % cz.page_size] for j in range(t + 1)])   # [t+1, G, d_v]
        for h in range(s.H):
            assert np.allclose(oz[n, h], rowsV[:, h // (s.H // s.G)].mean(axis=0), atol=1e-14)
        assert np.allclose(lz[n], math.log(t + 1), atol=1e-14)


def test_prefill_is_causal_and_chunking_invariant():
    # (a) changing a later token's cache rows or queries never changes an earlier row; (b) splitting the same
    # prompt into [context | chunk] at any point gives the same rows as prefilling it whole
    s = wl.HeadShape(H=4, G=2, d_v=8, d_c=6, d_r=4)
    whole = wl.make_prefill_case("w", s, [0], [11], page_size=4, cache_dtype="f32", paged=True, seed=35)
    out_w, lse_w = orc.prefill_case(whole)
    for cut in (1, 4, 10):
        part = wl.make_prefill_case("p", s, [cut], [11 - cut], page_size=4, cache_dtype="f32", paged=True, seed=35)
        assert np.array_equal(part.cache.v_pool, whole.cache.v_pool)           # same seeded cache
        part.q_c[:] = whole.q_c[cut:]; part.q_r[:] = whole.q_r[cut:]
        o, l = orc.prefill_case(part)
        assert np.allclose(o, out_w[cut:], atol=1e-14) and np.allclose(l, lse_w[cut:], atol=1e-14)
    c = whole.cache
    page, slot = c.page_of(0, 7 // 4), 7 % 4
    c.v_pool[page, :, slot] += 3.0
    c.kr_pool[page, slot] -= 2.0
    whole.q_c[8:] *= -1
    o2, _ = orc.prefill_case(whole)
    assert np.array_equal(o2[:7], out_w[:7]) and not np.allclose(o2[7], out_w[7])


def test_append_chunk_equals_token_by_token_append():
    pc = small_prefill("bf16", paged=True, seed=36)
    c = pc.cache
    v1, k1 = c.v_pool.copy(), c.kr_pool.copy()
    v2, k2 = c.v_pool.copy(), c.kr_pool.copy()
    assert orc.append_chunk(v1, k1, c.block_table, pc.v_new, pc.kr_new, pc.cu_q, pc.ctx_lens) == 0
    for n in range(pc.n_q):                       # Algorithm 1's append, one token at a time
        b = int(pc.q_seq[n])
        vn = np.zeros((c.B,) + pc.v_new.shape[1:], dtype=np.float32); kn = np.zeros((c.B, pc.kr_new.shape[1]), dtype=np.float32)
        vn[b], kn[b] = pc.v_new[n], pc.kr_new[n]
        # append only sequence b: a one-sequence view of the block table
        assert orc.append(v2, k2, c.block_table[b:b + 1], vn[b:b + 1], kn[b:b + 1], [int(pc.q_pos[n])]) == 0
    assert np.array_equal(v1, v2) and np.array_equal(k1, k2)
    changed = np.argwhere((v1 != c.v_pool).any(axis=(1, 3)))
    assert len(changed) <= pc.n_q                                  # at most one (page, slot) per new token


# ---------------------------------------------------------------- value-only cache (no positional slice, d_r = 0)
def test_value_only_cache_is_attention_with_keys_v_m():
    # without the positional slice the score is q^nope . (v M_h) alone and d_qk = d_c: plain attention whose keys
    # are the reconstructed content keys (library routine), and the cache is exactly half of matched GQA
    s = wl.HeadShape(H=8, G=2, d_v=16, d_c=12, d_r=0)
    c = wl.make_case("vo", s, [37, 5, 16, 1, 0], page_size=16, cache_dtype="bf16", paged=True, seed=41, poison_unused=True)
    assert c.kr_pool.size == 0 and c.cache_bytes() * 2 == int(c.seq_lens.sum()) * 2 * s.G * s.d_v * 2
    q_abs = orc.absorb_case(c)
    assert q_abs.shape == (c.B, s.H, s.d_v)
    out, lse = orc.decode_case(c)
    V = torch.from_numpy(wl.pool_to_f64(c.v_pool)); M = torch.from_numpy(c.M.astype(np.float64))
    for b in range(c.B):
        L = int(c.seq_lens[b])
        if L == 0:
            assert np.all(out[b] == 0) and np.all(np.isneginf(lse[b]))
            continue
        pages = [c.page_of(b, t // c.page_size) for t in range(L)]; slots = [t % c.page_size for t in range(L)]
        q = torch.from_numpy(c.q_c[b].astype(np.float64))
        K = torch.stack([V[pages, h // (s.H // s.G), slots] @ M[h] for h in range(s.H)])
        Vv = torch.stack([V[pages, h // (s.H // s.G), slots] for h in range(s.H)])
        ref = torch.nn.functional.scaled_dot_product_attention(q[None, :, None, :], K[None], Vv[None],
                                                               scale=1.0 / math.sqrt(s.d_c))[0, :, 0]
        assert np.allclose(out[b], ref.numpy(), atol=1e-12)
    # append writes value rows only
    v0 = c.v_pool.copy()
    live = c.seq_lens > 0
    c.append_pos[:] = np.maximum(c.seq_lens - 1, 0)
    assert orc.append_case(c) == 0
    assert (c.v_pool != v0).any() and c.kr_pool.size == 0


# ---------------------------------------------------------------- 8-bit (e4m3) cache codes
def test_e4m3_codec_against_library_cast_and_by_hand():
    codes = np.arange(256, dtype=np.uint8)
    lib_vals = torch.from_numpy(codes).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    mine = np.array([orc.e4m3_to_double(int(c)) for c in codes])
    gen = wl.e4m3_bits_to_f64(codes)
    finite = ~np.isnan(lib_vals)
    assert finite.sum() == 254 and np.isnan(mine[~finite]).all() and np.isnan(gen[~finite]).all()
    assert np.array_equal(mine[finite], lib_vals[finite]) and np.array_equal(gen[finite], lib_vals[finite])
    # every finite code survives a round trip through both encoders (0x80 is -0)
    for c in codes[finite]:
        assert orc.e4m3_from_double(mine[c]) == c
    assert np.array_equal(wl.f32_to_e4m3_bits(lib_vals[finite].astype(np.float32)), codes[finite])
    # random float32 values inside the finite range: both encoders agree with the library's cast
    rng = np.random.default_rng(61)
    x = np.concatenate([rng.standard_normal(20000), rng.uniform(-448, 448, 5000), rng.standard_normal(5000) * 1e-2]).astype(np.float32)
    lib_codes = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(wl.f32_to_e4m3_bits(x), lib_codes)
    assert np.array_equal(np.array([orc.e4m3_from_double(float(v)) for v in x[:4000]], dtype=np.uint8), lib_codes[:4000])
    # by hand: ties go to the even mantissa, the subnormal quantum is 2^-9, magnitudes beyond 448 saturate
    assert orc.e4m3_from_double(1.0625) == 0x38 and orc.e4m3_from_double(1.1875) == 0x3A        # 1.0 and 1.25
    assert orc.e4m3_from_double(2.0 ** -10) == 0x00 and orc.e4m3_from_double(3 * 2.0 ** -10) == 0x02
    assert orc.e4m3_from_double(2.0 ** -6 - 2.0 ** -10) == 0x08                                   # rounds up into the normals
    assert orc.e4m3_from_double(1e6) == 0x7E and orc.e4m3_from_double(-449.0) == 0xFE and orc.e4m3_from_double(float("nan")) == 0x7F


def test_fp8_cache_decode_and_append_through_the_oracle():
    # the oracle reads e4m3 codes exactly and appends with one rounding; the decode over such a cache is the same plain
    # attention over the widened values
    c = small_case(cache_dtype="fp8")
    assert c.v_pool.dtype == np.uint8 and c.cache_bytes() == int(c.seq_lens.sum()) * c.shape.row_elems
    out, lse = orc.decode_case(c)
    V = wl.pool_to_f64(c.v_pool); KR = wl.pool_to_f64(c.kr_pool)
    q_abs = orc.absorb_case(c)
    s = c.shape
    for b in range(c.B):
        L = int(c.seq_lens[b])
        for h in range(s.H):
            g = h // (s.H // s.G)
            rows = [(c.page_of(b, t // c.page_size), t % c.page_size) for t in range(L)]
            sc = np.array([q_abs[b, h, :s.d_v] @ V[p, g, sl] + q_abs[b, h, s.d_v:] @ KR[p, sl] for p, sl in rows]) / math.sqrt(s.d_c + s.d_r)
            w = np.exp(sc - sc.max()); w /= w.sum()
            assert np.allclose(out[b, h], sum(w[t] * V[rows[t][0], g, rows[t][1]] for t in range(L)), atol=1e-13)
    v0, k0 = c.v_pool.copy(), c.kr_pool.copy()
    assert orc.append_case(c) == 0
    for b in range(c.B):
        t = int(c.append_pos[b]); p, sl = c.page_of(b, t // c.page_size), t % c.page_size
        assert np.array_equal(c.v_pool[p, :, sl], wl.f32_to_e4m3_bits(c.v_new[b]))
        rot = orc.rope(c.kr_new[b], t)
        assert np.array_equal(c.kr_pool[p, sl], np.array([orc.e4m3_from_double(float(v)) for v in rot], dtype=np.uint8))
    assert (c.v_pool != v0).sum() <= c.B * s.G * s.d_v and (c.kr_pool != k0).sum() <= c.B * s.d_r
