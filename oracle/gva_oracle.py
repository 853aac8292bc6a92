"""ctypes front end of the fp64 CPU oracle (oracle/gva_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the benchmark's CPU-baseline
leg.  The CUDA library never imports or links it, and it never imports the CUDA package.

All functions take and return numpy arrays.  Cache pools are passed in storage dtype
(uint16 = bfloat16 bit patterns, or float32); everything else is float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gva_oracle.c")
_LIB = os.path.join(_HERE, "libgva_oracle.so")
_lib = None

F32, BF16, E4M3 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over (batch, head)); returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_bf16_from_double.restype = ctypes.c_uint16
        _lib.oracle_bf16_from_double.argtypes = [ctypes.c_double]
        _lib.oracle_e4m3_from_double.restype = ctypes.c_uint8
        _lib.oracle_e4m3_from_double.argtypes = [ctypes.c_double]
        _lib.oracle_e4m3_to_double.restype = ctypes.c_double
        _lib.oracle_e4m3_to_double.argtypes = [ctypes.c_uint8]
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_append.restype = ctypes.c_int
        _lib.oracle_append_chunk.restype = ctypes.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _dt(pool: np.ndarray) -> int:
    if pool.dtype == np.uint16:
        return BF16
    if pool.dtype == np.float32:
        return F32
    if pool.dtype == np.uint8:
        return E4M3
    raise TypeError("cache pools must be uint16 (bf16 bits), uint8 (e4m3 codes) or float32")


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_threads(n: int) -> None:
    lib().oracle_set_threads(ctypes.c_int(int(n)))


def bf16_from_double(x: float) -> int:
    return int(lib().oracle_bf16_from_double(ctypes.c_double(float(x))))


def e4m3_from_double(x: float) -> int:
    return int(lib().oracle_e4m3_from_double(float(x)))


def e4m3_to_double(code: int) -> float:
    return float(lib().oracle_e4m3_to_double(int(code)))


def rope(x, pos: float, base: float = 10000.0) -> np.ndarray:
    """y = x R_pos^T on the last axis (pairs (2i, 2i+1))."""
    x = _f64(x)
    y = np.empty_like(x)
    d_r = x.shape[-1]
    if d_r == 0:                     # value-only cache (Section 3.4): there is no positional slice to rotate
        return y
    xf, yf = x.reshape(-1, d_r), y.reshape(-1, d_r)
    for r in range(xf.shape[0]):
        lib().oracle_rope(_p(xf[r]), ctypes.c_int(d_r), ctypes.c_double(float(pos)), ctypes.c_double(base), _p(yf[r]))
    return y


def absorb(q_c, q_r, M, q_pos, base: float = 10000.0) -> np.ndarray:
    """q_abs [B,H,d_v+d_r]: absorbed content query q_c M_h^T, then q_r rotated at q_pos[b]."""
    q_c, q_r, M, q_pos = _f64(q_c), _f64(q_r), _f64(M), _i32(q_pos)
    B, H, d_c = q_c.shape
    d_r = q_r.shape[-1]
    d_v = M.shape[1]
    assert M.shape == (H, d_v, d_c)
    out = np.empty((B, H, d_v + d_r), dtype=np.float64)
    lib().oracle_absorb(_p(q_c), _p(q_r), _p(M), _p(q_pos), *map(ctypes.c_int, (B, H, d_v, d_c, d_r)),
                        ctypes.c_double(base), _p(out))
    return out


def append(v_pool, kr_pool, block_table, v_new, kr_new, pos, base: float = 10000.0,
           max_pages_per_seq: Optional[int] = None) -> int:
    """In-place cache append (Algorithm 1's append lines).  Returns 0 or 1+b of the first bad page."""
    dt = _dt(v_pool)
    assert v_pool.flags.c_contiguous and kr_pool.flags.c_contiguous and _dt(kr_pool) == dt
    num_pages, G, P, d_v = v_pool.shape
    d_r = kr_pool.shape[-1]
    v_new, kr_new, pos = _f64(v_new), _f64(kr_new), _i32(pos)
    B = pos.shape[0]
    bt = None if block_table is None else _i32(block_table)
    max_pages = bt.shape[1] if bt is not None else int(max_pages_per_seq)
    return int(lib().oracle_append(_p(v_pool), _p(kr_pool), ctypes.c_int(dt), _p(bt), ctypes.c_int(num_pages),
                                   ctypes.c_int(max_pages), ctypes.c_int(P), ctypes.c_int(G), ctypes.c_int(d_v),
                                   ctypes.c_int(d_r), ctypes.c_double(base), _p(v_new), _p(kr_new), _p(pos),
                                   ctypes.c_int(B)))


def decode(v_pool, kr_pool, block_table, seq_lens, q_abs, H: int, scale: Optional[float] = None,
           d_c: Optional[int] = None, max_pages_per_seq: Optional[int] = None):
    """(out [B,H,d_v], lse [B,H]) by the plain definition.  scale defaults to 1/sqrt(d_c+d_r)."""
    dt = _dt(v_pool)
    assert v_pool.flags.c_contiguous and kr_pool.flags.c_contiguous and _dt(kr_pool) == dt
    _, G, P, d_v = v_pool.shape
    d_r = kr_pool.shape[-1]
    q_abs, seq_lens = _f64(q_abs), _i32(seq_lens)
    B = seq_lens.shape[0]
    assert q_abs.shape == (B, H, d_v + d_r)
    if scale is None:
        scale = 1.0 / np.sqrt(float((d_v if d_c is None else d_c) + d_r))
    bt = None if block_table is None else _i32(block_table)
    max_pages = bt.shape[1] if bt is not None else int(max_pages_per_seq)
    out = np.empty((B, H, d_v), dtype=np.float64)
    lse = np.empty((B, H), dtype=np.float64)
    lib().oracle_decode(_p(v_pool), _p(kr_pool), ctypes.c_int(dt), _p(bt), ctypes.c_int(max_pages), ctypes.c_int(P),
                        _p(seq_lens), _p(q_abs), ctypes.c_double(scale), *map(ctypes.c_int, (B, H, G, d_v, d_r)),
                        _p(out), _p(lse))
    return out, lse


def decode_weights(v_pool, kr_pool, block_table, seq_lens, q_abs, H: int, b: int, h: int, scale: float,
                   max_pages_per_seq: Optional[int] = None) -> np.ndarray:
    """Softmax weights p_t of one (b, h) row."""
    dt = _dt(v_pool)
    _, G, P, d_v = v_pool.shape
    d_r = kr_pool.shape[-1]
    q_abs, seq_lens = _f64(q_abs), _i32(seq_lens)
    bt = None if block_table is None else _i32(block_table)
    max_pages = bt.shape[1] if bt is not None else int(max_pages_per_seq)
    p = np.empty(int(seq_lens[b]), dtype=np.float64)
    lib().oracle_decode_weights(_p(v_pool), _p(kr_pool), ctypes.c_int(dt), _p(bt), ctypes.c_int(max_pages),
                                ctypes.c_int(P), _p(seq_lens), _p(q_abs), ctypes.c_double(scale),
                                *map(ctypes.c_int, (H, G, d_v, d_r, b, h)), _p(p))
    return p


def gqa_decode(k_pool, v_pool, block_table, seq_lens, q, scale: Optional[float] = None,
               max_pages_per_seq: Optional[int] = None):
    """Matched GQA decode: (out [B,H,d_h], lse [B,H]); scale defaults to 1/sqrt(d_h)."""
    dt = _dt(v_pool)
    assert _dt(k_pool) == dt and k_pool.shape == v_pool.shape
    _, G, P, d_h = v_pool.shape
    q, seq_lens = _f64(q), _i32(seq_lens)
    B, H, _ = q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(float(d_h))
    bt = None if block_table is None else _i32(block_table)
    max_pages = bt.shape[1] if bt is not None else int(max_pages_per_seq)
    out = np.empty((B, H, d_h), dtype=np.float64)
    lse = np.empty((B, H), dtype=np.float64)
    lib().oracle_gqa_decode(_p(k_pool), _p(v_pool), ctypes.c_int(dt), _p(bt), ctypes.c_int(max_pages), ctypes.c_int(P),
                            _p(seq_lens), _p(q), ctypes.c_double(scale), *map(ctypes.c_int, (B, H, G, d_h)),
                            _p(out), _p(lse))
    return out, lse


# ---- projections around the attention (Algorithm 1's first lines and the output projection) ----
def matmul(x, W) -> np.ndarray:
    """y = x W by the plain triple loop in fp64."""
    x, W = _f64(x), _f64(W)
    B, K = x.shape
    K2, N = W.shape
    assert K == K2
    y = np.empty((B, N), dtype=np.float64)
    lib().oracle_matmul(_p(x), _p(W), *map(ctypes.c_int, (B, K, N)), _p(y))
    return y


def fold_maps(W_q_nope, M) -> np.ndarray:
    """W_abs[m,h,:] = W_q_nope[m,h,:] M_h^T  ([d_model,H,d_c] x [H,d_v,d_c] -> [d_model,H,d_v])."""
    W_q_nope, M = _f64(W_q_nope), _f64(M)
    d_model, H, d_c = W_q_nope.shape
    d_v = M.shape[1]
    out = np.empty((d_model, H, d_v), dtype=np.float64)
    lib().oracle_fold_maps(_p(W_q_nope), _p(M), *map(ctypes.c_int, (d_model, H, d_v, d_c)), _p(out))
    return out


def bf16_round(a) -> np.ndarray:
    """Values rounded to bfloat16 (nearest even, straight from fp64), returned as uint16 bit patterns."""
    a = _f64(a)
    out = np.empty(a.shape, dtype=np.uint16)
    flat, of = a.ravel(), out.ravel()
    for i in range(flat.size):
        of[i] = lib().oracle_bf16_from_double(ctypes.c_double(float(flat[i])))
    return out


def pack_input_weights(W_q_nope, W_q_rope, W_v, W_r, M) -> np.ndarray:
    """The packed input projection [d_model, H*(d_v+d_r) + G*d_v + d_r] in fp64: per head the folded content
    columns W_q_nope_h M_h^T then the positional query columns, then the value columns, then the positional key."""
    W_q_nope, W_q_rope, W_v, W_r = _f64(W_q_nope), _f64(W_q_rope), _f64(W_v), _f64(W_r)
    d_model, H, _ = W_q_nope.shape
    W_abs = fold_maps(W_q_nope, M)
    per_head = np.concatenate([W_abs, W_q_rope], axis=2)                  # [d_model, H, d_v + d_r]
    return np.concatenate([per_head.reshape(d_model, -1), W_v.reshape(d_model, -1), W_r.reshape(d_model, -1)], axis=1)


def project_in(x, W_in, H: int, G: int, d_v: int, d_r: int):
    """x W_in split into (q_tilde [B,H,d_v], q_rope [B,H,d_r] unrotated, v_new [B,G,d_v], kr_new [B,d_r] unrotated)."""
    y = matmul(x, W_in)
    B = y.shape[0]
    nq = H * (d_v + d_r)
    qh = y[:, :nq].reshape(B, H, d_v + d_r)
    v = y[:, nq:nq + G * d_v].reshape(B, G, d_v)
    kr = y[:, nq + G * d_v:]
    assert kr.shape[1] == d_r
    return qh[..., :d_v].copy(), qh[..., d_v:].copy(), v.copy(), kr.copy()


def layer_step(x, W_in, W_o, v_pool, kr_pool, block_table, pos, seq_lens, H: int, G: int, d_c: int,
               base: float = 10000.0, max_pages_per_seq: Optional[int] = None):
    """One whole decode step of a GVA layer from the hidden state (Algorithm 1, then the output projection):
    project, rotate, append to the cache (in place), attend, concatenate heads, project out.
    Returns (y [B,d_model], attention output [B,H,d_v], q_abs [B,H,d_v+d_r])."""
    _, Gp, P, d_v = v_pool.shape
    d_r = kr_pool.shape[-1]
    assert Gp == G
    q_t, q_r, v_new, kr_new = project_in(x, W_in, H, G, d_v, d_r)
    pos = _i32(pos)
    q_abs = np.concatenate([q_t, np.stack([rope(q_r[b], int(pos[b]), base) for b in range(len(pos))])], axis=2)
    rc = append(v_pool, kr_pool, block_table, v_new, kr_new, pos, base, max_pages_per_seq=max_pages_per_seq)
    assert rc == 0
    out, _ = decode(v_pool, kr_pool, block_table, seq_lens, q_abs, H, scale=1.0 / np.sqrt(float(d_c + d_r)),
                    max_pages_per_seq=max_pages_per_seq)
    y = matmul(out.reshape(out.shape[0], -1), W_o)
    return y, out, q_abs


def prefill(v_pool, kr_pool, block_table, cu_q, ctx_lens, q_c, q_r, M, base: float = 10000.0,
            scale: Optional[float] = None, max_pages_per_seq: Optional[int] = None):
    """Causal attention of a chunk of new tokens per sequence with explicitly formed keys K_h = V_g M_h.
    q_c [n_q,H,d_c], q_r [n_q,H,d_r] unrotated; query i of sequence b is at position ctx_lens[b] + i and its
    value rows / positional key are already cached.  Returns (out [n_q,H,d_v], lse [n_q,H])."""
    dt = _dt(v_pool)
    assert v_pool.flags.c_contiguous and kr_pool.flags.c_contiguous and _dt(kr_pool) == dt
    _, G, P, d_v = v_pool.shape
    d_r = kr_pool.shape[-1]
    q_c, q_r, M = _f64(q_c), _f64(q_r), _f64(M)
    cu_q, ctx_lens = _i32(cu_q), _i32(ctx_lens)
    B = ctx_lens.shape[0]
    n_q, H, d_c = q_c.shape
    assert cu_q.shape == (B + 1,) and int(cu_q[-1]) == n_q and q_r.shape == (n_q, H, d_r) and M.shape == (H, d_v, d_c)
    if scale is None:
        scale = 1.0 / np.sqrt(float(d_c + d_r))
    bt = None if block_table is None else _i32(block_table)
    max_pages = bt.shape[1] if bt is not None else int(max_pages_per_seq)
    out = np.zeros((n_q, H, d_v), dtype=np.float64)
    lse = np.zeros((n_q, H), dtype=np.float64)
    lib().oracle_prefill(_p(v_pool), _p(kr_pool), ctypes.c_int(dt), _p(bt), ctypes.c_int(max_pages), ctypes.c_int(P),
                         _p(cu_q), _p(ctx_lens), _p(q_c), _p(q_r), _p(M), ctypes.c_double(base), ctypes.c_double(scale),
                         *map(ctypes.c_int, (B, H, G, d_v, d_c, d_r)), _p(out), _p(lse))
    return out, lse


def append_chunk(v_pool, kr_pool, block_table, v_new, kr_new, cu_q, ctx_lens, base: float = 10000.0,
                 max_pages_per_seq: Optional[int] = None) -> int:
    """In-place append of a chunk: token i of sequence b goes to position ctx_lens[b] + i."""
    dt = _dt(v_pool)
    assert v_pool.flags.c_contiguous and kr_pool.flags.c_contiguous and _dt(kr_pool) == dt
    num_pages, G, P, d_v = v_pool.shape
    d_r = kr_pool.shape[-1]
    v_new, kr_new, cu_q, ctx_lens = _f64(v_new), _f64(kr_new), _i32(cu_q), _i32(ctx_lens)
    B = ctx_lens.shape[0]
    bt = None if block_table is None else _i32(block_table)
    max_pages = bt.shape[1] if bt is not None else int(max_pages_per_seq)
    return int(lib().oracle_append_chunk(_p(v_pool), _p(kr_pool), ctypes.c_int(dt), _p(bt), ctypes.c_int(num_pages),
                                         ctypes.c_int(max_pages), ctypes.c_int(P), ctypes.c_int(G), ctypes.c_int(d_v),
                                         ctypes.c_int(d_r), ctypes.c_double(base), _p(v_new), _p(kr_new), _p(cu_q),
                                         _p(ctx_lens), ctypes.c_int(B)))


def prefill_case(pc):
    """Oracle outputs of a workloads.PrefillCase-like object (duck-typed)."""
    c = pc.cache
    return prefill(c.v_pool, c.kr_pool, c.block_table, pc.cu_q, pc.ctx_lens, pc.q_c, pc.q_r, c.M, c.rope_base,
                   max_pages_per_seq=c.max_pages_per_seq)


# ---- convenience over a workloads.DecodeCase-like object (duck-typed; no import of the generator) ----
def absorb_case(case) -> np.ndarray:
    return absorb(case.q_c, case.q_r, case.M, case.q_pos, case.rope_base)


def decode_case(case, q_abs=None, seq_lens=None):
    if q_abs is None:
        q_abs = absorb_case(case)
    s = case.shape
    return decode(case.v_pool, case.kr_pool, case.block_table, case.seq_lens if seq_lens is None else seq_lens,
                  q_abs, s.H, scale=1.0 / np.sqrt(float(s.d_c + s.d_r)), max_pages_per_seq=case.max_pages_per_seq)


def append_case(case) -> int:
    return append(case.v_pool, case.kr_pool, case.block_table, case.v_new, case.kr_new, case.append_pos,
                  case.rope_base, max_pages_per_seq=case.max_pages_per_seq)
