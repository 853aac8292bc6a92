"""Seeded synthetic inputs for the GVA decode path.

This module only *draws* tensors: random numbers, page permutations, ragged
lengths and the storage cast of the generated cache.  It holds none of the
method's arithmetic (no RoPE, no absorption, no softmax), so both the CUDA
library's tests and the CPU oracle's tests can feed on the same bytes without
sharing any compute code.  It depends on numpy only.

The five named workloads mirror the decode configurations the repository is
measured on (shapes of a ~350M-parameter GVA decoder: G*d_h = 256, one shared
RoPE key per token; cache count N_GVA = T*G*d_h + T*d_r, Section 3.4 / Eq. ngva):

  cfg0  B=1,   H=16 G=4  d_v=64  d_c=64  d_r=16, T=128,   f32 contiguous cache
  cfg1  B=8,   same heads,                        T=4096,  bf16 contiguous cache
  cfg2  B=32,  same heads,                        T=32768, bf16, 64-token pages, permuted block table
  cfg3  B=64,  H=32 G=8  d_v=128 d_c=128 d_r=32, seq_lens ~ U{1024..16384}, bf16 paged
  cfg4  B=128, cfg0 heads, 24 layers, T=8192 cached + one appended token, bf16 paged

Values: cache rows, queries and new rows ~ N(0,1); the maps M_h ~ N(0, 1/d_v)
(variance, the scale-matched initialisation of Appendix A, Eq. scale-init with
sigma_Q = sigma_V = 1), so reconstructed keys have unit RMS.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

MASTER_SEED = 20260913


# ----------------------------------------------------------------------------
# storage cast used when *generating* a bf16 cache (not the library's append)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).reshape(-1)
    out = np.empty(u.shape, dtype=np.uint16)
    blk = 1 << 20                                   # small blocks: the temporaries stay in cache and are reused
    t = np.empty(min(blk, max(u.size, 1)), dtype=np.uint32)
    for lo in range(0, u.size, blk):
        hi = min(u.size, lo + blk)
        tv = t[:hi - lo]
        np.right_shift(u[lo:hi], np.uint32(16), out=tv)
        np.bitwise_and(tv, np.uint32(1), out=tv)
        np.add(tv, np.uint32(0x7FFF), out=tv)
        np.add(tv, u[lo:hi], out=tv)
        np.right_shift(tv, np.uint32(16), out=tv)
        out[lo:hi] = tv
    return out.reshape(np.shape(x))


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) exactly to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_e4m3_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the 8-bit e4m3 format (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; nearest,
    ties to even; magnitudes beyond the largest finite value 448 saturate to it); returns uint8 codes."""
    x = np.ascontiguousarray(x, dtype=np.float32).astype(np.float64)
    sign = np.where(np.signbit(x), 0x80, 0).astype(np.uint8)
    a = np.minimum(np.abs(x), 448.0)
    _, e = np.frexp(np.where(a > 0, a, 1.0))
    eu = np.maximum(e - 1, -6)                                  # below 2^-6 the quantum is fixed at 2^-9
    y = np.ldexp(np.rint(np.ldexp(a, 3 - eu)), eu - 3)         # rint: ties to even
    _, e2 = np.frexp(np.where(y > 0, y, 1.0))
    eu2 = e2 - 1
    normal = y >= 2.0 ** -6
    mant = np.where(normal, np.ldexp(y, 3 - eu2) - 8.0, np.ldexp(y, 9)).astype(np.int64)
    expo = np.where(normal, eu2 + 7, 0).astype(np.int64)
    code = ((expo << 3) | mant).astype(np.uint8)
    code = np.where(np.isnan(x), np.uint8(0x7F), code | sign)
    return code.astype(np.uint8)


def e4m3_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Widen e4m3 codes (uint8) exactly to float64."""
    b = np.ascontiguousarray(b, dtype=np.uint8).astype(np.int64)
    e, m = (b >> 3) & 15, b & 7
    v = np.where(e == 0, np.ldexp(m.astype(np.float64), -9), np.ldexp(1.0 + m / 8.0, e - 7))
    v = np.where((b & 0x7F) == 0x7F, np.nan, v)
    return np.where(b & 0x80, -v, v)


def pool_to_f64(pool: np.ndarray) -> np.ndarray:
    """Cache pool (uint16 bf16 bits, uint8 e4m3 codes or float32) widened exactly to float64."""
    if pool.dtype == np.uint16:
        return bf16_bits_to_f32(pool).astype(np.float64)
    if pool.dtype == np.uint8:
        return e4m3_bits_to_f64(pool)
    return pool.astype(np.float64)


BF16_NAN_BITS = np.uint16(0x7FC0)


# ----------------------------------------------------------------------------
@dataclass(frozen=True)
class HeadShape:
    H: int      # query heads
    G: int      # value groups; head h reads group h // (H // G)
    d_v: int    # value width (paper d_h)
    d_c: int    # content-key width (paper d_n)
    d_r: int    # RoPE width

    @property
    def row_elems(self) -> int:
        """Cached scalars per token: G*d_v + d_r (Eq. ngva)."""
        return self.G * self.d_v + self.d_r


SHAPE_A = HeadShape(H=16, G=4, d_v=64, d_c=64, d_r=16)
SHAPE_B = HeadShape(H=32, G=8, d_v=128, d_c=128, d_r=32)
SHAPE_C = HeadShape(H=16, G=4, d_v=64, d_c=64, d_r=24)      # the paper's second tested RoPE width (48-byte k_r rows)
SHAPE_A0 = HeadShape(H=16, G=4, d_v=64, d_c=64, d_r=0)      # value-only cache: no positional slice (half the bytes of matched GQA)
SHAPE_B0 = HeadShape(H=32, G=8, d_v=128, d_c=128, d_r=0)


@dataclass
class DecodeCase:
    """One batch of decode inputs.  Pools are host arrays in *storage* dtype."""
    name: str
    shape: HeadShape
    B: int
    page_size: int
    cache_dtype: str                      # "bf16" | "f32" | "fp8" (e4m3 codes)
    num_pages: int
    max_pages_per_seq: int
    v_pool: np.ndarray                    # [num_pages, G, page_size, d_v]  uint16 (bf16 bits) | float32
    kr_pool: np.ndarray                   # [num_pages, page_size, d_r]
    block_table: Optional[np.ndarray]     # int32 [B, max_pages_per_seq] or None (contiguous)
    seq_lens: np.ndarray                  # int32 [B]  tokens attended
    q_c: np.ndarray                       # f32 [B, H, d_c]
    q_r: np.ndarray                       # f32 [B, H, d_r]   (unrotated)
    M: np.ndarray                         # f32 [H, d_v, d_c]
    q_pos: np.ndarray                     # int32 [B]
    v_new: np.ndarray                     # f32 [B, G, d_v]   rows for cache append
    kr_new: np.ndarray                    # f32 [B, d_r]      unrotated positional key
    append_pos: np.ndarray                # int32 [B]
    rope_base: float = 10000.0
    meta: dict = field(default_factory=dict)

    @property
    def elem_size(self) -> int:
        return {"bf16": 2, "fp8": 1}.get(self.cache_dtype, 4)

    def cache_bytes(self) -> int:
        """Live cache bytes a decode step must stream: sum_b seq_len * (G*d_v + d_r) * elem."""
        return int(self.seq_lens.astype(np.int64).sum()) * self.shape.row_elems * self.elem_size

    def algorithmic_bytes(self) -> int:
        """Cache stream + absorbed queries read + outputs written (f32)."""
        s = self.shape
        return self.cache_bytes() + self.B * s.H * (s.d_v + s.d_r) * 4 + self.B * s.H * s.d_v * 4

    def page_of(self, b: int, j: int) -> int:
        if self.block_table is None:
            return b * self.max_pages_per_seq + j
        return int(self.block_table[b, j])


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(seed))


def _normal_pool(rng: np.random.Generator, shape, cache_dtype: str, chunk_elems: int = 1 << 25) -> np.ndarray:
    """N(0,1) pool in storage dtype, generated in slabs so the f32 temporary stays small.

    A pool of more than one slab is drawn slab by slab from independent streams -- slab k from the caller's Philox
    generator jumped k + 1 times (2^128 draws apart each) -- on a few threads; a pool of one slab is drawn from the
    caller's generator itself."""
    n = int(np.prod(shape))
    if cache_dtype == "f32" and n <= chunk_elems:
        return rng.standard_normal(n, dtype=np.float32).reshape(shape)
    fp8 = cache_dtype == "fp8"
    out = np.empty(n, dtype=np.float32 if cache_dtype == "f32" else (np.uint8 if fp8 else np.uint16))
    if fp8:
        chunk_elems = min(chunk_elems, 1 << 22)         # the e4m3 cast works in float64 temporaries
    cast = (lambda d: d) if cache_dtype == "f32" else (f32_to_e4m3_bits if fp8 else f32_to_bf16_bits)
    if n <= chunk_elems:
        out[:] = cast(rng.standard_normal(n, dtype=np.float32))
        return out.reshape(shape)
    slabs = [(k, lo, min(n, lo + chunk_elems)) for k, lo in enumerate(range(0, n, chunk_elems))]
    base = rng.bit_generator

    def fill(job):
        k, lo, hi = job
        sub = np.random.Generator(base.jumped(k + 1))
        out[lo:hi] = cast(sub.standard_normal(hi - lo, dtype=np.float32))

    from concurrent.futures import ThreadPoolExecutor
    import os
    with ThreadPoolExecutor(max_workers=max(1, min(8, len(os.sched_getaffinity(0))))) as pool:
        list(pool.map(fill, slabs))
    return out.reshape(shape)


def make_case(name: str, shape: HeadShape, seq_lens, *, page_size: int, cache_dtype: str = "bf16",
              paged: bool = True, seed: int = MASTER_SEED, q_pos=None, append_pos=None,
              extra_pages: int = 0, max_pages_per_seq: Optional[int] = None,
              poison_unused: bool = False, m_var: Optional[float] = None,
              q_gain: float = 1.0) -> DecodeCase:
    """General seeded generator.

    paged=True  : physical pages are a seeded random permutation; block-table entries beyond a
                  sequence's live range are -1.
    paged=False : block_table is None and page j of sequence b is b*max_pages_per_seq + j.
    poison_unused: page tails past seq_len and never-referenced pages are filled with NaN
                  (they must not influence any result).
    append_pos  : defaults to seq_len-1 clipped at 0 (the slot of the current token, so that an
                  append followed by a decode over seq_len tokens follows Algorithm 1's order).
    """
    rng = _rng(seed)
    seq_lens = np.asarray(seq_lens, dtype=np.int32)
    B = int(seq_lens.shape[0])
    P = int(page_size)
    pages_per = (seq_lens.astype(np.int64) + P - 1) // P
    pages_alloc = np.maximum(pages_per, 1)                      # every sequence owns >= 1 page (append target)
    if max_pages_per_seq is None:
        max_pages_per_seq = int(pages_alloc.max()) if B else 1
    if paged:
        num_pages = int(pages_alloc.sum()) + int(extra_pages)
        perm = rng.permutation(num_pages).astype(np.int32)
        block_table = np.full((B, max_pages_per_seq), -1, dtype=np.int32)
        off = 0
        for b in range(B):
            n = int(pages_alloc[b])
            block_table[b, :n] = perm[off:off + n]
            off += n
    else:
        num_pages = B * max_pages_per_seq + int(extra_pages)
        block_table = None

    v_pool = _normal_pool(rng, (num_pages, shape.G, P, shape.d_v), cache_dtype)
    kr_pool = _normal_pool(rng, (num_pages, P, shape.d_r), cache_dtype)
    q_c = (q_gain * rng.standard_normal((B, shape.H, shape.d_c), dtype=np.float32)).astype(np.float32)
    q_r = (q_gain * rng.standard_normal((B, shape.H, shape.d_r), dtype=np.float32)).astype(np.float32)
    var = (1.0 / shape.d_v) if m_var is None else m_var
    M = (rng.standard_normal((shape.H, shape.d_v, shape.d_c), dtype=np.float32) * np.float32(np.sqrt(var))).astype(np.float32)
    v_new = rng.standard_normal((B, shape.G, shape.d_v), dtype=np.float32)
    kr_new = rng.standard_normal((B, shape.d_r), dtype=np.float32)
    q_pos = seq_lens.copy() if q_pos is None else np.asarray(q_pos, dtype=np.int32)
    if append_pos is None:
        append_pos = np.maximum(seq_lens - 1, 0).astype(np.int32)
    else:
        append_pos = np.asarray(append_pos, dtype=np.int32)

    case = DecodeCase(name=name, shape=shape, B=B, page_size=P, cache_dtype=cache_dtype, num_pages=num_pages,
                      max_pages_per_seq=int(max_pages_per_seq), v_pool=v_pool, kr_pool=kr_pool,
                      block_table=block_table, seq_lens=seq_lens, q_c=q_c, q_r=q_r, M=M, q_pos=q_pos,
                      v_new=v_new, kr_new=kr_new, append_pos=append_pos,
                      meta={"seed": seed, "paged": paged, "total_tokens": int(seq_lens.astype(np.int64).sum())})
    if poison_unused:
        poison_unused_slots(case)
    return case


def poison_unused_slots(case: DecodeCase) -> None:
    """Overwrite every cache slot that no live token occupies with NaN (in place)."""
    P = case.page_size
    live = np.zeros((case.num_pages, P), dtype=bool)
    for b in range(case.B):
        L = int(case.seq_lens[b])
        for j in range((L + P - 1) // P):
            n = min(P, L - j * P)
            live[case.page_of(b, j), :n] = True
    dead = ~live
    if case.cache_dtype == "bf16":
        case.v_pool[np.broadcast_to(dead[:, None, :], case.v_pool.shape[:3])] = BF16_NAN_BITS
        case.kr_pool[dead] = BF16_NAN_BITS
    elif case.cache_dtype == "fp8":
        case.v_pool[np.broadcast_to(dead[:, None, :], case.v_pool.shape[:3])] = np.uint8(0x7F)     # the e4m3 NaN code
        case.kr_pool[dead] = np.uint8(0x7F)
    else:
        case.v_pool[np.broadcast_to(dead[:, None, :], case.v_pool.shape[:3])] = np.nan
        case.kr_pool[dead] = np.nan


# ----------------------------------------------------------------------------
# the five named workloads
# ----------------------------------------------------------------------------
def config0(seed: int = MASTER_SEED) -> DecodeCase:
    return make_case("cfg0", SHAPE_A, [128], page_size=64, cache_dtype="f32", paged=False, seed=seed)


def config1(seed: int = MASTER_SEED + 1000) -> DecodeCase:
    return make_case("cfg1", SHAPE_A, [4096] * 8, page_size=64, cache_dtype="bf16", paged=False, seed=seed)


def config2(seed: int = MASTER_SEED + 2000, B: int = 32, T: int = 32768) -> DecodeCase:
    return make_case("cfg2", SHAPE_A, [T] * B, page_size=64, cache_dtype="bf16", paged=True, seed=seed)


def config3_seq_lens(seed: int = MASTER_SEED + 3000, B: int = 64, lo: int = 1024, hi: int = 16384) -> np.ndarray:
    return _rng(seed ^ 0x5EED).integers(lo, hi + 1, size=B).astype(np.int32)


def config3(seed: int = MASTER_SEED + 3000, B: int = 64, poison: bool = False) -> DecodeCase:
    lens = config3_seq_lens(seed, B)
    return make_case("cfg3", SHAPE_B, lens, page_size=64, cache_dtype="bf16", paged=True, seed=seed,
                     poison_unused=poison)


def config4_layer(layer: int, seed: int = MASTER_SEED + 4000, B: int = 128, T: int = 8192) -> DecodeCase:
    """One layer of the 24-layer stack: cache holds T tokens, the step appends at position T and
    then attends over T+1 tokens with the query at position T (Algorithm 1's append-before-attend)."""
    lens = np.full(B, T + 1, dtype=np.int32)
    case = make_case(f"cfg4.L{layer}", SHAPE_A, lens, page_size=64, cache_dtype="bf16", paged=True,
                     seed=seed + layer, q_pos=np.full(B, T, dtype=np.int32),
                     append_pos=np.full(B, T, dtype=np.int32))
    case.meta["layer"] = layer
    return case


CONFIG4_LAYERS = 24


def gqa_case(name: str, H: int, G: int, d_h: int, seq_lens, *, page_size: int = 64, paged: bool = True,
             cache_dtype: str = "bf16", seed: int = MASTER_SEED + 5000) -> dict:
    """Matched GQA decode inputs: K (already rotated) and V pools [num_pages, G, P, d_h], q [B, H, d_h]."""
    rng = _rng(seed)
    seq_lens = np.asarray(seq_lens, dtype=np.int32)
    B = int(seq_lens.shape[0])
    P = page_size
    pages_alloc = np.maximum((seq_lens.astype(np.int64) + P - 1) // P, 1)
    max_pages = int(pages_alloc.max())
    if paged:
        num_pages = int(pages_alloc.sum())
        perm = rng.permutation(num_pages).astype(np.int32)
        bt = np.full((B, max_pages), -1, dtype=np.int32)
        off = 0
        for b in range(B):
            n = int(pages_alloc[b])
            bt[b, :n] = perm[off:off + n]
            off += n
    else:
        num_pages = B * max_pages
        bt = None
    k_pool = _normal_pool(rng, (num_pages, G, P, d_h), cache_dtype)
    v_pool = _normal_pool(rng, (num_pages, G, P, d_h), cache_dtype)
    q = rng.standard_normal((B, H, d_h), dtype=np.float32)
    return dict(name=name, H=H, G=G, d_h=d_h, B=B, page_size=P, num_pages=num_pages, max_pages_per_seq=max_pages,
                k_pool=k_pool, v_pool=v_pool, block_table=bt, seq_lens=seq_lens, q=q, cache_dtype=cache_dtype)


# ---- prefill / chunked prefill: several query tokens per sequence ------------------------------------
@dataclass
class PrefillCase:
    """A chunk of new tokens per sequence on top of a (possibly empty) cached context.

    `cache` is a DecodeCase whose pools already hold every token (context and chunk) and whose seq_lens are
    ctx_lens + q_lens; its per-sequence q_c / q_r / v_new / kr_new fields are not used.  Query token i of
    sequence b is row cu_q[b] + i of q_c / q_r and sits at position ctx_lens[b] + i."""
    name: str
    cache: DecodeCase
    ctx_lens: np.ndarray                  # int32 [B]   tokens cached before the chunk
    q_lens: np.ndarray                    # int32 [B]   new tokens
    cu_q: np.ndarray                      # int32 [B+1] exclusive prefix sums of q_lens
    q_c: np.ndarray                       # f32 [n_q, H, d_c]
    q_r: np.ndarray                       # f32 [n_q, H, d_r]   unrotated
    q_pos: np.ndarray                     # int32 [n_q] position of every query token
    q_seq: np.ndarray                     # int32 [n_q] sequence of every query token
    v_new: np.ndarray                     # f32 [n_q, G, d_v]  rows for a chunk append
    kr_new: np.ndarray                    # f32 [n_q, d_r]     unrotated positional keys for a chunk append

    @property
    def n_q(self) -> int:
        return int(self.cu_q[-1])

    def pairs(self) -> int:
        """(query, key) pairs under the causal mask, summed over sequences (per head)."""
        c, n = self.ctx_lens.astype(np.int64), self.q_lens.astype(np.int64)
        return int((n * c + n * (n + 1) // 2).sum())

    def flops(self) -> int:
        """Multiply-adds x 2 of the absorbed form: per pair and head (d_v + d_r) for the score, d_v for the value sum."""
        s = self.cache.shape
        return 2 * self.pairs() * s.H * (2 * s.d_v + s.d_r)


def make_prefill_case(name: str, shape: HeadShape, ctx_lens, q_lens, *, page_size: int = 64, cache_dtype: str = "bf16",
                      paged: bool = True, seed: int = MASTER_SEED + 7000, poison_unused: bool = False,
                      extra_pages: int = 0, q_gain: float = 1.0) -> PrefillCase:
    ctx_lens = np.asarray(ctx_lens, dtype=np.int32)
    q_lens = np.asarray(q_lens, dtype=np.int32)
    cache = make_case(name, shape, ctx_lens + q_lens, page_size=page_size, cache_dtype=cache_dtype, paged=paged, seed=seed,
                      extra_pages=extra_pages, poison_unused=poison_unused)
    rng = _rng(seed + 1)
    cu_q = np.zeros(len(q_lens) + 1, dtype=np.int32)
    cu_q[1:] = np.cumsum(q_lens)
    n_q = int(cu_q[-1])
    q_c = (q_gain * rng.standard_normal((n_q, shape.H, shape.d_c), dtype=np.float32)).astype(np.float32)
    q_r = (q_gain * rng.standard_normal((n_q, shape.H, shape.d_r), dtype=np.float32)).astype(np.float32)
    v_new = rng.standard_normal((n_q, shape.G, shape.d_v), dtype=np.float32)
    kr_new = rng.standard_normal((n_q, shape.d_r), dtype=np.float32)
    q_seq = np.repeat(np.arange(len(q_lens), dtype=np.int32), q_lens)
    q_pos = (ctx_lens[q_seq] + (np.arange(n_q, dtype=np.int32) - cu_q[q_seq])).astype(np.int32)
    return PrefillCase(name=name, cache=cache, ctx_lens=ctx_lens, q_lens=q_lens, cu_q=cu_q, q_c=q_c, q_r=q_r,
                       q_pos=q_pos, q_seq=q_seq, v_new=v_new, kr_new=kr_new)


def prefill_bench_case(seed: int = MASTER_SEED + 7100, B: int = 8, T: int = 8192) -> PrefillCase:
    """Whole-prompt prefill on the headline head shape: B prompts of T tokens, empty context, 64-token pages."""
    return make_prefill_case("prefill", SHAPE_A, [0] * B, [T] * B, page_size=64, seed=seed)


def prefill_bench_case_b(seed: int = MASTER_SEED + 7200, B: int = 4, T: int = 8192) -> PrefillCase:
    """Whole-prompt prefill on the wider head shape (H=32, G=8, d_v=128, d_c=128, d_r=32)."""
    return make_prefill_case("prefill_b", SHAPE_B, [0] * B, [T] * B, page_size=64, seed=seed)


def layer_weights(shape: HeadShape, d_model: int, B: int, seed: int = MASTER_SEED + 6000) -> dict:
    """Seeded projections around the attention of one layer and one hidden state per sequence.
    Every weight ~ N(0, 1/fan_in) (so projected activations stay unit-scale), x ~ N(0, 1):
      W_q_nope [d_model, H, d_c], W_q_rope [d_model, H, d_r], W_v [d_model, G, d_v], W_r [d_model, d_r],
      W_o [H*d_v, d_model], x [B, d_model]."""
    rng = _rng(seed)
    sd = np.float32(1.0 / np.sqrt(d_model))
    n = lambda *sh: (rng.standard_normal(sh, dtype=np.float32) * sd).astype(np.float32)
    return dict(d_model=d_model, W_q_nope=n(d_model, shape.H, shape.d_c), W_q_rope=n(d_model, shape.H, shape.d_r),
                W_v=n(d_model, shape.G, shape.d_v), W_r=n(d_model, shape.d_r),
                W_o=(rng.standard_normal((shape.H * shape.d_v, d_model), dtype=np.float32)
                     * np.float32(1.0 / np.sqrt(shape.H * shape.d_v))).astype(np.float32),
                x=rng.standard_normal((B, d_model), dtype=np.float32))
