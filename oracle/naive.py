"""Second, deliberately naive oracle path: Python lists and the `math` module only.

TEST INFRASTRUCTURE ONLY.  Used to brute-force hand-sized cases and to cross-check the C oracle
(oracle/gva_oracle.c); written separately from it, following Algorithm 1 of the paper line by
line in its notation (1-based steps of the algorithm are noted beside the code).  Cache values are
plain Python floats (already widened from whatever storage type).
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence


def rope(x: Sequence[float], p: float, base: float = 10000.0) -> List[float]:
    """x R_p^T : rotate each pair (x[2i], x[2i+1]) by the angle p * base**(-2i/d_r)."""
    d_r = len(x)
    y = [0.0] * d_r
    for i in range(d_r // 2):
        a = p * base ** (-2.0 * i / d_r)
        y[2 * i] = x[2 * i] * math.cos(a) - x[2 * i + 1] * math.sin(a)
        y[2 * i + 1] = x[2 * i] * math.sin(a) + x[2 * i + 1] * math.cos(a)
    return y


def absorb(q_nope: Sequence[float], M_h: Sequence[Sequence[float]]) -> List[float]:
    """q~ = q^nope M_h^T with M_h of shape [d_v][d_c]  (Eq. absorb)."""
    return [sum(q_nope[j] * M_h[i][j] for j in range(len(q_nope))) for i in range(len(M_h))]


def reconstruct_key(v: Sequence[float], M_h: Sequence[Sequence[float]]) -> List[float]:
    """k^nope = v M_h  (Eq. kvm / Eq. knope): a d_c-wide content key from a d_v-wide value."""
    d_v, d_c = len(M_h), len(M_h[0])
    return [sum(v[i] * M_h[i][j] for i in range(d_v)) for j in range(d_c)]


def softmax(s: Sequence[float]) -> List[float]:
    m = max(s)
    e = [math.exp(x - m) for x in s]
    z = sum(e)
    return [x / z for x in e]


def decode_head(q_tilde: Sequence[float], q_rope_rot: Sequence[float], V_g: Sequence[Sequence[float]],
                k_rope: Sequence[Sequence[float]], d_qk: int):
    """Algorithm 1, the two attention lines for one head:
    s_j = q~ . v_j + q^rope . k^rope_j ;  o = softmax(s / sqrt(d_qk)) V_g.   Returns (o, lse)."""
    T = len(V_g)
    d_v = len(q_tilde)
    if T == 0:
        return [0.0] * d_v, -math.inf
    s = []
    for j in range(T):
        sj = sum(q_tilde[i] * V_g[j][i] for i in range(d_v))
        sj += sum(q_rope_rot[k] * k_rope[j][k] for k in range(len(q_rope_rot)))
        s.append(sj / math.sqrt(d_qk))
    p = softmax(s)
    o = [sum(p[j] * V_g[j][i] for j in range(T)) for i in range(d_v)]
    m = max(s)
    lse = m + math.log(sum(math.exp(x - m) for x in s))
    return o, lse


def decode_step(q_c, q_r, M, q_pos, V_tokens, KR_tokens, H: int, G: int, d_c: int, base: float = 10000.0):
    """Whole-batch decode by explicit loops.

    q_c[b][h][d_c], q_r[b][h][d_r], M[h][d_v][d_c], q_pos[b];
    V_tokens[b][t][g] = value row (list of d_v floats) of token t, group g, already gathered in
    logical order; KR_tokens[b][t] = cached (already rotated) positional key.
    Returns out[b][h][d_v], lse[b][h].
    """
    out, lses = [], []
    for b in range(len(q_c)):
        ob, lb = [], []
        for h in range(H):
            g = h // (H // G)
            d_r = len(q_r[b][h])
            qt = absorb(q_c[b][h], M[h])
            qr = rope(q_r[b][h], q_pos[b], base) if d_r else []
            Vg = [V_tokens[b][t][g] for t in range(len(V_tokens[b]))]
            o, l = decode_head(qt, qr, Vg, KR_tokens[b], d_c + d_r)
            ob.append(o)
            lb.append(l)
        out.append(ob)
        lses.append(lb)
    return out, lses


def gather_tokens(v_pool, kr_pool, block_table: Optional[Sequence[Sequence[int]]], seq_lens, P: int,
                  max_pages_per_seq: int):
    """Resolve the paged layout by direct indexing: v_pool[page][g][slot][:], kr_pool[page][slot][:]."""
    V_tokens, KR_tokens = [], []
    for b, L in enumerate(seq_lens):
        vt, kt = [], []
        for t in range(int(L)):
            page = block_table[b][t // P] if block_table is not None else b * max_pages_per_seq + t // P
            slot = t % P
            vt.append([[float(x) for x in v_pool[page][g][slot]] for g in range(len(v_pool[page]))])
            kt.append([float(x) for x in kr_pool[page][slot]])
        V_tokens.append(vt)
        KR_tokens.append(kt)
    return V_tokens, KR_tokens
