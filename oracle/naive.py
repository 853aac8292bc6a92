"""Second, deliberately naive oracle path: Python lists and the `math` module only.

TEST INFRASTRUCTURE ONLY.  Used to brute-force hand-sized cases and to cross-check the C oracle
(oracle/gva_oracle.c); written separately from it, from the paper's equations (Eq. absorb, Eq. kvm,
Eq. krope, the score equation of Section 3.3) in its notation.  Cache values are plain Python floats
(already widened from whatever storage type).
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
    """One head's attention in the absorbed form (Section 3.3 with Eq. absorb):
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


def _vec_mat(x: Sequence[float], W, n_out: int, pick) -> List[float]:
    """y[c] = sum_m x[m] * pick(W[m], c) for c < n_out: a row vector times a matrix stored row by row."""
    return [sum(x[m] * pick(W[m], c) for m in range(len(x))) for c in range(n_out)]


def layer_decode_step(x, W_Q, W_V, W_r, W_O, M, t: int, V_cache, KR_cache, H: int, G: int, d_c: int, d_r: int,
                      base: float = 10000.0):
    """One sequence's decode step from the hidden state x (list of d_model floats), in the UNABSORBED form: every
    head's keys are written out as full (d_c + d_r)-wide vectors, the content part reconstructed from the cached
    values (Eq. kvm: K_h = V_g(h) M_h) and the shared rotated positional key appended to it (Eq. krope and the
    concatenated-key score of Section 3.3), and attention is plain softmax(q k^T / sqrt(d_qk)) v over those keys.

    W_Q[m][h] = list of d_r + d_c floats (positional slice first, then content slice), W_V[m][g] = list of d_v,
    W_r[m] = list of d_r, W_O[h*d_v + i] = list of d_model.  V_cache[g] = list of cached value rows, KR_cache = list
    of cached rotated positional keys; both are extended in place by the new token (position t) before anything
    attends, so the new token sees itself.  Returns (y, per-head outputs)."""
    d_model, d_v, d_qk = len(x), len(M[0]), d_c + d_r
    # 1. the new token's cache entries: one value row per group, one rotated positional key for all heads
    for g in range(G):
        V_cache[g].append(_vec_mat(x, W_V, d_v, lambda row, i, g=g: row[g][i]))
    KR_cache.append(rope(_vec_mat(x, W_r, d_r, lambda row, k: row[k]), t, base))
    n_tok = len(KR_cache)
    # 2. full queries [q^nope | q^rope R_t^T] and full keys [v_j M_h | k^rope_j], head by head
    outs = []
    for h in range(H):
        g = h // (H // G)
        q_full = _vec_mat(x, W_Q, d_qk, lambda row, c, h=h: row[h][c])
        query = q_full[d_r:] + rope(q_full[:d_r], t, base)
        keys = [reconstruct_key(V_cache[g][j], M[h]) + list(KR_cache[j]) for j in range(n_tok)]
        weights = softmax([sum(a * b for a, b in zip(query, keys[j])) / math.sqrt(d_qk) for j in range(n_tok)])
        outs.append([sum(weights[j] * V_cache[g][j][i] for j in range(n_tok)) for i in range(d_v)])
    # 3. heads side by side, then the output projection
    concat = [v for o in outs for v in o]
    y = [sum(concat[r] * W_O[r][m] for r in range(len(concat))) for m in range(d_model)]
    return y, outs


def prefill_sequence(q_c, q_r, M, ctx: int, V_tokens, KR_tokens, H: int, G: int, base: float = 10000.0):
    """Causal attention of a chunk for ONE sequence, with explicit keys (nothing absorbed) and plain loops.

    q_c[i][h][d_c], q_r[i][h][d_r] (unrotated) for the chunk's tokens i = 0..n-1 at positions ctx + i;
    V_tokens[t][g] / KR_tokens[t] as in decode_step, holding ctx + n tokens.  Returns out[i][h][d_v]."""
    out = []
    for i in range(len(q_c)):
        t = ctx + i
        row = []
        for h in range(H):
            g = h // (H // G)
            d_c, d_r = len(q_c[i][h]), len(q_r[i][h])
            qr = rope(q_r[i][h], t, base) if d_r else []
            s = []
            for j in range(t + 1):
                k = reconstruct_key(V_tokens[j][g], M[h])
                s.append((sum(a * b for a, b in zip(q_c[i][h], k)) + sum(a * b for a, b in zip(qr, KR_tokens[j])))
                         / math.sqrt(d_c + d_r))
            p = softmax(s)
            row.append([sum(p[j] * V_tokens[j][g][d] for j in range(t + 1)) for d in range(len(M[h]))])
        out.append(row)
    return out
