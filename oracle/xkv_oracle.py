"""CPU oracle for xKV cross-layer factorisation and the Selective Reconstruction decode step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
CUDA library must compute.  It shares no code with the CUDA path and imports
nothing from the product package; only tests, the smoke check and the
benchmark's CPU-baseline leg may call it.

Conventions
-----------
* Every tensor that the library receives in bf16 is handed to the oracle as the
  same bf16 values widened to float32/float64 (no extra rounding happens here
  except where a function says it produces a bf16 tensor).
* Floating point is fp64 everywhere except `landmark_scores`, whose fp32
  sequential accumulation is part of the contract: the scores decide an integer
  result (the selected indices), so both sides must take that decision in the
  same precision and the same order.
* Symbols follow the paper: L (here T) context rows, W (here G) layers per
  window, H_q / H_kv heads, d_h head width, d = H_kv*d_h, c chunk size,
  k token budget, k_ch = ceil(k/c), n_c = ceil(T/c), rho(h) = h // n_rep.

Parity pins (tests/test_oracle_*.py): every function below is pinned by closed
forms, invariants, brute force on tiny inputs, a library routine it must reduce
to, or numbers the paper prints; none is "parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np

# --------------------------------------------------------------------------
# bf16 helper (the oracle's own; round-to-nearest-even on the fp32 bit pattern)
# --------------------------------------------------------------------------


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); returns float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = (u + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


# --------------------------------------------------------------------------
# O1  Cross-Layer Factorization  (Sec. 3.1, Eq. 1)
# --------------------------------------------------------------------------


def clf_factorize(X_layers, r: int):
    """Rank-r factorisation of the column-wise concatenation of a window's caches.

    X_layers: list of W arrays (T x d), the pre-RoPE key cache or the value cache
    of the W adjacent layers of one window (Eq. 1).  Returns (A, [B_l], sigma):
    A = U_r Sigma_r (T x r) is the shared token basis, B_l (r x d) is the l-th
    column block of V_r^T, sigma are all singular values of the concatenation.
    No centring is applied (Eq. 1 has none).  This is the exact optimum the
    paper approximates with a randomised SVD.
    """
    X_cat = np.concatenate([np.asarray(x, dtype=np.float64) for x in X_layers], axis=1)
    U, s, Vt = np.linalg.svd(X_cat, full_matrices=False)
    if not (1 <= r <= s.shape[0]):
        raise ValueError("rank out of range")
    A = U[:, :r] * s[:r][None, :]
    d = X_layers[0].shape[1]
    B = [Vt[:r, i * d:(i + 1) * d].copy() for i in range(len(X_layers))]
    return A, B, s


# --------------------------------------------------------------------------
# RoPE (rotate-half convention).  The paper factorises pre-RoPE keys while
# landmarks and queries are post-RoPE, so reconstructed key rows must be
# rotated at their token position before they meet the query.
# --------------------------------------------------------------------------


def rope_rotate(x: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Rotate rows of x (n x d_h) at integer positions pos (n,), fp64.

    theta_i = base^(-2i/d_h) for i < d_h/2, phi = pos*theta_i,
    y[i] = x[i] cos(phi) - x[i+d_h/2] sin(phi),
    y[i+d_h/2] = x[i+d_h/2] cos(phi) + x[i] sin(phi).   base <= 0: identity.
    """
    x = np.asarray(x, dtype=np.float64)
    if base <= 0:
        return x.copy()
    d_h = x.shape[-1]
    half = d_h // 2
    i = np.arange(half, dtype=np.float64)
    theta = np.power(float(base), -2.0 * i / d_h)
    phi = np.asarray(pos, dtype=np.float64)[:, None] * theta[None, :]
    cs, sn = np.cos(phi), np.sin(phi)
    x1, x2 = x[:, :half], x[:, half:]
    return np.concatenate([x1 * cs - x2 * sn, x2 * cs + x1 * sn], axis=1)


# --------------------------------------------------------------------------
# O2  Landmark construction  (App. B.1, Algorithm 1, lines 1-3)
# --------------------------------------------------------------------------


def build_landmarks(K_pre: np.ndarray, c: int, rope_base: float) -> np.ndarray:
    """Chunk means of the post-RoPE keys of one layer, rounded to bf16.

    K_pre: (H_kv, T, d_h) pre-RoPE keys (the original cache, not a reconstruction).
    Chunk j covers rows [c*j, min(c*j+c, T)); its landmark is the mean over the
    rows actually present (the 1/|C_j| form, which also covers a ragged tail).
    Returns (H_kv, n_c, d_h) float32 holding bf16 values.
    """
    H_kv, T, d_h = K_pre.shape
    n_c = -(-T // c)
    out = np.zeros((H_kv, n_c, d_h), dtype=np.float64)
    pos = np.arange(T)
    for g in range(H_kv):
        Kr = rope_rotate(K_pre[g], pos, rope_base)
        for j in range(n_c):
            rows = Kr[c * j:min(c * j + c, T)]
            out[g, j] = rows.sum(axis=0) / rows.shape[0]
    return bf16_round(out.astype(np.float32))


# --------------------------------------------------------------------------
# O3  Landmark-guided top-k chunk selection  (App. B.1, Algorithm 2)
# --------------------------------------------------------------------------


def landmark_scores(q_heads: np.ndarray, L_g: np.ndarray) -> np.ndarray:
    """Algorithm 2 line 2 for the query heads mapped to one KV head.

    q_heads (n_rep x d_h) and L_g (n_c x d_h) hold bf16 values.  Canonical
    arithmetic: acc = +0; for i = 0..d_h-1 in order acc = acc + q[i]*L[j][i]
    in fp32 (each product of two bf16 values is exact in fp32, so only the
    order matters); P = acc * s with s = 1/sqrt(d_h) computed in fp32.
    """
    q = np.asarray(q_heads, dtype=np.float32)
    L = np.asarray(L_g, dtype=np.float32)
    n_rep, d_h = q.shape
    s = np.float32(1.0) / np.sqrt(np.float32(d_h))
    P = np.empty((n_rep, L.shape[0]), dtype=np.float32)
    for h in range(n_rep):
        acc = np.zeros(L.shape[0], dtype=np.float32)
        for i in range(d_h):
            acc = acc + q[h, i] * L[:, i]
        P[h] = acc * s
    return P


def pool_scores(P: np.ndarray) -> np.ndarray:
    """Algorithm 2 line 3: max over the query heads of one KV head."""
    return P.max(axis=0)


def topk_chunks(S: np.ndarray, k_ch: int) -> np.ndarray:
    """Algorithm 2 line 4 with a fixed tie rule.

    Total order: score descending, then chunk index ascending (-0 equals +0).
    Returns the first k_ch chunk ids of that order, sorted ascending.
    """
    order = np.argsort(-(S.astype(np.float32) + np.float32(0.0)), kind="stable")
    return np.sort(order[:k_ch]).astype(np.int64)


def expand_chunks(chunks: np.ndarray, c: int, T: int) -> np.ndarray:
    """Chunk ids -> token rows c*j .. min(c*j+c, T)-1, ascending."""
    rows = []
    for j in chunks:
        rows.extend(range(int(j) * c, min(int(j) * c + c, T)))
    return np.asarray(rows, dtype=np.int32)


def union_outliers(chunks: np.ndarray, outliers, n_c: int) -> np.ndarray:
    """Algorithm 2 line 5: the selected chunks united with the head's static outlier chunks, ascending.

    Ids outside [0, n_c) are ignored and a repeated id counts once (it is a set union)."""
    if outliers is None:
        return np.asarray(chunks, dtype=np.int64)
    keep = set(int(j) for j in chunks)
    for j in np.asarray(outliers).reshape(-1):
        if 0 <= int(j) < n_c:
            keep.add(int(j))
    return np.asarray(sorted(keep), dtype=np.int64)


def sr_select(q_heads: np.ndarray, L_g: np.ndarray, k: int, c: int, T: int, outliers=None) -> np.ndarray:
    """Selected token rows for one (layer, sequence, KV head): Algorithm 2 (line 5 only if `outliers` is given)."""
    n_c = L_g.shape[0]
    k_ch = min(-(-k // c), n_c)
    S = pool_scores(landmark_scores(q_heads, L_g))
    return expand_chunks(union_outliers(topk_chunks(S, k_ch), outliers, n_c), c, T)


def min_chunk_cosine(K_rope: np.ndarray, c: int) -> np.ndarray:
    """Algorithm 1 line 4-5 (first half): r_j = min over the tokens x of chunk j of cos(K(x), landmark_j), with the
    landmark the exact (unrounded) chunk mean.  K_rope (T, d_h) post-RoPE keys of one head; returns (n_c,) fp64.
    A zero vector has cosine 0 with everything."""
    K = np.asarray(K_rope, dtype=np.float64)
    T = K.shape[0]
    n_c = -(-T // c)
    out = np.empty(n_c)
    for j in range(n_c):
        rows = K[j * c:min(T, j * c + c)]
        lm = rows.mean(axis=0)
        den = np.linalg.norm(rows, axis=1) * np.linalg.norm(lm)
        cos = np.where(den > 0, (rows @ lm) / np.where(den > 0, den, 1.0), 0.0)
        out[j] = cos.min()
    return out


def static_outliers(K_rope: np.ndarray, c: int, o: int) -> np.ndarray:
    """Algorithm 1 line 5: the o chunks with the smallest minimum within-chunk cosine (ties to the lowest
    chunk id), i.e. ArgTopK(-m, o); returned ascending."""
    m = min_chunk_cosine(K_rope, c)
    order = np.argsort(m, kind="stable")
    return np.sort(order[:min(o, m.shape[0])]).astype(np.int64)


# --------------------------------------------------------------------------
# O4  Selective reconstruction  (Sec. 3.2, Eq. 3)
# --------------------------------------------------------------------------


def sr_reconstruct(A: np.ndarray, B_head: np.ndarray, rows: np.ndarray) -> np.ndarray:
    """X_hat[S,:] = A[S,:] @ B_{l,g}   (A: T x r, B_head: r x d_h), fp64."""
    gathered = np.asarray(A)[np.asarray(rows, dtype=np.int64)].astype(np.float64)
    return gathered @ np.asarray(B_head, dtype=np.float64)


def sr_reconstruct_keys(A_k, B_k_head, rows, rope_base: float) -> np.ndarray:
    """Reconstructed key rows rotated at their token positions (position = row index)."""
    return rope_rotate(sr_reconstruct(A_k, B_k_head, rows), np.asarray(rows), rope_base)


# --------------------------------------------------------------------------
# O5  Attention over the reconstructed rows
# --------------------------------------------------------------------------


def attend(q_heads: np.ndarray, K_hat: np.ndarray, V_hat: np.ndarray, scale: float):
    """softmax(q K_hat^T * scale) V_hat per query head; returns (o, lse) in fp64.

    An empty row set gives o = 0 and lse = -inf.
    """
    q = np.asarray(q_heads, dtype=np.float64)
    n_rep = q.shape[0]
    d_v = V_hat.shape[1] if V_hat.ndim == 2 else 0
    if K_hat.shape[0] == 0:
        return np.zeros((n_rep, d_v)), np.full((n_rep,), -np.inf)
    z = (q @ np.asarray(K_hat, dtype=np.float64).T) * float(scale)
    m = z.max(axis=1, keepdims=True)
    w = np.exp(z - m)
    l = w.sum(axis=1, keepdims=True)
    o = (w @ np.asarray(V_hat, dtype=np.float64)) / l
    lse = (m + np.log(l))[:, 0]
    return o, lse


def dense_attend(q_heads, K_all, V_all, scale: float):
    """Plain softmax attention over every row, written separately from `attend`
    (row by row, no max subtraction shared with it) so that the two can pin each other."""
    q = np.asarray(q_heads, dtype=np.float64)
    K = np.asarray(K_all, dtype=np.float64)
    V = np.asarray(V_all, dtype=np.float64)
    out = np.zeros((q.shape[0], V.shape[1]))
    for h in range(q.shape[0]):
        z = np.array([float(np.dot(q[h], K[j])) * float(scale) for j in range(K.shape[0])])
        e = np.exp(z - z.max())
        out[h] = (e[:, None] * V).sum(axis=0) / e.sum()
    return out


def merge_partials(parts):
    """Merge attention results over disjoint row sets by log-sum-exp.

    parts: list of (o, lse) as returned by `attend`.  Equals `attend` on the union.
    """
    lses = np.stack([p[1] for p in parts])            # (n_parts, n_rep)
    m = lses.max(axis=0)
    w = np.exp(lses - m[None, :])                     # weight of each part
    o = sum(w[i][:, None] * parts[i][0] for i in range(len(parts))) / w.sum(axis=0)[:, None]
    return o, m + np.log(w.sum(axis=0))


# --------------------------------------------------------------------------
# The decode step of one window: select -> reconstruct -> RoPE -> attend
# --------------------------------------------------------------------------


def sr_decode_problem(q_heads, L_g, A_k, A_v, B_k_head, B_v_head, k, c, T, rope_base, scale,
                      rows=None, outliers=None):
    """One (layer, sequence, KV head) problem.  rows=None: use Algorithm 2."""
    if rows is None:
        rows = sr_select(q_heads, L_g, k, c, T, outliers)
    K_hat = sr_reconstruct_keys(A_k, B_k_head, rows, rope_base)
    V_hat = sr_reconstruct(A_v, B_v_head, rows)
    o, lse = attend(q_heads, K_hat, V_hat, scale)
    return rows, o, lse


def sr_decode_step(A_k, A_v, B_k, B_v, landmarks, q, k, c, H_kv, rope_base, scale=None,
                   sel_idx=None, sel_cnt=None, problems=None, outliers=None):
    """Whole-window decode step in the library's tensor layouts.

    A_k (B,T,r_k)  A_v (B,T,r_v)  B_k (B,G,r_k,d)  B_v (B,G,r_v,d)
    landmarks (B,G,H_kv,n_c,d_h)  q (G,B,H_q,d_h)
    Returns sel_idx (G,B,H_kv,k_cap) int32 padded with -1, sel_cnt (G,B,H_kv),
    out (G,B,H_q,d_h) fp64, lse (G,B,H_q) fp64.
    If sel_idx/sel_cnt are given the selection is taken from them (any order,
    duplicates allowed) and Algorithm 2 is skipped.  `problems` restricts the
    work to a list of (l, b, g) triples (the rest of the outputs stay zero).
    `outliers` (G,B,H_kv,o) int: static outlier chunk ids united with every selection (Algorithm 2 line 5);
    the row stride of sel_idx is then (ceil(k/c) + o) * c.
    """
    Bsz, T, _ = A_k.shape
    G = B_k.shape[1]
    H_q, d_h = q.shape[2], q.shape[3]
    n_rep = H_q // H_kv
    if scale is None:
        scale = 1.0 / math.sqrt(d_h)
    n_out = 0 if outliers is None else outliers.shape[-1]
    k_cap = (-(-k // c) + n_out) * c if sel_idx is None else sel_idx.shape[-1]
    o_idx = np.full((G, Bsz, H_kv, k_cap), -1, dtype=np.int32)
    o_cnt = np.zeros((G, Bsz, H_kv), dtype=np.int32)
    out = np.zeros((G, Bsz, H_q, d_h))
    lse = np.zeros((G, Bsz, H_q))
    if problems is None:
        problems = [(l, b, g) for l in range(G) for b in range(Bsz) for g in range(H_kv)]
    for (l, b, g) in problems:
        qh = q[l, b, g * n_rep:(g + 1) * n_rep]
        rows = None
        if sel_idx is not None:
            rows = np.asarray(sel_idx[l, b, g, :int(sel_cnt[l, b, g])], dtype=np.int32)
        rows, o, ls = sr_decode_problem(
            qh, None if landmarks is None else landmarks[b, l, g], A_k[b], A_v[b],
            B_k[b, l][:, g * d_h:(g + 1) * d_h], B_v[b, l][:, g * d_h:(g + 1) * d_h],
            k, c, T, rope_base, scale, rows, None if outliers is None else outliers[l, b, g])
        o_idx[l, b, g, :len(rows)] = rows
        o_cnt[l, b, g] = len(rows)
        out[l, b, g * n_rep:(g + 1) * n_rep] = o
        lse[l, b, g * n_rep:(g + 1) * n_rep] = ls
    return o_idx, o_cnt, out, lse


# --------------------------------------------------------------------------
# Uncompressed tail  (Sec. 4 "Implementation details", Sec. 7 "Long Generation Scenario":
# tokens generated during decoding are not compressed; they are attended to densely)
# --------------------------------------------------------------------------


def sr_attend_with_tail(q_heads, K_hat, V_hat, K_tail, V_tail, scale: float):
    """Attention of the query heads of one KV head over the union of the reconstructed selected rows
    (K_hat already rotated) and the uncompressed tail rows (K_tail as the model stores it: post-RoPE).

    The definition written out: one softmax over the concatenated logits.  Returns (o, lse) in fp64.
    """
    K = np.concatenate([np.asarray(K_hat, dtype=np.float64), np.asarray(K_tail, dtype=np.float64)], axis=0)
    V = np.concatenate([np.asarray(V_hat, dtype=np.float64), np.asarray(V_tail, dtype=np.float64)], axis=0)
    return attend(q_heads, K, V, scale)


def sr_decode_step_with_tail(A_k, A_v, B_k, B_v, q, sel_idx, sel_cnt, tail_k, tail_v, tail_len, H_kv,
                             rope_base, scale=None, problems=None):
    """`sr_decode_step` with given selections plus an uncompressed tail.

    tail_k, tail_v (G,B,H_kv,tail_cap,d_h); tail_len (B,) rows of the tail that are valid for each sequence.
    Returns out (G,B,H_q,d_h) fp64, lse (G,B,H_q) fp64.
    """
    Bsz, T, _ = A_k.shape
    G = B_k.shape[1]
    H_q, d_h = q.shape[2], q.shape[3]
    n_rep = H_q // H_kv
    if scale is None:
        scale = 1.0 / math.sqrt(d_h)
    out = np.zeros((G, Bsz, H_q, d_h))
    lse = np.zeros((G, Bsz, H_q))
    if problems is None:
        problems = [(l, b, g) for l in range(G) for b in range(Bsz) for g in range(H_kv)]
    for (l, b, g) in problems:
        qh = q[l, b, g * n_rep:(g + 1) * n_rep]
        rows = np.asarray(sel_idx[l, b, g, :int(sel_cnt[l, b, g])], dtype=np.int32)
        K_hat = sr_reconstruct_keys(A_k[b], B_k[b, l][:, g * d_h:(g + 1) * d_h], rows, rope_base)
        V_hat = sr_reconstruct(A_v[b], B_v[b, l][:, g * d_h:(g + 1) * d_h], rows)
        n_t = int(tail_len[b])
        o, ls = sr_attend_with_tail(qh, K_hat, V_hat, tail_k[l, b, g, :n_t], tail_v[l, b, g, :n_t], scale)
        out[l, b, g * n_rep:(g + 1) * n_rep] = o
        lse[l, b, g * n_rep:(g + 1) * n_rep] = ls
    return out, lse


# --------------------------------------------------------------------------
# Cost and memory accounting  (App. C, "FLOPs & Memory Cost")
# --------------------------------------------------------------------------


def flops_dense(L: int, r_k: int, r_v: int, d: int) -> int:
    """Dense reconstruction cost of one layer (multiply-add counted once, as the paper does)."""
    return L * r_k * d + L * r_v * d


def flops_sr(M_per_head, d_h: int, r_k: int, r_v: int) -> int:
    """Selective reconstruction cost of one layer: sum_g M_g * d_h * (r_K + r_V)."""
    return sum(int(M) * d_h * (r_k + r_v) for M in M_per_head)


def factor_scalars(N: int, W: int, L: int, r_k: int, r_v: int, d: int) -> int:
    """Stored scalars of the CLF factors: one basis per window, one B per layer."""
    Gw = -(-N // W)
    return (Gw * L * r_k + N * r_k * d) + (Gw * L * r_v + N * r_v * d)


def landmark_scalars(N: int, L: int, c: int, d: int) -> int:
    return N * (-(-L // c)) * d


def compression_ratios(N: int, W: int, L: int, d: int, r_k: int, r_v: int, c: int) -> dict:
    """Compression ratios relative to the full cache of 2*N*L*d scalars."""
    Gw = -(-N // W)
    C_K = N * L * d / (Gw * L * r_k + N * r_k * d)
    C_V = N * L * d / (Gw * L * r_v + N * r_v * d) if r_v else float("inf")
    alpha = (-(-L // c)) / L
    return {
        "xkv": 2.0 / (1.0 / C_K + 1.0 / C_V),
        "xkv_sr": 2.0 / (1.0 / C_K + 1.0 / C_V + alpha),
        "xk_sr_gpu": 2.0 / (1.0 / C_K + alpha),
        "xk_sr_total": 2.0 / (1.0 / C_K + alpha + 1.0),
    }


# --------------------------------------------------------------------------
# Round-to-nearest quantisation of the compressed cache  (App. "Integrate with Quantization")
#
# The paper applies "a simple round-to-nearest (RTN) quantization method to the compressed cache" and prints the
# resulting compression: 8.03x -> 25.70x at 4 bits and -> 32.12x at 3 bits, i.e. exactly b + 1 stored bits per
# scalar.  The grouping is not stated; the reading taken here reproduces that overhead of one bit: groups of 32
# consecutive scalars of a row share a 16-bit scale and a 16-bit offset (asymmetric min/max quantisation).
# Canonical arithmetic (fp32, IEEE, so that the codes are the same integers on every implementation):
#   lo, hi = min, max of the group;  zero = bf16(lo);  scale = bf16((hi - lo) / (2^b - 1))
#   code   = clip(rint((x - zero) / scale), 0, 2^b - 1)        (rint: ties to even; scale == 0 -> code 0)
#   x_hat  = bf16(code * scale + zero)                          (the exact value, rounded once)
# --------------------------------------------------------------------------

RTN_GROUP = 32


def rtn_quantize(X: np.ndarray, bits: int, group: int = RTN_GROUP):
    """X (n, m) of bf16 values, m a multiple of `group`.  Returns codes (n, m) uint8, scale (n, m/group) and
    zero (n, m/group) as float32 arrays holding bf16 values."""
    X = np.ascontiguousarray(X, dtype=np.float32)
    n, m = X.shape
    assert m % group == 0 and 1 <= bits <= 8
    qmax = np.float32((1 << bits) - 1)
    Xg = X.reshape(n, m // group, group)
    lo = Xg.min(axis=2)
    hi = Xg.max(axis=2)
    zero = bf16_round(lo)
    scale = bf16_round((hi - lo) / qmax)
    codes = np.zeros_like(Xg)
    nz = scale > 0
    with np.errstate(divide="ignore", invalid="ignore"):
        q = (Xg - zero[:, :, None]) / scale[:, :, None]          # fp32 division, correctly rounded
    q = np.where(nz[:, :, None], np.rint(q), np.float32(0.0))
    codes = np.clip(q, 0.0, qmax).astype(np.uint8)
    return codes.reshape(n, m), scale, zero


def bf16_round_exact(x: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bf16 (8 significant bits, ties to even) in ONE step; returns float32.
    (Going through float32 first would round twice.)  Values in the normal range of bf16 only."""
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                                   # x = m * 2^e, 0.5 <= |m| < 1
    return np.ldexp(np.rint(m * 256.0) / 256.0, e).astype(np.float32)


def rtn_dequantize(codes: np.ndarray, scale: np.ndarray, zero: np.ndarray, group: int = RTN_GROUP) -> np.ndarray:
    """x_hat = bf16(code * scale + zero): the exact value (formed in fp64, where it is exact for any realistic
    exponent gap) rounded once.  float32 array holding bf16 values."""
    n, m = codes.shape
    c = codes.reshape(n, m // group, group).astype(np.float64)
    x = c * scale[:, :, None].astype(np.float64) + zero[:, :, None].astype(np.float64)
    return bf16_round_exact(x.reshape(n, m))


def quantized_bits_per_scalar(bits: int, group: int = RTN_GROUP, meta_bits: int = 32) -> float:
    """Stored bits per scalar: the code plus the group's scale and offset spread over its members."""
    return bits + meta_bits / group


def quantized_compression_ratio(base_ratio: float, bits: int, group: int = RTN_GROUP) -> float:
    """Compression of a 16-bit factorised cache of ratio `base_ratio` after RTN quantisation of every factor."""
    return base_ratio * 16.0 / quantized_bits_per_scalar(bits, group)


# --------------------------------------------------------------------------
# Randomised cross-layer factorisation  (App. "Custom SVD Kernel": randomised SVD, 16-bit matrix products in the
# power iterations, shifted Cholesky QR instead of Householder QR)
#
# The paper names the ingredients, not the steps.  The steps taken here are the textbook randomised subspace
# iteration (Halko, Martinsson, Tropp) run on the right side, because X (T x N, N = G d) is tall:
#   Z <- Omega (N x l, l = r + p);  repeat q + 1 times: Y = X Z; U = X^T Y; Z = orth(U)
#   Rayleigh-Ritz on span(Z): M = Z^T X^T X Z = P Lambda P^T; V = Z P_r; B = V^T; A = X bf16(V); sigma = sqrt(Lambda).
# orth = shifted Cholesky QR: G = U^T U + s I, s = shift * max diag(U^T U), G = L L^T, U <- U L^-T, in passes with
# relative shifts 1e-4, 1e-5 (inside the iteration) and 1e-4, 1e-5, 1e-6, 1e-8, 1e-10 (last iterate).  Matrices that the 16-bit products read are rounded to bf16 first (X is bf16 already).
# It approximates clf_factorize's optimum; it is compared with it through the residual, never factor by factor.
# --------------------------------------------------------------------------


CHOLQR_SHIFTS = (1e-4, 1e-5, 1e-6, 1e-8, 1e-10)


def cholesky_qr(U: np.ndarray, shifts=CHOLQR_SHIFTS) -> np.ndarray:
    """Orthonormalise the columns of U (n x l) by repeated shifted Cholesky QR (fp64 here); one pass per entry of
    `shifts` (each relative to the largest diagonal entry of the Gram matrix of that pass)."""
    Z = np.asarray(U, dtype=np.float64)
    for shift_rel in shifts:
        Gm = Z.T @ Z
        Gm = Gm + shift_rel * Gm.diagonal().max() * np.eye(Gm.shape[0])
        L = np.linalg.cholesky(Gm)
        Z = np.linalg.solve(L, Z.T).T                       # Z L^-T
    return Z


def clf_randomized(X_cat: np.ndarray, r: int, omega: np.ndarray, power_iters: int = 2):
    """Rank-r factorisation of X_cat (T x N, bf16 values) from the test matrix omega (N x l, bf16 values, l >= r).
    Returns A (T x r), V (N x r) with B = V^T, sigma (r,); A and V hold bf16 values (float32 arrays)."""
    X = np.asarray(X_cat, dtype=np.float64)
    Z = np.asarray(omega, dtype=np.float64)
    for it in range(power_iters + 1):
        Y = bf16_round((X @ bf16_round(Z.astype(np.float32)).astype(np.float64)).astype(np.float32)).astype(np.float64)
        U = X.T @ Y
        # inside the iteration the iterate only has to stay well conditioned (two passes); the last one has to be
        # orthonormal (five passes, decreasing shifts)
        Z = cholesky_qr(U, CHOLQR_SHIFTS if it == power_iters else CHOLQR_SHIFTS[:2])
    Zb = bf16_round(Z.astype(np.float32)).astype(np.float64)
    W = bf16_round((X @ Zb).astype(np.float32)).astype(np.float64)
    M = Z.T @ (X.T @ W)
    M = 0.5 * (M + M.T)
    lam, P = np.linalg.eigh(M)
    order = np.argsort(-lam)[:r]
    V = bf16_round((Z @ P[:, order]).astype(np.float32))
    A = bf16_round((X @ V.astype(np.float64)).astype(np.float32))
    return A, V, np.sqrt(np.maximum(lam[order], 0.0))
