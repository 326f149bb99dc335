"""Pins for the oracle's decode step: RoPE, landmarks (Alg. 1), selection (Alg. 2),
selective reconstruction (Eq. 3) and attention over the selected rows."""
import math

import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O


def _bf(x):
    return O.bf16_round(np.asarray(x, dtype=np.float32))


# ------------------------------------------------------------------ RoPE

def test_rope_is_complex_multiplication():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 8))
    pos = np.array([0, 1, 7, 1000, 131071])
    base = 10000.0
    y = O.rope_rotate(x, pos, base)
    theta = base ** (-2.0 * np.arange(4) / 8)
    z = (x[:, :4] + 1j * x[:, 4:]) * np.exp(1j * pos[:, None] * theta[None, :])
    np.testing.assert_allclose(y[:, :4], z.real, atol=1e-9)
    np.testing.assert_allclose(y[:, 4:], z.imag, atol=1e-9)
    np.testing.assert_allclose(y[0], x[0])                                  # p = 0 is the identity
    np.testing.assert_allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1))


def test_rope_d2_textbook_and_relative_property():
    # d_h = 2: one frequency theta_0 = 1, a plain rotation by p radians
    y = O.rope_rotate(np.array([[1.0, 0.0]]), np.array([2]), 10000.0)
    np.testing.assert_allclose(y, [[math.cos(2.0), math.sin(2.0)]])
    rng = np.random.default_rng(1)
    x, w = rng.standard_normal((1, 16)), rng.standard_normal((1, 16))
    a = O.rope_rotate(x, np.array([37]), 500.0) @ O.rope_rotate(w, np.array([37]), 500.0).T
    np.testing.assert_allclose(a, x @ w.T)
    # <R_p x, R_q w> depends on p - q only
    b = O.rope_rotate(x, np.array([50]), 500.0) @ O.rope_rotate(w, np.array([40]), 500.0).T
    c = O.rope_rotate(x, np.array([10]), 500.0) @ w.T
    np.testing.assert_allclose(b, c)
    np.testing.assert_array_equal(O.rope_rotate(x, np.array([9]), 0.0), x)  # base <= 0: no rotation


# ------------------------------------------------------------------ landmarks

def test_landmarks_constant_keys_and_plain_mean():
    key = _bf(np.linspace(-1, 1, 16))
    K = np.broadcast_to(key, (2, 37, 16)).copy()
    L = O.build_landmarks(K, 8, 0.0)
    assert L.shape == (2, 5, 16)
    np.testing.assert_array_equal(L, np.broadcast_to(key, (2, 5, 16)))
    rng = np.random.default_rng(2)
    K = _bf(rng.standard_normal((1, 21, 4)))
    L = O.build_landmarks(K, 8, 0.0)
    for j, (a, b) in enumerate([(0, 8), (8, 16), (16, 21)]):               # ragged tail: mean over 5 rows
        brute = np.zeros(4)
        for x in range(a, b):
            brute += K[0, x].astype(np.float64)
        np.testing.assert_array_equal(L[0, j], _bf(brute / (b - a)))


def test_landmarks_use_post_rope_keys():
    rng = np.random.default_rng(3)
    K = _bf(rng.standard_normal((1, 6, 8)))
    L = O.build_landmarks(K, 1, 10000.0)                                    # c = 1: landmark = rotated key
    np.testing.assert_array_equal(L[0], _bf(O.rope_rotate(K[0], np.arange(6), 10000.0)))
    L2 = O.build_landmarks(K, 2, 10000.0)
    R = O.rope_rotate(K[0], np.arange(6), 10000.0)
    np.testing.assert_array_equal(L2[0, 1], _bf((R[2] + R[3]) / 2))


# ------------------------------------------------------------------ selection

def _brute_select(q, L, k, c, T):
    """Algorithm 2 in scalar Python, fp32 by explicit np.float32 scalars."""
    n_rep, d_h = q.shape
    n_c = L.shape[0]
    s = np.float32(1.0) / np.float32(math.sqrt(np.float32(d_h)))
    S = []
    for j in range(n_c):
        best = None
        for h in range(n_rep):
            acc = np.float32(0.0)
            for i in range(d_h):
                acc = np.float32(acc + np.float32(np.float32(q[h, i]) * np.float32(L[j, i])))
            p = np.float32(acc * s)
            best = p if best is None or p > best else best
        S.append(best)
    k_ch = min(-(-k // c), n_c)
    order = sorted(range(n_c), key=lambda j: (-float(S[j]), j))[:k_ch]
    rows = []
    for j in sorted(order):
        rows += list(range(j * c, min(j * c + c, T)))
    return np.array(rows, dtype=np.int32)


@pytest.mark.parametrize("T,c,k,n_rep,d_h", [(64, 8, 16, 4, 16), (61, 8, 20, 3, 8), (40, 4, 9, 1, 32), (17, 8, 8, 7, 8)])
def test_select_matches_brute_force(T, c, k, n_rep, d_h):
    rng = np.random.default_rng(T + k)
    n_c = -(-T // c)
    q = _bf(rng.standard_normal((n_rep, d_h)))
    L = _bf(rng.standard_normal((n_c, d_h)))
    np.testing.assert_array_equal(O.sr_select(q, L, k, c, T), _brute_select(q, L, k, c, T))


def test_select_properties():
    rng = np.random.default_rng(7)
    T, c, n_rep, d_h = 1000, 8, 4, 32
    n_c = 125
    q = _bf(rng.standard_normal((n_rep, d_h)))
    L = _bf(rng.standard_normal((n_c, d_h)))
    prev = set()
    for k in (8, 64, 65, 200, 512):
        rows = O.sr_select(q, L, k, c, T)
        assert len(rows) == -(-k // c) * c                         # budget rounds up to whole chunks
        assert np.all(np.diff(rows) > 0)                           # ascending, distinct
        assert prev <= set(rows.tolist())                          # nested in k
        prev = set(rows.tolist())
    # the best chunk is always selected
    S = O.pool_scores(O.landmark_scores(q, L))
    j = int(np.argmax(S))
    assert j * c in O.sr_select(q, L, 8, c, T)
    # k >= T selects every row
    np.testing.assert_array_equal(O.sr_select(q, L, T, c, T), np.arange(T))
    np.testing.assert_array_equal(O.sr_select(q, L, 10 * T, c, T), np.arange(T))
    # permuting the query heads of the group changes nothing (max pooling)
    np.testing.assert_array_equal(O.sr_select(q[::-1], L, 64, c, T), O.sr_select(q, L, 64, c, T))
    # pooled score is the max over heads of the per-head scores, each a scaled inner product
    P64 = (q.astype(np.float64) @ L.astype(np.float64).T) / math.sqrt(d_h)
    np.testing.assert_allclose(S, P64.max(axis=0), rtol=0, atol=2e-5)


def test_select_ties_go_to_lowest_index():
    d_h = 8
    q = _bf(np.ones((2, d_h)))
    L = np.zeros((6, d_h), dtype=np.float32)
    L[[1, 3, 4]] = 1.0                                             # three identical best chunks
    rows = O.sr_select(q, L, 2 * 4, 4, 24)                         # budget: 2 chunks of 4
    np.testing.assert_array_equal(rows, [4, 5, 6, 7, 12, 13, 14, 15])
    # -0 and +0 scores tie: chunk 0 (score -0) beats chunk 2 (score +0) by index only
    L = np.zeros((3, d_h), dtype=np.float32)
    L[0, 0] = -0.0
    L[1] = -1.0
    S = np.array([-0.0, -1.0, 0.0], dtype=np.float32)
    np.testing.assert_array_equal(O.topk_chunks(S, 1), [0])
    np.testing.assert_array_equal(O.topk_chunks(S, 2), [0, 2])


def test_select_ragged_last_chunk():
    d_h = 4
    q = _bf(np.ones((1, d_h)))
    L = np.zeros((3, d_h), dtype=np.float32)
    L[2] = 1.0                                                     # last chunk (rows 16..18 of T=19) is best
    rows = O.sr_select(q, L, 16, 8, 19)
    np.testing.assert_array_equal(rows, list(range(0, 8)) + [16, 17, 18])


def test_select_fp32_order_agrees_with_fp64_when_margin_is_clear():
    rng = np.random.default_rng(11)
    n_c, d_h, k_ch = 512, 64, 32
    q = _bf(rng.standard_normal((4, d_h)))
    L = _bf(rng.standard_normal((n_c, d_h)))
    S64 = ((q.astype(np.float64) @ L.astype(np.float64).T) / math.sqrt(d_h)).max(axis=0)
    srt = np.sort(S64)[::-1]
    if srt[k_ch - 1] - srt[k_ch] > 1e-5:
        want = np.sort(np.argsort(-S64, kind="stable")[:k_ch])
        got = O.topk_chunks(O.pool_scores(O.landmark_scores(q, L)), k_ch)
        np.testing.assert_array_equal(got, want)
    else:
        pytest.skip("boundary margin too small for this seed")


# ------------------------------------------------------------------ reconstruction

def test_reconstruct_identity_B_is_a_gather():
    rng = np.random.default_rng(20)
    A = rng.standard_normal((50, 8))
    rows = np.array([3, 49, 0, 3, 17])
    np.testing.assert_array_equal(O.sr_reconstruct(A, np.eye(8), rows), A[rows])
    Kh = O.sr_reconstruct_keys(A, np.eye(8), rows, 10000.0)
    np.testing.assert_allclose(Kh, O.rope_rotate(A[rows], rows, 10000.0))


def test_reconstruct_rows_equal_rows_of_dense_reconstruction():
    rng = np.random.default_rng(21)
    A, B = rng.standard_normal((30, 6)), rng.standard_normal((6, 12))
    full = np.zeros((30, 12))
    for t in range(30):
        for j in range(12):
            full[t, j] = sum(A[t, m] * B[m, j] for m in range(6))
    rows = np.array([29, 4, 4, 11])
    np.testing.assert_allclose(O.sr_reconstruct(A, B, rows), full[rows], atol=1e-12)


def test_full_rank_clf_then_reconstruct_gives_original_rows():
    rng = np.random.default_rng(22)
    X = [rng.standard_normal((40, 8)) for _ in range(2)]            # 2 layers, H_kv=2, d_h=4
    A, B, _ = O.clf_factorize(X, 16)
    rows = np.array([5, 6, 7, 30])
    for l in range(2):
        for g in range(2):
            got = O.sr_reconstruct(A, B[l][:, 4 * g:4 * g + 4], rows)
            np.testing.assert_allclose(got, X[l][rows, 4 * g:4 * g + 4], atol=1e-10)


# ------------------------------------------------------------------ attention

def test_attend_all_rows_equals_dense_and_library_sdpa():
    rng = np.random.default_rng(30)
    q, K, V = rng.standard_normal((3, 16)), rng.standard_normal((41, 16)), rng.standard_normal((41, 16))
    scale = 1 / math.sqrt(16)
    o, lse = O.attend(q, K, V, scale)
    np.testing.assert_allclose(o, O.dense_attend(q, K, V, scale), atol=1e-12)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None])[0].numpy()
    np.testing.assert_allclose(o, ref, atol=1e-12)
    np.testing.assert_allclose(lse, torch.logsumexp(torch.from_numpy(q @ K.T * scale), dim=1).numpy(), atol=1e-12)


def test_attend_special_cases():
    rng = np.random.default_rng(31)
    q, K, V = rng.standard_normal((2, 8)), rng.standard_normal((9, 8)), rng.standard_normal((9, 8))
    o, lse = O.attend(q, K[:1], V[:1], 0.3)
    np.testing.assert_allclose(o, np.broadcast_to(V[0], (2, 8)))               # one row: output is that V row
    np.testing.assert_allclose(lse, (q @ K[0]) * 0.3)
    o, _ = O.attend(q, K, np.broadcast_to(V[3], (9, 8)), 0.3)
    np.testing.assert_allclose(o, np.broadcast_to(V[3], (2, 8)))               # all V rows equal
    o, lse = O.attend(np.zeros((2, 8)), K, V, 0.3)
    np.testing.assert_allclose(o, np.broadcast_to(V.mean(axis=0), (2, 8)))     # q = 0: uniform weights
    np.testing.assert_allclose(lse, math.log(9))
    # a constant added to every logit changes nothing: append a constant feature to q and K
    qa = np.concatenate([q, np.ones((2, 1))], axis=1)
    Ka = np.concatenate([K, np.full((9, 1), 5.0)], axis=1)
    np.testing.assert_allclose(O.attend(qa, Ka, V, 0.3)[0], O.attend(q, K, V, 0.3)[0], atol=1e-12)
    # duplicates count twice
    o2, _ = O.attend(q, np.concatenate([K, K[:1]]), np.concatenate([V, V[:1]]), 0.3)
    z = q @ K.T * 0.3
    w = np.exp(z)
    w[:, 0] *= 2
    np.testing.assert_allclose(o2, (w @ V) / w.sum(axis=1, keepdims=True), atol=1e-12)
    o, lse = O.attend(q, K[:0], V[:0], 0.3)                                    # empty selection
    assert np.all(o == 0) and np.all(np.isneginf(lse))


def test_split_and_merge_equals_single_pass():
    rng = np.random.default_rng(32)
    q, K, V = rng.standard_normal((4, 8)), 3 * rng.standard_normal((50, 8)), rng.standard_normal((50, 8))
    whole = O.attend(q, K, V, 0.35)
    parts = [O.attend(q, K[a:b], V[a:b], 0.35) for a, b in [(0, 7), (7, 33), (33, 50)]]
    o, lse = O.merge_partials(parts)
    np.testing.assert_allclose(o, whole[0], atol=1e-12)
    np.testing.assert_allclose(lse, whole[1], atol=1e-12)


# ------------------------------------------------------------------ the whole step

def test_full_rank_all_tokens_equals_dense_attention_on_original_cache():
    """Full-rank factorisation + selection of every token = textbook attention on the raw cache."""
    rng = np.random.default_rng(40)
    G, H_kv, n_rep, d_h, T, c = 2, 2, 2, 8, 48, 8
    d = H_kv * d_h
    K = [rng.standard_normal((T, d)) for _ in range(G)]
    V = [rng.standard_normal((T, d)) for _ in range(G)]
    A_k, B_k, _ = O.clf_factorize(K, G * d)
    A_v, B_v, _ = O.clf_factorize(V, G * d)
    lm = np.stack([O.build_landmarks(np.stack([K[l][:, g * d_h:(g + 1) * d_h] for g in range(H_kv)]), c, 10000.0)
                   for l in range(G)])[None]
    q = rng.standard_normal((G, 1, H_kv * n_rep, d_h))
    idx, cnt, out, lse = O.sr_decode_step(A_k[None], A_v[None], np.stack(B_k)[None], np.stack(B_v)[None],
                                          lm, q, k=T, c=c, H_kv=H_kv, rope_base=10000.0)
    assert np.all(cnt == T)
    for l in range(G):
        for g in range(H_kv):
            Kr = O.rope_rotate(K[l][:, g * d_h:(g + 1) * d_h], np.arange(T), 10000.0)
            ref = O.dense_attend(q[l, 0, g * n_rep:(g + 1) * n_rep], Kr, V[l][:, g * d_h:(g + 1) * d_h],
                                 1 / math.sqrt(d_h))
            np.testing.assert_allclose(out[l, 0, g * n_rep:(g + 1) * n_rep], ref, atol=1e-9)
            np.testing.assert_array_equal(idx[l, 0, g], np.arange(T))


def test_step_with_given_index_set_skips_selection():
    rng = np.random.default_rng(41)
    T, r, d_h = 64, 6, 8
    A_k, A_v = rng.standard_normal((1, T, r)), rng.standard_normal((1, T, r))
    B_k, B_v = rng.standard_normal((1, 1, r, d_h)), rng.standard_normal((1, 1, r, d_h))
    q = rng.standard_normal((1, 1, 2, d_h))
    sel = np.array([[[[40, 3, 17, 3, 0, 0]]]], dtype=np.int32)                  # unsorted, duplicate, padded
    cnt = np.array([[[4]]], dtype=np.int32)
    idx, c2, out, lse = O.sr_decode_step(A_k, A_v, B_k, B_v, None, q, k=0, c=8, H_kv=1, rope_base=0.0,
                                         sel_idx=sel, sel_cnt=cnt)
    rows = [40, 3, 17, 3]
    ref, _ = O.attend(q[0, 0], A_k[0][rows] @ B_k[0, 0], A_v[0][rows] @ B_v[0, 0], 1 / math.sqrt(d_h))
    np.testing.assert_allclose(out[0, 0], ref, atol=1e-12)
    assert c2[0, 0, 0] == 4


# ------------------------------------------------------------------ uncompressed tail (Sec. 4, Sec. 7)

def test_tail_union_equals_dense_and_merge_of_the_two_parts():
    """Attention over selected rows + tail is one softmax over the union: it must equal the row-by-row dense
    routine on the concatenation, the library SDPA, and the log-sum-exp merge of the two separate results."""
    rng = np.random.default_rng(40)
    q = rng.standard_normal((3, 8))
    Ks, Vs = 2 * rng.standard_normal((21, 8)), rng.standard_normal((21, 8))
    Kt, Vt = 2 * rng.standard_normal((6, 8)), rng.standard_normal((6, 8))
    o, lse = O.sr_attend_with_tail(q, Ks, Vs, Kt, Vt, 0.4)
    Kc, Vc = np.concatenate([Ks, Kt]), np.concatenate([Vs, Vt])
    np.testing.assert_allclose(o, O.dense_attend(q, Kc, Vc, 0.4), atol=1e-12)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(Kc)[None], torch.from_numpy(Vc)[None], scale=0.4)[0].numpy()
    np.testing.assert_allclose(o, ref, atol=1e-12)
    om, lm = O.merge_partials([O.attend(q, Ks, Vs, 0.4), O.attend(q, Kt, Vt, 0.4)])
    np.testing.assert_allclose(o, om, atol=1e-12)
    np.testing.assert_allclose(lse, lm, atol=1e-12)


def test_tail_special_cases():
    rng = np.random.default_rng(41)
    q = rng.standard_normal((2, 8))
    Ks, Vs = rng.standard_normal((5, 8)), rng.standard_normal((5, 8))
    Kt, Vt = rng.standard_normal((4, 8)), rng.standard_normal((4, 8))
    # empty tail: the plain SR result
    o, lse = O.sr_attend_with_tail(q, Ks, Vs, Kt[:0], Vt[:0], 0.3)
    np.testing.assert_allclose(o, O.attend(q, Ks, Vs, 0.3)[0], atol=1e-15)
    # empty selection: dense attention over the tail
    o, lse = O.sr_attend_with_tail(q, Ks[:0], Vs[:0], Kt, Vt, 0.3)
    np.testing.assert_allclose(o, O.dense_attend(q, Kt, Vt, 0.3), atol=1e-12)
    # a tail row whose logit dwarfs everything takes all the weight
    big = np.concatenate([Kt, 200.0 * q[:1]])
    o, _ = O.sr_attend_with_tail(q[:1], Ks, Vs, big, np.concatenate([Vt, np.full((1, 8), 7.0)]), 1.0)
    np.testing.assert_allclose(o, np.full((1, 8), 7.0), atol=1e-9)


def test_step_with_tail_layouts_and_per_sequence_lengths():
    """The window-level routine indexes (layer, sequence, head) and honours tail_len per sequence:
    compare with a direct per-problem evaluation from the definitions."""
    rng = np.random.default_rng(42)
    G, Bsz, H_kv, n_rep, d_h, T, r = 2, 2, 2, 2, 8, 40, 6
    A_k, A_v = _bf(rng.standard_normal((Bsz, T, r))), _bf(rng.standard_normal((Bsz, T, r)))
    B_k, B_v = _bf(rng.standard_normal((Bsz, G, r, H_kv * d_h))), _bf(rng.standard_normal((Bsz, G, r, H_kv * d_h)))
    q = _bf(rng.standard_normal((G, Bsz, H_kv * n_rep, d_h)))
    sel_idx = np.stack([np.sort(rng.choice(T, 12, replace=False)) for _ in range(G * Bsz * H_kv)]).reshape(G, Bsz, H_kv, 12).astype(np.int32)
    sel_cnt = rng.integers(0, 13, size=(G, Bsz, H_kv)).astype(np.int32)
    tk, tv = _bf(rng.standard_normal((G, Bsz, H_kv, 5, d_h))), _bf(rng.standard_normal((G, Bsz, H_kv, 5, d_h)))
    tail_len = np.array([5, 2], dtype=np.int32)
    out, lse = O.sr_decode_step_with_tail(A_k, A_v, B_k, B_v, q, sel_idx, sel_cnt, tk, tv, tail_len, H_kv, 10000.0)
    scale = 1 / math.sqrt(d_h)
    for l in range(G):
        for b in range(Bsz):
            for g in range(H_kv):
                rows = sel_idx[l, b, g, :sel_cnt[l, b, g]]
                Kh = O.rope_rotate(A_k[b][rows].astype(np.float64) @ B_k[b, l][:, g * d_h:(g + 1) * d_h].astype(np.float64), rows, 10000.0)
                Vh = A_v[b][rows].astype(np.float64) @ B_v[b, l][:, g * d_h:(g + 1) * d_h].astype(np.float64)
                n_t = tail_len[b]
                Kc = np.concatenate([Kh, tk[l, b, g, :n_t]]); Vc = np.concatenate([Vh, tv[l, b, g, :n_t]])
                ref = O.dense_attend(q[l, b, g * n_rep:(g + 1) * n_rep], Kc, Vc, scale)
                np.testing.assert_allclose(out[l, b, g * n_rep:(g + 1) * n_rep], ref, atol=1e-10)


# ------------------------------------------------------------------ static outliers (Alg. 1 lines 4-5, Alg. 2 line 5)

def test_union_with_outliers_is_a_set_union_and_keeps_the_topk():
    rng = np.random.default_rng(50)
    T, c, d_h = 333, 8, 16
    n_c = -(-T // c)
    L = _bf(rng.standard_normal((n_c, d_h)))
    q = _bf(rng.standard_normal((2, d_h)))
    plain = O.sr_select(q, L, 40, c, T)
    out = np.array([3, 3, n_c - 1, -5, 10 ** 6, int(plain[0]) // c, 17])       # repeats, out of range, one already in
    rows = O.sr_select(q, L, 40, c, T, outliers=out)
    want = set(plain.tolist())
    for j in (3, n_c - 1, 17, int(plain[0]) // c):
        want |= set(range(j * c, min(T, j * c + c)))
    assert rows.tolist() == sorted(want)                                      # brute force on sets
    assert set(plain.tolist()) <= set(rows.tolist())
    # outliers that the top-k already holds change nothing; an empty list changes nothing
    inside = np.unique(plain // c)[:3]
    np.testing.assert_array_equal(O.sr_select(q, L, 40, c, T, outliers=inside), plain)
    np.testing.assert_array_equal(O.sr_select(q, L, 40, c, T, outliers=np.array([], dtype=np.int64)), plain)


def test_min_chunk_cosine_and_static_outliers():
    c = 4
    e0, e1 = np.eye(6)[0], np.eye(6)[1]
    K = np.stack([e0, e0, e0, e0,                    # identical rows: cosine 1
                  e0, e0, e0, -e0 + 4 * e1,          # one row far from the mean
                  e0, e1, e0, e1,                    # two directions: each row at 45 degrees from the mean
                  2 * e0, 5 * e0])                   # ragged chunk, parallel rows of different length: cosine 1
    m = O.min_chunk_cosine(K, c)
    np.testing.assert_allclose(m[0], 1.0, atol=1e-12)
    np.testing.assert_allclose(m[2], math.cos(math.pi / 4), atol=1e-12)
    np.testing.assert_allclose(m[3], 1.0, atol=1e-12)
    mean1 = K[4:8].mean(axis=0)
    np.testing.assert_allclose(m[1], min(K[j] @ mean1 / np.linalg.norm(K[j]) / np.linalg.norm(mean1) for j in range(4, 8)), atol=1e-12)
    assert m[1] < m[2]
    np.testing.assert_array_equal(O.static_outliers(K, c, 2), [1, 2])          # the two least homogeneous chunks
    np.testing.assert_array_equal(O.static_outliers(K, c, 1), [1])
    np.testing.assert_array_equal(O.static_outliers(K, c, 9), [0, 1, 2, 3])    # o larger than n_c
    # scaling a row does not change its cosine; a zero row has cosine 0
    K2 = K.copy(); K2[0] *= 7.0
    np.testing.assert_allclose(O.min_chunk_cosine(K2, c)[0], 1.0, atol=1e-12)
    K3 = K.copy(); K3[1] = 0.0
    np.testing.assert_allclose(O.min_chunk_cosine(K3, c)[0], 0.0, atol=1e-12)


def test_step_with_outliers_layout_and_count():
    rng = np.random.default_rng(51)
    G, Bsz, H_kv, n_rep, d_h, T, r, c = 2, 2, 2, 2, 8, 70, 6, 8
    n_c = -(-T // c)
    A_k, A_v = _bf(rng.standard_normal((Bsz, T, r))), _bf(rng.standard_normal((Bsz, T, r)))
    B_k, B_v = _bf(rng.standard_normal((Bsz, G, r, H_kv * d_h))), _bf(rng.standard_normal((Bsz, G, r, H_kv * d_h)))
    lm = _bf(rng.standard_normal((Bsz, G, H_kv, n_c, d_h)))
    q = _bf(rng.standard_normal((G, Bsz, H_kv * n_rep, d_h)))
    outl = rng.integers(0, n_c, size=(G, Bsz, H_kv, 3))
    idx, cnt, out, lse = O.sr_decode_step(A_k, A_v, B_k, B_v, lm, q, 16, c, H_kv, 10000.0, outliers=outl)
    assert idx.shape[-1] == (2 + 3) * c
    for l in range(G):
        for b in range(Bsz):
            for g in range(H_kv):
                rows = O.sr_select(q[l, b, g * n_rep:(g + 1) * n_rep], lm[b, l, g], 16, c, T, outl[l, b, g])
                assert cnt[l, b, g] == len(rows)
                np.testing.assert_array_equal(idx[l, b, g, :len(rows)], rows)
                assert np.all(idx[l, b, g, len(rows):] == -1)
                for j in outl[l, b, g]:
                    assert j * c in rows
