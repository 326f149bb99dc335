"""Pins for the oracle's cross-layer factorisation (Sec. 3.1, Eq. 1)."""
import numpy as np
import pytest

from oracle import xkv_oracle as O


def _known_svd(T, n, s, seed):
    """X = U diag(s) V^T with orthonormal U, V drawn independently of the oracle."""
    rng = np.random.default_rng(seed)
    U, _ = np.linalg.qr(rng.standard_normal((T, len(s))))
    V, _ = np.linalg.qr(rng.standard_normal((n, len(s))))
    return (U * np.asarray(s)[None, :]) @ V.T


def _split(X, W):
    d = X.shape[1] // W
    return [X[:, i * d:(i + 1) * d] for i in range(W)]


def test_full_rank_reproduces_input():
    rng = np.random.default_rng(0)
    X = [rng.standard_normal((40, 8)) for _ in range(3)]          # T=40 > W*d=24
    A, B, _ = O.clf_factorize(X, 24)
    for l in range(3):
        np.testing.assert_allclose(A @ B[l], X[l], atol=1e-10)


def test_eckart_young_residual_closed_form():
    s = np.array([9.0, 7.0, 4.0, 2.5, 1.0, 0.5, 0.25, 0.1])
    X = _known_svd(50, 12, s, 1)
    for r in (1, 3, 5, 8):
        A, B, sig = O.clf_factorize(_split(X, 3), r)
        res = np.linalg.norm(X - A @ np.concatenate(B, axis=1)) ** 2
        assert abs(res - (s[r:] ** 2).sum()) < 1e-9
        np.testing.assert_allclose(sig[:8], s, rtol=1e-10)           # known singular values


def test_factor_invariants():
    rng = np.random.default_rng(2)
    X = [rng.standard_normal((64, 6)) for _ in range(4)]
    A, B, sig = O.clf_factorize(X, 10)
    Bcat = np.concatenate(B, axis=1)
    np.testing.assert_allclose(Bcat @ Bcat.T, np.eye(10), atol=1e-12)   # rows of V_r^T orthonormal
    gram = A.T @ A                                                      # A = U Sigma  =>  A^T A = Sigma^2
    np.testing.assert_allclose(gram, np.diag(sig[:10] ** 2), atol=1e-9)
    assert np.all(np.diff(sig) <= 1e-12)
    # Sigma sits in A, not in B: the columns of A carry the scale
    np.testing.assert_allclose(np.linalg.norm(A, axis=0), sig[:10], rtol=1e-10)


def test_exact_low_rank_input_is_recovered():
    rng = np.random.default_rng(3)
    Z = rng.standard_normal((80, 5))                                   # shared token subspace
    X = [Z @ rng.standard_normal((5, 16)) for _ in range(4)]
    A, B, sig = O.clf_factorize(X, 5)
    for l in range(4):
        np.testing.assert_allclose(A @ B[l], X[l], atol=1e-9)
    assert sig[5] < 1e-9 * sig[0]
    # the shared-basis point of the method: each layer alone also has rank 5, so a per-layer
    # factorisation at the same rank stores W bases where the window stores one
    A1, B1, _ = O.clf_factorize([X[0]], 5)
    np.testing.assert_allclose(A1 @ B1[0], X[0], atol=1e-9)


def test_single_layer_window_is_plain_truncated_svd():
    rng = np.random.default_rng(4)
    X = rng.standard_normal((30, 10))
    A, B, _ = O.clf_factorize([X], 4)
    # best rank-4 approximation projects X onto its top-4 right singular subspace
    w, V = np.linalg.eigh(X.T @ X)
    Vr = V[:, ::-1][:, :4]
    np.testing.assert_allclose(A @ B[0], X @ Vr @ Vr.T, atol=1e-9)


def test_no_centering_is_applied():
    # a constant offset is part of the signal: rank-1 input of all ones is reproduced exactly
    X = np.ones((20, 6))
    A, B, _ = O.clf_factorize([X[:, :3], X[:, 3:]], 1)
    np.testing.assert_allclose(A @ np.concatenate(B, axis=1), X, atol=1e-12)


def test_rank_out_of_range():
    with pytest.raises(ValueError):
        O.clf_factorize([np.ones((4, 3))], 4)


def test_bf16_round_ties_to_even_and_exact_values():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -7, -0.0, 3.140625], dtype=np.float32)
    # bf16 has 8 significand bits: spacing at 1.0 is 2^-7; halves round to even
    want = np.array([1.0, 1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, -0.0, 3.140625], dtype=np.float32)
    got = O.bf16_round(x)
    np.testing.assert_array_equal(got, want)
    assert np.signbit(got[4])
    import torch
    y = np.random.default_rng(5).standard_normal(1000).astype(np.float32)
    np.testing.assert_array_equal(O.bf16_round(y), torch.from_numpy(y).bfloat16().float().numpy())


# ---- the randomised factorisation (App. "Custom SVD Kernel"): pinned against the exact one above

def _decaying(T, N, rank, noise, seed):
    rng = np.random.default_rng(seed)
    s = 1.0 / np.arange(1, rank + 1)
    X = (rng.standard_normal((T, rank)) * s) @ rng.standard_normal((rank, N)) / np.sqrt(rank)
    X += noise * np.sqrt((X ** 2).mean()) * rng.standard_normal((T, N))
    return O.bf16_round(X.astype(np.float32)).astype(np.float64)


def test_cholesky_qr_gives_an_orthonormal_basis_of_the_same_span():
    rng = np.random.default_rng(0)
    U = rng.standard_normal((300, 40)) * np.logspace(0, -7, 40)          # condition number 1e7
    Z = O.cholesky_qr(U)
    assert np.abs(Z.T @ Z - np.eye(40)).max() < 1e-8
    # same column space: projecting U on span(Z) changes nothing
    assert np.abs(Z @ (Z.T @ U) - U).max() < 1e-9 * np.abs(U).max()
    # against the library's Householder QR: identical projector
    Q, _ = np.linalg.qr(U)
    assert np.abs(Z @ Z.T - Q @ Q.T).max() < 1e-6


def test_randomized_factorisation_is_close_to_the_optimum_and_b_is_orthonormal():
    X = _decaying(1500, 256, 48, 0.01, 1)
    r, l = 64, 128
    omega = O.bf16_round(np.random.default_rng(2).standard_normal((256, l)).astype(np.float32))
    A, V, sig = O.clf_randomized(X, r, omega, power_iters=2)
    sv = np.linalg.svd(X, compute_uv=False)
    res = ((X - A.astype(np.float64) @ V.astype(np.float64).T) ** 2).sum()
    assert res <= 1.15 * (sv[r:] ** 2).sum()      # Eckart-Young optimum; the flat noise tail is what the 32 extra directions cannot order
    assert np.abs(V.T.astype(np.float64) @ V - np.eye(r)).max() < 1e-2    # bf16 storage
    np.testing.assert_allclose(sig[:48], sv[:48], rtol=1e-2)
    # more power iterations never hurt, none at all is worse
    A0, V0, _ = O.clf_randomized(X, r, omega, power_iters=0)
    res0 = ((X - A0.astype(np.float64) @ V0.astype(np.float64).T) ** 2).sum()
    assert res <= res0 * 1.001


def test_randomized_factorisation_recovers_exactly_low_rank_input():
    rng = np.random.default_rng(3)
    X = O.bf16_round((rng.standard_normal((800, 20)) @ rng.standard_normal((20, 128)) / 4).astype(np.float32)).astype(np.float64)
    omega = O.bf16_round(rng.standard_normal((128, 64)).astype(np.float32))
    A, V, sig = O.clf_randomized(X, 32, omega, power_iters=1)
    res = ((X - A.astype(np.float64) @ V.astype(np.float64).T) ** 2).sum() / (X ** 2).sum()
    assert res < 1e-4                                                     # rounding of X, A and V to bf16 only
    # with l = N the subspace is everything and the result is the exact truncated SVD up to that rounding
    om_full = O.bf16_round(rng.standard_normal((128, 128)).astype(np.float32))
    Xn = _decaying(600, 128, 128, 0.0, 4)
    A2, V2, _ = O.clf_randomized(Xn, 32, om_full, power_iters=0)
    sv = np.linalg.svd(Xn, compute_uv=False)
    res2 = ((Xn - A2.astype(np.float64) @ V2.astype(np.float64).T) ** 2).sum()
    assert abs(res2 / (sv[32:] ** 2).sum() - 1.0) < 2e-2
