"""Cross-layer factorisation on the GPU (Eq. 1 by the randomised SVD of App. "Custom SVD Kernel") against the
oracle.  Factors are never compared element by element (signs and rotations inside close singular values are not
unique): the residual ||X - A B||_F^2 is compared with the Eckart-Young optimum of the oracle's exact SVD and with
the oracle's restatement of the same randomised algorithm, B must have orthonormal rows, A must be the projection
X B^T, and a decode step on the GPU-made factors must match the oracle on the same factors."""
import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2503_18893_b200 import synth, workload
from tests import _cases as C

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (192, 300, 520), (576, 2048, 256), (64, 1000, 4096)])
def test_tensor_core_product_against_fp64(M, N, K):
    from paper_2503_18893_b200 import xkv
    a = synth.normal(synth.stream_key(5, M, N, K), (K, M)).to(torch.bfloat16)
    b = synth.normal(synth.stream_key(6, M, N, K), (N, K)).to(torch.bfloat16)
    Cd = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    xkv.xkv_debug_gemm(a.cuda(), b.cuda(), Cd, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    ref = C.f32(a).astype(np.float64).T @ C.f32(b).astype(np.float64).T
    np.testing.assert_allclose(Cd.cpu().numpy(), ref, rtol=1e-4, atol=1e-3 * np.sqrt(K))


def _factorize_gpu(X, G, d, r, oversample, q, seed):
    from paper_2503_18893_b200 import xkv
    T = X.shape[0]
    cfg = xkv.make_clf_config(T=T, G=G, d=d, r=r, oversample=oversample, power_iters=q)
    l = xkv.xkv_clf_rank_l(cfg)
    omega = synth.normal(synth.stream_key(seed, 31), (G * d, l)).to(torch.bfloat16)
    ws = torch.empty(xkv.xkv_clf_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    A = torch.empty((T, r), dtype=torch.bfloat16, device="cuda")
    B = torch.empty((G, r, d), dtype=torch.bfloat16, device="cuda")
    sig = torch.empty(r, dtype=torch.float32, device="cuda")
    xkv.xkv_clf_factorize(cfg, X.cuda().contiguous(), omega.cuda(), ws, A, B, sig)
    torch.cuda.synchronize()
    st, flags = xkv.xkv_clf_status(ws)
    assert (st, flags) == (0, 0)
    return A, B, sig, omega


@pytest.mark.parametrize("name,over,r,p,q,near", [
    ("tiny_T2048_N256_r64", dict(T=2048), 64, 32, 2, 1.15),
    ("ragged_T1001_N256_r40", dict(T=1001), 40, 24, 2, 1.15),
    ("N1024_r128_decaying", dict(T=4096, G=4, H_kv=2, d_h=128, rho=64, decay=1.0, noise=0.01, noise_abs=False), 128, 64, 2, 1.15),
    # a sketch of 832 columns: wider than the blocked triangular solve holds in shared memory, so the row-wise one
    # runs.  Two thirds of the kept directions lie in the flat noise tail, which no sketch can order: the bound against
    # the optimum is loose here, the one against the oracle's run of the same algorithm is what counts.
    ("N1024_r768_wide_sketch", dict(T=4096, G=4, H_kv=2, d_h=128, rho=512, decay=1.0, noise=0.01, noise_abs=False), 768, 64, 1, 2.0),
])
def test_clf_residual_orthonormality_and_projection(name, over, r, p, q, near):
    s = synth.config(1, **over)
    K, _ = synth.make_kv(s)                                           # (G, T, d) bf16
    X = torch.cat([K[l] for l in range(s.G)], dim=1)                  # (T, G d): the layers side by side (Eq. 1)
    A, B, sig, omega = _factorize_gpu(X, s.G, s.d, r, p, q, seed=1234)
    Xf = C.f32(X).astype(np.float64)
    Af = C.f32(A).astype(np.float64)
    V = np.concatenate([C.f32(B[g]) for g in range(s.G)], axis=1).astype(np.float64).T      # (G d, r), B = V^T
    sv = np.linalg.svd(Xf, compute_uv=False)
    optimum = float((sv[r:] ** 2).sum())                              # Eckart-Young
    res = float(((Xf - Af @ V.T) ** 2).sum())
    # the oracle's restatement of the same algorithm on the same test matrix
    Ao, Vo, so = O.clf_randomized(Xf, r, C.f32(omega), q)
    res_o = float(((Xf - Ao.astype(np.float64) @ Vo.astype(np.float64).T) ** 2).sum())
    assert res <= near * optimum, (name, res / optimum)               # the randomised subspace is near the optimum
    assert res <= 1.03 * res_o, (name, res / res_o)                   # and the fp32/bf16 GPU pipeline loses nothing on fp64
    assert np.abs(V.T @ V - np.eye(r)).max() <= 2e-2                  # orthonormal rows of B (bf16 storage)
    proj = Xf @ V                                                     # A = X B^T
    assert np.abs(Af - proj).max() <= 2e-2 * np.abs(proj).max()
    np.testing.assert_allclose(C.f32(sig), sv[:r], rtol=2e-2, atol=2e-3 * sv[0])


def test_exactly_low_rank_input_is_recovered():
    T, G, d, rank = 1536, 2, 128, 24
    Z = synth.normal(synth.stream_key(9, 1), (T, rank))
    Mx = synth.normal(synth.stream_key(9, 2), (rank, G * d))
    X = (Z @ Mx / np.sqrt(rank)).to(torch.bfloat16)
    A, B, sig, _ = _factorize_gpu(X, G, d, 32, 32, 1, seed=77)
    Xf = C.f32(X).astype(np.float64)
    V = np.concatenate([C.f32(B[g]) for g in range(G)], axis=1).astype(np.float64).T
    res = ((Xf - C.f32(A).astype(np.float64) @ V.T) ** 2).sum() / (Xf ** 2).sum()
    assert res <= 1e-4                                                # bf16 rounding of X, A and B only


def test_decode_step_on_gpu_made_factors():
    """Factorise raw caches on the GPU, build landmarks with the library, run the decode step, compare with the
    oracle on the same factors (the factors are inputs of that comparison, whoever made them)."""
    from paper_2503_18893_b200 import xkv
    s = synth.config(1, T=2048, k=256)
    Kc, Vc = synth.make_kv(s)
    Xk = torch.cat([Kc[l] for l in range(s.G)], dim=1)
    Xv = torch.cat([Vc[l] for l in range(s.G)], dim=1)
    A_k, B_k, _, _ = _factorize_gpu(Xk, s.G, s.d, s.r_k, 32, 2, seed=1)
    A_v, B_v, _, _ = _factorize_gpu(Xv, s.G, s.d, s.r_v, 32, 2, seed=2)
    lm = torch.empty((1, s.G, s.H_kv, s.n_c, s.d_h), dtype=torch.bfloat16, device="cuda")
    xkv.xkv_build_landmarks(Kc.unsqueeze(0).cuda().contiguous(), lm, G=s.G, batch=1, T=s.T, H_kv=s.H_kv, d_h=s.d_h,
                            chunk=s.c, rope_base=s.rope_base)
    torch.cuda.synchronize()
    inp = workload.GroupInputs(A_k.unsqueeze(0).cpu(), A_v.unsqueeze(0).cpu(), B_k.unsqueeze(0).cpu(),
                               B_v.unsqueeze(0).cpu(), lm.cpu(), synth.make_queries(s, 1))
    g = C.GpuCase(s, inp)
    gidx, gcnt = g.select(0)
    gout, glse = g.attend(gidx, gcnt, 0)
    oidx, ocnt, oout, olse = C.oracle_step(s, inp, 0)
    np.testing.assert_array_equal(gidx, oidx)
    assert C.rel_err(gout, oout) <= 2e-2
    # and the compressed cache stands for the raw one: rank 64 of a rank-32 signal plus 0.25 % of noise energy
    Kf = C.f32(Kc[0]).astype(np.float64)
    rec = C.f32(A_k).astype(np.float64) @ C.f32(B_k[0]).astype(np.float64)
    assert ((rec - Kf) ** 2).sum() / (Kf ** 2).sum() <= 5e-3
    g.close()
