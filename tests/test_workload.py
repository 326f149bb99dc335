"""Input preparation (no GPU): the generator is deterministic, the recipes have the structure they claim, and
the test cases take their landmarks from the oracle's Algorithm 1."""
import numpy as np
import torch

from oracle import xkv_oracle as O
from paper_2503_18893_b200 import synth, workload


def test_generator_is_deterministic_and_standard_normal():
    a = synth.normal(synth.stream_key(7, 1, 2), (4096, 8))
    b = synth.normal(synth.stream_key(7, 1, 2), (4096, 8), chunk=1000)     # chunking does not change the stream
    assert torch.equal(a, b)
    assert not torch.equal(a, synth.normal(synth.stream_key(7, 1, 3), (4096, 8)))
    assert abs(a.mean()) < 0.03 and abs(a.std() - 1) < 0.03
    assert abs((a ** 4).mean() - 3.0) < 0.3                                # normal kurtosis
    # first words of the counter stream, recomputed with Python integers
    key = synth.stream_key(7, 1, 2)
    w = synth.uniform_bits(key, 0, 3, "cpu").tolist()
    for i, v in enumerate(w):
        assert (v & ((1 << 64) - 1)) == synth._mix_py(key + (i + 1) * 0x9E3779B97F4A7C15)


def test_kv_recipe_has_a_shared_low_rank_token_subspace():
    s = synth.config(1, T=512)
    K, V = synth.make_kv(s)
    assert K.shape == (2, 512, 128) and K.dtype == torch.bfloat16
    X = torch.cat([K[0], K[1]], dim=1).double()
    sv = torch.linalg.svdvals(X)
    assert sv[31] > 4 * sv[32]                                             # rank-32 signal over the noise floor
    assert abs(K.float().pow(2).mean() - 1) < 1e-2


def test_direct_factors_are_in_factorised_form():
    s = synth.config(1)
    A_k, A_v, B_k, B_v = synth.make_factors(s)
    Bcat = torch.cat([B_k[0, l].float() for l in range(s.G)], dim=1)
    assert torch.allclose(Bcat @ Bcat.T, torch.eye(s.r_k), atol=2e-2)      # orthonormal rows (bf16 rounding)
    X = A_k[0].float() @ B_k[0, 0].float()
    assert abs(X.pow(2).mean() - 1) < 0.1
    idx = synth.fixed_index_set(s)
    assert idx.shape == (2, 1, 2, 256) and idx.min() >= 0 and idx.max() < s.T
    assert len(set(idx[0, 0, 0].tolist())) == 256
    assert not torch.equal(idx[0, 0, 0], idx[0, 0, 0].sort().values)       # left unsorted


def test_test_cases_take_landmarks_from_the_oracle():
    from tests import _cases as C
    s = synth.config(1, T=203, r_k=16, r_v=16)                             # ragged last chunk (203 = 25*8 + 3)
    inp = C.case_from_factors(s)
    assert inp.landmarks.shape == (1, s.G, s.H_kv, 26, s.d_h) and inp.landmarks.dtype == torch.bfloat16
    # the last landmark is the mean of the three rows present, of the rotated bf16 keys A_k B_k
    K = O.bf16_round(C.f32(inp.A_k[0]) @ C.f32(inp.B_k[0, 1]))[:, s.d_h:2 * s.d_h]
    tail = O.rope_rotate(K[200:203], np.arange(200, 203), s.rope_base).mean(axis=0)
    np.testing.assert_allclose(C.f32(inp.landmarks[0, 1, 1, 25]), tail, rtol=1e-2, atol=1e-3)


def test_byte_and_flop_model():
    s = synth.config(3)
    b = workload.algorithmic_bytes(s)
    assert b["landmarks"] == 4 * 16384 * 1024 * 2                          # 134 MB: every landmark once
    assert b["rows_issued"] == 32 * 4096 * 1024 * 2                        # 268 MB
    assert b["B"] == 4 * 1024 * 1024 * 2
    assert workload.algorithmic_flops(s) == 2 * O.flops_sr([4096] * 8, 128, 512, 512) * 4
