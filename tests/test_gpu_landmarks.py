"""Parity of the prefill side of the selector (App. B.1, Algorithm 1) against the oracle: landmarks (chunk means
of the post-RoPE keys), minimum within-chunk cosines and the static outlier chunks."""
import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2503_18893_b200 import synth
from tests import _cases as C

pytestmark = pytest.mark.gpu


def _run(s, K_list, n_out, rope_base):
    """K_list: per sequence a bf16 tensor (G, T, d).  Returns landmarks (B,G,H_kv,n_c,d_h), min_cos, outliers."""
    from paper_2503_18893_b200 import xkv
    keys = torch.stack(K_list).cuda().contiguous()                     # (B, G, T, d)
    lm = torch.full((s.batch, s.G, s.H_kv, s.n_c, s.d_h), float("nan"), dtype=torch.bfloat16, device="cuda")
    mc = torch.full((s.G, s.batch, s.H_kv, s.n_c), float("nan"), dtype=torch.float32, device="cuda")
    outl = torch.full((s.G, s.batch, s.H_kv, max(n_out, 1)), -9, dtype=torch.int32, device="cuda")
    xkv.xkv_build_landmarks(keys, lm, G=s.G, batch=s.batch, T=s.T, H_kv=s.H_kv, d_h=s.d_h, chunk=s.c,
                            rope_base=rope_base, min_cos=mc, n_outliers=n_out, outliers=outl if n_out else None)
    torch.cuda.synchronize()
    return C.f32(lm), mc.cpu().numpy(), outl.cpu().numpy()


CASES = [
    ("llama_like", dict(T=1003, H_kv=2, H_q=8, d_h=128), 6, 10000.0),          # ragged last chunk
    ("d64_one_head", dict(T=512, H_kv=1, H_q=4, d_h=64, c=16), 3, 10000.0),
    ("long_chunks_no_rope", dict(T=700, H_kv=2, H_q=4, d_h=128, c=48), 2, 0.0),  # c larger than one 32-row pass
    ("two_sequences", dict(T=256, H_kv=2, H_q=4, d_h=128, batch=2), 40, 500000.0),  # more outliers than chunks (32)
]


@pytest.mark.parametrize("name,over,n_out,rope_base", CASES, ids=[c[0] for c in CASES])
def test_landmarks_min_cos_and_outliers(name, over, n_out, rope_base):
    s = synth.config(1, **over)
    K_list = [synth.make_kv(s, 0, b)[0] for b in range(s.batch)]
    lm, mc, outl = _run(s, K_list, n_out, rope_base)
    for b in range(s.batch):
        Kf = C.f32(K_list[b])
        for l in range(s.G):
            heads = Kf[l].reshape(s.T, s.H_kv, s.d_h).transpose(1, 0, 2)            # (H_kv, T, d_h) before rotation
            ref = O.build_landmarks(heads, s.c, rope_base)                          # bf16-rounded fp64 means
            # the rounding to bf16 is decided by a sum formed in a different order: allow one unit in the last place
            tol = np.maximum(np.abs(ref), 1e-3) * 2.0 ** -7
            assert np.all(np.abs(lm[b, l] - ref) <= tol), name
            assert np.mean(lm[b, l] == ref) > 0.95                                  # and almost always the same value
            for g in range(s.H_kv):
                Kr = O.rope_rotate(heads[g], np.arange(s.T), rope_base) if rope_base > 0 else heads[g].astype(np.float64)
                m = O.min_chunk_cosine(Kr, s.c)
                np.testing.assert_allclose(mc[l, b, g], m, atol=2e-5)
                # outliers: exact where the oracle's margin is clear, otherwise any chunk inside the margin is valid
                got = outl[l, b, g]
                o_eff = min(n_out, s.n_c)
                assert np.all(got[o_eff:] == -1)
                got = got[:o_eff]
                assert np.all(np.diff(got) > 0) and got.min() >= 0 and got.max() < s.n_c
                want = O.static_outliers(Kr, s.c, n_out)
                if o_eff < s.n_c:
                    srt = np.sort(m)
                    cut = srt[o_eff - 1]
                    must = set(np.nonzero(m < cut - 1e-4)[0].tolist())
                    may = set(np.nonzero(m <= cut + 1e-4)[0].tolist())
                    assert must <= set(got.tolist()) <= may
                    if srt[o_eff] - cut > 2e-4:
                        np.testing.assert_array_equal(got, want)
                else:
                    np.testing.assert_array_equal(got, np.arange(s.n_c))


def test_landmarks_feed_the_selector():
    """Landmarks and outliers computed on the GPU drive xkv_sr_select like the ones the harness computes."""
    s = synth.config(1, T=1024, k=64, H_kv=2, H_q=8)
    inp = C.case_from_factors(s)
    # keys of the window as the factors represent them (before rotation), rounded to bf16
    K = torch.stack([(inp.A_k[0].float() @ inp.B_k[0, l].float()) for l in range(s.G)]).to(torch.bfloat16)
    lm, mc, outl = _run(s, [K], 4, s.rope_base)
    g = C.GpuCase(s, inp)
    lm_dev = torch.from_numpy(lm).to(torch.bfloat16).cuda()
    from paper_2503_18893_b200 import xkv
    grp = xkv.create_from_tensors(g.inp.A_k, g.inp.A_v, g.inp.B_k, g.inp.B_v, lm_dev, H_kv=s.H_kv, H_q=s.H_q, k_max=s.k,
                                  chunk=s.c, rope_base=s.rope_base)
    o_dev = torch.from_numpy(outl).cuda()
    xkv.xkv_group_set_outliers(grp, o_dev, 4)
    k_cap = (-(-s.k // s.c) + 4) * s.c
    idx = torch.full((s.G, s.batch, s.H_kv, k_cap), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((s.G, s.batch, s.H_kv), -7, dtype=torch.int32, device="cuda")
    xkv.xkv_sr_select(grp, 0, s.G, g.inp.q[0], s.k, idx, cnt)
    torch.cuda.synchronize()
    oidx, ocnt, _, _ = O.sr_decode_step(C.f32(inp.A_k), C.f32(inp.A_v), C.f32(inp.B_k), C.f32(inp.B_v), lm,
                                        C.f32(inp.q[0]), k=s.k, c=s.c, H_kv=s.H_kv, rope_base=s.rope_base,
                                        outliers=outl)
    np.testing.assert_array_equal(idx.cpu().numpy(), oidx)
    np.testing.assert_array_equal(cnt.cpu().numpy(), ocnt)
    for j in outl.reshape(-1, 4)[0]:
        assert j * s.c in idx.cpu().numpy()[0, 0, 0]
    xkv.xkv_group_destroy(grp)
    g.close()
