"""Parity of the dense decode-attention baseline (plain softmax attention over an uncompressed bf16 cache, the
arm selective reconstruction is compared with) against the oracle's softmax attention over all rows (`attend`, itself pinned by the row-by-row `dense_attend`)."""
import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2503_18893_b200 import synth
from tests import _cases as C

pytestmark = pytest.mark.gpu
TOL = 2e-2       # max relative error per output vector

# (name, shape overrides on config 1, cache capacity, per-sequence lengths)
D128 = dict(d_h=128, r_k=64, r_v=64, T=256, k=64)
CASES = [
    ("one_tile_per_cta_ragged", dict(**D128), 1000, [1000]),
    ("two_tiles_per_cta_ragged", dict(**D128), 40000, [39999]),              # beyond the tail limit: several tiles per CTA
    ("three_tiles_per_cta_lengths", dict(batch=3, **D128), 70000, [70000, 0, 33001]),
    ("rep7", dict(H_kv=2, H_q=14, **D128), 33000, [32897]),
    ("rep16", dict(H_kv=1, H_q=16, **D128), 2000, [1999]),
    ("d64_cuda_cores", dict(T=256, k=64), 3000, [2500]),
]


@pytest.mark.parametrize("name,over,cap,lens", CASES, ids=[c[0] for c in CASES])
def test_dense_attend_parity(name, over, cap, lens):
    s = synth.config(1, **over)
    inp = C.case_from_factors(s)
    g = C.GpuCase(s, inp)
    x = g.xkv
    K, V = synth.make_tail(s, cap, key_rms=1.0, value_rms=1.0, device="cuda")
    ws = torch.empty(x.xkv_dense_workspace_bytes(g.grp, cap), dtype=torch.uint8, device="cuda")
    out = torch.zeros((s.G, s.batch, s.H_q, s.d_h), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((s.G, s.batch, s.H_q), dtype=torch.float32, device="cuda")
    ln = torch.tensor(lens, dtype=torch.int32, device="cuda")
    before = x.xkv_debug_launch_counts()
    x.xkv_dense_attend(g.grp, 0, s.G, g.inp.q[0], K, V, ln, cap, ws, out, lse)
    torch.cuda.synchronize()
    after = x.xkv_debug_launch_counts()
    assert g.status() == (0, 0)
    assert after["dense"] == before["dense"] + 1 and after["fused"] == before["fused"]
    assert after["tail_tc" if s.d_h == 128 else "tail_cuda"] == before["tail_tc" if s.d_h == 128 else "tail_cuda"] + 1
    gout, glse = C.f32(out), lse.cpu().numpy()
    q = C.f32(inp.q[0])
    Kc, Vc = C.f32(K), C.f32(V)
    scale = 1.0 / np.sqrt(s.d_h)
    for l in range(s.G):
        for b in range(s.batch):
            for hk in range(s.H_kv):
                hs = slice(hk * s.n_rep, (hk + 1) * s.n_rep)
                n = lens[b]
                if n == 0:
                    assert np.all(gout[l, b, hs] == 0) and np.all(np.isneginf(glse[l, b, hs]))
                    continue
                o, ls = O.attend(q[l, b, hs], Kc[l, b, hk, :n], Vc[l, b, hk, :n], scale)
                if n <= 2000 and l == 0:      # the row-by-row routine, where it is affordable
                    np.testing.assert_allclose(O.dense_attend(q[l, b, hs], Kc[l, b, hk, :n], Vc[l, b, hk, :n], scale), o,
                                               rtol=1e-9, atol=1e-12)
                assert C.rel_err(gout[l, b, hs], o) <= TOL, (name, l, b, hk)
                np.testing.assert_allclose(glse[l, b, hs], ls, atol=2e-2)
    g.close()


def test_dense_attend_argument_checks():
    s = synth.config(1, T=256, k=64)                                        # d_h = 64
    inp = C.case_from_factors(s)
    g = C.GpuCase(s, inp)
    x = g.xkv
    with pytest.raises(x.XKVError) as e:
        x.xkv_dense_workspace_bytes(g.grp, 0)
    assert e.value.status == x.XKV_ERR_INVALID_ARG
    with pytest.raises(x.XKVError) as e:
        x.xkv_dense_workspace_bytes(g.grp, x.XKV_TAIL_MAX_ROWS + 1)         # long caches need d_h = 128
    assert e.value.status == x.XKV_ERR_UNSUPPORTED
    g.close()
