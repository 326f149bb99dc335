"""The segment merge of windows with many problems (one CTA per group of query heads instead of one per head): parity
of reconstruct+attend against the oracle on shapes whose problem count takes that kernel, for both head widths,
group sizes 4, 7 and 16, ragged ranks, empty problems, and with an uncompressed tail."""
import numpy as np
import pytest

from paper_2503_18893_b200 import synth
from tests import _cases as C

pytestmark = pytest.mark.gpu
TOL = 2e-2

# (name, overrides on config 1).  Problems x heads per KV head must exceed twice the SM count (2 x 148).
CASES = [
    ("d128_rep4", dict(T=1024, k=256, G=4, batch=8, H_kv=4, H_q=16, d_h=128, r_k=64, r_v=64)),
    ("d128_rep7_ragged_rank", dict(T=1024, k=256, G=2, batch=8, H_kv=4, H_q=28, d_h=128, r_k=96, r_v=160)),
    ("d128_rep16", dict(T=1024, k=256, G=2, batch=6, H_kv=2, H_q=32, d_h=128, r_k=64, r_v=72)),
    ("d64_rep4", dict(T=1024, k=256, G=4, batch=8, H_kv=4, H_q=16, d_h=64, r_k=64, r_v=64)),
    ("d64_rep7", dict(T=1024, k=256, G=2, batch=8, H_kv=4, H_q=28, d_h=64, r_k=96, r_v=136)),
]


def _ran(before, after):
    return {f for f in ("merge", "merge_multi") if after[f] > before[f]}


@pytest.mark.parametrize("name,over", CASES, ids=[c[0] for c in CASES])
def test_reconstruct_attend_with_the_grouped_merge(name, over):
    from paper_2503_18893_b200 import xkv
    s = synth.config(1, **over)
    assert s.G * s.batch * s.H_kv * s.n_rep > 2 * 148
    inp = C.case_from_factors(s)
    idx = synth.fixed_index_set(s, 200).numpy()                    # unsorted, not chunk aligned: two tiles, one ragged
    cnt = np.full((s.G, s.batch, s.H_kv), 200, dtype=np.int32)
    cnt[0, 0, 0] = 0                                               # an empty problem
    cnt[s.G - 1, s.batch - 1, s.H_kv - 1] = 1                      # a one-row problem
    cnt[0, 1, 0] = 129
    g = C.GpuCase(s, inp)
    before = xkv.xkv_debug_launch_counts()
    gout, glse = g.attend(idx, cnt, 0)
    assert _ran(before, xkv.xkv_debug_launch_counts()) == {"merge_multi"}
    assert g.status() == (0, 0)
    _, _, oout, olse = C.oracle_step(s, inp, 0, sel_idx=idx, sel_cnt=cnt)
    empty = np.isneginf(olse)
    assert empty.sum() == s.n_rep and np.array_equal(np.isneginf(glse), empty)
    assert np.all(gout[empty] == 0)
    assert C.rel_err(gout[~empty], oout[~empty]) <= TOL, name
    np.testing.assert_allclose(glse[~empty], olse[~empty], atol=2e-2)
    g.close()


@pytest.mark.parametrize("name,over", [CASES[1], CASES[3]], ids=[CASES[1][0], CASES[3][0]])
def test_grouped_merge_with_an_uncompressed_tail(name, over):
    from oracle import xkv_oracle as O
    from paper_2503_18893_b200 import xkv
    s = synth.config(1, **over)
    inp = C.case_from_factors(s)
    rows = np.arange(0, 64)
    K = O.sr_reconstruct(C.f32(inp.A_k)[0], C.f32(inp.B_k)[0, 0][:, :s.d_h], rows)
    lens = [(37 * b) % 300 for b in range(s.batch)]                # per-sequence lengths, one of them 0
    tk, tv = synth.make_tail(s, 300, key_rms=float(np.sqrt((K ** 2).mean())), value_rms=1.0)
    idx = synth.fixed_index_set(s, 96).numpy()
    cnt = np.full((s.G, s.batch, s.H_kv), 96, dtype=np.int32)
    cnt[0, 0, 0] = 0                                               # sequence 0 has no tail either: an empty problem
    g = C.GpuCase(s, inp)
    before = xkv.xkv_debug_launch_counts()
    gout, glse = g.attend_tail(idx, cnt, tk, tv, lens)
    assert _ran(before, xkv.xkv_debug_launch_counts()) == {"merge_multi"}
    assert g.status() == (0, 0)
    oout, olse = C.oracle_step_with_tail(s, inp, idx, cnt, tk, tv, lens)
    empty = np.isneginf(olse)
    assert np.array_equal(np.isneginf(glse), empty) and np.all(gout[empty] == 0)
    assert C.rel_err(gout[~empty], oout[~empty]) <= TOL, name
    np.testing.assert_allclose(glse[~empty], olse[~empty], atol=2e-2)
    g.close()
