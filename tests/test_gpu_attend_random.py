"""Reconstruct+attend on randomly drawn shapes against the oracle: head widths, query heads per KV head from 1 to 16
(all three widths of the fused kernel), ragged ranks from 8 to 520, windows of one to 64 problems (both merge
kernels), unsorted index sets of random length per problem (empty ones included)."""
import numpy as np
import pytest

from paper_2503_18893_b200 import synth
from tests import _cases as C

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.mark.parametrize("case", range(24))
def test_attention_of_a_random_shape_is_the_oracles(case):
    rng = np.random.default_rng(9000 + case)
    d_h = int(rng.choice([64, 128]))
    H_kv = int(rng.choice([1, 2, 4]))
    n_rep = int(rng.choice([1, 2, 4, 7, 8, 16]))
    G = int(rng.choice([1, 2, 4]))
    B = int(rng.choice([1, 2, 8]))
    lim = G * H_kv * d_h                                       # a rank cannot exceed the width of the concatenated cache
    r_k = min(int(rng.choice([8, 64, 96, 256, 520])), lim) // 8 * 8
    r_v = min(int(rng.choice([8, 64, 136, 256, 512])), lim) // 8 * 8
    T = int(rng.integers(300, 3000))
    rows = min(int(rng.integers(1, 400)), T)
    s = synth.config(1, T=T, k=512, G=G, H_kv=H_kv, H_q=H_kv * n_rep, d_h=d_h, batch=B, r_k=r_k, r_v=r_v,
                     seed=9000 + case)
    inp = C.case_from_factors(s)
    idx = synth.fixed_index_set(s, rows).numpy()
    cnt = rng.integers(0, rows + 1, size=(s.G, s.batch, s.H_kv)).astype(np.int32)
    g = C.GpuCase(s, inp)
    gout, glse = g.attend(idx, cnt, 0)
    assert g.status() == (0, 0)
    _, _, oout, olse = C.oracle_step(s, inp, 0, sel_idx=idx, sel_cnt=cnt)
    what = dict(d_h=d_h, H_kv=H_kv, n_rep=n_rep, G=G, B=B, r_k=r_k, r_v=r_v, T=T, rows=rows)
    empty = np.isneginf(olse)
    assert np.array_equal(np.isneginf(glse), empty), what
    assert np.all(gout[empty] == 0), what
    if (~empty).any():
        assert C.rel_err(gout[~empty], oout[~empty]) <= TOL, what
        np.testing.assert_allclose(glse[~empty], olse[~empty], atol=2e-2, err_msg=str(what))
    g.close()
