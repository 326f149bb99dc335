"""Parity at the full size of the headline workload (one window of config 3: T = 131072, r = 512, k = 4096,
32 problems), in the launch configuration the benchmark times (all layers of the window per call), on sampled
problems that the oracle evaluates one by one, plus properties of every problem that hold at any size."""
import numpy as np
import pytest
import torch

from paper_2503_18893_b200 import synth, workload
from tests import _cases as C

pytestmark = pytest.mark.gpu
TOL = 2e-2       # max relative error per output vector


def test_config3_full_size_sampled_problems():
    s = synth.config(3, n_groups=1)
    dev_inp = workload.make_group_inputs(s, 0, 1, "cuda")
    g = C.GpuCase(s, dev_inp)
    gidx, gcnt = g.select(0)
    gout, glse = g.attend(gidx, gcnt, 0)
    assert g.status() == (0, 0)

    # ---- every problem: Algorithm 2's output format
    assert np.all(gcnt == s.k)
    rows = gidx.reshape(-1, s.k_cap)
    assert np.all(rows >= 0) and np.all(rows < s.T)
    assert np.all(np.diff(rows, axis=1) > 0)                              # ascending, no repeats
    ch = rows.reshape(rows.shape[0], -1, s.c)
    assert np.all(ch[:, :, 0] % s.c == 0) and np.all(np.diff(ch, axis=2) == 1)   # whole aligned chunks
    assert np.all(np.isfinite(gout)) and np.all(np.isfinite(glse))

    # ---- sampled problems against the oracle (first, middle and last (layer, head))
    cpu = workload.GroupInputs(*(t.cpu() for t in (dev_inp.A_k, dev_inp.A_v, dev_inp.B_k, dev_inp.B_v,
                                                   dev_inp.landmarks, dev_inp.q)))
    problems = [(0, 0, 0), (1, 0, 5), (s.G - 1, 0, s.H_kv - 1)]
    oidx, ocnt, oout, olse = C.oracle_step(s, cpu, 0, problems=problems)
    for (l, b, hk) in problems:
        np.testing.assert_array_equal(gidx[l, b, hk], oidx[l, b, hk])
        assert gcnt[l, b, hk] == ocnt[l, b, hk]
        hs = slice(hk * s.n_rep, (hk + 1) * s.n_rep)
        assert C.rel_err(gout[l, b, hs], oout[l, b, hs]) <= TOL, (l, b, hk)
        np.testing.assert_allclose(glse[l, b, hs], olse[l, b, hs], atol=2e-2)
    g.close()
    del dev_inp
    torch.cuda.empty_cache()
