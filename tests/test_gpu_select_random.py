"""Algorithm 2 on randomly drawn shapes against the oracle, bit for bit: head widths, group sizes, chunk sizes,
budgets from one token to more than the context, contexts beyond one top-k super-block, forced chunks (in and out
of range), and landmark/query values coarse enough that many scores tie exactly -- the cases where the order of
equal keys and the edges of the selection kernels' tiles decide the answer."""
import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2503_18893_b200 import synth, workload
from tests import _cases as C

pytestmark = pytest.mark.gpu


def _draw_case(case):
    rng = np.random.default_rng(7000 + case)
    d_h = int(rng.choice([64, 128]))
    H_kv = int(rng.choice([1, 2, 4]))
    n_rep = int(rng.choice([1, 2, 4, 7, 16]))
    G = int(rng.choice([1, 2]))
    B = int(rng.choice([1, 2]))
    c = int(rng.choice([8, 8, 8, 16, 4]))
    T = int(rng.integers(9, 70000)) if case % 4 else int(rng.integers(130000, 300000))
    k = int(rng.integers(1, min(T, 20000) + 50))
    n_out = int(rng.choice([0, 0, 3, 40]))
    return rng, dict(d_h=d_h, H_kv=H_kv, n_rep=n_rep, G=G, B=B, c=c, T=T, k=k, n_out=n_out, mode=case % 3)


@pytest.mark.parametrize("case", range(36))
def test_selection_of_a_random_shape_is_the_oracles(case):
    rng, p = _draw_case(case)
    d_h, H_kv, n_rep, G, B, c, T, k, n_out = (p[x] for x in ("d_h", "H_kv", "n_rep", "G", "B", "c", "T", "k", "n_out"))
    n_c = -(-T // c)
    s = synth.config(1, T=T, k=k, G=G, H_kv=H_kv, H_q=H_kv * n_rep, d_h=d_h, batch=B, c=c, r_k=8, r_v=8,
                     seed=7000 + case)
    lm = synth.normal(synth.stream_key(s.seed, 91), (B, G, H_kv, n_c, d_h))
    q = synth.normal(synth.stream_key(s.seed, 92), (1, G, B, H_kv * n_rep, d_h))
    if p["mode"] == 1:                    # half-integer landmarks, integer queries: scores on a coarse grid
        lm, q = torch.round(lm * 2) / 2, torch.round(q)
    if p["mode"] == 2:                    # +-1 landmarks, sparse +-1 queries: a handful of distinct scores
        lm, q = torch.sign(lm), torch.sign(q) * (torch.rand(q.shape, generator=torch.Generator().manual_seed(case)) < 0.1)
    lm, q = lm.to(torch.bfloat16), q.to(torch.bfloat16)
    A = torch.zeros((B, T, 8), dtype=torch.bfloat16)
    Bm = torch.zeros((B, G, 8, H_kv * d_h), dtype=torch.bfloat16)
    g = C.GpuCase(s, workload.GroupInputs(A, A.clone(), Bm, Bm.clone(), lm, q))
    outl = None
    if n_out:
        outl = rng.integers(-2, n_c + 3, size=(G, B, H_kv, n_out)).astype(np.int32)
        o_dev = torch.from_numpy(outl).cuda()
        g.xkv.xkv_group_set_outliers(g.grp, o_dev, n_out)
    k_cap = (-(-k // c) + n_out) * c
    idx = torch.full((G, B, H_kv, k_cap), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((G, B, H_kv), -7, dtype=torch.int32, device="cuda")
    g.xkv.xkv_sr_select(g.grp, 0, G, g.inp.q[0], k, idx, cnt)
    torch.cuda.synchronize()
    assert g.status() == (0, 0)
    gi, gc = idx.cpu().numpy(), cnt.cpu().numpy()
    qf, lf = C.f32(q[0]), C.f32(lm)
    for l in range(G):
        for b in range(B):
            for h in range(H_kv):
                rows = O.sr_select(qf[l, b, h * n_rep:(h + 1) * n_rep], lf[b, l, h], k, c, T,
                                   None if outl is None else outl[l, b, h])
                assert gc[l, b, h] == len(rows), (p, l, b, h)
                np.testing.assert_array_equal(gi[l, b, h, :len(rows)], rows, err_msg=str((p, l, b, h)))
                assert np.all(gi[l, b, h, len(rows):] == -1), (p, l, b, h)
    g.close()
