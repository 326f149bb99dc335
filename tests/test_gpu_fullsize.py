"""Parity at the full sizes of the benchmark configurations, in the launch configuration the benchmark times (all
layers of a window per call).  The oracle's selection is cheap, so the index sets of EVERY (layer, sequence, head)
problem are compared bit for bit; attention is compared on sampled problems that the oracle evaluates one by one;
format properties are checked on everything.  Inputs: factors drawn directly, landmarks made by the library's
Algorithm 1 kernel (its own parity is tests/test_gpu_landmarks.py) -- both sides read the same bf16 tensors."""
import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2503_18893_b200 import synth, workload
from tests import _cases as C

pytestmark = pytest.mark.gpu
TOL = 2e-2       # max relative error per output vector


def _cpu(t):
    return t.detach().float().cpu().numpy()


def _oracle_rows(s, inp, l, b, g, step=0):
    """Algorithm 2 for one problem: selected token rows, ascending."""
    q = _cpu(inp.q[step, l, b, g * s.n_rep:(g + 1) * s.n_rep])
    return O.sr_select(q, _cpu(inp.landmarks[b, l, g]), s.k, s.c, s.T)


def _oracle_attend(s, inp, l, b, g, rows, step=0, cache=None):
    """Eq. 3 + attention for one problem over the given rows.  `cache` keeps the widened bases of a sequence."""
    cache = {} if cache is None else cache
    if b not in cache:
        cache.clear()
        cache[b] = (_cpu(inp.A_k[b]), _cpu(inp.A_v[b]))
    A_k, A_v = cache[b]
    q = _cpu(inp.q[step, l, b, g * s.n_rep:(g + 1) * s.n_rep])
    hd = slice(g * s.d_h, (g + 1) * s.d_h)
    _, o, lse = O.sr_decode_problem(q, None, A_k, A_v, _cpu(inp.B_k[b, l][:, hd]), _cpu(inp.B_v[b, l][:, hd]), s.k,
                                    s.c, s.T, s.rope_base, 1.0 / np.sqrt(s.d_h), rows=rows)
    return o, lse


def _check_full_size(s, sample, step=0):
    """Select + attend on the GPU for one window of shape `s`; indices of all problems and attention of the
    problems in `sample` against the oracle."""
    inp = workload.make_group_inputs(s, 0, 1, "cuda")
    g = C.GpuCase(s, inp)
    gidx, gcnt = g.select(step)
    gout, glse = g.attend(gidx, gcnt, step)
    assert g.status() == (0, 0)

    # ---- every problem: Algorithm 2's output format
    k_rows = min(s.k_cap, s.T)
    assert np.all(gcnt == k_rows)
    rows = gidx.reshape(-1, s.k_cap)[:, :k_rows]
    assert np.all(rows >= 0) and np.all(rows < s.T)
    assert np.all(np.diff(rows, axis=1) > 0)                              # ascending, no repeats
    ch = rows.reshape(rows.shape[0], -1, s.c)
    assert np.all(ch[:, :, 0] % s.c == 0) and np.all(np.diff(ch, axis=2) == 1)   # whole aligned chunks
    assert np.all(np.isfinite(gout)) and np.all(np.isfinite(glse))

    # ---- every problem: the selected rows, bit for bit
    for l in range(s.G):
        for b in range(s.batch):
            for hk in range(s.H_kv):
                orows = _oracle_rows(s, inp, l, b, hk, step)
                assert gcnt[l, b, hk] == len(orows), (l, b, hk)
                np.testing.assert_array_equal(gidx[l, b, hk, :len(orows)], orows, err_msg=str((l, b, hk)))
                assert np.all(gidx[l, b, hk, len(orows):] == -1)

    # ---- sampled problems: attention
    cache = {}
    worst = 0.0
    for (l, b, hk) in sorted(sample, key=lambda p: p[1]):
        o, lse = _oracle_attend(s, inp, l, b, hk, gidx[l, b, hk, :gcnt[l, b, hk]], step, cache)
        hs = slice(hk * s.n_rep, (hk + 1) * s.n_rep)
        err = C.rel_err(gout[l, b, hs], o)
        worst = max(worst, err)
        assert err <= TOL, (l, b, hk, err)
        np.testing.assert_allclose(glse[l, b, hs], lse, atol=2e-2)
    g.close()
    del inp, g
    torch.cuda.empty_cache()
    return worst


def test_config3_batch1_every_index_set_and_six_sampled_problems():
    s = synth.config(3, n_groups=1)
    _check_full_size(s, [(0, 0, 0), (0, 0, 7), (1, 0, 5), (2, 0, 2), (3, 0, 4), (s.G - 1, 0, s.H_kv - 1)])


def test_config3_batch4():
    s = synth.config(3, n_groups=1, batch=4)
    _check_full_size(s, [(0, 0, 0), (1, 1, 3), (2, 2, 6), (3, 3, 7), (0, 3, 1), (2, 1, 4)])


def test_config4_qwen_shape_batch8_seven_heads_per_kv_head_heavy_rows():
    s = synth.config(4, n_groups=1)
    assert (s.T, s.batch, s.n_rep, s.r_k, s.k) == (65536, 8, 7, 256, 2048) and s.heavy_frac == 0.01
    _check_full_size(s, [(0, 0, 0), (1, 2, 3), (2, 5, 1), (3, 7, 3), (0, 4, 2), (2, 7, 0)])


@pytest.mark.parametrize("name,over", [
    ("rank_1024", dict(T=16384, r_k=1024, r_v=1024, k=4096)),            # the eight-block variant of the value side
    ("budget_16384", dict(T=65536, k=16384)),                             # 128 tiles per problem
    ("T_262144", dict(T=262144, k=4096)),                                 # more chunks than one top-k super-block
    ("tensor_bound_corner", dict(T=16384, r_k=1024, r_v=1024, k=16384)),  # the selection is every row
])
def test_config5_corners(name, over):
    s = synth.config(5, **over)
    _check_full_size(s, [(0, 0, 0), (1, 0, 3), (s.G - 1, 0, s.H_kv - 1)])


def test_config5_batch16_corner_many_problems():
    """512 problems in one call (the batch-16 corner of the stress sweep at T = 16K): every index set, and attention on
    problems of the first, a middle and the last sequence; the merge runs one CTA per problem here."""
    from paper_2503_18893_b200 import xkv
    s = synth.config(5, T=16384, r_k=256, r_v=256, k=1024, batch=16)
    before = xkv.xkv_debug_launch_counts()
    _check_full_size(s, [(0, 0, 0), (1, 7, 3), (2, 15, 7), (s.G - 1, 15, s.H_kv - 1), (0, 9, 5)])
    after = xkv.xkv_debug_launch_counts()
    assert after["merge_multi"] > before["merge_multi"] and after["merge"] == before["merge"]


def test_config3_window_with_an_8192_row_uncompressed_tail():
    """The default tail kernel at the headline head width and size: selected rows by the library, then one softmax
    over those rows and 8192 uncompressed rows, on sampled problems."""
    from paper_2503_18893_b200 import xkv
    s = synth.config(3, n_groups=1)
    inp = workload.make_group_inputs(s, 0, 1, "cuda")
    g = C.GpuCase(s, inp)
    gidx, gcnt = g.select(0)
    # tail keys of the size of the rebuilt keys, so that both parts carry weight
    rows = np.arange(64)
    K = O.sr_reconstruct(_cpu(inp.A_k[0]), _cpu(inp.B_k[0, 0][:, :s.d_h]), rows)
    tk, tv = synth.make_tail(s, 8192, key_rms=float(np.sqrt((K ** 2).mean())), value_rms=1.0, device="cuda")
    before = xkv.xkv_debug_launch_counts()
    gout, glse = g.attend_tail(gidx, gcnt, tk, tv, [8192])
    after = xkv.xkv_debug_launch_counts()
    assert after["tail_tc"] == before["tail_tc"] + 1 and after["tail_cuda"] == before["tail_cuda"]
    assert g.status() == (0, 0)
    sample = [(0, 0, 0), (1, 0, 6), (3, 0, 7)]
    A_k, A_v, q = _cpu(inp.A_k), _cpu(inp.A_v), _cpu(inp.q[0])
    shares = []
    for (l, b, hk) in sample:
        hd = slice(hk * s.d_h, (hk + 1) * s.d_h)
        hs = slice(hk * s.n_rep, (hk + 1) * s.n_rep)
        r = gidx[l, b, hk, :gcnt[l, b, hk]]
        K_hat = O.sr_reconstruct_keys(A_k[b], _cpu(inp.B_k[b, l][:, hd]), r, s.rope_base)
        V_hat = O.sr_reconstruct(A_v[b], _cpu(inp.B_v[b, l][:, hd]), r)
        o, lse = O.sr_attend_with_tail(q[l, b, hs], K_hat, V_hat, _cpu(tk[l, b, hk]), _cpu(tv[l, b, hk]),
                                       1.0 / np.sqrt(s.d_h))
        assert C.rel_err(gout[l, b, hs], o) <= TOL, (l, b, hk)
        np.testing.assert_allclose(glse[l, b, hs], lse, atol=2e-2)
        _, lse_sr = O.attend(q[l, b, hs], K_hat, V_hat, 1.0 / np.sqrt(s.d_h))
        shares.append(np.exp(lse_sr - lse))
    assert 0.01 < float(np.median(np.concatenate(shares))) < 0.99          # both parts matter
    g.close()


def test_config3_window_from_4bit_bases():
    """The headline window with the token bases as 4-bit round-to-nearest codes (App. "Integrate with
    Quantization"): sampled problems against the oracle on the dequantised bases."""
    from paper_2503_18893_b200 import xkv
    s = synth.config(3, n_groups=1)
    inp = workload.make_group_inputs(s, 0, 1, "cuda")
    g = C.GpuCase(s, inp)
    ck, mk = xkv.xkv_quantize_rtn(g.inp.A_k)
    cv, mv = xkv.xkv_quantize_rtn(g.inp.A_v)
    xkv.xkv_group_set_quantized_bases(g.grp, ck, mk, cv, mv)
    gidx, gcnt = g.select(0)
    gout, glse = g.attend(gidx, gcnt, 0)
    assert g.status() == (0, 0)
    deq = workload.GroupInputs(xkv.xkv_dequantize_rtn(ck, mk), xkv.xkv_dequantize_rtn(cv, mv), inp.B_k, inp.B_v,
                               inp.landmarks, inp.q)          # bit-equal to the oracle's dequantiser (tests/test_gpu_quant.py)
    cache = {}
    for (l, b, hk) in [(0, 0, 1), (2, 0, 6), (3, 0, 3)]:
        o, lse = _oracle_attend(s, deq, l, b, hk, gidx[l, b, hk, :gcnt[l, b, hk]], 0, cache)
        hs = slice(hk * s.n_rep, (hk + 1) * s.n_rep)
        assert C.rel_err(gout[l, b, hs], o) <= TOL, (l, b, hk)
        np.testing.assert_allclose(glse[l, b, hs], lse, atol=2e-2)
    g.close()
