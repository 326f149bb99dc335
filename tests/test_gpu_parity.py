"""Parity of the CUDA library (through the C ABI) with the CPU oracle on the same seeded inputs.

Bar: selected indices and counts bit-exact; attention outputs within 2e-2 max relative error per
output vector (max_i |gpu_i - ref_i| / max_i |ref_i|), bf16 storage with fp32 accumulation.
"""
import math

import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2503_18893_b200 import synth
from tests import _cases as C

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _check_select(gidx, gcnt, oidx, ocnt):
    np.testing.assert_array_equal(gcnt, ocnt)
    np.testing.assert_array_equal(gidx, oidx)        # includes the -1 padding beyond sel_cnt


def test_config1_full_pipeline_from_oracle_clf():
    """Tiny case: raw caches -> oracle CLF -> oracle landmarks -> library vs oracle."""
    s = synth.config(1)
    inp, _ = C.case_from_clf(s)
    g = C.GpuCase(s, inp)
    for step in (0, 1):
        oidx, ocnt, oout, olse = C.oracle_step(s, inp, step)
        gidx, gcnt = g.select(step)
        _check_select(gidx, gcnt, oidx, ocnt)
        gout, glse = g.attend(gidx, gcnt, step)
        assert C.rel_err(gout, oout) <= TOL
        np.testing.assert_allclose(glse, olse, atol=2e-2)
    assert g.status() == (0, 0)
    g.close()


def test_config1_fixed_index_set_reconstruct_attend_alone():
    s = synth.config(1)
    inp, _ = C.case_from_clf(s)
    sel = synth.fixed_index_set(s, 256, 4242).numpy()            # unsorted, not chunk aligned
    cnt = np.full((s.G, 1, s.H_kv), 256, dtype=np.int32)
    _, _, oout, olse = C.oracle_step(s, inp, 0, sel_idx=sel, sel_cnt=cnt)
    g = C.GpuCase(s, inp)
    gout, glse = g.attend(sel, cnt, 0)
    assert C.rel_err(gout, oout) <= TOL
    np.testing.assert_allclose(glse, olse, atol=2e-2)
    # a group-wide shared set (the same rows for every layer and head) is just a special case
    sel2 = np.broadcast_to(sel[0:1, :, 0:1], sel.shape).copy()
    _, _, oout2, _ = C.oracle_step(s, inp, 0, sel_idx=sel2, sel_cnt=cnt)
    gout2, _ = g.attend(sel2, cnt, 0)
    assert C.rel_err(gout2, oout2) <= TOL
    g.close()


RAGGED = [
    # name,                         overrides
    ("T_not_multiple_of_c", dict(T=2043, k=250)),
    ("k_not_multiple_of_c", dict(T=1500, k=251)),
    ("k_ge_T_dense", dict(T=700, k=700)),
    ("k_gt_T", dict(T=333, k=1000)),
    ("n_rep_7_dh128", dict(H_kv=2, H_q=14, d_h=128, T=1111, k=130, r_k=72, r_v=40)),
    ("n_rep_1", dict(H_kv=4, H_q=4, d_h=64, T=900, k=64)),
    ("rank_not_multiple_of_64", dict(T=1024, k=128, r_k=104, r_v=8)),
    ("chunk_16_no_rope", dict(T=1000, k=100, c=16, rope_base=0.0)),
    ("tiny_T", dict(T=5, k=8)),
    ("batch_3_G_3", dict(G=3, batch=3, T=777, k=96, r_k=32, r_v=48)),
    ("one_chunk_budget", dict(T=4096, k=1)),
    ("tile_tail_multi_tile", dict(T=6000, k=1000, H_kv=1, H_q=16, d_h=128, r_k=136, r_v=200)),
]


@pytest.mark.parametrize("name,over", RAGGED, ids=[r[0] for r in RAGGED])
def test_ragged_shapes(name, over):
    s = synth.config(1, **over)
    inp = C.case_from_factors(s)
    oidx, ocnt, oout, olse = C.oracle_step(s, inp, 0)
    g = C.GpuCase(s, inp)
    gidx, gcnt = g.select(0)
    _check_select(gidx, gcnt, oidx, ocnt)
    gout, glse = g.attend(gidx, gcnt, 0)
    assert C.rel_err(gout, oout) <= TOL, name
    np.testing.assert_allclose(glse, olse, atol=2e-2)
    assert g.status() == (0, 0)
    g.close()


def test_selection_ties_and_signed_zero():
    """Duplicated landmarks and all-zero landmarks: the lowest chunk index wins, on both sides."""
    s = synth.config(1, T=4096, k=64)
    inp = C.case_from_factors(s)
    lm = inp.landmarks.clone()
    lm[:, :, :, 100:140] = lm[:, :, :, 7:8]          # 40 copies of chunk 7
    lm[:, 1, :, 200:300] = 0.0                        # a run of exact zeros in layer 1
    lm[:, 1, 0, 250] = -0.0
    inp.landmarks = lm
    oidx, ocnt, _, _ = C.oracle_step(s, inp, 0)
    g = C.GpuCase(s, inp)
    gidx, gcnt = g.select(0)
    _check_select(gidx, gcnt, oidx, ocnt)
    # all landmarks identical: every score ties, the first k_ch chunks are selected
    inp.landmarks = torch.ones_like(lm)
    g2 = C.GpuCase(s, inp)
    gidx, gcnt = g2.select(0)
    np.testing.assert_array_equal(gidx[0, 0, 0], np.arange(64))
    g.close(); g2.close()


def test_budget_nesting_and_layer_ranges():
    s = synth.config(1, G=3, T=3000)
    inp = C.case_from_factors(s)
    g = C.GpuCase(s, inp, k_max=1024)
    prev = None
    for k in (8, 200, 256, 1024):
        oidx, ocnt, _, _ = C.oracle_step(s, inp, 0, k=k)
        gidx, gcnt = g.select(0, k=k)
        _check_select(gidx, gcnt, oidx, ocnt)
        cur = set(gidx[0, 0, 0][:gcnt[0, 0, 0]].tolist())
        assert prev is None or prev <= cur
        prev = cur
    # a sub-range of layers writes only its own slots
    gidx, gcnt = g.select(0, k=256, layers=(1, 2))
    oidx, ocnt, oout, _ = C.oracle_step(s, inp, 0, k=256)
    np.testing.assert_array_equal(gidx[1], oidx[1])
    assert np.all(gidx[0] == -7) and np.all(gidx[2] == -7) and np.all(gcnt[[0, 2]] == -7)
    gout, _ = g.attend(oidx, ocnt, 0, layers=(1, 2))
    assert C.rel_err(gout[1], oout[1]) <= TOL and np.all(gout[[0, 2]] == 0)
    g.close()


def test_attend_edge_cases_empty_duplicates_and_bad_indices():
    s = synth.config(1, T=512, k=64)
    inp = C.case_from_factors(s)
    g = C.GpuCase(s, inp)
    k_cap = 64
    sel = np.zeros((s.G, 1, s.H_kv, k_cap), dtype=np.int32)
    cnt = np.zeros((s.G, 1, s.H_kv), dtype=np.int32)
    sel[0, 0, 0, :5] = [9, 9, 300, 9, 511]; cnt[0, 0, 0] = 5            # duplicates count as often as listed
    sel[0, 0, 1, :1] = [17]; cnt[0, 0, 1] = 1                            # one row: output = its V row
    cnt[1, 0, 0] = 0                                                     # empty: output 0, lse -inf
    sel[1, 0, 1, :4] = [3, 100000, -5, 4]; cnt[1, 0, 1] = 4              # out of range rows are skipped
    gout, glse = g.attend(sel, cnt, 0)
    st, flags = g.status()
    assert st == g.xkv.XKV_ERR_INDEX_RANGE and flags & g.xkv.XKV_FLAG_INDEX_RANGE
    assert g.status() == (0, 0)                                          # reading clears the flag
    sel_ok = sel.copy(); cnt_ok = cnt.copy()
    sel_ok[1, 0, 1, :2] = [3, 4]; cnt_ok[1, 0, 1] = 2
    _, _, oout, olse = C.oracle_step(s, inp, 0, sel_idx=sel_ok, sel_cnt=cnt_ok)
    assert C.rel_err(gout, oout) <= TOL
    n = s.n_rep
    assert np.all(gout[1, 0, 0:n] == 0) and np.all(np.isneginf(glse[1, 0, 0:n]))
    np.testing.assert_allclose(np.delete(glse, np.s_[0:n], axis=2)[1:], np.delete(olse, np.s_[0:n], axis=2)[1:], atol=2e-2)
    vrow = C.f32(inp.A_v)[0, 17] @ C.f32(inp.B_v)[0, 0][:, s.d_h:2 * s.d_h]
    np.testing.assert_allclose(gout[0, 0, n:2 * n], np.broadcast_to(vrow, (n, s.d_h)), rtol=2e-2, atol=2e-2)
    g.close()


def test_select_all_then_attend_equals_dense_attention_on_reconstructed_cache():
    s = synth.config(1, T=1024, k=1024)
    inp = C.case_from_factors(s)
    g = C.GpuCase(s, inp)
    gidx, gcnt = g.select(0)
    assert np.all(gcnt == 1024) and np.all(gidx[0, 0, 0] == np.arange(1024))
    gout, _ = g.attend(gidx, gcnt, 0)
    A_k, A_v, B_k, B_v, q = (C.f32(t) for t in (inp.A_k, inp.A_v, inp.B_k, inp.B_v, inp.q[0]))
    for l in range(s.G):
        for h in range(s.H_q):
            hk = h // s.n_rep
            K = O.rope_rotate(A_k[0] @ B_k[0, l][:, hk * s.d_h:(hk + 1) * s.d_h], np.arange(1024), s.rope_base)
            V = A_v[0] @ B_v[0, l][:, hk * s.d_h:(hk + 1) * s.d_h]
            ref = O.dense_attend(q[l, 0, h:h + 1], K, V, 1 / math.sqrt(s.d_h))
            assert C.rel_err(gout[l, 0, h:h + 1], ref) <= TOL
    g.close()


@pytest.mark.parametrize("cfg_id,over", [(2, dict(T=8192)), (4, dict(T=4096, batch=2))],
                         ids=["cfg2_shape_T8192", "cfg4_shape_T4096_b2"])
def test_model_shapes_reduced_context(cfg_id, over):
    """Llama- and Qwen-shaped windows at a context the oracle finishes in seconds (several tiles, n_rep 4 and 7)."""
    s = synth.config(cfg_id, **over)
    inp = C.case_from_factors(s)
    problems = [(l, b, g) for l in (0, s.G - 1) for b in range(s.batch) for g in (0, s.H_kv - 1)]
    oidx, ocnt, oout, olse = C.oracle_step(s, inp, 0, problems=problems)
    g = C.GpuCase(s, inp)
    gidx, gcnt = g.select(0)
    gout, glse = g.attend(gidx, gcnt, 0)
    for (l, b, hk) in problems:
        np.testing.assert_array_equal(gidx[l, b, hk], oidx[l, b, hk])
        assert gcnt[l, b, hk] == ocnt[l, b, hk]
        hs = slice(hk * s.n_rep, (hk + 1) * s.n_rep)
        assert C.rel_err(gout[l, b, hs], oout[l, b, hs]) <= TOL
        np.testing.assert_allclose(glse[l, b, hs], olse[l, b, hs], atol=2e-2)
    assert g.status() == (0, 0)
    g.close()


def test_small_ranks_and_many_tiles_do_not_stall():
    """One 64-column slab per phase and many tiles per CTA: exercises the ring hand-offs with almost no work
    per tile (a regression test for a stall that the bounded waits turned into a TIMEOUT flag)."""
    s = synth.config(1, T=20000, k=6000, H_kv=1, H_q=4, d_h=128, r_k=64, r_v=8)
    inp = C.case_from_factors(s)
    oidx, ocnt, oout, olse = C.oracle_step(s, inp, 0)
    g = C.GpuCase(s, inp)
    gidx, gcnt = g.select(0)
    _check_select(gidx, gcnt, oidx, ocnt)
    gout, glse = g.attend(gidx, gcnt, 0)
    assert g.status() == (0, 0)
    assert C.rel_err(gout, oout) <= TOL
    g.close()


@pytest.mark.parametrize("T", [140001, 300001])
def test_more_chunks_than_one_topk_superblock(T):
    """n_c = 17501: 32 keys per thread in the list-based top-k; n_c = 37501: the kernel that re-reads the pooled
    scores super-block by super-block."""
    s = synth.config(1, T=T, k=3000, r_k=8, r_v=8)
    inp = C.case_from_factors(s)
    oidx, ocnt, _, _ = C.oracle_step(s, inp, 0, problems=[(0, 0, 0), (1, 0, 1)])
    g = C.GpuCase(s, inp)
    gidx, gcnt = g.select(0)
    for (l, hk) in ((0, 0), (1, 1)):
        np.testing.assert_array_equal(gidx[l, 0, hk], oidx[l, 0, hk])
        assert gcnt[l, 0, hk] == ocnt[l, 0, hk]
    g.close()


def test_selection_with_static_outliers_union():
    """Algorithm 2 line 5: outlier chunks are united with the top-k (ascending, no repeats, variable count), then
    reconstruct+attend runs on the longer selections."""
    s = synth.config(1, T=2045, k=128, batch=2)                          # ragged last chunk
    inp = C.case_from_factors(s)
    n_out = 5
    rng = np.random.default_rng(7)
    outl = rng.integers(0, s.n_c, size=(s.G, s.batch, s.H_kv, n_out)).astype(np.int32)
    outl[0, 0, 0] = [3, 3, s.n_c - 1, -4, 10 ** 6]                       # repeats, the ragged last chunk, out of range
    g = C.GpuCase(s, inp)
    plain_idx, plain_cnt = g.select(0)
    outl[1, 1, 1, :2] = plain_idx[1, 1, 1, [0, 8]] // s.c                 # two outliers that the top-k already holds
    o_dev = torch.from_numpy(outl).cuda()
    g.xkv.xkv_group_set_outliers(g.grp, o_dev, n_out)
    k_cap = (-(-s.k // s.c) + n_out) * s.c
    idx = torch.full((s.G, s.batch, s.H_kv, k_cap), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((s.G, s.batch, s.H_kv), -7, dtype=torch.int32, device="cuda")
    g.xkv.xkv_sr_select(g.grp, 0, s.G, g.inp.q[0], s.k, idx, cnt)
    torch.cuda.synchronize()
    gidx, gcnt = idx.cpu().numpy(), cnt.cpu().numpy()
    oidx, ocnt, oout, olse = O.sr_decode_step(C.f32(inp.A_k), C.f32(inp.A_v), C.f32(inp.B_k), C.f32(inp.B_v),
                                              C.f32(inp.landmarks), C.f32(inp.q[0]), k=s.k, c=s.c, H_kv=s.H_kv,
                                              rope_base=s.rope_base, outliers=outl)
    np.testing.assert_array_equal(gidx, oidx)
    np.testing.assert_array_equal(gcnt, ocnt)
    assert gcnt.min() >= plain_cnt.min() and gcnt.max() > plain_cnt.max()
    gout, glse = g.attend(gidx, gcnt, 0)
    assert C.rel_err(gout, oout) <= TOL
    np.testing.assert_allclose(glse, olse, atol=2e-2)
    # switching the union off restores the plain selection
    g.xkv.xkv_group_set_outliers(g.grp, None, 0)
    again_idx, again_cnt = g.select(0)
    np.testing.assert_array_equal(again_idx, plain_idx)
    np.testing.assert_array_equal(again_cnt, plain_cnt)
    assert g.status() == (0, 0)
    g.close()


@pytest.mark.parametrize("n_c", [20000, 40000])
def test_outliers_with_more_chunks_than_one_superblock(n_c):
    s = synth.config(1, T=8 * n_c, k=256, H_kv=1, H_q=2, G=1, r_k=16, r_v=16)       # both multi-super-block top-k kernels
    inp = C.case_from_factors(s)
    n_out = 7
    outl = np.array([[[[0, 16383, 16384, n_c - 1, 5, 5, 12345]]]], dtype=np.int32)
    g = C.GpuCase(s, inp)
    o_dev = torch.from_numpy(outl).cuda()
    g.xkv.xkv_group_set_outliers(g.grp, o_dev, n_out)
    k_cap = (-(-s.k // s.c) + n_out) * s.c
    idx = torch.full((s.G, s.batch, s.H_kv, k_cap), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((s.G, s.batch, s.H_kv), -7, dtype=torch.int32, device="cuda")
    g.xkv.xkv_sr_select(g.grp, 0, s.G, g.inp.q[0], s.k, idx, cnt)
    torch.cuda.synchronize()
    rows = O.sr_select(C.f32(inp.q[0])[0, 0], C.f32(inp.landmarks)[0, 0, 0], s.k, s.c, s.T, outl[0, 0, 0])
    assert cnt.item() == len(rows)
    np.testing.assert_array_equal(idx.cpu().numpy()[0, 0, 0, :len(rows)], rows)
    assert g.status() == (0, 0)
    g.close()


def test_plain_tile_kernel_agrees_with_the_tensor_core_path(monkeypatch):
    """The CUDA-core implementation that forms V_hat literally (the fallback for shapes the tensor-core kernel does
    not cover) against the oracle and against the fused path on the same inputs."""
    s = synth.config(1, T=2048, k=256)
    inp = C.case_from_factors(s)
    oidx, ocnt, oout, olse = C.oracle_step(s, inp, 0)
    g = C.GpuCase(s, inp)
    fout, flse = g.attend(oidx, ocnt, 0)
    g.close()
    monkeypatch.setenv("XKV_ATTEND_IMPL", "tile")
    g2 = C.GpuCase(s, inp)
    tout, tlse = g2.attend(oidx, ocnt, 0)
    assert g2.status() == (0, 0)
    g2.close()
    assert C.rel_err(tout, oout) <= TOL
    np.testing.assert_allclose(tlse, olse, atol=2e-2)
    assert C.rel_err(tout, fout.astype(np.float64)) <= TOL
