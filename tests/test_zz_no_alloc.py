"""xkv_sr_select_static: chunk selection for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not allowed: a serving process whose memory pool owns the
whole device, an allocator that forbids side allocations, a sandbox that only hands out fixed buffers.  They
cannot create a handle (creation allocates scratch), so the library offers one entry point whose scratch -- the
pooled landmark scores -- sits in a fixed array inside the library image.  This file checks, through the C ABI,
that it returns exactly what the handle-based xkv_sr_select returns, twice in a row on the shared scratch
(the second call with another budget and other queries, so that leftovers of the first call would show), and
that it refuses problems that do not fit.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2503_18893_b200 import synth
from tests import _cases as C

pytestmark = pytest.mark.gpu


def _static_select(xkv, s, lm, q, k, layers=None, bufs=None):
    k_cap = -(-k // s.c) * s.c
    if bufs is None:
        bufs = (torch.empty((s.G, s.batch, s.H_kv, k_cap), dtype=torch.int32, device="cuda"),
                torch.empty((s.G, s.batch, s.H_kv), dtype=torch.int32, device="cuda"))
    idx, cnt = bufs
    idx.fill_(-7)
    cnt.fill_(-7)
    l0, l1 = layers or (0, s.G)
    xkv.xkv_sr_select_static(G=s.G, batch=s.batch, T=s.T, H_kv=s.H_kv, H_q=s.H_q, d_h=s.d_h, landmarks=lm,
                             layer_begin=l0, layer_end=l1, q=q, k=k, sel_idx=idx, sel_cnt=cnt, chunk=s.c)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), cnt.cpu().numpy()


def test_static_select_matches_handle_select_twice_in_a_row():
    s = synth.config(1, G=3, batch=2, T=5003, k=400, r_k=16, r_v=16)
    inp = C.case_from_factors(s, n_steps=2)
    g = C.GpuCase(s, inp, k_max=1024)
    xkv = g.xkv
    # first call: budget 400, queries of step 0
    ref_idx, ref_cnt = g.select(0, k=400)
    got_idx, got_cnt = _static_select(xkv, s, g.inp.landmarks, g.inp.q[0], 400)
    np.testing.assert_array_equal(got_cnt, ref_cnt)
    np.testing.assert_array_equal(got_idx, ref_idx)
    # second call on the same scratch: other queries, larger budget, a sub-range of layers
    ref_idx, ref_cnt = g.select(1, k=1000, layers=(1, 3))
    got_idx, got_cnt = _static_select(xkv, s, g.inp.landmarks, g.inp.q[1], 1000, layers=(1, 3))
    np.testing.assert_array_equal(got_cnt, ref_cnt)
    np.testing.assert_array_equal(got_idx, ref_idx)
    assert np.all(got_idx[0] == -7)                                  # layer 0 was not in the range
    # and against the oracle, so that a fault shared by both entry points would still show
    oidx, ocnt, _, _ = C.oracle_step(s, inp, 1, k=1000, problems=[(1, 0, 0), (2, 1, 1)])
    np.testing.assert_array_equal(got_idx[1, 0, 0], oidx[1, 0, 0])
    np.testing.assert_array_equal(got_idx[2, 1, 1], oidx[2, 1, 1])
    # the entry point itself allocates nothing: with the output buffers made beforehand and the kernels already
    # loaded by the calls above, free device memory is the same before and after two more calls
    bufs = (torch.empty((s.G, s.batch, s.H_kv, 400), dtype=torch.int32, device="cuda"),
            torch.empty((s.G, s.batch, s.H_kv), dtype=torch.int32, device="cuda"))
    _static_select(xkv, s, g.inp.landmarks, g.inp.q[0], 400, bufs=bufs)
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(2):
        _static_select(xkv, s, g.inp.landmarks, g.inp.q[0], 400, bufs=bufs)
    assert abs(free_before - torch.cuda.mem_get_info()[0]) <= (1 << 20)
    g.close()


def test_static_select_rejects_what_does_not_fit():
    from paper_2503_18893_b200 import xkv
    s = synth.config(1, G=4, batch=4, H_kv=8, H_q=8, T=131072 * 4)  # 4*4*8*65536 scores = 8 Mi > 1 Mi
    lm = torch.zeros(16, dtype=torch.bfloat16, device="cuda")        # never read: the call is refused first
    q = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(xkv.XKVError) as e:
        xkv.xkv_sr_select_static(G=s.G, batch=s.batch, T=s.T, H_kv=s.H_kv, H_q=s.H_q, d_h=s.d_h, landmarks=lm,
                                 layer_begin=0, layer_end=1, q=q, k=8, sel_idx=idx, sel_cnt=idx)
    assert e.value.status == xkv.XKV_ERR_TOO_LARGE
    assert "scratch" in str(e.value)
    with pytest.raises(xkv.XKVError) as e:                           # bad layer range
        xkv.xkv_sr_select_static(G=2, batch=1, T=64, H_kv=1, H_q=1, d_h=64, landmarks=lm, layer_begin=1, layer_end=1,
                                 q=q, k=8, sel_idx=idx, sel_cnt=idx)
    assert e.value.status == xkv.XKV_ERR_INVALID_ARG
