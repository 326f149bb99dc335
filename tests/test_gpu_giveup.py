"""The give-up path: a wait inside a kernel that can never be satisfied runs into its limit, the kernel raises the
time-out flag and returns, xkv_group_status reports XKV_ERR_TIMEOUT, and the handle works again afterwards.
The failure is injected on the host (the loads that would satisfy the wait are simply not issued); nothing here
faults, traps or hangs the GPU."""
import numpy as np
import pytest

from paper_2503_18893_b200 import synth
from tests import _cases as C

pytestmark = pytest.mark.gpu


def _case():
    s = synth.config(1, T=1024, k=128)
    inp = C.case_from_factors(s)
    return s, inp, C.GpuCase(s, inp)


def test_landmark_scan_wait_runs_out_and_the_handle_recovers():
    s, inp, g = _case()
    x = g.xkv
    oidx, ocnt, oout, olse = C.oracle_step(s, inp, 0)
    x.xkv_debug_set_fault_injection(g.grp, x.XKV_INJECT_SCAN_NO_LOAD)
    gidx, gcnt = g.select(0)                                   # returns: every wait is bounded
    st, flags = g.status()
    assert st == x.XKV_ERR_TIMEOUT and flags & x.XKV_FLAG_TIMEOUT
    assert np.all(gidx < s.T) and np.all(gcnt <= s.k_cap)      # arbitrary, but in range
    assert g.status() == (0, 0)                                # reading the status cleared it
    x.xkv_debug_set_fault_injection(g.grp, 0)
    gidx, gcnt = g.select(0)
    np.testing.assert_array_equal(gidx, oidx)
    np.testing.assert_array_equal(gcnt, ocnt)
    assert g.status() == (0, 0)
    g.close()


def test_reconstruct_attend_wait_runs_out_and_the_handle_recovers():
    s, inp, g = _case()
    x = g.xkv
    oidx, ocnt, oout, olse = C.oracle_step(s, inp, 0)
    x.xkv_debug_set_fault_injection(g.grp, x.XKV_INJECT_FUSED_NO_B)
    g.attend(oidx, ocnt, 0)                                    # returns after the shortened limit; output unspecified
    st, flags = g.status()
    assert st == x.XKV_ERR_TIMEOUT and flags & x.XKV_FLAG_TIMEOUT
    x.xkv_debug_set_fault_injection(g.grp, 0)
    gout, glse = g.attend(oidx, ocnt, 0)
    assert g.status() == (0, 0)
    assert C.rel_err(gout, oout) <= 2e-2
    np.testing.assert_allclose(glse, olse, atol=2e-2)
    g.close()


def test_injection_mask_is_checked():
    s, inp, g = _case()
    with pytest.raises(g.xkv.XKVError) as e:
        g.xkv.xkv_debug_set_fault_injection(g.grp, 64)
    assert e.value.status == g.xkv.XKV_ERR_INVALID_ARG
    g.close()


def test_jacobi_grid_barrier_wait_runs_out_and_the_next_factorisation_is_fine():
    """One CTA of the cooperative Jacobi kernel skips its arrival at the first grid barrier: the others run into the
    (shortened) limit of their wait, raise the time-out flag and the abort word, and every CTA returns."""
    import torch
    from paper_2503_18893_b200 import xkv
    s = synth.config(1, T=2048)
    K, _ = synth.make_kv(s)
    X = torch.cat([K[l] for l in range(s.G)], dim=1).cuda().contiguous()          # (T, G d)
    r = 64
    cfg = xkv.make_clf_config(T=s.T, G=s.G, d=s.d, r=r, oversample=32, power_iters=1)
    l = xkv.xkv_clf_rank_l(cfg)
    omega = synth.normal(synth.stream_key(5, 31), (s.G * s.d, l)).to(torch.bfloat16).cuda()
    ws = torch.empty(xkv.xkv_clf_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    A = torch.empty((s.T, r), dtype=torch.bfloat16, device="cuda")
    B = torch.empty((s.G, r, s.d), dtype=torch.bfloat16, device="cuda")
    sig = torch.empty(r, dtype=torch.float32, device="cuda")
    xkv.xkv_debug_set_clf_fault_injection(xkv.XKV_INJECT_CLF_BARRIER)
    try:
        xkv.xkv_clf_factorize(cfg, X, omega, ws, A, B, sig)                        # returns: the barrier wait is bounded
        st, flags = xkv.xkv_clf_status(ws)
        assert st == xkv.XKV_ERR_TIMEOUT and flags & xkv.XKV_FLAG_TIMEOUT
    finally:
        xkv.xkv_debug_set_clf_fault_injection(0)
    xkv.xkv_clf_factorize(cfg, X, omega, ws, A, B, sig)
    assert xkv.xkv_clf_status(ws) == (0, 0)
    Xf = X.double()
    V = torch.cat([B[g] for g in range(s.G)], dim=1).double()                      # (r, G d)
    res = float(((Xf - A.double() @ V) ** 2).sum())
    sv = torch.linalg.svdvals(Xf)
    assert res <= 1.15 * float((sv[r:] ** 2).sum())
