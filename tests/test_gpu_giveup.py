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
