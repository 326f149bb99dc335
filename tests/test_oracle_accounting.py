"""The oracle's memory/FLOP accounting against numbers the paper prints (App. C)."""
import os

import pytest

from oracle import xkv_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden", "compression_ratios.txt")


def _rows():
    with open(GOLD) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                p = line.split()
                yield p[0], int(p[1]), int(p[2]), float(p[3])


@pytest.mark.parametrize("kind,r_k,r_v,printed", list(_rows()))
def test_compression_ratio_matches_paper(kind, r_k, r_v, printed):
    # Llama-3.1-8B: N=32, d=1024, W=4; 64K context; c=8.  Printed with two decimals.
    ratios = O.compression_ratios(N=32, W=4, L=65536, d=1024, r_k=r_k, r_v=r_v, c=8)
    if kind.startswith("xkv_rtn"):
        # the table multiplies the printed (two-decimal) 8.03x of xKV: do the same
        got = O.quantized_compression_ratio(round(ratios["xkv"], 2), int(kind[len("xkv_rtn"):]))
    else:
        got = ratios[kind]
    assert abs(got - printed) < 0.0075, (kind, got, printed)


def test_factor_and_landmark_scalars_closed_form():
    # M_fact = (G L r_K + N r_K d) + (G L r_V + N r_V d);  M_lm = N ceil(L/c) d
    assert O.factor_scalars(8, 4, 100, 3, 5, 16) == (2 * 100 * 3 + 8 * 3 * 16) + (2 * 100 * 5 + 8 * 5 * 16)
    assert O.landmark_scalars(8, 101, 8, 16) == 8 * 13 * 16
    # ratio of full cache to factors+landmarks equals R_xKV-SR
    N, W, L, d, rk, rv, c = 32, 4, 65536, 1024, 384, 576, 8
    full = 2 * N * L * d
    r = full / (O.factor_scalars(N, W, L, rk, rv, d) + O.landmark_scalars(N, L, c, d))
    assert abs(r - O.compression_ratios(N, W, L, d, rk, rv, c)["xkv_sr"]) < 1e-9


def test_flops_formulas():
    # dense: L r_K d + L r_V d ; SR: sum_g M_g d_h (r_K + r_V); SR with M_g = L for all heads = dense
    L, rk, rv, H, dh = 1000, 48, 72, 4, 32
    assert O.flops_dense(L, rk, rv, H * dh) == L * rk * H * dh + L * rv * H * dh
    assert O.flops_sr([L] * H, dh, rk, rv) == O.flops_dense(L, rk, rv, H * dh)
    assert O.flops_sr([10, 20], dh, rk, rv) == 30 * dh * (rk + rv)
