"""The C-ABI library: it loads, exports every declared symbol, and its host-only logic behaves (no GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def xkv():
    from paper_2503_18893_b200 import build
    build.build()
    from paper_2503_18893_b200 import xkv as m
    return m


def test_exports_every_declared_symbol(xkv):
    hdr = open(os.path.join(ROOT, "include", "xkv.h")).read()
    names = re.findall(r"XKV_API\s+[\w\s\*]+?\b(xkv_\w+)\s*\(", hdr)
    assert set(names) >= {"xkv_group_create", "xkv_sr_select", "xkv_sr_reconstruct_attend", "xkv_group_destroy"}
    lib = ctypes.CDLL(xkv.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n


def test_config_struct_matches_header(xkv):
    # 13 four-byte fields followed by five pointers
    assert ctypes.sizeof(xkv.xkv_group_config) == 13 * 4 + 4 + 5 * 8


def test_group_bytes_matches_paper_accounting(xkv):
    from oracle import xkv_oracle as O
    # one window of Llama-3.1-8B at 64K: bytes = 2 * scalars of the appendix formulas with N = W = G
    cfg = xkv.make_config(G=4, batch=1, T=65536, H_kv=8, H_q=32, d_h=128, r_k=384, r_v=576, k_max=2048)
    f, l = xkv.xkv_group_bytes(cfg)
    assert f == 2 * O.factor_scalars(4, 4, 65536, 384, 576, 1024)
    assert l == 2 * O.landmark_scalars(4, 65536, 8, 1024)
    # 8 windows reproduce the printed 5.35x of xKV-SR
    full = 2 * 32 * 65536 * 1024 * 2
    assert abs(full / (8 * (f + l)) - 5.35) < 0.0075
    cfg3 = xkv.make_config(G=4, batch=3, T=1001, H_kv=2, H_q=4, d_h=64, r_k=16, r_v=24, k_max=8, chunk=16)
    f, l = xkv.xkv_group_bytes(cfg3)
    assert f == 3 * 2 * (1001 * 16 + 4 * 16 * 128 + 1001 * 24 + 4 * 24 * 128)
    assert l == 3 * 2 * 4 * 63 * 128


@pytest.mark.parametrize("field,value", [
    ("struct_size", 8), ("G", 0), ("batch", 0), ("T", 0), ("T", 1 << 24), ("H_q", 30), ("H_q", 8 * 17),
    ("d_h", 96), ("r_k", 12), ("r_v", 0), ("k_max", 0), ("chunk", -1), ("softmax_scale", -1.0)])
def test_invalid_config_is_rejected_on_the_host(xkv, field, value):
    cfg = xkv.make_config(G=4, batch=1, T=4096, H_kv=8, H_q=32, d_h=128, r_k=64, r_v=64, k_max=256)
    setattr(cfg, field, value)
    with pytest.raises(xkv.XKVError) as e:
        xkv.xkv_group_bytes(cfg)
    assert e.value.status == xkv.XKV_ERR_INVALID_ARG


def test_create_rejects_null_and_misaligned_pointers(xkv):
    cfg = xkv.make_config(G=4, batch=1, T=4096, H_kv=8, H_q=32, d_h=128, r_k=64, r_v=64, k_max=256)
    with pytest.raises(xkv.XKVError) as e:                       # all factor pointers NULL
        xkv.xkv_group_create(cfg, stream=0)
    assert e.value.status == xkv.XKV_ERR_INVALID_ARG
    cfg.B_k = cfg.B_v = 0x1000
    cfg.A_k = 0x1000                                             # one basis without the other
    with pytest.raises(xkv.XKVError) as e:
        xkv.xkv_group_create(cfg, stream=0)
    assert e.value.status == xkv.XKV_ERR_INVALID_ARG
    cfg.A_k = cfg.A_v = cfg.B_k = cfg.B_v = 0x1000
    cfg.A_v = 0x1008                                             # not 16-byte aligned
    with pytest.raises(xkv.XKVError) as e:
        xkv.xkv_group_create(cfg, stream=0)
    assert e.value.status == xkv.XKV_ERR_INVALID_ARG


def test_null_handle_calls_fail_cleanly(xkv):
    lib = ctypes.CDLL(xkv.LIB_PATH)
    assert lib.xkv_group_destroy(None) == xkv.XKV_OK
    lib.xkv_sr_select.restype = ctypes.c_int
    assert lib.xkv_sr_select(None, 0, 1, None, 8, None, None, None) == xkv.XKV_ERR_INVALID_ARG
    assert lib.xkv_sr_reconstruct_attend(None, 0, 1, None, None, None, 8, None, None, None) == xkv.XKV_ERR_INVALID_ARG
    assert xkv.xkv_strerror(xkv.XKV_ERR_TIMEOUT) and xkv.xkv_strerror(12345) == "unknown status"


def test_create_without_gpu_reports_cuda_error_not_a_crash(xkv):
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    cfg = xkv.make_config(G=1, batch=1, T=64, H_kv=1, H_q=1, d_h=64, r_k=8, r_v=8, k_max=8)
    cfg.A_k = cfg.A_v = cfg.B_k = cfg.B_v = 0x1000
    with pytest.raises(xkv.XKVError) as e:
        xkv.xkv_group_create(cfg, stream=0)
    assert e.value.status in (xkv.XKV_ERR_CUDA, xkv.XKV_ERR_ARCH)


def test_budgets_that_overflow_32_bit_strides_are_rejected_on_the_host(xkv):
    # a caller may pass a huge k to mean "every row": the row stride ceil(k/c)*c must not wrap
    cfg = xkv.make_config(G=4, batch=1, T=4096, H_kv=8, H_q=32, d_h=128, r_k=64, r_v=64, k_max=2**31 - 1)
    with pytest.raises(xkv.XKVError) as e:
        xkv.xkv_group_bytes(cfg)
    assert e.value.status == xkv.XKV_ERR_INVALID_ARG
    # the allocation-free entry point checks k before it touches the device (fake, aligned, never dereferenced pointers)
    sc = xkv.xkv_select_static_config()
    sc.struct_size = ctypes.sizeof(xkv.xkv_select_static_config)
    sc.G, sc.batch, sc.T, sc.H_kv, sc.H_q, sc.d_h, sc.chunk = 1, 1, 4096, 2, 8, 64, 8
    sc.landmarks = 0x10000
    st = xkv._lib.xkv_sr_select_static(ctypes.byref(sc), 0, 1, 0x20000, 2**31 - 1, 0x30000, 0x40000, None)
    assert st == xkv.XKV_ERR_INVALID_ARG
    # sizes whose landmark rows do not fit a 32-bit coordinate are refused, not wrapped
    big = xkv.make_config(G=64, batch=64, T=(1 << 24) - 1, H_kv=8, H_q=8, d_h=64, r_k=8, r_v=8, k_max=8)
    with pytest.raises(xkv.XKVError) as e:
        xkv.xkv_group_bytes(big)
    assert e.value.status == xkv.XKV_ERR_UNSUPPORTED


def test_launch_counters_by_family(xkv):
    c = xkv.xkv_debug_launch_counts()
    assert set(c) == set(xkv.XKV_KERNEL_FAMILIES) and sum(c.values()) == xkv.xkv_kernel_launch_count()


def test_quantisation_entry_points_check_their_arguments_on_the_host(xkv):
    L = xkv._lib
    assert L.xkv_quantize_rtn(0x1000, 4, 48, 4, 0x2000, 0x3000, None) == xkv.XKV_ERR_INVALID_ARG      # cols % 32
    assert L.xkv_quantize_rtn(0x1000, 4, 64, 5, 0x2000, 0x3000, None) == xkv.XKV_ERR_UNSUPPORTED      # no 5-bit format
    assert L.xkv_quantize_rtn(0x1000, 4, 64, 4, 0x2000, None, None) == xkv.XKV_ERR_INVALID_ARG        # 4 bits need meta
    assert L.xkv_quantize_rtn(0x1000, 4, 64, 9, 0x2000, 0x3000, None) == xkv.XKV_ERR_INVALID_ARG
    assert L.xkv_dequantize_rtn(0x1008, 0x2000, 4, 64, 4, 0x3000, None) == xkv.XKV_ERR_INVALID_ARG    # alignment
    assert L.xkv_group_set_quantized_bases(None, None, None, None, None, 4) == xkv.XKV_ERR_INVALID_ARG


def test_clf_config_is_checked_on_the_host(xkv):
    ok = xkv.make_clf_config(T=131072, G=4, d=1024, r=512)
    assert xkv.xkv_clf_rank_l(ok) == 576                      # r + 32 rounded up to a multiple of 64
    assert xkv.xkv_clf_workspace_bytes(ok) > 131072 * 576 * 2
    for bad in (dict(T=0), dict(r=12), dict(d=100, G=1), dict(r=8192), dict(power_iters=9)):
        kw = dict(T=4096, G=2, d=128, r=64)
        kw.update(bad)
        with pytest.raises(xkv.XKVError) as e:
            xkv.xkv_clf_workspace_bytes(xkv.make_clf_config(**kw))
        assert e.value.status == xkv.XKV_ERR_INVALID_ARG, bad
    with pytest.raises(xkv.XKVError) as e:                    # l beyond what the eigen-solver's tables hold
        xkv.xkv_clf_workspace_bytes(xkv.make_clf_config(T=4096, G=4, d=1024, r=2048, oversample=64))
    assert e.value.status == xkv.XKV_ERR_UNSUPPORTED
