"""Thin ctypes binding of libxkv (argument marshalling only; every step runs in the CUDA library).

The functions carry the names of the C ABI (include/xkv.h).  Tensors are torch CUDA tensors used
for their device memory; the stream is torch's current stream unless one is given.  Importing this
module loads libxkv.so from the package directory and raises if it has not been built: there is no
CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libxkv.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2503_18893_b200.build` "
        "(nvcc, sm_100a). There is no fallback path.")

_lib = ctypes.CDLL(LIB_PATH)

XKV_OK = 0
XKV_ERR_INVALID_ARG = -1
XKV_ERR_UNSUPPORTED = -2
XKV_ERR_ARCH = -3
XKV_ERR_CUDA = -4
XKV_ERR_OOM = -5
XKV_ERR_INDEX_RANGE = -6
XKV_ERR_TIMEOUT = -7
XKV_ERR_TOO_LARGE = -8
XKV_FLAG_INDEX_RANGE = 1
XKV_FLAG_TIMEOUT = 2


class xkv_group_config(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("G", ctypes.c_int32), ("batch", ctypes.c_int32), ("T", ctypes.c_int32),
        ("H_kv", ctypes.c_int32), ("H_q", ctypes.c_int32), ("d_h", ctypes.c_int32),
        ("r_k", ctypes.c_int32), ("r_v", ctypes.c_int32), ("chunk", ctypes.c_int32),
        ("k_max", ctypes.c_int32),
        ("rope_base", ctypes.c_float), ("softmax_scale", ctypes.c_float),
        ("A_k", ctypes.c_void_p), ("A_v", ctypes.c_void_p),
        ("B_k", ctypes.c_void_p), ("B_v", ctypes.c_void_p),
        ("landmarks", ctypes.c_void_p),
    ]


class xkv_select_static_config(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("G", ctypes.c_int32), ("batch", ctypes.c_int32), ("T", ctypes.c_int32),
        ("H_kv", ctypes.c_int32), ("H_q", ctypes.c_int32), ("d_h", ctypes.c_int32),
        ("chunk", ctypes.c_int32),
        ("landmarks", ctypes.c_void_p),
    ]


XKV_STATIC_SELECT_MAX_SCORES = 1 << 20
_P = ctypes.c_void_p
_lib.xkv_group_create.argtypes = [ctypes.POINTER(xkv_group_config), _P, ctypes.POINTER(_P)]
_lib.xkv_group_create.restype = ctypes.c_int
_lib.xkv_sr_select.argtypes = [_P, ctypes.c_int, ctypes.c_int, _P, ctypes.c_int32, _P, _P, _P]
_lib.xkv_sr_select.restype = ctypes.c_int
_lib.xkv_sr_reconstruct_attend.argtypes = [_P, ctypes.c_int, ctypes.c_int, _P, _P, _P, ctypes.c_int32, _P, _P, _P]
_lib.xkv_sr_reconstruct_attend.restype = ctypes.c_int
_lib.xkv_sr_select_static.argtypes = [ctypes.POINTER(xkv_select_static_config), ctypes.c_int, ctypes.c_int, _P,
                                      ctypes.c_int32, _P, _P, _P]
_lib.xkv_sr_select_static.restype = ctypes.c_int
_lib.xkv_tail_workspace_bytes.argtypes = [_P, ctypes.c_int32, ctypes.POINTER(ctypes.c_uint64)]
_lib.xkv_tail_workspace_bytes.restype = ctypes.c_int
_lib.xkv_sr_reconstruct_attend_tail.argtypes = [_P, ctypes.c_int, ctypes.c_int, _P, _P, _P, ctypes.c_int32, _P, _P, _P,
                                                ctypes.c_int32, _P, ctypes.c_uint64, _P, _P, _P]
_lib.xkv_sr_reconstruct_attend_tail.restype = ctypes.c_int


_lib.xkv_dense_workspace_bytes.argtypes = [_P, ctypes.c_int32, ctypes.POINTER(ctypes.c_uint64)]
_lib.xkv_dense_workspace_bytes.restype = ctypes.c_int
_lib.xkv_dense_attend.argtypes = [_P, ctypes.c_int, ctypes.c_int, _P, _P, _P, _P, ctypes.c_int32, _P, ctypes.c_uint64,
                                  _P, _P, _P]
_lib.xkv_dense_attend.restype = ctypes.c_int
_lib.xkv_quantize_rtn.argtypes = [_P, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, _P, _P, _P]
_lib.xkv_quantize_rtn.restype = ctypes.c_int
_lib.xkv_dequantize_rtn.argtypes = [_P, _P, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, _P, _P]
_lib.xkv_dequantize_rtn.restype = ctypes.c_int
_lib.xkv_group_set_quantized_bases.argtypes = [_P, _P, _P, _P, _P, ctypes.c_int32]
_lib.xkv_group_set_quantized_bases.restype = ctypes.c_int
XKV_DENSE_MAX_ROWS = 1 << 22
XKV_TAIL_MAX_ROWS = 32768


class xkv_landmark_config(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("G", ctypes.c_int32), ("batch", ctypes.c_int32),
                ("T", ctypes.c_int32), ("H_kv", ctypes.c_int32), ("d_h", ctypes.c_int32), ("chunk", ctypes.c_int32),
                ("rope_base", ctypes.c_float)]


_lib.xkv_build_landmarks.argtypes = [ctypes.POINTER(xkv_landmark_config), _P, _P, _P, ctypes.c_int32, _P, _P]
_lib.xkv_build_landmarks.restype = ctypes.c_int
_lib.xkv_group_set_outliers.argtypes = [_P, _P, ctypes.c_int32, _P]
_lib.xkv_group_set_outliers.restype = ctypes.c_int
_lib.xkv_group_destroy.argtypes = [_P]
_lib.xkv_group_destroy.restype = ctypes.c_int
_lib.xkv_group_status.argtypes = [_P, ctypes.POINTER(ctypes.c_uint32), _P]
_lib.xkv_group_status.restype = ctypes.c_int
_lib.xkv_group_bytes.argtypes = [ctypes.POINTER(xkv_group_config), ctypes.POINTER(ctypes.c_uint64),
                                 ctypes.POINTER(ctypes.c_uint64)]
_lib.xkv_group_bytes.restype = ctypes.c_int
_lib.xkv_group_workspace_bytes.argtypes = [_P, ctypes.POINTER(ctypes.c_uint64)]
_lib.xkv_group_workspace_bytes.restype = ctypes.c_int
_lib.xkv_strerror.argtypes = [ctypes.c_int]
_lib.xkv_strerror.restype = ctypes.c_char_p
_lib.xkv_last_cuda_error.restype = ctypes.c_int
_lib.xkv_kernel_launch_count.restype = ctypes.c_uint64
_lib.xkv_debug_launch_counts.argtypes = [ctypes.POINTER(ctypes.c_uint64)]
_lib.xkv_debug_launch_counts.restype = ctypes.c_int
_lib.xkv_debug_set_fault_injection.argtypes = [_P, ctypes.c_uint32]
_lib.xkv_debug_set_fault_injection.restype = ctypes.c_int

XKV_KERNEL_FAMILIES = ("scan", "topk", "fused", "merge", "tile", "tail_tc", "tail_cuda", "landmarks", "prep", "dense",
                       "clf", "merge_multi")
XKV_FLAG_CLF_BREAKDOWN = 4
XKV_INJECT_SCAN_NO_LOAD = 1
XKV_INJECT_FUSED_NO_B = 2
XKV_INJECT_CLF_BARRIER = 4
_lib.xkv_debug_set_clf_fault_injection.argtypes = [ctypes.c_uint32]
_lib.xkv_debug_set_clf_fault_injection.restype = ctypes.c_int


class XKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {xkv_strerror(status)} (status {status}, cuda error {xkv_last_cuda_error()})")


def xkv_strerror(status: int) -> str:
    return _lib.xkv_strerror(int(status)).decode()


def xkv_last_cuda_error() -> int:
    return int(_lib.xkv_last_cuda_error())


def xkv_kernel_launch_count() -> int:
    return int(_lib.xkv_kernel_launch_count())


def xkv_debug_launch_counts() -> dict:
    """Launches since load, by kernel family (names in XKV_KERNEL_FAMILIES)."""
    a = (ctypes.c_uint64 * len(XKV_KERNEL_FAMILIES))()
    st = _lib.xkv_debug_launch_counts(a)
    if st != XKV_OK:
        raise XKVError(st, "xkv_debug_launch_counts")
    return {n: int(a[i]) for i, n in enumerate(XKV_KERNEL_FAMILIES)}


def xkv_debug_set_clf_fault_injection(mask: int) -> None:
    st = _lib.xkv_debug_set_clf_fault_injection(mask)
    if st != XKV_OK:
        raise XKVError(st, "xkv_debug_set_clf_fault_injection")


def xkv_debug_set_fault_injection(grp, mask: int) -> None:
    st = _lib.xkv_debug_set_fault_injection(grp.handle, mask)
    if st != XKV_OK:
        raise XKVError(st, "xkv_debug_set_fault_injection")


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def make_config(*, G, batch, T, H_kv, H_q, d_h, r_k, r_v, k_max, chunk=8, rope_base=10000.0,
                softmax_scale=0.0, A_k=None, A_v=None, B_k=None, B_v=None, landmarks=None) -> xkv_group_config:
    """Fill an xkv_group_config; tensor arguments contribute their device addresses only."""
    cfg = xkv_group_config()
    cfg.struct_size = ctypes.sizeof(xkv_group_config)
    cfg.G, cfg.batch, cfg.T, cfg.H_kv, cfg.H_q, cfg.d_h = G, batch, T, H_kv, H_q, d_h
    cfg.r_k, cfg.r_v, cfg.chunk, cfg.k_max = r_k, r_v, chunk, k_max
    cfg.rope_base, cfg.softmax_scale = rope_base, softmax_scale
    cfg.A_k, cfg.A_v, cfg.B_k, cfg.B_v, cfg.landmarks = _ptr(A_k), _ptr(A_v), _ptr(B_k), _ptr(B_v), _ptr(landmarks)
    return cfg


def xkv_group_bytes(cfg: xkv_group_config):
    """(factor_bytes, landmark_bytes) of one window; host only."""
    f, l = ctypes.c_uint64(), ctypes.c_uint64()
    st = _lib.xkv_group_bytes(ctypes.byref(cfg), ctypes.byref(f), ctypes.byref(l))
    if st != XKV_OK:
        raise XKVError(st, "xkv_group_bytes")
    return f.value, l.value


class Group:
    """Owner of one xkv_group handle.  Keeps the borrowed tensors alive."""

    def __init__(self, handle: int, cfg: xkv_group_config, keep):
        self.handle, self.cfg, self._keep = handle, cfg, keep

    @property
    def k_cap_max(self) -> int:
        c = self.cfg.chunk or 8
        return -(-self.cfg.k_max // c) * c

    def __del__(self):
        try:
            xkv_group_destroy(self)
        except Exception:
            pass


def xkv_group_create(cfg: xkv_group_config, stream=None, keep=None) -> Group:
    h = _P()
    st = _lib.xkv_group_create(ctypes.byref(cfg), _stream(stream), ctypes.byref(h))
    if st != XKV_OK:
        raise XKVError(st, "xkv_group_create")
    return Group(h.value, cfg, keep)


def xkv_group_destroy(grp: Group) -> None:
    if grp.handle:
        h, grp.handle = grp.handle, 0
        st = _lib.xkv_group_destroy(h)
        if st != XKV_OK:
            raise XKVError(st, "xkv_group_destroy")


def xkv_sr_select(grp: Group, layer_begin: int, layer_end: int, q, k: int, sel_idx, sel_cnt, stream=None) -> None:
    st = _lib.xkv_sr_select(grp.handle, layer_begin, layer_end, _ptr(q), k, _ptr(sel_idx), _ptr(sel_cnt),
                            _stream(stream))
    if st != XKV_OK:
        raise XKVError(st, "xkv_sr_select")


def xkv_sr_select_static(*, G, batch, T, H_kv, H_q, d_h, landmarks, layer_begin, layer_end, q, k, sel_idx, sel_cnt,
                         chunk=8, stream=None) -> None:
    """Selection without a handle and without any device allocation (fixed scratch inside the library, see
    include/xkv.h).  Same outputs as xkv_sr_select.  Raises XKVError(XKV_ERR_TOO_LARGE) beyond the fixed size."""
    cfg = xkv_select_static_config()
    cfg.struct_size = ctypes.sizeof(xkv_select_static_config)
    cfg.G, cfg.batch, cfg.T, cfg.H_kv, cfg.H_q, cfg.d_h, cfg.chunk = G, batch, T, H_kv, H_q, d_h, chunk
    cfg.landmarks = _ptr(landmarks)
    st = _lib.xkv_sr_select_static(ctypes.byref(cfg), layer_begin, layer_end, _ptr(q), k, _ptr(sel_idx), _ptr(sel_cnt),
                                   _stream(stream))
    if st != XKV_OK:
        raise XKVError(st, "xkv_sr_select_static")


def xkv_sr_reconstruct_attend(grp: Group, layer_begin: int, layer_end: int, q, sel_idx, sel_cnt, k_cap: int,
                              out, lse=None, stream=None) -> None:
    st = _lib.xkv_sr_reconstruct_attend(grp.handle, layer_begin, layer_end, _ptr(q), _ptr(sel_idx), _ptr(sel_cnt),
                                        k_cap, _ptr(out), _ptr(lse), _stream(stream))
    if st != XKV_OK:
        raise XKVError(st, "xkv_sr_reconstruct_attend")


def xkv_build_landmarks(keys, landmarks, *, G, batch, T, H_kv, d_h, chunk=8, rope_base=10000.0, min_cos=None,
                        n_outliers=0, outliers=None, stream=None) -> None:
    """Algorithm 1 on device tensors in the layouts of include/xkv.h."""
    cfg = xkv_landmark_config(ctypes.sizeof(xkv_landmark_config), G, batch, T, H_kv, d_h, chunk, rope_base)
    st = _lib.xkv_build_landmarks(ctypes.byref(cfg), _ptr(keys), _ptr(landmarks), _ptr(min_cos), n_outliers,
                                  _ptr(outliers), _stream(stream))
    if st != XKV_OK:
        raise XKVError(st, "xkv_build_landmarks")


def xkv_group_set_outliers(grp: Group, outliers, n_outliers: int, stream=None) -> None:
    """`outliers`: int32 device tensor [G][batch][H_kv][n_outliers]; the caller keeps it alive."""
    st = _lib.xkv_group_set_outliers(grp.handle, _ptr(outliers), n_outliers, _stream(stream))
    if st != XKV_OK:
        raise XKVError(st, "xkv_group_set_outliers")
    grp.outliers = outliers     # keep the borrowed tensor alive with the handle


def xkv_tail_workspace_bytes(grp: Group, tail_cap: int) -> int:
    b = ctypes.c_uint64()
    st = _lib.xkv_tail_workspace_bytes(grp.handle, tail_cap, ctypes.byref(b))
    if st != XKV_OK:
        raise XKVError(st, "xkv_tail_workspace_bytes")
    return b.value


def xkv_sr_reconstruct_attend_tail(grp: Group, layer_begin: int, layer_end: int, q, sel_idx, sel_cnt, k_cap: int,
                                   tail_k, tail_v, tail_len, tail_cap: int, workspace, out, lse=None,
                                   stream=None) -> None:
    """`workspace`: a device tensor of at least xkv_tail_workspace_bytes(grp, tail_cap) bytes."""
    st = _lib.xkv_sr_reconstruct_attend_tail(grp.handle, layer_begin, layer_end, _ptr(q), _ptr(sel_idx), _ptr(sel_cnt),
                                             k_cap, _ptr(tail_k), _ptr(tail_v), _ptr(tail_len), tail_cap,
                                             _ptr(workspace), workspace.numel() * workspace.element_size(),
                                             _ptr(out), _ptr(lse), _stream(stream))
    if st != XKV_OK:
        raise XKVError(st, "xkv_sr_reconstruct_attend_tail")


def xkv_quantize_rtn(x, bits: int = 4, stream=None):
    """RTN-quantise a bf16 device tensor [..., cols] along its last axis in groups of 32 (include/xkv.h).
    Returns (codes uint8 [..., cols/2], meta int32 [..., cols/32] or None for 3 bits) device tensors."""
    cols = x.shape[-1]
    rows = x.numel() // cols
    codes = torch.empty(x.shape[:-1] + (cols // 2,), dtype=torch.uint8, device=x.device)
    # 4 bits: one scale/offset word per group beside the codes; 3 bits: the 16-byte records hold them (meta is None)
    meta = torch.empty(x.shape[:-1] + (cols // 32,), dtype=torch.int32, device=x.device) if bits == 4 else None
    st = _lib.xkv_quantize_rtn(_ptr(x), rows, cols, bits, _ptr(codes), _ptr(meta), _stream(stream))
    if st != XKV_OK:
        raise XKVError(st, "xkv_quantize_rtn")
    return codes, meta


def xkv_dequantize_rtn(codes, meta, bits: int = 4, stream=None):
    """bf16 tensor [..., cols] of the dequantised values x_hat."""
    cols = codes.shape[-1] * 2
    rows = codes.numel() // (cols // 2)
    x = torch.empty(codes.shape[:-1] + (cols,), dtype=torch.bfloat16, device=codes.device)
    st = _lib.xkv_dequantize_rtn(_ptr(codes), _ptr(meta), rows, cols, bits, _ptr(x), _stream(stream))
    if st != XKV_OK:
        raise XKVError(st, "xkv_dequantize_rtn")
    return x


def xkv_group_set_quantized_bases(grp: Group, codes_k, meta_k, codes_v, meta_v, bits: int = 4) -> None:
    st = _lib.xkv_group_set_quantized_bases(grp.handle, _ptr(codes_k), _ptr(meta_k), _ptr(codes_v), _ptr(meta_v), bits)
    if st != XKV_OK:
        raise XKVError(st, "xkv_group_set_quantized_bases")
    grp.quantized = (codes_k, meta_k, codes_v, meta_v)      # keep the borrowed tensors alive with the handle


class xkv_clf_config(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("T", ctypes.c_int32), ("G", ctypes.c_int32), ("d", ctypes.c_int32),
                ("r", ctypes.c_int32), ("oversample", ctypes.c_int32), ("power_iters", ctypes.c_int32)]


_lib.xkv_clf_rank_l.argtypes = [ctypes.POINTER(xkv_clf_config), ctypes.POINTER(ctypes.c_int32)]
_lib.xkv_clf_rank_l.restype = ctypes.c_int
_lib.xkv_clf_workspace_bytes.argtypes = [ctypes.POINTER(xkv_clf_config), ctypes.POINTER(ctypes.c_uint64)]
_lib.xkv_clf_workspace_bytes.restype = ctypes.c_int
_lib.xkv_clf_factorize.argtypes = [ctypes.POINTER(xkv_clf_config), _P, _P, _P, ctypes.c_uint64, _P, _P, _P, _P]
_lib.xkv_clf_factorize.restype = ctypes.c_int
_lib.xkv_clf_status.argtypes = [_P, ctypes.POINTER(ctypes.c_uint32), _P]
_lib.xkv_clf_status.restype = ctypes.c_int
_lib.xkv_debug_gemm.argtypes = [_P, _P, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, _P, _P, _P]
_lib.xkv_debug_gemm.restype = ctypes.c_int


def make_clf_config(*, T, G, d, r, oversample=0, power_iters=2) -> xkv_clf_config:
    return xkv_clf_config(ctypes.sizeof(xkv_clf_config), T, G, d, r, oversample, power_iters)


def xkv_clf_rank_l(cfg: xkv_clf_config) -> int:
    l = ctypes.c_int32()
    st = _lib.xkv_clf_rank_l(ctypes.byref(cfg), ctypes.byref(l))
    if st != XKV_OK:
        raise XKVError(st, "xkv_clf_rank_l")
    return l.value


def xkv_clf_workspace_bytes(cfg: xkv_clf_config) -> int:
    b = ctypes.c_uint64()
    st = _lib.xkv_clf_workspace_bytes(ctypes.byref(cfg), ctypes.byref(b))
    if st != XKV_OK:
        raise XKVError(st, "xkv_clf_workspace_bytes")
    return b.value


def xkv_clf_factorize(cfg: xkv_clf_config, X, omega, workspace, A, B, sigma=None, stream=None) -> None:
    """Cross-layer factorisation of X bf16 [T][G*d] (include/xkv.h); A bf16 [T][r], B bf16 [G][r][d], sigma fp32 [r]."""
    st = _lib.xkv_clf_factorize(ctypes.byref(cfg), _ptr(X), _ptr(omega), _ptr(workspace),
                                workspace.numel() * workspace.element_size(), _ptr(A), _ptr(B), _ptr(sigma),
                                _stream(stream))
    if st != XKV_OK:
        raise XKVError(st, "xkv_clf_factorize")


def xkv_clf_status(workspace, stream=None):
    f = ctypes.c_uint32()
    st = _lib.xkv_clf_status(_ptr(workspace), ctypes.byref(f), _stream(stream))
    return st, f.value


def xkv_debug_gemm(a, b, C, flags, stream=None) -> None:
    """C (M x N, fp32) = A B^T for a bf16 [K][M] and b bf16 [N][K] on the tensor core (diagnostic)."""
    K, M = a.shape
    N = b.shape[0]
    st = _lib.xkv_debug_gemm(_ptr(a), _ptr(b), M, N, K, _ptr(C), _ptr(flags), _stream(stream))
    if st != XKV_OK:
        raise XKVError(st, "xkv_debug_gemm")


def xkv_dense_workspace_bytes(grp: Group, cap: int) -> int:
    b = ctypes.c_uint64()
    st = _lib.xkv_dense_workspace_bytes(grp.handle, cap, ctypes.byref(b))
    if st != XKV_OK:
        raise XKVError(st, "xkv_dense_workspace_bytes")
    return b.value


def xkv_dense_attend(grp: Group, layer_begin: int, layer_end: int, q, K, V, length, cap: int, workspace, out, lse=None,
                     stream=None) -> None:
    """Plain decode attention over an uncompressed cache K, V [G][batch][H_kv][cap][d_h] (the dense baseline)."""
    st = _lib.xkv_dense_attend(grp.handle, layer_begin, layer_end, _ptr(q), _ptr(K), _ptr(V), _ptr(length), cap,
                               _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(out), _ptr(lse),
                               _stream(stream))
    if st != XKV_OK:
        raise XKVError(st, "xkv_dense_attend")


def xkv_group_status(grp: Group, stream=None):
    """(status, flags): reads and clears the device flag word (blocks on the stream)."""
    f = ctypes.c_uint32()
    st = _lib.xkv_group_status(grp.handle, ctypes.byref(f), _stream(stream))
    return st, f.value


def xkv_group_workspace_bytes(grp: Group) -> int:
    b = ctypes.c_uint64()
    st = _lib.xkv_group_workspace_bytes(grp.handle, ctypes.byref(b))
    if st != XKV_OK:
        raise XKVError(st, "xkv_group_workspace_bytes")
    return b.value


def create_from_tensors(A_k, A_v, B_k, B_v, landmarks, *, H_kv, H_q, k_max, chunk=8, rope_base=10000.0,
                        softmax_scale=0.0, stream=None) -> Group:
    """Convenience: read the sizes off the tensors (layouts of xkv_group_config) and create the handle."""
    batch, T, r_k = A_k.shape
    r_v = A_v.shape[2]
    G = B_k.shape[1]
    d_h = B_k.shape[3] // H_kv
    for t in (A_k, A_v, B_k, B_v, landmarks):
        if t is not None:
            assert t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16
    cfg = make_config(G=G, batch=batch, T=T, H_kv=H_kv, H_q=H_q, d_h=d_h, r_k=r_k, r_v=r_v, k_max=k_max,
                      chunk=chunk, rope_base=rope_base, softmax_scale=softmax_scale, A_k=A_k, A_v=A_v,
                      B_k=B_k, B_v=B_v, landmarks=landmarks)
    return xkv_group_create(cfg, stream, keep=(A_k, A_v, landmarks))
