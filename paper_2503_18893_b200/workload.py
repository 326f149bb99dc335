"""Synthetic long-context workloads for the benchmark and the full-size tests.

Everything here prepares INPUTS of the decode path: factors drawn by `synth.make_factors`, and chunk
landmarks of the keys those factors represent, computed by the library's own prefill entry point
(`xkv_build_landmarks`, App. B.1, Algorithm 1 lines 1-3).  None of the method's arithmetic is restated in
Python here; the decode step and the landmarks are only ever run through the C ABI (`xkv.py`).
"""
from __future__ import annotations

import dataclasses

import torch

from . import synth


def landmarks_from_factors(A_k: torch.Tensor, B_k: torch.Tensor, shape: synth.SRShape) -> torch.Tensor:
    """Landmarks of the keys the factors stand for, made by the library's own prefill step.

    The synthetic "original" pre-RoPE keys of layer l are K_l = bf16(A_k @ B_k[l]) (one library matmul per layer:
    this only manufactures an input); `xkv_build_landmarks` (Algorithm 1) then rotates them and takes the chunk
    means.  A_k (batch,T,r) bf16, B_k (batch,G,r,d) bf16 on a CUDA device  ->  bf16 (batch,G,H_kv,n_c,d_h).
    """
    from . import xkv
    if not A_k.is_cuda:
        raise RuntimeError("workload inputs are prepared with the CUDA library: pass device='cuda'")
    s = shape
    lm = torch.empty((s.batch, s.G, s.H_kv, s.n_c, s.d_h), dtype=torch.bfloat16, device=A_k.device)
    for b in range(s.batch):
        keys = torch.stack([A_k[b] @ B_k[b, l] for l in range(s.G)]).unsqueeze(0).contiguous()   # (1,G,T,d)
        xkv.xkv_build_landmarks(keys, lm[b:b + 1], G=s.G, batch=1, T=s.T, H_kv=s.H_kv, d_h=s.d_h, chunk=s.c,
                                rope_base=s.rope_base)
        torch.cuda.synchronize()
        del keys
    return lm


@dataclasses.dataclass
class GroupInputs:
    A_k: torch.Tensor
    A_v: torch.Tensor
    B_k: torch.Tensor
    B_v: torch.Tensor
    landmarks: torch.Tensor
    q: torch.Tensor          # (n_steps, G, batch, H_q, d_h)


def make_group_inputs(shape: synth.SRShape, group: int = 0, n_steps: int = 1, device="cuda") -> GroupInputs:
    """Factors, landmarks and queries of one window on a CUDA device, drawn directly (no factorisation is run)."""
    A_k, A_v, B_k, B_v = synth.make_factors(shape, group, device)
    lm = landmarks_from_factors(A_k, B_k, shape)
    q = synth.make_queries(shape, n_steps, group, device)
    return GroupInputs(A_k, A_v, B_k, B_v, lm, q)


def algorithmic_bytes(shape: synth.SRShape, unique_rows=None, quant_bits: int = 0) -> dict:
    """Bytes one window-step has to move (bf16 storage), per term.

    landmarks: every landmark is read once;  rows_issued: every selected row of A_k and A_v;
    rows_unique: the rows of the union over the (layer, head) problems of each sequence
    (pass the measured count; default = min(issued, T));  B: both reconstruction matrices.
    """
    problems = shape.G * shape.H_kv * shape.batch
    M = min(shape.k_cap, shape.T)
    lm = shape.batch * shape.G * shape.n_c * shape.d * 2
    # bytes per stored scalar of a basis row: 2 (bf16), or (b + 1)/8 with b-bit codes and their scale/offset words
    bps = 2.0 if not quant_bits else (quant_bits + 1) / 8.0
    issued = problems * M * (shape.r_k + shape.r_v) * bps
    if unique_rows is None:
        unique_rows = shape.batch * min(shape.G * shape.H_kv * M, shape.T)
    uniq = unique_rows * (shape.r_k + shape.r_v) * bps
    Bm = shape.batch * shape.G * (shape.r_k + shape.r_v) * shape.d * 2
    small = shape.G * shape.batch * shape.H_q * shape.d_h * 2 * 2 + problems * (M + 1) * 4 * 2
    return {"landmarks": lm, "rows_issued": issued, "rows_unique": uniq, "B": Bm, "small": small,
            "bytes_min": lm + uniq + Bm + small, "bytes_issued": lm + issued + Bm + small}


def algorithmic_flops(shape: synth.SRShape) -> float:
    """2 * sum over problems of M * d_h * (r_K + r_V)  (the paper's SR cost with the multiply-add factor)."""
    problems = shape.G * shape.H_kv * shape.batch
    M = min(shape.k_cap, shape.T)
    return 2.0 * problems * M * shape.d_h * (shape.r_k + shape.r_v)


def executed_flops(shape: synth.SRShape) -> float:
    """Flops the tensor-core path issues for one window-step: keys as in the paper's formula, values re-associated
    (sum_j p_j (A_v[S_j] B_v) = (sum_j p_j A_v[S_j]) B_v): 2 M r_V n_pad for the weighted basis rows (n_pad = the
    query heads of a KV head padded to the smallest MMA width, 16) plus 2 r_V d_h per query head for the projection."""
    problems = shape.G * shape.H_kv * shape.batch
    M = min(shape.k_cap, shape.T)
    return problems * (2.0 * M * shape.d_h * shape.r_k + 2.0 * M * shape.r_v * 16 + 2.0 * shape.r_v * shape.d_h * shape.n_rep)


class DeviceWorkload:
    """All windows of a configuration resident on one GPU, with their handles and output buffers."""

    def __init__(self, shape: synth.SRShape, n_steps: int = 4, device="cuda", groups=None, tail_rows: int = 0,
                 quant_bits: int = 0):
        from . import xkv  # loads the CUDA library; raises if it is not built
        self.xkv = xkv
        self.shape = shape
        self.device = device
        self.groups = []
        self.inputs = []
        ids = range(shape.n_groups) if groups is None else groups
        for gi in ids:
            inp = make_group_inputs(shape, gi, n_steps, device)
            grp = xkv.create_from_tensors(inp.A_k, inp.A_v, inp.B_k, inp.B_v, inp.landmarks, H_kv=shape.H_kv,
                                          H_q=shape.H_q, k_max=shape.k, chunk=shape.c, rope_base=shape.rope_base)
            if quant_bits:      # the token bases as b-bit codes (App. "Integrate with Quantization"), made by the library
                ck, mk = xkv.xkv_quantize_rtn(inp.A_k, quant_bits)
                cv, mv = xkv.xkv_quantize_rtn(inp.A_v, quant_bits)
                xkv.xkv_group_set_quantized_bases(grp, ck, mk, cv, mv, quant_bits)
            self.inputs.append(inp)
            self.groups.append(grp)
        n = len(self.groups)
        s = shape
        self.sel_idx = torch.empty((n, s.G, s.batch, s.H_kv, s.k_cap), dtype=torch.int32, device=device)
        self.sel_cnt = torch.empty((n, s.G, s.batch, s.H_kv), dtype=torch.int32, device=device)
        self.out = torch.empty((n, s.G, s.batch, s.H_q, s.d_h), dtype=torch.bfloat16, device=device)
        self.lse = torch.empty((n, s.G, s.batch, s.H_q), dtype=torch.float32, device=device)
        self.n_steps = n_steps
        # optional uncompressed tail of generated tokens (Sec. 4): every sequence has `tail_rows` of them
        self.tail_rows = tail_rows
        self.tail = []
        self.tail_ws = None
        if tail_rows > 0:
            for gi in ids:
                self.tail.append(synth.make_tail(s, tail_rows, group=gi, device=device))
            self.tail_ws = torch.empty(xkv.xkv_tail_workspace_bytes(self.groups[0], tail_rows), dtype=torch.uint8,
                                       device=device)

    def attend(self, gi: int, q) -> None:
        """Reconstruct+attend of window gi over the rows selected last, plus the tail if there is one."""
        s, x, grp = self.shape, self.xkv, self.groups[gi]
        if self.tail_rows > 0:
            tk, tv = self.tail[gi]
            x.xkv_sr_reconstruct_attend_tail(grp, 0, s.G, q, self.sel_idx[gi], self.sel_cnt[gi], s.k_cap, tk, tv, None,
                                             self.tail_rows, self.tail_ws, self.out[gi], self.lse[gi])
        else:
            x.xkv_sr_reconstruct_attend(grp, 0, s.G, q, self.sel_idx[gi], self.sel_cnt[gi], s.k_cap,
                                        self.out[gi], self.lse[gi])

    def step(self, i: int, q_override=None) -> None:
        """One decode step: every window, select then reconstruct+attend, on the current stream."""
        s, x = self.shape, self.xkv
        for gi, grp in enumerate(self.groups):
            q = self.inputs[gi].q[i % self.n_steps] if q_override is None else q_override[gi]
            x.xkv_sr_select(grp, 0, s.G, q, s.k, self.sel_idx[gi], self.sel_cnt[gi])
            self.attend(gi, q)

    def close(self):
        for g in self.groups:
            self.xkv.xkv_group_destroy(g)
        self.groups = []
