"""Shared helpers of the parity tests: build a case on the CPU, run the oracle, run the library."""
import math

import numpy as np
import torch

from oracle import xkv_oracle as O
from paper_2503_18893_b200 import synth, workload


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def case_from_clf(shape: synth.SRShape):
    """Generate raw caches, factorise them with the oracle (Eq. 1), build landmarks with the oracle
    (Alg. 1) from the ORIGINAL keys, round everything to bf16.  CPU tensors (bf16)."""
    assert shape.batch == 1
    K, V = synth.make_kv(shape)                                  # (G,T,d) bf16
    Kf, Vf = f32(K), f32(V)
    A_k, B_k, _ = O.clf_factorize([Kf[l] for l in range(shape.G)], shape.r_k)
    A_v, B_v, _ = O.clf_factorize([Vf[l] for l in range(shape.G)], shape.r_v)
    lm = np.stack([O.build_landmarks(Kf[l].reshape(shape.T, shape.H_kv, shape.d_h).transpose(1, 0, 2),
                                     shape.c, shape.rope_base) for l in range(shape.G)])[None]
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)
    inp = workload.GroupInputs(to(A_k[None]), to(A_v[None]), to(np.stack(B_k)[None]), to(np.stack(B_v)[None]),
                               to(lm), synth.make_queries(shape, 2))
    return inp, (K, V)


def case_from_factors(shape: synth.SRShape, n_steps=1, group=0):
    """Factors drawn directly (CPU), landmarks by the oracle's Algorithm 1 from the keys those factors stand for:
    K_l = bf16(A_k B_k[l]), the synthetic "original" pre-RoPE cache.  CPU tensors (bf16)."""
    A_k, A_v, B_k, B_v = synth.make_factors(shape, group, "cpu")
    lm = np.empty((shape.batch, shape.G, shape.H_kv, shape.n_c, shape.d_h), dtype=np.float32)
    for b in range(shape.batch):
        for l in range(shape.G):
            K = O.bf16_round(f32(A_k[b]) @ f32(B_k[b, l]))                       # (T, d)
            lm[b, l] = O.build_landmarks(K.reshape(shape.T, shape.H_kv, shape.d_h).transpose(1, 0, 2), shape.c,
                                         shape.rope_base)
    return workload.GroupInputs(A_k, A_v, B_k, B_v, torch.from_numpy(lm).to(torch.bfloat16),
                                synth.make_queries(shape, n_steps, group))


def oracle_step(shape, inp, step=0, sel_idx=None, sel_cnt=None, problems=None, k=None):
    return O.sr_decode_step(f32(inp.A_k), f32(inp.A_v), f32(inp.B_k), f32(inp.B_v), f32(inp.landmarks),
                            f32(inp.q[step]), k=shape.k if k is None else k, c=shape.c, H_kv=shape.H_kv,
                            rope_base=shape.rope_base, sel_idx=sel_idx, sel_cnt=sel_cnt, problems=problems)


def oracle_step_with_tail(shape, inp, sel_idx, sel_cnt, tail_k, tail_v, tail_len, step=0, problems=None):
    return O.sr_decode_step_with_tail(f32(inp.A_k), f32(inp.A_v), f32(inp.B_k), f32(inp.B_v), f32(inp.q[step]),
                                      sel_idx, sel_cnt, f32(tail_k), f32(tail_v), np.asarray(tail_len),
                                      H_kv=shape.H_kv, rope_base=shape.rope_base, problems=problems)


def rel_err(gpu: np.ndarray, ref: np.ndarray) -> float:
    """max_i |gpu_i - ref_i| / max_i |ref_i| over the last axis, worst vector."""
    num = np.abs(gpu.astype(np.float64) - ref).max(axis=-1)
    den = np.maximum(np.abs(ref).max(axis=-1), 1e-30)
    return float((num / den).max())


class GpuCase:
    """The library on cuda:0 for one window."""

    def __init__(self, shape, inp, k_max=None):
        from paper_2503_18893_b200 import xkv
        self.xkv, self.shape = xkv, shape
        d = "cuda"
        self.inp = workload.GroupInputs(*(t.to(d).contiguous() for t in
                                          (inp.A_k, inp.A_v, inp.B_k, inp.B_v, inp.landmarks, inp.q)))
        i = self.inp
        self.grp = xkv.create_from_tensors(i.A_k, i.A_v, i.B_k, i.B_v, i.landmarks, H_kv=shape.H_kv, H_q=shape.H_q,
                                           k_max=k_max or max(shape.k, 1), chunk=shape.c, rope_base=shape.rope_base)

    def select(self, step=0, k=None, layers=None):
        s = self.shape
        k = s.k if k is None else k
        k_cap = -(-k // s.c) * s.c
        idx = torch.full((s.G, s.batch, s.H_kv, k_cap), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((s.G, s.batch, s.H_kv), -7, dtype=torch.int32, device="cuda")
        l0, l1 = layers or (0, s.G)
        self.xkv.xkv_sr_select(self.grp, l0, l1, self.inp.q[step], k, idx, cnt)
        torch.cuda.synchronize()
        return idx.cpu().numpy(), cnt.cpu().numpy()

    def attend(self, sel_idx, sel_cnt, step=0, layers=None, want_lse=True):
        s = self.shape
        idx = torch.as_tensor(sel_idx, dtype=torch.int32).cuda().contiguous()
        cnt = torch.as_tensor(sel_cnt, dtype=torch.int32).cuda().contiguous()
        out = torch.zeros((s.G, s.batch, s.H_q, s.d_h), dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros((s.G, s.batch, s.H_q), dtype=torch.float32, device="cuda") if want_lse else None
        l0, l1 = layers or (0, s.G)
        self.xkv.xkv_sr_reconstruct_attend(self.grp, l0, l1, self.inp.q[step], idx, cnt, idx.shape[-1], out, lse)
        torch.cuda.synchronize()
        return f32(out), (lse.cpu().numpy() if want_lse else None)

    def attend_tail(self, sel_idx, sel_cnt, tail_k, tail_v, tail_len, step=0, layers=None):
        s = self.shape
        idx = torch.as_tensor(sel_idx, dtype=torch.int32).cuda().contiguous()
        cnt = torch.as_tensor(sel_cnt, dtype=torch.int32).cuda().contiguous()
        tk, tv = tail_k.cuda().contiguous(), tail_v.cuda().contiguous()
        tl = None if tail_len is None else torch.as_tensor(tail_len, dtype=torch.int32).cuda().contiguous()
        cap = tk.shape[3]
        ws = torch.empty(self.xkv.xkv_tail_workspace_bytes(self.grp, cap), dtype=torch.uint8, device="cuda")
        out = torch.zeros((s.G, s.batch, s.H_q, s.d_h), dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros((s.G, s.batch, s.H_q), dtype=torch.float32, device="cuda")
        l0, l1 = layers or (0, s.G)
        self.xkv.xkv_sr_reconstruct_attend_tail(self.grp, l0, l1, self.inp.q[step], idx, cnt, idx.shape[-1], tk, tv, tl,
                                                cap, ws, out, lse)
        torch.cuda.synchronize()
        return f32(out), lse.cpu().numpy()

    def status(self):
        return self.xkv.xkv_group_status(self.grp)

    def close(self):
        self.xkv.xkv_group_destroy(self.grp)
