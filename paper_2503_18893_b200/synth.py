"""Seeded synthetic inputs for the xKV selective-reconstruction path.

This module only draws numbers: a counter-based generator (splitmix64 finaliser
plus Box-Muller, written out in integer tensor ops so the stream does not depend
on the torch version) and the recipes that shape those numbers like long-context
KV caches (a token subspace shared by the layers of a window, decaying spectrum,
noise floor, a few heavy rows).  It contains none of the method's arithmetic:
no factorisation, no landmarks, no selection, no attention.  Both the CPU oracle
tests and the CUDA tests/benchmark take their inputs from here.
"""
from __future__ import annotations

import dataclasses
import math

import torch

_MASK64 = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB


def _s64(v: int) -> int:
    """Python int (mod 2^64) -> the signed value torch.int64 holds for the same bits."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _mix_py(z: int) -> int:
    z &= _MASK64
    z = ((z ^ (z >> 30)) * _M1) & _MASK64
    z = ((z ^ (z >> 27)) * _M2) & _MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, *ids: int) -> int:
    """Hash a master seed and a tuple of small integers (tensor id, group, ...) to a 64-bit key."""
    k = _mix_py(seed + _GOLD)
    for i in ids:
        k = _mix_py(k ^ _mix_py((int(i) + 1) * _GOLD))
    return k


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 bit patterns."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix_t(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def uniform_bits(key: int, start: int, n: int, device) -> torch.Tensor:
    """n 64-bit words: word i = mix(key + (start+i+1)*GOLD)  (int64 bit patterns)."""
    ctr = torch.arange(start + 1, start + n + 1, dtype=torch.int64, device=device)
    return _mix_t(ctr * _s64(_GOLD) + _s64(key))


def normal(key: int, shape, device="cpu", dtype=torch.float32, chunk: int = 1 << 24) -> torch.Tensor:
    """Standard normals, element i from counter words 2i and 2i+1 (Box-Muller, fp64)."""
    n = int(math.prod(shape))
    out = torch.empty(n, dtype=dtype, device=device)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        w = uniform_bits(key, 2 * s, 2 * m, device).view(m, 2)
        u1 = (_lsr(w[:, 0], 11).to(torch.float64) + 1.0) * (1.0 / 9007199254740992.0)
        u2 = _lsr(w[:, 1], 11).to(torch.float64) * (1.0 / 9007199254740992.0)
        out[s:s + m] = (torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2)).to(dtype)
    return out.view(*shape)


def uniform_int(key: int, n: int, high: int, device="cpu") -> torch.Tensor:
    """n integers in [0, high) (modulo bias is irrelevant at these sizes)."""
    w = _lsr(uniform_bits(key, 0, n, device), 1)
    return (w % high).to(torch.int64)


def distinct_rows(key: int, n: int, high: int) -> torch.Tensor:
    """n distinct integers in [0, high), in the order drawn (unsorted)."""
    assert n <= high
    seen, out, start = set(), [], 0
    while len(out) < n:
        w = _lsr(uniform_bits(key, start, 2 * n, "cpu"), 1) % high
        start += 2 * n
        for v in w.tolist():
            if v not in seen:
                seen.add(v)
                out.append(v)
                if len(out) == n:
                    break
    return torch.tensor(out, dtype=torch.int32)


# --------------------------------------------------------------------------
# Workload shapes (the benchmark configurations)
# --------------------------------------------------------------------------


@dataclasses.dataclass(frozen=True)
class SRShape:
    """One window-group workload.  Names follow the paper (T is its L, G its W)."""
    name: str
    G: int
    H_kv: int
    H_q: int
    d_h: int
    T: int
    r_k: int
    r_v: int
    k: int
    batch: int = 1
    c: int = 8
    n_groups: int = 1
    rho: int = 32            # rank of the token subspace shared by the G layers
    decay: float = 0.0       # spectrum s_i = (i+1)^-decay
    noise: float = 0.05      # noise std (absolute if noise_abs else relative to signal rms)
    noise_abs: bool = False
    heavy_frac: float = 0.0  # fraction of token rows carrying 10x norm
    rope_base: float = 10000.0
    seed: int = 1000

    @property
    def d(self) -> int:
        return self.H_kv * self.d_h

    @property
    def n_rep(self) -> int:
        return self.H_q // self.H_kv

    @property
    def n_c(self) -> int:
        return -(-self.T // self.c)

    @property
    def k_cap(self) -> int:
        return (-(-self.k // self.c)) * self.c


def config(i: int, **over) -> SRShape:
    """The five benchmark configurations (1-based), optionally overridden."""
    base = {
        1: dict(name="cfg1_tiny", G=2, H_kv=2, H_q=8, d_h=64, T=2048, r_k=64, r_v=64, k=256,
                rho=32, decay=0.0, noise=0.05, noise_abs=True, seed=1001),
        2: dict(name="cfg2_llama_group", G=4, H_kv=8, H_q=32, d_h=128, T=32768, r_k=512, r_v=512,
                k=2048, rho=256, decay=1.0, noise=0.01, seed=1002),
        3: dict(name="cfg3_llama_128k", G=4, H_kv=8, H_q=32, d_h=128, T=131072, r_k=512, r_v=512,
                k=4096, n_groups=8, rho=256, decay=1.0, noise=0.01, seed=1003),
        4: dict(name="cfg4_qwen_64k", G=4, H_kv=4, H_q=28, d_h=128, T=65536, r_k=256, r_v=256,
                k=2048, batch=8, n_groups=7, rho=128, decay=0.8, noise=0.02, heavy_frac=0.01,
                seed=1004),
        5: dict(name="cfg5_stress", G=4, H_kv=8, H_q=32, d_h=128, T=65536, r_k=512, r_v=512,
                k=4096, rho=256, decay=1.0, noise=0.01, seed=1005),
    }[i]
    base.update(over)
    return SRShape(**base)


# --------------------------------------------------------------------------
# Recipes
# --------------------------------------------------------------------------

_T_K, _T_V, _T_Q, _T_IDX, _T_TAIL_K, _T_TAIL_V = 1, 2, 3, 4, 5, 6


def make_kv(shape: SRShape, group: int = 0, seq: int = 0, device="cpu"):
    """Raw caches of one window and one sequence, before any factorisation.

    For keys (pre-RoPE) and values independently: X_l = Z diag(s) M_l + noise with
    Z (T x rho) shared by the G layers, M_l (rho x d) per layer with N(0, 1/rho)
    entries, the whole scaled to unit rms and rounded to bf16.
    Returns (K, V), each a bf16 tensor (G, T, d).
    """
    out = []
    for which in (_T_K, _T_V):
        key = lambda *ids: stream_key(shape.seed, which, group, seq, *ids)
        Z = normal(key(0), (shape.T, shape.rho), device)
        s = torch.arange(1, shape.rho + 1, device=device, dtype=torch.float32) ** (-shape.decay)
        layers = []
        for l in range(shape.G):
            M = normal(key(1, l), (shape.rho, shape.d), device) / math.sqrt(shape.rho)
            sig = (Z * s) @ M
            srms = sig.pow(2).mean().sqrt()
            nstd = shape.noise if shape.noise_abs else shape.noise * srms
            layers.append(sig + nstd * normal(key(2, l), (shape.T, shape.d), device))
        X = torch.stack(layers)
        if shape.heavy_frac > 0:
            rows = uniform_int(stream_key(shape.seed, 9, group, seq), int(shape.heavy_frac * shape.T),
                               shape.T, device)
            X[:, rows, :] *= 10.0
        X = X / X.pow(2).mean().sqrt()
        out.append(X.to(torch.bfloat16))
    return out[0], out[1]


def make_factors(shape: SRShape, group: int = 0, device="cpu"):
    """Factors drawn directly in the form a cross-layer factorisation would return them.

    A = Z' diag(a): column i has std a_i, the spectrum of the recipe in `make_kv`
    (signal s_i over the first rho columns, a flat noise floor after) scaled so that
    A @ B has unit rms; B_cat (r x G*d) has orthonormal rows (QR of a Gaussian matrix).
    Returns bf16 tensors A_k (batch,T,r_k), A_v (batch,T,r_v), B_k (batch,G,r_k,d),
    B_v (batch,G,r_v,d).
    """
    res = {}
    for which, r in ((_T_K, shape.r_k), (_T_V, shape.r_v)):
        Gd = shape.G * shape.d
        i = torch.arange(r, device=device, dtype=torch.float32)
        sig = (i + 1.0) ** (-shape.decay)
        srms2 = float((sig[:min(shape.rho, r)] ** 2).sum()) / shape.rho
        floor = shape.noise if shape.noise_abs else shape.noise * math.sqrt(srms2)
        a = torch.where(i < shape.rho, sig * math.sqrt(Gd / shape.rho),
                        torch.full_like(sig, floor * (1.0 + math.sqrt(Gd / shape.T))))
        a = a * math.sqrt(Gd / float((a ** 2).sum()))
        A_all, B_all = [], []
        for b in range(shape.batch):
            key = lambda *ids: stream_key(shape.seed, 16 + which, group, b, *ids)
            A = normal(key(0), (shape.T, r), device) * a
            if shape.heavy_frac > 0:
                rows = uniform_int(stream_key(shape.seed, 9, group, b),
                                   int(shape.heavy_frac * shape.T), shape.T, device)
                A[rows, :] *= 10.0
            Q, _ = torch.linalg.qr(normal(key(1), (Gd, r), device).double())
            Bcat = Q.T.float().contiguous()                       # (r, G*d), orthonormal rows
            A_all.append(A.to(torch.bfloat16))
            B_all.append(Bcat.view(r, shape.G, shape.d).permute(1, 0, 2).contiguous().to(torch.bfloat16))
        res[which] = (torch.stack(A_all), torch.stack(B_all))
    return res[_T_K][0], res[_T_V][0], res[_T_K][1], res[_T_V][1]


def make_queries(shape: SRShape, n_steps: int = 1, group: int = 0, device="cpu") -> torch.Tensor:
    """Post-RoPE decode queries, N(0,1), bf16, shape (n_steps, G, batch, H_q, d_h)."""
    q = normal(stream_key(shape.seed, _T_Q, group), (n_steps, shape.G, shape.batch, shape.H_q, shape.d_h),
               device)
    return q.to(torch.bfloat16)


def make_tail(shape: SRShape, tail_cap: int, key_rms: float = 1.0, value_rms: float = 1.0, group: int = 0,
              device="cpu"):
    """Uncompressed K/V rows of the tokens generated so far (keys as the model stores them, already rotated):
    N(0, rms^2), bf16, shape (G, batch, H_kv, tail_cap, d_h) each.  The caller picks the scales so that the
    tail's logits are comparable with those of the reconstructed rows."""
    shp = (shape.G, shape.batch, shape.H_kv, tail_cap, shape.d_h)
    k = normal(stream_key(shape.seed, _T_TAIL_K, group), shp, device) * key_rms
    v = normal(stream_key(shape.seed, _T_TAIL_V, group), shp, device) * value_rms
    return k.to(torch.bfloat16), v.to(torch.bfloat16)


def fixed_index_set(shape: SRShape, n_rows: int = 256, seed: int = 4242) -> torch.Tensor:
    """Per (layer, sequence, KV head): n_rows distinct token rows, unsorted, not chunk aligned.

    Returns int32 (G, batch, H_kv, n_rows)."""
    out = torch.empty((shape.G, shape.batch, shape.H_kv, n_rows), dtype=torch.int32)
    for l in range(shape.G):
        for b in range(shape.batch):
            for g in range(shape.H_kv):
                out[l, b, g] = distinct_rows(stream_key(seed, _T_IDX, l, b, g), n_rows, shape.T)
    return out
