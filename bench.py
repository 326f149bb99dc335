#!/usr/bin/env python
"""Benchmark of the xKV selective-reconstruction decode step on B200.

    python bench.py --gpus N --steps K --warmup W            (ours; torchrun launches N>1)
    python bench.py --impl reference ...                      (the CPU oracle on a bounded sample)

One step = one decode step of the whole model-shaped workload: for every window of G layers,
xkv_sr_select then xkv_sr_reconstruct_attend.  The workload is Llama-3.1-8B-shaped: 8 windows of
G=4 layers, 8 KV heads x 128, 32 query heads, T=131072 context rows, r_K=r_V=512, budget k=4096,
batch 1, bf16, synthetic factors.  With N GPUs every rank serves its own sequence (windows and
sequences are independent units: weak scaling, no collective on the data path).

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "SR decode steps/sec per layer group at 128K ctx"
UNIT = "group-steps/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, help="workload id (3 = the headline 128K workload)")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--T", type=int, default=None)
    ap.add_argument("--k", type=int, default=None)
    ap.add_argument("--r", type=int, default=None)
    ap.add_argument("--r-k", type=int, default=None)
    ap.add_argument("--r-v", type=int, default=None)
    ap.add_argument("--rope-base", type=float, default=None)
    ap.add_argument("--groups", type=int, default=None, help="number of windows (default: the config's)")
    ap.add_argument("--tail", type=int, default=0,
                    help="rows of uncompressed generated tokens attended to besides the selected rows (default none)")
    ap.add_argument("--quant", type=int, default=0, choices=[0, 3, 4],
                    help="gather the token bases from b-bit round-to-nearest codes (0: bf16 bases, the headline)")
    ap.add_argument("--op", default="decode", choices=["decode", "landmarks", "clf"],
                    help="decode: the hot path (default).  landmarks: the prefill-side Algorithm 1 kernel alone "
                         "(not the headline metric; prints its own JSON line)")
    ap.add_argument("--repeats", type=int, default=0,
                    help="times the `steps`-step region is repeated (0: as many as make about a second of timed work)")
    ap.add_argument("--dense", action="store_true",
                    help="also time plain decode attention over an uncompressed bf16 cache of the same shape")
    ap.add_argument("--sweep", action="store_true",
                    help="run the other benchmark configurations and the corner points of the stress sweep, one JSON "
                         "line per point (each with the dense-attention arm and a parity check)")
    ap.add_argument("--sweep-out", default=None, help="with --sweep: also write a markdown table to this file")
    ap.add_argument("--sweep-filter", default=None, help="with --sweep: only the points whose label contains this text")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-problems", type=int, default=None, help="oracle sample size in (layer,head) problems")
    return ap.parse_args()


def make_shape(args):
    from paper_2503_18893_b200 import synth
    over = {}
    if args.batch is not None: over["batch"] = args.batch
    if args.T is not None: over["T"] = args.T
    if args.k is not None: over["k"] = args.k
    if args.r is not None: over["r_k"] = over["r_v"] = args.r
    if args.r_k is not None: over["r_k"] = args.r_k
    if args.r_v is not None: over["r_v"] = args.r_v
    if args.rope_base is not None: over["rope_base"] = args.rope_base
    if args.groups is not None: over["n_groups"] = args.groups
    return synth.config(args.config, **over)


def replica_units(n_windows: int, rank: int):
    """Ids of the synthetic windows that rank `rank` serves: every rank holds a full replica of the workload made of
    its own sequences (fixed work per GPU: weak scaling), so the ids of different ranks never overlap."""
    return list(range(rank * n_windows, (rank + 1) * n_windows))


def reduce_max(value: float, dist=None) -> float:
    """Max over ranks of a host scalar (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return value
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i", str(self.index),
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        rows = [r for (t, r) in self.rows if t0 - 0.05 <= t <= t1 + 0.15] or [r for (_, r) in self.rows]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def oracle_sample(shape, inp, n_problems, spread=False):
    """Time the CPU oracle (as it stands) on n_problems (layer, sequence, head) problems of a window: the first
    ones, or (spread) ones spread evenly over the window.  Returns (seconds, problems, cores, results) where cores is
    the CPU time the call used divided by its wall time (the oracle's scoring loop is serial numpy; only its
    BLAS calls use several threads) and results = (problem list, sel_idx, sel_cnt, out, lse) of the oracle."""
    import numpy as np
    from oracle import xkv_oracle as O
    f32 = lambda t: t.detach().float().cpu().numpy()
    allp = [(l, b, g) for l in range(shape.G) for b in range(shape.batch) for g in range(shape.H_kv)]
    n_problems = min(n_problems, len(allp))
    probs = [allp[(i * len(allp)) // n_problems] for i in range(n_problems)] if spread else allp[:n_problems]
    # only the sequences the sample touches are widened to fp32 on the host
    seqs = sorted({b for (_, b, _) in probs})
    pos = {b: i for i, b in enumerate(seqs)}
    A_k, A_v, B_k, B_v, lm = (f32(t[seqs]) for t in (inp.A_k, inp.A_v, inp.B_k, inp.B_v, inp.landmarks))
    q = f32(inp.q[0][:, seqs])
    sub = [(l, pos[b], g) for (l, b, g) in probs]
    c0, t0 = time.process_time(), time.perf_counter()
    res = O.sr_decode_step(A_k, A_v, B_k, B_v, lm, q, k=shape.k, c=shape.c, H_kv=shape.H_kv, rope_base=shape.rope_base,
                           problems=sub)
    dt, cpu = time.perf_counter() - t0, time.process_time() - c0
    # back to the full batch numbering
    full = []
    for a in res:
        z = np.zeros(a.shape[:1] + (shape.batch,) + a.shape[2:], dtype=a.dtype)
        z[:, seqs] = a
        full.append(z)
    return dt, len(probs), round(max(1.0, cpu / max(dt, 1e-9)), 1), (probs,) + tuple(full)


def parity_against(shape, oracle_results, gidx, gcnt, gout, glse):
    """Compare the library's results of one window-step with the oracle's on the problems the oracle evaluated:
    number of index-set mismatches, worst relative error per output vector, worst absolute LSE error."""
    import numpy as np
    probs, oidx, ocnt, oout, olse = oracle_results
    bad, err, lerr = 0, 0.0, 0.0
    for (l, b, g) in probs:
        if int(gcnt[l, b, g]) != int(ocnt[l, b, g]) or not np.array_equal(gidx[l, b, g], oidx[l, b, g]):
            bad += 1
        hs = slice(g * shape.n_rep, (g + 1) * shape.n_rep)
        num = np.abs(gout[l, b, hs].astype(np.float64) - oout[l, b, hs]).max(axis=-1)
        den = np.maximum(np.abs(oout[l, b, hs]).max(axis=-1), 1e-30)
        err = max(err, float((num / den).max()))
        lerr = max(lerr, float(np.abs(glse[l, b, hs] - olse[l, b, hs]).max()))
    return {"problems_checked": len(probs), "idx_mismatch": bad, "max_rel_err": err, "max_lse_abs_err": lerr,
            "tolerance": 2e-2}


def captured_traffic(kernel_file: str):
    """DRAM bytes per reconstruct_attend call from the ncu capture summarised under profiles/, if that capture was
    taken from the kernel source as it is now (the summary records the source file's hash); else None."""
    import glob
    import hashlib
    import re
    try:
        with open(os.path.join(ROOT, "paper_2503_18893_b200", "csrc", kernel_file), "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()[:16]
    except OSError:
        return None
    for path in glob.glob(os.path.join(ROOT, "profiles", "*.md")):
        for m in re.finditer(r"capture-of: (\S+) sha256=(\w+) attend_dram_bytes_per_launch=([0-9.e+]+)", open(path).read()):
            if m.group(1) == kernel_file and m.group(2) == digest:
                return float(m.group(3))
    return None


def reference_inputs(shape, n_problems):
    """Inputs of the reference arm, prepared on the host without the CUDA library: factors from the generator,
    landmarks by the oracle's Algorithm 1 from the keys the factors stand for -- only for the (layer, sequence,
    head) problems the sample covers (the others stay zero and are never read)."""
    import numpy as np
    import torch
    from oracle import xkv_oracle as O
    from paper_2503_18893_b200 import synth, workload
    f32 = lambda t: t.detach().float().cpu().numpy()
    A_k, A_v, B_k, B_v = synth.make_factors(shape, 0, "cpu")
    lm = np.zeros((shape.batch, shape.G, shape.H_kv, shape.n_c, shape.d_h), dtype=np.float32)
    allp = [(l, b, g) for l in range(shape.G) for b in range(shape.batch) for g in range(shape.H_kv)]
    for (l, b, g) in allp[:n_problems]:
        K = O.bf16_round(f32(A_k[b]) @ f32(B_k[b, l][:, g * shape.d_h:(g + 1) * shape.d_h]))      # (T, d_h)
        lm[b, l, g] = O.build_landmarks(K[None], shape.c, shape.rope_base)[0]
    return workload.GroupInputs(A_k, A_v, B_k, B_v, torch.from_numpy(lm).to(torch.bfloat16),
                                synth.make_queries(shape, 1, 0))


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores, a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    shape = make_shape(args)
    problems_per_group = shape.G * shape.batch * shape.H_kv
    n = args.cpu_problems or 2
    inp = reference_inputs(shape, n)
    times = []
    for i in range(args.warmup + args.steps):
        dt, np_, threads, _ = oracle_sample(shape, inp, n)
        if i >= args.warmup:
            times.append(dt)
    sec = sum(times)
    value = (args.steps * n / problems_per_group) / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sec / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(shape, 1),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"{n} of {problems_per_group} (layer,head) problems of one window per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


def workload_config(shape, n_gpus):
    return {"workload": f"{shape.name}: {shape.n_groups} windows x G={shape.G} layers, H_kv={shape.H_kv}x{shape.d_h}, "
                        f"H_q={shape.H_q}, T={shape.T}, r_K={shape.r_k}, r_V={shape.r_v}, k={shape.k}, c={shape.c}, "
                        f"batch={shape.batch} per GPU",
            "T": shape.T, "k": shape.k, "r_k": shape.r_k, "r_v": shape.r_v, "batch_per_gpu": shape.batch,
            "windows": shape.n_groups, "parallelism": f"replica x{n_gpus} (independent sequences)",
            "l2": "per-step inputs larger than L2 (windows visited round-robin; no operand survives in L2 "
                  "between steps)"}


def run_landmarks(args):
    """Times xkv_build_landmarks (Algorithm 1 with 48 outlier chunks per head) on one window of the workload's keys:
    the keys the factors represent, A_k @ B_k[l], formed with torch once outside the timed region."""
    import torch
    from paper_2503_18893_b200 import synth, xkv
    torch.cuda.set_device(0)
    s = make_shape(args)
    A_k, _, B_k, _ = synth.make_factors(s, 0, "cuda")
    keys = torch.stack([torch.stack([(A_k[b].float() @ B_k[b, l].float()).to(torch.bfloat16) for l in range(s.G)])
                        for b in range(s.batch)]).contiguous()                    # (batch, G, T, d)
    n_out = 48
    lm = torch.empty((s.batch, s.G, s.H_kv, s.n_c, s.d_h), dtype=torch.bfloat16, device="cuda")
    mc = torch.empty((s.G, s.batch, s.H_kv, s.n_c), dtype=torch.float32, device="cuda")
    outl = torch.empty((s.G, s.batch, s.H_kv, n_out), dtype=torch.int32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")              # larger than L2
    call = lambda mcos, n, o: xkv.xkv_build_landmarks(keys, lm, G=s.G, batch=s.batch, T=s.T, H_kv=s.H_kv, d_h=s.d_h,
                                                      chunk=s.c, rope_base=s.rope_base, min_cos=mcos, n_outliers=n,
                                                      outliers=o)
    res = {}
    for name, a in (("landmarks_only", (None, 0, None)), ("landmarks_min_cos_outliers", (mc, n_out, outl))):
        ts = []
        for i in range(args.warmup + args.steps):
            flush.zero_()
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(); call(*a); e1.record()
            torch.cuda.synchronize()
            if i >= args.warmup:
                ts.append(e0.elapsed_time(e1))
        res[name] = statistics.mean(ts)
    pk = peaks()
    key_bytes = keys.numel() * 2 + lm.numel() * 2
    print(json.dumps({"op": "xkv_build_landmarks", "config": workload_config(s, 1)["workload"] + " (one window)",
                      "key_bytes": key_bytes, "ms": res, "l2": "flushed between calls",
                      "achieved_gbs_landmarks_only": key_bytes / (res["landmarks_only"] * 1e-3) / 1e9,
                      "frac_of_hbm_peak": key_bytes / (res["landmarks_only"] * 1e-3) / 1e9 / pk["hbm_gbs"],
                      "peak_source": pk["source"]}))
    return 0


def run_clf(args):
    """Times xkv_clf_factorize (Eq. 1 by randomised SVD) on the raw key cache of one window and one sequence of the
    workload's shape, and compares its residual with the optimum (eigenvalues of the fp64 Gram matrix, by torch on
    the GPU: a harness cross-check).  Not the headline metric; prints its own JSON line."""
    import torch
    from paper_2503_18893_b200 import synth, xkv
    torch.cuda.set_device(0)
    s = make_shape(args)
    K, _ = synth.make_kv(s, device="cuda")                                          # (G, T, d) bf16
    X = torch.cat([K[l] for l in range(s.G)], dim=1).contiguous()
    del K
    r, q, p = s.r_k, 2, 32
    cfg = xkv.make_clf_config(T=s.T, G=s.G, d=s.d, r=r, oversample=p, power_iters=q)
    l = xkv.xkv_clf_rank_l(cfg)
    omega = synth.normal(synth.stream_key(s.seed, 31), (s.G * s.d, l), "cuda").to(torch.bfloat16)
    ws = torch.empty(xkv.xkv_clf_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    A = torch.empty((s.T, r), dtype=torch.bfloat16, device="cuda")
    B = torch.empty((s.G, r, s.d), dtype=torch.bfloat16, device="cuda")
    sig = torch.empty(r, dtype=torch.float32, device="cuda")
    ts = []
    for i in range(args.warmup + args.steps):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(); xkv.xkv_clf_factorize(cfg, X, omega, ws, A, B, sig); e1.record()
        torch.cuda.synchronize()
        if i >= args.warmup:
            ts.append(e0.elapsed_time(e1))
    st, flags = xkv.xkv_clf_status(ws)
    jacobi_sweeps = int(ws[:256].view(torch.int32)[11].item())       # diagnostic word of the workspace's flag block
    # residual against the optimum
    N = s.G * s.d
    gram = torch.zeros((N, N), dtype=torch.float64, device="cuda")
    for t0 in range(0, s.T, 16384):
        xb = X[t0:t0 + 16384].double()
        gram += xb.T @ xb
    ev = torch.linalg.eigvalsh(gram).flip(0).clamp_min(0)
    optimum = float(ev[r:].sum())
    Vm = torch.cat([B[g] for g in range(s.G)], dim=1).double()                      # (r, N)
    res = 0.0
    for t0 in range(0, s.T, 16384):
        res += float(((X[t0:t0 + 16384].double() - A[t0:t0 + 16384].double() @ Vm) ** 2).sum())
    ms = statistics.median(ts)
    tall_flops = (2 * (q + 2) + 1) * 2.0 * s.T * N * l                              # 2 products per iteration + A
    print(json.dumps({"op": "xkv_clf_factorize", "config": f"T={s.T}, G={s.G}, d={s.d} (X is {s.T} x {N}), r={r}, "
                      f"oversample={p} (l={l}), power_iters={q}", "ms": ms, "tall_product_tflops": tall_flops / (ms * 1e-3) / 1e12,
                      "residual_over_optimum": res / optimum, "relative_residual": res / float(ev.sum()),
                      "orthonormality_max_dev": float((Vm @ Vm.T - torch.eye(r, device="cuda", dtype=torch.float64)).abs().max()),
                      "sigma_max_rel_err": float(((sig.double() - ev[:r].sqrt()).abs() / ev[0].sqrt()).max()),
                      "jacobi_sweeps": jacobi_sweeps, "status": st, "flags": flags}))
    return 0


def measure_point(shape, args, world, rank, local_rank, dist, with_cpu=True, with_dense=False, cpu_problems=None):
    """Time the decode step of one workload on this rank's GPU and return the JSON line (a dict)."""
    import numpy as np
    import torch
    from paper_2503_18893_b200 import workload, xkv

    s = shape
    n_q = 8
    wl = workload.DeviceWorkload(shape, n_steps=n_q, device="cuda", groups=replica_units(shape.n_groups, rank),
                                 tail_rows=args.tail, quant_bits=getattr(args, "quant", 0))
    n_groups = len(wl.groups)
    q_bytes = n_groups * s.G * s.batch * s.H_q * s.d_h * 2
    out_bytes = q_bytes
    ddist = dist if world > 1 else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    for i in range(args.warmup):
        wl.step(i)
        if i == 0:
            st0, fl0 = xkv.xkv_group_status(wl.groups[0])
            if st0 != 0:   # a kernel gave up on a bounded wait or saw a bad index: do not time a broken run
                raise SystemExit(f"device status {st0} (flags {fl0}) after the first step: {xkv.xkv_strerror(st0)}")
    barrier()
    # how often the `steps`-step region is repeated: about a second of timed work, so that the clock sampler sees
    # the load and a slow outlier shows; one probe region decides
    e0 = ev(); e0.record(stream)
    for i in range(args.steps):
        wl.step(i)
    e1 = ev(); e1.record(stream)
    barrier()
    probe_ms = e0.elapsed_time(e1)
    repeats = args.repeats if args.repeats > 0 else int(min(200, max(3, round(1000.0 / max(probe_ms, 1e-3)))))
    if world > 1:       # every rank must run the same number of regions
        repeats = int(reduce_max(float(repeats), dist))

    # ---- timed region 1: inputs resident in HBM; `repeats` regions of exactly `steps` steps, each between two
    # events with a barrier on both sides; the reported region is the median one (max over ranks per region)
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    launches0 = xkv.xkv_kernel_launch_count()
    t_wall0 = time.time()
    regions = []
    for r in range(repeats):
        barrier()
        a = ev(); a.record(stream)
        for i in range(args.steps):
            wl.step(args.warmup + r * args.steps + i)
        b = ev(); b.record(stream)
        barrier()
        regions.append(reduce_max(a.elapsed_time(b), ddist))
    launches = (xkv.xkv_kernel_launch_count() - launches0) // repeats
    ms_total = statistics.median(regions)

    # ---- timed region 1b: the same steps again with an event around every ABI call, for the per-kernel roofline
    # (kept out of region 1: an event between two calls keeps the second call's kernels from starting under
    # programmatic dependent launch while the first call's kernels drain)
    marks = []
    for i in range(max(args.steps, 10)):
        for gi, grp in enumerate(wl.groups):
            q = wl.inputs[gi].q[(args.warmup + i) % n_q]
            a = ev(); a.record(stream)
            xkv.xkv_sr_select(grp, 0, s.G, q, s.k, wl.sel_idx[gi], wl.sel_cnt[gi])
            b = ev(); b.record(stream)
            wl.attend(gi, q)
            c = ev(); c.record(stream)
            marks.append((a, b, c))
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1)
    sel_ms = [a.elapsed_time(b) for (a, b, c) in marks]
    att_ms = [b.elapsed_time(c) for (a, b, c) in marks]
    st, flags = xkv.xkv_group_status(wl.groups[0])

    # unique rows actually gathered in the last step (compulsory bytes of the byte model)
    uniq = 0
    for gi in range(n_groups):
        for b_ in range(s.batch):
            rows = wl.sel_idx[gi][:, b_].reshape(-1)
            uniq += int(torch.unique(rows[rows >= 0]).numel())
    uniq_per_group = uniq / n_groups
    bytes_model = workload.algorithmic_bytes(s, unique_rows=uniq_per_group, quant_bits=getattr(args, "quant", 0))
    flops_paper = workload.algorithmic_flops(s)
    flops_exec = workload.executed_flops(s)
    pk = peaks()

    # ---- timed region 2: end to end through the C ABI with host buffers (pinned), copies inside
    q_host = [torch.stack([wl.inputs[gi].q[j] for gi in range(n_groups)]).cpu().pin_memory() for j in range(n_q)]
    q_dev = torch.empty_like(q_host[0], device="cuda")
    out_host = torch.empty(wl.out.shape, dtype=wl.out.dtype).pin_memory()
    e2e_steps = max(3, min(args.steps * repeats, 200) // 2)
    barrier()
    e0 = ev(); e0.record(stream)
    for i in range(e2e_steps):
        q_dev.copy_(q_host[i % n_q], non_blocking=True)
        wl.step(i, q_override=q_dev)
        out_host.copy_(wl.out, non_blocking=True)
        stream.synchronize()                      # the caller consumes the result before the next token
    e1 = ev(); e1.record(stream)
    barrier()
    e2e_ms = reduce_max(e0.elapsed_time(e1), ddist)

    total_group_steps = world * n_groups * args.steps
    value = total_group_steps / (ms_total * 1e-3)
    e2e_value = world * n_groups * e2e_steps / (e2e_ms * 1e-3)
    us_window = (ms_total / args.steps / n_groups) * 1e3

    # ---- dominant kernel: the reconstruct+attend call (gather, contraction, attention).  Its bound is the larger
    # of the byte term (unique gathered rows + B, at the measured HBM peak) and the tensor term of the flops the
    # kernel executes (the value side is re-associated); the paper's cost formula is kept as a labelled side field.
    att_s = statistics.mean(att_ms) * 1e-3
    sel_s = statistics.mean(sel_ms) * 1e-3
    att_bytes = bytes_model["rows_unique"] + bytes_model["B"] + bytes_model["small"]
    sel_bytes = bytes_model["landmarks"]
    hbm_t = att_bytes / (pk["hbm_gbs"] * 1e9)
    tc_t = flops_exec / (pk["bf16_tflops_sustained"] * 1e12)
    if hbm_t >= tc_t:
        roof = {"bound": "hbm", "achieved": att_bytes / att_s / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": flops_exec / att_s / 1e12, "peak": pk["bf16_tflops_sustained"],
                "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    headline_shape = (shape.name == "cfg3_llama_128k" and args.tail == 0 and not getattr(args, "quant", 0) and
                      (s.T, s.r_k, s.r_v, s.k, s.batch) == (131072, 512, 512, 4096, 1))
    roof.update({"traffic": captured_traffic("xkv_fused.cu") if headline_shape else None,
                 "kernel": "xkv_sr_reconstruct_attend (gather + reconstruct + attention)",
                 "peak_source": pk["source"], "us_per_launch": att_s * 1e6,
                 "algorithmic_bytes_per_launch": att_bytes,
                 "hbm_frac": att_bytes / att_s / 1e9 / pk["hbm_gbs"],
                 "executed_flops_per_launch": flops_exec,
                 "executed_tflops": flops_exec / att_s / 1e12,
                 "executed_frac_of_bf16_peak": flops_exec / att_s / 1e12 / pk["bf16_tflops_sustained"],
                 "paper_formula_flops_per_launch": flops_paper,
                 "paper_formula_tflops": flops_paper / att_s / 1e12})
    step_t = max(bytes_model["bytes_min"] / (pk["hbm_gbs"] * 1e9), tc_t)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": workload_config(shape, world),
        "repeats": {"regions": repeats, "steps_per_region": args.steps, "region_ms_median": ms_total,
                    "region_ms_min": min(regions), "region_ms_max": max(regions),
                    "value_from": "median region, max over ranks"},
        "tokens_per_s": world * s.batch * args.steps / (ms_total * 1e-3),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": q_bytes, "d2h_bytes_per_step": out_bytes,
                "steps": e2e_steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": roof,
        "select_kernel": {"us_per_launch": sel_s * 1e6, "algorithmic_bytes": sel_bytes,
                          "achieved_gbs": sel_bytes / sel_s / 1e9, "frac": sel_bytes / sel_s / 1e9 / pk["hbm_gbs"]},
        "step_roofline": {"bytes_min_per_group_step": bytes_model["bytes_min"],
                          "bytes_issued_per_group_step": bytes_model["bytes_issued"],
                          "executed_flops_per_group_step": flops_exec, "unique_rows_per_group_step": uniq_per_group,
                          "bound": "hbm" if bytes_model["bytes_min"] / (pk["hbm_gbs"] * 1e9) >= tc_t else "tensor",
                          "ideal_us": step_t * 1e6, "achieved_us": us_window, "frac": step_t * 1e6 / us_window,
                          "frac_of_nominal_8TBs": (bytes_model["bytes_min"] / 8e12) * 1e6 / us_window},
        "device_status": {"status": st, "flags": flags},
    }
    if getattr(args, "quant", 0):       # not the headline workload: 4-bit bases
        line["config"]["quant_bits"] = args.quant
        line["config"]["workload"] += f", token bases as {args.quant}-bit RTN codes (groups of 32)"
    if args.tail > 0:       # not the headline workload: the step also attends to uncompressed generated tokens
        line["config"]["tail_rows"] = args.tail
        line["config"]["workload"] += f", plus {args.tail} uncompressed tail rows per sequence"

    # ---- the dense arm: plain decode attention over an uncompressed bf16 cache of the same shape (what SR replaces)
    if with_dense:
        try:
            line["dense_attention"] = dense_arm(shape, wl, us_window, pk)
        except Exception as e:      # the arm is a side measurement: a failure there is reported, not fatal
            line["dense_attention"] = {"skipped": repr(e)[:200]}
            torch.cuda.empty_cache()

    # ---- the CPU oracle on the host cores (rank 0), timed on a bounded sample of window 0; the same oracle run also
    # serves as the parity check of what was just timed (window 0, query set 0)
    if rank == 0 and with_cpu:
        n_all = s.G * s.batch * s.H_kv
        n = cpu_problems or args.cpu_problems or min(n_all, 32)
        oinp = wl.inputs[0]
        if getattr(args, "quant", 0):       # the oracle works on what the codes stand for
            oinp = workload.GroupInputs(xkv.xkv_dequantize_rtn(*xkv.xkv_quantize_rtn(oinp.A_k, args.quant), bits=args.quant),
                                        xkv.xkv_dequantize_rtn(*xkv.xkv_quantize_rtn(oinp.A_v, args.quant), bits=args.quant),
                                        oinp.B_k, oinp.B_v, oinp.landmarks, oinp.q)
        dt, np_, cores, ores = oracle_sample(shape, oinp, n, spread=(n < n_all))
        line["cpu_baseline"] = {"value": (np_ / n_all) / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "seconds": dt,
                                "sample": f"{np_} of {n_all} (layer,head) problems of window 0, one step"}
        q0 = wl.inputs[0].q[0]
        xkv.xkv_sr_select(wl.groups[0], 0, s.G, q0, s.k, wl.sel_idx[0], wl.sel_cnt[0])
        wl.attend(0, q0)
        torch.cuda.synchronize()
        line["parity"] = parity_against(shape, ores, wl.sel_idx[0].cpu().numpy(), wl.sel_cnt[0].cpu().numpy(),
                                        wl.out[0].float().cpu().numpy(), wl.lse[0].cpu().numpy())
    wl.close()
    del wl
    torch.cuda.empty_cache()
    return line


def dense_arm(shape, wl, sr_us_window, pk):
    """Time xkv_dense_attend (and torch's scaled_dot_product_attention beside it, as a cross-check only) on window 0's
    shape with a synthetic uncompressed cache [G][batch][H_kv][T][d_h] for K and for V."""
    import torch
    from paper_2503_18893_b200 import synth, xkv
    s = shape
    cache_bytes = 2 * s.G * s.batch * s.H_kv * s.T * s.d_h * 2
    free, _ = torch.cuda.mem_get_info()
    if cache_bytes * 1.15 + (4 << 30) > free:
        return {"skipped": f"the uncompressed cache of one window is {cache_bytes / 1e9:.1f} GB; {free / 1e9:.1f} GB are free"}
    grp = wl.groups[0]
    try:
        need = xkv.xkv_dense_workspace_bytes(grp, s.T)
    except xkv.XKVError as e:
        return {"skipped": str(e)}
    # the cache is drawn layer by layer and sequence by sequence (the generator works in fp32: drawing 69 GB at once
    # would need twice that)
    K = torch.empty((s.G, s.batch, s.H_kv, s.T, s.d_h), dtype=torch.bfloat16, device="cuda")
    V = torch.empty_like(K)
    for l in range(s.G):
        for b in range(s.batch):
            for which, dst in ((21, K), (22, V)):
                dst[l, b] = synth.normal(synth.stream_key(s.seed, which, l, b), (s.H_kv, s.T, s.d_h), "cuda").to(torch.bfloat16)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    out = torch.empty((s.G, s.batch, s.H_q, s.d_h), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((s.G, s.batch, s.H_q), dtype=torch.float32, device="cuda")
    flush = torch.empty(192 << 20, dtype=torch.uint8, device="cuda") if cache_bytes < (512 << 20) else None
    ev = lambda: torch.cuda.Event(enable_timing=True)
    n_q = wl.n_steps

    def timed(fn, n_warm=3, n=10):
        ts = []
        for i in range(n_warm + n):
            if flush is not None:
                flush.zero_()                        # caches smaller than a few L2s: flush between calls
            a, b = ev(), ev()
            a.record(); fn(i); b.record()
            torch.cuda.synchronize()
            if i >= n_warm:
                ts.append(a.elapsed_time(b) * 1e3)
        return statistics.median(ts)

    ours = timed(lambda i: xkv.xkv_dense_attend(grp, 0, s.G, wl.inputs[0].q[i % n_q], K, V, None, s.T, ws, out, lse))
    res = {"kernel": "xkv_dense_attend", "us_per_window_step": ours, "cache_bytes": cache_bytes,
           "achieved_gbs": cache_bytes / (ours * 1e-6) / 1e9, "frac_of_hbm_peak": cache_bytes / (ours * 1e-6) / 1e9 / pk["hbm_gbs"],
           "sr_us_per_window_step": sr_us_window, "sr_speedup_over_dense": ours / sr_us_window,
           "l2": "flushed between calls" if flush is not None else "cache larger than L2"}
    try:
        import torch.nn.functional as F

        def sdpa(i):
            q = wl.inputs[0].q[i % n_q]
            for l in range(s.G):
                F.scaled_dot_product_attention(q[l].unsqueeze(2), K[l], V[l], enable_gqa=True)
        res["torch_sdpa_us_per_window_step"] = timed(sdpa)
    except Exception as e:      # a cross-check only
        res["torch_sdpa_us_per_window_step"] = None
        res["torch_sdpa_note"] = repr(e)[:120]
    del K, V, ws
    torch.cuda.empty_cache()
    return res


def sweep_points():
    """(label, shape) of the benchmark configurations besides the headline one and of the corner points of the
    stress sweep (config 5: T x r x k x batch on the Llama-shaped window).  Small points get several windows, visited
    round-robin, so that a step's inputs are several times the L2 and nothing survives in it between steps."""
    from paper_2503_18893_b200 import synth
    pts = [("cfg2 T=32K r=512 k=2048 B=1", synth.config(2, n_groups=4)),
           ("cfg3 T=128K r=512 k=4096 B=1 (headline)", synth.config(3, n_groups=8)),
           ("cfg3 T=128K r=512 k=4096 B=4", synth.config(3, batch=4, n_groups=2)),
           ("cfg4 Qwen-shaped T=64K r=256 k=2048 B=8 n_rep=7", synth.config(4, n_groups=2)),
           ("cfg5 T=64K r=512 k=4096 B=1 (centre)", synth.config(5, n_groups=4))]
    for T in (16384, 262144):
        for r in (256, 1024):
            for k in (1024, 16384):
                for B in (1, 16):
                    window_bytes = B * (T * 2 * r * 2 + 4 * (T // 8) * 1024 * 2)
                    n_groups = int(max(1, min(16, -(-(512 << 20) // window_bytes))))
                    pts.append((f"cfg5 T={T // 1024}K r={r} k={k} B={B}",
                                synth.config(5, T=T, r_k=r, r_v=r, k=k, batch=B, n_groups=n_groups,
                                             seed=1005 + (T // 1024) * 7 + r * 3 + k + B)))
    return pts


def run_sweep(args, world, rank, local_rank, dist):
    rows = []
    for label, shape in sweep_points():
        if args.sweep_filter and args.sweep_filter not in label:
            continue
        a = argparse.Namespace(**vars(args))
        a.steps, a.warmup, a.repeats, a.tail = 5, 3, 0, 0
        try:
            line = measure_point(shape, a, world, rank, local_rank, dist, with_cpu=True, with_dense=True, cpu_problems=2)
        except Exception as e:      # a point that does not fit or is not supported is reported, not fatal
            line = {"config": {"workload": label}, "skipped": repr(e)[:300]}
            import torch
            torch.cuda.empty_cache()
        line["point"] = label
        if rank == 0:
            print(json.dumps(line), flush=True)
        rows.append(line)
    if rank == 0 and args.sweep_out:
        with open(args.sweep_out, "w") as f:
            f.write(sweep_table(rows))
    return 0


def sweep_table(rows) -> str:
    out = ["| point | windows | SR us / window-step | window-steps/s | tokens/s | bytes_min MB | bound | roofline frac | "
           "select us | attend us | dense us (ours) | dense GB/s | torch SDPA us | SR speed-up over dense | parity (idx "
           "mismatch / max rel err) | SM MHz under load |", "|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|"]
    for r in rows:
        if "skipped" in r:
            out.append(f"| {r['point']} | skipped: {r['skipped']} |" + " |" * 14)
            continue
        sr, d = r["step_roofline"], r.get("dense_attention", {})
        par = r.get("parity", {})
        dense = (f"{d['us_per_window_step']:.0f} | {d['achieved_gbs']:.0f} | "
                 f"{(d.get('torch_sdpa_us_per_window_step') or float('nan')):.0f} | {d['sr_speedup_over_dense']:.2f}"
                 if "us_per_window_step" in d else f"{d.get('skipped', 'n/a')} | | | ")
        out.append(f"| {r['point']} | {r['config']['windows']} | {sr['achieved_us']:.1f} | {r['value']:.0f} | "
                   f"{r['tokens_per_s']:.0f} | {sr['bytes_min_per_group_step'] / 1e6:.1f} | {sr['bound']} | "
                   f"{sr['frac']:.3f} | {r['select_kernel']['us_per_launch']:.1f} | {r['roofline']['us_per_launch']:.1f} | "
                   f"{dense} | {par.get('idx_mismatch', 'n/a')} / {par.get('max_rel_err', float('nan')):.1e} | "
                   f"{r.get('clocks', {}).get('sm_mhz', float('nan')):.0f}"
                   f"{' (power cap)' if 'sw_power_cap' in r.get('clocks', {}).get('reasons', []) else ''} |")
    return "\n".join(out) + "\n"


def main():
    args = parse_args()
    if args.op == "landmarks":
        return run_landmarks(args)
    if args.op == "clf":
        return run_clf(args)
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if args.sweep:
        rc = run_sweep(args, world, rank, local_rank, dist)
    else:
        line = measure_point(make_shape(args), args, world, rank, local_rank, dist,
                             with_cpu=not args.no_cpu_baseline, with_dense=args.dense)
        if rank == 0:
            print(json.dumps(line))
        rc = 0
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return rc


if __name__ == "__main__":
    sys.exit(main())
