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

# dram__bytes_read.sum + dram__bytes_write.sum per launch, sr_fused_kernel (95.46 + 3.38 MB) + merge_segments_kernel
# (5.65 MB), one window of config 3
NCU_ATTEND_DRAM_BYTES = 104.5e6
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
    ap.add_argument("--op", default="decode", choices=["decode", "landmarks"],
                    help="decode: the hot path (default).  landmarks: the prefill-side Algorithm 1 kernel alone "
                         "(not the headline metric; prints its own JSON line)")
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


def shard_units(n_units: int, rank: int, world: int):
    """Contiguous share of n_units independent units for `rank` (sizes differ by at most one)."""
    lo = (n_units * rank) // world
    hi = (n_units * (rank + 1)) // world
    return list(range(lo, hi))


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


def oracle_sample(shape, inp, n_problems):
    """Time the CPU oracle (as it stands) on the first n_problems (layer, sequence, head) problems of a window.
    Returns (seconds, problems, threads)."""
    import numpy as np
    from oracle import xkv_oracle as O
    f32 = lambda t: t.detach().float().cpu().numpy()
    A_k, A_v, B_k, B_v, lm, q = (f32(t) for t in (inp.A_k, inp.A_v, inp.B_k, inp.B_v, inp.landmarks, inp.q[0]))
    allp = [(l, b, g) for l in range(shape.G) for b in range(shape.batch) for g in range(shape.H_kv)]
    probs = allp[:n_problems]
    t0 = time.perf_counter()
    O.sr_decode_step(A_k, A_v, B_k, B_v, lm, q, k=shape.k, c=shape.c, H_kv=shape.H_kv, rope_base=shape.rope_base,
                     problems=probs)
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        threads = max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    return dt, len(probs), threads


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
        dt, np_, threads = oracle_sample(shape, inp, n)
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


def main():
    args = parse_args()
    if args.op == "landmarks":
        return run_landmarks(args)
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    from paper_2503_18893_b200 import workload

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_2503_18893_b200 import xkv

    shape = make_shape(args)
    # Each rank owns one full replica of the workload (its own sequence): per-GPU work is fixed.
    n_q = 8
    wl = workload.DeviceWorkload(shape, n_steps=n_q, device="cuda", tail_rows=args.tail)
    n_groups = len(wl.groups)
    s = shape
    q_bytes = n_groups * s.G * s.batch * s.H_q * s.d_h * 2
    out_bytes = q_bytes

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    stream = torch.cuda.current_stream()
    for i in range(args.warmup):
        wl.step(i)
        if i == 0:
            st0, fl0 = xkv.xkv_group_status(wl.groups[0])
            if st0 != 0:   # a kernel gave up on a bounded wait or saw a bad index: do not time a broken run
                raise SystemExit(f"device status {st0} (flags {fl0}) after the first step: {xkv.xkv_strerror(st0)}")
    barrier()

    # ---- timed region 1: inputs resident in HBM, exactly `steps` steps between two events
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    launches0 = xkv.xkv_kernel_launch_count()
    barrier()
    t_wall0 = time.time()
    e_start = ev(); e_start.record(stream)
    for i in range(args.steps):
        wl.step(args.warmup + i)
    e_stop = ev(); e_stop.record(stream)
    barrier()
    launches = xkv.xkv_kernel_launch_count() - launches0
    ms_total = reduce_max(e_start.elapsed_time(e_stop), dist if world > 1 else None)

    # ---- timed region 1b: the same steps again with an event around every ABI call, for the per-kernel roofline
    # (kept out of region 1: an event between two calls keeps the second call's kernels from starting under
    # programmatic dependent launch while the first call's kernels drain)
    marks = []
    for i in range(args.steps):
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
    bytes_model = workload.algorithmic_bytes(s, unique_rows=uniq_per_group)
    flops = workload.algorithmic_flops(s)
    pk = peaks()

    # ---- timed region 2: end to end through the C ABI with host buffers (pinned), copies inside
    q_host = [torch.stack([wl.inputs[gi].q[j] for gi in range(n_groups)]).cpu().pin_memory() for j in range(n_q)]
    q_dev = torch.empty_like(q_host[0], device="cuda")
    out_host = torch.empty(wl.out.shape, dtype=wl.out.dtype).pin_memory()
    e2e_steps = max(3, args.steps // 2)
    barrier()
    e0 = ev(); e0.record(stream)
    for i in range(e2e_steps):
        q_dev.copy_(q_host[i % n_q], non_blocking=True)
        wl.step(i, q_override=q_dev)
        out_host.copy_(wl.out, non_blocking=True)
        stream.synchronize()                      # the caller consumes the result before the next token
    e1 = ev(); e1.record(stream)
    barrier()
    e2e_ms = reduce_max(e0.elapsed_time(e1), dist if world > 1 else None)

    total_group_steps = world * n_groups * args.steps
    value = total_group_steps / (ms_total * 1e-3)
    e2e_value = world * n_groups * e2e_steps / (e2e_ms * 1e-3)

    # dominant kernel: reconstruct+attend (gather, contraction, attention); HBM bound at this shape
    att_s = statistics.mean(att_ms) * 1e-3
    sel_s = statistics.mean(sel_ms) * 1e-3
    att_bytes = bytes_model["rows_unique"] + bytes_model["B"] + bytes_model["small"]
    sel_bytes = bytes_model["landmarks"]
    hbm_t = att_bytes / (pk["hbm_gbs"] * 1e9)
    tc_t = flops / (pk["bf16_tflops_sustained"] * 1e12)
    if hbm_t >= tc_t:
        roof = {"bound": "hbm", "achieved": att_bytes / att_s / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": flops / att_s / 1e12, "peak": pk["bf16_tflops_sustained"],
                "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    # DRAM bytes of one reconstruct_attend call (fused kernel + segment merge) from the ncu capture of one window of
    # this workload (profiles/kernels_one_window_cfg3.md); it only applies to the unmodified headline shape.
    traffic = None
    if shape.name == "cfg3_llama_128k" and (s.T, s.r_k, s.r_v, s.k, s.batch) == (131072, 512, 512, 4096, 1):
        traffic = NCU_ATTEND_DRAM_BYTES
    roof.update({"traffic": traffic, "kernel": "xkv_sr_reconstruct_attend (gather + reconstruct + attention)",
                 "peak_source": pk["source"], "us_per_launch": att_s * 1e6,
                 "algorithmic_bytes_per_launch": att_bytes, "algorithmic_flops_per_launch": flops})
    step_t = max(bytes_model["bytes_min"] / (pk["hbm_gbs"] * 1e9), tc_t)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": workload_config(shape, world),
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
                          "flops_per_group_step": flops, "unique_rows_per_group_step": uniq_per_group,
                          "ideal_us": step_t * 1e6, "achieved_us": (ms_total / args.steps / n_groups) * 1e3,
                          "frac": step_t / ((ms_total / args.steps / n_groups) * 1e-3),
                          "frac_of_nominal_8TBs": (bytes_model["bytes_min"] / 8e12) /
                                                  ((ms_total / args.steps / n_groups) * 1e-3)},
        "device_status": {"status": st, "flags": flags},
    }
    if args.tail > 0:       # not the headline workload: the step also attends to uncompressed generated tokens
        line["config"]["tail_rows"] = args.tail
        line["config"]["workload"] += f", plus {args.tail} uncompressed tail rows per sequence"
        line["roofline"]["traffic"] = None
    if rank == 0 and not args.no_cpu_baseline:
        n = args.cpu_problems or min(s.G * s.batch * s.H_kv, 32)
        dt, np_, threads = oracle_sample(shape, wl.inputs[0], n)
        line["cpu_baseline"] = {"value": (np_ / (s.G * s.batch * s.H_kv)) / dt, "unit": UNIT, "cores": threads,
                                "kind": "oracle", "seconds": dt,
                                "sample": f"{np_} of {s.G * s.batch * s.H_kv} (layer,head) problems of window 0, one step"}
    wl.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))
    return 0


if __name__ == "__main__":
    sys.exit(main())
