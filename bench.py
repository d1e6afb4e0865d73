"""Benchmark of the fused 4-bit AdamW step (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one pass of the whole hot path (rank-1 maxima pass, reciprocal pass, update/re-quantize pass)
over every tensor of the workload. The default workload is the LLaMA-7B-shaped parameter list with bf16
gradients (6.74 G fp32 parameters, about 47.5 GB resident), far larger than L2, so no flush is needed
between iterations. With N > 1 (one process per GPU under torch.distributed.run) every rank runs its own
copy of the per-GPU workload with no collective inside the step (weak scaling).

`--impl reference` times the CPU oracle (a deliberately plain program) on a bounded sample of the same
workload on the host cores; under a multi-rank launch only rank 0 runs it.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "4-bit AdamW step: Gparams/s and achieved HBM GB/s vs B200 peak"
UNIT = "Gparams/s"

# Algorithmic bytes per parameter (each operand read once and written once, scales included) for a
# 2-D rank-1 tensor: w 4+4, g 2 (bf16) or 4 (fp32), m codes 0.5+0.5, v codes 0.5+0.5, m block maxima 8/128.
# The update/re-quantize pass moves exactly these; the maxima pass re-reads g and the v codes.
PASS2_BYTES = {"bf16": 12.0625, "f32": 14.0625}
PASS1_BYTES = {"bf16": 2.5, "f32": 4.5}
# DRAM traffic of the update/re-quantize pass measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum)
# per parameter, from the capture of the 464.5 M-parameter LLaMA slice summarised in
# profiles/pass2_llama_7b_1l.txt (3.2950 GB read + 2.2835 GB written); traffic scales with the parameter count.
# fp32 gradients: capture of the RoBERTa-large list (355.4 M params, 3.2749 GB read + 1.7452 GB written), same file.
PASS2_TRAFFIC_BYTES_PER_PARAM = {"bf16": 12.009, "f32": 14.125}
# DRAM traffic of the whole step per parameter by schedule (ncu, same metrics): two-pass = the update pass above plus
# the maxima pass (2.503 B/param, profiles/pass1_llama_7b_1l.txt); fused = one launch, from the capture of the
# four-decoder-layer LLaMA slice (817.96 M params) summarised in profiles/schedules_llama_7b.txt, at the library's default
# tuning (7.931 GB read + 4.092 GB written; 13.98 B/param at the tuning that keeps most in L2).
STEP_TRAFFIC_BYTES_PER_PARAM = {"two_pass": {"bf16": 14.512}, "fused": {"bf16": 14.699}}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama_7b")
    ap.add_argument("--optimizer", choices=["adamw", "sgdm"], default="adamw",
                    help="sgdm: the compressed SGDM step (Alg. 2) instead of the AdamW step; no end-to-end leg")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--m-block", type=int, default=128, choices=[128, 2048], help="first-moment block size")
    ap.add_argument("--v-mode", default="rank1", choices=["rank1", "block", "factored"],
                    help="second moment of matrices: rank-1 or block-wise 4-bit, or factorized (fp32 row/column statistics)")
    ap.add_argument("--schedule", default="auto", choices=["auto", "two_pass", "fused", "overlap"],
                    help="order of the maxima and update work inside a step (lpmm_schedule)")
    ap.add_argument("--tile-elems", type=int, default=0)
    ap.add_argument("--tile-elems-maxima", type=int, default=0)
    ap.add_argument("--l2-keep-mb", type=int, default=0)
    ap.add_argument("--lead-melems", type=int, default=0)
    ap.add_argument("--gap-items", type=int, default=0)
    ap.add_argument("--no-l2-hints", action="store_true")
    ap.add_argument("--overlap-groups", type=int, default=0)
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        import torch
        self.proc = None
        self.path = None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            ident = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            ident = str(device_index)
        try:
            fd, self.path = tempfile.mkstemp(prefix="lpmm_clocks_", suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", ident, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t0: float, t1: float) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            from datetime import datetime
            for line in open(self.path):
                parts = [p.strip() for p in line.strip().split(",")]
                if len(parts) < 8:
                    continue
                try:
                    ts = datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(parts[1]), float(parts[2]), parts[4:8]))
                except Exception:
                    continue
        finally:
            try:
                os.unlink(self.path)
            except Exception:
                pass
        inside = [r for r in rows if t0 - 0.03 <= r[0] <= t1 + 0.03] or rows
        if not inside:
            return out
        sm = sorted(r[1] for r in inside)
        out["sm_mhz"] = sm[len(sm) // 2]
        out["sm_max_mhz"] = inside[0][2]
        out["samples"] = len(inside)
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        out["reasons"] = [n for k, n in enumerate(names) if any(r[3][k] == "Active" for r in inside)]
        return out


# ----------------------------------------------------------------------------- oracle legs

def oracle_sample(wl, small: bool = False, budget: int = 350_000_000):
    """The bounded sample of the workload the CPU oracle is timed on. Lists of up to 80 M parameters: all of it. The
    LLaMA list: the token embedding plus every tensor of one decoder layer (333 M parameters); other large lists: their
    first tensors up to about 350 M parameters. A smaller `budget` (parameters per step) drops tensors from the end of
    that sample. small=True: the first large matrix only (for the single-thread leg)."""
    items = list(enumerate(wl.tensors))
    if small:
        mats = [(i, t) for i, t in items if t.ndim >= 2 and t.numel >= 1 << 20] or items
        i, t = mats[1] if len(mats) > 1 else mats[0]
        return [(i, t)], f"one tensor ({t.name}, {t.rows}x{t.cols})"
    if wl.numel <= 80_000_000:
        return items, "whole workload"
    if wl.name.startswith("llama_7b") and not wl.name.endswith("flat"):
        cand = [(i, t) for i, t in items if t.name.startswith("l0.")] + [(i, t) for i, t in items if t.name == "embed"]
        if sum(t.numel for _, t in cand) <= budget:
            return cand, "every tensor of one decoder layer + the token embedding"
        label = "tensors of one decoder layer"
    else:
        cand, label = items, "tensors of the list"
    picked, total = [], 0
    for i, t in cand:
        if total + t.numel > budget and picked:
            break
        picked.append((i, t))
        total += t.numel
    return picked, f"the first {len(picked)} {label} ({', '.join(sorted({f'{t.rows}x{t.cols}' for _, t in picked if t.numel > 4096}))})"


def time_oracle(wl, steps: int, warmup: int, threads: int | None = None, small: bool = False, budget: int = 350_000_000):
    """Runs the oracle as it stands on the sample; returns (Gparams/s, threads, description, ms/step)."""
    import numpy as np
    import torch
    import oracle
    from paper_2309_01507_b200 import workloads
    sample, desc = oracle_sample(wl, small, budget)
    hyper = dict(lr=wl.lr, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, weight_decay=wl.weight_decay)
    gdt = torch.bfloat16 if wl.grad_dtype == "bf16" else torch.float32
    all_threads = oracle.threads()
    if threads is not None:
        oracle.set_threads(threads)
    try:
        ws, gs, sts = [], [], []
        for i, t in sample:
            ws.append(workloads.make_param(t, wl.index, i).numpy().ravel().copy())
            gs.append(workloads.make_grad(t, wl.index, i, 1, dtype=gdt).float().numpy().ravel())
            sts.append(oracle.state_init(t.rows, t.cols, oracle.kind_of(t.rows, t.cols, t.ndim, 4096, int(t.force_quant))))
        n = sum(t.numel for _, t in sample)
        step = 0
        for _ in range(warmup):
            step += 1
            for w, g, st in zip(ws, gs, sts):
                oracle.adamw4_step(w, g, st, step=step, **hyper)
        t0 = time.perf_counter()
        for _ in range(steps):
            step += 1
            for w, g, st in zip(ws, gs, sts):
                oracle.adamw4_step(w, g, st, step=step, **hyper)
        dt = time.perf_counter() - t0
        used = oracle.threads()
    finally:
        oracle.set_threads(all_threads)
    return n * steps / dt / 1e9, used, f"{desc}, {n / 1e6:.1f} M params per step, {steps} step(s)", dt / steps * 1e3


def run_reference(args):
    from paper_2309_01507_b200 import dist, workloads
    rank, _, _ = dist.env()
    if rank != 0:
        return
    wl = workloads.WORKLOADS[args.workload]()
    # about two minutes of oracle time in all at the ~0.06 Gparams/s it reaches on 16 cores: the sample shrinks with K + W
    steps, warmup = max(args.steps, 1), max(args.warmup, 0)
    budget = int(min(350e6, 0.06e9 * 120 / (steps + warmup)))
    value, threads, desc, ms = time_oracle(wl, steps, warmup, budget=budget)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "sample": desc, "grad_dtype": wl.grad_dtype},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- the CUDA arm

def run_ours(args):
    import torch
    from paper_2309_01507_b200 import build as cuda_build
    from paper_2309_01507_b200 import dist, lpmm, workloads

    rank, local_rank, world = dist.env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the fused step has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    cuda_build.build()
    dist.init("nccl")

    wl = workloads.WORKLOADS[args.workload]()
    gdt = torch.bfloat16 if wl.grad_dtype == "bf16" else torch.float32
    hyper = dict(lr=wl.lr, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, weight_decay=wl.weight_decay)
    params = [workloads.make_param(t, wl.index, i, device=dev) for i, t in enumerate(wl.tensors)]
    grads = [workloads.make_grad(t, wl.index, i, 1, device=dev, dtype=gdt) for i, t in enumerate(wl.tensors)]
    v_mode = {"rank1": lpmm.V_RANK1, "block": lpmm.V_BLOCK, "factored": lpmm.V_FACTORED}[args.v_mode]
    schedule = {"auto": lpmm.SCHEDULE_AUTO, "two_pass": lpmm.SCHEDULE_TWO_PASS, "fused": lpmm.SCHEDULE_FUSED,
                "overlap": lpmm.SCHEDULE_OVERLAP}[args.schedule]
    cfg = lpmm.default_config(m_block=args.m_block, v_mode=v_mode, schedule=schedule, tile_elems=args.tile_elems,
                              tile_elems_maxima=args.tile_elems_maxima, l2_keep_mbytes=args.l2_keep_mb,
                              lead_melems=args.lead_melems, gap_items=args.gap_items, no_l2_hints=int(args.no_l2_hints), overlap_groups=args.overlap_groups)
    state = lpmm.state_init(cfg, wl.tensors, device=dev)
    cache = lpmm.make_ptr_cache(params, grads)
    n_params = wl.numel
    torch.cuda.synchronize()

    sgdm = args.optimizer == "sgdm"

    def one_step(t):
        if sgdm:
            lpmm.sgdm4_step(state, params, grads, lr=wl.lr, beta=wl.beta1)
        else:
            lpmm.adamw4_step(state, params, grads, step=t, ptr_cache=cache, **hyper)

    step = 0
    for _ in range(max(args.warmup, 3)):
        step += 1
        one_step(step)
    torch.cuda.synchronize()
    dist.barrier()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    if state.schedule == lpmm.SCHEDULE_FUSED:
        lpmm.wait_stats(state)          # clear what the warm-up left
    lpmm.profile(state, True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t_wall0 = time.time()
    ev0.record()
    for _ in range(args.steps):
        step += 1
        one_step(step)
    ev1.record()
    torch.cuda.synchronize()
    t_wall1 = time.time()
    dist.barrier()
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    prof = lpmm.profile_read(state)
    waits = lpmm.wait_stats(state) if state.schedule == lpmm.SCHEDULE_FUSED else None
    lpmm.profile(state, False)
    launches = state.last_launches * args.steps
    ms_total = dist.max_over_ranks(ev0.elapsed_time(ev1), device=dev)
    ms_step = ms_total / args.steps
    value = world * n_params / (ms_step * 1e-3) / 1e9

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    e2e = None
    if not args.no_e2e and args.e2e_steps > 0 and not sgdm:
        gsz = 2 if wl.grad_dtype == "bf16" else 4
        nstage = lpmm.stage_bytes(state)
        d_pstage = torch.empty(nstage, dtype=torch.uint8, device=dev)
        d_gstage = torch.empty(nstage, dtype=torch.uint8, device=dev)
        h_p = torch.empty(n_params, dtype=torch.float32, pin_memory=True)
        h_g = torch.empty(n_params, dtype=gdt, pin_memory=True)
        hp, hg, off = [], [], 0
        for p, g in zip(params, grads):
            k = p.numel()
            hp.append(h_p[off:off + k]); hg.append(h_g[off:off + k])
            hp[-1].copy_(p.reshape(-1)); hg[-1].copy_(g.reshape(-1))
            off += k
        torch.cuda.synchronize()
        e2e_state = lpmm.state_init(cfg, wl.tensors, device=dev)
        t = 0
        for _ in range(1):
            t += 1
            lpmm.adamw4_step_host(e2e_state, hp, hg, d_pstage, d_gstage, step=t, **hyper)
        torch.cuda.synchronize()
        dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.e2e_steps):
            t += 1
            lpmm.adamw4_step_host(e2e_state, hp, hg, d_pstage, d_gstage, step=t, **hyper)
        e1.record()
        torch.cuda.synchronize()
        dist.barrier()
        e2e_ms = dist.max_over_ranks(e0.elapsed_time(e1), device=dev) / args.e2e_steps
        e2e = {"value": world * n_params / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": (4 + gsz) * n_params, "d2h_bytes_per_step": 4 * n_params,
               "ms_per_step": e2e_ms, "steps": args.e2e_steps,
               "note": "lpmm_adamw4_step_host: pinned host params+grads copied in, updated params copied out, every step; copies of neighbouring tensor groups overlap the kernels"}
        del d_pstage, d_gstage, h_p, h_g, hp, hg, e2e_state

    if rank != 0:
        dist.shutdown()
        return

    peak, peak_kind = measured_peak()
    fused = state.schedule == lpmm.SCHEDULE_FUSED and not sgdm
    p2_ms = prof["pass2_ms"] / max(prof["steps"], 1)
    p1_ms = prof["pass1_ms"] / max(prof["steps"], 1)
    if sgdm or fused:      # one kernel per step: its duration is the step time
        p2_ms, p1_ms = ms_step, 0.0
    # block maxima: 8 bytes per block of m (and of v when v is block-wise; then pass 1 has nothing to do).
    # A list of 1-D tensors only (flattened parameters) is block-wise whatever the mode (Sec. 4.2).
    v_kind = "block" if all(t.ndim == 1 for t in wl.tensors) else args.v_mode
    pass2_bpp = PASS2_BYTES[wl.grad_dtype] - 8 / 128 + 8 / args.m_block + (8 / 128 if v_kind == "block" else 0)
    pass1_bpp = {"rank1": PASS1_BYTES[wl.grad_dtype], "block": 0.0, "factored": PASS1_BYTES[wl.grad_dtype] - 0.5}[v_kind]
    if v_kind == "factored":
        pass2_bpp -= 1.0      # no second-moment codes are read or written
    if sgdm:                  # w 4+4, g, first-moment codes 1, block maxima
        pass2_bpp = 8.0 + (2.0 if wl.grad_dtype == "bf16" else 4.0) + 1.0 + 8 / args.m_block
        pass1_bpp = 0.0
    # The step as a whole. "Algorithmic" = what the method's two reads of every rank-1 tensor amount to (the maxima
    # pass re-reads the gradient and the second-moment codes): pass1_bpp + pass2_bpp per parameter. The single-pass
    # figure (each operand once) is printed beside it.
    step_bytes = (pass1_bpp + pass2_bpp) * n_params
    single_bytes = pass2_bpp * n_params
    step_gbs = step_bytes / (ms_step * 1e-3) / 1e9
    single_gbs = single_bytes / (ms_step * 1e-3) / 1e9
    default_quant = v_kind == "rank1" and args.m_block == 128 and not sgdm
    traffic_pp = None
    if default_quant:         # the captures cover the default quantizers only
        traffic_pp = STEP_TRAFFIC_BYTES_PER_PARAM["fused" if fused else "two_pass"].get(wl.grad_dtype)
    kernels = {}
    if not (sgdm or fused):
        p2_gbs = single_bytes / (p2_ms * 1e-3) / 1e9
        kernels["pass2_kernel (update + re-quantize)"] = {
            "ms_per_launch": p2_ms, "algorithmic_bytes_per_launch": single_bytes, "achieved": p2_gbs, "frac": p2_gbs / peak,
            "frac_of_nominal_8tbs": p2_gbs / 8000.0,
            "traffic": None if not default_quant else PASS2_TRAFFIC_BYTES_PER_PARAM[wl.grad_dtype] * n_params}
        if p1_ms > 0:
            p1_gbs = pass1_bpp * n_params / (p1_ms * 1e-3) / 1e9
            kernels["pass1_kernel (row/column maxima)"] = {
                "ms_per_launch": p1_ms, "algorithmic_bytes_per_launch": pass1_bpp * n_params, "achieved": p1_gbs,
                "frac": p1_gbs / peak, "frac_of_nominal_8tbs": p1_gbs / 8000.0}
    sm_mhz = (clocks or {}).get("sm_mhz")
    roofline = {"bound": "hbm",
                "kernel": "sgdm_kernel" if sgdm else ("step_fused_kernel (one launch per step)" if fused else
                                                      "whole step: pass1_kernel + rcp_kernel + pass2_kernel"),
                "achieved": step_gbs, "peak": peak, "unit": "GB/s", "frac": step_gbs / peak, "peak_kind": f"of {peak_kind}",
                "frac_of_nominal_8tbs": step_gbs / 8000.0,
                "traffic": None if traffic_pp is None else traffic_pp * n_params,
                "algorithmic_bytes_per_step": step_bytes, "bytes_per_param": pass1_bpp + pass2_bpp,
                "single_pass": {"bytes_per_param": pass2_bpp, "achieved": single_gbs, "frac": single_gbs / peak,
                                "frac_of_nominal_8tbs": single_gbs / 8000.0},
                "ms_per_step": ms_step, "ms_x_sm_ghz": None if not sm_mhz else ms_step * sm_mhz / 1000.0,
                "kernels": kernels}

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        v, threads, desc, _ = time_oracle(wl, 1, 1)
        v1, t1, desc1, _ = time_oracle(wl, 1, 1, threads=1, small=True)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
               "single_thread": {"value": v1, "unit": UNIT, "cores": t1, "sample": desc1}}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "tensors": len(wl.tensors), "params_per_gpu": n_params,
                       "grad_dtype": wl.grad_dtype, "param_dtype": "f32", "m": f"B{args.m_block}/DE 4-bit", "v": {"rank1": "Rank-1/Linear 4-bit", "block": "B128/Linear 4-bit", "factored": "factorized (fp32 row/column statistics)"}[v_kind] if not sgdm else "none (compressed SGDM, Alg. 2)",
                       "l2": f"inputs larger than L2 ({(n_params * (8 + (2 if wl.grad_dtype == 'bf16' else 4) + 1)) / 1e9:.1f} GB touched per step), no flush", "parallelism": f"replicas x{world}, no collective"},
            "clocks": clocks, "waits": waits, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)
    dist.shutdown()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
