#!/usr/bin/env python
"""Benchmark of the quantized-Adam-with-error-feedback step on B200.

A "step" is one pass of the whole path over one batch of synthetic input: every
worker's compress (max-abs scale, quantize, pack, residual) followed by the
server's decode-average-update-broadcast.  The metric is elements per second,
elements = d * n per step (parameters times workers), whole job.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload flat28] [--n 16]
    python bench.py --impl reference ...      # the CPU oracle on a bounded sample

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs
an independent replica of the workload: the path has no exchange step between
GPUs, so there is no collective in the data path; the time is the maximum over
ranks and the value the elements all ranks processed per second.

One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "qadam_ef_step_elements_per_s"
UNIT = "elements/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic per (worker, element) or per element measured with ncu
# (dram__bytes_read.sum + dram__bytes_write.sum of one launch divided by the units
# it processed; profiles/ holds the captures).  Valid only for the kernel sources
# whose digest is recorded beside it.
NCU_TRAFFIC = {
    # kernel: (bytes per unit, digest of csrc/ at capture time)
    # profiles/dram_traffic_flat28_n16_server_moments.txt: the benchmark's own workload
    # (flat28, n = 16, moments on the server), one-pass capture of the two byte counters
    "absmax": (8.00, "7bed1ed2fd2fbf57"),
    "quantize": (12.24, "7bed1ed2fd2fbf57"),
    "server": (28.03, "7bed1ed2fd2fbf57"),
    # profiles/worker_resident_bert_base_n4.md: the on-chip worker kernel on the BERT-base-shaped
    # set with n = 4 (a case small enough for a multi-pass capture), scaled by the pairs it takes
    "worker_fused:server": (12.12, "7bed1ed2fd2fbf57"),
    "worker_fused:worker": (28.10, "7bed1ed2fd2fbf57"),
}


def csrc_digest() -> str:
    h = hashlib.sha256()
    base = os.path.join(ROOT, "paper_2004_14180_b200", "csrc")
    for name in sorted(os.listdir(base)):
        with open(os.path.join(base, name), "rb") as f:
            h.update(name.encode())
            h.update(f.read())
    return h.hexdigest()[:16]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="flat28")
    ap.add_argument("--n", type=int, default=None, help="worker count (default: the workload's)")
    ap.add_argument("--placement", default="server", choices=["server", "worker"],
                    help="where Adam's moments live")
    ap.add_argument("--kg", type=int, default=None)
    ap.add_argument("--kx", type=int, default=None)
    ap.add_argument("--single-scale", action="store_true", help="one max-abs scale per worker")
    ap.add_argument("--scale-block-log2", type=int, default=0,
                    help="one max-abs scale per block of 2^K elements of a tensor (0: per tensor)")
    ap.add_argument("--weight-decay", type=float, default=0.0,
                    help="lambda of the l2 term g + lambda * (held weights); 0: none")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sample-log2", type=int, default=None,
                    help="log2 of the per-worker sample length the oracle is timed on")
    return ap.parse_args()


def get_workload(args):
    import qadam_inputs as qi
    w = qi.get_workload(args.workload, n=args.n)
    kw = {}
    if args.kg is not None:
        kw["kg"] = args.kg
    if args.kx is not None:
        kw["kx"] = args.kx
    if args.single_scale:
        kw["per_tensor_scale"] = False
    if args.scale_block_log2 > 0:
        kw["scale_block"] = 1 << args.scale_block_log2
    return w.with_(**kw) if kw else w


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- byte accounting

def algorithmic_bytes(kernel: str, w, placement: str, D: int, gbits: int, xbits: int,
                      pass_model=None, l2_term: bool = False) -> float:
    """Bytes one launch of `kernel` must move at its interface (fp32 state it has
    to read and write, packed codes), for all n workers.  The worker side is capacity
    aware: (worker, segment) pairs that fit on chip go through the fused kernel and are
    counted once (one pass); larger ones take the two streaming launches and are counted
    twice (the max-abs scale needs the whole pair before any of it can be quantized)."""
    n = w.n
    server_moments = placement == "server"
    # with the l2 term a worker also reads the weights it holds: the packed broadcast, or x
    held = ((xbits / 8.0) if xbits else 4.0) if l2_term else 0.0
    if kernel == "worker_fused":    # the on-chip kernel: the one-pass pairs, every array touched once
        one_pass, _ = pass_model
        # read g, e, write e and the codes; moments on the workers: also read and write m, v
        return one_pass * ((12.0 if server_moments else 28.0) + held + gbits / 8.0)
    # the split launches cover everything, or, beside the fused kernel, the two-pass pairs only
    split_units = pass_model[1] if pass_model and pass_model[0] > 0 else n * D
    if kernel == "absmax":      # phase 1: read g, e (worker moments: + read m, v, write m, v, u)
        per = (8.0 if server_moments else 28.0) + held
        return per * split_units
    if kernel == "quantize":    # phase 2: read g, e (or u), write e and the codes
        per = (12.0 + held if server_moments else 8.0) + gbits / 8.0
        return per * split_units
    if kernel == "identity":
        per = ((8.0 + 8.0) if server_moments else (16.0 + 16.0)) + held
        return per * n * D
    if kernel == "server":      # read n code streams and x (m, v); write x (m, v) and the broadcast
        state = 24.0 if server_moments else 8.0
        return (n * gbits / 8.0 + state + xbits / 8.0) * D
    if kernel == "broadcast":
        return (4.0 + xbits / 8.0) * D
    raise KeyError(kernel)


# ----------------------------------------------------------------------------- the oracle, timed

def time_oracle(w, placement: str, sample_log2: int, steps: int, warmup: int, weight_decay: float = 0.0):
    """Times the CPU oracle (single thread) on a bounded sample of the workload:
    the same n, quantizers and distributions, each worker's vector cut to
    2**sample_log2 elements.  Returns (elements/s, description, seconds per step)."""
    import numpy as np
    import oracle
    import qadam_inputs as qi
    oracle.build()
    d_s = min(w.d, 1 << sample_log2)
    sample_log2 = d_s.bit_length() - 1 if d_s & (d_s - 1) == 0 else sample_log2
    ws = w.with_(seg_len=(d_s,), fan_in=(0,), is_gamma=(False,), per_tensor_scale=True,
                 w0="gauss:0.05" if w.w0 == "he" else w.w0)
    place = oracle.PLACE_SERVER if placement == "server" else oracle.PLACE_WORKER
    st = oracle.OracleState([d_s], ws.n, ws.kg, ws.kx, place, ws.beta1, ws.beta2, ws.eps)
    st.set_weights(qi.initial_weights(ws, "cpu").numpy())
    st.set_regularization(weight_decay)
    g = st.to_padded(np.stack([qi.gradients(ws, 1, i, "cpu").numpy() for i in range(ws.n)]))
    for _ in range(warmup):
        st.step(g, ws.lr, threads=1)
    t0 = time.perf_counter()
    for _ in range(steps):
        st.step(g, ws.lr, threads=1)
    dt = (time.perf_counter() - t0) / max(1, steps)
    desc = (f"{w.name}: n={ws.n} workers, each cut to {d_s} elements "
            f"({steps} timed steps after {warmup} warm-up), one thread")
    return ws.n * d_s / dt, desc, dt


def run_reference(args):
    rank, _, _ = rank_env()
    if rank != 0:
        return
    w = get_workload(args)
    sample_log2 = args.sample_log2 or 22
    value, desc, dt = time_oracle(w, args.placement, sample_log2, args.steps, args.warmup, args.weight_decay)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(w, args, extra={"sample": desc}),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(w, args, extra=None):
    cfg = {
        "workload": f"{w.name} (d={w.d}, {w.num_segments} scale segment(s), n={w.n} workers)",
        "d": w.d, "n_workers": w.n, "segments": w.num_segments,
        "kg": w.kg, "kx": w.kx, "placement": args.placement, "weight_decay": args.weight_decay,
        "beta1": w.beta1, "beta2": w.beta2, "eps": w.eps, "lr": w.lr,
        "gradients": w.grad, "parallelism": f"replicas x{args.gpus} (no exchange between GPUs)",
        "l2": ("inputs larger than L2 (no flush between steps)" if 8 * w.n * w.d > (1 << 28) else
               "inputs fit in L2 and are not flushed: an L2-resident number, not HBM evidence"),
    }
    if extra:
        cfg.update(extra)
    return cfg


# ----------------------------------------------------------------------------- ranks

def rank_env():
    """(rank, world size, local rank) as torch.distributed.run exports them."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time: replicas finish when the last one does."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(d: int, n_workers: int, world: int, ms_per_step: float) -> float:
    """Whole-job elements per second: every rank steps its own replica of d*n elements."""
    return world * d * n_workers / (ms_per_step * 1e-3)


# ----------------------------------------------------------------------------- the CUDA path

def run_b200(args):
    import torch
    import torch.distributed as dist
    import qadam_inputs as qi
    import paper_2004_14180_b200 as qb

    rank, world, local = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); "
                         "use --impl reference for the oracle")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = get_workload(args)
    placement = qb.PLACE_SERVER if args.placement == "server" else qb.PLACE_WORKER
    x1 = qi.initial_weights(w, dev)
    q = qb.QAdam(w.scale_seg_len, w.n, kg=w.kg, kx=w.kx, placement=placement, beta1=w.beta1,
                 beta2=w.beta2, eps=w.eps, lr=w.lr, x1=x1, device=dev)
    q.set_regularization(args.weight_decay)
    del x1
    D = q.D
    if w.n * D * 4 <= (1 << 27):
        print(f"note: gradient input is {w.n * D * 4 >> 20} MiB, not larger than L2", file=sys.stderr)
    # one batch of gradients, resident in HBM; the same batch feeds every step
    g = torch.zeros(w.n, D, dtype=torch.float32, device=dev)
    for i in range(w.n):
        gi = qi.gradients(w, 1, i, dev)
        g[i].copy_(q.to_padded(gi))
        del gi
    torch.cuda.synchronize()

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    step = 0
    for _ in range(max(3, args.warmup)):
        step += 1
        q.step(step, g)
    sync_all()

    q.profile(True)
    q.profile_read()
    launches0 = q.launches
    clocks = ClockSampler(local)
    time.sleep(0.25)
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step += 1
        q.step(step, g)
    e1.record()
    sync_all()
    ms_total = e0.elapsed_time(e1)
    clock_info = clocks.stop()
    prof = q.profile_read()
    q.profile(False)
    gpu_launches = q.launches - launches0
    status = q.poll_status()

    ms_total = max_over_ranks(ms_total, world, dev)
    ms_step = ms_total / args.steps
    value = job_value(w.d, w.n, world, ms_step)

    # ---- end to end through the host-buffer entry point -------------------------------
    e2e = None
    if not args.no_e2e:
        g_host = torch.empty(w.n * D, dtype=torch.float32, pin_memory=True)
        g_host.copy_(g.view(-1))
        out_bytes = q.wcode_bytes if w.kx >= 0 else 4 * D
        out_host = torch.empty(out_bytes, dtype=torch.uint8, pin_memory=True)
        step += 1
        q.step_host(step, g_host, g, out_host)          # warm-up
        sync_all()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(args.e2e_steps):
            step += 1
            q.step_host(step, g_host, g, out_host)
        s1.record()
        sync_all()
        ms_e2e = max_over_ranks(s0.elapsed_time(s1), world, dev) / args.e2e_steps
        e2e = {"value": job_value(w.d, w.n, world, ms_e2e), "unit": UNIT,
               "h2d_bytes_per_step": w.n * D * 4, "d2h_bytes_per_step": out_bytes,
               "steps": args.e2e_steps, "ms_per_step": ms_e2e,
               "api": "qadam_step_host (pinned host gradients in, packed broadcast out)"}
        del g_host, out_host

    # ---- roofline of the dominant kernel ---------------------------------------------
    peak, peak_kind = measured_peak()
    kernels = {}
    for name, (ms, cnt) in prof.items():
        if cnt == 0:
            continue
        per = ms / cnt
        bytes_ = algorithmic_bytes(name, w, args.placement, D, q.gcode_bytes * 8 // D, q.wcode_bytes * 8 // D,
                                   pass_model=q.worker_pass_model(), l2_term=args.weight_decay != 0.0)
        kernels[name] = {"launches": int(cnt), "ms_per_launch": per,
                         "share": ms / sum(m for m, c in prof.values()),
                         "algorithmic_bytes": bytes_, "achieved_gbs": bytes_ / (per * 1e-3) / 1e9,
                         "frac": bytes_ / (per * 1e-3) / 1e9 / peak}
    dom = max(kernels, key=lambda k: kernels[k]["launches"] * kernels[k]["ms_per_launch"])
    traffic = None
    tkey = f"{dom}:{args.placement}" if dom == "worker_fused" else dom
    if tkey in NCU_TRAFFIC and NCU_TRAFFIC[tkey][1] == csrc_digest() and args.weight_decay == 0.0 \
            and (dom == "worker_fused" or args.placement == "server"):
        one_pass, two_pass = q.worker_pass_model()
        units = {"worker_fused": one_pass, "absmax": two_pass if one_pass else w.n * D,
                 "quantize": two_pass if one_pass else w.n * D}.get(dom, D)
        traffic = NCU_TRAFFIC[tkey][0] * units
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["achieved_gbs"],
                "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                "frac": kernels[dom]["frac"], "traffic": traffic,
                "step_frac": sum(k["algorithmic_bytes"] * k["launches"] for k in kernels.values())
                / args.steps / (ms_step * 1e-3) / 1e9 / peak}

    if rank == 0:
        cpu_baseline = None
        if not args.no_cpu_baseline and world == 1:
            sl = args.sample_log2 or 24
            v, desc, _ = time_oracle(w, args.placement, sl, steps=2, warmup=0, weight_decay=args.weight_decay)
            cpu_baseline = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc}
        sent = q.sent_bytes_per_step()
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": workload_config(w, args, extra={
                "D_padded": D, "gcode_bits": q.gcode_bytes * 8 // D, "wcode_bits": q.wcode_bytes * 8 // D,
                "sent_bytes_per_step": sent, "compression_ratio": q.compression_ratio(),
                "broadcast_bytes_per_step": q.wcode_bytes}),
            "clocks": clock_info, "e2e": e2e, "gpu_launches": int(gpu_launches),
            "roofline": roofline, "kernels": kernels, "cpu_baseline": cpu_baseline,
            "device_status": int(status),
        }
        print(json.dumps(line), flush=True)
    q.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_b200(args)


if __name__ == "__main__":
    main()
