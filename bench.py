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

NOMINAL_HBM_GBS = 8000.0     # the B200's HBM3e figure the 75 % target is stated against


def ncu_traffic():
    """DRAM bytes per unit (a (worker, element) pair for the worker kernels, an element for the
    server pass) taken with ncu on small cases of the same kernels, with the digest of the
    kernel sources they were taken on.  A record whose digest is not the current one is stale
    and not used."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as f:
            return json.load(f)
    except Exception:
        return {}


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
    ap.add_argument("--grad", default=None,
                    help="gradient distribution in place of the workload's, e.g. gauss_clip:5 (Gaussian clipped "
                         "at 5 sigma: about 1.2 %% of the ternary codes non-zero), gauss_clip:4 (4.6 %%), gauss_clip:2 (32 %%)")
    ap.add_argument("--scale-block-log2", type=int, default=0,
                    help="one max-abs scale per block of 2^K elements of a tensor (0: per tensor)")
    ap.add_argument("--weight-decay", type=float, default=0.0,
                    help="lambda of the l2 term g + lambda * (held weights); 0: none")
    ap.add_argument("--weight-feedback", action="store_true",
                    help="give the weight broadcast an error buffer of its own (Q_x applied to x + e^w)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--mode", default="replicas", choices=["replicas", "ps"],
                    help="with several GPUs: independent replicas (default), or ONE problem with the "
                         "workers dealt out to the ranks and the server sharded (codes exchanged over NCCL)")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the per-configuration records (key `configs` of the line)")
    ap.add_argument("--config-steps", type=int, default=5)
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
    if args.grad:
        kw["grad"] = args.grad
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
                      pass_model=None, l2_term: bool = False, weight_feedback: bool = False) -> float:
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
        if weight_feedback:     # the broadcast's own error buffer is read and written too
            state += 8.0
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
        "weight_feedback": bool(getattr(args, "weight_feedback", False)),
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

def alu_decode_peak():
    """Codes per second the decode of the server pass could sustain if nothing but its two
    busiest pipes mattered: a ternary code costs one logic operation (16 lanes per scheduler,
    2 cycles per warp instruction) and half an add.f32x2 plus half an fma.f32x2 (2 cycles per
    warp instruction each on the 32-lane fp32 pipe), so a scheduler retires 32 codes per 2
    cycles on either pipe: 64 codes per clock and SM at the maximum SM clock."""
    import torch
    props = torch.cuda.get_device_properties(torch.cuda.current_device())
    mhz = 1965.0
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            mhz = float(json.load(f).get("sm_max_mhz", mhz))
    except Exception:
        pass
    return props.multi_processor_count * 64.0 * mhz * 1e6


def kernel_table(prof, w, placement_name, q, weight_decay, peak, weight_feedback=False):
    """Per kernel: launches, time, algorithmic bytes, achieved rate and its fractions."""
    D = q.D
    kernels = {}
    total_ms = sum(m for m, c in prof.values()) or 1.0
    for name, (ms, cnt) in prof.items():
        if cnt == 0:
            continue
        per = ms / cnt
        bytes_ = algorithmic_bytes(name, w, placement_name, D, q.gcode_bytes * 8 // D, q.wcode_bytes * 8 // D,
                                   pass_model=q.worker_pass_model(), l2_term=weight_decay != 0.0,
                                   weight_feedback=weight_feedback)
        gbs = bytes_ / (per * 1e-3) / 1e9
        kernels[name] = {"launches": int(cnt), "ms_per_launch": per, "share": ms / total_ms,
                         "algorithmic_bytes": bytes_, "achieved_gbs": gbs,
                         "frac": gbs / peak, "frac_of_nominal": gbs / NOMINAL_HBM_GBS}
        if name == "server" and w.kg == 0:
            # second roofline of the server pass: with dense codes (always, when the moments are on
            # the workers) it is bound by the arithmetic of the decode, not by HBM
            codes = float(w.n) * D / (per * 1e-3)
            kernels[name]["alu"] = {"bound": "alu", "achieved": codes, "peak": alu_decode_peak(),
                                    "unit": "codes/s", "frac": codes / alu_decode_peak()}
    return kernels


class Measured:
    """One workload set up on the device and timed: the context stays open for the caller."""

    def __init__(self, w, placement_name, weight_decay, steps, warmup, dev, world, peak, sample_clocks,
                 weight_feedback=False):
        import torch
        import torch.distributed as dist
        import qadam_inputs as qi
        import paper_2004_14180_b200 as qb
        self.w, self.placement_name, self.weight_decay = w, placement_name, weight_decay
        placement = qb.PLACE_SERVER if placement_name == "server" else qb.PLACE_WORKER
        x1 = qi.initial_weights(w, dev)
        q = qb.QAdam(w.scale_seg_len, w.n, kg=w.kg, kx=w.kx, placement=placement, beta1=w.beta1,
                     beta2=w.beta2, eps=w.eps, lr=w.lr, x1=x1, device=dev, want_wfeedback=weight_feedback)
        q.set_regularization(weight_decay)
        del x1
        self.q, D = q, q.D
        # one batch of gradients, resident in HBM; the same batch feeds every step
        g = torch.zeros(w.n, D, dtype=torch.float32, device=dev)
        for i in range(w.n):
            gi = qi.gradients(w, 1, i, dev)
            g[i].copy_(q.to_padded(gi))
            del gi
        self.g = g
        torch.cuda.synchronize()

        def sync_all():
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
                torch.cuda.synchronize()
        self.sync_all = sync_all

        self.step = 0
        for _ in range(max(3, warmup)):
            self.step += 1
            q.step(self.step, g)
        sync_all()
        q.profile(True)
        q.profile_read()
        launches0 = q.launches
        clocks = ClockSampler(dev.index or 0) if sample_clocks else None
        if clocks:
            time.sleep(0.25)
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            self.step += 1
            q.step(self.step, g)
        e1.record()
        sync_all()
        ms_total = e0.elapsed_time(e1)
        self.clock_info = clocks.stop() if clocks else None
        prof = q.profile_read()
        q.profile(False)
        self.gpu_launches = q.launches - launches0
        self.status = q.poll_status()
        self.ms_step = max_over_ranks(ms_total, world, dev) / steps
        self.value = job_value(w.d, w.n, world, self.ms_step)
        self.kernels = kernel_table(prof, w, placement_name, q, weight_decay, peak, weight_feedback)
        self.step_bytes = sum(k["algorithmic_bytes"] * k["launches"] for k in self.kernels.values()) / steps

    def close(self):
        self.q.close()
        self.g = None
        self.q = None


# The configurations reported beside the headline: both large workloads over the worker-count
# sweep, the ResNet-18-shaped sets, both placements of the moments, one run with the l2 term,
# and (a fifth field) two with an error buffer of its own for the weight broadcast.
CONFIG_RUNS = (
    ("bert_base", None, "server", 0.0), ("bert_base", None, "worker", 0.0),
    ("bert_base", None, "server", 5e-4),
    ("bert_base", None, "server", 0.0, True), ("flat28", 16, "server", 0.0, True),
    ("flat28", 1, "server", 0.0), ("flat28", 4, "server", 0.0), ("flat28", 32, "server", 0.0),
    ("flat28", 1, "worker", 0.0), ("flat28", 4, "worker", 0.0), ("flat28", 16, "worker", 0.0),
    ("flat28", 32, "worker", 0.0),
    ("resnet18_qg", None, "server", 0.0), ("resnet18_qg", None, "worker", 0.0),
    ("resnet18_qg_qx_k0", None, "server", 0.0), ("resnet18_qg_qx_k0", None, "worker", 0.0),
    ("resnet18_qg_qx_k1", None, "server", 0.0), ("resnet18_qg_qx_k1", None, "worker", 0.0),
    ("flat20", None, "server", 0.0), ("flat20", None, "worker", 0.0),
)


def config_records(args, dev, world, peak):
    """One record per configuration: step time, elements/s and every kernel's fraction of the
    measured copy rate and of the nominal HBM rate."""
    import torch
    import qadam_inputs as qi
    out = []
    free_b, _total = torch.cuda.mem_get_info(dev)
    for name, n, placement_name, wd, *more in CONFIG_RUNS:
        wf = bool(more and more[0])
        w = qi.get_workload(name, n=n)
        # g, e (and the workers' m, v) dominate; skip what this device cannot hold
        need = w.n * w.d * 4 * (4 if placement_name == "worker" else 2) + 4 * w.d * 4
        rec = {"workload": w.name, "n_workers": w.n, "placement": placement_name, "weight_decay": wd,
               "weight_feedback": wf, "kg": w.kg, "kx": w.kx, "d": w.d, "segments": w.num_segments}
        if need > 0.92 * free_b:
            rec["skipped"] = f"needs {need >> 30} GiB of {free_b >> 30} GiB free"
            out.append(rec)
            continue
        m = Measured(w, placement_name, wd, args.config_steps, 3, dev, world, peak, sample_clocks=True,
                     weight_feedback=wf)
        rec.update({"ms_per_step": m.ms_step, "value": m.value, "unit": UNIT, "steps": args.config_steps,
                    "device_status": int(m.status), "clocks": m.clock_info,
                    "step_frac": m.step_bytes / (m.ms_step * 1e-3) / 1e9 / peak,
                    "step_frac_of_nominal": m.step_bytes / (m.ms_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                    "l2": ("inputs larger than L2" if 8 * w.n * w.d > (1 << 28)
                           else "fits in L2: not HBM evidence"),
                    "kernels": {k: {"ms_per_launch": v["ms_per_launch"], "launches": v["launches"],
                                    "achieved_gbs": v["achieved_gbs"], "frac": v["frac"],
                                    "frac_of_nominal": v["frac_of_nominal"],
                                    **({"alu_frac": v["alu"]["frac"]} if "alu" in v else {})}
                                for k, v in m.kernels.items()}})
        m.close()
        del m
        torch.cuda.empty_cache()
        out.append(rec)
    return out


def run_b200(args):
    import torch
    import torch.distributed as dist

    rank, world, local = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); "
                         "use --impl reference for the oracle")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = get_workload(args)
    peak, peak_kind = measured_peak()
    m = Measured(w, args.placement, args.weight_decay, args.steps, args.warmup, dev, world, peak,
                 sample_clocks=True, weight_feedback=args.weight_feedback)
    q, g, D = m.q, m.g, m.q.D
    if w.n * D * 4 <= (1 << 27):
        print(f"note: gradient input is {w.n * D * 4 >> 20} MiB, not larger than L2", file=sys.stderr)
    ms_step, value, kernels = m.ms_step, m.value, m.kernels
    step = m.step

    # ---- end to end through the host-buffer entry point -------------------------------
    e2e = None
    if not args.no_e2e:
        g_host = torch.empty(w.n * D, dtype=torch.float32, pin_memory=True)
        g_host.copy_(g.view(-1))
        out_bytes = q.wcode_bytes if w.kx >= 0 else 4 * D
        out_host = torch.empty(out_bytes, dtype=torch.uint8, pin_memory=True)
        step += 1
        q.step_host(step, g_host, g, out_host)          # warm-up
        m.sync_all()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(args.e2e_steps):
            step += 1
            q.step_host(step, g_host, g, out_host)
        s1.record()
        m.sync_all()
        ms_e2e = max_over_ranks(s0.elapsed_time(s1), world, dev) / args.e2e_steps
        e2e = {"value": job_value(w.d, w.n, world, ms_e2e), "unit": UNIT,
               "h2d_bytes_per_step": w.n * D * 4, "d2h_bytes_per_step": out_bytes,
               "steps": args.e2e_steps, "ms_per_step": ms_e2e,
               "api": "qadam_step_host (pinned host gradients in, packed broadcast out)"}
        del g_host, out_host

    # ---- roofline of the dominant kernel ---------------------------------------------
    dom = max(kernels, key=lambda k: kernels[k]["launches"] * kernels[k]["ms_per_launch"])
    traffic, traffic_note = None, None
    tkey = f"{dom}:{args.placement}"
    trec = ncu_traffic().get(tkey)
    if trec and args.weight_decay == 0.0:
        if trec.get("digest") == csrc_digest():
            one_pass, two_pass = q.worker_pass_model()
            units = {"worker_fused": one_pass, "absmax": two_pass if one_pass else w.n * D,
                     "quantize": two_pass if one_pass else w.n * D}.get(dom, D)
            traffic = trec["bytes_per_unit"] * units
            traffic_note = trec.get("case")
        else:
            traffic_note = "the kernel sources changed since the counters were taken"
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["achieved_gbs"],
                "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                "frac": kernels[dom]["frac"], "traffic": traffic, "traffic_note": traffic_note,
                "nominal_peak": NOMINAL_HBM_GBS, "frac_of_nominal": kernels[dom]["frac_of_nominal"],
                "step_frac": m.step_bytes / (ms_step * 1e-3) / 1e9 / peak,
                "step_frac_of_nominal": m.step_bytes / (ms_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                # the target is stated against the nominal rate: which kernels of this run meet it
                "target_0p75_of_nominal": {k: v["frac_of_nominal"] >= 0.75 for k, v in kernels.items()
                                           if k != "broadcast"}}
    sent = q.sent_bytes_per_step()
    cfg = workload_config(w, args, extra={
        "D_padded": D, "gcode_bits": q.gcode_bytes * 8 // D, "wcode_bits": q.wcode_bytes * 8 // D,
        "sent_bytes_per_step": sent, "compression_ratio": q.compression_ratio(),
        "broadcast_bytes_per_step": q.wcode_bytes})
    clock_info, gpu_launches, status = m.clock_info, m.gpu_launches, m.status
    m.close()
    del m, q, g
    torch.cuda.empty_cache()

    configs = None
    if not args.no_configs and world == 1:
        configs = config_records(args, dev, world, peak)

    if rank == 0:
        cpu_baseline = None
        if not args.no_cpu_baseline and world == 1:
            sl = args.sample_log2 or 24
            v, desc, _ = time_oracle(w, args.placement, sl, steps=2, warmup=0, weight_decay=args.weight_decay)
            cpu_baseline = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": cfg,
            "clocks": clock_info, "e2e": e2e, "gpu_launches": int(gpu_launches),
            "roofline": roofline, "kernels": kernels, "cpu_baseline": cpu_baseline,
            "device_status": int(status), "configs": configs,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_ps(args):
    """One problem over all ranks: rank r compresses its share of the workers, the packed codes
    are exchanged (all-to-all), each rank serves its range of the vector, and the packed weights
    are gathered back.  Total work is fixed as ranks are added: strong scaling."""
    import torch
    import torch.distributed as dist
    import qadam_inputs as qi
    import paper_2004_14180_b200 as qb
    from paper_2004_14180_b200 import ps

    rank, world, local = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py --mode ps needs a CUDA device")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if not dist.is_initialized():
        if world == 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    w = get_workload(args)
    if w.n % world:
        w = w.with_(n=(w.n + world - 1) // world * world)        # workers are dealt out evenly
    placement = qb.PLACE_SERVER if args.placement == "server" else qb.PLACE_WORKER
    x1 = qi.initial_weights(w, dev)
    q = qb.QAdam(w.scale_seg_len, w.n, kg=w.kg, kx=w.kx, placement=placement, beta1=w.beta1,
                 beta2=w.beta2, eps=w.eps, lr=w.lr, x1=x1, device=dev)
    q.set_regularization(args.weight_decay)
    del x1
    drv = ps.ShardedStep(q, always_communicate=True)
    k = drv.plan.workers_per_rank
    g = torch.zeros(k, q.D, dtype=torch.float32, device=dev)
    for j, i in enumerate(drv.plan.workers_of(rank)):
        g[j].copy_(q.to_padded(qi.gradients(w, 1, i, dev)))

    def sync_all():
        torch.cuda.synchronize()
        dist.barrier()
        torch.cuda.synchronize()

    step = 0
    for _ in range(max(3, args.warmup)):
        step += 1
        drv.step(step, g)
    sync_all()
    launches0 = q.launches
    clocks = ClockSampler(local)
    time.sleep(0.25)
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step += 1
        drv.step(step, g)
    e1.record()
    sync_all()
    ms_step = max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps
    clock_info = clocks.stop()
    status = q.poll_status()
    if rank == 0:
        wire = ps.wire_bytes_per_step(drv.plan, q.S)
        cfg = workload_config(w, args, extra={
            "parallelism": f"sharded parameter server over {world} rank(s): {k} worker(s) and 1/{world} of the "
                           "vector per rank; all-to-all of packed codes, all-gather of scales, broadcast of "
                           "the packed weights (NCCL)",
            "D_padded": q.D, "wire_bytes_per_step": wire, "shard_cuts": list(drv.plan.cuts)})
        line = {"metric": METRIC, "value": w.d * w.n / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_step,
                "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "mode": "ps", "config": cfg, "clocks": clock_info,
                "gpu_launches": int(q.launches - launches0), "device_status": int(status)}
        print(json.dumps(line), flush=True)
    q.close()
    dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.mode == "ps":
        run_ps(args)
    else:
        run_b200(args)


if __name__ == "__main__":
    main()
