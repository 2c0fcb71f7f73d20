#!/usr/bin/env python
"""Benchmark of the TSLT hot path on B200: one step = tslt_sparsify over all draft rows plus
tslt_verify over all target rows of the throughput-sweep workload (B=256, gamma=8, V=256000,
bf16, top-k 64, temperature 1), with the logits resident in HBM.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--extras]

* value        rows/s over the whole job (draft rows + target rows per step, all ranks),
               timed with CUDA events on the launching stream, max over ranks.
* roofline     the dominant kernel's achieved HBM GB/s (algorithmic bytes per launch over its
               mean event-timed duration inside the timed region) against the measured copy
               bandwidth in MEASURED_PEAKS.json.
* e2e          the same step driven from pinned HOST buffers: H2D of the logits and uniforms
               and D2H of the sparse payload and the verdicts are inside the timed region.
* cpu_baseline the CPU oracle, as it stands, on a bounded sample of the same rows (rank 0).
* --impl reference   times the oracle alone on the host cores (there is no reference
               implementation of this path to install; the oracle stands in for it).
With N > 1 every rank runs the same per-GPU workload on its own GPU (rows and sequences are
independent: weak scaling, no data-path collective); only timing is reduced.
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

import numpy as np
import torch

from paper_2512_16273_b200 import synth

WORKLOAD = synth.CONFIGS[4]
METRIC = "TSLT sparsify+verify rows/s and achieved HBM GB/s as fraction of B200 peak"
UNIT = "rows/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of each entry point's streaming kernel
# (sparsify_kernel, verify_stream_kernel) from the ncu captures summarised under profiles/.  Each
# entry point is two kernels on this workload (streaming, then finish / resolve: 4 launches per
# step); the event-timed duration of an entry point covers both.
NCU_TRAFFIC_BYTES = {"sparsify_kernel": 1108.9e6, "verify_kernel": 1188.1e6}


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ---- distributed plumbing (timing only) -----------------------------------------------------
def dist_setup(n_gpus: int, backend: str = "nccl"):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        if not dist.is_initialized():
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29511")
            dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local, world


def dist_barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def reduce_max(x: float, world: int, device="cpu") -> float:
    if world <= 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate(rows_per_rank: int, seconds_this_rank: float, world: int, device="cpu"):
    """Whole-job throughput: every rank processed rows_per_rank rows; the job took the slowest
    rank's time.  Returns (rows/s over all ranks, seconds)."""
    t = reduce_max(seconds_this_rank, world, device)
    return rows_per_rank * world / t, t


# ---- clocks ---------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.thread = [], None, None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        def pump():
            for line in self.proc.stdout:
                self.rows.append(line.strip())
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, smax, reasons = [], [], set()
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None, "samples": len(sm), "reasons": sorted(reasons)}


# ---- the CPU oracle leg ---------------------------------------------------------------------
def oracle_sample_run(zq_rows, zp_seqs, k, top_p, T, seed):
    """Time the oracle on draft rows [n, V] and target sequences [m, gamma+1, V] (CPU tensors),
    spread over the host cores with one thread per core (ctypes releases the GIL)."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    cores = len(os.sched_getaffinity(0))
    n, V = zq_rows.shape
    m, g1, _ = zp_seqs.shape
    gamma = g1 - 1
    ud = synth.uniforms((n, 1), seed, synth.TID_U_DRAFT).numpy()
    ua = synth.uniforms((m, gamma), seed, synth.TID_U_ACCEPT).numpy()
    us = synth.uniforms((m,), seed, synth.TID_U_SAMPLE).numpy()
    zq_np, _ = oracle.as_logits(zq_rows)
    zp_np, _ = oracle.as_logits(zp_seqs)
    oracle.lib()
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=cores) as ex:
        parts = list(ex.map(lambda r: oracle.sparsify(zq_np[r:r + 1], k, top_p, T, ud[r:r + 1]), range(n)))
    t1 = time.perf_counter()
    sp = {key: np.concatenate([p[key] for p in parts]) for key in ("idx", "logit", "count", "token")}
    # verifier sample: the first gamma draft rows of the sample stand in for each sequence's drafts
    reps = (m * gamma + n - 1) // n
    di = np.tile(sp["idx"], (reps, 1))[:m * gamma].reshape(m, gamma, k)
    dl = np.tile(sp["logit"], (reps, 1))[:m * gamma].reshape(m, gamma, k)
    dc = np.tile(sp["count"], reps)[:m * gamma].reshape(m, gamma)
    tk = np.tile(sp["token"][:, 0], reps)[:m * gamma].reshape(m, gamma)
    t2 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=cores) as ex:
        list(ex.map(lambda b: oracle.verify(zp_np[b:b + 1], di[b:b + 1], dl[b:b + 1], dc[b:b + 1], tk[b:b + 1],
                                            T, T, ua[b:b + 1], us[b:b + 1]), range(m)))
    t3 = time.perf_counter()
    rows = n + m * g1
    secs = (t1 - t0) + (t3 - t2)
    return rows / secs, rows, secs, min(cores, max(n, m))


def run_reference(args):
    """--impl reference: the oracle, as it stands, on a bounded sample of the workload per step."""
    rank, local, world = int(os.environ.get("RANK", "0")), 0, int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    w = WORKLOAD
    dt = synth.torch_dtype(w["dtype"])
    n_rows, n_seq = 8, 1
    zq, zp = synth.sequence_logits(n_seq + 1, w["gamma"], w["V"], dt, w["sigma_t"], 0, "cpu")
    zq_rows = zq.reshape(-1, w["V"])[:n_rows].contiguous()
    zp_seqs = zp[:n_seq].contiguous()
    for _ in range(args.warmup):
        oracle_sample_run(zq_rows[:2], zp_seqs[:1, :2], w["k"], w["top_p"], w["temperature"], 0)
    tot_rows, tot_secs, cores = 0, 0.0, 1
    for s in range(args.steps):
        _, rows, secs, cores = oracle_sample_run(zq_rows, zp_seqs, w["k"], w["top_p"], w["temperature"], s)
        tot_rows += rows
        tot_secs += secs
    value = tot_rows / tot_secs
    sample = "%d draft rows + %d sequence(s) x %d target rows of the workload per step" % (n_rows, n_seq, w["gamma"] + 1)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_secs / max(args.steps, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(B=None):
    w = WORKLOAD
    return {"workload": w["name"], "B": B or w["B"], "gamma": w["gamma"], "V": w["V"], "logits_dtype": w["dtype"],
            "k": w["k"], "top_p": w["top_p"], "temperature": w["temperature"],
            "l2": "inputs (1.05 GB draft + 1.18 GB target logits) are larger than L2, no flush needed"}


# ---- the GPU leg ----------------------------------------------------------------------------
def make_inputs(device, seed=0, B=None):
    w = WORKLOAD
    B = B or w["B"]
    dt = synth.torch_dtype(w["dtype"])
    zq, zp = synth.sequence_logits(B, w["gamma"], w["V"], dt, w["sigma_t"], seed, device)
    rows = B * w["gamma"]
    ud = synth.uniforms((rows, 1), seed, synth.TID_U_DRAFT, device)
    ua = synth.uniforms((B, w["gamma"]), seed, synth.TID_U_ACCEPT, device)
    us = synth.uniforms((B,), seed, synth.TID_U_SAMPLE, device)
    return zq, zp, ud, ua, us


def gpu_step(tslt, zq, zp, ud, ua, us, k, top_p, T, s_out, v_out, ws_s, ws_v, events=None):
    B, gamma, V = zq.shape
    if events:
        events[0].record()
    tslt.sparsify(zq, k, top_p, T, ud, out=s_out, ws=ws_s)
    if events:
        events[1].record()
    tslt.verify(zp, s_out["idx"], s_out["logit"], s_out["count"], s_out["token"], T, T, ua, us, out=v_out, ws=ws_v)
    if events:
        events[2].record()


def alloc_outputs(B, gamma, k, device, diag=False):
    rows = B * gamma
    s_out = {"idx": torch.empty(rows, k, dtype=torch.int32, device=device),
             "logit": torch.empty(rows, k, dtype=torch.float32, device=device),
             "count": torch.empty(rows, dtype=torch.int32, device=device),
             "token": torch.empty(rows, 1, dtype=torch.int32, device=device),
             "lse": torch.empty(rows, dtype=torch.float32, device=device),
             "mass": torch.empty(rows, dtype=torch.float32, device=device)}
    v_out = {"accepted_len": torch.empty(B, dtype=torch.int32, device=device),
             "out_token": torch.empty(B, dtype=torch.int32, device=device)}
    return s_out, v_out


def time_config(tslt, zq, zp, ud, ua, us, k, top_p, T, steps, warmup):
    """Event-timed loop; returns (seconds total, mean sparsify ms, mean verify ms)."""
    B, gamma, V = zq.shape
    dev = zq.device
    s_out, v_out = alloc_outputs(B, gamma, k, dev)
    ws_s = torch.empty(tslt.sparsify_workspace_bytes(B * gamma, V, k, 1), dtype=torch.uint8, device=dev)
    ws_v = torch.empty(tslt.verify_workspace_bytes(B, gamma, V, k), dtype=torch.uint8, device=dev)
    for _ in range(warmup):
        gpu_step(tslt, zq, zp, ud, ua, us, k, top_p, T, s_out, v_out, ws_s, ws_v)
    torch.cuda.synchronize()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    for i in range(steps):
        gpu_step(tslt, zq, zp, ud, ua, us, k, top_p, T, s_out, v_out, ws_s, ws_v, evs[i])
    torch.cuda.synchronize()
    total_ms = evs[0][0].elapsed_time(evs[-1][2])
    sp_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in evs)
    vf_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in evs)
    assert tslt.workspace_status(ws_s) == 0 and tslt.workspace_status(ws_v) == 0
    return total_ms / 1e3, sp_ms, vf_ms, s_out, v_out


def run_e2e(tslt, zq, zp, ud, ua, us, k, top_p, T, steps, warmup):
    """The same step from pinned host buffers, copies inside the timed region."""
    B, gamma, V = zq.shape
    dev = zq.device
    h = {name: torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
         for name, t in (("zq", zq), ("zp", zp), ("ud", ud), ("ua", ua), ("us", us))}
    d = {name: torch.empty_like(t) for name, t in (("zq", zq), ("zp", zp), ("ud", ud), ("ua", ua), ("us", us))}
    s_out, v_out = alloc_outputs(B, gamma, k, dev)
    ws_s = torch.empty(tslt.sparsify_workspace_bytes(B * gamma, V, k, 1), dtype=torch.uint8, device=dev)
    ws_v = torch.empty(tslt.verify_workspace_bytes(B, gamma, V, k), dtype=torch.uint8, device=dev)
    outs = [s_out["idx"], s_out["logit"], s_out["count"], s_out["token"], v_out["accepted_len"], v_out["out_token"]]
    h_out = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in outs]
    h2d = sum(t.numel() * t.element_size() for t in h.values())
    d2h = sum(t.numel() * t.element_size() for t in outs)

    def step():
        for name in ("zq", "ud"):
            d[name].copy_(h[name], non_blocking=True)
        tslt.sparsify(d["zq"], k, top_p, T, d["ud"], out=s_out, ws=ws_s)
        for name in ("zp", "ua", "us"):
            d[name].copy_(h[name], non_blocking=True)
        tslt.verify(d["zp"], s_out["idx"], s_out["logit"], s_out["count"], s_out["token"], T, T, d["ua"], d["us"],
                    out=v_out, ws=ws_v)
        for src, dst in zip(outs, h_out):
            dst.copy_(src, non_blocking=True)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    del h, d
    return e0.elapsed_time(e1) / 1e3 / steps, h2d, d2h


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--extras", action="store_true", help="also time the k / top-p sweep and the other configs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--batch", type=int, default=0,
                    help="override B (a smaller case of the same kernels, for profiler captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libtslt has no CPU path")
    from paper_2512_16273_b200 import tslt  # raises if libtslt.so is missing

    rank, local, world = dist_setup(args.gpus)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    w = WORKLOAD
    k, top_p, T = w["k"], w["top_p"], w["temperature"]
    B, gamma, V = (args.batch or w["B"]), w["gamma"], w["V"]
    zq, zp, ud, ua, us = make_inputs(dev, seed=rank, B=B)
    rows_step = B * gamma + B * (gamma + 1)
    eb = 2
    sparsify_bytes = B * gamma * (V * eb + 4 + 4) + B * gamma * k * 8 + B * gamma * 4
    verify_bytes = B * (gamma + 1) * V * eb + B * gamma * k * 8 + B * gamma * 12

    # warm-up outside the clock sampler, then the timed region
    sampler = ClockSampler(local)
    torch.cuda.synchronize()
    dist_barrier(world)
    sampler.start()
    secs, sp_ms, vf_ms, s_out, v_out = time_config(tslt, zq, zp, ud, ua, us, k, top_p, T, args.steps, max(args.warmup, 3))
    torch.cuda.synchronize()
    dist_barrier(world)
    clocks = sampler.stop()
    value, secs_max = aggregate(rows_step * args.steps, secs, world, dev)

    peak, peak_kind = measured_peak_gbs()
    kernels = {"sparsify_kernel": {"ms": sp_ms, "GBps": sparsify_bytes / (sp_ms * 1e-3) / 1e9,
                                   "rows_per_s": B * gamma / (sp_ms * 1e-3), "algorithmic_bytes": sparsify_bytes},
               "verify_kernel": {"ms": vf_ms, "GBps": verify_bytes / (vf_ms * 1e-3) / 1e9,
                                 "rows_per_s": B * (gamma + 1) / (vf_ms * 1e-3), "algorithmic_bytes": verify_bytes}}
    dom = max(kernels, key=lambda n: kernels[n]["ms"])
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["GBps"], "peak": peak,
                "peak_kind": "%s copy bandwidth (MEASURED_PEAKS.json)" % peak_kind if peak_kind == "measured"
                else "fallback 6650 GB/s", "unit": "GB/s", "frac": kernels[dom]["GBps"] / peak,
                "frac_of_nominal_8000": kernels[dom]["GBps"] / 8000.0, "traffic": NCU_TRAFFIC_BYTES.get(dom),
                "kernels": kernels}

    e2e = None
    if not args.no_e2e:
        e2e_secs, h2d, d2h = run_e2e(tslt, zq, zp, ud, ua, us, k, top_p, T, steps=min(args.steps, 3), warmup=1)
        e2e_secs = reduce_max(e2e_secs, world, dev)
        e2e = {"value": rows_step * world / e2e_secs, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_secs * 1e3}

    extras = {}
    if args.extras and rank == 0:
        for kk, pp in w["sweep"]:
            _, a, b, _, _ = time_config(tslt, zq, zp, ud, ua, us, kk, pp, T, 10, 3)
            extras["k%d_p%g" % (kk, pp)] = {"sparsify_ms": a, "verify_ms": b,
                                             "sparsify_GBps": (B * gamma * V * eb) / a / 1e6,
                                             "verify_GBps": (B * (gamma + 1) * V * eb) / b / 1e6}

    payload = None
    if args.extras and rank == 0:
        # the uplink payload of this step's draft rows (Section 2.2 of the paper: entries * (b_prob + b_idx) bits)
        s_o = tslt.sparsify(zq, k, top_p, T, ud)
        fmt = tslt.PROB_BF16 if w["dtype"] == "bf16" else tslt.PROB_F32
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        for it in range(4):  # the last round is the timed one
            evs[0].record()
            pk = tslt.pack_payload(s_o["idx"], s_o["logit"], s_o["count"], V, fmt)
            evs[1].record()
            tslt.unpack_payload(pk["payload"], k, V, fmt)
            evs[2].record()
        torch.cuda.synchronize()
        words, ebits = tslt.payload_words(k, V, fmt)
        payload = {"format": "bf16" if fmt == tslt.PROB_BF16 else "f32", "entry_bits": ebits,
                   "bits_per_row": float(pk["bits"].double().mean().item()),
                   "dense_row_bits": V * (16 if fmt == tslt.PROB_BF16 else 32), "record_words": words,
                   "pack_ms": evs[0].elapsed_time(evs[1]), "unpack_ms": evs[1].elapsed_time(evs[2])}

    cpu_baseline = None
    if rank == 0 and not args.no_cpu_baseline:
        n_rows, n_seq = B * gamma, B  # the whole step: a few seconds on the host cores
        zq_rows = zq.view(-1, V)[:n_rows].cpu()
        zp_seqs = zp[:n_seq].cpu()
        val, rows, cpu_secs, cores = oracle_sample_run(zq_rows, zp_seqs, k, top_p, T, 0)
        cpu_baseline = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": "%d draft rows + %d sequences x %d target rows of the same tensors (%.1f s)"
                                  % (n_rows, n_seq, gamma + 1, cpu_secs)}
    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": secs_max * 1e3 / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "config": workload_config(B), "clocks": clocks, "roofline": roofline,
                "e2e": e2e, "cpu_baseline": cpu_baseline, "gpu_launches": 4 * args.steps}
        if extras:
            line["sweep"] = extras
        if payload:
            line["payload"] = payload
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
