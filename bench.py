#!/usr/bin/env python
"""Benchmark of the TSLT hot path on B200.  One pass of the hot path = tslt_sparsify over all draft rows
plus tslt_verify over all target rows of the throughput workload (B=256, gamma=8, V=256000, bf16,
top-k 64, temperature 1), with the logits resident in HBM.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

* value        rows/s over the whole job (draft rows + target rows per pass, all ranks), timed with
               CUDA events on the launching stream, max over ranks.  A counted step is
               `config.passes_per_step` passes back to back, chosen so that the timed region lasts
               about a second whatever --steps is (the clock sampler then sees sustained clocks).
* roofline     the slower entry point's achieved HBM GB/s (algorithmic bytes per call over its mean
               event-timed duration inside the timed region) against the measured copy bandwidth in
               MEASURED_PEAKS.json, and against the nominal 8000 GB/s; `kernels` lists every entry
               point, tslt_tree_verify and its path walk (config 3) included.
* sweep        (1 GPU) the five (k, top_p) points of the throughput workload, each entry point timed.
* configs      (1 GPU) the four small configurations, every entry point timed on its own, L2-cold:
               the inputs rotate over copies that total at least four times the L2.
* e2e          the same pass driven from pinned HOST buffers: H2D of the logits and uniforms and D2H
               of the sparse payload and the verdicts are inside the timed region.
* cpu_baseline the CPU oracle, as it stands, on the same tensors over the host cores (rank 0); its
               outputs are also compared with the timed pass's (`parity`).
* --impl reference   times the oracle alone on the host cores (there is no reference implementation
               of this path to install; the oracle stands in for it).
With N > 1 every rank runs the same per-GPU workload on its own GPU (rows and sequences are
independent: weak scaling, no data-path collective); only timing is reduced.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
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
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126 * 1024 * 1024
TIMED_REGION_SECONDS = 1.0


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def kernel_source_digest() -> str:
    """Digest of the CUDA sources: DRAM traffic figures taken from a profiler capture are only quoted
    while the kernels are the ones that were captured."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2512_16273_b200", "csrc")
    for name in ("tslt_common.cuh", "tslt_rowmath.cuh", "tslt_payload.cuh", "tslt_sparsify.cu", "tslt_verify.cu"):  # the timed kernels
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def captured_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of each entry point's streaming kernel
    on the bench workload, from profiles/traffic.json (written with the ncu capture); {} if there is
    no capture of the current kernels."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            t = json.load(f)
    except Exception:
        return {}
    if t.get("kernel_source_digest") != kernel_source_digest():
        return {}
    return {k: v.get("bytes_per_bench_launch") for k, v in t.get("kernels", {}).items()}


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


# ---- the CPU oracle legs --------------------------------------------------------------------
def oracle_run(zq_rows, zp_seqs, k, top_p, T, ud, ua, us):
    """The oracle on draft rows [n, V] and target sequences [m, gamma+1, V] (CPU tensors, n = m * gamma),
    spread over the host cores with one task per row / sequence (ctypes releases the GIL).  The
    verifier consumes the oracle's own drafts.  Returns (rows/s, rows, seconds, threads used, outputs)."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    cores = len(os.sched_getaffinity(0))
    n, V = zq_rows.shape
    m, g1, _ = zp_seqs.shape
    gamma = g1 - 1
    zq_np, _ = oracle.as_logits(zq_rows)
    zp_np, _ = oracle.as_logits(zp_seqs)
    oracle.lib()
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=cores) as ex:
        parts = list(ex.map(lambda r: oracle.sparsify(zq_np[r:r + 1], k, top_p, T, ud[r:r + 1]), range(n)))
    t1 = time.perf_counter()
    sp = {key: np.concatenate([p[key] for p in parts]) for key in ("idx", "logit", "count", "token", "flags")}
    di = sp["idx"][:m * gamma].reshape(m, gamma, k)
    dl = sp["logit"][:m * gamma].reshape(m, gamma, k)
    dc = sp["count"][:m * gamma].reshape(m, gamma)
    tk = np.ascontiguousarray(sp["token"][:m * gamma, 0].reshape(m, gamma))
    t2 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=cores) as ex:
        vparts = list(ex.map(lambda b: oracle.verify(zp_np[b:b + 1], di[b:b + 1], dl[b:b + 1], dc[b:b + 1], tk[b:b + 1],
                                                     T, T, ua[b:b + 1], us[b:b + 1]), range(m)))
    t3 = time.perf_counter()
    vf = {key: np.concatenate([p[key] for p in vparts]) for key in ("accepted_len", "out_token", "flags")}
    rows = n + m * g1
    secs = (t1 - t0) + (t3 - t2)
    return rows / secs, rows, secs, min(cores, max(n, m)), (sp, vf)


def parity_report(s_out, v_out, sp, vf):
    """The timed pass's outputs against the oracle's on the same inputs: rows / sequences the oracle does
    not flag (a decision within 1e-6 of a boundary) must agree exactly.  (The full validity check of
    flagged rows is the test suite's; this is the bench run's own sanity line.)"""
    import oracle
    idx, cnt, tok = (s_out[n].cpu().numpy() for n in ("idx", "count", "token"))
    clean = (sp["flags"] & (oracle.FLAG_SEL | oracle.FLAG_SMP)) == 0
    bad_rows = int(((cnt != sp["count"]) | (idx != sp["idx"]).any(axis=1) | (tok[:, 0] != sp["token"][:, 0]))[clean].sum())
    al, ot = v_out["accepted_len"].cpu().numpy(), v_out["out_token"].cpu().numpy()
    vclean = (vf["flags"] & (oracle.FLAG_ACC | oracle.FLAG_RES | oracle.FLAG_DEGEN)) == 0
    # the GPU verifier consumed the GPU's drafts: equal to the oracle's wherever no draft row was flagged
    gamma = al.size and idx.shape[0] // al.size
    seq_clean = vclean & clean.reshape(al.size, gamma).all(axis=1)
    bad_seqs = int(((al != vf["accepted_len"]) | (ot != vf["out_token"]))[seq_clean].sum())
    return {"status": "ok" if bad_rows == 0 and bad_seqs == 0 else "mismatch", "draft_rows_compared": int(clean.sum()),
            "draft_rows_flagged": int((~clean).sum()), "sequences_compared": int(seq_clean.sum()),
            "sequences_flagged": int((~seq_clean).sum()), "mismatches": bad_rows + bad_seqs}


def run_reference(args):
    """--impl reference: the oracle, as it stands, on a bounded sample of the workload per step: two
    draft rows and two sequences per host core, so that every core has work in both legs."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = WORKLOAD
    dt = synth.torch_dtype(w["dtype"])
    cores = len(os.sched_getaffinity(0))
    n_seq = max(2, 2 * cores // w["gamma"] + 1)  # n_seq * gamma >= 2 * cores draft rows
    n_seq = max(n_seq, 2 * cores) if cores <= 8 else n_seq
    zq, zp = synth.sequence_logits(n_seq, w["gamma"], w["V"], dt, w["sigma_t"], 0, "cpu")
    zq_rows = zq.reshape(-1, w["V"]).contiguous()
    n_rows = zq_rows.shape[0]

    def uniforms(seed):
        return (synth.uniforms((n_rows, 1), seed, synth.TID_U_DRAFT).numpy(),
                synth.uniforms((n_seq, w["gamma"]), seed, synth.TID_U_ACCEPT).numpy(),
                synth.uniforms((n_seq,), seed, synth.TID_U_SAMPLE).numpy())
    for _ in range(min(args.warmup, 1)):
        oracle_run(zq_rows[:2 * w["gamma"]], zp[:2], w["k"], w["top_p"], w["temperature"], *[u[:2 * w["gamma"]] if i == 0 else u[:2]
                                                                                             for i, u in enumerate(uniforms(0))])
    steps = max(1, min(args.steps, 8))  # bounded: each step is seconds of CPU work
    tot_rows, tot_secs, used = 0, 0.0, 1
    for s in range(steps):
        _, rows, secs, used, _ = oracle_run(zq_rows, zp, w["k"], w["top_p"], w["temperature"], *uniforms(s))
        tot_rows += rows
        tot_secs += secs
    value = tot_rows / tot_secs
    sample = ("%d draft rows + %d sequences x %d target rows of the workload per step, %d of the %d requested steps "
              "(each step is seconds of CPU work)" % (n_rows, n_seq, w["gamma"] + 1, steps, args.steps))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * tot_secs / steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(B=None, passes_per_step=1):
    w = WORKLOAD
    return {"workload": w["name"], "B": B or w["B"], "gamma": w["gamma"], "V": w["V"], "logits_dtype": w["dtype"],
            "k": w["k"], "top_p": w["top_p"], "temperature": w["temperature"], "passes_per_step": passes_per_step,
            "l2": "inputs (1.05 GB draft + 1.18 GB target logits) are larger than L2, no flush needed"}


# ---- the GPU legs ---------------------------------------------------------------------------
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


def alloc_outputs(B, gamma, k, device, ns=1):
    rows = B * gamma
    s_out = {"idx": torch.empty(rows, k, dtype=torch.int32, device=device),
             "logit": torch.empty(rows, k, dtype=torch.float32, device=device),
             "count": torch.empty(rows, dtype=torch.int32, device=device),
             "token": torch.empty(rows, ns, dtype=torch.int32, device=device),
             "lse": torch.empty(rows, dtype=torch.float32, device=device),
             "mass": torch.empty(rows, dtype=torch.float32, device=device)}
    v_out = {"accepted_len": torch.empty(B, dtype=torch.int32, device=device),
             "out_token": torch.empty(B, dtype=torch.int32, device=device)}
    return s_out, v_out


def sparsify_bytes(rows, V, eb, k, ns=1):
    """Algorithmic bytes of one tslt_sparsify call: the logits once, one uniform per sample, the k
    (index, logit) pairs, count and tokens."""
    return rows * (V * eb + 4 * ns + 4) + rows * k * 8 + rows * 4 * ns


def verify_bytes(seqs, rows_per_seq, draft_rows, V, eb, k):
    """Algorithmic bytes of one verifier call: every target row once, the sparse drafts, the scalars."""
    return seqs * rows_per_seq * V * eb + draft_rows * k * 8 + draft_rows * 12


class Pass:
    """Buffers of one (k, top_p) point of the throughput workload and the calls of one pass over it."""

    def __init__(self, tslt, zq, zp, ud, ua, us, k, top_p, T):
        self.tslt, self.zq, self.zp, self.ud, self.ua, self.us = tslt, zq, zp, ud, ua, us
        self.k, self.top_p, self.T = k, top_p, T
        B, gamma, V = zq.shape
        dev = zq.device
        self.s_out, self.v_out = alloc_outputs(B, gamma, k, dev)
        self.ws_s = torch.empty(tslt.sparsify_workspace_bytes(B * gamma, V, k, 1), dtype=torch.uint8, device=dev)
        self.ws_v = torch.empty(tslt.verify_workspace_bytes(B, gamma, V, k), dtype=torch.uint8, device=dev)

    def sparsify(self):
        self.tslt.sparsify(self.zq, self.k, self.top_p, self.T, self.ud, out=self.s_out, ws=self.ws_s)

    def verify(self):
        s = self.s_out
        self.tslt.verify(self.zp, s["idx"], s["logit"], s["count"], s["token"], self.T, self.T, self.ua, self.us,
                         out=self.v_out, ws=self.ws_v)

    def run(self, events=None):
        if events:
            events[0].record()
        self.sparsify()
        if events:
            events[1].record()
        self.verify()
        if events:
            events[2].record()

    def status_ok(self):
        return self.tslt.workspace_status(self.ws_s) == 0 and self.tslt.workspace_status(self.ws_v) == 0


def time_passes(ps: Pass, passes: int, warmup: int):
    """Event-timed loop of `passes` passes; returns (seconds total, mean sparsify ms, mean verify ms).
    Every pass is bracketed by events on the launching stream (three records per pass)."""
    for _ in range(warmup):
        ps.run()
    torch.cuda.synchronize()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(passes)]
    for i in range(passes):
        ps.run(evs[i])
    torch.cuda.synchronize()
    total_ms = evs[0][0].elapsed_time(evs[-1][2])
    sp_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in evs)
    vf_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in evs)
    assert ps.status_ok(), "device status word set"
    return total_ms / 1e3, sp_ms, vf_ms


def run_e2e(ps: Pass, steps, warmup):
    """The same pass from pinned host buffers, copies inside the timed region."""
    tslt = ps.tslt
    ins = (("zq", ps.zq), ("zp", ps.zp), ("ud", ps.ud), ("ua", ps.ua), ("us", ps.us))
    h = {name: torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t) for name, t in ins}
    d = {name: torch.empty_like(t) for name, t in ins}
    s_out, v_out = ps.s_out, ps.v_out
    outs = [s_out["idx"], s_out["logit"], s_out["count"], s_out["token"], v_out["accepted_len"], v_out["out_token"]]
    h_out = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in outs]
    h2d = sum(t.numel() * t.element_size() for t in h.values())
    d2h = sum(t.numel() * t.element_size() for t in outs)

    def step():
        for name in ("zq", "ud"):
            d[name].copy_(h[name], non_blocking=True)
        tslt.sparsify(d["zq"], ps.k, ps.top_p, ps.T, d["ud"], out=s_out, ws=ps.ws_s)
        for name in ("zp", "ua", "us"):
            d[name].copy_(h[name], non_blocking=True)
        tslt.verify(d["zp"], s_out["idx"], s_out["logit"], s_out["count"], s_out["token"], ps.T, ps.T, d["ua"], d["us"],
                    out=v_out, ws=ps.ws_v)
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


def rotating_copies(nbytes: int) -> int:
    """Copies of an input over which calls rotate so that every call reads HBM: together at least four
    times the L2."""
    return max(2, min(4096, math.ceil(4 * L2_BYTES / max(nbytes, 1))))


def time_rotating(call, copies: int) -> float:
    """Mean microseconds per call of call(i), i the copy to read: one untimed round over all copies
    (which also leaves the oldest copies out of L2), then one timed round of at least 20 calls,
    back to back on the stream between two events."""
    for i in range(copies):
        call(i)
    torch.cuda.synchronize()
    n = max(copies, 20)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(n):
        call(i % copies)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / n


def entry(us, nbytes, rows, peak):
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"us_per_call": us, "rows_per_s": rows / (us * 1e-6), "GBps": gbs, "algorithmic_bytes": nbytes,
            "frac_of_measured": gbs / peak, "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS}


def time_small_configs(tslt, dev, peak):
    """Configurations 0 to 3, every entry point on its own, L2-cold (rotating input copies)."""
    out = {}
    for cfg in synth.CONFIGS[:4]:
        dt = synth.torch_dtype(cfg["dtype"])
        eb = 2 if cfg["dtype"] == "bf16" else 4
        V, k, T, top_p = cfg["V"], cfg["k"], cfg["temperature"], cfg["top_p"]
        res = {}
        if cfg["kind"] == "sequence":
            B, gamma = cfg["B"], cfg["gamma"]
            zq, zp = synth.sequence_logits(B, gamma, V, dt, cfg["sigma_t"], 0, dev)
            ud = synth.uniforms((B * gamma, 1), 0, synth.TID_U_DRAFT, dev)
            ua = synth.uniforms((B, gamma), 0, synth.TID_U_ACCEPT, dev)
            us = synth.uniforms((B,), 0, synth.TID_U_SAMPLE, dev)
            cq, cp = rotating_copies(zq.numel() * eb), rotating_copies(zp.numel() * eb)
            zq_all = zq.unsqueeze(0).repeat(cq, 1, 1, 1)
            zp_all = zp.unsqueeze(0).repeat(cp, 1, 1, 1)
            s_out, v_out = alloc_outputs(B, gamma, k, dev)
            ws_s = torch.empty(tslt.sparsify_workspace_bytes(B * gamma, V, k, 1), dtype=torch.uint8, device=dev)
            ws_v = torch.empty(tslt.verify_workspace_bytes(B, gamma, V, k), dtype=torch.uint8, device=dev)
            us_s = time_rotating(lambda i: tslt.sparsify(zq_all[i], k, top_p, T, ud, out=s_out, ws=ws_s), cq)
            us_v = time_rotating(lambda i: tslt.verify(zp_all[i], s_out["idx"], s_out["logit"], s_out["count"], s_out["token"],
                                                       T, T, ua, us, out=v_out, ws=ws_v), cp)
            assert tslt.workspace_status(ws_s) == 0 and tslt.workspace_status(ws_v) == 0
            res["tslt_sparsify"] = entry(us_s, sparsify_bytes(B * gamma, V, eb, k), B * gamma, peak)
            res["tslt_verify"] = entry(us_v, verify_bytes(B, gamma + 1, B * gamma, V, eb, k), B * (gamma + 1), peak)
            # the verifier on the uplink records themselves against unpacking them first (same verdicts)
            fmt = tslt.PROB_BF16 if cfg["dtype"] == "bf16" else tslt.PROB_F32
            wire = tslt.pack_payload(s_out["idx"], s_out["logit"], s_out["count"], V, fmt)["payload"]
            p_out = {n: torch.empty_like(t) for n, t in v_out.items()}
            us_p = time_rotating(lambda i: tslt.verify_packed(zp_all[i], wire, fmt, k, s_out["token"], T, T, ua, us,
                                                              out=p_out, ws=ws_v), cp)

            d = tslt.unpack_payload(wire, k, V, fmt)

            def unpack_then_verify(i):
                tslt.unpack_payload(wire, k, V, fmt, out=d)
                tslt.verify(zp_all[i], d["idx"], d["logit"], d["count"], s_out["token"], T, T, ua, us, out=v_out, ws=ws_v)
            us_u = time_rotating(unpack_then_verify, cp)
            torch.cuda.synchronize()
            assert all(torch.equal(p_out[n], v_out[n]) for n in ("accepted_len", "out_token")), "packed verifier disagrees"
            res["tslt_verify_packed"] = entry(us_p, verify_bytes(B, gamma + 1, B * gamma, V, eb, k), B * (gamma + 1), peak)
            res["tslt_unpack_payload+tslt_verify"] = entry(us_u, verify_bytes(B, gamma + 1, B * gamma, V, eb, k),
                                                           B * (gamma + 1), peak)
            res["input_copies"] = {"draft": cq, "target": cp}
            del zq_all, zp_all
        else:
            B = cfg["B"]
            parent, ndr, M, depth = synth.complete_tree(cfg["expansion"])
            N, ns = len(parent), max(cfg["expansion"])
            zq, zp = synth.tree_logits(B, parent, ndr, V, dt, cfg["sigma_t"], 0, dev)
            ud = synth.uniforms((B * M, ns), 0, synth.TID_U_DRAFT, dev)
            ua = synth.uniforms((B, N), 0, synth.TID_U_ACCEPT, dev)
            us = synth.uniforms((B, N), 0, synth.TID_U_SAMPLE, dev)
            cq, cp = rotating_copies(zq.numel() * eb), rotating_copies(zp.numel() * eb)
            zq_all = zq.unsqueeze(0).repeat(cq, 1, 1, 1)
            zp_all = zp.unsqueeze(0).repeat(cp, 1, 1, 1)
            s_out, _ = alloc_outputs(B, M, k, dev, ns=ns)
            ws_s = torch.empty(tslt.sparsify_workspace_bytes(B * M, V, k, ns), dtype=torch.uint8, device=dev)
            us_s = time_rotating(lambda i: tslt.sparsify(zq_all[i], k, top_p, T, ud, out=s_out, ws=ws_s), cq)
            st = s_out["token"].view(B, M, ns)
            toks = torch.zeros(B, N, dtype=torch.int32, device=dev)
            for n in range(N):
                if ndr[n] >= 0:
                    ch = [c for c in range(N) if parent[c] == n]
                    toks[:, ch] = st[:, ndr[n], :len(ch)]
            di, dl, dc = s_out["idx"].view(B, M, k), s_out["logit"].view(B, M, k), s_out["count"].view(B, M)
            t_out = {"accepted_path": torch.empty(B, depth, dtype=torch.int32, device=dev),
                     "accepted_len": torch.empty(B, dtype=torch.int32, device=dev),
                     "out_token": torch.empty(B, dtype=torch.int32, device=dev)}
            ws_t = torch.empty(tslt.tree_verify_workspace_bytes(B, N, V, k), dtype=torch.uint8, device=dev)
            ws_w = torch.empty(tslt.tree_verify_walk_workspace_bytes(B, N, V, k), dtype=torch.uint8, device=dev)
            us_t = time_rotating(lambda i: tslt.tree_verify(zp_all[i], parent, ndr, toks, di, dl, dc, T, T, ua, us, depth,
                                                            out=t_out, ws=ws_t), cp)
            names = ("accepted_path", "accepted_len", "out_token")
            all_nodes = {n: t_out[n].clone() for n in names}
            us_w = time_rotating(lambda i: tslt.tree_verify(zp_all[i], parent, ndr, toks, di, dl, dc, T, T, ua, us, depth,
                                                            out=t_out, ws=ws_w, walk=True), cp)
            torch.cuda.synchronize()
            differ = [n for n in names if not torch.equal(all_nodes[n], t_out[n])]
            assert not differ, ("path walk and all-nodes verifier disagree", differ)
            rows_walked = int((t_out["accepted_len"] + 1).sum().item())  # the root row and one per accepted node
            res["tslt_sparsify"] = entry(us_s, sparsify_bytes(B * M, V, eb, k, ns), B * M, peak)
            res["tslt_tree_verify"] = entry(us_t, verify_bytes(B, N, B * M, V, eb, k), B * N, peak)
            # the path walk is credited only with the rows it read: a latency figure, not a bandwidth one
            res["tslt_tree_verify_walk"] = entry(us_w, rows_walked * V * eb + rows_walked * k * 8, rows_walked, peak)
            res["tslt_tree_verify_walk"]["rows_read_of"] = [rows_walked, B * N]
            res["input_copies"] = {"draft": cq, "target": cp}
            del zq_all, zp_all
        res["l2"] = "inputs rotate over copies totalling >= 4 x L2 (126 MiB): every call reads HBM"
        out[cfg["name"]] = res
        torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the k / top-p sweep and the small configurations")
    ap.add_argument("--batch", type=int, default=0,
                    help="override B (a smaller case of the same kernels, for profiler captures)")
    ap.add_argument("--passes-per-step", type=int, default=0, help="override (default: enough for a timed region of ~1 s)")
    ap.add_argument("--k", type=int, default=0, help="override k of the timed workload (profiler captures of sweep points)")
    ap.add_argument("--top-p", type=float, default=0.0, help="override top_p of the timed workload")
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
    k, top_p, T = (args.k or w["k"]), (args.top_p or w["top_p"]), w["temperature"]
    B, gamma, V = (args.batch or w["B"]), w["gamma"], w["V"]
    zq, zp, ud, ua, us = make_inputs(dev, seed=rank, B=B)
    rows_pass = B * gamma + B * (gamma + 1)
    eb = 2
    warmup = max(args.warmup, 3)
    ps = Pass(tslt, zq, zp, ud, ua, us, k, top_p, T)
    # how many passes make a counted step: the timed region should last about a second
    est_s, _, _ = time_passes(ps, 5, warmup)
    R = args.passes_per_step or max(1, math.ceil(TIMED_REGION_SECONDS / max(args.steps, 1) / (est_s / 5)))

    sampler = ClockSampler(local)
    torch.cuda.synchronize()
    dist_barrier(world)
    sampler.start()
    secs, sp_ms, vf_ms = time_passes(ps, args.steps * R, warmup)
    torch.cuda.synchronize()
    dist_barrier(world)
    clocks = sampler.stop()
    value, secs_max = aggregate(rows_pass * args.steps * R, secs, world, dev)

    peak, peak_kind = measured_peak_gbs()
    traffic = captured_traffic()
    kernels = {"tslt_sparsify": entry(sp_ms * 1e3, sparsify_bytes(B * gamma, V, eb, k), B * gamma, peak),
               "tslt_verify": entry(vf_ms * 1e3, verify_bytes(B, gamma + 1, B * gamma, V, eb, k), B * (gamma + 1), peak)}
    dom = max(("tslt_sparsify", "tslt_verify"), key=lambda n: kernels[n]["us_per_call"])

    sweep, configs = None, None
    if world == 1 and not args.no_extras:
        sweep = {}
        for kk, pp in w["sweep"]:
            pt = ps if (kk, pp) == (k, top_p) else Pass(tslt, zq, zp, ud, ua, us, kk, pp, T)
            _, a, b = time_passes(pt, 30, 3)
            sweep["k%d_p%g" % (kk, pp)] = {"tslt_sparsify": entry(a * 1e3, sparsify_bytes(B * gamma, V, eb, kk), B * gamma, peak),
                                           "tslt_verify": entry(b * 1e3, verify_bytes(B, gamma + 1, B * gamma, V, eb, kk),
                                                                B * (gamma + 1), peak)}
            del pt
        configs = time_small_configs(tslt, dev, peak)
        t3 = configs[synth.CONFIGS[3]["name"]]
        kernels["tslt_tree_verify"] = dict(t3["tslt_tree_verify"], workload=synth.CONFIGS[3]["name"])
        kernels["tslt_tree_verify_walk"] = dict(t3["tslt_tree_verify_walk"], workload=synth.CONFIGS[3]["name"])
        ps.run()  # the headline pass's outputs again, for the parity line below
        torch.cuda.synchronize()

    roofline = {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["GBps"], "peak": peak,
                "peak_kind": "%s copy bandwidth (MEASURED_PEAKS.json)" % peak_kind if peak_kind == "measured"
                else "fallback 6650 GB/s", "unit": "GB/s", "frac": kernels[dom]["GBps"] / peak,
                "frac_of_nominal_8000": kernels[dom]["GBps"] / NOMINAL_HBM_GBS, "traffic": traffic.get(dom),
                "kernels": kernels}

    e2e = None
    if not args.no_e2e:
        e2e_secs, h2d, d2h = run_e2e(ps, steps=3, warmup=1)
        e2e_secs = reduce_max(e2e_secs, world, dev)
        e2e = {"value": rows_pass * world / e2e_secs, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_pass": e2e_secs * 1e3}
        ps.run()
        torch.cuda.synchronize()

    cpu_baseline, parity = None, None
    if rank == 0 and not args.no_cpu_baseline:
        zq_rows, zp_seqs = zq.view(-1, V).cpu(), zp.cpu()  # the whole pass: a few seconds on the host cores
        val, rows, cpu_secs, cores, (sp, vf) = oracle_run(zq_rows, zp_seqs, k, top_p, T, ud.cpu().numpy(), ua.cpu().numpy(),
                                                          us.cpu().numpy())
        cpu_baseline = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": "%d draft rows + %d sequences x %d target rows of the same tensors (%.1f s)"
                                  % (B * gamma, B, gamma + 1, cpu_secs)}
        parity = parity_report(ps.s_out, ps.v_out, sp, vf)
    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": warmup, "ms_per_step": secs_max * 1e3 / args.steps, "ms_per_pass": secs_max * 1e3 / (args.steps * R),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "config": dict(workload_config(B, R), k=k, top_p=top_p), "clocks": clocks,
                "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu_baseline, "parity": parity,
                "gpu_launches": 4 * args.steps * R}
        if sweep:
            line["sweep"] = sweep
        if configs:
            line["configs"] = configs
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
