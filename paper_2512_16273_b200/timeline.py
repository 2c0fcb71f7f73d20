"""Where the microseconds of one call go: builds the library a second time with -DTSLT_STAMPS (thread 0 of
every CTA writes %globaltimer at its phase boundaries; the ordinary build has none of this), runs
tslt_sparsify and tslt_verify on a synthetic configuration and prints the timeline and the per-phase
medians.  The stamped library is a separate file (libtslt_stamps.so); nothing else loads it.

    python -m paper_2512_16273_b200.timeline                 # config 4 (B = 256), k = 64
    python -m paper_2512_16273_b200.timeline --k 1024 --top-p 0.95
    python -m paper_2512_16273_b200.timeline --config 2      # a small batch, L2 flushed before each call
"""
from __future__ import annotations

import argparse
import ctypes
import os
import subprocess

import numpy as np
import torch

from . import build as _build
from . import synth

STAMP_CTAS, STAMP_SLOTS = 16384, 8
LIB = os.path.join(_build.HERE, "libtslt_stamps.so")


def build_stamped() -> str:
    deps = [os.path.join(_build.CSRC, f) for f in _build.SOURCES + _build.HEADERS]
    if os.path.exists(LIB) and all(os.path.getmtime(d) <= os.path.getmtime(LIB) for d in deps):
        return LIB
    cmd = [_build._nvcc()] + _build.NVCC_FLAGS + ["-DTSLT_STAMPS", "-o", LIB] + [os.path.join(_build.CSRC, f) for f in _build.SOURCES]
    subprocess.check_call(cmd)
    return LIB


def _stamps(fn) -> np.ndarray:
    a = np.zeros((STAMP_CTAS, STAMP_SLOTS), np.uint64)
    rc = fn(ctypes.c_void_p(a.ctypes.data), ctypes.c_size_t(a.nbytes))
    if rc != 0:
        raise RuntimeError("reading the stamps failed: %d" % rc)
    return a.astype(np.int64)


def _q(a):
    return "first %7.1f  median %7.1f  p90 %7.1f  last %7.1f" % (a.min(), np.median(a), np.percentile(a, 90), a.max())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--k", type=int, default=0)
    ap.add_argument("--top-p", type=float, default=0.0)
    args = ap.parse_args()
    from . import tslt
    tslt._LIB_PATH = build_stamped()  # before the first call loads the library
    L = tslt.lib()
    cfg = synth.CONFIGS[args.config]
    if cfg["kind"] != "sequence":
        raise SystemExit("sequence configurations only")
    B, g, V, T = cfg["B"], cfg["gamma"], cfg["V"], cfg["temperature"]
    k, top_p = args.k or cfg["k"], args.top_p or cfg["top_p"]
    rows = B * g
    if rows > STAMP_CTAS // 2:
        raise SystemExit("at most %d rows" % (STAMP_CTAS // 2))
    zq, zp = synth.sequence_logits(B, g, V, synth.torch_dtype(cfg["dtype"]), cfg["sigma_t"], 0, "cuda")
    ud = synth.uniforms((rows, 1), 0, synth.TID_U_DRAFT, "cuda")
    ua = synth.uniforms((B, g), 0, synth.TID_U_ACCEPT, "cuda")
    us = synth.uniforms((B,), 0, synth.TID_U_SAMPLE, "cuda")
    small = zq.numel() * zq.element_size() < (256 << 20)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if small else None
    s = tslt.sparsify(zq.reshape(rows, V), k, top_p, T, ud)
    for it in range(3):
        if flush is not None:
            flush.fill_(it)
        tslt.sparsify(zq.reshape(rows, V), k, top_p, T, ud, out=s, ws=s["workspace"])
    torch.cuda.synchronize()
    st = _stamps(L.tslt_debug_stamps_sparsify)
    sc = st[:STAMP_CTAS // 2]  # streaming CTAs (those that ran have a start stamp)
    fin = st[:rows]
    done = st[STAMP_CTAS // 2:STAMP_CTAS // 2 + rows, 0]
    t0 = sc[:, 0][sc[:, 0] > 0].min()
    us_ = lambda x: (x - t0) / 1e3
    print("tslt_sparsify  %s  k=%d top_p=%g  rows=%d  (us from the first streaming CTA's start)" % (cfg["name"], k, top_p, rows))
    live = sc[:, 0] > 0
    print("  streaming CTA starts      ", _q(us_(sc[live, 0])))
    print("  streaming loop ends       ", _q(us_(sc[live, 1])), "  loop: median %.1f" % np.median((sc[live, 1] - sc[live, 0]) / 1e3))
    print("  segment handed over       ", _q(us_(sc[live, 2])), "  end phase: median %.1f" % np.median((sc[live, 2] - sc[live, 1]) / 1e3))
    print("  finish CTA enters         ", _q(us_(fin[:, 3])))
    print("  finish CTA done           ", _q(us_(done)))
    names = ["wait for the row", "hand-over read (+ bound and list for segments)", "gather", "select", "cut + CDF + outputs"]
    ph = np.stack([fin[:, 4] - fin[:, 3], fin[:, 5] - fin[:, 4], fin[:, 6] - fin[:, 5], fin[:, 7] - fin[:, 6], done - fin[:, 7]], 1) / 1e3
    for n, col in zip(names, ph.T):
        print("    %-48s median %5.1f  p90 %5.1f" % (n, np.median(col), np.percentile(col, 90)))
    print("    finish chain: median %.1f us; rows finished before the last hand-over: %d of %d" % (
        np.median((done - fin[:, 4]) / 1e3), int((done <= sc[live, 2].max()).sum()), rows))

    tok = s["token"].view(B, g)
    v = tslt.verify(zp, s["idx"].view(B, g, k), s["logit"].view(B, g, k), s["count"].view(B, g), tok, T, T, ua, us)
    for it in range(3):
        if flush is not None:
            flush.fill_(it)
        tslt.verify(zp, s["idx"].view(B, g, k), s["logit"].view(B, g, k), s["count"].view(B, g), tok, T, T, ua, us, out=v,
                    ws=v["workspace"])
    torch.cuda.synchronize()
    sv = _stamps(L.tslt_debug_stamps_verify)[:B]
    t0 = sv[:, 0].min()
    print("tslt_verify  resolver CTAs (us from the first one's entry)")
    print("  enters                    ", _q((sv[:, 0] - t0) / 1e3))
    vn = ["wait for the streaming kernel", "positions (log-normaliser, acceptance test)", "accepted run + draft of the stop position",
          "correction token"]
    for i, n in enumerate(vn):
        col = (sv[:, i + 1] - sv[:, i]) / 1e3
        print("    %-48s median %5.1f  max %5.1f" % (n, np.median(col), col.max()))
    print("  last resolver done         %.1f" % ((sv[:, 4].max() - t0) / 1e3))


if __name__ == "__main__":
    main()
