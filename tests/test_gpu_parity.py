"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  Sizes span several tiles, ragged tails and split rows."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_16273_b200 import synth, tslt
from parity_utils import (compare_sparsify, compare_tree, compare_verify, oracle_sparsify_parallel,
                          oracle_tree_parallel, oracle_verify_parallel, run_sequence_case, to_gpu_rows, to_np,
                          verify_inputs)

pytestmark = pytest.mark.gpu


def small_logits(B, gamma, V, dtype, seed, sigma_t=0.5):
    return synth.sequence_logits(B, gamma, V, dtype, sigma_t, seed, "cpu")


@pytest.mark.parametrize("V", [8, 16, 100, 1000, 1001, 4099, 8192, 8200, 20011, 70001])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_sequence_small_vocab_sweep(V, dtype):
    """Tiny to mid vocabularies: single tile, ragged tails (V not a multiple of the vector
    width), several tiles, split rows."""
    B, gamma = 3, 2
    zq, zp = small_logits(B, gamma, V, dtype, seed=V)
    for k, top_p, T, ns in [(1, 1.0, 1.0, 1), (min(V, 5), 1.0, 0.7, 2), (min(V, 64), 0.9, 1.0, 1),
                            (min(V, 300), 0.95, 0.5, 3), (min(V, 1024), 1.0, 1.3, 1)]:
        run_sequence_case(zq, zp, k, top_p, T, seed=7 * V + k, num_samples=ns,
                          what="V=%d %s k=%d p=%g T=%g" % (V, dtype, k, top_p, T))


def test_k_equals_V_small():
    for V in (8, 16, 33, 1024):
        zq, zp = small_logits(2, 3, V, torch.float32, seed=100 + V)
        run_sequence_case(zq, zp, V, 1.0, 1.0, seed=V, what="k=V=%d" % V)
        run_sequence_case(zq, zp, V, 0.7, 0.8, seed=V + 1, what="k=V=%d top-p" % V)


@pytest.mark.parametrize("cfg_id", [0, 1, 2])
def test_config_full_size(cfg_id):
    """Benchmark configs 0-2 at full size, every row and sequence compared."""
    cfg = synth.CONFIGS[cfg_id]
    dt = synth.torch_dtype(cfg["dtype"])
    for seed in (0, 1):
        zq, zp = synth.sequence_logits(cfg["B"], cfg["gamma"], cfg["V"], dt, cfg["sigma_t"], seed, "cpu")
        run_sequence_case(zq, zp, cfg["k"], cfg["top_p"], cfg["temperature"], seed, what=cfg["name"])


def test_top_p_below_cap_and_second_temperature():
    """Low temperature so the nucleus cut lands below the cap (both branches of n = min(k, n*))."""
    zq, zp = small_logits(4, 4, 32000, torch.bfloat16, seed=77)
    _, _, ref_s, _ = run_sequence_case(zq, zp, 256, 0.9, 0.5, seed=5, what="top-p T=0.5")
    assert (ref_s["count"] < 256).any()
    _, _, ref_s, _ = run_sequence_case(zq, zp, 32, 0.9, 1.0, seed=6, what="top-p cap binds")
    assert (ref_s["count"] == 32).any()


def test_many_rows_take_the_two_launch_verifier():
    """At least 592 target rows (one per CTA slot of the machine): the verifier runs as a streaming
    kernel followed by a resolve kernel instead of one fused launch."""
    zq, zp = small_logits(100, 6, 4099, torch.bfloat16, seed=21)          # 700 target rows
    run_sequence_case(zq, zp, 32, 1.0, 1.0, seed=21, what="two-launch verify")
    run_sequence_case(zq, zp, 64, 0.9, 0.7, seed=22, num_samples=2, what="two-launch verify top-p")
    _, ref = run_tree_case(20, (3, 3, 3), 5000, torch.float32, 16, 1.0, 23, what="two-launch tree")  # 800 rows
    assert ref["accepted_len"].max() >= 1


def sparsify_only_case(z_cpu, k, top_p, T, seed, ns, what):
    rows, V = z_cpu.shape
    u = synth.uniforms((rows, ns), seed, synth.TID_U_DRAFT)
    ref = oracle_sparsify_parallel(z_cpu, k, top_p, T, u.numpy())
    got = tslt.sparsify(to_gpu_rows(z_cpu), k, top_p, T, u.cuda())
    torch.cuda.synchronize()
    assert tslt.workspace_status(got["workspace"]) == 0
    return compare_sparsify(got, ref, what, logits=z_cpu, uniforms=u, T=T)


def test_long_rows_in_both_forms():
    """Rows several times the benchmark's.  600 rows of 600 000 bf16 logits fill the machine, so each row
    is one streaming CTA whose tile maxima (37 KB) no longer fit one line per thread and whose groups span
    several lines; 3 rows of 3 000 000 logits are cut into 64 segments each, with thousands of groups at
    k = 1024 and groups of 2048 tiles at k = 16."""
    z = synth.draft_rows(600, 600000, torch.bfloat16, 41, "cuda").cpu()  # (drawn on the GPU: 360 M logits)
    sparsify_only_case(z, 64, 1.0, 1.0, 41, 1, "600 x 600000 k=64")
    sparsify_only_case(z, 1024, 0.95, 0.8, 42, 2, "600 x 600000 top-p cap 1024")
    del z
    z = synth.draft_rows(3, 3000000, torch.bfloat16, 43, "cuda").cpu()
    sparsify_only_case(z, 1024, 1.0, 1.0, 43, 1, "3 x 3000000 k=1024")
    sparsify_only_case(z, 16, 0.9, 1.0, 44, 3, "3 x 3000000 k=16 top-p")
    zf = synth.draft_rows(2, 1500000, torch.float32, 45, "cuda").cpu()
    sparsify_only_case(zf, 320, 1.0, 1.0, 45, 1, "2 x 1500000 fp32 k=320")


@pytest.mark.parametrize("rows", [591, 592, 593, 1184])
def test_row_counts_around_the_machine_size(rows):
    """One row fewer than the streaming kernel's CTA slots (rows cut in two), exactly as many and one more
    (one CTA per row), and two full waves."""
    z = synth.draft_rows(rows, 20011, torch.bfloat16, rows, "cpu")
    sparsify_only_case(z, 32, 0.9, 1.0, rows, 1, "rows=%d" % rows)


def test_verify_longest_rows():
    """The verifier's row limit (4 MiB per row: 2 097 152 bf16 logits, 2048 chunk partials per row) and an
    fp32 row of 586 chunks: more partials than a lane keeps in registers."""
    zq, zp = small_logits(2, 2, 2097152, torch.bfloat16, seed=51)
    run_sequence_case(zq, zp, 64, 1.0, 1.0, seed=51, what="V=2097152 bf16")
    zq, zp = small_logits(3, 3, 300000, torch.float32, seed=52)
    run_sequence_case(zq, zp, 300, 0.95, 0.9, seed=52, num_samples=2, what="V=300000 fp32")
    z = torch.zeros(1, 2, 2097160, dtype=torch.bfloat16, device="cuda")  # one vector beyond the limit
    d = tslt.sparsify(z[:, :1].reshape(1, -1), 4, 1.0, 1.0, torch.zeros(1, 1, device="cuda"))
    with pytest.raises(tslt.TsltError) as e:
        tslt.verify(z, d["idx"].view(1, 1, 4), d["logit"].view(1, 1, 4), d["count"].view(1, 1), d["token"].view(1, 1), 1.0, 1.0,
                    torch.zeros(1, 1, device="cuda"), torch.zeros(1, device="cuda"))
    assert e.value.status == tslt.ERR_UNSUPPORTED


@pytest.mark.parametrize("kk,top_p", synth.CONFIGS[4]["sweep"])
def test_config4_full_size_every_row_against_oracle(kk, top_p):
    """The benchmark workload at full size (B = 256, gamma = 8, V = 256000, bf16: 2048 draft rows and
    2304 target rows drawn on the GPU), in the launch configuration bench.py times, at every point of
    the k / top-p sweep.  The oracle (spread over the host cores) checks EVERY draft row and sequence."""
    cfg = synth.CONFIGS[4]
    B, gamma, V, T = cfg["B"], cfg["gamma"], cfg["V"], cfg["temperature"]
    zq, zp = synth.sequence_logits(B, gamma, V, torch.bfloat16, cfg["sigma_t"], 0, "cuda")
    ud = synth.uniforms((B * gamma, 1), 0, synth.TID_U_DRAFT, "cuda")
    ua = synth.uniforms((B, gamma), 0, synth.TID_U_ACCEPT, "cuda")
    us = synth.uniforms((B,), 0, synth.TID_U_SAMPLE, "cuda")
    gs = tslt.sparsify(zq, kk, top_p, T, ud)
    gv = tslt.verify(zp, gs["idx"].view(B, gamma, kk), gs["logit"].view(B, gamma, kk), gs["count"].view(B, gamma),
                     gs["token"].view(B, gamma), T, T, ua, us)
    torch.cuda.synchronize()
    assert tslt.workspace_status(gs["workspace"]) == 0 and tslt.workspace_status(gv["workspace"]) == 0
    zq_c, zp_c = zq.view(-1, V).cpu(), zp.cpu()
    ref_s = oracle_sparsify_parallel(zq_c, kk, top_p, T, ud)
    compare_sparsify(gs, ref_s, "config 4 k=%d p=%g" % (kk, top_p), logits=zq_c, uniforms=ud, T=T)
    # the verifier is compared on the GPU's own drafts (equal to the oracle's wherever the cut did not move)
    inp = verify_inputs(zp_c, {n: to_np(gs[n]) for n in ("idx", "logit", "count")}, B, gamma, kk,
                        to_np(gs["token"]).reshape(B, gamma), T, T, ua, us)
    ref_v = oracle_verify_parallel(zp_c, inp["idx"], inp["logit"], inp["count"], inp["token"], T, T, inp["ua"], inp["us"])
    compare_verify(gv, ref_v, "config 4 verify k=%d p=%g" % (kk, top_p), inputs=inp)


def tree_tokens(st, parent, ndr, B, N, device):
    """node_token [B, N] from the per-internal-node samples st [B, M, kmax] (children in ascending id)."""
    toks = torch.zeros(B, N, dtype=torch.int32, device=device)
    for n in range(N):
        if ndr[n] >= 0:
            ch = [c for c in range(N) if parent[c] == n]
            toks[:, ch] = st[:, ndr[n], :len(ch)]
    return toks


def test_tree_config3_full_batch_every_sequence():
    """Config 3 at full size (B = 16, 640 target rows), every draft row and every sequence checked."""
    cfg = synth.CONFIGS[3]
    B, V, k = cfg["B"], cfg["V"], cfg["k"]
    parent, ndr, M, depth = synth.complete_tree(cfg["expansion"])
    N = len(parent)
    zq, zp = synth.tree_logits(B, parent, ndr, V, torch.bfloat16, cfg["sigma_t"], 5, "cuda")
    ud = synth.uniforms((B * M, 3), 5, synth.TID_U_DRAFT, "cuda")
    gs = tslt.sparsify(zq, k, 1.0, 1.0, ud)
    toks = tree_tokens(gs["token"].view(B, M, 3), parent, ndr, B, N, "cuda")
    ua = synth.uniforms((B, N), 5, synth.TID_U_ACCEPT, "cuda")
    us = synth.uniforms((B, N), 5, synth.TID_U_SAMPLE, "cuda")
    gt = tslt.tree_verify(zp, parent, ndr, toks, gs["idx"].view(B, M, k), gs["logit"].view(B, M, k),
                          gs["count"].view(B, M), 1.0, 1.0, ua, us, depth)
    torch.cuda.synchronize()
    zq_c, zp_c = zq.view(-1, V).cpu(), zp.cpu()
    ref_s = oracle_sparsify_parallel(zq_c, k, 1.0, 1.0, ud)
    compare_sparsify(gs, ref_s, "config 3 drafts", logits=zq_c, uniforms=ud, T=1.0)
    inp = dict(zp=zp_c, parent=parent, ndr=ndr, toks=to_np(toks), idx=to_np(gs["idx"]).reshape(B, M, k),
               logit=to_np(gs["logit"]).reshape(B, M, k), count=to_np(gs["count"]).reshape(B, M), Tq=1.0, Tp=1.0,
               ua=to_np(ua), us=to_np(us), depth=depth)
    ref_t = oracle_tree_parallel(zp_c, parent, ndr, inp["toks"], inp["idx"], inp["logit"], inp["count"], 1.0, 1.0,
                                 inp["ua"], inp["us"], depth)
    compare_tree(gt, ref_t, "config 3 trees", inputs=inp)
    gw = tslt.tree_verify(zp, parent, ndr, toks, gs["idx"].view(B, M, k), gs["logit"].view(B, M, k),
                          gs["count"].view(B, M), 1.0, 1.0, ua, us, depth, walk=True)
    torch.cuda.synchronize()
    compare_tree(gw, ref_t, "config 3 trees (path walk)", inputs=inp)
    for n in ("accepted_path", "accepted_len", "out_token"):
        assert torch.equal(gw[n], gt[n]), n  # the two entry points agree bit for bit


def adversarial_rows(V, dtype):
    rows = []
    asc = torch.linspace(-8, 8, V)
    rows.append(asc)                                   # ascending: every element beats the threshold
    rows.append(asc.flip(0))                           # descending
    rows.append(torch.zeros(V))                        # all equal: ties everywhere
    t = torch.zeros(V); t[::7] = 1.0; rows.append(t)   # two values, heavy ties at the cut
    g = torch.Generator().manual_seed(3)
    r = torch.randn(V, generator=g); r[torch.rand(V, generator=g) < 0.3] = -float("inf"); rows.append(r)
    rows.append(torch.full((V,), -float("inf")))       # no finite logit at all
    r2 = torch.full((V,), -float("inf")); r2[V // 2] = 1.5; r2[5] = 0.5; rows.append(r2)  # fewer finite than k
    r3 = torch.randn(V, generator=g) * 30; rows.append(r3)  # wide dynamic range
    r4 = torch.randn(V, generator=g); r4[::3] = -0.0; r4[1::3] = 0.0; rows.append(r4)   # signed zeros
    # a few hundred equal maxima over a low background: more tied candidates than the small finish
    # kernel lists (400), and more tiles holding one than it lists (700)
    for n_top in (400, 700):
        r5 = torch.randn(V, generator=g) * 0.01 - 10.0
        r5[::max(1, V // n_top)] = 3.0
        rows.append(r5)
    # a run of 800 adjacent equal maxima: few vectors, more tied candidates than the finish kernel lists
    r6 = torch.randn(V, generator=g) * 0.01 - 10.0
    r6[V // 8: V // 8 + min(800, V // 2)] = 3.0
    rows.append(r6)
    # large offsets: thousands of logits crowd the threshold's histogram bin (bins are relative to
    # the logit's magnitude), so these rows leave the fast paths
    rows.append(torch.randn(V, generator=g) + 20.0)
    rows.append(torch.randn(V, generator=g) * 0.5 - 30.0)
    # the row's first 16 KB say nothing about the rest (masked to a large negative finite value):
    # the offset taken from them is useless and the bins are coarse again
    r7 = torch.randn(V, generator=g)
    r7[:min(V // 2, 8192)] = -1000.0
    rows.append(r7)
    return torch.stack(rows).to(dtype)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V", [1000, 40000])
def test_sparsify_adversarial_rows(V, dtype):
    z = adversarial_rows(V, dtype)
    rows = z.shape[0]
    # k = 80 / 96 run the 96-thread finish kernel, 128 the 128-thread one, 200 / 256 the 256-thread one,
    # 64 and below the 64-thread one, 257 and above the generic one
    for k, top_p in [(1, 1.0), (7, 1.0), (64, 1.0), (80, 1.0), (96, 0.95), (128, 1.0), (200, 1.0), (256, 0.95),
                     (257, 1.0), (1000, 1.0), (128, 0.9)]:
        u = synth.uniforms((rows, 2), k, synth.TID_U_DRAFT)
        ref = oracle.sparsify(z, k, top_p, 1.0, u.numpy())
        gpu = tslt.sparsify(z.cuda(), k, top_p, 1.0, u.cuda())
        torch.cuda.synchronize()
        assert tslt.workspace_status(gpu["workspace"]) == 0
        compare_sparsify(gpu, ref, "adversarial V=%d k=%d p=%g" % (V, k, top_p), logits=z, uniforms=u, T=1.0)


def test_verify_edge_tokens_and_uniforms():
    """u = 0, u just below 1 and u >= 1 (clamped) for every decision; draft token outside the
    transmitted set; target row with -inf at the drafted token."""
    B, gamma, V, k = 6, 3, 5000, 16
    zq, zp = small_logits(B, gamma, V, torch.bfloat16, seed=9)
    ud = synth.uniforms((B * gamma, 1), 1, synth.TID_U_DRAFT)
    ref_s = oracle.sparsify(zq.reshape(-1, V), k, 1.0, 1.0, ud.numpy())
    tok = ref_s["token"][:, 0].reshape(B, gamma).copy()
    tok[1, 0] = int(np.setdiff1d(np.arange(V), ref_s["idx"][gamma * 1])[0])  # not in S
    zp = zp.clone()
    zp[2, 0, tok[2, 0]] = -float("inf")                                      # p(x) = 0: never accepted
    one_m = float(np.nextafter(np.float32(1), np.float32(0)))
    ua = torch.tensor([[0.0] * gamma, [0.5] * gamma, [0.0] * gamma, [one_m] * gamma, [1.0] * gamma,
                       [0.0, 0.0, 3.0]], dtype=torch.float32)
    for us_val in (0.0, one_m, 1.0, 0.37):
        us = torch.full((B,), us_val, dtype=torch.float32)
        ref = oracle.verify(zp, ref_s["idx"].reshape(B, gamma, k), ref_s["logit"].reshape(B, gamma, k),
                            ref_s["count"].reshape(B, gamma), tok, 1.0, 1.0, ua.numpy(), us.numpy())
        gpu = tslt.verify(zp.cuda(), torch.from_numpy(ref_s["idx"]).cuda().view(B, gamma, k),
                          torch.from_numpy(ref_s["logit"]).cuda().view(B, gamma, k),
                          torch.from_numpy(ref_s["count"]).cuda().view(B, gamma),
                          torch.from_numpy(tok).cuda(), 1.0, 1.0, ua.cuda(), us.cuda())
        torch.cuda.synchronize()
        inp = verify_inputs(zp, ref_s, B, gamma, k, tok, 1.0, 1.0, ua, us)
        compare_verify(gpu, ref, "edge us=%g" % us_val, inputs=inp)
    assert ref["accepted_len"][2] == 0 and ref["accept_prob"][2, 0] == 0.0


def test_degenerate_residual_takes_the_same_fallback():
    """p = q~ on S and -inf elsewhere, drafted token outside S: the rejection leaves no residual mass.
    The oracle then samples the unmodified p (flag DEGEN); the kernel must land on the same token."""
    V, k, B = 5000, 3, 4
    S = np.array([11, 2047, 4999], np.int32)
    lg = np.array([0.5, 1.25, -0.75], np.float32)
    zp = torch.full((B, 2, V), -float("inf"))
    zp[:, 0, torch.from_numpy(S.astype(np.int64))] = torch.from_numpy(lg)
    zp[:, 1] = torch.randn(V, generator=torch.Generator().manual_seed(1))
    idx = np.tile(S, (B, 1, 1)); logit = np.tile(lg, (B, 1, 1)); count = np.full((B, 1), k, np.int32)
    tok = np.full((B, 1), 7, np.int32)  # not in S, target logit -inf
    ua = np.zeros((B, 1), np.float32)
    us = np.array([0.0, 0.3, 0.55, 0.999], np.float32)
    ref = oracle.verify(zp, idx, logit, count, tok, 1.0, 1.0, ua, us)
    assert (ref["flags"] & oracle.FLAG_DEGEN).all() and (ref["accepted_len"] == 0).all()
    gpu = tslt.verify(zp.cuda(), torch.from_numpy(idx).cuda(), torch.from_numpy(logit).cuda(), torch.from_numpy(count).cuda(),
                      torch.from_numpy(tok).cuda(), 1.0, 1.0, torch.from_numpy(ua).cuda(), torch.from_numpy(us).cuda())
    torch.cuda.synchronize()
    inp = dict(zp=zp, idx=idx, logit=logit, count=count, token=tok, Tq=1.0, Tp=1.0, ua=ua, us=us)
    compare_verify(gpu, ref, "degenerate residual", inputs=inp)
    assert np.array_equal(to_np(gpu["out_token"]), ref["out_token"])


def test_identical_models_accept_everything():
    B, gamma, V = 4, 5, 30000
    zq, _ = small_logits(B, gamma, V, torch.bfloat16, seed=12)
    zp = torch.cat([zq, zq[:, :1]], dim=1).contiguous()
    _, _, _, ref_v = run_sequence_case(zq, zp, 1024, 1.0, 1.0, seed=3, what="identical")
    # with k < V the truncated q~ exceeds p on S, so acceptance is p/q~ = rho < 1: not all accepted,
    # but beta^ equals the retained mass
    zq2, _ = small_logits(2, 2, 512, torch.float32, seed=13)
    zp2 = torch.cat([zq2, zq2[:, :1]], dim=1).contiguous()
    _, _, ref_s, ref_v = run_sequence_case(zq2, zp2, 512, 1.0, 1.0, seed=4, what="identical k=V")
    assert (ref_v["accepted_len"] == 2).all()


@pytest.mark.parametrize("offset,T", [(300.0, 1.0), (1000.0, 1.0), (-700.0, 1.0), (0.0, 0.3), (300.0, 0.3)])
def test_large_common_offsets_and_low_temperature(offset, T):
    """fp32 rows shifted by a large common offset, and a low temperature: the offset must cancel in
    every probability (the streaming pass and the per-token exponent use one and the same scale)."""
    B, gamma, V, k = 4, 3, 20011, 48
    zq, zp = synth.sequence_logits(B, gamma, V, torch.float32, 0.5, 31, "cpu")
    run_sequence_case(zq + offset, zp + offset, k, 1.0, T, seed=int(abs(offset)) + 3, what="offset %g T=%g" % (offset, T))
    run_sequence_case(zq + offset, zp + offset, 256, 0.9, T, seed=int(abs(offset)) + 4, what="offset %g T=%g top-p" % (offset, T))


def test_ready_wait_fall_back_sets_the_status_word_and_changes_nothing():
    """With a poll limit of 0 every finish CTA of tslt_sparsify gives up on its row's ready flags at
    once, records that in the status word and waits for the end of the streaming kernel instead:
    same outputs, status word non-zero (reported as TSLT_ERR_DEVICE_STATUS).  Nothing is left
    waiting: the fall-back is an ordinary kernel-boundary wait."""
    B, gamma, V, k = 40, 4, 32000, 64
    zq, _ = synth.sequence_logits(B, gamma, V, torch.bfloat16, 0.5, 17, "cuda")
    u = synth.uniforms((B * gamma, 1), 17, synth.TID_U_DRAFT, "cuda")
    ref = tslt.sparsify(zq, k, 0.95, 1.0, u)
    torch.cuda.synchronize()
    assert tslt.workspace_status(ref["workspace"]) == 0
    ws = torch.empty(tslt.sparsify_workspace_bytes(B * gamma, V, k, 1), dtype=torch.uint8, device="cuda")
    try:
        tslt.set_ready_poll_limit(0)
        got = tslt.sparsify(zq, k, 0.95, 1.0, u, ws=ws)
        torch.cuda.synchronize()
    finally:
        tslt.set_ready_poll_limit(1 << 22)
    assert tslt.workspace_status(ws) & tslt.STATUS_WAIT_FELL_BACK
    rc = tslt.lib().tslt_workspace_status(ws.data_ptr(), None, None)
    assert rc == tslt.ERR_DEVICE_STATUS
    for n in ("idx", "logit", "count", "token", "lse", "mass"):
        assert to_np(got[n]).tobytes() == to_np(ref[n]).tobytes(), n
    # the next ordinary call on the same workspace clears the word again
    tslt.sparsify(zq, k, 0.95, 1.0, u, ws=ws)
    torch.cuda.synchronize()
    assert tslt.workspace_status(ws) == 0


def test_strided_rows_and_zero_rows():
    V, k = 3000, 32
    stride = 3008  # multiple of 8 elements: rows stay 16-byte aligned
    buf = torch.randn(5, stride).to(torch.bfloat16)
    z = buf[:, :V]
    u = synth.uniforms((5, 1), 2, synth.TID_U_DRAFT)
    ref = oracle.sparsify(z.contiguous(), k, 1.0, 1.0, u.numpy())
    gpu = tslt.sparsify(buf.cuda()[:, :V], k, 1.0, 1.0, u.cuda())
    torch.cuda.synchronize()
    compare_sparsify(gpu, ref, "strided", logits=z.contiguous(), uniforms=u, T=1.0)
    empty = tslt.sparsify(torch.empty(0, V, dtype=torch.bfloat16, device="cuda"), k, 1.0, 1.0,
                          torch.empty(0, 1, device="cuda"))
    assert empty["idx"].shape == (0, k)


def test_determinism_and_canaries():
    """Same inputs twice give identical bytes; nothing is written outside the output buffers."""
    cfg = synth.CONFIGS[1]
    zq, zp = synth.sequence_logits(cfg["B"], cfg["gamma"], cfg["V"], torch.bfloat16, 0.5, 3, "cpu")
    B, gamma, V, k = cfg["B"], cfg["gamma"], cfg["V"], cfg["k"]
    rows = B * gamma
    u = synth.uniforms((rows, 2), 3, synth.TID_U_DRAFT).cuda()
    zq_d = zq.cuda()
    pad = 64
    CAN_I, CAN_F = -123456789, -1234.5

    def padded(n, dtype, val):
        t = torch.full((n + 2 * pad,), val, dtype=dtype, device="cuda")
        return t, t[pad:pad + n]

    outs = []
    for _ in range(2):
        bufs = {}
        o = {}
        for name, n, dt, val in (("idx", rows * k, torch.int32, CAN_I), ("logit", rows * k, torch.float32, CAN_F),
                                 ("count", rows, torch.int32, CAN_I), ("token", rows * 2, torch.int32, CAN_I),
                                 ("lse", rows, torch.float32, CAN_F), ("mass", rows, torch.float32, CAN_F)):
            bufs[name], o[name] = padded(n, dt, val)
        o["idx"] = o["idx"].view(rows, k); o["logit"] = o["logit"].view(rows, k); o["token"] = o["token"].view(rows, 2)
        tslt.sparsify(zq_d, k, cfg["top_p"], cfg["temperature"], u, out=o)
        torch.cuda.synchronize()
        for name, full in bufs.items():
            val = CAN_I if full.dtype == torch.int32 else CAN_F
            assert (full[:pad] == val).all() and (full[-pad:] == val).all(), name
        outs.append({n: to_np(o[n]).copy() for n in ("idx", "logit", "count", "token", "lse", "mass")})
    for n in outs[0]:
        assert outs[0][n].tobytes() == outs[1][n].tobytes(), n


def test_back_to_back_calls_reuse_workspace_and_outputs():
    """A serving loop calls the two entry points again and again on the same workspace and the
    same output buffers, with nothing in between.  Eight such steps on a batch of more rows than
    the machine holds at once (the small finish kernel and the two-launch verifier) must give the
    first step's bytes every time and leave both status words at zero."""
    B, gamma, V, k = 80, 8, 32000, 64
    zq, zp = synth.sequence_logits(B, gamma, V, torch.bfloat16, 0.5, 21, "cuda")
    rows = B * gamma
    ud = synth.uniforms((rows, 1), 21, synth.TID_U_DRAFT, "cuda")
    ua = synth.uniforms((B, gamma), 21, synth.TID_U_ACCEPT, "cuda")
    us = synth.uniforms((B,), 21, synth.TID_U_SAMPLE, "cuda")
    ws_s = torch.empty(tslt.sparsify_workspace_bytes(rows, V, k, 1), dtype=torch.uint8, device="cuda")
    ws_v = torch.empty(tslt.verify_workspace_bytes(B, gamma, V, k), dtype=torch.uint8, device="cuda")
    s = tslt.sparsify(zq, k, 1.0, 1.0, ud, ws=ws_s)
    v = tslt.verify(zp, s["idx"], s["logit"], s["count"], s["token"], 1.0, 1.0, ua, us, ws=ws_v)
    torch.cuda.synchronize()
    first = {n: to_np(s[n]).copy() for n in ("idx", "logit", "count", "token", "lse", "mass")}
    first.update({n: to_np(v[n]).copy() for n in ("accepted_len", "out_token")})
    for _ in range(8):
        tslt.sparsify(zq, k, 1.0, 1.0, ud, out=s, ws=ws_s)
        tslt.verify(zp, s["idx"], s["logit"], s["count"], s["token"], 1.0, 1.0, ua, us, out=v, ws=ws_v)
    torch.cuda.synchronize()
    assert tslt.workspace_status(ws_s) == 0 and tslt.workspace_status(ws_v) == 0
    for n in ("idx", "logit", "count", "token", "lse", "mass"):
        assert to_np(s[n]).tobytes() == first[n].tobytes(), n
    for n in ("accepted_len", "out_token"):
        assert to_np(v[n]).tobytes() == first[n].tobytes(), n


def run_tree_case(B, expansion, V, dtype, k, T, seed, sigma_t=0.5, what=""):
    parent, ndr, M, depth = synth.complete_tree(expansion)
    N = len(parent)
    zq, zp = synth.tree_logits(B, parent, ndr, V, dtype, sigma_t, seed, "cpu")
    kmax = max(expansion)
    ud = synth.uniforms((B * M, kmax), seed, synth.TID_U_DRAFT)
    ref_s = oracle.sparsify(zq.reshape(B * M, V), k, 1.0, T, ud.numpy())
    gpu_s = tslt.sparsify(to_gpu_rows(zq), k, 1.0, T, ud.cuda())
    torch.cuda.synchronize()
    compare_sparsify(gpu_s, ref_s, what + " tree sparsify", logits=zq.reshape(B * M, V), uniforms=ud, T=T)
    toks = np.zeros((B, N), np.int32)
    for n in range(N):
        if ndr[n] >= 0:
            ch = [c for c in range(N) if parent[c] == n]
            for b in range(B):
                toks[b, ch] = ref_s["token"][b * M + ndr[n], :len(ch)]
    ua = synth.uniforms((B, N), seed, synth.TID_U_ACCEPT)
    us = synth.uniforms((B, N), seed, synth.TID_U_SAMPLE)
    ref = oracle.tree_verify(zp, parent, ndr, toks, ref_s["idx"].reshape(B, M, k), ref_s["logit"].reshape(B, M, k),
                             ref_s["count"].reshape(B, M), T, T, ua.numpy(), us.numpy(), depth)
    gpu = tslt.tree_verify(to_gpu_rows(zp), parent, ndr, torch.from_numpy(toks).cuda(),
                           torch.from_numpy(ref_s["idx"]).cuda().view(B, M, k),
                           torch.from_numpy(ref_s["logit"]).cuda().view(B, M, k),
                           torch.from_numpy(ref_s["count"]).cuda().view(B, M), T, T, ua.cuda(), us.cuda(), depth)
    torch.cuda.synchronize()
    assert tslt.workspace_status(gpu["workspace"]) == 0
    inp = dict(zp=zp, parent=parent, ndr=ndr, toks=toks, idx=ref_s["idx"].reshape(B, M, k),
               logit=ref_s["logit"].reshape(B, M, k), count=ref_s["count"].reshape(B, M), Tq=T, Tp=T,
               ua=ua.numpy(), us=us.numpy(), depth=depth)
    # the path walk (only the rows on each sequence's path are read) must give the same outputs
    walk = tslt.tree_verify(to_gpu_rows(zp), parent, ndr, torch.from_numpy(toks).cuda(),
                            torch.from_numpy(ref_s["idx"]).cuda().view(B, M, k),
                            torch.from_numpy(ref_s["logit"]).cuda().view(B, M, k),
                            torch.from_numpy(ref_s["count"]).cuda().view(B, M), T, T, ua.cuda(), us.cuda(), depth,
                            walk=True, ws=torch.empty(tslt.tree_verify_walk_workspace_bytes(B, N, V, k) + 256,
                                                      dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    assert tslt.workspace_status(walk["workspace"]) == 0
    compare_tree(walk, ref, what + " (path walk)", inputs=inp)
    return compare_tree(gpu, ref, what, inputs=inp), ref


@pytest.mark.parametrize("expansion,V,dtype,k", [((2, 2, 2), 32000, torch.bfloat16, 64),
                                                  ((3,), 1000, torch.float32, 8),
                                                  ((1, 1, 1, 1), 5000, torch.bfloat16, 16),
                                                  ((4, 2), 20011, torch.float32, 300),
                                                  ((2, 3), 16, torch.float32, 4)])
def test_tree_small(expansion, V, dtype, k):
    lens = []
    for seed in range(3):
        _, ref = run_tree_case(6, expansion, V, dtype, k, 1.0, seed, what="tree %s V=%d" % (expansion, V))
        lens.append(ref["accepted_len"])
    assert np.concatenate(lens).max() >= 1  # some child is accepted somewhere


def test_tree_config3_reduced_batch():
    cfg = synth.CONFIGS[3]
    run_tree_case(4, cfg["expansion"], cfg["V"], torch.bfloat16, cfg["k"], 1.0, 0, what=cfg["name"])


def test_tree_duplicate_children_and_single_node():
    """Identical sibling tokens (drawn with replacement) and the degenerate root-only tree."""
    V, k, B = 2000, 4, 5
    parent, ndr, M, depth = synth.complete_tree((3,))
    N = len(parent)
    zq, zp = synth.tree_logits(B, parent, ndr, V, torch.float32, 0.5, 4, "cpu")
    ref_s = oracle.sparsify(zq.reshape(B * M, V), k, 1.0, 1.0, np.zeros((B * M, 1), np.float32))
    toks = np.zeros((B, N), np.int32)
    toks[:, 1:] = ref_s["token"][:, :1]  # all three children carry the same token
    one_m = float(np.nextafter(np.float32(1), np.float32(0)))
    ua = torch.full((B, N), one_m)
    us = synth.uniforms((B, N), 4, synth.TID_U_SAMPLE)
    ref = oracle.tree_verify(zp, parent, ndr, toks, ref_s["idx"].reshape(B, M, k), ref_s["logit"].reshape(B, M, k),
                             ref_s["count"].reshape(B, M), 1.0, 1.0, ua.numpy(), us.numpy(), depth)
    gpu = tslt.tree_verify(zp.cuda(), parent, ndr, torch.from_numpy(toks).cuda(),
                           torch.from_numpy(ref_s["idx"]).cuda().view(B, M, k),
                           torch.from_numpy(ref_s["logit"]).cuda().view(B, M, k),
                           torch.from_numpy(ref_s["count"]).cuda().view(B, M), 1.0, 1.0, ua.cuda(), us.cuda(), depth)
    torch.cuda.synchronize()
    inp = dict(zp=zp, parent=parent, ndr=ndr, toks=toks, idx=ref_s["idx"].reshape(B, M, k),
               logit=ref_s["logit"].reshape(B, M, k), count=ref_s["count"].reshape(B, M), Tq=1.0, Tp=1.0,
               ua=ua.numpy(), us=us.numpy(), depth=depth)
    compare_tree(gpu, ref, "duplicates", inputs=inp)
    gw = tslt.tree_verify(zp.cuda(), parent, ndr, torch.from_numpy(toks).cuda(),
                          torch.from_numpy(ref_s["idx"]).cuda().view(B, M, k),
                          torch.from_numpy(ref_s["logit"]).cuda().view(B, M, k),
                          torch.from_numpy(ref_s["count"]).cuda().view(B, M), 1.0, 1.0, ua.cuda(), us.cuda(), depth, walk=True)
    torch.cuda.synchronize()
    compare_tree(gw, ref, "duplicates (path walk)", inputs=inp)
    # root only: the "tree" is a leaf, the token is a plain sample of the root row
    z1 = zp[:, :1].contiguous()
    ref = oracle.tree_verify(z1, [-1], [-1], np.zeros((B, 1), np.int32), np.zeros((B, 0, 1), np.int32),
                             np.zeros((B, 0, 1), np.float32), np.zeros((B, 0), np.int32), 1.0, 1.0,
                             np.zeros((B, 1), np.float32), us[:, :1].numpy(), 0)
    e_i = torch.empty(0, dtype=torch.int32, device="cuda")
    gpu = tslt.tree_verify(z1.cuda(), [-1], [-1], torch.zeros(B, 1, dtype=torch.int32, device="cuda"), e_i,
                           torch.empty(0, device="cuda"), e_i, 1.0, 1.0, torch.zeros(B, 1, device="cuda"),
                           us[:, :1].contiguous().cuda(), 0)
    torch.cuda.synchronize()
    gw = tslt.tree_verify(z1.cuda(), [-1], [-1], torch.zeros(B, 1, dtype=torch.int32, device="cuda"), e_i,
                          torch.empty(0, device="cuda"), e_i, 1.0, 1.0, torch.zeros(B, 1, device="cuda"),
                          us[:, :1].contiguous().cuda(), 0, walk=True)
    torch.cuda.synchronize()
    assert torch.equal(gw["out_token"], gpu["out_token"]) and (to_np(gw["accepted_len"]) == 0).all()
    assert (to_np(gpu["accepted_len"]) == 0).all()
    inp = dict(zp=z1, parent=[-1], ndr=[-1], toks=np.zeros((B, 1), np.int32), idx=np.zeros((B, 0, 1), np.int32),
               logit=np.zeros((B, 0, 1), np.float32), count=np.zeros((B, 0), np.int32), Tq=1.0, Tp=1.0,
               ua=np.zeros((B, 1), np.float32), us=us[:, :1].numpy(), depth=0)
    compare_tree(gpu, ref, "root only", inputs=inp)


def test_argument_errors_leave_outputs_untouched():
    V, k = 1000, 8
    z = torch.randn(2, V, device="cuda")
    u = torch.rand(2, 1, device="cuda")
    out = tslt.sparsify(z, k, 1.0, 1.0, u)
    torch.cuda.synchronize()
    snapshot = out["idx"].clone()
    for kwargs in (dict(k=0), dict(k=V + 1), dict(top_p=0.0), dict(temperature=0.0), dict(temperature=float("nan")),
                   dict(k=2000)):
        args = dict(k=k, top_p=1.0, temperature=1.0)
        args.update(kwargs)
        o2 = {n: out[n] for n in ("idx", "logit", "count", "token", "lse", "mass")}
        if args["k"] != k:
            o2 = None
        with pytest.raises((tslt.TsltError, ValueError, RuntimeError)):
            tslt.sparsify(z if args["k"] <= V + 1 else torch.randn(2, 4000, device="cuda"), args["k"], args["top_p"],
                          args["temperature"], u, out=o2)
    torch.cuda.synchronize()
    assert torch.equal(out["idx"], snapshot)
    # misaligned base pointer
    zb = torch.randn(2 * V + 8, device="cuda")[1:1 + 2 * V].view(2, V)
    with pytest.raises(tslt.TsltError):
        tslt.sparsify(zb, k, 1.0, 1.0, u)
    # workspace too small
    with pytest.raises(tslt.TsltError):
        tslt.sparsify(z, k, 1.0, 1.0, u, ws=torch.empty(256, dtype=torch.uint8, device="cuda"))
    # bad tree: parent not before child
    with pytest.raises(tslt.TsltError):
        tslt.tree_verify(torch.randn(1, 3, V, device="cuda"), [-1, 2, 0], [0, 1, -1],
                         torch.zeros(1, 3, dtype=torch.int32, device="cuda"),
                         torch.zeros(1, 2, k, dtype=torch.int32, device="cuda"), torch.zeros(1, 2, k, device="cuda"),
                         torch.zeros(1, 2, dtype=torch.int32, device="cuda"), 1.0, 1.0,
                         torch.zeros(1, 3, device="cuda"), torch.zeros(1, 3, device="cuda"), 2)
