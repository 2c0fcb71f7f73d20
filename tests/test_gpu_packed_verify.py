"""GPU parity of the verifiers that read the uplink records directly (tslt_verify_packed,
tslt_tree_verify_packed; through the C ABI): against the CPU oracle's verifier given the logits as the
wire format leaves them, and bit for bit against tslt_verify / tslt_tree_verify on the unpacked arrays."""
import numpy as np
import pytest
import torch

import oracle
from oracle import payload as P
from paper_2512_16273_b200 import synth, tslt
from parity_utils import compare_tree, compare_verify, to_gpu_rows, to_np, verify_inputs

pytestmark = pytest.mark.gpu

FORMATS = [(tslt.PROB_F32, P.PROB_F32), (tslt.PROB_BF16, P.PROB_BF16), (tslt.PROB_F16, P.PROB_F16)]


def wire(ref_s, of):
    return np.where(ref_s["idx"] >= 0, P.round_value(ref_s["logit"], of), -np.inf).astype(np.float32)


@pytest.mark.parametrize("dtype,fmt,V,k", [(torch.bfloat16, FORMATS[1], 20011, 48), (torch.float32, FORMATS[0], 4099, 17),
                                           (torch.float32, FORMATS[2], 32000, 320), (torch.bfloat16, FORMATS[1], 256000, 1024),
                                           (torch.float32, FORMATS[1], 8, 8)])
def test_verify_packed(dtype, fmt, V, k):
    gf, of = fmt
    B, gamma, T = 6, 4, 0.9
    zq, zp = synth.sequence_logits(B, gamma, V, dtype, 0.5, 21, "cpu")
    rows = B * gamma
    ud = synth.uniforms((rows, 1), 21, synth.TID_U_DRAFT)
    ua = synth.uniforms((B, gamma), 21, synth.TID_U_ACCEPT)
    us = synth.uniforms((B,), 21, synth.TID_U_SAMPLE)
    ref_s = oracle.sparsify(zq.reshape(rows, V), k, 0.97, T, ud.numpy())
    wl = wire(ref_s, of)
    rec = P.pack(ref_s["idx"], ref_s["logit"], ref_s["count"], V, of)  # the oracle's records, not the GPU's
    tok = np.ascontiguousarray(ref_s["token"][:, 0].reshape(B, gamma))
    z = to_gpu_rows(zp)
    got = tslt.verify_packed(z, torch.from_numpy(rec.view(np.int32)).cuda(), gf, k, torch.from_numpy(tok).cuda(), T, T,
                             ua.cuda(), us.cuda())
    torch.cuda.synchronize()
    assert tslt.workspace_status(got["workspace"]) == 0
    ref_v = oracle.verify(zp, ref_s["idx"].reshape(B, gamma, k), wl.reshape(B, gamma, k), ref_s["count"].reshape(B, gamma),
                          tok, T, T, ua.numpy(), us.numpy())
    inp = verify_inputs(zp, dict(idx=ref_s["idx"], logit=wl, count=ref_s["count"]), B, gamma, k, tok, T, T, ua, us)
    compare_verify(got, ref_v, "packed %s fmt %d V=%d" % (dtype, gf, V), inputs=inp)
    # the same call on the unpacked arrays: identical bits
    u = tslt.unpack_payload(torch.from_numpy(rec.view(np.int32)).cuda(), k, V, gf)
    plain = tslt.verify(z, u["idx"].view(B, gamma, k), u["logit"].view(B, gamma, k), u["count"].view(B, gamma),
                        torch.from_numpy(tok).cuda(), T, T, ua.cuda(), us.cuda())
    torch.cuda.synchronize()
    for name in ("accepted_len", "out_token", "accept_prob", "beta_hat", "lse_p"):
        assert to_np(got[name]).tobytes() == to_np(plain[name]).tobytes(), name


def test_verify_packed_refuses_a_corrupt_record():
    B, gamma, V, k, T = 3, 2, 5000, 16, 1.0
    zq, zp = synth.sequence_logits(B, gamma, V, torch.bfloat16, 0.5, 3, "cpu")
    rows = B * gamma
    ud = synth.uniforms((rows, 1), 3, synth.TID_U_DRAFT)
    ref_s = oracle.sparsify(zq.reshape(rows, V), k, 1.0, T, ud.numpy())
    rec = P.pack(ref_s["idx"], ref_s["logit"], ref_s["count"], V, P.PROB_BF16).copy()
    rec[1, 0] = k + 5  # sequence 0, position 1: a count word no record of this library has
    tok = np.ascontiguousarray(ref_s["token"][:, 0].reshape(B, gamma))
    ua = synth.uniforms((B, gamma), 3, synth.TID_U_ACCEPT)
    us = synth.uniforms((B,), 3, synth.TID_U_SAMPLE)
    got = tslt.verify_packed(to_gpu_rows(zp), torch.from_numpy(rec.view(np.int32)).cuda(), tslt.PROB_BF16, k,
                             torch.from_numpy(tok).cuda(), T, T, ua.cuda(), us.cuda())
    torch.cuda.synchronize()
    assert tslt.workspace_status(got["workspace"]) & tslt.STATUS_BAD_RECORD
    # the row reads as empty: the oracle on a zero count gives the same verdicts
    cnt = ref_s["count"].copy()
    cnt[1] = 0
    ref_v = oracle.verify(zp, ref_s["idx"].reshape(B, gamma, k), ref_s["logit"].reshape(B, gamma, k), cnt.reshape(B, gamma),
                          tok, T, T, ua.numpy(), us.numpy())
    inp = verify_inputs(zp, dict(idx=ref_s["idx"], logit=ref_s["logit"], count=cnt), B, gamma, k, tok, T, T, ua, us)
    compare_verify(got, ref_v, "corrupt record", inputs=inp)


@pytest.mark.parametrize("expansion,V,dtype,k,fmt", [((2, 2, 2), 32000, torch.bfloat16, 64, FORMATS[1]),
                                                      ((3, 2), 20011, torch.float32, 40, FORMATS[0]),
                                                      ((3, 3, 3), 151936, torch.bfloat16, 64, FORMATS[1])])
def test_tree_verify_packed(expansion, V, dtype, k, fmt):
    gf, of = fmt
    B, T, seed = 4, 1.0, 9
    parent, ndr, M, depth = synth.complete_tree(expansion)
    N = len(parent)
    zq, zp = synth.tree_logits(B, parent, ndr, V, dtype, 0.5, seed, "cpu")
    kmax = max(expansion)
    ud = synth.uniforms((B * M, kmax), seed, synth.TID_U_DRAFT)
    ref_s = oracle.sparsify(zq.reshape(B * M, V), k, 1.0, T, ud.numpy())
    wl = wire(ref_s, of)
    rec = torch.from_numpy(P.pack(ref_s["idx"], ref_s["logit"], ref_s["count"], V, of).view(np.int32)).cuda()
    toks = np.zeros((B, N), np.int32)
    for n in range(N):
        if ndr[n] >= 0:
            ch = [c for c in range(N) if parent[c] == n]
            for b in range(B):
                toks[b, ch] = ref_s["token"][b * M + ndr[n], :len(ch)]
    ua = synth.uniforms((B, N), seed, synth.TID_U_ACCEPT)
    us = synth.uniforms((B, N), seed, synth.TID_U_SAMPLE)
    ref = oracle.tree_verify(zp, parent, ndr, toks, ref_s["idx"].reshape(B, M, k), wl.reshape(B, M, k),
                             ref_s["count"].reshape(B, M), T, T, ua.numpy(), us.numpy(), depth)
    inp = dict(zp=zp, parent=parent, ndr=ndr, toks=toks, idx=ref_s["idx"].reshape(B, M, k), logit=wl.reshape(B, M, k),
               count=ref_s["count"].reshape(B, M), Tq=T, Tp=T, ua=ua.numpy(), us=us.numpy(), depth=depth)
    z = to_gpu_rows(zp)
    outs = []
    for walk in (False, True):
        ws = torch.empty((tslt.tree_verify_walk_workspace_bytes if walk else tslt.tree_verify_workspace_bytes)(B, N, V, k) + 256,
                         dtype=torch.uint8, device="cuda")
        got = tslt.tree_verify_packed(z, parent, ndr, torch.from_numpy(toks).cuda(), rec, gf, k, T, T, ua.cuda(), us.cuda(),
                                      depth, walk=walk, ws=ws)
        torch.cuda.synchronize()
        assert tslt.workspace_status(got["workspace"]) == 0
        compare_tree(got, ref, "packed tree walk=%s %s" % (walk, expansion), inputs=inp)
        outs.append(got)
    for name in ("accepted_path", "accepted_len", "out_token"):
        assert to_np(outs[0][name]).tobytes() == to_np(outs[1][name]).tobytes(), name
