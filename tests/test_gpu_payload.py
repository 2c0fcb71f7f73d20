"""GPU parity of the uplink payload: tslt_pack_payload / tslt_unpack_payload against the numpy
oracle (oracle/payload.py), byte for byte, and the verifier on an unpacked payload against the
oracle's verifier on the logits the wire format leaves."""
import numpy as np
import pytest
import torch

import oracle
from oracle import payload as P
from paper_2512_16273_b200 import synth, tslt
from parity_utils import compare_verify, to_gpu_rows, to_np, verify_inputs

pytestmark = pytest.mark.gpu

FORMATS = [(tslt.PROB_F32, P.PROB_F32), (tslt.PROB_BF16, P.PROB_BF16), (tslt.PROB_F16, P.PROB_F16)]


def random_rows(rows, k, V, seed, special=True):
    rng = np.random.default_rng(seed)
    idx = np.full((rows, k), -1, np.int32)
    logit = np.full((rows, k), -np.inf, np.float32)
    count = rng.integers(0, k + 1, size=rows).astype(np.int32)
    count[0] = 0
    count[-1] = k
    for r in range(rows):
        n = min(int(count[r]), V)
        count[r] = n
        idx[r, :n] = np.sort(rng.choice(V, size=n, replace=False))
        logit[r, :n] = (rng.standard_normal(n) * 8).astype(np.float32)
    if special and rows > 2 and count[-1] >= 4:
        logit[-1, 0] = -np.inf
        logit[-1, 1] = 70000.0      # beyond half precision: becomes inf on a 16-bit IEEE wire
        logit[-1, 2] = np.float32(1.00390625)   # a tie of the bf16 rounding
        idx[-1, count[-1] - 1] = V - 1          # the largest index uses every index bit
    return idx, logit, count


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("V,k", [(2, 1), (8, 3), (1000, 37), (32000, 64), (151936, 320), (256000, 1024)])
def test_pack_and_unpack_match_the_oracle(V, k, fmt):
    gf, of = fmt
    rows = 23
    idx, logit, count = random_rows(rows, k, V, seed=V + k + gf)
    want = P.pack(idx, logit, count, V, of)
    words, ebits = tslt.payload_words(k, V, gf)
    assert words == P.words_per_row(k, V, of) == want.shape[1] and ebits == P.entry_bits(V, of)
    g = tslt.pack_payload(torch.from_numpy(idx).cuda(), torch.from_numpy(logit).cuda(), torch.from_numpy(count).cuda(), V, gf)
    torch.cuda.synchronize()
    got = to_np(g["payload"]).view(np.uint32)
    assert got.tobytes() == want.tobytes()
    assert (to_np(g["bits"]) == P.payload_bits(count, V, of)).all()
    # the other direction, from the oracle's records
    u = tslt.unpack_payload(torch.from_numpy(want.view(np.int32)).cuda(), k, V, gf)
    torch.cuda.synchronize()
    i2, l2, c2 = P.unpack(want, k, V, of)
    assert (to_np(u["count"]) == c2).all() and (to_np(u["idx"]) == i2).all()
    assert to_np(u["logit"]).tobytes() == l2.tobytes()
    assert int(to_np(u["flag"])[0]) == 0


def test_many_rows_and_corrupt_count():
    V, k, rows = 128256, 128, 3000
    idx, logit, count = random_rows(rows, k, V, seed=5, special=False)
    g = tslt.pack_payload(torch.from_numpy(idx).cuda(), torch.from_numpy(logit).cuda(), torch.from_numpy(count).cuda(), V,
                          tslt.PROB_BF16)
    u = tslt.unpack_payload(g["payload"], k, V, tslt.PROB_BF16)
    torch.cuda.synchronize()
    assert (to_np(u["count"]) == count).all() and (to_np(u["idx"]) == idx).all()
    assert to_np(u["logit"]).tobytes() == np.where(idx >= 0, P.round_value(logit, P.PROB_BF16), -np.inf).astype(np.float32).tobytes()
    # a record whose count word exceeds k is refused: flag set, row empty, nothing out of bounds
    bad = g["payload"].clone()
    bad[7, 0] = k + 1
    u = tslt.unpack_payload(bad, k, V, tslt.PROB_BF16)
    torch.cuda.synchronize()
    assert int(to_np(u["flag"])[0]) == 1 and int(to_np(u["count"])[7]) == 0 and (to_np(u["idx"])[7] == -1).all()
    assert int(to_np(u["count"])[8]) == int(count[8])


@pytest.mark.parametrize("dtype,fmt", [(torch.bfloat16, FORMATS[1]), (torch.float32, FORMATS[1]), (torch.float32, FORMATS[2]),
                                       (torch.float32, FORMATS[0])])
def test_round_trip_through_the_wire_then_verify(dtype, fmt):
    """sparsify -> pack -> unpack -> verify on the GPU against the oracle's verifier given the
    logits as the wire format leaves them.  bf16 logits on a bf16 wire are untouched."""
    gf, of = fmt
    B, gamma, V, k, T = 6, 4, 20011, 48, 0.9
    zq, zp = synth.sequence_logits(B, gamma, V, dtype, 0.5, 11, "cpu")
    rows = B * gamma
    ud = synth.uniforms((rows, 1), 11, synth.TID_U_DRAFT)
    ua = synth.uniforms((B, gamma), 11, synth.TID_U_ACCEPT)
    us = synth.uniforms((B,), 11, synth.TID_U_SAMPLE)
    ref_s = oracle.sparsify(zq.reshape(rows, V), k, 1.0, T, ud.numpy())
    wire_logit = np.where(ref_s["idx"] >= 0, P.round_value(ref_s["logit"], of), -np.inf).astype(np.float32)
    if dtype == torch.bfloat16 and of == P.PROB_BF16:
        assert wire_logit.tobytes() == ref_s["logit"].tobytes()
    g = tslt.pack_payload(torch.from_numpy(ref_s["idx"]).cuda(), torch.from_numpy(ref_s["logit"]).cuda(),
                          torch.from_numpy(ref_s["count"]).cuda(), V, gf)
    u = tslt.unpack_payload(g["payload"], k, V, gf)
    tok = np.ascontiguousarray(ref_s["token"][:, 0].reshape(B, gamma))
    gpu_v = tslt.verify(to_gpu_rows(zp), u["idx"].view(B, gamma, k), u["logit"].view(B, gamma, k), u["count"].view(B, gamma),
                        torch.from_numpy(tok).cuda(), T, T, ua.cuda(), us.cuda())
    torch.cuda.synchronize()
    ref_v = oracle.verify(zp, ref_s["idx"].reshape(B, gamma, k), wire_logit.reshape(B, gamma, k),
                          ref_s["count"].reshape(B, gamma), tok, T, T, ua.numpy(), us.numpy())
    inp = verify_inputs(zp, dict(idx=ref_s["idx"], logit=wire_logit, count=ref_s["count"]), B, gamma, k, tok, T, T, ua, us)
    compare_verify(gpu_v, ref_v, "wire %s / %d" % (dtype, gf), inputs=inp)


def test_argument_errors():
    t = torch.zeros(4, 8, dtype=torch.int32, device="cuda")
    with pytest.raises(tslt.TsltError):
        tslt.payload_words(8, 1000, 7)
    with pytest.raises(tslt.TsltError):
        tslt.payload_words(0, 1000, tslt.PROB_F32)
    with pytest.raises(ValueError):
        tslt.unpack_payload(t, 8, 1000, tslt.PROB_F32)  # wrong record width
