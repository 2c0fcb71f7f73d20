"""tslt_verify_static, the entry point for callers that are not allowed to allocate device memory
(a serving loop whose memory pool owns all of HBM, a plug-in without access to its host's
allocator): its scratch is an 8 MiB array inside the library instead of a caller's workspace.

The check: through the C ABI, on two calls in a row (the second finds the first call's leftovers
in the shared array), its outputs equal those of tslt_verify with an ordinary workspace: integer
outputs exactly, fp32 diagnostics within the 1e-5 relative bar of the other parity tests; and, like
every other entry point, they are held against the CPU oracle.  One case is large enough to fill
the machine (hundreds of target rows cut into 64 KB segments, 3.3 MiB of the array in use).  The
file sorts last so that a run stopping at the first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2512_16273_b200 import synth, tslt
from parity_utils import ATOL_LSE, ATOL_PROB, RTOL, close, compare_verify, to_gpu_rows, to_np, verify_inputs


def _outputs(B, gamma, device):
    return {"accepted_len": torch.full((B,), -7, dtype=torch.int32, device=device),
            "out_token": torch.full((B,), -7, dtype=torch.int32, device=device),
            "accept_prob": torch.full((B, gamma), -7.0, device=device),
            "beta_hat": torch.full((B, gamma), -7.0, device=device),
            "lse_p": torch.full((B, gamma + 1), -7.0, device=device)}


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_and_oracle_twice():
    k = 64
    cases = [(8, 8, 32000, torch.bfloat16, 0.8, 11),     # config-1 shape
             (3, 4, 20011, torch.float32, 1.0, 12),      # ragged fp32 rows, different sizes on the second case
             (120, 7, 110000, torch.bfloat16, 1.0, 13)]  # 960 target rows: more than the machine holds at once
    for B, gamma, V, dtype, T, seed in cases:
        zq, zp = synth.sequence_logits(B, gamma, V, dtype, 0.5, seed, "cpu")
        ud = synth.uniforms((B * gamma, 1), seed, synth.TID_U_DRAFT)
        ua = synth.uniforms((B, gamma), seed, synth.TID_U_ACCEPT)
        us = synth.uniforms((B,), seed, synth.TID_U_SAMPLE)
        ref_s = oracle.sparsify(zq.reshape(-1, V), k, 1.0, T, ud.numpy())
        tok = np.ascontiguousarray(ref_s["token"][:, 0].reshape(B, gamma))
        inp = verify_inputs(zp, ref_s, B, gamma, k, tok, T, T, ua, us)
        ref_o = oracle.verify(zp, inp["idx"], inp["logit"], inp["count"], inp["token"], T, T, inp["ua"], inp["us"])
        zp_d = to_gpu_rows(zp)
        args = (zp_d, torch.from_numpy(inp["idx"]).cuda(), torch.from_numpy(inp["logit"]).cuda(),
                torch.from_numpy(inp["count"]).cuda(), torch.from_numpy(inp["token"]).cuda(), T, T, ua.cuda(), us.cuda())
        assert tslt.verify_workspace_bytes(B, gamma, V, k) <= tslt.STATIC_SCRATCH_BYTES
        ref = tslt.verify(*args)
        torch.cuda.synchronize()
        for call in range(2):
            out = _outputs(B, gamma, "cuda")
            tslt.verify_static(*args, out=out)
            torch.cuda.synchronize()
            for name in ("accepted_len", "out_token"):
                assert np.array_equal(to_np(out[name]), to_np(ref[name])), (name, call, B, V)
            for name in ("accept_prob", "beta_hat"):
                assert close(to_np(out[name]), to_np(ref[name]), RTOL, ATOL_PROB).all(), (name, call)
            assert close(to_np(out["lse_p"]), to_np(ref["lse_p"]), RTOL, ATOL_LSE).all(), ("lse_p", call)
            compare_verify(out, ref_o, "static scratch B=%d V=%d call %d" % (B, V, call), inputs=inp)


def test_static_scratch_refuses_what_does_not_fit():
    """The size check runs on the host before anything touches a device, so it needs no GPU."""
    L = tslt.lib()
    fake = ctypes.c_void_p(0x1000)
    need = tslt.verify_workspace_bytes(4096, 8, 256000, 64)
    assert need > tslt.STATIC_SCRATCH_BYTES
    rc = L.tslt_verify_static(fake, tslt.BF16, 4096, 8, 256000, 256000, 64, fake, fake, fake, fake, 1.0, 1.0,
                              fake, fake, fake, fake, None, None, None, None)
    assert rc == tslt.ERR_STATIC_SCRATCH
    assert "scratch" in tslt.status_string(rc)
