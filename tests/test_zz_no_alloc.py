"""tslt_verify_static, the entry point for callers that are not allowed to allocate device memory
(a serving loop whose memory pool owns all of HBM, a plug-in without access to its host's
allocator): its scratch is an 8 MiB array inside the library instead of a caller's workspace.

The check: through the C ABI, on two calls in a row (the second finds the first call's leftovers
in the shared array), its outputs equal those of tslt_verify with an ordinary workspace: integer
outputs exactly, fp32 diagnostics within the 1e-5 relative bar of the other parity tests.  The
file sorts last so that a run stopping at the first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2512_16273_b200 import synth, tslt
from parity_utils import ATOL_PROB, RTOL, close, to_np


def _outputs(B, gamma, device):
    return {"accepted_len": torch.full((B,), -7, dtype=torch.int32, device=device),
            "out_token": torch.full((B,), -7, dtype=torch.int32, device=device),
            "accept_prob": torch.full((B, gamma), -7.0, device=device),
            "beta_hat": torch.full((B, gamma), -7.0, device=device),
            "lse_p": torch.full((B, gamma + 1), -7.0, device=device)}


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_twice():
    k = 64
    cases = [(8, 8, 32000, torch.bfloat16, 0.8, 11),     # config-1 shape
             (3, 4, 20011, torch.float32, 1.0, 12)]      # ragged fp32 rows, different sizes on the second call
    for B, gamma, V, dtype, T, seed in cases:
        zq, zp = synth.sequence_logits(B, gamma, V, dtype, 0.5, seed, "cpu")
        ud = synth.uniforms((B * gamma, 1), seed, synth.TID_U_DRAFT).cuda()
        ua = synth.uniforms((B, gamma), seed, synth.TID_U_ACCEPT).cuda()
        us = synth.uniforms((B,), seed, synth.TID_U_SAMPLE).cuda()
        from parity_utils import to_gpu_rows
        s = tslt.sparsify(to_gpu_rows(zq), k, 1.0, T, ud)
        zp_d = to_gpu_rows(zp)
        args = (zp_d, s["idx"].view(B, gamma, k), s["logit"].view(B, gamma, k), s["count"].view(B, gamma),
                s["token"].view(B, gamma).contiguous(), T, T, ua, us)
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
            assert close(to_np(out["lse_p"]), to_np(ref["lse_p"]), RTOL).all(), ("lse_p", call)


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
