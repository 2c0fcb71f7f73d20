"""GPU parity of tslt_diagnostics (through the C ABI) against the numpy oracle, element by element:
1e-5 relative + 1e-6 absolute on every probability, on fp32 and bf16 rows, ragged vocabularies, K lists
that reach beyond the finite entries, and the bench vocabulary at reduced batch."""
import numpy as np
import pytest
import torch

from oracle import diagnostics as D
from paper_2512_16273_b200 import synth, tslt
from parity_utils import ATOL_PROB, RTOL, close, to_gpu_rows, to_np

pytestmark = pytest.mark.gpu


def check(zq, zp, ks, c, Tq, Tp, what):
    ref = D.diagnostics(zq.double().numpy(), zp.double().numpy(), ks, c, Tq, Tp)
    got = tslt.diagnostics(to_gpu_rows(zq), to_gpu_rows(zp), ks, c, Tq, Tp)
    torch.cuda.synchronize()
    assert tslt.workspace_status(got["workspace"]) == 0
    for name in ("beta_j", "z_j", "theta", "rho", "beta_hat_j", "theta_hat"):
        ok = close(to_np(got[name]), ref[name], RTOL, ATOL_PROB)
        assert ok.all(), (what, name, np.argwhere(~ok)[:4], to_np(got[name])[~ok][:4], ref[name][~ok][:4])
    # Theorem 1 on the GPU's own numbers: |beta^ - beta| <= sigma (to fp32 rounding)
    sigma = 1.0 - to_np(got["rho"])
    assert (np.abs(to_np(got["beta_hat_j"])[:, :, 0] - to_np(got["beta_j"])[:, :1]) <= sigma + 1e-5).all(), what


@pytest.mark.parametrize("V,dtype", [(1000, torch.float32), (4099, torch.bfloat16), (32000, torch.bfloat16), (20011, torch.float32)])
def test_diagnostics_small(V, dtype):
    zq, zp = synth.sequence_logits(1, 6, V, dtype, 0.5, V, "cpu")
    check(zq[0], zp[0, :6], [1, 8, 64, 320, min(V, 1000)], 4, 1.0, 1.0, "V=%d" % V)
    check(zq[0], zp[0, :6], [32, 320], 2, 0.7, 1.3, "V=%d temperatures" % V)


def test_diagnostics_few_finite_and_identical_rows():
    V = 3000
    zq, zp = synth.sequence_logits(1, 4, V, torch.float32, 0.5, 5, "cpu")
    zq, zp = zq[0].clone(), zp[0, :4].clone()
    zq[0, 40:] = -float("inf")            # 40 finite draft logits: K = 64 uses them all
    zp[1] = zq[1]                          # identical models: beta = 1
    check(zq, zp, [16, 64, 256], 3, 1.0, 1.0, "few finite / identical")


def test_diagnostics_bench_vocabulary():
    cfg = synth.CONFIGS[4]
    zq, zp = synth.sequence_logits(2, 4, cfg["V"], torch.bfloat16, cfg["sigma_t"], 1, "cpu")
    check(zq.reshape(-1, cfg["V"]), zp[:, :4].reshape(-1, cfg["V"]), [16, 64, 256, 1024], 3, 1.0, 1.0, "V=256000")
