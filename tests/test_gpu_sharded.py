"""GPU parity of the vocabulary-sharded two-stage sparsify (tslt_sparsify_shard on every slice, then
tslt_sparsify_merge; both through the C ABI) against the CPU oracle run on the WHOLE rows, and against
tslt_sparsify on the whole rows: the truncated set, its logits and the count must be bit-identical,
samples and statistics to the bar of the other parity tests.  Shards are ragged, some hold fewer than
k finite logits, one case has a shard with none."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_16273_b200 import synth, tslt
from parity_utils import compare_sparsify, oracle_sparsify_parallel, to_gpu_rows, to_np

pytestmark = pytest.mark.gpu


def run_case(z_cpu, bounds, k, top_p, T, seed, ns, what):
    rows, V = z_cpu.shape
    u = synth.uniforms((rows, ns), seed, 11)
    ref = oracle_sparsify_parallel(z_cpu, k, top_p, T, u.numpy())
    z = to_gpu_rows(z_cpu)
    got = tslt.sparsify_sharded(z, bounds, k, top_p, T, u.cuda())
    torch.cuda.synchronize()
    assert tslt.workspace_status(got["workspace"]) == 0
    for ws in got["shard_workspaces"]:
        assert tslt.workspace_status(ws) == 0
    compare_sparsify(got, ref, what, logits=z_cpu, uniforms=u, T=T)
    whole = tslt.sparsify(z, k, top_p, T, u.cuda())
    torch.cuda.synchronize()
    same_cut = to_np(whole["count"]) == to_np(got["count"])  # (a cumulative mass on top_p may cut one entry apart)
    assert (same_cut | ((ref["flags"] & oracle.FLAG_SEL) != 0)).all(), (what, "count differs from tslt_sparsify")
    for name in ("idx", "logit"):
        a, b = to_np(whole[name])[same_cut], to_np(got[name])[same_cut]
        assert a.tobytes() == b.tobytes(), (what, name, "differs from tslt_sparsify")
    # every shard's own part is the oracle's top-k of that slice
    for s in range(len(bounds) - 1):
        sl = z_cpu[:, bounds[s]:bounds[s + 1]].contiguous()
        ks = min(k, sl.shape[1])
        if ks < k:
            continue  # (a shard narrower than k: not accepted by tslt_sparsify_shard, not built by these cases)
        r = oracle_sparsify_parallel(sl, k, 1.0, T, np.zeros((rows, 1), np.float32))
        assert np.array_equal(to_np(got["parts"]["idx"][s]), r["idx"]), (what, "shard idx", s)
        assert np.array_equal(to_np(got["parts"]["count"][s]), r["count"]), (what, "shard count", s)
        lse2 = to_np(got["parts"]["lse2"][s]) * np.log(2.0)
        fin = np.isfinite(r["lse"])
        assert np.allclose(lse2[fin], r["lse"][fin], rtol=1e-5, atol=1e-6) and np.isneginf(lse2[~fin]).all(), (what, "shard lse", s)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_sharded_small(dtype):
    V = 20016
    zq, _ = synth.sequence_logits(3, 4, V, dtype, 0.5, 31, "cpu")
    z = zq.reshape(-1, V)
    run_case(z, [0, 5000, 10008, 15016, V], 64, 1.0, 1.0, 1, 2, "4 shards k=64 %s" % dtype)
    run_case(z, [0, 8, 10000, V], 8, 0.9, 0.7, 2, 1, "3 ragged shards top-p %s" % dtype)
    run_case(z, [0, 2048, 4096, 6144, 8192, 10240, 12288, 14336, V], 256, 0.95, 1.0, 3, 1, "8 shards k=256 %s" % dtype)
    run_case(z, [0, 10008, V], 1024, 1.0, 1.3, 4, 1, "2 shards k=1024 %s" % dtype)


def test_sharded_sparse_and_empty_shards():
    V = 12000
    zq, _ = synth.sequence_logits(2, 3, V, torch.float32, 0.5, 5, "cpu")
    z = zq.reshape(-1, V).clone()
    z[:, 4000:8000] = -float("inf")      # a shard with no finite logit
    z[0, 40:4000] = -float("inf")        # a shard with fewer than k
    z[1, :] = -float("inf")              # a row with none at all
    z[2, 8000:] = 1.25                   # thousands of ties inside one shard
    run_case(z, [0, 4000, 8000, V], 64, 1.0, 1.0, 9, 2, "empty / thin shards")
    run_case(z, [0, 4000, 8000, V], 64, 0.8, 1.0, 10, 1, "empty / thin shards top-p")


def test_sharded_bench_vocabulary():
    cfg = synth.CONFIGS[4]
    V = cfg["V"]
    zq, _ = synth.sequence_logits(4, 4, V, torch.bfloat16, cfg["sigma_t"], 2, "cpu")
    z = zq.reshape(-1, V)
    run_case(z, [0, 32000, 64000, 96000, 128000, 160000, 192000, 224000, V], 64, 1.0, 1.0, 12, 1, "V=256000 8 shards")
    run_case(z, [0, 64000, 128000, 192000, V], 256, 0.95, 1.0, 13, 1, "V=256000 4 shards top-p")


def test_merge_rejects_what_it_cannot_hold():
    dev = "cuda"
    part = dict(idx=torch.zeros(4, 2, 1024, dtype=torch.int32, device=dev), logit=torch.zeros(4, 2, 1024, device=dev),
                count=torch.zeros(4, 2, dtype=torch.int32, device=dev), lse2=torch.zeros(4, 2, dtype=torch.float64, device=dev))
    with pytest.raises(tslt.TsltError) as e:
        tslt.sparsify_merge(part["idx"], part["logit"], part["count"], part["lse2"], [0, 10, 20, 30], torch.float32)
    assert e.value.status == tslt.ERR_UNSUPPORTED  # 4 * 1024 entries
    with pytest.raises(tslt.TsltError) as e:
        tslt.sparsify_merge(part["idx"][:2], part["logit"][:2], part["count"][:2], part["lse2"][:2], [10, 10], torch.float32)
    assert e.value.status == tslt.ERR_INVALID_ARG  # offsets must ascend


def test_vocab_parallel_glue_on_one_rank():
    """The glue with the library's own kernels and NCCL, as far as one GPU goes: a process group of one
    rank, whose single slice is the whole vocabulary; same outputs as tslt_sparsify."""
    import torch.distributed as dist
    from paper_2512_16273_b200 import vocab_parallel
    created = False
    if not dist.is_initialized():
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29877", rank=0, world_size=1)
        created = True
    try:
        V, k = 20016, 64
        z = synth.draft_rows(6, V, torch.bfloat16, 8, "cuda")
        u = synth.uniforms((6, 2), 8, 11, "cuda")
        got = vocab_parallel.sparsify_vocab_parallel(z, 0, k, 0.95, 0.8, u)
        want = tslt.sparsify(z, k, 0.95, 0.8, u)
        torch.cuda.synchronize()
        for name in ("idx", "logit", "count", "token"):
            assert to_np(got[name]).tobytes() == to_np(want[name]).tobytes(), name
        assert np.allclose(to_np(got["lse"]), to_np(want["lse"]), rtol=1e-6, atol=1e-6)
    finally:
        if created:
            dist.destroy_process_group()
