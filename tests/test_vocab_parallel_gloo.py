"""The vocabulary-parallel form of tslt_sparsify on two gloo ranks on the CPU: the plumbing around the
kernels (the order and layout of the all-gathered parts, the shard offsets, every rank getting the same
answer).  The two compute steps need a GPU, so the CPU oracle stands in for them here (per-shard top-k and
log-normaliser; the merge by its definition in numpy); the kernels themselves are held against the
oracle in tests/test_gpu_sharded.py."""
import os
import sys

import numpy as np
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
V, K, T, TOP_P, ROWS = 3001, 24, 0.9, 1.0, 5
BOUNDS = [0, 1296, V]  # ragged: the second rank's slice is longer


def _logits():
    g = torch.Generator().manual_seed(77)
    return (torch.randn(ROWS, V, generator=g) * 2.0).to(torch.float32)


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    import oracle
    from paper_2512_16273_b200 import vocab_parallel
    dist.init_process_group("gloo", rank=rank, world_size=world)
    z = _logits()
    local = z[:, BOUNDS[rank]:BOUNDS[rank + 1]].contiguous()
    u = np.full((ROWS, 1), 0.37, np.float32)

    def shard_fn(x, k, temperature):  # the oracle in place of tslt_sparsify_shard
        r = oracle.sparsify(x, k, 1.0, temperature, np.zeros((x.shape[0], 1), np.float32))
        return {"idx": torch.from_numpy(r["idx"]), "logit": torch.from_numpy(r["logit"]),
                "count": torch.from_numpy(r["count"]), "lse2": torch.from_numpy(r["lse"] / np.log(2.0))}

    def merge_fn(parts, offsets, dtype, top_p, temperature, uniforms):  # the merge by its definition
        idx = parts["idx"].numpy() + np.asarray(offsets, np.int64)[:, None, None]
        idx = np.where(parts["idx"].numpy() >= 0, idx, -1)
        out = np.full((ROWS, K), -1, np.int64)
        for r in range(ROWS):
            ci = np.concatenate([idx[s, r] for s in range(idx.shape[0])])
            cl = np.concatenate([parts["logit"].numpy()[s, r] for s in range(idx.shape[0])])
            assert (np.diff(ci[ci >= 0]) > 0).all()  # shard order is vocabulary order: one ascending list
            keep = ci >= 0
            order = np.lexsort((ci[keep], -cl[keep].astype(np.float64)))[:K]
            sel = np.sort(ci[keep][order])
            out[r, :len(sel)] = sel
        lse = np.logaddexp.reduce(parts["lse2"].numpy() * np.log(2.0), axis=0)
        return {"idx": out, "lse": lse, "offsets": list(offsets)}

    got = vocab_parallel.sparsify_vocab_parallel(local, BOUNDS[rank], K, TOP_P, T, u, shard_fn=shard_fn, merge_fn=merge_fn)
    whole = oracle.sparsify(z, K, TOP_P, T, u)
    ok = bool(np.array_equal(got["idx"], whole["idx"]) and np.allclose(got["lse"], whole["lse"], rtol=1e-12, atol=1e-12)
              and got["offsets"] == BOUNDS[:-1])
    # overlapping slices are refused on every rank
    refused = False
    try:
        vocab_parallel.sparsify_vocab_parallel(local, 0, K, TOP_P, T, u, shard_fn=shard_fn, merge_fn=merge_fn)
    except ValueError:
        refused = True
    q.put((rank, ok, refused))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gather_parts_in_vocabulary_order():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29900 + os.getpid() % 90
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, True, True), (1, True, True)]
