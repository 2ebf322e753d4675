"""World-size-2 gloo test of the data-parallel host logic: batch sharding, the all-reduce of the
clipped sums and the single shared noise draw.  The per-rank arithmetic is played by the oracle
(no GPU here); what is checked is that two ranks reproduce the single-process result."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    from oracle import dp_oracle as O
    from oracle import noise_oracle as NO
    from paper_2609_40335_b200 import parallel

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(0)                     # same global batch on every rank
    B, T, d, p, V, C = 5, 6, 4, 3, 9, 0.7
    A, G = rng.standard_normal((B, T, d)), rng.standard_normal((B, T, p))
    ids, Ge = rng.integers(0, V, (B, T)), rng.standard_normal((B, T, d))
    lo, hi = parallel.shard_range(B, rank, world)
    res = O.dp_step([(A[lo:hi], G[lo:hi])], ids[lo:hi], Ge[lo:hi], V, C)
    outs = {k: torch.from_numpy(v.copy()) for k, v in res["sums"].items()}

    def add_noise(t, tid):
        t.copy_(torch.from_numpy(NO.add_noise(t.numpy(), 0.5, C, 1.0, 3, tid, 11)))

    outs2 = {k: v.clone() for k, v in outs.items()}
    parallel.reduce_then_noise(outs, add_noise)
    ret[rank] = {k: v.numpy().copy() for k, v in outs.items()}

    # reduce-scatter form: each rank noises only the slice it owns, the slices are gathered back
    def add_noise_slice(t, first, tid):
        z = NO.standard_normals(t.numel(), 3, tid, 11, start=first)
        t.copy_(torch.from_numpy(1.0 * (t.numpy() + 0.5 * C * z)))

    owned = parallel.reduce_scatter_then_noise(outs2, add_noise_slice)
    ret[f"rs{rank}"] = {k: v.numpy().copy() for k, v in outs2.items()}
    ret[f"own{rank}"] = {k: (lo, hi) for k, (lo, hi, _) in owned.items()}
    ret[f"clip{rank}"] = (lo, hi, res["clip"])

    # bucketed form (what bench.py --gpus N runs): the tensors leave in the production order of the
    # clipped sums, each bucket as soon as it exists; the owned slices tile every tensor
    outs3 = {k: torch.from_numpy(v.copy()) for k, v in res["sums"].items()}
    for gather in (False, True):
        work = {k: v.clone() for k, v in outs3.items()}
        ex = parallel.BucketedExchange(work, lambda t, first, tid, st: add_noise_slice(t, first, tid),
                                       gather=gather)
        ex.begin_step()
        order = parallel.bucket_order(["linear0"], None, ["wte"], n_linear_buckets=3)
        for bucket in order:
            ex.submit(bucket)
        ex.finish()
        ret[f"bk{int(gather)}_{rank}"] = {k: (lo_, hi_, t.numpy().copy()) for k, (lo_, hi_, t) in ex.owned.items()}
        if gather:
            ret[f"bkfull{rank}"] = {k: v.numpy().copy() for k, v in work.items()}
        ret[f"wire{int(gather)}_{rank}"] = ex.bytes_on_wire
    try:                                   # a tensor that is never submitted is an error, not a silent skip
        ex2 = parallel.BucketedExchange({k: v.clone() for k, v in outs3.items()},
                                        lambda t, first, tid, st: None)
        ex2.begin_step()
        ex2.submit(["linear0"])
        ex2.finish()
        ret[f"missing{rank}"] = "not raised"
    except RuntimeError as e:
        ret[f"missing{rank}"] = str(e)
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_process_step():
    from oracle import dp_oracle as O
    from oracle import noise_oracle as NO
    from paper_2609_40335_b200 import parallel

    assert [parallel.shard_range(5, r, 2) for r in range(2)] == [(0, 3), (3, 5)]
    assert [parallel.shard_range(7, r, 3) for r in range(3)] == [(0, 3), (3, 5), (5, 7)]
    assert [parallel.slice_bounds(10, r, 3) for r in range(3)] == [(4, 0, 4), (4, 4, 8), (4, 8, 10)]
    assert parallel.slice_bounds(3, 1, 2) == (4, 3, 3)                     # empty trailing slice
    ctx = mp.get_context("spawn")
    ret = ctx.Manager().dict()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, ret)) for r in range(2)]
    for p_ in procs:
        p_.start()
    for p_ in procs:
        p_.join(120)
        assert p_.exitcode == 0
    rng = np.random.default_rng(0)
    B, T, d, p, V, C = 5, 6, 4, 3, 9, 0.7
    A, G = rng.standard_normal((B, T, d)), rng.standard_normal((B, T, p))
    ids, Ge = rng.integers(0, V, (B, T)), rng.standard_normal((B, T, d))
    full = O.dp_step([(A, G)], ids, Ge, V, C)
    for tid, k in enumerate(sorted(full["sums"])):
        want = NO.add_noise(full["sums"][k], 0.5, C, 1.0, 3, tid, 11)
        np.testing.assert_allclose(ret[0][k], want, rtol=1e-12, atol=1e-12)
        np.testing.assert_array_equal(ret[0][k], ret[1][k])       # replicas stay identical
        # the reduce-scatter form gives the same noised sums on both ranks
        np.testing.assert_allclose(ret["rs0"][k], want, rtol=1e-12, atol=1e-12)
        np.testing.assert_array_equal(ret["rs0"][k], ret["rs1"][k])
        n = want.size
        (lo0, hi0), (lo1, hi1) = ret["own0"][k], ret["own1"][k]
        assert lo0 == 0 and hi0 == lo1 and hi1 == n and lo1 % 4 == 0      # slices tile the tensor
    for r in range(2):
        lo, hi, clip = ret[f"clip{r}"]
        np.testing.assert_allclose(clip, full["clip"][lo:hi], rtol=1e-12)
    # bucketed exchange: every rank's owned slice holds the single-process values of that slice
    for tid, k in enumerate(sorted(full["sums"])):
        want = NO.add_noise(full["sums"][k], 0.5, C, 1.0, 3, tid, 11).reshape(-1)
        for gather in (0, 1):
            covered = 0
            for r in range(2):
                lo, hi, t = ret[f"bk{gather}_{r}"][k]
                np.testing.assert_allclose(t, want[lo:hi], rtol=1e-12, atol=1e-12)
                covered += hi - lo
            assert covered == want.size
        for r in range(2):
            np.testing.assert_allclose(ret[f"bkfull{r}"][k].reshape(-1), want, rtol=1e-12, atol=1e-12)
    assert ret["wire1_0"] == 2 * ret["wire0_0"] > 0
    assert "never exchanged" in ret["missing0"] and "wte" in ret["missing0"]
    # the bucket order: head first, the linears in contiguous groups, tables last, nothing lost
    order = parallel.bucket_order([f"linear{k}" for k in range(7)], "lm_head", ["wte", "wpe"], 3)
    assert order[0] == ["lm_head"] and order[-1] == ["wte", "wpe"]
    assert [n for b in order[1:-1] for n in b] == [f"linear{k}" for k in range(7)]
    assert len(order) == 5 and parallel.bucket_order([], None, ["wte"]) == [["wte"]]
