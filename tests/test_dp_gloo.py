"""Data-parallel path on CPU: two gloo ranks, each with its own token shard, run the
fp64 oracle's backward on the shard and all-reduce the parameter gradients through the
same helper bench.py uses on NCCL.  The reduced gradients must equal the oracle's
gradients on the whole batch (they are linear in G = dY^T X and the STE gate depends on
the replicated weights only), and dX must be the corresponding rows of the full dX."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import l4q_oracle as orc
from paper_2402_04902_b200 import dp, synth

CFG = synth.LayerConfig("dp_cpu", tokens=96, d_in=128, d_out=72, rank=8, alpha=16.0, bits=4, group_size=32,
                        io_dtype="f32")


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        arrays = {k: np.asarray(v, dtype=np.float64) for k, v in synth.make_layer_inputs(CFG, seed=3).items()}
        spec = orc.L4QSpec(rank=CFG.rank, alpha=CFG.alpha, bits=CFG.bits, group_size=CFG.group_size)
        sl = dp.token_shard(CFG.tokens, rank, world)
        g = orc.backward(spec, arrays["X"][sl], arrays["dY"][sl], arrays["W0"], arrays["A"], arrays["B"],
                         arrays["s"], arrays["b"])
        if True:
            # half of the test goes through the per-tensor helper, half through the bucket bench.py uses
            flat, views = dp.alloc_grad_bucket({k: g[k].shape for k in dp.PARAM_GRADS}, dtype=torch.float64)
            for k in dp.PARAM_GRADS:
                views[k].copy_(torch.from_numpy(np.ascontiguousarray(g[k])))
            dp.allreduce_grad_bucket(flat)
        grads = {k: torch.from_numpy(np.ascontiguousarray(g[k])) for k in dp.PARAM_GRADS}
        dp.allreduce_param_grads(grads)
        for k in dp.PARAM_GRADS:
            assert torch.equal(views[k], grads[k]), k
            assert views[k].data_ptr() % 16 == 0
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), dX=g["dX"], start=sl.start, stop=sl.stop,
                 **{k: v.numpy() for k, v in grads.items()})
    finally:
        dist.destroy_process_group()


def test_token_shards_are_balanced_and_cover_the_batch():
    for tokens, world in ((96, 2), (97, 2), (10, 4), (3, 4)):
        shards = [dp.token_shard(tokens, r, world) for r in range(world)]
        assert shards[0].start == 0 and shards[-1].stop == tokens
        assert all(a.stop == b.start for a, b in zip(shards, shards[1:]))
        sizes = [s.stop - s.start for s in shards]
        assert max(sizes) - min(sizes) <= 1


def test_two_gloo_ranks_reduce_to_the_full_batch_gradients(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    arrays = {k: np.asarray(v, dtype=np.float64) for k, v in synth.make_layer_inputs(CFG, seed=3).items()}
    spec = orc.L4QSpec(rank=CFG.rank, alpha=CFG.alpha, bits=CFG.bits, group_size=CFG.group_size)
    full = orc.backward(spec, arrays["X"], arrays["dY"], arrays["W0"], arrays["A"], arrays["B"], arrays["s"],
                        arrays["b"])
    outs = [np.load(os.path.join(tmp_path, f"rank{r}.npz")) for r in range(world)]
    for k in dp.PARAM_GRADS:
        assert np.array_equal(outs[0][k], outs[1][k]), k                # every rank holds the same reduced value
        assert np.allclose(outs[0][k], full[k], rtol=1e-12, atol=1e-12 * np.abs(full[k]).max()), k
    dX = np.vstack([outs[r]["dX"] for r in range(world)])
    assert int(outs[0]["stop"]) == int(outs[1]["start"])
    assert np.allclose(dX, full["dX"], rtol=1e-12, atol=1e-14)
