"""World-size-2 check of the multi-GPU recipe on CPU (gloo): heads are sharded across ranks with no collective
in the data path, every rank computes its slice on its own (here with the CPU oracle standing in for the
device library), and the gathered slices equal the unsharded result.  Also the max-over-ranks timing helper."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    from oracle import attn_jvp_numpy as onp
    from paper_2511_19797_b200 import inputs, sharding
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = inputs.custom(3, 3, 20, 8, seed=12)          # 9 heads over 2 ranks: 5 + 4
    lo, hi = sharding.head_range(wl.B * wl.H, rank, world)
    x = inputs.make_inputs(wl, heads=list(range(lo, hi)))
    xs = [x[k].to(torch.float64).numpy() for k in inputs.NAMES]
    O, tO, _, _ = onp.attn_jvp_fwd(*xs[:6], 0.3)
    dQ = onp.attn_jvp_bwd(*xs, 0.3)[0]
    np.save(os.path.join(out_dir, "r%d.npy" % rank), np.concatenate([O, tO, dQ], axis=1))
    slow = sharding.max_over_ranks(1.0 + rank, dist)   # rank 1 is "slower"
    assert slow == float(world), slow
    dist.barrier()
    dist.destroy_process_group()


def test_heads_shard_across_two_ranks_without_a_collective(tmp_path):
    from oracle import attn_jvp_numpy as onp
    from paper_2511_19797_b200 import inputs, sharding
    assert [sharding.head_range(9, r, 2) for r in range(2)] == [(0, 5), (5, 9)]
    assert [sharding.head_range(8, r, 4) for r in range(4)] == [(0, 2), (2, 4), (4, 6), (6, 8)]
    assert sharding.head_range(1, 1, 2) == (1, 1)
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    got = np.concatenate([np.load(os.path.join(str(tmp_path), "r%d.npy" % r)) for r in range(2)], axis=0)
    wl = inputs.custom(3, 3, 20, 8, seed=12)
    x = inputs.make_inputs(wl, heads=list(range(9)))
    xs = [x[k].to(torch.float64).numpy() for k in inputs.NAMES]
    O, tO, _, _ = onp.attn_jvp_fwd(*xs[:6], 0.3)
    dQ = onp.attn_jvp_bwd(*xs, 0.3)[0]
    ref = np.concatenate([O, tO, dQ], axis=1)
    assert got.shape == ref.shape and np.array_equal(got, ref)
