"""The N>1 path: token rows are sharded across ranks with no data-path collective.
Two gloo ranks on CPU each run the oracle on their shard; the gathered result must equal
the oracle on the whole tensor (this checks the shard planner and that rows really are
independent units).  No CUDA involved."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_21446_b200 import workloads as W


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, tokens, d, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import c_oracle as co
    spec = W.ActivationSpec("shard", tokens, d, seed=8, outlier_channels=3, outlier_gain=50.0,
                            spike_rows=2, spike_gain=8.0)
    Xb = W.gen_activations(spec)
    G = W.gen_factors(8)
    lo, hi = W.shard_rows(tokens, world, rank)
    q, s, _ = co.quantize(Xb[lo:hi], G)
    # gather variable-sized shards on rank 0 (gloo): pad to the largest shard
    n_max = -(-tokens // world)
    qpad = np.zeros((n_max, d // 2), np.uint8)
    spad = np.zeros((n_max, d // 32), np.uint8)
    qpad[:hi - lo], spad[:hi - lo] = q, s
    qt, stt = torch.from_numpy(qpad), torch.from_numpy(spad)
    qs = [torch.empty_like(qt) for _ in range(world)] if rank == 0 else None
    ss = [torch.empty_like(stt) for _ in range(world)] if rank == 0 else None
    dist.gather(qt, qs, dst=0)
    dist.gather(stt, ss, dst=0)
    if rank == 0:
        qf, sf, _ = co.quantize(Xb, G)
        qcat = np.concatenate([qs[r].numpy()[:W.shard_rows(tokens, world, r)[1] - W.shard_rows(tokens, world, r)[0]]
                               for r in range(world)])
        scat = np.concatenate([ss[r].numpy()[:W.shard_rows(tokens, world, r)[1] - W.shard_rows(tokens, world, r)[0]]
                               for r in range(world)])
        ok = np.array_equal(qcat, qf) and np.array_equal(scat, sf)
        with open(os.path.join(out_dir, "result.txt"), "w") as f:
            f.write("ok" if ok else "mismatch")
    dist.barrier()
    dist.destroy_process_group()


def test_shard_rows_partition():
    for tokens in (0, 1, 7, 4608, 65536):
        for world in (1, 2, 3, 8):
            ranges = [W.shard_rows(tokens, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == tokens
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
            sizes = [hi - lo for lo, hi in ranges]
            assert max(sizes) - min(sizes) <= 1


def test_two_rank_sharded_quantize_equals_whole(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, 257, 320, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "result.txt").read_text() == "ok"
