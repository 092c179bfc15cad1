"""Multi-GPU path on CPU: the batch is sharded by sequence (sequences are independent, no collective on
the data path), each rank verifies its own slice, and the gathered per-sequence results equal the
unsharded run. Two `gloo` ranks. What is under test here is the host logic of a sharded run: `shard_call`
(the slice of every per-sequence tensor and the `seq_index_base` a rank passes with it), ragged shards, and
the gather of the results. No GPU is present, so the verification of a slice is stood in for by the CPU
oracle, told the same thing the library is told -- the index of the slice's first sequence; that the
library itself returns the unsharded results for such a call is the GPU test
`test_sequence_base_makes_shards_reproduce_the_whole_batch`, which cuts its batch with the same `shard_call`."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, B, K_d, K_q, V, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2510_12966_b200 import workloads
    zd, zq, zt, tok = workloads.make_pyramid_inputs(B, K_d, K_q, V, "bf16", seed=77, sigma_q=0.5, sigma_d=0.9)
    lo, hi, seq_index_base = workloads.shard_call(B, rank, world)
    ids = seq_index_base + np.arange(hi - lo)
    res = oracle.verify(workloads.to_host_bits(zd[lo:hi]), workloads.to_host_bits(zq[lo:hi]),
                        workloads.to_host_bits(zt[lo:hi]), tok[lo:hi].numpy(), np.float32(0.3), np.float32(0.2),
                        oracle.STRICT, 5, 8, seq_ids=ids)
    mine = torch.tensor(np.stack([res["accept_len_q"], res["next_token_q"], res["accept_len"], res["next_token"]], 1),
                        dtype=torch.int32)
    sizes = [h - l for l, h in (workloads.shard_batch(B, r, world) for r in range(world))]
    padded = torch.zeros((max(sizes), 4), dtype=torch.int32)   # ragged shards: pad to the largest one
    padded[:hi - lo] = mine
    gathered = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(gathered, padded)   # result collection only: 4 ints per sequence, not on the data path
    if rank == 0:
        np.save(os.path.join(out_dir, "sharded.npy"), torch.cat([g[:n] for g, n in zip(gathered, sizes)]).numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_batch_shards_reproduce_the_unsharded_result(tmp_path, oracle):
    from paper_2510_12966_b200 import workloads
    B, K_d, K_q, V, world = 7, 5, 3, 1531, 2          # B not divisible by the world size: ragged shards
    port = _free_port()
    mp.spawn(_worker, args=(world, port, B, K_d, K_q, V, str(tmp_path)), nprocs=world, join=True)
    sharded = np.load(tmp_path / "sharded.npy")
    zd, zq, zt, tok = workloads.make_pyramid_inputs(B, K_d, K_q, V, "bf16", seed=77, sigma_q=0.5, sigma_d=0.9)
    full = oracle.verify(workloads.to_host_bits(zd), workloads.to_host_bits(zq), workloads.to_host_bits(zt),
                         tok.numpy(), np.float32(0.3), np.float32(0.2), oracle.STRICT, 5, 8)
    want = np.stack([full["accept_len_q"], full["next_token_q"], full["accept_len"], full["next_token"]], 1)
    assert np.array_equal(sharded, want)
    assert 0 < full["accept_len_q"].sum() < B * K_d       # the case has accepted and rejected positions


def test_shard_batch_covers_the_batch_exactly():
    from paper_2510_12966_b200 import workloads
    for B in (0, 1, 5, 64, 257):
        for world in (1, 2, 3, 8):
            spans = [workloads.shard_batch(B, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [h - l for l, h in spans]
            assert max(sizes) - min(sizes) <= 1
