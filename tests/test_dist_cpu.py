"""The N > 1 path on CPU (gloo, world size 2): units are independent, so ranks own disjoint batch rows
and exchange nothing on the data path.  Checked here: the row partition bench.py uses, that a rank's
inputs are exactly its rows of the global seeded workload, that the oracle's results for a rank's rows
equal the same rows of a single-process run (so sharding changes no result), and the max-over-ranks
timing reduction."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from oracle.lola_oracle import LolaOracle, config_for
    from paper_2505_23666_b200.workloads import WorkloadInputs, small_case
    per_rank = 2
    wl = small_case("dist", batch=per_rank, n_q_heads=4, n_kv_heads=2, head_dim=16, feat_half=8, tokens=96, chunk=16,
                    window=16, sparse=24, dtype="f32", seed=5, decode_steps=3)
    inputs = WorkloadInputs(wl.with_(batch=per_rank * world))      # the global workload
    rows = bench.rank_rows(rank, per_rank)
    orc = LolaOracle(config_for(wl, batch=per_rank), inputs.W.astype(np.float64))
    outs = []
    for t in range(0, wl.tokens, wl.chunk):
        q, k, v = inputs.prefill_tokens(t, wl.chunk, batch_rows=rows)
        outs.append(orc.prefill_chunk(q, k, v))
    for sidx in range(wl.decode_steps):
        q, k, v = inputs.decode_token(sidx, batch_rows=rows)
        outs.append(orc.decode_step(q, k, v)[:, None])
    np.save(os.path.join(out_dir, f"out{rank}.npy"), np.concatenate([o.reshape(per_rank, -1) for o in outs], axis=1))
    # timing reduction: every rank must see the slowest rank's time
    ms = bench.max_over_ranks(10.0 + rank, world)
    bench.barrier(world)
    assert ms == 10.0 + (world - 1), ms
    dist.destroy_process_group()


def test_two_ranks_shard_batch_rows_without_exchange(tmp_path):
    world = 2
    port = 29500 + (os.getpid() % 500)
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    import bench
    from oracle.lola_oracle import LolaOracle, config_for
    from paper_2505_23666_b200.workloads import WorkloadInputs, small_case
    per_rank = 2
    assert bench.rank_rows(0, per_rank) == [0, 1] and bench.rank_rows(1, per_rank) == [2, 3]
    wl = small_case("dist", batch=per_rank * world, n_q_heads=4, n_kv_heads=2, head_dim=16, feat_half=8, tokens=96,
                    chunk=16, window=16, sparse=24, dtype="f32", seed=5, decode_steps=3)
    inputs = WorkloadInputs(wl)
    orc = LolaOracle(config_for(wl), inputs.W.astype(np.float64))
    outs = []
    for t in range(0, wl.tokens, wl.chunk):
        outs.append(orc.prefill_chunk(*inputs.prefill_tokens(t, wl.chunk)))
    for sidx in range(wl.decode_steps):
        outs.append(orc.decode_step(*inputs.decode_token(sidx))[:, None])
    full = np.concatenate([o.reshape(per_rank * world, -1) for o in outs], axis=1)
    got = np.concatenate([np.load(tmp_path / f"out{r}.npy") for r in range(world)], axis=0)
    assert np.array_equal(full, got)          # same arithmetic on the same rows: identical, not merely close
