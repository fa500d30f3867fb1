"""Two gloo ranks on CPU: the token split covers a batch exactly once, the codec steps are
independent per token (so shards need no exchange), and timings are reduced with MAX."""

import os
import socket

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import ssn_oracle as oracle
from paper_2607_13332_b200 import dist_util, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert dist_util.rank_world() == (rank, world, rank)
        wl = synth.Workload("mr", d=64, k=8, vocab=50, batch=3, seq_len=11, dtype=synth.F32)
        t = synth.codec_inputs(wl, seed=77)           # same seed: every rank sees the same batch
        mine = synth.shard_tokens(wl.n_tokens, rank, world)
        sel = np.arange(mine.start, mine.stop)
        f = lambda a: synth.to_f64(a, wl.dtype)
        pos = oracle.token_positions(wl.n_tokens, wl.seq_len)
        Z, _ = oracle.compress(f(t["X"])[sel], f(t["U"]), f(t["E"]), t["ids"][sel], f(t["P"]), pos[sel])
        np.save(os.path.join(out_dir, f"z{rank}.npy"), Z)
        np.save(os.path.join(out_dir, f"sel{rank}.npy"), sel)
        dist_util.barrier()
        slowest = dist_util.max_over_ranks(1.0 + rank)
        assert slowest == float(world)
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_without_exchange(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = synth.Workload("mr", d=64, k=8, vocab=50, batch=3, seq_len=11, dtype=synth.F32)
    t = synth.codec_inputs(wl, seed=77)
    f = lambda a: synth.to_f64(a, wl.dtype)
    pos = oracle.token_positions(wl.n_tokens, wl.seq_len)
    full, _ = oracle.compress(f(t["X"]), f(t["U"]), f(t["E"]), t["ids"], f(t["P"]), pos)
    sels = [np.load(tmp_path / f"sel{r}.npy") for r in range(world)]
    assert np.array_equal(np.concatenate(sels), np.arange(wl.n_tokens))
    got = np.concatenate([np.load(tmp_path / f"z{r}.npy") for r in range(world)])
    np.testing.assert_array_equal(got, full)      # per-token independence: bit for bit


def test_single_process_helpers_are_no_ops():
    assert dist_util.max_over_ranks(3.5) == 3.5
    dist_util.barrier()
