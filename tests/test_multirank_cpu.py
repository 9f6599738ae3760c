"""World-size-2 run on CPU (gloo): the rank plumbing used for N > 1 GPUs.

Ranks take disjoint ciphertext-index ranges, never exchange polynomials, and the results of
the shards put together equal the single-process result; the step time is the max over ranks."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from paper_2207_04604_b200 import workloads as wl


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _shard_sums(rank, world, cts_per_rank, seed, total_cts):
    """The oracle stands in for the per-rank GPU work: the test is about the plumbing."""
    from common import make_oracle

    cfg = wl.RoundConfig("tiny", 3, 2, 5, 36, 2, 32 * total_cts, 0.0, int_range=500)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed)
    parties = list(range(cfg.num_parties))
    offsets, rows = wl.regular_graph(cfg.num_parties, cfg.degree, seed)
    first, cnt = wl.shard_ct_range(rank, world, cts_per_rank)
    values = wl.gradients(cfg, seed, first, cnt)
    pk = o.collective_pk(parties)
    ct = o.encrypt(pk, parties, first, o.encode(values))
    agg = o.aggregate(ct, offsets, rows)
    shares = o.partial_decrypt(agg, parties, parties, first)
    return o.decode(o.combine(agg, shares)), values, offsets, rows


def _worker(rank, world, port, out_dir):
    import sys

    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2207_04604_b200 import parallel

    r, lr, w = parallel.init("gloo")
    assert (r, w) == (rank, world)
    parallel.barrier()
    sums, _, _, _ = _shard_sums(rank, world, 2, seed=3, total_cts=2 * world)
    slowest = parallel.max_over_ranks(10.0 + rank)
    assert slowest == 10.0 + world - 1
    whole = parallel.gather_to_rank0(torch.from_numpy(sums))
    parallel.barrier()
    if rank == 0:
        np.save(os.path.join(out_dir, "whole.npy"), whole.numpy())
    else:
        assert whole is None
    parallel.finish()


def test_two_ranks_cover_the_round_without_exchange(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    got = np.load(tmp_path / "whole.npy")
    # single-process result over the whole index range
    sums, values, offsets, rows = _shard_sums(0, 1, 2 * world, seed=3, total_cts=2 * world)
    assert got.shape == sums.shape
    assert np.array_equal(got, sums)
    for i in range(3):
        assert np.array_equal(sums[i], values[rows[offsets[i]:offsets[i + 1]]].sum(axis=0))


def test_single_process_helpers_are_noops():
    from paper_2207_04604_b200 import parallel

    assert parallel.max_over_ranks(3.5) == 3.5
    t = torch.arange(6).reshape(1, 6)
    assert parallel.gather_to_rank0(t) is t
    parallel.barrier()
