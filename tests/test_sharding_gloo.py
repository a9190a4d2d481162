"""The multi-process path on CPU: two gloo ranks split one search by rank windows, each
searches its windows (with the CPU oracle standing in for the GPU library, which this test
does not need), and the merged result must equal the unsharded search."""
import os
import socket

import torch.multiprocessing as mp

import oracle
from paper_2505_02146_b200.sharding import merge_results, shard_rank_windows
from xp_instances import Hole, Sketch, Variable, constant_set, free_grammar, parse_expr


def _sketch(spec):
    vs = [Variable("i", 0, 16), Variable("j", 0, 16)]
    g = free_grammar(vs, constant_set(-8, 8))
    return Sketch(g, [Hole(0, 5, spec_expr=parse_expr(spec, vs))])


def _worker(rank, world, port, spec, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sk = _sketch(spec)
    cand = oracle.counts(sk.grammar, 0, 5)
    windows = shard_rank_windows(cand, world, rank)
    local = oracle.repair_hole(sk, rank_ranges={s: (b, e) for _, s, b, e in windows})
    merged = merge_results(local.match_count, local.solved, local.least_size, local.least_rank)
    out[rank] = (windows, merged)
    dist.destroy_process_group()


def test_windows_partition_every_size():
    cand = [0, 19, 0, 1805, 0, 342950]
    for world in (1, 2, 3, 7, 20):
        for size, n in enumerate(cand):
            if size == 0:
                continue
            pieces = [w for r in range(world) for w in shard_rank_windows(cand, world, r) if w[1] == size]
            assert pieces[0][2] == 0 and pieces[-1][3] == n
            assert all(a[3] == b[2] for a, b in zip(pieces[:-1], pieces[1:]))
            lens = [w[3] - w[2] for w in pieces]
            assert max(lens) - min(lens) <= 1


def test_two_gloo_ranks_merge_to_the_unsharded_result():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    for spec in ["(i*8)+j", "i%4", "100"]:
        full = oracle.repair_hole(_sketch(spec))
        out = mp.Manager().dict()
        mp.spawn(_worker, args=(2, port, spec, out), nprocs=2, join=True)
        assert out[0][1] == out[1][1]
        counts, solved, lsize, lrank = out[0][1]
        assert counts == full.match_count and solved == full.solved
        if solved:
            assert (lsize, lrank) == (full.least_size, full.least_rank)
