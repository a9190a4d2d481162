"""Writes the full-size expected results under tests/golden/ by running the CPU oracle (and
nothing else) over disjoint rank windows in parallel processes and merging them: counts add,
the least solution is the one of the lowest window that has a match.

    python tests/golden/make_full_goldens.py [--procs N] [config2 config3 config4 config5]

Single-core cost is about 1-2 h per large config; with N processes it divides by N.
"""
from __future__ import annotations

import argparse
import json
import multiprocessing as mp
import os
import sys
import time

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _sketch(name: str, seed: int, index: int = 0):
    from xp_instances import config2, config3, config4, config5_instance
    if name == "config2": return config2(seed)
    if name == "config3": return config3(seed)
    if name == "config4": return config4(seed)
    if name == "config5": return config5_instance(seed, index)
    raise KeyError(name)


def _corner_ids(sk):
    """Point ids of the box corners (tried first: results do not depend on the order)."""
    if sk.coords is not None:
        return list(range(min(64, sk.n_points)))
    ext = [v.hi - v.lo for v in sk.grammar.variables]
    ids = []
    for mask in range(1 << len(ext)):
        pid = 0
        for d, e in enumerate(ext):
            pid = pid * e + ((e - 1) if (mask >> d) & 1 else 0)
        ids.append(pid)
    return sorted(set(ids))


def _work(job):
    import oracle
    name, seed, index, hole, size, lo, hi = job
    sk = _sketch(name, seed, index)
    K = sk.holes[hole].max_size
    rr = {s: (0, 0) for s in range(1, K + 1)}
    rr[size] = (lo, hi)
    r = oracle.repair_hole(sk, hole, rank_ranges=rr, first_points=_corner_ids(sk))
    return (name, seed, index, hole, size, lo, r.match_count[size], r.solved, r.least_rank, r.least_text, r.cand_count)


def _work_whole(job):
    import oracle
    name, seed, index = job
    sk = _sketch(name, seed, index)
    r = oracle.repair_hole(sk, 0)
    return index, [r.match_count[1], r.match_count[3], r.match_count[5], r.least_size if r.solved else 0,
                   r.least_rank if r.solved else 0]


def run_large(pool, name: str, seed: int, shard: int):
    import oracle
    sk = _sketch(name, seed)
    jobs = []
    for h, hole in enumerate(sk.holes):
        cnt = oracle.counts(sk.grammar, hole.start_nt, hole.max_size)
        for size in range(1, hole.max_size + 1):
            for lo in range(0, cnt[size], shard):
                jobs.append((name, seed, 0, h, size, lo, min(cnt[size], lo + shard)))
    jobs.sort(key=lambda j: -(j[6] - j[5]))
    out = [{"cand_count": None, "match_count": [0] * (hole.max_size + 1), "solved": False, "least_size": 0,
            "least_rank": 0, "least_text": "", "planted": hole.note} for hole in sk.holes]
    best = [None] * len(sk.holes)
    t0 = time.time()
    for n, (_, _, _, h, size, lo, m, solved, lrank, ltext, cand) in enumerate(pool.imap_unordered(_work, jobs)):
        out[h]["cand_count"] = cand
        out[h]["match_count"][size] += m
        if solved and (best[h] is None or (size, lrank) < best[h][:2]):
            best[h] = (size, lrank, ltext)
        if n % 50 == 0:
            print(f"{name}: {n + 1}/{len(jobs)} windows, {time.time() - t0:.0f} s", flush=True)
    for h, b in enumerate(best):
        if b:
            out[h].update(solved=True, least_size=b[0], least_rank=b[1], least_text=b[2])
    path = os.path.join(HERE, f"{name}_seed{seed}_full.json")
    json.dump({"config": name, "seed": seed, "written_by": "tests/golden/make_full_goldens.py (CPU oracle only)",
               "holes": out}, open(path, "w"), indent=1)
    print("wrote", path, f"{time.time() - t0:.0f} s", flush=True)


def run_batch(pool, seed: int, n_instances: int):
    rows = [None] * n_instances
    for index, row in pool.imap_unordered(_work_whole, [("config5", seed, i) for i in range(n_instances)], chunksize=8):
        rows[index] = row
    path = os.path.join(HERE, f"config5_seed{seed}_full.txt")
    with open(path, "w") as f:
        f.write("# config 5, seed %d: one line per instance: match_count at sizes 1 3 5, least size (0 = no solution), least rank\n" % seed)
        f.write("# written by tests/golden/make_full_goldens.py (CPU oracle only)\n")
        for row in rows:
            f.write(" ".join(str(x) for x in row) + "\n")
    print("wrote", path, flush=True)


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--procs", type=int, default=max(1, (os.cpu_count() or 2) - 1))
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--shard", type=int, default=400_000_000)
    ap.add_argument("configs", nargs="*", default=["config5", "config3", "config2", "config4"])
    a = ap.parse_args()
    import oracle
    oracle.build()
    with mp.get_context("spawn").Pool(a.procs) as pool:
        for c in a.configs:
            if c == "config5":
                run_batch(pool, a.seed, 4096)
            else:
                run_large(pool, c, a.seed, a.shard)
