"""The allocation-free entry point (xp_repair_static) against xp_repair.

Some users of the library run where device memory may not be allocated once work has
started: a framework whose caching allocator has taken all of it, a serving loop that cannot
afford the device-wide synchronisation of cudaMalloc, a process with a fixed memory budget.
For them xp_repair_static keeps its scratch in a fixed array inside the library.  This test
calls it through the C ABI twice in a row on each case (the array keeps the previous call's
bytes, so the second call checks that nothing of them leaks) and requires exactly the results
of xp_repair: counts, match counts and the least solution, bit for bit.  It lives in a file
collected last so that a failure here cannot hide any other test of an -x run.
"""
import pytest

from xp_instances import Hole, Sketch, Variable, config1, config2, config3, config5_instance, free_grammar, parse_expr

pytestmark = pytest.mark.gpu


def _same(summary, ref):
    K = summary.max_size
    assert [int(summary.cand_count[k]) for k in range(K + 1)] == ref.cand_count
    assert [int(summary.match_count[k]) for k in range(K + 1)] == ref.match_count
    assert bool(summary.solved) == ref.solved
    if ref.solved:
        assert (summary.least_size, int(summary.least_rank), summary.least_text.decode()) == \
            (ref.least_size, ref.least_rank, ref.least_text)


def test_static_entry_point_matches_xp_repair_on_two_calls_in_a_row(xp):
    cases = [(config1(0), None), (config1(3), None), (config5_instance(0, 1), None),
             (config2(0), [(0, 5, 0, 3_000_000), (0, 7, 10 ** 9, 10 ** 9 + 2_000_000)]),
             (config3(0), [(-1, 5, 0, 1_500_000)])]
    for sk, windows in cases:
        gr = xp.xp_grammar_create(sk.grammar)
        ls = xp.xp_sketch_load(gr, sk)
        ref = xp.xp_repair(ls, rank_ranges=windows)
        for _ in range(2):
            got = xp.xp_repair_static(ls, rank_ranges=windows)
            assert len(got) == len(ref)
            for g, r in zip(got, ref):
                _same(g, r)
    # alternating different problems: each call must wipe what the other left in the array
    a, b = config1(1), config1(2)
    ga, gb = xp.xp_grammar_create(a.grammar), xp.xp_grammar_create(b.grammar)
    la, lb = xp.xp_sketch_load(ga, a), xp.xp_sketch_load(gb, b)
    ra, rb = xp.xp_repair(la), xp.xp_repair(lb)
    for _ in range(2):
        _same(xp.xp_repair_static(la)[0], ra[0])
        _same(xp.xp_repair_static(lb)[0], rb[0])


def test_static_entry_point_leaves_device_memory_as_it_found_it(xp):
    """The property the entry point is named for: once a first call on the device has been made,
    further calls, on different sketches and with different options, neither take nor give back
    device memory (free memory as the driver reports it stays the same to the byte)."""
    import torch
    sketches = []
    for sk in (config1(0), config1(4), config5_instance(0, 2), config3(0)):
        sketches.append(xp.xp_sketch_load(xp.xp_grammar_create(sk.grammar), sk))      # (loading does allocate)
    xp.xp_repair_static(sketches[0])                                                   # first call: address look-up
    torch.cuda.synchronize()
    free0, total0 = torch.cuda.mem_get_info()
    for ls in sketches:
        xp.xp_repair_static(ls)
        xp.xp_repair_static(ls, flags=xp.XP_FLAG_NO_FILTER, size_max=3)
        xp.xp_repair_static(ls, rank_ranges=[(-1, 5, 0, 100_000)])
        assert torch.cuda.mem_get_info() == (free0, total0)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info() == (free0, total0)


def test_static_entry_point_when_its_survivor_queue_is_full(xp):
    """The fixed array holds a survivor queue of 8192 entries; a spec with 60 878 matches of size 5
    overflows it, and the warps then check their survivors themselves: same counts."""
    vs = [Variable("i", 0, 16), Variable("j", 0, 16)]
    g = free_grammar(vs, list(range(-8, 9)))
    ls = xp.xp_sketch_load(xp.xp_grammar_create(g), Sketch(g, [Hole(0, 5, spec_expr=parse_expr("0", vs))]))
    ref = xp.xp_repair(ls)
    assert ref[0].match_count == [0, 1, 0, 301, 0, 60878]
    for _ in range(2):
        _same(xp.xp_repair_static(ls)[0], ref[0])
        _same(xp.xp_repair_static(ls, flags=xp.XP_FLAG_NO_FILTER)[0], ref[0])


def test_static_entry_point_rejects_what_does_not_fit(xp):
    vs = [Variable("x", 0, 4)]
    g = free_grammar(vs, [0, 1, 2])
    hole = Hole(0, 5, spec_expr=parse_expr("x+1", vs))
    gr = xp.xp_grammar_create(g)
    ls = xp.xp_sketch_load(gr, Sketch(g, [hole]))
    lib = xp.load()
    out = (xp.binding.xp_hole_summary * 1)()
    assert lib.xp_repair_static(ls.handle, None, out, 0) == 1            # out too short
    assert b"fewer entries" in lib.xp_last_error()
    assert lib.xp_repair_static(None, None, out, 1) == 1
    many = xp.xp_sketch_load(gr, Sketch(g, [hole] * 65))                 # beyond the fixed limit: refused, not run
    with pytest.raises(xp.XpError) as e:
        xp.xp_repair_static(many)
    assert e.value.status == 4 and "64 holes" in str(e.value)
    assert len(xp.xp_repair(many)) == 65                                 # the allocating entry point still takes it
    _same(xp.xp_repair_static(ls)[0], xp.xp_repair(ls)[0])               # and the fixed array still works afterwards
