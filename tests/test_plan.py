"""The host-side scheduler of evo_validate, through evo_plan_inspect (CPU only: the plan
looks at pointer values and sizes, never at tensor contents)."""
import ctypes as C

import numpy as np
import pytest

DESC = np.dtype([("n", "<u8"), ("ref", "<u8"), ("dtype", "<i4"), ("group", "<u4")], align=True)
RANGE = np.dtype([("tile_begin", "<u8"), ("tile_end", "<u8"), ("set_begin", "<u4"), ("set_end", "<u4")], align=True)
SUMMARY = np.dtype([("n_sets", "<u4"), ("n_ctas", "<u4"), ("n_parts", "<u4"), ("tile_elems", "<u4"), ("total_tiles", "<u8")], align=True)
F32, F16, BF16 = 1, 2, 3
ESIZE = {F32: 4, F16: 2, BF16: 2}


@pytest.fixture(scope="module")
def lib():
    from paper_2510_03760_b200 import build
    L = C.CDLL(build.build())
    L.evo_plan_inspect.restype = C.c_int
    L.evo_plan_inspect.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_int, C.c_uint32,
                                   C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    return L


def inspect(lib, cands, descs, max_ctas, ref=None, dtype=F32):
    cands = np.ascontiguousarray(cands, dtype=np.uint64)
    descs = np.ascontiguousarray(descs, dtype=DESC)
    summ = np.zeros(1, SUMMARY)
    ranges = np.zeros(max_ctas, RANGE)
    set_of = np.zeros(max(len(descs), 1), np.uint32)
    set_k = np.zeros(max(len(descs), 1), np.uint32)
    st = lib.evo_plan_inspect(cands.ctypes.data, ref, descs.ctypes.data, len(descs), dtype, max_ctas,
                              summ.ctypes.data, ranges.ctypes.data, set_of.ctypes.data, set_k.ctypes.data)
    return st, summ[0], ranges[: summ[0]["n_ctas"]], set_of[: len(descs)], set_k[: summ[0]["n_sets"]]


def coverage(summ, ranges, set_tiles):
    """Tiles walked per set, and that the runs are ordered, disjoint and gap-free."""
    walked = np.zeros(len(set_tiles), dtype=np.int64)
    cursor = (0, 0)
    weights = []
    for r in ranges:
        if r["set_begin"] > r["set_end"]:
            weights.append(0)
            continue
        sb, se, tb, te = int(r["set_begin"]), int(r["set_end"]), int(r["tile_begin"]), int(r["tile_end"])
        # skip sets without tiles when comparing with the cursor
        cs, ct = cursor
        while cs < len(set_tiles) and ct >= set_tiles[cs]:
            cs, ct = cs + 1, 0
        assert (sb, tb) == (cs, ct), "run does not start where the previous one ended"
        w = 0
        for s in range(sb, se + 1):
            t0 = tb if s == sb else 0
            t1 = te if s == se else set_tiles[s]
            assert 0 <= t0 <= t1 <= set_tiles[s]
            walked[s] += t1 - t0
            w += t1 - t0
        assert w > 0
        weights.append(w)
        cursor = (se, te)
    assert np.array_equal(walked, np.asarray(set_tiles)), "every tile exactly once"
    return weights


def tiles_of(n, dtype, tile_elems):
    per = tile_elems
    return (n + per - 1) // per


def test_shared_reference_becomes_one_set_and_cut_is_balanced(lib):
    n = 1 << 25
    descs = np.zeros(16, DESC)
    descs["n"], descs["ref"], descs["dtype"] = n, 0x7000_0000_0000, F32
    cands = 0x1000_0000_0000 + np.arange(16, dtype=np.uint64) * (n * 4)
    st, summ, ranges, set_of, set_k = inspect(lib, cands, descs, 444)
    assert st == 0 and summ["n_sets"] == 1 and set_k.tolist() == [16] and set(set_of.tolist()) == {0}
    tiles = tiles_of(n, F32, int(summ["tile_elems"]))
    assert summ["total_tiles"] == tiles and summ["n_ctas"] == 444 and tiles > 6 * 444
    w = coverage(summ, ranges, [tiles])
    assert max(w) - min(w) <= 1
    assert summ["n_parts"] == 444 * 16


def test_few_items_per_cta_split_a_large_set_for_balance(lib):
    """Every CTA gets work but fewer than six (set, tile) items: the members of one reference are spread over
    smaller sets (never below four members), so that the shares of the CTAs come out more even."""
    n = 1 << 22                                        # 1024 tiles for 444 CTAs
    descs = np.zeros(16, DESC)
    descs["n"], descs["ref"], descs["dtype"] = n, 0x7000_0000_0000, F32
    cands = 0x1000_0000_0000 + np.arange(16, dtype=np.uint64) * (n * 4)
    st, summ, ranges, set_of, set_k = inspect(lib, cands, descs, 444)
    assert st == 0 and summ["n_sets"] == 4 and set_k.tolist() == [4, 4, 4, 4]
    assert set_of.tolist() == [i // 4 for i in range(16)]
    tiles = tiles_of(n, F32, int(summ["tile_elems"]))
    w = coverage(summ, ranges, [tiles] * 4)
    assert max(w) <= 1.12 * (sum(w) / len(w))          # shares within one item (5 tiles) of a mean of 46
    # fewer items than CTAs (a small population): the members are spread over sets of 2 until there are items for
    # every CTA - 100 tiles x 8 sets = 800 items for 444 CTAs (sets of 4 would have given 400)
    descs["n"] = 100 * 4096
    st, summ, ranges, set_of, set_k = inspect(lib, cands, descs, 444)
    assert st == 0 and summ["n_sets"] == 8 and set_k.tolist() == [2] * 8 and summ["n_ctas"] == 444
    # a single tile per tensor: every member its own set, sixteen CTAs
    descs["n"] = 4096
    st, summ, ranges, set_of, set_k = inspect(lib, cands, descs, 444)
    assert st == 0 and summ["n_sets"] == 16 and set_k.tolist() == [1] * 16 and summ["n_ctas"] == 16


def test_more_members_than_a_set_holds(lib):
    descs = np.zeros(100, DESC)
    descs["n"], descs["ref"], descs["dtype"] = 50000, 0x7000_0000_0000, BF16
    cands = 0x1000_0000_0000 + np.arange(100, dtype=np.uint64) * 100096
    st, summ, ranges, set_of, set_k = inspect(lib, cands, descs, 8)
    assert st == 0 and set_k.tolist() == [32, 32, 32, 4]                  # 52 items for 8 CTAs: as large as sets get
    assert set_of.tolist() == [i // 32 for i in range(100)]
    tiles = tiles_of(50000, BF16, int(summ["tile_elems"]))
    coverage(summ, ranges, [tiles] * 4)
    st, summ, ranges, set_of, set_k = inspect(lib, cands, descs, 64)       # fewer items than CTAs: sets of 16
    assert st == 0 and set_k.tolist() == [16] * 6 + [4] and set_of.tolist() == [i // 16 for i in range(100)]
    coverage(summ, ranges, [tiles] * 7)


def test_ragged_mixed_population(lib):
    rng = np.random.default_rng(0)
    n_desc = 300
    descs = np.zeros(n_desc, DESC)
    descs["n"] = np.floor(2.0 ** rng.uniform(0, 22, n_desc)).astype(np.uint64)
    descs["n"][::17] = 0
    descs["dtype"] = rng.choice([F32, F16, BF16], n_desc)
    descs["ref"] = 0x7000_0000_0000 + np.arange(n_desc, dtype=np.uint64) * (1 << 26)
    descs["ref"][1::5] = descs["ref"][0]           # some share a reference (same n/dtype only if they match)
    descs["n"][1::5] = descs["n"][0]
    descs["dtype"][1::5] = descs["dtype"][0]
    cands = 0x1000_0000_0000 + np.arange(n_desc, dtype=np.uint64) * (1 << 26)
    for max_ctas in (1, 7, 148 * 3, 5000):
        st, summ, ranges, set_of, set_k = inspect(lib, cands, descs, max_ctas)
        assert st == 0
        tb = int(summ["tile_elems"])
        set_tiles = [None] * int(summ["n_sets"])
        weight_per_tile = [None] * int(summ["n_sets"])
        for i in range(n_desc):
            s = int(set_of[i])
            t = tiles_of(int(descs["n"][i]), int(descs["dtype"][i]), tb)
            assert set_tiles[s] in (None, t)
            set_tiles[s] = t
            weight_per_tile[s] = int(set_k[s]) + 1
        assert sum(set_k.tolist()) == n_desc
        assert 0 < summ["n_ctas"] <= min(max_ctas, sum(set_tiles))
        assert summ["n_ctas"] >= min(max_ctas, sum(set_tiles)) // 2         # few runs are lost to heavy items
        assert all(r["set_begin"] <= r["set_end"] for r in ranges)          # no idle CTA is launched
        coverage(summ, ranges, set_tiles)
        # weighted balance: no CTA carries more than its share plus one heaviest item
        total = sum(t * w for t, w in zip(set_tiles, weight_per_tile))
        heaviest = max(weight_per_tile)
        for r in ranges:
            if r["set_begin"] > r["set_end"]:
                continue
            wsum = 0
            for s in range(int(r["set_begin"]), int(r["set_end"]) + 1):
                t0 = int(r["tile_begin"]) if s == r["set_begin"] else 0
                t1 = int(r["tile_end"]) if s == r["set_end"] else set_tiles[s]
                wsum += (t1 - t0) * weight_per_tile[s]
            assert wsum <= total / len(ranges) + 2 * heaviest


def test_heavy_items_with_few_tiles_leave_no_idle_cta(lib):
    # 40 members of 3 tiles each: 12 items of very different weight, fewer runs than items
    descs = np.zeros(80, DESC)
    descs["n"], descs["dtype"] = 10000, F16
    descs["ref"][:40], descs["ref"][40:] = 0x7000_0000_0000, 0x7100_0000_0000
    cands = 0x1000_0000_0000 + np.arange(80, dtype=np.uint64) * 65536
    st, summ, ranges, set_of, set_k = inspect(lib, cands, descs, 2)
    assert st == 0 and set_k.tolist() == [32, 8, 32, 8] and summ["total_tiles"] == 12
    assert all(r["set_begin"] <= r["set_end"] for r in ranges) and 0 < summ["n_ctas"] <= 2
    coverage(summ, ranges, [3, 3, 3, 3])
    st, summ, ranges, set_of, set_k = inspect(lib, cands, descs, 11)       # boundaries inside heavy items: no empty run
    assert st == 0 and all(r["set_begin"] <= r["set_end"] for r in ranges) and 0 < summ["n_ctas"] <= 11
    coverage(summ, ranges, [3] * int(summ["n_sets"]))
    # with CTAs to spare the same tensors are spread out: one member per set, 240 light items
    st, summ, ranges, set_of, set_k = inspect(lib, cands, descs, 444)
    assert st == 0 and set_k.tolist() == [1] * 80 and summ["total_tiles"] == 240 and summ["n_ctas"] == 240
    coverage(summ, ranges, [3] * 80)


def test_empty_and_zero_length(lib):
    st, summ, ranges, _, _ = inspect(lib, [], np.zeros(0, DESC), 10)
    assert st == 0 and summ["n_ctas"] == 0 and summ["n_sets"] == 0
    descs = np.zeros(3, DESC)
    descs["dtype"] = F32
    st, summ, ranges, set_of, set_k = inspect(lib, [0, 0, 0], descs, 10)
    assert st == 0 and summ["n_ctas"] == 0 and summ["total_tiles"] == 0


def test_argument_errors(lib):
    good = np.zeros(1, DESC)
    good["n"], good["ref"], good["dtype"] = 10, 0x7000_0000_0000, F32
    assert inspect(lib, [0x1000], good, 4)[0] == 0
    bad = good.copy(); bad["dtype"] = 7
    assert inspect(lib, [0x1000], bad, 4)[0] == -3
    bad = good.copy(); bad["dtype"] = -1
    assert inspect(lib, [0x1000], bad, 4, dtype=0)[0] == -3          # raw words are not a tensor type here
    assert inspect(lib, [0x1000], bad, 4, dtype=F16)[0] == 0
    assert inspect(lib, [0x1002], good, 4)[0] == -2                   # candidate not 4-byte aligned
    bad = good.copy(); bad["ref"] = 0x7000_0000_0001
    assert inspect(lib, [0x1000], bad, 4)[0] == -2
    bad = good.copy(); bad["ref"] = 0
    assert inspect(lib, [0x1000], bad, 4)[0] == -1                    # no reference at all
    assert inspect(lib, [0x1000], bad, 4, ref=0x7000_0000_0000)[0] == 0   # call-level reference
    assert inspect(lib, [0], good, 4)[0] == -1
    assert inspect(lib, [0x1000], good, 0)[0] == -1


def test_unaligned_tensors_are_scheduled_too(lib):
    descs = np.zeros(2, DESC)
    descs["n"], descs["ref"], descs["dtype"] = 100000, 0x7000_0000_0004, F32
    st, summ, ranges, set_of, set_k = inspect(lib, [0x1000_0000, 0x2000_0008], descs, 16)
    assert st == 0 and summ["n_sets"] == 1
    coverage(summ, ranges, [tiles_of(100000, F32, int(summ["tile_elems"]))])
