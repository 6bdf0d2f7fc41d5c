"""Pins for the integer pool model: hand-computed block tables and the invariants the
paper states for fork and release (Section 2.3 "Decoding")."""
import os
import random

import pytest

from oracle import BlockModel, BookkeepingError

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def load_golden(name):
    out = {"table": {}, "len": {}}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, _, val = line.partition(":")
        parts = key.split()
        if parts[0] in ("table", "len"):
            vals = [int(x) for x in val.split()]
            out[parts[0]][int(parts[1])] = vals if parts[0] == "table" else vals[0]
        elif parts[0] == "copies":
            out["copies"] = [tuple(int(x) for x in c.split()) for c in val.split(",") if c.strip()]
        elif parts[0] in ("refcount", "in_use_after_event", "peak_after_event", "free_list"):
            out[parts[0]] = [int(x) for x in val.split()]
        else:
            out[parts[0]] = int(val)
    return out


def check_against_golden(m, g, copies):
    assert copies == g["copies"]
    for t, table in g["table"].items():
        assert m.tables[t] == table
        assert m.lens[t] == g["len"][t]
    n = len(g["refcount"])
    assert m.refcount[:n] == g["refcount"] and not any(m.refcount[n:])
    leaves = [1, 2, 3]
    assert len({b for t in leaves for b in m.tables[t]}) == g["unique_blocks"]
    assert sum(len(m.tables[t]) for t in leaves) == g["unshared_blocks"]
    assert m.unique_tokens(leaves) == g["unique_tokens"]
    assert m.attended_tokens(leaves) == g["unshared_tokens"]


def test_prompt64_hand_computed():
    g = load_golden("fork_tables_prompt64.txt")
    m = BlockModel(32, g["block_size"], 8, 16)
    (p,) = m.new_threads(1)
    m.append([p], [64])
    kids, copies = m.fork([p, p, p])
    assert kids == [1, 2, 3]
    m.append(kids, [31, 16, 39])
    slots = m.append(kids)
    assert slots == [[(5, 15)], [(10, 0)], [(9, 7)]]
    check_against_golden(m, g, copies)
    assert m.peak_used == g["peak_used_blocks"] == 11


def test_prompt70_hand_computed_copy_on_fork():
    g = load_golden("fork_tables_prompt70.txt")
    m = BlockModel(32, g["block_size"], 8, 16)
    (p,) = m.new_threads(1)
    m.append([p], [70])
    kids, copies = m.fork([p, p, p])
    check_against_golden(m, g, copies)
    assert m.peak_used == g["peak_used_blocks"] == 8
    assert m.cow_blocks == 3 and m.cow_rows == 18
    # parent keeps its own partial block and appends in place; children use their copies
    assert m.append([p] + kids) == [[(4, 6)], [(5, 6)], [(6, 6)], [(7, 6)]]


def release_refork_events():
    """The events of golden/release_refork_peak.txt as (method, arguments) on thread ids."""
    return [("new+append", 40), ("fork", 0), ("append", 1, 30), ("release", 1), ("fork", 0),
            ("append", 2, 9), ("append", 2, 17), ("append", 0, 1), ("append", 0, 24)]


def test_peak_of_blocks_in_use_hand_computed():
    g = load_golden("release_refork_peak.txt")
    m = BlockModel(g["num_blocks"], g["block_size"], 8, 16)
    in_use, peak = [], []
    for ev in release_refork_events():
        if ev[0] == "new+append":
            (t,) = m.new_threads(1)
            m.append([t], [ev[1]])
        elif ev[0] == "fork":
            m.fork([ev[1]])
        elif ev[0] == "append":
            m.append([ev[1]], [ev[2]])
        else:
            m.release([ev[1]])
        in_use.append(m.used_blocks())
        peak.append(m.peak_used)
    assert in_use == g["in_use_after_event"]
    assert peak == g["peak_after_event"]          # taking freed blocks again does not move it
    for t, table in g["table"].items():
        assert m.tables[t] == table and m.lens[t] == g["len"][t]


def invariants(m):
    entries = [b for t in m.tables.values() for b in t]
    assert sum(m.refcount) == len(entries)
    for b in range(m.num_blocks):
        assert m.refcount[b] == entries.count(b)
    used = {b for b in range(m.num_blocks) if m.refcount[b] > 0}
    assert len(m.free) == len(set(m.free)) and not (set(m.free) & used)
    assert len(m.free) + len(used) == m.num_blocks
    for t, table in m.tables.items():
        assert len(table) == -(-m.lens[t] // m.block_size)


def test_random_replay_keeps_invariants_and_fork_rule():
    rnd = random.Random(11)
    m = BlockModel(400, 16, 64, 40)
    live = m.new_threads(3)
    m.append(live, [rnd.randrange(1, 100) for _ in live])
    for step in range(300):
        op = rnd.random()
        try:
            if op < 0.25 and live:
                parents = [rnd.choice(live) for _ in range(rnd.randrange(1, 4))]
                before = {p: (list(m.tables[p]), m.lens[p]) for p in parents}
                used0 = m.used_blocks()
                kids, copies = m.fork(parents)
                assert len(copies) <= len(parents)
                assert m.used_blocks() - used0 == len(copies)     # <= 1 block per fork
                for p, c in zip(parents, kids):
                    tp, lp = before[p]
                    full, r = divmod(lp, 16)
                    assert m.tables[c][:full] == tp[:full]       # all full blocks shared
                    assert len(m.tables[c]) == -(-lp // 16) and m.lens[c] == lp
                    if r:
                        assert m.tables[c][-1] not in tp and m.refcount[m.tables[c][-1]] == 1
                    assert m.tables[p] == tp                     # parent untouched
                live += kids
            elif op < 0.85 and live:
                sub = rnd.sample(live, rnd.randrange(1, len(live) + 1))
                m.append(sub, [rnd.randrange(0, 20) for _ in sub])
            elif live:
                sub = rnd.sample(live, rnd.randrange(1, min(3, len(live)) + 1))
                m.release(sub)
                live = [t for t in live if t not in sub]
        except BookkeepingError as e:
            assert e.code in ("NO_BLOCKS", "NO_THREADS", "TABLE_FULL")
        invariants(m)
    m.release(live)
    assert len(m.free) == m.num_blocks and not any(m.refcount)   # only-own cache freed, all of it


def test_release_frees_only_blocks_no_one_else_holds():
    m = BlockModel(16, 16, 8, 8)
    (p,) = m.new_threads(1)
    m.append([p], [40])                 # blocks 0,1,2 (8 rows in block 2)
    (c,), copies = m.fork([p])
    assert copies == [(2, 3, 8)]
    m.append([c], [10])                 # fills block 3, opens block 4
    m.release([c])
    assert m.free_list()[:2] == [4, 3] and m.refcount[:3] == [1, 1, 1]
    (c2,), _ = m.fork([p])
    assert m.tables[c2] == [0, 1, 4]    # last-in first-out reuse
    m.release([p])
    assert m.refcount[:3] == [1, 1, 0] and m.free_list()[0] == 2
    with pytest.raises(BookkeepingError):
        m.append([p])


def test_failed_calls_change_nothing():
    m = BlockModel(6, 16, 4, 4)
    a, b = m.new_threads(2)
    m.append([a, b], [20, 17])          # 2 + 2 blocks, 2 free
    snap = (dict((t, list(v)) for t, v in m.tables.items()), dict(m.lens), list(m.free),
            list(m.refcount), m.next_tid)

    def same():
        return snap == (dict((t, list(v)) for t, v in m.tables.items()), dict(m.lens),
                        list(m.free), list(m.refcount), m.next_tid)

    for call, code in [
        (lambda: m.fork([a, b, a]), "NO_THREADS"),
        (lambda: m.append([a, b], [30, 30]), "NO_BLOCKS"),
        (lambda: m.append([a], [60]), "TABLE_FULL"),
        (lambda: m.append([a, a]), "INVALID_ARG"),
        (lambda: m.append([a, 99]), "BAD_THREAD"),
        (lambda: m.release([a, a]), "BAD_THREAD"),
        (lambda: m.fork([7]), "BAD_THREAD"),
    ]:
        with pytest.raises(BookkeepingError) as e:
            call()
        assert e.value.code == code and same()
    m2 = BlockModel(5, 16, 8, 3)
    x, y = m2.new_threads(2)
    m2.append([x, y], [20, 17])
    with pytest.raises(BookkeepingError) as e:
        m2.fork([x, y])                 # needs 2 copies, 1 block free
    assert e.value.code == "NO_BLOCKS" and len(m2.tables) == 2 and len(m2.free) == 1


def accept_events():
    """The events of tests/golden/accept_candidates.txt."""
    return [("new+append", 37), ("append", 0, 5), ("accept", 0, 5, 2), ("append", 0, 12),
            ("accept", 0, 12, 1), ("fork", 0), ("append", 0, 30), ("accept", 0, 30, 0),
            ("append", 1, 10), ("accept", 1, 10, 10), ("accept-refused", 0, 9, 0)]


def test_accept_of_speculated_rows_against_the_hand_worked_events():
    g = load_golden("accept_candidates.txt")
    m = BlockModel(g["num_blocks"], g["block_size"], 8, 16)
    in_use, peak = [], []
    for ev in accept_events():
        if ev[0] == "new+append":
            (t,) = m.new_threads(1)
            m.append([t], [ev[1]])
        elif ev[0] == "append":
            m.append([ev[1]], [ev[2]])
        elif ev[0] == "fork":
            m.fork([ev[1]])
        elif ev[0] == "accept":
            m.accept([ev[1]], [ev[2]], [ev[3]])
        else:
            before = (dict(m.lens), {t: list(b) for t, b in m.tables.items()}, list(m.free))
            with pytest.raises(BookkeepingError) as e:
                m.accept([ev[1]], [ev[2]], [ev[3]])
            assert e.value.code == "INVALID_ARG"
            assert before == (m.lens, m.tables, m.free)
        in_use.append(m.used_blocks())
        peak.append(m.peak_used)
    assert in_use == g["in_use_after_event"] and peak == g["peak_after_event"]
    assert m.tables == g["table"] and m.lens == g["len"]
    assert m.refcount == g["refcount"] and m.free_list() == g["free_list"]
