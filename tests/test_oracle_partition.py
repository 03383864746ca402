"""Pins for the oracle's hierarchical workload partitioning (paper Sec. 6.2, App. B to D):
expert windows, peer windows, transfer units with cost alpha + s/beta, LPT-style list scheduling under
a stripe-level fan-out cap.  None of these re-run the oracle's own greedy loop: they use hand-worked
schedules (Graham's tight instances), a brute-force optimum, closed-form unit counts, and the
requirement that window-major dispatch writes exactly what token-major dispatch writes."""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2607_26444_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
BIG = 1 << 40


def units_to_layout(units, R):
    """A layout whose peer windows are exactly the given units: one expert per rank (E = R), source rank r
    sends `cost` rows to expert d for the i-th unit (r, d) in id order.  Units are (cost, dest)."""
    sec = np.zeros((R, R), np.int32)
    r = 0
    last_d = -1
    for cost, d in units:
        if d <= last_d:          # unit ids enumerate (r, d): start a new source rank when d does not increase
            r += 1
        assert r < R and sec[r, d] == 0
        sec[r, d] = cost
        last_d = d
    off = np.concatenate([[0], np.cumsum(sec.sum(axis=0))]).astype(np.int32)
    return {"src_expert_count": sec, "expert_offset": off}


def parse_golden():
    rows = []
    with open(os.path.join(GOLDEN, "lpt_examples.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            name, cores, cap, units, loads, opt, stripes = [s.strip() for s in line.split("|")]
            us = [(int(u.split("@")[0]), int(u.split("@")[1])) for u in units.split()]
            rows.append((name, int(cores), int(cap), us, [int(v) for v in loads.split()], int(opt),
                         [[int(v) for v in core.split()] for core in stripes.split(";")]))
    return rows


@pytest.mark.parametrize("case", parse_golden(), ids=lambda c: c[0])
def test_hand_worked_schedules(case):
    name, cores, cap, units, loads, opt, stripes = case
    R = 8
    lay = units_to_layout(units, R)
    # cost = rows exactly: alpha 0, beta = row_bytes, one unit per peer window
    part = oracle.partition(lay, row_bytes=64, n_cores=cores, tiers=[(0, 64, BIG, cap)])
    assert part["n_units"] == len(units)
    assert part["unit_cost"].tolist() == [u[0] for u in units]
    assert part["unit_desc"][:, 1].tolist() == [u[1] for u in units]
    assert part["core_load"].tolist() == loads
    got = [part["task_stripe"][part["task_offset"][c]:part["task_offset"][c + 1]].tolist() for c in range(cores)]
    assert got == stripes
    assert max(loads) <= (4 / 3 - 1 / (3 * cores)) * opt + 1e-9      # the cap never costs makespan: classical bound


def brute_force_optimum(costs, C):
    best = sum(costs)
    for assign in itertools.product(range(C), repeat=len(costs)):
        loads = [0] * C
        for c, a in zip(costs, assign):
            loads[a] += c
        best = min(best, max(loads))
    return best


@pytest.mark.parametrize("seed", range(12))
def test_lpt_bound_against_brute_force_optimum(seed):
    rng = np.random.default_rng(seed)
    C = int(rng.choice([2, 3]))
    n = int(rng.integers(3, 9))
    R = 3
    costs = rng.integers(1, 30, size=n).tolist()
    dests = [i % R for i in range(n)]
    lay = units_to_layout(list(zip(costs, dests)), R=8)
    part = oracle.partition(lay, row_bytes=2, n_cores=C, tiers=[(0, 2, BIG, 99)])
    assert sorted(part["unit_cost"].tolist()) == sorted(costs)
    makespan = int(part["core_load"].max())
    assert part["core_load"].sum() == sum(costs)
    opt = brute_force_optimum(costs, C)
    assert opt <= makespan <= (4 / 3 - 1 / (3 * C)) * opt + 1e-9


def schedule_tables(part, R):
    """How often every unit is scheduled, and the fan-out table F[stripe][dest] rebuilt from the task lists and
    their stripes; also checks that a core's stripes strictly increase (at most one unit per core and stripe)."""
    C = part["task_offset"].size - 1
    U = part["n_units"]
    seen = np.zeros(U, np.int32)
    F = np.zeros((int(part["task_stripe"].max()) + 1 if U else 0, R), np.int32)
    for c in range(C):
        lo, hi = part["task_offset"][c], part["task_offset"][c + 1]
        assert np.all(np.diff(part["task_stripe"][lo:hi]) > 0)
        for j, k in zip(part["task_unit"][lo:hi], part["task_stripe"][lo:hi]):
            seen[j] += 1
            F[k, part["unit_desc"][j, 1]] += 1
    return seen, F


def test_structure_on_a_routed_batch():
    cfg = wl.shrink(wl.CONFIGS["skew"], R=8, T=96, H=256, E=32, K=4)
    inp = wl.generate(cfg)
    lay = oracle.layout(inp["ids"], cfg.E)
    row_bytes = cfg.H * 2
    # three tiers with different unit sizes and caps; ranks 0-1 share a "die", 0-3 a "node"
    tiers = [(20, 512, 24, 4), (70, 400, 16, 3), (210, 350, 8, 2)]
    C = 12
    part = oracle.partition(lay, row_bytes, C, tiers, g0=2, g1=4)
    U = part["n_units"]
    sec = lay["src_expert_count"]
    e_loc = cfg.E // cfg.R
    # level 2: window bases
    for e in range(cfg.E):
        assert part["win_base"][0, e] == lay["expert_offset"][e]
        assert np.array_equal(np.diff(part["win_base"][:, e]), sec[:-1, e])
    # level 3: closed-form unit count and exact tiling of every peer window
    B = sec.reshape(cfg.R, cfg.R, e_loc).sum(axis=2)
    def tier(r, d):
        return 0 if r // 2 == d // 2 else 1 if r // 4 == d // 4 else 2
    want_units = sum(-(-int(B[r, d]) // tiers[tier(r, d)][2]) for r in range(cfg.R) for d in range(cfg.R))
    assert U == want_units
    pos = {}
    for j in range(U):
        r, d, a, n = part["unit_desc"][j]
        assert a == pos.get((r, d), 0) and 1 <= n <= tiers[tier(r, d)][2]
        pos[(r, d)] = a + n
        al, be, _, _ = tiers[tier(r, d)]
        assert part["unit_cost"][j] == al + -(-int(n) * row_bytes // be)
    for r in range(cfg.R):
        for d in range(cfg.R):
            assert pos.get((r, d), 0) == B[r, d]
    # every unit scheduled exactly once; loads add up
    seen, F = schedule_tables(part, cfg.R)
    assert np.all(seen == 1)
    loads = np.zeros(C, np.int64)
    for c in range(C):
        for j in part["task_unit"][part["task_offset"][c]:part["task_offset"][c + 1]]:
            loads[c] += part["unit_cost"][j]
    assert np.array_equal(loads, part["core_load"])
    # units inside a core's list arrive in non-increasing cost (largest first)
    for c in range(C):
        lst = part["task_unit"][part["task_offset"][c]:part["task_offset"][c + 1]]
        assert np.all(np.diff(part["unit_cost"][lst]) <= 0)
    # balance: list scheduling keeps every core within one largest unit of the lightest, and the cap changes
    # no core's list (it only moves units to later stripes)
    free = oracle.partition(lay, row_bytes, C, [(a, b, s, 10 ** 6) for a, b, s, _ in tiers], g0=2, g1=4)
    assert free["core_load"].max() - free["core_load"].min() <= free["unit_cost"].max()
    assert np.array_equal(free["core_load"], part["core_load"]) and np.array_equal(free["task_unit"], part["task_unit"])
    assert np.array_equal(free["task_stripe"], np.concatenate([np.arange(n) for n in np.diff(free["task_offset"])]))
    # the cap holds unit by unit: replayed in list-scheduling order (largest cost first, ties by id), a unit
    # never enters a stripe that already holds H_t units for its destination, H_t the cap of the unit's tier
    stripe_of = np.zeros(U, np.int64)
    stripe_of[part["task_unit"]] = part["task_stripe"]
    F2 = np.zeros((int(part["task_stripe"].max()) + 1, cfg.R), np.int32)
    assert F2.shape == F.shape
    for j in sorted(range(U), key=lambda u: (-int(part["unit_cost"][u]), u)):
        r, d = part["unit_desc"][j, 0], part["unit_desc"][j, 1]
        assert F2[stripe_of[j], d] < tiers[tier(r, d)][3]
        F2[stripe_of[j], d] += 1
    assert F.max() <= max(t[3] for t in tiers) and (part["task_stripe"] != free["task_stripe"]).any()
    # window-major dispatch writes exactly what token-major dispatch writes, every row once
    got = oracle.dispatch_windows(lay, part, inp["x"], cfg.K)
    assert np.array_equal(got, oracle.dispatch_bf16(lay["dst_row"], inp["x"]))


def test_fanout_cap_holds_when_it_can():
    # cap 1, as many destinations as cores, units spread evenly: no stripe may hold two units to one rank
    units = [(5 - (i // 4), i % 4) for i in range(16)]
    lay = units_to_layout(units, R=8)
    part = oracle.partition(lay, row_bytes=8, n_cores=4, tiers=[(0, 8, BIG, 1)])
    _, F = schedule_tables(part, 8)
    assert F.max() == 1
    # and a generous cap reproduces the uncapped schedule
    a = oracle.partition(lay, row_bytes=8, n_cores=4, tiers=[(0, 8, BIG, 4)])
    b = oracle.partition(lay, row_bytes=8, n_cores=4, tiers=[(0, 8, BIG, 1000)])
    assert np.array_equal(a["task_unit"], b["task_unit"]) and np.array_equal(a["core_load"], b["core_load"])


def test_too_many_units_is_reported():
    lay = units_to_layout([(10, 0), (10, 1)], R=4)
    with pytest.raises(ValueError):
        oracle.partition(lay, row_bytes=8, n_cores=2, tiers=[(0, 8, 1, 9)], max_units=5)
