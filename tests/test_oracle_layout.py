"""Pins for the oracle's routing layout (paper App. D, token placement).

None of these retype the oracle's counting sort: they use a comparison sort of
(expert, rank, token, slot) tuples, a hand-worked example, closed forms and
structural invariants.
"""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def brute_force_layout(ids: np.ndarray, E: int):
    """Independent formulation: sort item tuples lexicographically; row = position."""
    R, T, K = ids.shape
    tuples = [(int(ids[r, t, k]), r, t, k) for r in range(R) for t in range(T) for k in range(K)]
    order = sorted(tuples)
    dst = np.empty((R, T, K), np.int32)
    for pos, (e, r, t, k) in enumerate(order):
        dst[r, t, k] = pos
    cnt = np.zeros(E, np.int32)
    src_cnt = np.zeros((R, E), np.int32)
    for e, r, _, _ in tuples:
        cnt[e] += 1
        src_cnt[r, e] += 1
    return dst, cnt, src_cnt


def check_invariants(ids, E, lay):
    R, T, K = ids.shape
    N = R * T * K
    e_loc = E // R
    assert lay["expert_count"].sum() == N                     # counts sum to R*T*K
    assert lay["expert_offset"][0] == 0 and lay["expert_offset"][E] == N
    assert np.all(np.diff(lay["expert_offset"]) == lay["expert_count"])
    assert np.array_equal(np.sort(lay["dst_row"].ravel()), np.arange(N))   # bijection
    assert np.array_equal(lay["rank_offset"][:R], lay["expert_offset"][0:E:e_loc])
    assert lay["rank_offset"][R] == N
    assert np.array_equal(np.diff(lay["rank_offset"]), lay["rank_count"])
    assert np.array_equal(lay["src_expert_count"].sum(axis=0), lay["expert_count"])
    assert np.all(lay["src_expert_count"].sum(axis=1) == T * K)
    src = lay["src_of_row"]
    assert np.array_equal(lay["dst_row"].ravel()[src], np.arange(N))       # inverse map
    flat = ids.ravel()
    # row lies inside its expert's segment
    d = lay["dst_row"].ravel()
    assert np.all(d >= lay["expert_offset"][flat]) and np.all(d < lay["expert_offset"][flat + 1])
    # inside a segment the source item index (= (r,t,k) lexicographic) strictly increases
    for e in range(E):
        seg = src[lay["expert_offset"][e]:lay["expert_offset"][e + 1]]
        assert np.all(flat[seg] == e)
        assert np.all(np.diff(seg) > 0)


def test_worked_example():
    rows = {}
    with open(os.path.join(GOLDEN, "layout_worked_example.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                rows[line[0]] = np.array(line[1:], dtype=np.int64)
    R, T, K, E = rows["shape"]
    lay = oracle.layout(rows["ids"].astype(np.int32).reshape(R, T, K), int(E))
    for key in ("expert_count", "expert_offset", "rank_count", "rank_offset",
                "src_expert_count", "dst_row", "src_of_row"):
        assert np.array_equal(lay[key].ravel(), rows[key]), key


@pytest.mark.parametrize("seed", range(8))
def test_matches_sort_brute_force(seed):
    rng = np.random.default_rng(seed)
    R = int(rng.choice([1, 2, 3, 4]))
    e_loc = int(rng.integers(1, 5))
    E = R * e_loc
    T = int(rng.integers(0, 40))
    K = int(rng.integers(1, 5))
    # duplicates inside a token are legal; some experts stay empty
    ids = rng.integers(0, max(1, E - (seed % 2)), size=(R, T, K)).astype(np.int32)
    lay = oracle.layout(ids, E)
    dst, cnt, src_cnt = brute_force_layout(ids, E)
    assert np.array_equal(lay["dst_row"], dst)
    assert np.array_equal(lay["expert_count"], cnt)
    assert np.array_equal(lay["src_expert_count"], src_cnt)
    check_invariants(ids, E, lay)


def test_all_to_one_expert_and_k1_and_r1():
    ids = np.full((3, 7, 2), 4, np.int32)
    lay = oracle.layout(ids, 6)
    assert np.array_equal(lay["dst_row"].ravel(), np.arange(42))
    assert lay["expert_count"].tolist() == [0, 0, 0, 0, 42, 0]
    assert lay["rank_count"].tolist() == [0, 0, 42]
    ids = np.arange(10, dtype=np.int32).reshape(1, 10, 1) % 3
    lay = oracle.layout(ids, 3)
    dst, _, _ = brute_force_layout(ids, 3)
    assert np.array_equal(lay["dst_row"], dst)


def test_closed_form_single_expert():
    ids = np.zeros((2, 5, 3), np.int32)
    lay = oracle.layout(ids, 2)          # E=2, only expert 0 used
    assert np.array_equal(lay["dst_row"].ravel(), np.arange(30))
    lay = oracle.layout(np.zeros((1, 5, 3), np.int32), 1)   # E = 1
    assert np.array_equal(lay["dst_row"].ravel(), np.arange(15))


def test_closed_form_round_robin():
    # ids[i] = i mod E with K = E: expert e receives item e of every token, in token order
    R, T, E = 4, 6, 8
    K = E
    n_tok = R * T
    ids = (np.arange(R * T * K) % E).astype(np.int32).reshape(R, T, K)
    lay = oracle.layout(ids, E)
    i = np.arange(R * T * K)
    assert np.array_equal(lay["dst_row"].ravel(), (i % E) * n_tok + i // E)
    assert np.all(lay["expert_count"] == n_tok)


def test_empty_batch():
    lay = oracle.layout(np.zeros((2, 0, 2), np.int32), 4)
    assert lay["expert_offset"].tolist() == [0, 0, 0, 0, 0]
    assert lay["rank_count"].tolist() == [0, 0]


def test_bad_expert_id_is_rejected():
    ids = np.zeros((2, 3, 2), np.int32)
    ids[1, 0, 1] = 4
    with pytest.raises(oracle.BadExpertId) as ei:
        oracle.layout(ids, 4)
    assert ei.value.item == 7
    ids[1, 0, 1] = -1
    with pytest.raises(oracle.BadExpertId):
        oracle.layout(ids, 4)
    with pytest.raises(ValueError):
        oracle.layout(np.zeros((3, 2, 1), np.int32), 4)    # E % R != 0


def test_invariants_on_tiny_config():
    from paper_2607_26444_b200 import workloads as wl
    cfg = wl.CONFIGS["tiny"]
    ids = wl.gen_topk_ids(cfg)
    lay = oracle.layout(ids, cfg.E)
    check_invariants(ids, cfg.E, lay)
    dst, cnt, _ = brute_force_layout(ids, cfg.E)
    assert np.array_equal(lay["dst_row"], dst)


# ---- production variants: aligned segments and the "not routed" sentinel ----------------------

def brute_force_layout_variants(ids, E, A, allow_unrouted):
    """Independent formulation: sort the routed item tuples; row = aligned segment start + position."""
    R, T, K = ids.shape
    tuples = [(int(ids[r, t, k]), r, t, k) for r in range(R) for t in range(T) for k in range(K)
              if not (allow_unrouted and ids[r, t, k] == -1)]
    cnt = np.zeros(E, np.int64)
    for e, _, _, _ in tuples:
        cnt[e] += 1
    off = np.zeros(E + 1, np.int64)
    for e in range(E):
        off[e + 1] = -(-(off[e] + cnt[e]) // A) * A
    dst = np.full((R, T, K), -1, np.int32)
    pos = np.zeros(E, np.int64)
    for e, r, t, k in sorted(tuples):
        dst[r, t, k] = off[e] + pos[e]
        pos[e] += 1
    return dst, cnt, off


def test_worked_example_padded_unrouted():
    rows = {}
    with open(os.path.join(GOLDEN, "layout_padded_unrouted_example.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                rows[line[0]] = np.array(line[1:], dtype=np.int64)
    R, T, K, E = rows["shape"]
    lay = oracle.layout(rows["ids"].astype(np.int32).reshape(R, T, K), int(E), segment_align=int(rows["align"][0]),
                        allow_unrouted=True)
    for key in ("expert_count", "expert_offset", "rank_count", "rank_offset", "src_expert_count", "dst_row",
                "src_of_row"):
        assert np.array_equal(lay[key].ravel(), rows[key]), key
    assert np.array_equal(oracle.row_experts(lay, int(R)), rows["row_expert"])


@pytest.mark.parametrize("seed", range(8))
def test_variants_match_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    R = int(rng.choice([1, 2, 4]))
    E = R * int(rng.integers(1, 5))
    T, K = int(rng.integers(1, 40)), int(rng.integers(1, 5))
    A = int(rng.choice([1, 2, 8, 16, 128]))
    ids = rng.integers(-1, E, size=(R, T, K)).astype(np.int32)
    lay = oracle.layout(ids, E, segment_align=A, allow_unrouted=True)
    dst, cnt, off = brute_force_layout_variants(ids, E, A, True)
    assert np.array_equal(lay["dst_row"], dst)
    assert np.array_equal(lay["expert_count"], cnt)
    assert np.array_equal(lay["expert_offset"], off)
    assert np.all(lay["expert_offset"] % A == 0)
    assert lay["rank_count"].sum() == (ids >= 0).sum()
    assert lay["rank_offset"][R] == off[E] and np.array_equal(lay["rank_offset"][:R], off[0:E:E // R])
    # inverse map: padding rows and nothing else hold -1
    src = lay["src_of_row"]
    assert src.size == off[E]
    routed = np.flatnonzero(ids.ravel() >= 0)
    assert np.array_equal(np.sort(src[src >= 0]), routed)
    assert np.array_equal(lay["dst_row"].ravel()[src[src >= 0]], np.flatnonzero(src >= 0))
    # without the flag, -1 is rejected like any bad id
    if (ids == -1).any():
        with pytest.raises(oracle.BadExpertId):
            oracle.layout(ids, E, segment_align=A)
    # align 1 without unrouted items is the plain layout
    ids2 = np.where(ids < 0, 0, ids).astype(np.int32)
    a = oracle.layout(ids2, E)
    b = oracle.layout(ids2, E, segment_align=1, allow_unrouted=True)
    assert all(np.array_equal(a[k], b[k]) for k in a)


def test_dispatch_and_combine_skip_unrouted_and_leave_padding():
    from paper_2607_26444_b200 import workloads as wl
    cfg = wl.shrink(wl.CONFIGS["tiny"], R=2, T=40, H=64, E=8, K=3)
    inp = wl.generate(cfg)
    ids = inp["ids"].copy()
    rng = np.random.default_rng(3)
    ids[rng.random(ids.shape) < 0.3] = -1
    ids[0, 0, :] = -1                                   # a token with no expert at all
    lay = oracle.layout(ids, cfg.E, segment_align=16, allow_unrouted=True)
    n_rows = int(lay["expert_offset"][cfg.E])
    recv = oracle.dispatch_bf16(lay["dst_row"], inp["x"], n_rows=n_rows)
    x2 = inp["x"].reshape(cfg.n_tok, cfg.H)
    src = lay["src_of_row"]
    assert np.all(recv[src < 0] == 0xDEAD)              # padding rows untouched
    assert np.array_equal(recv[src >= 0], x2[src[src >= 0] // cfg.K])
    out = oracle.combine(lay["dst_row"], recv, inp["w"])
    assert np.all(out[0] == 0)                          # nothing routed: the sum is empty, +0
    # against float64 over the routed slots only
    rows = lay["dst_row"].reshape(cfg.n_tok, cfg.K)
    w = inp["w"].reshape(cfg.n_tok, cfg.K).astype(np.float64)
    xv = wl.bf16_bits_to_f32(x2).astype(np.float64)
    exact = ((rows >= 0) * w).sum(axis=1, keepdims=True) * xv
    got = wl.bf16_bits_to_f32(out).astype(np.float64)
    assert np.all(np.abs(got - exact) <= np.abs(exact) * 2.0 ** -8 + 1e-30)


def test_ragged_ranks_are_padding_with_the_unrouted_sentinel():
    """Ranks with different token counts: pad every rank to T tokens whose ids are all -1.  Because the
    order is the flat (rank, token, slot) order, the rows of the real items are exactly those of the
    compacted ragged batch."""
    rng = np.random.default_rng(21)
    R, T, K, E = 4, 30, 3, 8
    tokens = [30, 7, 0, 19]                                   # per-rank token counts
    ids = np.full((R, T, K), -1, np.int32)
    for r, n in enumerate(tokens):
        ids[r, :n] = rng.integers(0, E, size=(n, K))
    lay = oracle.layout(ids, E, allow_unrouted=True)
    compact = np.concatenate([ids[r, :n].reshape(-1, K) for r, n in enumerate(tokens)])
    ref = oracle.layout(compact.reshape(1, -1, K), E)         # one "rank": same flat order
    valid = ids.ravel() >= 0
    assert np.array_equal(lay["dst_row"].ravel()[valid], ref["dst_row"].ravel())
    assert np.array_equal(lay["expert_count"], ref["expert_count"])
    assert np.array_equal(lay["expert_offset"], ref["expert_offset"])
    assert lay["src_expert_count"].sum(axis=1).tolist() == [n * K for n in tokens]


# ---- fixed-capacity layout -----------------------------------------------------------------------

def test_worked_example_fixed_capacity():
    rows = {}
    with open(os.path.join(GOLDEN, "layout_fixed_capacity_example.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                rows[line[0]] = np.array(line[1:], dtype=np.int64)
    R, T, K, E = rows["shape"]
    lay = oracle.layout(rows["ids"].astype(np.int32).reshape(R, T, K), int(E), slot_capacity=int(rows["capacity"][0]))
    for key in ("expert_count", "expert_offset", "rank_count", "rank_offset", "src_expert_count", "dst_row",
                "src_of_row"):
        assert np.array_equal(lay[key].ravel(), rows[key]), key
    assert lay["dropped"] == rows["dropped"][0]
    assert np.array_equal(oracle.row_experts(lay, int(R), int(rows["capacity"][0])), rows["row_expert"])


@pytest.mark.parametrize("seed", range(6))
def test_fixed_capacity_matches_brute_force(seed):
    rng = np.random.default_rng(300 + seed)
    R = int(rng.choice([1, 2, 4]))
    E = R * int(rng.integers(1, 4))
    T, K, C = int(rng.integers(1, 30)), int(rng.integers(1, 4)), int(rng.integers(1, 9))
    ids = rng.integers(-1, E, size=(R, T, K)).astype(np.int32)
    lay = oracle.layout(ids, E, allow_unrouted=True, slot_capacity=C)
    # independent formulation: group the routed items by (expert, rank) with a comparison sort
    tuples = sorted((int(ids[r, t, k]), r, t, k) for r in range(R) for t in range(T) for k in range(K) if ids[r, t, k] >= 0)
    dst = np.full((R, T, K), -1, np.int32)
    seen, dropped = {}, 0
    for e, r, t, k in tuples:
        j = seen.get((e, r), 0)
        seen[(e, r)] = j + 1
        if j < C:
            dst[r, t, k] = (e * R + r) * C + j
        else:
            dropped += 1
    assert np.array_equal(lay["dst_row"], dst) and lay["dropped"] == dropped
    kept = np.array([[min(seen.get((e, r), 0), C) for e in range(E)] for r in range(R)])
    assert np.array_equal(lay["src_expert_count"], kept)
    assert np.array_equal(lay["expert_count"], kept.sum(axis=0))
    assert np.array_equal(lay["expert_offset"], np.arange(E + 1) * R * C)
    assert lay["rank_offset"][R] == E * R * C
    src = lay["src_of_row"]
    assert src.size == E * R * C and (src >= 0).sum() == (dst >= 0).sum()
    assert np.array_equal(lay["dst_row"].ravel()[src[src >= 0]], np.flatnonzero(src >= 0))
    # a capacity nobody reaches: same slots, nothing dropped, counts are the plain counts
    big = oracle.layout(ids, E, allow_unrouted=True, slot_capacity=T * K + 1)
    assert big["dropped"] == 0
    assert np.array_equal(big["expert_count"], oracle.layout(ids, E, allow_unrouted=True)["expert_count"])
    with pytest.raises(ValueError):
        oracle.layout(ids, E, allow_unrouted=True, slot_capacity=C, segment_align=4)


@pytest.mark.parametrize("align,cap,frac", [(1, 0, 0.0), (8, 0, 0.15), (1, 5, 0.1), (128, 0, 0.0)])
def test_row_experts_is_the_id_of_the_item_placed_in_the_row(align, cap, frac):
    # independent statement: a row's expert is the id of the item that src_of_row names, -1 where nothing was placed
    rng = np.random.default_rng(align * 10 + cap)
    R, T, K, E = 4, 37, 3, 8
    ids = rng.integers(0, E, size=(R, T, K)).astype(np.int32)
    if frac:
        ids[rng.uniform(size=ids.shape) < frac] = -1
    lay = oracle.layout(ids, E, segment_align=align, allow_unrouted=frac > 0, slot_capacity=cap)
    src = lay["src_of_row"]
    want = np.where(src >= 0, ids.ravel()[np.maximum(src, 0)], -1)
    got = oracle.row_experts(lay, R, cap)
    assert np.array_equal(got, want)
    for e in range(E):
        assert (got == e).sum() == lay["expert_count"][e]
    if align > 1:                                   # every tile of `align` rows belongs to one expert (or is empty)
        tiles = got.reshape(-1, align)
        for t in tiles:
            assert len(set(t[t >= 0].tolist())) <= 1


def test_mask_ragged_marks_exactly_the_padding_tokens():
    rng = np.random.default_rng(3)
    R, T, K, E = 4, 9, 3, 8
    ids = rng.integers(0, E, size=(R, T, K)).astype(np.int32)
    tokens = np.array([9, 0, 4, 12], np.int32)              # a count above T keeps the whole rank
    got = oracle.mask_ragged(ids, tokens)
    t = np.arange(T)[None, :, None]
    want = np.where(t < tokens[:, None, None], ids, -1)
    assert np.array_equal(got, want)
    # and the layout of the masked batch is the layout of the compacted ragged batch
    lay = oracle.layout(got, E, allow_unrouted=True)
    compact = np.concatenate([ids[r, :min(int(n), T)].reshape(-1, K) for r, n in enumerate(tokens)])
    ref = oracle.layout(compact.reshape(1, -1, K), E)
    assert np.array_equal(lay["dst_row"].ravel()[got.ravel() >= 0], ref["dst_row"].ravel())
