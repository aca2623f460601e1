"""Host logic of the persistent multi-operation launch (no GPU): how rosaq_plan divides a list of
operations among the CTAs of its grid.  Checked here: every (operation, tile, group) is held exactly once;
an operation that reads another's output is processed after it by every CTA, with the operations that
depend on nothing and feed nothing in between; the holders of a shared tile
are consecutive in K, own consecutive partial-tile slots and one counter; at least one holder closes the
tile, the closers are exactly the holders whose range ends in the tile, and they split the token rows;
the shares of a phase are equal up to one work item."""
import collections

import pytest

from paper_2506_13472_b200 import binding as rb

COST_FP16, COST_QUANT, COST_TILE, COST_SCATTER_TILE = 12, 7, 1, 48

LAYER_7B = dict(  # rot(attn), rot(mlp), rot(o) head-wise, down, q, k, v, o, gate, up
    n_tiles=[32, 32, 32, 32, 32, 32, 32, 32, 86, 86], groups=[32, 32, 1, 86, 32, 32, 32, 32, 32, 32],
    g_fp16=[32, 32, 1, 1, 1, 1, 1, 1, 1, 1], x_from=[-1, -1, -1, -1, 0, 0, 0, 2, 1, 1],
    copies=[1, 1, 4, 1, 1, 1, 1, 1, 1, 1])         # the head-wise rotation writes a permuted output: four copies
CASES = {
    "7b-layer": (LAYER_7B, 148),
    "rot+qkv": (dict(n_tiles=[32, 32, 32, 32], groups=[32] * 4, g_fp16=[32, 1, 1, 1], x_from=[-1, 0, 0, 0]), 148),
    "single": (dict(n_tiles=[32], groups=[32], g_fp16=[1], x_from=[-1]), 148),
    "tiny": (dict(n_tiles=[4, 2], groups=[4, 4], g_fp16=[4, 1], x_from=[-1, 0]), 148),     # fewer items than CTAs
    "13b-gateup": (dict(n_tiles=[40, 108, 108], groups=[40] * 3, g_fp16=[40, 1, 1], x_from=[-1, 0, 0]), 148),
    "chain": (dict(n_tiles=[3, 5, 2], groups=[7, 3, 5], g_fp16=[0, 3, 1], x_from=[-1, 0, 1]), 5),
    "filler": (dict(n_tiles=[3, 4, 2], groups=[5, 6, 5], g_fp16=[5, 1, 1], x_from=[-1, -1, 0]), 6),   # op 1 feeds nobody
    "one-cta": (dict(n_tiles=[3, 2], groups=[2, 2], g_fp16=[1, 0], x_from=[-1, -1]), 1),
    "copies": (dict(n_tiles=[5, 3], groups=[3, 4], g_fp16=[3, 1], x_from=[-1, 0], copies=[3, 1]), 7),
}


def phases(x_from):
    """An operation runs after the one it reads from; operations that neither read nor feed another one are
    placed between the producers and their consumers (they fill the time the producers' exchange takes)."""
    feeds = {f for f in x_from if f >= 0}
    free = [i for i, f in enumerate(x_from) if f < 0 and i not in feeds]
    step = 2 if feeds and free else 1
    ph = []
    for i, f in enumerate(x_from):
        ph.append(ph[f] + step if f >= 0 else (1 if step == 2 and i in free else 0))
    return ph


def item_cost(geom, op, g):
    tile = COST_SCATTER_TILE if geom.get("copies", [1] * (op + 1))[op] > 1 else COST_TILE
    return (COST_FP16 if g < geom["g_fp16"][op] else COST_QUANT) + (tile if g == 0 else 0)


@pytest.mark.parametrize("name", sorted(CASES))
def test_schedule_covers_the_list_and_orders_the_exchange(name):
    geom, n_ctas = CASES[name]
    copies = geom.get("copies", [1] * len(geom["n_tiles"]))
    begin, pieces = rb.plan_schedule(geom["n_tiles"], geom["groups"], geom["g_fp16"], geom["x_from"], n_ctas, copies)
    assert begin[0] == 0 and begin[-1] == len(pieces) and all(a <= b for a, b in zip(begin, begin[1:]))
    ph = phases(geom["x_from"])
    n_ops = len(ph)
    # --- coverage: every group of every tile exactly once per copy; the copies of a tile split the 64 token rows
    seen = collections.Counter()
    for p in pieces:
        assert 0 <= p["g_begin"] < p["g_end"] <= geom["groups"][p["op"]] and 0 <= p["tile"] < geom["n_tiles"][p["op"]]
        c = copies[p["op"]]
        k = (p["tok_begin"] * c + 63) // 64
        assert (p["tok_begin"], p["tok_end"]) == (64 * k // c, 64 * (k + 1) // c)
        for g in range(p["g_begin"], p["g_end"]):
            seen[(p["op"], p["tile"], p["tok_begin"], g)] += 1
    want = {(o, t, 64 * k // copies[o], g) for o in range(n_ops) for t in range(geom["n_tiles"][o])
            for k in range(copies[o]) for g in range(geom["groups"][o])}
    assert set(seen) == want and set(seen.values()) == {1}
    # --- order inside a CTA: phases never go backwards; list order inside a phase
    share = collections.defaultdict(int)
    last_of_phase = {}
    for c in range(n_ctas):
        mine = pieces[begin[c]:begin[c + 1]]
        keys = [(ph[p["op"]], p["op"], p["tile"], p["tok_begin"], p["g_begin"]) for p in mine]
        assert keys == sorted(keys)
        for k, p in enumerate(mine):
            share[(ph[p["op"]], c)] += sum(item_cost(geom, p["op"], g) for g in range(p["g_begin"], p["g_end"]))
            last_of_phase[(ph[p["op"]], c)] = begin[c] + k
    # --- shared tiles
    by_tile = collections.defaultdict(list)
    owner = {}
    for c in range(n_ctas):
        for k in range(begin[c], begin[c + 1]):
            owner[k] = c
            by_tile[(pieces[k]["op"], pieces[k]["tile"], pieces[k]["tok_begin"])].append(k)
    slots, counters = set(), set()
    for (op, tile, _), ks in by_tile.items():
        hs = [pieces[k] for k in ks]
        S = len(hs)
        assert all(h["holders"] == S for h in hs)
        if S == 1:
            assert hs[0]["closer_idx"] == -1
            continue
        hs_sorted = sorted(zip(hs, ks), key=lambda hk: hk[0]["g_begin"])
        assert [h["holder_idx"] for h, _ in hs_sorted] == list(range(S))                  # ascending K
        assert all(a["g_end"] == b["g_begin"] for (a, _), (b, _) in zip(hs_sorted, hs_sorted[1:]))
        assert [owner[k] for _, k in hs_sorted] == sorted(owner[k] for _, k in hs_sorted)  # ... = ascending CTA
        assert len({h["slot0"] for h in hs}) == 1 and len({h["counter"] for h in hs}) == 1
        new_slots = set(range(hs[0]["slot0"], hs[0]["slot0"] + S))
        assert not (new_slots & slots) and hs[0]["counter"] not in counters               # never reused in a launch
        slots |= new_slots
        counters.add(hs[0]["counter"])
        closers = [(h, k) for h, k in hs_sorted if h["closer_idx"] >= 0]
        assert len(closers) >= 1 and all(h["closers"] == len(closers) for h in hs)
        assert sorted(h["closer_idx"] for h, _ in closers) == list(range(len(closers)))
        for h, k in hs_sorted:                                                            # closer <=> last piece of its range
            assert (h["closer_idx"] >= 0) == (last_of_phase[(ph[op], owner[k])] == k)
    # --- balance: a share exceeds the mean by less than one work item
    for phase in set(ph):
        total = sum(v for (p, _), v in share.items() if p == phase)
        worst = max(v for (p, _), v in share.items() if p == phase)
        assert worst - total / n_ctas <= COST_FP16 + COST_SCATTER_TILE + 1e-9


def test_schedule_argument_errors():
    with pytest.raises(rb.RosaqError) as e:
        rb.plan_schedule([4], [4], [5], [-1], 8)              # more fp16 groups than groups
    assert e.value.status == rb.ROSAQ_ERR_INVALID_ARG
    with pytest.raises(rb.RosaqError) as e:
        rb.plan_schedule([4, 4], [4, 4], [1, 1], [1, -1], 8)  # reads from a later operation
    assert e.value.status == rb.ROSAQ_ERR_INVALID_ARG
    with pytest.raises(rb.RosaqError) as e:
        rb.plan_schedule([4], [4], [1], [-1], 0)
    assert e.value.status == rb.ROSAQ_ERR_INVALID_ARG
