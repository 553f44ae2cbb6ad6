"""Host logic of the decode kernel's work schedule (no GPU): the banded flat tile space covers every
tile of every unit exactly once, the work items partition it in order and shrink geometrically,
every segment (the part of one unit inside one item) has a partial record of its own, and every
unit ends up with a small number of them."""
import numpy as np
import pytest


@pytest.fixture(scope="module")
def rl():
    from paper_2510_08525_b200 import build
    build.build()
    import paper_2510_08525_b200.binding as b
    return b


SHAPES = [
    # full units, tiles each, compressed units, tiles each, CTAs, item tiles
    (1, 1, 0, 1, 148, 4), (0, 1, 3, 2, 148, 4), (1, 9, 1, 1, 148, 4), (2, 47, 2, 2, 148, 4),
    (102, 129, 26, 2, 148, 4), (102, 129, 26, 2, 296, 2), (51, 257, 77, 2, 148, 4), (38, 65, 26, 4, 148, 4),
    (512, 33, 0, 2, 148, 4), (8, 1025, 56, 2, 148, 4), (7, 300, 5, 3, 7, 3), (512, 1025, 0, 2, 296, 4),
    (24, 47, 8, 2, 148, 9), (3, 2, 200, 2, 148, 2),
]


@pytest.mark.parametrize("U,tf,Uc,tc,ctas,item", SHAPES)
def test_banded_schedule(rl, U, tf, Uc, tc, ctas, item):
    starts, n_slots, tmap = rl.rlkv_debug_schedule(U, tf, Uc, tc, ctas, item, tile_map=True)
    T = U * tf + Uc * tc
    # ---- items partition the flat space in order
    assert starts[0] == 0 and starts[-1] == T
    sizes = np.diff(starts)
    assert (sizes >= 1).all()
    n_items = sizes.size
    rounds = 0
    while (rounds + 1) * ctas <= n_items and sizes[rounds * ctas:(rounds + 1) * ctas].min() >= 2 * item:
        rounds += 1
    tail = sizes[rounds * ctas:]
    if tail.size:                                           # last band: items of exactly `item` tiles
        assert (tail[:-1] == item).all() and 1 <= tail[-1] <= item
    for r in range(rounds):                                 # earlier bands: near-equal items, shrinking
        part = sizes[r * ctas:(r + 1) * ctas]
        assert part.max() - part.min() <= 1
        if r:
            assert part.max() <= sizes[(r - 1) * ctas:r * ctas].max()
    # ---- every tile of every unit exactly once
    uid, tile, run, slot = tmap[:, 0], tmap[:, 1], tmap[:, 2], tmap[:, 3]
    want = [(u, t) for u in range(U) for t in range(tf)] + [(U + u, t) for u in range(Uc) for t in range(tc)]
    assert sorted(zip(uid.tolist(), tile.tolist())) == want
    # ---- runs: from x on, `run` consecutive flat tiles are consecutive tiles of the same unit, and
    # the run ends where the unit's slice ends
    for x in range(T):
        assert run[x] >= 1
        if run[x] > 1:
            assert uid[x + 1] == uid[x] and tile[x + 1] == tile[x] + 1 and run[x + 1] == run[x] - 1
        elif x + 1 < T:
            assert (uid[x + 1], tile[x + 1]) != (uid[x], tile[x] + 1) or x + 1 == T
    # ---- segments and their partial records
    item_of = np.repeat(np.arange(n_items), sizes)
    new_seg = np.ones(T, bool)
    new_seg[1:] = (item_of[1:] != item_of[:-1]) | (uid[1:] != uid[:-1]) | (tile[1:] != tile[:-1] + 1)
    seg_id = np.cumsum(new_seg) - 1
    seg_slot = {}
    for x in range(T):
        seg_slot.setdefault(int(seg_id[x]), set()).add(int(slot[x]))
    assert all(len(v) == 1 for v in seg_slot.values())                  # one record per segment
    slots = [next(iter(v)) for v in seg_slot.values()]
    assert len(set(slots)) == len(slots)                                # and no two segments share one
    assert max(slots) < n_slots
    # ---- every unit is split into few segments: a handful per band, not one per small item
    per_unit = np.bincount(uid[new_seg], minlength=U + Uc)
    last_band_tiles = tf / 2 ** rounds + 1
    per_band = ctas / max(U, 1) + 2                     # a band of a unit spans about P/U items
    assert per_unit.max() <= rounds * per_band + last_band_tiles / item + 3, (per_unit.max(), rounds)


STEP_SHAPES = [
    # full units, tiles each, compressed units, tiles each, CTAs, largest item
    (3280, 129, 816, 2, 148, 32),       # 32 layers x batch 16, 205 of 256 heads full, n = 8193
    (1232, 65, 816, 4, 148, 32),        # batch 8, n = 4097, 16 + 240 rings
    (205, 33, 51, 2, 148, 32),          # batch 1, n = 2049: fewer tiles than 32 per CTA
    (51, 129, 205, 2, 148, 32),         # 80 % compressed
    (8, 1025, 248, 2, 148, 32),         # very few, very long full units
    (0, 1, 256, 2, 148, 32),            # no full unit at all
    (2, 3, 2, 1, 148, 32), (300, 1, 0, 1, 148, 32), (149, 2, 0, 1, 148, 2), (1000, 7, 24, 3, 7, 5),
]


@pytest.mark.parametrize("U,tf,Uc,tc,ctas,item", STEP_SHAPES)
def test_whole_step_schedule(rl, U, tf, Uc, tc, ctas, item):
    """The schedule of a whole decode step in one launch: most full units lie whole, unit after unit,
    in one static item per CTA (the prefix); the remaining units follow unit after unit in small items.
    Every tile exactly once, items in order, one partial record per segment, none shared; units of the
    prefix are split only where an item boundary falls into them."""
    starts, n_slots, tmap = rl.rlkv_debug_schedule(U, tf, Uc, tc, ctas, item, tile_map=True, whole_step=True)
    T = U * tf + Uc * tc
    assert starts[0] == 0 and starts[-1] == T
    sizes = np.diff(starts)
    assert (sizes >= 1).all()
    n_items = sizes.size
    uid, tile, run, slot = tmap[:, 0], tmap[:, 1], tmap[:, 2], tmap[:, 3]
    want = [(u, t) for u in range(U) for t in range(tf)] + [(U + u, t) for u in range(Uc) for t in range(tc)]
    assert list(zip(uid.tolist(), tile.tolist())) == want          # unit after unit, tile after tile
    for x in range(T - 1):
        if run[x] > 1:
            assert uid[x + 1] == uid[x] and run[x + 1] == run[x] - 1
    # the prefix: the first `ctas` items are near-equal and hold whole units except at their borders;
    # the items after it are small
    small = min(item, max(2, T // ctas))
    prefix_items = ctas if n_items > ctas and sizes[:ctas].min() > small else 0
    if prefix_items:
        part = sizes[:ctas]
        assert part.max() - part.min() <= 1
        x0 = int(starts[ctas])
        assert x0 % tf == 0 and x0 // tf <= U                      # whole units
        assert T - x0 >= 6 * ctas * small - tf                     # enough left for every CTA to claim a few items
        assert T - x0 < 6 * ctas * small + tf + Uc * tc            # and no more than that
        rest = sizes[ctas:]
        assert (rest[:-1] == small).all() and 1 <= rest[-1] <= small
    else:
        assert (sizes[:-1] == small).all()
    item_of = np.repeat(np.arange(n_items), sizes)
    new_seg = np.ones(T, bool)
    new_seg[1:] = (item_of[1:] != item_of[:-1]) | (uid[1:] != uid[:-1])
    seg_id = np.cumsum(new_seg) - 1
    seg_slot = {}
    for x in range(T):
        seg_slot.setdefault(int(seg_id[x]), set()).add(int(slot[x]))
    assert all(len(v) == 1 for v in seg_slot.values())
    slots = [next(iter(v)) for v in seg_slot.values()]
    assert len(set(slots)) == len(slots) and max(slots) < n_slots
    per_unit = np.bincount(uid[new_seg], minlength=U + Uc)
    if prefix_items:                                               # a prefix unit: one piece, or one more per item border inside it
        n_prefix = int(starts[ctas]) // tf
        assert per_unit[:n_prefix].max() <= 1 + -(-tf // int(sizes[:ctas].min()))
        assert (per_unit[:n_prefix] == 1).sum() >= n_prefix - 2 * ctas


@pytest.mark.parametrize("U,tf,Uc,tc,ctas,item", STEP_SHAPES)
def test_whole_step_schedule_with_units_as_items(rl, U, tf, Uc, tc, ctas, item):
    """The whole-step schedule of a paged batch of unequal lengths: the prefix is handed out unit by unit
    (item u = unit u, whole), the rest as in the other form.  Every tile exactly once, one partial record
    per segment, none shared; the hand-out order still starts CTA c with item c."""
    starts, n_slots, tmap = rl.rlkv_debug_schedule(U, tf, Uc, tc, ctas, item, tile_map=True, whole_step=2)
    T = U * tf + Uc * tc
    assert starts[0] == 0 and starts[-1] == T
    sizes = np.diff(starts)
    assert (sizes >= 1).all()
    n_items = sizes.size
    uid, tile, run, slot = tmap[:, 0], tmap[:, 1], tmap[:, 2], tmap[:, 3]
    want = [(u, t) for u in range(U) for t in range(tf)] + [(U + u, t) for u in range(Uc) for t in range(tc)]
    assert list(zip(uid.tolist(), tile.tolist())) == want
    small = min(item, max(2, T // ctas))
    n_prefix = 0
    while n_prefix < n_items and n_prefix < U and sizes[n_prefix] == tf and starts[n_prefix] == n_prefix * tf and tf > small:
        n_prefix += 1
    if n_prefix:
        assert n_prefix >= ctas                                    # every CTA starts with a unit of its own
        assert T - n_prefix * tf >= 6 * ctas * small - tf          # enough left for every CTA to claim a few items
        rest = sizes[n_prefix:]
        assert (rest[:-1] == small).all() and 1 <= rest[-1] <= small
    item_of = np.repeat(np.arange(n_items), sizes)
    new_seg = np.ones(T, bool)
    new_seg[1:] = (item_of[1:] != item_of[:-1]) | (uid[1:] != uid[:-1])
    seg_id = np.cumsum(new_seg) - 1
    seg_slot = {}
    for x in range(T):
        seg_slot.setdefault(int(seg_id[x]), set()).add(int(slot[x]))
    assert all(len(v) == 1 for v in seg_slot.values())
    slots = [next(iter(v)) for v in seg_slot.values()]
    assert len(set(slots)) == len(slots) and max(slots) < n_slots
    per_unit = np.bincount(uid[new_seg], minlength=U + Uc)
    assert (per_unit[:n_prefix] == 1).all()                        # a unit of the prefix is never cut
    order = rl.rlkv_debug_claim_order(U, tf, Uc, tc, ctas, item, n_items, whole_step=2)
    assert sorted(order.tolist()) == list(range(n_items))
    static = min(ctas, n_items)
    assert order[:static].tolist() == list(range(static))


@pytest.mark.parametrize("whole_step", [False, True])
@pytest.mark.parametrize("U,tf,Uc,tc,ctas,item", SHAPES[:8] + STEP_SHAPES[:6])
def test_items_of_compressed_units_are_claimed_first(rl, U, tf, Uc, tc, ctas, item, whole_step):
    """The hand-out order is a permutation of the items that keeps CTA c's first item (item c); among
    the claimed items those that hold only compressed units come first, both groups in their own order."""
    starts, _, tmap = rl.rlkv_debug_schedule(U, tf, Uc, tc, ctas, item, tile_map=True, whole_step=whole_step)
    n_items = starts.size - 1
    order = rl.rlkv_debug_claim_order(U, tf, Uc, tc, ctas, item, n_items, whole_step=whole_step)
    assert sorted(order.tolist()) == list(range(n_items))
    static = min(ctas, n_items)
    assert order[:static].tolist() == list(range(static))
    claimed = order[static:]
    only_comp = np.array([bool((tmap[starts[k]:starts[k + 1], 0] >= U).all()) for k in claimed], dtype=bool)
    n_c = int(only_comp.sum())
    assert only_comp[:n_c].all() and not only_comp[n_c:].any()
    assert (np.diff(claimed[:n_c]) > 0).all() and (np.diff(claimed[n_c:]) > 0).all()


def test_schedule_rejects_bad_arguments(rl):
    for bad in ((0, 1, 0, 1, 148, 4), (1, 0, 0, 1, 148, 4), (1, 1, 1, 0, 148, 4), (1, 1, 0, 1, 0, 4),
                (1, 1, 0, 1, 148, 0), (-1, 1, 2, 1, 148, 4)):
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_debug_schedule(*bad)
        assert e.value.code == rl.RLKV_EINVAL


def test_paged_launch_tickets_match_the_segments_that_exist():
    """Paged cache: sequences shorter than the longest one of a call own only the first tiles of
    their (uniformly sized) units.  Whatever the lengths, grid and item size, every unit must either
    be written directly by the one segment that holds all of its tiles, or receive exactly as many
    partial records as its tickets wait for -- otherwise its merge would never run, or run early."""
    import paper_2510_08525_b200.binding as rl
    rng = np.random.default_rng(11)
    cases = 0
    for trial in range(300):
        n = int(rng.integers(1, 40))
        hi = int(rng.choice([70, 700, 5000, 40000]))
        lens = rng.integers(1, hi + 1, size=n)
        if trial % 3 == 0:
            lens[rng.integers(n)] = hi                      # one long sequence beside short ones
        if trial % 7 == 0:
            lens[:] = int(lens[0])                          # a uniform batch
        n_full, n_comp = int(rng.integers(0, 5)), int(rng.integers(0, 4))
        if n_full + n_comp == 0:
            n_full = 1
        cap = int(rng.choice([5, 64, 128, 200, 384]))
        ctas = int(rng.choice([1, 7, 148, 160]))
        item_tiles = int(rng.choice([2, 3, 8, 32]))
        n_items, delivered, expected, complete = rl.rlkv_debug_paged_schedule(lens, n_full, n_comp, cap, ctas, item_tiles)
        assert n_items >= 1
        direct = complete == 1
        assert ((complete == 0) | direct).all()
        assert (delivered[direct] == 0).all()
        assert (delivered[~direct] == expected[~direct]).all() and (delivered[~direct] >= 1).all()
        cases += len(delivered)
    assert cases > 10000


@pytest.mark.parametrize("n,follows_append", [(1, True), (2, True), (7, True), (32, True), (5, False), (128, False)])
def test_two_launches_sharing_a_scratch_copy_are_never_in_flight_together(rl, n, follows_append):
    """The decode launches of a step alternate between two copies of the split-KV scratch.  Replay
    the launch rules with the slowest possible completions: a launch starts when it is allowed to
    and completes only when something waits for it.  Launch l must never start before launch l - 2
    (the other user of its scratch copy) has completed."""
    overlap, dep_wait, copy = rl.rlkv_debug_step_plan(n, follows_append)
    assert list(copy) == [l & 1 for l in range(n)]
    assert dep_wait[0] == (1 if follows_append else 0) and overlap[0] == (1 if follows_append else 0)
    # earliest moment launch l can start, in terms of which earlier launches must have COMPLETED by then
    must_be_complete = []
    for l in range(n):
        if not overlap[l]:
            done = set(range(l))                     # an ordinary launch waits for everything before it
        elif l == 0:
            done = set()
        else:
            # it starts once launch l - 1 has executed launch_dependents: at its own start if that
            # launch waits for nothing (then it was an ordinary launch, which implies its predecessors
            # were complete), else after the launch before it has completed
            prev_done = must_be_complete[l - 1]
            done = set(prev_done)
            if dep_wait[l - 1] == 0:
                assert not overlap[l - 1], "a launch that triggers at once must itself be an ordinary launch"
            elif dep_wait[l - 1] == 2:
                done |= set(range(l - 1))            # launch l - 2 complete, and by induction all before it
        must_be_complete.append(done)
        if l >= 2:
            assert l - 2 in done, f"launch {l} may start while launch {l - 2} still uses scratch copy {copy[l]}"
