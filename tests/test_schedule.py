"""Host logic of the decode kernel's work schedule (no GPU): the items partition the flat tile
space in order, shrink geometrically round by round, end in items of the requested size, and the
tile -> item map used by the split merge is the inverse of the item starts."""
import numpy as np
import pytest


@pytest.fixture(scope="module")
def rl():
    from paper_2510_08525_b200 import build
    build.build()
    import paper_2510_08525_b200.binding as b
    return b


@pytest.mark.parametrize("tiles,ctas,item", [
    (1, 148, 4), (3, 148, 4), (5, 1, 2), (147, 148, 4), (148, 148, 4), (1000, 148, 4), (2367, 148, 4),
    (13209, 148, 4), (13209, 296, 2), (13260, 148, 8), (131072, 148, 4), (524800, 296, 4), (40000, 7, 3),
    (3000000, 148, 2),
])
def test_items_partition_the_tile_space(rl, tiles, ctas, item):
    starts = rl.rlkv_debug_schedule(tiles, ctas, item)     # the library also checks the inverse map
    assert starts[0] == 0 and starts[-1] == tiles
    sizes = np.diff(starts)
    assert (sizes >= 1).all()                               # no empty item, strictly increasing starts
    n_items = sizes.size
    # factoring rounds: `ctas` near-equal items of at least 2*item tiles each
    rounds = 0
    while (rounds + 1) * ctas <= n_items and sizes[rounds * ctas:(rounds + 1) * ctas].min() >= 2 * item:
        rounds += 1
    # the final section: items of exactly `item` tiles (the last one may be shorter)
    tail = sizes[rounds * ctas:]
    if tail.size:
        assert (tail[:-1] == item).all() and 1 <= tail[-1] <= item
    # each round hands out half of what is left
    left = tiles
    for r in range(rounds):
        part = sizes[r * ctas:(r + 1) * ctas]
        assert part.sum() == left // 2 and part.max() - part.min() <= 1
        left -= part.sum()
    assert tail.sum() == left
    # few items while everything is busy, fine grain at the end
    assert n_items <= 14 * ctas + 2 or tiles > (1 << 20)


def test_schedule_rejects_bad_arguments(rl):
    for bad in ((0, 148, 4), (10, 0, 4), (10, 148, 0)):
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_debug_schedule(*bad)
        assert e.value.code == rl.RLKV_EINVAL
