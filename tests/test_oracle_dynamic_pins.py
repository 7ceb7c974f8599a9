"""Pins of the oracle's model of pages on demand (paper, Section 8 "Dynamic block size and prompt
selection": block sizes and summary lengths that are not known in advance).  The model is a few lines
of counting; it is pinned by hand-worked numbers, by conservation, and by planting the mistakes its
checker exists to catch."""
import numpy as np
import pytest

from oracle import plan as op


def test_hand_worked_small_case():
    # P = 4.  Blocks of 5 and 8 tokens, up to 6 new tokens each, ten free pages 10..19.
    #   block 0: 5 tokens -> 5 // 4 + 1 = 2 pages (10, 11); table holds ceil(11 / 4) = 3
    #   block 1: 8 tokens -> 8 // 4 + 1 = 3 pages (12, 13, 14); table holds ceil(14 / 4) = 4
    #   reserve: 5 pages (15..19)
    m = op.DynamicPages([5, 8], 6, 4, list(range(10, 20)))
    assert m.pages == [2, 3] and m.cap == [3, 4] and m.reserve == 5
    assert m.initial == [[10, 11], [12, 13, 14]]
    m.step([True, True])          # lengths 6, 9: nobody fills a page
    assert m.len == [6, 9] and m.pages == [2, 3] and m.reserve == 5
    m.step([True, False])         # 7, 9
    m.step([True, True])          # 8 (page 1 full -> third page), 10
    assert m.len == [8, 10] and m.pages == [3, 3] and m.reserve == 4
    m.step([False, True])         # 8, 11
    m.step([True, True])          # 9, 12 (block 1 fills page 2 -> fourth page)
    assert m.len == [9, 12] and m.pages == [3, 4] and m.reserve == 3
    m.release([0])
    assert m.pages == [0, 4] and m.reserve == 6 and m.live == [False, True]
    m.step([True, True])          # block 0 is gone: only block 1 moves
    assert m.len == [9, 13]


def test_block_never_holds_more_pages_than_its_table():
    # L = 8, T = 0, P = 4: the table holds 2 pages, and 8 // 4 + 1 = 3 is cut to 2
    m = op.DynamicPages([8], 0, 4, [0, 1, 2])
    assert m.pages == [2] and m.reserve == 1


def test_conservation_under_random_steps():
    rng = np.random.default_rng(0)
    lens = rng.integers(1, 60, 12).tolist()
    free = rng.permutation(200).tolist()
    m = op.DynamicPages(lens, 40, 16, free)
    total = len(free)
    for t in range(40):
        m.step((rng.random(12) < 0.7).tolist())
        if t % 9 == 8:
            m.release([int(rng.integers(0, 12))])
        assert sum(m.pages) + m.reserve == total
        for b in range(12):
            if m.live[b]:
                assert m.pages[b] == min(m.len[b] // 16 + 1, m.cap[b])


def test_empty_reserve_stops_a_block_at_its_page_end():
    m = op.DynamicPages([3, 3], 20, 4, [0, 1])        # one page each, nothing in reserve
    m.step([True, True])                               # both fill their page, no page to take
    assert m.len == [4, 4] and m.pages == [1, 1]
    with pytest.raises(MemoryError):
        m.step([True, False])
    with pytest.raises(MemoryError):
        op.DynamicPages([3, 3], 20, 4, [0])


def _state(m, extra=None):
    """A valid assignment for the model's counts: initial pages first, then pages from the reserve."""
    used = {x for row in m.initial for x in row}
    spare = [x for x in m.all_pages if x not in used]
    rows = []
    for b in range(len(m.len)):
        row = list(m.initial[b]) if m.live[b] else []
        while len(row) < m.pages[b]:
            row.append(spare.pop())
        rows.append(row + [0] * (m.cap[b] - len(row)))
    if extra:
        spare += extra
    return rows, list(m.pages), list(m.len), spare


def test_checker_accepts_a_valid_state_and_rejects_planted_mistakes():
    m = op.DynamicPages([5, 8, 17], 12, 4, list(range(100, 130)))
    for _ in range(7):
        m.step([True, True, True])
    m.release([1])                                # its pages go back to the reserve
    rows, assigned, lens, ring = _state(m)
    ring += [x for x in m.all_pages if x not in ring and all(x not in r[:a] for r, a in zip(rows, assigned))]
    m.check(rows, assigned, lens, ring)
    bad = [r[:] for r in rows]
    bad[0][1] = bad[2][0]                         # one page in two blocks
    with pytest.raises(AssertionError):
        m.check(bad, assigned, lens, ring)
    with pytest.raises(AssertionError):
        m.check(rows, assigned, lens, ring[:-1])  # a page lost from the reserve
    with pytest.raises(AssertionError):
        m.check(rows, assigned, lens, ring + [999])   # a foreign page
    with pytest.raises(AssertionError):
        m.check(rows, [assigned[0] - 1] + assigned[1:], lens, ring)
    with pytest.raises(AssertionError):
        m.check(rows, assigned, [lens[0] + 1] + lens[1:], ring)
    swapped = [r[:] for r in rows]
    swapped[0][0], swapped[0][1] = swapped[0][1], swapped[0][0]   # cached tokens would sit in the wrong page
    with pytest.raises(AssertionError):
        m.check(swapped, assigned, lens, ring)
