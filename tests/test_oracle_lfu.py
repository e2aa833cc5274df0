"""Pins of the capacity-management model (oracle/lfu.py) against hand-worked sequences."""
import pytest

from oracle import lfu


def test_hand_worked_sequence():
    m = lfu.LfuModel(limit_pages=6)
    # call 1: stores A (2 pages), B (2 pages); nothing evicted
    masks, ev = m.call([([1, 2], [32, 20])])
    assert masks == [[0, 0]] and ev == [] and m.used() == 4
    # call 2: hits A, stores C (1 page): fits (5 <= 6)
    masks, ev = m.call([([1, 3], [32, 16])])
    assert masks == [[1, 0]] and ev == []
    assert {c: e["count"] for c, e in m.entries.items()} == {1: 2, 2: 1, 3: 1}
    # call 3: stores D (3 pages): 5 + 3 - 6 = 2 over; candidates by (count, age): B(1, older), C(1), A(2)
    masks, ev = m.call([([4], [40])])
    assert ev == [2] and sorted(m.entries) == [1, 3, 4] and m.used() == 6
    # call 4: hits C and D, stores E (2 pages): over by 2; C and D are protected -> A goes although its count is highest
    masks, ev = m.call([([3, 4, 5], [16, 40, 30])])
    assert masks == [[1, 1, 0]] and ev == [1] and sorted(m.entries) == [3, 4, 5]
    # call 5: a chunk that cannot fit at all: 7 pages > limit even after evicting everything -> error, nothing changes
    before = {c: dict(e) for c, e in m.entries.items()}
    with pytest.raises(lfu.NoSpace):
        m.call([([9], [112])])
    assert m.entries == before


def test_ties_go_to_the_oldest_and_counts_per_occurrence():
    m = lfu.LfuModel(limit_pages=3)
    m.insert(10, 16)
    m.insert(11, 16)
    m.insert(12, 16)
    masks, ev = m.call([([11], [16]), ([11, 12], [16, 16])])      # 11 used twice, 12 once
    assert masks == [[1], [1, 1]] and ev == []
    assert {c: e["count"] for c, e in m.entries.items()} == {10: 1, 11: 3, 12: 2}
    assert m.insert(13, 16) == [10]
    assert m.insert(14, 16) == [13]          # 13 (count 1) is now the least used; 12 (2) and 11 (3) stay
    assert m.insert(15, 32) == [14, 12]


def test_no_eviction_without_the_policy_and_limit_changes():
    m = lfu.LfuModel(limit_pages=2, evict=False)
    m.insert(1, 32)
    with pytest.raises(lfu.NoSpace):
        m.insert(2, 1)
    m2 = lfu.LfuModel(limit_pages=4)
    for c in (1, 2, 3, 4):
        m2.insert(c, 10)
    m2.call([([2, 4], [10, 10])])
    assert m2.set_limit(2) == [1, 3]
    assert sorted(m2.entries) == [2, 4]
    assert m2.set_limit(4) == []


def test_same_new_chunk_in_two_prompts_is_stored_once():
    m = lfu.LfuModel(limit_pages=10)
    masks, ev = m.call([([7], [16]), ([7, 8], [16, 16])])
    assert masks == [[0], [0, 0]] and m.used() == 2
    assert m.entries[7]["count"] == 1 and m.entries[7]["serial"] < m.entries[8]["serial"]
