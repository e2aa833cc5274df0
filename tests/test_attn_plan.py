"""Host-side scheduling of the attention kernel (no GPU): every (tile, unit, block) is covered exactly once, parts of
a split unit are consecutive and use consecutive partial slots, CTAs get contiguous item ranges, and the deal is
balanced."""
import numpy as np
import pytest

from paper_2601_11553_b200 import percache as pcb


def check_plan(n_blocks, units, n_ctas=148, max_slots=298):
    items, ctas_used, n_split, makespan = pcb.debug_attn_plan(n_blocks, units, n_ctas, max_slots)
    assert 0 <= ctas_used <= n_ctas
    covered = {}
    for t, u, b0, b1, slot, cta in items.tolist():
        assert 0 <= b0 < b1 <= n_blocks[t] and 0 <= u < units and 0 <= cta < max(ctas_used, 1)
        covered.setdefault((t, u), []).append((b0, b1, slot, cta))
    assert set(covered) == {(t, u) for t in range(len(n_blocks)) for u in range(units)}
    # CTA index never decreases along the list (each CTA runs a contiguous range)
    assert np.all(np.diff(items[:, 5]) >= 0) if len(items) > 1 else True
    split_units, slots_seen = 0, []
    for (t, u), parts in covered.items():
        parts.sort()
        assert parts[0][0] == 0 and parts[-1][1] == n_blocks[t]
        for a, b in zip(parts, parts[1:]):
            assert a[1] == b[0]                       # no gap, no overlap
        if len(parts) == 1:
            assert parts[0][2] == -1                  # a whole unit writes final rows
        else:
            split_units += 1
            s = [p[2] for p in parts]
            assert s == list(range(s[0], s[0] + len(parts))) and s[0] >= 0
            slots_seen += s
            assert all(p[1] - p[0] >= 3 for p in parts)   # no part shorter than three blocks
    assert split_units == n_split
    assert sorted(slots_seen) == list(range(len(slots_seen))) and len(slots_seen) <= max_slots
    load = np.zeros(max(ctas_used, 1), dtype=np.int64)
    for t, u, b0, b1, slot, cta in items.tolist():
        load[cta] += b1 - b0
    return load, n_split, makespan


def test_empty():
    items, ctas, n_split, makespan = pcb.debug_attn_plan([], 8)
    assert len(items) == 0 and ctas == 0 and n_split == 0


def test_one_short_tile_is_not_split():
    load, n_split, _ = check_plan([1], 8)
    assert n_split == 0 and load.tolist() == [1] * 8


@pytest.mark.parametrize("n_blocks", [
    [5, 6, 7, 8, 9, 10, 11, 12, 15, 16, 17],                                # 11 tiles, fewer units than SMs
    [9, 10, 11, 12, 25, 26, 27, 28, 41, 42, 43, 44, 57, 58, 59, 60, 65],     # long ragged tiles
    list(range(1, 259)),                                                   # a 33 024-token prompt, nothing cached
    [3] * 40 + [200],
])
def test_balanced(n_blocks):
    units = 8
    load, n_split, makespan = check_plan(n_blocks, units)
    ideal = units * sum(n_blocks) / 148.0
    # no CTA gets more than the ideal share plus a few blocks of slack
    assert load.max() <= ideal * 1.05 + 6, (load.max(), ideal)


def test_random_shapes():
    rng = np.random.default_rng(11)
    for _ in range(60):
        n_tiles = int(rng.integers(1, 80))
        nb = rng.integers(1, int(rng.integers(2, 300)), size=n_tiles).tolist()
        units = int(rng.choice([1, 2, 4, 8]))
        n_ctas = int(rng.choice([1, 3, 16, 148]))
        check_plan(nb, units, n_ctas=n_ctas, max_slots=2 * n_ctas + 2)


def test_slot_limit_is_respected():
    nb = [64] * 10
    load, n_split, _ = check_plan(nb, 8, n_ctas=148, max_slots=4)
    items, *_ = pcb.debug_attn_plan(nb, 8, 148, 4)
    assert (items[:, 4] >= 0).sum() <= 4


def test_invalid():
    with pytest.raises(pcb.PerCacheError):
        pcb.debug_attn_plan([0], 8)
    with pytest.raises(pcb.PerCacheError):
        pcb.debug_attn_plan([4], 0)
