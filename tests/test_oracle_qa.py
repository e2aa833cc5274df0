"""Pins of the QA-bank lookup definition: hand cases and closed forms."""
import math

import numpy as np

from oracle import qa_bank as qa


def test_hand_cases():
    bank = np.array([[1.0, 0.0, 0.0, 0.0], [0.0, 2.0, 0.0, 0.0], [3.0, 3.0, 0.0, 0.0], [-1.0, 0.0, 0.0, 0.0]])
    queries = np.array([[5.0, 0.0, 0.0, 0.0], [1.0, 1.0, 0.0, 0.0], [0.0, 0.0, 1.0, 0.0]])
    idx, best, hit, s = qa.top1(bank, queries, 0.85)
    assert np.allclose(s[0], [1.0, 0.0, math.sqrt(0.5), -1.0])           # scale invariance, sign
    assert idx.tolist() == [0, 2, 0]                                       # query 2: all zeros -> lowest index
    assert np.allclose(best, [1.0, 1.0, 0.0])
    assert hit.tolist() == [1, 1, 0]
    # threshold is strict: a similarity equal to tau is not a hit
    assert qa.top1(bank, queries[:1], 1.0)[2].tolist() == [0]


def test_ties_take_the_lowest_index_and_known_angle():
    bank = np.array([[0.0, 1.0], [1.0, 0.0], [2.0, 0.0], [math.cos(0.3), math.sin(0.3)]])
    idx, best, hit, s = qa.top1(bank, np.array([[1.0, 0.0]]), 0.5)
    assert idx.tolist() == [1] and best[0] == 1.0
    assert abs(s[0, 3] - math.cos(0.3)) < 1e-15
