"""Pins for the oracle's decoder (decode + sum half of CommunicateAndUpdate).  CPU only."""
import numpy as np

import oracle

F32 = np.float32


def _word(idx, sign, d):
    return np.uint32((idx << 4) | (sign << 3) | d)


def test_appendix_b_round_trip():
    vals = np.array([0.04, 0.31, -6.25, 22.25, -35.75], F32)
    offs = np.array([0, 5], np.uint32)
    r = np.zeros(5, F32); v = np.zeros(5, F32)
    msg = oracle.compress(vals, np.zeros(5, F32), r, v, offs, 1.0, 0.999)
    u = np.zeros(5, F32)
    assert oracle.decode_accumulate([(msg.words, msg.group_exp)], offs, 1.0, u) == 0
    assert u.tolist() == [0.0, 0.25, -8.0, 16.0, -32.0]        # the rounded values the paper prints


def test_decode_by_hand_with_groups_and_scale():
    offs = np.array([0, 4, 4, 10], np.uint32)                   # middle group empty
    words = np.array([_word(0, 0, 0), _word(3, 1, 2), _word(4, 0, 7), _word(9, 1, 0)], np.uint32)
    gexp = np.array([3, oracle.EXP_NONE, -2], np.int32)
    u = np.ones(10, F32)
    oracle.decode_accumulate([(words, gexp)], offs, 0.5, u)
    want = np.ones(10); want[0] += 0.5 * 8; want[3] -= 0.5 * 2; want[4] += 0.5 * 2.0 ** -9; want[9] -= 0.5 * 0.25
    assert np.array_equal(u, want.astype(F32))


def test_identical_messages_sum_and_total():
    rng = np.random.default_rng(0)
    n, W = 5000, 6
    offs = np.array([0, 1200, 5000], np.uint32)
    idx = np.sort(rng.choice(n, 700, replace=False))
    words = ((idx.astype(np.uint32) << 4) | rng.integers(0, 16, idx.size).astype(np.uint32))
    gexp = np.array([-9, -14], np.int32)
    one = np.zeros(n, F32); many = np.zeros(n, F32)
    oracle.decode_accumulate([(words, gexp)], offs, 1.0, one)
    oracle.decode_accumulate([(words, gexp)] * W, offs, 1.0, many)
    assert np.array_equal(many, one * W)                        # powers of two: exact
    k = (idx >= 1200).astype(int)
    vals = np.where((words >> 3) & 1, -1.0, 1.0) * np.exp2(gexp[k] - (words & 7).astype(np.int64))
    assert one.astype(np.float64).sum() == vals.sum()
    assert np.array_equal(np.nonzero(one)[0], idx)


def test_out_of_range_words_are_skipped_and_counted():
    offs = np.array([0, 8], np.uint32)
    words = np.array([_word(1, 0, 0), _word(8, 0, 0), _word(100, 1, 1)], np.uint32)
    u = np.zeros(8, F32)
    assert oracle.decode_accumulate([(words, np.array([0], np.int32))], offs, 1.0, u) == 2
    assert u.tolist() == [0, 1, 0, 0, 0, 0, 0, 0]
