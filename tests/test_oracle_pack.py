"""Pins for the oracle's index compression (Sec. 4.2, last paragraph: the sorted index field stored as differences in
a variable-length code).  The paper gives no format, so what is pinned is the rule the oracle states: byte strings
worked out by hand from that rule, the stream's size in closed form, the standard base-128 code written a second time
here, and the round trip."""
import numpy as np
import pytest

import oracle


def word(idx, sign, d):
    return (idx << 4) | (sign << 3) | d


def test_hand_written_byte_strings():
    # one run of three words.  v = difference << 4 | low four bits:
    #   idx 0, (+, d=5):  v = 0<<4 | 5          = 5      -> 05
    #   idx 3, (-, d=7):  v = 3<<4 | 15         = 63     -> 3F
    #   idx 11, (+, d=0): v = 8<<4 | 0          = 128    -> 80 01   (seven low bits 0 with the continuation bit, then 1)
    # table: one run -> two entries: 0 and the payload length 4
    words = np.array([word(0, 0, 5), word(3, 1, 7), word(11, 0, 0)], np.uint32)
    assert oracle.pack_indices(words).tolist() == [0, 0, 0, 0, 4, 0, 0, 0, 0x05, 0x3F, 0x80, 0x01]
    # the largest index as a first word: v = (2^28 - 1) << 4 | 9 = 0xFFFFFFF9 -> F9 FF FF FF 0F
    words = np.array([word((1 << 28) - 1, 1, 1)], np.uint32)
    assert oracle.pack_indices(words).tolist() == [0, 0, 0, 0, 5, 0, 0, 0, 0xF9, 0xFF, 0xFF, 0xFF, 0x0F]
    # an empty message is a table with the single entry 0
    assert oracle.pack_indices(np.zeros(0, np.uint32)).tolist() == [0, 0, 0, 0]
    # difference 8 with a zero value field is the first two-byte number; 2^10 the first three-byte one
    two = oracle.pack_indices(np.array([word(7, 1, 7)], np.uint32))       # v = 127 -> 7F
    assert two.tolist()[8:] == [0x7F]
    three = oracle.pack_indices(np.array([word(1024, 0, 0)], np.uint32))  # v = 16384 = 2^14 -> 80 80 01
    assert three.tolist()[8:] == [0x80, 0x80, 0x01]


def test_runs_restart_and_the_table_points_at_them():
    # 257 consecutive indices 1000..1256, value field 2: the first word of each run carries its whole index
    idx = np.arange(1000, 1257, dtype=np.uint32)
    words = (idx << 4) | 2
    packed = oracle.pack_indices(words)
    table = packed[:12].view("<u4")
    # run 0: first number 1000<<4|2 = 16002 -> two bytes (< 2^14); then 255 times (1<<4|2) = 18 -> one byte each
    assert table.tolist() == [0, 2 + 255, 2 + 255 + 3]
    payload = packed[12:]
    assert payload[:3].tolist() == [(16002 & 0x7F) | 0x80, 16002 >> 7, 18]
    # run 1 starts afresh: 1256<<4|2 = 20098 = 1*2^14 + 29*2^7 + 2 -> three bytes 82 9D 01
    assert payload[257:].tolist() == [0x82, 0x9D, 0x01]


def leb128(v):
    """Unsigned LEB128 as the DWARF / protobuf documents define it (second, independent writing)."""
    out = bytearray()
    while True:
        byte = v & 0x7F
        v >>= 7
        out.append(byte | (0x80 if v else 0))
        if not v:
            return bytes(out)


@pytest.mark.parametrize("n,density,seed", [(1 << 20, 1e-2, 1), (1 << 22, 1e-3, 2), (1 << 28, 1e-5, 3), (5000, 0.9, 4),
                                            (100000, 0.2, 5)])
def test_size_in_closed_form_round_trip_and_second_writing(n, density, seed):
    rng = np.random.default_rng(seed)
    m = int(n * density)
    idx = np.sort(rng.choice(n, m, replace=False)).astype(np.uint32) if n <= (1 << 22) else \
        np.unique(rng.integers(0, n, m).astype(np.uint32))
    m = idx.size
    low = rng.integers(0, 16, m).astype(np.uint32)
    words = (idx << 4) | low
    packed = oracle.pack_indices(words)
    # size: every number takes ceil(bits / 7) bytes (one byte for zero), runs restart every 256 words
    prev = np.concatenate([[0], idx[:-1]]).astype(np.int64)
    prev[::oracle.PACK_RUN] = 0
    v = ((idx.astype(np.int64) - prev) << 4) | low
    nbytes = np.maximum((np.floor(np.log2(np.maximum(v, 1))).astype(np.int64) + 7) // 7, 1)
    runs = (m + oracle.PACK_RUN - 1) // oracle.PACK_RUN
    assert packed.size == 4 * (runs + 1) + int(nbytes.sum())
    assert packed.size <= 4 * (runs + 1) + 5 * m
    table = packed[:4 * (runs + 1)].view("<u4")
    run_bytes = np.add.reduceat(nbytes, np.arange(0, m, oracle.PACK_RUN)) if m else np.zeros(0, np.int64)
    assert np.array_equal(table, np.concatenate([[0], np.cumsum(run_bytes)]))
    # the payload is the concatenation of the standard code of every number
    head = min(m, 2000)
    want = b"".join(leb128(int(x)) for x in v[:head])
    assert packed[4 * (runs + 1):4 * (runs + 1) + len(want)].tobytes() == want
    # round trip
    assert np.array_equal(oracle.unpack_indices(packed, m), words)
    if 1e-3 <= density <= 1e-2 and m > 1000:
        assert packed.size < 0.7 * 4 * m            # the point of it: well under four bytes a word


def test_malformed_streams_are_refused():
    words = (np.arange(0, 3000, 3, dtype=np.uint32) << 4) | 1
    packed = oracle.pack_indices(words)
    broken = packed.copy()
    broken[4] ^= 1                                   # run 1 no longer starts where run 0 ends
    with pytest.raises(ValueError):
        oracle.unpack_indices(broken, words.size)
    runs = (words.size + oracle.PACK_RUN - 1) // oracle.PACK_RUN
    broken = packed.copy()
    broken[4 * (runs + 1):4 * (runs + 1) + 6] = 0x80   # a number that never ends within five bytes
    with pytest.raises(ValueError):
        oracle.unpack_indices(broken, words.size)
