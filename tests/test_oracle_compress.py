"""Pins for the CPU oracle's compressor (Algorithm 1 + Sec. 4.2/4.4 quantiser + packing).

None of these tests touches the CUDA path; they tie the oracle to what the paper prints and to
what the mathematics fixes, so that a dropped term, a wrong sign or a shifted index fails."""
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "appendix_b_quantisation.txt")
F32 = np.float32


def _read_appendix_b():
    rows, e = [], None
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            tok = line.split()
            if tok[0] == "floor_log2_Mk":
                e = int(tok[1])
            else:
                rows.append((float(tok[0]), float(tok[1]), int(tok[2]), int(tok[3]), tok[4]))
    return e, rows


def _send_all(vals, offsets=None, **kw):
    """Run one compress step in which every non-zero element passes the test (r=0, s=0, alpha=1)."""
    vals = np.asarray(vals, F32)
    n = vals.size
    r = np.zeros(n, F32); v = np.zeros(n, F32)
    offs = np.array([0, n], np.uint32) if offsets is None else offsets
    msg = oracle.compress(vals, np.zeros(n, F32), r, v, offs, 1.0, 0.999, **kw)
    return msg, r, v


def decode_words(words, gexp, offsets):
    idx = (words >> 4).astype(np.int64)
    sign = (words >> 3) & 1
    d = (words & 7).astype(np.int64)
    k = np.searchsorted(np.asarray(offsets, np.int64), idx, side="right") - 1
    mag = np.ldexp(1.0, (gexp[k].astype(np.int64) - d).astype(np.int64))
    return idx, np.where(sign == 1, -mag, mag)


# ---------------------------------------------------------------------------- Appendix B
def test_appendix_b_worked_example():
    e, rows = _read_appendix_b()
    vals = [r[0] for r in rows]
    msg, r, v = _send_all(vals)
    assert msg.n_criterion == 5
    assert msg.group_exp.tolist() == [e]
    sent = [(i, row) for i, row in enumerate(rows) if row[3] == 1]
    assert msg.nnz == len(sent) and msg.n_dropped == len(rows) - len(sent)
    for word, (i, row) in zip(msg.words.tolist(), sent):
        assert word >> 4 == i                      # 0-based flat index
        assert (word >> 3) & 1 == (1 if row[4] == "-" else 0)
        assert word & 7 == row[2]                  # d as printed
        assert 2.0 ** (e - (word & 7)) == row[1]   # rounded magnitude as printed
    # the unsendable element (d = 10) is rounded to zero: its state is reset like the others
    assert not r.any() and not v.any()
    assert msg.mask.tolist() == [1] * 5


# ---------------------------------------------------------------------------- state machine
def test_never_send_closed_form():
    rng = np.random.default_rng(1)
    n, T, zeta = 257, 40, F32(0.999)
    r = np.zeros(n, F32); v = np.zeros(n, F32)
    r_ref = np.zeros(n, F32); v_ref = np.zeros(n, np.float64)
    offs = np.array([0, 100, 257], np.uint32)
    for t in range(T):
        g = rng.standard_normal(n).astype(F32)
        s = (rng.standard_normal(n) ** 2).astype(F32)
        msg = oracle.compress(g, s, r, v, offs, 1e30, zeta)
        assert msg.nnz == 0 and msg.n_criterion == 0 and not msg.mask.any()
        assert (msg.group_exp == oracle.EXP_NONE).all()
        r_ref = (r_ref + g).astype(F32)                       # fp32 running sum, same order
        v_ref = (v_ref + s.astype(np.float64)) * float(zeta)  # v_t = zeta (v_{t-1} + s_t)
    assert np.array_equal(r, r_ref)
    np.testing.assert_allclose(v, v_ref, rtol=1e-5)
    # constant s: geometric series s * zeta (1 - zeta^T) / (1 - zeta)
    r[:] = 0; v[:] = 0
    for t in range(T):
        oracle.compress(np.zeros(n, F32), np.full(n, 0.25, F32), r, v, offs, 1e30, zeta)
    z = float(zeta)
    np.testing.assert_allclose(v, 0.25 * z * (1 - z ** T) / (1 - z), rtol=1e-5)


def test_always_send_alpha_zero():
    rng = np.random.default_rng(2)
    n = 1000
    offs = np.array([0, n], np.uint32)
    r = np.zeros(n, F32); v = np.zeros(n, F32)
    for t in range(3):
        g = rng.standard_normal(n).astype(F32)
        g[::7] = 0.0                                   # dead parameters: 0 > 0 is false
        s = (rng.standard_normal(n) ** 2).astype(F32)
        msg = oracle.compress(g, s, r, v, offs, 0.0, 0.999)
        assert np.array_equal(msg.mask, (g != 0).astype(np.uint8))
        assert msg.n_criterion == int((g != 0).sum())
        assert not r.any()                             # sent -> 0 ; dead -> 0 + 0
        assert np.all(v[g != 0] == 0)
    # dead parameters kept accumulating and decaying v, they were never reset
    assert np.all(v[::7] > 0)


def test_strict_inequality_and_single_sample():
    # a single sample per step gives g^2 == s exactly; alpha = 1 must not send (strict ">")
    a = np.array([0.5, -2.0, 3.0, 1.0], F32)
    r = np.zeros(4, F32); v = np.zeros(4, F32)
    msg = oracle.compress(a, a * a, r, v, np.array([0, 4], np.uint32), 1.0, 1.0)
    assert msg.n_criterion == 0
    assert np.array_equal(r, a) and np.array_equal(v, a * a)


def test_cauchy_schwarz_delay():
    # zeta = 1 and consistent inputs: after n accumulated samples (sum a)^2 <= n sum a^2, so
    # nothing can be sent while n <= alpha.
    rng = np.random.default_rng(3)
    nparam, alpha = 500, 4.0
    r = np.zeros(nparam, F32); v = np.zeros(nparam, F32)
    offs = np.array([0, nparam], np.uint32)
    sent_at = np.full(nparam, -1)
    for t in range(1, 9):
        a = (rng.standard_normal(nparam) + 2.0).astype(F32)   # strong mean: will send soon after
        msg = oracle.compress(a, a * a, r, v, offs, alpha, 1.0)
        new = (msg.mask == 1) & (sent_at < 0)
        sent_at[new] = t
    assert (sent_at[sent_at > 0] > alpha).all()
    assert (sent_at > 0).mean() > 0.5


def test_eq2_matches_eq1_variance_form():
    """Eq. 2 (sum of squares form) against Eq. 1 with the factor of Appendix A's last line:
    mean^2 > alpha (B-1)/(B-alpha) * V_B / B, V_B the unbiased sample variance."""
    rng = np.random.default_rng(4)
    B, n = 16, 4000
    for alpha in (1.0, 1.5, 2.0):
        per_ex = (rng.standard_normal((B, n)) + rng.standard_normal(n) * 0.7)   # per-example grads
        g = (per_ex.sum(0) / B)
        s = ((per_ex / B) ** 2).sum(0)
        mean = per_ex.mean(0)
        var = per_ex.var(0, ddof=1)
        lhs, rhs = mean ** 2, alpha * (B - 1) / (B - alpha) * var / B
        clear = np.abs(lhs - rhs) > 1e-4 * (lhs + rhs)        # stay away from ties
        r = np.zeros(n, F32); v = np.zeros(n, F32)
        msg = oracle.compress(g.astype(F32), s.astype(F32), r, v, np.array([0, n], np.uint32), alpha, 0.999)
        assert clear.mean() > 0.99
        assert np.array_equal(msg.mask[clear] == 1, (lhs > rhs)[clear])
        assert 0.05 < msg.mask.mean() < 0.95


def test_residual_accounting_multi_step():
    rng = np.random.default_rng(5)
    n, T = 3000, 25
    offs = np.array([0, 1000, 1000, 2500, 3000], np.uint32)      # includes an empty group
    alpha, zeta = F32(2.0), F32(0.999)
    r = np.zeros(n, F32); v = np.zeros(n, F32)
    total_g = np.zeros(n, np.float64)
    total_sent = np.zeros(n, np.float64)      # raw values handed to Encode()
    total_decoded = np.zeros(n, np.float64)
    for t in range(T):
        B = 8
        a = (rng.standard_normal((B, n)) * 1e-2 + 2e-3)
        g = (a.sum(0) / B).astype(F32); s = ((a / B) ** 2).sum(0).astype(F32)
        r0, v0 = r.copy(), v.copy()
        msg = oracle.compress(g, s, r, v, offs, alpha, zeta)
        m = msg.mask == 1
        r1 = (r0 + g).astype(F32); v1 = (v0 + s).astype(F32)
        # exact per-element rules of Algorithm 1
        assert np.array_equal(m, (r1 * r1).astype(F32) > (alpha * v1).astype(F32))
        assert np.all(r[m] == 0) and np.all(v[m] == 0)
        assert np.array_equal(r[~m], r1[~m])
        assert np.array_equal(v[~m], (v1 * zeta).astype(F32)[~m])
        # r_before + g == r_after + (value handed to the encoder, or 0): exact in fp32
        val = np.where(m, r1, F32(0))
        assert np.array_equal((r0 + g).astype(F32), (r + val).astype(F32))
        total_g += g; total_sent += val
        # the message: ascending unique indices, all inside the mask, decoded ~ raw value
        idx, dec = decode_words(msg.words, msg.group_exp, offs)
        assert np.all(np.diff(idx) > 0) and m[idx].all()
        assert msg.nnz + msg.n_dropped == msg.n_criterion == int(m.sum())
        ratio = dec / r1[idx]
        assert np.all(ratio > 0.5) and np.all(ratio <= 4.0 / 3.0)
        total_decoded[idx] += dec
        for k in range(4):
            lo, hi = offs[k], offs[k + 1]
            sel = m[lo:hi]
            if sel.any():
                assert msg.group_exp[k] == math.floor(math.log2(np.abs(r1[lo:hi][sel]).max()))
            else:
                assert msg.group_exp[k] == oracle.EXP_NONE
    # what was accumulated is either still in r or was handed to the encoder
    np.testing.assert_allclose(total_g, r.astype(np.float64) + total_sent, atol=1e-6)
    assert 0.0 < np.abs(total_decoded).sum()


# ---------------------------------------------------------------------------- quantiser
def test_quantiser_rounding_rule_by_definition():
    """Against Sec. 4.2 written with real logarithms: cut above 2^E, else nearer of the two
    neighbouring powers of two (midpoint up), d = E - log2 g', drop d > 7."""
    rng = np.random.default_rng(6)
    n = 20000
    vals = (rng.standard_normal(n) * np.exp2(rng.integers(-12, 4, n))).astype(F32)
    vals[vals == 0] = 1.0
    vals[:6] = [1.5, 3.0, -0.75, 2.9999998, 1.4999999, -6.0]      # exact midpoints and neighbours
    msg, _, _ = _send_all(vals)
    a = np.abs(vals.astype(np.float64))
    E = math.floor(math.log2(a.max()))
    assert msg.group_exp[0] == E
    lo = np.exp2(np.floor(np.log2(a))); hi = 2 * lo
    near = np.where(a - lo < hi - a, lo, hi)        # tie (a = 1.5 lo) goes up
    near = np.where(a == lo, lo, near)
    gq = np.minimum(near, 2.0 ** E)
    d = (E - np.log2(gq)).astype(np.int64)
    keep = d <= 7
    assert msg.nnz == int(keep.sum()) and msg.n_dropped == int((~keep).sum())
    idx = (msg.words >> 4).astype(np.int64)
    assert np.array_equal(idx, np.nonzero(keep)[0])
    assert np.array_equal((msg.words & 7).astype(np.int64), d[keep])
    assert np.array_equal(((msg.words >> 3) & 1).astype(bool), vals[keep] < 0)
    # dropped <=> |val| < 1.5 * 2^(E-8)
    assert np.array_equal(~keep, a < 1.5 * 2.0 ** (E - 8))
    # unclamped ratio in (2/3, 4/3], clamped in (1/2, 1]
    _, dec = decode_words(msg.words, msg.group_exp, [0, n])
    ratio = np.abs(dec) / a[keep]
    clamped = a[keep] > 2.0 ** E
    assert np.all((ratio[~clamped] > 2 / 3) & (ratio[~clamped] <= 4 / 3))
    assert np.all((ratio[clamped] > 0.5) & (ratio[clamped] < 1.0))


def test_group_max_is_over_sent_elements_of_the_group_only():
    # group 0 holds a huge residual that does NOT pass the test; it must not set the scale
    g = np.array([100.0, 0.5, 0.25, 8.0, 1.0], F32)
    s = np.array([1e6, 0.0, 0.0, 0.0, 0.0], F32)
    r = np.zeros(5, F32); v = np.zeros(5, F32)
    msg = oracle.compress(g, s, r, v, np.array([0, 3, 5], np.uint32), 1.0, 0.999)
    assert msg.mask.tolist() == [0, 1, 1, 1, 1]
    assert msg.group_exp.tolist() == [-1, 3]
    assert [(w >> 4, w & 7) for w in msg.words.tolist()] == [(1, 0), (2, 1), (3, 0), (4, 3)]
    assert r[0] == 100.0 and v[0] == F32(1e6) * F32(0.999)


def test_capacity_overflow_leaves_state_untouched():
    rng = np.random.default_rng(7)
    n = 500
    g = rng.standard_normal(n).astype(F32); s = np.zeros(n, F32)
    offs = np.array([0, n], np.uint32)
    r1 = np.zeros(n, F32); v1 = np.zeros(n, F32)
    r2 = np.zeros(n, F32); v2 = np.zeros(n, F32)
    full = oracle.compress(g, s, r1, v1, offs, 1.0, 0.999)
    cut = oracle.compress(g, s, r2, v2, offs, 1.0, 0.999, capacity=10)
    assert cut.overflow and not full.overflow
    assert cut.nnz == full.nnz and np.array_equal(cut.words, full.words[:10])
    assert np.array_equal(r1, r2) and np.array_equal(v1, v2)


# ---------------------------------------------------------------------------- second writing
def _compress_numpy(g, s, r, v, offs, alpha, zeta):
    """An independent vectorised writing of the same algorithm (numpy float32 array ops)."""
    alpha, zeta = F32(alpha), F32(zeta)
    r1 = r + g; v1 = v + s
    send = (r1 * r1) > (alpha * v1)
    r_new = np.where(send, F32(0), r1); v_new = np.where(send, F32(0), v1 * zeta)
    bits = r1.view(np.uint32)
    mag = bits & np.uint32(0x7FFFFFFF)
    words, gexp = [], []
    for k in range(len(offs) - 1):
        lo, hi = int(offs[k]), int(offs[k + 1])
        sel = np.nonzero(send[lo:hi])[0] + lo
        if sel.size == 0:
            gexp.append(oracle.EXP_NONE); continue
        E = int(mag[sel].max() >> 23) - 127
        gexp.append(E)
        e1 = ((mag[sel].astype(np.int64) + 0x00400000) >> 23) - 127
        d = E - np.minimum(e1, E)
        ok = d <= 7
        words.append((sel[ok].astype(np.uint32) << 4) | ((bits[sel][ok] >> 31) << 3) | d[ok].astype(np.uint32))
    words = np.concatenate(words) if words else np.zeros(0, np.uint32)
    return send, r_new, v_new, words.astype(np.uint32), np.array(gexp, np.int32)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_second_independent_writing_agrees(seed):
    rng = np.random.default_rng(100 + seed)
    n = 50000 + seed * 13
    cuts = np.sort(rng.integers(0, n, 6))
    offs = np.concatenate([[0], cuts, [n]]).astype(np.uint32)
    r = np.zeros(n, F32); v = np.zeros(n, F32)
    for t in range(6):
        a = rng.standard_normal((4, n)) * np.exp2(rng.integers(-10, 3, n))
        g = (a.sum(0) / 4).astype(F32); s = ((a / 4) ** 2).sum(0).astype(F32)
        send, r_np, v_np, words_np, gexp_np = _compress_numpy(g, s, r, v, offs, 2.0, 0.999)
        msg = oracle.compress(g, s, r, v, offs, 2.0, 0.999)
        assert np.array_equal(msg.mask == 1, send)
        assert np.array_equal(r, r_np) and np.array_equal(v, v_np)
        assert np.array_equal(msg.words, words_np) and np.array_equal(msg.group_exp, gexp_np)
