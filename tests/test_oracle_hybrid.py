"""Pins for the oracle's hybrid compressor (Algorithm 2 / Sec. 4.5).  CPU only.  The paper prints no worked example
for it, so the pins are what the text fixes: the threshold method it reduces to, the variance correction the
derivation of Sec. 4.5 demands, the always-on decay, and the relation to Algorithm 1."""
import numpy as np

import oracle

F32 = np.float32


def test_alpha_zero_is_the_threshold_method_with_exact_residual_accounting():
    # alpha = 0 leaves |r| > tau alone: accumulate, send +-tau, keep the remainder (Strom's rule as Sec. 4.5 uses it)
    rng = np.random.default_rng(0)
    n, T, tau = 4000, 30, 0.25                       # tau and the inputs are dyadic: every operation is exact
    r = np.zeros(n, F32); v = np.zeros(n, F32)
    total_g = np.zeros(n); sent = np.zeros(n)
    for t in range(T):
        g = (rng.integers(-64, 65, n) / 256.0).astype(F32)
        g[:7] = 0                                    # r == 0 never sends (strict tests)
        r_before = r.copy()
        msg = oracle.compress_hybrid(g, np.zeros(n, F32), r, v, 0.0, 0.999, tau)
        m = msg.mask == 1
        r1 = r_before + g
        assert np.array_equal(m, np.abs(r1) > tau)
        assert np.array_equal(r[m], r1[m] - np.sign(r1[m]) * tau) and np.array_equal(r[~m], r1[~m])
        idx = (msg.words >> 4).astype(np.int64)
        assert np.array_equal(idx, np.nonzero(m)[0]) and np.all(msg.words & 7 == 0)
        sign = np.where((msg.words >> 3) & 1, -1.0, 1.0)
        assert np.array_equal(sign, np.sign(r1[m]))
        total_g += g; sent[idx] += sign * tau
    assert np.array_equal(total_g, r.astype(np.float64) + sent)      # nothing is lost, only delayed
    assert np.all(np.abs(r) <= tau + 0.25)                            # |g| <= 0.25: the remainder stays bounded


def test_variance_correction_is_a_squared_minus_b_squared_for_one_sample():
    # Sec. 4.5: "modifying a^2 to (a-b)^2".  With one sample per step and r = v = 0 before it, v + s = r^2, so after
    # a send the corrected sum of squares must be the square of what is left: (|a| - tau)^2 (then decayed).
    a = np.array([3.0, -5.0, 1.5, -1.25, 0.5, 9.0], F32)
    tau, zeta = 1.0, F32(0.5)
    r = np.zeros(6, F32); v = np.zeros(6, F32)
    msg = oracle.compress_hybrid(a, a * a, r, v, 0.5, zeta, tau)     # alpha < 1 so that r^2 > alpha*v holds
    assert msg.mask.tolist() == [1, 1, 1, 1, 0, 1]
    left = np.where(msg.mask == 1, np.abs(a) - tau, np.abs(a))
    assert np.array_equal(np.abs(r), left)
    assert np.array_equal(v, (left * left * zeta).astype(F32))        # dyadic values: exact
    # the statement order of the listing (|r| taken after the subtraction) gives tau^2 more per unit of 2*tau
    r2 = np.zeros(6, F32); v2 = np.zeros(6, F32)
    oracle.compress_hybrid(a, a * a, r2, v2, 0.5, zeta, tau, pre_update_r=False)
    m = msg.mask == 1
    assert np.array_equal(v2[m], ((left[m] ** 2 + 2 * tau * tau) * zeta).astype(F32)) and np.array_equal(r2, r)


def test_never_send_limits_and_decay_at_every_step():
    rng = np.random.default_rng(1)
    n, T, zeta = 500, 20, 0.999
    for kw in (dict(alpha=1e30, tau=0.0), dict(alpha=0.0, tau=1e30)):
        r = np.zeros(n, F32); v = np.zeros(n, F32)
        v_ref = np.zeros(n); r_ref = np.zeros(n, F32)
        for t in range(T):
            g = rng.standard_normal(n).astype(F32); s = (rng.standard_normal(n) ** 2).astype(F32)
            msg = oracle.compress_hybrid(g, s, r, v, kw["alpha"], zeta, kw["tau"])
            assert msg.nnz == 0
            r_ref = (r_ref + g).astype(F32); v_ref = (v_ref + s.astype(np.float64)) * zeta
        assert np.array_equal(r, r_ref)
        np.testing.assert_allclose(v, v_ref, rtol=1e-5)


def test_same_send_decision_as_algorithm_1_when_tau_is_zero_and_v_never_negative():
    rng = np.random.default_rng(2)
    n = 20000
    a = rng.standard_normal((4, n)) * 0.01 + 0.004
    g = (a.sum(0) / 4).astype(F32); s = ((a / 4) ** 2).sum(0).astype(F32)
    r1 = np.zeros(n, F32); v1 = np.zeros(n, F32); r2 = np.zeros(n, F32); v2 = np.zeros(n, F32)
    basic = oracle.compress(g, s, r1, v1, np.array([0, n], np.uint32), 2.0, 0.999)
    hyb = oracle.compress_hybrid(g, s, r2, v2, 2.0, 0.999, 0.0)
    # tau = 0: |r| > 0 is implied by r^2 > alpha*v >= 0, so the masks coincide; the hybrid keeps r (sends only a sign)
    assert np.array_equal(basic.mask, hyb.mask) and 0.05 < hyb.mask.mean() < 0.95
    assert np.array_equal(r2, g) and np.all(v2 >= 0)
    # with a real threshold fewer elements qualify, and the correction never drives v below zero
    r3 = np.zeros(n, F32); v3 = np.zeros(n, F32)
    hyb2 = oracle.compress_hybrid(g, s, r3, v3, 2.0, 0.999, 0.004)
    assert 0 < hyb2.nnz < hyb.nnz and np.all(v3 >= 0)
    assert np.all((hyb2.mask == 1) <= (hyb.mask == 1))


def test_decode_hybrid_adds_plus_minus_tau():
    words = [np.array([(1 << 4), (3 << 4) | 8, (9 << 4)], np.uint32), np.array([(3 << 4) | 8, (40 << 4)], np.uint32)]
    u = np.zeros(10, F32)
    assert oracle.decode_hybrid(words, 0.125, 2.0, u) == 1           # index 40 is out of range
    assert u.tolist() == [0, 0.25, 0, -0.5, 0, 0, 0, 0, 0, 0.25]
