"""Pins for the oracle's squared per-example gradient sums (the right-hand side of Eq. 2,
the "v_i +=" line of Algorithm 1), dense and conv.  CPU only."""
import numpy as np
import pytest
import torch

import oracle

F32 = np.float32


def _dense_inputs(seed, B, n_in, n_out):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((B, n_in)).astype(F32), (rng.standard_normal((B, n_out)) * 1e-2).astype(F32)


def test_dense_against_materialised_per_example_gradients():
    x, d = _dense_inputs(0, 4, 7, 5)
    per_example = np.einsum("zj,zi->zji", d.astype(np.float64), x.astype(np.float64))   # [B,out,in]
    want = (per_example ** 2).sum(0)
    got = oracle.sqgrad_linear(x, d)
    assert got.shape == (5, 7)
    np.testing.assert_allclose(got, want, rtol=2e-7)
    # scale = 1/B^2 (Algorithm 1 accumulates (grad_z / B)^2)
    np.testing.assert_allclose(oracle.sqgrad_linear(x, d, scale=1 / 16), want / 16, rtol=2e-7)


def test_dense_equals_matmul_of_squared_operands():
    x, d = _dense_inputs(1, 32, 256, 128)
    want = (torch.from_numpy(d).double() ** 2).t() @ (torch.from_numpy(x).double() ** 2)
    np.testing.assert_allclose(oracle.sqgrad_linear(x, d), want.numpy(), rtol=2e-7)


def test_dense_accumulate_and_all_ones():
    B, n_in, n_out = 12, 9, 4
    ones = oracle.sqgrad_linear(np.ones((B, n_in), F32), np.ones((B, n_out), F32), scale=0.5)
    assert np.all(ones == 0.5 * B)
    x, d = _dense_inputs(2, B, n_in, n_out)
    S = oracle.sqgrad_linear(x, d)
    S2 = S.copy()
    oracle.sqgrad_linear(x, d, out=S2)
    np.testing.assert_allclose(S2, 2 * S, rtol=2e-7)


def test_dense_dead_inputs_and_cauchy_schwarz():
    B = 16
    x, d = _dense_inputs(3, B, 20, 10)
    x = np.maximum(x, 0); x[:, 3] = 0
    S = oracle.sqgrad_linear(x, d, scale=1.0 / B ** 2)
    assert np.all(S >= 0) and np.all(S[:, 3] == 0)
    g = (d.astype(np.float64).T @ x.astype(np.float64)) / B
    assert np.all(g ** 2 <= B * S.astype(np.float64) * (1 + 1e-6))     # (sum a)^2 <= B sum a^2


def _conv_inputs(seed, B, C, H, W, Cout, k, s, p):
    rng = np.random.default_rng(seed)
    Ho = (H + 2 * p - k) // s + 1
    Wo = (W + 2 * p - k) // s + 1
    x = np.abs(rng.standard_normal((B, C, H, W))).astype(F32)
    d = (rng.standard_normal((B, Cout, Ho, Wo)) * 1e-2).astype(F32)
    return x, d


def _conv_contributions(x, d, k, s, p):
    """Every (example, position) contribution a[z,o,c,kh,kw,ho,wo] as an explicit array."""
    B, C, H, W = x.shape
    _, Cout, Ho, Wo = d.shape
    xp = np.zeros((B, C, H + 2 * p, W + 2 * p)); xp[:, :, p:p + H, p:p + W] = x
    a = np.zeros((B, Cout, C, k, k, Ho, Wo))
    for kh in range(k):
        for kw in range(k):
            patch = xp[:, :, kh:kh + s * Ho:s, kw:kw + s * Wo:s]                 # [B,C,Ho,Wo]
            a[:, :, :, kh, kw] = d.astype(np.float64)[:, :, None] * patch[:, None]
    return a


@pytest.mark.parametrize("shape", [(2, 3, 6, 5, 4, 3, 1, 1), (3, 2, 7, 7, 3, 3, 2, 1), (2, 4, 5, 5, 2, 1, 1, 0),
                                   (2, 3, 9, 9, 2, 7, 2, 3), (2, 2, 6, 6, 3, 1, 2, 0)])
def test_conv_against_materialised_contributions(shape):
    B, C, H, W, Cout, k, s, p = shape
    x, d = _conv_inputs(10, B, C, H, W, Cout, k, s, p)
    a = _conv_contributions(x, d, k, s, p)
    got = oracle.sqgrad_conv(x, d, (k, k), (s, s), (p, p))
    np.testing.assert_allclose(got, (a ** 2).sum((0, 5, 6)), rtol=2e-7)
    # per-example reading: positions summed first, then squared
    got_exact = oracle.sqgrad_conv_exact(x, d, (k, k), (s, s), (p, p))
    np.testing.assert_allclose(got_exact, (a.sum((5, 6)) ** 2).sum(0), rtol=1e-6, atol=1e-12)
    # entries version = full version at those entries
    idx = np.random.default_rng(0).integers(0, got.size, 17)
    ent = oracle.sqgrad_conv_entries(x, d, (k, k), (s, s), (p, p), 1.0, idx)
    assert np.array_equal(ent, got.reshape(-1)[idx])


def test_conv_exact_against_autograd_per_example_gradients():
    B, C, H, W, Cout, k, s, p = 3, 2, 6, 6, 3, 3, 1, 1
    x, d = _conv_inputs(11, B, C, H, W, Cout, k, s, p)
    w = torch.zeros(Cout, C, k, k, dtype=torch.float64, requires_grad=True)
    tot = torch.zeros(Cout, C, k, k, dtype=torch.float64)
    for z in range(B):
        y = torch.nn.functional.conv2d(torch.from_numpy(x[z:z + 1]).double(), w, stride=s, padding=p)
        (gz,) = torch.autograd.grad((y * torch.from_numpy(d[z:z + 1]).double()).sum(), w)
        tot += gz ** 2
    np.testing.assert_allclose(oracle.sqgrad_conv_exact(x, d, (k, k), (s, s), (p, p)), tot.numpy(), rtol=1e-6)


def test_conv_single_output_position_equals_per_example():
    # kernel covers the whole image: one output position, so both readings coincide
    x, d = _conv_inputs(12, 4, 3, 5, 5, 6, 5, 1, 0)
    assert d.shape[2:] == (1, 1)
    np.testing.assert_allclose(oracle.sqgrad_conv(x, d, (5, 5)), oracle.sqgrad_conv_exact(x, d, (5, 5)), rtol=1e-6)


def test_conv_1x1_reduces_to_dense():
    x, d = _conv_inputs(13, 3, 5, 4, 6, 7, 1, 1, 0)
    xm = np.ascontiguousarray(x.transpose(0, 2, 3, 1).reshape(-1, 5))
    dm = np.ascontiguousarray(d.transpose(0, 2, 3, 1).reshape(-1, 7))
    np.testing.assert_allclose(oracle.sqgrad_conv(x, d, (1, 1), scale=0.25).reshape(7, 5),
                               oracle.sqgrad_linear(xm, dm, scale=0.25), rtol=2e-7)


def test_conv_all_ones_counts_valid_positions():
    B, C, H, W, Cout, k, s, p = 2, 1, 5, 5, 1, 3, 1, 1
    S = oracle.sqgrad_conv(np.ones((B, C, H, W), F32), np.ones((B, Cout, 5, 5), F32), (k, k), (s, s), (p, p))
    # a corner tap sees 4x4 valid positions, an edge tap 4x5, the centre 5x5
    assert S.reshape(3, 3).tolist() == [[32, 40, 32], [40, 50, 40], [32, 40, 32]]
