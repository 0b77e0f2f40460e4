"""GPU parity: the per-example conv statistic (vgc_sqgrad_conv_exact) against the CPU oracle's
sqgrad_conv_exact (per-example gradients materialised in fp64, squared, summed)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1802_06058_b200 as vgc

pytestmark = pytest.mark.gpu

SHAPES = [  # B, C, H, Cout, k, stride, pad
    (3, 96, 12, 160, 1, 1, 0),      # 1x1, TMA-fed, several slices per example
    (4, 64, 8, 64, 1, 1, 0),        # roles swapped (few output channels)
    (5, 40, 7, 130, 1, 1, 0),       # 7x7 planes: gathered tiles (no flat repacking in this form)
    (2, 24, 16, 130, 3, 1, 1),      # 3x3, three taps at a time (width % 4 == 0)
    (2, 24, 14, 130, 3, 1, 1),      # ... width % 4 == 2
    (2, 40, 12, 48, 3, 1, 1),       # 3x3 swapped
    (2, 40, 7, 130, 3, 1, 1),       # odd width: padded planes
    (2, 72, 16, 200, 3, 2, 1),      # strided 3x3: three taps at a time, stride-2 form
    (2, 32, 14, 96, 3, 2, 1),       # ... with odd output width: padded planes first
    (2, 20, 9, 40, 3, 2, 1),        # strided 3x3, odd input width: element-wise gather
    (2, 96, 16, 160, 1, 2, 0),      # strided 1x1: subsampled planes
    (2, 3, 32, 16, 7, 2, 3),        # first-layer shape
    (3, 16, 40, 24, 1, 1, 0),       # 50 slices per example: several drains inside one example
    (1, 8, 6, 8, 1, 1, 0), (6, 8, 6, 8, 3, 1, 1),
]


def run(x, d, k, s, p, scale, S0=None):
    B, C, H, W = x.shape
    Cout = d.shape[1]
    S = torch.empty(Cout, C, k, k, device="cuda") if S0 is None else S0.clone()
    ws = torch.zeros(max(vgc.vgc_sqgrad_conv_exact_workspace_bytes(B, C, H, W, Cout, k, k, s, s, p, p), 256),
                     dtype=torch.uint8, device="cuda")
    vgc.vgc_sqgrad_conv_exact(x, d, (k, k), (s, s), (p, p), scale, S, accumulate=S0 is not None, ws=ws)
    assert int(ws[:4].view(torch.int32).item()) == 0
    return S.cpu().numpy()


@pytest.mark.parametrize("B,C,H,Cout,k,s,p", SHAPES)
def test_exact_statistic(B, C, H, Cout, k, s, p):
    gen = torch.Generator(device="cuda"); gen.manual_seed(C * 100 + H)
    Ho = (H + 2 * p - k) // s + 1
    x = torch.randn(B, C, H, H, device="cuda", generator=gen)
    d = torch.randn(B, Cout, Ho, Ho, device="cuda", generator=gen) * 1e-2
    xn, dn = x.cpu().numpy(), d.cpu().numpy()
    want = oracle.sqgrad_conv_exact(xn, dn, (k, k), (s, s), (p, p), scale=0.5).astype(np.float64)
    bound = oracle.sqgrad_conv_exact(np.abs(xn), np.abs(dn), (k, k), (s, s), (p, p), scale=0.5).astype(np.float64)
    got = run(x, d, k, s, p, 0.5).astype(np.float64)
    assert np.all(np.abs(got - want) <= 1e-5 * bound), float((np.abs(got - want) / bound).max())
    # and it is not the position-as-sample statistic (cross terms matter) unless there is one position
    if Ho > 1:
        pos = oracle.sqgrad_conv(xn, dn, (k, k), (s, s), (p, p), scale=0.5).astype(np.float64)
        assert np.abs(pos - want).max() > 1e-3 * np.abs(want).max()


def test_same_sign_inputs_are_relative_1e5_and_accumulate():
    B, C, H, Cout = 4, 64, 14, 96
    gen = torch.Generator(device="cuda"); gen.manual_seed(3)
    x = torch.randn(B, C, H, H, device="cuda", generator=gen).abs_()
    d = torch.randn(B, Cout, H, H, device="cuda", generator=gen).abs_() * 1e-3
    S0 = torch.rand(Cout, C, 1, 1, device="cuda") * 1e-3
    want = oracle.sqgrad_conv_exact(x.cpu().numpy(), d.cpu().numpy(), (1, 1), (1, 1), (0, 0), scale=1.0).astype(np.float64)
    got = run(x, d, 1, 1, 0, 1.0).astype(np.float64)
    assert np.all(np.abs(got - want) <= 1e-5 * want)
    acc = run(x, d, 1, 1, 0, 1.0, S0=S0).astype(np.float64)
    assert np.all(np.abs(acc - (want + S0.cpu().numpy())) <= 1e-5 * (want + S0.cpu().numpy()))


def test_one_position_equals_the_position_statistic():
    B, C, Cout = 64, 96, 160
    x = torch.randn(B, C, 1, 1, device="cuda"); d = torch.randn(B, Cout, 1, 1, device="cuda")
    want = oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (1, 1), (1, 1), (0, 0), scale=1.0).astype(np.float64)
    got = run(x, d, 1, 1, 0, 1.0).astype(np.float64)
    assert np.all(np.abs(got - want) <= 1e-5 * want)


@pytest.mark.parametrize("n_layers", [3, 9])
@pytest.mark.parametrize("B,C,H,Cout,k,s,p", [(3, 96, 12, 160, 1, 1, 0), (2, 24, 16, 130, 3, 1, 1), (2, 40, 7, 130, 3, 1, 1)])
def test_exact_batch(n_layers, B, C, H, Cout, k, s, p):
    gen = torch.Generator(device="cuda"); gen.manual_seed(n_layers + C)
    Ho = (H + 2 * p - k) // s + 1
    xs = [torch.randn(B, C, H, H, device="cuda", generator=gen) for _ in range(n_layers)]
    ds = [torch.randn(B, Cout, Ho, Ho, device="cuda", generator=gen) * 1e-2 for _ in range(n_layers)]
    Ss = [torch.empty(Cout, C, k, k, device="cuda") for _ in range(n_layers)]
    ws = torch.zeros(vgc.vgc_sqgrad_conv_batch_workspace_bytes(n_layers, B, C, H, H, Cout, k, k, s, s, p, p, exact=True),
                     dtype=torch.uint8, device="cuda")
    vgc.vgc_sqgrad_conv_exact_batch(xs, ds, (k, k), (s, s), (p, p), 0.5, Ss, ws=ws)
    assert int(ws[:4].view(torch.int32).item()) == 0
    for l in range(n_layers):
        xn, dn = xs[l].cpu().numpy(), ds[l].cpu().numpy()
        want = oracle.sqgrad_conv_exact(xn, dn, (k, k), (s, s), (p, p), scale=0.5).astype(np.float64)
        bound = oracle.sqgrad_conv_exact(np.abs(xn), np.abs(dn), (k, k), (s, s), (p, p), scale=0.5).astype(np.float64)
        got = Ss[l].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - want) <= 1e-5 * bound)
