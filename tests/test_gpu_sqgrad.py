"""GPU parity: squared per-example gradient sums against the CPU oracle (relative 1e-5)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1802_06058_b200 as vgc
from gpu_harness import Guarded, guarded_like

pytestmark = pytest.mark.gpu
RTOL = 1e-5


def _ws(nbytes):
    return torch.zeros(max(nbytes, 256), dtype=torch.uint8, device="cuda")      # status word starts at 0


def _status(ws):
    return int(ws[:4].view(torch.int32).item())


def _check(got, want):
    want64 = want.astype(np.float64)
    err = np.abs(got.astype(np.float64) - want64)
    assert np.all(err <= RTOL * np.abs(want64)), float((err / np.maximum(np.abs(want64), 1e-300)).max())
    assert np.all(got[want == 0] == 0)


def _guarded_ws(nbytes):
    g = Guarded(max(nbytes, 256), torch.uint8)
    g.t.zero_()                                                               # status word starts at 0
    return g


def run_linear(x, d, scale, S0=None):
    """Result and workspace sit between guard bands: a store past either end of S or of the scratch fails the run."""
    B, n_in = x.shape
    n_out = d.shape[1]
    S = Guarded(n_out * n_in, fill=float("nan")) if S0 is None else guarded_like(S0)
    ws = _guarded_ws(vgc.vgc_sqgrad_linear_workspace_bytes(B, n_in, n_out))
    vgc.vgc_sqgrad_linear(x, d, scale, S.t, accumulate=S0 is not None, ws=ws.t)
    assert _status(ws.t) == 0
    S.check("S"); ws.check("sqgrad workspace")
    return S.t.cpu().numpy().reshape(n_out, n_in)


def run_conv(x, d, k, s, p, scale, S0=None):
    B, C, H, W = x.shape
    Cout = d.shape[1]
    S = Guarded(Cout * C * k * k, fill=float("nan")) if S0 is None else guarded_like(S0)
    ws = _guarded_ws(vgc.vgc_sqgrad_conv_workspace_bytes(B, C, H, W, Cout, k, k, s, s, p, p))
    vgc.vgc_sqgrad_conv(x, d, (k, k), (s, s), (p, p), scale, S.t, accumulate=S0 is not None, ws=ws.t)
    assert _status(ws.t) == 0
    S.check("S"); ws.check("sqgrad workspace")
    return S.t.cpu().numpy().reshape(Cout, C, k, k)


@pytest.mark.parametrize("B,n_in,n_out", [(32, 256, 128), (128, 784, 1024), (128, 1024, 10), (1, 5, 3),
                                          (7, 130, 67), (64, 1000, 333), (300, 64, 64), (2, 1, 1),
                                          (32, 2048, 1000), (64, 36, 260), (1000, 128, 132)])
def test_linear(B, n_in, n_out):
    gen = torch.Generator(device="cuda"); gen.manual_seed(B * 131 + n_in)
    x = torch.randn(B, n_in, device="cuda", generator=gen).clamp_(min=0)     # ReLU-dead inputs
    d = torch.randn(B, n_out, device="cuda", generator=gen) * 1e-3
    x[:, 0] = 0
    got = run_linear(x, d, 1.0 / (B * B))
    want = oracle.sqgrad_linear(x.cpu().numpy(), d.cpu().numpy(), scale=1.0 / (B * B))
    _check(got, want)


def test_linear_accumulate_and_all_ones():
    B, n_in, n_out = 4096, 72, 40
    ones = run_linear(torch.ones(B, n_in, device="cuda"), torch.ones(B, n_out, device="cuda"), 0.5)
    assert np.all(ones == 0.5 * B)
    x = torch.randn(16, n_in, device="cuda"); d = torch.randn(16, n_out, device="cuda")
    S0 = torch.rand(n_out, n_in, device="cuda")
    got = run_linear(x, d, 0.25, S0=S0)
    want = S0.cpu().numpy().copy()
    oracle.sqgrad_linear(x.cpu().numpy(), d.cpu().numpy(), scale=0.25, out=want)
    _check(got, want)


CONV_SHAPES = [  # B, C, H, Cout, k, stride, pad
    (2, 3, 9, 4, 3, 1, 1), (3, 5, 8, 6, 1, 1, 0), (2, 4, 9, 3, 1, 2, 0), (2, 3, 20, 8, 7, 2, 3),
    (4, 16, 14, 24, 3, 2, 1), (2, 64, 14, 64, 3, 1, 1), (2, 70, 7, 130, 1, 1, 0), (3, 8, 5, 5, 5, 1, 0),
    (1, 1, 3, 1, 3, 1, 1),
    # 1x1 / stride 1 / no padding: the tensor-core path (whole and ragged tiles, split reductions)
    (2, 64, 8, 64, 1, 1, 0), (3, 256, 14, 64, 1, 1, 0), (2, 100, 12, 200, 1, 1, 0), (4, 64, 56, 64, 1, 1, 0),
    (2, 8, 6, 8, 1, 1, 0), (5, 300, 10, 136, 1, 1, 0),
    # 1x1 layers that are repacked first: 7x7 planes (channel-major, flat reduction), strided (subsampled planes)
    (4, 70, 7, 130, 1, 1, 0), (4, 48, 14, 200, 1, 2, 0), (2, 96, 16, 160, 1, 2, 0), (3, 64, 28, 40, 1, 2, 0),
    (32, 160, 7, 144, 1, 1, 0),
    # 3x3, stride 1, pad 1 with an even width: three taps per gathered row segment (width % 4 == 0 and == 2,
    # many and few output channels, tiles whose first row is not the first tap of a triple)
    (2, 24, 16, 130, 3, 1, 1), (2, 24, 14, 130, 3, 1, 1), (3, 50, 8, 40, 3, 1, 1), (2, 50, 6, 200, 3, 1, 1),
    (1, 130, 4, 70, 3, 1, 1),
    # 3x3, stride 1, pad 1 on odd widths: planes padded to a multiple of 4 columns first
    (2, 40, 7, 130, 3, 1, 1), (4, 130, 7, 48, 3, 1, 1), (2, 16, 5, 72, 3, 1, 1),
    # 3x3, stride 2, pad 1, input width twice the output width: three taps per gathered segment, stride-2 form
    (2, 24, 12, 130, 3, 2, 1), (3, 50, 8, 40, 3, 2, 1), (2, 16, 24, 72, 3, 2, 1),
    # 7x7, stride 2, pad 3, few output channels: seven taps per gathered row segment
    (2, 3, 32, 16, 7, 2, 3), (1, 5, 24, 40, 7, 2, 3), (3, 20, 16, 64, 7, 2, 3),
]
REPACKED = [(4, 70, 7, 130, 1, 1, 0), (4, 48, 14, 200, 1, 2, 0), (2, 96, 16, 160, 1, 2, 0), (3, 64, 28, 40, 1, 2, 0),
            (2, 40, 7, 130, 3, 1, 1), (3, 24, 9, 20, 3, 1, 1), (4, 16, 14, 24, 3, 2, 1), (2, 64, 14, 130, 3, 2, 1)]


@pytest.mark.parametrize("B,C,H,Cout,k,s,p", CONV_SHAPES)
def test_conv(B, C, H, Cout, k, s, p):
    gen = torch.Generator(device="cuda"); gen.manual_seed(C * 1000 + H)
    Ho = (H + 2 * p - k) // s + 1
    x = torch.randn(B, C, H, H, device="cuda", generator=gen).abs_()
    d = torch.randn(B, Cout, Ho, Ho, device="cuda", generator=gen) * 1e-4
    got = run_conv(x, d, k, s, p, 1.0 / (B * B))
    want = oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (k, k), (s, s), (p, p), scale=1.0 / (B * B))
    _check(got, want)


def test_conv_rectangular_geometry_and_accumulate():
    B, C, H, W, Cout = 2, 3, 10, 7, 4
    Kh, Kw, sh, sw, ph, pw = 3, 2, 2, 1, 1, 0
    Ho, Wo = (H + 2 * ph - Kh) // sh + 1, (W + 2 * pw - Kw) // sw + 1
    x = torch.randn(B, C, H, W, device="cuda"); d = torch.randn(B, Cout, Ho, Wo, device="cuda")
    S0 = torch.rand(Cout, C, Kh, Kw, device="cuda")
    S = S0.clone()
    ws = _ws(vgc.vgc_sqgrad_conv_workspace_bytes(B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw))
    vgc.vgc_sqgrad_conv(x, d, (Kh, Kw), (sh, sw), (ph, pw), 2.0, S, accumulate=True, ws=ws)
    want = S0.cpu().numpy().copy()
    oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (Kh, Kw), (sh, sw), (ph, pw), scale=2.0, out=want)
    _check(S.cpu().numpy(), want)


def test_long_reduction_all_ones_is_exact():
    # K = 2*224*224 = 100352 terms of exactly 1: any one-sided rounding in the accumulation shows up
    x = torch.ones(2, 4, 224, 224, device="cuda"); d = torch.ones(2, 8, 224, 224, device="cuda")
    got = run_conv(x, d, 1, 1, 0, 1.0)
    assert np.all(got == 2 * 224 * 224)
    x = torch.ones(2, 8, 224, 224, device="cuda"); d = torch.ones(2, 16, 224, 224, device="cuda")
    got = run_conv(x, d, 1, 1, 0, 1.0)                      # tensor-core path
    assert np.all(got == 2 * 224 * 224)


@pytest.mark.parametrize("B,C,H,Cout,k,s,p", REPACKED)
def test_repacked_forms_agree_with_the_oracle(B, C, H, Cout, k, s, p):
    gen = torch.Generator(device="cuda"); gen.manual_seed(C + H)
    Ho = (H + 2 * p - k) // s + 1
    x = torch.randn(B, C, H, H, device="cuda", generator=gen)
    d = torch.randn(B, Cout, Ho, Ho, device="cuda", generator=gen) * 1e-3
    want = oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (k, k), (s, s), (p, p), scale=0.5)
    S0 = torch.rand(Cout, C, k, k, device="cuda")
    want_acc = S0.cpu().numpy().copy()
    oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (k, k), (s, s), (p, p), scale=0.5, out=want_acc)
    _check(run_conv(x, d, k, s, p, 0.5), want)
    _check(run_conv(x, d, k, s, p, 0.5, S0=S0), want_acc)


# The library picks a kernel form from the layer's geometry.  One shape (at least) per form that is left:
KERNEL_FORMS = [  # B, C, H, Cout, k, stride, pad
    (3, 96, 12, 160, 1, 1, 0),      # both tiles by TMA, errors as the tensor-memory operand, bf16 cross terms
    (3, 256, 14, 64, 1, 1, 0),      # ... few output channels: the input takes the 128-row side, result written transposed
    (2, 40, 12, 80, 5, 1, 2),       # errors by TMA, im2col rows gathered element-wise (5x5 kernel)
    (2, 40, 12, 48, 5, 1, 2),       # ... roles swapped: gathered im2col rows on the 128-row side
    (2, 40, 9, 80, 5, 1, 2),        # 9x9 planes: neither tile TMA-addressable, both gathered
    (2, 40, 9, 48, 5, 1, 2),        # ... roles swapped
    (2, 24, 16, 130, 3, 1, 1),      # three taps at a time
    (2, 24, 12, 130, 3, 2, 1),      # three taps, stride 2
    (2, 3, 32, 16, 7, 2, 3),        # seven taps, stride 2
    (2, 8, 10, 24, 3, 3, 0),        # stride 3, no padding, 3x3 output: gathered, one slice per example
]


@pytest.mark.parametrize("B,C,H,Cout,k,s,p", KERNEL_FORMS)
def test_every_kernel_form_gives_the_statistic(B, C, H, Cout, k, s, p):
    gen = torch.Generator(device="cuda"); gen.manual_seed(C + H)
    Ho = (H + 2 * p - k) // s + 1
    x = torch.randn(B, C, H, H, device="cuda", generator=gen).abs_()
    d = torch.randn(B, Cout, Ho, Ho, device="cuda", generator=gen) * 1e-4
    want = oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (k, k), (s, s), (p, p), scale=0.5)
    _check(run_conv(x, d, k, s, p, 0.5), want)
    S0 = torch.rand(Cout, C, k, k, device="cuda", generator=gen) * float(want.mean())
    _check(run_conv(x, d, k, s, p, 0.5, S0=S0), S0.cpu().numpy().astype(np.float64) + want)


@pytest.mark.parametrize("xv,dv", [(1.2345678, 0.0031415926), (1.7320508, 0.0027182818), (0.99999994, 1.0000001)])
def test_constant_inputs_rounding_errors_all_of_one_sign(xv, dv):
    """Every product has the same rounding error when all inputs are equal, so nothing averages out: the error of
    the split operands (and of the bf16 cross terms) shows at its full size and must still be inside the tolerance."""
    B, C, H, Cout = 8, 128, 28, 256
    x = torch.full((B, C, H, H), xv, device="cuda"); d = torch.full((B, Cout, H, H), dv, device="cuda")
    got = run_conv(x, d, 1, 1, 0, 1.0 / B)
    x2 = float(np.float32(xv)) ** 2; d2 = float(np.float32(dv)) ** 2        # exact squares of the fp32 inputs
    want = np.full((Cout, C, 1, 1), (1.0 / B) * B * H * H * x2 * d2)
    _check(got, want)


# How a launch's work is cut over the thread blocks depends on the number of tiles and the length of the reduction:
# whole tiles per block, or an even cut of all slices with tiles shared between blocks (partial tiles through the
# scratch, a block finishing one tile and starting the next).  Shapes on either side, results written in both layouts.
@pytest.mark.parametrize("B,C,H,Cout,n_layers", [(8, 256, 14, 1024, 3),      # 48 tiles, 49 slices each: even cut
                                                  (2, 640, 8, 1280, 1),       # 50 tiles, 4 slices: whole tiles
                                                  (16, 64, 28, 64, 2),        # 2 tiles, 400 slices: every block inside one tile
                                                  (4, 192, 16, 40, 5),        # swapped roles, ragged tiles, 10 tiles
                                                  (3, 1152, 8, 1408, 2)])     # 198 tiles of 6 slices: more tiles than blocks
def test_work_is_cut_evenly_over_the_blocks(B, C, H, Cout, n_layers):
    gen = torch.Generator(device="cuda"); gen.manual_seed(B + C + Cout)
    xs = [torch.randn(B, C, H, H, device="cuda", generator=gen).clamp_(min=0) for _ in range(n_layers)]
    ds = [torch.randn(B, Cout, H, H, device="cuda", generator=gen) * 1e-2 for _ in range(n_layers)]
    wants = [oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (1, 1), (1, 1), (0, 0), scale=0.25) for x, d in zip(xs, ds)]
    flat = Guarded(n_layers * Cout * C, fill=float("nan"))
    Ss = [flat.t[l * Cout * C:(l + 1) * Cout * C] for l in range(n_layers)]
    ws = _guarded_ws(vgc.vgc_sqgrad_conv_batch_workspace_bytes(n_layers, B, C, H, H, Cout, 1, 1, 1, 1, 0, 0))
    vgc.vgc_sqgrad_conv_batch(xs, ds, (1, 1), (1, 1), (0, 0), 0.25, Ss, ws=ws.t)
    assert _status(ws.t) == 0
    flat.check("S"); ws.check("sqgrad workspace")
    for S, want in zip(Ss, wants):
        _check(S.cpu().numpy().reshape(Cout, C, 1, 1), want)
    # accumulate on top of what is there
    before = flat.t.clone()
    vgc.vgc_sqgrad_conv_batch(xs, ds, (1, 1), (1, 1), (0, 0), 0.25, Ss, accumulate=True, ws=ws.t)
    flat.check("S"); ws.check("sqgrad workspace")
    for l, want in enumerate(wants):
        base = before[l * Cout * C:(l + 1) * Cout * C].cpu().numpy().astype(np.float64).reshape(Cout, C, 1, 1)
        _check(Ss[l].cpu().numpy().reshape(Cout, C, 1, 1), base + want)


def test_empty_batch_clears_or_keeps_the_result():
    """B = 0: the sum over the mini-batch is empty."""
    x = torch.empty(0, 72, device="cuda"); d = torch.empty(0, 40, device="cuda")
    S = torch.full((40, 72), 3.0, device="cuda")
    vgc.vgc_sqgrad_linear(x, d, 1.0, S, accumulate=True)
    assert float(S.min().item()) == 3.0
    vgc.vgc_sqgrad_linear(x, d, 1.0, S)
    assert float(S.abs().max().item()) == 0.0
    xc = torch.empty(0, 8, 6, 6, device="cuda"); dc = torch.empty(0, 16, 6, 6, device="cuda")
    Sc = torch.full((16 * 8 * 9,), 2.0, device="cuda")
    vgc.vgc_sqgrad_conv(xc, dc, (3, 3), (1, 1), (1, 1), 1.0, Sc, accumulate=True)
    assert float(Sc.min().item()) == 2.0
    vgc.vgc_sqgrad_conv(xc, dc, (3, 3), (1, 1), (1, 1), 1.0, Sc)
    assert float(Sc.abs().max().item()) == 0.0


@pytest.mark.parametrize("n_layers", [1, 3, 9])
@pytest.mark.parametrize("B,C,H,Cout,k,s,p", [(3, 96, 12, 160, 1, 1, 0), (2, 40, 12, 48, 3, 1, 1), (4, 70, 7, 130, 1, 1, 0),
                                              (2, 96, 16, 160, 1, 2, 0), (2, 24, 9, 20, 3, 2, 1), (8, 256, 14, 64, 1, 1, 0)])
def test_batch_of_layers_matches_the_oracle_layer_by_layer(n_layers, B, C, H, Cout, k, s, p):
    gen = torch.Generator(device="cuda"); gen.manual_seed(n_layers * 100 + C)
    Ho = (H + 2 * p - k) // s + 1
    xs = [torch.randn(B, C, H, H, device="cuda", generator=gen) for _ in range(n_layers)]
    ds = [torch.randn(B, Cout, Ho, Ho, device="cuda", generator=gen) * (10.0 ** -(l % 4)) for l in range(n_layers)]
    flat = torch.rand(n_layers * Cout * C * k * k, device="cuda", generator=gen)
    S0 = flat.clone()
    Ss = [flat[l * Cout * C * k * k:(l + 1) * Cout * C * k * k] for l in range(n_layers)]
    ws = _ws(vgc.vgc_sqgrad_conv_batch_workspace_bytes(n_layers, B, C, H, H, Cout, k, k, s, s, p, p))
    for accumulate in (False, True):
        flat.copy_(S0)
        vgc.vgc_sqgrad_conv_batch(xs, ds, (k, k), (s, s), (p, p), 0.5, Ss, accumulate=accumulate, ws=ws)
        assert _status(ws) == 0
        for l in range(n_layers):
            want = S0[l * Cout * C * k * k:(l + 1) * Cout * C * k * k].cpu().numpy().reshape(Cout, C, k, k).copy() \
                if accumulate else None
            want = oracle.sqgrad_conv(xs[l].cpu().numpy(), ds[l].cpu().numpy(), (k, k), (s, s), (p, p), scale=0.5, out=want)
            _check(Ss[l].cpu().numpy().reshape(Cout, C, k, k), want)


def test_batch_argument_checks():
    x = torch.randn(2, 8, 6, 6, device="cuda"); d = torch.randn(2, 8, 6, 6, device="cuda")
    S = torch.empty(8 * 8, device="cuda")
    with pytest.raises(ValueError):
        vgc.vgc_sqgrad_conv_batch([x, x], [d], (1, 1), (1, 1), (0, 0), 1.0, [S, S], ws=_ws(1 << 20))
    with pytest.raises(vgc.VgcError):                         # workspace too small for two layers
        vgc.vgc_sqgrad_conv_batch([x, x], [d, d], (1, 1), (1, 1), (0, 0), 1.0, [S, S.clone()], ws=_ws(256)[:16])
    assert vgc.vgc_sqgrad_conv_batch([], [], (1, 1), (1, 1), (0, 0), 1.0, []) == []


def test_plan_hint_changes_the_share_of_the_sms_not_the_result():
    B, C, H, Cout = 4, 256, 14, 512
    gen = torch.Generator(device="cuda"); gen.manual_seed(5)
    x = torch.randn(B, C, H, H, device="cuda", generator=gen)
    d = torch.randn(B, Cout, H, H, device="cuda", generator=gen) * 1e-2
    want = oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (1, 1), (1, 1), (0, 0), scale=1.0)
    try:
        for hint in (4, 148, 1000, 1):
            vgc.vgc_sqgrad_plan_hint(hint)
            _check(run_conv(x, d, 1, 1, 0, 1.0), want)
    finally:
        vgc.vgc_sqgrad_plan_hint(1)
