"""GPU parity: squared per-example gradient sums against the CPU oracle (relative 1e-5)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1802_06058_b200 as vgc

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


def run_linear(x, d, scale, S0=None):
    B, n_in = x.shape
    n_out = d.shape[1]
    S = torch.empty(n_out, n_in, device="cuda") if S0 is None else S0.clone()
    ws = _ws(vgc.vgc_sqgrad_linear_workspace_bytes(B, n_in, n_out))
    vgc.vgc_sqgrad_linear(x, d, scale, S, accumulate=S0 is not None, ws=ws)
    assert _status(ws) == 0
    return S.cpu().numpy()


def run_conv(x, d, k, s, p, scale, S0=None):
    B, C, H, W = x.shape
    Cout = d.shape[1]
    S = torch.empty(Cout, C, k, k, device="cuda") if S0 is None else S0.clone()
    ws = _ws(vgc.vgc_sqgrad_conv_workspace_bytes(B, C, H, W, Cout, k, k, s, s, p, p))
    vgc.vgc_sqgrad_conv(x, d, (k, k), (s, s), (p, p), scale, S, accumulate=S0 is not None, ws=ws)
    assert _status(ws) == 0
    return S.cpu().numpy()


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
def test_repacked_and_in_place_forms_agree_with_the_oracle(monkeypatch, B, C, H, Cout, k, s, p):
    gen = torch.Generator(device="cuda"); gen.manual_seed(C + H)
    Ho = (H + 2 * p - k) // s + 1
    x = torch.randn(B, C, H, H, device="cuda", generator=gen)
    d = torch.randn(B, Cout, Ho, Ho, device="cuda", generator=gen) * 1e-3
    want = oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (k, k), (s, s), (p, p), scale=0.5)
    S0 = torch.rand(Cout, C, k, k, device="cuda")
    want_acc = S0.cpu().numpy().copy()
    oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (k, k), (s, s), (p, p), scale=0.5, out=want_acc)
    for repack in ("1", "0"):
        monkeypatch.setenv("VGC_TC_REPACK", repack)
        _check(run_conv(x, d, k, s, p, 0.5), want)
        _check(run_conv(x, d, k, s, p, 0.5, S0=S0), want_acc)


@pytest.mark.parametrize("env", [{"VGC_TC_ATMEM": "0"}, {"VGC_TC_GATHER": "1"}, {"VGC_TC_GATHER": "2"},
                                 {"VGC_TC_GATHER": "3"}, {"VGC_SQGRAD_PATH": "simt"}, {"VGC_TC_TAPS": "0"}, {"VGC_TC_BF16": "0"}, {"VGC_TC_PAIR": "1"}, {"VGC_TC_WIDE": "1"}])
@pytest.mark.parametrize("B,C,H,Cout,k,s,p", [(3, 96, 12, 160, 1, 1, 0), (2, 40, 12, 48, 3, 1, 1), (2, 72, 16, 200, 3, 2, 1)])
def test_every_kernel_variant_gives_the_same_statistic(monkeypatch, env, B, C, H, Cout, k, s, p):
    """The library picks a kernel form per layer (TMA or gathered tiles, A operand in shared or tensor memory,
    roles swapped for few output channels, CUDA-core kernel); the switches force each form on shapes that would
    otherwise take another one."""
    for key, val in env.items():
        monkeypatch.setenv(key, val)
    gen = torch.Generator(device="cuda"); gen.manual_seed(C + H)
    Ho = (H + 2 * p - k) // s + 1
    x = torch.randn(B, C, H, H, device="cuda", generator=gen).abs_()
    d = torch.randn(B, Cout, Ho, Ho, device="cuda", generator=gen) * 1e-4
    got = run_conv(x, d, k, s, p, 0.5)
    want = oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (k, k), (s, s), (p, p), scale=0.5)
    _check(got, want)


@pytest.mark.parametrize("bf16_cross", ["1", "0"])
@pytest.mark.parametrize("xv,dv", [(1.2345678, 0.0031415926), (1.7320508, 0.0027182818), (0.99999994, 1.0000001)])
def test_constant_inputs_rounding_errors_all_of_one_sign(monkeypatch, bf16_cross, xv, dv):
    """Every product has the same rounding error when all inputs are equal, so nothing averages out: the error of
    the split operands (and of the bf16 cross terms) shows at its full size and must still be inside the tolerance."""
    monkeypatch.setenv("VGC_TC_BF16", bf16_cross)
    B, C, H, Cout = 8, 128, 28, 256
    x = torch.full((B, C, H, H), xv, device="cuda"); d = torch.full((B, Cout, H, H), dv, device="cuda")
    got = run_conv(x, d, 1, 1, 0, 1.0 / B)
    x2 = float(np.float32(xv)) ** 2; d2 = float(np.float32(dv)) ** 2        # exact squares of the fp32 inputs
    want = np.full((Cout, C, 1, 1), (1.0 / B) * B * H * H * x2 * d2)
    _check(got, want)


@pytest.mark.parametrize("form", ["VGC_TC_PAIR", "VGC_TC_WIDE"])
@pytest.mark.parametrize("B,C,H,Cout", [(2, 128, 8, 256), (3, 256, 14, 64), (2, 100, 12, 200), (4, 64, 56, 64),
                                        (8, 256, 14, 1024), (2, 130, 8, 520), (4, 512, 28, 128), (2, 384, 7, 640),
                                        (20, 256, 14, 512), (6, 256, 28, 384)])
def test_pair_forms_of_the_1x1_kernel(monkeypatch, form, B, C, H, Cout):
    """VGC_TC_PAIR=1: two CTAs of a cluster share a 256 x 128 tile (cta_group::2); VGC_TC_WIDE=1: a 256 x 256 tile with
    N = 256 instructions where the layer is wide and deep enough (the last two shapes; the last one only with the
    operands' roles exchanged and with a half-empty second tile), pairs or single CTAs elsewhere.  The shapes cover an
    even number of row tiles as given, one that is even only with the roles exchanged, one with no even side (falls back
    to single CTAs), ragged last tiles, the repacked 7x7 form and split reductions; one call and a batch of three layers."""
    monkeypatch.setenv(form, "1")
    gen = torch.Generator(device="cuda"); gen.manual_seed(B + C + Cout)
    xs = [torch.randn(B, C, H, H, device="cuda", generator=gen).clamp_(min=0) for _ in range(3)]
    ds = [torch.randn(B, Cout, H, H, device="cuda", generator=gen) * 1e-2 for _ in range(3)]
    wants = [oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (1, 1), (1, 1), (0, 0), scale=0.25) for x, d in zip(xs, ds)]
    _check(run_conv(xs[0], ds[0], 1, 1, 0, 0.25), wants[0])
    S0 = torch.rand(Cout, C, 1, 1, device="cuda", generator=gen) * float(wants[0].mean())
    _check(run_conv(xs[0], ds[0], 1, 1, 0, 0.25, S0=S0), S0.cpu().numpy().astype(np.float64) + wants[0])
    Ss = [torch.empty(Cout * C, device="cuda") for _ in range(3)]
    ws = _ws(vgc.vgc_sqgrad_conv_batch_workspace_bytes(3, B, C, H, H, Cout, 1, 1, 1, 1, 0, 0))
    vgc.vgc_sqgrad_conv_batch(xs, ds, (1, 1), (1, 1), (0, 0), 0.25, Ss, ws=ws)
    assert _status(ws) == 0
    for S, want in zip(Ss, wants):
        _check(S.cpu().numpy().reshape(Cout, C, 1, 1), want)


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


def test_plan_hint_changes_the_split_not_the_result():
    B, C, H, Cout = 4, 256, 14, 512
    gen = torch.Generator(device="cuda"); gen.manual_seed(5)
    x = torch.randn(B, C, H, H, device="cuda", generator=gen)
    d = torch.randn(B, Cout, H, H, device="cuda", generator=gen) * 1e-2
    want = oracle.sqgrad_conv(x.cpu().numpy(), d.cpu().numpy(), (1, 1), (1, 1), (0, 0), scale=1.0)
    try:
        for hint in (4, 1):
            vgc.vgc_sqgrad_plan_hint(hint)
            _check(run_conv(x, d, 1, 1, 0, 1.0), want)
    finally:
        vgc.vgc_sqgrad_plan_hint(1)


def test_mma_rate_probe_reports_the_instruction_floor():
    """The diagnostic behind the kernel's tensor-pipe ceiling: with M = 128 an instruction takes as long for N = 64 as
    for N = 128 (so half-width tiles run at half the rate) and less than twice as long for N = 256."""
    c64, _ = vgc.vgc_probe_mma_rate(0, True, 64, reps=2048, blocks=8)
    c128, tf128 = vgc.vgc_probe_mma_rate(0, True, 128, reps=2048, blocks=8)
    c256, tf256 = vgc.vgc_probe_mma_rate(0, True, 256, reps=2048, blocks=8)
    assert 20 < c128 < 1000 and tf128 > 0
    assert c64 > 0.9 * c128
    assert c128 < c256 < 1.9 * c128 and tf256 > tf128
    with pytest.raises(vgc.VgcError):
        vgc.vgc_probe_mma_rate(0, True, 100)
    with pytest.raises(vgc.VgcError):
        vgc.vgc_probe_mma_rate(2, True, 128)
