"""GPU parity: vgc_compress through the C ABI against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

import paper_1802_06058_b200 as vgc
from gpu_harness import (GpuCompressor, OracleCompressor, assert_same_message, assert_same_state, noise_gs,
                         random_offsets)

pytestmark = pytest.mark.gpu
F32 = np.float32


@pytest.mark.parametrize("n,K", [(1, 1), (5, 2), (4095, 3), (4096, 1), (4097, 4), (100003, 7),
                                 ((1 << 20) + 7, 54), (3 * 4096 * 37 + 2, 1500)])
def test_lockstep_random_buffers(n, K):
    rng = np.random.default_rng(n)
    offs = random_offsets(rng, n, K)
    gpu, cpu = GpuCompressor(n, offs), OracleCompressor(n, offs)
    for t in range(4):
        g, s = noise_gs(n, 4, seed=1000 * n % 9973 + t)
        got = gpu.step(g, s, 2.0, 0.999)
        want = cpu.step(g.cpu().numpy(), s.cpu().numpy(), 2.0, 0.999)
        assert_same_message(got, want)
        assert_same_state(gpu, cpu)
        if n > 1000:
            assert 0.01 < want.n_criterion / n < 0.9
            idx = got["words"] >> 4
            assert np.all(np.diff(idx.astype(np.int64)) > 0)


@pytest.mark.parametrize("alpha", [0.0, 1.0, 4.0, 1e30])
def test_alpha_extremes_and_dead_parameters(alpha):
    n = 50000
    offs = np.array([0, 10000, 10000, n], np.uint32)
    gpu, cpu = GpuCompressor(n, offs), OracleCompressor(n, offs)
    for t in range(3):
        g, s = noise_gs(n, 8, seed=77 + t)
        g[::5] = 0; s[::5] = 0                      # dead parameters: 0 > alpha*0 must stay false
        got = gpu.step(g, s, alpha, 0.999)
        want = cpu.step(g.cpu().numpy(), s.cpu().numpy(), alpha, 0.999)
        assert_same_message(got, want)
        assert_same_state(gpu, cpu)
    if alpha == 1e30:
        assert want.nnz == 0 and (got["group_exp"] == vgc.VGC_EXP_NONE).all()


def test_denormal_squares_are_not_flushed():
    # r1*r1 is a denormal here; with v1 = 0 the strict test must still pass (no flush-to-zero)
    n = 4096
    offs = np.array([0, n], np.uint32)
    g = torch.full((n,), 2.0 ** -70, dtype=torch.float32, device="cuda")
    g[1::2] = -(2.0 ** -74)
    g[7] = 2.0 ** -76                               # square underflows to zero: not sent
    s = torch.zeros(n, dtype=torch.float32, device="cuda")
    gpu, cpu = GpuCompressor(n, offs), OracleCompressor(n, offs)
    got = gpu.step(g, s, 1.0, 0.999)
    want = cpu.step(g.cpu().numpy(), s.cpu().numpy(), 1.0, 0.999)
    assert want.n_criterion == n - 1
    assert_same_message(got, want)
    assert_same_state(gpu, cpu)


def test_capacity_overflow_keeps_state_and_reports_needed_count():
    n = 200000
    offs = np.array([0, 70000, n], np.uint32)
    g, s = noise_gs(n, 4, seed=5)
    full, cpu = GpuCompressor(n, offs), OracleCompressor(n, offs)
    want = cpu.step(g.cpu().numpy(), s.cpu().numpy(), 2.0, 0.999)
    ref = full.step(g, s, 2.0, 0.999)
    assert_same_message(ref, want)
    # word buffer too small
    small = GpuCompressor(n, offs, capacity=1000)
    got = small.step(g, s, 2.0, 0.999)
    assert got["dev_status"] == vgc.VGC_DEV_CAPACITY
    assert got["nnz"] == want.nnz and got["n_criterion"] == want.n_criterion
    assert np.array_equal(got["words"], want.words[:1000])
    assert_same_state(small, cpu)
    # no room at all
    none = GpuCompressor(n, offs, capacity=0)
    got = none.step(g, s, 2.0, 0.999)
    assert got["dev_status"] == vgc.VGC_DEV_CAPACITY and got["nnz"] == want.nnz and got["words"].size == 0
    assert_same_state(none, cpu)


def test_checkpoint_resume_is_bit_identical():
    n = 300001
    offs = random_offsets(np.random.default_rng(3), n, 9)
    a, b = GpuCompressor(n, offs), GpuCompressor(n, offs)
    inputs = [noise_gs(n, 4, seed=900 + t) for t in range(6)]
    for g, s in inputs:
        last_a = a.step(g, s, 1.5, 0.999)
    for g, s in inputs[:3]:
        b.step(g, s, 1.5, 0.999)
    r_saved, v_saved = b.r.cpu(), b.v.cpu()          # the whole algorithm state is (r, v)
    c = GpuCompressor(n, offs)
    c.r.copy_(r_saved); c.v.copy_(v_saved)
    for g, s in inputs[3:]:
        last_c = c.step(g, s, 1.5, 0.999)
    assert np.array_equal(last_a["words"], last_c["words"])
    assert torch.equal(a.r, c.r) and torch.equal(a.v, c.v)


def test_without_mask_and_on_a_side_stream():
    n = 123457
    offs = np.array([0, n], np.uint32)
    gpu, cpu = GpuCompressor(n, offs, with_mask=False), OracleCompressor(n, offs)
    g, s = noise_gs(n, 4, seed=11)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        got = gpu.step(g, s, 2.0, 0.999)
    side.synchronize()
    want = cpu.step(g.cpu().numpy(), s.cpu().numpy(), 2.0, 0.999)
    assert_same_message(got, want)


def test_sqgrad_accumulated_into_v_then_compress_without_s():
    """The fused form: the squared-gradient kernels add their result straight into v (accumulate = 1) and the
    compressor is called without s.  v + s is one fp32 addition either way, so everything matches bit for bit."""
    from paper_1802_06058_b200 import workloads
    layers, B = workloads.mlp_layers(), 128
    offs = workloads.group_offsets(layers)
    n, scale = int(offs[-1]), 1.0 / (B * B)
    plain, cpu = GpuCompressor(n, offs), OracleCompressor(n, offs)
    fused = GpuCompressor(n, offs)
    ws = torch.zeros(1 << 26, dtype=torch.uint8, device="cuda")
    s = torch.empty(n, device="cuda")
    for t in range(4):
        ins = [workloads.layer_inputs(spec, B, 1, 0, t, li, "relu_normal", 1e-3, "cuda") for li, spec in enumerate(layers)]
        g = torch.cat([workloads.mean_gradient(spec, x, d) for spec, (x, d) in zip(layers, ins)])
        for li, (spec, (x, d)) in enumerate(zip(layers, ins)):
            lo, hi = int(offs[li]), int(offs[li + 1])
            vgc.vgc_sqgrad_linear(x, d, scale, s[lo:hi], ws=ws)
            vgc.vgc_sqgrad_linear(x, d, scale, fused.v[lo:hi], accumulate=True, ws=ws)
        got_plain = plain.step(g, s, 2.0, 0.999)
        fused.out.counters.zero_()
        vgc.vgc_compress(g, None, fused.r, fused.v, fused.offs_dev, 2.0, 0.999, fused.out, fused.ws)
        got_fused = fused.out.read()
        want = cpu.step(g.cpu().numpy(), s.cpu().numpy(), 2.0, 0.999)
        assert_same_message(got_plain, want)
        assert_same_message(got_fused, want)
        assert_same_state(plain, cpu)
        assert_same_state(fused, cpu)
