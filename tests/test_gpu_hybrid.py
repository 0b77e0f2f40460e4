"""GPU parity for the hybrid algorithm (Algorithm 2, Sec. 4.5): vgc_compress_hybrid and
vgc_decode_accumulate_hybrid through the C ABI against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1802_06058_b200 as vgc
from gpu_harness import noise_gs

pytestmark = pytest.mark.gpu
F32 = np.float32


class GpuHybrid:
    def __init__(self, n, capacity=None, with_mask=True):
        self.n = n
        self.r = torch.zeros(n, dtype=torch.float32, device="cuda")
        self.v = torch.zeros(n, dtype=torch.float32, device="cuda")
        self.out = vgc.HybridMessageBuffers(n if capacity is None else capacity, n, with_mask=with_mask)
        self.ws = torch.empty(max(vgc.vgc_compress_hybrid_workspace_bytes(n), 16), dtype=torch.uint8, device="cuda")

    def step(self, g, s, alpha, zeta, tau, post=False):
        vgc.vgc_compress_hybrid(g, s, self.r, self.v, alpha, zeta, tau, self.out, self.ws,
                                correction_from_updated_r=post)
        return self.out.read()


def check(got, want, gpu, r_cpu, v_cpu):
    assert got["nnz"] == want.nnz
    np.testing.assert_array_equal(got["words"], want.words)
    if got["mask"] is not None:
        np.testing.assert_array_equal(got["mask"], want.mask)
    np.testing.assert_array_equal(gpu.r.cpu().numpy().view(np.uint32), r_cpu.view(np.uint32))
    np.testing.assert_array_equal(gpu.v.cpu().numpy().view(np.uint32), v_cpu.view(np.uint32))


@pytest.mark.parametrize("post", [False, True])
@pytest.mark.parametrize("n", [1, 5, 2047, 2048, 2049, 100003, 32 * 2048 * 3 + 17, (1 << 21) + 7])
def test_lockstep(n, post):
    gpu = GpuHybrid(n)
    r, v = np.zeros(n, F32), np.zeros(n, F32)
    tau = 2.0 ** -5
    for t in range(5):
        g, s = noise_gs(n, 4, seed=n % 9973 + 31 * t)
        got = gpu.step(g, s, 1.5, 0.999, tau, post=post)
        want = oracle.compress_hybrid(g.cpu().numpy(), s.cpu().numpy(), r, v, 1.5, 0.999, tau, pre_update_r=not post)
        check(got, want, gpu, r, v)
        assert got["dev_status"] == 0
        if n > 1000:
            assert 0.005 < want.nnz / n < 0.9
            assert np.all(np.diff((got["words"] >> 4).astype(np.int64)) > 0)
            assert np.all((got["words"] & 7) == 0)


@pytest.mark.parametrize("alpha,tau", [(0.0, 2.0 ** -4), (2.0, 0.0), (1e30, 2.0 ** -4), (1.0, 1e30)])
def test_limits(alpha, tau):
    # alpha = 0: plain threshold method; tau = 0: the variance test alone; huge alpha or tau: nothing is sent
    n = 70001
    gpu = GpuHybrid(n)
    r, v = np.zeros(n, F32), np.zeros(n, F32)
    for t in range(3):
        g, s = noise_gs(n, 8, seed=500 + t)
        g[::7] = 0; s[::7] = 0
        got = gpu.step(g, s, alpha, 0.9, tau)
        want = oracle.compress_hybrid(g.cpu().numpy(), s.cpu().numpy(), r, v, alpha, 0.9, tau)
        check(got, want, gpu, r, v)
    if alpha == 1e30 or tau == 1e30:
        assert got["nnz"] == 0


def test_s_null_equals_s_added_to_v_first():
    n = 50003
    a, b = GpuHybrid(n), GpuHybrid(n)
    for t in range(3):
        g, s = noise_gs(n, 4, seed=900 + t)
        ga = a.step(g, s, 1.0, 0.99, 2.0 ** -6)
        b.v += s                                            # one rounded add per element, as the kernel would do
        gb = b.step(g, None, 1.0, 0.99, 2.0 ** -6)
        np.testing.assert_array_equal(ga["words"], gb["words"])
        assert torch.equal(a.r, b.r) and torch.equal(a.v, b.v)


def test_capacity_overflow_sets_flag_and_keeps_prefix():
    n = 40000
    g, s = noise_gs(n, 4, seed=5)
    full = GpuHybrid(n).step(g, s, 1.0, 0.999, 2.0 ** -6)
    cap = full["nnz"] // 3
    small = GpuHybrid(n, capacity=cap)
    got = small.step(g, s, 1.0, 0.999, 2.0 ** -6)
    assert got["nnz"] == full["nnz"] and got["dev_status"] & vgc.VGC_DEV_CAPACITY
    np.testing.assert_array_equal(got["words"], full["words"][:cap])


def test_argument_checks():
    n = 100
    gpu = GpuHybrid(n)
    g, s = noise_gs(n, 4, seed=1)
    with pytest.raises(vgc.VgcError):
        gpu.step(g, s, 1.0, 0.9, -1.0)
    with pytest.raises(vgc.VgcError):
        gpu.step(g, s, 1.0, 0.9, float("nan"))
    with pytest.raises(vgc.VgcError):
        vgc.vgc_compress_hybrid(g, s, gpu.r, gpu.v, 1.0, 0.9, 0.1, gpu.out, gpu.ws[:16])


def hybrid_message(rng, n, density):
    idx = np.flatnonzero(rng.random(n) < density).astype(np.uint32)
    sign = rng.integers(0, 2, idx.size).astype(np.uint32)
    return (idx << 4) | (sign << 3)


def assert_within_the_roundings(got, want, u0, msgs, tau, scale):
    """The decoder may sum an element's +-tau words exactly and round once, the oracle rounds after every message:
    the two differ by at most W + 2 half-ulps of |u0| + hits * |scale * tau| (and by nothing where at most two
    words meet)."""
    W = len(msgs)
    mag = np.abs(u0).astype(np.float64)
    hits = np.zeros(u0.size, np.int64)
    for m in msgs:
        idx = (np.asarray(m, np.uint32) >> 4).astype(np.int64)
        np.add.at(hits, idx[idx < u0.size], 1)
    mag += hits * abs(float(np.float32(scale) * np.float32(tau)))
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    assert np.all(err <= (W + 2) * 2.0 ** -24 * mag)
    assert np.array_equal(got[hits == 0].view(np.uint32), u0[hits == 0].view(np.uint32))


@pytest.mark.parametrize("n,W,density", [(1, 1, 1.0), (4097, 3, 0.3), (300007, 8, 0.05), (300007, 2, 0.0005),
                                         ((1 << 21) + 3, 16, 0.02), (70000, 70, 0.2)])
def test_decode(n, W, density):
    rng = np.random.default_rng(n + W)
    msgs = [hybrid_message(rng, n, density) for _ in range(W)]
    tau, scale = 0.0123, 1.0 / W
    u0 = rng.standard_normal(n).astype(F32)
    want = u0.copy()
    assert oracle.decode_hybrid(msgs, tau, scale, want) == 0
    u = torch.from_numpy(u0).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dev = []
    for m in msgs:
        buf = np.zeros(max(m.size, 4), np.uint32); buf[:m.size] = m
        dev.append((torch.from_numpy(buf.view(np.int32)).cuda(), torch.tensor([m.size], dtype=torch.int32, device="cuda")))
    vgc.vgc_decode_accumulate_hybrid(dev, tau, scale, u, status)
    assert int(status.item()) == 0
    assert_within_the_roundings(u.cpu().numpy(), want, u0, msgs, tau, scale)


def test_compress_then_decode_round_trip():
    # W workers, one step: the decoded sum equals the oracle's decode of the oracle's messages
    n, W, tau = 123457, 4, 2.0 ** -6
    workers = [GpuHybrid(n, with_mask=False) for _ in range(W)]
    want = np.zeros(n, F32)
    msgs = []
    for w, wk in enumerate(workers):
        g, s = noise_gs(n, 4, seed=40 + w)
        wk.step(g, s, 1.0, 0.999, tau)
        r, v = np.zeros(n, F32), np.zeros(n, F32)
        msgs.append(oracle.compress_hybrid(g.cpu().numpy(), s.cpu().numpy(), r, v, 1.0, 0.999, tau).words)
    oracle.decode_hybrid(msgs, tau, 1.0 / W, want)
    u = torch.zeros(n, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    vgc.vgc_decode_accumulate_hybrid([wk.out for wk in workers], tau, 1.0 / W, u, status)
    assert int(status.item()) == 0
    np.testing.assert_allclose(u.cpu().numpy(), want, rtol=0, atol=1e-6)


@pytest.mark.parametrize("n,W,density", [(4097, 3, 0.3), (300007, 2, 0.0005), ((1 << 21) + 3, 9, 0.05)])
def test_decode_sum(n, W, density):
    rng = np.random.default_rng(n + W)
    msgs = [hybrid_message(rng, n, density) for _ in range(W)]
    tau, scale = 0.0123, 1.0 / W
    want = np.zeros(n, F32)
    assert oracle.decode_hybrid(msgs, tau, scale, want) == 0
    u = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dev = []
    for m in msgs:
        buf = np.zeros(max(m.size, 4), np.uint32); buf[:m.size] = m
        dev.append((torch.from_numpy(buf.view(np.int32)).cuda(), torch.tensor([m.size], dtype=torch.int32, device="cuda")))
    vgc.vgc_decode_sum_hybrid(dev, tau, scale, u, status)
    assert int(status.item()) == 0
    np.testing.assert_allclose(u.cpu().numpy(), want, rtol=0, atol=1e-6)
    assert_within_the_roundings(u.cpu().numpy(), want, np.zeros(n, F32), msgs, tau, scale)
