"""Helpers shared by the GPU parity tests: run the CUDA path through the binding and the CPU
oracle on identical bytes and compare."""
import numpy as np
import torch

import oracle
import paper_1802_06058_b200 as vgc

F32 = np.float32


class GpuCompressor:
    """State + buffers for repeated vgc_compress calls on one flat buffer."""

    def __init__(self, n, offsets, with_mask=True, capacity=None):
        self.n = n
        self.offsets = np.asarray(offsets, np.uint32)
        self.K = len(self.offsets) - 1
        self.offs_dev = vgc.offsets_tensor(self.offsets)
        self.r = torch.zeros(n, dtype=torch.float32, device="cuda")
        self.v = torch.zeros(n, dtype=torch.float32, device="cuda")
        self.out = vgc.MessageBuffers(n if capacity is None else capacity, self.K, n, with_mask=with_mask)
        ws_bytes = vgc.vgc_compress_workspace_bytes(n, self.K)
        self.ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")

    def step(self, g, s, alpha, zeta):
        self.out.counters.zero_()
        vgc.vgc_compress(g, s, self.r, self.v, self.offs_dev, alpha, zeta, self.out, self.ws)
        return self.out.read()


class OracleCompressor:
    def __init__(self, n, offsets):
        self.offsets = np.asarray(offsets, np.uint32)
        self.r = np.zeros(n, F32)
        self.v = np.zeros(n, F32)

    def step(self, g, s, alpha, zeta, capacity=None, want_mask=True):
        return oracle.compress(g, s, self.r, self.v, self.offsets, alpha, zeta, capacity=capacity,
                               want_mask=want_mask)


def assert_same_message(got, want, check_mask=True):
    """got: dict from MessageBuffers.read(); want: oracle.Message.  Bit-exact."""
    assert got["dev_status"] == 0
    assert got["n_criterion"] == want.n_criterion
    assert got["nnz"] == want.nnz
    assert got["n_dropped"] == want.n_dropped
    assert np.array_equal(got["group_exp"], want.group_exp)
    assert np.array_equal(got["words"], want.words)
    if check_mask and want.mask is not None and got["mask"] is not None:
        assert np.array_equal(got["mask"], want.mask)


def assert_same_state(gpu: GpuCompressor, cpu: OracleCompressor):
    assert np.array_equal(gpu.r.cpu().numpy().view(np.uint32), cpu.r.view(np.uint32))
    assert np.array_equal(gpu.v.cpu().numpy().view(np.uint32), cpu.v.view(np.uint32))


def random_offsets(rng, n, K):
    """K groups over [0, n): random cut points (duplicates give empty groups)."""
    cuts = np.sort(rng.integers(0, n + 1, K - 1)) if K > 1 else np.zeros(0, np.int64)
    return np.concatenate([[0], cuts, [n]]).astype(np.uint32)


def noise_gs(n, batch, seed, device="cuda", sigma_exp_range=(-12, 2)):
    """g = sum a / B, s = sum (a/B)^2 from per-parameter noise with a small mean and a
    per-parameter magnitude spread over many binades (exercises the quantiser's range)."""
    gen = torch.Generator(device=device); gen.manual_seed(seed)
    a = torch.empty((batch, n), dtype=torch.float32, device=device).normal_(generator=gen)
    mag = torch.randint(sigma_exp_range[0], sigma_exp_range[1], (n,), generator=gen, device=device).float().exp2()
    a = (a + 0.3) * mag
    g = a.sum(0) / batch
    s = (a / batch).square().sum(0)
    return g.contiguous(), s.contiguous()
