"""Helpers shared by the GPU parity tests: run the CUDA path through the binding and the CPU
oracle on identical bytes and compare."""
import numpy as np
import torch

import oracle
import paper_1802_06058_b200 as vgc

F32 = np.float32


class Guarded:
    """A device buffer with a 4-KB band of 0xA5 bytes on either side (the stand-in for a memory checker: a kernel
    that writes one element before or after a buffer it was given changes a band, and ``check`` sees it).
    ``t`` is the buffer itself, 256-byte aligned, its last byte directly followed by the upper band."""
    BAND = 4096

    def __init__(self, numel, dtype=torch.float32, fill=None, device="cuda"):
        item = torch.empty(0, dtype=dtype).element_size()
        self.nbytes = int(numel) * item
        self.raw = torch.full((2 * self.BAND + self.nbytes,), 0xA5, dtype=torch.uint8, device=device)
        self.t = self.raw[self.BAND:self.BAND + self.nbytes].view(dtype)
        if fill is not None:
            self.t.fill_(fill)

    def check(self, what="buffer"):
        lower, upper = self.raw[:self.BAND], self.raw[self.BAND + self.nbytes:]
        assert bool((lower == 0xA5).all()), f"{what}: bytes below the buffer were overwritten"
        assert bool((upper == 0xA5).all()), f"{what}: bytes above the buffer were overwritten"


def guarded_like(t):
    g = Guarded(t.numel(), t.dtype, device=t.device)
    g.t.copy_(t.reshape(-1))
    return g


class GpuCompressor:
    """State + buffers for repeated vgc_compress calls on one flat buffer."""

    def __init__(self, n, offsets, with_mask=True, capacity=None):
        self.n = n
        self.offsets = np.asarray(offsets, np.uint32)
        self.K = len(self.offsets) - 1
        self.offs_dev = vgc.offsets_tensor(self.offsets)
        # every buffer the kernels write sits between guard bands
        self._r, self._v = Guarded(n, fill=0.0), Guarded(n, fill=0.0)
        self.r, self.v = self._r.t, self._v.t
        cap = n if capacity is None else capacity
        self.out = vgc.MessageBuffers(cap, self.K, n, with_mask=with_mask)
        self._words = Guarded(max(cap, 1), torch.int32)
        self._gexp = Guarded(max(self.K, 1), torch.int32)
        self.out.words, self.out.group_exp = self._words.t, self._gexp.t
        self._mask = None
        if with_mask:
            self._mask = Guarded(n, torch.uint8, fill=0)
            self.out.mask = self._mask.t
        ws_bytes = vgc.vgc_compress_workspace_bytes(n, self.K)
        self._ws = Guarded(ws_bytes, torch.uint8)
        self.ws = self._ws.t

    def check_guards(self):
        for name, gd in (("r", self._r), ("v", self._v), ("words", self._words), ("group_exp", self._gexp),
                         ("mask", self._mask), ("workspace", self._ws)):
            if gd is not None:
                gd.check(name)

    def step(self, g, s, alpha, zeta):
        self.out.counters.zero_()
        vgc.vgc_compress(g, s, self.r, self.v, self.offs_dev, alpha, zeta, self.out, self.ws)
        res = self.out.read()
        self.check_guards()
        return res


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
