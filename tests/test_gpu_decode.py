"""GPU parity: vgc_decode_accumulate against the CPU oracle (absolute error <= 1e-6)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1802_06058_b200 as vgc
from paper_1802_06058_b200 import workloads
from gpu_harness import random_offsets

pytestmark = pytest.mark.gpu
F32 = np.float32
ATOL = 1e-6


def _decode_both(n, offs, msgs, scale, u0=None):
    """msgs: list of (words int32 cuda, gexp int32 cuda)."""
    u = torch.zeros(n, dtype=torch.float32, device="cuda") if u0 is None else u0.clone()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    pad = torch.zeros(4, dtype=torch.int32, device="cuda")      # an empty message still needs a valid pointer
    triples = [(w if w.numel() else pad, torch.tensor([w.numel()], dtype=torch.int32, device="cuda"), e)
               for w, e in msgs]
    vgc.vgc_decode_accumulate(triples, vgc.offsets_tensor(offs), scale, u, status)
    u_ref = np.zeros(n, F32) if u0 is None else u0.cpu().numpy().copy()
    bad = oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy()) for w, e in msgs],
                                   offs, scale, u_ref)
    return u.cpu().numpy(), u_ref, int(status.item()), bad


@pytest.mark.parametrize("n,K,W,density", [(1000, 1, 1, 0.5), (100003, 7, 4, 0.01), (1 << 20, 54, 8, 0.1),
                                           (3000001, 16, 70, 0.003), (65537, 1200, 3, 0.2)])
def test_random_messages(n, K, W, density):
    offs = random_offsets(np.random.default_rng(n + W), n, K)
    msgs = [workloads.random_message(n, offs, density, seed=workloads.seed_for(5, w, 0, 0, 2), device="cuda")
            for w in range(W)]
    got, want, status, bad = _decode_both(n, offs, msgs, 1.0 / 4)
    assert status == 0 and bad == 0
    assert np.abs(got.astype(np.float64) - want).max() <= ATOL
    assert (want != 0).mean() > density * 0.5


def test_max_contention_and_existing_content():
    n, W = 50000, 16
    offs = np.array([0, 20000, n], np.uint32)
    one = workloads.random_message(n, offs, 0.05, seed=9, device="cuda")
    u0 = torch.randn(n, device="cuda") * 1e-3
    got, want, status, _ = _decode_both(n, offs, [one] * W, 1.0, u0=u0)
    assert status == 0
    assert np.abs(got.astype(np.float64) - want).max() <= ATOL


def test_out_of_range_word_sets_flag_and_is_skipped():
    n = 4096
    offs = np.array([0, n], np.uint32)
    words, gexp = workloads.random_message(n, offs, 0.1, seed=3, device="cuda")
    words = torch.cat([words, torch.tensor([(n << 4) | 1, ((n + 77) << 4) | 9], dtype=torch.int32, device="cuda")])
    got, want, status, bad = _decode_both(n, offs, [(words, gexp)], 1.0)
    assert status == vgc.VGC_DEV_RANGE and bad == 2
    assert np.array_equal(got, want)                      # single message, distinct indices: exact


def test_empty_messages_and_unaligned_word_pointer():
    n = 10000
    offs = np.array([0, n], np.uint32)
    words, gexp = workloads.random_message(n, offs, 0.3, seed=4, device="cuda")
    empty = (words[:0], gexp)
    shifted = (words[1:], gexp)                           # 4-byte aligned only
    got, want, status, _ = _decode_both(n, offs, [empty, shifted], 2.0)
    assert status == 0 and np.array_equal(got, want)


def test_round_trip_of_compressed_messages():
    """Messages produced by vgc_compress on the GPU are consumed straight from device memory."""
    from gpu_harness import GpuCompressor, OracleCompressor, noise_gs
    n, W = 200003, 4
    offs = random_offsets(np.random.default_rng(8), n, 5)
    comps, cpu_msgs = [], []
    for w in range(W):
        gpu, cpu = GpuCompressor(n, offs), OracleCompressor(n, offs)
        g, s = noise_gs(n, 4, seed=40 + w)
        gpu.out.counters.zero_()
        vgc.vgc_compress(g, s, gpu.r, gpu.v, gpu.offs_dev, 2.0, 0.999, gpu.out, gpu.ws)
        m = cpu.step(g.cpu().numpy(), s.cpu().numpy(), 2.0, 0.999)
        comps.append(gpu); cpu_msgs.append((m.words, m.group_exp))
    u = torch.zeros(n, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    vgc.vgc_decode_accumulate([c.out for c in comps], comps[0].offs_dev, 1.0 / W, u, status)
    want = np.zeros(n, F32)
    oracle.decode_accumulate(cpu_msgs, offs, 1.0 / W, want)
    assert int(status.item()) == 0
    assert np.abs(u.cpu().numpy().astype(np.float64) - want).max() <= ATOL


@pytest.mark.parametrize("n,K,W", [(400003, 9, 5), (3 * 24576 * 2 + 5, 3, 9), (2500000, 40, 17)])
def test_every_decode_form_agrees_with_the_oracle(monkeypatch, n, K, W):
    """Default: large tiles through shared memory; VGC_DECODE_PATH=merge: the 4096-element tile form;
    VGC_DECODE_PATH=scatter: one atomic per word."""
    offs = random_offsets(np.random.default_rng(21), n, K)
    msgs = [workloads.random_message(n, offs, 0.15 if w % 2 else 0.002, seed=900 + w, device="cuda") for w in range(W)]
    u0 = torch.randn(n, device="cuda") * 1e-2
    for path in (None, "merge", "scatter"):
        if path:
            monkeypatch.setenv("VGC_DECODE_PATH", path)
        got, want, status, _ = _decode_both(n, offs, msgs, 0.5, u0=u0)
        assert status == 0
        assert np.abs(got.astype(np.float64) - want).max() <= ATOL


@pytest.mark.parametrize("path", [None, "merge", "scatter"])
@pytest.mark.parametrize("n,K,W,density", [(5, 1, 1, 1.0), (100003, 7, 4, 0.0005), (1 << 20, 54, 8, 0.1),
                                           (2500001, 16, 70, 0.02)])
def test_decode_sum_overwrites_whatever_u_held(monkeypatch, path, n, K, W, density):
    if path:
        monkeypatch.setenv("VGC_DECODE_PATH", path)
    offs = random_offsets(np.random.default_rng(n + W), n, K)
    msgs = [workloads.random_message(n, offs, density, seed=workloads.seed_for(6, w, 0, 0, 2), device="cuda")
            for w in range(W)]
    u = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    pad = torch.zeros(4, dtype=torch.int32, device="cuda")
    triples = [(w if w.numel() else pad, torch.tensor([w.numel()], dtype=torch.int32, device="cuda"), e) for w, e in msgs]
    vgc.vgc_decode_sum(triples, vgc.offsets_tensor(offs), 0.25, u, status)
    want = np.zeros(n, F32)
    oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy()) for w, e in msgs], offs, 0.25, want)
    assert int(status.item()) == 0
    assert np.abs(u.cpu().numpy().astype(np.float64) - want).max() <= ATOL


def test_decode_sum_of_no_messages_is_zero():
    n = 12345
    u = torch.full((n,), 3.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    vgc.vgc_decode_sum([], vgc.offsets_tensor(np.array([0, n], np.uint32)), 1.0, u, status)
    assert float(u.abs().max().item()) == 0.0


def test_exchange_and_decode_single_rank():
    """Without a process group the exchange is the identity: the worker decodes its own message."""
    from gpu_harness import GpuCompressor, OracleCompressor, noise_gs
    from paper_1802_06058_b200 import exchange
    n = 150001
    offs = random_offsets(np.random.default_rng(3), n, 6)
    gpu, cpu = GpuCompressor(n, offs), OracleCompressor(n, offs)
    g, s = noise_gs(n, 4, seed=77)
    gpu.out.counters.zero_()
    vgc.vgc_compress(g, s, gpu.r, gpu.v, gpu.offs_dev, 2.0, 0.999, gpu.out, gpu.ws)
    m = cpu.step(g.cpu().numpy(), s.cpu().numpy(), 2.0, 0.999)
    u = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    exchange.exchange_and_decode(gpu.out, gpu.offs_dev, u, status)
    want = np.zeros(n, F32)
    oracle.decode_accumulate([(m.words, m.group_exp)], offs, 1.0, want)
    assert int(status.item()) == 0
    assert np.array_equal(u.cpu().numpy(), want)
