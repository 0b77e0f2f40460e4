"""GPU parity: index compression of packed messages (vgc_pack_indices / vgc_unpack_indices) against the CPU oracle --
the byte stream must be the oracle's, byte for byte, and the round trip must give the words back."""
import numpy as np
import pytest
import torch

import oracle
import paper_1802_06058_b200 as vgc
from paper_1802_06058_b200 import workloads
from gpu_harness import Guarded

pytestmark = pytest.mark.gpu


def gpu_pack(words_dev, nnz, capacity=None):
    max_words = words_dev.numel()
    cap = vgc.vgc_pack_bound_bytes(max_words) if capacity is None else capacity
    packed = Guarded(cap, torch.uint8, fill=0xEE)
    ws = Guarded(vgc.vgc_pack_workspace_bytes(max_words), torch.uint8)
    nbytes = torch.zeros(1, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    count = torch.tensor([nnz], dtype=torch.int32, device="cuda")
    vgc.vgc_pack_indices(words_dev, count, packed.t, nbytes, status, ws.t)
    torch.cuda.synchronize()
    packed.check("packed stream"); ws.check("pack workspace")
    return packed.t, int(nbytes.item()), int(status.item()), count


@pytest.mark.parametrize("n,density", [(1 << 20, 1e-2), (1 << 22, 1e-3), (1 << 28, 2e-5), (5000, 0.9), (100000, 0.2),
                                       (300, 1.0), (25502912, 0.05)])
def test_stream_is_the_oracles_and_round_trips(n, density):
    offs = np.array([0, n], np.uint32)
    words, _ = workloads.random_message(n, offs, density, seed=int(n * density) + 7, device="cuda")
    m = words.numel()
    host = words.cpu().numpy().view(np.uint32)
    want = oracle.pack_indices(host)
    packed, nbytes, status, count = gpu_pack(words, m)
    assert status == 0 and nbytes == want.size
    assert np.array_equal(packed[:nbytes].cpu().numpy(), want)
    if 1e-3 <= density <= 1e-2 and m > 1000:
        assert nbytes < 0.7 * 4 * m
    back = Guarded(m, torch.int32, fill=0)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    vgc.vgc_unpack_indices(packed, count, back.t, st)
    torch.cuda.synchronize()
    back.check("unpacked words")
    assert int(st.item()) == 0
    assert np.array_equal(back.t.cpu().numpy().view(np.uint32), host)
    assert np.array_equal(oracle.unpack_indices(packed[:nbytes].cpu().numpy(), m), host)


def test_count_below_the_buffer_and_edge_counts():
    n = 200000
    words, _ = workloads.random_message(n, np.array([0, n], np.uint32), 0.05, seed=3, device="cuda")
    host = words.cpu().numpy().view(np.uint32)
    for m in (0, 1, 255, 256, 257, 512, 2049, host.size):
        want = oracle.pack_indices(host[:m])
        packed, nbytes, status, count = gpu_pack(words, m)
        assert status == 0 and nbytes == want.size, m
        assert np.array_equal(packed[:nbytes].cpu().numpy(), want), m
        back = torch.full((max(m, 1),), -1, dtype=torch.int32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        vgc.vgc_unpack_indices(packed, count, back, st)
        assert int(st.item()) == 0 and np.array_equal(back[:m].cpu().numpy().view(np.uint32), host[:m]), m


def test_small_buffer_is_reported_not_overrun():
    n = 100000
    words, _ = workloads.random_message(n, np.array([0, n], np.uint32), 0.1, seed=5, device="cuda")
    host = words.cpu().numpy().view(np.uint32)
    want = oracle.pack_indices(host)
    packed, nbytes, status, _ = gpu_pack(words, host.size, capacity=want.size // 2)
    assert status == vgc.VGC_DEV_CAPACITY and nbytes == want.size
    assert np.array_equal(packed.cpu().numpy(), want[:want.size // 2])


def test_damaged_stream_is_refused_run_by_run():
    n = 100000
    words, _ = workloads.random_message(n, np.array([0, n], np.uint32), 0.1, seed=6, device="cuda")
    host = words.cpu().numpy().view(np.uint32)
    packed, nbytes, _, count = gpu_pack(words, host.size)
    runs = (host.size + 255) // 256
    damaged = packed.clone()
    table = damaged[:4 * (runs + 1)].cpu().numpy().view("<u4").copy()
    table[3] += 1                                             # run 2 ends one byte late, run 3 starts one byte late
    damaged[:4 * (runs + 1)] = torch.from_numpy(table.view(np.uint8)).cuda()
    back = torch.zeros(host.size, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    vgc.vgc_unpack_indices(damaged, count, back, st)
    got = back.cpu().numpy().view(np.uint32)
    assert int(st.item()) & vgc.VGC_DEV_RANGE
    ok = np.ones(host.size, bool); ok[2 * 256:4 * 256] = False
    assert np.array_equal(got[ok], host[ok])                 # the other runs are untouched by the damage
    assert np.all(got[2 * 256:3 * 256] == 0xFFFFFFFF)        # run 2 no longer ends on a number's last byte: refused


def test_packed_message_decodes_to_the_same_update():
    """compress -> pack -> (the wire) -> unpack -> decode gives the update of the unpacked message, bit for bit."""
    from gpu_harness import GpuCompressor, noise_gs, random_offsets
    n = 400003
    offs = random_offsets(np.random.default_rng(12), n, 6)
    gpu = GpuCompressor(n, offs, with_mask=False)
    g, s = noise_gs(n, 4, seed=91)
    msg = gpu.step(g, s, 2.0, 0.999)
    packed, nbytes, status, _ = gpu_pack(gpu.out.words, msg["nnz"])
    assert status == 0 and nbytes < 4 * msg["nnz"]
    back = torch.zeros(msg["nnz"], dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    vgc.vgc_unpack_indices(packed, gpu.out.counters[0:1], back, st)
    u0 = torch.zeros(n, device="cuda"); u1 = torch.zeros(n, device="cuda")
    vgc.vgc_decode_sum([gpu.out], gpu.offs_dev, 1.0, u0, st)
    vgc.vgc_decode_sum([(back, gpu.out.counters[0:1], gpu.out.group_exp)], gpu.offs_dev, 1.0, u1, st)
    assert int(st.item()) == 0 and torch.equal(u0, u1)
    ref = np.zeros(n, np.float32)
    oracle.decode_accumulate([(oracle.unpack_indices(packed[:nbytes].cpu().numpy(), msg["nnz"]), msg["group_exp"])], offs, 1.0, ref)
    assert np.array_equal(u1.cpu().numpy(), ref)
