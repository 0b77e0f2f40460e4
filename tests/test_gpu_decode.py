"""GPU parity: vgc_decode_accumulate / vgc_decode_sum against the CPU oracle.  The bound is 1e-6 absolute.  Where the
decoder adds in message order (the ordered form of dense calls, and any element hit by at most two messages) and where
it sums exactly under a power-of-two scale (vgc_decode_sum's exact form) the result must be the oracle's bit for bit;
where it applies the scale to the exact sum, the difference is bounded by the roundings of the sequential sum."""
import numpy as np
import pytest
import torch

import oracle
import paper_1802_06058_b200 as vgc
from paper_1802_06058_b200 import workloads
from gpu_harness import Guarded, guarded_like, random_offsets

pytestmark = pytest.mark.gpu
F32 = np.float32
ATOL = 1e-6


def _decode_both(n, offs, msgs, scale, u0=None):
    """msgs: list of (words int32 cuda, gexp int32 cuda)."""
    gu = Guarded(n, fill=0.0) if u0 is None else guarded_like(u0)      # u between guard bands
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    pad = torch.zeros(4, dtype=torch.int32, device="cuda")      # an empty message still needs a valid pointer
    triples = [(w if w.numel() else pad, torch.tensor([w.numel()], dtype=torch.int32, device="cuda"), e)
               for w, e in msgs]
    vgc.vgc_decode_accumulate(triples, vgc.offsets_tensor(offs), scale, gu.t, status)
    gu.check("u")
    u_ref = np.zeros(n, F32) if u0 is None else u0.cpu().numpy().copy()
    bad = oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy()) for w, e in msgs],
                                   offs, scale, u_ref)
    return gu.t.cpu().numpy(), u_ref, int(status.item()), bad


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


DENSE_CASES = [(400003, 9, 5, 0.1), (3 * 24576 * 2 + 5, 3, 9, 0.15), (2500000, 40, 17, 0.05), (1 << 20, 54, 8, 0.14),
               (700001, 5, 3, 0.9), (300000, 2, 64, 0.004), (33, 1, 2, 1.0), (5000, 1, 1, 0.5)]


def _off_boundary(words):
    """The same words at an address that is 4 bytes past a 16-byte boundary: such a message takes the ordered form."""
    buf = torch.empty(words.numel() + 1, dtype=words.dtype, device=words.device)
    buf[1:] = words
    return buf[1:]


@pytest.mark.parametrize("n,K,W,density", DENSE_CASES)
def test_ordered_form_adds_in_message_order_bit_for_bit(n, K, W, density):
    """At one word per eight elements or more the decoder moves u through shared memory; messages that do not start on
    16-byte boundaries are added message after message -- the oracle's own sequence of fp32 additions -- so the result
    is the oracle's, bit for bit, with several messages hitting most elements and a scale that is not a power of two."""
    offs = random_offsets(np.random.default_rng(21), n, K)
    msgs = [workloads.random_message(n, offs, density * (1.5 if w % 2 else 0.5), seed=900 + w, device="cuda",
                                     exp_lo=-12, exp_hi=3) for w in range(W)]
    msgs = [(_off_boundary(w), e) for w, e in msgs]
    assert sum(m[0].numel() for m in msgs) * 8 >= n
    u0 = torch.randn(n, device="cuda") * 1e-2
    got, want, status, _ = _decode_both(n, offs, msgs, 1.0 / 3, u0=u0)
    assert status == 0
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # the same messages written instead of added
    gu = Guarded(n, fill=float("nan"))
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    triples = [(w, torch.tensor([w.numel()], dtype=torch.int32, device="cuda"), e) for w, e in msgs]
    vgc.vgc_decode_sum(triples, vgc.offsets_tensor(offs), 1.0 / 3, gu.t, st)
    gu.check("u")
    ref = np.zeros(n, F32)
    oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy()) for w, e in msgs], offs, 1.0 / 3, ref)
    assert int(st.item()) == 0 and np.array_equal(gu.t.cpu().numpy().view(np.uint32), ref.view(np.uint32))


@pytest.mark.parametrize("scale", [1.0 / 3, 0.25, -1.0 / 7])
@pytest.mark.parametrize("n,K,W,density", DENSE_CASES)
def test_exact_form_differs_from_the_sequential_sum_by_its_roundings_only(n, K, W, density, scale):
    """Messages on 16-byte boundaries whose exponents lie close together are summed exactly and scaled once; the
    sequential sum rounds after every message.  Per element the two differ by at most the sequential sum's W roundings
    plus the exact form's two, each half an ulp of a number no larger than |u0| + sum |scale * value|.  Elements no
    word points at keep their bits.  (Tensors whose exponents lie too far apart take the ordered form: no difference.)"""
    offs = random_offsets(np.random.default_rng(21), n, K)
    msgs = [workloads.random_message(n, offs, density * (1.5 if w % 2 else 0.5), seed=900 + w, device="cuda",
                                     exp_lo=-9, exp_hi=-4) for w in range(W)]
    assert sum(m[0].numel() for m in msgs) * 8 >= n
    u0 = torch.randn(n, device="cuda") * 1e-2
    u0[::7] = -0.0
    got, want, status, _ = _decode_both(n, offs, msgs, scale, u0=u0)
    assert status == 0
    mag = np.abs(u0.cpu().numpy()).astype(np.float64)
    touched = np.zeros(n, bool)
    for w, e in msgs:
        one = np.zeros(n, F32)
        oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy())], offs, scale, one)
        mag += np.abs(one)
        touched[w.cpu().numpy().view(np.uint32) >> 4] = True
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    assert np.all(err <= (W + 2) * 2.0 ** -24 * mag) and err.max() <= ATOL
    assert np.array_equal(got.view(np.uint32)[~touched], u0.cpu().numpy().view(np.uint32)[~touched])
    # the same messages written instead of added: scale times the exact sum, one rounding
    gu = Guarded(n, fill=float("nan"))
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    triples = [(w, torch.tensor([w.numel()], dtype=torch.int32, device="cuda"), e) for w, e in msgs]
    vgc.vgc_decode_sum(triples, vgc.offsets_tensor(offs), scale, gu.t, st)
    gu.check("u")
    ref = np.zeros(n, F32)
    oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy()) for w, e in msgs], offs, scale, ref)
    err = np.abs(gu.t.cpu().numpy().astype(np.float64) - ref.astype(np.float64))
    assert int(st.item()) == 0 and np.all(err <= (W + 2) * 2.0 ** -24 * (mag - np.abs(u0.cpu().numpy())))
    if scale == 0.25:                                         # a power of two: every product exact, the same bits
        assert np.array_equal(gu.t.cpu().numpy().view(np.uint32), ref.view(np.uint32))


@pytest.mark.parametrize("n,K,W,density,exps,scale", [(1 << 20, 54, 8, 0.14, (-10, -8), 0.125), (2500000, 40, 17, 0.05, (-14, -9), 1.0),
                                                      (700001, 5, 64, 0.05, (-3, 0), 2.0 ** -6), (400003, 9, 5, 0.3, (-20, -6), 0.5),
                                                      (300000, 3, 4, 0.5, (-125, -120), 1.0), (300000, 3, 4, 0.5, (100, 110), 0.25)])
def test_decode_sum_over_the_exponent_range_bit_for_bit(n, K, W, density, exps, scale):
    """vgc_decode_sum with a power-of-two scale and per-tensor exponents that lie close together accumulates integer
    multiples of one power of two in any order (no barrier between messages, no search for the runs' ends); the sums
    are exact, so the result is still the oracle's sequential sum, bit for bit.  Wider exponent ranges (fourth case),
    values next to the smallest normal number and large ones take whichever form applies tile by tile."""
    offs = random_offsets(np.random.default_rng(31), n, K)
    msgs = [workloads.random_message(n, offs, density, seed=700 + w, device="cuda", exp_lo=exps[0], exp_hi=exps[1])
            for w in range(W)]
    gu = Guarded(n, fill=float("nan"))
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    triples = [(w, torch.tensor([w.numel()], dtype=torch.int32, device="cuda"), e) for w, e in msgs]
    vgc.vgc_decode_sum(triples, vgc.offsets_tensor(offs), scale, gu.t, st)
    gu.check("u")
    ref = np.zeros(n, F32)
    oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy()) for w, e in msgs], offs, scale, ref)
    assert int(st.item()) == 0 and np.array_equal(gu.t.cpu().numpy().view(np.uint32), ref.view(np.uint32))


def test_more_messages_than_one_launch_takes():
    """70 messages are decoded by two launches (64 + 6); the second adds to what the first wrote.  With the workers'
    exponents close together both take the exact form: the result is within the roundings of the sequential sum."""
    n, K, W, scale = 500003, 6, 70, 1.0 / 70
    offs = random_offsets(np.random.default_rng(3), n, K)
    msgs = [workloads.random_message(n, offs, 0.01, seed=1500 + w, device="cuda", exp_seed=77) for w in range(W)]
    assert sum(m[0].numel() for m in msgs) * 8 >= n
    for entry in ("vgc_decode_sum", "vgc_decode_accumulate"):
        gu = Guarded(n, fill=0.0)
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        triples = [(w, torch.tensor([w.numel()], dtype=torch.int32, device="cuda"), e) for w, e in msgs]
        getattr(vgc, entry)(triples, vgc.offsets_tensor(offs), scale, gu.t, st)
        gu.check("u")
        ref = np.zeros(n, F32)
        mag = np.zeros(n, np.float64)
        for w, e in msgs:
            one = np.zeros(n, F32)
            oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy())], offs, scale, one)
            mag += np.abs(one)
        oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy()) for w, e in msgs], offs, scale, ref)
        err = np.abs(gu.t.cpu().numpy().astype(np.float64) - ref.astype(np.float64))
        assert int(st.item()) == 0 and np.all(err <= (W + 4) * 2.0 ** -24 * mag) and err.max() <= ATOL


@pytest.mark.parametrize("shift", [0, 1, 2, 3])
def test_decode_sum_reads_messages_at_any_word_alignment(shift):
    """The exact form reads the messages 16 bytes at a time from the boundary before each cursor; a message that does
    not start on a 16-byte boundary takes the ordered form.  Same bits either way, and nothing before a message's
    first word or after its last one changes the result: each message sits between two words that point at element 0."""
    n, K, W = 600001, 7, 6
    offs = random_offsets(np.random.default_rng(77), n, K)
    msgs = [workloads.random_message(n, offs, 0.2, seed=1200 + w, device="cuda", exp_lo=-9, exp_hi=-7) for w in range(W)]
    triples = []
    for w, (words, exps) in enumerate(msgs):
        m = words.numel() - (w % 4)                                 # counts that are not multiples of four
        buf = torch.full((m + shift + 8,), 0x0000000F, dtype=words.dtype, device="cuda")      # element 0, largest code
        buf[shift:shift + m] = words[:m]
        msgs[w] = (words[:m], exps)
        triples.append((buf[shift:shift + m], torch.tensor([m], dtype=torch.int32, device="cuda"), exps))
    gu = Guarded(n, fill=float("nan"))
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    vgc.vgc_decode_sum(triples, vgc.offsets_tensor(offs), 0.25, gu.t, st)
    gu.check("u")
    ref = np.zeros(n, F32)
    oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy()) for w, e in msgs], offs, 0.25, ref)
    assert int(st.item()) == 0 and np.array_equal(gu.t.cpu().numpy().view(np.uint32), ref.view(np.uint32))


@pytest.mark.parametrize("n,K,W,density", [(400003, 9, 5, 0.002), (2500000, 40, 17, 0.0005)])
def test_sparse_calls_are_relative_to_the_sum(n, K, W, density):
    """Sparse calls add with atomics in any order: an element hit by three or more messages may differ from the
    sequential sum in the last bit, so the bound is a few ulps of the element's own sum, far inside 1e-6."""
    offs = random_offsets(np.random.default_rng(22), n, K)
    msgs = [workloads.random_message(n, offs, density, seed=950 + w, device="cuda", exp_lo=-12, exp_hi=3) for w in range(W)]
    u0 = torch.randn(n, device="cuda") * 1e-2
    got, want, status, _ = _decode_both(n, offs, msgs, 0.5, u0=u0)
    assert status == 0
    mag = np.abs(u0.cpu().numpy()).astype(np.float64)
    np.add.at(mag, np.concatenate([(m[0].cpu().numpy().view(np.uint32) >> 4) for m in msgs]), 8.0)   # |value| <= 2^3
    err = np.abs(got.astype(np.float64) - want)
    assert np.all(err <= 4 * 2.0 ** -24 * mag)


def test_truncated_message_is_decoded_up_to_its_buffer():
    """A message cut short at the sender (VGC_DEV_CAPACITY) carries the count that was needed, not the count that was
    written: the decoder applies the words the buffer holds, reports VGC_DEV_CAPACITY and reads nothing beyond."""
    from gpu_harness import noise_gs
    n = 300007
    offs = random_offsets(np.random.default_rng(5), n, 4)
    offs_dev = vgc.offsets_tensor(offs)
    g, s = noise_gs(n, 4, seed=61)
    r = torch.zeros(n, device="cuda"); v = torch.zeros(n, device="cuda")
    full = vgc.MessageBuffers(n, 4, n)
    ws = torch.empty(vgc.vgc_compress_workspace_bytes(n, 4), dtype=torch.uint8, device="cuda")
    vgc.vgc_compress(g, s, r, v, offs_dev, 2.0, 0.999, full, ws)
    whole = full.read()
    cap = whole["nnz"] // 2
    short = vgc.MessageBuffers(cap, 4, n)
    guard = Guarded(cap, torch.int32)
    short.words = guard.t
    r.zero_(); v.zero_()
    vgc.vgc_compress(g, s, r, v, offs_dev, 2.0, 0.999, short, ws)
    guard.check("words")
    cut = short.read()
    assert cut["dev_status"] == vgc.VGC_DEV_CAPACITY and cut["nnz"] == whole["nnz"]
    assert np.array_equal(cut["words"], whole["words"][:cap])
    for overwrite in (False, True):
        u = torch.zeros(n, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        vgc.vgc_decode_accumulate([short, full], offs_dev, 1.0, u, status, overwrite=overwrite)
        want = np.zeros(n, F32)
        oracle.decode_accumulate([(whole["words"][:cap], whole["group_exp"]), (whole["words"], whole["group_exp"])],
                                 offs, 1.0, want)
        assert int(status.item()) == vgc.VGC_DEV_CAPACITY
        assert np.array_equal(u.cpu().numpy(), want)


@pytest.mark.parametrize("density", [0.3, 0.001])
@pytest.mark.parametrize("entry", ["vgc_decode_accumulate", "vgc_decode_sum"])
def test_unsorted_words_never_touch_a_wrong_element(density, entry):
    """Messages must be sorted; one that is not may lose words (VGC_DEV_RANGE says so), but no word is ever added to
    an element other than its own and nothing outside u is written."""
    n, W = 200003, 3
    offs = np.array([0, 70000, n], np.uint32)
    msgs = [workloads.random_message(n, offs, density, seed=30 + w, device="cuda") for w in range(W)]
    words = msgs[1][0].clone()
    m = words.numel()
    words[m // 3], words[2 * m // 3] = words[2 * m // 3].clone(), words[m // 3].clone()      # two words far out of place
    msgs[1] = (words, msgs[1][1])
    gu = Guarded(n, fill=0.0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    triples = [(w, torch.tensor([w.numel()], dtype=torch.int32, device="cuda"), e) for w, e in msgs]
    getattr(vgc, entry)(triples, vgc.offsets_tensor(offs), 1.0, gu.t, status)        # u starts as zeros: same result
    gu.check("u")
    ref = np.zeros(n, F32)
    oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy()) for w, e in msgs], offs, 1.0, ref)
    got = gu.t.cpu().numpy()
    differs = np.flatnonzero(got != ref)
    # only elements the damaged message points at may differ, and only by that message's own words being left out
    pointed = set((words.cpu().numpy().view(np.uint32) >> 4).tolist())
    assert all(int(i) in pointed for i in differs)
    if differs.size:
        assert int(status.item()) & vgc.VGC_DEV_RANGE


@pytest.mark.parametrize("n,K,W,density", [(5, 1, 1, 1.0), (100003, 7, 4, 0.0005), (1 << 20, 54, 8, 0.1),
                                           (2500001, 16, 70, 0.02)])
def test_decode_sum_overwrites_whatever_u_held(n, K, W, density):
    offs = random_offsets(np.random.default_rng(n + W), n, K)
    msgs = [workloads.random_message(n, offs, density, seed=workloads.seed_for(6, w, 0, 0, 2), device="cuda")
            for w in range(W)]
    gu = Guarded(n, fill=float("nan"))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    pad = torch.zeros(4, dtype=torch.int32, device="cuda")
    triples = [(w if w.numel() else pad, torch.tensor([w.numel()], dtype=torch.int32, device="cuda"), e) for w, e in msgs]
    vgc.vgc_decode_sum(triples, vgc.offsets_tensor(offs), 0.25, gu.t, status)
    gu.check("u")
    want = np.zeros(n, F32)
    oracle.decode_accumulate([(w.cpu().numpy().view(np.uint32), e.cpu().numpy()) for w, e in msgs], offs, 0.25, want)
    assert int(status.item()) == 0
    assert np.abs(gu.t.cpu().numpy().astype(np.float64) - want).max() <= ATOL


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
