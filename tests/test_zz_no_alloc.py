"""vgc_compress_static: the variant of vgc_compress for callers that cannot allocate device memory
(memory planned in full beforehand, plug-ins called inside another framework's step, hosts that lend
only the call's tensors).  Its scratch is a fixed array inside the library, so it must give exactly what
vgc_compress gives with a caller-provided workspace -- also on a second call, which finds the first
call's leftovers in the shared array.  Collected last on purpose: a run that stops at the first failure
has then already run every other test."""
import numpy as np
import pytest
import torch

import paper_1802_06058_b200 as vgc
from gpu_harness import noise_gs, random_offsets

pytestmark = pytest.mark.gpu


def _run(n, offs, gs_list, use_static):
    offs_dev = vgc.offsets_tensor(offs)
    K = len(offs) - 1
    r = torch.zeros(n, device="cuda"); v = torch.zeros(n, device="cuda")
    out = vgc.MessageBuffers(n, K, n, with_mask=True)
    ws = None if use_static else torch.empty(vgc.vgc_compress_workspace_bytes(n, K), dtype=torch.uint8, device="cuda")
    results = []
    for g, s in gs_list:
        out.counters.zero_()
        if use_static:
            vgc.vgc_compress_static(g, s, r, v, offs_dev, 2.0, 0.999, out)
        else:
            vgc.vgc_compress(g, s, r, v, offs_dev, 2.0, 0.999, out, ws)
        res = out.read()
        res["r"] = r.cpu().numpy().copy(); res["v"] = v.cpu().numpy().copy()
        results.append(res)
    return results


def test_static_scratch_matches_workspace_variant_on_two_calls_in_a_row():
    n = 1_000_003                                   # ragged tail, several hundred tiles
    offs = random_offsets(np.random.default_rng(11), n, 7)
    # second call: a different, sparser problem, so stale counts and staged pairs of the first call are
    # still lying in the scratch beyond what the second call writes
    gs = [noise_gs(n, 4, seed=501), noise_gs(n, 16, seed=502)]
    want = _run(n, offs, gs, use_static=False)
    got = _run(n, offs, gs, use_static=True)
    for a, b in zip(got, want):
        assert a["dev_status"] == 0 and b["dev_status"] == 0
        for key in ("nnz", "n_criterion", "n_dropped"):
            assert a[key] == b[key]
        assert a["nnz"] > 1000
        for key in ("words", "group_exp", "mask", "r", "v"):
            assert np.array_equal(a[key], b[key]), key


def test_static_scratch_rejects_buffers_beyond_its_size():
    n = vgc.VGC_COMPRESS_STATIC_MAX_PARAMS + 4
    t = torch.zeros(n, device="cuda")
    offs = vgc.offsets_tensor(np.array([0, n], np.uint32))
    out = vgc.MessageBuffers(16, 1, n)
    with pytest.raises(vgc.VgcError) as err:
        vgc.vgc_compress_static(t, t, t.clone(), t.clone(), offs, 2.0, 0.999, out)
    assert err.value.status == 2                   # VGC_ERR_UNSUPPORTED, nothing was enqueued
