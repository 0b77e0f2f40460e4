"""World-size-2 checks on CPU (gloo): the benchmark's per-rank sharding is by worker (independent replicas,
different seeds, no data-path collective); what the ranks share is the max-over-ranks timing reduction and
the rule that only rank 0 reports."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
from paper_1802_06058_b200 import workloads
dist.init_process_group("gloo")
rank = dist.get_rank()
got = bench.max_over_ranks(10.0 + rank)             # device-timed ms of this rank -> max over ranks
assert got == 10.0 + dist.get_world_size() - 1, got
# replicas draw different inputs: seeds differ by worker, equal for equal worker
a = workloads.seed_for(2, worker=rank * 16, step=0, layer=3, tensor=0)
gathered = [None, None]
dist.all_gather_object(gathered, a)
assert gathered[0] != gathered[1]
assert workloads.seed_for(2, 16, 0, 3, 0) == workloads.seed_for(2, 16, 0, 3, 0)
dist.barrier()
dist.destroy_process_group()
sys.stdout.write("rank%dok\n" % rank); sys.stdout.flush()
"""


def _free_port():
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


def _torchrun(args, timeout=600):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    for attempt in range(2):                     # a port can be taken between the probe and the launch
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
               "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), *args]
        res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)
        if res.returncode == 0:
            break
    return res


def test_max_over_ranks_and_seeding_world_size_2(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    res = _torchrun([str(script)])
    assert res.returncode == 0, res.stdout + res.stderr
    assert "rank0ok" in res.stdout and "rank1ok" in res.stdout


def test_reference_arm_under_torchrun_prints_one_line_from_rank_0():
    res = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--workload", "dense", "--steps", "1",
                     "--warmup", "0"])
    assert res.returncode == 0, res.stdout + res.stderr
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["cpu_baseline"]["kind"] == "oracle"
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["value"] > 0


EXCHANGE_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import numpy as np, torch, torch.distributed as dist
from paper_1802_06058_b200 import exchange
dist.init_process_group("gloo")
rank, W = dist.get_rank(), dist.get_world_size()
# messages of different lengths (rank 0: 5 words, rank 1: 11 words), K = 3 per-tensor exponents
def message(r):
    n = 5 + 6 * r
    words = (torch.arange(n, dtype=torch.int32) * 7 + r) * 16 + r
    return words, torch.tensor([n], dtype=torch.int32), torch.tensor([r, -r, 3 * r], dtype=torch.int32)
words, nnz, gexp = message(rank)
padded = torch.cat([words, torch.full((9,), -1, dtype=torch.int32)])        # capacity larger than the message
for pad_to in (None, 16):
    all_words, all_nnz, all_exp = exchange.allgather_messages(padded, nnz, gexp, pad_to=pad_to)
    assert all_words.shape == (W, 12 if pad_to is None else 16), all_words.shape   # the longest message (11), rounded up to 16-byte rows
    for r in range(W):
        w, c, e = message(r)
        assert int(all_nnz[r]) == int(c[0])
        assert torch.equal(all_words[r, :int(c[0])], w)
        assert torch.equal(all_exp[r], e)
dist.barrier()
dist.destroy_process_group()
sys.stdout.write("rank%dok\n" % rank); sys.stdout.flush()
"""


def test_allgather_of_messages_world_size_2(tmp_path):
    script = tmp_path / "exchange_worker.py"
    script.write_text(EXCHANGE_WORKER.format(root=ROOT))
    res = _torchrun([str(script)])
    assert res.returncode == 0, res.stdout + res.stderr
    assert "rank0ok" in res.stdout and "rank1ok" in res.stdout
