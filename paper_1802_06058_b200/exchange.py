"""The exchange step of CommunicateAndUpdate (Sec. 4.3): every worker receives every worker's packed message
(an allgatherv -- messages differ in length) and decodes their sum into the dense update.

The collective is torch.distributed's (NCCL on GPUs, gloo in the CPU tests); the decode is the library's
``vgc_decode_sum``.  The messages are padded to a common length for the gather: the length is either given
(``pad_to``: no host synchronisation, e.g. a capacity agreed once) or the largest count among the ranks (one
small gather of the counts and one host read).  Padding words are never decoded: each message's own count
travels with it.
"""
from typing import Optional, Tuple

import torch
import torch.distributed as dist


def allgather_messages(words: torch.Tensor, nnz: torch.Tensor, group_exp: torch.Tensor, group=None,
                       pad_to: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """words int32 [>= nnz], nnz int32 [1], group_exp int32 [K] of this rank ->
    (all_words int32 [W, L], all_nnz int32 [W], all_exp int32 [W, K]); row w is rank w's message."""
    if not dist.is_available() or not dist.is_initialized():
        L = int(nnz.item()) if pad_to is None else int(pad_to)
        L = max((L + 3) // 4 * 4, 4)
        buf = torch.zeros(L, dtype=torch.int32, device=words.device)
        take = min(L, words.numel())
        buf[:take] = words[:take]
        return buf.unsqueeze(0), nnz.reshape(1).clone(), group_exp.unsqueeze(0).clone()
    W = dist.get_world_size(group)
    all_nnz = torch.empty(W, dtype=torch.int32, device=nnz.device)
    dist.all_gather_into_tensor(all_nnz, nnz.reshape(1).contiguous(), group=group)
    L = int(all_nnz.max().item()) if pad_to is None else int(pad_to)       # host read only when no length is agreed
    L = max((L + 3) // 4 * 4, 4)        # rows on 16-byte boundaries: the decoder then reads them 16 bytes at a time
    mine = torch.zeros(L, dtype=torch.int32, device=words.device)
    take = min(L, words.numel())
    mine[:take] = words[:take]
    all_words = torch.empty(W * L, dtype=torch.int32, device=words.device)
    dist.all_gather_into_tensor(all_words, mine, group=group)
    all_exp = torch.empty(W * group_exp.numel(), dtype=torch.int32, device=group_exp.device)
    dist.all_gather_into_tensor(all_exp, group_exp.contiguous(), group=group)
    return all_words.view(W, L), all_nnz, all_exp.view(W, group_exp.numel())


def exchange_and_decode(out, group_offsets: torch.Tensor, u: torch.Tensor, dev_status: torch.Tensor, group=None,
                        pad_to: Optional[int] = None, stream=None) -> torch.Tensor:
    """Gather every rank's message (``out``: this rank's MessageBuffers after vgc_compress) and write the mean
    of the decoded messages into ``u`` (every element written)."""
    from . import vgc_decode_sum
    all_words, all_nnz, all_exp = allgather_messages(out.words, out.counters[0:1], out.group_exp[:out.K], group, pad_to)
    W = all_words.shape[0]
    views = [(all_words[w], all_nnz[w:w + 1], all_exp[w]) for w in range(W)]
    return vgc_decode_sum(views, group_offsets, 1.0 / W, u, dev_status, stream=stream)
