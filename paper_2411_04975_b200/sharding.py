"""Host-side plumbing for running one store replica per GPU.

Requests are independent given the global tree, so the batch is sharded by
request and every rank keeps a full replica of the global tree.  The only data
the ranks ever exchange is the text of finished outputs, which every replica
must insert into its global tree in the same order (the paper inserts a
finished request's output into the global tree, Section 3 "Suffix Tree
Construction").  Nothing here touches the trees; it only moves token arrays
and scalars with torch.distributed (NCCL on GPUs, gloo on CPU).
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np
import torch
import torch.distributed as dist


def request_range(rank: int, world: int, batch_per_rank: int) -> range:
    """Global request indices served by `rank` (weak scaling: fixed batch per rank)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    return range(rank * batch_per_rank, (rank + 1) * batch_per_rank)


def max_over_ranks(value: float, device: torch.device) -> float:
    """Slowest rank's time: the figure every multi-GPU number is reported on."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def all_gather_sequences(local: Sequence[np.ndarray], device: torch.device) -> List[np.ndarray]:
    """Every rank's finished outputs, concatenated in rank order (then local order), the
    same list on every rank."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [np.asarray(s, dtype=np.int32) for s in local]
    world = dist.get_world_size()
    lens = np.asarray([len(s) for s in local], dtype=np.int64)
    meta = torch.tensor([len(local), int(lens.sum())], dtype=torch.int64, device=device)
    metas = [torch.zeros_like(meta) for _ in range(world)]
    dist.all_gather(metas, meta)
    max_n = max(int(m[0]) for m in metas)
    max_tok = max(int(m[1]) for m in metas)
    if max_n == 0:
        return []
    pad_len = torch.zeros(max_n, dtype=torch.int64, device=device)
    pad_len[:len(local)] = torch.as_tensor(lens, device=device)
    pad_tok = torch.zeros(max(max_tok, 1), dtype=torch.int32, device=device)
    if lens.sum():
        pad_tok[:int(lens.sum())] = torch.as_tensor(np.concatenate([np.asarray(s, dtype=np.int32) for s in local]),
                                                    device=device)
    all_len = [torch.zeros_like(pad_len) for _ in range(world)]
    all_tok = [torch.zeros_like(pad_tok) for _ in range(world)]
    dist.all_gather(all_len, pad_len)
    dist.all_gather(all_tok, pad_tok)
    out: List[np.ndarray] = []
    for r in range(world):
        n = int(metas[r][0])
        ln = all_len[r][:n].cpu().numpy()
        tok = all_tok[r].cpu().numpy()
        off = 0
        for k in range(n):
            out.append(tok[off:off + int(ln[k])].astype(np.int32))
            off += int(ln[k])
    return out
