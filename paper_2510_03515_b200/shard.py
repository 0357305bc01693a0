"""Spreading ONE mini-batch over several GPUs (host logic only; no arithmetic of the method).

The path couples generations only inside a prompt group (Eq. 5), so a mini-batch is split by
WHOLE groups and no rank ever needs another rank's logits.  What crosses ranks is:

  * before the call: the global normaliser Z of Eq. 3 -- the global number of generations (known
    without communication) or, with token normalisation, the global token count (one scalar
    all-reduce of the ranks' mask sums) -- which every rank passes as desc.norm_z with
    RAPID_FLAG_NORM_GIVEN, so that per-rank losses and gradients add up to the whole batch's;
  * after the call: the scalar loss and the side statistics, reduced here in one all-reduce of
    eight doubles (plus one MAX all-reduce of the status word).

dlogits (or dhidden) stay on the rank that owns the rows.  For the fused LM-head form dW is a
plain sum over ranks: the ordinary data-parallel gradient all-reduce, which the caller's training
framework already does.

Works with any torch.distributed backend: tensors are created on `device` ("cpu" for gloo).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch


def partition_groups(tokens_per_group: Sequence[int], world: int) -> List[List[int]]:
    """Assign whole groups to ranks, balancing the unmasked-token count (largest group first, to the
    least loaded rank; ties by lower index).  Deterministic, so every rank computes the same plan."""
    if world <= 0:
        raise ValueError("world must be positive")
    loads = [0] * world
    out: List[List[int]] = [[] for _ in range(world)]
    order = sorted(range(len(tokens_per_group)), key=lambda k: (-int(tokens_per_group[k]), k))
    for k in order:
        r = min(range(world), key=lambda i: (loads[i], i))
        out[r].append(k)
        loads[r] += int(tokens_per_group[k])
    return [sorted(g) for g in out]


@dataclass
class LocalShard:
    groups: List[int]              # global group indices owned by this rank, ascending
    seq_index: np.ndarray          # global generation index of each local generation
    group_offsets: np.ndarray      # local [K_local + 1] int32 offsets (contiguous groups)
    n_seq_global: int

    @property
    def n_seq(self) -> int:
        return int(self.seq_index.shape[0])


def plan(group_offsets: Sequence[int], tokens_per_seq: Sequence[int], world: int, rank: int) -> LocalShard:
    """This rank's part of a mini-batch given the global group offsets and per-generation token counts."""
    go = np.asarray(group_offsets, dtype=np.int64)
    tps = np.asarray(tokens_per_seq, dtype=np.int64)
    K = go.shape[0] - 1
    per_group = [int(tps[go[k]:go[k + 1]].sum()) for k in range(K)]
    mine = partition_groups(per_group, world)[rank]
    seqs, offs = [], [0]
    for k in mine:
        seqs.extend(range(int(go[k]), int(go[k + 1])))
        offs.append(len(seqs))
    return LocalShard(mine, np.asarray(seqs, dtype=np.int64), np.asarray(offs, dtype=np.int32), int(go[-1]))


def global_token_count(local_tokens: int, device="cpu", group=None) -> int:
    """Z for token normalisation: the sum of the ranks' unmasked-token counts."""
    import torch.distributed as dist
    t = torch.tensor([float(local_tokens)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return int(round(t.item()))


def reduce_stats(local: Dict[str, float], n_seq_local: int, n_seq_global: int, device="cpu",
                 group=None) -> Dict[str, float]:
    """Combine per-rank results of calls made with RAPID_FLAG_NORM_GIVEN into the mini-batch's.

    `local` holds this rank's loss, n_tokens, n_clipped, n_bad_token, n_empty_group, mean_log_cw,
    mean_abs_log_cw and status (e.g. from binding.read_stats).  Means are re-weighted by the
    number of generations each rank holds; counts and the loss add; the status is the worst one.
    """
    import torch.distributed as dist
    v = torch.tensor([
        float(local["loss"]), float(local["n_tokens"]), float(local["n_clipped"]),
        float(local["n_bad_token"]), float(local["n_empty_group"]),
        float(local["mean_log_cw"]) * n_seq_local, float(local["mean_abs_log_cw"]) * n_seq_local,
        float(n_seq_local)], dtype=torch.float64, device=device)
    s = torch.tensor([float(local.get("status", 0))], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(v, op=dist.ReduceOp.SUM, group=group)
        dist.all_reduce(s, op=dist.ReduceOp.MAX, group=group)
    v = v.cpu().tolist()
    if int(round(v[7])) != n_seq_global:
        raise RuntimeError(f"shards cover {int(round(v[7]))} generations, the mini-batch has {n_seq_global}")
    return {"loss": v[0], "n_tokens": int(round(v[1])), "n_clipped": int(round(v[2])),
            "n_bad_token": int(round(v[3])), "n_empty_group": int(round(v[4])),
            "mean_log_cw": v[5] / n_seq_global, "mean_abs_log_cw": v[6] / n_seq_global,
            "status": int(round(s.item()))}
