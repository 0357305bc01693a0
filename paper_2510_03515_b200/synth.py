"""Seeded synthetic mini-batches shaped like the paper's SLM rollouts.

The paper trains on MBPP+/MATH/MiniF2F rollouts of Qwen2.5 / Llama-3.2 / Gemma-3 models (Sec. 4.1);
neither the datasets nor the weights are available here, so these generators stand in for them.
Shapes echo the paper's hyper-parameter table (several generations per prompt, completions of up
to a few thousand tokens, mini-batches of 4-32 generations, bf16).

This module only draws random numbers and arranges them.  It contains none of the method's
arithmetic: in particular the behaviour policy's log-probabilities are returned as a NOISE term
that the caller adds to whatever "current" log-probabilities it obtained elsewhere.  Both the
test oracle and the CUDA path are fed from here; neither is imported here.

"N(0, x)" always means standard deviation x.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, Optional

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n_prompts: int          # K, number of groups
    group_size: int         # N_k, generations per prompt
    seq_len: int            # L, padded response length
    vocab: int              # V
    dtype: str              # "f32" or "bf16"
    logit_std: float
    boost: float            # added to the sampled token's logit (peaked softmax)
    length_mode: str        # "full" | "uniform" | "trailing"
    len_lo: int = 0         # "uniform": lengths drawn from {len_lo..seq_len}
    trailing_frac: float = 0.0  # "trailing": this share of every row of the grid is padding
    behav_sigma: float = 0.1
    reward_mode: str = "half"   # "half" | "per_prompt" | "per_prompt_const" | "const_first_two" | "p03"
    seed: int = 0
    hidden: int = 0         # fused-head form only: D

    @property
    def n_seq(self) -> int:
        return self.n_prompts * self.group_size

    @property
    def n_rows(self) -> int:
        return self.n_seq * self.seq_len

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five configurations of the benchmark definition, full size.
CONFIGS: Dict[str, Workload] = {
    "tiny": Workload("tiny", 4, 8, 64, 4096, "f32", 2.0, 0.0, "full",
                     behav_sigma=0.1, reward_mode="half", seed=0),
    "slm": Workload("slm", 8, 8, 1024, 151936, "bf16", 3.0, 8.0, "uniform", len_lo=256,
                    behav_sigma=0.2, reward_mode="per_prompt", seed=1),
    "stale": Workload("stale", 16, 8, 512, 151936, "bf16", 3.0, 8.0, "full",
                      behav_sigma=0.5, reward_mode="per_prompt_const", seed=2),
    "long": Workload("long", 4, 16, 4096, 32000, "f32", 2.0, 0.0, "trailing", trailing_frac=0.3,
                     behav_sigma=0.1, reward_mode="const_first_two", seed=3),
    "fused": Workload("fused", 8, 8, 256, 151936, "bf16", 0.0, 0.0, "full",
                      behav_sigma=0.2, reward_mode="p03", seed=4, hidden=1536),
}
STALE_SIGMAS = (0.0, 0.1, 0.5, 1.0, 2.0)


def _gen(seed: int, stream: int, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 1_000_003 + int(stream))
    return g


def torch_dtype(w: Workload) -> torch.dtype:
    return torch.float32 if w.dtype == "f32" else torch.bfloat16


def make_tokens(w: Workload) -> Dict[str, torch.Tensor]:
    """Everything except the logits, on the CPU (small): targets, mask, rewards, groups, noise."""
    N, L, V, K = w.n_seq, w.seq_len, w.vocab, w.n_prompts
    g = _gen(w.seed, 1)
    targets = torch.randint(0, V, (N, L), generator=g, dtype=torch.int64).to(torch.int32)

    if w.length_mode == "full":
        lengths = torch.full((N,), L, dtype=torch.int64)
    elif w.length_mode == "uniform":
        lengths = torch.randint(w.len_lo, L + 1, (N,), generator=g)
    elif w.length_mode == "trailing":
        lengths = torch.full((N,), L - int(round(w.trailing_frac * L)), dtype=torch.int64)
    else:
        raise ValueError(w.length_mode)
    mask = (torch.arange(L)[None, :] < lengths[:, None]).to(torch.uint8)

    u = torch.rand((K, w.group_size), generator=g)
    if w.reward_mode == "half":
        p = torch.full((K, 1), 0.5)
    elif w.reward_mode == "p03":
        p = torch.full((K, 1), 0.3)
    elif w.reward_mode in ("per_prompt", "per_prompt_const"):
        p = torch.rand((K, 1), generator=g)
    elif w.reward_mode == "const_first_two":
        p = torch.full((K, 1), 0.5)
    else:
        raise ValueError(w.reward_mode)
    rewards = (u < p).to(torch.float32)
    if w.reward_mode in ("per_prompt_const", "const_first_two") and K >= 2:
        rewards[0, :] = 0.0   # a group whose rewards are all zero
        rewards[1, :] = 1.0   # a group whose rewards are all one
    rewards = rewards.reshape(N)

    group_offsets = (torch.arange(K + 1) * w.group_size).to(torch.int32)
    noise = torch.randn((N, L), generator=g) * w.behav_sigma
    return {
        "targets": targets.reshape(N * L).contiguous(),
        "mask": mask.reshape(N * L).contiguous(),
        "lengths": lengths,
        "rewards": rewards.contiguous(),
        "group_offsets": group_offsets.contiguous(),
        "behav_noise": noise.reshape(N * L).to(torch.float32).contiguous(),
    }


def logits_for_sequences(w: Workload, targets: torch.Tensor, seq0: int, n_seqs: int,
                         device="cpu", out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Logits rows of generations [seq0, seq0 + n_seqs), shape [n_seqs * L, V], in w's dtype.

    Each generation has its own random stream, so any range can be regenerated on its own.
    Drawn in float32 on `device`, the sampled token's logit boosted, then rounded to the dtype.
    """
    L, V = w.seq_len, w.vocab
    dt = torch_dtype(w)
    if out is None:
        out = torch.empty((n_seqs * L, V), dtype=dt, device=device)
    tg = targets.reshape(-1, L)
    for i in range(n_seqs):
        n = seq0 + i
        g = _gen(w.seed, 1000 + n, device=device)
        z = torch.randn((L, V), generator=g, device=device, dtype=torch.float32) * w.logit_std
        if w.boost != 0.0:
            idx = tg[n].to(device=device, dtype=torch.int64).unsqueeze(1)
            z.scatter_add_(1, idx, torch.full((L, 1), w.boost, device=device))
        out[i * L:(i + 1) * L].copy_(z)
    return out


def make_batch(w: Workload, device="cpu") -> Dict[str, torch.Tensor]:
    """A whole mini-batch with dense logits [N*L, V] on `device` (small per-token arrays too)."""
    b = make_tokens(w)
    b["logits"] = logits_for_sequences(w, b["targets"], 0, w.n_seq, device=device)
    for k in ("targets", "mask", "rewards", "group_offsets", "behav_noise"):
        b[k] = b[k].to(device)
    return b


def make_head(w: Workload, device="cpu") -> Dict[str, torch.Tensor]:
    """Fused-head form: hidden states [N*L, D] ~ N(0, 1) and the LM-head weight [D, V] ~ N(0, 0.02)."""
    assert w.hidden > 0
    b = make_tokens(w)
    g = _gen(w.seed, 2, device=device)
    h = torch.randn((w.n_rows, w.hidden), generator=g, device=device, dtype=torch.float32)
    W = torch.randn((w.hidden, w.vocab), generator=g, device=device, dtype=torch.float32) * 0.02
    b["hidden"] = h.to(torch.bfloat16)
    b["w_vocab"] = W.to(torch.bfloat16)
    for k in ("targets", "mask", "rewards", "group_offsets", "behav_noise"):
        b[k] = b[k].to(device)
    return b


def bits_numpy(t: torch.Tensor):
    """CPU numpy view of a tensor as the GPU stores it: float32 as is, bf16 as uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view("uint16")
    return t.numpy()
