"""ctypes binding over librapid_pg.so: same names as the C ABI (include/rapid_pg.h), argument
marshalling only.  Tensors are PyTorch CUDA tensors used purely as device memory; every step of
the computation runs in the library's kernels on torch's current stream.

There is no fallback: if the shared library is missing the first call raises.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librapid_pg.so")

RAPID_OK = 0
RAPID_ERR_INVALID_ARG = 1
RAPID_ERR_ALIGNMENT = 2
RAPID_ERR_UNSUPPORTED = 3
RAPID_ERR_WORKSPACE = 4
RAPID_ERR_CUDA = 5
RAPID_ERR_TIMEOUT = 6

RAPID_F32 = 0
RAPID_BF16 = 1

FLAG_OUTER_UNCLIPPED = 1
FLAG_NORM_TOKENS = 2
FLAG_ADV_INPUT_IS_WEIGHT = 4
FLAG_LEAVE_ONE_OUT = 8
FLAG_LOO_LITERAL_DIVISOR = 16
FLAG_NORM_GIVEN = 32
FLAG_HEAD_STORE_LOGITS = 64
FLAG_HEAD_CTA_PAIRS = 128
FLAG_HEAD_SINGLE_CTA = 256
FLAG_HEAD_DW_BF16 = 512

# every symbol declared in include/rapid_pg.h
EXPORTS = (
    "rapid_status_string", "rapid_version", "rapid_workspace_bytes", "rapid_group_advantage",
    "rapid_pg_loss_fwd_bwd", "rapid_pg_stats_chunk", "rapid_pg_finalize", "rapid_pg_dlogits_chunk",
    "rapid_pg_loss_fwd_bwd_noalloc", "rapid_fused_head_workspace_bytes", "rapid_pg_loss_fused_head",
    "rapid_pg_loss_onpolicy_fwd_bwd", "rapid_pg_loss_fwd_bwd_hostlogits", "rapid_selftest_bounded_wait",
)


class RapidDesc(C.Structure):
    _fields_ = [("n_seq", C.c_int32), ("seq_len", C.c_int32), ("vocab", C.c_int32),
                ("n_groups", C.c_int32), ("ld", C.c_int64), ("dtype", C.c_int32),
                ("flags", C.c_uint32), ("eta", C.c_double), ("norm_z", C.c_double)]


class RapidStats(C.Structure):
    _fields_ = [("n_tokens", C.c_int64), ("n_clipped", C.c_int32), ("n_bad_token", C.c_int32),
                ("n_empty_group", C.c_int32), ("status", C.c_int32), ("mean_log_cw", C.c_double),
                ("mean_abs_log_cw", C.c_double), ("loss", C.c_double)]


STATS_BYTES = C.sizeof(RapidStats)


class RapidError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


_lib = None


def lib():
    """Load librapid_pg.so (once).  Raises if it has not been built: there is no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2510_03515_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i64, sz = C.c_void_p, C.c_int64, C.c_size_t
        dp = C.POINTER(RapidDesc)
        L.rapid_status_string.restype = C.c_char_p
        L.rapid_status_string.argtypes = [C.c_int]
        L.rapid_version.restype = C.c_int32
        L.rapid_workspace_bytes.restype = C.c_int
        L.rapid_workspace_bytes.argtypes = [dp, C.POINTER(C.c_size_t)]
        L.rapid_group_advantage.restype = C.c_int
        L.rapid_group_advantage.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp]
        L.rapid_pg_loss_fwd_bwd.restype = C.c_int
        L.rapid_pg_loss_fwd_bwd.argtypes = [dp] + [vp] * 12 + [sz, vp]
        L.rapid_pg_loss_fwd_bwd_noalloc.restype = C.c_int
        L.rapid_pg_loss_fwd_bwd_noalloc.argtypes = [dp] + [vp] * 12
        L.rapid_pg_loss_fwd_bwd_hostlogits.restype = C.c_int
        L.rapid_pg_loss_fwd_bwd_hostlogits.argtypes = [dp] + [vp] * 13 + [sz, vp]
        L.rapid_pg_loss_onpolicy_fwd_bwd.restype = C.c_int
        L.rapid_pg_loss_onpolicy_fwd_bwd.argtypes = [dp] + [vp] * 11 + [sz, vp]
        L.rapid_fused_head_workspace_bytes.restype = C.c_int
        L.rapid_fused_head_workspace_bytes.argtypes = [dp, C.c_int32, C.POINTER(C.c_size_t)]
        L.rapid_pg_loss_fused_head.restype = C.c_int
        L.rapid_pg_loss_fused_head.argtypes = [dp, C.c_int32] + [vp] * 14 + [sz, vp]
        L.rapid_selftest_bounded_wait.restype = C.c_int
        L.rapid_selftest_bounded_wait.argtypes = [C.c_uint64, vp, vp]
        L.rapid_pg_stats_chunk.restype = C.c_int
        L.rapid_pg_stats_chunk.argtypes = [dp, vp, i64, i64, vp, vp, vp, sz, vp]
        L.rapid_pg_finalize.restype = C.c_int
        L.rapid_pg_finalize.argtypes = [dp] + [vp] * 8 + [sz, vp]
        L.rapid_pg_dlogits_chunk.restype = C.c_int
        L.rapid_pg_dlogits_chunk.argtypes = [dp, vp, vp, i64, i64, vp, vp, vp, sz, vp]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().rapid_status_string(int(code)).decode()


def rapid_version() -> int:
    return int(lib().rapid_version())


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code: int, where: str) -> None:
    if code != RAPID_OK:
        raise RapidError(code, where)


def make_desc(n_seq: int, seq_len: int, vocab: int, n_groups: int, dtype: torch.dtype,
              ld: Optional[int] = None, eta: float = 2.0, flags: int = 0,
              norm_z: float = 0.0) -> RapidDesc:
    if dtype == torch.float32:
        dt = RAPID_F32
    elif dtype == torch.bfloat16:
        dt = RAPID_BF16
    else:
        raise TypeError("logits must be float32 or bfloat16")
    return RapidDesc(n_seq, seq_len, vocab, n_groups, vocab if ld is None else ld, dt, flags,
                     float(eta), float(norm_z))


def rapid_workspace_bytes(desc: RapidDesc) -> int:
    n = C.c_size_t(0)
    _check(lib().rapid_workspace_bytes(C.byref(desc), C.byref(n)), "rapid_workspace_bytes")
    return int(n.value)


def alloc_workspace(desc: RapidDesc, device="cuda") -> torch.Tensor:
    """Device memory for the scratch workspace (torch's allocator returns >= 256-byte alignment)."""
    return torch.empty(rapid_workspace_bytes(desc), dtype=torch.uint8, device=device)


def alloc_stats(device="cuda") -> torch.Tensor:
    return torch.zeros(STATS_BYTES, dtype=torch.uint8, device=device)


def read_stats(stats: torch.Tensor) -> dict:
    """Copy a device rapid_stats_t to the host (synchronises) and return it as a dict."""
    raw = bytes(stats.cpu().numpy().tobytes())
    s = RapidStats.from_buffer_copy(raw)
    return {k: getattr(s, k) for k, _ in RapidStats._fields_}


def rapid_group_advantage(desc: RapidDesc, rewards: torch.Tensor,
                          seq_log_ratio: Optional[torch.Tensor], group_offsets: torch.Tensor,
                          adv: torch.Tensor, clipped_w: Optional[torch.Tensor] = None,
                          stats: Optional[torch.Tensor] = None) -> None:
    _check(lib().rapid_group_advantage(C.byref(desc), _ptr(rewards), _ptr(seq_log_ratio),
                                       _ptr(group_offsets), _ptr(adv), _ptr(clipped_w),
                                       _ptr(stats), _stream()), "rapid_group_advantage")


def rapid_pg_loss_fwd_bwd(desc: RapidDesc, logits: torch.Tensor, targets: torch.Tensor,
                          mask: Optional[torch.Tensor], behav_logp: torch.Tensor,
                          rewards: torch.Tensor, group_offsets: torch.Tensor,
                          dlogits: torch.Tensor, loss: torch.Tensor,
                          token_logp: Optional[torch.Tensor], adv: Optional[torch.Tensor],
                          stats: Optional[torch.Tensor], workspace: torch.Tensor) -> None:
    _check(lib().rapid_pg_loss_fwd_bwd(
        C.byref(desc), _ptr(logits), _ptr(targets), _ptr(mask), _ptr(behav_logp), _ptr(rewards),
        _ptr(group_offsets), _ptr(dlogits), _ptr(loss), _ptr(token_logp), _ptr(adv), _ptr(stats),
        _ptr(workspace), workspace.numel(), _stream()), "rapid_pg_loss_fwd_bwd")


NOALLOC_SCRATCH_BYTES = 4 << 20


def rapid_pg_loss_fwd_bwd_noalloc(desc: RapidDesc, logits: torch.Tensor, targets: torch.Tensor,
                                  mask: Optional[torch.Tensor], behav_logp: torch.Tensor,
                                  rewards: torch.Tensor, group_offsets: torch.Tensor,
                                  dlogits: torch.Tensor, loss: torch.Tensor,
                                  token_logp: Optional[torch.Tensor], adv: Optional[torch.Tensor],
                                  stats: Optional[torch.Tensor]) -> None:
    """rapid_pg_loss_fwd_bwd for callers that cannot allocate a workspace: the scratch is a fixed
    array inside the library (at most NOALLOC_SCRATCH_BYTES; larger problems raise
    RAPID_ERR_UNSUPPORTED).  Calls on one device share that array, so do not let two overlap."""
    _check(lib().rapid_pg_loss_fwd_bwd_noalloc(
        C.byref(desc), _ptr(logits), _ptr(targets), _ptr(mask), _ptr(behav_logp), _ptr(rewards),
        _ptr(group_offsets), _ptr(dlogits), _ptr(loss), _ptr(token_logp), _ptr(adv), _ptr(stats),
        _stream()), "rapid_pg_loss_fwd_bwd_noalloc")


def rapid_pg_stats_chunk(desc: RapidDesc, logits_chunk: torch.Tensor, row0: int, n_rows: int,
                         targets: torch.Tensor, mask: Optional[torch.Tensor],
                         workspace: torch.Tensor) -> None:
    _check(lib().rapid_pg_stats_chunk(C.byref(desc), _ptr(logits_chunk), row0, n_rows,
                                      _ptr(targets), _ptr(mask), _ptr(workspace),
                                      workspace.numel(), _stream()), "rapid_pg_stats_chunk")


def rapid_pg_finalize(desc: RapidDesc, behav_logp: torch.Tensor, rewards: torch.Tensor,
                      group_offsets: torch.Tensor, loss: torch.Tensor,
                      token_logp: Optional[torch.Tensor], adv: Optional[torch.Tensor],
                      stats: Optional[torch.Tensor], workspace: torch.Tensor) -> None:
    _check(lib().rapid_pg_finalize(C.byref(desc), _ptr(behav_logp), _ptr(rewards),
                                   _ptr(group_offsets), _ptr(loss), _ptr(token_logp), _ptr(adv),
                                   _ptr(stats), _ptr(workspace), workspace.numel(), _stream()),
           "rapid_pg_finalize")


def rapid_pg_dlogits_chunk(desc: RapidDesc, logits_chunk: torch.Tensor,
                           dlogits_chunk: torch.Tensor, row0: int, n_rows: int,
                           targets: torch.Tensor, stats: Optional[torch.Tensor],
                           workspace: torch.Tensor) -> None:
    _check(lib().rapid_pg_dlogits_chunk(C.byref(desc), _ptr(logits_chunk), _ptr(dlogits_chunk),
                                        row0, n_rows, _ptr(targets), _ptr(stats), _ptr(workspace),
                                        workspace.numel(), _stream()), "rapid_pg_dlogits_chunk")


def rapid_pg_loss_fwd_bwd_hostlogits(desc: RapidDesc, logits_host: torch.Tensor, logits_staging: torch.Tensor,
                                     targets: torch.Tensor, mask: Optional[torch.Tensor],
                                     behav_logp: torch.Tensor, rewards: torch.Tensor,
                                     group_offsets: torch.Tensor, dlogits: torch.Tensor, loss: torch.Tensor,
                                     token_logp: Optional[torch.Tensor], adv: Optional[torch.Tensor],
                                     stats: Optional[torch.Tensor], workspace: torch.Tensor) -> None:
    """`logits_host` is a PINNED CPU tensor; everything else lives on the device."""
    _check(lib().rapid_pg_loss_fwd_bwd_hostlogits(
        C.byref(desc), _ptr(logits_host), _ptr(logits_staging), _ptr(targets), _ptr(mask), _ptr(behav_logp),
        _ptr(rewards), _ptr(group_offsets), _ptr(dlogits), _ptr(loss), _ptr(token_logp), _ptr(adv),
        _ptr(stats), _ptr(workspace), workspace.numel(), _stream()), "rapid_pg_loss_fwd_bwd_hostlogits")


def rapid_pg_loss_onpolicy_fwd_bwd(desc: RapidDesc, logits: torch.Tensor, targets: torch.Tensor,
                                   mask: Optional[torch.Tensor], rewards: torch.Tensor,
                                   group_offsets: torch.Tensor, dlogits: torch.Tensor, loss: torch.Tensor,
                                   token_logp: Optional[torch.Tensor], adv: Optional[torch.Tensor],
                                   stats: Optional[torch.Tensor], workspace: torch.Tensor) -> None:
    _check(lib().rapid_pg_loss_onpolicy_fwd_bwd(
        C.byref(desc), _ptr(logits), _ptr(targets), _ptr(mask), _ptr(rewards), _ptr(group_offsets),
        _ptr(dlogits), _ptr(loss), _ptr(token_logp), _ptr(adv), _ptr(stats), _ptr(workspace),
        workspace.numel(), _stream()), "rapid_pg_loss_onpolicy_fwd_bwd")


def rapid_selftest_bounded_wait(limit_ns: int, stats: torch.Tensor) -> None:
    _check(lib().rapid_selftest_bounded_wait(int(limit_ns), _ptr(stats), _stream()), "rapid_selftest_bounded_wait")


def rapid_fused_head_workspace_bytes(desc: RapidDesc, hidden_dim: int) -> int:
    n = C.c_size_t(0)
    _check(lib().rapid_fused_head_workspace_bytes(C.byref(desc), int(hidden_dim), C.byref(n)),
           "rapid_fused_head_workspace_bytes")
    return int(n.value)


def alloc_fused_head_workspace(desc: RapidDesc, hidden_dim: int, device="cuda") -> torch.Tensor:
    """Device scratch for rapid_pg_loss_fused_head, on a 1024-byte boundary."""
    n = rapid_fused_head_workspace_bytes(desc, hidden_dim)
    buf = torch.empty(n + 1024, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 1024
    return buf[off:off + n]


def rapid_pg_loss_fused_head(desc: RapidDesc, hidden: torch.Tensor, w_vocab: torch.Tensor,
                             targets: torch.Tensor, mask: Optional[torch.Tensor],
                             behav_logp: torch.Tensor, rewards: torch.Tensor,
                             group_offsets: torch.Tensor, loss: torch.Tensor, dhidden: torch.Tensor,
                             dW: torch.Tensor, token_logp: Optional[torch.Tensor],
                             adv: Optional[torch.Tensor], stats: Optional[torch.Tensor],
                             workspace: torch.Tensor) -> None:
    _check(lib().rapid_pg_loss_fused_head(
        C.byref(desc), int(hidden.shape[1]), _ptr(hidden), _ptr(w_vocab), _ptr(targets), _ptr(mask),
        _ptr(behav_logp), _ptr(rewards), _ptr(group_offsets), _ptr(loss), _ptr(dhidden), _ptr(dW),
        _ptr(token_logp), _ptr(adv), _ptr(stats), _ptr(workspace), workspace.numel(), _stream()),
        "rapid_pg_loss_fused_head")


@dataclass
class PgResult:
    loss: torch.Tensor        # [1] float32, device
    dlogits: torch.Tensor     # [T, ld]
    token_logp: torch.Tensor  # [T] float32
    adv: torch.Tensor         # [N] float32
    stats: torch.Tensor       # raw rapid_stats_t bytes, device


def pg_loss(logits: torch.Tensor, targets, mask, behav_logp, rewards, group_offsets, n_seq: int,
            seq_len: int, eta: float = 2.0, flags: int = 0, in_place: bool = False,
            workspace: Optional[torch.Tensor] = None, norm_z: float = 0.0) -> PgResult:
    """Convenience wrapper: allocate the outputs and make ONE rapid_pg_loss_fwd_bwd call."""
    T, ld = logits.shape[0], logits.stride(0)
    vocab = logits.shape[1]
    assert T == n_seq * seq_len
    desc = make_desc(n_seq, seq_len, vocab, group_offsets.numel() - 1, logits.dtype, ld, eta, flags, norm_z)
    dev = logits.device
    ws = workspace if workspace is not None else alloc_workspace(desc, dev)
    dlogits = logits if in_place else torch.empty_like(logits)
    loss = torch.empty(1, dtype=torch.float32, device=dev)
    token_logp = torch.empty(T, dtype=torch.float32, device=dev)
    adv = torch.empty(n_seq, dtype=torch.float32, device=dev)
    stats = alloc_stats(dev)
    rapid_pg_loss_fwd_bwd(desc, logits, targets, mask, behav_logp, rewards, group_offsets, dlogits,
                          loss, token_logp, adv, stats, ws)
    return PgResult(loss, dlogits, token_logp, adv, stats)
