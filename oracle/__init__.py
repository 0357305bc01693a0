"""ctypes wrapper around the float64 CPU oracle (oracle/rapid_oracle.c).

TEST INFRASTRUCTURE.  Only the test-suite, the smoke check and the benchmark's CPU-baseline leg
may import this package.  It shares no code with the CUDA library; arrays go in and out as numpy.

Logits are handed over exactly as the GPU sees them: float32 arrays, or bf16 bit patterns held
in a uint16 array.  Everything the oracle computes is float64.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional

import numpy as np

from . import build as _build

F32 = 0
BF16 = 1

FLAG_OUTER_UNCLIPPED = 1
FLAG_NORM_TOKENS = 2
FLAG_ADV_INPUT_IS_WEIGHT = 4
FLAG_LEAVE_ONE_OUT = 8
FLAG_LOO_LITERAL_DIVISOR = 16

_lib = None


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.rapid_oracle_token_logp.restype = C.c_int64
        L.rapid_oracle_token_logp.argtypes = [
            C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_void_p, C.c_void_p]
        L.rapid_oracle_seq_reduce.restype = None
        L.rapid_oracle_seq_reduce.argtypes = [C.c_int32, C.c_int32] + [C.c_void_p] * 6
        L.rapid_oracle_group_advantage.restype = C.c_int
        L.rapid_oracle_group_advantage.argtypes = [
            C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_double, C.c_uint32,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.rapid_oracle_coef_loss.restype = C.c_double
        L.rapid_oracle_coef_loss.argtypes = [C.c_int32] + [C.c_void_p] * 6 + [
            C.c_double, C.c_uint32, C.c_void_p, C.c_void_p]
        L.rapid_oracle_dlogits_rows.restype = None
        L.rapid_oracle_dlogits_rows.argtypes = [
            C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_void_p,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        L.rapid_oracle_pg_loss.restype = C.c_int
        L.rapid_oracle_pg_loss.argtypes = [
            C.c_void_p, C.c_int, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_double, C.c_uint32,
        ] + [C.c_void_p] * 15
        L.rapid_oracle_head_logits.restype = None
        L.rapid_oracle_head_logits.argtypes = [
            C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p]
        L.rapid_oracle_token_logp_f64.restype = None
        L.rapid_oracle_token_logp_f64.argtypes = [
            C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.rapid_oracle_dlogits_f64.restype = None
        L.rapid_oracle_dlogits_f64.argtypes = [
            C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.rapid_oracle_head_dhidden.restype = None
        L.rapid_oracle_head_dhidden.argtypes = [
            C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int64, C.c_void_p]
        L.rapid_oracle_head_dweight_accum.restype = None
        L.rapid_oracle_head_dweight_accum.argtypes = [
            C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p]
        L.rapid_oracle_set_threads.argtypes = [C.c_int]
        L.rapid_oracle_max_threads.restype = C.c_int
        _lib = L
    return _lib


def set_threads(n: int) -> None:
    lib().rapid_oracle_set_threads(int(n))


def max_threads() -> int:
    return int(lib().rapid_oracle_max_threads())


def _dtype_code(logits: np.ndarray) -> int:
    if logits.dtype == np.float32:
        return F32
    if logits.dtype == np.uint16:
        return BF16
    raise TypeError("logits must be float32, or bf16 bit patterns as uint16")


def _c(a, dt):
    return None if a is None else np.ascontiguousarray(a, dtype=dt)


def token_logp(logits: np.ndarray, vocab: int, targets, mask=None):
    """Step 1 for every row of `logits` ([n_rows, ld]).  Returns a dict of float64/uint8 arrays."""
    logits = np.ascontiguousarray(logits)
    n_rows, ld = logits.shape
    targets = _c(targets, np.int32)
    mask = _c(mask, np.uint8)
    lse = np.zeros(n_rows)
    lp = np.zeros(n_rows)
    ok = np.zeros(n_rows, np.uint8)
    bad = lib().rapid_oracle_token_logp(_p(logits), _dtype_code(logits), ld, n_rows, vocab,
                                        _p(targets), _p(mask), _p(lse), _p(lp), _p(ok))
    return {"lse": lse, "token_logp": lp, "row_ok": ok, "n_bad_token": int(bad)}


def seq_reduce(n_seq: int, seq_len: int, token_logp_, behav_logp, row_ok):
    """Step 2.  Returns (s_n, S_n, token counts)."""
    tl = _c(token_logp_, np.float64)
    bl = _c(behav_logp, np.float32)
    ok = _c(row_ok, np.uint8)
    s = np.zeros(n_seq)
    S = np.zeros(n_seq)
    cnt = np.zeros(n_seq, np.int32)
    lib().rapid_oracle_seq_reduce(n_seq, seq_len, _p(tl), _p(bl), _p(ok), _p(s), _p(S), _p(cnt))
    return s, S, cnt


def group_advantage(rewards, seq_log_ratio, group_offsets, eta: float = 2.0, flags: int = 0):
    """Steps 3-4.  seq_log_ratio None => on-policy (Eq. 2).  Returns a dict."""
    rewards = _c(rewards, np.float32)
    slr = _c(seq_log_ratio, np.float64)
    go = _c(group_offsets, np.int32)
    n = rewards.shape[0]
    k = go.shape[0] - 1
    w = np.zeros(n)
    c = np.zeros(n)
    a64 = np.zeros(n)
    a32 = np.zeros(n, np.float32)
    rc = lib().rapid_oracle_group_advantage(n, k, _p(rewards), _p(slr), _p(go), float(eta),
                                            int(flags), _p(w), _p(c), _p(a64), _p(a32))
    if rc:
        raise ValueError("group_offsets is not a monotone cover of [0, n_seq)")
    return {"weight": w, "clipped_w": c, "adv64": a64, "adv32": a32}


def dlogits_rows(logits: np.ndarray, vocab: int, seq_len: int, targets, row_ok, lse, coef, rows,
                 row_base: int = 0) -> np.ndarray:
    """Step 6 for the listed global rows; `logits` starts at global row `row_base`."""
    logits = np.ascontiguousarray(logits)
    ld = logits.shape[1]
    rows = _c(rows, np.int64)
    out = np.zeros((rows.shape[0], vocab))
    lib().rapid_oracle_dlogits_rows(_p(logits), _dtype_code(logits), ld, int(row_base), vocab,
                                    seq_len, _p(_c(targets, np.int32)), _p(_c(row_ok, np.uint8)),
                                    _p(_c(lse, np.float64)), _p(_c(coef, np.float64)), _p(rows),
                                    rows.shape[0], _p(out))
    return out


def coef_loss(seq_log_ratio, seq_logp, seq_tokens, weight, clipped_w, adv64, eta=2.0, flags=0):
    """Step 5.  Returns (loss, coef, stats dict)."""
    n = len(seq_logp)
    coef = np.zeros(n)
    st = np.zeros(4)
    loss = lib().rapid_oracle_coef_loss(
        n, _p(_c(seq_log_ratio, np.float64)), _p(_c(seq_logp, np.float64)),
        _p(_c(seq_tokens, np.int32)), _p(_c(weight, np.float64)), _p(_c(clipped_w, np.float64)),
        _p(_c(adv64, np.float64)), float(eta), int(flags), _p(coef), _p(st))
    stats = {"n_clipped": int(st[0]), "mean_log_cw": st[1], "mean_abs_log_cw": st[2],
             "n_tokens": int(st[3])}
    return float(loss), coef, stats


def pg_loss(logits: np.ndarray, n_seq: int, seq_len: int, vocab: int, targets, mask, behav_logp,
            rewards, group_offsets, eta: float = 2.0, flags: int = 0, want_dlogits: bool = False):
    """Steps 1-6 over one mini-batch.  Returns a dict with every intermediate."""
    logits = np.ascontiguousarray(logits)
    T = n_seq * seq_len
    assert logits.shape[0] == T
    ld = logits.shape[1]
    targets = _c(targets, np.int32)
    mask = _c(mask, np.uint8)
    behav_logp = _c(behav_logp, np.float32)
    rewards = _c(rewards, np.float32)
    go = _c(group_offsets, np.int32)
    K = go.shape[0] - 1
    o = {
        "loss": np.zeros(1), "lse": np.zeros(T), "token_logp": np.zeros(T),
        "row_ok": np.zeros(T, np.uint8), "seq_log_ratio": np.zeros(n_seq),
        "seq_logp": np.zeros(n_seq), "seq_tokens": np.zeros(n_seq, np.int32),
        "weight": np.zeros(n_seq), "clipped_w": np.zeros(n_seq), "adv64": np.zeros(n_seq),
        "adv32": np.zeros(n_seq, np.float32), "coef": np.zeros(n_seq), "stats": np.zeros(4),
        "n_bad_token": np.zeros(1, np.int64),
        "dlogits": np.zeros((T, vocab)) if want_dlogits else None,
    }
    rc = lib().rapid_oracle_pg_loss(
        _p(logits), _dtype_code(logits), ld, n_seq, seq_len, vocab, K, _p(targets), _p(mask),
        _p(behav_logp), _p(rewards), _p(go), float(eta), int(flags),
        _p(o["loss"]), _p(o["lse"]), _p(o["token_logp"]), _p(o["row_ok"]),
        _p(o["seq_log_ratio"]), _p(o["seq_logp"]), _p(o["seq_tokens"]), _p(o["weight"]),
        _p(o["clipped_w"]), _p(o["adv64"]), _p(o["adv32"]), _p(o["coef"]), _p(o["stats"]),
        _p(o["n_bad_token"]), _p(o["dlogits"]))
    if rc:
        raise ValueError("group_offsets is not a monotone cover of [0, n_seq)")
    st = o.pop("stats")
    o["loss"] = float(o["loss"][0])
    o["n_bad_token"] = int(o["n_bad_token"][0])
    o["n_clipped"] = int(st[0])
    o["mean_log_cw"] = float(st[1])
    o["mean_abs_log_cw"] = float(st[2])
    o["n_tokens"] = int(st[3])
    return o


# ---- fused-head form -----------------------------------------------------------------------------

def head_logits(hidden_bits: np.ndarray, w_bits: np.ndarray, rows=None) -> np.ndarray:
    """z[rows] = h[rows] @ W in float64 from bf16 bit patterns (uint16 arrays)."""
    hidden_bits = _c(hidden_bits, np.uint16)
    w_bits = _c(w_bits, np.uint16)
    D, V = w_bits.shape
    if rows is None:
        rows = np.arange(hidden_bits.shape[0], dtype=np.int64)
    rows = _c(rows, np.int64)
    out = np.zeros((rows.shape[0], V))
    lib().rapid_oracle_head_logits(_p(hidden_bits), _p(w_bits), D, V, _p(rows), rows.shape[0],
                                   _p(out))
    return out


def decode_bf16(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> the float64 values they stand for (exact)."""
    bits = _c(bits, np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def head_logits_dgemm(hidden_bits: np.ndarray, w_f64: np.ndarray, rows=None) -> np.ndarray:
    """z[rows] = h[rows] @ W in float64 with the library's matrix product as the step.

    Same definition as head_logits (the fused-head form's z = h W); the sum over the hidden
    dimension is taken by float64 GEMM instead of the plain loops, which is what makes all
    16 384 rows of the full-size configuration affordable (3.8e12 multiply-adds).  `w_f64` is
    decode_bf16(w_bits), decoded once by the caller.  The two differ only in summation order."""
    h = decode_bf16(hidden_bits if rows is None else _c(hidden_bits, np.uint16)[_c(rows, np.int64)])
    return h @ w_f64


def token_logp_f64(z: np.ndarray, targets_of_list):
    z = _c(z, np.float64)
    n, V = z.shape
    t = _c(targets_of_list, np.int32)
    lse = np.zeros(n)
    lp = np.zeros(n)
    lib().rapid_oracle_token_logp_f64(_p(z), n, V, _p(t), _p(lse), _p(lp))
    return lse, lp


def dlogits_f64_inplace(z: np.ndarray, targets_of_list, lse, coef_of_list) -> np.ndarray:
    assert z.dtype == np.float64 and z.flags.c_contiguous
    n, V = z.shape
    lib().rapid_oracle_dlogits_f64(_p(z), n, V, _p(_c(targets_of_list, np.int32)),
                                   _p(_c(lse, np.float64)), _p(_c(coef_of_list, np.float64)))
    return z


def head_dhidden(dz: np.ndarray, w_bits: np.ndarray) -> np.ndarray:
    dz = _c(dz, np.float64)
    w_bits = _c(w_bits, np.uint16)
    D, V = w_bits.shape
    out = np.zeros((dz.shape[0], D))
    lib().rapid_oracle_head_dhidden(_p(dz), _p(w_bits), D, V, dz.shape[0], _p(out))
    return out


def head_dweight_accum(dW: np.ndarray, dz: np.ndarray, hidden_bits: np.ndarray, rows=None) -> None:
    assert dW.dtype == np.float64 and dW.flags.c_contiguous
    dz = _c(dz, np.float64)
    hidden_bits = _c(hidden_bits, np.uint16)
    D, V = dW.shape
    rows_ = None if rows is None else _c(rows, np.int64)
    lib().rapid_oracle_head_dweight_accum(_p(dz), _p(hidden_bits), D, V, _p(rows_), dz.shape[0],
                                          _p(dW))
