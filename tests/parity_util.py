"""Shared helpers for the GPU parity tests: run the oracle and the CUDA library on the same
seeded inputs and compare element by element.  Tolerances are the ones the benchmark definition
states: loss relative error 1e-5 (fp32 logits) / 2e-3 (bf16), dlogits max abs error 1e-6 / 4e-3.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2510_03515_b200 import binding as rb
from paper_2510_03515_b200 import synth

LOSS_RTOL = {torch.float32: 1e-5, torch.bfloat16: 2e-3}
DLOGITS_ATOL = {torch.float32: 1e-6, torch.bfloat16: 4e-3}
# token log-probs are returned as float32: half an ulp at |x| in [16, 32) is 1e-6, which is what is
# observed (worst 9.6e-7 at full size); the kernels' own error is below 2e-7
LOGP_ATOL = {torch.float32: 2e-6, torch.bfloat16: 4e-6}
ADV_ATOL = {torch.float32: 2e-6, torch.bfloat16: 2e-5}
# the fused LM-head form takes its row statistics in float inside the GEMM epilogue, 256 columns at a
# time (observed at full size: token log-probs 7e-6, advantages 1.8e-5)
HEAD_LOGP_ATOL = 2e-5
HEAD_ADV_ATOL = 2e-4


def report_observed(case: str, **ratios) -> None:
    """Print the worst observed error of each compared quantity as a fraction of its bound (shown by
    `pytest -s` or `-rP`), and append the same record to the file named by RAPID_OBSERVED_LOG when
    that variable is set, so that the slack in every tolerance can be read off one run."""
    import json
    import os
    rec = {"case": case, **{k: float(f"{float(v):.3g}") for k, v in ratios.items()}}
    print("[observed error / bound]", json.dumps(rec))
    path = os.environ.get("RAPID_OBSERVED_LOG")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps(rec) + "\n")


def adv_atol(dtype, seq_len: int) -> float:
    """Advantages of the whole path depend on w_n = exp(sum of up to seq_len token log-probs).
    With float32 logits each row's log-sum-exp carries a few 1e-9 of error (float32 exponentials
    and differences, averaged over the vocabulary), with bf16 logits up to 2e-8 where the softmax
    is very peaked (2e-9 on the benchmark's logits); it adds up over the generation, and the
    advantage inherits it through mean(c R) with c <= eta = 2.  So the bound grows with L."""
    per_token = 4e-9 if dtype == torch.float32 else 5e-8
    return max(ADV_ATOL[dtype], per_token * seq_len)


def head_adv_atol(seq_len: int) -> float:
    """The same for the fused LM-head form (bf16 operands, float statistics per 256-column tile)."""
    return max(HEAD_ADV_ATOL, 4e-7 * seq_len)


def loss_scale(o) -> float:
    """The loss is a signed sum; its relative error is measured against
    max(|loss|, 1e-3 * sum_n |g_n S_n|).  When every token has probability one (a vocabulary of a
    single entry) both are exactly zero and a relative error has no meaning; the floor
    1e-9 * sum_n |g_n| len_n then turns the relative tolerance into an absolute one that
    corresponds to a log-probability error of rtol * 1e-9 per token."""
    floor = 1e-9 * float(np.abs(o["coef"] * o["seq_tokens"]).sum()) if "seq_tokens" in o else 0.0
    return max(abs(o["loss"]), 1e-3 * float(np.abs(o["coef"] * o["seq_logp"]).sum()), floor, 1e-30)


def behaviour_logp(batch, oracle_logp: np.ndarray) -> torch.Tensor:
    """log mu = current log-prob + the generator's noise, stored as float32 (as a sampler would)."""
    cur = torch.from_numpy(oracle_logp).to(torch.float64)
    return (cur + batch["behav_noise"].cpu().to(torch.float64)).to(torch.float32)


def bf16_round(x: np.ndarray) -> np.ndarray:
    return torch.from_numpy(np.ascontiguousarray(x, np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def run_both(batch, n_seq, seq_len, eta=2.0, flags=0, in_place=False, want_dlogits=True,
             ld_pad=0, device="cuda"):
    """Returns (oracle dict, gpu dict of numpy arrays).  `batch` holds CPU tensors."""
    logits = batch["logits"]
    T, V = logits.shape
    per = 16 // logits.element_size()
    if (V + ld_pad) % per:  # the row pitch must be a multiple of 16 bytes
        ld_pad += (-(V + ld_pad)) % per
    if ld_pad:
        padded = torch.full((T, V + ld_pad), 77.0, dtype=logits.dtype)
        padded[:, :V] = logits
        logits_host = padded
    else:
        logits_host = logits
    bits = synth.bits_numpy(logits_host)
    mask = batch.get("mask")
    pre = oracle.token_logp(bits, V, batch["targets"].numpy(), None if mask is None else mask.numpy())
    behav = batch.get("behav_logp")
    if behav is None:
        behav = behaviour_logp(batch, pre["token_logp"])
    o = oracle.pg_loss(bits, n_seq, seq_len, V, batch["targets"].numpy(),
                       None if mask is None else mask.numpy(), behav.numpy(),
                       batch["rewards"].numpy(), batch["group_offsets"].numpy(), eta, flags,
                       want_dlogits=want_dlogits)

    dev = torch.device(device)
    # guard rows before and after the logits / dlogits buffers
    G = 2
    ld = V + ld_pad
    zbuf = torch.full((T + 2 * G, ld), 55.0, dtype=logits.dtype, device=dev)
    zbuf[G:G + T].copy_(logits_host)
    z = zbuf[G:G + T]
    if in_place:
        dbuf, dz = zbuf, z
    else:
        dbuf = torch.full((T + 2 * G, ld), 33.0, dtype=logits.dtype, device=dev)
        dz = dbuf[G:G + T]
    desc = rb.make_desc(n_seq, seq_len, V, batch["group_offsets"].numel() - 1, logits.dtype, ld, eta, flags)
    ws = rb.alloc_workspace(desc, dev)
    loss = torch.full((1,), float("nan"), device=dev)
    tl = torch.full((T,), float("nan"), device=dev)
    adv = torch.full((n_seq,), float("nan"), device=dev)
    stats = rb.alloc_stats(dev)
    rb.rapid_pg_loss_fwd_bwd(desc, z, batch["targets"].to(dev), None if mask is None else mask.to(dev),
                             behav.to(dev), batch["rewards"].to(dev), batch["group_offsets"].to(dev),
                             dz, loss, tl, adv, stats, ws)
    torch.cuda.synchronize()
    g = {
        "loss": float(loss.item()), "token_logp": tl.cpu().numpy(), "adv": adv.cpu().numpy(),
        "stats": rb.read_stats(stats), "dlogits": dz[:, :V].float().cpu().numpy(),
    }
    # canaries: guard rows and pad columns untouched
    guard_val = 55.0 if in_place else 33.0
    assert torch.all(dbuf[:G] == guard_val) and torch.all(dbuf[G + T:] == guard_val), "guard rows overwritten"
    if ld_pad:
        pad_val = 77.0 if in_place else 33.0
        assert torch.all(dz[:, V:] == pad_val), "columns >= vocab overwritten"
    if not in_place:
        assert torch.equal(z.cpu(), logits_host), "logits modified"
    return o, g


def compare(o, g, dtype, seq_len, check_dlogits=True):
    """Element-by-element comparison at the stated tolerances; returns the worst errors."""
    ok = o["row_ok"].astype(bool)
    np.testing.assert_allclose(g["token_logp"], o["token_logp"], rtol=0, atol=LOGP_ATOL[dtype])
    assert np.all(g["token_logp"][~ok] == 0.0)
    np.testing.assert_allclose(g["adv"], o["adv64"], rtol=0, atol=adv_atol(dtype, seq_len))
    rel = abs(g["loss"] - o["loss"]) / loss_scale(o)
    out = {"loss_rel": rel, "loss_vs_bound": rel / LOSS_RTOL[dtype],
           "logp_vs_bound": float(np.abs(g["token_logp"] - o["token_logp"]).max()) / LOGP_ATOL[dtype],
           "adv_vs_bound": float(np.abs(g["adv"] - o["adv64"]).max()) / adv_atol(dtype, seq_len)}
    # the float32 loss output itself carries half an ulp
    assert rel <= LOSS_RTOL[dtype] + 6e-8 * abs(o["loss"]) / loss_scale(o), f"loss rel err {rel}"
    st = g["stats"]
    assert st["status"] == 0
    assert st["n_tokens"] == o["n_tokens"]
    assert st["n_bad_token"] == o["n_bad_token"]
    near_tie = np.abs(o["weight"] - 2.0) < 1e-3
    if not near_tie.any():
        assert st["n_clipped"] == o["n_clipped"]
    assert st["mean_log_cw"] == np.float64(st["mean_log_cw"])
    tol_s = 1e-4 if dtype == torch.float32 else 1e-2
    assert abs(st["mean_log_cw"] - o["mean_log_cw"]) <= tol_s
    assert abs(st["mean_abs_log_cw"] - o["mean_abs_log_cw"]) <= tol_s
    relst = abs(st["loss"] - o["loss"]) / loss_scale(o)
    assert relst <= LOSS_RTOL[dtype]
    if check_dlogits and o.get("dlogits") is not None:
        d = g["dlogits"].astype(np.float64)
        ref = o["dlogits"]
        err = np.abs(d - ref).max()
        assert err <= DLOGITS_ATOL[dtype], f"dlogits max abs err {err}"
        # rows that must be exactly zero: masked rows and generations with zero coefficient
        zero_rows = (~ok) | (np.repeat(o["coef"], seq_len) == 0.0)
        assert np.all(d[zero_rows] == 0.0)
        out["dlogits_abs"] = err
        out["dlogits_vs_bound"] = err / DLOGITS_ATOL[dtype]
    return out
