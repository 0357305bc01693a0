"""GPU parity of the fused LM-head form against the float64 oracle: z = h W in float64 from the
same bf16 bits, steps 1-6 on z, then dh = dz W^T and dW = h^T dz.

Tolerances.  Loss and token log-probabilities: the bf16-logits class (2e-3 relative, 2e-5).
dh and dW: the library rounds dlogits to bf16 before the two products, an independent relative
error of at most 2^-9 per element, so an output element sum_k a_k dz_k carries a random error of
standard deviation about 2^-9 sqrt(sum_k a_k^2 dz_k^2) / sqrt(3); the test allows 2^-6 times that
root-sum-square (many standard deviations), plus 2^-8 |ref| for dh's own rounding to bf16.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2510_03515_b200 import binding as rb  # noqa: E402
from paper_2510_03515_b200 import synth  # noqa: E402
from parity_util import LOGP_ATOL, LOSS_RTOL, adv_atol  # noqa: E402


def bf16_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def oracle_head(b, w, eta=2.0, flags=0):
    """Everything the oracle computes for one fused-head batch (small sizes: dense float64)."""
    T, V, L = w.n_rows, w.vocab, w.seq_len
    h_bits, w_bits = synth.bits_numpy(b["hidden"]), synth.bits_numpy(b["w_vocab"])
    tg, mk = b["targets"].numpy(), b["mask"].numpy()
    z = oracle.head_logits(h_bits, w_bits)
    ok = (mk != 0) & (tg >= 0) & (tg < V)
    lse, lp = oracle.token_logp_f64(z, np.where(ok, tg, 0))
    lp = np.where(ok, lp, 0.0)
    behav = b.get("behav_logp")
    if behav is None:
        behav = (torch.from_numpy(lp) + b["behav_noise"].double()).float()
    s, S, cnt = oracle.seq_reduce(w.n_seq, L, lp, behav.numpy(), ok.astype(np.uint8))
    ga = oracle.group_advantage(b["rewards"].numpy(), s, b["group_offsets"].numpy(), eta, flags)
    loss, coef, st = oracle.coef_loss(s, S, cnt, ga["weight"], ga["clipped_w"], ga["adv64"], eta, flags)
    g_row = np.repeat(coef, L) * ok
    dz = oracle.dlogits_f64_inplace(z.copy(), np.where(ok, tg, 0), lse, g_row)
    dh = oracle.head_dhidden(dz, w_bits)
    dW = np.zeros((w.hidden, V))
    oracle.head_dweight_accum(dW, dz, h_bits)
    return {"loss": loss, "coef": coef, "seq_logp": S, "token_logp": lp, "adv64": ga["adv64"], "stats": st,
            "dz": dz, "dh": dh, "dW": dW, "behav": behav, "ok": ok,
            "h": bf16_to_f64(h_bits), "W": bf16_to_f64(w_bits)}


def run_head(b, w, behav, ld_pad=0, eta=2.0, flags=0):
    dev = torch.device("cuda")
    T, V, D = w.n_rows, w.vocab, w.hidden
    ld = V + ld_pad
    Wd = torch.full((D, ld), 9.0, dtype=torch.bfloat16, device=dev)
    Wd[:, :V] = b["w_vocab"].to(dev)
    desc = rb.make_desc(w.n_seq, w.seq_len, V, w.n_prompts, torch.bfloat16, ld, eta, flags)
    ws = rb.alloc_fused_head_workspace(desc, D, dev)
    loss = torch.full((1,), float("nan"), device=dev)
    dh = torch.full((T + 2, D), 7.0, dtype=torch.bfloat16, device=dev)   # one guard row on each side
    dW = torch.full((D + 2, ld), 5.0, dtype=torch.float32, device=dev)
    tl = torch.full((T,), float("nan"), device=dev)
    adv = torch.full((w.n_seq,), float("nan"), device=dev)
    stats = rb.alloc_stats(dev)
    rb.rapid_pg_loss_fused_head(desc, b["hidden"].to(dev), Wd, b["targets"].to(dev), b["mask"].to(dev),
                                behav.to(dev), b["rewards"].to(dev), b["group_offsets"].to(dev), loss,
                                dh[1:T + 1], dW[1:D + 1], tl, adv, stats, ws)
    torch.cuda.synchronize()
    assert torch.all(dh[0] == 7.0) and torch.all(dh[T + 1] == 7.0), "dhidden guard rows overwritten"
    assert torch.all(dW[0] == 5.0) and torch.all(dW[D + 1] == 5.0), "dW guard rows overwritten"
    if ld_pad:
        v4 = (V + 3) // 4 * 4   # stores go out in 16-byte units: up to 3 pad columns become zero
        assert torch.all(dW[1:D + 1, v4:] == 5.0), "dW columns beyond the 16-byte unit overwritten"
        assert torch.all((dW[1:D + 1, V:v4] == 5.0) | (dW[1:D + 1, V:v4] == 0.0))
    return {"loss": loss.item(), "dh": dh[1:T + 1].float().cpu().numpy().astype(np.float64),
            "dW": dW[1:D + 1, :V].cpu().numpy().astype(np.float64), "token_logp": tl.cpu().numpy(),
            "adv": adv.cpu().numpy(), "stats": rb.read_stats(stats)}


def compare_head(o, g, w):
    dt = torch.bfloat16
    assert g["stats"]["status"] == 0
    np.testing.assert_allclose(g["token_logp"], o["token_logp"], rtol=0, atol=LOGP_ATOL[dt])
    np.testing.assert_allclose(g["adv"], o["adv64"], rtol=0, atol=adv_atol(dt, w.seq_len))
    scale = max(abs(o["loss"]), 1e-3 * float(np.abs(o["coef"] * o["seq_logp"]).sum()), 1e-30)
    assert abs(g["loss"] - o["loss"]) / scale <= LOSS_RTOL[dt]
    assert g["stats"]["n_tokens"] == o["stats"]["n_tokens"]
    rss_h = np.sqrt((o["dz"] ** 2) @ (o["W"] ** 2).T)
    tol_h = 2.0 ** -6 * rss_h + 2.0 ** -8 * np.abs(o["dh"]) + 1e-12
    bad = np.abs(g["dh"] - o["dh"]) > tol_h
    assert not bad.any(), f"dhidden: {bad.sum()} elements out of tolerance, worst ratio " \
                          f"{(np.abs(g['dh'] - o['dh']) / tol_h).max():.2f}"
    rss_w = np.sqrt((o["h"] ** 2).T @ (o["dz"] ** 2))
    tol_w = 2.0 ** -6 * rss_w + 1e-6 * np.abs(o["dW"]) + 1e-12
    bad = np.abs(g["dW"] - o["dW"]) > tol_w
    assert not bad.any(), f"dW: {bad.sum()} elements out of tolerance, worst ratio " \
                          f"{(np.abs(g['dW'] - o['dW']) / tol_w).max():.2f}"
    # rows without gradient are exactly zero
    dead = ~(o["ok"] & (np.repeat(o["coef"], w.seq_len) != 0.0))
    assert np.all(g["dh"][dead] == 0.0)
    # the gradients are not trivially small: the test would notice a missing term
    assert np.abs(o["dh"]).max() > 100 * tol_h.mean() or np.abs(o["dh"]).max() > 1e-4


@pytest.mark.parametrize("V,D,L,pad", [(1000, 192, 40, 0), (777, 200, 50, 7), (256, 64, 32, 0), (5000, 1536, 33, 8)])
def test_fused_head_scaled(V, D, L, pad):
    """Ragged everything: rows not a multiple of 128, vocabulary not a multiple of 256 (or of 8),
    hidden size not a multiple of 64, ragged generation lengths, a padded weight pitch."""
    pad = (-V) % 8 + pad if (V + pad) % 8 else pad
    w = synth.CONFIGS["fused"].scaled(n_prompts=3, group_size=4, seq_len=L, vocab=V, hidden=D,
                                      length_mode="uniform", len_lo=L // 3, reward_mode="per_prompt_const",
                                      seed=300 + V)
    b = synth.make_head(w)
    o = oracle_head(b, w)
    g = run_head(b, w, o["behav"], ld_pad=pad)
    compare_head(o, g, w)
    assert np.all(o["adv64"][:4] == 0.0)   # the all-zero-reward group: its rows give no gradient


@pytest.mark.parametrize("flags,eta", [(rb.FLAG_OUTER_UNCLIPPED, 2.0), (rb.FLAG_NORM_TOKENS, 0.5),
                                       (rb.FLAG_LEAVE_ONE_OUT, float("inf"))])
def test_fused_head_flags(flags, eta):
    w = synth.CONFIGS["fused"].scaled(n_prompts=2, group_size=3, seq_len=20, vocab=520, hidden=128, seed=77)
    b = synth.make_head(w)
    b["rewards"] = torch.randn(w.n_seq, generator=torch.Generator().manual_seed(5))
    o = oracle_head(b, w, eta, flags)
    g = run_head(b, w, o["behav"], eta=eta, flags=flags)
    compare_head(o, g, w)


def test_fused_head_equals_logits_in_path_on_materialised_logits():
    """Special case that pins the fused form to the logits-in form: feed z = h W, rounded to
    float32, to rapid_pg_loss_fwd_bwd; losses agree to float32-path accuracy."""
    w = synth.CONFIGS["fused"].scaled(n_prompts=2, group_size=4, seq_len=24, vocab=1024, hidden=256, seed=9)
    b = synth.make_head(w)
    o = oracle_head(b, w)
    g = run_head(b, w, o["behav"])
    dev = torch.device("cuda")
    z = (b["hidden"].to(dev).float() @ b["w_vocab"].to(dev).float()).contiguous()
    res = rb.pg_loss(z, b["targets"].to(dev), b["mask"].to(dev), o["behav"].to(dev), b["rewards"].to(dev),
                     b["group_offsets"].to(dev), w.n_seq, w.seq_len)
    torch.cuda.synchronize()
    assert abs(res.loss.item() - g["loss"]) <= 2e-3 * max(abs(g["loss"]), 1e-6)
