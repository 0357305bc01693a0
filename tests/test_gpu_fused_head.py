"""GPU parity of the fused LM-head form against the float64 oracle: z = h W in float64 from the
same bf16 bits, steps 1-6 on z, then dh = dz W^T and dW = h^T dz.

Tolerances.  Loss and token log-probabilities: the bf16-logits class (2e-3 relative, 2e-5).
dh and dW: the library rounds dlogits to bf16 before the two products, an independent relative
error of at most 2^-9 per element, so an output element sum_k a_k dz_k carries a random error of
standard deviation about 2^-9 sqrt(sum_k a_k^2 dz_k^2) / sqrt(3); the test allows 2^-6 times that
root-sum-square (many standard deviations), plus 2^-8 |ref| for dh's own rounding to bf16.

With RAPID_FLAG_HEAD_STORE_LOGITS the library works on bf16(h W): the oracle then rounds its float64
logits to bf16 before step 1.  The library rounds a float32 accumulator, the oracle the exact
product; where the exact logit lies within the accumulator's error (taken as 2^-20 sum_k |h_k W_kv|:
sixteen float32 ulps of the sum of magnitudes) of a rounding boundary the two may land on
neighbouring bf16 values.  A token log-probability z_y - lse then moves
by one bf16 ulp of z_y if the sampled token's logit is such an element, and by p_v ulp(z_v) for every
other such element v of the row (d lse / d z_v = p_v).  The test computes exactly that bound per row
from the oracle's own logits and adds it to the usual tolerance; it is far below the tolerance for
the typical row and matters where a high-probability token sits on a boundary.
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


def round_to_bf16(x):
    """float64 -> nearest bf16 value, as float64."""
    return torch.from_numpy(np.ascontiguousarray(x, np.float32)).to(torch.bfloat16).double().numpy()


def oracle_head(b, w, eta=2.0, flags=0):
    """Everything the oracle computes for one fused-head batch (small sizes: dense float64)."""
    T, V, L = w.n_rows, w.vocab, w.seq_len
    h_bits, w_bits = synth.bits_numpy(b["hidden"]), synth.bits_numpy(b["w_vocab"])
    tg, mk = b["targets"].numpy(), b["mask"].numpy()
    z = oracle.head_logits(h_bits, w_bits)
    ok = (mk != 0) & (tg >= 0) & (tg < V)
    logp_slack = np.zeros(T)
    if flags & rb.FLAG_HEAD_STORE_LOGITS:
        acc_err = 2.0 ** -20 * (np.abs(bf16_to_f64(h_bits)) @ np.abs(bf16_to_f64(w_bits)))
        either = np.abs(round_to_bf16(z + acc_err) - round_to_bf16(z - acc_err))   # one ulp where the rounding may go either way
        z = round_to_bf16(z)
        prob = np.exp(z - z.max(1, keepdims=True))
        prob /= prob.sum(1, keepdims=True)
        rows = np.arange(T)
        ycol = np.where(ok, tg, 0)
        prob[rows, ycol] = 1.0                               # the sampled token's own logit counts in full
        logp_slack = np.where(ok, (prob * either).sum(1), 0.0)
        flags &= ~rb.FLAG_HEAD_STORE_LOGITS                  # the rest of the oracle does not know the flag
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
            "dz": dz, "dh": dh, "dW": dW, "behav": behav, "ok": ok, "logp_slack": logp_slack,
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
    slack = o["logp_slack"]
    assert (np.abs(g["token_logp"] - o["token_logp"]) <= LOGP_ATOL[dt] + slack).all()
    assert np.median(slack) < 5 * LOGP_ATOL[dt], "the relaxation must stay small against the tolerance itself"
    seq_slack = slack.reshape(w.n_seq, w.seq_len).sum(1).max() * 2.0    # w_n = exp(sum of them), c <= 2
    np.testing.assert_allclose(g["adv"], o["adv64"], rtol=0, atol=adv_atol(dt, w.seq_len) + seq_slack)
    scale = max(abs(o["loss"]), 1e-3 * float(np.abs(o["coef"] * o["seq_logp"]).sum()), 1e-30)
    assert abs(g["loss"] - o["loss"]) / scale <= LOSS_RTOL[dt] + float(np.abs(np.repeat(o["coef"], w.seq_len)) @ slack) / scale
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


def test_fused_head_mid_size_many_tiles_per_cta():
    """2048 rows x 32000 columns x 512 hidden: 16 x 125 output tiles, i.e. about 14 per CTA through
    both accumulator buffers, a ragged last vocabulary tile, and K loops of 8, 500 and 32 blocks.
    Everything is compared against the dense float64 oracle."""
    w = synth.CONFIGS["fused"].scaled(n_prompts=2, group_size=4, seq_len=256, vocab=32000, hidden=512,
                                      length_mode="uniform", len_lo=100, reward_mode="per_prompt", seed=31)
    b = synth.make_head(w)
    o = oracle_head(b, w)
    g = run_head(b, w, o["behav"])
    compare_head(o, g, w)


def test_fused_head_full_size_config():
    """The full benchmark configuration (16384 x 1536 x 151936).  The float64 oracle forms the
    logits of ONE whole prompt group (2048 rows), which fixes that group's token log-probabilities,
    generation weights, advantages and coefficients independently of the GPU; dhidden is then
    compared on sampled rows of the group.  dW and the loss need every row, which the oracle
    cannot afford at this size: they are covered by properties that hold at any size -- the
    adjoint identity <dW, W> = <dhidden, h> (both equal sum z dz), finiteness, exact zeros -- and
    by the dense comparisons at smaller sizes above."""
    w = synth.CONFIGS["fused"]
    dev = torch.device("cuda")
    b = synth.make_head(w, device=dev)
    T, V, D, L, G = w.n_rows, w.vocab, w.hidden, w.seq_len, w.group_size
    rows_g = np.arange(G * L, dtype=np.int64)                     # group 0
    h_bits, w_bits = synth.bits_numpy(b["hidden"]), synth.bits_numpy(b["w_vocab"])
    tg = b["targets"].cpu().numpy()
    z = oracle.head_logits(h_bits, w_bits, rows_g)
    lse, lp = oracle.token_logp_f64(z, tg[rows_g])
    # behaviour log-probs: group 0 from the oracle, the other groups from a library logsumexp
    # (input synthesis only; any plausible values serve there)
    noise = b["behav_noise"].cpu().double()
    behav = torch.empty(T, dtype=torch.float64)
    behav[:G * L] = torch.from_numpy(lp) + noise[:G * L]
    for r0 in range(G * L, T, 1024):
        zz = b["hidden"][r0:r0 + 1024].float() @ b["w_vocab"].float()
        cur = zz.gather(1, b["targets"][r0:r0 + 1024].long().unsqueeze(1)).squeeze(1) - torch.logsumexp(zz, 1)
        behav[r0:r0 + 1024] = cur.double().cpu() + noise[r0:r0 + 1024]
    behav = behav.float()
    s, S, cnt = oracle.seq_reduce(G, L, lp, behav[:G * L].numpy(), np.ones(G * L, np.uint8))
    ga = oracle.group_advantage(b["rewards"][:G].cpu().numpy(), s, np.array([0, G], np.int32), 2.0, 0)
    coef = ga["clipped_w"] * ga["adv64"] / w.n_seq

    desc = rb.make_desc(w.n_seq, L, V, w.n_prompts, torch.bfloat16, V, 2.0, 0)
    ws = rb.alloc_fused_head_workspace(desc, D, dev)
    loss = torch.full((1,), float("nan"), device=dev)
    dh = torch.empty((T, D), dtype=torch.bfloat16, device=dev)
    dW = torch.empty((D, V), dtype=torch.float32, device=dev)
    tl = torch.empty(T, device=dev)
    adv = torch.empty(w.n_seq, device=dev)
    stats = rb.alloc_stats(dev)
    rb.rapid_pg_loss_fused_head(desc, b["hidden"], b["w_vocab"], b["targets"], b["mask"], behav.to(dev),
                                b["rewards"], b["group_offsets"], loss, dh, dW, tl, adv, stats, ws)
    torch.cuda.synchronize()
    st = rb.read_stats(stats)
    assert st["status"] == 0 and st["n_tokens"] == T and np.isfinite(loss.item())
    np.testing.assert_allclose(tl[:G * L].cpu().numpy(), lp, rtol=0, atol=LOGP_ATOL[torch.bfloat16])
    np.testing.assert_allclose(adv[:G].cpu().numpy(), ga["adv64"], rtol=0, atol=adv_atol(torch.bfloat16, L))

    sel = np.random.default_rng(4).choice(G * L, 48, replace=False)
    sel.sort()
    dz = oracle.dlogits_f64_inplace(z[sel].copy(), tg[sel], lse[sel], np.repeat(coef, L)[sel])
    ref = oracle.head_dhidden(dz, w_bits)
    Wf = bf16_to_f64(w_bits)
    tol = 2.0 ** -6 * np.sqrt((dz ** 2) @ (Wf ** 2).T) + 2.0 ** -8 * np.abs(ref) + 1e-12
    got = dh[torch.from_numpy(sel).to(dev)].float().cpu().numpy().astype(np.float64)
    assert (np.abs(got - ref) <= tol).all(), f"worst ratio {(np.abs(got - ref) / tol).max():.2f}"
    assert np.abs(ref).max() > 0

    assert torch.isfinite(dh.float()).all() and torch.isfinite(dW).all()
    a = sum((dW[d0:d0 + 128].double() * b["w_vocab"][d0:d0 + 128].double()).sum().item() for d0 in range(0, D, 128))
    c = (dh.double() * b["hidden"].double()).sum().item()
    assert abs(a - c) <= 1e-3 * max(abs(a), abs(c)) + 1e-2, (a, c)
    dead = (adv == 0).repeat_interleave(L)
    assert (dh[dead] == 0).all()


def test_fused_head_more_rows_than_one_backward_chunk():
    """18000 rows: the backward part runs as a chunk of 16384 rows and a ragged second one, whose
    contribution is ADDED to dW; everything against the dense float64 oracle."""
    w = synth.CONFIGS["fused"].scaled(n_prompts=3, group_size=3, seq_len=2000, vocab=600, hidden=64,
                                      length_mode="uniform", len_lo=1500, reward_mode="per_prompt", seed=71)
    b = synth.make_head(w)
    b["rewards"] = torch.randn(w.n_seq, generator=torch.Generator().manual_seed(8))
    o = oracle_head(b, w)
    g = run_head(b, w, o["behav"])
    compare_head(o, g, w)
    # the second chunk's rows really contribute: dW restricted to the first chunk differs from the total
    first = 16384
    part = (o["h"][:first].T @ o["dz"][:first])
    assert np.abs(part - o["dW"]).max() > 100 * 2.0 ** -6 * np.sqrt((o["h"][first:] ** 2).T @ (o["dz"][first:] ** 2)).mean()


def test_fused_head_bad_tokens_and_empty_generation():
    """Token ids outside [0, V) count as masked and are reported; a generation with no unmasked
    token has weight 1 and no gradient; an empty group is skipped."""
    w = synth.CONFIGS["fused"].scaled(n_prompts=2, group_size=3, seq_len=10, vocab=304, hidden=64, seed=5)
    b = synth.make_head(w)
    b["targets"][3] = 304
    b["targets"][17] = -5
    b["mask"][20:30] = 0                                  # generation 2: nothing counts
    b["rewards"] = torch.tensor([1.0, 0.0, 0.5, 0.0, 1.0, 1.0])
    b["group_offsets"] = torch.tensor([0, 3, 3, 6], dtype=torch.int32)   # an empty group in the middle
    w = w.scaled(n_prompts=3, group_size=2)               # three groups now; the same six generations
    o = oracle_head(b, w)
    g = run_head(b, w, o["behav"])
    compare_head(o, g, w)
    assert g["stats"]["n_bad_token"] == 2 and g["stats"]["n_empty_group"] == 1
    assert g["stats"]["n_tokens"] == 60 - 10 - 2
    assert np.all(g["dh"][20:30] == 0.0) and np.all(g["dh"][[3, 17]] == 0.0)


@pytest.mark.parametrize("V,D,L", [(40, 8, 3), (8, 16, 1), (300 - 4, 24, 2)])
def test_fused_head_shapes_smaller_than_one_tile(V, D, L):
    """Vocabulary, hidden size and row count all below one 128 x 256 x 64 tile: the TMA boxes hang
    over every edge of every matrix."""
    w = synth.CONFIGS["fused"].scaled(n_prompts=1, group_size=3, seq_len=L, vocab=V, hidden=D, seed=90 + V)
    b = synth.make_head(w)
    b["rewards"] = torch.tensor([1.0, 0.0, -0.5])
    o = oracle_head(b, w)
    g = run_head(b, w, o["behav"])
    compare_head(o, g, w)


@pytest.mark.parametrize("V,D,L,pad", [(1000, 192, 40, 0), (777, 200, 50, 7), (5000, 1536, 33, 8), (40, 8, 3, 0)])
def test_fused_head_stored_logits(V, D, L, pad):
    """RAPID_FLAG_HEAD_STORE_LOGITS: three contractions, the logits kept in bf16 between forward and
    backward.  Same ragged shapes as above; the oracle works on its own bf16 rounding of h W."""
    pad = (-V) % 8 + pad if (V + pad) % 8 else pad
    w = synth.CONFIGS["fused"].scaled(n_prompts=3, group_size=4, seq_len=L, vocab=V, hidden=D,
                                      length_mode="uniform", len_lo=max(1, L // 3), reward_mode="per_prompt_const",
                                      seed=300 + V)
    b = synth.make_head(w)
    o = oracle_head(b, w, flags=rb.FLAG_HEAD_STORE_LOGITS)
    g = run_head(b, w, o["behav"], ld_pad=pad, flags=rb.FLAG_HEAD_STORE_LOGITS)
    compare_head(o, g, w)


def test_fused_head_stored_logits_more_rows_than_one_backward_chunk():
    """18000 rows with stored logits: the bf16 matrix covers all rows, dh and dW still run per chunk."""
    w = synth.CONFIGS["fused"].scaled(n_prompts=3, group_size=3, seq_len=2000, vocab=600, hidden=64,
                                      length_mode="uniform", len_lo=1500, reward_mode="per_prompt", seed=71)
    b = synth.make_head(w)
    b["rewards"] = torch.randn(w.n_seq, generator=torch.Generator().manual_seed(8))
    o = oracle_head(b, w, flags=rb.FLAG_HEAD_STORE_LOGITS)
    g = run_head(b, w, o["behav"], flags=rb.FLAG_HEAD_STORE_LOGITS)
    compare_head(o, g, w)


def test_fused_head_stored_logits_bad_tokens_and_flags():
    """Out-of-range token ids, an empty generation, an empty group, token normalisation and the
    unclipped outer weight, all with stored logits."""
    w = synth.CONFIGS["fused"].scaled(n_prompts=2, group_size=3, seq_len=10, vocab=304, hidden=64, seed=5)
    b = synth.make_head(w)
    b["targets"][3] = 304
    b["targets"][17] = -5
    b["mask"][20:30] = 0
    b["rewards"] = torch.tensor([1.0, 0.0, 0.5, 0.0, 1.0, 1.0])
    b["group_offsets"] = torch.tensor([0, 3, 3, 6], dtype=torch.int32)
    w = w.scaled(n_prompts=3, group_size=2)
    flags = rb.FLAG_HEAD_STORE_LOGITS | rb.FLAG_NORM_TOKENS | rb.FLAG_OUTER_UNCLIPPED
    o = oracle_head(b, w, 0.5, flags)
    g = run_head(b, w, o["behav"], eta=0.5, flags=flags)
    compare_head(o, g, w)
    assert g["stats"]["n_bad_token"] == 2 and g["stats"]["n_empty_group"] == 1
    assert np.all(g["dh"][20:30] == 0.0) and np.all(g["dh"][[3, 17]] == 0.0)
