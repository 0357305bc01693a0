"""GPU parity of the fused LM-head form against the float64 oracle: z = h W in float64 from the
same bf16 bits, steps 1-6 on z, then dh = dz W^T and dW = h^T dz.

Tolerances.  Loss and token log-probabilities: the bf16-logits class (2e-3 relative, 2e-5).
dh and dW: the library rounds dlogits to bf16 before the two products, an independent relative
error of at most 2^-8 per element (half a unit in the last place of an 8-bit significand; 2^-9 at
the top of a binade), so an output element sum_k a_k dz_k carries a random error of standard
deviation about 0.4 * 2^-8 sqrt(sum_k a_k^2 dz_k^2); the test allows 2^-6 times that root-sum-square
(ten standard deviations; where one term dominates the sum -- the sampled token's g (p_y - 1) in
dh -- its single rounding error of up to 2^-8 is a quarter of the allowance), plus 2^-8 |ref| for
dh's own rounding to bf16.  At full size a third term enters: dh and dW are linear in the
coefficient g_n = c_n A_n / N, and A_n is only held to the advantage tolerance (absolute), so a
generation whose advantage nearly cancels has a relatively uncertain coefficient; the allowance is
the advantage tolerance propagated through g_n, i.e. |contribution of generation n| * dg_n / |g_n|
with dg_n = c_n (1 + |A_n|) * (advantage tolerance) / N.

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
from parity_util import HEAD_LOGP_ATOL, LOSS_RTOL, head_adv_atol  # noqa: E402


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
    dw_bf16 = bool(flags & rb.FLAG_HEAD_DW_BF16)
    dW = torch.full((D + 2, ld), 5.0, dtype=torch.bfloat16 if dw_bf16 else torch.float32, device=dev)
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
        unit = 8 if dw_bf16 else 4
        v4 = (V + unit - 1) // unit * unit   # stores go out in 16-byte units: the pad columns of the last unit become zero
        assert torch.all(dW[1:D + 1, v4:] == 5.0), "dW columns beyond the 16-byte unit overwritten"
        assert torch.all((dW[1:D + 1, V:v4] == 5.0) | (dW[1:D + 1, V:v4] == 0.0))
    return {"loss": loss.item(), "dh": dh[1:T + 1].float().cpu().numpy().astype(np.float64),
            "dW": dW[1:D + 1, :V].float().cpu().numpy().astype(np.float64), "dw_bf16": dw_bf16,
            "token_logp": tl.cpu().numpy(),
            "adv": adv.cpu().numpy(), "stats": rb.read_stats(stats)}


def compare_head(o, g, w):
    dt = torch.bfloat16
    assert g["stats"]["status"] == 0
    slack = o["logp_slack"]
    assert (np.abs(g["token_logp"] - o["token_logp"]) <= HEAD_LOGP_ATOL + slack).all()
    assert np.median(slack) < 5 * HEAD_LOGP_ATOL, "the relaxation must stay small against the tolerance itself"
    seq_slack = slack.reshape(w.n_seq, w.seq_len).sum(1).max() * 2.0    # w_n = exp(sum of them), c <= 2
    np.testing.assert_allclose(g["adv"], o["adv64"], rtol=0, atol=head_adv_atol(w.seq_len) + seq_slack)
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
    if g.get("dw_bf16"):
        # dW itself rounded to bf16: once per backward chunk of 16384 rows (2^-8 relative each), and
        # the chunks' sums are added in bf16
        n_chunks = (w.n_rows + 16383) // 16384
        tol_w = tol_w + (2 * n_chunks - 1) * 2.0 ** -8 * np.abs(o["dW"]) + (n_chunks - 1) * 2.0 ** -8 * np.abs(o["h"]).T @ np.abs(o["dz"])
    bad = np.abs(g["dW"] - o["dW"]) > tol_w
    assert not bad.any(), f"dW: {bad.sum()} elements out of tolerance, worst ratio " \
                          f"{(np.abs(g['dW'] - o['dW']) / tol_w).max():.2f}"
    # rows without gradient are exactly zero
    dead = ~(o["ok"] & (np.repeat(o["coef"], w.seq_len) != 0.0))
    assert np.all(g["dh"][dead] == 0.0)
    # the gradients are not trivially small: the test would notice a missing term
    assert np.abs(o["dh"]).max() > 100 * tol_h.mean() or np.abs(o["dh"]).max() > 1e-4


@pytest.mark.parametrize("extra", [0, rb.FLAG_HEAD_SINGLE_CTA])
@pytest.mark.parametrize("V,D,L,pad", [(1000, 192, 40, 0), (777, 200, 50, 7), (256, 64, 32, 0), (5000, 1536, 33, 8)])
def test_fused_head_scaled(V, D, L, pad, extra):
    """Ragged everything: rows not a multiple of 128, vocabulary not a multiple of 256 (or of 8),
    hidden size not a multiple of 64, ragged generation lengths, a padded weight pitch.  Once with
    the default mix of kernels (forward and recompute on CTA pairs, dhidden and dW on single CTAs) and
    once with every contraction on single CTAs."""
    pad = (-V) % 8 + pad if (V + pad) % 8 else pad
    w = synth.CONFIGS["fused"].scaled(n_prompts=3, group_size=4, seq_len=L, vocab=V, hidden=D,
                                      length_mode="uniform", len_lo=L // 3, reward_mode="per_prompt_const",
                                      seed=300 + V)
    b = synth.make_head(w)
    o = oracle_head(b, w)
    g = run_head(b, w, o["behav"], ld_pad=pad, flags=extra)
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


@pytest.mark.parametrize("V,D,L,pad,extra", [(1000, 192, 40, 0, 0), (777, 200, 50, 7, 0), (5000, 1536, 33, 8, 0),
                                             (40, 8, 3, 0, 0), (1000, 192, 40, 0, rb.FLAG_HEAD_STORE_LOGITS),
                                             (5000, 1536, 33, 8, rb.FLAG_HEAD_STORE_LOGITS)])
def test_fused_head_cta_pairs(V, D, L, pad, extra):
    """RAPID_FLAG_HEAD_CTA_PAIRS: every contraction on pairs of CTAs (256 x 256 tiles, tcgen05 cta_group::2).
    Ragged rows (not a multiple of 256, so the second CTA of the last pair is partly or wholly past the
    end), vocabulary and hidden size; both forms of the head; everything against the dense oracle."""
    pad = (-V) % 8 + pad if (V + pad) % 8 else pad
    w = synth.CONFIGS["fused"].scaled(n_prompts=3, group_size=4, seq_len=L, vocab=V, hidden=D,
                                      length_mode="uniform", len_lo=max(1, L // 3), reward_mode="per_prompt_const",
                                      seed=300 + V)
    b = synth.make_head(w)
    o = oracle_head(b, w, flags=extra)
    g = run_head(b, w, o["behav"], ld_pad=pad, flags=extra | rb.FLAG_HEAD_CTA_PAIRS)
    compare_head(o, g, w)


@pytest.mark.parametrize("extra", [0, rb.FLAG_HEAD_CTA_PAIRS, rb.FLAG_HEAD_STORE_LOGITS])
@pytest.mark.parametrize("V,D,L,pad", [(1000, 192, 40, 0), (777, 200, 50, 7), (40, 8, 3, 0)])
def test_fused_head_weight_gradient_in_bf16(V, D, L, pad, extra):
    """RAPID_FLAG_HEAD_DW_BF16: dW comes out as bf16 (guard rows and pad columns untouched), through the
    single-CTA and the CTA-pair kernels."""
    pad = (-V) % 8 + pad if (V + pad) % 8 else pad
    w = synth.CONFIGS["fused"].scaled(n_prompts=3, group_size=4, seq_len=L, vocab=V, hidden=D,
                                      length_mode="uniform", len_lo=max(1, L // 3), reward_mode="per_prompt_const",
                                      seed=300 + V)
    b = synth.make_head(w)
    o = oracle_head(b, w, flags=extra & rb.FLAG_HEAD_STORE_LOGITS)
    g = run_head(b, w, o["behav"], ld_pad=pad, flags=extra | rb.FLAG_HEAD_DW_BF16)
    compare_head(o, g, w)


def test_fused_head_weight_gradient_in_bf16_over_two_backward_chunks():
    """18000 rows: the second chunk's contribution is added to a bf16 dW."""
    w = synth.CONFIGS["fused"].scaled(n_prompts=3, group_size=3, seq_len=2000, vocab=600, hidden=64,
                                      length_mode="uniform", len_lo=1500, reward_mode="per_prompt", seed=71)
    b = synth.make_head(w)
    b["rewards"] = torch.randn(w.n_seq, generator=torch.Generator().manual_seed(8))
    o = oracle_head(b, w)
    compare_head(o, run_head(b, w, o["behav"], flags=rb.FLAG_HEAD_DW_BF16), w)


def test_fused_head_cta_pairs_many_tiles_and_two_backward_chunks():
    """Pairs of CTAs over many tiles per pair (2048 x 32000 x 512) and over two backward chunks (18000
    rows, the second one ragged, its contribution added to dW)."""
    w = synth.CONFIGS["fused"].scaled(n_prompts=2, group_size=4, seq_len=256, vocab=32000, hidden=512,
                                      length_mode="uniform", len_lo=100, reward_mode="per_prompt", seed=31)
    b = synth.make_head(w)
    o = oracle_head(b, w)
    compare_head(o, run_head(b, w, o["behav"], flags=rb.FLAG_HEAD_CTA_PAIRS), w)
    w = synth.CONFIGS["fused"].scaled(n_prompts=3, group_size=3, seq_len=2000, vocab=600, hidden=64,
                                      length_mode="uniform", len_lo=1500, reward_mode="per_prompt", seed=71)
    b = synth.make_head(w)
    b["rewards"] = torch.randn(w.n_seq, generator=torch.Generator().manual_seed(8))
    o = oracle_head(b, w)
    compare_head(o, run_head(b, w, o["behav"], flags=rb.FLAG_HEAD_CTA_PAIRS), w)


@pytest.fixture(scope="module")
def full_size_oracle():
    """The float64 oracle over ALL 16 384 rows of the full benchmark configuration
    (16384 x 1536 x 151936), for both forms of the head: logits as the exact product, and logits
    rounded to bf16 (what RAPID_FLAG_HEAD_STORE_LOGITS keeps).

    z = h W is formed a block of 1024 rows at a time with the library's float64 matrix product
    (oracle.head_logits_dgemm: 3.8e12 multiply-adds in all; its plain-loop twin is checked against
    it on sampled rows of every block) and dropped again; what is kept per row is the log-sum-exp
    and the sampled token's log-probability, plus the logits of a seeded sample of 48 rows (six
    from each prompt group, for dhidden) and of 40 vocabulary columns over all rows (24 random, 8
    inside the ragged last 256-column tile, 8 that are some row's sampled token; for dW)."""
    return _oracle_over_all_rows(synth.CONFIGS["fused"], torch.device("cuda"), block=1024)


def _oracle_over_all_rows(w, dev, block):
    from concurrent.futures import ThreadPoolExecutor
    b = synth.make_head(w, device=dev)
    T, V, D, L, G = w.n_rows, w.vocab, w.hidden, w.seq_len, w.group_size
    h_bits, w_bits = synth.bits_numpy(b["hidden"]), synth.bits_numpy(b["w_vocab"])
    tg = b["targets"].cpu().numpy()
    Wf = oracle.decode_bf16(w_bits)
    absW = np.abs(Wf)

    rng = np.random.default_rng(4)
    per_group = G * L
    sel_rows = np.sort(np.concatenate([k * per_group + rng.choice(per_group, 6, replace=False)
                                       for k in range(w.n_prompts)])).astype(np.int64)
    last_tile = V // 256 * 256
    cols = np.unique(np.concatenate([rng.choice(V, 24, replace=False), last_tile + rng.choice(V - last_tile, 8, replace=False),
                                     tg[rng.choice(T, 8, replace=False)]])).astype(np.int64)

    forms = {f: {"lse": np.zeros(T), "lp": np.zeros(T), "slack": np.zeros(T), "z_rows": np.zeros((len(sel_rows), V)),
                 "z_cols": np.zeros((T, len(cols)))} for f in ("exact", "bf16")}
    pool = ThreadPoolExecutor(oracle.max_threads())

    def stats_of(z, r0):
        """oracle step 1 on the rows of a block, its rows spread over the host's cores"""
        n = z.shape[0]
        cuts = list(range(0, n, 32))
        parts = list(pool.map(lambda c: oracle.token_logp_f64(z[c:c + 32], tg[r0 + c:r0 + c + 32]), cuts))
        return np.concatenate([p[0] for p in parts]), np.concatenate([p[1] for p in parts])

    assert T % block == 0
    worst_twin = 0.0
    for r0 in range(0, T, block):
        rows = np.arange(r0, r0 + block, dtype=np.int64)
        z = oracle.head_logits_dgemm(h_bits, Wf, rows)
        probe = rows[[3, block // 2, block - 1]]
        twin = oracle.head_logits(h_bits, w_bits, probe)
        worst_twin = max(worst_twin, float(np.abs(twin - z[probe - r0]).max()))
        mine = (sel_rows >= r0) & (sel_rows < r0 + block)
        for form, f in forms.items():
            if form == "bf16":
                mag = np.abs(oracle.decode_bf16(h_bits[rows])) @ absW
                mag *= 2.0 ** -20                                   # the float32 accumulator's error
                either = np.abs(round_to_bf16(z + mag) - round_to_bf16(z - mag))
                del mag
                z = round_to_bf16(z)
            lse, lp = stats_of(z, r0)
            f["lse"][rows], f["lp"][rows] = lse, lp
            f["z_rows"][mine] = z[sel_rows[mine] - r0]
            f["z_cols"][rows] = z[:, cols]
            if form == "bf16":
                # a token log-probability moves by ulp(z_y) if the sampled token's logit may round either
                # way, and by p_v ulp(z_v) for every other such element of the row
                ar, y = np.arange(block), tg[rows]
                ey = either[ar, y].copy()
                either *= np.exp(z - lse[:, None])
                f["slack"][rows] = either.sum(1) + (1.0 - np.exp(lp)) * ey
                del either
    pool.shutdown()
    assert worst_twin <= 1e-11, worst_twin

    noise = b["behav_noise"].cpu().double()
    go = b["group_offsets"].cpu().numpy()
    for f in forms.values():
        f["behav"] = (torch.from_numpy(f["lp"]) + noise).float()
        s, S, cnt = oracle.seq_reduce(w.n_seq, L, f["lp"], f["behav"].numpy(), np.ones(T, np.uint8))
        ga = oracle.group_advantage(b["rewards"].cpu().numpy(), s, go, 2.0, 0)
        f["loss"], f["coef"], f["stats"] = oracle.coef_loss(s, S, cnt, ga["weight"], ga["clipped_w"], ga["adv64"], 2.0, 0)
        f["adv64"], f["seq_logp"], f["weight"] = ga["adv64"], S, ga["weight"]
        g_row = np.repeat(f["coef"], L)
        # relative uncertainty of each generation's coefficient that the advantage tolerance leaves
        seq_slack = f["slack"].reshape(w.n_seq, L).sum(1).max() * 2.0
        dg = ga["clipped_w"] * (1.0 + np.abs(ga["adv64"])) * (head_adv_atol(L) + seq_slack) / w.n_seq
        g_rel = np.repeat(np.where(f["coef"] != 0.0, dg / np.maximum(np.abs(f["coef"]), 1e-300), 0.0), L)
        dz = oracle.dlogits_f64_inplace(f["z_rows"].copy(), tg[sel_rows], f["lse"][sel_rows], g_row[sel_rows])
        f["dh_rows"] = oracle.head_dhidden(dz, w_bits)
        f["dh_tol"] = 2.0 ** -6 * np.sqrt((dz ** 2) @ (Wf ** 2).T) + \
            (2.0 ** -8 + g_rel[sel_rows][:, None]) * np.abs(f["dh_rows"]) + 1e-12
        f["dh_coef_share"] = g_rel[sel_rows][:, None] * np.abs(f["dh_rows"]) / f["dh_tol"]
        pos = np.full(T, -1, np.int32)                              # the sampled token's place among the columns
        hit = np.isin(tg, cols)
        pos[hit] = np.searchsorted(cols, tg[hit])
        dzc = oracle.dlogits_f64_inplace(f["z_cols"].copy(), pos, f["lse"], g_row)
        f["dW_cols"] = np.zeros((D, len(cols)))
        oracle.head_dweight_accum(f["dW_cols"], dzc, h_bits)
        hf = oracle.decode_bf16(h_bits)
        f["dW_tol"] = 2.0 ** -6 * np.sqrt((hf ** 2).T @ (dzc ** 2)) + 1e-6 * np.abs(f["dW_cols"]) + \
            np.abs(hf).T @ (np.abs(dzc) * g_rel[:, None]) + 1e-12
        f["onehot_cols"] = int(hit.sum())
    return {"w": w, "b": b, "forms": forms, "sel_rows": sel_rows, "cols": cols}


@pytest.mark.parametrize("form,flags", [("exact", 0), ("bf16", rb.FLAG_HEAD_STORE_LOGITS),
                                        ("exact", rb.FLAG_HEAD_CTA_PAIRS), ("exact", rb.FLAG_HEAD_SINGLE_CTA),
                                        ("bf16", rb.FLAG_HEAD_STORE_LOGITS | rb.FLAG_HEAD_SINGLE_CTA)])
def test_fused_head_full_size_config(full_size_oracle, form, flags):
    """The full benchmark configuration against the oracle on every row: all 16 384 token
    log-probabilities, all 64 advantages, the loss, the statistics; dhidden on 48 sampled rows
    spread over all eight prompt groups; dW on 40 sampled vocabulary columns (all 1536 entries of
    each), some in the ragged last tile, some carrying a sampled token's one-hot term.  Beside
    that, properties that hold for every element: finiteness, exact zeros for generations with
    zero advantage, and the adjoint identity <dW, W> = <dhidden, h> (both equal sum z dz)."""
    from parity_util import report_observed
    fx, f = full_size_oracle, full_size_oracle["forms"][form]
    w, b = fx["w"], fx["b"]
    dev = torch.device("cuda")
    T, V, D, L = w.n_rows, w.vocab, w.hidden, w.seq_len
    dt = torch.bfloat16

    desc = rb.make_desc(w.n_seq, L, V, w.n_prompts, dt, V, 2.0, flags)
    ws = rb.alloc_fused_head_workspace(desc, D, dev)
    loss = torch.full((1,), float("nan"), device=dev)
    dh = torch.empty((T, D), dtype=dt, device=dev)
    dW = torch.empty((D, V), dtype=torch.float32, device=dev)
    tl = torch.empty(T, device=dev)
    adv = torch.empty(w.n_seq, device=dev)
    stats = rb.alloc_stats(dev)
    rb.rapid_pg_loss_fused_head(desc, b["hidden"], b["w_vocab"], b["targets"], b["mask"], f["behav"].to(dev),
                                b["rewards"], b["group_offsets"], loss, dh, dW, tl, adv, stats, ws)
    torch.cuda.synchronize()
    del ws
    st = rb.read_stats(stats)
    assert st["status"] == 0 and st["n_tokens"] == T and st["n_bad_token"] == 0

    slack = f["slack"]
    lp_err = np.abs(tl.cpu().numpy() - f["lp"])
    assert (lp_err <= HEAD_LOGP_ATOL + slack).all(), f"token log-prob: worst {(lp_err / (HEAD_LOGP_ATOL + slack)).max():.2f} x bound"
    assert np.median(slack) < 5 * HEAD_LOGP_ATOL
    seq_slack = slack.reshape(w.n_seq, L).sum(1).max() * 2.0
    adv_err = np.abs(adv.cpu().numpy() - f["adv64"])
    assert (adv_err <= head_adv_atol(L) + seq_slack).all()
    scale = max(abs(f["loss"]), 1e-3 * float(np.abs(f["coef"] * f["seq_logp"]).sum()), 1e-30)
    loss_bound = LOSS_RTOL[dt] + float(np.abs(np.repeat(f["coef"], L)) @ slack) / scale
    loss_rel = abs(loss.item() - f["loss"]) / scale
    assert loss_rel <= loss_bound, (loss.item(), f["loss"])
    assert abs(st["loss"] - f["loss"]) / scale <= loss_bound
    if not (np.abs(f["weight"] - 2.0) < 1e-3 + 2.0 * seq_slack).any():
        assert st["n_clipped"] == f["stats"]["n_clipped"]
    assert abs(st["mean_log_cw"] - f["stats"]["mean_log_cw"]) <= 1e-2 + seq_slack

    got = dh[torch.from_numpy(fx["sel_rows"]).to(dev)].float().cpu().numpy().astype(np.float64)
    dh_ratio = np.abs(got - f["dh_rows"]) / f["dh_tol"]
    assert (dh_ratio <= 1.0).all(), f"dhidden: worst {dh_ratio.max():.2f} x bound"
    assert np.abs(f["dh_rows"]).max() > 0
    gotW = dW[:, torch.from_numpy(fx["cols"]).to(dev)].cpu().numpy().astype(np.float64)
    dW_ratio = np.abs(gotW - f["dW_cols"]) / f["dW_tol"]
    assert (dW_ratio <= 1.0).all(), f"dW: worst {dW_ratio.max():.2f} x bound (column {fx['cols'][dW_ratio.max(0).argmax()]})"
    assert f["onehot_cols"] >= 8 and np.abs(f["dW_cols"]).max() > 100 * f["dW_tol"].mean()

    assert torch.isfinite(dh.float()).all() and torch.isfinite(dW).all()
    a = sum((dW[d0:d0 + 128].double() * b["w_vocab"][d0:d0 + 128].double()).sum().item() for d0 in range(0, D, 128))
    c = (dh.double() * b["hidden"].double()).sum().item()
    assert abs(a - c) <= 1e-3 * max(abs(a), abs(c)) + 1e-2, (a, c)
    dead = torch.from_numpy(np.repeat(f["coef"] == 0.0, L)).to(dev)
    assert (dh[dead] == 0).all()
    report_observed(f"fused head full size ({form} logits{', CTA pairs' if flags & rb.FLAG_HEAD_CTA_PAIRS else ', single CTAs' if flags & rb.FLAG_HEAD_SINGLE_CTA else ''})", token_logp=(lp_err / (HEAD_LOGP_ATOL + slack)).max(),
                    adv=(adv_err / (head_adv_atol(L) + seq_slack)).max(), loss=loss_rel / loss_bound,
                    dh=dh_ratio.max(), dW=dW_ratio.max(), loss_rel_abs=loss_rel,
                    coef_term_share_of_dh_bound_at_worst=f["dh_coef_share"].flat[dh_ratio.argmax()])


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
