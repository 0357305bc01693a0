"""GPU parity at the FULL sizes of the benchmark configurations, in the launch configuration the
benchmark times (statistics pass, finalize, dlogits pass over the whole resident batch; the
chunked three-step form for the long-sequence configuration).

The oracle runs steps 1-5 on every row, so token log-probabilities, advantages, the loss and the
statistics are compared in full.  dlogits (step 6) is compared against the oracle on a seeded
sample of rows (a few thousand, plus the rows around every mask boundary of a few generations),
and on ALL rows through properties that hold at any size: masked rows and zero-coefficient
generations are exactly zero, every row sums to zero within rounding, and nothing is non-finite.
Logits are drawn on the device (the host generator would take minutes) and the oracle is handed
the very bits the device holds.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2510_03515_b200 import binding as rb  # noqa: E402
from paper_2510_03515_b200 import synth  # noqa: E402
from parity_util import DLOGITS_ATOL, LOGP_ATOL, LOSS_RTOL, adv_atol, report_observed  # noqa: E402


def _oracle_steps_2_to_5(w, tok, lp, row_ok, behav, eta=2.0, flags=0):
    s, S, cnt = oracle.seq_reduce(w.n_seq, w.seq_len, lp, behav, row_ok)
    ga = oracle.group_advantage(tok["rewards"].numpy(), s, tok["group_offsets"].numpy(), eta, flags)
    loss, coef, st = oracle.coef_loss(s, S, cnt, ga["weight"], ga["clipped_w"], ga["adv64"], eta, flags)
    return {"loss": loss, "coef": coef, "seq_logp": S, "adv64": ga["adv64"], "weight": ga["weight"],
            "stats": st}


def _check_scalars(o, loss_gpu, adv_gpu, st, dt, seq_len):
    scale = max(abs(o["loss"]), 1e-3 * float(np.abs(o["coef"] * o["seq_logp"]).sum()), 1e-30)
    assert abs(loss_gpu - o["loss"]) / scale <= LOSS_RTOL[dt] + 6e-8 * abs(o["loss"]) / scale
    assert abs(st["loss"] - o["loss"]) / scale <= LOSS_RTOL[dt]
    np.testing.assert_allclose(adv_gpu, o["adv64"], rtol=0, atol=adv_atol(dt, seq_len))
    assert st["status"] == 0 and st["n_tokens"] == o["stats"]["n_tokens"] and st["n_bad_token"] == 0
    if not (np.abs(o["weight"] - 2.0) < 1e-3).any():
        assert st["n_clipped"] == o["stats"]["n_clipped"]
    assert abs(st["mean_log_cw"] - o["stats"]["mean_log_cw"]) <= (1e-4 if dt == torch.float32 else 1e-2)


def _sample_rows(w, tok, n_random, seed):
    """Seeded random rows plus the rows on both sides of the mask boundary of four generations."""
    rng = np.random.default_rng(seed)
    rows = set(rng.integers(0, w.n_rows, n_random).tolist())
    rows |= {0, w.n_rows - 1}
    for n in (0, 1, w.n_seq // 2, w.n_seq - 1):
        ln = int(tok["lengths"][n])
        for t in (0, ln - 1, ln, w.seq_len - 1):
            if 0 <= t < w.seq_len:
                rows.add(n * w.seq_len + t)
    return np.array(sorted(rows), dtype=np.int64)


def _property_checks(dz, live_row, dt, block=4096):
    """All rows, on the device: dead rows exactly zero, live rows sum to ~0, everything finite."""
    tol = 1e-5 if dt == torch.float32 else 1e-3  # |g| <= ~0.06; a row sums V values rounded to the dtype
    T = dz.shape[0]
    for r0 in range(0, T, block):
        blk = dz[r0:r0 + block].float()
        live = live_row[r0:r0 + block]
        assert torch.isfinite(blk).all()
        assert (blk[~live] == 0).all(), "a masked / zero-coefficient row is not zero"
        assert blk.sum(1).abs().max().item() <= tol


def _resident_batch_full_size(w, cases):
    """`cases`: list of (label, sigma, shift) -- behaviour log-probs = the oracle's current ones +
    N(0, sigma) + shift[n] per token of generation n.  Step 1 of the oracle (and the logits) do not
    depend on the behaviour policy, so they are computed once and shared by all cases."""
    dt = synth.torch_dtype(w)
    dev = torch.device("cuda")
    tok = synth.make_tokens(w.scaled(behav_sigma=1.0))           # unit noise, scaled per case below
    T, V, N = w.n_rows, w.vocab, w.n_seq
    logits = synth.logits_for_sequences(w, tok["targets"], 0, N, device=dev)
    host = logits.cpu()
    bits = synth.bits_numpy(host)
    pre = oracle.token_logp(bits, V, tok["targets"].numpy(), tok["mask"].numpy())
    targets, mask = tok["targets"].to(dev), tok["mask"].to(dev)
    desc = rb.make_desc(N, w.seq_len, V, w.n_prompts, dt, logits.stride(0), 2.0, 0)
    ws = rb.alloc_workspace(desc, dev)
    dz = torch.empty_like(logits)
    rows = _sample_rows(w, tok, 3000, seed=w.seed)
    outs = {}
    for label, sigma, shift in cases:
        noise = tok["behav_noise"].double() * sigma
        if shift is not None:
            noise = noise + torch.from_numpy(np.repeat(shift, w.seq_len))
        behav = (torch.from_numpy(pre["token_logp"]) + noise).float()
        o = _oracle_steps_2_to_5(w, tok, pre["token_logp"], pre["row_ok"], behav.numpy())

        loss = torch.zeros(1, device=dev)
        tl = torch.empty(T, device=dev)
        adv = torch.empty(N, device=dev)
        stats = rb.alloc_stats(dev)
        dz.fill_(float("nan"))
        rb.rapid_pg_stats_chunk(desc, logits, 0, T, targets, mask, ws)
        rb.rapid_pg_finalize(desc, behav.to(dev), tok["rewards"].to(dev), tok["group_offsets"].to(dev), loss,
                             tl, adv, stats, ws)
        rb.rapid_pg_dlogits_chunk(desc, logits, dz, 0, T, targets, stats, ws)
        torch.cuda.synchronize()

        np.testing.assert_allclose(tl.cpu().numpy(), pre["token_logp"], rtol=0, atol=LOGP_ATOL[dt])
        st = rb.read_stats(stats)
        _check_scalars(o, loss.item(), adv.cpu().numpy(), st, dt, w.seq_len)

        worst = 0.0
        for i in range(0, len(rows), 256):
            sel = rows[i:i + 256]
            ref = oracle.dlogits_rows(bits, V, w.seq_len, tok["targets"].numpy(), pre["row_ok"], pre["lse"],
                                      o["coef"], sel)
            got = dz[torch.from_numpy(sel).to(dev)].float().cpu().numpy().astype(np.float64)
            worst = max(worst, float(np.abs(got - ref).max()))
        assert worst <= DLOGITS_ATOL[dt], f"{label}: dlogits max abs err {worst}"

        live = torch.from_numpy(pre["row_ok"].astype(bool) & (np.repeat(o["coef"], w.seq_len) != 0.0)).to(dev)
        _property_checks(dz, live, dt)
        scale = max(abs(o["loss"]), 1e-3 * float(np.abs(o["coef"] * o["seq_logp"]).sum()), 1e-30)
        report_observed(f"{w.name} full size, {label}", loss=abs(loss.item() - o["loss"]) / scale / LOSS_RTOL[dt],
                        token_logp=np.abs(tl.cpu().numpy() - pre["token_logp"]).max() / LOGP_ATOL[dt],
                        adv=np.abs(adv.cpu().numpy() - o["adv64"]).max() / adv_atol(dt, w.seq_len),
                        dlogits=worst / DLOGITS_ATOL[dt])
        outs[label] = (o, st)
    assert torch.equal(logits.cpu(), host), "logits modified"
    return outs


def test_slm_batch_full_size():
    w = synth.CONFIGS["slm"]
    _resident_batch_full_size(w, [("sigma 0.2", w.behav_sigma, None)])


def test_staleness_sweep_full_size():
    """128 x 512 tokens at every staleness level of the sweep, sigma in {0, 0.1, 0.5, 1, 2}: from
    weights that are all one to log-weights with a standard deviation of 2 sqrt(512) = 45, where
    nearly every weight is either clipped at eta or vanishes.  A sixth case shifts three
    generations' behaviour log-probs by -2 per token, so that their log-weight passes 709 and the
    exponential overflows to +inf in double precision, which the clip turns into eta."""
    w = synth.CONFIGS["stale"]
    shift = np.zeros(w.n_seq)
    shift[[20, 21, 77]] = -2.0                                   # members of groups 2 and 9
    cases = [(f"sigma {s:g}", s, None) for s in synth.STALE_SIGMAS] + [("sigma 2 + overflow", 2.0, shift)]
    outs = _resident_batch_full_size(w, cases)
    for label, (o, st) in outs.items():
        assert np.all(o["adv64"][:w.group_size] == 0.0)          # the all-zero-reward group
        assert np.all(np.isfinite(o["coef"])) and np.isfinite(o["loss"])
    o0, st0 = outs["sigma 0"]
    assert st0["n_clipped"] == 0 and abs(st0["mean_log_cw"]) < 1e-3 and np.all(np.abs(o0["weight"] - 1.0) < 1e-3)
    o2, st2 = outs["sigma 2"]
    assert o2["weight"].max() > 3.4e38, "some weight should lie beyond the float32 range at sigma = 2"
    assert st2["n_clipped"] >= w.n_seq // 4
    oo, sto = outs["sigma 2 + overflow"]
    assert np.isinf(oo["weight"][[20, 21, 77]]).all() and sto["n_clipped"] == oo["stats"]["n_clipped"]


def test_long_config_full_size_chunked():
    """64 x 4096 tokens, V = 32000 fp32, 30 % trailing padding: 33.5 GB of logits, produced and
    consumed a block of generations at a time through the chunked three-step form."""
    w = synth.CONFIGS["long"]
    dt = torch.float32
    dev = torch.device("cuda")
    tok = synth.make_tokens(w)
    T, V, N, L = w.n_rows, w.vocab, w.n_seq, w.seq_len
    per = 4                                   # generations per chunk: 16 384 rows, 2.1 GB
    targets, mask = tok["targets"].to(dev), tok["mask"].to(dev)
    tg_np, mk_np = tok["targets"].numpy(), tok["mask"].numpy()
    desc = rb.make_desc(N, L, V, w.n_prompts, dt)
    ws = rb.alloc_workspace(desc, dev)
    buf = torch.empty((per * L, V), dtype=dt, device=dev)

    lse = np.zeros(T)
    lp = np.zeros(T)
    ok = np.zeros(T, np.uint8)
    for n0 in range(0, N, per):
        synth.logits_for_sequences(w, tok["targets"], n0, per, device=dev, out=buf)
        r0, nr = n0 * L, per * L
        rb.rapid_pg_stats_chunk(desc, buf, r0, nr, targets, mask, ws)
        pre = oracle.token_logp(synth.bits_numpy(buf), V, tg_np[r0:r0 + nr], mk_np[r0:r0 + nr])
        lse[r0:r0 + nr], lp[r0:r0 + nr], ok[r0:r0 + nr] = pre["lse"], pre["token_logp"], pre["row_ok"]
    behav = (torch.from_numpy(lp) + tok["behav_noise"].double()).float()
    o = _oracle_steps_2_to_5(w, tok, lp, ok, behav.numpy())

    loss = torch.zeros(1, device=dev)
    tl = torch.empty(T, device=dev)
    adv = torch.empty(N, device=dev)
    stats = rb.alloc_stats(dev)
    rb.rapid_pg_finalize(desc, behav.to(dev), tok["rewards"].to(dev), tok["group_offsets"].to(dev), loss,
                         tl, adv, stats, ws)
    torch.cuda.synchronize()
    np.testing.assert_allclose(tl.cpu().numpy(), lp, rtol=0, atol=LOGP_ATOL[dt])
    _check_scalars(o, loss.item(), adv.cpu().numpy(), rb.read_stats(stats), dt, L)
    assert np.all(o["adv64"][:w.group_size] == 0.0)

    rows_all = _sample_rows(w, tok, 6000, seed=w.seed)
    live_all = ok.astype(bool) & (np.repeat(o["coef"], L) != 0.0)
    worst = 0.0
    for n0 in range(0, N, per):
        synth.logits_for_sequences(w, tok["targets"], n0, per, device=dev, out=buf)
        r0, nr = n0 * L, per * L
        bits = synth.bits_numpy(buf)          # host copy before the in-place pass overwrites it
        rb.rapid_pg_dlogits_chunk(desc, buf, buf, r0, nr, targets, stats, ws)   # in place
        sel = rows_all[(rows_all >= r0) & (rows_all < r0 + nr)]
        if len(sel):
            ref = oracle.dlogits_rows(bits, V, L, tg_np, ok, lse, o["coef"], sel, row_base=r0)
            got = buf[torch.from_numpy(sel - r0).to(dev)].cpu().numpy().astype(np.float64)
            worst = max(worst, float(np.abs(got - ref).max()))
        _property_checks(buf, torch.from_numpy(live_all[r0:r0 + nr]).to(dev), dt)
    assert worst <= DLOGITS_ATOL[dt], f"dlogits max abs err {worst}"
    assert rb.read_stats(stats)["status"] == 0
    scale = max(abs(o["loss"]), 1e-3 * float(np.abs(o["coef"] * o["seq_logp"]).sum()), 1e-30)
    report_observed("long full size (chunked)", loss=abs(loss.item() - o["loss"]) / scale / LOSS_RTOL[dt],
                    token_logp=np.abs(tl.cpu().numpy() - lp).max() / LOGP_ATOL[dt],
                    adv=np.abs(adv.cpu().numpy() - o["adv64"]).max() / adv_atol(dt, L),
                    dlogits=worst / DLOGITS_ATOL[dt])
