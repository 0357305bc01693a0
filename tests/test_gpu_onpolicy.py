"""GPU parity of the single-pass on-policy form (Eq. 1 with the Eq. 2 group advantage) against the
float64 oracle.  The oracle side is its own steps with every weight set to one: step 1 (token
log-probs), step 2 (per-generation sums), Eq. 2 advantages (no log-ratios), step 5 with
w = c = 1, step 6."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2510_03515_b200 import binding as rb  # noqa: E402
from paper_2510_03515_b200 import synth  # noqa: E402
from parity_util import ADV_ATOL, DLOGITS_ATOL, LOGP_ATOL, LOSS_RTOL  # noqa: E402


def oracle_onpolicy(b, N, L, V, flags=0, want_dlogits=True, bits=None):
    bits = synth.bits_numpy(b["logits"]) if bits is None else bits
    mask = b.get("mask")
    mk = None if mask is None else mask.numpy()
    pre = oracle.token_logp(bits, V, b["targets"].numpy(), mk)
    s, S, cnt = oracle.seq_reduce(N, L, pre["token_logp"], np.zeros(N * L, np.float32), pre["row_ok"])
    ga = oracle.group_advantage(b["rewards"].numpy(), None, b["group_offsets"].numpy(), 2.0, flags)
    ones = np.ones(N)
    loss, coef, st = oracle.coef_loss(np.zeros(N), S, cnt, ones, ones, ga["adv64"], 2.0, flags)
    o = {"loss": loss, "coef": coef, "seq_logp": S, "adv64": ga["adv64"], "token_logp": pre["token_logp"],
         "row_ok": pre["row_ok"], "lse": pre["lse"], "n_tokens": st["n_tokens"], "n_bad_token": pre["n_bad_token"]}
    if want_dlogits:
        rows = np.arange(N * L, dtype=np.int64)
        o["dlogits"] = oracle.dlogits_rows(bits, V, L, b["targets"].numpy(), pre["row_ok"], pre["lse"], coef, rows)
    return o


def run_gpu(b, N, L, flags=0, in_place=False, want_logp=True, ld_pad=0):
    logits = b["logits"]
    T, V = logits.shape
    dev = torch.device("cuda")
    G = 2
    ld = V + ld_pad
    zbuf = torch.full((T + 2 * G, ld), 55.0, dtype=logits.dtype, device=dev)
    zbuf[G:G + T, :V].copy_(logits)
    z = zbuf[G:G + T]
    if in_place:
        dbuf, dz = zbuf, z
    else:
        dbuf = torch.full((T + 2 * G, ld), 33.0, dtype=logits.dtype, device=dev)
        dz = dbuf[G:G + T]
    mask = b.get("mask")
    desc = rb.make_desc(N, L, V, b["group_offsets"].numel() - 1, logits.dtype, ld, 2.0, flags)
    ws = rb.alloc_workspace(desc, dev)
    loss = torch.full((1,), float("nan"), device=dev)
    tl = torch.full((T,), float("nan"), device=dev) if want_logp else None
    adv = torch.full((N,), float("nan"), device=dev)
    stats = rb.alloc_stats(dev)
    rb.rapid_pg_loss_onpolicy_fwd_bwd(desc, z, b["targets"].to(dev), None if mask is None else mask.to(dev),
                                      b["rewards"].to(dev), b["group_offsets"].to(dev), dz, loss, tl, adv, stats, ws)
    torch.cuda.synchronize()
    guard = 55.0 if in_place else 33.0
    assert torch.all(dbuf[:G] == guard) and torch.all(dbuf[G + T:] == guard), "guard rows overwritten"
    if ld_pad:
        assert torch.all(dz[:, V:] == (55.0 if in_place else 33.0)), "columns >= vocab overwritten"
    return {"loss": loss.item(), "token_logp": None if tl is None else tl.cpu().numpy(), "adv": adv.cpu().numpy(),
            "stats": rb.read_stats(stats), "dlogits": dz[:, :V].float().cpu().numpy().astype(np.float64)}


def compare(o, g, dt, L, want_logp=True):
    ok = o["row_ok"].astype(bool)
    live = ok & (np.repeat(o["coef"], L) != 0.0)
    if want_logp:
        np.testing.assert_allclose(g["token_logp"], o["token_logp"], rtol=0, atol=LOGP_ATOL[dt])
    np.testing.assert_allclose(g["adv"], o["adv64"], rtol=0, atol=ADV_ATOL[dt])
    scale = max(abs(o["loss"]), 1e-3 * float(np.abs(o["coef"] * o["seq_logp"]).sum()), 1e-30)
    assert abs(g["loss"] - o["loss"]) / scale <= LOSS_RTOL[dt] + 6e-8 * abs(o["loss"]) / scale
    st = g["stats"]
    assert st["status"] == 0 and st["n_tokens"] == o["n_tokens"] and st["n_bad_token"] == o["n_bad_token"]
    assert st["n_clipped"] == 0 and st["mean_log_cw"] == 0.0
    err = np.abs(g["dlogits"] - o["dlogits"]).max()
    assert err <= DLOGITS_ATOL[dt], f"dlogits max abs err {err}"
    assert np.all(g["dlogits"][~live] == 0.0)


def test_tiny_config_full_size():
    w = synth.CONFIGS["tiny"]
    b = synth.make_batch(w)
    o = oracle_onpolicy(b, w.n_seq, w.seq_len, w.vocab)
    compare(o, run_gpu(b, w.n_seq, w.seq_len), torch.float32, w.seq_len)


@pytest.mark.parametrize("in_place", [False, True])
@pytest.mark.parametrize("want_logp", [True, False])
def test_slm_scaled(in_place, want_logp):
    """Full vocabulary, bf16, ragged lengths; one prompt's generations all get reward 0, so its
    rows have no gradient (read only when token log-probs are asked for)."""
    w = synth.CONFIGS["slm"].scaled(n_prompts=3, group_size=4, seq_len=36, len_lo=9, reward_mode="per_prompt_const")
    b = synth.make_batch(w)
    o = oracle_onpolicy(b, w.n_seq, w.seq_len, w.vocab)
    g = run_gpu(b, w.n_seq, w.seq_len, in_place=in_place, want_logp=want_logp)
    compare(o, g, torch.bfloat16, w.seq_len, want_logp)
    assert np.all(o["coef"][:8] == 0.0) and np.any(o["coef"] != 0.0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,pad", [(1, 7), (7, 1), (8, 0), (9, 7), (257, 7), (1000, 0), (4099, 5), (8200, 0), (33000, 8)])
def test_ragged_vocab_and_row_pitch(dtype, V, pad):
    per = 4 if dtype == "f32" else 8
    pad = (-V) % per + (per if pad else 0)
    w = synth.Workload("edge", 2, 3, 5, V, dtype, 2.0, 3.0 if V > 1 else 0.0, "uniform", len_lo=0,
                       behav_sigma=0.3, reward_mode="per_prompt", seed=200 + V)
    b = synth.make_batch(w)
    b["rewards"] = torch.randn(w.n_seq, generator=torch.Generator().manual_seed(V))
    o = oracle_onpolicy(b, w.n_seq, w.seq_len, V)
    compare(o, run_gpu(b, w.n_seq, w.seq_len, ld_pad=pad), synth.torch_dtype(w), w.seq_len)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, rb.FLAG_NORM_TOKENS, rb.FLAG_LEAVE_ONE_OUT,
                                   rb.FLAG_LEAVE_ONE_OUT | rb.FLAG_LOO_LITERAL_DIVISOR])
def test_flags(dtype, flags):
    w = synth.Workload("flags", 3, 4, 9, 515 if dtype == "f32" else 520, dtype, 2.0, 4.0, "uniform", len_lo=1,
                       behav_sigma=0.25, reward_mode="per_prompt", seed=7)
    b = synth.make_batch(w)
    b["rewards"] = torch.randn(w.n_seq, generator=torch.Generator().manual_seed(3))
    V = w.vocab
    pad = (-V) % (4 if dtype == "f32" else 8)
    o = oracle_onpolicy(b, w.n_seq, w.seq_len, V, flags)
    compare(o, run_gpu(b, w.n_seq, w.seq_len, flags=flags, ld_pad=pad), synth.torch_dtype(w), w.seq_len)


def test_degenerate_shapes_and_bad_groups():
    V, N, L = 300, 6, 1
    gen = torch.Generator().manual_seed(11)
    b = {"logits": torch.randn((N * L, V), generator=gen) * 2,
         "targets": torch.randint(0, V, (N * L,), generator=gen, dtype=torch.int64).to(torch.int32),
         "mask": torch.tensor([1, 1, 0, 1, 1, 1], dtype=torch.uint8),
         "rewards": torch.tensor([1.0, 0.0, 1.0, 1.0, 0.5, -2.0]),
         "group_offsets": torch.tensor([0, 1, 1, 3, 6], dtype=torch.int32)}
    b["targets"][4] = V
    b["targets"][5] = -1
    o = oracle_onpolicy(b, N, L, V)
    g = run_gpu(b, N, L)
    compare(o, g, torch.float32, L)
    assert g["stats"]["n_bad_token"] == 2 and g["stats"]["n_empty_group"] == 1
    b["group_offsets"] = torch.tensor([0, 3, 2, 6, 6], dtype=torch.int32)
    g = run_gpu(b, N, L)
    assert g["stats"]["status"] == rb.RAPID_ERR_INVALID_ARG and np.isnan(g["loss"]) and np.all(g["dlogits"] == 0)


def test_equals_two_pass_path_when_behaviour_equals_current():
    """The special case that ties the two forms together: feed the two-pass path behaviour
    log-probs equal to the current ones (as float32); weights are 1 up to that rounding."""
    w = synth.CONFIGS["slm"].scaled(n_prompts=2, group_size=4, seq_len=20, len_lo=5, vocab=4096)
    b = synth.make_batch(w)
    g1 = run_gpu(b, w.n_seq, w.seq_len)
    dev = torch.device("cuda")
    res = rb.pg_loss(b["logits"].to(dev), b["targets"].to(dev), b["mask"].to(dev),
                     torch.from_numpy(g1["token_logp"]).to(dev), b["rewards"].to(dev), b["group_offsets"].to(dev),
                     w.n_seq, w.seq_len)
    torch.cuda.synchronize()
    assert abs(res.loss.item() - g1["loss"]) <= 2e-3 * max(abs(g1["loss"]), 1e-6)   # two bf16-class kernels
    assert np.abs(res.dlogits.float().cpu().numpy() - g1["dlogits"]).max() <= 4e-3


def test_slm_config_full_size():
    """The benchmark's mini-batch (64 x 1024 x 151936 bf16) through the single-pass form: steps 1-5
    against the oracle on every row, dlogits on sampled rows plus whole-batch properties."""
    w = synth.CONFIGS["slm"]
    dt, dev = torch.bfloat16, torch.device("cuda")
    tok = synth.make_tokens(w)
    T, V, N, L = w.n_rows, w.vocab, w.n_seq, w.seq_len
    logits = synth.logits_for_sequences(w, tok["targets"], 0, N, device=dev)
    bits = synth.bits_numpy(logits)
    b = dict(tok)
    o = oracle_onpolicy(b, N, L, V, want_dlogits=False, bits=bits)
    desc = rb.make_desc(N, L, V, w.n_prompts, dt)
    ws = rb.alloc_workspace(desc, dev)
    loss = torch.zeros(1, device=dev)
    tl = torch.empty(T, device=dev)
    adv = torch.empty(N, device=dev)
    stats = rb.alloc_stats(dev)
    rb.rapid_pg_loss_onpolicy_fwd_bwd(desc, logits, tok["targets"].to(dev), tok["mask"].to(dev), tok["rewards"].to(dev),
                                      tok["group_offsets"].to(dev), logits, loss, tl, adv, stats, ws)   # in place
    torch.cuda.synchronize()
    np.testing.assert_allclose(tl.cpu().numpy(), o["token_logp"], rtol=0, atol=LOGP_ATOL[dt])
    np.testing.assert_allclose(adv.cpu().numpy(), o["adv64"], rtol=0, atol=ADV_ATOL[dt])
    scale = max(abs(o["loss"]), 1e-3 * float(np.abs(o["coef"] * o["seq_logp"]).sum()))
    assert abs(loss.item() - o["loss"]) / scale <= LOSS_RTOL[dt]
    st = rb.read_stats(stats)
    assert st["status"] == 0 and st["n_tokens"] == o["n_tokens"]
    rows = np.unique(np.random.default_rng(5).integers(0, T, 2000))
    worst = 0.0
    for i in range(0, len(rows), 256):
        sel = rows[i:i + 256]
        ref = oracle.dlogits_rows(bits, V, L, tok["targets"].numpy(), o["row_ok"], o["lse"], o["coef"], sel)
        got = logits[torch.from_numpy(sel).to(dev)].float().cpu().numpy().astype(np.float64)
        worst = max(worst, float(np.abs(got - ref).max()))
    assert worst <= DLOGITS_ATOL[dt], worst
    live = torch.from_numpy(o["row_ok"].astype(bool) & (np.repeat(o["coef"], L) != 0.0)).to(dev)
    for r0 in range(0, T, 4096):
        blk = logits[r0:r0 + 4096].float()
        assert torch.isfinite(blk).all() and (blk[~live[r0:r0 + 4096]] == 0).all()
        assert blk.sum(1).abs().max().item() <= 1e-3


@pytest.mark.parametrize("fill", ["-inf", "lowest"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_minus_infinity_logits(dtype, fill):
    """-inf logits (a masked part of the vocabulary): a padded tail on every row, the whole first 9000
    columns of every third row, a scattered 30 % of every fifth row; never the sampled token."""
    V = 20000 + (4 if dtype == "f32" else 0)
    w = synth.Workload("ninf", 2, 3, 7, V, dtype, 2.0, 4.0, "uniform", len_lo=3, behav_sigma=0.3,
                       reward_mode="per_prompt", seed=812)
    b = synth.make_batch(w)
    b["rewards"] = torch.randn(w.n_seq, generator=torch.Generator().manual_seed(3))
    z = b["logits"]
    T = z.shape[0]
    ninf = torch.zeros(z.shape, dtype=torch.bool)
    ninf[:, V - 613:] = True
    ninf[0::3, :9000] = True
    ninf[1::5] |= torch.rand((len(range(1, T, 5)), V), generator=torch.Generator().manual_seed(77)) < 0.3
    ninf[torch.arange(T), b["targets"].long().clamp(0, V - 1)] = False
    z[ninf] = float("-inf") if fill == "-inf" else torch.finfo(z.dtype).min
    o = oracle_onpolicy(b, w.n_seq, w.seq_len, V)
    g = run_gpu(b, w.n_seq, w.seq_len)
    compare(o, g, torch.float32 if dtype == "f32" else torch.bfloat16, w.seq_len)
    assert np.isfinite(g["dlogits"]).all() and np.isfinite(g["token_logp"]).all()
    assert np.all(g["dlogits"][ninf.numpy()] == 0.0)
