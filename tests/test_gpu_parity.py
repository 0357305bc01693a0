"""GPU parity: the CUDA library (through its C ABI) against the float64 CPU oracle on the same
seeded inputs, element by element, at sizes the oracle finishes in seconds."""
import math

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2510_03515_b200 import binding as rb  # noqa: E402
from paper_2510_03515_b200 import synth  # noqa: E402
from parity_util import compare, report_observed, run_both  # noqa: E402


def _dt(w):
    return synth.torch_dtype(w)


def test_config_tiny_full_size():
    """4 prompts x 8 samples, 64 tokens, V = 4096, fp32, seed 0: every element compared."""
    w = synth.CONFIGS["tiny"]
    b = synth.make_batch(w)
    o, g = run_both(b, w.n_seq, w.seq_len)
    r = compare(o, g, _dt(w), w.seq_len)
    assert np.abs(g["dlogits"].sum(1)).max() < 1e-6
    report_observed("tiny (every element)", loss=r["loss_vs_bound"], token_logp=r["logp_vs_bound"],
                    adv=r["adv_vs_bound"], dlogits=r["dlogits_vs_bound"])


@pytest.mark.parametrize("in_place", [False, True])
def test_config_slm_scaled(in_place):
    """SLM mini-batch shape at full vocabulary (151936, bf16, boosted sampled logit, ragged
    lengths with trailing padding), fewer and shorter generations so the oracle takes seconds."""
    w = synth.CONFIGS["slm"].scaled(n_prompts=2, group_size=4, seq_len=40, len_lo=10)
    b = synth.make_batch(w)
    o, g = run_both(b, w.n_seq, w.seq_len, in_place=in_place)
    r = compare(o, g, _dt(w), w.seq_len)
    assert (b["mask"] == 0).any()
    report_observed(f"slm scaled (every element, in_place={in_place})", loss=r["loss_vs_bound"],
                    token_logp=r["logp_vs_bound"], adv=r["adv_vs_bound"], dlogits=r["dlogits_vs_bound"])


@pytest.mark.parametrize("sigma", synth.STALE_SIGMAS)
def test_config_stale_scaled(sigma):
    """Staleness sweep: sigma in {0, .1, .5, 1, 2}; includes an all-zero and an all-one group."""
    w = synth.CONFIGS["stale"].scaled(n_prompts=4, group_size=4, seq_len=24, behav_sigma=sigma)
    b = synth.make_batch(w)
    o, g = run_both(b, w.n_seq, w.seq_len)
    compare(o, g, _dt(w), w.seq_len)
    assert np.all(o["adv64"][:4] == 0.0)  # all-zero rewards: no std division, exactly zero
    if sigma >= 1:
        assert o["n_clipped"] > 0


def test_config_long_scaled_chunked():
    """Long sequences, V = 32000 fp32, 30% trailing padding, through the chunked three-step API
    with a ragged last chunk; also equals the one-call form."""
    w = synth.CONFIGS["long"].scaled(n_prompts=2, group_size=4, seq_len=640)
    b = synth.make_batch(w)
    o, g = run_both(b, w.n_seq, w.seq_len)
    compare(o, g, _dt(w), w.seq_len)

    dev = torch.device("cuda")
    T, V = b["logits"].shape
    behav = torch.from_numpy(o["token_logp"]).double().add(b["behav_noise"].double()).float().to(dev)
    desc = rb.make_desc(w.n_seq, w.seq_len, V, w.n_prompts, torch.float32)
    ws = rb.alloc_workspace(desc, dev)
    tg, mk = b["targets"].to(dev), b["mask"].to(dev)
    chunk = 1500
    starts = list(range(0, T, chunk))
    for r0 in reversed(starts):  # any order
        n = min(chunk, T - r0)
        rb.rapid_pg_stats_chunk(desc, b["logits"][r0:r0 + n].to(dev), r0, n, tg, mk, ws)
    loss = torch.zeros(1, device=dev)
    tl = torch.zeros(T, device=dev)
    adv = torch.zeros(w.n_seq, device=dev)
    st = rb.alloc_stats(dev)
    rb.rapid_pg_finalize(desc, behav, b["rewards"].to(dev), b["group_offsets"].to(dev), loss, tl, adv, st, ws)
    dz = torch.empty((T, V), device=dev)
    for r0 in starts:
        n = min(chunk, T - r0)
        zc = b["logits"][r0:r0 + n].to(dev)
        rb.rapid_pg_dlogits_chunk(desc, zc, dz[r0:r0 + n], r0, n, tg, st, ws)
    torch.cuda.synchronize()
    g2 = {"loss": loss.item(), "token_logp": tl.cpu().numpy(), "adv": adv.cpu().numpy(),
          "stats": rb.read_stats(st), "dlogits": dz.cpu().numpy()}
    compare(o, g2, torch.float32, w.seq_len)
    # the chunked form and the one-call form run the same kernels on the same rows
    assert g2["loss"] == g["loss"]
    np.testing.assert_array_equal(g2["dlogits"], g["dlogits"])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,pad", [(1, 7), (2, 6), (7, 1), (8, 0), (9, 7), (255, 1), (257, 7),
                                   (1000, 0), (4099, 5), (33000, 0)])
def test_ragged_vocab_and_row_pitch(dtype, V, pad):
    """Vocabulary sizes around the vector width and the per-thread batch, with a padded pitch."""
    per = 4 if dtype == "f32" else 8
    pad = (-V) % per + (per if pad else 0)  # pitch must be a multiple of 16 bytes
    w = synth.Workload("edge", 2, 3, 5, V, dtype, 2.0, 3.0 if V > 1 else 0.0, "uniform", len_lo=0,
                       behav_sigma=0.3, reward_mode="per_prompt", seed=100 + V)
    b = synth.make_batch(w)
    o, g = run_both(b, w.n_seq, w.seq_len, ld_pad=pad)
    compare(o, g, _dt(w), w.seq_len)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, rb.FLAG_OUTER_UNCLIPPED, rb.FLAG_NORM_TOKENS,
                                   rb.FLAG_LEAVE_ONE_OUT, rb.FLAG_LEAVE_ONE_OUT | rb.FLAG_LOO_LITERAL_DIVISOR,
                                   rb.FLAG_OUTER_UNCLIPPED | rb.FLAG_NORM_TOKENS])
@pytest.mark.parametrize("eta", [2.0, math.inf, 0.5])
def test_flags_and_eta(dtype, flags, eta):
    w = synth.Workload("flags", 3, 4, 9, 515, dtype, 2.0, 4.0, "uniform", len_lo=1,
                       behav_sigma=0.25, reward_mode="per_prompt", seed=7)
    b = synth.make_batch(w)
    b["rewards"] = torch.randn(w.n_seq, generator=torch.Generator().manual_seed(3))  # real-valued rewards
    o, g = run_both(b, w.n_seq, w.seq_len, eta=eta, flags=flags)
    compare(o, g, _dt(w), w.seq_len)


def test_degenerate_shapes():
    """L = 1; groups of one; an empty group; a generation with no unmasked token; bad token ids."""
    V = 300
    N, L = 6, 1
    gen = torch.Generator().manual_seed(11)
    b = {
        "logits": torch.randn((N * L, V), generator=gen) * 2,
        "targets": torch.randint(0, V, (N * L,), generator=gen, dtype=torch.int64).to(torch.int32),
        "mask": torch.tensor([1, 1, 0, 1, 1, 1], dtype=torch.uint8),
        "rewards": torch.tensor([1.0, 0.0, 1.0, 1.0, 0.5, -2.0]),
        "group_offsets": torch.tensor([0, 1, 1, 3, 6], dtype=torch.int32),  # sizes 1, 0, 2, 3
        "behav_noise": torch.randn(N * L, generator=gen) * 0.5,
    }
    b["targets"][4] = V        # out of range: row counts as masked, is reported
    b["targets"][5] = -1
    o, g = run_both(b, N, L)
    compare(o, g, torch.float32, L)
    assert g["stats"]["n_bad_token"] == 2 and g["stats"]["n_empty_group"] == 1
    assert g["stats"]["n_tokens"] == 3


def test_everything_masked():
    w = synth.Workload("allmasked", 2, 2, 4, 64, "bf16", 1.0, 0.0, "full", seed=5)
    b = synth.make_batch(w)
    b["mask"] = torch.zeros_like(b["mask"])
    o, g = run_both(b, w.n_seq, w.seq_len)
    assert g["loss"] == 0.0 and np.all(g["dlogits"] == 0.0) and g["stats"]["n_tokens"] == 0
    compare(o, g, torch.bfloat16, w.seq_len)
    o, g = run_both(b, w.n_seq, w.seq_len, flags=rb.FLAG_NORM_TOKENS)  # Z = 0 tokens: still finite
    assert g["loss"] == 0.0 and np.all(g["dlogits"] == 0.0)


def test_mask_null_means_all_ones():
    w = synth.Workload("nomask", 2, 2, 6, 1024, "f32", 2.0, 0.0, "full", seed=6)
    b = synth.make_batch(w)
    del b["mask"]
    o, g = run_both(b, w.n_seq, w.seq_len)
    compare(o, g, torch.float32, w.seq_len)
    assert g["stats"]["n_tokens"] == w.n_rows


def test_invalid_group_offsets_reported_by_device():
    w = synth.Workload("badgroups", 2, 2, 3, 128, "f32", 1.0, 0.0, "full", seed=8)
    b = synth.make_batch(w)
    dev = torch.device("cuda")
    for bad in ([0, 3, 2, 4], [1, 2, 4], [0, 2, 5]):
        go = torch.tensor(bad, dtype=torch.int32, device=dev)
        z = b["logits"].to(dev)
        res = rb.pg_loss(z, b["targets"].to(dev), b["mask"].to(dev), torch.zeros(w.n_rows, device=dev),
                         b["rewards"].to(dev), go, w.n_seq, w.seq_len)
        torch.cuda.synchronize()
        st = rb.read_stats(res.stats)
        assert st["status"] == rb.RAPID_ERR_INVALID_ARG
        assert math.isnan(res.loss.item())
        assert torch.all(res.dlogits == 0)


# ---- rapid_group_advantage on its own: bit-exact ----------------------------------------------------

def _adv_gpu(R, slr, go, eta, flags):
    dev = torch.device("cuda")
    N, K = len(R), len(go) - 1
    desc = rb.RapidDesc(N, 1, 1, K, 1, rb.RAPID_F32, flags, eta)
    adv = torch.full((N,), float("nan"), device=dev)
    cw = torch.full((N,), float("nan"), dtype=torch.float64, device=dev)
    st = rb.alloc_stats(dev)
    rb.rapid_group_advantage(desc, torch.from_numpy(R).to(dev),
                             None if slr is None else torch.from_numpy(slr).to(dev),
                             torch.from_numpy(go).to(dev), adv, cw, st)
    torch.cuda.synchronize()
    return adv.cpu().numpy(), cw.cpu().numpy(), rb.read_stats(st)


@pytest.mark.parametrize("flags", [0, rb.FLAG_LEAVE_ONE_OUT, rb.FLAG_LEAVE_ONE_OUT | rb.FLAG_LOO_LITERAL_DIVISOR])
@pytest.mark.parametrize("eta", [2.0, math.inf])
def test_group_advantage_bit_exact(flags, eta):
    rng = np.random.default_rng(17)
    sizes = [8] * 16 + [1, 3, 16, 5, 2, 7] + [4] * 300
    go = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    N = int(go[-1])
    for R in ((rng.random(N) < 0.4).astype(np.float32), rng.normal(0, 1, N).astype(np.float32)):
        s = rng.normal(0, 1.0, N)
        # (a) identical weights on both sides: bit-exact by construction
        w = np.exp(s)
        ref = oracle.group_advantage(R, w, go, eta, flags | oracle.FLAG_ADV_INPUT_IS_WEIGHT)
        adv, cw, st = _adv_gpu(R, w, go, eta, flags | rb.FLAG_ADV_INPUT_IS_WEIGHT)
        assert np.array_equal(adv.view(np.uint32), ref["adv32"].view(np.uint32))
        assert np.array_equal(cw, ref["clipped_w"])
        assert st["n_clipped"] == int((w > eta).sum()) and st["status"] == 0
        assert st["mean_log_cw"] == pytest.approx(np.log(np.minimum(w, eta)).mean(), abs=1e-12)
        # (b) log-ratios in: exp() may differ in the last double bit between the two libraries;
        #     any float32 difference is then at most one ulp
        ref = oracle.group_advantage(R, s, go, eta, flags)
        adv, cw, st = _adv_gpu(R, s, go, eta, flags)
        ulp = np.abs(adv.view(np.int32).astype(np.int64) - ref["adv32"].view(np.int32).astype(np.int64))
        assert ulp.max() <= 1
        # (c) on-policy (Eq. 2): no weights at all, exact
        ref = oracle.group_advantage(R, None, go, eta, flags)
        adv, cw, st = _adv_gpu(R, None, go, eta, flags)
        assert np.array_equal(adv.view(np.uint32), ref["adv32"].view(np.uint32))
        assert st["n_clipped"] == 0 and st["mean_log_cw"] == 0.0


@pytest.mark.parametrize("flags", [0, rb.FLAG_LEAVE_ONE_OUT, rb.FLAG_LEAVE_ONE_OUT | rb.FLAG_LOO_LITERAL_DIVISOR])
@pytest.mark.parametrize("sizes", [[3000], [5, 0, 0, 2900, 0, 7, 1, 0]])
def test_group_advantage_groups_of_thousands(flags, sizes):
    """The single-path baseline (every generation in one group) with thousands of generations, and the
    same beside small and empty groups: the leave-one-out sums run one thread per member and find
    the member's group by bisection over offsets that repeat where a group is empty.  Bit-exact."""
    rng = np.random.default_rng(23)
    go = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    N = int(go[-1])
    R = rng.normal(0, 1, N).astype(np.float32)
    w = np.exp(rng.normal(0, 1.0, N))
    ref = oracle.group_advantage(R, w, go, 2.0, flags | oracle.FLAG_ADV_INPUT_IS_WEIGHT)
    adv, cw, st = _adv_gpu(R, w, go, 2.0, flags | rb.FLAG_ADV_INPUT_IS_WEIGHT)
    assert np.array_equal(adv.view(np.uint32), ref["adv32"].view(np.uint32))
    assert np.array_equal(cw, ref["clipped_w"]) and st["status"] == 0
    assert st["n_empty_group"] == sizes.count(0)
    ref = oracle.group_advantage(R, None, go, 2.0, flags)
    adv, _, _ = _adv_gpu(R, None, go, 2.0, flags)
    assert np.array_equal(adv.view(np.uint32), ref["adv32"].view(np.uint32))


def test_group_advantage_zero_sum_on_device():
    """Eq. 2 advantages sum to zero within each group (checked on the device's own output)."""
    rng = np.random.default_rng(19)
    go = (np.arange(65) * 8).astype(np.int32)
    R = (rng.random(512) < 0.3).astype(np.float32)
    adv, _, _ = _adv_gpu(R, None, go, 2.0, 0)
    assert np.abs(adv.reshape(64, 8).astype(np.float64).sum(1)).max() < 1e-6


# ---- one mini-batch spread over ranks by whole prompt groups -------------------------------------------

@pytest.mark.parametrize("flags", [0, rb.FLAG_NORM_TOKENS])
def test_shards_with_given_normaliser_add_up_to_the_whole_batch(flags):
    """Three 'ranks' (run one after another on this GPU; their kernels do not depend on each other)
    each take whole groups and pass the global Z with RAPID_FLAG_NORM_GIVEN: losses add up to the
    oracle's loss on the whole mini-batch and every dlogits row equals the oracle's."""
    from paper_2510_03515_b200 import shard
    w = synth.Workload("shards", 5, 3, 11, 1000, "bf16", 3.0, 6.0, "uniform", len_lo=3, behav_sigma=0.3,
                       reward_mode="per_prompt", seed=29)
    b = synth.make_batch(w)
    L, V, N = w.seq_len, w.vocab, w.n_seq
    bits = synth.bits_numpy(b["logits"])
    pre = oracle.token_logp(bits, V, b["targets"].numpy(), b["mask"].numpy())
    behav = (torch.from_numpy(pre["token_logp"]) + b["behav_noise"].double()).float()
    full = oracle.pg_loss(bits, N, L, V, b["targets"].numpy(), b["mask"].numpy(), behav.numpy(),
                          b["rewards"].numpy(), b["group_offsets"].numpy(), 2.0, flags, want_dlogits=True)
    z_global = float(full["n_tokens"]) if flags & rb.FLAG_NORM_TOKENS else float(N)
    dev = torch.device("cuda")
    world, loss_sum, tok_sum = 3, 0.0, 0
    for rank in range(world):
        sh = shard.plan(b["group_offsets"].numpy(), b["lengths"].numpy(), world, rank)
        rows = torch.from_numpy((sh.seq_index[:, None] * L + np.arange(L)[None, :]).reshape(-1))
        res = rb.pg_loss(b["logits"][rows].contiguous().to(dev), b["targets"][rows].to(dev), b["mask"][rows].to(dev),
                         behav[rows].to(dev), b["rewards"][torch.from_numpy(sh.seq_index)].to(dev),
                         torch.from_numpy(sh.group_offsets).to(dev), sh.n_seq, L,
                         flags=flags | rb.FLAG_NORM_GIVEN, norm_z=z_global)
        torch.cuda.synchronize()
        st = rb.read_stats(res.stats)
        assert st["status"] == 0
        loss_sum += st["loss"]
        tok_sum += st["n_tokens"]
        err = np.abs(res.dlogits.float().cpu().numpy() - full["dlogits"][rows.numpy()]).max()
        assert err <= 4e-3
        np.testing.assert_allclose(res.adv.cpu().numpy(), full["adv64"][sh.seq_index], rtol=0, atol=2e-4)
    scale = max(abs(full["loss"]), 1e-3 * float(np.abs(full["coef"] * full["seq_logp"]).sum()))
    assert abs(loss_sum - full["loss"]) / scale <= 2e-3
    assert tok_sum == full["n_tokens"]


def test_single_path_baseline_is_one_group():
    """The single-path baseline of Sec. 3.3 (A = R - batch-mean reward) is the one-group case of the
    group advantage: all N generations in one group."""
    w = synth.Workload("onegroup", 1, 6, 7, 520, "bf16", 2.0, 4.0, "uniform", len_lo=2, behav_sigma=0.0,
                       reward_mode="per_prompt", seed=13)
    b = synth.make_batch(w)
    b["rewards"] = torch.tensor([1.0, 0.0, 0.0, 1.0, 1.0, 0.0])
    o, g = run_both(b, w.n_seq, w.seq_len)
    compare(o, g, _dt(w), w.seq_len)
    # sigma = 0: weights are 1 up to float32 rounding of the stored behaviour log-probs
    np.testing.assert_allclose(g["adv"], b["rewards"].numpy() - 0.5, atol=1e-5)


def test_runs_on_the_callers_stream():
    """Work is enqueued on the stream handed over (here torch's current, non-default stream) and is
    ordered after that stream's earlier work: the logits are produced on the same stream just before."""
    w = synth.Workload("stream", 2, 3, 6, 2048, "bf16", 2.0, 3.0, "uniform", len_lo=2, behav_sigma=0.2,
                       reward_mode="per_prompt", seed=37)
    b = synth.make_batch(w)
    dev = torch.device("cuda")
    ref = rb.pg_loss(b["logits"].to(dev), b["targets"].to(dev), b["mask"].to(dev), torch.full((w.n_rows,), -7.0, device=dev),
                     b["rewards"].to(dev), b["group_offsets"].to(dev), w.n_seq, w.seq_len)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    staged = b["logits"].to(dev)
    tg, mk, rw, go = b["targets"].to(dev), b["mask"].to(dev), b["rewards"].to(dev), b["group_offsets"].to(dev)
    bh = torch.full((w.n_rows,), -7.0, device=dev)
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        z = torch.empty_like(staged)
        for _ in range(20):                  # keep the stream busy, then produce the input on it
            z.copy_(staged * 0.5)
        z.copy_(staged)
        got = rb.pg_loss(z, tg, mk, bh, rw, go, w.n_seq, w.seq_len)
    side.synchronize()
    assert got.loss.item() == ref.loss.item()
    assert torch.equal(got.dlogits, ref.dlogits)


def test_many_small_generations():
    """5000 generations in 1250 groups: the per-generation and per-group steps loop well past one CTA."""
    N, L, V = 5000, 2, 64
    gen = torch.Generator().manual_seed(3)
    b = {"logits": torch.randn((N * L, V), generator=gen),
         "targets": torch.randint(0, V, (N * L,), generator=gen, dtype=torch.int64).to(torch.int32),
         "mask": (torch.rand(N * L, generator=gen) < 0.8).to(torch.uint8),
         "rewards": (torch.rand(N, generator=gen) < 0.5).float(),
         "group_offsets": (torch.arange(1251) * 4).to(torch.int32),
         "behav_noise": torch.randn(N * L, generator=gen) * 0.3}
    o, g = run_both(b, N, L)
    compare(o, g, torch.float32, L)


@pytest.mark.parametrize("form", ["two_pass", "on_policy"])
def test_masked_rows_are_never_read(form):
    """Masked rows may hold anything (here NaN): outputs are bit-identical to a clean run."""
    w = synth.Workload("nanmask", 2, 3, 8, 4096, "bf16", 2.0, 3.0, "uniform", len_lo=2, behav_sigma=0.2,
                       reward_mode="per_prompt", seed=43)
    b = synth.make_batch(w)
    dev = torch.device("cuda")
    poisoned = b["logits"].clone()
    poisoned[b["mask"] == 0] = float("nan")
    bh = torch.full((w.n_rows,), -7.0, device=dev)
    outs = []
    for z in (b["logits"], poisoned):
        if form == "two_pass":
            r = rb.pg_loss(z.to(dev), b["targets"].to(dev), b["mask"].to(dev), bh, b["rewards"].to(dev),
                           b["group_offsets"].to(dev), w.n_seq, w.seq_len)
            outs.append((r.loss.item(), r.dlogits.clone()))
        else:
            desc = rb.make_desc(w.n_seq, w.seq_len, w.vocab, w.n_prompts, torch.bfloat16)
            ws = rb.alloc_workspace(desc, dev)
            loss = torch.zeros(1, device=dev)
            dz = torch.empty((w.n_rows, w.vocab), dtype=torch.bfloat16, device=dev)
            tl = torch.empty(w.n_rows, device=dev)
            rb.rapid_pg_loss_onpolicy_fwd_bwd(desc, z.to(dev), b["targets"].to(dev), b["mask"].to(dev),
                                              b["rewards"].to(dev), b["group_offsets"].to(dev), dz, loss, tl, None,
                                              None, ws)
            outs.append((loss.item(), dz.clone()))
        torch.cuda.synchronize()
    assert outs[0][0] == outs[1][0] and torch.equal(outs[0][1], outs[1][1])
    assert torch.isfinite(outs[1][1].float()).all()


def test_two_pass_call_can_be_captured_in_a_cuda_graph():
    """The library keeps no state and only enqueues kernels, so one rapid_pg_loss_fwd_bwd call can be
    captured once and replayed (useful for small, launch-bound mini-batches): replays on fresh inputs
    give the same bits as a direct call."""
    w = synth.CONFIGS["tiny"]
    b = synth.make_batch(w)
    dev = torch.device("cuda")
    z = b["logits"].to(dev)
    tg, mk, rw, go = b["targets"].to(dev), b["mask"].to(dev), b["rewards"].to(dev), b["group_offsets"].to(dev)
    bh = torch.full((w.n_rows,), -8.5, device=dev)
    desc = rb.make_desc(w.n_seq, w.seq_len, w.vocab, w.n_prompts, torch.float32)
    ws = rb.alloc_workspace(desc, dev)
    out = {k: torch.zeros(s, device=dev) for k, s in (("loss", 1), ("tl", w.n_rows), ("adv", w.n_seq))}
    dz = torch.zeros_like(z)
    st = rb.alloc_stats(dev)

    def call():
        rb.rapid_pg_loss_fwd_bwd(desc, z, tg, mk, bh, rw, go, dz, out["loss"], out["tl"], out["adv"], st, ws)

    call()                                   # warm-up outside capture (sets kernel attributes)
    torch.cuda.synchronize()
    direct = (out["loss"].item(), dz.clone())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    for scale in (1.0, 0.5):
        z.copy_(b["logits"].to(dev) * scale)
        dz.zero_()
        graph.replay()
        torch.cuda.synchronize()
        if scale == 1.0:
            assert out["loss"].item() == direct[0] and torch.equal(dz, direct[1])
        else:
            call_loss = out["loss"].item()
            ref = rb.pg_loss(z, tg, mk, bh, rw, go, w.n_seq, w.seq_len)
            torch.cuda.synchronize()
            assert call_loss == ref.loss.item() and torch.equal(dz, ref.dlogits)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_logits_read_from_pinned_host_memory(dtype):
    """The host-logits form gives the same bits as copying the logits over first; rows that are
    masked never reach the staging buffer; pointers that are not page-locked host memory are refused
    before anything runs."""
    import ctypes as C
    w = synth.Workload("hostz", 2, 3, 9, 4100 if dtype == "f32" else 4104, dtype, 2.0, 3.0, "uniform", len_lo=3,
                       behav_sigma=0.2, reward_mode="per_prompt", seed=47)
    b = synth.make_batch(w)
    dev = torch.device("cuda")
    dt = synth.torch_dtype(w)
    tg, mk, rw, go = b["targets"].to(dev), b["mask"].to(dev), b["rewards"].to(dev), b["group_offsets"].to(dev)
    bh = torch.full((w.n_rows,), -7.5, device=dev)
    ref = rb.pg_loss(b["logits"].to(dev), tg, mk, bh, rw, go, w.n_seq, w.seq_len)
    torch.cuda.synchronize()

    pinned = b["logits"].clone().pin_memory()
    staging = torch.full_like(b["logits"], 7.0, device=dev)
    desc = rb.make_desc(w.n_seq, w.seq_len, w.vocab, w.n_prompts, dt)
    ws = rb.alloc_workspace(desc, dev)
    loss = torch.zeros(1, device=dev)
    dz = torch.empty_like(staging)
    tl = torch.empty(w.n_rows, device=dev)
    adv = torch.empty(w.n_seq, device=dev)
    st = rb.alloc_stats(dev)
    rb.rapid_pg_loss_fwd_bwd_hostlogits(desc, pinned, staging, tg, mk, bh, rw, go, dz, loss, tl, adv, st, ws)
    torch.cuda.synchronize()
    assert loss.item() == ref.loss.item() and torch.equal(dz, ref.dlogits) and torch.equal(tl, ref.token_logp)
    on = b["mask"].bool()
    assert torch.equal(staging[on.to(dev)].cpu(), b["logits"][on])          # what was read is what was staged
    assert torch.all(staging[(~on).to(dev)] == 7.0)                          # masked rows never came over
    assert rb.read_stats(st)["status"] == 0

    L = rb.lib()
    args = lambda z: (C.byref(desc), z, staging.data_ptr(), tg.data_ptr(), mk.data_ptr(), bh.data_ptr(), rw.data_ptr(),
                      go.data_ptr(), dz.data_ptr(), loss.data_ptr(), None, None, None, ws.data_ptr(), ws.numel(), None)
    pageable = b["logits"].clone()
    assert L.rapid_pg_loss_fwd_bwd_hostlogits(*args(pageable.data_ptr())) == rb.RAPID_ERR_INVALID_ARG
    assert L.rapid_pg_loss_fwd_bwd_hostlogits(*args(staging.data_ptr())) == rb.RAPID_ERR_INVALID_ARG
    torch.cuda.synchronize()


def _with_minus_infinity(b, V, fill="-inf"):
    """Masks parts of the vocabulary with -inf, never the sampled token: a padded tail on every row
    (as a model whose vocabulary is padded to a round size produces), the whole first 9000 columns of
    every third row (every thread's first loads see nothing but -inf there), and a scattered 30 % of
    every fifth row."""
    z = b["logits"]
    T = z.shape[0]
    ninf = torch.zeros(z.shape, dtype=torch.bool)
    ninf[:, V - 613:] = True
    ninf[0::3, :9000] = True
    g = torch.Generator().manual_seed(1234)
    ninf[1::5] |= torch.rand((len(range(1, T, 5)), V), generator=g) < 0.3
    ninf[torch.arange(T), b["targets"].long().clamp(0, V - 1)] = False
    # "lowest": the most negative finite value of the dtype, which some pipelines use as their mask value
    z[ninf] = float("-inf") if fill == "-inf" else torch.finfo(z.dtype).min
    return ninf


@pytest.mark.parametrize("fill", ["-inf", "lowest"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_minus_infinity_logits(dtype, fill):
    """-inf logits (a masked part of the vocabulary) contribute exp(-inf) = 0 to every sum and get a zero
    gradient; long runs of them at the start of a row must not poison the running maximum."""
    V = 20000 + (4 if dtype == "f32" else 0)
    w = synth.Workload("ninf", 2, 3, 7, V, dtype, 2.0, 4.0, "uniform", len_lo=3, behav_sigma=0.3,
                       reward_mode="per_prompt", seed=811)
    b = synth.make_batch(w)
    b["rewards"] = torch.randn(w.n_seq, generator=torch.Generator().manual_seed(3))
    ninf = _with_minus_infinity(b, V, fill)
    o, g = run_both(b, w.n_seq, w.seq_len)
    compare(o, g, _dt(w), w.seq_len)
    assert np.isfinite(g["dlogits"]).all() and np.isfinite(g["token_logp"]).all()
    assert np.all(g["dlogits"][ninf.numpy()] == 0.0)
