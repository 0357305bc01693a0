"""The workspace-free entry point, rapid_pg_loss_fwd_bwd_noalloc.

Who needs it: code that is not allowed to allocate device memory -- a plug-in living inside an
application whose own pool owns the device, a loop whose memory budget is fully handed out before
it starts, a latency-critical step that must not risk the stall an allocation can cause.  Such a
caller cannot create the workspace that rapid_pg_loss_fwd_bwd asks for, so this variant keeps its
scratch in a fixed array inside the library instead.

What is checked: through the C ABI, on two calls in a row (the second on a different, smaller
problem, so that the shared array still holds the first call's leftovers), every output equals
what rapid_pg_loss_fwd_bwd gives with an ordinary workspace, within the tolerances used by the
parity tests; and a problem that does not fit the fixed array is refused with a clear status
before anything reaches the device.

This file sorts last on purpose: if it fails under `-x`, every other test has already run.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2510_03515_b200 import binding as rb
from paper_2510_03515_b200 import synth
from parity_util import DLOGITS_ATOL, LOGP_ATOL, LOSS_RTOL


def _inputs(w, dev):
    b = synth.make_batch(w)
    gen = torch.Generator().manual_seed(w.seed + 77)
    # behaviour log-probs only need to be plausible here: both entry points get the same array
    behav = (-6.0 + 0.5 * torch.randn(w.n_rows, generator=gen)).float()
    return {
        "logits": b["logits"].to(dev), "targets": b["targets"].to(dev), "mask": b["mask"].to(dev),
        "behav": behav.to(dev), "rewards": b["rewards"].to(dev),
        "group_offsets": b["group_offsets"].to(dev),
    }


def _outputs(w, dev):
    dt = synth.torch_dtype(w)
    return {
        "dlogits": torch.full((w.n_rows, w.vocab), float("nan"), dtype=dt, device=dev),
        "loss": torch.full((1,), float("nan"), device=dev),
        "token_logp": torch.full((w.n_rows,), float("nan"), device=dev),
        "adv": torch.full((w.n_seq,), float("nan"), device=dev),
        "stats": rb.alloc_stats(dev),
    }


def _run_pair(w, dev):
    """Same inputs through the workspace form and the workspace-free form; compare everything."""
    x = _inputs(w, dev)
    dt = synth.torch_dtype(w)
    desc = rb.make_desc(w.n_seq, w.seq_len, w.vocab, w.n_prompts, dt)
    assert rb.rapid_workspace_bytes(desc) <= rb.NOALLOC_SCRATCH_BYTES

    ref = _outputs(w, dev)
    ws = rb.alloc_workspace(desc, dev)
    rb.rapid_pg_loss_fwd_bwd(desc, x["logits"], x["targets"], x["mask"], x["behav"], x["rewards"],
                             x["group_offsets"], ref["dlogits"], ref["loss"], ref["token_logp"],
                             ref["adv"], ref["stats"], ws)
    got = _outputs(w, dev)
    rb.rapid_pg_loss_fwd_bwd_noalloc(desc, x["logits"], x["targets"], x["mask"], x["behav"],
                                     x["rewards"], x["group_offsets"], got["dlogits"], got["loss"],
                                     got["token_logp"], got["adv"], got["stats"])
    torch.cuda.synchronize()

    a, b = ref["loss"].item(), got["loss"].item()
    assert np.isfinite(a) and np.isfinite(b)
    assert abs(a - b) <= LOSS_RTOL[dt] * max(abs(a), 1e-30)
    err = (ref["dlogits"].float() - got["dlogits"].float()).abs().max().item()
    assert err <= DLOGITS_ATOL[dt], f"dlogits differ by {err}"
    assert torch.isfinite(got["dlogits"].float()).all()
    assert (ref["token_logp"] - got["token_logp"]).abs().max().item() <= LOGP_ATOL[dt]
    assert torch.equal(ref["adv"], got["adv"])
    sa, sb = rb.read_stats(ref["stats"]), rb.read_stats(got["stats"])
    assert sb["status"] == rb.RAPID_OK
    for k in ("n_tokens", "n_clipped", "n_bad_token", "n_empty_group"):
        assert sa[k] == sb[k]
    assert sb["n_tokens"] > 0 and got["dlogits"].float().abs().max().item() > 0


@pytest.mark.gpu
def test_noalloc_matches_workspace_form_on_two_calls_in_a_row():
    dev = torch.device("cuda")
    first = synth.Workload("noalloc-a", 3, 4, 24, 5000, "bf16", 3.0, 8.0, "uniform", len_lo=6,
                           behav_sigma=0.2, reward_mode="per_prompt", seed=41)
    second = synth.Workload("noalloc-b", 2, 3, 9, 1000, "f32", 2.0, 0.0, "uniform", len_lo=2,
                            behav_sigma=0.2, reward_mode="per_prompt", seed=42)
    _run_pair(first, dev)
    _run_pair(second, dev)   # the array now starts out holding the first call's state


def test_noalloc_refuses_what_does_not_fit():
    """Needs no GPU: the size check comes before the device is touched."""
    fake = 0x10000
    too_big = rb.make_desc(64, 4096, 32000, 4, torch.float32)      # 262 144 rows: ~5.5 MB of scratch
    assert rb.rapid_workspace_bytes(too_big) > rb.NOALLOC_SCRATCH_BYTES
    code = rb.lib().rapid_pg_loss_fwd_bwd_noalloc(C.byref(too_big), fake, fake, None, fake, fake, fake,
                                                 fake + (1 << 40), fake, None, None, None, None)
    assert code == rb.RAPID_ERR_UNSUPPORTED
    bad = rb.make_desc(0, 8, 64, 2, torch.float32)
    code = rb.lib().rapid_pg_loss_fwd_bwd_noalloc(C.byref(bad), fake, fake, None, fake, fake, fake,
                                                 fake + (1 << 40), fake, None, None, None, None)
    assert code == rb.RAPID_ERR_INVALID_ARG
