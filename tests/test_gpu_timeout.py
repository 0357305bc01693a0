"""The time-out path of the pipelined kernels, exercised without breaking anything: the library's
bounded barrier wait is run on a barrier that nothing arrives at and must give up after its limit,
report RAPID_ERR_TIMEOUT through the statistics block and leave the context usable."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2510_03515_b200 import binding as rb  # noqa: E402
from paper_2510_03515_b200 import synth  # noqa: E402


@pytest.mark.parametrize("limit_ms", [2, 20])
def test_a_wait_that_nothing_satisfies_gives_up_and_reports_it(limit_ms):
    dev = torch.device("cuda")
    st = rb.alloc_stats(dev)
    rb.rapid_selftest_bounded_wait(limit_ms * 1_000_000, st)
    torch.cuda.synchronize()                       # returns: the kernel ended by itself
    s = rb.read_stats(st)
    assert s["status"] == rb.RAPID_ERR_TIMEOUT
    waited_ms = s["n_tokens"] / 1e6
    assert limit_ms <= waited_ms <= limit_ms + 25, waited_ms

    # the context is still good: an ordinary call right after it works and reports no error
    w = synth.CONFIGS["tiny"].scaled(n_prompts=2, group_size=2, seq_len=4, vocab=512)
    b = synth.make_batch(w)
    res = rb.pg_loss(b["logits"].to(dev), b["targets"].to(dev), b["mask"].to(dev),
                     torch.full((w.n_rows,), -6.0, device=dev), b["rewards"].to(dev), b["group_offsets"].to(dev),
                     w.n_seq, w.seq_len)
    torch.cuda.synchronize()
    assert rb.read_stats(res.stats)["status"] == 0 and np.isfinite(res.loss.item())
