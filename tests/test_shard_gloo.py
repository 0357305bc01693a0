"""The multi-GPU sharding logic, run as two gloo ranks on the CPU.  Each rank takes its whole
prompt groups of one seeded mini-batch; the per-rank compute is stood in for by the float64 oracle
(there is no GPU here), with the loss rescaled from the rank's own N to the global N exactly as
RAPID_FLAG_NORM_GIVEN makes the library do; the reduced result must equal the oracle's on the
whole mini-batch."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_03515_b200 import shard, synth


def test_partition_is_balanced_and_complete():
    tokens = [900, 100, 500, 500, 300, 700, 50, 950]
    parts = shard.partition_groups(tokens, 3)
    assert sorted(sum(parts, [])) == list(range(8))
    loads = [sum(tokens[k] for k in p) for p in parts]
    assert max(loads) - min(loads) <= max(tokens)
    assert shard.partition_groups(tokens, 3) == parts                       # deterministic
    assert shard.partition_groups([5, 5], 4) == [[0], [1], [], []]         # more ranks than groups
    with pytest.raises(ValueError):
        shard.partition_groups(tokens, 0)


def test_plan_local_offsets():
    go = [0, 2, 5, 6, 10]                      # group sizes 2, 3, 1, 4
    tps = [10, 10, 1, 1, 1, 50, 2, 2, 2, 2]
    a = shard.plan(go, tps, 2, 0)
    b = shard.plan(go, tps, 2, 1)
    assert sorted(a.groups + b.groups) == [0, 1, 2, 3]
    assert sorted(a.seq_index.tolist() + b.seq_index.tolist()) == list(range(10))
    for s in (a, b):
        sizes = np.diff(s.group_offsets).tolist()
        assert sizes == [go[k + 1] - go[k] for k in s.groups]
        assert s.n_seq_global == 10 and s.group_offsets[0] == 0


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_path):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.Workload("shard", 5, 3, 7, 130, "f32", 2.0, 3.0, "uniform", len_lo=2, behav_sigma=0.4,
                           reward_mode="per_prompt", seed=23)
        b = synth.make_batch(w)
        L, V = w.seq_len, w.vocab
        bits = synth.bits_numpy(b["logits"])
        tg, mk = b["targets"].numpy(), b["mask"].numpy()
        behav = (-5.0 + b["behav_noise"]).float().numpy()
        sh = shard.plan(b["group_offsets"].numpy(), b["lengths"].numpy(), world, rank)
        rows = (sh.seq_index[:, None] * L + np.arange(L)[None, :]).reshape(-1)
        for flags in (0, oracle.FLAG_NORM_TOKENS):
            o = oracle.pg_loss(bits[rows], sh.n_seq, L, V, tg[rows], mk[rows], behav[rows],
                               b["rewards"].numpy()[sh.seq_index], sh.group_offsets, 2.0, flags)
            # the library run with RAPID_FLAG_NORM_GIVEN divides by the global Z; the oracle divided
            # by this rank's own count, so rescale
            if flags & oracle.FLAG_NORM_TOKENS:
                z_local = o["n_tokens"]
                z_global = shard.global_token_count(z_local)
            else:
                z_local, z_global = sh.n_seq, sh.n_seq_global
            local = {"loss": o["loss"] * z_local / z_global, "n_tokens": o["n_tokens"], "n_clipped": o["n_clipped"],
                     "n_bad_token": o["n_bad_token"], "n_empty_group": 0, "mean_log_cw": o["mean_log_cw"],
                     "mean_abs_log_cw": o["mean_abs_log_cw"], "status": 0}
            red = shard.reduce_stats(local, sh.n_seq, sh.n_seq_global)
            full = oracle.pg_loss(bits, w.n_seq, L, V, tg, mk, behav, b["rewards"].numpy(),
                                  b["group_offsets"].numpy(), 2.0, flags)
            assert abs(red["loss"] - full["loss"]) <= 1e-12 * max(1.0, abs(full["loss"]))
            assert red["n_tokens"] == full["n_tokens"] and red["n_clipped"] == full["n_clipped"]
            assert abs(red["mean_log_cw"] - full["mean_log_cw"]) <= 1e-12
            assert abs(red["mean_abs_log_cw"] - full["mean_abs_log_cw"]) <= 1e-12
            # groups are whole, so advantages need no communication at all
            np.testing.assert_array_equal(o["adv64"], full["adv64"][sh.seq_index])
        # a failing rank is seen by all
        red = shard.reduce_stats(dict(local, status=6 if rank == 1 else 0), sh.n_seq, sh.n_seq_global)
        assert red["status"] == 6
        if rank == 0:
            open(out_path, "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reduce_to_the_whole_batch(tmp_path):
    out = tmp_path / "done.txt"
    mp.spawn(_rank_main, args=(2, _free_port(), str(out)), nprocs=2, join=True)
    assert out.read_text() == "ok"
