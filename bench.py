#!/usr/bin/env python
"""Benchmark of the hot path: importance-weighted group-advantage PG loss, forward + backward.

A "step" is one pass of the whole path (row statistics, finalize, dlogits) over one synthetic
mini-batch of the SLM shape: 8 prompts x 8 generations, responses of 256-1024 tokens padded to
1024 and masked, V = 151936, bf16 logits.  The metric is unmasked tokens per second.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload ...]

N ranks, one per GPU: either start this file under torch.distributed.run (WORLD_SIZE etc. in the
environment), or give --gpus N > 1 to a plain `python bench.py`, which then starts
`python -m torch.distributed.run --nnodes=1 --nproc-per-node N --master-addr 127.0.0.1 ...` on
itself after checking that the machine has N devices (it refuses otherwise).  Every rank runs
its own mini-batch (the path partitions by prompt group, so there is no collective on the data
path: weak scaling); the time is the maximum over ranks, the tokens the sum.

The default single-GPU run appends short timed runs of the other forms of the path to the same
JSON line (`roofline_onpolicy`, `roofline_fused`, `roofline_fused_stored`, `roofline_long`),
each with its own clock record; --no-extras leaves them out.

--impl reference times the float64 CPU oracle, as it stands, on the host cores (the paper ships
no implementation to run); each of its steps is a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2510_03515_b200 import synth  # noqa: E402

METRIC = "PG loss fwd+bwd tokens/sec at V=151936 bf16"
UNIT = "tokens/s"
WORKLOAD = "slm"


# ------------------------------------------------------------------------------------------------
# helpers
# ------------------------------------------------------------------------------------------------

def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def load_tensor_peaks():
    """(burst, sustained) dense bf16 TFLOP/s and where they come from."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            j = json.load(f)
        return float(j["bf16_tflops"]), float(j.get("bf16_tflops_sustained", j["bf16_tflops"])), "measured"
    return 1590.0, 1400.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons for one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.rows = []
        self.proc = None
        self.thread = None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            self.gpu_id = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            self.gpu_id = str(device_index)

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_id}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for ts, line in self.rows:
            if ts < t0 or ts > t1 + 0.1:
                continue
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                  "sw_power_cap"), parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def torch_token_logp(logits: torch.Tensor, targets: torch.Tensor, rows_per_block: int = 2048):
    """'Current' log-probs used only to synthesise the behaviour policy's stored log-probs
    (input generation with library ops; not part of the measured path)."""
    out = torch.empty(logits.shape[0], dtype=torch.float32, device=logits.device)
    for r0 in range(0, logits.shape[0], rows_per_block):
        z = logits[r0:r0 + rows_per_block].float()
        lse = torch.logsumexp(z, dim=1)
        zy = z.gather(1, targets[r0:r0 + rows_per_block].long().unsqueeze(1)).squeeze(1)
        out[r0:r0 + rows_per_block] = zy - lse
    return out


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------

def oracle_sample(w: synth.Workload, target_seconds: float = 10.0, single_thread: bool = True):
    """Time the oracle, as it stands, on a bounded sample of the workload: whole groups of the
    same vocabulary and dtype with proportionally shorter generations.  Returns a dict."""
    import numpy as np

    import oracle
    cores = oracle.max_threads()

    def run(seq_len: int, n_prompts: int = 1):
        ws = w.scaled(n_prompts=n_prompts, seq_len=seq_len, len_lo=max(1, w.len_lo * seq_len // w.seq_len))
        b = synth.make_batch(ws)
        bits = synth.bits_numpy(b["logits"])
        tg, mk = b["targets"].numpy(), b["mask"].numpy()
        behav = b["behav_noise"].numpy() - 10.0
        t0 = time.perf_counter()
        o = oracle.pg_loss(bits, ws.n_seq, ws.seq_len, ws.vocab, tg, mk, behav, b["rewards"].numpy(),
                           b["group_offsets"].numpy(), 2.0, 0, want_dlogits=False)
        blk = 128
        for r0 in range(0, ws.n_rows, blk):  # step 6 in blocks so the float64 rows fit in memory
            rows = np.arange(r0, min(r0 + blk, ws.n_rows), dtype=np.int64)
            oracle.dlogits_rows(bits, ws.vocab, ws.seq_len, tg, o["row_ok"], o["lse"], o["coef"], rows)
        dt = time.perf_counter() - t0
        return dt, int(o["n_tokens"]), ws

    dt, ntok, ws = run(16)
    seq_len = int(min(w.seq_len, max(16, 16 * target_seconds / max(dt, 1e-3))))
    seq_len = max(16, min(seq_len, w.seq_len))
    dt, ntok, ws = run(seq_len)
    if seq_len == w.seq_len and dt < 0.5 * target_seconds:
        # whole generations already: take more prompt groups (at most 4; drawing their logits on the
        # host is what takes the wall-clock time, not the oracle)
        k = int(min(w.n_prompts, 4, max(1, target_seconds // max(dt, 1e-3))))
        if k > 1:
            dt, ntok, ws = run(seq_len, k)
    # the same on one thread, on a sample shorter by the core count (one prompt group)
    single = None
    if cores > 1 and single_thread:
        oracle.set_threads(1)
        try:
            dt1, ntok1, ws1 = run(max(16, min(ws.seq_len, ws.seq_len * ws.n_prompts // cores)))
            single = {"value": ntok1 / dt1, "unit": UNIT, "cores": 1,
                      "sample": f"{ws1.n_seq} generations x {ws1.seq_len} padded tokens ({ntok1} unmasked), {dt1:.2f} s"}
        finally:
            oracle.set_threads(cores)
    return {"value": ntok / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{ws.n_seq} generations x {ws.seq_len} padded tokens ({ntok} unmasked), "
                      f"V={ws.vocab} {ws.dtype}, float64 steps 1-6, {dt:.2f} s",
            "single_thread": single, "seconds": dt, "tokens": ntok}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.CONFIGS[WORKLOAD]
    for _ in range(max(0, min(args.warmup, 1))):
        oracle_sample(w, target_seconds=1.0, single_thread=False)
    steps = max(1, min(args.steps, 3))
    tot_tok, tot_s, last = 0, 0.0, None
    for _ in range(steps):
        last = oracle_sample(w, target_seconds=8.0, single_thread=(_ == steps - 1))
        tot_tok += last["tokens"]
        tot_s += last["seconds"]
    value = tot_tok / tot_s
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * tot_s / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": WORKLOAD + " (bounded sample per step)", "vocab": w.vocab,
                   "logits_dtype": w.dtype},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["cores"], "kind": "oracle",
                         "sample": last["sample"], "single_thread": last["single_thread"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# ranks, launching, timing
# ------------------------------------------------------------------------------------------------

def launch_command(gpus: int, env: dict, argv: list, device_count: int, port: int):
    """What a plain `python bench.py --gpus N` has to do.  Returns
       ("run", None)     this process is the (or a) rank: go on;
       ("exec", [cmd])   start N ranks with torch.distributed.run on this file;
       ("error", text)   the request cannot be met (too few devices, or ranks that contradict --gpus)."""
    if "WORLD_SIZE" in env:
        world = int(env["WORLD_SIZE"])
        if gpus != world:
            return "error", f"--gpus {gpus} but the launcher started WORLD_SIZE={world} ranks"
        return "run", None
    if gpus <= 1:
        return "run", None
    if device_count < gpus:
        return "error", (f"--gpus {gpus} asked for, but this machine has {device_count} CUDA device(s): "
                         f"refusing to print a line for fewer ranks than asked")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return "exec", cmd


def free_port() -> int:
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def reduce_over_ranks(dist, device, x: float, op: str) -> float:
    """MAX or SUM of one number over the ranks of `dist` (the only things that ever cross ranks here:
    the timed interval and the token count); the number itself when there is one rank."""
    if dist is None:
        return float(x)
    t = torch.tensor([x], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())


class Rank:
    """This process's place among the ranks; the NCCL group carries only timings and token counts."""

    def __init__(self):
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
        if self.local_rank >= torch.cuda.device_count():
            raise SystemExit(f"rank {self.rank}: no CUDA device {self.local_rank} "
                             f"({torch.cuda.device_count()} on this machine)")
        torch.cuda.set_device(self.local_rank)
        self.dev = torch.device("cuda", self.local_rank)
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            if not dist.is_initialized():
                dist.init_process_group("nccl", device_id=self.dev)
            self.dist = dist

    def barrier(self):
        if self.dist:
            self.dist.barrier()

    def max_over_ranks(self, x: float) -> float:
        return reduce_over_ranks(self.dist, self.dev, x, "max")

    def sum_over_ranks(self, x: float) -> float:
        return reduce_over_ranks(self.dist, self.dev, x, "sum")

    def close(self):
        if self.dist and self.dist.is_initialized():
            self.dist.destroy_process_group()


def timed_region(rk: Rank, step, steps: int, n_marks: int):
    """Barrier + synchronize, `steps` calls of step(events), synchronize + barrier.  `step` records
    its `n_marks` events (first = start of the step, last = its end) on the current stream, which is
    the stream the library launches on.  Returns (total ms, maximum over ranks; per-step lists of
    the n_marks - 1 intervals in ms, this rank's; the clock record taken meanwhile)."""
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(n_marks)] for _ in range(steps)]
    sampler = ClockSampler(rk.local_rank) if rk.rank == 0 else None
    rk.barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
        time.sleep(0.25)
    t0w = time.time()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for k in range(steps):
        step(evs[k])
    end.record()
    torch.cuda.synchronize()
    t1w = time.time()
    rk.barrier()
    clocks = sampler.stop(t0w, t1w) if sampler else None
    total_ms = rk.max_over_ranks(start.elapsed_time(end))
    parts = [[e[i].elapsed_time(e[i + 1]) for e in evs] for i in range(n_marks - 1)]
    whole = [e[0].elapsed_time(e[-1]) for e in evs]
    return total_ms, parts, whole, clocks


def mean_median(xs):
    return statistics.mean(xs), statistics.median(xs)


# ------------------------------------------------------------------------------------------------
# the logits-in path (--workload slm, the metric's configuration; --workload long, chunked form)
# ------------------------------------------------------------------------------------------------

# DRAM traffic per algorithmic byte, from the ncu captures summarised under profiles/ (counters
# dram__bytes_read.sum + dram__bytes_write.sum of a smaller launch of the same kernel; traffic grows
# in proportion to the rows processed).  NOT counters of this run: the line says so.
TRAFFIC_P2_PER_BYTE = 0.9873
TRAFFIC_P2_SOURCE = "profiles/logits_in_path_slm_bf16.md: ncu dram bytes of a 2.5 GB launch x rows of this one"
# the on-policy kernel: dram__bytes_read.sum per byte of live rows, dram__bytes_write.sum per byte of all rows
TRAFFIC_OP_READ_PER_LIVE_BYTE = 1.280
TRAFFIC_OP_WRITE_PER_ROW_BYTE = 0.978
TRAFFIC_OP_SOURCE = "profiles/onpolicy_rows_kernel_slm_bf16.md: ncu dram bytes of an 8192-row launch x rows of this one"
# pass 1's secondary ceiling: share of cycles the MUFU (ex2) pipe is busy, same captures
MUFU_PIPE_PCT_PASS1 = 81.1
MUFU_SOURCE = "profiles/logits_in_path_slm_bf16.md (ncu pipe utilisation of row_stats_kernel)"


def run_ours(args, rk: Rank):
    from paper_2510_03515_b200 import binding as rb
    rank, dev, world = rk.rank, rk.dev, rk.world
    rb.lib()

    name = args.workload if args.workload in ("slm", "long") else WORKLOAD
    w = synth.CONFIGS[name].scaled(seed=synth.CONFIGS[name].seed + 1000 * rank)
    if args.seq_len:
        w = w.scaled(seq_len=args.seq_len, len_lo=max(1, args.seq_len // 4))
    # the long-sequence configuration goes through the chunked three-step form, four generations at a time
    chunk_rows = 4 * w.seq_len if name == "long" else w.n_rows
    tok = synth.make_tokens(w)
    T, V, N = w.n_rows, w.vocab, w.n_seq
    esize = 2 if w.dtype == "bf16" else 4
    logits = synth.logits_for_sequences(w, tok["targets"], 0, N, device=dev)
    targets, mask = tok["targets"].to(dev), tok["mask"].to(dev)
    rewards, go = tok["rewards"].to(dev), tok["group_offsets"].to(dev)
    behav = (torch_token_logp(logits, targets) + tok["behav_noise"].to(dev)).contiguous()
    dlogits = torch.empty_like(logits)
    desc = rb.make_desc(N, w.seq_len, V, w.n_prompts, logits.dtype, logits.stride(0), 2.0, 0)
    ws = rb.alloc_workspace(desc, dev)
    loss = torch.zeros(1, device=dev)
    token_logp = torch.empty(T, device=dev)
    adv = torch.empty(N, device=dev)
    stats = rb.alloc_stats(dev)
    n_tokens = int(tok["mask"].sum().item())

    def step(ev=None):
        if ev:
            ev[0].record()
        for r0 in range(0, T, chunk_rows):
            n = min(chunk_rows, T - r0)
            rb.rapid_pg_stats_chunk(desc, logits[r0:r0 + n], r0, n, targets, mask, ws)
        if ev:
            ev[1].record()
        rb.rapid_pg_finalize(desc, behav, rewards, go, loss, token_logp, adv, stats, ws)
        if ev:
            ev[2].record()
        for r0 in range(0, T, chunk_rows):
            n = min(chunk_rows, T - r0)
            rb.rapid_pg_dlogits_chunk(desc, logits[r0:r0 + n], dlogits[r0:r0 + n], r0, n, targets, stats, ws)
        if ev:
            ev[3].record()

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    st = rb.read_stats(stats)
    # rows pass 2 really streams: unmasked rows of generations with a non-zero coefficient
    coef_live = (adv != 0).repeat_interleave(w.seq_len)
    live_rows = int((coef_live & (mask != 0)).sum().item())

    elapsed_ms, parts, whole, clocks = timed_region(rk, step, args.steps, 4)
    total_tokens = rk.sum_over_ranks(n_tokens)
    ms_per_step = elapsed_ms / args.steps
    value = total_tokens / (ms_per_step * 1e-3)
    ms_median = rk.max_over_ranks(statistics.median(whole))

    (p1, p1_med), (fin, _), (p2, p2_med) = (mean_median(x) for x in parts)
    peak, peak_kind = load_peaks()
    row_bytes = V * esize
    # algorithmic bytes: pass 1 reads every unmasked row once; pass 2 re-reads the live rows and
    # writes every row (zeros for the rest)
    bytes_p1 = n_tokens * row_bytes
    bytes_p2 = live_rows * row_bytes + T * row_bytes
    ach_p1 = bytes_p1 / (p1 * 1e-3) / 1e9
    ach_p2 = bytes_p2 / (p2 * 1e-3) / 1e9
    ach_all = (bytes_p1 + bytes_p2) / (ms_per_step * 1e-3) / 1e9

    # ---- end to end through the public call with HOST buffers ------------------------------------
    e2e = e2e_grad = None
    if not args.skip_e2e and name == "slm":
        e2e, e2e_grad = run_e2e(rb, args, desc, w, logits, tok, behav, dlogits, ws, loss, token_logp, adv, stats,
                                n_tokens, rk)

    if rank != 0:
        return None
    cpu = None
    if not args.skip_cpu:
        cpu = oracle_sample(w, target_seconds=args.cpu_seconds)
        for k in ("seconds", "tokens"):
            cpu.pop(k, None)
    n_chunks = (T + chunk_rows - 1) // chunk_rows
    line = {
        "metric": METRIC if name == "slm" else f"PG loss fwd+bwd tokens/sec at V={V} {w.dtype} (chunked form)",
        "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "ms_per_step_median": ms_median, "value_at_median": total_tokens / (ms_median * 1e-3),
        "config": {"workload": name, "chunk_rows": chunk_rows, "prompts": w.n_prompts,
                   "generations_per_prompt": w.group_size,
                   "padded_len": w.seq_len, "vocab": V, "logits_dtype": w.dtype,
                   "unmasked_tokens_per_gpu": n_tokens, "rows_per_gpu": T,
                   "l2_policy": f"inputs larger than L2 ({T * row_bytes / 1e9:.1f} GB logits per step)",
                   "eta": 2.0, "parallelism": f"dp{world} (by prompt group, no data-path collective)"},
        "clocks": clocks,
        "e2e": e2e,
        "e2e_gradient_to_host": e2e_grad,
        "gpu_launches": (2 + 2 * n_chunks) * args.steps,
        "roofline": {"bound": "hbm", "kernel": "dlogits_kernel (pass 2)", "achieved": ach_p2,
                     "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": ach_p2 / peak,
                     "frac_of_8TBs_nominal": ach_p2 / 8000.0, "ms_per_launch": p2 / n_chunks,
                     "ms_per_step": p2, "ms_per_step_median": p2_med,
                     "achieved_at_median": bytes_p2 / (p2_med * 1e-3) / 1e9,
                     "algorithmic_bytes_per_launch": bytes_p2 / n_chunks, "launches_per_step": n_chunks,
                     "traffic": (TRAFFIC_P2_PER_BYTE * bytes_p2) if name == "slm" else None,
                     "traffic_source": TRAFFIC_P2_SOURCE if name == "slm" else None},
        "roofline_pass1": {"bound": "hbm", "kernel": "row_stats_kernel (pass 1)", "achieved": ach_p1,
                           "peak": peak, "unit": "GB/s", "frac": ach_p1 / peak,
                           "frac_of_8TBs_nominal": ach_p1 / 8000.0, "ms_per_launch": p1 / n_chunks,
                           "ms_per_step": p1, "ms_per_step_median": p1_med,
                           "achieved_at_median": bytes_p1 / (p1_med * 1e-3) / 1e9,
                           "algorithmic_bytes_per_launch": bytes_p1 / n_chunks, "launches_per_step": n_chunks,
                           "secondary_ceiling": {"pipe": "MUFU ex2", "pipe_active_pct": MUFU_PIPE_PCT_PASS1,
                                                 "source": MUFU_SOURCE} if w.dtype == "bf16" else None},
        "roofline_step": {"achieved": ach_all, "peak": peak, "unit": "GB/s", "frac": ach_all / peak,
                          "frac_of_8TBs_nominal": ach_all / 8000.0, "finalize_ms": fin},
        "cpu_baseline": cpu,
        "stats": {"n_clipped": st["n_clipped"], "mean_log_cw": st["mean_log_cw"], "loss": st["loss"]},
    }
    return line


def run_e2e(rb, args, desc, w, logits, tok, behav, dlogits, ws, loss, token_logp, adv, stats, n_tokens, rk: Rank):
    """Same step, but the inputs start in pinned HOST memory and the loss is read back to the host
    every step.  Uses a full pinned copy of the logits when the host has room, otherwise a
    2 GiB pinned buffer copied repeatedly into successive device slices (same bytes moved).

    Two figures.  `e2e`: inputs in, loss out; dlogits, the path's main output, stays in device
    memory, where the transformer's backward pass consumes it (the method alternates inference and
    training on the same GPUs, so nothing downstream wants the gradient on the host).
    `e2e_gradient_to_host`: the same plus a copy of all of dlogits to pinned host memory, for a
    caller that does want it there; only taken when the host has room for the second buffer."""
    import psutil
    dev = rk.dev
    T = logits.shape[0]
    nbytes = logits.numel() * logits.element_size()
    steps = max(1, min(args.e2e_steps, args.steps))
    mode = "full pinned copy"
    host_logits = None
    try:
        if psutil.virtual_memory().available > 3 * nbytes:
            host_logits = torch.empty(logits.shape, dtype=logits.dtype, pin_memory=True)
            host_logits.copy_(logits)
    except Exception:
        host_logits = None
    if host_logits is None:
        rows = max(1, min(T, (2 << 30) // (logits.shape[1] * logits.element_size())))
        host_logits = torch.empty((rows, logits.shape[1]), dtype=logits.dtype, pin_memory=True)
        host_logits.copy_(logits[:rows])
        mode = f"{rows}-row pinned buffer reused for every slice"
    small = {k: tok[k].pin_memory() for k in ("targets", "mask", "rewards", "group_offsets")}
    h_behav = behav.cpu().pin_memory()
    d = {k: torch.empty_like(v, device=dev) for k, v in small.items()}
    d_behav = torch.empty_like(behav)
    d_logits = torch.empty_like(logits)
    h_loss = torch.empty(1, dtype=torch.float32).pin_memory()
    h2d = nbytes + sum(v.numel() * v.element_size() for v in small.values()) + h_behav.numel() * 4

    direct = host_logits.shape[0] == T   # the whole batch is pinned: let the kernels read it from there
    if direct:
        mode = "full pinned copy, read in place by the statistics pass (masked rows never cross the bus)"
        h2d = n_tokens * logits.shape[1] * logits.element_size() + \
            sum(v.numel() * v.element_size() for v in small.values()) + h_behav.numel() * 4
    host_grad = None

    def step():
        for k in small:
            d[k].copy_(small[k], non_blocking=True)
        d_behav.copy_(h_behav, non_blocking=True)
        if direct:
            rb.rapid_pg_loss_fwd_bwd_hostlogits(desc, host_logits, d_logits, d["targets"], d["mask"], d_behav,
                                                d["rewards"], d["group_offsets"], dlogits, loss, token_logp, adv,
                                                stats, ws)
        else:
            R = host_logits.shape[0]
            for r0 in range(0, T, R):
                n = min(R, T - r0)
                d_logits[r0:r0 + n].copy_(host_logits[:n], non_blocking=True)
            rb.rapid_pg_loss_fwd_bwd(desc, d_logits, d["targets"], d["mask"], d_behav, d["rewards"],
                                     d["group_offsets"], dlogits, loss, token_logp, adv, stats, ws)
        h_loss.copy_(loss, non_blocking=True)
        if host_grad is not None:
            host_grad.copy_(dlogits, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        return float(h_loss[0])

    def timed():
        step()
        rk.barrier()
        torch.cuda.synchronize()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for _ in range(steps):
            step()
        e.record()
        torch.cuda.synchronize()
        return rk.max_over_ranks(s.elapsed_time(e))

    ms = timed()
    tokens = rk.sum_over_ranks(n_tokens)
    out = {"value": tokens * steps / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
           "d2h_bytes_per_step": 4, "steps": steps, "ms_per_step": ms / steps, "host_buffer": mode,
           "d2h_is": "the loss", "result_left_on_device_bytes": int(nbytes),
           "result_left_on_device": "dlogits (consumed on the device by the backward pass of the model)"}
    # the second figure needs a second pinned buffer on every rank: each rank tries, all agree, then all
    # time it or none does (a rank that skipped the timed loop would leave the others at its barrier)
    out_grad = None
    why = ""
    try:
        if psutil.virtual_memory().available > 2 * nbytes:
            host_grad = torch.empty(logits.shape, dtype=logits.dtype, pin_memory=True)
        else:
            why = "not enough host memory for a second pinned buffer"
    except RuntimeError as ex:
        host_grad, why = None, str(ex).splitlines()[0][:200]
    if rk.sum_over_ranks(0.0 if host_grad is not None else 1.0) == 0.0:
        ms2 = timed()
        out_grad = {"value": tokens * steps / (ms2 * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                    "d2h_bytes_per_step": int(nbytes) + 4, "steps": steps, "ms_per_step": ms2 / steps,
                    "d2h_is": "the loss and all of dlogits"}
    else:
        host_grad = None
        out_grad = {"unavailable": why or "another rank could not pin its buffer"}
    del d_logits, host_logits, host_grad
    return out, out_grad


# ------------------------------------------------------------------------------------------------
# the fused LM-head form (--workload fused): hidden states and the LM-head weight in, no logits
# ------------------------------------------------------------------------------------------------

def run_fused(args, rk: Rank):
    from paper_2510_03515_b200 import binding as rb
    rank, dev, world = rk.rank, rk.dev, rk.world
    rb.lib()
    w = synth.CONFIGS["fused"].scaled(seed=synth.CONFIGS["fused"].seed + 1000 * rank)
    if args.seq_len:
        w = w.scaled(seq_len=args.seq_len)
    b = synth.make_head(w, device=dev)
    T, V, D, N = w.n_rows, w.vocab, w.hidden, w.n_seq
    stored = args.head == "stored"
    desc = rb.make_desc(N, w.seq_len, V, w.n_prompts, torch.bfloat16, V, 2.0,
                        (rb.FLAG_HEAD_STORE_LOGITS if stored else 0) |
                        (rb.FLAG_HEAD_CTA_PAIRS if getattr(args, "cta_pairs", False) else 0) |
                        (rb.FLAG_HEAD_SINGLE_CTA if getattr(args, "single_cta", False) else 0))
    ws = rb.alloc_fused_head_workspace(desc, D, dev)
    loss = torch.zeros(1, device=dev)
    dh = torch.empty((T, D), dtype=torch.bfloat16, device=dev)
    dW = torch.empty((D, V), dtype=torch.float32, device=dev)
    tl = torch.empty(T, device=dev)
    adv = torch.empty(N, device=dev)
    stats = rb.alloc_stats(dev)
    behav = torch.full((T,), -12.0, device=dev)

    def step(ev=None, hid=None, wv=None, bh=None):
        if ev:
            ev[0].record()
        rb.rapid_pg_loss_fused_head(desc, b["hidden"] if hid is None else hid, b["w_vocab"] if wv is None else wv,
                                    b["targets"], b["mask"], behav if bh is None else bh, b["rewards"],
                                    b["group_offsets"], loss, dh, dW, tl, adv, stats, ws)
        if ev:
            ev[1].record()

    step()   # the library's own token log-probs seed the synthetic behaviour log-probs (input synthesis)
    torch.cuda.synchronize()
    behav = (tl + b["behav_noise"]).contiguous()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    ms, _, whole, clocks = timed_region(rk, step, args.steps, 2)
    n_tokens = int(b["mask"].sum().item())
    tokens = rk.sum_over_ranks(n_tokens)
    ms_per_step = ms / args.steps
    ms_median = rk.max_over_ranks(statistics.median(whole))
    st = rb.read_stats(stats)

    # end to end: hidden states, weight and per-token arrays start in pinned host memory
    e2e = None
    if not args.skip_e2e:
        names = ("hidden", "w_vocab")
        host = {k: b[k].cpu().pin_memory() for k in names}
        h_behav = behav.cpu().pin_memory()
        d_in = {k: torch.empty_like(b[k]) for k in names}
        d_behav = torch.empty_like(behav)
        h_loss = torch.empty(1, dtype=torch.float32).pin_memory()
        h2d = sum(v.numel() * v.element_size() for v in host.values()) + h_behav.numel() * 4

        def e2e_step():
            for k in names:
                d_in[k].copy_(host[k], non_blocking=True)
            d_behav.copy_(h_behav, non_blocking=True)
            step(None, d_in["hidden"], d_in["w_vocab"], d_behav)
            h_loss.copy_(loss, non_blocking=True)
            torch.cuda.current_stream().synchronize()

        e2e_step()
        rk.barrier()
        torch.cuda.synchronize()
        k = max(1, min(args.e2e_steps, args.steps))
        s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s2.record()
        for _ in range(k):
            e2e_step()
        e2.record()
        torch.cuda.synchronize()
        ems = rk.max_over_ranks(s2.elapsed_time(e2))
        e2e = {"value": tokens * k / (ems * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": 4, "steps": k, "ms_per_step": ems / k, "d2h_is": "the loss",
               "result_left_on_device_bytes": int(dh.numel() * 2 + dW.numel() * 4),
               "result_left_on_device": "dhidden and dW (consumed on the device by the model's backward pass and optimizer)"}
    if rank != 0:
        return None
    cpu = None
    if not args.skip_cpu:
        cpu = oracle_head_sample(w, target_seconds=args.cpu_seconds)
    burst, sustained, kind = load_tensor_peaks()
    n_gemm = 3 if stored else 4   # forward, (recompute,) dhidden, dW
    flops = n_gemm * 2.0 * T * D * V
    ach = flops / (ms_per_step * 1e-3) / 1e12
    mhz = (clocks or {}).get("sm_mhz")
    line = {
        "metric": "fused LM-head PG loss fwd+bwd tokens/sec at V=151936 bf16", "value": tokens / (ms_per_step * 1e-3),
        "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "ms_per_step_median": ms_median,
        "config": {"workload": "fused", "head": args.head, "ctas_per_tile": ("pairs" if getattr(args, "cta_pairs", False) else "single" if getattr(args, "single_cta", False)
                                             else "pairs for forward and recompute, single for dhidden and dW"), "prompts": w.n_prompts, "generations_per_prompt": w.group_size,
                   "padded_len": w.seq_len, "rows_per_gpu": T, "hidden": D, "vocab": V,
                   "l2_policy": "inputs larger than L2 (0.47 GB weight, 5 GB dlogits scratch per step)",
                   "eta": 2.0, "parallelism": f"dp{world} (by prompt group, no data-path collective)"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": 9 * args.steps,
        "roofline": {"bound": "tensor",
                     "kernel": ("umma gemm_kernel x3 (forward statistics + logits store, dhidden, dW); dlogits in place "
                                "by the logits-in second pass") if stored else
                               "umma gemm_kernel x4 (forward statistics, dlogits, dhidden, dW)",
                     "achieved": ach, "peak": sustained, "peak_kind": kind + " sustained", "unit": "TFLOP/s",
                     "frac": ach / sustained, "frac_of_burst": ach / burst, "flops_per_step": flops,
                     "ms_x_sm_mhz": (ms_per_step * mhz) if mhz else None,
                     "traffic": None},
        "cpu_baseline": cpu,
        "stats": {"n_clipped": st["n_clipped"], "mean_log_cw": st["mean_log_cw"], "loss": st["loss"],
                  "status": st["status"]},
    }
    return line


def oracle_head_sample(w: synth.Workload, target_seconds: float = 6.0):
    """The oracle's fused-head steps (float64 product by plain loops, steps 1-6, dhidden, dW), as they
    stand, on a bounded sample: a few generations of the same hidden size and vocabulary."""
    import numpy as np

    import oracle
    cores = oracle.max_threads()

    def run(n_rows):
        L = max(1, n_rows // 2)
        ws_ = w.scaled(n_prompts=1, group_size=2, seq_len=L)
        b = synth.make_head(ws_)
        hb, wb = synth.bits_numpy(b["hidden"]), synth.bits_numpy(b["w_vocab"])
        tg = b["targets"].numpy()
        t0 = time.perf_counter()
        z = oracle.head_logits(hb, wb)
        lse, lp = oracle.token_logp_f64(z, tg)
        behav = (lp + b["behav_noise"].numpy()).astype(np.float32)
        s_, S_, cnt = oracle.seq_reduce(ws_.n_seq, L, lp, behav, np.ones(ws_.n_rows, np.uint8))
        ga = oracle.group_advantage(b["rewards"].numpy(), s_, b["group_offsets"].numpy(), 2.0, 0)
        _, coef, _ = oracle.coef_loss(s_, S_, cnt, ga["weight"], ga["clipped_w"], ga["adv64"], 2.0, 0)
        dz = oracle.dlogits_f64_inplace(z, tg, lse, np.repeat(coef, L))
        oracle.head_dhidden(dz, wb)
        dW = np.zeros((ws_.hidden, ws_.vocab))
        oracle.head_dweight_accum(dW, dz, hb)
        return time.perf_counter() - t0, ws_.n_rows

    dt, n = run(8)
    rows = int(max(8, min(512, 8 * target_seconds / max(dt, 1e-3)))) // 2 * 2
    if rows > n:
        dt, n = run(rows)
    return {"value": n / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n} rows of hidden size {w.hidden}, V={w.vocab}, float64 product by plain loops, "
                      f"steps 1-6, dhidden and dW, {dt:.2f} s"}


# ------------------------------------------------------------------------------------------------
# the on-policy single-pass form (--workload onpolicy): same mini-batch as slm, weights all one
# ------------------------------------------------------------------------------------------------

def run_onpolicy(args, rk: Rank):
    from paper_2510_03515_b200 import binding as rb
    rank, dev, world = rk.rank, rk.dev, rk.world
    w = synth.CONFIGS["slm"].scaled(seed=synth.CONFIGS["slm"].seed + 1000 * rank)
    if args.seq_len:
        w = w.scaled(seq_len=args.seq_len, len_lo=max(1, args.seq_len // 4))
    tok = synth.make_tokens(w)
    T, V, N = w.n_rows, w.vocab, w.n_seq
    logits = synth.logits_for_sequences(w, tok["targets"], 0, N, device=dev)
    targets, mask = tok["targets"].to(dev), tok["mask"].to(dev)
    rewards, go = tok["rewards"].to(dev), tok["group_offsets"].to(dev)
    dlogits = torch.empty_like(logits)
    desc = rb.make_desc(N, w.seq_len, V, w.n_prompts, logits.dtype, logits.stride(0), 2.0, 0)
    ws = rb.alloc_workspace(desc, dev)
    loss = torch.zeros(1, device=dev)
    adv = torch.empty(N, device=dev)
    stats = rb.alloc_stats(dev)
    n_tokens = int(tok["mask"].sum().item())

    def step(ev=None):
        if ev:
            ev[0].record()
        rb.rapid_pg_loss_onpolicy_fwd_bwd(desc, logits, targets, mask, rewards, go, dlogits, loss, None, adv, stats, ws)
        if ev:
            ev[1].record()

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    live_rows = int(((adv != 0).repeat_interleave(w.seq_len) & (mask != 0)).sum().item())
    ms, _, whole, clocks = timed_region(rk, step, args.steps, 2)
    tokens = rk.sum_over_ranks(n_tokens)
    ms_median = rk.max_over_ranks(statistics.median(whole))
    if rank != 0:
        return None
    ms_per_step = ms / args.steps
    st = rb.read_stats(stats)
    cpu = None
    if not args.skip_cpu:   # the oracle's steps 1-6 on a bounded sample of the same mini-batch shape
        cpu = oracle_sample(w, target_seconds=args.cpu_seconds, single_thread=False)
        for k in ("seconds", "tokens", "single_thread"):
            cpu.pop(k, None)
    peak, peak_kind = load_peaks()
    row_bytes = V * (2 if w.dtype == "bf16" else 4)
    algo = live_rows * 2 * row_bytes + (T - live_rows) * row_bytes   # live rows: one read + one write
    # reads grow with the live rows (the second sweep misses L2 for part of each), writes with all rows
    traffic = TRAFFIC_OP_READ_PER_LIVE_BYTE * live_rows * row_bytes + TRAFFIC_OP_WRITE_PER_ROW_BYTE * T * row_bytes
    ach = algo / (ms_per_step * 1e-3) / 1e9
    line = {
        "metric": "on-policy PG loss fwd+bwd tokens/sec at V=151936 bf16 (single pass)",
        "value": tokens / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "ms_per_step_median": ms_median,
        "config": {"workload": "onpolicy (slm mini-batch, mu = pi_theta)", "prompts": w.n_prompts,
                   "generations_per_prompt": w.group_size, "padded_len": w.seq_len, "vocab": V,
                   "logits_dtype": w.dtype, "unmasked_tokens_per_gpu": n_tokens, "live_rows_per_gpu": live_rows,
                   "rows_per_gpu": T, "l2_policy": "inputs larger than L2",
                   "parallelism": f"dp{world} (by prompt group, no data-path collective)"},
        "clocks": clocks, "e2e": None, "gpu_launches": 4 * args.steps,
        "roofline": {"bound": "hbm", "kernel": "onpolicy_rows_kernel", "achieved": ach, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": ach / peak, "frac_of_8TBs_nominal": ach / 8000.0,
                     "achieved_at_median": algo / (ms_median * 1e-3) / 1e9,
                     "algorithmic_bytes_per_launch": algo, "traffic": traffic, "traffic_source": TRAFFIC_OP_SOURCE},
        "cpu_baseline": cpu, "stats": {"loss": st["loss"], "status": st["status"]},
    }
    return line


# ------------------------------------------------------------------------------------------------
# the other forms of the path, appended to the default line
# ------------------------------------------------------------------------------------------------

def run_extras(args, rk: Rank) -> dict:
    """Short timed runs of the on-policy, fused-head (both variants) and long-sequence workloads, each
    with the same timing protocol and its own clock record, condensed to one object per workload."""
    import copy
    import gc
    out = {}
    plan = [("roofline_onpolicy", run_onpolicy, {"workload": "onpolicy", "steps": 30}),
            ("roofline_fused", run_fused, {"workload": "fused", "head": "recompute", "steps": 12}),
            ("roofline_fused_stored", run_fused, {"workload": "fused", "head": "stored", "steps": 12}),
            ("roofline_long", run_ours, {"workload": "long", "steps": 20})]
    for key, fn, over in plan:
        a = copy.copy(args)
        for k, v in over.items():
            setattr(a, k, v)
        a.warmup, a.skip_e2e, a.seq_len, a.cpu_seconds = 3, True, 0, 4.0
        gc.collect()
        torch.cuda.empty_cache()
        try:
            ln = fn(a, rk)
        except Exception as ex:      # a workload that cannot run here must not take the headline line down
            out[key] = {"unavailable": f"{type(ex).__name__}: {str(ex).splitlines()[0][:200]}"}
            continue
        if ln is None:
            continue
        r = dict(ln["roofline"])
        r.update({"workload": ln["config"]["workload"], "metric": ln["metric"], "value": ln["value"],
                  "value_unit": ln["unit"], "steps": ln["steps"], "warmup": ln["warmup"], "ms_per_step": ln["ms_per_step"],
                  "ms_per_step_median": ln.get("ms_per_step_median"), "clocks": ln["clocks"],
                  "gpu_launches": ln["gpu_launches"], "cpu_baseline": ln.get("cpu_baseline")})
        if "roofline_pass1" in ln:
            r["pass1"] = ln["roofline_pass1"]
            r["step"] = ln["roofline_step"]
        out[key] = r
    # the oracle on a bounded slice of the two configurations that have no timed GPU run of their own
    # (tiny: launch-bound, parity only; stale: the shape class of slm), so that every configuration has one
    if rk.rank == 0 and not args.skip_cpu:
        other = {}
        for name in ("tiny", "stale"):
            c = oracle_sample(synth.CONFIGS[name], target_seconds=3.0, single_thread=False)
            for k in ("seconds", "tokens", "single_thread"):
                c.pop(k, None)
            other[name] = c
        out["cpu_baseline_other_configs"] = other
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="slm", choices=["slm", "fused", "onpolicy", "long"],
                    help="slm: the logits-in path the metric is quoted on (default); long: the 64 x 4096 x 32000 fp32 configuration through the chunked form; onpolicy: single pass; fused: the LM-head form")
    ap.add_argument("--cta-pairs", action="store_true",
                    help="--workload fused: all four contractions on pairs of CTAs (256 x 256 tiles, tcgen05 cta_group::2)")
    ap.add_argument("--single-cta", action="store_true",
                    help="--workload fused: all four contractions on one CTA per 128 x 256 tile (default: the measured-best mix)")
    ap.add_argument("--head", default="recompute", choices=["recompute", "stored"],
                    help="--workload fused: form the logits twice on the tensor cores (four contractions), or keep "
                         "them in bf16 between forward and backward (three contractions)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--skip-e2e", action="store_true", help="leave out the host-buffer leg (profiling)")
    ap.add_argument("--skip-cpu", action="store_true", help="leave out the CPU oracle timing (profiling)")
    ap.add_argument("--no-extras", action="store_true",
                    help="default workload on one GPU: leave out the appended runs of the other workloads")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="size of the CPU oracle's timed sample")
    ap.add_argument("--seq-len", type=int, default=0,
                    help="shorter padded length (smaller device footprint, e.g. for profiling)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    what, arg = launch_command(args.gpus, os.environ, sys.argv[1:],
                               torch.cuda.device_count() if torch.cuda.is_available() else 0, free_port())
    if what == "error":
        raise SystemExit("bench.py: " + arg)
    if what == "exec":
        sys.stdout.flush()
        os.execv(arg[0], arg)
    args.warmup = max(args.warmup, 3)
    rk = Rank()
    try:
        if args.workload == "fused":
            line = run_fused(args, rk)
        elif args.workload == "onpolicy":
            line = run_onpolicy(args, rk)
        else:
            line = run_ours(args, rk)
        if args.workload == "slm" and rk.world == 1 and not args.no_extras and not args.seq_len:
            line.update(run_extras(args, rk))
        if rk.rank == 0:
            print(json.dumps(line), flush=True)
    finally:
        rk.close()


if __name__ == "__main__":
    main()
