"""Benchmark of the fused COBS decode step (cobs_decode_step) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one pass of the whole per-decode-step path (block scoring from the summaries, top-k
selection, block-sparse attention over the selected blocks plus the window) over one batch of a
synthetic long-context workload whose KV cache and summaries are resident in HBM.  The reported
value is the whole-job achieved HBM bandwidth: algorithmic bytes per step (summary records of every
summarised block + K and V of the selected and window blocks + q + out) times the number of ranks,
divided by the step time (CUDA events, max over ranks).  Prints ONE JSON line on rank 0.

With N > 1 every rank holds its own batch of sequences: the path shards over (sequence, KV head) with no
collective, so scaling is weak.  `--gpus N` with no rank environment (plain `python bench.py --gpus N`) starts the
N ranks itself through torch.distributed.run on 127.0.0.1; under torchrun the ranks are taken from the environment.
The line also carries `other_workloads`: the step time and roofline fraction of the other named configurations
(fewer steps each), so that one run covers the 32k configurations as well as the 128k one.
"""

from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2607_09052_b200 import shard, synth  # noqa: E402

DEFAULT_WORKLOAD = "cfg4_128k"
L2_FLUSH_BYTES = 256 << 20
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the fused kernel (ncu; see profiles/)
TRAFFIC_BYTES = {"cfg4_128k": 4 * (128485376 + 3605760)}   # batch-4 capture x 4 (traffic is proportional to batch)


def algorithmic_bytes(wl: synth.Workload, record_bytes: int) -> int:
    """Bytes one step must read or write: summary records of every summarised block, K and V of the
    selected and window blocks, q, out, the page-table entries of the blocks read, and U_Q."""
    total = 0
    L, D = wl.block_size, wl.head_dim
    for t in wl.lens():
        n_sum = t // L
        ws = (max(0, t - wl.window) // L) * L
        n_cand = ws // L
        n_sel = min(wl.topk, n_cand)
        kv_tokens = n_sel * L + (t - ws)
        total += wl.n_kv_heads * (n_sum * record_bytes + kv_tokens * D * 2 * 2)
        total += (kv_tokens + wl.page_size - 1) // wl.page_size * 4
    total += wl.batch * wl.n_q_heads * D * (2 + 4)
    if wl.sub_dim:
        total += wl.n_kv_heads * D * wl.sub_dim * 4
    return total


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class L2Flush:
    """Between timed steps: write a buffer twice the size of L2.  That alone leaves L2 full of DIRTY lines, whose
    write-back then competes with the next step's reads for HBM (up to 126 MB of extra DRAM writes inside the timed
    region: an artefact of the flush, not of the workload), so the default mode reads a second buffer of the same
    size afterwards: L2 then holds clean lines of an unrelated buffer.  Mode "write" is the plain write."""

    def __init__(self, dev, mode="write+read"):
        self.mode = mode
        self.buf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
        self.src = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device=dev) if mode == "write+read" else None

    def zero_(self):
        self.buf.zero_()
        if self.src is not None:
            torch.max(self.src)

    def describe(self):
        what = "write" if self.src is None else "write, then read of a second buffer of that size (leaves L2 clean)"
        return f"{L2_FLUSH_BYTES >> 20} MiB {what} between timed steps (outside the events)"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def ensure_ranks(args):
    """Make `--gpus N` mean N ranks.  Under a launcher (WORLD_SIZE set) the environment decides and must agree with
    the flag; without one and N > 1 this process replaces itself by `python -m torch.distributed.run` with N
    workers on this node (rendezvous on 127.0.0.1), each of which re-enters this script with its rank set."""
    if "WORLD_SIZE" in os.environ:
        world = int(os.environ["WORLD_SIZE"])
        if args.gpus != world:
            if int(os.environ.get("RANK", "0")) == 0:
                sys.stderr.write(f"bench.py: --gpus {args.gpus} but the launcher started {world} ranks; using {world}\n")
            args.gpus = world
        return
    if args.gpus <= 1:
        return
    if args.impl == "ours" and not args.launch_selftest:
        have = torch.cuda.device_count()
        if args.gpus > have:
            sys.stderr.write(f"bench.py: --gpus {args.gpus} but this node has {have} CUDA device(s)\n")
            sys.exit(2)
    cmd = shard.launcher_command(os.path.abspath(__file__), args.gpus, sys.argv[1:])
    sys.stdout.flush()
    os.execvp(cmd[0], cmd)


OTHER_WORKLOADS = ["cfg2_32k", "cfg3a_32k_subspace", "cfg3b_32k_k85", "cfg5_64k_g8"]


class Measurement:
    """One workload resident on one GPU: inputs, summaries built by the library, and the timed loops."""

    def __init__(self, B, wl, dev):
        self.B, self.wl, self.dev = B, wl, dev
        self.inp = synth.generate(wl, dev)
        self.cfg = B.make_config(wl)
        self.kv = B.make_kv(self.inp)
        self.summ = B.SummaryBuffers(self.cfg, dev, self.inp.get("u_q"))
        self.ws = B.alloc_workspace(self.cfg, dev)
        self.stream = torch.cuda.current_stream()
        nb, hq, hkv, D = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
        self.out = torch.zeros((nb, hq, D), dtype=torch.float32, device=dev)
        self.sel = torch.zeros((nb, hkv, wl.topk), dtype=torch.int32, device=dev)
        self.cnt = torch.zeros((nb, hkv), dtype=torch.int32, device=dev)
        mb, xb, sb = B.cobs_summary_bytes(self.cfg)
        self.record = (mb + xb + sb) // (nb * hkv * wl.max_blocks)
        self.step_bytes = algorithmic_bytes(wl, self.record)
        self.summary_bytes = sum(hkv * (t // wl.block_size) * self.record for t in wl.lens())
        # summaries of every block, built by the library (set-up, timed separately)
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(self.stream)
        B.cobs_build_summaries(self.cfg, self.kv, 0, wl.max_blocks, self.summ, self.ws)
        ev1.record(self.stream)
        torch.cuda.synchronize()
        self.build_ms = ev0.elapsed_time(ev1)
        self.check("cobs_build_summaries")

    def check(self, where):
        if self.B.cobs_read_status(self.ws) != 0:
            raise RuntimeError(f"device status after {where}")

    def step(self):
        self.B.cobs_decode_step(self.cfg, self.inp["q"], self.kv, self.summ, self.out, None, self.sel, self.cnt, self.ws)

    def timed(self, fn, n, flush):
        """n calls of fn, each bracketed by CUDA events on the launching stream, an L2 flush (not timed) before
        each.  Returns the per-call milliseconds."""
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for a, b_ in evs:
            if flush is not None:
                flush.zero_()
            a.record(self.stream)
            fn()
            b_.record(self.stream)
        torch.cuda.synchronize()
        return [a.elapsed_time(b_) for a, b_ in evs]

    def e2e_seconds(self, n, flush):
        """n calls of the host-buffer entry point (pinned host q in, host out back, synchronised): wall clock around
        each call alone; the L2 flush and its synchronise come before the clock starts."""
        B, wl = self.B, self.wl
        q_host = self.inp["q"].cpu().pin_memory()
        out_host = torch.zeros((wl.batch, wl.n_q_heads, wl.head_dim), dtype=torch.float32).pin_memory()
        for _ in range(2):
            B.cobs_decode_step_host(self.cfg, q_host, self.kv, self.summ, out_host, None, None, self.ws)
        total = 0.0
        for _ in range(n):
            if flush is not None:
                flush.zero_()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            B.cobs_decode_step_host(self.cfg, q_host, self.kv, self.summ, out_host, None, None, self.ws)
            total += time.perf_counter() - t0
        return total, q_host.numel() * 2, out_host.numel() * 4


def measure_other(B, name, dev, flush, peak, steps):
    """Step time of another named configuration on this GPU (fewer steps; same timing rules).  These workloads move
    11 - 106 MB per step, less than L2 holds: how L2 is emptied between steps matters, so the plain write flush is
    timed as well (it leaves part of the workload resident)."""
    wl = synth.named_workloads()[name]
    m = Measurement(B, wl, dev)
    for _ in range(5):
        flush.zero_()
        m.step()
    torch.cuda.synchronize()
    launches0 = B.cobs_kernel_launches()
    ms = m.timed(m.step, steps, flush)
    launches = B.cobs_kernel_launches() - launches0
    m.check("the timed steps")
    ms_write = m.timed(m.step, steps, flush.buf)            # the 256 MiB write alone
    e2e_s, _, _ = m.e2e_seconds(steps, flush)
    us = statistics.mean(ms) * 1e3
    gbs = m.step_bytes / (us * 1e-6) / 1e9
    return {"workload": name, "us_per_step": round(us, 2), "us_per_step_median": round(statistics.median(ms) * 1e3, 2),
            "us_per_step_write_only_flush": round(statistics.mean(ms_write) * 1e3, 2),
            "algorithmic_bytes_per_step": m.step_bytes, "achieved_gbs": round(gbs, 1), "frac": round(gbs / peak, 4),
            "e2e_us_per_step": round(e2e_s / steps * 1e6, 2), "kernels_per_step": launches / steps, "steps": steps,
            "build_summaries_ms": round(m.build_ms, 3),
            "hbm_time_us_at_peak": round(m.step_bytes / (peak * 1e9) * 1e6, 2)}


def run_phase_times(args):
    """Where the time of one step goes, from the library build that carries timing code (libcobs_timing.so):
    per-warp global-timer stamps at the phase boundaries, clock cycles per category inside the phases, and per
    unit the moments its scores were complete and its selection was published.  One JSON line; times in
    microseconds from the earliest warp's start.  Numbers of this build are not benchmark values."""
    import ctypes as C
    import numpy as np
    from paper_2607_09052_b200 import binding as B
    from paper_2607_09052_b200 import build as build_mod
    B.use_library(build_mod.build(timing=True))
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    wl = synth.named_workloads()[args.workload]
    if args.batch:
        wl = wl.replace(batch=args.batch)
    if args.seq_len:
        wl = wl.replace(seq_len=args.seq_len)
    m = Measurement(B, wl, dev)
    flush = L2Flush(dev, args.flush_mode)
    score_only = args.phase_times == "score"
    def step():
        if score_only:
            B.cobs_score_select(m.cfg, m.inp["q"], m.summ, m.inp["seq_lens"], m.sel, m.cnt, None, m.ws)
        else:
            m.step()
    for _ in range(5):
        flush.zero_()
        step()
    torch.cuda.synchronize()
    acc = (C.c_ulonglong * (8 * 4096))()
    B.lib().cobs_debug_acc(acc, 1)                          # clear the accumulators
    flush.zero_()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(m.stream)
    step()
    ev1.record(m.stream)
    torch.cuda.synchronize()
    buf = (C.c_ulonglong * (4 * 4096))()
    assert B.lib().cobs_debug_times(buf) == 0 and B.lib().cobs_debug_acc(acc, 1) == 0
    t = np.frombuffer(buf, dtype=np.uint64).reshape(4, 4096).astype(np.int64)
    n = int((t[0] > 0).sum())
    t = t[:, :n]
    t0 = int(t[0].min())
    raw = np.frombuffer(acc, dtype=np.uint64).reshape(8, 4096).astype(np.int64)
    mhz = 1965.0

    def stats(x):
        return {k: round(float(v), 2) for k, v in zip(("min", "p10", "p50", "p90", "max"),
                                                      [x.min(), *np.percentile(x, [10, 50, 90]), x.max()])}
    out = {"phase_times": True, "workload": wl.name, "mode": args.phase_times, "streaming_warps": n,
           "step_us_this_build": round(ev0.elapsed_time(ev1) * 1e3, 2),
           "warp_stamps_us": {name: stats((t[k] - t0) / 1e3) for k, name in
                              enumerate(["start", "scoring_done", "attention_start", "attention_done"])}}
    sc = raw[:, 1200:1200 + n].astype(np.float64) / mhz
    busy = sc.sum(0) > 0.5
    names_s = ["next position", "after issue", "wait for copies", "arithmetic", "epilogue", "issue copies", "seek", "fence + count"]
    out["scoring_us_per_working_warp"] = {nm: round(float(sc[k][busy].mean()), 2) for k, nm in enumerate(names_s)}
    out["scoring_working_warps"] = int(busy.sum())
    if not score_only:
        at = raw[:, :n].astype(np.float64) / mhz
        names_a = ["after the draw", "item set-up", "wait for selection", "group table + query", "stream loop",
                   "write partial + fence + count", "draw the next item", "merge (last closer of a unit)"]
        out["attention_us_per_warp"] = {nm: round(float(at[k].mean()), 2) for k, nm in enumerate(names_a)}
        late = np.argsort(t[3])[-8:]
        out["latest_warps"] = [{"warp": int(w), "attention_start": round(float((t[2][w] - t0) / 1e3), 1),
                                "attention_done": round(float((t[3][w] - t0) / 1e3), 1),
                                **{nm: round(float(at[k][w]), 1) for k, nm in enumerate(names_a)}} for w in late]
    nu = wl.batch * wl.n_kv_heads
    st = [(raw[k, 3000:3000 + min(nu, 1024)] - t0) / 1e3 for k in (0, 2, 3, 4, 5, 1)]
    out["selection_us"] = {"unit_scored_at": stats(st[0]), "unit_ready_at": stats(st[5]),
                           "duration": stats(st[5] - st[0]),
                           "parts_mean": {nm: round(float((st[i + 1] - st[i]).mean()), 2) for i, nm in
                                          enumerate(["loads + lse", "scores", "bisection", "compaction", "fence + flag"])}}
    out["status"] = B.cobs_read_status(m.ws)
    print(json.dumps(out), flush=True)


def run_launch_selftest(args):
    """The N-rank launch path without a GPU: every rank joins a gloo group, runs a stub step whose duration grows
    with the rank, and rank 0 prints the line with the real world size and the max-over-ranks time.  What
    tests/test_shard_gloo.py drives."""
    import torch.distributed as dist
    rank, local_rank, world = dist_env()
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    sys.stderr.write(f"bench.py: rank {rank} of {world} up (local rank {local_rank}, launch self-test, no GPU work)\n")
    wl = shard.rank_workload(synth.named_workloads()["cfg1_tiny"], rank)
    local_ms = args.steps * (1.0 + rank)                      # the last rank is the slow one
    total_ms, = shard.job_times([local_ms])
    if rank == 0:
        step_bytes = 1000
        print(json.dumps({"launch_selftest": True, "n_gpus": world, "steps": args.steps, "ms_per_step": total_ms / args.steps,
                          "value": shard.job_throughput(step_bytes, world, total_ms / args.steps * 1e-3),
                          "seed_rank0": wl.seed}), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_ours(args):
    from paper_2607_09052_b200 import binding as B
    from paper_2607_09052_b200 import build as build_mod

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the decode path has no CPU fallback")
    if local_rank >= torch.cuda.device_count():
        raise RuntimeError(f"rank {rank}: local rank {local_rank} has no GPU ({torch.cuda.device_count()} visible)")
    torch.cuda.set_device(local_rank)
    if rank == 0:
        build_mod.build()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    sys.stderr.write(f"bench.py: rank {rank} of {world} on cuda:{local_rank} ({torch.cuda.get_device_name(local_rank)})\n")
    B.lib()

    wl = synth.named_workloads()[args.workload]
    if args.batch:
        wl = wl.replace(batch=args.batch, name=f"{wl.name}[batch={args.batch}]")
    if args.seq_len:
        wl = wl.replace(seq_len=args.seq_len, name=f"{wl.name}[context={args.seq_len}]")
    if args.contiguous_pages:
        wl = wl.replace(shuffle_pages=False, name=f"{wl.name}[contiguous pages]")
    wl = shard.rank_workload(wl, rank)                  # every rank draws its own sequences
    dev = torch.device("cuda", local_rank)
    m = Measurement(B, wl, dev)
    cfg, inp, kv, summ, ws, out, sel, cnt, stream = m.cfg, m.inp, m.kv, m.summ, m.ws, m.out, m.sel, m.cnt, m.stream
    nb, hq, hkv, D = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
    record, step_bytes, build_ms = m.record, m.step_bytes, m.build_ms
    flush_buf = L2Flush(dev, args.flush_mode)
    flush = None if args.no_l2_flush else flush_buf
    step = m.step

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    t_warm = time.perf_counter()
    n_warm = 0
    while n_warm < args.warmup or time.perf_counter() - t_warm < args.clock_warm_s:   # >= W steps, and long enough for clock samples
        if flush is not None:
            flush.zero_()
        step()
        n_warm += 1
        if n_warm % 16 == 0:
            torch.cuda.synchronize()
    barrier()

    # ---- timed region: exactly K steps, an L2 flush (not timed) before each ----------------------------
    launches0 = B.cobs_kernel_launches()
    t_wall0 = time.perf_counter()
    step_ms = m.timed(step, args.steps, flush)
    barrier()
    wall_s = time.perf_counter() - t_wall0
    launches = B.cobs_kernel_launches() - launches0
    clocks = sampler.stop() if sampler else None
    total_ms = sum(step_ms)
    m.check("the timed steps")

    # ---- the two halves of the step through their own entry points (context for the roofline line) ----
    n_sub = max(3, min(args.steps, 20))
    score_ms = statistics.mean(m.timed(lambda: B.cobs_score_select(cfg, inp["q"], summ, inp["seq_lens"], sel, cnt, None, ws),
                                       n_sub, flush_buf))
    attend_ms = statistics.mean(m.timed(lambda: B.cobs_sparse_decode(cfg, inp["q"], kv, sel, cnt, out, None, ws),
                                        n_sub, flush_buf))
    summary_bytes = m.summary_bytes
    kv_bytes = step_bytes - summary_bytes

    # ---- end to end through the host-buffer entry point ------------------------------------------------
    barrier()
    e2e_s, h2d_bytes, d2h_bytes = m.e2e_seconds(args.steps, flush_buf)

    # ---- optional: consecutive decode steps (append a token, rebuild a block's summary when it fills, step) ----
    loop_info = None
    if args.decode_loop > 0:
        from paper_2607_09052_b200.decode_loop import DecodeLoop
        n_loop = args.decode_loop
        start_len = wl.seq_len - n_loop - 7                  # not a multiple of the block size; ends below capacity
        inp["seq_lens"].fill_(start_len)
        loop = DecodeLoop(wl.replace(seq_lens=[start_len] * nb), inp, summ=summ, ws=ws)
        gen = torch.Generator(device=dev).manual_seed(1234)
        pool = [(torch.randn((nb, hq, D), generator=gen, device=dev).to(torch.bfloat16),
                 torch.randn((nb, hkv, D), generator=gen, device=dev).to(torch.bfloat16),
                 torch.randn((nb, hkv, D), generator=gen, device=dev).to(torch.bfloat16)) for _ in range(8)]
        ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev_a.record(stream)
        for i in range(n_loop):
            q_i, k_i, v_i = pool[i % len(pool)]
            loop.step(q_i, k_i, v_i, out, None, sel, cnt)
        ev_b.record(stream)
        torch.cuda.synchronize()
        m.check("the decode loop")
        loop_info = {"steps": n_loop, "start_len": start_len, "rebuilds": loop.rebuilds,
                     "us_per_step_amortised": round(ev_a.elapsed_time(ev_b) * 1e3 / n_loop, 2),
                     "note": "append + summary rebuild of the block that filled (one launch per block boundary, all "
                             "sequences) + fused step, back to back on one stream, no L2 flush between steps"}

    total_ms, e2e_s = shard.job_times([total_ms, e2e_s], device=dev)   # the job is as slow as its slowest rank
    ms_per_step = total_ms / args.steps
    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    peak, peak_kind = read_peaks()
    value = world * step_bytes / (ms_per_step * 1e-3) / 1e9
    # the step is ONE launch of the persistent kernel, so its launch duration is the step time
    kernels_per_step = launches / args.steps
    achieved = step_bytes / (ms_per_step * 1e-3) / 1e9 if world == 1 else value / world
    line = {
        "metric": "fused COBS decode step: achieved HBM GB/s (algorithmic bytes per step / step time)",
        "value": round(value, 2), "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(ms_per_step, 6), "us_per_step": round(ms_per_step * 1e3, 3),
        "us_per_step_median": round(statistics.median(step_ms) * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "batch_per_gpu": nb, "global_batch": nb * world, "context": wl.seq_len,
                   "n_q_heads": hq, "n_kv_heads": hkv, "head_dim": D, "block_size": wl.block_size,
                   "page_size": wl.page_size, "topk": wl.topk, "window": wl.window, "rank": wl.rank,
                   "sub_dim": wl.sub_dim, "summary_dtype": wl.summary_dtype, "scale_dtype": wl.scale_dtype,
                   "record_bytes": record, "algorithmic_bytes_per_step": step_bytes,
                   "l2": ("no flush (the step's own traffic exceeds L2); " if args.no_l2_flush else flush_buf.describe() + "; ") +
                         f"step traffic {step_bytes / 2**20:.1f} MiB",
                   "sharding": "independent sequences per rank, no collective"},
        "frac_of_measured_peak": round(value / (world * peak), 4), "peak_gbs": peak, "peak_kind": peak_kind,
        "frac_of_nominal_8tbs": round(value / (world * 8000.0), 4),
        "roofline": {"bound": "hbm", "kernel": "fused_step_kernel (scoring + selection + attention + merge)",
                     "achieved": round(achieved, 2), "peak": peak, "unit": "GB/s", "frac": round(achieved / peak, 4),
                     "traffic": TRAFFIC_BYTES.get(wl.name), "algorithmic_bytes": step_bytes,
                     "launch_ms": round(ms_per_step, 6), "kernels_per_step": kernels_per_step,
                     "note": f"of {peak_kind} (copy bandwidth); the same kernel run for one half of the step alone: "
                             f"scoring + selection {score_ms * 1e3:.1f} us for {summary_bytes} B, attention "
                             f"{attend_ms * 1e3:.1f} us for {kv_bytes} B; traffic = DRAM bytes per launch from the ncu "
                             f"capture summarised under profiles/ (null when not captured for this workload)"},
        "e2e": {"value": round(world * step_bytes / (e2e_s / args.steps) / 1e9, 2), "unit": "GB/s",
                "us_per_step": round(e2e_s / args.steps * 1e6, 2),
                "h2d_bytes_per_step": h2d_bytes, "d2h_bytes_per_step": d2h_bytes,
                "note": "cobs_decode_step_host: pinned host q copied in, step, output written to pinned host memory, "
                        "stream synchronised; wall clock around each call alone"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "build_summaries_ms": round(build_ms, 3),
        "wall_s_timed_region": round(wall_s, 4),
    }
    if loop_info:
        line["decode_loop"] = loop_info
    if world == 1 and not args.no_other_workloads and args.workload == DEFAULT_WORKLOAD and not (args.batch or args.seq_len):
        del m, step, inp, kv, summ, ws, out, sel, cnt
        torch.cuda.empty_cache()
        line["other_workloads"] = [measure_other(B, name, dev, flush_buf, peak, args.other_steps) for name in OTHER_WORKLOADS]
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(wl, record, budget_s=20.0)
    print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------------------------------
# CPU baseline / reference arm: the oracle as it stands, on the host cores, on a bounded sample.
# ----------------------------------------------------------------------------------------------------------

def oracle_sample(wl: synth.Workload, n_units: int):
    """Inputs and oracle-built summaries for the first n_units (sequence 0, KV heads 0..) of a workload
    reduced to one sequence (same shapes per unit as the full workload)."""
    from oracle import cobs_oracle as O
    small = wl.replace(batch=1, seq_lens=None)
    inp = synth.generate(small, "cpu")
    units = []
    for h in range(min(n_units, small.n_kv_heads)):
        K, V = synth.unit_kv(inp, small, 0, h)
        q = synth.unit_q(inp, small, 0, h).numpy()
        u_q = inp["u_q"][h].double().numpy() if small.sub_dim else None
        mean, xi, _ = O.build_summaries(K.numpy(), small.block_size, small.rank, u_q)
        st = O.store_summaries(mean, xi, small.summary_dtype, small.scale_dtype)
        units.append((q, K.numpy(), V.numpy(), st, u_q))
    return small, units


def oracle_time_steps(small, units, repeats: int):
    from oracle import cobs_oracle as O
    t0 = time.perf_counter()
    for _ in range(repeats):
        for q, K, V, st, u_q in units:
            O.decode_step(q, K, V, small.seq_len, st, small.block_size, small.topk, small.window, u_q)
    return time.perf_counter() - t0


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(wl, record, budget_s: float):
    n_units = 2
    small, units = oracle_sample(wl, n_units)
    one = oracle_time_steps(small, units, 1)
    repeats = max(1, min(5000, int(budget_s / max(one, 1e-6))))
    elapsed = oracle_time_steps(small, units, repeats)
    unit_bytes = algorithmic_bytes(small, record) / small.n_kv_heads
    gbs = repeats * len(units) * unit_bytes / elapsed / 1e9
    return {"value": round(gbs, 4), "unit": "GB/s", "cores": host_threads(), "kind": "oracle",
            "sample": f"{len(units)} (sequence, KV head) units of {wl.name} x {repeats} repeats, "
                      f"score + select + attend per unit (summaries prebuilt), {elapsed:.1f} s",
            "us_per_step_extrapolated": round(elapsed / (repeats * len(units)) * wl.batch * wl.n_kv_heads * 1e6, 1)}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    wl = synth.named_workloads()[args.workload]
    mb = wl.head_dim * (4 if wl.summary_dtype == "fp32" else 2)
    ds = wl.sub_dim or wl.head_dim
    if wl.summary_dtype == "fp4":
        pad = (ds + 7) // 8 * 8
        while wl.rank and (wl.rank * pad // 2) % 16:
            pad += 8
        record = mb + wl.rank * pad // 2 + wl.rank * (2 if wl.scale_dtype == "fp16" else 4)
    else:
        record = mb + wl.rank * ds * (4 if wl.summary_dtype == "fp32" else 2)
    small, units = oracle_sample(wl, 2)
    for _ in range(args.warmup):
        oracle_time_steps(small, units, 1)
    times = [oracle_time_steps(small, units, 1) for _ in range(args.steps)]
    per_step_s = sum(times) / len(times)
    unit_bytes = algorithmic_bytes(small, record) / small.n_kv_heads
    gbs = len(units) * unit_bytes / per_step_s / 1e9
    sample = f"each step = {len(units)} (sequence, KV head) units of {wl.name} (of {wl.batch * wl.n_kv_heads}), " \
             f"score + select + attend by the CPU oracle, summaries prebuilt"
    line = {"impl": "reference",
            "metric": "fused COBS decode step: achieved HBM GB/s (algorithmic bytes per step / step time)",
            "value": round(gbs, 4), "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(per_step_s * 1e3, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "context": wl.seq_len, "sample": sample},
            "cpu_baseline": {"value": round(gbs, 4), "unit": "GB/s", "kind": "oracle", "cores": host_threads(),
                             "sample": sample},
            "e2e": {"value": round(gbs, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.named_workloads()))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling on a small case)")
    ap.add_argument("--seq-len", type=int, default=0, help="override the workload's context (profiling on a small case)")
    ap.add_argument("--contiguous-pages", action="store_true",
                    help="diagnostic: identity page table instead of the workload's shuffled pages")
    ap.add_argument("--no-l2-flush", action="store_true",
                    help="do not write 256 MiB between timed steps (valid only where the step's own traffic exceeds L2)")
    ap.add_argument("--flush-mode", default="write+read", choices=["write", "write+read"],
                    help="how L2 is flushed between timed steps (see L2Flush)")
    ap.add_argument("--decode-loop", type=int, default=0,
                    help="also time this many consecutive decode steps (append, rebuild on block fill, step) and "
                         "report the amortised time per step")
    ap.add_argument("--clock-warm-s", type=float, default=0.6,
                    help="keep warming up at least this long so that the clock sampler has samples")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the other named configurations (the `other_workloads` list of the line)")
    ap.add_argument("--other-steps", type=int, default=20, help="timed steps per other configuration")
    ap.add_argument("--phase-times", nargs="?", const="step", default=None, choices=["step", "score"],
                    help="diagnostic, one GPU: run the timing build of the library and print where the time of one step "
                         "(or of cobs_score_select alone) goes; not a benchmark value")
    ap.add_argument("--launch-selftest", action="store_true",
                    help="no GPU work: bring the N ranks up on gloo, run a stub step, print the line (tests the launch path)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if not args.phase_times:
        ensure_ranks(args)
    if args.phase_times:
        run_phase_times(args)
    elif args.launch_selftest:
        run_launch_selftest(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
