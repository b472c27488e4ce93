#!/usr/bin/env python
"""Benchmark of the shared-prefix decode-attention step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

One "step" is one pass of the whole hot path over the workload: append one token per candidate (for
the configurations that sweep appends), prefix pass, suffix pass, merge.  The metric is the unique
K/V + Q + O (+LSE) bytes of a step divided by its device time, in GB/s.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2601_05475_b200 import workload as wl  # noqa: E402

METRIC = "decode_attn_unique_kv_gbs"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of the dominant kernel relative to its algorithmic bytes (dram__bytes_read.sum +
# dram__bytes_write.sum per launch, one ncu capture per regime: chunks of a few hundred tokens as on cfg2, and
# 4096-token chunks on a small problem of cfg4's shape; the traffic grows in proportion to the tokens streamed,
# so the ratio is scaled by the units of the timed workload).  A ratio is only reported while the kernel source
# still has the hash it had when the counters were taken.
SUFFIX_TRAFFIC_RATIO = {"short_chunks": 1.0122, "long_chunks": 1.0024}
SUFFIX_KERNEL_SHA1 = "b1c5d052742adae3d483a7572013b2a9de2a4403"


def suffix_traffic(algorithmic_bytes, suffix_part_tokens):
    import hashlib
    ratio = SUFFIX_TRAFFIC_RATIO["long_chunks" if suffix_part_tokens >= 2048 else "short_chunks"]
    if ratio is None:
        return None
    src = os.path.join(ROOT, "paper_2601_05475_b200", "csrc", "mc_suffix_tma.cu")
    try:
        if hashlib.sha1(open(src, "rb").read()).hexdigest() != SUFFIX_KERNEL_SHA1:
            return None
    except OSError:
        return None
    return algorithmic_bytes * ratio


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f), "measured"
    except Exception:
        return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


# ---------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------------
def host_rows(cfg: wl.Config, rows):
    """Logical K/V histories of the sampled (b, hq) rows, drawn on the host with the workload's
    distributions (lengths are the workload's own draws)."""
    prefix_len, suffix_len = wl.draw_lengths(cfg)
    q_all = wl.draw_q(cfg, 0)
    out = []
    for i, (b, hq) in enumerate(rows):
        j = b // cfg.C
        n = int(prefix_len[j]) + int(suffix_len[b])
        k, v = wl.draw_single_head_history(cfg, i, n)
        out.append((q_all[b, hq], k, v))
    return out, prefix_len, suffix_len


def time_oracle(cfg: wl.Config, n_rows: int, repeats: int = 1):
    """Times oracle.attend over n_rows sampled rows on the host cores; returns (seconds per repeat list,
    cores used, bytes-equivalent of the sample in the metric's accounting)."""
    from concurrent.futures import ThreadPoolExecutor

    from oracle import attention as orc
    import contextlib
    try:
        from threadpoolctl import threadpool_limits
        blas_one_thread = lambda: threadpool_limits(limits=1)
    except Exception:  # pragma: no cover
        blas_one_thread = contextlib.nullcontext
    rng = np.random.default_rng(12345)
    rows = [(int(rng.integers(cfg.B)), int(rng.integers(cfg.Hq))) for _ in range(n_rows)]
    data, prefix_len, suffix_len = host_rows(cfg, rows)
    cores = max(1, min(os.cpu_count() or 1, n_rows))
    ub = wl.unique_bytes(cfg, prefix_len, suffix_len)
    # A whole step is B*Hq rows; the sample's share of the step's unique bytes is n_rows / (B*Hq).
    sample_bytes = ub["total"] * n_rows / float(cfg.B * cfg.Hq)

    def one(item):
        q, k, v = item
        return orc.attend(q, k, v, cfg.scale)[1]

    times = []
    with blas_one_thread(), ThreadPoolExecutor(max_workers=cores) as ex:
        for _ in range(repeats):
            t0 = time.perf_counter()
            list(ex.map(one, data))
            times.append(time.perf_counter() - t0)
    return times, cores, sample_bytes


def oracle_sample_rows(cfg: wl.Config) -> int:
    """Rows whose fp64 attention costs roughly 10-20 s of CPU work in total."""
    prefix_len, suffix_len = wl.draw_lengths(cfg)
    mean_n = float(prefix_len.mean() + suffix_len.mean())
    per_row_s = max(1e-4, mean_n * cfg.d * 1.2e-8)          # ~12 ns per (token, channel) for convert + 2 gemv + exp
    return int(max(8, min(cfg.B * cfg.Hq, 12.0 / per_row_s)))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    cfg = wl.CONFIGS[args.workload]
    n_rows = max(8, oracle_sample_rows(cfg) // 4)
    times, cores, sample_bytes = time_oracle(cfg, n_rows, repeats=args.warmup + args.steps)
    timed = times[args.warmup:]
    sec = sum(timed) / len(timed)
    value = sample_bytes / sec / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "sample": "%d of %d (candidate, head) rows per step" % (n_rows, cfg.B * cfg.Hq)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "%d of %d rows of %s, fp64 numpy, one thread per row" % (n_rows, cfg.B * cfg.Hq, cfg.name)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------------------------------------------
# multi-process aggregation (replicas only: no data-path collective; ranks only agree on the time)
# ---------------------------------------------------------------------------------------------------
def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks of the default process group (identity when
    no group is initialised).  The step time of the job is the slowest rank's."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def aggregate_value(bytes_per_replica_step, ms_per_step, world):
    """Whole-job metric of `world` independent replicas that each move bytes_per_replica_step per step."""
    return world * bytes_per_replica_step / (ms_per_step * 1e-3) / 1e9


def free_port() -> int:
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        return so.getsockname()[1]


def spawn_replicas(n: int, argv, extra_env=None, script=None) -> int:
    """`bench.py --gpus N` started as ONE process: starts N workers of this same script (or of `script`), one per
    GPU, with the environment a torchrun launch would give them (rank 0 prints the line); returns the first
    non-zero exit code."""
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable, script or os.path.abspath(__file__)] + list(argv), env=env))
    rc = 0
    for p in procs:
        p.wait()
        rc = rc or p.returncode
    return rc


def timed_blocks(run_block, sync, steps, min_seconds, max_blocks):
    """Runs `run_block(block_index)` (which enqueues `steps` steps between two events and returns them) until
    `min_seconds` of device time have been timed or `max_blocks` blocks have run; returns the per-block
    milliseconds.  `sync` is the barrier + device synchronisation on both sides of every block."""
    ms = []
    while len(ms) < max_blocks and (not ms or sum(ms) * 1e-3 < min_seconds):
        sync()
        e0, e1 = run_block(len(ms))
        sync()
        ms.append(e0.elapsed_time(e1))
    return ms


# ---------------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.idx = device_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_2601_05475_b200 import binding as mc
    from paper_2601_05475_b200.harness import device_append, device_q, make_device_problem

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    mc.lib()  # fail loudly here if the extension is missing

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def agree_seconds(x):
        # every rank must run the same number of blocks (each block has a barrier): the ranks time different
        # things, so the target is turned into "never stop on time" for N > 1 and the block cap decides
        return x if world == 1 else (1e9 if x > 0 else 0.0)

    def measure(name, steps, warmup, want_kernel_split, outer=(), min_seconds=0.0, max_timed_steps=None):
        """Blocks of `steps` steps, each between a barrier + synchronize and timed with two events on the launching
        stream, repeated until `min_seconds` have been timed (at most `max_timed_steps` steps in all, so that the
        appends do not move the workload away from the configuration); the step time is the median block's."""
        cfg = wl.CONFIGS[name]
        appends = cfg.append_steps > 0
        if max_timed_steps is None:
            max_timed_steps = 640 if appends else 4000
        max_blocks = max(1, max_timed_steps // steps)
        total_steps = warmup + max_blocks * steps + 16
        dp = make_device_problem(cfg, headroom_tokens=total_steps + 1 if appends else 1, outer=outer)
        stream = torch.cuda.current_stream().cuda_stream
        qs = [device_q(cfg, i) for i in range(4)]
        kv = [device_append(cfg, i) for i in range(4)] if appends else None
        len0 = dp.suffix_len.clone()
        ub0 = wl.unique_bytes(cfg, dp.prefix_len.cpu().numpy(), len0.cpu().numpy())
        per_tok = 2 * cfg.Hkv * cfg.d * cfg.kv_elem_bytes + (2 * cfg.Hkv * 4 / wl.PAGE if cfg.dtype == "fp8" else 0)
        outer_tokens = sum(int(np.sum(lens)) for (_, lens) in outer)          # each outer token is unique once
        ub0["total"] += outer_tokens * per_tok

        def step(i):
            mc.mc_decode_step(dp.layout, kv[i % 4][0] if appends else None, kv[i % 4][1] if appends else None,
                              qs[i % 4], cfg.scale, dp.o, dp.lse, dp.ws_ptr, dp.ws_bytes, stream)

        for i in range(warmup):
            step(i)
        barrier()
        sampler = ClockSampler(torch.cuda.current_device())
        if rank == 0 and min_seconds > 0:
            sampler.start()
        n0 = mc.mc_launch_count()

        def run_block(blk):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps):
                step(warmup + blk * steps + i)
            e1.record()
            return e0, e1

        block_ms = timed_blocks(run_block, barrier, steps, agree_seconds(min_seconds), max_blocks)
        launches = (mc.mc_launch_count() - n0) // len(block_ms)
        clocks = sampler.stop() if (rank == 0 and min_seconds > 0) else None
        if mc.mc_get_last_status(dp.layout) != mc.MC_OK:
            raise RuntimeError("device status word reports an error")
        # the median block (lower median: a block that was really run) and the bytes of ITS average step (suffixes
        # grow by one token per step when appending)
        order = sorted(range(len(block_ms)), key=lambda i: block_ms[i])
        mid = order[(len(order) - 1) // 2]
        ms = block_ms[mid] / steps
        grow = (warmup + mid * steps + (steps + 1) / 2.0) * cfg.B * per_tok if appends else 0.0
        step_bytes = ub0["total"] + grow + (2 * cfg.B * cfg.Hkv * cfg.d * cfg.elem_bytes if appends else 0)
        res = {"ms": ms, "bytes": step_bytes, "launches": launches, "clocks": clocks, "cfg": cfg,
               "blocks": len(block_ms), "block_ms_min": min(block_ms) / steps, "block_ms_max": max(block_ms) / steps,
               "prefix_ctas": int(dp.geom.prefix_ctas), "n_parts": int(dp.geom.n_parts),
               "n_prefix_parts": int(dp.geom.n_prefix_parts), "suffix_part_tokens": int(dp.geom.suffix_part_tokens)}

        # what making the layout object costs on the host (it reads lengths back, plans both passes, encodes the
        # tensor maps and allocates its small device state): median of five create / destroy pairs
        if not outer:
            t_create = []
            for _ in range(5):
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                h = mc.mc_kv_layout_create(dp.desc)
                t_create.append((time.perf_counter() - t0) * 1e3)
                mc.mc_kv_layout_destroy(h)
            res["layout_create_ms"] = statistics.median(t_create)

        # end to end through the host-buffer entry point: pinned host q / k_new / v_new in, o / lse out
        pin = lambda t: t.cpu().pin_memory()
        hq = [pin(x) for x in qs]
        hkv = [(pin(a), pin(b)) for a, b in kv] if appends else None
        ho = torch.empty(dp.o.shape, dtype=dp.o.dtype).pin_memory()
        hl = torch.empty(dp.lse.shape, dtype=torch.float32).pin_memory()
        e2e_steps = max(3, min(steps, 10))

        def host_step(i):
            mc.mc_decode_step_host(dp.layout, hkv[i % 4][0] if appends else None, hkv[i % 4][1] if appends else None,
                                   hq[i % 4], cfg.scale, ho, hl, dp.ws_ptr, dp.ws_bytes, stream)

        host_step(0)
        barrier()
        t0 = time.perf_counter()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(e2e_steps):
            host_step(1 + i)
        e1.record()
        barrier()
        wall_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
        res["e2e_ms"] = max(e0.elapsed_time(e1) / e2e_steps, wall_ms if world == 1 else 0.0)
        res["h2d"] = hq[0].numel() * hq[0].element_size() + (2 * hkv[0][0].numel() * hkv[0][0].element_size() if appends else 0)
        res["d2h"] = ho.numel() * ho.element_size() + hl.numel() * 4

        if want_kernel_split:
            # the dominant kernel alone, on the launching stream, same data
            g = dp.geom
            lse_off = (g.rows * g.n_parts * g.head_dim * 4 + 255) // 256 * 256
            o_ptr, l_ptr = dp.ws_ptr, dp.ws_ptr + lse_off
            for fn_name, fn in (("suffix", mc.mc_suffix_attn), ("prefix", mc.mc_prefix_attn)):
                for _ in range(3):
                    fn(dp.layout, qs[0], cfg.scale, o_ptr, l_ptr, stream)
                torch.cuda.synchronize()
                k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                k0.record()
                for i in range(steps):
                    fn(dp.layout, qs[i % 4], cfg.scale, o_ptr, l_ptr, stream)
                k1.record()
                torch.cuda.synchronize()
                res[fn_name + "_ms"] = k0.elapsed_time(k1) / steps
            cur = dp.suffix_len.cpu().numpy().astype(np.int64)
            res["suffix_bytes"] = float(cur.sum()) * per_tok
            res["prefix_bytes"] = (float(dp.prefix_len.cpu().numpy().astype(np.int64).sum()) + outer_tokens) * per_tok
            res["prefix_flops"] = 4.0 * cfg.Hq * cfg.d * (float(
                (dp.prefix_len.cpu().numpy().astype(np.int64) * cfg.C).sum()) + sum(
                float(np.sum(np.asarray(lens, dtype=np.int64) * np.diff(np.asarray(go, dtype=np.int64))))
                for (go, lens) in outer))
        dp.close()
        del dp
        torch.cuda.empty_cache()
        return res

    def measure_prefix_cold(name, steps, warmup, copies=6):
        """The same step with the shared prefix NOT left in L2 by the step before: `copies` independent instances of
        the configuration (own pools, own tables) take turns, so that between two steps on one instance the others
        have streamed several times the L2 capacity, their own evict-last prefix lines included - what a decode
        loop over the layers of a model does to one layer's prefix.  No appends (the lengths stay at step 0)."""
        cfg = wl.CONFIGS[name]
        dps = [make_device_problem(cfg, headroom_tokens=1) for _ in range(copies)]      # same lengths, own memory
        stream = torch.cuda.current_stream().cuda_stream
        qs = [device_q(cfg, i) for i in range(4)]
        per_tok = 2 * cfg.Hkv * cfg.d * cfg.elem_bytes
        total = sum(wl.unique_bytes(cfg, dp.prefix_len.cpu().numpy(), dp.suffix_len.cpu().numpy())["total"] for dp in dps)

        def step(i):
            dp = dps[i % copies]
            mc.mc_decode_step(dp.layout, None, None, qs[i % 4], cfg.scale, dp.o, dp.lse, dp.ws_ptr, dp.ws_bytes, stream)

        for i in range(max(warmup, copies)):
            step(i)
        barrier()
        n = (steps + copies - 1) // copies * copies          # every instance equally often
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n):
            step(i)
        e1.record()
        barrier()
        ms = e0.elapsed_time(e1) / n
        for dp in dps:
            dp.close()
        del dps
        torch.cuda.empty_cache()
        return {"ms_per_step": ms, "gbs": total / copies / (ms * 1e-3) / 1e9, "instances": copies}

    def measure_read_peak():
        """Read-only streaming rate of this GPU: the library's probe kernel over 4 GiB (33 x L2), best of 5."""
        n = 4 << 30
        buf = torch.empty(n, dtype=torch.uint8, device="cuda")
        buf.zero_()
        sink = torch.zeros(1, dtype=torch.int32, device="cuda")
        stream = torch.cuda.current_stream().cuda_stream
        best = 0.0
        for i in range(7):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            mc.mc_hbm_read_probe(buf, n, sink, stream)
            e1.record()
            torch.cuda.synchronize()
            if i >= 2:
                best = max(best, n / (e0.elapsed_time(e1) * 1e-3) / 1e9)
        del buf
        torch.cuda.empty_cache()
        return best

    def measure_search():
        """The search bookkeeping on 2^17 problems x 8 trajectories x 8 steps (Section 3.1: K = 8, depth 8): one pass
        = rewards / best-so-far / value targets / labels / returns (mc_search_returns), then value head, selection of
        tau* and of the state to expand in one launch (mc_search_select).  Algorithmic bytes per (trajectory, step):
        5 read + 10 written; per trajectory 4 (length) + 4 (return, written) + 20 (logits) + 4 (expected) + 4 (return,
        read by the selection)."""
        b = wl.draw_search_batch(problems=1 << 17, K=8, T=8, seed=0)
        N, T, P = b["N"], b["T"], b["P"]
        dev = lambda a: torch.from_numpy(a).cuda()
        sp, ok, ln, lg, go = dev(b["speedup"]), dev(b["correct"]), dev(b["len"]), dev(b["logits"]), dev(b["group_offsets"])
        r = torch.empty((T, N), dtype=torch.uint8, device="cuda")
        lab = torch.empty_like(r)
        u, v = torch.empty((T, N), device="cuda"), torch.empty((T, N), device="cuda")
        G, ev = torch.empty(N, device="cuda"), torch.empty(N, device="cuda")
        best_t, best_s = (torch.empty(P, dtype=torch.int32, device="cuda") for _ in range(2))
        s1, s2, s3 = wl.SEARCH_THRESHOLDS
        stream = torch.cuda.current_stream().cuda_stream

        def returns():
            mc.mc_search_returns(sp, ok, ln, N, T, s1, s2, s3, 0.95, r, u, v, lab, G, stream)

        def select():
            mc.mc_search_select(lg, G, go, P, None, ev, best_t, best_s, stream)

        def one():
            returns()
            select()

        def timed(fn, reps=10):
            for _ in range(3):
                fn()
            total = 0.0
            for _ in range(reps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn()
                e1.record()
                torch.cuda.synchronize()
                total += e0.elapsed_time(e1)
            return total / reps

        ms, ms_returns, ms_select = timed(one), timed(returns), timed(select)
        nbytes = N * T * 15 + N * (4 + 4 + 20 + 4 + 4) + 2 * P * 8
        return {"trajectories": N, "steps": T, "ms": round(ms, 5), "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
                "launches": 2, "ms_returns_alone": round(ms_returns, 5), "ms_select_alone": round(ms_select, 5),
                "gbs_returns_alone": round((N * T * 15 + N * 8) / (ms_returns * 1e-3) / 1e9, 1),
                "algorithmic_bytes": nbytes, "trajectory_steps_per_s": round(N * T / (ms * 1e-3), 1),
                "l2": "arrays of one pass (170 MB) larger than L2, no flush"}

    def measure_scoring():
        """Scoring of whole candidates by the value model's attention (Section 2.3): 4 problems x 8 candidates x 512
        tokens behind a 4096-token prompt, every token a query, causal inside the candidate; Hq 32 / Hkv 8 / d 128.
        One pass = mc_decode_attn on the cascade layout (prompt level + own-token level with row limits)."""
        from paper_2601_05475_b200.harness import ScoringDeviceProblem, to_device
        scfg = wl.Config("scoring", "bf16", 4, 8, 32, 8, 128, ("fixed", 4096), ("fixed", (0,)), permute_pages=True)
        seq_len = [512] * scfg.B
        hp = wl.make_scoring_host_problem(scfg, [4096] * scfg.G, seq_len)
        dp = ScoringDeviceProblem(hp)
        q = to_device(scfg, np.concatenate(wl.draw_scoring_q(scfg, seq_len), axis=0))
        stream = torch.cuda.current_stream().cuda_stream
        for _ in range(3):
            dp.score(q, stream)
        torch.cuda.synchronize()
        reps = 10
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches = mc.mc_launch_count()
        e0.record()
        for _ in range(reps):
            dp.score(q, stream)
        e1.record()
        torch.cuda.synchronize()
        launches = (mc.mc_launch_count() - launches) // reps
        ms = e0.elapsed_time(e1) / reps
        ok = mc.mc_get_last_status(dp.layout) == mc.MC_OK
        seen = sum(n * 4096 + n * (n + 1) // 2 for n in seq_len)               # (query, key) pairs that are not masked
        flops = 4.0 * scfg.Hq * scfg.d * seen
        ctas, n_parts, nv = int(dp.geom.prefix_ctas), int(dp.geom.n_parts), dp.n_virtual
        dp.close()
        return {"sequences": scfg.B, "tokens_per_sequence": 512, "prompt_tokens": 4096, "queries": nv, "ms": round(ms, 4),
                "tflops": round(flops / (ms * 1e-3) / 1e12, 1), "flops": flops, "prefix_ctas": ctas, "n_parts": n_parts,
                "launches_per_pass": int(launches), "scored_tokens_per_s": round(nv / (ms * 1e-3), 1), "status_ok": ok}

    def measure_qkv():
        """The decode layer's step in front of the attention (q/k/v projection + rotary embedding + append, fused):
        configuration 4's 128 candidates, Hq 64 / Hkv 8 / d 128 and a hidden size of 8192 (the width of the 70B-class
        models those head counts belong to): 168 MB of weights per call, streamed once.  Bytes = weights + hidden
        states + the bf16 rows written; the plain library GEMM of the same shape (torch.matmul, no rotation, no
        append) is timed beside it for context."""
        qcfg = wl.scaled_down(wl.CONFIGS["cfg4"], "qkv", prefix=("fixed", 64), suffix=("fixed", (0,)), append_steps=0)
        hidden, reps = 8192, 100
        n = (qcfg.Hq + 2 * qcfg.Hkv) * qcfg.d
        dp = make_device_problem(qcfg, headroom_tokens=4 * reps)
        gen = torch.Generator(device="cuda")
        gen.manual_seed(1234)
        w = (torch.randn(n, hidden, device="cuda", generator=gen) * hidden ** -0.5).to(torch.bfloat16)
        xs = [torch.randn(qcfg.B, hidden, device="cuda", generator=gen).to(torch.bfloat16) for _ in range(4)]
        q_out = torch.empty(qcfg.B, qcfg.Hq, qcfg.d, dtype=torch.bfloat16, device="cuda")
        plan = mc.mc_qkv_plan_create(dp.layout, w, None, hidden)
        stream = torch.cuda.current_stream().cuda_stream
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def timed(fn):
            for i in range(5):
                fn(i)
            torch.cuda.synchronize()
            e0.record()
            for i in range(reps):
                fn(i)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / reps

        launches = mc.mc_launch_count()
        ms = timed(lambda i: mc.mc_qkv_append(plan, xs[i % 4], q_out, None, 500000.0, stream))
        launches = (mc.mc_launch_count() - launches) // (reps + 5)
        ok = mc.mc_get_last_status(dp.layout) == mc.MC_OK
        y = torch.empty(qcfg.B, n, dtype=torch.bfloat16, device="cuda")
        ms_lib = timed(lambda i: torch.matmul(xs[i % 4], w.t(), out=y))
        pieces, ctas, ws = mc.mc_qkv_plan_geometry(plan)
        mc.mc_qkv_plan_destroy(plan)
        dp.close()
        nbytes = n * hidden * 2 + qcfg.B * hidden * 2 + qcfg.B * n * 2
        return {"candidates": qcfg.B, "hidden": hidden, "features": n, "ms": round(ms, 5),
                "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1), "tflops": round(2.0 * qcfg.B * n * hidden / (ms * 1e-3) / 1e12, 1),
                "algorithmic_bytes": nbytes, "launches": int(launches), "ctas": ctas, "pieces": pieces,
                "workspace_bytes": ws, "status_ok": ok, "library_gemm_alone_ms": round(ms_lib, 5),
                "l2": "weights (168 MB) larger than L2, no flush"}

    if args.qkv_only:          # profiling aid: only the fused projection, one small JSON line
        if rank == 0:
            print(json.dumps({"qkv_projection": measure_qkv()}))
        return 0

    if args.pass_only:         # profiling aid: one pass alone on the launching stream, one small JSON line
        cfg = wl.CONFIGS[args.workload]
        if args.kv_dtype:
            import dataclasses
            cfg = dataclasses.replace(cfg, dtype=args.kv_dtype)
        dp = make_device_problem(cfg, headroom_tokens=1)
        g = dp.geom
        lse_off = (g.rows * g.n_parts * g.head_dim * 4 + 255) // 256 * 256
        fn = {"suffix": mc.mc_suffix_attn, "prefix": mc.mc_prefix_attn}[args.pass_only]
        q, stream = device_q(cfg, 0), torch.cuda.current_stream().cuda_stream
        for _ in range(args.warmup):
            fn(dp.layout, q, cfg.scale, dp.ws_ptr, dp.ws_ptr + lse_off, stream)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            fn(dp.layout, q, cfg.scale, dp.ws_ptr, dp.ws_ptr + lse_off, stream)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.steps
        tokens = float((dp.suffix_len if args.pass_only == "suffix" else dp.prefix_len).sum().item())
        nbytes = tokens * 2 * cfg.Hkv * cfg.d * cfg.kv_elem_bytes
        ok = mc.mc_get_last_status(dp.layout) == mc.MC_OK
        if rank == 0:
            print(json.dumps({"pass": args.pass_only, "workload": cfg.name, "ms": ms, "algorithmic_bytes": nbytes,
                              "gbs": nbytes / (ms * 1e-3) / 1e9, "suffix_part_tokens": int(g.suffix_part_tokens),
                              "n_parts": int(g.n_parts), "prefix_ctas": int(g.prefix_ctas), "status_ok": ok,
                              "forced_alu": os.environ.get("MC_FORCE_FMA", "0") not in ("", "0")}))
        dp.close()
        return 0

    if args.scoring_only:      # profiling aid: only the scoring pass, one small JSON line
        if rank == 0:
            print(json.dumps({"scoring_attention": measure_scoring()}))
        return 0

    main = measure(args.workload, args.steps, args.warmup, True, min_seconds=args.min_seconds)
    others = {}
    cold = None
    if args.all_configs:
        for name in ("cfg2", "cfg3", "cfg4", "cfg4_fp8"):
            if name != args.workload:
                others[name] = measure(name, args.steps, args.warmup, True)
        cold = measure_prefix_cold("cfg2", max(args.steps, 60), args.warmup)
        # a cascade deeper than two levels: configuration 3 behind a 4096-token prompt shared by all 256 candidates
        c3 = wl.CONFIGS["cfg3"]
        others["cfg3+root4096"] = measure("cfg3", args.steps, args.warmup, True, outer=[([0, c3.B], [4096])])

    search = measure_search() if args.all_configs else None
    read_peak = measure_read_peak() if args.all_configs else None

    scoring = measure_scoring() if args.all_configs else None
    qkv = measure_qkv() if args.all_configs else None

    # max over ranks of the step time
    ms, e2e_ms = max_over_ranks([main["ms"], main["e2e_ms"]], device="cuda")

    if rank == 0:
        cfg = main["cfg"]
        peaks, peak_kind = measured_peaks()
        peak = float(peaks["hbm_gbs"])
        value = aggregate_value(main["bytes"], ms, world)
        suffix_gbs = main["suffix_bytes"] / (main["suffix_ms"] * 1e-3) / 1e9

        def prefix_summary(r, pk):
            tf = r["prefix_flops"] / (r["prefix_ms"] * 1e-3) / 1e12
            ctas = r["prefix_ctas"]
            peak = pk.get("bf16_tflops")
            return {"kernel": "prefix_rp_kernel / prefix_tc_kernel (tcgen05)" if ctas else "attn_mma_kernel<prefix>",
                    "ms_alone": r["prefix_ms"],
                    "ctas": ctas, "tflops": tf, "bf16_peak_tflops": peak,
                    # the pass deliberately holds only `ctas` of the 148 SMs: utilisation of the SMs it holds
                    "frac_of_bf16_peak_of_held_sms": (tf / (peak * ctas / 148.0)) if (peak and ctas) else None,
                    "note": "timed alone; in a step it runs beside the suffix pass and is sized to finish under it"}

        def summary(r):
            gbs = r["bytes"] / (r["ms"] * 1e-3) / 1e9
            out = {"gbs": round(gbs, 1), "frac_of_8tbs": round(gbs / NOMINAL_HBM_GBS, 4), "ms_per_step": round(r["ms"], 5),
                   "candidate_tokens_per_s": round(r["cfg"].B / (r["ms"] * 1e-3), 1)}
            if "layout_create_ms" in r:
                out["layout_create_ms"] = round(r["layout_create_ms"], 3)
            if "suffix_ms" in r:
                out["suffix_ms"] = round(r["suffix_ms"], 5)
                out["suffix_gbs"] = round(r["suffix_bytes"] / (r["suffix_ms"] * 1e-3) / 1e9, 1)
                out["prefix_ms"] = round(r["prefix_ms"], 5)
                out["prefix_tflops"] = round(r["prefix_flops"] / (r["prefix_ms"] * 1e-3) / 1e12, 2)
                out["prefix_ctas"] = r["prefix_ctas"]
            return out

        if args.cpu_baseline:
            n_rows = oracle_sample_rows(cfg)
            times, cores, sample_bytes = time_oracle(cfg, n_rows, repeats=1)
            cpu_value = sample_bytes / times[0] / 1e9
        else:
            n_rows, cores, cpu_value = 0, 0, None
        per_config = {**{cfg.name: summary(main)}, **{k: summary(v) for k, v in others.items()}}
        if cold and "cfg2" in per_config:
            # two readings of configuration 2: `frac_of_8tbs` with the 33.6 MB prefix still in L2 from the step before
            # (consecutive steps on ONE layout, as the configuration is worded), and this one with the prefix coming
            # from HBM at every step (instances taking turns)
            per_config["cfg2"]["frac_of_8tbs_prefix_cold"] = round(cold["gbs"] / NOMINAL_HBM_GBS, 4)
            per_config["cfg2"]["ms_per_step_prefix_cold"] = round(cold["ms_per_step"], 5)
            per_config["cfg2"]["prefix_cold_instances"] = cold["instances"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": cfg.name, "groups": cfg.G, "candidates_per_group": cfg.C, "q_heads": cfg.Hq,
                       "kv_heads": cfg.Hkv, "head_dim": cfg.d, "page_tokens": wl.PAGE,
                       "step": ("append + " if cfg.append_steps else "") + "prefix + suffix + merge",
                       "bytes_per_step": main["bytes"], "l2": "inputs larger than L2 (no flush needed)",
                       "multi_gpu": "replicas only"},
            "frac_of_8tbs": value / world / NOMINAL_HBM_GBS,
            "candidate_tokens_per_s": world * cfg.B / (ms * 1e-3),
            "roofline": {"bound": "hbm", "kernel": "suffix_tma_kernel", "achieved": suffix_gbs, "peak": peak,
                         "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": suffix_gbs / peak,
                         "frac_of_8tbs": suffix_gbs / NOMINAL_HBM_GBS,
                         "traffic": suffix_traffic(main["suffix_bytes"], main["suffix_part_tokens"]),
                         "kernel_ms": main["suffix_ms"], "algorithmic_bytes": main["suffix_bytes"],
                         # the measured peak is a copy (reads + writes); this kernel only reads: the read-only
                         # streaming rate of the library's probe kernel on this GPU, in this run, and the fraction of it
                         "read_only_peak": read_peak,
                         "frac_of_read_only_peak": (suffix_gbs / read_peak) if read_peak else None},
            "prefix_pass": prefix_summary(main, peaks),
            "cpu_baseline": {"value": cpu_value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "%d of %d (candidate, head) rows of %s, fp64 numpy, one thread per row"
                                       % (n_rows, cfg.B * cfg.Hq, cfg.name)},
            "e2e": {"value": world * main["bytes"] / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": main["h2d"], "d2h_bytes_per_step": main["d2h"], "ms_per_step": e2e_ms},
            "gpu_launches": int(main["launches"]),
            "clocks": main["clocks"],
            "timed": {"blocks": main["blocks"], "steps_per_block": args.steps, "ms_per_step_is": "median block",
                      "ms_per_step_min_block": main["block_ms_min"], "ms_per_step_max_block": main["block_ms_max"]},
            "per_config": per_config,
            "search_bookkeeping": (dict(search, frac_of_measured_hbm=round(search["gbs"] / peak, 4)) if search else None),
            "scoring_attention": (dict(scoring, bound="tensor", frac_of_measured_bf16=(
                round(scoring["tflops"] / peaks["bf16_tflops"], 4) if peaks.get("bf16_tflops") else None)) if scoring else None),
            "qkv_projection": (dict(qkv, bound="hbm", frac_of_measured_hbm=round(qkv["gbs"] / peak, 4)) if qkv else None),
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg4", choices=sorted(wl.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false",
                    help="skip the CPU-oracle leg (profiling runs only; the default run reports it)")
    ap.add_argument("--scoring-only", action="store_true", help="run only the scoring pass (profiling aid)")
    ap.add_argument("--qkv-only", action="store_true", help="run only the fused q/k/v projection (profiling aid)")
    ap.add_argument("--pass-only", choices=["suffix", "prefix"], default=None,
                    help="run only that pass of --workload, alone (profiling aid)")
    ap.add_argument("--kv-dtype", choices=["bf16", "fp8"], default=None,
                    help="with --pass-only: the cache type, if not the workload's own")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="repeat the block of --steps steps until this much device time has been timed (0: one block)")
    ap.add_argument("--no-all-configs", dest="all_configs", action="store_false",
                    help="time only --workload (default: also cfg2/cfg3/cfg4 summaries under per_config)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as one process: become the launcher of N replicas (one per GPU), as a torchrun launch would
        return spawn_replicas(args.gpus, sys.argv[1:])
    if args.impl == "reference":
        return run_reference(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
