#!/usr/bin/env python
"""Benchmark of the suffix-automaton draft + greedy-verify step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config I]

One "step" = one closed-loop iteration of the whole hot path over one batch: vocabulary argmax
over [B, K+1, V] bf16 logits, prefix accept, automaton walk over the accepted tokens, next draft
(`sam_step`).  The workload is synthetic (see workload/agent_memory.py); the default is the
B=256, K=16, 16M-token-corpus configuration.  Prints ONE JSON line on rank 0.

`--gpus N` with N > 1 starts N ranks, one per GPU (it re-runs itself under
`python -m torch.distributed.run`; started under such a launcher already, it checks that the world size
is N).  Every rank owns B streams of its own and a replica of the index; no collective touches the data
path, the ranks only meet for the final sum of tokens and maximum of time (weak scaling).

Timing: every step is bracketed by CUDA events on the launching stream; the stand-in target
model (sparse planting of the wanted tokens into the resident noise logits between steps) is
outside the events.  `--impl reference` times the CPU oracle instead (host cores, wall clock).
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workload as W  # noqa: E402

METRIC = "sam_draft_verify_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
# DRAM traffic of one argmax_bulk_kernel launch from the ncu captures summarised in
# profiles/argmax_bulk_kernel_cfg1_ncu_full.md and profiles/argmax_direct_kernel_cfg1_dram.md (config 1, launches of the
# kernel as it stands): dram__bytes_read.sum per
# logits row (every row is read once, so the reads grow in proportion to the rows) and dram__bytes_write.sum per launch
# (write-backs of the harness' sparse planting, which do not grow with the rows; the kernel writes 8 bytes per row)
NCU_DRAM_READ_BYTES_PER_ROW = 304105.3
NCU_DRAM_WRITE_BYTES_PER_LAUNCH = 2.82e6
# the same for argmax_direct_kernel (profiles/argmax_direct_kernel_cfg1_dram.md), captured at V = 151,936 and only
# reported for that row length
NCU_DRAM_READ_BYTES_PER_ROW_DIRECT = 304549.0
# dram__sectors_read.sum of one accept_kernel launch per stream, config 2 (profiles/walk_kernels_cfg2_sectors.md)
NCU_ACCEPT_DRAM_SECTORS_PER_STREAM = 45.8


# ----------------------------------------------------------------------------- helpers
def dist_env():
    from harness.launcher import rank_env
    return rank_env()


RANK_SEED_STRIDE = 7919      # rank r draws its stream scripts and planting decisions from seed + 7919 * r


def plan_rank(args, rank: int):
    """(cfg, stream_cfg) of one rank.  cfg describes what every rank shares (corpus, noise logits, sizes);
    stream_cfg differs only in the seed of the B streams the rank owns."""
    base = W.CONFIGS[args.config]
    if args.streams > 0:
        base = base.scaled(B=args.streams, name=f"{base.name}_B{args.streams}")
    # long enough for every leg of either arm (the oracle leg replays the scripts from step 0), and the same in
    # both arms: the script generator's draws depend on the script length
    n_script_steps = max(args.warmup + args.steps + args.split_steps + 2 * args.e2e_steps + 1, args.cpu_steps + 8)
    cfg = base.scaled(steps=n_script_steps)
    stream_cfg = cfg.scaled(seed=cfg.seed + RANK_SEED_STRIDE * rank) if rank > 0 else cfg
    return cfg, stream_cfg


def init_ranks(backend: str, args, device_of=None):
    """Joins the process group when started under a launcher; (rank, local_rank, world).  Refuses to run when
    the launcher's world size is not the --gpus that was asked for."""
    rank, local_rank, world = dist_env()
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if world > 1:
        import torch.distributed as dist
        kw = {}
        if device_of is not None:
            kw["device_id"] = device_of(local_rank)
        dist.init_process_group(backend, **kw)
    return rank, local_rank, world


def gather_over_ranks(obj, world: int):
    """List of every rank's (picklable) object, in rank order."""
    if world == 1:
        return [obj]
    import torch.distributed as dist
    out = [None] * world
    dist.all_gather_object(out, obj)
    return out


NOISE_ON_HOST_MAX_BYTES = 3 << 30


def noise_on_host(cfg) -> bool:
    """The noise logits of both arms come from one host generator whenever that is affordable; only the
    10 GB workload draws them on the device (minutes on the host), and its two arms then differ in bytes."""
    return cfg.rows * cfg.vocab * 2 <= NOISE_ON_HOST_MAX_BYTES


def workload_block(cfg) -> dict:
    """The `config` object of the JSON line; the same for both arms."""
    big = cfg.rows * cfg.vocab * 2 > 252e6
    return {"workload": cfg.name, "B_per_gpu": cfg.B, "K": cfg.K, "V": cfg.vocab, "min_match": cfg.min_match,
            "corpus_tokens": cfg.n_corpus, "accept_p": cfg.accept_p,
            "logits_bytes_per_step": cfg.rows * cfg.vocab * 2,
            "l2": "inputs larger than L2 (logits re-read from HBM every step)" if big
            else "inputs smaller than 2x L2: bandwidth figures are not HBM figures",
            "noise": "numpy PCG64 on the host, same bytes in both arms" if noise_on_host(cfg)
            else "torch generator on the device (ours) / numpy on the host (reference): same distribution"}


def headline(cfg, world, args, tokens, ms, **more) -> dict:
    """The contract keys of the JSON line from the job totals (tokens summed and ms maximised over ranks)."""
    out = {"metric": METRIC, "value": tokens / (ms / 1e3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "bf16 compare / int32", "data": "synthetic", "config": workload_block(cfg)}
    out.update(more)
    return out


def reduce_over_ranks(tokens: int, ms: float, world: int, backend_device=None):
    """(sum of tokens, max of milliseconds) over all ranks; identity when world == 1."""
    if world == 1:
        return tokens, ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(tokens)], dtype=torch.float64, device=backend_device)
    m = torch.tensor([float(ms)], dtype=torch.float64, device=backend_device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    dist.all_reduce(m, op=dist.ReduceOp.MAX)
    return int(round(t.item())), float(m.item())


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock, power and throttle reasons while the timed region runs: NVML from a thread of this
    process (a sample every millisecond, so that even a 20-step window holds many), nvidia-smi as a fallback.
    Read-only: nothing on the GPU is set."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int, period_s: float = 0.001):
        self.samples = []            # (time, sm MHz, max MHz, set of reasons)
        self.gpu = gpu_index
        self.period = period_s
        self.proc = None
        self.thread = None
        self.how = None
        self._stop = threading.Event()

    def _physical_index(self):
        vis = os.environ.get("CUDA_VISIBLE_DEVICES")
        if vis:
            ids = [x.strip() for x in vis.split(",") if x.strip()]
            if self.gpu < len(ids) and ids[self.gpu].isdigit():
                return int(ids[self.gpu])
        return self.gpu

    def start(self):
        try:
            import pynvml as N
            N.nvmlInit()
            h = N.nvmlDeviceGetHandleByIndex(self._physical_index())
            mx = float(N.nvmlDeviceGetMaxClockInfo(h, N.NVML_CLOCK_SM))
            bits = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}
            reasons_fn = getattr(N, "nvmlDeviceGetCurrentClocksEventReasons", None) or N.nvmlDeviceGetCurrentClocksThrottleReasons
            reasons_fn(h)       # must work before the thread relies on it

            def pump():
                while not self._stop.is_set():
                    try:
                        r = int(reasons_fn(h))
                        self.samples.append((time.time(), float(N.nvmlDeviceGetClockInfo(h, N.NVML_CLOCK_SM)), mx,
                                             {k for k, b in bits.items() if r & b}))
                    except Exception:
                        pass
                    time.sleep(self.period)
            self.thread = threading.Thread(target=pump, daemon=True)
            self.thread.start()
            self.how = f"NVML, one sample per {self.period * 1e3:g} ms"
            return
        except Exception:
            self.thread = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self._physical_index()}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "5"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True, bufsize=1)
            self.thread = threading.Thread(target=self._pump_smi, daemon=True)
            self.thread.start()
            self.how = "nvidia-smi -lms 5"
        except Exception:
            self.proc = None

    def _pump_smi(self):
        for line in self.proc.stdout:
            f = [x.strip() for x in line.strip().split(",")]
            if len(f) < 8:
                continue
            try:
                self.samples.append((time.time(), float(f[0]), float(f[1]),
                                     {n for n, v in zip(self.NAMES, f[4:8]) if v.lower().startswith("active")}))
            except ValueError:
                continue

    def stop(self, t_begin: float = 0.0, t_end: float = float("inf")):
        """Summary of the samples that arrived inside [t_begin, t_end] (the timed region)."""
        self._stop.set()
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        if self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["no clock source available"]}
        self.thread.join(timeout=2)
        inside = [x for x in self.samples if t_begin <= x[0] <= t_end]
        sm = [x[1] for x in inside]
        reasons = set().union(*[x[3] for x in inside]) if inside else set()
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(x[2] for x in inside) if inside else None,
                "samples": len(sm), "reasons": sorted(reasons), "source": self.how}


def make_inputs_gpu(cfg, device):
    """Corpus (host) and the noise logits on the device.  The noise is drawn on the host by the generator
    the reference arm uses and uploaded once, so both arms read the same bytes; only a workload too large
    for that draws it on the device."""
    import torch
    corpus = W.make_corpus(cfg)
    if noise_on_host(cfg):
        bits = W.make_noise_logits(cfg)
        rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(bits).max(axis=1))
        logits = torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
        del bits
    else:
        logits, rowmax = W.make_noise_logits_device(cfg, device)
    return corpus, logits, rowmax


# ----------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2512_18337_b200 as S
    from paper_2512_18337_b200.build import build
    from harness.cuda_backend import CudaBackend

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    rank, local_rank, world = init_ranks("nccl", args, lambda lr: torch.device(f"cuda:{lr}"))
    device = f"cuda:{local_rank}"
    torch.cuda.set_device(device)
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    S.sam_set_argmax_variant(args.variant)

    # weak scaling: every rank owns B streams of its own (distinct scripts / planting draws), the
    # read-only automaton is replicated; no data-path collective
    cfg, stream_cfg = plan_rank(args, rank)

    t0 = time.time()
    corpus, logits, rowmax = make_inputs_gpu(cfg, device)
    scripts = W.make_scripts(stream_cfg, corpus)
    t_inputs = time.time() - t0
    t0 = time.time()
    index = S.SamIndex(corpus, [cfg.separator], device=device, upload=False)
    t_build = time.time() - t0
    t0 = time.time()
    index.blob = torch.empty(index.device_bytes, dtype=torch.uint8, device=device)
    S.sam_upload(index.handle, index.blob)
    t_upload = time.time() - t0

    feeder = W.ClosedLoopFeeder(stream_cfg, scripts, rowmax)
    be = CudaBackend(cfg, corpus, logits, index=index, device=device)
    be.counters = torch.zeros(S.SAM_N_COUNTERS, dtype=torch.int64, device=device)
    if args.skip_unused_rows:
        be.flags |= S.SAM_STEP_SKIP_UNUSED_ROWS
        be.chain_row_lists = True       # every step's accept kernel lists the rows of the next step: two launches per step
    toks, n = feeder.prime_tokens()
    drafts, n_draft = be.prime(toks, n)

    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    tokens = 0
    stats_trace = []

    def one_step(t, timed_slot=None):
        nonlocal drafts, n_draft, tokens
        ow = feeder.overwrites(t, drafts, n_draft)
        keep = np.arange(ow["row"].shape[0])
        saved = be.poke(ow["row"], ow["col"], ow["bits"], keep)
        in_nd = n_draft
        if timed_slot is not None:
            # keep the stream busy (a spin kernel, outside the events) while the host enqueues the step, so
            # the events bracket device execution and not the host's launch latency on an idle GPU
            torch.cuda._sleep(args.presleep_cycles)
            ev[timed_slot][0].record()
            be.launch_step()
            ev[timed_slot][1].record()
        else:
            be.launch_step()
        torch.cuda.synchronize()
        n_acc = be.n_accepted.cpu().numpy()
        drafts, n_draft = be.drafts.cpu().numpy(), be.n_draft.cpu().numpy()
        be.unpoke(ow["row"], ow["col"], saved)
        feeder.advance(n_acc)
        if timed_slot is not None:
            tokens += int(n_acc.sum())
            stats_trace.append(dict(n_accepted=n_acc, in_n_draft=in_nd))

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()           # started early: nvidia-smi needs a moment before its first sample
    for t in range(args.warmup):
        one_step(t)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    graph_launches = None
    direct_launch = be.launch_step
    if args.graph:
        # the step's launches recorded once (after ordinary calls have done the first-use set-up) and replayed:
        # same kernels, same buffers, no per-launch host work and no gaps between the two kernels
        l0 = S.sam_launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            direct_launch()
        graph_launches = S.sam_launch_count() - l0
        be.launch_step = graph.replay
        torch.cuda.synchronize()
    launches0 = S.sam_launch_count()
    be.counters.zero_()
    torch.cuda.synchronize()
    wall0 = time.time()
    for i in range(args.steps):
        one_step(args.warmup + i, timed_slot=i)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    wall = time.time() - wall0
    launches = S.sam_launch_count() - launches0
    if args.graph:
        launches = graph_launches * args.steps      # kernel nodes of the replayed graph
        be.launch_step = direct_launch
    dev_counters = [int(x) for x in be.counters.cpu().numpy()]
    clocks = sampler.stop(wall0, wall0 + wall) if rank == 0 else None
    step_ms = [a.elapsed_time(b) for a, b in ev]
    total_ms = float(sum(step_ms))
    launches_per_step = launches / args.steps

    # ---- per-kernel split, outside the timed region: the same loop continues with the accept step in a kernel
    # of its own, so that the library's events separate the vocabulary argmax from accept + walk + draft
    split = None
    if args.split_steps > 0:
        S.sam_set_argmax_variant(3 if args.variant == 2 else args.variant)
        S.sam_profile_enable(args.split_steps)
        n_before = len(stats_trace)
        for i in range(args.split_steps):
            t = args.warmup + args.steps + i
            ow = feeder.overwrites(t, drafts, n_draft)
            saved = be.poke(ow["row"], ow["col"], ow["bits"], np.arange(ow["row"].shape[0]))
            in_nd = n_draft
            torch.cuda._sleep(args.presleep_cycles)
            be.launch_step()
            torch.cuda.synchronize()
            n_acc = be.n_accepted.cpu().numpy()
            drafts, n_draft = be.drafts.cpu().numpy(), be.n_draft.cpu().numpy()
            be.unpoke(ow["row"], ow["col"], saved)
            feeder.advance(n_acc)
            stats_trace.append(dict(n_accepted=n_acc, in_n_draft=in_nd))
        sp = [S.sam_profile_read(i) for i in range(S.sam_profile_count())]
        S.sam_profile_enable(0)
        S.sam_set_argmax_variant(args.variant)
        split_trace = stats_trace[n_before:]
        del stats_trace[n_before:]
        split = {"steps": args.split_steps, "argmax_ms": statistics.mean(p[0] for p in sp),
                 "accept_walk_draft_ms": statistics.mean(p[1] for p in sp),
                 "committed": int(sum(int(o["n_accepted"].sum()) for o in split_trace)),
                 "drafted": int(sum(int(o["in_n_draft"].sum()) for o in split_trace))}

    # ---- end to end through the host-buffer entry point: logits and bookkeeping start in pinned host memory
    e2e = None
    if args.e2e_steps > 0:
        B, K, V = cfg.B, cfg.K, cfg.vocab
        host_logits = torch.empty(logits.shape, dtype=torch.bfloat16).pin_memory()
        host_logits.copy_(logits)
        torch.cuda.synchronize()
        hraw = host_logits.view(torch.int16).numpy().view(np.uint16)
        i32 = dict(dtype=torch.int32)
        h = {k: torch.zeros(s, **i32).pin_memory() for k, s in dict(
            drafts=(B, K), n_draft=(B,), argmax=(B, K + 1), accepted=(B, K + 1), n_accepted=(B,),
            state=(B,), mlen=(B,)).items()}
        h["drafts"].copy_(be.drafts)
        h["n_draft"].copy_(be.n_draft)
        h["state"].copy_(be.state)
        h["mlen"].copy_(be.mlen)
        torch.cuda.synchronize()
        sb = S.sam_step_host_staging_bytes(V, B, K, V)
        staging = torch.empty(sb, dtype=torch.uint8, device=device)
        def host_loop(flags, t_base):
            toks, secs, rows = 0, 0.0, 0
            for i in range(args.e2e_steps):
                t = t_base + i
                ow = feeder.overwrites(t, h["drafts"].numpy(), h["n_draft"].numpy())
                saved = hraw[ow["row"], ow["col"]].copy()
                hraw[ow["row"], ow["col"]] = ow["bits"]
                used_rows = int(np.clip(h["n_draft"].numpy(), 0, K).sum()) + B
                torch.cuda.synchronize()
                c0 = time.perf_counter()
                S.sam_step_host_ex(index.handle, host_logits, V, B, K, V, h["drafts"], h["n_draft"], h["argmax"],
                                   h["accepted"], h["n_accepted"], h["state"], h["mlen"], cfg.min_match,
                                   h["drafts"], h["n_draft"], flags, staging, sb)
                c1 = time.perf_counter()
                hraw[ow["row"], ow["col"]] = saved
                n_acc = h["n_accepted"].numpy().copy()
                feeder.advance(n_acc)
                if i > 0 or args.e2e_steps == 1:       # first host step warms the pinned path
                    toks += int(n_acc.sum())
                    secs += c1 - c0
                    rows += used_rows
            return toks, secs, rows

        t_e2e = args.warmup + args.steps + args.split_steps
        e2e_tokens, e2e_s, _ = host_loop(0, t_e2e)
        skip_tokens, skip_s, skip_rows = host_loop(S.SAM_STEP_SKIP_UNUSED_ROWS, t_e2e + args.e2e_steps)
        n_timed = max(1, args.e2e_steps - 1)
        small = (B * K + 3 * B) * 4
        h2d = logits.numel() * 2 + small
        d2h = (2 * B * (K + 1) + B * K + 4 * B) * 4
        e2e_tokens, e2e_ms = reduce_over_ranks(e2e_tokens, e2e_s * 1e3, world, device)
        skip_tokens, skip_ms = reduce_over_ranks(skip_tokens, skip_s * 1e3, world, device)
        e2e = {"value": e2e_tokens / (e2e_ms / 1e3) if e2e_ms > 0 else None, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "steps": n_timed, "api": "sam_step_host (pinned host buffers, wall clock incl. sync)",
               "skip_unused_rows": {"value": skip_tokens / (skip_ms / 1e3) if skip_ms > 0 else None, "unit": UNIT,
                                    "h2d_bytes_per_step": skip_rows / n_timed * V * 2 + small,
                                    "api": "sam_step_host_ex with SAM_STEP_SKIP_UNUSED_ROWS: only rows 0..n_draft[b] "
                                           "cross the bus (a different contract: the other rows are not arg-maxed)"}}
        del staging, host_logits

    # ---- with --graph: what a serving loop that issues steps back to back sees, direct calls against replays of
    # the recorded step (one event pair around the whole run; the logits stay as they are, so most drafts are
    # rejected, but every row is arg-maxed and every stream accepted, walked and drafted as in any other step)
    back_to_back = None
    if args.graph:
        n_b2b = 300
        back_to_back = {"steps": n_b2b}
        for name, fn in (("direct_calls_us_per_step", direct_launch), ("graph_replay_us_per_step", graph.replay)):
            for _ in range(10):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            w0 = time.perf_counter()
            e0.record()
            for _ in range(n_b2b):
                fn()
            e1.record()
            torch.cuda.synchronize()
            w1 = time.perf_counter()
            back_to_back[name] = e0.elapsed_time(e1) * 1e3 / n_b2b
            back_to_back[name.replace("_us_per_step", "_wall_us_per_step")] = (w1 - w0) * 1e6 / n_b2b
        assert be.status() == 0

    all_tokens, max_ms = reduce_over_ranks(tokens, total_ms, world, device)
    rank_seeds = gather_over_ranks(stream_cfg.seed, world)      # one distinct script seed per rank
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    R = cfg.rows
    rows_read_per_step = dev_counters[5] / max(1, dev_counters[0]) * cfg.B     # all rows unless rows are skipped
    alg_bytes = R * (2 * cfg.vocab + 4)
    if args.skip_unused_rows:
        alg_bytes = rows_read_per_step * (2 * cfg.vocab + 4)
    # dominant kernel: with one launch per step the step's event bracket IS that kernel's duration (vocabulary
    # argmax with the accept / walk / draft tail inside); with two launches per step the argmax kernel's own
    # time comes from the split measurement
    if launches_per_step == 1:
        kernel_ms, kernel_name = total_ms / args.steps, "argmax_bulk_kernel (argmax + fused accept/walk/draft tail)"
    else:
        kernel_ms, kernel_name = (split["argmax_ms"] if split else total_ms / args.steps), "argmax kernel alone"
    # counters exist for the two argmax kernels at the full vocabulary
    # the library's own rule for variant 0: direct loads up to 768 MiB of logits and K <= 16
    direct = args.variant == 1 or (args.variant == 0 and cfg.K <= 16 and R * cfg.vocab * 2 <= (768 << 20))
    traffic_per_row = None
    if cfg.vocab == 151936:
        traffic_per_row = NCU_DRAM_READ_BYTES_PER_ROW_DIRECT if direct else NCU_DRAM_READ_BYTES_PER_ROW
    achieved = alg_bytes / (kernel_ms * 1e-3) / 1e9
    walk = None
    if split is not None:
        walk_s = split["accept_walk_draft_ms"] * split["steps"] / 1e3
        walk = {"draft_tokens_per_s": split["drafted"] / walk_s, "committed_tokens_per_s_kernel_only": split["committed"] / walk_s,
                "argmax_only_GBps": alg_bytes / (split["argmax_ms"] * 1e-3) / 1e9,
                "bound": "latency (dependent random accesses)",
                "dram_sector_GBps": NCU_ACCEPT_DRAM_SECTORS_PER_STREAM * cfg.B * 32 / (split["accept_walk_draft_ms"] * 1e-3) / 1e9,
                "dram_sector_frac_of_peak": NCU_ACCEPT_DRAM_SECTORS_PER_STREAM * cfg.B * 32
                                            / (split["accept_walk_draft_ms"] * 1e-3) / 1e9 / peak,
                "note": f"{split['steps']} further steps of the same loop after the timed region, accept + walk + draft "
                        "in a kernel of its own (library events around it)", **split}
    st = W.trace_stats(cfg, stats_trace)
    out = headline(cfg, world, args, all_tokens, max_ms)
    out.update({
        "timing": "CUDA events around each sam_step on the launching stream, summed over steps, maximum over ranks; "
                  "sparse logits planting between steps excluded; a spin kernel ahead of the first "
                  "event keeps the queue full so host launch latency is not timed",
        "rank_seeds": rank_seeds,
        "steps_per_s": args.steps / (max_ms / 1e3),
        "stream_steps_per_s": world * cfg.B * args.steps / (max_ms / 1e3),
        "gpu_launches": launches,
        "launches_per_step": launches_per_step, "variant": args.variant, "cuda_graph": bool(args.graph), "back_to_back": back_to_back,
        "roofline": {"kernel": kernel_name + (" (argmax_direct_kernel)" if direct else " (argmax_bulk_kernel)" if launches_per_step != 1 else ""), "kernel_ms": kernel_ms, "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_8TBs": achieved / 8000.0,
                     "traffic": (traffic_per_row * (rows_read_per_step if args.skip_unused_rows else R)
                                 + NCU_DRAM_WRITE_BYTES_PER_LAUNCH) if traffic_per_row else None,
                     "algorithmic_bytes": alg_bytes,
                     "whole_step": {"ms": total_ms / args.steps, "achieved": alg_bytes / (total_ms / args.steps * 1e-3) / 1e9,
                                    "frac": alg_bytes / (total_ms / args.steps * 1e-3) / 1e9 / peak,
                                    "note": "the same bytes over the event bracket of the whole step in the timed region "
                                            "(argmax + accept + walk + draft)"}},
        "walk": walk,
        "ote": st["ote"], "shr": st["shr"], "shr_per_K_of_nonempty_proposals": st["shr_k"],
        "mean_n_draft": st["mean_n_draft"],
        "device_counters": {"passes": dev_counters[0], "committed": dev_counters[1], "proposed": dev_counters[2],
                            "accepted_drafts": dev_counters[3], "nonempty_proposals": dev_counters[4],
                            "rows_read": dev_counters[5], "ote": dev_counters[1] / max(1, dev_counters[0]),
                            "shr": dev_counters[3] / max(1, dev_counters[2])},
        "skip_unused_rows": bool(args.skip_unused_rows), "rows_read_per_step": rows_read_per_step,
        "e2e": e2e, "clocks": clocks,
        "setup_s": {"inputs": t_inputs, "sam_build": t_build, "sam_upload": t_upload,
                    "sam_build_tokens_per_s": cfg.n_corpus / t_build,
                    "states": index.n_states, "edges": index.n_edges, "device_bytes": index.device_bytes},
        "wall_s_timed_loop_incl_harness": wall,
    })
    if args.cpu_baseline and world == 1:
        out["cpu_baseline"] = cpu_baseline(cfg, corpus, scripts, logits, rowmax, args.cpu_steps)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- oracle arm
def oracle_loop(cfg, corpus, scripts, host_bits, rowmax, warmup, steps, threads, single_thread_steps=0, backend=None):
    """Times the oracle's step (wall clock, planting excluded) on the same closed loop; optionally goes on for a
    few steps on one thread.  Returns (tokens, seconds, build seconds[, single-thread tokens, seconds]).
    `backend`: an OracleBackend to reuse (its automaton is kept, its stream state starts afresh)."""
    from oracle.backend import OracleBackend
    feeder = W.ClosedLoopFeeder(cfg, scripts, rowmax)
    t0 = time.time()
    if backend is None:
        be = OracleBackend(cfg, corpus, host_bits, threads)
    else:
        be = backend
        be.state[:] = 0
        be.mlen[:] = 0
        be.threads = threads
    t_build = time.time() - t0
    toks, n = feeder.prime_tokens()
    drafts, n_draft = be.prime(toks, n)
    tokens, secs, tokens1, secs1 = 0, 0.0, 0, 0.0
    for t in range(warmup + steps + single_thread_steps):
        if t == warmup + steps:
            be.threads = 1
        ow = feeder.overwrites(t, drafts, n_draft)
        keep = np.arange(ow["row"].shape[0])
        saved = be.poke(ow["row"], ow["col"], ow["bits"], keep)
        c0 = time.perf_counter()
        out = be.step(drafts, n_draft)
        c1 = time.perf_counter()
        be.unpoke(ow["row"], ow["col"], saved)
        feeder.advance(out["n_accepted"])
        drafts, n_draft = out["drafts"], out["n_draft"]
        if t >= warmup + steps:
            tokens1 += int(out["n_accepted"].sum())
            secs1 += c1 - c0
        elif t >= warmup:
            tokens += int(out["n_accepted"].sum())
            secs += c1 - c0
    if single_thread_steps > 0:
        return tokens, secs, t_build, tokens1, secs1
    return tokens, secs, t_build


def cpu_baseline(cfg, corpus, scripts, logits_dev, rowmax, steps):
    import oracle
    host_bits = W.device_bits_to_host(logits_dev)
    threads = oracle.host_threads()
    tokens, secs, t_build, tokens1, secs1 = oracle_loop(cfg, corpus, scripts, host_bits, rowmax, 1, steps, threads, 4)
    return {"value": tokens / secs, "unit": UNIT, "cores": threads, "kind": "oracle",
            "single_thread": {"value": tokens1 / secs1, "unit": UNIT, "steps": 4,
                              "argmax_GBps": cfg.rows * cfg.vocab * 2 * 4 / secs1 / 1e9},
            "sample": f"all {cfg.B} streams, first {steps} closed-loop steps after 1 warm-up step "
                      f"({secs:.2f} s of oracle stepping; oracle automaton build {t_build:.1f} s not included)",
            "ms_per_step": secs / steps * 1e3,
            "argmax_GBps": cfg.rows * cfg.vocab * 2 * steps / secs / 1e9}


REFERENCE_MAX_STEPS = 400      # oracle steps per run over all rank shares (about 20 s at the default workload)


def run_reference(args):
    """The oracle, as it stands, on the host cores: the work of all --gpus rank shares, one after the other (the
    host cores are one pool, so the shares' times add up).  Under a launcher rank 0 alone does this."""
    rank, _, world = dist_env()
    if world > 1 and world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if rank != 0:
        return
    import oracle
    from oracle.backend import OracleBackend
    n_shares = args.gpus
    per_share_cap = max(1, REFERENCE_MAX_STEPS // n_shares)
    steps = min(args.steps, per_share_cap)
    warmup = min(args.warmup, per_share_cap)
    cfg, _ = plan_rank(args, 0)
    corpus = W.make_corpus(cfg)
    host_bits = W.make_noise_logits(cfg)
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(host_bits).max(axis=1))
    threads = oracle.host_threads()
    t0 = time.time()
    be = OracleBackend(cfg, corpus, host_bits, threads)
    t_build = time.time() - t0
    tokens, secs, seeds = 0, 0.0, []
    for r in range(n_shares):
        _, stream_cfg = plan_rank(args, r)
        scripts = W.make_scripts(stream_cfg, corpus)
        tk, sc, _ = oracle_loop(stream_cfg, corpus, scripts, host_bits, rowmax, warmup, steps, threads, backend=be)
        tokens += tk
        secs += sc
        seeds.append(stream_cfg.seed)
    v = tokens / secs
    capped = steps != args.steps or warmup != args.warmup
    sample = (f"all {cfg.B} streams of each of {n_shares} rank share(s) of {cfg.name}, {steps} closed-loop steps per share "
              f"after {warmup} warm-up" + (f" (requested {args.steps}/{args.warmup}; capped so the run stays within minutes)"
                                          if capped else ""))
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": n_shares, "steps": steps,
            "warmup": warmup, "ms_per_step": secs / steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16 compare / int32", "data": "synthetic", "config": workload_block(cfg),
            "timing": "wall clock around each oracle step on the host cores, summed over steps and rank shares; "
                      "planting between steps excluded",
            "rank_seeds": seeds,
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "oracle_build_s": t_build}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- growing index
def run_growing(args):
    """Same closed loop on an index that keeps growing: every step the tokens all streams committed are
    queued for the builder thread (one new session per step), and before each step whatever the thread has
    finished is brought to the device (sam_sync) and the stream states are renormalised.  Prints its own JSON
    line; the timed bracket of a step holds sync + renormalise + sam_step."""
    import torch
    import paper_2512_18337_b200 as S
    from paper_2512_18337_b200.build import build
    from harness.cuda_backend import CudaBackend

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    device = "cuda:0"
    torch.cuda.set_device(device)
    build()
    base = W.CONFIGS[args.config]
    cfg = base.scaled(steps=args.warmup + args.steps + 1)
    corpus, logits, rowmax = make_inputs_gpu(cfg, device)
    scripts = W.make_scripts(cfg, corpus)
    room = (cfg.K + 2) * cfg.B * (args.warmup + args.steps + 2) + (1 << 20) + 32768
    t0 = time.time()
    index = S.SamIndex(corpus, [cfg.separator], device=device, max_tokens=cfg.n_corpus + room, max_token_id=cfg.separator)
    t_build_upload = time.time() - t0
    # builder throughput on its own: one large piece of fresh text, waited for
    extra = W.make_corpus(cfg.scaled(sessions=max(1, (1 << 19) // cfg.session_len), seed=cfg.seed + 101))
    t0 = time.time()
    S.sam_extend(index.handle, extra)
    t_extend = time.time() - t0
    t0 = time.time()
    S.sam_sync(index.handle)
    torch.cuda.synchronize()
    t_first_sync = time.time() - t0
    # a 30k-token prompt arriving at once (the paper's asynchronous-construction experiment uses such a prompt):
    # time until the builder thread has indexed it and the device copy is up to date
    prompt = W.make_corpus(cfg.scaled(sessions=8, seed=cfg.seed + 202))[:30000]
    t0 = time.time()
    S.sam_extend(index.handle, prompt)
    t_prompt_build = time.time() - t0
    S.sam_sync(index.handle)
    torch.cuda.synchronize()
    t_prompt_total = time.time() - t0
    stats0 = S.sam_update_stats(index.handle)

    feeder = W.ClosedLoopFeeder(cfg, scripts, rowmax)
    be = CudaBackend(cfg, corpus, logits, index=index, device=device)
    toks, n = feeder.prime_tokens()
    drafts, n_draft = be.prime(toks, n)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    tokens = appended = 0
    lag = []
    for t in range(args.warmup + args.steps):
        ow = feeder.overwrites(t, drafts, n_draft)
        saved = be.poke(ow["row"], ow["col"], ow["bits"], np.arange(ow["row"].shape[0]))
        i = t - args.warmup
        if i >= 0:
            torch.cuda._sleep(args.presleep_cycles)
            ev[i][0].record()
        S.sam_sync_renormalize(index.handle, cfg.B, be.state, be.mlen)
        be.launch_step()
        if i >= 0:
            ev[i][1].record()
        torch.cuda.synchronize()
        n_acc = be.n_accepted.cpu().numpy()
        acc = be.accepted.cpu().numpy()
        drafts, n_draft = be.drafts.cpu().numpy(), be.n_draft.cpu().numpy()
        be.unpoke(ow["row"], ow["col"], saved)
        feeder.advance(n_acc)
        piece = np.concatenate([[cfg.separator]] + [acc[b, :n_acc[b]] for b in range(cfg.B)]).astype(np.int32)
        S.sam_extend(index.handle, piece, wait=False)
        if i >= 0:
            tokens += int(n_acc.sum())
            appended += piece.shape[0]
            q, bt, dv = S.sam_pending(index.handle)
            lag.append(q - dv)
    S.sam_extend(index.handle, np.zeros(0, np.int32))
    S.sam_sync(index.handle)
    torch.cuda.synchronize()
    stats1 = S.sam_update_stats(index.handle)
    ms = float(sum(a.elapsed_time(b) for a, b in ev))
    print(json.dumps({
        "metric": METRIC + "_growing_index", "value": tokens / (ms / 1e3), "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "dtype": "bf16 compare / int32", "data": "synthetic",
        "config": {"workload": cfg.name + " + one appended session per step (all committed tokens)",
                   "B": cfg.B, "K": cfg.K, "V": cfg.vocab, "timing": "CUDA events around sam_sync_renormalize + sam_step"},
        "appended_tokens_per_step": appended / args.steps,
        "mean_tokens_not_yet_on_device_at_step_end": statistics.mean(lag),
        "updates": {"incremental": stats1[0] - stats0[0], "full_images": stats1[1] - stats0[1],
                    "h2d_bytes_per_step": (stats1[2] - stats0[2]) / args.steps},
        "builder_thread_tokens_per_s": extra.shape[0] / t_extend,
        "prompt_30k_tokens": {"indexed_on_host_ms": t_prompt_build * 1e3, "visible_on_device_ms": t_prompt_total * 1e3,
                              "note": "drafting from the older text goes on meanwhile; nothing on the decoding path waits"},
        "first_sync_s": t_first_sync, "first_sync_bytes": stats0[2], "build_and_upload_s": t_build_upload,
        "device_bytes": index.device_bytes,
    }))


# ----------------------------------------------------------------------------- vocabulary-parallel verification
def run_vocab_parallel(args):
    """The closed loop with the vocabulary split into column shards (tensor-parallel output layer).
    Under torchrun every rank owns one shard of the same logits and the per-row words are combined by one
    NCCL MAX all-reduce; on a single process all shards are reduced one after the other on the one GPU and
    merged there.  Prints its own JSON line."""
    import torch
    import torch.distributed as dist
    import paper_2512_18337_b200 as S
    from paper_2512_18337_b200.build import build
    from paper_2512_18337_b200.parallel import reduce_argmax_keys, shard_bounds
    from harness.cuda_backend import CudaBackend

    rank, local_rank, world = init_ranks("nccl", args, lambda lr: torch.device(f"cuda:{lr}"))
    device = f"cuda:{local_rank}"
    torch.cuda.set_device(device)
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    shards = world if world > 1 else args.vocab_shards
    mine = [rank] if world > 1 else list(range(shards))
    cfg, _ = plan_rank(args, 0)          # every rank holds a column shard of the SAME streams' logits
    corpus, logits, rowmax = make_inputs_gpu(cfg, device)       # same seed on every rank: same logits
    scripts = W.make_scripts(cfg, corpus)
    feeder = W.ClosedLoopFeeder(cfg, scripts, rowmax)
    be = CudaBackend(cfg, corpus, logits, device=device)
    toks, n = feeder.prime_tokens()
    drafts, n_draft = be.prime(toks, n)
    R, c = cfg.rows, cfg
    keys = [torch.zeros(R + 1, dtype=torch.int64, device=device) for _ in mine]
    merged = torch.zeros(R, dtype=torch.int64, device=device)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    shard_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(mine) + 1)] for _ in range(args.steps)]
    tokens = 0
    for t in range(args.warmup + args.steps):
        ow = feeder.overwrites(t, drafts, n_draft)
        saved = be.poke(ow["row"], ow["col"], ow["bits"], np.arange(ow["row"].shape[0]))
        i = t - args.warmup
        if i >= 0:
            torch.cuda._sleep(args.presleep_cycles)
            ev[i][0].record()
        for q, (k, r) in enumerate(zip(keys, mine)):
            lo, hi = shard_bounds(c.vocab, r, shards)
            if i >= 0:
                shard_ev[i][q].record()
            S.sam_argmax_partial(be.logits.data_ptr() + 2 * lo, be.stride, R, hi - lo, lo, k)
        if i >= 0:
            shard_ev[i][len(mine)].record()
        if world > 1:
            reduce_argmax_keys(keys[0], R)
            words = keys[0]
        else:
            merged.copy_(keys[0][:R])
            for k in keys[1:]:
                torch.maximum(merged, k[:R], out=merged)
            words = merged
        S.sam_step_from_keys(be.index.handle, words, c.B, c.K, be.drafts, be.n_draft, be.argmax, be.accepted,
                             be.n_accepted, be.state, be.mlen, c.min_match, be.drafts, be.n_draft)
        if i >= 0:
            ev[i][1].record()
        torch.cuda.synchronize()
        n_acc = be.n_accepted.cpu().numpy()
        drafts, n_draft = be.drafts.cpu().numpy(), be.n_draft.cpu().numpy()
        be.unpoke(ow["row"], ow["col"], saved)
        feeder.advance(n_acc)
        if i >= 0:
            tokens += int(n_acc.sum())
    ms = float(sum(a.elapsed_time(b) for a, b in ev))
    _, ms = reduce_over_ranks(0, ms, world, device)
    # one shard's sam_argmax_partial (zero-fill of its words + the argmax kernel), from the events between the calls
    shard_ms = [e[q].elapsed_time(e[q + 1]) for e in shard_ev for q in range(len(mine))]
    shard_bytes = [R * (2 * (shard_bounds(c.vocab, r, shards)[1] - shard_bounds(c.vocab, r, shards)[0]) + 4) for r in mine]
    peak, peak_kind = measured_peaks()
    if rank == 0:
        per_shard_gbs = statistics.mean(shard_bytes) / (statistics.mean(shard_ms) * 1e-3) / 1e9
        print(json.dumps({
            "metric": METRIC + "_vocab_parallel",
            "shard_argmax": {"us_per_shard": statistics.mean(shard_ms) * 1e3, "GBps": per_shard_gbs, "frac": per_shard_gbs / peak,
                             "peak_kind": f"of {peak_kind}", "bytes_per_shard": statistics.mean(shard_bytes),
                             "note": "events around each sam_argmax_partial call (memset of the words + argmax kernel)"}, "value": tokens / (ms / 1e3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "strong", "dtype": "bf16 compare / int32", "data": "synthetic",
            "config": {"workload": cfg.name, "B": c.B, "K": c.K, "V": c.vocab, "vocab_shards": shards,
                       "shards_reduced_per_gpu": len(mine),
                       "timing": "CUDA events around sam_argmax_partial (per shard) + merge + sam_step_from_keys"},
            "bytes_reduced_per_gpu_per_step": sum(R * 2 * (shard_bounds(c.vocab, r, shards)[1] - shard_bounds(c.vocab, r, shards)[0]) for r in mine),
            "allreduce_bytes_per_step": R * 8 if world > 1 else 0,
        }))
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- composite drafting
def run_multi(args):
    """Closed loop with composite drafting: the corpus of the chosen workload is split into M member
    automata (sessions dealt round-robin), every stream holds all M with weights from {0.5, 1, 1.5}; a step is
    sam_verify followed by sam_multi_draft on the accepted tokens.  Prints its own JSON line."""
    import torch
    import paper_2512_18337_b200 as S
    from paper_2512_18337_b200.build import build

    device = "cuda:0"
    torch.cuda.set_device(device)
    build()
    M = args.multi
    cfg = W.CONFIGS[args.config].scaled(steps=args.warmup + args.steps + 1)
    corpus, logits, rowmax = make_inputs_gpu(cfg, device)
    scripts = W.make_scripts(cfg, corpus)
    ln = cfg.session_len + 1
    padded = np.concatenate([corpus, [cfg.separator]]).reshape(cfg.sessions, ln)
    t0 = time.time()
    members = [S.SamIndex(np.ascontiguousarray(padded[m::M]).reshape(-1)[:-1], [cfg.separator], device=device) for m in range(M)]
    t_build = time.time() - t0
    sset = S.SamSet(members, device=device)
    B, K, V = cfg.B, cfg.K, cfg.vocab
    rng = np.random.default_rng(cfg.seed)
    i32 = dict(dtype=torch.int32, device=device)
    slots = torch.arange(M, **i32).repeat(B, 1).contiguous()
    weights = torch.from_numpy(rng.choice(np.array([0.5, 1.0, 1.5], np.float32), size=(B, M))).to(device)
    st, ml = torch.zeros((B, M), **i32), torch.zeros((B, M), **i32)
    drafts, n_draft, chosen = torch.full((B, K), -1, **i32), torch.zeros(B, **i32), torch.zeros(B, **i32)
    am, acc, nacc = torch.zeros((B, K + 1), **i32), torch.zeros((B, K + 1), **i32), torch.zeros(B, **i32)
    wsb = S.sam_multi_workspace_bytes(B, K, M)
    ws = torch.empty(wsb, dtype=torch.uint8, device=device)
    S.sam_workspace_init(ws, wsb)
    raw = logits.view(torch.int16)
    feeder = W.ClosedLoopFeeder(cfg, scripts, rowmax)
    toks, n = feeder.prime_tokens()
    S.sam_multi_draft(sset.handle, B, M, slots, weights, st, ml, torch.from_numpy(toks).to(device), toks.shape[1],
                      torch.from_numpy(n).to(device), K, cfg.min_match, drafts, n_draft, chosen)
    torch.cuda.synchronize()
    ev = [tuple(torch.cuda.Event(enable_timing=True) for _ in range(3)) for _ in range(args.steps)]
    tokens = drafted = 0
    for t in range(args.warmup + args.steps):
        ow = feeder.overwrites(t, drafts.cpu().numpy(), n_draft.cpu().numpy())
        r, c = torch.from_numpy(ow["row"]).to(device), torch.from_numpy(ow["col"]).to(device)
        saved = raw[r, c].clone()
        raw[r, c] = torch.from_numpy(ow["bits"].view(np.int16)).to(device)
        i = t - args.warmup
        if i >= 0:
            drafted += int(n_draft.sum())
            torch.cuda._sleep(args.presleep_cycles)
            ev[i][0].record()
        if args.multi_unfused:
            S.sam_verify(logits, V, B, K, V, drafts, n_draft, am, acc, nacc, ws, wsb)
            if i >= 0:
                ev[i][1].record()
            S.sam_multi_draft(sset.handle, B, M, slots, weights, st, ml, acc, K + 1, nacc, K, cfg.min_match, drafts, n_draft, chosen)
        else:
            if i >= 0:
                ev[i][1].record()
            S.sam_multi_step(sset.handle, logits, V, B, K, V, drafts, n_draft, am, acc, nacc, M, slots, weights, st, ml,
                             cfg.min_match, drafts, n_draft, chosen, ws, wsb)
        if i >= 0:
            ev[i][2].record()
        torch.cuda.synchronize()
        raw[r, c] = saved
        n_acc = nacc.cpu().numpy()
        feeder.advance(n_acc)
        if i >= 0:
            tokens += int(n_acc.sum())
    ms = float(sum(e[0].elapsed_time(e[2]) for e in ev))
    ms_multi = float(sum(e[1].elapsed_time(e[2]) for e in ev))
    print(json.dumps({
        "metric": METRIC + "_composite", "value": tokens / (ms / 1e3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "dtype": "bf16 compare / int32",
        "data": "synthetic",
        "config": {"workload": cfg.name + f" split into {M} member automata, every stream holds all {M}", "B": B, "K": K,
                   "V": V, "api": "sam_verify + sam_multi_draft" if args.multi_unfused else "sam_multi_step",
                   "timing": "CUDA events around the step"},
        "multi_draft_kernel_ms": (ms_multi / args.steps) if args.multi_unfused else None,
        "mean_n_draft": drafted / (B * args.steps), "ote": tokens / (B * args.steps), "members_build_s": t_build,
    }))


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload index 0..5 (default 2: B=256, K=16; 5: the paper's evaluation shape, B=4, K=3)")
    ap.add_argument("--streams", type=int, default=0, help="override the workload's number of streams B (per GPU)")
    ap.add_argument("--e2e-steps", type=int, default=11,
                    help="steps of each end-to-end loop through the host-buffer entry point (the first one warms "
                         "the pinned path and is not timed)")
    ap.add_argument("--presleep-cycles", type=int, default=300000,
                    help="length of the spin kernel enqueued before each timed step (outside the events)")
    ap.add_argument("--variant", type=int, default=0, choices=[0, 1, 2, 3],
                    help="kernel selection of the library (0 = default: by size - bulk-copy argmax kernel above 768 MiB of "
                         "logits or K > 16, direct-load kernel below, each + accept kernel; 1 = direct-load argmax + accept; "
                         "2 = bulk-copy kernel with the accept step inside, one launch per step; 3 = bulk-copy + accept)")
    ap.add_argument("--split-steps", type=int, default=50,
                    help="steps run after the timed region with two kernels per step, to report each kernel's time")
    ap.add_argument("--cpu-steps", type=int, default=200)
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--skip-unused-rows", action="store_true",
                    help="verify only rows 0..n_draft[b] of every stream (SAM_STEP_SKIP_UNUSED_ROWS); a different "
                         "workload from the default one, which reads all B*(K+1) rows")
    ap.add_argument("--vocab-shards", type=int, default=0,
                    help="> 0: time verification over a column-sharded vocabulary (one shard per rank under torchrun; "
                         "all shards one after the other on a single GPU); prints a separate JSON line")
    ap.add_argument("--multi", type=int, default=0,
                    help="> 0: closed loop with composite drafting over that many member automata (1..8); separate JSON line")
    ap.add_argument("--multi-unfused", action="store_true", help="with --multi: sam_verify + sam_multi_draft instead of sam_multi_step")
    ap.add_argument("--graph", action="store_true",
                    help="capture one sam_step in a CUDA graph after the warm-up and replay it for every timed step")
    ap.add_argument("--growing", action="store_true",
                    help="run the closed loop on a growing index instead (prints a separate JSON line)")
    args = ap.parse_args(argv)
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    return args


def main():
    args = parse_args()
    from harness.launcher import spawn_ranks, under_launcher
    single_process_modes = args.growing or args.multi > 0 or (args.impl == "reference")
    if args.gpus > 1 and not under_launcher() and not single_process_modes:
        # one process per GPU: this script again, under the torch launcher, with the same arguments
        sys.exit(spawn_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args)
    elif args.growing:
        run_growing(args)
    elif args.multi > 0:
        run_multi(args)
    elif args.vocab_shards > 0:
        run_vocab_parallel(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
