#!/usr/bin/env python
"""Benchmark of the tree-verification step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole hot path over one batch of synthetic input:
tree_build_mask, tree_verify_attn for every layer, tree_accept, kv_commit.
Prints one JSON line (rank 0).  With --gpus N (launched under torchrun) every
rank runs its own batch of the same shape (sequence sharding, no data-path
collective) and the value is the aggregate over ranks, timed as the max over
ranks.  --impl reference times the fp64 CPU oracle on a bounded sample.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import CONFIGS, get_config, make_case, bf16_bits  # noqa: E402

METRIC = "tree_verify_steps_per_sec"
UNIT = "steps/s"
# DRAM bytes per tree_verify_attn launch from ncu (dram__bytes_read.sum + dram__bytes_write.sum), as a ratio to
# the algorithmic bytes.  Captured on gqa8b_ragged (162.0 MB / 160.1 MB) and long_context (547.9 MB / 547.4 MB),
# see profiles/tree_attn_kernel_*.md; full_step_32l holds too much memory for a full capture and takes the ratio of
# a 4-layer launch of its own shape (613.5 MB / 616.1 MB); llama7b_layer holds too little work for
# a capture larger than L2 and takes the ragged-batch ratio; traffic grows with the sum of (prefix + tree) keys.
L2_BYTES = 126 * 1024 * 1024
NCU_TRAFFIC_RATIO = {"gqa8b_ragged": 1.012, "long_context": 1.001, "full_step_32l": 0.996, "llama7b_layer": 1.012}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index, period_s=0.004):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.period = period_s
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or getattr(
            nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = get_reasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def attn_algorithmic_bytes(cfg, prefix_len):
    """K and V once over prefix + tree keys, Q in and O out, per layer (bf16)."""
    keys = int(np.sum(prefix_len.astype(np.int64) + cfg.N))
    return 2 * 2 * cfg.Hkv * cfg.d * keys + 2 * 2 * cfg.B * cfg.N * cfg.Hq * cfg.d


def attn_flops(cfg, prefix_len):
    keys = int(np.sum(prefix_len.astype(np.int64) + cfg.N))
    return 4 * cfg.Hq * cfg.N * cfg.d * keys


def input_copies(cfg):
    """(copies of a step's inputs that are used in turn, bytes of one copy, note for the JSON line).  A step whose
    inputs fit the 126 MB L2 would be timed L2-warm: such workloads cycle through copies of the big inputs (same
    values, distinct memory), enough of them to exceed L2 between two uses of one copy."""
    e = 2
    per_layer = cfg.B * (cfg.N * cfg.Hq * cfg.d + 2 * cfg.N * cfg.Hkv * cfg.d + 2 * cfg.Hkv * cfg.Scap * cfg.d)   # q, tree K/V, cache
    step_bytes = e * (cfg.L * per_layer + cfg.B * cfg.N * cfg.V)                                                  # + logits
    n_sets = 1 if step_bytes > 2 * L2_BYTES else min(8, int(2 * L2_BYTES // max(step_bytes, 1)) + 2)
    if n_sets == 1:
        note = "inputs larger than L2 (each step streams the whole KV cache and the logits)"
    elif n_sets * step_bytes > L2_BYTES:
        note = (f"{n_sets} copies of the inputs ({step_bytes / 1e6:.0f} MB each) used in turn, so that a copy has left "
                "L2 before it is read again")
    else:
        note = (f"L2-resident: {n_sets} copies of the inputs ({step_bytes / 1e6:.2f} MB each) used in turn still fit L2; "
                "a launch-latency-scale workload")
    return n_sets, step_bytes, note


def workload_config(cfg, world, sum_prefix, layers_overridden):
    """The `config` object of the JSON line: the workload, the same on both arms."""
    return {"workload": cfg.name + (f" with {cfg.L} layers" if layers_overridden else ""), "B": cfg.B, "L": cfg.L,
            "N": cfg.N, "D": cfg.D, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "d": cfg.d, "V": cfg.V, "prefix": [cfg.S_lo, cfg.S_hi],
            "sum_prefix": int(sum_prefix), "parallelism": f"sequence-sharded x{world}", "l2": input_copies(cfg)[2]}


# --------------------------------------------------------------------------- oracle legs
def oracle_sample_seconds(cfg, seed):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload and
    scales each stage to a full step.  Returns (estimated seconds per full step, description, threads)."""
    from oracle import tree_verify_oracle as orc
    small = cfg.scaled(L=1, B=min(cfg.B, 4), V=min(cfg.V, 65536) if cfg.V else 0)
    case = make_case(small, seed, device="cpu")
    from workloads import case_to_numpy
    cn = case_to_numpy(case)
    Dp1 = cn["retrieve"].shape[2]
    wall_0, cpu_0 = time.perf_counter(), time.process_time()
    t0 = time.perf_counter()
    mk = orc.build_mask(cn["parent"], cn["n_nodes"], Dp1 - 1, cn["retrieve"].shape[1])
    t_mask = time.perf_counter() - t0
    # attention: one layer, the sampled sequences, all KV heads
    hk_n = small.Hkv
    G = small.Hq // small.Hkv
    t0 = time.perf_counter()
    orc.tree_attention(cn["q"][0][:, :, :hk_n * G], cn["k_cache"][0][:, :hk_n], cn["v_cache"][0][:, :hk_n],
                       cn["k_tree"][0][:, :, :hk_n], cn["v_tree"][0][:, :, :hk_n], cn["prefix_len"],
                       cn["n_nodes"], mk["dense"][:, 0], small.d ** -0.5)
    t_attn = time.perf_counter() - t0
    keys_sample = float(np.sum(cn["prefix_len"].astype(np.int64) + small.N)) * hk_n
    # full-step key count uses the expected prefix length of the config
    keys_full = cfg.B * ((cfg.S_lo + cfg.S_hi) / 2 + cfg.N) * cfg.Hkv * cfg.L
    est = t_mask * cfg.B / small.B + t_attn * keys_full / keys_sample
    desc = (f"oracle on {small.B} of {cfg.B} sequences: mask; attention of 1 layer x {hk_n} KV heads "
            f"(scaled by keys x heads x layers)")
    if cfg.V:
        t0 = time.perf_counter()
        am = orc.argmax_rows(cn["logits"], cn["n_nodes"])
        t_arg = time.perf_counter() - t0
        t0 = time.perf_counter()
        acc = orc.greedy_accept(cn["retrieve"], cn["tokens"], cn["n_nodes"], am)
        t_acc = time.perf_counter() - t0
        t0 = time.perf_counter()
        orc.kv_commit(cn["k_cache"], cn["v_cache"], cn["k_tree"], cn["v_tree"], acc["accepted_nodes"],
                      acc["accept_len"], cn["prefix_len"])
        t_com = time.perf_counter() - t0
        est += t_arg * (cfg.B * cfg.V) / (small.B * small.V) + t_acc * cfg.B / small.B + t_com * cfg.B * cfg.L / small.B
        desc += f"; argmax over {small.V} of {cfg.V} logits per row; accept; commit of 1 layer"
    # Threads the timed code actually used: CPU seconds of the process over wall seconds of the sample.  The oracle
    # is Python loops on one core around numpy calls; only the per-head matmuls can fan out into numpy's BLAS pool.
    wall, cpu = time.perf_counter() - wall_0, time.process_time() - cpu_0
    used = cpu / max(wall, 1e-9)
    try:
        from threadpoolctl import threadpool_info
        pool = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        pool = os.cpu_count() or 1
    desc += f"; CPU seconds / wall seconds of the sample = {used:.2f} (numpy BLAS pool: {pool} threads)"
    return est, desc, max(1, int(round(used)))


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    for _ in range(args.warmup):
        pass      # the oracle has no warm-up state; a warm-up step would only repeat the sample
    ests = []
    t_all = time.perf_counter()
    for s in range(args.steps):
        est, desc, threads = oracle_sample_seconds(cfg, args.seed + s)
        ests.append(est)
        if time.perf_counter() - t_all > 120:
            break
    sec = float(np.mean(ests))
    value = 1.0 / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": len(ests), "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        # the same workload object as the CUDA arm prints (prefix lengths of the same seed; no cache is drawn for it)
        "config": workload_config(cfg, int(os.environ.get("WORLD_SIZE", "1")),
                                  make_case(cfg.scaled(L=1), args.seed, device="cpu", with_cache=False,
                                            with_logits=False)["prefix_len"].sum().item(), args.layers > 0),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- CUDA arm
def run_ours(args, cfg):
    import paper_2603_08088_b200 as tv
    from paper_2603_08088_b200 import dist as tvd
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the treeverify library has no CPU path")
    rank, world, local = tvd.init_from_env("nccl")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    tv.load()
    scale = cfg.d ** -0.5
    case = make_case(cfg, args.seed + rank, device=dev)
    P, Dp1 = case["retrieve"].shape[1], cfg.D + 1
    given_rows = cfg.P > 0
    buf = tv.StepBuffers(cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap, cfg.V, P, Dp1, device=dev)
    prefix0 = case["prefix_len"].clone()
    S_host = prefix0.cpu().numpy()
    has_accept = cfg.V > 0
    ev = lambda: torch.cuda.Event(enable_timing=True)
    # A step whose inputs fit the 126 MB L2 would be timed L2-warm: such workloads cycle through copies of the big
    # inputs (same values, distinct memory), enough of them to exceed L2 between two uses of one copy.
    big = ("q", "k_cache", "v_cache", "k_tree", "v_tree") + (("logits",) if has_accept else ())
    n_sets, step_bytes, l2_note = input_copies(cfg)
    assert step_bytes == sum(case[k].numel() * case[k].element_size() for k in big)
    sets = [case] + [dict(case, **{k: case[k].clone() for k in big}) for _ in range(n_sets - 1)]
    step_no = [0]

    def rest():
        """A second without work before a leg of its own: the headline runs in the first tens of milliseconds, before
        the board reaches its power limit, and a leg that follows it at once would be timed at lower clocks."""
        torch.cuda.synchronize()
        time.sleep(1.0)

    def one_step(marks=None):
        case = sets[step_no[0] % n_sets]
        step_no[0] += 1
        # the commit advances prefix_len; every step starts from the same committed state
        case["prefix_len"].copy_(prefix0)
        if marks is not None and marks[0] is not None:
            marks[0].record()
        tv.tree_build_mask(case["parent"], case["n_nodes"], Dp1 - 1, buf.retrieve.shape[1], buf.anc_bits,
                           buf.status, retrieve_indices=None if given_rows else buf.retrieve, n_paths=buf.n_paths)
        if marks is not None:
            marks[1].record()
        # all layers in one call; the mask kernel in front writes none of the attention's early inputs
        tv.tree_verify_attn_layers(case["q"], case["k_cache"], case["v_cache"], case["k_tree"], case["v_tree"],
                                   case["prefix_len"], case["n_nodes"], buf.anc_bits, scale, buf.out, buf.attn_ws,
                                   buf.status, flags=tv.TV_ATTN_STABLE_INPUTS)
        if marks is not None:
            marks[2].record()
        if has_accept:
            rows = case["retrieve"] if given_rows else buf.retrieve
            tv.tree_accept(case["logits"], case["tokens"], rows, case["n_nodes"], buf.argmax_tok, buf.accept_len,
                           buf.best_path, buf.accepted_nodes, buf.next_token, buf.accept_ws, buf.status)
            tv.kv_commit(case["k_cache"], case["v_cache"], case["k_tree"], case["v_tree"], buf.accepted_nodes,
                         buf.accept_len, case["prefix_len"], buf.status)
        if marks is not None and marks[3] is not None:
            marks[3].record()

    for _ in range(max(args.warmup, 3)):
        one_step()
    torch.cuda.synchronize()
    status = buf.status.cpu().numpy()
    if (status & 15).any():
        raise SystemExit(f"bench.py: fatal per-sequence status after warm-up: {status}")

    # Inside the timed region only the attention launch is bracketed by events (the roofline entry needs its
    # duration there).  An event record between two launches takes the programmatic overlap of the two away, so
    # the mask and accept/commit stages are timed in a short pass of their own behind the timed region.
    sampler = ClockSampler(local)
    marks = [[None, ev(), ev(), None] for _ in range(args.steps)]
    tvd.barrier()
    torch.cuda.synchronize()
    launches0 = tv.tv_launch_count()
    sampler.start()
    t_start, t_end = ev(), ev()
    t_start.record()
    for s in range(args.steps):
        one_step(marks[s])
    t_end.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    launches = tv.tv_launch_count() - launches0
    tvd.barrier()
    elapsed_ms = tvd.max_over_ranks(t_start.elapsed_time(t_end), dev)
    total_steps = tvd.sum_over_ranks(args.steps, dev)
    attn_ms = sum(m[1].elapsed_time(m[2]) for m in marks) / (args.steps * cfg.L)
    n_staged = min(args.steps, 10)
    staged = [[ev() for _ in range(4)] for _ in range(n_staged)]
    for s in range(n_staged):
        one_step(staged[s])
    torch.cuda.synchronize()
    per_step_ms = sorted(m[0].elapsed_time(m[3]) for m in staged)
    tail_us = sum(m[2].elapsed_time(m[3]) for m in staged) / n_staged * 1e3
    mask_us = sum(m[0].elapsed_time(m[1]) for m in staged) / n_staged * 1e3
    mean_accept = float(buf.accept_len.float().mean().item()) if has_accept else None

    # ---- end-to-end through the host-buffer entry point (rank-local, timed with the host clock around
    # the call, which returns after the stream has drained)
    e2e = None
    if has_accept:
        torch.cuda.synchronize()
        pin = lambda t: t.cpu().contiguous().pin_memory()
        host = {k: pin(case[k]) for k in ("parent", "n_nodes", "tokens", "q", "k_tree", "v_tree", "logits")}
        host["retrieve_indices"] = pin(case["retrieve"]) if given_rows else None
        host["P"] = P
        host["out"] = torch.empty(cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.d, dtype=torch.bfloat16).pin_memory()
        for k, shape in (("accept_len", (cfg.B,)), ("accepted_nodes", (cfg.B, Dp1)), ("next_token", (cfg.B,)),
                         ("status", (cfg.B,))):
            host[k] = torch.zeros(shape, dtype=torch.int32).pin_memory()
        staging = torch.empty(tv.tv_step_staging_bytes(cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap,
                                                       cfg.V, P, Dp1), dtype=torch.uint8, device=dev)
        h2d = sum(host[k].numel() * host[k].element_size() for k in
                  ("parent", "n_nodes", "tokens", "q", "k_tree", "v_tree", "logits"))
        if given_rows:
            h2d += host["retrieve_indices"].numel() * 4
        d2h = sum(host[k].numel() * host[k].element_size() for k in
                  ("out", "accept_len", "accepted_nodes", "next_token", "status"))
        e2e_steps = max(3, min(args.steps, 10))
        for _ in range(2):
            case["prefix_len"].copy_(prefix0)
            tv.tv_verify_step_host(host, case["k_cache"], case["v_cache"], case["prefix_len"], staging, scale, cfg.V)
        tvd.barrier()
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(e2e_steps):
            case["prefix_len"].copy_(prefix0)
            tv.tv_verify_step_host(host, case["k_cache"], case["v_cache"], case["prefix_len"], staging, scale, cfg.V)
        e1.record()
        torch.cuda.synchronize()
        e2e_ms = tvd.max_over_ranks(e0.elapsed_time(e1), dev)
        e2e = {"value": tvd.sum_over_ranks(e2e_steps, dev) / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
               "ms_per_step": e2e_ms / e2e_steps}
        if (host["status"].numpy() & 15).any():
            raise SystemExit(f"bench.py: fatal status from the host-buffer step: {host['status'].numpy()}")

    # ---- the same step replayed from a captured CUDA graph (one graph per input copy): what the step costs
    # once the host's launch path is out of the way
    graph_leg = None
    if args.graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            graphs = []
            with torch.cuda.stream(side):
                for i in range(n_sets):
                    step_no[0] = i
                    one_step()
                    torch.cuda.synchronize()
                    step_no[0] = i
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=side):
                        one_step()
                    graphs.append(g)
            torch.cuda.current_stream().wait_stream(side)
            for i in range(3):
                graphs[i % n_sets].replay()
            torch.cuda.synchronize()
            g0, g1 = ev(), ev()
            g0.record()
            for i in range(args.steps):
                graphs[i % n_sets].replay()
            g1.record()
            torch.cuda.synchronize()
            gms = g0.elapsed_time(g1)           # this rank's own clock: no collective inside an optional leg
            graph_leg = {"steps": args.steps, "ms_per_step": gms / args.steps,
                         "steps_per_sec_per_gpu": args.steps / (gms * 1e-3)}
            if (buf.status.cpu().numpy() & 15).any():
                raise SystemExit(f"bench.py: fatal status in the graph replay: {buf.status.cpu().numpy()}")

        except SystemExit:
            raise
        except Exception as exc:      # the optional leg never takes the main line down
            graph_leg = {"error": f"{type(exc).__name__}: {exc}"[:200]}
            torch.cuda.synchronize()

    # ---- multi-layer workloads: the same layers issued as L separate tree_verify_attn calls, back to back (what a
    # caller whose layers depend on each other has to issue: every call is a launch of its own with its own pipeline
    # fill, tail and merges, and reads nothing before the call in front has finished)
    attn_single = None
    if cfg.L > 1:
        rest()
        case["prefix_len"].copy_(prefix0)

        def layer_by_layer():      # issued from C, so that the host's launch path does not bound the figure
            tv.tree_verify_attn_layers(case["q"], case["k_cache"], case["v_cache"], case["k_tree"], case["v_tree"],
                                       case["prefix_len"], case["n_nodes"], buf.anc_bits, scale, buf.out, buf.attn_ws,
                                       buf.status, flags=tv.TV_ATTN_LAUNCH_PER_LAYER)

        layer_by_layer()
        torch.cuda.synchronize()
        reps = 5
        c0, c1 = ev(), ev()
        c0.record()
        for _ in range(reps):
            layer_by_layer()
        c1.record()
        torch.cuda.synchronize()
        attn_single = {"calls": reps * cfg.L, "us_per_layer": c0.elapsed_time(c1) / (reps * cfg.L) * 1e3}

    # ---- the kernel's memory side alone (test entry point of treeverify_debug.h): the same launch, schedule and TMA
    # copies, every shared-memory slot handed back as soon as it has landed, no MMA, no softmax, no output
    stream_only = None
    if hasattr(tv.load(), "tv_debug_attn_stream_only"):      # every rank, like the legs around it
        rest()
        for c in sets:
            c["prefix_len"].copy_(prefix0)

        def stream_pass(i):
            c = sets[i % n_sets]
            tv.tv_debug_attn_stream_only(c["q"], c["k_cache"], c["v_cache"], c["k_tree"], c["v_tree"], c["prefix_len"],
                                         c["n_nodes"], buf.anc_bits, buf.out, buf.attn_ws, buf.status)

        n_so = 5 if cfg.L > 1 else 120
        for i in range(3):
            stream_pass(i)
        torch.cuda.synchronize()
        s0, s1 = ev(), ev()
        s0.record()
        for i in range(n_so):
            stream_pass(i)
        s1.record()
        torch.cuda.synchronize()
        stream_only = {"calls": n_so, "us_per_layer": s0.elapsed_time(s1) / (n_so * cfg.L) * 1e3,
                       "note": "tv_debug_attn_stream_only: the launch's K/V stream with nothing computed"}

    # ---- one-layer workloads: the attention launches alone, back to back on one stream (the step loop above is
    # bound by the host's launch path when a step is a handful of short kernels); inputs cycle through the copies
    attn_b2b = None
    if cfg.L == 1:
        n_b2b = 240
        tv.tree_build_mask(case["parent"], case["n_nodes"], Dp1 - 1, buf.retrieve.shape[1], buf.anc_bits, buf.status,
                           retrieve_indices=None if given_rows else buf.retrieve, n_paths=buf.n_paths)
        for c in sets:
            c["prefix_len"].copy_(prefix0)

        def attn_only(i):
            c = sets[i % n_sets]
            tv.tree_verify_attn(c["q"][0], c["k_cache"][0], c["v_cache"][0], c["k_tree"][0], c["v_tree"][0],
                                c["prefix_len"], c["n_nodes"], buf.anc_bits, scale, buf.out[0], buf.attn_ws, buf.status)

        for i in range(8):
            attn_only(i)
        torch.cuda.synchronize()
        b0, b1 = ev(), ev()
        b0.record()
        for i in range(n_b2b):
            attn_only(i)
        b1.record()
        torch.cuda.synchronize()
        b2b_us = b0.elapsed_time(b1) / n_b2b * 1e3
        attn_b2b = {"launches": n_b2b, "us": b2b_us, "input_copies": n_sets}

    # ---- the same step loop kept running for --sustain seconds (this rank's own clock; the legs that
    # are timed on their own come before it or rest first): what the step costs once the board has
    # reached that limit, with the clocks seen over the region
    def run_sustained():
        sustained = None
        if args.sustain <= 0:
            return None
        n_sus = max(args.steps, int(args.sustain / max(elapsed_ms / args.steps * 1e-3, 1e-6)) + 1)
        every = max(1, n_sus // 64)                       # per-stage events on a subset of the steps
        sm = {i: [ev() for _ in range(4)] for i in range(0, n_sus, every)}
        sus_sampler = ClockSampler(local, period_s=0.02)
        torch.cuda.synchronize()
        sus_sampler.start()
        s0, s1 = ev(), ev()
        s0.record()
        for i in range(n_sus):
            one_step(sm.get(i))
        s1.record()
        torch.cuda.synchronize()
        sus_clocks = sus_sampler.stop()
        sus_ms = s0.elapsed_time(s1)
        late = [m for i, m in sm.items() if i >= n_sus // 2]          # stages over the second half of the region
        sustained = {"seconds": sus_ms * 1e-3, "steps": n_sus, "value": n_sus / (sus_ms * 1e-3), "unit": UNIT + " per GPU",
                     "ms_per_step": sus_ms / n_sus,
                     "attn_per_layer_us": sum(m[1].elapsed_time(m[2]) for m in late) / (len(late) * cfg.L) * 1e3,
                     "accept_commit_us": sum(m[2].elapsed_time(m[3]) for m in late) / len(late) * 1e3,
                     "clocks": sus_clocks}
        if (buf.status.cpu().numpy() & 15).any():
            raise SystemExit(f"bench.py: fatal status in the sustained run: {buf.status.cpu().numpy()}")
        return sustained

    sustained = run_sustained()       # every rank, so that the ranks stay together; the legs behind it rest first

    if rank != 0:
        return
    peak, peak_kind = measured_peaks()
    alg_bytes = attn_algorithmic_bytes(cfg, S_host)
    achieved = alg_bytes / (attn_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": total_steps / (elapsed_ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": elapsed_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(cfg, world, S_host.sum(), args.layers > 0),
        "sequence_steps_per_sec": total_steps * cfg.B / (elapsed_ms * 1e-3),
        "stage_us": {"mask": mask_us, "attn_per_layer": attn_ms * 1e3, "accept_commit": tail_us,
                     "source": f"attn_per_layer: events inside the timed region; mask, accept_commit: {n_staged} "
                               "steps behind it with an event between all stages"},
        "step_ms": {"median": per_step_ms[len(per_step_ms) // 2], "min": per_step_ms[0], "max": per_step_ms[-1],
                    "source": "the staged steps behind the timed region"},
        "mean_accept_len": mean_accept,
        "roofline": {"bound": "hbm", "kernel": "tree_verify_attn", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     # one launch covers all cfg.L layers of the step
                     "traffic": (int(NCU_TRAFFIC_RATIO[cfg.name] * alg_bytes * cfg.L) if cfg.name in NCU_TRAFFIC_RATIO else None),
                     "traffic_source": "ncu dram bytes, scaled by algorithmic bytes from the captured config",
                     "layers_per_launch": cfg.L,
                     "algorithmic_bytes_per_launch": alg_bytes * cfg.L,
                     "avg_launch_us": attn_ms * 1e3 * cfg.L,
                     "tensor_tflops": attn_flops(cfg, S_host) / (attn_ms * 1e-3) / 1e12},
        "clocks": clocks, "gpu_launches": int(launches), "e2e": e2e,
    }
    if graph_leg is not None:
        line["graph_replay"] = graph_leg
    if attn_single is not None:
        attn_single["hbm_gbs"] = alg_bytes / (attn_single["us_per_layer"] * 1e-6) / 1e9
        attn_single["frac"] = attn_single["hbm_gbs"] / peak
        line["attn_single_call"] = attn_single
    if stream_only is not None:
        stream_only["hbm_gbs"] = alg_bytes / (stream_only["us_per_layer"] * 1e-6) / 1e9
        stream_only["frac"] = stream_only["hbm_gbs"] / peak
        line["attn_stream_only"] = stream_only
    if attn_b2b is not None:
        attn_b2b["hbm_gbs"] = alg_bytes / (attn_b2b["us"] * 1e-6) / 1e9
        attn_b2b["frac"] = attn_b2b["hbm_gbs"] / peak
        attn_b2b["tensor_tflops"] = attn_flops(cfg, S_host) / (attn_b2b["us"] * 1e-6) / 1e12
        line["attn_back_to_back"] = attn_b2b
    if args.budget_sweep:
        line["budget_sweep"] = budget_sweep(args.seed, dev)
    if args.in_cache and has_accept:
        rest()
        line["in_cache"] = in_cache_step(cfg, case, buf, prefix0, scale, given_rows, min(args.steps, 20), dev)
        case["prefix_len"].copy_(prefix0)
    if args.sample_accept and has_accept:
        rest()
        line["sample_accept"] = sample_accept_leg(cfg, case, min(args.steps, 20), dev, args.seed)
    if args.paged and has_accept:
        rest()
        line["paged"] = paged_step(cfg, case, buf, prefix0, scale, given_rows, min(args.steps, 20), dev, args.seed)
        case["prefix_len"].copy_(prefix0)
    if args.context_split > 1:
        case["prefix_len"].copy_(prefix0)
        line["context_split"] = context_split_member(cfg, case, buf, args.context_split, dev)
    if args.cpu_baseline:
        sec, desc, threads = oracle_sample_seconds(cfg, args.seed)
        line["cpu_baseline"] = {"value": 1.0 / sec, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": desc, "est_seconds_per_step": sec}
    if sustained is not None:
        sustained["attn_hbm_frac"] = alg_bytes / (sustained["attn_per_layer_us"] * 1e-6) / 1e9 / peak
        line["sustained"] = sustained
    print(json.dumps(line))


def budget_sweep(seed, dev):
    """tree_verify_attn over the node budgets and depths of the paper's sensitivity sweep (Table 2: M from 16 to
    256 draft nodes, depth bounds 4 to 16) on the ragged GQA batch of config 3: one layer, 20 back-to-back
    launches per shape, CUDA events.  M counts draft nodes; the tree has M + 1 rows with the root, capped at
    256 rows (the kernel's limit)."""
    import paper_2603_08088_b200 as tv
    peak, _ = measured_peaks()
    rows = []
    for M, D in ((16, 4), (32, 6), (64, 8), (128, 12), (256, 16)):
        N = min(M + 1, 256)
        cfg = get_config("gqa8b_ragged").scaled(N=N, D=D, tree="spine", L=1, V=0, P=0)
        case = make_case(cfg, seed, device=dev, with_logits=False)
        B = cfg.B
        bits = torch.zeros(B, N, (N + 31) // 32, dtype=torch.int32, device=dev)
        status = torch.zeros(B, dtype=torch.int32, device=dev)
        tv.tree_build_mask(case["parent"], case["n_nodes"], N - 1, 1, bits, status)
        out = torch.empty(B, N, cfg.Hq, cfg.d, dtype=torch.bfloat16, device=dev)
        ws = torch.zeros(tv.tv_attn_workspace_bytes(B, N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap), dtype=torch.uint8, device=dev)

        def run():
            tv.tree_verify_attn(case["q"][0], case["k_cache"][0], case["v_cache"][0], case["k_tree"][0], case["v_tree"][0],
                                case["prefix_len"], case["n_nodes"], bits, cfg.d ** -0.5, out, ws, status)

        for _ in range(3):
            run()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(20):
            run()
        b.record()
        torch.cuda.synchronize()
        us = a.elapsed_time(b) / 20 * 1e3
        S = case["prefix_len"].cpu().numpy()
        if int(status.cpu().numpy().max()) != 0:
            raise SystemExit(f"bench.py: budget sweep M={M}: status {status.cpu().numpy()}")
        rows.append({"M": M, "rows": N, "Dmax": D, "attn_us": us,
                     "hbm_frac": attn_algorithmic_bytes(cfg, S) / (us * 1e-6) / 1e9 / peak,
                     "tensor_tflops": attn_flops(cfg, S) / (us * 1e-6) / 1e12})
    return rows


def in_cache_step(cfg, case, buf, prefix0, scale, given_rows, steps, dev):
    """The same step with the in-cache layout (Section 3.1: the forward pass extends the cache in place; the
    commit is a reorder inside the cache): the tree's K/V are written behind each prefix once, outside the
    timed region, then mask, L x attention (tree tiles read from the cache), accept and kv_commit_inplace are
    timed.  Every step starts from the same state: prefix_len is reset and the rows the commit moved are
    written again (both outside the events of the commit, inside those of the step)."""
    import paper_2603_08088_b200 as tv
    N = cfg.N
    S = prefix0.cpu().tolist()
    if max(s + N for s in S) > cfg.Scap:
        return {"skipped": "a tree does not fit behind its prefix"}
    rows = [(b, s) for b, s in enumerate(S)]
    tree_k = [case["k_tree"][:, b].permute(0, 2, 1, 3).contiguous() for b, _ in rows]
    tree_v = [case["v_tree"][:, b].permute(0, 2, 1, 3).contiguous() for b, _ in rows]

    def place():
        for (b, s), tk, tvv in zip(rows, tree_k, tree_v):
            case["k_cache"][:, b, :, s:s + N] = tk
            case["v_cache"][:, b, :, s:s + N] = tvv

    ev = lambda: torch.cuda.Event(enable_timing=True)
    t_step, t_attn, t_commit = [], [], []
    for it in range(3 + steps):
        case["prefix_len"].copy_(prefix0)
        place()
        m = [ev() for _ in range(5)]
        m[0].record()
        tv.tree_build_mask(case["parent"], case["n_nodes"], cfg.D, buf.retrieve.shape[1], buf.anc_bits, buf.status,
                           retrieve_indices=None if given_rows else buf.retrieve, n_paths=buf.n_paths)
        m[1].record()
        tv.tree_verify_attn_layers(case["q"], case["k_cache"], case["v_cache"], None, None, case["prefix_len"],
                                   case["n_nodes"], buf.anc_bits, scale, buf.out, buf.attn_ws, buf.status,
                                   flags=tv.TV_ATTN_STABLE_INPUTS)
        m[2].record()
        tv.tree_accept(case["logits"], case["tokens"], case["retrieve"] if given_rows else buf.retrieve, case["n_nodes"],
                       buf.argmax_tok, buf.accept_len, buf.best_path, buf.accepted_nodes, buf.next_token, buf.accept_ws,
                       buf.status)
        m[3].record()
        tv.kv_commit_inplace(case["k_cache"], case["v_cache"], buf.accepted_nodes, buf.accept_len, case["prefix_len"], N,
                             buf.status)
        m[4].record()
        torch.cuda.synchronize()
        if it >= 3:
            t_step.append(m[0].elapsed_time(m[4]))
            t_attn.append(m[1].elapsed_time(m[2]) / cfg.L)
            t_commit.append(m[3].elapsed_time(m[4]))
    if (buf.status.cpu().numpy() & 15).any():
        raise SystemExit(f"bench.py: fatal status in the in-cache step: {buf.status.cpu().numpy()}")
    med = lambda v: sorted(v)[len(v) // 2]
    return {"steps": steps, "ms_per_step_median": med(t_step), "steps_per_sec": 1e3 / med(t_step),
            "attn_per_layer_us": med(t_attn) * 1e3, "commit_inplace_us": med(t_commit) * 1e3,
            "note": "tree K/V read from the cache rows behind the prefix; commit = reorder inside the cache"}


def sample_accept_leg(cfg, case, steps, dev, seed):
    """tree_accept_sample (temperature 1, seeded uniforms) on the workload's logits, L2 flushed between calls,
    beside the greedy tree_accept of the step."""
    import paper_2603_08088_b200 as tv
    B, N, V, Dp1 = cfg.B, cfg.N, cfg.V, cfg.D + 1
    g = torch.Generator(device=dev).manual_seed(seed)
    u_node = torch.rand(B, N, device=dev, generator=g)
    u_bonus = torch.rand(B, device=dev, generator=g)
    z = lambda *s_: torch.zeros(s_, dtype=torch.int32, device=dev)
    alen, nodes, nxt, status = z(B), z(B, Dp1), z(B), z(B)
    ws = torch.zeros(max(16, tv.tv_sample_workspace_bytes(B, N, V)), dtype=torch.uint8, device=dev)
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)
    ts = []
    for it in range(2 + steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        tv.tree_accept_sample(case["logits"], case["tokens"], case["parent"], case["n_nodes"], u_node, u_bonus, 1.0, alen,
                              nodes, nxt, ws, status)
        e1.record()
        torch.cuda.synchronize()
        if it >= 2:
            ts.append(e0.elapsed_time(e1) * 1e3)
    ts.sort()
    return {"steps": steps, "temperature": 1.0, "us_median": ts[len(ts) // 2], "us_min": ts[0],
            "mean_accept_len": float(alen.float().mean().item()), "logits_mb": case["logits"].numel() * 2 / 1e6}


def paged_step(cfg, case, buf, prefix0, scale, given_rows, steps, dev, seed):
    """The same step over a paged committed cache: every sequence's rows cut into pages of 128 rows that are
    scattered over a pool in a seeded random order (one block table for all layers), then mask, L x
    tree_verify_attn_paged, accept and kv_commit_paged are timed.  The pool is built once, outside the timed
    region; every step starts from the same prefix lengths (the commit rewrites the same rows)."""
    import paper_2603_08088_b200 as tv
    L, B, Hkv, Scap, d = case["k_cache"].shape
    nb = (Scap + 127) // 128
    n_pages = B * nb
    g = torch.Generator().manual_seed(seed)
    order = torch.randperm(n_pages, generator=g).to(dev)
    bt = order.view(B, nb).to(torch.int32).contiguous()
    def paginate(cache):
        pool = torch.zeros(L, n_pages, Hkv, 128, d, dtype=cache.dtype, device=dev)
        for b in range(B):
            rows = torch.zeros(L, Hkv, nb * 128, d, dtype=cache.dtype, device=dev)
            rows[:, :, :Scap] = cache[:, b]
            pool[:, bt[b].long()] = rows.view(L, Hkv, nb, 128, d).permute(0, 2, 1, 3, 4)
        return pool
    k_pages, v_pages = paginate(case["k_cache"]), paginate(case["v_cache"])
    ev = lambda: torch.cuda.Event(enable_timing=True)
    t_step, t_attn, t_commit = [], [], []
    for it in range(3 + steps):
        case["prefix_len"].copy_(prefix0)
        m = [ev() for _ in range(5)]
        m[0].record()
        tv.tree_build_mask(case["parent"], case["n_nodes"], cfg.D, buf.retrieve.shape[1], buf.anc_bits, buf.status,
                           retrieve_indices=None if given_rows else buf.retrieve, n_paths=buf.n_paths)
        m[1].record()
        tv.tree_verify_attn_paged_layers(case["q"], k_pages, v_pages, bt, case["k_tree"], case["v_tree"], case["prefix_len"],
                                         case["n_nodes"], buf.anc_bits, scale, buf.out, buf.attn_ws, buf.status,
                                         flags=tv.TV_ATTN_STABLE_INPUTS)
        m[2].record()
        tv.tree_accept(case["logits"], case["tokens"], case["retrieve"] if given_rows else buf.retrieve, case["n_nodes"],
                       buf.argmax_tok, buf.accept_len, buf.best_path, buf.accepted_nodes, buf.next_token, buf.accept_ws,
                       buf.status)
        m[3].record()
        tv.kv_commit_paged(k_pages, v_pages, bt, case["k_tree"], case["v_tree"], buf.accepted_nodes, buf.accept_len,
                           case["prefix_len"], buf.status)
        m[4].record()
        torch.cuda.synchronize()
        if it >= 3:
            t_step.append(m[0].elapsed_time(m[4]))
            t_attn.append(m[1].elapsed_time(m[2]) / L)
            t_commit.append(m[3].elapsed_time(m[4]))
    if (buf.status.cpu().numpy() & 15).any():
        raise SystemExit(f"bench.py: fatal status in the paged step: {buf.status.cpu().numpy()}")
    med = lambda v: sorted(v)[len(v) // 2]
    return {"steps": steps, "page_rows": 128, "n_pages": n_pages, "ms_per_step_median": med(t_step),
            "steps_per_sec": 1e3 / med(t_step), "attn_per_layer_us": med(t_attn) * 1e3,
            "commit_paged_us": med(t_commit) * 1e3,
            "note": "committed cache in pages of 128 rows scattered over the pool, one block table for all layers"}


def context_split_member(cfg, case, buf, R, dev):
    """What one member of an R-way context split of this workload does per layer, timed on this GPU: attention
    over its 1/R of every prefix (it owns the tree keys, the worst case) and the merge of R gathered partials.
    The all-gather itself needs R GPUs and is not timed here; its payload is reported."""
    import paper_2603_08088_b200 as tv
    from paper_2603_08088_b200 import dist as tvd
    B, N, Hq, d = cfg.B, cfg.N, cfg.Hq, cfg.d
    lo, hi = tvd.split_prefix(case["prefix_len"], R - 1, R)
    local_len = (hi - lo).to(torch.int32)
    out = torch.empty(B, N, Hq, d, dtype=torch.bfloat16, device=dev)
    lse = torch.empty(B, Hq, N, dtype=torch.float32, device=dev)
    o_parts = torch.randn(R, B, N, Hq, d, device=dev).to(torch.bfloat16)
    l_parts = torch.randn(R, B, Hq, N, device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def attn():
        tv.tree_verify_attn(case["q"][0], case["k_cache"][0], case["v_cache"][0], case["k_tree"][0], case["v_tree"][0],
                            local_len, case["n_nodes"], buf.anc_bits, d ** -0.5, out, buf.attn_ws, buf.status, lse=lse)

    def merge():
        tv.tree_merge_partials(o_parts, l_parts, out, lse)

    res = {}
    for name, fn in (("attn", attn), ("merge", merge)):
        for _ in range(3):
            fn()
        a, b = ev(), ev()
        torch.cuda.synchronize()
        a.record()
        for _ in range(20):
            fn()
        b.record()
        torch.cuda.synchronize()
        res[name] = a.elapsed_time(b) / 20 * 1e3
    gather_bytes = (R - 1) * (B * N * Hq * d * 2 + B * Hq * N * 4)
    merge_bytes = R * (B * N * Hq * d * 2 + B * Hq * N * 4) + B * N * Hq * d * 2 + B * Hq * N * 4
    return {"members": R, "member_attn_us": res["attn"], "merge_us": res["merge"],
            "merge_gbs": merge_bytes / (res["merge"] * 1e-6) / 1e9,
            "allgather_bytes_received_per_member": gather_bytes,
            "note": "one member timed on one GPU (back-to-back launches, inputs re-read from L2 where they fit); "
                    "the all-gather is not timed"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="full_step_32l", choices=[c.name for c in CONFIGS])
    ap.add_argument("--seed", type=int, default=4000)
    ap.add_argument("--layers", type=int, default=0,
                    help="override the workload's layer count (a smaller case of the same shape, e.g. for an ncu capture)")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--budget-sweep", action="store_true",
                    help="also time tree_verify_attn over the node budgets of the paper's sweep (extra key in the JSON line)")
    ap.add_argument("--in-cache", action="store_true",
                    help="also time the step with the tree's K/V inside the cache and the in-place commit")
    ap.add_argument("--sustain", type=float, default=2.0,
                    help="seconds the step loop is kept running after the headline for the power-capped figure (0: skip)")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="skip the extra leg that times the step replayed from a captured CUDA graph")
    ap.add_argument("--sample-accept", action="store_true",
                    help="also time the sampling-mode acceptance (tree_accept_sample) on the workload's logits")
    ap.add_argument("--paged", action="store_true",
                    help="also time the step over a paged committed cache (pages of 128 rows, block table)")
    ap.add_argument("--context-split", type=int, default=1,
                    help="also time one member of an R-way context split of the workload (extra key in the JSON line)")
    args = ap.parse_args()
    cfg = get_config(args.workload)
    if args.layers > 0:
        cfg = cfg.scaled(L=args.layers)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        if int(os.environ.get("WORLD_SIZE", "1")) > 1:
            args.cpu_baseline = False      # the CPU baseline is reported at N=1 only
        run_ours(args, cfg)
    try:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()
    except Exception:
        pass


if __name__ == "__main__":
    main()
