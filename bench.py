"""Benchmark of the Lazy Attention decode step (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--mode vla_qc|vla_eq8|gla]
    python bench.py --impl reference ...      # times the CPU oracle on the same workload

A step is one qc_decode_step over the whole batch (append + Q Cache write + split-KV partial
attention + log-sum-exp merge, all layers).  `value` is decode tokens/s with inputs resident
in HBM under the in-order schedule (one launch per layer, each using nothing of later layers);
`e2e` is the same through qc_decode_step_host with pinned HOST buffers (q, k, v copied in, out
copied back, inside the timed region).  Without --workload the headline is the largest
configuration and `per_config` holds a record for each of the other model-shaped ones.  With
N > 1 every rank runs its own batch of the same shape on its own GPU (independent sequences: no
collective on the data path); the time is the maximum over ranks.  `--gpus N` starts the N
ranks itself unless a launcher already did.
"""

from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "decode_attention_tokens_per_s"
UNIT = "tokens/s"
MODES = {"vla_qc": 0, "vla_eq8": 1, "gla": 2}

# (dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic K/V bytes of one attention launch of the
# in-order schedule, from ncu captures of small cases of the same shapes (first 8 layers: launches of
# 181-257 MB for the MHA kernel, 74-107 MB for the GQA kernel).  Every tile is fetched once and the
# partial rows are written once per piece, so traffic grows in proportion to the K/V bytes swept and a
# full-size launch's traffic is this ratio times its algorithmic bytes.
NCU_TRAFFIC_RATIO = {"attend_kernel": 1.028, "attend_tc_kernel": 1.057}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the GPU is timed."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def _physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# ------------------------------------------------------------------------------------------
# CPU oracle leg (bounded, fixed sample)
# ------------------------------------------------------------------------------------------

ORACLE_STEPS = 16         # decode steps each sampled sub-problem is advanced through


def _host_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def _oracle_unit(job):
    """One sampled sub-problem on one core: the whole layer stack of one (sequence, KV head) with its
    query heads, advanced through ORACLE_STEPS decode steps.  Returns the seconds spent inside the
    oracle's decode_step (input generation is not the oracle's work)."""
    name, mode, first_step, unit = job
    from threadpoolctl import threadpool_limits

    from oracle.lazy_attention import LazyAttentionOracle
    from paper_2602_01901_b200 import workloads as W

    w = W.get_workload(name)
    f64 = W.bf16_bits_to_f64
    g = w.group
    seq, kvh = unit % w.batch, (unit // w.batch) % w.n_kv_heads
    heads = list(range(kvh * g, (kvh + 1) * g))
    spent = 0.0
    with threadpool_limits(limits=1):
        o = LazyAttentionOracle(w.n_layers, g, 1, w.head_dim, w.layer_kind().tolist(), mode, n_seqs=1)
        kind, k, v = W.prefill_kv_np(w, seq, heads=[kvh])
        o.prefill_append(0, kind.tolist(), f64(k), f64(v))
        for step in range(first_step):   # untimed catch-up to the first timed context (only the appends matter)
            q, kk, vv = W.decode_qkv_np(w, step, seqs=[seq], q_heads=heads, kv_heads=[kvh])
            for l in range(w.n_layers):
                o.V_T[l][0].append(f64(vv[l, 0]))
                if o.K_T[l][0] is not None:
                    o.K_T[l][0].append(f64(kk[l, 0]))
        for step in range(first_step, first_step + ORACLE_STEPS):
            q, kk, vv = W.decode_qkv_np(w, step, seqs=[seq], q_heads=heads, kv_heads=[kvh])
            qf, kf, vf = f64(q[:, 0]), f64(kk[:, 0]), f64(vv[:, 0])
            t0 = time.perf_counter()
            o.decode_step(0, qf, kf, vf)
            spent += time.perf_counter() - t0
    return spent


def cpu_oracle_sample(w, mode: int, first_step: int):
    """Time the fp64 oracle, as it stands, on a fixed sample of the workload, on all host cores.

    Sample: four whole-stack sub-problems per core (all layers, one sequence, one KV head with its
    query heads; sub-problem i is sequence i mod batch, KV head i div batch), each advanced through
    ORACLE_STEPS decode steps from the context of the benchmark's first timed step, one process per
    core.  One generated token of the workload costs n_kv_heads sub-problem steps, so tokens/s =
    sub-problem steps / (core-seconds inside the oracle / cores) / n_kv_heads.
    """
    import multiprocessing as mp

    cores = _host_cores()
    n_units = min(4 * cores, w.batch * w.n_kv_heads)
    cores = min(cores, n_units)
    jobs = [(w.name, mode, first_step, u) for u in range(n_units)]
    ctx = mp.get_context("spawn")
    with ctx.Pool(cores) as pool:
        spent = pool.map(_oracle_unit, jobs, chunksize=1)
    # throughput of the cores together: sub-problem steps per core-second inside the oracle, times the cores
    # (the mean over sub-problems, so that one straggler on a shared host does not decide the figure)
    core_seconds = float(sum(spent))
    tokens_per_s = n_units * ORACLE_STEPS / (core_seconds / cores) / w.n_kv_heads
    return {
        "value": tokens_per_s, "unit": UNIT, "cores": cores, "kind": "oracle",
        "sample": f"{n_units} (sequence, KV head) sub-problems x all {w.n_layers} layers x {ORACLE_STEPS} decode steps "
                  f"from context {w.n_prompt + first_step} of {w.name}, one process per core; {core_seconds:.1f} core-seconds "
                  f"inside the oracle (slowest sub-problem {max(spent):.2f} s); scaled by 1/{w.n_kv_heads} KV heads per token",
    }


# ------------------------------------------------------------------------------------------
# GPU arms
# ------------------------------------------------------------------------------------------

def _gen_inputs(w, first, count, device, seq_offset=0):
    from paper_2602_01901_b200 import workloads as W

    return [W.decode_qkv_torch(w, s, device, seq_offset) for s in range(first, first + count)]


class _Arms:
    """The timed arms of one workload on one GPU, all on one cache: consecutive decode steps under
    different schedules (a schedule changes how a step is cut into launches, never its result).  The
    context grows by one token per step, so a later arm sweeps more bytes per step than an earlier one:
    every record carries its context range, and GB/s figures are the ones to compare across arms."""

    def __init__(self, args, w, mode, group, local_rank, seq_offset, all_full=False):
        import torch

        from paper_2602_01901_b200 import binding as qc
        from paper_2602_01901_b200.session import Session

        self.torch, self.w, self.group, self.args = torch, w, group, args
        self.dev = torch.device("cuda", local_rank)
        self.s = Session.for_workload(w, lazy_mode=mode, device=local_rank, split_tokens=args.split_tokens,
                                      all_full=all_full)
        self.s.prefill_workload(w, seq_offset)
        self.ids = qc._i32_array(list(range(w.batch)))
        self.out = torch.empty((w.n_layers, w.batch, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device=self.dev)
        self.step = 0
        self.seq_offset = seq_offset

    def barrier(self):
        self.group.barrier()
        self.torch.cuda.synchronize()

    def set(self, options):
        for key, value in options:
            self.s.set_option(key, value)

    def run(self, n, timed=True, profile=0):
        """n consecutive decode steps; returns ms per step (max over ranks), K/V bytes per step, the
        library's profile of the region (if asked for) and its kernel launches."""
        torch = self.torch
        if self.step + n > self.w.decode_steps:
            raise SystemExit(f"{self.w.name}: the arms need more than the workload's {self.w.decode_steps} decode steps")
        inputs = _gen_inputs(self.w, self.step, n, self.dev, self.seq_offset)
        self.s.set_option("profile", profile)
        st0 = self.s.stats()
        self.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n):
            self.s.decode_step(self.ids, *inputs[i], self.out)
        e1.record()
        self.barrier()
        ms = self.group.max_over_ranks(e0.elapsed_time(e1)) / n
        prof = self.s.profile() if profile else None
        self.s.set_option("profile", 0)
        st1 = self.s.stats()
        if st1.device_error:
            raise SystemExit(f"device error word = {st1.device_error}")
        self.step += n
        return {"ms_per_step": ms, "kv_bytes_per_step": (st1.kv_bytes_swept - st0.kv_bytes_swept) / n,
                "launches_per_step": (st1.kernel_launches - st0.kernel_launches) / n,
                "context_first": self.w.n_prompt + self.step - n + 1, "context_last": self.w.n_prompt + self.step,
                "prof": prof}

    def run_layer_calls(self, n):
        """n steps through qc_decode_begin / qc_decode_layer, every layer's tensors passed on their own."""
        torch = self.torch
        inputs = _gen_inputs(self.w, self.step, n + 2, self.dev, self.seq_offset)
        outs = [torch.empty(self.out.shape[1:], dtype=torch.bfloat16, device=self.dev) for _ in range(self.w.n_layers)]

        from paper_2602_01901_b200 import binding as qc

        # raw pointers of every (step, layer) slice, taken ahead of the timed loop: the loop itself is
        # one C call per layer, as a model's runtime would make them
        ptrs = [[(q[l].data_ptr(), k[l].data_ptr(), v[l].data_ptr(), outs[l].data_ptr()) for l in range(self.w.n_layers)]
                for q, k, v in inputs]
        cache, ids = self.s.cache, self.ids

        def step(i):
            qc.qc_decode_begin(cache, ids)
            for l, (qp, kp, vp, op) in enumerate(ptrs[i]):
                qc.qc_decode_layer(cache, l, qp, kp, vp, op)

        for i in range(2):
            step(i)
        st0 = self.s.stats()
        self.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(2, n + 2):
            step(i)
        e1.record()
        self.barrier()
        ms = self.group.max_over_ranks(e0.elapsed_time(e1)) / n
        st1 = self.s.stats()
        if st1.device_error:
            raise SystemExit(f"device error word = {st1.device_error}")
        self.step += n + 2
        return {"ms_per_step": ms, "kv_bytes_per_step": (st1.kv_bytes_swept - st0.kv_bytes_swept) / n,
                "context_first": self.w.n_prompt + self.step - n + 1, "context_last": self.w.n_prompt + self.step}

    def run_host(self, n):
        """n steps through qc_decode_step_host with pinned host buffers; returns tokens/s inputs."""
        torch = self.torch
        warm = 3   # untimed: the entry point's launch plan, copy streams and events are made on its first call
        dev_in = _gen_inputs(self.w, self.step, warm + n, self.dev, self.seq_offset)
        host_in = [tuple(t.cpu().pin_memory() for t in step) for step in dev_in]
        host_out = torch.empty(self.out.shape, dtype=torch.bfloat16).pin_memory()
        del dev_in
        for i in range(warm):
            self.s.decode_step_host(self.ids, *host_in[i], host_out)
        self.barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for i in range(warm, warm + n):
            self.s.decode_step_host(self.ids, *host_in[i], host_out)   # returns after the copy back has finished
        g1.record()
        self.barrier()
        ms = self.group.max_over_ranks(g0.elapsed_time(g1)) / n
        self.step += warm + n
        return {"ms_per_step": ms, "h2d": sum(t.numel() * 2 for t in host_in[0]), "d2h": host_out.numel() * 2,
                "context_first": self.w.n_prompt + self.step - n + 1, "context_last": self.w.n_prompt + self.step}

    def check_output(self):
        checksum = float(self.out.float().abs().sum().item())
        if not np.isfinite(checksum) or checksum == 0.0:
            raise SystemExit("output is not finite / all zero")

    def close(self):
        st = self.s.stats()
        self.s.close()
        del self.s, self.out
        self.torch.cuda.empty_cache()
        return st


IN_ORDER = [("in_order_launches", 1)]
ONE_LAUNCH = [("in_order_launches", 0), ("layers_per_launch", 0)]


def measure_workload(args, w, mode, group, local_rank, world, rank, K, W_, Ke, extra_arms):
    """All arms of one workload.  The headline arm is the in-order schedule (one launch per layer,
    each using nothing of later layers: what a model that computes layer after layer can issue),
    timed with the library's profiling off; the same schedule is then run with events around every
    attention launch for the kernel's own time.  The one-launch schedule (every layer's q/k/v known
    up front, which only a harness has) is reported beside it."""
    peak, peak_kind = _peaks()
    kernel = "attend_tc_kernel" if w.group > 1 else "attend_kernel"
    a = _Arms(args, w, mode, group, local_rank, rank * w.batch)
    a.set(IN_ORDER)
    for kv in args.option:
        key, value = kv.split("=")
        a.s.set_option(key, int(value))
    a.run(W_, timed=False)
    launches0 = a.s.stats().kernel_launches
    with ClockSampler(_physical_gpu_index(local_rank)) as clocks:
        main = a.run(K)
    gpu_launches = int(a.s.stats().kernel_launches - launches0)
    a.check_output()
    kp = a.run(min(K, 16), profile=2)           # the kernel's own time, launch by launch
    prof = kp["prof"]
    n_launch = max(1, prof.attend_kernel_launches)
    kernel_gbs = prof.kv_bytes_read / (prof.attend_kernel_ms / 1e3) / 1e9
    host = a.run_host(Ke)                       # next to the headline steps: nearly the same contexts
    a.set(ONE_LAUNCH)
    a.run(3, timed=False)
    one = a.run(K)
    onep = a.run(min(K, 16), profile=1)["prof"]
    one_attend_ms = onep.attend_ms / max(1, onep.steps)
    one_gbs = onep.kv_bytes_read / (onep.attend_ms / 1e3) / 1e9
    extra = {}
    if extra_arms and world == 1:
        a.set([("layers_per_launch", 1)])
        a.run(3, timed=False)
        pb = a.run(min(K, 24))
        extra["per_block_launches"] = {
            "ms_per_step": pb["ms_per_step"], "kv_gb_per_s_whole_step": pb["kv_bytes_per_step"] / pb["ms_per_step"] / 1e6,
            "context": [pb["context_first"], pb["context_last"]],
            "note": "one attention + merge launch per lazy block, blocks in layer order (needs a block's q/k/v at once)"}
        a.set([("per_layer_logit_cache", 1)])
        a.run(3, timed=False)
        pl = a.run(min(K, 24))
        extra["per_layer_logit_cache"] = {
            "ms_per_step": pl["ms_per_step"], "kv_gb_per_s_whole_step": pl["kv_bytes_per_step"] / pl["ms_per_step"] / 1e6,
            "context": [pl["context_first"], pl["context_last"]],
            "note": "one launch per layer; followers sweep their V with the leader's scores from a logit cache"}
        a.set(IN_ORDER)
        lc = a.run_layer_calls(min(K, 24))
        extra["layer_calls"] = {
            "ms_per_step": lc["ms_per_step"], "kv_gb_per_s_whole_step": lc["kv_bytes_per_step"] / lc["ms_per_step"] / 1e6,
            "context": [lc["context_first"], lc["context_last"]],
            "note": "the in-order step through qc_decode_begin + one qc_decode_layer per layer (each call gets only "
                    "that layer's q/k/v and also appends them: one more small launch per layer)"}
    st = a.close()
    tokens = w.batch * world
    res = {
        "workload": w.name, "mode": args.mode, "schedule": "in_order (one launch per layer, layers in order)",
        "tokens_per_s": tokens / (main["ms_per_step"] / 1e3), "ms_per_step": main["ms_per_step"],
        "context": [main["context_first"], main["context_last"]],
        "kv_bytes_per_step": main["kv_bytes_per_step"],
        "whole_step_gb_per_s": main["kv_bytes_per_step"] / main["ms_per_step"] / 1e6,
        "whole_step_frac": main["kv_bytes_per_step"] / main["ms_per_step"] / 1e6 / peak,
        "attend_launches_per_step": n_launch / max(1, prof.steps),
        "attend_ms_per_step": prof.attend_kernel_ms / max(1, prof.steps),
        "algorithmic_bytes_per_launch": prof.kv_bytes_read / n_launch,
        "avg_launch_ms": prof.attend_kernel_ms / n_launch,
        "kernel_gb_per_s": kernel_gbs, "frac": kernel_gbs / peak, "frac_of_nominal_8TBs": kernel_gbs / 8000.0,
        "kernel": kernel, "gpu_launches": gpu_launches, "launches_per_step": main["launches_per_step"],
        "one_launch": {"harness_only": True, "ms_per_step": one["ms_per_step"],
                       "tokens_per_s": tokens / (one["ms_per_step"] / 1e3), "attend_ms": one_attend_ms,
                       "kernel_gb_per_s": one_gbs, "frac": one_gbs / peak, "context": [one["context_first"], one["context_last"]],
                       "note": "all layers in one attention launch: needs every layer's q/k/v before the step starts"},
        "e2e": {"value": tokens / (host["ms_per_step"] / 1e3), "unit": UNIT, "h2d_bytes_per_step": host["h2d"],
                "d2h_bytes_per_step": host["d2h"], "steps": Ke, "ms_per_step": host["ms_per_step"],
                "context": [host["context_first"], host["context_last"]]},
        "kv_saved": {"token_exact": 1 - st.kv_bytes_stored / st.kv_bytes_all_full,
                     "paged": 1 - st.kv_bytes_stored_paged / st.kv_bytes_all_full_paged,
                     "bytes_stored": st.kv_bytes_stored, "bytes_all_full": st.kv_bytes_all_full,
                     "qcache_bytes": st.qcache_bytes},
        "clocks": clocks.summary(),
    }
    res["e2e"]["over_value"] = res["e2e"]["value"] / res["tokens_per_s"]
    res.update(extra)
    if extra_arms and world == 1 and not args.no_all_full:
        # the same steps on a cache whose layers are all ordinary (Eq. 2 only), same schedule
        f = _Arms(args, w, mode, group, local_rank, rank * w.batch, all_full=True)
        f.set(IN_ORDER)
        f.run(W_, timed=False)
        full = f.run(K)
        stf = f.close()
        res["vs_all_full"] = {"ms_per_step": full["ms_per_step"], "tokens_per_s": tokens / (full["ms_per_step"] / 1e3),
                              "kv_bytes_stored": stf.kv_bytes_stored, "speedup_of_lazy": full["ms_per_step"] / main["ms_per_step"],
                              "context": [full["context_first"], full["context_last"]],
                              "note": "same inputs, steps and schedule, every layer ordinary (Eq. 2 only)"}
    return res


def measure_tiny(args, mode, group, local_rank):
    """The small contiguous workload: launch-latency-bound (1.4 MB per layer), reported in us per step."""
    from paper_2602_01901_b200 import workloads as W

    w = W.get_workload("tiny")
    a = _Arms(args, w, mode, group, local_rank, 0)
    a.set(IN_ORDER)
    a.run(3, timed=False)
    io = a.run(5)
    a.set(ONE_LAUNCH)
    a.run(3, timed=False)
    one = a.run(5)
    a.close()
    return {"workload": "tiny", "us_per_step": io["ms_per_step"] * 1e3, "us_per_step_one_launch": one["ms_per_step"] * 1e3,
            "note": "L2-resident, launch-latency-bound: no HBM fraction is meaningful"}


HEADLINE = "llava_next_anyres"                       # the largest configuration by bytes per step
OTHERS = ("llava15_7b", "qwen2vl_gqa", "long_video_pruned")


def run_gpu(args, rank, world, local_rank):
    from paper_2602_01901_b200 import workloads as W
    from paper_2602_01901_b200.ranks import RankGroup

    group = RankGroup(backend=args.dist_backend)   # NCCL when launched with WORLD_SIZE > 1
    mode = MODES[args.mode]
    W_, K, Ke = args.warmup, args.steps, min(args.steps, args.e2e_steps)
    single = args.workload is not None
    head_w = _shape(args, W.get_workload(args.workload or HEADLINE))
    head = measure_workload(args, head_w, mode, group, local_rank, world, rank, K, W_, Ke,
                            extra_arms=single and not args.no_per_block)
    per_config, tiny = [], None
    if not single and world == 1:
        for name in OTHERS:
            w = W.get_workload(name)
            k = min(K, 48)
            per_config.append(measure_workload(args, w, mode, group, local_rank, world, rank, k, W_, min(Ke, 16),
                                               extra_arms=(name == "llava15_7b" and not args.no_per_block)))
        tiny = measure_tiny(args, mode, group, local_rank)
    group.close()
    if rank != 0:
        return None
    peak, peak_kind = _peaks()
    traffic = NCU_TRAFFIC_RATIO[head["kernel"]] * head["algorithmic_bytes_per_launch"]
    line = {
        "metric": METRIC, "value": head["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W_,
        "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": head_w.name, "mode": args.mode, "schedule": head["schedule"], "batch_per_gpu": head_w.batch,
            "n_layers": head_w.n_layers, "lazy_layers": len(head_w.lazy_layers), "q_heads": head_w.n_q_heads,
            "kv_heads": head_w.n_kv_heads, "head_dim": head_w.head_dim, "context_first_timed_step": head["context"][0],
            "context_last_timed_step": head["context"][1], "page_tokens": head_w.page_size,
            "l2": "inputs larger than L2: every step streams the whole KV cache",
            "arithmetic": "bf16 storage, fp32 accumulate",
        },
        "roofline": {
            "bound": "hbm", "achieved": head["kernel_gb_per_s"], "peak": peak, "unit": "GB/s", "frac": head["frac"],
            "traffic": traffic, "traffic_source": "ncu dram bytes of launches of the same kernel and schedule on the first 8 "
                                                  "layers of llava15_7b / qwen2vl_gqa, scaled by the K/V bytes of a launch",
            "peak_kind": f"of {peak_kind}", "kernel": head["kernel"],
            "algorithmic_bytes_per_launch": head["algorithmic_bytes_per_launch"], "avg_launch_ms": head["avg_launch_ms"],
            "launches_per_step": head["attend_launches_per_step"], "frac_of_nominal_8TBs": head["frac_of_nominal_8TBs"],
            "whole_step_frac": head["whole_step_frac"],
            "note": "achieved = K/V bytes of the attention launches / their summed durations (events around every "
                    "launch, second pass); whole_step_frac = the same bytes / the profiling-off step time",
        },
        "e2e": head["e2e"], "gpu_launches": head["gpu_launches"], "clocks": head["clocks"],
        "kv_cache": head["kv_saved"], "one_launch": head["one_launch"],
        "per_config": per_config, "tiny": tiny,
        "paper_context": "paper reports ~35% KV saved and 1.5x-1.6x decode throughput for LLaVA-NeXT-7B on one 80GB A100 (whole model)",
    }
    for key in ("vs_all_full", "per_block_launches", "per_layer_logit_cache", "layer_calls"):
        if key in head:
            line[key] = head[key]
    return line


def _shape(args, w):
    if not (args.layers or args.batch):
        return w
    # a smaller case of the same shape, e.g. for a profiler capture that must stay a few GB
    import dataclasses

    n_layers = args.layers or w.n_layers
    batch = args.batch or w.batch
    return dataclasses.replace(w, name=f"{w.name}[layers={n_layers},batch={batch}]", n_layers=n_layers, batch=batch,
                               lazy_layers=tuple(l for l in w.lazy_layers if l < n_layers))


def run_prefill(args, w, mode, local_rank):
    """Secondary measurement: prefill Lazy Attention (qc_prefill_attend) over the workload's prompts.
    One JSON line: prompt tokens/s through the call, and the attention kernel against the tensor peak."""
    import torch

    from paper_2602_01901_b200 import workloads as W
    from paper_2602_01901_b200.session import Session

    dev = torch.device("cuda", local_rank)
    s = Session.for_workload(w, lazy_mode=mode, device=local_rank)
    s.set_option("prefill_tcgen05", 1 if args.prefill_kernel == "tcgen05" else 0)
    s.set_option("prefill_shared_scores", 0 if args.no_prefill_sharing else 1)
    for kv in args.option:
        key, _, val = kv.partition("=")
        s.set_option(key, int(val))
    n_seqs = min(w.batch, max(4, args.warmup + 1))
    prompts = []
    for b in range(n_seqs):
        kind, k, v = W.prefill_kv_torch(w, b, dev)
        prompts.append((kind, W.prefill_q_torch(w, b, dev), k, v))
    out = torch.empty_like(prompts[0][1])
    from paper_2602_01901_b200 import binding as qc

    n_chunks = max(1, args.prefill_chunks)
    T = len(prompts[0][0])
    cuts = [T * i // n_chunks for i in range(n_chunks + 1)]

    chunks = None
    if n_chunks > 1:   # a chunk's tensors must be dense: materialise them before the timed region
        chunks = []
        for kind, q, k, v in prompts:
            chunks.append([(kind[a:e], q[:, a:e].contiguous(), k[:, a:e].contiguous(), v[:, a:e].contiguous(),
                            torch.empty_like(q[:, a:e].contiguous())) for a, e in zip(cuts[:-1], cuts[1:])])

    def prefill(b):   # the prompt in one call, or as consecutive chunks (later ones see the cached tokens)
        if n_chunks == 1:
            s.prefill_attend(b, *prompts[b], out)
            return
        for kind_c, q_c, k_c, v_c, out_c in chunks[b]:
            s.prefill_attend(b, kind_c, q_c, k_c, v_c, out_c)

    prefill(0)          # warm-up on sequence 0, then release it
    qc.qc_free_seq(s.cache, 0)
    s.set_option("profile", 1)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(_physical_gpu_index(local_rank)) as clocks:
        e0.record()
        for b in range(n_seqs):
            prefill(b)
        e1.record()
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    prof = s.profile()
    st = s.stats()
    s.close()
    peak_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak, peak_kind = 1590.0, "of fallback"
    if os.path.exists(peak_path):
        with open(peak_path) as f:
            peak, peak_kind = float(json.load(f)["bf16_tflops"]), "of measured"
    achieved = prof.prefill_flops / (prof.prefill_attend_ms / 1e3) / 1e12
    return {
        "metric": "prefill_attention_tokens_per_s", "value": n_seqs * T / (ms / 1e3), "unit": UNIT, "n_gpus": 1,
        "steps": n_seqs, "warmup": 1, "ms_per_step": ms / n_seqs, "higher_is_better": True, "dtype": "bf16",
        "data": "synthetic", "config": {"workload": w.name, "mode": args.mode, "prompt_tokens": T, "prompt_chunks": n_chunks,
                                        "shared_score_passes": (args.mode == "gla" and not args.no_prefill_sharing),
                                        "n_layers": w.n_layers, "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads},
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved / peak, "traffic": None,
                     "kernel": "prefill_attend_tcgen05_kernel" if (args.prefill_kernel == "tcgen05" and w.head_dim == 128)
                     else "prefill_attend_kernel",
                     "avg_launch_ms": prof.prefill_attend_ms / max(1, prof.prefill_calls),
                     "flops_per_launch": prof.prefill_flops / max(1, prof.prefill_calls), "peak_kind": peak_kind},
        "clocks": clocks.summary(), "device_error": st.device_error,
    }


def _self_launch(argv, n):
    """`python bench.py --gpus N` without a launcher: start N ranks of this script on this node."""
    import socket
    import subprocess

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + argv
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=48)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None,
                    help="one workload only (default: the headline on the largest configuration plus a record per "
                         "other model-shaped configuration and the tiny one)")
    ap.add_argument("--mode", default="vla_qc", choices=sorted(MODES))
    ap.add_argument("--e2e-steps", type=int, default=32)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-prefill", action="store_true", help="skip the prefill records of the default run")
    ap.add_argument("--no-all-full", action="store_true", help="skip the all-ordinary-layers comparison run")
    ap.add_argument("--no-per-block", action="store_true",
                    help="skip the comparison arms (one launch per lazy block, per layer with the logit cache, "
                         "all layers ordinary)")
    ap.add_argument("--option", action="append", default=[], help="key=value passed to qc_set_option (headline arm)")
    ap.add_argument("--dist-backend", default=None, help="torch.distributed backend (default: nccl on GPUs)")
    ap.add_argument("--force-device", type=int, default=-1,
                    help="use this CUDA device on every rank (to exercise the multi-rank plumbing on one GPU)")
    ap.add_argument("--phase", default="decode", choices=["decode", "prefill"],
                    help="decode (the benchmark) or prefill (secondary: qc_prefill_attend over the prompts)")
    ap.add_argument("--no-prefill-sharing", action="store_true",
                    help="prefill phase, mode gla: one score pass per layer instead of one per run of up to three "
                         "layers of a lazy block")
    ap.add_argument("--prefill-chunks", type=int, default=1,
                    help="prefill phase: give each prompt as this many consecutive calls (chunked prefill)")
    ap.add_argument("--prefill-kernel", default="tcgen05", choices=["tcgen05", "mma"],
                    help="prefill phase, head_dim 128: tcgen05 kernel (default) or the mma.sync kernel")
    ap.add_argument("--split-tokens", type=int, default=0, help="keys per split-KV work item (0 = library default)")
    ap.add_argument("--layers", type=int, default=0, help="cut the stack to its first N layers (profiling-size case)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch (profiling-size case)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(_self_launch(sys.argv[1:], args.gpus))

    from paper_2602_01901_b200 import workloads as W

    mode = MODES[args.mode]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.force_device >= 0:     # several ranks on one GPU: a plumbing check, not a measurement
        local_rank = args.force_device

    if args.impl == "reference":
        # the oracle on the host cores; under a multi-rank launch rank 0 alone works, the others only
        # answer the roll call that fills n_gpus
        from paper_2602_01901_b200.ranks import RankGroup

        group = RankGroup(backend=args.dist_backend or "gloo")
        ranks = int(group.sum_over_ranks(1.0))
        group.close()
        if rank != 0:
            return
        w = _shape(args, W.get_workload(args.workload or HEADLINE))
        t0 = time.perf_counter()
        base = cpu_oracle_sample(w, mode, args.warmup)
        line = {
            "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": ranks,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.batch / base["value"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "mode": args.mode, "schedule": "oracle (one layer, sequence and head at a time)",
                       "batch_per_gpu": w.batch, "n_layers": w.n_layers, "lazy_layers": len(w.lazy_layers),
                       "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
                       "page_tokens": w.page_size, "arithmetic": "fp64"},
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "wall_s": time.perf_counter() - t0,
        }
        print(json.dumps(line))
        return

    if args.phase == "prefill":
        if rank == 0:
            w = _shape(args, W.get_workload(args.workload or "llava15_7b"))
            print(json.dumps(run_prefill(args, w, mode, local_rank)))
        return
    line = run_gpu(args, rank, world, local_rank)
    if rank == 0:
        if world == 1 and args.workload is None and not args.no_prefill:
            # secondary: prefill Lazy Attention (qc_prefill_attend) over the prompts of configs 2 and 3
            line["prefill"] = []
            for name in ("llava15_7b", HEADLINE):
                r = run_prefill(args, W.get_workload(name), mode, local_rank)
                line["prefill"].append({"workload": name, "prompt_tokens": r["config"]["prompt_tokens"],
                                        "prompt_tokens_per_s": r["value"], "ms_per_prompt": r["ms_per_step"],
                                        "kernel": r["roofline"]["kernel"], "tflops": r["roofline"]["achieved"],
                                        "frac_of_measured_bf16_peak": r["roofline"]["frac"],
                                        "avg_launch_ms": r["roofline"]["avg_launch_ms"]})
        if world == 1 and not args.no_cpu_baseline:
            w = _shape(args, W.get_workload(args.workload or HEADLINE))
            line["cpu_baseline"] = cpu_oracle_sample(w, mode, args.warmup)
        print(json.dumps(line))


if __name__ == "__main__":
    main()
