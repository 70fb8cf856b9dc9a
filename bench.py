"""Benchmark of the Lazy Attention decode step (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--mode vla_qc|vla_eq8|gla]
    python bench.py --impl reference ...      # times the CPU oracle on the same workload

A step is one qc_decode_step over the whole batch (append + Q Cache write + split-KV partial
attention + log-sum-exp merge, all layers).  `value` is decode tokens/s with inputs resident
in HBM; `e2e` is the same through qc_decode_step_host with pinned HOST buffers (q, k, v copied
in, out copied back, inside the timed region).  With N > 1 (torchrun) every rank runs its own
batch of the same shape on its own GPU (independent sequences: no collective on the data
path); the time is the maximum over ranks.
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

# (dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic K/V bytes of one attention launch,
# from the ncu captures of small cases summarised in profiles/attend_kernels_small_cases_ncu_full.md.
# Traffic grows in proportion to the K/V bytes swept (every tile is fetched once; partial results are
# written once per chunk), so a full launch's traffic is this ratio times its algorithmic bytes.
NCU_TRAFFIC_RATIO = {"attend_kernel": 1.069, "attend_tc_kernel": 1.070}


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
# CPU oracle leg (bounded sample)
# ------------------------------------------------------------------------------------------

def cpu_oracle_sample(w, mode: int, first_step: int, budget_s: float = 12.0):
    """Time the fp64 oracle, as it stands, on a bounded sample of the workload.

    Sample: whole-stack sub-problems (all layers, one sequence, one KV head with its query
    heads), each advanced through decode steps starting at `first_step` context length, until
    the time budget is used.  One generated token of the full workload costs n_kv_heads such
    sub-problem steps, so tokens/s = sub-problem steps per second / n_kv_heads.
    """
    from threadpoolctl import threadpool_limits

    from oracle.lazy_attention import LazyAttentionOracle
    from paper_2602_01901_b200 import workloads as W

    f64 = W.bf16_bits_to_f64
    g = w.group
    done, spent, units = 0, 0.0, 0
    with threadpool_limits(limits=1):
        unit = 0
        while spent < budget_s and unit < w.batch * w.n_kv_heads:
            seq, kvh = unit % w.batch, (unit // w.batch) % w.n_kv_heads
            heads = list(range(kvh * g, (kvh + 1) * g))
            o = LazyAttentionOracle(w.n_layers, g, 1, w.head_dim, w.layer_kind().tolist(), mode, n_seqs=1)
            kind, k, v = W.prefill_kv_np(w, seq, heads=[kvh])
            o.prefill_append(0, kind.tolist(), f64(k), f64(v))
            # untimed catch-up to the benchmark's first timed step (appends only matter)
            for step in range(first_step):
                q, kk, vv = W.decode_qkv_np(w, step, seqs=[seq], q_heads=heads, kv_heads=[kvh])
                for l in range(w.n_layers):
                    o.V_T[l][0].append(f64(vv[l, 0]))
                    if o.K_T[l][0] is not None:
                        o.K_T[l][0].append(f64(kk[l, 0]))
            for step in range(first_step, first_step + 16):
                q, kk, vv = W.decode_qkv_np(w, step, seqs=[seq], q_heads=heads, kv_heads=[kvh])
                qf, kf, vf = f64(q[:, 0]), f64(kk[:, 0]), f64(vv[:, 0])
                t0 = time.perf_counter()
                o.decode_step(0, qf, kf, vf)
                spent += time.perf_counter() - t0
                done += 1
            unit += 1
            units += 1
    tokens_per_s = done / spent / w.n_kv_heads
    return {
        "value": tokens_per_s, "unit": UNIT, "cores": 1, "kind": "oracle",
        "sample": f"{units} (sequence, KV head) sub-problems x all {w.n_layers} layers x 16 decode steps from "
                  f"context {w.n_prompt + first_step}; {done} sub-problem steps in {spent:.1f} s, "
                  f"scaled by 1/{w.n_kv_heads} KV heads per token",
    }


# ------------------------------------------------------------------------------------------
# GPU arms
# ------------------------------------------------------------------------------------------

def _gen_inputs(w, first, count, device, seq_offset=0):
    from paper_2602_01901_b200 import workloads as W

    return [W.decode_qkv_torch(w, s, device, seq_offset) for s in range(first, first + count)]


def run_gpu(args, w, mode, rank, world, local_rank):
    import torch

    from paper_2602_01901_b200 import binding as qc
    from paper_2602_01901_b200.session import Session

    from paper_2602_01901_b200.ranks import RankGroup

    group = RankGroup(backend=args.dist_backend)   # NCCL when launched by torchrun with WORLD_SIZE > 1
    seq_offset = rank * w.batch  # every rank serves its own sequences of the global batch

    def barrier():
        group.barrier()
        torch.cuda.synchronize()

    max_over_ranks = group.max_over_ranks

    W_, K = args.warmup, args.steps
    total_steps = W_ + K
    if total_steps > w.decode_steps:
        raise SystemExit(f"warmup + steps = {total_steps} exceeds the workload's {w.decode_steps} decode steps")
    ids = qc._i32_array(list(range(w.batch)))
    dev = torch.device("cuda", local_rank)
    shape_o = (w.n_layers, w.batch, w.n_q_heads, w.head_dim)

    # ---- arm 1: inputs resident in HBM ---------------------------------------------------
    s = Session.for_workload(w, lazy_mode=mode, device=local_rank, split_tokens=args.split_tokens)
    s.prefill_workload(w, seq_offset)
    if args.blocks_per_launch:
        s.set_option("layers_per_launch", args.blocks_per_launch)
    if args.per_layer:
        s.set_option("per_layer_logit_cache", 1)
    if args.in_order:
        s.set_option("in_order_launches", 1)
    for kv in args.option:
        key, value = kv.split("=")
        s.set_option(key, int(value))
    inputs = _gen_inputs(w, 0, total_steps, dev, seq_offset)
    out = torch.empty(shape_o, dtype=torch.bfloat16, device=dev)
    for i in range(W_):
        s.decode_step(ids, *inputs[i], out)
    s.set_option("profile", 1)
    launches_before = s.stats().kernel_launches
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(_physical_gpu_index(local_rank)) as clocks:
        e0.record()
        for i in range(W_, total_steps):
            s.decode_step(ids, *inputs[i], out)
        e1.record()
        barrier()
    ms = max_over_ranks(e0.elapsed_time(e1))
    prof = s.profile()
    s.set_option("profile", 0)
    st = s.stats()
    if st.device_error:
        raise SystemExit(f"device error word = {st.device_error}")
    checksum = float(out.float().abs().sum().item())
    if not np.isfinite(checksum) or checksum == 0.0:
        raise SystemExit("output is not finite / all zero")
    s.close()
    del s

    # ---- arm 1b (one GPU only): the same steps on a cache whose layers are all ordinary -------
    all_full = None
    if world == 1 and not args.no_all_full:
        s = Session.for_workload(w, lazy_mode=mode, device=local_rank, split_tokens=args.split_tokens, all_full=True)
        s.prefill_workload(w, seq_offset)
        for i in range(W_):
            s.decode_step(ids, *inputs[i], out)
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for i in range(W_, total_steps):
            s.decode_step(ids, *inputs[i], out)
        f1.record()
        torch.cuda.synchronize()
        ms_full = f0.elapsed_time(f1)
        st_full = s.stats()
        s.close()
        del s
        all_full = {"ms_per_step": ms_full / K, "tokens_per_s": w.batch * K / (ms_full / 1e3),
                    "kv_bytes_stored": st_full.kv_bytes_stored, "speedup_of_lazy": ms_full / ms,
                    "note": "same inputs and steps, every layer ordinary (Eq. 2 only)"}
    # ---- arms 1c, 1d (one GPU only): the same steps under the two schedules that issue layers in order.
    # per_block: one attention + merge launch per lazy block (needs a block's q/k/v at once).
    # per_layer: one launch pair per layer, followers reading the leader's scores from the logit
    # cache: the schedule of a model in which a layer's q/k/v only exist after the previous layer.
    def ordered_arm(option, value, note):
        s2 = Session.for_workload(w, lazy_mode=mode, device=local_rank, split_tokens=args.split_tokens)
        s2.prefill_workload(w, seq_offset)
        s2.set_option(option, value)
        for i in range(W_):
            s2.decode_step(ids, *inputs[i], out)
        s2.set_option("profile", 1)
        torch.cuda.synchronize()
        launches0 = s2.stats().kernel_launches
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for i in range(W_, total_steps):
            s2.decode_step(ids, *inputs[i], out)
        f1.record()
        torch.cuda.synchronize()
        ms2 = f0.elapsed_time(f1)
        prof2 = s2.profile()
        res = {"ms_per_step": ms2 / K, "tokens_per_s": w.batch * K / (ms2 / 1e3),
               "gpu_launches": int(s2.stats().kernel_launches - launches0),
               "kv_gb_per_s_whole_step": prof2.kv_bytes_read / (ms2 / 1e3) / 1e9,
               "kv_bytes_read_per_step": prof2.kv_bytes_read / max(1, prof2.steps), "note": note}
        s2.close()
        return res

    per_block = per_layer = in_order = None
    if world == 1 and not args.no_per_block and not args.blocks_per_launch and not args.per_layer and not args.in_order:
        in_order = ordered_arm("in_order_launches", 1,
                               "one attention + merge launch per layer, layers in order; a leader's launch also "
                               "sweeps its followers' cached V rows")
        per_block = ordered_arm("layers_per_launch", 1,
                                "one attention + merge launch per lazy block, blocks in layer order")
        per_layer = ordered_arm("per_layer_logit_cache", 1,
                                "one attention + merge launch per layer, layers in order; followers take the "
                                "leader's scores from the logit cache instead of reading its K")
    del inputs
    torch.cuda.empty_cache()

    # ---- arm 2: host buffers through qc_decode_step_host -----------------------------------
    Ke = min(K, args.e2e_steps)
    s = Session.for_workload(w, lazy_mode=mode, device=local_rank, split_tokens=args.split_tokens)
    s.prefill_workload(w, seq_offset)
    dev_in = _gen_inputs(w, 0, W_ + Ke, dev, seq_offset)
    for i in range(W_):
        s.decode_step(ids, *dev_in[i], out)
    host_in = [tuple(t.cpu().pin_memory() for t in dev_in[i]) for i in range(W_, W_ + Ke)]
    host_out = torch.empty(shape_o, dtype=torch.bfloat16).pin_memory()
    del dev_in
    barrier()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for i in range(Ke):
        s.decode_step_host(ids, *host_in[i], host_out)     # returns after the copy back has finished
    g1.record()
    barrier()
    e2e_s = max_over_ranks(g0.elapsed_time(g1)) / 1e3
    h2d = sum(t.numel() * 2 for t in host_in[0])
    d2h = host_out.numel() * 2
    s.close()

    group.close()
    if rank != 0:
        return None
    peak, peak_kind = _peaks()
    tokens = w.batch * K * world
    attend_s = prof.attend_ms / 1e3
    achieved = prof.kv_bytes_read / attend_s / 1e9
    launches_attend = K
    kernel = "attend_tc_kernel" if w.group > 1 else "attend_kernel"
    traffic = NCU_TRAFFIC_RATIO[kernel] * prof.kv_bytes_read / launches_attend
    line = {
        "metric": METRIC, "value": tokens / (ms / 1e3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W_,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": w.name, "mode": args.mode, "batch_per_gpu": w.batch, "n_layers": w.n_layers,
            "lazy_layers": len(w.lazy_layers), "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads,
            "head_dim": w.head_dim, "context_first_timed_step": w.n_prompt + W_ + 1,
            "context_last_timed_step": w.n_prompt + total_steps, "page_tokens": w.page_size,
            "l2": "inputs larger than L2: every step streams the whole KV cache", "arithmetic": "bf16 storage, fp32 accumulate",
        },
        "roofline": {
            "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": traffic, "traffic_source": "ncu dram bytes of a small case, scaled by K/V bytes per launch",
            "peak_kind": f"of {peak_kind}", "kernel": kernel,
            "algorithmic_bytes_per_launch": prof.kv_bytes_read / launches_attend,
            "avg_launch_ms": prof.attend_ms / launches_attend, "frac_of_nominal_8TBs": achieved / 8000.0,
        },
        "e2e": {"value": w.batch * Ke * world / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": Ke},
        "gpu_launches": int(st.kernel_launches - launches_before),
        "clocks": clocks.summary(),
        "kv_cache": {
            "bytes_stored": st.kv_bytes_stored, "bytes_all_full": st.kv_bytes_all_full,
            "saved_frac_token_exact": 1 - st.kv_bytes_stored / st.kv_bytes_all_full,
            "saved_frac_paged": 1 - st.kv_bytes_stored_paged / st.kv_bytes_all_full_paged,
            "qcache_bytes": st.qcache_bytes,
        },
        "vs_all_full": all_full,
        "per_block_launches": per_block,
        "per_layer_launches": per_layer,
        "in_order_launches": in_order,
        "step_ms_by_events": prof.step_ms / max(1, prof.steps),
        "paper_context": "paper reports ~35% KV saved and 1.5x-1.6x decode throughput for LLaVA-NeXT-7B on one 80GB A100 (whole model)",
    }
    return line


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
    with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
        peak = float(json.load(f)["bf16_tflops"])
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
                     "flops_per_launch": prof.prefill_flops / max(1, prof.prefill_calls), "peak_kind": "of measured"},
        "clocks": clocks.summary(), "device_error": st.device_error,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=240)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llava15_7b")
    ap.add_argument("--mode", default="vla_qc", choices=sorted(MODES))
    ap.add_argument("--e2e-steps", type=int, default=64)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-all-full", action="store_true", help="skip the all-ordinary-layers comparison run")
    ap.add_argument("--no-per-block", action="store_true",
                    help="skip the comparison runs with one launch per lazy block / per layer")
    ap.add_argument("--per-layer", action="store_true",
                    help="run the main arm under the per-layer schedule with the logit cache (for profiling it)")
    ap.add_argument("--in-order", action="store_true",
                    help="run the main arm under the in-order schedule (for profiling it)")
    ap.add_argument("--option", action="append", default=[], help="key=value passed to qc_set_option (main arm)")
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
    ap.add_argument("--blocks-per-launch", type=int, default=0,
                    help="0 = one attention launch per step; k = one launch per k lazy blocks, in layer order")
    ap.add_argument("--layers", type=int, default=0, help="cut the stack to its first N layers (profiling-size case)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch (profiling-size case)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    from paper_2602_01901_b200 import workloads as W

    w = W.get_workload(args.workload)
    if args.layers or args.batch:
        # a smaller case of the same shape, e.g. for a profiler capture that must stay a few GB
        import dataclasses

        n_layers = args.layers or w.n_layers
        batch = args.batch or w.batch
        w = dataclasses.replace(w, name=f"{w.name}[layers={n_layers},batch={batch}]", n_layers=n_layers, batch=batch,
                                lazy_layers=tuple(l for l in w.lazy_layers if l < n_layers))
    mode = MODES[args.mode]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.force_device >= 0:     # several ranks on one GPU: a plumbing check, not a measurement
        local_rank = args.force_device

    if args.impl == "reference":
        if rank != 0:
            return
        t0 = time.perf_counter()
        base = cpu_oracle_sample(w, mode, args.warmup, budget_s=20.0)
        line = {
            "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.batch / base["value"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "mode": args.mode, "batch_per_gpu": w.batch},
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "wall_s": time.perf_counter() - t0,
        }
        print(json.dumps(line))
        return

    if args.phase == "prefill":
        if rank == 0:
            print(json.dumps(run_prefill(args, w, mode, local_rank)))
        return
    line = run_gpu(args, w, mode, rank, world, local_rank)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_oracle_sample(w, mode, args.warmup)
        print(json.dumps(line))


if __name__ == "__main__":
    main()
