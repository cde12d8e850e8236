#!/usr/bin/env python
"""Benchmark of the adapter-aware MoE layer forward (ExpertWeave hot path) on B200.

A step is one pass of the whole hot path (router + top-k + batched rerouting + histogram, permute,
grouped SwiGLU GEMM-1, GEMM-2, combine) over one decode batch of the DeepSeek-V2-Lite-shaped layer
(workload c1: 256 tokens, 64 routed + 2 shared experts, top-6, 4 adapters x 8 re-tuned experts).

  python bench.py [--gpus N] [--steps K] [--warmup W]      the CUDA path (prints one JSON line)
  python bench.py --impl reference ...                     the CPU oracle as it stands, same metric

The line's `value` is workload c1.  Its `extra` object carries the other parts of the metric, each with the
clocks seen while it ran: the prefill layer (c2: tokens/s and the tensor-core fraction of the two GEMMs), a slice
of the stacked decode configuration (c3: ms per layer, weight stream), the rerouting operator alone (c4: GB/s at
65,536 and 4 M tokens, fused with the gate, and as separate kernels) and the padding-mode pool against the
on-demand one.  `--no-extras` leaves them out.

With N > 1 every rank runs its own replica of the batch on its own GPU (the path has no exchange step); the timed
region is bracketed by barriers and the slowest rank's time is used.  Launched plainly with --gpus N the script
spawns the N ranks itself; under torchrun it takes its rank from the environment.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel (GEMM-1 + SwiGLU at
# workload c1) from an ncu capture of this build; reported beside the algorithmic bytes, not used in any ratio.
NCU_TRAFFIC_BYTES = {"c1": 1.1451e9}
# route_logits4_kernel at the c4 shape: issue-slot lanes per token from one ncu capture (smsp__inst_executed x 32 /
# tokens; 3,208 of them carry an active thread), and the issue peak of the GPU
ALU_INSTR_PER_TOKEN_C4 = 127 * 32
ALU_PEAK_TINSTR = 148 * 4 * 32 * 1.965e9 / 1e12

METRIC = "adapter-aware MoE layer tokens/s"
UNIT = "tokens/s"
WORKLOADS = {
    "c1": "c1: DeepSeek-V2-Lite-shaped MoE layer, decode batch 256, 4 adapters x 8 experts",
    "c2": "c2: DeepSeek-V2-Lite-shaped MoE layer, prefill 8192 tokens (32 requests x 256), 20 adapters x 4-16 experts",
}
WORKLOAD = WORKLOADS["c1"]
MIN_TIMED_S = 0.5          # the K-step region is repeated until this much has been timed; the median region is reported


def load_peaks():
    """-> (HBM GB/s, bf16 TFLOP/s burst, bf16 TFLOP/s sustained under the power cap, kind)"""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return (float(d["hbm_gbs"]), float(d["bf16_tflops"]),
                float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "measured")
    return 6650.0, 1590.0, 1400.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while `active` is set."""

    def __init__(self, index: int, period: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.active = False
        self.err = None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = int(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
            names = {
                getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
                getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
            }
            get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
            while not self._stop_evt.is_set():
                if self.active:
                    self.samples.append(int(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                    mask = int(get_reasons(h))
                    for bit, name in names.items():
                        if mask & bit:
                            self.reasons.add(name)
                time.sleep(self.period)
        except Exception as e:  # clocks are evidence, not part of the computation
            self.err = repr(e)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)

    def window(self):
        """Context manager: samples are taken only inside it (the timed regions, not the set-up around them)."""
        import contextlib

        @contextlib.contextmanager
        def cm():
            self.active = True
            try:
                yield
            finally:
                self.active = False
        return cm()

    def take(self):
        """Summary of the samples since the last call (the sampler keeps running)."""
        s, r = self.samples, self.reasons
        self.samples, self.reasons = [], set()
        out = {"sm_mhz": float(np.median(s)) if s else None, "sm_max_mhz": self.max_mhz,
               "reasons": sorted(r), "samples": len(s)}
        if self.err:
            out["error"] = self.err
        return out


def reduce_max_over_ranks(values, device="cpu"):
    """Element-wise MAX of per-rank measurements over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_tokens_per_s(world: int, tokens_per_step_per_rank: int, steps: int, ms_slowest_rank: float) -> float:
    """Replicas only: every rank pushes its own batch, the job's time is the slowest rank's."""
    return world * tokens_per_step_per_rank * steps / (ms_slowest_rank * 1e-3)


def physical_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except (ValueError, IndexError):
            pass
    return local_rank


def timed_regions(step, steps, barrier, min_total_s=MIN_TIMED_S, max_regions=400, reduce=None):
    """Time `steps` calls of step() between CUDA events, bracketed by barrier(), again and again until at least
    `min_total_s` has been timed (at least three regions).  Returns the per-region milliseconds (max over ranks when
    `reduce` is given, so that every rank takes the same number of regions)."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    regions, total = [], 0.0
    while (total < min_total_s * 1e3 or len(regions) < 3) and len(regions) < max_regions:
        barrier()
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        barrier()
        ms = e0.elapsed_time(e1)
        if reduce is not None:
            ms = reduce([ms])[0]
        regions.append(ms)
        total += ms
    return regions


def layer_bytes_and_flops(cfg, live):
    B, H, k = cfg.n_tokens, cfg.hidden, cfg.top_k
    groups = live + cfg.num_shared
    pairs = B * k
    rows_act = cfg.num_shared * B + pairs
    blk = cfg.inter * cfg.hidden * 2
    return {
        "bytes_gemm1": groups * 2 * blk + (pairs + B) * H * 2 + rows_act * cfg.inter * 2,     # weights + rows in + act out
        # weights + act rows in + Y rows out (the shared experts are chained along K: one Y row per token for all of them)
        "bytes_gemm2": groups * blk + rows_act * cfg.inter * 2 + (pairs + (B if cfg.num_shared else 0)) * H * 4,
        "bytes_layer": groups * 3 * blk,
        "flops_gemm1": 2.0 * rows_act * 2 * cfg.inter * H,
        "flops_gemm2": 2.0 * rows_act * cfg.inter * H,
    }


def setup_layer(cfg, device, **pool_kw):
    import torch
    from paper_2508_17624_b200 import binding, workloads as wl
    pool = binding.Pool.from_config(cfg, device=device, **pool_kw)
    binding.load_model(pool, cfg)
    x_bits, aid_np = wl.gen_tokens(cfg), wl.gen_adapter_ids(cfg)
    x = torch.from_numpy(x_bits.view(np.int16)).cuda().view(torch.bfloat16)
    aid = torch.from_numpy(aid_np).cuda()
    return pool, x, aid, x_bits, aid_np


def kernel_pass(pool, step, n, barrier):
    """`n` forwards with the library's per-kernel CUDA events on the same stream (the events sit between the kernels,
    so this pass runs without launch overlap).  -> (ms per kernel per forward, ms per forward of this pass)"""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pool.profile_enable(True)
    pool.profile_read()
    barrier()
    e0.record()
    for _ in range(n):
        step()
    e1.record()
    barrier()
    kern_ms, n_prof = pool.profile_read()
    pool.profile_enable(False)
    return {kname: v / max(n_prof, 1) for kname, v in kern_ms.items()}, e0.elapsed_time(e1) / n


def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2508_17624_b200 import build, workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    own_group = world > 1 and not dist.is_initialized()      # under torchrun; ranks spawned by this script come with a group
    if own_group:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    cfg = wl.CONFIGS[args.workload]
    workload = WORKLOADS[args.workload]
    B, H, k = cfg.n_tokens, cfg.hidden, cfg.top_k
    pool, x, aid, x_bits, aid_np = setup_layer(cfg, local)
    out = torch.empty_like(x)

    # structure of this batch (for the algorithmic bytes): live slots from one debug forward
    dbg = pool.moe_forward_debug(0, x, aid)
    torch.cuda.synchronize()
    live = int((dbg["counts"].cpu().numpy() > 0).sum())
    w = layer_bytes_and_flops(cfg, live)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def reduce(v):
        return reduce_max_over_ranks(v, device="cuda")

    def step():
        pool.moe_forward(0, x, aid, out)

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    barrier()
    sampler = ClockSampler(physical_index(local))
    sampler.start()
    if args.minimal:                                    # profiler captures: warm-up and K timed steps, nothing else
        regions = timed_regions(step, args.steps, barrier, min_total_s=0.0, max_regions=1, reduce=reduce)
        sampler.stop()
        pool.destroy()
        if own_group:
            dist.destroy_process_group()
        if rank == 0:
            print(json.dumps({"metric": METRIC, "minimal": True, "ms_per_step": regions[0] / args.steps}))
        return

    # ---- timed regions: K forwards back to back (the kernels of a forward chain by programmatic dependent launch),
    #      repeated until at least MIN_TIMED_S has been timed; the clocks are sampled while they run
    sampler.active = True
    regions = timed_regions(step, args.steps, barrier, reduce=reduce)
    sampler.active = False
    clocks = sampler.take()
    ms_total = float(np.median(regions))

    # ---- the same forwards with per-kernel events
    kern, ms_with_events = kernel_pass(pool, step, min(max(args.steps, 50), 500), barrier)

    # ---- end to end through the C ABI with host buffers (pinned): H2D + forward + D2H every step.  Pipelined
    #      throughput (the entry point overlaps step n's copies with its neighbours' kernels) and, beside it, the
    #      latency of one call from upload to result on the host.
    xh = torch.from_numpy(x_bits.view(np.int16).copy()).pin_memory()
    ah = torch.from_numpy(aid_np.copy()).pin_memory()
    oh = torch.empty((B, H), dtype=torch.int16).pin_memory()

    def step_host():
        pool.moe_forward_host(0, xh, ah, oh)

    for _ in range(3):
        step_host()
    barrier()
    regions_e2e = timed_regions(step_host, args.steps, barrier, reduce=reduce)
    ms_e2e = float(np.median(regions_e2e))
    assert torch.equal(oh.cuda().view(torch.bfloat16), out), "host-buffer path disagrees with the device path"
    lat = []
    for _ in range(30):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        step_host()
        torch.cuda.synchronize()
        lat.append((time.perf_counter() - t0) * 1e3)
    err = pool.last_device_error()
    assert err == 0, f"device error word {err}"

    result = None
    if rank == 0:
        peak, peak_tf, peak_tf_sustained, peak_kind = load_peaks()
        g1_ms = kern["gemm1"]
        achieved = w["bytes_gemm1"] / (g1_ms * 1e-3) / 1e9
        tensor_bound = w["flops_gemm1"] / (peak_tf * 1e12) > w["bytes_gemm1"] / (peak * 1e9)
        if tensor_bound:
            tf = w["flops_gemm1"] / (g1_ms * 1e-3) / 1e12
            roof = {"bound": "tensor", "kernel": "GEMM-1 + SwiGLU (grouped_gemm_kernel + fat_gemm_kernel)",
                    "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": tf / peak_tf, "of": peak_kind + " (bf16 burst)",
                    "traffic": None, "algorithmic_flops": w["flops_gemm1"], "avg_launch_ms": g1_ms, "hbm_gbs": achieved,
                    # the timed loop runs for seconds under the power cap: the sustained cuBLAS figure beside it
                    "peak_sustained": peak_tf_sustained, "frac_of_sustained": tf / peak_tf_sustained}
        else:
            roof = {"bound": "hbm", "kernel": "grouped_gemm_kernel<GLU> (GEMM-1 + SwiGLU)",
                    "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "of": peak_kind, "traffic": NCU_TRAFFIC_BYTES.get(args.workload), "algorithmic_bytes": w["bytes_gemm1"],
                    "avg_launch_ms": g1_ms}
        kernels_per_forward = pool.stats()["last_forward_kernels"]     # 4, 5 or 7: the library reports what it launched
        result = {
            "metric": METRIC, "value": whole_job_tokens_per_s(world, B, args.steps, ms_total), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": warmup, "ms_per_step": ms_total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload, "tokens_per_step_per_gpu": B, "hidden": H, "inter": cfg.inter,
                       "experts": cfg.num_experts, "shared": cfg.num_shared, "top_k": k,
                       "adapters": cfg.max_adapters, "e_max": cfg.e_max, "live_slots": live,
                       "parallelism": f"replicas x{world}",
                       "l2": "no flush: each step streams %.2f GB of live expert weights, far above the 126 MB L2"
                             % (w["bytes_layer"] / 1e9)},
            "timed_regions": {"count": len(regions), "steps_each": args.steps, "ms_total": float(np.sum(regions)),
                              "ms_per_step_min": float(np.min(regions)) / args.steps,
                              "ms_per_step_max": float(np.max(regions)) / args.steps, "reported": "median region"},
            "e2e": {"value": whole_job_tokens_per_s(world, B, args.steps, ms_e2e), "unit": UNIT,
                    "h2d_bytes_per_step": B * H * 2 + B * 4, "d2h_bytes_per_step": B * H * 2,
                    "kind": "pipelined across calls (double-buffered staging inside ew_moe_forward_host)",
                    "single_call_latency_ms": float(np.median(lat)),
                    "single_call_tokens_per_s": B / (float(np.median(lat)) * 1e-3)},
            "gpu_launches": kernels_per_forward * args.steps,
            "clocks": clocks,
            "roofline": roof,
            "kernels_ms_per_step": kern,
            "gemm2": {"achieved": w["bytes_gemm2"] / (kern["gemm2"] * 1e-3) / 1e9, "unit": "GB/s",
                      "algorithmic_bytes": w["bytes_gemm2"], "tflops": w["flops_gemm2"] / (kern["gemm2"] * 1e-3) / 1e12},
            "layer_weight_stream": {"achieved": w["bytes_layer"] / (ms_total / args.steps * 1e-3) / 1e9, "unit": "GB/s",
                                    "frac": w["bytes_layer"] / (ms_total / args.steps * 1e-3) / 1e9 / peak},
            "ms_per_step_with_kernel_events": ms_with_events,
        }
    pool.destroy()
    del pool
    if rank == 0 and world == 1 and not args.no_extras and args.workload == "c1":
        result["extra"] = run_extras(sampler, local)
    sampler.stop()
    if rank == 0 and not args.no_cpu_baseline and world == 1:
        result["cpu_baseline"] = cpu_baseline(cfg, budget_s=24.0)
    if world > 1:
        dist.barrier()
    if own_group:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(result))


# ------------------------------------------------------------------------------------------------------ extras
def run_extras(sampler, device):
    """The other parts of the metric, one record each, every one with the clocks sampled while it ran."""
    out = {}
    for name, fn in (("c2_prefill", extra_prefill), ("c3_stack_slice", extra_stack), ("c4_reroute", extra_reroute),
                     ("padding_mode", extra_padding), ("expert_parallel_emulated", extra_expert_parallel)):
        try:
            sampler.take()
            rec = fn(device, sampler)
            rec["clocks"] = sampler.take()
            out[name] = rec
        except Exception as e:                           # an extra never takes the headline down with it
            out[name] = {"error": repr(e)}
    return out


def _sync_barrier():
    import torch
    torch.cuda.synchronize()


def extra_prefill(device, sampler):
    """c2: 8192-token prefill batch, 20 adapters.  Sustained: regions of 200 forwards for at least 1.5 s."""
    import torch
    from paper_2508_17624_b200 import workloads as wl
    cfg = wl.CONFIGS["c2"]
    pool, x, aid, _, _ = setup_layer(cfg, device)
    out = torch.empty_like(x)
    dbg = pool.moe_forward_debug(0, x, aid)
    torch.cuda.synchronize()
    counts = dbg["counts"].cpu().numpy()
    live = int((counts > 0).sum())
    w = layer_bytes_and_flops(cfg, live)

    def step():
        pool.moe_forward(0, x, aid, out)

    for _ in range(10):
        step()
    with sampler.window():
        regions = timed_regions(step, 200, _sync_barrier, min_total_s=1.5)
    ms = float(np.median(regions)) / 200
    kern, _ = kernel_pass(pool, step, 200, _sync_barrier)
    assert pool.last_device_error() == 0
    pool.destroy()
    _, peak_tf, peak_tf_sus, kind = load_peaks()
    rec = {"workload": WORKLOADS["c2"], "tokens_per_s": cfg.n_tokens / (ms * 1e-3), "ms_per_step": ms,
           "timed_s": float(np.sum(regions)) / 1e3, "live_slots": live,
           "thin_slots": int(((counts > 0) & (counts <= 128)).sum()), "kernels_ms_per_step": kern, "of": kind}
    for g, fl in (("gemm1", w["flops_gemm1"]), ("gemm2", w["flops_gemm2"])):
        tf = fl / (kern[g] * 1e-3) / 1e12
        rec[g] = {"tflops": tf, "frac_of_burst": tf / peak_tf, "frac_of_sustained": tf / peak_tf_sus,
                  "peak_burst": peak_tf, "peak_sustained": peak_tf_sus}
    tf = (w["flops_gemm1"] + w["flops_gemm2"]) / (ms * 1e-3) / 1e12
    rec["layer"] = {"tflops": tf, "frac_of_burst": tf / peak_tf, "frac_of_sustained": tf / peak_tf_sus}
    return rec


def extra_stack(device, sampler, layers=4):
    """c3: a slice of the 26-layer stack (1024 tokens per layer, 20 adapters, Zipf ids), layers back to back."""
    import torch
    from paper_2508_17624_b200 import binding, workloads as wl
    cfg = wl.with_(wl.CONFIGS["c3"], num_layers=layers)
    pool = binding.Pool.from_config(cfg, device=device)
    binding.load_model(pool, cfg)
    aid = torch.from_numpy(wl.gen_adapter_ids(cfg)).cuda()
    xs = [torch.from_numpy(wl.gen_tokens(cfg, l).view(np.int16)).cuda().view(torch.bfloat16) for l in range(layers)]
    outs = [torch.empty_like(x) for x in xs]
    lives = []
    for l in range(layers):
        d = pool.moe_forward_debug(l, xs[l], aid)
        lives.append(int((d["counts"] > 0).sum()) + cfg.num_shared)

    def step():
        for l in range(layers):
            pool.moe_forward(l, xs[l], aid, outs[l])

    for _ in range(5):
        step()
    with sampler.window():
        regions = timed_regions(step, 50, _sync_barrier)
    ms_layer = float(np.median(regions)) / 50 / layers
    assert pool.last_device_error() == 0
    st = pool.stats()
    pool.destroy()
    peak, _, _, kind = load_peaks()
    gb = float(np.mean(lives)) * 3 * cfg.inter * cfg.hidden * 2 / 1e9
    return {"workload": f"c3: {layers} of the 26 stacked decode layers, 1024 tokens per layer, 20 adapters x 7-9 experts, Zipf(1) ids",
            "ms_per_layer": ms_layer, "tokens_per_s_through_26_layers": cfg.n_tokens / (ms_layer * 26e-3),
            "token_layers_per_s": cfg.n_tokens / (ms_layer * 1e-3), "live_experts_per_layer": float(np.mean(lives)),
            "weight_stream": {"achieved": gb / ms_layer * 1e3, "unit": "GB/s", "peak": peak, "frac": gb / ms_layer * 1e3 / peak,
                              "of": kind, "algorithmic_bytes_per_layer": gb * 1e9},
            "pool": {"physical_bytes": st["physical_bytes"], "padding_bytes": st["padding_bytes"]}}


def _reroute_pool(e=32):
    from paper_2508_17624_b200 import binding, workloads as wl
    cfg = wl.CONFIGS["c4"]
    M, k, N = cfg.num_experts, cfg.top_k, cfg.max_adapters
    pool = binding.Pool(hidden=64, inter=64, num_experts=M, num_shared=0, top_k=k, max_adapters=N, e_max=cfg.e_max,
                        max_tokens=8)
    z = np.zeros((M, 64, 64), np.uint16)
    pool.load_base(0, np.zeros((M, 64), np.uint16), z, z, z)
    tuned = wl.tuned_sets(cfg, np.full((N, 1), e))
    za = np.zeros((e, 64, 64), np.uint16)
    for i in range(N):
        pool.load_adapter(i, np.array([e], np.int32), tuned[i][0], za, za, za)
    return pool, cfg


def _reroute_sets(pool, cfg, B, logits_too=False):
    """Rotating buffer sets whose total exceeds the L2 (cold-cache launches)."""
    import torch
    M, k, N, P = cfg.num_experts, cfg.top_k, cfg.max_adapters, cfg.num_slots
    per = (2 * B * k * 4 + B * 4) + (B * M * 4 + B * k * 4 if logits_too else 0)
    n_sets = min(96 if not logits_too else 24, max(2, int((256 << 20) // per) + 1))
    g = torch.Generator(device="cuda").manual_seed(4)
    sets = []
    for _ in range(n_sets):
        logits = torch.randn((B, M), device="cuda", generator=g)
        ids = torch.topk(logits, k, dim=1).indices.to(torch.int32).contiguous()
        aid = torch.randint(-1, N, (B,), device="cuda", generator=g, dtype=torch.int32)
        s = {"ids": ids, "aid": aid, "slots": torch.empty_like(ids), "counts": torch.empty(P, dtype=torch.int32, device="cuda")}
        if logits_too:
            s["logits"] = logits
            s["w"] = torch.empty((B, k), dtype=torch.float32, device="cuda")
            s["ids_out"] = torch.empty_like(ids)
        sets.append(s)
    return sets


def _time_calls(call, sets, iters):
    import torch
    for i in range(3):
        call(sets[i % len(sets)])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(iters):
        call(sets[i % len(sets)])
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def reroute_measurements(pool, cfg, B, iters, with_unfused=True):
    """-> dict of ms per call at B tokens for the stand-alone operator, the gate-fused kernel and the unfused variant."""
    import torch
    from paper_2508_17624_b200 import binding
    M, k, N = cfg.num_experts, cfg.top_k, cfg.max_adapters
    lib, h, st, dp = binding.lib(), pool._h, binding._stream, binding._dp
    peak, _, _, kind = load_peaks()
    sets = _reroute_sets(pool, cfg, B)
    rec = {"tokens": B, "l2": f"cold: {len(sets)} rotating buffer sets", "of": kind}
    ms = _time_calls(lambda s: binding._check(lib.ew_reroute(h, 0, dp(s["ids"]), dp(s["aid"]), B, dp(s["slots"]), dp(s["counts"]), st()), "ew_reroute"), sets, iters)
    nbytes = 2 * B * k * 4 + B * 4 + N * M * 4
    rec["reroute"] = {"us_per_call": ms * 1e3, "GB/s": nbytes / (ms * 1e-3) / 1e9, "frac": nbytes / (ms * 1e-3) / 1e9 / peak,
                      "algorithmic_bytes": nbytes, "tokens_per_s": B / (ms * 1e-3)}
    if with_unfused:
        scratch = torch.empty(2 * B * k, dtype=torch.int32, device="cuda")
        ms_u = _time_calls(lambda s: binding._check(lib.ew_reroute_unfused(h, 0, dp(s["ids"]), dp(s["aid"]), B, dp(s["slots"]), dp(s["counts"]), dp(scratch), st()), "ew_reroute_unfused"), sets, iters)
        rec["unfused"] = {"us_per_call": ms_u * 1e3, "kernels": 4, "slowdown_vs_operator": ms_u / ms}
        del scratch
    del sets
    sets = _reroute_sets(pool, cfg, B, logits_too=True)
    ms_l = _time_calls(lambda s: binding._check(lib.ew_route_logits(h, 0, dp(s["logits"]), dp(s["aid"]), B, dp(s["ids_out"]), dp(s["w"]), dp(s["slots"]), dp(s["counts"]), st()), "ew_route_logits"), sets, iters)
    nb_l = B * M * 4 + B * 4 + 3 * B * k * 4 + N * M * 4
    rec["gate_fused"] = {"us_per_call": ms_l * 1e3, "GB/s": nb_l / (ms_l * 1e-3) / 1e9, "frac": nb_l / (ms_l * 1e-3) / 1e9 / peak,
                         "algorithmic_bytes": nb_l, "tokens_per_s": B / (ms_l * 1e-3)}
    return rec


def extra_reroute(device, sampler):
    """c4: the batched rerouting operator alone (ids in; slot ids + per-slot counts out), the same step fused with the
    gate function before it (fp32 logits in), and the unfused variant (one kernel per tensor operation), at the
    workload's 65,536 tokens and at 4 M tokens; 20 adapters re-tuning 50 % of the experts."""
    pool, cfg = _reroute_pool(32)
    with sampler.window():
        rec = {"workload": "c4: reroute only, 64 experts, top-6, 20 adapters x 32 experts, adapter ids per token",
               "peak_hbm_gbs": load_peaks()[0],
               "65536": reroute_measurements(pool, cfg, 65536, 300),
               "4194304": reroute_measurements(pool, cfg, 1 << 22, 40)}
    assert pool.last_device_error() == 0
    pool.destroy()
    return rec


def extra_padding(device, sampler, pairs=7):
    """Padding baseline (pool_mode = 1, the whole tensor backed at creation) against pages mapped on demand: the decode
    layer of c1 with 16 slots reserved per adapter of which 8 are tuned (half of every adapter's range is padding);
    alternating A/B timing pairs, median difference."""
    import torch
    from paper_2508_17624_b200 import workloads as wl
    cfg = wl.with_(wl.CONFIGS["c1"], e_max=16)
    pools = {}
    for mode in (0, 1):
        pool, x, aid, _, _ = setup_layer(cfg, device, pool_mode=mode)
        pools[mode] = (pool, x, aid, torch.empty_like(x))
    ms = {0: [], 1: []}
    with sampler.window():
        for _ in range(pairs):
            for mode in (0, 1):
                pool, x, aid, out = pools[mode]
                for _ in range(20):
                    pool.moe_forward(0, x, aid, out)
                r = timed_regions(lambda: pool.moe_forward(0, x, aid, out), 300, _sync_barrier, min_total_s=0.0, max_regions=3)
                ms[mode].append(float(np.median(r)) / 300)
    assert torch.equal(pools[0][3], pools[1][3])
    stats = {m: pools[m][0].stats() for m in (0, 1)}
    for m in (0, 1):
        pools[m][0].destroy()
    delta = [(b - a) / a for a, b in zip(ms[0], ms[1])]
    return {"workload": WORKLOADS["c1"] + ", 16 slots reserved per adapter", "pairs": pairs, "ms_on_demand": float(np.median(ms[0])), "ms_padding": float(np.median(ms[1])),
            "latency_delta_median": float(np.median(delta)), "latency_delta_min": float(np.min(delta)),
            "latency_delta_max": float(np.max(delta)),
            "physical_bytes_on_demand": stats[0]["physical_bytes"], "physical_bytes_padding": stats[1]["physical_bytes"],
            "saved_frac": 1.0 - stats[0]["physical_bytes"] / stats[1]["physical_bytes"]}


def extra_expert_parallel(device, sampler):
    """Expert parallelism with the ranks emulated on this one GPU: each rank's pool holds its block of the experts
    (ep_size = R), the ranks run one after the other, and each rank's partial forward is timed alone - the time one
    GPU of an R-GPU deployment would spend per layer before the all-reduce, which is not measured here (one GPU)."""
    import torch
    from paper_2508_17624_b200 import binding, workloads as wl
    cfg = wl.CONFIGS["c1"]
    bank = wl.NoiseBank(cfg.seed)
    tuned = wl.tuned_sets(cfg)
    base = wl.gen_base_layer(cfg, 0, bank)
    ads = [wl.gen_adapter_layer(cfg, i, 0, tuned[i][0], bank) for i in range(cfg.max_adapters)]
    x = torch.from_numpy(wl.gen_tokens(cfg).view(np.int16)).cuda().view(torch.bfloat16)
    aid = torch.from_numpy(wl.gen_adapter_ids(cfg)).cuda()
    rec = {"workload": WORKLOADS["c1"], "all_reduce": "not measured (one GPU): fp32 [tokens, H] per layer = %d bytes" % (cfg.n_tokens * cfg.hidden * 4),
           "ranks": {}}
    for R, ranks in ((2, (0, 1)), (8, (0, 1, 7))):
        per_rank = {}
        for r in ranks:
            pool = binding.Pool.from_config(cfg, device=device, ep_size=R, ep_rank=r)
            pool.load_base(0, base.router_w, base.routed.w_gate, base.routed.w_up, base.routed.w_down, base.shared.w_gate,
                           base.shared.w_up, base.shared.w_down)
            for i, e in enumerate(ads):
                pool.load_adapter(i, np.array([len(tuned[i][0])], np.int32), tuned[i][0].astype(np.int32), e.w_gate, e.w_up, e.w_down)
            part = torch.empty((cfg.n_tokens, cfg.hidden), dtype=torch.float32, device="cuda")
            for _ in range(20):
                pool.moe_forward_partial(0, x, aid, part)
            with sampler.window():
                reg = timed_regions(lambda: pool.moe_forward_partial(0, x, aid, part), 300, _sync_barrier, min_total_s=0.2, max_regions=5)
            st = pool.stats()
            per_rank[str(r)] = {"ms_per_partial_forward": float(np.median(reg)) / 300, "live_experts": st["live_experts"],
                                "physical_bytes": st["physical_bytes"], "kernels_per_forward": st["last_forward_kernels"]}
            assert pool.last_device_error() == 0
            pool.destroy()
        rec["ranks"]["ep%d" % R] = per_rank
    return rec


def run_reroute(args):
    """--workload c4: the rerouting operator alone, one JSON line per coverage (10 / 25 / 50 % of the experts
    re-tuned) at 65536 tokens (or --tokens), then a size sweep of the 50 % case up to 2^24 tokens."""
    import torch
    from paper_2508_17624_b200 import build
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    build.build()
    for e in ((32,) if args.tokens else (6, 16, 32)):
        pool, cfg = _reroute_pool(e)
        rec = reroute_measurements(pool, cfg, args.tokens or cfg.n_tokens, args.steps)
        rec["config"] = {"workload": f"c4: reroute only, {rec['tokens']} tokens, 20 adapters x {e} of 64 experts"}
        gf = rec["gate_fused"]
        gf["roofline_alu"] = {"bound": "alu", "instructions_per_token": ALU_INSTR_PER_TOKEN_C4, "peak": ALU_PEAK_TINSTR,
                              "unit": "T thread-instructions/s",
                              "achieved": gf["tokens_per_s"] * ALU_INSTR_PER_TOKEN_C4 / 1e12,
                              "frac": gf["tokens_per_s"] * ALU_INSTR_PER_TOKEN_C4 / 1e12 / ALU_PEAK_TINSTR}
        print(json.dumps(rec))
        if e == 32 and not args.tokens:
            sweep = [reroute_measurements(pool, cfg, 1 << lg, max(20, args.steps >> max(0, lg - 17)), with_unfused=False)
                     for lg in (16, 18, 20, 22, 24)]
            print(json.dumps({"metric": "batched reroute, size sweep (50 % coverage)", "sweep": sweep}))
        assert pool.last_device_error() == 0
        pool.destroy()


def build_oracle_layer(cfg):
    import oracle
    from paper_2508_17624_b200 import workloads as wl
    bank = wl.NoiseBank(cfg.seed)
    base = wl.gen_base_layer(cfg, 0, bank)
    tuned = wl.tuned_sets(cfg)
    ads = []
    for i in range(cfg.max_adapters):
        ew = wl.gen_adapter_layer(cfg, i, 0, tuned[i][0], bank)
        ads.append((tuned[i][0], ew.w_gate, ew.w_up, ew.w_down))
    oc = oracle.OracleConfig(cfg.hidden, cfg.inter, cfg.num_experts, cfg.num_shared, cfg.top_k, cfg.max_adapters,
                             cfg.e_max)
    return oracle.OracleLayer(oc, base.router_w, base.routed.w_gate, base.routed.w_up, base.routed.w_down,
                              base.shared.w_gate, base.shared.w_up, base.shared.w_down, ads)


def cpu_baseline(cfg, budget_s: float):
    """The oracle as it stands, timed on the host cores on a bounded sample of the same batch."""
    import oracle
    from paper_2508_17624_b200 import workloads as wl
    layer = build_oracle_layer(cfg)
    x, aid = wl.gen_tokens(cfg), wl.gen_adapter_ids(cfg)
    n = min(32, cfg.n_tokens)
    t0 = time.time()
    oracle.layer_forward(layer, x[:n], aid[:n])
    per_tok = (time.time() - t0) / n
    n = int(max(1, min(cfg.n_tokens, budget_s / max(per_tok, 1e-9))))
    passes = int(max(1, min(64, budget_s / max(per_tok * n, 1e-9))))     # the whole batch fits the budget: repeat it
    t0 = time.time()
    for _ in range(passes):
        oracle.layer_forward(layer, x[:n], aid[:n])
    dt = time.time() - t0
    return {"value": n * passes / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"first {n} of the {cfg.n_tokens} tokens of the same batch, {passes} passes, {dt:.2f} s"}


def run_reference(args):
    """--impl reference: the CPU oracle, same metric and config; each step a bounded sample of the batch."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2508_17624_b200 import workloads as wl
    cfg = wl.CONFIGS["c1"]
    layer = build_oracle_layer(cfg)
    x, aid = wl.gen_tokens(cfg), wl.gen_adapter_ids(cfg)
    t0 = time.time()
    oracle.layer_forward(layer, x[:16], aid[:16])
    per_tok = (time.time() - t0) / 16
    total_steps = args.steps + max(args.warmup, 0)
    n = int(max(1, min(cfg.n_tokens, 150.0 / max(per_tok * total_steps, 1e-9))))
    for _ in range(max(args.warmup, 0)):
        oracle.layer_forward(layer, x[:n], aid[:n])
    t0 = time.time()
    for _ in range(args.steps):
        oracle.layer_forward(layer, x[:n], aid[:n])
    dt = time.time() - t0
    value = n * args.steps / dt
    cores = oracle.num_threads()
    sample = f"each step = the first {n} of the batch's {cfg.n_tokens} tokens"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------------ N ranks, one node
def _free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_entry(rank, world, port, backend, body, body_args):
    """One spawned rank: the environment torchrun would have set, a process group, then the per-rank body."""
    import torch.distributed as dist
    os.environ.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world),
                       "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    if backend == "nccl":
        import torch
        torch.cuda.set_device(rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", rank))
    else:
        dist.init_process_group(backend)
    try:
        body(*body_args)
    finally:
        if dist.is_initialized():
            dist.destroy_process_group()


def spawn_ranks(world, body, body_args=(), backend="nccl"):
    """`python bench.py --gpus N` typed as is: start N ranks on this node (one per GPU), each running body(*body_args)
    with RANK / LOCAL_RANK / WORLD_SIZE set and a process group up.  Replicas only: the group serves the barrier and
    the max-over-ranks reduction of the timings."""
    import torch.multiprocessing as mp
    port = _free_port()
    mp.spawn(_rank_entry, args=(world, port, backend, body, body_args), nprocs=world, join=True)


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="only the headline workload (no c2 / c3 / c4 / padding records)")
    ap.add_argument("--workload", default="c1", choices=sorted(WORKLOADS) + ["c4"],
                    help="c1 (decode, the benchmark's workload), c2 (prefill) or c4 (reroute operator only)")
    ap.add_argument("--tokens", type=int, default=0, help="c4 only: one run at this many tokens (50 %% coverage)")
    ap.add_argument("--minimal", action="store_true",
                    help="warm-up and K timed steps only (for profiler captures)")
    return ap.parse_args(argv)


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "c4":
        run_reroute(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args.gpus, run_cuda, (args,))
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
