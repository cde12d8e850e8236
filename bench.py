#!/usr/bin/env python
"""Benchmark of the adapter-aware MoE layer forward (ExpertWeave hot path) on B200.

A step is one pass of the whole hot path (router + top-k + batched rerouting + histogram, permute,
grouped SwiGLU GEMM-1, GEMM-2, combine) over one decode batch of the DeepSeek-V2-Lite-shaped layer
(workload c1: 256 tokens, 64 routed + 2 shared experts, top-6, 4 adapters x 8 re-tuned experts).

  python bench.py [--gpus N] [--steps K] [--warmup W]      the CUDA path (prints one JSON line)
  python bench.py --impl reference ...                     the CPU oracle as it stands, same metric

With N > 1 (torchrun) every rank runs its own replica of the batch on its own GPU (the path has no
exchange step), the timed region is bracketed by barriers and the slowest rank's time is used.
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

# DRAM bytes (read + write) per launch of the dominant kernel from the committed ncu captures
# (profiles/c1_decode_grouped_gemm_full.md); reported beside the algorithmic bytes, not used in any ratio.
NCU_TRAFFIC_BYTES = {"c1": 1.1529e9}
# route_logits_kernel at the c4 shape: thread instructions per token from one ncu capture (smsp__inst_executed x 32 /
# tokens, profiles/c4_reroute_operator.md), and the issue peak of the GPU
ALU_INSTR_PER_TOKEN_C4 = 215 * 32
ALU_PEAK_TINSTR = 148 * 4 * 32 * 1.965e9 / 1e12

METRIC = "adapter-aware MoE layer tokens/s"
UNIT = "tokens/s"
WORKLOADS = {
    "c1": "c1: DeepSeek-V2-Lite-shaped MoE layer, decode batch 256, 4 adapters x 8 experts",
    "c2": "c2: DeepSeek-V2-Lite-shaped MoE layer, prefill 8192 tokens (32 requests x 256), 20 adapters x 4-16 experts",
}
WORKLOAD = WORKLOADS["c1"]


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
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

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

    def summary(self):
        out = {"sm_mhz": float(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
               "reasons": sorted(self.reasons), "samples": len(self.samples)}
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


def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2508_17624_b200 import binding, build, workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    cfg = wl.CONFIGS[args.workload]
    workload = WORKLOADS[args.workload]
    B, H, k = cfg.n_tokens, cfg.hidden, cfg.top_k
    pool = binding.Pool.from_config(cfg, device=local)
    binding.load_model(pool, cfg)
    x_bits, aid_np = wl.gen_tokens(cfg), wl.gen_adapter_ids(cfg)
    x = torch.from_numpy(x_bits.view(np.int16)).cuda().view(torch.bfloat16)
    aid = torch.from_numpy(aid_np).cuda()
    out = torch.empty_like(x)

    # structure of this batch (for the algorithmic bytes): live slots from one debug forward
    dbg = pool.moe_forward_debug(0, x, aid)
    torch.cuda.synchronize()
    counts = dbg["counts"].cpu().numpy()
    live = int((counts > 0).sum())
    groups = live + cfg.num_shared
    pairs = B * k
    rows_act = cfg.num_shared * B + pairs
    blk = cfg.inter * cfg.hidden * 2
    bytes_gemm1 = groups * 2 * blk + (pairs + B) * H * 2 + rows_act * cfg.inter * 2     # weights + rows in + act out
    bytes_gemm2 = groups * blk + rows_act * cfg.inter * 2 + rows_act * H * 4
    bytes_layer = groups * 3 * blk

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        pool.moe_forward(0, x, aid, out)
    barrier()
    sampler = ClockSampler(physical_index(local))
    sampler.start()

    # ---- timed region: K forwards back to back (the kernels of a forward chain by programmatic dependent launch)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.active = True
    e0.record()
    for _ in range(args.steps):
        pool.moe_forward(0, x, aid, out)
    e1.record()
    barrier()
    sampler.active = False
    ms_total = e0.elapsed_time(e1)
    extended = False
    if len(sampler.samples) < 3 and not args.minimal:   # short runs: keep the same load going until the sampler has seen it
        extended = True
        sampler.active = True
        t_end = time.time() + 1.5
        while time.time() < t_end and len(sampler.samples) < 5:
            for _ in range(50):
                pool.moe_forward(0, x, aid, out)
            torch.cuda.synchronize()
        sampler.active = False

    # ---- the same K forwards again with the library's per-kernel CUDA events on the same stream: the events
    #      sit between the kernels, so this pass runs without launch overlap and is a little slower
    side_steps = args.steps
    pool.profile_enable(True)
    pool.profile_read()
    barrier()
    e0.record()
    for _ in range(side_steps):
        pool.moe_forward(0, x, aid, out)
    e1.record()
    barrier()
    ms_plain = e0.elapsed_time(e1)
    kern_ms, n_prof = pool.profile_read()
    pool.profile_enable(False)
    if args.minimal:
        side_steps = 0

    # ---- end to end through the C ABI with host buffers (pinned): H2D + forward + D2H every step
    xh = torch.from_numpy(x_bits.view(np.int16).copy()).pin_memory()
    ah = torch.from_numpy(aid_np.copy()).pin_memory()
    oh = torch.empty((B, H), dtype=torch.int16).pin_memory()
    for _ in range(3 if side_steps else 1):
        pool.moe_forward_host(0, xh, ah, oh)
    barrier()
    e0.record()
    for _ in range(max(side_steps, 1)):
        pool.moe_forward_host(0, xh, ah, oh)
    e1.record()
    barrier()
    ms_e2e = e0.elapsed_time(e1)
    assert torch.equal(oh.cuda().view(torch.bfloat16), out), "host-buffer path disagrees with the device path"
    sampler.stop()
    err = pool.last_device_error()
    assert err == 0, f"device error word {err}"

    ms_total, ms_e2e, ms_plain = reduce_max_over_ranks([ms_total, ms_e2e, ms_plain], device="cuda")

    result = None
    if rank == 0:
        peak, peak_tf, peak_tf_sustained, peak_kind = load_peaks()
        g1_ms = kern_ms["gemm1"] / max(n_prof, 1)
        achieved = bytes_gemm1 / (g1_ms * 1e-3) / 1e9
        flops_gemm1 = 2.0 * rows_act * 2 * cfg.inter * H
        flops_gemm2 = 2.0 * rows_act * cfg.inter * H
        tensor_bound = flops_gemm1 / (peak_tf * 1e12) > bytes_gemm1 / (peak * 1e9)
        if tensor_bound:
            roof = {"bound": "tensor", "kernel": "grouped_gemm_kernel<GLU> (GEMM-1 + SwiGLU)",
                    "achieved": flops_gemm1 / (g1_ms * 1e-3) / 1e12, "peak": peak_tf, "unit": "TFLOP/s",
                    "frac": flops_gemm1 / (g1_ms * 1e-3) / 1e12 / peak_tf, "of": peak_kind + " (bf16 burst)",
                    "traffic": None, "algorithmic_flops": flops_gemm1, "avg_launch_ms": g1_ms,
                    "hbm_gbs": achieved,
                    # the timed loop runs for seconds under the power cap: the sustained cuBLAS figure beside it
                    "peak_sustained": peak_tf_sustained,
                    "frac_of_sustained": flops_gemm1 / (g1_ms * 1e-3) / 1e12 / peak_tf_sustained}
        else:
            roof = {"bound": "hbm", "kernel": "grouped_gemm_kernel<GLU> (GEMM-1 + SwiGLU)",
                    "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "of": peak_kind, "traffic": NCU_TRAFFIC_BYTES.get(args.workload), "algorithmic_bytes": bytes_gemm1,
                    "avg_launch_ms": g1_ms}
        result = {
            "metric": METRIC, "value": whole_job_tokens_per_s(world, B, args.steps, ms_total), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload, "tokens_per_step_per_gpu": B, "hidden": H, "inter": cfg.inter,
                       "experts": cfg.num_experts, "shared": cfg.num_shared, "top_k": k,
                       "adapters": cfg.max_adapters, "e_max": cfg.e_max, "live_slots": live,
                       "parallelism": f"replicas x{world}",
                       "l2": "no flush: each step streams %.2f GB of live expert weights, far above the 126 MB L2"
                             % (bytes_layer / 1e9)},
            "e2e": {"value": whole_job_tokens_per_s(world, B, max(side_steps, 1), ms_e2e), "unit": UNIT,
                    "h2d_bytes_per_step": B * H * 2 + B * 4, "d2h_bytes_per_step": B * H * 2},
            "gpu_launches": 5 * args.steps,
            "clocks": dict(sampler.summary(), extended=extended),
            "roofline": roof,
            "kernels_ms_per_step": {kname: v / max(n_prof, 1) for kname, v in kern_ms.items()},
            "gemm2": {"achieved": bytes_gemm2 / (kern_ms["gemm2"] / max(n_prof, 1) * 1e-3) / 1e9, "unit": "GB/s",
                      "algorithmic_bytes": bytes_gemm2,
                      "tflops": flops_gemm2 / (kern_ms["gemm2"] / max(n_prof, 1) * 1e-3) / 1e12},
            "layer_weight_stream": {"achieved": bytes_layer / (ms_total / args.steps * 1e-3) / 1e9, "unit": "GB/s",
                                    "frac": bytes_layer / (ms_total / args.steps * 1e-3) / 1e9 / peak},
            "ms_per_step_with_kernel_events": ms_plain / args.steps,
        }
        if not args.no_cpu_baseline and not args.minimal and world == 1:
            result["cpu_baseline"] = cpu_baseline(cfg, budget_s=24.0)
    pool.destroy()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(result))


def run_reroute(args):
    """--workload c4: the batched rerouting operator alone (ids in, slot ids + per-slot counts out), and the same
    step fused with the gate function before it (fp32 logits in).

    One JSON line per coverage (10 / 25 / 50 % of the experts re-tuned) at 65536 tokens, plus a size sweep
    up to 2^24 tokens.  Cold L2: consecutive launches work on different buffer sets whose total exceeds the
    L2 (256 MB).  GB/s = algorithmic bytes (ids in + slots out + adapter ids in + map) / mean launch time.
    """
    import torch
    from paper_2508_17624_b200 import binding, build, workloads as wl
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    build.build()
    cfg = wl.CONFIGS["c4"]
    M, k, N, P = cfg.num_experts, cfg.top_k, cfg.max_adapters, cfg.num_slots
    pool = binding.Pool(hidden=64, inter=64, num_experts=M, num_shared=0, top_k=k, max_adapters=N, e_max=cfg.e_max,
                        max_tokens=8)
    z = np.zeros((M, 64, 64), np.uint16)
    pool.load_base(0, np.zeros((M, 64), np.uint16), z, z, z)
    peak, _, _, peak_kind = load_peaks()
    lines = []

    def measure(B, iters):
        pair_bytes = 2 * B * k * 4 + B * 4 + N * M * 4
        n_sets = max(2, int((256 << 20) // pair_bytes) + 1)
        g = torch.Generator(device="cuda").manual_seed(4)
        sets = []
        for _ in range(min(n_sets, 96)):
            logits = torch.randn((B, M), device="cuda", generator=g)
            ids = torch.topk(logits, k, dim=1).indices.to(torch.int32).contiguous()
            aid = torch.randint(-1, N, (B,), device="cuda", generator=g, dtype=torch.int32)
            sets.append((ids, aid, torch.empty_like(ids), torch.empty(P, dtype=torch.int32, device="cuda")))
            del logits
        for i in range(3):
            pool.reroute(0, *sets[i % len(sets)][:2], slot_ids=sets[i % len(sets)][2], counts=sets[i % len(sets)][3])
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for i in range(iters):
            s_ = sets[i % len(sets)]
            pool.reroute(0, s_[0], s_[1], slot_ids=s_[2], counts=s_[3])
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        return pair_bytes, ms, len(sets)

    for e in ((32,) if args.tokens else (6, 16, 32)):
        tuned = wl.tuned_sets(cfg, np.full((N, 1), e))
        za = np.zeros((e, 64, 64), np.uint16)
        for i in range(N):
            pool.load_adapter(i, np.array([e], np.int32), tuned[i][0], za, za, za)
        nbytes, ms, n_sets = measure(args.tokens or cfg.n_tokens, args.steps)
        gbs = nbytes / (ms * 1e-3) / 1e9
        lines.append({"metric": "batched reroute GB/s", "value": gbs, "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
                      "ms_per_launch": ms, "tokens": args.tokens or cfg.n_tokens,
                      "tokens_per_s": (args.tokens or cfg.n_tokens) / (ms * 1e-3),
                      "dtype": "int32", "data": "synthetic",
                      "config": {"workload": f"c4: reroute only, {args.tokens or cfg.n_tokens} tokens, 20 adapters x {e} of 64 experts",
                                 "l2": f"cold: {n_sets} rotating buffer sets", "includes": "zeroing of counts + kernel"},
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                                   "of": peak_kind, "algorithmic_bytes": nbytes, "traffic": None}})
        if e != 32:
            for i in range(N):
                pool.unload_adapter(i)
    # ---- the same step fused with the gate function before it: fp32 logits in; ids, weights, slot ids and counts out
    def measure_logits(B, iters):
        nbytes = B * M * 4 + B * 4 + 3 * B * k * 4 + N * M * 4
        n_sets = min(24, max(2, int((256 << 20) // nbytes) + 1))
        g = torch.Generator(device="cuda").manual_seed(5)
        sets = [(torch.randn((B, M), device="cuda", generator=g),
                 torch.randint(-1, N, (B,), device="cuda", generator=g, dtype=torch.int32)) for _ in range(n_sets)]
        for i in range(3):
            pool.route_logits(0, *sets[i % n_sets])
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        outs = pool.route_logits(0, *sets[0])                      # output tensors reused below: no allocation in the loop
        torch.cuda.synchronize()
        e0.record()
        for i in range(iters):
            lg_, aid_ = sets[i % n_sets]
            binding._check(binding.lib().ew_route_logits(pool._h, 0, binding._dp(lg_), binding._dp(aid_), B, binding._dp(outs[0]),
                                                         binding._dp(outs[1]), binding._dp(outs[2]), binding._dp(outs[3]),
                                                         binding._stream()), "ew_route_logits")
        e1.record()
        torch.cuda.synchronize()
        return nbytes, e0.elapsed_time(e1) / iters, n_sets

    Bt = args.tokens or cfg.n_tokens
    nbytes, ms, n_sets = measure_logits(Bt, args.steps)
    gbs = nbytes / (ms * 1e-3) / 1e9
    lines.append({"metric": "gate + reroute from logits GB/s", "value": gbs, "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
                  "ms_per_launch": ms, "tokens": Bt, "tokens_per_s": Bt / (ms * 1e-3), "dtype": "f32", "data": "synthetic",
                  "config": {"workload": f"c4: softmax + top-k + reroute + counts from fp32 logits, {Bt} tokens, 20 adapters x 32 of 64 experts",
                             "l2": f"cold: {n_sets} rotating buffer sets", "includes": "zeroing of counts + kernel"},
                  # bound by arithmetic (softmax + k selection rounds over M probabilities), not by memory: ncu counts 215
                  # warp instructions per token (M = 64, k = 6); peak = 148 SMs x 4 schedulers x 32 lanes x 1.965 GHz
                  "roofline": {"bound": "alu", "achieved": Bt / (ms * 1e-3) * ALU_INSTR_PER_TOKEN_C4 / 1e12, "peak": ALU_PEAK_TINSTR,
                               "unit": "T thread-instructions/s", "of": "derived: SM count x issue slots x lanes x max clock",
                               "frac": Bt / (ms * 1e-3) * ALU_INSTR_PER_TOKEN_C4 / 1e12 / ALU_PEAK_TINSTR,
                               "instructions_per_token": ALU_INSTR_PER_TOKEN_C4, "hbm_gbs": gbs, "hbm_frac": gbs / peak,
                               "algorithmic_bytes": nbytes, "traffic": None}})
    sweep = []
    for lg in (() if args.tokens else (16, 18, 20, 22)):
        nb_, ms_, _ = measure_logits(1 << lg, max(20, args.steps >> max(0, lg - 16)))
        sweep.append({"tokens": 1 << lg, "ms_per_launch": ms_, "GB/s": nb_ / (ms_ * 1e-3) / 1e9,
                      "frac": nb_ / (ms_ * 1e-3) / 1e9 / peak})
    lines.append({"metric": "gate + reroute from logits GB/s, size sweep", "sweep": sweep, "peak": peak, "of": peak_kind})
    sweep = []
    for lg in (() if args.tokens else (16, 18, 20, 22, 24)):
        nbytes, ms, n_sets = measure(1 << lg, max(20, args.steps >> max(0, lg - 18)))
        sweep.append({"tokens": 1 << lg, "ms_per_launch": ms, "GB/s": nbytes / (ms * 1e-3) / 1e9,
                      "frac": nbytes / (ms * 1e-3) / 1e9 / peak})
    lines.append({"metric": "batched reroute GB/s, size sweep (50 % coverage)", "sweep": sweep, "peak": peak, "of": peak_kind})
    assert pool.last_device_error() == 0
    pool.destroy()
    for ln in lines:
        print(json.dumps(ln))


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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="c1", choices=sorted(WORKLOADS) + ["c4"],
                    help="c1 (decode, the benchmark's workload), c2 (prefill) or c4 (reroute operator only)")
    ap.add_argument("--tokens", type=int, default=0, help="c4 only: one run at this many tokens (50 %% coverage)")
    ap.add_argument("--minimal", action="store_true",
                    help="warm-up and timed steps only (for profiler captures): no CPU baseline, no side measurements")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "c4":
        run_reroute(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
