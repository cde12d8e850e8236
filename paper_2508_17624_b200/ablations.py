"""In-house analogues of the paper's micro-benchmarks (Section 5.3 / 5.4), on synthetic layers.

  python -m paper_2508_17624_b200.ablations [--steps K]

Prints one JSON object:
  adapters_vs_base   layer time with 4 adapters in the batch vs the same layer serving base-model tokens only
                     (the paper's "overhead vs Base-Only", Section 5.2, restated for one layer)
  vmm_vs_padding     layer time and physical bytes, pages on demand vs the fully backed padding tensor
                     (Section 5.3 "virtual weight tensor vs padding", Section 5.4 memory)
  churn              evicting and re-loading one adapter (8 experts, 132 MiB) while forwards are in flight:
                     host-side latency of ew_unload_adapter / ew_load_adapter and page reuse (Section 4.2)
  batch_sweep        the c1 layer (4 adapters) from 1 to 8192 tokens per call: ms, tokens/s, live experts, weight
                     stream TB/s and TFLOP/s (where the layer turns from weight-bound to tensor-bound)
  reroute            the batched rerouting step three ways: fused into the router kernel (its share of the
                     layer), the stand-alone operator, and the unfused formulation from stock tensor ops
                     (broadcast the adapter ids, compute offsets into the map, gather: the paper's
                     "SingleOp" variant, Section 5.3)
All inputs are seeded and synthetic (workloads.py); timings are CUDA events over K back-to-back calls.
"""
import argparse
import json

import numpy as np


def _time(fn, steps, torch):
    for _ in range(5):
        fn()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def table1_shaped_counts(max_e: int, avg_e: float, layers: int, seed: int) -> np.ndarray:
    """Per-layer expert counts with the given maximum and (rounded) average: the paper prints only these two
    summary numbers per adapter (Table 1), not the per-layer counts."""
    rng = np.random.default_rng(seed)
    target = int(round(avg_e * layers))
    e = rng.integers(1, max_e + 1, size=layers)
    e[rng.integers(layers)] = max_e
    while e.sum() != target:
        i = rng.integers(layers)
        if e.sum() > target and e[i] > 1 and (e[i] < max_e or (e == max_e).sum() > 1):
            e[i] -= 1
        elif e.sum() < target and e[i] < max_e:
            e[i] += 1
    return e.astype(np.int32)


def memory_table1_shapes(page_bytes: int = 0):
    """Adapter memory, pages on demand vs padding, for Table-1-shaped adapters of the DeepSeek-V2-Lite shape
    (26 layers, 64 experts, 16.5 MiB per expert), on the accounting-only backend (no GPU needed).  The paper's
    Section 5.4 loads gate-math, then gate-intent, then token-math and reports 40.4 %, 28.9 % and 37.3 % less.
    `page_bytes` = 0 takes the driver's minimum granularity (2 MiB); larger pages cost rounding at every adapter's
    two ends (Section 4.2's sub-page sharing removes it between neighbours only)."""
    from . import binding, workloads as wl
    shapes = [("gate-math", 12, 7.04), ("gate-intent", 12, 9.50), ("token-math", 9, 6.12)]
    L, M, e_max = 26, 64, 12
    out = []
    pools = {}
    for mode in (0, 1):
        pools[mode] = binding.Pool(device=-1, num_layers=L, hidden=2048, inter=1408, num_experts=M, num_shared=2,
                                   top_k=6, max_adapters=3, e_max=e_max, max_tokens=16, pool_mode=mode,
                                   page_bytes=page_bytes)
        for l in range(L):
            pools[mode].load_base(l, None, None, None, None, None, None, None)
    base = {m: pools[m].stats()["physical_bytes"] for m in pools}
    base_pad_reserved = 3 * e_max * L * 3 * 1408 * 2048 * 2
    for i, (name, mx, avg) in enumerate(shapes):
        counts = table1_shaped_counts(mx, avg, L, seed=100 + i)
        ids = np.concatenate([np.arange(c, dtype=np.int32) for c in counts])
        for m in pools:
            pools[m].load_adapter(i, counts, ids, None, None, None)
        vmm = pools[0].stats()["physical_bytes"] - base[0]
        # the padding tensor reserves E_max slots for every adapter that is loaded
        pad = (i + 1) * e_max * L * 3 * 1408 * 2048 * 2
        out.append({"adapters": i + 1, "added": name, "adapter_bytes_vmm": vmm, "adapter_bytes_padding": pad,
                    "saving": 1.0 - vmm / pad})
    assert pools[1].stats()["physical_bytes"] - pools[0].stats()["physical_bytes"] > 0
    for m in pools:
        pools[m].destroy()
    return out


def page_size_sweep(gpu: bool):
    """Page size of the physical pool (Section 4.2): larger pages mean fewer map/unmap driver calls per adapter
    (the load latency is mostly those calls) and more rounding at the adapters' ends.  Memory side on the
    accounting backend (Table-1-shaped adapters), latency side (if `gpu`) on one c1-shaped adapter of 8 experts
    with its weights in page-locked host memory and no forward in flight."""
    from . import binding, workloads as wl
    rows = []
    for mib in (2, 4, 8, 32):
        row = {"page_MiB": mib, "table1_saving": [r["saving"] for r in memory_table1_shapes(mib << 20)]}
        if gpu:
            import time
            import torch
            cfg = wl.CONFIGS["c1"]
            bank = wl.NoiseBank(cfg.seed)
            pool = binding.Pool.from_config(cfg, page_bytes=mib << 20)
            binding.load_model(pool, cfg, bank)
            tuned = wl.tuned_sets(cfg)
            ew3 = wl.gen_adapter_layer(cfg, 3, 0, tuned[3][0], bank)
            src = [torch.from_numpy(a.view(np.int16)).pin_memory().numpy().view(np.uint16)
                   for a in (ew3.w_gate, ew3.w_up, ew3.w_down)]
            t_un, t_ld = [], []
            for _ in range(6):
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                pool.unload_adapter(3)
                t1 = time.perf_counter()
                pool.load_adapter(3, np.array([len(tuned[3][0])], np.int32), tuned[3][0], *src)
                t2 = time.perf_counter()
                t_un.append((t1 - t0) * 1e3)
                t_ld.append((t2 - t1) * 1e3)
            row.update(unload_ms=float(np.median(t_un)), load_ms=float(np.median(t_ld)),
                       pages_per_adapter=int(-(-ew3.w_gate.nbytes * 3 // (mib << 20))))
            pool.destroy()
        rows.append(row)
    return rows


def main():
    import torch
    from . import binding, build, workloads as wl
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=500)
    args = ap.parse_args()
    assert torch.cuda.is_available(), "needs a CUDA device"
    build.build()
    cfg = wl.CONFIGS["c1"]
    bank = wl.NoiseBank(cfg.seed)
    x = torch.from_numpy(wl.gen_tokens(cfg).view(np.int16)).cuda().view(torch.bfloat16)
    aid = torch.from_numpy(wl.gen_adapter_ids(cfg)).cuda()
    base_aid = torch.full_like(aid, -1)
    out = torch.empty_like(x)
    res = {}

    # ---- pages on demand
    pool = binding.Pool.from_config(cfg)
    binding.load_model(pool, cfg, bank, adapters=[])
    t_base_only = _time(lambda: pool.moe_forward(0, x, base_aid, out), args.steps, torch)
    st_base = pool.stats()
    binding.load_model(pool, cfg, bank, layers=[])           # now the four adapters
    t_mixed = _time(lambda: pool.moe_forward(0, x, aid, out), args.steps, torch)
    t_base_tokens = _time(lambda: pool.moe_forward(0, x, base_aid, out), args.steps, torch)
    pool.profile_enable(True)
    pool.profile_read()
    for _ in range(200):
        pool.moe_forward(0, x, aid, out)
    kern, n = pool.profile_read()
    pool.profile_enable(False)
    st_vmm = pool.stats()
    d = pool.moe_forward_debug(0, x, aid)
    torch.cuda.synchronize()
    live = int((d["counts"] > 0).sum())
    res["adapters_vs_base"] = {
        "ms_base_only_pool": t_base_only, "ms_adapters_loaded_base_tokens": t_base_tokens, "ms_mixed_batch": t_mixed,
        "overhead_mixed_vs_base_only": t_mixed / t_base_only - 1.0,
        "live_slots_mixed": live, "live_weight_bytes_ratio": (live + cfg.num_shared) / (cfg.num_experts + cfg.num_shared)}
    res["reroute"] = {"router_kernel_ms": kern["route"] / n, "layer_ms_with_kernel_events": sum(kern.values()) / n,
                      "router_share_of_layer": kern["route"] / sum(kern.values())}

    # ---- churn: evict and re-load adapter 3 with 20 forwards queued each time
    import time
    tuned = wl.tuned_sets(cfg)
    ew3 = wl.gen_adapter_layer(cfg, 3, 0, tuned[3][0], bank)
    aid_wo3 = torch.where(aid == 3, torch.full_like(aid, -1), aid)
    created0 = pool.stats()["pages_created_total"]
    # the same weights in page-locked host memory: the copy then runs at the host link's speed, and what is left
    # of the load latency is the page mapping
    pinned = [torch.from_numpy(a.view(np.int16)).pin_memory().numpy().view(np.uint16) for a in (ew3.w_gate, ew3.w_up, ew3.w_down)]
    on_device = [torch.from_numpy(a.view(np.int16)).cuda() for a in (ew3.w_gate, ew3.w_up, ew3.w_down)]
    t_un, t_ld, t_ld_pinned, t_ld_device = [], [], [], []
    for it in range(15):
        src = on_device if it >= 10 else pinned if it >= 5 else (ew3.w_gate, ew3.w_up, ew3.w_down)
        for _ in range(20):
            pool.moe_forward(0, x, aid, out)
        t0 = time.perf_counter()
        pool.unload_adapter(3)                       # waits for the 20 forwards, flips the map rows, unmaps
        t1 = time.perf_counter()
        for _ in range(20):
            pool.moe_forward(0, x, aid_wo3, out)
        t2 = time.perf_counter()
        pool.load_adapter(3, np.array([len(tuned[3][0])], np.int32), tuned[3][0], *src)
        t3 = time.perf_counter()
        t_un.append((t1 - t0) * 1e3)
        (t_ld_device if it >= 10 else t_ld_pinned if it >= 5 else t_ld).append((t3 - t2) * 1e3)
    torch.cuda.synchronize()
    res["churn"] = {"unload_ms_median": float(np.median(t_un)), "load_ms_median": float(np.median(t_ld)),
                    "load_ms_median_pinned_source": float(np.median(t_ld_pinned)),
                    "load_ms_median_device_source": float(np.median(t_ld_device)),
                    "adapter_bytes": int(ew3.w_gate.nbytes * 3), "forwards_in_flight": 20,
                    "pages_created_during_churn": pool.stats()["pages_created_total"] - created0,
                    "device_error": pool.last_device_error()}

    res["page_size_sweep"] = page_size_sweep(gpu=True)

    # ---- batch-size sweep on a pool sized for 8192 tokens
    big = binding.Pool.from_config(cfg, max_tokens=8192)
    binding.load_model(big, cfg, bank)
    rng = np.random.default_rng(0)
    sweep = []
    for B in (1, 4, 16, 64, 128, 256, 512, 1024, 2048, 4096, 8192):
        xb = torch.from_numpy(wl.f32_to_bf16_bits(rng.standard_normal((B, cfg.hidden)).astype(np.float32)).view(np.int16)).cuda().view(torch.bfloat16)
        ab = torch.from_numpy(rng.integers(-1, cfg.max_adapters, size=B).astype(np.int32)).cuda()
        ob = torch.empty_like(xb)
        dd = big.moe_forward_debug(0, xb, ab)
        torch.cuda.synchronize()
        live_b = int((dd["counts"] > 0).sum()) + cfg.num_shared
        ms = _time(lambda: big.moe_forward(0, xb, ab, ob), min(args.steps, 200 if B <= 1024 else 50), torch)
        gb = live_b * 3 * cfg.inter * cfg.hidden * 2 / 1e9
        fl = (B * cfg.top_k + cfg.num_shared * B) * 6 * cfg.inter * cfg.hidden / 1e12
        sweep.append({"tokens": B, "ms": ms, "tokens_per_s": B / ms * 1e3, "live_experts": live_b,
                      "weight_stream_TBps": gb / ms, "TFLOPps": fl / ms * 1e3})
    big.destroy()
    res["batch_sweep"] = sweep

    # ---- stand-alone operator vs unfused tensor ops, at the decode batch and at 65536 tokens
    pi_dev = torch.from_numpy(pool.get_expert_map(0)).cuda()
    for B in (cfg.n_tokens, 65536):
        g = torch.Generator(device="cuda").manual_seed(7)
        ids = torch.topk(torch.randn((B, cfg.num_experts), device="cuda", generator=g), cfg.top_k, dim=1).indices.to(torch.int32)
        a = torch.randint(-1, cfg.max_adapters, (B,), device="cuda", generator=g, dtype=torch.int32)
        slots = torch.empty_like(ids)
        counts = torch.empty(pool.num_slots, dtype=torch.int32, device="cuda")

        def unfused():
            a_b = a.to(torch.int64).unsqueeze(1).expand(-1, cfg.top_k)              # broadcast the adapter ids
            off = a_b.clamp(min=0) * cfg.num_experts + ids.to(torch.int64)           # offsets into the map
            red = pi_dev.reshape(-1).gather(0, off.reshape(-1)).reshape(B, cfg.top_k)   # gather
            return torch.where(a_b < 0, ids, red)

        want = unfused()
        pool.reroute(0, ids, a, slot_ids=slots, counts=counts)
        torch.cuda.synchronize()
        assert torch.equal(want, slots), (B, int((want != slots).sum()), pool.last_device_error())
        res["reroute"][f"B={B}"] = {
            "operator_ms": _time(lambda: pool.reroute(0, ids, a, slot_ids=slots, counts=counts), args.steps, torch),
            "operator_no_counts_ms": _time(lambda: pool.reroute(0, ids, a, slot_ids=slots, want_counts=False), args.steps, torch),
            "unfused_tensor_ops_ms": _time(unfused, args.steps, torch)}
    pool.destroy()

    # ---- padding baseline: the whole [M + N*E_max + S] tensor is physically backed
    pad = binding.Pool.from_config(cfg, pool_mode=1)
    binding.load_model(pad, cfg, bank)
    t_pad = _time(lambda: pad.moe_forward(0, x, aid, out), args.steps, torch)
    st_pad = pad.stats()
    pad.destroy()
    res["vmm_vs_padding"] = {"ms_vmm": t_mixed, "ms_padding": t_pad, "latency_delta": t_mixed / t_pad - 1.0,
                             "physical_bytes_vmm": st_vmm["physical_bytes"], "physical_bytes_padding": st_pad["physical_bytes"],
                             "physical_bytes_base_only": st_base["physical_bytes"],
                             "adapter_bytes_vmm": st_vmm["physical_bytes"] - st_base["physical_bytes"],
                             "adapter_bytes_padding": st_pad["physical_bytes"] - st_base["physical_bytes"]}
    res["memory_table1_shapes"] = memory_table1_shapes()
    print(json.dumps(res))


if __name__ == "__main__":
    main()
