"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest

import oracle
from paper_2508_17624_b200 import binding, build
from paper_2508_17624_b200 import workloads as wl

from helpers import WEIGHT_RTOL, bf16_to_f32, check_output, check_routing, oracle_layer, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    build.build()
    binding.lib()


def edge_tokens(r, n_extra, seed):
    """Tokens that own the first and the last row of every live slot's chunk (so that every slot's first and last
    token block, ragged tails included, is compared), plus `n_extra` seeded random ones."""
    inv = r["inv"].cpu().numpy()
    off = r["offsets"].cpu().numpy()
    B, k = inv.shape
    row_tok = np.empty(B * k, np.int64)
    row_tok[inv.reshape(-1)] = np.repeat(np.arange(B), k)
    live = np.nonzero(off[1:] > off[:-1])[0]
    picks = set(row_tok[off[live]].tolist()) | set(row_tok[off[live + 1] - 1].tolist())
    picks |= set(np.random.default_rng(seed).choice(B, size=min(B, n_extra), replace=False).tolist())
    return np.array(sorted(picks))


def run_layer(cfg, layer=0, n_tokens=None, aid_mode=None, adapters=None, sample=None, pool=None, bank=None,
              tuned=None, bases=None, **pool_kw):
    """One debug forward against the oracle.  `sample`: None = the output of every token is compared; an index
    array; or a function of the debug results that returns one."""
    import torch
    bank = bank or wl.NoiseBank(cfg.seed)
    own = pool is None
    if own:
        pool = binding.Pool.from_config(cfg, max_tokens=n_tokens or cfg.n_tokens, **pool_kw)
        tuned, bases = binding.load_model(pool, cfg, bank, adapters=adapters)
    olayer = oracle_layer(cfg, layer, bank, tuned, base=(bases or {}).get(layer), adapters=adapters)
    x = wl.gen_tokens(cfg, layer, n_tokens)
    aid = wl.gen_adapter_ids(cfg, n_tokens, aid_mode)
    r = pool.moe_forward_debug(layer, to_dev(x), to_dev(aid))
    torch.cuda.synchronize()
    assert pool.last_device_error() == 0
    ids, w, slots, flips = check_routing(cfg, olayer, x, aid, r)
    if callable(sample):
        sample = sample(r)
    rel, mx = check_output(olayer, x, slots, w, bf16_to_f32(r["out"]), sample)
    # the plain entry point gives the same bits as the debug one
    out2 = pool.moe_forward(layer, to_dev(x), to_dev(aid))
    torch.cuda.synchronize()
    assert torch.equal(out2, r["out"])
    if own:
        pool.destroy()
    return dict(flips=flips, rel=rel, max_abs=mx, slots=slots, out=r["out"],
                n_checked=x.shape[0] if sample is None else len(sample))


def oracle_check(pool, cfg, olayer, x_bits, aid_np, out, layer=0):
    """`out` (a forward's result obtained some other way: another entry point, another stream, a graph replay) has
    the bits of a debug forward on the same inputs, and that forward matches the oracle stage by stage."""
    import torch
    r = pool.moe_forward_debug(layer, to_dev(x_bits), to_dev(aid_np))
    torch.cuda.synchronize()
    assert torch.equal(r["out"], out)
    ids, w, slots, _ = check_routing(cfg, olayer, x_bits, aid_np, r)
    check_output(olayer, x_bits, slots, w, bf16_to_f32(r["out"]))


def test_c0_tiny_layer():
    res = run_layer(wl.CONFIGS["c0"])
    assert res["flips"] <= 2
    assert (res["slots"] >= 16).any()


@pytest.mark.parametrize("n_tokens", [1, 7, 33, 64, 100])
def test_c0_ragged_token_counts(n_tokens):
    run_layer(wl.CONFIGS["c0"], n_tokens=n_tokens)


def test_c1_decode_layer():
    res = run_layer(wl.CONFIGS["c1"])
    print("c1", {k: v for k, v in res.items() if k in ("flips", "rel", "max_abs")})
    assert res["flips"] <= 4


def test_c1_base_only_equals_no_adapters():
    """All tokens base: adapters loaded or not, the output is the base model's."""
    import torch
    cfg = wl.CONFIGS["c1"]
    a = run_layer(cfg, aid_mode="base")
    b = run_layer(cfg, aid_mode="base", adapters=[])
    assert torch.equal(a["out"], b["out"])
    assert (a["slots"] < cfg.num_experts).all()


@pytest.mark.parametrize("name", ["c0", "c1"])
def test_padding_mode_pool(name):
    """The padding baseline of Section 3.1 (pool_mode = 1: the whole [M + N*E_max] tensor is backed by pages at
    creation): the same kernels give the oracle's result, bit-identical to the pool that maps pages on demand,
    while holding the full tensor's worth of pages."""
    import torch
    cfg = wl.CONFIGS[name]
    vmm = run_layer(cfg)
    pad = run_layer(cfg, pool_mode=1)
    assert torch.equal(vmm["out"], pad["out"]) and np.array_equal(vmm["slots"], pad["slots"])
    pools = {m: binding.Pool.from_config(cfg, pool_mode=m) for m in (0, 1)}
    for pool in pools.values():
        binding.load_model(pool, cfg, adapters=[0])          # one adapter: most of the adapter range is padding
    st0, st1 = pools[0].stats(), pools[1].stats()
    assert st1["pages_mapped"] * st1["page_bytes"] >= st1["padding_bytes"]        # fully backed
    assert st0["pages_mapped"] <= st1["pages_mapped"] and (name == "c0" or st0["pages_mapped"] < 0.8 * st1["pages_mapped"])
    assert st0["physical_bytes"] - st0["live_expert_bytes"] <= 4 * st0["page_bytes"]   # page rounding only
    for pool in pools.values():
        pool.destroy()


def test_slot_address_reads_back_the_loaded_weights():
    """ew_slot_address: start_addr = base + slot * expert_size (Section 4.2); the bytes there are the expert's
    weights as loaded (gate block then up block in the fused tensor), for base, adapter and shared slots."""
    import torch
    from cuda.bindings import runtime as rt
    cfg = wl.CONFIGS["c0"]
    bank = wl.NoiseBank(cfg.seed)
    pool = binding.Pool.from_config(cfg)
    tuned, bases = binding.load_model(pool, cfg, bank)
    torch.cuda.synchronize()
    blk = cfg.inter * cfg.hidden            # elements per matrix

    def read(which, slot, n_elems):
        host = np.empty(n_elems, np.uint16)
        err, = rt.cudaMemcpy(host.ctypes.data, pool.slot_address(0, which, slot), n_elems * 2,
                             rt.cudaMemcpyKind.cudaMemcpyDeviceToHost)
        assert int(err) == 0
        return host

    base13, base2 = pool.slot_address(0, 0, 0), pool.slot_address(0, 1, 0)
    for slot in (0, 7, cfg.num_experts - 1):
        assert pool.slot_address(0, 0, slot) == base13 + slot * 2 * blk * 2
        assert pool.slot_address(0, 1, slot) == base2 + slot * blk * 2
        got = read(0, slot, 2 * blk)
        assert np.array_equal(got[:blk], bases[0].routed.w_gate[slot].reshape(-1))
        assert np.array_equal(got[blk:], bases[0].routed.w_up[slot].reshape(-1))
        assert np.array_equal(read(1, slot, blk), bases[0].routed.w_down[slot].reshape(-1))
    ew = wl.gen_adapter_layer(cfg, 1, 0, tuned[1][0], bank)
    slot = cfg.num_experts + 1 * cfg.e_max + 2                     # adapter 1, third tuned expert
    assert np.array_equal(read(0, slot, blk), ew.w_gate[2].reshape(-1))
    assert np.array_equal(read(1, slot, blk), ew.w_down[2].reshape(-1))
    shared = cfg.num_slots                                         # first shared expert sits behind the P routed slots
    assert np.array_equal(read(0, shared, blk), bases[0].shared.w_gate[0].reshape(-1))
    with pytest.raises(binding.EwError):
        pool.slot_address(0, 0, cfg.num_slots + cfg.num_shared)
    with pytest.raises(binding.EwError):
        pool.slot_address(0, 2, 0)
    pool.destroy()


@pytest.mark.parametrize("switch", ["EW_DISABLE_PDL", "EW_DISABLE_FAT", "EW_DISABLE_KSPLIT", "EW_DISABLE_SELFPLAN",
                                    "EW_DISABLE_TAIL_OVERLAP"])
def test_debugging_switches_in_a_fresh_process(switch):
    """The environment switches of the library (plain stream order instead of overlapped launches; every block on
    the weight-streaming kernel; no K split in the router; the planning kernel at every batch size; the CTA-pair kernel
    waiting for the weight-streaming kernel of its GEMM) are read once per process, so each is exercised in a process of its own: the
    tiny layer, the decode layer and a prefill-sized odd shape against the oracle."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, **{switch: "1"})
    here = os.path.dirname(os.path.abspath(__file__))
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", os.path.join(here, "test_gpu_parity.py"), "-k",
                        "test_c0_tiny_layer or test_c1_decode_layer or (test_odd_shapes and shape10)"],
                       env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "4 passed" in r.stdout, r.stdout[-500:]


def test_zero_tokens_and_errors():
    import torch
    cfg = wl.CONFIGS["c0"]
    pool = binding.Pool.from_config(cfg)
    x = torch.zeros((4, cfg.hidden), dtype=torch.bfloat16, device="cuda")
    aid = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.EwError) as ei:
        pool.moe_forward(0, x, aid)                     # base weights not loaded yet
    assert ei.value.status == 4
    binding.load_model(pool, cfg, adapters=[0])
    pool.moe_forward(0, x[:0], aid[:0])                 # n_tokens = 0 is a no-op
    with pytest.raises(binding.EwError):
        pool.moe_forward(0, torch.zeros((cfg.n_tokens + 1, cfg.hidden), dtype=torch.bfloat16, device="cuda"),
                         torch.zeros(cfg.n_tokens + 1, dtype=torch.int32, device="cuda"))
    pool.destroy()


def test_bad_and_unloaded_adapter_ids_against_the_oracle():
    """Adapter 1 is not loaded, 5 and 2^30 are past N, -7 is below -1: the oracle's reading makes all of them base
    tokens; the GPU must give the oracle's slots, counts and output for them and raise its flag."""
    import torch
    cfg = wl.CONFIGS["c0"]
    bank = wl.NoiseBank(cfg.seed)
    pool = binding.Pool.from_config(cfg)
    tuned, bases = binding.load_model(pool, cfg, bank, adapters=[0])
    olayer = oracle_layer(cfg, 0, bank, tuned, base=bases[0], adapters=[0])
    x = wl.gen_tokens(cfg)
    aid = np.resize(np.array([1, 5, -7, -1, 0, 2**30, 0, 1, -2**31, 0], np.int32), cfg.n_tokens)
    r = pool.moe_forward_debug(0, to_dev(x), to_dev(aid))
    torch.cuda.synchronize()
    assert pool.last_device_error() == 8
    ids, w, slots, _ = check_routing(cfg, olayer, x, aid, r)
    check_output(olayer, x, slots, w, bf16_to_f32(r["out"]))
    _, n_bad = oracle.reroute(ids, aid, olayer.build_map(), loaded=olayer.loaded, return_bad=True)
    assert n_bad == int(((aid != 0) & (aid != -1)).sum()) > 30
    assert (slots[aid == 0] >= cfg.num_experts).any() and (slots[aid != 0] < cfg.num_experts).all()
    good = pool.moe_forward(0, to_dev(x), to_dev(np.where(aid == 0, 0, -1).astype(np.int32)))
    torch.cuda.synchronize()
    assert pool.last_device_error() == 0
    assert torch.equal(r["out"], good)
    pool.destroy()


def test_load_unload_on_device():
    """Evicting an adapter returns its tokens to the base path; reloading restores the adapter path."""
    import torch
    cfg = wl.CONFIGS["c0"]
    bank = wl.NoiseBank(cfg.seed)
    pool = binding.Pool.from_config(cfg)
    tuned, bases = binding.load_model(pool, cfg, bank)
    x, aid = to_dev(wl.gen_tokens(cfg)), to_dev(wl.gen_adapter_ids(cfg))
    full = pool.moe_forward(0, x, aid).clone()
    st_full = pool.stats()
    pool.unload_adapter(1)
    aid_wo1 = torch.where(aid == 1, torch.full_like(aid, -1), aid)
    part = pool.moe_forward(0, x, aid_wo1).clone()
    torch.cuda.synchronize()
    assert pool.last_device_error() == 0
    changed = (aid == 1).cpu().numpy()
    same = torch.equal(part[~torch.from_numpy(changed).cuda()], full[~torch.from_numpy(changed).cuda()])
    assert same
    x_bits, aid_np = wl.gen_tokens(cfg), wl.gen_adapter_ids(cfg)
    oracle_check(pool, cfg, oracle_layer(cfg, 0, bank, tuned, base=bases[0], adapters=[0]), x_bits,
                 np.where(aid_np == 1, -1, aid_np).astype(np.int32), part)
    ew = wl.gen_adapter_layer(cfg, 1, 0, tuned[1][0], bank)
    pool.load_adapter(1, np.array([3], np.int32), tuned[1][0], ew.w_gate, ew.w_up, ew.w_down)
    again = pool.moe_forward(0, x, aid)
    torch.cuda.synchronize()
    assert torch.equal(again, full)
    oracle_check(pool, cfg, oracle_layer(cfg, 0, bank, tuned, base=bases[0]), x_bits, aid_np, again)
    assert pool.stats()["pages_mapped"] == st_full["pages_mapped"]
    pool.destroy()


def test_adapter_weights_from_device_memory():
    """ew_load_adapter takes its weights from device memory as well as from host memory: same forward either way."""
    import torch
    cfg = wl.CONFIGS["c0"]
    bank = wl.NoiseBank(cfg.seed)
    pool = binding.Pool.from_config(cfg)
    binding.load_model(pool, cfg, bank)
    x, aid = to_dev(wl.gen_tokens(cfg)), to_dev(wl.gen_adapter_ids(cfg))
    ref = pool.moe_forward(0, x, aid).clone()
    torch.cuda.synchronize()
    tuned = wl.tuned_sets(cfg)
    ew = wl.gen_adapter_layer(cfg, 1, 0, tuned[1][0], bank)
    pool.unload_adapter(1)
    dev = [torch.from_numpy(a.view(np.int16)).cuda() for a in (ew.w_gate, ew.w_up, ew.w_down)]
    pool.load_adapter(1, np.array([len(tuned[1][0])], np.int32), tuned[1][0], *dev)
    out = pool.moe_forward(0, x, aid)
    torch.cuda.synchronize()
    assert torch.equal(out, ref)
    oracle_check(pool, cfg, oracle_layer(cfg, 0, bank, tuned), wl.gen_tokens(cfg), wl.gen_adapter_ids(cfg), out)
    pool.destroy()


def test_reroute_operator_c4_sample():
    """The rerouting operator alone: slot ids and per-slot counts are bit-exact."""
    import torch
    cfg = wl.with_(wl.CONFIGS["c4"], n_tokens=4099)      # several tiles and a ragged tail
    oc = oracle.OracleConfig(cfg.hidden, cfg.inter, cfg.num_experts, 0, cfg.top_k, cfg.max_adapters, cfg.e_max)
    ids, _, _ = oracle.topk_from_logits(oc, wl.gen_logits(cfg))
    aid = wl.gen_adapter_ids(cfg, mode="uniform")
    pool = binding.Pool(hidden=64, inter=64, num_experts=cfg.num_experts, num_shared=0, top_k=cfg.top_k,
                        max_adapters=cfg.max_adapters, e_max=cfg.e_max, max_tokens=8)
    z = np.zeros((cfg.num_experts, 64, 64), np.uint16)
    pool.load_base(0, np.zeros((cfg.num_experts, 64), np.uint16), z, z, z)
    counts = np.array([16], np.int32)
    tuned = wl.tuned_sets(cfg, np.full((cfg.max_adapters, 1), 16))
    for i in range(cfg.max_adapters):
        za = np.zeros((16, 64, 64), np.uint16)
        pool.load_adapter(i, counts, tuned[i][0], za, za, za)
    Pi = oracle.build_map(cfg.num_experts, cfg.max_adapters, cfg.e_max, [t[0] for t in tuned])
    assert np.array_equal(pool.get_expert_map(0), Pi)
    slots, cnt = pool.reroute(0, to_dev(ids), to_dev(aid))
    torch.cuda.synchronize()
    want = oracle.reroute(ids, aid, Pi)
    assert np.array_equal(slots.cpu().numpy(), want)
    assert np.array_equal(cnt.cpu().numpy(), oracle.counts(want, cfg.num_slots))
    assert pool.last_device_error() == 0
    # buffers that are not 16-byte aligned (views starting one row in) take the generic kernel
    big_ids = torch.zeros((ids.shape[0] + 1, cfg.top_k), dtype=torch.int32, device="cuda")
    big_ids[1:] = to_dev(ids)
    big_aid = torch.zeros(aid.shape[0] + 1, dtype=torch.int32, device="cuda")
    big_aid[1:] = to_dev(aid)
    assert big_ids[1:].data_ptr() % 16 != 0
    slots2, cnt2 = pool.reroute(0, big_ids[1:], big_aid[1:])
    torch.cuda.synchronize()
    assert np.array_equal(slots2.cpu().numpy(), want) and torch.equal(cnt2, cnt)
    # ids outside [0, M) pass through unchanged and raise the flag; bad adapter ids act as base tokens
    bad_ids = to_dev(ids).clone()
    bad_ids[5, 2] = cfg.num_experts + 7
    bad_aid = to_dev(aid).clone()
    bad_aid[9] = cfg.max_adapters
    slots3, _ = pool.reroute(0, bad_ids, bad_aid)
    torch.cuda.synchronize()
    assert int(slots3[5, 2]) == cfg.num_experts + 7
    assert torch.equal(slots3[9], bad_ids[9])
    assert pool.last_device_error() in (1, 8)
    # bad adapter ids against the oracle's reading (base tokens), with counts; adapter 3 evicted = not loaded
    pool.unload_adapter(3)
    loaded = np.ones(cfg.max_adapters, np.int32)
    loaded[3] = 0
    aid4 = aid.copy()
    aid4[[0, 17, 4098]] = [cfg.max_adapters, -5, 2**30]
    Pi4 = pool.get_expert_map(0)
    assert np.array_equal(Pi4[3], np.arange(cfg.num_experts))
    slots4, cnt4 = pool.reroute(0, to_dev(ids), to_dev(aid4))
    torch.cuda.synchronize()
    want4, n_bad = oracle.reroute(ids, aid4, Pi, loaded=loaded, return_bad=True)     # Pi: the stale map, row 3 included
    assert n_bad == 3 + int((aid4 == 3).sum())
    assert np.array_equal(slots4.cpu().numpy(), want4)
    assert np.array_equal(cnt4.cpu().numpy(), oracle.counts(want4, cfg.num_slots))
    assert pool.last_device_error() == 8
    slots5, cnt5 = pool.reroute_unfused(0, to_dev(ids), to_dev(aid4))
    torch.cuda.synchronize()
    assert np.array_equal(slots5.cpu().numpy(), want4) and np.array_equal(cnt5.cpu().numpy(), cnt4.cpu().numpy())
    assert pool.last_device_error() == 8
    # in place, on a batch whose pair count is not a multiple of four (vector body + scalar tail on the same buffer)
    n_odd = 4097
    assert (n_odd * cfg.top_k) % 4 != 0
    buf = to_dev(ids[:n_odd]).clone()
    pool.reroute(0, buf, to_dev(aid4[:n_odd]), slot_ids=buf, want_counts=False)
    torch.cuda.synchronize()
    assert np.array_equal(buf.cpu().numpy(), want4[:n_odd])
    assert pool.last_device_error() == 8
    pool.destroy()


@pytest.mark.parametrize("M,k,n,renorm,quant", [(64, 6, 65536, 0, 0), (64, 6, 4099, 1, 0), (16, 2, 130, 0, 0), (80, 3, 1000, 0, 0),
                                                (256, 8, 777, 1, 0), (4, 4, 33, 0, 0), (64, 16, 1000, 1, 0), (32, 32, 200, 0, 0),
                                                (64, 6, 3000, 0, 1), (48, 12, 500, 1, 1), (128, 6, 300, 0, 1)])
def test_route_from_logits(M, k, n, renorm, quant):
    """Softmax + top-k + rerouting + counts from given fp32 logits (the c4 recipe: N(0,1) logits, adapter ids per
    token; also k > 8, k = M, and logits with many exact ties): ids equal the oracle's except where the k-th and
    (k+1)-th probabilities are within rounding of each other,
    weights to 2e-6 relative (same logits, different summation order), slots and counts bit-exact given the ids."""
    import torch
    N, e_max = 5, 3
    rng = np.random.default_rng(100 + M + k)
    logits = rng.standard_normal((n, M)).astype(np.float32)
    if quant:                  # logits on a grid of 0.5: many exact ties, inside a lane's experts and between lanes
        logits = (np.round(logits * 2) / 2).astype(np.float32)
    aid = rng.integers(-1, N, size=n).astype(np.int32)
    scale = 1.5 if renorm else 1.0
    pool = binding.Pool(hidden=64, inter=64, num_experts=M, num_shared=0, top_k=k, max_adapters=N, e_max=e_max,
                        max_tokens=8, renormalize=renorm, routed_scale=scale)
    z = np.zeros((M, 64, 64), np.uint16)
    pool.load_base(0, np.zeros((M, 64), np.uint16), z, z, z)
    tuned = [np.sort(rng.choice(M, size=min(e_max, M), replace=False)).astype(np.int32) for _ in range(N - 1)]
    for i, ts in enumerate(tuned):                       # the last adapter stays unloaded
        za = np.zeros((len(ts), 64, 64), np.uint16)
        pool.load_adapter(i, np.array([len(ts)], np.int32), ts, za, za, za)
    aid_loaded = np.where(aid == N - 1, -1, aid).astype(np.int32)
    oc = oracle.OracleConfig(64, 64, M, 0, k, N, e_max)
    oc.renormalize, oc.routed_scale = renorm, scale
    ids_o, w_o, gap = oracle.topk_from_logits(oc, logits)
    Pi = oracle.build_map(M, N, e_max, tuned + [np.zeros(0, np.int32)])
    ids, w, slots, cnt = pool.route_logits(0, to_dev(logits), to_dev(aid_loaded))
    torch.cuda.synchronize()
    assert pool.last_device_error() == 0
    ids, w, slots, cnt = ids.cpu().numpy(), w.cpu().numpy(), slots.cpu().numpy(), cnt.cpu().numpy()
    same = (ids == ids_o).all(axis=1)
    if quant:                  # equal logits give equal probabilities on both sides: the tie rule decides, exactly
        assert same.all(), "ties must go to the lower expert index, in the oracle's order"
    assert np.all(gap[~same] < 1e-6), "a routing decision differs where the probabilities are not tied"
    assert (~same).sum() <= max(1, n // 1000)
    assert np.allclose(w[same], w_o[same], rtol=2e-6, atol=1e-9)
    assert np.array_equal(slots, oracle.reroute(ids, aid_loaded, Pi))
    assert np.array_equal(cnt, oracle.counts(slots, M + N * e_max))
    # an unloaded adapter's id behaves as -1 and raises the error word; so does an id out of range
    aid_bad = aid.copy()
    aid_bad[0] = N + 3
    ids2, w2, slots2, cnt2 = pool.route_logits(0, to_dev(logits), to_dev(aid_bad))
    torch.cuda.synchronize()
    assert pool.last_device_error() in (1, 8)
    assert np.array_equal(ids2.cpu().numpy(), ids)
    loaded = np.ones(N, np.int32)
    loaded[N - 1] = 0
    want2, n_bad = oracle.reroute(ids, aid_bad, Pi, loaded=loaded, return_bad=True)
    assert n_bad == int(((aid_bad == N - 1) | (aid_bad == N + 3)).sum()) > 0
    assert np.array_equal(slots2.cpu().numpy(), want2)
    assert np.array_equal(cnt2.cpu().numpy(), oracle.counts(want2, M + N * e_max))
    # empty batch: counts zeroed, nothing else touched
    e_ids, e_w, e_slots, e_cnt = pool.route_logits(0, to_dev(logits[:0]), to_dev(aid[:0]))
    torch.cuda.synchronize()
    assert int(e_cnt.sum()) == 0
    # logits that are not 16-byte aligned are refused
    if M % 4 == 0 and n > 1:
        shifted = torch.zeros(n * M + 1, dtype=torch.float32, device="cuda")[1:].view(n, M)
        with pytest.raises(binding.EwError):
            pool.route_logits(0, shifted, to_dev(aid_loaded))
    pool.destroy()


def test_c2_prefill_layer():
    """8192 tokens, 20 adapters: routing and the layer output are checked for every token."""
    cfg = wl.CONFIGS["c2"]
    res = run_layer(cfg)
    assert res["n_checked"] == cfg.n_tokens
    print("c2", {k: v for k, v in res.items() if k in ("flips", "rel", "max_abs", "n_checked")})
    assert res["flips"] <= 40
    counts = np.bincount(res["slots"].reshape(-1), minlength=cfg.num_slots)
    assert counts[:cfg.num_experts].min() > 256            # base slots are fat (several token blocks) ...
    assert ((counts[cfg.num_experts:] > 0) & (counts[cfg.num_experts:] < 256)).any()   # ... adapter slots thin


def test_c4_reroute_full_size():
    """65536 tokens, 20 adapters re-tuning 10 %, 25 % and 50 % of the experts: ids and counts bit-exact."""
    import torch
    cfg = wl.CONFIGS["c4"]
    oc = oracle.OracleConfig(cfg.hidden, cfg.inter, cfg.num_experts, 0, cfg.top_k, cfg.max_adapters, cfg.e_max)
    ids, _, _ = oracle.topk_from_logits(oc, wl.gen_logits(cfg))
    aid = wl.gen_adapter_ids(cfg, mode="uniform")
    assert set(np.unique(aid)) == set(range(-1, cfg.max_adapters))
    pool = binding.Pool(hidden=64, inter=64, num_experts=cfg.num_experts, num_shared=0, top_k=cfg.top_k,
                        max_adapters=cfg.max_adapters, e_max=cfg.e_max, max_tokens=8)
    z = np.zeros((cfg.num_experts, 64, 64), np.uint16)
    pool.load_base(0, np.zeros((cfg.num_experts, 64), np.uint16), z, z, z)
    d_ids, d_aid = to_dev(ids), to_dev(aid)
    for e in (6, 16, 32):
        tuned = wl.tuned_sets(cfg, np.full((cfg.max_adapters, 1), e))
        za = np.zeros((e, 64, 64), np.uint16)
        for i in range(cfg.max_adapters):
            pool.load_adapter(i, np.array([e], np.int32), tuned[i][0], za, za, za)
        Pi = oracle.build_map(cfg.num_experts, cfg.max_adapters, cfg.e_max, [t[0] for t in tuned])
        slots, cnt = pool.reroute(0, d_ids, d_aid)
        torch.cuda.synchronize()
        want = oracle.reroute(ids, aid, Pi)
        assert np.array_equal(slots.cpu().numpy(), want)
        assert np.array_equal(cnt.cpu().numpy(), oracle.counts(want, cfg.num_slots))
        redirected = float((want >= cfg.num_experts).mean())
        assert abs(redirected - (e / 64) * 20 / 21) < 0.02      # tuned fraction x share of non-base tokens
        # in place (slot_ids aliasing topk_ids) gives the same result
        buf = d_ids.clone()
        pool.reroute(0, buf, d_aid, slot_ids=buf, want_counts=False)
        torch.cuda.synchronize()
        assert np.array_equal(buf.cpu().numpy(), want)
        # the unfused formulation (one kernel per tensor operation) gives the oracle's result as well
        slots_u, cnt_u = pool.reroute_unfused(0, d_ids, d_aid)
        torch.cuda.synchronize()
        assert np.array_equal(slots_u.cpu().numpy(), want)
        assert np.array_equal(cnt_u.cpu().numpy(), oracle.counts(want, cfg.num_slots))
        buf = d_ids.clone()
        pool.reroute_unfused(0, buf, d_aid, slot_ids=buf, want_counts=False)
        torch.cuda.synchronize()
        assert np.array_equal(buf.cpu().numpy(), want)
        for i in range(cfg.max_adapters):
            pool.unload_adapter(i)
    assert pool.last_device_error() == 0
    pool.destroy()


def test_c3_stacked_layers():
    """26 layers of the decode shape resident in one pool through the virtual weight tensors (fewer layers
    if the device has less free memory), 20 adapters, Zipf adapter popularity.  Every layer is checked against the
    oracle: routing for all 1024 tokens, the output for the tokens that own the first and the last row of every
    live slot plus 160 random ones (about 450 tokens per layer)."""
    import torch
    cfg = wl.CONFIGS["c3"]
    per_layer = (66 + 20 * 9) * 3 * cfg.inter * cfg.hidden * 2
    free, _ = torch.cuda.mem_get_info()
    L = int(min(cfg.num_layers, max(2, (free - (12 << 30)) // per_layer)))
    cfg = wl.with_(cfg, num_layers=L)
    print(f"c3: {L} layers resident")
    bank = wl.NoiseBank(cfg.seed)
    pool = binding.Pool.from_config(cfg)
    tuned = wl.tuned_sets(cfg)
    for l in range(L):
        b = wl.gen_base_layer(cfg, l, bank)
        pool.load_base(l, b.router_w, b.routed.w_gate, b.routed.w_up, b.routed.w_down,
                       b.shared.w_gate, b.shared.w_up, b.shared.w_down)
        del b
    for i in range(cfg.max_adapters):
        per = [wl.gen_adapter_layer(cfg, i, l, tuned[i][l], bank) for l in range(L)]
        pool.load_adapter(i, np.array([len(tuned[i][l]) for l in range(L)], np.int32),
                          np.concatenate([tuned[i][l] for l in range(L)]),
                          np.concatenate([e.w_gate for e in per]), np.concatenate([e.w_up for e in per]),
                          np.concatenate([e.w_down for e in per]))
        del per
    st = pool.stats()
    assert st["adapters_loaded"] == cfg.max_adapters
    assert st["physical_bytes"] < 0.90 * st["padding_bytes"]           # ~8 of the 10 reserved slots per adapter are live
    assert st["physical_bytes"] - st["live_expert_bytes"] < 0.02 * st["live_expert_bytes"]   # page rounding only
    aid = wl.gen_adapter_ids(cfg)
    assert aid.min() >= 0                                              # every token belongs to an adapter
    single = []
    for l in range(L):                   # the oracle's copy of a layer's weights is regenerated from the seed
        res = run_layer(cfg, layer=l, sample=lambda r, l=l: edge_tokens(r, 160, 300 + l), pool=pool, bank=bank,
                        tuned=tuned)
        assert res["n_checked"] >= 128
        single.append(res["out"].clone())
        if l in (0, L // 2, L - 1):
            print("c3 layer", l, {k: v for k, v in res.items() if k in ("flips", "rel", "max_abs", "n_checked")})
    # all layers back to back on one stream, each on its own input: the same bits as one at a time
    xs = [to_dev(wl.gen_tokens(cfg, l)) for l in range(L)]
    d_aid = to_dev(aid)
    outs = [pool.moe_forward(l, xs[l], d_aid) for l in range(L)]
    torch.cuda.synchronize()
    assert pool.last_device_error() == 0
    assert all(torch.equal(o, s_) for o, s_ in zip(outs, single))
    pool.destroy()


def test_bounded_wait_expires_and_reports():
    """A device-side wait that nothing satisfies gives up after its limit, raises the timeout bit and the
    kernel returns; the context stays usable (a forward right after is still correct)."""
    import torch
    cfg = wl.CONFIGS["c0"]
    pool = binding.Pool.from_config(cfg)
    binding.load_model(pool, cfg)
    x, aid = to_dev(wl.gen_tokens(cfg)), to_dev(wl.gen_adapter_ids(cfg))
    before = pool.moe_forward(0, x, aid).clone()
    pool.selftest_bounded_wait()
    assert pool.last_device_error() == 7          # EW_ERR_TIMEOUT, reported once
    assert pool.last_device_error() == 0
    after = pool.moe_forward(0, x, aid)
    torch.cuda.synchronize()
    assert torch.equal(before, after)
    pool.destroy()


def test_adapter_churn_under_load():
    """Adapters come and go while forwards are in flight (Section 4.2: pages are handed out at load time,
    returned on eviction and reused).  Small experts (192 KiB) make neighbouring adapters share 2 MiB pages at
    every alignment.  After every change the layer output is checked against the oracle for the adapters that
    are loaded at that moment."""
    import torch
    cfg = wl.with_(wl.CONFIGS["c0"], max_adapters=6, e_max=5, n_tokens=96, seed=11)
    bank = wl.NoiseBank(cfg.seed)
    rng = np.random.default_rng(11)
    pool = binding.Pool.from_config(cfg, prealloc_pages=2)
    base = wl.gen_base_layer(cfg, 0, bank)
    pool.load_base(0, base.router_w, base.routed.w_gate, base.routed.w_up, base.routed.w_down,
                   base.shared.w_gate, base.shared.w_up, base.shared.w_down)
    counts0 = rng.integers(1, cfg.e_max + 1, size=(cfg.max_adapters, 1))
    tuned = wl.tuned_sets(cfg, counts0)
    weights = {i: wl.gen_adapter_layer(cfg, i, 0, tuned[i][0], bank) for i in range(cfg.max_adapters)}
    x_bits = wl.gen_tokens(cfg)
    x = to_dev(x_bits)
    loaded = set()
    created = []
    for step in range(24):
        # keep the GPU busy with forwards of the current population, then change the population
        pop = sorted(loaded)
        aid_np = rng.choice([-1] + pop, size=cfg.n_tokens).astype(np.int32)
        aid = to_dev(aid_np)
        for _ in range(20):
            pool.moe_forward(0, x, aid)
        i = int(rng.integers(cfg.max_adapters))
        if i in loaded:
            pool.unload_adapter(i)                       # must wait for the forwards above, not fault
            loaded.discard(i)
        else:
            ew = weights[i]
            pool.load_adapter(i, np.array([len(tuned[i][0])], np.int32), tuned[i][0], ew.w_gate, ew.w_up, ew.w_down)
            loaded.add(i)
        created.append(pool.stats()["pages_created_total"])
        # the new population, checked against the oracle
        pop = sorted(loaded)
        aid_np = rng.choice([-1] + pop, size=cfg.n_tokens).astype(np.int32)
        r = pool.moe_forward_debug(0, x, to_dev(aid_np))
        torch.cuda.synchronize()
        assert pool.last_device_error() == 0, step
        olayer = oracle_layer(cfg, 0, bank, tuned, base=base, adapters=loaded)
        ids, w, slots, flips = check_routing(cfg, olayer, x_bits, aid_np, r)
        check_output(olayer, x_bits, slots, w, bf16_to_f32(r["out"]))
        # a token of an evicted adapter is served as a base token and flagged
        gone = [a for a in range(cfg.max_adapters) if a not in loaded]
        if gone:
            bad = aid_np.copy()
            bad[0] = gone[0]
            pool.moe_forward(0, x, to_dev(bad))
            torch.cuda.synchronize()
            assert pool.last_device_error() == 8
    st = pool.stats()
    assert st["pages_mapped"] + st["pages_free"] == st["pages_created_total"]
    assert created[-1] == max(created) and created[-1] <= created[len(created) // 2] + 1   # pages are reused, not re-created
    pool.destroy()


@pytest.mark.parametrize("shape", [
    dict(hidden=64, inter=8, num_experts=4, num_shared=0, top_k=1, max_adapters=1, e_max=1, n_tokens=5),      # smallest legal sizes
    dict(hidden=128, inter=200, num_experts=40, num_shared=1, top_k=5, max_adapters=3, e_max=4, n_tokens=77),  # I, M off the tile sizes
    dict(hidden=192, inter=136, num_experts=8, num_shared=2, top_k=8, max_adapters=2, e_max=8, n_tokens=40),   # k = M: dense mixture
    dict(hidden=256, inter=128, num_experts=80, num_shared=0, top_k=3, max_adapters=2, e_max=2, n_tokens=130), # M > 64: shared-memory softmax path
    dict(hidden=64, inter=64, num_experts=256, num_shared=1, top_k=4, max_adapters=1, e_max=3, n_tokens=33),   # the largest M
    dict(hidden=64, inter=64, num_experts=256, num_shared=0, top_k=2, max_adapters=20, e_max=1, n_tokens=70),  # expert map too large for shared memory
    dict(hidden=64, inter=64, num_experts=64, num_shared=1, top_k=32, max_adapters=2, e_max=4, n_tokens=50),    # the largest k
    dict(hidden=64, inter=64, num_experts=64, num_shared=1, top_k=32, max_adapters=2, e_max=4, n_tokens=600),   # and with prefill tiles
    dict(hidden=320, inter=96, num_experts=12, num_shared=1, top_k=3, max_adapters=2, e_max=2, n_tokens=40),   # router K split over 4 CTAs, 5 K-atoms: one CTA has none
    dict(hidden=576, inter=64, num_experts=24, num_shared=0, top_k=4, max_adapters=2, e_max=3, n_tokens=90),   # router K split over 8 CTAs, 9 K-atoms: ragged shares
    # prefill-sized batches (128-row gather tiles in GEMM-1, 256-row CTA-pair tiles in GEMM-2) on shapes off the tile sizes
    dict(hidden=128, inter=200, num_experts=8, num_shared=1, top_k=2, max_adapters=3, e_max=3, n_tokens=3001),  # H = one weight tile: half-empty tile pair
    dict(hidden=192, inter=72, num_experts=4, num_shared=0, top_k=4, max_adapters=2, e_max=4, n_tokens=1500),   # k = M, I < one tile
    dict(hidden=320, inter=264, num_experts=80, num_shared=2, top_k=3, max_adapters=4, e_max=5, n_tokens=5000), # M > 64 with 64-token router tiles
    dict(hidden=64, inter=64, num_experts=8, num_shared=1, top_k=2, max_adapters=2, e_max=2, n_tokens=12000),   # 128-token router tiles, 47 fat blocks per shared expert
])
@pytest.mark.parametrize("renorm", [0, 1])
def test_odd_shapes(shape, renorm):
    """Shapes off every tile size, degenerate top-k, no shared experts, renormalised and scaled weights."""
    check_shape(shape, renorm, seed=21)


def _random_shape(rng):
    M = int(rng.choice([2, 3, 5, 8, 12, 16, 24, 33, 48, 64, 72, 100]))
    return dict(hidden=64 * int(rng.integers(1, 7)), inter=8 * int(rng.integers(1, 40)), num_experts=M,
                num_shared=int(rng.integers(0, 3)), top_k=int(rng.integers(1, min(M, 8) + 1)),
                max_adapters=int(rng.integers(1, 5)), e_max=int(rng.integers(1, min(M, 5) + 1)),
                n_tokens=int(rng.choice([1, 3, 17, 32, 33, 63, 64, 100, 129, 257, 600, 1100])))


@pytest.mark.parametrize("case", range(32))
def test_random_shapes(case):
    """Seeded random layer shapes and batch sizes (sizes, expert counts, top-k, shared experts, adapters all drawn
    independently), each checked against the oracle like the hand-picked ones above."""
    rng = np.random.default_rng(1000 + case)
    check_shape(_random_shape(rng), renorm=case % 2, seed=1000 + case)


def check_shape(shape, renorm, seed):
    import torch
    cfg = wl.MoEConfig(name="odd", num_layers=1, seed=seed, **shape)
    bank = wl.NoiseBank(cfg.seed)
    rng = np.random.default_rng(seed)
    scale = 2.5 if renorm else 1.0
    pool = binding.Pool.from_config(cfg, renormalize=renorm, routed_scale=scale)
    counts = rng.integers(0, cfg.e_max + 1, size=(cfg.max_adapters, 1))
    counts[0, 0] = cfg.e_max
    tuned = wl.tuned_sets(cfg, counts)
    _, bases = binding.load_model(pool, cfg, bank, tuned=tuned)
    olayer = oracle_layer(cfg, 0, bank, tuned, base=bases[0])
    olayer.cfg.renormalize, olayer.cfg.routed_scale = renorm, scale
    x = wl.gen_tokens(cfg)
    x_scale = 1.0
    if cfg.num_experts > 64:      # spread the logits so that the 1e-5 near-tie window stays rare with many experts
        x_scale = 6.0
        x = wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(x) * x_scale)
    aid = wl.gen_adapter_ids(cfg, mode="uniform")
    # The absolute bound of 2e-2 is stated for outputs the size of the five workloads' (|y| < 4): the final rounding
    # to bf16 alone is half an ulp = 1.6e-2 for |y| in [4, 8) and 3.1e-2 beyond.  So the inputs are drawn to stay
    # there instead of the bound being stretched: while the oracle's output reaches 3.5 the activations are halved
    # (exact in bf16; decided by the oracle alone, before the GPU runs).
    for _ in range(8):
        ref_full, *_ = oracle.layer_forward(olayer, x, aid)
        if float(np.abs(ref_full).max()) < 3.5:
            break
        x = wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(x) * np.float32(0.5))
        x_scale *= 0.5
    assert float(np.abs(ref_full).max()) < 3.5
    r = pool.moe_forward_debug(0, to_dev(x), to_dev(aid))
    torch.cuda.synchronize()
    assert pool.last_device_error() == 0
    ids, w, slots, flips = check_routing(cfg, olayer, x, aid, r, weight_rtol=WEIGHT_RTOL * max(1.0, x_scale))
    assert flips <= max(2, cfg.n_tokens // 20)
    check_output(olayer, x, slots, w, bf16_to_f32(r["out"]))
    kernels = pool.stats()["last_forward_kernels"]
    pool.destroy()
    return kernels


def test_kernels_per_forward_and_the_planning_fallback():
    """Which form of the forward ran is reported by the pool: four kernels for a decode-sized batch (the GEMM kernels
    derive their own work items), seven for a prefill-sized one (planning kernel, two kernels per GEMM), and five - the
    planning kernel kept - for a decode-sized batch whose items a GEMM CTA could not hold in its shared memory: here
    704 slots x 32 weight tiles of GEMM-2 are up to 170 items per CTA.  Each against the oracle."""
    assert check_shape(dict(hidden=128, inter=200, num_experts=40, num_shared=1, top_k=5, max_adapters=3, e_max=4, n_tokens=77), 0, 5) == 4
    assert check_shape(dict(hidden=192, inter=72, num_experts=4, num_shared=0, top_k=4, max_adapters=2, e_max=4, n_tokens=1500), 0, 5) == 7
    assert check_shape(dict(hidden=4096, inter=64, num_experts=64, num_shared=2, top_k=8, max_adapters=20, e_max=32, n_tokens=1024), 0, 5) == 5


def test_c3_stack_throughput_report():
    """Timing of a 4-layer slice of the stacked configuration (1024 tokens per layer, 20 adapters, Zipf ids):
    layers back to back on one stream.  Reported, with a loose sanity bound (the per-layer weight stream is
    ~3.8 GB, so a layer cannot take less than 0.5 ms nor, on a healthy B200, more than 3 ms)."""
    import torch
    cfg = wl.with_(wl.CONFIGS["c3"], num_layers=4)
    bank = wl.NoiseBank(cfg.seed)
    pool = binding.Pool.from_config(cfg)
    binding.load_model(pool, cfg, bank)
    aid = to_dev(wl.gen_adapter_ids(cfg))
    xs = [to_dev(wl.gen_tokens(cfg, l)) for l in range(cfg.num_layers)]
    outs = [torch.empty_like(x) for x in xs]
    for _ in range(3):
        for l in range(cfg.num_layers):
            pool.moe_forward(l, xs[l], aid, outs[l])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    reps = 20
    for _ in range(reps):
        for l in range(cfg.num_layers):
            pool.moe_forward(l, xs[l], aid, outs[l])
    e1.record()
    torch.cuda.synchronize()
    ms_layer = e0.elapsed_time(e1) / (reps * cfg.num_layers)
    d = pool.moe_forward_debug(0, xs[0], aid)
    live = int((d["counts"] > 0).sum()) + cfg.num_shared
    gb = live * 3 * cfg.inter * cfg.hidden * 2 / 1e9
    print(f"c3: {ms_layer:.4f} ms per layer, {live} live experts, {gb:.2f} GB of weights per layer, "
          f"{gb / ms_layer:.2f} TB/s, {cfg.n_tokens / ms_layer / 26:.1f} k tokens/s through a 26-layer stack")
    assert 0.5 < ms_layer < 3.0
    pool.destroy()


def test_side_stream_and_cuda_graph():
    """The forward is asynchronous on the caller's stream: it runs on a side stream, and it can be captured
    into a CUDA graph (after a warm-up call) and replayed with the same bits as a direct call."""
    import torch
    cfg = wl.CONFIGS["c0"]
    pool = binding.Pool.from_config(cfg)
    binding.load_model(pool, cfg)
    x, aid = to_dev(wl.gen_tokens(cfg)), to_dev(wl.gen_adapter_ids(cfg))
    ref = pool.moe_forward(0, x, aid).clone()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    out = torch.empty_like(x)
    with torch.cuda.stream(side):
        pool.moe_forward(0, x, aid, out)
    side.synchronize()
    assert torch.equal(out, ref)
    g = torch.cuda.CUDAGraph()
    out2 = torch.zeros_like(x)
    with torch.cuda.graph(g):
        pool.moe_forward(0, x, aid, out2)
    for _ in range(3):
        out2.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out2, ref)
    assert pool.last_device_error() == 0
    # a direct call after the replays still works (the slot counters were left clean by the graph's last kernel)
    assert torch.equal(pool.moe_forward(0, x, aid), ref)
    pool.destroy()


def test_cuda_graph_of_a_prefill_sized_forward():
    """A prefill-sized batch (thin and fat item lists, CTA-pair kernels launched as clusters with programmatic
    dependent launch) captured into a CUDA graph after one warm-up call replays with the bits of a direct call."""
    import torch
    cfg = wl.MoEConfig(name="odd", num_layers=1, seed=31, hidden=192, inter=136, num_experts=6, num_shared=1, top_k=2,
                       max_adapters=8, e_max=2, n_tokens=2500)
    bank = wl.NoiseBank(cfg.seed)
    pool = binding.Pool.from_config(cfg)
    tuned = wl.tuned_sets(cfg, np.array([[2], [1], [2], [1], [2], [2], [1], [2]]))
    binding.load_model(pool, cfg, bank, tuned=tuned)
    x, aid = to_dev(wl.gen_tokens(cfg)), to_dev(wl.gen_adapter_ids(cfg, mode="uniform"))
    ref = pool.moe_forward(0, x, aid).clone()            # the warm-up call
    torch.cuda.synchronize()
    counts = pool.moe_forward_debug(0, x, aid)["counts"].cpu().numpy()
    assert counts.max() > 256 and ((counts > 0) & (counts <= 128)).any()      # both item lists are in play
    g = torch.cuda.CUDAGraph()
    out = torch.zeros_like(x)
    with torch.cuda.graph(g):
        pool.moe_forward(0, x, aid, out)
    for _ in range(3):
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, ref)
    assert torch.equal(pool.moe_forward(0, x, aid), ref)
    assert pool.last_device_error() == 0
    oracle_check(pool, cfg, oracle_layer(cfg, 0, bank, tuned), wl.gen_tokens(cfg), wl.gen_adapter_ids(cfg, mode="uniform"), out)
    pool.destroy()


def test_two_pools_on_one_device():
    import torch
    c0, c1 = wl.CONFIGS["c0"], wl.with_(wl.CONFIGS["c0"], seed=5, max_adapters=1)
    pa, pb = binding.Pool.from_config(c0), binding.Pool.from_config(c1)
    binding.load_model(pa, c0)
    binding.load_model(pb, c1)
    xa, xb = to_dev(wl.gen_tokens(c0)), to_dev(wl.gen_tokens(c1))
    aa, ab = to_dev(wl.gen_adapter_ids(c0)), to_dev(wl.gen_adapter_ids(c1))
    ra, rb = pa.moe_forward(0, xa, aa).clone(), pb.moe_forward(0, xb, ab).clone()
    for _ in range(5):                               # interleaved calls do not disturb each other's workspaces
        oa, ob = pa.moe_forward(0, xa, aa), pb.moe_forward(0, xb, ab)
    torch.cuda.synchronize()
    assert torch.equal(oa, ra) and torch.equal(ob, rb) and not torch.equal(ra, rb)
    pa.destroy()
    pb.destroy()


@pytest.mark.parametrize("name", ["c0", "c1"])
def test_back_to_back_forwards_with_changing_inputs(name):
    """The kernels of consecutive forwards overlap their launches; with a different batch in every call any
    read that slipped ahead of its producer would pick up the previous batch's intermediate results."""
    import torch
    cfg = wl.CONFIGS[name]
    pool = binding.Pool.from_config(cfg)
    binding.load_model(pool, cfg)
    rng = np.random.default_rng(0)
    batches = []
    for i in range(6):
        n = cfg.n_tokens if i % 2 == 0 else max(1, cfg.n_tokens - 17 * i)
        x = wl.f32_to_bf16_bits(rng.standard_normal((n, cfg.hidden)).astype(np.float32))
        aid = rng.integers(-1, cfg.max_adapters, size=n).astype(np.int32)
        batches.append((to_dev(x), to_dev(aid)))
    ref = []
    for x, aid in batches:                      # one at a time, fully synchronised
        ref.append(pool.moe_forward(0, x, aid).clone())
        torch.cuda.synchronize()
    outs = [torch.empty_like(b[0]) for b in batches]
    busy = torch.empty(1 << 28, dtype=torch.uint8, device="cuda")
    for rep in range(6):
        busy.zero_()                            # keeps the GPU busy so that the following launches queue up densely
        order = rng.permutation(len(batches))
        for i in order:
            pool.moe_forward(0, batches[i][0], batches[i][1], outs[i])
        torch.cuda.synchronize()
        for i in range(len(batches)):
            assert torch.equal(outs[i], ref[i]), (rep, i)
            outs[i].zero_()
    assert pool.last_device_error() == 0
    pool.destroy()


def test_back_to_back_forwards_of_every_form_on_one_pool():
    """One pool, batches of very different sizes queued back to back without host synchronisation: each call picks its
    own form of the forward (four kernels for the decode-sized ones, seven for the prefill-sized ones) and leaves
    tables of the other forms behind in the shared workspace.  Every output against the oracle, and against the same
    call made alone."""
    import torch
    cfg = wl.CONFIGS["c0"]
    sizes = [7, 3000, 64, 1500, 256, 2999, 1, 640]
    bank = wl.NoiseBank(cfg.seed)
    pool = binding.Pool.from_config(cfg, max_tokens=max(sizes))
    tuned, bases = binding.load_model(pool, cfg, bank)
    olayer = oracle_layer(cfg, 0, bank, tuned, base=bases[0])
    rng = np.random.default_rng(11)
    batches, alone, forms = [], [], []
    for n in sizes:
        x = wl.f32_to_bf16_bits(rng.standard_normal((n, cfg.hidden)).astype(np.float32))
        aid = rng.integers(-1, cfg.max_adapters, size=n).astype(np.int32)
        r = pool.moe_forward_debug(0, to_dev(x), to_dev(aid))
        torch.cuda.synchronize()
        forms.append(pool.stats()["last_forward_kernels"])
        ids, w, slots, _ = check_routing(cfg, olayer, x, aid, r)
        check_output(olayer, x, slots, w, bf16_to_f32(r["out"]))
        batches.append((to_dev(x), to_dev(aid)))
        alone.append(r["out"].clone())
    assert 4 in forms and 7 in forms
    outs = [torch.empty_like(b[0]) for b in batches]
    busy = torch.empty(1 << 28, dtype=torch.uint8, device="cuda")
    for rep in range(4):
        busy.zero_()
        order = rng.permutation(len(batches))
        for i in order:
            pool.moe_forward(0, batches[i][0], batches[i][1], outs[i])
        torch.cuda.synchronize()
        for i in range(len(batches)):
            assert torch.equal(outs[i], alone[i]), (rep, i, sizes[i])
            outs[i].zero_()
    assert pool.last_device_error() == 0
    pool.destroy()


def test_forwards_on_two_streams_share_the_workspace_in_order():
    """One pool, two streams, no host synchronisation between the calls: the pool makes a forward wait for the one
    issued before it on the other stream, so the single workspace is never used by two forwards at once."""
    import torch
    cfg = wl.CONFIGS["c1"]
    pool = binding.Pool.from_config(cfg)
    binding.load_model(pool, cfg)
    rng = np.random.default_rng(5)
    batches = []
    for i in range(6):
        n = cfg.n_tokens - 13 * i
        x = wl.f32_to_bf16_bits(rng.standard_normal((n, cfg.hidden)).astype(np.float32))
        aid = rng.integers(-1, cfg.max_adapters, size=n).astype(np.int32)
        batches.append((to_dev(x), to_dev(aid)))
    ref = []
    for x, aid in batches:
        ref.append(pool.moe_forward(0, x, aid).clone())
        torch.cuda.synchronize()
    outs = [torch.empty_like(b[0]) for b in batches]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    busy = torch.empty(1 << 28, dtype=torch.uint8, device="cuda")
    for rep in range(4):
        torch.cuda.synchronize()
        for s in streams:
            with torch.cuda.stream(s):
                busy.zero_()                    # both streams start behind a long kernel: the launches queue up
        for i in range(len(batches)):
            with torch.cuda.stream(streams[i % 2]):
                pool.moe_forward(0, batches[i][0], batches[i][1], outs[i])
        torch.cuda.synchronize()
        for i in range(len(batches)):
            assert torch.equal(outs[i], ref[i]), (rep, i)
            outs[i].zero_()
    assert pool.last_device_error() == 0
    pool.destroy()


def test_many_short_lived_streams():
    """A caller that uses a fresh stream for every call: the pool's per-stream bookkeeping must stay bounded and the
    results must not change."""
    import torch
    cfg = wl.CONFIGS["c0"]
    pool = binding.Pool.from_config(cfg)
    binding.load_model(pool, cfg)
    x, aid = to_dev(wl.gen_tokens(cfg)), to_dev(wl.gen_adapter_ids(cfg))
    ref = pool.moe_forward(0, x, aid).clone()
    torch.cuda.synchronize()
    for i in range(100):
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            out = pool.moe_forward(0, x, aid)
        s.synchronize()
        assert torch.equal(out, ref), i
        del s
    pool.unload_adapter(0)                      # walks the bookkeeping of every stream still listed
    assert pool.last_device_error() == 0
    pool.destroy()


def test_host_buffer_pipeline():
    """ew_moe_forward_host overlaps upload, kernels and download across calls with double-buffered staging:
    different batches issued back to back (and mixed with direct device-side calls) give the direct results."""
    import torch
    cfg = wl.CONFIGS["c0"]
    pool = binding.Pool.from_config(cfg)
    binding.load_model(pool, cfg)
    rng = np.random.default_rng(3)
    host, ref = [], []
    for i in range(7):
        n = cfg.n_tokens - 5 * i
        xb = wl.f32_to_bf16_bits(rng.standard_normal((n, cfg.hidden)).astype(np.float32))
        ab = rng.integers(-1, cfg.max_adapters, size=n).astype(np.int32)
        xh = torch.from_numpy(xb.view(np.int16).copy()).pin_memory()
        ah = torch.from_numpy(ab.copy()).pin_memory()
        oh = torch.zeros((n, cfg.hidden), dtype=torch.int16).pin_memory()
        host.append((xh, ah, oh))
        ref.append(pool.moe_forward(0, to_dev(xb), to_dev(ab)).clone())
        torch.cuda.synchronize()
    xd, ad = to_dev(wl.gen_tokens(cfg)), to_dev(wl.gen_adapter_ids(cfg))
    direct_ref = pool.moe_forward(0, xd, ad).clone()
    torch.cuda.synchronize()
    for rep in range(3):
        for i, (xh, ah, oh) in enumerate(host):
            pool.moe_forward_host(0, xh, ah, oh)
            if i == 3:
                direct = pool.moe_forward(0, xd, ad)          # a device-side call in the middle of the pipeline
        torch.cuda.synchronize()
        assert torch.equal(direct, direct_ref)
        for (xh, ah, oh), r in zip(host, ref):
            assert torch.equal(oh.cuda().view(torch.bfloat16), r), rep
            if rep < 2:
                oh.zero_()
    assert pool.last_device_error() == 0
    # what arrived in the host buffer of the first batch is the oracle's layer output
    xh, ah, oh = host[0]
    bank = wl.NoiseBank(cfg.seed)
    oracle_check(pool, cfg, oracle_layer(cfg, 0, bank, wl.tuned_sets(cfg)), xh.numpy().view(np.uint16), ah.numpy(),
                 oh.cuda().view(torch.bfloat16))
    pool.destroy()


def test_token_tile_of_128_rows():
    """640 tokens on the decode-shaped layer give ~60 rows per expert: the 128-row token tile (the one size the
    five workloads do not reach) with its double-buffered accumulators and 128-row activation boxes."""
    cfg = wl.CONFIGS["c1"]
    sample = np.sort(np.random.default_rng(6).choice(640, size=96, replace=False))
    res = run_layer(cfg, n_tokens=640, sample=sample)
    counts = np.bincount(res["slots"].reshape(-1), minlength=cfg.num_slots)
    assert 64 < counts[:cfg.num_experts].max() <= 128
    assert res["flips"] <= 6
