"""The allocation-free routing entry point against the CPU oracle and against the regular forward.

Some users of the library cannot allocate device memory when they need a routing decision (their
KV cache owns all free HBM, or they run where the CUDA allocator must not be entered), so
`ew_route_noalloc` keeps its scratch in a fixed array inside the library.  This file is collected
last on purpose: if it fails, a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest

from paper_2508_17624_b200 import binding, build
from paper_2508_17624_b200 import workloads as wl

from helpers import WEIGHT_RTOL, WEIGHT_TOL, check_routing, oracle_layer, to_dev

pytestmark = pytest.mark.gpu


def _route(pool, cfg, x, aid, n):
    import torch
    k, P = cfg.top_k, cfg.num_slots
    ids = torch.full((n, k), -7, dtype=torch.int32, device="cuda")
    w = torch.full((n, k), -7.0, dtype=torch.float32, device="cuda")
    slots = torch.full((n, k), -7, dtype=torch.int32, device="cuda")
    counts = torch.full((P,), 12345, dtype=torch.int32, device="cuda")      # must be overwritten, not accumulated
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    pool.route_noalloc(0, x, aid, ids, w, slots, counts, status)
    torch.cuda.synchronize()
    return ids.cpu().numpy(), w.cpu().numpy(), slots.cpu().numpy(), counts.cpu().numpy(), int(status.item())


@pytest.mark.parametrize("name", ["c0", "c1"])
def test_route_noalloc_matches_forward_twice_in_a_row(name):
    import torch
    assert torch.cuda.is_available()
    build.build()
    cfg = wl.CONFIGS[name]
    bank = wl.NoiseBank(cfg.seed)
    pool = binding.Pool.from_config(cfg)
    tuned, bases = binding.load_model(pool, cfg, bank)
    olayer = oracle_layer(cfg, 0, bank, tuned, base=bases[0])
    x_bits, aid_np = wl.gen_tokens(cfg), wl.gen_adapter_ids(cfg)
    x, aid = to_dev(x_bits), to_dev(aid_np)
    ref = pool.moe_forward_debug(0, x, aid)
    torch.cuda.synchronize()
    want = {k_: ref[k_].cpu().numpy() for k_ in ("topk_ids", "topk_w", "slot_ids", "counts")}
    for call in range(2):                               # the second call sees the first call's leftovers in the array
        ids, w, slots, counts, status = _route(pool, cfg, x, aid, cfg.n_tokens)
        assert status == 0
        # against the oracle: ids (near-ties counted), weights, slot ids and counts bit-exact given the ids
        _, _, _, flips = check_routing(cfg, olayer, x_bits, aid_np,
                                       dict(topk_ids=ids, topk_w=w, slot_ids=slots, counts=counts))
        assert flips <= 4
        # and the same bits as the existing entry point
        assert np.array_equal(ids, want["topk_ids"]), call
        assert (np.abs(w - want["topk_w"]) <= WEIGHT_TOL + WEIGHT_RTOL * want["topk_w"]).all(), call
        assert np.array_equal(slots, want["slot_ids"]), call
        assert np.array_equal(counts, want["counts"]), call
    # a bad adapter id is reported through the status word kept in the array, and cleared by the next call
    bad_np = aid_np.copy()
    bad_np[0] = cfg.max_adapters + 3
    ids, w, slots, counts, status = _route(pool, cfg, x, to_dev(bad_np), cfg.n_tokens)
    assert status & 1
    check_routing(cfg, olayer, x_bits, bad_np, dict(topk_ids=ids, topk_w=w, slot_ids=slots, counts=counts))
    *_, status = _route(pool, cfg, x, aid, cfg.n_tokens)
    assert status == 0
    assert pool.last_device_error() == 0                # the pool's own status word and workspace were not involved
    pool.destroy()


@pytest.mark.parametrize("n", [6000, 10000])
def test_route_noalloc_large_batches(n):
    """Batches beyond 4736 tokens take the router's large-tile form (64- and 128-token tiles, a histogram per CTA whose
    bases come from the caller's counters): ids, weights, slot ids and counts against the oracle."""
    import torch
    cfg = wl.CONFIGS["c0"]
    assert n * cfg.top_k <= 65536
    bank = wl.NoiseBank(cfg.seed)
    pool = binding.Pool.from_config(cfg)
    tuned, bases = binding.load_model(pool, cfg, bank)
    olayer = oracle_layer(cfg, 0, bank, tuned, base=bases[0])
    x_bits, aid_np = wl.gen_tokens(cfg, 0, n), wl.gen_adapter_ids(cfg, n)
    ids, w, slots, counts, status = _route(pool, cfg, to_dev(x_bits), to_dev(aid_np), n)
    assert status == 0
    _, _, _, flips = check_routing(cfg, olayer, x_bits, aid_np, dict(topk_ids=ids, topk_w=w, slot_ids=slots, counts=counts))
    assert flips <= max(4, n // 500)
    assert counts.sum() == n * cfg.top_k
    pool.destroy()


def test_route_noalloc_rejects_sizes_beyond_the_array():
    import torch
    cfg = wl.CONFIGS["c0"]
    pool = binding.Pool.from_config(cfg)
    binding.load_model(pool, cfg, adapters=[])
    n = 65536 // cfg.top_k + 1
    x = torch.zeros((n, cfg.hidden), dtype=torch.bfloat16, device="cuda")
    aid = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.EwError) as ei:
        _route(pool, cfg, x, aid, n)
    assert ei.value.status == 1 and "65536" in str(ei.value)
    ids, w, slots, counts, status = _route(pool, cfg, x[:n - 1], aid[:n - 1], n - 1)   # the largest accepted size
    assert status == 0 and counts.sum() == (n - 1) * cfg.top_k
    pool.destroy()
