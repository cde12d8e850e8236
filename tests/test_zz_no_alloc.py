"""The allocation-free routing entry point against the regular forward's routing results.

Some users of the library cannot allocate device memory when they need a routing decision (their
KV cache owns all free HBM, or they run where the CUDA allocator must not be entered), so
`ew_route_noalloc` keeps its scratch in a fixed array inside the library.  This file is collected
last on purpose: if it fails, a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest

from paper_2508_17624_b200 import binding, build
from paper_2508_17624_b200 import workloads as wl

from helpers import WEIGHT_RTOL, WEIGHT_TOL, to_dev

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
    pool = binding.Pool.from_config(cfg)
    binding.load_model(pool, cfg)
    x, aid = to_dev(wl.gen_tokens(cfg)), to_dev(wl.gen_adapter_ids(cfg))
    ref = pool.moe_forward_debug(0, x, aid)
    torch.cuda.synchronize()
    want = {k_: ref[k_].cpu().numpy() for k_ in ("topk_ids", "topk_w", "slot_ids", "counts")}
    for call in range(2):                               # the second call sees the first call's leftovers in the array
        ids, w, slots, counts, status = _route(pool, cfg, x, aid, cfg.n_tokens)
        assert status == 0
        assert np.array_equal(ids, want["topk_ids"]), call
        assert (np.abs(w - want["topk_w"]) <= WEIGHT_TOL + WEIGHT_RTOL * want["topk_w"]).all(), call
        assert np.array_equal(slots, want["slot_ids"]), call
        assert np.array_equal(counts, want["counts"]), call
    # a bad adapter id is reported through the status word kept in the array, and cleared by the next call
    bad = aid.clone()
    bad[0] = cfg.max_adapters + 3
    *_, status = _route(pool, cfg, x, bad, cfg.n_tokens)
    assert status & 1
    *_, status = _route(pool, cfg, x, aid, cfg.n_tokens)
    assert status == 0
    assert pool.last_device_error() == 0                # the pool's own status word and workspace were not involved
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
