"""Soak test of the forward path: many batch sizes (every token-tile class, ragged tails) in random order on two
streams with no host synchronisation in between, and an adapter evicted and re-loaded while forwards are in flight.
The forward is deterministic, so every output must be bit-identical to the one computed for the same batch in
isolation; a read that overtook its producer, a workspace shared by two forwards or a stale table would show up as a
mismatch."""
import numpy as np
import pytest

from paper_2508_17624_b200 import binding, build, workloads as wl

pytestmark = pytest.mark.gpu


def test_random_sizes_two_streams_and_churn():
    import torch
    build.build()
    cfg = wl.CONFIGS["c1"]
    bank = wl.NoiseBank(cfg.seed)
    pool = binding.Pool.from_config(cfg, max_tokens=8192)
    binding.load_model(pool, cfg, bank)
    tuned = wl.tuned_sets(cfg)
    last = cfg.max_adapters - 1
    ew_last = wl.gen_adapter_layer(cfg, last, 0, tuned[last][0], bank)
    rng = np.random.default_rng(123)
    sizes = [1, 2, 7, 31, 64, 65, 200, 256, 300, 511, 777, 1024, 1500, 2048, 3000, 4096, 5000, 8192]

    def batch(n, with_last):
        x = wl.f32_to_bf16_bits(rng.standard_normal((n, cfg.hidden)).astype(np.float32))
        aid = rng.integers(-1, cfg.max_adapters if with_last else last, size=n).astype(np.int32)
        return (torch.from_numpy(x.view(np.int16)).cuda().view(torch.bfloat16), torch.from_numpy(aid).cuda())

    sets = {w: [batch(n, w) for n in sizes] for w in (True, False)}       # with / without tokens of the last adapter
    refs = {}
    for w in (True, False):
        refs[w] = []
        for x, aid in sets[w]:
            refs[w].append(pool.moe_forward(0, x, aid).clone())
            torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    loaded = True
    for it in range(48):
        outs = []
        for j, i in enumerate(rng.integers(0, len(sizes), size=24)):
            x, aid = sets[loaded][i]
            out = torch.empty_like(x)
            with torch.cuda.stream(streams[j % 2]):
                pool.moe_forward(0, x, aid, out)
            outs.append((int(i), out))
        if it % 6 == 3:                        # churn with the 24 forwards above still queued
            if loaded:
                pool.unload_adapter(last)      # waits for them: they complete with the adapter in place
            else:
                pool.load_adapter(last, np.array([len(tuned[last][0])], np.int32), tuned[last][0], ew_last.w_gate,
                                  ew_last.w_up, ew_last.w_down)
        torch.cuda.synchronize()
        for i, out in outs:
            assert torch.equal(out, refs[loaded][i]), (it, sizes[i])
        if it % 6 == 3:
            loaded = not loaded
    assert pool.last_device_error() == 0
    pool.destroy()
