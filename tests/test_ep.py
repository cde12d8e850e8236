"""Expert parallelism on CPU: the placement rule, the page accounting of a rank's pool (accounting backend), and the
exchange step with two gloo ranks whose stand-in pools compute their partial sums with the oracle."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2508_17624_b200 import binding, ep, workloads as wl  # noqa: E402
from helpers import oracle_layer, oracle_partial  # noqa: E402


def _load_accounting_only(pool, cfg):
    """The loads of binding.load_model without generating any weights (an accounting pool never reads them)."""
    tuned = wl.tuned_sets(cfg)
    for l in range(cfg.num_layers):
        pool.load_base(l, None, None, None, None)
    for i in range(cfg.max_adapters):
        counts = np.array([len(tuned[i][l]) for l in range(cfg.num_layers)], np.int32)
        ids = np.concatenate([tuned[i][l] for l in range(cfg.num_layers)]).astype(np.int32)
        pool.load_adapter(i, counts, ids, None, None, None)
    return tuned


@pytest.mark.parametrize("n,size", [(64, 1), (64, 2), (64, 8), (66, 4), (2, 8), (0, 3), (7, 7), (5, 2)])
def test_owned_ranges_partition_the_items(n, size):
    seen = []
    for r in range(size):
        lo, hi = ep.owned_range(n, size, r)
        assert 0 <= lo <= hi <= n
        seen += list(range(lo, hi))
        for j in range(lo, hi):
            assert ep.owner_of(j, n, size) == r
    assert seen == list(range(n))                      # disjoint, in rank order, complete
    sizes = [ep.owned_range(n, size, r)[1] - ep.owned_range(n, size, r)[0] for r in range(size)]
    assert max(sizes) == -(-n // size) if n else max(sizes) == 0


def test_a_rerouted_pair_stays_on_the_rank_of_its_base_expert():
    """Section 4.1's map sends base expert j to an adapter's copy of j; the library keeps that copy on j's rank, so the
    mask over base ids is also the mask over slots: every slot an adapter row maps j to is held where j is."""
    cfg = wl.CONFIGS["c0"]
    tuned = wl.tuned_sets(cfg)
    R = 2
    for r in range(R):
        pool = binding.Pool.from_config(cfg, device=-1, ep_size=R, ep_rank=r)
        _load_accounting_only(pool, cfg)
        lo, hi = ep.owned_range(cfg.num_experts, R, r)
        st = pool.stats()
        own_tuned = sum(int(((t >= lo) & (t < hi)).sum()) for i in range(cfg.max_adapters) for t in tuned[i])
        assert st["live_experts"] == cfg.num_layers * (hi - lo) + own_tuned
        Pi = pool.get_expert_map(0)
        full = oracle.build_map(cfg.num_experts, cfg.max_adapters, cfg.e_max, [tuned[i][0] for i in range(cfg.max_adapters)])
        assert np.array_equal(Pi, full)                # the map itself is the same on every rank
        pool.destroy()


def test_rank_pools_back_only_their_share():
    cfg = wl.CONFIGS["c1"]
    single = binding.Pool.from_config(cfg, device=-1)
    _load_accounting_only(single, cfg)
    s1 = single.stats()
    for R in (2, 4, 8):
        tot_live, tot_bytes, tot_pages = 0, 0, 0
        for r in range(R):
            pool = binding.Pool.from_config(cfg, device=-1, ep_size=R, ep_rank=r)
            _load_accounting_only(pool, cfg)
            st = pool.stats()
            tot_live += st["live_experts"]
            tot_bytes += st["live_expert_bytes"]
            tot_pages += st["pages_mapped"]
            assert st["pages_mapped"] <= s1["pages_mapped"] // R + 4 * 2 * cfg.num_layers * (cfg.max_adapters + 2)
            for i in range(cfg.max_adapters):           # eviction returns exactly what the adapter's share took
                pool.unload_adapter(i)
            lo, hi = ep.owned_range(cfg.num_experts, R, r)
            assert pool.stats()["live_experts"] == cfg.num_layers * (hi - lo)
            pool.destroy()
        assert tot_live == s1["live_experts"] and tot_bytes == s1["live_expert_bytes"]
        assert tot_pages >= s1["pages_mapped"]          # page rounding at the blocks' edges can only add
    with pytest.raises(binding.EwError):
        binding.Pool.from_config(cfg, device=-1, ep_size=2, ep_rank=2)
    single.destroy()


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


class _OraclePool:
    """Stand-in for a rank's pool on CPU: the partial sums come from the oracle, the rounding from torch."""

    def __init__(self, cfg, world, rank, n_tokens):
        self.cfg, self.world, self.rank = cfg, world, rank
        self.bank = wl.NoiseBank(cfg.seed)
        self.tuned = wl.tuned_sets(cfg)
        self.olayer = oracle_layer(cfg, 0, self.bank, self.tuned)

    def moe_forward_partial(self, layer, x, adapter_ids):
        xb = x.view(torch.int16).numpy().view(np.uint16)
        aid = adapter_ids.numpy()
        _, ids, w, slots = oracle.layer_forward(self.olayer, xb, aid)
        part = oracle_partial(self.cfg, layer, self.bank, self.tuned, xb, ids, slots, w, self.world, self.rank)
        return torch.from_numpy(part)

    def ep_finish(self, summed, out=None):
        return summed.to(torch.bfloat16)

    def ep_finish_gathered(self, gathered, out=None):
        acc = gathered[0].clone()
        for r in range(1, gathered.shape[0]):          # rank order
            acc += gathered[r]
        return acc.to(torch.bfloat16)


def _ep_worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.CONFIGS["c0"]
    n = 24
    x = torch.from_numpy(wl.gen_tokens(cfg, 0, n).view(np.int16)).view(torch.bfloat16)
    aid = torch.from_numpy(wl.gen_adapter_ids(cfg, n))
    layer = ep.ExpertParallelLayer(_OraclePool(cfg, world, rank, n))
    assert layer.world() == world
    out = layer.forward(0, x, aid)
    np.save(os.path.join(out_dir, f"out{rank}.npy"), out.view(torch.int16).numpy())
    out_g = layer.forward_gathered(0, x, aid)
    np.save(os.path.join(out_dir, f"gathered{rank}.npy"), out_g.view(torch.int16).numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_add_up_to_the_oracle_layer(tmp_path):
    world = 2
    mp.spawn(_ep_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    cfg = wl.CONFIGS["c0"]
    n = 24
    bank = wl.NoiseBank(cfg.seed)
    xb, aid = wl.gen_tokens(cfg, 0, n), wl.gen_adapter_ids(cfg, n)
    ref, ids, w, slots = oracle.layer_forward(oracle_layer(cfg, 0, bank, wl.tuned_sets(cfg)), xb, aid)
    outs = [np.load(tmp_path / f"out{r}.npy") for r in range(world)]
    assert np.array_equal(outs[0], outs[1])            # every rank ends with the same result
    got = torch.from_numpy(outs[0]).view(torch.bfloat16).float().numpy()
    want = torch.from_numpy(ref).to(torch.bfloat16).float().numpy()
    # the partial sums are added in rank order, the oracle adds pair by pair: the fp32 sums differ in their last
    # bits, so a few results fall on the other side of a bf16 rounding boundary
    assert np.abs(got - want).max() <= 2.0 ** -7 * np.abs(want).max()
    assert (got != want).mean() < 0.02
    # the all-gather form adds the partial sums in rank order on every rank: identical bits on both ranks, and the same
    # closeness to the oracle
    gath = [np.load(tmp_path / f"gathered{r}.npy") for r in range(world)]
    assert np.array_equal(gath[0], gath[1])
    got_g = torch.from_numpy(gath[0]).view(torch.bfloat16).float().numpy()
    assert np.abs(got_g - want).max() <= 2.0 ** -7 * np.abs(want).max()
    # and no rank alone gives the answer: both hold experts the batch uses
    mask0 = ep.local_pair_mask(ids, cfg.num_experts, world, 0)
    assert mask0.any() and (~mask0).any()


def test_single_rank_layer_needs_no_process_group():
    cfg = wl.CONFIGS["c0"]
    n = 5
    x = torch.from_numpy(wl.gen_tokens(cfg, 0, n).view(np.int16)).view(torch.bfloat16)
    aid = torch.from_numpy(wl.gen_adapter_ids(cfg, n))
    out = ep.ExpertParallelLayer(_OraclePool(cfg, 1, 0, n)).forward(0, x, aid)
    ref, *_ = oracle.layer_forward(oracle_layer(cfg, 0, wl.NoiseBank(cfg.seed), wl.tuned_sets(cfg)), wl.gen_tokens(cfg, 0, n),
                                   wl.gen_adapter_ids(cfg, n))
    assert torch.equal(out, torch.from_numpy(ref).to(torch.bfloat16))
