"""Page accounting of the virtual weight tensors (Section 4.2) on the accounting-only backend.

The expected numbers are re-derived in this file from the definition alone: a page is mapped iff the
byte range of at least one live expert intersects it; start_addr = base_addr + slot * expert_size.
"""
import os

import numpy as np
import pytest

from paper_2508_17624_b200 import binding, build

MiB = 1 << 20
PAGE = 2 * MiB


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def pages_of(slots, expert_bytes, page=PAGE):
    s = set()
    for slot in slots:
        lo, hi = slot * expert_bytes, (slot + 1) * expert_bytes
        s.update(range(lo // page, (hi - 1) // page + 1))
    return s


def expect_mapped(cfg, live_slots_per_layer):
    """live_slots_per_layer: list over layers of the set of live slot indices (including shared)."""
    e13, e2 = 2 * cfg["inter"] * cfg["hidden"] * 2, cfg["inter"] * cfg["hidden"] * 2
    return sum(len(pages_of(s, e13)) + len(pages_of(s, e2)) for s in live_slots_per_layer)


def mk(**kw):
    base = dict(device=-1, num_layers=1, hidden=1024, inter=768, num_experts=4, num_shared=0, top_k=2,
                max_adapters=2, e_max=3, max_tokens=16)
    base.update(kw)
    return binding.Pool(**base), base


def load(pool, a, per_layer_ids):
    counts = np.array([len(x) for x in per_layer_ids], np.int32)
    ids = np.concatenate([np.asarray(x, np.int32) for x in per_layer_ids]) if counts.sum() else np.zeros(0, np.int32)
    pool.load_adapter(a, counts, ids, None, None, None)


def test_fig3_virtual_tensor_example():
    """Figure 3: E_max = 3, e_0 = 2, e_1 = 1, every expert is 1.5 pages."""
    g = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "fig3_virtual_tensor.txt")):
        if line.strip() and not line.startswith("#"):
            k, *v = line.split()
            g[k] = v
    pool, cfg = mk(e_max=int(g["E_max"][0]))                       # gate|up tensor: 2*768*1024*2 B = 3 MiB = 1.5 pages
    assert 2 * cfg["inter"] * cfg["hidden"] * 2 == float(g["expert_pages"][0]) * PAGE
    s0 = pool.stats()
    assert s0["pages_mapped"] == 0 and s0["page_bytes"] == PAGE   # reservation maps nothing
    assert s0["va_reserved_bytes"] >= (4 + 2 * 3) * (3 + 1.5) * MiB
    pool.load_base(0, None, None, None, None)
    base_pages = pool.stats()["pages_mapped"]
    assert base_pages == 6 + 3                                    # 4 x 3 MiB and 4 x 1.5 MiB
    e0, e1 = int(g["e"][0]), int(g["e"][1])
    load(pool, 0, [list(range(e0))])
    after0 = pool.stats()["pages_mapped"]
    # the gate|up tensor gains exactly 3 pages under adapter 0's two experts (the down tensor 2)
    assert after0 - base_pages == int(g["adapter0_new_pages"][0]) + 2
    load(pool, 1, [[2][:e1]])
    after1 = pool.stats()["pages_mapped"]
    # adapter 1 starts mid-page at slot 7: bytes [21,24) MiB of gate|up -> pages 10,11; down [10.5,12) -> page 5
    assert after1 - after0 == 2 + 1
    live = {0, 1, 2, 3, 4, 5, 7}
    assert after1 == expect_mapped(cfg, [live])
    # adapter 0's padding slot 6 holds no page of its own: page 9 = [18,20) MiB stays unmapped
    assert 9 not in pages_of(live, 3 * MiB) and 9 in pages_of({6}, 3 * MiB)
    pm = pool.get_expert_map(0)
    assert pm[0].tolist() == [4, 5, 2, 3] and pm[1].tolist() == [0, 1, 7, 3]
    pool.destroy()


def test_fig4_shapes_at_deepseek_sizes():
    """M=64, N=2, E_max=8, e_0=3, e_1=7 with 11 MiB / 5.5 MiB experts (5.5 and 2.75 pages)."""
    pool, cfg = mk(hidden=2048, inter=1408, num_experts=64, num_shared=0, top_k=6, max_adapters=2, e_max=8)
    pool.load_base(0, None, None, None, None)
    assert pool.stats()["pages_mapped"] == 352 + 176
    load(pool, 0, [[3, 10, 40]])
    assert pool.stats()["pages_mapped"] == 352 + 176 + 17 + 9
    load(pool, 1, [[0, 3, 9, 10, 11, 50, 63]])
    st = pool.stats()
    assert st["pages_mapped"] == 352 + 176 + 17 + 9 + 39 + 20
    assert st["pages_mapped"] == expect_mapped(cfg, [set(range(64)) | {64, 65, 66} | set(range(72, 79))])
    assert st["live_experts"] == 64 + 10 and st["adapters_loaded"] == 2
    assert st["padding_bytes"] == 80 * 3 * 1408 * 2048 * 2
    assert st["physical_bytes"] < st["padding_bytes"]
    pool.destroy()


def test_tiny_config_shares_pages_between_adapters():
    """c0 shapes: 128 KiB / 64 KiB experts, so both adapters live inside pages the base already holds."""
    pool, cfg = mk(hidden=256, inter=128, num_experts=16, num_shared=1, top_k=2, max_adapters=2, e_max=3)
    pool.load_base(0, None, None, None, None, None, None, None)
    base_live = set(range(16)) | {22}
    assert pool.stats()["pages_mapped"] == expect_mapped(cfg, [base_live]) == 2 + 1
    load(pool, 0, [[1, 5, 9]])
    load(pool, 1, [[5, 6, 14]])
    assert pool.stats()["pages_mapped"] == expect_mapped(cfg, [base_live | {16, 17, 18, 19, 20, 21}]) == 3
    pool.unload_adapter(0)
    pool.unload_adapter(1)
    assert pool.stats()["pages_mapped"] == 3                # shared pages stay: the base still lives there
    pool.destroy()


def test_churn_reuses_pages_and_returns_to_the_same_state():
    rng = np.random.default_rng(0)
    L = 3
    pool, cfg = mk(num_layers=L, hidden=1024, inter=768, num_experts=8, num_shared=1, max_adapters=4, e_max=4,
                   prealloc_pages=5)
    assert pool.stats()["pages_free"] == 5
    for l in range(L):
        pool.load_base(l, None, None, None, None, None, None, None)
    base = pool.stats()
    P = 8 + 4 * 4
    live = [set(range(8)) | {P} for _ in range(L)]
    assert base["pages_mapped"] == expect_mapped(cfg, live)
    loaded = {}
    peak_created = 0
    for step in range(60):
        a = int(rng.integers(0, 4))
        if a in loaded:
            pool.unload_adapter(a)
            for l in range(L):
                live[l] -= {8 + a * 4 + d for d in range(len(loaded[a][l]))}
            del loaded[a]
        else:
            per_layer = [sorted(rng.choice(8, size=int(rng.integers(0, 5)), replace=False).tolist()) for _ in range(L)]
            load(pool, a, per_layer)
            loaded[a] = per_layer
            for l in range(L):
                live[l] |= {8 + a * 4 + d for d in range(len(per_layer[l]))}
        st = pool.stats()
        assert st["pages_mapped"] == expect_mapped(cfg, live), step
        assert st["pages_mapped"] + st["pages_free"] <= st["pages_created_total"]
        peak_created = max(peak_created, st["pages_created_total"])
        for l in range(L):
            pm = pool.get_expert_map(l)
            for i in range(4):
                want = list(range(8))
                for d, j in enumerate(loaded.get(i, [[]] * L)[l]):
                    want[j] = 8 + i * 4 + d
                assert pm[i].tolist() == want
    for a in list(loaded):
        pool.unload_adapter(a)
    end = pool.stats()
    assert end["pages_mapped"] == base["pages_mapped"] and end["live_experts"] == base["live_experts"]
    # freed pages are kept for reuse; creation stops growing once the pool has seen its peak
    assert end["pages_free"] == end["pages_created_total"] - end["pages_mapped"]
    pool.trim()
    assert pool.stats()["pages_free"] == 0
    pool.destroy()


def test_load_is_all_or_nothing_under_a_page_budget():
    pool, cfg = mk(num_layers=2, max_pages=2 * 9 + 4)
    for l in range(2):
        pool.load_base(l, None, None, None, None)
    before = pool.stats()
    with pytest.raises(binding.EwError) as ei:
        load(pool, 0, [[0, 1, 2], [0, 1, 2]])            # needs 2 * (5 + 3) pages > 4 left
    assert ei.value.status == 2
    after = pool.stats()
    assert after["pages_mapped"] == before["pages_mapped"] and after["adapters_loaded"] == 0
    assert (pool.get_expert_map(0) == np.arange(4)).all() and (pool.get_expert_map(1) == np.arange(4)).all()
    load(pool, 0, [[0], []])                              # a smaller adapter still fits (e = 0 in a layer is legal)
    assert pool.stats()["adapters_loaded"] == 1
    pool.destroy()


def test_load_errors():
    pool, cfg = mk()
    pool.load_base(0, None, None, None, None)
    for bad, status in (([[0, 1, 2, 3]], 5), ([[2, 1]], 1), ([[1, 1]], 1), ([[4]], 1), ([[-1]], 1)):
        with pytest.raises(binding.EwError) as ei:
            load(pool, 0, bad)
        assert ei.value.status == status
    load(pool, 0, [[1]])
    with pytest.raises(binding.EwError) as ei:
        load(pool, 0, [[2]])
    assert ei.value.status == 3
    with pytest.raises(binding.EwError) as ei:
        load(pool, 2, [[2]])
    assert ei.value.status == 1
    pool.destroy()


def test_padding_mode_backs_everything():
    pool, cfg = mk(pool_mode=1)
    st = pool.stats()
    slots = 4 + 2 * 3
    assert st["pages_mapped"] == expect_mapped(cfg, [set(range(slots))])
    pool.load_base(0, None, None, None, None)
    load(pool, 0, [[0, 1]])
    assert pool.stats()["pages_mapped"] == st["pages_mapped"]
    pool.unload_adapter(0)
    assert pool.stats()["pages_mapped"] == st["pages_mapped"]
    pool.destroy()


def test_base_load_is_counted_once_and_a_failed_one_not_at_all():
    """ew_load_base maps the base range on its first successful call only; loading a layer again overwrites in place
    (same pages, same counters), and a first load that fails on the page budget leaves nothing mapped or counted, so
    that a retry does not double anything."""
    pool, cfg = mk(num_layers=2)
    pool.load_base(0, None, None, None, None)
    once = pool.stats()
    pool.load_base(0, None, None, None, None)
    again = pool.stats()
    assert again == once and once["live_experts"] == 4
    assert once["pages_mapped"] == expect_mapped(cfg, [set(range(4))])
    pool.destroy()
    # 4 experts of 3 MiB + 1.5 MiB: 6 + 3 pages per layer; a budget of 10 lets layer 0 in and stops layer 1 midway
    pool, cfg = mk(num_layers=2, max_pages=10)
    pool.load_base(0, None, None, None, None)
    before = pool.stats()
    for _ in range(2):                                   # the retry fails the same way and changes nothing either
        with pytest.raises(binding.EwError) as ei:
            pool.load_base(1, None, None, None, None)
        assert ei.value.status == 2
        st = pool.stats()
        for key in ("pages_mapped", "live_experts", "live_expert_bytes"):     # nothing of layer 1 stays mapped or counted
            assert st[key] == before[key], key
        assert st["pages_mapped"] + st["pages_free"] == st["pages_created_total"] <= 10   # pages made on the way wait in the free list
    pool.destroy()
