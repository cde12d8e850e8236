"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test is chosen so that a plausible mistake in `oracle/ew_oracle.c` (a dropped term, a wrong
sign or index, a transposed operand, a wrong tie rule) fails at least one of them.
"""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import brute, stats
from paper_2508_17624_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_kv(name):
    out = {}
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, *v = line.split()
        out[k] = v
    return out


# ----------------------------------------------------------------------------- expert map, reroute

def test_fig4_expert_map():
    """Figure 4's parameters: adapter 0 owns slots 64..66, adapter 1 slots 72..78, first dim 80."""
    g = _read_kv("fig4_batched_rerouting.txt")
    M, N, E_max = int(g["M"][0]), int(g["N"][0]), int(g["E_max"][0])
    e = [int(v) for v in g["e"]]
    rng = np.random.default_rng(4)
    tuned = [np.sort(rng.choice(M, size=e[i], replace=False)).astype(np.int32) for i in range(N)]
    Pi = oracle.build_map(M, N, E_max, tuned)
    assert Pi.shape == (N, M)
    for i in range(N):
        assert [int(v) for v in g[f"adapter{i}_slots"]] == [int(Pi[i, j]) for j in tuned[i]]
        assert int(g["Delta"][i]) == M + i * E_max
        untuned = np.setdiff1d(np.arange(M), tuned[i])
        assert np.array_equal(Pi[i, untuned], untuned)          # untuned experts keep their index
    assert Pi.max() < int(g["first_dim"][0]) == M + N * E_max


def test_reroute_definition():
    """TopK'(x) = {Pi[A(x), j]}; -1 = base model; token granularity (any interleaving of adapters)."""
    M, N, E_max, k, B = 64, 2, 8, 6, 200
    rng = np.random.default_rng(5)
    tuned = [np.array([3, 10, 40], np.int32), np.array([0, 3, 9, 10, 11, 50, 63], np.int32)]
    Pi = oracle.build_map(M, N, E_max, tuned)
    ids = np.stack([rng.choice(M, size=k, replace=False) for _ in range(B)]).astype(np.int32)
    aid = rng.integers(-1, N, size=B).astype(np.int32)
    slots = oracle.reroute(ids, aid, Pi)
    for t in range(B):
        for r in range(k):
            j, a = int(ids[t, r]), int(aid[t])
            if a < 0 or j not in tuned[a]:
                assert slots[t, r] == j                        # never redirected
            else:
                assert slots[t, r] == M + a * E_max + list(tuned[a]).index(j)
    cnt = oracle.counts(slots, M + N * E_max)
    assert cnt.sum() == B * k
    # every pair that selected base expert j lands on j or one of its adapter copies
    for j in range(M):
        group = {j} | {int(Pi[i, j]) for i in range(N)}
        assert sum(int(cnt[s]) for s in group) == int((ids == j).sum())
    # padding slots are never hit
    for i in range(N):
        for d in range(len(tuned[i]), E_max):
            assert cnt[M + i * E_max + d] == 0


def test_reroute_bad_and_unloaded_adapter_ids_are_base_tokens():
    """The paper defines the adapter id as -1 (base model) or an adapter index (Section 4.3) and is silent on
    anything else.  Reading pinned here: an id outside [-1, N), or the id of an adapter that is not loaded, makes
    the token a base-model token (ids unchanged) and is counted; nothing is read outside the map.  The expected
    values are spelled out by hand for a map small enough to check by eye."""
    M, N, E_max = 4, 3, 2
    tuned = [np.array([1, 2], np.int32), np.array([0], np.int32), np.array([3], np.int32)]
    Pi = oracle.build_map(M, N, E_max, tuned)
    assert Pi.tolist() == [[0, 4, 5, 3], [6, 1, 2, 3], [0, 1, 2, 8]]
    ids = np.array([[1, 2], [0, 3], [3, 0], [2, 1], [1, 0], [3, 2], [0, 1]], np.int32)
    aid = np.array([0, 1, 2, -1, 3, -2, 2**30], np.int32)
    slots, bad = oracle.reroute(ids, aid, Pi, return_bad=True)             # every adapter loaded
    assert slots.tolist() == [[4, 5], [6, 3], [8, 0], [2, 1], [1, 0], [3, 2], [0, 1]] and bad == 3
    # adapter 1 not loaded: its token keeps the base ids even though a (stale) row for it exists in the map
    slots, bad = oracle.reroute(ids, aid, Pi, loaded=np.array([1, 0, 1], np.int32), return_bad=True)
    assert slots.tolist() == [[4, 5], [0, 3], [8, 0], [2, 1], [1, 0], [3, 2], [0, 1]] and bad == 4
    # a large negative id is not an index into the map either
    slots, bad = oracle.reroute(ids[:1], np.array([-2**31], np.int32), Pi, return_bad=True)
    assert slots.tolist() == [[1, 2]] and bad == 1
    # with the ids rewritten to -1 by hand the result is the same and nothing is counted
    fixed = np.where((aid < -1) | (aid >= N), -1, aid).astype(np.int32)
    slots2, bad2 = oracle.reroute(ids, fixed, Pi, return_bad=True)
    assert bad2 == 0 and np.array_equal(slots2, oracle.reroute(ids, aid, Pi))


def test_build_map_rejects_bad_lists():
    with pytest.raises(ValueError):
        oracle.build_map(8, 1, 2, [np.array([1, 2, 3], np.int32)])      # e > E_max
    with pytest.raises(ValueError):
        oracle.build_map(8, 1, 4, [np.array([2, 1], np.int32)])         # not ascending
    with pytest.raises(ValueError):
        oracle.build_map(8, 1, 4, [np.array([1, 8], np.int32)])         # id out of range


# ----------------------------------------------------------------------------- closed-form metrics

def test_table1_sparsity_and_fragmentation():
    rows = []
    for line in open(os.path.join(GOLD, "table1_adapter_sparsity.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, mx, avg, s = line.split()
        rows.append((name, float(mx), float(avg), float(s)))
    assert len(rows) == 10
    for name, mx, avg, s in rows:
        assert abs(stats.adapter_sparsity_from_summary(mx, avg) - s) <= 0.0051, name
    f = stats.fragmentation_from_summary(64, 13, [r[2] for r in rows])
    assert 1.495 <= f <= 1.515            # printed 1.51; the rounded averages give 1.502
    # the per-layer form agrees with the summary form
    rng = np.random.default_rng(0)
    e = rng.integers(0, 14, size=(10, 26))
    e[:, 0] = 13
    assert abs(stats.adapter_sparsity(e[3]) - stats.adapter_sparsity_from_summary(e[3].max(), e[3].mean())) < 1e-12
    assert abs(stats.fragmentation(64, 13, e) - stats.fragmentation_from_summary(64, 13, e.mean(axis=1))) < 1e-12
    assert stats.fragmentation(64, 13, np.full((10, 26), 13)) == 1.0


# ----------------------------------------------------------------------------- helpers for layer tests

def _tiny(H=32, I=16, M=6, S=1, k=2, N=2, E_max=2, seed=0, tuned=None, w_std=0.5):
    rng = np.random.default_rng(seed)

    def w(*shape):
        return wl.f32_to_bf16_bits((rng.standard_normal(shape) * w_std / np.sqrt(shape[-1])).astype(np.float32))

    cfg = oracle.OracleConfig(H, I, M, S, k, N, E_max)
    tuned = tuned if tuned is not None else [np.array([1, 4], np.int32), np.array([4], np.int32)][:N]
    base = dict(router_w=wl.f32_to_bf16_bits(rng.standard_normal((M, H)).astype(np.float32) * 0.3),
                w_gate=w(M, I, H), w_up=w(M, I, H), w_down=w(M, H, I),
                s_gate=w(S, I, H), s_up=w(S, I, H), s_down=w(S, H, I))
    adapters = [(t, w(len(t), I, H), w(len(t), I, H), w(len(t), H, I)) for t in tuned]
    return cfg, base, adapters, rng


def _x(rng, B, H):
    return wl.f32_to_bf16_bits(rng.standard_normal((B, H)).astype(np.float32))


# ----------------------------------------------------------------------------- the paper's invariants

def test_merged_model_equivalence_bitwise():
    """Section 5.5 / Table 3: serving through the map gives exactly the merged models' results."""
    cfg, base, adapters, rng = _tiny()
    B = 40
    x = _x(rng, B, cfg.H)
    aid = rng.integers(-1, cfg.N, size=B).astype(np.int32)
    layer = oracle.OracleLayer(cfg, **base, adapters=adapters)
    out, ids, w, slots = oracle.layer_forward(layer, x, aid)
    ref = oracle.layer_forward_merged(layer, x, aid)
    assert np.array_equal(out.view(np.uint32), ref.view(np.uint32))
    assert (slots >= cfg.M).any() and (slots < cfg.M).any()
    # and against explicitly merged weight tensors run through the base-only path, adapter by adapter
    for a in range(cfg.N):
        t_ids, ag, au, ad = adapters[a]
        merged = {k_: v.copy() for k_, v in base.items()}
        merged["w_gate"][t_ids], merged["w_up"][t_ids], merged["w_down"][t_ids] = ag, au, ad
        ml = oracle.OracleLayer(cfg, **merged, adapters=None)
        sel = np.nonzero(aid == a)[0]
        o2, *_ = oracle.layer_forward(ml, x[sel], np.full(len(sel), -1, np.int32))
        assert np.array_equal(o2.view(np.uint32), out[sel].view(np.uint32))


def test_base_only_and_identical_copies():
    cfg, base, adapters, rng = _tiny()
    B = 24
    x = _x(rng, B, cfg.H)
    aid = rng.integers(0, cfg.N, size=B).astype(np.int32)
    plain = oracle.OracleLayer(cfg, **base, adapters=None)
    base_out, *_ = oracle.layer_forward(plain, x, np.full(B, -1, np.int32))
    # no adapter loaded: adapter ids fall through identity rows
    o, _, _, slots = oracle.layer_forward(plain, x, aid)
    assert np.array_equal(o, base_out) and (slots < cfg.M).all()
    # adapters loaded but every token is a base token
    full = oracle.OracleLayer(cfg, **base, adapters=adapters)
    o, _, _, slots = oracle.layer_forward(full, x, np.full(B, -1, np.int32))
    assert np.array_equal(o, base_out) and (slots < cfg.M).all()
    # adapter copies equal to the base weights: redirected, yet the same output bit for bit
    same = [(t, base["w_gate"][t], base["w_up"][t], base["w_down"][t]) for t, *_ in adapters]
    clone = oracle.OracleLayer(cfg, **base, adapters=same)
    o, _, _, slots = oracle.layer_forward(clone, x, aid)
    assert np.array_equal(o, base_out) and (slots >= cfg.M).any()
    # an adapter that is not loaded: its tokens (and tokens with an id past N) are base tokens, whether the map
    # holds an identity row for it or a stale one; the merged-model path agrees
    part = oracle.OracleLayer(cfg, **base, adapters=[adapters[0], None])
    aid_bad = aid.copy()
    aid_bad[0] = cfg.N + 5
    want = np.where((aid_bad == 1) | (aid_bad >= cfg.N), -1, aid_bad).astype(np.int32)
    o_want, *_ = oracle.layer_forward(full, x, want)
    for Pi in (None, full.build_map()):
        o, _, _, slots = oracle.layer_forward(part, x, aid_bad, Pi)
        assert np.array_equal(o, o_want)
        assert (slots[(aid_bad == 1) | (aid_bad >= cfg.N)] < cfg.M).all()
    assert np.array_equal(oracle.layer_forward_merged(part, x, aid_bad), o_want)
    # adapter copies that differ change exactly the tokens whose routed set meets the tuned set
    o, ids, _, slots = oracle.layer_forward(full, x, aid)
    touched = (slots >= cfg.M).any(axis=1)
    assert touched.any() and (~touched).any()
    assert np.array_equal(o[~touched], base_out[~touched])
    assert not np.any(np.all(o[touched] == base_out[touched], axis=1))


def test_batch_and_permutation_invariance():
    cfg, base, adapters, rng = _tiny(seed=3)
    B = 17
    x = _x(rng, B, cfg.H)
    aid = rng.integers(-1, cfg.N, size=B).astype(np.int32)
    layer = oracle.OracleLayer(cfg, **base, adapters=adapters)
    out, *_ = oracle.layer_forward(layer, x, aid)
    for t in (0, 5, 16):
        o1, *_ = oracle.layer_forward(layer, x[t:t + 1], aid[t:t + 1])
        assert np.array_equal(o1[0], out[t])
    perm = rng.permutation(B)
    op, *_ = oracle.layer_forward(layer, x[perm], aid[perm])
    assert np.array_equal(op, out[perm])


def test_padding_slot_is_an_error():
    cfg, base, adapters, rng = _tiny()
    layer = oracle.OracleLayer(cfg, **base, adapters=adapters)
    x = _x(rng, 1, cfg.H)
    bad = np.array([[cfg.M + 1 * cfg.E_max + 1, 0]], np.int32)     # adapter 1 tunes one expert: delta 1 is padding
    with pytest.raises(ValueError):
        oracle.ffn_given_slots(layer, x, bad, np.ones((1, 2), np.float32))


# ----------------------------------------------------------------------------- brute force, fp64

@pytest.mark.parametrize("seed,M,k,renorm", [(0, 4, 2, False), (1, 6, 3, False), (2, 5, 1, True), (3, 6, 2, True)])
def test_brute_force_fp64(seed, M, k, renorm):
    cfg, base, adapters, rng = _tiny(H=8, I=8, M=M, S=1, k=k, N=2, E_max=2, seed=seed,
                                     tuned=[np.array([0, 2], np.int32), np.array([2], np.int32)])
    cfg.renormalize = int(renorm)
    cfg.routed_scale = 1.5 if renorm else 1.0
    B = 12
    x = _x(rng, B, cfg.H)
    aid = rng.integers(-1, cfg.N, size=B).astype(np.int32)
    layer = oracle.OracleLayer(cfg, **base, adapters=adapters)
    out, ids, w, slots = oracle.layer_forward(layer, x, aid)
    ref, chosen = brute.layer_forward_fp64(x, aid, base["router_w"], base["w_gate"], base["w_up"], base["w_down"],
                                           base["s_gate"], base["s_up"], base["s_down"], adapters, k,
                                           renormalize=renorm, routed_scale=cfg.routed_scale)
    for t in range(B):
        assert tuple(sorted(int(j) for j in ids[t])) == chosen[t]
    assert np.abs(out - ref).max() <= 1e-5 * max(1.0, np.abs(ref).max())


def test_topk_order_and_tie_break():
    """Rows come out by (probability descending, index ascending); exact ties go to the lower index."""
    H, M, k = 16, 8, 3
    rng = np.random.default_rng(7)
    rw = rng.standard_normal((M, H)).astype(np.float32)
    rw[5] = rw[2]                       # experts 2 and 5 always tie exactly
    rw[7] = rw[2]
    rw_bits = wl.f32_to_bf16_bits(rw)
    x = _x(rng, 64, H)
    cfg = oracle.OracleConfig(H, 4, M, 0, k, 1, 1)
    ids, w, gap, probs = oracle.gate_topk(cfg, x, rw_bits, want_probs=True)
    assert np.allclose(probs.sum(axis=1), 1.0, atol=1e-5)
    seen_tie_cut = False
    for t in range(64):
        order = sorted(range(M), key=lambda j: (-probs[t, j], j))
        assert list(ids[t]) == order[:k]
        assert np.array_equal(w[t], probs[t, order[:k]])
        assert abs(gap[t] - (probs[t, order[k - 1]] - probs[t, order[k]])) < 1e-7
        if 2 in ids[t] and 7 not in ids[t]:
            seen_tie_cut = True         # the tie group {2,5,7} was cut: lower indices won
            assert gap[t] == 0.0
    assert seen_tie_cut
    # fp64 library witness for the probabilities
    z = torch.from_numpy(wl.bf16_bits_to_f32(x)).double() @ torch.from_numpy(wl.bf16_bits_to_f32(rw_bits)).double().T
    assert np.abs(torch.softmax(z, dim=1).numpy() - probs).max() < 1e-6


# ----------------------------------------------------------------------------- library special cases

def _torch_ffn(x, g, u, d):
    gg, uu = x @ g.T, x @ u.T
    return (torch.nn.functional.silu(gg) * uu) @ d.T


def test_single_expert_is_a_swiglu_mlp():
    """M = 1, k = 1: p = 1, the layer is one SwiGLU MLP (plus the shared one)."""
    cfg, base, adapters, rng = _tiny(H=48, I=24, M=1, S=1, k=1, N=1, E_max=1, tuned=[np.array([0], np.int32)])
    B = 9
    x = _x(rng, B, cfg.H)
    layer = oracle.OracleLayer(cfg, **base, adapters=adapters)
    tx = torch.from_numpy(wl.bf16_bits_to_f32(x)).double()
    T = lambda b: torch.from_numpy(wl.bf16_bits_to_f32(b)).double()
    shared = _torch_ffn(tx, T(base["s_gate"][0]), T(base["s_up"][0]), T(base["s_down"][0]))
    out, _, w, _ = oracle.layer_forward(layer, x, np.full(B, -1, np.int32))
    assert np.all(w == 1.0)
    ref = _torch_ffn(tx, T(base["w_gate"][0]), T(base["w_up"][0]), T(base["w_down"][0])) + shared
    assert np.abs(out - ref.numpy()).max() < 2e-5
    out, *_ = oracle.layer_forward(layer, x, np.zeros(B, np.int32))          # adapter 0 replaces the expert
    _, ag, au, ad = adapters[0]
    ref = _torch_ffn(tx, T(ag[0]), T(au[0]), T(ad[0])) + shared
    assert np.abs(out - ref.numpy()).max() < 2e-5


def test_dense_mixture_when_k_equals_m():
    cfg, base, adapters, rng = _tiny(H=32, I=16, M=4, S=0, k=4, N=1, E_max=1, tuned=[np.array([2], np.int32)])
    B = 7
    x = _x(rng, B, cfg.H)
    layer = oracle.OracleLayer(cfg, **base, adapters=adapters)
    out, ids, w, _ = oracle.layer_forward(layer, x, np.full(B, -1, np.int32))
    T = lambda b: torch.from_numpy(wl.bf16_bits_to_f32(b)).double()
    tx = T(x)
    p = torch.softmax(tx @ T(base["router_w"]).T, dim=1)
    ref = sum(p[:, j:j + 1] * _torch_ffn(tx, T(base["w_gate"][j]), T(base["w_up"][j]), T(base["w_down"][j]))
              for j in range(4))
    assert np.abs(out - ref.numpy()).max() < 2e-5
    assert np.allclose(w.sum(axis=1), 1.0, atol=1e-6)


def test_staged_path_equals_whole_path_on_c0():
    """The stages (gate_topk, reroute, ffn_given_slots) compose to layer_forward on the tiny config."""
    cfg = wl.CONFIGS["c0"]
    bank = wl.NoiseBank(cfg.seed)
    base = wl.gen_base_layer(cfg, 0, bank)
    tuned = wl.tuned_sets(cfg)
    ads = []
    for i in range(cfg.max_adapters):
        ew = wl.gen_adapter_layer(cfg, i, 0, tuned[i][0], bank)
        ads.append((tuned[i][0], ew.w_gate, ew.w_up, ew.w_down))
    oc = oracle.OracleConfig(cfg.hidden, cfg.inter, cfg.num_experts, cfg.num_shared, cfg.top_k,
                             cfg.max_adapters, cfg.e_max)
    layer = oracle.OracleLayer(oc, base.router_w, base.routed.w_gate, base.routed.w_up, base.routed.w_down,
                               base.shared.w_gate, base.shared.w_up, base.shared.w_down, ads)
    x, aid = wl.gen_tokens(cfg), wl.gen_adapter_ids(cfg)
    out, ids, w, slots = oracle.layer_forward(layer, x, aid)
    Pi = layer.build_map()
    assert Pi[0, 5] == 16 + 1 and Pi[1, 5] == 16 + 3 + 0 and Pi[1, 14] == 16 + 3 + 2
    ids2, w2, gap, _ = oracle.gate_topk(oc, x, base.router_w)
    slots2 = oracle.reroute(ids2, aid, Pi)
    assert np.array_equal(ids, ids2) and np.array_equal(w, w2) and np.array_equal(slots, slots2)
    out2 = oracle.ffn_given_slots(layer, x, slots2, w2)
    assert np.array_equal(out, out2)
    assert np.array_equal(out, oracle.layer_forward_merged(layer, x, aid))
    assert set(np.unique(aid)) == {-1, 0, 1}


def test_counts_is_a_histogram():
    """Tokens per slot (Section 2.1 dispatch) is a plain histogram of the slot ids: numpy's bincount."""
    rng = np.random.default_rng(11)
    P = 37
    slots = rng.integers(0, P, size=(500, 3)).astype(np.int32)
    slots[slots == 5] = 6                                     # an empty slot in the middle
    assert np.array_equal(oracle.counts(slots, P), np.bincount(slots.reshape(-1), minlength=P))
    assert np.array_equal(oracle.counts(np.zeros((0, 3), np.int32), P), np.zeros(P, np.int64))


def test_topk_from_logits_against_library_topk():
    """Given logits (the stand-alone operator's input recipe), ids and weights are the library's softmax + top-k
    in fp64 wherever the k-th and (k+1)-th probabilities are not within rounding of each other."""
    rng = np.random.default_rng(12)
    B, M, k = 300, 64, 6
    logits = rng.standard_normal((B, M)).astype(np.float32)
    cfg = oracle.OracleConfig(16, 4, M, 0, k, 1, 1)
    ids, w, gap = oracle.topk_from_logits(cfg, logits)
    p = torch.softmax(torch.from_numpy(logits).double(), dim=1)
    tw, ti = torch.topk(p, k, dim=1)                          # sorted descending
    clear = gap > 1e-6
    assert clear.mean() > 0.9
    assert np.array_equal(ids[clear], ti.numpy()[clear].astype(np.int32))
    assert np.abs(w[clear] - tw.numpy()[clear]).max() < 1e-6
    full = np.sort(p.numpy(), axis=1)[:, ::-1]
    assert np.abs(gap - (full[:, k - 1] - full[:, k])).max() < 1e-6
