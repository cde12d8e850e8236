"""Shared test plumbing: build the oracle's layer and the GPU pool from the same seeded bits, and the
staged comparison of a GPU forward against the oracle."""
from __future__ import annotations

import numpy as np

import oracle
from paper_2508_17624_b200 import workloads as wl

NEAR_TIE = 1e-5          # a token whose k-th and (k+1)-th probabilities differ by less is a near-tie
REL_L2_TOL = 1e-2        # bf16 layer output vs the fp32 oracle
MAX_ABS_TOL = 2e-2
# Combine weights: both sides accumulate the H-term logit in fp32 but in a different order (sequential in the
# oracle, the tensor core's tree on the GPU).  A selected expert has one of the largest logits, |z| in [2, 4) for
# H = 2048, x ~ N(0,1), router rows ~ N(0, 0.02); while the running sum is that large every addition rounds by up
# to half an ulp = 1.2e-7 (rms 7e-8), and about half of the 2048 additions happen there: rms 2.2e-6 per logit,
# 5 sigma = 1.1e-5 over the ~1e5 weights of a test.  d p / p = (1 - p) d z, so the weights agree to a relative
# 1.5e-5 (largest seen: 1.1e-5 on the 26-layer stack, 6e-6 on the 8192-token prefill batch).  The bound is
# proportional to the size of the products x_h w_h: a test that scales its activations by c passes c * WEIGHT_RTOL.
WEIGHT_RTOL = 1.5e-5
WEIGHT_TOL = 1e-7        # absolute floor


def oracle_config(cfg: wl.MoEConfig) -> oracle.OracleConfig:
    return oracle.OracleConfig(cfg.hidden, cfg.inter, cfg.num_experts, cfg.num_shared, cfg.top_k,
                               cfg.max_adapters, cfg.e_max)


def oracle_layer(cfg, layer, bank, tuned, base=None, adapters=None) -> oracle.OracleLayer:
    base = base or wl.gen_base_layer(cfg, layer, bank)
    ads = []
    for i in range(cfg.max_adapters):
        if adapters is not None and i not in adapters:
            ads.append(None)
            continue
        ew = wl.gen_adapter_layer(cfg, i, layer, tuned[i][layer], bank)
        ads.append((tuned[i][layer], ew.w_gate, ew.w_up, ew.w_down))
    return oracle.OracleLayer(oracle_config(cfg), base.router_w, base.routed.w_gate, base.routed.w_up,
                              base.routed.w_down, base.shared.w_gate, base.shared.w_up, base.shared.w_down, ads)


def oracle_partial(cfg, layer, bank, tuned, x_bits, ids, slots, w, ep_size, ep_rank, base=None, adapters=None):
    """What rank `ep_rank` of `ep_size` contributes to the layer output under expert parallelism, from the oracle:
    the pairs whose base expert id lies in the rank's block keep their weight, all others get weight 0, and only
    the rank's shared experts are present.  fp32 [B, H]; the sum over ranks is the oracle's layer output up to the
    order of the fp32 additions."""
    from paper_2508_17624_b200 import ep
    base = base or wl.gen_base_layer(cfg, layer, bank)
    s_lo, s_hi = ep.owned_range(cfg.num_shared, ep_size, ep_rank)
    ocfg = oracle.OracleConfig(cfg.hidden, cfg.inter, cfg.num_experts, s_hi - s_lo, cfg.top_k, cfg.max_adapters, cfg.e_max)
    ads = []
    for i in range(cfg.max_adapters):
        if adapters is not None and i not in adapters:
            ads.append(None)
            continue
        ew = wl.gen_adapter_layer(cfg, i, layer, tuned[i][layer], bank)
        ads.append((tuned[i][layer], ew.w_gate, ew.w_up, ew.w_down))
    ol = oracle.OracleLayer(ocfg, base.router_w, base.routed.w_gate, base.routed.w_up, base.routed.w_down,
                            base.shared.w_gate[s_lo:s_hi], base.shared.w_up[s_lo:s_hi], base.shared.w_down[s_lo:s_hi], ads)
    mask = ep.local_pair_mask(ids, cfg.num_experts, ep_size, ep_rank)
    return oracle.ffn_given_slots(ol, x_bits, slots, np.where(mask, w, np.float32(0)).astype(np.float32))


def to_dev(bits_or_ids, dtype=None):
    import torch
    a = np.ascontiguousarray(bits_or_ids)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def bf16_to_f32(t) -> np.ndarray:
    return t.float().cpu().numpy()


def _np(v):
    return v if isinstance(v, np.ndarray) else v.cpu().numpy()


def check_gate(oc, router_w, x_bits, ids_g, w_g, weight_rtol=WEIGHT_RTOL):
    """Top-k ids and combine weights of the GPU against the oracle's gate.  Ids: exact as sets, except counted
    near-ties, for which either set is accepted.  Weights: every one, the flipped tokens' included, against the
    oracle's probabilities of the experts the GPU chose (renormalised and scaled as the configuration says).
    Returns (weights to feed the staged oracle with, number of near-tie flips)."""
    B, k = ids_g.shape
    ids_o, w_o, gap, probs = oracle.gate_topk(oc, x_bits, router_w, want_probs=True)
    flips = 0
    w_ffn = np.empty_like(w_g)
    for t in range(B):
        flipped = set(ids_g[t].tolist()) != set(ids_o[t].tolist())
        if flipped:
            assert gap[t] < NEAR_TIE, f"token {t}: top-k differs with gap {gap[t]}"
            # whatever the GPU picked instead is itself within the window of the oracle's k-th probability
            extra = sorted(set(ids_g[t].tolist()) - set(ids_o[t].tolist()))
            assert all(probs[t, j] > probs[t, ids_o[t, k - 1]] - NEAR_TIE for j in extra), (t, extra)
            flips += 1
            wt = probs[t, ids_g[t]].astype(np.float32)       # the oracle's probabilities of the GPU's choice
            if oc.renormalize:
                wt = wt / wt.sum(dtype=np.float32)
            wt = wt * np.float32(oc.routed_scale)
            lut = {int(j): float(w) for j, w in zip(ids_g[t], wt)}
        else:
            lut = {int(j): float(w) for j, w in zip(ids_o[t], w_o[t])}
        for c in range(k):
            wo = lut[int(ids_g[t, c])]
            assert abs(wo - w_g[t, c]) <= WEIGHT_TOL + weight_rtol * wo, (t, c, wo, w_g[t, c])
            w_ffn[t, c] = wo
        if not flipped and gap[t] >= NEAR_TIE and \
                (k == 1 or np.min(np.abs(np.diff(np.sort(w_o[t])))) >= NEAR_TIE * max(1.0, w_o[t].sum())):
            assert ids_g[t].tolist() == ids_o[t].tolist(), f"token {t}: order differs"
    assert len(set(map(len, map(set, ids_g.tolist())))) == 1 and len(set(ids_g[0].tolist())) == k
    return w_ffn, flips


def check_routing(cfg, olayer, x_bits, aid, r, Pi=None, weight_rtol=WEIGHT_RTOL):
    """Compare the routing-side results of a debug forward `r` (dict of torch tensors) with the oracle.
    Returns (ids_gpu, w_for_ffn, slots_gpu, n_near_tie_flips)."""
    oc = olayer.cfg
    B, k, P = x_bits.shape[0], oc.k, oc.P
    ids_g = _np(r["topk_ids"])
    w_g = _np(r["topk_w"])
    slots_g = _np(r["slot_ids"])
    counts_g = _np(r["counts"])
    w_ffn, flips = check_gate(oc, olayer.router_w, x_bits, ids_g, w_g, weight_rtol)
    # rerouted slots and counts: bit-exact given the same top-k ids (adapters that are not loaded and ids
    # outside [-1, N) behave as base tokens on both sides)
    Pi = olayer.build_map() if Pi is None else Pi
    slots_o = oracle.reroute(ids_g, aid, Pi, loaded=olayer.loaded)
    assert np.array_equal(slots_g, slots_o)
    counts_o = oracle.counts(slots_g, P)
    assert np.array_equal(counts_g, counts_o)
    if "inv" not in r:
        return ids_g, w_ffn, slots_g, flips
    inv_g = _np(r["inv"])
    off_g = _np(r["offsets"])
    # offsets: exclusive scan; inv: a bijection onto [0, B*k) that respects the slot chunks
    assert np.array_equal(off_g, np.concatenate([[0], np.cumsum(counts_o)]).astype(np.int32))
    flat = inv_g.reshape(-1)
    assert np.array_equal(np.sort(flat), np.arange(B * k))
    s = slots_g.reshape(-1)
    assert np.all(flat >= off_g[s]) and np.all(flat < off_g[s + 1])
    return ids_g, w_ffn, slots_g, flips


def check_output(olayer, x_bits, slots, w, out_gpu_f32, sample=None):
    """Layer output against the fp32 oracle fed with the given slots/weights (optionally on a sample)."""
    idx = np.arange(x_bits.shape[0]) if sample is None else np.asarray(sample)
    ref = oracle.ffn_given_slots(olayer, x_bits[idx], slots[idx], w[idx])
    got = out_gpu_f32[idx]
    rel = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30))
    mx = float(np.abs(got - ref).max())
    assert rel <= REL_L2_TOL, f"relative L2 error {rel}"
    assert mx <= MAX_ABS_TOL, f"max abs error {mx}"
    return rel, mx
