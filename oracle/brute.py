"""Independent fp64 witness for tiny inputs (test infrastructure only).

Written separately from `ew_oracle.c`: no expert map, no slots.  For each token it enumerates every
size-k subset of the M experts, keeps the subset with the largest probability sum (ties: the
lexicographically smallest sorted index tuple, which is what "lowest index wins" selects), and
evaluates the merged model of the token's adapter (Section 3.2: a token of adapter i must be
processed by adapter i's copy of an expert when the adapter tunes it, by the base expert otherwise)
with numpy fp64 matmuls.
"""
import itertools

import numpy as np


def _f64(bits):
    return (np.asarray(bits, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def layer_forward_fp64(x_bits, aid, router_w, w_gate, w_up, w_down, s_gate, s_up, s_down, adapters, k,
                       renormalize=False, routed_scale=1.0):
    """adapters[i] = None or (tuned_ids, w_gate, w_up, w_down) with bf16 bits.  Returns (out, chosen)."""
    x = _f64(x_bits)
    rw = _f64(router_w)
    B, H = x.shape
    M = rw.shape[0]
    out = np.zeros((B, H))
    chosen = []
    for t in range(B):
        z = rw @ x[t]
        p = np.exp(z - z.max())
        p = p / p.sum()
        best, best_sum = None, -1.0
        for sub in itertools.combinations(range(M), k):      # ascending tuples in lexicographic order
            s = sum(p[j] for j in sub)
            if s > best_sum + 1e-12:     # equal sums: keep the lexicographically first subset
                best, best_sum = sub, s
        chosen.append(best)
        wts = np.array([p[j] for j in best])
        if renormalize:
            wts = wts / wts.sum()
        wts = wts * routed_scale
        a = int(aid[t])
        y = np.zeros(H)
        for j, wj in zip(best, wts):
            g, u, d = w_gate[j], w_up[j], w_down[j]
            if a >= 0 and adapters[a] is not None:
                ids, ag, au, ad = adapters[a]
                for pos, jj in enumerate(ids):
                    if int(jj) == j:
                        g, u, d = ag[pos], au[pos], ad[pos]
            gg = _f64(g) @ x[t]
            uu = _f64(u) @ x[t]
            y += wj * (_f64(d) @ ((gg / (1.0 + np.exp(-gg))) * uu))
        for s in range(len(s_gate)):
            gg = _f64(s_gate[s]) @ x[t]
            uu = _f64(s_up[s]) @ x[t]
            y += _f64(s_down[s]) @ ((gg / (1.0 + np.exp(-gg))) * uu)
        out[t] = y
    return out, chosen
