/*
 * CPU oracle for the adapter-aware MoE layer forward of ExpertWeave.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the layer computes,
 * written from the paper; it shares no code with the CUDA path and must never be called from the
 * product path.  Only the test-suite, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Arithmetic: inputs are bf16 bit patterns (uint16), widened exactly to fp32; every product and
 * sum is fp32, accumulated sequentially in ascending index order; the graded layer output is the
 * unrounded fp32 vector.
 *
 * What each function follows:
 *   ewo_build_map          ESFT expert map, Section 4.1, the two-case definition of Pi^(l)[i,j]
 *                          with Delta_i = M + i*E_max and 0 <= delta < e_i^(l).
 *   ewo_reroute            batched rerouting, Section 4.1: TopK'(x) = { Pi[A(x), j] : j in TopK(x) };
 *                          adapter id -1 marks a base-model token (Section 4.3).  The paper leaves two
 *                          inputs undefined: an id outside [-1, N) and the id of an adapter that is not
 *                          loaded.  Reading taken here: such a token is a base-model token (its ids are
 *                          kept) and it is counted in the function's return value.
 *   ewo_gate_topk          the router of Section 2.1 (g(x), top-k ids [B,k]); the paper does not fix
 *                          g, so: softmax over all M logits, the k largest probabilities, ties to
 *                          the lower index, weights = the selected probabilities (optionally
 *                          renormalised / scaled).
 *   ewo_counts             tokens per slot for the dispatch step of Section 2.1.
 *   ewo_ffn_given_slots    Section 2.1 expert computation + weighted combine, reading each expert
 *                          through its slot in the unified pool [M + N*E_max, ...] of Section 4.1.
 *   ewo_layer_forward      the adapter-aware path: gate -> top-k -> reroute -> FFN through slots.
 *   ewo_layer_forward_merged  the plain definition the method must reproduce (Section 3.2 and the
 *                          "Merged" deployment of Section 5.1): each token is processed by the merged
 *                          model of its own adapter; no map, no slots, an explicit "is expert j
 *                          tuned by adapter a" test per token.
 *
 * Parity pins (tests, "not gpu"): Figure 4's parameters for the map; merged-model equivalence,
 * base-only equivalence, identical-copy equivalence, batch and permutation invariance; fp64 brute
 * force over all C(M,k) subsets on tiny inputs; M=1,k=1 and k=M special cases against library
 * matmuls in fp64.  The paper prints no numerical layer outputs, so ewo_ffn_given_slots has no
 * golden-value fixture: its values are pinned by those library special cases, the brute force and
 * the bit-for-bit equality with the merged-model path.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t H, I, M, S, k, N, E_max;
    int32_t renormalize;   /* 1: divide the k weights by their sum */
    float routed_scale;    /* multiplies the k weights */
} ewo_cfg;

/* All weights of one layer, as the caller holds them on the host (bf16 bits). */
typedef struct {
    const uint16_t *router_w;                  /* [M, H] */
    const uint16_t *w_gate, *w_up, *w_down;    /* base routed experts [M,I,H], [M,I,H], [M,H,I] */
    const uint16_t *s_gate, *s_up, *s_down;    /* shared experts      [S,I,H], [S,I,H], [S,H,I] */
    const int32_t *e;                          /* [N] experts tuned by adapter i in this layer (0 when not loaded) */
    const int32_t *loaded;                     /* [N] 1 = adapter i is loaded (it may still tune nothing in this layer) */
    const int32_t *const *tuned;               /* [N] -> ascending base expert ids, length e[i] */
    const uint16_t *const *a_gate;             /* [N] -> [e_i, I, H] */
    const uint16_t *const *a_up;               /* [N] -> [e_i, I, H] */
    const uint16_t *const *a_down;             /* [N] -> [e_i, H, I] */
} ewo_layer;

static inline float bf(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

int ewo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Pi[i*M + j] = j if adapter i does not tune j, else M + i*E_max + (rank of j in tuned[i]). */
int ewo_build_map(int M, int N, int E_max, const int32_t *e, const int32_t *const *tuned, int32_t *Pi) {
    for (int i = 0; i < N; ++i) {
        for (int j = 0; j < M; ++j) Pi[i * M + j] = j;
        if (e[i] > E_max) return -1;
        for (int d = 0; d < e[i]; ++d) {
            int j = tuned[i][d];
            if (j < 0 || j >= M) return -2;
            if (d > 0 && tuned[i][d - 1] >= j) return -3;
            Pi[i * M + j] = M + i * E_max + d;
        }
    }
    return 0;
}

/* slots[t,r] = aid[t] == -1 ? ids[t,r] : Pi[aid[t], ids[t,r]].
 * loaded[i] != 0 marks adapter i as loaded (null = all N loaded).  A token whose id is outside [-1, N) or names
 * an adapter that is not loaded is treated as a base-model token; the return value counts such tokens. */
int ewo_reroute(int B, int k, int M, int N, const int32_t *ids, const int32_t *aid, const int32_t *Pi,
                const int32_t *loaded, int32_t *slots) {
    int bad = 0;
    for (int t = 0; t < B; ++t) {
        int a = aid[t];
        if (a < -1 || a >= N || (a >= 0 && loaded && !loaded[a])) { a = -1; ++bad; }
        for (int r = 0; r < k; ++r) {
            int j = ids[t * k + r];
            slots[t * k + r] = a < 0 ? j : Pi[a * M + j];
        }
    }
    return bad;
}

void ewo_counts(int n_pairs, int P, const int32_t *slots, int32_t *cnt) {
    for (int s = 0; s < P; ++s) cnt[s] = 0;
    for (int q = 0; q < n_pairs; ++q) cnt[slots[q]] += 1;
}

/* softmax over M fp32 logits, then the k largest (value descending, index ascending on ties) */
static void softmax_topk(const ewo_cfg *c, const float *z, float *p, int32_t *ids, float *w, float *gap) {
    int M = c->M, k = c->k;
    float mx = z[0];
    for (int j = 1; j < M; ++j) mx = z[j] > mx ? z[j] : mx;
    float sum = 0.f;
    for (int j = 0; j < M; ++j) { p[j] = expf(z[j] - mx); sum += p[j]; }
    for (int j = 0; j < M; ++j) p[j] = p[j] / sum;
    float last = 0.f;
    for (int r = 0; r <= k && r < M; ++r) {  /* one extra round finds the (k+1)-th value for the gap */
        int best = -1;
        for (int j = 0; j < M; ++j) {
            int taken = 0;
            for (int q = 0; q < r && q < k; ++q) taken |= (ids[q] == j);
            if (taken) continue;
            if (best < 0 || p[j] > p[best]) best = j;   /* strict >: the lower index keeps a tie */
        }
        if (r < k) { ids[r] = best; w[r] = p[best]; last = p[best]; }
        else if (gap) *gap = last - p[best];
    }
    if (k >= M && gap) *gap = 1.f;
    if (c->renormalize) {
        float s = 0.f;
        for (int r = 0; r < k; ++r) s += w[r];
        for (int r = 0; r < k; ++r) w[r] = w[r] / s;
    }
    for (int r = 0; r < k; ++r) w[r] = w[r] * c->routed_scale;
}

/* logits (fp32, h ascending) -> softmax -> top-k.  probs [B,M] and gap [B] are optional outputs;
 * gap[t] = p_(k) - p_(k+1), used to flag near-ties. */
void ewo_gate_topk(const ewo_cfg *c, int B, const uint16_t *x, const uint16_t *router_w,
                   int32_t *ids, float *w, float *probs, float *gap) {
    int H = c->H, M = c->M, k = c->k;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < B; ++t) {
        float *z = (float *)malloc(sizeof(float) * 2 * M);
        float *p = z + M;
        for (int j = 0; j < M; ++j) {
            float acc = 0.f;
            for (int h = 0; h < H; ++h) acc += bf(x[(size_t)t * H + h]) * bf(router_w[(size_t)j * H + h]);
            z[j] = acc;
        }
        softmax_topk(c, z, p, ids + (size_t)t * k, w + (size_t)t * k, gap ? gap + t : 0);
        if (probs) memcpy(probs + (size_t)t * M, p, sizeof(float) * M);
        free(z);
    }
}

/* same selection starting from given fp32 logits [B,M] (reroute-only workload) */
void ewo_topk_from_logits(const ewo_cfg *c, int B, const float *logits, int32_t *ids, float *w, float *gap) {
    int M = c->M, k = c->k;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < B; ++t) {
        float *p = (float *)malloc(sizeof(float) * M);
        softmax_topk(c, logits + (size_t)t * M, p, ids + (size_t)t * k, w + (size_t)t * k, gap ? gap + t : 0);
        free(p);
    }
}

/* y += scale * FFN(x) with one expert's matrices: g = Wg x, u = Wu x, a = silu(g)*u, y += scale * (Wd a) */
static void expert_ffn(const ewo_cfg *c, const float *xf, const uint16_t *wg, const uint16_t *wu,
                       const uint16_t *wd, float scale, float *act, float *y) {
    int H = c->H, I = c->I;
    for (int i = 0; i < I; ++i) {
        float g = 0.f, u = 0.f;
        const uint16_t *rg = wg + (size_t)i * H, *ru = wu + (size_t)i * H;
        for (int h = 0; h < H; ++h) g += bf(rg[h]) * xf[h];
        for (int h = 0; h < H; ++h) u += bf(ru[h]) * xf[h];
        act[i] = (g / (1.f + expf(-g))) * u;
    }
    for (int o = 0; o < H; ++o) {
        float d = 0.f;
        const uint16_t *rd = wd + (size_t)o * I;
        for (int i = 0; i < I; ++i) d += bf(rd[i]) * act[i];
        y[o] += scale * d;
    }
}

/* slot -> the three matrices stored there in the unified pool; 0 on success.
 * slot < M: base expert; else adapter i = (slot-M)/E_max, position d = (slot-M)%E_max, d < e_i. */
static int resolve_slot(const ewo_cfg *c, const ewo_layer *L, int slot, const uint16_t **wg,
                        const uint16_t **wu, const uint16_t **wd) {
    size_t sz = (size_t)c->I * c->H;
    if (slot < 0) return -1;
    if (slot < c->M) {
        *wg = L->w_gate + sz * slot; *wu = L->w_up + sz * slot; *wd = L->w_down + sz * slot;
        return 0;
    }
    int i = (slot - c->M) / c->E_max, d = (slot - c->M) % c->E_max;
    if (i >= c->N || d >= L->e[i]) return -2;     /* a padding slot: nothing is mapped there */
    *wg = L->a_gate[i] + sz * d; *wu = L->a_up[i] + sz * d; *wd = L->a_down[i] + sz * d;
    return 0;
}

/* out[t] = sum_r w[t,r] * FFN_{slot[t,r]}(x[t]) + sum_shared FFN(x[t]); r in the given order. */
int ewo_ffn_given_slots(const ewo_cfg *c, const ewo_layer *L, int B, const uint16_t *x,
                        const int32_t *slots, const float *w, float *out) {
    int H = c->H, I = c->I, k = c->k, err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int t = 0; t < B; ++t) {
        float *xf = (float *)malloc(sizeof(float) * (H + I));
        float *act = xf + H, *y = out + (size_t)t * H;
        for (int h = 0; h < H; ++h) { xf[h] = bf(x[(size_t)t * H + h]); y[h] = 0.f; }
        for (int r = 0; r < k; ++r) {
            const uint16_t *wg, *wu, *wd;
            if (resolve_slot(c, L, slots[t * k + r], &wg, &wu, &wd)) {
#pragma omp atomic write
                err = 1;
                continue;
            }
            expert_ffn(c, xf, wg, wu, wd, w[t * k + r], act, y);
        }
        size_t sz = (size_t)I * H;
        for (int s = 0; s < c->S; ++s)
            expert_ffn(c, xf, L->s_gate + sz * s, L->s_up + sz * s, L->s_down + sz * s, 1.f, act, y);
        free(xf);
    }
    return err ? -1 : 0;
}

/* Adapter-aware path.  ids/w/slots are optional outputs ([B,k]); Pi is [N,M]. */
int ewo_layer_forward(const ewo_cfg *c, const ewo_layer *L, int B, const uint16_t *x, const int32_t *aid,
                      const int32_t *Pi, float *out, int32_t *ids_out, float *w_out, int32_t *slots_out) {
    size_t n = (size_t)B * c->k;
    int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * n * 2);
    int32_t *slots = ids + n;
    float *w = (float *)malloc(sizeof(float) * n);
    ewo_gate_topk(c, B, x, L->router_w, ids, w, 0, 0);
    ewo_reroute(B, c->k, c->M, c->N, ids, aid, Pi, L->loaded, slots);
    int rc = ewo_ffn_given_slots(c, L, B, x, slots, w, out);
    if (ids_out) memcpy(ids_out, ids, sizeof(int32_t) * n);
    if (slots_out) memcpy(slots_out, slots, sizeof(int32_t) * n);
    if (w_out) memcpy(w_out, w, sizeof(float) * n);
    free(ids); free(w);
    return rc;
}

/* The definition: token t goes through the merged model of adapter aid[t] (base model if -1):
 * expert j's matrices are the adapter's copy when the adapter tunes j, otherwise the base ones. */
int ewo_layer_forward_merged(const ewo_cfg *c, const ewo_layer *L, int B, const uint16_t *x,
                             const int32_t *aid, float *out) {
    int H = c->H, I = c->I, k = c->k;
    size_t n = (size_t)B * k, sz = (size_t)I * H;
    int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * n);
    float *w = (float *)malloc(sizeof(float) * n);
    ewo_gate_topk(c, B, x, L->router_w, ids, w, 0, 0);
#pragma omp parallel for schedule(dynamic, 1)
    for (int t = 0; t < B; ++t) {
        float *xf = (float *)malloc(sizeof(float) * (H + I));
        float *act = xf + H, *y = out + (size_t)t * H;
        for (int h = 0; h < H; ++h) { xf[h] = bf(x[(size_t)t * H + h]); y[h] = 0.f; }
        int a = aid[t];
        for (int r = 0; r < k; ++r) {
            int j = ids[t * k + r];
            const uint16_t *wg = L->w_gate + sz * j, *wu = L->w_up + sz * j, *wd = L->w_down + sz * j;
            if (a >= 0 && a < c->N)
                for (int d = 0; d < L->e[a]; ++d)
                    if (L->tuned[a][d] == j) {
                        wg = L->a_gate[a] + sz * d; wu = L->a_up[a] + sz * d; wd = L->a_down[a] + sz * d;
                    }
            expert_ffn(c, xf, wg, wu, wd, w[t * k + r], act, y);
        }
        for (int s = 0; s < c->S; ++s)
            expert_ffn(c, xf, L->s_gate + sz * s, L->s_up + sz * s, L->s_down + sz * s, 1.f, act, y);
        free(xf);
    }
    free(ids); free(w);
    return 0;
}
