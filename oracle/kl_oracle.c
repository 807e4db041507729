/*
 * CPU oracle for one decode step of a decoder-only transformer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file defines what the CUDA path must compute;
 * it is never part of the product path and shares no code with it.  Only the
 * tests, the smoke check and the bench's CPU-baseline leg may call it.
 *
 * The paper (Sections 1-2) names the blocks of a decode step -- Embedding,
 * L x Decoder, Classifier, Sampling -- and the operators inside a decoder
 * (RMSNorm, GEMM, SDPA, SiLU) but prints no operator arithmetic.  The chain
 * implemented here is the standard pre-norm Llama block:
 *
 *   x = E[token]
 *   for l in 0..L-1:
 *     a = rmsnorm(x; g1[l]);  q,k,v = Wq a, Wk a, Wv a
 *     q,k = rope(q,k; position p)          (half-split pairing i <-> i + hd/2)
 *     cache[l].K[p] = bf16(k); cache[l].V[p] = bf16(v)
 *     o[hq] = softmax(q[hq] . K[g]^T / sqrt(hd)) V[g],  g = hq div (nq/nkv), over 0..p
 *     x = x + Wo o
 *     m = rmsnorm(x; g2[l]);  x = x + Wd (silu(Wg m) * (Wu m))
 *       (mixture-of-experts layers: r = Wr m; the top_k largest r_e, lowest index first among equals, chosen in
 *        descending order; their weights = softmax over the chosen logits;
 *        x = x + sum over the chosen e, in that order, of weight_e * Wd_e (silu(Wg_e m) * (Wu_e m)))
 *   hidden = x;  logits = Wlm rmsnorm(x; gf);  next = argmax(logits) (lowest index on ties)
 *
 * Precision: weights, gains, embedding and cached K/V are bf16 VALUES; every
 * other quantity is an IEEE double and every sum is accumulated in double, in
 * index order.  No blocking, fusion or reordering.  The only rounding steps are
 * the two bf16 stores into the KV cache.
 *
 * Accounting (Section 1, operation-intensity table): every routine adds the
 * multiply-accumulates it performs and the distinct parameter / KV bytes it
 * touches to a ko_counters record.  With count_only != 0 the loops are skipped
 * and only the counters advance, so the table's rows can be reproduced at
 * shapes far too large to execute.
 *
 * parity pins: see tests/test_oracle_pins.py (closed forms, invariants, brute
 * force, a library re-statement with torch CPU operators, the paper's table).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab, max_ctx;
    double rms_eps, rope_theta;
} ko_desc;

typedef struct {
    uint64_t macs;            /* multiply-accumulates in matrix products (linear layers + QK^T + PV) */
    uint64_t weight_bytes;    /* distinct parameter bytes read (matrices, gains) */
    uint64_t embed_bytes;     /* embedding rows read */
    uint64_t kv_read_bytes;   /* distinct KV-cache bytes read */
    uint64_t kv_write_bytes;  /* KV-cache bytes written */
} ko_counters;

typedef struct {
    const uint16_t *wq, *wk, *wv, *wo, *wgate, *wup, *wdown, *norm1, *norm2;
    const uint16_t *bq, *bk, *bv; /* optional biases of the q, k, v projections (NULL: none), bf16 */
    /* Mixture-of-experts MLP (n_experts > 0; the paper's Table 2 lists such a decoder, Mixtral 8x7B): a router matrix
     * [n_experts, hidden] and, per expert, gate / up [ffn, hidden] and down [hidden, ffn]; wgate / wup / wdown are then
     * unused.  n_experts == 0: the dense MLP above. */
    int32_t n_experts, top_k;
    const uint16_t *router;
    const uint16_t *const *ex_gate, *const *ex_up, *const *ex_down;
} ko_layer_weights;

/* ---------------------------------------------------------------- bf16 */

double ko_bf16_to_double(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* Nearest bf16 to a double, ties to even mantissa (decided in double, so no double rounding). */
uint16_t ko_bf16_rne(double v) {
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, 4);
    uint16_t c = (uint16_t)(u >> 16); /* truncation: |c| <= |v| up to float rounding */
    uint16_t cand[3];
    cand[0] = c;
    cand[1] = (uint16_t)(c + 1); /* next larger magnitude */
    cand[2] = (uint16_t)(c - 1); /* next smaller magnitude (c == 0 wraps; harmless, it loses) */
    uint16_t best = c;
    double bd = fabs(ko_bf16_to_double(c) - v);
    for (int i = 1; i < 3; ++i) {
        if ((cand[i] & 0x7F80) == 0x7F80) continue; /* inf/nan encodings */
        if (c == 0 && i == 2) continue;
        double d = fabs(ko_bf16_to_double(cand[i]) - v);
        if (d < bd || (d == bd && (cand[i] & 1) == 0 && (best & 1) == 1)) {
            bd = d;
            best = cand[i];
        }
    }
    return best;
}

/* ---------------------------------------------------------------- operators */

/* y[r] = sum_k W[r,k] x[k];  W row-major [R,K] bf16, no bias. */
void ko_matvec(const uint16_t *W, int R, int K, const double *x, double *y, ko_counters *c, int count_only) {
    if (c) {
        c->macs += (uint64_t)R * (uint64_t)K;
        c->weight_bytes += (uint64_t)R * (uint64_t)K * 2u;
    }
    if (count_only) return;
#pragma omp parallel for schedule(static)
    for (int r = 0; r < R; ++r) {
        const uint16_t *w = W + (size_t)r * (size_t)K;
        double acc = 0.0;
        for (int k = 0; k < K; ++k) acc += ko_bf16_to_double(w[k]) * x[k];
        y[r] = acc;
    }
}

/* y = x / sqrt(mean(x^2) + eps) * g   (eps inside the root, gain applied last). */
void ko_rmsnorm(const double *x, const uint16_t *g, int H, double eps, double *y, ko_counters *c, int count_only) {
    if (c) c->weight_bytes += (uint64_t)H * 2u;
    if (count_only) return;
    double ss = 0.0;
    for (int i = 0; i < H; ++i) ss += x[i] * x[i];
    double inv = 1.0 / sqrt(ss / (double)H + eps);
    for (int i = 0; i < H; ++i) y[i] = x[i] * inv * ko_bf16_to_double(g[i]);
}

/* Rotary embedding of one head vector u[hd] at position p, in place (half-split pairing). */
void ko_rope(double *u, int hd, int p, double theta) {
    int half = hd / 2;
    for (int i = 0; i < half; ++i) {
        double ang = (double)p * pow(theta, -2.0 * (double)i / (double)hd);
        double cs = cos(ang), sn = sin(ang);
        double a = u[i], b = u[i + half];
        u[i] = a * cs - b * sn;
        u[i + half] = b * cs + a * sn;
    }
}

/* w = softmax(s) over n entries (subtract max, exponentiate, normalise). */
void ko_softmax(const double *s, int n, double *w) {
    double mx = s[0];
    for (int j = 1; j < n; ++j)
        if (s[j] > mx) mx = s[j];
    double sum = 0.0;
    for (int j = 0; j < n; ++j) {
        w[j] = exp(s[j] - mx);
        sum += w[j];
    }
    for (int j = 0; j < n; ++j) w[j] /= sum;
}

double ko_silu(double z) { return z / (1.0 + exp(-z)); }

/* One query head against n cached positions of one KV head.
 * K, V: [n][hd] bf16 rows with row stride `stride` elements.  out[hd]. */
void ko_attention_head(const double *q, const uint16_t *K, const uint16_t *V, int n, int hd, size_t stride,
                       double *out, double *scratch /* 2n doubles */) {
    double *s = scratch, *w = scratch + n;
    double scale = 1.0 / sqrt((double)hd);
    for (int j = 0; j < n; ++j) {
        const uint16_t *kr = K + (size_t)j * stride;
        double acc = 0.0;
        for (int d = 0; d < hd; ++d) acc += q[d] * ko_bf16_to_double(kr[d]);
        s[j] = acc * scale;
    }
    ko_softmax(s, n, w);
    for (int d = 0; d < hd; ++d) {
        double acc = 0.0;
        for (int j = 0; j < n; ++j) acc += w[j] * ko_bf16_to_double(V[(size_t)j * stride + d]);
        out[d] = acc;
    }
}

/* Router of a mixture-of-experts layer: the k largest of E logits in descending order (among equal logits the lower
 * index first), and the softmax over those k as their weights.  Equal to a softmax over all E followed by top-k and
 * renormalisation. */
void ko_moe_route(const double *logits, int E, int k, int32_t *idx, double *w) {
    double chosen[64];
    for (int s = 0; s < k; ++s) {
        int best = -1;
        for (int e = 0; e < E; ++e) {
            int taken = 0;
            for (int t = 0; t < s; ++t)
                if (idx[t] == e) taken = 1;
            if (taken) continue;
            if (best < 0 || logits[e] > logits[best]) best = e;
        }
        idx[s] = best;
        chosen[s] = logits[best];
    }
    ko_softmax(chosen, k, w);
}

/* ---------------------------------------------------------------- blocks */

/* Embedding block: x = E[token]. */
void ko_embed(const ko_desc *d, const uint16_t *E, int token, double *x, ko_counters *c, int count_only) {
    if (c) c->embed_bytes += (uint64_t)d->hidden * 2u;
    if (count_only) return;
    for (int i = 0; i < d->hidden; ++i) x[i] = ko_bf16_to_double(E[(size_t)token * (size_t)d->hidden + i]);
}

/* Same, from a single already-extracted row. */
void ko_embed_row(const ko_desc *d, const uint16_t *row, double *x, ko_counters *c, int count_only) {
    ko_embed(d, row, 0, x, c, count_only);
}

/* Decoder block l for one sequence.
 * kcache, vcache: this layer's and this sequence's slices, [n_kv_heads][max_ctx][head_dim] bf16.
 * p = number of valid cached positions = index written by this step; attention covers 0..p.
 * x[hidden] is updated in place.  Returns 0, or -1 on bad arguments / allocation failure. */
int ko_decoder_layer(const ko_desc *d, const ko_layer_weights *w, uint16_t *kcache, uint16_t *vcache, int p, double *x,
                     ko_counters *c, int count_only) {
    const int H = d->hidden, nq = d->n_q_heads, nkv = d->n_kv_heads, hd = d->head_dim, F = d->ffn;
    if (p < 0 || p >= d->max_ctx || nq % nkv != 0 || hd % 2 != 0) return -1;
    const int G = nq / nkv, n = p + 1;
    const size_t head_stride = (size_t)d->max_ctx * (size_t)hd;

    double *a = NULL, *q = NULL, *k = NULL, *v = NULL, *o = NULL, *t = NULL, *gate = NULL, *up = NULL, *sc = NULL;
    if (!count_only) {
        a = malloc(sizeof(double) * H);
        q = malloc(sizeof(double) * nq * hd);
        k = malloc(sizeof(double) * nkv * hd);
        v = malloc(sizeof(double) * nkv * hd);
        o = malloc(sizeof(double) * nq * hd);
        t = malloc(sizeof(double) * H);
        gate = malloc(sizeof(double) * F);
        up = malloc(sizeof(double) * F);
        sc = malloc(sizeof(double) * 2 * (size_t)n * (size_t)nq);
        if (!a || !q || !k || !v || !o || !t || !gate || !up || !sc) return -1;
    }

    /* attention half */
    ko_rmsnorm(x, w->norm1, H, d->rms_eps, a, c, count_only);
    ko_matvec(w->wq, nq * hd, H, a, q, c, count_only);
    ko_matvec(w->wk, nkv * hd, H, a, k, c, count_only);
    ko_matvec(w->wv, nkv * hd, H, a, v, c, count_only);
    /* q, k, v = W a + b for decoders with projection biases; the bias is added before the rotation */
    if (w->bq && !count_only) for (int i = 0; i < nq * hd; ++i) q[i] += ko_bf16_to_double(w->bq[i]);
    if (w->bk && !count_only) for (int i = 0; i < nkv * hd; ++i) k[i] += ko_bf16_to_double(w->bk[i]);
    if (w->bv && !count_only) for (int i = 0; i < nkv * hd; ++i) v[i] += ko_bf16_to_double(w->bv[i]);
    if (c && w->bq) c->weight_bytes += (uint64_t)2 * (uint64_t)(nq + 2 * nkv) * hd;
    if (c) {
        c->kv_write_bytes += (uint64_t)2 * nkv * hd * 2u;
        c->kv_read_bytes += (uint64_t)2 * nkv * (uint64_t)n * hd * 2u; /* each cached row once */
        c->macs += (uint64_t)2 * (uint64_t)n * (uint64_t)nq * hd;      /* QK^T and PV */
    }
    if (!count_only) {
        for (int h = 0; h < nq; ++h) ko_rope(q + (size_t)h * hd, hd, p, d->rope_theta);
        for (int g = 0; g < nkv; ++g) {
            ko_rope(k + (size_t)g * hd, hd, p, d->rope_theta);
            for (int e = 0; e < hd; ++e) {
                kcache[(size_t)g * head_stride + (size_t)p * hd + e] = ko_bf16_rne(k[(size_t)g * hd + e]);
                vcache[(size_t)g * head_stride + (size_t)p * hd + e] = ko_bf16_rne(v[(size_t)g * hd + e]);
            }
        }
#pragma omp parallel for schedule(static)
        for (int h = 0; h < nq; ++h) {
            int g = h / G;
            ko_attention_head(q + (size_t)h * hd, kcache + (size_t)g * head_stride, vcache + (size_t)g * head_stride, n,
                              hd, (size_t)hd, o + (size_t)h * hd, sc + (size_t)h * 2 * (size_t)n);
        }
    }
    ko_matvec(w->wo, H, nq * hd, o, t, c, count_only);
    if (!count_only)
        for (int i = 0; i < H; ++i) x[i] += t[i];

    /* MLP half */
    ko_rmsnorm(x, w->norm2, H, d->rms_eps, a, c, count_only);
    if (w->n_experts > 0) {
        const int E = w->n_experts, K = w->top_k;
        if (K < 1 || K > E || E > 64) return -1;
        double r[64], wt[64];
        int32_t idx[64];
        ko_matvec(w->router, E, H, a, r, c, count_only);
        if (!count_only) ko_moe_route(r, E, K, idx, wt);
        for (int s = 0; s < K; ++s) {
            const int e = count_only ? 0 : idx[s];
            ko_matvec(count_only ? NULL : w->ex_gate[e], F, H, a, gate, c, count_only);
            ko_matvec(count_only ? NULL : w->ex_up[e], F, H, a, up, c, count_only);
            if (!count_only)
                for (int f = 0; f < F; ++f) gate[f] = ko_silu(gate[f]) * up[f];
            ko_matvec(count_only ? NULL : w->ex_down[e], H, F, gate, t, c, count_only);
            if (!count_only)
                for (int i = 0; i < H; ++i) x[i] += wt[s] * t[i];
        }
    } else {
        ko_matvec(w->wgate, F, H, a, gate, c, count_only);
        ko_matvec(w->wup, F, H, a, up, c, count_only);
        if (!count_only)
            for (int f = 0; f < F; ++f) gate[f] = ko_silu(gate[f]) * up[f];
        ko_matvec(w->wdown, H, F, gate, t, c, count_only);
        if (!count_only)
            for (int i = 0; i < H; ++i) x[i] += t[i];
    }

    free(a); free(q); free(k); free(v); free(o); free(t); free(gate); free(up); free(sc);
    return 0;
}

/* Classifier block: logits = Wlm rmsnorm(x; gf). */
int ko_classifier(const ko_desc *d, const uint16_t *norm_f, const uint16_t *lm_head, const double *x, double *logits,
                  ko_counters *c, int count_only) {
    double *a = NULL;
    if (!count_only) {
        a = malloc(sizeof(double) * d->hidden);
        if (!a) return -1;
    }
    ko_rmsnorm(x, norm_f, d->hidden, d->rms_eps, a, c, count_only);
    ko_matvec(lm_head, d->vocab, d->hidden, a, logits, c, count_only);
    free(a);
    return 0;
}

/* Sampling block (greedy): index of the largest logit, lowest index on ties. */
int ko_argmax(const double *logits, int n) {
    int best = 0;
    for (int i = 1; i < n; ++i)
        if (logits[i] > logits[best]) best = i;
    return best;
}

int ko_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
