/*
 * River-LLM decode-with-exit: the CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, step-by-step CPU statement of
 * what the token-level early-exit decode step computes.  Only the tests, the smoke check
 * and the benchmark's cpu_baseline / reference legs may build or call it; the product
 * (the CUDA library) shares no code, header, table or helper with it.
 *
 * What it follows (River-LLM paper):
 *   - Section 4.1 "KV-Shared Exit Layer": every exit (river) layer is a copy of its
 *     backbone decoder block whose Attention and FFN weights are 4-bit weight-only
 *     quantised, and it uses the *same KV cache addressing* as the backbone block, so
 *     the K/V of bypassed backbone layers appear in the backbone's own slots as a
 *     by-product of running the river.
 *   - Section 4.2 "Inference with Seamless Exit", Eq. 1: after backbone block l the
 *     state-transition similarity s = cos(h^(l-1), h^(l)) is compared with the threshold
 *     tau (strict >); on exit the remaining depth runs in the river and ends at the
 *     original LM head.  Prefill uses one unified exit depth for all prompt tokens,
 *     generation exits per token.
 *
 * Arithmetic: weights are the given bf16 / packed-u4 inputs, values are stored as fp32,
 * every reduction (dot products, norms, softmax sums) accumulates in fp64.  The exit
 * comparison is taken on the fp32-rounded score, strict ">" (NaN never exits; a zero
 * norm gives s = 0).
 *
 * Pins (tests/test_oracle_*.py): full-depth equivalence with the separate plain decoder
 * below, a no-cache brute-force recompute written in numpy, the identity-river
 * invariance, cache completeness, monotonicity in tau, closed forms of Eq. 1, textbook
 * attention / RoPE special cases, the cache-size figure of the paper's memory table, and
 * the 4-bit grid bounds.  The paper's accuracy figures (match rate, KV cosine >= 0.97,
 * r = 0.5536) need trained checkpoints and datasets: parity unpinned for those.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t L, d, Hq, Hkv, dh, F, V;
    float rms_eps, rope_theta;
    int32_t entry_layer; /* L_s: first block after which an exit may be taken */
    int32_t group;       /* quantisation group along the input dimension */
    int32_t max_seqs, max_len;
    int32_t exit_mode;   /* 0 = per token, 1 = whole batch switches together (Eq. 1 literal) */
    int32_t kv_store;    /* 0 = cache holds fp32 values; 1 = cache entries are rounded to bf16 when stored: the
                            method keeps the KV cache in a 16-bit format (Section 4.1) */
    int32_t kv_strategy; /* what happens in the blocks a token skips (Section 3, the strategies the method is compared
                            with): 0 = the KV-Shared Exit River (Section 4.1: the quantised copy of the block runs and
                            writes K/V into the shared slot); 1 = State Propagation: the hidden state at the exit is the
                            input of every later block's K/V projection (backbone weights), nothing else runs there;
                            2 = Mono-Decreasing Exit: nothing runs in a skipped block, and a token leaves no later than
                            the previous token of its sequence did, so no cache entry it needs is ever missing;
                            3 = KV Mask: nothing runs in a skipped block, and a later token's attention in block l sees
                            only the positions whose token ran block l (and itself) */
} orc_config;

/* backbone pointers per layer: attn_norm, wq, wk, wv, wo, ffn_norm, wg, wu, wd (all bf16) */
enum { BB_ATTN_NORM, BB_WQ, BB_WK, BB_WV, BB_WO, BB_FFN_NORM, BB_WG, BB_WU, BB_WD, BB_N };
/* river pointers per layer: for each of the 7 matrices (q,k,v,o,g,u,d): codes, scale, zero */
enum { RV_N = 21 };

typedef struct {
    orc_config c;
    const uint16_t *embed, *lm_head, *final_norm;
    const void **bb; /* [L][BB_N] */
    const void **rv; /* [L][RV_N], all NULL for a layer without a river copy */
    float *K, *V;    /* [L][max_seqs][max_len][Hkv*dh] */
    uint8_t *written;/* [L][max_seqs][max_len] number of writes (saturating) */
    int32_t *len;    /* [max_seqs] */
    int32_t *cap;    /* [max_seqs] Mono-Decreasing Exit: the depth the sequence's last token reached (L to begin with) */
    uint8_t *depth;  /* [max_seqs][max_len] KV Mask: number of backbone blocks the token at each position ran */
    /* lists of the last decode step: rows in the backbone / in the river entering layer l (1-based) */
    int32_t *act_idx, *riv_idx, *n_act, *n_riv; /* [(L+1)][maxB], [(L+1)] */
    int32_t lists_cap;
} orc_ctx;

/* round an fp32 value to the nearest bf16 (ties to even) and return it as fp32 */
static inline float round_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return f; /* inf / nan unchanged */
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return f;
}

static inline float bf16_to_f32(uint16_t v) {
    uint32_t u = ((uint32_t)v) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* a projection matrix in either representation */
typedef struct {
    const uint16_t *w;     /* bf16 [out][in] or NULL */
    const uint8_t *codes;  /* u8 [out][in/2], low nibble = even input index */
    const uint16_t *scale; /* bf16 [out][in/G] */
    const uint16_t *zero;  /* bf16 [out][in/G] */
    int G;
} mat_t;

/* y[o] = sum_k W[o][k] x[k]; river weights dequantise as w = (q - z) * s (Section 4.1: W4A16) */
static void matvec(const mat_t *m, int out, int in, const float *x, float *y) {
    if (m->w) {
#pragma omp parallel for schedule(static)
        for (int o = 0; o < out; ++o) {
            const uint16_t *row = m->w + (size_t)o * in;
            double acc = 0.0;
#pragma omp simd reduction(+ : acc)
            for (int k = 0; k < in; ++k) acc += (double)bf16_to_f32(row[k]) * (double)x[k];
            y[o] = (float)acc;
        }
    } else {
        const int G = m->G, ng = in / G;
#pragma omp parallel for schedule(static)
        for (int o = 0; o < out; ++o) {
            const uint8_t *row = m->codes + (size_t)o * (in / 2);
            double acc = 0.0;
            for (int g = 0; g < ng; ++g) {
                const float s = bf16_to_f32(m->scale[(size_t)o * ng + g]);
                const float z = bf16_to_f32(m->zero[(size_t)o * ng + g]);
                for (int k = g * G; k < (g + 1) * G; ++k) {
                    const int q = (k & 1) ? (row[k >> 1] >> 4) : (row[k >> 1] & 15);
                    const float w = ((float)q - z) * s;
                    acc += (double)w * (double)x[k];
                }
            }
            y[o] = (float)acc;
        }
    }
}

static void rmsnorm(const float *h, const uint16_t *gain, int d, float eps, float *x) {
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += (double)h[i] * (double)h[i];
    const double r = 1.0 / sqrt(ss / d + (double)eps);
    for (int i = 0; i < d; ++i) x[i] = (float)((double)h[i] * r * (double)bf16_to_f32(gain[i]));
}

/* rotate-half RoPE on one head vector: pairs (i, i + dh/2), angle = pos * theta^(-2i/dh) */
static void rope(float *v, int dh, int pos, float theta) {
    const int half = dh / 2;
    for (int i = 0; i < half; ++i) {
        const double ang = (double)pos * pow((double)theta, -2.0 * i / dh);
        const double c = cos(ang), s = sin(ang);
        const double a = v[i], b = v[i + half];
        v[i] = (float)(a * c - b * s);
        v[i + half] = (float)(b * c + a * s);
    }
}

static size_t kv_off(const orc_ctx *o, int l0, int slot, int pos) {
    const orc_config *c = &o->c;
    return (((size_t)l0 * c->max_seqs + slot) * c->max_len + pos) * ((size_t)c->Hkv * c->dh);
}

static void get_mats(const orc_ctx *o, int l0, int river, mat_t m[7]) {
    static const int bbi[7] = {BB_WQ, BB_WK, BB_WV, BB_WO, BB_WG, BB_WU, BB_WD};
    for (int j = 0; j < 7; ++j) {
        memset(&m[j], 0, sizeof(mat_t));
        m[j].G = o->c.group;
        if (!river) {
            m[j].w = (const uint16_t *)o->bb[l0 * BB_N + bbi[j]];
        } else {
            m[j].codes = (const uint8_t *)o->rv[l0 * RV_N + 3 * j + 0];
            m[j].scale = (const uint16_t *)o->rv[l0 * RV_N + 3 * j + 1];
            m[j].zero = (const uint16_t *)o->rv[l0 * RV_N + 3 * j + 2];
        }
    }
}

/*
 * Causal GQA attention for one row: query heads q [Hq][dh] (already rotated) against the
 * cached positions 0..pos of sequence slot at layer l0; head i reads kv head i/(Hq/Hkv);
 * att [Hq][dh] = softmax_p(q_i . K_p / sqrt(dh)) . V_p.
 * KV Mask (kv_strategy 3, Section 3): an earlier position whose token did not run block l0 + 1 has no K/V there and is
 * invisible (the softmax runs over the other positions; the row's own position is always among them).
 */
static void attend(const orc_ctx *o, int l0, int slot, int pos, const float *q, float *att) {
    const orc_config *c = &o->c;
    const int Hq = c->Hq, dh = c->dh, grp = c->Hq / c->Hkv;
    const double scale = 1.0 / sqrt((double)dh);
    const uint8_t *depth = c->kv_strategy == 3 ? o->depth + (size_t)slot * c->max_len : NULL;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < Hq; ++i) {
        const int kvh = i / grp;
        double *sc = (double *)malloc(sizeof(double) * (size_t)(pos + 1));
        double mx = -INFINITY;
        for (int p = 0; p <= pos; ++p) {
            if (depth && p < pos && depth[p] < l0 + 1) { sc[p] = -INFINITY; continue; }
            const float *kp = o->K + kv_off(o, l0, slot, p) + (size_t)kvh * dh;
            double a = 0.0;
            for (int e = 0; e < dh; ++e) a += (double)q[(size_t)i * dh + e] * (double)kp[e];
            sc[p] = a * scale;
            if (sc[p] > mx) mx = sc[p];
        }
        double den = 0.0;
        for (int p = 0; p <= pos; ++p) {
            sc[p] = exp(sc[p] - mx);  /* exactly 0 for an invisible position */
            den += sc[p];
        }
        for (int e = 0; e < dh; ++e) {
            double a = 0.0;
            for (int p = 0; p <= pos; ++p)
                if (sc[p] != 0.0) a += sc[p] * (double)(o->V + kv_off(o, l0, slot, p))[(size_t)kvh * dh + e];
            att[(size_t)i * dh + e] = (float)(a / den);
        }
        free(sc);
    }
}

/*
 * One decoder block (0-based layer l0) on one row: h (in) -> h_out, for the token at
 * position pos of sequence slot.  river != 0 selects the quantised copy; the norms are
 * shared and the K/V go to the same cache slot either way (Section 4.1).
 */
static void block(orc_ctx *o, int l0, int river, int slot, int pos, const float *h, float *h_out) {
    const orc_config *c = &o->c;
    const int d = c->d, Hq = c->Hq, Hkv = c->Hkv, dh = c->dh, F = c->F;
    mat_t m[7];
    get_mats(o, l0, river, m);
    float *x = (float *)malloc(sizeof(float) * (size_t)(d > F ? d : F));
    float *q = (float *)malloc(sizeof(float) * (size_t)Hq * dh);
    float *att = (float *)malloc(sizeof(float) * (size_t)Hq * dh);
    float *hmid = (float *)malloc(sizeof(float) * (size_t)d);
    float *tmp = (float *)malloc(sizeof(float) * (size_t)d);
    float *gate = (float *)malloc(sizeof(float) * (size_t)F);
    float *up = (float *)malloc(sizeof(float) * (size_t)F);

    rmsnorm(h, (const uint16_t *)o->bb[l0 * BB_N + BB_ATTN_NORM], d, c->rms_eps, x);
    float *kdst = o->K + kv_off(o, l0, slot, pos);
    float *vdst = o->V + kv_off(o, l0, slot, pos);
    matvec(&m[0], Hq * dh, d, x, q);
    matvec(&m[1], Hkv * dh, d, x, kdst);
    matvec(&m[2], Hkv * dh, d, x, vdst);
    for (int i = 0; i < Hq; ++i) rope(q + (size_t)i * dh, dh, pos, c->rope_theta);
    for (int j = 0; j < Hkv; ++j) rope(kdst + (size_t)j * dh, dh, pos, c->rope_theta);
    if (c->kv_store == 1)
        for (int i = 0; i < Hkv * dh; ++i) { kdst[i] = round_to_bf16(kdst[i]); vdst[i] = round_to_bf16(vdst[i]); }
    {
        uint8_t *w = &o->written[((size_t)l0 * c->max_seqs + slot) * c->max_len + pos];
        if (*w < 255) ++*w;
    }

    attend(o, l0, slot, pos, q, att);

    matvec(&m[3], d, Hq * dh, att, tmp);
    for (int i = 0; i < d; ++i) hmid[i] = h[i] + tmp[i];
    rmsnorm(hmid, (const uint16_t *)o->bb[l0 * BB_N + BB_FFN_NORM], d, c->rms_eps, x);
    matvec(&m[4], F, d, x, gate);
    matvec(&m[5], F, d, x, up);
    for (int i = 0; i < F; ++i) {
        const double g = gate[i];
        gate[i] = (float)(g / (1.0 + exp(-g)) * (double)up[i]);
    }
    matvec(&m[6], d, F, gate, tmp);
    for (int i = 0; i < d; ++i) h_out[i] = hmid[i] + tmp[i];

    free(x); free(q); free(att); free(hmid); free(tmp); free(gate); free(up);
}

/*
 * State Propagation (Section 3): block l0 + 1 is skipped, but its K/V for this position are computed from the hidden
 * state the token left the backbone with - that block's attention norm and its backbone K / V projections - and
 * stored in the block's cache slot.  No attention, no feed-forward: the hidden state itself is unchanged.
 */
static void propagate_kv(orc_ctx *o, int l0, int slot, int pos, const float *h) {
    const orc_config *c = &o->c;
    const int d = c->d, Hkv = c->Hkv, dh = c->dh;
    mat_t m[7];
    get_mats(o, l0, 0, m);
    float *x = (float *)malloc(sizeof(float) * (size_t)d);
    rmsnorm(h, (const uint16_t *)o->bb[l0 * BB_N + BB_ATTN_NORM], d, c->rms_eps, x);
    float *kdst = o->K + kv_off(o, l0, slot, pos);
    float *vdst = o->V + kv_off(o, l0, slot, pos);
    matvec(&m[1], Hkv * dh, d, x, kdst);
    matvec(&m[2], Hkv * dh, d, x, vdst);
    for (int j = 0; j < Hkv; ++j) rope(kdst + (size_t)j * dh, dh, pos, c->rope_theta);
    if (c->kv_store == 1)
        for (int i = 0; i < Hkv * dh; ++i) { kdst[i] = round_to_bf16(kdst[i]); vdst[i] = round_to_bf16(vdst[i]); }
    uint8_t *w = &o->written[((size_t)l0 * c->max_seqs + slot) * c->max_len + pos];
    if (*w < 255) ++*w;
    free(x);
}

/* Eq. 1: s = <a,b> / (|a| |b|); zero norm -> 0 */
static float transition_similarity(const float *a, const float *b, int d) {
    double ab = 0.0, aa = 0.0, bb = 0.0;
    for (int i = 0; i < d; ++i) {
        ab += (double)a[i] * (double)b[i];
        aa += (double)a[i] * (double)a[i];
        bb += (double)b[i] * (double)b[i];
    }
    if (aa == 0.0 || bb == 0.0) return 0.0f;
    return (float)(ab / (sqrt(aa) * sqrt(bb)));
}

static void lm_head(const orc_ctx *o, const float *h, float *logits, int32_t *next) {
    const orc_config *c = &o->c;
    float *x = (float *)malloc(sizeof(float) * (size_t)c->d);
    float *lg = logits ? logits : (float *)malloc(sizeof(float) * (size_t)c->V);
    rmsnorm(h, o->final_norm, c->d, c->rms_eps, x);
    mat_t m;
    memset(&m, 0, sizeof m);
    m.w = o->lm_head;
    matvec(&m, c->V, c->d, x, lg);
    int best = 0;
    for (int v = 1; v < c->V; ++v)
        if (lg[v] > lg[best]) best = v; /* greedy; ties -> lowest id */
    *next = best;
    if (!logits) free(lg);
    free(x);
}

static void embed_row(const orc_ctx *o, int tok, float *h) {
    const uint16_t *e = o->embed + (size_t)tok * o->c.d;
    for (int i = 0; i < o->c.d; ++i) h[i] = bf16_to_f32(e[i]);
}

/* ------------------------------------------------------------------ public API */

orc_ctx *orc_create(const orc_config *cfg, const void *embed, const void *lm_head_w, const void *final_norm,
                    const void **bb, const void **rv) {
    if (!cfg || cfg->L <= 0 || cfg->Hq % cfg->Hkv || cfg->dh % 2 || cfg->d % cfg->group || cfg->F % cfg->group ||
        (cfg->Hq * cfg->dh) % cfg->group || cfg->entry_layer < 0 || cfg->entry_layer >= cfg->L)
        return NULL;
    orc_ctx *o = (orc_ctx *)calloc(1, sizeof(orc_ctx));
    o->c = *cfg;
    o->embed = (const uint16_t *)embed;
    o->lm_head = (const uint16_t *)lm_head_w;
    o->final_norm = (const uint16_t *)final_norm;
    o->bb = (const void **)malloc(sizeof(void *) * (size_t)cfg->L * BB_N);
    o->rv = (const void **)malloc(sizeof(void *) * (size_t)cfg->L * RV_N);
    memcpy(o->bb, bb, sizeof(void *) * (size_t)cfg->L * BB_N);
    memcpy(o->rv, rv, sizeof(void *) * (size_t)cfg->L * RV_N);
    const size_t n = (size_t)cfg->L * cfg->max_seqs * cfg->max_len;
    o->K = (float *)calloc(n * cfg->Hkv * cfg->dh, sizeof(float));
    o->V = (float *)calloc(n * cfg->Hkv * cfg->dh, sizeof(float));
    o->written = (uint8_t *)calloc(n, 1);
    o->len = (int32_t *)calloc((size_t)cfg->max_seqs, sizeof(int32_t));
    o->cap = (int32_t *)malloc(sizeof(int32_t) * (size_t)cfg->max_seqs);
    if (!o->K || !o->V || !o->written || !o->cap) return NULL;
    for (int s = 0; s < cfg->max_seqs; ++s) o->cap[s] = cfg->L;
    if (cfg->kv_strategy < 0 || cfg->kv_strategy > 3 || cfg->L > 255) return NULL;
    o->depth = (uint8_t *)calloc((size_t)cfg->max_seqs * cfg->max_len, 1);
    if (!o->depth) return NULL;
    return o;
}

void orc_destroy(orc_ctx *o) {
    if (!o) return;
    free(o->K); free(o->V); free(o->written); free(o->len); free(o->cap); free(o->depth);
    free((void *)o->bb); free((void *)o->rv);
    free(o->act_idx); free(o->riv_idx); free(o->n_act); free(o->n_riv);
    free(o);
}

int orc_seq_len(const orc_ctx *o, int slot) { return o->len[slot]; }
void orc_set_len(orc_ctx *o, int slot, int n) { o->len[slot] = n; }
void orc_release(orc_ctx *o, int slot) {
    o->len[slot] = 0;
    o->cap[slot] = o->c.L;
    for (int l = 0; l < o->c.L; ++l)
        memset(&o->written[((size_t)l * o->c.max_seqs + slot) * o->c.max_len], 0, (size_t)o->c.max_len);
}
int orc_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static int river_exists(const orc_ctx *o, int l0) { return o->rv[l0 * RV_N] != NULL; }

/*
 * One token-level early-exit decode step (Section 4.2).  Row b feeds token tok[b] at
 * position len[slots[b]] of its sequence.  forced_exit (may be NULL) is a test hook:
 * forced_exit[b] >= 0 replaces the score test by "exit after block forced_exit[b]"
 * (L = never, 0 = river from the first block on, which needs entry_layer == 0).
 * Outputs: logits [B][V] (may be NULL), next_tok [B], exit_layer [B] = number of
 * backbone blocks run, scores [B][L] (may be NULL; NaN where no score was taken).
 * Returns 0, or a negative code on a bad argument.
 */
int orc_decode_step(orc_ctx *o, int B, const int32_t *slots, const int32_t *tok, const float *tau,
                    const int32_t *forced_exit, float *logits, int32_t *next_tok, int32_t *exit_layer,
                    float *scores) {
    const orc_config *c = &o->c;
    const int L = c->L, d = c->d;
    if (B <= 0) return -1;
    for (int b = 0; b < B; ++b) {
        if (slots[b] < 0 || slots[b] >= c->max_seqs || o->len[slots[b]] >= c->max_len) return -2;
        if (tok[b] < 0 || tok[b] >= c->V) return -3;
        for (int b2 = 0; b2 < b; ++b2)
            if (slots[b2] == slots[b]) return -4;
        if (forced_exit && forced_exit[b] >= 0) {
            if (forced_exit[b] > L || forced_exit[b] < c->entry_layer) return -5;
        }
    }
    if (o->lists_cap < B) {
        free(o->act_idx); free(o->riv_idx); free(o->n_act); free(o->n_riv);
        o->act_idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)(L + 1) * B);
        o->riv_idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)(L + 1) * B);
        o->n_act = (int32_t *)malloc(sizeof(int32_t) * (size_t)(L + 1));
        o->n_riv = (int32_t *)malloc(sizeof(int32_t) * (size_t)(L + 1));
        o->lists_cap = B;
    }
    float *h = (float *)malloc(sizeof(float) * (size_t)B * d);
    float *h2 = (float *)malloc(sizeof(float) * (size_t)B * d);
    uint8_t *exited = (uint8_t *)calloc((size_t)B, 1);
    float *s_now = (float *)malloc(sizeof(float) * (size_t)B);
    for (int b = 0; b < B; ++b) {
        embed_row(o, tok[b], h + (size_t)b * d);
        exit_layer[b] = L;
        if (forced_exit && forced_exit[b] == 0) { exited[b] = 1; exit_layer[b] = 0; }
        if (scores) for (int l = 0; l < L; ++l) scores[(size_t)b * L + l] = NAN;
    }
    for (int l = 1; l <= L; ++l) {
        /* the two row lists entering block l, ascending (what a stream compaction must produce) */
        int na = 0, nr = 0;
        for (int b = 0; b < B; ++b) {
            if (exited[b]) o->riv_idx[(size_t)(l - 1) * o->lists_cap + nr++] = b;
            else o->act_idx[(size_t)(l - 1) * o->lists_cap + na++] = b;
        }
        o->n_act[l - 1] = na; o->n_riv[l - 1] = nr;
        for (int b = 0; b < B; ++b) {
            if (exited[b] && c->kv_strategy != 0) {  /* a skipped block under one of the other strategies (2, 3: nothing) */
                if (c->kv_strategy == 1) propagate_kv(o, l - 1, slots[b], o->len[slots[b]], h + (size_t)b * d);
                memcpy(h2 + (size_t)b * d, h + (size_t)b * d, sizeof(float) * (size_t)d);
                continue;
            }
            if (exited[b] && !river_exists(o, l - 1)) { free(h); free(h2); free(exited); free(s_now); return -6; }
            block(o, l - 1, exited[b], slots[b], o->len[slots[b]], h + (size_t)b * d, h2 + (size_t)b * d);
        }
        /* exit evaluation on h^(l-1) -> h^(l), before the next block; only for rows still in the backbone */
        int all_pass = 1, any_active = 0;
        for (int b = 0; b < B; ++b) {
            s_now[b] = NAN;
            if (exited[b]) continue;
            any_active = 1;
            s_now[b] = transition_similarity(h + (size_t)b * d, h2 + (size_t)b * d, d);
            if (scores) scores[(size_t)b * L + (l - 1)] = s_now[b];
            if (!(s_now[b] > tau[b])) all_pass = 0;
        }
        for (int b = 0; b < B; ++b) {
            if (exited[b]) continue;
            int leave;
            if (forced_exit && forced_exit[b] >= 0) {
                leave = (forced_exit[b] == l) && (l < L);
            } else {
                const int eligible = (l >= c->entry_layer) && (l < L) && (l >= 1);
                if (c->exit_mode == 0) leave = eligible && (s_now[b] > tau[b]);
                else leave = eligible && any_active && all_pass;
            }
            /* Mono-Decreasing Exit: never deeper than the sequence's previous token */
            if (c->kv_strategy == 2 && l < L && l >= o->cap[slots[b]]) leave = 1;
            if (leave) { exited[b] = 1; exit_layer[b] = l; }
        }
        float *t = h; h = h2; h2 = t;
    }
    {
        int na = 0, nr = 0;
        for (int b = 0; b < B; ++b) {
            if (exited[b]) o->riv_idx[(size_t)L * o->lists_cap + nr++] = b;
            else o->act_idx[(size_t)L * o->lists_cap + na++] = b;
        }
        o->n_act[L] = na; o->n_riv[L] = nr;
    }
    for (int b = 0; b < B; ++b) {
        lm_head(o, h + (size_t)b * d, logits ? logits + (size_t)b * c->V : NULL, &next_tok[b]);
        o->len[slots[b]] += 1;
        if (c->kv_strategy == 2) o->cap[slots[b]] = exit_layer[b];
        o->depth[(size_t)slots[b] * c->max_len + (o->len[slots[b]] - 1)] = (uint8_t)exit_layer[b];
    }
    free(h); free(h2); free(exited); free(s_now);
    return 0;
}

/* lists of the last decode step: act/riv [(L+1)][B] (row-major with stride B), counts [(L+1)] */
void orc_last_lists(const orc_ctx *o, int B, int32_t *act, int32_t *n_act, int32_t *riv, int32_t *n_riv) {
    for (int l = 0; l <= o->c.L; ++l) {
        n_act[l] = o->n_act[l]; n_riv[l] = o->n_riv[l];
        for (int i = 0; i < B; ++i) {
            act[(size_t)l * B + i] = i < o->n_act[l] ? o->act_idx[(size_t)l * o->lists_cap + i] : -1;
            riv[(size_t)l * B + i] = i < o->n_riv[l] ? o->riv_idx[(size_t)l * o->lists_cap + i] : -1;
        }
    }
}

/*
 * A separate plain decoder with no exit logic at all: every block of every row runs on
 * one weight set (use_river = 0: the backbone; 1: the dequantised river, i.e. the
 * "full quantisation" limit).  It exists so that the exit loop can be pinned against it.
 */
int orc_plain_step(orc_ctx *o, int B, const int32_t *slots, const int32_t *tok, int use_river, float *logits,
                   int32_t *next_tok) {
    const orc_config *c = &o->c;
    float *a = (float *)malloc(sizeof(float) * (size_t)c->d);
    float *b2 = (float *)malloc(sizeof(float) * (size_t)c->d);
    for (int b = 0; b < B; ++b) {
        const int slot = slots[b], pos = o->len[slot];
        if (pos >= c->max_len) { free(a); free(b2); return -2; }
        embed_row(o, tok[b], a);
        for (int l0 = 0; l0 < c->L; ++l0) {
            block(o, l0, use_river, slot, pos, a, b2);
            float *t = a; a = b2; b2 = t;
        }
        lm_head(o, a, logits ? logits + (size_t)b * c->V : NULL, &next_tok[b]);
        o->len[slot] = pos + 1;
    }
    free(a); free(b2);
    return 0;
}

/*
 * Prefill with sequence-level exit (Section 4.2): every prompt token runs the backbone
 * for blocks 1..e_p and the river for blocks e_p+1..L, causal attention.  Token by token
 * this is a decode step with the exit forced at e_p.  Writes the last token's logits.
 */
int orc_prefill(orc_ctx *o, int slot, const int32_t *tokens, int n, int e_p, float *logits_last, int32_t *next) {
    int32_t nt = 0, el = 0;
    const float tau = INFINITY;
    for (int i = 0; i < n; ++i) {
        const int32_t fe = e_p;
        const int rc = orc_decode_step(o, 1, &slot, &tokens[i], &tau, &fe, (i == n - 1) ? logits_last : NULL, &nt,
                                       &el, NULL);
        if (rc) return rc;
    }
    if (next) *next = nt;
    return 0;
}

/*
 * Prefill whose unified depth is chosen by the exit rule itself (Section 4.2, "Prefill Phase": all tokens of the
 * prompt exit at one depth; Eq. 1 with the prompt's positions as the batch): the depth is the first block l with
 * max(entry_layer, 1) <= l <= L-1 after which EVERY prompt position has s^l > tau, else L.  The scores up to that
 * block involve backbone blocks only, so a first pass runs the whole backbone over the prompt and collects the
 * scores; the prompt is then redone with orc_prefill at the depth found.  Returns the depth, or a negative code.
 */
int orc_prefill_auto(orc_ctx *o, int slot, const int32_t *tokens, int n, float tau, float *logits_last, int32_t *next) {
    const int L = o->c.L;
    int32_t nt = 0, el = 0;
    const int32_t never = L;
    const float inf = INFINITY;
    float *sc = (float *)malloc(sizeof(float) * (size_t)L);
    unsigned char *some_fail = (unsigned char *)calloc((size_t)L + 1, 1);
    for (int i = 0; i < n; ++i) {
        const int rc = orc_decode_step(o, 1, &slot, &tokens[i], &inf, &never, NULL, &nt, &el, sc);
        if (rc) { free(sc); free(some_fail); return rc; }
        for (int l = 1; l <= L; ++l)
            if (!(sc[l - 1] > tau)) some_fail[l] = 1;
    }
    int depth = L;
    for (int l = (o->c.entry_layer > 1 ? o->c.entry_layer : 1); l < L; ++l)
        if (!some_fail[l]) { depth = l; break; }
    free(sc); free(some_fail);
    orc_release(o, slot);
    const int rc = orc_prefill(o, slot, tokens, n, depth, logits_last, next);
    return rc ? rc : depth;
}

/* cache access, fp32 [n][Hkv*dh]; K is stored after RoPE */
int orc_read_kv(const orc_ctx *o, int slot, int layer0, int pos0, int n, float *k_out, float *v_out) {
    const size_t w = (size_t)o->c.Hkv * o->c.dh;
    if (slot < 0 || slot >= o->c.max_seqs || layer0 < 0 || layer0 >= o->c.L || pos0 < 0 || pos0 + n > o->c.max_len)
        return -1;
    for (int i = 0; i < n; ++i) {
        memcpy(k_out + i * w, o->K + kv_off(o, layer0, slot, pos0 + i), w * sizeof(float));
        memcpy(v_out + i * w, o->V + kv_off(o, layer0, slot, pos0 + i), w * sizeof(float));
    }
    return 0;
}
int orc_write_kv(orc_ctx *o, int slot, int layer0, int pos0, int n, const float *k_in, const float *v_in) {
    const size_t w = (size_t)o->c.Hkv * o->c.dh;
    if (slot < 0 || slot >= o->c.max_seqs || layer0 < 0 || layer0 >= o->c.L || pos0 < 0 || pos0 + n > o->c.max_len)
        return -1;
    for (int i = 0; i < n; ++i) {
        memcpy(o->K + kv_off(o, layer0, slot, pos0 + i), k_in + i * w, w * sizeof(float));
        memcpy(o->V + kv_off(o, layer0, slot, pos0 + i), v_in + i * w, w * sizeof(float));
    }
    return 0;
}
/* number of cache writes seen at (layer, slot, pos) since the slot was released */
int orc_write_count(const orc_ctx *o, int slot, int layer0, int pos) {
    return o->written[((size_t)layer0 * o->c.max_seqs + slot) * o->c.max_len + pos];
}

/* ---- small pieces exported on their own so that the tests can pin them one by one ---- */
float orc_similarity(const float *a, const float *b, int d) { return transition_similarity(a, b, d); }
void orc_rope(float *v, int dh, int pos, float theta) { rope(v, dh, pos, theta); }
void orc_attention(const orc_ctx *o, int layer0, int slot, int pos, const float *q, float *att) {
    attend(o, layer0, slot, pos, q, att);
}
void orc_rmsnorm(const float *h, const uint16_t *gain, int d, float eps, float *x) { rmsnorm(h, gain, d, eps, x); }
void orc_matvec_bf16(const uint16_t *w, int out, int in, const float *x, float *y) {
    mat_t m; memset(&m, 0, sizeof m); m.w = w; matvec(&m, out, in, x, y);
}
void orc_matvec_w4(const uint8_t *codes, const uint16_t *scale, const uint16_t *zero, int G, int out, int in,
                   const float *x, float *y) {
    mat_t m; memset(&m, 0, sizeof m); m.codes = codes; m.scale = scale; m.zero = zero; m.G = G;
    matvec(&m, out, in, x, y);
}
/* dequantise a W4 matrix to fp32 [out][in]: w = (q - z) * s */
void orc_dequant_w4(const uint8_t *codes, const uint16_t *scale, const uint16_t *zero, int G, int out, int in,
                    float *w) {
    const int ng = in / G;
    for (int o = 0; o < out; ++o)
        for (int k = 0; k < in; ++k) {
            const uint8_t byte = codes[(size_t)o * (in / 2) + (k >> 1)];
            const int q = (k & 1) ? (byte >> 4) : (byte & 15);
            const float s = bf16_to_f32(scale[(size_t)o * ng + k / G]);
            const float z = bf16_to_f32(zero[(size_t)o * ng + k / G]);
            w[(size_t)o * in + k] = ((float)q - z) * s;
        }
}
/* bytes of a 16-bit K+V cache for n_tokens tokens (the paper's memory table, KV column) */
uint64_t orc_kv_bytes_16bit(const orc_config *c, uint64_t n_tokens) {
    return n_tokens * (uint64_t)c->L * 2u * (uint64_t)c->Hkv * (uint64_t)c->dh * 2u;
}
