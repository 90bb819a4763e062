/*
 * Crystal-KV decode-path oracle: TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow CPU statement of what the library's hot path computes, written from
 * the paper's Section 2.2 (attention), Section 5.2 with Algorithm 1 (attention-based
 * LRFU) and Section 5.3 with Algorithm 2 (adaptive budget allocation).  Only tests,
 * the smoke check and the bench's cpu-baseline leg may call it.  It shares no code
 * with the CUDA path: per-unit explicit entry arrays, a real sort for the nucleus and
 * for the eviction order, and a real compaction (memmove) when entries leave.
 *
 * Precision: attention, softmax and the nucleus walk are fp64 computed from the bf16
 * input bits.  CRF state is fp32 with separately rounded multiply and add (compile
 * with -ffp-contract=off), the decay factor coming from a host table
 * tab[D] = (float)pow((double)lambda, (double)D).  Algorithm 2 is fp64 in a fixed
 * index order with integer (2^-32 fixed-point) CRF sums.
 *
 * Pins (tests/test_oracle_pins.py): attention against an independent naive routine
 * and a library scaled-dot-product attention; the hit mask against subset
 * enumeration; CRF against the closed form of Section 5.2 and the lambda = 0 / 1
 * limits; eviction against a full sort; Algorithm 2 against hand examples and its
 * invariants, the re-share after the cap against a second set of hand examples;
 * "budget = entries per head" against Table 1's HBM-saving column; the
 * observation-window prefill, the buffered eviction cadence and the literal early
 * return against the same definition-level simulator as the plain trajectory; the
 * shrink after a reallocation and after okv_set_budget against that simulator's
 * ranking by the closed-form CRF at the time of the last step; the tie log against
 * hand-built inputs on both sides of the window and against the conditions evaluated
 * from the definitions along a run; export and import as a round trip.
 * Whole trajectories (which tokens survive thousands of steps) have no value printed
 * in the paper: parity unpinned for those beyond the per-step pins above.
 *
 * Readings of points the paper leaves open are marked "Reading:" at the place used.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define OKV_OK 0
#define OKV_ERR (-1)
#define OKV_STAGE_THINK 0
#define OKV_STAGE_ANSWER 1
#define OKV_MODE_EVICT 0
#define OKV_MODE_FULLKV 1
#define OKV_TIE_EVICT 1
#define OKV_TIE_NUCLEUS 2

typedef struct {
    int32_t n_layers, n_q_heads, n_kv_heads, head_dim, batch;
    int32_t budget_per_head, min_budget, max_budget;
    int32_t max_context;
    int32_t mode;
    float top_p, lambda, sm_scale;
    double tie_eps; /* relative window for the tie log (1e-6) */
    int32_t evict_every;    /* m: step 4 runs once a head is m entries over its budget (0, 1: every step) */
    int32_t literal_return; /* 1: Algorithm 1's first line taken literally (nothing runs while Len(K) < B) */
    float budget_ratio;     /* r > 0: budgets follow the context, r x tokens per head on average (0: fixed) */
} okv_config;

typedef struct {
    int32_t pos;
    float crf;
    int32_t tau;
    double *k, *v; /* the bf16 inputs converted exactly to fp64, head_dim each */
} okv_entry;

typedef struct {
    okv_entry *e;
    int n, room;
    int budget;
} okv_unit;

typedef struct {
    int32_t layer, seq, head, t, kind;
} okv_tie;

typedef struct okv {
    okv_config c;
    okv_unit *u; /* [batch][L][H] */
    float *tab;  /* lambda^D, D in [0, max_context] */
    int *t_layer; /* time of the last completed step per layer; -1 before prefill */
    int stage;
    okv_tie *ties;
    int n_ties, room_ties;
} okv;

/* ------------------------------------------------------------------ helpers */

static double bf16_to_double(uint16_t b) {
    uint32_t w = (uint32_t)b << 16;
    float f;
    memcpy(&f, &w, 4);
    return (double)f;
}

static okv_unit *unit_of(okv *o, int seq, int layer, int head) {
    return &o->u[((size_t)seq * o->c.n_layers + layer) * o->c.n_kv_heads + head];
}

static void unit_append(okv *o, okv_unit *u, int pos, const uint16_t *k, const uint16_t *v,
                        float crf, int tau) {
    int d = o->c.head_dim;
    if (u->n == u->room) {
        u->room = u->room ? 2 * u->room : 64;
        u->e = (okv_entry *)realloc(u->e, (size_t)u->room * sizeof(okv_entry));
    }
    okv_entry *e = &u->e[u->n++];
    e->pos = pos;
    e->crf = crf;
    e->tau = tau;
    e->k = (double *)malloc((size_t)d * sizeof(double));
    e->v = (double *)malloc((size_t)d * sizeof(double));
    for (int c = 0; c < d; ++c) { e->k[c] = bf16_to_double(k[c]); e->v[c] = bf16_to_double(v[c]); }
}

/* remove entry i, keeping the order of the others (a real compaction) */
static void unit_erase(okv_unit *u, int i) {
    free(u->e[i].k);
    free(u->e[i].v);
    memmove(&u->e[i], &u->e[i + 1], (size_t)(u->n - 1 - i) * sizeof(okv_entry));
    u->n--;
}

static void log_tie(okv *o, int layer, int seq, int head, int t, int kind) {
#pragma omp critical(okv_tielog)
    {
        if (o->n_ties == o->room_ties) {
            o->room_ties = o->room_ties ? 2 * o->room_ties : 256;
            o->ties = (okv_tie *)realloc(o->ties, (size_t)o->room_ties * sizeof(okv_tie));
        }
        okv_tie *x = &o->ties[o->n_ties++];
        x->layer = layer; x->seq = seq; x->head = head; x->t = t; x->kind = kind;
    }
}

/* ------------------------------------------------------------------ Section 2.2 */

/*
 * AttnScore = softmax(q K^T), y = AttnScore V  (Section 2.2), for the G query heads
 * that share one KV head.  Reading: the logits carry a scale factor (1/sqrt(d) by
 * default); the paper's formula leaves it out.  Every dot product and every output
 * channel is summed in ascending index order; the G heads are only evaluated side by
 * side.
 *   q: [G][d]; krows/vrows: n pointers to d values; prob: [G][n] out; y: [G][d] out.
 */
static void attention_f64(const double *q, const double *const *krows, const double *const *vrows,
                          int n, int G, int d, double scale, double *prob, double *y) {
    double s[64];
    for (int i = 0; i < n; ++i) {
        const double *k = krows[i];
        for (int g = 0; g < G; ++g) s[g] = 0.0;
        for (int c = 0; c < d; ++c)
            for (int g = 0; g < G; ++g) s[g] += q[g * d + c] * k[c];
        for (int g = 0; g < G; ++g) prob[(size_t)g * n + i] = scale * s[g];
    }
    for (int g = 0; g < G; ++g) {
        double *p = prob + (size_t)g * n;
        double m = -INFINITY;
        for (int i = 0; i < n; ++i) if (p[i] > m) m = p[i];
        double l = 0.0;
        for (int i = 0; i < n; ++i) { p[i] = exp(p[i] - m); l += p[i]; }
        for (int i = 0; i < n; ++i) p[i] /= l;
    }
    for (int i = 0; i < G * d; ++i) y[i] = 0.0;
    for (int i = 0; i < n; ++i) {
        const double *v = vrows[i];
        for (int g = 0; g < G; ++g) {
            const double pi = prob[(size_t)g * n + i];
            double *yg = y + (size_t)g * d;
            for (int c = 0; c < d; ++c) yg[c] += pi * v[c];
        }
    }
}

/* the same from bf16 bit patterns: q [G][d], krows/vrows n pointers to d bf16 values */
void okv_attention(const uint16_t *q, const uint16_t *const *krows, const uint16_t *const *vrows,
                   int n, int G, int d, double scale, double *prob, double *y) {
    double *qd = (double *)malloc((size_t)G * d * sizeof(double));
    double *kv = (double *)malloc((size_t)2 * (n > 0 ? n : 1) * d * sizeof(double));
    const double **kr = (const double **)malloc((size_t)(n > 0 ? n : 1) * sizeof(void *));
    const double **vr = (const double **)malloc((size_t)(n > 0 ? n : 1) * sizeof(void *));
    for (int i = 0; i < G * d; ++i) qd[i] = bf16_to_double(q[i]);
    for (int i = 0; i < n; ++i) {
        kr[i] = kv + (size_t)i * d;
        vr[i] = kv + (size_t)(n + i) * d;
        for (int c = 0; c < d; ++c) {
            kv[(size_t)i * d + c] = bf16_to_double(krows[i][c]);
            kv[(size_t)(n + i) * d + c] = bf16_to_double(vrows[i][c]);
        }
    }
    attention_f64(qd, kr, vr, n, G, d, scale, prob, y);
    free(qd); free(kv); free(kr); free(vr);
}

/* ------------------------------------------------------------------ Section 5.2: hits */

typedef struct { double p; int32_t pos; int idx; } nuc_item;

static int nuc_cmp(const void *a, const void *b) {
    const nuc_item *x = (const nuc_item *)a, *y = (const nuc_item *)b;
    if (x->p > y->p) return -1;
    if (x->p < y->p) return 1;
    return (x->pos > y->pos) - (x->pos < y->pos);
}

/*
 * Hit entries = the smallest set of entries whose cumulative attention score reaches
 * the threshold p (Section 5.2; Algorithm 1 step 1).  Reading: walk the entries by
 * descending score (equal scores by ascending position) with an exclusive running sum
 * C; an entry is a hit iff C < p when it is reached.
 * near_tie (optional) is set when the decision sits within rel_eps of a boundary:
 * |C_incl(last hit) - p|/p, |C_excl(last hit) - p|/p, or the relative gap between the
 * last hit's score and the first miss's score.
 * Returns the number of hits.
 */
static int hit_mask_ex(const double *pbar, const int32_t *pos, int n, double p, uint8_t *hit,
                       double rel_eps, int *near_tie, int *last_hit, int *first_miss) {
    nuc_item *it = (nuc_item *)malloc((size_t)(n > 0 ? n : 1) * sizeof(nuc_item));
    for (int i = 0; i < n; ++i) { it[i].p = pbar[i]; it[i].pos = pos[i]; it[i].idx = i; hit[i] = 0; }
    qsort(it, (size_t)n, sizeof(nuc_item), nuc_cmp);
    double C = 0.0, C_excl_last = 0.0;
    int nh = 0;
    for (int r = 0; r < n; ++r) {
        if (!(C < p)) break;
        hit[it[r].idx] = 1;
        C_excl_last = C;
        C += it[r].p;
        nh = r + 1;
    }
    if (near_tie) {
        *near_tie = 0;
        if (nh > 0 && p > 0.0) {
            double last = it[nh - 1].p;
            if (fabs(C - p) / p < rel_eps) *near_tie = 1;
            if (fabs(C_excl_last - p) / p < rel_eps) *near_tie = 1;
            if (nh < n && last > 0.0 && fabs(last - it[nh].p) / last < rel_eps) *near_tie = 1;
        }
    }
    /* the two entries on either side of the boundary, for the harness's flipped replays */
    if (last_hit) *last_hit = nh > 0 ? it[nh - 1].idx : -1;
    if (first_miss) *first_miss = nh < n ? it[nh].idx : -1;
    free(it);
    return nh;
}

int okv_hit_mask(const double *pbar, const int32_t *pos, int n, double p, uint8_t *hit,
                 double rel_eps, int *near_tie) {
    return hit_mask_ex(pbar, pos, n, p, hit, rel_eps, near_tie, NULL, NULL);
}

/* ------------------------------------------------------------------ Algorithm 1 steps 2-4 */

typedef struct { float crf_temp; int32_t tau; int32_t pos; int idx; } ev_item;

static int ev_cmp(const void *a, const void *b) {
    const ev_item *x = (const ev_item *)a, *y = (const ev_item *)b;
    if (x->crf_temp < y->crf_temp) return -1;
    if (x->crf_temp > y->crf_temp) return 1;
    if (x->tau != y->tau) return (x->tau > y->tau) - (x->tau < y->tau);
    return (x->pos > y->pos) - (x->pos < y->pos);
}

/*
 * Algorithm 1 steps 2-3 at time t.  Hits: CRF_temp = lambda^(t-tau)*CRF + 1, recorded
 * together with tau = t.  Misses: CRF_temp = lambda^(t-tau)*CRF, not recorded.
 * Multiply and add are separate fp32 roundings.  crf_temp: [n] out.
 */
static void crf_update(okv *o, okv_unit *u, int t, const uint8_t *hit, float *crf_temp) {
    for (int i = 0; i < u->n; ++i) {
        float dec = o->tab[t - u->e[i].tau];
        volatile float prod = dec * u->e[i].crf;
        float ct = prod;
        if (hit[i]) {
            volatile float sum = ct + 1.0f;
            ct = sum;
            u->e[i].crf = ct;
            u->e[i].tau = t;
        }
        crf_temp[i] = ct;
    }
}

/*
 * Algorithm 1 step 4: Retain = TopK(CRF_temp, B); everything else leaves the cache.
 * Reading: the k = n - B leaving entries are the first k under the total order
 * (CRF_temp ascending, tau ascending, position ascending).  With lambda = 0 every
 * un-hit entry has CRF_temp 0 and the tau key makes this least-recently-hit first.
 * Returns 1 if the k-th and (k+1)-th keys are within rel_eps but not bit-equal.
 */
static int evict_lowest(okv_unit *u, const float *crf_temp, int k, double rel_eps) {
    int n = u->n, near = 0;
    if (k <= 0) return 0;
    if (k > n) k = n;
    ev_item *it = (ev_item *)malloc((size_t)n * sizeof(ev_item));
    for (int i = 0; i < n; ++i) {
        it[i].crf_temp = crf_temp[i]; it[i].tau = u->e[i].tau; it[i].pos = u->e[i].pos; it[i].idx = i;
    }
    qsort(it, (size_t)n, sizeof(ev_item), ev_cmp);
    if (k < n) {
        double a = it[k - 1].crf_temp, b = it[k].crf_temp;
        if (a != b && fabs(b - a) < rel_eps * fmax(fabs(a), fabs(b))) near = 1;
    }
    uint8_t *gone = (uint8_t *)calloc((size_t)n, 1);
    for (int r = 0; r < k; ++r) gone[it[r].idx] = 1;
    for (int i = n - 1; i >= 0; --i)
        if (gone[i]) unit_erase(u, i);
    free(gone);
    free(it);
    return near;
}

/*
 * One pass of Algorithm 1 over a unit with the G queries of its group at time t.
 * Reading (GQA): the cache, CRF and budget belong to the KV head; the hit mask is
 * taken from the mean of the group's G probability vectors, itself a distribution.
 * Reading (step 1 early return): scoring and CRF tracking run on every think step;
 * only the eviction is gated by Len(K) > B.  With literal_return the algorithm's first
 * line is taken as printed instead: while Len(K) < B steps 1-4 are all skipped.
 * Reading (buffered cadence, evict_every = m > 1): step 4 waits until the head is m
 * entries over its budget and then removes all of them at once (k = m per call).
 * hold: steps 1-3 only (the observation-window replay of the prompt evicts once, at
 * its last query).
 * y (may be NULL): [G][d] fp32 attention output.
 * flip (0 in every ordinary call): the harness's "what if the near-tie had gone the other
 * way" replays move the hit boundary by one entry after the mask is taken: 1 = the first
 * miss is a hit too, 2 = the last hit is a miss, 3 = those two trade places.
 */
static void lrfu_pass_unit(okv *o, okv_unit *u, int seq, int layer, int head, const uint16_t *q, int t,
                           int track, int hold, float *y, int flip) {
    int n = u->n, d = o->c.head_dim, G = o->c.n_q_heads / o->c.n_kv_heads;
    if (track && o->c.literal_return && n < u->budget) track = 0;
    const double **kr = (const double **)malloc((size_t)n * sizeof(void *));
    const double **vr = (const double **)malloc((size_t)n * sizeof(void *));
    for (int i = 0; i < n; ++i) { kr[i] = u->e[i].k; vr[i] = u->e[i].v; }
    double *prob = (double *)malloc((size_t)G * n * sizeof(double));
    double *yy = (double *)malloc((size_t)G * d * sizeof(double));
    double *qd = (double *)malloc((size_t)G * d * sizeof(double));
    for (int i = 0; i < G * d; ++i) qd[i] = bf16_to_double(q[i]);
    attention_f64(qd, kr, vr, n, G, d, (double)o->c.sm_scale, prob, yy);
    free(qd);
    if (y) for (int i = 0; i < G * d; ++i) y[i] = (float)yy[i];
    if (track) {
        double *pbar = (double *)malloc((size_t)n * sizeof(double));
        int32_t *pos = (int32_t *)malloc((size_t)n * sizeof(int32_t));
        uint8_t *hit = (uint8_t *)malloc((size_t)n);
        float *ct = (float *)malloc((size_t)n * sizeof(float));
        for (int i = 0; i < n; ++i) {
            double s = 0.0;
            for (int g = 0; g < G; ++g) s += prob[(size_t)g * n + i];
            pbar[i] = s / (double)G;
            pos[i] = u->e[i].pos;
        }
        int near = 0, last_hit = -1, first_miss = -1;
        hit_mask_ex(pbar, pos, n, (double)o->c.top_p, hit, o->c.tie_eps, &near, &last_hit, &first_miss);
        if (near && layer >= 0) log_tie(o, layer, seq, head, t, OKV_TIE_NUCLEUS);
        if ((flip == 1 || flip == 3) && first_miss >= 0) hit[first_miss] = 1;
        if ((flip == 2 || flip == 3) && last_hit >= 0) hit[last_hit] = 0;
        crf_update(o, u, t, hit, ct);
        int m = o->c.evict_every > 1 ? o->c.evict_every : 1;
        int over = n - u->budget;
        if (!hold && over >= m && evict_lowest(u, ct, over, o->c.tie_eps) && layer >= 0)
            log_tie(o, layer, seq, head, t, OKV_TIE_EVICT);
        free(pbar); free(pos); free(hit); free(ct);
    }
    free(kr); free(vr); free(prob); free(yy);
}

static void lrfu_pass(okv *o, int seq, int layer, int head, const uint16_t *q, int t,
                      int track, int hold, float *y) {
    lrfu_pass_unit(o, unit_of(o, seq, layer, head), seq, layer, head, q, t, track, hold, y, 0);
}

/*
 * Ratio budgets (Section 6.1 and Table 1's "Ratio-10 %" rows: a budget of 10 % of the tokens,
 * 935 entries per head of 9 350 tokens, 1 870 of 18 700).  Reading: the average budget per head
 * after `tokens` tokens is floor(r * tokens), evaluated in fp64 from the fp32 ratio, kept
 * between max(1, min_budget) and budget_per_head (which sizes the storage); it is applied when
 * the prompt is loaded (uniformly) and as Algorithm 2's B_total at every reallocation.
 */
static int32_t ratio_budget(const okv_config *c, int tokens) {
    int64_t b = (int64_t)floor((double)c->budget_ratio * (double)tokens);
    int64_t lo = c->min_budget > 1 ? c->min_budget : 1;
    if (b < lo) b = lo;
    if (b > c->budget_per_head) b = c->budget_per_head;
    return (int32_t)b;
}

int32_t okv_ratio_budget(okv *o, int tokens) { return ratio_budget(&o->c, tokens); }

/* ------------------------------------------------------------------ lifecycle */

okv *okv_create(const okv_config *c) {
    if (!c || c->n_layers < 1 || c->n_kv_heads < 1 || c->batch < 1 || c->head_dim < 1 ||
        c->n_q_heads % c->n_kv_heads || c->n_q_heads / c->n_kv_heads > 64 || c->max_context < 1)
        return NULL;
    okv *o = (okv *)calloc(1, sizeof(okv));
    o->c = *c;
    if (o->c.sm_scale == 0.0f) o->c.sm_scale = (float)(1.0 / sqrt((double)c->head_dim));
    if (o->c.tie_eps == 0.0) o->c.tie_eps = 1e-6;
    size_t nu = (size_t)c->batch * c->n_layers * c->n_kv_heads;
    o->u = (okv_unit *)calloc(nu, sizeof(okv_unit));
    for (size_t i = 0; i < nu; ++i) o->u[i].budget = c->budget_per_head;
    o->tab = (float *)malloc(((size_t)c->max_context + 1) * sizeof(float));
    /* lambda^D; pow(0, 0) = 1 makes lambda = 0 keep only same-step hits */
    for (int D = 0; D <= c->max_context; ++D) o->tab[D] = (float)pow((double)c->lambda, (double)D);
    o->t_layer = (int *)malloc((size_t)c->n_layers * sizeof(int));
    for (int l = 0; l < c->n_layers; ++l) o->t_layer[l] = -1;
    o->stage = OKV_STAGE_THINK;
    return o;
}

void okv_destroy(okv *o) {
    if (!o) return;
    size_t nu = (size_t)o->c.batch * o->c.n_layers * o->c.n_kv_heads;
    for (size_t i = 0; i < nu; ++i) {
        for (int j = 0; j < o->u[i].n; ++j) { free(o->u[i].e[j].k); free(o->u[i].e[j].v); }
        free(o->u[i].e);
    }
    free(o->u); free(o->tab); free(o->t_layer); free(o->ties); free(o);
}

int okv_set_stage(okv *o, int stage) { o->stage = stage; return OKV_OK; }

/*
 * Prompt: k, v [batch][P][H][d]; q_last [batch][Hq][d] is the query of prompt token
 * P-1.  Reading: the P entries arrive with CRF 0 and tau = P-1, then one Algorithm 1
 * pass with Q^last at t = P-1 seeds CRF/tau and evicts down to the budget.
 */
int okv_prefill(okv *o, int layer, const uint16_t *k, const uint16_t *v, const uint16_t *q_last, int P) {
    const okv_config *c = &o->c;
    if (layer < 0 || layer >= c->n_layers || P < 1 || o->t_layer[layer] >= 0) return OKV_ERR;
    int H = c->n_kv_heads, d = c->head_dim, G = c->n_q_heads / H;
    int track = (c->mode == OKV_MODE_EVICT);
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < c->batch; ++b)
        for (int h = 0; h < H; ++h) {
            okv_unit *u = unit_of(o, b, layer, h);
            if (c->budget_ratio > 0.0f) u->budget = ratio_budget(c, P);
            for (int i = 0; i < P; ++i) {
                size_t off = (((size_t)b * P + i) * H + h) * d;
                unit_append(o, u, i, k + off, v + off, 0.0f, P - 1);
            }
            const uint16_t *q = q_last + ((size_t)b * c->n_q_heads + (size_t)h * G) * d;
            if (track) lrfu_pass(o, b, layer, h, q, P - 1, 1, 0, NULL);
        }
    o->t_layer[layer] = P - 1;
    return OKV_OK;
}

/*
 * Prompt with an observation window: k, v [batch][P][H][d]; q_win [W][batch][Hq][d] are
 * the queries of prompt tokens P-W .. P-1; y_win (may be NULL) [W][batch][Hq][d] their
 * causal attention outputs.  Reading: the last W prompt tokens are replayed as decode
 * steps whose eviction is deferred: token i arrives with CRF 0 and tau = i, the query
 * of token t in the window attends to tokens 0..t and runs Algorithm 1 steps 1-3 at
 * time t, and step 4 runs once, after the last query (t = P-1).
 */
int okv_prefill_window(okv *o, int layer, const uint16_t *k, const uint16_t *v, const uint16_t *q_win,
                       int P, int W, float *y_win) {
    const okv_config *c = &o->c;
    if (layer < 0 || layer >= c->n_layers || P < 1 || W < 1 || W > P || o->t_layer[layer] >= 0) return OKV_ERR;
    int H = c->n_kv_heads, d = c->head_dim, G = c->n_q_heads / H;
    int track = (c->mode == OKV_MODE_EVICT);
    size_t qn = (size_t)c->batch * c->n_q_heads * d;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < c->batch; ++b)
        for (int h = 0; h < H; ++h) {
            okv_unit *u = unit_of(o, b, layer, h);
            if (c->budget_ratio > 0.0f) u->budget = ratio_budget(c, P);
            for (int i = 0; i < P; ++i) {
                size_t off = (((size_t)b * P + i) * H + h) * d;
                unit_append(o, u, i, k + off, v + off, 0.0f, i);
                int w = i - (P - W);
                if (w < 0) continue;
                size_t qo = (size_t)w * qn + ((size_t)b * c->n_q_heads + (size_t)h * G) * d;
                lrfu_pass(o, b, layer, h, q_win + qo, i, track, i < P - 1, y_win ? y_win + qo : NULL);
            }
        }
    o->t_layer[layer] = P - 1;
    return OKV_OK;
}

/*
 * One decode step of one layer: q, out [batch][Hq][d]; k_new, v_new [batch][H][d].
 * The new (k, v) is appended (Section 2.2) as a PotentialKV entry; reading: CRF 0,
 * tau = arrival time.  Think stage in evict mode: Algorithm 1.  Answer stage or
 * FullKV mode: attention only, nothing tracked, nothing evicted.
 */
int okv_decode_step(okv *o, int layer, const uint16_t *q, const uint16_t *k_new,
                    const uint16_t *v_new, float *out) {
    const okv_config *c = &o->c;
    if (layer < 0 || layer >= c->n_layers || o->t_layer[layer] < 0) return OKV_ERR;
    int t = o->t_layer[layer] + 1;
    if (t > c->max_context) return OKV_ERR;
    int H = c->n_kv_heads, d = c->head_dim, G = c->n_q_heads / H;
    int track = (c->mode == OKV_MODE_EVICT && o->stage == OKV_STAGE_THINK);
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < c->batch; ++b)
        for (int h = 0; h < H; ++h) {
            okv_unit *u = unit_of(o, b, layer, h);
            size_t kvo = ((size_t)b * H + h) * d;
            unit_append(o, u, t, k_new + kvo, v_new + kvo, 0.0f, t);
            size_t qo = ((size_t)b * c->n_q_heads + (size_t)h * G) * d;
            lrfu_pass(o, b, layer, h, q + qo, t, track, 0, out + qo);
        }
    o->t_layer[layer] = t;
    return OKV_OK;
}

/* ------------------------------------------------------------------ Algorithm 2 */

typedef struct { double frac; int idx; } rem_item;

static int rem_cmp(const void *a, const void *b) {
    const rem_item *x = (const rem_item *)a, *y = (const rem_item *)b;
    if (x->frac > y->frac) return -1;
    if (x->frac < y->frac) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

/*
 * Hand `extra` whole slots to the members of `who` (m indices into add[]) in
 * proportion to weight[]: floor of the real share, then one more each by largest
 * fractional part (ties to the lower index).  All-zero weights mean equal shares.
 */
static void share_out(int64_t extra, const int *who, int m, const double *weight, int64_t *add) {
    if (m <= 0 || extra <= 0) return;
    double W = 0.0;
    for (int j = 0; j < m; ++j) W += weight[who[j]];
    rem_item *r = (rem_item *)malloc((size_t)m * sizeof(rem_item));
    int64_t given = 0;
    for (int j = 0; j < m; ++j) {
        double x = (W > 0.0) ? ((double)extra * weight[who[j]]) / W : (double)extra / (double)m;
        double f = floor(x);
        add[who[j]] += (int64_t)f;
        given += (int64_t)f;
        r[j].frac = x - f;
        r[j].idx = who[j];
    }
    qsort(r, (size_t)m, sizeof(rem_item), rem_cmp);
    int64_t left = extra - given;
    for (int64_t j = 0; left > 0; ++j, --left) add[r[j % m].idx] += 1;
    /* rounding can only over-give when the real shares sum above `extra` */
    for (int64_t j = m - 1; left < 0; --j) {
        if (j < 0) j = m - 1;
        if (add[r[j].idx] > 0) { add[r[j].idx] -= 1; ++left; }
    }
    free(r);
}

/*
 * Algorithm 2 for one inference: A[L*H] aggregated CRF (real), B[L*H] current budgets.
 *   step 1  eta_i  = sum_j A_ij / sum_j B_ij
 *   step 2  B'_i   = B_total * eta_i / sum_i eta_i
 *   step 3  eta_ij = A_ij / B_ij
 *   step 4  B'_ij  = B'_i * eta_ij / sum_j eta_ij
 * Reading (integers): a floor of min_b per head is set aside first and the rule
 * divides the remainder R = B_total - L*H*min_b; shares are floored and the left-over
 * slots go to the largest fractional parts, so sum B' = B_total exactly; heads above
 * max_b are clamped and their excess is shared among the others by the same
 * proportions until none exceeds it.  With min_b = 0 and max_b = B_total this is
 * Algorithm 2 itself.  sum_i eta_i = 0 keeps the budgets; sum_j eta_ij = 0 splits the
 * layer's share equally.
 */
void okv_alg2(const double *A, const int32_t *B, int L, int H, int64_t B_total,
              int32_t min_b, int32_t max_b, int32_t *B_out) {
    int N = L * H;
    double *eta_l = (double *)malloc((size_t)L * sizeof(double));
    double *S_l = (double *)malloc((size_t)L * sizeof(double));
    double *x = (double *)malloc((size_t)N * sizeof(double));
    int64_t *add = (int64_t *)calloc((size_t)N, sizeof(int64_t));
    int *who = (int *)malloc((size_t)N * sizeof(int));
    double S = 0.0;
    for (int i = 0; i < L; ++i) {
        double sa = 0.0, sb = 0.0, sl = 0.0;
        for (int j = 0; j < H; ++j) {
            sa += A[i * H + j];
            sb += (double)B[i * H + j];
            sl += A[i * H + j] / (double)B[i * H + j];
        }
        eta_l[i] = sa / sb;
        S_l[i] = sl;
        S += eta_l[i];
    }
    if (!(S > 0.0)) {
        for (int k = 0; k < N; ++k) B_out[k] = B[k];
        goto done;
    }
    {
        int64_t R = B_total - (int64_t)N * min_b;
        for (int i = 0; i < L; ++i)
            for (int j = 0; j < H; ++j) {
                double layer_share = ((double)R * eta_l[i]) / S;
                double head_part = (S_l[i] > 0.0) ? (A[i * H + j] / (double)B[i * H + j]) / S_l[i]
                                                  : 1.0 / (double)H;
                x[i * H + j] = layer_share * head_part;
            }
        for (int k = 0; k < N; ++k) who[k] = k;
        share_out(R, who, N, x, add);
        for (;;) {
            int64_t excess = 0;
            int m = 0;
            for (int k = 0; k < N; ++k) {
                int64_t b = (int64_t)min_b + add[k];
                if (b > max_b) { excess += b - max_b; add[k] = (int64_t)max_b - min_b; }
            }
            if (excess == 0) break;
            for (int k = 0; k < N; ++k)
                if ((int64_t)min_b + add[k] < max_b) who[m++] = k;
            if (m == 0) break;
            share_out(excess, who, m, x, add);
        }
        for (int k = 0; k < N; ++k) B_out[k] = (int32_t)(min_b + add[k]);
    }
done:
    free(eta_l); free(S_l); free(x); free(add); free(who);
}

/*
 * Periodic trigger of Algorithm 2 (Section 5.3), per sequence, at the time t_last of
 * the last completed step (all layers must agree on it).  Reading: a head's
 * "aggregated CRF" is the sum over its retained entries of the CRF decayed to t_last,
 * each term truncated to 2^-32 fixed point so the sum is order independent.  Heads
 * whose budget shrank evict down to it at once, lowest (decayed CRF, tau, pos) first.
 */
int okv_rebudget(okv *o) {
    const okv_config *c = &o->c;
    int L = c->n_layers, H = c->n_kv_heads;
    int t_last = o->t_layer[0];
    for (int l = 0; l < L; ++l)
        if (o->t_layer[l] != t_last || t_last < 0) return OKV_ERR;
    if (c->mode != OKV_MODE_EVICT) return OKV_ERR;
    int64_t B_total = (int64_t)c->budget_per_head * L * H;
    if (c->budget_ratio > 0.0f) B_total = (int64_t)ratio_budget(c, t_last + 1) * L * H;
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < c->batch; ++b) {
        double *A = (double *)malloc((size_t)L * H * sizeof(double));
        int32_t *B = (int32_t *)malloc((size_t)L * H * sizeof(int32_t));
        int32_t *Bn = (int32_t *)malloc((size_t)L * H * sizeof(int32_t));
        for (int l = 0; l < L; ++l)
            for (int h = 0; h < H; ++h) {
                okv_unit *u = unit_of(o, b, l, h);
                int64_t acc = 0;
                for (int i = 0; i < u->n; ++i) {
                    volatile float dcrf = o->tab[t_last - u->e[i].tau] * u->e[i].crf;
                    acc += (int64_t)((double)dcrf * 4294967296.0);
                }
                A[l * H + h] = (double)acc / 4294967296.0;
                B[l * H + h] = u->budget;
            }
        okv_alg2(A, B, L, H, B_total, c->min_budget, c->max_budget, Bn);
        for (int l = 0; l < L; ++l)
            for (int h = 0; h < H; ++h) {
                okv_unit *u = unit_of(o, b, l, h);
                u->budget = Bn[l * H + h];
                if (u->n > u->budget) {
                    float *ct = (float *)malloc((size_t)u->n * sizeof(float));
                    for (int i = 0; i < u->n; ++i) {
                        volatile float dcrf = o->tab[t_last - u->e[i].tau] * u->e[i].crf;
                        ct[i] = dcrf;
                    }
                    if (evict_lowest(u, ct, u->n - u->budget, c->tie_eps))
                        log_tie(o, l, b, h, t_last, OKV_TIE_EVICT);
                    free(ct);
                }
            }
        free(A); free(B); free(Bn);
    }
    return OKV_OK;
}

/* ------------------------------------------------------------------ inspection */

static int pos_cmp(const void *a, const void *b) {
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/* ascending token positions retained by (layer, seq, head); returns the count */
int okv_get_retained(okv *o, int layer, int seq, int head, int32_t *pos_out, int cap) {
    okv_unit *u = unit_of(o, seq, layer, head);
    if (u->n > cap) return -u->n;
    for (int i = 0; i < u->n; ++i) pos_out[i] = u->e[i].pos;
    qsort(pos_out, (size_t)u->n, sizeof(int32_t), pos_cmp);
    return u->n;
}

int okv_get_budgets(okv *o, int32_t *out) { /* [batch][L][H] */
    size_t nu = (size_t)o->c.batch * o->c.n_layers * o->c.n_kv_heads;
    for (size_t i = 0; i < nu; ++i) out[i] = o->u[i].budget;
    return OKV_OK;
}

/*
 * Sets one head's budget by hand; a head holding more than its new budget evicts down
 * to it at once, exactly as after a reallocation (lowest CRF decayed to the time of the
 * last step first).
 */
int okv_set_budget(okv *o, int layer, int seq, int head, int budget) {
    okv_unit *u = unit_of(o, seq, layer, head);
    int t_last = o->t_layer[layer];
    u->budget = budget;
    if (t_last >= 0 && u->n > budget) {
        float *ct = (float *)malloc((size_t)u->n * sizeof(float));
        for (int i = 0; i < u->n; ++i) {
            volatile float dcrf = o->tab[t_last - u->e[i].tau] * u->e[i].crf;
            ct[i] = dcrf;
        }
        if (evict_lowest(u, ct, u->n - budget, o->c.tie_eps)) log_tie(o, layer, seq, head, t_last, OKV_TIE_EVICT);
        free(ct);
    }
    return OKV_OK;
}

int okv_time(okv *o, int layer) { return o->t_layer[layer]; }

/* per-entry records sorted by position: rec[3*i] = pos, [3*i+1] = CRF bits, [3*i+2] = tau */
int okv_export_state(okv *o, int layer, int seq, int head, int32_t *rec, int cap) {
    okv_unit *u = unit_of(o, seq, layer, head);
    if (u->n > cap) return -u->n;
    ev_item *it = (ev_item *)malloc((size_t)(u->n ? u->n : 1) * sizeof(ev_item));
    for (int i = 0; i < u->n; ++i) { it[i].pos = u->e[i].pos; it[i].idx = i; }
    for (int i = 1; i < u->n; ++i) { /* insertion sort by pos: entries are nearly ordered */
        ev_item x = it[i];
        int j = i - 1;
        while (j >= 0 && it[j].pos > x.pos) { it[j + 1] = it[j]; --j; }
        it[j + 1] = x;
    }
    for (int i = 0; i < u->n; ++i) {
        okv_entry *e = &u->e[it[i].idx];
        uint32_t bits;
        memcpy(&bits, &e->crf, 4);
        rec[3 * i] = e->pos; rec[3 * i + 1] = (int32_t)bits; rec[3 * i + 2] = e->tau;
    }
    free(it);
    return u->n;
}

/*
 * Replace a unit's contents (used by the harness to re-synchronise after a logged
 * tie): n records as above plus the K/V rows [n][d] of those positions.
 */
int okv_import_state(okv *o, int layer, int seq, int head, const int32_t *rec, int n,
                     const uint16_t *k, const uint16_t *v) {
    okv_unit *u = unit_of(o, seq, layer, head);
    int d = o->c.head_dim;
    while (u->n > 0) unit_erase(u, u->n - 1);
    for (int i = 0; i < n; ++i) {
        float crf;
        uint32_t bits = (uint32_t)rec[3 * i + 1];
        memcpy(&crf, &bits, 4);
        unit_append(o, u, rec[3 * i], k + (size_t)i * d, v + (size_t)i * d, crf, rec[3 * i + 2]);
    }
    return OKV_OK;
}

/*
 * Replays think-stage decode steps of ONE head outside the oracle's own state, for the
 * harness: when the GPU's state differs from the oracle's after a logged near-tie, the
 * difference is only forgiven if this replay, with the tie taken the other way, lands on the
 * GPU's state exactly.  The head starts from n records (as okv_export_state writes them)
 * with their K/V rows and a budget, then takes nsteps steps at times t_first, t_first+1, ..
 * with the given queries [nsteps][G][d] and arriving rows [nsteps][d]; flips[s] is the flip
 * of step s (see lrfu_pass_unit).  With append_first = 0 the first step appends nothing: it
 * is the scoring pass of a prefill over the records given.  Uses the handle's configuration
 * and decay table only; logs nothing.  Writes the final records (sorted by position) and returns their count, or the
 * negated count if cap is too small.
 */
int okv_replay_unit(okv *o, const int32_t *rec, const uint16_t *k, const uint16_t *v, int n, int budget,
                    int t_first, int append_first, int nsteps, const uint16_t *q, const uint16_t *k_new, const uint16_t *v_new,
                    const int32_t *flips, int32_t *rec_out, int cap) {
    int d = o->c.head_dim, G = o->c.n_q_heads / o->c.n_kv_heads;
    okv_unit u;
    memset(&u, 0, sizeof u);
    u.budget = budget;
    for (int i = 0; i < n; ++i) {
        float crf;
        uint32_t bits = (uint32_t)rec[3 * i + 1];
        memcpy(&crf, &bits, 4);
        unit_append(o, &u, rec[3 * i], k + (size_t)i * d, v + (size_t)i * d, crf, rec[3 * i + 2]);
    }
    for (int s = 0; s < nsteps; ++s) {
        int t = t_first + s;
        if (s > 0 || append_first) unit_append(o, &u, t, k_new + (size_t)s * d, v_new + (size_t)s * d, 0.0f, t);
        lrfu_pass_unit(o, &u, 0, -1, 0, q + (size_t)s * G * d, t, 1, 0, NULL, flips ? flips[s] : 0);
    }
    int n_out = u.n;
    if (n_out <= cap) {
        int32_t *order = (int32_t *)malloc((size_t)(n_out ? n_out : 1) * sizeof(int32_t));
        for (int i = 0; i < n_out; ++i) order[i] = i;
        for (int i = 1; i < n_out; ++i) { /* insertion sort by position */
            int32_t x = order[i];
            int j = i - 1;
            while (j >= 0 && u.e[order[j]].pos > u.e[x].pos) { order[j + 1] = order[j]; --j; }
            order[j + 1] = x;
        }
        for (int i = 0; i < n_out; ++i) {
            okv_entry *e = &u.e[order[i]];
            uint32_t bits;
            memcpy(&bits, &e->crf, 4);
            rec_out[3 * i] = e->pos; rec_out[3 * i + 1] = (int32_t)bits; rec_out[3 * i + 2] = e->tau;
        }
        free(order);
    }
    for (int j = 0; j < u.n; ++j) { free(u.e[j].k); free(u.e[j].v); }
    free(u.e);
    return n_out <= cap ? n_out : -n_out;
}

int okv_tie_count(okv *o) { return o->n_ties; }

/* copies up to cap records of 5 int32 {layer, seq, head, t, kind}; returns the count copied */
int okv_get_ties(okv *o, int32_t *out, int cap) {
    int n = o->n_ties < cap ? o->n_ties : cap;
    for (int i = 0; i < n; ++i) {
        out[5 * i] = o->ties[i].layer; out[5 * i + 1] = o->ties[i].seq; out[5 * i + 2] = o->ties[i].head;
        out[5 * i + 3] = o->ties[i].t; out[5 * i + 4] = o->ties[i].kind;
    }
    return n;
}

void okv_clear_ties(okv *o) { o->n_ties = 0; }

/* decay table entry, for tests */
float okv_decay(okv *o, int D) { return o->tab[D]; }
