/*
 * OBCache checker ("oracle"): a plain, slow, double-precision CPU statement of what the
 * score -> pool -> select -> compact path computes.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be compared with
 * something written directly from the paper.  It shares no code, header, table or constant
 * with the CUDA path; nothing in the product may call it.  Only the tests, the smoke check
 * and the benchmark's CPU-baseline leg load it.
 *
 * What each function follows:
 *   attention recompute        Sec. 3 (Z = Q K^T / sqrt(d), A = softmax_row(Z), O = A V),
 *                              restricted to the perturbation window (Eq. 9, App. A.1)
 *   value score                Eq. 4  (App. A.2 boxed form)
 *   key score                  Eq. 5  (App. A.3 boxed form)
 *   joint score                Eq. 6  (App. A.4 boxed form)
 *   "alg1" formulation         Algorithm 1 (expanded norms: |o|^2 + |v|^2 - 2 v.o, |v|^2 - v.o)
 *   attention-only score       Sec. 4.3 (sum_i |A_ip|)
 *   value-aware l1 score       remark after Eq. 4 and App. C.2 "VATP": Eq. 4 with l1 norms,
 *                              sum_i |A_ip| * ||v_p||_1
 *   scores from a given O/LSE  Eq. 4-6 with A = exp(Z - lse) and o_i as supplied by the caller
 *                              (the attention kernel's own outputs instead of a recompute)
 *   GQA reduction              App. A.5 (sum over the query heads of a KV head's group)
 *   head-adaptive select       the AdaKV budget allocation the paper pairs its scores with (Sec. 5.1,
 *                              App. C.2.1): global ranking across heads with a per-head safeguard
 *   pool / select / compact    Algorithm 2 (top-k below the cutoff, indices sorted ascending,
 *                              gather, recent tail appended) with SnapKV-style 1-D pooling
 *   decode step pieces         Sec. 3 "Decoding"/"Cache Eviction", Sec. 4.2 last paragraph
 *                              (scores accumulated over decode steps), App. C.2.2
 *
 * Parity pins (tests/test_oracle_*.py) check these functions against brute-force row zeroing,
 * finite-difference limits, closed-form special cases and sort-based brute force; every
 * exported scoring/selection function is pinned (none is "parity unpinned").
 *
 * Readings taken where the paper is silent (all listed in the design notes):
 *   - window rows are the last W query positions; with causal != 0 row i sees keys
 *     p <= N - W + i; masked pairs contribute exactly 0;
 *   - Z is the scaled logit q.k/sqrt(d) itself (no max subtraction);
 *   - pooling runs over the candidate range [n_sink, N - n_recent) only, stride 1, "same"
 *     length, in fp32: max pads with -inf, avg pads with zeros and divides by the kernel size,
 *     adding taps in ascending index order;
 *   - ties in the top-k keep the lowest index.
 */
#define _GNU_SOURCE
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ work sharing */
typedef void (*item_fn)(void* ctx, long item);
typedef struct { item_fn fn; void* ctx; long n_items; long next; pthread_mutex_t mu; } pool_t;

static void* pool_worker(void* arg) {
    pool_t* p = (pool_t*)arg;
    for (;;) {
        pthread_mutex_lock(&p->mu);
        long it = p->next++;
        pthread_mutex_unlock(&p->mu);
        if (it >= p->n_items) break;
        p->fn(p->ctx, it);
    }
    return NULL;
}

/* Every item writes outputs no other item writes, so results do not depend on n_threads. */
static void run_items(item_fn fn, void* ctx, long n_items, int n_threads) {
    pool_t p; p.fn = fn; p.ctx = ctx; p.n_items = n_items; p.next = 0;
    pthread_mutex_init(&p.mu, NULL);
    if (n_threads < 1) n_threads = 1;
    if (n_threads > 256) n_threads = 256;
    if (n_threads == 1 || n_items <= 1) { pool_worker(&p); pthread_mutex_destroy(&p.mu); return; }
    pthread_t th[256];
    for (int t = 0; t < n_threads; ++t) pthread_create(&th[t], NULL, pool_worker, &p);
    for (int t = 0; t < n_threads; ++t) pthread_join(th[t], NULL);
    pthread_mutex_destroy(&p.mu);
}

/* ------------------------------------------------------------------ small helpers */
static double dot_fd(const float* a, const float* b, int d) {
    double s = 0.0;
    for (int c = 0; c < d; ++c) s += (double)a[c] * (double)b[c];
    return s;
}
static double dot_fD(const float* a, const double* b, int d) {
    double s = 0.0;
    for (int c = 0; c < d; ++c) s += (double)a[c] * b[c];
    return s;
}

/* ------------------------------------------------------------------ score */
typedef struct {
    const float *q, *k, *v;            /* q [B,Hq,W,d]; k, v [B,Hkv,Nmax,d] */
    int B, Hq, Hkv, d, W, Nmax;
    const int32_t* seq_lens;           /* [B] or NULL (all = Nmax) */
    double scale; int causal; int formulation;
    /* per (b, g, r): softmax statistics and window outputs */
    double *m, *l, *o;                 /* [B*Hkv*R], [B*Hkv*R], [B*Hkv*R*d] */
    double *s_value, *s_key, *s_joint, *s_attn, *s_vatp;   /* [B,Hkv,Nmax], any may be NULL */
    long chunk;                        /* tokens per phase-2 item */
    long chunks_per_unit;
} score_ctx;

static int seq_len_of(const score_ctx* c, int b) { return c->seq_lens ? c->seq_lens[b] : c->Nmax; }

/* row r of KV head g = (query head g*G + r / W, window index i = r % W) */
static const float* q_row(const score_ctx* c, int b, int g, int r) {
    int G = c->Hq / c->Hkv;
    int h = g * G + r / c->W, i = r % c->W;
    return c->q + (((long)b * c->Hq + h) * c->W + i) * c->d;
}
/* last key position row r may attend to (Sec. 3: decoding query s attends to keys 1..s) */
static long last_visible(const score_ctx* c, int N, int r) {
    if (!c->causal) return N - 1;
    return (long)N - c->W + (r % c->W);
}

/* Phase 1, one item per (b, g, r): m_r = max_p z_rp, l_r = sum_p exp(z_rp - m_r),
 * o_r = sum_p A_rp v_p with A_rp = exp(z_rp - m_r) / l_r          (Sec. 3)               */
static void phase1_item(void* vctx, long item) {
    score_ctx* c = (score_ctx*)vctx;
    int G = c->Hq / c->Hkv, R = G * c->W, d = c->d;
    int r = (int)(item % R); long u = item / R; int g = (int)(u % c->Hkv), b = (int)(u / c->Hkv);
    int N = seq_len_of(c, b);
    const float* qr = q_row(c, b, g, r);
    const float* K = c->k + ((long)b * c->Hkv + g) * c->Nmax * d;
    const float* V = c->v + ((long)b * c->Hkv + g) * c->Nmax * d;
    long last = last_visible(c, N, r);
    double* z = (double*)malloc(sizeof(double) * (size_t)(last + 1 > 0 ? last + 1 : 1));
    double m = -INFINITY;
    for (long p = 0; p <= last; ++p) { z[p] = c->scale * dot_fd(qr, K + p * d, d); if (z[p] > m) m = z[p]; }
    double l = 0.0;
    for (long p = 0; p <= last; ++p) l += exp(z[p] - m);
    double* o = c->o + item * d;
    for (int cc = 0; cc < d; ++cc) o[cc] = 0.0;
    for (long p = 0; p <= last; ++p) {
        double a = exp(z[p] - m) / l;
        for (int cc = 0; cc < d; ++cc) o[cc] += a * (double)V[p * d + cc];
    }
    c->m[item] = m; c->l[item] = l;
    free(z);
}

/* Phase 2, one item per (b, g, token chunk): the three scores of every token in the chunk. */
static void phase2_item(void* vctx, long item) {
    score_ctx* c = (score_ctx*)vctx;
    int G = c->Hq / c->Hkv, R = G * c->W, d = c->d;
    long ch = item % c->chunks_per_unit; long u = item / c->chunks_per_unit;
    int g = (int)(u % c->Hkv), b = (int)(u / c->Hkv);
    int N = seq_len_of(c, b);
    const float* K = c->k + ((long)b * c->Hkv + g) * c->Nmax * d;
    const float* V = c->v + ((long)b * c->Hkv + g) * c->Nmax * d;
    long p0 = ch * c->chunk, p1 = p0 + c->chunk; if (p1 > N) p1 = N;
    for (long p = p0; p < p1; ++p) {
        const float* kp = K + p * d; const float* vp = V + p * d;
        double nv = dot_fd(vp, vp, d);                       /* ||v_p||^2 */
        double nv1 = 0.0;                                    /* ||v_p||_1 */
        for (int cc = 0; cc < d; ++cc) nv1 += fabs((double)vp[cc]);
        double sv = 0.0, sk = 0.0, sj = 0.0, sa = 0.0;
        for (int r = 0; r < R; ++r) {
            if (p > last_visible(c, N, r)) continue;         /* masked pair: contributes 0 */
            long ur = u * R + r;
            const double* o = c->o + ur * d;
            double Z = c->scale * dot_fd(q_row(c, b, g, r), kp, d);
            double A = exp(Z - c->m[ur]) / c->l[ur];
            double vo = dot_fD(vp, o, d);                    /* v_p . o_r */
            sa += fabs(A);                                   /* Sec. 4.3 */
            sv += A * A * nv;                                /* Eq. 4 */
            double key_term, cross_term;
            if (c->formulation == 0) {
                /* Eq. 5: |A Z|^2 ||v_p - o_r||^2, the norm taken of the difference vector */
                double dn = 0.0;
                for (int cc = 0; cc < d; ++cc) { double df = (double)vp[cc] - o[cc]; dn += df * df; }
                key_term = (A * Z) * (A * Z) * dn;
                /* Eq. 6 cross term: 2 A^2 Z (||v_p||^2 - v_p . o_r) */
                cross_term = 2.0 * A * A * Z * (nv - vo);
            } else {
                /* Algorithm 1: ||v - o||^2 expanded as |o|^2 + |v|^2 - 2 v.o */
                double no = 0.0;
                for (int cc = 0; cc < d; ++cc) no += o[cc] * o[cc];
                double vmo = no + nv - 2.0 * vo;
                key_term = (A * Z) * (A * Z) * vmo;
                cross_term = 2.0 * (A * A) * Z * (nv - vo);
            }
            sk += key_term;
            sj += cross_term;
        }
        sj += sv + sk;                                       /* Eq. 6 */
        long idx = u * c->Nmax + p;
        if (c->s_value) c->s_value[idx] = sv;
        if (c->s_key)   c->s_key[idx]   = sk;
        if (c->s_joint) c->s_joint[idx] = sj;
        if (c->s_attn)  c->s_attn[idx]  = sa;
        if (c->s_vatp)  c->s_vatp[idx]  = sa * nv1;          /* remark after Eq. 4: l1 norms */
    }
}

/*
 * Scores of every cached token for every (batch item, KV head).
 *   q [B,Hq,W,d], k, v [B,Hkv,Nmax,d]: host float arrays (values exact in the storage dtype).
 *   seq_lens: host int32 [B] or NULL.  scale <= 0 means 1/sqrt(d).
 *   formulation: 0 = Eq. 4-6 as printed, 1 = Algorithm 1's expanded form.
 *   outputs: host double [B,Hkv,Nmax] each, NULL to skip; entries past seq_len are 0.
 *   o_out [B,Hkv,R,d], m_out, l_out [B,Hkv,R]: optional copies of the window outputs / stats.
 * Returns 0, or -1 on a bad argument / allocation failure.
 */
static int score_run(const float* q, const float* k, const float* v,
                     const float* o_given, const float* lse_given,
                     int B, int Hq, int Hkv, int d, int W, int Nmax, const int32_t* seq_lens,
                     double scale, int causal, int formulation,
                     double* s_value, double* s_key, double* s_joint, double* s_attn, double* s_vatp,
                     double* o_out, double* m_out, double* l_out, int n_threads) {
    if (!q || !k || !v || B < 1 || Hkv < 1 || Hq % Hkv || d < 1 || W < 1 || Nmax < 1) return -1;
    if ((o_given == NULL) != (lse_given == NULL)) return -1;
    for (int b = 0; b < B; ++b) { int n = seq_lens ? seq_lens[b] : Nmax; if (n < W || n > Nmax) return -1; }
    score_ctx c; memset(&c, 0, sizeof c);
    c.q = q; c.k = k; c.v = v; c.B = B; c.Hq = Hq; c.Hkv = Hkv; c.d = d; c.W = W; c.Nmax = Nmax;
    c.seq_lens = seq_lens; c.scale = scale > 0 ? scale : 1.0 / sqrt((double)d);
    c.causal = causal; c.formulation = formulation;
    int R = (Hq / Hkv) * W; long units = (long)B * Hkv;
    c.m = (double*)malloc(sizeof(double) * units * R);
    c.l = (double*)malloc(sizeof(double) * units * R);
    c.o = (double*)malloc(sizeof(double) * units * R * d);
    if (!c.m || !c.l || !c.o) { free(c.m); free(c.l); free(c.o); return -1; }
    c.s_value = s_value; c.s_key = s_key; c.s_joint = s_joint; c.s_attn = s_attn; c.s_vatp = s_vatp;
    double* outs[5] = { s_value, s_key, s_joint, s_attn, s_vatp };
    for (int i = 0; i < 5; ++i) if (outs[i]) memset(outs[i], 0, sizeof(double) * units * Nmax);
    if (o_given) {
        /* Row r of KV head g is (query head g*G + r / W, window index r % W), so [B,Hq,W,d] and
         * [B,Hkv,R,d] are the same memory order.  A_ip = exp(z_ip - lse_i): m = lse, l = 1. */
        for (long i = 0; i < units * R; ++i) { c.m[i] = (double)lse_given[i]; c.l[i] = 1.0; }
        for (long i = 0; i < units * R * d; ++i) c.o[i] = (double)o_given[i];
    } else {
        run_items(phase1_item, &c, units * R, n_threads);
    }
    c.chunk = 256; c.chunks_per_unit = (Nmax + c.chunk - 1) / c.chunk;
    run_items(phase2_item, &c, units * c.chunks_per_unit, n_threads);
    if (o_out) memcpy(o_out, c.o, sizeof(double) * units * R * d);
    if (m_out) memcpy(m_out, c.m, sizeof(double) * units * R);
    if (l_out) memcpy(l_out, c.l, sizeof(double) * units * R);
    free(c.m); free(c.l); free(c.o);
    return 0;
}

int obc_oracle_score(const float* q, const float* k, const float* v,
                     int B, int Hq, int Hkv, int d, int W, int Nmax, const int32_t* seq_lens,
                     double scale, int causal, int formulation,
                     double* s_value, double* s_key, double* s_joint, double* s_attn, double* s_vatp,
                     double* o_out, double* m_out, double* l_out, int n_threads) {
    return score_run(q, k, v, NULL, NULL, B, Hq, Hkv, d, W, Nmax, seq_lens, scale, causal, formulation,
                     s_value, s_key, s_joint, s_attn, s_vatp, o_out, m_out, l_out, n_threads);
}

/*
 * The same scores from attention outputs the caller already has (what a fused attention kernel
 * returns for the window rows) instead of a recompute:
 *   o_given   [B,Hq,W,d]  host float, the window rows of O = A V
 *   lse_given [B,Hq,W]    host float, natural-log log-sum-exp of the scaled logits of each row
 * Eq. 4-6 are evaluated with A_ip = exp(z_ip - lse_i) and o_i = o_given row i.  Other arguments
 * and outputs as obc_oracle_score.
 */
int obc_oracle_score_given(const float* q, const float* k, const float* v,
                           const float* o_given, const float* lse_given,
                           int B, int Hq, int Hkv, int d, int W, int Nmax, const int32_t* seq_lens,
                           double scale, int causal, int formulation,
                           double* s_value, double* s_key, double* s_joint, double* s_attn, double* s_vatp,
                           int n_threads) {
    if (!o_given || !lse_given) return -1;
    return score_run(q, k, v, o_given, lse_given, B, Hq, Hkv, d, W, Nmax, seq_lens, scale, causal, formulation,
                     s_value, s_key, s_joint, s_attn, s_vatp, NULL, NULL, NULL, n_threads);
}

/* ------------------------------------------------------------------ pool */
/*
 * 1-D pooling of one head's fp32 scores over the candidate range [lo, hi) (stride 1, same
 * length, odd kernel).  mode 0: copy; 1: average (zero padding, divide by the kernel size,
 * taps added in ascending index order, fp32); 2: max (padding never wins).  Entries outside
 * [lo, hi) are copied unchanged.  Returns 0 or -1.
 */
int obc_oracle_pool(const float* s, int N, int lo, int hi, int mode, int kernel, float* out) {
    if (!s || !out || N < 0 || lo < 0 || hi > N || lo > hi) return -1;
    if (mode != 0 && (kernel < 1 || kernel % 2 == 0)) return -1;
    for (int p = 0; p < N; ++p) out[p] = s[p];
    if (mode == 0 || kernel == 1) return 0;
    int half = kernel / 2;
    for (int p = lo; p < hi; ++p) {
        if (mode == 1) {
            volatile float acc = 0.0f;                     /* volatile: one fp32 rounding per add */
            for (int t = p - half; t <= p + half; ++t) if (t >= lo && t < hi) acc = acc + s[t];
            out[p] = acc / (float)kernel;
        } else {
            float mx = -INFINITY;
            for (int t = p - half; t <= p + half; ++t) if (t >= lo && t < hi && s[t] > mx) mx = s[t];
            out[p] = mx;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ select */
typedef struct { float s; int32_t i; } cand_t;
static int cand_cmp(const void* a, const void* b) {
    const cand_t* x = (const cand_t*)a; const cand_t* y = (const cand_t*)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->i > y->i) - (x->i < y->i);                  /* equal scores: lowest index first */
}
static int i32_cmp(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b; return (x > y) - (x < y);
}

/*
 * Algorithm 2's index selection for one head.  Keeps the first n_sink and the last n_recent
 * tokens, plus the (budget - n_sink - n_recent) highest-scoring tokens of the candidate range
 * [n_sink, N - n_recent) (ties: lowest index).  idx receives `budget` indices in ascending
 * order followed by (idx_len - budget) entries of -1.  Returns 0 or -1.
 */
int obc_oracle_select(const float* pooled, int N, int budget, int n_sink, int n_recent,
                      int32_t* idx, int idx_len) {
    if (!pooled || !idx || N < 1 || budget > N || budget > idx_len) return -1;
    if (n_sink < 0 || n_recent < 0 || budget < n_sink + n_recent) return -1;
    int lo = n_sink, hi = N - n_recent, n_hh = budget - n_sink - n_recent;
    if (hi - lo < n_hh) return -1;
    cand_t* c = (cand_t*)malloc(sizeof(cand_t) * (size_t)(hi - lo > 0 ? hi - lo : 1));
    if (!c) return -1;
    for (int p = lo; p < hi; ++p) { c[p - lo].s = pooled[p]; c[p - lo].i = p; }
    qsort(c, (size_t)(hi - lo), sizeof(cand_t), cand_cmp);
    int w = 0;
    for (int p = 0; p < n_sink; ++p) idx[w++] = p;
    for (int j = 0; j < n_hh; ++j) idx[w++] = c[j].i;
    qsort(idx + n_sink, (size_t)n_hh, sizeof(int32_t), i32_cmp);
    for (int p = hi; p < N; ++p) idx[w++] = p;
    for (; w < idx_len; ++w) idx[w] = -1;
    free(c);
    return 0;
}

/* ------------------------------------------------------------------ head-adaptive select */
typedef struct { float s; int32_t h; int32_t i; } hcand_t;
static int hcand_cmp(const void* a, const void* b) {
    const hcand_t* x = (const hcand_t*)a; const hcand_t* y = (const hcand_t*)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    if (x->h != y->h) return (x->h > y->h) - (x->h < y->h);  /* equal scores: lowest head, then lowest index */
    return (x->i > y->i) - (x->i < y->i);
}

/*
 * Head-adaptive budgets (the AdaKV allocation of App. C.2.1 and Sec. 5.1: the top-k eviction scores are
 * ranked globally across the heads of a layer, with a safeguard fraction of the budget guaranteed to
 * every head), for one batch item.
 *   pooled [H, N]   the heads' pooled scores (row stride N)
 *   budget          kept tokens per head on average; n_hh = budget - n_sink - n_recent slots per head
 *                   are for scored tokens, H * n_hh in total
 *   safeguard       fraction of n_hh every head keeps by its own ranking: s = floor(safeguard * n_hh)
 * Every head first takes its s best candidates of [n_sink, N - n_recent) (ties: lowest index); the
 * other H * (n_hh - s) slots go to the best remaining candidates of all heads ranked together (ties:
 * lowest head, then lowest index).  idx [H, idx_len]: per head the sinks, the selected tokens in
 * ascending order and the recent tail, padded with -1; counts [H] = kept tokens of the head.
 * Returns 0, or -1 on bad arguments or when a head would keep more than idx_len tokens.
 */
int obc_oracle_select_adaptive(const float* pooled, int H, int N, int budget, int n_sink, int n_recent,
                               float safeguard, int32_t* idx, int32_t* counts, int idx_len) {
    if (!pooled || !idx || !counts || H < 1 || N < 1 || budget > N) return -1;
    if (n_sink < 0 || n_recent < 0 || budget < n_sink + n_recent) return -1;
    if (!(safeguard >= 0.0f && safeguard <= 1.0f)) return -1;
    const int lo = n_sink, hi = N - n_recent, n_hh = budget - n_sink - n_recent, n = hi - lo;
    if (n < n_hh) return -1;
    int s = (int)floor((double)safeguard * (double)n_hh);
    if (s > n_hh) s = n_hh;
    const long extra = (long)H * (n_hh - s);
    char* taken = (char*)calloc((size_t)H * (size_t)(n > 0 ? n : 1), 1);
    cand_t* c = (cand_t*)malloc(sizeof(cand_t) * (size_t)(n > 0 ? n : 1));
    hcand_t* rest = (hcand_t*)malloc(sizeof(hcand_t) * (size_t)H * (size_t)(n > 0 ? n : 1));
    if (!taken || !c || !rest) { free(taken); free(c); free(rest); return -1; }
    long n_rest = 0;
    for (int h = 0; h < H; ++h) {                          /* the safeguarded share of every head */
        for (int p = lo; p < hi; ++p) { c[p - lo].s = pooled[(long)h * N + p]; c[p - lo].i = p; }
        qsort(c, (size_t)n, sizeof(cand_t), cand_cmp);
        for (int j = 0; j < s; ++j) taken[(long)h * n + (c[j].i - lo)] = 1;
        for (int j = s; j < n; ++j) { rest[n_rest].s = c[j].s; rest[n_rest].h = h; rest[n_rest].i = c[j].i; ++n_rest; }
    }
    qsort(rest, (size_t)n_rest, sizeof(hcand_t), hcand_cmp);   /* all heads ranked together */
    for (long j = 0; j < extra; ++j) taken[(long)rest[j].h * n + (rest[j].i - lo)] = 1;
    int rc = 0;
    for (int h = 0; h < H && rc == 0; ++h) {
        int w = 0;
        int32_t* out = idx + (long)h * idx_len;
        int kept = n_sink + n_recent;
        for (int p = 0; p < n; ++p) kept += taken[(long)h * n + p];
        if (kept > idx_len) { rc = -1; break; }
        for (int p = 0; p < n_sink; ++p) out[w++] = p;
        for (int p = lo; p < hi; ++p) if (taken[(long)h * n + (p - lo)]) out[w++] = p;
        for (int p = hi; p < N; ++p) out[w++] = p;
        counts[h] = w;
        for (; w < idx_len; ++w) out[w] = -1;
    }
    free(taken); free(c); free(rest);
    return rc;
}

/* ------------------------------------------------------------------ compact */
/*
 * Algorithm 2's gather for one head: out[j,:] = src[idx[j],:] for j < budget.  `elem` is the
 * element size in bytes (2 or 4); rows j >= budget of `out` are left untouched.
 */
int obc_oracle_compact(const void* src, int d, int elem, const int32_t* idx, int budget, void* out) {
    if (!src || !idx || !out || d < 1 || elem < 1) return -1;
    size_t row = (size_t)d * (size_t)elem;
    for (int j = 0; j < budget; ++j) {
        if (idx[j] < 0) return -1;
        memcpy((char*)out + row * (size_t)j, (const char*)src + row * (size_t)idx[j], row);
    }
    return 0;
}

/* ------------------------------------------------------------------ decode pieces */
/*
 * W = 1 scores of one KV head's live cache for the newest query of each of its G query heads.
 *   qg [G,d]; kc, vc [cap,d]; pos [cap] (token position of a slot, < 0 = free slot);
 *   slots [0, hi) are examined.  variant: 1 value, 2 key, 4 joint, 8 attention-only.
 *   out [cap] double: the score of each live slot (0 for free slots and slots >= hi).
 * The newest query attends to every live slot (they are all earlier or equal positions).
 */
int obc_oracle_decode_scores(const float* qg, const float* kc, const float* vc, const int32_t* pos,
                             int G, int d, int cap, int hi, double scale, int variant, double* out) {
    if (!qg || !kc || !vc || !pos || !out || hi > cap) return -1;
    if (scale <= 0) scale = 1.0 / sqrt((double)d);
    for (int p = 0; p < cap; ++p) out[p] = 0.0;
    double* o = (double*)malloc(sizeof(double) * (size_t)d);
    double* z = (double*)malloc(sizeof(double) * (size_t)(hi > 0 ? hi : 1));
    if (!o || !z) { free(o); free(z); return -1; }
    for (int r = 0; r < G; ++r) {
        const float* qr = qg + (long)r * d;
        double m = -INFINITY, l = 0.0;
        for (int p = 0; p < hi; ++p) if (pos[p] >= 0) { z[p] = scale * dot_fd(qr, kc + (long)p * d, d); if (z[p] > m) m = z[p]; }
        for (int p = 0; p < hi; ++p) if (pos[p] >= 0) l += exp(z[p] - m);
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        for (int p = 0; p < hi; ++p) if (pos[p] >= 0) {
            double a = exp(z[p] - m) / l;
            for (int c = 0; c < d; ++c) o[c] += a * (double)vc[(long)p * d + c];
        }
        for (int p = 0; p < hi; ++p) if (pos[p] >= 0) {
            const float* vp = vc + (long)p * d;
            double A = exp(z[p] - m) / l, Z = z[p];
            double nv = dot_fd(vp, vp, d), vo = dot_fD(vp, o, d), dn = 0.0;
            for (int c = 0; c < d; ++c) { double df = (double)vp[c] - o[c]; dn += df * df; }
            double sv = A * A * nv, sk = (A * Z) * (A * Z) * dn;
            double sj = sv + sk + 2.0 * A * A * Z * (nv - vo);
            out[p] += variant == 1 ? sv : variant == 2 ? sk : variant == 4 ? sj : fabs(A);
        }
    }
    free(o); free(z);
    return 0;
}

/*
 * Which slot to evict after a decode step, from fp32 accumulated scores: the live slot with
 * the smallest accumulator among tokens that are neither sinks (pos < n_sink) nor recent
 * (pos > step_pos - n_recent, the newest token has pos == step_pos); equal accumulators evict
 * the highest position.  Returns the slot, or -1 if no slot is evictable.
 */
int obc_oracle_decode_evict(const float* s_acc, const int32_t* pos, int hi, int step_pos,
                            int n_sink, int n_recent) {
    int best = -1;
    for (int p = 0; p < hi; ++p) {
        if (pos[p] < 0 || pos[p] < n_sink || pos[p] > step_pos - n_recent) continue;
        if (best < 0 || s_acc[p] < s_acc[best] || (s_acc[p] == s_acc[best] && pos[p] > pos[best])) best = p;
    }
    return best;
}
