/*
 * SubGen oracle: a plain, slow, single-threaded CPU statement of the streaming
 * attention data structure of "SubGen: Token Generation in Sublinear Time and
 * Memory" (Algorithm 1 with its three procedures UpdateSoftmaxNormalizer,
 * UpdateMatrixProduct and QueryStreamAttn), plus the recent-token sliding
 * window of the paper's end-to-end experiments (Section 3.2).
 *
 * THIS IS TEST INFRASTRUCTURE. It exists so that the CUDA library can be
 * checked against something written directly from the paper. It shares no
 * code, header, table or helper with the CUDA path and must never be used by
 * it. Only tests, the smoke check and the CPU-baseline leg of the benchmark
 * may load it.
 *
 * One oracle object is one stream, i.e. one (sequence, KV head) unit. It keeps
 * every key and value it has seen (the whole point of an oracle is to be able
 * to look everything up) and represents the paper's state by token indices:
 *   D  = { (x_i, S_i, n_i) }   -> centre_tok[i], slot_tok[i*t + j], count[i]
 *   M  = list of s (k, v)      -> m_tok[j]  (-1 = null)
 *   mu = sum of ||v||^2         -> mu (fixed point, see below)
 *   window                      -> the last `window` token indices
 *
 * Readings of points the paper leaves open:
 *  - Window (Section 3.2 keeps "the most recent r tokens" next to the
 *    clustered rest and gives no estimator for the combination): a token
 *    enters D and M when it LEAVES the window; window tokens enter numerator
 *    and partition function exactly, with weight one. window = 0 is
 *    Algorithm 1 verbatim; a stream no longer than the window is exact
 *    attention (Eq. 1).
 *  - Order inside one stream step follows the main loop of Algorithm 1:
 *    UpdateSoftmaxNormalizer, then UpdateMatrixProduct with the OLD mu, then
 *    mu += ||v||^2, then the query.
 *  - "<= delta" joins, "> delta" opens (the algorithm and Lemma 2, not the
 *    prose). Ties in the argmin go to the lowest cluster index.
 *  - Decisions are integer decisions, so they are taken in exact integer
 *    arithmetic that does not depend on summation order:
 *      D2(x,k) = sum_j floor( fl32( fl32(x_j - k_j)^2 ) * 2^32 )   (uint64)
 *      join  <=>  D2 <= floor( fl32(delta)^2 (in double) * 2^32 )
 *      W(v)    = sum_j floor( fl32(v_j * v_j) * 2^24 )             (uint64)
 *      mu      = sum of W over inserted tokens                      (uint64)
 *    fl32 is IEEE binary32 round-to-nearest-even; inputs are binary32 (bf16
 *    inputs are widened exactly).
 *  - Coins come from Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11):
 *      key     = (seed low 32 bits, seed high 32 bits)
 *      counter = (token index, unit id, slot / 4, domain)
 *      word    = slot % 4;  domain 0 = cluster slots, 1 = value slots
 *    cluster coin (probability 1/n):   u * n          <  2^32
 *    value coin (prob. W/(mu+W)):      u * (mu + W)   <  W * 2^32   (128 bit)
 *  - The estimator weight of a value sample is mu / (s * W), the same
 *    fixed-point numbers the coin used, so it is unbiased for the
 *    distribution actually sampled. Null slots contribute nothing.
 *  - exp() is shifted by the maximum score over everything scored; z / tau
 *    does not depend on the shift.
 *  - No 1/sqrt(d): Eq. 1 has none.
 *
 * Pins (tests/test_oracle_*.py): published Philox known answers, exact
 * attention when the stream fits the window, z/tau = v_1 after one token,
 * delta = 0 gives the exact partition function, the five invariants of
 * Lemma 2, the sampling laws of Lemma 1 and Lemma 2(5) (chi-square),
 * unbiasedness of z and tau, the closed-form variance of row-norm sampling.
 * The 0.99 success probability of Theorem 1 hides constants in Omega() and is
 * parity unpinned.
 *
 * Build: gcc -O2 -ffp-contract=off -shared -fPIC (binary32 products must not
 * be fused or kept in wider registers).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;

/* ------------------------------------------------------------------------ */
/* Philox4x32-10, from its published definition.                             */

static void philox_round(uint32_t c[4], const uint32_t k[2]) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
    uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    uint32_t n0 = hi1 ^ c[1] ^ k[0];
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c[3] ^ k[1];
    uint32_t n3 = lo0;
    c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
}

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
    uint32_t k[2] = {key[0], key[1]};
    for (int r = 0; r < 10; ++r) {
        if (r > 0) { k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u; }
        philox_round(c, k);
    }
    out[0] = c[0]; out[1] = c[1]; out[2] = c[2]; out[3] = c[3];
}

/* ------------------------------------------------------------------------ */

typedef struct oracle_unit {
    int d, t, s, window, m_max;
    float delta;
    uint64_t delta2_fx;          /* floor(delta^2 * 2^32) */
    uint32_t key[2];
    uint32_t unit_id;

    /* every token seen so far */
    int n, cap;
    float *K, *V;                /* [cap, d] */
    uint64_t *W;                 /* [cap] fixed-point ||v||^2 */
    int *assign;                 /* [cap] cluster id of an inserted token, -1 while in the window */
    uint64_t *ins_d2;            /* [cap] D2 to the nearest centre at insertion (UINT64_MAX if D was empty) */
    int *ins_near;               /* [cap] index of that nearest centre (-1 if D was empty) */

    int inserted;                /* tokens that have left the window = tokens in D and M */
    int m;                       /* clusters */
    int *centre_tok;             /* [m_max] */
    int *count;                  /* [m_max] */
    int *slot_tok;               /* [m_max * t] */
    int *m_tok;                  /* [s], -1 = null */
    uint64_t mu;
    int overflow_at;             /* token whose insertion found D full, or -1 */

    /* bounded-m variant (see doubling_sweep): the threshold in force and how often it has doubled */
    int bounded;
    uint64_t thr2_fx;            /* starts as delta2_fx */
    int level;
} oracle_unit;

oracle_unit *oracle_create(int d, float delta, int t, int s, int window, uint64_t seed,
                           uint32_t unit_id, int m_max) {
    if (d <= 0 || t <= 0 || s <= 0 || window < 0 || m_max <= 0 || !(delta >= 0.0f)) return NULL;
    oracle_unit *u = (oracle_unit *)calloc(1, sizeof(oracle_unit));
    if (!u) return NULL;
    u->d = d; u->t = t; u->s = s; u->window = window; u->m_max = m_max;
    u->delta = delta;
    u->delta2_fx = (uint64_t)floor((double)delta * (double)delta * 4294967296.0);
    u->thr2_fx = u->delta2_fx;
    u->key[0] = (uint32_t)seed; u->key[1] = (uint32_t)(seed >> 32);
    u->unit_id = unit_id;
    u->centre_tok = (int *)malloc(sizeof(int) * (size_t)m_max);
    u->count = (int *)malloc(sizeof(int) * (size_t)m_max);
    u->slot_tok = (int *)malloc(sizeof(int) * (size_t)m_max * (size_t)t);
    u->m_tok = (int *)malloc(sizeof(int) * (size_t)s);
    for (int i = 0; i < s; ++i) u->m_tok[i] = -1;     /* M starts as s nulls */
    u->overflow_at = -1;
    return u;
}

void oracle_destroy(oracle_unit *u) {
    if (!u) return;
    free(u->K); free(u->V); free(u->W); free(u->assign); free(u->ins_d2); free(u->ins_near);
    free(u->centre_tok); free(u->count); free(u->slot_tok); free(u->m_tok);
    free(u);
}

/* D2(x, k): squared distance in order-independent fixed point. */
static uint64_t dist2_fx(const float *x, const float *k, int d) {
    uint64_t acc = 0;
    for (int j = 0; j < d; ++j) {
        float diff = x[j] - k[j];
        float sq = diff * diff;
        acc += (uint64_t)(sq * 4294967296.0f);
    }
    return acc;
}

/* W(v): squared norm in order-independent fixed point. */
static uint64_t norm2_fx(const float *v, int d) {
    uint64_t acc = 0;
    for (int j = 0; j < d; ++j) {
        float sq = v[j] * v[j];
        acc += (uint64_t)(sq * 16777216.0f);
    }
    return acc;
}

static uint32_t coin_word(const oracle_unit *u, int token, int slot, uint32_t domain) {
    uint32_t ctr[4] = {(uint32_t)token, u->unit_id, (uint32_t)(slot / 4), domain};
    uint32_t out[4];
    oracle_philox4x32_10(ctr, u->key, out);
    return out[slot % 4];
}

/*
 * Bounded-m variant. The paper bounds the number of clusters only through the clusterability assumption and cites
 * the incremental clustering of Charikar, Chekuri, Feder and Motwani as the inspiration of its online clustering;
 * it does not say what to do when a budget of m_max clusters is exhausted. This is the reading taken, in the
 * spirit of that doubling algorithm:
 *   when token e has no representative within the threshold and m = m_max, the threshold doubles
 *   (thr2 <- max(4 thr2, 1) in fixed point, capped at 2^62) and the clusters are swept in index order: cluster i
 *   is kept if no already kept representative lies within the new threshold of x_i, otherwise it is merged into
 *   the nearest kept one (ties: lowest kept index). Kept clusters are renumbered in order. Token e is then placed
 *   against the kept representatives with the new threshold; if it still has to open a cluster and there is still
 *   no room, the threshold doubles again.
 * Merging cluster i (n_i members) into kept cluster j (n_j members): the count becomes n_j + n_i and every sample
 * slot q of j independently takes slot q of i with probability n_i / (n_j + n_i), which keeps each slot uniform
 * over the union, exactly as property (5) of Lemma 2 needs. The coin is
 *   u * (n_j + n_i) < n_i * 2^32,  u = word q % 4 of Philox(counter = (e, unit, q / 4 + 256 * i, 2 + 4 * level)),
 * i the index the merged cluster had before this sweep, level the number of doublings including this one.
 */
static uint32_t merge_coin_word(const oracle_unit *u, int token, int slot, int old_index) {
    uint32_t ctr[4] = {(uint32_t)token, u->unit_id, (uint32_t)(slot / 4) + 256u * (uint32_t)old_index,
                       2u + 4u * (uint32_t)u->level};
    uint32_t out[4];
    oracle_philox4x32_10(ctr, u->key, out);
    return out[slot % 4];
}

static void doubling_sweep(oracle_unit *u, int e) {
    u->level++;
    if (u->thr2_fx >= ((uint64_t)1 << 60)) u->thr2_fx = (uint64_t)1 << 62;
    else u->thr2_fx = u->thr2_fx ? 4 * u->thr2_fx : 1;
    int *remap = (int *)malloc(sizeof(int) * (size_t)u->m);
    int kept = 0;
    for (int i = 0; i < u->m; ++i) {
        const float *xi = u->K + (size_t)u->centre_tok[i] * u->d;
        int best = -1;
        uint64_t best_d2 = UINT64_MAX;
        for (int j = 0; j < kept; ++j) {
            uint64_t d2 = dist2_fx(u->K + (size_t)u->centre_tok[j] * u->d, xi, u->d);
            if (d2 < best_d2) { best_d2 = d2; best = j; }
        }
        if (best >= 0 && best_d2 <= u->thr2_fx) {
            uint64_t n_i = (uint64_t)u->count[i], n_new = (uint64_t)u->count[best] + n_i;
            for (int q = 0; q < u->t; ++q) {
                uint32_t w = merge_coin_word(u, e, q, i);
                if ((uint64_t)w * n_new < (n_i << 32)) u->slot_tok[(size_t)best * u->t + q] = u->slot_tok[(size_t)i * u->t + q];
            }
            u->count[best] = (int)n_new;
            remap[i] = best;
        } else {
            u->centre_tok[kept] = u->centre_tok[i];
            u->count[kept] = u->count[i];
            for (int q = 0; q < u->t; ++q) u->slot_tok[(size_t)kept * u->t + q] = u->slot_tok[(size_t)i * u->t + q];
            remap[i] = kept++;
        }
    }
    for (int tok = 0; tok < u->inserted; ++tok) u->assign[tok] = remap[u->assign[tok]];
    u->m = kept;
    free(remap);
}

/* Procedure UpdateSoftmaxNormalizer for token e. Returns 0, or -1 if D is full. */
static int update_softmax_normalizer(oracle_unit *u, int e) {
    const float *k = u->K + (size_t)e * u->d;
    for (int round = 0;; ++round) {
        int best = -1;
        uint64_t best_d2 = UINT64_MAX;
        for (int i = 0; i < u->m; ++i) {                    /* argmin over representatives */
            uint64_t d2 = dist2_fx(u->K + (size_t)u->centre_tok[i] * u->d, k, u->d);
            if (d2 < best_d2) { best_d2 = d2; best = i; }  /* strict: ties keep the lowest index */
        }
        u->ins_d2[e] = best_d2;
        u->ins_near[e] = best;
        if (best >= 0 && best_d2 <= u->thr2_fx) {
            int n_new = ++u->count[best];
            for (int j = 0; j < u->t; ++j) {               /* t independent size-1 reservoirs */
                uint32_t w = coin_word(u, e, j, 0u);
                if ((uint64_t)w * (uint64_t)n_new < 4294967296ull) u->slot_tok[(size_t)best * u->t + j] = e;
            }
            u->assign[e] = best;
            return 0;
        }
        if (u->m < u->m_max) {
            int c = u->m++;
            u->centre_tok[c] = e;                           /* representative = first key of the cluster */
            u->count[c] = 1;
            for (int j = 0; j < u->t; ++j) u->slot_tok[(size_t)c * u->t + j] = e;   /* t copies */
            u->assign[e] = c;
            return 0;
        }
        if (!u->bounded || round >= 40) { if (u->overflow_at < 0) u->overflow_at = e; return -1; }
        doubling_sweep(u, e);
    }
}

/* Procedure UpdateMatrixProduct for token e, with the mu of before this token. */
static void update_matrix_product(oracle_unit *u, int e) {
    uint64_t w_e = u->W[e];
    u128 rhs = (u128)w_e << 32;
    u128 tot = (u128)u->mu + (u128)w_e;
    for (int i = 0; i < u->s; ++i) {
        uint32_t w = coin_word(u, e, i, 1u);
        if ((u128)w * tot < rhs) u->m_tok[i] = e;
    }
}

static int insert_token(oracle_unit *u, int e) {
    int rc = update_softmax_normalizer(u, e);
    if (rc) return rc;
    update_matrix_product(u, e);
    u->mu += u->W[e];
    u->inserted++;
    return 0;
}

/* Append one token to the stream. The token enters the window; the token it
 * pushes out (itself when window = 0) is inserted into D and M.
 * Returns 0, -1 on cluster capacity overflow (state then stops being meaningful). */
int oracle_push(oracle_unit *u, const float *k, const float *v) {
    if (u->n == u->cap) {
        int nc = u->cap ? u->cap * 2 : 1024;
        u->K = (float *)realloc(u->K, sizeof(float) * (size_t)nc * u->d);
        u->V = (float *)realloc(u->V, sizeof(float) * (size_t)nc * u->d);
        u->W = (uint64_t *)realloc(u->W, sizeof(uint64_t) * (size_t)nc);
        u->assign = (int *)realloc(u->assign, sizeof(int) * (size_t)nc);
        u->ins_d2 = (uint64_t *)realloc(u->ins_d2, sizeof(uint64_t) * (size_t)nc);
        u->ins_near = (int *)realloc(u->ins_near, sizeof(int) * (size_t)nc);
        u->cap = nc;
    }
    int e_new = u->n;
    memcpy(u->K + (size_t)e_new * u->d, k, sizeof(float) * u->d);
    memcpy(u->V + (size_t)e_new * u->d, v, sizeof(float) * u->d);
    u->W[e_new] = norm2_fx(v, u->d);
    u->assign[e_new] = -1;
    u->ins_d2[e_new] = 0;
    u->ins_near[e_new] = -1;
    u->n++;
    if (u->n - u->inserted > u->window) return insert_token(u, u->inserted);
    return 0;
}

int oracle_push_many(oracle_unit *u, const float *K, const float *V, int n) {
    for (int i = 0; i < n; ++i) {
        int rc = oracle_push(u, K + (size_t)i * u->d, V + (size_t)i * u->d);
        if (rc) return rc;
    }
    return 0;
}

static double dot_d(const float *a, const float *b, int d) {
    double acc = 0.0;
    for (int j = 0; j < d; ++j) acc += (double)a[j] * (double)b[j];
    return acc;
}

/* Procedure QueryStreamAttn plus the window terms.
 *   z   = sum_{(k,v) in M} mu/(s ||v||^2) exp(<q,k>) v  +  sum_{window} exp(<q,k>) v
 *   tau = sum_{(x,S,n') in D} (n'/t) sum_{k in S} exp(<q,k>)  +  sum_{window} exp(<q,k>)
 * Everything is scaled by exp(-shift), shift = the largest score met.
 * z_out[d], *tau_out, *shift_out may be NULL; out[d] = z / tau. */
void oracle_query_parts(const oracle_unit *u, const float *q, double *out,
                        double *z_out, double *tau_out, double *shift_out) {
    const int d = u->d;
    double shift = -INFINITY;
    for (int c = 0; c < u->m; ++c)
        for (int j = 0; j < u->t; ++j) {
            double a = dot_d(q, u->K + (size_t)u->slot_tok[(size_t)c * u->t + j] * d, d);
            if (a > shift) shift = a;
        }
    for (int i = 0; i < u->s; ++i)
        if (u->m_tok[i] >= 0) {
            double a = dot_d(q, u->K + (size_t)u->m_tok[i] * d, d);
            if (a > shift) shift = a;
        }
    for (int e = u->inserted; e < u->n; ++e) {
        double a = dot_d(q, u->K + (size_t)e * d, d);
        if (a > shift) shift = a;
    }
    double *z = (double *)calloc((size_t)d, sizeof(double));
    double tau = 0.0;
    if (shift > -INFINITY) {
        for (int i = 0; i < u->s; ++i) {
            int e = u->m_tok[i];
            if (e < 0) continue;
            double wgt = (double)u->mu / ((double)u->s * (double)u->W[e]);
            double p = wgt * exp(dot_d(q, u->K + (size_t)e * d, d) - shift);
            for (int j = 0; j < d; ++j) z[j] += p * (double)u->V[(size_t)e * d + j];
        }
        for (int c = 0; c < u->m; ++c) {
            double acc = 0.0;
            for (int j = 0; j < u->t; ++j)
                acc += exp(dot_d(q, u->K + (size_t)u->slot_tok[(size_t)c * u->t + j] * d, d) - shift);
            tau += (double)u->count[c] / (double)u->t * acc;
        }
        for (int e = u->inserted; e < u->n; ++e) {
            double p = exp(dot_d(q, u->K + (size_t)e * d, d) - shift);
            for (int j = 0; j < d; ++j) z[j] += p * (double)u->V[(size_t)e * d + j];
            tau += p;
        }
    }
    if (out) for (int j = 0; j < d; ++j) out[j] = tau > 0.0 ? z[j] / tau : 0.0;
    if (z_out) memcpy(z_out, z, sizeof(double) * (size_t)d);
    if (tau_out) *tau_out = tau;
    if (shift_out) *shift_out = shift;
    free(z);
}

void oracle_query(const oracle_unit *u, const float *q, double *out) {
    oracle_query_parts(u, q, out, NULL, NULL, NULL);
}

/* One pass of the main loop of Algorithm 1: update with (k, v), then query with q. */
int oracle_step(oracle_unit *u, const float *q, const float *k, const float *v, double *out) {
    int rc = oracle_push(u, k, v);
    if (rc) return rc;
    oracle_query(u, q, out);
    return 0;
}

/* Eq. 1 written out: softmax(K q)^T V over n rows, no scaling. */
void oracle_exact_attention(const float *K, const float *V, int n, int d, const float *q, double *out) {
    double shift = -INFINITY;
    for (int i = 0; i < n; ++i) {
        double a = dot_d(q, K + (size_t)i * d, d);
        if (a > shift) shift = a;
    }
    double denom = 0.0;
    for (int j = 0; j < d; ++j) out[j] = 0.0;
    for (int i = 0; i < n; ++i) {
        double p = exp(dot_d(q, K + (size_t)i * d, d) - shift);
        denom += p;
        for (int j = 0; j < d; ++j) out[j] += p * (double)V[(size_t)i * d + j];
    }
    for (int j = 0; j < d; ++j) out[j] = denom > 0.0 ? out[j] / denom : 0.0;
}

/* ------------------------------------------------------------------------ */
/* Read-only views of the state, for the tests.                              */

int oracle_n(const oracle_unit *u) { return u->n; }
int oracle_inserted(const oracle_unit *u) { return u->inserted; }
int oracle_m(const oracle_unit *u) { return u->m; }
uint64_t oracle_mu(const oracle_unit *u) { return u->mu; }
uint64_t oracle_delta2_fx(const oracle_unit *u) { return u->delta2_fx; }
/* Switch on the bounded-m variant; valid only before the first token. */
int oracle_set_bounded(oracle_unit *u, int on) { if (u->n) return -1; u->bounded = on != 0; return 0; }
uint64_t oracle_thr2_fx(const oracle_unit *u) { return u->thr2_fx; }
int oracle_level(const oracle_unit *u) { return u->level; }
int oracle_overflow_at(const oracle_unit *u) { return u->overflow_at; }
const int *oracle_counts(const oracle_unit *u) { return u->count; }
const int *oracle_centre_tok(const oracle_unit *u) { return u->centre_tok; }
const int *oracle_slot_tok(const oracle_unit *u) { return u->slot_tok; }
const int *oracle_m_tok(const oracle_unit *u) { return u->m_tok; }
const int *oracle_assign(const oracle_unit *u) { return u->assign; }
const uint64_t *oracle_w(const oracle_unit *u) { return u->W; }
const uint64_t *oracle_ins_d2(const oracle_unit *u) { return u->ins_d2; }
const int *oracle_ins_near(const oracle_unit *u) { return u->ins_near; }
uint64_t oracle_dist2_fx(const float *x, const float *k, int d) { return dist2_fx(x, k, d); }
uint64_t oracle_norm2_fx(const float *v, int d) { return norm2_fx(v, d); }

/* ------------------------------------------------------------------------ */
/* Offline greedy k-center compression with a recent-token window: the variant the paper's end-to-end
 * experiment ran (Section 3.2: keep the most recent r tokens and k centres chosen from the remaining tokens by
 * the greedy k-center algorithm, applied once to the whole cache).
 *
 * Greedy k-center (farthest-point traversal, Dyer and Frieze 1985 / Gonzalez 1985) over the n_old = n - r
 * oldest keys: the first centre is the first key; every further centre is the key farthest from its nearest
 * chosen centre. Readings where the paper is silent: distances are the fixed-point D2 above, so the argmax is an
 * integer decision; ties go to the lowest token index; when n_old <= k every old token is kept. The retained
 * tokens are then attended exactly (Eq. 1 over centres and window), the same budget semantics as the eviction
 * baselines it is compared with.
 *
 * centres[k_out] receives the chosen token indices in selection order, radius2 (may be NULL) the largest
 * fixed-point D2 of an old key to its nearest centre after the selection. Returns k_out = min(k, n_old). */
int oracle_kcenter(const float *K, int n_old, int d, int k, int *centres, uint64_t *radius2) {
    if (n_old <= 0 || k <= 0) { if (radius2) *radius2 = 0; return 0; }
    int k_out = k < n_old ? k : n_old;
    uint64_t *dist = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)n_old);
    for (int i = 0; i < n_old; ++i) dist[i] = UINT64_MAX;
    int c = 0;
    for (int t = 0; t < k_out; ++t) {
        centres[t] = c;
        uint64_t far = 0;
        int far_i = 0;
        for (int i = 0; i < n_old; ++i) {
            uint64_t d2 = dist2_fx(K + (size_t)c * d, K + (size_t)i * d, d);
            if (d2 < dist[i]) dist[i] = d2;
            if (dist[i] > far) { far = dist[i]; far_i = i; }       /* strict: ties keep the lowest index */
        }
        c = far_i;
        if (radius2) *radius2 = far;
    }
    free(dist);
    return k_out;
}
