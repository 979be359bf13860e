/*
 * CPU ORACLE -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.
 *
 * A plain, slow C restatement (single-threaded; one entry point shares the token loop of a
 * sweep among host threads, unchanged, for the benchmark's all-cores figure) of one frozen-counts sweep of
 * the LightLDA Metropolis-Hastings token sampler, written from the paper's
 * equations.  It exists so that the CUDA path can be compared with something
 * that can be checked against the paper by eye.  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may load it.  It shares no code
 * with the CUDA path: everything it needs (Philox, alias construction, the
 * count tables, the acceptance ratios, the log-likelihood) is written out here.
 *
 * What it follows:
 *   - collapsed-LDA target conditional           : Eq. 1 / Eq. 4
 *   - word-proposal and its acceptance ratio     : Eq. 6, Eq. 7, Eq. 8
 *   - sparse-plus-dense mixture for the word side: Section 4.2 (after Eq. 8)
 *   - doc-proposal and its acceptance ratio      : Eq. 9, Eq. 10, Eq. 11
 *   - "the z array is the alias table" for n_kd  : Eq. 12
 *   - alternating (cycle) proposal               : Section 4.3, Eq. 13
 *   - immutable model during sampling            : Section 6, "Multi-thread Efficiency"
 *   - count tables as sufficient statistics      : Section 3 (after Eq. 1)
 *   - log-likelihood, doc part + word part       : Section 7.2 / Figure 11
 *
 * Pins (tests/, CPU only): Philox known-answer vectors and an independent
 * big-integer restatement; alias tables against exact rational masses and two
 * hand-worked tables; proposal histograms against Eq. 6 / Eq. 9 by chi-square;
 * Eq. 8 / Eq. 11 against p(t)q(s)/(p(s)q(t)) built from Eq. 4, 6, 9; the chain
 * against the brute-force Eq. 4 conditional (histogram and exact transition
 * matrix); count invariants and brute-force recount; log-likelihood against a
 * dense double loop.  Sampler QUALITY over many sweeps (how fast the
 * log-likelihood rises) is compared only in trend with a sequential collapsed
 * Gibbs sampler: the paper prints no number for it -- parity unpinned there.
 *
 * Readings taken where the paper is silent are stated at the function that
 * takes them.
 */
#define _POSIX_C_SOURCE 199309L
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <time.h>

#define LDAREF_OK 0
#define LDAREF_EINVAL (-1)
#define LDAREF_ERANGE (-2)
#define LDAREF_ESTATE (-3)
#define LDAREF_ENOMEM (-4)

#define LDAREF_NK 0
#define LDAREF_NWK 1
#define LDAREF_NDK 2

static double wall_seconds(void)
{
    struct timespec ts;
    clock_gettime(CLOCK_MONOTONIC, &ts);
    return (double)ts.tv_sec + 1e-9 * (double)ts.tv_nsec;
}

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as    */
/* easy as 1, 2, 3", SC'11).  The paper under test names no generator; a      */
/* counter-based one makes every random choice a function of (seed, sweep,    */
/* token, step) and therefore independent of execution order.                 */
/* ------------------------------------------------------------------------- */
void ldaref_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Map a 32-bit random word to {0..n-1}: floor(r * n / 2^32). */
static uint32_t scale_to_range(uint32_t r, uint32_t n)
{
    return (uint32_t)(((uint64_t)r * (uint64_t)n) >> 32);
}

static int bit_length(uint64_t x)
{
    int b = 0;
    while (x) { ++b; x >>= 1; }
    return b;
}

/* ------------------------------------------------------------------------- */
/* Alias table (Walker / Vose, the paper's refs [13],[20]; Section 4.2 says    */
/* each bin stores a split point and an alias).  The paper's worked example    */
/* (Figure 2) is not reproduced in the text and many valid tables exist for    */
/* one distribution, so one construction is fixed here, in integers, so that   */
/* a second implementation can reproduce it bit for bit:                       */
/*   - weights arrive as integers wt[i] (fixed point, see weight functions);   */
/*   - W44 = sum wt; all weights are shifted right by                          */
/*       sh = max(0, bitlen(W44) + bitlen(n) - 62)                             */
/*     so that n * sum(w) < 2^62; w[i] = wt[i] >> sh, W = sum w;               */
/*   - every bin has capacity W and item i brings mass a[i] = n * w[i];        */
/*   - items with a[i] <= W are "light", the others "heavy"; both are taken    */
/*     in ascending item order.  Lights are filled from the current heavy      */
/*     item; a heavy item whose remaining mass drops to <= W becomes a bin     */
/*     itself, keeps that remainder, and is topped up by the next heavy item.  */
/* thr[i] is the mass of bin i that stays with item i, alias[i] the item that  */
/* owns the rest (alias[i] == i when the bin is full).                         */
/* Stored split point: thr32 = floor(thr * 2^32 / W) computed on the top 32    */
/* bits of W, saturated to 2^32-1.                                             */
/* ------------------------------------------------------------------------- */
int ldaref_alias_build(int32_t n, const uint64_t *wt, uint32_t *thr32, int32_t *alias,
                       uint64_t *thr_raw /* may be NULL */, uint64_t *W_out, uint64_t *W44_out,
                       int32_t *shift_out)
{
    if (n <= 0 || !wt || !thr32 || !alias) return LDAREF_EINVAL;
    uint64_t W44 = 0;
    for (int32_t i = 0; i < n; ++i) W44 += wt[i];
    int sh = bit_length(W44) + bit_length((uint64_t)n) - 62;
    if (sh < 0) sh = 0;
    uint64_t W = 0;
    for (int32_t i = 0; i < n; ++i) W += wt[i] >> sh;
    if (W == 0) return LDAREF_ERANGE;

    uint64_t *a = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)n);
    uint64_t *thr = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)n);
    int32_t *heavy = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
    if (!a || !thr || !heavy) { free(a); free(thr); free(heavy); return LDAREF_ENOMEM; }
    int32_t H = 0;
    for (int32_t i = 0; i < n; ++i) {
        a[i] = (uint64_t)n * (wt[i] >> sh);
        if (a[i] > W) heavy[H++] = i;
    }
    int32_t h = 0;                       /* current heavy item: heavy[h] */
    uint64_t rest = H ? a[heavy[0]] : 0; /* mass it still holds */
    for (int32_t i = 0; i < n; ++i) {
        if (a[i] > W) continue;          /* lights only, ascending */
        thr[i] = a[i];
        uint64_t deficit = W - a[i];
        if (deficit == 0) { alias[i] = i; continue; }
        alias[i] = heavy[h];
        rest -= deficit;
        while (h < H && rest <= W) {     /* the heavy item became a bin */
            int32_t j = heavy[h];
            thr[j] = rest;
            uint64_t gap = W - rest;
            ++h;
            if (gap == 0) {
                alias[j] = j;
                if (h < H) rest = a[heavy[h]];
            } else {
                alias[j] = heavy[h];     /* exists: total mass is n*W */
                rest = a[heavy[h]] - gap;
            }
        }
    }
    int wsh = bit_length(W) - 32;
    if (wsh < 0) wsh = 0;
    for (int32_t i = 0; i < n; ++i) {
        uint64_t q = ((thr[i] >> wsh) << 32) / (W >> wsh);
        thr32[i] = q > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)q;
        if (thr_raw) thr_raw[i] = thr[i];
    }
    if (W_out) *W_out = W;
    if (W44_out) *W44_out = W44;
    if (shift_out) *shift_out = sh;
    free(a); free(thr); free(heavy);
    return LDAREF_OK;
}

/* One draw from an alias table: r1 picks the bin, r2 is the coin. */
int32_t ldaref_alias_draw(int32_t n, const uint32_t *thr32, const int32_t *alias, uint32_t r1,
                          uint32_t r2)
{
    int32_t b = (int32_t)scale_to_range(r1, (uint32_t)n);
    return (alias[b] == b || r2 < thr32[b]) ? b : alias[b];
}

/* Share of the sparse term in the word-proposal mixture as a 32-bit
 * threshold: floor(S * 2^32 / (S + B)), on the top 32 bits of S + B. */
static uint32_t mixture_threshold(uint64_t S, uint64_t B)
{
    if (S == 0) return 0;
    uint64_t T = S + B;
    int sh = bit_length(T) - 32;
    if (sh < 0) sh = 0;
    uint64_t q = ((S >> sh) << 32) / (T >> sh);
    return q > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)q;
}

/* ------------------------------------------------------------------------- */
/* Sampler state                                                             */
/* ------------------------------------------------------------------------- */
typedef struct ldaref_ctx {
    int32_t V, K;
    double alpha, beta;
    double Vbeta;    /* beta-bar = sum_w beta_w = V*beta (symmetric prior) */
    double Kalpha;   /* sum_k alpha_k = K*alpha */
    int64_t N, D;
    int32_t *word;       /* [N] word of token i (caller's document order) */
    int64_t *doc_off;    /* [D+1] */
    int32_t *doc_of;     /* [N] document of token i */
    int64_t *word_off;   /* [V+1] tokens of word w: word_tok[word_off[w]..word_off[w+1]) */
    int32_t *word_tok;   /* [N] token ids grouped by word, ascending inside a word */
    int32_t *z;          /* [N] current assignments */
    int32_t *z_new;      /* [N] */
    /* cached sufficient statistics (Section 3): n_k dense, n_kw as per-word
     * lists of (topic, count) over the nonzero entries, topics ascending.
     * n_kd is not cached: it is counted from the document's z (Eq. 12). */
    int64_t *nk;         /* [K] */
    int64_t *row_off;    /* [V+1] */
    int32_t *row_topic;  /* [nnz] */
    int32_t *row_count;  /* [nnz] */
    /* proposal tables built from the frozen counts */
    uint32_t *sp_thr32;  /* [nnz] per-word sparse alias tables (same indexing as rows) */
    int32_t *sp_alias;   /* [nnz] item index inside the word's row */
    uint32_t *mix32;     /* [V] */
    uint32_t *dn_thr32;  /* [K] dense table shared by all words */
    int32_t *dn_alias;   /* [K] */
    uint64_t dense_mass; /* B: sum of the dense fixed-point weights */
    int tables_valid;
    uint64_t seed;
    uint32_t sweep;      /* number of sweeps done since init */
    int proposals;       /* 0 cycle (word, doc, word, ...), 1 word-proposal only, 2 doc-proposal only */
    uint32_t tok_base;   /* Philox token key of token 0 (nonzero when the corpus is one shard of a larger one) */
    int64_t row_cap;     /* entries the four row arrays (row_*, sp_*) can hold */
    int64_t moves[2];    /* steps of the last sweep call that moved a chain: word-, doc-proposals */
    int loaded, inited;
} ldaref_ctx;

static const double FIXED_ONE = 17592186044416.0; /* 2^44 */

/* Fixed-point weight of a nonzero entry of the sparse term n_kw / (n_k + beta-bar). */
static uint64_t sparse_weight(const ldaref_ctx *c, int32_t n_kw, int64_t n_k)
{
    double den = (double)n_k + c->Vbeta;
    return (uint64_t)(((double)n_kw / den) * FIXED_ONE);
}

/* Fixed-point weight of topic k in the dense term beta_w / (n_k + beta-bar). */
static uint64_t dense_weight(const ldaref_ctx *c, int64_t n_k)
{
    double den = (double)n_k + c->Vbeta;
    return (uint64_t)((c->beta / den) * FIXED_ONE);
}

int ldaref_create(int32_t V, int32_t K, double alpha, double beta, ldaref_ctx **out)
{
    if (!out) return LDAREF_EINVAL;
    *out = NULL;
    if (V <= 0 || K <= 0 || !(alpha > 0) || !(beta > 0) || !isfinite(alpha) || !isfinite(beta))
        return LDAREF_EINVAL;
    if (K > 131072) return LDAREF_ERANGE;
    ldaref_ctx *c = (ldaref_ctx *)calloc(1, sizeof(ldaref_ctx));
    if (!c) return LDAREF_ENOMEM;
    c->V = V; c->K = K; c->alpha = alpha; c->beta = beta;
    c->Vbeta = (double)V * beta;
    c->Kalpha = (double)K * alpha;
    *out = c;
    return LDAREF_OK;
}

static void free_corpus(ldaref_ctx *c)
{
    free(c->word); free(c->doc_off); free(c->doc_of); free(c->word_off); free(c->word_tok);
    free(c->z); free(c->z_new); free(c->nk); free(c->row_off); free(c->row_topic);
    free(c->row_count); free(c->sp_thr32); free(c->sp_alias); free(c->mix32);
    free(c->dn_thr32); free(c->dn_alias);
    c->word = NULL; c->doc_off = NULL; c->doc_of = NULL; c->word_off = NULL; c->word_tok = NULL;
    c->z = NULL; c->z_new = NULL; c->nk = NULL; c->row_off = NULL; c->row_topic = NULL;
    c->row_count = NULL; c->sp_thr32 = NULL; c->sp_alias = NULL; c->mix32 = NULL;
    c->dn_thr32 = NULL; c->dn_alias = NULL;
    c->loaded = c->inited = c->tables_valid = 0;
}

void ldaref_destroy(ldaref_ctx *c)
{
    if (!c) return;
    free_corpus(c);
    free(c);
}

int ldaref_load_corpus(ldaref_ctx *c, const int32_t *word_ids, int64_t n_tokens,
                       const int64_t *doc_offsets, int64_t n_docs)
{
    if (!c || !doc_offsets || n_tokens < 0 || n_docs < 0 || (n_tokens > 0 && !word_ids))
        return LDAREF_EINVAL;
    if (n_tokens >= 2147483648LL) return LDAREF_ERANGE;
    if (doc_offsets[0] != 0 || doc_offsets[n_docs] != n_tokens) return LDAREF_ERANGE;
    for (int64_t d = 0; d < n_docs; ++d)
        if (doc_offsets[d + 1] < doc_offsets[d]) return LDAREF_ERANGE;
    for (int64_t i = 0; i < n_tokens; ++i)
        if (word_ids[i] < 0 || word_ids[i] >= c->V) return LDAREF_ERANGE;
    free_corpus(c);
    int64_t N = n_tokens, D = n_docs;
    size_t n1 = (size_t)(N > 0 ? N : 1);
    c->N = N; c->D = D;
    c->row_cap = (int64_t)n1;
    c->word = (int32_t *)malloc(sizeof(int32_t) * n1);
    c->doc_off = (int64_t *)malloc(sizeof(int64_t) * (size_t)(D + 1));
    c->doc_of = (int32_t *)malloc(sizeof(int32_t) * n1);
    c->word_off = (int64_t *)calloc((size_t)c->V + 1, sizeof(int64_t));
    c->word_tok = (int32_t *)malloc(sizeof(int32_t) * n1);
    c->z = (int32_t *)malloc(sizeof(int32_t) * n1);
    c->z_new = (int32_t *)malloc(sizeof(int32_t) * n1);
    c->nk = (int64_t *)calloc((size_t)c->K, sizeof(int64_t));
    c->row_off = (int64_t *)calloc((size_t)c->V + 1, sizeof(int64_t));
    c->row_topic = (int32_t *)malloc(sizeof(int32_t) * n1);
    c->row_count = (int32_t *)malloc(sizeof(int32_t) * n1);
    c->sp_thr32 = (uint32_t *)malloc(sizeof(uint32_t) * n1);
    c->sp_alias = (int32_t *)malloc(sizeof(int32_t) * n1);
    c->mix32 = (uint32_t *)calloc((size_t)c->V, sizeof(uint32_t));
    c->dn_thr32 = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)c->K);
    c->dn_alias = (int32_t *)malloc(sizeof(int32_t) * (size_t)c->K);
    if (!c->word || !c->doc_off || !c->doc_of || !c->word_off || !c->word_tok || !c->z ||
        !c->z_new || !c->nk || !c->row_off || !c->row_topic || !c->row_count || !c->sp_thr32 ||
        !c->sp_alias || !c->mix32 || !c->dn_thr32 || !c->dn_alias) {
        free_corpus(c);
        return LDAREF_ENOMEM;
    }
    if (N > 0) memcpy(c->word, word_ids, sizeof(int32_t) * (size_t)N);
    memcpy(c->doc_off, doc_offsets, sizeof(int64_t) * (size_t)(D + 1));
    for (int64_t d = 0; d < D; ++d)
        for (int64_t i = doc_offsets[d]; i < doc_offsets[d + 1]; ++i) c->doc_of[i] = (int32_t)d;
    /* group token ids by word (counting sort; ascending token id inside a word) */
    for (int64_t i = 0; i < N; ++i) c->word_off[c->word[i] + 1] += 1;
    for (int32_t w = 0; w < c->V; ++w) c->word_off[w + 1] += c->word_off[w];
    int64_t *cursor = (int64_t *)malloc(sizeof(int64_t) * (size_t)c->V);
    if (!cursor) { free_corpus(c); return LDAREF_ENOMEM; }
    memcpy(cursor, c->word_off, sizeof(int64_t) * (size_t)c->V);
    for (int64_t i = 0; i < N; ++i) c->word_tok[cursor[c->word[i]]++] = (int32_t)i;
    free(cursor);
    c->loaded = 1;
    return LDAREF_OK;
}

static int cmp_i32(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/* Count tables from the assignments (Section 3: n_k, n_kw are counts of
 * tokens; Eq. 12 for n_kd, which is counted on demand). */
static int rebuild_counts(ldaref_ctx *c)
{
    int32_t K = c->K;
    memset(c->nk, 0, sizeof(int64_t) * (size_t)K);
    for (int64_t i = 0; i < c->N; ++i) c->nk[c->z[i]] += 1;
    int32_t *tally = (int32_t *)calloc((size_t)K, sizeof(int32_t));
    int32_t *seen = (int32_t *)malloc(sizeof(int32_t) * (size_t)K);
    if (!tally || !seen) { free(tally); free(seen); return LDAREF_ENOMEM; }
    int64_t nnz = 0;
    for (int32_t w = 0; w < c->V; ++w) {
        c->row_off[w] = nnz;
        int32_t n_seen = 0;
        for (int64_t p = c->word_off[w]; p < c->word_off[w + 1]; ++p) {
            int32_t k = c->z[c->word_tok[p]];
            if (tally[k]++ == 0) seen[n_seen++] = k;
        }
        qsort(seen, (size_t)n_seen, sizeof(int32_t), cmp_i32);
        for (int32_t j = 0; j < n_seen; ++j) {
            c->row_topic[nnz] = seen[j];
            c->row_count[nnz] = tally[seen[j]];
            tally[seen[j]] = 0;
            ++nnz;
        }
    }
    c->row_off[c->V] = nnz;
    free(tally); free(seen);
    c->tables_valid = 0;
    return LDAREF_OK;
}

/* n_kw lookup in the word's sorted nonzero list. */
static int32_t count_wk(const ldaref_ctx *c, int32_t w, int32_t k)
{
    int64_t lo = c->row_off[w], hi = c->row_off[w + 1];
    while (lo < hi) {
        int64_t mid = lo + (hi - lo) / 2;
        if (c->row_topic[mid] < k) lo = mid + 1; else hi = mid;
    }
    return (lo < c->row_off[w + 1] && c->row_topic[lo] == k) ? c->row_count[lo] : 0;
}

/* n_kd = sum_i [z_di = k]  (Eq. 12), counted from the document's z. */
static int32_t count_dk(const ldaref_ctx *c, int32_t d, int32_t k)
{
    int32_t n = 0;
    for (int64_t j = c->doc_off[d]; j < c->doc_off[d + 1]; ++j) n += (c->z[j] == k);
    return n;
}

/* Initial assignments.  The paper does not say how z starts; taken here:
 * z_i uniform on {0..K-1} from Philox counter (i, 0, 0, 1), word 0. */
int ldaref_init(ldaref_ctx *c, uint64_t seed)
{
    if (!c) return LDAREF_EINVAL;
    if (!c->loaded) return LDAREF_ESTATE;
    c->seed = seed;
    c->sweep = 0;
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    for (int64_t i = 0; i < c->N; ++i) {
        uint32_t ctr[4] = {c->tok_base + (uint32_t)i, 0u, 0u, 1u}, r[4];
        ldaref_philox4x32_10(ctr, key, r);
        c->z[i] = (int32_t)scale_to_range(r[0], (uint32_t)c->K);
    }
    int rc = rebuild_counts(c);
    if (rc) return rc;
    c->inited = 1;
    return LDAREF_OK;
}

/* Warm start from given assignments (Section 6: counts are re-initialised from z). */
int ldaref_set_assignments(ldaref_ctx *c, const int32_t *z, uint64_t seed, uint32_t sweep)
{
    if (!c || (c->N > 0 && !z)) return LDAREF_EINVAL;
    if (!c->loaded) return LDAREF_ESTATE;
    for (int64_t i = 0; i < c->N; ++i)
        if (z[i] < 0 || z[i] >= c->K) return LDAREF_ERANGE;
    if (c->N > 0) memcpy(c->z, z, sizeof(int32_t) * (size_t)c->N);
    c->seed = seed;
    c->sweep = sweep;
    int rc = rebuild_counts(c);
    if (rc) return rc;
    c->inited = 1;
    return LDAREF_OK;
}

/* Proposal tables for the word side (Section 4.2): the word-proposal
 * (n_kw + beta_w)/(n_k + beta-bar) is split into a sparse term over the
 * word's nonzero n_kw (one alias table per word) and a dense term
 * beta_w/(n_k + beta-bar) whose alias table is shared by all words.  A term
 * is picked with probability proportional to its mass. */
int ldaref_build_tables(ldaref_ctx *c)
{
    if (!c) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    int32_t K = c->K;
    uint64_t *wt = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)K);
    if (!wt) return LDAREF_ENOMEM;
    for (int32_t k = 0; k < K; ++k) wt[k] = dense_weight(c, c->nk[k]);
    int rc = ldaref_alias_build(K, wt, c->dn_thr32, c->dn_alias, NULL, NULL, &c->dense_mass, NULL);
    if (rc) { free(wt); return rc; }
    for (int32_t w = 0; w < c->V; ++w) {
        int64_t off = c->row_off[w];
        int32_t n = (int32_t)(c->row_off[w + 1] - off);
        if (n == 0) { c->mix32[w] = 0; continue; }
        for (int32_t j = 0; j < n; ++j)
            wt[j] = sparse_weight(c, c->row_count[off + j], c->nk[c->row_topic[off + j]]);
        uint64_t S = 0;
        rc = ldaref_alias_build(n, wt, c->sp_thr32 + off, c->sp_alias + off, NULL, NULL, &S, NULL);
        if (rc) { free(wt); return rc; }
        c->mix32[w] = mixture_threshold(S, c->dense_mass);
    }
    free(wt);
    c->tables_valid = 1;
    return LDAREF_OK;
}

/* Draw from the word-proposal of word w (Eq. 6 via the mixture):
 * r0 picks the term, r1 the bin, r2 is the alias coin. */
static int32_t draw_word_proposal(const ldaref_ctx *c, int32_t w, uint32_t r0, uint32_t r1,
                                  uint32_t r2)
{
    if (r0 < c->mix32[w]) {
        int64_t off = c->row_off[w];
        int32_t n = (int32_t)(c->row_off[w + 1] - off);
        int32_t item = ldaref_alias_draw(n, c->sp_thr32 + off, c->sp_alias + off, r1, r2);
        return c->row_topic[off + item];
    }
    return ldaref_alias_draw(c->K, c->dn_thr32, c->dn_alias, r1, r2);
}

/* Draw from the doc-proposal of document d (Eq. 9): with probability
 * n_d / (n_d + sum_k alpha_k) copy the topic of a uniformly chosen token of
 * the document (Eq. 12: z itself is the alias table for n_kd; the token
 * being sampled is included, since Eq. 9 carries no "-di"), else a uniform
 * topic.  r0 picks the term, r1 the position / topic. */
static int32_t draw_doc_proposal(const ldaref_ctx *c, int32_t d, uint32_t r0, uint32_t r1)
{
    int64_t n_d = c->doc_off[d + 1] - c->doc_off[d];
    double u = (double)r0 * (1.0 / 4294967296.0);
    if (u * ((double)n_d + c->Kalpha) < (double)n_d)
        return c->z[c->doc_off[d] + scale_to_range(r1, (uint32_t)n_d)];
    return (int32_t)scale_to_range(r1, (uint32_t)c->K);
}

/* Numerator and denominator of the acceptance ratio for moving token i from
 * state s to state t.  kind 0: word-proposal, Eq. 8.  kind 1: doc-proposal,
 * Eq. 11.  The "-di" counts exclude the token's own contribution; with
 * counts frozen at sweep start that contribution sits at z0 = the
 * assignment the token had when the counts were taken, whatever the chain's
 * current state is.  Proposal factors carry no "-di" (Eq. 6, Eq. 9). */
static void accept_ratio(const ldaref_ctx *c, int64_t i, int32_t s, int32_t t, int kind,
                         double *num, double *den)
{
    int32_t w = c->word[i], d = c->doc_of[i], z0 = c->z[i];
    int32_t e_s = (s == z0), e_t = (t == z0);
    int32_t n_sd = count_dk(c, d, s), n_td = count_dk(c, d, t);
    int32_t n_sw = count_wk(c, w, s), n_tw = count_wk(c, w, t);
    int64_t n_s = c->nk[s], n_t = c->nk[t];
    double a = c->alpha, b = c->beta, bb = c->Vbeta;
    double nu = (double)(n_td - e_t) + a;
    nu = nu * ((double)(n_tw - e_t) + b);
    nu = nu * ((double)(n_s - e_s) + bb);
    double de = (double)(n_sd - e_s) + a;
    de = de * ((double)(n_sw - e_s) + b);
    de = de * ((double)(n_t - e_t) + bb);
    if (kind == 0) {
        nu = nu * ((double)n_sw + b);
        nu = nu * ((double)n_t + bb);
        de = de * ((double)n_tw + b);
        de = de * ((double)n_s + bb);
    } else {
        nu = nu * ((double)n_sd + a);
        de = de * ((double)n_td + a);
    }
    *num = nu;
    *den = de;
}

/* The MH chain of one token for one sweep (Section 4.3): `steps` individual
 * proposals, word-proposal on even steps and doc-proposal on odd steps (the
 * paper alternates the two and does not fix which comes first or how a
 * "step" is counted; taken here: one step = one proposal, word first).
 * Every step uses one Philox block, counter (token, sweep, step, 0):
 * r0 term choice, r1 index, r2 alias coin, r3 acceptance.  A proposal equal
 * to the current state changes nothing; otherwise accept iff u*den < num
 * with u = r3 / 2^32, which accepts with probability min{1, num/den}
 * (Eq. 7, Eq. 10). */
static int32_t run_chain(const ldaref_ctx *c, int64_t i, uint32_t sweep, int32_t steps, int64_t *moves)
{
    uint32_t key[2] = {(uint32_t)c->seed, (uint32_t)(c->seed >> 32)};
    int32_t s = c->z[i];
    for (int32_t m = 0; m < steps; ++m) {
        uint32_t ctr[4] = {c->tok_base + (uint32_t)i, sweep, (uint32_t)m, 0u}, r[4];
        ldaref_philox4x32_10(ctr, key, r);
        /* Section 4.3: the cycle alternates the two proposals; each alone is a valid MH kernel
         * for the same target (the variants compared in Figure 11) */
        int kind = c->proposals == 0 ? (m & 1) : c->proposals - 1;
        int32_t t = kind == 0 ? draw_word_proposal(c, c->word[i], r[0], r[1], r[2])
                              : draw_doc_proposal(c, c->doc_of[i], r[0], r[1]);
        if (t == s) continue;
        double num, den;
        accept_ratio(c, i, s, t, kind, &num, &den);
        double u = (double)r[3] * (1.0 / 4294967296.0);
        if (u * den < num) {
            s = t;
            if (moves) moves[kind] += 1; /* accepted, and the state changed (t != s) */
        }
    }
    return s;
}

/* Which proposals a chain uses (Section 4.3, Figure 11): 0 = cycle (default), 1 = word-proposal
 * on every step, 2 = doc-proposal on every step. */
int ldaref_set_proposals(ldaref_ctx *c, int mode)
{
    if (!c || mode < 0 || mode > 2) return LDAREF_EINVAL;
    c->proposals = mode;
    return LDAREF_OK;
}

/* `iters` sweeps.  During a sweep every count and every z that is read is the
 * sweep-start value (Section 6: the model is immutable while sampled and
 * updates are applied afterwards; here the document side is frozen as well,
 * so a sweep does not depend on the order tokens are visited in). */
int ldaref_sweep(ldaref_ctx *c, int32_t iters, int32_t mh_steps)
{
    if (!c || iters < 0 || mh_steps < 1) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    c->moves[0] = c->moves[1] = 0;
    for (int32_t it = 0; it < iters; ++it) {
        int rc = ldaref_build_tables(c);
        if (rc) return rc;
        for (int64_t i = 0; i < c->N; ++i) c->z_new[i] = run_chain(c, i, c->sweep, mh_steps, c->moves);
        int32_t *tmp = c->z; c->z = c->z_new; c->z_new = tmp;
        rc = rebuild_counts(c);
        if (rc) return rc;
        c->sweep += 1;
    }
    return LDAREF_OK;
}

/* New assignments of a bounded set of tokens for the NEXT sweep, without
 * changing state (used where a whole sweep is too slow to run). */
int ldaref_sample_tokens(ldaref_ctx *c, const int64_t *tokens, int64_t n, int32_t mh_steps,
                         int32_t *z_out)
{
    if (!c || !tokens || !z_out || n < 0 || mh_steps < 1) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if (!c->tables_valid) { int rc = ldaref_build_tables(c); if (rc) return rc; }
    for (int64_t j = 0; j < n; ++j) {
        if (tokens[j] < 0 || tokens[j] >= c->N) return LDAREF_ERANGE;
        z_out[j] = run_chain(c, tokens[j], c->sweep, mh_steps, NULL);
    }
    return LDAREF_OK;
}

/* The first `n` tokens of one sweep, timed by the benchmark's CPU leg. */
int ldaref_sweep_prefix(ldaref_ctx *c, int64_t n, int32_t mh_steps, int32_t *z_out)
{
    if (!c || !z_out || n < 0 || n > (c ? c->N : 0) || mh_steps < 1) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if (!c->tables_valid) { int rc = ldaref_build_tables(c); if (rc) return rc; }
    for (int64_t i = 0; i < n; ++i) z_out[i] = run_chain(c, i, c->sweep, mh_steps, NULL);
    return LDAREF_OK;
}

/* The same sweep with the token loop shared among `threads` host threads (OpenMP).  Every chain
 * reads only the sweep-start state and writes only its own z_new[i] (Section 6: the model is
 * immutable while sampled), so the result is the serial sweep's, token for token; the table build
 * and the count rebuild stay serial.  seconds[0..2], when given, receive the wall time of the
 * table build, the token loop and the count rebuild, summed over the iterations. */
int ldaref_sweep_threads(ldaref_ctx *c, int32_t iters, int32_t mh_steps, int32_t threads,
                         double *seconds)
{
    if (!c || iters < 0 || mh_steps < 1 || threads < 1) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if (seconds) seconds[0] = seconds[1] = seconds[2] = 0.0;
    int64_t moves_w = 0, moves_d = 0;
    for (int32_t it = 0; it < iters; ++it) {
        double t0 = wall_seconds();
        int rc = ldaref_build_tables(c);
        if (rc) return rc;
        double t1 = wall_seconds();
        const int64_t N = c->N;
        const uint32_t sweep = c->sweep;
        int32_t *z_new = c->z_new;
#pragma omp parallel for num_threads(threads) schedule(static) reduction(+ : moves_w, moves_d)
        for (int64_t i = 0; i < N; ++i) {
            int64_t mv[2] = {0, 0};
            z_new[i] = run_chain(c, i, sweep, mh_steps, mv);
            moves_w += mv[0];
            moves_d += mv[1];
        }
        double t2 = wall_seconds();
        int32_t *tmp = c->z; c->z = c->z_new; c->z_new = tmp;
        rc = rebuild_counts(c);
        if (rc) return rc;
        c->sweep += 1;
        double t3 = wall_seconds();
        if (seconds) { seconds[0] += t1 - t0; seconds[1] += t2 - t1; seconds[2] += t3 - t2; }
    }
    c->moves[0] = moves_w;
    c->moves[1] = moves_d;
    return LDAREF_OK;
}

/* Chain of token i under an arbitrary sweep index and step count, state
 * untouched: lets a test replicate the chain over many Philox streams. */
int ldaref_chain(ldaref_ctx *c, int64_t token, uint32_t sweep, int32_t steps, int32_t *z_out)
{
    if (!c || !z_out || steps < 0) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if (token < 0 || token >= c->N) return LDAREF_ERANGE;
    if (!c->tables_valid) { int rc = ldaref_build_tables(c); if (rc) return rc; }
    *z_out = run_chain(c, token, sweep, steps, NULL);
    return LDAREF_OK;
}

int ldaref_word_proposal(ldaref_ctx *c, int32_t w, uint32_t r0, uint32_t r1, uint32_t r2,
                         int32_t *t_out)
{
    if (!c || !t_out) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if (w < 0 || w >= c->V) return LDAREF_ERANGE;
    if (!c->tables_valid) { int rc = ldaref_build_tables(c); if (rc) return rc; }
    *t_out = draw_word_proposal(c, w, r0, r1, r2);
    return LDAREF_OK;
}

int ldaref_doc_proposal(ldaref_ctx *c, int32_t d, uint32_t r0, uint32_t r1, int32_t *t_out)
{
    if (!c || !t_out) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if (d < 0 || d >= c->D || c->doc_off[d + 1] == c->doc_off[d]) return LDAREF_ERANGE;
    *t_out = draw_doc_proposal(c, d, r0, r1);
    return LDAREF_OK;
}

int ldaref_accept_ratio(ldaref_ctx *c, int64_t token, int32_t s, int32_t t, int32_t kind,
                        double *num, double *den)
{
    if (!c || !num || !den || (kind != 0 && kind != 1)) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if (token < 0 || token >= c->N || s < 0 || s >= c->K || t < 0 || t >= c->K)
        return LDAREF_ERANGE;
    accept_ratio(c, token, s, t, kind, num, den);
    return LDAREF_OK;
}

/* Collapsed joint log p(w, z | alpha, beta) split into its word part and its
 * document part (the decomposition plotted in Figure 11; the paper defers the
 * formula to its ref. [18] -- this is the standard Dirichlet-multinomial one):
 *   word = K*lgamma(V*beta) + sum_{n_kw>0} [lgamma(n_kw+beta) - lgamma(beta)]
 *          - sum_k lgamma(n_k + V*beta)
 *   doc  = D*lgamma(K*alpha) + sum_{n_kd>0} [lgamma(n_kd+alpha) - lgamma(alpha)]
 *          - sum_d lgamma(n_d + K*alpha)                                       */
/* ------------------------------------------------------------------------- */
/* Exact-conditional yardstick (Section 3, Eq. 1; Section 4, Eq. 3).           */
/*                                                                             */
/* What the MH chain approximates with a few O(1) steps per token is one draw  */
/* from the collapsed conditional of Eq. 1.  Two samplers draw it exactly:     */
/*   - the frozen sweep: every token draws from Eq. 1 under the sweep-start    */
/*     counts (the token's own contribution removed), the like-for-like        */
/*     yardstick of the frozen MH sweep above;                                  */
/*   - the sequential sweep: the textbook collapsed Gibbs sampler, counts      */
/*     updated after every token (the samplers of Figures 12-14 work so).      */
/* The frozen sweep splits Eq. 1 as Eq. 3 does,                                 */
/*   p(k) ~ n_kd'(n_kw'+beta)/(n_k'+V beta)  +  alpha (n_kw'+beta)/(n_k'+V beta) */
/* (primes: token removed), a term over the document's topics plus a term over  */
/* all topics, and draws by inverse CDF over integer masses (each term floored  */
/* at 2^-44), so that the draw is a function of the counts alone, whatever the  */
/* order a second implementation adds the terms in.  One Philox word per        */
/* token and sweep: counter (token, sweep, 0, 2) for the frozen sweep,          */
/* (token, sweep, 0, 3) for the sequential one.  The paper is silent on all of  */
/* this (its Gibbs samplers are other people's systems): these are readings.    */
/* ------------------------------------------------------------------------- */

/* floor(x * 2^44) of the document term and of the smoothing term of Eq. 3 */
static uint64_t gibbs_doc_term(const ldaref_ctx *c, int32_t n_kd, int32_t n_kw, int64_t n_k)
{
    double x = ((double)n_kd * ((double)n_kw + c->beta)) / ((double)n_k + c->Vbeta);
    return (uint64_t)(x * FIXED_ONE);
}

static uint64_t gibbs_prior_term(const ldaref_ctx *c, int32_t n_kw, int64_t n_k)
{
    double x = (c->alpha * ((double)n_kw + c->beta)) / ((double)n_k + c->Vbeta);
    return (uint64_t)(x * FIXED_ONE);
}

/* Integer masses of token i under the frozen counts: doc_mass[k] (zero outside the document's
 * topics) and prior_mass[k], k = 0..K-1; `tally` holds the document's n_kd (all K entries). */
static void gibbs_masses(const ldaref_ctx *c, int64_t i, const int32_t *tally, uint64_t *doc_mass,
                         uint64_t *prior_mass)
{
    int32_t w = c->word[i], z0 = c->z[i];
    for (int32_t k = 0; k < c->K; ++k) {
        int32_t own = (k == z0);
        int32_t n_kd = tally[k] - own, n_kw = count_wk(c, w, k) - own;
        int64_t n_k = c->nk[k] - own;
        doc_mass[k] = n_kd > 0 ? gibbs_doc_term(c, n_kd, n_kw, n_k) : 0;
        prior_mass[k] = gibbs_prior_term(c, n_kw, n_k);
    }
}

/* Inverse CDF: the document term's topics first (ascending), then the smoothing term's. */
static int32_t gibbs_pick(int32_t K, const uint64_t *doc_mass, const uint64_t *prior_mass, uint32_t r0)
{
    uint64_t sum_doc = 0, sum_prior = 0;
    for (int32_t k = 0; k < K; ++k) { sum_doc += doc_mass[k]; sum_prior += prior_mass[k]; }
    uint64_t total = sum_doc + sum_prior;
    uint64_t x = (uint64_t)(((unsigned __int128)total * r0) >> 32); /* floor(total * r0 / 2^32) < total */
    const uint64_t *m = doc_mass;
    if (x >= sum_doc) { x -= sum_doc; m = prior_mass; }
    uint64_t cum = 0;
    for (int32_t k = 0; k < K; ++k) {
        cum += m[k];
        if (cum > x) return k;
    }
    return K - 1; /* not reached: x < the bucket's sum */
}

static int gibbs_limits(const ldaref_ctx *c)
{
    /* the document term is at most n_d * 2^44: sums stay below 2^63 for documents shorter than 2^19 */
    for (int64_t d = 0; d < c->D; ++d)
        if (c->doc_off[d + 1] - c->doc_off[d] >= (1 << 19)) return LDAREF_ERANGE;
    return LDAREF_OK;
}

/* `iters` frozen exact-conditional sweeps, the documents shared among `threads` host threads. */
int ldaref_gibbs_sweep(ldaref_ctx *c, int32_t iters, int32_t threads)
{
    if (!c || iters < 0 || threads < 1) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    int rc = gibbs_limits(c);
    if (rc) return rc;
    uint32_t key[2] = {(uint32_t)c->seed, (uint32_t)(c->seed >> 32)};
    for (int32_t it = 0; it < iters; ++it) {
        int failed = 0;
#pragma omp parallel num_threads(threads)
        {
            int32_t *tally = (int32_t *)calloc((size_t)c->K, sizeof(int32_t));
            uint64_t *dm = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)c->K);
            uint64_t *pm = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)c->K);
            if (!tally || !dm || !pm) {
#pragma omp atomic write
                failed = 1;
            } else {
#pragma omp for schedule(dynamic, 64)
                for (int64_t d = 0; d < c->D; ++d) {
                    int64_t lo = c->doc_off[d], hi = c->doc_off[d + 1];
                    for (int64_t j = lo; j < hi; ++j) tally[c->z[j]] += 1;
                    for (int64_t i = lo; i < hi; ++i) {
                        uint32_t ctr[4] = {c->tok_base + (uint32_t)i, c->sweep, 0u, 2u}, r[4];
                        ldaref_philox4x32_10(ctr, key, r);
                        gibbs_masses(c, i, tally, dm, pm);
                        c->z_new[i] = gibbs_pick(c->K, dm, pm, r[0]);
                    }
                    for (int64_t j = lo; j < hi; ++j) tally[c->z[j]] = 0;
                }
            }
            free(tally); free(dm); free(pm);
        }
        if (failed) return LDAREF_ENOMEM;
        int32_t *tmp = c->z; c->z = c->z_new; c->z_new = tmp;
        rc = rebuild_counts(c);
        if (rc) return rc;
        c->sweep += 1;
    }
    return LDAREF_OK;
}

/* The integer masses of one token under the current counts -- doc_mass_out[K] (document term) and
 * prior_mass_out[K] (smoothing term) -- and the topic the frozen sweep would pick for it given the
 * random word r0. */
int ldaref_gibbs_masses(ldaref_ctx *c, int64_t token, uint64_t *doc_mass_out, uint64_t *prior_mass_out,
                        uint32_t r0, int32_t *pick_out)
{
    if (!c || !doc_mass_out || !prior_mass_out) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if (token < 0 || token >= c->N) return LDAREF_ERANGE;
    int32_t *tally = (int32_t *)calloc((size_t)c->K, sizeof(int32_t));
    uint64_t *dm = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)c->K);
    uint64_t *pm = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)c->K);
    if (!tally || !dm || !pm) { free(tally); free(dm); free(pm); return LDAREF_ENOMEM; }
    int32_t d = c->doc_of[token];
    for (int64_t j = c->doc_off[d]; j < c->doc_off[d + 1]; ++j) tally[c->z[j]] += 1;
    gibbs_masses(c, token, tally, dm, pm);
    for (int32_t k = 0; k < c->K; ++k) { doc_mass_out[k] = dm[k]; prior_mass_out[k] = pm[k]; }
    if (pick_out) *pick_out = gibbs_pick(c->K, dm, pm, r0);
    free(tally); free(dm); free(pm);
    return LDAREF_OK;
}

/* `iters` sweeps of the sequential collapsed Gibbs sampler (Eq. 1): tokens in document order,
 * every count updated as soon as a token is redrawn; plain floating-point inverse CDF. */
int ldaref_gibbs_sweep_sequential(ldaref_ctx *c, int32_t iters)
{
    if (!c || iters < 0) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if ((int64_t)c->V * c->K > ((int64_t)1 << 31)) return LDAREF_ERANGE; /* a dense n_kw is kept */
    uint32_t key[2] = {(uint32_t)c->seed, (uint32_t)(c->seed >> 32)};
    int32_t K = c->K;
    int32_t *n_wk = (int32_t *)calloc((size_t)c->V * (size_t)K, sizeof(int32_t));
    int32_t *n_dk = (int32_t *)calloc((size_t)K, sizeof(int32_t));
    int64_t *n_k = (int64_t *)calloc((size_t)K, sizeof(int64_t));
    double *cum = (double *)malloc(sizeof(double) * (size_t)K);
    if (!n_wk || !n_dk || !n_k || !cum) { free(n_wk); free(n_dk); free(n_k); free(cum); return LDAREF_ENOMEM; }
    for (int64_t i = 0; i < c->N; ++i) { n_wk[(size_t)c->word[i] * K + c->z[i]] += 1; n_k[c->z[i]] += 1; }
    for (int32_t it = 0; it < iters; ++it) {
        for (int64_t d = 0; d < c->D; ++d) {
            int64_t lo = c->doc_off[d], hi = c->doc_off[d + 1];
            for (int64_t j = lo; j < hi; ++j) n_dk[c->z[j]] += 1;
            for (int64_t i = lo; i < hi; ++i) {
                int32_t *row = n_wk + (size_t)c->word[i] * K;
                int32_t s = c->z[i];
                n_dk[s] -= 1; row[s] -= 1; n_k[s] -= 1;       /* the counts without token i */
                double total = 0.0;
                for (int32_t k = 0; k < K; ++k) {
                    total += ((double)n_dk[k] + c->alpha) * ((double)row[k] + c->beta) /
                             ((double)n_k[k] + c->Vbeta);      /* Eq. 1 */
                    cum[k] = total;
                }
                uint32_t ctr[4] = {c->tok_base + (uint32_t)i, c->sweep, 0u, 3u}, r[4];
                ldaref_philox4x32_10(ctr, key, r);
                double u = (double)r[0] * (1.0 / 4294967296.0) * total;
                int32_t t = 0;
                while (t < K - 1 && cum[t] <= u) ++t;
                c->z[i] = t;
                n_dk[t] += 1; row[t] += 1; n_k[t] += 1;
            }
            for (int64_t j = lo; j < hi; ++j) n_dk[c->z[j]] = 0;
        }
        c->sweep += 1;
    }
    free(n_wk); free(n_dk); free(n_k); free(cum);
    return rebuild_counts(c);
}

/* ------------------------------------------------------------------------- */
/* Document shards (Section 6, "Parameter Server and Data Placement": the      */
/* documents are partitioned over the workers, the word-topic table is        */
/* shared).  An oracle context may hold a run of consecutive documents of a   */
/* larger corpus: first_token is the index of its first token there and       */
/* offsets the Philox token key; n_kw travels as a dense V x K matrix, the    */
/* caller adds the shards' matrices up and hands the sum back before a sweep. */
/* ------------------------------------------------------------------------- */
int ldaref_set_shard(ldaref_ctx *c, int64_t first_token)
{
    if (!c || first_token < 0 || first_token >= ((int64_t)1 << 32)) return LDAREF_EINVAL;
    c->tok_base = (uint32_t)first_token;
    return LDAREF_OK;
}

int ldaref_word_counts_to_dense(const ldaref_ctx *c, int32_t *out)
{
    if (!c || !out) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    memset(out, 0, sizeof(int32_t) * (size_t)c->V * (size_t)c->K);
    for (int32_t w = 0; w < c->V; ++w)
        for (int64_t p = c->row_off[w]; p < c->row_off[w + 1]; ++p)
            out[(size_t)w * c->K + c->row_topic[p]] = c->row_count[p];
    return LDAREF_OK;
}

int ldaref_word_counts_from_dense(ldaref_ctx *c, const int32_t *in)
{
    if (!c || !in) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    int64_t nnz = 0;
    for (size_t q = 0; q < (size_t)c->V * (size_t)c->K; ++q) {
        if (in[q] < 0) return LDAREF_ERANGE;
        nnz += in[q] > 0;
    }
    if (nnz > c->row_cap) {
        size_t n = (size_t)nnz;
        int32_t *a = (int32_t *)realloc(c->row_topic, sizeof(int32_t) * n);
        if (a) c->row_topic = a;
        int32_t *b = (int32_t *)realloc(c->row_count, sizeof(int32_t) * n);
        if (b) c->row_count = b;
        uint32_t *t = (uint32_t *)realloc(c->sp_thr32, sizeof(uint32_t) * n);
        if (t) c->sp_thr32 = t;
        int32_t *l = (int32_t *)realloc(c->sp_alias, sizeof(int32_t) * n);
        if (l) c->sp_alias = l;
        if (!a || !b || !t || !l) return LDAREF_ENOMEM;
        c->row_cap = nnz;
    }
    memset(c->nk, 0, sizeof(int64_t) * (size_t)c->K);
    nnz = 0;
    for (int32_t w = 0; w < c->V; ++w) {
        c->row_off[w] = nnz;
        for (int32_t k = 0; k < c->K; ++k) {
            int32_t n = in[(size_t)w * c->K + k];
            if (n > 0) {
                c->row_topic[nnz] = k;
                c->row_count[nnz] = n;
                c->nk[k] += n;          /* n_k = sum_w n_kw (Section 3) */
                ++nnz;
            }
        }
    }
    c->row_off[c->V] = nnz;
    c->tables_valid = 0;
    return LDAREF_OK;
}

/* Compensated sum (Neumaier's form of Kahan summation): `sum` plus the rounding errors collected in `err`. */
typedef struct { double sum, err; } ksum;
static void ksum_add(ksum *a, double x)
{
    double t = a->sum + x;
    if (fabs(a->sum) >= fabs(x)) a->err += (a->sum - t) + x;
    else a->err += (x - t) + a->sum;
    a->sum = t;
}
static double ksum_value(const ksum *a) { return a->sum + a->err; }

int ldaref_loglik(ldaref_ctx *c, double *total, double *word_ll, double *doc_ll)
{
    if (!c) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    /* Each of the formula's sums is taken with compensated (Kahan-Neumaier) addition and the groups
     * are combined at the end.  Plain one-by-one addition is not good enough here: K*lgamma(V*beta)
     * and sum_k lgamma(n_k + V*beta) are ~1e10 each at V = 1e6, K = 1e5 and nearly cancel, and the
     * millions of equal terms lgamma(1 + prior) - lgamma(prior) round the same way every time, so
     * the error grows with their number (measured: 0.3 absolute on -2.4e8). */
    double lg_beta = lgamma(c->beta), lg_alpha = lgamma(c->alpha);
    ksum w_nonzero = {0.0, 0.0}, w_topics = {0.0, 0.0}, d_nonzero = {0.0, 0.0}, d_lengths = {0.0, 0.0};
    for (int64_t p = 0; p < c->row_off[c->V]; ++p)
        ksum_add(&w_nonzero, lgamma((double)c->row_count[p] + c->beta) - lg_beta);
    for (int32_t k = 0; k < c->K; ++k) ksum_add(&w_topics, lgamma((double)c->nk[k] + c->Vbeta));
    double lw = ((double)c->K * lgamma(c->Vbeta) - ksum_value(&w_topics)) + ksum_value(&w_nonzero);
    int32_t *tally = (int32_t *)calloc((size_t)c->K, sizeof(int32_t));
    if (!tally) return LDAREF_ENOMEM;
    for (int64_t d = 0; d < c->D; ++d) {
        int64_t lo = c->doc_off[d], hi = c->doc_off[d + 1];
        for (int64_t j = lo; j < hi; ++j) tally[c->z[j]] += 1;
        for (int64_t j = lo; j < hi; ++j) {
            int32_t n = tally[c->z[j]];
            if (n) { ksum_add(&d_nonzero, lgamma((double)n + c->alpha) - lg_alpha); tally[c->z[j]] = 0; }
        }
        ksum_add(&d_lengths, lgamma((double)(hi - lo) + c->Kalpha));
    }
    free(tally);
    double ld = ((double)c->D * lgamma(c->Kalpha) - ksum_value(&d_lengths)) + ksum_value(&d_nonzero);
    if (word_ll) *word_ll = lw;
    if (doc_ll) *doc_ll = ld;
    if (total) *total = lw + ld;
    return LDAREF_OK;
}

/* Counts as CSR (topics ascending inside a row).  NULL buffers: only nnz. */
int ldaref_get_counts(ldaref_ctx *c, int which, int64_t *row_offsets, int32_t *topics,
                      int32_t *counts, int64_t capacity, int64_t *nnz_out)
{
    if (!c) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if (which == LDAREF_NK) {
        if (nnz_out) *nnz_out = c->K;
        if (counts) {
            if (capacity < c->K) return LDAREF_ERANGE;
            for (int32_t k = 0; k < c->K; ++k) counts[k] = (int32_t)c->nk[k];
        }
        return LDAREF_OK;
    }
    if (which == LDAREF_NWK) {
        int64_t nnz = c->row_off[c->V];
        if (nnz_out) *nnz_out = nnz;
        if (!topics && !counts && !row_offsets) return LDAREF_OK;
        if (capacity < nnz) return LDAREF_ERANGE;
        if (row_offsets) memcpy(row_offsets, c->row_off, sizeof(int64_t) * ((size_t)c->V + 1));
        if (topics) memcpy(topics, c->row_topic, sizeof(int32_t) * (size_t)nnz);
        if (counts) memcpy(counts, c->row_count, sizeof(int32_t) * (size_t)nnz);
        return LDAREF_OK;
    }
    if (which == LDAREF_NDK) {
        int32_t *tally = (int32_t *)calloc((size_t)c->K, sizeof(int32_t));
        int32_t *seen = (int32_t *)malloc(sizeof(int32_t) * (size_t)c->K);
        if (!tally || !seen) { free(tally); free(seen); return LDAREF_ENOMEM; }
        int64_t nnz = 0;
        int fill = (topics || counts || row_offsets);
        int rc = LDAREF_OK;
        for (int64_t d = 0; d < c->D && rc == LDAREF_OK; ++d) {
            if (row_offsets) row_offsets[d] = nnz;
            int32_t n_seen = 0;
            for (int64_t j = c->doc_off[d]; j < c->doc_off[d + 1]; ++j)
                if (tally[c->z[j]]++ == 0) seen[n_seen++] = c->z[j];
            qsort(seen, (size_t)n_seen, sizeof(int32_t), cmp_i32);
            for (int32_t j = 0; j < n_seen; ++j) {
                if (fill) {
                    if (nnz >= capacity) rc = LDAREF_ERANGE;
                    else {
                        if (topics) topics[nnz] = seen[j];
                        if (counts) counts[nnz] = tally[seen[j]];
                    }
                }
                tally[seen[j]] = 0;
                ++nnz;
            }
        }
        if (row_offsets && rc == LDAREF_OK) row_offsets[c->D] = nnz;
        free(tally); free(seen);
        if (nnz_out) *nnz_out = nnz;
        return rc;
    }
    return LDAREF_EINVAL;
}

int ldaref_get_assignments(ldaref_ctx *c, int32_t *z_out)
{
    if (!c || (c->N > 0 && !z_out)) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if (c->N > 0) memcpy(z_out, c->z, sizeof(int32_t) * (size_t)c->N);
    return LDAREF_OK;
}

/* Proposal tables as built from the current counts, for table-by-table
 * comparison: per-word sparse tables indexed like the NWK rows, the shared
 * dense table, the per-word mixture thresholds and the dense mass. */
int ldaref_get_tables(ldaref_ctx *c, uint32_t *sp_thr32, int32_t *sp_alias, int64_t capacity,
                      uint32_t *mix32, uint32_t *dn_thr32, int32_t *dn_alias, uint64_t *dense_mass)
{
    if (!c) return LDAREF_EINVAL;
    if (!c->inited) return LDAREF_ESTATE;
    if (!c->tables_valid) { int rc = ldaref_build_tables(c); if (rc) return rc; }
    int64_t nnz = c->row_off[c->V];
    if ((sp_thr32 || sp_alias) && capacity < nnz) return LDAREF_ERANGE;
    if (sp_thr32) memcpy(sp_thr32, c->sp_thr32, sizeof(uint32_t) * (size_t)nnz);
    if (sp_alias) memcpy(sp_alias, c->sp_alias, sizeof(int32_t) * (size_t)nnz);
    if (mix32) memcpy(mix32, c->mix32, sizeof(uint32_t) * (size_t)c->V);
    if (dn_thr32) memcpy(dn_thr32, c->dn_thr32, sizeof(uint32_t) * (size_t)c->K);
    if (dn_alias) memcpy(dn_alias, c->dn_alias, sizeof(int32_t) * (size_t)c->K);
    if (dense_mass) *dense_mass = c->dense_mass;
    return LDAREF_OK;
}

uint32_t ldaref_sweeps_done(const ldaref_ctx *c) { return c ? c->sweep : 0; }

/* Steps of the last ldaref_sweep / ldaref_sweep_threads call that moved a chain (the proposed topic
 * differed from the current one and passed the test of Eq. 7 / Eq. 10): [0] word-, [1] doc-proposals. */
int ldaref_get_moves(const ldaref_ctx *c, int64_t *out2)
{
    if (!c || !out2) return LDAREF_EINVAL;
    out2[0] = c->moves[0];
    out2[1] = c->moves[1];
    return LDAREF_OK;
}
