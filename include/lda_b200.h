/*
 * lda_b200.h -- C ABI of the B200 (sm_100a) LightLDA sweep library.
 *
 * The library runs the data-parallel hot path of the LightLDA sampler on one
 * GPU: per sweep it rebuilds the word-proposal alias tables from the counts
 * frozen at sweep start, runs `mh_steps` Metropolis-Hastings proposals per
 * token (word-proposal on even steps, doc-proposal on odd steps) and rebuilds
 * the count tables n_kw, n_k, n_kd from the new assignments.
 *
 * Conventions
 *   - every function returns an int status: LDA_OK or a negative LDA_E* code;
 *     nothing throws, exits or prints.  lda_last_error() gives a message.
 *   - pointers are HOST pointers unless the parameter says DEVICE.
 *   - the caller owns every buffer it passes; inputs are copied, so they may
 *     be freed once the call returns.  The context owns all device memory it
 *     allocates and frees it in lda_destroy().
 *   - a context is bound to the CUDA device that is current in lda_create()
 *     and to one stream (the legacy default stream unless lda_set_stream() is
 *     called).  One host thread per context.
 *   - all calls are synchronous: results are complete when they return.
 *   - limits: n_tokens < 2^31, K <= 131072; bitlen(K-1) + bitlen(longest
 *     document + 1) <= 32 (n_kd entries are stored as one packed 32-bit word).
 *
 * There is no CPU fallback: every entry point that computes needs the GPU.
 */
#ifndef LDA_B200_H
#define LDA_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LDA_OK 0
#define LDA_EINVAL (-1)    /* NULL pointer, V/K <= 0, alpha/beta not finite and > 0, iters < 0, mh_steps outside 1..1024 */
#define LDA_ERANGE (-2)    /* word id outside [0,V), bad offsets, sizes beyond the limits, capacity too small */
#define LDA_ESTATE (-3)    /* call order: load before init, init before sweep */
#define LDA_ENOMEM (-4)    /* host or device allocation failed */
#define LDA_ECUDA (-5)     /* a CUDA call or launch failed */
#define LDA_EINTERNAL (-6) /* a kernel raised the device error word (inconsistent tables) */

#define LDA_NK 0
#define LDA_NWK 1
#define LDA_NDK 2

typedef struct lda_ctx lda_ctx; /* opaque, owned by the library */

/* Timings and counters of the most recent lda_sweep() call (all its iterations summed). */
typedef struct lda_stats {
    int64_t n_tokens, n_docs;
    int64_t nnz_wk, nnz_dk;   /* nonzeros of n_kw and n_kd after the last rebuild */
    int64_t n_dense_words;    /* words whose n_kw row is kept dense */
    int64_t device_bytes;     /* device memory held by the context */
    int64_t kernel_launches;  /* kernels launched by the last lda_sweep() */
    int32_t sweeps_done;      /* sweeps since lda_init()/lda_set_assignments() */
    int32_t iters;            /* iterations of the last lda_sweep() */
    float ms_alias_dense;     /* dense smoothing table            (Section 4.2) */
    float ms_alias_sparse;    /* per-word sparse alias tables     (Section 4.2) */
    float ms_sample;          /* token MH step, all passes        (Eq. 6-13)    */
    float ms_count_wk;        /* n_kw rebuild                     (Section 3)   */
    float ms_count_k;         /* n_k rebuild                                    */
    float ms_count_dk;        /* always 0: n_kd is rebuilt inside the MH step's document pass (Eq. 12), tile by
                                 tile in shared memory; its time is part of ms_doc_side */
    float ms_total;           /* first launch to last kernel end                */
    float ms_propose;         /* MH step, pass 1: word-proposals   (part of ms_sample) */
    float ms_doc_side;        /* MH step, pass 2: document side    (part of ms_sample) */
    float ms_accept;          /* MH step, pass 3: accept / reject  (part of ms_sample) */
    /* Proposals of the last lda_sweep() by kind (Section 4.2: Eq. 7 / Eq. 10 acceptance): how many
     * steps drew the word-proposal / the doc-proposal (every token takes every step), and how many of
     * them moved the chain (proposed topic differs from the current one and was accepted). */
    int64_t word_proposed, word_accepted;
    int64_t doc_proposed, doc_accepted;
} lda_stats;

/* Model dimensions and symmetric priors of the collapsed LDA model (Section 3,
 * Eq. 1: alpha_k = alpha, beta_w = beta, beta-bar = V*beta). */
int lda_create(int32_t V, int32_t K, double alpha, double beta, lda_ctx** out);

/* Run all later work of this context on `cuda_stream` (a cudaStream_t); NULL = default stream. */
int lda_set_stream(lda_ctx* ctx, void* cuda_stream);

/* Where the context's device memory comes from.  By default cudaMalloc / cudaFree; a caller that runs
 * inside a framework with a memory pool of its own (PyTorch's caching allocator, say) hands the
 * pool's routines in, and every later allocation of the context -- the corpus layout, the count and
 * alias tables, the exchange buffers, transient buffers of lda_load_corpus / lda_get_counts /
 * lda_gibbs_sweep -- goes through them.  alloc_fn returns DEVICE memory of at least `bytes` bytes,
 * 256-byte aligned, usable on the context's stream, or NULL when it has none; free_fn takes such a
 * pointer back (the library calls it only after the work that used the memory has finished on the
 * context's stream).  Both or neither (NULL, NULL = back to cudaMalloc).  Must be called before
 * lda_load_corpus (LDA_ESTATE afterwards); `user` is passed through. */
typedef void* (*lda_alloc_fn)(size_t bytes, void* user);
typedef void (*lda_free_fn)(void* ptr, void* user);
int lda_set_allocator(lda_ctx* ctx, lda_alloc_fn alloc_fn, lda_free_fn free_fn, void* user);

/* Tunables that never change results.  Must be set before lda_load_corpus().
 *   "dense_frac"   fraction of the vocabulary (by term frequency) whose n_kw rows are dense (Section 5)
 *   "dense_min_tf" words rarer than this (or than K/8) stay sparse even inside dense_frac
 *   "block_log2"   log2 of the tokens per block of documents in the block-major token order that the
 *                  document-side pass of the MH step walks (default 22: the exchange buffers
 *                  of one block, 20 bytes per token, stay in L2 while the document pass is on it)
 *   "copy_chunk_log2" log2 of the tokens per chunk in which assignments cross the host link (default 25):
 *                  a chunk is copied on the context's copy stream while its neighbour is spread into, or
 *                  collected from, the device layout.  Whole number in [10, 30]; no result depends on it.
 *   "alias_slices" number of vocabulary slices (Section 3, Figure 1: the model is visited one slice at a
 *                  time, and only that slice's alias tables are in memory; Section 6 "Pipelining").  Whole
 *                  number in [1, 256], default 1.  The words are cut into runs of about equal row
 *                  capacity; the word-proposal tables of Section 4.2 and their construction scratch
 *                  (28-36 bytes per row slot, the largest part of the model's working set) are allocated
 *                  for the largest slice only, and pass 1 of the MH step goes slice by slice: build the
 *                  slice's tables, draw the word-proposals of its tokens.  The n_kw rows themselves stay
 *                  resident (the accept pass and the rebuild need them).  No result depends on it; with
 *                  more than one slice lda_stats.ms_alias_sparse is ~0 and ms_propose covers both.         */
int lda_set_option(lda_ctx* ctx, const char* key, double value);

/* Which proposal the steps of a token's chain draw (Section 4.3; the variants compared in
 * Figure 11).  Either proposal alone is a valid MH kernel for Eq. 4; the cycle mixes best.
 *   LDA_PROPOSALS_CYCLE  step m draws the word-proposal (Eq. 6-8) when m is even and the
 *                        doc-proposal (Eq. 9-11) when m is odd (default)
 *   LDA_PROPOSALS_WORD   every step draws the word-proposal
 *   LDA_PROPOSALS_DOC    every step draws the doc-proposal
 * May be called at any time between sweeps; it changes results (not only speed) from the next
 * lda_sweep() on and keeps the Philox counter layout.  Other values: LDA_EINVAL. */
#define LDA_PROPOSALS_CYCLE 0
#define LDA_PROPOSALS_WORD 1
#define LDA_PROPOSALS_DOC 2
int lda_set_proposals(lda_ctx* ctx, int mode);

/* Storage of n_kw (Section 5): words with many tokens keep a dense row of K counters; the long tail
 * keeps sparse rows.  The paper's sparse rows are hash tables because it updates them in place;
 * here every row is rebuilt from the assignments each sweep, so a tail row is stored SORTED by
 * topic (binary search instead of probing; the same order defines the items of the word's alias
 * table).  Hashed rows in the paper's sense are what the document side uses for n_kd.  Which form a
 * word gets never changes a result.
 *
 * Corpus in document order: token i has word word_ids[i]; document d owns tokens
 * [doc_offsets[d], doc_offsets[d+1]); doc_offsets has n_docs+1 entries, [0] = 0,
 * [n_docs] = n_tokens; empty documents are legal.  Builds the word-sorted token
 * layout once (Section 6, item 3) and chooses the dense/sparse class of every
 * word (Section 5).  Both arrays are HOST memory. */
int lda_load_corpus(lda_ctx* ctx, const int32_t* word_ids, int64_t n_tokens,
                    const int64_t* doc_offsets, int64_t n_docs);

/* Same, with both arrays in DEVICE memory of the context's GPU. */
int lda_load_corpus_device(lda_ctx* ctx, const int32_t* word_ids_dev, int64_t n_tokens,
                           const int64_t* doc_offsets_dev, int64_t n_docs);

/* z_i uniform on {0..K-1} from Philox4x32-10 keyed by `seed`, counter
 * (token, 0, 0, 1); builds n_kw, n_k, n_kd (Section 3, Eq. 12); sweep counter = 0. */
int lda_init(lda_ctx* ctx, uint64_t seed);

/* Warm start (Section 6: counts are re-initialised from z).  z has n_tokens
 * entries in the caller's document order, each in [0,K). */
int lda_set_assignments(lda_ctx* ctx, const int32_t* z, uint64_t seed, uint32_t sweep);

/* The same with 16-bit topics: half the bytes over the host link.  Needs K <= 65536 (the library
 * then stores topics in 16 bits itself); LDA_ERANGE otherwise. */
int lda_set_assignments_u16(lda_ctx* ctx, const uint16_t* z, uint64_t seed, uint32_t sweep);

/* `iters` frozen-counts sweeps of `mh_steps` proposals per token (Section 4.2-4.3,
 * Eq. 6-13; Section 6 "immutable model"), the proposal of each step chosen by
 * lda_set_proposals().  Randomness: one Philox block per (token, sweep, step), counter
 * (token, sweep, step, 0). */
int lda_sweep(lda_ctx* ctx, int32_t iters, int32_t mh_steps);

/* Document-sharded data parallelism (Section 6, "Parameter Server and Data Placement": documents are
 * partitioned over the workers, the word-topic table n_kw and its column sums n_k are shared and the
 * workers' updates are aggregated after sampling).  A context may hold ONE SHARD of a corpus -- a
 * run of consecutive documents.  Its n_kd is its own; n_kw and n_k must be the sums over all shards
 * whenever a sweep starts.  The library does the local halves, the caller the sum (one all-reduce of
 * a dense int32 matrix per sweep, e.g. ncclAllReduce / torch.distributed.all_reduce):
 *
 *   lda_set_shard(ctx, first_token, global_term_freq)      before lda_load_corpus
 *   lda_load_corpus(shard's documents); lda_init(seed)      the same seed on every shard
 *   repeat:  lda_word_counts_to_dense(ctx, M)               M = this shard's n_kw, DEVICE int32 [V*K]
 *            M <- sum of M over the shards                  (the caller's collective)
 *            lda_word_counts_from_dense(ctx, M)             n_kw, n_k := the sums
 *            lda_sweep(ctx, 1, mh_steps)                    leaves the shard's own counts again
 *
 * first_token is the index of the shard's first token in the whole corpus: it offsets the Philox
 * token key, so a sharded run draws exactly the random numbers of a single context holding all the
 * documents and, the counts being frozen during a sweep, produces exactly its assignments.
 * global_term_freq (HOST, V entries, copied; NULL = this corpus is the whole) is every word's token
 * count over ALL shards: it sizes the rows and picks the dense/sparse class of a word.
 * lda_word_counts_from_dense returns LDA_ERANGE (and the context must be initialised again) if a
 * row of the matrix has more nonzeros than min(global_term_freq[w], K) or a negative entry.
 * lda_loglik() on a shard gives the word part of the counts last imported and the document part of
 * the shard's own documents: sum the document parts over the shards, take the word part once.
 * Needs V*K*4 bytes per matrix (the caller's buffer). */
int lda_set_shard(lda_ctx* ctx, int64_t first_token, const int32_t* global_term_freq);
int lda_word_counts_to_dense(lda_ctx* ctx, int32_t* nwk_dev);
int lda_word_counts_from_dense(lda_ctx* ctx, const int32_t* nwk_dev);

/* Yardstick, not a fast path: `iters` frozen sweeps in which every token draws its new topic from the
 * collapsed conditional itself (Section 3, Eq. 1) under the sweep-start counts with the token's own
 * contribution removed -- the law the MH chain of lda_sweep() converges to as mh_steps grows
 * (Section 4.1).  The conditional is split as in Section 4, Eq. 3 (a term over the document's topics
 * + a smoothing term over all topics); every term is floored to a multiple of 2^-44 and the draw is
 * the inverse CDF over these integer masses (document term first, topics ascending), so results do
 * not depend on summation order.  Randomness: Philox counter (token, sweep, 0, 2), word 0.
 * Cost per token O(K_d log K_w + log K); keeps V*K running sums of 8 bytes while it runs.
 * Limits (LDA_ERANGE): K <= 16384, V*K*8 bytes <= 24 GiB, K*alpha < 2^17, documents < 2^19 tokens.
 * Counts, sweep counter and lda_loglik() behave as after lda_sweep(); lda_stats is left alone. */
int lda_gibbs_sweep(lda_ctx* ctx, int32_t iters);

/* Collapsed joint log p(w,z): word part + document part (Section 7.2, Figure 11).
 * Any output pointer may be NULL. */
int lda_loglik(lda_ctx* ctx, double* total, double* word_ll, double* doc_ll);

/* Count tables as CSR, topics ascending inside a row.
 *   LDA_NK : counts[0..K) dense, `capacity` >= K; row_offsets/topics unused.
 *   LDA_NWK: V rows; LDA_NDK: n_docs rows.  row_offsets has rows+1 entries.
 * With topics == counts == row_offsets == NULL only *nnz_out is written. */
int lda_get_counts(lda_ctx* ctx, int which, int64_t* row_offsets, int32_t* topics,
                   int32_t* counts, int64_t capacity, int64_t* nnz_out);

/* Current assignments, n_tokens entries in the caller's document order. */
int lda_get_assignments(lda_ctx* ctx, int32_t* z_out);

/* The same as 16-bit topics; needs K <= 65536, LDA_ERANGE otherwise. */
int lda_get_assignments_u16(lda_ctx* ctx, uint16_t* z_out);

/* The two calls above without the wait at the end (the paper has no counterpart: Section 6 overlaps
 * its transfers by pipelining data blocks; here the one transfer of a sweep's result is overlapped
 * with what the caller does next).  The assignments are collected and copied to z_out (host memory;
 * pinned, or the copy is not asynchronous) chunk by chunk on a stream of the context's own; the call
 * returns once that is queued.  z_out is complete, and may be read, after lda_wait() has returned
 * LDA_OK.  Calls made in between are legal: lda_loglik(), lda_get_stats() and lda_get_tables() run
 * beside the transfer; a call that changes the state (lda_sweep, lda_set_assignments, lda_init, ...)
 * is ordered after it on the device.  z_out stays owned by the caller and must stay valid until
 * lda_wait() or lda_destroy(). */
int lda_get_assignments_async(lda_ctx* ctx, int32_t* z_out);
int lda_get_assignments_u16_async(lda_ctx* ctx, uint16_t* z_out);

/* Waits for everything the context has queued (its stream and its copy stream).  LDA_ECUDA if the
 * device reports an error. */
int lda_wait(lda_ctx* ctx);

/* Word-proposal tables built from the current counts (Section 4.2): per-word sparse
 * alias tables indexed like the LDA_NWK rows (split point as a 32-bit fraction,
 * alias as an item index inside the row), per-word mixture thresholds [V], the
 * dense table [K] and the dense term's fixed-point mass.  Any pointer may be NULL. */
int lda_get_tables(lda_ctx* ctx, uint32_t* sp_thr32, int32_t* sp_alias, int64_t capacity,
                   uint32_t* mix32, uint32_t* dn_thr32, int32_t* dn_alias, uint64_t* dense_mass);

/* Dense smoothing table without any allocation (the paper has no counterpart: this exists for
 * callers of the library, not for the method).
 *
 * Who needs it: code that may not allocate device memory when it runs -- a component living
 * inside another framework's memory pool, a latency-critical loop that cannot afford the
 * device-wide synchronisation an allocation can imply, a process whose memory was budgeted
 * at start-up.  Every other entry point here may allocate; this one calls no cudaMalloc,
 * cudaFree or allocating library routine.
 *
 * Computes exactly what lda_get_tables() reports as dn_thr32 / dn_alias / dense_mass: the alias
 * table over k of beta / (n_k[k] + V*beta).  All pointers are DEVICE memory owned by the caller:
 *   n_k_dev[K] in; dn_thr32_dev[K], dn_alias_dev[K], dense_mass_dev[1] out;
 *   status_dev[1] out, may be NULL: 0 on success, else the library's device error bits.
 * The work is queued on `cuda_stream` (a cudaStream_t, NULL = default stream) and the call
 * returns without waiting for it.
 *
 * The construction scratch is a fixed device array inside the library, sized for
 * LDA_NOALLOC_MAX_K topics (20 bytes per topic, about 2.6 MB); every GPU that loads the library
 * holds it until the process exits.  K above LDA_NOALLOC_MAX_K is refused with LDA_ERANGE.
 * The first call on each device looks up the array's device address (one runtime query, made
 * with that device current; the runtime may load the library's device code at that moment too, if
 * nothing of it ran on the device before); make that first call before starting any stream capture.
 * The looked-up address is cached per device without a lock: if two host threads may make the
 * FIRST call on a device at the same time, serialise those two calls (later calls only read it).
 * A caller that passes status_dev == NULL cannot learn of a failed construction (e.g. beta so small
 * against n_k that every fixed-point weight is zero): the call still returns LDA_OK and the
 * outputs stay unwritten.  Pass a status word wherever the inputs are not known to be sane.
 * All calls share the one array and it keeps the previous call's contents; nothing in it needs
 * clearing because each call overwrites what it later reads, and the status word is zeroed on
 * the stream before the kernel.  Two calls that overlap on the GPU (different streams, or
 * different host threads) race on the array and give undefined tables: serialise them. */
#define LDA_NOALLOC_MAX_K 131072
int lda_dense_table_noalloc(const int32_t* n_k_dev, int32_t K, int32_t V, double beta,
                            uint32_t* dn_thr32_dev, int32_t* dn_alias_dev, uint64_t* dense_mass_dev,
                            int32_t* status_dev, void* cuda_stream);

int lda_get_stats(lda_ctx* ctx, lda_stats* out);

/* Message of the last failure on this context (library-owned, valid until the next call). */
const char* lda_last_error(const lda_ctx* ctx);

void lda_destroy(lda_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* LDA_B200_H */
