// Internal declarations shared by the library's translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/lda_b200.h"

namespace lda {

// The proposal schedule of a chain (Section 4.3): whether step m draws the doc-proposal, and the
// running index of step m among the steps of its own kind.
template <int MODE>
__host__ __device__ constexpr bool step_is_doc(int m)
{
    return MODE == LDA_PROPOSALS_CYCLE ? (m & 1) != 0 : MODE == LDA_PROPOSALS_DOC;
}
template <int MODE>
__host__ __device__ constexpr int step_kind_index(int m)
{
    return MODE == LDA_PROPOSALS_CYCLE ? m >> 1 : m;
}

// Words of the record the document side leaves per token for a chain of m steps: the token's own
// (topic, n_kd) word, one (topic, n_kd) word per step, one acceptance uniform per doc step.
template <int MODE>
__host__ __device__ constexpr int step_record_words(int m)
{
    return 1 + m + (MODE == LDA_PROPOSALS_CYCLE ? m / 2 : MODE == LDA_PROPOSALS_DOC ? m : 0);
}

// Device error word bits (set by kernels, read by the host after a sweep).
enum : int {
    ERR_WORD_RANGE = 1,   // a word id outside [0,V) at load
    ERR_COUNT_ZERO = 2,   // a token's own topic has a zero count (tables inconsistent)
    ERR_ROW_OVERFLOW = 4, // a count row needed more entries than its capacity
    ERR_TOPIC_RANGE = 8,  // an assignment outside [0,K)
    ERR_ALIAS = 16,       // alias construction met an impossible state
    ERR_STAGE = 32,       // a bulk copy into shared memory did not complete within its wait limit
};

constexpr uint32_t DK_EMPTY = 0xFFFFFFFFu;  // == DK_EMPTY_SLOT of the device helpers
constexpr int DK_SLOTS_PER_TOKEN_HOST = 4;   // == DK_SLOTS_PER_TOKEN of the device helpers
constexpr int SORT_TILE = 2048;      // tokens per segmented-sort tile (one CTA)
// Tiles of whole documents (one CTA each) of the document-side kernels: tokens per tile and
// threads per CTA, chosen per corpus from these shapes; longer documents get a CTA of their own.
constexpr int DOC_TILE_SHAPES = 4;
#ifndef LDA_DOC_TILE_ROUNDS
#define LDA_DOC_TILE_ROUNDS 3
#endif
constexpr int DOC_TILE_ROUNDS = LDA_DOC_TILE_ROUNDS;  // tokens per thread: every shape holds this many times its thread count
constexpr int DOC_TILE_THREADS[DOC_TILE_SHAPES] = {128, 256, 512, 1024};
constexpr int DOC_TILE_TOKENS[DOC_TILE_SHAPES] = {DOC_TILE_ROUNDS * 128, DOC_TILE_ROUNDS * 256, DOC_TILE_ROUNDS * 512,
                                                  DOC_TILE_ROUNDS * 1024};
constexpr int DOC_TILE_MAX = DOC_TILE_ROUNDS * 1024;
// shared memory per token of a tile: 4 table slots, document offset, topic/slot (4 bytes each)
#ifndef LDA_DOC_TILE_SLOTS
#define LDA_DOC_TILE_SLOTS 4
#endif
constexpr int DOC_TILE_SLOTS = LDA_DOC_TILE_SLOTS;  // slots per token of a tile's tables in shared memory
static_assert(DOC_TILE_SLOTS % 4 == 0, "a tile's tables are cleared 16 bytes at a time");
constexpr int DOC_TILE_SMEM_PER_TOKEN = 4 * DOC_TILE_SLOTS + 4 + 4;
// partial sums of the log-likelihood kernels: word part; document part (tiles + long documents)
constexpr int LL_WORD_PARTIALS = 592;
constexpr int LL_DOC_PARTIALS = 148 * 16 + 592 + 1024;
constexpr int HIST_BINS = 32768;     // shared-memory histogram window (32-bit bins)
constexpr int WORD_ROWS_BITMAP_MAX_K = 16384;  // tail rows: topic bitmap up to this K, key sort above
constexpr int HIST16_BINS = 106496;  // window of a warm word's n_kw histogram (16-bit bins, 208 KB)
constexpr int HIST32_BINS = 49152;   // window of a hot word's n_kw histogram (32-bit bins, 192 KB)
#ifndef LDA_HIST_CHUNK
#define LDA_HIST_CHUNK 262144
#endif
constexpr int HIST_CHUNK = LDA_HIST_CHUNK;    // tokens per CTA (one run of a word) in the histogram path
#ifndef LDA_HOT_TILE
#define LDA_HOT_TILE 32768
#endif
#ifndef LDA_HOT_TILE_PROPOSE
#define LDA_HOT_TILE_PROPOSE 8192
#endif
constexpr int HOT_TILE = LDA_HOT_TILE;  // accept pass: tokens of one hot word per CTA (the word's row is staged once per CTA)
constexpr int HOT_TILE_PROPOSE = LDA_HOT_TILE_PROPOSE;  // propose pass: nothing is staged, shorter runs balance better
constexpr int COLD_TILE = 2048;      // MH kernel: tokens of a tile of whole tail words
constexpr int COLD_WORDS = 512;      // MH kernel: words per tail tile
constexpr int HOT_STAGE_MAX_K = 16384;  // dense rows up to this many topics are staged in shared memory
// Beyond that K a dense row (4 K bytes) only pays for frequent words.  Words with more tokens than
// a tail tile holds but at most WARM_MAX_TF keep a sorted sparse row only ("warm" words): rebuilt by
// one CTA per word from a 16-bit histogram over the topics, and staged whole in shared memory by
// the accept pass (a row has at most as many entries as the word has tokens).
constexpr int WARM_MAX_TF = 12288;
#ifndef LDA_ALIAS_WARP_MAX
#define LDA_ALIAS_WARP_MAX 512
#endif
constexpr int ALIAS_WARP_MAX = LDA_ALIAS_WARP_MAX;  // rows up to this many items are built by one warp
constexpr int ALIAS_WARP_SMEM = 8 * ALIAS_WARP_MAX * 12;  // eight warps per CTA, 12 bytes of scratch per item
constexpr int ALIAS_SCRATCH_PER_ITEM = 20;   // bytes of construction scratch per item
#ifndef LDA_ALIAS_SMEM_ITEMS_MID
#define LDA_ALIAS_SMEM_ITEMS_MID 2048
#endif
constexpr int ALIAS_SMEM_ITEMS_MID = LDA_ALIAS_SMEM_ITEMS_MID;   // rows a 256-thread CTA builds entirely in shared memory
constexpr int ALIAS_SMEM_ITEMS_BIG = 4096;   // ... and a 512-thread CTA

// Everything a kernel needs, passed by value.
struct View {
    int32_t V, K, N, D;
    double alpha, beta, Vbeta, Kalpha;
    uint32_t tok_base;  // Philox token key of the corpus' first token (0 unless the corpus is a shard)
    int topic_bits;  // bits of K-1
    int count_bits;  // low bits of a packed n_kd entry that hold the count
    // tokens in word-sorted order (position p)
    const uint32_t* tok_orig;  // index of the token in the caller's document order
    // block-major order (index m): the tokens sorted by (block of the document-order index,
    // word-sorted position).  Buffers in this order are reached from word order in runs of
    // consecutive positions and from document order within one L2-sized block at a time.
    const uint32_t* inv;        // [N] block-major index of the token at word-sorted position p
    const uint32_t* bm_of_tok;  // [N] block-major index of the token with document-order index i
    // per-sweep exchange buffers between the word-order and the document-order passes
    void* prop;        // [word steps][N] block-major: topics proposed by the word-proposals after the first
    uint32_t* ua_w;    // [word steps][N] word order: acceptance uniforms of the word-proposal steps
    uint32_t* dside;   // [N][side_stride] block-major: own record, per step (topic << count_bits) | n_kd,
                       // per doc step its acceptance uniform
    int32_t side_stride;  // words per token in dside, a multiple of 4
    // assignments (topic type: u16 or i32) after the last MH step or initialisation
    void* zw;   // word-sorted order: read by the n_kw / n_k rebuild
    void* zbm;  // block-major order, two entries per token: its topic, read (through bm_of_tok) by everything
                // that works per document, and beside it the first word-proposal of the running MH step
    // One word per token in document order: scratch (slot indices of long documents during the MH
    // step, staging of assignments on their way in and out, z in document order for export.cu).
    uint32_t* rec;
    const int32_t* word_off;  // [V+1] token range of each word in word-sorted order
    const int32_t* doc_off;   // [D+1]
    // n_kw: every word has a sorted (topic, count) row of fixed capacity; hot words also a dense row
    const int32_t* row_start;  // [V+1] first slot of each word's row
    int32_t* wk_nnz;           // [V]
    uint32_t* wk_topic;        // [row_start[V]]
    uint32_t* wk_count;
    const int32_t* dense_slot;  // [V] index of the word's dense row or -1
    int32_t* dense_rows;        // [n_dense * dense_stride]
    int32_t dense_stride;       // K rounded up to a multiple of 4 (rows start 16-byte aligned)
    // word-proposal tables
    uint32_t* al_thr;  // split point of each sparse bin as a 32-bit fraction
    uint32_t* al_idx;  // alias item of each sparse bin
    uint2* al_pk;      // 16-bit topics only: bin as (split point, topic of the bin's item | topic of
                       // its alias item << 16), so a draw costs one read
    uint32_t* mix32;   // [V] share of the sparse term
    uint32_t* dn_thr;  // [K]
    uint32_t* dn_idx;  // [K]
    uint2* dn_pk;      // [K] (split point, alias) of the dense table in one word pair
    unsigned long long* dense_mass;
    int32_t* nk;  // [K]
    // n_kd of the documents longer than a tile (the others' tables only ever live in shared memory):
    // the i-th long document owns the open-addressing table dk_slots[long_slot_off[i] .. long_slot_off[i+1])
    // (four slots per token, load <= 0.25); layout and probe order: dk_insert in lda_device.cuh.
    uint32_t* dk_slots;
    const long long* long_slot_off;
    int* err;
    unsigned long long* moves;  // [2] steps of the running lda_sweep() that moved a chain: word-, doc-proposals
};

struct Ctx {
    int32_t V = 0, K = 0;
    double alpha = 0, beta = 0;
    int device = 0;
    int n_sm = 148;  // multiprocessors of the device
    cudaStream_t stream = nullptr;
    bool wide_topics = false;  // false: 16-bit topic storage, true: 32-bit
    int block_shift = 22;  // log2 of the tokens per block of the block-major order
    int doc_tile = DOC_TILE_TOKENS[0], doc_threads = DOC_TILE_THREADS[0];  // shape of the document tiles
    int side_steps = 0;    // number of steps the exchange buffers are allocated for
    int side_mode = 0;     // ... and the proposal schedule they are laid out for
    int proposals = 0;     // LDA_PROPOSALS_*: which proposal each step of a chain draws
    int64_t shard_first_token = 0;        // lda_set_shard(): global index of this corpus' first token
    std::vector<int32_t> shard_global_tf;  // ... and the term frequencies over all shards (empty: this corpus alone)
    double dense_frac = 0.05;
    double dense_min_tf = 64;
    int alias_slices = 1;  // vocabulary slices whose word-proposal tables are alive one at a time
    bool loaded = false, inited = false, tables_valid = false;
    int64_t n_nonempty_docs = 0;
    uint64_t seed = 0;
    uint32_t sweep = 0;
    int64_t N = 0, D = 0;
    View v{};
    // host-side work lists (device copies below)
    int32_t n_word_tiles = 0, n_doc_tiles = 0, n_dense = 0, n_hist_chunks = 0, n_long_docs = 0,
            n_alias_big = 0, n_alias_mid = 0, n_hot_tiles = 0, n_hot_tiles_propose = 0, n_cold_tiles = 0;
    int32_t* word_tiles = nullptr;   // [n_word_tiles*2] word ranges sorted per CTA
    int32_t* doc_tiles = nullptr;    // [n_doc_tiles*2]
    int32_t* dense_words = nullptr;  // [n_dense]
    int32_t* hist_chunks = nullptr;  // [n_hist_chunks*4] (word, first token, count, 1 if the word's only run)
    int32_t* long_docs = nullptr;    // [n_long_docs]
    // sorted n_kd rows (export.cu): tiles of whole documents of at most SORT_TILE tokens, and the longer documents
    int32_t n_doc_sort_tiles = 0, n_doc_sort_long = 0;
    int32_t* doc_sort_tiles = nullptr;
    int32_t* doc_sort_long = nullptr;
    int32_t* alias_big = nullptr;    // [n_alias_big] words whose row can exceed ALIAS_WARP_MAX; the first
                                     // n_alias_mid of them cannot exceed ALIAS_SMEM_ITEMS_MID
    int32_t n_warm = 0, n_hot_tiles_warm = 0;
    int32_t* warm_words = nullptr;      // [n_warm] words with a sorted row and more tokens than a tail tile holds
    int32_t* hot_tiles_warm = nullptr;  // [n_hot_tiles_warm*3] their runs for the accept pass
    int32_t* hot_tiles = nullptr;    // [n_hot_tiles*3] (word, first token, count): MH kernel, words with a dense row (accept pass)
    int32_t* hot_tiles_propose = nullptr;  // the same cut into the shorter runs of the propose passs
    int32_t* cold_tiles = nullptr;   // [n_cold_tiles*2] word ranges of whole tail words: MH kernel
    // Vocabulary slices (Section 3, Fig. 1: the model is visited slice by slice): the words are cut into
    // runs of about equal row capacity; the sparse alias tables and their construction scratch hold one
    // slice at a time (entry of row slot r of the running slice: r - row_lo), so pass 1 goes slice by
    // slice: build the slice's tables, draw the word-proposals of its tokens.  One slice = everything.
    struct Slice {
        int32_t w_lo = 0, w_hi = 0;        // words [w_lo, w_hi)
        int64_t row_lo = 0, row_n = 0;     // their row slots [row_lo, row_lo + row_n)
        int32_t mid_lo = 0, mid_n = 0;     // their part of alias_big[0 .. n_alias_mid)
        int32_t big_lo = 0, big_n = 0;     // ... of alias_big[n_alias_mid .. n_alias_big), relative to n_alias_mid
        int32_t hotp_lo = 0, hotp_n = 0;   // ... of hot_tiles_propose
        int32_t cold_lo = 0, cold_n = 0;   // ... of cold_tiles
    };
    std::vector<Slice> slices;
    int cur_slice = 0;
    uint32_t* al_thr0 = nullptr;  // the slice-sized buffers View::al_thr, al_idx, al_pk and sc_w, sc_de, sc_item
    uint32_t* al_idx0 = nullptr;  // point into, shifted by the running slice's row_lo
    uint2* al_pk0 = nullptr;
    unsigned long long* sc_w0 = nullptr;
    unsigned long long* sc_de0 = nullptr;
    uint32_t* sc_item0 = nullptr;
    // alias-construction scratch
    unsigned long long* sc_w = nullptr;   // [row capacity total] scaled masses
    unsigned long long* sc_de = nullptr;  // deficits prefix (front) / surpluses prefix (back)
    uint32_t* sc_item = nullptr;          // light items (front) / heavy items (back)
    unsigned long long* sc_dense = nullptr;  // same three for the dense table, [3*K]
    double* ll_tab = nullptr;        // [2 * 512] lgamma tables of the log-likelihood's document part
    double* ll_tile_part = nullptr;  // [n_doc_tiles] its partial sums, one per tile of documents
    uint32_t* ll_tile_nnz = nullptr; // [n_doc_tiles] filled table slots of the tile: its share of nnz(n_kd)
    bool ll_tables_ready = false;
    double* red = nullptr;                   // reduction partials for the log-likelihood
    int64_t* red_i = nullptr;
    // device memory comes from cudaMalloc / cudaFree unless lda_set_allocator() gave other routines
    lda_alloc_fn alloc_fn = nullptr;
    lda_free_fn free_fn = nullptr;
    void* alloc_user = nullptr;
    std::vector<void*> allocs;
    std::vector<size_t> alloc_bytes;  // size of every entry of `allocs`
    std::vector<char> alloc_own;      // 1: the entry came from the caller's allocator, 0: from cudaMalloc
    int64_t device_bytes = 0;
    lda_stats stats{};
    int64_t launches = 0;
    // Events of up to EV_RING iterations of a sweep call (per iteration: 0..6 bracket the phases, 8 and
    // 9 the passes of the MH step); the host waits and reads them once per EV_RING iterations.
    static constexpr int EV_RING = 8;
    cudaEvent_t ev_ring[EV_RING][10] = {};
    cudaEvent_t* ev = ev_ring[0];  // the running iteration's
    bool have_events = false;
    // Two more streams for kernels of one phase that touch different words: fork_streams() makes them
    // wait for the work queued on `stream` so far, join_streams() makes `stream` wait for theirs.
    cudaStream_t side[2] = {};
    cudaEvent_t ev_fork = nullptr, ev_join[2] = {};
    bool have_side = false;
    // Assignments travel between host and device in chunks on a stream of their own, so that the copy
    // of one chunk runs beside the kernel that spreads (or collects) its neighbour.  ev_chunk orders a
    // chunk's two halves; ev_export completes when the last chunk of an export has reached the host:
    // whatever touches the staging buffer next waits for it on the device (order_after_export()).
    int64_t copy_chunk = 1 << 25;  // tokens per chunk (option "copy_chunk_log2")
    cudaStream_t copy = nullptr;
    cudaEvent_t ev_chunk = nullptr, ev_export = nullptr;
    bool export_pending = false;
    std::string err;
};

inline void fork_streams(Ctx& c)
{
    cudaEventRecord(c.ev_fork, c.stream);
    for (int i = 0; i < 2; ++i) cudaStreamWaitEvent(c.side[i], c.ev_fork, 0);
}

inline void join_streams(Ctx& c)
{
    for (int i = 0; i < 2; ++i) {
        cudaEventRecord(c.ev_join[i], c.side[i]);
        cudaStreamWaitEvent(c.stream, c.ev_join[i], 0);
    }
}

// --- launchers (each returns the number of kernels it launched) -----------------
int launch_init(Ctx& c);
int launch_spread_assignments(Ctx& c, const void* z_dev, bool narrow);  // z (doc order; u16 if narrow, else i32) -> both layouts
int launch_spread_chunk(Ctx& c, const void* z_dev, bool narrow, int64_t first, int64_t count);  // ... tokens [first, first+count) -> block-major
int launch_word_order_topics(Ctx& c);                                  // block-major -> word order, all tokens
int launch_export_assignments(Ctx& c, void* z_dev, bool narrow);
int launch_export_chunk(Ctx& c, void* z_dev, bool narrow, int64_t first, int64_t count);
int launch_count_wk(Ctx& c);
int launch_count_k(Ctx& c);
int launch_alias_dense(Ctx& c);
int launch_alias_sparse(Ctx& c);            // the running slice's tables
void set_slice(Ctx& c, int slice);          // makes `slice` the running one (moves the table pointers)
int launch_sample(Ctx& c, int mh_steps);   // all passes of the MH step; needs ensure_exchange()
int launch_doc_side(Ctx& c, int mh_steps);  // pass 2 of the MH step
size_t doc_tile_smem_bytes(int tile_tokens);  // dynamic shared memory of the document-tile kernels
int ensure_exchange(Ctx& c, int mh_steps);  // (re)allocates View::prop / View::dside; LDA_* status
int launch_loglik(Ctx& c, double* out3_host);
int launch_count_nnz(Ctx& c, int64_t* nnz_wk_host, int64_t* nnz_dk_host);

// n_kd as sorted rows in device memory (export.cu): row_off[D+1], and unless sizes_only the entries.
// The caller releases the arrays with free_dk_csr().
struct DkCsr {
    long long* row_off = nullptr;
    int32_t* nnz = nullptr;
    int32_t* topic = nullptr;
    int32_t* count = nullptr;
    long long total = 0;
};
int build_dk_csr(Ctx& c, DkCsr& r, bool sizes_only);  // LDA_* status; queued on c.stream, rows complete after a sync
void free_dk_csr(Ctx& c, DkCsr& r);

// n_kw as a dense V x K matrix in device memory and back (shard.cu): the exchange format of the
// document-sharded mode.  Return the number of kernels launched.
int launch_word_counts_to_dense(Ctx& c, int32_t* nwk_dev);
int launch_word_counts_from_dense(Ctx& c, const int32_t* nwk_dev);

// Exact-conditional yardstick (gibbs.cu): `iters` frozen sweeps drawing from Eq. 1.  LDA_* status.
constexpr int GIBBS_MAX_K = 16384;              // a word's dense n_kw row is staged in shared memory
constexpr long long GIBBS_MAX_PREFIX_BYTES = 24ll << 30;  // V * K running sums of 8 bytes
int gibbs_sweep(Ctx& c, int32_t iters);
void set_gibbs_smem_limits();

// load-time layout (sort + offsets); fills c.v token arrays. Returns LDA_* status.
int build_layout(Ctx& c, const int32_t* word_ids_dev, const int64_t* doc_off_host);

void* raw_alloc(Ctx& c, size_t bytes);  // the context's allocator (cudaMalloc by default); nullptr on failure
void raw_free(Ctx& c, void* p);
template <typename P>
inline bool tmp_alloc(Ctx& c, P** p, size_t bytes)  // transient buffer, released with raw_free()
{
    *p = static_cast<P*>(raw_alloc(c, bytes ? bytes : 1));
    return *p != nullptr;
}
void* dev_alloc(Ctx& c, size_t bytes);  // tracked allocation held by the context; nullptr on failure
void dev_free(Ctx& c, void* p);         // releases one tracked allocation (nullptr: nothing)
void dev_free_all(Ctx& c);

}  // namespace lda
