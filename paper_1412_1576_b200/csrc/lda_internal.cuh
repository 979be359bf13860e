// Internal declarations shared by the library's translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/lda_b200.h"

namespace lda {

// Device error word bits (set by kernels, read by the host after a sweep).
enum : int {
    ERR_WORD_RANGE = 1,   // a word id outside [0,V) at load
    ERR_COUNT_ZERO = 2,   // a token's own topic has a zero count (tables inconsistent)
    ERR_ROW_OVERFLOW = 4, // a count row needed more entries than its capacity
    ERR_TOPIC_RANGE = 8,  // an assignment outside [0,K)
    ERR_ALIAS = 16,       // alias construction met an impossible state
};

constexpr uint32_t DK_EMPTY = 0xFFFFFFFFu;
constexpr uint32_t DK_HASH = 0x9E3779B1u;
constexpr int SORT_TILE = 2048;      // tokens per segmented-sort tile (one CTA)
constexpr int HIST_BINS = 32768;     // shared-memory histogram window (bins)
constexpr int HIST_CHUNK = 16384;    // tokens per CTA in the histogram path
constexpr int SAMPLE_TILE = 1024;    // tokens per CTA in the MH kernel
constexpr int ALIAS_WARP_MAX = 256;  // rows up to this many items are built by one warp

// Everything a kernel needs, passed by value.
struct View {
    int32_t V, K, N, D;
    double alpha, beta, Vbeta, Kalpha;
    int topic_bits;  // bits of K-1
    int count_bits;  // low bits of a packed n_kd entry that hold the count
    // tokens in word-sorted order
    const uint2* tok_dinfo;  // per token: (first token of its document, document length)
    const uint32_t* tok_orig;
    void* zw[2];  // assignments in word-sorted order (topic type: u16 or i32)
    void* zd[2];  // assignments in the caller's document order
    const int32_t* word_off;  // [V+1] token range of each word in word-sorted order
    const int32_t* doc_off;   // [D+1]
    // n_kw: every word has a sorted (topic, count) row of fixed capacity; hot words also a dense row
    const int32_t* row_start;  // [V+1] first slot of each word's row
    int32_t* wk_nnz;           // [V]
    uint32_t* wk_topic;        // [row_start[V]]
    uint32_t* wk_count;
    const int32_t* dense_slot;  // [V] index of the word's dense row or -1
    int32_t* dense_rows;        // [n_dense * K]
    // word-proposal tables
    uint32_t* al_thr;  // split point of each sparse bin as a 32-bit fraction
    uint32_t* al_idx;  // alias item of each sparse bin
    uint32_t* mix32;   // [V] share of the sparse term
    uint32_t* dn_thr;  // [K]
    uint32_t* dn_idx;  // [K]
    unsigned long long* dense_mass;
    int32_t* nk;  // [K]
    // n_kd: document d owns the open-addressing table dk_slots[2*doc_off[d] .. 2*doc_off[d+1])
    // (capacity twice the document length, load <= 0.5); a slot is (topic << count_bits) | count
    // or DK_EMPTY; topic k starts probing at umulhi(k * DK_HASH, capacity), linear, wrapping.
    uint32_t* dk_slots;
    int* err;
};

struct Ctx {
    int32_t V = 0, K = 0;
    double alpha = 0, beta = 0;
    int device = 0;
    cudaStream_t stream = nullptr;
    bool wide_topics = false;  // false: 16-bit topic storage, true: 32-bit
    double dense_frac = 0.05;
    double dense_min_tf = 64;
    bool loaded = false, inited = false, tables_valid = false;
    int cur = 0;  // which of the two z buffers is current
    uint64_t seed = 0;
    uint32_t sweep = 0;
    int64_t N = 0, D = 0;
    View v{};
    // host-side work lists (device copies below)
    int32_t n_word_tiles = 0, n_doc_tiles = 0, n_dense = 0, n_hist_chunks = 0, n_long_docs = 0,
            n_alias_big = 0;
    int32_t* word_tiles = nullptr;   // [n_word_tiles*2] word ranges sorted per CTA
    int32_t* doc_tiles = nullptr;    // [n_doc_tiles*2]
    int32_t* dense_words = nullptr;  // [n_dense]
    int32_t* hist_chunks = nullptr;  // [n_hist_chunks*3] (word, first token, count)
    int32_t* long_docs = nullptr;    // [n_long_docs]
    int32_t* alias_big = nullptr;    // [n_alias_big] words whose row can exceed ALIAS_WARP_MAX
    // alias-construction scratch
    unsigned long long* sc_w = nullptr;   // [row capacity total] scaled masses
    unsigned long long* sc_de = nullptr;  // deficits prefix (front) / surpluses prefix (back)
    uint32_t* sc_item = nullptr;          // light items (front) / heavy items (back)
    unsigned long long* sc_dense = nullptr;  // same three for the dense table, [3*K]
    double* red = nullptr;                   // reduction partials for the log-likelihood
    int64_t* red_i = nullptr;
    std::vector<void*> allocs;
    int64_t device_bytes = 0;
    lda_stats stats{};
    int64_t launches = 0;
    cudaEvent_t ev[8] = {};
    bool have_events = false;
    std::string err;
};

// --- launchers (each returns the number of kernels it launched) -----------------
int launch_init(Ctx& c);
int launch_spread_assignments(Ctx& c, const int32_t* z_dev);  // z (doc order, i32) -> both layouts
int launch_export_assignments(Ctx& c, int32_t* z_dev);
int launch_count_wk(Ctx& c);
int launch_count_k(Ctx& c);
int launch_count_dk(Ctx& c);
int launch_alias_dense(Ctx& c);
int launch_alias_sparse(Ctx& c);
int launch_sample(Ctx& c, int mh_steps);
int launch_loglik(Ctx& c, double* out3_host);
int launch_count_nnz(Ctx& c, int64_t* nnz_wk_host, int64_t* nnz_dk_host);

// load-time layout (sort + offsets); fills c.v token arrays. Returns LDA_* status.
int build_layout(Ctx& c, const int32_t* word_ids_dev, const int64_t* doc_off_host);

void* dev_alloc(Ctx& c, size_t bytes);  // tracked cudaMalloc; nullptr on failure
void dev_free_all(Ctx& c);

}  // namespace lda
