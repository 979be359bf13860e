// C ABI of the library: argument checks, device memory, work lists, launch order.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "lda_internal.cuh"

namespace lda {
void set_hist_smem_limits();
void set_sample_smem_limits();
void set_doc_smem_limits();
void set_alias_smem_limits();
void set_export_smem_limits();
void set_loglik_smem_limits();

void* raw_alloc(Ctx& c, size_t bytes)
{
    if (c.alloc_fn) return c.alloc_fn(bytes, c.alloc_user);
    void* p = nullptr;
    if (cudaMalloc(&p, bytes) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return p;
}

void raw_free(Ctx& c, void* p)
{
    if (!p) return;
    if (c.free_fn) c.free_fn(p, c.alloc_user);
    else cudaFree(p);
}

void* dev_alloc(Ctx& c, size_t bytes)
{
    if (bytes == 0) bytes = 16;
    void* p = raw_alloc(c, bytes);
    if (!p) return nullptr;
    c.allocs.push_back(p);
    c.alloc_bytes.push_back(bytes);
    c.alloc_own.push_back(c.alloc_fn ? 1 : 0);
    c.device_bytes += (int64_t)bytes;
    return p;
}

void dev_free(Ctx& c, void* p)
{
    if (!p) return;
    for (size_t i = 0; i < c.allocs.size(); ++i)
        if (c.allocs[i] == p) {
            c.device_bytes -= (int64_t)c.alloc_bytes[i];
            const bool own = c.alloc_own[i] != 0;
            c.allocs.erase(c.allocs.begin() + i);
            c.alloc_bytes.erase(c.alloc_bytes.begin() + i);
            c.alloc_own.erase(c.alloc_own.begin() + i);
            if (own && c.free_fn) c.free_fn(p, c.alloc_user);
            else cudaFree(p);
            return;
        }
}

void dev_free_all(Ctx& c)
{
    for (size_t i = 0; i < c.allocs.size(); ++i) {
        if (c.alloc_own[i] && c.free_fn) c.free_fn(c.allocs[i], c.alloc_user);
        else cudaFree(c.allocs[i]);
    }
    c.allocs.clear();
    c.alloc_bytes.clear();
    c.alloc_own.clear();
    c.device_bytes = 0;
}

static int fail(Ctx* c, int code, const char* msg)
{
    if (c) c->err = msg;
    return code;
}

static int cuda_fail(Ctx* c, const char* where)
{
    cudaError_t e = cudaGetLastError();
    if (c) c->err = std::string(where) + ": " + cudaGetErrorString(e);
    return LDA_ECUDA;
}

// Reads and clears the device error word.
static int read_err(Ctx& c, int* bits)
{
    if (cudaMemcpyAsync(bits, c.v.err, sizeof(int), cudaMemcpyDeviceToHost, c.stream) != cudaSuccess ||
        cudaStreamSynchronize(c.stream) != cudaSuccess)
        return cuda_fail(&c, "reading the device error word");
    if (*bits) cudaMemsetAsync(c.v.err, 0, sizeof(int), c.stream);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        c.err = std::string("kernel launch: ") + cudaGetErrorString(e);
        return LDA_ECUDA;
    }
    return LDA_OK;
}

static int check_device(Ctx& c)
{
    if (cudaSetDevice(c.device) != cudaSuccess) return cuda_fail(&c, "cudaSetDevice");
    return LDA_OK;
}

// An export started by lda_get_assignments*_async() may still be copying out of the staging buffer:
// whatever is queued on the context's stream from here on starts after it (no host wait).
static void order_after_export(Ctx& c)
{
    if (!c.export_pending) return;
    cudaStreamWaitEvent(c.stream, c.ev_export, 0);
    c.export_pending = false;
}

// Host wait for everything the context has queued, the copy stream included.
static int wait_all(Ctx& c)
{
    cudaError_t e = cudaStreamSynchronize(c.stream);
    if (e == cudaSuccess && c.copy) e = cudaStreamSynchronize(c.copy);
    c.export_pending = false;
    return e == cudaSuccess ? LDA_OK : cuda_fail(&c, "waiting for the context's streams");
}

template <typename T>
static T* upload(Ctx& c, const std::vector<T>& h)
{
    T* d = (T*)dev_alloc(c, h.size() * sizeof(T));
    if (d && !h.empty() &&
        cudaMemcpyAsync(d, h.data(), h.size() * sizeof(T), cudaMemcpyHostToDevice, c.stream) != cudaSuccess)
        return nullptr;
    return d;
}

static void free_corpus(Ctx& c)
{
    if (c.copy) cudaStreamSynchronize(c.copy);  // an export may still read the staging buffer
    c.export_pending = false;
    int* err = c.v.err;
    // the error word is allocated in lda_create and outlives corpora
    std::vector<void*> drop;
    for (void* p : c.allocs)
        if (p != (void*)err) drop.push_back(p);
    for (void* p : drop) dev_free(c, p);
    View nv{};
    nv.V = c.V; nv.K = c.K; nv.alpha = c.alpha; nv.beta = c.beta;
    nv.Vbeta = (double)c.V * c.beta;
    nv.Kalpha = (double)c.K * c.alpha;
    nv.dense_stride = (c.K + 3) & ~3;
    nv.err = err;
    nv.moves = c.v.moves;
    c.v = nv;
    c.loaded = c.inited = c.tables_valid = false;
    c.N = c.D = 0;
    c.side_steps = 0;
    c.slices.clear();
    c.cur_slice = 0;
    c.al_thr0 = c.al_idx0 = c.sc_item0 = c.sc_item = nullptr;
    c.al_pk0 = nullptr;
    c.sc_w0 = c.sc_de0 = c.sc_w = c.sc_de = nullptr;
}

// Row slot r of the running slice lives at entry r - row_lo of the slice-sized buffers: the pointers the
// kernels index with row slots are the buffers' moved back by row_lo entries (and only ever used with
// slots of that slice).
template <typename P>
static P* moved_back(P* base, int64_t entries)
{
    return base ? reinterpret_cast<P*>(reinterpret_cast<uintptr_t>(base) - (uintptr_t)entries * sizeof(P)) : nullptr;
}

void set_slice(Ctx& c, int slice)
{
    const Ctx::Slice& q = c.slices[(size_t)slice];
    c.cur_slice = slice;
    c.v.al_thr = moved_back(c.al_thr0, q.row_lo);
    c.v.al_idx = moved_back(c.al_idx0, q.row_lo);
    c.v.al_pk = moved_back(c.al_pk0, q.row_lo);
    c.sc_w = moved_back(c.sc_w0, q.row_lo);
    c.sc_de = moved_back(c.sc_de0, q.row_lo);
    c.sc_item = moved_back(c.sc_item0, q.row_lo);
}

}  // namespace lda

// Buffers the passes of the MH step hand results to each other in; sized by the number of steps.
int lda::ensure_exchange(Ctx& c, int mh_steps)
{
    if (c.N == 0) return LDA_OK;
    auto bytes_for = [&](int mode, int steps, size_t& prop_b, size_t& side_b, size_t& ua_b, int& stride) {
        const size_t zt = c.wide_topics ? 4 : 2, n = (size_t)c.N;
        const int n_word = mode == LDA_PROPOSALS_CYCLE ? (steps + 1) / 2 : mode == LDA_PROPOSALS_WORD ? steps : 0;
        const int n_doc = steps - n_word;
        const size_t planes = (size_t)(n_word > 0 ? n_word : 1);
        stride = (1 + steps + n_doc + 3) & ~3;  // own, one word per step, one uniform per doc step
        prop_b = zt * planes * n;
        side_b = 4 * (size_t)stride * n;
        ua_b = 4 * planes * n;
    };
    size_t pb = 0, sb = 0, ub = 0;
    int stride = 0;
    if (mh_steps <= c.side_steps && c.side_mode == c.proposals && c.v.dside) {
        // buffers laid out for more steps of the same schedule are large enough: only the record
        // stride follows the step count (a chain of two steps keeps its 16-byte records after a
        // chain of four has run)
        bytes_for(c.proposals, mh_steps, pb, sb, ub, stride);
        c.v.side_stride = stride;
        return LDA_OK;
    }
    cudaStreamSynchronize(c.stream);
    dev_free(c, c.v.prop);
    dev_free(c, c.v.dside);
    dev_free(c, c.v.ua_w);
    c.v.prop = nullptr;
    c.v.dside = nullptr;
    c.v.ua_w = nullptr;
    c.side_steps = 0;
    bytes_for(c.proposals, mh_steps, pb, sb, ub, stride);
    c.v.prop = dev_alloc(c, pb);
    c.v.dside = (uint32_t*)dev_alloc(c, sb);
    c.v.ua_w = (uint32_t*)dev_alloc(c, ub);
    if (!c.v.prop || !c.v.dside || !c.v.ua_w) {
        c.err = "device allocation failed";
        return LDA_ENOMEM;
    }
    c.v.side_stride = stride;
    c.side_steps = mh_steps;
    c.side_mode = c.proposals;
    return LDA_OK;
}

namespace lda {

static int rebuild_counts(Ctx& c, int64_t* launches)
{
    int n = launch_count_wk(c);
    n += launch_count_k(c);
    if (launches) *launches += n;
    c.tables_valid = false;
    return LDA_OK;
}

static int ensure_tables(Ctx& c)
{
    if (c.tables_valid) return LDA_OK;
    launch_alias_dense(c);
    launch_alias_sparse(c);  // the running slice's (lda_get_tables walks the slices itself)
    int bits = 0;
    int rc = read_err(c, &bits);
    if (rc) return rc;
    if (bits) return fail(&c, LDA_EINTERNAL, "alias construction raised the device error word");
    c.tables_valid = true;
    return LDA_OK;
}

static int load_common(Ctx& c, const int32_t* words_dev, int64_t n_tokens, const int64_t* doc_off,
                       int64_t n_docs)
{
    free_corpus(c);
    c.N = n_tokens;
    c.D = n_docs;
    View& v = c.v;
    v.N = (int32_t)n_tokens;
    v.D = (int32_t)n_docs;
    const int32_t V = c.V, K = c.K;
    const int32_t N = v.N, D = v.D;

    int64_t max_len = 0;
    for (int64_t d = 0; d < n_docs; ++d) max_len = std::max(max_len, doc_off[d + 1] - doc_off[d]);
    int tb = 1;
    while ((1ll << tb) < (long long)K) ++tb;
    int cb = 1;  // a count never has all bits set, so no entry equals the empty-slot marker
    while ((1ll << cb) <= max_len + 1) ++cb;
    if (tb + cb > 32) {
        free_corpus(c);
        return fail(&c, LDA_ERANGE, "bits(K-1) + bits(longest document) exceeds 32");
    }
    v.topic_bits = tb;
    v.count_bits = cb;
    v.tok_base = (uint32_t)c.shard_first_token;

    int rc = build_layout(c, words_dev, doc_off);
    if (rc != LDA_OK) { free_corpus(c); return fail(&c, rc, "building the word-sorted layout failed"); }
    int bits = 0;
    rc = read_err(c, &bits);
    if (rc) { free_corpus(c); return rc; }
    if (bits & ERR_WORD_RANGE) { free_corpus(c); return fail(&c, LDA_ERANGE, "word id outside [0,V)"); }

    std::vector<int32_t> word_off((size_t)V + 1);
    if (cudaMemcpy(word_off.data(), v.word_off, ((size_t)V + 1) * 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
        free_corpus(c);
        return cuda_fail(&c, "copying word offsets");
    }

    // --- dense / sparse class of every word (Section 5) ---------------------------------
    // tf_here: the word's tokens in this corpus (its token range); tf: what the word's row and class
    // are sized for -- the same, unless the corpus is one shard of a larger one (lda_set_shard), in
    // which case the row has to hold the counts of all shards
    std::vector<int32_t> tf_here((size_t)V), tf((size_t)V);
    for (int32_t w = 0; w < V; ++w) {
        tf_here[w] = word_off[w + 1] - word_off[w];
        tf[w] = c.shard_global_tf.empty() ? tf_here[w] : std::max(tf_here[w], c.shard_global_tf[(size_t)w]);
    }
    int32_t tf_cut = INT32_MAX;
    const int64_t n_top = (int64_t)std::floor(c.dense_frac * (double)V);
    if (n_top > 0) {
        std::vector<int32_t> tmp(tf);
        const size_t nth = (size_t)std::min<int64_t>(n_top, V) - 1;
        std::nth_element(tmp.begin(), tmp.begin() + nth, tmp.end(), std::greater<int32_t>());
        // a dense row of K counters only pays for a word with a fair share of K tokens
        tf_cut = std::max<int32_t>({tmp[nth], (int32_t)std::max(1.0, c.dense_min_tf), K / 8});
    }
    // K above the staging limit: only words with more than WARM_MAX_TF tokens get a dense row, the
    // others with more tokens than a tail tile holds a sorted row built by a CTA of their own
    const bool warm_class = K > HOT_STAGE_MAX_K;
    std::vector<int32_t> warm_words;
    std::vector<int32_t> dense_slot((size_t)V, -1), dense_words, row_start((size_t)V + 1), alias_big, alias_mid;
    std::vector<int32_t> hist_chunks, word_tiles;
    int64_t cap_total = 0;
    for (int32_t w = 0; w < V; ++w) {
        row_start[w] = (int32_t)cap_total;
        const int32_t cap = std::min(tf[w], K);
        cap_total += cap;
        if (cap > ALIAS_SMEM_ITEMS_MID) alias_big.push_back(w);
        else if (cap > ALIAS_WARP_MAX) alias_mid.push_back(w);
        if (warm_class && tf[w] > SORT_TILE && tf[w] <= WARM_MAX_TF) {
            warm_words.push_back(w);
        } else if (tf[w] > SORT_TILE || (tf[w] > 0 && tf[w] >= tf_cut)) {
            dense_slot[w] = (int32_t)dense_words.size();
            dense_words.push_back(w);
            for (int32_t o = 0; o < tf_here[w]; o += HIST_CHUNK) {
                hist_chunks.push_back(w);
                hist_chunks.push_back(word_off[w] + o);
                hist_chunks.push_back(std::min(HIST_CHUNK, tf_here[w] - o));
                hist_chunks.push_back(tf_here[w] <= HIST_CHUNK ? 1 : 0);
            }
        }
    }
    row_start[V] = (int32_t)cap_total;
    // vocabulary slices of about equal row capacity; slice_w[s] = first word of slice s
    const int n_slices = std::max(1, c.alias_slices);
    std::vector<int32_t> slice_w((size_t)n_slices + 1, V);
    slice_w[0] = 0;
    for (int sl = 1; sl < n_slices; ++sl) {
        const int32_t target = (int32_t)(cap_total * sl / n_slices);
        slice_w[sl] = (int32_t)(std::lower_bound(row_start.begin(), row_start.begin() + V, target) - row_start.begin());
    }
    std::vector<char> slice_starts((size_t)V + 1, 0);
    for (int sl = 1; sl < n_slices; ++sl) slice_starts[(size_t)slice_w[sl]] = 1;
    // tiles of consecutive sparse words: <= SORT_TILE tokens and <= SORT_TILE words each
    {
        int32_t s0 = 0, tok = 0;
        auto close = [&](int32_t s1) {
            if (s1 > s0) { word_tiles.push_back(s0); word_tiles.push_back(s1); }
        };
        for (int32_t w = 0; w < V; ++w) {
            if (dense_slot[w] >= 0 || tf[w] > SORT_TILE) { close(w); s0 = w + 1; tok = 0; continue; }
            if (tok + tf[w] > SORT_TILE || w - s0 >= SORT_TILE) { close(w); s0 = w; tok = 0; }
            tok += tf[w];
        }
        close(V);
    }
    // MH kernel work lists: a hot word (more tokens than a tail tile holds; it has a dense row by
    // the rule above) is cut into runs of HOT_TILE tokens, tail words are packed whole into tiles
    std::vector<int32_t> hot_tiles, hot_tiles_warm, hot_tiles_propose, cold_tiles;
    {
        static_assert(COLD_TILE >= SORT_TILE, "every word longer than a tail tile must have a dense row or a warm one");
        int32_t s0 = 0, tok = 0;
        auto close = [&](int32_t s1) {
            if (s1 > s0 && tok > 0) { cold_tiles.push_back(s0); cold_tiles.push_back(s1); }
        };
        for (int32_t w = 0; w < V; ++w) {
            if (slice_starts[w]) { close(w); s0 = w; tok = 0; }  // no tile reaches across two slices
            if (tf[w] > COLD_TILE) {
                close(w); s0 = w + 1; tok = 0;
                std::vector<int32_t>& runs = dense_slot[w] >= 0 ? hot_tiles : hot_tiles_warm;
                for (int32_t o = 0; o < tf_here[w]; o += HOT_TILE) {
                    runs.push_back(w);
                    runs.push_back(word_off[w] + o);
                    runs.push_back(std::min(HOT_TILE, tf_here[w] - o));
                }
                for (int32_t o = 0; o < tf_here[w]; o += HOT_TILE_PROPOSE) {
                    hot_tiles_propose.push_back(w);
                    hot_tiles_propose.push_back(word_off[w] + o);
                    hot_tiles_propose.push_back(std::min(HOT_TILE_PROPOSE, tf_here[w] - o));
                }
                continue;
            }
            if (tok + tf[w] > COLD_TILE || w - s0 >= COLD_WORDS) { close(w); s0 = w; tok = 0; }
            tok += tf[w];
        }
        close(V);
    }
    // document tiles: the smallest tile shape that leaves at most 5 % of the tokens in documents
    // too long for a tile (those get a CTA of their own and a table in device memory)
    std::vector<int32_t> doc_tiles, long_docs;
    {
        int shape = DOC_TILE_SHAPES - 1;
        for (int sft = 0; sft < DOC_TILE_SHAPES; ++sft) {
            int64_t over = 0;
            for (int32_t d = 0; d < D; ++d) {
                const int64_t len = doc_off[d + 1] - doc_off[d];
                if (len > DOC_TILE_TOKENS[sft]) over += len;
            }
            if (over * 20 <= (int64_t)N) { shape = sft; break; }
        }
        c.doc_tile = DOC_TILE_TOKENS[shape];
        c.doc_threads = DOC_TILE_THREADS[shape];
        const int32_t tile = c.doc_tile;
        int32_t s0 = 0;
        int64_t tok = 0;
        auto close = [&](int32_t s1) {
            if (s1 > s0) { doc_tiles.push_back(s0); doc_tiles.push_back(s1); }
        };
        for (int32_t d = 0; d < D; ++d) {
            const int64_t len = doc_off[d + 1] - doc_off[d];
            if (len > tile) { close(d); s0 = d + 1; tok = 0; long_docs.push_back(d); continue; }
            if (tok + len > tile || d - s0 >= tile) { close(d); s0 = d; tok = 0; }
            tok += len;
        }
        close(D);
    }
    // tiles of whole documents for the sorted n_kd rows: <= SORT_TILE tokens and <= SORT_TILE documents each
    std::vector<int32_t> doc_sort_tiles, doc_sort_long;
    {
        int32_t s0 = 0;
        int64_t tok = 0;
        auto close = [&](int32_t s1) {
            if (s1 > s0) { doc_sort_tiles.push_back(s0); doc_sort_tiles.push_back(s1); }
        };
        for (int32_t d = 0; d < D; ++d) {
            const int64_t len = doc_off[d + 1] - doc_off[d];
            if (len > SORT_TILE) { close(d); s0 = d + 1; tok = 0; doc_sort_long.push_back(d); continue; }
            if (tok + len > SORT_TILE || d - s0 >= SORT_TILE) { close(d); s0 = d; tok = 0; }
            tok += len;
        }
        close(D);
    }
    c.n_doc_sort_tiles = (int32_t)(doc_sort_tiles.size() / 2);
    c.n_doc_sort_long = (int32_t)doc_sort_long.size();
    c.n_word_tiles = (int32_t)(word_tiles.size() / 2);
    c.n_doc_tiles = (int32_t)(doc_tiles.size() / 2);
    c.n_dense = (int32_t)dense_words.size();
    c.n_hist_chunks = (int32_t)(hist_chunks.size() / 4);
    c.n_long_docs = (int32_t)long_docs.size();
    c.n_alias_mid = (int32_t)alias_mid.size();
    alias_big.insert(alias_big.begin(), alias_mid.begin(), alias_mid.end());
    c.n_alias_big = (int32_t)alias_big.size();
    c.n_hot_tiles = (int32_t)(hot_tiles.size() / 3);
    c.n_hot_tiles_warm = (int32_t)(hot_tiles_warm.size() / 3);
    c.n_warm = (int32_t)warm_words.size();
    c.n_hot_tiles_propose = (int32_t)(hot_tiles_propose.size() / 3);
    c.n_cold_tiles = (int32_t)(cold_tiles.size() / 2);
    c.slices.assign((size_t)n_slices, Ctx::Slice{});
    int64_t slice_rows_max = 1;
    {
        // every list is in ascending word order: a slice's part is a run of it
        auto first_at = [](const std::vector<int32_t>& list, size_t lo, size_t hi, int stride, int32_t w) {
            size_t a = lo, b = hi;  // first entry of [lo, hi) whose word is >= w
            while (a < b) {
                const size_t m = (a + b) / 2;
                if (list[m * stride] < w) a = m + 1; else b = m;
            }
            return (int32_t)a;
        };
        const size_t n_mid = (size_t)c.n_alias_mid, n_big = (size_t)c.n_alias_big;
        for (int sl = 0; sl < n_slices; ++sl) {
            Ctx::Slice& q = c.slices[(size_t)sl];
            q.w_lo = slice_w[(size_t)sl];
            q.w_hi = slice_w[(size_t)sl + 1];
            q.row_lo = row_start[(size_t)q.w_lo];
            q.row_n = row_start[(size_t)q.w_hi] - q.row_lo;
            slice_rows_max = std::max(slice_rows_max, q.row_n);
            q.mid_lo = first_at(alias_big, 0, n_mid, 1, q.w_lo);
            q.mid_n = first_at(alias_big, 0, n_mid, 1, q.w_hi) - q.mid_lo;
            q.big_lo = first_at(alias_big, n_mid, n_big, 1, q.w_lo) - (int32_t)n_mid;
            q.big_n = first_at(alias_big, n_mid, n_big, 1, q.w_hi) - (int32_t)n_mid - q.big_lo;
            q.hotp_lo = first_at(hot_tiles_propose, 0, (size_t)c.n_hot_tiles_propose, 3, q.w_lo);
            q.hotp_n = first_at(hot_tiles_propose, 0, (size_t)c.n_hot_tiles_propose, 3, q.w_hi) - q.hotp_lo;
            q.cold_lo = first_at(cold_tiles, 0, (size_t)c.n_cold_tiles, 2, q.w_lo);
            q.cold_n = first_at(cold_tiles, 0, (size_t)c.n_cold_tiles, 2, q.w_hi) - q.cold_lo;
        }
    }
    const size_t cap_alias = (size_t)slice_rows_max;

    const size_t n1 = (size_t)std::max<int64_t>(N, 1), cap1 = (size_t)std::max<int64_t>(cap_total, 1);
    const size_t zt = c.wide_topics ? 4 : 2;
    bool ok = true;
    auto A = [&](size_t bytes) { void* p = dev_alloc(c, bytes); ok = ok && p; return p; };
    v.zw = A(n1 * zt);
    v.zbm = A(2 * n1 * zt);  // (topic, first word-proposal) pairs
    v.rec = (uint32_t*)A(n1 * 4 + 16);  // + one aligned group of four words past the last record
    v.row_start = upload(c, row_start);
    v.dense_slot = upload(c, dense_slot);
    c.word_tiles = upload(c, word_tiles);
    c.doc_tiles = upload(c, doc_tiles);
    c.dense_words = upload(c, dense_words);
    c.hist_chunks = upload(c, hist_chunks);
    c.long_docs = upload(c, long_docs);
    c.doc_sort_tiles = upload(c, doc_sort_tiles);
    c.doc_sort_long = upload(c, doc_sort_long);
    c.alias_big = upload(c, alias_big);
    c.hot_tiles = upload(c, hot_tiles);
    c.hot_tiles_warm = upload(c, hot_tiles_warm);
    c.warm_words = upload(c, warm_words);
    c.hot_tiles_propose = upload(c, hot_tiles_propose);
    c.cold_tiles = upload(c, cold_tiles);
    ok = ok && v.row_start && v.dense_slot && c.word_tiles && c.doc_tiles && c.dense_words &&
         c.hist_chunks && c.long_docs && c.doc_sort_tiles && c.doc_sort_long && c.alias_big && c.hot_tiles && c.hot_tiles_warm && c.warm_words && c.hot_tiles_propose && c.cold_tiles;
    v.wk_nnz = (int32_t*)A((size_t)V * 4);
    v.wk_topic = (uint32_t*)A(cap1 * 4);
    v.wk_count = (uint32_t*)A(cap1 * 4);
    v.dense_rows = (int32_t*)A(std::max<size_t>((size_t)c.n_dense * v.dense_stride, 1) * 4);
    c.al_thr0 = (uint32_t*)A(cap_alias * 4);
    c.al_idx0 = (uint32_t*)A(cap_alias * 4);
    c.al_pk0 = c.wide_topics ? nullptr : (uint2*)A(cap_alias * 8);
    v.dn_pk = (uint2*)A((size_t)K * 8);
    v.mix32 = (uint32_t*)A((size_t)V * 4);
    v.dn_thr = (uint32_t*)A((size_t)K * 4);
    v.dn_idx = (uint32_t*)A((size_t)K * 4);
    v.dense_mass = (unsigned long long*)A(8);
    v.nk = (int32_t*)A((size_t)v.dense_stride * 4);  // padded like a dense row: copied in 16-byte units
    // scratch tables of the documents longer than a tile: four slots per token, one document after the other
    std::vector<long long> long_slot_off(long_docs.size() + 1, 0);
    for (size_t i = 0; i < long_docs.size(); ++i)
        long_slot_off[i + 1] = long_slot_off[i] + 4ll * (doc_off[long_docs[i] + 1] - doc_off[long_docs[i]]);
    v.dk_slots = (uint32_t*)A((size_t)long_slot_off.back() * 4 + 32);
    v.long_slot_off = upload(c, long_slot_off);
    ok = ok && v.long_slot_off;
    c.sc_w0 = (unsigned long long*)A(cap_alias * 8);
    c.sc_de0 = (unsigned long long*)A(cap_alias * 8);
    c.sc_item0 = (uint32_t*)A(cap_alias * 4);
    c.sc_dense = (unsigned long long*)A((size_t)K * 8 * 3);
    c.red = (double*)A(sizeof(double) * (LL_WORD_PARTIALS + LL_DOC_PARTIALS));
    c.red_i = (int64_t*)A(16);
    c.ll_tab = (double*)A(sizeof(double) * 2 * 512);
    c.ll_tile_part = (double*)A(sizeof(double) * std::max<size_t>((size_t)c.n_doc_tiles, 1));
    c.ll_tile_nnz = (uint32_t*)A(4 * std::max<size_t>((size_t)c.n_doc_tiles, 1));
    c.ll_tables_ready = false;
    if (!ok) { free_corpus(c); return fail(&c, LDA_ENOMEM, "device allocation failed"); }
    set_slice(c, 0);
    cudaMemsetAsync(v.wk_nnz, 0, (size_t)V * 4, c.stream);
    cudaMemsetAsync(v.mix32, 0, (size_t)V * 4, c.stream);
    cudaMemsetAsync(v.nk, 0, (size_t)K * 4, c.stream);
    if (cudaStreamSynchronize(c.stream) != cudaSuccess) { free_corpus(c); return cuda_fail(&c, "load"); }
    c.stats = lda_stats{};
    c.stats.n_tokens = N;
    c.stats.n_docs = D;
    c.stats.n_dense_words = c.n_dense;
    c.n_nonempty_docs = 0;
    for (int64_t d = 0; d < n_docs; ++d) c.n_nonempty_docs += doc_off[d + 1] > doc_off[d];
    c.loaded = true;
    return LDA_OK;
}

static int validate_offsets(Ctx* c, int64_t n_tokens, const int64_t* doc_off, int64_t n_docs)
{
    if (n_tokens >= 2147483648ll || n_docs >= 2147483647ll) return fail(c, LDA_ERANGE, "n_tokens and n_docs must be below 2^31");
    if (doc_off[0] != 0 || doc_off[n_docs] != n_tokens)
        return fail(c, LDA_ERANGE, "doc_offsets must start at 0 and end at n_tokens");
    for (int64_t d = 0; d < n_docs; ++d)
        if (doc_off[d + 1] < doc_off[d]) return fail(c, LDA_ERANGE, "doc_offsets must be non-decreasing");
    return LDA_OK;
}

}  // namespace lda

using namespace lda;

struct lda_ctx {
    Ctx c;
};

extern "C" {

int lda_create(int32_t V, int32_t K, double alpha, double beta, lda_ctx** out)
{
    if (!out) return LDA_EINVAL;
    *out = nullptr;
    if (V <= 0 || K <= 0 || !(alpha > 0) || !(beta > 0) || !std::isfinite(alpha) || !std::isfinite(beta))
        return LDA_EINVAL;
    if (K > 131072) return LDA_ERANGE;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return LDA_ECUDA; }
    lda_ctx* h = new (std::nothrow) lda_ctx();
    if (!h) return LDA_ENOMEM;
    Ctx& c = h->c;
    c.V = V; c.K = K; c.alpha = alpha; c.beta = beta; c.device = dev;
    if (cudaDeviceGetAttribute(&c.n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || c.n_sm < 1) {
        cudaGetLastError();
        c.n_sm = 148;
    }
    c.wide_topics = K > 65536;
    c.v.V = V; c.v.K = K; c.v.alpha = alpha; c.v.beta = beta;
    c.v.Vbeta = (double)V * beta;
    c.v.Kalpha = (double)K * alpha;
    c.v.dense_stride = (K + 3) & ~3;
    c.v.err = (int*)dev_alloc(c, 32);  // the error word and, 16 bytes on, the two move counters
    c.v.moves = c.v.err ? reinterpret_cast<unsigned long long*>(reinterpret_cast<char*>(c.v.err) + 16) : nullptr;
    if (!c.v.err || cudaMemset(c.v.err, 0, 32) != cudaSuccess) {
        dev_free_all(c);
        delete h;
        cudaGetLastError();
        return LDA_ECUDA;
    }
    for (int i = 0; i < Ctx::EV_RING * 10; ++i)
        if (cudaEventCreate(&c.ev_ring[i / 10][i % 10]) != cudaSuccess) {
            for (int j = 0; j < i; ++j) cudaEventDestroy(c.ev_ring[j / 10][j % 10]);
            dev_free_all(c);
            delete h;
            cudaGetLastError();
            return LDA_ECUDA;
        }
    c.have_events = true;
    {
        bool ok = cudaEventCreateWithFlags(&c.ev_fork, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < 2 && ok; ++i)
            ok = cudaEventCreateWithFlags(&c.ev_join[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaStreamCreateWithFlags(&c.side[i], cudaStreamNonBlocking) == cudaSuccess;
        ok = ok && cudaStreamCreateWithFlags(&c.copy, cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&c.ev_chunk, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c.ev_export, cudaEventDisableTiming) == cudaSuccess;
        c.have_side = true;  // lda_destroy() releases whatever was created
        if (!ok) {
            lda_destroy(h);
            return LDA_ECUDA;
        }
    }
    set_hist_smem_limits();
    set_sample_smem_limits();
    set_doc_smem_limits();
    set_alias_smem_limits();
    set_export_smem_limits();
    set_loglik_smem_limits();
    set_gibbs_smem_limits();
    *out = h;
    return LDA_OK;
}

void lda_destroy(lda_ctx* h)
{
    if (!h) return;
    Ctx& c = h->c;
    cudaSetDevice(c.device);
    cudaStreamSynchronize(c.stream);
    if (c.have_side) {
        for (int i = 0; i < 2; ++i) {
            if (c.side[i]) {
                cudaStreamSynchronize(c.side[i]);
                cudaStreamDestroy(c.side[i]);
            }
            if (c.ev_join[i]) cudaEventDestroy(c.ev_join[i]);
        }
        if (c.ev_fork) cudaEventDestroy(c.ev_fork);
        if (c.copy) {
            cudaStreamSynchronize(c.copy);
            cudaStreamDestroy(c.copy);
        }
        if (c.ev_chunk) cudaEventDestroy(c.ev_chunk);
        if (c.ev_export) cudaEventDestroy(c.ev_export);
    }
    if (c.have_events)
        for (int i = 0; i < Ctx::EV_RING * 10; ++i) cudaEventDestroy(c.ev_ring[i / 10][i % 10]);
    dev_free_all(c);
    cudaGetLastError();
    delete h;
}

const char* lda_last_error(const lda_ctx* h) { return h ? h->c.err.c_str() : "null context"; }

int lda_set_stream(lda_ctx* h, void* cuda_stream)
{
    if (!h) return LDA_EINVAL;
    cudaStreamSynchronize(h->c.stream);
    h->c.stream = (cudaStream_t)cuda_stream;
    return LDA_OK;
}

int lda_set_allocator(lda_ctx* h, lda_alloc_fn alloc_fn, lda_free_fn free_fn, void* user)
{
    if (!h || (alloc_fn == nullptr) != (free_fn == nullptr)) return LDA_EINVAL;
    Ctx& c = h->c;
    if (c.loaded) return fail(&c, LDA_ESTATE, "lda_set_allocator must come before lda_load_corpus");
    c.alloc_fn = alloc_fn;
    c.free_fn = free_fn;
    c.alloc_user = user;
    return LDA_OK;
}

int lda_set_option(lda_ctx* h, const char* key, double value)
{
    if (!h || !key) return LDA_EINVAL;
    Ctx& c = h->c;
    if (c.loaded) return fail(&c, LDA_ESTATE, "options must be set before lda_load_corpus");
    if (!std::strcmp(key, "dense_frac")) {
        if (!(value >= 0.0 && value <= 1.0)) return fail(&c, LDA_EINVAL, "dense_frac must be in [0,1]");
        c.dense_frac = value;
        return LDA_OK;
    }
    if (!std::strcmp(key, "alias_slices")) {
        if (!(value >= 1.0 && value <= 256.0) || value != std::floor(value))
            return fail(&c, LDA_EINVAL, "alias_slices must be a whole number in [1,256]");
        c.alias_slices = (int)value;
        return LDA_OK;
    }
    if (!std::strcmp(key, "copy_chunk_log2")) {
        if (!(value >= 10.0 && value <= 30.0) || value != std::floor(value))
            return fail(&c, LDA_EINVAL, "copy_chunk_log2 must be a whole number in [10,30]");
        c.copy_chunk = (int64_t)1 << (int)value;
        return LDA_OK;
    }
    if (!std::strcmp(key, "dense_min_tf")) {
        if (!(value >= 1.0)) return fail(&c, LDA_EINVAL, "dense_min_tf must be >= 1");
        c.dense_min_tf = value;
        return LDA_OK;
    }
    if (!std::strcmp(key, "block_log2")) {
        if (!(value >= 10.0 && value <= 30.0)) return fail(&c, LDA_EINVAL, "block_log2 must be in [10,30]");
        c.block_shift = (int)value;
        return LDA_OK;
    }
    return fail(&c, LDA_EINVAL, "unknown option");
}

int lda_set_proposals(lda_ctx* h, int mode)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (mode != LDA_PROPOSALS_CYCLE && mode != LDA_PROPOSALS_WORD && mode != LDA_PROPOSALS_DOC)
        return fail(&c, LDA_EINVAL, "unknown proposal mode");
    c.proposals = mode;  // the exchange buffers are laid out again by the next sweep
    return LDA_OK;
}

int lda_load_corpus(lda_ctx* h, const int32_t* word_ids, int64_t n_tokens, const int64_t* doc_offsets,
                    int64_t n_docs)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (!doc_offsets || n_tokens < 0 || n_docs < 0 || (n_tokens > 0 && !word_ids))
        return fail(&c, LDA_EINVAL, "null pointer or negative size");
    int rc = validate_offsets(&c, n_tokens, doc_offsets, n_docs);
    if (rc) return rc;
    if ((rc = check_device(c))) return rc;
    int32_t* wd = nullptr;
    if (!tmp_alloc(c, &wd, (size_t)std::max<int64_t>(n_tokens, 1) * 4)) return fail(&c, LDA_ENOMEM, "device allocation failed");
    if (n_tokens > 0 &&
        cudaMemcpyAsync(wd, word_ids, (size_t)n_tokens * 4, cudaMemcpyHostToDevice, c.stream) != cudaSuccess) {
        raw_free(c, wd);
        return cuda_fail(&c, "copying word ids");
    }
    rc = load_common(c, wd, n_tokens, doc_offsets, n_docs);
    cudaStreamSynchronize(c.stream);
    raw_free(c, wd);
    return rc;
}

int lda_load_corpus_device(lda_ctx* h, const int32_t* word_ids_dev, int64_t n_tokens,
                           const int64_t* doc_offsets_dev, int64_t n_docs)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (!doc_offsets_dev || n_tokens < 0 || n_docs < 0 || (n_tokens > 0 && !word_ids_dev))
        return fail(&c, LDA_EINVAL, "null pointer or negative size");
    if (n_docs >= 2147483647ll) return fail(&c, LDA_ERANGE, "n_docs must be below 2^31");
    int rc = check_device(c);
    if (rc) return rc;
    std::vector<int64_t> off((size_t)n_docs + 1);
    if (cudaMemcpy(off.data(), doc_offsets_dev, ((size_t)n_docs + 1) * 8, cudaMemcpyDeviceToHost) != cudaSuccess)
        return cuda_fail(&c, "copying doc offsets");
    if ((rc = validate_offsets(&c, n_tokens, off.data(), n_docs))) return rc;
    return load_common(c, word_ids_dev, n_tokens, off.data(), n_docs);
}

int lda_init(lda_ctx* h, uint64_t seed)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (!c.loaded) return fail(&c, LDA_ESTATE, "lda_init before lda_load_corpus");
    int rc = check_device(c);
    if (rc) return rc;
    order_after_export(c);
    c.seed = seed;
    c.sweep = 0;
    launch_init(c);
    rebuild_counts(c, nullptr);
    int bits = 0;
    if ((rc = read_err(c, &bits))) return rc;
    if (bits) return fail(&c, LDA_EINTERNAL, "count rebuild raised the device error word");
    c.inited = true;
    return LDA_OK;
}

static int set_assignments(lda_ctx* h, const void* z, bool narrow, uint64_t seed, uint32_t sweep)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (!c.loaded) return fail(&c, LDA_ESTATE, "lda_set_assignments before lda_load_corpus");
    if (narrow && c.wide_topics) return fail(&c, LDA_ERANGE, "16-bit assignments need K <= 65536");
    if (c.N > 0 && !z) return fail(&c, LDA_EINVAL, "null assignments");
    int rc = check_device(c);
    if (rc) return rc;
    // the record array (one word per token, only meaningful while the exported n_kd is valid)
    // doubles as the staging buffer: no allocation here
    char* zdev = reinterpret_cast<char*>(c.v.rec);
    order_after_export(c);
    // chunk by chunk on the copy stream, each chunk spread into the block-major order (on the context's
    // stream) while the next one is on its way
    const size_t zt = narrow ? 2 : 4;
    cudaEventRecord(c.ev_chunk, c.stream);
    cudaStreamWaitEvent(c.copy, c.ev_chunk, 0);  // the staging buffer's earlier users are done
    for (int64_t first = 0; first < c.N; first += c.copy_chunk) {
        const int64_t count = std::min<int64_t>(c.copy_chunk, c.N - first);
        if (cudaMemcpyAsync(zdev + (size_t)first * zt, reinterpret_cast<const char*>(z) + (size_t)first * zt,
                            (size_t)count * zt, cudaMemcpyHostToDevice, c.copy) != cudaSuccess)
            return cuda_fail(&c, "copying assignments");
        cudaEventRecord(c.ev_chunk, c.copy);
        cudaStreamWaitEvent(c.stream, c.ev_chunk, 0);
        launch_spread_chunk(c, zdev, narrow, first, count);
    }
    launch_word_order_topics(c);
    int bits = 0;
    rc = read_err(c, &bits);
    if (rc) return rc;
    if (bits & ERR_TOPIC_RANGE) { c.inited = false; return fail(&c, LDA_ERANGE, "assignment outside [0,K)"); }
    c.seed = seed;
    c.sweep = sweep;
    rebuild_counts(c, nullptr);
    if ((rc = read_err(c, &bits))) return rc;
    if (bits) return fail(&c, LDA_EINTERNAL, "count rebuild raised the device error word");
    c.inited = true;
    return LDA_OK;
}

int lda_set_assignments(lda_ctx* h, const int32_t* z, uint64_t seed, uint32_t sweep)
{
    return set_assignments(h, z, false, seed, sweep);
}

int lda_set_assignments_u16(lda_ctx* h, const uint16_t* z, uint64_t seed, uint32_t sweep)
{
    return set_assignments(h, z, true, seed, sweep);
}

int lda_sweep(lda_ctx* h, int32_t iters, int32_t mh_steps)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (iters < 0 || mh_steps < 1 || mh_steps > 1024)
        return fail(&c, LDA_EINVAL, "iters must be >= 0 and mh_steps in 1..1024");
    if (!c.inited) return fail(&c, LDA_ESTATE, "lda_sweep before lda_init");
    int rc = check_device(c);
    if (rc) return rc;
    order_after_export(c);
    if ((rc = ensure_exchange(c, mh_steps))) return rc;
    lda_stats& s = c.stats;
    s.ms_alias_dense = s.ms_alias_sparse = s.ms_sample = s.ms_count_wk = s.ms_count_k = s.ms_count_dk =
        s.ms_total = s.ms_propose = s.ms_doc_side = s.ms_accept = 0.f;
    s.kernel_launches = 0;
    s.iters = iters;
    s.word_proposed = s.word_accepted = s.doc_proposed = s.doc_accepted = 0;
    if (cudaMemsetAsync(c.v.moves, 0, 16, c.stream) != cudaSuccess) return cuda_fail(&c, "clearing the move counters");
    // Iterations are queued without waiting for each other; the host waits once per EV_RING of them
    // (and after the last) to read the error word, the move counters and the phase timings.
    for (int32_t it0 = 0; it0 < iters; it0 += Ctx::EV_RING) {
        const int32_t batch = std::min<int32_t>(Ctx::EV_RING, iters - it0);
        for (int32_t b = 0; b < batch; ++b) {
            c.ev = c.ev_ring[b];
            int64_t n = 0;
            cudaEventRecord(c.ev[0], c.stream);
            n += launch_alias_dense(c);
            cudaEventRecord(c.ev[1], c.stream);
            if (c.slices.size() == 1) n += launch_alias_sparse(c);  // else slice by slice inside pass 1
            cudaEventRecord(c.ev[2], c.stream);
            n += launch_sample(c, mh_steps);
            cudaEventRecord(c.ev[3], c.stream);
            n += launch_count_wk(c);
            cudaEventRecord(c.ev[4], c.stream);
            n += launch_count_k(c);
            cudaEventRecord(c.ev[5], c.stream);
            cudaEventRecord(c.ev[6], c.stream);  // n_kd is rebuilt inside the next MH step, per tile
            c.tables_valid = false;
            c.sweep += 1;
            s.kernel_launches += n;
        }
        c.ev = c.ev_ring[0];
        int bits = 0;
        if ((rc = read_err(c, &bits))) { c.inited = false; return rc; }
        if (bits) {
            // some iteration of this batch met inconsistent tables: the state is not to be trusted
            c.inited = false;
            c.err = "a kernel raised the device error word: " + std::to_string(bits) +
                    " (call lda_init or lda_set_assignments again)";
            return LDA_EINTERNAL;
        }
        for (int32_t b = 0; b < batch; ++b) {
            cudaEvent_t* ev = c.ev_ring[b];
            float ms[7] = {0};
            for (int i = 0; i < 6; ++i) cudaEventElapsedTime(&ms[i], ev[i], ev[i + 1]);
            cudaEventElapsedTime(&ms[6], ev[0], ev[6]);
            if (c.N > 0) {
                float a = 0.f, bb = 0.f, d = 0.f;
                cudaEventElapsedTime(&a, ev[2], ev[8]);
                cudaEventElapsedTime(&bb, ev[8], ev[9]);
                cudaEventElapsedTime(&d, ev[9], ev[3]);
                s.ms_propose += a; s.ms_doc_side += bb; s.ms_accept += d;
            }
            s.ms_alias_dense += ms[0]; s.ms_alias_sparse += ms[1]; s.ms_sample += ms[2];
            s.ms_count_wk += ms[3]; s.ms_count_k += ms[4]; s.ms_count_dk += ms[5]; s.ms_total += ms[6];
        }
    }
    {
        unsigned long long moves[2] = {0, 0};
        if (cudaMemcpyAsync(moves, c.v.moves, 16, cudaMemcpyDeviceToHost, c.stream) != cudaSuccess ||
            cudaStreamSynchronize(c.stream) != cudaSuccess)
            return cuda_fail(&c, "reading the move counters");
        const int64_t n_word = c.proposals == LDA_PROPOSALS_CYCLE  ? (mh_steps + 1) / 2
                               : c.proposals == LDA_PROPOSALS_WORD ? mh_steps
                                                                   : 0;
        s.word_proposed = (int64_t)iters * c.N * n_word;
        s.doc_proposed = (int64_t)iters * c.N * (mh_steps - n_word);
        s.word_accepted = (int64_t)moves[0];
        s.doc_accepted = (int64_t)moves[1];
    }
    return LDA_OK;
}

int lda_set_shard(lda_ctx* h, int64_t first_token, const int32_t* global_term_freq)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (c.loaded) return fail(&c, LDA_ESTATE, "lda_set_shard must come before lda_load_corpus");
    if (first_token < 0 || first_token >= 4294967296ll) return fail(&c, LDA_ERANGE, "first_token must be in [0, 2^32)");
    c.shard_first_token = first_token;
    c.shard_global_tf.clear();
    if (global_term_freq) {
        for (int32_t w = 0; w < c.V; ++w)
            if (global_term_freq[w] < 0) return fail(&c, LDA_ERANGE, "negative term frequency");
        c.shard_global_tf.assign(global_term_freq, global_term_freq + c.V);
    }
    return LDA_OK;
}

int lda_word_counts_to_dense(lda_ctx* h, int32_t* nwk_dev)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (!nwk_dev) return fail(&c, LDA_EINVAL, "null matrix");
    if (!c.inited) return fail(&c, LDA_ESTATE, "lda_word_counts_to_dense before lda_init");
    int rc = check_device(c);
    if (rc) return rc;
    launch_word_counts_to_dense(c, nwk_dev);
    if (cudaStreamSynchronize(c.stream) != cudaSuccess || cudaGetLastError() != cudaSuccess)
        return cuda_fail(&c, "writing the count matrix");
    return LDA_OK;
}

int lda_word_counts_from_dense(lda_ctx* h, const int32_t* nwk_dev)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (!nwk_dev) return fail(&c, LDA_EINVAL, "null matrix");
    if (!c.inited) return fail(&c, LDA_ESTATE, "lda_word_counts_from_dense before lda_init");
    int rc = check_device(c);
    if (rc) return rc;
    launch_word_counts_from_dense(c, nwk_dev);
    c.tables_valid = false;
    int bits = 0;
    if ((rc = read_err(c, &bits))) { c.inited = false; return rc; }
    if (bits) {
        c.inited = false;
        return fail(&c, LDA_ERANGE,
                    "the matrix has negative entries or more nonzeros in a row than the term frequencies given to lda_set_shard allow");
    }
    return LDA_OK;
}

int lda_gibbs_sweep(lda_ctx* h, int32_t iters)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (iters < 0) return fail(&c, LDA_EINVAL, "iters must be >= 0");
    if (!c.inited) return fail(&c, LDA_ESTATE, "lda_gibbs_sweep before lda_init");
    if (c.K > GIBBS_MAX_K) return fail(&c, LDA_ERANGE, "the exact-conditional sweep takes K <= 16384");
    if ((long long)c.V * c.K * 8 > GIBBS_MAX_PREFIX_BYTES)
        return fail(&c, LDA_ERANGE, "the exact-conditional sweep keeps V*K running sums: V*K*8 bytes must stay below 24 GiB");
    if ((double)c.K * c.alpha >= 131072.0) return fail(&c, LDA_ERANGE, "the exact-conditional sweep needs K*alpha < 2^17");
    if (c.v.count_bits > 19) return fail(&c, LDA_ERANGE, "the exact-conditional sweep takes documents shorter than 2^19 tokens");
    int rc = check_device(c);
    if (rc) return rc;
    order_after_export(c);
    rc = gibbs_sweep(c, iters);
    if (rc) return fail(&c, rc, "the exact-conditional sweep failed");
    int bits = 0;
    if ((rc = read_err(c, &bits))) { c.inited = false; return rc; }
    if (bits) {
        c.inited = false;
        return fail(&c, LDA_EINTERNAL, "a kernel of the exact-conditional sweep raised the device error word");
    }
    return LDA_OK;
}

int lda_loglik(lda_ctx* h, double* total, double* word_ll, double* doc_ll)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (!c.inited) return fail(&c, LDA_ESTATE, "lda_loglik before lda_init");
    int rc = check_device(c);
    if (rc) return rc;
    double out[3];
    if (launch_loglik(c, out) < 0) return cuda_fail(&c, "log-likelihood");
    int bits = 0;
    if ((rc = read_err(c, &bits))) return rc;
    if (bits) return fail(&c, LDA_EINTERNAL, "the log-likelihood kernels raised the device error word");
    if (total) *total = out[0];
    if (word_ll) *word_ll = out[1];
    if (doc_ll) *doc_ll = out[2];
    return LDA_OK;
}

int lda_get_counts(lda_ctx* h, int which, int64_t* row_offsets, int32_t* topics, int32_t* counts,
                   int64_t capacity, int64_t* nnz_out)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (!c.inited) return fail(&c, LDA_ESTATE, "lda_get_counts before lda_init");
    int rc = check_device(c);
    if (rc) return rc;
    order_after_export(c);
    const View& v = c.v;
    cudaStreamSynchronize(c.stream);
    if (which == LDA_NK) {
        if (nnz_out) *nnz_out = c.K;
        if (counts) {
            if (capacity < c.K) return fail(&c, LDA_ERANGE, "capacity below K");
            if (cudaMemcpy(counts, v.nk, (size_t)c.K * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
                return cuda_fail(&c, "copying n_k");
        }
        return LDA_OK;
    }
    if (which == LDA_NDK) {
        // sorted rows are built on the device; only the row offsets and the nonzeros cross to the host
        const bool sizes_only = !row_offsets && !topics && !counts;
        DkCsr r;
        if ((rc = build_dk_csr(c, r, sizes_only))) return fail(&c, rc, "building the n_kd rows failed");
        int bits = 0;
        if ((rc = read_err(c, &bits))) { free_dk_csr(c, r); return rc; }
        if (bits) { free_dk_csr(c, r); return fail(&c, LDA_EINTERNAL, "the n_kd rows raised the device error word"); }
        const int64_t total = (int64_t)r.total;
        if (nnz_out) *nnz_out = total;
        if (sizes_only) { free_dk_csr(c, r); return LDA_OK; }
        if (capacity < total) { free_dk_csr(c, r); return fail(&c, LDA_ERANGE, "capacity below the number of nonzeros"); }
        static_assert(sizeof(long long) == sizeof(int64_t), "row offsets are copied as they are");
        bool ok = true;
        if (row_offsets) ok = ok && cudaMemcpy(row_offsets, r.row_off, ((size_t)c.D + 1) * 8, cudaMemcpyDeviceToHost) == cudaSuccess;
        if (topics && total) ok = ok && cudaMemcpy(topics, r.topic, (size_t)total * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
        if (counts && total) ok = ok && cudaMemcpy(counts, r.count, (size_t)total * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
        free_dk_csr(c, r);
        if (!ok) return cuda_fail(&c, "copying the n_kd rows");
        return LDA_OK;
    }
    if (which != LDA_NWK) return fail(&c, LDA_EINVAL, "unknown table");
    const int64_t rows = c.V;
    std::vector<int32_t> nnz((size_t)rows), start((size_t)rows + 1);
    if (cudaMemcpy(nnz.data(), v.wk_nnz, (size_t)rows * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
        return cuda_fail(&c, "copying row sizes");
    if (cudaMemcpy(start.data(), v.row_start, ((size_t)rows + 1) * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
        return cuda_fail(&c, "copying row starts");
    int64_t total = 0;
    for (int64_t r = 0; r < rows; ++r) total += nnz[(size_t)r];
    if (nnz_out) *nnz_out = total;
    if (!row_offsets && !topics && !counts) return LDA_OK;
    if (capacity < total) return fail(&c, LDA_ERANGE, "capacity below the number of nonzeros");
    const size_t cap = (size_t)start[(size_t)rows];
    std::vector<uint32_t> a(std::max<size_t>(cap, 1)), b(std::max<size_t>(cap, 1));
    if (cap && (cudaMemcpy(a.data(), v.wk_topic, cap * 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
                cudaMemcpy(b.data(), v.wk_count, cap * 4, cudaMemcpyDeviceToHost) != cudaSuccess))
        return cuda_fail(&c, "copying n_kw rows");
    int64_t o = 0;
    for (int64_t r = 0; r < rows; ++r) {
        if (row_offsets) row_offsets[r] = o;
        const size_t s0 = (size_t)start[(size_t)r];
        for (int32_t j = 0; j < nnz[(size_t)r]; ++j, ++o) {
            if (topics) topics[o] = (int32_t)a[s0 + j];
            if (counts) counts[o] = (int32_t)b[s0 + j];
        }
    }
    if (row_offsets) row_offsets[rows] = o;
    return LDA_OK;
}

static int get_assignments(lda_ctx* h, void* z_out, bool narrow, bool wait)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (!c.inited) return fail(&c, LDA_ESTATE, "lda_get_assignments before lda_init");
    if (narrow && c.wide_topics) return fail(&c, LDA_ERANGE, "16-bit assignments need K <= 65536");
    if (c.N > 0 && !z_out) return fail(&c, LDA_EINVAL, "null output");
    if (c.N == 0) return LDA_OK;
    int rc = check_device(c);
    if (rc) return rc;
    order_after_export(c);
    char* zdev = reinterpret_cast<char*>(c.v.rec);  // staging, see set_assignments()
    // chunk by chunk: collected into document order on the context's stream, copied out on the copy
    // stream while the next chunk is collected
    const size_t zt = narrow ? 2 : 4;
    for (int64_t first = 0; first < c.N; first += c.copy_chunk) {
        const int64_t count = std::min<int64_t>(c.copy_chunk, c.N - first);
        launch_export_chunk(c, zdev, narrow, first, count);
        cudaEventRecord(c.ev_chunk, c.stream);
        cudaStreamWaitEvent(c.copy, c.ev_chunk, 0);
        if (cudaMemcpyAsync(reinterpret_cast<char*>(z_out) + (size_t)first * zt, zdev + (size_t)first * zt,
                            (size_t)count * zt, cudaMemcpyDeviceToHost, c.copy) != cudaSuccess)
            return cuda_fail(&c, "copying assignments");
    }
    cudaEventRecord(c.ev_export, c.copy);
    c.export_pending = true;
    return wait ? wait_all(c) : LDA_OK;
}

int lda_get_assignments(lda_ctx* h, int32_t* z_out) { return get_assignments(h, z_out, false, true); }

int lda_get_assignments_u16(lda_ctx* h, uint16_t* z_out) { return get_assignments(h, z_out, true, true); }

int lda_get_assignments_async(lda_ctx* h, int32_t* z_out) { return get_assignments(h, z_out, false, false); }

int lda_get_assignments_u16_async(lda_ctx* h, uint16_t* z_out) { return get_assignments(h, z_out, true, false); }

int lda_wait(lda_ctx* h)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    int rc = check_device(c);
    if (rc) return rc;
    return wait_all(c);
}

int lda_get_tables(lda_ctx* h, uint32_t* sp_thr32, int32_t* sp_alias, int64_t capacity, uint32_t* mix32,
                   uint32_t* dn_thr32, int32_t* dn_alias, uint64_t* dense_mass)
{
    if (!h) return LDA_EINVAL;
    Ctx& c = h->c;
    if (!c.inited) return fail(&c, LDA_ESTATE, "lda_get_tables before lda_init");
    int rc = check_device(c);
    if (rc) return rc;
    const View& v = c.v;
    const size_t V = (size_t)c.V, K = (size_t)c.K;
    const bool want_sparse = sp_thr32 || sp_alias;
    std::vector<int32_t> nnz(V), start(V + 1);
    std::vector<uint32_t> a, b;
    if (want_sparse) {
        if (cudaMemcpy(nnz.data(), v.wk_nnz, V * 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
            cudaMemcpy(start.data(), v.row_start, (V + 1) * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
            return cuda_fail(&c, "copy");
        int64_t total = 0;
        for (size_t w = 0; w < V; ++w) total += nnz[w];
        if (capacity < total) return fail(&c, LDA_ERANGE, "capacity below the number of nonzeros");
        a.resize(std::max<size_t>((size_t)start[V], 1));
        b.resize(a.size());
    }
    // The device holds the sparse tables of one vocabulary slice at a time: build slice after slice
    // (one slice: the whole vocabulary, built once and kept until the counts change).
    const bool one = c.slices.size() == 1;
    if (one) {
        if ((rc = ensure_tables(c))) return rc;
    } else {
        c.tables_valid = false;
        launch_alias_dense(c);
    }
    for (size_t sl = 0; sl < c.slices.size(); ++sl) {
        const Ctx::Slice& q = c.slices[sl];
        if (!one) {
            set_slice(c, (int)sl);
            launch_alias_sparse(c);
            int bits = 0;
            if ((rc = read_err(c, &bits))) return rc;
            if (bits) return fail(&c, LDA_EINTERNAL, "alias construction raised the device error word");
        }
        if (want_sparse && q.row_n &&
            (cudaMemcpy(a.data() + q.row_lo, c.al_thr0, (size_t)q.row_n * 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
             cudaMemcpy(b.data() + q.row_lo, c.al_idx0, (size_t)q.row_n * 4, cudaMemcpyDeviceToHost) != cudaSuccess))
            return cuda_fail(&c, "copy");
    }
    if (mix32 && cudaMemcpy(mix32, v.mix32, V * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return cuda_fail(&c, "copy");
    if (dn_thr32 && cudaMemcpy(dn_thr32, v.dn_thr, K * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return cuda_fail(&c, "copy");
    if (dn_alias && cudaMemcpy(dn_alias, v.dn_idx, K * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return cuda_fail(&c, "copy");
    if (dense_mass && cudaMemcpy(dense_mass, v.dense_mass, 8, cudaMemcpyDeviceToHost) != cudaSuccess) return cuda_fail(&c, "copy");
    if (!want_sparse) return LDA_OK;
    int64_t o = 0;
    for (size_t w = 0; w < V; ++w)
        for (int32_t j = 0; j < nnz[w]; ++j, ++o) {
            if (sp_thr32) sp_thr32[o] = a[(size_t)start[w] + j];
            if (sp_alias) sp_alias[o] = (int32_t)b[(size_t)start[w] + j];
        }
    return LDA_OK;
}

int lda_get_stats(lda_ctx* h, lda_stats* out)
{
    if (!h || !out) return LDA_EINVAL;
    Ctx& c = h->c;
    if (c.inited) {
        if (check_device(c)) return LDA_ECUDA;
        int64_t a = 0, b = 0;
        launch_count_nnz(c, &a, &b);
        c.stats.nnz_wk = a;
        c.stats.nnz_dk = b;
    }
    c.stats.device_bytes = c.device_bytes;
    c.stats.sweeps_done = (int32_t)c.sweep;
    *out = c.stats;
    return LDA_OK;
}

}  // extern "C"
