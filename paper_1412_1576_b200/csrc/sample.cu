// Token Metropolis-Hastings step (Section 4.2-4.3) and the assignment initialisation / import /
// export kernels.
//
// Everything a token's chain reads is the sweep-start state (Section 6: the model is immutable
// while sampled) and a thread writes only its own output slots, so the result does not depend
// on scheduling.  Because the counts are frozen, a proposal never depends on the chain's current
// state.  The step is therefore split into passes that each stay on one side of the model:
//   1. word order : draw the word-proposals (alias bins of the word staged per tile);
//   2. doc order  : the document side -- own record, doc-proposals, n_kd at every proposed topic --
//                   from per-document tables built in shared memory (docside.cu);
//   3. word order : accept/reject chain in registers, n_kw rows staged in shared memory (hot
//                   words: the dense row, by one bulk asynchronous copy; tail words: the sorted rows
//                   of a tile of whole words);
// Pass 3 leaves the new assignments in word order (for the n_kw / n_k rebuild) and in block-major
// order, where the next document-side pass picks them up.
// A random access to HBM costs far more than the bytes it returns.  The passes exchange their
// results through buffers in block-major order (tokens sorted by block of documents, then by
// word-order position): the word-order passes reach them in runs of consecutive positions, the
// document-order pass within one L2-sized block at a time.
#include "lda_device.cuh"
#include "lda_internal.cuh"

namespace lda {

constexpr double INV_2_32 = 1.0 / 4294967296.0;
// launch shapes of the hot-word kernel: threads per CTA and CTAs per SM the compiler must allow
#ifndef LDA_PROPOSE_THREADS
#define LDA_PROPOSE_THREADS 512
#endif
#ifndef LDA_PROPOSE_MIN_CTAS
#define LDA_PROPOSE_MIN_CTAS 2
#endif
#ifndef LDA_PROPOSE_FIXED_MIN_CTAS
#define LDA_PROPOSE_FIXED_MIN_CTAS 4
#endif
#ifndef LDA_PROPOSE_TOKENS
#define LDA_PROPOSE_TOKENS 3
#endif
constexpr int PROPOSE_TOKENS = LDA_PROPOSE_TOKENS;  // tokens a thread of the two-step propose kernel takes per turn
#ifndef LDA_ACCEPT_FIXED2_THREADS
#define LDA_ACCEPT_FIXED2_THREADS 768
#endif
#ifndef LDA_ACCEPT_THREADS
#define LDA_ACCEPT_THREADS 512
#endif
#ifndef LDA_ACCEPT_MIN_CTAS
#define LDA_ACCEPT_MIN_CTAS 2
#endif
constexpr int PROPOSE_THREADS = LDA_PROPOSE_THREADS;
// the two-step chain needs few enough registers for two CTAs of 768 threads per SM
__host__ __device__ constexpr int accept_threads(int fixed)
{
    return fixed == 2 ? LDA_ACCEPT_FIXED2_THREADS : LDA_ACCEPT_THREADS;
}
constexpr int COLD_THREADS = 256;
constexpr int STAGE_WAIT_LIMIT = 1 << 20;

// --- shared-memory barrier and bulk-copy primitives ------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(void* bar, uint32_t arrivals)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(void* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}

// Global -> shared bulk copy; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, void* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// Waits for the barrier's phase `parity`; gives up after `limit` polls and returns false.
__device__ __forceinline__ bool mbar_wait_bounded(void* bar, uint32_t parity, int limit)
{
    uint32_t done = 0;
    for (int i = 0; i < limit && !done; ++i)
        asm volatile(
            "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
            : "=r"(done)
            : "r"(smem_addr(bar)), "r"(parity)
            : "memory");
    return done != 0;
}

// --- word side -------------------------------------------------------------------------------
// What a word-proposal draw keeps between issuing its table read and using the result.
struct Draw {
    uint2 e;      // the bin read from global memory (hot words; dense term of tail words)
    uint32_t b;   // bin index
    uint32_t rz;  // the alias coin
    bool sparse;  // sparse term (the word's own table) or dense smoothing term
};

// A hot word: dense n_kw row (in shared memory when STAGED), alias bins read from global memory.
template <bool STAGED, bool PACKED>
struct HotTile {
    struct Ref {};
    const int32_t* row;
    const int32_t* nk_tab;    // n_k: shared memory when STAGED, else global
    const uint2* pk;          // PACKED: the word's bins
    const uint32_t* thr;      // otherwise the three separate arrays
    const uint32_t* idx;
    const uint32_t* topic;
    int32_t nnz;
    uint32_t mix;
    void* bar;   // STAGED: barrier the bulk copy of the row completes on
    bool ready;  // the row has landed
    bool gave_up;  // STAGED: the wait for the copy ran out
    __device__ __forceinline__ Ref ref(int32_t) const { return Ref{}; }
    // Called before the first lookup: the row must have landed by then.  If the bounded wait runs
    // out, the error word is raised and false returned: the caller must not touch the staged rows
    // (it drops its remaining tokens; the host refuses to go on from a sweep that raised the word).
    __device__ __forceinline__ bool prepare(const View& v)
    {
        if (STAGED && !ready) {
            if (!mbar_wait_bounded(bar, 0, STAGE_WAIT_LIMIT)) {
                atomicOr(v.err, ERR_STAGE);
                gave_up = true;
                return false;
            }
            ready = true;
        }
        return true;
    }
    __device__ __forceinline__ int32_t count(const Ref&, uint32_t k) const
    {
        return STAGED ? row[k] : __ldg(row + k);
    }
    __device__ __forceinline__ int32_t nk(uint32_t k) const { return STAGED ? nk_tab[k] : __ldg(nk_tab + k); }
    __device__ __forceinline__ Draw draw_issue(const Ref&, const View& v, const uint4& r) const
    {
        Draw d;
        d.sparse = r.x < mix;
        d.rz = r.z;
        d.b = scale_to_range(r.y, d.sparse ? (uint32_t)nnz : (uint32_t)v.K);
        if (PACKED) {
            d.e = __ldg((d.sparse ? pk : v.dn_pk) + d.b);
        } else if (d.sparse) {
            const uint32_t al = __ldg(idx + d.b);
            const uint32_t item = (al == d.b || r.z < __ldg(thr + d.b)) ? d.b : al;
            d.e = make_uint2(0u, __ldg(topic + item));
        } else {
            d.e = __ldg(v.dn_pk + d.b);
        }
        return d;
    }
    __device__ __forceinline__ void draw_finish(const Ref&, const Draw& d, uint32_t& t, int32_t& n_tw) const
    {
        if (d.sparse) {
            if (PACKED) t = (d.rz < d.e.x) ? (d.e.y & 0xFFFFu) : (d.e.y >> 16);
            else t = d.e.y;
        } else {
            t = (d.e.y == d.b || d.rz < d.e.x) ? d.b : d.e.y;
        }
        n_tw = -1;  // looked up with the other counts
    }
};

// A tile of tail words: sorted n_kw rows and alias bins in shared memory.
struct ColdTile {
    struct Ref {
        int32_t rs, nnz;  // the word's row inside the tile's arrays
        uint32_t mix;
    };
    const int32_t* woff;  // [nw+1] first token of each word, relative to the tile
    const int32_t* rs;    // [nw+1] first row slot of each word, relative to the tile
    const int32_t* nnz;
    const uint32_t* mix;
    const uint32_t* topic;
    const uint32_t* cnt;
    const uint32_t* thr;
    const uint32_t* idx;
    int32_t nw;
    const int32_t* nk_tab;  // n_k in global memory
    static constexpr bool gave_up = false;
    __device__ __forceinline__ int32_t nk(uint32_t k) const { return __ldg(nk_tab + k); }
    __device__ __forceinline__ Ref ref(int32_t q) const
    {
        int32_t lo = 0, hi = nw;  // last word with woff[word] <= q
        while (hi - lo > 1) {
            const int32_t mid = (lo + hi) >> 1;
            if (woff[mid] <= q) lo = mid; else hi = mid;
        }
        return Ref{rs[lo], nnz[lo], mix[lo]};
    }
    __device__ __forceinline__ bool prepare(const View&) { return true; }
    __device__ __forceinline__ int32_t count(const Ref& w, uint32_t k) const
    {
        int32_t lo = 0, hi = w.nnz;
        while (lo < hi) {
            const int32_t mid = (lo + hi) >> 1;
            if (topic[w.rs + mid] < k) lo = mid + 1; else hi = mid;
        }
        return (lo < w.nnz && topic[w.rs + lo] == k) ? (int32_t)cnt[w.rs + lo] : 0;
    }
    __device__ __forceinline__ Draw draw_issue(const Ref& w, const View& v, const uint4& r) const
    {
        Draw d;
        d.sparse = r.x < w.mix;
        d.rz = r.z;
        d.b = scale_to_range(r.y, d.sparse ? (uint32_t)w.nnz : (uint32_t)v.K);
        d.e = make_uint2(0u, 0u);
        if (!d.sparse) d.e = __ldg(v.dn_pk + d.b);
        return d;
    }
    __device__ __forceinline__ void draw_finish(const Ref& w, const Draw& d, uint32_t& t, int32_t& n_tw) const
    {
        if (d.sparse) {
            const uint32_t al = idx[w.rs + d.b];
            const uint32_t item = (al == d.b || d.rz < thr[w.rs + d.b]) ? d.b : al;
            t = topic[w.rs + item];
            n_tw = (int32_t)cnt[w.rs + item];
        } else {
            t = (d.e.y == d.b || d.rz < d.e.x) ? d.b : d.e.y;
            n_tw = -1;
        }
    }
};

// A warm word: sorted n_kw row without a dense one, staged in shared memory and looked up by binary
// search inside one bucket of 2^shift consecutive topics: start[b] is the row position of bucket
// b's first entry (WARM_BUCKETS + 1 positions, the last one the row's end).
constexpr int WARM_BUCKETS = 1024;
struct WarmTile {
    struct Ref {};
    const uint32_t* topic;
    const uint32_t* cnt;
    const int32_t* nk_tab;  // n_k in global memory
    const uint32_t* start;
    int shift;
    static constexpr bool gave_up = false;
    __device__ __forceinline__ Ref ref(int32_t) const { return Ref{}; }
    __device__ __forceinline__ bool prepare(const View&) { return true; }
    __device__ __forceinline__ int32_t nk(uint32_t k) const { return __ldg(nk_tab + k); }
    __device__ __forceinline__ int32_t count(const Ref&, uint32_t k) const
    {
        int32_t lo = (int32_t)start[k >> shift];
        const int32_t end = (int32_t)start[(k >> shift) + 1];
        int32_t hi = end;
        while (lo < hi) {
            const int32_t mid = (lo + hi) >> 1;
            if (topic[mid] < k) lo = mid + 1; else hi = mid;
        }
        return (lo < end && topic[lo] == k) ? (int32_t)cnt[lo] : 0;
    }
};

// --- pass 1: word-proposals (word order) ---------------------------------------------------------
// Draws the topic proposed by every word-proposal step (Eq. 6; the even steps of the cycle) of the
// tile's tokens.
// A proposal depends on (token, sweep, step) and the frozen tables only, never on the chain's
// state, so all of them can be drawn before anything is accepted.
template <typename T, int MODE, int FIXED, class Tile>
__device__ __forceinline__ void propose_tokens(const View& v, const Tile& tile, const int32_t p_begin,
                                               const int32_t p_end, const int32_t nthreads, const uint2 key,
                                               const uint32_t sweep, const int32_t mh_steps)
{
    T* prop = reinterpret_cast<T*>(v.prop);
    if (FIXED == 2 && MODE == LDA_PROPOSALS_CYCLE) {
        // One word step per token: a thread takes PROPOSE_TOKENS tokens per turn, so that their
        // table reads (the pass waits for little else) are in flight together.
        constexpr int U = PROPOSE_TOKENS;
        for (int32_t p0 = p_begin + (int32_t)threadIdx.x; p0 < p_end; p0 += U * nthreads) {
            uint32_t tok[U], at[U], ua[U];
            Draw d[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int32_t p = p0 + u * nthreads;
                const bool live = p < p_end;
                tok[u] = live ? v.tok_base + __ldcs(v.tok_orig + p) : 0u;
                at[u] = live ? __ldcs(v.inv + p) : 0u;
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int32_t p = p0 + u * nthreads;
                const uint4 r = philox4x32_10(make_uint4(tok[u], sweep, 0u, 0u), key);
                ua[u] = r.w;
                d[u] = tile.draw_issue(tile.ref((p < p_end ? p : p0) - p_begin), v, r);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int32_t p = p0 + u * nthreads;
                uint32_t t;
                int32_t n_tw;
                tile.draw_finish(tile.ref((p < p_end ? p : p0) - p_begin), d[u], t, n_tw);
                if (p < p_end) {
                    __stcs(reinterpret_cast<T*>(v.zbm) + 2 * (size_t)at[u] + 1, (T)t);
                    __stcs(v.ua_w + p, ua[u]);
                }
            }
        }
    } else {
        for (int32_t p = p_begin + (int32_t)threadIdx.x; p < p_end; p += nthreads) {
            const uint32_t tok = v.tok_base + __ldcs(v.tok_orig + p);
            const uint32_t at = __ldcs(v.inv + p);  // the document-side pass reads block-major
            const typename Tile::Ref w = tile.ref(p - p_begin);
            for (int32_t m = 0; m < mh_steps; m += (MODE == LDA_PROPOSALS_CYCLE ? 2 : 1)) {
                const int32_t wi = step_kind_index<MODE>(m);
                const uint4 r = philox4x32_10(make_uint4(tok, sweep, (uint32_t)m, 0u), key);
                const Draw d = tile.draw_issue(w, v, r);
                uint32_t t;
                int32_t n_tw;
                tile.draw_finish(w, d, t, n_tw);
                // the first proposal goes beside the token's topic, the later ones to arrays of their own
                if (wi == 0) __stcs(reinterpret_cast<T*>(v.zbm) + 2 * (size_t)at + 1, (T)t);
                else __stcs(prop + (size_t)wi * v.N + at, (T)t);
                __stcs(v.ua_w + (size_t)wi * v.N + p, r.w);  // the step's acceptance uniform, for pass 3
            }
        }
    }
}

// The new topic goes out together with the other half of its pair (the word-proposal of this step,
// which nobody reads any more; pass 1 of the next step overwrites it): a whole word per token, so
// that the runs the tile writes fill their sectors and L2 has nothing to merge them with.
__device__ __forceinline__ void store_topic_pair(uint16_t* zbm, uint32_t at, uint32_t s)
{
    __stcs(reinterpret_cast<uint32_t*>(zbm) + at, s);
}
__device__ __forceinline__ void store_topic_pair(int32_t* zbm, uint32_t at, uint32_t s)
{
    __stcs(reinterpret_cast<uint2*>(zbm) + at, make_uint2(s, 0u));
}

// --- pass 3: accept / reject (word order) -----------------------------------------------------------
// Runs the chain of every token of the tile: everything the document side contributes was
// gathered by pass 2, the word side comes from the tile's staged rows.
template <typename T, int CH, int MODE, int FIXED, class Tile>
__device__ __forceinline__ void accept_tokens(const View& v, Tile& tile, const int32_t p_begin, const int32_t p_end,
                                              const int32_t nthreads, const uint2 key, const uint32_t sweep,
                                              const int32_t mh_steps)
{
    const int cb = v.count_bits;
    const uint32_t cmask = (1u << cb) - 1u;
    const double alpha = v.alpha, beta = v.beta, Vb = v.Vbeta;
    static_assert(CH % 2 == 0, "in the cycle a group of steps starts on a word-proposal");
    const size_t N = (size_t)v.N;
    T* zw = reinterpret_cast<T*>(v.zw);
    bool bad = false;
    // steps of this thread's tokens that moved the chain: word-proposals in the low half, doc-proposals
    // in the high half (a thread takes fewer than 65536 steps of either kind: lda_sweep bounds mh_steps)
    uint32_t moved = 0;
    bool staged_ok = true;
    // The reads of a token are issued ahead of its turn: its block-major index two iterations
    // early, the gathered record (which needs that index) one iteration early.
    const uint4* side4 = reinterpret_cast<const uint4*>(v.dside);
    const int32_t quads = v.side_stride >> 2;
    // with the step count fixed at compile time a record of more than four words is read ahead whole
    constexpr bool TWO = FIXED > 0 && step_record_words<MODE>(FIXED) > 4;
    static_assert(FIXED == 0 || step_record_words<MODE>(FIXED) <= 8, "the record is read as two 16-byte words");
    int32_t p = p_begin + (int32_t)threadIdx.x;
    uint32_t at_c = 0, at_n = 0;
    uint4 rec_c = make_uint4(0u, 0u, 0u, 0u), rec2_c = make_uint4(0u, 0u, 0u, 0u);
    if (p < p_end) at_c = __ldcs(v.inv + p);
    if (p + nthreads < p_end) at_n = __ldcs(v.inv + p + nthreads);
    if (p < p_end) {
        rec_c = __ldcs(side4 + (size_t)at_c * quads);
        if (TWO) rec2_c = __ldcs(side4 + (size_t)at_c * quads + 1);
    }
    for (; p < p_end; p += nthreads) {
        const uint32_t at = at_c;
        const uint4 rec = rec_c, rec2 = rec2_c;  // own record, then the words pass 2 gathered
        at_c = at_n;
        if (p + nthreads < p_end) {
            rec_c = __ldcs(side4 + (size_t)at_c * quads);
            if (TWO) rec2_c = __ldcs(side4 + (size_t)at_c * quads + 1);
        }
        if (p + 2 * nthreads < p_end) at_n = __ldcs(v.inv + p + 2 * nthreads);
        const uint32_t* side = v.dside + (size_t)at * v.side_stride;
        auto side_word = [&](int32_t i) {
            if (TWO && i >= 4) return i == 4 ? rec2.x : i == 5 ? rec2.y : i == 6 ? rec2.z : rec2.w;
            return i == 1 ? rec.y : i == 2 ? rec.z : i == 3 ? rec.w : __ldcs(side + i);
        };
        const uint32_t own = rec.x;
        const typename Tile::Ref w = tile.ref(p - p_begin);
        uint32_t z0 = 0, s = 0;
        int32_t n_sd = 0, n_sw = 0, n_s = 0;
        for (int32_t m0 = 0; m0 < mh_steps; m0 += CH) {
            uint32_t e[CH], ua[CH];
#pragma unroll
            for (int i = 0; i < CH; ++i) {
                e[i] = 0;
                ua[i] = 0;
                if (m0 + i < mh_steps) {
                    e[i] = side_word(1 + m0 + i);
                    // acceptance uniform: word 3 of the step's Philox block, drawn by the pass that made
                    // the proposal (pass 1: word steps, pass 2: doc steps) and left for this one
                    ua[i] = step_is_doc<MODE>(i) ? side_word(1 + mh_steps + step_kind_index<MODE>(m0 + i))
                                                 : __ldcs(v.ua_w + (size_t)step_kind_index<MODE>(m0 + i) * N + p);
                }
            }
            if (m0 == 0) {
                // counts at the start state s = z0, where all three are >= 1
                staged_ok = tile.prepare(v);
                if (!staged_ok) break;
                z0 = s = own >> cb;
                n_sd = (int32_t)(own & cmask);
                n_sw = tile.count(w, z0);
                n_s = tile.nk(z0);
                bad = bad || n_sd < 1 || n_sw < 1 || n_s < 1;
            }
            // counts at the proposed topics, all read before the first acceptance test
            uint32_t t[CH];
            int32_t n_tw[CH], n_t[CH];
#pragma unroll
            for (int i = 0; i < CH; ++i) {
                t[i] = e[i] >> cb;
                n_tw[i] = tile.count(w, t[i]);
                n_t[i] = tile.nk(t[i]);
            }
            // Eq. 8 (word steps) / Eq. 11 (doc steps), products taken left to right
#pragma unroll
            for (int i = 0; i < CH; ++i) {
                const bool live = m0 + i < mh_steps && t[i] != s;
                const int32_t n_td = (int32_t)(e[i] & cmask);
                const int32_t e_s = (s == z0), e_t = (t[i] == z0);
                double num = __dadd_rn(u32_to_double((uint32_t)(n_td - e_t)), alpha);
                num = __dmul_rn(num, __dadd_rn(u32_to_double((uint32_t)(n_tw[i] - e_t)), beta));
                num = __dmul_rn(num, __dadd_rn(u32_to_double((uint32_t)(n_s - e_s)), Vb));
                double den = __dadd_rn(u32_to_double((uint32_t)(n_sd - e_s)), alpha);
                den = __dmul_rn(den, __dadd_rn(u32_to_double((uint32_t)(n_sw - e_s)), beta));
                den = __dmul_rn(den, __dadd_rn(u32_to_double((uint32_t)(n_t[i] - e_t)), Vb));
                if (!step_is_doc<MODE>(i)) {
                    num = __dmul_rn(num, __dadd_rn(u32_to_double((uint32_t)n_sw), beta));
                    num = __dmul_rn(num, __dadd_rn(u32_to_double((uint32_t)n_t[i]), Vb));
                    den = __dmul_rn(den, __dadd_rn(u32_to_double((uint32_t)n_tw[i]), beta));
                    den = __dmul_rn(den, __dadd_rn(u32_to_double((uint32_t)n_s), Vb));
                } else {
                    num = __dmul_rn(num, __dadd_rn(u32_to_double((uint32_t)n_sd), alpha));
                    den = __dmul_rn(den, __dadd_rn(u32_to_double((uint32_t)n_td), alpha));
                }
                const double u = __dmul_rn(u32_to_double((uint32_t)ua[i]), INV_2_32);
                if (live && __dmul_rn(u, den) < num) {
                    moved += step_is_doc<MODE>(i) ? 0x10000u : 1u;
                    s = t[i];
                    n_sd = n_td;
                    n_sw = n_tw[i];
                    n_s = n_t[i];
                }
            }
        }
        if (!staged_ok) break;
        __stcs(zw + p, (T)s);
        store_topic_pair(reinterpret_cast<T*>(v.zbm), at, s);
    }
    if (bad) atomicOr(v.err, ERR_COUNT_ZERO);
    // one add per CTA and kind to the sweep's counters
    __shared__ uint32_t moved_s[2];
    if (threadIdx.x == 0) moved_s[0] = moved_s[1] = 0u;
    __syncthreads();
    const uint32_t moved_w = warp_reduce_sum<uint32_t>(moved & 0xFFFFu);
    const uint32_t moved_d = warp_reduce_sum<uint32_t>(moved >> 16);
    if ((threadIdx.x & 31) == 0) {
        if (moved_w) atomicAdd(&moved_s[0], moved_w);
        if (moved_d) atomicAdd(&moved_s[1], moved_d);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (moved_s[0]) atomicAdd(v.moves + 0, (unsigned long long)moved_s[0]);
        if (moved_s[1]) atomicAdd(v.moves + 1, (unsigned long long)moved_s[1]);
    }
}

// Hot words: tile = (word, first token, count).  ACCEPT = false: pass 1, true: pass 3.
// FIXED > 0: the number of steps is this compile-time constant (the argument is ignored), which
// removes the step loops and their predicates (and, in pass 1, enough registers for a third CTA per SM).
template <typename T, int CH, bool STAGED, bool ACCEPT, int MODE, int FIXED>
__global__ void __launch_bounds__(ACCEPT ? accept_threads(FIXED) : PROPOSE_THREADS,
                                  ACCEPT      ? LDA_ACCEPT_MIN_CTAS
                                  : FIXED > 0 ? LDA_PROPOSE_FIXED_MIN_CTAS
                                              : LDA_PROPOSE_MIN_CTAS)
k_word_hot(View v, const int32_t* __restrict__ tiles, uint2 key, uint32_t sweep, int32_t mh_steps_arg)
{
    const int32_t mh_steps = FIXED > 0 ? FIXED : mh_steps_arg;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ __align__(8) unsigned long long bar;
    constexpr bool PACKED = sizeof(T) == 2;
    const int32_t w = tiles[3 * blockIdx.x], p0 = tiles[3 * blockIdx.x + 1], cnt = tiles[3 * blockIdx.x + 2];
    const int32_t* row_g = v.dense_rows + (size_t)__ldg(v.dense_slot + w) * v.dense_stride;
    int32_t* row_s = reinterpret_cast<int32_t*>(dyn_smem);
    int32_t* nk_s = row_s + v.dense_stride;
    if (STAGED && ACCEPT) {
        if (threadIdx.x == 0) {
            // the word's dense n_kw row and n_k, one bulk copy each, both signalling the same barrier
            const uint32_t bytes = (uint32_t)v.dense_stride * 4u;
            mbar_init(&bar, 1);
            mbar_expect_tx(&bar, 2u * bytes);
            bulk_copy_g2s(row_s, row_g, bytes, &bar);
            bulk_copy_g2s(nk_s, v.nk, bytes, &bar);
        }
        __syncthreads();
    }
    const int32_t r0 = __ldg(v.row_start + w);
    HotTile<STAGED && ACCEPT, PACKED> tile;
    tile.row = (STAGED && ACCEPT) ? row_s : row_g;
    tile.nk_tab = (STAGED && ACCEPT) ? nk_s : v.nk;
    tile.pk = v.al_pk + r0;
    tile.thr = v.al_thr + r0;
    tile.idx = v.al_idx + r0;
    tile.topic = v.wk_topic + r0;
    tile.nnz = __ldg(v.wk_nnz + w);
    tile.mix = __ldg(v.mix32 + w);
    tile.bar = &bar;
    tile.ready = !(STAGED && ACCEPT);
    tile.gave_up = false;
    if (ACCEPT) accept_tokens<T, CH, MODE, FIXED>(v, tile, p0, p0 + cnt, accept_threads(FIXED), key, sweep, mh_steps);
    else propose_tokens<T, MODE, FIXED>(v, tile, p0, p0 + cnt, PROPOSE_THREADS, key, sweep, mh_steps);
    // ACCEPT: every thread that had a token waited for the copy; thread 0 always has one.  A thread
    // whose wait ran out waits once more (bounded again) before the CTA may retire: a bulk copy still
    // in flight must not land in shared memory that belongs to the next CTA.
    if (STAGED && ACCEPT && tile.gave_up) mbar_wait_bounded(&bar, 0, STAGE_WAIT_LIMIT);
}

// Warm words, accept pass: tile = (word, first token, count) like a hot word's, the sorted row
// instead of a dense one.
template <typename T, int CH, int MODE, int FIXED>
__global__ void __launch_bounds__(accept_threads(FIXED), LDA_ACCEPT_MIN_CTAS)
k_word_warm(View v, const int32_t* __restrict__ tiles, uint2 key, uint32_t sweep, int32_t mh_steps_arg)
{
    const int32_t mh_steps = FIXED > 0 ? FIXED : mh_steps_arg;
    extern __shared__ __align__(16) uint32_t warm_smem[];  // [2 * WARM_MAX_TF] topics, counts
    __shared__ uint32_t start_s[WARM_BUCKETS + 1];
    const int32_t w = tiles[3 * blockIdx.x], p0 = tiles[3 * blockIdx.x + 1], cnt = tiles[3 * blockIdx.x + 2];
    const int32_t r0 = __ldg(v.row_start + w);
    const int32_t nnz = min(__ldg(v.wk_nnz + w), WARM_MAX_TF);  // never more entries than tokens
    uint32_t* topic_s = warm_smem;
    uint32_t* count_s = warm_smem + WARM_MAX_TF;
    for (int32_t j = threadIdx.x; j < nnz; j += blockDim.x) {
        topic_s[j] = __ldg(v.wk_topic + r0 + j);
        count_s[j] = __ldg(v.wk_count + r0 + j);
    }
    __syncthreads();
    int shift = 0;
    while (((v.K - 1) >> shift) >= WARM_BUCKETS) ++shift;
    for (int32_t b = threadIdx.x; b <= WARM_BUCKETS; b += blockDim.x) {
        const uint32_t k = (uint32_t)b << shift;
        int32_t lo = 0, hi = nnz;
        while (lo < hi) {
            const int32_t mid = (lo + hi) >> 1;
            if (topic_s[mid] < k) lo = mid + 1; else hi = mid;
        }
        start_s[b] = (uint32_t)lo;
    }
    __syncthreads();
    WarmTile tile{topic_s, count_s, v.nk, start_s, shift};
    accept_tokens<T, CH, MODE, FIXED>(v, tile, p0, p0 + cnt, accept_threads(FIXED), key, sweep, mh_steps);
}

// Tail words: tile = range of whole words [w0, w1) with at most COLD_TILE tokens.
template <typename T, int CH, bool ACCEPT, int MODE, int FIXED>
__global__ void __launch_bounds__(COLD_THREADS)
k_word_cold(View v, const int32_t* __restrict__ tiles, uint2 key, uint32_t sweep, int32_t mh_steps_arg)
{
    const int32_t mh_steps = FIXED > 0 ? FIXED : mh_steps_arg;
    __shared__ int32_t woff_s[COLD_WORDS + 1];  // first token of each word, relative to the tile
    __shared__ int32_t rs_s[COLD_WORDS + 1];    // first row slot of each word, relative to the tile
    __shared__ int32_t nnz_s[COLD_WORDS];
    __shared__ uint32_t mix_s[COLD_WORDS];
    __shared__ uint32_t topic_s[COLD_TILE], count_s[COLD_TILE], thr_s[COLD_TILE], idx_s[COLD_TILE];
    const int tid = threadIdx.x;
    const int32_t w0 = tiles[2 * blockIdx.x], w1 = tiles[2 * blockIdx.x + 1];
    const int32_t nw = w1 - w0;
    const int32_t p0 = __ldg(v.word_off + w0), cnt = __ldg(v.word_off + w1) - p0;
    const int32_t e0 = __ldg(v.row_start + w0), ne = __ldg(v.row_start + w1) - e0;
    if (cnt == 0) return;
    for (int j = tid; j <= nw; j += COLD_THREADS) {
        woff_s[j] = __ldg(v.word_off + w0 + j) - p0;
        rs_s[j] = __ldg(v.row_start + w0 + j) - e0;
    }
    for (int j = tid; j < nw; j += COLD_THREADS) {
        nnz_s[j] = __ldg(v.wk_nnz + w0 + j);
        mix_s[j] = __ldg(v.mix32 + w0 + j);
    }
    for (int j = tid; j < ne; j += COLD_THREADS) {
        topic_s[j] = __ldcs(v.wk_topic + e0 + j);
        if (ACCEPT) {
            count_s[j] = __ldcs(v.wk_count + e0 + j);
        } else {
            thr_s[j] = __ldcs(v.al_thr + e0 + j);
            idx_s[j] = __ldcs(v.al_idx + e0 + j);
        }
    }
    __syncthreads();
    ColdTile tile{woff_s, rs_s, nnz_s, mix_s, topic_s, count_s, thr_s, idx_s, nw, v.nk};
    if (ACCEPT) accept_tokens<T, CH, MODE, FIXED>(v, tile, p0, p0 + cnt, COLD_THREADS, key, sweep, mh_steps);
    else propose_tokens<T, MODE, FIXED>(v, tile, p0, p0 + cnt, COLD_THREADS, key, sweep, mh_steps);
}

// z_i uniform on {0..K-1}: Philox counter (token, 0, 0, 1), word 0.
template <typename T>
__global__ void k_init(View v, uint2 key)
{
    T* zw = reinterpret_cast<T*>(v.zw);
    T* zbm = reinterpret_cast<T*>(v.zbm);
    for (int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; p < v.N;
         p += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t tok = v.tok_base + v.tok_orig[p];
        const uint4 r = philox4x32_10(make_uint4(tok, 0u, 0u, 1u), key);
        const T z = (T)scale_to_range(r.x, (uint32_t)v.K);
        zw[p] = z;
        zbm[2 * (size_t)v.inv[p]] = z;
    }
}

// Import of assignments given in the caller's document order (IN = int32_t or uint16_t), in two
// steps that each stay coalesced on one side: document order -> block-major order (the scattered
// writes stay inside one block of that order at a time), then block-major -> word order.
template <typename T, typename IN>
__global__ void k_spread(View v, const IN* __restrict__ z_in, int64_t first, int64_t count)
{
    // one token per thread, CTAs in document order: the scattered writes of the CTAs in flight stay
    // inside one block of the block-major order (a grid-stride loop would let them drift apart)
    T* zbm = reinterpret_cast<T*>(v.zbm);
    const int64_t i = first + blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i >= first + count) return;
    int64_t a = (int64_t)z_in[i];
    if (a < 0 || a >= v.K) {
        atomicOr(v.err, ERR_TOPIC_RANGE);
        a = 0;
    }
    store_topic_pair(zbm, __ldcs(v.bm_of_tok + i), (uint32_t)a);  // the proposal half means nothing between sweeps
}

template <typename T>
__global__ void k_word_order_topics(View v)
{
    T* zw = reinterpret_cast<T*>(v.zw);
    const T* zbm = reinterpret_cast<const T*>(v.zbm);
    for (int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; p < v.N;
         p += (int64_t)gridDim.x * blockDim.x)
        zw[p] = zbm[2 * (size_t)__ldcs(v.inv + p)];
}

template <typename T, typename OUT>
__global__ void k_export(View v, OUT* __restrict__ out, int64_t first, int64_t count)
{
    // one token per thread, CTAs in document order (see k_spread)
    const T* zbm = reinterpret_cast<const T*>(v.zbm);
    const int64_t i = first + blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i < first + count) out[i] = (OUT)zbm[2 * (size_t)__ldcs(v.bm_of_tok + i)];
}

static int grid_for(int64_t n, int block)
{
    int64_t g = (n + block - 1) / block;
    if (g > 148 * 16) g = 148 * 16;
    return g < 1 ? 1 : (int)g;
}

template <typename T, int CH, int MODE, int FIXED>
static int launch_accept(Ctx& c, uint2 key, int mh_steps)
{
    const View& v = c.v;
    int launches = 0;
    if (c.n_hot_tiles) {
        if (c.K <= HOT_STAGE_MAX_K)
            k_word_hot<T, CH, true, true, MODE, FIXED>
                <<<c.n_hot_tiles, accept_threads(FIXED), (size_t)v.dense_stride * 8, c.stream>>>(v, c.hot_tiles, key, c.sweep,
                                                                                          mh_steps);
        else
            k_word_hot<T, CH, false, true, MODE, FIXED>
                <<<c.n_hot_tiles, accept_threads(FIXED), 0, c.stream>>>(v, c.hot_tiles, key, c.sweep, mh_steps);
        ++launches;
    }
    if (c.n_hot_tiles_warm) {
        k_word_warm<T, CH, MODE, FIXED><<<c.n_hot_tiles_warm, accept_threads(FIXED), WARM_MAX_TF * 8, c.stream>>>(
            v, c.hot_tiles_warm, key, c.sweep, mh_steps);
        ++launches;
    }
    if (c.n_cold_tiles) {
        k_word_cold<T, CH, true, MODE, FIXED><<<c.n_cold_tiles, COLD_THREADS, 0, c.stream>>>(v, c.cold_tiles, key,
                                                                                           c.sweep, mh_steps);
        ++launches;
    }
    return launches;
}

template <typename T, int CH, int MODE, int FIXED>
static int launch_propose(Ctx& c, uint2 key, int mh_steps)
{
    // the running vocabulary slice's tokens (its tables are the ones in memory)
    const View& v = c.v;
    const Ctx::Slice& q = c.slices[(size_t)c.cur_slice];
    int launches = 0;
    if (q.hotp_n) {
        k_word_hot<T, CH, false, false, MODE, FIXED><<<q.hotp_n, PROPOSE_THREADS, 0, c.stream>>>(
            v, c.hot_tiles_propose + 3 * (size_t)q.hotp_lo, key, c.sweep, mh_steps);
        ++launches;
    }
    if (q.cold_n) {
        k_word_cold<T, CH, false, MODE, FIXED><<<q.cold_n, COLD_THREADS, 0, c.stream>>>(
            v, c.cold_tiles + 2 * (size_t)q.cold_lo, key, c.sweep, mh_steps);
        ++launches;
    }
    return launches;
}

template <typename T, int CH, int MODE>
static int sample_tc(Ctx& c, int mh_steps)
{
    const uint2 key = make_uint2((uint32_t)c.seed, (uint32_t)(c.seed >> 32));
    int launches = 0;
    // pass 1: word-proposals (none in a doc-proposal-only chain).  With more than one vocabulary
    // slice the sparse alias tables exist for one slice at a time: build a slice's, draw from them,
    // go on to the next (one slice: the caller has built them already).
    if (MODE != LDA_PROPOSALS_DOC) {
        const int n_slices = (int)c.slices.size();
        for (int sl = 0; sl < n_slices; ++sl) {
            if (n_slices > 1) {
                set_slice(c, sl);
                launches += launch_alias_sparse(c);
            }
            if (CH == 2 && mh_steps == 2)
                launches += launch_propose<T, 2, MODE, 2>(c, key, mh_steps);
            else
                launches += launch_propose<T, CH, MODE, 0>(c, key, mh_steps);
        }
    }
    // pass 2: document side
    cudaEventRecord(c.ev[8], c.stream);
    launches += launch_doc_side(c, mh_steps);
    // pass 3: accept / reject; chains of two steps (and the cycle with four) have kernels of their own
    cudaEventRecord(c.ev[9], c.stream);
    if (CH == 2 && mh_steps == 2)
        launches += launch_accept<T, 2, MODE, 2>(c, key, mh_steps);
    else if (CH == 4 && MODE == LDA_PROPOSALS_CYCLE && mh_steps == 4)
        launches += launch_accept<T, 4, LDA_PROPOSALS_CYCLE, 4>(c, key, mh_steps);
    else
        launches += launch_accept<T, CH, MODE, 0>(c, key, mh_steps);
    return launches;
}

// The accept/reject pass handles proposals in groups of two (mh_steps <= 2) or four.
template <typename T>
static int sample_t(Ctx& c, int mh_steps)
{
    switch (c.proposals) {
        case LDA_PROPOSALS_WORD:
            return mh_steps <= 2 ? sample_tc<T, 2, LDA_PROPOSALS_WORD>(c, mh_steps)
                                 : sample_tc<T, 4, LDA_PROPOSALS_WORD>(c, mh_steps);
        case LDA_PROPOSALS_DOC:
            return mh_steps <= 2 ? sample_tc<T, 2, LDA_PROPOSALS_DOC>(c, mh_steps)
                                 : sample_tc<T, 4, LDA_PROPOSALS_DOC>(c, mh_steps);
        default:
            return mh_steps <= 2 ? sample_tc<T, 2, LDA_PROPOSALS_CYCLE>(c, mh_steps)
                                 : sample_tc<T, 4, LDA_PROPOSALS_CYCLE>(c, mh_steps);
    }
}

// Reads the records and tables of the sweep-start state; writes zw and zbm.
int launch_sample(Ctx& c, int mh_steps)
{
    if (c.N == 0) return 0;
    return c.wide_topics ? sample_t<int32_t>(c, mh_steps) : sample_t<uint16_t>(c, mh_steps);
}

template <typename T, int CH, int MODE, int FIXED>
static void set_hot_limit_one()
{
    cudaFuncSetAttribute(k_word_hot<T, CH, true, true, MODE, FIXED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         HOT_STAGE_MAX_K * 8);
    cudaFuncSetAttribute(k_word_warm<T, CH, MODE, FIXED>, cudaFuncAttributeMaxDynamicSharedMemorySize, WARM_MAX_TF * 8);
}

template <typename T, int CH>
static void set_hot_limit()
{
    set_hot_limit_one<T, CH, LDA_PROPOSALS_CYCLE, 0>();
    set_hot_limit_one<T, CH, LDA_PROPOSALS_WORD, 0>();
    set_hot_limit_one<T, CH, LDA_PROPOSALS_DOC, 0>();
    if (CH == 2) {
        set_hot_limit_one<T, 2, LDA_PROPOSALS_CYCLE, 2>();
        set_hot_limit_one<T, 2, LDA_PROPOSALS_WORD, 2>();
        set_hot_limit_one<T, 2, LDA_PROPOSALS_DOC, 2>();
    }
    if (CH == 4) set_hot_limit_one<T, 4, LDA_PROPOSALS_CYCLE, 4>();
}

void set_sample_smem_limits()
{
    set_hot_limit<uint16_t, 2>();
    set_hot_limit<uint16_t, 4>();
    set_hot_limit<int32_t, 2>();
    set_hot_limit<int32_t, 4>();
}

int launch_init(Ctx& c)
{
    if (c.N == 0) return 0;
    const uint2 key = make_uint2((uint32_t)c.seed, (uint32_t)(c.seed >> 32));
    const int g = grid_for(c.N, 256);
    if (c.wide_topics) k_init<int32_t><<<g, 256, 0, c.stream>>>(c.v, key);
    else k_init<uint16_t><<<g, 256, 0, c.stream>>>(c.v, key);
    return 1;
}

// `narrow`: the caller's array holds 16-bit topics (only with 16-bit topic storage), else int32.
int launch_spread_chunk(Ctx& c, const void* z_dev, bool narrow, int64_t first, int64_t count)
{
    if (count <= 0) return 0;
    const unsigned full = (unsigned)((count + 255) / 256);  // one token per thread
    if (c.wide_topics) k_spread<int32_t, int32_t><<<full, 256, 0, c.stream>>>(c.v, (const int32_t*)z_dev, first, count);
    else if (narrow) k_spread<uint16_t, uint16_t><<<full, 256, 0, c.stream>>>(c.v, (const uint16_t*)z_dev, first, count);
    else k_spread<uint16_t, int32_t><<<full, 256, 0, c.stream>>>(c.v, (const int32_t*)z_dev, first, count);
    return 1;
}

int launch_word_order_topics(Ctx& c)
{
    if (c.N == 0) return 0;
    const int g = grid_for(c.N, 256);
    if (c.wide_topics) k_word_order_topics<int32_t><<<g, 256, 0, c.stream>>>(c.v);
    else k_word_order_topics<uint16_t><<<g, 256, 0, c.stream>>>(c.v);
    return 1;
}

int launch_spread_assignments(Ctx& c, const void* z_dev, bool narrow)
{
    if (c.N == 0) return 0;
    return launch_spread_chunk(c, z_dev, narrow, 0, c.N) + launch_word_order_topics(c);
}

int launch_export_chunk(Ctx& c, void* z_dev, bool narrow, int64_t first, int64_t count)
{
    if (count <= 0) return 0;
    const unsigned full = (unsigned)((count + 255) / 256);  // one token per thread
    if (c.wide_topics) k_export<int32_t, int32_t><<<full, 256, 0, c.stream>>>(c.v, (int32_t*)z_dev, first, count);
    else if (narrow) k_export<uint16_t, uint16_t><<<full, 256, 0, c.stream>>>(c.v, (uint16_t*)z_dev, first, count);
    else k_export<uint16_t, int32_t><<<full, 256, 0, c.stream>>>(c.v, (int32_t*)z_dev, first, count);
    return 1;
}

int launch_export_assignments(Ctx& c, void* z_dev, bool narrow)
{
    return launch_export_chunk(c, z_dev, narrow, 0, c.N);
}

}  // namespace lda
