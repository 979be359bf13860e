// Document side of the MH step (pass 2), one tile of whole documents per CTA.
//
// The sweep-start n_kd of a document (Eq. 12) is a function of that document's assignments
// alone, so the tile's tables are built where they are used: in shared memory, by insertion
// (Section 5's hashed rows: claim a slot with compare-and-swap, then add one to its count), and
// thrown away afterwards.  Every token then gathers what the accept/reject pass needs from this
// side:
//   - the token's own (topic, n_kd) record,
//   - for every word-proposal (drawn by pass 1): n_kd at the proposed topic,
//   - for every doc-proposal (Eq. 9, Eq. 12): the Philox block of the step, the proposed topic
//     -- the topic of a random token of the document, or a uniform topic with probability
//     K*alpha / (n_d + K*alpha) -- its n_kd, and the step's acceptance uniform.
// The current assignments and the word-proposals arrive in block-major order and the results go
// back in block-major order: a tile's documents lie in one block of that order (two at a block
// border), so these scattered reads and writes stay in L2.
#include "lda_device.cuh"
#include "lda_internal.cuh"

namespace lda {

constexpr double INV_2_32 = 1.0 / 4294967296.0;
// slots per token of the tables a tile builds in shared memory (DOC_TILE_SLOTS, a multiple of 4)
constexpr int TILE_SLOTS = DOC_TILE_SLOTS;

// A token's current topic and its first word-proposal sit side by side at its block-major index:
// one read brings both.
__device__ __forceinline__ void load_topic_pair(const uint16_t* zbm, uint32_t bm, uint32_t& z, uint32_t& t1)
{
    const uint32_t w = __ldcg(reinterpret_cast<const uint32_t*>(zbm) + bm);
    z = w & 0xFFFFu;
    t1 = w >> 16;
}
__device__ __forceinline__ void load_topic_pair(const int32_t* zbm, uint32_t bm, uint32_t& z, uint32_t& t1)
{
    const uint2 w = __ldcg(reinterpret_cast<const uint2*>(zbm) + bm);
    z = w.x;
    t1 = w.y;
}

// Everything pass 3 needs from the document side for one token, written at the token's
// block-major index `bm`.
//   tab     : the document's table, 4 * doc_len slots
//   slot_at : slot holding the topic of the document's j-th token
template <typename T, int MODE, int FIXED, int SLOTS, class SlotAt>
__device__ __forceinline__ void doc_side_token(const View& v, const uint32_t* tab, uint32_t tok, uint32_t doc_len,
                                               uint32_t own, uint32_t t_first, uint32_t bm, const SlotAt& slot_at,
                                               uint2 key, uint32_t sweep, int32_t mh_steps)
{
    const uint32_t cap = SLOTS * doc_len;
    const int cb = v.count_bits;
    const T* prop = reinterpret_cast<const T*>(v.prop);
    const size_t N = (size_t)v.N;
    uint32_t* out = v.dside + (size_t)bm * v.side_stride;
    const double n_d = (double)doc_len;
    // words 0..3 (the whole record when the step count is fixed at compile time) are collected in
    // registers and go out as 16-byte stores at the end, the rest one by one
    constexpr int REGW = (FIXED > 0 && step_record_words<MODE>(FIXED) > 4) ? 8 : 4;
    static_assert(FIXED == 0 || step_record_words<MODE>(FIXED) <= 8, "the record is kept in eight registers");
    uint32_t wr[REGW];
#pragma unroll
    for (int q = 0; q < REGW; ++q) wr[q] = 0u;
    auto put = [&](int at, uint32_t val) {
        if (FIXED > 0) {
            wr[at] = val;  // the step loops are unrolled: `at` is a constant
        } else {
            if (at == 1) wr[1] = val;
            else if (at == 2) wr[2] = val;
            else if (at == 3) wr[3] = val;
            else __stcs(out + at, val);
        }
    };
    // word-proposal of step st, the wi-th of its kind: n_kd at the topic pass 1 drew
    auto word_step = [&](int32_t st, int32_t wi) {
        const uint32_t t1 = wi == 0 ? t_first : (uint32_t)__ldcg(prop + (size_t)wi * N + bm);
        const uint32_t e1 = dk_lookup(tab, cap, t1, cb);
        put(1 + st, e1 ? e1 : t1 << cb);
    };
    // doc-proposal of step st, the di-th of its kind
    auto doc_step = [&](int32_t st, int32_t di) {
        const uint4 r = philox4x32_10(make_uint4(v.tok_base + tok, sweep, (uint32_t)st, 0u), key);
        const double uu = __dmul_rn((double)r.x, INV_2_32);
        uint32_t o2;
        if (__dmul_rn(uu, __dadd_rn(n_d, v.Kalpha)) < n_d) {
            o2 = tab[slot_at(scale_to_range(r.y, doc_len))];
        } else {
            const uint32_t t2 = scale_to_range(r.y, (uint32_t)v.K);
            const uint32_t e2 = dk_lookup(tab, cap, t2, cb);
            o2 = e2 ? e2 : t2 << cb;
        }
        put(1 + st, o2);
        put(1 + mh_steps + di, r.w);  // the step's acceptance uniform
    };
    if (MODE == LDA_PROPOSALS_CYCLE) {
#pragma unroll
        for (int32_t st = 0; st < mh_steps; st += 2) {
            word_step(st, st >> 1);
            if (st + 1 < mh_steps) doc_step(st + 1, st >> 1);
        }
    } else if (MODE == LDA_PROPOSALS_WORD) {
#pragma unroll
        for (int32_t st = 0; st < mh_steps; ++st) word_step(st, st);
    } else {
#pragma unroll
        for (int32_t st = 0; st < mh_steps; ++st) doc_step(st, st);
    }
    __stcs(reinterpret_cast<uint4*>(out), make_uint4(own, wr[1], wr[2], wr[3]));
    if (REGW == 8) __stcs(reinterpret_cast<uint4*>(out) + 1, make_uint4(wr[4], wr[5], wr[6], wr[7]));
}

// `cap` = tokens a tile can hold (the shared-memory carve-up) = DOC_TILE_ROUNDS x blockDim.x: a
// thread owns at most DOC_TILE_ROUNDS tokens and keeps what it read about them in registers across
// the phases.  Small tiles keep many CTAs per SM, which is what hides the gathers of the first phase.
// FIXED > 0: the number of steps is this compile-time constant (the argument is ignored).
// Threads the compiler must leave room for per SM: the two-step kernels with a word step need few
// enough registers to fill the SM (16 CTAs of 128 threads), the others three quarters of it.
__host__ __device__ constexpr int doc_resident_threads(int mode, int fixed)
{
    return (fixed == 2 && mode != LDA_PROPOSALS_DOC) ? 2048 : 1536;
}
template <typename T, int THREADS, int MODE, int FIXED>
__global__ void __launch_bounds__(THREADS, doc_resident_threads(MODE, FIXED) / THREADS)
k_doc_tile(View v, const int32_t* __restrict__ tiles, uint2 key, uint32_t sweep, int32_t mh_steps_arg)
{
    const int32_t mh_steps = FIXED > 0 ? FIXED : mh_steps_arg;
    constexpr int cap = DOC_TILE_ROUNDS * THREADS;
    extern __shared__ __align__(16) uint32_t doc_smem[];
    uint32_t* slots = doc_smem;                                  // [TILE_SLOTS * cap] the tile's tables
    int32_t* soff = reinterpret_cast<int32_t*>(slots + TILE_SLOTS * cap);  // [cap + 1] document offsets
    uint32_t* slot_s = reinterpret_cast<uint32_t*>(soff + cap + 1);  // [cap] slot (inside its table) of a token's topic
    const int tid = threadIdx.x;
    const int32_t s0 = tiles[2 * blockIdx.x], s1 = tiles[2 * blockIdx.x + 1];
    const int32_t nseg = s1 - s0;
    const int32_t base = v.doc_off[s0];
    const int32_t cnt = v.doc_off[s1] - base;
    if (cnt == 0) return;
    const T* zbm = reinterpret_cast<const T*>(v.zbm);
    uint32_t bm[DOC_TILE_ROUNDS], z[DOC_TILE_ROUNDS], t1[DOC_TILE_ROUNDS];
    int32_t first[DOC_TILE_ROUNDS], len[DOC_TILE_ROUNDS];
#pragma unroll
    for (int r = 0; r < DOC_TILE_ROUNDS; ++r) {
        const int j = tid + r * THREADS;
        bm[r] = z[r] = t1[r] = 0;
        if (j < cnt) {
            bm[r] = __ldcs(v.bm_of_tok + base + j);
            load_topic_pair(zbm, bm[r], z[r], t1[r]);
        }
    }
    for (int j = tid; j <= nseg; j += blockDim.x) soff[j] = v.doc_off[s0 + j] - base;
    const uint4 empty4 = make_uint4(DK_EMPTY, DK_EMPTY, DK_EMPTY, DK_EMPTY);
    for (int j = tid; j < cnt * (TILE_SLOTS / 4); j += blockDim.x) reinterpret_cast<uint4*>(slots)[j] = empty4;
    __syncthreads();
    // every token finds its document, adds itself to the document's table and notes the slot
#pragma unroll
    for (int r = 0; r < DOC_TILE_ROUNDS; ++r) {
        const int j = tid + r * THREADS;
        first[r] = 0;
        len[r] = 1;
        if (j < cnt) {
            int lo = 0, hi = nseg;  // last document with soff[doc] <= j
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (soff[mid] <= j) lo = mid; else hi = mid;
            }
            first[r] = soff[lo];
            len[r] = soff[lo + 1] - first[r];
            uint32_t at = 0xFFFFFFFFu;
            if (z[r] < (uint32_t)v.K)
                at = dk_insert(slots + TILE_SLOTS * first[r], TILE_SLOTS * (uint32_t)len[r], z[r],
                               v.count_bits);
            if (at == 0xFFFFFFFFu) {
                atomicOr(v.err, z[r] < (uint32_t)v.K ? ERR_ROW_OVERFLOW : ERR_TOPIC_RANGE);
                at = 0;
            }
            slot_s[j] = at;
            z[r] = at;  // from here on: the slot
        }
    }
    __syncthreads();
    // the tables are complete: every token gathers its share
#pragma unroll
    for (int r = 0; r < DOC_TILE_ROUNDS; ++r) {
        const int j = tid + r * THREADS;
        if (j < cnt) {
            const uint32_t* tab = slots + TILE_SLOTS * first[r];
            const uint32_t* slot_of = slot_s + first[r];
            auto slot_at = [slot_of](uint32_t jj) { return slot_of[jj]; };
            doc_side_token<T, MODE, FIXED, TILE_SLOTS>(v, tab, (uint32_t)(base + j), (uint32_t)len[r], tab[z[r]], t1[r], bm[r], slot_at, key,
                              sweep, mh_steps);
        }
    }
}

// Documents longer than a tile: one CTA per document; the table lives in the document's range of
// the scratch slots in device memory (long_slot_off: four slots per token of the long documents,
// one after the other) and the slot indices in its range of the record array.
template <typename T, int MODE, int FIXED>
__global__ void __launch_bounds__(512)
k_long_doc_tile(View v, const int32_t* __restrict__ long_docs, uint2 key, uint32_t sweep, int32_t mh_steps_arg)
{
    const int32_t mh_steps = FIXED > 0 ? FIXED : mh_steps_arg;
    const int32_t d = long_docs[blockIdx.x];
    const int32_t first = v.doc_off[d], cnt = v.doc_off[d + 1] - first;
    const uint32_t cap = DK_SLOTS_PER_TOKEN * (uint32_t)cnt;
    const T* zbm = reinterpret_cast<const T*>(v.zbm);
    uint32_t* tab = v.dk_slots + v.long_slot_off[blockIdx.x];
    uint32_t* slot_of = v.rec + first;
    for (uint32_t j = threadIdx.x; j < cap; j += blockDim.x) tab[j] = DK_EMPTY;
    __syncthreads();
    for (int j = threadIdx.x; j < cnt; j += blockDim.x) {
        const uint32_t k = (uint32_t)zbm[2 * (size_t)v.bm_of_tok[first + j]];
        uint32_t at = 0xFFFFFFFFu;
        if (k < (uint32_t)v.K) at = dk_insert(tab, cap, k, v.count_bits);
        if (at == 0xFFFFFFFFu) {
            atomicOr(v.err, k < (uint32_t)v.K ? ERR_ROW_OVERFLOW : ERR_TOPIC_RANGE);
            at = 0;
        }
        slot_of[j] = at;
    }
    __syncthreads();
    auto slot_at = [slot_of](uint32_t j) { return slot_of[j]; };
    for (int j = threadIdx.x; j < cnt; j += blockDim.x) {
        const uint32_t bm = v.bm_of_tok[first + j];
        doc_side_token<T, MODE, FIXED, DK_SLOTS_PER_TOKEN>(v, tab, (uint32_t)(first + j), (uint32_t)cnt, tab[slot_of[j]], (uint32_t)zbm[2 * (size_t)bm + 1], bm,
                          slot_at, key, sweep, mh_steps);
    }
}

size_t doc_tile_smem_bytes(int tile_tokens) { return (size_t)tile_tokens * DOC_TILE_SMEM_PER_TOKEN + 16; }

template <typename T, int MODE, int FIXED>
static void set_doc_limit()
{
    cudaFuncSetAttribute(k_doc_tile<T, 1024, MODE, FIXED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         (int)doc_tile_smem_bytes(DOC_TILE_MAX));
}

void set_doc_smem_limits()
{
    set_doc_limit<uint16_t, LDA_PROPOSALS_CYCLE, 0>();
    set_doc_limit<uint16_t, LDA_PROPOSALS_CYCLE, 2>();
    set_doc_limit<uint16_t, LDA_PROPOSALS_CYCLE, 4>();
    set_doc_limit<uint16_t, LDA_PROPOSALS_WORD, 0>();
    set_doc_limit<uint16_t, LDA_PROPOSALS_WORD, 2>();
    set_doc_limit<uint16_t, LDA_PROPOSALS_DOC, 0>();
    set_doc_limit<uint16_t, LDA_PROPOSALS_DOC, 2>();
    set_doc_limit<int32_t, LDA_PROPOSALS_CYCLE, 0>();
    set_doc_limit<int32_t, LDA_PROPOSALS_CYCLE, 2>();
    set_doc_limit<int32_t, LDA_PROPOSALS_CYCLE, 4>();
    set_doc_limit<int32_t, LDA_PROPOSALS_WORD, 0>();
    set_doc_limit<int32_t, LDA_PROPOSALS_WORD, 2>();
    set_doc_limit<int32_t, LDA_PROPOSALS_DOC, 0>();
    set_doc_limit<int32_t, LDA_PROPOSALS_DOC, 2>();
}

template <typename T, int MODE, int FIXED>
static int doc_side_tm(Ctx& c, int mh_steps)
{
    const uint2 key = make_uint2((uint32_t)c.seed, (uint32_t)(c.seed >> 32));
    int launches = 0;
    if (c.n_doc_tiles) {
        const size_t smem = doc_tile_smem_bytes(c.doc_tile);
        switch (c.doc_threads) {
            case 128: k_doc_tile<T, 128, MODE, FIXED><<<c.n_doc_tiles, 128, smem, c.stream>>>(c.v, c.doc_tiles, key, c.sweep, mh_steps); break;
            case 256: k_doc_tile<T, 256, MODE, FIXED><<<c.n_doc_tiles, 256, smem, c.stream>>>(c.v, c.doc_tiles, key, c.sweep, mh_steps); break;
            case 512: k_doc_tile<T, 512, MODE, FIXED><<<c.n_doc_tiles, 512, smem, c.stream>>>(c.v, c.doc_tiles, key, c.sweep, mh_steps); break;
            default: k_doc_tile<T, 1024, MODE, FIXED><<<c.n_doc_tiles, 1024, smem, c.stream>>>(c.v, c.doc_tiles, key, c.sweep, mh_steps); break;
        }
        ++launches;
    }
    if (c.n_long_docs) {
        k_long_doc_tile<T, MODE, FIXED><<<c.n_long_docs, 512, 0, c.stream>>>(c.v, c.long_docs, key, c.sweep, mh_steps);
        ++launches;
    }
    return launches;
}

template <typename T>
static int doc_side_t(Ctx& c, int mh_steps)
{
    switch (c.proposals) {
        // chains of two steps (and the cycle with four) have kernels of their own
        case LDA_PROPOSALS_WORD:
            return mh_steps == 2 ? doc_side_tm<T, LDA_PROPOSALS_WORD, 2>(c, mh_steps)
                                 : doc_side_tm<T, LDA_PROPOSALS_WORD, 0>(c, mh_steps);
        case LDA_PROPOSALS_DOC:
            return mh_steps == 2 ? doc_side_tm<T, LDA_PROPOSALS_DOC, 2>(c, mh_steps)
                                 : doc_side_tm<T, LDA_PROPOSALS_DOC, 0>(c, mh_steps);
        default:
            return mh_steps == 2   ? doc_side_tm<T, LDA_PROPOSALS_CYCLE, 2>(c, mh_steps)
                   : mh_steps == 4 ? doc_side_tm<T, LDA_PROPOSALS_CYCLE, 4>(c, mh_steps)
                                   : doc_side_tm<T, LDA_PROPOSALS_CYCLE, 0>(c, mh_steps);
    }
}

int launch_doc_side(Ctx& c, int mh_steps)
{
    if (c.N == 0) return 0;
    return c.wide_topics ? doc_side_t<int32_t>(c, mh_steps) : doc_side_t<uint16_t>(c, mh_steps);
}

}  // namespace lda
