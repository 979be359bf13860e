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

// Everything pass 3 needs from the document side for one token, written at the token's
// block-major index `bm`.
//   tab     : the document's table, 4 * doc_len slots
//   slot_at : slot holding the topic of the document's j-th token
template <typename T, class SlotAt>
__device__ __forceinline__ void doc_side_token(const View& v, const uint32_t* tab, uint32_t tok, uint32_t doc_len,
                                               uint32_t own, uint32_t t_first, uint32_t bm, const SlotAt& slot_at,
                                               uint2 key, uint32_t sweep, int32_t mh_steps)
{
    const uint32_t cap = DK_SLOTS_PER_TOKEN * doc_len;
    const int cb = v.count_bits;
    const T* prop = reinterpret_cast<const T*>(v.prop);
    const size_t N = (size_t)v.N;
    uint32_t* out = v.dside + (size_t)bm * v.side_stride;
    const double n_d = (double)doc_len;
    // words 0..3 go out as one 16-byte store at the end, the rest one by one
    uint32_t w1 = 0u, w2 = 0u, w3 = 0u;
    auto put = [&](int at, uint32_t val) {
        if (at == 1) w1 = val;
        else if (at == 2) w2 = val;
        else if (at == 3) w3 = val;
        else __stcs(out + at, val);
    };
    for (int32_t st = 0; st < mh_steps; st += 2) {
        // word-proposal of step st: n_kd at the topic pass 1 drew
        const uint32_t t1 = st == 0 ? t_first : (uint32_t)__ldcg(prop + (size_t)(st >> 1) * N + bm);
        const uint32_t e1 = dk_lookup(tab, cap, t1, cb);
        put(1 + st, e1 ? e1 : t1 << cb);
        if (st + 1 < mh_steps) {
            // doc-proposal of step st+1
            const uint4 r = philox4x32_10(make_uint4(tok, sweep, (uint32_t)(st + 1), 0u), key);
            const double uu = __dmul_rn((double)r.x, INV_2_32);
            uint32_t o2;
            if (__dmul_rn(uu, __dadd_rn(n_d, v.Kalpha)) < n_d) {
                o2 = tab[slot_at(scale_to_range(r.y, doc_len))];
            } else {
                const uint32_t t2 = scale_to_range(r.y, (uint32_t)v.K);
                const uint32_t e2 = dk_lookup(tab, cap, t2, cb);
                o2 = e2 ? e2 : t2 << cb;
            }
            put(2 + st, o2);
            put(1 + mh_steps + (st >> 1), r.w);  // the step's acceptance uniform
        }
    }
    __stcs(reinterpret_cast<uint4*>(out), make_uint4(own, w1, w2, w3));
}

// `cap` = tokens a tile can hold (the shared-memory carve-up); small tiles keep many CTAs per SM,
// which is what hides the gathers of the first phase.
template <typename T>
__global__ void __launch_bounds__(1024)
k_doc_tile(View v, const int32_t* __restrict__ tiles, int32_t cap, uint2 key, uint32_t sweep, int32_t mh_steps)
{
    extern __shared__ __align__(16) uint32_t doc_smem[];
    uint32_t* slots = doc_smem;                                  // [4 * cap] the tile's tables
    int32_t* soff = reinterpret_cast<int32_t*>(slots + DK_SLOTS_PER_TOKEN * cap);  // [cap + 1] document offsets
    uint32_t* topic = reinterpret_cast<uint32_t*>(soff + cap + 1);  // [cap] a token's topic, later its slot
    uint32_t* bm_s = topic + cap;                                // [cap] a token's block-major index
    uint32_t* t1_s = bm_s + cap;                                 // [cap] the first word-proposal's topic
    uint16_t* doc_s = reinterpret_cast<uint16_t*>(t1_s + cap);   // [cap] a token's document, relative to the tile
    const int tid = threadIdx.x;
    const int32_t s0 = tiles[2 * blockIdx.x], s1 = tiles[2 * blockIdx.x + 1];
    const int32_t nseg = s1 - s0;
    const int32_t base = v.doc_off[s0];
    const int32_t cnt = v.doc_off[s1] - base;
    if (cnt == 0) return;
    const T* zbm = reinterpret_cast<const T*>(v.zbm);
    const T* prop = reinterpret_cast<const T*>(v.prop);
    for (int j = tid; j < cnt; j += blockDim.x) {
        const uint32_t bm = __ldcs(v.bm_of_tok + base + j);
        bm_s[j] = bm;
        topic[j] = (uint32_t)__ldcg(zbm + bm);
        t1_s[j] = (uint32_t)__ldcg(prop + bm);
    }
    for (int j = tid; j <= nseg; j += blockDim.x) soff[j] = v.doc_off[s0 + j] - base;
    for (int j = tid; j < DK_SLOTS_PER_TOKEN * cnt; j += blockDim.x) slots[j] = DK_EMPTY;
    __syncthreads();
    // which document each token belongs to: one warp per document writes its index
    const int lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    for (int d = warp; d < nseg; d += nwarps)
        for (int j = soff[d] + lane; j < soff[d + 1]; j += 32) doc_s[j] = (uint16_t)d;
    __syncthreads();
    // every token adds itself to its document's table and notes the slot
    for (int j = tid; j < cnt; j += blockDim.x) {
        const int32_t first = soff[doc_s[j]], len = soff[doc_s[j] + 1] - first;
        const uint32_t k = topic[j];
        uint32_t at = 0xFFFFFFFFu;
        if (k < (uint32_t)v.K)
            at = dk_insert(slots + DK_SLOTS_PER_TOKEN * first, DK_SLOTS_PER_TOKEN * (uint32_t)len, k, v.count_bits);
        if (at == 0xFFFFFFFFu) {
            atomicOr(v.err, k < (uint32_t)v.K ? ERR_ROW_OVERFLOW : ERR_TOPIC_RANGE);
            at = 0;
        }
        topic[j] = at;
    }
    __syncthreads();
    // the tables are complete: every token gathers its share
    for (int j = tid; j < cnt; j += blockDim.x) {
        const int32_t first = soff[doc_s[j]], len = soff[doc_s[j] + 1] - first;
        const uint32_t* tab = slots + DK_SLOTS_PER_TOKEN * first;
        const uint32_t* slot_of = topic + first;
        auto slot_at = [slot_of](uint32_t jj) { return slot_of[jj]; };
        doc_side_token<T>(v, tab, (uint32_t)(base + j), (uint32_t)len, tab[topic[j]], t1_s[j], bm_s[j], slot_at, key,
                          sweep, mh_steps);
    }
}

// Documents longer than a tile: one CTA per document; the table lives in the document's range of
// the global slot array and the slot indices in its range of the record array (both are scratch
// here: the exported n_kd tables are rebuilt on demand).
template <typename T>
__global__ void __launch_bounds__(512)
k_long_doc_tile(View v, const int32_t* __restrict__ long_docs, uint2 key, uint32_t sweep, int32_t mh_steps)
{
    const int32_t d = long_docs[blockIdx.x];
    const int32_t first = v.doc_off[d], cnt = v.doc_off[d + 1] - first;
    const uint32_t cap = DK_SLOTS_PER_TOKEN * (uint32_t)cnt;
    const T* zbm = reinterpret_cast<const T*>(v.zbm);
    const T* prop = reinterpret_cast<const T*>(v.prop);
    uint32_t* tab = v.dk_slots + DK_SLOTS_PER_TOKEN * (size_t)first;
    uint32_t* slot_of = v.rec + first;
    for (uint32_t j = threadIdx.x; j < cap; j += blockDim.x) tab[j] = DK_EMPTY;
    __syncthreads();
    for (int j = threadIdx.x; j < cnt; j += blockDim.x) {
        const uint32_t k = (uint32_t)zbm[v.bm_of_tok[first + j]];
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
        doc_side_token<T>(v, tab, (uint32_t)(first + j), (uint32_t)cnt, tab[slot_of[j]], (uint32_t)prop[bm], bm,
                          slot_at, key, sweep, mh_steps);
    }
}

size_t doc_tile_smem_bytes(int tile_tokens) { return (size_t)tile_tokens * DOC_TILE_SMEM_PER_TOKEN + 16; }

void set_doc_smem_limits()
{
    const int bytes = (int)doc_tile_smem_bytes(DOC_TILE_MAX);
    cudaFuncSetAttribute(k_doc_tile<uint16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    cudaFuncSetAttribute(k_doc_tile<int32_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

template <typename T>
static int doc_side_t(Ctx& c, int mh_steps)
{
    const uint2 key = make_uint2((uint32_t)c.seed, (uint32_t)(c.seed >> 32));
    int launches = 0;
    if (c.n_doc_tiles) {
        k_doc_tile<T><<<c.n_doc_tiles, c.doc_threads, doc_tile_smem_bytes(c.doc_tile), c.stream>>>(
            c.v, c.doc_tiles, c.doc_tile, key, c.sweep, mh_steps);
        ++launches;
    }
    if (c.n_long_docs) {
        k_long_doc_tile<T><<<c.n_long_docs, 512, 0, c.stream>>>(c.v, c.long_docs, key, c.sweep, mh_steps);
        ++launches;
    }
    return launches;
}

int launch_doc_side(Ctx& c, int mh_steps)
{
    if (c.N == 0) return 0;
    return c.wide_topics ? doc_side_t<int32_t>(c, mh_steps) : doc_side_t<uint16_t>(c, mh_steps);
}

}  // namespace lda
