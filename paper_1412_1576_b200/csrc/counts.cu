// Count-table rebuild from the assignments (Section 3: n_kw, n_k; Eq. 12: n_kd).
//
// n_kw (segments = words over the word-sorted z): per word, the sorted list of
// (topic, count).  Two paths, chosen per word at load time:
//   - tail words: whole words are packed into tiles of <= SORT_TILE tokens; one
//     CTA counts each word's topics in a shared-memory hash table and reads them
//     back in topic order through a bitmap over the topics (K <= 16384), or sorts
//     the tile's (word, topic) keys (larger K);
//   - hot words: shared-memory histogram over a window of topics, merged into
//     the word's dense row, then compacted into the sorted row.
// n_k: column sums of the rows just written.
// n_kd (segments = documents): the MH step builds every document's table itself, per tile, in
// shared memory (docside.cu), and so does the log-likelihood (loglik.cu); lda_get_counts gets
// sorted rows from export.cu.
// No per-token global atomics: a CTA touches global counters once per bin it
// actually filled (documents longer than a tile are the one exception).
#include <algorithm>

#include "lda_device.cuh"
#include "lda_internal.cuh"

namespace lda {

struct EmitWord {
    const int32_t* row_start;
    uint32_t* topic;
    uint32_t* count;
    int32_t* nnz;
    __device__ __forceinline__ void entry(int32_t seg, int32_t rank, uint32_t k, uint32_t n) const
    {
        const int32_t slot = row_start[seg] + rank;
        topic[slot] = k;
        count[slot] = n;
    }
    __device__ __forceinline__ void rows(int32_t seg, int32_t n) const { nnz[seg] = n; }
};

// Tail words when K is large (the bitmap of k_word_rows would cost more than the sort): one CTA per
// tile of whole words [s0, s1) holding <= SORT_TILE tokens and <= SORT_TILE words sorts the tile's
// (word, topic) keys in shared memory (bitonic) and run-length encodes them.
template <typename T, class Emit>
__global__ void __launch_bounds__(256)
k_seg_count_sorted(const int32_t* __restrict__ tiles, const int32_t* __restrict__ seg_off,
                   const T* __restrict__ z, int topic_bits, int32_t K, Emit emit, int* err)
{
    __shared__ uint32_t keys[SORT_TILE];
    __shared__ int32_t soff[SORT_TILE + 1];
    __shared__ int32_t hidx[SORT_TILE + 1];
    __shared__ int32_t headpos[SORT_TILE + 1];
    __shared__ int32_t scan_tmp[33];

    const int tid = threadIdx.x;
    const int32_t s0 = tiles[2 * blockIdx.x], s1 = tiles[2 * blockIdx.x + 1];
    const int32_t nseg = s1 - s0;
    const int32_t base = seg_off[s0];
    const int32_t cnt = seg_off[s1] - base;
    for (int j = tid; j <= nseg; j += blockDim.x) soff[j] = seg_off[s0 + j] - base;
    int npad = 1;
    while (npad < cnt) npad <<= 1;
    __syncthreads();
    if (cnt == 0) {
        for (int j = tid; j < nseg; j += blockDim.x) emit.rows(s0 + j, 0);
        return;
    }
    for (int j = tid; j < npad; j += blockDim.x) {
        uint32_t key = 0xFFFFFFFFu;
        if (j < cnt) {
            int lo = 0, hi = nseg;  // last segment with soff[seg] <= j
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (soff[mid] <= j) lo = mid; else hi = mid;
            }
            const uint32_t k = (uint32_t)z[base + j];
            if (k >= (uint32_t)K) atomicOr(err, ERR_TOPIC_RANGE);
            key = ((uint32_t)lo << topic_bits) | k;
        }
        keys[j] = key;
    }
    __syncthreads();
    // bitonic sort, ascending
    for (int size = 2; size <= npad; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int t = tid; t < (npad >> 1); t += blockDim.x) {
                const int i = ((t & ~(stride - 1)) << 1) | (t & (stride - 1));
                const int j = i | stride;
                const bool up = ((i & size) == 0);
                const uint32_t a = keys[i], b = keys[j];
                if ((a > b) == up) { keys[i] = b; keys[j] = a; }
            }
            __syncthreads();
        }
    }
    // head flags -> exclusive scan (8 consecutive entries per thread)
    constexpr int PER = SORT_TILE / 256;
    int32_t flags[PER];
    int32_t local = 0;
#pragma unroll
    for (int q = 0; q < PER; ++q) {
        const int j = tid * PER + q;
        flags[q] = (j < cnt && (j == 0 || keys[j] != keys[j - 1])) ? 1 : 0;
        local += flags[q];
    }
    int32_t total;
    int32_t run = block_scan_excl<int32_t>(local, scan_tmp, total);
#pragma unroll
    for (int q = 0; q < PER; ++q) {
        const int j = tid * PER + q;
        if (j < cnt) {
            hidx[j] = run;
            if (flags[q]) headpos[run] = j;
            run += flags[q];
        }
    }
    if (tid == 0) { hidx[cnt] = total; headpos[total] = cnt; }
    __syncthreads();
    const uint32_t kmask = (1u << topic_bits) - 1u;
    for (int h = tid; h < total; h += blockDim.x) {
        const int j = headpos[h];
        const uint32_t key = keys[j];
        const int32_t seg = (int32_t)(key >> topic_bits);
        const int32_t rank = h - hidx[soff[seg]];
        emit.entry(s0 + seg, rank, key & kmask, (uint32_t)(headpos[h + 1] - j));
    }
    for (int j = tid; j < nseg; j += blockDim.x) emit.rows(s0 + j, hidx[soff[j + 1]] - hidx[soff[j]]);
}

// Tail words: one CTA per tile of whole words [s0, s1) holding <= SORT_TILE tokens; the words are
// taken one after the other.  A word's tokens are counted in a shared-memory hash table (same
// tables as n_kd: 4 slots per token) and marked in a bitmap over the K topics; the bitmap, read in
// order, gives the sorted row: the rank of a topic is the number of set bits before it.
template <typename T>
__global__ void __launch_bounds__(256)
k_word_rows(const int32_t* __restrict__ tiles, const int32_t* __restrict__ word_off, const T* __restrict__ z,
            const int32_t* __restrict__ row_start, uint32_t* __restrict__ wk_topic, uint32_t* __restrict__ wk_count,
            int32_t* __restrict__ wk_nnz, int32_t K, int* err)
{
    constexpr int CB = 12;  // count bits of a table entry: a tail word has at most SORT_TILE = 2048 tokens
    static_assert(SORT_TILE < (1 << CB), "count bits");
    extern __shared__ uint32_t word_smem[];
    __shared__ uint32_t table[DK_SLOTS_PER_TOKEN * SORT_TILE];
    __shared__ int32_t scan_tmp[33];
    const int32_t bw = (K + 31) >> 5;
    uint32_t* bitmap = word_smem;  // [bw] topics present in the word
    uint32_t* before = word_smem + bw;  // [bw] set bits before each bitmap word
    const int tid = threadIdx.x;
    const int32_t s0 = tiles[2 * blockIdx.x], s1 = tiles[2 * blockIdx.x + 1];
    // Words of at most 32 tokens (most of the vocabulary) take one warp each and no barrier: a lane
    // holds a token, lanes with the same topic find each other, the lowest of them writes the entry at
    // the rank of its topic among the word's distinct topics.
    {
        const int lane = tid & 31;
        for (int32_t w = s0 + (tid >> 5); w < s1; w += (int32_t)(blockDim.x >> 5)) {
            const int32_t first = word_off[w], n = word_off[w + 1] - first;
            if (n > 32) continue;
            uint32_t k = 0xFFFFFFFFu;
            if (lane < n) {
                k = (uint32_t)__ldcs(z + first + lane);
                if (k >= (uint32_t)K) { atomicOr(err, ERR_TOPIC_RANGE); k = 0xFFFFFFFFu; }
            }
            const uint32_t same = __match_any_sync(0xFFFFFFFFu, k);
            const bool lead = k != 0xFFFFFFFFu && (uint32_t)(__ffs((int)same) - 1) == (uint32_t)lane;
            const uint32_t leaders = __ballot_sync(0xFFFFFFFFu, lead);
            int32_t rank = 0;
            for (uint32_t m = leaders; m; m &= m - 1u) {
                const uint32_t other = __shfl_sync(0xFFFFFFFFu, k, __ffs((int)m) - 1);
                rank += other < k ? 1 : 0;
            }
            if (lead) {
                const int32_t r = row_start[w] + rank;
                wk_topic[r] = k;
                wk_count[r] = (uint32_t)__popc(same);
            }
            if (lane == 0) wk_nnz[w] = __popc(leaders);
        }
    }
    for (int32_t w = s0; w < s1; ++w) {
        const int32_t first = word_off[w], n = word_off[w + 1] - first;
        if (n <= 32) continue;  // done above
        const uint32_t cap = DK_SLOTS_PER_TOKEN * (uint32_t)n;
        for (int32_t i = tid; i < bw; i += blockDim.x) bitmap[i] = 0;
        for (uint32_t i = tid; i < cap; i += blockDim.x) table[i] = DK_EMPTY;
        __syncthreads();
        for (int32_t j = tid; j < n; j += blockDim.x) {
            const uint32_t k = (uint32_t)__ldcs(z + first + j);
            if (k >= (uint32_t)K) { atomicOr(err, ERR_TOPIC_RANGE); continue; }
            atomicOr(&bitmap[k >> 5], 1u << (k & 31u));
            if (dk_insert(table, cap, k, CB) == DK_EMPTY) atomicOr(err, ERR_ROW_OVERFLOW);
        }
        __syncthreads();
        int32_t running = 0;
        for (int32_t i0 = 0; i0 < bw; i0 += blockDim.x) {
            const int32_t i = i0 + tid;
            const int32_t c = i < bw ? __popc(bitmap[i]) : 0;
            int32_t total;
            const int32_t pos = block_scan_excl<int32_t>(c, scan_tmp, total);
            if (i < bw) before[i] = (uint32_t)(running + pos);
            running += total;
        }
        __syncthreads();
        const int32_t out0 = row_start[w];
        for (int32_t i = tid; i < bw; i += blockDim.x) {
            uint32_t m = bitmap[i];
            int32_t r = out0 + (int32_t)before[i];
            while (m) {
                const uint32_t k = 32u * (uint32_t)i + (uint32_t)(__ffs((int)m) - 1);
                m &= m - 1u;
                wk_topic[r] = k;
                wk_count[r] = dk_lookup(table, cap, k, CB) & ((1u << CB) - 1u);
                ++r;
            }
        }
        if (tid == 0) wk_nnz[w] = running;
        __syncthreads();
    }
}

// Warm words (more tokens than a tail tile holds, no dense row): one CTA per word.  The word's
// tokens are counted in 16-bit bins over a window of topics in shared memory (two bins per word of
// shared memory; a warm word has fewer than 65536 tokens), and the nonzero bins, read in order,
// are the sorted row: every warp owns a run of consecutive bin pairs, counts its nonzero bins, the
// warps' totals are scanned, and a second walk writes the entries.
template <typename T>
__global__ void __launch_bounds__(512)
k_warm_rows(const int32_t* __restrict__ words, const int32_t* __restrict__ word_off, const T* __restrict__ z,
            const int32_t* __restrict__ row_start, uint32_t* __restrict__ wk_topic, uint32_t* __restrict__ wk_count,
            int32_t* __restrict__ wk_nnz, int32_t K, int32_t window, int* err)
{
    extern __shared__ __align__(16) uint32_t bins2[];
    __shared__ int32_t warp_total[17];
    const int32_t w = words[blockIdx.x];
    const int32_t first = word_off[w], cnt = word_off[w + 1] - first;
    const int32_t out0 = row_start[w], cap = row_start[w + 1] - out0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    int32_t done = 0;
    for (int32_t k0 = 0; k0 < K; k0 += window) {
        const int32_t nb = min(window, K - k0), nw = (nb + 1) >> 1;
        const int32_t nw4 = (nw + 3) >> 2;
        for (int b = threadIdx.x; b < nw4; b += blockDim.x) reinterpret_cast<uint4*>(bins2)[b] = make_uint4(0u, 0u, 0u, 0u);
        __syncthreads();
        for (int32_t j = threadIdx.x; j < cnt; j += blockDim.x) {
            const uint32_t k = (uint32_t)__ldcs(z + first + j);
            if (k >= (uint32_t)K) { atomicOr(err, ERR_TOPIC_RANGE); continue; }
            const uint32_t b = k - (uint32_t)k0;
            if (b < (uint32_t)nb) atomicAdd(&bins2[b >> 1], (b & 1u) ? 0x10000u : 1u);
        }
        __syncthreads();
        // a warp's run of bin pairs
        const int32_t per_warp = ((nw + nwarps - 1) / nwarps + 31) & ~31;
        const int32_t q0 = min(nw, warp * per_warp), q1 = min(nw, q0 + per_warp);
        int32_t mine = 0;
        for (int32_t q = q0 + lane; q < q1; q += 32) {
            const uint32_t n2 = bins2[q];
            mine += ((n2 & 0xFFFFu) != 0u) + ((n2 >> 16) != 0u);
        }
        mine = warp_reduce_sum<int32_t>(mine);
        if (lane == 0) warp_total[warp] = mine;
        __syncthreads();
        if (threadIdx.x == 0) {
            int32_t run = 0;
            for (int i = 0; i < nwarps; ++i) { const int32_t t = warp_total[i]; warp_total[i] = run; run += t; }
            warp_total[16] = run;
        }
        __syncthreads();
        int32_t at = done + warp_total[warp];
        const int32_t total = warp_total[16];
        if (done + total > cap) {
            if (threadIdx.x == 0) atomicOr(err, ERR_ROW_OVERFLOW);
        } else {
            const uint32_t below = (1u << lane) - 1u;
            for (int32_t q = q0 + lane; q - lane < q1; q += 32) {
                const uint32_t n2 = q < q1 ? bins2[q] : 0u;
                const bool lo = (n2 & 0xFFFFu) != 0u, hi = (n2 >> 16) != 0u;
                const uint32_t m_lo = __ballot_sync(0xffffffffu, lo), m_hi = __ballot_sync(0xffffffffu, hi);
                int32_t pos = at + __popc(m_lo & below) + __popc(m_hi & below);
                if (lo) {
                    wk_topic[out0 + pos] = (uint32_t)(k0 + 2 * q);
                    wk_count[out0 + pos] = n2 & 0xFFFFu;
                    ++pos;
                }
                if (hi) {
                    wk_topic[out0 + pos] = (uint32_t)(k0 + 2 * q + 1);
                    wk_count[out0 + pos] = n2 >> 16;
                }
                at += __popc(m_lo) + __popc(m_hi);
            }
        }
        done += total;
        __syncthreads();
    }
    if (threadIdx.x == 0) wk_nnz[w] = done;
}

// Hot words: one CTA per run of a word's tokens (up to HIST_CHUNK of them); histogram of a window
// of topics in shared memory (32-bit bins), merged into the word's dense row.  A word that fits
// one run owns its row: its nonzero bins are stored.  A longer word's runs add theirs, one global
// add per nonzero bin and run -- a few runs per word, so a row takes few adds per bin.
template <typename T>
__global__ void __launch_bounds__(512)
k_hist_chunks(const int32_t* __restrict__ chunks, const T* __restrict__ z,
              const int32_t* __restrict__ dense_slot, int32_t* __restrict__ dense_rows, int32_t K,
              int32_t stride, int32_t window, int* err)
{
    extern __shared__ __align__(16) int32_t hist_bins[];
    const int32_t w = chunks[4 * blockIdx.x], first = chunks[4 * blockIdx.x + 1],
                  cnt = chunks[4 * blockIdx.x + 2];
    const bool alone = chunks[4 * blockIdx.x + 3] != 0;  // the word's only run
    int32_t* row = dense_rows + (size_t)dense_slot[w] * stride;
    for (int32_t k0 = 0; k0 < K; k0 += window) {
        const int32_t nb = min(window, K - k0);
        for (int b = threadIdx.x; b < (nb + 3) / 4; b += blockDim.x)
            reinterpret_cast<int4*>(hist_bins)[b] = make_int4(0, 0, 0, 0);
        __syncthreads();
        auto add = [&](uint32_t k) {
            if (k >= (uint32_t)K) { atomicOr(err, ERR_TOPIC_RANGE); return; }
            const uint32_t b = k - (uint32_t)k0;
            if (b < (uint32_t)nb) atomicAdd(&hist_bins[b], 1);
        };
        // the run's topics are read 16 bytes at a time; what lies before the first and after the
        // last 16-byte boundary one by one
        constexpr int E = 16 / (int)sizeof(T);
        const int32_t head = min(cnt, (int32_t)((E - (first & (E - 1))) & (E - 1)));
        const int32_t nvec = (cnt - head) / E;
        const uint4* zv = reinterpret_cast<const uint4*>(z + first + head);
        for (int q = threadIdx.x; q < nvec; q += blockDim.x) {
            const uint4 x = k0 == 0 ? __ldcs(zv + q) : __ldg(zv + q);
            const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (sizeof(T) == 2) {
                    add(xs[u] & 0xFFFFu);
                    add(xs[u] >> 16);
                } else {
                    add(xs[u]);
                }
            }
        }
        for (int j = threadIdx.x; j < cnt - nvec * E; j += blockDim.x)
            add((uint32_t)z[first + (j < head ? j : nvec * E + j)]);
        __syncthreads();
        for (int b = threadIdx.x; b < nb; b += blockDim.x) {
            const int32_t n = hist_bins[b];
            if (n) {
                if (alone) row[k0 + b] = n;  // the row was cleared before the launch
                else atomicAdd(&row[k0 + b], n);
            }
        }
        __syncthreads();
    }
}

// Dense row -> sorted (topic, count) row, one CTA per dense word.
__global__ void __launch_bounds__(256)
k_compact_dense(const int32_t* __restrict__ dense_words, const int32_t* __restrict__ dense_slot,
                const int32_t* __restrict__ dense_rows, const int32_t* __restrict__ row_start,
                uint32_t* __restrict__ wk_topic, uint32_t* __restrict__ wk_count,
                int32_t* __restrict__ wk_nnz, int32_t K, int32_t stride, int* err)
{
    __shared__ int32_t scan_tmp[33];
    const int32_t w = dense_words[blockIdx.x];
    const int32_t* row = dense_rows + (size_t)dense_slot[w] * stride;
    const int32_t out0 = row_start[w], cap = row_start[w + 1] - out0;
    // four consecutive topics per thread and step (rows are padded to a multiple of four and start
    // 16-byte aligned; the padding is never written, so it reads as zero)
    int32_t done = 0;
    for (int32_t k0 = 0; k0 < stride; k0 += 4 * blockDim.x) {
        const int32_t k = k0 + 4 * (int32_t)threadIdx.x;
        int4 n = make_int4(0, 0, 0, 0);
        if (k < stride) n = __ldcs(reinterpret_cast<const int4*>(row + k));
        const int32_t mine = (n.x > 0) + (n.y > 0) + (n.z > 0) + (n.w > 0);
        int32_t total;
        int32_t pos = done + block_scan_excl<int32_t>(mine, scan_tmp, total);
        if (pos + mine > cap) {
            atomicOr(err, ERR_ROW_OVERFLOW);
        } else {
            const int32_t nv[4] = {n.x, n.y, n.z, n.w};
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (nv[q] > 0) {
                    wk_topic[out0 + pos] = (uint32_t)(k + q);
                    wk_count[out0 + pos] = (uint32_t)nv[q];
                    ++pos;
                }
        }
        done += total;
    }
    if (threadIdx.x == 0) wk_nnz[w] = done;
}

// n_k = sum over words of n_kw (Section 3), taken from the rows the n_kw rebuild has just written
// instead of from another pass over the assignments:
//   - dense rows: column sums, one thread per topic and group of rows;
//   - sorted rows of the words without a dense row: CTA-private shared-memory bins over a chunk
//     of words, flushed with one global add per nonzero bin.
__global__ void __launch_bounds__(256)
k_nk_from_dense(const int32_t* __restrict__ dense_rows, int32_t n_dense, int32_t K, int32_t stride,
                int32_t* __restrict__ nk)
{
    // four consecutive topics per thread (rows are padded to a multiple of four and 16-byte aligned;
    // the padding is never written, so it reads as zero), a slice of the rows per blockIdx.y
    const int32_t k = 4 * (blockIdx.x * blockDim.x + threadIdx.x);
    if (k >= stride) return;
    int4 s = make_int4(0, 0, 0, 0);
#pragma unroll 4
    for (int32_t r = blockIdx.y; r < n_dense; r += gridDim.y) {
        const int4 x = __ldcs(reinterpret_cast<const int4*>(dense_rows + (size_t)r * stride + k));
        s.x += x.x; s.y += x.y; s.z += x.z; s.w += x.w;
    }
    if (s.x) atomicAdd(&nk[k], s.x);
    if (s.y && k + 1 < K) atomicAdd(&nk[k + 1], s.y);
    if (s.z && k + 2 < K) atomicAdd(&nk[k + 2], s.z);
    if (s.w && k + 3 < K) atomicAdd(&nk[k + 3], s.w);
}

__global__ void __launch_bounds__(512)
k_nk_from_sparse(const int32_t* __restrict__ row_start, const int32_t* __restrict__ wk_nnz,
                 const uint32_t* __restrict__ wk_topic, const uint32_t* __restrict__ wk_count,
                 const int32_t* __restrict__ dense_slot, int32_t V, int32_t* __restrict__ nk, int32_t K,
                 int32_t window)
{
    extern __shared__ int32_t bins[];
    const int32_t per = (V + gridDim.x - 1) / gridDim.x;
    const int32_t w_lo = per * blockIdx.x, w_hi = min(V, w_lo + per);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int32_t k0 = 0; k0 < K; k0 += window) {
        const int32_t nb = min(window, K - k0);
        for (int b = threadIdx.x; b < nb; b += blockDim.x) bins[b] = 0;
        __syncthreads();
        for (int32_t w = w_lo + warp; w < w_hi; w += nwarps) {
            if (dense_slot[w] >= 0) continue;
            const int32_t r0 = row_start[w], n = wk_nnz[w];
            for (int32_t j = lane; j < n; j += 32) {
                const uint32_t b = wk_topic[r0 + j] - (uint32_t)k0;
                if (b < (uint32_t)nb) atomicAdd(&bins[b], (int32_t)wk_count[r0 + j]);
            }
        }
        __syncthreads();
        for (int b = threadIdx.x; b < nb; b += blockDim.x) {
            const int32_t n = bins[b];
            if (n) atomicAdd(&nk[k0 + b], n);
        }
        __syncthreads();
    }
}

// The same sums when K is too large for bins in shared memory: one global add per row entry (the
// adds of one warp go to different topics: a row holds a topic once).
__global__ void __launch_bounds__(256)
k_nk_from_sparse_direct(const int32_t* __restrict__ row_start, const int32_t* __restrict__ wk_nnz,
                        const uint32_t* __restrict__ wk_topic, const uint32_t* __restrict__ wk_count,
                        const int32_t* __restrict__ dense_slot, int32_t V, int32_t* __restrict__ nk)
{
    const int lane = threadIdx.x & 31;
    const int32_t warps = (gridDim.x * blockDim.x) >> 5;
    for (int32_t w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < V; w += warps) {
        if (dense_slot[w] >= 0) continue;
        const int32_t r0 = row_start[w], n = wk_nnz[w];
        for (int32_t j = lane; j < n; j += 32) atomicAdd(&nk[__ldcs(wk_topic + r0 + j)], (int32_t)__ldcs(wk_count + r0 + j));
    }
}

struct EmitRowSizes {
    int32_t* nnz;
    __device__ __forceinline__ void entry(int32_t, int32_t, uint32_t, uint32_t) const {}
    __device__ __forceinline__ void rows(int32_t seg, int32_t n) const { nnz[seg] = n; }
};

struct EmitRowEntries {
    const long long* row_off;
    int32_t* topic;
    int32_t* count;
    __device__ __forceinline__ void entry(int32_t seg, int32_t rank, uint32_t k, uint32_t n) const
    {
        const long long at = row_off[seg] + rank;
        topic[at] = (int32_t)k;
        count[at] = (int32_t)n;
    }
    __device__ __forceinline__ void rows(int32_t, int32_t) const {}
};

// Sorted rows of the segments (documents) of `tiles` from z given in segment order: sizes only, or
// the entries at the row offsets (export.cu).
template <typename T>
void launch_doc_rows(Ctx& c, const int32_t* tiles, int32_t n_tiles, const T* z, int32_t* nnz, const long long* row_off,
                     int32_t* topic, int32_t* count)
{
    if (nnz)
        k_seg_count_sorted<T, EmitRowSizes><<<n_tiles, 256, 0, c.stream>>>(tiles, c.v.doc_off, z, c.v.topic_bits, c.K,
                                                                            EmitRowSizes{nnz}, c.v.err);
    else
        k_seg_count_sorted<T, EmitRowEntries><<<n_tiles, 256, 0, c.stream>>>(
            tiles, c.v.doc_off, z, c.v.topic_bits, c.K, EmitRowEntries{row_off, topic, count}, c.v.err);
}
template void launch_doc_rows<uint16_t>(Ctx&, const int32_t*, int32_t, const uint16_t*, int32_t*, const long long*, int32_t*, int32_t*);
template void launch_doc_rows<int32_t>(Ctx&, const int32_t*, int32_t, const int32_t*, int32_t*, const long long*, int32_t*, int32_t*);

static int hist_window(const Ctx& c) { return c.K < HIST_BINS ? c.K : HIST_BINS; }

template <typename T>
static int count_wk_t(Ctx& c)
{
    View& v = c.v;
    int launches = 0;
    const T* z = (const T*)v.zw;
    // the tail words' rows and the hot words' rows are built side by side
    fork_streams(c);
    if (c.n_word_tiles) {
        if (c.K <= WORD_ROWS_BITMAP_MAX_K) {
            const size_t smem = 2 * (size_t)((c.K + 31) / 32) * 4;
            k_word_rows<T><<<c.n_word_tiles, 256, smem, c.side[0]>>>(c.word_tiles, v.word_off, z, v.row_start,
                                                                    v.wk_topic, v.wk_count, v.wk_nnz, c.K, v.err);
        } else {
            EmitWord e{v.row_start, v.wk_topic, v.wk_count, v.wk_nnz};
            k_seg_count_sorted<T, EmitWord><<<c.n_word_tiles, 256, 0, c.side[0]>>>(
                c.word_tiles, v.word_off, z, v.topic_bits, c.K, e, v.err);
        }
        ++launches;
    }
    if (c.n_warm) {
        const int win = c.K < HIST16_BINS ? c.K : HIST16_BINS;
        k_warm_rows<T><<<c.n_warm, 512, (size_t)((win + 7) / 8) * 16, c.side[1]>>>(
            c.warm_words, v.word_off, z, v.row_start, v.wk_topic, v.wk_count, v.wk_nnz, c.K, win, v.err);
        ++launches;
    }
    if (c.n_dense) {
        cudaMemsetAsync(v.dense_rows, 0, (size_t)c.n_dense * v.dense_stride * 4, c.stream);
        const int win = c.K < HIST32_BINS ? c.K : HIST32_BINS;
        k_hist_chunks<T><<<c.n_hist_chunks, 512, (size_t)((win + 3) / 4) * 16, c.stream>>>(
            c.hist_chunks, z, v.dense_slot, v.dense_rows, c.K, v.dense_stride, win, v.err);
        k_compact_dense<<<c.n_dense, 256, 0, c.stream>>>(c.dense_words, v.dense_slot, v.dense_rows,
                                                         v.row_start, v.wk_topic, v.wk_count,
                                                         v.wk_nnz, c.K, v.dense_stride, v.err);
        launches += 2;
    }
    join_streams(c);
    return launches;
}

// Must follow launch_count_wk(): reads the rows it wrote.
static int count_k(Ctx& c)
{
    View& v = c.v;
    cudaMemsetAsync(v.nk, 0, (size_t)c.K * 4, c.stream);
    if (c.N == 0) return 0;
    int launches = 0;
    // both kernels add into n_k (integer adds: any order gives the same sums)
    fork_streams(c);
    if (c.n_dense) {
        const dim3 grid((unsigned)((v.dense_stride / 4 + 255) / 256), (unsigned)std::min(c.n_dense, 256));
        k_nk_from_dense<<<grid, 256, 0, c.stream>>>(v.dense_rows, c.n_dense, c.K, v.dense_stride, v.nk);
        ++launches;
    }
    if (c.n_dense < c.V) {
        if (c.K <= HIST_BINS) {
            const int win = hist_window(c);
            const int grid = std::min(148 * 4, (int)((c.V + 255) / 256));
            k_nk_from_sparse<<<grid, 512, (size_t)win * 4, c.side[0]>>>(v.row_start, v.wk_nnz, v.wk_topic, v.wk_count,
                                                                       v.dense_slot, c.V, v.nk, c.K, win);
        } else {
            const int grid = (int)std::min<int64_t>(148 * 16, ((int64_t)c.V * 32 + 255) / 256);
            k_nk_from_sparse_direct<<<grid, 256, 0, c.side[0]>>>(v.row_start, v.wk_nnz, v.wk_topic, v.wk_count,
                                                                v.dense_slot, c.V, v.nk);
        }
        ++launches;
    }
    join_streams(c);
    return launches;
}

int launch_count_wk(Ctx& c) { return c.wide_topics ? count_wk_t<int32_t>(c) : count_wk_t<uint16_t>(c); }
int launch_count_k(Ctx& c) { return count_k(c); }

void set_hist_smem_limits()
{
    cudaFuncSetAttribute(k_warm_rows<uint16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST16_BINS * 2 + 16);
    cudaFuncSetAttribute(k_warm_rows<int32_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST16_BINS * 2 + 16);
    cudaFuncSetAttribute(k_hist_chunks<uint16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST32_BINS * 4);
    cudaFuncSetAttribute(k_hist_chunks<int32_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST32_BINS * 4);
    cudaFuncSetAttribute(k_nk_from_sparse, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST_BINS * 4);
}

}  // namespace lda
