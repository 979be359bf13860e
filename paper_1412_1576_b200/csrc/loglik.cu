// Collapsed joint log-likelihood log p(w, z), split as in Figure 11 into a word
// part and a document part (Dirichlet-multinomial closed form):
//   word = K lgamma(V beta) + sum_{n_kw>0} [lgamma(n_kw+beta) - lgamma(beta)] - sum_k lgamma(n_k + V beta)
//   doc  = D lgamma(K alpha) + sum_{n_kd>0} [lgamma(n_kd+alpha) - lgamma(alpha)] - sum_d lgamma(n_d + K alpha)
// Each CTA writes one partial sum; the host adds the partials in a fixed order.
#include <algorithm>
#include <cmath>

#include "lda_device.cuh"
#include "lda_internal.cuh"

namespace lda {

constexpr int LL_BLOCKS = LL_WORD_PARTIALS;
// Counts below this take lgamma(count + prior) - lgamma(prior) from a table in shared memory that
// every CTA fills with the same expression: same values as calling lgamma() per entry.
constexpr int LL_TABLE = 512;

__device__ __forceinline__ void fill_ll_table(double* tab, double prior, double lg_prior)
{
    for (int c = threadIdx.x; c < LL_TABLE; c += blockDim.x) tab[c] = lgamma((double)c + prior) - lg_prior;
    __syncthreads();
}

__global__ void __launch_bounds__(256) k_ll_word(View v, double lg_beta, double* __restrict__ out)
{
    __shared__ double tmp[32];
    __shared__ double small[LL_TABLE];
    fill_ll_table(small, v.beta, lg_beta);
    const int warps = (gridDim.x * blockDim.x) >> 5, lane = threadIdx.x & 31;
    double s = 0.0;
    for (int32_t w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < v.V; w += warps) {
        const int32_t r0 = v.row_start[w], n = v.wk_nnz[w];
        for (int32_t j = lane; j < n; j += 32) {
            const uint32_t c = v.wk_count[r0 + j];
            s += c < (uint32_t)LL_TABLE ? small[c] : lgamma((double)c + v.beta) - lg_beta;
        }
    }
    for (int32_t k = blockIdx.x * blockDim.x + threadIdx.x; k < v.K; k += gridDim.x * blockDim.x)
        s -= lgamma((double)v.nk[k] + v.Vbeta);
    s = block_reduce_sum<double>(s, tmp);
    if (threadIdx.x == 0) out[blockIdx.x] = s;
}

__global__ void k_sum_nnz(const int32_t* __restrict__ a, int64_t n, unsigned long long* out)
{
    __shared__ unsigned long long tmp[32];
    unsigned long long s = 0;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        s += (unsigned long long)a[i];
    s = block_reduce_sum<unsigned long long>(s, tmp);
    if (threadIdx.x == 0 && s) atomicAdd(out, s);
}

// Document part.  n_kd is not kept between sweeps (the MH step builds it per tile of documents
// and drops it), so it is built here the same way: a CTA takes tiles of whole documents in turns
// (tile t, t + gridDim.x, ...: a fixed assignment, so a CTA's partial sum is the same on every
// run), inserts the tile's topics into the documents' hashed tables in shared memory, and adds up
// lgamma(n_kd + alpha) - lgamma(alpha) over the filled slots and -lgamma(n_d + K alpha) per document.
// It also counts the filled slots: nnz(n_kd).
template <typename T>
__global__ void __launch_bounds__(1024)
k_ll_doc_tiles(View v, const int32_t* __restrict__ tiles, int32_t n_tiles, int32_t cap, double lg_alpha,
               double* __restrict__ out, unsigned long long* __restrict__ nnz_out)
{
    extern __shared__ __align__(16) uint32_t doc_smem[];  // carved up for tiles of `cap` tokens
    __shared__ double tmp[32];
    __shared__ double small[LL_TABLE];
    uint32_t* slots = doc_smem;
    int32_t* soff = reinterpret_cast<int32_t*>(slots + DK_SLOTS_PER_TOKEN * cap);
    uint32_t* topic = reinterpret_cast<uint32_t*>(soff + cap + 1);
    __shared__ double by_len[LL_TABLE];  // lgamma(n_d + K alpha) for documents shorter than LL_TABLE tokens
    fill_ll_table(small, v.alpha, lg_alpha);
    for (int c = threadIdx.x; c < LL_TABLE; c += blockDim.x) by_len[c] = lgamma((double)c + v.Kalpha);
    __syncthreads();
    const T* zbm = reinterpret_cast<const T*>(v.zbm);
    const int tid = threadIdx.x;
    const uint32_t cmask = (1u << v.count_bits) - 1u;
    double s = 0.0;
    unsigned long long filled = 0;
    // A thread's tokens of a tile (cap = DOC_TILE_ROUNDS x blockDim.x): their block-major indices are
    // read one tile ahead, so that a tile starts with its gathers already issued side by side.
    uint32_t bm[DOC_TILE_ROUNDS];
    auto tile_range = [&](int32_t t, int32_t& s0, int32_t& s1, int32_t& base, int32_t& cnt) {
        s0 = tiles[2 * t];
        s1 = tiles[2 * t + 1];
        base = v.doc_off[s0];
        cnt = v.doc_off[s1] - base;
    };
    auto read_bm = [&](int32_t base, int32_t cnt) {
#pragma unroll
        for (int r = 0; r < DOC_TILE_ROUNDS; ++r) {
            const int j = tid + r * (int)blockDim.x;
            bm[r] = j < cnt ? __ldcs(v.bm_of_tok + base + j) : 0u;
        }
    };
    int32_t s0 = 0, s1 = 0, base = 0, cnt = 0;
    if ((int32_t)blockIdx.x < n_tiles) {
        tile_range(blockIdx.x, s0, s1, base, cnt);
        read_bm(base, cnt);
    }
    for (int32_t t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        const int32_t nseg = s1 - s0;
        const int32_t first_doc = s0, tile_base = base, tile_cnt = cnt;
        uint32_t zt[DOC_TILE_ROUNDS];
#pragma unroll
        for (int r = 0; r < DOC_TILE_ROUNDS; ++r) {
            const int j = tid + r * (int)blockDim.x;
            zt[r] = j < tile_cnt ? (uint32_t)__ldcg(zbm + 2 * (size_t)bm[r]) : 0u;
        }
        if (t + (int32_t)gridDim.x < n_tiles) {
            tile_range(t + gridDim.x, s0, s1, base, cnt);
            read_bm(base, cnt);
        }
#pragma unroll
        for (int r = 0; r < DOC_TILE_ROUNDS; ++r) {
            const int j = tid + r * (int)blockDim.x;
            if (j < tile_cnt) topic[j] = zt[r];
        }
        for (int j = tid; j <= nseg; j += blockDim.x) soff[j] = v.doc_off[first_doc + j] - tile_base;
        for (int j = tid; j < DK_SLOTS_PER_TOKEN * tile_cnt; j += blockDim.x) slots[j] = DK_EMPTY;
        __syncthreads();
        // one warp per document: its lanes insert the document's tokens
        const int lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
        for (int d = warp; d < nseg; d += nwarps) {
            const int32_t first = soff[d], len = soff[d + 1] - first;
            for (int j = first + lane; j < first + len; j += 32) {
                const uint32_t k = topic[j];
                if (k >= (uint32_t)v.K) atomicOr(v.err, ERR_TOPIC_RANGE);
                else if (dk_insert(slots + DK_SLOTS_PER_TOKEN * first, DK_SLOTS_PER_TOKEN * (uint32_t)len, k,
                                   v.count_bits) == DK_EMPTY)
                    atomicOr(v.err, ERR_ROW_OVERFLOW);
            }
            if (lane == 0 && len > 0) s -= len < LL_TABLE ? by_len[len] : lgamma((double)len + v.Kalpha);
        }
        __syncthreads();
        for (int j = tid; j < DK_SLOTS_PER_TOKEN * tile_cnt; j += blockDim.x) {
            const uint32_t e = slots[j];
            if (e != DK_EMPTY) {
                const uint32_t c = e & cmask;
                s += c < (uint32_t)LL_TABLE ? small[c] : lgamma((double)c + v.alpha) - lg_alpha;
                ++filled;
            }
        }
        __syncthreads();
    }
    s = block_reduce_sum<double>(s, tmp);
    if (threadIdx.x == 0) out[blockIdx.x] = s;
    __syncthreads();
    filled = block_reduce_sum<unsigned long long>(filled, reinterpret_cast<unsigned long long*>(tmp));
    if (threadIdx.x == 0 && filled) atomicAdd(nnz_out, filled);
}

// Documents longer than a tile: a CTA takes them in turns, with the table in the document's range
// of the scratch slots in device memory (the same scratch the MH step uses for these documents).
template <typename T>
__global__ void __launch_bounds__(512)
k_ll_doc_long(View v, const int32_t* __restrict__ long_docs, int32_t n_long, double lg_alpha,
              double* __restrict__ out, unsigned long long* __restrict__ nnz_out)
{
    __shared__ double tmp[32];
    __shared__ double small[LL_TABLE];
    fill_ll_table(small, v.alpha, lg_alpha);
    const T* zbm = reinterpret_cast<const T*>(v.zbm);
    const uint32_t cmask = (1u << v.count_bits) - 1u;
    double s = 0.0;
    unsigned long long filled = 0;
    for (int32_t i = blockIdx.x; i < n_long; i += gridDim.x) {
        const int32_t d = long_docs[i];
        const int32_t first = v.doc_off[d], cnt = v.doc_off[d + 1] - first;
        const uint32_t cap = DK_SLOTS_PER_TOKEN * (uint32_t)cnt;
        uint32_t* tab = v.dk_slots + v.long_slot_off[i];
        for (uint32_t j = threadIdx.x; j < cap; j += blockDim.x) tab[j] = DK_EMPTY;
        __syncthreads();
        for (int j = threadIdx.x; j < cnt; j += blockDim.x) {
            const uint32_t k = (uint32_t)zbm[2 * (size_t)v.bm_of_tok[first + j]];
            if (k >= (uint32_t)v.K) atomicOr(v.err, ERR_TOPIC_RANGE);
            else if (dk_insert(tab, cap, k, v.count_bits) == DK_EMPTY) atomicOr(v.err, ERR_ROW_OVERFLOW);
        }
        __syncthreads();
        for (uint32_t j = threadIdx.x; j < cap; j += blockDim.x) {
            const uint32_t e = tab[j];
            if (e != DK_EMPTY) {
                const uint32_t c = e & cmask;
                s += c < (uint32_t)LL_TABLE ? small[c] : lgamma((double)c + v.alpha) - lg_alpha;
                ++filled;
            }
        }
        if (threadIdx.x == 0) s -= lgamma((double)cnt + v.Kalpha);
        __syncthreads();
    }
    s = block_reduce_sum<double>(s, tmp);
    if (threadIdx.x == 0) out[blockIdx.x] = s;
    __syncthreads();
    filled = block_reduce_sum<unsigned long long>(filled, reinterpret_cast<unsigned long long*>(tmp));
    if (threadIdx.x == 0 && filled) atomicAdd(nnz_out, filled);
}

// Grids of the document part: as many CTAs as the GPU holds at once (a CTA that had to wait for a
// free slot would run its whole share of the tiles after the others, at low occupancy), each taking
// tiles in turns.
template <typename T>
static int doc_ll_resident(const Ctx& c)
{
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_ll_doc_tiles<T>, c.doc_threads,
                                                      doc_tile_smem_bytes(c.doc_tile)) != cudaSuccess || per_sm < 1)
        per_sm = 1;
    return c.n_sm * per_sm;
}
static int doc_ll_grid(const Ctx& c)
{
    const int resident = c.wide_topics ? doc_ll_resident<int32_t>(c) : doc_ll_resident<uint16_t>(c);
    return std::max(1, std::min<int>(c.n_doc_tiles, resident));
}
static int long_ll_grid(const Ctx& c) { return std::max(1, std::min<int>(c.n_long_docs, LL_BLOCKS)); }

// Queues the document part: partial sums to part[0 .. number returned), nnz(n_kd) to *nnz_dev (cleared here).
static int queue_doc_part(Ctx& c, double* part, unsigned long long* nnz_dev)
{
    cudaMemsetAsync(nnz_dev, 0, 8, c.stream);
    const double lg_alpha = std::lgamma(c.alpha);
    int n = 0;
    if (c.n_doc_tiles) {
        const int g = std::min(doc_ll_grid(c), LL_DOC_PARTIALS - LL_BLOCKS);
        const size_t smem = doc_tile_smem_bytes(c.doc_tile);
        if (c.wide_topics)
            k_ll_doc_tiles<int32_t><<<g, c.doc_threads, smem, c.stream>>>(c.v, c.doc_tiles, c.n_doc_tiles, c.doc_tile,
                                                                         lg_alpha, part, nnz_dev);
        else
            k_ll_doc_tiles<uint16_t><<<g, c.doc_threads, smem, c.stream>>>(c.v, c.doc_tiles, c.n_doc_tiles, c.doc_tile,
                                                                          lg_alpha, part, nnz_dev);
        n += g;
    }
    if (c.n_long_docs) {
        const int g = long_ll_grid(c);
        if (c.wide_topics)
            k_ll_doc_long<int32_t><<<g, 512, 0, c.stream>>>(c.v, c.long_docs, c.n_long_docs, lg_alpha, part + n, nnz_dev);
        else
            k_ll_doc_long<uint16_t><<<g, 512, 0, c.stream>>>(c.v, c.long_docs, c.n_long_docs, lg_alpha, part + n, nnz_dev);
        n += g;
    }
    return n;
}

int launch_loglik(Ctx& c, double* out3_host)
{
    double* part = c.red;  // [LL_WORD_PARTIALS + LL_DOC_PARTIALS]
    k_ll_word<<<LL_BLOCKS, 256, 0, c.stream>>>(c.v, std::lgamma(c.beta), part);
    const int n_doc = queue_doc_part(c, part + LL_BLOCKS, reinterpret_cast<unsigned long long*>(c.red_i) + 1);
    std::vector<double> h((size_t)LL_BLOCKS + n_doc);
    if (cudaMemcpyAsync(h.data(), part, sizeof(double) * h.size(), cudaMemcpyDeviceToHost, c.stream) != cudaSuccess ||
        cudaStreamSynchronize(c.stream) != cudaSuccess)
        return -1;
    // every document with tokens contributes lgamma(K alpha) - lgamma(n_d + K alpha); an empty one nothing
    double lw = (double)c.K * std::lgamma(c.v.Vbeta), ld = (double)c.n_nonempty_docs * std::lgamma(c.v.Kalpha);
    for (int i = 0; i < LL_BLOCKS; ++i) lw += h[i];
    for (int i = 0; i < n_doc; ++i) ld += h[LL_BLOCKS + i];
    out3_host[0] = lw + ld;
    out3_host[1] = lw;
    out3_host[2] = ld;
    return 2 + (c.n_doc_tiles ? 1 : 0) + (c.n_long_docs ? 1 : 0);
}

// nnz(n_kw) and nnz(n_kd) of the current assignments (the latter by the document part's kernels).
int launch_count_nnz(Ctx& c, int64_t* nnz_wk_host, int64_t* nnz_dk_host)
{
    unsigned long long* acc = (unsigned long long*)c.red_i;
    cudaMemsetAsync(acc, 0, 8, c.stream);
    k_sum_nnz<<<296, 256, 0, c.stream>>>(c.v.wk_nnz, c.V, acc);
    queue_doc_part(c, c.red + LL_BLOCKS, acc + 1);
    unsigned long long h[2] = {0, 0};
    cudaMemcpyAsync(h, acc, 16, cudaMemcpyDeviceToHost, c.stream);
    cudaStreamSynchronize(c.stream);
    *nnz_wk_host = (int64_t)h[0];
    *nnz_dk_host = (int64_t)h[1];
    return 3;
}

void set_loglik_smem_limits()
{
    const int doc_bytes = (int)doc_tile_smem_bytes(DOC_TILE_MAX);
    cudaFuncSetAttribute(k_ll_doc_tiles<uint16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, doc_bytes);
    cudaFuncSetAttribute(k_ll_doc_tiles<int32_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, doc_bytes);
}

}  // namespace lda
