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

// Tables of the document part in device memory, filled once per corpus: [0, LL_TABLE) holds
// lgamma(c + alpha) - lgamma(alpha), [LL_TABLE, 2 LL_TABLE) holds lgamma(n + K alpha).
__global__ void k_ll_fill_tables(View v, double lg_alpha, double* __restrict__ tab)
{
    for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < LL_TABLE; c += gridDim.x * blockDim.x) {
        tab[c] = lgamma((double)c + v.alpha) - lg_alpha;
        tab[LL_TABLE + c] = lgamma((double)c + v.Kalpha);
    }
}

// lgamma() for the rare count beyond the tables, kept out of line so that the kernel below fits the
// register budget of a full multiprocessor.
__device__ __noinline__ double lgamma_out_of_line(double x) { return lgamma(x); }

// Document part.  n_kd is not kept between sweeps (the MH step builds it per tile of documents
// and drops it), so it is built here the same way and by the same shape of kernel as pass 2 of the
// MH step: one CTA per tile of whole documents, a thread owns DOC_TILE_ROUNDS tokens, inserts their
// topics into the documents' hashed tables in shared memory, and the CTA then adds up
// lgamma(n_kd + alpha) - lgamma(alpha) over the filled slots and -lgamma(n_d + K alpha) per document.
// One partial sum per tile (a second kernel adds them in a fixed order) and the number of filled
// slots, nnz(n_kd).
template <typename T, int THREADS>
__global__ void __launch_bounds__(THREADS, 1536 / THREADS)
k_ll_doc_tiles(View v, const int32_t* __restrict__ tiles, double lg_alpha, const double* __restrict__ tab,
               double* __restrict__ tile_part, uint32_t* __restrict__ tile_nnz)
{
    constexpr int cap = DOC_TILE_ROUNDS * THREADS;
    extern __shared__ __align__(16) uint32_t doc_smem[];
    __shared__ double tmp[32];
    uint32_t* slots = doc_smem;                                                            // [DK_SLOTS_PER_TOKEN * cap]
    int32_t* soff = reinterpret_cast<int32_t*>(slots + DK_SLOTS_PER_TOKEN * cap);          // [cap + 1]
    const int tid = threadIdx.x;
    const int32_t s0 = tiles[2 * blockIdx.x], s1 = tiles[2 * blockIdx.x + 1];
    const int32_t nseg = s1 - s0;
    const int32_t base = v.doc_off[s0];
    const int32_t cnt = v.doc_off[s1] - base;
    const T* zbm = reinterpret_cast<const T*>(v.zbm);
    uint32_t z[DOC_TILE_ROUNDS];
#pragma unroll
    for (int r = 0; r < DOC_TILE_ROUNDS; ++r) {
        const int j = tid + r * THREADS;
        z[r] = 0;
        if (j < cnt) z[r] = (uint32_t)__ldcg(zbm + 2 * (size_t)__ldcs(v.bm_of_tok + base + j));
    }
    for (int j = tid; j <= nseg; j += THREADS) soff[j] = v.doc_off[s0 + j] - base;
    const uint4 empty4 = make_uint4(DK_EMPTY, DK_EMPTY, DK_EMPTY, DK_EMPTY);
    for (int j = tid; j < cnt * (DK_SLOTS_PER_TOKEN / 4); j += THREADS) reinterpret_cast<uint4*>(slots)[j] = empty4;
    __syncthreads();
#pragma unroll
    for (int r = 0; r < DOC_TILE_ROUNDS; ++r) {
        const int j = tid + r * THREADS;
        if (j < cnt) {
            int lo = 0, hi = nseg;  // last document with soff[doc] <= j
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (soff[mid] <= j) lo = mid; else hi = mid;
            }
            const int32_t first = soff[lo], len = soff[lo + 1] - first;
            if (z[r] >= (uint32_t)v.K) atomicOr(v.err, ERR_TOPIC_RANGE);
            else if (dk_insert(slots + DK_SLOTS_PER_TOKEN * first, DK_SLOTS_PER_TOKEN * (uint32_t)len, z[r],
                               v.count_bits) == DK_EMPTY)
                atomicOr(v.err, ERR_ROW_OVERFLOW);
        }
    }
    __syncthreads();
    const uint32_t cmask = (1u << v.count_bits) - 1u;
    double s = 0.0;
    uint32_t filled = 0;
    for (int j = tid; j < cnt; j += THREADS) {  // a token's worth of slots at a time
        const uint4 e4 = reinterpret_cast<const uint4*>(slots)[j];
        const uint32_t e[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (e[q] != DK_EMPTY) {
                const uint32_t c = e[q] & cmask;
                s += c < (uint32_t)LL_TABLE ? __ldg(tab + c) : lgamma_out_of_line((double)c + v.alpha) - lg_alpha;
                ++filled;
            }
        }
    }
    for (int d = tid; d < nseg; d += THREADS) {
        const int32_t len = soff[d + 1] - soff[d];
        if (len > 0) s -= len < LL_TABLE ? __ldg(tab + LL_TABLE + len) : lgamma_out_of_line((double)len + v.Kalpha);
    }
    s = block_reduce_sum<double>(s, tmp);
    if (tid == 0) tile_part[blockIdx.x] = s;
    __syncthreads();
    filled = block_reduce_sum<uint32_t>(filled, reinterpret_cast<uint32_t*>(tmp));
    if (tid == 0) tile_nnz[blockIdx.x] = filled;
}

// Adds the tiles' partial sums: CTA b takes the b-th run of `per` consecutive tiles, always in the same order.
__global__ void __launch_bounds__(256) k_ll_sum_tiles(const double* __restrict__ tile_part,
                                                      const uint32_t* __restrict__ tile_nnz, int32_t n_tiles, int32_t per,
                                                      double* __restrict__ out, unsigned long long* __restrict__ nnz_out)
{
    __shared__ double tmp[32];
    const int32_t t0 = blockIdx.x * per, t1 = min(n_tiles, t0 + per);
    double s = 0.0;
    unsigned long long filled = 0;
    for (int32_t t = t0 + threadIdx.x; t < t1; t += blockDim.x) {
        s += tile_part[t];
        filled += tile_nnz[t];
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

constexpr int LL_TILE_SUMS = 1024;  // partial sums the tiles' sums are folded into

static int long_ll_grid(const Ctx& c) { return std::max(1, std::min<int>(c.n_long_docs, LL_BLOCKS)); }

template <typename T>
static void launch_ll_tiles_t(Ctx& c, size_t smem, double lg_alpha)
{
    switch (c.doc_threads) {
        case 128: k_ll_doc_tiles<T, 128><<<c.n_doc_tiles, 128, smem, c.stream>>>(c.v, c.doc_tiles, lg_alpha, c.ll_tab, c.ll_tile_part, c.ll_tile_nnz); break;
        case 256: k_ll_doc_tiles<T, 256><<<c.n_doc_tiles, 256, smem, c.stream>>>(c.v, c.doc_tiles, lg_alpha, c.ll_tab, c.ll_tile_part, c.ll_tile_nnz); break;
        case 512: k_ll_doc_tiles<T, 512><<<c.n_doc_tiles, 512, smem, c.stream>>>(c.v, c.doc_tiles, lg_alpha, c.ll_tab, c.ll_tile_part, c.ll_tile_nnz); break;
        default: k_ll_doc_tiles<T, 1024><<<c.n_doc_tiles, 1024, smem, c.stream>>>(c.v, c.doc_tiles, lg_alpha, c.ll_tab, c.ll_tile_part, c.ll_tile_nnz); break;
    }
}
static void launch_ll_tiles(Ctx& c, size_t smem, double lg_alpha)
{
    if (c.wide_topics) launch_ll_tiles_t<int32_t>(c, smem, lg_alpha);
    else launch_ll_tiles_t<uint16_t>(c, smem, lg_alpha);
}

// Queues the document part: partial sums to part[0 .. number returned), nnz(n_kd) to *nnz_dev (cleared here).
static int queue_doc_part(Ctx& c, double* part, unsigned long long* nnz_dev)
{
    cudaMemsetAsync(nnz_dev, 0, 8, c.stream);
    const double lg_alpha = std::lgamma(c.alpha);
    int n = 0;
    if (c.n_doc_tiles) {
        if (!c.ll_tables_ready) {
            k_ll_fill_tables<<<2, 256, 0, c.stream>>>(c.v, lg_alpha, c.ll_tab);
            c.ll_tables_ready = true;
        }
        const size_t smem = doc_tile_smem_bytes(c.doc_tile);
        launch_ll_tiles(c, smem, lg_alpha);
        const int per = (c.n_doc_tiles + LL_TILE_SUMS - 1) / LL_TILE_SUMS;
        const int g = (c.n_doc_tiles + per - 1) / per;
        k_ll_sum_tiles<<<g, 256, 0, c.stream>>>(c.ll_tile_part, c.ll_tile_nnz, c.n_doc_tiles, per, part, nnz_dev);
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
    return 2 + (c.n_doc_tiles ? 2 : 0) + (c.n_long_docs ? 1 : 0);
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
    cudaFuncSetAttribute(k_ll_doc_tiles<uint16_t, 1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, doc_bytes);
    cudaFuncSetAttribute(k_ll_doc_tiles<int32_t, 1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, doc_bytes);
}

}  // namespace lda
