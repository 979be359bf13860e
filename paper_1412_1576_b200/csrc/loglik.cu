// Collapsed joint log-likelihood log p(w, z), split as in Figure 11 into a word
// part and a document part (Dirichlet-multinomial closed form):
//   word = K lgamma(V beta) + sum_{n_kw>0} [lgamma(n_kw+beta) - lgamma(beta)] - sum_k lgamma(n_k + V beta)
//   doc  = D lgamma(K alpha) + sum_{n_kd>0} [lgamma(n_kd+alpha) - lgamma(alpha)] - sum_d lgamma(n_d + K alpha)
// Each CTA writes one partial sum; the host adds the partials in a fixed order.
#include <cmath>

#include "lda_device.cuh"
#include "lda_internal.cuh"

namespace lda {

constexpr int LL_BLOCKS = 592;
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

__global__ void __launch_bounds__(256) k_ll_doc(View v, double lg_alpha, double* __restrict__ out)
{
    __shared__ double tmp[32];
    __shared__ double small[LL_TABLE];
    fill_ll_table(small, v.alpha, lg_alpha);
    const int warps = (gridDim.x * blockDim.x) >> 5, lane = threadIdx.x & 31;
    const uint32_t cmask = (1u << v.count_bits) - 1u;
    double s = 0.0;
    for (int32_t d = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; d < v.D; d += warps) {
        // a document's table: four slots per token, read 16 bytes at a time
        static_assert(DK_SLOTS_PER_TOKEN == 4, "one 16-byte read per token of the document");
        const int32_t d0 = v.doc_off[d], len = v.doc_off[d + 1] - d0;
        const uint4* tab = reinterpret_cast<const uint4*>(v.dk_slots) + (size_t)d0;
        for (int32_t j = lane; j < len; j += 32) {
            const uint4 q = __ldcs(tab + j);
            const uint32_t es[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (es[u] != DK_EMPTY) {
                    const uint32_t c = es[u] & cmask;
                    s += c < (uint32_t)LL_TABLE ? small[c] : lgamma((double)c + v.alpha) - lg_alpha;
                }
            }
        }
        if (lane == 0) s -= lgamma((double)(v.doc_off[d + 1] - d0) + v.Kalpha);
    }
    s = block_reduce_sum<double>(s, tmp);
    if (threadIdx.x == 0) out[blockIdx.x] = s;
}

int launch_loglik(Ctx& c, double* out3_host)
{
    double* part = c.red;  // [2 * LL_BLOCKS]
    k_ll_word<<<LL_BLOCKS, 256, 0, c.stream>>>(c.v, std::lgamma(c.beta), part);
    k_ll_doc<<<LL_BLOCKS, 256, 0, c.stream>>>(c.v, std::lgamma(c.alpha), part + LL_BLOCKS);
    std::vector<double> h(2 * LL_BLOCKS);
    if (cudaMemcpyAsync(h.data(), part, sizeof(double) * 2 * LL_BLOCKS, cudaMemcpyDeviceToHost,
                        c.stream) != cudaSuccess ||
        cudaStreamSynchronize(c.stream) != cudaSuccess)
        return -1;
    double lw = (double)c.K * std::lgamma(c.v.Vbeta), ld = (double)c.D * std::lgamma(c.v.Kalpha);
    for (int i = 0; i < LL_BLOCKS; ++i) lw += h[i];
    for (int i = 0; i < LL_BLOCKS; ++i) ld += h[LL_BLOCKS + i];
    out3_host[0] = lw + ld;
    out3_host[1] = lw;
    out3_host[2] = ld;
    return 2;
}

}  // namespace lda
