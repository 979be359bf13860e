// Exact-conditional yardstick (Section 3, Eq. 1; the split of Section 4, Eq. 3): a frozen sweep in
// which every token draws its new topic from the collapsed conditional itself instead of running a
// short MH chain towards it.  It is what the MH sweep is measured against (log-likelihood per sweep),
// not a fast path: a token costs O(K_d log K_w + log K).
//
//   p(k) ~ n_kd'(n_kw'+beta)/(n_k'+V beta)  +  alpha (n_kw'+beta)/(n_k'+V beta)      (primes: token removed)
//
// Every term is floored to a multiple of 2^-44 and the draw is the inverse CDF over these integer
// masses -- the document term's topics first (ascending), then all topics -- so the result does
// not depend on the order the terms are added in.  The second term differs between two tokens of
// a word only at the token's own topic, so its running sums over k are built once per word and
// sweep; the first term walks the document's sorted n_kd row (export.cu) and looks n_kw up in the
// word's sorted row.  One Philox word per token and sweep: counter (token, sweep, 0, 2).
#include <algorithm>

#include "lda_device.cuh"
#include "lda_internal.cuh"

namespace lda {

typedef unsigned long long ull;
constexpr double GIBBS_FIXED_ONE = 17592186044416.0;  // 2^44

__device__ __forceinline__ ull gibbs_doc_term(double beta, double Vbeta, int32_t n_kd, int32_t n_kw, int32_t n_k)
{
    const double x = __ddiv_rn(__dmul_rn((double)n_kd, __dadd_rn((double)n_kw, beta)), __dadd_rn((double)n_k, Vbeta));
    return __double2ull_rz(__dmul_rn(x, GIBBS_FIXED_ONE));
}

__device__ __forceinline__ ull gibbs_prior_term(double alpha, double beta, double Vbeta, int32_t n_kw, int32_t n_k)
{
    const double x = __ddiv_rn(__dmul_rn(alpha, __dadd_rn((double)n_kw, beta)), __dadd_rn((double)n_k, Vbeta));
    return __double2ull_rz(__dmul_rn(x, GIBBS_FIXED_ONE));
}

// word_of[i] = word of the token with document-order index i (the layout keeps tokens by word).
__global__ void k_word_of_tokens(View v, int32_t* __restrict__ word_of)
{
    for (int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; p < v.N; p += (int64_t)gridDim.x * blockDim.x) {
        int32_t lo = 0, hi = v.V;  // last word with word_off[word] <= p
        while (hi - lo > 1) {
            const int32_t mid = lo + ((hi - lo) >> 1);
            if (v.word_off[mid] <= (int32_t)p) lo = mid; else hi = mid;
        }
        word_of[v.tok_orig[p]] = lo;
    }
}

// One CTA per word: running sums over k of the smoothing term under the frozen counts.
__global__ void __launch_bounds__(256) k_gibbs_prior_prefix(View v, ull* __restrict__ prefix)
{
    extern __shared__ int32_t row_s[];  // [K] the word's n_kw as a dense row
    __shared__ ull scan_tmp[33];
    const int32_t w = blockIdx.x, K = v.K;
    for (int32_t k = threadIdx.x; k < K; k += blockDim.x) row_s[k] = 0;
    __syncthreads();
    const int32_t r0 = v.row_start[w], n = v.wk_nnz[w];
    for (int32_t j = threadIdx.x; j < n; j += blockDim.x) row_s[v.wk_topic[r0 + j]] = (int32_t)v.wk_count[r0 + j];
    __syncthreads();
    ull carry = 0;
    for (int32_t k0 = 0; k0 < K; k0 += blockDim.x) {
        const int32_t k = k0 + (int32_t)threadIdx.x;
        const ull term = k < K ? gibbs_prior_term(v.alpha, v.beta, v.Vbeta, row_s[k], v.nk[k]) : 0ull;
        ull total;
        const ull before = block_scan_excl<ull>(term, scan_tmp, total);
        if (k < K) prefix[(size_t)w * K + k] = carry + before + term;
        carry += total;
        __syncthreads();
    }
}

// n_kw[w][k] from the word's sorted row.
__device__ __forceinline__ int32_t word_count(const View& v, int32_t row0, int32_t nnz, uint32_t k)
{
    int32_t lo = 0, hi = nnz;
    while (lo < hi) {
        const int32_t mid = (lo + hi) >> 1;
        if (__ldg(v.wk_topic + row0 + mid) < k) lo = mid + 1; else hi = mid;
    }
    return (lo < nnz && __ldg(v.wk_topic + row0 + lo) == k) ? (int32_t)__ldg(v.wk_count + row0 + lo) : 0;
}

// One warp per document, a lane per token.
template <typename T>
__global__ void __launch_bounds__(256)
k_gibbs_tokens(View v, const T* __restrict__ z, const int32_t* __restrict__ word_of, const long long* __restrict__ row_off,
               const int32_t* __restrict__ dk_topic, const int32_t* __restrict__ dk_count, const ull* __restrict__ prefix,
               int32_t* __restrict__ z_new, uint2 key, uint32_t sweep)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int32_t K = v.K;
    for (int64_t d = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; d < v.D; d += warps) {
        const int32_t first = v.doc_off[d], n = v.doc_off[d + 1] - first;
        const long long e0 = row_off[d];
        const int32_t rows = (int32_t)(row_off[d + 1] - e0);
        for (int32_t j = lane; j < n; j += 32) {
            const int32_t i = first + j;
            const uint32_t z0 = (uint32_t)z[i];
            const int32_t w = word_of[i];
            const int32_t row0 = v.row_start[w], nnz = v.wk_nnz[w];
            // document term over the document's topics (ascending)
            auto doc_mass = [&](int32_t e) -> ull {
                const uint32_t k = (uint32_t)dk_topic[e0 + e];
                const int32_t own = (k == z0);
                const int32_t n_kd = dk_count[e0 + e] - own;
                if (n_kd <= 0) return 0ull;
                return gibbs_doc_term(v.beta, v.Vbeta, n_kd, word_count(v, row0, nnz, k) - own, v.nk[k] - own);
            };
            ull sum_doc = 0;
            for (int32_t e = 0; e < rows; ++e) sum_doc += doc_mass(e);
            // smoothing term: the word's running sums, set right at the token's own topic
            const ull* pre = prefix + (size_t)w * K;
            const int32_t n_zw = word_count(v, row0, nnz, z0), n_z = v.nk[z0];
            const long long delta = (long long)gibbs_prior_term(v.alpha, v.beta, v.Vbeta, n_zw - 1, n_z - 1) -
                                    (long long)gibbs_prior_term(v.alpha, v.beta, v.Vbeta, n_zw, n_z);
            const ull sum_prior = (ull)((long long)pre[K - 1] + delta);
            const ull total = sum_doc + sum_prior;
            const uint4 r = philox4x32_10(make_uint4(v.tok_base + (uint32_t)i, sweep, 0u, 2u), key);
            ull x = __umul64hi(total, (ull)r.x << 32);  // floor(total * r.x / 2^32)
            uint32_t pick = (uint32_t)(K - 1);
            if (x < sum_doc) {
                ull cum = 0;
                for (int32_t e = 0; e < rows; ++e) {
                    cum += doc_mass(e);
                    if (cum > x) { pick = (uint32_t)dk_topic[e0 + e]; break; }
                }
            } else {
                x -= sum_doc;
                int32_t lo = 0, hi = K - 1;  // first k whose running sum exceeds x
                while (lo < hi) {
                    const int32_t mid = (lo + hi) >> 1;
                    const ull c = (ull)((long long)pre[mid] + ((uint32_t)mid >= z0 ? delta : 0ll));
                    if (c > x) hi = mid; else lo = mid + 1;
                }
                pick = (uint32_t)lo;
            }
            z_new[i] = (int32_t)pick;
        }
    }
}

}  // namespace lda

using namespace lda;

int lda::gibbs_sweep(Ctx& c, int32_t iters)
{
    const View& v = c.v;
    const size_t n1 = (size_t)std::max<int64_t>(c.N, 1);
    int32_t* word_of = nullptr;
    int32_t* z_new = nullptr;
    ull* prefix = nullptr;
    int rc = LDA_OK;
    if (!tmp_alloc(c, &word_of, n1 * 4) || !tmp_alloc(c, &z_new, n1 * 4) || !tmp_alloc(c, &prefix, (size_t)c.V * c.K * 8))
        rc = LDA_ENOMEM;
    const uint2 key = make_uint2((uint32_t)c.seed, (uint32_t)(c.seed >> 32));
    if (rc == LDA_OK && c.N > 0) k_word_of_tokens<<<1184, 256, 0, c.stream>>>(v, word_of);
    for (int32_t it = 0; rc == LDA_OK && it < iters && c.N > 0; ++it) {
        DkCsr r;
        if ((rc = build_dk_csr(c, r, false))) break;  // also leaves z in document order in the record array
        k_gibbs_prior_prefix<<<c.V, 256, (size_t)c.K * 4, c.stream>>>(v, prefix);
        const int grid = (int)std::min<int64_t>(148 * 8, (c.D + 7) / 8);
        if (c.wide_topics)
            k_gibbs_tokens<int32_t><<<grid, 256, 0, c.stream>>>(v, (const int32_t*)v.rec, word_of, r.row_off, r.topic, r.count,
                                                               prefix, z_new, key, c.sweep);
        else
            k_gibbs_tokens<uint16_t><<<grid, 256, 0, c.stream>>>(v, (const uint16_t*)v.rec, word_of, r.row_off, r.topic,
                                                                r.count, prefix, z_new, key, c.sweep);
        launch_spread_assignments(c, z_new, false);
        launch_count_wk(c);
        launch_count_k(c);
        c.tables_valid = false;
            c.sweep += 1;
        if (cudaStreamSynchronize(c.stream) != cudaSuccess) rc = LDA_ECUDA;
        free_dk_csr(c, r);
    }
    if (iters > 0 && c.N == 0) c.sweep += (uint32_t)iters;
    cudaStreamSynchronize(c.stream);
    raw_free(c, word_of);
    raw_free(c, z_new);
    raw_free(c, prefix);
    if (rc == LDA_OK && cudaGetLastError() != cudaSuccess) rc = LDA_ECUDA;
    return rc;
}

void lda::set_gibbs_smem_limits()
{
    cudaFuncSetAttribute(k_gibbs_prior_prefix, cudaFuncAttributeMaxDynamicSharedMemorySize, GIBBS_MAX_K * 4);
}
