// n_kd (Eq. 12) as sorted rows in device memory: for every document the (topic, count) pairs of its
// nonzero counts, topics ascending.  The MH step never needs this form (its document pass builds
// hashed tables per tile and drops them); it is what lda_get_counts(LDA_NDK) hands out and what the
// exact-conditional sweep (gibbs.cu) walks.  Documents are packed whole into tiles of at most
// SORT_TILE tokens, sorted and run-length encoded by k_seg_count_sorted (counts.cu); a longer document
// gets a CTA of its own and a histogram over the topics.  Two passes: row sizes, a prefix sum for
// the row offsets (CUB's device scan: this path is off the sweep), then the entries.
#include <cub/device/device_scan.cuh>

#include "lda_device.cuh"
#include "lda_internal.cuh"

namespace lda {

// A document longer than a sort tile: topics counted window by window in shared memory.
// EMIT false: nnz[d] = number of distinct topics; true: the row's entries at row_off[d].
template <typename T, bool EMIT>
__global__ void __launch_bounds__(512)
k_long_doc_rows(const int32_t* __restrict__ long_docs, const int32_t* __restrict__ doc_off, const T* __restrict__ z,
                int32_t K, int32_t window, int32_t* __restrict__ nnz, const long long* __restrict__ row_off,
                int32_t* __restrict__ topic, int32_t* __restrict__ count, int* err)
{
    extern __shared__ int32_t bins[];
    __shared__ int32_t scan_tmp[33];
    const int32_t d = long_docs[blockIdx.x];
    const int32_t first = doc_off[d], n = doc_off[d + 1] - first;
    int32_t done = 0;
    for (int32_t k0 = 0; k0 < K; k0 += window) {
        const int32_t nb = min(window, K - k0);
        for (int32_t b = threadIdx.x; b < nb; b += blockDim.x) bins[b] = 0;
        __syncthreads();
        for (int32_t j = threadIdx.x; j < n; j += blockDim.x) {
            const uint32_t k = (uint32_t)z[first + j];
            if (k >= (uint32_t)K) { atomicOr(err, ERR_TOPIC_RANGE); continue; }
            const uint32_t b = k - (uint32_t)k0;
            if (b < (uint32_t)nb) atomicAdd(&bins[b], 1);
        }
        __syncthreads();
        for (int32_t b0 = 0; b0 < nb; b0 += blockDim.x) {
            const int32_t b = b0 + (int32_t)threadIdx.x;
            const int32_t c = b < nb ? bins[b] : 0;
            int32_t total;
            const int32_t pos = block_scan_excl<int32_t>(c > 0 ? 1 : 0, scan_tmp, total);
            if (EMIT && c > 0) {
                const long long at = row_off[d] + done + pos;
                topic[at] = k0 + b;
                count[at] = c;
            }
            done += total;
        }
        __syncthreads();
    }
    if (!EMIT && threadIdx.x == 0) nnz[d] = done;
}

template <typename T>
void launch_doc_rows(Ctx& c, const int32_t* tiles, int32_t n_tiles, const T* z, int32_t* nnz, const long long* row_off,
                     int32_t* topic, int32_t* count);  // counts.cu

void free_dk_csr(Ctx& c, DkCsr& r)
{
    raw_free(c, r.row_off);
    raw_free(c, r.nnz);
    raw_free(c, r.topic);
    raw_free(c, r.count);
    r = DkCsr{};
}

template <typename T>
static int build_dk_csr_t(Ctx& c, DkCsr& r, bool sizes_only)
{
    const View& v = c.v;
    const int32_t D = (int32_t)c.D;
    r = DkCsr{};
    if (!tmp_alloc(c, &r.row_off, ((size_t)D + 1) * 8) || !tmp_alloc(c, &r.nnz, ((size_t)D + 1) * 4)) {
        free_dk_csr(c, r);
        return LDA_ENOMEM;
    }
    cudaMemsetAsync(r.nnz, 0, ((size_t)D + 1) * 4, c.stream);
    // the assignments in document order, in the record array (scratch between calls)
    T* z = reinterpret_cast<T*>(v.rec);
    launch_export_assignments(c, z, sizeof(T) == 2);
    const int win = c.K < HIST_BINS ? c.K : HIST_BINS;
    if (c.n_doc_sort_tiles)
        launch_doc_rows<T>(c, c.doc_sort_tiles, c.n_doc_sort_tiles, z, r.nnz, nullptr, nullptr, nullptr);
    if (c.n_doc_sort_long)
        k_long_doc_rows<T, false><<<c.n_doc_sort_long, 512, (size_t)win * 4, c.stream>>>(
            c.doc_sort_long, v.doc_off, z, c.K, win, r.nnz, nullptr, nullptr, nullptr, v.err);
    void* temp = nullptr;
    size_t temp_bytes = 0;
    // nnz(n_kd) <= n_tokens < 2^31: the 32-bit running sum cannot overflow
    if (cub::DeviceScan::ExclusiveSum(nullptr, temp_bytes, r.nnz, r.row_off, D + 1, c.stream) != cudaSuccess ||
        !tmp_alloc(c, &temp, temp_bytes)) {
        cudaGetLastError();
        free_dk_csr(c, r);
        return LDA_ENOMEM;
    }
    const cudaError_t e = cub::DeviceScan::ExclusiveSum(temp, temp_bytes, r.nnz, r.row_off, D + 1, c.stream);
    long long total = 0;
    if (e != cudaSuccess ||
        cudaMemcpyAsync(&total, r.row_off + D, 8, cudaMemcpyDeviceToHost, c.stream) != cudaSuccess ||
        cudaStreamSynchronize(c.stream) != cudaSuccess) {
        cudaGetLastError();
        raw_free(c, temp);
        free_dk_csr(c, r);
        return LDA_ECUDA;
    }
    raw_free(c, temp);
    r.total = total;
    if (sizes_only) return LDA_OK;
    const size_t cap = (size_t)(total > 0 ? total : 1);
    if (!tmp_alloc(c, &r.topic, cap * 4) || !tmp_alloc(c, &r.count, cap * 4)) {
        free_dk_csr(c, r);
        return LDA_ENOMEM;
    }
    if (c.n_doc_sort_tiles)
        launch_doc_rows<T>(c, c.doc_sort_tiles, c.n_doc_sort_tiles, z, nullptr, r.row_off, r.topic, r.count);
    if (c.n_doc_sort_long)
        k_long_doc_rows<T, true><<<c.n_doc_sort_long, 512, (size_t)win * 4, c.stream>>>(
            c.doc_sort_long, v.doc_off, z, c.K, win, nullptr, r.row_off, r.topic, r.count, v.err);
    return LDA_OK;
}

int build_dk_csr(Ctx& c, DkCsr& r, bool sizes_only)
{
    return c.wide_topics ? build_dk_csr_t<int32_t>(c, r, sizes_only) : build_dk_csr_t<uint16_t>(c, r, sizes_only);
}

void set_export_smem_limits()
{
    cudaFuncSetAttribute(k_long_doc_rows<uint16_t, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST_BINS * 4);
    cudaFuncSetAttribute(k_long_doc_rows<uint16_t, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST_BINS * 4);
    cudaFuncSetAttribute(k_long_doc_rows<int32_t, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST_BINS * 4);
    cudaFuncSetAttribute(k_long_doc_rows<int32_t, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST_BINS * 4);
}

}  // namespace lda
