// Document-sharded data parallelism (Section 6, "Parameter Server and Data Placement": the
// documents are partitioned over the workers, the word-topic table is shared and the workers'
// updates are aggregated after sampling).  A context may hold one shard of the documents: its n_kd
// stays local, n_kw and n_k have to be the sums over all shards before the next sweep.  The
// exchange format is n_kw as a dense V x K matrix of int32 in device memory -- a plain buffer a
// collective library can add up across GPUs:
//   after lda_init / lda_sweep:  lda_word_counts_to_dense()   (the shard's own counts)
//   all-reduce (sum) of the matrix over the shards, by the caller
//   lda_word_counts_from_dense()  (rows, dense rows and n_k rebuilt from the summed matrix)
// No kernel here reads another GPU's memory; the reduction is the caller's (NCCL) call.
#include <algorithm>

#include "lda_device.cuh"
#include "lda_internal.cuh"

namespace lda {

// One warp per word: the sorted row scattered into the word's line of the matrix (cleared before).
__global__ void __launch_bounds__(256)
k_rows_to_dense(View v, int32_t* __restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < v.V; w += warps) {
        const int32_t r0 = v.row_start[w], n = v.wk_nnz[w];
        int32_t* line = out + (size_t)w * v.K;
        for (int32_t j = lane; j < n; j += 32) line[v.wk_topic[r0 + j]] = (int32_t)v.wk_count[r0 + j];
    }
}

// One CTA per word: the word's line of the matrix -> sorted row (and dense row, if the word has one).
__global__ void __launch_bounds__(256)
k_rows_from_dense(View v, const int32_t* __restrict__ in)
{
    __shared__ int32_t scan_tmp[33];
    const int32_t w = blockIdx.x, K = v.K;
    const int32_t* line = in + (size_t)w * K;
    const int32_t out0 = v.row_start[w], cap = v.row_start[w + 1] - out0;
    const int32_t slot = v.dense_slot[w];
    int32_t* dense = slot >= 0 ? v.dense_rows + (size_t)slot * v.dense_stride : nullptr;
    int32_t done = 0;
    for (int32_t k0 = 0; k0 < K; k0 += blockDim.x) {
        const int32_t k = k0 + (int32_t)threadIdx.x;
        const int32_t n = k < K ? line[k] : 0;
        if (n < 0) atomicOr(v.err, ERR_COUNT_ZERO);
        if (dense && k < K) dense[k] = n;
        int32_t total;
        const int32_t pos = done + block_scan_excl<int32_t>(n > 0 ? 1 : 0, scan_tmp, total);
        if (n > 0) {
            if (pos < cap) {
                v.wk_topic[out0 + pos] = (uint32_t)k;
                v.wk_count[out0 + pos] = (uint32_t)n;
            } else {
                atomicOr(v.err, ERR_ROW_OVERFLOW);  // more nonzeros than the word has tokens over all shards
            }
        }
        done += total;
        __syncthreads();
    }
    if (threadIdx.x == 0) v.wk_nnz[w] = min(done, cap);
}

int launch_word_counts_to_dense(Ctx& c, int32_t* nwk_dev)
{
    cudaMemsetAsync(nwk_dev, 0, (size_t)c.V * c.K * 4, c.stream);
    const int grid = (int)std::min<int64_t>(148 * 16, ((int64_t)c.V * 32 + 255) / 256);
    k_rows_to_dense<<<grid, 256, 0, c.stream>>>(c.v, nwk_dev);
    return 1;
}

int launch_word_counts_from_dense(Ctx& c, const int32_t* nwk_dev)
{
    k_rows_from_dense<<<c.V, 256, 0, c.stream>>>(c.v, nwk_dev);
    return 1 + launch_count_k(c);  // n_k = column sums of the rows just written
}

}  // namespace lda
