// One-time corpus layout (Section 6, item 3: token-topic pairs are sorted by
// word once, so that the tokens of a word -- and of a slice of words -- are
// contiguous).  Tokens are sorted stably by word id, so inside a word they
// stay in document order.  The sort itself uses CUB's device radix sort: it
// runs once per corpus, outside the per-sweep path.
#include <cub/device/device_radix_sort.cuh>

#include "lda_device.cuh"
#include "lda_internal.cuh"

namespace lda {

__global__ void k_check_words_iota(const int32_t* __restrict__ words, uint32_t* __restrict__ iota,
                                   int32_t n, int32_t V, int* err)
{
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n;
         i += (int64_t)gridDim.x * blockDim.x) {
        iota[i] = (uint32_t)i;
        const int32_t w = words[i];
        if (w < 0 || w >= V) atomicOr(err, ERR_WORD_RANGE);
    }
}

// word_off[w] = first position whose word is >= w (positions are word-sorted).
__global__ void k_word_offsets(const int32_t* __restrict__ sorted_words, int32_t n, int32_t V,
                               int32_t* __restrict__ word_off)
{
    const int32_t w = blockIdx.x * blockDim.x + threadIdx.x;
    if (w > V) return;
    int32_t lo = 0, hi = n;
    while (lo < hi) {
        const int32_t mid = lo + ((hi - lo) >> 1);
        if (sorted_words[mid] < w) lo = mid + 1; else hi = mid;
    }
    word_off[w] = lo;
}

// Keys of the block-major order: the block of a token is the high part of its document-order index.
__global__ void k_block_keys(const uint32_t* __restrict__ tok_orig, int32_t n, int shift,
                             uint32_t* __restrict__ keys, uint32_t* __restrict__ iota)
{
    for (int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; p < n;
         p += (int64_t)gridDim.x * blockDim.x) {
        keys[p] = tok_orig[p] >> shift;
        iota[p] = (uint32_t)p;
    }
}

// The block-major index of every token, by word-sorted position and by document-order index.
__global__ void k_block_major_maps(const uint32_t* __restrict__ order, const uint32_t* __restrict__ tok_orig,
                                   int32_t n, uint32_t* __restrict__ inv, uint32_t* __restrict__ bm_of_tok)
{
    for (int64_t m = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; m < n;
         m += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t p = order[m];
        inv[p] = (uint32_t)m;
        bm_of_tok[tok_orig[p]] = (uint32_t)m;
    }
}

int build_layout(Ctx& c, const int32_t* word_ids_dev, const int64_t* doc_off_host)
{
    const int32_t N = (int32_t)c.N, D = (int32_t)c.D, V = c.V;
    cudaStream_t st = c.stream;
    const size_t n1 = (size_t)(N > 0 ? N : 1);

    uint32_t* tok_orig = (uint32_t*)dev_alloc(c, n1 * 4);
    uint32_t* inv = (uint32_t*)dev_alloc(c, n1 * 4);
    uint32_t* bm_of_tok = (uint32_t*)dev_alloc(c, n1 * 4);
    int32_t* word_off = (int32_t*)dev_alloc(c, ((size_t)V + 1) * 4);
    int32_t* doc_off = (int32_t*)dev_alloc(c, ((size_t)D + 1) * 4);
    if (!tok_orig || !inv || !bm_of_tok || !word_off || !doc_off) return LDA_ENOMEM;

    std::vector<int32_t> doc32((size_t)D + 1);
    for (int64_t d = 0; d <= D; ++d) doc32[(size_t)d] = (int32_t)doc_off_host[d];
    if (cudaMemcpyAsync(doc_off, doc32.data(), ((size_t)D + 1) * 4, cudaMemcpyHostToDevice, st) !=
        cudaSuccess)
        return LDA_ECUDA;

    // transient buffers of the sort
    int32_t* keys_out = nullptr;
    uint32_t* iota = nullptr;
    uint32_t* keys_blk = nullptr;
    uint32_t* order = nullptr;
    void* temp = nullptr;
    void* temp2 = nullptr;
    size_t temp_bytes = 0, temp2_bytes = 0;
    int rc = LDA_OK;
    do {
        if (!tmp_alloc(c, &keys_out, n1 * 4) || !tmp_alloc(c, &iota, n1 * 4) || !tmp_alloc(c, &keys_blk, n1 * 4) ||
            !tmp_alloc(c, &order, n1 * 4)) {
            rc = LDA_ENOMEM;
            break;
        }
        if (N > 0) {
            k_check_words_iota<<<1184, 256, 0, st>>>(word_ids_dev, iota, N, V, c.v.err);
            int end_bit = 1;
            while (end_bit < 31 && (1ll << end_bit) < (long long)V) ++end_bit;
            if (cub::DeviceRadixSort::SortPairs(nullptr, temp_bytes, word_ids_dev, keys_out, iota,
                                                tok_orig, N, 0, end_bit, st) != cudaSuccess) {
                rc = LDA_ECUDA;
                break;
            }
            if (!tmp_alloc(c, &temp, temp_bytes)) {
                rc = LDA_ENOMEM;
                break;
            }
            if (cub::DeviceRadixSort::SortPairs(temp, temp_bytes, word_ids_dev, keys_out, iota,
                                                tok_orig, N, 0, end_bit, st) != cudaSuccess) {
                rc = LDA_ECUDA;
                break;
            }
            // block-major order: tokens sorted by (block of their document-order index, word-sorted
            // position); a stable sort of the positions by block
            uint32_t* keys_tmp = reinterpret_cast<uint32_t*>(keys_out);  // the word keys are no longer needed
            k_block_keys<<<1184, 256, 0, st>>>(tok_orig, N, c.block_shift, keys_blk, iota);
            int blk_bits = 1;
            while (blk_bits < 32 && (((long long)N - 1) >> c.block_shift) >= (1ll << blk_bits)) ++blk_bits;
            if (cub::DeviceRadixSort::SortPairs(nullptr, temp2_bytes, keys_blk, keys_tmp, iota, order, N, 0,
                                                blk_bits, st) != cudaSuccess) {
                rc = LDA_ECUDA;
                break;
            }
            if (!tmp_alloc(c, &temp2, temp2_bytes)) {
                rc = LDA_ENOMEM;
                break;
            }
            // the word offsets are taken from keys_out first: the next sort overwrites it
            k_word_offsets<<<(V + 1 + 255) / 256, 256, 0, st>>>(keys_out, N, V, word_off);
            if (cub::DeviceRadixSort::SortPairs(temp2, temp2_bytes, keys_blk, keys_tmp, iota, order, N, 0,
                                                blk_bits, st) != cudaSuccess) {
                rc = LDA_ECUDA;
                break;
            }
            k_block_major_maps<<<1184, 256, 0, st>>>(order, tok_orig, N, inv, bm_of_tok);
        } else {
            k_word_offsets<<<(V + 1 + 255) / 256, 256, 0, st>>>(keys_out, N, V, word_off);
        }
        if (cudaStreamSynchronize(st) != cudaSuccess || cudaGetLastError() != cudaSuccess)
            rc = LDA_ECUDA;
    } while (0);
    raw_free(c, keys_out);
    raw_free(c, iota);
    raw_free(c, keys_blk);
    raw_free(c, order);
    raw_free(c, temp);
    raw_free(c, temp2);
    if (rc != LDA_OK) return rc;
    c.v.inv = inv;
    c.v.bm_of_tok = bm_of_tok;
    c.v.tok_orig = tok_orig;
    c.v.word_off = word_off;
    c.v.doc_off = doc_off;
    return LDA_OK;
}

}  // namespace lda
