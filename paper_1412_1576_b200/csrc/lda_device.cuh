// Device-side helpers: Philox4x32-10, range scaling, block/warp scans.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace lda {

// Philox4x32 with 10 rounds (Salmon et al., SC'11): counter-based, so a random
// word depends only on (seed, token, sweep, step) and not on which thread asks.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}

// floor(r * n / 2^32): a 32-bit random word mapped to {0..n-1}.
__device__ __forceinline__ uint32_t scale_to_range(uint32_t r, uint32_t n) { return __umulhi(r, n); }

__device__ __forceinline__ int bit_length(unsigned long long x) { return 64 - __clzll((long long)x); }

// --- n_kd tables --------------------------------------------------------------------------------
// Document d owns slots [t0, t1) = [2*doc_off[d], 2*doc_off[d+1]) of one global slot array (twice
// its length, so the load factor stays <= 0.5; Section 5, fn. 5).  A slot is
// (topic << count_bits) | count, or DK_EMPTY_SLOT.  The table is bucketed by aligned groups of
// four slots (one 16-byte read): topic k starts at group DkProbe::first() and tries the group's
// slots that lie inside [t0, t1) in order, then the next group, wrapping to the table's first
// group.  An empty slot met on the way means "absent".
constexpr uint32_t DK_EMPTY_SLOT = 0xFFFFFFFFu;
constexpr uint32_t DK_HASH_MULT = 0x9E3779B1u;

struct DkProbe {
    uint32_t t0, t1;          // the table's slot range
    uint32_t g_first, g_cnt;  // first group (slot index / 4) and number of groups it touches
    __device__ __forceinline__ DkProbe(uint32_t doc_first_token, uint32_t doc_len)
        : t0(2u * doc_first_token), t1(2u * (doc_first_token + doc_len))
    {
        g_first = t0 >> 2;
        g_cnt = ((t1 - 1u) >> 2) - g_first + 1u;
    }
    __device__ __forceinline__ uint32_t first(uint32_t k) const { return g_first + __umulhi(k * DK_HASH_MULT, g_cnt); }
    __device__ __forceinline__ uint32_t next(uint32_t g) const { return g + 1u - g_first == g_cnt ? g_first : g + 1u; }
    __device__ __forceinline__ bool inside(uint32_t slot) const { return slot >= t0 && slot < t1; }
};

// Looks topic k up in one group of four slots `q` (group index g).  Returns true when the search
// is over (found, or an empty slot proves absence) and sets `entry` (0 when absent).
__device__ __forceinline__ bool dk_match_group(const DkProbe& pr, uint32_t g, const uint4& q, uint32_t k,
                                               int count_bits, uint32_t& entry)
{
    const uint32_t qv[4] = {q.x, q.y, q.z, q.w};
    bool done = false;
    entry = 0;
#pragma unroll
    for (uint32_t l = 0; l < 4; ++l) {
        const uint32_t e = qv[l];
        if (!done && pr.inside(4u * g + l)) {
            if (e == DK_EMPTY_SLOT) done = true;
            else if ((e >> count_bits) == k) { entry = e; done = true; }
        }
    }
    return done;
}

template <typename T>
__device__ __forceinline__ T warp_reduce_sum(T v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Inclusive scan across the 32 lanes of a warp.
template <typename T>
__device__ __forceinline__ T warp_scan_incl(T v)
{
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        T u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
    }
    return v;
}

// Block-wide sum; `smem` holds at least 32 T; result returned to every thread.
template <typename T>
__device__ __forceinline__ T block_reduce_sum(T v, T* smem)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_reduce_sum(v);
    __syncthreads();
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    T t = (lane < nw) ? smem[lane] : T(0);
    t = warp_reduce_sum(t);
    return t;
}

// Block-wide exclusive scan of one value per thread; returns the exclusive
// prefix and writes the block total to `total`.  `smem` holds at least 33 T.
template <typename T>
__device__ __forceinline__ T block_scan_excl(T v, T* smem, T& total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    T incl = warp_scan_incl(v);
    __syncthreads();
    if (lane == 31) smem[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        T w = (lane < nw) ? smem[lane] : T(0);
        T wi = warp_scan_incl(w);
        smem[lane] = wi - w;
        if (lane == 31) smem[32] = wi;
    }
    __syncthreads();
    total = smem[32];
    return smem[warp] + incl - v;
}

}  // namespace lda
