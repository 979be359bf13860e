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

// (double)x for an unsigned 32-bit x, exactly, without the (slow) integer-to-double conversion
// instruction: x placed in the low mantissa bits of 2^52, then 2^52 subtracted.
__device__ __forceinline__ double u32_to_double(uint32_t x)
{
    return __dsub_rn(__hiloint2double(0x43300000, (int)x), 4503599627370496.0);
}

// floor(r * n / 2^32): a 32-bit random word mapped to {0..n-1}.
__device__ __forceinline__ uint32_t scale_to_range(uint32_t r, uint32_t n) { return __umulhi(r, n); }

__device__ __forceinline__ int bit_length(unsigned long long x) { return 64 - __clzll((long long)x); }

// --- n_kd tables --------------------------------------------------------------------------------
// Section 5's hashed rows (fn. 5 asks for at least twice as many slots as entries), one table per
// document: `cap` = 4 * (document length) slots, so the load factor stays <= 0.25.  A slot is
// (topic << count_bits) | count, or DK_EMPTY_SLOT.  Open addressing with linear probing: topic k
// starts at slot floor(k * DK_HASH_MULT mod 2^32 * cap / 2^32) and moves up one slot at a time,
// wrapping; an empty slot met on the way means "absent".  At this load a search takes about 1.2
// probes (found) or 1.4 (absent).
constexpr uint32_t DK_EMPTY_SLOT = 0xFFFFFFFFu;
constexpr uint32_t DK_HASH_MULT = 0x9E3779B1u;
constexpr int DK_SLOTS_PER_TOKEN = 4;

__device__ __forceinline__ uint32_t dk_home(uint32_t k, uint32_t cap) { return __umulhi(k * DK_HASH_MULT, cap); }

// Adds one occurrence of topic k to the table `tab[0..cap)`: claims an empty slot with one
// compare-and-swap that also sets the count to 1, or finds the topic's slot and adds one to its
// count bits.  Safe against concurrent insertions into the same table.  Returns the slot, or
// DK_EMPTY_SLOT if the table had no room (which the load factor rules out).
__device__ __forceinline__ uint32_t dk_insert(uint32_t* tab, uint32_t cap, uint32_t k, int count_bits)
{
    const uint32_t first = (k << count_bits) | 1u;
    uint32_t h = dk_home(k, cap);
    for (uint32_t n = 0; n < cap; ++n) {
        const uint32_t prev = atomicCAS(&tab[h], DK_EMPTY_SLOT, first);
        if (prev == DK_EMPTY_SLOT) return h;
        if ((prev >> count_bits) == k) {
            atomicAdd(&tab[h], 1u);
            return h;
        }
        if (++h == cap) h = 0;
    }
    return DK_EMPTY_SLOT;
}

// n_kd[k] as a packed entry (0 when absent).
__device__ __forceinline__ uint32_t dk_lookup(const uint32_t* tab, uint32_t cap, uint32_t k, int count_bits)
{
    uint32_t h = dk_home(k, cap);
    for (uint32_t n = 0; n < cap; ++n) {
        const uint32_t e = tab[h];
        if (e == DK_EMPTY_SLOT) return 0u;
        if ((e >> count_bits) == k) return e;
        if (++h == cap) h = 0;
    }
    return 0u;
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
