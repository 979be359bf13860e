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
// Document d owns slots [4*doc_off[d], 4*doc_off[d+1]) of one global slot array: four slots per
// token, so the load factor stays <= 0.25 (Section 5, fn. 5 asks for at least twice the number
// of entries).  A slot is (topic << count_bits) | count, or DK_EMPTY_SLOT.  The table is
// bucketed by aligned groups of eight slots (one 32-byte sector): topic k starts at group
// DkProbe::first(k) and tries the group's slots that belong to the document in order, then the
// next group, wrapping to the table's first group.  An empty slot met on the way means "absent".
// At this load a lookup almost never needs a second group.
constexpr uint32_t DK_EMPTY_SLOT = 0xFFFFFFFFu;
constexpr uint32_t DK_HASH_MULT = 0x9E3779B1u;
constexpr int DK_SLOTS_PER_TOKEN = 4;
constexpr int DK_GROUP = 8;

struct DkProbe {
    uint32_t g_first, g_cnt;  // first group (slot index / 8) and number of groups the table touches
    bool head_half, tail_half;  // the table starts / ends in the middle of a group
    __device__ __forceinline__ DkProbe(uint32_t doc_first_token, uint32_t doc_len)
    {
        const uint32_t end = doc_first_token + doc_len;  // tokens; the document is not empty
        g_first = doc_first_token >> 1;
        g_cnt = ((end - 1u) >> 1) - g_first + 1u;
        head_half = doc_first_token & 1u;
        tail_half = end & 1u;
    }
    __device__ __forceinline__ uint32_t first(uint32_t k) const { return g_first + __umulhi(k * DK_HASH_MULT, g_cnt); }
    __device__ __forceinline__ uint32_t next(uint32_t g) const { return g + 1u - g_first == g_cnt ? g_first : g + 1u; }
    // bit l set: slot l of group g belongs to this table
    __device__ __forceinline__ uint32_t lanes(uint32_t g) const
    {
        uint32_t m = 0xFFu;
        if (head_half && g == g_first) m &= 0xF0u;
        if (tail_half && g + 1u - g_first == g_cnt) m &= 0x0Fu;
        return m;
    }
};

// Looks topic k up in group g, whose eight slots are (qa, qb).  Returns true when the search is
// over (found, or an empty slot proves absence) and sets `entry` (0 when absent).
__device__ __forceinline__ bool dk_match_group(const DkProbe& pr, uint32_t g, const uint4& qa, const uint4& qb,
                                               uint32_t k, int count_bits, uint32_t& entry)
{
    const uint32_t qv[8] = {qa.x, qa.y, qa.z, qa.w, qb.x, qb.y, qb.z, qb.w};
    const uint32_t lanes = pr.lanes(g);
    bool done = false;
    entry = 0;
#pragma unroll
    for (uint32_t l = 0; l < 8; ++l) {
        const uint32_t e = qv[l];
        if (!done && ((lanes >> l) & 1u)) {
            if (e == DK_EMPTY_SLOT) done = true;
            else if ((e >> count_bits) == k) { entry = e; done = true; }
        }
    }
    return done;
}

// `tab` points at the copy of group `g0`; slot l of group g is tab[(g - g0) * 8 + l].
// Returns the index into `tab` the topic lives at (or 0xFFFFFFFF if the table had no room,
// which the load factor rules out).
__device__ __forceinline__ uint32_t dk_insert(uint32_t* tab, uint32_t g0, const DkProbe& pr, uint32_t k,
                                              int count_bits)
{
    const uint32_t fresh = k << count_bits;
    uint32_t g = pr.first(k);
    for (uint32_t n = 0; n < pr.g_cnt; ++n, g = pr.next(g)) {
        const uint32_t lanes = pr.lanes(g);
#pragma unroll
        for (uint32_t l = 0; l < DK_GROUP; ++l) {
            if (!((lanes >> l) & 1u)) continue;
            const uint32_t at = (g - g0) * DK_GROUP + l;
            const uint32_t prev = atomicCAS(&tab[at], DK_EMPTY_SLOT, fresh);
            if (prev == DK_EMPTY_SLOT || (prev >> count_bits) == k) {
                atomicAdd(&tab[at], 1u);
                return at;
            }
        }
    }
    return 0xFFFFFFFFu;
}

// n_kd[k] as a packed entry (0 when absent) from a table held as in dk_insert(); `tab` is 16-byte
// aligned.
__device__ __forceinline__ uint32_t dk_lookup(const uint32_t* tab, uint32_t g0, const DkProbe& pr, uint32_t k,
                                              int count_bits)
{
    uint32_t g = pr.first(k), entry = 0;
    for (uint32_t n = 0; n < pr.g_cnt; ++n, g = pr.next(g)) {
        const uint4* q = reinterpret_cast<const uint4*>(tab + (size_t)(g - g0) * DK_GROUP);
        if (dk_match_group(pr, g, q[0], q[1], k, count_bits, entry)) break;
    }
    return entry;
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
