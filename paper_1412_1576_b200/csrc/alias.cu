// Word-proposal tables (Section 4.2): the word-proposal (n_kw + beta)/(n_k + V*beta)
// is sampled as a mixture of a sparse term over the word's nonzero n_kw (one alias
// table per word, O(K_w) to build) and a dense term beta/(n_k + V*beta) whose alias
// table is shared by all words.
//
// Alias construction is cooperative (a warp for short rows, a CTA for long ones)
// and exact in integers, so the table is a function of the counts alone:
//   - fixed-point weights wt_i = floor(weight_i * 2^44), W44 = sum wt_i;
//   - pre-shift sh = max(0, bitlen(W44) + bitlen(n) - 62), w_i = wt_i >> sh, W = sum w_i;
//   - bin capacity W, item i brings a_i = n * w_i; a_i <= W is "light", else "heavy";
//   - with D_l = deficits of the lights before light l (ascending item order) and
//     E_m = surpluses of heavies 0..m, light l is filled by heavy #{m : E_m <= D_l};
//     heavy m keeps W + E_m - D_lam with lam = min{l : D_l >= E_m} and is filled by
//     heavy m+1 (or is full).
// This is the closed form of "fill lights in order from the current heavy item; an
// exhausted heavy item becomes a bin topped up by the next heavy item".
#include "lda_device.cuh"
#include "lda_internal.cuh"

namespace lda {

typedef unsigned long long ull;

#ifndef LDA_ALIAS_BINS_AT_ONCE
#define LDA_ALIAS_BINS_AT_ONCE 2
#endif
constexpr int ALIAS_BINS_AT_ONCE = LDA_ALIAS_BINS_AT_ONCE;  // bins a thread finishes side by side

template <bool BLOCK>
struct Group {
    ull* smem;  // CTA groups only: >= 99 entries
    __device__ __forceinline__ int rank() const { return BLOCK ? (int)threadIdx.x : (int)(threadIdx.x & 31); }
    __device__ __forceinline__ int size() const { return BLOCK ? (int)blockDim.x : 32; }
    __device__ __forceinline__ void sync() const
    {
        if (BLOCK) __syncthreads(); else __syncwarp();
    }
    __device__ __forceinline__ ull reduce(ull v) const
    {
        if (BLOCK) return block_reduce_sum<ull>(v, smem);
        return warp_reduce_sum<ull>(v);
    }
    // Exclusive scans of three values at once (one pass, one set of barriers); v[] in, prefixes
    // out in v[], totals in tot[].  CTA groups need 99 entries of `smem`.
    __device__ __forceinline__ void scan_excl3(ull (&v)[3], ull (&tot)[3]) const
    {
        ull incl[3];
#pragma unroll
        for (int q = 0; q < 3; ++q) incl[q] = warp_scan_incl<ull>(v[q]);
        if (!BLOCK) {
#pragma unroll
            for (int q = 0; q < 3; ++q) {
                tot[q] = __shfl_sync(0xffffffffu, incl[q], 31);
                v[q] = incl[q] - v[q];
            }
            return;
        }
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
        __syncthreads();
        if (lane == 31) {
#pragma unroll
            for (int q = 0; q < 3; ++q) smem[33 * q + warp] = incl[q];
        }
        __syncthreads();
        if (warp == 0) {
#pragma unroll
            for (int q = 0; q < 3; ++q) {
                const ull w = (lane < nw) ? smem[33 * q + lane] : 0ull;
                const ull wi = warp_scan_incl<ull>(w);
                smem[33 * q + lane] = wi - w;
                if (lane == 31) smem[33 * q + 32] = wi;
            }
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < 3; ++q) {
            tot[q] = smem[33 * q + 32];
            v[q] = smem[33 * q + warp] + incl[q] - v[q];
        }
    }
};

__device__ __forceinline__ uint32_t to_frac32(ull part, ull whole)
{
    int sh = bit_length(whole) - 32;
    if (sh < 0) sh = 0;
    const ull q = ((part >> sh) << 32) / (whole >> sh);
    return q > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)q;
}

// to_frac32(part, whole) for many parts <= whole of one whole: the quotient from a double
// reciprocal of the (shifted) whole, then set right with the exact integer remainder.  The
// estimate is within 2^-20 of the true quotient (two roundings of 2^-53 on a value <= 2^32), so
// its integer part is off by one at most.
struct Frac32 {
    int sh;
    uint32_t w;  // whole >> sh, < 2^32
    double inv;  // 1 / w
    __device__ __forceinline__ explicit Frac32(ull whole)
    {
        sh = bit_length(whole) - 32;
        if (sh < 0) sh = 0;
        w = (uint32_t)(whole >> sh);
        inv = __ddiv_rn(1.0, u32_to_double(w));
    }
    __device__ __forceinline__ uint32_t operator()(ull part) const
    {
        const uint32_t p = (uint32_t)(part >> sh);  // part <= whole
        const ull x = (ull)p << 32;
        ull q = __double2ull_rz(__dmul_rn(__dmul_rn(u32_to_double(p), 4294967296.0), inv));
        const long long r = (long long)(x - q * (ull)w);
        if (r < 0) --q;
        else if (r >= (long long)w) ++q;
        return q > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)q;
    }
};

// One bin in the form the MH kernel reads with a single load.  With `topic` (a word's sorted
// row) the second word holds the topics of the bin's own item and of its alias item, 16 bits
// each; without it (the dense table, whose items are the topics) it holds the alias.
__device__ __forceinline__ void store_packed_bin(uint2* out_pk, const uint32_t* topic, uint32_t i, uint32_t thr32,
                                                 uint32_t al)
{
    if (!out_pk) return;
    out_pk[i] = make_uint2(thr32, topic ? (topic[i] | (topic[al] << 16)) : al);
}

// Builds one table of n items.  weight(i) gives the fixed-point weight of item i.
// sc_w, sc_de, sc_item: scratch of n entries each, private to this row.
// out_pk (may be null) receives the packed form of every bin, see store_packed_bin().
// Returns W44 (the sum of the fixed-point weights) to every thread of the group.
template <bool BLOCK, class Weight>
__device__ ull build_alias_row(const Group<BLOCK>& g, int32_t n, Weight weight, ull* __restrict__ sc_w,
                               ull* __restrict__ sc_de, uint32_t* __restrict__ sc_item,
                               uint32_t* __restrict__ out_thr, uint32_t* __restrict__ out_idx,
                               uint2* __restrict__ out_pk, const uint32_t* __restrict__ pk_topic, int* err)
{
    const int r = g.rank(), gs = g.size();
    // Items are taken four (weights) or two (bins) at a time per thread, their loads issued side by
    // side: a row is built by one warp or one CTA, so what a pass costs is the latency of its chain of
    // dependent reads, not the number of instructions.
    ull s = 0;
    for (int32_t i0 = r; i0 < n; i0 += 4 * gs) {
        ull wt[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int32_t i = i0 + u * gs;
            wt[u] = i < n ? weight(i) : 0ull;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int32_t i = i0 + u * gs;
            if (i < n) sc_w[i] = wt[u];
            s += wt[u];
        }
    }
    const ull W44 = g.reduce(s);
    int sh = bit_length(W44) + bit_length((ull)n) - 62;
    if (sh < 0) sh = 0;
    s = 0;
#pragma unroll 4
    for (int32_t i = r; i < n; i += gs) s += sc_w[i] >> sh;
    const ull W = g.reduce(s);
    if (W == 0) {
        if (r == 0) atomicOr(err, ERR_ALIAS);
        return W44;
    }
    // Every thread takes a run of consecutive items (lights and heavies are numbered in ascending
    // item order): one pass to count them and add up their deficits and surpluses, one scan of the
    // threads' totals, one pass to write the prefix of every item.  An odd run length keeps the
    // threads of a warp on different shared-memory banks.
    g.sync();  // the weights were written item by item across the group
    const int32_t seg = ((n + gs - 1) / gs) | 1;
    const int32_t i_first = min(n, r * seg), i_last = min(n, i_first + seg);
    ull cnt = 0, d_mine = 0, e_mine = 0;
#pragma unroll 4
    for (int32_t i = i_first; i < i_last; ++i) {
        const ull a = (ull)n * (sc_w[i] >> sh);
        if (a <= W) { cnt += 1ull; d_mine += W - a; } else { cnt += 1ull << 32; e_mine += a - W; }
    }
    ull pre[3] = {cnt, d_mine, e_mine}, tot[3];
    g.scan_excl3(pre, tot);
    {
        uint32_t l = (uint32_t)pre[0], m = (uint32_t)(pre[0] >> 32);
        ull d_at = pre[1], e_at = pre[2];
#pragma unroll 2
        for (int32_t i = i_first; i < i_last; ++i) {
            const ull a = (ull)n * (sc_w[i] >> sh);
            sc_w[i] = a;
            if (a <= W) {
                sc_de[l] = d_at;  // deficits of the lights before this one
                sc_item[l] = (uint32_t)i;
                ++l;
                d_at += W - a;
            } else {
                e_at += a - W;
                sc_de[n - 1 - m] = e_at;  // surpluses of the heavies up to and including this one
                sc_item[n - 1 - m] = (uint32_t)i;
                ++m;
            }
        }
    }
    const uint32_t L = (uint32_t)tot[0], H = (uint32_t)(tot[0] >> 32);
    const ull d_sum = tot[1];
    g.sync();
    const Frac32 frac(W);
    // The searches below count the entries of a sorted prefix array under a bound, one bit of the
    // answer per step from the top: the same number of steps for every item, so two items' searches
    // run in one loop.
    constexpr int U = ALIAS_BINS_AT_ONCE;
    const uint32_t top_h = H ? 1u << (31 - __clz((int)H)) : 0u;
    const uint32_t top_l = L ? 1u << (31 - __clz((int)L)) : 0u;
    for (uint32_t l0 = r; l0 < L; l0 += U * gs) {
        uint32_t it[U], pos[U];
        ull a[U], D[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t l = l0 + u * gs;
            it[u] = l < L ? sc_item[l] : 0u;
            D[u] = l < L ? sc_de[l] : 0ull;
            pos[u] = 0;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) a[u] = l0 + u * gs < L ? sc_w[it[u]] : W;
        for (uint32_t step = top_h; step; step >>= 1) {  // number of heavies with E_m <= D
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t q = pos[u] + step;
                if (q <= H && sc_de[n - q] <= D[u]) pos[u] = q;
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (l0 + u * gs >= L) continue;
            const uint32_t i = it[u];
            uint32_t al = i;
            if (a[u] != W) {
                uint32_t lo = pos[u];
                if (lo >= H) { atomicOr(err, ERR_ALIAS); lo = H ? H - 1 : 0; }
                al = H ? sc_item[n - 1 - lo] : i;
            }
            const uint32_t thr32 = frac(a[u]);
            out_thr[i] = thr32;
            out_idx[i] = al;
            store_packed_bin(out_pk, pk_topic, i, thr32, al);
        }
    }
    for (uint32_t m0 = r; m0 < H; m0 += U * gs) {
        uint32_t it[U], pos[U];
        ull E[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t m = m0 + u * gs;
            it[u] = m < H ? sc_item[n - 1 - m] : 0u;
            E[u] = m < H ? sc_de[n - 1 - m] : 0ull;
            pos[u] = 0;
        }
        for (uint32_t step = top_l; step; step >>= 1) {  // number of lights with D_l < E: the first light with D_l >= E
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t q = pos[u] + step;
                if (q <= L && sc_de[q - 1] < E[u]) pos[u] = q;
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t m = m0 + u * gs;
            if (m >= H) continue;
            const uint32_t i = it[u], lo = pos[u];  // lo == L stands for the total deficit
            const ull Dl = lo < L ? sc_de[lo] : d_sum;
            const ull thr = W + E[u] - Dl;
            uint32_t al = i;
            if (thr != W) {
                if (m + 1 >= H) atomicOr(err, ERR_ALIAS);
                else al = sc_item[n - 1 - (m + 1)];
            }
            const uint32_t thr32 = frac(thr);
            out_thr[i] = thr32;
            out_idx[i] = al;
            store_packed_bin(out_pk, pk_topic, i, thr32, al);
        }
    }
    return W44;
}

constexpr double FIXED_ONE = 17592186044416.0;  // 2^44

struct DenseWeight {
    const int32_t* nk;
    double beta, Vbeta;
    __device__ __forceinline__ ull operator()(int32_t k) const
    {
        const double den = __dadd_rn((double)nk[k], Vbeta);
        return __double2ull_rz(__dmul_rn(__ddiv_rn(beta, den), FIXED_ONE));
    }
};

struct SparseWeight {
    const uint32_t* topic;
    const uint32_t* count;
    const int32_t* nk;
    double Vbeta;
    __device__ __forceinline__ ull operator()(int32_t i) const
    {
        const double den = __dadd_rn((double)nk[topic[i]], Vbeta);
        return __double2ull_rz(__dmul_rn(__ddiv_rn((double)count[i], den), FIXED_ONE));
    }
};

__global__ void __launch_bounds__(1024) k_alias_dense(View v, ull* sc)
{
    __shared__ ull smem[99];
    Group<true> g{smem};
    const int32_t K = v.K;
    DenseWeight wf{v.nk, v.beta, v.Vbeta};
    const ull B = build_alias_row<true>(g, K, wf, sc, sc + K, (uint32_t*)(sc + 2 * (size_t)K), v.dn_thr,
                                        v.dn_idx, v.dn_pk, nullptr, v.err);
    if (threadIdx.x == 0) *v.dense_mass = B;
}

__device__ __forceinline__ uint32_t mixture_threshold(ull S, ull B)
{
    if (S == 0) return 0;
    return to_frac32(S, S + B);
}

// One warp per word, rows of at most ALIAS_WARP_MAX items.  The two scratch arrays the binary
// searches run over live in shared memory (12 bytes per item and warp), the third in the row's
// range of the scratch array in device memory.
__global__ void __launch_bounds__(256) k_alias_sparse_warp(View v, ull* sc_w, int32_t w_lo, int32_t w_hi)
{
    extern __shared__ __align__(16) unsigned char alias_scratch[];
    Group<false> g{nullptr};
    const int warps = (gridDim.x * blockDim.x) >> 5;
    const int wic = threadIdx.x >> 5;
    ull* de_s = reinterpret_cast<ull*>(alias_scratch) + (size_t)wic * ALIAS_WARP_MAX;
    uint32_t* item_s = reinterpret_cast<uint32_t*>(reinterpret_cast<ull*>(alias_scratch) + 8 * ALIAS_WARP_MAX) +
                       (size_t)wic * ALIAS_WARP_MAX;
    const ull B = *v.dense_mass;
    for (int32_t w = w_lo + ((blockIdx.x * blockDim.x + threadIdx.x) >> 5); w < w_hi; w += warps) {
        const int32_t n = v.wk_nnz[w];
        if (n > ALIAS_WARP_MAX) continue;
        if (n == 0) {
            if ((threadIdx.x & 31) == 0) v.mix32[w] = 0;
            continue;
        }
        const int32_t r0 = v.row_start[w];
        SparseWeight wf{v.wk_topic + r0, v.wk_count + r0, v.nk, v.Vbeta};
        const ull S = build_alias_row<false>(g, n, wf, sc_w + r0, de_s, item_s, v.al_thr + r0, v.al_idx + r0,
                                             v.al_pk ? v.al_pk + r0 : nullptr, v.wk_topic + r0, v.err);
        if ((threadIdx.x & 31) == 0) v.mix32[w] = mixture_threshold(S, B);
        __syncwarp();
    }
}

// One CTA per word whose row can be longer than ALIAS_WARP_MAX.  The construction's scratch
// (20 bytes per item) lives in shared memory when the row has at most `smem_items` items; a longer
// row keeps the array its binary searches run over (8 bytes per item) there as long as that fits,
// and the rest -- or, beyond that, everything -- in the row's range of the scratch arrays in
// device memory.
#ifndef LDA_ALIAS_MID_MIN_CTAS
#define LDA_ALIAS_MID_MIN_CTAS 1
#endif
template <int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? LDA_ALIAS_MID_MIN_CTAS : 1)
k_alias_sparse_block(View v, const int32_t* __restrict__ words, ull* sc_w, ull* sc_de, uint32_t* sc_item,
                     int32_t smem_items)
{
    extern __shared__ __align__(16) unsigned char alias_scratch[];
    __shared__ ull smem[99];
    Group<true> g{smem};
    const int32_t w = words[blockIdx.x];
    const int32_t n = v.wk_nnz[w];
    if (n <= ALIAS_WARP_MAX) return;
    const int32_t r0 = v.row_start[w];
    SparseWeight wf{v.wk_topic + r0, v.wk_count + r0, v.nk, v.Vbeta};
    uint2* pk = v.al_pk ? v.al_pk + r0 : nullptr;
    ull S;
    if (n <= smem_items) {
        ull* w_s = reinterpret_cast<ull*>(alias_scratch);
        ull* de_s = w_s + smem_items;
        uint32_t* item_s = reinterpret_cast<uint32_t*>(de_s + smem_items);
        S = build_alias_row<true>(g, n, wf, w_s, de_s, item_s, v.al_thr + r0, v.al_idx + r0, pk, v.wk_topic + r0, v.err);
    } else if ((int64_t)n * 8 <= (int64_t)smem_items * ALIAS_SCRATCH_PER_ITEM) {
        S = build_alias_row<true>(g, n, wf, sc_w + r0, reinterpret_cast<ull*>(alias_scratch), sc_item + r0,
                                  v.al_thr + r0, v.al_idx + r0, pk, v.wk_topic + r0, v.err);
    } else {
        S = build_alias_row<true>(g, n, wf, sc_w + r0, sc_de + r0, sc_item + r0, v.al_thr + r0, v.al_idx + r0, pk,
                                  v.wk_topic + r0, v.err);
    }
    if (threadIdx.x == 0) v.mix32[w] = mixture_threshold(S, *v.dense_mass);
}

int launch_alias_dense(Ctx& c)
{
    k_alias_dense<<<1, 1024, 0, c.stream>>>(c.v, c.sc_dense);
    return 1;
}

// The three kernels build the tables of different words: they run side by side, the one with the
// longest rows (and the longest tail) first.
int launch_alias_sparse(Ctx& c)
{
    const Ctx::Slice& q = c.slices[(size_t)c.cur_slice];
    if (q.w_hi <= q.w_lo) return 0;
    int launches = 0;
    fork_streams(c);
    // words whose row cannot exceed ALIAS_SMEM_ITEMS_MID come first in the list
    if (q.big_n) {
        k_alias_sparse_block<512><<<q.big_n, 512, ALIAS_SMEM_ITEMS_BIG * ALIAS_SCRATCH_PER_ITEM, c.stream>>>(
            c.v, c.alias_big + c.n_alias_mid + q.big_lo, c.sc_w, c.sc_de, c.sc_item, ALIAS_SMEM_ITEMS_BIG);
        ++launches;
    }
    if (q.mid_n) {
        k_alias_sparse_block<256><<<q.mid_n, 256, ALIAS_SMEM_ITEMS_MID * ALIAS_SCRATCH_PER_ITEM, c.side[0]>>>(
            c.v, c.alias_big + q.mid_lo, c.sc_w, c.sc_de, c.sc_item, ALIAS_SMEM_ITEMS_MID);
        ++launches;
    }
    int grid = (int)(((int64_t)(q.w_hi - q.w_lo) * 32 + 255) / 256);
    if (grid > 148 * 16) grid = 148 * 16;
    k_alias_sparse_warp<<<grid, 256, ALIAS_WARP_SMEM, c.side[1]>>>(c.v, c.sc_w, q.w_lo, q.w_hi);
    ++launches;
    join_streams(c);
    return launches;
}

void set_alias_smem_limits()
{
    cudaFuncSetAttribute(k_alias_sparse_warp, cudaFuncAttributeMaxDynamicSharedMemorySize, ALIAS_WARP_SMEM);
    cudaFuncSetAttribute(k_alias_sparse_block<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         ALIAS_SMEM_ITEMS_MID * ALIAS_SCRATCH_PER_ITEM);
    cudaFuncSetAttribute(k_alias_sparse_block<512>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         ALIAS_SMEM_ITEMS_BIG * ALIAS_SCRATCH_PER_ITEM);
}

}  // namespace lda

// ---------------------------------------------------------------------------------------
// Allocation-free entry point.
//
// Some callers cannot allocate device memory at the moment they need a table: code that
// runs inside a framework's memory pool and must not touch cudaMalloc behind its back, a
// real-time loop where an allocation's implicit device synchronisation is not acceptable,
// or a process whose memory budget was fixed at start-up.  For them the dense smoothing
// table can be built with the construction scratch held in a file-scope device array.
// Every GPU that loads the library holds that array (20 bytes per topic of LDA_NOALLOC_MAX_K,
// about 2.6 MB) until exit.
// ---------------------------------------------------------------------------------------
namespace lda {

constexpr int NOALLOC_MAX_K = LDA_NOALLOC_MAX_K;
// per topic: one 64-bit mass, one 64-bit prefix sum, one 32-bit item index = 20 bytes
constexpr size_t NOALLOC_SCRATCH_WORDS = 2 * (size_t)NOALLOC_MAX_K + (size_t)NOALLOC_MAX_K / 2;

static __device__ __align__(256) unsigned long long g_noalloc_scratch[NOALLOC_SCRATCH_WORDS];
static __device__ __align__(256) int g_noalloc_status[4];

// Device addresses of the two arrays above, looked up once per device.  In host code the
// array names are only handles for the runtime, not addresses a kernel could use.
struct NoallocAddr {
    bool ready = false;
    unsigned long long* scratch = nullptr;
    int* status = nullptr;
};
static NoallocAddr g_noalloc_addr[64];

static int noalloc_setup(int dev, NoallocAddr** out)
{
    if (dev < 0 || dev >= 64) return LDA_ERANGE;
    NoallocAddr& a = g_noalloc_addr[dev];
    if (!a.ready) {
        void* p = nullptr;
        void* q = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess ||
            cudaGetSymbolAddress(&q, g_noalloc_status) != cudaSuccess) {
            cudaGetLastError();
            return LDA_ECUDA;
        }
        a.scratch = (unsigned long long*)p;
        a.status = (int*)q;
        a.ready = true;
    }
    *out = &a;
    return LDA_OK;
}

}  // namespace lda

extern "C" int lda_dense_table_noalloc(const int32_t* n_k_dev, int32_t K, int32_t V, double beta,
                                       uint32_t* dn_thr32_dev, int32_t* dn_alias_dev,
                                       uint64_t* dense_mass_dev, int32_t* status_dev, void* cuda_stream)
{
    using namespace lda;
    if (!n_k_dev || !dn_thr32_dev || !dn_alias_dev || !dense_mass_dev) return LDA_EINVAL;
    if (K <= 0 || V <= 0 || !(beta > 0) || !isfinite(beta)) return LDA_EINVAL;
    if (K > NOALLOC_MAX_K) return LDA_ERANGE;  // the fixed scratch array holds LDA_NOALLOC_MAX_K topics
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return LDA_ECUDA; }
    NoallocAddr* addr = nullptr;
    int rc = noalloc_setup(dev, &addr);
    if (rc != LDA_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int* status = status_dev ? (int*)status_dev : addr->status;
    // the status word must start at zero; the scratch itself is fully overwritten before it is read
    if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) { cudaGetLastError(); return LDA_ECUDA; }
    View v{};
    v.V = V;
    v.K = K;
    v.beta = beta;
    v.Vbeta = (double)V * beta;
    v.nk = const_cast<int32_t*>(n_k_dev);
    v.dn_thr = dn_thr32_dev;
    v.dn_idx = (uint32_t*)dn_alias_dev;
    v.dense_mass = (unsigned long long*)dense_mass_dev;
    v.err = status;
    k_alias_dense<<<1, 1024, 0, st>>>(v, addr->scratch);
    if (cudaGetLastError() != cudaSuccess) return LDA_ECUDA;
    return LDA_OK;
}
