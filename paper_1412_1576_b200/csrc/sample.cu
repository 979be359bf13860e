// Token Metropolis-Hastings kernel (Section 4.2-4.3) and the assignment
// initialisation / import / export kernels.
//
// One thread owns one token for the whole chain.  Everything it reads is the
// sweep-start state (Section 6: the model is immutable while sampled), it writes
// only its own two output slots, so the result does not depend on scheduling.
#include "lda_device.cuh"
#include "lda_internal.cuh"

namespace lda {

constexpr double INV_2_32 = 1.0 / 4294967296.0;

// n_kw lookup: dense row if the word has one, else binary search in its sorted row.
__device__ __forceinline__ int32_t lookup_wk(const View& v, int32_t dslot, int32_t r0, int32_t nnz,
                                             uint32_t k)
{
    if (dslot >= 0) return __ldg(v.dense_rows + (size_t)dslot * v.K + k);
    int32_t lo = 0, hi = nnz;
    while (lo < hi) {
        const int32_t mid = (lo + hi) >> 1;
        if (__ldg(v.wk_topic + r0 + mid) < k) lo = mid + 1; else hi = mid;
    }
    return (lo < nnz && __ldg(v.wk_topic + r0 + lo) == k) ? (int32_t)__ldg(v.wk_count + r0 + lo) : 0;
}

// n_kd lookup in the document's open-addressing table (capacity 2*n_d, linear probing).
__device__ __forceinline__ int32_t lookup_dk(const View& v, const uint32_t* __restrict__ tab, uint32_t cap,
                                             uint32_t k)
{
    uint32_t h = __umulhi(k * DK_HASH, cap);
    for (uint32_t probe = 0; probe < cap; ++probe) {
        const uint32_t e = __ldg(tab + h);
        if (e == DK_EMPTY) return 0;
        if ((e >> v.count_bits) == k) return (int32_t)(e & ((1u << v.count_bits) - 1u));
        if (++h == cap) h = 0;
    }
    return 0;
}

template <typename T>
__global__ void __launch_bounds__(256)
k_sample(View v, const T* __restrict__ zw_cur, const T* __restrict__ zd_cur, T* __restrict__ zw_nxt,
         T* __restrict__ zd_nxt, uint2 key, uint32_t sweep, int32_t mh_steps)
{
    __shared__ int32_t w_lo_s, w_hi_s;
    const int32_t p0 = blockIdx.x * SAMPLE_TILE;
    const int32_t p1 = min(v.N, p0 + SAMPLE_TILE);
    if (threadIdx.x < 2) {
        // word of the tile's first / last token: last w with word_off[w] <= p
        const int32_t p = threadIdx.x == 0 ? p0 : p1 - 1;
        int32_t lo = 0, hi = v.V;
        while (hi - lo > 1) {
            const int32_t mid = (lo + hi) >> 1;
            if (__ldg(v.word_off + mid) <= p) lo = mid; else hi = mid;
        }
        if (threadIdx.x == 0) w_lo_s = lo; else w_hi_s = lo;
    }
    __syncthreads();
    const int32_t w_lo = w_lo_s, w_hi = w_hi_s;
    const double alpha = v.alpha, beta = v.beta, Vb = v.Vbeta, Ka = v.Kalpha;

    for (int32_t p = p0 + threadIdx.x; p < p1; p += blockDim.x) {
        int32_t lo = w_lo, hi = w_hi + 1;
        while (hi - lo > 1) {
            const int32_t mid = (lo + hi) >> 1;
            if (__ldg(v.word_off + mid) <= p) lo = mid; else hi = mid;
        }
        const int32_t w = lo;
        const uint2 dinfo = __ldg(v.tok_dinfo + p);
        const uint32_t tok = __ldg(v.tok_orig + p);
        const uint32_t z0 = (uint32_t)zw_cur[p];

        const int32_t r0 = __ldg(v.row_start + w), wnnz = __ldg(v.wk_nnz + w);
        const int32_t dslot = __ldg(v.dense_slot + w);
        const uint32_t mix = __ldg(v.mix32 + w);
        const int32_t d0 = (int32_t)dinfo.x, n_d = (int32_t)dinfo.y;
        const uint32_t* dtab = v.dk_slots + 2 * (size_t)dinfo.x;
        const uint32_t dcap = 2u * dinfo.y;

        // counts at the current state s (start: s = z0, where all three are >= 1)
        uint32_t s = z0;
        int32_t n_sd = lookup_dk(v, dtab, dcap, s);
        int32_t n_sw = lookup_wk(v, dslot, r0, wnnz, s);
        int32_t n_s = __ldg(v.nk + s);
        if (n_sd < 1 || n_sw < 1 || n_s < 1) atomicOr(v.err, ERR_COUNT_ZERO);

        for (int32_t m = 0; m < mh_steps; ++m) {
            const uint4 r = philox4x32_10(make_uint4(tok, sweep, (uint32_t)m, 0u), key);
            uint32_t t;
            int32_t n_tw = -1;
            const bool word_step = (m & 1) == 0;
            if (word_step) {
                // word-proposal (Eq. 6): sparse term with probability mix/2^32, else dense term
                if (r.x < mix) {
                    const uint32_t b = scale_to_range(r.y, (uint32_t)wnnz);
                    const uint32_t al = __ldg(v.al_idx + r0 + b);
                    const uint32_t item = (al == b || r.z < __ldg(v.al_thr + r0 + b)) ? b : al;
                    t = __ldg(v.wk_topic + r0 + item);
                    n_tw = (int32_t)__ldg(v.wk_count + r0 + item);
                } else {
                    const uint32_t b = scale_to_range(r.y, (uint32_t)v.K);
                    const uint32_t al = __ldg(v.dn_idx + b);
                    t = (al == b || r.z < __ldg(v.dn_thr + b)) ? b : al;
                }
            } else {
                // doc-proposal (Eq. 9, Eq. 12): copy the topic of a random token of the document,
                // or a uniform topic with probability K*alpha / (n_d + K*alpha)
                const double u = __dmul_rn((double)r.x, INV_2_32);
                if (__dmul_rn(u, __dadd_rn((double)n_d, Ka)) < (double)n_d)
                    t = (uint32_t)zd_cur[d0 + scale_to_range(r.y, (uint32_t)n_d)];
                else
                    t = scale_to_range(r.y, (uint32_t)v.K);
            }
            if (t == s) continue;
            if (n_tw < 0) n_tw = lookup_wk(v, dslot, r0, wnnz, t);
            const int32_t n_td = lookup_dk(v, dtab, dcap, t);
            const int32_t n_t = __ldg(v.nk + t);
            const int32_t e_s = (s == z0), e_t = (t == z0);
            // Eq. 8 (word step) / Eq. 11 (doc step), products taken left to right
            double num = __dadd_rn((double)(n_td - e_t), alpha);
            num = __dmul_rn(num, __dadd_rn((double)(n_tw - e_t), beta));
            num = __dmul_rn(num, __dadd_rn((double)(n_s - e_s), Vb));
            double den = __dadd_rn((double)(n_sd - e_s), alpha);
            den = __dmul_rn(den, __dadd_rn((double)(n_sw - e_s), beta));
            den = __dmul_rn(den, __dadd_rn((double)(n_t - e_t), Vb));
            if (word_step) {
                num = __dmul_rn(num, __dadd_rn((double)n_sw, beta));
                num = __dmul_rn(num, __dadd_rn((double)n_t, Vb));
                den = __dmul_rn(den, __dadd_rn((double)n_tw, beta));
                den = __dmul_rn(den, __dadd_rn((double)n_s, Vb));
            } else {
                num = __dmul_rn(num, __dadd_rn((double)n_sd, alpha));
                den = __dmul_rn(den, __dadd_rn((double)n_td, alpha));
            }
            const double ua = __dmul_rn((double)r.w, INV_2_32);
            if (__dmul_rn(ua, den) < num) {
                s = t;
                n_sd = n_td;
                n_sw = n_tw;
                n_s = n_t;
            }
        }
        zw_nxt[p] = (T)s;
        zd_nxt[tok] = (T)s;
    }
}

// z_i uniform on {0..K-1}: Philox counter (token, 0, 0, 1), word 0.
template <typename T>
__global__ void k_init(View v, T* __restrict__ zw, T* __restrict__ zd, uint2 key)
{
    for (int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; p < v.N;
         p += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t tok = v.tok_orig[p];
        const uint4 r = philox4x32_10(make_uint4(tok, 0u, 0u, 1u), key);
        const T z = (T)scale_to_range(r.x, (uint32_t)v.K);
        zw[p] = z;
        zd[tok] = z;
    }
}

template <typename T>
__global__ void k_spread(View v, const int32_t* __restrict__ z_in, T* __restrict__ zw, T* __restrict__ zd)
{
    for (int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; p < v.N;
         p += (int64_t)gridDim.x * blockDim.x) {
        const int32_t a = z_in[p];
        if (a < 0 || a >= v.K) atomicOr(v.err, ERR_TOPIC_RANGE);
        zd[p] = (T)a;
        zw[p] = (T)z_in[v.tok_orig[p]];
    }
}

template <typename T>
__global__ void k_export(int32_t n, const T* __restrict__ zd, int32_t* __restrict__ out)
{
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n;
         i += (int64_t)gridDim.x * blockDim.x)
        out[i] = (int32_t)zd[i];
}

static int grid_for(int64_t n, int block)
{
    int64_t g = (n + block - 1) / block;
    if (g > 148 * 16) g = 148 * 16;
    return g < 1 ? 1 : (int)g;
}

template <typename T>
static int sample_t(Ctx& c, int mh_steps)
{
    if (c.N == 0) return 0;
    View& v = c.v;
    const int nxt = c.cur ^ 1;
    const int grid = (int)((c.N + SAMPLE_TILE - 1) / SAMPLE_TILE);
    const uint2 key = make_uint2((uint32_t)c.seed, (uint32_t)(c.seed >> 32));
    k_sample<T><<<grid, 256, 0, c.stream>>>(v, (const T*)v.zw[c.cur], (const T*)v.zd[c.cur],
                                            (T*)v.zw[nxt], (T*)v.zd[nxt], key, c.sweep, mh_steps);
    return 1;
}

int launch_sample(Ctx& c, int mh_steps)
{
    return c.wide_topics ? sample_t<int32_t>(c, mh_steps) : sample_t<uint16_t>(c, mh_steps);
}

int launch_init(Ctx& c)
{
    if (c.N == 0) return 0;
    const uint2 key = make_uint2((uint32_t)c.seed, (uint32_t)(c.seed >> 32));
    const int g = grid_for(c.N, 256);
    if (c.wide_topics)
        k_init<int32_t><<<g, 256, 0, c.stream>>>(c.v, (int32_t*)c.v.zw[c.cur], (int32_t*)c.v.zd[c.cur], key);
    else
        k_init<uint16_t><<<g, 256, 0, c.stream>>>(c.v, (uint16_t*)c.v.zw[c.cur], (uint16_t*)c.v.zd[c.cur], key);
    return 1;
}

int launch_spread_assignments(Ctx& c, const int32_t* z_dev)
{
    if (c.N == 0) return 0;
    const int g = grid_for(c.N, 256);
    if (c.wide_topics)
        k_spread<int32_t><<<g, 256, 0, c.stream>>>(c.v, z_dev, (int32_t*)c.v.zw[c.cur], (int32_t*)c.v.zd[c.cur]);
    else
        k_spread<uint16_t><<<g, 256, 0, c.stream>>>(c.v, z_dev, (uint16_t*)c.v.zw[c.cur], (uint16_t*)c.v.zd[c.cur]);
    return 1;
}

int launch_export_assignments(Ctx& c, int32_t* z_dev)
{
    if (c.N == 0) return 0;
    const int g = grid_for(c.N, 256);
    if (c.wide_topics)
        k_export<int32_t><<<g, 256, 0, c.stream>>>((int32_t)c.N, (const int32_t*)c.v.zd[c.cur], z_dev);
    else
        k_export<uint16_t><<<g, 256, 0, c.stream>>>((int32_t)c.N, (const uint16_t*)c.v.zd[c.cur], z_dev);
    return 1;
}

}  // namespace lda
