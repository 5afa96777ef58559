// Channel-wise variant of the path (a variant of this library: the paper, Sec. 3, uses one clip
// range per tensor; channel-wise ranges are what its cited PTQ work uses for activations with
// outlier channels).  The tensor is [rows, channels], row-major: element i belongs to channel
// i mod channels.  Every channel gets the statistics, clip range and quantizer that the
// per-tensor functions give for its column alone; bit-width and packed layout are shared.
//
//   ch_stats_a / ch_stats_b   column reductions, HBM-bound: a thread owns V consecutive channels
//                             (one 16-byte load per row when the layout allows), a block walks
//                             rows blockIdx.x, blockIdx.x + gridDim.x, ... with 8 rows in flight (4 for
//                             bf16), fp32 sums over those rows folded into fp64; block partials
//                             [block][channel] are merged per channel in block order by
//                             ch_merge_a / ch_merge_b (bit-reproducible)
//   ch_clip_kernel            one thread per channel: closed-form clip -> quantizer
//   ch_pack_kernel            warp tile of 1024 elements: coalesced loads, quantize with the channel's
//                             parameters (table in shared memory), 16-bit codes into the warp's
//                             padded staging rows; then each lane packs 32 consecutive codes
//   ch_unpack_kernel          mirror image: words -> codes in the staging rows -> coalesced stores
#include "qp_internal.cuh"

QP_CK_UNIT

namespace {

constexpr int CH_THREADS = 256;
template <int V> struct ChRows { static constexpr int N = V >= 8 ? 4 : 8; };   // rows in flight per thread
constexpr int CH_STATS_MAX_THREADS = 512;      // column-reduction blocks: one thread per group of V channels

struct ChPart {                                   // one per (row block, channel)
    double s0, s1;                                // pass A: sum x, sum |x|;  pass B: sum |x-mean|, sum (x-mean)^2
    float mn, mx;
    unsigned bad, pad;
};

template <typename T, int V>
__device__ __forceinline__ void ch_load(const T* p, float (&e)[V])
{
    if constexpr (V == 1) {
        e[0] = qp_load_one(p);
    } else {
        qp_load_vec(p, e);
    }
}

template <typename T, int V>
__global__ void __launch_bounds__(CH_STATS_MAX_THREADS) ch_stats_a(const T* __restrict__ x, uint64_t rows, uint32_t C,
                                                         ChPart* __restrict__ part)
{
    const uint32_t col0 = (blockIdx.y * blockDim.x + threadIdx.x) * V;
    if (col0 >= C) return;
    const float inf = __int_as_float(0x7F800000);
    double s[V], sa[V];
    float mn[V], mx[V];
    unsigned bad[V];
#pragma unroll
    for (int i = 0; i < V; ++i) { s[i] = 0.0; sa[i] = 0.0; mn[i] = inf; mx[i] = -inf; bad[i] = 0u; }
    constexpr int CH_ROWS_IN_FLIGHT = ChRows<V>::N;
    const uint64_t step = gridDim.x;
    for (uint64_t r0 = blockIdx.x; r0 < rows; r0 += CH_ROWS_IN_FLIGHT * step) {
        float e[CH_ROWS_IN_FLIGHT][V];
#pragma unroll
        for (int u = 0; u < CH_ROWS_IN_FLIGHT; ++u) {
            const uint64_t r = r0 + u * step;
            if (r < rows) ch_load<T, V>(x + r * C + col0, e[u]);
        }
        float ps[V], psa[V];
#pragma unroll
        for (int i = 0; i < V; ++i) { ps[i] = 0.f; psa[i] = 0.f; }
#pragma unroll
        for (int u = 0; u < CH_ROWS_IN_FLIGHT; ++u) {
            if (r0 + u * step >= rows) break;
#pragma unroll
            for (int i = 0; i < V; ++i) {
                const float v = e[u][i];
                if (qp_is_finite(v)) {
                    ps[i] += v;
                    psa[i] += fabsf(v);
                    mn[i] = fminf(mn[i], v);
                    mx[i] = fmaxf(mx[i], v);
                } else {
                    ++bad[i];
                }
            }
        }
#pragma unroll
        for (int i = 0; i < V; ++i) { s[i] += (double)ps[i]; sa[i] += (double)psa[i]; }
    }
    ChPart* dst = part + (size_t)blockIdx.x * C + col0;
#pragma unroll
    for (int i = 0; i < V; ++i) {
        ChPart p;
        p.s0 = s[i]; p.s1 = sa[i]; p.mn = mn[i]; p.mx = mx[i]; p.bad = bad[i]; p.pad = 0u;
        dst[i] = p;
    }
}

// Merge of the row blocks' partials: a block takes 32 channels (lane = channel, so a warp reads
// 1 KB rows of partials), warp w adds row blocks w, w + 32, ... in order with four loads in
// flight, and the 32 warp sums are combined in warp order: the same bits on every run.
constexpr int CH_MERGE_THREADS = 1024;
constexpr int CH_MERGE_WARPS = CH_MERGE_THREADS / 32;
__global__ void __launch_bounds__(CH_MERGE_THREADS) ch_merge_a(const ChPart* __restrict__ part, int blocks, uint64_t rows,
                                                         uint32_t C, qp_stats_t* __restrict__ out,
                                                         unsigned* __restrict__ status)
{
    __shared__ double s_s[CH_MERGE_WARPS][32], s_sa[CH_MERGE_WARPS][32];
    __shared__ float s_mn[CH_MERGE_WARPS][32], s_mx[CH_MERGE_WARPS][32];
    __shared__ unsigned long long s_bad[CH_MERGE_WARPS][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t c = blockIdx.x * 32 + lane;
    const float inf = __int_as_float(0x7F800000);
    double s = 0.0, sa = 0.0;
    float mn = inf, mx = -inf;
    unsigned long long bad = 0;
    if (c < C) {
        for (int b0 = warp; b0 < blocks; b0 += 4 * CH_MERGE_WARPS) {
            ChPart p[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int b = b0 + u * CH_MERGE_WARPS;
                if (b < blocks) p[u] = part[(size_t)b * C + c];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (b0 + u * CH_MERGE_WARPS >= blocks) break;
                s += p[u].s0;
                sa += p[u].s1;
                mn = fminf(mn, p[u].mn);
                mx = fmaxf(mx, p[u].mx);
                bad += p[u].bad;
            }
        }
    }
    s_s[warp][lane] = s; s_sa[warp][lane] = sa; s_mn[warp][lane] = mn; s_mx[warp][lane] = mx; s_bad[warp][lane] = bad;
    __syncthreads();
    if (warp != 0 || c >= C) return;
    for (int w = 1; w < CH_MERGE_WARPS; ++w) {
        s += s_s[w][lane];
        sa += s_sa[w][lane];
        mn = fminf(mn, s_mn[w][lane]);
        mx = fmaxf(mx, s_mx[w][lane]);
        bad += s_bad[w][lane];
    }
    const unsigned long long nf = rows - bad;
    qp_stats_t st;
    st.n = rows;
    st.nonfinite = bad;
    st.mean = nf ? s / (double)nf : 0.0;
    st.mean_abs = nf ? sa / (double)nf : 0.0;
    st.mad = 0.0;
    st.var = 0.0;
    st.min = nf ? (double)mn : 0.0;
    st.max = nf ? (double)mx : 0.0;
    st.hist_peak = 0;
    st.hist_bins = 0;
    st.reserved = 0;
    out[c] = st;
    if (bad) atomicOr(status, QP_DEV_NONFINITE);
}

template <typename T, int V>
__global__ void __launch_bounds__(CH_STATS_MAX_THREADS) ch_stats_b(const T* __restrict__ x, uint64_t rows, uint32_t C,
                                                         const qp_stats_t* __restrict__ st, ChPart* __restrict__ part)
{
    const uint32_t col0 = (blockIdx.y * blockDim.x + threadIdx.x) * V;
    if (col0 >= C) return;
    float m_hi[V], m_lo[V];                               // each channel's mean as an unevaluated fp32 pair
    double sd[V], sv[V];
#pragma unroll
    for (int i = 0; i < V; ++i) {
        const double mean = st[col0 + i].mean;
        m_hi[i] = (float)mean;
        m_lo[i] = (float)(mean - (double)m_hi[i]);
        sd[i] = 0.0;
        sv[i] = 0.0;
    }
    constexpr int CH_ROWS_IN_FLIGHT = ChRows<V>::N;
    const uint64_t step = gridDim.x;
    for (uint64_t r0 = blockIdx.x; r0 < rows; r0 += CH_ROWS_IN_FLIGHT * step) {
        float e[CH_ROWS_IN_FLIGHT][V];
#pragma unroll
        for (int u = 0; u < CH_ROWS_IN_FLIGHT; ++u) {
            const uint64_t r = r0 + u * step;
            if (r < rows) ch_load<T, V>(x + r * C + col0, e[u]);
        }
        float d1[V], d2[V];
#pragma unroll
        for (int i = 0; i < V; ++i) { d1[i] = 0.f; d2[i] = 0.f; }
#pragma unroll
        for (int u = 0; u < CH_ROWS_IN_FLIGHT; ++u) {
            if (r0 + u * step >= rows) break;
#pragma unroll
            for (int i = 0; i < V; ++i) {
                const float v = e[u][i];
                if (!qp_is_finite(v)) continue;
                const float d = __fsub_rn(__fsub_rn(v, m_hi[i]), m_lo[i]);
                d1[i] += fabsf(d);
                d2[i] = fmaf(d, d, d2[i]);
            }
        }
#pragma unroll
        for (int i = 0; i < V; ++i) { sd[i] += (double)d1[i]; sv[i] += (double)d2[i]; }
    }
    ChPart* dst = part + (size_t)blockIdx.x * C + col0;
#pragma unroll
    for (int i = 0; i < V; ++i) {
        dst[i].s0 = sd[i];
        dst[i].s1 = sv[i];
    }
}

__global__ void __launch_bounds__(CH_MERGE_THREADS) ch_merge_b(const ChPart* __restrict__ part, int blocks, uint32_t C,
                                                         qp_stats_t* __restrict__ out)
{
    __shared__ double s_d[CH_MERGE_WARPS][32], s_v[CH_MERGE_WARPS][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t c = blockIdx.x * 32 + lane;
    double sd = 0.0, sv = 0.0;
    if (c < C) {
        for (int b0 = warp; b0 < blocks; b0 += 4 * CH_MERGE_WARPS) {
            double a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int bb = b0 + u * CH_MERGE_WARPS;
                if (bb < blocks) {
                    a[u] = part[(size_t)bb * C + c].s0;
                    b[u] = part[(size_t)bb * C + c].s1;
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (b0 + u * CH_MERGE_WARPS >= blocks) break;
                sd += a[u];
                sv += b[u];
            }
        }
    }
    s_d[warp][lane] = sd;
    s_v[warp][lane] = sv;
    __syncthreads();
    if (warp != 0 || c >= C) return;
    for (int w = 1; w < CH_MERGE_WARPS; ++w) {
        sd += s_d[w][lane];
        sv += s_v[w][lane];
    }
    const unsigned long long nf = out[c].n - out[c].nonfinite;
    out[c].mad = nf ? sd / (double)nf : 0.0;
    out[c].var = nf ? sv / (double)nf : 0.0;
}

__global__ void __launch_bounds__(128) ch_clip_kernel(const qp_stats_t* __restrict__ st, uint32_t C, int bits, int method,
                                                      int dist, int bmode, double F, qp_qparams_t* __restrict__ qp_out,
                                                      unsigned* __restrict__ status)
{
    const uint32_t c = blockIdx.x * 128 + threadIdx.x;
    if (c >= C) return;
    double lo, hi;
    qp_clip_ends(st[c], method, dist, bmode, bits, F, lo, hi);
    qp_qparams_t q;
    const int rc = qp_fill_qparams(lo, hi, bits, &q);
    qp_out[c] = q;
    if (rc == QP_WARN_DEGENERATE) atomicOr(status, QP_DEV_DEGENERATE);
}

// ---- quantize + pack
//
// A warp owns a tile of 1024 consecutive elements (= 32 * bits output words) and never waits for
// another warp: coalesced 16-byte loads (lane l takes vectors l, l + 32, ..., all issued first),
// every element quantized with its channel's parameters from the table in shared memory, 16-bit
// codes into the warp's own 32 x 17-word staging rows (row = 32 consecutive elements, one pad
// word: conflict-free both ways), then lane l packs row l into `bits` words.

constexpr int CH_WARPS = CH_THREADS / 32;
constexpr int CH_WTILE = 1024;                    // elements per warp tile
constexpr int CH_STAGE_WORDS = 32 * 17;           // per warp

// staging word that holds the codes of tile elements le, le + 1 (le even)
__device__ __forceinline__ int ch_code_word(int le) { return (le >> 1) + (le >> 5); }

// Per-channel parameters in shared memory as four arrays [C] (lo, hi, scale, inv_scale): a lane
// reads the parameters of its 4 consecutive channels as one 16-byte vector per array, and the
// lanes of a warp read consecutive vectors (no bank conflicts).
struct ChTable {
    const float *lo, *hi, *scale, *inv;
};
__device__ __forceinline__ ChTable ch_load_table(const qp_qparams_t* __restrict__ d_qp, uint32_t C, int bits, float* tab,
                                                 unsigned* status)
{
    bool mismatch = false;
    for (uint32_t c = threadIdx.x; c < C; c += CH_THREADS) {
        const qp_qparams_t q = d_qp[c];
        tab[c] = q.lo;
        tab[C + c] = q.hi;
        tab[2 * C + c] = q.scale;
        tab[3 * C + c] = q.inv_scale;
        mismatch |= q.bits != bits;
    }
    if (mismatch && blockIdx.x == 0) atomicOr(status, QP_DEV_BITS_MISMATCH);
    ChTable t = {tab, tab + C, tab + 2 * C, tab + 3 * C};
    return t;
}
__device__ __forceinline__ void ch_lds4(const float* p, float (&v)[4])
{
    const float4 a = *reinterpret_cast<const float4*>(p);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
}

// BITS > 0: the bit-width as a compile-time constant (shifts become immediates); 0: `bits_rt`.
template <typename T, bool VEC, int BITS>
__global__ void __launch_bounds__(CH_THREADS) ch_pack_kernel(const T* __restrict__ x, uint64_t n, uint32_t C, int bits_rt,
                                                             const qp_qparams_t* __restrict__ d_qp,
                                                             uint32_t* __restrict__ out, uint64_t total_words,
                                                             uint64_t ntiles, uint64_t el0, unsigned* __restrict__ status)
{
    // x, n, out, total_words and ntiles describe the part of the tensor this launch packs; el0 = index of
    // x[0] in the whole tensor (a multiple of the warp tile), which fixes the channel of every element
    extern __shared__ __align__(16) unsigned char raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int bits = BITS ? BITS : bits_rt;
    uint32_t* codes = reinterpret_cast<uint32_t*>(raw + (size_t)C * sizeof(float4)) + warp * CH_STAGE_WORDS;
    const ChTable tab = ch_load_table(d_qp, C, bits, reinterpret_cast<float*>(raw), status);
    __syncthreads();
    constexpr int EPV = qp_span<T>::EPV;
    constexpr int NV = CH_WTILE / (32 * EPV);                  // vectors per lane and tile: 8 (f32) or 4 (bf16)
    const unsigned mask = (1u << bits) - 1u;
    const uint32_t cstep = (uint32_t)((32u * EPV) % C);        // channel advance from one of a lane's vectors to the next
    const uint64_t wstride = (uint64_t)gridDim.x * CH_WARPS;
    for (uint64_t tile = (uint64_t)blockIdx.x * CH_WARPS + warp; tile < ntiles; tile += wstride) {
        const uint64_t base = tile * CH_WTILE;
        if (VEC) {
            const bool full = base + CH_WTILE <= n;              // no element of the tile lies beyond the tensor
            float e[NV][EPV];
#pragma unroll
            for (int j = 0; j < NV; ++j) {
                const uint64_t el = base + (uint64_t)(j * 32 + lane) * EPV;
                if (full || el + EPV <= n) {
                    qp_load_vec(x + el, e[j]);
                } else {
#pragma unroll
                    for (int i = 0; i < EPV; ++i) e[j][i] = el + i < n ? qp_load_one(x + el + i) : 0.f;
                }
            }
            uint32_t c = (uint32_t)((el0 + base + (uint64_t)lane * EPV) % C);
#pragma unroll
            for (int j = 0; j < NV; ++j) {
                const int le = (j * 32 + lane) * EPV;
                const uint64_t el = base + le;
                unsigned cd[EPV];
#pragma unroll
                for (int h = 0; h < EPV; h += 4) {               // EPV divides C: the vector stays in one row
                    float lo[4], hi[4], inv[4];
                    ch_lds4(tab.lo + QP_CK(c + h, C - 3), lo);
                    ch_lds4(tab.hi + QP_CK(c + h, C - 3), hi);
                    ch_lds4(tab.inv + QP_CK(c + h, C - 3), inv);
#pragma unroll
                    for (int i = 0; i < 4; ++i) cd[h + i] = qp_code(e[j][h + i], lo[i], hi[i], inv[i], mask);
                }
                if (!full) {
#pragma unroll
                    for (int i = 0; i < EPV; ++i) cd[i] = el + i < n ? cd[i] : 0u;
                }
#pragma unroll
                for (int i = 0; i < EPV; i += 2) codes[QP_CK(ch_code_word(le + i), CH_STAGE_WORDS)] = cd[i] | (cd[i + 1] << 16);
                c += cstep;
                if (c >= C) c -= C;
            }
        } else {
            unsigned short* ch = reinterpret_cast<unsigned short*>(codes);
            for (int k = 0; k < 32; ++k) {
                const int le = k * 32 + lane;
                const uint64_t el = base + le;
                unsigned cd = 0u;
                if (el < n) {
                    const uint32_t c = (uint32_t)((el0 + el) % C);
                    cd = qp_code(qp_load_one(x + el), tab.lo[c], tab.hi[c], tab.inv[c], mask);
                }
                ch[le + ((le >> 5) << 1)] = (unsigned short)cd;
            }
        }
        __syncwarp();
        {
            const uint64_t w0 = (tile * 32 + lane) * (uint64_t)bits;          // this lane's group of 32 elements
            if (w0 < total_words) {
                uint32_t w[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) w[j] = codes[17 * lane + j];
                unsigned long long acc = 0ull;
                int fill = 0;
                uint32_t* dst = out + w0;
                const uint32_t* end = out + total_words;
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const unsigned cd = (w[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu;
                    acc |= (unsigned long long)cd << fill;
                    fill += bits;
                    if (fill >= 32) {
                        if (dst < end) *dst = (uint32_t)acc;
                        ++dst;
                        acc >>= 32;
                        fill -= 32;
                    }
                }
            }
        }
        __syncwarp();
    }
}

// ---- unpack + dequantize (mirror image)

__device__ __forceinline__ float ch_code_to_float(unsigned c) { return __fsub_rn(__uint_as_float(0x4B000000u | c), 8388608.0f); }

__device__ __forceinline__ void ch_store4(float* y, uint64_t el, const float (&v)[4])
{
    __stcs(reinterpret_cast<float4*>(y + el), make_float4(v[0], v[1], v[2], v[3]));   // streaming: not read again here
}
__device__ __forceinline__ void ch_store4(unsigned short* y, uint64_t el, const float (&v)[4])
{
    uint2 o;
    o.x = (unsigned)qp_f32_to_bf16(v[0]) | ((unsigned)qp_f32_to_bf16(v[1]) << 16);
    o.y = (unsigned)qp_f32_to_bf16(v[2]) | ((unsigned)qp_f32_to_bf16(v[3]) << 16);
    __stcs(reinterpret_cast<uint2*>(y + el), o);
}
__device__ __forceinline__ void ch_store1(float* y, uint64_t el, float v) { y[el] = v; }
__device__ __forceinline__ void ch_store1(unsigned short* y, uint64_t el, float v) { y[el] = qp_f32_to_bf16(v); }

template <typename TO, bool VEC, int BITS>
__global__ void __launch_bounds__(CH_THREADS) ch_unpack_kernel(const uint32_t* __restrict__ in, uint64_t n, uint32_t C,
                                                               int bits_rt, const qp_qparams_t* __restrict__ d_qp,
                                                               TO* __restrict__ y, uint64_t total_words, uint64_t ntiles,
                                                               uint64_t el0, unsigned* __restrict__ status)
{
    // in, n, y, total_words, ntiles: the part this launch unpacks; el0 = index of y[0] in the whole tensor
    extern __shared__ __align__(16) unsigned char raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int bits = BITS ? BITS : bits_rt;
    uint32_t* codes = reinterpret_cast<uint32_t*>(raw + (size_t)C * sizeof(float4)) + warp * CH_STAGE_WORDS;
    const ChTable tab = ch_load_table(d_qp, C, bits, reinterpret_cast<float*>(raw), status);
    __syncthreads();
    const unsigned mask = (1u << bits) - 1u;
    const uint32_t cstep = (uint32_t)(128u % C);               // a lane's vectors of 4 are 128 elements apart
    const uint64_t wstride = (uint64_t)gridDim.x * CH_WARPS;
    for (uint64_t tile = (uint64_t)blockIdx.x * CH_WARPS + warp; tile < ntiles; tile += wstride) {
        const uint64_t base = tile * CH_WTILE;
        {
            // this lane's group of 32 elements: `bits` words -> 32 codes -> its staging row
            const uint64_t w0 = (tile * 32 + lane) * (uint64_t)bits;
            uint32_t w[16];
#pragma unroll
            for (int m = 0; m < 16; ++m) w[m] = (m < bits && w0 + m < total_words) ? __ldg(in + w0 + m) : 0u;
            if (BITS) {
#pragma unroll
                for (int i = 0; i < 32; i += 2) {              // positions known at compile time
                    unsigned two[2];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int bit = (i + h) * (BITS ? BITS : 1), word = bit >> 5, sh = bit & 31;
                        unsigned cd = w[word] >> sh;
                        if (sh + (BITS ? BITS : 1) > 32) cd |= w[(word + 1) & 15] << (32 - sh);
                        two[h] = cd & mask;
                    }
                    codes[17 * lane + (i >> 1)] = two[0] | (two[1] << 16);
                }
            } else {
                unsigned long long acc = 0ull;                 // bits not yet consumed, oldest lowest
                int have = 0, i = 0;
                unsigned prev = 0u;
#pragma unroll
                for (int m = 0; m < 16; ++m) {
                    if (m < bits) {
                        acc |= (unsigned long long)w[m] << have;
                        have += 32;
                        while (have >= bits) {
                            const unsigned cd = (unsigned)acc & mask;
                            acc >>= bits;
                            have -= bits;
                            if (i & 1) codes[17 * lane + (i >> 1)] = prev | (cd << 16);
                            else       prev = cd;
                            ++i;
                        }
                    }
                }
            }
        }
        __syncwarp();
        if (VEC) {
            uint32_t c = (uint32_t)((el0 + base + (uint64_t)lane * 4) % C);
#pragma unroll
            for (int j = 0; j < CH_WTILE / 128; ++j) {
                const int le = (j * 32 + lane) * 4;
                const uint64_t el = base + le;
                const uint32_t a = codes[ch_code_word(le)], b = codes[ch_code_word(le + 2)];
                const unsigned cd[4] = {a & 0xFFFFu, a >> 16, b & 0xFFFFu, b >> 16};
                float v[4], lo[4], sc[4];
                ch_lds4(tab.lo + QP_CK(c, C - 3), lo);
                ch_lds4(tab.scale + QP_CK(c, C - 3), sc);
#pragma unroll
                for (int i = 0; i < 4; ++i) v[i] = fmaf(ch_code_to_float(cd[i]), sc[i], lo[i]);
                if (el + 4 <= n) {
                    ch_store4(y, el, v);
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (el + i < n) ch_store1(y, el + i, v[i]);
                }
                c += cstep;
                if (c >= C) c -= C;
            }
        } else {
            const unsigned short* ch = reinterpret_cast<const unsigned short*>(codes);
            for (int k = 0; k < 32; ++k) {
                const int le = k * 32 + lane;
                const uint64_t el = base + le;
                if (el < n) {
                    const uint32_t c = (uint32_t)((el0 + el) % C);
                    ch_store1(y, el, fmaf(ch_code_to_float(ch[le + ((le >> 5) << 1)]), tab.scale[c], tab.lo[c]));
                }
            }
        }
        __syncwarp();
    }
}

// ---- whole warp tiles on the fast path (aligned tensor, channels a multiple of the vector, 1..8 bits)
//
// The per-tensor packer's warp tile (1024 elements = 32 * BITS words: coalesced 16-byte loads, four codes
// to a "quad", quads across the warp through a swizzled 1 KB buffer, a lane then owns 32 consecutive
// elements = BITS words, coalesced word stores) with the quantizers of a vector's four channels read
// from the shared table as one 16-byte vector per array.  The staging of 16-bit codes and the
// element-by-element bit assembly of the generic kernel above took it to 0.6 of the copy peak; the
// generic kernel keeps the last partial tile, 16 bits and the unaligned shapes.
__device__ __forceinline__ int ch_swz(int p) { return ((((p >> 2) ^ ((p >> 5) & 1)) << 2) | (p & 3)); }

template <int BITS, typename T>
__global__ void __launch_bounds__(CH_THREADS) ch_pack_fast(const T* __restrict__ x, uint64_t ntiles, uint32_t C,
                                                           const qp_qparams_t* __restrict__ d_qp,
                                                           uint32_t* __restrict__ out, unsigned* __restrict__ status)
{
    extern __shared__ __align__(16) unsigned char raw[];
    constexpr int EPV = qp_span<T>::EPV;
    constexpr int NLOAD = CH_WTILE / (32 * EPV);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* sw = reinterpret_cast<uint32_t*>(raw + (size_t)C * sizeof(float4)) + warp * 256;
    const ChTable tab = ch_load_table(d_qp, C, BITS, reinterpret_cast<float*>(raw), status);
    __syncthreads();
    constexpr unsigned mask = (1u << BITS) - 1u;
    const uint32_t cstep = (uint32_t)((32u * EPV) % C);        // channel advance from one of a lane's vectors to the next
    const uint64_t wstride = (uint64_t)gridDim.x * CH_WARPS;
    for (uint64_t tile = (uint64_t)blockIdx.x * CH_WARPS + warp; tile < ntiles; tile += wstride) {
        const T* xt = x + tile * CH_WTILE;
        float e[NLOAD][EPV];
#pragma unroll
        for (int j = 0; j < NLOAD; ++j) qp_load_vec(xt + (j * 32 + lane) * EPV, e[j]);
        uint32_t c = (uint32_t)((tile * CH_WTILE + (uint64_t)lane * EPV) % C);
#pragma unroll
        for (int j = 0; j < NLOAD; ++j) {
            unsigned quads[EPV / 4];
#pragma unroll
            for (int h = 0; h < EPV / 4; ++h) {                  // EPV divides C: the vector stays in one row
                float lo[4], hi[4], inv[4];
                ch_lds4(tab.lo + QP_CK(c + 4 * h, C - 3), lo);
                ch_lds4(tab.hi + QP_CK(c + 4 * h, C - 3), hi);
                ch_lds4(tab.inv + QP_CK(c + 4 * h, C - 3), inv);
                unsigned r = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) r |= qp_code(e[j][4 * h + i], lo[i], hi[i], inv[i], mask) << (BITS * i);
                quads[h] = r;
            }
            if constexpr (EPV == 4) sw[ch_swz(j * 32 + lane)] = quads[0];
            else *reinterpret_cast<uint2*>(&sw[ch_swz(2 * (j * 32 + lane))]) = make_uint2(quads[0], quads[1]);
            c += cstep;
            if (c >= C) c -= C;
        }
        __syncwarp();
        const uint4 a = *reinterpret_cast<const uint4*>(&sw[ch_swz(8 * lane)]);
        const uint4 b = *reinterpret_cast<const uint4*>(&sw[ch_swz(8 * lane + 4)]);
        const uint32_t qd[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        uint32_t w[BITS];
#pragma unroll
        for (int m = 0; m < BITS; ++m) w[m] = 0u;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            constexpr int QB = 4 * BITS;
            const int bit = QB * k, word = bit >> 5, sh = bit & 31;
            w[word] |= qd[k] << sh;
            if (sh + QB > 32) w[(word + 1) % BITS] |= qd[k] >> (32 - sh);
        }
        uint32_t* ot = out + tile * (32 * BITS);
        __syncwarp();
#pragma unroll
        for (int m = 0; m < BITS; ++m) sw[lane * BITS + m] = w[m];
        __syncwarp();
#pragma unroll
        for (int m = 0; m < BITS; ++m) ot[m * 32 + lane] = sw[m * 32 + lane];
        __syncwarp();
    }
}

template <int BITS, typename TO>
__global__ void __launch_bounds__(CH_THREADS) ch_unpack_fast(const uint32_t* __restrict__ in, uint64_t ntiles, uint32_t C,
                                                             const qp_qparams_t* __restrict__ d_qp, TO* __restrict__ y,
                                                             unsigned* __restrict__ status)
{
    extern __shared__ __align__(16) unsigned char raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* sw = reinterpret_cast<uint32_t*>(raw + (size_t)C * sizeof(float4)) + warp * 256;
    const ChTable tab = ch_load_table(d_qp, C, BITS, reinterpret_cast<float*>(raw), status);
    __syncthreads();
    constexpr unsigned MASK = (1u << BITS) - 1u;
    constexpr int QB = 4 * BITS;
    constexpr unsigned QMASK = QB >= 32 ? 0xFFFFFFFFu : ((1u << (QB & 31)) - 1u);
    const uint32_t cstep = (uint32_t)(128u % C);               // a lane's vectors of 4 are 128 elements apart
    const uint64_t wstride = (uint64_t)gridDim.x * CH_WARPS;
    for (uint64_t tile = (uint64_t)blockIdx.x * CH_WARPS + warp; tile < ntiles; tile += wstride) {
        const uint32_t* it = in + tile * (32 * BITS);
        uint32_t w[BITS];
#pragma unroll
        for (int m = 0; m < BITS; ++m) sw[m * 32 + lane] = __ldg(it + m * 32 + lane);
        __syncwarp();
#pragma unroll
        for (int m = 0; m < BITS; ++m) w[m] = sw[lane * BITS + m];
        __syncwarp();
        uint32_t qd[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int bit = QB * k, word = bit >> 5, sh = bit & 31;
            uint32_t v = w[word] >> sh;
            if (sh + QB > 32) v |= w[(word + 1) % BITS] << (32 - sh);
            qd[k] = v & QMASK;
        }
        *reinterpret_cast<uint4*>(&sw[ch_swz(8 * lane)]) = make_uint4(qd[0], qd[1], qd[2], qd[3]);
        *reinterpret_cast<uint4*>(&sw[ch_swz(8 * lane + 4)]) = make_uint4(qd[4], qd[5], qd[6], qd[7]);
        __syncwarp();
        uint32_t mine[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) mine[j] = sw[ch_swz(j * 32 + lane)];
        uint32_t c = (uint32_t)((tile * CH_WTILE + (uint64_t)lane * 4) % C);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float v[4], lo[4], sc[4];
            ch_lds4(tab.lo + QP_CK(c, C - 3), lo);
            ch_lds4(tab.scale + QP_CK(c, C - 3), sc);
#pragma unroll
            for (int i = 0; i < 4; ++i) v[i] = fmaf(ch_code_to_float((mine[j] >> (BITS * i)) & MASK), sc[i], lo[i]);
            ch_store4(y, tile * CH_WTILE + (uint64_t)(j * 32 + lane) * 4, v);
            c += cstep;
            if (c >= C) c -= C;
        }
        __syncwarp();
    }
}

// ---- host side

int32_t ch_check(qp_ctx* ctx, uint64_t rows, uint32_t channels)
{
    if (channels < 1 || channels > QP_MAX_CHANNELS) return qp_fail(ctx, QP_ERR_INVALID_ARG, "channels must be 1..QP_MAX_CHANNELS");
    if (rows >= (1ull << 40) / channels) return qp_fail(ctx, QP_ERR_INVALID_ARG, "tensor too large");
    return QP_OK;
}

// block partials of the column reductions: grown on demand, kept by the context
int32_t ch_scratch(qp_ctx* ctx, size_t bytes)
{
    if (ctx->ch_part_bytes >= bytes) return QP_OK;
    if (ctx->d_ch_part) cudaFree(ctx->d_ch_part);
    ctx->d_ch_part = nullptr;
    ctx->ch_part_bytes = 0;
    if (cudaMalloc(&ctx->d_ch_part, bytes) != cudaSuccess) {
        cudaGetLastError();
        return qp_fail(ctx, QP_ERR_CUDA, "cannot allocate the channel partials");
    }
    ctx->ch_part_bytes = bytes;
    return QP_OK;
}

template <typename T>
int32_t stats_channels_typed(qp_ctx* ctx, const T* x, uint64_t rows, uint32_t C, qp_stats_t* d_out, cudaStream_t s)
{
    constexpr int EPV = qp_span<T>::EPV;
    const bool vec = (C % EPV == 0) && (((uintptr_t)x & 15u) == 0);
    const int V = vec ? EPV : 1;
    // one thread per group of V channels; a block spans all of them where 512 threads suffice
    const unsigned groups = C / V;
    unsigned threads = (groups + 31) / 32 * 32;
    if (threads > CH_STATS_MAX_THREADS) threads = CH_STATS_MAX_THREADS;
    const unsigned col_blocks = (groups + threads - 1) / threads;
    // about 640 threads per SM in all: 8 x 16-byte loads in flight per thread keep HBM busy, and the
    // partials (32 bytes per row block and channel) stay a few percent of the tensor
    uint64_t want = (uint64_t)ctx->sm_count * 640 / ((uint64_t)threads * col_blocks);
    if (want < 1) want = 1;
    if (want > 1024) want = 1024;
    const int row_blocks = (int)(rows < want ? rows : want);
    int32_t rc = ch_scratch(ctx, sizeof(ChPart) * (size_t)row_blocks * C);
    if (rc) return rc;
    ChPart* part = static_cast<ChPart*>(ctx->d_ch_part);
    const dim3 grid(row_blocks, col_blocks);
    const unsigned merge_blocks = (C + 31) / 32;
    if (vec) ch_stats_a<T, EPV><<<grid, threads, 0, s>>>(x, rows, C, part);
    else     ch_stats_a<T, 1><<<grid, threads, 0, s>>>(x, rows, C, part);
    ch_merge_a<<<merge_blocks, CH_MERGE_THREADS, 0, s>>>(part, row_blocks, rows, C, d_out, ctx->d_status);
    if (vec) ch_stats_b<T, EPV><<<grid, threads, 0, s>>>(x, rows, C, d_out, part);
    else     ch_stats_b<T, 1><<<grid, threads, 0, s>>>(x, rows, C, d_out, part);
    ch_merge_b<<<merge_blocks, CH_MERGE_THREADS, 0, s>>>(part, row_blocks, C, d_out);
    ctx->launches += 4;
    return qp_check_launch(ctx, "qp_stats_channels");
}

size_t ch_pack_smem(uint32_t C) { return (size_t)C * sizeof(float4) + (size_t)CH_WARPS * CH_STAGE_WORDS * sizeof(uint32_t); }

template <typename K>
bool ch_allow_smem(K kernel, size_t bytes)
{
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess;
}

}  // namespace

extern "C" int32_t qp_stats_channels(qp_ctx* ctx, const void* d_x, int dtype, uint64_t rows, uint32_t channels,
                                     qp_stats_t* d_out, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (dtype != QP_F32 && dtype != QP_BF16) return qp_fail(ctx, QP_ERR_UNSUPPORTED_DTYPE, "dtype must be QP_F32 or QP_BF16");
    int32_t rc = ch_check(ctx, rows, channels);
    if (rc) return rc;
    if (!d_out || (rows > 0 && !d_x)) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null pointer");
    if (((uintptr_t)d_x & (dtype == QP_F32 ? 3u : 1u)) || ((uintptr_t)d_out & 7u))
        return qp_fail(ctx, QP_ERR_ALIGNMENT, "tensor or d_out not aligned");
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (rows == 0) {
        if (cudaMemsetAsync(d_out, 0, sizeof(qp_stats_t) * channels, s) != cudaSuccess)
            return qp_check_launch(ctx, "qp_stats_channels");
        return QP_OK;
    }
    if (dtype == QP_F32) return stats_channels_typed<float>(ctx, static_cast<const float*>(d_x), rows, channels, d_out, s);
    return stats_channels_typed<unsigned short>(ctx, static_cast<const unsigned short*>(d_x), rows, channels, d_out, s);
}

extern "C" int32_t qp_clip_qparams_channels_device(qp_ctx* ctx, const qp_stats_t* d_stats, uint32_t channels, int bits,
                                                   int method, int dist, int bmode, qp_qparams_t* d_qp_out, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    int32_t rc = ch_check(ctx, 0, channels);
    if (rc) return rc;
    if (!d_stats || !d_qp_out) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null pointer");
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    if (!qp_clip_method_closed_form(method))
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "method must be ACIQ (| INTERSECT) or MINMAX, optionally | MIDRISE");
    if ((dist != QP_DIST_LAPLACE && dist != QP_DIST_GAUSS) || (bmode != QP_B_MAD && bmode != QP_B_MEAN_ABS))
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "dist/bmode");
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    ch_clip_kernel<<<(channels + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        d_stats, channels, bits, method, dist, bmode, qp_host_aciq_F(bits, dist), d_qp_out, ctx->d_status);
    ctx->launches += 1;
    return qp_check_launch(ctx, "qp_clip_qparams_channels_device");
}

extern "C" int32_t qp_quantize_pack_channels(qp_ctx* ctx, const void* d_x, int dtype, uint64_t rows, uint32_t channels,
                                             int bits, const qp_qparams_t* d_qp, void* d_packed,
                                             uint64_t packed_capacity, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (dtype != QP_F32 && dtype != QP_BF16) return qp_fail(ctx, QP_ERR_UNSUPPORTED_DTYPE, "dtype must be QP_F32 or QP_BF16");
    int32_t rc = ch_check(ctx, rows, channels);
    if (rc) return rc;
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    uint64_t n = rows * channels;
    const uint64_t need = qp_packed_bytes(n, bits);
    if (packed_capacity < need) return qp_fail(ctx, QP_ERR_BUFFER_TOO_SMALL, "packed_capacity < qp_packed_bytes(n, bits)");
    if (!d_qp || (n > 0 && (!d_x || !d_packed))) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null pointer");
    if (((uintptr_t)d_x & (dtype == QP_F32 ? 3u : 1u)) || ((uintptr_t)d_packed & 15u) || ((uintptr_t)d_qp & 3u))
        return qp_fail(ctx, QP_ERR_ALIGNMENT, "tensor, d_packed (16 bytes) or d_qp not aligned");
    if (n == 0) return QP_OK;
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t smem = ch_pack_smem(channels);
    const uint64_t cap = (uint64_t)ctx->sm_count * 6;
    const int esz = dtype == QP_F32 ? 4 : 2;
    const bool vec = channels % (16 / esz) == 0 && ((uintptr_t)d_x & 15u) == 0;
    // whole warp tiles of an aligned tensor at 1..8 bits go through the fast kernel; the generic one takes
    // what is left (the last partial tile and the pad words), or everything
    const uint64_t nfast = (vec && bits <= 8) ? n / CH_WTILE : 0;
    const uint64_t el0 = nfast * CH_WTILE;
    uint32_t* out = static_cast<uint32_t*>(d_packed) + nfast * 32 * (uint64_t)bits;
    const uint64_t n_all = n;
    n = n_all - el0;
    const uint64_t total_words = need / 4 - nfast * 32 * (uint64_t)bits;
    const uint64_t groups = (total_words + bits - 1) / bits;
    const uint64_t ntiles = (groups + 31) / 32;                               // warp tiles, pad words included
    const uint64_t want = (ntiles + CH_WARPS - 1) / CH_WARPS;
    const unsigned blocks = (unsigned)(want < cap ? want : cap);
    bool ok = true;
    if (nfast) {
        const uint64_t fwant = (nfast + CH_WARPS - 1) / CH_WARPS;
        const unsigned fblocks = (unsigned)(fwant < cap ? fwant : cap);
        uint32_t* fout = static_cast<uint32_t*>(d_packed);
#define QP_CH_FAST(T, B)                                                                                               \
    do {                                                                                                               \
        ok = ch_allow_smem(ch_pack_fast<B, T>, smem);                                                                  \
        if (ok) ch_pack_fast<B, T><<<fblocks, CH_THREADS, smem, s>>>(static_cast<const T*>(d_x), nfast, channels,     \
                                                                    d_qp, fout, ctx->d_status);                       \
    } while (0)
#define QP_CH_FAST_BITS(T)                                                                                             \
    switch (bits) {                                                                                                    \
        case 1: QP_CH_FAST(T, 1); break;                                                                               \
        case 2: QP_CH_FAST(T, 2); break;                                                                               \
        case 3: QP_CH_FAST(T, 3); break;                                                                               \
        case 4: QP_CH_FAST(T, 4); break;                                                                               \
        case 5: QP_CH_FAST(T, 5); break;                                                                               \
        case 6: QP_CH_FAST(T, 6); break;                                                                               \
        case 7: QP_CH_FAST(T, 7); break;                                                                               \
        default: QP_CH_FAST(T, 8); break;                                                                              \
    }
        if (dtype == QP_F32) { QP_CH_FAST_BITS(float) } else { QP_CH_FAST_BITS(unsigned short) }
#undef QP_CH_FAST_BITS
#undef QP_CH_FAST
        if (!ok) return qp_check_launch(ctx, "qp_quantize_pack_channels (shared memory)");
        ctx->launches += 1;
        if (total_words == 0) return qp_check_launch(ctx, "qp_quantize_pack_channels");
    }
#define QP_CH_PACK(T, VEC, B)                                                                                          \
    do {                                                                                                               \
        ok = ch_allow_smem(ch_pack_kernel<T, VEC, B>, smem);                                                           \
        if (ok) ch_pack_kernel<T, VEC, B><<<blocks, CH_THREADS, smem, s>>>(x, n, channels, bits, d_qp, out,           \
                                                                          total_words, ntiles, el0, ctx->d_status);   \
    } while (0)
#define QP_CH_PACK_BITS(T)                                                                                             \
    switch (bits) {                                                                                                    \
        case 1: QP_CH_PACK(T, true, 1); break;                                                                         \
        case 2: QP_CH_PACK(T, true, 2); break;                                                                         \
        case 3: QP_CH_PACK(T, true, 3); break;                                                                         \
        case 4: QP_CH_PACK(T, true, 4); break;                                                                         \
        case 5: QP_CH_PACK(T, true, 5); break;                                                                         \
        case 6: QP_CH_PACK(T, true, 6); break;                                                                         \
        case 7: QP_CH_PACK(T, true, 7); break;                                                                         \
        case 8: QP_CH_PACK(T, true, 8); break;                                                                         \
        default: QP_CH_PACK(T, true, 16); break;                                                                       \
    }
    if (dtype == QP_F32) {
        const float* x = static_cast<const float*>(d_x) + el0;
        if (vec) { QP_CH_PACK_BITS(float) }
        else QP_CH_PACK(float, false, 0);
    } else {
        const unsigned short* x = static_cast<const unsigned short*>(d_x) + el0;
        if (vec) { QP_CH_PACK_BITS(unsigned short) }
        else QP_CH_PACK(unsigned short, false, 0);
    }
#undef QP_CH_PACK_BITS
#undef QP_CH_PACK
    if (!ok) return qp_check_launch(ctx, "qp_quantize_pack_channels (shared memory)");
    ctx->launches += 1;
    return qp_check_launch(ctx, "qp_quantize_pack_channels");
}

extern "C" int32_t qp_unpack_dequantize_channels(qp_ctx* ctx, const void* d_packed, uint64_t rows, uint32_t channels,
                                                 int bits, const qp_qparams_t* d_qp, void* d_y, int out_dtype,
                                                 void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (out_dtype != QP_F32 && out_dtype != QP_BF16) return qp_fail(ctx, QP_ERR_UNSUPPORTED_DTYPE, "out_dtype");
    int32_t rc = ch_check(ctx, rows, channels);
    if (rc) return rc;
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    const uint64_t n = rows * channels;
    if (!d_qp || (n > 0 && (!d_packed || !d_y))) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null pointer");
    if (((uintptr_t)d_packed & 15u) || ((uintptr_t)d_qp & 3u) || ((uintptr_t)d_y & (out_dtype == QP_F32 ? 3u : 1u)))
        return qp_fail(ctx, QP_ERR_ALIGNMENT, "d_packed (16 bytes), d_qp or d_y not aligned");
    if (n == 0) return QP_OK;
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t smem = ch_pack_smem(channels);
    const uint64_t cap = (uint64_t)ctx->sm_count * 6;
    const bool vec = channels % 4 == 0 && ((uintptr_t)d_y & (out_dtype == QP_F32 ? 15u : 7u)) == 0;
    // whole warp tiles at 1..8 bits go through the fast kernel, the generic one takes what is left
    const uint64_t nfast = (vec && bits <= 8) ? n / CH_WTILE : 0;
    const uint64_t el0 = nfast * CH_WTILE;
    const uint64_t total_words = qp_packed_bytes(n, bits) / 4 - nfast * 32 * (uint64_t)bits;
    const uint32_t* in = static_cast<const uint32_t*>(d_packed) + nfast * 32 * (uint64_t)bits;
    bool ok = true;
    if (nfast) {
        const uint64_t fwant = (nfast + CH_WARPS - 1) / CH_WARPS;
        const unsigned fblocks = (unsigned)(fwant < cap ? fwant : cap);
        const uint32_t* fin = static_cast<const uint32_t*>(d_packed);
#define QP_CH_FAST(T, B)                                                                                               \
    do {                                                                                                               \
        ok = ch_allow_smem(ch_unpack_fast<B, T>, smem);                                                                \
        if (ok) ch_unpack_fast<B, T><<<fblocks, CH_THREADS, smem, s>>>(fin, nfast, channels, d_qp,                    \
                                                                      static_cast<T*>(d_y), ctx->d_status);           \
    } while (0)
#define QP_CH_FAST_BITS(T)                                                                                             \
    switch (bits) {                                                                                                    \
        case 1: QP_CH_FAST(T, 1); break;                                                                               \
        case 2: QP_CH_FAST(T, 2); break;                                                                               \
        case 3: QP_CH_FAST(T, 3); break;                                                                               \
        case 4: QP_CH_FAST(T, 4); break;                                                                               \
        case 5: QP_CH_FAST(T, 5); break;                                                                               \
        case 6: QP_CH_FAST(T, 6); break;                                                                               \
        case 7: QP_CH_FAST(T, 7); break;                                                                               \
        default: QP_CH_FAST(T, 8); break;                                                                              \
    }
        if (out_dtype == QP_F32) { QP_CH_FAST_BITS(float) } else { QP_CH_FAST_BITS(unsigned short) }
#undef QP_CH_FAST_BITS
#undef QP_CH_FAST
        if (!ok) return qp_check_launch(ctx, "qp_unpack_dequantize_channels (shared memory)");
        ctx->launches += 1;
        if (n == el0) return qp_check_launch(ctx, "qp_unpack_dequantize_channels");
    }
    const uint64_t n_rest = n - el0;
    const uint64_t ntiles = (n_rest + CH_WTILE - 1) / CH_WTILE;
    const uint64_t want = (ntiles + CH_WARPS - 1) / CH_WARPS;
    const unsigned blocks = (unsigned)(want < cap ? want : cap);
#define QP_CH_UNPACK(T, VEC, B)                                                                                        \
    do {                                                                                                               \
        ok = ch_allow_smem(ch_unpack_kernel<T, VEC, B>, smem);                                                         \
        if (ok) ch_unpack_kernel<T, VEC, B><<<blocks, CH_THREADS, smem, s>>>(in, n_rest, channels, bits, d_qp, y,     \
                                                                            total_words, ntiles, el0, ctx->d_status); \
    } while (0)
#define QP_CH_UNPACK_BITS(T)                                                                                           \
    switch (bits) {                                                                                                    \
        case 1: QP_CH_UNPACK(T, true, 1); break;                                                                       \
        case 2: QP_CH_UNPACK(T, true, 2); break;                                                                       \
        case 3: QP_CH_UNPACK(T, true, 3); break;                                                                       \
        case 4: QP_CH_UNPACK(T, true, 4); break;                                                                       \
        case 5: QP_CH_UNPACK(T, true, 5); break;                                                                       \
        case 6: QP_CH_UNPACK(T, true, 6); break;                                                                       \
        case 7: QP_CH_UNPACK(T, true, 7); break;                                                                       \
        case 8: QP_CH_UNPACK(T, true, 8); break;                                                                       \
        default: QP_CH_UNPACK(T, true, 16); break;                                                                     \
    }
    if (out_dtype == QP_F32) {
        float* y = static_cast<float*>(d_y) + el0;
        if (vec) { QP_CH_UNPACK_BITS(float) }
        else QP_CH_UNPACK(float, false, 0);
    } else {
        unsigned short* y = static_cast<unsigned short*>(d_y) + el0;
        if (vec) { QP_CH_UNPACK_BITS(unsigned short) }
        else QP_CH_UNPACK(unsigned short, false, 0);
    }
#undef QP_CH_UNPACK_BITS
#undef QP_CH_UNPACK
    if (!ok) return qp_check_launch(ctx, "qp_unpack_dequantize_channels (shared memory)");
    ctx->launches += 1;
    return qp_check_launch(ctx, "qp_unpack_dequantize_channels");
}

// The channel-wise sender in one call: statistics -> per-channel clip -> quantize+pack, nothing read
// back to the host.  The statistics go to d_stats_out, or to a buffer the context keeps when that is NULL.
extern "C" int32_t qp_sender_channels_device(qp_ctx* ctx, const void* d_x, int dtype, uint64_t rows, uint32_t channels,
                                             int bits, int method, int bmode, void* d_packed, uint64_t packed_capacity,
                                             qp_qparams_t* d_qp_out, qp_stats_t* d_stats_out, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    int32_t rc = ch_check(ctx, rows, channels);
    if (rc) return rc;
    if (!d_qp_out) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null d_qp_out");
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    const bool use_ds = (method & ~QP_CLIP_MIDRISE) == QP_CLIP_DSACIQ;
    if (!use_ds && !qp_clip_method_closed_form(method))
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "method must be ACIQ (| INTERSECT), MINMAX or DSACIQ, optionally | MIDRISE");
    if (use_ds && bits > 8) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "the search supports 1..8 bits");
    if (packed_capacity < qp_packed_bytes(rows * channels, bits))
        return qp_fail(ctx, QP_ERR_BUFFER_TOO_SMALL, "packed_capacity < qp_packed_bytes(rows * channels, bits)");
    qp_stats_t* st = d_stats_out;
    if (!st) {
        const size_t need = sizeof(qp_stats_t) * (size_t)channels;
        if (ctx->ch_stats_bytes < need) {
            qp_device_guard guard(ctx->device);
            if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
            if (ctx->d_ch_stats) cudaFree(ctx->d_ch_stats);
            ctx->d_ch_stats = nullptr;
            ctx->ch_stats_bytes = 0;
            if (cudaMalloc(&ctx->d_ch_stats, need) != cudaSuccess) {
                cudaGetLastError();
                return qp_fail(ctx, QP_ERR_CUDA, "cannot allocate the channel statistics");
            }
            ctx->ch_stats_bytes = need;
        }
        st = static_cast<qp_stats_t*>(ctx->d_ch_stats);
    }
    rc = qp_stats_channels(ctx, d_x, dtype, rows, channels, st, stream);
    if (rc < 0) return rc;
    if (use_ds)
        rc = qp_dsaciq_search_channels(ctx, d_x, dtype, rows, channels, st, bits,
                                       bmode | ((method & QP_CLIP_MIDRISE) ? QP_B_MIDRISE : 0), QP_DEFAULT_STEPS,
                                       QP_DEFAULT_HIST_BINS, nullptr, d_qp_out, stream);
    else
        rc = qp_clip_qparams_channels_device(ctx, st, channels, bits, method, QP_DIST_LAPLACE, bmode, d_qp_out, stream);
    if (rc < 0) return rc;
    return qp_quantize_pack_channels(ctx, d_x, dtype, rows, channels, bits, d_qp_out, d_packed, packed_capacity, stream);
}
