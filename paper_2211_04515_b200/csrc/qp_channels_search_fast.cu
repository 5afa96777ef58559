// Channel-wise directed search (paper Sec. 3 "Directed Search", Eq. 1, run per column) through interval
// moments: the squared error of every candidate of every channel from ONE pass over the tensor, in
// place of scoring every element under every candidate (qp_channels_search.cu: (steps + 1) * 9 fp32
// instructions per element).
//
// For one candidate the code is a non-decreasing step function of x, so candidate k cuts the line at
// L - 1 thresholds T(k, j) = smallest float whose code is >= j.  Between two neighbours of the sorted
// union of a channel's thresholds every candidate's code is constant, so per channel
//     sum (x - Q_k(x))^2 = SXX + sum over codes j of [ N_j q_j^2 - 2 q_j SX_j ],
// with N_j, SX_j the count and the sum of (x - ref0) over the intervals that candidate k maps to code j
// (a difference of two prefix sums over the sorted intervals), q_j = level_k(j) - ref0, ref0 = the
// channel's minimum, and SXX = sum (x - ref0)^2, the same for every candidate.
//
//   ci_tables_kernel    block per channel: all thresholds by bisection over float bit patterns WITH THE
//                       QUANTIZER'S OWN CODE FUNCTION (exact), sorted in shared memory (bitonic)
//   ci_moments_kernel   the pass over x: a block owns a few neighbouring channels and all rows; an
//                       element finds its interval by binary search among its channel's sorted
//                       thresholds in shared memory and adds 1 to the interval's count and d to its sum,
//                       d = offset from the interval's reference point in units of u (a power of two;
//                       the difference is taken in fp64, where it is exact: integer sums, exact and
//                       order-independent).  d has 31 bits and goes in as two halves, so that all three
//                       additions are 32-bit shared-memory atomics (one 64-bit atomic per element is a
//                       compare-and-swap loop that collapses when many elements meet in one interval:
//                       1.6 ms at 2 bits on the ViT-Huge tensor)
//   ci_curve_kernel     block per channel: prefix sums over the intervals, then thread k evaluates
//                       candidate k from 2^bits prefix differences
// The only approximation is the rounding of each offset to u <= range / 2^30 (a channel of a few hundred
// elements whose range is set by outliers needs that: with 2^22 steps a candidate's error was off by 2e-6);
// the results do not depend on the order of execution.  The pick is
// the candidate-scoring path's kernel, fed with these sums.
#include "qp_internal.cuh"

QP_CK_UNIT

namespace {

constexpr int CI_TAB_THREADS = 256;
constexpr int CI_MOM_THREADS = 1024;
constexpr int CI_CURVE_THREADS = 128;
constexpr float CI_MAGIC = 8388608.0f;                 // 2^23: 0x4B000000 | j is the float 2^23 + j
constexpr unsigned long long CI_SUM_MASK = (1ull << 48) - 1ull;
constexpr size_t CI_SMEM_BUDGET = 226 * 1024;          // dynamic shared memory the moments kernel may ask for (of 227 KB)

// ---------------------------------------------------------------- thresholds, sorted

// block c: thresholds of channel c.  thr[c][k * L1 + j - 1] = T(k, j) (+inf: candidate not valid),
// bb[c][0 .. nthr) = the same values in ascending order, m[c] = how many are finite; the offsets' unit
// and the reference point go into setup[c] (u, inv_u, g_lo = the channel's minimum).
__global__ void __launch_bounds__(CI_TAB_THREADS) ci_tables_kernel(const qp_stats_t* __restrict__ st,
                                                                   const float4* __restrict__ cand,
                                                                   const int* __restrict__ valid, int ncp, int ncand,
                                                                   int bits, int nthr, int p2,
                                                                   qp_ds_setup* __restrict__ setup, float* __restrict__ thr,
                                                                   float* __restrict__ bb, unsigned* __restrict__ m_out)
{
    extern __shared__ float s_key[];                   // [p2]
    __shared__ float s_lo[CI_TAB_THREADS / 32], s_hi[CI_TAB_THREADS / 32];
    __shared__ float sg_lo, sg_hi;
    const uint32_t c = blockIdx.x;
    const int L1 = (1 << bits) - 1;
    const float inf = __int_as_float(0x7F800000);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    float lo = inf, hi = -inf;                         // union of the valid candidates' clip ranges
    for (int k = threadIdx.x; k < ncand; k += CI_TAB_THREADS)
        if (valid[(size_t)c * ncp + k]) {
            const float4 q = cand[(size_t)c * ncp + k];
            lo = fminf(lo, q.x);
            hi = fmaxf(hi, q.y);
        }
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_down_sync(0xFFFFFFFFu, lo, o));
        hi = fmaxf(hi, __shfl_down_sync(0xFFFFFFFFu, hi, o));
    }
    if (lane == 0) { s_lo[warp] = lo; s_hi[warp] = hi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < CI_TAB_THREADS / 32; ++w) { lo = fminf(lo, s_lo[w]); hi = fmaxf(hi, s_hi[w]); }
        sg_lo = lo;
        sg_hi = hi;
        // offsets are taken from a point at or above the channel's minimum and stay below max - min < 2^e:
        // in units of 2^(e - 31) they stay below 2^31, and 65535 of them add up to less than 2^47
        const double width = st[c].max - st[c].min;
        double u = 1.0;
        if (width > 0.0) {
            int e;
            frexp(width, &e);
            u = ldexp(1.0, e - 31);
        }
        setup[c].u = u;
        setup[c].inv_u = (float)(1.0 / u);             // a power of two
        setup[c].g_lo = (float)st[c].min;              // exact: the minimum is one of the elements
        setup[c].g_hi = (float)st[c].max;
    }
    __syncthreads();
    const float g_lo = sg_lo, g_hi = sg_hi;
    for (int t = threadIdx.x; t < p2; t += CI_TAB_THREADS) {
        float out = inf;
        if (t < nthr) {
            const int k = t / L1, j = 1 + t % L1;
            if (valid[(size_t)c * ncp + k] && g_hi > g_lo) {
                const float4 q = cand[(size_t)c * ncp + k];
                const unsigned mask = (unsigned)L1;
                auto pred = [&](float x) { return (int)qp_code(x, q.x, q.y, q.w, mask) >= j; };
                if (!pred(g_lo) && pred(g_hi)) out = qp_first_true(g_lo, g_hi, pred);
            }
            thr[(size_t)c * nthr + t] = out;
        }
        s_key[t] = out;
    }
    __syncthreads();
    // bitonic sort, ascending (p2 is a power of two; the padding is +inf)
    for (int k = 2; k <= p2; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = threadIdx.x; i < p2; i += CI_TAB_THREADS) {
                const int ixj = i ^ j;
                if (ixj > i) {
                    const float a = s_key[i], b = s_key[ixj];
                    const bool up = (i & k) == 0;
                    if ((a > b) == up) { s_key[i] = b; s_key[ixj] = a; }
                }
            }
            __syncthreads();
        }
    for (int t = threadIdx.x; t < nthr; t += CI_TAB_THREADS) bb[(size_t)c * nthr + t] = s_key[t];
    if (threadIdx.x == 0) {                            // finite entries come first
        int a = 0, b = nthr;
        while (a < b) {
            const int mid = (a + b) >> 1;
            if (s_key[mid] < inf) a = mid + 1; else b = mid;
        }
        m_out[c] = (unsigned)a;
    }
}

// ---------------------------------------------------------------- the pass over x

// Block b owns channels [b * cpb, b * cpb + cpb) and every row.  Thread = (channel slot, row lane): a warp
// reads cpb neighbouring elements of a few rows.  Shared memory per slot: the sorted thresholds (1-based)
// and three counters per interval, nthr + 1 words each.  tot[c][i] = count << 48 | sum of offsets of
// interval i (i = number of the channel's thresholds <= x), sumd2[c] = sum of squared offsets.
template <typename T>
__global__ void __launch_bounds__(CI_MOM_THREADS, 1) ci_moments_kernel(const T* __restrict__ x, uint64_t rows, uint32_t C,
                                                                       int cpb, int nthr, const float* __restrict__ bb,
                                                                       const unsigned* __restrict__ m_in,
                                                                       const qp_ds_setup* __restrict__ setup,
                                                                       unsigned long long* __restrict__ tot,
                                                                       double* __restrict__ sumd2)
{
    extern __shared__ __align__(16) unsigned char raw[];
    const int stride = nthr + 1;
    float* s_bb = reinterpret_cast<float*>(raw);                                  // [cpb][stride]
    unsigned* s_cnt = reinterpret_cast<unsigned*>(s_bb + (size_t)cpb * stride);   // [cpb][stride] elements
    unsigned* s_lo = s_cnt + (size_t)cpb * stride;                                // [cpb][stride] sum of the offsets' low 16 bits
    unsigned* s_hi = s_lo + (size_t)cpb * stride;                                 // [cpb][stride] sum of their high 15 bits
    double* s_d2 = reinterpret_cast<double*>(raw + ((size_t)cpb * stride * 16 + 7) / 8 * 8);   // [CI_MOM_THREADS]
    const float inf = __int_as_float(0x7F800000);
    const uint32_t c0 = blockIdx.x * (uint32_t)cpb;
    const int nch = (int)min((uint32_t)cpb, C - c0);
    for (int i = threadIdx.x; i < cpb * stride; i += CI_MOM_THREADS) {
        const int slot = i / stride, j = i - slot * stride;
        s_cnt[i] = 0u;
        s_lo[i] = 0u;
        s_hi[i] = 0u;
        s_bb[i] = (slot < nch && j >= 1) ? bb[(size_t)(c0 + slot) * nthr + (j - 1)] : inf;
    }
    __syncthreads();

    const int slot = threadIdx.x % cpb, rl = threadIdx.x / cpb, nl = CI_MOM_THREADS / cpb;
    double d2 = 0.0;
    if (rl < nl && slot < nch) {
        const uint32_t c = c0 + slot;
        const unsigned m = m_in[c];
        const float ref0 = setup[c].g_lo;
        const double inv_u = 1.0 / setup[c].u;          // a power of two
        const float* sb = s_bb + (size_t)slot * stride;
        unsigned* cnt = s_cnt + (size_t)slot * stride;
        unsigned* sl = s_lo + (size_t)slot * stride;
        unsigned* sh = s_hi + (size_t)slot * stride;
        const T* px = x + c;
        auto one = [&](float e, double& p) {
            if (!qp_is_finite(e)) return;
            unsigned lo = 0u, hi = m;
            while (lo < hi) {                           // largest i in [0, m] with sb[i] <= e (sb[0] counts as -inf)
                const unsigned mid = (lo + hi + 1u) >> 1;
                if (sb[QP_CK(mid, stride)] <= e) lo = mid; else hi = mid - 1u;
            }
            lo = QP_CK(lo, stride);
            const float ref = lo ? fmaxf(sb[lo], ref0) : ref0;
            const unsigned d = __double2uint_rn(((double)e - (double)ref) * inv_u);     // e >= ref; exact difference
            const double df = (double)d;
            p = fma(df, df, p);
            atomicAdd(&cnt[lo], 1u);
            atomicAdd(&sl[lo], d & 0xFFFFu);
            atomicAdd(&sh[lo], d >> 16);
        };
        uint64_t r = (uint64_t)rl;
        for (; r + 3ull * nl < rows; r += 4ull * nl) {   // four loads ahead of their look-ups
            float e[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) e[q] = qp_load_one(px + (r + (uint64_t)q * nl) * C);
#pragma unroll
            for (int q = 0; q < 4; ++q) one(e[q], d2);
        }
        for (; r < rows; r += nl) one(qp_load_one(px + r * C), d2);
    }
    s_d2[threadIdx.x] = d2;
    __syncthreads();
    if (rl == 0 && slot < nch) {                         // the row lanes of a channel, in lane order
        double t = 0.0;
        for (int l = 0; l < nl; ++l) t += s_d2[l * cpb + slot];
        sumd2[c0 + slot] = t;
    }
    for (int i = threadIdx.x; i < nch * stride; i += CI_MOM_THREADS) {
        const int sl = i / stride, j = i - sl * stride;
        tot[(size_t)(c0 + sl) * stride + j] =
            ((unsigned long long)s_cnt[i] << 48) | ((unsigned long long)s_lo[i] + ((unsigned long long)s_hi[i] << 16));
    }
}

// ---------------------------------------------------------------- every candidate from prefix sums

// block c.  Interval i (0..m) lies at offset r_i = max(bb[i], ref0) - ref0 from the channel's reference
// point (r_0 = 0), so its sum of (x - ref0) is N_i r_i + u S1_i.  PN / PSX are the exclusive prefix sums of
// the counts and of those sums; candidate k's code j covers the intervals [pos(T(k, j)), pos(T(k, j + 1))),
// pos(T) = number of thresholds <= T (all intervals from there on hold elements >= T, the ones before
// it elements < T), and the total of its squared error goes to part[c][k] for the pick.
__global__ void __launch_bounds__(CI_CURVE_THREADS) ci_curve_kernel(const unsigned long long* __restrict__ tot,
                                                                    const float* __restrict__ bb, const float* __restrict__ thr,
                                                                    const unsigned* __restrict__ m_in,
                                                                    const qp_ds_setup* __restrict__ setup,
                                                                    const double* __restrict__ sumd2,
                                                                    const float4* __restrict__ cand,
                                                                    const int* __restrict__ valid, int ncp, int ncand, int bits,
                                                                    int nthr, double* __restrict__ part)
{
    extern __shared__ __align__(16) unsigned char raw[];
    const int stride = nthr + 1;
    double* PN = reinterpret_cast<double*>(raw);                      // [nthr + 2]
    double* PSX = PN + (nthr + 2);                                    // [nthr + 2]
    float* s_bb = reinterpret_cast<float*>(PSX + (nthr + 2));         // [nthr + 1], 1-based
    __shared__ double c_n[CI_CURVE_THREADS], c_sx[CI_CURVE_THREADS], c_sxx[CI_CURVE_THREADS];
    __shared__ double s_sxx;
    const uint32_t c = blockIdx.x;
    const unsigned m = m_in[c];
    const qp_ds_setup s = setup[c];
    const double u = s.u, ref0 = (double)s.g_lo;
    const float inf = __int_as_float(0x7F800000);
    for (int i = threadIdx.x; i < stride; i += CI_CURVE_THREADS) s_bb[i] = i >= 1 ? bb[(size_t)c * nthr + (i - 1)] : -inf;
    __syncthreads();

    // exclusive prefix sums over intervals 0..m: thread t takes the chunk [t * per, t * per + per)
    const int count = (int)m + 1, per = (count + CI_CURVE_THREADS - 1) / CI_CURVE_THREADS;
    const int i0 = threadIdx.x * per, i1 = min(i0 + per, count);
    auto interval = [&](int i, double& n, double& sx, double& sxx) {
        const unsigned long long w = tot[(size_t)c * stride + i];
        n = (double)(w >> 48);
        const double s1 = u * (double)(w & CI_SUM_MASK);
        const double r = i ? fmax((double)s_bb[QP_CK(i, stride)], ref0) - ref0 : 0.0;
        sx = n * r + s1;
        sxx = n * r * r + 2.0 * r * s1;
    };
    {
        double a = 0.0, b = 0.0, d = 0.0;
        for (int i = i0; i < i1; ++i) {
            double n, sx, sxx;
            interval(i, n, sx, sxx);
            a += n; b += sx; d += sxx;
        }
        c_n[threadIdx.x] = a; c_sx[threadIdx.x] = b; c_sxx[threadIdx.x] = d;
    }
    __syncthreads();
    if (threadIdx.x == 0) {                              // chunk sums -> chunk offsets, in chunk order
        double a = 0.0, b = 0.0, d = 0.0;
        for (int t = 0; t < CI_CURVE_THREADS; ++t) {
            const double n = c_n[t], sx = c_sx[t];
            c_n[t] = a; c_sx[t] = b;
            a += n; b += sx; d += c_sxx[t];
        }
        s_sxx = d + u * u * sumd2[c];
    }
    __syncthreads();
    {
        double a = c_n[threadIdx.x], b = c_sx[threadIdx.x];
        for (int i = i0; i < i1; ++i) {
            double n, sx, sxx;
            interval(i, n, sx, sxx);
            PN[QP_CK(i, nthr + 2)] = a; PSX[QP_CK(i, nthr + 2)] = b;
            a += n; b += sx;
        }
        if (i1 == count && i0 < i1) { PN[count] = a; PSX[count] = b; }
    }
    if (count <= 0 && threadIdx.x == 0) { PN[0] = 0.0; PSX[0] = 0.0; }
    __syncthreads();

    const int L1 = (1 << bits) - 1;
    for (int k = threadIdx.x; k < ncp; k += CI_CURVE_THREADS) {
        double total = 0.0;
        if (k < ncand && valid[(size_t)c * ncp + k]) {
            const float4 q = cand[(size_t)c * ncp + k];
            total = s_sxx;
            unsigned prev = 0u;
            for (int j = 0; j <= L1; ++j) {
                unsigned next = m + 1u;                  // the last code runs to the end
                if (j < L1) {
                    const float T = thr[(size_t)c * nthr + (size_t)k * L1 + j];      // T(k, j + 1)
                    if (T < inf) {                       // pos(T): thresholds <= T among s_bb[1..m]
                        unsigned lo = 0u, hi = m;
                        while (lo < hi) {
                            const unsigned mid = (lo + hi + 1u) >> 1;
                            if (s_bb[QP_CK(mid, stride)] <= T) lo = mid; else hi = mid - 1u;
                        }
                        next = lo;
                    }
                }
                if (next < prev) next = prev;
                const double n = PN[QP_CK(next, nthr + 2)] - PN[QP_CK(prev, nthr + 2)];
                const double sx = PSX[next] - PSX[prev];
                const float level = fmaf(__fsub_rn(__uint_as_float(0x4B000000u | (unsigned)j), CI_MAGIC), q.z, q.x);
                const double a = (double)level - ref0;
                total += n * a * a - 2.0 * a * sx;
                prev = next;
            }
        }
        part[(size_t)c * ncp + k] = total;
    }
}

}  // namespace

// Scratch the interval form needs beyond the candidate path's (bytes), for `C` channels and `nthr` thresholds.
size_t qp_channel_interval_scratch_bytes(uint32_t C, int nthr)
{
    auto al = [](size_t v) { return (v + 255) / 256 * 256; };
    return al(sizeof(float) * (size_t)C * nthr) * 2 + al(sizeof(unsigned) * (size_t)C) + al(sizeof(double) * (size_t)C) +
           al(sizeof(unsigned long long) * (size_t)C * (nthr + 1));
}

// Whether the interval form applies: thresholds per channel that fit the shared-memory tables, and row
// counts that the packed count / carry fields hold.
bool qp_channel_interval_applies(uint64_t rows, int bits, int steps)
{
    const long long nthr = (long long)(steps + 1) * ((1 << bits) - 1);
    return nthr <= 2048 && rows >= 1 && rows <= 65535;
}

// Fills part[c][k] (one row block) with every candidate's total squared error.  `scratch` holds
// qp_channel_interval_scratch_bytes(C, nthr) bytes.
int32_t qp_launch_channel_interval_sums(qp_ctx* ctx, const void* d_x, int dtype, uint64_t rows, uint32_t C, int bits, int steps,
                                        int ncp, const qp_stats_t* d_stats, const float4* cand, const int* valid,
                                        qp_ds_setup* setup, char* scratch, double* part, cudaStream_t s)
{
    auto al = [](size_t v) { return (v + 255) / 256 * 256; };
    const int ncand = steps + 1, L1 = (1 << bits) - 1, nthr = ncand * L1;
    int p2 = 2;
    while (p2 < nthr) p2 <<= 1;
    size_t off = 0;
    float* thr = reinterpret_cast<float*>(scratch + off);            off += al(sizeof(float) * (size_t)C * nthr);
    float* bb = reinterpret_cast<float*>(scratch + off);             off += al(sizeof(float) * (size_t)C * nthr);
    unsigned* m = reinterpret_cast<unsigned*>(scratch + off);        off += al(sizeof(unsigned) * (size_t)C);
    double* sumd2 = reinterpret_cast<double*>(scratch + off);        off += al(sizeof(double) * (size_t)C);
    unsigned long long* tot = reinterpret_cast<unsigned long long*>(scratch + off);

    ci_tables_kernel<<<C, CI_TAB_THREADS, sizeof(float) * (size_t)p2, s>>>(d_stats, cand, valid, ncp, ncand, bits, nthr, p2,
                                                                         setup, thr, bb, m);
    // channels per block: one block per SM where the tables of that many channels fit in shared memory
    const size_t per_channel = 16 * (size_t)(nthr + 1);
    const size_t fixed = sizeof(double) * CI_MOM_THREADS + 8;
    int cpb = (int)((C + (uint32_t)ctx->sm_count - 1) / (uint32_t)ctx->sm_count);
    const int cap = (int)((CI_SMEM_BUDGET - fixed) / per_channel);
    if (cpb > cap) cpb = cap;
    if (cpb < 1) cpb = 1;
    const size_t smem = fixed + per_channel * (size_t)cpb;
    const unsigned blocks = (C + (unsigned)cpb - 1) / (unsigned)cpb;
    if (dtype == QP_F32) {
        if (cudaFuncSetAttribute(ci_moments_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return qp_check_launch(ctx, "qp_dsaciq_search_channels (interval shared memory)");
        ci_moments_kernel<float><<<blocks, CI_MOM_THREADS, smem, s>>>(static_cast<const float*>(d_x), rows, C, cpb, nthr, bb, m,
                                                                     setup, tot, sumd2);
    } else {
        if (cudaFuncSetAttribute(ci_moments_kernel<unsigned short>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess)
            return qp_check_launch(ctx, "qp_dsaciq_search_channels (interval shared memory)");
        ci_moments_kernel<unsigned short><<<blocks, CI_MOM_THREADS, smem, s>>>(static_cast<const unsigned short*>(d_x), rows, C,
                                                                              cpb, nthr, bb, m, setup, tot, sumd2);
    }
    const size_t csmem = sizeof(double) * 2 * (size_t)(nthr + 2) + sizeof(float) * (size_t)(nthr + 1);
    ci_curve_kernel<<<C, CI_CURVE_THREADS, csmem, s>>>(tot, bb, thr, m, setup, sumd2, cand, valid, ncp, ncand, bits, nthr, part);
    ctx->launches += 3;
    return qp_check_launch(ctx, "qp_dsaciq_search_channels (interval path)");
}
