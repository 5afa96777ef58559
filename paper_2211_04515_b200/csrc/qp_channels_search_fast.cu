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
//                       QUANTIZER'S OWN CODE FUNCTION (exact), sorted in shared memory (the monotone runs
//                       they come in, merged pairwise)
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

constexpr int CI_TAB_THREADS = 128;                    // small blocks: all channels of a ViT layer in one wave
constexpr int CI_MOM_THREADS = 1024;
constexpr int CI_CURVE_THREADS = 128;
constexpr float CI_MAGIC = 8388608.0f;                 // 2^23: 0x4B000000 | j is the float 2^23 + j
constexpr unsigned long long CI_SUM_MASK = (1ull << 48) - 1ull;
constexpr int CI_CELLS = 128;                          // uniform cells over the union of a channel's clip ranges
constexpr size_t CI_SMEM_BUDGET = 226 * 1024;          // dynamic shared memory the moments kernel may ask for (of 227 KB)

// Cell of x on a channel's grid (origin g0, inv_cw cells per unit): each operation rounded on its own, so
// the function is monotone in x; values beyond the grid go to the end cells.
__device__ __forceinline__ int ci_cell(float x, float g0, float inv_cw)
{
    const float t = __fmul_rn(__fsub_rn(x, g0), inv_cw);
    return __float2int_rd(fminf(fmaxf(t, 0.f), (float)(CI_CELLS - 1)));
}

// ---------------------------------------------------------------- thresholds, sorted

// block c: thresholds T(k, j) of channel c (+inf: candidate not valid).  bb[c][0 .. nthr) = their values in
// ascending order, pos[c][(j - 1) * ncand + k] = the number of thresholds <= T(k, j) (0xFFFF for +inf),
// m[c] = how many are finite; the offsets' unit, the reference point and the look-up
// grid go into setup[c] (u, inv_u, g_lo = the channel's minimum, gw / inv_gw = the grid).
__global__ void __launch_bounds__(CI_TAB_THREADS) ci_tables_kernel(const qp_stats_t* __restrict__ st,
                                                                   const float4* __restrict__ cand,
                                                                   const int* __restrict__ valid, int ncp, int ncand,
                                                                   int bits, int nthr, int p2,
                                                                   qp_ds_setup* __restrict__ setup,
                                                                   float* __restrict__ bb, unsigned* __restrict__ m_out,
                                                                   unsigned* __restrict__ cells,
                                                                   unsigned short* __restrict__ pos)
{
    extern __shared__ float s_key[];                   // p2 = nthr rounded up to 4: [p2] sorted, [p2] in (k, j) order, [p2] ordered runs
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
        setup[c].gw = lo;                              // origin of the look-up grid: the union of the clip ranges
        setup[c].inv_gw = hi > lo ? (float)((double)CI_CELLS / ((double)hi - (double)lo)) : 0.f;
    }
    __syncthreads();
    const float g_lo = sg_lo, g_hi = sg_hi;
    float* s_thr = s_key + p2;                         // [p2] thresholds in (k, j) order; s_key: the same, sorted
    // (threads walk the thresholds run by run: the lanes of a warp then work on one code boundary j, and
    // what costs more for some boundaries than for others - a wide bracket near zero, the rank sort of the
    // middle run below - does not hold up the lanes of the other boundaries)
    for (int r = threadIdx.x; r < p2; r += CI_TAB_THREADS) {
        float out = inf;
        const int k = r % ncand, t = r < nthr ? k * L1 + r / ncand : r;
        if (r < nthr) {
            const int j = 1 + r / ncand;
            if (valid[(size_t)c * ncp + k] && g_hi > g_lo) {
                const float4 q = cand[(size_t)c * ncp + k];
                const unsigned mask = (unsigned)L1;
                auto pred = [&](float x) { return (int)qp_code(x, q.x, q.y, q.w, mask) >= j; };
                // real arithmetic puts the threshold at lo + (j - 1/2) scale, and the rounding of the ends, the
                // scale and its reciprocal moves it by a few ulps of the larger end: a bracket of that width
                // takes a handful of evaluations of the code function instead of 32; the whole range is the
                // fall-back (the result is the same smallest float either way)
                const float est = fmaf((float)j - 0.5f, q.z, q.x);
                const float w = 2e-6f * fmaxf(fabsf(q.x), fabsf(q.y));
                const float xa = fmaxf(est - w, g_lo), xb = fminf(est + w, g_hi);
                if (xa < xb && !pred(xa) && pred(xb)) out = qp_first_true(xa, xb, pred);
                else if (!pred(g_lo) && pred(g_hi)) out = qp_first_true(g_lo, g_hi, pred);
            }
        }
        s_thr[t] = out;
    }
    __syncthreads();
    // Sorting.  The thresholds of one code boundary j ("run" j: k = 0 .. ncand - 1) move one way with k (the
    // middle boundary stays at the mean and only wobbles in its last bits), so the array is L1 short runs that
    // are cheap to put in order (a run that rises or falls with k is copied as it is or reversed, any other
    // run gets a rank sort of its own, ncand^2 comparisons) and are then merged pairwise.  (A bitonic sort of
    // the whole array took 170 us for 1280 channels at 4 bits, ranks summed over all runs 300 us.)
    float* s_run = s_thr + p2;                          // [L1][ncand] every run in ascending order
    __shared__ unsigned char s_up[256], s_down[256];
    for (int jr = threadIdx.x; jr < L1; jr += CI_TAB_THREADS) { s_up[jr] = 1; s_down[jr] = 1; }
    __syncthreads();
    for (int t = threadIdx.x; t + L1 < nthr; t += CI_TAB_THREADS) {
        const float a = s_thr[t], b = s_thr[t + L1];
        if (!(a <= b)) s_up[t % L1] = 0;                // benign races: every writer writes 0
        if (!(a >= b)) s_down[t % L1] = 0;
    }
    __syncthreads();
    for (int r = threadIdx.x; r < nthr; r += CI_TAB_THREADS) {
        const int jj = r / ncand, k = r - jj * ncand;
        const float T = s_thr[k * L1 + jj];
        int place;
        if (s_up[jj]) place = k;
        else if (s_down[jj]) place = ncand - 1 - k;
        else {
            place = 0;
            for (int k2 = 0; k2 < ncand; ++k2) {
                const float o = s_thr[k2 * L1 + jj];
                place += (o < T) || (o == T && k2 < k);
            }
        }
        s_run[jj * ncand + place] = T;
    }
    __syncthreads();
    // merge the ordered runs pairwise, log2(L1) rounds: an element's place in the merged pair is its place in
    // its own run plus the elements of the partner run below it (ties: the left run first), by binary search
    float* src = s_run;
    float* dst = s_key;
    for (int len = ncand; len < nthr; len <<= 1) {
        for (int i = threadIdx.x; i < nthr; i += CI_TAB_THREADS) {
            const int a0 = i / (2 * len) * (2 * len), a1 = min(a0 + len, nthr), b1 = min(a0 + 2 * len, nthr);
            const float v = src[i];
            int lo, hi, at;
            if (i < a1) {                               // left run: partner elements < v
                lo = a1; hi = b1;
                while (lo < hi) { const int mid = (lo + hi) >> 1; if (src[mid] < v) lo = mid + 1; else hi = mid; }
                at = i + (lo - a1);
            } else {                                    // right run: partner elements <= v
                lo = a0; hi = a1;
                while (lo < hi) { const int mid = (lo + hi) >> 1; if (src[mid] <= v) lo = mid + 1; else hi = mid; }
                at = (i - a1) + lo;
            }
            dst[QP_CK(at, nthr)] = v;
        }
        __syncthreads();
        float* t2 = src; src = dst; dst = t2;
    }
    if (src != s_key) {
        for (int t = threadIdx.x; t < nthr; t += CI_TAB_THREADS) s_key[t] = src[t];
        __syncthreads();
    }
    for (int r = threadIdx.x; r < nthr; r += CI_TAB_THREADS) {         // pos(T) = sorted thresholds <= T, run by run
        const int jj = r / ncand, k = r - jj * ncand;
        const float T = s_thr[k * L1 + jj];
        int lo = 0, hi = nthr;
        while (lo < hi) { const int mid = (lo + hi) >> 1; if (s_key[mid] <= T) lo = mid + 1; else hi = mid; }
        pos[(size_t)c * nthr + r] = T < inf ? (unsigned short)lo : (unsigned short)0xFFFFu;
    }
    for (int t = threadIdx.x; t < nthr; t += CI_TAB_THREADS) bb[(size_t)c * nthr + t] = s_key[t];
    __shared__ int s_m;
    __shared__ unsigned s_first[CI_CELLS + 1];
    if (threadIdx.x == 0) {                            // finite entries come first
        int a = 0, b = nthr;
        while (a < b) {
            const int mid = (a + b) >> 1;
            if (s_key[mid] < inf) a = mid + 1; else b = mid;
        }
        m_out[c] = (unsigned)a;
        s_m = a;
    }
    __syncthreads();
    // cell table: first[g] = sorted thresholds that lie in cells below g.  An element of cell g has all of
    // them below it and all thresholds of higher cells above it, so its interval is first[g] .. first[g + 1].
    const int m = s_m;
    const float g0 = sg_lo, inv_cw = g_hi > g_lo ? (float)((double)CI_CELLS / ((double)g_hi - (double)g_lo)) : 0.f;
    for (int g = threadIdx.x; g <= CI_CELLS; g += CI_TAB_THREADS) {
        int a = 0, b = m;                              // first position whose threshold's cell is >= g
        while (a < b) {
            const int mid = (a + b) >> 1;
            if (ci_cell(s_key[mid], g0, inv_cw) < g) a = mid + 1; else b = mid;
        }
        s_first[g] = g == CI_CELLS ? (unsigned)m : (unsigned)a;
    }
    __syncthreads();
    for (int g = threadIdx.x; g < CI_CELLS; g += CI_TAB_THREADS)
        cells[(size_t)c * CI_CELLS + g] = s_first[g] | (s_first[g + 1] << 16);
}

// ---------------------------------------------------------------- the pass over x

// Block b owns channels [b * cpb, b * cpb + cpb) and every row.  Thread = (channel slot, row lane): a warp
// reads cpb neighbouring elements of a few rows.  Shared memory per slot: the sorted thresholds (1-based)
// and three counters per interval, nthr + 1 words each.  tot[c][i] = count << 48 | sum of offsets of
// interval i (i = number of the channel's thresholds <= x), sumd2[c] = sum of squared offsets.
template <typename T>
__global__ void __launch_bounds__(CI_MOM_THREADS, 1) ci_moments_kernel(const T* __restrict__ x, uint64_t rows, uint32_t C,
                                                                       int cpb, int nthr, const float* __restrict__ bb,
                                                                       const unsigned* __restrict__ cells,
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
    unsigned* s_cell = s_hi + (size_t)cpb * stride;                               // [cpb][CI_CELLS] interval range of a cell
    double* s_d2 = reinterpret_cast<double*>(raw + ((size_t)cpb * (stride * 16 + CI_CELLS * 4) + 7) / 8 * 8);   // [CI_MOM_THREADS]
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
    for (int i = threadIdx.x; i < cpb * CI_CELLS; i += CI_MOM_THREADS)
        s_cell[i] = (i / CI_CELLS) < nch ? cells[(size_t)c0 * CI_CELLS + i] : 0u;
    __syncthreads();

    const int slot = threadIdx.x % cpb, rl = threadIdx.x / cpb, nl = CI_MOM_THREADS / cpb;
    double d2 = 0.0;
    if (rl < nl && slot < nch) {
        const uint32_t c = c0 + slot;
        const float ref0 = setup[c].g_lo, g0 = setup[c].gw, inv_cw = setup[c].inv_gw;
        const unsigned* cell = s_cell + (size_t)slot * CI_CELLS;
        const double inv_u = 1.0 / setup[c].u;          // a power of two
        const float* sb = s_bb + (size_t)slot * stride;
        unsigned* cnt = s_cnt + (size_t)slot * stride;
        unsigned* sl = s_lo + (size_t)slot * stride;
        unsigned* sh = s_hi + (size_t)slot * stride;
        const T* px = x + c;
        auto one = [&](float e, double& p) {
            if (!qp_is_finite(e)) return;
            const unsigned range = cell[QP_CK(ci_cell(e, g0, inv_cw), CI_CELLS)];
            unsigned lo = range & 0xFFFFu, hi = range >> 16;
            while (lo < hi) {                           // largest i in [lo, hi] with sb[i] <= e (sb[i] <= e for i <= lo)
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
                                                                    const float* __restrict__ bb,
                                                                    const unsigned short* __restrict__ pos,
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
    __shared__ double c_n[CI_CURVE_THREADS], c_sx[CI_CURVE_THREADS], c_sxx[CI_CURVE_THREADS];
    __shared__ double s_sxx;
    const uint32_t c = blockIdx.x;
    const unsigned m = m_in[c];
    const qp_ds_setup s = setup[c];
    const double u = s.u, ref0 = (double)s.g_lo;

    // per interval: count and sum of (x - ref0), into PN / PSX (loads independent of one another), and every
    // thread's share of SXX
    const int count = (int)m + 1;
    {
        double d = 0.0;
        for (int i = threadIdx.x; i < count; i += CI_CURVE_THREADS) {
            const unsigned long long w = tot[(size_t)c * stride + i];
            const double n = (double)(w >> 48);
            const double s1 = u * (double)(w & CI_SUM_MASK);
            const double r = i ? fmax((double)bb[(size_t)c * nthr + QP_CK(i - 1, nthr)], ref0) - ref0 : 0.0;
            PN[QP_CK(i, nthr + 2)] = n;
            PSX[QP_CK(i, nthr + 2)] = n * r + s1;
            d += n * r * r + 2.0 * r * s1;
        }
        c_sxx[threadIdx.x] = d;
    }
    __syncthreads();
    // exclusive prefix sums in place: thread t takes the chunk [t * per, t * per + per)
    const int per = (count + CI_CURVE_THREADS - 1) / CI_CURVE_THREADS;
    const int i0 = min((int)threadIdx.x * per, count), i1 = min(i0 + per, count);
    {
        double a = 0.0, b = 0.0;
        for (int i = i0; i < i1; ++i) { a += PN[i]; b += PSX[i]; }
        c_n[threadIdx.x] = a; c_sx[threadIdx.x] = b;
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
        PN[count] = a; PSX[count] = b;                   // the totals: the end of the last code's range
    }
    __syncthreads();
    {
        double a = c_n[threadIdx.x], b = c_sx[threadIdx.x];
        for (int i = i0; i < i1; ++i) {
            const double n = PN[i], sx = PSX[i];
            PN[i] = a; PSX[i] = b;
            a += n; b += sx;
        }
    }
    __syncthreads();

    const int L1 = (1 << bits) - 1;
    for (int k = threadIdx.x; k < ncp; k += CI_CURVE_THREADS) {
        double total = 0.0;
        if (k < ncand && valid[(size_t)c * ncp + k]) {
            const float4 q = cand[(size_t)c * ncp + k];
            const unsigned short* pk = pos + (size_t)c * nthr + k;    // T(k, j + 1) at pk[j * ncand]
            total = s_sxx;
            unsigned prev = 0u;
            for (int j0 = 0; j0 <= L1; j0 += 8) {        // eight positions loaded ahead of their use
                unsigned p8[8];
#pragma unroll
                for (int h = 0; h < 8; ++h) p8[h] = j0 + h < L1 ? (unsigned)pk[(size_t)(j0 + h) * ncand] : 0xFFFFu;
#pragma unroll
                for (int h = 0; h < 8; ++h) {
                    const int j = j0 + h;
                    if (j > L1) break;
                    unsigned next = p8[h] == 0xFFFFu ? m + 1u : p8[h];   // the last code (and a code never reached) runs to the end
                    if (next < prev) next = prev;
                    const double n = PN[QP_CK(next, nthr + 2)] - PN[QP_CK(prev, nthr + 2)];
                    const double sx = PSX[next] - PSX[prev];
                    const float level = fmaf(__fsub_rn(__uint_as_float(0x4B000000u | (unsigned)j), CI_MAGIC), q.z, q.x);
                    const double a = (double)level - ref0;
                    total += n * a * a - 2.0 * a * sx;
                    prev = next;
                }
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
    return al(sizeof(float) * (size_t)C * nthr) + al(sizeof(unsigned) * (size_t)C) + al(sizeof(double) * (size_t)C) +
           al(sizeof(unsigned long long) * (size_t)C * (nthr + 1)) + al(sizeof(unsigned) * (size_t)C * 128) +
           al(sizeof(unsigned short) * (size_t)C * nthr);
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
    const int p2 = (nthr + 3) & ~3;                      // the three arrays of the tables kernel, a multiple of 16 bytes each
    size_t off = 0;
    float* bb = reinterpret_cast<float*>(scratch + off);             off += al(sizeof(float) * (size_t)C * nthr);
    unsigned* m = reinterpret_cast<unsigned*>(scratch + off);        off += al(sizeof(unsigned) * (size_t)C);
    double* sumd2 = reinterpret_cast<double*>(scratch + off);        off += al(sizeof(double) * (size_t)C);
    unsigned long long* tot = reinterpret_cast<unsigned long long*>(scratch + off);  off += al(sizeof(unsigned long long) * (size_t)C * (nthr + 1));
    unsigned* cells = reinterpret_cast<unsigned*>(scratch + off);    off += al(sizeof(unsigned) * (size_t)C * CI_CELLS);
    unsigned short* pos = reinterpret_cast<unsigned short*>(scratch + off);

    ci_tables_kernel<<<C, CI_TAB_THREADS, 3 * sizeof(float) * (size_t)p2, s>>>(d_stats, cand, valid, ncp, ncand, bits, nthr,
                                                                             p2, setup, bb, m, cells, pos);
    // channels per block: one block per SM where the tables of that many channels fit in shared memory
    const size_t per_channel = 16 * (size_t)(nthr + 1) + 4 * (size_t)CI_CELLS;
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
        ci_moments_kernel<float><<<blocks, CI_MOM_THREADS, smem, s>>>(static_cast<const float*>(d_x), rows, C, cpb, nthr, bb,
                                                                     cells, setup, tot, sumd2);
    } else {
        if (cudaFuncSetAttribute(ci_moments_kernel<unsigned short>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess)
            return qp_check_launch(ctx, "qp_dsaciq_search_channels (interval shared memory)");
        ci_moments_kernel<unsigned short><<<blocks, CI_MOM_THREADS, smem, s>>>(static_cast<const unsigned short*>(d_x), rows, C,
                                                                              cpb, nthr, bb, cells, setup, tot, sumd2);
    }
    const size_t csmem = sizeof(double) * 2 * (size_t)(nthr + 2);
    ci_curve_kernel<<<C, CI_CURVE_THREADS, csmem, s>>>(tot, bb, pos, m, setup, sumd2, cand, valid, ncp, ncand, bits, nthr, part);
    ctx->launches += 3;
    return qp_check_launch(ctx, "qp_dsaciq_search_channels (interval path)");
}
