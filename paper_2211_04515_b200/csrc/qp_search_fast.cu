// a4, second implementation: the directed search (paper Sec. 3, Eq. 1) scored through
// per-interval moments instead of per-candidate passes.
//
// For a fixed candidate the quantizer's code is a non-decreasing step function of x, so each
// candidate k cuts the real line at L-1 thresholds T(k,j) = smallest float whose code is >= j.
// Merge the thresholds of all candidates (and the edges of a uniform grid that is used to
// find intervals quickly): between two neighbouring boundaries EVERY candidate's code is
// constant.  One pass over x accumulates, per interval i with left end r_i,
//     N_i = count,  S1_i = sum (x - r_i),  S2_i = sum (x - r_i)^2,
// and the squared error of candidate k follows exactly from the moments:
//     sum_i  N_i a^2 - 2 a S1_i + S2_i,   a = dq_k(r_i) - r_i,
// dq_k the reconstruction level of r_i under candidate k.  Elements outside the union
// [g_lo, g_hi] of all clip ranges are clipped by every candidate and enter through three
// global moments on each side.  Cost: one pass of ~30 instructions per element instead of
// 909, for any number of candidates.
//
// The thresholds come from bisection over float bit patterns with the quantizer's own code
// function, so the partition is exact.  Offsets x - r_i are smaller than one grid cell and
// are accumulated in fixed point with unit u (a power of two below cell/2^16), as
// integers: sums are exact and order-independent (bit-reproducible); the only approximation
// is the rounding of each offset to u, which moves a candidate's MSE by less than 1e-6
// relative in the worst case (all roundings aligned) and by ~1e-11 in practice.
#include <type_traits>

#include "qp_internal.cuh"

namespace {

constexpr int G = QP_IV_CELLS;
constexpr int MAXB = QP_IV_MAXB;
constexpr unsigned long long S1_MASK = (1ull << 40) - 1ull;

// monotone map float -> uint32 (finite values; -0 sorts directly below +0)
__device__ __forceinline__ unsigned key_of(float x)
{
    const unsigned u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float float_of(unsigned k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// grid cell of x (x >= g_lo): fp32, each operation rounded on its own
__device__ __forceinline__ int cell_of(float x, float g_lo, float inv_gw)
{
    return min(__float2int_rz(__fmul_rn(__fsub_rn(x, g_lo), inv_gw)), G - 1);
}

// smallest float in (lo_x, hi_x] for which pred holds, given !pred(lo_x) and pred(hi_x), pred monotone
template <typename P>
__device__ __forceinline__ float first_true(float lo_x, float hi_x, P pred)
{
    unsigned lo = key_of(lo_x), hi = key_of(hi_x);
    while (hi - lo > 1u) {
        const unsigned mid = lo + ((hi - lo) >> 1);
        if (pred(float_of(mid))) hi = mid; else lo = mid;
    }
    return float_of(hi);
}

// ------------------------------------------------------------------ grid + boundaries

// one block: the grid that covers all valid candidates, and the fixed-point unit
__global__ void iv_grid_kernel(const float4* __restrict__ cand, const int* __restrict__ valid, int ncand,
                               qp_ds_setup* __restrict__ setup)
{
    if (threadIdx.x != 0) return;
    float lo = cand[0].x, hi = cand[0].y;
    for (int k = 1; k < ncand; ++k)
        if (valid[k]) { lo = fminf(lo, cand[k].x); hi = fmaxf(hi, cand[k].y); }
    const double width = (double)hi - (double)lo;
    float inv_gw = 0.f;
    double u = 1.0;
    if (width > 0.0) {
        inv_gw = (float)((double)G / width);
        int e;
        frexp(width / (double)G, &e);               // cell width in (2^(e-1), 2^e]
        u = ldexp(1.0, e - 17);                     // offsets inside a cell stay below 2^17 units
    }
    setup->g_lo = lo;
    setup->g_hi = hi;
    setup->inv_gw = inv_gw;
    setup->u = u;
    setup->inv_u = (float)(1.0 / u);
}

// thread t < nthr: threshold (k, j) of candidate k = t / (L-1), code j = 1 + t % (L-1);
// thread nthr + c - 1: left edge of grid cell c = 1..G-1.  Entries that do not exist are +inf.
__global__ void __launch_bounds__(256) iv_bounds_kernel(const float4* __restrict__ cand, const int* __restrict__ valid,
                                                        int ncand, int bits, const qp_ds_setup* __restrict__ setup,
                                                        float* __restrict__ bnd, float* __restrict__ edges)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int L1 = (1 << bits) - 1;
    const int nthr = ncand * L1;
    const float inf = __int_as_float(0x7F800000);
    const float g_lo = setup->g_lo, g_hi = setup->g_hi, inv_gw = setup->inv_gw;
    if (t < nthr) {
        const int k = t / L1, j = 1 + t % L1;
        float out = inf;
        if (valid[k] && g_hi > g_lo) {
            const float4 q = cand[k];
            const unsigned mask = (unsigned)L1;
            auto pred = [&](float x) { return (int)qp_code(x, q.x, q.y, q.w, mask) >= j; };
            if (!pred(g_lo) && pred(g_hi)) out = first_true(g_lo, g_hi, pred);
        }
        bnd[t] = out;
    } else if (t < nthr + G - 1) {
        const int c = t - nthr + 1;
        float out = inf;
        if (g_hi > g_lo) {
            auto pred = [&](float x) { return cell_of(x, g_lo, inv_gw) >= c; };
            if (!pred(g_lo) && pred(g_hi)) out = first_true(g_lo, g_hi, pred);
        }
        bnd[t] = out;
        edges[c] = out;
    } else if (t < MAXB) {
        bnd[t] = inf;
    }
    if (t == 0) { edges[0] = g_lo; edges[G] = inf; }
}

// one block of 1024 threads: bitonic sort of the MAXB boundaries, then the per-cell lookup
__global__ void __launch_bounds__(1024) iv_sort_kernel(const float* __restrict__ bnd, const float* __restrict__ edges,
                                                       const qp_ds_setup* __restrict__ setup, float* __restrict__ bb,
                                                       unsigned* __restrict__ first)
{
    __shared__ float s[MAXB];
    for (int i = threadIdx.x; i < MAXB; i += 1024) s[i] = bnd[i];
    __syncthreads();
    for (int size = 2; size <= MAXB; size <<= 1)
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int t = threadIdx.x; t < MAXB / 2; t += 1024) {
                const int i = ((t / stride) * stride * 2) + (t % stride);
                const int j = i + stride;
                const bool up = ((i & size) == 0);
                const float a = s[i], b = s[j];
                if ((a > b) == up) { s[i] = b; s[j] = a; }
            }
            __syncthreads();
        }
    const float inf = __int_as_float(0x7F800000);
    // bb[0] = g_lo, bb[i + 1] = i-th smallest boundary (+inf beyond the finite ones)
    for (int i = threadIdx.x; i < MAXB; i += 1024) bb[i + 1] = s[i];
    if (threadIdx.x == 0) bb[0] = setup->g_lo;
    // m = number of finite boundaries.  first[c] = number of boundaries <= left edge of cell c
    // (the edge itself included), so the intervals that meet cell c are first[c] .. first[c+1]-1;
    // a cell whose edge does not exist (+inf) gets m + 1, which ends its left neighbour at m.
    for (int c = threadIdx.x; c <= G + 1; c += 1024) {
        const float e = (c <= G) ? edges[c] : inf;
        int lo = 0, hi = MAXB;                       // count of s[i] <= e (for e = inf: the finite ones)
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            const bool le = (e == inf) ? (s[mid] < inf) : (s[mid] <= e);
            if (le) lo = mid + 1; else hi = mid;
        }
        if (c <= G) first[c] = (e == inf) ? (unsigned)lo + 1u : (unsigned)lo;
        else first[G + 1] = (unsigned)lo;
    }
}

// ------------------------------------------------------------------------ moments

struct IvShared {
    float* bb;                      // [MAXB + 1]
    unsigned short* first;          // [G + 1]
    unsigned long long* A;          // [MAXB + 1] count << 40 | sum of offsets
    unsigned long long* B;          // [MAXB + 1] sum of squared offsets
};

struct IvOuter {
    double s1_lo, s2_lo, s1_hi, s2_hi;
    unsigned n_lo, n_hi;
};

template <bool GUARD>
__device__ __forceinline__ void iv_one(float x, const IvShared& sh, float g_lo, float g_hi, float inv_gw, float inv_u,
                                       IvOuter& o)
{
    if (GUARD && !qp_is_finite(x)) return;
    if (x < g_lo) {
        const double d = (double)__fsub_rn(g_lo, x);
        ++o.n_lo; o.s1_lo += d; o.s2_lo += d * d;
    } else if (x > g_hi) {
        const double d = (double)__fsub_rn(x, g_hi);
        ++o.n_hi; o.s1_hi += d; o.s2_hi += d * d;
    } else {
        const int c = cell_of(x, g_lo, inv_gw);
        unsigned lo = sh.first[c], hi = sh.first[c + 1] - 1u;
        while (lo < hi) {                                   // largest i in [lo, hi] with bb[i] <= x
            const unsigned mid = (lo + hi + 1u) >> 1;
            if (sh.bb[mid] <= x) lo = mid; else hi = mid - 1u;
        }
        const unsigned d1 = __float2uint_rn(__fmul_rn(__fsub_rn(x, sh.bb[lo]), inv_u));
        atomicAdd(&sh.A[lo], (1ull << 40) + (unsigned long long)d1);
        atomicAdd(&sh.B[lo], (unsigned long long)d1 * (unsigned long long)d1);
    }
}

template <typename T>
__global__ void __launch_bounds__(QP_IV_THREADS) iv_moments_kernel(const T* __restrict__ x, uint64_t n,
                                                                   const qp_stats_t* __restrict__ st,
                                                                   const qp_ds_setup* __restrict__ setup,
                                                                   const float* __restrict__ g_bb,
                                                                   const unsigned* __restrict__ g_first,
                                                                   ulonglong2* __restrict__ part,
                                                                   double* __restrict__ outer)
{
    extern __shared__ __align__(16) unsigned char raw[];
    IvShared sh;
    sh.A = reinterpret_cast<unsigned long long*>(raw);
    sh.B = sh.A + (MAXB + 1);
    sh.bb = reinterpret_cast<float*>(sh.B + (MAXB + 1));
    sh.first = reinterpret_cast<unsigned short*>(sh.bb + (MAXB + 1));
    const unsigned m = g_first[G + 1];                       // finite boundaries; intervals 0..m
    for (unsigned i = threadIdx.x; i <= (unsigned)MAXB; i += QP_IV_THREADS) { sh.A[i] = 0ull; sh.B[i] = 0ull; }
    for (unsigned i = threadIdx.x; i <= (unsigned)MAXB; i += QP_IV_THREADS) sh.bb[i] = g_bb[i];
    for (unsigned c = threadIdx.x; c <= (unsigned)G; c += QP_IV_THREADS) sh.first[c] = (unsigned short)g_first[c];
    __syncthreads();
    const float g_lo = setup->g_lo, g_hi = setup->g_hi, inv_gw = setup->inv_gw, inv_u = setup->inv_u;
    const bool guard = st->nonfinite != 0;
    IvOuter o = {0.0, 0.0, 0.0, 0.0, 0u, 0u};

    constexpr int EPV = qp_span<T>::EPV;
    const qp_span<T> sp(x, n);
    const T* xv = x + sp.head;
    const uint64_t stride = (uint64_t)gridDim.x * QP_IV_THREADS;
    auto body = [&](auto guard_tag) {
        constexpr bool GD = decltype(guard_tag)::value;
        uint64_t v = (uint64_t)blockIdx.x * QP_IV_THREADS + threadIdx.x;
        for (; v + stride < sp.nvec; v += 2 * stride) {
            float a[EPV], b[EPV];
            qp_load_vec(xv + v * EPV, a);
            qp_load_vec(xv + (v + stride) * EPV, b);
#pragma unroll
            for (int i = 0; i < EPV; ++i) iv_one<GD>(a[i], sh, g_lo, g_hi, inv_gw, inv_u, o);
#pragma unroll
            for (int i = 0; i < EPV; ++i) iv_one<GD>(b[i], sh, g_lo, g_hi, inv_gw, inv_u, o);
        }
        for (; v < sp.nvec; v += stride) {
            float a[EPV];
            qp_load_vec(xv + v * EPV, a);
#pragma unroll
            for (int i = 0; i < EPV; ++i) iv_one<GD>(a[i], sh, g_lo, g_hi, inv_gw, inv_u, o);
        }
        if (blockIdx.x == 0) {
            for (uint64_t i = threadIdx.x; i < sp.head; i += QP_IV_THREADS)
                iv_one<GD>(qp_load_one(x + i), sh, g_lo, g_hi, inv_gw, inv_u, o);
            const uint64_t t0 = sp.head + sp.nvec * EPV;
            for (uint64_t i = threadIdx.x; i < sp.tail; i += QP_IV_THREADS)
                iv_one<GD>(qp_load_one(x + t0 + i), sh, g_lo, g_hi, inv_gw, inv_u, o);
        }
    };
    if (guard) body(std::true_type{}); else body(std::false_type{});
    __syncthreads();
    ulonglong2* mine = part + (size_t)blockIdx.x * (MAXB + 1);
    for (unsigned i = threadIdx.x; i <= m; i += QP_IV_THREADS) mine[i] = make_ulonglong2(sh.A[i], sh.B[i]);

    __shared__ double red[QP_IV_THREADS / 32];
    const double r0 = qp_block_sum(o.s1_lo, red), r1 = qp_block_sum(o.s2_lo, red);
    const double r2 = qp_block_sum(o.s1_hi, red), r3 = qp_block_sum(o.s2_hi, red);
    const double r4 = qp_block_sum((double)o.n_lo, red), r5 = qp_block_sum((double)o.n_hi, red);
    if (threadIdx.x == 0) {
        double* dst = outer + (size_t)blockIdx.x * 8;
        dst[0] = r0; dst[1] = r1; dst[2] = r2; dst[3] = r3; dst[4] = r4; dst[5] = r5;
    }
}

// totals over the blocks' partials, in block order
__global__ void __launch_bounds__(256) iv_reduce_kernel(const ulonglong2* __restrict__ part, int blocks,
                                                        const unsigned* __restrict__ g_first,
                                                        qp_iv_total* __restrict__ tot)
{
    const unsigned m = g_first[G + 1];
    const unsigned i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i > m) return;
    unsigned long long n = 0, s1 = 0, s2 = 0;
    for (int b = 0; b < blocks; ++b) {
        const ulonglong2 p = part[(size_t)b * (MAXB + 1) + i];
        n += p.x >> 40;
        s1 += p.x & S1_MASK;
        s2 += p.y;
    }
    qp_iv_total t;
    t.n = n; t.s1 = s1; t.s2 = s2;
    tot[i] = t;
}

// block k: squared error of candidate k from the interval moments, fixed summation order
__global__ void __launch_bounds__(QP_THREADS) iv_curve_kernel(const qp_iv_total* __restrict__ tot,
                                                              const float* __restrict__ bb,
                                                              const unsigned* __restrict__ g_first,
                                                              const double* __restrict__ outer, int blocks,
                                                              const float4* __restrict__ cand,
                                                              const int* __restrict__ valid, int bits,
                                                              const qp_ds_setup* __restrict__ setup,
                                                              double* __restrict__ curve)
{
    const int k = blockIdx.x;
    __shared__ double red[QP_THREADS / 32];
    if (!valid[k]) {
        if (threadIdx.x == 0) curve[k] = __longlong_as_double(0x7FF0000000000000ll);
        return;
    }
    const float4 q = cand[k];
    const unsigned mask = (1u << bits) - 1u;
    const unsigned m = g_first[G + 1];
    const double u = setup->u;
    auto level = [&](float r) {      // reconstruction level that candidate k assigns to r
        const unsigned c = qp_code(r, q.x, q.y, q.w, mask);
        return (double)fmaf(__fsub_rn(__uint_as_float(0x4B000000u | c), 8388608.0f), q.z, q.x);
    };
    double acc = 0.0;
    for (unsigned i = threadIdx.x; i <= m; i += QP_THREADS) {
        const qp_iv_total t = tot[i];
        if (t.n == 0) continue;
        const float r = bb[i];
        const double a = level(r) - (double)r;
        acc += (double)t.n * a * a - 2.0 * a * ((double)t.s1 * u) + (double)t.s2 * (u * u);
    }
    double total = qp_block_sum(acc, red);
    if (threadIdx.x == 0) {
        double s1_lo = 0, s2_lo = 0, s1_hi = 0, s2_hi = 0, n_lo = 0, n_hi = 0;
        for (int b = 0; b < blocks; ++b) {
            const double* o = outer + (size_t)b * 8;
            s1_lo += o[0]; s2_lo += o[1]; s1_hi += o[2]; s2_hi += o[3]; n_lo += o[4]; n_hi += o[5];
        }
        const double a_lo = level(setup->g_lo) - (double)setup->g_lo;      // >= 0: below every clip range
        const double a_hi = level(setup->g_hi) - (double)setup->g_hi;      // <= 0: above every clip range
        total += n_lo * a_lo * a_lo + 2.0 * a_lo * s1_lo + s2_lo;
        total += n_hi * a_hi * a_hi - 2.0 * a_hi * s1_hi + s2_hi;
        const unsigned long long nf = setup->n_finite;
        curve[k] = nf ? total / (double)nf : 0.0;
    }
}

template <typename T>
int32_t interval_typed(qp_ctx* ctx, const T* x, uint64_t n, const qp_stats_t* d_stats, int bits, int steps,
                       cudaStream_t s)
{
    const int ncand = steps + 1;
    const int L1 = (1 << bits) - 1;
    const int nbnd = ncand * L1 + G - 1;
    if (nbnd > MAXB) return qp_fail(ctx, QP_ERR_INVALID_ARG, "too many boundaries for the interval path");
    constexpr size_t smem = (size_t)(MAXB + 1) * (8 + 8 + 4) + (size_t)(G + 1) * 2 + 16;
    if (cudaFuncSetAttribute(iv_moments_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return qp_check_launch(ctx, "qp_dsaciq_search (interval shared memory)");
    iv_grid_kernel<<<1, 32, 0, s>>>(ctx->d_cand, ctx->d_valid, ncand, ctx->d_setup);
    iv_bounds_kernel<<<MAXB / 256, 256, 0, s>>>(ctx->d_cand, ctx->d_valid, ncand, bits, ctx->d_setup, ctx->d_iv_bnd,
                                                ctx->d_iv_edges);
    iv_sort_kernel<<<1, 1024, 0, s>>>(ctx->d_iv_bnd, ctx->d_iv_edges, ctx->d_setup, ctx->d_iv_bb, ctx->d_iv_first);
    const int blocks = ctx->iv_blocks;
    iv_moments_kernel<T><<<blocks, QP_IV_THREADS, smem, s>>>(x, n, d_stats, ctx->d_setup, ctx->d_iv_bb, ctx->d_iv_first,
                                                             ctx->d_iv_part, ctx->d_iv_outer);
    iv_reduce_kernel<<<(MAXB + 1 + 255) / 256, 256, 0, s>>>(ctx->d_iv_part, blocks, ctx->d_iv_first, ctx->d_iv_tot);
    iv_curve_kernel<<<ncand, QP_THREADS, 0, s>>>(ctx->d_iv_tot, ctx->d_iv_bb, ctx->d_iv_first, ctx->d_iv_outer, blocks,
                                                 ctx->d_cand, ctx->d_valid, bits, ctx->d_setup, ctx->d_curve);
    ctx->launches += 6;
    return qp_check_launch(ctx, "qp_dsaciq_search (interval path)");
}

}  // namespace

int32_t qp_launch_interval_search(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, const qp_stats_t* d_stats,
                                  int bits, int steps, cudaStream_t s)
{
    if (dtype == QP_F32) return interval_typed<float>(ctx, static_cast<const float*>(d_x), n, d_stats, bits, steps, s);
    return interval_typed<unsigned short>(ctx, static_cast<const unsigned short*>(d_x), n, d_stats, bits, steps, s);
}
