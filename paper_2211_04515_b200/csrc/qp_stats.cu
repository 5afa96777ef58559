// a1: per-tensor statistics (paper Sec. 3: min/max, mean, Laplace scale).
//
// Two streaming passes, both HBM-bound (the second one is served from L2 for tensors that
// fit there):
//   pass A  sum x, sum |x|, min, max, non-finite count            -> mean, mean_abs, min, max
//   pass B  sum |x - mean|, sum (x - mean)^2                      -> mad, var
// Each thread keeps fp32 partial sums over a run of 16 (f32) or 32 (bf16) elements and
// folds them into fp64; blocks write fp64 partials; the last block to finish (ticket
// counter, no waiting) merges all partials in index order, so results do not depend on
// block scheduling.
#include <type_traits>

#include "qp_gridbar.cuh"
#include "qp_internal.cuh"
#include "qp_stream.cuh"

QP_CK_UNIT

namespace {

constexpr int UNROLL = 4;   // 16-byte loads in flight per thread

struct AccA {
    double s, sa, mn, mx;
    unsigned long long bad;
    __device__ void add_scalar(float v)
    {
        if (qp_is_finite(v)) {
            s += (double)v;
            sa += (double)fabsf(v);
            mn = fmin(mn, (double)v);
            mx = fmax(mx, (double)v);
        } else {
            ++bad;
        }
    }
};

template <typename T>
__global__ void __launch_bounds__(QP_THREADS) stats_pass_a(const T* __restrict__ x, uint64_t n,
                                                           qp_stats_partial* __restrict__ part,
                                                           unsigned* __restrict__ ticket, qp_stats_t* __restrict__ out,
                                                           unsigned* __restrict__ status)
{
    constexpr int EPV = qp_span<T>::EPV;
    const qp_span<T> sp(x, n);
    const T* xv = x + sp.head;
    const float inf = __int_as_float(0x7F800000);

    AccA acc = {0.0, 0.0, (double)inf, (double)-inf, 0ull};
    const uint64_t stride = (uint64_t)gridDim.x * QP_THREADS;
    uint64_t v = (uint64_t)blockIdx.x * QP_THREADS + threadIdx.x;

    for (; v + (UNROLL - 1) * stride < sp.nvec; v += UNROLL * stride) {
        float e[UNROLL][EPV];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) qp_load_vec(xv + (v + u * stride) * EPV, e[u]);
        float s = 0.f, sa = 0.f, mn = inf, mx = -inf;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
#pragma unroll
            for (int i = 0; i < EPV; ++i) {
                s += e[u][i];
                sa += fabsf(e[u][i]);
                mn = fminf(mn, e[u][i]);
                mx = fmaxf(mx, e[u][i]);
            }
        if (sa < inf) {                       // every element finite (and no fp32 overflow)
            acc.s += (double)s;
            acc.sa += (double)sa;
            acc.mn = fmin(acc.mn, (double)mn);
            acc.mx = fmax(acc.mx, (double)mx);
        } else {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u)
#pragma unroll
                for (int i = 0; i < EPV; ++i) acc.add_scalar(e[u][i]);
        }
    }
    for (; v < sp.nvec; v += stride) {
        float e[EPV];
        qp_load_vec(xv + v * EPV, e);
#pragma unroll
        for (int i = 0; i < EPV; ++i) acc.add_scalar(e[i]);
    }
    if (blockIdx.x == 0) {                    // unaligned head and ragged tail
        for (uint64_t i = threadIdx.x; i < sp.head; i += QP_THREADS) acc.add_scalar(qp_load_one(x + i));
        const uint64_t t0 = sp.head + sp.nvec * EPV;
        for (uint64_t i = threadIdx.x; i < sp.tail; i += QP_THREADS) acc.add_scalar(qp_load_one(x + t0 + i));
    }

    __shared__ double sh[QP_THREADS / 32];
    __shared__ bool last;
    const double bs = qp_block_sum(acc.s, sh);
    const double bsa = qp_block_sum(acc.sa, sh);
    const double bmn = qp_block_min(acc.mn, sh);
    const double bmx = qp_block_max(acc.mx, sh);
    const double bbad = qp_block_sum((double)acc.bad, sh);   // exact: counts are far below 2^53
    if (threadIdx.x == 0) {
        qp_stats_partial p;
        p.s0 = bs; p.s1 = bsa; p.mn = bmn; p.mx = bmx; p.bad = (unsigned long long)bbad; p.pad = 0;
        part[blockIdx.x] = p;
        __threadfence();
        last = (atomicAdd(&ticket[0], 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!last) return;
    __threadfence();

    double s = 0.0, sa = 0.0, mn = (double)inf, mx = (double)-inf, bad = 0.0;
    for (unsigned b = threadIdx.x; b < gridDim.x; b += QP_THREADS) {
        s += __ldcg(&part[b].s0);
        sa += __ldcg(&part[b].s1);
        mn = fmin(mn, __ldcg(&part[b].mn));
        mx = fmax(mx, __ldcg(&part[b].mx));
        bad += (double)__ldcg(&part[b].bad);
    }
    s = qp_block_sum(s, sh);
    sa = qp_block_sum(sa, sh);
    mn = qp_block_min(mn, sh);
    mx = qp_block_max(mx, sh);
    bad = qp_block_sum(bad, sh);
    if (threadIdx.x == 0) {
        const unsigned long long nbad = (unsigned long long)bad;
        const unsigned long long nf = n - nbad;
        out->n = n;
        out->nonfinite = nbad;
        out->mean = nf ? s / (double)nf : 0.0;
        out->mean_abs = nf ? sa / (double)nf : 0.0;
        out->min = nf ? mn : 0.0;
        out->max = nf ? mx : 0.0;
        out->mad = 0.0;
        out->var = 0.0;
        out->hist_peak = 0;
        out->hist_bins = 0;
        out->reserved = 0;
        if (nbad) atomicOr(status, QP_DEV_NONFINITE);
        ticket[0] = 0;
    }
}

template <typename T, bool GUARD>
__device__ __forceinline__ void pass_b_body(const T* __restrict__ x, uint64_t n, float m_hi, float m_lo, double& sd,
                                            double& sv)
{
    constexpr int EPV = qp_span<T>::EPV;
    const qp_span<T> sp(x, n);
    const T* xv = x + sp.head;
    const uint64_t stride = (uint64_t)gridDim.x * QP_THREADS;
    uint64_t v = (uint64_t)blockIdx.x * QP_THREADS + threadIdx.x;

    auto one = [&](float e, float& d1, float& d2) {
        // x - mean with the mean held as an unevaluated fp32 pair
        const float d = __fsub_rn(__fsub_rn(e, m_hi), m_lo);
        if (!GUARD || qp_is_finite(e)) {
            d1 += fabsf(d);
            d2 = fmaf(d, d, d2);
        }
    };
    for (; v + (UNROLL - 1) * stride < sp.nvec; v += UNROLL * stride) {
        float e[UNROLL][EPV];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) qp_load_vec(xv + (v + u * stride) * EPV, e[u]);
        float d1 = 0.f, d2 = 0.f;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
#pragma unroll
            for (int i = 0; i < EPV; ++i) one(e[u][i], d1, d2);
        sd += (double)d1;
        sv += (double)d2;
    }
    for (; v < sp.nvec; v += stride) {
        float e[EPV];
        qp_load_vec(xv + v * EPV, e);
        float d1 = 0.f, d2 = 0.f;
#pragma unroll
        for (int i = 0; i < EPV; ++i) one(e[i], d1, d2);
        sd += (double)d1;
        sv += (double)d2;
    }
    if (blockIdx.x == 0) {
        float d1 = 0.f, d2 = 0.f;
        for (uint64_t i = threadIdx.x; i < sp.head; i += QP_THREADS) one(qp_load_one(x + i), d1, d2);
        const uint64_t t0 = sp.head + sp.nvec * EPV;
        for (uint64_t i = threadIdx.x; i < sp.tail; i += QP_THREADS) one(qp_load_one(x + t0 + i), d1, d2);
        sd += (double)d1;
        sv += (double)d2;
    }
}

template <typename T>
__global__ void __launch_bounds__(QP_THREADS) stats_pass_b(const T* __restrict__ x, uint64_t n,
                                                           qp_stats_partial* __restrict__ part,
                                                           unsigned* __restrict__ ticket, qp_stats_t* __restrict__ out)
{
    const double mean = out->mean;
    const unsigned long long nbad = out->nonfinite;
    const float m_hi = (float)mean;
    const float m_lo = (float)(mean - (double)m_hi);
    double sd = 0.0, sv = 0.0;
    if (nbad == 0) pass_b_body<T, false>(x, n, m_hi, m_lo, sd, sv);
    else           pass_b_body<T, true>(x, n, m_hi, m_lo, sd, sv);

    __shared__ double sh[QP_THREADS / 32];
    __shared__ bool last;
    const double bsd = qp_block_sum(sd, sh);
    const double bsv = qp_block_sum(sv, sh);
    if (threadIdx.x == 0) {
        part[blockIdx.x].s0 = bsd;
        part[blockIdx.x].s1 = bsv;
        __threadfence();
        last = (atomicAdd(&ticket[1], 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    double a = 0.0, b = 0.0;
    for (unsigned k = threadIdx.x; k < gridDim.x; k += QP_THREADS) {
        a += __ldcg(&part[k].s0);
        b += __ldcg(&part[k].s1);
    }
    a = qp_block_sum(a, sh);
    b = qp_block_sum(b, sh);
    if (threadIdx.x == 0) {
        const unsigned long long nf = n - nbad;
        out->mad = nf ? a / (double)nf : 0.0;
        out->var = nf ? b / (double)nf : 0.0;
        ticket[1] = 0;
    }
}

// ---------------------------------------------------------------------------------------
// Streamed versions for 16-byte aligned tensors: tiles of 16 KB arrive in shared memory
// through the bulk-copy ring (qp_stream.cuh), 4 stages per block, so about 190 KB per SM are
// in flight whatever the consumers are doing.  Same arithmetic and merge as above.  Pass B
// walks the tiles in the opposite direction to pass A, so it starts on the part of the
// tensor that pass A left in L2.

constexpr int ST_TILE = 16384;
constexpr int ST_STAGES = 4;
constexpr int ST_BLOCKS_PER_SM = 2;
constexpr int ST_FUSED_HIST_MAX = 4096;     // largest histogram that pass B carries along

template <typename T>
__device__ __forceinline__ void lds_vec(const unsigned char* p, float (&v)[qp_span<T>::EPV])
{
    if constexpr (sizeof(T) == 4) {
        const float4 a = *reinterpret_cast<const float4*>(p);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    } else {
        const uint4 a = *reinterpret_cast<const uint4*>(p);
        v[0] = __uint_as_float(a.x << 16); v[1] = __uint_as_float(a.x & 0xFFFF0000u);
        v[2] = __uint_as_float(a.y << 16); v[3] = __uint_as_float(a.y & 0xFFFF0000u);
        v[4] = __uint_as_float(a.z << 16); v[5] = __uint_as_float(a.z & 0xFFFF0000u);
        v[6] = __uint_as_float(a.w << 16); v[7] = __uint_as_float(a.w & 0xFFFF0000u);
    }
}

template <typename T>
__global__ void __launch_bounds__(QP_THREADS) stats_stream_a(const T* __restrict__ x, uint64_t n, uint64_t ntiles,
                                                             qp_stats_partial* __restrict__ part,
                                                             unsigned* __restrict__ ticket, qp_stats_t* __restrict__ out,
                                                             unsigned* __restrict__ status, long long wait_limit)
{
    extern __shared__ __align__(128) unsigned char ring[];
    constexpr int EPV = qp_span<T>::EPV;
    constexpr int VPT = ST_TILE / 16 / QP_THREADS;           // 16-byte vectors per thread and tile (4)
    const float inf = __int_as_float(0x7F800000);
    AccA acc = {0.0, 0.0, (double)inf, (double)-inf, 0ull};
    float tmn = inf, tmx = -inf;                             // exact in fp32: kept out of the fp64 path

    qp_stream::for_each_tile<ST_TILE, ST_STAGES>(
        reinterpret_cast<const unsigned char*>(x), ntiles, false, ring, status, wait_limit,
        [&](const unsigned char* tile, uint64_t) {
            float e[VPT][EPV];
#pragma unroll
            for (int u = 0; u < VPT; ++u) lds_vec<T>(tile + (size_t)(u * QP_THREADS + threadIdx.x) * 16, e[u]);
            float s = 0.f, sa = 0.f, mn = inf, mx = -inf;
#pragma unroll
            for (int u = 0; u < VPT; ++u)
#pragma unroll
                for (int i = 0; i < EPV; ++i) {
                    s += e[u][i];
                    sa += fabsf(e[u][i]);
                    mn = fminf(mn, e[u][i]);
                    mx = fmaxf(mx, e[u][i]);
                }
            if (sa < inf) {
                acc.s += (double)s;
                acc.sa += (double)sa;
                tmn = fminf(tmn, mn);
                tmx = fmaxf(tmx, mx);
            } else {
#pragma unroll
                for (int u = 0; u < VPT; ++u)
#pragma unroll
                    for (int i = 0; i < EPV; ++i) acc.add_scalar(e[u][i]);
            }
        });
    acc.mn = fmin(acc.mn, (double)tmn);
    acc.mx = fmax(acc.mx, (double)tmx);
    if (blockIdx.x == 0) {                                   // elements after the last whole tile
        const uint64_t t0 = ntiles * (ST_TILE / sizeof(T));
        for (uint64_t i = t0 + threadIdx.x; i < n; i += QP_THREADS) acc.add_scalar(qp_load_one(x + i));
    }

    __shared__ double sh[QP_THREADS / 32];
    __shared__ bool last;
    const double bs = qp_block_sum(acc.s, sh);
    const double bsa = qp_block_sum(acc.sa, sh);
    const double bmn = qp_block_min(acc.mn, sh);
    const double bmx = qp_block_max(acc.mx, sh);
    const double bbad = qp_block_sum((double)acc.bad, sh);
    if (threadIdx.x == 0) {
        qp_stats_partial p;
        p.s0 = bs; p.s1 = bsa; p.mn = bmn; p.mx = bmx; p.bad = (unsigned long long)bbad; p.pad = 0;
        part[blockIdx.x] = p;
        __threadfence();
        last = (atomicAdd(&ticket[0], 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    double s = 0.0, sa = 0.0, mn = (double)inf, mx = (double)-inf, bad = 0.0;
    for (unsigned b = threadIdx.x; b < gridDim.x; b += QP_THREADS) {
        s += __ldcg(&part[b].s0);
        sa += __ldcg(&part[b].s1);
        mn = fmin(mn, __ldcg(&part[b].mn));
        mx = fmax(mx, __ldcg(&part[b].mx));
        bad += (double)__ldcg(&part[b].bad);
    }
    s = qp_block_sum(s, sh);
    sa = qp_block_sum(sa, sh);
    mn = qp_block_min(mn, sh);
    mx = qp_block_max(mx, sh);
    bad = qp_block_sum(bad, sh);
    if (threadIdx.x == 0) {
        const unsigned long long nbad = (unsigned long long)bad;
        const unsigned long long nf = n - nbad;
        out->n = n;
        out->nonfinite = nbad;
        out->mean = nf ? s / (double)nf : 0.0;
        out->mean_abs = nf ? sa / (double)nf : 0.0;
        out->min = nf ? mn : 0.0;
        out->max = nf ? mx : 0.0;
        out->mad = 0.0;
        out->var = 0.0;
        out->hist_peak = 0;
        out->hist_bins = 0;
        out->reserved = 0;
        if (nbad) atomicOr(status, QP_DEV_NONFINITE);
        ticket[0] = 0;
    }
}

// Pass B, optionally with the histogram of the directed search fused in (HIST): nb equal bins
// over [min, max], bin = floor((x - min) * inv_w) in fp32 with the last bin closed, counted in
// shared memory with one replica of every bin per lane group (no same-address contention),
// merged into 64-bit global counters; the last block extracts the peak count.
template <typename T, bool HIST>
__global__ void __launch_bounds__(QP_THREADS) stats_stream_b(const T* __restrict__ x, uint64_t n, uint64_t ntiles,
                                                             qp_stats_partial* __restrict__ part,
                                                             unsigned* __restrict__ ticket, qp_stats_t* __restrict__ out,
                                                             unsigned* __restrict__ status, int nb, int rep_shift,
                                                             unsigned long long* __restrict__ hist, long long wait_limit)
{
    extern __shared__ __align__(128) unsigned char ring[];
    constexpr int EPV = qp_span<T>::EPV;
    constexpr int VPT = ST_TILE / 16 / QP_THREADS;
    unsigned* sh_hist = reinterpret_cast<unsigned*>(ring + qp_stream::ring_bytes<ST_TILE, ST_STAGES>());
    const double mean = out->mean;
    const bool guard = out->nonfinite != 0;
    const float m_hi = (float)mean;
    const float m_lo = (float)(mean - (double)m_hi);
    const double dmn = out->min, dmx = out->max;
    const bool hist_on = HIST && dmx > dmn;
    const float mn = (float)dmn;
    const float inv_w = hist_on ? (float)((double)nb / (dmx - dmn)) : 0.f;
    // every lane counts in its own replica of the bins: my_hist[bin << rep_shift]
    unsigned* my_hist = sh_hist + (threadIdx.x & ((1 << rep_shift) - 1));
    const int top_bin = nb - 1;
    if (HIST) {
        for (int i = threadIdx.x; i < (nb << rep_shift); i += QP_THREADS) sh_hist[i] = 0u;
        __syncthreads();
    }
    double sd = 0.0, sv = 0.0;
    auto run = [&](auto guard_tag) {
        constexpr bool GD = decltype(guard_tag)::value;
        auto one = [&](float e, float& d1, float& d2) {
            const float d = __fsub_rn(__fsub_rn(e, m_hi), m_lo);
            if (!GD || qp_is_finite(e)) {
                d1 += fabsf(d);
                d2 = fmaf(d, d, d2);
                if (HIST) {      // x >= min, so the position is never negative; an empty range gives bin 0
                    const int b = min(__float2int_rz(__fmul_rn(__fsub_rn(e, mn), inv_w)), top_bin);
                    atomicAdd(&my_hist[QP_CK(b << rep_shift, nb << rep_shift)], 1u);
                }
            }
        };
        qp_stream::for_each_tile<ST_TILE, ST_STAGES>(
            reinterpret_cast<const unsigned char*>(x), ntiles, true, ring, status, wait_limit,
            [&](const unsigned char* tile, uint64_t) {
                float e[VPT][EPV];
#pragma unroll
                for (int u = 0; u < VPT; ++u) lds_vec<T>(tile + (size_t)(u * QP_THREADS + threadIdx.x) * 16, e[u]);
                float d1 = 0.f, d2 = 0.f;
#pragma unroll
                for (int u = 0; u < VPT; ++u)
#pragma unroll
                    for (int i = 0; i < EPV; ++i) one(e[u][i], d1, d2);
                sd += (double)d1;
                sv += (double)d2;
            });
        if (blockIdx.x == 0) {
            float d1 = 0.f, d2 = 0.f;
            const uint64_t t0 = ntiles * (ST_TILE / sizeof(T));
            for (uint64_t i = t0 + threadIdx.x; i < n; i += QP_THREADS) one(qp_load_one(x + i), d1, d2);
            sd += (double)d1;
            sv += (double)d2;
        }
    };
    if (guard) run(std::true_type{}); else run(std::false_type{});
    if (HIST) {
        __syncthreads();
        const int reps = 1 << rep_shift;
        for (int b = threadIdx.x; b < nb; b += QP_THREADS) {
            unsigned long long c = 0;
            for (int r = 0; r < reps; ++r) c += sh_hist[(b << rep_shift) + ((r + threadIdx.x) & (reps - 1))];
            if (c) atomicAdd(&hist[b], c);
        }
        __threadfence();                          // counts are out before this block takes its ticket
    }
    __shared__ double sh[QP_THREADS / 32];
    __shared__ bool last;
    const double bsd = qp_block_sum(sd, sh);
    const double bsv = qp_block_sum(sv, sh);
    if (threadIdx.x == 0) {
        part[blockIdx.x].s0 = bsd;
        part[blockIdx.x].s1 = bsv;
        __threadfence();
        last = (atomicAdd(&ticket[1], 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    double a = 0.0, b = 0.0;
    for (unsigned k = threadIdx.x; k < gridDim.x; k += QP_THREADS) {
        a += __ldcg(&part[k].s0);
        b += __ldcg(&part[k].s1);
    }
    a = qp_block_sum(a, sh);
    b = qp_block_sum(b, sh);
    double top = 0.0;
    if (HIST) {
        for (int k = threadIdx.x; k < nb; k += QP_THREADS) top = fmax(top, (double)__ldcg(&hist[k]));   // counts < 2^53
        top = qp_block_max(top, sh);
    }
    if (threadIdx.x == 0) {
        const unsigned long long nf = n - out->nonfinite;
        out->mad = nf ? a / (double)nf : 0.0;
        out->var = nf ? b / (double)nf : 0.0;
        if (HIST) {
            out->hist_peak = hist_on ? (unsigned long long)top : 0ull;     // empty range: no histogram
            out->hist_bins = nb;
        }
        ticket[1] = 0;
    }
}

template <typename T>
int32_t launch_streamed(qp_ctx* ctx, const T* x, uint64_t n, uint64_t ntiles, int hist_bins, qp_stats_t* d_out,
                        cudaStream_t s)
{
    constexpr size_t ring = qp_stream::ring_bytes<ST_TILE, ST_STAGES>();
    // fused histogram: as many lane replicas of each bin as fit in 16 KB of shared memory
    const bool fuse = hist_bins >= 1 && hist_bins <= ST_FUSED_HIST_MAX;
    int rep_shift = 5;
    while (fuse && rep_shift > 0 && ((size_t)hist_bins << rep_shift) * sizeof(unsigned) > 16 * 1024) --rep_shift;
    const size_t smem_b = ring + (fuse ? ((size_t)hist_bins << rep_shift) * sizeof(unsigned) : 0);
    // per device, cheap: done on every call so that every device the process uses is covered
    if (cudaFuncSetAttribute(stats_stream_a<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring) != cudaSuccess ||
        cudaFuncSetAttribute(stats_stream_b<T, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring) != cudaSuccess ||
        cudaFuncSetAttribute(stats_stream_b<T, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(ring + 16 * 1024)) != cudaSuccess)
        return qp_check_launch(ctx, "qp_stats (shared memory attribute)");
    if (fuse && cudaMemsetAsync(ctx->d_hist, 0, sizeof(unsigned long long) * hist_bins, s) != cudaSuccess)
        return qp_check_launch(ctx, "qp_stats (histogram reset)");
    const uint64_t cap = (uint64_t)ctx->sm_count * ST_BLOCKS_PER_SM;
    const int blocks = (int)(ntiles > cap ? cap : ntiles);
    stats_stream_a<T><<<blocks, QP_THREADS, ring, s>>>(x, n, ntiles, ctx->d_part, ctx->d_ticket, d_out, ctx->d_status,
                                                       ctx->wait_cycles);
    if (fuse)
        stats_stream_b<T, true><<<blocks, QP_THREADS, smem_b, s>>>(x, n, ntiles, ctx->d_part, ctx->d_ticket, d_out,
                                                                   ctx->d_status, hist_bins, rep_shift, ctx->d_hist,
                                                                   ctx->wait_cycles);
    else
        stats_stream_b<T, false><<<blocks, QP_THREADS, ring, s>>>(x, n, ntiles, ctx->d_part, ctx->d_ticket, d_out,
                                                                  ctx->d_status, 0, 0, ctx->d_hist, ctx->wait_cycles);
    ctx->launches += 2;
    return qp_check_launch(ctx, "qp_stats");
}

// ---------------------------------------------------------------------------------------
// Both passes in ONE cooperative launch (one block per SM).  What the two streamed kernels
// spend twice - a launch, the start of the copy ring, a last-block merge - is spent once, and
// the second pass reads less: every warp keeps the last tile of its first pass in shared memory,
// and the second pass, which walks the warp's tiles in the opposite order, starts on that
// resident tile and fetches only the rest (all SMs together hold ~19 MB; with what L2 still holds
// of the tensor's end, a 129 MB tensor costs ~173 MB of DRAM reads instead of 258, and one that
// fits in L2 is read once).
//
// Every warp has a ring of its own (qp_stream::warp_ring): the tile loops hold no block barrier,
// a warp refills its stage as soon as its lanes have the tile in registers, and a lane works on
// 64 elements per tile in four independent chains per sum.  Measured on a 129 MB tensor: fewer
// and larger tiles beat more stages (16 warps x 1 stage of 8 KB: 43.6 us; 3 stages of 4 KB: 45.3;
// 6 stages of 2 KB: 51.7; 32 warps x 3 x 2 KB: 57.0), because the work per tile outside the sums
// (wait, address, refill, the fp64 adds) is what the issue slots go to; the block-wide ring of 6 x 32 KB
// with two block barriers per tile that came before took 53 us.
//
//   pass A    warp w of block b takes 8 KB tiles 16 b + w, + 16 G, ...: sum x, sum |x|, min, max, non-finite
//   barrier   grid-wide (bounded); every block merges the G partials in index order: same mean everywhere
//   pass B    the same tiles backwards: sum |x - mean|, sum (x - mean)^2, histogram over [min, max]
//   exit      every block counts itself out; the last one merges pass B's partials, takes the
//             histogram's peak, writes the statistics and leaves the barrier scratch at zero
//
// A warp whose wait runs out flags its block; the block then (after its loops) raises the abort
// flag beside the barrier counter and QP_DEV_STREAM_TIMEOUT in the status word, every warp waits
// for its own copies in flight, and the block still arrives at the barrier and counts itself out,
// so nobody waits for it and the scratch is clean afterwards; no statistics are written then.
constexpr int SF_THREADS = 512;
constexpr int SF_WARPS = SF_THREADS / 32;
constexpr int SF_TILE = 8192;                     // bytes of one warp's tile
constexpr int SF_STAGES = 1;
constexpr int SF_VPT = SF_TILE / 16 / 32;         // 16-byte vectors per lane and tile (16)

struct SfArgs {
    const void* x;
    uint64_t n, ntiles;                           // ntiles: whole SF_TILE-byte tiles
    qp_stats_partial* part;                       // [2 * grid]: pass A, then pass B
    qp_stats_t* out;
    unsigned* status;
    int nb, rep_shift;                            // histogram bins (0: none) and log2 of the lane replicas per bin
    unsigned long long* hist;                     // [nb] global counters (zeroed by block 0 before the barrier)
    unsigned* bar;                                // [0] arrivals, [1] blocks that have left, [2] abort flag; zero at entry
    long long wait_limit;
    unsigned spin_limit, bar_extra;
};

// element k of a 16-byte vector held as four words
template <typename T>
__device__ __forceinline__ float sf_elem(const uint4& v, int k)
{
    if constexpr (sizeof(T) == 4) {
        return __uint_as_float(k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w);
    } else {
        const unsigned w = (k >> 1) == 0 ? v.x : (k >> 1) == 1 ? v.y : (k >> 1) == 2 ? v.z : v.w;
        return __uint_as_float((k & 1) ? (w & 0xFFFF0000u) : (w << 16));
    }
}

template <typename T, bool HIST>
__global__ void __launch_bounds__(SF_THREADS, 1) stats_fused_kernel(const SfArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int EPV = qp_span<T>::EPV;
    using Ring = qp_stream::warp_ring<SF_TILE, SF_STAGES>;
    __shared__ double sh[SF_THREADS / 32];
    __shared__ int s_flag, s_ok;
    __shared__ bool s_last;
    __shared__ double s_mean, s_mean_abs, s_mn, s_mx;
    __shared__ unsigned long long s_bad;
    unsigned* sh_hist = reinterpret_cast<unsigned*>(smem + Ring::bytes(SF_WARPS));
    const T* x = static_cast<const T*>(a.x);
    const unsigned char* base = static_cast<const unsigned char*>(a.x);
    const int lane = threadIdx.x & 31;
    const uint64_t G = gridDim.x;
    const uint64_t GW = G * SF_WARPS, first = (uint64_t)blockIdx.x * SF_WARPS + (threadIdx.x >> 5);
    const uint64_t m = first < a.ntiles ? (a.ntiles - first + GW - 1) / GW : 0;   // tiles of this warp
    const float inf = __int_as_float(0x7F800000);
    auto tile_src = [&](uint64_t i) { return base + (first + i * GW) * (uint64_t)SF_TILE; };
    Ring ring;
    if (threadIdx.x == 0) s_flag = 0;
    ring.init(smem, SF_WARPS);
    bool ok = true;

    // ---- pass A
    for (uint64_t i = 0; i < (uint64_t)SF_STAGES && i < m; ++i) ring.issue((int)i, tile_src(i));
    AccA acc = {0.0, 0.0, (double)inf, (double)-inf, 0ull};
    float tmn = inf, tmx = -inf;                             // exact in fp32: kept out of the fp64 path
    {
        int s = 0;
        for (uint64_t i = 0; i < m; ++i) {
            if (!ring.wait(s, a.wait_limit)) { s_flag = 1; break; }      // benign race: every writer writes 1
            const unsigned char* tile = ring.stage(s);
            uint4 v[SF_VPT];
#pragma unroll
            for (int u = 0; u < SF_VPT; ++u) v[u] = *reinterpret_cast<const uint4*>(tile + (size_t)(u * 32 + lane) * 16);
            __syncwarp();
            if (i + SF_STAGES < m) ring.issue(s, tile_src(i + SF_STAGES));   // the last ones stay resident
            float cs[4] = {0.f, 0.f, 0.f, 0.f}, ca[4] = {0.f, 0.f, 0.f, 0.f};
            float cmn[4] = {inf, inf, inf, inf}, cmx[4] = {-inf, -inf, -inf, -inf};
#pragma unroll
            for (int u = 0; u < SF_VPT; ++u)
#pragma unroll
                for (int k = 0; k < EPV; ++k) {
                    const float e = sf_elem<T>(v[u], k);
                    cs[k & 3] += e;
                    ca[k & 3] += fabsf(e);
                    cmn[k & 3] = fminf(cmn[k & 3], e);
                    cmx[k & 3] = fmaxf(cmx[k & 3], e);
                }
            const float psa = (ca[0] + ca[1]) + (ca[2] + ca[3]);
            if (psa < inf) {                                 // every element finite (and no fp32 overflow)
                acc.s += (double)((cs[0] + cs[1]) + (cs[2] + cs[3]));
                acc.sa += (double)psa;
                tmn = fminf(tmn, fminf(fminf(cmn[0], cmn[1]), fminf(cmn[2], cmn[3])));
                tmx = fmaxf(tmx, fmaxf(fmaxf(cmx[0], cmx[1]), fmaxf(cmx[2], cmx[3])));
            } else {
#pragma unroll
                for (int u = 0; u < SF_VPT; ++u)
#pragma unroll
                    for (int k = 0; k < EPV; ++k) acc.add_scalar(sf_elem<T>(v[u], k));
            }
            s = s + 1 == SF_STAGES ? 0 : s + 1;
        }
    }
    __syncthreads();
    ok = s_flag == 0;
    if (ok) {
        acc.mn = fmin(acc.mn, (double)tmn);
        acc.mx = fmax(acc.mx, (double)tmx);
        if (blockIdx.x == 0) {                               // elements after the last whole tile
            const uint64_t t0 = a.ntiles * (SF_TILE / sizeof(T));
            for (uint64_t i = t0 + threadIdx.x; i < a.n; i += SF_THREADS) acc.add_scalar(qp_load_one(x + i));
            if (HIST)
                for (int b = threadIdx.x; b < a.nb; b += SF_THREADS) a.hist[b] = 0ull;
        }
        const double bs = qp_block_sum(acc.s, sh);
        const double bsa = qp_block_sum(acc.sa, sh);
        const double bmn = qp_block_min(acc.mn, sh);
        const double bmx = qp_block_max(acc.mx, sh);
        const double bbad = qp_block_sum((double)acc.bad, sh);   // exact: counts are far below 2^53
        if (threadIdx.x == 0) {
            qp_stats_partial p;
            p.s0 = bs; p.s1 = bsa; p.mn = bmn; p.mx = bmx; p.bad = (unsigned long long)bbad; p.pad = 0;
            a.part[blockIdx.x] = p;
        }
    }
    // a failed block drains its copies, flags the launch, and still arrives so that nobody waits for it
    auto give_up = [&]() {
        if (threadIdx.x == 0) {
            atomicOr(a.status, QP_DEV_STREAM_TIMEOUT);
            atomicExch(a.bar + 2, 1u);
        }
        ring.drain();
        __syncthreads();
    };
    if (!ok) give_up();
    const bool met = qp_grid::barrier(a.bar, (unsigned)G + a.bar_extra, a.spin_limit, a.status, &s_ok);
    if (!met && threadIdx.x == 0) atomicExch(a.bar + 2, 1u);
    ok = ok && met && qp_grid::ld_acquire(a.bar + 2) == 0u;  // (the flag is read by all threads after the barrier's block barrier)

    // ---- every block: tensor-wide first moments, merged in index order (the same bits everywhere)
    if (ok) {
        double s = 0.0, sa = 0.0, mn = (double)inf, mx = (double)-inf, bad = 0.0;
        for (unsigned b = threadIdx.x; b < (unsigned)G; b += SF_THREADS) {
            s += __ldcg(&a.part[b].s0);
            sa += __ldcg(&a.part[b].s1);
            mn = fmin(mn, __ldcg(&a.part[b].mn));
            mx = fmax(mx, __ldcg(&a.part[b].mx));
            bad += (double)__ldcg(&a.part[b].bad);
        }
        s = qp_block_sum(s, sh);
        sa = qp_block_sum(sa, sh);
        mn = qp_block_min(mn, sh);
        mx = qp_block_max(mx, sh);
        bad = qp_block_sum(bad, sh);
        if (threadIdx.x == 0) {
            const unsigned long long nbad = (unsigned long long)bad;
            const unsigned long long nf = a.n - nbad;
            s_bad = nbad;
            s_mean = nf ? s / (double)nf : 0.0;
            s_mean_abs = nf ? sa / (double)nf : 0.0;
            s_mn = nf ? mn : 0.0;
            s_mx = nf ? mx : 0.0;
        }
        __syncthreads();
    }

    // ---- pass B: the warp's tiles backwards; tile i lives in stage i % SF_STAGES in both passes, so the
    // last SF_STAGES tiles of pass A are there already and each stage is refilled as it is consumed
    double sd = 0.0, sv = 0.0;
    if (ok) {
        const double mean = s_mean;
        const bool guard = s_bad != 0;
        const float m_hi = (float)mean;
        const float m_lo = (float)(mean - (double)m_hi);
        const double dmn = s_mn, dmx = s_mx;
        const bool hist_on = HIST && dmx > dmn;
        const float fmn = (float)dmn;
        const float inv_w = hist_on ? (float)((double)a.nb / (dmx - dmn)) : 0.f;
        unsigned* my_hist = sh_hist + (threadIdx.x & ((1 << a.rep_shift) - 1));   // this lane's replica of the bins
        const float top_bin = (float)(a.nb - 1);
        const int rep_shift = a.rep_shift;
        if (HIST) {
            for (int i = threadIdx.x; i < (a.nb << rep_shift); i += SF_THREADS) sh_hist[i] = 0u;
            __syncthreads();
        }
        auto run = [&](auto guard_tag) {
            constexpr bool GD = decltype(guard_tag)::value;
            auto one = [&](float e, float& d1, float& d2) {
                const float d = __fsub_rn(__fsub_rn(e, m_hi), m_lo);       // the mean as an unevaluated fp32 pair
                if (!GD || qp_is_finite(e)) {
                    d1 += fabsf(d);
                    d2 = fmaf(d, d, d2);
                    if (HIST) {
                        // bin = floor((x - min) * inv_w), the last bin closed; x >= min, so the position is
                        // never negative (an empty range gives bin 0).  The floor is taken by adding 2^23
                        // rounding down, which leaves it in the low mantissa bits: no conversion instruction
                        // (conversions issue at a quarter of the rate of an addition).
                        const float pos = fminf(__fmul_rn(__fsub_rn(e, fmn), inv_w), top_bin);
                        const unsigned b = __float_as_uint(__fadd_rd(pos, 8388608.0f)) & 0x7FFFFFu;
                        atomicAdd(&my_hist[QP_CK(b << rep_shift, (unsigned)a.nb << rep_shift)], 1u);
                    }
                }
            };
            int s = m ? (int)((m - 1) % SF_STAGES) : 0;
            for (uint64_t j = 0; j < m; ++j) {
                const uint64_t i = m - 1 - j;
                if (j >= (uint64_t)SF_STAGES && !ring.wait(s, a.wait_limit)) { s_flag = 1; break; }   // fetched in this pass
                const unsigned char* tile = ring.stage(s);
                uint4 v[SF_VPT];
#pragma unroll
                for (int u = 0; u < SF_VPT; ++u)
                    v[u] = *reinterpret_cast<const uint4*>(tile + (size_t)(u * 32 + lane) * 16);
                __syncwarp();
                if (i >= (uint64_t)SF_STAGES) ring.issue(s, tile_src(i - SF_STAGES));
                float c1[4] = {0.f, 0.f, 0.f, 0.f}, c2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int u = 0; u < SF_VPT; ++u)
#pragma unroll
                    for (int k = 0; k < EPV; ++k) one(sf_elem<T>(v[u], k), c1[k & 3], c2[k & 3]);
                sd += (double)((c1[0] + c1[1]) + (c1[2] + c1[3]));
                sv += (double)((c2[0] + c2[1]) + (c2[2] + c2[3]));
                s = s == 0 ? SF_STAGES - 1 : s - 1;
            }
            if (blockIdx.x == 0) {
                float d1 = 0.f, d2 = 0.f;
                const uint64_t t0 = a.ntiles * (SF_TILE / sizeof(T));
                for (uint64_t i = t0 + threadIdx.x; i < a.n; i += SF_THREADS) one(qp_load_one(x + i), d1, d2);
                sd += (double)d1;
                sv += (double)d2;
            }
        };
        if (guard) run(std::true_type{}); else run(std::false_type{});
        __syncthreads();
        ok = s_flag == 0;
        if (!ok) give_up();
        if (ok && HIST) {
            const int reps = 1 << rep_shift;
            for (int b = threadIdx.x; b < a.nb; b += SF_THREADS) {
                unsigned long long c = 0;
                for (int r = 0; r < reps; ++r) c += sh_hist[(b << rep_shift) + ((r + threadIdx.x) & (reps - 1))];
                if (c) atomicAdd(&a.hist[b], c);
            }
        }
    }
    {
        const double bsd = qp_block_sum(sd, sh);
        const double bsv = qp_block_sum(sv, sh);
        if (threadIdx.x == 0) {
            a.part[G + blockIdx.x].s0 = bsd;
            a.part[G + blockIdx.x].s1 = bsv;
        }
    }
    __syncthreads();
    ring.fini();

    // ---- exit: every block counts itself out (on every path); the last one finishes the call
    __threadfence();                                         // partials and histogram counts are out first
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(a.bar + 1, 1u) == (unsigned)G - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const bool good = qp_grid::ld_acquire(a.bar + 2) == 0u;  // nobody gave up: this block holds the first moments too
    if (good) {
        double sa = 0.0, sb = 0.0;
        for (unsigned k = threadIdx.x; k < (unsigned)G; k += SF_THREADS) {
            sa += __ldcg(&a.part[G + k].s0);
            sb += __ldcg(&a.part[G + k].s1);
        }
        sa = qp_block_sum(sa, sh);
        sb = qp_block_sum(sb, sh);
        double top = 0.0;
        if (HIST) {
            for (int k = threadIdx.x; k < a.nb; k += SF_THREADS) top = fmax(top, (double)__ldcg(&a.hist[k]));   // counts < 2^53
            top = qp_block_max(top, sh);
        }
        if (threadIdx.x == 0) {
            const unsigned long long nf = a.n - s_bad;
            qp_stats_t st;
            st.n = a.n;
            st.nonfinite = s_bad;
            st.mean = s_mean;
            st.mean_abs = s_mean_abs;
            st.mad = nf ? sa / (double)nf : 0.0;
            st.var = nf ? sb / (double)nf : 0.0;
            st.min = s_mn;
            st.max = s_mx;
            st.hist_peak = (HIST && s_mx > s_mn) ? (unsigned long long)top : 0ull;   // empty range: no histogram
            st.hist_bins = HIST ? a.nb : 0;
            st.reserved = 0;
            *a.out = st;
            if (s_bad) atomicOr(a.status, QP_DEV_NONFINITE);
        }
    }
    if (threadIdx.x == 0) {                                  // everybody has left: the scratch goes back to zero
        a.bar[0] = 0u;
        a.bar[1] = 0u;
        a.bar[2] = 0u;
    }
}

constexpr size_t SF_RING_BYTES = qp_stream::warp_ring<SF_TILE, SF_STAGES>::bytes(SF_WARPS);
constexpr size_t SF_HIST_BYTES = 16 * 1024;

// Whether this device can hold the one-launch statistics (checked once per context).
bool stats_fused_usable(qp_ctx* ctx)
{
    if (!ctx->stats_fused_checked) {
        ctx->stats_fused_checked = 1;
        int coop = 0, optin = 0;
        bool ok = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, ctx->device) == cudaSuccess && coop &&
                  cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, ctx->device) == cudaSuccess &&
                  2 * ctx->sm_count <= QP_MAX_BLOCKS;
        void* kernels[4] = {(void*)stats_fused_kernel<float, false>, (void*)stats_fused_kernel<float, true>,
                            (void*)stats_fused_kernel<unsigned short, false>, (void*)stats_fused_kernel<unsigned short, true>};
        for (int t = 0; ok && t < 4; ++t) {
            const size_t dyn = SF_RING_BYTES + ((t & 1) ? SF_HIST_BYTES : 0);
            cudaFuncAttributes fa;
            int per_sm = 0;
            ok = cudaFuncGetAttributes(&fa, kernels[t]) == cudaSuccess && (size_t)optin >= fa.sharedSizeBytes + dyn &&
                 cudaFuncSetAttribute(kernels[t], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) == cudaSuccess &&
                 cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernels[t], SF_THREADS, dyn) == cudaSuccess &&
                 per_sm >= 1;
        }
        if (!ok) cudaGetLastError();
        ctx->stats_fused_ok = ok ? 1 : 0;
    }
    return ctx->stats_fused_ok != 0;
}

template <typename T>
int32_t launch_fused(qp_ctx* ctx, const T* x, uint64_t n, int hist_bins, qp_stats_t* d_out, cudaStream_t s)
{
    const bool fuse = hist_bins >= 1 && hist_bins <= ST_FUSED_HIST_MAX;
    int rep_shift = 5;
    while (fuse && rep_shift > 0 && ((size_t)hist_bins << rep_shift) * sizeof(unsigned) > SF_HIST_BYTES) --rep_shift;
    SfArgs a;
    a.x = x;
    a.n = n;
    a.ntiles = n * sizeof(T) / SF_TILE;
    a.part = ctx->d_part;
    a.out = d_out;
    a.status = ctx->d_status;
    a.nb = fuse ? hist_bins : 0;
    a.rep_shift = fuse ? rep_shift : 0;
    a.hist = ctx->d_hist;
    a.bar = reinterpret_cast<unsigned*>(ctx->d_fused) + 8;       // words 8..10 of the barrier scratch (the sender uses 0, 1)
    a.wait_limit = ctx->wait_cycles;
    a.spin_limit = ctx->spin_limit;
    a.bar_extra = (unsigned)ctx->bar_extra;
    const uint64_t want = (a.ntiles + SF_WARPS - 1) / SF_WARPS;                 // a tile per warp at least
    const unsigned G = (unsigned)(want < (uint64_t)ctx->sm_count ? want : (uint64_t)ctx->sm_count);
    const size_t dyn = SF_RING_BYTES + (fuse ? SF_HIST_BYTES : 0);
    void* kernel = fuse ? (void*)stats_fused_kernel<T, true> : (void*)stats_fused_kernel<T, false>;
    void* params[] = {&a};
    if (cudaLaunchCooperativeKernel(kernel, dim3(G), dim3(SF_THREADS), params, dyn, s) != cudaSuccess)
        return qp_check_launch(ctx, "qp_stats (cooperative launch)");
    ctx->launches += 1;
    return qp_check_launch(ctx, "qp_stats");
}

template <typename T>
int32_t launch_typed(qp_ctx* ctx, const T* x, uint64_t n, qp_stats_t* d_out, cudaStream_t s)
{
    const uint64_t per_block = (uint64_t)QP_THREADS * UNROLL * qp_span<T>::EPV;
    uint64_t want = (n + per_block - 1) / per_block;
    const uint64_t cap = (uint64_t)ctx->sm_count * 6;
    int blocks = (int)(want < 1 ? 1 : (want > cap ? cap : want));
    if (blocks > QP_MAX_BLOCKS) blocks = QP_MAX_BLOCKS;
    stats_pass_a<T><<<blocks, QP_THREADS, 0, s>>>(x, n, ctx->d_part, ctx->d_ticket, d_out, ctx->d_status);
    stats_pass_b<T><<<blocks, QP_THREADS, 0, s>>>(x, n, ctx->d_part, ctx->d_ticket, d_out);
    ctx->launches += 2;
    return qp_check_launch(ctx, "qp_stats");
}

}  // namespace

extern "C" int qp_stats_carries_histogram(const void* d_x, int dtype, uint64_t n, int hist_bins)
{
    if (dtype != QP_F32 && dtype != QP_BF16) return 0;
    // the streamed kernels (aligned, at least 8 tiles) with a histogram small enough to ride along
    const uint64_t ntiles = ((uintptr_t)d_x & 15u) ? 0 : n * (dtype == QP_F32 ? 4 : 2) / ST_TILE;
    return (ntiles >= 8 && hist_bins >= 1 && hist_bins <= ST_FUSED_HIST_MAX) ? 1 : 0;
}

int32_t qp_launch_stats(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int hist_bins, qp_stats_t* d_out,
                        cudaStream_t s)
{
    if (n == 0) {
        if (cudaMemsetAsync(d_out, 0, sizeof(qp_stats_t), s) != cudaSuccess) return qp_check_launch(ctx, "qp_stats");
        return QP_OK;
    }
    const uint64_t ntiles = ((uintptr_t)d_x & 15u) ? 0 : n * (dtype == QP_F32 ? 4 : 2) / ST_TILE;
    // One launch or two.  Alone, the one-launch form is the faster with and without the histogram (129 MB:
    // 43.6 / 51.8 us against 51.0 / 59.0).  Inside the sender chain, where the pass runs while the receiver's
    // output of the step before is still being written back from L2, the two kernels are the faster once the
    // histogram rides along (66.3 us against 72.5; equal without it, 59 us): QP_STATS_AUTO takes the one launch
    // without the histogram and the two kernels with it; QP_STATS_FUSED and QP_STATS_TWO_KERNELS force either.
    const bool with_hist = hist_bins >= 1 && hist_bins <= ST_FUSED_HIST_MAX;
    const bool one_launch = ctx->stats_path == QP_STATS_FUSED || (ctx->stats_path == QP_STATS_AUTO && !with_hist);
    if (ntiles >= 8 && one_launch && stats_fused_usable(ctx)) {
        if (dtype == QP_F32) return launch_fused<float>(ctx, static_cast<const float*>(d_x), n, hist_bins, d_out, s);
        return launch_fused<unsigned short>(ctx, static_cast<const unsigned short*>(d_x), n, hist_bins, d_out, s);
    }
    if (ntiles >= 8) {                        // aligned and large enough for the streamed kernels to pay
        if (dtype == QP_F32)
            return launch_streamed<float>(ctx, static_cast<const float*>(d_x), n, ntiles, hist_bins, d_out, s);
        return launch_streamed<unsigned short>(ctx, static_cast<const unsigned short*>(d_x), n, ntiles, hist_bins, d_out, s);
    }
    if (dtype == QP_F32) return launch_typed<float>(ctx, static_cast<const float*>(d_x), n, d_out, s);
    return launch_typed<unsigned short>(ctx, static_cast<const unsigned short*>(d_x), n, d_out, s);
}

// ---------------------------------------------------------------------------------------
// Statistics without a context and without any allocation.
//
// Some callers must not allocate device memory at all: code that runs while a memory pool
// is frozen, inside a region where the allocator may not be re-entered, or in a process
// whose whole device budget was handed out before this library was loaded.  For them the
// scratch that qp_stats keeps in its qp_ctx (block partials, two tickets, a status word)
// lives in the fixed array below, which every GPU that loads the library holds until the
// process exits.  Its size bounds the grid (QP_STATIC_BLOCKS partials), not the tensor.
#include <mutex>

namespace {

constexpr int QP_STATIC_BLOCKS = 1024;
constexpr size_t QP_STATIC_PART_BYTES = sizeof(qp_stats_partial) * QP_STATIC_BLOCKS;      // 48 KiB
constexpr size_t QP_STATIC_BYTES = QP_STATIC_PART_BYTES + 256;                            // + tickets, status

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char qp_static_scratch[QP_STATIC_BYTES];

constexpr int QP_STATIC_MAX_DEVICES = 64;
std::mutex g_static_mu;
unsigned char* g_static_ptr[QP_STATIC_MAX_DEVICES] = {};
int g_static_sms[QP_STATIC_MAX_DEVICES] = {};

template <typename T>
int32_t static_typed(const T* x, uint64_t n, qp_stats_t* d_out, unsigned char* scratch, int sms, cudaStream_t s)
{
    qp_stats_partial* part = reinterpret_cast<qp_stats_partial*>(scratch);
    unsigned* ticket = reinterpret_cast<unsigned*>(scratch + QP_STATIC_PART_BYTES);        // [0], [1]
    unsigned* status = ticket + 4;
    // the array keeps whatever the last call left: tickets and status must start at zero
    if (cudaMemsetAsync(ticket, 0, 256, s) != cudaSuccess) { cudaGetLastError(); return QP_ERR_CUDA; }
    const uint64_t per_block = (uint64_t)QP_THREADS * UNROLL * qp_span<T>::EPV;
    uint64_t want = (n + per_block - 1) / per_block;
    const uint64_t cap = (uint64_t)sms * 6;
    int blocks = (int)(want < 1 ? 1 : (want > cap ? cap : want));
    if (blocks > QP_STATIC_BLOCKS) blocks = QP_STATIC_BLOCKS;
    stats_pass_a<T><<<blocks, QP_THREADS, 0, s>>>(x, n, part, ticket, d_out, status);
    stats_pass_b<T><<<blocks, QP_THREADS, 0, s>>>(x, n, part, ticket, d_out);
    return cudaGetLastError() == cudaSuccess ? QP_OK : QP_ERR_CUDA;
}

}  // namespace

extern "C" int32_t qp_stats_static(const void* d_x, int dtype, uint64_t n, qp_stats_t* d_out, void* stream)
{
    if (dtype != QP_F32 && dtype != QP_BF16) return QP_ERR_UNSUPPORTED_DTYPE;
    if (!d_out || (n > 0 && !d_x)) return QP_ERR_INVALID_ARG;
    if (((uintptr_t)d_x & (dtype == QP_F32 ? 3u : 1u)) || ((uintptr_t)d_out & 7u)) return QP_ERR_ALIGNMENT;
    if (n > QP_STATS_STATIC_MAX_N) return QP_ERR_TOO_LARGE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return QP_ERR_CUDA; }
    if (dev < 0 || dev >= QP_STATIC_MAX_DEVICES) return QP_ERR_INVALID_ARG;
    unsigned char* scratch = nullptr;
    int sms = 0;
    {
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!g_static_ptr[dev]) {
            // once per device, with that device current: resolve the array's device address
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, qp_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return QP_ERR_CUDA; }
            int count = 0;
            if (cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || count < 1) {
                cudaGetLastError();
                return QP_ERR_CUDA;
            }
            g_static_sms[dev] = count;
            g_static_ptr[dev] = static_cast<unsigned char*>(p);
        }
        scratch = g_static_ptr[dev];
        sms = g_static_sms[dev];
    }
    if (n == 0) return cudaMemsetAsync(d_out, 0, sizeof(qp_stats_t), s) == cudaSuccess ? QP_OK : QP_ERR_CUDA;
    if (dtype == QP_F32) return static_typed<float>(static_cast<const float*>(d_x), n, d_out, scratch, sms, s);
    return static_typed<unsigned short>(static_cast<const unsigned short*>(d_x), n, d_out, scratch, sms, s);
}
