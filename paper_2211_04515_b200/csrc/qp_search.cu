// a2 + a3 + a4: histogram peak, ACIQ clip on the device, and the directed search DS-ACIQ
// (paper Sec. 3 "Directed Search", Eq. 1).
//
//   hist      count histogram of x over [min, max] in shared memory (lane-replicated
//             counters, no same-address contention), merged into global 64-bit counters
//   setup     peak -> b_R, the steps+1 candidate scales b_k and their quantizers
//   eval      every thread scores QP_EVAL_K candidates against each element it loads and
//             keeps K error sums (fp32 over 8 elements, then fp64); blockIdx.x picks the
//             candidate group, groups of the same chunk of x run next to each other so x
//             is fetched from HBM once and re-read from L2; the kernel is bound by fp32
//             ALU throughput, not by memory
//   finalize  fixed-order merge of the block sums, MSE per candidate, first minimum wins
#include "qp_internal.cuh"

namespace {

constexpr int K = QP_EVAL_K;

// -------------------------------------------------------------------- histogram

template <typename T, bool GUARD>
__device__ __forceinline__ void hist_body(const T* __restrict__ x, uint64_t n, float mn, float inv_w, int nb, int rep_mask,
                                          int rep_shift, unsigned* __restrict__ sh)
{
    constexpr int EPV = qp_span<T>::EPV;
    const qp_span<T> sp(x, n);
    const T* xv = x + sp.head;
    const uint64_t stride = (uint64_t)gridDim.x * QP_THREADS;
    const int lane_rep = threadIdx.x & rep_mask;
    auto one = [&](float e) {
        if (GUARD && !qp_is_finite(e)) return;
        // bin = floor((x - min) * inv_w), the last bin closed; fp32, each op rounded once
        int b = __float2int_rz(__fmul_rn(__fsub_rn(e, mn), inv_w));
        b = min(max(b, 0), nb - 1);
        atomicAdd(&sh[(b << rep_shift) + lane_rep], 1u);
    };
    for (uint64_t v = (uint64_t)blockIdx.x * QP_THREADS + threadIdx.x; v < sp.nvec; v += 2 * stride) {
        float e0[EPV], e1[EPV];
        const bool two = v + stride < sp.nvec;
        qp_load_vec(xv + v * EPV, e0);
        if (two) qp_load_vec(xv + (v + stride) * EPV, e1);
#pragma unroll
        for (int i = 0; i < EPV; ++i) one(e0[i]);
        if (two) {
#pragma unroll
            for (int i = 0; i < EPV; ++i) one(e1[i]);
        }
    }
    if (blockIdx.x == 0) {
        for (uint64_t i = threadIdx.x; i < sp.head; i += QP_THREADS) one(qp_load_one(x + i));
        const uint64_t t0 = sp.head + sp.nvec * EPV;
        for (uint64_t i = threadIdx.x; i < sp.tail; i += QP_THREADS) one(qp_load_one(x + t0 + i));
    }
}

template <typename T>
__global__ void __launch_bounds__(QP_THREADS) hist_kernel(const T* __restrict__ x, uint64_t n,
                                                          const qp_stats_t* __restrict__ st, int nb, int rep_shift,
                                                          unsigned long long* __restrict__ hist)
{
    extern __shared__ unsigned sh[];
    if (st->hist_bins == nb) return;                 // the statistics already carry this histogram's peak
    const int reps = 1 << rep_shift;
    for (int i = threadIdx.x; i < nb * reps; i += QP_THREADS) sh[i] = 0u;
    __syncthreads();
    const double mn = st->min, mx = st->max;
    if (mx > mn) {
        const float inv_w = (float)((double)nb / (mx - mn));
        if (st->nonfinite == 0) hist_body<T, false>(x, n, (float)mn, inv_w, nb, reps - 1, rep_shift, sh);
        else                    hist_body<T, true>(x, n, (float)mn, inv_w, nb, reps - 1, rep_shift, sh);
    }
    __syncthreads();
    for (int b = threadIdx.x; b < nb; b += QP_THREADS) {
        unsigned long long c = 0;
        for (int r = 0; r < reps; ++r) c += sh[(b << rep_shift) + ((r + threadIdx.x) & (reps - 1))];
        if (c) atomicAdd(&hist[b], c);
    }
}

// ------------------------------------------------------------------------ setup

__global__ void __launch_bounds__(QP_THREADS) setup_kernel(const qp_stats_t* __restrict__ st,
                                                           const unsigned long long* __restrict__ hist, int nb, int bits,
                                                           int bmode, int steps, double F, float4* __restrict__ cand,
                                                           int* __restrict__ valid, qp_ds_setup* __restrict__ setup,
                                                           unsigned* __restrict__ status)
{
    __shared__ unsigned long long sh_top[QP_THREADS];
    __shared__ qp_ds_setup s;
    unsigned long long top = 0;
    const bool from_stats = st->hist_bins == nb;
    const bool promised = (bmode & QP_B_HIST_IN_STATS) != 0;      // then nobody has counted into hist
    if (promised && !from_stats && threadIdx.x == 0) atomicOr(status, QP_DEV_HIST_MISSING);
    for (int b = threadIdx.x; !from_stats && !promised && b < nb; b += QP_THREADS) {
        const unsigned long long c = hist[b];
        top = c > top ? c : top;
    }
    sh_top[threadIdx.x] = top;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < QP_THREADS; ++i) top = sh_top[i] > top ? sh_top[i] : top;
        if (from_stats) top = st->hist_peak;
        qp_ds_make_setup(st, top, nb, bmode, F, s);
        *setup = s;
    }
    __syncthreads();
    for (int k = threadIdx.x; k <= steps; k += QP_THREADS) {
        float4 c;
        int ok;
        qp_ds_candidate(s, k, steps, bits, bmode & QP_B_MIDRISE, c, ok);
        cand[k] = c;
        valid[k] = ok;
    }
}

// ------------------------------------------------------------------------- eval

template <bool GUARD, int NE>
__device__ __forceinline__ void score(const float (&e)[NE], const float (&lo)[K], const float (&hi)[K],
                                      const float (&sc)[K], const float (&iv)[K], double (&acc)[K])
{
    float p[K];
#pragma unroll
    for (int k = 0; k < K; ++k) p[k] = 0.f;
#pragma unroll
    for (int i = 0; i < NE; ++i) {
        const float x = e[i];
        const bool fin = !GUARD || qp_is_finite(x);
#pragma unroll
        for (int k = 0; k < K; ++k) {
            // level index as a float: (pos + 1.5*2^23) - 1.5*2^23 rounds to nearest, ties to even
            const float pos = qp_grid_pos(x, lo[k], hi[k], iv[k]);
            const float r = __fsub_rn(__fadd_rn(pos, QP_MAGIC), QP_MAGIC);
            const float d = __fsub_rn(fmaf(r, sc[k], lo[k]), x);
            if (GUARD) { if (fin) p[k] = fmaf(d, d, p[k]); }
            else       p[k] = fmaf(d, d, p[k]);
        }
    }
#pragma unroll
    for (int k = 0; k < K; ++k) acc[k] += (double)p[k];
}

template <typename T, bool GUARD>
__device__ __forceinline__ void eval_body(const T* __restrict__ x, uint64_t n, unsigned chunk, unsigned chunks,
                                          const float (&lo)[K], const float (&hi)[K], const float (&sc)[K],
                                          const float (&iv)[K], double (&acc)[K])
{
    constexpr int EPV = qp_span<T>::EPV;
    constexpr int NV = 8 / EPV;                       // 8 elements per scoring round
    const qp_span<T> sp(x, n);
    const T* xv = x + sp.head;
    const uint64_t stride = (uint64_t)chunks * QP_THREADS;
    uint64_t v = (uint64_t)chunk * QP_THREADS + threadIdx.x;
    for (; v + (NV - 1) * stride < sp.nvec; v += NV * stride) {
        float e[8];
        if (NV == 2) {
            float a[EPV], b[EPV];
            qp_load_vec(xv + v * EPV, a);
            qp_load_vec(xv + (v + stride) * EPV, b);
#pragma unroll
            for (int i = 0; i < EPV; ++i) { e[i] = a[i]; e[EPV + i] = b[i]; }
        } else {
            float a[EPV];
            qp_load_vec(xv + v * EPV, a);
#pragma unroll
            for (int i = 0; i < EPV; ++i) e[i] = a[i];
        }
        score<GUARD, 8>(e, lo, hi, sc, iv, acc);
    }
    for (; v < sp.nvec; v += stride) {
        float a[EPV];
        qp_load_vec(xv + v * EPV, a);
        score<GUARD, EPV>(a, lo, hi, sc, iv, acc);
    }
    if (chunk == 0) {
        for (uint64_t i = threadIdx.x; i < sp.head; i += QP_THREADS) {
            const float a[1] = {qp_load_one(x + i)};
            score<GUARD, 1>(a, lo, hi, sc, iv, acc);
        }
        const uint64_t t0 = sp.head + sp.nvec * EPV;
        for (uint64_t i = threadIdx.x; i < sp.tail; i += QP_THREADS) {
            const float a[1] = {qp_load_one(x + t0 + i)};
            score<GUARD, 1>(a, lo, hi, sc, iv, acc);
        }
    }
}

// grid = (groups, chunks): the candidate group is the fastest-varying block index, so the
// groups of one chunk are scheduled together and share its lines in L2.
template <typename T>
__global__ void __launch_bounds__(QP_THREADS) eval_kernel(const T* __restrict__ x, uint64_t n,
                                                          const qp_stats_t* __restrict__ st,
                                                          const float4* __restrict__ cand, int ncand,
                                                          double* __restrict__ sums)
{
    const int g = blockIdx.x;
    const unsigned chunk = blockIdx.y, chunks = gridDim.y;
    float lo[K], hi[K], sc[K], iv[K];
    double acc[K];
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const int c = min(g * K + k, ncand - 1);
        const float4 q = cand[c];
        lo[k] = q.x; hi[k] = q.y; sc[k] = q.z; iv[k] = q.w;
        acc[k] = 0.0;
    }
    if (st->nonfinite == 0) eval_body<T, false>(x, n, chunk, chunks, lo, hi, sc, iv, acc);
    else                    eval_body<T, true>(x, n, chunk, chunks, lo, hi, sc, iv, acc);

    __shared__ double sh[QP_THREADS / 32];
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const double t = qp_block_sum(acc[k], sh);
        if (threadIdx.x == 0) sums[((size_t)g * chunks + chunk) * K + k] = t;
    }
}

// --------------------------------------------------------------------- finalize

__global__ void __launch_bounds__(QP_THREADS) finalize_kernel(const double* __restrict__ sums, int chunks, int steps,
                                                              int from_sums,
                                                              int nb, int bits, const int* __restrict__ valid,
                                                              const float4* __restrict__ cand,
                                                              const qp_ds_setup* __restrict__ setup,
                                                              double* __restrict__ curve, qp_ds_result_t* __restrict__ out,
                                                              qp_qparams_t* __restrict__ qp_out,
                                                              unsigned* __restrict__ status)
{
    const qp_ds_setup s = *setup;
    for (int k = threadIdx.x; from_sums && k <= steps; k += QP_THREADS) {
        const int g = k / K, j = k % K;
        double t = 0.0;
        for (int b = 0; b < chunks; ++b) t += sums[((size_t)g * chunks + b) * K + j];
        double mse = s.n_finite ? t / (double)s.n_finite : 0.0;
        if (!valid[k]) mse = __longlong_as_double(0x7FF0000000000000ll);
        curve[k] = mse;
    }
    __syncthreads();
    __threadfence_block();
    __shared__ double s_curve[QP_MAX_STEPS + 1];
    qp_ds_pick(curve, steps, nb, bits, cand, setup, out, qp_out, status, s_curve);
}

// one thread: closed-form clip (ACIQ, ACIQ cut back to the data range, or min/max) from
// device-resident statistics
__global__ void aciq_kernel(const qp_stats_t* __restrict__ st, int bits, int method, int dist, int bmode, double F,
                            qp_qparams_t* __restrict__ qp_out, unsigned* __restrict__ status)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    double lo, hi;
    qp_clip_ends(*st, method, dist, bmode, bits, F, lo, hi);
    qp_qparams_t q;
    const int rc = qp_fill_qparams(lo, hi, bits, &q);
    *qp_out = q;
    if (rc == QP_WARN_DEGENERATE) atomicOr(status, QP_DEV_DEGENERATE);
}

template <typename T>
int32_t search_typed(qp_ctx* ctx, const T* x, uint64_t n, const qp_stats_t* d_stats, int bits, int bmode, int steps,
                     int nb, double F, qp_ds_result_t* d_out, qp_qparams_t* d_qp_out, cudaStream_t s)
{
    // histogram: as many lane replicas of each bin as fit in 64 KB of shared memory
    int rep_shift = 5;
    while (rep_shift > 0 && ((size_t)nb << rep_shift) * sizeof(unsigned) > 64 * 1024) --rep_shift;
    const size_t sh_bytes = ((size_t)nb << rep_shift) * sizeof(unsigned);
    if (cudaFuncSetAttribute(hist_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024) != cudaSuccess)
        return qp_check_launch(ctx, "qp_dsaciq_search (histogram attribute)");
    const uint64_t per_block = (uint64_t)QP_THREADS * 2 * qp_span<T>::EPV;
    uint64_t want = (n + per_block - 1) / per_block;
    const uint64_t hcap = (uint64_t)ctx->sm_count * 3;
    const int hblocks = (int)(want < 1 ? 1 : (want > hcap ? hcap : want));
    if (!(bmode & QP_B_HIST_IN_STATS)) {
        // returns at once when the statistics already carry this histogram's peak
        if (cudaMemsetAsync(ctx->d_hist, 0, sizeof(unsigned long long) * nb, s) != cudaSuccess)
            return qp_check_launch(ctx, "qp_dsaciq_search (histogram reset)");
        hist_kernel<T><<<hblocks, QP_THREADS, sh_bytes, s>>>(x, n, d_stats, nb, rep_shift, ctx->d_hist);
        ctx->launches += 1;
    }

    const int ncand = steps + 1;
    // interval-moment scoring where its tables fit and its fixed-point sums cannot overflow
    const bool iv_fits = ncand * ((1 << bits) - 1) + QP_IV_CELLS <= QP_IV_MAXB &&
                         n / (uint64_t)ctx->iv_blocks + 65536 < (1ull << 22);
    const bool use_iv = iv_fits && (ctx->search_path == QP_SEARCH_INTERVALS ||
                                    (ctx->search_path == QP_SEARCH_AUTO && n >= (1ull << 20)));
    if (use_iv)
        return qp_launch_interval_search(ctx, x, sizeof(T) == 4 ? QP_F32 : QP_BF16, n, d_stats, bits, bmode, steps, nb, F,
                                         d_out, d_qp_out, s);
    setup_kernel<<<1, QP_THREADS, 0, s>>>(d_stats, ctx->d_hist, nb, bits, bmode, steps, F, ctx->d_cand, ctx->d_valid,
                                          ctx->d_setup, ctx->d_status);
    const int groups = (ncand + K - 1) / K;
    const uint64_t per_chunk = (uint64_t)QP_THREADS * 8;
    want = (n + per_chunk - 1) / per_chunk;
    uint64_t ccap = (uint64_t)ctx->sm_count * 4 / (uint64_t)groups;     // about 4 resident blocks per SM in all
    if (ccap < 1) ccap = 1;
    if (ccap * groups > QP_MAX_BLOCKS) ccap = QP_MAX_BLOCKS / groups;
    const int chunks = (int)(want < 1 ? 1 : (want > ccap ? ccap : want));
    eval_kernel<T><<<dim3(groups, chunks), QP_THREADS, 0, s>>>(x, n, d_stats, ctx->d_cand, ncand, ctx->d_sums);
    finalize_kernel<<<1, QP_THREADS, 0, s>>>(ctx->d_sums, chunks, steps, 1, nb, bits, ctx->d_valid, ctx->d_cand,
                                             ctx->d_setup, ctx->d_curve, d_out, d_qp_out, ctx->d_status);
    ctx->launches += 3;
    return qp_check_launch(ctx, "qp_dsaciq_search");
}

}  // namespace

int32_t qp_launch_search(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, const qp_stats_t* d_stats, int bits,
                         int bmode, int steps, int hist_bins, double F, qp_ds_result_t* d_out, qp_qparams_t* d_qp_out,
                         cudaStream_t s)
{
    if (dtype == QP_F32)
        return search_typed<float>(ctx, static_cast<const float*>(d_x), n, d_stats, bits, bmode, steps, hist_bins, F,
                                   d_out, d_qp_out, s);
    return search_typed<unsigned short>(ctx, static_cast<const unsigned short*>(d_x), n, d_stats, bits, bmode, steps,
                                        hist_bins, F, d_out, d_qp_out, s);
}

int32_t qp_launch_aciq_device(qp_ctx* ctx, const qp_stats_t* d_stats, int bits, int method, int dist, int bmode, double F,
                              qp_qparams_t* d_qp_out, cudaStream_t s)
{
    aciq_kernel<<<1, 32, 0, s>>>(d_stats, bits, method, dist, bmode, F, d_qp_out, ctx->d_status);
    ctx->launches += 1;
    return qp_check_launch(ctx, "qp_aciq_qparams_device");
}
