// Channel-wise variant of a2 + a4: the directed search (paper Sec. 3 "Directed Search", Eq. 1)
// run for every channel of a [rows, channels] tensor on its column alone.  The paper searches
// one clip per tensor; per-channel ranges are what its cited PTQ work uses for activations with
// outlier channels, and this is the same search with the column in place of the tensor.
//
// Four kernels, all indexed so that a warp reads consecutive channels of one row (coalesced):
//   ch_hist_kernel    per-channel histogram of hist_bins equal bins over the channel's [min, max]
//                     (the per-tensor bin expression), shared-memory counters per block of 64
//                     channels, merged into global counters
//   ch_setup_kernel   block per channel: peak -> b_R, the candidates and their quantizers
//   ch_eval_kernel    thread = (channel, group of 8 candidates, row lane): the candidate path's
//                     arithmetic on the column, fp32 error sums over 8 rows folded into fp64,
//                     block partials per (row block, channel, candidate)
//   ch_pick_kernel    block per channel: partials merged in row-block order, first minimum wins
// Work is (steps + 1) * 9 fp32 instructions per element, as in the per-tensor candidate path.  Where the
// interval form applies (qp_channels_search_fast.cu: one pass over the tensor instead of the scoring) it
// takes ch_eval_kernel's place and hands the pick one row block of sums.
#include <stdlib.h>

#include "qp_internal.cuh"

QP_CK_UNIT

namespace {

constexpr int CK = QP_EVAL_K;                       // candidates per thread
constexpr int CS_HIST_CH = 64;                      // channels per histogram block
constexpr int CS_HIST_ROWS = 512;                   // rows per histogram block
constexpr int CS_EVAL_CH = 32;                      // channels per scoring block (one warp wide)
constexpr int CS_EVAL_LANES = 8;                    // row lanes per scoring block
constexpr int CS_MAX_ROW_BLOCKS = 64;

template <typename T>
__device__ __forceinline__ float cs_load(const T* p)
{
    return qp_load_one(p);
}

template <typename T>
__global__ void __launch_bounds__(256) ch_hist_kernel(const T* __restrict__ x, uint64_t rows, uint32_t C,
                                                      const qp_stats_t* __restrict__ st, int nb,
                                                      unsigned* __restrict__ hist)
{
    extern __shared__ unsigned sh[];                // [CS_HIST_CH][nb]
    const uint32_t c0 = blockIdx.y * CS_HIST_CH;
    const uint32_t cl = threadIdx.x % CS_HIST_CH, rl = threadIdx.x / CS_HIST_CH;
    const uint32_t c = c0 + cl;
    for (int i = threadIdx.x; i < CS_HIST_CH * nb; i += 256) sh[i] = 0u;
    __syncthreads();
    if (c < C) {
        const double mn = st[c].min, mx = st[c].max;
        if (mx > mn) {
            // bin = floor((x - min) * inv_w), the last bin closed; fp32, each op rounded once
            const float fmn = (float)mn, inv_w = (float)((double)nb / (mx - mn));
            const uint64_t r0 = (uint64_t)blockIdx.x * CS_HIST_ROWS;
            const uint64_t r1 = r0 + CS_HIST_ROWS < rows ? r0 + CS_HIST_ROWS : rows;
            unsigned* mine = sh + cl * nb;
            constexpr uint64_t RL = 256 / CS_HIST_CH;           // row lanes of a block
            auto count = [&](float e) {
                if (!qp_is_finite(e)) return;
                int b = __float2int_rz(__fmul_rn(__fsub_rn(e, fmn), inv_w));
                b = min(max(b, 0), nb - 1);
                atomicAdd(&mine[QP_CK(b, nb)], 1u);
            };
            uint64_t r = r0 + rl;
            for (; r + 7 * RL < r1; r += 8 * RL) {              // eight loads ahead of their counting
                float e[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) e[q] = cs_load(x + (r + q * RL) * C + c);
#pragma unroll
                for (int q = 0; q < 8; ++q) count(e[q]);
            }
            for (; r < r1; r += RL) count(cs_load(x + r * C + c));
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < CS_HIST_CH * nb; i += 256) {
        const uint32_t cc = c0 + i / nb;
        const unsigned v = sh[i];
        if (v && cc < C) atomicAdd(&hist[(size_t)cc * nb + i % nb], v);
    }
}

__global__ void __launch_bounds__(128) ch_setup_kernel(const qp_stats_t* __restrict__ st, const unsigned* __restrict__ hist,
                                                       int nb, int bits, int bmode, int steps, int ncp, double F,
                                                       float4* __restrict__ cand, int* __restrict__ valid,
                                                       qp_ds_setup* __restrict__ setup)
{
    const uint32_t c = blockIdx.x;
    __shared__ unsigned s_top[128];
    __shared__ qp_ds_setup s;
    unsigned top = 0;
    for (int b = threadIdx.x; b < nb; b += 128) top = max(top, hist[(size_t)c * nb + b]);
    s_top[threadIdx.x] = top;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 128; ++i) top = max(top, s_top[i]);
        qp_ds_make_setup(&st[c], (unsigned long long)top, nb, bmode, F, s);
        s.g_lo = s.g_hi = s.inv_gw = s.inv_u = s.gw = s.pad2 = 0.f;
        s.u = 0.0;
        setup[c] = s;
    }
    __syncthreads();
    for (int k = threadIdx.x; k < ncp; k += 128) {
        float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
        int ok = 0;
        if (k <= steps) qp_ds_candidate(s, k, steps, bits, bmode & QP_B_MIDRISE, q, ok);
        cand[(size_t)c * ncp + k] = q;
        valid[(size_t)c * ncp + k] = ok;
    }
}

// grid = (channel tiles, candidate groups, row blocks); block = 32 channels x 8 row lanes
template <typename T>
__global__ void __launch_bounds__(CS_EVAL_CH * CS_EVAL_LANES, 4) ch_eval_kernel(const T* __restrict__ x, uint64_t rows,
                                                                             uint32_t C, uint64_t rows_per_block,
                                                                             const float4* __restrict__ cand, int ncp,
                                                                             double* __restrict__ part)
{
    const uint32_t cl = threadIdx.x & 31, rl = threadIdx.x >> 5;
    const uint32_t c = blockIdx.x * CS_EVAL_CH + cl;
    const int g = blockIdx.y;
    const uint64_t r0 = (uint64_t)blockIdx.z * rows_per_block;
    const uint64_t r1 = r0 + rows_per_block < rows ? r0 + rows_per_block : rows;
    float lo[CK], hi[CK], sc[CK], iv[CK];
    double acc[CK];
#pragma unroll
    for (int k = 0; k < CK; ++k) {
        const float4 q = c < C ? cand[(size_t)c * ncp + g * CK + k] : make_float4(0.f, 0.f, 0.f, 0.f);
        lo[k] = q.x; hi[k] = q.y; sc[k] = q.z; iv[k] = q.w;
        acc[k] = 0.0;
    }
    if (c < C && r0 + rl < r1) {
        // this lane's rows r0 + rl, r0 + rl + 8, ...: batches of 8 (fp32 sums per batch, then fp64)
        const T* px = x + (r0 + rl) * C + c;
        const size_t step = (size_t)CS_EVAL_LANES * C;
        const uint64_t mine = (r1 - r0 - rl + CS_EVAL_LANES - 1) / CS_EVAL_LANES;
        auto batch = [&](int count) {                       // count <= 8 rows from px on
            float p[CK];
#pragma unroll
            for (int k = 0; k < CK; ++k) p[k] = 0.f;
#pragma unroll
            for (int half = 0; half < 2; ++half) {          // four loads ahead of their scoring
                float e[4];
#pragma unroll
                for (int it = 0; it < 4; ++it)
                    e[it] = half * 4 + it < count ? cs_load(px + (half * 4 + it) * step) : __int_as_float(0x7FC00000);
#pragma unroll
                for (int it = 0; it < 4; ++it) {
                    const float v = e[it];
                    const bool fin = qp_is_finite(v);       // also skips the rows beyond `count`
#pragma unroll
                    for (int k = 0; k < CK; ++k) {
                        const float pos = qp_grid_pos(v, lo[k], hi[k], iv[k]);
                        const float lev = __fsub_rn(__fadd_rn(pos, QP_MAGIC), QP_MAGIC);
                        const float d = __fsub_rn(fmaf(lev, sc[k], lo[k]), v);
                        if (fin) p[k] = fmaf(d, d, p[k]);
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < CK; ++k) acc[k] += (double)p[k];
        };
        for (uint64_t b = 0; b < mine / 8; ++b) {
            batch(8);
            px += 8 * step;
        }
        if (mine % 8) batch((int)(mine % 8));
    }
    // the 8 row lanes of a channel, merged in lane order
    __shared__ double sh[CS_EVAL_LANES][CK][CS_EVAL_CH];
#pragma unroll
    for (int k = 0; k < CK; ++k) sh[rl][k][cl] = acc[k];
    __syncthreads();
    if (rl == 0 && c < C) {
#pragma unroll
        for (int k = 0; k < CK; ++k) {
            double t = 0.0;
            for (int l = 0; l < CS_EVAL_LANES; ++l) t += sh[l][k][cl];
            part[((size_t)blockIdx.z * C + c) * ncp + g * CK + k] = t;
        }
    }
}

__global__ void __launch_bounds__(128) ch_pick_kernel(const double* __restrict__ part, int row_blocks, uint32_t C, int steps,
                                                      int ncp, int nb, int bits, const int* __restrict__ valid,
                                                      const float4* __restrict__ cand,
                                                      const qp_ds_setup* __restrict__ setup, double* __restrict__ curve,
                                                      qp_ds_result_t* __restrict__ out, qp_qparams_t* __restrict__ qp_out,
                                                      unsigned* __restrict__ status)
{
    const uint32_t c = blockIdx.x;
    __shared__ double s_curve[128];
    const qp_ds_setup s = setup[c];
    for (int k = threadIdx.x; k <= steps; k += 128) {
        double t = 0.0;
        for (int b = 0; b < row_blocks; ++b) t += part[((size_t)b * C + c) * ncp + k];
        double mse = s.n_finite ? t / (double)s.n_finite : 0.0;
        if (!valid[(size_t)c * ncp + k]) mse = __longlong_as_double(0x7FF0000000000000ll);
        s_curve[k] = mse;
        curve[(size_t)c * ncp + k] = mse;
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    int best = 0;
    double best_mse = s_curve[0];
    for (int k = 1; k <= steps; ++k)
        if (s_curve[k] < best_mse) { best_mse = s_curve[k]; best = k; }
    qp_ds_write_result(best, s_curve, s, steps, nb, bits, cand[(size_t)c * ncp + best], out ? out + c : nullptr,
                       qp_out ? qp_out + c : nullptr, status);
}

size_t align256(size_t v) { return (v + 255) / 256 * 256; }

template <typename T>
int32_t search_channels_typed(qp_ctx* ctx, const T* x, uint64_t rows, uint32_t C, const qp_stats_t* d_stats, int bits,
                              int bmode, int steps, int nb, double F, qp_ds_result_t* d_out, qp_qparams_t* d_qp_out,
                              cudaStream_t s)
{
    const int ncp = (steps + 1 + CK - 1) / CK * CK;          // candidates padded to whole groups
    const int groups = ncp / CK;
    // row blocks of the scoring: enough blocks to fill the GPU, at most CS_MAX_ROW_BLOCKS partial rows
    const uint64_t tiles = ((uint64_t)C + CS_EVAL_CH - 1) / CS_EVAL_CH * (uint64_t)groups;
    uint64_t row_blocks = ((uint64_t)ctx->sm_count * 16 + tiles - 1) / tiles;
    if (row_blocks > CS_MAX_ROW_BLOCKS) row_blocks = CS_MAX_ROW_BLOCKS;
    const uint64_t min_rows = 8 * CS_EVAL_LANES;             // no point in blocks of less than one batch per lane
    if (row_blocks > (rows + min_rows - 1) / min_rows) row_blocks = (rows + min_rows - 1) / min_rows;
    if (row_blocks < 1) row_blocks = 1;
    // interval moments where they apply (qp_set_search_path(QP_SEARCH_CANDIDATES) keeps the scoring of every candidate)
    const bool intervals = ctx->search_path != QP_SEARCH_CANDIDATES && qp_channel_interval_applies(rows, bits, steps);
    if (intervals) row_blocks = 1;
    const uint64_t rows_per_block = (rows + row_blocks - 1) / row_blocks;

    size_t off = 0;
    const size_t o_hist = off;  off = align256(off + sizeof(unsigned) * (size_t)C * nb);
    const size_t o_cand = off;  off = align256(off + sizeof(float4) * (size_t)C * ncp);
    const size_t o_valid = off; off = align256(off + sizeof(int) * (size_t)C * ncp);
    const size_t o_setup = off; off = align256(off + sizeof(qp_ds_setup) * (size_t)C);
    const size_t o_curve = off; off = align256(off + sizeof(double) * (size_t)C * ncp);
    const size_t o_part = off;  off = align256(off + sizeof(double) * (size_t)row_blocks * C * ncp);
    const size_t o_iv = off;
    if (intervals) off = align256(off + qp_channel_interval_scratch_bytes(C, (steps + 1) * ((1 << bits) - 1)));
    if (ctx->ch_search_bytes < off) {                        // grown on demand, kept by the context
        if (ctx->d_ch_search) cudaFree(ctx->d_ch_search);
        ctx->d_ch_search = nullptr;
        ctx->ch_search_bytes = 0;
        if (cudaMalloc(&ctx->d_ch_search, off) != cudaSuccess) {
            cudaGetLastError();
            return qp_fail(ctx, QP_ERR_CUDA, "cannot allocate the channel search scratch");
        }
        ctx->ch_search_bytes = off;
    }
    char* b = static_cast<char*>(ctx->d_ch_search);
    unsigned* hist = reinterpret_cast<unsigned*>(b + o_hist);
    float4* cand = reinterpret_cast<float4*>(b + o_cand);
    int* valid = reinterpret_cast<int*>(b + o_valid);
    qp_ds_setup* setup = reinterpret_cast<qp_ds_setup*>(b + o_setup);
    double* curve = reinterpret_cast<double*>(b + o_curve);
    double* part = reinterpret_cast<double*>(b + o_part);

    if (cudaMemsetAsync(hist, 0, sizeof(unsigned) * (size_t)C * nb, s) != cudaSuccess)
        return qp_check_launch(ctx, "qp_dsaciq_search_channels (histogram reset)");
    const size_t hist_smem = sizeof(unsigned) * CS_HIST_CH * (size_t)nb;
    if (cudaFuncSetAttribute(ch_hist_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)hist_smem) != cudaSuccess)
        return qp_check_launch(ctx, "qp_dsaciq_search_channels (histogram attribute)");
    if (rows > 0) {
        const dim3 hgrid((unsigned)((rows + CS_HIST_ROWS - 1) / CS_HIST_ROWS), (C + CS_HIST_CH - 1) / CS_HIST_CH);
        ch_hist_kernel<T><<<hgrid, 256, hist_smem, s>>>(x, rows, C, d_stats, nb, hist);
        ctx->launches += 1;
    }
    ch_setup_kernel<<<C, 128, 0, s>>>(d_stats, hist, nb, bits, bmode, steps, ncp, F, cand, valid, setup);
    ctx->launches += 1;
    if (intervals) {
        const int32_t rc = qp_launch_channel_interval_sums(ctx, x, sizeof(T) == 4 ? QP_F32 : QP_BF16, rows, C, bits, steps, ncp,
                                                           d_stats, cand, valid, setup, b + o_iv, part, s);
        if (rc != QP_OK) return rc;
    } else {
        const dim3 egrid((C + CS_EVAL_CH - 1) / CS_EVAL_CH, groups, (unsigned)row_blocks);
        ch_eval_kernel<T><<<egrid, CS_EVAL_CH * CS_EVAL_LANES, 0, s>>>(x, rows, C, rows_per_block, cand, ncp, part);
        ctx->launches += 1;
    }
    ch_pick_kernel<<<C, 128, 0, s>>>(part, (int)row_blocks, C, steps, ncp, nb, bits, valid, cand, setup, curve, d_out,
                                     d_qp_out, ctx->d_status);
    ctx->launches += 1;
    ctx->ch_last_steps = steps;
    ctx->ch_last_ncp = ncp;
    ctx->ch_last_channels = C;
    ctx->ch_curve_offset = o_curve;
    ctx->ch_cand_offset = o_cand;
    ctx->ch_last_bits = bits;
    return qp_check_launch(ctx, "qp_dsaciq_search_channels");
}

}  // namespace

extern "C" int32_t qp_dsaciq_search_channels(qp_ctx* ctx, const void* d_x, int dtype, uint64_t rows, uint32_t channels,
                                             const qp_stats_t* d_stats, int bits, int bmode, int steps, int hist_bins,
                                             qp_ds_result_t* d_out, qp_qparams_t* d_qp_out, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (dtype != QP_F32 && dtype != QP_BF16) return qp_fail(ctx, QP_ERR_UNSUPPORTED_DTYPE, "dtype must be QP_F32 or QP_BF16");
    if (channels < 1 || channels > QP_MAX_CHANNELS) return qp_fail(ctx, QP_ERR_INVALID_ARG, "channels must be 1..QP_MAX_CHANNELS");
    if (rows >= (1ull << 40) / channels) return qp_fail(ctx, QP_ERR_INVALID_ARG, "tensor too large");
    if ((rows > 0 && !d_x) || !d_stats || !d_qp_out) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null pointer");
    if ((uintptr_t)d_x & (dtype == QP_F32 ? 3u : 1u)) return qp_fail(ctx, QP_ERR_ALIGNMENT, "d_x must be aligned to its element size");
    if (((uintptr_t)d_stats & 7u) || ((uintptr_t)d_out & 7u) || ((uintptr_t)d_qp_out & 3u))
        return qp_fail(ctx, QP_ERR_ALIGNMENT, "statistics / result pointers");
    if (bits < 1 || bits > 8) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "the search supports 1..8 bits");
    {
        const int base = bmode & ~(QP_B_MIDRISE | QP_B_GAUSS);
        if ((base != QP_B_MAD && base != QP_B_MEAN_ABS) || ((bmode & QP_B_GAUSS) && base != QP_B_MAD))
            return qp_fail(ctx, QP_ERR_INVALID_ARG, "bmode");
    }
    if (steps < 1 || steps > QP_CH_MAX_STEPS) return qp_fail(ctx, QP_ERR_INVALID_ARG, "steps must be 1..QP_CH_MAX_STEPS");
    if (hist_bins < 1 || hist_bins > QP_CH_MAX_HIST_BINS)
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "hist_bins must be 1..QP_CH_MAX_HIST_BINS");
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const double F = qp_host_aciq_F(bits, (bmode & QP_B_GAUSS) ? QP_DIST_GAUSS : QP_DIST_LAPLACE);
    if (dtype == QP_F32)
        return search_channels_typed<float>(ctx, static_cast<const float*>(d_x), rows, channels, d_stats, bits, bmode, steps,
                                            hist_bins, F, d_out, d_qp_out, s);
    return search_channels_typed<unsigned short>(ctx, static_cast<const unsigned short*>(d_x), rows, channels, d_stats, bits,
                                                 bmode, steps, hist_bins, F, d_out, d_qp_out, s);
}

extern "C" int32_t qp_dsaciq_curve_channels(qp_ctx* ctx, uint32_t channel, double* h_curve, int capacity, void* stream)
{
    if (!ctx || !h_curve) return QP_ERR_INVALID_ARG;
    if (ctx->ch_last_steps < 1 || !ctx->d_ch_search) return qp_fail(ctx, QP_ERR_INVALID_ARG, "no channel search has run on this context");
    if (channel >= ctx->ch_last_channels) return qp_fail(ctx, QP_ERR_INVALID_ARG, "channel out of range");
    if (capacity < ctx->ch_last_steps + 1) return qp_fail(ctx, QP_ERR_BUFFER_TOO_SMALL, "curve buffer");
    qp_device_guard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const double* src = reinterpret_cast<const double*>(static_cast<char*>(ctx->d_ch_search) + ctx->ch_curve_offset) +
                        (size_t)channel * ctx->ch_last_ncp;
    cudaError_t e = cudaMemcpyAsync(h_curve, src, sizeof(double) * (ctx->ch_last_steps + 1), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return qp_fail(ctx, QP_ERR_CUDA, "copying the curve");
    }
    return QP_OK;
}

extern "C" int32_t qp_dsaciq_candidates_channels(qp_ctx* ctx, qp_qparams_t* h_out, uint64_t capacity, void* stream)
{
    if (!ctx || !h_out) return QP_ERR_INVALID_ARG;
    if (ctx->ch_last_steps < 1 || !ctx->d_ch_search) return qp_fail(ctx, QP_ERR_INVALID_ARG, "no channel search has run on this context");
    const int ncand = ctx->ch_last_steps + 1, ncp = ctx->ch_last_ncp;
    const uint32_t C = ctx->ch_last_channels;
    if (capacity < (uint64_t)C * ncand) return qp_fail(ctx, QP_ERR_BUFFER_TOO_SMALL, "candidate buffer");
    qp_device_guard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t count = (size_t)C * ncp;
    float4* tmp = static_cast<float4*>(malloc(sizeof(float4) * count));
    if (!tmp) return qp_fail(ctx, QP_ERR_CUDA, "out of host memory");
    cudaError_t e = cudaMemcpyAsync(tmp, static_cast<char*>(ctx->d_ch_search) + ctx->ch_cand_offset, sizeof(float4) * count,
                                    cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        free(tmp);
        cudaGetLastError();
        return qp_fail(ctx, QP_ERR_CUDA, "copying the candidates");
    }
    for (uint32_t c = 0; c < C; ++c)
        for (int k = 0; k < ncand; ++k) {
            const float4 q = tmp[(size_t)c * ncp + k];
            qp_qparams_t& o = h_out[(size_t)c * ncand + k];
            o.lo = q.x; o.hi = q.y; o.scale = q.z; o.inv_scale = q.w;
            o.bits = ctx->ch_last_bits;
            o.flags = q.y > q.x ? 0 : 1;
        }
    free(tmp);
    return QP_OK;
}
