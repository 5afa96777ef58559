// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "quantpipe.h"

// ------------------------------------------------------------------ context

constexpr int QP_THREADS = 256;          // block size of the streaming kernels
constexpr int QP_MAX_BLOCKS = 4096;      // upper bound on blocks that write partials
constexpr int QP_EVAL_K = 8;             // candidates scored per thread in one pass

struct qp_stats_partial {                // one per block, written by the two statistics passes
    double s0, s1;                       // pass A: sum x, sum |x|;  pass B: sum |x-mean|, sum (x-mean)^2
    double mn, mx;
    unsigned long long bad;
    unsigned long long pad;
};

struct qp_ds_setup {                     // written by the search's set-up kernel
    double b_e, b_r, F, mean;
    unsigned long long n_finite;
    int degenerate;
    int pad;
    // interval-moment path: the grid that covers every candidate's clip range
    float g_lo, g_hi;                    // min lo_k, max hi_k over the valid candidates
    float inv_gw;                        // QP_IV_CELLS / (g_hi - g_lo), 0 for an empty range
    float inv_u;                         // 1 / u, u = fixed-point unit of offsets inside an interval (a power of two)
    float gw;                            // cell width (g_hi - g_lo) / QP_IV_CELLS
    float pad2;
    double u;
};

constexpr int QP_IV_CELLS = 2048;        // uniform cells over [g_lo, g_hi]
constexpr int QP_IV_MAXB = 4096;         // most interval boundaries (candidate thresholds + cell edges)
constexpr int QP_IV_THREADS = 512;
constexpr int QP_IV_BLOCKS_PER_SM = 3;

struct qp_iv_total { unsigned long long n, s1; };       // per interval: count, sum of offsets (fixed point)

// One instantiated graph of a multi-kernel call, keyed by every argument that the kernels bake in.
constexpr int QP_GRAPH_KEY_WORDS = 12;
struct qp_graph_entry {
    unsigned long long key[QP_GRAPH_KEY_WORDS];
    cudaGraphExec_t exec;
    unsigned launches;                   // kernels inside the graph
    int32_t rc;                          // status the recorded call returned (QP_OK or a warning)
    unsigned long long used;
};
#define QP_GRAPH_SLOTS 64

struct qp_ctx {
    int device;
    int sm_count;
    void* d_base;                        // single allocation, carved below
    qp_stats_partial* d_part;            // [QP_MAX_BLOCKS]
    unsigned long long* d_hist;          // [QP_MAX_HIST_BINS]
    float4* d_cand;                      // [QP_MAX_STEPS + 1]  (lo, hi, scale, inv_scale)
    int* d_valid;                        // [QP_MAX_STEPS + 1]
    double* d_sums;                      // [QP_MAX_BLOCKS * QP_EVAL_K] block partial error sums
    double* d_curve;                     // [QP_MAX_STEPS + 1]  MSE per candidate
    qp_ds_setup* d_setup;
    unsigned int* d_ticket;              // [4] last-block tickets (always left at 0)
    unsigned int* d_status;              // device status word
    float* d_iv_bnd;                     // [QP_IV_MAXB] unsorted boundaries
    float* d_iv_bb;                      // [QP_IV_MAXB + 1] g_lo followed by the sorted boundaries
    float* d_iv_edges;                   // [QP_IV_CELLS + 1] left edge of every cell
    unsigned* d_iv_first;                // [c], c = 0..G+1: boundaries <= left edge of cell c; [G + 2]: finite boundaries m
    unsigned long long* d_iv_part;       // [blocks][QP_IV_MAXB + 1] per-block count << 40 | sum of offsets
    double* d_iv_outer;                  // [blocks + 1][8] per-block sums that need no interval, then their totals
    qp_iv_total* d_iv_tot;               // [QP_IV_MAXB + 1]
    int iv_blocks;                       // blocks of the interval-moment kernel (fixed per context)
    int search_path;                     // 0 auto, 1 candidate scoring, 2 interval moments
    int moments_form;                    // interval moments: 0 auto (second form where it applies), 1 always the first form
    int sender_path;                     // 0 auto, 1 kernel chain, 2 single cooperative launch where it applies
    int stats_path;                      // 0 auto, 1 two kernels, 2 one cooperative launch where it applies
    int fused_checked, fused_ok;         // whether this device can hold the cooperative sender's grid
    int stats_fused_checked, stats_fused_ok;   // the same for the one-launch statistics
    long long wait_cycles;               // limit of a wait for a tile copy (clock cycles)
    unsigned spin_limit;                 // limit of a grid-barrier wait (polls)
    int bar_extra;                       // test only: arrivals a grid barrier waits for beyond the grid size
    size_t fused_dyn_max;                // largest slice (bytes of dynamic shared memory) per block
    void* d_fused;                       // scratch of the cooperative kernels (QP_FUSED_BYTES, see below)
    void* d_ch_part;                     // channel-wise statistics: block partials, allocated on first use
    size_t ch_part_bytes;
    void* d_ch_search;                   // channel-wise search: histograms, candidates, partials, curves; on first use
    size_t ch_search_bytes;
    int ch_last_steps, ch_last_ncp;      // of the last channel-wise search (for qp_dsaciq_curve_channels)
    uint32_t ch_last_channels;
    size_t ch_curve_offset;
    size_t ch_cand_offset;               // candidates of the last channel-wise search inside d_ch_search
    int ch_last_bits;
    void* d_ch_stats;                    // channel-wise sender: statistics when the caller wants none back
    size_t ch_stats_bytes;
    qp_stats_t* d_tmp_stats;             // statistics / quantizer of the host-buffer entry points
    qp_qparams_t* d_tmp_qp;
    unsigned long long launches;         // kernels launched through this context (host count)
    int graphs_on;                       // replay repeated multi-kernel calls as CUDA graphs (qp_set_graph_replay)
    int n_graphs;
    unsigned long long graph_clock;      // use counter for least-recently-used eviction
    unsigned long long graph_hits;       // calls served by replaying a stored graph
    qp_graph_entry graphs[QP_GRAPH_SLOTS];
    int last_steps;                      // steps of the last search (for qp_dsaciq_curve)
    int last_bits;                       // its bit-width (for qp_dsaciq_candidates)
    const void* last_x;                  // tensor of the last full pass on this context and where that pass
    int last_x_end;                      // stopped (1 = at the end of the tensor): the next pass starts there (L2)
    char err[256];
};

// Scratch of the cooperative kernels (d_fused): 256 bytes of barrier counters and the whole-sender
// kernel's histogram (4096 x 8 bytes).
constexpr size_t QP_FUSED_BYTES = 256 + sizeof(unsigned long long) * 4096;

constexpr long long QP_WAIT_CYCLES_DEFAULT = 4000000000ll;   // about two seconds
constexpr unsigned QP_SPIN_LIMIT_DEFAULT = 1u << 22;          // x 64 ns sleeps: a quarter of a second at least

int32_t qp_fail(qp_ctx* ctx, int32_t status, const char* what);
int32_t qp_check_launch(qp_ctx* ctx, const char* what);

struct qp_device_guard {                 // makes ctx->device current for the scope
    int prev;
    bool ok;
    explicit qp_device_guard(int dev) : prev(-1), ok(true)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~qp_device_guard() { if (prev >= 0) cudaSetDevice(prev); }
};

// Shared host arithmetic (one definition each, in qp_api.cu).
double qp_host_aciq_F(int bits, int dist);
static inline bool qp_bits_ok(int bits) { return (bits >= 1 && bits <= 8) || bits == 16; }
bool qp_clip_method_closed_form(int method);     // ACIQ (| INTERSECT) or MINMAX, optionally | MIDRISE

// ------------------------------------------------------------- device helpers
#ifdef __CUDACC__

// Index checks of the debug build (-DQP_CHECK_BOUNDS; python -m paper_2211_04515_b200.build --check).
// QP_CK(i, n) is `i` in the ordinary build.  In the debug build an index outside [0, n) is replaced by
// 0, so the access stays inside its table, and a flag of the translation unit is raised, which
// qp_get_status reports as QP_DEV_INDEX_RANGE: nothing traps and nothing faults.  Every translation
// unit that uses QP_CK says QP_CK_UNIT once at file scope (it registers the unit's flag with the host).
#ifdef QP_CHECK_BOUNDS
static __device__ unsigned qp_ck_flag;
template <typename I, typename N>
__device__ __forceinline__ I qp_ck(I i, N n)
{
    if ((unsigned long long)(long long)i >= (unsigned long long)(long long)n) {
        atomicOr(&qp_ck_flag, 1u);
        return (I)0;
    }
    return i;
}
#define QP_CK(i, n) qp_ck((i), (n))
struct qp_ck_unit { qp_ck_unit* next; unsigned (*read_and_clear)(); };
void qp_ck_register(qp_ck_unit* u);
#define QP_CK_UNIT                                                                                          \
    static unsigned qp_ck_read_and_clear()                                                                  \
    {                                                                                                       \
        unsigned v = 0, z = 0;                                                                              \
        if (cudaMemcpyFromSymbol(&v, qp_ck_flag, sizeof v) != cudaSuccess) { cudaGetLastError(); return 0; } \
        if (v) cudaMemcpyToSymbol(qp_ck_flag, &z, sizeof z);                                                \
        return v;                                                                                           \
    }                                                                                                       \
    static qp_ck_unit qp_ck_this_unit = {nullptr, qp_ck_read_and_clear};                                    \
    static const int qp_ck_registered = (qp_ck_register(&qp_ck_this_unit), 0);
#else
#define QP_CK(i, n) (i)
#define QP_CK_UNIT
#endif

// Quantizer set-up from a clip range, same on host and device: ends rounded to fp32, scale
// and reciprocal from the rounded ends in fp64, rounded once.
__host__ __device__ inline int qp_fill_qparams(double lo, double hi, int bits, qp_qparams_t* q)
{
    const double levels_m1 = (double)((1u << bits) - 1u);
    const float lo_f = (float)lo, hi_f = (float)hi;
    q->lo = lo_f;
    q->hi = hi_f;
    q->bits = bits;
    q->flags = 0;
    const bool finite = (lo_f - lo_f == 0.0f) && (hi_f - hi_f == 0.0f);
    if (!(hi_f > lo_f) || !finite) {
        q->scale = 0.0f;
        q->inv_scale = 0.0f;
        q->flags = 1;
        return QP_WARN_DEGENERATE;
    }
    const double range = (double)hi_f - (double)lo_f;
    q->scale = (float)(range / levels_m1);
    q->inv_scale = (float)(levels_m1 / range);
    return QP_OK;
}

constexpr float QP_MAGIC = 12582912.0f;         // 1.5 * 2^23: adding it rounds to an integer, ties to even
constexpr unsigned QP_MAGIC_BITS = 0x4B400000u;

// Position of x on the level grid: clamp (NaN -> lo), subtract, scale; each op rounded to fp32.
__device__ __forceinline__ float qp_grid_pos(float x, float lo, float hi, float inv_scale)
{
    const float t = fminf(fmaxf(x, lo), hi);
    return __fmul_rn(__fsub_rn(t, lo), inv_scale);
}

// Code of x as the low bits of (pos + 1.5*2^23): for 0 <= pos < 2^22 the float addition
// rounds pos to the nearest integer, ties to even, and leaves it in the low mantissa bits.
__device__ __forceinline__ unsigned qp_code(float x, float lo, float hi, float inv_scale, unsigned mask)
{
    return __float_as_uint(__fadd_rn(qp_grid_pos(x, lo, hi, inv_scale), QP_MAGIC)) & mask;
}

// monotone map float -> uint32 (finite values; -0 sorts directly below +0), and back
__device__ __forceinline__ unsigned qp_key_of(float x)
{
    const unsigned u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float qp_float_of(unsigned k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// smallest float in (lo_x, hi_x] for which pred holds, given !pred(lo_x) and pred(hi_x), pred monotone:
// bisection over the floats' bit patterns (at most 32 evaluations of pred)
template <typename P>
__device__ __forceinline__ float qp_first_true(float lo_x, float hi_x, P pred)
{
    unsigned lo = qp_key_of(lo_x), hi = qp_key_of(hi_x);
    while (hi - lo > 1u) {
        const unsigned mid = lo + ((hi - lo) >> 1);
        if (pred(qp_float_of(mid))) hi = mid; else lo = mid;
    }
    return qp_float_of(hi);
}

__device__ __forceinline__ float qp_bf16_to_f32(unsigned short h) { return __uint_as_float((unsigned)h << 16); }

__device__ __forceinline__ unsigned short qp_f32_to_bf16(float f)   // round to nearest even
{
    unsigned u = __float_as_uint(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (unsigned short)((u >> 16) | 0x0040u);
    return (unsigned short)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}

__device__ __forceinline__ bool qp_is_finite(float x) { return fabsf(x) < __int_as_float(0x7F800000); }

// A contiguous array seen as [head scalars][nvec aligned 16-byte vectors][tail scalars].
template <typename T>
struct qp_span {
    uint64_t head, nvec, tail;
    static constexpr int EPV = 16 / sizeof(T);
    __host__ __device__ qp_span(const T* p, uint64_t n)
    {
        const uint64_t mis = ((uintptr_t)p & 15u) / sizeof(T);
        head = mis ? (EPV - mis) : 0;
        if (head > n) head = n;
        nvec = (n - head) / EPV;
        tail = n - head - nvec * EPV;
    }
};

// Load one 16-byte vector of T as EPV floats.
__device__ __forceinline__ void qp_load_vec(const float* p, float (&v)[4])
{
    const float4 a = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
}
__device__ __forceinline__ void qp_load_vec(const unsigned short* p, float (&v)[8])
{
    const uint4 a = __ldg(reinterpret_cast<const uint4*>(p));
    v[0] = __uint_as_float(a.x << 16); v[1] = __uint_as_float(a.x & 0xFFFF0000u);
    v[2] = __uint_as_float(a.y << 16); v[3] = __uint_as_float(a.y & 0xFFFF0000u);
    v[4] = __uint_as_float(a.z << 16); v[5] = __uint_as_float(a.z & 0xFFFF0000u);
    v[6] = __uint_as_float(a.w << 16); v[7] = __uint_as_float(a.w & 0xFFFF0000u);
}
__device__ __forceinline__ float qp_load_one(const float* p) { return __ldg(p); }
__device__ __forceinline__ float qp_load_one(const unsigned short* p) { return qp_bf16_to_f32(__ldg(p)); }

// Deterministic block-wide sum of a double (result valid in thread 0).  `sh` holds one
// double per warp.
__device__ __forceinline__ double qp_block_sum(double v, double* sh)
{
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
    __syncthreads();
    if (lane == 0) sh[warp] = v;
    __syncthreads();
    double r = 0.0;
    if (threadIdx.x == 0)
        for (int w = 0; w < nwarp; ++w) r += sh[w];
    return r;
}
__device__ __forceinline__ double qp_block_min(double v, double* sh)
{
    for (int o = 16; o > 0; o >>= 1) v = fmin(v, __shfl_down_sync(0xFFFFFFFFu, v, o));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
    __syncthreads();
    if (lane == 0) sh[warp] = v;
    __syncthreads();
    double r = v;
    if (threadIdx.x == 0)
        for (int w = 0; w < nwarp; ++w) r = fmin(r, sh[w]);
    return r;
}
__device__ __forceinline__ double qp_block_max(double v, double* sh)
{
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_down_sync(0xFFFFFFFFu, v, o));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
    __syncthreads();
    if (lane == 0) sh[warp] = v;
    __syncthreads();
    double r = v;
    if (threadIdx.x == 0)
        for (int w = 0; w < nwarp; ++w) r = fmax(r, sh[w]);
    return r;
}

// Mid-rise grid on a clip range: 2^bits equal bins over [lo, hi], reconstruction at the bin
// centres.  The centres are the 2^bits levels of the uniform quantizer on the range pulled in
// by half a bin on each side, and its rounding boundaries are the bin edges, so the grid is a
// change of the clip range and nothing else.
__host__ __device__ inline void qp_midrise_ends(int bits, double& lo, double& hi)
{
    const double half = (hi - lo) / (double)(2ull << bits);
    lo += half;
    hi -= half;
}

// Closed-form clip range from the statistics: ACIQ (optionally cut back to [min, max]) or the
// tensor's own range, optionally on the mid-rise grid; same on host and device.
__host__ __device__ inline void qp_clip_ends(const qp_stats_t& st, int method, int dist, int bmode, int bits, double F,
                                             double& lo, double& hi)
{
    if ((method & 0xF) == QP_CLIP_MINMAX) {
        lo = st.min;
        hi = st.max;
    } else {
        const double b = dist == QP_DIST_GAUSS ? sqrt(st.var) : (bmode == QP_B_MEAN_ABS ? st.mean_abs : st.mad);
        const double alpha = F * b;
        lo = st.mean - alpha;
        hi = st.mean + alpha;
        if (method & QP_CLIP_INTERSECT) {
            if (st.min > lo) lo = st.min;
            if (st.max < hi) hi = st.max;
        }
    }
    if (method & QP_CLIP_MIDRISE) qp_midrise_ends(bits, lo, hi);
}

// ---- pieces of the directed search shared by its two scoring paths

// b_E, b_R and friends from the statistics and the histogram's peak count `top`
__device__ inline void qp_ds_make_setup(const qp_stats_t* __restrict__ st, unsigned long long top, int nb, int bmode,
                                        double F, qp_ds_setup& s)
{
    const unsigned long long nf = st->n - st->nonfinite;
    const double mn = st->min, mx = st->max;
    const bool gauss = (bmode & QP_B_GAUSS) != 0;       // normal model: scale = standard deviation
    const double b_e = gauss ? sqrt(st->var) : ((bmode & 0xF) == QP_B_MEAN_ABS ? st->mean_abs : st->mad);
    double peak = 0.0;
    if (mx > mn && nf > 0) {
        const double w = (mx - mn) / (double)nb;
        peak = (double)top / ((double)nf * w);
    }
    s.degenerate = !(mx > mn) || !(peak > 0.0) || !(b_e > 0.0);
    s.b_e = b_e;
    // the model's density peaks at 1 / (factor * scale): factor 2 (Laplace) or sqrt(2 pi) (normal)
    s.b_r = s.degenerate ? b_e : 1.0 / ((gauss ? 2.5066282746310002 : 2.0) * peak);
    s.F = F;
    s.mean = st->mean;
    s.n_finite = nf;
    s.pad = 0;
}

// candidate k: b_k = b_E + k (b_R - b_E) / steps, evaluated in this order in fp64; its quantizer
// (midrise != 0: on the mid-rise grid)
__device__ inline void qp_ds_candidate(const qp_ds_setup& s, int k, int steps, int bits, int midrise, float4& c, int& ok)
{
    const double b_k = s.b_e + (double)k * (s.b_r - s.b_e) / (double)steps;
    ok = ((k == 0) || (!s.degenerate && b_k > 0.0)) ? 1 : 0;
    qp_qparams_t q;
    q.lo = q.hi = q.scale = q.inv_scale = 0.f;
    if (ok) {
        const double alpha = s.F * b_k;
        double lo = s.mean - alpha, hi = s.mean + alpha;
        if (midrise) qp_midrise_ends(bits, lo, hi);
        qp_fill_qparams(lo, hi, bits, &q);
    }
    c = make_float4(q.lo, q.hi, q.scale, q.inv_scale);
}

// One thread: the search's result record and the winning quantizer for the chosen step `best`.
__device__ inline void qp_ds_write_result(int best, const double* s_curve, const qp_ds_setup& s, int steps, int nb, int bits,
                                          float4 c, qp_ds_result_t* __restrict__ out, qp_qparams_t* __restrict__ qp_out,
                                          unsigned* __restrict__ status)
{
    const double b_star = s.b_e + (double)best * (s.b_r - s.b_e) / (double)steps;
    if (out) {
        out->b_e = s.b_e;
        out->b_r = s.b_r;
        out->b_star = b_star;
        out->alpha_e = s.F * s.b_e;
        out->alpha_star = s.F * b_star;
        out->mse_e = s_curve[0];
        out->mse_star = s_curve[best];
        out->k_star = best;
        out->steps = steps;
        out->hist_bins = nb;
        out->bits = bits;
    }
    const bool degenerate_q = !(c.y > c.x);
    if (qp_out) {
        qp_out->lo = c.x; qp_out->hi = c.y; qp_out->scale = c.z; qp_out->inv_scale = c.w;
        qp_out->bits = bits;
        qp_out->flags = degenerate_q ? 1 : 0;
    }
    if (s.degenerate || degenerate_q) atomicOr(status, QP_DEV_DEGENERATE);
}

// Block-wide: first minimum of the MSE curve wins (k = 0 keeps b_E); writes the result and
// the winning quantizer.  s_curve: shared scratch of steps + 1 doubles.
__device__ inline void qp_ds_pick(const double* __restrict__ curve, int steps, int nb, int bits,
                                  const float4* __restrict__ cand, const qp_ds_setup* __restrict__ setup,
                                  qp_ds_result_t* __restrict__ out, qp_qparams_t* __restrict__ qp_out,
                                  unsigned* __restrict__ status, double* s_curve)
{
    for (int k = threadIdx.x; k <= steps; k += blockDim.x) s_curve[k] = __ldcg(&curve[k]);
    __syncthreads();
    if (threadIdx.x != 0) return;
    const qp_ds_setup s = *setup;
    int best = 0;
    double best_mse = s_curve[0];
    for (int k = 1; k <= steps; ++k)
        if (s_curve[k] < best_mse) { best_mse = s_curve[k]; best = k; }
    qp_ds_write_result(best, s_curve, s, steps, nb, bits, __ldcg(&cand[best]), out, qp_out, status);
}

#endif  // __CUDACC__

// Kernel launchers (one per translation unit).
int32_t qp_launch_stats(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int hist_bins, qp_stats_t* d_out,
                        cudaStream_t s);
int32_t qp_launch_search(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, const qp_stats_t* d_stats, int bits,
                         int bmode, int steps, int hist_bins, double F, qp_ds_result_t* d_out,
                         qp_qparams_t* d_qp_out, cudaStream_t s);
// channel-wise search through interval moments (qp_channels_search_fast.cu)
size_t qp_channel_interval_scratch_bytes(uint32_t C, int nthr);
bool qp_channel_interval_applies(uint64_t rows, int bits, int steps);
int32_t qp_launch_channel_interval_sums(qp_ctx* ctx, const void* d_x, int dtype, uint64_t rows, uint32_t C, int bits, int steps,
                                        int ncp, const qp_stats_t* d_stats, const float4* cand, const int* valid,
                                        qp_ds_setup* setup, char* scratch, double* part, cudaStream_t s);
int32_t qp_launch_interval_search(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, const qp_stats_t* d_stats,
                                  int bits, int bmode, int steps, int hist_bins, double F, qp_ds_result_t* d_out,
                                  qp_qparams_t* d_qp_out, cudaStream_t s);
bool qp_sender_fused_applies(uint64_t n, int use_ds, int steps, int hist_bins, bool forced);
int32_t qp_launch_sender_fused(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int bits, int method, int bmode,
                               int steps, int hist_bins, double F, void* d_packed, qp_qparams_t* d_qp_out,
                               qp_stats_t* d_stats_out, cudaStream_t s);
int32_t qp_launch_aciq_device(qp_ctx* ctx, const qp_stats_t* d_stats, int bits, int method, int dist, int bmode, double F,
                              qp_qparams_t* d_qp_out, cudaStream_t s);
int32_t qp_launch_pack(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int bits, const qp_qparams_t* d_qp,
                       qp_qparams_t h_qp, void* d_packed, cudaStream_t s);
int32_t qp_launch_unpack(qp_ctx* ctx, const void* d_packed, uint64_t n, int bits, const qp_qparams_t* d_qp,
                         qp_qparams_t h_qp, void* d_y, int out_dtype, cudaStream_t s);
