// The whole sender (paper Sec. 3: statistics -> ACIQ clip or directed search -> uniform
// quantization) for small tensors in ONE cooperative launch.
//
// At the sizes of a small micro-batch the kernel chain of the separate calls is bound by
// launches, not by data: 4 to 10 kernels of a few microseconds each.  Here every SM takes a
// slice of x into shared memory once, and the steps that need a tensor-wide result (mean
// before the deviations; statistics and histogram peak before the candidates; the error
// curve before the winner) are separated by grid barriers instead of kernel boundaries.
// x is read from global memory exactly once and every later step works on the resident
// slice.
//
//   phase 0   slice -> shared memory; sum x, sum |x|, min, max, non-finite count
//   barrier   every block merges all block partials in index order (all get the same bits)
//   phase 1   sum |x - mean|, sum (x - mean)^2; histogram over [min, max] (search only)
//   barrier
//   phase 2   statistics; ACIQ clip, or: histogram peak -> b_R, candidates, squared error of
//             every candidate over the slice (each element quantized under each candidate)
//   barrier   (search only)
//   phase 3   error curve, first minimum wins
//   phase 4   quantize + pack the slice, 32 elements (= `bits` words) per thread
//
// The grid barrier is an arrival counter in global memory; blocks are co-resident because
// the launch is cooperative, and the wait is bounded all the same: a block that gives up
// sets QP_DEV_STREAM_TIMEOUT in the status word and leaves.
#include "qp_gridbar.cuh"
#include "qp_internal.cuh"

QP_CK_UNIT

namespace {

constexpr int FS_THREADS = 512;
constexpr int FS_WARPS = FS_THREADS / 32;
constexpr int FS_MAX_STEPS = 127;                 // candidates fit the per-block tables
constexpr int FS_MAX_BINS = 4096;
constexpr uint64_t FS_MAX_N_SEARCH = 1ull << 20;  // above this the per-candidate scoring stops paying
constexpr uint64_t FS_AUTO_N = 1ull << 21;
constexpr uint64_t FS_MAX_N = 6500000;            // slices of 148 SMs x ~190 KB of shared memory (checked per device)
constexpr int FS_PART = 8;                        // doubles per block partial
constexpr int K = QP_EVAL_K;

struct FsArgs {
    const void* x;
    uint64_t n;
    int bits, use_ds, method, bmode, steps, nb;         // use_ds: method is the directed search
    double F;
    uint32_t* out;
    uint64_t total_words;
    unsigned groups_per_block;                    // 32-element groups per block
    qp_qparams_t* qp_out;
    qp_stats_t* st_out;
    qp_ds_result_t* ds_out;                       // optional
    double* part;                                 // [grid][FS_PART]
    unsigned long long* hist;                     // [nb], zero at entry
    double* sums;                                 // [grid][FS_MAX_STEPS + 1]
    double* curve;                                // [steps + 1]
    float4* cand;                                 // [steps + 1]
    qp_ds_setup* setup;
    unsigned* bar;                                // arrival counter, zero at entry
    unsigned* status;
    unsigned spin_limit;                          // polls a grid-barrier wait may take
    unsigned bar_extra;                           // 0; a test makes the barriers wait for more arrivals than blocks
};

// Block reduction of N values at once; every thread gets the results, merged in warp order (the
// same bits in every block).  OPS: 0 sum, 1 min, 2 max.  sh: FS_WARPS * N doubles.
template <int... OPS>
__device__ __forceinline__ void fs_reduce(double (&v)[sizeof...(OPS)], double* sh)
{
    constexpr int N = sizeof...(OPS);
    constexpr int ops[N] = {OPS...};
#pragma unroll
    for (int j = 0; j < N; ++j)
        for (int o = 16; o > 0; o >>= 1) {
            const double t = __shfl_down_sync(0xFFFFFFFFu, v[j], o);
            v[j] = ops[j] == 0 ? v[j] + t : (ops[j] == 1 ? fmin(v[j], t) : fmax(v[j], t));
        }
    __syncthreads();                               // sh may still be read from the reduction before
    if ((threadIdx.x & 31) == 0)
#pragma unroll
        for (int j = 0; j < N; ++j) sh[(threadIdx.x >> 5) * N + j] = v[j];
    __syncthreads();
#pragma unroll
    for (int j = 0; j < N; ++j) {
        double r = sh[j];
        for (int w = 1; w < FS_WARPS; ++w) {
            const double t = sh[w * N + j];
            r = ops[j] == 0 ? r + t : (ops[j] == 1 ? fmin(r, t) : fmax(r, t));
        }
        v[j] = r;
    }
}

template <typename T>
__global__ void __launch_bounds__(FS_THREADS, 1) sender_fused_kernel(const FsArgs a)
{
    extern __shared__ __align__(16) float xs[];   // this block's slice of x: element i at i + (i >> 5), rows of 33 words
    __shared__ double s_red[FS_WARPS * 5];
    __shared__ int s_ok;
    // histogram counters in phase 1; per-thread candidate error sums in phase 2
    __shared__ __align__(16) unsigned char s_union[FS_THREADS * K * sizeof(double)];
    __shared__ float4 s_cand[FS_MAX_STEPS + 1];
    __shared__ int s_valid[FS_MAX_STEPS + 1];
    __shared__ double s_curve[FS_MAX_STEPS + 1];
    __shared__ qp_stats_t s_st;
    __shared__ qp_ds_setup s_setup;
    __shared__ qp_qparams_t s_qp;
    __shared__ int s_best;
    unsigned* s_hist = reinterpret_cast<unsigned*>(s_union);                 // [FS_MAX_BINS]
    double (*s_acc)[K] = reinterpret_cast<double (*)[K]>(s_union);           // [FS_THREADS][K]
    static_assert(sizeof(s_union) >= FS_MAX_BINS * sizeof(unsigned), "histogram fits the union");

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned G = gridDim.x;
    const double inf = __longlong_as_double(0x7FF0000000000000ll);

    // ---- phase 0: slice into shared memory, first moments
    const uint64_t g0 = (uint64_t)blockIdx.x * a.groups_per_block;
    const uint64_t e0 = g0 * 32;
    const int cap = (int)a.groups_per_block * 32;
    const int cnt = e0 < a.n ? (int)(a.n - e0 < (uint64_t)cap ? a.n - e0 : (uint64_t)cap) : 0;
    {
        const T* x = static_cast<const T*>(a.x);
        double v5[5] = {0.0, 0.0, inf, -inf, 0.0};            // sum, sum |x|, min, max, non-finite
        auto one = [&](float v) {                             // element by element: skips and counts NaN/Inf
            if (qp_is_finite(v)) {
                v5[0] += (double)v;
                v5[1] += (double)fabsf(v);
                v5[2] = fmin(v5[2], (double)v);
                v5[3] = fmax(v5[3], (double)v);
            } else {
                v5[4] += 1.0;
            }
        };
        constexpr int EPV = qp_span<T>::EPV;
        const T* xb = x + e0;
        const float finf = __int_as_float(0x7F800000);
        // 16-byte loads where the slice is aligned (its start is a multiple of 32 elements from x),
        // four in flight per thread; fp32 partial sums over one vector, folded into fp64
        const int nvec = (((uintptr_t)xb & 15u) == 0) ? cnt / EPV : 0;
        for (int v0 = tid; v0 < nvec; v0 += 4 * FS_THREADS) {
            float e[4][EPV];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int v = v0 + u * FS_THREADS;
                if (v < nvec) qp_load_vec(xb + (size_t)v * EPV, e[u]);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int v = v0 + u * FS_THREADS;
                if (v >= nvec) break;
                const int i0 = v * EPV;                       // EPV consecutive elements stay inside one 32-element row
                float* dst = xs + QP_CK(i0 + (i0 >> 5), (int)a.groups_per_block * 33 - (EPV - 1));
                float ps = 0.f, psa = 0.f, pmn = finf, pmx = -finf;
#pragma unroll
                for (int i = 0; i < EPV; ++i) {
                    const float val = e[u][i];
                    dst[i] = val;
                    ps += val;
                    psa += fabsf(val);
                    pmn = fminf(pmn, val);
                    pmx = fmaxf(pmx, val);
                }
                if (psa < finf) {                             // every element finite (and no fp32 overflow)
                    v5[0] += (double)ps;
                    v5[1] += (double)psa;
                    v5[2] = fmin(v5[2], (double)pmn);
                    v5[3] = fmax(v5[3], (double)pmx);
                } else {
#pragma unroll
                    for (int i = 0; i < EPV; ++i) one(e[u][i]);
                }
            }
        }
        for (int i = nvec * EPV + tid; i < cnt; i += FS_THREADS) {   // unaligned slice, ragged end
            const float v = qp_load_one(xb + i);
            xs[QP_CK(i + (i >> 5), (int)a.groups_per_block * 33)] = v;
            one(v);
        }
        fs_reduce<0, 0, 1, 2, 0>(v5, s_red);
        if (tid == 0) {
            double* p = a.part + (size_t)blockIdx.x * FS_PART;
            p[0] = v5[0]; p[1] = v5[1]; p[2] = v5[2]; p[3] = v5[3]; p[4] = v5[4];
        }
    }
    if (!qp_grid::barrier(a.bar, G + a.bar_extra, a.spin_limit, a.status, &s_ok)) return;

    // ---- phase 1: tensor-wide first moments (same in every block), then deviations and histogram
    double mean, mean_abs, mn_all, mx_all;
    unsigned long long nbad, nf;
    {
        double v5[5] = {0.0, 0.0, inf, -inf, 0.0};
        for (unsigned b = tid; b < G; b += FS_THREADS) {
            const double* p = a.part + (size_t)b * FS_PART;
            v5[0] += __ldcg(p + 0);
            v5[1] += __ldcg(p + 1);
            v5[2] = fmin(v5[2], __ldcg(p + 2));
            v5[3] = fmax(v5[3], __ldcg(p + 3));
            v5[4] += __ldcg(p + 4);                            // exact: counts are far below 2^53
        }
        fs_reduce<0, 0, 1, 2, 0>(v5, s_red);
        nbad = (unsigned long long)v5[4];
        nf = a.n - nbad;
        mean = nf ? v5[0] / (double)nf : 0.0;
        mean_abs = nf ? v5[1] / (double)nf : 0.0;
        mn_all = nf ? v5[2] : 0.0;
        mx_all = nf ? v5[3] : 0.0;
    }
    const bool want_hist = a.use_ds && mx_all > mn_all;
    if (want_hist)
        for (int b = tid; b < a.nb; b += FS_THREADS) s_hist[b] = 0u;
    __syncthreads();
    {
        // x - mean with the mean held as an unevaluated fp32 pair
        const float m_hi = (float)mean;
        const float m_lo = (float)(mean - (double)m_hi);
        const float h_mn = (float)mn_all;
        const float inv_w = want_hist ? (float)((double)a.nb / (mx_all - mn_all)) : 0.f;
        double v2[2] = {0.0, 0.0};
        for (int i0 = tid; i0 < cnt; i0 += 8 * FS_THREADS) {  // fp32 sums over 8 elements, then fp64
            float d1 = 0.f, d2 = 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = i0 + u * FS_THREADS;
                if (i >= cnt) break;
                const float v = xs[i + (i >> 5)];
                if (!qp_is_finite(v)) continue;
                const float d = __fsub_rn(__fsub_rn(v, m_hi), m_lo);
                d1 += fabsf(d);
                d2 = fmaf(d, d, d2);
                if (want_hist) {
                    // bin = floor((x - min) * inv_w), the last bin closed; fp32, each op rounded once
                    int b = __float2int_rz(__fmul_rn(__fsub_rn(v, h_mn), inv_w));
                    b = min(max(b, 0), a.nb - 1);
                    atomicAdd(&s_hist[QP_CK(b, FS_MAX_BINS)], 1u);
                }
            }
            v2[0] += (double)d1;
            v2[1] += (double)d2;
        }
        fs_reduce<0, 0>(v2, s_red);                            // (its barriers also order the shared atomics)
        if (tid == 0) {
            a.part[(size_t)blockIdx.x * FS_PART + 5] = v2[0];
            a.part[(size_t)blockIdx.x * FS_PART + 6] = v2[1];
        }
        if (want_hist)
            for (int b = tid; b < a.nb; b += FS_THREADS) {
                const unsigned c = s_hist[b];
                if (c) atomicAdd(&a.hist[b], (unsigned long long)c);
            }
    }
    if (!qp_grid::barrier(a.bar, 2 * G + a.bar_extra, a.spin_limit, a.status, &s_ok)) return;

    // ---- phase 2: statistics, then the clip range
    {
        double v3[3] = {0.0, 0.0, 0.0};                        // sum |x-mean|, sum (x-mean)^2, histogram peak
        for (unsigned b = tid; b < G; b += FS_THREADS) {
            const double* p = a.part + (size_t)b * FS_PART;
            v3[0] += __ldcg(p + 5);
            v3[1] += __ldcg(p + 6);
        }
        if (want_hist)
            for (int b = tid; b < a.nb; b += FS_THREADS) v3[2] = fmax(v3[2], (double)__ldcg(&a.hist[b]));
        fs_reduce<0, 0, 2>(v3, s_red);
        if (tid == 0) {
            s_st.n = a.n;
            s_st.nonfinite = nbad;
            s_st.mean = mean;
            s_st.mean_abs = mean_abs;
            s_st.mad = nf ? v3[0] / (double)nf : 0.0;
            s_st.var = nf ? v3[1] / (double)nf : 0.0;
            s_st.min = mn_all;
            s_st.max = mx_all;
            s_st.hist_peak = a.use_ds ? (unsigned long long)v3[2] : 0ull;
            s_st.hist_bins = a.use_ds ? a.nb : 0;
            s_st.reserved = 0;
            if (blockIdx.x == 0) {
                *a.st_out = s_st;
                if (nbad) atomicOr(a.status, QP_DEV_NONFINITE);
            }
            if (a.use_ds) {
                qp_ds_make_setup(&s_st, (unsigned long long)v3[2], a.nb, a.bmode, a.F, s_setup);
                s_setup.g_lo = s_setup.g_hi = s_setup.inv_gw = s_setup.inv_u = s_setup.gw = s_setup.pad2 = 0.f;
                s_setup.u = 0.0;
            } else {
                double lo, hi;
                qp_clip_ends(s_st, a.method, QP_DIST_LAPLACE, a.bmode, a.bits, a.F, lo, hi);
                const int rc = qp_fill_qparams(lo, hi, a.bits, &s_qp);
                if (blockIdx.x == 0) {
                    *a.qp_out = s_qp;
                    if (rc == QP_WARN_DEGENERATE) atomicOr(a.status, QP_DEV_DEGENERATE);
                }
            }
        }
        __syncthreads();
    }

    if (a.use_ds) {
        const int ncand = a.steps + 1;
        for (int k = tid; k < ncand; k += FS_THREADS) {
            float4 c;
            int ok;
            qp_ds_candidate(s_setup, k, a.steps, a.bits, a.method & QP_CLIP_MIDRISE, c, ok);
            s_cand[k] = c;
            s_valid[k] = ok;
        }
        __syncthreads();
        // Squared error of every candidate over the slice.  Thread t scores the K candidates of
        // group t % groups against the elements i = t / groups (mod lanes_per_group), so all
        // threads are busy whatever the slice length; the K sums stay in registers.
        const int groups = (ncand + K - 1) / K;
        const int per_group = FS_THREADS / groups;             // threads that share one candidate group
        const int g = tid % groups, sub = tid / groups;
        {
            float lo[K], hi[K], sc[K], iv[K];
            double acc[K];
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const float4 q = s_cand[min(g * K + k, ncand - 1)];
                lo[k] = q.x; hi[k] = q.y; sc[k] = q.z; iv[k] = q.w;
                acc[k] = 0.0;
            }
            if (sub < per_group) {
                for (int i0 = sub; i0 < cnt; i0 += 8 * per_group) {
                    float p[K];
#pragma unroll
                    for (int k = 0; k < K; ++k) p[k] = 0.f;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {               // fp32 sums over 8 elements, then fp64
                        const int i = i0 + u * per_group;
                        if (i >= cnt) break;
                        const float v = xs[i + (i >> 5)];
                        if (!qp_is_finite(v)) continue;
#pragma unroll
                        for (int k = 0; k < K; ++k) {
                            // level index as a float: (pos + 1.5*2^23) - 1.5*2^23 rounds to nearest, ties to even
                            const float pos = qp_grid_pos(v, lo[k], hi[k], iv[k]);
                            const float r = __fsub_rn(__fadd_rn(pos, QP_MAGIC), QP_MAGIC);
                            const float d = __fsub_rn(fmaf(r, sc[k], lo[k]), v);
                            p[k] = fmaf(d, d, p[k]);
                        }
                    }
#pragma unroll
                    for (int k = 0; k < K; ++k) acc[k] += (double)p[k];
                }
            }
#pragma unroll
            for (int k = 0; k < K; ++k) s_acc[tid][k] = acc[k];
        }
        __syncthreads();
        for (int c = tid; c < ncand; c += FS_THREADS) {        // this block's sum for candidate c, fixed order
            const int cg = c / K, ck = c % K;
            double t = 0.0;
            for (int j = 0; j < per_group; ++j) t += s_acc[j * groups + cg][ck];
            a.sums[(size_t)blockIdx.x * (FS_MAX_STEPS + 1) + c] = t;
        }
        if (!qp_grid::barrier(a.bar, 3 * G + a.bar_extra, a.spin_limit, a.status, &s_ok)) return;

        // ---- phase 3: error curve, first minimum wins.  The G block sums of a candidate are merged
        // by four threads, each over a quarter of the blocks in index order (loads issued in
        // batches so that they overlap), then the quarters in order: the same bits in every block.
        {
            constexpr int QUARTERS = FS_THREADS / (FS_MAX_STEPS + 1);
            double (*s_q)[FS_MAX_STEPS + 1] = reinterpret_cast<double (*)[FS_MAX_STEPS + 1]>(s_union);
            const int k = tid % (FS_MAX_STEPS + 1), qtr = tid / (FS_MAX_STEPS + 1);
            const unsigned per = (G + QUARTERS - 1) / QUARTERS;
            const unsigned b0 = qtr * per, b1 = min(b0 + per, G);
            double t = 0.0;
            if (k < ncand) {
                for (unsigned b = b0; b < b1; b += 20) {
                    double v[20];
#pragma unroll
                    for (int u = 0; u < 20; ++u)
                        v[u] = b + u < b1 ? __ldcg(&a.sums[(size_t)(b + u) * (FS_MAX_STEPS + 1) + k]) : 0.0;
#pragma unroll
                    for (int u = 0; u < 20; ++u) t += v[u];
                }
            }
            __syncthreads();                                   // s_acc (same storage) has been read by everyone
            s_q[qtr][k] = t;
            __syncthreads();
            if (tid < ncand) {
                double sum = 0.0;
                for (int q = 0; q < QUARTERS; ++q) sum += s_q[q][tid];
                double mse = nf ? sum / (double)nf : 0.0;
                if (!s_valid[tid]) mse = inf;
                s_curve[tid] = mse;
            }
        }
        __syncthreads();
        if (warp == 0) {                                       // smallest value, lowest step among equals
            double bv = inf;
            int bk = FS_MAX_STEPS + 1;
            for (int k = lane; k < ncand; k += 32)
                if (s_curve[k] < bv) { bv = s_curve[k]; bk = k; }
            for (int o = 16; o > 0; o >>= 1) {
                const double ov = __shfl_down_sync(0xFFFFFFFFu, bv, o);
                const int ok = __shfl_down_sync(0xFFFFFFFFu, bk, o);
                if (ov < bv || (ov == bv && ok < bk)) { bv = ov; bk = ok; }
            }
            if (lane == 0) {
                const int best = bk <= a.steps ? bk : 0;        // (every MSE infinite or NaN: keep b_E)
                s_best = best;
                const float4 c = s_cand[best];
                s_qp.lo = c.x; s_qp.hi = c.y; s_qp.scale = c.z; s_qp.inv_scale = c.w;
                s_qp.bits = a.bits;
                s_qp.flags = !(c.y > c.x) ? 1 : 0;
            }
        }
        __syncthreads();
        if (blockIdx.x == 0) {                                 // the search's outputs, as the separate call leaves them
            for (int k = tid; k < ncand; k += FS_THREADS) {
                a.curve[k] = s_curve[k];
                a.cand[k] = s_cand[k];
            }
            if (tid == 0) {
                *a.setup = s_setup;
                qp_ds_write_result(s_best, s_curve, s_setup, a.steps, a.nb, a.bits, s_cand[s_best], a.ds_out, a.qp_out,
                                   a.status);
            }
            for (int b = tid; b < a.nb; b += FS_THREADS) a.hist[b] = 0ull;   // every block has read it: clean for the next call
        }
    }

    // ---- phase 4: quantize + pack.  A thread takes the 32 elements of one group (= `bits` whole
    // words): all loads first, then the codes, then the words through a 64-bit shift register.
    {
        const float lo = s_qp.lo, hi = s_qp.hi, inv = s_qp.inv_scale;
        const int bits = a.bits;
        const unsigned mask = (1u << bits) - 1u;
        for (unsigned j = tid; j < a.groups_per_block; j += FS_THREADS) {
            const uint64_t w0 = (g0 + j) * (uint64_t)bits;
            if (w0 >= a.total_words) break;
            const float* row = xs + j * 33;
            const int have = cnt - (int)j * 32;                // elements of this group that exist
            float e[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) e[i] = row[i];
            unsigned c[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) c[i] = i < have ? qp_code(e[i], lo, hi, inv, mask) : 0u;
            unsigned long long acc = 0ull;
            int fill = 0;
            uint32_t* dst = a.out + w0;
            const uint32_t* end = a.out + a.total_words;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                acc |= (unsigned long long)c[i] << fill;
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

    // ---- leave the arrival counter at zero: the last block out resets it (nobody waits any more)
    __syncthreads();
    if (tid == 0) {
        const unsigned gone = atomicInc(a.bar + 1, G - 1);     // wraps to 0 with the last block
        if (gone == G - 1) atomicExch(a.bar, 0u);
    }
}

}  // namespace

bool qp_sender_fused_applies(uint64_t n, int use_ds, int steps, int hist_bins, bool forced)
{
    // measured against the kernel chain: the single launch wins up to ~2^21 elements with a
    // closed-form clip and up to 2^20 with the search; when forced it runs up to what the
    // shared memory of all SMs holds
    const uint64_t max_n = use_ds ? FS_MAX_N_SEARCH : (forced ? FS_MAX_N : FS_AUTO_N);
    if (n == 0 || n > max_n) return false;
    if (use_ds && (steps > FS_MAX_STEPS || hist_bins > FS_MAX_BINS)) return false;
    return true;
}

// Returns QP_OK when the launch was enqueued, a negative status on an error, and
// QP_WARN_INFEASIBLE when this device cannot hold the grid (the caller then runs the chain).
int32_t qp_launch_sender_fused(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int bits, int method, int bmode,
                               int steps, int hist_bins, double F, void* d_packed, qp_qparams_t* d_qp_out,
                               qp_stats_t* d_stats_out, cudaStream_t s)
{
    const int use_ds = (method & 0xF) == QP_CLIP_DSACIQ;
    const uint64_t total_words = qp_packed_bytes(n, bits) / 4;
    const uint64_t groups = (total_words + bits - 1) / bits;             // 32-element groups, pad words included
    const unsigned G = (unsigned)ctx->sm_count;
    const unsigned gpb = (unsigned)((groups + G - 1) / G);
    const size_t dyn = (size_t)gpb * 33 * sizeof(float);
    void* kernel = dtype == QP_F32 ? (void*)sender_fused_kernel<float> : (void*)sender_fused_kernel<unsigned short>;

    if (!ctx->fused_checked) {                   // once: how large a slice can one block per SM hold?
        ctx->fused_checked = 1;
        ctx->fused_ok = 0;
        ctx->fused_dyn_max = 0;
        int coop = 0, optin = 0;
        bool ok = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, ctx->device) == cudaSuccess && coop &&
                  cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, ctx->device) == cudaSuccess &&
                  (size_t)G * (FS_MAX_STEPS + 1) <= (size_t)QP_MAX_BLOCKS * QP_EVAL_K && G <= QP_MAX_BLOCKS;
        size_t dyn_max = 0;
        for (int t = 0; ok && t < 2; ++t) {
            void* kf = t ? (void*)sender_fused_kernel<unsigned short> : (void*)sender_fused_kernel<float>;
            cudaFuncAttributes fa;
            int per_sm = 0;
            ok = cudaFuncGetAttributes(&fa, kf) == cudaSuccess && (size_t)optin > fa.sharedSizeBytes + 2048;
            if (!ok) break;
            const size_t room = (size_t)optin - fa.sharedSizeBytes - 1024;     // 1 KB the system keeps per block
            dyn_max = t ? (room < dyn_max ? room : dyn_max) : room;
            ok = cudaFuncSetAttribute(kf, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)room) == cudaSuccess &&
                 cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kf, FS_THREADS, room) == cudaSuccess &&
                 per_sm >= 1;
        }
        if (!ok) cudaGetLastError();
        ctx->fused_ok = ok ? 1 : 0;
        ctx->fused_dyn_max = ok ? dyn_max : 0;
    }
    if (!ctx->fused_ok || dyn > ctx->fused_dyn_max) return QP_WARN_INFEASIBLE;   // the caller runs the chain

    // The arrival counter and the histogram start at zero: the context allocates them zeroed and
    // every completed launch leaves them so (a timed-out one does not: qp_get_status clears them).
    FsArgs a;
    a.x = d_x; a.n = n; a.bits = bits; a.use_ds = use_ds; a.method = method; a.bmode = bmode; a.steps = steps; a.nb = hist_bins; a.F = F;
    a.out = static_cast<uint32_t*>(d_packed);
    a.total_words = total_words;
    a.groups_per_block = gpb;
    a.qp_out = d_qp_out;
    a.st_out = d_stats_out;
    a.ds_out = nullptr;
    a.part = reinterpret_cast<double*>(ctx->d_part);
    a.hist = reinterpret_cast<unsigned long long*>(reinterpret_cast<unsigned char*>(ctx->d_fused) + 256);
    a.sums = ctx->d_sums;
    a.curve = ctx->d_curve;
    a.cand = ctx->d_cand;
    a.setup = ctx->d_setup;
    a.bar = reinterpret_cast<unsigned*>(ctx->d_fused);
    a.status = ctx->d_status;
    a.spin_limit = ctx->spin_limit;
    a.bar_extra = (unsigned)ctx->bar_extra;
    void* params[] = {&a};
    if (cudaLaunchCooperativeKernel(kernel, dim3(G), dim3(FS_THREADS), params, dyn, s) != cudaSuccess)
        return qp_check_launch(ctx, "qp_sender_device (cooperative launch)");
    ctx->launches += 1;
    return qp_check_launch(ctx, "qp_sender_device");
}
