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
// (taken from a reference point per cell) are accumulated in fixed point with unit u (a
// power of two below cell/2^15) by two 32-bit shared-memory atomics per element, as
// integers: sums are exact and order-independent (bit-reproducible); the only approximation
// is the rounding of each offset to u, which moves a candidate's MSE by less than 1e-6
// relative in the worst case (all roundings aligned) and by ~1e-11 in practice.
#include <type_traits>

#include "qp_internal.cuh"

QP_CK_UNIT

namespace {

constexpr int G = QP_IV_CELLS;
constexpr int MAXB = QP_IV_MAXB;
constexpr unsigned long long S1_MASK = (1ull << 40) - 1ull;

// Grid cell of x in [g_lo, g_hi]: its position in cell units, rounded to the nearest integer
// (0..G, so G + 1 cells).  The rounding is done by adding 2^23 (no conversion instruction):
// `pm` keeps the cell number in its low mantissa bits.  Each operation is rounded on its own,
// so the function is monotone in x.
constexpr float IV_MAGIC = 8388608.0f;
__device__ __forceinline__ float cell_pm(float x, float g_lo, float inv_gw)
{
    return __fadd_rn(__fmul_rn(__fsub_rn(x, g_lo), inv_gw), IV_MAGIC);
}
__device__ __forceinline__ int cell_of(float x, float g_lo, float inv_gw)
{
    return (int)(__float_as_uint(cell_pm(x, g_lo, inv_gw)) & 0x7FFFFFu);
}

// Reference point of every interval inside the cell whose `pm` is given: one cell below the
// cell's centre, so that offsets x - ref are positive (between ~0.5 and ~1.5 cells).  Any
// fixed function of the cell would do; it only has to be the same where the moments are
// gathered and where they are used.
__device__ __forceinline__ float cell_ref(float pm, float g_lo, float gw)
{
    return fmaf(__fsub_rn(pm, IV_MAGIC + 1.0f), gw, g_lo);      // (cell - 1) * gw + g_lo
}

// ------------------------------------------------------------------ grid + boundaries

// Set-up and boundaries in one launch.  Every block repeats the cheap part (peak of the
// histogram -> b_R, the candidates and their quantizers, the grid that covers all valid
// candidates; block 0 stores them for the later kernels), then: thread t < nthr finds
// threshold (k, j) of candidate k = t / (L-1), code j = 1 + t % (L-1); thread nthr + c - 1
// finds the left edge of grid cell c = 1..G.  Entries that do not exist are +inf.
constexpr int IV_MAX_CAND = 1024;
__global__ void __launch_bounds__(256) iv_bounds_kernel(const qp_stats_t* __restrict__ st,
                                                        const unsigned long long* __restrict__ hist, int nb, int bits,
                                                        int bmode, int steps, double F, float4* __restrict__ cand,
                                                        int* __restrict__ valid, qp_ds_setup* __restrict__ setup,
                                                        float* __restrict__ bnd, unsigned* __restrict__ status)
{
    __shared__ unsigned long long s_top[8];
    __shared__ float s_lo[8], s_hi[8];
    __shared__ float sg_lo, sg_hi, sg_inv;
    __shared__ qp_ds_setup s;
    __shared__ float4 s_cand[IV_MAX_CAND];
    __shared__ unsigned char s_valid[IV_MAX_CAND];
    const float inf = __int_as_float(0x7F800000);
    const int ncand = steps + 1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    unsigned long long top = 0;
    const bool from_stats = st->hist_bins == nb;
    const bool promised = (bmode & QP_B_HIST_IN_STATS) != 0;      // then nobody has counted into hist
    if (promised && !from_stats && blockIdx.x == 0 && threadIdx.x == 0) atomicOr(status, QP_DEV_HIST_MISSING);
    for (int b = threadIdx.x; !from_stats && !promised && b < nb; b += 256) {
        const unsigned long long c = hist[b];
        top = c > top ? c : top;
    }
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_down_sync(0xFFFFFFFFu, top, o);
        top = other > top ? other : top;
    }
    if (lane == 0) s_top[warp] = top;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) top = s_top[w] > top ? s_top[w] : top;
        if (from_stats) top = st->hist_peak;
        qp_ds_make_setup(st, top, nb, bmode, F, s);
    }
    __syncthreads();
    float lo = inf, hi = -inf;
    for (int k = threadIdx.x; k < ncand; k += 256) {
        float4 c;
        int ok;
        qp_ds_candidate(s, k, steps, bits, bmode & QP_B_MIDRISE, c, ok);
        s_cand[k] = c;
        s_valid[k] = (unsigned char)ok;
        if (blockIdx.x == 0) { cand[k] = c; valid[k] = ok; }
        if (ok) { lo = fminf(lo, c.x); hi = fmaxf(hi, c.y); }
    }
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_down_sync(0xFFFFFFFFu, lo, o));
        hi = fmaxf(hi, __shfl_down_sync(0xFFFFFFFFu, hi, o));
    }
    if (lane == 0) { s_lo[warp] = lo; s_hi[warp] = hi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) { lo = fminf(lo, s_lo[w]); hi = fmaxf(hi, s_hi[w]); }
        const double width = (double)hi - (double)lo;
        float inv_gw = 0.f;
        double u = 1.0;
        if (width > 0.0) {
            inv_gw = (float)((double)G / width);
            int e;
            frexp(width / (double)G, &e);               // cell width in [2^(e-1), 2^e)
            u = ldexp(1.0, e - 16);                     // offsets (up to ~1.5 cells) stay below 2^17.6 units
        }
        sg_lo = lo; sg_hi = hi; sg_inv = inv_gw;
        if (blockIdx.x == 0) {
            s.g_lo = lo;
            s.g_hi = hi;
            s.inv_gw = inv_gw;
            s.u = u;
            s.inv_u = (float)(1.0 / u);
            s.gw = (float)(width / (double)G);
            s.pad2 = 0.f;
            *setup = s;
        }
    }
    __syncthreads();
    const float g_lo = sg_lo, g_hi = sg_hi, inv_gw = sg_inv;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int L1 = (1 << bits) - 1;
    const int nthr = ncand * L1;
    if (t < nthr) {
        const int k = t / L1, j = 1 + t % L1;
        float out = inf;
        if (s_valid[k] && g_hi > g_lo) {
            const float4 q = s_cand[k];
            const unsigned mask = (unsigned)L1;
            auto pred = [&](float x) { return (int)qp_code(x, q.x, q.y, q.w, mask) >= j; };
            if (!pred(g_lo) && pred(g_hi)) out = qp_first_true(g_lo, g_hi, pred);
        }
        bnd[t] = out;
    } else if (t < nthr + G) {
        const int c = t - nthr + 1;
        float out = inf;
        if (g_hi > g_lo) {
            auto pred = [&](float x) { return cell_of(x, g_lo, inv_gw) >= c; };
            if (!pred(g_lo) && pred(g_hi)) out = qp_first_true(g_lo, g_hi, pred);
        }
        bnd[t] = out;
    } else if (t < MAXB) {
        bnd[t] = inf;
    }
}

// Rank sort of the MAXB boundaries (rank = entries that are smaller, or equal with a lower
// index).  The array is [nthr thresholds in any order][cell edges, then +inf fillers]; the
// second part is already non-decreasing (the edge of a cell is never below the edge of the
// cell before it, missing cells are +inf at the end), so only the thresholds need comparing:
//   threshold:  rank = thresholds before it + tail entries strictly below it (binary search)
//   tail entry: rank = thresholds <= it + its own position in the tail
// Block b places entries [32b, 32b+32): thread t compares entry 32b + (t & 31) with the
// thresholds of slice t >> 5, the 16 slice counts are merged in shared memory.
// bb[0] = g_lo, bb[1 + r] = entry of rank r; +inf entries end up behind the finite ones.
// For the entry that is the left edge of grid cell c it also stores
// first[c] = number of boundaries <= that edge (the edge included), or ~0 if the cell does
// not exist: cell c then meets the intervals first[c] .. first[c+1] - 1.
constexpr int IV_RANK_PER_BLOCK = 32;
__global__ void __launch_bounds__(512) iv_rank_kernel(const float* __restrict__ bnd, const qp_ds_setup* __restrict__ setup,
                                                      int nthr, float* __restrict__ bb, unsigned* __restrict__ first)
{
    __shared__ float s[MAXB];
    __shared__ int rank[IV_RANK_PER_BLOCK], le[IV_RANK_PER_BLOCK];
    for (int i = threadIdx.x; i < MAXB; i += 512) s[i] = bnd[i];
    if (threadIdx.x < IV_RANK_PER_BLOCK) { rank[threadIdx.x] = 0; le[threadIdx.x] = 0; }
    __syncthreads();
    const int local = threadIdx.x & 31, slice = threadIdx.x >> 5;
    const int me = blockIdx.x * IV_RANK_PER_BLOCK + local;
    const float v = s[me];
    int cnt = 0, cnt_le = 0;
    const int per = (nthr + 15) / 16;                         // thresholds per slice
    const int j1 = min(nthr, (slice + 1) * per);
    for (int j = slice * per; j < j1; ++j) {
        const float w = s[j];
        cnt += (w < v || (w == v && j < me)) ? 1 : 0;
        cnt_le += (w <= v) ? 1 : 0;
    }
    if (slice == 0) {                                         // the sorted tail: binary searches
        const float* tail = s + nthr;
        const int len = MAXB - nthr;
        int lo = 0, hi = len;                                 // entries strictly below v
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (tail[mid] < v) lo = mid + 1; else hi = mid;
        }
        const int below = lo;
        hi = len;                                             // entries <= v (continue from `below`)
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (tail[mid] <= v) lo = mid + 1; else hi = mid;
        }
        cnt_le += lo;
        // a threshold counts the tail entries below it; a tail entry counts its own position (equal
        // tail entries before it have lower indices; the loop above has counted the thresholds <= it,
        // which all have lower indices too)
        cnt += me < nthr ? below : (me - nthr);
    }
    atomicAdd(&rank[local], cnt);
    atomicAdd(&le[local], cnt_le);
    __syncthreads();
    if (threadIdx.x < IV_RANK_PER_BLOCK) {
        const int t = blockIdx.x * IV_RANK_PER_BLOCK + threadIdx.x;
        const float mine = s[t];
        bb[1 + rank[threadIdx.x]] = mine;
        if (t >= nthr && t < nthr + G)
            first[t - nthr + 1] = (mine < __int_as_float(0x7F800000)) ? (unsigned)le[threadIdx.x] : 0xFFFFFFFFu;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        bb[0] = setup->g_lo;
        first[0] = 0u;                   // every boundary lies above g_lo
        first[G + 1] = 0xFFFFFFFFu;
    }
}

// ------------------------------------------------------------------------ moments

struct IvShared {
    float* bb;                      // [MAXB + 1]
    unsigned* cell;                 // [G + 1] first interval of the cell | last interval << 16
    unsigned* cnt;                  // [MAXB + 1] count (bits 0-23) | carries out of s1 (bits 24-31)
    unsigned* s1;                   // [MAXB + 1] low 32 bits of the sum of offsets
};

// Elements outside [g_lo, g_hi] are clipped by every candidate.  They go through the interval
// of the end they were clamped to (which contributes (level - end)^2 for them), and the rest of
// their error, -2 (level - end) e + e^2 with e = signed distance beyond the end (negative below
// g_lo, positive above g_hi, zero inside), needs only the sums of e on each side and of e^2.
// Kept per thread as sum e, sum |e| (the two sides are their half sum and half difference) and
// sum e^2: one subtraction and three accumulations per element.
struct IvOuter {                    // per thread, fp64
    double s1, s1a, s2, s2_in;
};
struct IvBatch {                    // the same over one batch of <= 8 elements, fp32
    float s1, s1a, s2, s2_in;
};
__device__ __forceinline__ void iv_flush(IvOuter& o, const IvBatch& b)
{
    o.s1 += (double)b.s1; o.s1a += (double)b.s1a; o.s2 += (double)b.s2;
    o.s2_in += (double)b.s2_in;
}

struct IvConst { float g_lo, g_hi, inv_gw, gw, inv_u; };

template <bool GUARD>
__device__ __forceinline__ void iv_one(float x, const IvShared& sh, const IvConst& k, IvBatch& b)
{
    if (GUARD && !qp_is_finite(x)) return;
    {
        const float xc = fminf(fmaxf(x, k.g_lo), k.g_hi);
        const float e = __fsub_rn(x, xc);
        b.s1 += e; b.s1a += fabsf(e); b.s2 = fmaf(e, e, b.s2);
        x = xc;
        const float pm = cell_pm(x, k.g_lo, k.inv_gw);
        const unsigned ci = sh.cell[QP_CK(__float_as_uint(pm) & 0x7FFFFFu, G + 1)];
        unsigned lo = ci & 0xFFFFu, hi = ci >> 16;
        while (lo < hi) {                                   // largest i in [lo, hi] with bb[i] <= x
            const unsigned mid = (lo + hi + 1u) >> 1;
            if (sh.bb[QP_CK(mid, MAXB + 1)] <= x) lo = mid; else hi = mid - 1u;
        }
        lo = QP_CK(lo, MAXB + 1);
        // offset in units of u, rounded to an integer by the same 2^23 trick (u is a power of two,
        // so the product is exact and the only rounding is the one to the integer)
        const float dm = fmaf(__fsub_rn(x, cell_ref(pm, k.g_lo, k.gw)), k.inv_u, IV_MAGIC);
        const unsigned d1 = __float_as_uint(dm) & 0x7FFFFFu;
        const float d1f = __fsub_rn(dm, IV_MAGIC);
        b.s2_in = fmaf(d1f, d1f, b.s2_in);
        // two 32-bit atomics (fewer bank conflicts than one 64-bit one); a wrap of the low word
        // of the sum is carried into the top byte of the count word, so nothing is lost
        atomicAdd(&sh.cnt[lo], 1u);
        const unsigned old = atomicAdd(&sh.s1[lo], d1);
        if (old + d1 < old) atomicAdd(&sh.cnt[lo], 1u << 24);
    }
}

template <typename T>
__global__ void __launch_bounds__(QP_IV_THREADS) iv_moments_kernel(const T* __restrict__ x, uint64_t n,
                                                                   const qp_stats_t* __restrict__ st,
                                                                   const qp_ds_setup* __restrict__ setup,
                                                                   const float* __restrict__ g_bb,
                                                                   const unsigned* __restrict__ g_first,
                                                                   unsigned* __restrict__ g_m,
                                                                   unsigned long long* __restrict__ part,
                                                                   double* __restrict__ outer)
{
    extern __shared__ __align__(16) unsigned char raw[];
    IvShared sh;
    sh.cnt = reinterpret_cast<unsigned*>(raw);
    sh.s1 = sh.cnt + (MAXB + 1);
    sh.bb = reinterpret_cast<float*>(sh.s1 + (MAXB + 1));
    sh.cell = reinterpret_cast<unsigned*>(sh.bb + (MAXB + 1));
    const float inf = __int_as_float(0x7F800000);
    for (unsigned i = threadIdx.x; i <= (unsigned)MAXB; i += QP_IV_THREADS) {
        sh.cnt[i] = 0u;
        sh.s1[i] = 0u;
        sh.bb[i] = g_bb[i];
    }
    __syncthreads();
    __shared__ unsigned s_m;
    if (threadIdx.x == 0) {                                  // m = finite boundaries (sorted: a binary search)
        int lo = 0, hi = MAXB;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (sh.bb[1 + mid] < inf) lo = mid + 1; else hi = mid;
        }
        s_m = (unsigned)lo;
        if (blockIdx.x == 0) *g_m = (unsigned)lo;
    }
    __syncthreads();
    const unsigned m = s_m;                                  // intervals 0..m
    // cell c meets intervals first[c] .. first[c+1]-1; a cell that does not exist counts as m + 1
    for (unsigned c = threadIdx.x; c <= (unsigned)G; c += QP_IV_THREADS) {
        unsigned f0 = g_first[c], f1 = g_first[c + 1];
        f0 = (f0 == 0xFFFFFFFFu) ? m + 1u : f0;
        f1 = (f1 == 0xFFFFFFFFu) ? m + 1u : f1;
        sh.cell[c] = (f0 & 0xFFFFu) | ((f1 - 1u) << 16);
    }
    __syncthreads();

    const IvConst k = {setup->g_lo, setup->g_hi, setup->inv_gw, setup->gw, setup->inv_u};
    const bool guard = st->nonfinite != 0;
    IvOuter o = {0.0, 0.0, 0.0, 0.0};

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
            IvBatch bt = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < EPV; ++i) iv_one<GD>(a[i], sh, k, bt);
#pragma unroll
            for (int i = 0; i < EPV; ++i) iv_one<GD>(b[i], sh, k, bt);
            iv_flush(o, bt);
        }
        for (; v < sp.nvec; v += stride) {
            float a[EPV];
            qp_load_vec(xv + v * EPV, a);
            IvBatch bt = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < EPV; ++i) iv_one<GD>(a[i], sh, k, bt);
            iv_flush(o, bt);
        }
        if (blockIdx.x == 0) {
            const uint64_t t0 = sp.head + sp.nvec * EPV;
            for (uint64_t i = threadIdx.x; i < sp.head + sp.tail; i += QP_IV_THREADS) {
                IvBatch bt = {0.f, 0.f, 0.f, 0.f};
                iv_one<GD>(qp_load_one(x + (i < sp.head ? i : t0 + (i - sp.head))), sh, k, bt);
                iv_flush(o, bt);
            }
        }
    };
    if (guard) body(std::true_type{}); else body(std::false_type{});
    __syncthreads();
    unsigned long long* mine = part + (size_t)blockIdx.x * (MAXB + 1);
    for (unsigned i = threadIdx.x; i <= m; i += QP_IV_THREADS) {      // count << 40 | 40-bit sum of offsets
        const unsigned c = sh.cnt[i];
        mine[i] = ((unsigned long long)(c & 0xFFFFFFu) << 40) | ((unsigned long long)(c >> 24) << 32) | sh.s1[i];
    }

    __shared__ double red[QP_IV_THREADS / 32];
    const double r0 = qp_block_sum(o.s1, red), r1 = qp_block_sum(o.s1a, red);
    const double r2 = qp_block_sum(o.s2, red), r3 = 0.0;
    const double r4 = 0.0, r5 = 0.0;
    const double r6 = qp_block_sum(o.s2_in, red);
    if (threadIdx.x == 0) {
        double* dst = outer + (size_t)blockIdx.x * 8;
        dst[0] = r0; dst[1] = r1; dst[2] = r2; dst[3] = r3; dst[4] = r4; dst[5] = r5; dst[6] = r6;
    }
}

// ---------------------------------------------------------------- moments, second form
//
// Same result as iv_moments_kernel (the same per-block rows of count << 40 | sum of offsets,
// the same outer sums), gathered with less work per element.  Most grid cells hold no
// threshold: such a cell is one interval, and its two sums need neither the table look-up nor
// the search.  They are kept in a table indexed by cell and replica (8 replicas of every cell,
// chosen by lane, so that elements of one value do not queue up behind one counter and a warp's
// atomics spread over the banks).  Cells that do hold thresholds ("split" cells) carry a mark
// in the top bit of their replica counters; the counter's old value, which the atomic returns
// anyway, tells the thread that its element needs the exact treatment.  Those elements are not
// handled on the spot (a warp would run the whole search for a few active lanes): each warp
// collects them in a small buffer of its own and works them off 32 at a time with all lanes
// busy, through the same cell table, search and interval sums as the first form.
// One block of 1024 threads per SM (the replica table takes 131 KB).  512 cells x 32 replicas
// (conflict-free, but more split cells) and 1024 x 16 were tried too: within 3 % of each other.
constexpr int IV2_THREADS = 1024;
constexpr int IV2_WARPS = IV2_THREADS / 32;
constexpr int IV2_STAGE = 64;                        // buffered elements per warp (worked off from 32 on)
constexpr unsigned IV2_SPLIT = 0x80000000u;
constexpr int IV2_RS = 3;                            // log2 of the replicas per cell
constexpr unsigned IV2_R = 1u << IV2_RS;
// replica sums are 32 bit: elements per block * largest offset (1.5 * 2^16 units) / 8 replicas < 2^32
constexpr uint64_t IV2_MAX_PER_BLOCK = 340000;

struct Iv2Shared {
    unsigned* rcnt;                 // [(G + 1) * IV2_R] per cell and replica: count (| IV2_SPLIT in split cells)
    unsigned* rs1;                  // [(G + 1) * IV2_R] per cell and replica: sum of offsets
    float* stage;                   // [IV2_WARPS][IV2_STAGE]
};

// exact treatment of one clamped, finite element of a split cell: as iv_one without the sums
// that the fast path has already taken
__device__ __forceinline__ void iv2_exact(float x, const IvShared& sh, const IvConst& k)
{
    const float pm = cell_pm(x, k.g_lo, k.inv_gw);
    const unsigned ci = sh.cell[QP_CK(__float_as_uint(pm) & 0x7FFFFFu, G + 1)];
    unsigned lo = ci & 0xFFFFu, hi = ci >> 16;
    while (lo < hi) {                                   // largest i in [lo, hi] with bb[i] <= x
        const unsigned mid = (lo + hi + 1u) >> 1;
        if (sh.bb[QP_CK(mid, MAXB + 1)] <= x) lo = mid; else hi = mid - 1u;
    }
    lo = QP_CK(lo, MAXB + 1);
    const float dm = fmaf(__fsub_rn(x, cell_ref(pm, k.g_lo, k.gw)), k.inv_u, IV_MAGIC);
    const unsigned d1 = __float_as_uint(dm) & 0x7FFFFFu;
    atomicAdd(&sh.cnt[lo], 1u);
    const unsigned old = atomicAdd(&sh.s1[lo], d1);
    if (old + d1 < old) atomicAdd(&sh.cnt[lo], 1u << 24);
}

// A batch of N elements per lane: clamp, outer sums, cell, offset and the two replica atomics of ALL of
// them first (independent: their latencies overlap), then one vote on whether any element of the warp
// met a split cell (the mark comes back with the count atomic's old value).  Only then, element by
// element, the split ones go into the warp's buffer; from 32 buffered elements on, the warp works 32 of
// them off with every lane busy.  (Asking after every element instead made each element wait for its
// own atomic to return: the pass was bound by that latency, not by issue slots or the shared-memory
// pipe.)  Called by all 32 lanes together (lanes without an element pass a non-finite value to the
// guarded form).
template <bool GUARD, int N>
__device__ __forceinline__ void iv2_batch(const float (&x)[N], const IvShared& sh, const Iv2Shared& s2, const IvConst& k,
                                          IvBatch& b, float* my_stage, unsigned& staged, unsigned lane)
{
    const unsigned full = 0xFFFFFFFFu;
    float xc[N];
    unsigned flags = 0u;                                 // bit i: element i lies in a split cell
#pragma unroll
    for (int i = 0; i < N; ++i) {
        xc[i] = x[i];
        if (!GUARD || qp_is_finite(x[i])) {
            xc[i] = fminf(fmaxf(x[i], k.g_lo), k.g_hi);
            const float e = __fsub_rn(x[i], xc[i]);
            b.s1 += e; b.s1a += fabsf(e); b.s2 = fmaf(e, e, b.s2);
            const float pm = cell_pm(xc[i], k.g_lo, k.inv_gw);
            const float dm = fmaf(__fsub_rn(xc[i], cell_ref(pm, k.g_lo, k.gw)), k.inv_u, IV_MAGIC);
            const float d1f = __fsub_rn(dm, IV_MAGIC);
            b.s2_in = fmaf(d1f, d1f, b.s2_in);
            const unsigned idx = QP_CK(((__float_as_uint(pm) & 0x7FFFFFu) << IV2_RS) + (lane & (IV2_R - 1u)), (G + 1) * IV2_R);
            const unsigned old = atomicAdd(&s2.rcnt[idx], 1u);
            atomicAdd(&s2.rs1[idx], __float_as_uint(dm) & 0x7FFFFFu);     // ignored later if the cell is split
            flags |= (old >> 31) << i;                   // IV2_SPLIT is the top bit
        }
    }
    if (!__any_sync(full, flags != 0u)) return;          // warp-uniform
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const bool split = (flags >> i) & 1u;
        const unsigned m = __ballot_sync(full, split);
        if (m) {                                         // warp-uniform
            if (split) my_stage[QP_CK(staged + __popc(m & ((1u << lane) - 1u)), IV2_STAGE)] = xc[i];
            staged += __popc(m);
            if (staged >= 32u) {
                __syncwarp();
                staged -= 32u;
                iv2_exact(my_stage[staged + lane], sh, k);
                __syncwarp();
            }
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(IV2_THREADS, 1) iv_moments2_kernel(const T* __restrict__ x, uint64_t n,
                                                                     const qp_stats_t* __restrict__ st,
                                                                     const qp_ds_setup* __restrict__ setup,
                                                                     const float* __restrict__ g_bb,
                                                                     const unsigned* __restrict__ g_first,
                                                                     unsigned* __restrict__ g_m,
                                                                     unsigned long long* __restrict__ part,
                                                                     double* __restrict__ outer)
{
    extern __shared__ __align__(16) unsigned char raw[];
    IvShared sh;
    Iv2Shared s2;
    s2.rcnt = reinterpret_cast<unsigned*>(raw);
    s2.rs1 = s2.rcnt + (G + 1) * IV2_R;
    sh.cnt = s2.rs1 + (G + 1) * IV2_R;
    sh.s1 = sh.cnt + (MAXB + 1);
    sh.bb = reinterpret_cast<float*>(sh.s1 + (MAXB + 1));
    sh.cell = reinterpret_cast<unsigned*>(sh.bb + (MAXB + 1));
    s2.stage = reinterpret_cast<float*>(sh.cell + (G + 1));
    const float inf = __int_as_float(0x7F800000);
    for (unsigned i = threadIdx.x; i <= (unsigned)MAXB; i += IV2_THREADS) {
        sh.cnt[i] = 0u;
        sh.s1[i] = 0u;
        sh.bb[i] = g_bb[i];
    }
    __syncthreads();
    __shared__ unsigned s_m;
    if (threadIdx.x == 0) {                                  // m = finite boundaries (sorted: a binary search)
        int lo = 0, hi = MAXB;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (sh.bb[1 + mid] < inf) lo = mid + 1; else hi = mid;
        }
        s_m = (unsigned)lo;
        if (blockIdx.x == 0) *g_m = (unsigned)lo;
    }
    __syncthreads();
    const unsigned m = s_m;                                  // intervals 0..m
    // cell c meets intervals first[c] .. first[c+1]-1 (a cell that does not exist counts as m + 1);
    // more than one interval = the cell holds a threshold
    for (unsigned c = threadIdx.x; c <= (unsigned)G; c += IV2_THREADS) {
        unsigned f0 = g_first[c], f1 = g_first[c + 1];
        f0 = (f0 == 0xFFFFFFFFu) ? m + 1u : f0;
        f1 = (f1 == 0xFFFFFFFFu) ? m + 1u : f1;
        sh.cell[c] = (f0 & 0xFFFFu) | ((f1 - 1u) << 16);
    }
    __syncthreads();
    for (unsigned i = threadIdx.x; i < (unsigned)(G + 1) * IV2_R; i += IV2_THREADS) {
        const unsigned ci = sh.cell[i >> IV2_RS];
        s2.rcnt[i] = ((ci >> 16) != (ci & 0xFFFFu)) ? IV2_SPLIT : 0u;
        s2.rs1[i] = 0u;
    }
    __syncthreads();

    const IvConst k = {setup->g_lo, setup->g_hi, setup->inv_gw, setup->gw, setup->inv_u};
    const bool guard = st->nonfinite != 0;
    IvOuter o = {0.0, 0.0, 0.0, 0.0};
    const unsigned lane = threadIdx.x & 31u;
    float* my_stage = s2.stage + (threadIdx.x >> 5) * IV2_STAGE;
    unsigned staged = 0;                                     // warp-uniform

    constexpr int EPV = qp_span<T>::EPV;
    const qp_span<T> sp(x, n);
    const T* xv = x + sp.head;
    const uint64_t stride = (uint64_t)gridDim.x * IV2_THREADS;
    // every lane of a warp runs the same number of iterations (ballots inside): the loops below
    // are bounded by warp-uniform conditions and lanes without an element pass a non-finite one
    auto body = [&](auto guard_tag) {
        constexpr bool GD = decltype(guard_tag)::value;
        const float skip = __int_as_float(0x7FC00000);       // NaN: ignored by the guarded form
        uint64_t v = (uint64_t)blockIdx.x * IV2_THREADS + threadIdx.x;
        // two vectors per lane while the warp's last lane still has both (v - lane + 31 is its first vector)
        // (the next pair is loaded before the current one is worked on, so a warp does not sit out the load latency)
        auto both = [&](uint64_t vv) { return vv - lane + 31u + stride < sp.nvec; };   // warp-uniform
        if (both(v)) {
            float a[EPV], b[EPV];
            qp_load_vec(xv + v * EPV, a);
            qp_load_vec(xv + (v + stride) * EPV, b);
            for (;;) {
                const uint64_t vn = v + 2 * stride;
                const bool more = both(vn);
                float na[EPV], nb[EPV];
                if (more) {
                    qp_load_vec(xv + vn * EPV, na);
                    qp_load_vec(xv + (vn + stride) * EPV, nb);
                }
                IvBatch bt = {0.f, 0.f, 0.f, 0.f};
                iv2_batch<GD>(a, sh, s2, k, bt, my_stage, staged, lane);
                iv2_batch<GD>(b, sh, s2, k, bt, my_stage, staged, lane);
                iv_flush(o, bt);
                v = vn;
                if (!more) break;
#pragma unroll
                for (int i = 0; i < EPV; ++i) { a[i] = na[i]; b[i] = nb[i]; }
            }
        }
        // the rest: warps may be partly filled, so every lane of a warp that still has work goes on
        const uint64_t warp_v0 = v - lane;                   // vector of lane 0 (v advanced alike in all lanes)
        for (uint64_t w0 = warp_v0; w0 < sp.nvec; w0 += stride) {
            const uint64_t mine = w0 + lane;
            const bool have = mine < sp.nvec;
            float a[EPV];
            if (have) qp_load_vec(xv + mine * EPV, a);
#pragma unroll
            for (int i = 0; i < EPV; ++i) a[i] = have ? a[i] : skip;
            IvBatch bt = {0.f, 0.f, 0.f, 0.f};
            iv2_batch<true>(a, sh, s2, k, bt, my_stage, staged, lane);
            iv_flush(o, bt);
        }
        if (blockIdx.x == 0) {
            const uint64_t t0 = sp.head + sp.nvec * EPV;
            const uint64_t extra = sp.head + sp.tail;
            for (uint64_t i0 = (threadIdx.x & ~31u); i0 < extra; i0 += IV2_THREADS) {
                const uint64_t i = i0 + lane;
                const bool have = i < extra;
                IvBatch bt = {0.f, 0.f, 0.f, 0.f};
                const float x1[1] = {have ? qp_load_one(x + (i < sp.head ? i : t0 + (i - sp.head))) : skip};
                iv2_batch<true>(x1, sh, s2, k, bt, my_stage, staged, lane);
                iv_flush(o, bt);
            }
        }
    };
    if (guard) body(std::true_type{}); else body(std::false_type{});
    __syncwarp();
    if (lane < staged) iv2_exact(my_stage[lane], sh, k);     // what is left in the warp's buffer (< 32)
    __syncthreads();

    // this block's row: a whole cell is its one interval (replicas added up); a split cell's
    // intervals come from the exact sums
    unsigned long long* mine = part + (size_t)blockIdx.x * (MAXB + 1);
    for (unsigned c = threadIdx.x; c <= (unsigned)G; c += IV2_THREADS) {
        const unsigned ci = sh.cell[c];
        const unsigned i0 = ci & 0xFFFFu, i1 = ci >> 16;
        if (i0 > m) continue;                                // the cell does not exist
        if (i0 == i1) {
            unsigned long long cn = 0, cs = 0;
            for (unsigned r = 0; r < IV2_R; ++r) {
                const unsigned rr = (r + lane) & (IV2_R - 1u);   // lanes start at different replicas
                cn += s2.rcnt[(c << IV2_RS) + rr];
                cs += s2.rs1[(c << IV2_RS) + rr];
            }
            mine[i0] = (cn << 40) | cs;
        } else {
            for (unsigned i = i0; i <= i1 && i <= m; ++i) {
                const unsigned cw = sh.cnt[i];
                mine[i] = ((unsigned long long)(cw & 0xFFFFFFu) << 40) | ((unsigned long long)(cw >> 24) << 32) | sh.s1[i];
            }
        }
    }

    __shared__ double red[IV2_THREADS / 32];
    const double r0 = qp_block_sum(o.s1, red), r1 = qp_block_sum(o.s1a, red);
    const double r2 = qp_block_sum(o.s2, red);
    const double r6 = qp_block_sum(o.s2_in, red);
    if (threadIdx.x == 0) {
        double* dst = outer + (size_t)blockIdx.x * 8;
        dst[0] = r0; dst[1] = r1; dst[2] = r2; dst[3] = 0.0; dst[4] = 0.0; dst[5] = 0.0; dst[6] = r6;
    }
}

// Totals over the blocks' partials.  A block takes 32 consecutive intervals: lane = interval
// (one 256-byte row segment per warp load), warp w adds the partials of blocks w, w + 32, ...
// (all of its loads in flight at once), the 32 warp sums are merged through shared memory and written
// once.  Integer sums, so the order does not matter.  Block 0 also adds up the outer sums
// in block order.
constexpr int IV_RED_THREADS = 1024;
constexpr int IV_RED_WARPS = IV_RED_THREADS / 32;
__global__ void __launch_bounds__(IV_RED_THREADS) iv_reduce_kernel(const unsigned long long* __restrict__ part, int blocks,
                                                                   const unsigned* __restrict__ g_m,
                                                                   qp_iv_total* __restrict__ tot,
                                                                   const double* __restrict__ outer,
                                                                   double* __restrict__ outer_tot)
{
    __shared__ unsigned long long s_n[IV_RED_WARPS][32], s_s[IV_RED_WARPS][32];
    const unsigned m = *g_m;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned i = blockIdx.x * 32 + lane;
    unsigned long long n = 0, s1 = 0;
    if (i <= m) {
        for (int b0 = warp; b0 < blocks; b0 += IV_RED_WARPS * 16) {
            unsigned long long p[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int b = b0 + u * IV_RED_WARPS;
                p[u] = b < blocks ? part[(size_t)b * (MAXB + 1) + i] : 0ull;
            }
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                n += p[u] >> 40;
                s1 += p[u] & S1_MASK;
            }
        }
    }
    s_n[warp][lane] = n;
    s_s[warp][lane] = s1;
    __syncthreads();
    if (warp == 0 && i <= m) {
        for (int w = 1; w < IV_RED_WARPS; ++w) {
            n += s_n[w][lane];
            s1 += s_s[w][lane];
        }
        tot[i].n = n;
        tot[i].s1 = s1;
    }
    if (blockIdx.x == 0 && threadIdx.x < 7 * 32) {
        // warp w adds up quantity w: lane l takes blocks l, l+32, ... then a fixed shuffle tree
        const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
        double t = 0.0;
        for (int b = l; b < blocks; b += 32) t += outer[(size_t)b * 8 + w];
        for (int o = 16; o > 0; o >>= 1) t += __shfl_down_sync(0xFFFFFFFFu, t, o);
        if (l == 0) outer_tot[w] = t;
    }
}

// block k: squared error of candidate k from the interval moments, fixed summation order;
// the last block to finish (ticket, no waiting) picks the winner
constexpr int IV_CURVE_THREADS = 512;
__global__ void __launch_bounds__(IV_CURVE_THREADS) iv_curve_kernel(const qp_iv_total* __restrict__ tot,
                                                                    const float* __restrict__ bb,
                                                                    const unsigned* __restrict__ g_m,
                                                                    const double* __restrict__ outer_tot,
                                                                    const float4* __restrict__ cand,
                                                                    const int* __restrict__ valid, int bits, int steps,
                                                                    int nb, const qp_ds_setup* __restrict__ setup,
                                                                    double* __restrict__ curve,
                                                                    unsigned* __restrict__ ticket,
                                                                    qp_ds_result_t* __restrict__ out,
                                                                    qp_qparams_t* __restrict__ qp_out,
                                                                    unsigned* __restrict__ status)
{
    const int k = blockIdx.x;
    __shared__ double red[IV_CURVE_THREADS / 32];
    __shared__ bool last;
    __shared__ double s_curve[IV_MAX_CAND];
    double total = 0.0;
    const bool ok = valid[k] != 0;
    const float4 q = cand[k];
    const unsigned mask = (1u << bits) - 1u;
    const unsigned m = *g_m;
    const double u = setup->u;
    const float g_lo = setup->g_lo, inv_gw = setup->inv_gw, gw = setup->gw;
    auto level = [&](float r) {      // reconstruction level that candidate k assigns to r
        const unsigned c = qp_code(r, q.x, q.y, q.w, mask);
        return (double)fmaf(__fsub_rn(__uint_as_float(0x4B000000u | c), 8388608.0f), q.z, q.x);
    };
    if (ok) {
        double acc = 0.0;
        // all loads first (independent), then the arithmetic; same summation order as a plain loop
        constexpr int PER = (MAXB + 1 + IV_CURVE_THREADS - 1) / IV_CURVE_THREADS;
        ulonglong2 t[PER];
        float left[PER];
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const unsigned i = threadIdx.x + j * IV_CURVE_THREADS;
            t[j] = make_ulonglong2(0ull, 0ull);
            left[j] = 0.f;
            if (i <= m) {
                t[j] = *reinterpret_cast<const ulonglong2*>(&tot[i]);
                left[j] = bb[i];                                        // an element of the interval: fixes its codes
            }
        }
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if (t[j].x == 0) continue;
            const float r = cell_ref(cell_pm(left[j], g_lo, inv_gw), g_lo, gw);
            const double a = level(left[j]) - (double)r;
            acc += (double)t[j].x * a * a - 2.0 * a * ((double)t[j].y * u);
        }
        total = qp_block_sum(acc, red);
    }
    if (threadIdx.x == 0) {
        double mse = __longlong_as_double(0x7FF0000000000000ll);
        if (ok) {
            const double s1 = outer_tot[0], s1a = outer_tot[1], s2 = outer_tot[2];
            const double s1_lo = 0.5 * (s1a - s1), s1_hi = 0.5 * (s1a + s1);   // sums of the distances beyond each end
            const double s2_in = outer_tot[6];
            const double a_lo = level(setup->g_lo) - (double)setup->g_lo;      // >= 0: below every clip range
            const double a_hi = level(setup->g_hi) - (double)setup->g_hi;      // <= 0: above every clip range
            total += s2_in * (u * u);                  // sum of squared offsets: the same for every candidate
            total += 2.0 * a_lo * s1_lo - 2.0 * a_hi * s1_hi + s2;   // what lies beyond the ends (see IvOuter)
            const unsigned long long nf = setup->n_finite;
            mse = nf ? total / (double)nf : 0.0;
        }
        curve[k] = mse;
        __threadfence();
        last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    if (threadIdx.x == 0) *ticket = 0;
    qp_ds_pick(curve, steps, nb, bits, cand, setup, out, qp_out, status, s_curve);
}

template <typename T>
int32_t interval_typed(qp_ctx* ctx, const T* x, uint64_t n, const qp_stats_t* d_stats, int bits, int bmode, int steps,
                       int nb, double F, qp_ds_result_t* d_out, qp_qparams_t* d_qp_out, cudaStream_t s)
{
    const int ncand = steps + 1;
    const int L1 = (1 << bits) - 1;
    const int nbnd = ncand * L1 + G;
    if (nbnd > MAXB || ncand > IV_MAX_CAND)
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "too many boundaries for the interval path");
    constexpr size_t smem = (size_t)(MAXB + 1) * (8 + 4) + (size_t)(G + 1) * 4 + 16;
    if (cudaFuncSetAttribute(iv_moments_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return qp_check_launch(ctx, "qp_dsaciq_search (interval shared memory)");
    unsigned* g_m = ctx->d_iv_first + G + 2;                 // behind first[0..G+1]
    iv_bounds_kernel<<<MAXB / 256, 256, 0, s>>>(d_stats, ctx->d_hist, nb, bits, bmode, steps, F, ctx->d_cand, ctx->d_valid,
                                                ctx->d_setup, ctx->d_iv_bnd, ctx->d_status);
    iv_rank_kernel<<<MAXB / IV_RANK_PER_BLOCK, 512, 0, s>>>(ctx->d_iv_bnd, ctx->d_setup, ncand * L1, ctx->d_iv_bb,
                                                            ctx->d_iv_first);
    // second form where its 32-bit replica sums cannot wrap: one block per SM, more for longer tensors
    constexpr size_t smem2 = (size_t)(G + 1) * IV2_R * 8 + (size_t)(MAXB + 1) * 12 + (size_t)(G + 1) * 4 +
                             (size_t)IV2_WARPS * IV2_STAGE * 4 + 16;
    uint64_t blocks2 = (uint64_t)ctx->sm_count;
    while (n / blocks2 > IV2_MAX_PER_BLOCK && blocks2 + (uint64_t)ctx->sm_count <= (uint64_t)ctx->iv_blocks)
        blocks2 += (uint64_t)ctx->sm_count;
    const bool second = ctx->moments_form != 1 && n / blocks2 <= IV2_MAX_PER_BLOCK;
    const int blocks = second ? (int)blocks2 : ctx->iv_blocks;
    if (second) {
        if (cudaFuncSetAttribute(iv_moments2_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2) != cudaSuccess)
            return qp_check_launch(ctx, "qp_dsaciq_search (interval shared memory)");
        iv_moments2_kernel<T><<<blocks, IV2_THREADS, smem2, s>>>(x, n, d_stats, ctx->d_setup, ctx->d_iv_bb, ctx->d_iv_first,
                                                                g_m, ctx->d_iv_part, ctx->d_iv_outer);
    } else {
        iv_moments_kernel<T><<<blocks, QP_IV_THREADS, smem, s>>>(x, n, d_stats, ctx->d_setup, ctx->d_iv_bb, ctx->d_iv_first,
                                                                 g_m, ctx->d_iv_part, ctx->d_iv_outer);
    }
    iv_reduce_kernel<<<(MAXB + 1 + 31) / 32, IV_RED_THREADS, 0, s>>>(ctx->d_iv_part, blocks, g_m, ctx->d_iv_tot, ctx->d_iv_outer,
                                                                    ctx->d_iv_outer + (size_t)blocks * 8);
    iv_curve_kernel<<<ncand, IV_CURVE_THREADS, 0, s>>>(ctx->d_iv_tot, ctx->d_iv_bb, g_m, ctx->d_iv_outer + (size_t)blocks * 8,
                                                       ctx->d_cand, ctx->d_valid, bits, steps, nb, ctx->d_setup, ctx->d_curve,
                                                       ctx->d_ticket + 2, d_out, d_qp_out, ctx->d_status);
    ctx->launches += 5;
    return qp_check_launch(ctx, "qp_dsaciq_search (interval path)");
}

}  // namespace

int32_t qp_launch_interval_search(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, const qp_stats_t* d_stats,
                                  int bits, int bmode, int steps, int hist_bins, double F, qp_ds_result_t* d_out,
                                  qp_qparams_t* d_qp_out, cudaStream_t s)
{
    if (dtype == QP_F32)
        return interval_typed<float>(ctx, static_cast<const float*>(d_x), n, d_stats, bits, bmode, steps, hist_bins, F,
                                     d_out, d_qp_out, s);
    return interval_typed<unsigned short>(ctx, static_cast<const unsigned short*>(d_x), n, d_stats, bits, bmode, steps,
                                          hist_bins, F, d_out, d_qp_out, s);
}
