// Token-wise variant of the path (a variant of this library: the paper, Sec. 3, uses one clip range
// per tensor).  The tensor is [tokens, channels], row-major; a token is a row of `channels`
// contiguous elements (one position of a ViT sequence) and gets the statistics, clip range and
// quantizer that the per-tensor functions give for its row alone.  Bit-width and packed layout
// are shared, so the receiver needs the `tokens` quantizers (24 bytes each) with the stream.
//
//   tok_stats_kernel    a warp per token: the row is read once from HBM (sums, min, max), the mean
//                       comes out of a warp reduction, and the second pass over the row (deviations)
//                       finds it in L1; fp32 partials per lane folded into fp64, fixed shuffle order
//   tok_pack_kernel     the per-tensor packer's warp tile (1024 elements = 32 * bits words, coalesced
//                       16-byte loads, quads across the warp through swizzled shared memory) with the
//                       quantizer looked up per 16-byte vector: a vector never straddles two tokens
//                       when `channels` is a multiple of the vector's elements, and a lane's vectors
//                       are 128 elements apart, so the token index moves on by a compare instead of
//                       a division
//   tok_unpack_kernel   the mirror image
//   tok_*_scalar        any shape and alignment: a thread per 32 elements, token by division
#include "qp_internal.cuh"

namespace {

constexpr int TILE = 1024;
constexpr int WARPS = QP_THREADS / 32;

// ---------------------------------------------------------------------------- statistics

template <typename T, bool VEC>
__global__ void __launch_bounds__(QP_THREADS) tok_stats_kernel(const T* __restrict__ x, uint64_t tokens, uint32_t C,
                                                               qp_stats_t* __restrict__ out, unsigned* __restrict__ status)
{
    constexpr int EPV = qp_span<T>::EPV;
    const int lane = threadIdx.x & 31;
    const uint64_t wstride = (uint64_t)gridDim.x * WARPS;
    const float inf = __int_as_float(0x7F800000);
    bool any_bad = false;
    for (uint64_t t = (uint64_t)blockIdx.x * WARPS + (threadIdx.x >> 5); t < tokens; t += wstride) {
        const T* row = x + t * C;
        double s = 0.0, sa = 0.0;
        float mn = inf, mx = -inf;
        unsigned bad = 0;
        auto first = [&](float v) {
            if (qp_is_finite(v)) { s += (double)v; sa += (double)fabsf(v); mn = fminf(mn, v); mx = fmaxf(mx, v); }
            else ++bad;
        };
        if (VEC) {
            for (uint32_t v0 = lane; v0 < C / EPV; v0 += 32) {
                float e[EPV];
                qp_load_vec(row + (size_t)v0 * EPV, e);
                float ps = 0.f, psa = 0.f;
#pragma unroll
                for (int i = 0; i < EPV; ++i) { ps += e[i]; psa += fabsf(e[i]); mn = fminf(mn, e[i]); mx = fmaxf(mx, e[i]); }
                if (psa < inf) { s += (double)ps; sa += (double)psa; }
                else {                                       // a NaN or Inf among them (min/max may hold it: redone below)
                    mn = inf; mx = -inf; bad = 0xFFFFFFFFu;
                }
            }
            if (__any_sync(0xFFFFFFFFu, bad == 0xFFFFFFFFu)) {   // rare: the whole row again, element by element
                s = 0.0; sa = 0.0; mn = inf; mx = -inf; bad = 0;
                for (uint32_t i = lane; i < C; i += 32) first(qp_load_one(row + i));
            }
        } else {
            for (uint32_t i = lane; i < C; i += 32) first(qp_load_one(row + i));
        }
        for (int o = 16; o > 0; o >>= 1) {                   // fixed order: bit-reproducible
            s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
            sa += __shfl_xor_sync(0xFFFFFFFFu, sa, o);
            mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, o));
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
            bad += __shfl_xor_sync(0xFFFFFFFFu, bad, o);
        }
        const unsigned nf = C - bad;
        const double mean = nf ? s / (double)nf : 0.0;
        const float m_hi = (float)mean, m_lo = (float)(mean - (double)m_hi);   // the mean as an unevaluated fp32 pair
        double sd = 0.0, sv = 0.0;
        auto second = [&](float v, float& d1, float& d2) {
            if (qp_is_finite(v)) {
                const float d = __fsub_rn(__fsub_rn(v, m_hi), m_lo);
                d1 += fabsf(d);
                d2 = fmaf(d, d, d2);
            }
        };
        if (VEC) {
            for (uint32_t v0 = lane; v0 < C / EPV; v0 += 32) {
                float e[EPV];
                qp_load_vec(row + (size_t)v0 * EPV, e);
                float d1 = 0.f, d2 = 0.f;
#pragma unroll
                for (int i = 0; i < EPV; ++i) second(e[i], d1, d2);
                sd += (double)d1;
                sv += (double)d2;
            }
        } else {
            for (uint32_t i = lane; i < C; i += 32) {
                float d1 = 0.f, d2 = 0.f;
                second(qp_load_one(row + i), d1, d2);
                sd += (double)d1;
                sv += (double)d2;
            }
        }
        for (int o = 16; o > 0; o >>= 1) {
            sd += __shfl_xor_sync(0xFFFFFFFFu, sd, o);
            sv += __shfl_xor_sync(0xFFFFFFFFu, sv, o);
        }
        if (lane == 0) {
            qp_stats_t st;
            st.n = C;
            st.nonfinite = bad;
            st.mean = mean;
            st.mean_abs = nf ? sa / (double)nf : 0.0;
            st.mad = nf ? sd / (double)nf : 0.0;
            st.var = nf ? sv / (double)nf : 0.0;
            st.min = nf ? (double)mn : 0.0;
            st.max = nf ? (double)mx : 0.0;
            st.hist_peak = 0;
            st.hist_bins = 0;
            st.reserved = 0;
            out[t] = st;
        }
        any_bad |= bad != 0;
    }
    if (any_bad && lane == 0) atomicOr(status, QP_DEV_NONFINITE);
}

__global__ void __launch_bounds__(128) tok_clip_kernel(const qp_stats_t* __restrict__ st, uint64_t tokens, int bits, int method,
                                                       int dist, int bmode, double F, qp_qparams_t* __restrict__ qp_out,
                                                       unsigned* __restrict__ status)
{
    const uint64_t t = (uint64_t)blockIdx.x * 128 + threadIdx.x;
    if (t >= tokens) return;
    double lo, hi;
    qp_clip_ends(st[t], method, dist, bmode, bits, F, lo, hi);
    qp_qparams_t q;
    const int rc = qp_fill_qparams(lo, hi, bits, &q);
    qp_out[t] = q;
    if (rc == QP_WARN_DEGENERATE) atomicOr(status, QP_DEV_DEGENERATE);
}

// ---------------------------------------------------------------------------- quantize + pack

__device__ __forceinline__ int swz(int p) { return ((((p >> 2) ^ ((p >> 5) & 1)) << 2) | (p & 3)); }

// token and position inside it of element `el`; then moved on by `step` elements at a time
struct TokCursor {
    uint64_t tok;
    uint32_t rem, C;
    __device__ __forceinline__ TokCursor(uint64_t el, uint32_t channels) : tok(el / channels), rem((uint32_t)(el % channels)), C(channels) {}
    __device__ __forceinline__ void advance(uint32_t step)
    {
        rem += step;
        while (rem >= C) { rem -= C; ++tok; }
    }
};

// Fast path: x 16-byte aligned, channels a multiple of the vector's elements (a vector lies in one token).
template <int BITS, typename T>
__global__ void __launch_bounds__(QP_THREADS) tok_pack_kernel(const T* __restrict__ x, uint64_t ntiles, uint32_t C,
                                                              const qp_qparams_t* __restrict__ d_qp,
                                                              uint32_t* __restrict__ out, unsigned* __restrict__ status)
{
    constexpr int EPV = qp_span<T>::EPV;
    constexpr int NLOAD = TILE / (32 * EPV);
    __shared__ __align__(16) uint32_t stage[WARPS][256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* sw = stage[warp];
    const uint64_t wstride = (uint64_t)gridDim.x * WARPS;
    constexpr unsigned mask = (1u << BITS) - 1u;
    bool mismatch = false;
    for (uint64_t tile = (uint64_t)blockIdx.x * WARPS + warp; tile < ntiles; tile += wstride) {
        const T* xt = x + tile * TILE;
        float e[NLOAD][EPV];
#pragma unroll
        for (int j = 0; j < NLOAD; ++j) qp_load_vec(xt + (j * 32 + lane) * EPV, e[j]);
        TokCursor cur(tile * TILE + (uint64_t)lane * EPV, C);
#pragma unroll
        for (int j = 0; j < NLOAD; ++j) {
            const qp_qparams_t* q = d_qp + cur.tok;
            const float lo = __ldg(&q->lo), hi = __ldg(&q->hi), inv = __ldg(&q->inv_scale);
            mismatch |= __ldg(&q->bits) != BITS;
            unsigned quads[EPV / 4];
#pragma unroll
            for (int h = 0; h < EPV / 4; ++h) {
                unsigned r = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) r |= qp_code(e[j][4 * h + i], lo, hi, inv, mask) << (BITS * i);
                quads[h] = r;
            }
            if constexpr (EPV == 4) sw[swz(j * 32 + lane)] = quads[0];
            else *reinterpret_cast<uint2*>(&sw[swz(2 * (j * 32 + lane))]) = make_uint2(quads[0], quads[1]);
            cur.advance(32 * EPV);
        }
        __syncwarp();
        const uint4 a = *reinterpret_cast<const uint4*>(&sw[swz(8 * lane)]);
        const uint4 b = *reinterpret_cast<const uint4*>(&sw[swz(8 * lane + 4)]);
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
    if (mismatch) atomicOr(status, QP_DEV_BITS_MISMATCH);
}

// Any shape: thread t packs elements [first + 32t, first + 32t + 32) that exist into `bits` words (16 bits:
// 16 words) and writes those below nwords.
template <typename T>
__global__ void __launch_bounds__(QP_THREADS) tok_pack_scalar(const T* __restrict__ x, uint64_t first, uint64_t n, uint32_t C,
                                                              int bits, const qp_qparams_t* __restrict__ d_qp,
                                                              uint32_t* __restrict__ out, uint64_t nwords,
                                                              unsigned* __restrict__ status)
{
    const uint64_t t = (uint64_t)blockIdx.x * QP_THREADS + threadIdx.x;
    const uint64_t w0 = t * (uint64_t)bits;
    if (w0 >= nwords) return;
    const unsigned mask = (1u << bits) - 1u;
    uint32_t w[16];
#pragma unroll
    for (int m = 0; m < 16; ++m) w[m] = 0u;
    const uint64_t e0 = first + t * 32;
    bool mismatch = false;
    if (e0 < n) {
        TokCursor cur(e0, C);
        for (int i = 0; i < 32 && e0 + i < n; ++i) {
            const qp_qparams_t* q = d_qp + cur.tok;
            mismatch |= __ldg(&q->bits) != bits;
            const unsigned c = qp_code(qp_load_one(x + e0 + i), __ldg(&q->lo), __ldg(&q->hi), __ldg(&q->inv_scale), mask);
            const int bit = i * bits, word = bit >> 5, sh = bit & 31;
            w[word] |= c << sh;
            if (sh + bits > 32) w[word + 1] |= c >> (32 - sh);
            cur.advance(1);
        }
    }
    for (int m = 0; m < bits; ++m)
        if (w0 + m < nwords) out[w0 + m] = w[m];
    if (mismatch) atomicOr(status, QP_DEV_BITS_MISMATCH);
}

// ---------------------------------------------------------------------------- unpack + dequantize

__device__ __forceinline__ float tok_code_to_float(unsigned c) { return __fsub_rn(__uint_as_float(0x4B000000u | c), 8388608.0f); }

__device__ __forceinline__ void tok_store4(float* y, uint64_t el, const float (&v)[4])
{
    __stcs(reinterpret_cast<float4*>(y + el), make_float4(v[0], v[1], v[2], v[3]));
}
__device__ __forceinline__ void tok_store4(unsigned short* y, uint64_t el, const float (&v)[4])
{
    uint2 o;
    o.x = (unsigned)qp_f32_to_bf16(v[0]) | ((unsigned)qp_f32_to_bf16(v[1]) << 16);
    o.y = (unsigned)qp_f32_to_bf16(v[2]) | ((unsigned)qp_f32_to_bf16(v[3]) << 16);
    __stcs(reinterpret_cast<uint2*>(y + el), o);
}
__device__ __forceinline__ void tok_store1(float* y, uint64_t el, float v) { y[el] = v; }
__device__ __forceinline__ void tok_store1(unsigned short* y, uint64_t el, float v) { y[el] = qp_f32_to_bf16(v); }

// Fast path: y aligned for 4-element stores, channels a multiple of 4.
template <int BITS, typename TO>
__global__ void __launch_bounds__(QP_THREADS) tok_unpack_kernel(const uint32_t* __restrict__ in, uint64_t ntiles, uint32_t C,
                                                                const qp_qparams_t* __restrict__ d_qp, TO* __restrict__ y,
                                                                unsigned* __restrict__ status)
{
    __shared__ __align__(16) uint32_t stage[WARPS][256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* sw = stage[warp];
    const uint64_t wstride = (uint64_t)gridDim.x * WARPS;
    constexpr unsigned MASK = (1u << BITS) - 1u;
    constexpr int QB = 4 * BITS;
    constexpr unsigned QMASK = QB >= 32 ? 0xFFFFFFFFu : ((1u << (QB & 31)) - 1u);
    bool mismatch = false;
    for (uint64_t tile = (uint64_t)blockIdx.x * WARPS + warp; tile < ntiles; tile += wstride) {
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
        *reinterpret_cast<uint4*>(&sw[swz(8 * lane)]) = make_uint4(qd[0], qd[1], qd[2], qd[3]);
        *reinterpret_cast<uint4*>(&sw[swz(8 * lane + 4)]) = make_uint4(qd[4], qd[5], qd[6], qd[7]);
        __syncwarp();
        uint32_t mine[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) mine[j] = sw[swz(j * 32 + lane)];
        TokCursor cur(tile * TILE + (uint64_t)lane * 4, C);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const qp_qparams_t* q = d_qp + cur.tok;
            const float lo = __ldg(&q->lo), scale = __ldg(&q->scale);
            mismatch |= __ldg(&q->bits) != BITS;
            float v[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) v[i] = fmaf(tok_code_to_float((mine[j] >> (BITS * i)) & MASK), scale, lo);
            tok_store4(y, tile * TILE + (uint64_t)(j * 32 + lane) * 4, v);
            cur.advance(128);
        }
        __syncwarp();
    }
    if (mismatch) atomicOr(status, QP_DEV_BITS_MISMATCH);
}

template <typename TO>
__global__ void __launch_bounds__(QP_THREADS) tok_unpack_scalar(const uint32_t* __restrict__ in, uint64_t first, uint64_t n,
                                                                uint32_t C, int bits, const qp_qparams_t* __restrict__ d_qp,
                                                                TO* __restrict__ y, unsigned* __restrict__ status)
{
    const uint64_t t = (uint64_t)blockIdx.x * QP_THREADS + threadIdx.x;
    const uint64_t e0 = first + t * 32;
    if (e0 >= n) return;
    const uint32_t* wp = in + t * (uint64_t)bits;          // `in` already points at the word of element `first`
    const unsigned mask = (1u << bits) - 1u;
    const int cnt = (int)((n - e0) < 32 ? (n - e0) : 32);
    const int nw = (cnt * bits + 31) >> 5;
    uint32_t w[17];
#pragma unroll
    for (int m = 0; m < 17; ++m) w[m] = 0u;
    for (int m = 0; m < nw; ++m) w[m] = __ldg(wp + m);
    TokCursor cur(e0, C);
    bool mismatch = false;
    for (int i = 0; i < cnt; ++i) {
        const qp_qparams_t* q = d_qp + cur.tok;
        mismatch |= __ldg(&q->bits) != bits;
        const int bit = i * bits, word = bit >> 5, sh = bit & 31;
        uint32_t c = w[word] >> sh;
        if (sh + bits > 32) c |= w[word + 1] << (32 - sh);
        tok_store1(y, e0 + i, fmaf(tok_code_to_float(c & mask), __ldg(&q->scale), __ldg(&q->lo)));
        cur.advance(1);
    }
    if (mismatch) atomicOr(status, QP_DEV_BITS_MISMATCH);
}

// ---------------------------------------------------------------------------- host side

int32_t tok_check(qp_ctx* ctx, uint64_t tokens, uint32_t channels)
{
    if (channels < 1) return qp_fail(ctx, QP_ERR_INVALID_ARG, "channels must be at least 1");
    if (tokens >= (1ull << 40) / channels) return qp_fail(ctx, QP_ERR_INVALID_ARG, "tensor too large");
    return QP_OK;
}

unsigned tok_grid(qp_ctx* ctx, uint64_t warps_wanted)
{
    const uint64_t want = (warps_wanted + WARPS - 1) / WARPS;
    const uint64_t cap = (uint64_t)ctx->sm_count * 64;
    return (unsigned)(want < 1 ? 1 : (want < cap ? want : cap));
}

template <typename T>
int32_t pack_tokens_typed(qp_ctx* ctx, const T* x, uint64_t n, uint32_t C, int bits, const qp_qparams_t* d_qp, void* d_packed,
                          cudaStream_t s)
{
    constexpr int EPV = qp_span<T>::EPV;
    uint32_t* out = static_cast<uint32_t*>(d_packed);
    const bool fast = bits <= 8 && C % EPV == 0 && ((uintptr_t)x & 15u) == 0;
    const uint64_t ntiles = fast ? n / TILE : 0;
    if (ntiles) {
        const unsigned blocks = tok_grid(ctx, ntiles);
        ctx->launches += 1;
#define QP_TOK_PACK(B) case B: tok_pack_kernel<B, T><<<blocks, QP_THREADS, 0, s>>>(x, ntiles, C, d_qp, out, ctx->d_status); break;
        switch (bits) {
            QP_TOK_PACK(1) QP_TOK_PACK(2) QP_TOK_PACK(3) QP_TOK_PACK(4) QP_TOK_PACK(5) QP_TOK_PACK(6) QP_TOK_PACK(7) QP_TOK_PACK(8)
        }
#undef QP_TOK_PACK
    }
    const uint64_t done_words = ntiles * 32 * (uint64_t)bits;
    const uint64_t total_words = qp_packed_bytes(n, bits) / 4;
    if (total_words > done_words) {
        const uint64_t nwords = total_words - done_words;
        const uint64_t threads = (nwords + bits - 1) / bits;
        const uint64_t blocks = (threads + QP_THREADS - 1) / QP_THREADS;
        ctx->launches += 1;
        tok_pack_scalar<T><<<(unsigned)blocks, QP_THREADS, 0, s>>>(x, ntiles * TILE, n, C, bits, d_qp, out + done_words, nwords,
                                                                    ctx->d_status);
    }
    return qp_check_launch(ctx, "qp_quantize_pack_tokens");
}

template <typename TO>
int32_t unpack_tokens_typed(qp_ctx* ctx, const void* d_packed, uint64_t n, uint32_t C, int bits, const qp_qparams_t* d_qp, TO* y,
                            cudaStream_t s)
{
    const uint32_t* in = static_cast<const uint32_t*>(d_packed);
    const bool fast = bits <= 8 && C % 4 == 0 && ((uintptr_t)y & (4 * sizeof(TO) - 1)) == 0;
    const uint64_t ntiles = fast ? n / TILE : 0;
    if (ntiles) {
        const unsigned blocks = tok_grid(ctx, ntiles);
        ctx->launches += 1;
#define QP_TOK_UNPACK(B) case B: tok_unpack_kernel<B, TO><<<blocks, QP_THREADS, 0, s>>>(in, ntiles, C, d_qp, y, ctx->d_status); break;
        switch (bits) {
            QP_TOK_UNPACK(1) QP_TOK_UNPACK(2) QP_TOK_UNPACK(3) QP_TOK_UNPACK(4) QP_TOK_UNPACK(5) QP_TOK_UNPACK(6) QP_TOK_UNPACK(7)
            QP_TOK_UNPACK(8)
        }
#undef QP_TOK_UNPACK
    }
    const uint64_t first = ntiles * TILE;
    if (n > first) {
        const uint64_t threads = (n - first + 31) / 32;
        const uint64_t blocks = (threads + QP_THREADS - 1) / QP_THREADS;
        ctx->launches += 1;
        tok_unpack_scalar<TO><<<(unsigned)blocks, QP_THREADS, 0, s>>>(in + ntiles * 32 * (uint64_t)bits, first, n, C, bits, d_qp, y,
                                                                      ctx->d_status);
    }
    return qp_check_launch(ctx, "qp_unpack_dequantize_tokens");
}

}  // namespace

extern "C" int32_t qp_stats_tokens(qp_ctx* ctx, const void* d_x, int dtype, uint64_t tokens, uint32_t channels,
                                   qp_stats_t* d_out, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (dtype != QP_F32 && dtype != QP_BF16) return qp_fail(ctx, QP_ERR_UNSUPPORTED_DTYPE, "dtype must be QP_F32 or QP_BF16");
    int32_t rc = tok_check(ctx, tokens, channels);
    if (rc) return rc;
    if ((tokens > 0 && (!d_x || !d_out))) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null pointer");
    if (((uintptr_t)d_x & (dtype == QP_F32 ? 3u : 1u)) || ((uintptr_t)d_out & 7u))
        return qp_fail(ctx, QP_ERR_ALIGNMENT, "tensor or d_out not aligned");
    if (tokens == 0) return QP_OK;
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const unsigned blocks = tok_grid(ctx, tokens);
    const bool aligned = ((uintptr_t)d_x & 15u) == 0;
    if (dtype == QP_F32) {
        const float* x = static_cast<const float*>(d_x);
        if (aligned && channels % 4 == 0) tok_stats_kernel<float, true><<<blocks, QP_THREADS, 0, s>>>(x, tokens, channels, d_out, ctx->d_status);
        else tok_stats_kernel<float, false><<<blocks, QP_THREADS, 0, s>>>(x, tokens, channels, d_out, ctx->d_status);
    } else {
        const unsigned short* x = static_cast<const unsigned short*>(d_x);
        if (aligned && channels % 8 == 0) tok_stats_kernel<unsigned short, true><<<blocks, QP_THREADS, 0, s>>>(x, tokens, channels, d_out, ctx->d_status);
        else tok_stats_kernel<unsigned short, false><<<blocks, QP_THREADS, 0, s>>>(x, tokens, channels, d_out, ctx->d_status);
    }
    ctx->launches += 1;
    return qp_check_launch(ctx, "qp_stats_tokens");
}

extern "C" int32_t qp_clip_qparams_tokens_device(qp_ctx* ctx, const qp_stats_t* d_stats, uint64_t tokens, int bits, int method,
                                                 int dist, int bmode, qp_qparams_t* d_qp_out, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (tokens >= (1ull << 40)) return qp_fail(ctx, QP_ERR_INVALID_ARG, "too many tokens");
    if (tokens > 0 && (!d_stats || !d_qp_out)) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null pointer");
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    if (!qp_clip_method_closed_form(method))
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "method must be ACIQ (| INTERSECT) or MINMAX, optionally | MIDRISE");
    if ((dist != QP_DIST_LAPLACE && dist != QP_DIST_GAUSS) || (bmode != QP_B_MAD && bmode != QP_B_MEAN_ABS))
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "dist/bmode");
    if (tokens == 0) return QP_OK;
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    tok_clip_kernel<<<(unsigned)((tokens + 127) / 128), 128, 0, static_cast<cudaStream_t>(stream)>>>(
        d_stats, tokens, bits, method, dist, bmode, qp_host_aciq_F(bits, dist), d_qp_out, ctx->d_status);
    ctx->launches += 1;
    return qp_check_launch(ctx, "qp_clip_qparams_tokens_device");
}

extern "C" int32_t qp_quantize_pack_tokens(qp_ctx* ctx, const void* d_x, int dtype, uint64_t tokens, uint32_t channels, int bits,
                                           const qp_qparams_t* d_qp, void* d_packed, uint64_t packed_capacity, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (dtype != QP_F32 && dtype != QP_BF16) return qp_fail(ctx, QP_ERR_UNSUPPORTED_DTYPE, "dtype must be QP_F32 or QP_BF16");
    int32_t rc = tok_check(ctx, tokens, channels);
    if (rc) return rc;
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    const uint64_t n = tokens * channels;
    const uint64_t need = qp_packed_bytes(n, bits);
    if (packed_capacity < need) return qp_fail(ctx, QP_ERR_BUFFER_TOO_SMALL, "packed_capacity < qp_packed_bytes(n, bits)");
    if (n > 0 && (!d_qp || !d_x || !d_packed)) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null pointer");
    if (((uintptr_t)d_x & (dtype == QP_F32 ? 3u : 1u)) || ((uintptr_t)d_packed & 15u) || ((uintptr_t)d_qp & 3u))
        return qp_fail(ctx, QP_ERR_ALIGNMENT, "tensor, d_packed (16 bytes) or d_qp not aligned");
    if (n == 0) return QP_OK;
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (dtype == QP_F32) return pack_tokens_typed<float>(ctx, static_cast<const float*>(d_x), n, channels, bits, d_qp, d_packed, s);
    return pack_tokens_typed<unsigned short>(ctx, static_cast<const unsigned short*>(d_x), n, channels, bits, d_qp, d_packed, s);
}

extern "C" int32_t qp_unpack_dequantize_tokens(qp_ctx* ctx, const void* d_packed, uint64_t tokens, uint32_t channels, int bits,
                                               const qp_qparams_t* d_qp, void* d_y, int out_dtype, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (out_dtype != QP_F32 && out_dtype != QP_BF16) return qp_fail(ctx, QP_ERR_UNSUPPORTED_DTYPE, "out_dtype");
    int32_t rc = tok_check(ctx, tokens, channels);
    if (rc) return rc;
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    const uint64_t n = tokens * channels;
    if (n > 0 && (!d_qp || !d_packed || !d_y)) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null pointer");
    if (((uintptr_t)d_packed & 15u) || ((uintptr_t)d_qp & 3u) || ((uintptr_t)d_y & (out_dtype == QP_F32 ? 3u : 1u)))
        return qp_fail(ctx, QP_ERR_ALIGNMENT, "d_packed (16 bytes), d_qp or d_y not aligned");
    if (n == 0) return QP_OK;
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (out_dtype == QP_F32) return unpack_tokens_typed<float>(ctx, d_packed, n, channels, bits, d_qp, static_cast<float*>(d_y), s);
    return unpack_tokens_typed<unsigned short>(ctx, d_packed, n, channels, bits, d_qp, static_cast<unsigned short*>(d_y), s);
}

// The token-wise sender in one call: statistics -> per-token clip -> quantize+pack, nothing read back to the
// host.  d_stats_work: device memory for `tokens` statistics (80 bytes each), the caller's.
extern "C" int32_t qp_sender_tokens_device(qp_ctx* ctx, const void* d_x, int dtype, uint64_t tokens, uint32_t channels, int bits,
                                           int method, int bmode, void* d_packed, uint64_t packed_capacity,
                                           qp_qparams_t* d_qp_out, qp_stats_t* d_stats_work, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (tokens > 0 && (!d_qp_out || !d_stats_work)) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null d_qp_out / d_stats_work");
    int32_t rc = qp_stats_tokens(ctx, d_x, dtype, tokens, channels, d_stats_work, stream);
    if (rc < 0) return rc;
    rc = qp_clip_qparams_tokens_device(ctx, d_stats_work, tokens, bits, method, QP_DIST_LAPLACE, bmode, d_qp_out, stream);
    if (rc < 0) return rc;
    return qp_quantize_pack_tokens(ctx, d_x, dtype, tokens, channels, bits, d_qp_out, d_packed, packed_capacity, stream);
}
