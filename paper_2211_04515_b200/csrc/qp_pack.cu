// a5: clamp + uniform quantize + bit-pack (paper Sec. 3: uniform quantization of the clipped
// activation; the packed layout is this library's: element i owns stream bits
// [i*bits, (i+1)*bits), LSB first).
//
// HBM-bound: 4 (or 2) bytes read and bits/8 bytes written per element.
//
// Fast path, bits 1..8.  A warp owns a tile of 1024 consecutive elements, which is exactly
// 32*bits output words.  Loads are fully coalesced 16-byte vectors (lane l takes vector
// j*32+l, all of them issued before first use).  Each group of 4 consecutive elements is
// quantized to a "quad" of 4*bits bits; quads cross the warp through 1 KB of shared memory
// (chunk-swizzled, conflict-free both ways) so that every lane ends up with the 8 quads of
// 32 consecutive elements = `bits` whole 32-bit words, which it stores as the widest aligned
// vector (bits 1,2,4,8) or, for the other widths, through shared memory again so that global
// stores are 128-byte coalesced.
//
// bits = 16: one uint16 per element, plain vectorised map.
// Ragged tails (n mod 1024), pad bytes and misaligned inputs go through a scalar kernel.
#include "qp_internal.cuh"

namespace {

constexpr int TILE = 1024;                 // elements per warp tile
constexpr int WARPS = QP_THREADS / 32;

struct QP4 { float lo, hi, inv; unsigned mask; };

__device__ __forceinline__ QP4 load_qp(const qp_qparams_t* __restrict__ d_qp, const qp_qparams_t& h_qp, int bits,
                                       unsigned* status)
{
    QP4 q;
    if (d_qp) {
        q.lo = __ldg(&d_qp->lo); q.hi = __ldg(&d_qp->hi); q.inv = __ldg(&d_qp->inv_scale);
        if (blockIdx.x == 0 && threadIdx.x == 0 && __ldg(&d_qp->bits) != bits) atomicOr(status, QP_DEV_BITS_MISMATCH);
    } else {
        q.lo = h_qp.lo; q.hi = h_qp.hi; q.inv = h_qp.inv_scale;
    }
    q.mask = (bits >= 32) ? 0xFFFFFFFFu : ((1u << bits) - 1u);
    return q;
}

// physical word of quad p in a warp's 256-word staging buffer: 16-byte chunk index XOR bit 3
__device__ __forceinline__ int swz(int p) { return ((((p >> 2) ^ ((p >> 5) & 1)) << 2) | (p & 3)); }

template <int BITS>
__device__ __forceinline__ unsigned quad_of(const float* e, const QP4& q)
{
    unsigned r = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) r |= qp_code(e[i], q.lo, q.hi, q.inv, q.mask) << (BITS * i);
    return r;
}

template <int BITS, typename T>
__global__ void __launch_bounds__(QP_THREADS) pack_kernel(const T* __restrict__ x, uint64_t ntiles,
                                                          const qp_qparams_t* __restrict__ d_qp, qp_qparams_t h_qp,
                                                          uint32_t* __restrict__ out, unsigned* __restrict__ status,
                                                          int reverse)
{
    constexpr int EPV = qp_span<T>::EPV;          // 4 (f32) or 8 (bf16) elements per 16-byte vector
    constexpr int NLOAD = TILE / (32 * EPV);      // 8 or 4 vector loads per lane
    __shared__ __align__(16) uint32_t stage[WARPS][256];
    const QP4 q = load_qp(d_qp, h_qp, BITS, status);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* sw = stage[warp];
    const uint64_t wstride = (uint64_t)gridDim.x * WARPS;

    // `reverse`: the grid walks the tensor from its end (the tiles are the same), for a call that
    // follows a pass which ended there and left that part of x in L2
    for (uint64_t it = (uint64_t)blockIdx.x * WARPS + warp; it < ntiles; it += wstride) {
        const uint64_t tile = reverse ? ntiles - 1 - it : it;
        const T* xt = x + tile * TILE;
        float e[NLOAD][EPV];
#pragma unroll
        for (int j = 0; j < NLOAD; ++j) qp_load_vec(xt + (j * 32 + lane) * EPV, e[j]);
#pragma unroll
        for (int j = 0; j < NLOAD; ++j) {
            if constexpr (EPV == 4) {
                sw[swz(j * 32 + lane)] = quad_of<BITS>(e[j], q);
            } else {
                uint2 two;
                two.x = quad_of<BITS>(e[j], q);
                two.y = quad_of<BITS>(e[j] + 4, q);
                *reinterpret_cast<uint2*>(&sw[swz(2 * (j * 32 + lane))]) = two;
            }
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
        if constexpr (BITS == 8) {
            uint4* o = reinterpret_cast<uint4*>(ot + lane * 8);
            o[0] = make_uint4(w[0], w[1], w[2], w[3]);
            o[1] = make_uint4(w[4], w[5], w[6], w[7]);
        } else if constexpr (BITS == 4) {
            *reinterpret_cast<uint4*>(ot + lane * 4) = make_uint4(w[0], w[1], w[2], w[3]);
        } else if constexpr (BITS == 2) {
            *reinterpret_cast<uint2*>(ot + lane * 2) = make_uint2(w[0], w[1]);
        } else if constexpr (BITS == 1) {
            ot[lane] = w[0];
        } else {
            __syncwarp();
#pragma unroll
            for (int m = 0; m < BITS; ++m) sw[lane * BITS + m] = w[m];
            __syncwarp();
#pragma unroll
            for (int m = 0; m < BITS; ++m) ot[m * 32 + lane] = sw[m * 32 + lane];
        }
        __syncwarp();
    }
}

// Scalar path: thread t packs elements [first + 32t, first + 32t + 32) that exist (missing
// ones count as code 0) into `bits` words, and writes those below nwords.
template <typename T>
__global__ void __launch_bounds__(QP_THREADS) pack_tail_kernel(const T* __restrict__ x, uint64_t first, uint64_t n,
                                                               int bits, const qp_qparams_t* __restrict__ d_qp,
                                                               qp_qparams_t h_qp, uint32_t* __restrict__ out,
                                                               uint64_t nwords, unsigned* __restrict__ status)
{
    const QP4 q = load_qp(d_qp, h_qp, bits, status);
    const uint64_t t = (uint64_t)blockIdx.x * QP_THREADS + threadIdx.x;
    const uint64_t w0 = t * (uint64_t)bits;
    if (w0 >= nwords) return;
    uint32_t w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const uint64_t e0 = first + t * 32;
    for (int i = 0; i < 32; ++i) {
        const uint64_t idx = e0 + i;
        if (idx >= n) break;
        const unsigned c = qp_code(qp_load_one(x + idx), q.lo, q.hi, q.inv, q.mask);
        const int bit = i * bits, word = bit >> 5, sh = bit & 31;
        w[word] |= c << sh;
        if (sh + bits > 32) w[word + 1] |= c >> (32 - sh);
    }
    for (int m = 0; m < bits; ++m)
        if (w0 + m < nwords) out[w0 + m] = w[m];
}

// bits = 16: thread t converts the 8 elements [8t, 8t+8) to one 16-byte vector of uint16 codes.
template <typename T, bool ALIGNED>
__global__ void __launch_bounds__(QP_THREADS) pack16_kernel(const T* __restrict__ x, uint64_t n,
                                                            const qp_qparams_t* __restrict__ d_qp, qp_qparams_t h_qp,
                                                            uint4* __restrict__ out, uint64_t nvec_out,
                                                            unsigned* __restrict__ status)
{
    const QP4 q = load_qp(d_qp, h_qp, 16, status);
    const uint64_t stride = (uint64_t)gridDim.x * QP_THREADS;
    for (uint64_t v = (uint64_t)blockIdx.x * QP_THREADS + threadIdx.x; v < nvec_out; v += stride) {
        float e[8];
        const uint64_t e0 = v * 8;
        if (ALIGNED && e0 + 8 <= n) {
            if constexpr (sizeof(T) == 4) {
                float a[4], b[4];
                qp_load_vec(x + e0, a);
                qp_load_vec(x + e0 + 4, b);
#pragma unroll
                for (int i = 0; i < 4; ++i) { e[i] = a[i]; e[4 + i] = b[i]; }
            } else {
                qp_load_vec(x + e0, e);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) e[i] = (e0 + i < n) ? qp_load_one(x + e0 + i) : __int_as_float(0x7FC00000);
        }
        unsigned c[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) c[i] = (e0 + i < n) ? qp_code(e[i], q.lo, q.hi, q.inv, q.mask) : 0u;
        out[v] = make_uint4(c[0] | (c[1] << 16), c[2] | (c[3] << 16), c[4] | (c[5] << 16), c[6] | (c[7] << 16));
    }
}

template <typename T>
int32_t pack_typed(qp_ctx* ctx, const T* x, uint64_t n, int bits, const qp_qparams_t* d_qp, const qp_qparams_t& h_qp,
                   void* d_packed, cudaStream_t s)
{
    const bool aligned = ((uintptr_t)x & 15u) == 0;
    if (bits == 16) {
        const uint64_t nvec_out = qp_packed_bytes(n, 16) / 16;
        uint64_t want = (nvec_out + QP_THREADS - 1) / QP_THREADS;
        const uint64_t cap = (uint64_t)ctx->sm_count * 64;
        const int blocks = (int)(want > cap ? cap : want);
        ctx->launches += 1;
        if (aligned)
            pack16_kernel<T, true><<<blocks, QP_THREADS, 0, s>>>(x, n, d_qp, h_qp, static_cast<uint4*>(d_packed), nvec_out, ctx->d_status);
        else
            pack16_kernel<T, false><<<blocks, QP_THREADS, 0, s>>>(x, n, d_qp, h_qp, static_cast<uint4*>(d_packed), nvec_out, ctx->d_status);
        return qp_check_launch(ctx, "qp_quantize_pack");
    }
    const uint64_t ntiles = aligned ? n / TILE : 0;
    uint32_t* out = static_cast<uint32_t*>(d_packed);
    // a hint, not a dependency: start where the last pass over this tensor stopped
    const int reverse = (ctx->last_x == static_cast<const void*>(x) && ctx->last_x_end) ? 1 : 0;
    ctx->last_x = x;
    ctx->last_x_end = reverse ? 0 : 1;
    if (ntiles) {
        uint64_t want = (ntiles + WARPS - 1) / WARPS;
        const uint64_t cap = (uint64_t)ctx->sm_count * 64;
        const int blocks = (int)(want > cap ? cap : want);
        ctx->launches += 1;
#define QP_PACK_CASE(B) case B: pack_kernel<B, T><<<blocks, QP_THREADS, 0, s>>>(x, ntiles, d_qp, h_qp, out, ctx->d_status, reverse); break;
        switch (bits) {
            QP_PACK_CASE(1) QP_PACK_CASE(2) QP_PACK_CASE(3) QP_PACK_CASE(4)
            QP_PACK_CASE(5) QP_PACK_CASE(6) QP_PACK_CASE(7) QP_PACK_CASE(8)
        }
#undef QP_PACK_CASE
    }
    const uint64_t done_words = ntiles * 32 * (uint64_t)bits;
    const uint64_t total_words = qp_packed_bytes(n, bits) / 4;
    if (total_words > done_words) {
        const uint64_t nwords = total_words - done_words;
        const uint64_t threads = (nwords + bits - 1) / bits;
        const uint64_t blocks = (threads + QP_THREADS - 1) / QP_THREADS;
        ctx->launches += 1;
        pack_tail_kernel<T><<<(unsigned)blocks, QP_THREADS, 0, s>>>(x, ntiles * TILE, n, bits, d_qp, h_qp,
                                                                     out + done_words, nwords, ctx->d_status);
    }
    return qp_check_launch(ctx, "qp_quantize_pack");
}

}  // namespace

int32_t qp_launch_pack(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int bits, const qp_qparams_t* d_qp,
                       qp_qparams_t h_qp, void* d_packed, cudaStream_t s)
{
    if (dtype == QP_F32) return pack_typed<float>(ctx, static_cast<const float*>(d_x), n, bits, d_qp, h_qp, d_packed, s);
    return pack_typed<unsigned short>(ctx, static_cast<const unsigned short*>(d_x), n, bits, d_qp, h_qp, d_packed, s);
}
