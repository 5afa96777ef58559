// a6: unpack + dequantize, the receiver's side (paper Sec. 3).  y_i = fma(code_i, scale, lo).
//
// HBM-bound and write-dominated: bits/8 bytes read, 4 (or 2) bytes written per element.
//
// Fast path, bits 1..8: the mirror image of the packer.  A warp owns 1024 elements
// (= 32*bits packed words).  Lane l fetches its `bits` words (widest aligned vector for
// bits 1,2,4,8; 128-byte coalesced through shared memory otherwise), cuts them into the 8
// "quads" (4 codes each) of its 32 consecutive elements, and the quads cross the warp
// through a chunk-swizzled 1 KB staging buffer so that lane l then expands quad j*32+l and
// stores 16-byte vectors that are fully coalesced across the warp.
#include "qp_internal.cuh"

namespace {

constexpr int TILE = 1024;
constexpr int WARPS = QP_THREADS / 32;

struct DQ { float lo, scale; };

__device__ __forceinline__ DQ load_dq(const qp_qparams_t* __restrict__ d_qp, const qp_qparams_t& h_qp, int bits,
                                      unsigned* status)
{
    DQ q;
    if (d_qp) {
        q.lo = __ldg(&d_qp->lo); q.scale = __ldg(&d_qp->scale);
        if (blockIdx.x == 0 && threadIdx.x == 0 && __ldg(&d_qp->bits) != bits) atomicOr(status, QP_DEV_BITS_MISMATCH);
    } else {
        q.lo = h_qp.lo; q.scale = h_qp.scale;
    }
    return q;
}

__device__ __forceinline__ int swz(int p) { return ((((p >> 2) ^ ((p >> 5) & 1)) << 2) | (p & 3)); }

// integer code (< 2^23) to float without a conversion instruction: 2^23 + c, minus 2^23
__device__ __forceinline__ float code_to_float(unsigned c) { return __fsub_rn(__uint_as_float(0x4B000000u | c), 8388608.0f); }

__device__ __forceinline__ float dequant(unsigned c, const DQ& q) { return fmaf(code_to_float(c), q.scale, q.lo); }

__device__ __forceinline__ void store_out(float* y, uint64_t i4, const float (&v)[4])
{
    __stcs(reinterpret_cast<float4*>(y) + i4, make_float4(v[0], v[1], v[2], v[3]));
}
__device__ __forceinline__ void store_out(unsigned short* y, uint64_t i4, const float (&v)[4])
{
    uint2 o;
    o.x = (unsigned)qp_f32_to_bf16(v[0]) | ((unsigned)qp_f32_to_bf16(v[1]) << 16);
    o.y = (unsigned)qp_f32_to_bf16(v[2]) | ((unsigned)qp_f32_to_bf16(v[3]) << 16);
    __stcs(reinterpret_cast<uint2*>(y) + i4, o);
}
__device__ __forceinline__ void store_one(float* y, uint64_t i, float v) { y[i] = v; }
__device__ __forceinline__ void store_one(unsigned short* y, uint64_t i, float v) { y[i] = qp_f32_to_bf16(v); }

template <int BITS, typename TO>
__global__ void __launch_bounds__(QP_THREADS) unpack_kernel(const uint32_t* __restrict__ in, uint64_t ntiles,
                                                            const qp_qparams_t* __restrict__ d_qp, qp_qparams_t h_qp,
                                                            TO* __restrict__ y, unsigned* __restrict__ status)
{
    __shared__ __align__(16) uint32_t stage[WARPS][256];
    const DQ q = load_dq(d_qp, h_qp, BITS, status);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* sw = stage[warp];
    const uint64_t wstride = (uint64_t)gridDim.x * WARPS;
    constexpr unsigned MASK = (1u << BITS) - 1u;
    constexpr int QB = 4 * BITS;
    constexpr unsigned QMASK = QB >= 32 ? 0xFFFFFFFFu : ((1u << (QB & 31)) - 1u);

    for (uint64_t tile = (uint64_t)blockIdx.x * WARPS + warp; tile < ntiles; tile += wstride) {
        const uint32_t* it = in + tile * (32 * BITS);
        uint32_t w[BITS];
        if constexpr (BITS == 8) {
            const uint4 a = __ldg(reinterpret_cast<const uint4*>(it + lane * 8));
            const uint4 b = __ldg(reinterpret_cast<const uint4*>(it + lane * 8) + 1);
            w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
        } else if constexpr (BITS == 4) {
            const uint4 a = __ldg(reinterpret_cast<const uint4*>(it + lane * 4));
            w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
        } else if constexpr (BITS == 2) {
            const uint2 a = __ldg(reinterpret_cast<const uint2*>(it + lane * 2));
            w[0] = a.x; w[1] = a.y;
        } else if constexpr (BITS == 1) {
            w[0] = __ldg(it + lane);
        } else {
#pragma unroll
            for (int m = 0; m < BITS; ++m) sw[m * 32 + lane] = __ldg(it + m * 32 + lane);
            __syncwarp();
#pragma unroll
            for (int m = 0; m < BITS; ++m) w[m] = sw[lane * BITS + m];
            __syncwarp();
        }
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
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float v[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) v[i] = dequant((mine[j] >> (BITS * i)) & MASK, q);
            store_out(y, tile * (TILE / 4) + j * 32 + lane, v);
        }
        __syncwarp();
    }
}

// Scalar path: thread t expands elements [first + 32t, first + 32t + 32) that exist.
template <typename TO>
__global__ void __launch_bounds__(QP_THREADS) unpack_tail_kernel(const uint32_t* __restrict__ in, uint64_t first,
                                                                 uint64_t n, int bits,
                                                                 const qp_qparams_t* __restrict__ d_qp, qp_qparams_t h_qp,
                                                                 TO* __restrict__ y, unsigned* __restrict__ status)
{
    const DQ q = load_dq(d_qp, h_qp, bits, status);
    const uint64_t t = (uint64_t)blockIdx.x * QP_THREADS + threadIdx.x;
    const uint64_t e0 = first + t * 32;
    if (e0 >= n) return;
    const uint32_t* wp = in + t * (uint64_t)bits;          // `in` already points at the word of element `first`
    const unsigned mask = (1u << bits) - 1u;
    const int cnt = (int)((n - e0) < 32 ? (n - e0) : 32);
    const int nw = (cnt * bits + 31) >> 5;                  // words that hold existing elements
    uint32_t w[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
    for (int m = 0; m < nw; ++m) w[m] = __ldg(wp + m);
    for (int i = 0; i < cnt; ++i) {
        const int bit = i * bits, word = bit >> 5, sh = bit & 31;
        uint32_t c = w[word] >> sh;
        if (sh + bits > 32) c |= w[word + 1] << (32 - sh);
        store_one(y, e0 + i, dequant(c & mask, q));
    }
}

// bits = 16: thread t expands one 16-byte vector of 8 codes.
template <typename TO, bool ALIGNED>
__global__ void __launch_bounds__(QP_THREADS) unpack16_kernel(const uint4* __restrict__ in, uint64_t n,
                                                              const qp_qparams_t* __restrict__ d_qp, qp_qparams_t h_qp,
                                                              TO* __restrict__ y, unsigned* __restrict__ status)
{
    const DQ q = load_dq(d_qp, h_qp, 16, status);
    const uint64_t nvec = (n + 7) / 8;
    const uint64_t stride = (uint64_t)gridDim.x * QP_THREADS;
    for (uint64_t v = (uint64_t)blockIdx.x * QP_THREADS + threadIdx.x; v < nvec; v += stride) {
        const uint4 a = __ldg(in + v);
        const unsigned c[8] = {a.x & 0xFFFFu, a.x >> 16, a.y & 0xFFFFu, a.y >> 16,
                               a.z & 0xFFFFu, a.z >> 16, a.w & 0xFFFFu, a.w >> 16};
        float f[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = dequant(c[i], q);
        const uint64_t e0 = v * 8;
        if (ALIGNED && e0 + 8 <= n) {
            const float lo4[4] = {f[0], f[1], f[2], f[3]}, hi4[4] = {f[4], f[5], f[6], f[7]};
            store_out(y, v * 2, lo4);
            store_out(y, v * 2 + 1, hi4);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (e0 + i < n) store_one(y, e0 + i, f[i]);
        }
    }
}

template <typename TO>
int32_t unpack_typed(qp_ctx* ctx, const void* d_packed, uint64_t n, int bits, const qp_qparams_t* d_qp,
                     const qp_qparams_t& h_qp, TO* y, cudaStream_t s)
{
    const bool aligned = ((uintptr_t)y & 15u) == 0;
    if (bits == 16) {
        const uint64_t nvec = (n + 7) / 8;
        uint64_t want = (nvec + QP_THREADS - 1) / QP_THREADS;
        const uint64_t cap = (uint64_t)ctx->sm_count * 64;
        const int blocks = (int)(want > cap ? cap : want);
        ctx->launches += 1;
        if (aligned)
            unpack16_kernel<TO, true><<<blocks, QP_THREADS, 0, s>>>(static_cast<const uint4*>(d_packed), n, d_qp, h_qp, y, ctx->d_status);
        else
            unpack16_kernel<TO, false><<<blocks, QP_THREADS, 0, s>>>(static_cast<const uint4*>(d_packed), n, d_qp, h_qp, y, ctx->d_status);
        return qp_check_launch(ctx, "qp_unpack_dequantize");
    }
    const uint32_t* in = static_cast<const uint32_t*>(d_packed);
    const uint64_t ntiles = aligned ? n / TILE : 0;
    if (ntiles) {
        uint64_t want = (ntiles + WARPS - 1) / WARPS;
        const uint64_t cap = (uint64_t)ctx->sm_count * 64;
        const int blocks = (int)(want > cap ? cap : want);
        ctx->launches += 1;
#define QP_UNPACK_CASE(B) case B: unpack_kernel<B, TO><<<blocks, QP_THREADS, 0, s>>>(in, ntiles, d_qp, h_qp, y, ctx->d_status); break;
        switch (bits) {
            QP_UNPACK_CASE(1) QP_UNPACK_CASE(2) QP_UNPACK_CASE(3) QP_UNPACK_CASE(4)
            QP_UNPACK_CASE(5) QP_UNPACK_CASE(6) QP_UNPACK_CASE(7) QP_UNPACK_CASE(8)
        }
#undef QP_UNPACK_CASE
    }
    const uint64_t first = ntiles * TILE;
    if (n > first) {
        const uint64_t threads = (n - first + 31) / 32;
        const uint64_t blocks = (threads + QP_THREADS - 1) / QP_THREADS;
        ctx->launches += 1;
        unpack_tail_kernel<TO><<<(unsigned)blocks, QP_THREADS, 0, s>>>(in + ntiles * 32 * (uint64_t)bits, first, n, bits,
                                                                       d_qp, h_qp, y, ctx->d_status);
    }
    return qp_check_launch(ctx, "qp_unpack_dequantize");
}

}  // namespace

int32_t qp_launch_unpack(qp_ctx* ctx, const void* d_packed, uint64_t n, int bits, const qp_qparams_t* d_qp,
                         qp_qparams_t h_qp, void* d_y, int out_dtype, cudaStream_t s)
{
    if (out_dtype == QP_F32) return unpack_typed<float>(ctx, d_packed, n, bits, d_qp, h_qp, static_cast<float*>(d_y), s);
    return unpack_typed<unsigned short>(ctx, d_packed, n, bits, d_qp, h_qp, static_cast<unsigned short*>(d_y), s);
}
