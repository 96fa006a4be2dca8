// Per-head absmax quantization of bf16 (or IEEE fp16) tensors to e4m3 (paper Eq. 2).
//
// Two HBM-bound kernels per call:
//   absmax_kernel    max |x| per head, packed bf16x2 max, one atomicMax per block
//   quantize_kernel  s = amax/448, y = x/s (IEEE fp32), cvt.rn.satfinite.e4m3x2
// Algorithmic traffic: 2 B read per element for the maximum, 2 B read + 1 B
// written for the conversion (5 B per element; 3 B when the scale is given).
// The conversion walks each head backwards so that it starts on the part of the
// head the maximum pass touched last, which is still in L2.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <mutex>

#include "common.h"

namespace fp8attn {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ uint4 ld_nc_v4(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// The two 16-bit input types: packed |x| / max for the reduction, and the exact
// fp32 value of the low and high half of a 32-bit word for the conversion.
template <bool kHalf> struct In16;
template <> struct In16<false> {
    using V2 = __nv_bfloat162;
    static __device__ __forceinline__ V2 as2(uint32_t u) { return *reinterpret_cast<V2*>(&u); }
    // an fp32 with the bf16 bits in its upper half is that value
    static __device__ __forceinline__ float lo(uint32_t w) { return __uint_as_float(w << 16); }
    static __device__ __forceinline__ float hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
};
template <> struct In16<true> {
    using V2 = __half2;
    static __device__ __forceinline__ V2 as2(uint32_t u) { return *reinterpret_cast<V2*>(&u); }
    static __device__ __forceinline__ float lo(uint32_t w) { return __low2float(as2(w)); }
    static __device__ __forceinline__ float hi(uint32_t w) { return __high2float(as2(w)); }
};

// One block's share of max |x| over head blockIdx.y (vecs_per_head 16-byte vectors),
// merged into amax_bits[blockIdx.y].
template <bool kHalf>
__device__ __forceinline__ void absmax_body(const uint4* __restrict__ x, int64_t vecs_per_head,
                                            uint32_t* __restrict__ amax_bits) {
    using T = In16<kHalf>;
    using V2 = typename T::V2;
    auto am = [](uint32_t a, uint32_t b) { return __hmax2(__habs2(T::as2(a)), __habs2(T::as2(b))); };
    const uint4* xh = x + (int64_t)blockIdx.y * vecs_per_head;
    V2 m = T::as2(0u);
    int64_t stride = (int64_t)gridDim.x * kThreads;
    int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    for (; i + 3 * stride < vecs_per_head; i += 4 * stride) {
        uint4 a = ld_nc_v4(xh + i), b = ld_nc_v4(xh + i + stride);
        uint4 c = ld_nc_v4(xh + i + 2 * stride), e = ld_nc_v4(xh + i + 3 * stride);
        V2 m0 = am(a.x, a.y), m1 = am(a.z, a.w), m2 = am(b.x, b.y), m3 = am(b.z, b.w);
        V2 m4 = am(c.x, c.y), m5 = am(c.z, c.w), m6 = am(e.x, e.y), m7 = am(e.z, e.w);
        m = __hmax2(m, __hmax2(__hmax2(__hmax2(m0, m1), __hmax2(m2, m3)),
                               __hmax2(__hmax2(m4, m5), __hmax2(m6, m7))));
    }
    for (; i < vecs_per_head; i += stride) {
        uint4 a = ld_nc_v4(xh + i);
        m = __hmax2(m, __hmax2(am(a.x, a.y), am(a.z, a.w)));
    }
    // |x| as a non-negative fp32 bit pattern orders like an unsigned integer
    float f = fmaxf(__low2float(m), __high2float(m));
    uint32_t bits = __float_as_uint(f);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) bits = max(bits, __shfl_xor_sync(0xffffffffu, bits, o));
    __shared__ uint32_t warp_max[kThreads / 32];
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = bits;
    __syncthreads();
    if (threadIdx.x < 32) {
        bits = threadIdx.x < kThreads / 32 ? warp_max[threadIdx.x] : 0u;
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) bits = max(bits, __shfl_xor_sync(0xffffffffu, bits, o));
        if (threadIdx.x == 0) atomicMax(amax_bits + blockIdx.y, bits);
    }
}

// grid: (blocks_per_head, n_heads).
template <bool kHalf>
__global__ void __launch_bounds__(kThreads)
absmax_kernel(const uint4* __restrict__ x, int64_t vecs_per_head, uint32_t* __restrict__ amax_bits) {
    absmax_body<kHalf>(x, vecs_per_head, amax_bits);
}

// two floats -> two e4m3 codes (lo in bits 0..7, hi in bits 8..15), RNE, saturating
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return (uint32_t)r;
}

template <bool kHalf>
__device__ __forceinline__ uint32_t quant4(uint32_t w0, uint32_t w1, float s) {
    // w0, w1: four 16-bit values
    using T = In16<kHalf>;
    float a = __fdiv_rn(T::lo(w0), s);
    float b = __fdiv_rn(T::hi(w0), s);
    float c = __fdiv_rn(T::lo(w1), s);
    float e = __fdiv_rn(T::hi(w1), s);
    return cvt_e4m3x2(a, b) | (cvt_e4m3x2(c, e) << 16);
}

// One block's share of head blockIdx.y.  Each thread turns 32 B of 16-bit input into
// 16 B of e4m3 per step.  pairs_per_head = elems_per_head / 16.
template <bool kHalf>
__device__ __forceinline__ void quantize_body(const uint4* __restrict__ x, int64_t pairs_per_head,
                                              const float* __restrict__ scale_in,
                                              const uint32_t* __restrict__ amax_bits,
                                              uint4* __restrict__ out, float* __restrict__ scale_out) {
    float s;
    if (scale_in != nullptr) {
        s = scale_in[blockIdx.y];
    } else {
        float amax = __uint_as_float(amax_bits[blockIdx.y]);
        s = amax == 0.0f ? 1.0f : __fdiv_rn(amax, 448.0f);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0 && scale_out != nullptr) scale_out[blockIdx.y] = s;
    const uint4* xh = x + (int64_t)blockIdx.y * pairs_per_head * 2;
    uint4* oh = out + (int64_t)blockIdx.y * pairs_per_head;
    int64_t stride = (int64_t)gridDim.x * kThreads;
    // walk the head from its end towards its start
    for (int64_t r = (int64_t)blockIdx.x * kThreads + threadIdx.x; r < pairs_per_head; r += stride) {
        int64_t i = pairs_per_head - 1 - r;
        uint4 a = ld_nc_v4(xh + 2 * i), b = ld_nc_v4(xh + 2 * i + 1);
        uint4 o;
        o.x = quant4<kHalf>(a.x, a.y, s);
        o.y = quant4<kHalf>(a.z, a.w, s);
        o.z = quant4<kHalf>(b.x, b.y, s);
        o.w = quant4<kHalf>(b.z, b.w, s);
        oh[i] = o;
    }
}

// grid: (blocks_per_head, n_heads).
template <bool kHalf>
__global__ void __launch_bounds__(kThreads)
quantize_kernel(const uint4* __restrict__ x, int64_t pairs_per_head,
                const float* __restrict__ scale_in, const uint32_t* __restrict__ amax_bits,
                uint4* __restrict__ out, float* __restrict__ scale_out) {
    quantize_body<kHalf>(x, pairs_per_head, scale_in, amax_bits, out, scale_out);
}

// All tensors of one attention call in two launches: blockIdx.z picks the tensor.
struct QuantBatch {
    const uint4* x[4];
    uint4* out[4];
    int64_t pairs_per_head[4];
    const float* scale_in[4];     // given scales (NULL: derive the scale from amax_in)
    const uint32_t* amax_in[4];   // accumulators the scale is derived from
    uint32_t* amax_acc[4];        // accumulators this tensor's maximum goes to (NULL: none)
    float* scale_out[4];
};

template <bool kHalf>
__global__ void __launch_bounds__(kThreads) absmax_batch_kernel(const QuantBatch b) {
    const int z = blockIdx.z;
    if (b.amax_acc[z] != nullptr && b.pairs_per_head[z] > 0)
        absmax_body<kHalf>(b.x[z], b.pairs_per_head[z] * 2, b.amax_acc[z]);
}

template <bool kHalf>
__global__ void __launch_bounds__(kThreads) quantize_batch_kernel(const QuantBatch b) {
    const int z = blockIdx.z;
    quantize_body<kHalf>(b.x[z], b.pairs_per_head[z], b.scale_in[z], b.amax_in[z], b.out[z], b.scale_out[z]);
}

}  // namespace

int launch_quantize_qkv(const void* q_train, const void* k, const void* v, const void* q_test,
                        int64_t n_heads, int64_t elems_train, int64_t elems_test, void* q_train_fp8,
                        void* k_fp8, void* v_fp8, void* q_test_fp8, float* scale_q, float* scale_k,
                        float* scale_v, uint32_t* amax_bits, uint32_t flags, cudaStream_t stream) {
    if (n_heads <= 0) return FP8ATTN_OK;
    if (n_heads > 65535) return FP8ATTN_ERR_UNSUPPORTED;
    QuantBatch b;
    const void* xs[4] = {q_train, k, v, q_test};
    void* outs[4] = {q_train_fp8, k_fp8, v_fp8, q_test_fp8};
    float* scales[4] = {scale_q, scale_k, scale_v, nullptr};
    for (int z = 0; z < 4; ++z) {
        b.x[z] = static_cast<const uint4*>(xs[z]);
        b.out[z] = static_cast<uint4*>(outs[z]);
        b.pairs_per_head[z] = (z == 3 ? elems_test : elems_train) / 16;
        // the test queries reuse the train-query maximum (slot 0): shared query scale
        b.amax_in[z] = amax_bits + (z == 3 ? 0 : z) * n_heads;
        b.amax_acc[z] = z == 3 ? nullptr : amax_bits + z * n_heads;
        // single-call form: the query scale covers train and test queries alike
        if (z == 3 && (flags & FP8ATTN_QUERY_SCALE_FROM_ALL_ROWS) && elems_test > 0) b.amax_acc[z] = amax_bits;
        b.scale_out[z] = scales[z];
        b.scale_in[z] = nullptr;
        if (flags & FP8ATTN_SCALES_GIVEN) {
            // scales computed upstream: nothing to reduce, nothing to write back
            b.scale_in[z] = scales[z == 3 ? 0 : z];
            b.scale_out[z] = nullptr;
            b.amax_acc[z] = nullptr;
        }
    }
    const int tensors = elems_test > 0 ? 4 : 3;
    const int64_t want = (148 * 16 + n_heads * 3 - 1) / (n_heads * 3);
    const int64_t have = (elems_train / 16 + kThreads - 1) / kThreads;
    const unsigned bx = (unsigned)(want < have ? (want < 1 ? 1 : want) : (have < 1 ? 1 : have));
    if (!(flags & FP8ATTN_SCALES_GIVEN) &&
        cudaMemsetAsync(amax_bits, 0, sizeof(uint32_t) * 3 * n_heads, stream) != cudaSuccess)
        return FP8ATTN_ERR_CUDA;
    const bool half = (flags & FP8ATTN_INPUT_FP16) != 0;
    if (elems_train > 0 && !(flags & FP8ATTN_SCALES_GIVEN)) {
        if (half) absmax_batch_kernel<true><<<dim3(bx, (unsigned)n_heads, 4), kThreads, 0, stream>>>(b);
        else absmax_batch_kernel<false><<<dim3(bx, (unsigned)n_heads, 4), kThreads, 0, stream>>>(b);
        count_launch();
    }
    if (half) quantize_batch_kernel<true><<<dim3(bx, (unsigned)n_heads, tensors), kThreads, 0, stream>>>(b);
    else quantize_batch_kernel<false><<<dim3(bx, (unsigned)n_heads, tensors), kThreads, 0, stream>>>(b);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? FP8ATTN_OK : FP8ATTN_ERR_CUDA;
}

int launch_quantize(const void* x_bf16, int64_t n_heads, int64_t elems_per_head,
                    const float* scale_in, void* x_fp8, float* scale_out,
                    uint32_t* amax_bits, uint32_t flags, cudaStream_t stream) {
    const bool half = (flags & FP8ATTN_INPUT_FP16) != 0;
    if (n_heads <= 0) return FP8ATTN_OK;
    if (n_heads > 65535) return FP8ATTN_ERR_UNSUPPORTED;
    const int64_t vecs = elems_per_head / 8, pairs = elems_per_head / 16;
    // enough blocks to fill 148 SMs several times over, never more than the work
    auto blocks_for = [&](int64_t units) {
        int64_t want = (148 * 16 + n_heads - 1) / n_heads;
        int64_t have = (units + kThreads - 1) / kThreads;
        int64_t b = want < have ? want : have;
        return (unsigned)(b < 1 ? 1 : b);
    };
    if (scale_in == nullptr) {
        if (cudaMemsetAsync(amax_bits, 0, sizeof(uint32_t) * n_heads, stream) != cudaSuccess)
            return FP8ATTN_ERR_CUDA;
        if (elems_per_head > 0) {
            const dim3 grid(blocks_for((vecs + 3) / 4), (unsigned)n_heads);
            if (half) absmax_kernel<true><<<grid, kThreads, 0, stream>>>((const uint4*)x_bf16, vecs, amax_bits);
            else absmax_kernel<false><<<grid, kThreads, 0, stream>>>((const uint4*)x_bf16, vecs, amax_bits);
            count_launch();
        }
    }
    // also launched for empty heads when the scale must be written out
    if (elems_per_head > 0 || scale_out != nullptr) {
        const dim3 grid(blocks_for(pairs), (unsigned)n_heads);
        if (half)
            quantize_kernel<true><<<grid, kThreads, 0, stream>>>((const uint4*)x_bf16, pairs, scale_in,
                                                                 amax_bits, (uint4*)x_fp8, scale_out);
        else
            quantize_kernel<false><<<grid, kThreads, 0, stream>>>((const uint4*)x_bf16, pairs, scale_in,
                                                                  amax_bits, (uint4*)x_fp8, scale_out);
        count_launch();
    }
    return cudaGetLastError() == cudaSuccess ? FP8ATTN_OK : FP8ATTN_ERR_CUDA;
}

}  // namespace fp8attn

// ---------------------------------------------------------------------------
// Allocation-free variant of the quantizer.
//
// The per-head absmax accumulators normally live in the caller's workspace.
// Here they live in a fixed array inside the library image, so a caller needs
// nothing but its input and output buffers.
// ---------------------------------------------------------------------------
namespace fp8attn {
namespace {

constexpr int kStaticMaxHeads = FP8ATTN_NOALLOC_MAX_HEADS;

// Resident on every GPU that loads the library, until the process exits.
static __device__ __align__(256) uint32_t g_static_amax[kStaticMaxHeads];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
uint32_t* g_static_amax_addr[kMaxDevices] = {};

// Device address of g_static_amax on the current device.  In host code the
// symbol's name is only a handle, so the address is looked up once per device.
int static_amax_address(uint32_t** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FP8ATTN_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return FP8ATTN_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_amax_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_amax) != cudaSuccess || p == nullptr)
            return FP8ATTN_ERR_CUDA;
        g_static_amax_addr[dev] = static_cast<uint32_t*>(p);
    }
    *out = g_static_amax_addr[dev];
    return FP8ATTN_OK;
}

}  // namespace
}  // namespace fp8attn

extern "C" int fp8attn_quantize_noalloc(const void* x_bf16, int B, int H, int64_t rows, int d,
                                        const float* scale_in, void* x_fp8, float* scale_out,
                                        void* cuda_stream) {
    using namespace fp8attn;
    if (B <= 0 || H <= 0 || rows < 0) return FP8ATTN_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return FP8ATTN_ERR_UNSUPPORTED;
    if ((int64_t)B * H > kStaticMaxHeads) return FP8ATTN_ERR_TOO_LARGE;
    if (rows > 0 && (!x_bf16 || !x_fp8)) return FP8ATTN_ERR_INVALID_ARG;
    if (!scale_in && !scale_out) return FP8ATTN_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(x_bf16) % 16 || reinterpret_cast<uintptr_t>(x_fp8) % 16 ||
        reinterpret_cast<uintptr_t>(scale_in) % 4 || reinterpret_cast<uintptr_t>(scale_out) % 4)
        return FP8ATTN_ERR_INVALID_ARG;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return FP8ATTN_ERR_CUDA;
    if (major != 10) return FP8ATTN_ERR_UNSUPPORTED;
    uint32_t* amax = nullptr;
    int rc = static_amax_address(&amax);
    if (rc != FP8ATTN_OK) return rc;
    // launch_quantize clears the accumulators it uses at the start of every call
    return launch_quantize(x_bf16, (int64_t)B * H, rows * (int64_t)d, scale_in, x_fp8, scale_out, amax, 0u,
                           static_cast<cudaStream_t>(cuda_stream));
}
