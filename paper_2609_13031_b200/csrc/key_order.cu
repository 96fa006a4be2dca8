// Key order for the online softmax: the keys of largest norm first.
//
// Attention sums over keys, so K and V may be permuted together without changing the result.
// The order matters to the kernel all the same: whenever a row's running maximum moves, O of
// that row's warp is rescaled, and with keys in arbitrary order that happens in about a
// quarter of the steps.  A key of large norm is, for most queries, where a large score comes
// from, so with those keys in the first step the running maximum settles there and the later
// steps seldom move it.  (Measured: 3.5 % of the attention time where row norms vary, nothing
// where they do not.)
//
//   key_norm_kernel   sum of squares of every key row (fp32), stored as its bit pattern in `dest`
//   key_order_kernel  per head: histogram of the norms, the bin from which on at least
//                     kFirstKeys rows lie, then a stable partition (rows at or above that bin
//                     first, the others behind, both in their old order); `dest` becomes the
//                     destination row of every key
//   reorder_rows_kernel  applies such a map to a 16-bit tensor (the FP8 path applies it while
//                     it writes the codes)
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.h"

namespace fp8attn {
namespace {

constexpr int kFirstKeys = 256;          // keys to bring to the front (two steps' worth)
constexpr int kOrderThreads = 1024;
constexpr int kBins = 4096;              // fp32 bit pattern >> 19: exponent and four mantissa bits

template <bool kHalf>
__device__ __forceinline__ float sumsq8(uint4 v) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float lo, hi;
        if (kHalf) {
            const __half2 h = *reinterpret_cast<const __half2*>(&w[i]);
            lo = __low2float(h);
            hi = __high2float(h);
        } else {
            lo = __uint_as_float(w[i] << 16);
            hi = __uint_as_float(w[i] & 0xffff0000u);
        }
        s = fmaf(lo, lo, s);
        s = fmaf(hi, hi, s);
    }
    return s;
}

// One 16-byte vector per thread, kD / 8 neighbouring threads per row.  grid: (blocks, heads).
template <bool kHalf, int kD>
__global__ void __launch_bounds__(256) key_norm_kernel(const uint4* __restrict__ k, int64_t rows,
                                                      uint32_t* __restrict__ dest) {
    constexpr int kVecs = kD / 8;
    const int64_t vec = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int64_t row = vec / kVecs;
    float s = 0.f;
    if (row < rows) s = sumsq8<kHalf>(k[(int64_t)blockIdx.y * rows * kVecs + vec]);
#pragma unroll
    for (int o = kVecs / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (row < rows && vec % kVecs == 0) dest[(int64_t)blockIdx.y * rows + row] = __float_as_uint(s);
}

// One block per head.  On entry dest holds the rows' norms (fp32 bit patterns, non-negative, so
// they order like unsigned integers); on exit the destination row of every row.
__global__ void __launch_bounds__(kOrderThreads) key_order_kernel(int64_t rows, uint32_t* __restrict__ dest) {
    __shared__ uint32_t hist[kBins];
    __shared__ uint32_t warp_sum[kOrderThreads / 32];
    __shared__ uint32_t threshold_bin, first_count;
    uint32_t* d = dest + (int64_t)blockIdx.x * rows;
    for (int i = threadIdx.x; i < kBins; i += kOrderThreads) hist[i] = 0u;
    __syncthreads();
    for (int64_t i = threadIdx.x; i < rows; i += kOrderThreads) atomicAdd(&hist[d[i] >> 19], 1u);
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t count = 0;
        int bin = kBins - 1;
        for (; bin > 0; --bin) {
            count += hist[bin];
            if (count >= (uint32_t)kFirstKeys) break;
        }
        if (bin == 0) count += hist[0];
        threshold_bin = (uint32_t)bin;
        first_count = count;
    }
    __syncthreads();
    const uint32_t thr = threshold_bin;
    uint32_t first_off = 0, rest_off = first_count;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int64_t base = 0; base < rows; base += kOrderThreads) {
        const int64_t i = base + threadIdx.x;
        const bool in = i < rows;
        const bool first = in && (d[i] >> 19) >= thr;
        const uint32_t ballot = __ballot_sync(0xffffffffu, first);
        const uint32_t before_in_warp = __popc(ballot & ((1u << lane) - 1u));
        if (lane == 0) warp_sum[warp] = __popc(ballot);
        __syncthreads();
        uint32_t before = before_in_warp, total = 0;
        for (int w = 0; w < kOrderThreads / 32; ++w) {
            const uint32_t c = warp_sum[w];
            if (w < warp) before += c;
            total += c;
        }
        if (in) d[i] = first ? first_off + before : rest_off + ((uint32_t)threadIdx.x - before);
        const uint32_t chunk = (uint32_t)min((int64_t)kOrderThreads, rows - base);
        first_off += total;
        rest_off += chunk - total;
        __syncthreads();
    }
}

template <int kD>
__global__ void __launch_bounds__(256) reorder_rows_kernel(const uint4* __restrict__ x, int64_t rows,
                                                          const int32_t* __restrict__ dest,
                                                          uint4* __restrict__ out) {
    constexpr int kVecs = kD / 8;
    const int64_t vec = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int64_t row = vec / kVecs;
    if (row >= rows) return;
    const int64_t head = (int64_t)blockIdx.y * rows;
    out[(head + dest[head + row]) * kVecs + vec % kVecs] = x[head * kVecs + vec];
}

}  // namespace

int launch_key_order(const void* k16, int64_t n_heads, int64_t n_train, int d, bool half, int32_t* dest,
                     cudaStream_t stream) {
    if (n_heads <= 0 || n_train <= 0) return FP8ATTN_OK;
    if (n_heads > 65535) return FP8ATTN_ERR_UNSUPPORTED;
    const int64_t vecs = n_train * (d / 8);
    const dim3 grid((unsigned)((vecs + 255) / 256), (unsigned)n_heads);
    const uint4* k = static_cast<const uint4*>(k16);
    uint32_t* dst = reinterpret_cast<uint32_t*>(dest);
    if (d == 64) {
        if (half) key_norm_kernel<true, 64><<<grid, 256, 0, stream>>>(k, n_train, dst);
        else key_norm_kernel<false, 64><<<grid, 256, 0, stream>>>(k, n_train, dst);
    } else {
        if (half) key_norm_kernel<true, 128><<<grid, 256, 0, stream>>>(k, n_train, dst);
        else key_norm_kernel<false, 128><<<grid, 256, 0, stream>>>(k, n_train, dst);
    }
    count_launch();
    key_order_kernel<<<(unsigned)n_heads, kOrderThreads, 0, stream>>>(n_train, dst);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? FP8ATTN_OK : FP8ATTN_ERR_CUDA;
}

int launch_reorder_rows(const void* x16, int64_t n_heads, int64_t rows, int d, const int32_t* dest, void* out16,
                        cudaStream_t stream) {
    if (n_heads <= 0 || rows <= 0) return FP8ATTN_OK;
    if (n_heads > 65535) return FP8ATTN_ERR_UNSUPPORTED;
    const int64_t vecs = rows * (d / 8);
    const dim3 grid((unsigned)((vecs + 255) / 256), (unsigned)n_heads);
    if (d == 64)
        reorder_rows_kernel<64><<<grid, 256, 0, stream>>>(static_cast<const uint4*>(x16), rows, dest,
                                                          static_cast<uint4*>(out16));
    else
        reorder_rows_kernel<128><<<grid, 256, 0, stream>>>(static_cast<const uint4*>(x16), rows, dest,
                                                           static_cast<uint4*>(out16));
    count_launch();
    return cudaGetLastError() == cudaSuccess ? FP8ATTN_OK : FP8ATTN_ERR_CUDA;
}

}  // namespace fp8attn
