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
//   key_order_kernel  per head: histogram of the norms of a sample, the bin from which on about
//                     kFirstKeys rows lie, then a stable partition (rows at or above that bin
//                     first, the others behind, both in their old order; left alone where that
//                     would be more than kMaxFirst rows); `dest` becomes the destination row of
//                     every key
//   reorder_rows_kernel  applies such a map to a 16-bit tensor (the FP8 path applies it while
//                     it writes the codes)
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.h"

namespace fp8attn {
namespace {

constexpr int kFirstKeys = 256;          // keys to bring to the front, about (two steps' worth)
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
// `norm`: rows fp32 bit patterns per head, heads norm_stride words apart.
template <bool kHalf, int kD>
__global__ void __launch_bounds__(256) key_norm_kernel(const uint4* __restrict__ k, int64_t rows,
                                                      uint32_t* __restrict__ norm, int64_t norm_stride) {
    constexpr int kVecs = kD / 8;
    const int64_t vec = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int64_t row = vec / kVecs;
    float s = 0.f;
    if (row < rows) s = sumsq8<kHalf>(k[(int64_t)blockIdx.y * rows * kVecs + vec]);
#pragma unroll
    for (int o = kVecs / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (row < rows && vec % kVecs == 0) norm[(int64_t)blockIdx.y * norm_stride + row] = __float_as_uint(s);
}

// grid: (kOrderBlocks, heads).  `norm` holds the rows' squared norms (fp32 bit patterns,
// non-negative, so they order like unsigned integers).  Every block of a head works out the
// same threshold and the same list, and writes the destinations of its own share of the rows:
// the rows at or above the threshold bin are collected in a list (at most kMaxFirst: where more
// rows than that share the leading bins, the norms single out no small group and the order is
// left alone), the list is sorted, and every row finds its place by a binary search: a listed
// row goes to its rank in the list, any other row r to r + (listed rows behind it).
constexpr int kMaxFirst = 2048;
constexpr int kSample = 8;
constexpr int kOrderBlocks = 16;

__global__ void __launch_bounds__(kOrderThreads)
key_order_kernel(int64_t rows, const uint32_t* __restrict__ norm, int64_t norm_stride, uint32_t* __restrict__ dest) {
    __shared__ uint32_t hist[kBins];
    __shared__ uint32_t suffix[kOrderThreads];
    __shared__ uint32_t list[kMaxFirst];
    __shared__ uint32_t threshold_bin, first_count;
    const uint32_t* d = norm + (int64_t)blockIdx.y * norm_stride;
    uint32_t* out = dest + (int64_t)blockIdx.y * rows;
    // this block's share of the rows
    const int64_t r0 = rows * blockIdx.x / kOrderBlocks, r1 = rows * (blockIdx.x + 1) / kOrderBlocks;
    const int tid = threadIdx.x;
    for (int i = tid; i < kBins; i += kOrderThreads) hist[i] = 0u;
    if (tid == 0) first_count = 0u;
    __syncthreads();
    // Histogram of a sample (every kSample-th row): the norms of a table crowd into few bins,
    // and shared-memory atomics on them are what this kernel would otherwise spend its time on.
    // The threshold then brings about kFirstKeys rows to the front instead of at least that many.
    const int64_t sampled = (rows + kSample - 1) / kSample;
    for (int64_t i = tid; i < sampled; i += kOrderThreads) atomicAdd(&hist[d[i * kSample] >> 19], 1u);
    __syncthreads();
    constexpr uint32_t want = kFirstKeys / kSample;
    // suffix[t] = rows in the bins from 4t on (kBins = 4 * kOrderThreads)
    static_assert(kBins == 4 * kOrderThreads, "four bins per thread");
    const uint32_t own = hist[4 * tid] + hist[4 * tid + 1] + hist[4 * tid + 2] + hist[4 * tid + 3];
    suffix[tid] = own;
    __syncthreads();
    for (int o = 1; o < kOrderThreads; o <<= 1) {
        const uint32_t add = tid + o < kOrderThreads ? suffix[tid + o] : 0u;
        __syncthreads();
        suffix[tid] += add;
        __syncthreads();
    }
    // the thread whose four bins contain the kFirstKeys-th largest row picks the bin
    const uint32_t above = suffix[tid] - own;     // rows in the bins of the threads behind this one
    if (above < want && suffix[tid] >= want) {
        uint32_t count = above;
        int bin = 4 * tid + 3;
        for (;; --bin) {
            count += hist[bin];
            if (count >= want || bin == 4 * tid) break;
        }
        threshold_bin = (uint32_t)bin;
    }
    if (tid == 0 && suffix[0] < want) threshold_bin = 0u;   // fewer rows than that: all of them
    __syncthreads();
    const uint32_t thr = threshold_bin;
    constexpr int kIlp = 8;   // independent loads in flight per thread: one block reads the whole head
    for (int64_t base = tid; base < rows; base += (int64_t)kIlp * kOrderThreads) {
        uint32_t v[kIlp];
#pragma unroll
        for (int u = 0; u < kIlp; ++u) {
            const int64_t i = base + (int64_t)u * kOrderThreads;
            v[u] = i < rows ? d[i] : 0xffffffffu;
        }
#pragma unroll
        for (int u = 0; u < kIlp; ++u) {
            if (v[u] != 0xffffffffu && (v[u] >> 19) >= thr) {
                const uint32_t pos = atomicAdd(&first_count, 1u);
                if (pos < (uint32_t)kMaxFirst) list[pos] = (uint32_t)(base + (int64_t)u * kOrderThreads);
            }
        }
    }
    __syncthreads();
    const uint32_t count = first_count;
    if (count > (uint32_t)kMaxFirst || count == (uint32_t)rows) {
        for (int64_t i = r0 + tid; i < r1; i += kOrderThreads) out[i] = (uint32_t)i;
        return;
    }
    // bitonic sort of the list, padded with the largest value
    for (int i = tid; i < kMaxFirst; i += kOrderThreads)
        if ((uint32_t)i >= count) list[i] = 0xffffffffu;
    __syncthreads();
    for (int k = 2; k <= kMaxFirst; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < kMaxFirst; i += kOrderThreads) {
                const int p = i ^ j;
                if (p > i) {
                    const uint32_t a = list[i], b = list[p];
                    if (((i & k) == 0) ? a > b : a < b) { list[i] = b; list[p] = a; }
                }
            }
            __syncthreads();
        }
    }
    for (int64_t i = r0 + tid; i < r1; i += kOrderThreads) {
        // listed rows below i (lower bound of i in the sorted list)
        int lo = 0, hi = (int)count;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (list[mid] < (uint32_t)i) lo = mid + 1; else hi = mid;
        }
        const bool listed = lo < (int)count && list[lo] == (uint32_t)i;
        out[i] = listed ? (uint32_t)lo : (uint32_t)i + (count - (uint32_t)lo);
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
                     void* norm_scratch, int64_t norm_stride_bytes, bool compute_norms, cudaStream_t stream) {
    if (n_heads <= 0 || n_train <= 0) return FP8ATTN_OK;
    if (n_heads > 65535) return FP8ATTN_ERR_UNSUPPORTED;
    const int64_t vecs = n_train * (d / 8);
    const dim3 grid((unsigned)((vecs + 255) / 256), (unsigned)n_heads);
    const uint4* k = static_cast<const uint4*>(k16);
    uint32_t* norm = static_cast<uint32_t*>(norm_scratch);
    const int64_t stride = norm_stride_bytes / 4;
    if (compute_norms) {
        if (d == 64) {
            if (half) key_norm_kernel<true, 64><<<grid, 256, 0, stream>>>(k, n_train, norm, stride);
            else key_norm_kernel<false, 64><<<grid, 256, 0, stream>>>(k, n_train, norm, stride);
        } else {
            if (half) key_norm_kernel<true, 128><<<grid, 256, 0, stream>>>(k, n_train, norm, stride);
            else key_norm_kernel<false, 128><<<grid, 256, 0, stream>>>(k, n_train, norm, stride);
        }
        count_launch();
    }
    key_order_kernel<<<dim3(kOrderBlocks, (unsigned)n_heads), kOrderThreads, 0, stream>>>(
        n_train, norm, stride, reinterpret_cast<uint32_t*>(dest));
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
