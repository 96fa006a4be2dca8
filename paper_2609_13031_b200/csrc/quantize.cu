// Per-head absmax quantization of bf16 (or IEEE fp16) tensors to e4m3 (paper Eq. 2).
//
// Two HBM-bound kernels per call:
//   absmax_kernel    max |x| per head, packed bf16x2 max, one atomicMax per block
//   quantize_kernel  s = amax/448, y = x/s (IEEE fp32), cvt.rn.satfinite.e4m3x2
// Algorithmic traffic: 2 B read per element for the maximum, 2 B read + 1 B
// written for the conversion (5 B per element; 3 B when the scale is given).
// The conversion walks each head backwards so that it starts on the part of the
// head the maximum pass touched last, which is still in L2.
// The IEEE division x/s is not evaluated per element: a 16-bit input is (1.m) * 2^e with a
// 7-bit (bf16) or 10-bit (fp16) m, and RN((1.m) * 2^e / s) = RN((1.m) / s) * 2^e exactly
// (scaling by a power of two is exact; where the product leaves the normal range the code
// saturates or is zero either way).  Each block therefore divides once per mantissa into a
// small table with the IEEE division, and an element costs a lookup and one multiplication
// by +-2^e.  Codes are identical to those of the per-element division by construction.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <mutex>

#include "common.h"

namespace fp8attn {
namespace {

constexpr int kThreads = 256;

// SMs of the current device (0 on error)
int sm_count() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return 0;
    return sms;
}

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
    static constexpr int kMantBits = 7;
    static __device__ __forceinline__ V2 as2(uint32_t u) { return *reinterpret_cast<V2*>(&u); }
    // an fp32 with the bf16 bits in its upper half is that value
    static __device__ __forceinline__ float lo(uint32_t w) { return __uint_as_float(w << 16); }
    static __device__ __forceinline__ float hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
};
template <> struct In16<true> {
    using V2 = __half2;
    static constexpr int kMantBits = 10;
    static __device__ __forceinline__ V2 as2(uint32_t u) { return *reinterpret_cast<V2*>(&u); }
    static __device__ __forceinline__ float lo(uint32_t w) { return __low2float(as2(w)); }
    static __device__ __forceinline__ float hi(uint32_t w) { return __high2float(as2(w)); }
};

// One block's share of max |x| over head blockIdx.y (vecs_per_head 16-byte vectors),
// merged into amax_bits[blockIdx.y].
// With kNorm it also leaves the squared norm of every row (vecs_per_row 16-byte vectors, 8 or
// 16; fp32 bit pattern) in row_norm[row] of the head: the vectors of a row sit in neighbouring
// lanes, whose loop conditions agree (all bounds are multiples of the row length), so the lanes
// of a row add up under a mask of their own.
template <bool kHalf, bool kNorm = false>
__device__ __forceinline__ void absmax_body(const uint4* __restrict__ x, int64_t vecs_per_head,
                                            uint32_t* __restrict__ amax_bits,
                                            uint32_t* __restrict__ row_norm = nullptr, int vecs_per_row = 8) {
    using T = In16<kHalf>;
    using V2 = typename T::V2;
    auto am = [](uint32_t a, uint32_t b) { return __hmax2(__habs2(T::as2(a)), __habs2(T::as2(b))); };
    const uint32_t row_mask = (vecs_per_row == 16 ? 0xffffu : 0xffu) << (threadIdx.x & 31 & ~(vecs_per_row - 1));
    auto norm_of = [&](const uint4& v, int64_t vec) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        float q = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float lo = T::lo(w[k]), hi = T::hi(w[k]);
            q = fmaf(lo, lo, q);
            q = fmaf(hi, hi, q);
        }
        for (int o = vecs_per_row >> 1; o > 0; o >>= 1) q += __shfl_xor_sync(row_mask, q, o);
        if ((vec & (vecs_per_row - 1)) == 0) row_norm[vec / vecs_per_row] = __float_as_uint(q);
    };
    const uint4* xh = x + (int64_t)blockIdx.y * vecs_per_head;
    V2 m = T::as2(0u);
    int64_t stride = (int64_t)gridDim.x * kThreads;
    int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    for (; i + 3 * stride < vecs_per_head; i += 4 * stride) {
        uint4 a = ld_nc_v4(xh + i), b = ld_nc_v4(xh + i + stride);
        uint4 c = ld_nc_v4(xh + i + 2 * stride), e = ld_nc_v4(xh + i + 3 * stride);
        if (kNorm) {
            norm_of(a, i);
            norm_of(b, i + stride);
            norm_of(c, i + 2 * stride);
            norm_of(e, i + 3 * stride);
        }
        V2 m0 = am(a.x, a.y), m1 = am(a.z, a.w), m2 = am(b.x, b.y), m3 = am(b.z, b.w);
        V2 m4 = am(c.x, c.y), m5 = am(c.z, c.w), m6 = am(e.x, e.y), m7 = am(e.z, e.w);
        m = __hmax2(m, __hmax2(__hmax2(__hmax2(m0, m1), __hmax2(m2, m3)),
                               __hmax2(__hmax2(m4, m5), __hmax2(m6, m7))));
    }
    for (; i < vecs_per_head; i += stride) {
        uint4 a = ld_nc_v4(xh + i);
        if (kNorm) norm_of(a, i);
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

// x / s for a 16-bit x given as its exact fp32 value: the quotient of its mantissa from the
// table, times its sign and power of two.  (Every fp32 that comes from a normal bf16, or from
// any fp16, has at most kMantBits leading mantissa bits set.)  With kDirect the division is
// evaluated per element: the block's scale is so small that subnormal inputs, which have no
// normalised mantissa, can still give non-zero codes.
template <bool kHalf, bool kDirect>
__device__ __forceinline__ float quotient(float x, float s, const float* tab) {
    if (kDirect) return __fdiv_rn(x, s);
    const uint32_t u = __float_as_uint(x);
    return tab[(u >> (23 - In16<kHalf>::kMantBits)) & ((1u << In16<kHalf>::kMantBits) - 1u)] *
           __uint_as_float(u & 0xff800000u);
}
template <bool kHalf, bool kDirect>
__device__ __forceinline__ uint32_t quant4(uint32_t w0, uint32_t w1, float s, const float* tab) {
    // w0, w1: four 16-bit values
    using T = In16<kHalf>;
    float a = quotient<kHalf, kDirect>(T::lo(w0), s, tab);
    float b = quotient<kHalf, kDirect>(T::hi(w0), s, tab);
    float c = quotient<kHalf, kDirect>(T::lo(w1), s, tab);
    float e = quotient<kHalf, kDirect>(T::hi(w1), s, tab);
    return cvt_e4m3x2(a, b) | (cvt_e4m3x2(c, e) << 16);
}

// One block's share of head blockIdx.y.  Each thread turns 32 B of 16-bit input into
// 16 B of e4m3 per step.  pairs_per_head = elems_per_head / 16.
// `row_dest` (NULL: none) sends the codes of row r of a head to row row_dest[r] of the output;
// a row is 2^pairs_per_row_shift pairs.
template <bool kHalf>
__device__ __forceinline__ void quantize_body(const uint4* __restrict__ x, int64_t pairs_per_head,
                                              const float* __restrict__ scale_in,
                                              const uint32_t* __restrict__ amax_bits,
                                              uint4* __restrict__ out, float* __restrict__ scale_out,
                                              const int32_t* __restrict__ row_dest = nullptr,
                                              int pairs_per_row_shift = 0) {
    float s;
    if (scale_in != nullptr) {
        s = scale_in[blockIdx.y];
    } else {
        float amax = __uint_as_float(amax_bits[blockIdx.y]);
        s = amax == 0.0f ? 1.0f : __fdiv_rn(amax, 448.0f);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0 && scale_out != nullptr) scale_out[blockIdx.y] = s;
    // (1.m) / s for every mantissa m of the input type, by the IEEE division
    constexpr int kTab = 1 << In16<kHalf>::kMantBits;
    __shared__ float tab[kTab];
    for (int m = threadIdx.x; m < kTab; m += kThreads)
        tab[m] = __fdiv_rn(__uint_as_float(0x3f800000u | ((uint32_t)m << (23 - In16<kHalf>::kMantBits))), s);
    __syncthreads();
    const uint4* xh = x + (int64_t)blockIdx.y * pairs_per_head * 2;
    uint4* oh = out + (int64_t)blockIdx.y * pairs_per_head;
    int64_t stride = (int64_t)gridDim.x * kThreads;
    // A bf16 subnormal (below 2^-126) is no (1.m) * 2^e; it can only give a non-zero code
    // (|x/s| >= 2^-10) if s < 2^-116.  And (1.m) / s must itself be a normal number for the
    // table entry to be the exact quotient's mantissa: s < 2^126.  Heads outside a scale range
    // kept well inside both limits (and given scales that are zero, negative or not finite)
    // take the per-element division.
    const bool direct = !(s >= 1e-30f && s <= 1e30f);
    // walk the head from its end towards its start
    for (int64_t r = (int64_t)blockIdx.x * kThreads + threadIdx.x; r < pairs_per_head; r += stride) {
        int64_t i = pairs_per_head - 1 - r;
        uint4 a = ld_nc_v4(xh + 2 * i), b = ld_nc_v4(xh + 2 * i + 1);
        uint4 o;
        if (direct) {
            o.x = quant4<kHalf, true>(a.x, a.y, s, tab);
            o.y = quant4<kHalf, true>(a.z, a.w, s, tab);
            o.z = quant4<kHalf, true>(b.x, b.y, s, tab);
            o.w = quant4<kHalf, true>(b.z, b.w, s, tab);
        } else {
            o.x = quant4<kHalf, false>(a.x, a.y, s, tab);
            o.y = quant4<kHalf, false>(a.z, a.w, s, tab);
            o.z = quant4<kHalf, false>(b.x, b.y, s, tab);
            o.w = quant4<kHalf, false>(b.z, b.w, s, tab);
        }
        int64_t dst = i;
        if (row_dest != nullptr) {
            const int64_t row = i >> pairs_per_row_shift;
            dst = ((int64_t)row_dest[(int64_t)blockIdx.y * (pairs_per_head >> pairs_per_row_shift) + row]
                   << pairs_per_row_shift) + (i - (row << pairs_per_row_shift));
        }
        oh[dst] = o;
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
    const int32_t* row_dest[4];   // output row of every input row, per head (NULL: the same row)
    int pairs_per_row_shift;      // log2(d / 16)
};

// kNorm: the pass over K (z = 1) also leaves the keys' squared norms in key_norm (one word per
// key, the heads key_norm_stride words apart).
template <bool kHalf, bool kNorm = false>
__global__ void __launch_bounds__(kThreads)
absmax_batch_kernel(const QuantBatch b, uint32_t* key_norm = nullptr, int64_t key_norm_stride = 0) {
    const int z = blockIdx.z;
    if (b.amax_acc[z] == nullptr || b.pairs_per_head[z] <= 0) return;
    if (kNorm && z == 1)
        absmax_body<kHalf, true>(b.x[z], b.pairs_per_head[z] * 2, b.amax_acc[z],
                                 key_norm + (int64_t)blockIdx.y * key_norm_stride, 2 << b.pairs_per_row_shift);
    else
        absmax_body<kHalf>(b.x[z], b.pairs_per_head[z] * 2, b.amax_acc[z]);
}

template <bool kHalf>
__global__ void __launch_bounds__(kThreads) quantize_batch_kernel(const QuantBatch b) {
    const int z = blockIdx.z;
    quantize_body<kHalf>(b.x[z], b.pairs_per_head[z], b.scale_in[z], b.amax_in[z], b.out[z], b.scale_out[z],
                         b.row_dest[z], b.pairs_per_row_shift);
}


// ---------------------------------------------------------------------------
// One launch for a small call (everything stays in L2): maximum, grid barrier, conversion.
//
// The 16-element pairs of all tensors and heads of the call form one flat range, cut into
// equal shares, one per block; a block walks its share segment by segment (segment = the part
// of one head of one tensor inside the share).  Pass 1 leaves the maximum of every segment
// in a slot of its own (slot = block + ordinal of the head, which is unique along the
// staircase of shares and heads), so nothing has to be cleared beforehand and no atomic
// maximum is needed.  All blocks then arrive on a counter and wait for the others (the launch
// has at most two blocks per SM, so on an otherwise idle GPU they are all resident; the wait
// is bounded all the same and records FP8ATTN_ERR_TIMEOUT on expiry).  Pass 2 takes the
// maximum of a head over the slots of the blocks that share it, builds the mantissa table
// and converts.  The last block to finish resets the two counters.
// ---------------------------------------------------------------------------
constexpr int kOneThreads = 512;
constexpr int64_t kOneLaunchMaxBytes = 48ll << 20;   // 16-bit input bytes of a call that takes this path
constexpr uint64_t kGridWaitLimitNs = 2000000000ull;

struct OneLaunchArgs {
    QuantBatch b;
    int tensors, n_heads;
    int query_scale_from_all_rows;
    uint32_t* status;     // workspace status words
    uint32_t* counters;   // [0] arrivals after pass 1, [1] blocks done
    float* partial;       // kOneLaunchMaxBlocks + 4 * n_heads slots
};

template <bool kHalf>
__global__ void __launch_bounds__(kOneThreads) quantize_one_launch_kernel(const OneLaunchArgs a) {
    using T = In16<kHalf>;
    using V2 = typename T::V2;
    constexpr int kTab = 1 << T::kMantBits;
    __shared__ float tab[kTab];
    __shared__ uint32_t warp_max[kOneThreads / 32];
    __shared__ float seg_amax;
    __shared__ int give_up;
    const int nb = gridDim.x, bid = blockIdx.x;
    int64_t total = 0, t_base[5];
    for (int z = 0; z < 4; ++z) {
        t_base[z] = total;
        if (z < a.tensors) total += a.b.pairs_per_head[z] * a.n_heads;
    }
    t_base[4] = total;
    auto share_lo = [&](int blk) { return total * blk / nb; };
    const int64_t lo = share_lo(bid), hi = share_lo(bid + 1);
    // a device error recorded earlier is sticky: nothing runs until the host has read it
    // (one thread decides for the block)
    if (threadIdx.x == 0) give_up = *reinterpret_cast<volatile uint32_t*>(a.status) != 0u;
    __syncthreads();
    if (give_up) return;

    // ---- pass 1: the maximum of every segment of this block's share ----
    for (int z = 0; z < a.tensors; ++z) {
        const int64_t pph = a.b.pairs_per_head[z];
        const bool counts = z < 3 || a.query_scale_from_all_rows;
        const int64_t t_lo = lo > t_base[z] ? lo : t_base[z], t_hi = hi < t_base[z + 1] ? hi : t_base[z + 1];
        if (pph <= 0 || !counts || t_lo >= t_hi) continue;
        for (int64_t head = (t_lo - t_base[z]) / pph; t_base[z] + head * pph < t_hi; ++head) {
            const int64_t h_base = t_base[z] + head * pph;
            const int64_t p0 = (t_lo > h_base ? t_lo : h_base) - h_base;
            const int64_t p1 = (t_hi < h_base + pph ? t_hi : h_base + pph) - h_base;
            const uint4* xh = a.b.x[z] + head * pph * 2;
            auto am = [](uint32_t u, uint32_t v) { return __hmax2(__habs2(T::as2(u)), __habs2(T::as2(v))); };
            V2 m = T::as2(0u);
            int64_t i = 2 * p0 + threadIdx.x;
            for (; i + 3 * kOneThreads < 2 * p1; i += 4 * kOneThreads) {   // four loads in flight
                const uint4 v0 = xh[i], v1 = xh[i + kOneThreads], v2 = xh[i + 2 * kOneThreads],
                            v3 = xh[i + 3 * kOneThreads];
                m = __hmax2(m, __hmax2(__hmax2(__hmax2(am(v0.x, v0.y), am(v0.z, v0.w)),
                                               __hmax2(am(v1.x, v1.y), am(v1.z, v1.w))),
                                       __hmax2(__hmax2(am(v2.x, v2.y), am(v2.z, v2.w)),
                                               __hmax2(am(v3.x, v3.y), am(v3.z, v3.w)))));
            }
            for (; i < 2 * p1; i += kOneThreads) {
                const uint4 v = xh[i];
                m = __hmax2(m, __hmax2(am(v.x, v.y), am(v.z, v.w)));
            }
            uint32_t bits = __float_as_uint(fmaxf(__low2float(m), __high2float(m)));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) bits = max(bits, __shfl_xor_sync(0xffffffffu, bits, o));
            __syncthreads();   // warp_max of the last segment has been read
            if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = bits;
            __syncthreads();
            if (threadIdx.x == 0) {
                for (int w = 0; w < kOneThreads / 32; ++w) bits = max(bits, warp_max[w]);
                a.partial[bid + z * a.n_heads + (int)head] = __uint_as_float(bits);
            }
        }
    }
    // ---- grid barrier: every block's maxima are visible before any block converts ----
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(a.counters, 1u);
        uint64_t t0;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
        int bad = 0;
        while (*reinterpret_cast<volatile uint32_t*>(a.counters) < (uint32_t)nb) {
            __nanosleep(64);
            uint64_t t1;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
            if (t1 - t0 > kGridWaitLimitNs || *reinterpret_cast<volatile uint32_t*>(a.status) != 0u) {
                if (atomicCAS(a.status, 0u, (uint32_t)FP8ATTN_ERR_TIMEOUT) == 0u)
                    a.status[1] = (kDetailQuantizeGridWait << 24) | ((uint32_t)bid & 0xFFFFFFu);
                bad = 1;
                break;
            }
        }
        __threadfence();
        give_up = bad;
    }
    __syncthreads();
    if (give_up) return;

    // ---- pass 2: scale of each segment's head, mantissa table, conversion ----
    for (int z = 0; z < a.tensors; ++z) {
        const int64_t pph = a.b.pairs_per_head[z];
        const int64_t t_lo = lo > t_base[z] ? lo : t_base[z], t_hi = hi < t_base[z + 1] ? hi : t_base[z + 1];
        if (pph <= 0 || t_lo >= t_hi) continue;
        for (int64_t head = (t_lo - t_base[z]) / pph; t_base[z] + head * pph < t_hi; ++head) {
            const int64_t h_base = t_base[z] + head * pph;
            const int64_t p0 = (t_lo > h_base ? t_lo : h_base) - h_base;
            const int64_t p1 = (t_hi < h_base + pph ? t_hi : h_base + pph) - h_base;
            if (threadIdx.x == 0) {
                // the head's maximum: over the slots of all blocks whose share touches the
                // head (of the tensor the scale comes from: the test queries take the train
                // queries' maximum; with the single-call form both query tensors count)
                float amax = 0.f;
                for (int src = 0; src < 2; ++src) {
                    const int zs = src == 0 ? (z == 3 ? 0 : z) : (z == 0 || z == 3 ? 3 : -1);
                    if (zs < 0 || (src == 1 && !a.query_scale_from_all_rows) || zs >= a.tensors) continue;
                    const int64_t pz = a.b.pairs_per_head[zs];
                    if (pz <= 0) continue;
                    const int64_t s0 = t_base[zs] + head * pz, s1 = s0 + pz;
                    int b0 = (int)(s0 * nb / total);
                    while (b0 > 0 && share_lo(b0) > s0) --b0;
                    while (share_lo(b0 + 1) <= s0) ++b0;
                    for (int blk = b0; blk < nb && share_lo(blk) < s1; ++blk)
                        amax = fmaxf(amax, a.partial[blk + zs * a.n_heads + (int)head]);
                }
                seg_amax = amax;
            }
            __syncthreads();   // also: the lookups of the last segment are done
            const float amax = seg_amax;
            const float s = amax == 0.0f ? 1.0f : __fdiv_rn(amax, 448.0f);
            if (p0 == 0 && threadIdx.x == 0 && a.b.scale_out[z] != nullptr) a.b.scale_out[z][head] = s;
            for (int mnt = threadIdx.x; mnt < kTab; mnt += kOneThreads)
                tab[mnt] = __fdiv_rn(__uint_as_float(0x3f800000u | ((uint32_t)mnt << (23 - T::kMantBits))), s);
            __syncthreads();
            const bool direct = !(s >= 1e-30f && s <= 1e30f);
            const uint4* xh = a.b.x[z] + head * pph * 2;
            uint4* oh = a.b.out[z] + head * pph;
            auto convert = [&](const uint4& u, const uint4& v) {
                uint4 o;
                if (direct) {
                    o.x = quant4<kHalf, true>(u.x, u.y, s, tab);
                    o.y = quant4<kHalf, true>(u.z, u.w, s, tab);
                    o.z = quant4<kHalf, true>(v.x, v.y, s, tab);
                    o.w = quant4<kHalf, true>(v.z, v.w, s, tab);
                } else {
                    o.x = quant4<kHalf, false>(u.x, u.y, s, tab);
                    o.y = quant4<kHalf, false>(u.z, u.w, s, tab);
                    o.z = quant4<kHalf, false>(v.x, v.y, s, tab);
                    o.w = quant4<kHalf, false>(v.z, v.w, s, tab);
                }
                return o;
            };
            int64_t i = p0 + threadIdx.x;
            for (; i + kOneThreads < p1; i += 2 * kOneThreads) {   // four loads in flight
                const uint4 u0 = xh[2 * i], v0 = xh[2 * i + 1];
                const uint4 u1 = xh[2 * (i + kOneThreads)], v1 = xh[2 * (i + kOneThreads) + 1];
                oh[i] = convert(u0, v0);
                oh[i + kOneThreads] = convert(u1, v1);
            }
            for (; i < p1; i += kOneThreads) oh[i] = convert(xh[2 * i], xh[2 * i + 1]);
        }
    }
    // ---- the last block to finish leaves the counters at zero for the next call ----
    __syncthreads();
    if (threadIdx.x == 0) {
        if (atomicAdd(a.counters + 1, 1u) == (uint32_t)nb - 1u) {
            a.counters[0] = 0u;
            a.counters[1] = 0u;
        }
    }
}

}  // namespace

int launch_quantize_qkv(const void* q_train, const void* k, const void* v, const void* q_test,
                        int64_t n_heads, int64_t elems_train, int64_t elems_test, void* q_train_fp8,
                        void* k_fp8, void* v_fp8, void* q_test_fp8, float* scale_q, float* scale_k,
                        float* scale_v, uint32_t* amax_bits, uint32_t flags, uint32_t* status,
                        uint32_t* counters, float* partial, cudaStream_t stream, int32_t* key_dest, int d) {
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
        // a key order applies to K and V alike: the attention sums over keys
        b.row_dest[z] = (z == 1 || z == 2) ? key_dest : nullptr;
        if (flags & FP8ATTN_SCALES_GIVEN) {
            // scales computed upstream: nothing to reduce, nothing to write back
            b.scale_in[z] = scales[z == 3 ? 0 : z];
            b.scale_out[z] = nullptr;
            b.amax_acc[z] = nullptr;
        }
    }
    b.pairs_per_row_shift = d == 128 ? 3 : 2;
    const int tensors = elems_test > 0 ? 4 : 3;
    const int sms = sm_count();
    if (sms <= 0) return FP8ATTN_ERR_CUDA;
    const bool half = (flags & FP8ATTN_INPUT_FP16) != 0;
    // small call: one launch (maximum, grid barrier, conversion)
    const int64_t total_pairs = (3 * elems_train + elems_test) / 16 * n_heads;
    if (!(flags & (FP8ATTN_SCALES_GIVEN | FP8ATTN_QKV_TWO_LAUNCHES)) && key_dest == nullptr && status != nullptr &&
        total_pairs > 0 &&
        total_pairs * 32 <= kOneLaunchMaxBytes) {
        OneLaunchArgs a;
        a.b = b;
        a.tensors = tensors;
        a.n_heads = (int)n_heads;
        a.query_scale_from_all_rows = (flags & FP8ATTN_QUERY_SCALE_FROM_ALL_ROWS) ? 1 : 0;
        a.status = status;
        a.counters = counters;
        a.partial = partial;
        // At most two blocks of 512 threads per SM: on a GPU that runs nothing else all blocks
        // are resident at once.  (Where other work holds SMs, the blocks that are resident wait
        // for the rest; the wait is bounded.)
        int64_t nb = (total_pairs + kOneThreads - 1) / kOneThreads;
        if (nb > 2 * sms) nb = 2 * sms;
        if (nb > kOneLaunchMaxBlocks) nb = kOneLaunchMaxBlocks;
        if (half) quantize_one_launch_kernel<true><<<(unsigned)nb, kOneThreads, 0, stream>>>(a);
        else quantize_one_launch_kernel<false><<<(unsigned)nb, kOneThreads, 0, stream>>>(a);
        count_launch();
        return cudaGetLastError() == cudaSuccess ? FP8ATTN_OK : FP8ATTN_ERR_CUDA;
    }
    const int64_t want = ((int64_t)sms * 16 + n_heads * 3 - 1) / (n_heads * 3);
    const int64_t have = (elems_train / 16 + kThreads - 1) / kThreads;
    const unsigned bx = (unsigned)(want < have ? (want < 1 ? 1 : want) : (have < 1 ? 1 : have));
    if (!(flags & FP8ATTN_SCALES_GIVEN) &&
        cudaMemsetAsync(amax_bits, 0, sizeof(uint32_t) * 3 * n_heads, stream) != cudaSuccess)
        return FP8ATTN_ERR_CUDA;
    // A key order is built between the two passes: the keys' norms come out of the maximum pass
    // (or, where the scales are given and there is none, out of a pass of their own) and sit in
    // the K8 buffer until the conversion overwrites them.
    uint32_t* key_norm = reinterpret_cast<uint32_t*>(k_fp8);
    const int64_t key_norm_stride = elems_train / 4;        // K8 bytes per head, in words
    const int64_t keys = elems_train / d;
    if (elems_train > 0 && !(flags & FP8ATTN_SCALES_GIVEN)) {
        const dim3 grid(bx, (unsigned)n_heads, 4);
        if (key_dest != nullptr) {
            if (half) absmax_batch_kernel<true, true><<<grid, kThreads, 0, stream>>>(b, key_norm, key_norm_stride);
            else absmax_batch_kernel<false, true><<<grid, kThreads, 0, stream>>>(b, key_norm, key_norm_stride);
        } else {
            if (half) absmax_batch_kernel<true><<<grid, kThreads, 0, stream>>>(b);
            else absmax_batch_kernel<false><<<grid, kThreads, 0, stream>>>(b);
        }
        count_launch();
    }
    if (key_dest != nullptr && elems_train > 0) {
        const int rc = launch_key_order(k, n_heads, keys, d, half, key_dest, key_norm,
                                        key_norm_stride * 4, (flags & FP8ATTN_SCALES_GIVEN) != 0, stream);
        if (rc != FP8ATTN_OK) return rc;
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
    // enough blocks to fill the SMs several times over, never more than the work
    const int sms = sm_count();
    if (sms <= 0) return FP8ATTN_ERR_CUDA;
    auto blocks_for = [&](int64_t units) {
        int64_t want = ((int64_t)sms * 16 + n_heads - 1) / n_heads;
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
