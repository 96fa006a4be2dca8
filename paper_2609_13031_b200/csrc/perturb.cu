// Seeded Gaussian perturbation of a bf16 tensor, per head (paper Eq. 3):
//   x~ = x + eps * rho[b,h] * z,   rho = sqrt(mean x^2 over the head),   z ~ N(0,1) iid.
// Two HBM-bound kernels: sum of squares per head, then the perturbation itself
// (2 B + 2 B read, 2 B written per element).  z is a pure function of
// (seed, stream, head, element pair): a 64-bit mix of the counters gives two
// 32-bit uniforms, Box-Muller gives two normals for two neighbouring elements.
#include <cuda_bf16.h>

#include "common.h"

namespace fp8attn {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ uint4 ld_nc_v4(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// grid: (blocks_per_head, n_heads); a head is vecs_per_head 16-byte vectors (8 bf16 each)
__global__ void __launch_bounds__(kThreads)
sumsq_kernel(const uint4* __restrict__ x, int64_t vecs_per_head, double* __restrict__ sumsq) {
    const uint4* xh = x + (int64_t)blockIdx.y * vecs_per_head;
    float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
    double total = 0.0;
    int n = 0;
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < vecs_per_head;
         i += (int64_t)gridDim.x * kThreads) {
        const uint4 v = ld_nc_v4(xh + i);
        acc0 = fmaf(bf16_lo(v.x), bf16_lo(v.x), fmaf(bf16_hi(v.x), bf16_hi(v.x), acc0));
        acc1 = fmaf(bf16_lo(v.y), bf16_lo(v.y), fmaf(bf16_hi(v.y), bf16_hi(v.y), acc1));
        acc2 = fmaf(bf16_lo(v.z), bf16_lo(v.z), fmaf(bf16_hi(v.z), bf16_hi(v.z), acc2));
        acc3 = fmaf(bf16_lo(v.w), bf16_lo(v.w), fmaf(bf16_hi(v.w), bf16_hi(v.w), acc3));
        if (++n == 64) {   // keep the fp32 partial sums short
            total += ((double)acc0 + (double)acc1) + ((double)acc2 + (double)acc3);
            acc0 = acc1 = acc2 = acc3 = 0.f;
            n = 0;
        }
    }
    total += ((double)acc0 + (double)acc1) + ((double)acc2 + (double)acc3);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    __shared__ double warp_sum[kThreads / 32];
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = total;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < kThreads / 32; ++w) s += warp_sum[w];
        atomicAdd(sumsq + blockIdx.y, s);
    }
}

// two bf16 values of 32-bit word number `word` of the head, perturbed
__device__ __forceinline__ uint32_t perturb_word(uint32_t w, uint64_t key, int64_t word, float amp) {
    const uint64_t h = mix64(key ^ ((uint64_t)word * 0x9E3779B97F4A7C15ull));
    const float u1 = ((float)(uint32_t)(h >> 32) + 0.5f) * 2.3283064365386963e-10f;   // (0,1]
    const float u2 = ((float)(uint32_t)h + 0.5f) * 2.3283064365386963e-10f;
    const float r = sqrtf(-2.0f * __logf(u1));
    float sn, cs;
    __sincosf(6.283185307179586f * u2, &sn, &cs);
    const float a = fmaf(amp, r * cs, bf16_lo(w));
    const float b = fmaf(amp, r * sn, bf16_hi(w));
    uint32_t packed;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(packed) : "f"(b), "f"(a));
    return packed;
}

// x and out may be the same buffer (each vector is read, then written, by one thread), so
// neither is __restrict__ and x is read with ordinary coherent loads.
__global__ void __launch_bounds__(kThreads)
perturb_kernel(const uint4* x, int64_t vecs_per_head, const double* __restrict__ sumsq,
               float epsilon, uint64_t seed, uint32_t stream_id, uint4* out,
               float* __restrict__ rho_out) {
    const int64_t head = blockIdx.y;
    const float rho = (float)sqrt(sumsq[head] / (double)(vecs_per_head * 8));
    if (blockIdx.x == 0 && threadIdx.x == 0 && rho_out != nullptr) rho_out[head] = rho;
    const float amp = epsilon * rho;
    const uint64_t key = mix64(mix64(mix64(seed) ^ ((uint64_t)stream_id * 0xD6E8FEB86659FD93ull)) ^ (uint64_t)head);
    const uint4* xh = x + head * vecs_per_head;
    uint4* oh = out + head * vecs_per_head;
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < vecs_per_head;
         i += (int64_t)gridDim.x * kThreads) {
        const uint4 v = xh[i];
        uint4 o;
        o.x = perturb_word(v.x, key, 4 * i + 0, amp);
        o.y = perturb_word(v.y, key, 4 * i + 1, amp);
        o.z = perturb_word(v.z, key, 4 * i + 2, amp);
        o.w = perturb_word(v.w, key, 4 * i + 3, amp);
        oh[i] = o;
    }
}

}  // namespace

int launch_perturb(const void* x_bf16, int64_t n_heads, int64_t elems_per_head, float epsilon,
                   uint64_t seed, uint32_t stream_id, void* out_bf16, float* rho_out, double* sumsq,
                   cudaStream_t stream) {
    if (n_heads <= 0 || elems_per_head <= 0) return FP8ATTN_OK;
    if (n_heads > 65535) return FP8ATTN_ERR_UNSUPPORTED;
    const int64_t vecs = elems_per_head / 8;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return FP8ATTN_ERR_CUDA;
    int64_t want = ((int64_t)sms * 16 + n_heads - 1) / n_heads, have = (vecs + kThreads - 1) / kThreads;
    const unsigned bx = (unsigned)(want < have ? (want < 1 ? 1 : want) : (have < 1 ? 1 : have));
    if (cudaMemsetAsync(sumsq, 0, sizeof(double) * n_heads, stream) != cudaSuccess) return FP8ATTN_ERR_CUDA;
    sumsq_kernel<<<dim3(bx, (unsigned)n_heads), kThreads, 0, stream>>>((const uint4*)x_bf16, vecs, sumsq);
    count_launch();
    perturb_kernel<<<dim3(bx, (unsigned)n_heads), kThreads, 0, stream>>>(
        (const uint4*)x_bf16, vecs, sumsq, epsilon, seed, stream_id, (uint4*)out_bf16, rho_out);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? FP8ATTN_OK : FP8ATTN_ERR_CUDA;
}

}  // namespace fp8attn
