// Internal declarations shared by the translation units of libfp8attn.so.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "fp8attn.h"

namespace fp8attn {

// Workspace layout (device memory, caller-owned, zero-filled once):
//   [0,4)    device status word (fp8attn_status_t, 0 = ok); first error wins
//   [4,8)    detail code of that error (which wait expired, which CTA)
//   [256, 256 + 12*B*H) three sets of per-(b,h) absmax accumulators (fp32 bit
//                       patterns): one is used by fp8attn_quantize, all three (Q, K, V)
//                       by fp8attn_quantize_qkv; cleared at the start of every call.
//                       fp8attn_perturb keeps its per-head sums of squares (fp64) here too.
//   [16,24)  the two grid-wide arrival counters of the one-launch quantizer; zero between calls
//   after the accumulators: partial maxima of the one-launch quantizer, one fp32 per
//                       (block, head segment) pair: kOneLaunchMaxBlocks + 4*B*H slots
constexpr size_t kWsStatusOffset = 0;
constexpr size_t kWsDetailOffset = 4;
constexpr size_t kWsCounterOffset = 16;
constexpr size_t kWsAmaxOffset = 256;
constexpr int kOneLaunchMaxBlocks = 1024;
// detail code (bits 24..31 of the detail word) of an expired wait at the one-launch quantizer's grid barrier
constexpr uint32_t kDetailQuantizeGridWait = 32;

inline size_t ws_amax_bytes(int B, int H) {
    size_t amax = (size_t)12 * (size_t)B * (size_t)H;
    return ((amax + 255) / 256) * 256;
}
inline size_t ws_partial_offset(int B, int H) { return kWsAmaxOffset + ws_amax_bytes(B, H); }
inline size_t workspace_bytes(int B, int H) {
    size_t partial = sizeof(float) * ((size_t)kOneLaunchMaxBlocks + (size_t)4 * (size_t)B * (size_t)H);
    return ws_partial_offset(B, H) + ((partial + 255) / 256) * 256;
}

// Scratch of the tail split (FP8ATTN_SPLIT_TAIL), appended to the workspace: partial results
// of fewer than one CTA per SM of the current device, 256 rows of d + 4 floats each (api.cu).
size_t split_scratch_bytes(int d);

void count_launch();

// quantize.cu
int launch_quantize(const void* x_bf16, int64_t n_heads, int64_t elems_per_head,
                    const float* scale_in, void* x_fp8, float* scale_out,
                    uint32_t* amax_bits, uint32_t flags, cudaStream_t stream);

// `status`, `counters`, `partial`: the workspace's status words, arrival counters and
// partial-maximum slots (the one-launch path for small calls uses them).
int launch_quantize_qkv(const void* q_train, const void* k, const void* v, const void* q_test,
                        int64_t n_heads, int64_t elems_train, int64_t elems_test, void* q_train_fp8,
                        void* k_fp8, void* v_fp8, void* q_test_fp8, float* scale_q, float* scale_k,
                        float* scale_v, uint32_t* amax_bits, uint32_t flags, uint32_t* status,
                        uint32_t* counters, float* partial, cudaStream_t stream,
                        int32_t* key_dest = nullptr, int d = 64);

// key_order.cu
// dest[b,h,r] = the row that key r of head (b,h) moves to: the keys of largest norm first.
// norm_scratch: device memory for one fp32 per key (its squared norm), the heads
// norm_stride_bytes apart; compute_norms: fill it from k16 first (else it is filled already).
int launch_key_order(const void* k16, int64_t n_heads, int64_t n_train, int d, bool half, int32_t* dest,
                     void* norm_scratch, int64_t norm_stride_bytes, bool compute_norms, cudaStream_t stream);
// out[b,h,dest[b,h,r],:] = x[b,h,r,:] for a 16-bit tensor
int launch_reorder_rows(const void* x16, int64_t n_heads, int64_t rows, int d, const int32_t* dest, void* out16,
                        cudaStream_t stream);

// perturb.cu
int launch_perturb(const void* x_bf16, int64_t n_heads, int64_t elems_per_head, float epsilon,
                   uint64_t seed, uint32_t stream_id, void* out_bf16, float* rho_out, double* sumsq,
                   cudaStream_t stream);

// attention.cu
struct AttnParams {
    const void* q_train; const void* q_test; const void* k; const void* v;
    const float* scale_q; const float* scale_k; const float* scale_v;  // NULL for bf16
    int B, H; int64_t n_train, n_test; int d;
    float softmax_scale;
    uint32_t flags;    // FP8ATTN_* forward flags
    void* out_train; void* out_test;
    uint32_t* status;  // workspace status words
    float* partial;    // scratch of the tail split (NULL: none)
    size_t partial_bytes;
};
int launch_icl_attention(const AttnParams& p, bool fp8, cudaStream_t stream);
// Query rows per CTA that a forward call of these sizes uses on a device with `sms` SMs: 256, or
// 384 at d = 64 where the grid of 384-row blocks fills the SMs at least eight times over.
int attention_rows_per_cta(int B, int H, int64_t n_train, int64_t n_test, int d, uint32_t flags, int sms);
int launch_wait_timeout_selftest(uint32_t* status, uint64_t limit_ns, cudaStream_t stream);

}  // namespace fp8attn
