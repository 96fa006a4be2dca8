// One whole step of the path (quantize + both attention calls) from HOST tensors to HOST
// results: fp8attn_icl_step_host.  The heads of a call are independent (per-head scales,
// per-head attention), so the call is cut into chunks of whole heads that run as a three-stage
// pipeline on three streams: copy-in of chunk c+1, quantize + attention of chunk c and copy-out
// of chunk c-1 overlap.  Two sets of device buffers inside the caller's scratch alternate
// between chunks.  Everything is enqueued; the host is not synchronised.
#include <cuda_runtime.h>

#include "common.h"

namespace fp8attn {
namespace {

constexpr int kMaxChunks = 8;
constexpr int64_t kPipelineMinBytes = 32ll << 20;   // 16-bit input bytes below which one chunk is used

size_t up256(size_t x) { return (x + 255) / 256 * 256; }

struct Plan {
    int heads;            // B*H
    int chunk_heads;      // heads per chunk
    int chunks;
    int sets;             // device buffer sets (1 or 2)
    size_t in_train, in_test, out_train, out_test;   // bytes per chunk (16-bit tensors)
    size_t ws;            // workspace bytes per set
    // offsets inside one set
    size_t off_ws, off_q, off_k, off_v, off_t, off_q8, off_k8, off_v8, off_t8, off_scales, off_otr, off_ote, off_order;
    size_t set_bytes;
};

Plan make_plan(int B, int H, int64_t n_train, int64_t n_test, int d, uint32_t flags) {
    Plan p{};
    p.heads = B * H;
    const int64_t head_in = (3 * n_train + n_test) * (int64_t)d * 2;
    p.chunk_heads = p.heads;
    if (!(flags & FP8ATTN_HOST_ONE_CHUNK) && head_in * p.heads >= kPipelineMinBytes && p.heads > 1)
        p.chunk_heads = (p.heads + kMaxChunks - 1) / kMaxChunks;
    p.chunks = (p.heads + p.chunk_heads - 1) / p.chunk_heads;
    p.sets = p.chunks > 1 ? 2 : 1;
    const size_t g = (size_t)p.chunk_heads;
    p.in_train = g * (size_t)n_train * d * 2;
    p.in_test = g * (size_t)n_test * d * 2;
    p.out_train = p.in_train;
    p.out_test = p.in_test;
    p.ws = up256(fp8attn_workspace_bytes(1, p.chunk_heads, n_train, n_test, d));
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o += up256(bytes); return at; };
    p.off_ws = take(p.ws);
    p.off_q = take(p.in_train);
    p.off_k = take(p.in_train);
    p.off_v = take(p.in_train);
    p.off_t = take(p.in_test);
    p.off_q8 = take(p.in_train / 2);
    p.off_k8 = take(p.in_train / 2);
    p.off_v8 = take(p.in_train / 2);
    p.off_t8 = take(p.in_test / 2);
    p.off_scales = take(3 * g * sizeof(float));
    p.off_otr = take(p.out_train);
    p.off_ote = take(p.out_test);
    p.off_order = take((flags & FP8ATTN_HOST_ORDER_KEYS) ? g * (size_t)n_train * sizeof(int32_t) : 0);
    p.set_bytes = o;
    return p;
}

bool args_ok(int B, int H, int64_t n_train, int64_t n_test, int d) {
    return B > 0 && H > 0 && n_train >= 1 && n_test >= 0 && (int64_t)B * H <= 65535 &&
           n_train < (1ll << 31) - 256 && n_test < (1ll << 31) - 256 && (d == 64 || d == 128);
}

}  // namespace
}  // namespace fp8attn

extern "C" size_t fp8attn_host_step_scratch_bytes(int B, int H, int64_t n_train, int64_t n_test, int d,
                                                  uint32_t flags) {
    using namespace fp8attn;
    if (!args_ok(B, H, n_train, n_test, d)) return 0;
    const Plan p = make_plan(B, H, n_train, n_test, d, flags);
    return p.set_bytes * (size_t)p.sets;
}

extern "C" int fp8attn_host_step_chunks(int B, int H, int64_t n_train, int64_t n_test, int d, uint32_t flags) {
    using namespace fp8attn;
    if (!args_ok(B, H, n_train, n_test, d)) return 0;
    return make_plan(B, H, n_train, n_test, d, flags).chunks;
}

extern "C" int fp8attn_icl_step_host(const void* q_train, const void* k, const void* v, const void* q_test,
                                     int B, int H, int64_t n_train, int64_t n_test, int d,
                                     float softmax_scale, uint32_t flags, void* out_train, void* out_test,
                                     void* device_scratch, size_t device_scratch_bytes, void* cuda_stream) {
    using namespace fp8attn;
    if (flags & ~(FP8ATTN_HOST_ONE_CHUNK | FP8ATTN_HOST_FP16 | FP8ATTN_HOST_ORDER_KEYS)) return FP8ATTN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || n_train < 1 || n_test < 0) return FP8ATTN_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return FP8ATTN_ERR_UNSUPPORTED;
    if (!args_ok(B, H, n_train, n_test, d)) return FP8ATTN_ERR_UNSUPPORTED;
    if (!q_train || !k || !v || !out_train) return FP8ATTN_ERR_INVALID_ARG;
    if (n_test > 0 && (!q_test || !out_test)) return FP8ATTN_ERR_INVALID_ARG;
    const Plan p = make_plan(B, H, n_train, n_test, d, flags);
    if (!device_scratch || reinterpret_cast<uintptr_t>(device_scratch) % 256 ||
        device_scratch_bytes < p.set_bytes * (size_t)p.sets)
        return FP8ATTN_ERR_WORKSPACE;
    cudaStream_t user = static_cast<cudaStream_t>(cuda_stream);
    // the two-launch quantizer: host steps of different streams may share the GPU, and the blocks
    // of the one-launch form wait for one another
    const uint32_t qflags = FP8ATTN_QKV_TWO_LAUNCHES | ((flags & FP8ATTN_HOST_FP16) ? FP8ATTN_INPUT_FP16 : 0u);
    const uint32_t fflags = FP8ATTN_SPLIT_TAIL | ((flags & FP8ATTN_HOST_FP16) ? FP8ATTN_IO_FP16 : 0u);

    // streams and events of this call; destroying them at the end only marks them for release
    // once the work enqueued on them has completed
    cudaStream_t s_in = nullptr, s_cmp = nullptr, s_out = nullptr;
    cudaEvent_t e_start = nullptr, e_in[kMaxChunks] = {}, e_q[kMaxChunks] = {}, e_c[kMaxChunks] = {},
                e_o[kMaxChunks] = {}, e_end[3] = {};
    // (a call of one chunk has nothing to overlap: it runs on the caller's stream as it is)
    const bool own_streams = p.chunks > 1;
    bool ok = true;
    if (own_streams)
        ok = cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking) == cudaSuccess &&
             cudaStreamCreateWithFlags(&s_cmp, cudaStreamNonBlocking) == cudaSuccess &&
             cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&e_start, cudaEventDisableTiming) == cudaSuccess;
    else
        s_in = s_cmp = s_out = user;
    for (int c = 0; ok && own_streams && c < p.chunks; ++c)
        ok = cudaEventCreateWithFlags(&e_in[c], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&e_q[c], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&e_c[c], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&e_o[c], cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && own_streams && i < 3; ++i) ok = cudaEventCreateWithFlags(&e_end[i], cudaEventDisableTiming) == cudaSuccess;
    int rc = ok ? FP8ATTN_OK : FP8ATTN_ERR_CUDA;
    auto cu = [&](cudaError_t e) {
        if (e != cudaSuccess && rc == FP8ATTN_OK) rc = FP8ATTN_ERR_CUDA;
        return e == cudaSuccess;
    };
    // event calls order the internal streams; on the caller's own stream the order is given
    auto record = [&](cudaEvent_t e, cudaStream_t s) { if (own_streams) cu(cudaEventRecord(e, s)); };
    auto wait = [&](cudaStream_t s, cudaEvent_t e) { if (own_streams) cu(cudaStreamWaitEvent(s, e, 0)); };

    if (rc == FP8ATTN_OK) {
        // everything of this call comes after what the caller's stream holds so far
        record(e_start, user);
        wait(s_in, e_start);
        wait(s_cmp, e_start);
        wait(s_out, e_start);
        char* base = static_cast<char*>(device_scratch);
        // the small head of each set's workspace (status words, counters, accumulators) starts at zero
        const size_t ws_head = fp8attn_workspace_bytes(1, p.chunk_heads, 0, 0, d);
        for (int s = 0; s < p.sets; ++s) cu(cudaMemsetAsync(base + (size_t)s * p.set_bytes + p.off_ws, 0, ws_head, s_cmp));
        const size_t head_train = (size_t)n_train * d * 2, head_test = (size_t)n_test * d * 2;
        for (int c = 0; c < p.chunks && rc == FP8ATTN_OK; ++c) {
            const int h0 = c * p.chunk_heads;
            const int g = p.heads - h0 < p.chunk_heads ? p.heads - h0 : p.chunk_heads;
            char* set = base + (size_t)(c % p.sets) * p.set_bytes;
            const size_t bt = (size_t)g * head_train, be = (size_t)g * head_test;
            const char* hq = static_cast<const char*>(q_train) + (size_t)h0 * head_train;
            const char* hk = static_cast<const char*>(k) + (size_t)h0 * head_train;
            const char* hv = static_cast<const char*>(v) + (size_t)h0 * head_train;
            // ---- copy in (the set's 16-bit inputs are free once the quantizer of its last chunk is done) ----
            if (c >= p.sets) wait(s_in, e_q[c - p.sets]);
            cu(cudaMemcpyAsync(set + p.off_k, hk, bt, cudaMemcpyHostToDevice, s_in));
            cu(cudaMemcpyAsync(set + p.off_v, hv, bt, cudaMemcpyHostToDevice, s_in));
            cu(cudaMemcpyAsync(set + p.off_q, hq, bt, cudaMemcpyHostToDevice, s_in));
            if (n_test > 0)
                cu(cudaMemcpyAsync(set + p.off_t, static_cast<const char*>(q_test) + (size_t)h0 * head_test, be,
                                   cudaMemcpyHostToDevice, s_in));
            record(e_in[c], s_in);
            // ---- quantize + attention ----
            wait(s_cmp, e_in[c]);
            if (c >= p.sets) wait(s_cmp, e_o[c - p.sets]);   // the set's outputs have left
            float* scales = reinterpret_cast<float*>(set + p.off_scales);
            void* t16 = n_test > 0 ? set + p.off_t : nullptr;
            void* t8 = n_test > 0 ? set + p.off_t8 : nullptr;
            void* ote = n_test > 0 ? set + p.off_ote : nullptr;
            int r = (flags & FP8ATTN_HOST_ORDER_KEYS)
                        ? fp8attn_quantize_qkv_ordered(set + p.off_q, set + p.off_k, set + p.off_v, t16, 1, g, n_train,
                                                       n_test, d, set + p.off_q8, set + p.off_k8, set + p.off_v8, t8,
                                                       scales, scales + g, scales + 2 * g,
                                                       reinterpret_cast<int32_t*>(set + p.off_order), qflags,
                                                       set + p.off_ws, p.ws, s_cmp)
                        : fp8attn_quantize_qkv_ex(set + p.off_q, set + p.off_k, set + p.off_v, t16, 1, g, n_train,
                                                  n_test, d, set + p.off_q8, set + p.off_k8, set + p.off_v8, t8,
                                                  scales, scales + g, scales + 2 * g, qflags, set + p.off_ws, p.ws,
                                                  s_cmp);
            record(e_q[c], s_cmp);
            if (r == FP8ATTN_OK)
                r = fp8attn_icl_forward_ex(set + p.off_q8, t8, set + p.off_k8, set + p.off_v8, scales, scales + g,
                                           scales + 2 * g, 1, g, n_train, n_test, d, softmax_scale, fflags,
                                           set + p.off_otr, ote, set + p.off_ws, p.ws, s_cmp);
            if (r != FP8ATTN_OK && rc == FP8ATTN_OK) rc = r;
            record(e_c[c], s_cmp);
            // ---- copy out ----
            wait(s_out, e_c[c]);
            cu(cudaMemcpyAsync(static_cast<char*>(out_train) + (size_t)h0 * head_train, set + p.off_otr, bt,
                               cudaMemcpyDeviceToHost, s_out));
            if (n_test > 0)
                cu(cudaMemcpyAsync(static_cast<char*>(out_test) + (size_t)h0 * head_test, set + p.off_ote, be,
                                   cudaMemcpyDeviceToHost, s_out));
            record(e_o[c], s_out);
        }
        // the caller's stream continues after all three
        cudaStream_t all[3] = {s_in, s_cmp, s_out};
        for (int i = 0; i < 3; ++i) {
            record(e_end[i], all[i]);
            wait(user, e_end[i]);
        }
    }
    for (int c = 0; c < kMaxChunks; ++c) {
        if (e_in[c]) cudaEventDestroy(e_in[c]);
        if (e_q[c]) cudaEventDestroy(e_q[c]);
        if (e_c[c]) cudaEventDestroy(e_c[c]);
        if (e_o[c]) cudaEventDestroy(e_o[c]);
    }
    for (int i = 0; i < 3; ++i)
        if (e_end[i]) cudaEventDestroy(e_end[i]);
    if (e_start) cudaEventDestroy(e_start);
    if (own_streams) {
        if (s_in) cudaStreamDestroy(s_in);
        if (s_cmp) cudaStreamDestroy(s_cmp);
        if (s_out) cudaStreamDestroy(s_out);
    }
    return rc;
}

extern "C" int fp8attn_host_step_status(void* device_scratch, int B, int H, int64_t n_train, int64_t n_test,
                                        int d, uint32_t flags, void* cuda_stream, uint32_t* detail) {
    using namespace fp8attn;
    if (!device_scratch || !args_ok(B, H, n_train, n_test, d)) return FP8ATTN_ERR_INVALID_ARG;
    const Plan p = make_plan(B, H, n_train, n_test, d, flags);
    int rc = FP8ATTN_OK;
    for (int s = 0; s < p.sets; ++s) {
        uint32_t dt = 0;
        const int r = fp8attn_last_device_status(static_cast<char*>(device_scratch) + (size_t)s * p.set_bytes + p.off_ws,
                                                 cuda_stream, &dt);
        if (r != FP8ATTN_OK && rc == FP8ATTN_OK) {
            rc = r;
            if (detail) *detail = dt;
        }
    }
    if (rc == FP8ATTN_OK && detail) *detail = 0;
    return rc;
}
