// extern "C" entry points of libfp8attn.so: argument checking and dispatch.
#include <atomic>
#include <math.h>

#include "common.h"

namespace fp8attn {

static std::atomic<uint64_t> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

size_t split_scratch_bytes(int d) {
    // one unit per SM at most; without a device to ask (size queries on a host without
    // a GPU) the size assumes the largest sm_100 part
    constexpr int kSmsWithoutDevice = 160;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = kSmsWithoutDevice;
    return (size_t)sms * 256 * (size_t)(d + 4) * sizeof(float);
}

namespace {

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_shape(int B, int H, int d) {
    if (B <= 0 || H <= 0) return FP8ATTN_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return FP8ATTN_ERR_UNSUPPORTED;
    return FP8ATTN_OK;
}

int check_workspace(const void* ws, size_t bytes, int B, int H) {
    if (ws == nullptr || !aligned(ws, 256) || bytes < workspace_bytes(B, H)) return FP8ATTN_ERR_WORKSPACE;
    return FP8ATTN_OK;
}

// The kernels are built for sm_100a only.
int check_device() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FP8ATTN_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return FP8ATTN_ERR_CUDA;
    return major == 10 ? FP8ATTN_OK : FP8ATTN_ERR_UNSUPPORTED;
}

int forward(bool fp8, const void* q_train, const void* q_test, const void* k, const void* v,
            const float* sq, const float* sk, const float* sv, int B, int H, int64_t n_train,
            int64_t n_test, int d, float softmax_scale, void* out_train, void* out_test,
            void* workspace, size_t workspace_bytes_, void* stream, uint32_t flags = 0) {
    int rc = check_shape(B, H, d);
    if (rc != FP8ATTN_OK) return rc;
    if (n_train < 1 || n_test < 0 || n_train > 0x7fffff00ll || n_test > 0x7fffff00ll)
        return FP8ATTN_ERR_INVALID_ARG;
    if (flags & ~(uint32_t)(FP8ATTN_TEST_ROWS_USE_KV_HEAD0 | FP8ATTN_TEST_ROWS_ONLY | FP8ATTN_IO_FP16 |
                            FP8ATTN_SPLIT_TAIL))
        return FP8ATTN_ERR_INVALID_ARG;
    const bool test_only = (flags & FP8ATTN_TEST_ROWS_ONLY) != 0;
    if (test_only && n_test < 1) return FP8ATTN_ERR_INVALID_ARG;
    if (!k || !v || (!test_only && (!q_train || !out_train))) return FP8ATTN_ERR_INVALID_ARG;
    if (n_test > 0 && (!q_test || !out_test)) return FP8ATTN_ERR_INVALID_ARG;
    if (fp8 && (!sq || !sk || !sv)) return FP8ATTN_ERR_INVALID_ARG;
    if (!aligned(k, 16) || !aligned(v, 16) ||
        (!test_only && (!aligned(q_train, 16) || !aligned(out_train, 16))) ||
        (n_test > 0 && (!aligned(q_test, 16) || !aligned(out_test, 16))))
        return FP8ATTN_ERR_INVALID_ARG;
    if (!(softmax_scale == softmax_scale) || isinf(softmax_scale)) return FP8ATTN_ERR_INVALID_ARG;
    rc = check_workspace(workspace, workspace_bytes_, B, H);
    if (rc != FP8ATTN_OK) return rc;
    if ((flags & FP8ATTN_SPLIT_TAIL) && workspace_bytes_ < workspace_bytes(B, H) + split_scratch_bytes(d))
        return FP8ATTN_ERR_WORKSPACE;
    rc = check_device();
    if (rc != FP8ATTN_OK) return rc;
    AttnParams p;
    p.partial = nullptr;
    p.partial_bytes = 0;
    if (flags & FP8ATTN_SPLIT_TAIL) {
        p.partial = reinterpret_cast<float*>(static_cast<char*>(workspace) + workspace_bytes(B, H));
        p.partial_bytes = workspace_bytes_ - workspace_bytes(B, H);
    }
    p.q_train = q_train; p.q_test = q_test; p.k = k; p.v = v;
    p.scale_q = sq; p.scale_k = sk; p.scale_v = sv;
    p.B = B; p.H = H; p.n_train = n_train; p.n_test = n_test; p.d = d;
    p.softmax_scale = softmax_scale;
    p.flags = flags;
    p.out_train = out_train; p.out_test = out_test;
    p.status = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + kWsStatusOffset);
    return launch_icl_attention(p, fp8, static_cast<cudaStream_t>(stream));
}

}  // namespace
}  // namespace fp8attn

using namespace fp8attn;

extern "C" {

int fp8attn_quantize(const void* x_bf16, int B, int H, int64_t rows, int d, const float* scale_in,
                     void* x_fp8, float* scale_out, void* workspace, size_t workspace_bytes_,
                     void* cuda_stream) {
    return fp8attn_quantize_ex(x_bf16, B, H, rows, d, scale_in, x_fp8, scale_out, 0u, workspace,
                               workspace_bytes_, cuda_stream);
}

int fp8attn_quantize_ex(const void* x_bf16, int B, int H, int64_t rows, int d, const float* scale_in,
                        void* x_fp8, float* scale_out, uint32_t flags, void* workspace,
                        size_t workspace_bytes_, void* cuda_stream) {
    int rc = check_shape(B, H, d);
    if (rc != FP8ATTN_OK) return rc;
    if (flags & ~(uint32_t)FP8ATTN_INPUT_FP16) return FP8ATTN_ERR_INVALID_ARG;
    if (rows < 0) return FP8ATTN_ERR_INVALID_ARG;
    if (rows > 0 && (!x_bf16 || !x_fp8)) return FP8ATTN_ERR_INVALID_ARG;
    if (!scale_in && !scale_out) return FP8ATTN_ERR_INVALID_ARG;
    if (!aligned(x_bf16, 16) || !aligned(x_fp8, 16) || !aligned(scale_in, 4) || !aligned(scale_out, 4))
        return FP8ATTN_ERR_INVALID_ARG;
    rc = check_workspace(workspace, workspace_bytes_, B, H);
    if (rc != FP8ATTN_OK) return rc;
    rc = check_device();
    if (rc != FP8ATTN_OK) return rc;
    uint32_t* amax = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + kWsAmaxOffset);
    return launch_quantize(x_bf16, (int64_t)B * H, rows * (int64_t)d, scale_in, x_fp8, scale_out, amax,
                           flags, static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"

namespace {
// key_dest: NULL for the plain call; else the keys are ordered first and K, V written in that order
int quantize_qkv_impl(const void* q_train, const void* k, const void* v, const void* q_test, int B,
                      int H, int64_t n_train, int64_t n_test, int d, void* q_train_fp8, void* k_fp8,
                      void* v_fp8, void* q_test_fp8, float* scale_q, float* scale_k, float* scale_v,
                      int32_t* key_dest, uint32_t flags, void* workspace, size_t workspace_bytes_,
                      void* cuda_stream) {
    int rc = check_shape(B, H, d);
    if (rc != FP8ATTN_OK) return rc;
    if (n_train < 1 || n_test < 0) return FP8ATTN_ERR_INVALID_ARG;
    if (flags & ~(uint32_t)(FP8ATTN_QUERY_SCALE_FROM_ALL_ROWS | FP8ATTN_INPUT_FP16 | FP8ATTN_SCALES_GIVEN |
                            FP8ATTN_QKV_TWO_LAUNCHES))
        return FP8ATTN_ERR_INVALID_ARG;
    if ((flags & FP8ATTN_SCALES_GIVEN) && (flags & FP8ATTN_QUERY_SCALE_FROM_ALL_ROWS))
        return FP8ATTN_ERR_INVALID_ARG;
    if (!q_train || !k || !v || !q_train_fp8 || !k_fp8 || !v_fp8 || !scale_q || !scale_k || !scale_v)
        return FP8ATTN_ERR_INVALID_ARG;
    if (n_test > 0 && (!q_test || !q_test_fp8)) return FP8ATTN_ERR_INVALID_ARG;
    const void* ptrs[8] = {q_train, k, v, q_test, q_train_fp8, k_fp8, v_fp8, q_test_fp8};
    for (const void* p : ptrs)
        if (!aligned(p, 16)) return FP8ATTN_ERR_INVALID_ARG;
    rc = check_workspace(workspace, workspace_bytes_, B, H);
    if (rc != FP8ATTN_OK) return rc;
    rc = check_device();
    if (rc != FP8ATTN_OK) return rc;
    uint32_t* amax = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + kWsAmaxOffset);
    char* ws = static_cast<char*>(workspace);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    return launch_quantize_qkv(q_train, k, v, q_test, (int64_t)B * H, n_train * (int64_t)d,
                               n_test * (int64_t)d, q_train_fp8, k_fp8, v_fp8, q_test_fp8, scale_q, scale_k,
                               scale_v, amax, flags, reinterpret_cast<uint32_t*>(ws + kWsStatusOffset),
                               reinterpret_cast<uint32_t*>(ws + kWsCounterOffset),
                               reinterpret_cast<float*>(ws + ws_partial_offset(B, H)), stream, key_dest, d);
}
}  // namespace

extern "C" {

int fp8attn_quantize_qkv_ex(const void* q_train, const void* k, const void* v, const void* q_test, int B,
                         int H, int64_t n_train, int64_t n_test, int d, void* q_train_fp8, void* k_fp8,
                         void* v_fp8, void* q_test_fp8, float* scale_q, float* scale_k, float* scale_v,
                         uint32_t flags, void* workspace, size_t workspace_bytes_, void* cuda_stream) {
    return quantize_qkv_impl(q_train, k, v, q_test, B, H, n_train, n_test, d, q_train_fp8, k_fp8, v_fp8,
                             q_test_fp8, scale_q, scale_k, scale_v, nullptr, flags, workspace, workspace_bytes_,
                             cuda_stream);
}

int fp8attn_quantize_qkv_ordered(const void* q_train, const void* k, const void* v, const void* q_test, int B,
                                 int H, int64_t n_train, int64_t n_test, int d, void* q_train_fp8, void* k_fp8,
                                 void* v_fp8, void* q_test_fp8, float* scale_q, float* scale_k,
                                 float* scale_v, int32_t* key_dest, uint32_t flags, void* workspace,
                                 size_t workspace_bytes_, void* cuda_stream) {
    if (!key_dest || !aligned(key_dest, 4)) return FP8ATTN_ERR_INVALID_ARG;
    return quantize_qkv_impl(q_train, k, v, q_test, B, H, n_train, n_test, d, q_train_fp8, k_fp8, v_fp8,
                             q_test_fp8, scale_q, scale_k, scale_v, key_dest, flags, workspace, workspace_bytes_,
                             cuda_stream);
}

int fp8attn_reorder_rows(const void* x_16bit, int B, int H, int64_t rows, int d, const int32_t* dest,
                         void* out_16bit, void* cuda_stream) {
    int rc = check_shape(B, H, d);
    if (rc != FP8ATTN_OK) return rc;
    if (rows < 0) return FP8ATTN_ERR_INVALID_ARG;
    if (rows > 0 && (!x_16bit || !dest || !out_16bit || x_16bit == out_16bit)) return FP8ATTN_ERR_INVALID_ARG;
    if (!aligned(x_16bit, 16) || !aligned(out_16bit, 16) || !aligned(dest, 4)) return FP8ATTN_ERR_INVALID_ARG;
    rc = check_device();
    if (rc != FP8ATTN_OK) return rc;
    return launch_reorder_rows(x_16bit, (int64_t)B * H, rows, d, dest, out_16bit,
                               static_cast<cudaStream_t>(cuda_stream));
}

int fp8attn_quantize_qkv(const void* q_train, const void* k, const void* v, const void* q_test, int B,
                         int H, int64_t n_train, int64_t n_test, int d, void* q_train_fp8, void* k_fp8,
                         void* v_fp8, void* q_test_fp8, float* scale_q, float* scale_k, float* scale_v,
                         void* workspace, size_t workspace_bytes_, void* cuda_stream) {
    return fp8attn_quantize_qkv_ex(q_train, k, v, q_test, B, H, n_train, n_test, d, q_train_fp8, k_fp8,
                                   v_fp8, q_test_fp8, scale_q, scale_k, scale_v, 0u, workspace,
                                   workspace_bytes_, cuda_stream);
}

int fp8attn_icl_forward(const void* q_train_fp8, const void* q_test_fp8, const void* k_fp8,
                        const void* v_fp8, const float* scale_q, const float* scale_k,
                        const float* scale_v, int B, int H, int64_t n_train, int64_t n_test, int d,
                        float softmax_scale, void* out_train_bf16, void* out_test_bf16,
                        void* workspace, size_t workspace_bytes_, void* cuda_stream) {
    return forward(true, q_train_fp8, q_test_fp8, k_fp8, v_fp8, scale_q, scale_k, scale_v, B, H, n_train,
                   n_test, d, softmax_scale, out_train_bf16, out_test_bf16, workspace, workspace_bytes_,
                   cuda_stream);
}

int bf16attn_icl_forward(const void* q_train, const void* q_test, const void* k, const void* v, int B,
                         int H, int64_t n_train, int64_t n_test, int d, float softmax_scale,
                         void* out_train_bf16, void* out_test_bf16, void* workspace,
                         size_t workspace_bytes_, void* cuda_stream) {
    return forward(false, q_train, q_test, k, v, nullptr, nullptr, nullptr, B, H, n_train, n_test, d,
                   softmax_scale, out_train_bf16, out_test_bf16, workspace, workspace_bytes_, cuda_stream);
}

int fp8attn_icl_forward_ex(const void* q_train_fp8, const void* q_test_fp8, const void* k_fp8,
                           const void* v_fp8, const float* scale_q, const float* scale_k,
                           const float* scale_v, int B, int H, int64_t n_train, int64_t n_test, int d,
                           float softmax_scale, uint32_t flags, void* out_train_bf16,
                           void* out_test_bf16, void* workspace, size_t workspace_bytes_,
                           void* cuda_stream) {
    return forward(true, q_train_fp8, q_test_fp8, k_fp8, v_fp8, scale_q, scale_k, scale_v, B, H, n_train,
                   n_test, d, softmax_scale, out_train_bf16, out_test_bf16, workspace, workspace_bytes_,
                   cuda_stream, flags);
}

int bf16attn_icl_forward_ex(const void* q_train, const void* q_test, const void* k, const void* v, int B,
                            int H, int64_t n_train, int64_t n_test, int d, float softmax_scale,
                            uint32_t flags, void* out_train_bf16, void* out_test_bf16, void* workspace,
                            size_t workspace_bytes_, void* cuda_stream) {
    return forward(false, q_train, q_test, k, v, nullptr, nullptr, nullptr, B, H, n_train, n_test, d,
                   softmax_scale, out_train_bf16, out_test_bf16, workspace, workspace_bytes_, cuda_stream,
                   flags);
}

int fp8attn_perturb(const void* x_bf16, int B, int H, int64_t rows, int d, float epsilon, uint64_t seed,
                    uint32_t stream_id, void* out_bf16, float* rho_out, void* workspace,
                    size_t workspace_bytes_, void* cuda_stream) {
    int rc = check_shape(B, H, d);
    if (rc != FP8ATTN_OK) return rc;
    if (rows < 0 || !(epsilon == epsilon)) return FP8ATTN_ERR_INVALID_ARG;
    if (rows > 0 && (!x_bf16 || !out_bf16)) return FP8ATTN_ERR_INVALID_ARG;
    if (!aligned(x_bf16, 16) || !aligned(out_bf16, 16) || !aligned(rho_out, 4)) return FP8ATTN_ERR_INVALID_ARG;
    rc = check_workspace(workspace, workspace_bytes_, B, H);
    if (rc != FP8ATTN_OK) return rc;
    rc = check_device();
    if (rc != FP8ATTN_OK) return rc;
    double* sumsq = reinterpret_cast<double*>(static_cast<char*>(workspace) + kWsAmaxOffset);
    return launch_perturb(x_bf16, (int64_t)B * H, rows * (int64_t)d, epsilon, seed, stream_id, out_bf16,
                          rho_out, sumsq, static_cast<cudaStream_t>(cuda_stream));
}

int fp8attn_selftest_wait_timeout(void* workspace, size_t workspace_bytes_, uint32_t limit_us,
                                  void* cuda_stream) {
    if (limit_us == 0 || limit_us > 100000) return FP8ATTN_ERR_INVALID_ARG;
    int rc = check_workspace(workspace, workspace_bytes_, 1, 1);
    if (rc != FP8ATTN_OK) return rc;
    rc = check_device();
    if (rc != FP8ATTN_OK) return rc;
    return launch_wait_timeout_selftest(reinterpret_cast<uint32_t*>(workspace), (uint64_t)limit_us * 1000ull,
                                        static_cast<cudaStream_t>(cuda_stream));
}

int fp8attn_gate_use_fp8(int64_t n_train) { return n_train > FP8ATTN_GATE_TRAIN_ROWS ? 1 : 0; }

int fp8attn_attention_rows_per_cta(int B, int H, int64_t n_train, int64_t n_test, int d, uint32_t flags) {
    if (B <= 0 || H <= 0 || n_train < 0 || n_test < 0 || (d != 64 && d != 128)) return 0;
    // without a device to ask (a host without a GPU): the SM count of a B200
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    return fp8attn::attention_rows_per_cta(B, H, n_train, n_test, d, flags, sms);
}

size_t fp8attn_workspace_bytes(int B, int H, int64_t n_train, int64_t, int d) {
    if (B <= 0 || H <= 0) return 0;
    // with the size of an attention call: room for the tail split's partial results as well
    if (n_train > 0 && (d == 64 || d == 128)) return workspace_bytes(B, H) + split_scratch_bytes(d);
    return workspace_bytes(B, H);
}

int fp8attn_last_device_status(void* workspace, void* cuda_stream, uint32_t* detail) {
    if (!workspace) return FP8ATTN_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (cudaStreamSynchronize(s) != cudaSuccess) return FP8ATTN_ERR_CUDA;
    uint32_t words[2] = {0, 0};
    if (cudaMemcpy(words, workspace, sizeof(words), cudaMemcpyDeviceToHost) != cudaSuccess)
        return FP8ATTN_ERR_CUDA;
    if (detail) *detail = words[1];
    // after an error: clear the status words, and the arrival counters a one-launch
    // quantization that gave up may have left behind
    if (words[0] != 0 && cudaMemset(workspace, 0, kWsAmaxOffset) != cudaSuccess) return FP8ATTN_ERR_CUDA;
    return (int)words[0];
}

const char* fp8attn_status_string(int status) {
    switch (status) {
        case FP8ATTN_OK: return "ok";
        case FP8ATTN_ERR_INVALID_ARG: return "invalid argument";
        case FP8ATTN_ERR_UNSUPPORTED: return "unsupported head dimension, size or device";
        case FP8ATTN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case FP8ATTN_ERR_CUDA: return "CUDA call failed";
        case FP8ATTN_ERR_TIMEOUT: return "device-side wait timed out";
        case FP8ATTN_ERR_TOO_LARGE:
            return "more heads than the built-in scratch of fp8attn_quantize_noalloc holds";
        default: return "unknown status";
    }
}

uint64_t fp8attn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
