/* fp8attn -- FP8 in-context-learning (ICL) attention for tabular foundation
 * models on NVIDIA B200 (sm_100a).  C ABI of libfp8attn.so.
 *
 * Conventions shared by every entry point
 *   - Every tensor pointer is a DEVICE pointer owned by the caller; the library
 *     allocates no device memory and keeps no pointer after a call returns.
 *   - Tensors are dense row-major [B, H, rows, d] with d innermost; base
 *     addresses must be 16-byte aligned.  bf16 tensors hold IEEE bfloat16 bit
 *     patterns, FP8 tensors hold e4m3fn codes (1-4-3, bias 7, no infinities,
 *     0x7F/0xFF = NaN, largest finite value 448).
 *   - `cuda_stream` is a cudaStream_t (NULL = the legacy default stream).  All
 *     work is enqueued on it; no entry point synchronises the host unless its
 *     description says so.
 *   - `workspace` is caller-owned device memory of at least
 *     fp8attn_workspace_bytes(...) bytes, 256-byte aligned, that must have been
 *     zero-filled once before its first use (cudaMemset).  Calls that share a
 *     workspace must be ordered on one stream; overlapping them races.
 *   - Return value: an fp8attn_status_t.  Argument errors are detected on the
 *     host before anything is launched.  Device-side problems (a bounded wait
 *     that ran out) are recorded in the workspace and read back with
 *     fp8attn_last_device_status(); the kernels never trap or spin forever.  A
 *     recorded device error is sticky: attention launches on that workspace do
 *     nothing until fp8attn_last_device_status() has read and cleared it.
 *   - Supported head dims: d = 64 and d = 128.  n_train >= 1, n_test >= 0, each
 *     below 2^31 - 256; B*H <= 65535.
 */
#ifndef FP8ATTN_H_
#define FP8ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FP8ATTN_OK = 0,
    FP8ATTN_ERR_INVALID_ARG = 1, /* null pointer, bad size, misaligned address   */
    FP8ATTN_ERR_UNSUPPORTED = 2, /* head dim other than 64/128, device not sm_100 */
    FP8ATTN_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small    */
    FP8ATTN_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed           */
    FP8ATTN_ERR_TIMEOUT = 5,     /* a device-side bounded wait expired            */
    FP8ATTN_ERR_TOO_LARGE = 6    /* more heads than the built-in scratch of the
                                    allocation-free entry point can hold          */
} fp8attn_status_t;

/* Per-head absmax quantization to e4m3 (paper Eq. 2, Method section).
 *
 *   s[b,h]  = max_{r,c} |x[b,h,r,c]| / 448        (fp32, IEEE division; 1.0 for an all-zero head)
 *   x8      = round_to_nearest_even_e4m3( clamp( x / s, -448, 448 ) )   (fp32 IEEE division)
 *
 *   x_bf16   in   bf16 [B,H,rows,d]
 *   scale_in in   NULL            -> the scale is computed from x itself (train queries, keys, values)
 *                 fp32 [B,H]      -> this scale is used instead and values outside its range saturate at
 *                                    +-448: the paper's shared train-query scale for the test queries,
 *                                    which keeps test predictions independent of the test batch.
 *   x_fp8    out  e4m3 [B,H,rows,d]
 *   scale_out out fp32 [B,H], the dequantization scale actually used (may be NULL when scale_in is given)
 *
 * rows may be 0 (nothing is written except scale_out when scale_in is given).
 * Inputs containing NaN or infinity are not supported.
 */
int fp8attn_quantize(const void* x_bf16, int B, int H, int64_t rows, int d,
                     const float* scale_in, void* x_fp8, float* scale_out,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/* fp8attn_quantize with a flags word.  FP8ATTN_INPUT_FP16: x holds IEEE fp16
 * instead of bf16 (the paper's kernel benchmark table runs in float16); the
 * arithmetic is the same, on the exact fp32 value of each input.  flags = 0 is
 * fp8attn_quantize.  Unknown flag bits return FP8ATTN_ERR_INVALID_ARG. */
#define FP8ATTN_INPUT_FP16 2u
int fp8attn_quantize_ex(const void* x_16bit, int B, int H, int64_t rows, int d,
                        const float* scale_in, void* x_fp8, float* scale_out, uint32_t flags,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The four quantizations of one ICL attention call in one or two launches
 * instead of seven (same arithmetic and bit-identical results to four
 * fp8attn_quantize calls): per-head absmax scales for Q_train, K and V (paper
 * Eq. 2), and Q_test quantized with the train-query scale (Method section, shared
 * query scale).  It removes most of the launch overhead that makes quantization
 * dominate at small train-row counts (the paper's latency tables below ~8k rows).
 * A call whose 16-bit inputs total at most 48 MB (they stay in L2) runs as ONE
 * launch of at most two thread blocks per SM: maximum, a grid-wide arrival
 * counter, conversion.  The blocks wait for one another, which presumes that they
 * are all resident at once, as they are on a GPU that runs nothing else; the wait
 * is bounded (2 s) and ends in FP8ATTN_ERR_TIMEOUT in the workspace's status word.
 * Callers that share the GPU with long-running kernels of other streams can ask
 * for the two-launch form with FP8ATTN_QKV_TWO_LAUNCHES (the _ex call).  Larger
 * calls always take two launches (maximum; conversion).
 *
 *   q_train, k, v   in  bf16 [B,H,n_train,d]      q_test in bf16 [B,H,n_test,d] (NULL iff n_test == 0)
 *   *_fp8           out e4m3, same shapes          scale_q/k/v out fp32 [B,H]
 * n_train >= 1, n_test >= 0.
 */
int fp8attn_quantize_qkv(const void* q_train, const void* k, const void* v, const void* q_test,
                         int B, int H, int64_t n_train, int64_t n_test, int d,
                         void* q_train_fp8, void* k_fp8, void* v_fp8, void* q_test_fp8,
                         float* scale_q, float* scale_k, float* scale_v,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/* fp8attn_quantize_qkv with a flags word.
 * FP8ATTN_QUERY_SCALE_FROM_ALL_ROWS: the query scale is the per-head absmax over
 * the train AND the test queries (the single-call form the paper uses for
 * TabICLv2, appendix: one attention call over all rows, quantized with per-head
 * dynamic scales).  Test predictions then depend on the test batch.  Without
 * the flag the scale comes from the train queries alone (the paper's proposal).
 * The "per-call query scale" ablation arm needs no flag: quantize the test
 * queries with fp8attn_quantize and scale_in = NULL.
 * FP8ATTN_INPUT_FP16 (above): all four inputs are IEEE fp16.
 * FP8ATTN_SCALES_GIVEN: scale_q, scale_k and scale_v are INPUTS, e.g. amax/448 with
 * the per-head maxima taken in the epilogue of the projection that produced Q, K
 * and V (the paper's method section notes that the quantization overhead is what
 * limits small tables).  No maximum pass runs: one launch, each element read
 * once; values outside a given scale's range saturate at +-448.  Not combinable
 * with FP8ATTN_QUERY_SCALE_FROM_ALL_ROWS.
 * FP8ATTN_QKV_TWO_LAUNCHES: never take the one-launch path of small calls. */
#define FP8ATTN_QUERY_SCALE_FROM_ALL_ROWS 1u
#define FP8ATTN_SCALES_GIVEN 4u
#define FP8ATTN_QKV_TWO_LAUNCHES 8u
int fp8attn_quantize_qkv_ex(const void* q_train, const void* k, const void* v, const void* q_test,
                            int B, int H, int64_t n_train, int64_t n_test, int d,
                            void* q_train_fp8, void* k_fp8, void* v_fp8, void* q_test_fp8,
                            float* scale_q, float* scale_k, float* scale_v, uint32_t flags,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);

/* fp8attn_quantize_qkv_ex that also chooses an order for the keys (the paper has no
 * counterpart: its kernel takes the keys as they come).  Attention sums over keys, so K and
 * V may be permuted together without changing the result; the order matters to the kernel
 * all the same, because every time a row's running maximum moves the accumulated output is
 * rescaled.  This call brings the keys of largest norm to the front (about 256 per head:
 * the rows whose squared norm, binned by exponent and four mantissa bits, lies at or above
 * the bin that the 32nd largest of every eighth row falls in), where, for most queries, the row maximum then
 * settles in the first step; all other keys follow in their old order.  Where more than 2048
 * rows of a head qualify (norms that single out no small group), that head keeps its order.
 *
 *   key_dest  out int32 [B,H,n_train] (device): the row that key r of head (b,h) was moved to,
 *             a permutation per head.  K8 and V8 are written in that order
 *             (k_fp8[b,h,key_dest[b,h,r],:] = code of k[b,h,r,:]); scales, Q8 and Q_test8 are
 *             those of fp8attn_quantize_qkv_ex.  It takes the two-launch form (whose maximum
 *             pass also leaves the key norms in the k_fp8 buffer, until the codes are written
 *             there) with one small launch for the order in between; with FP8ATTN_SCALES_GIVEN
 *             a pass of its own computes the norms.  Other arguments and flags as
 *             fp8attn_quantize_qkv_ex.
 *
 * The forward calls need nothing: pass the reordered K8 and V8.  Measured on B200: 3.5 % of
 * the attention time on tables whose row norms vary (log-normal, sigma 0.5), nothing on
 * tables whose rows have equal norms.  fp8attn_reorder_rows applies such a map to a 16-bit
 * tensor (out[b,h,dest[b,h,r],:] = x[b,h,r,:]; out must not be x), for callers that feed the
 * 16-bit forward with the same key order. */
int fp8attn_quantize_qkv_ordered(const void* q_train, const void* k, const void* v, const void* q_test,
                                 int B, int H, int64_t n_train, int64_t n_test, int d,
                                 void* q_train_fp8, void* k_fp8, void* v_fp8, void* q_test_fp8,
                                 float* scale_q, float* scale_k, float* scale_v, int32_t* key_dest,
                                 uint32_t flags, void* workspace, size_t workspace_bytes, void* cuda_stream);
int fp8attn_reorder_rows(const void* x_16bit, int B, int H, int64_t rows, int d, const int32_t* dest,
                         void* out_16bit, void* cuda_stream);

/* Fused FP8 ICL attention (paper Eq. 1 with the Method section's two-call
 * structure and quantization placement).
 *
 * For every (b,h): the n_train train queries attend to all n_train train keys
 * (non-causal, the diagonal included) and the n_test test queries attend to the
 * same n_train train keys only; both read the same quantized K and V.
 *
 *   S   = Q8 K8^T                         FP8 tensor-core product, fp32 accumulation
 *   x   = softmax_scale * s_q * s_k * S   (the Q and K scales are folded into the softmax scale)
 *   P   = exp(x - rowmax) lifted by 2^8 and rounded to e4m3 inside the kernel
 *         (the row maximum maps to 256 < 448); the normaliser sums the unrounded fp32 values
 *   out = bf16( s_v * (P8 V8) / rowsum )  (the V scale is applied in the epilogue)
 *
 *   q_train_fp8 in  e4m3 [B,H,n_train,d]     q_test_fp8 in e4m3 [B,H,n_test,d] (NULL iff n_test == 0)
 *   k_fp8,v_fp8 in  e4m3 [B,H,n_train,d]
 *   scale_q/k/v in  fp32 [B,H] device arrays (scale_q serves train AND test queries)
 *   softmax_scale   <= 0 selects 1/sqrt(d)
 *   out_train_bf16 out bf16 [B,H,n_train,d]  out_test_bf16 out bf16 [B,H,n_test,d] (NULL iff n_test == 0)
 */
int fp8attn_icl_forward(const void* q_train_fp8, const void* q_test_fp8,
                        const void* k_fp8, const void* v_fp8,
                        const float* scale_q, const float* scale_k, const float* scale_v,
                        int B, int H, int64_t n_train, int64_t n_test, int d,
                        float softmax_scale,
                        void* out_train_bf16, void* out_test_bf16,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same ICL attention on unquantized bf16 Q/K/V with bf16 probabilities: the
 * 16-bit comparison path (the paper's "ours 16-bit" control in its latency
 * tables).  Arguments as above without scales; all tensors bf16.
 */
int bf16attn_icl_forward(const void* q_train, const void* q_test, const void* k, const void* v,
                         int B, int H, int64_t n_train, int64_t n_test, int d,
                         float softmax_scale,
                         void* out_train_bf16, void* out_test_bf16,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Variants of the two forward calls with a flags word.
 *
 * FP8ATTN_TEST_ROWS_USE_KV_HEAD0: grouped-query test->train attention as in
 * TabPFN-v3 (paper appendix, noise-experiment details, where the test->train call
 * uses K/V head 0 only): the test queries of every head h of a table attend to the
 * keys and values of head 0 of that table (and use head 0's K and V scales; the
 * query scale stays head h's train-query scale).  Train rows are unaffected.
 * K and V are still passed, and were quantized, as full [B,H,n_train,d] tensors,
 * so both attention calls consume the same quantized K/V entries.
 *
 * FP8ATTN_TEST_ROWS_ONLY runs the test->train call alone: only out_test is
 * written, q_train and out_train are not read or written and may be NULL, and
 * n_test must be >= 1.  Together with the plain call at n_test = 0 (the
 * train->train call alone) this gives the arms of the paper's precision
 * ablation (results section, table of quantization arms: FP8 in the train
 * context only, in the test context only, in both): run one call through
 * fp8attn_icl_forward_ex and the other through bf16attn_icl_forward_ex.  The
 * test rows' results are bit-identical to those of the combined call.
 *
 * FP8ATTN_IO_FP16 switches the 16-bit tensors of the call from bf16 to IEEE
 * fp16 (the paper's kernel benchmark table runs in float16): the outputs of
 * fp8attn_icl_forward_ex, and the inputs, the on-chip probabilities and the
 * outputs of bf16attn_icl_forward_ex (which then is an fp16 kernel).
 *
 * FP8ATTN_SPLIT_TAIL balances the last, partly filled round of the launch.  The
 * grid is one CTA per 256 query rows of a head (per 384 at d = 64 in launches of
 * eight rounds and more, which the split does not apply to); when the number of CTAs is not
 * a multiple of the number of SMs, the CTAs left over after the last full
 * round would run alone on a fraction of the GPU.  With this flag each of them
 * is replaced by up to 16 CTAs that share its query rows and divide the train
 * keys between them, followed by a small kernel that combines their partial
 * results (the online softmax of the paper's kernel, applied once more across
 * key ranges).  The workspace must then be at least
 * fp8attn_workspace_bytes(B, H, n_train, n_test, d) with n_train > 0, which
 * includes the scratch for the partial results, else
 * FP8ATTN_ERR_WORKSPACE.  The split is applied only where it was measured to
 * pay (launches of fewer than 8 CTAs per SM whose key ranges keep at least
 * four steps); elsewhere the flag changes nothing.  Results stay within the same tolerances, but which
 * rows take the split path depends on the sizes of the call, so a row's result
 * is no longer bit-identical across calls with different n_test.
 *
 * Unknown flag bits return FP8ATTN_ERR_INVALID_ARG.  flags = 0 is the plain call.
 */
#define FP8ATTN_TEST_ROWS_USE_KV_HEAD0 1u
#define FP8ATTN_TEST_ROWS_ONLY 2u
#define FP8ATTN_IO_FP16 4u
#define FP8ATTN_SPLIT_TAIL 8u
int fp8attn_icl_forward_ex(const void* q_train_fp8, const void* q_test_fp8,
                           const void* k_fp8, const void* v_fp8,
                           const float* scale_q, const float* scale_k, const float* scale_v,
                           int B, int H, int64_t n_train, int64_t n_test, int d,
                           float softmax_scale, uint32_t flags,
                           void* out_train_bf16, void* out_test_bf16,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);
int bf16attn_icl_forward_ex(const void* q_train, const void* q_test, const void* k, const void* v,
                            int B, int H, int64_t n_train, int64_t n_test, int d,
                            float softmax_scale, uint32_t flags,
                            void* out_train_bf16, void* out_test_bf16,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The paper's dispatch gate (Method section: the quantization overhead is
 * amortised for N > 8192 train rows, and the final configuration uses FP8 only
 * then).  Host-only helper, returns 1 if the FP8 path should be used for this
 * many train rows, else 0 (use bf16attn_icl_forward).  Policy, not enforced:
 * fp8attn_icl_forward itself runs at any size. */
#define FP8ATTN_GATE_TRAIN_ROWS 8192
int fp8attn_gate_use_fp8(int64_t n_train);

/* Informational, host only (the paper has no counterpart): the number of query rows that
 * one CTA of the forward calls takes for a call of these sizes and flags on the current
 * device: 256 (two 128-row tiles), or 384 (three) at d = 64 when the grid of 384-row
 * blocks fills the SMs at least eight times over.  Without a device the SM count of a
 * B200 (148) is assumed.  0 for unsupported sizes.  Results do not depend on it beyond the
 * order of the online softmax (steps of 128 or 96 keys). */
int fp8attn_attention_rows_per_cta(int B, int H, int64_t n_train, int64_t n_test, int d, uint32_t flags);

/* Seeded Gaussian perturbation of Q, K or V (paper appendix, Eq. 3: the noise
 * experiment that replaces quantization by an explicit perturbation):
 *
 *   x~[b,h] = x[b,h] + epsilon * rho[b,h] * Z,   rho[b,h] = sqrt( mean over the head of x^2 ),
 *   Z iid N(0,1), independent per head; the paper sweeps epsilon over {1..5} x 0.0265.
 *
 *   x_bf16 in bf16 [B,H,rows,d]; out_bf16 out, same shape (may alias x_bf16);
 *   rho_out out fp32 [B,H] or NULL.
 * Z is a pure function of (seed, stream_id, b*H+h, element index): the noise
 * field is reproducible from the seed, and different stream_id values (one per
 * tensor and layer, say) give independent fields.  rho is summed with fp64 atomic
 * additions whose order varies between runs, so rho can differ in its last bit from
 * run to run, and with it (rarely) the rounding of an output element.  Perturbing K and V once and passing the
 * result to fp8attn_icl_forward / bf16attn_icl_forward is the paper's
 * "coordinated" arm: both attention calls then consume the same noisy K, V.
 * The normals come from Box-Muller in fp32 (hardware log / sin / cos), the sum of
 * squares is accumulated in fp64; results agree with an fp64 evaluation to within
 * one bf16 rounding step of the result (plus ~1e-6 of the two terms where they cancel).
 */
int fp8attn_perturb(const void* x_bf16, int B, int H, int64_t rows, int d,
                    float epsilon, uint64_t seed, uint32_t stream_id,
                    void* out_bf16, float* rho_out,
                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Allocation-free quantizer (the paper has no counterpart; this is a
 * packaging variant of fp8attn_quantize, same arithmetic, same results).
 *
 * Some hosts can give this library nothing but input and output buffers and may
 * not allocate device memory on its behalf: an inference runtime's plugin slot
 * that has no workspace argument, a serving process whose memory pool already
 * owns all of HBM (a cudaMalloc there fails or fragments the pool), or a
 * latency-critical loop that cannot afford the device-wide synchronisation
 * cudaMalloc implies.  For them the per-head absmax accumulators live in a
 * fixed array inside the library image instead of a caller-provided workspace.
 * The array holds FP8ATTN_NOALLOC_MAX_HEADS 32-bit slots (16 KiB) and stays
 * resident on every GPU that loads the library until the process exits.
 *
 *   - Arguments as fp8attn_quantize, without the workspace.  The caller still
 *     passes x_bf16, x_fp8 and scale_out (device pointers it owns).
 *   - B*H > FP8ATTN_NOALLOC_MAX_HEADS returns FP8ATTN_ERR_TOO_LARGE and
 *     launches nothing.
 *   - The call performs no cudaMalloc / cudaFree and calls no allocating
 *     library routine.  The first call on each device looks up the device
 *     address of the built-in array (cudaGetSymbolAddress, with that device
 *     current); make that first call outside any stream capture.
 *   - Every call on a device shares the one array and the array keeps the last
 *     call's contents: each call clears the slots it uses before accumulating,
 *     and two calls that overlap on the GPU (different streams, no ordering
 *     between them) race on it.  Order them on one stream or with events.
 */
#define FP8ATTN_NOALLOC_MAX_HEADS 4096
int fp8attn_quantize_noalloc(const void* x_bf16, int B, int H, int64_t rows, int d,
                             const float* scale_in, void* x_fp8, float* scale_out,
                             void* cuda_stream);

/* One whole step of the path from HOST memory to HOST memory: the four tensors of an
 * ICL attention call are copied to the device, quantized (fp8attn_quantize_qkv, paper
 * Eq. 2 with the shared train-query scale), both attention calls run
 * (fp8attn_icl_forward_ex with FP8ATTN_SPLIT_TAIL), and the 16-bit results are copied
 * back.  The paper has no counterpart; this is the form a caller with host-resident
 * tables uses, and the one the end-to-end latency of a call is measured on.
 *
 * Heads are independent in every step of the path, so a large call is cut into up to 8
 * chunks of whole heads that run as a pipeline on three internal streams (copy-in of the
 * next chunk, compute of the current one, copy-out of the previous one overlap; two sets
 * of device buffers alternate).  Calls whose 16-bit inputs total less than 32 MB, and
 * calls with FP8ATTN_HOST_ONE_CHUNK, run as one chunk.  Results are those of the
 * device-pointer calls on the same data (a chunk is a call with B = 1 and the chunk's
 * heads; with FP8ATTN_SPLIT_TAIL, which rows take the split path depends on the chunking).
 *
 *   q_train, k, v  in  HOST bf16 [B,H,n_train,d]    q_test in HOST bf16 [B,H,n_test,d] (NULL iff n_test == 0)
 *   out_train      out HOST bf16 [B,H,n_train,d]    out_test out HOST bf16 [B,H,n_test,d] (NULL iff n_test == 0)
 *   device_scratch DEVICE memory owned by the caller, 256-byte aligned, at least
 *                  fp8attn_host_step_scratch_bytes(...) bytes with the same sizes and flags;
 *                  its contents on entry do not matter
 *   flags          FP8ATTN_HOST_ONE_CHUNK (no pipeline), FP8ATTN_HOST_FP16 (all 16-bit tensors
 *                  are IEEE fp16), FP8ATTN_HOST_ORDER_KEYS (quantize with
 *                  fp8attn_quantize_qkv_ordered: the keys of largest norm first); other bits:
 *                  FP8ATTN_ERR_INVALID_ARG
 *
 * The host buffers should be page-locked: copies from pageable memory are staged by the
 * CUDA runtime and do not overlap.  The call only enqueues work (after everything already
 * in `cuda_stream`; `cuda_stream` continues after the last copy-out), so the host buffers
 * must stay valid, and the outputs are complete, once `cuda_stream` has been synchronised.
 * Calls made on different streams (each with its own scratch and host buffers) may be in
 * flight together: the copies and kernels of one overlap those of the other.
 * The library allocates no device memory here either; it creates and releases three
 * streams and a few events per call.  fp8attn_host_step_status synchronises `cuda_stream`
 * and returns the device status of the call's workspaces (inside the scratch), like
 * fp8attn_last_device_status.  fp8attn_host_step_chunks returns the number of chunks
 * the call is cut into (0 for unsupported sizes, like the scratch size). */
#define FP8ATTN_HOST_ONE_CHUNK 1u
#define FP8ATTN_HOST_FP16 2u
#define FP8ATTN_HOST_ORDER_KEYS 4u
size_t fp8attn_host_step_scratch_bytes(int B, int H, int64_t n_train, int64_t n_test, int d,
                                       uint32_t flags);
int fp8attn_host_step_chunks(int B, int H, int64_t n_train, int64_t n_test, int d, uint32_t flags);
int fp8attn_icl_step_host(const void* q_train, const void* k, const void* v, const void* q_test,
                          int B, int H, int64_t n_train, int64_t n_test, int d,
                          float softmax_scale, uint32_t flags, void* out_train, void* out_test,
                          void* device_scratch, size_t device_scratch_bytes, void* cuda_stream);
int fp8attn_host_step_status(void* device_scratch, int B, int H, int64_t n_train, int64_t n_test,
                             int d, uint32_t flags, void* cuda_stream, uint32_t* detail);

/* Bytes of workspace the calls above need: a few KB for the status words and the
 * per-head accumulators (all that is returned for n_train = 0), plus, for
 * n_train > 0 and d in {64, 128}, the scratch of FP8ATTN_SPLIT_TAIL (about 13 MB
 * at d = 64, 26 MB at d = 128; independent of n_train and n_test).  A workspace
 * of the smaller size serves every call that does not set that flag. */
size_t fp8attn_workspace_bytes(int B, int H, int64_t n_train, int64_t n_test, int d);

/* Synchronises `cuda_stream`, reads and clears the device status word of
 * `workspace`, and returns it (FP8ATTN_OK, FP8ATTN_ERR_TIMEOUT, or
 * FP8ATTN_ERR_CUDA if the stream reported an error).  `detail`, if not NULL,
 * receives a kernel-specific code saying which wait expired.  For tests. */
int fp8attn_last_device_status(void* workspace, void* cuda_stream, uint32_t* detail);

/* Self-test of the device-side error path (no counterpart in the paper).  Every
 * wait inside the attention kernels is bounded; this launches one warp that
 * waits, with a limit of limit_us microseconds (1..100000), on a barrier nothing
 * ever signals, so the wait expires, FP8ATTN_ERR_TIMEOUT is recorded in the
 * workspace and the kernel returns normally.  fp8attn_last_device_status() then
 * reports it; until that call has cleared it, attention launches on the
 * workspace do nothing.  The GPU context stays usable throughout. */
int fp8attn_selftest_wait_timeout(void* workspace, size_t workspace_bytes, uint32_t limit_us,
                                  void* cuda_stream);

/* Static, human-readable name of a status code. */
const char* fp8attn_status_string(int status);

/* Number of kernels the library has launched in this process so far (all
 * entry points, all threads).  Used by benchmarks to report launch counts. */
uint64_t fp8attn_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* FP8ATTN_H_ */
