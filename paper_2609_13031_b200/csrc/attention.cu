// Fused ICL attention for sm_100a: train->train and test->train in one launch.
//
// One CTA owns up to 256 query rows (two 128-row tiles) of one (b,h) and walks
// over all train keys in tiles of 128.  Warp roles:
//   warps 0-3  softmax of query tile 0 (one row per thread)
//   warps 4-7  softmax of query tile 1
//   warp  8    issues every tcgen05.mma (one elected thread)
//   warp  9    TMA producer for Q, K and V tiles
// Tensor memory (512 columns): S0 | S1 | O0 | O1.  The probability tile P_t is
// written over the first columns of S_t (as e4m3 with the row maximum lifted to
// 2^8, or as bf16 in the 16-bit path) and is the tensor-memory A operand of
// O_t += P_t V.  While one tile's softmax runs on the CUDA cores, the tensor
// core works on the other tile.
//
// Scale placement (FP8 path): x = (alpha * s_q * s_k * log2 e) * S feeds exp2;
// the V scale and 1/rowsum are applied to O in the epilogue.
#include <cuda_bf16.h>

#include "common.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace fp8attn {
namespace {

using namespace ptx;

constexpr int kTileM = 128;         // query rows per tile
constexpr int kTileN = 128;         // keys per step
constexpr int kNumThreads = 320;
constexpr uint32_t kTmemCols = 512;
constexpr uint64_t kWaitLimitNs = 4000000000ull;

// detail codes written next to FP8ATTN_ERR_TIMEOUT
enum : uint32_t {
    kWaitQFull = 1, kWaitKFull, kWaitVFull, kWaitKEmpty, kWaitVEmpty, kWaitSFull, kWaitPFull, kWaitOFull
};

template <bool kFp8, int kD>
struct Cfg {
    static constexpr int kES = kFp8 ? 1 : 2;                    // element bytes
    static constexpr int kRowBytes = kD * kES;
    static constexpr int kBoxBytes = kRowBytes > 128 ? 128 : kRowBytes;  // swizzle span
    static constexpr int kBoxes = kRowBytes / kBoxBytes;        // TMA boxes per tile
    static constexpr int kBoxCols = kBoxBytes / kES;
    static constexpr int kTileBytes = 128 * kRowBytes;          // Q, K or V tile
    static constexpr int kUmmaK = 32 / kES;                     // elements per MMA K step
    static constexpr int kStages = kTileBytes >= 32768 ? 2 : 4; // K ring and V ring depth
    static constexpr uint32_t kSwizzle = kBoxBytes == 128 ? kSwizzle128 : kSwizzle64;
    static constexpr uint32_t kFmt = kFp8 ? 0u : 1u;            // e4m3 / bf16
    static constexpr uint32_t kIdescQK = idesc(kFmt, kFmt, false, false, kTileM, kTileN);
    static constexpr uint32_t kIdescPV = idesc(kFmt, kFmt, false, true, kTileM, kD);
    static constexpr uint32_t kColS = 0, kColO = 256;           // TMEM columns: S_t at t*128, O_t at 256+t*kD
    static constexpr int kPCols = kTileN * kES / 4;             // TMEM columns of a P tile
    static constexpr size_t kSmemBytes = (size_t)(2 + 2 * kStages) * kTileBytes + 1024;
};

struct Barriers {
    uint64_t q_full;
    uint64_t k_full[4], k_empty[4], v_full[4], v_empty[4];
    uint64_t s_full[2], p_full[2], o_full[2];
};

__device__ __forceinline__ uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Bounded mbarrier wait.  On expiry records (FP8ATTN_ERR_TIMEOUT, detail) once,
// marks the thread dead so that its later waits fall through, and returns false.
struct Waiter {
    uint32_t* status;
    bool dead;
    __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity, uint32_t what) {
        if (dead) return false;
        if (mbar_try_wait(bar, parity)) return true;
        uint64_t t0 = globaltimer_ns();
        for (;;) {
            for (int i = 0; i < 64; ++i)
                if (mbar_try_wait(bar, parity)) return true;
            if (globaltimer_ns() - t0 > kWaitLimitNs) break;
        }
        dead = true;
        if (atomicCAS(status, 0u, (uint32_t)FP8ATTN_ERR_TIMEOUT) == 0u)
            status[1] = (what << 24) | (blockIdx.x & 0xFFFFFFu);
        return false;
    }
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_e4m3x4(float a, float b, float c, float d) {
    uint16_t lo, hi;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(b), "f"(a));
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(d), "f"(c));
    return (uint32_t)lo | ((uint32_t)hi << 16);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

struct KernelArgs {
    const float* scale_q; const float* scale_k; const float* scale_v;
    void* out_train; void* out_test;
    int64_t n_train, n_test;
    int blocks_train, blocks_test;   // 256-row query blocks per head
    float softmax_scale;
    uint32_t* status;
};

template <bool kFp8, int kD>
__global__ void __launch_bounds__(kNumThreads, 1)
icl_attention_kernel(const __grid_constant__ CUtensorMap map_q_train,
                     const __grid_constant__ CUtensorMap map_q_test,
                     const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const KernelArgs args) {
    using C = Cfg<kFp8, kD>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ Barriers bars;
    __shared__ uint32_t tmem_slot;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + 2 * C::kTileBytes;
    const uint32_t sV = sK + C::kStages * C::kTileBytes;

    // ---- which query block is this CTA's ----
    const int blocks_per_head = args.blocks_train + args.blocks_test;
    const int bh = blockIdx.x / blocks_per_head;
    const int blk = blockIdx.x % blocks_per_head;
    const bool is_test = blk >= args.blocks_train;
    const int64_t q_rows = is_test ? args.n_test : args.n_train;
    const int64_t row0 = (int64_t)(is_test ? blk - args.blocks_train : blk) * (2 * kTileM);
    const int ntiles = (q_rows - row0 > kTileM) ? 2 : 1;
    const int64_t n_keys = args.n_train;
    const int nkv = (int)((n_keys + kTileN - 1) / kTileN);
    const CUtensorMap* map_q = is_test ? &map_q_test : &map_q_train;

    // ---- set-up ----
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars.q_full), 1);
        for (int s = 0; s < 4; ++s) {
            mbar_init(smem_u32(&bars.k_full[s]), 1);
            mbar_init(smem_u32(&bars.k_empty[s]), 1);
            mbar_init(smem_u32(&bars.v_full[s]), 1);
            mbar_init(smem_u32(&bars.v_empty[s]), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_u32(&bars.s_full[t]), 1);
            mbar_init(smem_u32(&bars.p_full[t]), kTileM);
            mbar_init(smem_u32(&bars.o_full[t]), 1);
        }
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 9 && lane == 0) {
        prefetch_tensormap(map_q);
        prefetch_tensormap(&map_k);
        prefetch_tensormap(&map_v);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    Waiter w{args.status, false};

    if (warp == 9) {
        // =========================== TMA producer ===========================
        if (lane == 0) {
            mbar_arrive_expect_tx(smem_u32(&bars.q_full), ntiles * C::kTileBytes);
            for (int t = 0; t < ntiles; ++t)
                for (int b = 0; b < C::kBoxes; ++b)
                    tma_load_3d(sQ + t * C::kTileBytes + b * 128 * C::kBoxBytes, map_q,
                                b * C::kBoxCols, (int)(row0 + t * kTileM), bh,
                                smem_u32(&bars.q_full));
            for (int j = 0; j < nkv; ++j) {
                const int s = j % C::kStages;
                const uint32_t ph = (j / C::kStages) & 1;
                w.wait(smem_u32(&bars.k_empty[s]), ph ^ 1, kWaitKEmpty);
                mbar_arrive_expect_tx(smem_u32(&bars.k_full[s]), C::kTileBytes);
                for (int b = 0; b < C::kBoxes; ++b)
                    tma_load_3d(sK + s * C::kTileBytes + b * 128 * C::kBoxBytes, &map_k,
                                b * C::kBoxCols, j * kTileN, bh, smem_u32(&bars.k_full[s]));
                w.wait(smem_u32(&bars.v_empty[s]), ph ^ 1, kWaitVEmpty);
                mbar_arrive_expect_tx(smem_u32(&bars.v_full[s]), C::kTileBytes);
                for (int b = 0; b < C::kBoxes; ++b)
                    tma_load_3d(sV + s * C::kTileBytes + b * 128 * C::kBoxBytes, &map_v,
                                b * C::kBoxCols, j * kTileN, bh, smem_u32(&bars.v_full[s]));
            }
            if (w.dead) {
                // let copies that are still in flight land before the CTA exits
                Waiter d{args.status, false};
                for (int j = (nkv > C::kStages ? nkv - C::kStages : 0); j < nkv; ++j) {
                    d.wait(smem_u32(&bars.k_full[j % C::kStages]), (j / C::kStages) & 1, kWaitKFull);
                    d.wait(smem_u32(&bars.v_full[j % C::kStages]), (j / C::kStages) & 1, kWaitVFull);
                }
            }
        }
    } else if (warp == 8) {
        // ============================ MMA issuer ============================
        if (lane == 0) {
            auto issue_qk = [&](int t, int stage) {
#pragma unroll
                for (int kk = 0; kk < kD / C::kUmmaK; ++kk) {
                    const int off = kk * 32;
                    const uint32_t in_box = off % C::kBoxBytes, box = off / C::kBoxBytes;
                    uint64_t a = smem_desc(sQ + t * C::kTileBytes + box * 128 * C::kBoxBytes + in_box,
                                           0, 8 * C::kBoxBytes, C::kSwizzle);
                    uint64_t b = smem_desc(sK + stage * C::kTileBytes + box * 128 * C::kBoxBytes + in_box,
                                           0, 8 * C::kBoxBytes, C::kSwizzle);
                    mma_ss<kFp8>(tmem + C::kColS + t * kTileN, a, b, C::kIdescQK, kk > 0);
                }
            };
            auto issue_pv = [&](int t, int stage, bool accumulate) {
#pragma unroll
                for (int kk = 0; kk < kTileN / C::kUmmaK; ++kk) {
                    uint64_t b = smem_desc(sV + stage * C::kTileBytes + kk * C::kUmmaK * C::kBoxBytes,
                                           128 * C::kBoxBytes, 8 * C::kBoxBytes, C::kSwizzle);
                    mma_ts<kFp8>(tmem + C::kColO + t * kD, tmem + C::kColS + t * kTileN + kk * 8, b,
                                 C::kIdescPV, (accumulate || kk > 0) ? 1u : 0u);
                }
            };
            w.wait(smem_u32(&bars.q_full), 0, kWaitQFull);
            w.wait(smem_u32(&bars.k_full[0]), 0, kWaitKFull);
            tc_fence_after_sync();
            for (int t = 0; t < ntiles; ++t) {
                issue_qk(t, 0);
                mma_commit(smem_u32(&bars.s_full[t]));
            }
            mma_commit(smem_u32(&bars.k_empty[0]));
            for (int j = 0; j < nkv; ++j) {
                const int sv = j % C::kStages;
                const bool has_next = j + 1 < nkv;
                const int sk = (j + 1) % C::kStages;
                w.wait(smem_u32(&bars.v_full[sv]), (j / C::kStages) & 1, kWaitVFull);
                if (has_next) w.wait(smem_u32(&bars.k_full[sk]), ((j + 1) / C::kStages) & 1, kWaitKFull);
                for (int t = 0; t < ntiles; ++t) {
                    w.wait(smem_u32(&bars.p_full[t]), j & 1, kWaitPFull);
                    tc_fence_after_sync();
                    issue_pv(t, sv, j > 0);
                    if (!has_next) mma_commit(smem_u32(&bars.o_full[t]));
                    if (has_next) {
                        issue_qk(t, sk);
                        mma_commit(smem_u32(&bars.s_full[t]));
                    }
                }
                mma_commit(smem_u32(&bars.v_empty[sv]));
                if (has_next) mma_commit(smem_u32(&bars.k_empty[sk]));
            }
        }
    } else {
        // ========================= softmax + epilogue =========================
        const int t = warp >> 2;                 // query tile of this warpgroup
        if (t < ntiles) {
            const int row_in_tile = threadIdx.x & 127;
            const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
            const uint32_t tS = tmem + lane_addr + C::kColS + t * kTileN;
            const uint32_t tO = tmem + lane_addr + C::kColO + t * kD;
            float c = (args.softmax_scale > 0.f ? args.softmax_scale : rsqrtf((float)kD)) *
                      1.4426950408889634f;
            float sv_scale = 1.0f;
            if (kFp8) {
                c *= args.scale_q[bh] * args.scale_k[bh];
                sv_scale = args.scale_v[bh];
            }
            const float lift = kFp8 ? 8.0f : 0.0f;
            float m = -INFINITY, l = 0.f;
            for (int j = 0; j < nkv; ++j) {
                w.wait(smem_u32(&bars.s_full[t]), j & 1, kWaitSFull);
                tc_fence_after_sync();
                float s[kTileN];
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld_x32(tS + q * 32, reinterpret_cast<uint32_t*>(s) + q * 32);
                tmem_wait_ld();
                const int valid = (int)min((int64_t)kTileN, n_keys - (int64_t)j * kTileN);
                if (valid < kTileN) {
#pragma unroll
                    for (int i = 0; i < kTileN; ++i)
                        if (i >= valid) s[i] = -INFINITY;
                }
                float mx = s[0];
#pragma unroll
                for (int i = 1; i < kTileN; ++i) mx = fmaxf(mx, s[i]);
                const float m_new = fmaxf(m, mx);
                if (j > 0 && __any_sync(0xffffffffu, m_new > m)) {
                    // the running maximum moved for some row of this warp: rescale O and l
                    const float f = ex2((m - m_new) * c);
                    l *= f;
#pragma unroll
                    for (int q = 0; q < kD / 32; ++q) {
                        float o[32];
                        tmem_ld_x32(tO + q * 32, reinterpret_cast<uint32_t*>(o));
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] *= f;
                        tmem_st_x32(tO + q * 32, reinterpret_cast<uint32_t*>(o));
                    }
                }
                m = m_new;
                const float nb = lift - m * c;
                float sum = 0.f;
                uint32_t p[C::kPCols];
                if (kFp8) {
#pragma unroll
                    for (int i = 0; i < kTileN; i += 4) {
                        float p0 = ex2(fmaf(s[i], c, nb)), p1 = ex2(fmaf(s[i + 1], c, nb));
                        float p2 = ex2(fmaf(s[i + 2], c, nb)), p3 = ex2(fmaf(s[i + 3], c, nb));
                        sum += (p0 + p1) + (p2 + p3);
                        p[i / 4] = pack_e4m3x4(p0, p1, p2, p3);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < kTileN; i += 2) {
                        float p0 = ex2(fmaf(s[i], c, nb)), p1 = ex2(fmaf(s[i + 1], c, nb));
                        sum += p0 + p1;
                        p[i / 2] = pack_bf16x2(p0, p1);
                    }
                }
                l += sum;
#pragma unroll
                for (int q = 0; q < C::kPCols / 32; ++q) tmem_st_x32(tS + q * 32, p + q * 32);
                tmem_wait_st();
                tc_fence_before_sync();
                mbar_arrive(smem_u32(&bars.p_full[t]));
            }
            // ---- epilogue: out = s_v * O / l ----
            w.wait(smem_u32(&bars.o_full[t]), 0, kWaitOFull);
            tc_fence_after_sync();
            const int64_t row = row0 + t * kTileM + row_in_tile;
            const float inv = sv_scale / l;
            __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(is_test ? args.out_test : args.out_train) +
                                 ((int64_t)bh * q_rows + row) * kD;
#pragma unroll
            for (int q = 0; q < kD / 32; ++q) {
                float o[32];
                tmem_ld_x32(tO + q * 32, reinterpret_cast<uint32_t*>(o));
                tmem_wait_ld();
                if (row < q_rows && !w.dead) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 v;
                        v.x = pack_bf16x2(o[i] * inv, o[i + 1] * inv);
                        v.y = pack_bf16x2(o[i + 2] * inv, o[i + 3] * inv);
                        v.z = pack_bf16x2(o[i + 4] * inv, o[i + 5] * inv);
                        v.w = pack_bf16x2(o[i + 6] * inv, o[i + 7] * inv);
                        *reinterpret_cast<uint4*>(out + q * 32 + i) = v;
                    }
                }
            }
        }
    }
    // ---- teardown ----
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

template <bool kFp8, int kD>
int launch(const AttnParams& p, cudaStream_t stream) {
    using C = Cfg<kFp8, kD>;
    const int64_t heads = (int64_t)p.B * p.H;
    CUtensorMap mq_train, mq_test, mk, mv;
    if (!make_tensor_map(&mq_train, p.q_train, C::kES, heads, p.n_train, kD, kTileM, C::kBoxCols) ||
        !make_tensor_map(&mk, p.k, C::kES, heads, p.n_train, kD, kTileN, C::kBoxCols) ||
        !make_tensor_map(&mv, p.v, C::kES, heads, p.n_train, kD, kTileN, C::kBoxCols))
        return FP8ATTN_ERR_CUDA;
    if (p.n_test > 0) {
        if (!make_tensor_map(&mq_test, p.q_test, C::kES, heads, p.n_test, kD, kTileM, C::kBoxCols))
            return FP8ATTN_ERR_CUDA;
    } else {
        mq_test = mq_train;
    }
    KernelArgs a;
    a.scale_q = p.scale_q; a.scale_k = p.scale_k; a.scale_v = p.scale_v;
    a.out_train = p.out_train; a.out_test = p.out_test;
    a.n_train = p.n_train; a.n_test = p.n_test;
    a.blocks_train = (int)((p.n_train + 2 * kTileM - 1) / (2 * kTileM));
    a.blocks_test = (int)((p.n_test + 2 * kTileM - 1) / (2 * kTileM));
    a.softmax_scale = p.softmax_scale;
    a.status = p.status;
    const int64_t grid = heads * (a.blocks_train + a.blocks_test);
    if (grid > 0x7fffffffll) return FP8ATTN_ERR_UNSUPPORTED;
    auto kern = icl_attention_kernel<kFp8, kD>;
    static bool attr_set = false;   // per instantiation
    if (!attr_set) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)C::kSmemBytes) != cudaSuccess)
            return FP8ATTN_ERR_CUDA;
        attr_set = true;
    }
    kern<<<(unsigned)grid, kNumThreads, C::kSmemBytes, stream>>>(mq_train, mq_test, mk, mv, a);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? FP8ATTN_OK : FP8ATTN_ERR_CUDA;
}

}  // namespace

int launch_icl_attention(const AttnParams& p, bool fp8, cudaStream_t stream) {
    if (fp8) return p.d == 64 ? launch<true, 64>(p, stream) : launch<true, 128>(p, stream);
    return p.d == 64 ? launch<false, 64>(p, stream) : launch<false, 128>(p, stream);
}

}  // namespace fp8attn
