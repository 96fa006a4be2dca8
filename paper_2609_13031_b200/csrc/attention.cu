// Fused ICL attention for sm_100a: train->train and test->train in one launch.
//
// One CTA owns the query rows of up to T 128-row tiles of one (b,h) (T = 3 at d = 64, 2 at
// d = 128) and walks over all train keys in steps of kKeys keys.  Warp roles:
//   warps 4t .. 4t+3   softmax of query tile t, one row per thread
//   warp  4T           issues the Q K^T tcgen05.mma of all tiles (one elected lane)
//   warp  4T+1         TMA producer for Q, K and V tiles
//   warps 4T+2, 4T+3   issue the P V tcgen05.mma of tiles {0, 2} and {1}
// Q K^T and P V are issued from different warps because a single warp cannot
// issue tcgen05 instructions of this size fast enough to keep the tensor core fed.
// A share of the exponentials (Cfg::kPolyPer16 pairs of every 16) is computed by a
// polynomial on the FMA pipe instead of the MUFU.
// Tensor memory (512 columns) holds S | P_0 .. P_(T-1) | O_0 .. O_(T-1): the tiles take
// turns in ONE S region.  A softmax thread pulls its whole score row into registers
// and gives S up at once, so that the Q K^T of the next tile in the rotation can run
// underneath the softmax, and writes the probability tile P_t (e4m3 with the row
// maximum lifted to 2^8, or bf16 / fp16 in the 16-bit path) to its own tensor-memory
// region (two alternating buffers in the FP8 path), from where it is the A operand of
// O_t += P_t V.
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

constexpr int kTileM = 128;           // query rows per tile
// Query tiles per CTA (kT): two, or at d = 64 three for launches of many rounds (tensor memory
// holds 512 columns and every tile's O takes d of them).  Three tiles put a third softmax warp
// on every scheduler, at the price of a smaller register budget per thread (96-key steps) and
// coarser blocks (384 rows), which small grids pay for in their last round.  Warps: four
// softmax warps per tile, then the Q K^T issuer, the TMA producer and two P V issuers (tiles
// {0, 2} and {1}).
template <int kT> constexpr int kRowsPerBlock = kT * kTileM;
static_assert(kRowsPerBlock<2> == 256, "split_scratch_bytes() in api.cu sizes the scratch for blocks of 256 rows");
template <int kT> constexpr int kNumThreads = (4 * kT + 4) * 32;
// Register budgets after setmaxnreg.  The CTA's register pool is what it was launched with
// (threads x registers at launch, as ptxas reports them for the launch bound);
// setmaxnreg.inc waits in hardware until the pool can serve it, so the budgets must fit in it.
template <int kT> constexpr int kLaunchRegs = kT == 3 ? 128 : 168;
template <int kT> constexpr int kRegsSoftmax = kT == 3 ? 152 : 224;
constexpr int kRegsOther = 56;
template <int kT> constexpr bool kRegsFit =
    4 * kT * 32 * kRegsSoftmax<kT> + 4 * 32 * kRegsOther <= kNumThreads<kT> * kLaunchRegs<kT>;
static_assert(kRegsFit<2> && kRegsFit<3>, "setmaxnreg budgets exceed the CTA's register pool");
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxSplits = 16;        // key ranges a split query block is divided into, at most
constexpr uint64_t kWaitLimitNs = 2000000000ull;

// detail codes written next to FP8ATTN_ERR_TIMEOUT
enum : uint32_t {
    kWaitQFull = 1, kWaitKFull, kWaitVFull, kWaitKEmpty, kWaitVEmpty, kWaitSFull, kWaitPFull, kWaitOFull,
    kWaitSFree, kWaitPFree, kWaitSelfTest
};

// kFp8: e4m3 operands and P (else 16-bit operands and P).  kHalf: the 16-bit type of the
// call is IEEE fp16 instead of bf16: the outputs of both kernels, and the operands and P
// of the 16-bit kernel.  (A run-time switch for the FP8 kernel's output type cost 4 % at
// d = 64 through register allocation, hence a template parameter.)
template <bool kFp8, int kD, bool kHalf, int kT>
struct Cfg {
    static_assert(kT == 2 || (kT == 3 && kD == 64), "tiles per CTA");
    static constexpr int kES = kFp8 ? 1 : 2;                    // element bytes
    static constexpr int kRowBytes = kD * kES;
    static constexpr int kBoxBytes = kRowBytes > 128 ? 128 : kRowBytes;  // swizzle span
    static constexpr int kBoxes = kRowBytes / kBoxBytes;        // TMA boxes per tile
    static constexpr int kBoxCols = kBoxBytes / kES;
    static constexpr int kTiles = kT;
    // keys per step: a softmax thread holds the scores of one row of a step in registers,
    // 128 of them in a budget of 224 registers, 96 in a budget of 152
    static constexpr int kKeys = kTiles == 3 ? 96 : 128;
    static constexpr int kQTileBytes = kTileM * kRowBytes;
    static constexpr int kKVTileBytes = kKeys * kRowBytes;
    static constexpr int kUmmaK = 32 / kES;                     // elements per MMA K step
    static constexpr int kStages = kKVTileBytes >= 32768 ? 2 : 4;  // K ring and V ring depth
    static constexpr uint32_t kSwizzle = kBoxBytes == 128 ? kSwizzle128 : kSwizzle64;
    static constexpr uint32_t kFmt = (kFp8 || kHalf) ? 0u : 1u; // e4m3 (kind::f8f6f4); f16 / bf16 (kind::f16)
    static constexpr uint32_t kIdescQK = idesc(kFmt, kFmt, false, false, kTileM, kKeys);
    static constexpr uint32_t kIdescPV = idesc(kFmt, kFmt, false, true, kTileM, kD);
    static constexpr int kPCols = kKeys * kES / 4;              // TMEM columns of a P tile
    // Tensor memory (512 columns): one S region that the query tiles of the CTA take turns in,
    // the P tiles behind it, and O_t at 256 + t*kD.  A tile's scores sit in S only from its
    // Q K^T until its softmax warps have loaded them into registers (a small part of a step),
    // and the tiles run a fraction of a step apart anyway; the Q K^T of a tile waits for the
    // load of the tile before it in the rotation.  Two tiles: S | P0 | P1 | O0 | O1 (128,
    // 2 x 64, 2 x kD columns); three tiles (d = 64): S | P0 | P1 | P2 | - | O0 | O1 | O2 (96,
    // 3 x 48, 3 x 64).
    // (Layouts before this one, d = 128: FP8 with 96-key steps and an S region per tile,
    // 3.6 % more time; P written over S, where Q K^T has to wait for P V: the 16-bit kernel
    // took 10 % more time and 20 % more cycles that way.)
    static constexpr uint32_t kColS = 0, kColO = 256;
    static constexpr uint32_t kColP0 = kKeys, kPStride = kKeys / 2;   // P_t at kColP0 + t*kPStride
    // FP8: P alternates between two buffers per tile (the second kPCols columns after the
    // first), so that writing P of one step never waits for the P V of the step before.
    static constexpr int kPBufs = kFp8 ? 2 : 1;
    // pairs of exponentials, out of every 16 pairs, that go to the FMA pipe (measured best)
    static constexpr int kPolyPer16 = kFp8 ? (kT == 3 ? 2 : 4) : 2;
    static_assert(kPBufs * kPCols <= (int)kPStride, "TMEM layout: P tiles overlap");
    static_assert(kColP0 + kTiles * kPStride <= kColO && kColO + kTiles * kD <= 512, "TMEM layout");
    static constexpr size_t kSmemBytes = (size_t)kTiles * kQTileBytes + (size_t)2 * kStages * kKVTileBytes + 1024;
};

struct Barriers {
    uint64_t q_full;
    uint64_t k_full[4], k_empty[4], v_full[4], v_empty[4];
    uint64_t s_full[3], p_free[3], o_full[3], s_free[3];
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
    uint64_t limit_ns = kWaitLimitNs;
    // kBackoffNs > 0: sleep that long between polls.  For waits with plenty of slack
    // (the TMA producer runs several stages ahead) this keeps the polling out of
    // the instruction queue that the softmax warps' MUFU and barrier traffic uses.
    template <uint32_t kBackoffNs = 0>
    __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity, uint32_t what) {
        if (dead) return false;
        if (mbar_test_wait(bar, parity)) return true;
        uint64_t t0 = globaltimer_ns();
        for (;;) {
            for (int i = 0; i < 64; ++i) {
                if (mbar_try_wait(bar, parity)) return true;
                if (kBackoffNs > 0) __nanosleep(kBackoffNs);
            }
            // another CTA already gave up: do not wait out the limit here as well
            if (*reinterpret_cast<volatile uint32_t*>(status) != 0u) { dead = true; return false; }
            if (globaltimer_ns() - t0 > limit_ns) break;
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
    uint32_t r;
    asm("{\n"
        ".reg .b16 lo, hi;\n"
        "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n"
        "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n"
        "mov.b32 %0, {lo, hi};\n"
        "}\n"
        : "=r"(r)
        : "f"(a), "f"(b), "f"(c), "f"(d));
    return r;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// two fp32 -> two 16-bit values of the call's 16-bit type (bf16, or IEEE fp16)
template <bool kHalf>
__device__ __forceinline__ uint32_t pack_16x2(float lo, float hi) {
    return kHalf ? pack_f16x2(lo, hi) : pack_bf16x2(lo, hi);
}

// ---- packed fp32x2 arithmetic (two lanes per instruction on sm_100) ----
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// 2^x for a pair of lanes on the FMA pipe instead of the MUFU: x = n + f with
// n = round(x) taken from the mantissa after adding 1.5*2^23, f in [-0.5, 0.5],
// 2^f by a minimax polynomial (degree 2: 1.7e-3 relative, enough for an e4m3
// result; degree 3: 7.5e-5 for bf16), and n added into the exponent field.
// x must be >= -126 (the caller clamps) and < 128.
template <bool kDegree3>
__device__ __forceinline__ void exp2_poly2(uint64_t x, float& r0, float& r1) {
    const uint64_t magic = pack2(12582912.f, 12582912.f);
    const uint64_t neg_magic = pack2(-12582912.f, -12582912.f);
    const uint64_t neg_one = pack2(-1.f, -1.f);
    const uint64_t t = add2(x, magic);
    const uint64_t n = add2(t, neg_magic);
    const uint64_t f = fma2(n, neg_one, x);
    uint64_t p;
    if (kDegree3) {
        p = fma2(f, pack2(0.05517132f, 0.05517132f), pack2(0.24261054f, 0.24261054f));
        p = fma2(p, f, pack2(0.69326097f, 0.69326097f));
        p = fma2(p, f, pack2(0.99992812f, 0.99992812f));
    } else {
        p = fma2(f, pack2(0.23842570f, 0.23842570f), pack2(0.70344281f, 0.70344281f));
        p = fma2(p, f, pack2(1.00044298f, 1.00044298f));
    }
    float p0, p1, t0, t1;
    unpack2(p, p0, p1);
    unpack2(t, t0, t1);
    r0 = __uint_as_float(__float_as_uint(p0) + (__float_as_uint(t0) << 23));
    r1 = __uint_as_float(__float_as_uint(p1) + (__float_as_uint(t1) << 23));
}

// Blocks until this thread's tcgen05.ld results have landed; naming the 32
// destination registers keeps every use of them after the wait.
__device__ __forceinline__ void tmem_wait_ld_x16(uint32_t* r) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]),
                   "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]),
                   "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
                 :
                 : "memory");
}
__device__ __forceinline__ void named_barrier_arrive(uint32_t id, uint32_t threads) {
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void named_barrier_sync(uint32_t id, uint32_t threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld_x32(uint32_t* r) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]),
                   "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]),
                   "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]),
                   "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
                   "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]),
                   "+r"(r[31])
                 :
                 : "memory");
}

template <int kRegs>
__device__ __forceinline__ void setmaxnreg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegs));
}
template <int kRegs>
__device__ __forceinline__ void setmaxnreg_dec() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegs));
}

// tcgen05.ld / wait / st of kCols consecutive columns (multiple of 16) in as few
// instructions as possible
template <int kCols>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t* r) {
#pragma unroll
    for (int q = 0; q + 32 <= kCols; q += 32) tmem_ld_x32(taddr + q, r + q);
    if (kCols % 32) tmem_ld_x16(taddr + (kCols / 32) * 32, r + (kCols / 32) * 32);
}
template <int kCols>
__device__ __forceinline__ void tmem_wait_ld_cols(uint32_t* r) {
#pragma unroll
    for (int q = 0; q + 32 <= kCols; q += 32) tmem_wait_ld_x32(r + q);
    if (kCols % 32) tmem_wait_ld_x16(r + (kCols / 32) * 32);
}
template <int kCols>
__device__ __forceinline__ void tmem_st_cols(uint32_t taddr, const uint32_t* r) {
    static_assert(kCols == 4 || kCols == 8 || kCols == 16 || kCols == 32, "store width");
    if (kCols == 4) tmem_st_x4(taddr, r);
    else if (kCols == 8) tmem_st_x8(taddr, r);
    else if (kCols == 16) tmem_st_x16(taddr, r);
    else tmem_st_x32(taddr, r);
}

// Named barrier (hardware-blocking, no polling), one per query tile t:
//   kPFullBarrier0 + t  "P_t is in tensor memory"    softmax warps -> P V issuer of tile t
constexpr uint32_t kPFullBarrier0 = 1;
constexpr uint32_t kSignalThreads = 128 + 32;   // one tile's softmax threads + the issuer warp

// floats per row of a partial result: kD values of O, c*m, l, and padding to 16 bytes
template <int kD> constexpr int kPartialStride = kD + 4;

struct KernelArgs {
    const float* scale_q; const float* scale_k; const float* scale_v;
    void* out_train; void* out_test;
    int64_t n_train, n_test;
    int blocks_train, blocks_test;   // query blocks (one CTA's rows) per head
    int heads;                       // H, to find head 0 of a table
    int test_kv_head0;               // test rows read K, V and their scales from head 0 of their table
    // Tail split: the query blocks from full_blocks on (the part of the grid that would
    // fill less than one CTA per SM) are each run by `splits` CTAs over disjoint key ranges;
    // those CTAs write unnormalised partial results to `partial`, combined afterwards.
    int full_blocks, splits;
    float* partial;                  // [unit][split][rows of a block][kD + 4] fp32: O, c*m, l, pad
    float softmax_scale;
    uint32_t* status;
};

// kSplit: this launch runs the split query blocks (see KernelArgs); kept out of the main
// instantiation, whose softmax warps have no register to spare for the extra indices.
template <bool kFp8, int kD, bool kHalf, int kT, bool kSplit>
__global__ void __launch_bounds__(kNumThreads<kT>, 1)
icl_attention_kernel(const __grid_constant__ CUtensorMap map_q_train,
                     const __grid_constant__ CUtensorMap map_q_test,
                     const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const KernelArgs args) {
    using C = Cfg<kFp8, kD, kHalf, kT>;
    constexpr int kKeys = C::kKeys;
    constexpr int kQkWarp = 4 * C::kTiles, kTmaWarp = kQkWarp + 1, kPvWarp0 = kQkWarp + 2;
    constexpr int kRows = kRowsPerBlock<kT>;       // query rows per CTA
    extern __shared__ uint8_t smem_raw[];
    __shared__ Barriers bars;
    __shared__ uint32_t tmem_slot;
    __shared__ uint32_t sticky_status;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + C::kTiles * C::kQTileBytes;
    const uint32_t sV = sK + C::kStages * C::kKVTileBytes;

    // ---- which query block is this CTA's ----
    const int blocks_per_head = args.blocks_train + args.blocks_test;
    const int vblk = kSplit ? args.full_blocks + (int)blockIdx.x / args.splits : (int)blockIdx.x;
    const int split = kSplit ? (int)blockIdx.x % args.splits : 0;
    const int nsplit = kSplit ? args.splits : 1;
    const int bh = vblk / blocks_per_head;
    const int blk = vblk % blocks_per_head;
    const bool is_test = blk >= args.blocks_train;
    const int64_t q_rows = is_test ? args.n_test : args.n_train;
    const int64_t row0 = (int64_t)(is_test ? blk - args.blocks_train : blk) * kRows;
    const int ntiles = (int)min((int64_t)C::kTiles, (q_rows - row0 + kTileM - 1) / kTileM);
    const int64_t n_keys = args.n_train;
    // this CTA's key steps: [j0, j0 + nkv) of the nkv_all steps over the train keys
    const int nkv_all = (int)((n_keys + kKeys - 1) / kKeys);
    const int j0 = (int)((int64_t)split * nkv_all / nsplit);
    const int nkv = (int)((int64_t)(split + 1) * nkv_all / nsplit) - j0;
    const CUtensorMap* map_q = is_test ? &map_q_test : &map_q_train;
    // grouped-query variant: every test query head attends to the first K/V head of its table
    const int bh_kv = (is_test && args.test_kv_head0) ? (bh / args.heads) * args.heads : bh;

    // A device error recorded earlier (and not yet read back by the host) is sticky:
    // nothing runs until fp8attn_last_device_status() has cleared it.
    // One thread reads it for the whole CTA, so that either every warp leaves or none does
    // (a warp that left alone would leave the others blocked on the named barriers).
    if (threadIdx.x == 0) sticky_status = *reinterpret_cast<volatile uint32_t*>(args.status);
    __syncthreads();
    if (sticky_status != 0u) return;

    // ---- set-up ----
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars.q_full), 1);
        for (int s = 0; s < 4; ++s) {
            mbar_init(smem_u32(&bars.k_full[s]), 1);
            mbar_init(smem_u32(&bars.k_empty[s]), 1);
            mbar_init(smem_u32(&bars.v_full[s]), 1);
            mbar_init(smem_u32(&bars.v_empty[s]), ntiles);   // one commit per P V issuer
        }
        for (int t = 0; t < C::kTiles; ++t) {
            mbar_init(smem_u32(&bars.s_full[t]), 1);
            mbar_init(smem_u32(&bars.p_free[t]), 1);
            mbar_init(smem_u32(&bars.o_full[t]), 1);
            mbar_init(smem_u32(&bars.s_free[t]), 4);   // one arrival per softmax warp of the tile
        }
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    if (warp == kTmaWarp && lane == 0) {
        prefetch_tensormap(map_q);
        prefetch_tensormap(&map_k);
        prefetch_tensormap(&map_v);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = __shfl_sync(0xffffffffu, tmem_slot, 0);
    Waiter w{args.status, false};

    if (warp == kTmaWarp) {
        setmaxnreg_dec<kRegsOther>();
        // =========================== TMA producer ===========================
        // The whole warp walks the loop (waits included); one elected lane issues.
        if (elect_one()) {
            mbar_arrive_expect_tx(smem_u32(&bars.q_full), ntiles * C::kQTileBytes);
            for (int t = 0; t < ntiles; ++t)
                for (int b = 0; b < C::kBoxes; ++b)
                    tma_load_3d(sQ + t * C::kQTileBytes + b * kTileM * C::kBoxBytes, map_q,
                                b * C::kBoxCols, (int)(row0 + t * kTileM), bh,
                                smem_u32(&bars.q_full));
        }
        for (int j = 0; j < nkv; ++j) {
            const int s = j % C::kStages;
            const uint32_t ph = (j / C::kStages) & 1;
            w.wait<400>(smem_u32(&bars.k_empty[s]), ph ^ 1, kWaitKEmpty);
            if (elect_one()) {
                mbar_arrive_expect_tx(smem_u32(&bars.k_full[s]), C::kKVTileBytes);
                for (int b = 0; b < C::kBoxes; ++b)
                    tma_load_3d(sK + s * C::kKVTileBytes + b * kKeys * C::kBoxBytes, &map_k,
                                b * C::kBoxCols, (j0 + j) * kKeys, bh_kv, smem_u32(&bars.k_full[s]));
            }
            w.wait<400>(smem_u32(&bars.v_empty[s]), ph ^ 1, kWaitVEmpty);
            if (elect_one()) {
                mbar_arrive_expect_tx(smem_u32(&bars.v_full[s]), C::kKVTileBytes);
                for (int b = 0; b < C::kBoxes; ++b)
                    tma_load_3d(sV + s * C::kKVTileBytes + b * kKeys * C::kBoxBytes, &map_v,
                                b * C::kBoxCols, (j0 + j) * kKeys, bh_kv, smem_u32(&bars.v_full[s]));
            }
            __syncwarp();
        }
        if (__any_sync(0xffffffffu, w.dead)) {
            // let copies that are still in flight land before the CTA exits
            Waiter d{args.status, false};
            for (int j = (nkv > C::kStages ? nkv - C::kStages : 0); j < nkv; ++j) {
                d.wait(smem_u32(&bars.k_full[j % C::kStages]), (j / C::kStages) & 1, kWaitKFull);
                d.wait(smem_u32(&bars.v_full[j % C::kStages]), (j / C::kStages) & 1, kWaitVFull);
            }
        }
    } else if (warp == kQkWarp) {
        setmaxnreg_dec<kRegsOther>();
        // ====================== Q K^T issuer (all query tiles) ======================
        // The whole warp walks the loop (waits included); one elected lane issues the
        // MMAs and commits.  Q K^T and P V are issued from different warps because one
        // warp cannot issue tcgen05 instructions fast enough to feed the tensor core
        // with instructions of this size; every dependency between the two streams
        // already goes through an mbarrier.
        const uint64_t dQ = smem_desc(sQ, 0, 8 * C::kBoxBytes, C::kSwizzle);
        const uint64_t dK = smem_desc(sK, 0, 8 * C::kBoxBytes, C::kSwizzle);
        auto issue_qk = [&](int t, int stage) {
            const uint64_t a0 = dQ + (uint64_t)((t * C::kQTileBytes) >> 4);
            const uint64_t b0 = dK + (uint64_t)((stage * C::kKVTileBytes) >> 4);
            const uint32_t d = tmem + C::kColS;
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kD / C::kUmmaK; ++kk) {
                    constexpr int kB = C::kBoxBytes;
                    const int off = kk * 32;
                    const uint64_t a = a0 + (uint64_t)(((off / kB) * kTileM * kB + off % kB) >> 4);
                    const uint64_t b = b0 + (uint64_t)(((off / kB) * kKeys * kB + off % kB) >> 4);
                    mma_ss<kFp8>(d, a, b, C::kIdescQK, kk > 0);
                }
                mma_commit(smem_u32(&bars.s_full[t]));
            }
            __syncwarp();
        };
        w.wait(smem_u32(&bars.q_full), 0, kWaitQFull);
        w.wait(smem_u32(&bars.k_full[0]), 0, kWaitKFull);
        tc_fence_after_sync();
        for (int t = 0; t < ntiles; ++t) {
            if (t > 0) {
                // the S region is the tile's before this one until its rows sit in registers
                w.wait(smem_u32(&bars.s_free[t - 1]), 0, kWaitSFree);
                tc_fence_after_sync();
            }
            issue_qk(t, 0);
        }
        if (elect_one()) mma_commit(smem_u32(&bars.k_empty[0]));
        __syncwarp();
        for (int j = 0; j + 1 < nkv; ++j) {
            const int sk = (j + 1) % C::kStages;
            w.wait(smem_u32(&bars.k_full[sk]), ((j + 1) / C::kStages) & 1, kWaitKFull);
            for (int t = 0; t < ntiles; ++t) {
                // The S region is free once its last occupant's rows sit in registers: that
                // is the tile before this one in the rotation (step j+1 of tile t-1, or step j
                // of the block's last tile for tile 0).  s_free[t] counts the loads of tile t
                // in step order, and a tile can be at most one load ahead of the issuer, so
                // the step's parity names the phase.
                if (t == 0) w.wait(smem_u32(&bars.s_free[ntiles - 1]), j & 1, kWaitSFree);
                else w.wait(smem_u32(&bars.s_free[t - 1]), (j + 1) & 1, kWaitSFree);
                tc_fence_after_sync();
                issue_qk(t, sk);
            }
            if (elect_one()) mma_commit(smem_u32(&bars.k_empty[sk]));
            __syncwarp();
        }
    } else if (warp >= kPvWarp0) {
        setmaxnreg_dec<kRegsOther>();
        // ============ P V issuers: the first takes tiles 0 and 2, the second tile 1 ============
        // (the tiles' P become ready in the order of the rotation, so the tiles of one issuer
        // never wait for each other)
        const int pw = warp - kPvWarp0;
        const uint64_t dV = smem_desc(sV, kKeys * C::kBoxBytes, 8 * C::kBoxBytes, C::kSwizzle);
        for (int j = 0; j < nkv; ++j) {
            const int sv = j % C::kStages;
            for (int t = pw; t < ntiles; t += 2) {
                const uint32_t d = tmem + C::kColO + t * kD;
                const uint32_t a = tmem + C::kColP0 + (uint32_t)t * C::kPStride;
                w.wait(smem_u32(&bars.v_full[sv]), (j / C::kStages) & 1, kWaitVFull);
                named_barrier_sync(kPFullBarrier0 + t, kSignalThreads);
                tc_fence_after_sync();
                if (elect_one()) {
                    const uint64_t b0 = dV + (uint64_t)((sv * C::kKVTileBytes) >> 4);
#pragma unroll
                    for (int kk = 0; kk < kKeys / C::kUmmaK; ++kk) {
                        const uint64_t b = b0 + (uint64_t)((kk * C::kUmmaK * C::kBoxBytes) >> 4);
                        const uint32_t pa = (uint32_t)((C::kPBufs == 2 ? (j & 1) * C::kPCols : 0) + kk * 8);
                        mma_ts<kFp8>(d, a + pa, b, C::kIdescPV,
                                     (j > 0 || kk > 0) ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&bars.p_free[t]));
                    mma_commit(smem_u32(&bars.v_empty[sv]));
                    if (j + 1 == nkv) mma_commit(smem_u32(&bars.o_full[t]));
                }
                __syncwarp();
            }
        }
    } else {
        // ========================= softmax + epilogue =========================
        setmaxnreg_inc<kRegsSoftmax<kT>>();
        const int t = warp >> 2;                       // query tile
        if (t < ntiles) {
            const int row_in_tile = (warp & 3) * 32 + lane;
            const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
            const uint32_t tS = tmem + lane_addr + C::kColS;
            const uint32_t tP = tmem + lane_addr + C::kColP0 + (uint32_t)t * C::kPStride;
            const uint32_t tO = tmem + lane_addr + C::kColO + t * kD;
            float c = (args.softmax_scale > 0.f ? args.softmax_scale : rsqrtf((float)kD)) *
                      1.4426950408889634f;
            float sv_scale = 1.0f;
            if (kFp8) {
                c *= args.scale_q[bh] * args.scale_k[bh_kv];
                sv_scale = args.scale_v[bh_kv];
            }
            const float lift = kFp8 ? 8.0f : 0.0f;
            const uint64_t cc = pack2(c, c);
            float m = -INFINITY;
            uint64_t l2a = pack2(0.f, 0.f), l2b = pack2(0.f, 0.f);   // partial row sums
            constexpr uint32_t kNegInf = 0xff800000u;
            for (int j = 0; j < nkv; ++j) {
                w.wait(smem_u32(&bars.s_full[t]), j & 1, kWaitSFull);
                tc_fence_after_sync();
                // ---- the whole score row of this thread into registers ----
                uint32_t s[kKeys];
                tmem_ld_cols<kKeys>(tS, s);
                tmem_wait_ld_cols<kKeys>(s);
                // the S region goes to the next tile's Q K^T of this step or, from the block's
                // last tile, to tile 0's of the next step
                if (j + 1 < nkv || t < ntiles - 1) {
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars.s_free[t]));
                }
                const int valid = (int)min((int64_t)kKeys, n_keys - (int64_t)(j0 + j) * kKeys);
                if (valid < kKeys) {
#pragma unroll
                    for (int i = 0; i < kKeys; ++i)
                        if (i >= valid) s[i] = kNegInf;
                }
                // ---- row maximum of the raw scores ----
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int i = 0; i < kKeys; i += 8) {
                    mx0 = max3(mx0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
                    mx1 = max3(mx1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
                    mx2 = max3(mx2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
                    mx3 = max3(mx3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
                }
                const float m_tile = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                // The reference maximum is the exact running maximum: the row maximum of
                // the keys seen so far maps to 2^lift.
                const float m_new = fmaxf(m, m_tile);
                // P V of the previous step must be done before O is rescaled or P rewritten
                bool pv_done = j == 0;
                if (C::kPBufs == 1 && !pv_done && !w.dead) {
                    // ask now, use the answer a chunk of exponentials later: the usual case
                    // (P V long done) then costs no stall in the middle of the chunk
                    pv_done = mbar_test_wait(smem_u32(&bars.p_free[t]), (j - 1) & 1);
                    tc_fence_after_sync();
                }
                // Where the maximum moved for some row of this warp, l is rescaled now and O at
                // the end of the step: by then the score registers are free, so the O columns
                // go through registers in pipelined 64-column halves instead of dependent
                // 16-column round trips, and the P V that has to precede it is long done.
                const bool rescale = j > 0 && __any_sync(0xffffffffu, m_new > m);
                float f = 1.0f;
                if (rescale) {
                    f = ex2((m - m_new) * c);
                    const uint64_t ff = pack2(f, f);
                    l2a = mul2(l2a, ff);
                    l2b = mul2(l2b, ff);
                }
                m = m_new;
                const float nb = lift - m * c;
                const uint64_t nbnb = pack2(nb, nb);
                // ---- p = 2^(c*s - c*m + lift), row sums, P tile into tensor memory ----
#pragma unroll
                for (int k0 = 0; k0 < kKeys; k0 += 32) {
                    constexpr int kPPer32 = kFp8 ? 8 : 16;
                    uint32_t p[kPPer32];
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        const uint32_t* cur = s + k0 + i;
                        const uint64_t xa = fma2(pack2(__uint_as_float(cur[0]), __uint_as_float(cur[1])), cc, nbnb);
                        const uint64_t xb = fma2(pack2(__uint_as_float(cur[2]), __uint_as_float(cur[3])), cc, nbnb);
                        float p0, p1, p2, p3, x0, x1, x2, x3;
                        unpack2(xa, x0, x1);
                        unpack2(xb, x2, x3);
                        // pair q of the chunk goes to the FMA pipe if the running count
                        // q * kPolyPer16 / 16 steps up there: an even spread over the chunk
                        constexpr int kPP = C::kPolyPer16;
                        const int qa = i / 2, qb = i / 2 + 1;
                        if (((qa + 1) * kPP) / 16 != (qa * kPP) / 16) {
                            exp2_poly2<!kFp8>(pack2(fmaxf(x0, -120.f), fmaxf(x1, -120.f)), p0, p1);
                        } else {
                            p0 = ex2(x0);
                            p1 = ex2(x1);
                        }
                        if (((qb + 1) * kPP) / 16 != (qb * kPP) / 16) {
                            exp2_poly2<!kFp8>(pack2(fmaxf(x2, -120.f), fmaxf(x3, -120.f)), p2, p3);
                        } else {
                            p2 = ex2(x2);
                            p3 = ex2(x3);
                        }
                        l2a = add2(l2a, pack2(p0, p1));
                        l2b = add2(l2b, pack2(p2, p3));
                        if (kFp8) {
                            p[i / 4] = pack_e4m3x4(p0, p1, p2, p3);
                        } else {
                            p[i / 2] = pack_16x2<kHalf>(p0, p1);
                            p[i / 2 + 1] = pack_16x2<kHalf>(p2, p3);
                        }
                    }
                    if (C::kPBufs == 1 && k0 == 0 && !pv_done) {
                        w.wait(smem_u32(&bars.p_free[t]), (j - 1) & 1, kWaitPFree);
                        tc_fence_after_sync();
                        pv_done = true;
                    }
                    tmem_st_cols<kPPer32>(tP + (uint32_t)((C::kPBufs == 2 ? (j & 1) * C::kPCols : 0) + (k0 / 32) * kPPer32), p);
                }
                if (C::kPBufs == 2 && !pv_done) {
                    // P V of the previous step has had this whole step to finish; once it
                    // has, the buffer that the NEXT step writes (the one it read) is free.
                    // That write comes after the next step's fence behind its wait for S.
                    w.wait(smem_u32(&bars.p_free[t]), (j - 1) & 1, kWaitPFree);
                    pv_done = true;
                    if (rescale) tc_fence_after_sync();
                }
                if (rescale) {
                    if (!pv_done) {
                        w.wait(smem_u32(&bars.p_free[t]), (j - 1) & 1, kWaitPFree);
                        tc_fence_after_sync();
                    }
#pragma unroll
                    for (int q = 0; q < kD / 64; ++q) {
                        uint32_t o[64];
                        tmem_ld_cols<64>(tO + q * 64, o);
                        tmem_wait_ld_cols<64>(o);
#pragma unroll
                        for (int i = 0; i < 64; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                        tmem_st_x32(tO + q * 64, o);
                        tmem_st_x32(tO + q * 64 + 32, o + 32);
                    }
                }
                tmem_wait_st();
                tc_fence_before_sync();
                named_barrier_arrive(kPFullBarrier0 + t, kSignalThreads);
            }
            // ---- row sum ----
            float l;
            {
                float a0, a1, b0, b1;
                unpack2(l2a, a0, a1);
                unpack2(l2b, b0, b1);
                l = (a0 + a1) + (b0 + b1);
            }
            // ---- epilogue: out = s_v * O / l ----
            w.wait(smem_u32(&bars.o_full[t]), 0, kWaitOFull);
            tc_fence_after_sync();
            const int64_t row = row0 + t * kTileM + row_in_tile;
            if (kSplit) {
                // partial result of this key range: unnormalised O, the reference maximum in
                // exp2 units and the row sum; the combine kernel weighs and normalises
                float* dst = args.partial +
                             ((size_t)((vblk - args.full_blocks) * nsplit + split) * kRowsPerBlock<kT> +
                              (size_t)(t * kTileM + row_in_tile)) * kPartialStride<kD>;
#pragma unroll
                for (int q = 0; q < kD / 32; ++q) {
                    uint32_t o[32];
                    tmem_ld_x32(tO + q * 32, o);
                    tmem_wait_ld_x32(o);
                    if (!w.dead) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            *reinterpret_cast<uint4*>(dst + q * 32 + i) = make_uint4(o[i], o[i + 1], o[i + 2], o[i + 3]);
                    }
                }
                if (!w.dead) *reinterpret_cast<float2*>(dst + kD) = make_float2(m * c, l);
            } else {
            const float inv = sv_scale / l;
            constexpr bool out_half = kHalf;   // 16-bit type of the outputs
            __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(is_test ? args.out_test : args.out_train) +
                                 ((int64_t)bh * q_rows + row) * kD;
#pragma unroll
            for (int q = 0; q < kD / 32; ++q) {
                uint32_t o[32];
                tmem_ld_x32(tO + q * 32, o);
                tmem_wait_ld_x32(o);
                if (row < q_rows && !w.dead) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 v;
                        auto val = [&](int k) { return __uint_as_float(o[i + k]) * inv; };
                        if (out_half) {
                            v.x = pack_f16x2(val(0), val(1));
                            v.y = pack_f16x2(val(2), val(3));
                            v.z = pack_f16x2(val(4), val(5));
                            v.w = pack_f16x2(val(6), val(7));
                        } else {
                            v.x = pack_bf16x2(val(0), val(1));
                            v.y = pack_bf16x2(val(2), val(3));
                            v.z = pack_bf16x2(val(4), val(5));
                            v.w = pack_bf16x2(val(6), val(7));
                        }
                        *reinterpret_cast<uint4*>(out + q * 32 + i) = v;
                    }
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

// Combines the partial results of the split query blocks: with M = max_s c*m_s,
// out = s_v * sum_s 2^(c*m_s - M) O_s / sum_s 2^(c*m_s - M) l_s.  One thread per row and
// eight output columns.
template <int kD, int kT>
__global__ void __launch_bounds__(256)
combine_split_kernel(const KernelArgs args, int units, int out_half, int fp8) {
    const int per_row = kD / 8;
    const int64_t tid = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int64_t unit = tid / (kRowsPerBlock<kT> * per_row);
    if (unit >= units) return;
    const int r = (int)(tid / per_row) % kRowsPerBlock<kT>;
    const int g = (int)(tid % per_row);
    const int blocks_per_head = args.blocks_train + args.blocks_test;
    const int vblk = args.full_blocks + (int)unit;
    const int bh = vblk / blocks_per_head, blk = vblk % blocks_per_head;
    const bool is_test = blk >= args.blocks_train;
    const int64_t q_rows = is_test ? args.n_test : args.n_train;
    const int64_t row = (int64_t)(is_test ? blk - args.blocks_train : blk) * kRowsPerBlock<kT> + r;
    if (row >= q_rows) return;
    const int bh_kv = (is_test && args.test_kv_head0) ? (bh / args.heads) * args.heads : bh;
    const float* base = args.partial + ((size_t)unit * args.splits * kRowsPerBlock<kT> + r) * kPartialStride<kD>;
    const size_t split_stride = (size_t)kRowsPerBlock<kT> * kPartialStride<kD>;
    float mmax = -INFINITY;
    for (int s = 0; s < args.splits; ++s) mmax = fmaxf(mmax, base[s * split_stride + kD]);
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    float lsum = 0.f;
    for (int s = 0; s < args.splits; ++s) {
        const float* ps = base + s * split_stride;
        const float wgt = exp2f(ps[kD] - mmax);
        lsum = fmaf(wgt, ps[kD + 1], lsum);
        const float4 a = *reinterpret_cast<const float4*>(ps + g * 8);
        const float4 b = *reinterpret_cast<const float4*>(ps + g * 8 + 4);
        acc[0] = fmaf(wgt, a.x, acc[0]); acc[1] = fmaf(wgt, a.y, acc[1]);
        acc[2] = fmaf(wgt, a.z, acc[2]); acc[3] = fmaf(wgt, a.w, acc[3]);
        acc[4] = fmaf(wgt, b.x, acc[4]); acc[5] = fmaf(wgt, b.y, acc[5]);
        acc[6] = fmaf(wgt, b.z, acc[6]); acc[7] = fmaf(wgt, b.w, acc[7]);
    }
    const float inv = (fp8 ? args.scale_v[bh_kv] : 1.0f) / lsum;
    uint4 v;
    if (out_half) {
        v.x = pack_f16x2(acc[0] * inv, acc[1] * inv); v.y = pack_f16x2(acc[2] * inv, acc[3] * inv);
        v.z = pack_f16x2(acc[4] * inv, acc[5] * inv); v.w = pack_f16x2(acc[6] * inv, acc[7] * inv);
    } else {
        v.x = pack_bf16x2(acc[0] * inv, acc[1] * inv); v.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
        v.z = pack_bf16x2(acc[4] * inv, acc[5] * inv); v.w = pack_bf16x2(acc[6] * inv, acc[7] * inv);
    }
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(is_test ? args.out_test : args.out_train) +
                         ((int64_t)bh * q_rows + row) * kD;
    *reinterpret_cast<uint4*>(out + g * 8) = v;
}

template <bool kFp8, int kD, bool kHalf, int kT>
int launch(const AttnParams& p, cudaStream_t stream) {
    using C = Cfg<kFp8, kD, kHalf, kT>;
    const int64_t heads = (int64_t)p.B * p.H;
    const bool test_only = (p.flags & FP8ATTN_TEST_ROWS_ONLY) != 0;
    CUtensorMap mq_train, mq_test, mk, mv;
    if (!make_tensor_map(&mk, p.k, C::kES, heads, p.n_train, kD, C::kKeys, C::kBoxCols) ||
        !make_tensor_map(&mv, p.v, C::kES, heads, p.n_train, kD, C::kKeys, C::kBoxCols))
        return FP8ATTN_ERR_CUDA;
    if (!test_only &&
        !make_tensor_map(&mq_train, p.q_train, C::kES, heads, p.n_train, kD, kTileM, C::kBoxCols))
        return FP8ATTN_ERR_CUDA;
    if (p.n_test > 0) {
        if (!make_tensor_map(&mq_test, p.q_test, C::kES, heads, p.n_test, kD, kTileM, C::kBoxCols))
            return FP8ATTN_ERR_CUDA;
    } else {
        mq_test = mq_train;
    }
    if (test_only) mq_train = mq_test;   // never used: the work list has no train blocks
    KernelArgs a;
    a.scale_q = p.scale_q; a.scale_k = p.scale_k; a.scale_v = p.scale_v;
    a.out_train = p.out_train; a.out_test = p.out_test;
    a.n_train = p.n_train; a.n_test = p.n_test;
    a.blocks_train = test_only ? 0 : (int)((p.n_train + kRowsPerBlock<kT> - 1) / kRowsPerBlock<kT>);
    a.blocks_test = (int)((p.n_test + kRowsPerBlock<kT> - 1) / kRowsPerBlock<kT>);
    a.softmax_scale = p.softmax_scale;
    a.heads = p.H;
    a.test_kv_head0 = (p.flags & FP8ATTN_TEST_ROWS_USE_KV_HEAD0) ? 1 : 0;
    a.status = p.status;
    int64_t grid = heads * (a.blocks_train + a.blocks_test);
    if (grid > 0x7fffffffll) return FP8ATTN_ERR_UNSUPPORTED;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FP8ATTN_ERR_CUDA;
    // Tail split: what is left of the grid after the last full round of one CTA per SM runs
    // as several CTAs per query block, each over its own share of the keys.
    a.full_blocks = (int)grid;
    a.splits = 1;
    a.partial = nullptr;
    int units = 0;
    // (three-tile launches have at least eight rounds, where the split does not pay)
    if (kT == 2 && (p.flags & FP8ATTN_SPLIT_TAIL) && p.partial != nullptr) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            return FP8ATTN_ERR_CUDA;
        const int64_t full = (grid / sms) * sms, left = grid - full;
        const int64_t steps = (p.n_train + C::kKeys - 1) / C::kKeys;
        // Measured: it pays from about one round up to about eight (1.4x at 1.1 rounds, 1.27x
        // at 2.2, 1.1x at 4.3, nothing beyond 8: after many rounds the SMs have drifted apart
        // and the last round is no longer a round), provided a key range keeps at least four
        // steps; below that the extra launches cost more than the split saves.
        if (left > 0 && grid < 8 * (int64_t)sms && steps >= 16) {
            int64_t splits = sms / left;
            if (splits > steps / 4) splits = steps / 4;
            if (splits > kMaxSplits) splits = kMaxSplits;
            const size_t per_split = (size_t)left * kRowsPerBlock<kT> * kPartialStride<kD> * sizeof(float);
            while (splits >= 2 && per_split * (size_t)splits > p.partial_bytes) --splits;
            if (splits >= 2) {
                a.full_blocks = (int)full;
                a.splits = (int)splits;
                a.partial = p.partial;
                units = (int)left;
            }
        }
    }
    auto kern = icl_attention_kernel<kFp8, kD, kHalf, kT, false>;
    auto kern_split = icl_attention_kernel<kFp8, kD, kHalf, 2, true>;
    // The opt-in to large dynamic shared memory is per device and per context; it is set on
    // every call (a cached flag would go stale when the context is destroyed).
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::kSmemBytes) !=
            cudaSuccess ||
        (units > 0 && cudaFuncSetAttribute(kern_split, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)C::kSmemBytes) != cudaSuccess))
        return FP8ATTN_ERR_CUDA;
    if (units > 0) {
        // The split blocks go first; the main grid and the combine kernel follow in stream
        // order.  (Releasing the main grid early behind the split grid by programmatic dependent
        // launch gained 1-2.5 % on launches of one to three rounds, but made the main grid's CTAs
        // wait for the split grid before they exit, the only wait of the library that no
        // time limit bounds.)
        kern_split<<<(unsigned)(units * a.splits), kNumThreads<kT>, C::kSmemBytes, stream>>>(mq_train, mq_test,
                                                                                      mk, mv, a);
        if (cudaGetLastError() != cudaSuccess) return FP8ATTN_ERR_CUDA;
        count_launch();
    }
    if (a.full_blocks > 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)a.full_blocks);
        cfg.blockDim = dim3(kNumThreads<kT>);
        cfg.dynamicSmemBytes = C::kSmemBytes;
        cfg.stream = stream;
        cfg.attrs = nullptr;
        cfg.numAttrs = 0;
        if (cudaLaunchKernelEx(&cfg, kern, mq_train, mq_test, mk, mv, a) != cudaSuccess)
            return FP8ATTN_ERR_CUDA;
        count_launch();
    }
    if (units > 0) {
        const int64_t threads = (int64_t)units * kRowsPerBlock<kT> * (kD / 8);
        combine_split_kernel<kD, 2><<<(unsigned)((threads + 255) / 256), 256, 0, stream>>>(
            a, units, kHalf ? 1 : 0, kFp8 ? 1 : 0);
        count_launch();
    }
    return cudaGetLastError() == cudaSuccess ? FP8ATTN_OK : FP8ATTN_ERR_CUDA;
}

}  // namespace

// Exercises the error path of the bounded waits without touching any real work:
// one warp waits, with the given limit, on a barrier that nothing ever arrives on,
// records the timeout in the status words and returns normally.
__global__ void wait_timeout_selftest_kernel(uint32_t* status, uint64_t limit_ns) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
    }
    __syncthreads();
    Waiter w{status, false, limit_ns};
    w.wait(smem_u32(&bar), 0, kWaitSelfTest);
}

int launch_wait_timeout_selftest(uint32_t* status, uint64_t limit_ns, cudaStream_t stream) {
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? FP8ATTN_OK : FP8ATTN_ERR_CUDA;
}

// d = 64: three tiles per CTA where the grid of 384-row blocks still fills the SMs at least
// eight times over (there the last, partly filled round no longer matters, and neither does
// the tail split); two tiles per CTA for smaller launches.
template <bool kFp8, bool kHalf>
int launch_d64(const AttnParams& p, cudaStream_t stream) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return FP8ATTN_ERR_CUDA;
    if (attention_rows_per_cta(p.B, p.H, p.n_train, p.n_test, 64, p.flags, sms) == kRowsPerBlock<3>)
        return launch<kFp8, 64, kHalf, 3>(p, stream);
    return launch<kFp8, 64, kHalf, 2>(p, stream);
}

int attention_rows_per_cta(int B, int H, int64_t n_train, int64_t n_test, int d, uint32_t flags, int sms) {
    if (d != 64) return kRowsPerBlock<2>;
    const int64_t rows3 = kRowsPerBlock<3>;
    const int64_t blocks = ((flags & FP8ATTN_TEST_ROWS_ONLY) ? 0 : (n_train + rows3 - 1) / rows3) +
                           (n_test + rows3 - 1) / rows3;
    return (int64_t)B * H * blocks >= 8 * (int64_t)sms ? kRowsPerBlock<3> : kRowsPerBlock<2>;
}

int launch_icl_attention(const AttnParams& p, bool fp8, cudaStream_t stream) {
    const bool half = (p.flags & FP8ATTN_IO_FP16) != 0;
    if (fp8) {
        if (half) return p.d == 64 ? launch_d64<true, true>(p, stream) : launch<true, 128, true, 2>(p, stream);
        return p.d == 64 ? launch_d64<true, false>(p, stream) : launch<true, 128, false, 2>(p, stream);
    }
    if (half) return p.d == 64 ? launch_d64<false, true>(p, stream) : launch<false, 128, true, 2>(p, stream);
    return p.d == 64 ? launch_d64<false, false>(p, stream) : launch<false, 128, false, 2>(p, stream);
}

}  // namespace fp8attn
