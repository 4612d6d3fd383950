// Actuator, tensor-core regime: the FFN over a list of active groups as two grouped GEMMs on the
// 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory, operands fed by TMA).
//
//   gate/up  (ffn_gateup_mma_kernel):  for group g of the list and a tile of 128 tokens
//        D[128 tokens, 256] = X[128, d] * [W_gate[g rows]; W_up[g rows]]^T      (bf16 x bf16 -> f32)
//        act[token, slot*128 + c] = silu(D[:, c]) * D[:, 128 + c]  (* membership mask), as bf16
//   down     (ffn_down_mma_kernel):    for a tile of 128 tokens, 256 output columns, a slice of the list
//        P[128, 256] = act[128, slice] * Wd_t[slice rows, 256 columns]
//   then out = residual + sum over slices of P (reduce_slices_kernel).
//
// The same kernels serve both uses of the paper's method: the prompt-level variant (one support
// shared by every token: list = that support, no mask) and large decode batches with independent
// supports (list = union of the supports, mask = which token owns which group).  With at most 128
// tokens a single 128-row MMA tile holds every token, so "bucketing tokens by group" costs nothing
// extra: the bucket of a group is the set of rows whose mask bit is set, and rows outside the bucket
// are zeroed in the epilogue.  (Smaller MMA tiles would not be cheaper: the instruction's cost is
// set by the 128-row weight operand it reads from shared memory.)
//
// Operand layouts (all 128-byte swizzled, written by TMA, read through shared-memory descriptors):
//   X, act, W_gate, W_up tiles are K-major: [rows][64 k] with 128-byte rows, 8-row swizzle atoms.
//   Wd_t tiles are N-major (the 256 output columns are contiguous in memory): four blocks of
//   [64 k rows][64 columns], 8 KB each.
//
// One CTA per tile, six warps: warp 0 issues TMA, warp 1 owns tensor memory and issues the MMAs
// (one elected lane), warps 2-5 run the epilogue (one warp per 32 TMEM lanes).  Every wait on an
// mbarrier is bounded; a wait that runs out records CS_ERR_TIMEOUT in the plan's status word and the
// CTA drains and exits.
#include <cuda.h>

#include <algorithm>
#include <vector>

#include "cs_internal.cuh"

namespace cs {

namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kMaxStages = 8;
constexpr int kABytes = BM * BK * 2;   // 16 KB
constexpr int kBBytes = BN * BK * 2;   // 32 KB
constexpr int kRingBytesMma = 4 * (kABytes + kBBytes);   // 192 KB of operand tiles
constexpr int kMmaThreads = 192;
// Epilogue warps come in slices of four (a warp may read the tensor-memory lane quarter warp % 4); a kernel
// launched with 64 + 128 S threads drains its accumulators with S slices, each taking every S-th chunk.
constexpr int kSwapMaxThreads = 64 + 4 * 128;
constexpr int kTileThreads = kSwapMaxThreads;   // the 128-token-tile kernels: four slices
constexpr uint32_t kSpinLimit = 1u << 20;
constexpr size_t kMmaSmem = 1024 + (size_t)kRingBytesMma + 256;

struct Barriers {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t acc_ready;
    uint32_t tmem_base;
    uint32_t aborted;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bounded wait on a phase parity.  Returns false (after flagging the timeout) if the limit is hit.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, Barriers *bars, DeviceStatus *status) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        uint32_t done;
        asm volatile(
            "{\n.reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n}"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (*reinterpret_cast<volatile uint32_t *>(&bars->aborted)) return false;
    }
    bars->aborted = 1;
    atomicCAS(&status->code, 0, (int)CS_ERR_TIMEOUT);
    return false;
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 consecutive f32 columns of this warp's 32 TMEM lanes.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors (version 1, 128-byte swizzle).  Offsets are in 16-byte units.
//   K-major:  rows 128 bytes apart, 8-row atoms 1024 bytes apart (SBO); LBO unused.
//   MN-major: 64-element blocks `lbo_bytes` apart (LBO), 8-row k groups 1024 bytes apart (SBO).
__device__ __forceinline__ uint64_t desc_sw128(uint32_t saddr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3ffff) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;   // descriptor version
    d |= (uint64_t)2 << 61;   // SWIZZLE_128B
    return d;
}
// Instruction descriptor: bf16 x bf16 -> f32, M = 128, N = 256; b_mn = B operand is N-major.
__host__ __device__ constexpr uint32_t make_idesc(bool b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) |
           ((uint32_t)(BM >> 4) << 24);
}

// General form: N columns, either operand MN-major.
__device__ __forceinline__ uint32_t make_idesc_rt(int n, bool a_mn, bool b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}
// 16 consecutive f32 columns of this warp's 32 TMEM lanes.
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
// Barriers + tensor memory of `ncols` columns (a power of two >= 32), owned by warp 1.
__device__ __forceinline__ void setup_cta(Barriers *bars, int warp, uint32_t ncols) {
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
        mbar_init(&bars->acc_ready, 1);
        bars->aborted = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&bars->tmem_base)), "r"(ncols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
}
__device__ __forceinline__ void teardown_cta(Barriers *bars, int warp, uint32_t ncols) {
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(bars->tmem_base), "r"(ncols) : "memory");
    }
}

// SPLIT: the activation operand comes as two bf16 matrices (high part and remainder, whose sum
// carries ~16 mantissa bits), each stage holds both A tiles and every MMA is issued twice.  The
// ring then has three stages of 64 KB instead of four of 48 KB.
template <bool SPLIT> struct Ring {
    static constexpr int kStages = SPLIT ? 3 : 4;
    static constexpr int kStageBytes = (SPLIT ? 2 : 1) * kABytes + kBBytes;
    static constexpr int kTxBytes = kStageBytes;
};
template <bool SPLIT> struct Tiles {
    uint8_t *base;    // 1024-byte aligned; stage s holds its A tile(s) then its B tile
    Barriers *bars;
    __device__ __forceinline__ uint8_t *a(int s) const { return base + (size_t)s * Ring<SPLIT>::kStageBytes; }
    __device__ __forceinline__ uint8_t *a_lo(int s) const { return a(s) + kABytes; }
    __device__ __forceinline__ uint8_t *b(int s) const { return a(s) + (SPLIT ? 2 : 1) * kABytes; }
};
template <bool SPLIT> __device__ __forceinline__ Tiles<SPLIT> carve(uint8_t *raw) {
    Tiles<SPLIT> t;
    t.base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~(uintptr_t)1023);
    t.bars = reinterpret_cast<Barriers *>(t.base + (size_t)kRingBytesMma);
    return t;
}

// Common prologue: barriers, tensor memory (256 columns, owned by warp 1).
template <bool SPLIT> __device__ __forceinline__ void prologue(const Tiles<SPLIT> &t, int warp, int lane) {
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(&t.bars->full[s], 1); mbar_init(&t.bars->empty[s], 1); }
        mbar_init(&t.bars->acc_ready, 1);
        t.bars->aborted = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&t.bars->tmem_base)), "r"(256) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    (void)lane;
}
template <bool SPLIT> __device__ __forceinline__ void epilogue_done(const Tiles<SPLIT> &t, int warp) {
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(t.bars->tmem_base), "r"(256) : "memory");
    }
}

// The MMA issue loop shared by both kernels: `kblocks` stages of four K=16 instructions.
template <bool B_MN, bool SPLIT>
__device__ __forceinline__ void mma_loop(const Tiles<SPLIT> &t, int kblocks, DeviceStatus *status) {
    constexpr uint32_t idesc = make_idesc(B_MN);
    constexpr int kStages = Ring<SPLIT>::kStages;
    const uint32_t tmem = t.bars->tmem_base;
    for (int kb = 0; kb < kblocks; ++kb) {
        const int s = kb % kStages;
        if (!mbar_wait(&t.bars->full[s], (kb / kStages) & 1, t.bars, status)) return;
        tc_fence_after();
        const uint32_t a0 = smem_u32(t.a(s)), a1 = smem_u32(t.a_lo(s)), b0 = smem_u32(t.b(s));
#pragma unroll
        for (int k4 = 0; k4 < BK / 16; ++k4) {
            const uint64_t bd = B_MN ? desc_sw128(b0 + k4 * 2048, 64 * BK * 2) : desc_sw128(b0 + k4 * 32, 16);
            tc_mma(tmem, desc_sw128(a0 + k4 * 32, 16), bd, idesc, (kb | k4) != 0);
            if (SPLIT) tc_mma(tmem, desc_sw128(a1 + k4 * 32, 16), bd, idesc, 1);
        }
        tc_commit(&t.bars->empty[s]);   // frees the stage once these MMAs have read it
    }
    tc_commit(&t.bars->acc_ready);
}

__device__ __forceinline__ float silu_f(float x) { return x / (1.f + __expf(-x)); }

}  // namespace

// ---- gate / up --------------------------------------------------------------------------------
template <bool SPLIT>
__global__ void __launch_bounds__(kTileThreads, 1)
ffn_gateup_mma_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_x_lo,
                      const __grid_constant__ CUtensorMap tm_g, const __grid_constant__ CUtensorMap tm_u,
                      const int32_t *__restrict__ glist, const int32_t *__restrict__ ng_dev, int ng_host, int M,
                      int d, int act_ld, const uint32_t *__restrict__ mask, __nv_bfloat16 *__restrict__ act,
                      __nv_bfloat16 *__restrict__ act_lo, DeviceStatus *status) {
    constexpr int kStages = Ring<SPLIT>::kStages;
    extern __shared__ uint8_t smem_raw[];
    const int gi = blockIdx.x, mt = blockIdx.y;
    const int ng = ng_dev != nullptr ? *ng_dev : ng_host;
    if (gi >= ng) return;
    const int g = glist[gi];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Tiles<SPLIT> t = carve<SPLIT>(smem_raw);
    prologue(t, warp, lane);
    const int kblocks = d / BK;

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < kblocks; ++kb) {
                const int s = kb % kStages;
                if (kb >= kStages && !mbar_wait(&t.bars->empty[s], ((kb / kStages) - 1) & 1, t.bars, status)) break;
                mbar_expect_tx(&t.bars->full[s], Ring<SPLIT>::kTxBytes);
                tma_load_2d(t.a(s), &tm_x, kb * BK, mt * BM, &t.bars->full[s]);
                if (SPLIT) tma_load_2d(t.a_lo(s), &tm_x_lo, kb * BK, mt * BM, &t.bars->full[s]);
                tma_load_2d(t.b(s), &tm_g, kb * BK, g * 128, &t.bars->full[s]);
                tma_load_2d(t.b(s) + kBBytes / 2, &tm_u, kb * BK, g * 128, &t.bars->full[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) mma_loop<false, SPLIT>(t, kblocks, status);
    } else {
        const int q = warp & 3;                    // TMEM lane quarter this warp may read
        const int slice = (warp - 2) >> 2, nslice = ((int)(blockDim.x >> 5) - 2) >> 2;
        const int row = q * 32 + lane, m = mt * BM + row;
        if (mbar_wait(&t.bars->acc_ready, 0, t.bars, status)) {
            tc_fence_after();
            const uint32_t tbase = t.bars->tmem_base + ((uint32_t)(q * 32) << 16);
            float keep = 1.f;
            if (mask != nullptr && m < M) keep = ((mask[(size_t)m * 4 + (g >> 5)] >> (g & 31)) & 1u) ? 1.f : 0.f;
#pragma unroll 1
            for (int c = slice; c < 4; c += nslice) {
                uint32_t gv[32], uv[32];
                tc_ld32(tbase + c * 32, gv);
                tc_ld32(tbase + 128 + c * 32, uv);
                tc_wait_ld();
                uint32_t packed[16], packed_lo[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float a0 = silu_f(__uint_as_float(gv[2 * j])) * __uint_as_float(uv[2 * j]) * keep;
                    const float a1 = silu_f(__uint_as_float(gv[2 * j + 1])) * __uint_as_float(uv[2 * j + 1]) * keep;
                    const __nv_bfloat162 p = __floats2bfloat162_rn(a0, a1);
                    packed[j] = *reinterpret_cast<const uint32_t *>(&p);
                    if (SPLIT) {
                        const __nv_bfloat162 r = __floats2bfloat162_rn(a0 - __low2float(p), a1 - __high2float(p));
                        packed_lo[j] = *reinterpret_cast<const uint32_t *>(&r);
                    }
                }
                if (m < M) {
                    const size_t off = (size_t)m * act_ld + (size_t)gi * 128 + c * 32;
                    uint4 *dst = reinterpret_cast<uint4 *>(act + off);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        dst[j] = make_uint4(packed[4 * j], packed[4 * j + 1], packed[4 * j + 2], packed[4 * j + 3]);
                    if (SPLIT) {
                        uint4 *dlo = reinterpret_cast<uint4 *>(act_lo + off);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            dlo[j] = make_uint4(packed_lo[4 * j], packed_lo[4 * j + 1], packed_lo[4 * j + 2], packed_lo[4 * j + 3]);
                    }
                }
            }
        }
    }
    epilogue_done(t, warp);
}

// ---- gate / up for one shared support (the prompt-level variant): single and paired token tiles ---------
// A 128 x 256 tile with both operands streamed per 64-wide k block takes in 0.0117 bytes per flop, which at
// the rate of the tensor pipe is more than the SMs can take in from L2 (the kernel above sits at 13.5 TB/s
// of ingest with the pipe 63 % busy).  A CTA that owns TWO token tiles of one group shares every weight
// tile between them: 64 KB per stage for twice the flops, two accumulators in the 512 tensor-memory
// columns.  Paired tiles alone would waste the last wave (a pair is twice the work), so one launch mixes
// them: CTAs [0, n_pair) take pair slots, the CTAs behind them split the remaining pair slots into single
// tiles; the hardware hands CTAs out in index order, so the singles fill the SMs as the pairs finish.
// Pair slot q = (group q % ng, token tiles 2 (q / ng) and 2 (q / ng) + 1).
__global__ void __launch_bounds__(kTileThreads, 1)
ffn_gateup_tiles_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_g,
                        const __grid_constant__ CUtensorMap tm_u, const int32_t *__restrict__ glist, int ng, int n_pair,
                        int mtiles, int M, int d, int act_ld, __nv_bfloat16 *__restrict__ act, DeviceStatus *status) {
    extern __shared__ uint8_t smem_raw[];
    const int c = blockIdx.x;
    const bool pair = c < n_pair;
    const int q = pair ? c : n_pair + ((c - n_pair) >> 1);
    const int gi = q % ng, mt0 = 2 * (q / ng) + (pair ? 0 : ((c - n_pair) & 1));
    if (mt0 >= mtiles) return;                                   // the odd half of a last, incomplete pair slot
    const int ntile = (pair && mt0 + 1 < mtiles) ? 2 : 1;
    const int g = glist[gi];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Barriers *bars = reinterpret_cast<Barriers *>(base + kRingBytesMma);
    const int stage_bytes = ntile * kABytes + kBBytes;           // 48 KB or 64 KB
    const int stages = kRingBytesMma / stage_bytes;              // 4 or 3
    const uint32_t tcols = ntile == 2 ? 512u : 256u;
    setup_cta(bars, warp, tcols);
    const int kblocks = d / BK;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0, ph = 1;                                   // ring slot and the parity of its previous use
            for (int kb = 0; kb < kblocks; ++kb, ++s) {
                if (s == stages) { s = 0; ph ^= 1; }
                if (kb >= stages && !mbar_wait(&bars->empty[s], ph, bars, status)) break;
                uint8_t *st = base + (size_t)s * stage_bytes;
                mbar_expect_tx(&bars->full[s], stage_bytes);
                tma_load_2d(st, &tm_x, kb * BK, mt0 * BM, &bars->full[s]);
                if (ntile == 2) tma_load_2d(st + kABytes, &tm_x, kb * BK, (mt0 + 1) * BM, &bars->full[s]);
                uint8_t *b = st + ntile * kABytes;
                tma_load_2d(b, &tm_g, kb * BK, g * 128, &bars->full[s]);
                tma_load_2d(b + kBBytes / 2, &tm_u, kb * BK, g * 128, &bars->full[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(false);
            const uint32_t tmem = bars->tmem_base;
            bool ok = true;
            int s = 0, ph = 0;
            for (int kb = 0; kb < kblocks && ok; ++kb, ++s) {
                if (s == stages) { s = 0; ph ^= 1; }
                ok = mbar_wait(&bars->full[s], ph, bars, status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a0 = smem_u32(base + (size_t)s * stage_bytes), b0 = a0 + ntile * kABytes;
#pragma unroll
                for (int k4 = 0; k4 < BK / 16; ++k4) {
                    const uint64_t bd = desc_sw128(b0 + k4 * 32, 16);
                    tc_mma(tmem, desc_sw128(a0 + k4 * 32, 16), bd, idesc, (kb | k4) != 0);
                    if (ntile == 2) tc_mma(tmem + 256, desc_sw128(a0 + kABytes + k4 * 32, 16), bd, idesc, (kb | k4) != 0);
                }
                tc_commit(&bars->empty[s]);
            }
            if (ok) tc_commit(&bars->acc_ready);
        }
    } else {
        const int qd = warp & 3;                   // TMEM lane quarter this warp may read
        const int row = qd * 32 + lane;
        const int slice = (warp - 2) >> 2, nslice = ((int)(blockDim.x >> 5) - 2) >> 2;
        if (mbar_wait(&bars->acc_ready, 0, bars, status)) {
            tc_fence_after();
#pragma unroll 1
            for (int e = slice; e < ntile * 4; e += nslice) {   // chunk e: token tile e / 4, 32 channels e % 4
                const int tt = e >> 2, cc = e & 3;
                const int m = (mt0 + tt) * BM + row;
                const uint32_t tbase = bars->tmem_base + ((uint32_t)(qd * 32) << 16) + (uint32_t)(tt * 256);
                {
                    uint32_t gv[32], uv[32];
                    tc_ld32(tbase + cc * 32, gv);
                    tc_ld32(tbase + 128 + cc * 32, uv);
                    tc_wait_ld();
                    uint32_t packed[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float a0 = silu_f(__uint_as_float(gv[2 * j])) * __uint_as_float(uv[2 * j]);
                        const float a1 = silu_f(__uint_as_float(gv[2 * j + 1])) * __uint_as_float(uv[2 * j + 1]);
                        const __nv_bfloat162 p = __floats2bfloat162_rn(a0, a1);
                        packed[j] = *reinterpret_cast<const uint32_t *>(&p);
                    }
                    if (m < M) {
                        uint4 *dst = reinterpret_cast<uint4 *>(act + (size_t)m * act_ld + (size_t)gi * 128 + cc * 32);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            dst[j] = make_uint4(packed[4 * j], packed[4 * j + 1], packed[4 * j + 2], packed[4 * j + 3]);
                    }
                }
            }
        }
    }
    teardown_cta(bars, warp, tcols);
}

// ---- gate / up for one shared support on CTA pairs (M = 256 across two SMs) ------------------------------
// The single-CTA tiles above sit at shared-memory bandwidth: per 128 x 256 x 16 instruction the tensor pipe
// reads 12 KB of operands while TMA refills the ring, 192 bytes per clock asked of a port that serves 128.
// A pair of CTAs on neighbouring SMs (a cluster of two) issues ONE instruction of 256 token rows: each CTA
// holds its own 128 token rows (A) and only HALF of the 256 weight columns (B: the even CTA the gate rows, the
// odd CTA the up rows of the group), so a k block is 32 KB written and 32 KB read per CTA, which the port
// can serve at the tensor pipe's full rate.  No multicast load: each CTA fetches its own tiles; its loads
// signal the even CTA's barrier, whose MMA thread issues for both and frees both CTAs' slots with a
// multicast commit.  Pair slot q = (group q % ng, token tiles 2 (q / ng) and 2 (q / ng) + 1); the launch is
// persistent, at most one cluster per SM pair, each taking every nc-th slot.  A token tile beyond the batch is
// loaded as zeros and not stored.
constexpr int kPairStageBytes = 2 * kABytes;                 // 16 KB of tokens + 16 KB of weights per CTA
constexpr int kPairStages = kRingBytesMma / kPairStageBytes; // 6
static_assert(kPairStages + 2 <= kMaxStages, "the two accumulator barriers of each kind follow the ring's");

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {   // the same offset in CTA `rank`
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load of a CTA pair: data into this CTA's shared memory, bytes counted on a barrier given by its
// cluster address (the even CTA's).
__device__ __forceinline__ void tma_load_2d_pair(void *dst, const CUtensorMap *map, int x, int y, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives (once the MMAs issued so far have completed) on the barrier at this offset in both CTAs of the pair.
__device__ __forceinline__ void tc_commit_pair(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((uint16_t)3) : "memory");
}

// Remote arrive on a barrier of the pair's even CTA (cluster address).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}

// Persistent: the launch has at most one cluster per SM pair, and cluster c takes the pair slots c, c + nc, ...
// The TMA ring runs on across slot boundaries, and the accumulators alternate between the two halves of the 512
// tensor-memory columns, so the set-up, the first loads and the epilogue of a slot (8.4 us of a 36 us round
// when every slot was a cluster of its own) overlap the main loop of the next.  An accumulator half is reused
// two slots later, once all epilogue warps of BOTH CTAs have arrived on its `acc_empty` barrier in the even CTA.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kTileThreads, 1)
ffn_gateup_pair_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_g,
                       const __grid_constant__ CUtensorMap tm_u, const int32_t *__restrict__ glist, int ng, int slots,
                       int M, int d, int act_ld, __nv_bfloat16 *__restrict__ act, DeviceStatus *status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t rank = cluster_ctarank();                  // 0: gate half, issues the MMAs; 1: up half
    const int c0 = blockIdx.x >> 1, nc = gridDim.x >> 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nepi = (int)(blockDim.x >> 5) - 2;              // epilogue warps of one CTA
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Barriers *bars = reinterpret_cast<Barriers *>(base + kRingBytesMma);
    uint64_t *acc_full = &bars->full[kPairStages], *acc_empty = &bars->empty[kPairStages];   // two each
    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
        mbar_init(&acc_full[0], 1); mbar_init(&acc_full[1], 1);
        mbar_init(&acc_empty[0], 2 * nepi); mbar_init(&acc_empty[1], 2 * nepi);
        bars->aborted = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // the same warp of both CTAs allocates for the pair
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&bars->tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();        // the peer's barriers exist before anything signals them
    tc_fence_after();
    const int kblocks = d / BK;

    if (warp == 0) {
        if (lane == 0) {
            const uint32_t full0 = map_to_cta(smem_u32(&bars->full[0]), 0);   // the even CTA's full barriers
            const CUtensorMap *tm_w = rank ? &tm_u : &tm_g;
            int s = 0, ph = 1, it = 0;
            bool ok = true;
            for (int q = c0; q < slots && ok; q += nc) {
                const int g = glist[q % ng], mt = 2 * (q / ng) + (int)rank;
                for (int kb = 0; kb < kblocks; ++kb, ++s, ++it) {
                    if (s == kPairStages) { s = 0; ph ^= 1; }
                    if (it >= kPairStages && !mbar_wait(&bars->empty[s], ph, bars, status)) { ok = false; break; }
                    uint8_t *st = base + (size_t)s * kPairStageBytes;
                    if (rank == 0) mbar_expect_tx(&bars->full[s], 2 * kPairStageBytes);   // both CTAs' bytes
                    tma_load_2d_pair(st, &tm_x, kb * BK, mt * BM, full0 + 8u * s);
                    tma_load_2d_pair(st + kABytes, tm_w, kb * BK, g * 128, full0 + 8u * s);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
            bool ok = true;
            int s = 0, ph = 0, j = 0;
            for (int q = c0; q < slots && ok; q += nc, ++j) {
                const int a = j & 1;
                // the epilogues of the slot before last have left this half
                if (j >= 2) { ok = mbar_wait(&acc_empty[a], ((j >> 1) - 1) & 1, bars, status); if (!ok) break; tc_fence_after(); }
                const uint32_t tmem = bars->tmem_base + (uint32_t)(a * 256);
                for (int kb = 0; kb < kblocks; ++kb, ++s) {
                    if (s == kPairStages) { s = 0; ph ^= 1; }
                    ok = mbar_wait(&bars->full[s], ph, bars, status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a0 = smem_u32(base + (size_t)s * kPairStageBytes), b0 = a0 + kABytes;
#pragma unroll
                    for (int k4 = 0; k4 < BK / 16; ++k4)   // the descriptors' offsets hold in both CTAs' shared memory
                        tc_mma_pair(tmem, desc_sw128(a0 + k4 * 32, 16), desc_sw128(b0 + k4 * 32, 16), idesc, (kb | k4) != 0);
                    tc_commit_pair(&bars->empty[s]);
                }
                if (ok) tc_commit_pair(&acc_full[a]);
            }
        }
    } else {
        const int qd = warp & 3;
        const int slice = (warp - 2) >> 2, nslice = nepi >> 2;
        const uint32_t empty0 = map_to_cta(smem_u32(&acc_empty[0]), 0);   // the even CTA's acc_empty barriers
        int j = 0;
        for (int q = c0; q < slots; q += nc, ++j) {
            const int a = j & 1;
            const int gi = q % ng, mt = 2 * (q / ng) + (int)rank;
            const int m = mt * BM + qd * 32 + lane;
            if (!mbar_wait(&acc_full[a], (j >> 1) & 1, bars, status)) break;
            tc_fence_after();
            const uint32_t tbase = bars->tmem_base + ((uint32_t)(qd * 32) << 16) + (uint32_t)(a * 256);
#pragma unroll 1
            for (int cc = slice; cc < 4; cc += nslice) {
                uint32_t gv[32], uv[32];
                tc_ld32(tbase + cc * 32, gv);
                tc_ld32(tbase + 128 + cc * 32, uv);
                tc_wait_ld();
                uint32_t packed[16];
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) {
                    const float a0 = silu_f(__uint_as_float(gv[2 * jj])) * __uint_as_float(uv[2 * jj]);
                    const float a1 = silu_f(__uint_as_float(gv[2 * jj + 1])) * __uint_as_float(uv[2 * jj + 1]);
                    const __nv_bfloat162 p = __floats2bfloat162_rn(a0, a1);
                    packed[jj] = *reinterpret_cast<const uint32_t *>(&p);
                }
                if (m < M) {
                    uint4 *dst = reinterpret_cast<uint4 *>(act + (size_t)m * act_ld + (size_t)gi * 128 + cc * 32);
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj)
                        dst[jj] = make_uint4(packed[4 * jj], packed[4 * jj + 1], packed[4 * jj + 2], packed[4 * jj + 3]);
                }
            }
            // this warp has taken what it needs from the half: one arrival per warp, of both CTAs, frees it
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(empty0 + 8u * a);
        }
    }
    // Neither CTA leaves (or frees tensor memory) while the other may still read its shared memory or signal
    // its barriers; every wait above is bounded, so both reach this point.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(bars->tmem_base), "r"(512) : "memory");
    }
}

// ---- down -------------------------------------------------------------------------------------
// grid (d / 256, token tiles, slices).  Slice z covers list entries [z*ng/Z, (z+1)*ng/Z).
template <bool SPLIT>
__global__ void __launch_bounds__(kTileThreads, 1)
ffn_down_mma_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_act_lo,
                    const __grid_constant__ CUtensorMap tm_wd, const int32_t *__restrict__ glist,
                    const int32_t *__restrict__ ng_dev, int ng_host, int M, int m_pad, int d,
                    float *__restrict__ partial, const float *residual, float *out_f32,
                    __nv_bfloat16 *__restrict__ out_bf16, DeviceStatus *status) {
    constexpr int kStages = Ring<SPLIT>::kStages;
    extern __shared__ uint8_t smem_raw[];
    const int nt = blockIdx.x, mt = blockIdx.y, z = blockIdx.z, Z = gridDim.z;
    const int ng = ng_dev != nullptr ? *ng_dev : ng_host;
    const int gi0 = (int)(((long long)ng * z) / Z), gi1 = (int)(((long long)ng * (z + 1)) / Z);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Tiles<SPLIT> t = carve<SPLIT>(smem_raw);
    prologue(t, warp, lane);
    const int kblocks = (gi1 - gi0) * 2;   // two 64-row k blocks per 128-channel group

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < kblocks; ++kb) {
                const int s = kb % kStages;
                if (kb >= kStages && !mbar_wait(&t.bars->empty[s], ((kb / kStages) - 1) & 1, t.bars, status)) break;
                const int gi = gi0 + (kb >> 1), half = kb & 1;
                const int wrow = glist[gi] * 128 + half * BK;
                mbar_expect_tx(&t.bars->full[s], Ring<SPLIT>::kTxBytes);
                tma_load_2d(t.a(s), &tm_act, gi * 128 + half * BK, mt * BM, &t.bars->full[s]);
                if (SPLIT) tma_load_2d(t.a_lo(s), &tm_act_lo, gi * 128 + half * BK, mt * BM, &t.bars->full[s]);
#pragma unroll
                for (int j = 0; j < BN / 64; ++j)
                    tma_load_2d(t.b(s) + j * (64 * BK * 2), &tm_wd, nt * BN + j * 64, wrow, &t.bars->full[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && kblocks > 0) mma_loop<true, SPLIT>(t, kblocks, status);
    } else {
        const int q = warp & 3;
        const int slice = (warp - 2) >> 2, nslice = ((int)(blockDim.x >> 5) - 2) >> 2;
        const int row = q * 32 + lane, m = mt * BM + row;
        float *dst = partial + ((size_t)z * m_pad + m) * d + (size_t)nt * BN;
        if (kblocks == 0) {   // empty slice: its partial is zero
            if (m < M && slice == 0) for (int c = 0; c < BN; c += 4) *reinterpret_cast<float4 *>(dst + c) = make_float4(0.f, 0.f, 0.f, 0.f);
        } else if (mbar_wait(&t.bars->acc_ready, 0, t.bars, status)) {
            tc_fence_after();
            const uint32_t tbase = t.bars->tmem_base + ((uint32_t)(q * 32) << 16);
            const size_t o = (size_t)m * d + (size_t)nt * BN;      // one slice: the tile is the output itself
#pragma unroll 1
            for (int c = slice; c < BN / 32; c += nslice) {
                uint32_t v[32];
                tc_ld32(tbase + c * 32, v);
                tc_wait_ld();
                if (Z == 1) {
                    if (m < M) {
                        if (residual != nullptr) {
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float4 r = *reinterpret_cast<const float4 *>(residual + o + c * 32 + 4 * j);
                                v[4 * j] = __float_as_uint(__uint_as_float(v[4 * j]) + r.x);
                                v[4 * j + 1] = __float_as_uint(__uint_as_float(v[4 * j + 1]) + r.y);
                                v[4 * j + 2] = __float_as_uint(__uint_as_float(v[4 * j + 2]) + r.z);
                                v[4 * j + 3] = __float_as_uint(__uint_as_float(v[4 * j + 3]) + r.w);
                            }
                        }
                        if (out_f32 != nullptr) {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                *reinterpret_cast<uint4 *>(out_f32 + o + c * 32 + 4 * j) = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                uint32_t pk[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[8 * j + 2 * e]), __uint_as_float(v[8 * j + 2 * e + 1]));
                                    pk[e] = *reinterpret_cast<const uint32_t *>(&h2);
                                }
                                *reinterpret_cast<uint4 *>(out_bf16 + o + c * 32 + 8 * j) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            }
                        }
                    }
                } else if (m < M) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<uint4 *>(dst + c * 32 + 4 * j) = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                }
            }
        }
    }
    epilogue_done(t, warp);
}


// ---- down, one slice, tiles of 128 tokens x 320 columns -----------------------------------------------
// With one list slice the number of tiles decides how evenly the SMs are loaded: 2048 tokens x 5120
// columns are 320 tiles of 256 columns, 2.16 per SM, i.e. three rounds; tiles of 320 columns are 256,
// two rounds of 1.25 times the work.  The accumulator takes 320 of the 512 tensor-memory columns and
// every k step is two instructions (256 + 64 columns).  Activations bf16 (no remainder operand); the
// epilogue writes the output itself.  grid (d / 320, token tiles).
constexpr int BNW = 320;
constexpr int kWideStage = kABytes + BNW * BK * 2;       // 16 KB + 40 KB
constexpr int kWideStages = kRingBytesMma / kWideStage;  // 3

__global__ void __launch_bounds__(kTileThreads, 1)
ffn_down_wide_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_wd,
                     const int32_t *__restrict__ glist, const int32_t *__restrict__ ng_dev, int ng_host, int M, int d,
                     const float *residual, float *out_f32, __nv_bfloat16 *__restrict__ out_bf16, DeviceStatus *status) {
    extern __shared__ uint8_t smem_raw[];
    const int nt = blockIdx.x, mt = blockIdx.y;
    const int ng = ng_dev != nullptr ? *ng_dev : ng_host;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Barriers *bars = reinterpret_cast<Barriers *>(base + kRingBytesMma);
    setup_cta(bars, warp, 512);
    const int kblocks = ng * 2;   // two 64-row k blocks per 128-channel group

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < kblocks; ++kb) {
                const int s = kb % kWideStages;
                if (kb >= kWideStages && !mbar_wait(&bars->empty[s], ((kb / kWideStages) - 1) & 1, bars, status)) break;
                const int gi = kb >> 1, half = kb & 1;
                const int wrow = glist[gi] * 128 + half * BK;
                uint8_t *st = base + (size_t)s * kWideStage;
                mbar_expect_tx(&bars->full[s], kWideStage);
                tma_load_2d(st, &tm_act, gi * 128 + half * BK, mt * BM, &bars->full[s]);
#pragma unroll
                for (int j = 0; j < BNW / 64; ++j)
                    tma_load_2d(st + kABytes + j * (64 * BK * 2), &tm_wd, nt * BNW + j * 64, wrow, &bars->full[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && kblocks > 0) {
            const uint32_t idesc256 = make_idesc_rt(256, false, true), idesc64 = make_idesc_rt(64, false, true);
            const uint32_t tmem = bars->tmem_base;
            bool ok = true;
            for (int kb = 0; kb < kblocks && ok; ++kb) {
                const int s = kb % kWideStages;
                ok = mbar_wait(&bars->full[s], (kb / kWideStages) & 1, bars, status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a0 = smem_u32(base + (size_t)s * kWideStage), b0 = a0 + kABytes;
#pragma unroll
                for (int k4 = 0; k4 < BK / 16; ++k4) {
                    const uint64_t ad = desc_sw128(a0 + k4 * 32, 16);
                    tc_mma(tmem, ad, desc_sw128(b0 + k4 * 2048, 64 * BK * 2), idesc256, (kb | k4) != 0);
                    tc_mma(tmem + 256, ad, desc_sw128(b0 + 4 * (64 * BK * 2) + k4 * 2048, 64 * BK * 2), idesc64, (kb | k4) != 0);
                }
                tc_commit(&bars->empty[s]);
            }
            if (ok) tc_commit(&bars->acc_ready);
        }
    } else {
        const int q = warp & 3;
        const int slice = (warp - 2) >> 2, nslice = ((int)(blockDim.x >> 5) - 2) >> 2;
        const int m = mt * BM + q * 32 + lane;
        if (kblocks > 0 && mbar_wait(&bars->acc_ready, 0, bars, status)) {
            tc_fence_after();
            const uint32_t tbase = bars->tmem_base + ((uint32_t)(q * 32) << 16);
            const size_t o = (size_t)m * d + (size_t)nt * BNW;
#pragma unroll 1
            for (int c = slice; c < BNW / 32; c += nslice) {
                uint32_t v[32];
                tc_ld32(tbase + c * 32, v);
                tc_wait_ld();
                if (m < M) {
                    if (residual != nullptr) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float4 r = *reinterpret_cast<const float4 *>(residual + o + c * 32 + 4 * j);
                            v[4 * j] = __float_as_uint(__uint_as_float(v[4 * j]) + r.x);
                            v[4 * j + 1] = __float_as_uint(__uint_as_float(v[4 * j + 1]) + r.y);
                            v[4 * j + 2] = __float_as_uint(__uint_as_float(v[4 * j + 2]) + r.z);
                            v[4 * j + 3] = __float_as_uint(__uint_as_float(v[4 * j + 3]) + r.w);
                        }
                    }
                    if (out_f32 != nullptr) {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            *reinterpret_cast<uint4 *>(out_f32 + o + c * 32 + 4 * j) = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint32_t pk[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[8 * j + 2 * e]), __uint_as_float(v[8 * j + 2 * e + 1]));
                                pk[e] = *reinterpret_cast<const uint32_t *>(&h2);
                            }
                            *reinterpret_cast<uint4 *>(out_bf16 + o + c * 32 + 8 * j) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        }
                    }
                }
            }
        }
    }
    teardown_cta(bars, warp, 512);
}


// ---- decode batches of at most 128 tokens: weights on the M side -------------------------------
// With few tokens the cheap orientation is the transposed one: the 128 channel rows of a weight
// block are the MMA's M operand and the tokens its N columns (N = batch rounded up to 16), so an
// instruction costs in proportion to the batch instead of a fixed 256 columns.
//   gate/up:  D_g[128 ch, N] = W_gate[g rows] X^T,  D_u likewise;  actT[slot*128 + ch, token] = silu(D_g) D_u
//   down:     D[128 out columns, N] = Wd_t[slice rows, 128 columns]^T actT[slice rows, tokens]
// actT is stored channel-major (tokens contiguous, pitch 128), which makes it an N-major B operand for
// the down GEMM; the Wd_t tile is the M-major A operand.
template <bool SPLIT>
__global__ void __launch_bounds__(kSwapMaxThreads, 1)
ffn_gateup_swap_kernel(const __grid_constant__ CUtensorMap tm_g, const __grid_constant__ CUtensorMap tm_u,
                       const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_x_lo,
                       const int32_t *__restrict__ glist, const int32_t *__restrict__ ng_dev, int N, int d,
                       const uint32_t *__restrict__ gmask, __nv_bfloat16 *__restrict__ actT,
                       __nv_bfloat16 *__restrict__ actT_lo, DeviceStatus *status) {
    extern __shared__ uint8_t smem_raw[];
    // glist == NULL: one CTA per group of the layer, activations stored at the group's own index and
    // left unmasked (the supports are still being recovered on another stream; mask_act_kernel
    // applies them afterwards).
    const int gi = blockIdx.x;
    if (glist != nullptr && gi >= *ng_dev) return;
    const int g = glist != nullptr ? glist[gi] : gi;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Barriers *bars = reinterpret_cast<Barriers *>(base + kRingBytesMma);
    const int xbytes = N * 128;                                    // X tile: N tokens x 64 k
    const int stage_bytes = 2 * kABytes + (SPLIT ? 2 : 1) * xbytes;
    const int stages = min(6, kRingBytesMma / stage_bytes);
    const int NB = (SPLIT ? 2 : 1) * N;                            // columns per accumulator
    const uint32_t tcols = 2 * NB <= 256 ? 256u : 512u;
    setup_cta(bars, warp, tcols);
    const int kblocks = d / BK;

    if (warp == 0) {
        if (lane == 0) {
            // Weights are parameters: the first ring of weight tiles is requested before the wait for the
            // kernel that produces the token tiles (programmatic dependent launch), so the stream from
            // HBM starts while that kernel is still running.
            const int pre = min(stages, kblocks);
            for (int kb = 0; kb < pre; ++kb) {
                uint8_t *st = base + (size_t)kb * stage_bytes;
                mbar_expect_tx(&bars->full[kb], stage_bytes);
                tma_load_2d(st, &tm_g, kb * BK, g * 128, &bars->full[kb]);
                tma_load_2d(st + kABytes, &tm_u, kb * BK, g * 128, &bars->full[kb]);
            }
            pdl_wait();
            for (int kb = 0; kb < pre; ++kb) {
                uint8_t *st = base + (size_t)kb * stage_bytes;
                tma_load_2d(st + 2 * kABytes, &tm_x, kb * BK, 0, &bars->full[kb]);
                if (SPLIT) tma_load_2d(st + 2 * kABytes + xbytes, &tm_x_lo, kb * BK, 0, &bars->full[kb]);
            }
            for (int kb = pre; kb < kblocks; ++kb) {
                const int s = kb % stages;
                if (!mbar_wait(&bars->empty[s], ((kb / stages) - 1) & 1, bars, status)) break;
                uint8_t *st = base + (size_t)s * stage_bytes;
                mbar_expect_tx(&bars->full[s], stage_bytes);
                tma_load_2d(st, &tm_g, kb * BK, g * 128, &bars->full[s]);
                tma_load_2d(st + kABytes, &tm_u, kb * BK, g * 128, &bars->full[s]);
                tma_load_2d(st + 2 * kABytes, &tm_x, kb * BK, 0, &bars->full[s]);
                if (SPLIT) tma_load_2d(st + 2 * kABytes + xbytes, &tm_x_lo, kb * BK, 0, &bars->full[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc_rt(NB, false, false);
            const uint32_t tmem = bars->tmem_base;
            bool ok = true;
            int s = 0, ph = 0;
            for (int kb = 0; kb < kblocks && ok; ++kb, ++s) {
                if (s == stages) { s = 0; ph ^= 1; }
                ok = mbar_wait(&bars->full[s], ph, bars, status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_g = smem_u32(base + (size_t)s * stage_bytes), a_u = a_g + kABytes;
                const uint32_t x0 = a_g + 2 * kABytes;
#pragma unroll
                for (int k4 = 0; k4 < BK / 16; ++k4) {
                    // x_hi and x_lo tiles are adjacent: one B operand of NB rows gives W x_hi in the first
                    // N columns and W x_lo in the next N, at the cost of a single instruction
                    const uint64_t bd = desc_sw128(x0 + k4 * 32, 16);
                    tc_mma(tmem, desc_sw128(a_g + k4 * 32, 16), bd, idesc, (kb | k4) != 0);
                    tc_mma(tmem + NB, desc_sw128(a_u + k4 * 32, 16), bd, idesc, (kb | k4) != 0);
                }
                tc_commit(&bars->empty[s]);
            }
            if (ok) tc_commit(&bars->acc_ready);
        }
    } else {
        // Warps 2.. are the epilogue: four consecutive warps cover the four lane quarters of tensor memory
        // (a warp may read quarter warp % 4), and each such slice of four warps takes every nslice-th
        // chunk of 16 tokens, so the accumulators drain in one or two rounds instead of N / 16 (measured at
        // 64 tokens: 1.5 us instead of 4.6 us after the last MMA).
        const int q = warp & 3, ch = q * 32 + lane;
        const int slice = (warp - 2) >> 2, nslice = ((int)(blockDim.x >> 5) - 2) >> 2;
        pdl_wait();   // nothing is stored before the kernels before this one are complete
        if (mbar_wait(&bars->acc_ready, 0, bars, status)) {
            tc_fence_after();
            const uint32_t tbase = bars->tmem_base + ((uint32_t)(q * 32) << 16);
            const uint4 gm = gmask != nullptr ? *reinterpret_cast<const uint4 *>(gmask + (size_t)g * 4)
                                              : make_uint4(~0u, ~0u, ~0u, ~0u);
            const uint32_t gw[4] = {gm.x, gm.y, gm.z, gm.w};
            const size_t row = ((size_t)gi * 128 + ch) * 128;
#pragma unroll 1
            for (int c = slice; c < N / 16; c += nslice) {
                uint32_t gv[16], uv[16];
                tc_ld16(tbase + c * 16, gv);
                tc_ld16(tbase + NB + c * 16, uv);
                if (SPLIT) {   // add the x_lo halves
                    uint32_t g2[16], u2[16];
                    tc_ld16(tbase + N + c * 16, g2);
                    tc_ld16(tbase + NB + N + c * 16, u2);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        gv[j] = __float_as_uint(__uint_as_float(gv[j]) + __uint_as_float(g2[j]));
                        uv[j] = __float_as_uint(__uint_as_float(uv[j]) + __uint_as_float(u2[j]));
                    }
                } else {
                    tc_wait_ld();
                }
                const uint32_t bits = gw[(c * 16) >> 5] >> ((c * 16) & 31);
                uint32_t hi[8], lo[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float k0 = (bits >> (2 * j)) & 1u ? 1.f : 0.f, k1 = (bits >> (2 * j + 1)) & 1u ? 1.f : 0.f;
                    const float a0 = silu_f(__uint_as_float(gv[2 * j])) * __uint_as_float(uv[2 * j]) * k0;
                    const float a1 = silu_f(__uint_as_float(gv[2 * j + 1])) * __uint_as_float(uv[2 * j + 1]) * k1;
                    const __nv_bfloat162 p = __floats2bfloat162_rn(a0, a1);
                    hi[j] = *reinterpret_cast<const uint32_t *>(&p);
                    if (SPLIT) {
                        const __nv_bfloat162 r = __floats2bfloat162_rn(a0 - __low2float(p), a1 - __high2float(p));
                        lo[j] = *reinterpret_cast<const uint32_t *>(&r);
                    }
                }
                uint4 *dst = reinterpret_cast<uint4 *>(actT + row + c * 16);
                dst[0] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                dst[1] = make_uint4(hi[4], hi[5], hi[6], hi[7]);
                if (SPLIT) {
                    uint4 *dl = reinterpret_cast<uint4 *>(actT_lo + row + c * 16);
                    dl[0] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                    dl[1] = make_uint4(lo[4], lo[5], lo[6], lo[7]);
                }
            }
        }
    }
    teardown_cta(bars, warp, tcols);
}

// grid (d / 128 / CPC, slices).  partial [slice][128 tokens][d].  A CTA owns CPC adjacent tiles of
// 128 output columns, which share every activation tile: these kernels are bound by the bytes the SMs
// take in, from DRAM and L2 alike (about 6.5 TB/s in all), and with one column tile per CTA the
// activation tiles that every CTA fetches again are as many bytes as the weights.
template <bool SPLIT, int CPC>
__global__ void __launch_bounds__(kSwapMaxThreads, 1)
ffn_down_swap_kernel(const __grid_constant__ CUtensorMap tm_wd, const __grid_constant__ CUtensorMap tm_act,
                     const __grid_constant__ CUtensorMap tm_act_lo, const int32_t *__restrict__ glist,
                     const int32_t *__restrict__ ng_dev, int N, int B, int d, int act_by_group,
                     float *__restrict__ partial, DeviceStatus *status) {
    extern __shared__ uint8_t smem_raw[];
    const int c0 = blockIdx.x * 128 * CPC, z = blockIdx.y, Z = gridDim.y;
    const int ng = *ng_dev;
    const int gi0 = (int)(((long long)ng * z) / Z), gi1 = (int)(((long long)ng * (z + 1)) / Z);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Barriers *bars = reinterpret_cast<Barriers *>(base + kRingBytesMma);
    const int nblk = (N + 63) / 64;                                // token blocks of 64
    const int bbytes = nblk * 64 * BK * 2;                         // actT tile: 64 k rows x tokens
    const int stage_bytes = CPC * kABytes + (SPLIT ? 2 : 1) * bbytes;
    const int stages = min(6, kRingBytesMma / stage_bytes);
    const int NB = SPLIT ? 2 * nblk * 64 : N;                      // MMA columns: value blocks then remainder blocks
    const uint32_t tcols = CPC * NB <= 128 ? 128u : CPC * NB <= 256 ? 256u : 512u;
    setup_cta(bars, warp, tcols);
    const int kblocks = (gi1 - gi0) * 2;

    if (warp == 0) {
        if (lane == 0) {
            auto load_w = [&](int kb, int s) {   // weight tile of column tile j / 2: two blocks of 64 columns
                const int wrow = glist[gi0 + (kb >> 1)] * 128 + (kb & 1) * BK;
                uint8_t *st = base + (size_t)s * stage_bytes;
#pragma unroll
                for (int j = 0; j < 2 * CPC; ++j)
                    tma_load_2d(st + j * (64 * BK * 2), &tm_wd, c0 + j * 64, wrow, &bars->full[s]);
            };
            auto load_act = [&](int kb, int s) {
                const int gi = gi0 + (kb >> 1);
                const int arow = (act_by_group ? glist[gi] : gi) * 128 + (kb & 1) * BK;
                uint8_t *st = base + (size_t)s * stage_bytes;
                for (int i = 0; i < nblk; ++i) {
                    tma_load_2d(st + CPC * kABytes + i * (64 * BK * 2), &tm_act, i * 64, arow, &bars->full[s]);
                    if (SPLIT) tma_load_2d(st + CPC * kABytes + bbytes + i * (64 * BK * 2), &tm_act_lo, i * 64, arow, &bars->full[s]);
                }
            };
            // as in the gate/up kernel: the first ring of weight tiles goes out before the wait for the
            // kernel that completes the activations (the group list was final before that kernel began)
            const int pre = min(stages, kblocks);
            for (int kb = 0; kb < pre; ++kb) { mbar_expect_tx(&bars->full[kb], stage_bytes); load_w(kb, kb); }
            pdl_wait();
            for (int kb = 0; kb < pre; ++kb) load_act(kb, kb);
            for (int kb = pre; kb < kblocks; ++kb) {
                const int s = kb % stages;
                if (!mbar_wait(&bars->empty[s], ((kb / stages) - 1) & 1, bars, status)) break;
                mbar_expect_tx(&bars->full[s], stage_bytes);
                load_w(kb, s);
                load_act(kb, s);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && kblocks > 0) {
            const uint32_t idesc = make_idesc_rt(NB, true, true);
            const uint32_t tmem = bars->tmem_base;
            bool ok = true;
            int s = 0, ph = 0;
            for (int kb = 0; kb < kblocks && ok; ++kb, ++s) {
                if (s == stages) { s = 0; ph ^= 1; }
                ok = mbar_wait(&bars->full[s], ph, bars, status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a0 = smem_u32(base + (size_t)s * stage_bytes), b0 = a0 + CPC * kABytes;
#pragma unroll
                for (int k4 = 0; k4 < BK / 16; ++k4) {   // remainder blocks follow the value blocks: one operand
                    const uint64_t bd = desc_sw128(b0 + k4 * 2048, 64 * BK * 2);
#pragma unroll
                    for (int ct = 0; ct < CPC; ++ct)
                        tc_mma(tmem + ct * NB, desc_sw128(a0 + ct * kABytes + k4 * 2048, 64 * BK * 2), bd, idesc, (kb | k4) != 0);
                }
                tc_commit(&bars->empty[s]);
            }
            if (ok) tc_commit(&bars->acc_ready);
        }
    } else {
        const int q = warp & 3;                     // epilogue slices as in the gate/up kernel
        const int slice = (warp - 2) >> 2, nslice = ((int)(blockDim.x >> 5) - 2) >> 2;
        pdl_wait();   // nothing is stored before the kernels before this one are complete
        if (kblocks == 0) {
            for (int ct = 0; ct < CPC; ++ct) {
                float *dst = partial + (size_t)z * 128 * d + c0 + ct * 128 + q * 32 + lane;
                for (int tkn = slice; tkn < B; tkn += nslice) dst[(size_t)tkn * d] = 0.f;
            }
        } else if (mbar_wait(&bars->acc_ready, 0, bars, status)) {
            tc_fence_after();
            for (int ct = 0; ct < CPC; ++ct) {
                const uint32_t tbase = bars->tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ct * NB);
                float *dst = partial + (size_t)z * 128 * d + c0 + ct * 128 + q * 32 + lane;
#pragma unroll 1
                for (int c = slice; c < N / 16; c += nslice) {
                    uint32_t v[16];
                    tc_ld16(tbase + c * 16, v);
                    if (SPLIT) {
                        uint32_t v2[16];
                        tc_ld16(tbase + nblk * 64 + c * 16, v2);
                        tc_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(v2[j]));
                    } else {
                        tc_wait_ld();
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int tkn = c * 16 + j;
                        if (tkn < B) dst[(size_t)tkn * d] = __uint_as_float(v[j]);
                    }
                }
            }
        }
    }
    teardown_cta(bars, warp, tcols);
}


// Zeroes the activations of (group, token) pairs outside the supports: row r of actT belongs to
// group r / 128; bit t of gmask[group] says whether token t owns the group.  One thread per row
// and 8-token chunk, for the value and the remainder matrix.
__global__ void mask_act_kernel(__nv_bfloat16 *__restrict__ actT, __nv_bfloat16 *__restrict__ actT_lo,
                                const uint32_t *__restrict__ gmask, int rows, int N) {
    pdl_launch_dependents();   // the down GEMM may start streaming its weights
    const int chunks = N / 8;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows * chunks) return;
    const int r = i / chunks, c = i - r * chunks;
    const uint32_t bits = (gmask[(size_t)(r >> 7) * 4 + ((c * 8) >> 5)] >> ((c * 8) & 31)) & 0xffu;
    if (bits == 0xffu) return;
    const uint32_t m0 = (bits & 1u ? 0xffffu : 0u) | (bits & 2u ? 0xffff0000u : 0u);
    const uint32_t m1 = (bits & 4u ? 0xffffu : 0u) | (bits & 8u ? 0xffff0000u : 0u);
    const uint32_t m2 = (bits & 16u ? 0xffffu : 0u) | (bits & 32u ? 0xffff0000u : 0u);
    const uint32_t m3 = (bits & 64u ? 0xffffu : 0u) | (bits & 128u ? 0xffff0000u : 0u);
    uint4 *p = reinterpret_cast<uint4 *>(actT + (size_t)r * 128 + c * 8);
    uint4 v = *p; v.x &= m0; v.y &= m1; v.z &= m2; v.w &= m3; *p = v;
    uint4 *q = reinterpret_cast<uint4 *>(actT_lo + (size_t)r * 128 + c * 8);
    uint4 w = *q; w.x &= m0; w.y &= m1; w.z &= m2; w.w &= m3; *q = w;
}

// out[m, :] = residual[m, :] + sum_z partial[z, m, :], slices added in index order.
template <typename OutT>
__global__ void reduce_slices_kernel(const float *__restrict__ partial, int Z, int M, int m_pad, int d,
                                     const float *__restrict__ residual, OutT *__restrict__ out) {
    const size_t i4 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;   // float4 index
    const size_t total4 = (size_t)M * d / 4;
    if (i4 >= total4) return;
    const size_t m = (i4 * 4) / d, c = (i4 * 4) % d;
    float4 s = residual != nullptr ? *reinterpret_cast<const float4 *>(residual + m * d + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int z = 0; z < Z; ++z) {
        const float4 v = *reinterpret_cast<const float4 *>(partial + ((size_t)z * m_pad + m) * d + c);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    if constexpr (sizeof(OutT) == 4) {
        *reinterpret_cast<float4 *>(reinterpret_cast<float *>(out) + m * d + c) = s;
    } else {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(s.x, s.y), hi = __floats2bfloat162_rn(s.z, s.w);
        uint2 p;
        p.x = *reinterpret_cast<const uint32_t *>(&lo);
        p.y = *reinterpret_cast<const uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(out) + m * d + c) = p;
    }
}

// x = y_hi + y_lo with both parts bf16: y_hi = round(x), y_lo = round(x - y_hi).
__global__ void split_bf16_kernel(const float *__restrict__ x, __nv_bfloat16 *__restrict__ y_hi,
                                  __nv_bfloat16 *__restrict__ y_lo, size_t n4) {
    pdl_launch_dependents();   // the gate/up GEMM may start streaming its weights
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    const float4 v = reinterpret_cast<const float4 *>(x)[i];
    const __nv_bfloat162 h0 = __floats2bfloat162_rn(v.x, v.y), h1 = __floats2bfloat162_rn(v.z, v.w);
    const __nv_bfloat162 l0 = __floats2bfloat162_rn(v.x - __low2float(h0), v.y - __high2float(h0));
    const __nv_bfloat162 l1 = __floats2bfloat162_rn(v.z - __low2float(h1), v.w - __high2float(h1));
    uint2 p, q;
    p.x = *reinterpret_cast<const uint32_t *>(&h0); p.y = *reinterpret_cast<const uint32_t *>(&h1);
    q.x = *reinterpret_cast<const uint32_t *>(&l0); q.y = *reinterpret_cast<const uint32_t *>(&l1);
    reinterpret_cast<uint2 *>(y_hi)[i] = p;
    reinterpret_cast<uint2 *>(y_lo)[i] = q;
}

// The same with the RMSNorm of the stacked workload in front: n = x * rsqrt(mean(x^2) + eps) * gamma,
// one CTA per token.  The GEMM's operand does not have to wait for the sketch kernel, which forms the
// same n for itself on the other stream.
constexpr int kNormSplitThreads = 256;
__global__ void __launch_bounds__(kNormSplitThreads)
norm_split_bf16_kernel(const float *__restrict__ x, const float *__restrict__ gamma, float eps, int d,
                       __nv_bfloat16 *__restrict__ y_hi, __nv_bfloat16 *__restrict__ y_lo) {
    __shared__ float red[kNormSplitThreads / 32];
    pdl_launch_dependents();   // the gate/up GEMM may start streaming its weights
    const int t = blockIdx.x, tid = threadIdx.x;
    const float4 *xr = reinterpret_cast<const float4 *>(x + (size_t)t * d);
    const float4 *gr = reinterpret_cast<const float4 *>(gamma);
    float ss = 0.f;
    for (int c = tid; c < d / 4; c += kNormSplitThreads) {
        const float4 v = xr[c];
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    ss = warp_sum(ss);
    if ((tid & 31) == 0) red[tid >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kNormSplitThreads / 32; ++w) tot += red[w];
    const float rscale = rsqrtf(tot / (float)d + eps);
    for (int c = tid; c < d / 4; c += kNormSplitThreads) {
        float4 v = xr[c];
        const float4 g = gr[c];
        v.x = v.x * g.x * rscale; v.y = v.y * g.y * rscale; v.z = v.z * g.z * rscale; v.w = v.w * g.w * rscale;
        const __nv_bfloat162 h0 = __floats2bfloat162_rn(v.x, v.y), h1 = __floats2bfloat162_rn(v.z, v.w);
        const __nv_bfloat162 l0 = __floats2bfloat162_rn(v.x - __low2float(h0), v.y - __high2float(h0));
        const __nv_bfloat162 l1 = __floats2bfloat162_rn(v.z - __low2float(h1), v.w - __high2float(h1));
        uint2 p, q;
        p.x = *reinterpret_cast<const uint32_t *>(&h0); p.y = *reinterpret_cast<const uint32_t *>(&h1);
        q.x = *reinterpret_cast<const uint32_t *>(&l0); q.y = *reinterpret_cast<const uint32_t *>(&l1);
        reinterpret_cast<uint2 *>(y_hi + (size_t)t * d)[c] = p;
        reinterpret_cast<uint2 *>(y_lo + (size_t)t * d)[c] = q;
    }
}

// ---- bucketing: supports [B,k] -> membership masks, per-group token lists, union list ------------
// One CTA.  mask [B][4] (bit g of token t), counts [G], offsets [G+1], token_ids [B*k] (tokens of
// group g ascending at offsets[g]..offsets[g+1]), glist [G] (groups with a non-empty bucket,
// ascending), *nu = their number.
constexpr int kBucketSmemTokens = 2048;   // masks of this many tokens are kept in shared memory

__global__ void __launch_bounds__(1024)
bucket_kernel(const int32_t *__restrict__ support, int B, int k, int G, uint32_t *__restrict__ mask,
              uint32_t *__restrict__ gmask, int32_t *__restrict__ counts, int32_t *__restrict__ offsets,
              int32_t *__restrict__ token_ids, int32_t *__restrict__ glist, int32_t *__restrict__ nu) {
    extern __shared__ uint32_t mask_s[];            // [min(B, kBucketSmemTokens)][4]
    __shared__ int warp_tot[kMaxG / 32], warp_used[kMaxG / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int Bs = min(B, kBucketSmemTokens);
    // membership masks: one (token, slot) pair per thread, OR-ed into shared memory (tokens beyond
    // the shared table go straight to global memory)
    for (int i = tid; i < Bs * 4; i += blockDim.x) mask_s[i] = 0u;
    for (int i = Bs * 4 + tid; i < B * 4; i += blockDim.x) mask[i] = 0u;
    __syncthreads();
    for (int i = tid; i < B * k; i += blockDim.x) {
        const int t = i / k;
        const int g = support[i];
        if (g >= 0 && g < G) {
            if (t < Bs) atomicOr(&mask_s[(size_t)t * 4 + (g >> 5)], 1u << (g & 31));
            else atomicOr(&mask[(size_t)t * 4 + (g >> 5)], 1u << (g & 31));
        }
    }
    __syncthreads();
    for (int i = tid; i < Bs * 4; i += blockDim.x) mask[i] = mask_s[i];
    __threadfence_block();
    __syncthreads();
    if (tid >= kMaxG) return;   // one thread per group from here on (warps 0..3)
    const int g = tid;
    const int word = g >> 5;
    const uint32_t bit = 1u << (g & 31);
    auto member = [&](int t) -> bool {
        return ((t < Bs ? mask_s[(size_t)t * 4 + word] : mask[(size_t)t * 4 + word]) & bit) != 0u;
    };
    // the transposed mask (bit t of group g) for the first 128 tokens, in four scalar words, and the
    // bucket size
    uint32_t w0 = 0u, w1 = 0u, w2 = 0u, w3 = 0u;
    int cnt = 0;
    if (g < G) {
        const int sh = g & 31;
        auto gather32 = [&](int t0) -> uint32_t {
            uint32_t wd = 0u;
#pragma unroll 8
            for (int tt = 0; tt < 32; ++tt) {
                const int t = t0 + tt;
                if (t < Bs) wd |= ((mask_s[(size_t)t * 4 + word] >> sh) & 1u) << tt;
            }
            return wd;
        };
        w0 = gather32(0);
        if (B > 32) w1 = gather32(32);
        if (B > 64) w2 = gather32(64);
        if (B > 96) w3 = gather32(96);
        cnt = __popc(w0) + __popc(w1) + __popc(w2) + __popc(w3);
        for (int t = 128; t < B; ++t) cnt += member(t);
    }
    // exclusive prefix sums over groups of the bucket sizes and of the non-empty flags
    int inc = cnt, used = cnt > 0, uinc = used;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, inc, o), b = __shfl_up_sync(0xffffffffu, uinc, o);
        if (lane >= o) { inc += a; uinc += b; }
    }
    if (lane == 31) { warp_tot[warp] = inc; warp_used[warp] = uinc; }
    // only warps 0..3 are alive: a named barrier over their 128 threads
    asm volatile("bar.sync 1, 128;" ::: "memory");
    int off = inc - cnt, uoff = uinc - used;
    for (int w2 = 0; w2 < warp; ++w2) { off += warp_tot[w2]; uoff += warp_used[w2]; }
    if (g < G) {
        counts[g] = cnt;
        offsets[g] = off;
        if (used) glist[uoff] = g;
        *reinterpret_cast<uint4 *>(gmask + (size_t)g * 4) = make_uint4(w0, w1, w2, w3);
        int o = off;   // tokens of the bucket in ascending order: walk the set bits, then the tail
        auto emit = [&](uint32_t wd, int t0) {
            while (wd) { token_ids[o++] = t0 + __ffs(wd) - 1; wd &= wd - 1; }
        };
        emit(w0, 0); emit(w1, 32); emit(w2, 64); emit(w3, 96);
        for (int t = 128; t < B; ++t)
            if (member(t)) token_ids[o++] = t;
    }
    if (g == kMaxG - 1) { offsets[G] = off + cnt; *nu = uoff + used; }
}

// ---- host side ----------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 matrix [outer, inner] row-major with `ld` elements per row; box = [box_outer rows, 64 columns].
bool make_map(CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer, uint64_t ld, uint32_t box_outer) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {64, box_outer};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// How many of the pair slots a mixed launch runs as paired tiles: CTAs are handed out in index order to
// whichever SM is free first, pairs first.  Measured on B200, a pair takes about 1.8 single-tile times
// (both kinds are bound by what shared memory can serve: the tensor pipe reads 12 KB of operands per
// 128 x 256 x 16 instruction while TMA refills the ring, and a pair saves only the second refill of
// the weight tile), so pairs pay off where they fix the last wave: 176 tiles on 148 SMs (two waves
// of singles, one of pairs), 864 tiles (six waves against three), not 432 (three full waves).
// The count with the shortest predicted makespan wins if it beats all-singles by 8 % or more.
constexpr double kPairCost = 1.8;
static int best_pair_count(int slots, int mtiles, int ng, int sms) {
    int best = 0;
    double best_t = 1e30;
    std::vector<double> free_at(sms);
    for (int n_pair = 0; n_pair <= slots; ++n_pair) {
        std::fill(free_at.begin(), free_at.end(), 0.0);
        auto run = [&](double cost) {
            auto it = std::min_element(free_at.begin(), free_at.end());
            *it += cost;
        };
        for (int q = 0; q < n_pair; ++q) run(2 * (q / ng) + 1 < mtiles ? kPairCost : 1.0);
        for (int q = n_pair; q < slots; ++q) {
            run(1.0);
            if (2 * (q / ng) + 1 < mtiles) run(1.0);
        }
        const double t = *std::max_element(free_at.begin(), free_at.end());
        if (n_pair == 0) { best_t = t * 0.92; continue; }   // what pairs have to beat
        if (t <= best_t + 1e-9) { best_t = t; best = n_pair; }
    }
    return best;
}

cs_status prepare_ffn_mma(cs_plan *plan) {
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(ffn_gateup_tiles_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMmaSmem));
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(ffn_gateup_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMmaSmem));
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(ffn_down_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMmaSmem));
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(ffn_gateup_mma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMmaSmem));
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(ffn_gateup_mma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMmaSmem));
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(ffn_down_mma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMmaSmem));
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(ffn_down_mma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMmaSmem));
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(ffn_gateup_swap_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMmaSmem));
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(ffn_down_swap_kernel<true, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMmaSmem));
    return CS_OK;
}

cs_status launch_bucket(cs_plan *plan, const int32_t *support, int B, cudaStream_t st, int32_t *counts,
                        int32_t *offsets, int32_t *token_ids) {
    const size_t smem = (size_t)min(B, kBucketSmemTokens) * 16;
    bucket_kernel<<<1, 1024, smem, st>>>(support, B, plan->cfg.k, plan->G, plan->mask, plan->gmask,
                                      counts ? counts : plan->counts, offsets ? offsets : plan->offsets,
                                      token_ids ? token_ids : plan->token_ids, plan->glist, plan->nu);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

// X [M, d] bf16 (plus X_lo, the bf16 remainder, when split precision is wanted); list / count on the
// device (ng_dev) or count on the host; mask may be NULL.  Writes out [M, d] as f32 (out_f32) or bf16
// (out_bf16), plus residual (f32, may be NULL).
cs_status launch_ffn_mma(cs_plan *plan, const cs_layer *L, const void *X, const void *X_lo, int M,
                         const int32_t *glist, const int32_t *ng_dev, int ng_host, const uint32_t *mask,
                         const float *residual, float *out_f32, void *out_bf16, cudaStream_t st) {
    const cs_config &c = plan->cfg;
    const bool split = X_lo != nullptr;
    const int grid_g = ng_dev != nullptr ? plan->G : ng_host;       // CTAs past the device count exit at once
    const int act_ld = plan->G * 128;
    const int mtiles = (M + BM - 1) / BM, m_pad = mtiles * BM;
    __nv_bfloat16 *act = static_cast<__nv_bfloat16 *>(plan->act);
    __nv_bfloat16 *act_lo = act + (size_t)plan->cfg.max_tokens * act_ld;
    CUtensorMap tm_x, tm_x_lo, tm_g, tm_u, tm_act, tm_act_lo, tm_wd;
    if (!make_map(&tm_x, X, c.d, M, c.d, BM) || !make_map(&tm_x_lo, split ? X_lo : X, c.d, M, c.d, BM) ||
        !make_map(&tm_g, L->W_gate, c.d, c.d_ff, c.d, 128) || !make_map(&tm_u, L->W_up, c.d, c.d_ff, c.d, 128) ||
        !make_map(&tm_act, act, act_ld, M, act_ld, BM) ||
        !make_map(&tm_act_lo, split ? act_lo : act, act_ld, M, act_ld, BM) ||
        !make_map(&tm_wd, L->Wd_t, c.d, c.d_ff, c.d, BK))
        return record_cuda(plan, cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    // One shared support whose size the host knows: how many pair slots run as paired token tiles (the
    // schedule of this shape, computed once); none leaves the launch to the single-tile kernel.
    int n_pair = 0;
    const int slots = ng_host * ((mtiles + 1) / 2);
    const bool shared = !split && ng_dev == nullptr && mask == nullptr && ng_host > 0;
    if (shared) {
        if (plan->pair_key_ng != ng_host || plan->pair_key_mtiles != mtiles) {
            plan->pair_count = best_pair_count(slots, mtiles, ng_host, plan->sm_count);
            plan->pair_key_ng = ng_host; plan->pair_key_mtiles = mtiles;
        }
        n_pair = plan->pair_count;
    }
    {
        StageTimer timer(plan, CS_STAGE_EXEC, st);
        if (split)
            ffn_gateup_mma_kernel<true><<<dim3(grid_g, mtiles), kTileThreads, kMmaSmem, st>>>(
                tm_x, tm_x_lo, tm_g, tm_u, glist, ng_dev, ng_host, M, c.d, act_ld, mask, act, act_lo, plan->status);
        else if (shared && n_pair == 0) {
            // one shared support and no gain from paired tiles (measured at k = 27 of 108 groups, 2048 tokens:
            // 214 us for the GEMM pair against 223 us with single tiles; with paired tiles in play, k = 11 and
            // 54, the mixed launch below is faster): CTA pairs, one M = 256 instruction over two token tiles
            ffn_gateup_pair_kernel<<<dim3(2 * min(slots, plan->sm_count / 2)), kTileThreads, kMmaSmem, st>>>(
                tm_x, tm_g, tm_u, glist, ng_host, slots, M, c.d, act_ld, act, plan->status);
        } else if (n_pair > 0) {
            // one shared support, its size known on the host: paired and single token tiles in one launch
            ffn_gateup_tiles_kernel<<<dim3(n_pair + 2 * (slots - n_pair)), kTileThreads, kMmaSmem, st>>>(
                tm_x, tm_g, tm_u, glist, ng_host, n_pair, mtiles, M, c.d, act_ld, act, plan->status);
        } else
            ffn_gateup_mma_kernel<false><<<dim3(grid_g, mtiles), kTileThreads, kMmaSmem, st>>>(
                tm_x, tm_x_lo, tm_g, tm_u, glist, ng_dev, ng_host, M, c.d, act_ld, mask, act, act_lo, plan->status);
        plan->launches++;
        CS_CUDA_TRY(plan, cudaGetLastError());
        // slices: fill the machine when one token tile cannot (decode), one slice otherwise (prompt)
        const int ntiles = c.d / BN;
        int Z = 1;
        if (mtiles * ntiles < plan->sm_count) Z = max(1, min(plan->sm_count / (mtiles * ntiles), plan->mma_slices));
        // one slice, bf16 activations: tiles of 320 columns when they need fewer rounds over the SMs
        const int sms = plan->sm_count;
        const bool wide = !split && Z == 1 && c.d % BNW == 0 && ng_host > 0 &&
                          ((mtiles * (c.d / BNW) + sms - 1) / sms) * BNW < ((mtiles * ntiles + sms - 1) / sms) * BN;
        if (wide)
            ffn_down_wide_kernel<<<dim3(c.d / BNW, mtiles), kTileThreads, kMmaSmem, st>>>(
                tm_act, tm_wd, glist, ng_dev, ng_host, M, c.d, residual, out_f32, static_cast<__nv_bfloat16 *>(out_bf16), plan->status);
        else if (split)
            ffn_down_mma_kernel<true><<<dim3(ntiles, mtiles, Z), kTileThreads, kMmaSmem, st>>>(
                tm_act, tm_act_lo, tm_wd, glist, ng_dev, ng_host, M, m_pad, c.d, plan->mma_partial, residual, out_f32,
                static_cast<__nv_bfloat16 *>(out_bf16), plan->status);
        else
            ffn_down_mma_kernel<false><<<dim3(ntiles, mtiles, Z), kTileThreads, kMmaSmem, st>>>(
                tm_act, tm_act_lo, tm_wd, glist, ng_dev, ng_host, M, m_pad, c.d, plan->mma_partial, residual, out_f32,
                static_cast<__nv_bfloat16 *>(out_bf16), plan->status);
        plan->launches++;
        CS_CUDA_TRY(plan, cudaGetLastError());
        plan->last_slices = Z;
    }
    if (plan->last_slices > 1) {   // a single slice has written the output itself
        StageTimer timer(plan, CS_STAGE_REDUCE, st);
        const size_t total4 = (size_t)M * c.d / 4;
        const int blocks = (int)((total4 + 255) / 256);
        if (out_f32 != nullptr)
            reduce_slices_kernel<float><<<blocks, 256, 0, st>>>(plan->mma_partial, plan->last_slices, M, m_pad, c.d, residual, out_f32);
        else
            reduce_slices_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(plan->mma_partial, plan->last_slices, M, m_pad, c.d,
                                                                       residual, static_cast<__nv_bfloat16 *>(out_bf16));
        plan->launches++;
        CS_CUDA_TRY(plan, cudaGetLastError());
    }
    return CS_OK;
}


// Decode batches from the crossover batch up to 128 tokens in three launches that the caller orders
// (the gate/up GEMM can run while the supports are still being recovered on another stream):
//   launch_decode_gateup(masked = false)  every group of the layer, activations unmasked, stored at the
//                                         group's own index;   (masked = true: union list + masks)
//   launch_decode_mask                    zeroes the (group, token) pairs outside the supports
//   launch_decode_down                    down GEMM over the union list, slice reduction, residual
static bool decode_maps(cs_plan *plan, const cs_layer *L, const void *X, const void *X_lo, int B, int N,
                        CUtensorMap *tm) {
    const cs_config &c = plan->cfg;
    __nv_bfloat16 *actT = static_cast<__nv_bfloat16 *>(plan->act);
    __nv_bfloat16 *actT_lo = actT + (size_t)plan->G * 128 * 128;
    return make_map(&tm[0], L->W_gate, c.d, c.d_ff, c.d, 128) && make_map(&tm[1], L->W_up, c.d, c.d_ff, c.d, 128) &&
           make_map(&tm[2], X ? X : plan->x_bf16, c.d, B, c.d, N) &&
           make_map(&tm[3], X_lo ? X_lo : plan->x_bf16, c.d, B, c.d, N) &&
           make_map(&tm[4], L->Wd_t, c.d, c.d_ff, c.d, BK) &&
           make_map(&tm[5], actT, 128, (uint64_t)plan->G * 128, 128, BK) &&
           make_map(&tm[6], actT_lo, 128, (uint64_t)plan->G * 128, 128, BK);
}

cs_status launch_decode_gateup(cs_plan *plan, const cs_layer *L, const void *X, const void *X_lo, int B,
                               bool masked, cudaStream_t st) {
    const cs_config &c = plan->cfg;
    const int N = (B + 15) / 16 * 16;
    __nv_bfloat16 *actT = static_cast<__nv_bfloat16 *>(plan->act);
    __nv_bfloat16 *actT_lo = actT + (size_t)plan->G * 128 * 128;
    CUtensorMap tm[7];
    if (!decode_maps(plan, L, X, X_lo, B, N, tm)) return record_cuda(plan, cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    StageTimer timer(plan, CS_STAGE_EXEC, st);
    const int threads = 64 + 128 * min(4, N / 16);   // one epilogue slice per chunk of 16 tokens, at most four
    launch_pdl(true, ffn_gateup_swap_kernel<true>, dim3(plan->G), dim3(threads), kMmaSmem, st,
               tm[0], tm[1], tm[2], tm[3], masked ? (const int32_t *)plan->glist : (const int32_t *)nullptr,
               (const int32_t *)plan->nu, N, c.d, masked ? (const uint32_t *)plan->gmask : (const uint32_t *)nullptr,
               actT, actT_lo, plan->status);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

cs_status launch_decode_mask(cs_plan *plan, int B, cudaStream_t st) {
    const int N = (B + 15) / 16 * 16;
    __nv_bfloat16 *actT = static_cast<__nv_bfloat16 *>(plan->act);
    __nv_bfloat16 *actT_lo = actT + (size_t)plan->G * 128 * 128;
    const int rows = plan->G * 128, total = rows * (N / 8);
    mask_act_kernel<<<(total + 255) / 256, 256, 0, st>>>(actT, actT_lo, plan->gmask, rows, N);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

cs_status launch_decode_down(cs_plan *plan, const cs_layer *L, int B, bool act_by_group, const float *residual,
                             float *out, cudaStream_t st) {
    const cs_config &c = plan->cfg;
    const int N = (B + 15) / 16 * 16;
    CUtensorMap tm[7];
    if (!decode_maps(plan, L, nullptr, nullptr, B, N, tm)) return record_cuda(plan, cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    const int Z = max(1, min(plan->sm_count / (c.d / 256), 8));   // two column tiles per CTA (d is a multiple of 256)
    {
        StageTimer timer(plan, CS_STAGE_EXEC2, st);
        const int threads = 64 + 128 * min(4, N / 16);
        launch_pdl(true, ffn_down_swap_kernel<true, 2>, dim3(c.d / 256, Z), dim3(threads), kMmaSmem, st,
                   tm[4], tm[5], tm[6], (const int32_t *)plan->glist, (const int32_t *)plan->nu, N, B, c.d,
                   act_by_group ? 1 : 0, plan->mma_partial, plan->status);
        plan->launches++;
        CS_CUDA_TRY(plan, cudaGetLastError());
    }
    {
        StageTimer timer(plan, CS_STAGE_REDUCE, st);
        const size_t total4 = (size_t)B * c.d / 4;
        reduce_slices_kernel<float><<<(int)((total4 + 255) / 256), 256, 0, st>>>(plan->mma_partial, Z, B, 128, c.d, residual, out);
        plan->launches++;
        CS_CUDA_TRY(plan, cudaGetLastError());
    }
    return CS_OK;
}

cs_status launch_norm_split_bf16(cs_plan *plan, const float *x, const float *gamma, int B, void *y_hi, void *y_lo,
                                 cudaStream_t st) {
    norm_split_bf16_kernel<<<B, kNormSplitThreads, 0, st>>>(x, gamma, plan->cfg.rms_eps, plan->cfg.d,
                                                            static_cast<__nv_bfloat16 *>(y_hi), static_cast<__nv_bfloat16 *>(y_lo));
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

cs_status launch_split_bf16(cs_plan *plan, const float *x, void *y_hi, void *y_lo, size_t n, cudaStream_t st) {
    const size_t n4 = n / 4;
    split_bf16_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(x, static_cast<__nv_bfloat16 *>(y_hi),
                                                                   static_cast<__nv_bfloat16 *>(y_lo), n4);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

}  // namespace cs
