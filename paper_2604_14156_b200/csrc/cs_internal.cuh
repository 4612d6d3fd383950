// Internal declarations shared by the library's translation units (not part of the C boundary).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cs.h"

namespace cs {

constexpr int kMaxG = 128;        // groups per layer
constexpr int kMaxM = 64;         // sketch rows
constexpr int kMaxD = 8192;       // hidden size
constexpr int kGatherThreads = 512;
constexpr int kGatherMaxRows = 32;   // channel rows one gather CTA owns at most
constexpr int kGatherMaxTokens = 16; // tokens per gather launch (scratch for partial sums)
constexpr int kSlotTableSlots = 32;  // slots per token of the recovery's slot table (small-batch step) ...
constexpr int kSlotTablePitch = 40;  // ... and ints per token: the slots, then a word that says "final"
constexpr int kReduceGroups = 32;    // partial-sum groups of the deterministic cross-CTA reduction
constexpr int kMmaMinTokens = 16;    // decode batches at least this large always run on the tensor cores; a plan
                                     // lowers the bound by its G / k (cs_plan_set_crossover overrides it)

// Device status word values mirror cs_status (0 = ok).
struct DeviceStatus {
    int code;
};

}  // namespace cs

struct cs_plan {
    cs_config cfg;
    int G;
    int device;
    int sm_count;
    // device scratch
    float *n_buf;      // [max_tokens, d]  normalised FFN input
    float *y_buf;      // [max_tokens, m]
    int32_t *sup_buf;  // [max_tokens, k]
    float *partial;    // [kGatherMaxTokens, nx_max, d] partial down-projections of the gather path
    float *gram;       // [G, pitch] I - mu Phi^T Phi of the layer being recovered, pitch = 32 ceil(G/32)
    float *resid_buf;     // [max_tokens] residual norms when the caller wants none (confidence fallback)
    int32_t *fb_flags;    // [max_tokens] confidence fallback: 1 = the token's recovery is not trusted
    int32_t *fb_list;     // [max_tokens] those tokens, ascending
    int32_t *fb_count;    // [1] their number
    int32_t *slot_table;  // [max_tokens, kSlotTablePitch] small-batch step: slot -> group of the recovery in flight
    unsigned *ticket;     // [max_tokens] arrival counters of the sketch CTAs (zero between launches)
    float *hbar;       // [d] mean prompt hidden state
    float *colsum;     // [mean_row_blocks, d]
    cs::DeviceStatus *status;  // device status word
    // tensor-core path (bf16 weights, 128-channel groups, d a multiple of 256)
    uint32_t *mask;      // [max_tokens, 4] membership bits: bit g of token t
    uint32_t *gmask;     // [G, 4] membership bits the other way round: bit t of group g (t < 128)
    int32_t *counts;     // [G] tokens per group
    int32_t *offsets;    // [G + 1]
    int32_t *token_ids;  // [max_tokens * k] tokens of each group, ascending
    int32_t *glist;      // [G] groups with a non-empty bucket, ascending
    int32_t *nu;         // [1] their number
    void *x_bf16;        // [2][max_tokens, d] bf16 activations: rounded value, then remainder
    void *act;           // [2][max_tokens, d_ff] bf16 SwiGLU activations over the group list (value, remainder)
    float *mma_partial;  // [slices, padded tokens, d] f32 partial down projections
    int speculative;     // small batches, on the recovery's first iterate: 1 = start the weight stream, 2 = warm L2 only
    int mma_ok;          // shape qualifies for the tensor-core path
    int mma_min_tokens;  // smallest decode batch that takes it
    int mma_slices;      // most list slices the down GEMM is split into
    int last_slices;
    int pair_key_ng, pair_key_mtiles, pair_count;   // prompt gate/up: paired-tile count of the last shape seen
    float *x_host_in;  // [max_tokens, d] staging for the host-buffer entry point
    float *x_host_out; // [max_tokens, d]
    cudaEvent_t ev[2 * CS_STAGE_COUNT];  // start/stop per stage
    cudaStream_t side;                   // second stream: recovery runs beside the gate/up GEMM
    cudaEvent_t ev_fork, ev_join;
    int timing;
    int stage_seen[CS_STAGE_COUNT];
    int nx_max;
    int mean_row_blocks;
    int64_t launches;
    char cuda_error[256];
};

namespace cs {

cs_status record_cuda(cs_plan *plan, cudaError_t e, const char *what);

#define CS_CUDA_TRY(plan, expr)                                                     \
    do {                                                                            \
        cudaError_t e_ = (expr);                                                    \
        if (e_ != cudaSuccess) return ::cs::record_cuda((plan), e_, #expr);         \
    } while (0)

// Brackets one stage's launches with events when timing is enabled.  On a capturing stream the
// records become event-record nodes of the graph (external events), which can be timed after a
// replay and cost far less than a record issued from the host between two launches.
struct StageTimer {
    cs_plan *p; int stage; cudaStream_t st;
    static void record(cudaEvent_t ev, cudaStream_t s) {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(s, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusActive)
            cudaEventRecordWithFlags(ev, s, cudaEventRecordExternal);
        else
            cudaEventRecord(ev, s);
    }
    StageTimer(cs_plan *plan, int s, cudaStream_t stream) : p(plan), stage(s), st(stream) {
        if (p->timing) record(p->ev[2 * stage], st);
    }
    ~StageTimer() {
        if (p->timing) { record(p->ev[2 * stage + 1], st); p->stage_seen[stage] = 1; }
    }
};

// Kernel launchers (each enqueues on `st`, bumps plan->launches, returns a status).
// Phi != NULL: the launch also forms the recovery's matrix I - mu Phi^T Phi (plan->gram) in spare CTAs.
cs_status launch_sketch(cs_plan *plan, const float *S, const float *x, const float *gamma, int B,
                        float *y, float *n_out, const float *Phi, float mu, cudaStream_t st);
// gram_ready: plan->gram already holds this Phi's matrix (the sketch launch before formed it).
cs_status launch_recover(cs_plan *plan, const float *Phi, float mu, const float *y, int B,
                         int32_t *support, float *z, float *resid, bool gram_ready, cudaStream_t st,
                         int T = -1 /* the plan's */, const int32_t *sup0 = nullptr, const float *z0 = nullptr,
                         float gamma = 0.f /* temporal term */, const int32_t *sup_prev = nullptr,
                         const float *z_prev = nullptr);
// the other estimators (solvers.cu)
cs_status prepare_solvers(cs_plan *plan);
cs_status launch_niht(cs_plan *plan, const float *Phi, float mu_fallback, const float *y, int B, int T,
                      int32_t *support, float *z, float *resid, cudaStream_t st);
cs_status launch_omp(cs_plan *plan, const float *Phi, const float *y, int B, int32_t *support, float *z, float *resid,
                     cudaStream_t st);
// the structured sketch (srht.cu)
cs_status launch_sketch_srht(cs_plan *plan, const uint32_t *sign_bits, const int32_t *rows, const float *h, int B, float *y,
                             cudaStream_t st);
// check: validate the supports on the device (ascending, distinct, in range) inside the same launch.
// warm: slot tables of a recovery still running in the launch ahead (launch_sketch_recover); the kernel
// asks L2 for the weight blocks they name before it waits for the final supports.
cs_status launch_ffn_gather(cs_plan *plan, const cs_layer *layer, const float *h, const int32_t *support,
                            int B, const float *residual, float *out, bool check, cudaStream_t st,
                            const int32_t *warm = nullptr);
// The small-batch step: sketch and recovery in one launch, whose programmatic trigger fires when the
// first iterate's slot table is in memory; the gather FFN launched behind it starts on that table,
// follows the table while the iteration runs, and settles on the final one.
bool sketch_recover_ok(const cs_plan *plan);
cs_status prepare_sketch(cs_plan *plan);
cs_status launch_sketch_recover(cs_plan *plan, const cs_layer *L, const float *x, int B, float *y, float *n_out,
                                int32_t *support, float *z, float *resid, cudaStream_t st);
cs_status launch_ffn_gather_spec(cs_plan *plan, const cs_layer *layer, const float *h, int B, const float *residual,
                                 float *out, cudaStream_t st);
cs_status prepare_ffn_gather(cs_plan *plan);
cs_status launch_support_drift(cs_plan *plan, const int32_t *prev, const int32_t *cur, int B, int32_t *drift,
                               float *ratio, cudaStream_t st);
// confidence fallback (control.cu): flags tokens whose relative residual exceeds tau, lists them, moves rows
cs_status launch_confidence(cs_plan *plan, const float *y, const float *resid, int B, float tau, int32_t *flags,
                            int32_t *list, int32_t *count, cudaStream_t st);
cs_status launch_gather_rows(cs_plan *plan, const float *src, const int32_t *list, int n, float *dst, cudaStream_t st);
cs_status launch_scatter_rows(cs_plan *plan, const float *src, const int32_t *list, int n, float *dst, cudaStream_t st);
cs_status launch_uds_budget(cs_plan *plan, const float *logits, int B, int V, float m_base, float gamma,
                            int m_min, int m_max, float *H, int32_t *m_t, cudaStream_t st);
cs_status launch_check_support(cs_plan *plan, const int32_t *support, int B, cudaStream_t st);
cs_status prepare_ffn_mma(cs_plan *plan);
cs_status launch_bucket(cs_plan *plan, const int32_t *support, int B, cudaStream_t st, int32_t *counts = nullptr,
                        int32_t *offsets = nullptr, int32_t *token_ids = nullptr);
cs_status launch_split_bf16(cs_plan *plan, const float *x, void *y_hi, void *y_lo, size_t n, cudaStream_t st);
cs_status launch_norm_split_bf16(cs_plan *plan, const float *x, const float *gamma, int B, void *y_hi, void *y_lo,
                                 cudaStream_t st);
cs_status launch_ffn_mma(cs_plan *plan, const cs_layer *L, const void *X, const void *X_lo, int M, const int32_t *glist,
                         const int32_t *ng_dev, int ng_host, const uint32_t *mask, const float *residual,
                         float *out_f32, void *out_bf16, cudaStream_t st);
cs_status launch_decode_gateup(cs_plan *plan, const cs_layer *L, const void *X, const void *X_lo, int B,
                               bool masked, cudaStream_t st);
cs_status launch_decode_mask(cs_plan *plan, int B, cudaStream_t st);
cs_status launch_decode_down(cs_plan *plan, const cs_layer *L, int B, bool act_by_group, const float *residual,
                             float *out, cudaStream_t st);
cs_status launch_prompt_mean(cs_plan *plan, const void *H, int n, float *hbar, cudaStream_t st);

// Programmatic dependent launch: a kernel launched through launch_pdl may start while its
// predecessor in the stream is still running (its CTAs become resident, run their prologue and
// then block in pdl_wait until the predecessor's writes are complete and visible).  Kernels call
// pdl_launch_dependents early so that their successor can do the same.  Both are no-ops for a
// kernel launched the ordinary way (pdl = false).  Only the small-batch chain uses it: its kernels are
// a few microseconds long and launch latency matters; with the large tensor-core kernels early-resident
// dependents measurably slowed the step down.
inline bool pdl_for(const cs_plan *plan, int B) { return !(plan->mma_ok && B >= plan->mma_min_tokens); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Loads of data that the kernel before this one produced.  They are volatile asm statements, like
// the wait itself, so the compiler keeps them after it; a plain load through a const __restrict__
// pointer (or __ldg) may be turned into a non-coherent load and moved above the wait, which reads
// what the buffer held before (seen as rare wrong recoveries when a plan's scratch was reused).
__device__ __forceinline__ float ld_dep(const float *p) {
    float v;
    asm volatile("ld.global.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ int ld_dep(const int32_t *p) {
    int v;
    asm volatile("ld.global.s32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ float4 ld_dep4(const float *p) {
    float4 v;
    asm volatile("ld.global.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- small device helpers -------------------------------------------------------------------
// Rows 2*blk and 2*blk+1 of M = I - mu Phi^T Phi by a CTA of kGramThreads threads.  M is stored
// row-major with a pitch of 32 * ceil(G / 32) floats, the columns past G zero, so that a recovery
// thread can read its row with aligned 16-byte loads and needs no bounds in its inner loop.
// The values depend on parameters only and are computed at once; the store waits for the kernels
// before this one, which may still be reading the previous layer's matrix.
constexpr int kGramThreads = 256;
inline int gram_blocks(int G) { return (G + 1) / 2; }
__host__ __device__ inline int gram_pitch(int G) { return (G + 31) & ~31; }
__device__ __forceinline__ void gram_rows(const float *__restrict__ Phi, float mu, int m, int G, int blk,
                                          float *__restrict__ gram) {
    const int a = blk * 2 + (threadIdx.x >> 7), b = threadIdx.x & 127;
    const int pitch = gram_pitch(G);
    const bool valid = a < G && b < G;
    float s0 = 0.f, s1 = 0.f;
    if (valid) {
        int i = 0;
        for (; i + 1 < m; i += 2) {
            s0 = fmaf(__ldg(Phi + i * G + a), __ldg(Phi + i * G + b), s0);
            s1 = fmaf(__ldg(Phi + (i + 1) * G + a), __ldg(Phi + (i + 1) * G + b), s1);
        }
        if (i < m) s0 = fmaf(__ldg(Phi + i * G + a), __ldg(Phi + i * G + b), s0);
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (a < G && b < pitch) gram[a * pitch + b] = valid ? (a == b ? 1.f : 0.f) - mu * (s0 + s1) : 0.f;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// 16-byte read-only streaming load (weights are read once per step: keep them out of L1).
__device__ __forceinline__ uint4 ldg_stream(const void *p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// Widen one 16-byte chunk of weights to floats: 8 values for bf16, 4 for f32.
template <typename WT> struct Chunk;
template <> struct Chunk<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static __forceinline__ void widen(const uint4 &q, float (&f)[8]) {
        f[0] = bf16_lo(q.x); f[1] = bf16_hi(q.x); f[2] = bf16_lo(q.y); f[3] = bf16_hi(q.y);
        f[4] = bf16_lo(q.z); f[5] = bf16_hi(q.z); f[6] = bf16_lo(q.w); f[7] = bf16_hi(q.w);
    }
};
template <> struct Chunk<float> {
    static constexpr int kElems = 4;
    __device__ static __forceinline__ void widen(const uint4 &q, float (&f)[4]) {
        f[0] = __uint_as_float(q.x); f[1] = __uint_as_float(q.y);
        f[2] = __uint_as_float(q.z); f[3] = __uint_as_float(q.w);
    }
};

}  // namespace cs
