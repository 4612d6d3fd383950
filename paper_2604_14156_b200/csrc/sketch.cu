// Sensor: y = S n, with the optional RMSNorm of the stacked workload folded in.
//
// y[t,r] = sum_i S[r,i] n[t,i],  n = x * rsqrt(mean(x^2) + eps) * gamma  (or n = x).
// Since the normalisation is one scalar per token, y = rscale * (S (x .* gamma)) and the sum of
// squares is taken in the same pass over x.
//
// Grid (row blocks, tokens).  All threads of a CTA cooperate on every row of its row block: a
// thread owns the float4 chunks tid, tid+256, ... of the row, keeps the matching x chunks in
// registers, and the per-row partial sums are folded by warp shuffles and one shared-memory hop.
// With one token the grid is m CTAs of one row each, so the m*d*4 bytes of S are pulled by m SMs
// at once; with a decode batch a CTA takes several rows per token.  When the recovery follows, a few
// extra CTAs of the same launch form its matrix I - mu Phi^T Phi, which needs the parameters only.
//
// RECOVER (the small-batch step): the recovery runs in this launch too.  Every CTA draws a ticket
// when its rows of y are in memory, and the CTA of a token that draws the last one runs the
// iteration (recover_core.cuh) on four of its warps, with I - mu Phi^T Phi in shared memory (every CTA
// forms it from a copy of Phi before the wait for the kernel ahead: parameters only), so that the
// iteration issues no global load while the actuator saturates the memory system.  Nothing waits for anything: the other CTAs are gone by then.  The launch's
// programmatic trigger is held back until the slot table of the FIRST iterate is in global memory;
// the actuator's kernel starts on it and takes the final table when this kernel has completed.
#include "recover_core.cuh"

namespace cs {

constexpr int kSketchThreads = 256;
constexpr int kSketchMaxRows = 16;
constexpr int kSketchRecNW = 4, kSketchRecKC = 4;     // recovery in this launch: G <= 128, k <= 32
// dynamic shared memory: Phi transposed [G][32] (16 KB at most) and the hand-over array of the first fill
// [32 slots][128] (16 KB); the size also keeps an actuator CTA off the recovery's SM
constexpr int kSketchRecSmem = (16 + 16) * 1024;

struct SketchRecoverArgs {
    float mu;
    int G, k, T;
    int32_t *table;       // [B, kSlotTablePitch] slot -> group of the current iterate
    unsigned *ticket;     // [B], zero between launches
    int32_t *support;     // [B, k] ascending (may be NULL)
    float *z, *resid;     // [B, k], [B] (may be NULL)
    DeviceStatus *status;
};

__device__ __forceinline__ void st_visible(int32_t *p, int v) {
    asm volatile("st.volatile.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Ticket: the release half orders this CTA's stores (made before the barrier that precedes the call)
// ahead of the increment, the acquire half orders the last CTA's loads behind it.
__device__ __forceinline__ unsigned ticket_draw(unsigned *p) {
    unsigned old;
    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(old) : "l"(p) : "memory");
    return old;
}

template <int CPT, bool RECOVER>
__global__ void __launch_bounds__(kSketchThreads, 2)
sketch_kernel(const float *__restrict__ S, const float *__restrict__ x, const float *__restrict__ gamma,
              float eps, int m, int d, int rows_per_cta, float *__restrict__ y, float *__restrict__ n_out,
              int sketch_blocks, const float *__restrict__ Phi, float mu, int G, float *__restrict__ gram,
              SketchRecoverArgs ra) {
    __shared__ float red[kSketchMaxRows + 1][kSketchThreads / 32];
    __shared__ float total[kSketchMaxRows + 1];
    extern __shared__ float4 phiT_s[];   // RECOVER: Phi transposed, [G][8] float4 (32 rows, those past m zero)
    if ((int)blockIdx.x >= sketch_blocks) {   // spare CTAs: the recovery's matrix for this layer
        pdl_launch_dependents();
        if (blockIdx.y == 0) gram_rows(Phi, mu, m, G, blockIdx.x - sketch_blocks, gram);
        return;
    }
    const int t = blockIdx.y;
    const int r0 = blockIdx.x * rows_per_cta;
    const int nrows = min(rows_per_cta, m - r0);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunks = d >> 2;
    if constexpr (!RECOVER) pdl_launch_dependents();
    if constexpr (RECOVER) {   // Phi is a parameter: every CTA copies it before the wait, one of them will use it
        float *pt = reinterpret_cast<float *>(phiT_s);
        // coalesced reads of Phi (four in flight per thread), transposed writes
        for (int i0 = tid; i0 < 32 * G; i0 += 4 * kSketchThreads) {
            float v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * kSketchThreads;
                v[u] = i < m * G ? __ldg(Phi + i) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * kSketchThreads;
                if (i < 32 * G) { const int row = i / G; pt[(i - row * G) * 32 + row] = v[u]; }
            }
        }
    }
    float phc[32];   // RECOVER: column (tid mod 128) of Phi
    if constexpr (RECOVER) {
        recover_load_phi<kSketchRecNW>(Phi, m, G, tid & (32 * kSketchRecNW - 1), phc);
    }
    // S is a parameter: with a single row per CTA (small batches) its chunks are requested before the
    // wait for the kernel that produces x, which takes the DRAM latency of S off the chain.
    const bool early = nrows == 1;
    float4 s0[CPT];
    if (early) {
        const float4 *row = reinterpret_cast<const float4 *>(S + (size_t)r0 * d);
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
            const int c = tid + j * kSketchThreads;
            s0[j] = c < chunks ? __ldg(row + c) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
    pdl_wait();   // x may be the previous kernel's output

    float4 xv[CPT];
    float ss = 0.f;
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
        const int c = tid + j * kSketchThreads;
        xv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < chunks) {
            xv[j] = ld_dep4(x + (size_t)t * d + 4 * (size_t)c);
            ss += xv[j].x * xv[j].x + xv[j].y * xv[j].y + xv[j].z * xv[j].z + xv[j].w * xv[j].w;
            if (gamma != nullptr) {
                const float4 g = reinterpret_cast<const float4 *>(gamma)[c];
                xv[j].x *= g.x; xv[j].y *= g.y; xv[j].z *= g.z; xv[j].w *= g.w;
            }
        }
    }
    for (int r = 0; r < nrows; ++r) {
        const float4 *row = reinterpret_cast<const float4 *>(S + (size_t)(r0 + r) * d);
        float acc = 0.f;
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
            const int c = tid + j * kSketchThreads;
            if (c < chunks) {
                const float4 s = early ? s0[j] : __ldg(row + c);
                acc = fmaf(s.x, xv[j].x, acc); acc = fmaf(s.y, xv[j].y, acc);
                acc = fmaf(s.z, xv[j].z, acc); acc = fmaf(s.w, xv[j].w, acc);
            }
        }
        acc = warp_sum(acc);
        if (lane == 0) red[r][warp] = acc;
    }
    ss = warp_sum(ss);
    if (lane == 0) red[kSketchMaxRows][warp] = ss;
    __syncthreads();
    if (tid <= kSketchMaxRows && (tid < nrows || tid == kSketchMaxRows)) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kSketchThreads / 32; ++w) s += red[tid][w];
        total[tid] = s;
    }
    __syncthreads();
    const float rscale = (gamma != nullptr) ? rsqrtf(total[kSketchMaxRows] / (float)d + eps) : 1.f;
    if (tid < nrows) y[(size_t)t * m + r0 + tid] = total[tid] * rscale;
    if (n_out != nullptr && blockIdx.x == 0) {
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
            const int c = tid + j * kSketchThreads;
            if (c < chunks) {
                float4 v = xv[j];
                v.x *= rscale; v.y *= rscale; v.z *= rscale; v.w *= rscale;
                reinterpret_cast<float4 *>(n_out + (size_t)t * d)[c] = v;
            }
        }
    }
    if constexpr (RECOVER) {
        __shared__ int last_s;
        int32_t *table = ra.table + (size_t)t * kSlotTablePitch;
        if (blockIdx.x == 0 && tid == 0) st_visible(table + kSlotTableSlots, 0);   // this step's table is not final yet
        __syncthreads();   // this CTA's rows of y (and n) are written ...
        if (tid == 0) last_s = ticket_draw(ra.ticket + t) == (unsigned)(sketch_blocks - 1);   // ... before its ticket is drawn
        __syncthreads();
        if (!last_s) return;                   // a CTA that has exited counts as having triggered
        if (tid == 0) ra.ticket[t] = 0u;       // for the next launch
        typedef PhiSource<5, 6, kSketchThreads> Source;
        const Source src{phiT_s, mu, reinterpret_cast<float *>(phiT_s) + 32 * kMaxG};
        __shared__ RecoverSmem<kSketchRecNW, kSketchRecKC> rs;
        if (tid >= 32 * kSketchRecNW) {   // helpers of the first fill (recover_core.cuh), then gone
            const int b = tid - 32 * kSketchRecNW;
            if (ra.T > 0) src.help(rs.idx, ra.k, b, b < G ? b : 0, phc);
            return;
        }
        const int g = tid;
        const int k = ra.k;
        recover_token<kSketchRecNW, kSketchRecKC, 1>(
            rs, g, Phi, src, mu, y + (size_t)t * m, m, G, k, ra.T,
            ra.support != nullptr ? ra.support + (size_t)t * k : nullptr, ra.z != nullptr ? ra.z + (size_t)t * k : nullptr,
            ra.resid != nullptr ? ra.resid + t : nullptr, nullptr, nullptr, 0.f, nullptr, nullptr, ra.status, phc,
            [&] {   // the first iterate's table goes out, then the launch's trigger
                if (g < k) st_visible(table + g, rs.idx[g]);
                __threadfence();
                bar_sync<1, 32 * kSketchRecNW>();
                if (g == 0) pdl_launch_dependents();
            },
            [&](int slot, int entry) { st_visible(table + slot, entry); },
            [&] {   // the table is final: say so (the actuator need not wait for the outputs below)
                __threadfence();
                bar_sync<1, 32 * kSketchRecNW>();
                if (g == 0) st_visible(table + kSlotTableSlots, 1);
            });
    }
}

static_assert(kGramThreads == kSketchThreads, "the spare CTAs of the sketch launch form the Gram rows");
static_assert(8 * kSketchRecKC == kSlotTableSlots, "one table row holds the list form's slots");

// Rows per CTA: enough CTAs to cover the SMs about twice, at most kSketchMaxRows rows per CTA.
static int sketch_rows_per_cta(const cs_plan *plan, int B) {
    const int rpc = (plan->cfg.m * B + 2 * plan->sm_count - 1) / (2 * plan->sm_count);
    return max(1, min(rpc, min(plan->cfg.m, kSketchMaxRows)));
}

cs_status launch_sketch(cs_plan *plan, const float *S, const float *x, const float *gamma, int B,
                        float *y, float *n_out, const float *Phi, float mu, cudaStream_t st) {
    const cs_config &c = plan->cfg;
    StageTimer timer(plan, CS_STAGE_SKETCH, st);
    const int rpc = sketch_rows_per_cta(plan, B);
    const int sblocks = (c.m + rpc - 1) / rpc;
    dim3 grid(sblocks + (Phi != nullptr ? gram_blocks(plan->G) : 0), B);
    const int cpt = (c.d / 4 + kSketchThreads - 1) / kSketchThreads;
#define CS_SKETCH_CASE(N)                                                                            \
    launch_pdl(pdl_for(plan, B), sketch_kernel<N, false>, grid, dim3(kSketchThreads), 0, st, S, x, gamma, c.rms_eps, c.m, c.d, rpc, y, n_out, sblocks, Phi, mu, plan->G, plan->gram, SketchRecoverArgs{})
    if (cpt <= 1) CS_SKETCH_CASE(1);
    else if (cpt <= 2) CS_SKETCH_CASE(2);
    else if (cpt <= 4) CS_SKETCH_CASE(4);
    else CS_SKETCH_CASE(8);
#undef CS_SKETCH_CASE
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

bool sketch_recover_ok(const cs_plan *plan) {
    return plan->cfg.k <= 8 * kSketchRecKC && plan->G <= 32 * kSketchRecNW && plan->cfg.m <= 32;
}

cs_status prepare_sketch(cs_plan *plan) {
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(sketch_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSketchRecSmem));
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(sketch_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSketchRecSmem));
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(sketch_kernel<4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSketchRecSmem));
    CS_CUDA_TRY(plan, cudaFuncSetAttribute(sketch_kernel<8, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSketchRecSmem));
    return CS_OK;
}

// Sketch and recovery in one launch (see the head of this file).  Writes y, the slot tables
// (plan->slot_table) and, when the kernel has completed, support / z / resid.
cs_status launch_sketch_recover(cs_plan *plan, const cs_layer *L, const float *x, int B, float *y, float *n_out,
                                int32_t *support, float *z, float *resid, cudaStream_t st) {
    const cs_config &c = plan->cfg;
    StageTimer timer(plan, CS_STAGE_SKETCH, st);
    const int rpc = sketch_rows_per_cta(plan, B);
    const int sblocks = (c.m + rpc - 1) / rpc;
    dim3 grid(sblocks, B);
    const int cpt = (c.d / 4 + kSketchThreads - 1) / kSketchThreads;
    SketchRecoverArgs ra;
    ra.mu = L->mu; ra.G = plan->G; ra.k = c.k; ra.T = c.T;
    ra.table = plan->slot_table; ra.ticket = plan->ticket;
    ra.support = support; ra.z = z; ra.resid = resid; ra.status = plan->status;
#define CS_SKETCH_CASE(N)                                                                            \
    launch_pdl(true, sketch_kernel<N, true>, grid, dim3(kSketchThreads), kSketchRecSmem, st, L->S, x, L->rms_gamma, c.rms_eps, c.m, c.d, rpc, y, n_out, sblocks, L->Phi, L->mu, plan->G, (float *)nullptr, ra)
    if (cpt <= 1) CS_SKETCH_CASE(1);
    else if (cpt <= 2) CS_SKETCH_CASE(2);
    else if (cpt <= 4) CS_SKETCH_CASE(4);
    else CS_SKETCH_CASE(8);
#undef CS_SKETCH_CASE
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

}  // namespace cs
