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
#include "cs_internal.cuh"

namespace cs {

constexpr int kSketchThreads = 256;
constexpr int kSketchMaxRows = 16;

template <int CPT>
__global__ void __launch_bounds__(kSketchThreads)
sketch_kernel(const float *__restrict__ S, const float *__restrict__ x, const float *__restrict__ gamma,
              float eps, int m, int d, int rows_per_cta, float *__restrict__ y, float *__restrict__ n_out,
              int sketch_blocks, const float *__restrict__ Phi, float mu, int G, float *__restrict__ gram) {
    __shared__ float red[kSketchMaxRows + 1][kSketchThreads / 32];
    __shared__ float total[kSketchMaxRows + 1];
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
    pdl_launch_dependents();
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
}

static_assert(kGramThreads == kSketchThreads, "the spare CTAs of the sketch launch form the Gram rows");

cs_status launch_sketch(cs_plan *plan, const float *S, const float *x, const float *gamma, int B,
                        float *y, float *n_out, const float *Phi, float mu, cudaStream_t st) {
    const cs_config &c = plan->cfg;
    StageTimer timer(plan, CS_STAGE_SKETCH, st);
    // Enough CTAs to cover the SMs about twice, at most kSketchMaxRows rows per CTA.
    int rpc = (c.m * B + 2 * plan->sm_count - 1) / (2 * plan->sm_count);
    rpc = max(1, min(rpc, min(c.m, kSketchMaxRows)));
    const int sblocks = (c.m + rpc - 1) / rpc;
    dim3 grid(sblocks + (Phi != nullptr ? gram_blocks(plan->G) : 0), B);
    const int cpt = (c.d / 4 + kSketchThreads - 1) / kSketchThreads;
#define CS_SKETCH_CASE(N)                                                                            \
    launch_pdl(pdl_for(plan, B), sketch_kernel<N>, grid, dim3(kSketchThreads), 0, st, S, x, gamma, c.rms_eps, c.m, c.d, rpc, y, n_out, sblocks, Phi, mu, plan->G, plan->gram)
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
