// Prompt-level support: the mean hidden state of the prompt (the mean sketch is S applied to it).
//
// hbar[i] = (1/n) sum_t H[t,i], H [n,d] bf16.  Two passes with a fixed summation order:
// column sums over row blocks (coalesced 4-byte loads, one pair of columns per thread), then the
// row-block partials are added in index order and scaled by 1/n.
#include "cs_internal.cuh"

namespace cs {

constexpr int kMeanThreads = 256;

__global__ void __launch_bounds__(kMeanThreads)
colsum_kernel(const __nv_bfloat16 *__restrict__ H, int n, int d, int rows_per_block, float *__restrict__ colsum) {
    const int col2 = blockIdx.x * kMeanThreads + threadIdx.x;  // pair of columns
    if (col2 * 2 >= d) return;
    const int r0 = blockIdx.y * rows_per_block, r1 = min(n, r0 + rows_per_block);
    float s0 = 0.f, s1 = 0.f;
    const uint32_t *src = reinterpret_cast<const uint32_t *>(H) + col2;
    const size_t pitch = (size_t)d / 2;
#pragma unroll 8
    for (int r = r0; r < r1; ++r) {
        const uint32_t u = __ldg(src + (size_t)r * pitch);
        s0 += bf16_lo(u);
        s1 += bf16_hi(u);
    }
    float2 *dst = reinterpret_cast<float2 *>(colsum + (size_t)blockIdx.y * d) + col2;
    *dst = make_float2(s0, s1);
}

__global__ void __launch_bounds__(kMeanThreads)
mean_finish_kernel(const float *__restrict__ colsum, int blocks, int n, int d, float *__restrict__ hbar) {
    const int col = blockIdx.x * kMeanThreads + threadIdx.x;
    if (col >= d) return;
    float s = 0.f;
    for (int b = 0; b < blocks; ++b) s += colsum[(size_t)b * d + col];
    hbar[col] = s / (float)n;
}

cs_status launch_prompt_mean(cs_plan *plan, const void *H, int n, float *hbar, cudaStream_t st) {
    const int d = plan->cfg.d;
    const int blocks = min(plan->mean_row_blocks, n);
    const int rpb = (n + blocks - 1) / blocks;
    const int used = (n + rpb - 1) / rpb;
    dim3 grid((d / 2 + kMeanThreads - 1) / kMeanThreads, used);
    colsum_kernel<<<grid, kMeanThreads, 0, st>>>(static_cast<const __nv_bfloat16 *>(H), n, d, rpb, plan->colsum);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    mean_finish_kernel<<<(d + kMeanThreads - 1) / kMeanThreads, kMeanThreads, 0, st>>>(plan->colsum, used, n, d, hbar);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

}  // namespace cs
