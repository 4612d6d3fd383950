// Confidence fallback (Sec. 12 online phase: "If the recovery confidence falls below a threshold, the
// system may revert temporarily to a denser support or a fallback kernel"): the confidence of a token's
// recovery is its relative residual ||y - Phi z_T|| / ||y||; tokens above the caller's threshold are
// flagged and listed, and small row movers carry them through a second, denser step.
#include "cs_internal.cuh"

namespace cs {

// One CTA.  flags[t] = resid[t] > tau * ||y_t||  (a NaN residual counts as not trusted); list = the flagged
// tokens in ascending order, *count = their number.
__global__ void __launch_bounds__(1024)
confidence_kernel(const float *__restrict__ y, const float *__restrict__ resid, int B, int m, float tau,
                  int32_t *__restrict__ flags, int32_t *__restrict__ list, int32_t *__restrict__ count) {
    __shared__ int warp_tot[32];
    __shared__ int base_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) base_s = 0;
    __syncthreads();
    for (int t0 = 0; t0 < B; t0 += 1024) {
        const int t = t0 + tid;
        int low = 0;
        if (t < B) {
            float ss = 0.f;
            for (int i = 0; i < m; ++i) { const float v = y[(size_t)t * m + i]; ss = fmaf(v, v, ss); }
            low = !(resid[t] <= tau * sqrtf(ss));
            if (flags != nullptr) flags[t] = low;
        }
        const unsigned bal = __ballot_sync(0xffffffffu, low);
        if (lane == 0) warp_tot[warp] = __popc(bal);
        __syncthreads();
        int off = base_s + __popc(bal & ((1u << lane) - 1u));
        for (int w = 0; w < warp; ++w) off += warp_tot[w];
        if (low) list[off] = t;
        __syncthreads();
        if (tid == 0) { int s = 0; for (int w = 0; w < 32; ++w) s += warp_tot[w]; base_s += s; }
        __syncthreads();
    }
    if (tid == 0) *count = base_s;
}

// dst[i, :] = src[list[i], :]  (gather)  /  dst[list[i], :] = src[i, :]  (scatter); rows of d floats, d a multiple of 4
__global__ void move_rows_kernel(const float *__restrict__ src, const int32_t *__restrict__ list, int d4, int scatter,
                                 float *__restrict__ dst) {
    const int i = blockIdx.y, row = list[i];
    const float4 *s = reinterpret_cast<const float4 *>(src) + (size_t)(scatter ? i : row) * d4;
    float4 *o = reinterpret_cast<float4 *>(dst) + (size_t)(scatter ? row : i) * d4;
    for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < d4; c += gridDim.x * blockDim.x) o[c] = s[c];
}

cs_status launch_confidence(cs_plan *plan, const float *y, const float *resid, int B, float tau, int32_t *flags,
                            int32_t *list, int32_t *count, cudaStream_t st) {
    confidence_kernel<<<1, 1024, 0, st>>>(y, resid, B, plan->cfg.m, tau, flags, list, count);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

static cs_status move_rows(cs_plan *plan, const float *src, const int32_t *list, int n, int scatter, float *dst,
                           cudaStream_t st) {
    const int d4 = plan->cfg.d / 4;
    move_rows_kernel<<<dim3((d4 + 255) / 256, n), 256, 0, st>>>(src, list, d4, scatter, dst);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}
cs_status launch_gather_rows(cs_plan *plan, const float *src, const int32_t *list, int n, float *dst, cudaStream_t st) {
    return move_rows(plan, src, list, n, 0, dst, st);
}
cs_status launch_scatter_rows(cs_plan *plan, const float *src, const int32_t *list, int n, float *dst, cudaStream_t st) {
    return move_rows(plan, src, list, n, 1, dst, st);
}

}  // namespace cs
