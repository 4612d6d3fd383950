// Sensor, structured: a subsampled randomized Hadamard operator (Sec. 8, "structured transforms such as
// subsampled randomized Hadamard operators when implementation efficiency is important"):
//
//     y[t, r] = (1 / sqrt(m)) sum_i H[rows[r], i] sign[i] h[t, i],   H[a, i] = (-1)^popcount(a & i),
//
// d a power of two.  Instead of the m x d matrix of the dense sketch (0.5 MB at the 7B shape, read from
// memory by every step) the operator is d sign bits and m row indices, and the transform is the fast
// Walsh-Hadamard butterfly: d log2(d) additions in shared memory, one CTA per token.  Each thread
// first runs the butterflies that stay inside its own run of consecutive elements in registers, the
// remaining stages go through shared memory with one barrier each.
#include "cs_internal.cuh"

namespace cs {

constexpr int kSrhtThreads = 256;

template <int EPT>   // elements per thread, a power of two: d = EPT * kSrhtThreads
__global__ void __launch_bounds__(kSrhtThreads)
srht_kernel(const uint32_t *__restrict__ sign_bits, const int32_t *__restrict__ rows, const float *__restrict__ h,
            int m, float *__restrict__ y) {
    constexpr int d = EPT * kSrhtThreads;
    extern __shared__ float buf[];   // [d]
    const int tid = threadIdx.x, t = blockIdx.x;
    pdl_launch_dependents();
    pdl_wait();   // h may be the kernel before's output
    float v[EPT];
    const int base = tid * EPT;
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        const int i = base + e;
        const float x = ld_dep(h + (size_t)t * d + i);
        v[e] = (sign_bits[i >> 5] >> (i & 31)) & 1u ? -x : x;
    }
    // stages with stride < EPT: inside the thread's own run
#pragma unroll
    for (int len = 1; len < EPT; len <<= 1) {
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            if ((e & len) == 0) {
                const float a = v[e], b = v[e | len];
                v[e] = a + b;
                v[e | len] = a - b;
            }
        }
    }
#pragma unroll
    for (int e = 0; e < EPT; ++e) buf[base + e] = v[e];
    __syncthreads();
    // stages with stride >= EPT: pairs (i, i + len) through shared memory, d / 2 pairs per stage
    for (int len = EPT; len < d; len <<= 1) {
        for (int p = tid; p < d / 2; p += kSrhtThreads) {
            const int i = ((p & ~(len - 1)) << 1) | (p & (len - 1));
            const float a = buf[i], b = buf[i + len];
            buf[i] = a + b;
            buf[i + len] = a - b;
        }
        __syncthreads();
    }
    const float scale = rsqrtf((float)m);
    for (int r = tid; r < m; r += kSrhtThreads) {
        const int a = rows[r];
        y[(size_t)t * m + r] = (unsigned)a < (unsigned)d ? scale * buf[a] : 0.f;   // a row index out of range reads nothing
    }
}

cs_status launch_sketch_srht(cs_plan *plan, const uint32_t *sign_bits, const int32_t *rows, const float *h, int B, float *y,
                             cudaStream_t st) {
    const int d = plan->cfg.d, m = plan->cfg.m;
    StageTimer timer(plan, CS_STAGE_SKETCH, st);
    const size_t smem = (size_t)d * sizeof(float);
#define CS_SRHT_CASE(E)                                                                                       \
    case E * kSrhtThreads:                                                                                    \
        launch_pdl(pdl_for(plan, B), srht_kernel<E>, dim3(B), dim3(kSrhtThreads), smem, st, sign_bits, rows, h, m, y); \
        break
    switch (d) {
        CS_SRHT_CASE(1); CS_SRHT_CASE(2); CS_SRHT_CASE(4); CS_SRHT_CASE(8); CS_SRHT_CASE(16); CS_SRHT_CASE(32);
        default: return CS_ERR_UNSUPPORTED;   // d must be a power of two between 256 and 8192
    }
#undef CS_SRHT_CASE
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

}  // namespace cs
