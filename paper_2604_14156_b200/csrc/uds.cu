// Uncertainty-driven sensing controller (Sec. 8.1): the predictive entropy of the previous step's
// distribution over the vocabulary, H = -sum_v p_v log p_v with p = softmax(logits), and the
// measurement budget it sets, m = clip(floor(m_base (1 + gamma H)), m_min, m_max).
//
// One pass over the logits.  Every thread keeps the three moments of its elements
//     M = max l,   Z = sum e^(l - M),   W = sum e^(l - M) (l - M),
// which merge associatively under a change of M, so the row is split over several CTAs (a single
// token still uses a good part of the GPU) and folded in a fixed order: per warp by shuffles, per
// CTA through shared memory, per row by a second small kernel, which ends with
//     H = log Z - W / Z.
// Bandwidth-bound: 4 V bytes per token, read once.
#include "cs_internal.cuh"

namespace cs {

constexpr int kUdsThreads = 512;
constexpr int kUdsMaxSplits = 32;
constexpr int kUdsBatch = 8;
constexpr int kUdsMinSplitElems = kUdsBatch * kUdsThreads;

struct Moments { float M, Z, W; };   // Z == 0: no element yet

__device__ __forceinline__ Moments merge(const Moments &a, const Moments &b) {
    if (b.Z == 0.f) return a;
    if (a.Z == 0.f) return b;
    const float M = fmaxf(a.M, b.M);
    const float da = a.M - M, db = b.M - M;       // one of them is exactly 0
    const float sa = expf(da), sb = expf(db);
    Moments r;
    r.M = M;
    r.Z = sa * a.Z + sb * b.Z;
    r.W = sa * (a.W + da * a.Z) + sb * (b.W + db * b.Z);
    return r;
}

// Folds a batch of N elements: one rescale to the batch maximum, then N independent exponentials.
// Entries of -inf contribute nothing (p = 0, 0 log 0 = 0).
template <int N>
__device__ __forceinline__ void add_logits(Moments &s, const float (&v)[N]) {
    float m = v[0];
#pragma unroll
    for (int j = 1; j < N; ++j) m = fmaxf(m, v[j]);
    if (m == -INFINITY) return;
    if (s.Z == 0.f) {
        s.M = m;
    } else if (m > s.M) {                         // new maximum: rescale what has been summed
        const float dm = s.M - m, sc = expf(dm);
        s.W = sc > 0.f ? sc * (s.W + dm * s.Z) : 0.f;
        s.Z = sc * s.Z;
        s.M = m;
    }
    float z0 = 0.f, z1 = 0.f, w0 = 0.f, w1 = 0.f;
#pragma unroll
    for (int j = 0; j < N; j += 2) {
        const float d0 = v[j] - s.M, d1 = v[j + 1] - s.M;
        const float e0 = __expf(d0), e1 = __expf(d1);   // d <= 0: the fast exponential's error (about
                                                        // 1e-7 |d| relative) is far inside the 1e-5 asked of H
        z0 += e0; z1 += e1;
        w0 += e0 > 0.f ? e0 * d0 : 0.f;           // e = 0 (underflow, or a -inf entry): no term
        w1 += e1 > 0.f ? e1 * d1 : 0.f;
    }
    s.Z += z0 + z1;
    s.W += w0 + w1;
}

__device__ __forceinline__ Moments warp_merge(Moments s) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Moments other;
        other.M = __shfl_xor_sync(0xffffffffu, s.M, o);
        other.Z = __shfl_xor_sync(0xffffffffu, s.Z, o);
        other.W = __shfl_xor_sync(0xffffffffu, s.W, o);
        // the lower lane's value goes first on both sides, so all lanes end with the same bits
        s = (threadIdx.x & o) ? merge(other, s) : merge(s, other);
    }
    return s;
}

// grid (splits, B): CTA (s, t) folds elements [s * per, min(V, (s + 1) * per)) of row t.
__global__ void __launch_bounds__(kUdsThreads)
uds_moments_kernel(const float *__restrict__ logits, int V, int per, Moments *__restrict__ part) {
    __shared__ Moments ws[kUdsThreads / 32];
    const int t = blockIdx.y, s = blockIdx.x;
    const int lo = s * per, hi = min(V, lo + per);
    const float *row = logits + (size_t)t * V;
    Moments acc{0.f, 0.f, 0.f};
    pdl_launch_dependents();
    // kUdsBatch loads in flight per thread before any of them is used
    for (int i = lo + threadIdx.x; i < hi; i += kUdsBatch * kUdsThreads) {
        float v[kUdsBatch];
#pragma unroll
        for (int j = 0; j < kUdsBatch; ++j) {
            const int idx = i + j * kUdsThreads;
            v[j] = idx < hi ? __ldg(row + idx) : -INFINITY;
        }
        add_logits(acc, v);
    }
    acc = warp_merge(acc);
    if ((threadIdx.x & 31) == 0) ws[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x < 32) {
        Moments v = threadIdx.x < kUdsThreads / 32 ? ws[threadIdx.x] : Moments{0.f, 0.f, 0.f};
        v = warp_merge(v);
        if (threadIdx.x == 0) part[(size_t)t * gridDim.x + s] = v;
    }
}

// One warp per token: folds the splits, then the entropy and the budget.  The floor is taken in
// double precision from the f32 entropy; a NaN entropy (a NaN or +inf logit) asks for m_max.
__global__ void __launch_bounds__(32)
uds_finish_kernel(const Moments *__restrict__ part, int splits, float m_base, float gamma, int m_min, int m_max,
                  float *__restrict__ H_out, int32_t *__restrict__ m_out) {
    const int t = blockIdx.x, lane = threadIdx.x;
    pdl_wait();   // the moments come from the kernel before
    Moments v{0.f, 0.f, 0.f};
    if (lane < splits) {
        const float *p = reinterpret_cast<const float *>(part + (size_t)t * splits + lane);
        v.M = ld_dep(p); v.Z = ld_dep(p + 1); v.W = ld_dep(p + 2);
    }
    v = warp_merge(v);
    if (lane == 0) {
        float H = v.Z > 0.f ? fmaxf(logf(v.Z) - v.W / v.Z, 0.f) : (v.Z == 0.f ? 0.f : v.Z);
        if (v.Z != v.Z || v.W != v.W) H = NAN;
        int m = m_max;
        if (H == H) {
            const double x = floor((double)m_base * (1.0 + (double)gamma * (double)H));
            m = x >= (double)m_max ? m_max : (x <= (double)m_min ? m_min : (int)x);
        }
        if (H_out != nullptr) H_out[t] = H;
        m_out[t] = m;
    }
}

cs_status launch_uds_budget(cs_plan *plan, const float *logits, int B, int V, float m_base, float gamma,
                            int m_min, int m_max, float *H, int32_t *m_t, cudaStream_t st) {
    int splits = (2 * plan->sm_count + B - 1) / B;   // about two CTAs per SM
    splits = max(1, min(splits, min(kUdsMaxSplits, V / kUdsMinSplitElems)));
    const size_t capacity = (size_t)kGatherMaxTokens * plan->nx_max * plan->cfg.d * sizeof(float);
    while (splits > 1 && (size_t)B * splits * sizeof(Moments) > capacity) --splits;
    if ((size_t)B * splits * sizeof(Moments) > capacity) return CS_ERR_SHAPE;
    const int per = (V + splits - 1) / splits;
    Moments *part = reinterpret_cast<Moments *>(plan->partial);
    uds_moments_kernel<<<dim3(splits, B), kUdsThreads, 0, st>>>(logits, V, per, part);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    launch_pdl(true, uds_finish_kernel, dim3(B), dim3(32), 0, st, (const Moments *)part, splits, m_base, gamma, m_min, m_max, H, m_t);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

}  // namespace cs
