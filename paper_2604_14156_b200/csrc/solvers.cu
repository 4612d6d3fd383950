// Estimators beside the fixed-step iteration (Sec. 8 lists them: "orthogonal matching pursuit over a
// constrained support dictionary", "projected proximal methods with a small fixed number of
// iterations"), one CTA of 128 threads per token, thread g owning entry g:
//
//   normalised step:  g = Phi^T (y - Phi z);  S = supp(z) (the k largest |g| when z = 0);
//                     mu_t = ||g_S||^2 / ||Phi g_S||^2 (the caller's mu when the denominator is 0);
//                     z = H_k(z + mu_t g).                    No line search follows the step.
//   matching pursuit: k times: the group whose normalised column correlates most with the residual
//                     joins the support (ties: lowest index), then z_S = argmin ||y - Phi_S z|| through an
//                     orthonormal basis Q of the chosen columns (Gram-Schmidt, applied twice) and the
//                     triangular factor R, Phi_S = Q R.
//
// Both are written for clarity, not for the last microsecond: they are the estimators a caller turns
// to when the fixed step does not recover enough, and neither is on the decode step's default path.
// Phi (at most 64 x 128 floats) sits in shared memory; every choice between groups uses the total
// order (value descending, index ascending) by exact rank counting, as the fixed-step kernel does.
#include "cs_internal.cuh"

namespace cs {

namespace {

constexpr int kSolverThreads = kMaxG;   // one thread per group
constexpr int kOmpMaxK = 64;

struct Reduce {
    float part[kSolverThreads / 32];
};
// Sum over the CTA (every thread gets it); two barriers.
__device__ __forceinline__ float block_sum(float v, Reduce &r) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) r.part[threadIdx.x >> 5] = v;
    __syncthreads();
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kSolverThreads / 32; ++w) s += r.part[w];
    return s;
}

// Number of entries that precede entry g in the order (key descending, index ascending); key_s holds
// every thread's key (entries past G: -1, they precede nothing and nothing real ties with them).
__device__ __forceinline__ int rank_of(const float *key_s, int G, int g) {
    const float mine = key_s[g];
    int rank = 0;
    for (int j = 0; j < G; ++j) {
        const float o = key_s[j];
        rank += (o > mine) || (o == mine && j < g);
    }
    return rank;
}
__device__ __forceinline__ float abs_key(float v) {   // |v|, a NaN ranked as a zero
    const uint32_t b = __float_as_uint(v) & 0x7fffffffu;
    return b > 0x7f800000u ? 0.f : __uint_as_float(b);
}

// Writes the kept entries in ascending index order: support[o] = g, z[o] = value.
__device__ __forceinline__ void write_ascending(bool kept, float value, int g, int k, int32_t *support, float *z,
                                                int *cnt_s) {
    const int lane = g & 31, warp = g >> 5;
    const unsigned kb = __ballot_sync(0xffffffffu, kept);
    __syncthreads();
    if (lane == 0) cnt_s[warp] = __popc(kb);
    __syncthreads();
    if (kept) {
        int o = __popc(kb & ((1u << lane) - 1u));
        for (int w = 0; w < warp; ++w) o += cnt_s[w];
        if (o < k) {
            support[o] = g;
            if (z != nullptr) z[o] = value;
        }
    }
}

}  // namespace

// ---- normalised step -------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSolverThreads)
niht_kernel(const float *__restrict__ Phi, float mu_fallback, const float *__restrict__ y, int m, int G, int k, int T,
            int32_t *__restrict__ support, float *__restrict__ z_out, float *__restrict__ resid_out, DeviceStatus *status) {
    __shared__ float phi_s[kMaxM * kMaxG];
    __shared__ float key_s[kSolverThreads], vec_s[kSolverThreads], r_s[kMaxM];
    __shared__ int cnt_s[kSolverThreads / 32];
    __shared__ Reduce red;
    const int g = threadIdx.x, t = blockIdx.x;
    const bool valid = g < G;
    for (int i = g; i < m * G; i += kSolverThreads) phi_s[i] = Phi[i];
    if (g < m) r_s[g] = y[(size_t)t * m + g];   // z = 0: r = y
    bool kept = g < k;                          // what the order gives an all-zero vector
    float z = 0.f;
    __syncthreads();
    for (int it = 0; it < T; ++it) {
        float grad = 0.f;
        if (valid)
            for (int i = 0; i < m; ++i) grad = fmaf(phi_s[i * G + g], r_s[i], grad);
        if (it == 0) {   // z = 0 has no support of its own yet: the k entries H_k keeps of the gradient
            key_s[g] = valid ? abs_key(grad) : -1.f;
            __syncthreads();
            kept = valid && rank_of(key_s, G, g) < k;
        }
        vec_s[g] = kept ? grad : 0.f;           // g_S
        const float num = block_sum(kept ? grad * grad : 0.f, red);   // (its barriers also publish vec_s)
        float pg = 0.f;                          // row g of Phi g_S
        if (g < m)
            for (int j = 0; j < G; ++j) pg = fmaf(phi_s[g * G + j], vec_s[j], pg);
        const float den = block_sum(g < m ? pg * pg : 0.f, red);
        const float mu_t = den > 0.f ? num / den : mu_fallback;
        const float v = fmaf(mu_t, grad, z);
        key_s[g] = valid ? abs_key(v) : -1.f;
        __syncthreads();
        kept = valid && rank_of(key_s, G, g) < k;
        z = kept ? v : 0.f;
        vec_s[g] = z;
        __syncthreads();
        if (g < m) {                             // r = y - Phi z
            float a = 0.f;
            for (int j = 0; j < G; ++j) a = fmaf(phi_s[g * G + j], vec_s[j], a);
            r_s[g] = y[(size_t)t * m + g] - a;
        }
        __syncthreads();
    }
    const float rr = block_sum(g < m ? r_s[g] * r_s[g] : 0.f, red);
    if (g == 0 && resid_out != nullptr) resid_out[t] = sqrtf(rr);
    if (valid && T > 0 && !(fabsf(z) <= 3.402823466e38f)) atomicCAS(&status->code, 0, (int)CS_ERR_NONFINITE);
    write_ascending(kept, z, g, k, support + (size_t)t * k, z_out != nullptr ? z_out + (size_t)t * k : nullptr, cnt_s);
}

// ---- orthogonal matching pursuit ----------------------------------------------------------------------
// Dynamic shared memory: Phi [m][G], Q [k][m], R [k][k].  A column whose norm after the two
// orthogonalisation passes is below 1e-5 of its own (float32: an exact duplicate leaves about 1e-7)
// lies in the span of the columns chosen before it and enters with coefficient 0.
constexpr float kOmpDependent = 1e-5f;

__global__ void __launch_bounds__(kSolverThreads)
omp_kernel(const float *__restrict__ Phi, const float *__restrict__ y, int m, int G, int k,
           int32_t *__restrict__ support, float *__restrict__ z_out, float *__restrict__ resid_out, DeviceStatus *status) {
    extern __shared__ float smem[];
    float *phi_s = smem, *Q = phi_s + m * G, *R = Q + k * m;
    __shared__ float key_s[kSolverThreads], r_s[kMaxM], col_s[kMaxM], y_s[kMaxM], dot_s[kOmpMaxK], qty_s[kOmpMaxK], coef_s[kOmpMaxK];
    __shared__ int live_s[kOmpMaxK], cnt_s[kSolverThreads / 32], pick_s;
    __shared__ Reduce red;
    const int g = threadIdx.x, t = blockIdx.x;
    const bool valid = g < G;
    for (int i = g; i < m * G; i += kSolverThreads) phi_s[i] = Phi[i];
    for (int i = g; i < k * k; i += kSolverThreads) R[i] = 0.f;
    if (g < m) { y_s[g] = y[(size_t)t * m + g]; r_s[g] = y_s[g]; }
    if (g < k) { live_s[g] = 0; qty_s[g] = 0.f; coef_s[g] = 0.f; }
    __syncthreads();
    float cn = 0.f;   // norm of this thread's column
    if (valid) {
        for (int i = 0; i < m; ++i) cn = fmaf(phi_s[i * G + g], phi_s[i * G + g], cn);
        cn = sqrtf(cn);
    }
    bool in = false;
    int my_pick = -1;   // the step at which this thread's group joined
    for (int s = 0; s < k; ++s) {
        // the candidate that comes first in the order (normalised correlation descending, index ascending)
        float c = -1.f;
        if (valid && !in && cn > 0.f) {
            float a = 0.f;
            for (int i = 0; i < m; ++i) a = fmaf(phi_s[i * G + g], r_s[i], a);
            c = abs_key(a) / cn;
        }
        key_s[g] = c;
        if (g == 0) pick_s = -1;
        __syncthreads();
        if (c > 0.f && rank_of(key_s, G, g) == 0) pick_s = g;
        __syncthreads();
        if (pick_s < 0) {   // nothing correlates: the lowest unused index joins with coefficient 0
            key_s[g] = (valid && !in) ? (float)(kMaxG - g) : -1.f;
            __syncthreads();
            if (valid && !in && rank_of(key_s, G, g) == 0) pick_s = g;
            __syncthreads();
            if (pick_s == g) { in = true; my_pick = s; }
            __syncthreads();
            continue;
        }
        const int j = pick_s;
        if (j == g) { in = true; my_pick = s; }
        if (g < m) col_s[g] = phi_s[g * G + j];
        __syncthreads();
        const float cnj = sqrtf(block_sum(g < m ? col_s[g] * col_s[g] : 0.f, red));
        for (int pass = 0; pass < 2; ++pass) {   // orthogonalise against the basis, twice
            if (g < s) {
                float d = 0.f;
                if (live_s[g])
                    for (int i = 0; i < m; ++i) d = fmaf(Q[g * m + i], col_s[i], d);
                dot_s[g] = d;
                R[g * k + s] += d;
            }
            __syncthreads();
            if (g < m) {
                float sub = 0.f;
                for (int a = 0; a < s; ++a) sub = fmaf(dot_s[a], Q[a * m + g], sub);
                col_s[g] -= sub;
            }
            __syncthreads();
        }
        const float nn = sqrtf(block_sum(g < m ? col_s[g] * col_s[g] : 0.f, red));
        if (nn > kOmpDependent * cnj) {
            if (g < m) Q[s * m + g] = col_s[g] / nn;
            const float qy = block_sum(g < m ? (col_s[g] / nn) * y_s[g] : 0.f, red);
            if (g == 0) { live_s[s] = 1; R[s * k + s] = nn; qty_s[s] = qy; }
            __syncthreads();
            if (g < m) {                         // r = y - Q Q^T y over the basis so far
                float a = y_s[g];
                for (int b = 0; b <= s; ++b)
                    if (live_s[b]) a -= qty_s[b] * Q[b * m + g];
                r_s[g] = a;
            }
        }
        __syncthreads();
    }
    // z_S = R^{-1} Q^T y by back substitution (first warp: lanes stride over the later picks)
    if (g < 32) {
        for (int s = k - 1; s >= 0; --s) {
            float acc = 0.f;
            for (int b = s + 1 + g; b < k; b += 32)
                if (live_s[b]) acc = fmaf(R[s * k + b], coef_s[b], acc);
            acc = warp_sum(acc);
            if (g == 0 && live_s[s]) coef_s[s] = (qty_s[s] - acc) / R[s * k + s];
            __syncwarp();
        }
    }
    __syncthreads();
    const float zg = in && my_pick >= 0 ? coef_s[my_pick] : 0.f;
    const float rr = block_sum(g < m ? r_s[g] * r_s[g] : 0.f, red);
    if (g == 0 && resid_out != nullptr) resid_out[t] = sqrtf(rr);
    if (in && !(fabsf(zg) <= 3.402823466e38f)) atomicCAS(&status->code, 0, (int)CS_ERR_NONFINITE);
    write_ascending(in, zg, g, k, support + (size_t)t * k, z_out != nullptr ? z_out + (size_t)t * k : nullptr, cnt_s);
}

static size_t omp_smem(int m, int G, int k) { return ((size_t)m * G + (size_t)k * m + (size_t)k * k) * sizeof(float); }

cs_status prepare_solvers(cs_plan *plan) {
    const cs_config &c = plan->cfg;
    if (c.k <= kOmpMaxK)
        CS_CUDA_TRY(plan, cudaFuncSetAttribute(omp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               (int)omp_smem(c.m, plan->G, c.k)));
    return CS_OK;
}

cs_status launch_niht(cs_plan *plan, const float *Phi, float mu_fallback, const float *y, int B, int T,
                      int32_t *support, float *z, float *resid, cudaStream_t st) {
    StageTimer timer(plan, CS_STAGE_RECOVER, st);
    niht_kernel<<<B, kSolverThreads, 0, st>>>(Phi, mu_fallback, y, plan->cfg.m, plan->G, plan->cfg.k, T, support, z, resid,
                                              plan->status);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

cs_status launch_omp(cs_plan *plan, const float *Phi, const float *y, int B, int32_t *support, float *z, float *resid,
                     cudaStream_t st) {
    if (plan->cfg.k > kOmpMaxK) return CS_ERR_UNSUPPORTED;
    StageTimer timer(plan, CS_STAGE_RECOVER, st);
    omp_kernel<<<B, kSolverThreads, omp_smem(plan->cfg.m, plan->G, plan->cfg.k), st>>>(
        Phi, y, plan->cfg.m, plan->G, plan->cfg.k, support, z, resid, plan->status);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

}  // namespace cs
