// Estimator: block iterative hard thresholding, one small CTA per token (the iteration itself is
// recover_core.cuh), plus the support-drift count.
#include "recover_core.cuh"

namespace cs {

// M = I - mu Phi^T Phi, row-major with padded rows; only Phi and mu enter, so it can be formed beside the sketch.
__global__ void __launch_bounds__(kGramThreads) gram_kernel(const float *__restrict__ Phi, float mu, int m, int G,
                                                            float *__restrict__ gram) {
    pdl_launch_dependents();
    gram_rows(Phi, mu, m, G, blockIdx.x, gram);
}

// NW = warps = ceil(G / 32).  KC = ceil(k / 8) for k <= 56 (list form), 0 otherwise (dense form).
template <int NW, int KC>
__global__ void __launch_bounds__(32 * NW)
recover_kernel(const float *__restrict__ Phi, const float *__restrict__ gram, float mu, const float *__restrict__ y,
               int m, int G, int k, int T, int32_t *__restrict__ support, float *__restrict__ z_out,
               float *__restrict__ resid_out, const int32_t *__restrict__ sup0, const float *__restrict__ z0,
               float tgamma, const int32_t *__restrict__ sup_prev, const float *__restrict__ z_prev, DeviceStatus *status) {
    __shared__ RecoverSmem<NW, KC> s;
    const int g = threadIdx.x, t = blockIdx.x;
    pdl_launch_dependents();
    // Phi is a parameter: this thread's column is requested before the wait for the kernel that
    // produces y and M, when it fits 32 registers
    float phc[32];
    if (m <= 32) recover_load_phi<NW>(Phi, m, G, g, phc);
    pdl_wait();   // y and M come from the kernel before
    recover_token<NW, KC, 0>(s, g, Phi, GramSource{gram, 32 * NW}, mu, y + (size_t)t * m, m, G, k, T, support + (size_t)t * k,
                             z_out != nullptr ? z_out + (size_t)t * k : nullptr,
                             resid_out != nullptr ? resid_out + t : nullptr,
                             sup0 != nullptr ? sup0 + (size_t)t * k : nullptr, z0 != nullptr ? z0 + (size_t)t * k : nullptr,
                             tgamma, sup_prev != nullptr ? sup_prev + (size_t)t * k : nullptr,
                             z_prev != nullptr ? z_prev + (size_t)t * k : nullptr, status, phc, [] {}, [](int, int) {}, [] {});
}

typedef void (*RecoverFn)(const float *, const float *, float, const float *, int, int, int, int, int32_t *, float *, float *,
                          const int32_t *, const float *, float, const int32_t *, const float *, DeviceStatus *);
static int recover_kc(int k) { return k <= 56 ? (k + 7) / 8 : 0; }
template <int NW> static RecoverFn recover_fn_kc(int k) {
    switch (recover_kc(k)) {
        case 1: return recover_kernel<NW, 1>;
        case 2: return recover_kernel<NW, 2>;
        case 3: return recover_kernel<NW, 3>;
        case 4: return recover_kernel<NW, 4>;
        case 5: return recover_kernel<NW, 5>;
        case 6: return recover_kernel<NW, 6>;
        case 7: return recover_kernel<NW, 7>;
        default: return recover_kernel<NW, 0>;
    }
}
static RecoverFn recover_fn(int G, int k) {
    switch ((G + 31) / 32) {
        case 1: return recover_fn_kc<1>(k);
        case 2: return recover_fn_kc<2>(k);
        case 3: return recover_fn_kc<3>(k);
        default: return recover_fn_kc<4>(k);
    }
}
cs_status launch_recover(cs_plan *plan, const float *Phi, float mu, const float *y, int B, int32_t *support,
                         float *z, float *resid, bool gram_ready, cudaStream_t st, int T, const int32_t *sup0,
                         const float *z0, float gamma, const int32_t *sup_prev, const float *z_prev) {
    const cs_config &c = plan->cfg;
    const int G = plan->G;
    StageTimer timer(plan, CS_STAGE_RECOVER, st);
    if (!gram_ready) {
        launch_pdl(pdl_for(plan, B), gram_kernel, dim3(gram_blocks(G)), dim3(kGramThreads), 0, st, Phi, mu, c.m, G, plan->gram);
        plan->launches++;
        CS_CUDA_TRY(plan, cudaGetLastError());
    }
    launch_pdl(pdl_for(plan, B), recover_fn(G, c.k), dim3(B), dim3(gram_pitch(G)), 0, st, Phi,
               (const float *)plan->gram, mu, y, c.m, G, c.k, T < 0 ? c.T : T, support, z, resid, sup0, z0, 2.f * mu * gamma, sup_prev,
               z_prev, plan->status);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

// Support drift between consecutive decoding steps (Sec. 11): Delta_t = |S_t symmetric-difference
// S_{t-1}|.  Both rows are ascending and distinct, so entry j of the new row is looked up in the old
// one by bisection; the rows have k entries each, so the symmetric difference is twice the misses.
constexpr int kDriftThreads = kMaxG;
__global__ void __launch_bounds__(kDriftThreads)
support_drift_kernel(const int32_t *__restrict__ prev, const int32_t *__restrict__ cur, int k,
                     int32_t *__restrict__ drift, float *__restrict__ ratio) {
    const int t = blockIdx.x, j = threadIdx.x;
    const int32_t *p = prev + (size_t)t * k;
    int missing = 0;
    if (j < k) {
        const int e = cur[(size_t)t * k + j];
        int lo = 0, hi = k;                       // first index whose entry is >= e
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (p[mid] < e) lo = mid + 1; else hi = mid;
        }
        missing = !(lo < k && p[lo] == e);
    }
    const int n = __syncthreads_count(missing);
    if (j == 0) {
        if (drift != nullptr) drift[t] = 2 * n;
        // D_t = |S_t sym.diff S_{t-1}| / |S_t union S_{t-1}| (Sec. 15): both rows have k entries, so the union has k + n
        if (ratio != nullptr) ratio[t] = (float)(2 * n) / (float)(k + n);
    }
}

cs_status launch_support_drift(cs_plan *plan, const int32_t *prev, const int32_t *cur, int B, int32_t *drift,
                               float *ratio, cudaStream_t st) {
    support_drift_kernel<<<B, kDriftThreads, 0, st>>>(prev, cur, plan->cfg.k, drift, ratio);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

}  // namespace cs
