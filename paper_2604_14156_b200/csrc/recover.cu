// Estimator: block iterative hard thresholding, one warp per token.
//
//   z_0 = 0;  T times:  r = y - Phi z;  v = z + mu Phi^T r;  z = H_k(v)
//
// Phi (m x G, padded to an odd row pitch so that both access patterns are bank-conflict free)
// lives in shared memory.  A lane owns the entries g = lane + 32 i of v and z (G <= 128: four
// per lane) and the rows r = lane + 32 q of the residual (m <= 64: two per lane).  z is carried
// as a compact (index, value) list of exactly k entries in shared memory, in ascending index
// order, which is also the output format.
//
// H_k is exact under the total order (|v| descending, index ascending): the k-th largest
// magnitude is found by bisection on the float bit pattern (monotone for non-negative floats),
// everything strictly above it is kept, and ties at the threshold are kept lowest index first.
#include "cs_internal.cuh"

namespace cs {

__device__ __forceinline__ int pitch_of(int G) { return G | 1; }

template <int SLOTS, int ROWS>
__global__ void recover_kernel(const float *__restrict__ Phi, float mu, const float *__restrict__ y, int B,
                               int m, int G, int k, int T, int32_t *__restrict__ support,
                               float *__restrict__ z_out, float *__restrict__ resid_out) {
    extern __shared__ float smem[];
    const int warps = blockDim.x >> 5;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int Gp = pitch_of(G);
    float *phi_s = smem;                                  // [m][Gp]
    float *r_s = phi_s + m * Gp + warp * kMaxM;           // [warps][kMaxM]
    float *val_s = phi_s + m * Gp + warps * kMaxM + warp * kMaxG;          // [warps][kMaxG]
    int *idx_s = reinterpret_cast<int *>(phi_s + m * Gp + warps * (kMaxM + kMaxG)) + warp * kMaxG;

    for (int i = threadIdx.x; i < m * G; i += blockDim.x) phi_s[(i / G) * Gp + (i % G)] = Phi[i];
    __syncthreads();

    const int t = blockIdx.x * warps + warp;
    if (t >= B) return;
    const unsigned lt_mask = (1u << lane) - 1u;

    float yv[ROWS];
#pragma unroll
    for (int q = 0; q < ROWS; ++q) {
        const int row = lane + 32 * q;
        yv[q] = row < m ? y[(size_t)t * m + row] : 0.f;
    }
    // z_0 = 0 with the support the order assigns to an all-zero vector: indices 0..k-1.
    for (int c = lane; c < k; c += 32) { idx_s[c] = c; val_s[c] = 0.f; }
    float zv[SLOTS];
#pragma unroll
    for (int i = 0; i < SLOTS; ++i) zv[i] = 0.f;
    __syncwarp();

    for (int it = 0; it <= T; ++it) {
        // r = y - Phi z  (z through its compact list, ascending index = the order of a dense sum)
        float rr[ROWS];
#pragma unroll
        for (int q = 0; q < ROWS; ++q) {
            const int row = lane + 32 * q;
            float acc = 0.f;
            if (row < m) {
                const float *prow = phi_s + row * Gp;
                for (int c = 0; c < k; ++c) acc = fmaf(prow[idx_s[c]], val_s[c], acc);
            }
            rr[q] = yv[q] - acc;
            if (row < m) r_s[row] = rr[q];
        }
        if (it == T) {  // final residual norm, then done
            float ss = 0.f;
#pragma unroll
            for (int q = 0; q < ROWS; ++q) ss += (lane + 32 * q < m) ? rr[q] * rr[q] : 0.f;
            ss = warp_sum(ss);
            if (lane == 0 && resid_out != nullptr) resid_out[t] = sqrtf(ss);
            break;
        }
        __syncwarp();
        // v = z + mu Phi^T r
        float v[SLOTS];
        unsigned key[SLOTS];
#pragma unroll
        for (int i = 0; i < SLOTS; ++i) {
            const int g = lane + 32 * i;
            float acc = 0.f;
            if (g < G) {
                for (int row = 0; row < m; ++row) acc = fmaf(phi_s[row * Gp + g], r_s[row], acc);
            }
            v[i] = fmaf(mu, acc, zv[i]);
            key[i] = g < G ? (__float_as_uint(v[i]) & 0x7fffffffu) : 0u;
        }
        // threshold = k-th largest key: largest tau with count(key >= tau) >= k
        unsigned tau = 0u;
        for (int bit = 30; bit >= 0; --bit) {
            const unsigned cand = tau | (1u << bit);
            int cnt = 0;
#pragma unroll
            for (int i = 0; i < SLOTS; ++i) cnt += key[i] >= cand;
            cnt = __reduce_add_sync(0xffffffffu, cnt);
            if (cnt >= k) tau = cand;
        }
        int above = 0;
#pragma unroll
        for (int i = 0; i < SLOTS; ++i) above += key[i] > tau;
        above = __reduce_add_sync(0xffffffffu, above);
        int need = k - above;  // ties at tau to keep, lowest index first
        int pos = 0;           // running position in the compact list
        __syncwarp();
#pragma unroll
        for (int i = 0; i < SLOTS; ++i) {
            const int g = lane + 32 * i;
            const bool tie = (g < G) && key[i] == tau;
            const unsigned tb = __ballot_sync(0xffffffffu, tie);
            const bool keep = (g < G) && (key[i] > tau || (tie && __popc(tb & lt_mask) < need));
            need -= __popc(tb);
            const unsigned kb = __ballot_sync(0xffffffffu, keep);
            if (keep) {
                const int p = pos + __popc(kb & lt_mask);
                idx_s[p] = g;
                val_s[p] = v[i];
            }
            pos += __popc(kb);
            zv[i] = keep ? v[i] : 0.f;
        }
        __syncwarp();
    }
    for (int c = lane; c < k; c += 32) {
        support[(size_t)t * k + c] = idx_s[c];
        if (z_out != nullptr) z_out[(size_t)t * k + c] = val_s[c];
    }
}

cs_status launch_recover(cs_plan *plan, const float *Phi, float mu, const float *y, int B,
                         int32_t *support, float *z, float *resid, cudaStream_t st) {
    const cs_config &c = plan->cfg;
    const int G = plan->G;
    StageTimer timer(plan, CS_STAGE_RECOVER, st);
    // One warp per CTA while that still fills the machine; four once tokens outnumber the SMs.
    const int warps = B > 2 * plan->sm_count ? 4 : 1;
    const int grid = (B + warps - 1) / warps;
    const size_t smem = sizeof(float) * ((size_t)c.m * (G | 1) + (size_t)warps * (kMaxM + 2 * kMaxG));
    const int slots = (G + 31) / 32, rows = (c.m + 31) / 32;
#define CS_RECOVER_CASE(SL, RW)                                                                       \
    recover_kernel<SL, RW><<<grid, warps * 32, smem, st>>>(Phi, mu, y, B, c.m, G, c.k, c.T, support, z, resid)
    if (rows <= 1) {
        if (slots <= 1) CS_RECOVER_CASE(1, 1);
        else if (slots <= 2) CS_RECOVER_CASE(2, 1);
        else if (slots <= 3) CS_RECOVER_CASE(3, 1);
        else CS_RECOVER_CASE(4, 1);
    } else {
        if (slots <= 1) CS_RECOVER_CASE(1, 2);
        else if (slots <= 2) CS_RECOVER_CASE(2, 2);
        else if (slots <= 3) CS_RECOVER_CASE(3, 2);
        else CS_RECOVER_CASE(4, 2);
    }
#undef CS_RECOVER_CASE
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

}  // namespace cs
