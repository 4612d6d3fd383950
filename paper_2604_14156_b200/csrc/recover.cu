// Estimator: block iterative hard thresholding, one CTA per token.
//
//   z_0 = 0;  T times:  r = y - Phi z;  v = z + mu Phi^T r;  z = H_k(v)
//
// The iteration is a latency chain (T sequential steps of two tiny mat-vecs and a top-k), so the
// kernel is organised to keep each step short rather than to save work:
//   - Phi (m x G) sits in shared memory with an odd row pitch.
//   - z is carried as a compact list of exactly k (index, value) pairs.  Every warp rebuilds the
//     residual r from that list on its own (lane i owns rows i and i+32), so no block-wide
//     synchronisation separates the two mat-vecs.
//   - Entry g of v belongs to a group of kRecParts adjacent lanes; each lane sums a strided subset
//     of the m rows of Phi^T r and the group folds with shuffles.
//   - H_k is exact under the total order (|v| descending, group index ascending): every entry
//     counts the entries that precede it (keys are the float bit patterns, which are monotone
//     for non-negative floats; an equal key precedes only from a lower index), again split over
//     the lanes of the group.  rank < k  <=>  kept, and the rank is the entry's slot in the new
//     list, so no prefix sum is needed inside the loop.
// Two block barriers per iteration: keys visible, list visible.  After the last iteration the
// kept entries are written in ascending index order, which is the output format.
#include "cs_internal.cuh"

namespace cs {

constexpr int kRecParts = 4;
constexpr int kRecThreads = kMaxG * kRecParts;  // 512
constexpr int kRecWarps = kRecThreads / 32;
static_assert(kMaxG == 32 * kRecParts, "each lane of a group scans one block of 32 entries");

template <int ROWS>  // residual rows per lane: ceil(m / 32)
__global__ void __launch_bounds__(kRecThreads)
recover_kernel(const float *__restrict__ Phi, float mu, const float *__restrict__ y, int m, int G, int k,
               int T, int32_t *__restrict__ support, float *__restrict__ z_out, float *__restrict__ resid_out) {
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = tid / kRecParts, part = tid % kRecParts;
    const int Gp = G | 1;
    int *key_s = reinterpret_cast<int *>(smem);   // [kMaxG] keys of the current v
    int *flag_s = key_s + kMaxG;                  // [kMaxG] kept flags (epilogue)
    int *idx_s = flag_s + kMaxG;                  // [kMaxG] list indices
    float *val_s = smem + 3 * kMaxG;              // [kMaxG] list values
    float *r_w = smem + 4 * kMaxG + warp * kMaxM; // [kRecWarps][kMaxM] per-warp residual
    float *phi_s = smem + 4 * kMaxG + kRecWarps * kMaxM;  // [m][Gp]

    const int t = blockIdx.x;
    for (int i = tid; i < m * G; i += kRecThreads) phi_s[(i / G) * Gp + (i % G)] = __ldg(Phi + i);
    float yv[ROWS];
#pragma unroll
    for (int q = 0; q < ROWS; ++q) {
        const int row = lane + 32 * q;
        yv[q] = row < m ? y[(size_t)t * m + row] : 0.f;
    }
    // z_0 = 0 with the support the order assigns to an all-zero vector: indices 0..k-1.
    if (tid < k) { idx_s[tid] = tid; val_s[tid] = 0.f; }
    float zv = 0.f;
    bool kept = g < k;
    __syncthreads();

    for (int it = 0; it < T; ++it) {
        // r = y - Phi z, rebuilt by every warp (two accumulators shorten the dependency chain)
#pragma unroll
        for (int q = 0; q < ROWS; ++q) {
            const int row = lane + 32 * q;
            if (row < m) {
                const float *prow = phi_s + row * Gp;
                float a0 = 0.f, a1 = 0.f;
                int c = 0;
                for (; c + 1 < k; c += 2) {
                    a0 = fmaf(prow[idx_s[c]], val_s[c], a0);
                    a1 = fmaf(prow[idx_s[c + 1]], val_s[c + 1], a1);
                }
                if (c < k) a0 = fmaf(prow[idx_s[c]], val_s[c], a0);
                r_w[row] = yv[q] - (a0 + a1);
            }
        }
        __syncwarp();
        // v_g = z_g + mu sum_i Phi[i,g] r_i, rows split over the lanes of the group
        float acc = 0.f;
        if (g < G) {
            for (int row = part; row < m; row += kRecParts) acc = fmaf(phi_s[row * Gp + g], r_w[row], acc);
        }
#pragma unroll
        for (int o = 1; o < kRecParts; o <<= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        const float v = fmaf(mu, acc, zv);
        const int key = g < G ? (int)(__float_as_uint(v) & 0x7fffffffu) : 0;
        if (part == 0) key_s[g] = key;
        __syncthreads();
        // rank = number of entries that precede entry g; this lane scans entries [32 part, 32 part + 32)
        int rank = 0;
        {
            const int4 *kq = reinterpret_cast<const int4 *>(key_s + 32 * part);
            const int split = g - 32 * part;  // entries below `split` in this block have a lower index
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
                const int4 kk = kq[jj];
                rank += kk.x > key - (int)(4 * jj + 0 < split);
                rank += kk.y > key - (int)(4 * jj + 1 < split);
                rank += kk.z > key - (int)(4 * jj + 2 < split);
                rank += kk.w > key - (int)(4 * jj + 3 < split);
            }
        }
#pragma unroll
        for (int o = 1; o < kRecParts; o <<= 1) rank += __shfl_xor_sync(0xffffffffu, rank, o);
        kept = g < G && rank < k;
        zv = kept ? v : 0.f;
        if (kept && part == 0) { idx_s[rank] = g; val_s[rank] = v; }
        __syncthreads();
    }

    // final residual norm (warp 0), from the list of the last iteration
    if (warp == 0 && resid_out != nullptr) {
        float ss = 0.f;
#pragma unroll
        for (int q = 0; q < ROWS; ++q) {
            const int row = lane + 32 * q;
            if (row < m) {
                const float *prow = phi_s + row * Gp;
                float a = 0.f;
                for (int c = 0; c < k; ++c) a = fmaf(prow[idx_s[c]], val_s[c], a);
                const float r = yv[q] - a;
                ss += r * r;
            }
        }
        ss = warp_sum(ss);
        if (lane == 0) resid_out[t] = sqrtf(ss);
    }
    // ascending index order: a kept entry goes to slot (number of kept entries with a lower index)
    if (part == 0) flag_s[g] = kept ? 1 : 0;
    __syncthreads();
    int slot = 0;
    {
        const int4 *fq = reinterpret_cast<const int4 *>(flag_s + 32 * part);
        const int split = g - 32 * part;
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
            const int4 f = fq[jj];
            slot += f.x & (int)(4 * jj + 0 < split);
            slot += f.y & (int)(4 * jj + 1 < split);
            slot += f.z & (int)(4 * jj + 2 < split);
            slot += f.w & (int)(4 * jj + 3 < split);
        }
    }
#pragma unroll
    for (int o = 1; o < kRecParts; o <<= 1) slot += __shfl_xor_sync(0xffffffffu, slot, o);
    if (kept && part == 0) {
        support[(size_t)t * k + slot] = g;
        if (z_out != nullptr) z_out[(size_t)t * k + slot] = zv;
    }
}

cs_status launch_recover(cs_plan *plan, const float *Phi, float mu, const float *y, int B,
                         int32_t *support, float *z, float *resid, cudaStream_t st) {
    const cs_config &c = plan->cfg;
    const int G = plan->G;
    StageTimer timer(plan, CS_STAGE_RECOVER, st);
    const size_t smem = sizeof(float) * ((size_t)c.m * (G | 1) + (size_t)kRecWarps * kMaxM + 4 * kMaxG);
    if (c.m <= 32)
        recover_kernel<1><<<B, kRecThreads, smem, st>>>(Phi, mu, y, c.m, G, c.k, c.T, support, z, resid);
    else
        recover_kernel<2><<<B, kRecThreads, smem, st>>>(Phi, mu, y, c.m, G, c.k, c.T, support, z, resid);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

}  // namespace cs
