// Estimator: block iterative hard thresholding, one small CTA per token.
//
//   z_0 = 0;  T times:  r = y - Phi z;  v = z + mu Phi^T r;  z = H_k(v)
//
// The iteration is a latency chain (T sequential steps of two tiny mat-vecs and a top-k) whose
// cost is the number of instructions on the critical path, so the CTA is as small as the data
// allows: warp w owns entries 32w .. 32w+31 of v and z (one entry per lane, ceil(G/32) warps).
//   - Phi (m x G) sits in shared memory with an odd row pitch (both access patterns conflict-free).
//   - z is carried as a compact list of exactly k (index, value) pairs in shared memory.  Every
//     warp rebuilds the residual r from that list on its own (lane i owns rows i and i+32), so no
//     block barrier separates the two mat-vecs.
//   - H_k is exact under the total order (|v| descending, group index ascending).  Keys are the
//     float bit patterns of |v| (monotone for non-negative floats).  An entry's rank is the number
//     of entries that precede it: key greater, or equal from a lower index.  Blocks of 32 keys
//     owned by lower warps count with >=, by higher warps with >, and inside the own warp
//     equal keys are found with one match instruction.  rank < k  <=>  kept, and the rank is the
//     entry's slot in the new list, so the loop needs no prefix sum.
// Two block barriers per iteration: keys visible, list visible.  After the last iteration the
// kept entries are written in ascending index order, which is the output format.
#include "cs_internal.cuh"

namespace cs {

constexpr int kRecMaxWarps = kMaxG / 32;

template <int ROWS>  // residual rows per lane: ceil(m / 32)
__global__ void __launch_bounds__(32 * kRecMaxWarps)
recover_kernel(const float *__restrict__ Phi, float mu, const float *__restrict__ y, int m, int G, int k,
               int T, int32_t *__restrict__ support, float *__restrict__ z_out, float *__restrict__ resid_out) {
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nwarps = blockDim.x >> 5;
    const int g = tid;  // entry owned by this thread
    const int Gp = G | 1;
    int *key_s = reinterpret_cast<int *>(smem);                          // [kMaxG] keys of the current v
    float2 *list_s = reinterpret_cast<float2 *>(smem + kMaxG);           // [kMaxG] (index bits, value), 16-byte aligned
    float *r_w = smem + 3 * kMaxG + warp * kMaxM;                        // [warps][kMaxM] residual
    int *cnt_s = reinterpret_cast<int *>(smem + 3 * kMaxG + kRecMaxWarps * kMaxM);  // [kRecMaxWarps]
    int *slot_s = cnt_s + kRecMaxWarps;                                             // [kMaxG] rank claims
    float *phi_s = smem + 4 * kMaxG + kRecMaxWarps * kMaxM + kRecMaxWarps;          // [m][Gp]

    const int t = blockIdx.x;
    pdl_launch_dependents();
    for (int col = tid; col < G; col += blockDim.x) {
#pragma unroll 8
        for (int row = 0; row < m; ++row) phi_s[row * Gp + col] = __ldg(Phi + row * G + col);
    }
    pdl_wait();   // Phi is a parameter and was staged above; y comes from the sketch kernel
    float yv[ROWS];
#pragma unroll
    for (int q = 0; q < ROWS; ++q) {
        const int row = lane + 32 * q;
        yv[q] = row < m ? y[(size_t)t * m + row] : 0.f;
    }
    // z_0 = 0 with the support the order assigns to an all-zero vector: indices 0..k-1.
    // The list is padded to a multiple of 8 with (index 0, value 0) so that loops over it need no tail.
    const int k8 = (k + 7) & ~7;
    if (tid < k8) list_s[tid] = make_float2(__int_as_float(tid < k ? tid : 0), 0.f);
    if (tid + blockDim.x < k8) list_s[tid + blockDim.x] = make_float2(__int_as_float(0), 0.f);
    float zv = 0.f;
    bool kept = g < k;
    const unsigned lt_mask = (1u << lane) - 1u;
    __syncthreads();

    // r = y - Phi z from the list (four accumulators shorten the dependency chain); returns the
    // residual of this lane's rows and leaves it in r_w for the whole warp
    auto residual = [&](float (&rr)[ROWS]) {
#pragma unroll
        for (int q = 0; q < ROWS; ++q) {
            const int row = min(lane + 32 * q, m - 1);
            const float *prow = phi_s + row * Gp;
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            for (int c = 0; c < k8; c += 8) {
                // eight list entries at a time: all list loads, then all Phi loads, then the FMAs
                const float4 *lq = reinterpret_cast<const float4 *>(list_s + c);
                const float4 e01 = lq[0], e23 = lq[1], e45 = lq[2], e67 = lq[3];
                const float p0 = prow[__float_as_int(e01.x)], p1 = prow[__float_as_int(e01.z)];
                const float p2 = prow[__float_as_int(e23.x)], p3 = prow[__float_as_int(e23.z)];
                const float p4 = prow[__float_as_int(e45.x)], p5 = prow[__float_as_int(e45.z)];
                const float p6 = prow[__float_as_int(e67.x)], p7 = prow[__float_as_int(e67.z)];
                a0 = fmaf(p0, e01.y, a0); a1 = fmaf(p1, e01.w, a1);
                a2 = fmaf(p2, e23.y, a2); a3 = fmaf(p3, e23.w, a3);
                a0 = fmaf(p4, e45.y, a0); a1 = fmaf(p5, e45.w, a1);
                a2 = fmaf(p6, e67.y, a2); a3 = fmaf(p7, e67.w, a3);
            }
            rr[q] = yv[q] - ((a0 + a1) + (a2 + a3));
            if (lane + 32 * q < m) r_w[lane + 32 * q] = rr[q];
        }
    };

    for (int it = 0; it < T; ++it) {
        float rr[ROWS];
        residual(rr);
        __syncwarp();
        // v_g = z_g + mu sum_i Phi[i,g] r_i
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        if (g < G) {
            const float *pcol = phi_s + g;
            int row = 0;
            for (; row + 7 < m; row += 8) {
                const float4 r4 = *reinterpret_cast<const float4 *>(r_w + row);
                const float4 r8 = *reinterpret_cast<const float4 *>(r_w + row + 4);
                const float q0 = pcol[row * Gp], q1 = pcol[(row + 1) * Gp], q2 = pcol[(row + 2) * Gp],
                            q3 = pcol[(row + 3) * Gp], q4 = pcol[(row + 4) * Gp], q5 = pcol[(row + 5) * Gp],
                            q6 = pcol[(row + 6) * Gp], q7 = pcol[(row + 7) * Gp];
                a0 = fmaf(q0, r4.x, a0); a1 = fmaf(q1, r4.y, a1); a2 = fmaf(q2, r4.z, a2); a3 = fmaf(q3, r4.w, a3);
                a0 = fmaf(q4, r8.x, a0); a1 = fmaf(q5, r8.y, a1); a2 = fmaf(q6, r8.z, a2); a3 = fmaf(q7, r8.w, a3);
            }
            for (; row < m; ++row) a0 = fmaf(pcol[row * Gp], r_w[row], a0);
        }
        const float v = fmaf(mu, (a0 + a1) + (a2 + a3), zv);
        // invalid entries get key -1: they precede nothing and nothing needs their rank
        const int key = g < G ? (int)(__float_as_uint(v) & 0x7fffffffu) : -1;
        key_s[g] = key;
        __syncthreads();
        int c0 = 0, c1 = 0, c2 = 0, c3 = 0, c4 = 0, c5 = 0, c6 = 0, c7 = 0;  // independent counters
        for (int blk = 0; blk < nwarps; ++blk) {
            const int4 *kq = reinterpret_cast<const int4 *>(key_s + 32 * blk);
            // entries of lower warps precede on ties (>=), own and higher warps only when greater
            const int thr = key - (blk < warp ? 1 : 0);
#pragma unroll
            for (int jj = 0; jj < 8; jj += 2) {
                const int4 ka = kq[jj], kb2 = kq[jj + 1];
                c0 += ka.x > thr; c1 += ka.y > thr; c2 += ka.z > thr; c3 += ka.w > thr;
                c4 += kb2.x > thr; c5 += kb2.y > thr; c6 += kb2.z > thr; c7 += kb2.w > thr;
            }
        }
        int rank = ((c0 + c1) + (c2 + c3)) + ((c4 + c5) + (c6 + c7));
        // Equal keys inside the own warp were not ordered above, so they share a rank.  That is
        // rare (exact ties), and shows as two lanes claiming one slot of a scratch table; only then
        // is the slower match instruction used to put the lower lane first.
        if (g < G) slot_s[rank] = g;
        __syncwarp();
        const bool clash = g < G && slot_s[rank] != g;
        if (__any_sync(0xffffffffu, clash)) rank += __popc(__match_any_sync(0xffffffffu, key) & lt_mask);
        kept = g < G && rank < k;
        zv = kept ? v : 0.f;
        if (kept) list_s[rank] = make_float2(__int_as_float(g), v);
        __syncthreads();
    }

    // final residual norm (warp 0), from the list of the last iteration
    if (warp == 0 && resid_out != nullptr) {
        float rr[ROWS];
        residual(rr);
        float ss = 0.f;
#pragma unroll
        for (int q = 0; q < ROWS; ++q) ss += (lane + 32 * q < m) ? rr[q] * rr[q] : 0.f;
        ss = warp_sum(ss);
        if (lane == 0) resid_out[t] = sqrtf(ss);
    }
    // ascending index order: a kept entry goes to slot (number of kept entries with a lower index)
    const unsigned kb = __ballot_sync(0xffffffffu, kept);
    if (lane == 0) cnt_s[warp] = __popc(kb);
    __syncthreads();
    if (kept) {
        int slot = __popc(kb & lt_mask);
        for (int w = 0; w < warp; ++w) slot += cnt_s[w];
        support[(size_t)t * k + slot] = g;
        if (z_out != nullptr) z_out[(size_t)t * k + slot] = zv;
    }
}

cs_status launch_recover(cs_plan *plan, const float *Phi, float mu, const float *y, int B,
                         int32_t *support, float *z, float *resid, cudaStream_t st) {
    const cs_config &c = plan->cfg;
    const int G = plan->G;
    StageTimer timer(plan, CS_STAGE_RECOVER, st);
    const int warps = (G + 31) / 32;
    const size_t smem = sizeof(float) * ((size_t)c.m * (G | 1) + 4 * kMaxG + kRecMaxWarps * kMaxM + kRecMaxWarps);
    if (c.m <= 32)
        launch_pdl(pdl_for(plan, B), recover_kernel<1>, dim3(B), dim3(32 * warps), smem, st, Phi, mu, y, c.m, G, c.k, c.T, support, z, resid);
    else
        launch_pdl(pdl_for(plan, B), recover_kernel<2>, dim3(B), dim3(32 * warps), smem, st, Phi, mu, y, c.m, G, c.k, c.T, support, z, resid);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

}  // namespace cs
