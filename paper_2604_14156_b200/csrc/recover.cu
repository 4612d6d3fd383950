// Estimator: block iterative hard thresholding, one small CTA per token.
//
//   z_0 = 0;  T times:  v = z + mu Phi^T (y - Phi z);  z = H_k(v)
//
// The iteration is a latency chain (T sequential steps of a small mat-vec and a top-k), so the cost
// is the number of instructions on the critical path.  Two things keep it short.
//   - The update is evaluated in its expanded form  v = c + M z  with  c = mu Phi^T y  (once per
//     token) and  M = I - mu Phi^T Phi  (once per layer, gram_rows below).  Since z has exactly k
//     non-zeros, one iteration is k multiply-adds per entry instead of the two mat-vecs through
//     the m-dimensional residual, and nothing but z crosses threads.
//   - Thread g owns entry g of v and z (one entry per lane, ceil(G/32) warps).  z is a compact list
//     of its k values in shared memory, read by broadcast, and the thread keeps the k matrix entries
//     M[g, idx_j] that go with the list in registers (fetched from global memory when the support
//     changes), so the mat-vec has no indexed load.  (For k > 56 z is a dense vector instead and
//     the thread keeps its whole row of M.)
//   - H_k is exact under the total order (|v| descending, group index ascending), but most
//     iterations do not change the support, which is the case exactly when every kept |v| exceeds
//     every other |v|: two warp reductions and one barrier decide that, and only otherwise are the
//     exact ranks computed.  A rank is the number of entries that precede: key greater, or equal
//     from a lower index.  Blocks of 32 keys owned by lower warps count with >=, by higher warps
//     with >.  Equal keys inside the own warp are rare (exact ties); they make the ranks add up to
//     less than those of a permutation, which every thread checks, and only then is the slow match
//     instruction used to put the lower index first.  rank < k  <=>  kept, and the rank is the
//     entry's slot in the new list.
// A shared-memory round trip costs about 30 cycles and a barrier about 20, so an iteration that
// keeps the support is one round trip, one barrier and k multiply-adds.  After the last iteration
// the kept entries are written in ascending index order (the output format) and ||y - Phi z||_2 is
// formed from Phi, y and z.
#include "cs_internal.cuh"

namespace cs {


// M = I - mu Phi^T Phi, row-major with padded rows; only Phi and mu enter, so it can be formed beside the sketch.
__global__ void __launch_bounds__(kGramThreads) gram_kernel(const float *__restrict__ Phi, float mu, int m, int G,
                                                            float *__restrict__ gram) {
    pdl_launch_dependents();
    gram_rows(Phi, mu, m, G, blockIdx.x, gram);
}

// 1.0f if a > b else 0.0f.
__device__ __forceinline__ float gt01(float a, float b) {
    float r;
    asm("set.gt.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
// NW = warps = ceil(G / 32).  KC = ceil(k / 8) for k <= 56: the iterate is a compact list of k
// values whose matrix entries M[idx_j, g] the thread keeps in registers; KC = 0: any k, the iterate
// is a dense vector and the thread keeps its whole row of M.
template <int NW, int KC>
__global__ void __launch_bounds__(32 * NW)
recover_kernel(const float *__restrict__ Phi, const float *__restrict__ gram, float mu, const float *__restrict__ y,
               int m, int G, int k, int T, int32_t *__restrict__ support, float *__restrict__ z_out,
               float *__restrict__ resid_out, const int32_t *__restrict__ sup0, const float *__restrict__ z0) {
    constexpr int GP = 32 * NW;                    // padded number of entries = pitch of M
    constexpr int NV = KC > 0 ? KC * 8 : GP;       // length of the iterate as the mat-vec reads it
    constexpr int NR = KC > 0 ? KC * 8 : GP;       // matrix entries a thread keeps
    __shared__ __align__(16) float key_s[GP];      // |v| of the current iterate
    __shared__ __align__(16) float val_s[2][NV];   // the iterate, by iteration parity: list values, or dense z
    __shared__ int idx_s[NV];                      // list form: entry index of each list slot
    __shared__ float y_s[kMaxM];
    __shared__ uint32_t mm_s[2][2][4];             // per parity: min kept key / max other key, per warp
    __shared__ int sum_s[4];                       // rank sums per warp
    __shared__ int cnt_s[4];
    __shared__ float red_s[kMaxM];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = tid;  // entry owned by this thread
    const bool valid = g < G;
    const int t = blockIdx.x;
    pdl_launch_dependents();
    // Phi is a parameter: this thread's column (needed for c) is requested before the wait for the
    // kernel that produces y and M, when it fits 32 registers
    const bool early_phi = m <= 32;
    float phc[32];
    if (early_phi) {
#pragma unroll
        for (int row = 0; row < 32; ++row) phc[row] = (valid && row < m) ? __ldg(Phi + row * G + g) : 0.f;
    }
    pdl_wait();   // y and M come from the kernel before
    float mreg[NR];
    const float *mcol = gram + (valid ? g : 0);
    if constexpr (KC > 0) {
        // List form: the entries M[idx_j, g] that go with the list come straight from global memory (M is
        // 30 to 60 KB and stays in L1/L2) and are fetched again only when the support changes, which
        // keeps the CTA's shared memory at 2 KB.  The first list is 0..k-1: requested at once.
#pragma unroll
        for (int j = 0; j < NR; ++j) mreg[j] = ld_dep(mcol + (j < k ? j : 0) * GP);
    }
    if constexpr (KC == 0) {   // row g of M (M is symmetric: row g is the column that multiplies into entry g)
        const float *src = gram + (size_t)(valid ? g : 0) * GP;
#pragma unroll
        for (int j = 0; j < GP / 4; ++j) {
            const float4 q = ld_dep4(src + 4 * j);
            mreg[4 * j] = q.x; mreg[4 * j + 1] = q.y; mreg[4 * j + 2] = q.z; mreg[4 * j + 3] = q.w;
        }
    }
    for (int row = tid; row < m; row += GP) y_s[row] = ld_dep(y + (size_t)t * m + row);
    // z_0 = 0 with the support the order assigns to an all-zero vector (indices 0..k-1), or, warm
    // started, the k-sparse iterate handed in (sup0 ascending and distinct, z0 its values).
    __shared__ int slot_s[GP];                     // warm start: list slot of each entry, -1 outside
    const bool warm = sup0 != nullptr;
    slot_s[g] = -1;
    for (int i = tid; i < NV; i += GP) { val_s[0][i] = 0.f; val_s[1][i] = 0.f; idx_s[i] = i < k ? i : 0; }
    __syncthreads();
    if (warm) {
        for (int j = tid; j < k; j += GP) {
            const int e = ld_dep(sup0 + (size_t)t * k + j);
            const float zv = ld_dep(z0 + (size_t)t * k + j);
            if ((unsigned)e >= (unsigned)G) continue;   // reported by the support check that ran before
            slot_s[e] = j;
            if constexpr (KC > 0) { idx_s[j] = e; val_s[0][j] = zv; }
            else val_s[0][e] = zv;
        }
    }
    __syncthreads();
    bool kept = warm ? slot_s[g] >= 0 : g < k;
    int slot = warm ? max(slot_s[g], 0) : g;
    float v = 0.f;
    if constexpr (KC > 0) {
        if (warm) {   // the entries that go with the warm list
#pragma unroll
            for (int j = 0; j < NR; ++j) mreg[j] = ld_dep(mcol + idx_s[j] * GP);
        }
    }
    // c_g = mu sum_i Phi[i,g] y_i
    float cg = 0.f;
    if (valid && early_phi) {
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
        for (int row = 0; row < 32; row += 4) {   // rows past m hold zeros
            const float y0 = row < m ? y_s[row] : 0.f, y1 = row + 1 < m ? y_s[row + 1] : 0.f;
            const float y2 = row + 2 < m ? y_s[row + 2] : 0.f, y3 = row + 3 < m ? y_s[row + 3] : 0.f;
            a0 = fmaf(phc[row], y0, a0); a1 = fmaf(phc[row + 1], y1, a1);
            a2 = fmaf(phc[row + 2], y2, a2); a3 = fmaf(phc[row + 3], y3, a3);
        }
        cg = mu * ((a0 + a1) + (a2 + a3));
    } else if (valid) {
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        const float *pcol = Phi + g;
        int row = 0;
#pragma unroll 4
        for (; row + 3 < m; row += 4) {
            a0 = fmaf(__ldg(pcol + row * G), y_s[row], a0); a1 = fmaf(__ldg(pcol + (row + 1) * G), y_s[row + 1], a1);
            a2 = fmaf(__ldg(pcol + (row + 2) * G), y_s[row + 2], a2); a3 = fmaf(__ldg(pcol + (row + 3) * G), y_s[row + 3], a3);
        }
        for (; row < m; ++row) a0 = fmaf(__ldg(pcol + row * G), y_s[row], a0);
        cg = mu * ((a0 + a1) + (a2 + a3));
    }
    const unsigned lt_mask = (1u << lane) - 1u;
    const int rank_total = G * (G - 1) / 2;   // what the ranks of G distinct positions add up to

    for (int it = 0; it < T; ++it) {
        const int par = it & 1;
        // v_g = c_g + sum_j M[g, idx_j] z_j, the iterate read by broadcast
        float a0 = cg, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
        for (int j = 0; j < NV / 4; ++j) {
            const float4 zq = reinterpret_cast<const float4 *>(val_s[par])[j];
            a0 = fmaf(mreg[4 * j], zq.x, a0); a1 = fmaf(mreg[4 * j + 1], zq.y, a1);
            a2 = fmaf(mreg[4 * j + 2], zq.z, a2); a3 = fmaf(mreg[4 * j + 3], zq.w, a3);
        }
        v = (a0 + a1) + (a2 + a3);
        // Keys are |v| (entries past G get -2: they precede nothing).
        const uint32_t kbits = __float_as_uint(v) & 0x7fffffffu;
        const float key = valid ? __uint_as_float(kbits) : -2.f;
        // Most iterations leave the support as it is.  That is the case exactly when every kept key is
        // greater than every other key, which two warp reductions and one barrier decide; the next
        // iterate is written on that assumption and rewritten below when it fails.
        const uint32_t wmin = __reduce_min_sync(0xffffffffu, kept ? kbits : 0xffffffffu);
        const uint32_t wmax = __reduce_max_sync(0xffffffffu, (valid && !kept) ? kbits : 0u);
        key_s[g] = key;
        if constexpr (KC > 0) { if (kept) val_s[par ^ 1][slot] = v; }
        else val_s[par ^ 1][g] = kept ? v : 0.f;
        if (lane == 0) { mm_s[par][0][warp] = wmin; mm_s[par][1][warp] = wmax; }
        __syncthreads();
        uint32_t gmin = 0xffffffffu, gmax = 0u;
#pragma unroll
        for (int w = 0; w < NW; ++w) { gmin = min(gmin, mm_s[par][0][w]); gmax = max(gmax, mm_s[par][1][w]); }
        if (gmin > gmax) continue;

        // The support may change: exact ranks.  "a >= key" is evaluated as "a > the next float below
        // key" (-1 below zero), so that one kind of compare serves both cases.
        const float key_lo = kbits == 0u ? -1.f : __uint_as_float(kbits - 1u);
        float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f, c4 = 0.f, c5 = 0.f, c6 = 0.f, c7 = 0.f;  // independent counters
#pragma unroll
        for (int blk = 0; blk < NW; ++blk) {
            const float4 *kq = reinterpret_cast<const float4 *>(key_s + 32 * blk);
            // entries of lower warps precede on ties (>=), own and higher warps only when greater
            const float thr = blk < warp ? key_lo : key;
#pragma unroll
            for (int jj = 0; jj < 8; jj += 2) {
                const float4 ka = kq[jj], kb2 = kq[jj + 1];
                c0 += gt01(ka.x, thr); c1 += gt01(ka.y, thr); c2 += gt01(ka.z, thr); c3 += gt01(ka.w, thr);
                c4 += gt01(kb2.x, thr); c5 += gt01(kb2.y, thr); c6 += gt01(kb2.z, thr); c7 += gt01(kb2.w, thr);
            }
        }
        int rank = valid ? (int)(((c0 + c1) + (c2 + c3)) + ((c4 + c5) + (c6 + c7))) : 0;
        // Equal keys inside the own warp were ordered by neither side, so they share a rank and the
        // ranks no longer add up to those of a permutation; only then is the slow match instruction
        // used to put the lower index first.
        const int wsum = __reduce_add_sync(0xffffffffu, rank);
        if (lane == 0) sum_s[warp] = wsum;
        __syncthreads();
        int total = 0;
#pragma unroll
        for (int w = 0; w < NW; ++w) total += sum_s[w];
        if (total != rank_total) rank += __popc(__match_any_sync(0xffffffffu, __float_as_uint(key)) & lt_mask);
        kept = valid && rank < k;   // the rank is the entry's slot in the new list
        slot = rank;
        if constexpr (KC > 0) { if (kept) { idx_s[slot] = g; val_s[par ^ 1][slot] = v; } }
        else val_s[par ^ 1][g] = kept ? v : 0.f;
        __syncthreads();
        if constexpr (KC > 0) {
#pragma unroll
            for (int j = 0; j < NR; ++j) mreg[j] = ld_dep(mcol + idx_s[j] * GP);
        }
    }

    // residual norm ||y - Phi z||_2: warp w takes rows w, w + NW, ...; lanes stride over the entries
    if (resid_out != nullptr) {
        __syncthreads();
        key_s[g] = (kept && T > 0) ? v : 0.f;   // dense z
        __syncthreads();
        for (int row = warp; row < m; row += NW) {
            float a = 0.f;
#pragma unroll
            for (int j = 0; j < NW; ++j) {
                const int col = lane + 32 * j;
                if (col < G) a = fmaf(__ldg(Phi + row * G + col), key_s[col], a);
            }
            a = warp_sum(a);
            if (lane == 0) { const float r = y_s[row] - a; red_s[row] = r * r; }
        }
    }
    // ascending index order: a kept entry goes to slot (number of kept entries with a lower index)
    const unsigned kb = __ballot_sync(0xffffffffu, kept);
    if (lane == 0) cnt_s[warp] = __popc(kb);
    __syncthreads();
    if (kept) {
        int o = __popc(kb & lt_mask);
        for (int w = 0; w < warp; ++w) o += cnt_s[w];
        support[(size_t)t * k + o] = g;
        if (z_out != nullptr) z_out[(size_t)t * k + o] = T > 0 ? v : 0.f;
    }
    if (resid_out != nullptr && tid == 0) {
        float ss = 0.f;
        for (int row = 0; row < m; ++row) ss += red_s[row];
        resid_out[t] = sqrtf(ss);
    }
}

typedef void (*RecoverFn)(const float *, const float *, float, const float *, int, int, int, int, int32_t *, float *, float *,
                          const int32_t *, const float *);
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
                         const float *z0) {
    const cs_config &c = plan->cfg;
    const int G = plan->G;
    StageTimer timer(plan, CS_STAGE_RECOVER, st);
    if (!gram_ready) {
        launch_pdl(pdl_for(plan, B), gram_kernel, dim3(gram_blocks(G)), dim3(kGramThreads), 0, st, Phi, mu, c.m, G, plan->gram);
        plan->launches++;
        CS_CUDA_TRY(plan, cudaGetLastError());
    }
    launch_pdl(pdl_for(plan, B), recover_fn(G, c.k), dim3(B), dim3(gram_pitch(G)), 0, st, Phi,
               (const float *)plan->gram, mu, y, c.m, G, c.k, T < 0 ? c.T : T, support, z, resid, sup0, z0);
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
                     int32_t *__restrict__ drift) {
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
    if (j == 0) drift[t] = 2 * n;
}

cs_status launch_support_drift(cs_plan *plan, const int32_t *prev, const int32_t *cur, int B, int32_t *drift,
                               cudaStream_t st) {
    support_drift_kernel<<<B, kDriftThreads, 0, st>>>(prev, cur, plan->cfg.k, drift);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

}  // namespace cs
