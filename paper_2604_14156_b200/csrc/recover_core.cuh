// Block iterative hard thresholding for ONE token, run by a group of 32 * NW threads that may be a
// whole CTA (recover_kernel) or a few warps beside others (the fused small-batch step, where the
// weight stream of the actuator starts on the support of the first iteration while the remaining
// iterations run).
//
//   z_0 = 0 (or a k-sparse warm start);  T times:  v = z + mu Phi^T (y - Phi z);  z = H_k(v)
//
// The iteration is a latency chain (T sequential steps of a small mat-vec and a top-k), so the cost
// is the number of instructions on the critical path.
//   - The update is evaluated in its expanded form  v = c + M z  with  c = mu Phi^T y  (once per
//     token) and  M = I - mu Phi^T Phi  (once per layer, gram_rows).  Since z has exactly k
//     non-zeros, one iteration is k multiply-adds per entry instead of the two mat-vecs through
//     the m-dimensional residual, and nothing but z crosses threads.
//   - Thread g owns entry g of v and z.  In the list form (k <= 56) z is a list of k slots in shared
//     memory, read by broadcast: slot j holds the value of entry idx[j], and the thread keeps the k
//     matrix entries M[idx[j], g] that go with the list in registers, so the mat-vec has no indexed
//     load.  Slots are stable: an entry that stays in the support keeps its slot, an entry that
//     enters takes the slot of one that left, and only the matrix entries of those slots are fetched
//     again.  (In the first iteration from z = 0 the slots are handed out by rank, which lists the
//     support by decreasing magnitude.)  For k > 56 z is a dense vector and the thread keeps its
//     whole row of M.
//   - H_k is exact under the total order (|v| descending, group index ascending), but most
//     iterations do not change the support, which is the case exactly when every kept |v| exceeds
//     every other |v|: two warp reductions and one barrier decide that, and only otherwise are the
//     exact ranks computed.  A rank is the number of entries that precede: key greater, or equal
//     from a lower index.  Blocks of 32 keys owned by lower warps count with >=, by higher warps
//     with >.  Equal keys inside the own warp are rare (exact ties); they make the ranks add up to
//     less than those of a permutation, which every thread checks, and only then is the slow match
//     instruction used to put the lower index first.  rank < k  <=>  kept.
// After the last iteration the kept entries are written in ascending index order (the output
// format) and ||y - Phi z||_2 is formed from Phi, y and z.
#pragma once

#include "cs_internal.cuh"

namespace cs {

// 1.0f if a > b else 0.0f.
__device__ __forceinline__ float gt01(float a, float b) {
    float r;
    asm("set.gt.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}

template <int ID, int N> __device__ __forceinline__ void bar_sync() {
    asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(N) : "memory");
}
template <int ID, int N> __device__ __forceinline__ void bar_arrive() {
    asm volatile("bar.arrive %0, %1;" ::"n"(ID), "n"(N) : "memory");
}

// NW = warps = ceil(G / 32).  KC = ceil(k / 8) for k <= 56 (list form); KC = 0: any k, dense form.
template <int NW, int KC> struct RecoverSmem {
    static constexpr int GP = 32 * NW;                 // padded number of entries = pitch of M
    static constexpr int NV = KC > 0 ? KC * 8 : GP;    // length of the iterate as the mat-vec reads it
    alignas(16) float key[GP];        // |v| of the current iterate
    alignas(16) float red[kMaxM];     // residual r of the two-step form; partial sums of the residual norm
    alignas(16) float val[2][NV];     // the iterate, by iteration parity: slot values, or dense z
    int idx[NV];                      // list form: entry held by each slot (the support, in slot order)
    float y[kMaxM];
    uint32_t mm[2][2][4];             // per parity: min kept key / max other key, per warp
    int sum[4];                       // rank sums per warp
    int cnt[4];                       // entries that left the support (or, at the end, kept entries) per warp
    int cnt_in[4];                    // entries that entered, per warp
    int vac[4][32];                   // slots vacated by the entries that left, per warp
    int slot[GP];                     // warm start: slot of each entry, -1 outside
};

// Where the entries of M = I - mu Phi^T Phi come from.
//   GramSource: the matrix formed by gram_rows in global memory (pitch floats per row); get(j, g) is a
//   dependent load from L1/L2, issued only when a slot changes hands.
//   PhiSource: no matrix at all.  Phi TRANSPOSED sits in shared memory ([G][32], rows past m zero;
//   m <= 32) and the thread's own column of Phi in registers; get(j, g) = delta_jg - mu Phi[:, j] .
//   Phi[:, g] is eight broadcast 16-byte reads and 32 multiply-adds, and no global load, which is what
//   a recovery needs that runs while the rest of the GPU saturates the memory system.  The k entries
//   of the first support are formed together with 32 * NW helper threads (PhiSource::help), which
//   take every other slot and hand their values over through shared memory.
struct GramSource {
    const float *gram;
    int pitch;
    __device__ __forceinline__ float get(int j, int g, const float (&)[32]) const {
        return ld_dep(gram + (size_t)j * pitch + g);
    }
    __device__ __forceinline__ float phi(const float *Phi, int row, int col, int G) const { return __ldg(Phi + row * G + col); }
    // the entries of all k slots: independent loads, issued together (tid: unused)
    template <int NR> __device__ __forceinline__ void fill(const int *idx, int k, int, int g, const float (&own)[32],
                                                           float (&mreg)[NR]) const {
#pragma unroll
        for (int j = 0; j < NR; ++j)
            if (j < k) mreg[j] = get(idx[j], g, own);
    }
    // the entries of the slots in `chg`: independent loads again
    template <int NR> __device__ __forceinline__ void reload(unsigned long long chg, const int *idx, int g,
                                                             const float (&own)[32], float (&mreg)[NR]) const {
#pragma unroll
        for (int j = 0; j < NR; ++j)
            if ((chg >> j) & 1ull) mreg[j] = get(idx[j], g, own);
    }
};
template <int BAR_A, int BAR_B, int THREADS> struct PhiSource {
    const float4 *phiT_s;   // shared memory, [G][8] float4
    float mu;
    float *fill_s;          // shared memory, [slots][THREADS / 2]
    __device__ __forceinline__ float get(int j, int g, const float (&own)[32]) const {
        const float4 *col = phiT_s + j * 8;
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float4 c = col[q];
            a0 = fmaf(c.x, own[4 * q], a0); a1 = fmaf(c.y, own[4 * q + 1], a1);
            a2 = fmaf(c.z, own[4 * q + 2], a2); a3 = fmaf(c.w, own[4 * q + 3], a3);
        }
        return (j == g ? 1.f : 0.f) - mu * ((a0 + a1) + (a2 + a3));
    }
    __device__ __forceinline__ float phi(const float *, int row, int col, int) const {
        return reinterpret_cast<const float *>(phiT_s)[col * 32 + row];
    }
    // slots `first`, first + 2, ... for column g into the hand-over array (place tid: one per thread)
    __device__ __forceinline__ void half(const int *idx, int k, int tid, int g, const float (&own)[32], int first) const {
#pragma unroll 2
        for (int j = first; j < k; j += 2) fill_s[j * (THREADS / 2) + tid] = get(idx[j], g, own);
    }
    template <int NR> __device__ __forceinline__ void fill(const int *idx, int k, int tid, int g, const float (&own)[32],
                                                           float (&mreg)[NR]) const {
        bar_sync<BAR_A, THREADS>();   // the helpers may read the table
        half(idx, k, tid, g, own, 0);
        __threadfence_block();
        bar_sync<BAR_B, THREADS>();   // both halves are in the hand-over array
#pragma unroll
        for (int j = 0; j < NR; ++j)
            if (j < k) mreg[j] = fill_s[j * (THREADS / 2) + tid];
    }
    // what helper thread tid (0 .. THREADS/2 - 1) runs, once, for a cold start with T >= 1: column g, the odd slots
    __device__ __forceinline__ void help(const int *idx, int k, int tid, int g, const float (&own)[32]) const {
        bar_sync<BAR_A, THREADS>();
        half(idx, k, tid, g, own, 1);
        __threadfence_block();
        bar_sync<BAR_B, THREADS>();
    }
    // one entry per changed slot, moved into its register by a select (the slot index is the same in
    // every thread, and changes are few): keeps the code of a support change a few hundred bytes
    template <int NR> __device__ __forceinline__ void reload(unsigned long long chg, const int *idx, int g,
                                                             const float (&own)[32], float (&mreg)[NR]) const {
        while (chg != 0ull) {
            const int js = __ffsll((long long)chg) - 1;
            chg &= chg - 1ull;
            const float mv = get(idx[js], g, own);
#pragma unroll
            for (int j = 0; j < NR; ++j) mreg[j] = j == js ? mv : mreg[j];
        }
    }
};

// This thread's column of Phi (needed for c): Phi is a parameter, so a caller under programmatic
// dependent launch requests it before the wait for the kernel that produces y and M.
template <int NW>
__device__ __forceinline__ void recover_load_phi(const float *__restrict__ Phi, int m, int G, int g, float (&phc)[32]) {
    const bool valid = g < G;
#pragma unroll
    for (int row = 0; row < 32; ++row) phc[row] = (valid && row < m) ? __ldg(Phi + row * G + g) : 0.f;
}

// Runs the recovery of one token.  g = this thread's entry (0 .. 32*NW-1); all 32*NW threads call it
// together and synchronise on named barrier BAR.  M: where the entries of I - mu Phi^T Phi come from
// (the dense form reads whole rows of the global matrix, whose pitch must be 32 * NW).  phc: the thread's column of Phi when m <= 32
// (recover_load_phi), unused otherwise.  y, gram, sup0, z0 may come from the kernel before: they are
// read with dependent loads, after the caller's wait.  table_ready() is called once by every thread
// when the slot table s.idx first holds a support worth acting on (that of the first iterate, or the
// start's own when T == 0 or the start is warm); from then on s.idx always holds k valid groups and changes only where the
// support changes: slot_changed(slot, g) is called by the thread whose entry g has just taken `slot`.
// table_final() is called once by every thread after the last iteration, before the outputs are
// written.
template <int NW, int KC, int BAR, typename MSource, typename TableReady, typename SlotChanged, typename TableFinal>
__device__ __forceinline__ void recover_token(RecoverSmem<NW, KC> &s, const int g, const float *__restrict__ Phi,
                                              const MSource M, float mu, const float *__restrict__ y, int m, int G, int k, int T, int32_t *__restrict__ support,
                                              float *__restrict__ z_out, float *__restrict__ resid_out,
                                              const int32_t *__restrict__ sup0, const float *__restrict__ z0,
                                              const float tgamma, const int32_t *__restrict__ sup_prev,
                                              const float *__restrict__ z_prev, DeviceStatus *status, const float (&phc)[32], TableReady table_ready,
                                              SlotChanged slot_changed, TableFinal table_final) {
    constexpr int GP = 32 * NW;
    constexpr int NV = RecoverSmem<NW, KC>::NV;
    constexpr int NR = NV;                         // matrix entries a thread keeps
    const int lane = g & 31, warp = g >> 5;
    const bool valid = g < G;
    const bool early_phi = m <= 32;
    float mreg[NR];
    const int gm = valid ? g : 0;
    if constexpr (KC > 0) {
        // List form: the entries M[idx_j, g] that go with the list.  The first list (0..k-1) holds zeros
        // unless the start is warm, and a cold first iteration hands the slots out anew: nothing to fetch yet.
#pragma unroll
        for (int j = 0; j < NR; ++j) mreg[j] = 0.f;
    }
    if constexpr (KC == 0) {   // row g of M (M is symmetric: row g is the column that multiplies into entry g)
        const float *src = M.gram + (size_t)gm * GP;
#pragma unroll
        for (int j = 0; j < GP / 4; ++j) {
            const float4 q = ld_dep4(src + 4 * j);
            mreg[4 * j] = q.x; mreg[4 * j + 1] = q.y; mreg[4 * j + 2] = q.z; mreg[4 * j + 3] = q.w;
        }
    }
    for (int row = g; row < m; row += GP) s.y[row] = ld_dep(y + row);
    // z_0 = 0 with the support the order assigns to an all-zero vector (indices 0..k-1), or, warm
    // started, the k-sparse iterate handed in (sup0 ascending and distinct, z0 its values).
    const bool warm = sup0 != nullptr;
    s.slot[g] = -1;
    for (int i = g; i < NV; i += GP) { s.val[0][i] = 0.f; s.val[1][i] = 0.f; s.idx[i] = i < k ? i : 0; }
    bar_sync<BAR, GP>();
    if (warm) {
        for (int j = g; j < k; j += GP) {
            const int e = ld_dep(sup0 + j);
            const float zv = ld_dep(z0 + j);
            if ((unsigned)e >= (unsigned)G) continue;   // reported by the support check that ran before
            s.slot[e] = j;
            if constexpr (KC > 0) { s.idx[j] = e; s.val[0][j] = zv; }
            else s.val[0][e] = zv;
        }
    }
    bar_sync<BAR, GP>();
    bool kept = warm ? s.slot[g] >= 0 : g < k;
    int slot = warm ? max(s.slot[g], 0) : g;
    float v = 0.f;
    // Temporal regulariser (Sec. 5), tgamma = 2 mu gamma: the step gains  tgamma (z_prev - z)_g.  z_prev is the
    // k-sparse estimate of the previous decoding step (sup_prev ascending, z_prev its values).
    float zprev_g = 0.f;
    if (tgamma != 0.f && sup_prev != nullptr) {
        for (int j = 0; j < k; ++j)
            if (ld_dep(sup_prev + j) == g) zprev_g = ld_dep(z_prev + j);
        if (warm && kept) {   // v holds this entry's value in the current iterate
            if constexpr (KC > 0) v = s.val[0][slot]; else v = s.val[0][g];
        }
    }
    if constexpr (KC > 0) {
        if (warm) {   // the entries that go with the warm list
#pragma unroll
            for (int j = 0; j < NR; ++j) mreg[j] = M.get(s.idx[j], gm, phc);
        }
    }
    // c_g = mu sum_i Phi[i,g] y_i
    float cg = 0.f;
    if (valid && early_phi) {
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
        for (int row = 0; row < 32; row += 4) {   // rows past m hold zeros
            const float y0 = row < m ? s.y[row] : 0.f, y1 = row + 1 < m ? s.y[row + 1] : 0.f;
            const float y2 = row + 2 < m ? s.y[row + 2] : 0.f, y3 = row + 3 < m ? s.y[row + 3] : 0.f;
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
            a0 = fmaf(__ldg(pcol + row * G), s.y[row], a0); a1 = fmaf(__ldg(pcol + (row + 1) * G), s.y[row + 1], a1);
            a2 = fmaf(__ldg(pcol + (row + 2) * G), s.y[row + 2], a2); a3 = fmaf(__ldg(pcol + (row + 3) * G), s.y[row + 3], a3);
        }
        for (; row < m; ++row) a0 = fmaf(__ldg(pcol + row * G), s.y[row], a0);
        cg = mu * ((a0 + a1) + (a2 + a3));
    }
    const unsigned lt_mask = (1u << lane) - 1u;
    const int rank_total = G * (G - 1) / 2;   // what the ranks of G distinct positions add up to
    if (T == 0 || warm || KC == 0) table_ready();

    for (int it = 0; it < T; ++it) {
        const int par = it & 1;
        {
            // v_g = c_g + sum_j M[g, idx_j] z_j, the iterate read by broadcast
            float a0 = cg, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
            for (int j = 0; j < NV / 4; ++j) {
                const float4 zq = reinterpret_cast<const float4 *>(s.val[par])[j];
                a0 = fmaf(mreg[4 * j], zq.x, a0); a1 = fmaf(mreg[4 * j + 1], zq.y, a1);
                a2 = fmaf(mreg[4 * j + 2], zq.z, a2); a3 = fmaf(mreg[4 * j + 3], zq.w, a3);
            }
            const float zcur = kept ? v : 0.f;   // this entry of the current iterate (v: its value from the step before)
            v = (a0 + a1) + (a2 + a3);
            if (tgamma != 0.f) v = fmaf(tgamma, zprev_g - zcur, v);
        }
        // Keys are |v| (entries past G get -2: they precede nothing).  A NaN has no place in the order:
        // it is ranked as a zero, so that the fast test below (integer order) and the exact ranks
        // (float order) agree and every iteration still keeps exactly k entries.
        uint32_t kbits = __float_as_uint(v) & 0x7fffffffu;
        if (kbits > 0x7f800000u) kbits = 0u;
        const float key = valid ? __uint_as_float(kbits) : -2.f;
        // Most iterations leave the support as it is.  That is the case exactly when every kept key is
        // greater than every other key, which two warp reductions and one barrier decide; the next
        // iterate is written on that assumption and rewritten below when it fails.
        const uint32_t wmin = __reduce_min_sync(0xffffffffu, kept ? kbits : 0xffffffffu);
        const uint32_t wmax = __reduce_max_sync(0xffffffffu, (valid && !kept) ? kbits : 0u);
        s.key[g] = key;
        if constexpr (KC > 0) { if (kept) s.val[par ^ 1][slot] = v; }
        else s.val[par ^ 1][g] = kept ? v : 0.f;
        if (lane == 0) { s.mm[par][0][warp] = wmin; s.mm[par][1][warp] = wmax; }
        bar_sync<BAR, GP>();
        uint32_t gmin = 0xffffffffu, gmax = 0u;
#pragma unroll
        for (int w = 0; w < NW; ++w) { gmin = min(gmin, s.mm[par][0][w]); gmax = max(gmax, s.mm[par][1][w]); }
        // (a cold first iteration always takes the exact path: it hands out the slots and fetches their
        // matrix entries)
        if (gmin > gmax && (it > 0 || warm || KC == 0)) continue;

        // The support may change: exact ranks.  "a >= key" is evaluated as "a > the next float below
        // key" (-1 below zero), so that one kind of compare serves both cases.
        const float key_lo = kbits == 0u ? -1.f : __uint_as_float(kbits - 1u);
        float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f, c4 = 0.f, c5 = 0.f, c6 = 0.f, c7 = 0.f;  // independent counters
#pragma unroll
        for (int blk = 0; blk < NW; ++blk) {
            const float4 *kq = reinterpret_cast<const float4 *>(s.key + 32 * blk);
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
        if (lane == 0) s.sum[warp] = wsum;
        bar_sync<BAR, GP>();
        int total = 0;
#pragma unroll
        for (int w = 0; w < NW; ++w) total += s.sum[w];
        if (total != rank_total) rank += __popc(__match_any_sync(0xffffffffu, __float_as_uint(key)) & lt_mask);
        const bool kept_new = valid && rank < k;
        if constexpr (KC == 0) {
            kept = kept_new;
            s.val[par ^ 1][g] = kept ? v : 0.f;
            bar_sync<BAR, GP>();
        } else {
            // Stable slots: the i-th entry that enters (by index) takes the slot of the i-th that left.
            // In a cold first iteration no slot holds anything yet: every kept entry "enters", and the
            // slots go out by rank, so that the table lists the support by decreasing magnitude.  (One
            // code path for both on purpose: whatever runs later has then run once before anything
            // else competes for the instruction cache's way to memory.)
            const bool first = it == 0 && !warm;
            const bool leaving = !first && kept && !kept_new, entering = (first || !kept) && kept_new;
            const unsigned bl = __ballot_sync(0xffffffffu, leaving), be = __ballot_sync(0xffffffffu, entering);
            if (leaving) s.vac[warp][__popc(bl & lt_mask)] = slot;
            if (lane == 0) { s.cnt[warp] = __popc(bl); s.cnt_in[warp] = __popc(be); }
            bar_sync<BAR, GP>();
            if (entering) {
                if (first) {
                    slot = rank;
                } else {
                    int e = __popc(be & lt_mask);
                    for (int w = 0; w < warp; ++w) e += s.cnt_in[w];
                    int w2 = 0;
                    while (w2 < NW - 1 && e >= s.cnt[w2]) { e -= s.cnt[w2]; ++w2; }
                    // (the bound only matters for an invalid warm start, whose counts need not match)
                    slot = (int)min((unsigned)s.vac[w2][e & 31], (unsigned)(NV - 1));
                }
                s.idx[slot] = g;
                slot_changed(slot, g);
            }
            kept = kept_new;
            if (kept) s.val[par ^ 1][slot] = v;
            unsigned long long chg = 0ull;   // slots whose entry changed
            if (first) {
                chg = k >= 64 ? ~0ull : (1ull << k) - 1ull;
            } else {
#pragma unroll
                for (int w = 0; w < NW; ++w)
                    for (int i = 0; i < s.cnt[w]; ++i) chg |= 1ull << s.vac[w][i];
            }
            bar_sync<BAR, GP>();
            if (first) table_ready();   // the table holds the first iterate's support
            if (first) M.fill(s.idx, k, g, gm, phc, mreg);   // the entries of all k slots
            else M.reload(chg, s.idx, gm, phc, mreg);        // those of the slots that changed hands
        }
    }
    table_final();

    // residual norm ||y - Phi z||_2
    if (resid_out != nullptr) {
        if constexpr (KC > 0) {
            // z has k non-zeros, held by the slots: a thread takes rows g, g + GP, ... and sums over the slots
            // (the last iterate's values are in val[T & 1]; every path above ends on a barrier)
            float ss = 0.f;
            for (int row = g; row < m; row += GP) {
                float a = 0.f;
#pragma unroll 8
                for (int j = 0; j < k; ++j) a = fmaf(M.phi(Phi, row, s.idx[j], G), s.val[T & 1][j], a);
                const float r = s.y[row] - a;
                ss = fmaf(r, r, ss);
            }
            ss = warp_sum(ss);
            if (lane == 0) s.red[warp] = ss;
        } else {   // dense form: warp w takes rows w, w + NW, ...; lanes stride over the entries
            bar_sync<BAR, GP>();
            s.key[g] = (kept && T > 0) ? v : 0.f;   // dense z
            bar_sync<BAR, GP>();
            for (int row = warp; row < m; row += NW) {
                float a = 0.f;
#pragma unroll
                for (int j = 0; j < NW; ++j) {
                    const int col = lane + 32 * j;
                    if (col < G) a = fmaf(M.phi(Phi, row, col, G), s.key[col], a);
                }
                a = warp_sum(a);
                if (lane == 0) { const float r = s.y[row] - a; s.red[row] = r * r; }
            }
        }
    }
    // ascending index order: a kept entry goes to position (number of kept entries with a lower index)
    const unsigned kb = __ballot_sync(0xffffffffu, kept);
    if (lane == 0) s.cnt[warp] = __popc(kb);
    bar_sync<BAR, GP>();
    if (kept) {
        int o = __popc(kb & lt_mask);
        for (int w = 0; w < warp; ++w) o += s.cnt[w];
        if (o < k) {   // always true for k kept entries; the bound keeps a broken count from leaving the row
            if (support != nullptr) support[o] = g;
            if (z_out != nullptr) z_out[o] = T > 0 ? v : 0.f;
        }
    }
    // a NaN or infinite iterate (non-finite y, or a diverging step size): indices above are valid, values are not
    if (valid && T > 0 && !(fabsf(v) <= 3.402823466e38f) && status != nullptr)
        atomicCAS(&status->code, 0, (int)CS_ERR_NONFINITE);
    if (resid_out != nullptr && g == 0) {
        float ss = 0.f;
        const int parts = KC > 0 ? NW : m;   // per-warp sums in the list form, per-row squares in the dense form
        for (int i = 0; i < parts; ++i) ss += s.red[i];
        *resid_out = sqrtf(ss);
    }
}

}  // namespace cs
