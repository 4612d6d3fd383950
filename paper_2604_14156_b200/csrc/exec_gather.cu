// Actuator, small-batch regime: a gather GEMV that streams every active weight row exactly once.
//
// The k*b active channel rows of a token (row R = slot * b + channel, slot = position in the
// token's support list) are dealt out to the CTAs of its grid row like cards: CTA x owns rows
// x, x + nx, x + 2 nx, ...  For its rows a CTA does
//     a[c]      = silu(W_gate[c,:] . h) * (W_up[c,:] . h)
//     partial[:] = sum_c a[c] * Wd_t[c,:]
// so gate, up and down rows of a channel are consumed by the same CTA and nothing but the
// d-vector of partial sums crosses CTAs.
//
// The kernel is a pure HBM stream (3 * rows * d weight elements, each used once), so two things
// matter: bytes in flight, and few instructions per byte.
//   - Every lane copies its own 16-byte chunks with cp.async (L2 -> shared, bypassing L1 and
//     registers) into slots only it reads back, so the rings need no barrier: each warp keeps
//     kWarpRing bytes in flight, kRingBytes per CTA.
//   - Gate/up phase: a warp takes (row, segment) units, a segment being kUnitChunks chunks per lane
//     of the gate row and of the up row; the two warp reductions per unit are amortised over
//     2 * kUnitChunks chunks per lane.  Segment partials are kept apart and added in segment order.
//   - Down phase: thread i owns chunk i (+512, ...) of every row, so the partial output stays in
//     registers; the down rows are copied into the warp's ring as soon as the warp has finished
//     its gate/up units, i.e. they are in flight while the activations are being folded.
// The partial d-vectors are summed in a fixed order by reduce_partials_kernel (deterministic,
// no atomics), which also adds the residual.
//
// SPEC (cs_layer_step at small batches): the supports are not an input; the recovery is still running
// (in the launch before this one, whose programmatic trigger fired when the slot table of its FIRST
// iterate was in global memory) while this kernel streams.  The recovery keeps its support as a
// table of k stable slots (slot -> group); a 17th warp of every CTA keeps copying the table of the
// CTA's token from global to shared memory, the streaming warps read that copy when they request a
// row and remember which group they requested.  The first iteration hands the slots out by
// decreasing magnitude and rows are dealt to CTAs and requested in slot order, so the rows requested
// first belong to the entries least likely to leave the support, and a slot that does change costs
// every CTA at most one row (not one CTA all of its rows).  After the gate/up pass the kernel waits
// for the launch before it to complete, reads the final table, fetches and computes again the units
// whose remembered group is not the slot's final one, and runs the down phase on the final table.
#include "recover_core.cuh"

namespace cs {

__device__ __forceinline__ float silu(float x) { return x / (1.f + __expf(-x)); }

constexpr int kGatherWarps = kGatherThreads / 32;
constexpr int kRingBytes = 192 * 1024;
constexpr int kWarpRing = kRingBytes / kGatherWarps;       // 12 KB per warp
constexpr int kUnitChunks = 4;                             // chunks per lane, matrix and unit
constexpr int kUnitBytes = 2 * kUnitChunks * 32 * 16;      // gate + up: 4 KB
constexpr int kUnitStages = kWarpRing / kUnitBytes;        // 3 units in flight per warp
constexpr int kLaneSlots = kWarpRing / (32 * 16);          // 24 chunks per lane in the down phase
constexpr int kMaxSegs = kMaxD * 4 / (kUnitChunks * 32 * 16);  // 16 (f32 rows of 8192)

constexpr int kSpecThreads = kGatherThreads + 32;   // the streaming warps + the warp that follows the slot table
constexpr uint32_t kFollowLimit = 1u << 16;         // polls of the table after which the following warp gives up

__device__ __forceinline__ int ld_visible(const int32_t *p) {
    int v;
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_acquire(const int32_t *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
    const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// CPT = 16-byte chunks per thread and row in the down phase (row bytes / (512 * 16), rounded up).
// FULL = every row is a whole number of units and of 512-chunk slices: no bounds checks inside.
// check: the CTAs with blockIdx.x == 0 also validate their token's support row (ascending, distinct).
// SPEC: `support` is the recovery's slot table, [tokens, kSlotTablePitch], still changing.
template <typename WT, int CPT, bool FULL, bool SPEC>
__global__ void __launch_bounds__(SPEC ? kSpecThreads : kGatherThreads, 1)
ffn_gather_kernel(const WT *__restrict__ Wg, const WT *__restrict__ Wu, const WT *__restrict__ Wdt,
                  const float *__restrict__ h, const int32_t *__restrict__ support, int d, int lb, int k, int G,
                  float *__restrict__ partial, DeviceStatus *status, int check, const int32_t *__restrict__ warm) {
    constexpr int E = Chunk<WT>::kElems;
    constexpr int DR = kLaneSlots / CPT;               // down rows in flight per thread
    constexpr int kSegElems = kUnitChunks * 32 * E;    // elements of one row segment
    extern __shared__ __align__(16) uint4 ring[];      // [kGatherWarps][kWarpRing / 16]
    __shared__ float red[kGatherMaxRows][kMaxSegs][2];
    __shared__ float a_s[kGatherMaxRows];
    __shared__ int chan_s[kGatherMaxRows];
    __shared__ int bad_s[kGatherMaxRows];   // row belongs to a group index outside [0, G): contributes nothing
    __shared__ short ugrp_s[SPEC ? kGatherMaxRows : 1][SPEC ? kMaxSegs : 1];   // group each unit was requested for
    __shared__ int table_s[SPEC ? kSlotTableSlots : 1];                       // the slot table as last seen
    __shared__ int done_s, final_s;                                           // pass over; table_s is the final table
    __shared__ short stale_s[SPEC ? kGatherMaxRows * kMaxSegs : 1];           // units to fetch and fold once more
    __shared__ int nstale_s;

    const int t = blockIdx.y, nx = gridDim.x, bx = blockIdx.x;
    const int b = 1 << lb;
    const int rows_total = k << lb;
    const int nrows = (rows_total - bx + nx - 1) / nx;     // rows bx, bx + nx, ...
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    auto cta_sync = [] {   // the streaming warps only
        if constexpr (SPEC) bar_sync<1, kGatherThreads>(); else __syncthreads();
    };
    pdl_launch_dependents();
    if constexpr (SPEC) {
        // No wait here: the launch before this one triggered when its first slot table was in memory,
        // and everything before THAT launch had completed by then.
        const int32_t *table_g = support + (size_t)t * kSlotTablePitch;
        if (tid == 0) { done_s = 0; final_s = 0; }
        if (tid >= kGatherThreads) {   // the following warp
            const int j = tid - kGatherThreads;
            int g = j < k ? ld_visible(table_g + j) : 0;
            table_s[j] = (unsigned)g < (unsigned)G ? g : 0;
            bar_sync<2, kSpecThreads>();
            // Keeps copying until the streaming warps have finished their pass, or the recovery has marked
            // the table final (the mark is read first: slots read after it are the final ones).
            for (uint32_t poll = 0; poll < kFollowLimit && *(volatile int *)&done_s == 0; ++poll) {
                const int fin = ld_acquire(table_g + kSlotTableSlots);
                g = j < k ? ld_visible(table_g + j) : 0;
                table_s[j] = (unsigned)g < (unsigned)G ? g : 0;
                if (fin != 0) {
                    __threadfence_block();
                    __syncwarp();
                    if (j == 0) *(volatile int *)&final_s = 1;
                    break;
                }
            }
            return;
        }
    }
    const int chunks = d / E;                                       // chunks per row
    const int nseg = (chunks + kUnitChunks * 32 - 1) / (kUnitChunks * 32);
    const int nunits = nrows * nseg;
    if constexpr (!SPEC) {
        // L2 warm-up (launched behind the sketch-and-recovery kernel, which triggers on its FIRST iterate):
        // before the wait for the final support, every CTA asks L2 for its share of the weight blocks of the
        // groups in the first iterate's slot table — nine tenths of them are in the final support, and HBM
        // streams them while the remaining iterations run.  Only a hint: whatever the table holds at this
        // moment, nothing but the range check stands between it and the request, and the pass below reads
        // the final support as always.
        if (warm != nullptr && tid < 3 * k) {
            const int mat = tid / k, j = tid - mat * k;
            const size_t chunk = ((size_t)d << lb) * sizeof(WT);            // one group's rows are contiguous
            const size_t seg = ((chunk / nx) + 127) & ~(size_t)127;         // this CTA's share of each block
            const size_t off = (size_t)bx * seg;
            const int g = ld_visible(warm + (size_t)t * kSlotTablePitch + j);
            if ((unsigned)g < (unsigned)G && off < chunk) {
                const char *src = reinterpret_cast<const char *>(mat == 0 ? Wg : mat == 1 ? Wu : Wdt) + (size_t)g * chunk + off;
                const uint32_t bytes = (uint32_t)min(seg, chunk - off);
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
            }
        }
        pdl_wait();   // supports and activations come from the kernels before
    }

    if constexpr (!SPEC) {
        if (tid < nrows) {
            const int R = bx + nx * tid;
            // A group index outside [0, G) must not become an address: the row is read from group 0
            // instead, its activation is forced to zero, and the call's status word (if any) says so.
            int g = ld_dep(support + (size_t)t * k + (R >> lb));
            const bool bad = (unsigned)g >= (unsigned)G;
            if (bad) {
                g = 0;
                if (status != nullptr) atomicCAS(&status->code, 0, (int)CS_ERR_SUPPORT);
            }
            bad_s[tid] = bad;
            chan_s[tid] = (g << lb) + (R & (b - 1));
        }
        if (check && bx == 0 && status != nullptr && tid >= kGatherThreads - kMaxG && tid - (kGatherThreads - kMaxG) < k) {
            // the last warps of the first CTA check the row: ascending, hence distinct (the range is checked above)
            const int j = tid - (kGatherThreads - kMaxG);
            if (j > 0 && ld_dep(support + (size_t)t * k + j) <= ld_dep(support + (size_t)t * k + j - 1))
                atomicCAS(&status->code, 0, (int)CS_ERR_SUPPORT);
        }
        __syncthreads();
    }
    volatile const int *table = table_s;               // SPEC: the slot table as the following warp last saw it

    uint4 *wring = ring + (size_t)warp * (kWarpRing / 16) + lane;   // this lane's column of the warp ring
    // ---- gate / up: units u = warp, warp + 16, ... ; unit u = (row u / nseg, segment u % nseg).
    // Two cursors (copy issue, consumption) walk the units incrementally: no division in the loop.
    const int step_r = kGatherWarps / nseg, step_s = kGatherWarps % nseg;
    struct Cursor { int u, r, seg; };
    auto advance = [&](Cursor &c) {
        c.u += kGatherWarps; c.r += step_r; c.seg += step_s;
        if (c.seg >= nseg) { c.seg -= nseg; ++c.r; }
    };
    Cursor ci{warp, warp / nseg, warp % nseg}, cc = ci;
    const WT *wg_lane = Wg + lane * E, *wu_lane = Wu + lane * E;
    const float *h_lane = h + (size_t)t * d + lane * E;

    // requests the gate and up chunks of unit (r, seg) into ring stage `stage`; settled: the final
    // rows (chan_s) are known, otherwise (SPEC) the row's group is read from the table and remembered
    auto request_unit = [&](int r, int seg, int stage, bool settled) {
        int chan;
        if (SPEC && !settled) {
            const int R = bx + nx * r;
            const int grp = table[R >> lb];
            if (lane == 0) ugrp_s[r][seg] = (short)grp;
            chan = (grp << lb) + (R & (b - 1));
        } else {
            chan = chan_s[r];
        }
        const size_t off = (size_t)chan * d + (size_t)seg * kSegElems;
        const WT *pg = wg_lane + off, *pu = wu_lane + off;
        uint4 *dst = wring + stage * (2 * kUnitChunks * 32);
#pragma unroll
        for (int j = 0; j < kUnitChunks; ++j) {
            if (FULL || (seg * kUnitChunks + j) * 32 + lane < chunks) {
                cp_async16(dst + j * 32, pg + j * 32 * E);
                cp_async16(dst + (kUnitChunks + j) * 32, pu + j * 32 * E);
            }
        }
    };
    auto issue_unit = [&](int stage) {
        if (ci.u < nunits) request_unit(ci.r, ci.seg, stage, false);
        cp_async_commit();  // one group per unit, empty past the end, so the wait count stays fixed
        advance(ci);
    };
    // When the number of segments divides the number of warps, a warp meets the same segment in every
    // unit and its slice of h is loaded once; otherwise it is fetched (from L1) per unit.
    const bool fixed_seg = kGatherWarps % nseg == 0;
    float hv[kUnitChunks][E];
    auto load_h = [&](int seg) {
        const float *hp = h_lane + seg * kSegElems;
#pragma unroll
        for (int j = 0; j < kUnitChunks; ++j) {
#pragma unroll
            for (int e = 0; e < E; e += 4) {
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (FULL || (seg * kUnitChunks + j) * 32 + lane < chunks) v = ld_dep4(hp + j * 32 * E + e);
                hv[j][e] = v.x; hv[j][e + 1] = v.y; hv[j][e + 2] = v.z; hv[j][e + 3] = v.w;
            }
        }
    };
    // dot products of the unit in ring stage `stage` with the h slice in hv; lane 0 files them under (r, seg)
    auto fold_unit = [&](int r, int seg, int stage) {
        const uint4 *src = wring + stage * (2 * kUnitChunks * 32);
        float g = 0.f, up = 0.f;
#pragma unroll
        for (int j = 0; j < kUnitChunks; ++j) {
            if (FULL || (seg * kUnitChunks + j) * 32 + lane < chunks) {
                float wg[E], wu[E];
                Chunk<WT>::widen(src[j * 32], wg);
                Chunk<WT>::widen(src[(kUnitChunks + j) * 32], wu);
#pragma unroll
                for (int e = 0; e < E; ++e) { g = fmaf(wg[e], hv[j][e], g); up = fmaf(wu[e], hv[j][e], up); }
            }
        }
        return make_float2(g, up);
    };
    if (fixed_seg) load_h(cc.seg);
    if constexpr (SPEC) bar_sync<2, kSpecThreads>();   // the table copy holds (at least) the first iterate's support
#pragma unroll
    for (int i = 0; i < kUnitStages; ++i) issue_unit(i);
    int stage = 0;
#pragma unroll 1
    for (; cc.u < nunits; advance(cc)) {
        if (!fixed_seg) load_h(cc.seg);
        cp_async_wait<kUnitStages - 1>();
        float2 gu = fold_unit(cc.r, cc.seg, stage);
        issue_unit(stage);  // refill the stage just consumed (its values were used above)
        stage = stage + 1 == kUnitStages ? 0 : stage + 1;
        gu.x = warp_sum(gu.x); gu.y = warp_sum(gu.y);
        if (lane == 0) { red[cc.r][cc.seg][0] = gu.x; red[cc.r][cc.seg][1] = gu.y; }
    }
    cp_async_wait<0>();

    if constexpr (SPEC) {
        cta_sync();
        const bool settled = *(volatile int *)&final_s != 0;   // the copy in shared memory is the final table
        if (tid == 0) *(volatile int *)&done_s = 1;            // the following warp may leave
        if (!settled) pdl_wait();   // else: the launch before has completed, so the table in global memory is final
        if (tid < nrows) {
            const int R = bx + nx * tid;
            int g = settled ? table[R >> lb] : ld_visible(support + (size_t)t * kSlotTablePitch + (R >> lb));
            if ((unsigned)g >= (unsigned)G) g = 0;   // a recovery always leaves valid groups; never an address otherwise
            bad_s[tid] = 0;
            chan_s[tid] = (g << lb) + (R & (b - 1));
        }
        cta_sync();
        // Units that were requested for a group that has since left its slot are fetched and folded once
        // more.  (Few: the rows requested early belong to the largest entries of the first iterate.)  They
        // are listed and dealt out over the warps, one per warp and round, and a round's request goes out
        // AHEAD of the down rows, into the ring stage the down rows leave free.
        if (tid == 0) nstale_s = 0;
        cta_sync();
        for (Cursor c{warp, warp / nseg, warp % nseg}; c.u < nunits; advance(c))
            if (lane == 0 && (int)ugrp_s[c.r][c.seg] != (chan_s[c.r] >> lb)) stale_s[atomicAdd(&nstale_s, 1)] = (short)c.u;
        cta_sync();
    }
    constexpr int kRedoStage = kUnitStages - 1;                       // the last unit stage = the last 8 lane slots
    constexpr int DRS = SPEC ? (kLaneSlots - 2 * kUnitChunks) / CPT : DR;   // down rows in flight beside it
    static_assert(DRS >= 1, "a down row must fit beside the stage kept for stale units");
    int nstale = 0, redo_u = -1;
    if constexpr (SPEC) {
        nstale = nstale_s;
        if (warp < nstale) {
            redo_u = stale_s[warp];
            load_h(redo_u % nseg);
            request_unit(redo_u / nseg, redo_u % nseg, kRedoStage, true);
        }
        cp_async_commit();
    }

    // ---- down rows: thread i owns chunks i, i + 512, ... of every row; lane slots of the warp ring
    const WT *wd_thread = Wdt + tid * E;
    int issue_r = 0, issue_stage = 0;
    auto issue_down = [&]() {
        if (issue_r < nrows) {
            const WT *p = wd_thread + (size_t)chan_s[issue_r] * d;
            uint4 *dst = wring + issue_stage * (CPT * 32);
#pragma unroll
            for (int j = 0; j < CPT; ++j)
                if (FULL || tid + j * kGatherThreads < chunks) cp_async16(dst + j * 32, p + j * kGatherThreads * E);
        }
        cp_async_commit();
        ++issue_r;
        issue_stage = issue_stage + 1 == DRS ? 0 : issue_stage + 1;
    };
#pragma unroll 1
    for (int r = 0; r < DRS; ++r) issue_down();

    if constexpr (SPEC) {
        auto finish_unit = [&](int u) {
            const int r = u / nseg, seg = u % nseg;
            float2 gu = fold_unit(r, seg, kRedoStage);
            gu.x = warp_sum(gu.x); gu.y = warp_sum(gu.y);
            if (lane == 0) { red[r][seg][0] = gu.x; red[r][seg][1] = gu.y; }
        };
        if (redo_u >= 0) {
            cp_async_wait<DRS>();   // the stale unit's group is older than the down rows'
            finish_unit(redo_u);
        }
        // more stale units than warps (rare): the rest one at a time, each behind the down rows already in flight
#pragma unroll 1
        for (int i = warp + kGatherWarps; i < nstale; i += kGatherWarps) {
            const int u = stale_s[i];
            load_h(u % nseg);
            request_unit(u / nseg, u % nseg, kRedoStage, true);
            cp_async_commit();
            cp_async_wait<0>();
            finish_unit(u);
        }
    }

    cta_sync();
    if (tid < nrows) {
        float g = 0.f, up = 0.f;
        for (int sgm = 0; sgm < nseg; ++sgm) { g += red[tid][sgm][0]; up += red[tid][sgm][1]; }
        a_s[tid] = bad_s[tid] ? 0.f : silu(g) * up;
    }
    cta_sync();

    float acc[CPT][E];
#pragma unroll
    for (int j = 0; j < CPT; ++j)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[j][e] = 0.f;
    stage = 0;
#pragma unroll 1
    for (int r = 0; r < nrows; ++r) {
        cp_async_wait<DRS - 1>();
        const uint4 *src = wring + stage * (CPT * 32);
        const float a = a_s[r];
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
            if (FULL || tid + j * kGatherThreads < chunks) {
                float w[E];
                Chunk<WT>::widen(src[j * 32], w);
#pragma unroll
                for (int e = 0; e < E; ++e) acc[j][e] = fmaf(a, w[e], acc[j][e]);
            }
        }
        issue_down();
        stage = stage + 1 == DRS ? 0 : stage + 1;
    }
    cp_async_wait<0>();
    // SPEC: nothing is written, and this launch does not end, before the launch that runs the recovery has
    // completed (its outputs, and the scratch the next step will reuse)
    if constexpr (SPEC) pdl_wait();
    float *dst = partial + ((size_t)t * nx + blockIdx.x) * d + tid * E;
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
        if (FULL || tid + j * kGatherThreads < chunks) {
#pragma unroll
            for (int e = 0; e < E; e += 4)
                *reinterpret_cast<float4 *>(dst + j * kGatherThreads * E + e) =
                    make_float4(acc[j][e], acc[j][e + 1], acc[j][e + 2], acc[j][e + 3]);
        }
    }
}

// out[t, :] = residual[t, :] + sum_{p < nx} partial[t, p, :], p ascending within fixed groups.
// CTA = kReduceCols float4 columns x kReduceGroups partial groups; a thread sums the partials p with
// p % kReduceGroups == its group, then the groups are folded in index order through shared memory.
// Small CTAs (256 threads, few registers) on purpose: under programmatic dependent launch they fit
// on the SMs beside the gather kernel's CTAs and are in place when its last partial lands.
constexpr int kReduceCols = 8;
__global__ void __launch_bounds__(kReduceCols * kReduceGroups)
reduce_partials_kernel(const float *__restrict__ partial, int nx, int d, const float *__restrict__ residual,
                       float *__restrict__ out) {
    __shared__ float4 fold[kReduceGroups][kReduceCols];
    const int t = blockIdx.y;
    const int cl = threadIdx.x & (kReduceCols - 1);
    const int col = blockIdx.x * kReduceCols + cl;          // float4 column
    const int grp = threadIdx.x / kReduceCols;
    const int cols = d >> 2;
    pdl_launch_dependents();
    pdl_wait();
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    // everything this thread needs is requested in one go after the wait: the residual (first group only)
    // and its partials p = grp, grp + 32, ..., eight at a time, added in index order
    float4 res = make_float4(0.f, 0.f, 0.f, 0.f);
    if (col < cols) {
        if (grp == 0 && residual != nullptr) res = ld_dep4(residual + (size_t)t * d + 4 * (size_t)col);
        const float4 *src = reinterpret_cast<const float4 *>(partial + (size_t)t * nx * d) + col;
        for (int p0 = grp; p0 < nx; p0 += 8 * kReduceGroups) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int p = p0 + u * kReduceGroups;
                v[u] = p < nx ? ld_dep4(reinterpret_cast<const float *>(src + (size_t)p * cols)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) { s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w; }
        }
    }
    fold[grp][cl] = s;
    __syncthreads();
    if (grp == 0 && col < cols) {
        float4 r = res;
#pragma unroll
        for (int g = 0; g < kReduceGroups; ++g) {
            const float4 v = fold[g][cl];
            r.x += v.x; r.y += v.y; r.z += v.z; r.w += v.w;
        }
        reinterpret_cast<float4 *>(out + (size_t)t * d)[col] = r;
    }
}

// Device-side validation of supports (ascending, distinct, in range); records CS_ERR_SUPPORT.
__global__ void check_support_kernel(const int32_t *__restrict__ support, int B, int k, int G,
                                     DeviceStatus *status) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= B) return;
    int prev = -1;
    bool ok = true;
    for (int c = 0; c < k; ++c) {
        const int g = support[(size_t)t * k + c];
        ok = ok && g > prev && g < G;
        prev = g;
    }
    if (!ok) atomicCAS(&status->code, 0, (int)CS_ERR_SUPPORT);
}

cs_status launch_check_support(cs_plan *plan, const int32_t *support, int B, cudaStream_t st) {
    check_support_kernel<<<(B + 127) / 128, 128, 0, st>>>(support, B, plan->cfg.k, plan->G, plan->status);
    plan->launches++;
    CS_CUDA_TRY(plan, cudaGetLastError());
    return CS_OK;
}

// Picks the instantiation: chunks per thread in the down phase, and whether rows need bounds checks.
template <typename WT, bool SPEC>
static void launch_gather_kernel(dim3 grid, cudaStream_t st, int cpt, int chunks, const WT *Wg, const WT *Wu,
                                 const WT *Wd, const float *h, const int32_t *sup, int d, int b, int k, int G,
                                 float *partial, DeviceStatus *status, int check, const int32_t *warm) {
    const bool full = chunks % kGatherThreads == 0 && (cpt == 1 || cpt == 2 || cpt == 4);
    const int lb = b == 64 ? 6 : 7;
#define CS_GATHER_CASE(N, F)                                                                              \
    launch_pdl(true, ffn_gather_kernel<WT, N, F, SPEC>, grid, dim3(SPEC ? kSpecThreads : kGatherThreads), kRingBytes, st, \
               Wg, Wu, Wd, h, sup, d, lb, k, G, partial, status, check, warm)
    if (cpt <= 1) { if (full) CS_GATHER_CASE(1, true); else CS_GATHER_CASE(1, false); }
    else if (cpt <= 2) { if (full) CS_GATHER_CASE(2, true); else CS_GATHER_CASE(2, false); }
    else { if (full) CS_GATHER_CASE(4, true); else CS_GATHER_CASE(4, false); }
#undef CS_GATHER_CASE
}

// CTAs per token: one CTA per SM when a single token is in flight, never more than kGatherMaxRows rows per CTA.
static int gather_nx(int sm_count, int nb, int rows_total, int nx_max) {
    int nx = max(sm_count / nb, (rows_total + kGatherMaxRows - 1) / kGatherMaxRows);
    return max(1, min(nx, min(rows_total, nx_max)));
}

// spec: `support` is the slot table of a recovery that is still running (the small-batch step), and one SM
// per token is left to the CTA that runs it; otherwise the supports are given (`check`: validate them).
template <typename WT>
static cs_status gather_typed(cs_plan *plan, const cs_layer *L, const float *h, const int32_t *support,
                              int B, const float *residual, float *out, int check, bool spec, cudaStream_t st,
                              const int32_t *warm = nullptr) {
    const cs_config &c = plan->cfg;
    constexpr int E = Chunk<WT>::kElems;
    const int rows_total = c.k * c.group;
    const int cpt = (c.d / E + kGatherThreads - 1) / kGatherThreads;
    const WT *Wg = static_cast<const WT *>(L->W_gate), *Wu = static_cast<const WT *>(L->W_up),
             *Wd = static_cast<const WT *>(L->Wd_t);
    for (int t0 = 0; t0 < B; t0 += kGatherMaxTokens) {
        const int nb = min(kGatherMaxTokens, B - t0);
        const int nx = gather_nx(spec ? plan->sm_count - nb : plan->sm_count, nb, rows_total, plan->nx_max);
        dim3 grid(nx, nb);
        const float *hp = h + (size_t)t0 * c.d;
        {
            StageTimer timer(plan, CS_STAGE_EXEC, st);
            if (spec)
                launch_gather_kernel<WT, true>(grid, st, cpt, c.d / E, Wg, Wu, Wd, hp, support + (size_t)t0 * kSlotTablePitch,
                                               c.d, c.group, c.k, plan->G, plan->partial, plan->status, 0, nullptr);
            else
                launch_gather_kernel<WT, false>(grid, st, cpt, c.d / E, Wg, Wu, Wd, hp, support + (size_t)t0 * c.k, c.d,
                                                c.group, c.k, plan->G, plan->partial, plan->status, check,
                                                warm != nullptr ? warm + (size_t)t0 * kSlotTablePitch : nullptr);
        }
        plan->launches++;
        CS_CUDA_TRY(plan, cudaGetLastError());
        dim3 rgrid((c.d / 4 + kReduceCols - 1) / kReduceCols, nb);
        {
            StageTimer timer(plan, CS_STAGE_REDUCE, st);
            launch_pdl(true, reduce_partials_kernel, rgrid, dim3(kReduceCols * kReduceGroups), 0, st, (const float *)plan->partial, nx,
                       c.d, residual ? residual + (size_t)t0 * c.d : (const float *)nullptr, out + (size_t)t0 * c.d);
        }
        plan->launches++;
        CS_CUDA_TRY(plan, cudaGetLastError());
    }
    return CS_OK;
}

// The ring needs more dynamic shared memory than the default limit: opt in once per kernel.
template <typename WT, int N>
static cudaError_t gather_attrs(bool fused_too) {
    cudaError_t e = cudaFuncSetAttribute(ffn_gather_kernel<WT, N, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(ffn_gather_kernel<WT, N, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes);
    if (e == cudaSuccess && fused_too)
        e = cudaFuncSetAttribute(ffn_gather_kernel<WT, N, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes);
    if (e == cudaSuccess && fused_too)
        e = cudaFuncSetAttribute(ffn_gather_kernel<WT, N, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes);
    return e;
}
static cudaError_t gather_attrs_all(bool fused_too) {
    cudaError_t e = gather_attrs<__nv_bfloat16, 1>(fused_too);
    if (e == cudaSuccess) e = gather_attrs<__nv_bfloat16, 2>(fused_too);
    if (e == cudaSuccess) e = gather_attrs<__nv_bfloat16, 4>(fused_too);
    if (e == cudaSuccess) e = gather_attrs<float, 1>(fused_too);
    if (e == cudaSuccess) e = gather_attrs<float, 2>(fused_too);
    if (e == cudaSuccess) e = gather_attrs<float, 4>(fused_too);
    return e;
}

cs_status prepare_ffn_gather(cs_plan *plan) {
    CS_CUDA_TRY(plan, gather_attrs_all(true));
    return CS_OK;
}

cs_status launch_ffn_gather(cs_plan *plan, const cs_layer *layer, const float *h, const int32_t *support,
                            int B, const float *residual, float *out, bool check, cudaStream_t st, const int32_t *warm) {
    if (plan->cfg.w_dtype == CS_BF16)
        return gather_typed<__nv_bfloat16>(plan, layer, h, support, B, residual, out, check, false, st, warm);
    return gather_typed<float>(plan, layer, h, support, B, residual, out, check, false, st, warm);
}

// The gather FFN behind launch_sketch_recover: starts on the recovery's first slot table (plan->slot_table).
cs_status launch_ffn_gather_spec(cs_plan *plan, const cs_layer *layer, const float *h, int B, const float *residual,
                                 float *out, cudaStream_t st) {
    if (plan->cfg.w_dtype == CS_BF16)
        return gather_typed<__nv_bfloat16>(plan, layer, h, plan->slot_table, B, residual, out, 0, true, st);
    return gather_typed<float>(plan, layer, h, plan->slot_table, B, residual, out, 0, true, st);
}


// ---- cs_ffn_exec_static: the same gather FFN for callers that must not allocate ------------------
//
// The partial down-projections normally live in scratch a plan allocates with cudaMalloc.  This
// entry point instead keeps them in the fixed array below, which is part of the library image: each
// GPU that loads the library carries these 8 MiB until the process exits, and no call ever
// allocates or frees anything.
constexpr size_t kStaticScratchBytes = 8u << 20;
static __device__ __align__(256) unsigned char g_static_partial[kStaticScratchBytes];

constexpr int kStaticMaxDevices = 64;
static float *g_static_ptr[kStaticMaxDevices];   // device address of g_static_partial, per device
static int g_static_sms[kStaticMaxDevices];

// Once per device, with that device current: look up where the array lives on the GPU (its name
// in host code is only a handle, not an address a kernel could use) and opt the kernels in to the
// shared-memory ring.  Neither call allocates.
static cudaError_t static_setup(int dev) {
    if (g_static_ptr[dev] != nullptr) return cudaSuccess;
    void *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_partial);
    if (e != cudaSuccess) return e;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (e == cudaSuccess) e = gather_attrs_all(false);
    if (e != cudaSuccess) return e;
    g_static_sms[dev] = sms;
    g_static_ptr[dev] = static_cast<float *>(p);
    return cudaSuccess;
}

template <typename WT>
static cudaError_t static_launch(const cs_config &c, const cs_layer *L, const float *h, const int32_t *support,
                                 int B, int nx, float *partial, const float *residual, float *out,
                                 cudaStream_t st) {
    constexpr int E = Chunk<WT>::kElems;
    const int cpt = (c.d / E + kGatherThreads - 1) / kGatherThreads;
    const WT *Wg = static_cast<const WT *>(L->W_gate), *Wu = static_cast<const WT *>(L->W_up),
             *Wd = static_cast<const WT *>(L->Wd_t);
    dim3 grid(nx, B);
    launch_gather_kernel<WT, false>(grid, st, cpt, c.d / E, Wg, Wu, Wd, h, support, c.d, c.group, c.k, c.d_ff / c.group,
                                    partial, static_cast<DeviceStatus *>(nullptr), 0, nullptr);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    dim3 rgrid((c.d / 4 + kReduceCols - 1) / kReduceCols, B);
    reduce_partials_kernel<<<rgrid, kReduceCols * kReduceGroups, 0, st>>>(partial, nx, c.d, residual, out);
    return cudaGetLastError();
}

}  // namespace cs

extern "C" cs_status cs_ffn_exec_static(const cs_config *cfg, const cs_layer *layer, const float *h,
                                        const int32_t *support, int32_t B, const float *residual, float *out,
                                        void *stream) {
    using namespace cs;
    if (cfg == nullptr || layer == nullptr || h == nullptr || support == nullptr || out == nullptr) return CS_ERR_NULL;
    if (layer->W_gate == nullptr || layer->W_up == nullptr || layer->Wd_t == nullptr) return CS_ERR_NULL;
    if (cfg->d <= 0 || cfg->group <= 0 || cfg->k <= 0 || cfg->d_ff <= 0 || cfg->d_ff % cfg->group != 0 ||
        cfg->k > cfg->d_ff / cfg->group || B <= 0)
        return CS_ERR_SHAPE;
    if ((cfg->group != 64 && cfg->group != 128) || cfg->d > kMaxD || cfg->d % 64 != 0 ||
        cfg->d_ff / cfg->group > kMaxG || (cfg->w_dtype != CS_F32 && cfg->w_dtype != CS_BF16))
        return CS_ERR_UNSUPPORTED;
    // the kernels move 16-byte chunks: the same alignment rule as cs_ffn_exec, checked before anything runs
    auto misaligned = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (misaligned(layer->W_gate) || misaligned(layer->W_up) || misaligned(layer->Wd_t) || misaligned(h) ||
        misaligned(out) || (residual != nullptr && misaligned(residual)))
        return CS_ERR_UNSUPPORTED;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return CS_ERR_CUDA;
    if (static_setup(dev) != cudaSuccess) return CS_ERR_CUDA;
    // B * nx partial vectors of d floats must fit the fixed array; nx may shrink down to the point
    // where a CTA would own more than kGatherMaxRows rows, beyond that the request is too large.
    const int rows_total = cfg->k * cfg->group;
    const int nx_min = (rows_total + kGatherMaxRows - 1) / kGatherMaxRows;
    const size_t per_vec = (size_t)cfg->d * sizeof(float);
    const size_t fit = kStaticScratchBytes / (per_vec * (size_t)B);
    if (fit < (size_t)nx_min) return CS_ERR_SHAPE;
    int nx = max(g_static_sms[dev] / B, nx_min);
    nx = (int)min((size_t)min(nx, rows_total), fit);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cfg->w_dtype == CS_BF16
        ? static_launch<__nv_bfloat16>(*cfg, layer, h, support, B, nx, g_static_ptr[dev], residual, out, st)
        : static_launch<float>(*cfg, layer, h, support, B, nx, g_static_ptr[dev], residual, out, st);
    return e == cudaSuccess ? CS_OK : CS_ERR_CUDA;
}
