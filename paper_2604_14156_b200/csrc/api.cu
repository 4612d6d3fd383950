// The C boundary: plan life cycle, host-side validation and dispatch.  See include/cs.h.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "cs_internal.cuh"

namespace cs {

cs_status record_cuda(cs_plan *plan, cudaError_t e, const char *what) {
    if (plan != nullptr)
        snprintf(plan->cuda_error, sizeof plan->cuda_error, "%s: %s", what, cudaGetErrorString(e));
    return CS_ERR_CUDA;
}

static cs_status check_config(const cs_config *c) {
    if (c->d <= 0 || c->d_ff <= 0 || c->group <= 0 || c->m <= 0 || c->k <= 0 || c->T < 0 || c->max_tokens <= 0)
        return CS_ERR_SHAPE;
    if (c->d_ff % c->group != 0) return CS_ERR_SHAPE;
    const int G = c->d_ff / c->group;
    if (c->k > G) return CS_ERR_SHAPE;
    if (!(c->rms_eps > 0.f) || !isfinite(c->rms_eps)) return CS_ERR_NONFINITE;
    if (c->group != 64 && c->group != 128) return CS_ERR_UNSUPPORTED;
    if (G > kMaxG || c->m > kMaxM || c->d > kMaxD || c->d % 64 != 0) return CS_ERR_UNSUPPORTED;
    if (c->w_dtype != CS_F32 && c->w_dtype != CS_BF16) return CS_ERR_UNSUPPORTED;
    return CS_OK;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace cs

using namespace cs;

// Device-visible address of page-locked host memory (unified addressing), or NULL for pageable memory.
static void *device_alias(const void *host) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
}

constexpr size_t kZeroCopyBytes = 64 * 1024;
constexpr size_t kZeroCopyBytesLarge = 4 * 1024 * 1024;

// x (page-locked host memory) -> plan scratch.  Both the load and the store come after the
// programmatic-launch wait: whatever ran before on the stream may have written the host buffer (a
// previous step that stored its result there, when layers are chained through one buffer) and may
// still be reading the scratch copy.
__global__ void __launch_bounds__(256) stage_in_kernel(const float4 *src, float4 *dst, int n4) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    cs::pdl_launch_dependents();
    cs::pdl_wait();
    if (i < n4) {
        float4 v;   // volatile and uncached: the host (or the step before) rewrites the buffer between steps
        asm volatile("ld.volatile.global.v4.f32 {%0, %1, %2, %3}, [%4];"
                     : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(src + i) : "memory");
        dst[i] = v;
    }
}

extern "C" {

cs_status cs_plan_create(const cs_config *cfg, cs_plan **out) {
    if (cfg == nullptr || out == nullptr) return CS_ERR_NULL;
    cs_status s = check_config(cfg);
    if (s != CS_OK) return s;
    cs_plan *p = new (std::nothrow) cs_plan();
    if (p == nullptr) return CS_ERR_CUDA;
    memset(p, 0, sizeof *p);
    p->cfg = *cfg;
    p->G = cfg->d_ff / cfg->group;
    cudaError_t e = cudaGetDevice(&p->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
    const size_t nt = (size_t)cfg->max_tokens;
    p->nx_max = max(p->sm_count, (cfg->k * cfg->group + kGatherMaxRows - 1) / kGatherMaxRows);
    p->mean_row_blocks = 32;
    auto alloc = [&](void **ptr, size_t bytes) {
        if (e == cudaSuccess) e = cudaMalloc(ptr, bytes);
    };
    alloc((void **)&p->n_buf, nt * cfg->d * sizeof(float));
    alloc((void **)&p->y_buf, nt * cfg->m * sizeof(float));
    alloc((void **)&p->sup_buf, nt * cfg->k * sizeof(int32_t));
    alloc((void **)&p->partial, (size_t)kGatherMaxTokens * p->nx_max * cfg->d * sizeof(float));
    alloc((void **)&p->gram, (size_t)kMaxG * kMaxG * sizeof(float));
    alloc((void **)&p->resid_buf, nt * sizeof(float));
    alloc((void **)&p->fb_flags, nt * sizeof(int32_t));
    alloc((void **)&p->fb_list, nt * sizeof(int32_t));
    alloc((void **)&p->fb_count, sizeof(int32_t));
    alloc((void **)&p->slot_table, nt * kSlotTablePitch * sizeof(int32_t));
    alloc((void **)&p->ticket, nt * sizeof(unsigned));
    alloc((void **)&p->hbar, (size_t)cfg->d * sizeof(float));
    alloc((void **)&p->colsum, (size_t)p->mean_row_blocks * cfg->d * sizeof(float));
    alloc((void **)&p->status, sizeof(DeviceStatus));
    p->mma_ok = cfg->w_dtype == CS_BF16 && cfg->group == 128 && cfg->d % 256 == 0;
    // The gather path streams B * k groups, the tensor-core path every group once: it takes over where
    // the first exceeds the second by the ~15 % the GEMM path costs extra (measured crossover between
    // 4 and 5 tokens at G / k = 3.9).
    p->mma_min_tokens = max(2, min(kMmaMinTokens, (int)ceilf(1.15f * (float)p->G / (float)cfg->k)));
    alloc((void **)&p->mask, nt * 4 * sizeof(uint32_t));
    alloc((void **)&p->gmask, (size_t)kMaxG * 4 * sizeof(uint32_t));
    alloc((void **)&p->counts, (size_t)kMaxG * sizeof(int32_t));
    alloc((void **)&p->offsets, (size_t)(kMaxG + 1) * sizeof(int32_t));
    alloc((void **)&p->token_ids, nt * cfg->k * sizeof(int32_t));
    alloc((void **)&p->glist, (size_t)kMaxG * sizeof(int32_t));
    alloc((void **)&p->nu, sizeof(int32_t));
    if (p->mma_ok) {
        const size_t m_pad = (nt + 127) / 128 * 128;
        p->mma_slices = max(1, min(16, p->sm_count / max(1, cfg->d / 256)));
        alloc((void **)&p->x_bf16, 2 * nt * cfg->d * 2);
        alloc((void **)&p->act, 2 * max(nt, (size_t)128) * cfg->d_ff * 2);
        // slices * padded tokens never exceeds 128 * (SMs / column tiles): see launch_ffn_mma
        const size_t slice_rows = (size_t)128 * (p->sm_count / max(1, cfg->d / 256) + 1);
        alloc((void **)&p->mma_partial, max(slice_rows, m_pad) * cfg->d * sizeof(float));
    }
    alloc((void **)&p->x_host_in, nt * cfg->d * sizeof(float));
    alloc((void **)&p->x_host_out, nt * cfg->d * sizeof(float));
    for (int i = 0; i < 2 * CS_STAGE_COUNT; ++i)
        if (e == cudaSuccess) e = cudaEventCreate(&p->ev[i]);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->side, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_join, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaMemset(p->status, 0, sizeof(DeviceStatus));
    if (e == cudaSuccess) e = cudaMemset(p->ticket, 0, nt * sizeof(unsigned));
    if (e == cudaSuccess) e = cudaMemset(p->slot_table, 0, nt * kSlotTablePitch * sizeof(int32_t));
    if (e == cudaSuccess && prepare_sketch(p) != CS_OK) e = cudaErrorUnknown;
    if (e == cudaSuccess && prepare_solvers(p) != CS_OK) e = cudaErrorUnknown;
    if (e == cudaSuccess && prepare_ffn_gather(p) != CS_OK) e = cudaErrorUnknown;
    if (e == cudaSuccess && p->mma_ok && prepare_ffn_mma(p) != CS_OK) e = cudaErrorUnknown;
    if (e != cudaSuccess) {
        cs_plan_destroy(p);
        return CS_ERR_CUDA;
    }
    *out = p;
    return CS_OK;
}

cs_status cs_plan_destroy(cs_plan *p) {
    if (p == nullptr) return CS_ERR_NULL;
    cudaFree(p->n_buf); cudaFree(p->y_buf); cudaFree(p->sup_buf);
    cudaFree(p->partial); cudaFree(p->gram); cudaFree(p->slot_table); cudaFree(p->ticket);
    cudaFree(p->resid_buf); cudaFree(p->fb_flags); cudaFree(p->fb_list); cudaFree(p->fb_count); cudaFree(p->hbar); cudaFree(p->colsum);
    cudaFree(p->status); cudaFree(p->x_host_in); cudaFree(p->x_host_out);
    cudaFree(p->mask); cudaFree(p->gmask); cudaFree(p->counts); cudaFree(p->offsets); cudaFree(p->token_ids); cudaFree(p->glist);
    cudaFree(p->nu); cudaFree(p->x_bf16); cudaFree(p->act); cudaFree(p->mma_partial);
    for (int i = 0; i < 2 * CS_STAGE_COUNT; ++i)
        if (p->ev[i] != nullptr) cudaEventDestroy(p->ev[i]);
    if (p->ev_fork != nullptr) cudaEventDestroy(p->ev_fork);
    if (p->ev_join != nullptr) cudaEventDestroy(p->ev_join);
    if (p->side != nullptr) cudaStreamDestroy(p->side);
    delete p;
    return CS_OK;
}

cs_status cs_sketch(cs_plan *plan, const float *S, const float *h, int32_t B, float *y, void *stream) {
    if (plan == nullptr || S == nullptr || h == nullptr || y == nullptr) return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    if (!aligned16(S) || !aligned16(h)) return CS_ERR_UNSUPPORTED;
    return launch_sketch(plan, S, h, nullptr, B, y, nullptr, nullptr, 0.f, static_cast<cudaStream_t>(stream));
}

cs_status cs_recover(cs_plan *plan, const float *Phi, float mu, const float *y, int32_t B,
                     int32_t *support, float *z, float *resid, void *stream) {
    if (plan == nullptr || Phi == nullptr || y == nullptr || support == nullptr) return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    if (!isfinite(mu) || !(mu > 0.f)) return CS_ERR_NONFINITE;
    return launch_recover(plan, Phi, mu, y, B, support, z, resid, false, static_cast<cudaStream_t>(stream));
}

cs_status cs_recover_warm(cs_plan *plan, const float *Phi, float mu, const float *y, int32_t B, int32_t T,
                          const int32_t *support0, const float *z0, int32_t *support, float *z, float *resid,
                          void *stream) {
    if (plan == nullptr || Phi == nullptr || y == nullptr || support0 == nullptr || z0 == nullptr || support == nullptr)
        return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens || T < 1) return CS_ERR_SHAPE;
    if (!isfinite(mu) || !(mu > 0.f)) return CS_ERR_NONFINITE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cs_status s = launch_check_support(plan, support0, B, st);
    if (s != CS_OK) return s;
    return launch_recover(plan, Phi, mu, y, B, support, z, resid, false, st, T, support0, z0);
}

cs_status cs_support_drift(cs_plan *plan, const int32_t *support_prev, const int32_t *support_cur, int32_t B,
                           int32_t *drift, void *stream) {
    if (plan == nullptr || support_prev == nullptr || support_cur == nullptr || drift == nullptr) return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cs_status s = launch_check_support(plan, support_prev, B, st);
    if (s == CS_OK) s = launch_check_support(plan, support_cur, B, st);
    if (s != CS_OK) return s;
    return launch_support_drift(plan, support_prev, support_cur, B, drift, nullptr, st);
}

cs_status cs_support_drift_ratio(cs_plan *plan, const int32_t *support_prev, const int32_t *support_cur, int32_t B,
                                 int32_t *delta, float *D, void *stream) {
    if (plan == nullptr || support_prev == nullptr || support_cur == nullptr || (delta == nullptr && D == nullptr))
        return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cs_status s = launch_check_support(plan, support_prev, B, st);
    if (s == CS_OK) s = launch_check_support(plan, support_cur, B, st);
    if (s != CS_OK) return s;
    return launch_support_drift(plan, support_prev, support_cur, B, delta, D, st);
}

static cs_status check_options(const cs_plan *plan, const cs_step_options *o, bool step) {
    if (o->solver != CS_SOLVER_IHT && o->solver != CS_SOLVER_NIHT && o->solver != CS_SOLVER_OMP) return CS_ERR_UNSUPPORTED;
    if (o->solver == CS_SOLVER_OMP && plan->cfg.k > 64) return CS_ERR_UNSUPPORTED;
    if (!isfinite(o->gamma) || o->gamma < 0.f) return CS_ERR_NONFINITE;
    const bool needs_prev = o->warm_start || o->gamma > 0.f;
    if (needs_prev && (o->support_prev == nullptr || o->z_prev == nullptr)) return CS_ERR_NULL;
    if ((o->delta_out != nullptr || o->drift_out != nullptr || (step && o->reuse_support)) && o->support_prev == nullptr)
        return CS_ERR_NULL;
    if ((o->warm_start || o->gamma > 0.f) && o->solver != CS_SOLVER_IHT) return CS_ERR_UNSUPPORTED;
    if (o->warm_start && o->T == 0) return CS_ERR_SHAPE;
    if ((o->srht_sign == nullptr) != (o->srht_rows == nullptr)) return CS_ERR_NULL;
    return CS_OK;
}

// The estimator an options struct asks for, on y; gram_ready: plan->gram holds this Phi's matrix.
static cs_status recover_with(cs_plan *plan, const float *Phi, float mu, const float *y, int B, const cs_step_options *o,
                              int32_t *support, float *z, float *resid, bool gram_ready, cudaStream_t st) {
    const int T = o->T < 0 ? plan->cfg.T : o->T;
    if (o->solver == CS_SOLVER_NIHT) return launch_niht(plan, Phi, mu, y, B, T, support, z, resid, st);
    if (o->solver == CS_SOLVER_OMP) return launch_omp(plan, Phi, y, B, support, z, resid, st);
    return launch_recover(plan, Phi, mu, y, B, support, z, resid, gram_ready, st, T,
                          o->warm_start ? o->support_prev : nullptr, o->warm_start ? o->z_prev : nullptr, o->gamma,
                          o->gamma > 0.f ? o->support_prev : nullptr, o->gamma > 0.f ? o->z_prev : nullptr);
}

cs_status cs_recover_ex(cs_plan *plan, const float *Phi, float mu, const float *y, int32_t B,
                        const cs_step_options *opt, int32_t *support, float *z, float *resid, void *stream) {
    if (opt == nullptr) return cs_recover(plan, Phi, mu, y, B, support, z, resid, stream);
    if (plan == nullptr || Phi == nullptr || y == nullptr || support == nullptr) return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    if (!isfinite(mu) || !(mu > 0.f)) return CS_ERR_NONFINITE;
    cs_status s = check_options(plan, opt, false);
    if (s != CS_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (opt->support_prev != nullptr) {
        s = launch_check_support(plan, opt->support_prev, B, st);
        if (s != CS_OK) return s;
    }
    s = recover_with(plan, Phi, mu, y, B, opt, support, z, resid, false, st);
    if (s != CS_OK) return s;
    if (opt->delta_out != nullptr || opt->drift_out != nullptr)
        s = launch_support_drift(plan, opt->support_prev, support, B, opt->delta_out, opt->drift_out, st);
    return s;
}

cs_status cs_sketch_srht(cs_plan *plan, const uint32_t *sign_bits, const int32_t *rows, const float *h, int32_t B,
                         float *y, void *stream) {
    if (plan == nullptr || sign_bits == nullptr || rows == nullptr || h == nullptr || y == nullptr) return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    return launch_sketch_srht(plan, sign_bits, rows, h, B, y, static_cast<cudaStream_t>(stream));
}

cs_status cs_uds_budget(cs_plan *plan, const float *logits, int32_t B, int32_t V, float m_base, float gamma,
                        int32_t m_min, int32_t m_max, float *H, int32_t *m_t, void *stream) {
    if (plan == nullptr || logits == nullptr || m_t == nullptr) return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens || V <= 0 || m_min < 1 || m_max < m_min) return CS_ERR_SHAPE;
    if (!isfinite(m_base) || !(m_base > 0.f) || !isfinite(gamma) || gamma < 0.f) return CS_ERR_NONFINITE;
    return launch_uds_budget(plan, logits, B, V, m_base, gamma, m_min, m_max, H, m_t, static_cast<cudaStream_t>(stream));
}

static cs_status check_weights(const cs_layer *L) {
    if (L == nullptr || L->W_gate == nullptr || L->W_up == nullptr || L->Wd_t == nullptr) return CS_ERR_NULL;
    if (!aligned16(L->W_gate) || !aligned16(L->W_up) || !aligned16(L->Wd_t)) return CS_ERR_UNSUPPORTED;
    return CS_OK;
}

extern "C++" {
static bool use_decode_mma(const cs_plan *plan, int B) { return plan->mma_ok && B >= plan->mma_min_tokens && B <= 128; }

// Tensor-core decode path from the crossover batch (mma_min_tokens) up to 128 tokens.  The gate/up
// GEMM needs no supports (at these batch sizes the union of the supports is, to within a group or two, every group), so it runs on the
// caller's stream while `side_work` -- sketch / recovery / bucketing -- runs on the plan's second
// stream; the two join before the activations are masked and the down GEMM starts.
// gamma != NULL: h is the un-normalised x and the operand split applies the RMSNorm itself.
template <typename SideWork>
static cs_status exec_decode_overlapped(cs_plan *plan, const cs_layer *layer, const float *h, int B,
                                        const float *residual, float *out, cudaStream_t st, SideWork side_work,
                                        const float *gamma = nullptr) {
    __nv_bfloat16 *x_hi = static_cast<__nv_bfloat16 *>(plan->x_bf16);
    __nv_bfloat16 *x_lo = x_hi + (size_t)plan->cfg.max_tokens * plan->cfg.d;
    CS_CUDA_TRY(plan, cudaEventRecord(plan->ev_fork, st));
    CS_CUDA_TRY(plan, cudaStreamWaitEvent(plan->side, plan->ev_fork, 0));
    cs_status s = side_work(plan->side);
    if (s != CS_OK) return s;
    CS_CUDA_TRY(plan, cudaEventRecord(plan->ev_join, plan->side));
    // f32 activations go in as two bf16 parts so that the result keeps f32-level accuracy
    s = gamma != nullptr ? launch_norm_split_bf16(plan, h, gamma, B, x_hi, x_lo, st)
                         : launch_split_bf16(plan, h, x_hi, x_lo, (size_t)B * plan->cfg.d, st);
    if (s != CS_OK) return s;
    s = launch_decode_gateup(plan, layer, x_hi, x_lo, B, false, st);
    if (s != CS_OK) return s;
    CS_CUDA_TRY(plan, cudaStreamWaitEvent(st, plan->ev_join, 0));
    s = launch_decode_mask(plan, B, st);
    if (s != CS_OK) return s;
    return launch_decode_down(plan, layer, B, true, residual, out, st);
}

}  // extern "C++"

// Dispatch of the actuator by batch size: gather GEMV, tensor-core decode path, or (more than 128
// tokens) the token-tiled grouped GEMMs over the union list.
// check: the supports come from the caller and are validated on the device (inside the gather
// kernel, or by a small kernel ahead of the tensor-core paths).
static cs_status exec_dispatch(cs_plan *plan, const cs_layer *layer, const float *h, const int32_t *support,
                               int B, const float *residual, float *out, bool check, cudaStream_t st) {
    if (!plan->mma_ok || B < plan->mma_min_tokens)
        return launch_ffn_gather(plan, layer, h, support, B, residual, out, check, st);
    if (check) {
        cs_status s = launch_check_support(plan, support, B, st);
        if (s != CS_OK) return s;
    }
    __nv_bfloat16 *x_hi = static_cast<__nv_bfloat16 *>(plan->x_bf16);
    __nv_bfloat16 *x_lo = x_hi + (size_t)plan->cfg.max_tokens * plan->cfg.d;
    if (use_decode_mma(plan, B)) {
        // The supports are known before the GEMMs here.  While the batch is small enough that a fair share
        // of the groups is in nobody's support (expected unused fraction (1 - k/G)^B of about 8 % or more),
        // the buckets are formed first and gate/up runs over the union list only, with the membership masks
        // applied in its epilogue; beyond that the union is (nearly) every group and bucketing runs beside
        // the dense gate/up GEMM instead.
        if (2 * B * plan->cfg.k <= 5 * plan->G) {
            cs_status s = launch_bucket(plan, support, B, st);
            if (s == CS_OK) s = launch_split_bf16(plan, h, x_hi, x_lo, (size_t)B * plan->cfg.d, st);
            if (s == CS_OK) s = launch_decode_gateup(plan, layer, x_hi, x_lo, B, true, st);
            if (s == CS_OK) s = launch_decode_down(plan, layer, B, false, residual, out, st);
            return s;
        }
        return exec_decode_overlapped(plan, layer, h, B, residual, out, st,
                                      [&](cudaStream_t side) { return launch_bucket(plan, support, B, side); });
    }
    cs_status s = launch_split_bf16(plan, h, x_hi, x_lo, (size_t)B * plan->cfg.d, st);
    if (s != CS_OK) return s;
    s = launch_bucket(plan, support, B, st);
    if (s != CS_OK) return s;
    return launch_ffn_mma(plan, layer, x_hi, x_lo, B, plan->glist, plan->nu, 0, plan->mask, residual, out, nullptr, st);
}

cs_status cs_ffn_exec(cs_plan *plan, const cs_layer *layer, const float *h, const int32_t *support,
                      int32_t B, const float *residual, float *out, void *stream) {
    if (plan == nullptr || h == nullptr || support == nullptr || out == nullptr) return CS_ERR_NULL;
    cs_status s = check_weights(layer);
    if (s != CS_OK) return s;
    if (B <= 0 || B > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    if (!aligned16(h) || !aligned16(out) || (residual != nullptr && !aligned16(residual))) return CS_ERR_UNSUPPORTED;
    return exec_dispatch(plan, layer, h, support, B, residual, out, true, static_cast<cudaStream_t>(stream));
}

cs_status cs_bucket(cs_plan *plan, const int32_t *support, int32_t B, int32_t *counts, int32_t *offsets,
                    int32_t *token_ids, void *stream) {
    if (plan == nullptr || support == nullptr || counts == nullptr || offsets == nullptr || token_ids == nullptr)
        return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cs_status s = launch_check_support(plan, support, B, st);
    if (s != CS_OK) return s;
    return launch_bucket(plan, support, B, st, counts, offsets, token_ids);
}

cs_status cs_layer_step(cs_plan *plan, const cs_layer *layer, const float *x, int32_t B, float *x_out,
                        int32_t *support_out, float *z_out, float *resid_out, void *stream) {
    if (plan == nullptr || x == nullptr || x_out == nullptr) return CS_ERR_NULL;
    cs_status s = check_weights(layer);
    if (s != CS_OK) return s;
    if (layer->S == nullptr || layer->Phi == nullptr) return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    if (!isfinite(layer->mu) || !(layer->mu > 0.f)) return CS_ERR_NONFINITE;
    if (!aligned16(x) || !aligned16(x_out) || !aligned16(layer->S) ||
        (layer->rms_gamma != nullptr && !aligned16(layer->rms_gamma)))
        return CS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool norm = layer->rms_gamma != nullptr;
    const float *n = norm ? plan->n_buf : x;
    int32_t *sup = support_out != nullptr ? support_out : plan->sup_buf;
    if (use_decode_mma(plan, B)) {
        // sketch, recovery and bucketing run beside the gate/up GEMM; with a normalisation the GEMM's
        // operand split normalises for itself, so that it does not wait for the sketch kernel either
        return exec_decode_overlapped(plan, layer, x, B, layer->add_residual ? x : nullptr, x_out, st,
                                      [&](cudaStream_t side) {
            cs_status r = launch_sketch(plan, layer->S, x, layer->rms_gamma, B, plan->y_buf, norm ? plan->n_buf : nullptr,
                                        layer->Phi, layer->mu, side);
            if (r == CS_OK) r = launch_recover(plan, layer->Phi, layer->mu, plan->y_buf, B, sup, z_out, resid_out, true, side);
            if (r == CS_OK) r = launch_bucket(plan, sup, B, side);
            return r;
        }, layer->rms_gamma);
    }
    const bool gather = !plan->mma_ok || B < plan->mma_min_tokens;
    if (gather && plan->speculative && sketch_recover_ok(plan) && !plan->timing) {
        // Opt-in (cs_plan_set_speculative): sketch and recovery in one launch, and the gather FFN behind it
        // starts its weight stream on the first iterate while the other iterations run.  (Not while stages
        // are being timed: event records between the launches would serialise them.)
        if (plan->speculative == 2) {
            // L2 warm-up only: the plain gather kernel, which asks L2 for the first iterate's blocks before it
            // waits for the final supports
            s = launch_sketch_recover(plan, layer, x, B, plan->y_buf, norm ? plan->n_buf : nullptr, sup, z_out, resid_out, st);
            if (s != CS_OK) return s;
            return launch_ffn_gather(plan, layer, n, sup, B, layer->add_residual ? x : nullptr, x_out, false, st, plan->slot_table);
        }
        s = launch_sketch_recover(plan, layer, x, B, plan->y_buf, norm ? plan->n_buf : nullptr, support_out, z_out, resid_out, st);
        if (s != CS_OK) return s;
        return launch_ffn_gather_spec(plan, layer, n, B, layer->add_residual ? x : nullptr, x_out, st);
    }
    s = launch_sketch(plan, layer->S, x, layer->rms_gamma, B, plan->y_buf, norm ? plan->n_buf : nullptr, layer->Phi, layer->mu, st);
    if (s != CS_OK) return s;
    s = launch_recover(plan, layer->Phi, layer->mu, plan->y_buf, B, sup, z_out, resid_out, true, st);
    if (s != CS_OK) return s;
    // supports produced by the recovery are valid by construction: no device check here
    return exec_dispatch(plan, layer, n, sup, B, layer->add_residual ? x : nullptr, x_out, false, st);
}

cs_status cs_layer_step_ex(cs_plan *plan, const cs_layer *layer, const float *x, int32_t B,
                           const cs_step_options *opt, float *x_out, int32_t *support_out, float *z_out,
                           float *resid_out, void *stream) {
    if (opt == nullptr) return cs_layer_step(plan, layer, x, B, x_out, support_out, z_out, resid_out, stream);
    if (plan == nullptr || x == nullptr || x_out == nullptr) return CS_ERR_NULL;
    cs_status s = check_weights(layer);
    if (s != CS_OK) return s;
    const bool srht = opt->srht_sign != nullptr;
    if (layer->Phi == nullptr || (!srht && layer->S == nullptr)) return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    if (!isfinite(layer->mu) || !(layer->mu > 0.f)) return CS_ERR_NONFINITE;
    if (!aligned16(x) || !aligned16(x_out) || (!srht && !aligned16(layer->S)) ||
        (layer->rms_gamma != nullptr && !aligned16(layer->rms_gamma)))
        return CS_ERR_UNSUPPORTED;
    s = check_options(plan, opt, true);
    if (s != CS_OK) return s;
    const bool norm = layer->rms_gamma != nullptr;
    if (srht && norm) return CS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (opt->support_prev != nullptr) {
        s = launch_check_support(plan, opt->support_prev, B, st);
        if (s != CS_OK) return s;
    }
    const float *n = norm ? plan->n_buf : x;
    const float *residual = layer->add_residual ? x : nullptr;
    if (opt->reuse_support) {   // no estimation this step: the previous supports execute
        if (norm) {   // the sketch kernel also forms the normalised input
            s = launch_sketch(plan, layer->S, x, layer->rms_gamma, B, plan->y_buf, plan->n_buf, nullptr, 0.f, st);
            if (s != CS_OK) return s;
        }
        if (support_out != nullptr)
            CS_CUDA_TRY(plan, cudaMemcpyAsync(support_out, opt->support_prev, (size_t)B * plan->cfg.k * sizeof(int32_t),
                                              cudaMemcpyDeviceToDevice, st));
        return exec_dispatch(plan, layer, n, opt->support_prev, B, residual, x_out, false, st);
    }
    if (srht) s = launch_sketch_srht(plan, opt->srht_sign, opt->srht_rows, x, B, plan->y_buf, st);
    else s = launch_sketch(plan, layer->S, x, layer->rms_gamma, B, plan->y_buf, norm ? plan->n_buf : nullptr, layer->Phi,
                           layer->mu, st);
    if (s != CS_OK) return s;
    int32_t *sup = support_out != nullptr ? support_out : plan->sup_buf;
    s = recover_with(plan, layer->Phi, layer->mu, plan->y_buf, B, opt, sup, z_out, resid_out, !srht, st);
    if (s != CS_OK) return s;
    if (opt->delta_out != nullptr || opt->drift_out != nullptr) {
        s = launch_support_drift(plan, opt->support_prev, sup, B, opt->delta_out, opt->drift_out, st);
        if (s != CS_OK) return s;
    }
    return exec_dispatch(plan, layer, n, sup, B, residual, x_out, false, st);
}

cs_status cs_layer_step_fallback(cs_plan *plan, cs_plan *dense, const cs_layer *layer, const float *x, int32_t B,
                                 const cs_step_options *opt, float tau, float *x_out, int32_t *support_out,
                                 float *z_out, float *resid_out, int32_t *flags_out, int32_t *n_fallback,
                                 void *stream) {
    if (plan == nullptr || dense == nullptr || n_fallback == nullptr) return CS_ERR_NULL;
    const cs_config &a = plan->cfg, &b = dense->cfg;
    if (a.d != b.d || a.d_ff != b.d_ff || a.group != b.group || a.m != b.m || a.w_dtype != b.w_dtype || b.k < a.k ||
        B > b.max_tokens)
        return CS_ERR_SHAPE;
    if (!isfinite(tau) || tau < 0.f) return CS_ERR_NONFINITE;
    if (opt != nullptr && opt->reuse_support) return CS_ERR_UNSUPPORTED;
    if (x_out == x) return CS_ERR_UNSUPPORTED;   // the second pass reads x again
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float *resid = resid_out != nullptr ? resid_out : plan->resid_buf;
    cs_status s = cs_layer_step_ex(plan, layer, x, B, opt, x_out, support_out, z_out, resid, stream);
    if (s != CS_OK) return s;
    s = launch_confidence(plan, plan->y_buf, resid, B, tau, flags_out != nullptr ? flags_out : plan->fb_flags, plan->fb_list,
                          plan->fb_count, st);
    if (s != CS_OK) return s;
    int32_t n_low = 0;
    CS_CUDA_TRY(plan, cudaMemcpyAsync(&n_low, plan->fb_count, sizeof n_low, cudaMemcpyDeviceToHost, st));
    CS_CUDA_TRY(plan, cudaStreamSynchronize(st));
    *n_fallback = n_low;
    if (n_low == 0) return CS_OK;
    // the untrusted tokens alone, through the denser plan, and back into their rows
    s = launch_gather_rows(plan, x, plan->fb_list, n_low, dense->x_host_in, st);
    if (s != CS_OK) return s;
    cs_step_options second;
    memset(&second, 0, sizeof second);
    second.T = -1;
    if (opt != nullptr) { second.solver = opt->solver; second.srht_sign = opt->srht_sign; second.srht_rows = opt->srht_rows; }
    if (second.solver == CS_SOLVER_OMP && b.k > 64) second.solver = CS_SOLVER_IHT;
    s = cs_layer_step_ex(dense, layer, dense->x_host_in, n_low, &second, dense->x_host_out, nullptr, nullptr, nullptr, stream);
    if (s != CS_OK) return s;
    return launch_scatter_rows(plan, dense->x_host_out, plan->fb_list, n_low, x_out, st);
}

cs_status cs_layer_step_host(cs_plan *plan, const cs_layer *layer, const float *x_host, int32_t B,
                             float *x_out_host, int32_t *support_host, void *stream) {
    if (plan == nullptr || x_host == nullptr || x_out_host == nullptr) return CS_ERR_NULL;
    if (B <= 0 || B > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t bytes = (size_t)B * plan->cfg.d * sizeof(float);
    // validate before the first copy so that nothing is enqueued on an error
    cs_status s = check_weights(layer);
    if (s != CS_OK) return s;
    if (layer->S == nullptr || layer->Phi == nullptr) return CS_ERR_NULL;
    if (!isfinite(layer->mu) || !(layer->mu > 0.f)) return CS_ERR_NONFINITE;
    // Small transfers from and to page-locked memory: the copy engine's set-up costs as much as the
    // transfer or more, so a kernel of the launch chain fetches x over the bus and the last kernel of
    // the step stores the result straight into the caller's buffer.  Anything else goes through the
    // copy engine.
    const float *x_alias = nullptr;
    float *out_alias = nullptr;
    if (bytes <= (pdl_for(plan, B) ? kZeroCopyBytes : kZeroCopyBytesLarge)) {
        x_alias = static_cast<const float *>(device_alias(x_host));
        out_alias = static_cast<float *>(device_alias(x_out_host));
        if (x_alias == nullptr || out_alias == nullptr || !aligned16(x_alias) || !aligned16(out_alias)) x_alias = nullptr;
    }
    if (x_alias != nullptr) {
        const int n4 = (int)(bytes / 16);
        launch_pdl(pdl_for(plan, B), stage_in_kernel, dim3((n4 + 255) / 256), dim3(256), 0, st,
                   reinterpret_cast<const float4 *>(x_alias), reinterpret_cast<float4 *>(plan->x_host_in), n4);
        plan->launches++;
        CS_CUDA_TRY(plan, cudaGetLastError());
        s = cs_layer_step(plan, layer, plan->x_host_in, B, out_alias, support_host != nullptr ? plan->sup_buf : nullptr, nullptr,
                          nullptr, stream);
        if (s != CS_OK) return s;
    } else {
        CS_CUDA_TRY(plan, cudaMemcpyAsync(plan->x_host_in, x_host, bytes, cudaMemcpyHostToDevice, st));
        s = cs_layer_step(plan, layer, plan->x_host_in, B, plan->x_host_out, support_host != nullptr ? plan->sup_buf : nullptr,
                          nullptr, nullptr, stream);
        if (s != CS_OK) return s;
        CS_CUDA_TRY(plan, cudaMemcpyAsync(x_out_host, plan->x_host_out, bytes, cudaMemcpyDeviceToHost, st));
    }
    if (support_host != nullptr)
        CS_CUDA_TRY(plan, cudaMemcpyAsync(support_host, plan->sup_buf, (size_t)B * plan->cfg.k * sizeof(int32_t),
                                          cudaMemcpyDeviceToHost, st));
    return CS_OK;
}

cs_status cs_plan_set_crossover(cs_plan *plan, int32_t tokens) {
    if (plan == nullptr) return CS_ERR_NULL;
    if (tokens < 1 || tokens > 129) return CS_ERR_SHAPE;
    plan->mma_min_tokens = tokens;
    return CS_OK;
}

int32_t cs_plan_crossover(const cs_plan *plan) { return plan != nullptr ? plan->mma_min_tokens : 0; }

cs_status cs_plan_set_speculative(cs_plan *plan, int32_t on) {
    if (plan == nullptr) return CS_ERR_NULL;
    if (on && !sketch_recover_ok(plan)) return CS_ERR_UNSUPPORTED;
    if (on < 0 || on > 2) return CS_ERR_SHAPE;
    plan->speculative = on;
    return CS_OK;
}

cs_status cs_plan_enable_timing(cs_plan *plan, int32_t on) {
    if (plan == nullptr) return CS_ERR_NULL;
    plan->timing = on != 0;
    for (int i = 0; i < CS_STAGE_COUNT; ++i) plan->stage_seen[i] = 0;
    return CS_OK;
}

cs_status cs_plan_stage_times(cs_plan *plan, void *stream, float ms[CS_STAGE_COUNT]) {
    if (plan == nullptr || ms == nullptr) return CS_ERR_NULL;
    CS_CUDA_TRY(plan, cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    for (int i = 0; i < CS_STAGE_COUNT; ++i) {
        ms[i] = 0.f;
        if (plan->stage_seen[i]) CS_CUDA_TRY(plan, cudaEventElapsedTime(&ms[i], plan->ev[2 * i], plan->ev[2 * i + 1]));
    }
    return CS_OK;
}

cs_status cs_prompt_support(cs_plan *plan, const float *S, const float *Phi, float mu, const void *H,
                            int32_t n, int32_t *support, float *z, float *resid, void *stream) {
    if (plan == nullptr || S == nullptr || Phi == nullptr || H == nullptr || support == nullptr) return CS_ERR_NULL;
    if (n <= 0 || n > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    if (!isfinite(mu) || !(mu > 0.f)) return CS_ERR_NONFINITE;
    if (!aligned16(S) || !aligned16(H)) return CS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cs_status s = launch_prompt_mean(plan, H, n, plan->hbar, st);
    if (s != CS_OK) return s;
    s = launch_sketch(plan, S, plan->hbar, nullptr, 1, plan->y_buf, nullptr, Phi, mu, st);
    if (s != CS_OK) return s;
    return launch_recover(plan, Phi, mu, plan->y_buf, 1, support, z, resid, true, st);
}

cs_status cs_ffn_exec_shared(cs_plan *plan, const cs_layer *layer, const void *H, int32_t n,
                             const int32_t *support, void *out, void *stream) {
    if (plan == nullptr || H == nullptr || support == nullptr || out == nullptr) return CS_ERR_NULL;
    cs_status s = check_weights(layer);
    if (s != CS_OK) return s;
    if (n <= 0 || n > plan->cfg.max_tokens) return CS_ERR_SHAPE;
    if (!plan->mma_ok || !aligned16(H) || !aligned16(out)) return CS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    s = launch_check_support(plan, support, 1, st);
    if (s != CS_OK) return s;
    return launch_ffn_mma(plan, layer, H, nullptr, n, support, nullptr, plan->cfg.k, nullptr, nullptr, nullptr, out, st);
}

cs_status cs_last_device_status(cs_plan *plan, void *stream, int32_t *code) {
    if (plan == nullptr || code == nullptr) return CS_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DeviceStatus hs;
    CS_CUDA_TRY(plan, cudaMemcpyAsync(&hs, plan->status, sizeof hs, cudaMemcpyDeviceToHost, st));
    CS_CUDA_TRY(plan, cudaMemsetAsync(plan->status, 0, sizeof hs, st));
    CS_CUDA_TRY(plan, cudaStreamSynchronize(st));
    *code = hs.code;
    return CS_OK;
}

int64_t cs_launch_count(const cs_plan *plan) { return plan != nullptr ? plan->launches : 0; }

const char *cs_last_cuda_error(const cs_plan *plan) { return plan != nullptr ? plan->cuda_error : ""; }

const char *cs_status_string(cs_status s) {
    switch (s) {
        case CS_OK: return "ok";
        case CS_ERR_NULL: return "null pointer";
        case CS_ERR_SHAPE: return "inconsistent shape";
        case CS_ERR_UNSUPPORTED: return "unsupported shape, dtype or alignment";
        case CS_ERR_SUPPORT: return "invalid support (must be ascending, distinct, in range)";
        case CS_ERR_NONFINITE: return "non-finite or non-positive scalar parameter";
        case CS_ERR_CUDA: return "CUDA runtime error";
        case CS_ERR_TIMEOUT: return "bounded device wait gave up";
    }
    return "unknown status";
}

}  // extern "C"
