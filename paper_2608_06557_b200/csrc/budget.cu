// cascade_budget: per-request latency budget (Eq. 3, Eq. 4, Eq. 5) and 64-bit priority key.
// One thread per request; int64 multiply/add/shift only, no division.  The work is a few
// dozen integer operations on ~37 bytes per request, so the kernel is launch-latency bound at
// every queue size this library accepts; loads are coalesced SoA reads.
#include "common.cuh"

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
budget_kernel(const __grid_constant__ cascade_params p, const __grid_constant__ LoadConsts lc,
              const __grid_constant__ cascade_reqs r, int n, int64_t now_ns, int64_t *__restrict__ budget_out,
              uint64_t *__restrict__ key_out, int32_t *__restrict__ want_out, uint32_t *__restrict__ status) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int i = blockIdx.x * kThreads + threadIdx.x;
    if (i >= n) return;
    const int64_t P = r.prompt[i];
    const int64_t O = r.pred_out[i];
    const int64_t n0 = r.n0[i], n1 = r.n1[i], n2 = r.n2[i];
    const uint32_t cls = r.cls[i];
    const uint32_t id = r.id[i] & 0x7FFFFFu;
    const int64_t elapsed = now_ns - r.arrival_ns[i];
    const int64_t lim = int64_t(1) << 50;
    bool ok = dev_request_valid(p.bt, P, n0, n1, n2) && O >= 0 && O <= (int64_t(1) << 20) &&
              cls < (uint32_t)p.n_classes && elapsed <= lim && elapsed >= -lim;
    if (!ok) {
        // out-of-bounds request: flagged and parked at the very end of the Tier-2 queue
        atomicOr(status, CASCADE_ST_EPRECOND);
        budget_out[i] = -(int64_t(1) << 62);
        key_out[i] = (uint64_t(1) << 63) | id;
        // parked, but still a request: with a usable shape it is offered tokens like any other (its budget
        // allows no restore, so the offer is everything behind its HBM blocks), in both admission modes
        if (p.plan_first) want_out[i] = dev_request_valid(p.bt, P, n0, n1, n2) ? (int32_t)(P - n0 * p.bt) : 0;
        return;
    }
    const int64_t s_hit = (n0 + n1 + n2) * p.bt;
    // matched prefix outside HBM is priced by tier (Eq. 6), the rest of the prompt is computed
    const int64_t tp = dev_restore_time(p, 1, n1) + dev_restore_time(p, 2, n2);
    const int64_t L_act = tp + (dev_comp_q(lc.A_act, p.c_attn_q20, P, s_hit) >> 20);
    const int64_t L_max = tp + (dev_comp_q(lc.A_max, p.c_attn_q20, P, s_hit) >> 20);
    const int64_t L = ((L_act + L_max) * p.gamma_q16) >> 17;   // Eq. 3
    const int64_t B = p.ttft_ns[cls] - L;                      // Eq. 4
    const int64_t B_rem = B - elapsed;                         // Eq. 5
    // one decode step of this request, co-scheduled with a full prefill chunk
    const int64_t kv = P * p.c_dkv_q20;
    const int64_t tdec_act = (lc.dec_act + kv) >> 20;
    const int64_t tdec_max = (lc.dec_max + kv) >> 20;
    const int64_t tdec = ((tdec_act + tdec_max) * p.gamma_q16) >> 17;
    const int64_t tpot = p.tpot_ns[cls];
    int64_t over = tdec - tpot;
    if (over < 0 || tpot == 0) over = 0;
    const int64_t budget = B_rem - O * over;
    // ordering value: the budget, or the comparison policies' arrival time / deadline / tokens left
    int64_t v = budget;
    bool tier2 = B <= 0;
    if (p.policy != CASCADE_POLICY_BUDGET) {
        tier2 = false;
        v = p.policy == CASCADE_POLICY_FCFS ? -elapsed
          : p.policy == CASCADE_POLICY_EDF  ? p.ttft_ns[cls] - elapsed
                                            : P - s_hit;
    }
    const int64_t clampv = int64_t(1) << 39;
    int64_t u = v < -clampv ? -clampv : (v > clampv - 1 ? clampv - 1 : v);
    u += clampv;
    budget_out[i] = budget;
    key_out[i] = (uint64_t(tier2) << 63) | (uint64_t(u) << 23) | id;
    if (p.plan_first) {
        // plan-first admission: the request's own restore choice fixes what it is offered
        int64_t x1, x2;
        dev_choose_restore(p, lc.A_act, P, n0, n1, n2, budget, &x1, &x2);
        want_out[i] = x2 > 0 ? 0 : (int32_t)(P - (n0 + x1) * p.bt);
    }
}

__global__ void __launch_bounds__(kThreads)
regimes_kernel(const __grid_constant__ cascade_params p, const __grid_constant__ LoadConsts lc, int64_t A_idle,
               const __grid_constant__ cascade_reqs r, int n, int64_t *__restrict__ lat4, uint32_t *__restrict__ status) {
    const int i = blockIdx.x * kThreads + threadIdx.x;
    if (i >= n) return;
    const int64_t P = r.prompt[i];
    const int64_t n0 = r.n0[i], n1 = r.n1[i], n2 = r.n2[i];
    longlong4 out = make_longlong4(0, 0, 0, 0);
    if (!dev_request_valid(p.bt, P, n0, n1, n2)) {
        atomicOr(status, CASCADE_ST_EPRECOND);
    } else {
        const int64_t s_hit = (n0 + n1 + n2) * p.bt;
        const int64_t tp = dev_restore_time(p, 1, n1) + dev_restore_time(p, 2, n2);
        out.x = dev_comp_q(A_idle, p.c_attn_q20, P, 0) >> 20;
        out.y = dev_comp_q(lc.A_act, p.c_attn_q20, P, 0) >> 20;
        out.z = tp + (dev_comp_q(lc.A_act, p.c_attn_q20, P, s_hit) >> 20);
        out.w = tp + (dev_comp_q(lc.A_max, p.c_attn_q20, P, s_hit) >> 20);
    }
    lat4[4 * (size_t)i + 0] = out.x;
    lat4[4 * (size_t)i + 1] = out.y;
    lat4[4 * (size_t)i + 2] = out.z;
    lat4[4 * (size_t)i + 3] = out.w;
}

__global__ void __launch_bounds__(kThreads)
reqs_update_kernel(const __grid_constant__ cascade_reqs dst, int cap, const __grid_constant__ cascade_reqs src,
                   const int32_t *__restrict__ slots, int m, uint32_t *__restrict__ status) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int i = blockIdx.x * kThreads + threadIdx.x;
    if (i >= m) return;
    const int s = slots[i];
    // all loads first (they may cross the host link: one round trip, not nine), then the stores
    const int64_t v_arr = src.arrival_ns[i];
    const int32_t v_prompt = src.prompt[i], v_out = src.pred_out[i], v_n0 = src.n0[i], v_n1 = src.n1[i], v_n2 = src.n2[i];
    const uint32_t v_id = src.id[i];
    const uint8_t v_cls = src.cls[i], v_flags = src.flags[i];
    if (s < 0 || s >= cap) {
        atomicOr(status, CASCADE_ST_EBOUNDS);
        return;
    }
    const_cast<int64_t *>(dst.arrival_ns)[s] = v_arr;
    const_cast<int32_t *>(dst.prompt)[s] = v_prompt;
    const_cast<int32_t *>(dst.pred_out)[s] = v_out;
    const_cast<int32_t *>(dst.n0)[s] = v_n0;
    const_cast<int32_t *>(dst.n1)[s] = v_n1;
    const_cast<int32_t *>(dst.n2)[s] = v_n2;
    const_cast<uint32_t *>(dst.id)[s] = v_id;
    const_cast<uint8_t *>(dst.cls)[s] = v_cls;
    const_cast<uint8_t *>(dst.flags)[s] = v_flags;
}

}  // namespace

extern "C" int cascade_reqs_update(cascade_ctx *ctx, const cascade_reqs *dst, int cap, const cascade_reqs *src,
                                   const int32_t *slots, int m, void *stream) {
    CascadeRange nvtx_range("cascade_reqs_update");
    if (!ctx || !dst || !src || cap < 0 || m < 0) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    if (m == 0) return CASCADE_OK;
    const cascade_reqs *both[2] = {dst, src};
    for (const cascade_reqs *q : both)
        if (!q->arrival_ns || !q->prompt || !q->pred_out || !q->n0 || !q->n1 || !q->n2 || !q->id || !q->cls || !q->flags)
            return CASCADE_EINVAL;
    if (!slots) return CASCADE_EINVAL;
    const int grid = (m + kThreads - 1) / kThreads;
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(grid), dim3(kThreads), 0, (cudaStream_t)stream,
                                         reqs_update_kernel, *dst, cap, *src, slots, m, ctx->status_dev));
    return CASCADE_OK;
}

extern "C" int cascade_budget(cascade_ctx *ctx, const cascade_reqs *r, int n, int64_t now_ns, int32_t D_act,
                              int64_t K_act, int64_t *budget_out, uint64_t *key_out, void *stream) {
    CascadeRange nvtx_range("cascade_budget");
    if (!ctx || !r || n < 0 || n > ctx->max_requests) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    if (n == 0) return CASCADE_OK;
    if (!budget_out || !key_out || !r->arrival_ns || !r->prompt || !r->pred_out || !r->n0 || !r->n1 || !r->n2 ||
        !r->id || !r->cls)
        return CASCADE_EINVAL;
    if (D_act < 0 || D_act > (1 << 16) || K_act < 0 || K_act > (int64_t(1) << 32)) return CASCADE_ERANGE;
    const LoadConsts lc = make_load_consts(ctx->params, D_act, K_act);
    const int grid = (n + kThreads - 1) / kThreads;
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(grid), dim3(kThreads), 0, (cudaStream_t)stream, budget_kernel,
                                         ctx->params, lc, *r, n, (int64_t)now_ns, budget_out, key_out,
                                         ctx->want_by_slot, ctx->status_dev));
    return CASCADE_OK;
}

extern "C" int cascade_latency_regimes(cascade_ctx *ctx, const cascade_reqs *r, int n, int32_t D_act, int64_t K_act,
                                       int64_t *lat4_out, void *stream) {
    CascadeRange nvtx_range("cascade_latency_regimes");
    if (!ctx || !r || n < 0 || n > ctx->max_requests) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    if (n == 0) return CASCADE_OK;
    if (!lat4_out || !r->prompt || !r->n0 || !r->n1 || !r->n2) return CASCADE_EINVAL;
    if (D_act < 0 || D_act > (1 << 16) || K_act < 0 || K_act > (int64_t(1) << 32)) return CASCADE_ERANGE;
    const LoadConsts lc = make_load_consts(ctx->params, D_act, K_act);
    const int64_t A_idle = make_load_consts(ctx->params, 0, 0).A_act;
    const int grid = (n + kThreads - 1) / kThreads;
    regimes_kernel<<<grid, kThreads, 0, (cudaStream_t)stream>>>(ctx->params, lc, A_idle, *r, n, lat4_out,
                                                               ctx->status_dev);
    CASCADE_CUDA_TRY(ctx, cudaGetLastError());
    return CASCADE_OK;
}
