// C-ABI entry points of librr (declared and documented in include/rr.h):
// argument checks, workspace layout, launches.  No device memory is allocated here.
#include "rr_common.cuh"
#include "rr_ffn.cuh"

namespace {

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

namespace rr {

static unsigned long long g_test_wait_limit_ns = 0;
unsigned long long test_wait_limit_ns() { return g_test_wait_limit_ns; }

rr_status check_route_shape(int T, int E, int k, int C, int G, unsigned mode)
{
    if (T < 0 || E < 1 || k < 1 || C < 0 || G < 1) return RR_ERR_INVALID_ARG;
    if (k > kMaxK || E > kMaxE || k > E) return RR_ERR_INVALID_ARG;
    if ((mode & RR_FR) && k >= E) return RR_ERR_INVALID_ARG;
    if (mode & ~(RR_IR | RR_FR | RR_SCORE | RR_FR_SOFTMAX | RR_LOCAL_CAP)) return RR_ERR_INVALID_ARG;
    if ((mode & RR_LOCAL_CAP) && C % G != 0) return RR_ERR_INVALID_ARG;
    if ((mode & RR_FR_SOFTMAX) && !(mode & RR_FR)) return RR_ERR_INVALID_ARG;
    if (T % G != 0 || E % G != 0) return RR_ERR_INVALID_ARG;
    if ((long long)E * C + T >= (1ll << 31)) return RR_ERR_INVALID_ARG;
    return RR_OK;
}

rr_status check_route_tables(const rr_route_tables *t)
{
    if (!t) return RR_ERR_INVALID_ARG;
    const void *p[] = {t->topk_expert, t->route_slot, t->slot_token, t->slot_rank, t->drop_count,
                       t->ir_expert, t->ir_pos, t->ir_offset, t->ir_token, t->expert_count,
                       t->n_routed, t->row_offset, t->row_token, t->row_weight, t->token_rows,
                       t->combine_w};
    for (const void *q : p)
        if (!q || !aligned(q, 16)) return RR_ERR_INVALID_ARG;
    return RR_OK;
}

}  // namespace rr

namespace {

using rr::check_route_shape;
rr_status check_tables(const rr_route_tables *t) { return rr::check_route_tables(t); }

rr_status check_moe_shape(const rr_moe_shape *s)
{
    if (!s) return RR_ERR_INVALID_ARG;
    rr_status rc = check_route_shape(s->T, s->E, s->k, s->capacity, s->G, s->mode);
    if (rc) return rc;
    if (s->d < 64 || s->d_ff < 64 || s->d % 64 || s->d_ff % 64) return RR_ERR_INVALID_ARG;
    if (s->dtype != RR_BF16 && s->dtype != RR_F32) return RR_ERR_INVALID_ARG;
    if (s->flags & ~RR_GRAD_EXACT) return RR_ERR_INVALID_ARG;
    return RR_OK;
}

}  // namespace

extern "C" {

rr_status rr_route_workspace_bytes(int T, int E, int k, int capacity, int G, unsigned mode, size_t *bytes)
{
    if (!bytes) return RR_ERR_INVALID_ARG;
    rr_status rc = check_route_shape(T, E, k, capacity, G, mode);
    if (rc) return rc;
    rr::RouteScratch s;
    *bytes = rr::route_scratch_layout(nullptr, T, E, k, &s, mode, G);
    return RR_OK;
}

rr_status rr_route(const float *logits, int T, int E, int k, int capacity, int G, unsigned mode,
                   const rr_route_tables *out, void *workspace, size_t workspace_bytes, void *stream)
{
    rr_status rc = check_route_shape(T, E, k, capacity, G, mode);
    if (rc) return rc;
    rc = check_tables(out);
    if (rc) return rc;
    if ((T > 0 && !logits) || !aligned(logits, 16) || !workspace || !aligned(workspace, 256))
        return RR_ERR_INVALID_ARG;
    rr::RouteScratch s;
    if (rr::route_scratch_layout(workspace, T, E, k, &s, mode, G) > workspace_bytes) return RR_ERR_WORKSPACE_TOO_SMALL;
    cudaError_t err = rr::launch_route(logits, T, E, k, capacity, G, mode, *out, s,
                                       static_cast<cudaStream_t>(stream));
    return err == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

rr_status rr_moe_workspace_bytes(const rr_moe_shape *s, size_t *fwd_bytes, size_t *bwd_bytes, size_t *saved_bytes)
{
    rr_status rc = check_moe_shape(s);
    if (rc) return rc;
    rr::FfnScratch f;
    if (fwd_bytes) *fwd_bytes = rr::ffn_fwd_layout(nullptr, nullptr, *s, &f);
    // (the backward pass exists for bf16 only: an fp32 shape has nothing to save and no workspace)
    if (saved_bytes) *saved_bytes = s->dtype == RR_BF16 ? rr::ffn_saved_bytes(*s) : 0;
    if (bwd_bytes) *bwd_bytes = s->dtype == RR_BF16 ? rr::ffn_bwd_layout(nullptr, *s, nullptr) : 0;
    return RR_OK;
}

rr_status rr_moe_fwd(const rr_moe_shape *s, const void *hidden, const void *W1, const void *W3,
                     const void *W2, const float *logits, const rr_route_tables *tables, float *out,
                     void *saved, void *workspace, size_t workspace_bytes, void *stream)
{
    (void)logits;
    rr_status rc = check_moe_shape(s);
    if (rc) return rc;
    rc = check_tables(tables);
    if (rc) return rc;
    if (s->T == 0) return RR_OK;  // no tokens: `out` has no elements
    if (!hidden || !W1 || !W3 || !W2 || !out || !workspace) return RR_ERR_INVALID_ARG;
    if (!aligned(hidden, 128) || !aligned(W1, 128) || !aligned(W3, 128) || !aligned(W2, 128) ||
        !aligned(out, 16) || !aligned(workspace, 256) || !aligned(saved, 256))
        return RR_ERR_INVALID_ARG;
    rr::FfnScratch f;
    if (rr::ffn_fwd_layout(workspace, saved, *s, &f) > workspace_bytes) return RR_ERR_WORKSPACE_TOO_SMALL;
    return rr::launch_ffn_fwd(*s, hidden, W1, W3, W2, *tables, out, f, static_cast<cudaStream_t>(stream));
}

rr_status rr_moe_bwd(const rr_moe_shape *s, const void *dout, const void *hidden, const void *W1,
                     const void *W3, const void *W2, const float *logits, const rr_route_tables *tables,
                     const void *saved, float *dhidden, float *dlogits, float *dW1, float *dW3,
                     float *dW2, void *workspace, size_t workspace_bytes, void *stream)
{
    rr_status rc = check_moe_shape(s);
    if (rc) return rc;
    rc = check_tables(tables);
    if (rc) return rc;
    if (s->dtype != RR_BF16) return RR_ERR_UNSUPPORTED;  // training configurations are bf16
    if (s->T == 0) {  // no tokens: the weight gradients are zero, the per-token outputs have no elements
        if (!dW1 || !dW3 || !dW2) return RR_ERR_INVALID_ARG;
        cudaStream_t st0 = static_cast<cudaStream_t>(stream);
        const size_t wbytes = (size_t)s->E * s->d * s->d_ff * sizeof(float);
        if (cudaMemsetAsync(dW1, 0, wbytes, st0) != cudaSuccess || cudaMemsetAsync(dW3, 0, wbytes, st0) != cudaSuccess ||
            cudaMemsetAsync(dW2, 0, wbytes, st0) != cudaSuccess)
            return RR_ERR_CUDA;
        return RR_OK;
    }
    if (!dout || !hidden || !W1 || !W3 || !W2 || !logits || !saved || !dhidden || !dlogits || !dW1 ||
        !dW3 || !dW2 || !workspace)
        return RR_ERR_INVALID_ARG;
    if (!aligned(dout, 128) || !aligned(hidden, 128) || !aligned(W1, 128) || !aligned(W3, 128) ||
        !aligned(W2, 128) || !aligned(saved, 256) || !aligned(workspace, 256) || !aligned(dhidden, 16) ||
        !aligned(dlogits, 16) || !aligned(dW1, 16) || !aligned(dW3, 16) || !aligned(dW2, 16))
        return RR_ERR_INVALID_ARG;
    rr::BwdScratch b;
    if (rr::ffn_bwd_layout(workspace, *s, &b) > workspace_bytes) return RR_ERR_WORKSPACE_TOO_SMALL;
    return rr::launch_ffn_bwd(*s, dout, hidden, W1, W3, W2, logits, *tables, saved, dhidden, dlogits,
                              dW1, dW3, dW2, b, static_cast<cudaStream_t>(stream));
}

namespace {

rr_status check_gate_shape(int T, int E, int d, int dtype)
{
    if (T < 0 || E < 1 || E > rr::kMaxE || d < 64 || d % 64) return RR_ERR_INVALID_ARG;
    if (dtype != RR_BF16 && dtype != RR_F32) return RR_ERR_INVALID_ARG;
    return RR_OK;
}

}  // namespace

rr_status rr_gate_workspace_bytes(int T, int E, int d, size_t *fwd_bytes, size_t *bwd_bytes)
{
    rr_status rc = check_gate_shape(T, E, d, RR_BF16);
    if (rc) return rc;
    if (fwd_bytes) *fwd_bytes = rr::gate_fwd_workspace(T, E, d);
    if (bwd_bytes) *bwd_bytes = rr::gate_bwd_workspace(T, E, d);
    return RR_OK;
}

rr_status rr_gate_fwd(int T, int E, int d, int dtype, const void *hidden, const void *Wg, float *logits,
                      void *workspace, size_t workspace_bytes, void *stream)
{
    rr_status rc = check_gate_shape(T, E, d, dtype);
    if (rc) return rc;
    if (T == 0) return RR_OK;
    if (!hidden || !Wg || !logits || !workspace) return RR_ERR_INVALID_ARG;
    if (!aligned(hidden, 128) || !aligned(Wg, 128) || !aligned(logits, 16) || !aligned(workspace, 256))
        return RR_ERR_INVALID_ARG;
    if (rr::gate_fwd_workspace(T, E, d) > workspace_bytes) return RR_ERR_WORKSPACE_TOO_SMALL;
    return rr::launch_gate_fwd(T, E, d, dtype, hidden, Wg, logits, workspace, static_cast<cudaStream_t>(stream));
}

rr_status rr_gate_bwd(int T, int E, int d, int dtype, const float *dlogits, const void *hidden, const void *Wg,
                      float *dWg, float *dhidden, void *workspace, size_t workspace_bytes, void *stream)
{
    rr_status rc = check_gate_shape(T, E, d, dtype);
    if (rc) return rc;
    if (!dWg) return RR_ERR_INVALID_ARG;
    if (T == 0)
        return cudaMemsetAsync(dWg, 0, (size_t)E * d * sizeof(float), static_cast<cudaStream_t>(stream)) == cudaSuccess
                   ? RR_OK : RR_ERR_CUDA;
    if (!dlogits || !hidden || !Wg || !dhidden || !workspace) return RR_ERR_INVALID_ARG;
    if (!aligned(hidden, 16) || !aligned(Wg, 16) || !aligned(dlogits, 16) || !aligned(dWg, 16) ||
        !aligned(dhidden, 16) || !aligned(workspace, 256))
        return RR_ERR_INVALID_ARG;
    if (rr::gate_bwd_workspace(T, E, d) > workspace_bytes) return RR_ERR_WORKSPACE_TOO_SMALL;
    return rr::launch_gate_bwd(T, E, d, dtype, dlogits, hidden, Wg, dWg, dhidden, workspace,
                               static_cast<cudaStream_t>(stream));
}

namespace {

// rr_gate_route: the routing scratch (header first) followed by what the projection's epilogue hands over
struct GateRouteExtra {
    int *tabs;
    float *val;
    int *h;
    float *a_h;
    float *psum;
    float *cta_psum;
};

size_t gate_route_layout(void *ws, int T, int E, int k, unsigned mode, int G, rr::RouteScratch *s, GateRouteExtra *x)
{
    const size_t Tn = T > 0 ? T : 1;
    rr::Carver c(ws);
    c.off = rr::route_scratch_layout(ws, T, E, k, s, mode, G);
    x->tabs = c.take<int>(4);
    x->val = c.take<float>(Tn * (k + 1));
    x->h = c.take<int>(Tn);
    x->a_h = c.take<float>(Tn);
    x->psum = c.take<float>((Tn + 31) / 32 * E);
    x->cta_psum = c.take<float>((size_t)rr::kMaxRouteCtas * E);
    return rr::align_up(c.off, 256);
}

rr_status check_gate_route(int T, int E, int k, int C, int G, unsigned mode, int d, int dtype)
{
    rr_status rc = check_route_shape(T, E, k, C, G, mode);
    if (rc) return rc;
    rc = check_gate_shape(T, E, d, dtype);
    if (rc) return rc;
    if (!rr::route_is_fused(mode, T) || (mode & RR_FR_SOFTMAX)) return RR_ERR_UNSUPPORTED;
    return RR_OK;
}

}  // namespace

rr_status rr_gate_route_workspace_bytes(int T, int E, int k, int capacity, int G, unsigned mode, int d, size_t *bytes)
{
    if (!bytes) return RR_ERR_INVALID_ARG;
    rr_status rc = check_gate_route(T, E, k, capacity, G, mode, d, RR_BF16);
    if (rc) return rc;
    rr::RouteScratch s;
    GateRouteExtra x;
    *bytes = gate_route_layout(nullptr, T, E, k, mode, G, &s, &x);
    return RR_OK;
}

rr_status rr_gate_route(int T, int E, int k, int capacity, int G, unsigned mode, int d, int dtype, const void *hidden,
                        const void *Wg, float *logits, const rr_route_tables *out, float alpha, float *loss, float *f,
                        float *P, void *workspace, size_t workspace_bytes, void *stream)
{
    rr_status rc = check_gate_route(T, E, k, capacity, G, mode, d, dtype);
    if (rc) return rc;
    rc = check_tables(out);
    if (rc) return rc;
    const bool want_loss = loss || f || P;
    if (want_loss && !(loss && f && P)) return RR_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256)) return RR_ERR_INVALID_ARG;
    rr::RouteScratch s;
    GateRouteExtra x;
    if (gate_route_layout(workspace, T, E, k, mode, G, &s, &x) > workspace_bytes) return RR_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (T == 0) {  // no tokens: empty tables, a zero loss
        if (want_loss && (cudaMemsetAsync(loss, 0, sizeof(float), st) != cudaSuccess ||
                          cudaMemsetAsync(f, 0, E * sizeof(float), st) != cudaSuccess ||
                          cudaMemsetAsync(P, 0, E * sizeof(float), st) != cudaSuccess))
            return RR_ERR_CUDA;
        return rr::launch_route(nullptr, 0, E, k, capacity, G, mode, *out, s, st) == cudaSuccess ? RR_OK : RR_ERR_CUDA;
    }
    if (!hidden || !Wg || !logits || !aligned(hidden, 128) || !aligned(Wg, 128) || !aligned(logits, 16))
        return RR_ERR_INVALID_ARG;
    rc = rr::launch_gate_sel(T, E, d, dtype, hidden, Wg, logits, k, G, out->topk_expert, x.val, x.h, x.a_h,
                             want_loss ? x.psum : nullptr, s.status, x.tabs, st);
    if (rc) return rc;
    rr::RoutePresel pre{};
    pre.val = x.val;
    pre.h = x.h;
    pre.a_h = x.a_h;
    pre.psum = want_loss ? x.psum : nullptr;
    pre.cta_psum = x.cta_psum;
    pre.alpha = alpha;
    pre.loss = loss;
    pre.f = f;
    pre.P = P;
    return rr::launch_route_fused(logits, T, E, k, capacity, G, mode, *out, s, st, &pre) == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

namespace {

// rr_route_loss: the routing scratch followed by the softmax sums per 32-token unit and per block
size_t route_loss_layout(void *ws, int T, int E, int k, unsigned mode, int G, rr::RouteScratch *s, float **psum, float **cta_psum)
{
    const size_t Tn = T > 0 ? T : 1;
    rr::Carver c(ws);
    c.off = rr::route_scratch_layout(ws, T, E, k, s, mode, G);
    *psum = c.take<float>((Tn + 31) / 32 * E);
    *cta_psum = c.take<float>((size_t)rr::kMaxRouteCtas * E);
    return rr::align_up(c.off, 256);
}

}  // namespace

rr_status rr_route_loss_workspace_bytes(int T, int E, int k, int capacity, int G, unsigned mode, size_t *bytes)
{
    if (!bytes) return RR_ERR_INVALID_ARG;
    rr_status rc = check_route_shape(T, E, k, capacity, G, mode);
    if (rc) return rc;
    if (!rr::route_is_fused(mode, T)) return RR_ERR_UNSUPPORTED;
    rr::RouteScratch s;
    float *a, *b;
    *bytes = route_loss_layout(nullptr, T, E, k, mode, G, &s, &a, &b);
    return RR_OK;
}

rr_status rr_route_loss(const float *logits, int T, int E, int k, int capacity, int G, unsigned mode,
                        const rr_route_tables *out, float alpha, float *loss, float *f, float *P, void *workspace,
                        size_t workspace_bytes, void *stream)
{
    rr_status rc = check_route_shape(T, E, k, capacity, G, mode);
    if (rc) return rc;
    rc = check_tables(out);
    if (rc) return rc;
    if (!rr::route_is_fused(mode, T)) return RR_ERR_UNSUPPORTED;
    if (!loss || !f || !P) return RR_ERR_INVALID_ARG;
    if ((T > 0 && !logits) || !aligned(logits, 16) || !workspace || !aligned(workspace, 256)) return RR_ERR_INVALID_ARG;
    rr::RouteScratch s;
    rr::RoutePresel pre{};
    float *psum, *cta_psum;
    if (route_loss_layout(workspace, T, E, k, mode, G, &s, &psum, &cta_psum) > workspace_bytes) return RR_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (T == 0) {
        if (cudaMemsetAsync(loss, 0, sizeof(float), st) != cudaSuccess || cudaMemsetAsync(f, 0, E * sizeof(float), st) != cudaSuccess ||
            cudaMemsetAsync(P, 0, E * sizeof(float), st) != cudaSuccess)
            return RR_ERR_CUDA;
        return rr::launch_route(logits, 0, E, k, capacity, G, mode, *out, s, st) == cudaSuccess ? RR_OK : RR_ERR_CUDA;
    }
    pre.psum = psum;
    pre.cta_psum = cta_psum;
    pre.alpha = alpha;
    pre.loss = loss;
    pre.f = f;
    pre.P = P;
    return rr::launch_route_fused(logits, T, E, k, capacity, G, mode, *out, s, st, &pre) == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

rr_status rr_aux_workspace_bytes(int T, int E, size_t *bytes)
{
    if (T < 0 || E < 1 || E > rr::kMaxE || !bytes) return RR_ERR_INVALID_ARG;
    *bytes = rr::aux_workspace(T, E);
    return RR_OK;
}

rr_status rr_aux_loss_fwd(int T, int E, int stride, const float *logits, const int32_t *first_choice, float alpha,
                          float *loss, float *f, float *P, void *workspace, size_t workspace_bytes, void *stream)
{
    if (T < 0 || E < 1 || E > rr::kMaxE || stride < 1 || !loss || !f) return RR_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (T == 0) {  // no tokens: the loss and both factors are zero
        if (cudaMemsetAsync(loss, 0, sizeof(float), st) != cudaSuccess ||
            cudaMemsetAsync(f, 0, E * sizeof(float), st) != cudaSuccess ||
            (P && cudaMemsetAsync(P, 0, E * sizeof(float), st) != cudaSuccess))
            return RR_ERR_CUDA;
        return RR_OK;
    }
    if (!logits || !first_choice || !workspace || !aligned(workspace, 256) || !aligned(logits, 16))
        return RR_ERR_INVALID_ARG;
    if (rr::aux_workspace(T, E) > workspace_bytes) return RR_ERR_WORKSPACE_TOO_SMALL;
    return rr::launch_aux_fwd(T, E, stride, logits, first_choice, alpha, loss, f, P, workspace, st);
}

rr_status rr_aux_loss_bwd(int T, int E, const float *logits, const float *f, float alpha, float scale,
                          int accumulate, float *dlogits, void *stream)
{
    if (T < 0 || E < 1 || E > rr::kMaxE) return RR_ERR_INVALID_ARG;
    if (T == 0) return RR_OK;
    if (!logits || !f || !dlogits || !aligned(logits, 16) || !aligned(dlogits, 16)) return RR_ERR_INVALID_ARG;
    const float coef = (float)((double)scale * alpha * E / T);
    return rr::launch_aux_bwd(T, E, logits, f, coef, accumulate ? 1 : 0, dlogits, static_cast<cudaStream_t>(stream));
}

rr_status rr_check(const void *workspace, void *stream)
{
    if (!workspace) return RR_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return RR_ERR_CUDA;
    int status = 0;
    if (cudaMemcpyAsync(&status, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return RR_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return RR_ERR_CUDA;
    if (status != 0) {
        // hand the error to the caller once, then start clean
        if (cudaMemsetAsync(const_cast<void *>(workspace), 0, sizeof(int), st) != cudaSuccess) return RR_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return RR_ERR_CUDA;
    }
    return status;
}

void rr_test_set_wait_limit_ns(unsigned long long ns) { rr::g_test_wait_limit_ns = ns; }

const char *rr_status_string(rr_status s)
{
    switch (s) {
    case RR_OK: return "ok";
    case RR_ERR_INVALID_ARG: return "invalid argument";
    case RR_ERR_UNSUPPORTED: return "unsupported request";
    case RR_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case RR_ERR_CUDA: return "CUDA call failed";
    case RR_ERR_NONFINITE: return "non-finite logit";
    case RR_ERR_TIMEOUT: return "bounded wait ran out on the device";
    case RR_ERR_STATIC_SCRATCH_EXCEEDED: return "shape needs more scratch than the fixed in-library array holds";
    default: return "unknown status";
    }
}

}  // extern "C"
