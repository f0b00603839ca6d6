// Expert FFN (grouped tcgen05 GEMMs) -- internal declarations.
#pragma once
#include "rr_common.cuh"

namespace rr {

constexpr int kTileM = 128;  // rows of one GEMM tile (= TMEM lanes)

// Scratch of the forward pass (device pointers).  Row-indexed buffers use the padded row space:
// expert e owns rows [128*mt_off[e], 128*mt_off[e+1]).
struct FfnScratch {
    Header *hdr;
    int *mt_off;  // [E+1] exclusive prefix of the number of 128-row tiles per expert
    void *xg;     // [Rp,d] token rows in padded row order (layer's element type), zero rows for padding
    void *act;    // [Rp,d_ff] silu(h1)*h3 in the layer's element type
    float *h1;    // [Rp,d_ff] fp32 gate pre-activation, in `saved`, only when training
    float *h3;    // [Rp,d_ff] fp32 up projection, in `saved`, only when training
};

// Scratch of the backward pass.
struct BwdScratch {
    Header *hdr;
    int *mt_off;   // [E+1]
    float *delta;  // [R] <dout_i, E_e(x_i)> per live row (public row index)
    void *dg;      // [Rp,d]    dout rows in padded row order (bf16), zero rows for padding
    void *dh1;     // [Rp,d_ff] bf16
    void *dh3;     // [Rp,d_ff] bf16
    void *wact;    // [Rp,d_ff] bf16 w_row * silu(h1) * h3
};

inline size_t rows_max(const rr_moe_shape &s) { return (size_t)s.E * s.capacity + (size_t)s.T; }
// upper bound of the padded row count: every expert adds fewer than 128 padding rows
inline size_t rows_pad_max(const rr_moe_shape &s) { return ((rows_max(s) + kTileM - 1) / kTileM + s.E) * kTileM; }
inline size_t elem_bytes(const rr_moe_shape &s) { return s.dtype == RR_F32 ? 4 : 2; }

size_t ffn_saved_bytes(const rr_moe_shape &s);
size_t ffn_fwd_layout(void *ws, void *saved, const rr_moe_shape &s, FfnScratch *f);
size_t ffn_bwd_layout(void *ws, const rr_moe_shape &s, BwdScratch *b);

rr_status launch_ffn_fwd(const rr_moe_shape &s, const void *hidden, const void *W1, const void *W3,
                         const void *W2, const rr_route_tables &t, float *out, const FfnScratch &f,
                         cudaStream_t st);

rr_status launch_ffn_bwd(const rr_moe_shape &s, const void *dout, const void *hidden, const void *W1,
                         const void *W3, const void *W2, const float *logits, const rr_route_tables &t,
                         const void *saved, float *dhidden, float *dlogits, float *dW1, float *dW3,
                         float *dW2, const BwdScratch &b, cudaStream_t st);

// Gate projection (rr_gate.cu)
size_t gate_fwd_workspace(int T, int E, int d);
size_t gate_bwd_workspace(int T, int E, int d);
rr_status launch_gate_fwd(int T, int E, int d, int dtype, const void *hidden, const void *Wg, float *logits,
                          void *workspace, cudaStream_t st);
rr_status launch_gate_bwd(int T, int E, int d, int dtype, const float *dlogits, const void *hidden, const void *Wg,
                          float *dWg, float *dhidden, void *workspace, cudaStream_t st);
rr_status launch_gate_sel(int T, int E, int d, int dtype, const void *hidden, const void *Wg, float *logits, int k, int G,
                          int *sel_expert, float *sel_val, int *sel_h, float *sel_ah, float *psum, int *status, int *tabs,
                          cudaStream_t st);

// Load-balance loss (rr_aux.cu)
size_t aux_workspace(int T, int E);
rr_status launch_aux_fwd(int T, int E, int stride, const float *logits, const int32_t *first, float alpha,
                         float *loss, float *f, float *P, void *workspace, cudaStream_t st);
rr_status launch_aux_bwd(int T, int E, const float *logits, const float *f, float coef, int accumulate,
                         float *dlogits, cudaStream_t st);

}  // namespace rr
