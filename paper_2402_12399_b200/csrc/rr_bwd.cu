// Backward pass of the rectified MoE layer (Appendix A for the gate gradient).
//
// For every live row r (token i at expert e with combine weight w_r, multiplicity mu_r):
//   z_r     = W2_e^T dout_i                         kDAct GEMM (dout rows copied into expert order first)
//   delta_r = <z_r, act_r> = <dout_i, E_e(x_i)>     fused into its epilogue
//   dact_r  = w_r z_r ; dh3 = dact * silu(h1) ; dh1 = dact * h3 * silu'(h1)
//   dx_r    = dH1_r W1_e + dH3_r W3_e               kDX GEMM, epilogue adds into dhidden[i]
//   dW2_e   = sum_r dout_i (x) (w_r act_r)          kWgrad GEMMs, contraction over the expert's rows
//   dW1_e   = sum_r dh1_r (x) x_i ;  dW3_e likewise
//   dlogits_i from delta (straight-through, Eq. 6, or exact)        k_dlogits
// Gradient w.r.t. hidden flows through the experts only; the gate projection that produced the
// logits belongs to the caller, who receives dlogits.
#include "rr_gemm.cuh"

namespace rr {

using namespace gemm;

namespace {

// Dg[p] = dout[token(p)] for live padded rows, zeros for padding rows (the row operand of kDAct and of
// the dW2 GEMM; the hidden rows in the same order were saved by the forward pass).  One warp per padded row.
__global__ void __launch_bounds__(256)
k_bwd_prep(int E, int d, const int *__restrict__ mt_off, const int *__restrict__ row_offset,
           const int *__restrict__ row_token, const __nv_bfloat16 *__restrict__ dout, __nv_bfloat16 *__restrict__ dg)
{
    __shared__ int mt_s[kMaxE + 1];
    for (int e = threadIdx.x; e <= E; e += blockDim.x) mt_s[e] = mt_off[e];
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int rows_pad = mt_s[E] * kTileM;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    for (int prow = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; prow < rows_pad; prow += warps) {
        const int tile = prow / kTileM;
        int lo = 0, hi = E;  // largest e with mt_s[e] <= tile
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (mt_s[mid] <= tile) lo = mid; else hi = mid;
        }
        const int row = row_offset[lo] + (prow - mt_s[lo] * kTileM);
        const bool live = row < row_offset[lo + 1];
        const int tok = live ? row_token[row] : 0;
        const uint4 *gx = reinterpret_cast<const uint4 *>(dout + (size_t)tok * d);
        uint4 *oy = reinterpret_cast<uint4 *>(dg + (size_t)prow * d);
        for (int c = lane; c < d / 8; c += 32) oy[c] = live ? gx[c] : make_uint4(0, 0, 0, 0);
    }
}

// Gate gradient, one warp per token (Appendix A).
//   exact:            dL/da_ij = sum_{r: e_r = j} w_r (delta_r - sum_r' w_r' delta_r')
//   straight-through: g = softmax(a_i) over all E experts, S = sum_r mu_r g_{e_r} held constant,
//                     dL/dg_j = sum_{r: e_r = j} mu_r delta_r / S, dL/da_l = g_l (dL/dg_l - <g, dL/dg>)
__global__ void __launch_bounds__(256)
k_dlogits(int T, int E, int k, int exact, const float *__restrict__ logits, const int *__restrict__ topk_expert,
          const int *__restrict__ ir_expert, const int *__restrict__ drop_count, const int *__restrict__ token_rows,
          const float *__restrict__ combine_w, const float *__restrict__ delta, float *__restrict__ dlogits)
{
    const int lane = threadIdx.x & 31;
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= T) return;
    const int K1 = k + 1, K2 = k + 2;
    int ex[kMaxK + 2];
    float dl[kMaxK + 2], mu[kMaxK + 2], wr[kMaxK + 2];
    int routes = 0;
    for (int r = 0; r < K2; ++r) {
        const int row = token_rows[(size_t)i * K2 + r];
        ex[r] = -1;
        dl[r] = 0.f; mu[r] = 0.f; wr[r] = 0.f;
        if (row >= 0) {
            ex[r] = r < K1 ? topk_expert[(size_t)i * K1 + r] : ir_expert[i];
            dl[r] = delta[row];
            mu[r] = r < K1 ? 1.0f : (float)drop_count[i];
            wr[r] = combine_w[(size_t)i * K2 + r];
            ++routes;
        }
    }
    const float *a = logits + (size_t)i * E;
    float *out = dlogits + (size_t)i * E;
    if (routes == 0) {
        for (int j = lane; j < E; j += 32) out[j] = 0.0f;
        return;
    }
    if (exact) {
        float mean = 0.f;
        for (int r = 0; r < K2; ++r) mean += wr[r] * dl[r];
        for (int j = lane; j < E; j += 32) {
            float g = 0.f;
            for (int r = 0; r < K2; ++r)
                if (ex[r] == j) g += wr[r] * (dl[r] - mean);
            out[j] = g;
        }
        return;
    }
    float m = -3.4e38f;
    for (int j = lane; j < E; j += 32) m = fmaxf(m, a[j]);
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float z = 0.f;
    for (int j = lane; j < E; j += 32) z += expf(a[j] - m);
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    const float inv_z = 1.0f / z;
    float S = 0.f;
    for (int r = 0; r < K2; ++r)
        if (ex[r] >= 0) S += mu[r] * expf(a[ex[r]] - m) * inv_z;
    float dot = 0.f;  // <g, dL/dg> = sum_r g_{e_r} mu_r delta_r / S
    for (int r = 0; r < K2; ++r)
        if (ex[r] >= 0) dot += expf(a[ex[r]] - m) * inv_z * mu[r] * dl[r] / S;
    for (int j = lane; j < E; j += 32) {
        float dg = 0.f;
        for (int r = 0; r < K2; ++r)
            if (ex[r] == j) dg += mu[r] * dl[r] / S;
        out[j] = expf(a[j] - m) * inv_z * (dg - dot);
    }
}

}  // namespace

size_t ffn_bwd_layout(void *ws, const rr_moe_shape &s, BwdScratch *b)
{
    BwdScratch tmp;
    if (!b) b = &tmp;
    Carver c(ws);
    const size_t Rp = rows_pad_max(s);
    b->hdr = c.take<Header>(1);
    b->mt_off = c.take<int>(s.E + 1);
    b->delta = c.take<float>(rows_max(s) + 1);
    b->dg = c.take<char>(Rp * s.d * 2);
    // three matrices at one stride: the kDAct epilogue writes them as the planes of one tensor
    const size_t plane = align_up(Rp * s.d_ff * 2, 256);
    char *planes = c.take<char>(3 * plane);
    b->dh1 = planes;
    b->dh3 = planes ? planes + plane : nullptr;
    b->wact = planes ? planes + 2 * plane : nullptr;
    return align_up(c.off, 256);
}

rr_status launch_ffn_bwd(const rr_moe_shape &s, const void *dout, const void *hidden, const void *W1, const void *W3,
                         const void *W2, const float *logits, const rr_route_tables &t, const void *saved,
                         float *dhidden, float *dlogits, float *dW1, float *dW3, float *dW2, const BwdScratch &b,
                         cudaStream_t st)
{
    if (s.dtype != RR_BF16) return RR_ERR_UNSUPPORTED;  // training configurations are bf16
    (void)hidden;  // its rows, in expert order, are in `saved`
    const int grid = sm_count();
    if (grid <= 0) return RR_ERR_CUDA;
    const size_t Rp = rows_pad_max(s);
    const size_t h_bytes = align_up(Rp * s.d_ff * sizeof(float), 256);
    const float *h1 = static_cast<const float *>(saved);
    const void *xg = static_cast<const char *>(saved) + 2 * h_bytes;  // token rows in expert order, kept by the forward pass

    CUtensorMap mDgk, mW2, mDh1, mDh3, mW1, mW3, mDg, mWact, mXg, mDh1p, mDh3p, mdW1, mdW3, mdW2;
    CUtensorMap mH, mOut;
    const size_t out_stride = align_up(Rp * s.d_ff * 2, 256);  // as laid out by ffn_bwd_layout
    if (!make_map(&mDgk, b.dg, Rp, s.d, false, kTileM) ||                   // K-major A tiles of kDAct
        !make_map(&mW2, W2, (size_t)s.E * s.d, s.d_ff, false, 64) ||        // MN-major panels
        !make_map(&mW1, W1, (size_t)s.E * s.d_ff, s.d, false, 64) ||
        !make_map(&mW3, W3, (size_t)s.E * s.d_ff, s.d, false, 64) ||
        !make_map(&mDh1, b.dh1, Rp, s.d_ff, false, kTileM) ||               // K-major A tiles of kDX
        !make_map(&mDh3, b.dh3, Rp, s.d_ff, false, kTileM) ||
        !make_map(&mDh1p, b.dh1, Rp, s.d_ff, false, 64) ||                  // MN-major panels of kWgrad
        !make_map(&mDh3p, b.dh3, Rp, s.d_ff, false, 64) ||
        !make_map(&mDg, b.dg, Rp, s.d, false, 64) ||
        !make_map(&mXg, xg, Rp, s.d, false, 64) ||
        !make_map(&mWact, b.wact, Rp, s.d_ff, false, 64) ||
        // 32 x 16 tiles of the kDAct epilogue: {h1, h3} and {dH1, dH3, w*act} as the planes of two 3-D tensors
        !make_map_stack(&mH, h1, 2, h_bytes, Rp, s.d_ff, 4, true, 32, 64) ||
        !make_map_stack(&mOut, b.dh1, 3, out_stride, Rp, s.d_ff, 2, false, 32, 32) ||
        !make_map_3d_f32(&mdW2, dW2, s.E, s.d, s.d_ff) ||                   // store views of the gradients
        !make_map_3d_f32(&mdW1, dW1, s.E, s.d_ff, s.d) ||
        !make_map_3d_f32(&mdW3, dW3, s.E, s.d_ff, s.d))
        return RR_ERR_CUDA;

    if (cudaMemsetAsync(dhidden, 0, (size_t)s.T * s.d * sizeof(float), st) != cudaSuccess) return RR_ERR_CUDA;
    if (cudaMemsetAsync(b.delta, 0, (rows_max(s) + 1) * sizeof(float), st) != cudaSuccess) return RR_ERR_CUDA;
    k_tiles<<<1, 256, 0, st>>>(s.E, t.row_offset, b.mt_off);
    k_bwd_prep<<<grid * 8, 256, 0, st>>>(s.E, s.d, b.mt_off, t.row_offset, t.row_token,
                                         static_cast<const __nv_bfloat16 *>(dout), static_cast<__nv_bfloat16 *>(b.dg));
    auto mark = [&](int i) {
        if (s.trace && s.trace[i]) cudaEventRecord(static_cast<cudaEvent_t>(s.trace[i]), st);
    };
    mark(0);

    Params p{};
    p.E = s.E;
    p.mt_off = b.mt_off;
    p.row_offset = t.row_offset;
    p.row_token = t.row_token;
    p.row_weight = t.row_weight;
    p.status = &b.hdr->status;

    // z = dout_rows W2_e, SwiGLU backward, delta
    p.KB = s.d / 64;
    p.N = s.d_ff;
    p.n_tiles = (s.d_ff + 255) / 256;
    p.w_rows = s.d;
    p.delta = b.delta;
    if ((s.d <= 1024 ? launch<kDActShortK, false>(mDgk, mH, mW2, mW2, mOut, mOut, mOut, p, grid, st)
                     : launch<kDAct, false>(mDgk, mH, mW2, mW2, mOut, mOut, mOut, p, grid, st)) != cudaSuccess)
        return RR_ERR_CUDA;
    mark(1);

    // dx = dH1 W1_e + dH3 W3_e, added into dhidden[token]
    p.KB = 2 * (s.d_ff / 64);
    p.N = s.d;
    p.n_tiles = (s.d + 255) / 256;
    p.w_rows = s.d_ff;
    p.out = dhidden;
    if (launch<kDX, false>(mDh1, mDh3, mW1, mW3, mW1, mW3, mW3, p, grid, st) != cudaSuccess) return RR_ERR_CUDA;
    mark(2);

    // weight gradients: contraction over each expert's (padded) rows
    p.KB = 0;
    p.M = s.d; p.m_tiles = (s.d + 2 * kTileM - 1) / (2 * kTileM);  // 256 rows of dW per CTA pair
    p.N = s.d_ff; p.n_tiles = (s.d_ff + 255) / 256;
    p.dw = dW2;
    if (launch<kWgrad, false>(mDg, mDg, mWact, mWact, mdW2, mdW2, mdW2, p, grid, st) != cudaSuccess) return RR_ERR_CUDA;
    p.M = s.d_ff; p.m_tiles = (s.d_ff + 2 * kTileM - 1) / (2 * kTileM);
    p.N = s.d; p.n_tiles = (s.d + 255) / 256;
    p.dw = dW1;
    if (launch<kWgrad, false>(mDh1p, mDh1p, mXg, mXg, mdW1, mdW1, mdW1, p, grid, st) != cudaSuccess) return RR_ERR_CUDA;
    p.dw = dW3;
    if (launch<kWgrad, false>(mDh3p, mDh3p, mXg, mXg, mdW3, mdW3, mdW3, p, grid, st) != cudaSuccess) return RR_ERR_CUDA;
    mark(3);

    const int warps_per_block = 8;
    k_dlogits<<<(s.T + warps_per_block - 1) / warps_per_block > 0 ? (s.T + warps_per_block - 1) / warps_per_block : 1,
                256, 0, st>>>(s.T, s.E, s.k, (s.flags & RR_GRAD_EXACT) ? 1 : 0, logits, t.topk_expert, t.ir_expert,
                              t.drop_count, t.token_rows, t.combine_w, b.delta, dlogits);
    mark(4);
    return cudaGetLastError() == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

}  // namespace rr
