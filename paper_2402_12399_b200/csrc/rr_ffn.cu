// Expert FFN forward (Section 5.1: every expert is a copy of the LLaMA2 gated FFN; Eq. 2 / Eq. 3
// for the combine): two launches of the GEMM template in rr_gemm.cuh.
//
//   gather  : Xg[row] = hidden[token(row)]                       (rows of each expert made contiguous)
//   gate/up : H = Xg [W1_e ; W3_e]^T,  Act = silu(H1) * H3       (SwiGLU in the epilogue)
//   down    : Y = Act W2_e^T,  out[token] += w_row * Y            (combine fused into the epilogue
//             as vector fp32 reductions)
//
// Only live rows are computed: padding slots cost nothing, dropped tokens appear in no row.
#include "rr_gemm.cuh"

namespace rr {

using namespace gemm;

namespace {

// Xg[p] = hidden[token(p)] for live padded rows, zeros for padding rows.  One warp per padded
// row, 16 bytes per lane and step; `row_bytes` is a multiple of 16.
__global__ void __launch_bounds__(256)
k_gather_rows(int E, int row_bytes, const int *__restrict__ mt_off, const int *__restrict__ row_offset,
              const int *__restrict__ row_token, const char *__restrict__ src, char *__restrict__ dst)
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
        const uint4 *in = reinterpret_cast<const uint4 *>(src + (size_t)tok * row_bytes);
        uint4 *out = reinterpret_cast<uint4 *>(dst + (size_t)prow * row_bytes);
        for (int c = lane; c < row_bytes / 16; c += 32) out[c] = live ? in[c] : make_uint4(0, 0, 0, 0);
    }
}

}  // namespace

size_t ffn_saved_bytes(const rr_moe_shape &s)
{
    // h1, h3 in fp32, then the token rows in expert order (the A operand of the forward's first GEMM and of
    // two of the three weight-gradient GEMMs: gathered once)
    return 2 * align_up(rows_pad_max(s) * s.d_ff * sizeof(float), 256) + align_up(rows_pad_max(s) * s.d * 2, 256);
}

size_t ffn_fwd_layout(void *ws, void *saved, const rr_moe_shape &s, FfnScratch *f)
{
    Carver c(ws);
    f->hdr = c.take<Header>(1);
    f->mt_off = c.take<int>(s.E + 1);
    const size_t act_bytes = align_up(rows_pad_max(s) * s.d_ff * elem_bytes(s), 256);
    const size_t h_bytes = align_up(rows_pad_max(s) * s.d_ff * sizeof(float), 256);
    f->xg = c.take<char>(align_up(rows_pad_max(s) * s.d * elem_bytes(s), 256));
    f->act = c.take<char>(act_bytes);
    // What the backward pass needs goes to `saved` (bf16 layers only: fp32 layers have no backward pass and
    // save nothing).  The pre-activations are kept in fp32: rounded to bf16 they put errors of 2-7 % of its
    // RMS into the gate gradient.
    const bool keep = saved && s.dtype == RR_BF16;
    f->h1 = keep ? static_cast<float *>(saved) : nullptr;
    f->h3 = keep ? reinterpret_cast<float *>(static_cast<char *>(saved) + h_bytes) : nullptr;
    if (keep) f->xg = static_cast<char *>(saved) + 2 * h_bytes;
    return align_up(c.off, 256);
}

rr_status launch_ffn_fwd(const rr_moe_shape &s, const void *hidden, const void *W1, const void *W3, const void *W2,
                         const rr_route_tables &t, float *out, const FfnScratch &f, cudaStream_t st)
{
    const bool f32 = s.dtype == RR_F32;
    const int bk = f32 ? 32 : 64;
    const int grid = sm_count();
    if (grid <= 0) return RR_ERR_CUDA;
    const size_t Rp = rows_pad_max(s);

    CUtensorMap mXg, mW1, mW3, mAct, mActS, mW2, mH1, mH3;
    if (!make_map(&mXg, f.xg, Rp, s.d, f32, kTileM) ||
        !make_map(&mW1, W1, (size_t)s.E * s.d_ff, s.d, f32, 128) ||
        !make_map(&mW3, W3, (size_t)s.E * s.d_ff, s.d, f32, 128) ||
        !make_map(&mAct, f.act, Rp, s.d_ff, f32, kTileM) ||
        !make_map_bytes(&mActS, f.act, Rp, s.d_ff, f32 ? 4 : 2, f32, 32, f32 ? 128 : 64) ||   // 32 x 32 store boxes
        !make_map(&mW2, W2, (size_t)s.E * s.d, s.d_ff, f32, 128))   // each CTA of a pair stages 128 of the 256 rows
        return RR_ERR_CUDA;
    if (f.h1 && (!make_map_bytes(&mH1, f.h1, Rp, s.d_ff, 4, true, 32) ||   // 32 x 32 fp32 store boxes
                 !make_map_bytes(&mH3, f.h3, Rp, s.d_ff, 4, true, 32)))
        return RR_ERR_CUDA;

    if (cudaMemsetAsync(out, 0, (size_t)s.T * s.d * sizeof(float), st) != cudaSuccess) return RR_ERR_CUDA;
    k_tiles<<<1, 256, 0, st>>>(s.E, t.row_offset, f.mt_off);
    k_gather_rows<<<grid * 8, 256, 0, st>>>(s.E, (int)(s.d * elem_bytes(s)), f.mt_off, t.row_offset, t.row_token,
                                            static_cast<const char *>(hidden), static_cast<char *>(f.xg));
    auto mark = [&](int i) {
        if (s.trace && s.trace[i]) cudaEventRecord(static_cast<cudaEvent_t>(s.trace[i]), st);
    };
    mark(0);

    Params p{};
    p.E = s.E;
    p.mt_off = f.mt_off;
    p.row_offset = t.row_offset;
    p.row_token = t.row_token;
    p.row_weight = t.row_weight;
    p.status = &f.hdr->status;
    p.test_tfull_limit_ns = test_wait_limit_ns();

    // gate / up + SwiGLU
    p.KB = s.d / bk;
    p.N = s.d_ff;
    p.n_tiles = (s.d_ff + 127) / 128;
    cudaError_t err;
    if (f.h1)
        err = f32 ? launch<kGateUpTrain, true>(mXg, mXg, mW1, mW3, mH1, mH3, mActS, p, grid, st)
                  : launch<kGateUpTrain, false>(mXg, mXg, mW1, mW3, mH1, mH3, mActS, p, grid, st);
    else
        err = f32 ? launch<kGateUp, true>(mXg, mXg, mW1, mW3, mXg, mXg, mActS, p, grid, st)
                  : launch<kGateUp, false>(mXg, mXg, mW1, mW3, mXg, mXg, mActS, p, grid, st);
    if (err != cudaSuccess) return RR_ERR_CUDA;
    mark(1);

    // down + combine
    p.KB = s.d_ff / bk;
    p.N = s.d;
    p.n_tiles = (s.d + 255) / 256;
    p.out = out;
    err = f32 ? launch<kDown, true>(mAct, mAct, mW2, mW2, mAct, mAct, mAct, p, grid, st)
              : launch<kDown, false>(mAct, mAct, mW2, mW2, mAct, mAct, mAct, p, grid, st);
    mark(2);
    return err == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

}  // namespace rr
