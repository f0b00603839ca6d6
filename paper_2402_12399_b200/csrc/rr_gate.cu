// Gate projection (Section 3, Eq. 1): a_ij = w_j^T x_i, the scores the router starts from, and its
// gradients.
//   forward : logits[T,E] = hidden[T,d] Wg[E,d]^T on the tensor cores (mode kGate of the GEMM
//             template: 256 tokens per CTA pair, the E <= 256 experts are the accumulator columns);
//             bound by the single read of `hidden`
//   backward: dhidden[T,d] += dlogits[T,E] Wg[E,d]   and   dWg[E,d] = dlogits^T hidden, both with a
//             contraction too short (E) or an output too small (E x d) for the tensor-core tiles:
//             register-tiled fp32 kernels, dWg summed over token slabs in a fixed order
#include "rr_gemm.cuh"

namespace rr {

using namespace gemm;

namespace {

constexpr int kMaxSlabs = 256;                   // token slabs of the dWg reduction, at most
constexpr size_t kMaxPartBytes = (size_t)64 << 20;  // ... and at most this much for their partial sums

// eight consecutive elements (16-byte aligned for bf16, 32-byte for fp32) as fp32
__device__ __forceinline__ void load8(const float *p, float (&v)[8])
{
    const float4 a = *reinterpret_cast<const float4 *>(p), b = *reinterpret_cast<const float4 *>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&v)[8])
{
    const uint4 u = *reinterpret_cast<const uint4 *>(p);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// rows [r0, r0+32) x columns [c0, c0+256) of a row-major [rows_total, d] matrix into a [32][256]
// fp32 tile (zeros outside); d is a multiple of 8
template <class TIn>
__device__ __forceinline__ void stage_32x256(float (*tile)[256], const TIn *__restrict__ src, int r0, int rows_end, int c0,
                                             int d)
{
    for (int q = threadIdx.x; q < 32 * 32; q += 256) {
        const int r = r0 + (q >> 5), c = c0 + (q & 31) * 8;
        float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (r < rows_end && c < d) load8(src + (size_t)r * d + c, v);
#pragma unroll
        for (int i = 0; i < 8; ++i) tile[q >> 5][(q & 31) * 8 + i] = v[i];
    }
}

// dhidden[t, c] += sum_e dlogits[t, e] * Wg[e, c].  Block: 64 tokens x 256 columns; thread
// (ty, tx) = (tid / 32, tid % 32) owns tokens ty*8..+8 and columns tx + 32 j; experts in chunks
// of 32 through shared memory.  Every output element has one owner: no atomics.
template <class TIn>
__global__ void __launch_bounds__(256)
k_gate_dhidden(int T, int E, int d, const float *__restrict__ dlogits, const TIn *__restrict__ Wg,
               float *dhidden)
{
    __shared__ float ws[32][256];
    __shared__ float dls[64][33];
    const int tid = threadIdx.x, ty = tid >> 5, tx = tid & 31;
    const int t0 = blockIdx.y * 64, c0 = blockIdx.x * 256;
    // the accumulators start from the values already in dhidden: their loads are in flight while
    // the first operands are staged, and the end of the kernel is plain stores
    float acc[8][8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const int t = t0 + ty * 8 + a, c = c0 + tx + 32 * b;
            acc[a][b] = (t < T && c < d) ? dhidden[(size_t)t * d + c] : 0.0f;
        }
    for (int e0 = 0; e0 < E; e0 += 32) {
        __syncthreads();
        stage_32x256<TIn>(ws, Wg, e0, E, c0, d);
        for (int q = tid; q < 64 * 32; q += 256) {
            const int t = t0 + (q >> 5), e = e0 + (q & 31);
            dls[q >> 5][q & 31] = (t < T && e < E) ? dlogits[(size_t)t * E + e] : 0.0f;
        }
        __syncthreads();
        const int ne = min(32, E - e0);
#pragma unroll 4
        for (int e = 0; e < ne; ++e) {
            float a[8], b[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) a[i] = dls[ty * 8 + i][e];
#pragma unroll
            for (int j = 0; j < 8; ++j) b[j] = ws[e][tx + 32 * j];
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int t = t0 + ty * 8 + i;
        if (t >= T) continue;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int c = c0 + tx + 32 * j;
            if (c < d) dhidden[(size_t)t * d + c] = acc[i][j];
        }
    }
}

// part[slab][e, c] = sum over the slab's tokens of dlogits[t, e] * hidden[t, c].  Block: 8*EPT
// experts x 256 columns x one slab; thread (ty, tx) owns experts ty*EPT..+EPT, columns tx + 32 j;
// tokens in chunks of 32 through shared memory.
template <class TIn, int EPT>
__global__ void __launch_bounds__(256)
k_gate_dwg_partial(int T, int E, int d, int slab_tokens, const float *__restrict__ dlogits,
                   const TIn *__restrict__ hidden, float *__restrict__ part)
{
    __shared__ float hs[32][256];
    __shared__ float dls[32][65];
    const int tid = threadIdx.x, ty = tid >> 5, tx = tid & 31;
    const int c0 = blockIdx.x * 256, e0 = blockIdx.y * (8 * EPT), slab = blockIdx.z;
    const int t_begin = slab * slab_tokens, t_end = min(T, t_begin + slab_tokens);
    float acc[EPT][8];
#pragma unroll
    for (int a = 0; a < EPT; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) acc[a][b] = 0.0f;
    for (int tb = t_begin; tb < t_end; tb += 32) {
        __syncthreads();
        stage_32x256<TIn>(hs, hidden, tb, t_end, c0, d);
        for (int q = tid; q < 32 * 8 * EPT; q += 256) {
            const int t = tb + q / (8 * EPT), e = e0 + q % (8 * EPT);
            dls[q / (8 * EPT)][q % (8 * EPT)] = (t < t_end && e < E) ? dlogits[(size_t)t * E + e] : 0.0f;
        }
        __syncthreads();
#pragma unroll 4
        for (int t = 0; t < 32; ++t) {
            float a[EPT], b[8];
#pragma unroll
            for (int i = 0; i < EPT; ++i) a[i] = dls[t][ty * EPT + i];
#pragma unroll
            for (int j = 0; j < 8; ++j) b[j] = hs[t][tx + 32 * j];
#pragma unroll
            for (int i = 0; i < EPT; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
    }
    float *dst = part + (size_t)slab * E * d;
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
        const int e = e0 + ty * EPT + i;
        if (e >= E) continue;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int c = c0 + tx + 32 * j;
            if (c < d) dst[(size_t)e * d + c] = acc[i][j];
        }
    }
}

// dWg = sum of the slabs' partial sums, in slab order.
__global__ void __launch_bounds__(256)
k_gate_dwg_reduce(size_t n, int slabs, const float *__restrict__ part, float *__restrict__ dWg)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float s = 0.0f;
    for (int k = 0; k < slabs; ++k) s += part[(size_t)k * n + i];
    dWg[i] = s;
}

}  // namespace

size_t gate_fwd_workspace(int T, int E, int d)
{
    (void)T; (void)E; (void)d;
    Carver c(nullptr);
    c.take<Header>(1);
    c.take<int>(2);
    c.take<int>(2);
    return align_up(c.off, 256);
}

// Experts per thread of the dWg kernel and the number of token slabs: enough blocks to fill the
// GPU about four times over, within the budget for the partial sums.
static int gate_ept(int E) { return E <= 8 ? 1 : E <= 16 ? 2 : E <= 32 ? 4 : 8; }
static int gate_slabs(int T, int E, int d)
{
    const int ept = gate_ept(E);
    const long tiles = (long)((d + 255) / 256) * ((E + 8 * ept - 1) / (8 * ept));
    long slabs = (600 + tiles - 1) / tiles;
    const long by_bytes = (long)(kMaxPartBytes / ((size_t)E * d * sizeof(float)));
    slabs = slabs < by_bytes ? slabs : by_bytes;
    slabs = slabs < kMaxSlabs ? slabs : kMaxSlabs;
    const long by_tokens = (T + 31) / 32;
    slabs = slabs < by_tokens ? slabs : by_tokens;
    return (int)(slabs < 1 ? 1 : slabs);
}

struct GateBwdTc;
static size_t gate_bwd_tc_layout(void *ws, int T, int E, int d, GateBwdTc *g);
static size_t gate_bwd_tc_bytes(int T, int E, int d);

size_t gate_bwd_workspace(int T, int E, int d)
{
    // (the element type is not known here: room for the tensor-core path of bf16 and for the fp32 path)
    const size_t a = align_up((size_t)gate_slabs(T, E, d) * E * d * sizeof(float), 256), b = gate_bwd_tc_bytes(T, E, d);
    return a > b ? a : b;
}

rr_status launch_gate_fwd(int T, int E, int d, int dtype, const void *hidden, const void *Wg, float *logits,
                          void *workspace, cudaStream_t st)
{
    const bool f32 = dtype == RR_F32;
    const int grid = sm_count();
    if (grid <= 0) return RR_ERR_CUDA;
    Carver c(workspace);
    Header *hdr = c.take<Header>(1);
    int *mt_off = c.take<int>(2);
    int *row_offset = c.take<int>(2);
    // the MMA is 256 tokens x gate_n experts: gate_n = E rounded up to 16, each CTA of a pair stages
    // gate_n / 2 rows of Wg per k-block (1 KB for E <= 16), which leaves room for a deep ring of
    // `hidden` tiles: the kernel lives on bytes in flight
    const int gate_n = (E + 15) / 16 * 16;
    const int stage_bytes = kABytes + gate_n * 64;
    int stages = (int)((232448 - 1024 - sizeof(Shared)) / stage_bytes);
    stages = stages > 12 ? 12 : stages;
    CUtensorMap mH, mW;
    if (!make_map(&mH, hidden, T, d, f32, kTileM) ||       // rows beyond T read as zeros
        !make_map(&mW, Wg, E, d, f32, gate_n / 2))         // rows beyond E read as zeros
        return RR_ERR_CUDA;
    Params p{};
    p.E = 1;
    p.KB = d / (f32 ? 32 : 64);
    p.N = E;
    p.n_tiles = 1;
    p.mt_off = mt_off;
    p.row_offset = row_offset;
    p.out = logits;
    p.gate_T = T;
    p.gate_n = gate_n;
    p.gate_stages = stages;
    p.status = &hdr->status;
    const size_t smem = 1024 + (size_t)stages * stage_bytes + sizeof(Shared);
    const cudaError_t err = f32 ? launch<kGate, true>(mH, mH, mW, mW, mH, mH, mH, p, grid, st, smem)
                                : launch<kGate, false>(mH, mH, mW, mW, mH, mH, mH, p, grid, st, smem);
    return err == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

// The projection with the selection of Eq. 1 and Section 4.1 in its epilogue (mode kGateSel of the GEMM
// template): logits are written once and never read back by the router.  `tabs` = 4 ints of scratch.
rr_status launch_gate_sel(int T, int E, int d, int dtype, const void *hidden, const void *Wg, float *logits, int k, int G,
                          int *sel_expert, float *sel_val, int *sel_h, float *sel_ah, float *psum, int *status, int *tabs,
                          cudaStream_t st)
{
    const bool f32 = dtype == RR_F32;
    const int grid = sm_count();
    if (grid <= 0) return RR_ERR_CUDA;
    int *mt_off = tabs, *row_offset = tabs + 2;
    const int gate_n = (E + 15) / 16 * 16;
    const int stage_bytes = kABytes + gate_n * 64;
    int stages = (int)((232448 - 1024 - sizeof(Shared)) / stage_bytes);
    stages = stages > 12 ? 12 : stages;
    CUtensorMap mH, mW;
    if (!make_map(&mH, hidden, T, d, f32, kTileM) || !make_map(&mW, Wg, E, d, f32, gate_n / 2)) return RR_ERR_CUDA;
    Params p{};
    p.E = 1;
    p.KB = d / (f32 ? 32 : 64);
    p.N = E;
    p.n_tiles = 1;
    p.mt_off = mt_off;
    p.row_offset = row_offset;
    p.out = logits;
    p.gate_T = T;
    p.gate_n = gate_n;
    p.gate_stages = stages;
    p.status = status;
    p.sel_k = k;
    p.sel_G = G;
    p.sel_T = T;
    p.sel_expert = sel_expert;
    p.sel_val = sel_val;
    p.sel_h = sel_h;
    p.sel_ah = sel_ah;
    p.sel_psum = psum;
    const size_t smem = 1024 + (size_t)stages * stage_bytes + sizeof(Shared);
    const cudaError_t err = f32 ? launch<kGateSel, true>(mH, mH, mW, mW, mH, mH, mH, p, grid, st, smem)
                                : launch<kGateSel, false>(mH, mH, mW, mW, mH, mH, mH, p, grid, st, smem);
    return err == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

// ---- backward on the tensor cores (bf16 inputs) -------------------------------------------------------
// dlogits is fp32; the MMAs take bf16.  It is split into a bf16 head and a bf16 remainder (together 16
// mantissa bits: 2^-17 relative), laid side by side as P[T, Mp] = [head | remainder | 0], Mp a multiple of
// 64.  Then
//   dhidden += P . [Wg ; Wg ; 0]            runs as mode kDenseAdd of the GEMM template (rows = tokens, K = Mp, 32 x 32
//                                            pieces added by TMA reduce), against WgT2[d, Mp] = [Wg^T | Wg^T | 0];
//   dWg      = head^T hidden + rem^T hidden  runs as mode kWgrad over slabs of tokens ("experts" = slabs, M = the
//                                            2 E8 columns of P), partial[slab][2 E8][d], added up in slab order.
struct GateBwdTc {
    int E8, Mp, nslabs, slab_tiles;
    float *partial;        // [nslabs][2 E8][d]
    __nv_bfloat16 *P;      // [T][Mp]
    __nv_bfloat16 *WgT2;   // [d][Mp]
    int *mt_off;           // [nslabs + 1] tiles of 128 tokens per slab (prefix); [kMaxE + 2 ..]: the one-expert tables of kDenseAdd
    int *status;
};

static size_t gate_bwd_tc_layout(void *ws, int T, int E, int d, GateBwdTc *g)
{
    const size_t Tn = T > 0 ? T : 1;
    g->E8 = (E + 7) & ~7;
    g->Mp = (2 * g->E8 + 63) & ~63;
    const int tiles = (int)((Tn + kTileM - 1) / kTileM);
    const int per = ((2 * g->E8 + 255) / 256) * ((d + 255) / 256);   // work items per slab
    int want = (4 * 74 + per - 1) / per;                              // about four items per CTA pair
    want = want < 1 ? 1 : (want > kMaxE ? kMaxE : want);
    want = want > tiles ? tiles : want;
    g->slab_tiles = (tiles + want - 1) / want;
    g->nslabs = (tiles + g->slab_tiles - 1) / g->slab_tiles;
    Carver c(ws);
    Header *hdr = c.take<Header>(1);
    g->status = hdr ? &hdr->status : nullptr;
    g->partial = c.take<float>((size_t)g->nslabs * 2 * g->E8 * d);
    g->P = c.take<__nv_bfloat16>(Tn * g->Mp);
    g->WgT2 = c.take<__nv_bfloat16>((size_t)d * g->Mp);
    g->mt_off = c.take<int>(kMaxE + 8);
    return align_up(c.off, 256);
}

static size_t gate_bwd_tc_bytes(int T, int E, int d)
{
    GateBwdTc g;
    return gate_bwd_tc_layout(nullptr, T, E, d, &g);
}

// P; one thread per (token, column of P)
__global__ void __launch_bounds__(256)
k_gate_split(int T, int E, int E8, int Mp, const float *__restrict__ dl, __nv_bfloat16 *__restrict__ P)
{
    const size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= (size_t)T * Mp) return;
    const int i = (int)(q / Mp), c = (int)(q - (size_t)i * Mp);
    float v = 0.0f;
    if (c < E) {
        v = dl[(size_t)i * E + c];
    } else if (c >= E8 && c < E8 + E) {
        const float x = dl[(size_t)i * E + (c - E8)];
        v = x - __bfloat162float(__float2bfloat16_rn(x));   // what the head leaves (exact in fp32)
    }
    P[q] = __float2bfloat16_rn(v);
}

// WgT2[c][m] = Wg[m][c] for m < E and Wg[m - E8][c] for E8 <= m < E8 + E, 0 elsewhere; the slab and tile tables
__global__ void __launch_bounds__(256)
k_gate_wt(int T, int E, int E8, int Mp, int d, int nslabs, int slab_tiles, const __nv_bfloat16 *__restrict__ Wg,
          __nv_bfloat16 *__restrict__ WgT2, int *__restrict__ mt_off)
{
    const size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q < (size_t)d * Mp) {
        const int c = (int)(q / Mp), m = (int)(q - (size_t)c * Mp);
        const int e = m < E ? m : ((m >= E8 && m < E8 + E) ? m - E8 : -1);
        WgT2[q] = e >= 0 ? Wg[(size_t)e * d + c] : __float2bfloat16_rn(0.0f);
    }
    if (q <= (size_t)nslabs) {
        const int tiles = (T + kTileM - 1) / kTileM;
        const int t = (int)q * slab_tiles;
        mt_off[q] = t < tiles ? t : tiles;
    }
    if (q == 0) {  // the tables of the one "expert" whose rows are the tokens (kDenseAdd)
        mt_off[kMaxE + 2] = 0;
        mt_off[kMaxE + 3] = (T + kTileM - 1) / kTileM;
        mt_off[kMaxE + 4] = 0;
        mt_off[kMaxE + 5] = T;
    }
}

// dWg[e][c] = sum over the slabs, in slab order, of the head's and the remainder's partial products
__global__ void __launch_bounds__(256)
k_gate_dwg_sum(int E, int E8, int d, int nslabs, const float *__restrict__ partial, float *__restrict__ dWg)
{
    const size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= (size_t)E * d) return;
    const int e = (int)(q / d), c = (int)(q - (size_t)e * d);
    float acc = 0.0f;
    for (int s = 0; s < nslabs; ++s) {
        const float *base = partial + (size_t)s * 2 * E8 * d;
        acc += base[(size_t)e * d + c] + base[(size_t)(E8 + e) * d + c];
    }
    dWg[q] = acc;
}

static rr_status launch_gate_bwd_tc(int T, int E, int d, const float *dlogits, const void *hidden, const void *Wg,
                                    float *dWg, float *dhidden, void *workspace, cudaStream_t st)
{
    const int grid = sm_count();
    if (grid <= 0) return RR_ERR_CUDA;
    GateBwdTc g;
    gate_bwd_tc_layout(workspace, T, E, d, &g);
    if (cudaMemsetAsync(g.status, 0, sizeof(int), st) != cudaSuccess) return RR_ERR_CUDA;
    const size_t nP = (size_t)T * g.Mp, nW = (size_t)d * g.Mp;
    k_gate_split<<<(unsigned)((nP + 255) / 256), 256, 0, st>>>(T, E, g.E8, g.Mp, dlogits, g.P);
    const size_t nq = nW > (size_t)g.nslabs + 1 ? nW : (size_t)g.nslabs + 1;
    k_gate_wt<<<(unsigned)((nq + 255) / 256), 256, 0, st>>>(T, E, g.E8, g.Mp, d, g.nslabs, g.slab_tiles,
                                                            static_cast<const __nv_bfloat16 *>(Wg), g.WgT2, g.mt_off);
    CUtensorMap mPk, mWt, mPm, mH, mS, mDh;
    if (!make_map(&mPk, g.P, T, g.Mp, false, kTileM) ||          // K-major A tiles of kDown
        !make_map(&mWt, g.WgT2, d, g.Mp, false, 128) ||          // K-major B tiles: 128 of the pair's 256 output columns per CTA
        !make_map(&mPm, g.P, T, g.Mp, false, 64) ||              // MN-major panels of kWgrad
        !make_map(&mH, hidden, T, d, false, 64) ||
        !make_map_3d_f32(&mS, g.partial, g.nslabs, 2 * g.E8, d) ||
        !make_map_bytes(&mDh, dhidden, T, d, 4, true, 32))       // 32 x 32 fp32 boxes of the reduce-add
        return RR_ERR_CUDA;
    Params p{};
    p.status = g.status;
    // dhidden[token] += P . WgT2^T
    p.E = 1;
    p.KB = g.Mp / 64;
    p.N = d;
    p.n_tiles = (d + 255) / 256;
    p.mt_off = g.mt_off + kMaxE + 2;
    p.row_offset = g.mt_off + kMaxE + 4;
    p.out = dhidden;
    if (launch<kDenseAdd, false>(mPk, mPk, mWt, mWt, mDh, mDh, mDh, p, grid, st) != cudaSuccess) return RR_ERR_CUDA;
    // partial[slab] = P_slab^T hidden_slab
    p.E = g.nslabs;
    p.KB = 0;
    p.M = 2 * g.E8;
    p.m_tiles = (2 * g.E8 + 2 * kTileM - 1) / (2 * kTileM);
    p.N = d;
    p.n_tiles = (d + 255) / 256;
    p.mt_off = g.mt_off;
    p.dw = g.partial;
    if (launch<kWgrad, false>(mPm, mPm, mH, mH, mS, mS, mS, p, grid, st) != cudaSuccess) return RR_ERR_CUDA;
    const size_t n = (size_t)E * d;
    k_gate_dwg_sum<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(E, g.E8, d, g.nslabs, g.partial, dWg);
    return cudaGetLastError() == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

rr_status launch_gate_bwd(int T, int E, int d, int dtype, const float *dlogits, const void *hidden, const void *Wg,
                          float *dWg, float *dhidden, void *workspace, cudaStream_t st)
{
    if (dtype == RR_BF16) return launch_gate_bwd_tc(T, E, d, dlogits, hidden, Wg, dWg, dhidden, workspace, st);
    float *part = static_cast<float *>(workspace);
    const int ept = gate_ept(E);
    const int want = gate_slabs(T, E, d);
    const int slab_tokens = ((T + want - 1) / want + 31) / 32 * 32;
    const int slabs = (T + slab_tokens - 1) / slab_tokens;   // <= want
    const dim3 gh((d + 255) / 256, (T + 63) / 64), gw((d + 255) / 256, (E + 8 * ept - 1) / (8 * ept), slabs);
    const bool f32 = dtype == RR_F32;
    if (f32)
        k_gate_dhidden<float><<<gh, 256, 0, st>>>(T, E, d, dlogits, static_cast<const float *>(Wg), dhidden);
    else
        k_gate_dhidden<__nv_bfloat16><<<gh, 256, 0, st>>>(T, E, d, dlogits, static_cast<const __nv_bfloat16 *>(Wg), dhidden);
#define RR_GATE_DWG(TIN, EPT) \
    k_gate_dwg_partial<TIN, EPT><<<gw, 256, 0, st>>>(T, E, d, slab_tokens, dlogits, static_cast<const TIN *>(hidden), part)
    if (f32) {
        if (ept == 1) RR_GATE_DWG(float, 1); else if (ept == 2) RR_GATE_DWG(float, 2);
        else if (ept == 4) RR_GATE_DWG(float, 4); else RR_GATE_DWG(float, 8);
    } else {
        if (ept == 1) RR_GATE_DWG(__nv_bfloat16, 1); else if (ept == 2) RR_GATE_DWG(__nv_bfloat16, 2);
        else if (ept == 4) RR_GATE_DWG(__nv_bfloat16, 4); else RR_GATE_DWG(__nv_bfloat16, 8);
    }
#undef RR_GATE_DWG
    const size_t n = (size_t)E * d;
    k_gate_dwg_reduce<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(n, slabs, part, dWg);
    return cudaGetLastError() == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

}  // namespace rr
