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

__global__ void k_gate_tables(int T, int *mt_off, int *row_offset)
{
    mt_off[0] = 0;
    mt_off[1] = (T + kTileM - 1) / kTileM;
    row_offset[0] = 0;
    row_offset[1] = T;
}

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

size_t gate_bwd_workspace(int T, int E, int d)
{
    return align_up((size_t)gate_slabs(T, E, d) * E * d * sizeof(float), 256);
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
    k_gate_tables<<<1, 1, 0, st>>>(T, mt_off, row_offset);
    Params p{};
    p.E = 1;
    p.KB = d / (f32 ? 32 : 64);
    p.N = E;
    p.n_tiles = 1;
    p.mt_off = mt_off;
    p.row_offset = row_offset;
    p.out = logits;
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
    k_gate_tables<<<1, 1, 0, st>>>(T, mt_off, row_offset);
    Params p{};
    p.E = 1;
    p.KB = d / (f32 ? 32 : 64);
    p.N = E;
    p.n_tiles = 1;
    p.mt_off = mt_off;
    p.row_offset = row_offset;
    p.out = logits;
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

rr_status launch_gate_bwd(int T, int E, int d, int dtype, const float *dlogits, const void *hidden, const void *Wg,
                          float *dWg, float *dhidden, void *workspace, cudaStream_t st)
{
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
