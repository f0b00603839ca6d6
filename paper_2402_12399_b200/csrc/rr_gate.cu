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

constexpr int kSlabs = 32;  // token slabs of the dWg reduction

__global__ void k_gate_tables(int T, int *mt_off, int *row_offset)
{
    mt_off[0] = 0;
    mt_off[1] = (T + kTileM - 1) / kTileM;
    row_offset[0] = 0;
    row_offset[1] = T;
}

template <class TIn>
__device__ __forceinline__ float to_f32(TIn v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// dhidden[t, c] += sum_e dlogits[t, e] * Wg[e, c].  Block: 64 tokens x 256 columns; thread
// (ty, tx) = (tid / 32, tid % 32) owns tokens ty*8..+8 and columns tx + 32 j; experts in chunks
// of 32 through shared memory.  Every output element has one owner: no atomics.
template <class TIn>
__global__ void __launch_bounds__(256)
k_gate_dhidden(int T, int E, int d, const float *__restrict__ dlogits, const TIn *__restrict__ Wg,
               float *__restrict__ dhidden)
{
    __shared__ float ws[32][256];
    __shared__ float dls[64][33];
    const int tid = threadIdx.x, ty = tid >> 5, tx = tid & 31;
    const int t0 = blockIdx.y * 64, c0 = blockIdx.x * 256;
    float acc[8][8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) acc[a][b] = 0.0f;
    for (int e0 = 0; e0 < E; e0 += 32) {
        __syncthreads();
        for (int q = tid; q < 32 * 256; q += 256) {
            const int e = e0 + (q >> 8), c = c0 + (q & 255);
            ws[q >> 8][q & 255] = (e < E && c < d) ? to_f32<TIn>(Wg[(size_t)e * d + c]) : 0.0f;
        }
        for (int q = tid; q < 64 * 32; q += 256) {
            const int t = t0 + (q >> 5), e = e0 + (q & 31);
            dls[q >> 5][q & 31] = (t < T && e < E) ? dlogits[(size_t)t * E + e] : 0.0f;
        }
        __syncthreads();
#pragma unroll 4
        for (int e = 0; e < 32; ++e) {
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
            if (c < d) dhidden[(size_t)t * d + c] += acc[i][j];
        }
    }
}

// part[slab][e, c] = sum over the slab's tokens of dlogits[t, e] * hidden[t, c].  Block: 64
// experts x 256 columns x one slab; thread (ty, tx) owns experts ty*8..+8, columns tx + 32 j;
// tokens in chunks of 32 through shared memory.
template <class TIn>
__global__ void __launch_bounds__(256)
k_gate_dwg_partial(int T, int E, int d, int slab_tokens, const float *__restrict__ dlogits,
                   const TIn *__restrict__ hidden, float *__restrict__ part)
{
    __shared__ float hs[32][256];
    __shared__ float dls[32][65];
    const int tid = threadIdx.x, ty = tid >> 5, tx = tid & 31;
    const int c0 = blockIdx.x * 256, e0 = blockIdx.y * 64, slab = blockIdx.z;
    const int t_begin = slab * slab_tokens, t_end = min(T, t_begin + slab_tokens);
    float acc[8][8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) acc[a][b] = 0.0f;
    for (int tb = t_begin; tb < t_end; tb += 32) {
        __syncthreads();
        for (int q = tid; q < 32 * 256; q += 256) {
            const int t = tb + (q >> 8), c = c0 + (q & 255);
            hs[q >> 8][q & 255] = (t < t_end && c < d) ? to_f32<TIn>(hidden[(size_t)t * d + c]) : 0.0f;
        }
        for (int q = tid; q < 32 * 64; q += 256) {
            const int t = tb + (q >> 6), e = e0 + (q & 63);
            dls[q >> 6][q & 63] = (t < t_end && e < E) ? dlogits[(size_t)t * E + e] : 0.0f;
        }
        __syncthreads();
#pragma unroll 4
        for (int t = 0; t < 32; ++t) {
            float a[8], b[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) a[i] = dls[t][ty * 8 + i];
#pragma unroll
            for (int j = 0; j < 8; ++j) b[j] = hs[t][tx + 32 * j];
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
    }
    float *dst = part + (size_t)slab * E * d;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int e = e0 + ty * 8 + i;
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

size_t gate_bwd_workspace(int T, int E, int d)
{
    (void)T;
    return align_up((size_t)kSlabs * E * d * sizeof(float), 256);
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
    CUtensorMap mH, mW;
    if (!make_map(&mH, hidden, T, d, f32, kTileM) ||   // rows beyond T read as zeros
        !make_map(&mW, Wg, E, d, f32, 128))            // rows beyond E read as zeros
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
    p.status = &hdr->status;
    const cudaError_t err = f32 ? launch<kGate, true>(mH, mH, mW, mW, mH, mH, mH, p, grid, st)
                                : launch<kGate, false>(mH, mH, mW, mW, mH, mH, mH, p, grid, st);
    return err == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

rr_status launch_gate_bwd(int T, int E, int d, int dtype, const float *dlogits, const void *hidden, const void *Wg,
                          float *dWg, float *dhidden, void *workspace, cudaStream_t st)
{
    float *part = static_cast<float *>(workspace);
    const int slab_tokens = ((T + kSlabs - 1) / kSlabs + 31) / 32 * 32;
    const int slabs = (T + slab_tokens - 1) / slab_tokens;
    const dim3 gh((d + 255) / 256, (T + 63) / 64), gw((d + 255) / 256, (E + 63) / 64, slabs);
    if (dtype == RR_F32) {
        k_gate_dhidden<float><<<gh, 256, 0, st>>>(T, E, d, dlogits, static_cast<const float *>(Wg), dhidden);
        k_gate_dwg_partial<float><<<gw, 256, 0, st>>>(T, E, d, slab_tokens, dlogits, static_cast<const float *>(hidden), part);
    } else {
        k_gate_dhidden<__nv_bfloat16><<<gh, 256, 0, st>>>(T, E, d, dlogits, static_cast<const __nv_bfloat16 *>(Wg), dhidden);
        k_gate_dwg_partial<__nv_bfloat16><<<gw, 256, 0, st>>>(T, E, d, slab_tokens, dlogits,
                                                             static_cast<const __nv_bfloat16 *>(hidden), part);
    }
    const size_t n = (size_t)E * d;
    k_gate_dwg_reduce<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(n, slabs, part, dWg);
    return cudaGetLastError() == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

}  // namespace rr
