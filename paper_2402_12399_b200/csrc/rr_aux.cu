// Load-balance loss of the top-k router (Section 5.1 gives its weight; the formula is the one of
// the work cited there):
//     f_e = (1/T) #{ i : first choice of token i is e },   P_e = (1/T) sum_i softmax(a_i)_e,
//     L = alpha E sum_e f_e P_e,     dL/da_ij = alpha E / T  g_ij ( f_j - sum_e f_e g_ie )   (f constant).
// One read of the logits forward, one read and one write (or read-modify-write) backward: both are
// bound by HBM at sizes above L2 and by launch latency below.  A token is handled by a group of GS
// lanes (a power of two, 1..32), each keeping up to eight columns in registers.
// Column sums are carried per lane over a contiguous slab of tokens, then added over the groups of a
// warp, the warps of a block and the blocks in a fixed order: the result repeats bit for bit.
#include "rr_ffn.cuh"

namespace rr {

namespace {

constexpr int kAuxThreads = 256;
constexpr int kAuxWarps = kAuxThreads / 32;
constexpr int kAuxMaxBlocks = 1184;  // 8 per SM
constexpr int kFwdMaxBlocks = 592;   // forward: 4 per SM (the second kernel's one block reads a row per block)
constexpr int kFinalThreads = 1024;

template <int GS>
__device__ __forceinline__ float group_max(float v)
{
#pragma unroll
    for (int o = GS / 2; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
template <int GS>
__device__ __forceinline__ float group_sum(float v)
{
#pragma unroll
    for (int o = GS / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Which columns a lane keeps.  Vector layout (E a multiple of 4): float4 pieces, piece q of lane gl
// covers columns q*4*GS + 4*gl .. + 3, so one load instruction of a group reads 16*GS contiguous bytes.
// Scalar layout (any E): element c is column c*GS + gl.
template <int GS, bool VEC>
__device__ __forceinline__ int column_of(int c, int gl)
{
    return VEC ? (c >> 2) * (4 * GS) + 4 * gl + (c & 3) : c * GS + gl;
}

// softmax of one token over the group's lanes; a lane without a token (ok == false) takes part in
// the shuffles and gets zeros
template <int GS, int CPL, bool VEC>
__device__ __forceinline__ void softmax_row(const float *__restrict__ a, bool ok, int E, int gl, float (&g)[CPL])
{
    if constexpr (VEC) {
#pragma unroll
        for (int q = 0; q < CPL / 4; ++q) {
            const int j = column_of<GS, true>(4 * q, gl);
            float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            if (ok && j < E) v = __ldg(reinterpret_cast<const float4 *>(a + j));
            g[4 * q] = v.x; g[4 * q + 1] = v.y; g[4 * q + 2] = v.z; g[4 * q + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int c = 0; c < CPL; ++c) {
            const int j = column_of<GS, false>(c, gl);
            g[c] = (ok && j < E) ? __ldg(a + j) : -INFINITY;
        }
    }
    float m = -INFINITY;
#pragma unroll
    for (int c = 0; c < CPL; ++c) m = fmaxf(m, g[c]);
    m = group_max<GS>(m);
    float z = 0.f;
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
        g[c] = ok ? expf(g[c] - m) : 0.f;  // exp(-inf) = 0 for the columns past E
        z += g[c];
    }
    z = group_sum<GS>(z);
    const float inv = ok ? 1.0f / z : 0.f;
#pragma unroll
    for (int c = 0; c < CPL; ++c) g[c] *= inv;
}

// one first choice into the block's histogram; a value outside 0..E-1 is reported and skipped
constexpr int kNoToken = INT32_MIN;
__device__ __forceinline__ void count_first(int e, int E, int *cnt, int *status)
{
    if (e == kNoToken) return;
    if (e >= 0 && e < E) atomicAdd(&cnt[e], 1);
    else latch_status(status, RR_ERR_INVALID_ARG);
}

// Forward, first kernel: softmax column sums and first-choice counts of a slab of tokens per block.
template <int GS, int CPL, bool VEC>
__global__ void __launch_bounds__(kAuxThreads) k_aux_partial(const float *__restrict__ logits,
                                                             const int32_t *__restrict__ first, int stride, int T,
                                                             int E, int slab, float *__restrict__ partial,
                                                             int *__restrict__ pcount, int *status)
{
    constexpr int TPW = 32 / GS;
    __shared__ float red[kAuxWarps][kMaxE];
    __shared__ int cnt[kMaxE];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, grp = lane / GS, gl = lane % GS;
    // the second kernel is launched as a programmatic dependent: it may be made ready at once (it waits for the
    // whole of this grid before it reads the partial sums)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int j = threadIdx.x; j < kMaxE; j += kAuxThreads) cnt[j] = 0;
    __syncthreads();
    const int t0 = blockIdx.x * slab, t1 = min(T, t0 + slab);
    float acc[CPL] = {};
    for (int base = t0 + warp * TPW; base < t1; base += 2 * kAuxWarps * TPW) {  // two tokens in flight per group
        const int ta = base + grp, tb = ta + kAuxWarps * TPW;
        const bool oka = ta < t1, okb = tb < t1;
        int ea = kNoToken, eb = kNoToken;  // fetched ahead of the rows: the two latencies overlap
        if (gl == 0 && oka) ea = __ldg(first + (size_t)ta * stride);
        if (gl == 0 && okb) eb = __ldg(first + (size_t)tb * stride);
        float ga[CPL], gb[CPL];
        softmax_row<GS, CPL, VEC>(logits + (size_t)(oka ? ta : 0) * E, oka, E, gl, ga);
        softmax_row<GS, CPL, VEC>(logits + (size_t)(okb ? tb : 0) * E, okb, E, gl, gb);
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[c] += ga[c];
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[c] += gb[c];
        count_first(ea, E, cnt, status);
        count_first(eb, E, cnt, status);
    }
    // groups of the warp, then warps of the block, in a fixed order
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
#pragma unroll
        for (int o = GS; o < 32; o <<= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], o);
        const int j = column_of<GS, VEC>(c, gl);
        if (grp == 0 && j < E) red[warp][j] = acc[c];
    }
    __syncthreads();
    for (int j = threadIdx.x; j < E; j += kAuxThreads) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kAuxWarps; ++w) s += red[w][j];
        partial[(size_t)blockIdx.x * E + j] = s;
        pcount[(size_t)blockIdx.x * E + j] = cnt[j];
    }
}

// Forward, second kernel (one block): thread (r, j) adds the rows r, r + R, ... of column j (of the four
// columns from j on when VEC); the R sums of a column are then added in the order of r (a tree over r
// with a block barrier per level measured slower than this loop).
template <bool VEC>
__global__ void __launch_bounds__(kFinalThreads) k_aux_final(const float *__restrict__ partial,
                                                             const int *__restrict__ pcount, int nb, int T, int E,
                                                             int epad, float alpha, float *loss, float *f, float *P)
{
    constexpr int V = VEC ? 4 : 1;
    __shared__ float sp[kFinalThreads * V];
    __shared__ int sc[kFinalThreads * V];
    __shared__ float prod[kMaxE];
    const int cols = epad / V, R = kFinalThreads / cols, r = threadIdx.x / cols, j = (threadIdx.x % cols) * V;
    float s[V] = {};
    int n[V] = {};
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the first kernel has completed and its sums are visible
    if (j < E) {
#pragma unroll 4
        for (int b = r; b < nb; b += R) {
            if constexpr (VEC) {
                const float4 x = *reinterpret_cast<const float4 *>(partial + (size_t)b * E + j);
                const int4 y = *reinterpret_cast<const int4 *>(pcount + (size_t)b * E + j);
                s[0] += x.x; s[1] += x.y; s[2] += x.z; s[3] += x.w;
                n[0] += y.x; n[1] += y.y; n[2] += y.z; n[3] += y.w;
            } else {
                s[0] += partial[(size_t)b * E + j];
                n[0] += pcount[(size_t)b * E + j];
            }
        }
    }
#pragma unroll
    for (int v = 0; v < V; ++v) {
        sp[r * epad + j + v] = s[v];
        sc[r * epad + j + v] = n[v];
    }
    __syncthreads();
    if (threadIdx.x < E) {
        float tot = 0.f;
        int cnt = 0;
        for (int q = 0; q < R; ++q) {
            tot += sp[q * epad + threadIdx.x];
            cnt += sc[q * epad + threadIdx.x];
        }
        const float fj = (float)cnt / (float)T, pj = tot / (float)T;
        f[threadIdx.x] = fj;
        if (P) P[threadIdx.x] = pj;
        prod[threadIdx.x] = fj * pj;
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        float tot = 0.f;
        for (int e = threadIdx.x; e < E; e += 32) tot += prod[e];
        tot = group_sum<32>(tot);
        if (threadIdx.x == 0) *loss = alpha * (float)E * tot;
    }
}

template <int GS, int CPL, bool VEC>
__global__ void __launch_bounds__(kAuxThreads) k_aux_bwd(const float *__restrict__ logits, const float *__restrict__ f,
                                                         int T, int E, float coef, int accumulate,
                                                         float *__restrict__ dlogits)
{
    constexpr int TPW = 32 / GS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, grp = lane / GS, gl = lane % GS;
    float fj[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
        const int j = column_of<GS, VEC>(c, gl);
        fj[c] = j < E ? __ldg(f + j) : 0.f;
    }
    const int step = gridDim.x * kAuxWarps * TPW;
    for (int base = (blockIdx.x * kAuxWarps + warp) * TPW; base < T; base += step) {
        const int t = base + grp;
        const bool ok = t < T;
        float g[CPL];
        softmax_row<GS, CPL, VEC>(logits + (size_t)(ok ? t : 0) * E, ok, E, gl, g);
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < CPL; ++c) dot += fj[c] * g[c];
        dot = group_sum<GS>(dot);
        if (!ok) continue;
        float *o = dlogits + (size_t)t * E;
#pragma unroll
        for (int c = 0; c < CPL; ++c) g[c] = coef * g[c] * (fj[c] - dot);
        if constexpr (VEC) {
#pragma unroll
            for (int q = 0; q < CPL / 4; ++q) {
                const int j = column_of<GS, true>(4 * q, gl);
                if (j >= E) continue;
                float4 *dst = reinterpret_cast<float4 *>(o + j);
                float4 v = make_float4(g[4 * q], g[4 * q + 1], g[4 * q + 2], g[4 * q + 3]);
                if (accumulate) {  // no contraction: the sum of what the other mode writes
                    const float4 old = *dst;
                    v = make_float4(__fadd_rn(old.x, v.x), __fadd_rn(old.y, v.y), __fadd_rn(old.z, v.z),
                                    __fadd_rn(old.w, v.w));
                }
                *dst = v;
            }
        } else {
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                const int j = column_of<GS, false>(c, gl);
                if (j < E) o[j] = accumulate ? __fadd_rn(o[j], g[c]) : g[c];
            }
        }
    }
}

// Lane layout for E experts: with E a multiple of 4 a lane keeps up to eight columns as float4 pieces
// and the group is as small as that allows (few shuffle steps: the reductions over the group, not the
// loads, bound these kernels otherwise); any other E takes scalar columns over up to 32 lanes.
struct Layout {
    bool vec;
    int gs, cpl;
};
Layout layout_of(int E)
{
    int epad = 1;
    while (epad < E) epad <<= 1;
    if (E % 4 == 0) {
        const int cpl = epad < 8 ? 4 : 8;
        return {true, epad / cpl, cpl};
    }
    return {false, epad < 32 ? epad : 32, epad <= 32 ? 1 : epad / 32};
}

int aux_blocks(int T, int E)
{
    const int per_pass = 2 * kAuxWarps * (32 / layout_of(E).gs);  // tokens a block takes per loop pass
    const int nb = (T + 2 * per_pass - 1) / (2 * per_pass);
    return nb < 1 ? 1 : (nb > kFwdMaxBlocks ? kFwdMaxBlocks : nb);
}

struct AuxScratch {
    Header *hdr;
    int *pcount;      // [blocks][E] first choices counted per block
    float *partial;   // [blocks][E] softmax column sums per block
};

size_t aux_layout(void *ws, int T, int E, AuxScratch *s)
{
    Carver c(ws);
    AuxScratch a;
    a.hdr = c.take<Header>(1);
    a.pcount = c.take<int>((size_t)aux_blocks(T, E) * E);
    a.partial = c.take<float>((size_t)aux_blocks(T, E) * E);
    if (s) *s = a;
    return align_up(c.off, 256);
}

template <int GS, int CPL, bool VEC>
rr_status run_fwd(int T, int E, int stride, const float *logits, const int32_t *first, float alpha, float *loss,
                  float *f, float *P, const AuxScratch &a, cudaStream_t st)
{
    const int nb = aux_blocks(T, E), slab = (T + nb - 1) / nb;
    int epad = 1;
    while (epad < E) epad <<= 1;
    k_aux_partial<GS, CPL, VEC><<<nb, kAuxThreads, 0, st>>>(logits, first, stride, T, E, slab, a.partial, a.pcount,
                                                            &a.hdr->status);
    // the one-block second kernel as a programmatic dependent of the first: its launch overlaps the first's run
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(kFinalThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float *partial = a.partial;
    const int *pcount = a.pcount;
    if (cudaLaunchKernelEx(&cfg, k_aux_final<VEC>, partial, pcount, nb, T, E, epad, alpha, loss, f, P) != cudaSuccess) {
        (void)cudaGetLastError();
        k_aux_final<VEC><<<1, kFinalThreads, 0, st>>>(a.partial, a.pcount, nb, T, E, epad, alpha, loss, f, P);
    }
    return cudaGetLastError() == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

template <int GS, int CPL, bool VEC>
rr_status run_bwd(int T, int E, const float *logits, const float *f, float coef, int accumulate, float *dlogits,
                  cudaStream_t st)
{
    const int per_block = kAuxWarps * (32 / GS);
    int nb = (T + per_block - 1) / per_block;
    if (nb > kAuxMaxBlocks) nb = kAuxMaxBlocks;
    k_aux_bwd<GS, CPL, VEC><<<nb, kAuxThreads, 0, st>>>(logits, f, T, E, coef, accumulate, dlogits);
    return cudaGetLastError() == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

// calls F<GS, CPL, VEC>::run(args...) for the layout of E
#define RR_AUX_DISPATCH(FN, ...)                                                   \
    do {                                                                           \
        const Layout l = layout_of(E);                                             \
        if (l.vec) {                                                               \
            if (l.cpl == 4) return FN<1, 4, true>(__VA_ARGS__);                    \
            switch (l.gs) {                                                        \
            case 1: return FN<1, 8, true>(__VA_ARGS__);                            \
            case 2: return FN<2, 8, true>(__VA_ARGS__);                            \
            case 4: return FN<4, 8, true>(__VA_ARGS__);                            \
            case 8: return FN<8, 8, true>(__VA_ARGS__);                            \
            case 16: return FN<16, 8, true>(__VA_ARGS__);                          \
            default: return FN<32, 8, true>(__VA_ARGS__);                          \
            }                                                                      \
        }                                                                          \
        if (l.cpl == 2) return FN<32, 2, false>(__VA_ARGS__);                      \
        if (l.cpl == 4) return FN<32, 4, false>(__VA_ARGS__);                      \
        if (l.cpl == 8) return FN<32, 8, false>(__VA_ARGS__);                      \
        switch (l.gs) {                                                            \
        case 1: return FN<1, 1, false>(__VA_ARGS__);                               \
        case 2: return FN<2, 1, false>(__VA_ARGS__);                               \
        case 4: return FN<4, 1, false>(__VA_ARGS__);                               \
        case 8: return FN<8, 1, false>(__VA_ARGS__);                               \
        case 16: return FN<16, 1, false>(__VA_ARGS__);                             \
        default: return FN<32, 1, false>(__VA_ARGS__);                             \
        }                                                                          \
    } while (0)

}  // namespace

size_t aux_workspace(int T, int E) { return aux_layout(nullptr, T, E, nullptr); }

rr_status launch_aux_fwd(int T, int E, int stride, const float *logits, const int32_t *first, float alpha,
                         float *loss, float *f, float *P, void *workspace, cudaStream_t st)
{
    AuxScratch a;
    aux_layout(workspace, T, E, &a);
    RR_AUX_DISPATCH(run_fwd, T, E, stride, logits, first, alpha, loss, f, P, a, st);
}

rr_status launch_aux_bwd(int T, int E, const float *logits, const float *f, float coef, int accumulate,
                         float *dlogits, cudaStream_t st)
{
    RR_AUX_DISPATCH(run_bwd, T, E, logits, f, coef, accumulate, dlogits, st);
}

}  // namespace rr
