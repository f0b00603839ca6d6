// Expert FFN forward: two persistent, warp-specialised grouped GEMMs on the 5th-generation
// tensor cores (tcgen05.mma, accumulators in TMEM, operands staged by TMA).
//
//   gate/up : H = X_rows [W1_e ; W3_e]^T,  Act = silu(H1) * H3         (rows gathered by TMA
//             row-gather straight from hidden[T,d]; SwiGLU in the epilogue)
//   down    : Y = Act W2_e^T,  out[token] += w_row * Y                  (Eq. 2 / Eq. 3 combine
//             fused into the epilogue as vector fp32 reductions)
//
// Each expert's live rows (occupied slots, then its IR list; Section 3, 4.1, 4.2) form a
// contiguous range of the compact row space, cut into 128-row tiles.  Padding slots are never
// computed.  One CTA per SM walks the (expert, n-tile, m-tile) list, m fastest, so that CTAs
// running together share the same weight tile through L2.
//
// Warp roles (192 threads): warp 0 TMA producer, warp 1 MMA issuer (one lane) and TMEM owner,
// warps 2-5 epilogue (one TMEM lane quarter each).  4-stage shared-memory ring
// (A 128x128 B + B 256x128 B per stage), two 256-column TMEM accumulators.
#include <cuda.h>
#include <cuda_bf16.h>

#include "rr_ffn.cuh"
#include "rr_tc.cuh"

namespace rr {
namespace {

using namespace tc;

constexpr int kStages = 4;
constexpr int kABytes = kTileM * 128;  // 128 rows x 128 B
constexpr int kBBytes = 256 * 128;     // 256 rows x 128 B
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kGemmThreads = 192;
constexpr int kAccCols = 256;
constexpr int kTmemCols = 512;

enum { kGateUp = 0, kDown = 1 };

struct GemmShared {
    uint64_t full[kStages], empty[kStages], tfull[2], tempty[2];
    uint32_t tmem_base;
    int abort_flag;
    int mt_off[kMaxE + 1];
    int row_off[kMaxE + 1];
};

constexpr size_t kGemmSmem = 1024 + (size_t)kStages * kStageBytes + sizeof(GemmShared);

struct GemmParams {
    int E;
    int KB;       // number of 128-byte k-blocks of the contraction
    int N;        // output columns (d_ff for gate/up, d for down)
    int n_tiles;  // tiles along N (128 wide for gate/up, 256 wide for down)
    const int *mt_off;
    const int *row_offset;
    const int *row_token;
    const float *row_weight;
    void *act, *h1, *h3;  // gate/up outputs [R, N]
    float *out;           // down output [T, N]
    int *status;
};

struct Work {
    int e, n, row0, rows;
};

__device__ __forceinline__ Work decode(const GemmShared *sh, int E, int n_tiles, int w)
{
    // largest e with mt_off[e] * n_tiles <= w
    int lo = 0, hi = E;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (sh->mt_off[mid] * n_tiles <= w) lo = mid; else hi = mid;
    }
    Work k;
    k.e = lo;
    const int local = w - sh->mt_off[lo] * n_tiles;
    const int mt = sh->mt_off[lo + 1] - sh->mt_off[lo];
    k.n = local / mt;
    const int m = local - k.n * mt;
    k.row0 = sh->row_off[lo] + m * kTileM;
    const int left = sh->row_off[lo + 1] - k.row0;
    k.rows = left < kTileM ? left : kTileM;
    return k;
}

__device__ __forceinline__ float silu(float z) { return z / (1.0f + __expf(-z)); }

template <bool kF32>
__device__ __forceinline__ void store32(void *base, size_t elem_index, const float *v)
{
    if constexpr (kF32) {
        float4 *p = reinterpret_cast<float4 *>(static_cast<float *>(base) + elem_index);
#pragma unroll
        for (int j = 0; j < 8; ++j) p[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
    } else {
        uint4 *p = reinterpret_cast<uint4 *>(static_cast<__nv_bfloat16 *>(base) + elem_index);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            __nv_bfloat162 a = __floats2bfloat162_rn(v[8 * j + 0], v[8 * j + 1]);
            __nv_bfloat162 b = __floats2bfloat162_rn(v[8 * j + 2], v[8 * j + 3]);
            __nv_bfloat162 c = __floats2bfloat162_rn(v[8 * j + 4], v[8 * j + 5]);
            __nv_bfloat162 d = __floats2bfloat162_rn(v[8 * j + 6], v[8 * j + 7]);
            uint4 u;
            u.x = *reinterpret_cast<uint32_t *>(&a);
            u.y = *reinterpret_cast<uint32_t *>(&b);
            u.z = *reinterpret_cast<uint32_t *>(&c);
            u.w = *reinterpret_cast<uint32_t *>(&d);
            p[j] = u;
        }
    }
}

template <int kMode, bool kF32>
__global__ void __launch_bounds__(kGemmThreads, 1)
k_ffn_gemm(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB0,
           const __grid_constant__ CUtensorMap mapB1, const GemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    GemmShared *sh = reinterpret_cast<GemmShared *>(tiles + (size_t)kStages * kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kBK = kF32 ? 32 : 64;  // elements per 128-byte k-block
    constexpr int kTileN = kMode == kGateUp ? 128 : 256;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&sh->tfull[b], 1); mbar_init(&sh->tempty[b], 128); }
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_map(&mapA);
        prefetch_map(&mapB0);
        if (kMode == kGateUp) prefetch_map(&mapB1);
    }
    for (int e = threadIdx.x; e <= p.E; e += kGemmThreads) {
        sh->mt_off[e] = p.mt_off[e];
        sh->row_off[e] = p.row_offset[e];
    }
    if (warp == 1) {
        tmem_alloc(&sh->tmem_base, kTmemCols);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;
    volatile int *abort_flag = &sh->abort_flag;
    const int total = sh->mt_off[p.E] * p.n_tiles;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        uint32_t it = 0;
        bool ok = true;
        for (int w = blockIdx.x; ok && w < total; w += gridDim.x) {
            const Work k = decode(sh, p.E, p.n_tiles, w);
            int tok[4] = {0, 0, 0, 0};
            if (kMode == kGateUp) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int r = lane * 4 + q;
                    tok[q] = p.row_token[k.row0 + (r < k.rows ? r : 0)];  // tail rows repeat a live row
                }
            }
            for (int kb = 0; kb < p.KB; ++kb, ++it) {
                const int s = it % kStages;
                const uint32_t ph = (it / kStages) & 1u;
                if (!warp_wait(&sh->empty[s], ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                uint8_t *a = tiles + (size_t)s * kStageBytes;
                uint8_t *b = a + kABytes;
                if (lane == 0) mbar_expect_tx(&sh->full[s], kStageBytes);
                __syncwarp();
                if (kMode == kGateUp) {
                    tma_gather4(a + lane * 512, &mapA, kb * kBK, tok[0], tok[1], tok[2], tok[3], &sh->full[s]);
                    if (lane == 0) {
                        tma_tile_2d(b, &mapB0, kb * kBK, k.e * p.N + k.n * kTileN, &sh->full[s]);
                        tma_tile_2d(b + kBBytes / 2, &mapB1, kb * kBK, k.e * p.N + k.n * kTileN, &sh->full[s]);
                    }
                } else if (lane == 0) {
                    tma_tile_2d(a, &mapA, kb * kBK, k.row0, &sh->full[s]);
                    tma_tile_2d(b, &mapB0, kb * kBK, k.e * p.N + k.n * kTileN, &sh->full[s]);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        constexpr uint32_t idesc = instr_desc(kF32 ? 2u : 1u, 0u, 0u, kTileM, 256);
        uint32_t it = 0, tile_it = 0;
        bool ok = true;
        for (int w = blockIdx.x; ok && w < total; w += gridDim.x, ++tile_it) {
            const uint32_t buf = tile_it & 1u;
            if (!warp_wait(&sh->tempty[buf], ((tile_it >> 1) & 1u) ^ 1u, abort_flag, p.status)) break;
            fence_after_sync();
            const uint32_t d_tmem = tmem_base + buf * kAccCols;
            for (int kb = 0; kb < p.KB; ++kb, ++it) {
                const int s = it % kStages;
                const uint32_t ph = (it / kStages) & 1u;
                if (!warp_wait(&sh->full[s], ph, abort_flag, p.status)) { ok = false; break; }
                fence_after_sync();
                if (lane == 0) {
                    const uint32_t a = smem_u32(tiles + (size_t)s * kStageBytes);
                    const uint64_t adesc = smem_desc(a, 16, 1024);
                    const uint64_t bdesc = smem_desc(a + kABytes, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)  // 32 bytes of K per instruction
                        mma_ss<kF32>(d_tmem, adesc + 2 * kk, bdesc + 2 * kk, idesc, (kb | kk) != 0);
                    mma_commit(&sh->empty[s]);
                }
                __syncwarp();
            }
            if (ok && lane == 0) mma_commit(&sh->tfull[buf]);
            __syncwarp();
        }
    } else {
        // ---------------- epilogue ----------------
        const int q = warp & 3;  // TMEM lane quarter this warp may read
        const int r_in_tile = q * 32 + lane;
        uint32_t tile_it = 0;
        for (int w = blockIdx.x; w < total; w += gridDim.x, ++tile_it) {
            const Work k = decode(sh, p.E, p.n_tiles, w);
            const uint32_t buf = tile_it & 1u;
            if (!warp_wait(&sh->tfull[buf], (tile_it >> 1) & 1u, abort_flag, p.status)) break;
            fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kAccCols;
            const bool live = r_in_tile < k.rows;
            const size_t row = (size_t)k.row0 + r_in_tile;
            if (kMode == kGateUp) {
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    float g[32], u[32];
                    tmem_ld32(taddr + c * 32, g);
                    tmem_ld32(taddr + 128 + c * 32, u);
                    const int col0 = k.n * kTileN + c * 32;
                    if (live && col0 < p.N) {
                        const size_t at = row * p.N + col0;
                        if (p.h1) { store32<kF32>(p.h1, at, g); store32<kF32>(p.h3, at, u); }
#pragma unroll
                        for (int j = 0; j < 32; ++j) g[j] = silu(g[j]) * u[j];
                        store32<kF32>(p.act, at, g);
                    }
                }
            } else {
                const int tok = live ? p.row_token[row] : 0;
                const float wgt = live ? p.row_weight[row] : 0.0f;
#pragma unroll 1
                for (int c = 0; c < 8; ++c) {
                    float y[32];
                    tmem_ld32(taddr + c * 32, y);
                    const int col0 = k.n * kTileN + c * 32;
                    if (live && col0 < p.N) {
                        float *dst = p.out + (size_t)tok * p.N + col0;
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            red_add_v4(dst + 4 * j, wgt * y[4 * j], wgt * y[4 * j + 1], wgt * y[4 * j + 2], wgt * y[4 * j + 3]);
                    }
                }
            }
            fence_before_sync();
            mbar_arrive(&sh->tempty[buf]);
        }
    }

    __syncthreads();
    if (sh->abort_flag) __nanosleep(2000000);  // let copies that are still in flight land
    if (warp == 1) {
        fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// Number of 128-row tiles per expert, as an exclusive prefix.
__global__ void k_ffn_tiles(int E, const int *__restrict__ row_offset, int *__restrict__ mt_off)
{
    __shared__ int mt[kMaxE];
    for (int e = threadIdx.x; e < E; e += blockDim.x)
        mt[e] = (row_offset[e + 1] - row_offset[e] + kTileM - 1) / kTileM;
    __syncthreads();
    if (threadIdx.x == 0) {
        int acc = 0;
        for (int e = 0; e < E; ++e) { mt_off[e] = acc; acc += mt[e]; }
        mt_off[E] = acc;
    }
}

// ---- host side ------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Row-major [rows, cols] matrix, box = 128 bytes of columns x box_rows rows, 128-byte swizzle.
bool make_map(CUtensorMap *m, const void *base, size_t rows, size_t cols, bool f32, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const size_t es = f32 ? 4 : 2;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)(rows ? rows : 1)};
    cuuint64_t strides[1] = {(cuuint64_t)(cols * es)};
    cuuint32_t box[2] = {(cuuint32_t)(128 / es), (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
              const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return n;
}

template <int kMode, bool kF32>
cudaError_t launch_gemm(const CUtensorMap &a, const CUtensorMap &b0, const CUtensorMap &b1, const GemmParams &p,
                        int grid, cudaStream_t st)
{
    cudaError_t err = cudaFuncSetAttribute(k_ffn_gemm<kMode, kF32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)kGemmSmem);
    if (err != cudaSuccess) return err;
    k_ffn_gemm<kMode, kF32><<<grid, kGemmThreads, kGemmSmem, st>>>(a, b0, b1, p);
    return cudaGetLastError();
}

}  // namespace

size_t ffn_saved_bytes(const rr_moe_shape &s)
{
    return 3 * align_up(rows_max(s) * s.d_ff * elem_bytes(s), 256);
}

size_t ffn_fwd_layout(void *ws, void *saved, const rr_moe_shape &s, FfnScratch *f)
{
    Carver c(ws);
    f->hdr = c.take<Header>(1);
    f->mt_off = c.take<int>(s.E + 1);
    const size_t act_bytes = align_up(rows_max(s) * s.d_ff * elem_bytes(s), 256);
    if (saved) {
        f->act = saved;
        f->h1 = static_cast<char *>(saved) + act_bytes;
        f->h3 = static_cast<char *>(saved) + 2 * act_bytes;
    } else {
        f->act = c.take<char>(act_bytes);
        f->h1 = nullptr;
        f->h3 = nullptr;
    }
    return align_up(c.off, 256);
}

rr_status launch_ffn_fwd(const rr_moe_shape &s, const void *hidden, const void *W1, const void *W3, const void *W2,
                         const rr_route_tables &t, float *out, const FfnScratch &f, cudaStream_t st)
{
    const bool f32 = s.dtype == RR_F32;
    const int bk = f32 ? 32 : 64;
    const int grid = sm_count();
    if (grid <= 0) return RR_ERR_CUDA;
    const size_t R = rows_max(s);

    CUtensorMap mX, mW1, mW3, mAct, mW2;
    if (!make_map(&mX, hidden, s.T, s.d, f32, 1) ||  // one-row box: rows are gathered four at a time
        !make_map(&mW1, W1, (size_t)s.E * s.d_ff, s.d, f32, 128) ||
        !make_map(&mW3, W3, (size_t)s.E * s.d_ff, s.d, f32, 128) ||
        !make_map(&mAct, f.act, R, s.d_ff, f32, kTileM) ||
        !make_map(&mW2, W2, (size_t)s.E * s.d, s.d_ff, f32, 256))
        return RR_ERR_CUDA;

    if (cudaMemsetAsync(out, 0, (size_t)s.T * s.d * sizeof(float), st) != cudaSuccess) return RR_ERR_CUDA;
    k_ffn_tiles<<<1, 256, 0, st>>>(s.E, t.row_offset, f.mt_off);
    auto mark = [&](int i) {
        if (s.trace && s.trace[i]) cudaEventRecord(static_cast<cudaEvent_t>(s.trace[i]), st);
    };
    mark(0);

    GemmParams p{};
    p.E = s.E;
    p.mt_off = f.mt_off;
    p.row_offset = t.row_offset;
    p.row_token = t.row_token;
    p.row_weight = t.row_weight;
    p.status = &f.hdr->status;

    // gate / up + SwiGLU
    p.KB = s.d / bk;
    p.N = s.d_ff;
    p.n_tiles = (s.d_ff + 127) / 128;
    p.act = f.act; p.h1 = f.h1; p.h3 = f.h3; p.out = nullptr;
    cudaError_t err = f32 ? launch_gemm<kGateUp, true>(mX, mW1, mW3, p, grid, st)
                          : launch_gemm<kGateUp, false>(mX, mW1, mW3, p, grid, st);
    if (err != cudaSuccess) return RR_ERR_CUDA;
    mark(1);

    // down + combine
    p.KB = s.d_ff / bk;
    p.N = s.d;
    p.n_tiles = (s.d + 255) / 256;
    p.out = out;
    err = f32 ? launch_gemm<kDown, true>(mAct, mW2, mW2, p, grid, st)
              : launch_gemm<kDown, false>(mAct, mW2, mW2, p, grid, st);
    mark(2);
    return err == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

size_t ffn_bwd_layout(void *, const rr_moe_shape &, BwdScratch *) { return 256; }

rr_status launch_ffn_bwd(const rr_moe_shape &, const void *, const void *, const void *, const void *, const void *,
                         const float *, const rr_route_tables &, const void *, float *, float *, float *, float *,
                         float *, const BwdScratch &, cudaStream_t)
{
    return RR_ERR_UNSUPPORTED;
}

}  // namespace rr
