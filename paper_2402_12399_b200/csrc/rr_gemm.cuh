// One persistent, warp-specialised tcgen05 GEMM kernel template serving every dense
// contraction of the layer.  CTA pairs: one cta_group::2 MMA of 256 x 256 x 16 drives the tensor
// cores of two SMs; each CTA of the pair owns 128 rows of the 256-row tile (its TMEM lanes) and
// stages its own A rows plus half of the B operand, so a k-block of 128 bytes (64 bf16 / 32 tf32)
// costs each CTA 16 KB + 16 KB of shared memory.  A ring of 4 or 6 such stages is filled by TMA;
// two TMEM accumulators let the epilogue of one tile overlap the main loop of the next.
//
//   mode      A operand (K-major unless noted)  B operand                        epilogue
//   kGateUp   token rows in expert order        [W1_e tile ; W3_e tile], K-major  Act = silu(g)*u
//   kGateUpTrain  as kGateUp, and keeps g, u in fp32 for the backward pass (TMA stores from a
//             swizzled staging buffer per epilogue warp)
//   kDown     Act tile                          W2_e tile, K-major                out[token] += w_row * y
//   kDAct     dout rows in expert order         W2_e, MN-major (no transpose      dH1, dH3, w*act, delta_row
//                                               copy of the weights is made)
//   kDX       dH1 tile then dH3 tile            W1_e then W3_e, MN-major          dhidden[token] += dx
//   kWgrad    P[rows, M] MN-major               Q[rows, N] MN-major               dW_e[M, N] = P^T Q
//   kGate     hidden (token order)              Wg [E, d], K-major (rows beyond   logits[token, 0..E)
//                                               E read as zeros)
//   kDenseAdd as kDown with one "expert" whose rows are the rows of `out` in order: out[row0 + r, :] += tile,
//             32 x 32 pieces through a staging tile per warp and TMA reduce-add (no per-row atomics)
//   kGateSel  as kGate; the epilogue also selects every token's k+1 best experts and the best of its
//             group straight from the accumulators (Eq. 1; Section 4.1) and sums the softmax values per
//             expert over each 32 tokens (for the load-balance loss)
//
// Rows live in a padded internal row space: expert e owns rows [128*mt_off[e], 128*mt_off[e+1]),
// its live rows first (occupied slots, then its IR list: Sections 3, 4.1, 4.2), zero rows after.
// Tiles therefore never straddle experts and the weight-gradient contraction over rows needs
// no masking.  Token rows are brought into that order by a copy kernel before the first GEMM
// (gathering them inside the GEMM ties it to single-CTA tiles, whose operand traffic saturates
// the shared-memory port: every k-block is written once by the loads and read once by the MMA).
//
// Warps: 0-2 = TMA producers (lane 0 of each; k-blocks dealt round-robin, because one thread
// cannot issue barrier waits and tile loads fast enough to keep up with the tensor cores),
// 3 = MMA issuer (lane 0, leader CTA only) and TMEM owner, 4-11 = epilogue (two warps per TMEM
// lane quarter, alternating column chunks).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "rr_ffn.cuh"
#include "rr_route_dev.cuh"
#include "rr_tc.cuh"

namespace rr {
namespace gemm {

using namespace tc;

constexpr int kABytes = kTileM * 128;   // A rows of this CTA, one k-block
constexpr int kBBytes = 128 * 128;      // this CTA's half of the B operand, one k-block
constexpr int kStageBytes = kABytes + kBBytes;

constexpr int kPanelBytes = 64 * 128;  // MN-major panel: 64 k-rows x 128 B
constexpr int kProducers = 3;                  // warps 0..2 (twelve warps in all: three per scheduler,
                                               // which leaves each thread up to 168 registers)
constexpr int kMmaWarp = kProducers;           // warp 3
constexpr int kFirstEpiWarp = kMmaWarp + 1;    // warps 4 and up
constexpr int kMaxEpiWarps = 12;
constexpr int kAccCols = 256;
constexpr int kTmemCols = 512;

enum Mode { kGateUp = 0, kDown = 1, kDAct = 2, kDX = 3, kWgrad = 4, kGateUpTrain = 5, kGate = 6, kGateSel = 7, kDenseAdd = 8,
            kDActShortK = 9 };  // kDAct in another launch shape (below); the kernel body is the same

// Epilogue warps: two per TMEM lane quarter (twelve warps in all, three per scheduler, up to 168
// registers a thread).  The kDAct epilogue is a long dependent chain per step (tile in, SwiGLU
// backward, three tiles out) that only more warps overlap: with a short contraction (d_model <= 1024)
// it bounds the kernel, and kDActShortK runs three warps per quarter on a ring of four stages
// (c5: 1.04 -> 0.91 ms); with a longer one the ring depth matters more (c4: 0.85 -> 0.90 ms), and
// kDAct keeps two warps per quarter and five stages.
template <int kMode>
__host__ __device__ constexpr int epi_warps_of() { return kMode == kDActShortK ? 12 : 8; }
template <int kMode>
__host__ __device__ constexpr int threads_of() { return 32 * (kFirstEpiWarp + epi_warps_of<kMode>()); }

struct Shared {
    uint64_t full[12], empty[12], tfull[2], tempty[2];
    uint64_t ebar[kMaxEpiWarps];  // kDAct: one per epilogue warp, counts the bytes of its h1 / h3 tiles
    uint32_t tmem_base;
    int abort_flag;
    int mt_off[kMaxE + 1];
    // number of experts before e with an odd tile count: the exclusive prefix of the number of
    // 256-row pair tiles per expert is (mt_off[e] + odd_before[e]) / 2
    // kWgrad instead: the experts by falling tile count (ties by index)
    union {
        uint16_t odd_before[kMaxE + 2];
        uint16_t order[kMaxE + 2];
    };
    __device__ __forceinline__ int pt_off(int e) const { return (mt_off[e] + odd_before[e]) >> 1; }
};

// kDAct epilogue, per warp: tiles of saved h1 and h3 (32 rows x 16 fp32, brought in by TMA) and
// staging tiles of dH1, dH3, w*act (32 rows x 16 bf16, taken out by TMA)
constexpr int kDActWarpBytes = 2 * 2048 + 3 * 1024;

// Ring depth: six stages; five for kDAct, whose epilogue needs 56 KB of shared memory for itself
// (four and 84 KB for kDActShortK); seven for kDown and kDX, whose epilogues need none.
// The depth matters: measured cycles per k-block are about 560 with six stages, 800 with four and
// 1200 with three (the loads need that much data in flight to cover their latency).
template <int kMode>
__host__ __device__ constexpr int stages_of()
{
    return kMode == kDAct ? 5 : kMode == kDActShortK ? 4 : (kMode == kDown || kMode == kDX) ? 7 : 6;
}
// Epilogue tiles in shared memory.  kGateUpTrain, kWgrad: per epilogue warp one 32 x 128-byte staging
// tile (g, then u; a piece of dW); kDAct: see kDActWarpBytes.
template <int kMode>
__host__ __device__ constexpr int epi_bytes_of()
{
    return (kMode == 0 || kMode == 5 || kMode == 4 || kMode == 8) ? epi_warps_of<kMode>() * 4096
           : (kMode == kDAct || kMode == kDActShortK)                   ? epi_warps_of<kMode>() * kDActWarpBytes
                                                                        : 0;
}
template <int kMode>
constexpr size_t smem_bytes_of()
{
    static_assert(sizeof(Shared) <= 2048, "six stages and 32 KB of epilogue tiles leave 2048 bytes for the barriers and expert tables");
    return 1024 + (size_t)stages_of<kMode>() * kStageBytes + sizeof(Shared) + epi_bytes_of<kMode>();
}

struct Params {
    int E;
    int KB;        // k-blocks per tile (row-tiled modes); kDX: both segments together
    int N;         // output columns
    int n_tiles;   // tiles along N
    int M;         // kWgrad: output rows per expert
    int m_tiles;   // kWgrad: tiles along M
    int w_rows;    // MN-major weight operand: rows of the weight matrix per expert
    const int *mt_off;
    const int *row_offset;
    const int *row_token;
    const float *row_weight;
    float *out;                   // kDown / kDX output, [T, N]; kGate: logits [T, N]
    int gate_T;                   // kGate: number of tokens (its tile tables are computed, not read)
    int gate_n;                   // kGate: N of the MMA (E rounded up to 16); each CTA stages gate_n/2 rows of Wg
    int gate_stages;              // kGate: ring depth (the small B tile leaves room for more stages)
    // kGateSel: what the epilogue's selection writes (Eq. 1, Section 4.1), per token
    int sel_k, sel_G, sel_T;      //   top-k, groups, tokens
    int *sel_expert;              //   [T, k+1] experts by (score desc, index asc), -1 beyond E
    float *sel_val;               //   [T, k+1] their scores
    int *sel_h;                   //   [T] best expert of the token's own group
    float *sel_ah;                //   [T] its score
    float *sel_psum;              //   [ceil(T/32), E] softmax values summed over each 32 tokens, or null
    float *delta;                 // kDAct output, [R] by public row
    float *dw;                    // kWgrad output, [E, M, N]
    int *status;
    unsigned long long test_tfull_limit_ns;  // testing aid: limit of the epilogue's accumulator wait (0: the usual 2 s)
};

struct Work {
    int e, n, m;     // expert, tile along N, tile along rows (row-tiled) or along M (kWgrad)
    int prow0;       // first padded row of the tile (row-tiled) / of the expert (kWgrad)
    int row0, rows;  // first public row of the tile and number of live rows in it
    int kblocks;     // k-blocks of this work item
    bool dead;       // second half of a pair whose expert has an odd number of tiles
};

template <int kMode>
__device__ __forceinline__ int total_work(const Shared *sh, const Params &p)
{
    if (kMode == kWgrad) return p.E * p.m_tiles * p.n_tiles;
    return sh->pt_off(p.E) * p.n_tiles;
}

// Work item `w` of the CTA pair, seen from the CTA of rank `rank` (0 = leader): the pair owns 256
// rows (two consecutive 128-row tiles of one expert, or 256 rows of dW_e), this CTA the rows
// [128*rank, 128*rank+128) of them.
template <int kMode, bool kRows = false>
__device__ __forceinline__ Work decode(const Shared *sh, const Params &p, int w, int rank)
{
    Work k;
    k.dead = false;
    if (kMode == kWgrad) {
        // An item costs as many k-blocks as its expert has rows, and the pairs take items w, w + npairs, ...:
        // the items are laid out by falling cost (experts by falling tile count) and every second band of
        // npairs items is walked backwards, so that each pair gets one item of every band and the bands'
        // dearer and cheaper ends alternate (c5: the busiest pair 2 % above the mean instead of 20 %).
        const int per = p.m_tiles * p.n_tiles;
        const int npairs = (int)(gridDim.x >> 1);
        const int band = w / npairs;
        if ((band & 1) && (band + 1) * npairs <= p.E * per) w = band * npairs + (npairs - 1 - (w - band * npairs));
        const int es = w / per;
        k.e = sh->order[es];
        const int rem = w - es * per;
        const int pm = rem / p.n_tiles;
        k.n = rem - pm * p.n_tiles;
        k.m = 2 * pm + rank;
        k.prow0 = sh->mt_off[k.e] * kTileM;
        k.row0 = 0;
        k.rows = 0;
        k.kblocks = (sh->mt_off[k.e + 1] - sh->mt_off[k.e]) * 2;  // 64 rows per k-block
        return k;
    }
    int lo = 0, hi = p.E;  // largest e with pt_off[e] * n_tiles <= w
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (sh->pt_off(mid) * p.n_tiles <= w) lo = mid; else hi = mid;
    }
    k.e = lo;
    const int pt0 = sh->pt_off(lo);
    const int local = w - pt0 * p.n_tiles;
    const int pt = sh->pt_off(lo + 1) - pt0;
    // m fastest: pairs running together share one weight tile.  (For kDown / kDX, whose A rows are as long
    // as a weight tile, blocks of eight n-tiles times several row tiles were measured instead: more DRAM
    // traffic, not less -- 3.9 GB against 3.0 GB on half of the 7B-width layer -- and 5 % slower.)
    k.n = local / pt;
    const int pm = local - k.n * pt;
    const int mt = sh->mt_off[lo + 1] - sh->mt_off[lo];
    k.m = 2 * pm + rank;
    if (k.m >= mt) {  // odd number of tiles: the second half of the last pair has no rows;
        k.dead = true;  // it reads its partner's rows (any valid memory) and stores nothing
        k.m = 2 * pm;
    }
    k.prow0 = (sh->mt_off[lo] + k.m) * kTileM;
    k.row0 = 0;
    k.rows = 0;
    if (kRows) {  // public row range of the tile (epilogue only; two cached global loads)
        // (kGate / kGateSel: the one "expert" owns the tokens 0 .. gate_T-1 in order, no tables in memory)
        constexpr bool kTokens = kMode == kGate || kMode == kGateSel;
        k.row0 = (kTokens ? 0 : __ldg(p.row_offset + lo)) + k.m * kTileM;
        const int left = (kTokens ? p.gate_T : __ldg(p.row_offset + lo + 1)) - k.row0;
        k.rows = k.dead ? 0 : (left < kTileM ? left : kTileM);
    }
    k.kblocks = p.KB;
    return k;
}

__device__ __forceinline__ float sigmoidf_fast(float z) { return __fdividef(1.0f, 1.0f + __expf(-z)); }
__device__ __forceinline__ float exp2f_fast(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_fast(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 8 fp32 values -> 8 bf16 in one 16-byte word
__device__ __forceinline__ uint4 pack8_bf16(const float *v)
{
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(v[2], v[3]);
    __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]);
    __nv_bfloat162 d = __floats2bfloat162_rn(v[6], v[7]);
    uint4 u;
    u.x = *reinterpret_cast<uint32_t *>(&a);
    u.y = *reinterpret_cast<uint32_t *>(&b);
    u.z = *reinterpret_cast<uint32_t *>(&c);
    u.w = *reinterpret_cast<uint32_t *>(&d);
    return u;
}

// kGateSel epilogue, one thread per token: the k+1 best experts and the best expert of the token's group
// from the fp32 scores in its TMEM lane, eight columns per step (a short loop body that is reused: the
// epilogue warps run alone on their schedulers, and long straight-line code costs them more in
// instruction fetch than the arithmetic does).  A score that is not finite latches RR_ERR_NONFINITE;
// the indices written still name experts.
template <int KK>
__device__ __forceinline__ void gate_select(const Params &p, uint32_t taddr, int tok, bool live)
{
    const int E = p.N, K1 = p.sel_k + 1;
    float bv[KK], gv = -CUDART_INF_F, chk = 0.0f;
    int bj[KK], gj = INT_MAX;
#pragma unroll
    for (int r = 0; r < KK; ++r) { bv[r] = empty_place(); bj[r] = INT_MAX; }
    const int tpg = p.sel_T / p.sel_G > 0 ? p.sel_T / p.sel_G : 1, epg = E / p.sel_G;
    const int lo = live ? (tok / tpg) * epg : 0, hi = lo + epg;
#pragma unroll 1
    for (int c = 0; c * 8 < E; ++c) {
        float y[8];
        tmem_ld8(taddr + c * 8, y);  // (every lane of the warp, live or not)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int col = 8 * c + j;
            if (col < E) {
                chk = fmaf(y[j], 0.0f, chk);
                insert_strict<KK>(y[j], col, bv, bj);
                if (col >= lo && col < hi && y[j] > gv) { gv = y[j]; gj = col; }
            }
        }
    }
    if (!live) return;
    if (chk != 0.0f) {
        latch_status(p.status, RR_ERR_NONFINITE);
#pragma unroll
        for (int r = 0; r < KK; ++r)
            if (bj[r] == INT_MAX && r < E) { bj[r] = r; bv[r] = 0.0f; }
    }
    if (gj == INT_MAX) { gj = lo; gv = 0.0f; }
#pragma unroll
    for (int r = 0; r < KK; ++r) {
        if (r < K1) {
            p.sel_expert[(size_t)tok * K1 + r] = bj[r] < E ? bj[r] : -1;
            p.sel_val[(size_t)tok * K1 + r] = bj[r] < E ? bv[r] : 0.0f;
        }
    }
    p.sel_h[tok] = gj;
    p.sel_ah[tok] = gv;
}

// kGateSel epilogue: softmax of every token's scores, summed per expert over the warp's 32 tokens (a
// fixed tree of exchanges, so the sums repeat bit for bit); tokens beyond T count as zero.  The
// exponentials are the hardware's (ex2.approx of the scaled argument, relative error about 1e-6: the sums
// are compared at 6e-5).
__device__ __forceinline__ void gate_softmax_sums(const Params &p, uint32_t taddr, int tok, bool live, int lane)
{
    const int E = p.N;
    float m = -CUDART_INF_F;
#pragma unroll 1
    for (int c = 0; c * 8 < E; ++c) {
        float y[8];
        tmem_ld8(taddr + c * 8, y);
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (8 * c + j < E) m = fmaxf(m, y[j]);
    }
    float Z = 0.0f;
#pragma unroll 1
    for (int c = 0; c * 8 < E; ++c) {
        float y[8];
        tmem_ld8(taddr + c * 8, y);
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (8 * c + j < E) Z += __expf(y[j] - m);
    }
    const float inv = live ? 1.0f / Z : 0.0f;
    const int unit = (tok - lane) >> 5;  // the warp's tokens are 32 consecutive ones starting at a multiple of 32
#pragma unroll 1
    for (int c = 0; c * 32 < E; ++c) {
        float v[32];
        tmem_ld32(taddr + c * 32, v);
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = 32 * c + j < E ? __expf(v[j] - m) * inv : 0.0f;
        warp_transpose_add(v, lane);  // lane j ends with column j summed over all 32 tokens
        if (32 * c + lane < E && tok - lane < p.sel_T) p.sel_psum[(size_t)unit * E + 32 * c + lane] = v[0];
    }
}

template <int kModeT, bool kF32>
__global__ void __launch_bounds__(threads_of<kModeT>(), 1)
k_gemm(const __grid_constant__ CUtensorMap mapA0, const __grid_constant__ CUtensorMap mapA1,
       const __grid_constant__ CUtensorMap mapB0, const __grid_constant__ CUtensorMap mapB1,
       const __grid_constant__ CUtensorMap mapS0, const __grid_constant__ CUtensorMap mapS1,
       const __grid_constant__ CUtensorMap mapS2, const Params p)
{
    constexpr int kMode = kModeT == kDActShortK ? (int)kDAct : kModeT;  // kModeT only sets the launch shape
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // kGate stages only gate_n/2 rows of Wg per CTA and k-block, so its stages are smaller and its
    // ring deeper (set by the host); every other mode has compile-time values
    constexpr bool kIsGate = kMode == kGate || kMode == kGateSel;
    const int kNS = kIsGate ? p.gate_stages : stages_of<kModeT>();
    const int stage_bytes = kIsGate ? kABytes + p.gate_n * 64 : kStageBytes;
    uint8_t *store_stage = tiles + (size_t)kNS * stage_bytes;  // epilogue tiles of kGateUpTrain, kWgrad, kDAct; 1024-byte aligned
    Shared *sh = reinterpret_cast<Shared *>(store_stage + epi_bytes_of<kModeT>());
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kEpiWarps = epi_warps_of<kModeT>();
    constexpr int kEpiGroups = kEpiWarps / 4;  // warps per TMEM lane quarter
    constexpr int kBK = kF32 ? 32 : 64;  // elements per 128-byte k-block (K-major operands)
    constexpr bool kGU = kMode == kGateUp || kMode == kGateUpTrain;
    constexpr int kTileN = kGU ? 128 : 256;
    constexpr bool kAmn = kMode == kWgrad;
    constexpr bool kBmn = kMode == kDAct || kMode == kDX || kMode == kWgrad;

    // rank 0 is the leader of the CTA pair: its full / tempty barriers count the loads and the
    // accumulator releases of both CTAs, and its MMA thread issues for both tensor cores
    const int rank = (int)cluster_ctarank();
    const int pair = (int)(blockIdx.x >> 1);
    const int npairs = (int)(gridDim.x >> 1);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kNS; ++s) {
            mbar_init(&sh->full[s], 1);
            mbar_init(&sh->empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(&sh->tfull[b], 1); mbar_init(&sh->tempty[b], 2 * 32 * kEpiWarps); }
        for (int i = 0; i < kEpiWarps; ++i) mbar_init(&sh->ebar[i], 1);
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_map(&mapA0);
        prefetch_map(&mapB0);
        if (kMode == kDX || kMode == kDAct) prefetch_map(&mapA1);
        if (kGU || kMode == kDX) prefetch_map(&mapB1);
        if (kMode == kGateUpTrain) { prefetch_map(&mapS0); prefetch_map(&mapS1); }
        if (kGU) prefetch_map(&mapS2);
        if (kMode == kWgrad || kMode == kDenseAdd) prefetch_map(&mapS0);
        if (kMode == kDAct) prefetch_map(&mapS0);
    }
    for (int e = threadIdx.x; e <= p.E; e += threads_of<kModeT>()) {
        sh->mt_off[e] = kIsGate ? (e == 0 ? 0 : (p.gate_T + kTileM - 1) / kTileM) : p.mt_off[e];
    }
    __syncthreads();
    if (kMode == kWgrad) {
        for (int e = threadIdx.x; e < p.E; e += threads_of<kModeT>()) {
            const int mine = sh->mt_off[e + 1] - sh->mt_off[e];
            int before = 0;  // experts that come first: more tiles, or as many and a smaller index
            for (int j = 0; j < p.E; ++j) {
                const int other = sh->mt_off[j + 1] - sh->mt_off[j];
                before += (other > mine || (other == mine && j < e)) ? 1 : 0;
            }
            sh->order[before] = (uint16_t)e;
        }
    } else if (threadIdx.x == 0) {
        int acc = 0;
        for (int e = 0; e < p.E; ++e) { sh->odd_before[e] = (uint16_t)acc; acc += (sh->mt_off[e + 1] - sh->mt_off[e]) & 1; }
        sh->odd_before[p.E] = (uint16_t)acc;
    }
    if (warp == kMmaWarp) {
        tmem_alloc_pair(&sh->tmem_base, kTmemCols);
        tmem_relinquish_pair();
    }
    fence_before_sync();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers are initialised before anything signals them
    fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;
    volatile int *abort_flag = &sh->abort_flag;
    const int total = total_work<kMode>(sh, p);
    // the leader's barriers as shared::cluster addresses
    const uint32_t lead_full = map_to_cta(&sh->full[0], 0);
    const uint32_t lead_tempty = map_to_cta(&sh->tempty[0], 0);

    if (warp < kProducers) {
        // ---------------- TMA producers ----------------
        // Producer j takes the k-blocks j, j+3, ... of this CTA's stream (counted across tiles).
        // Both CTAs load their own A rows and their half of B; all bytes are counted on the
        // leader's stage barrier, which the peer names by its shared::cluster address.
        if (lane == 0) {
            uint32_t s = warp % kNS, ph = 0;  // stage and phase parity of this producer's next k-block
            uint32_t next = warp;             // its index in the stream
            uint32_t it0 = 0;                 // stream index of the first k-block of the tile
            bool ok = true;
            for (int w = pair; ok && w < total; w += npairs) {
                const Work k = decode<kMode>(sh, p, w, rank);
                const int bn = k.n * kTileN + 128 * rank;  // this CTA's half of the B rows / columns
                int kb = (int)(next - it0);
                for (; kb < k.kblocks; kb += kProducers) {
                    if (!mbar_wait(&sh->empty[s], ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    uint8_t *a = tiles + (size_t)s * stage_bytes;
                    uint8_t *b = a + kABytes;
                    const uint32_t bar = lead_full + 8u * s;
                    if (rank == 0) mbar_expect_tx(&sh->full[s], 2u * stage_bytes);  // bytes of both CTAs
                    if (kGU) {
                        tma_tile_2d_pair(a, &mapA0, kb * kBK, k.prow0, bar);
                        // accumulator columns 0..127 = gate (W1, staged by the leader), 128..255 = up (W3)
                        tma_tile_2d_pair(b, rank == 0 ? &mapB0 : &mapB1, kb * kBK, k.e * p.N + k.n * kTileN, bar);
                    } else if (kIsGate) {  // one "expert", its rows are the tokens; B = this CTA's rows of Wg
                        tma_tile_2d_pair(a, &mapA0, kb * kBK, k.prow0, bar);
                        tma_tile_2d_pair(b, &mapB0, kb * kBK, (p.gate_n >> 1) * rank, bar);
                    } else if (kMode == kDown || kMode == kDenseAdd) {
                        tma_tile_2d_pair(a, &mapA0, kb * kBK, k.prow0, bar);
                        tma_tile_2d_pair(b, &mapB0, kb * kBK, k.e * p.N + bn, bar);
                    } else if (kMode == kDAct) {
                        tma_tile_2d_pair(a, &mapA0, kb * 64, k.prow0, bar);
#pragma unroll
                        for (int q = 0; q < 2; ++q)
                            tma_tile_2d_pair(b + q * kPanelBytes, &mapB0, bn + 64 * q, k.e * p.w_rows + kb * 64, bar);
                    } else if (kMode == kDX) {
                        const int half = p.KB >> 1;
                        const bool second = kb >= half;
                        const int kl = second ? kb - half : kb;
                        tma_tile_2d_pair(a, second ? &mapA1 : &mapA0, kl * 64, k.prow0, bar);
#pragma unroll
                        for (int q = 0; q < 2; ++q)
                            tma_tile_2d_pair(b + q * kPanelBytes, second ? &mapB1 : &mapB0, bn + 64 * q,
                                             k.e * p.w_rows + kl * 64, bar);
                    } else {  // kWgrad
#pragma unroll
                        for (int q = 0; q < 2; ++q)
                            tma_tile_2d_pair(a + q * kPanelBytes, &mapA0, k.m * kTileM + 64 * q, k.prow0 + kb * 64, bar);
#pragma unroll
                        for (int q = 0; q < 2; ++q)
                            tma_tile_2d_pair(b + q * kPanelBytes, &mapB0, bn + 64 * q, k.prow0 + kb * 64, bar);
                    }
                    s += kProducers;
                    if (s >= (uint32_t)kNS) { s -= kNS; ph ^= 1u; }
                }
                next = it0 + kb;
                it0 += k.kblocks;
            }
        }
    } else if (warp == kMmaWarp) {
        // ---------------- MMA issuer: one thread of the leader drives both tensor cores ----------------
        if (rank == 0 && lane == 0) {
            const uint32_t idesc = instr_desc(kF32 ? 2u : 1u, kAmn ? 1u : 0u, kBmn ? 1u : 0u, 2 * kTileM,
                                              kIsGate ? (uint32_t)p.gate_n : 256u);
            // descriptors carry this CTA's addresses, the peer uses the same offsets; one
            // instruction consumes 32 bytes of K: 32 B along a K-major row, or 16 k-rows
            // (2048 B) of an MN-major panel
            const uint32_t a0 = smem_u32(tiles);
            const uint64_t adesc0 = kAmn ? smem_desc(a0, kPanelBytes, 1024) : smem_desc(a0, 16, 1024);
            const uint64_t bdesc0 = kBmn ? smem_desc(a0 + kABytes, kPanelBytes, 1024) : smem_desc(a0 + kABytes, 16, 1024);
            constexpr uint32_t a_step = kAmn ? 128u : 2u, b_step = kBmn ? 128u : 2u;
            uint32_t s = 0, ph = 0, tile_it = 0;
            bool ok = true;
            for (int w = pair; ok && w < total; w += npairs) {
                const Work k = decode<kMode>(sh, p, w, rank);
                if (k.kblocks == 0) continue;  // kWgrad of an expert without rows: the epilogue writes zeros
                const uint32_t buf = tile_it & 1u;
                if (!mbar_wait(&sh->tempty[buf], ((tile_it >> 1) & 1u) ^ 1u, abort_flag, p.status)) break;
                fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * kAccCols;
                for (int kb = 0; kb < k.kblocks; ++kb) {
                    if (!mbar_wait(&sh->full[s], ph, abort_flag, p.status)) { ok = false; break; }
                    const uint32_t off = s * (uint32_t)(stage_bytes >> 4);  // descriptor addresses count 16-byte units
                    const uint64_t adesc = adesc0 + off, bdesc = bdesc0 + off;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_ss_pair<kF32>(d_tmem, adesc + a_step * kk, bdesc + b_step * kk, idesc, (kb | kk) != 0);
                    mma_commit_pair(&sh->empty[s]);  // frees the stage in both CTAs
                    if (++s == (uint32_t)kNS) { s = 0; ph ^= 1u; }
                }
                if (ok) mma_commit_pair(&sh->tfull[buf]);  // accumulators ready in both CTAs
                ++tile_it;
            }
        }
    } else {
        // ---------------- epilogue (warps 4 .. 4 + kEpiWarps - 1) ----------------
        // kEpiGroups warps per TMEM lane quarter; the warp of group eg takes the column chunks eg, eg + kEpiGroups, ...
        const int eg = (warp - kFirstEpiWarp) >> 2;
        const int q = warp & 3;  // TMEM lane quarter this warp may read
        const int wi = eg * 4 + q;
        const int r_in_tile = q * 32 + lane;
        uint32_t tile_it = 0, store_it = 0, ld_it = 0;
        for (int w = pair; w < total; w += npairs) {
            const Work k = decode<kMode, true>(sh, p, w, rank);
            if (kMode == kWgrad && k.kblocks == 0) {
                const int mrow = k.m * kTileM + r_in_tile;
                if (mrow < p.M) {
                    float4 *dst = reinterpret_cast<float4 *>(p.dw + ((size_t)k.e * p.M + mrow) * p.N + k.n * kTileN);
                    const int cols = min(kTileN, p.N - k.n * kTileN);
                    for (int j = eg; j < cols / 4; j += 2) dst[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                continue;
            }
            const uint32_t buf = tile_it & 1u;
            const bool live = r_in_tile < k.rows;
            const size_t row = (size_t)k.row0 + r_in_tile;
            const int ncol = min(kTileN, p.N - k.n * kTileN);  // multiple of 64
            // kDAct: this warp's tiles: saved h1, h3 in (mapA1: both matrices as the planes of one 3-D
            // tensor), dH1, dH3, w*act out (mapS0: three planes).  Issuing a tile copy costs the warp well
            // over a hundred cycles whatever its size, so one copy carries the tiles of all planes.
            // The first input tiles are requested while the tensor cores still work on the tile.
            uint8_t *ib = store_stage + (size_t)wi * kDActWarpBytes;
            uint8_t *ob = ib + 4096;
            auto h_load = [&](int c) {  // 32 rows x columns [16c, 16c+16) of h1 (at ib) and h3 (at ib + 2048)
                if (lane == 0) {
                    mbar_expect_tx(&sh->ebar[wi], 4096);
                    tma_tile_3d(ib, &mapA1, k.n * kTileN + c * 16, k.prow0 + q * 32, 0, &sh->ebar[wi]);
                }
            };
            if (kMode == kDAct && !k.dead && eg * 16 < ncol) h_load(eg);
            if (!warp_wait(&sh->tfull[buf], (tile_it >> 1) & 1u, abort_flag, p.status,
                           p.test_tfull_limit_ns ? p.test_tfull_limit_ns : kWaitLimitNs))
                break;
            fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kAccCols;

            if (!k.dead) {  // a dead half stores nothing (its accumulator rows are its partner's rows again)
            if (kGU) {
#pragma unroll 1
                for (int c = eg; c < 4; c += 2) {
                    float g[32], u[32];
                    tmem_ld32(taddr + c * 32, g);
                    tmem_ld32(taddr + 128 + c * 32, u);
                    const int col0 = k.n * kTileN + c * 32;
                    if (col0 < p.N) {
                        if (!live) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) { g[j] = 0.f; u[j] = 0.f; }
                        }
                        // Results leave through shared memory: each lane writes its row into a
                        // swizzled 32 x 32 tile and a TMA store writes whole lines (training:
                        // mapS0 = g, mapS1 = u).  The one staging tile of the warp carries g, then
                        // Act, then u, each once the store before it has read the tile.
                        uint8_t *bt = store_stage + (size_t)wi * 4096;
                        auto stage_wait = [&]() {
                            if (store_it >= 1) {  // the previous store has read the staging tile
                                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                                __syncwarp();
                            }
                        };
                        auto stage_send = [&](const CUtensorMap *map) {
                            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                            __syncwarp();
                            if (lane == 0) {
                                tma_store_2d(map, bt, col0, k.prow0 + q * 32);
                                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                            }
                            ++store_it;
                        };
                        auto stage_f32 = [&](const float *v, const CUtensorMap *map) {
                            stage_wait();
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                *reinterpret_cast<float4 *>(bt + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                                    make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                            stage_send(map);
                        };
                        if (kMode == kGateUpTrain) stage_f32(g, &mapS0);
#pragma unroll
                        for (int j = 0; j < 32; ++j) g[j] = g[j] * sigmoidf_fast(g[j]) * u[j];
                        // Act (mapS2) leaves the same way: 32 x 32 elements, 64-byte rows for bf16
                        // (piece j of row r at j ^ ((r >> 1) & 3))
                        if constexpr (kF32) {
                            stage_f32(g, &mapS2);
                        } else {
                            stage_wait();
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                *reinterpret_cast<uint4 *>(bt + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4)) = pack8_bf16(g + 8 * j);
                            stage_send(&mapS2);
                        }
                        if (kMode == kGateUpTrain) stage_f32(u, &mapS1);
                    }
                }
            } else if (kMode == kDown || kMode == kDX) {
                const int tok = live ? p.row_token[row] : 0;
                const float wgt = kMode == kDown ? (live ? p.row_weight[row] : 0.0f) : 1.0f;
#pragma unroll 1
                for (int c = eg; c < 8; c += 2) {
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
            } else if (kMode == kDenseAdd) {
                // The rows of the tile are rows row0 .. of `out` (mapS0: [rows, N] fp32, 32 x 32 boxes): each
                // 32 x 32 piece goes through the warp's swizzled staging tile and is added to `out` by one
                // TMA reduce; rows and columns beyond the tensor are clipped.
#pragma unroll 1
                for (int c = eg; c < 8; c += 2) {
                    float y[32];
                    tmem_ld32(taddr + c * 32, y);
                    const int col0 = k.n * kTileN + c * 32;
                    if (col0 < p.N) {
                        uint8_t *bt = store_stage + (size_t)wi * 4096;
                        if (store_it >= 1) {  // the previous reduce has read the staging tile
                            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                            __syncwarp();
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            *reinterpret_cast<float4 *>(bt + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                                make_float4(y[4 * j], y[4 * j + 1], y[4 * j + 2], y[4 * j + 3]);
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                        if (lane == 0) {
                            tma_reduce_add_2d(&mapS0, bt, col0, k.row0 + q * 32);
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        }
                        ++store_it;
                    }
                }
            } else if (kMode == kDAct) {
                // z = W2_e^T dout_i for this row; delta = <z, act>; dact = w z; SwiGLU backward.
                // 16 columns per step.  Rows are 4 * N bytes apart in memory, so per-thread copies
                // would cost one memory transaction per row and instruction; the tiles travel by
                // TMA instead and each lane touches only shared memory: it reads its row of h1, h3
                // (64-byte rows, 16-byte piece j of row r at j ^ ((r >> 1) & 3)) and writes its row
                // of the three results (32-byte rows, piece j at j ^ ((r >> 2) & 1)).
                const float wgt = live ? p.row_weight[row] : 0.0f;
                float dsum = 0.0f;
                bool ok = true;
#pragma unroll 1
                for (int c = eg; c * 16 < ncol; c += kEpiGroups) {
                    if (!warp_wait(&sh->ebar[wi], ld_it & 1u, abort_flag, p.status)) { ok = false; break; }
                    ++ld_it;
                    float a1[16], a3[16], z[16];
                    uint32_t o1[8], o3[8], ow[8];  // dH1, dH3, w*act of the 16 columns as bf16 pairs
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int off = lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4);
                        const float4 x = *reinterpret_cast<const float4 *>(ib + off);
                        const float4 y = *reinterpret_cast<const float4 *>(ib + 2048 + off);
                        a1[4 * j] = x.x; a1[4 * j + 1] = x.y; a1[4 * j + 2] = x.z; a1[4 * j + 3] = x.w;
                        a3[4 * j] = y.x; a3[4 * j + 1] = y.y; a3[4 * j + 2] = y.z; a3[4 * j + 3] = y.w;
                    }
                    // Every lane holds its inputs: the input tiles may be refilled.  The refill is a
                    // write through the async proxy; without the proxy fence it can overtake the
                    // shared-memory loads just issued (measured: wrong h3 values now and then).
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if ((c + kEpiGroups) * 16 < ncol) h_load(c + kEpiGroups);
                    tmem_ld16(taddr + c * 16, z);
                    if (live) {
                        // two columns at a time in packed fp32 pairs (the epilogue warps are bound by the
                        // instructions they issue; only the exponential and the reciprocal stay scalar)
                        const f32x2 one2 = pack2(1.0f, 1.0f), mone2 = pack2(-1.0f, -1.0f), w2 = pack2(wgt, wgt);
                        const f32x2 nl2e = pack2(-1.4426950408889634f, -1.4426950408889634f);
                        f32x2 dsum2 = pack2(0.0f, 0.0f);
#pragma unroll
                        for (int j = 0; j < 16; j += 2) {
                            const f32x2 g = pack2(a1[j], a1[j + 1]), u = pack2(a3[j], a3[j + 1]), zz = pack2(z[j], z[j + 1]);
                            float t0, t1;
                            unpack2(mul2(g, nl2e), t0, t1);                       // -g log2(e)
                            const f32x2 den = add2(pack2(exp2f_fast(t0), exp2f_fast(t1)), one2);
                            unpack2(den, t0, t1);
                            const f32x2 sg = pack2(rcp_fast(t0), rcp_fast(t1));   // sigmoid(g)
                            const f32x2 sl = mul2(g, sg);                          // silu(g)
                            const f32x2 ac = mul2(sl, u);                          // act = silu(g) u
                            dsum2 = fma2(zz, ac, dsum2);
                            const f32x2 wa2 = mul2(w2, ac), da = mul2(w2, zz);
                            // d silu / dg = sg (1 + g (1 - sg))
                            const f32x2 dg = mul2(mul2(mul2(da, u), sg), fma2(g, fma2(sg, mone2, one2), one2));
                            const f32x2 du = mul2(da, sl);
                            ow[j >> 1] = pack_bf16x2(wa2);
                            o1[j >> 1] = pack_bf16x2(dg);
                            o3[j >> 1] = pack_bf16x2(du);
                        }
                        {
                            float s0, s1;
                            unpack2(dsum2, s0, s1);
                            dsum += s0 + s1;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j) { o1[j] = 0u; o3[j] = 0u; ow[j] = 0u; }
                    }
                    if (store_it >= 1) {  // the previous store has read the staging tiles
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        __syncwarp();
                    }
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        const int off = lane * 32 + ((t ^ ((lane >> 2) & 1)) << 4);
                        *reinterpret_cast<uint4 *>(ob + off) = make_uint4(o1[4 * t], o1[4 * t + 1], o1[4 * t + 2], o1[4 * t + 3]);
                        *reinterpret_cast<uint4 *>(ob + 1024 + off) = make_uint4(o3[4 * t], o3[4 * t + 1], o3[4 * t + 2], o3[4 * t + 3]);
                        *reinterpret_cast<uint4 *>(ob + 2048 + off) = make_uint4(ow[4 * t], ow[4 * t + 1], ow[4 * t + 2], ow[4 * t + 3]);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_3d(&mapS0, ob, k.n * kTileN + c * 16, k.prow0 + q * 32, 0);
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                    ++store_it;
                }
                if (!ok) break;
                if (live) atomicAdd(p.delta + row, dsum);
            } else if (kIsGate) {
                // the rows of the tile are tokens in order, the first N accumulator columns their scores
#pragma unroll 1
                for (int c = eg; c * 32 < p.N; c += 2) {
                    float y[32];
                    tmem_ld32(taddr + c * 32, y);
                    if (live) {
                        float *dst = p.out + row * p.N + c * 32;
                        const int nv = min(32, p.N - c * 32);
                        if ((p.N & 3) == 0) {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                if (4 * j < nv)
                                    *reinterpret_cast<float4 *>(dst + 4 * j) = make_float4(y[4 * j], y[4 * j + 1], y[4 * j + 2], y[4 * j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < nv) dst[j] = y[j];
                        }
                    }
                }
                if (kMode == kGateSel) {
                    // The token's scores are still in this thread's TMEM lane: the first warp of each lane
                    // quarter selects (Eq. 1: the k+1 best by (score desc, index asc), walked in ascending
                    // column order with strict ">"; Section 4.1: the best expert of the token's group), the
                    // second one adds up the softmax values of its 32 tokens per expert.
                    if (eg == 0) {
                        if (p.sel_k + 1 <= 3) gate_select<3>(p, taddr, (int)row, live);
                        else gate_select<kMaxK + 1>(p, taddr, (int)row, live);
                    } else if (p.sel_psum) {
                        gate_softmax_sums(p, taddr, (int)row, live, lane);
                    }
                }
            } else {  // kWgrad: row of the tile = row of dW_e
                // 32 x 32 fp32 pieces go through a swizzled staging tile (two per warp, in
                // rotation) and leave by TMA stores on the 3-D view [E][M][N] of dW (mapS0), which
                // clips rows beyond M and columns beyond N
#pragma unroll 1
                for (int c = eg; c < 8; c += 2) {
                    float y[32];
                    tmem_ld32(taddr + c * 32, y);
                    const int col0 = k.n * kTileN + c * 32;
                    if (col0 < p.N) {
                        uint8_t *bs = store_stage + (size_t)wi * 4096;
                        if (store_it >= 1) {  // the previous store has read the staging tile
                            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                            __syncwarp();
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            *reinterpret_cast<float4 *>(bs + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                                make_float4(y[4 * j], y[4 * j + 1], y[4 * j + 2], y[4 * j + 3]);
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                        if (lane == 0) {
                            tma_store_3d(&mapS0, bs, col0, k.m * kTileM + q * 32, k.e);
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        }
                        ++store_it;
                    }
                }
            }
            }
            fence_before_sync();
            mbar_arrive_cluster(lead_tempty + 8u * buf);  // both CTAs free the accumulator at the leader
            ++tile_it;
        }
        if ((kGU || kMode == kWgrad || kMode == kDenseAdd) && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        if (kMode == kDAct && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    __syncwarp();  // the single-lane loops above rejoin their warps
    __syncthreads();
    if (sh->abort_flag) __nanosleep(2000000);  // let copies that are still in flight land
    cluster_sync_all();  // neither CTA leaves while its peer may still signal its barriers
    if (warp == kMmaWarp) {
        fence_after_sync();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

// ---- host helpers ---------------------------------------------------------------------
inline int sm_count()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return n;
}

// a0, a1: A operand(s); b0, b1: B operand(s); s0..s2: store views of the epilogue (kDAct: a1, b1 =
// saved h1, h3 as read by its epilogue).  Unused maps may repeat another one.  The grid is rounded down to whole CTA pairs.
template <int kMode, bool kF32>
cudaError_t launch(const CUtensorMap &a0, const CUtensorMap &a1, const CUtensorMap &b0, const CUtensorMap &b1,
                   const CUtensorMap &s0, const CUtensorMap &s1, const CUtensorMap &s2, const Params &p, int grid,
                   cudaStream_t st, size_t smem_bytes = smem_bytes_of<kMode>())
{
    cudaError_t err = cudaFuncSetAttribute(k_gemm<kMode, kF32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)smem_bytes);
    if (err != cudaSuccess) return err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid & ~1);
    cfg.blockDim = dim3(threads_of<kMode>());
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_gemm<kMode, kF32>, a0, a1, b0, b1, s0, s1, s2, p);
}

// Number of 128-row tiles per expert, as an exclusive prefix (a template only so that every
// translation unit that launches it carries its own copy).
template <int kUnused = 0>
__global__ void k_tiles(int E, const int *__restrict__ row_offset, int *__restrict__ mt_off)
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

}  // namespace gemm
}  // namespace rr
