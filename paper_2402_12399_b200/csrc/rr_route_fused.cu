// The router as ONE persistent kernel (arXiv 2402.12399, Section 3 Eq. 1-2, Section 4.1 Eq. 3,
// Section 4.2): every mode except RR_SCORE and RR_LOCAL_CAP.
//
// The grid is at most one block per SM, launched cooperatively; every block owns a contiguous range
// of 32-token units and every warp a contiguous part of it, so "token order" is (block, warp, unit,
// lane) order and a position in an expert's queue is
//     slots taken by lower ranks (all tokens)  +  same (rank, expert) in earlier blocks
//   + same (rank, expert) in earlier warps of the block  +  running count inside the warp.
// The phases are separated by grid-wide barriers (an arrival counter in the workspace header; every
// wait has a time limit and latches RR_ERR_TIMEOUT):
//   1  one pass over logits[T,E]: the rows of 32 tokens arrive in shared memory as 128-byte-swizzled
//      boxes by TMA (several in flight per warp), one thread per token walks its row in ascending
//      column order -- conflict-free thanks to the swizzle -- and keeps the k+1 best entries by
//      insertion with strict ">" (ties stay with the lower index, Eq. 1), in two levels for wide
//      rows; in-group best expert (Section 4.1); running per-warp counts of every (rank, expert)
//   -- barrier: counts of all blocks are known --
//   2  slots (Section 3: kept iff position < capacity), drops, nominee lists (Section 4.2, stage
//      one), running counts of the IR tokens per expert
//   -- barrier --
//   3  Fill-in Rectification, stage two: blocks share out the experts, each picks the best nominees
//      by radix select and places them in token order
//   -- barrier --
//   4  IR lists, combine weights (Eq. 2 / Eq. 3), row space, marks outside the live ranges
// Per-token records between the phases stay in shared memory when the block's range is short enough
// and go through the workspace (L2) otherwise.
#include <float.h>
#include <string.h>

#include "rr_common.cuh"
#include "rr_route_dev.cuh"
#include "rr_tc.cuh"

namespace rr {

namespace {

constexpr int kMaxWarps = 16;
constexpr int kSmemBudget = 220 * 1024;

struct FusedParams {
    const float *logits;
    int T, E, k, C, G;
    unsigned mode;
    int nblk;         // 32-token units
    int bpc;          // units per block
    int bpw;          // units per warp
    int ns;           // row stages per warp
    int tma;          // 1: swizzled boxes by TMA (E % 32 == 0); 0: lanes copy rows into padded rows
    int pitch;        // floats per staged row of the padded layout
    int stage_bytes;  // one stage = the rows of 32 tokens
    int rec_smem;     // records of the block's tokens stay in shared memory
    unsigned long long wait_limit_ns;  // time limit of the grid barriers
    int presel;       // 1: the selection was made by the gate projection's epilogue (`pre`), logits are not read
    RoutePresel pre;
    rr_route_tables t;
    RouteScratch s;
};

// Shared-memory plan, the same on host (size) and device (pointers).
struct Plan {
    size_t stages, bars, wcnt, wir, pre, tot, base, kept, take, nnom, loff, occ, irpre, irtot, iro, row, sel, misc, rec, end;
};
__host__ __device__ inline Plan make_plan(int nw, int ns, int stage_bytes, int E, int k, int rec_words)
{
    const size_t cols = (size_t)(k + 1) * E;
    Plan p;
    size_t o = 0;
    auto take = [&](size_t bytes, size_t align) { o = (o + align - 1) / align * align; const size_t at = o; o += bytes; return at; };
    p.stages = take((size_t)nw * ns * stage_bytes, 1024);
    p.bars = take((size_t)nw * ns * 8, 8);
    p.wcnt = take((size_t)nw * cols * 4, 16);
    p.wir = take((size_t)nw * E * 4, 16);
    p.pre = take((cols + 7) / 8 * 8 * 4, 16);  // (column sums come in groups of eight)
    p.tot = take((cols + 7) / 8 * 8 * 4, 16);
    p.base = take((size_t)k * E * 4, 16);
    p.kept = take((size_t)E * 4, 16);
    p.take = take((size_t)E * 4, 16);
    p.nnom = take((size_t)E * 4, 16);
    p.loff = take((size_t)(E + 1) * 4, 16);
    p.occ = take((size_t)E * 4, 16);
    p.irpre = take((size_t)(E + 7) / 8 * 8 * 4, 16);
    p.irtot = take((size_t)(E + 7) / 8 * 8 * 4, 16);
    p.iro = take((size_t)(E + 1) * 4, 16);
    p.row = take((size_t)(E + 1) * 4, 16);
    p.sel = take(sizeof(SelectShared), 16);
    p.misc = take(64, 16);
    p.rec = take((size_t)rec_words * 4, 16);
    p.end = o;
    return p;
}

// 16-byte piece g of a staged row: rowbase + (g / 8) * box_stride + (((g % 8) ^ x) * 16).  Swizzled
// boxes: box_stride = 4096, x = row % 8, rowbase = stage + row * 128; padded rows: box_stride = 128,
// x = 0, rowbase = stage + row * pitch * 4.
struct RowView {
    const uint8_t *base;
    int box_stride, x;
    __device__ __forceinline__ float4 piece(int g) const
    {
        return *reinterpret_cast<const float4 *>(base + (g >> 3) * box_stride + (((g & 7) ^ x) << 4));
    }
    __device__ __forceinline__ float at(int j) const
    {
        const int g = j >> 2;
        return *reinterpret_cast<const float *>(base + (g >> 3) * box_stride + (((g & 7) ^ x) << 4) + ((j & 3) << 2));
    }
};

__device__ __forceinline__ void nonfinite_probe(const float4 &f, float &chk)
{
    // x * 0 is NaN for a NaN and for both infinities
    chk = fmaf(f.x, 0.0f, chk); chk = fmaf(f.y, 0.0f, chk);
    chk = fmaf(f.z, 0.0f, chk); chk = fmaf(f.w, 0.0f, chk);
}

// The k+1 best columns of one row by (value desc, index asc): the row is walked in ascending column
// order and an entry enters the list only ahead of strictly smaller values, so equal values keep
// their index order.  Wide rows (E >= 8 KK, E % 4 == 0) in two levels: first the KK best groups of
// four columns by group maximum (every one of the KK best columns lies in one of them: a column
// outside has, in each chosen group, that group's maximum ahead of it -- larger, or equal at a lower
// index), then only those groups' columns, again in ascending order.  `np` = pieces of the row.
template <int KK>
__device__ __forceinline__ void select_row(const RowView &rv, int E, int np, float (&bv)[KK], int (&bj)[KK], float &chk)
{
#pragma unroll
    for (int r = 0; r < KK; ++r) { bv[r] = empty_place(); bj[r] = INT_MAX; }
    if ((E & 3) == 0 && E >= 8 * KK) {
        float gv[KK];
        int gs[KK];
#pragma unroll
        for (int r = 0; r < KK; ++r) { gv[r] = empty_place(); gs[r] = INT_MAX; }
#pragma unroll 4
        for (int g = 0; g < np; ++g) {
            const float4 f = rv.piece(g);
            nonfinite_probe(f, chk);
            insert_strict<KK>(fmaxf(fmaxf(f.x, f.y), fmaxf(f.z, f.w)), g, gv, gs);
        }
        // A row of NaNs or of -inf leaves places empty (nothing exceeds -inf, NaN compares false):
        // such a place takes the lowest group not yet chosen (E >= 8 KK: it exists), so that every
        // piece read below lies inside the row.  `chk` reports the row in any case.
#pragma unroll
        for (int r = 0; r < KK; ++r) {
            if (gs[r] == INT_MAX) {
                int cand = 0;
#pragma unroll
                for (int t = 0; t < KK; ++t) {
                    bool used = false;
#pragma unroll
                    for (int q = 0; q < KK; ++q) used |= (q < r && gs[q] == cand);
                    cand += used ? 1 : 0;
                }
                gs[r] = cand;
            }
        }
#pragma unroll
        for (int a = 0; a < KK - 1; ++a)  // the chosen groups in ascending order
#pragma unroll
            for (int b = 0; b < KK - 1 - a; ++b) {
                const int lo_g = min(gs[b], gs[b + 1]), hi_g = max(gs[b], gs[b + 1]);
                gs[b] = lo_g;
                gs[b + 1] = hi_g;
            }
#pragma unroll
        for (int r = 0; r < KK; ++r) {
            const float4 f = rv.piece(gs[r]);
            const int j = 4 * gs[r];
            insert_strict<KK>(f.x, j, bv, bj); insert_strict<KK>(f.y, j + 1, bv, bj);
            insert_strict<KK>(f.z, j + 2, bv, bj); insert_strict<KK>(f.w, j + 3, bv, bj);
        }
    } else {
        // every piece; in the padded layout the columns beyond E hold -FLT_MAX and sit above every
        // real column, so they can only fill places no real column claims
#pragma unroll 2
        for (int g = 0; g < np; ++g) {
            const float4 f = rv.piece(g);
            nonfinite_probe(f, chk);
            const int j = 4 * g;
            insert_strict<KK>(f.x, j, bv, bj); insert_strict<KK>(f.y, j + 1, bv, bj);
            insert_strict<KK>(f.z, j + 2, bv, bj); insert_strict<KK>(f.w, j + 3, bv, bj);
        }
    }
}

// Grid-wide barrier number `epoch` (1, 2, ...) of this launch: every block adds one to the arrival word
// and has passed when it reads epoch * gridDim.x.  (Spreading the arrivals over several words was
// measured and is slower: the blocks then poll several words.)  Returns false when the wait ran out or
// another block gave up; the caller then leaves the kernel.
__device__ __forceinline__ bool grid_barrier(int *sync, int *status, int epoch, int *sh_ok, unsigned long long limit_ns)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(&sync[0], 1);
        const int target = epoch * (int)gridDim.x;
        int ok = 1, seen;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(sync) : "memory");
        if (seen < target) {
            const unsigned long long t0 = tc::globaltimer();
            unsigned it = 0;
            for (;;) {
                asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(sync) : "memory");
                if (seen >= target) break;
                if ((++it & 63u) == 0 || limit_ns < 1000000ull) {  // (a limit below 1 ms is a test's: look at the clock every time)
                    int gave_up;
                    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(gave_up) : "l"(sync + 1) : "memory");
                    if (gave_up) { ok = 0; break; }
                    if (tc::globaltimer() - t0 > limit_ns) {
                        atomicExch(&sync[1], 1);
                        latch_status(status, RR_ERR_TIMEOUT);
                        ok = 0;
                        break;
                    }
                }
            }
        }
        *sh_ok = ok;
    }
    __syncthreads();
    return *sh_ok != 0;
}

// counts[block][column], 16-bit (a block's range holds fewer than 65536 tokens), `stride` counts per
// block (a multiple of 8), `ncta` rows written.  For every column: the sum over the blocks before this
// one is added onto pre[c], the sum over all blocks onto tot[c] (shared memory, zero on entry).  Every
// block reads every row, so this costs L2 traffic and one round of loads: a thread takes eight
// neighbouring columns (one 16-byte load per row) of up to eight rows, all in flight together; the threads
// that share columns meet in shared-memory atomics (different words inside a warp).
__device__ __forceinline__ void column_sums(const uint16_t *counts, int stride, int ncta, int *pre, int *tot, int tid, int nthr)
{
    // (run by the threads tid = 0 .. nthr-1 of the block, all of them or a part)
    const int bid = (int)blockIdx.x;
    const int nvec = stride >> 3;                               // 16-byte pieces per row
    const int ngrp = nthr >= nvec ? nthr / nvec : 1;            // groups of threads, each a share of the rows
    for (int item = tid; item < nvec * ngrp; item += nthr) {
        const int g = item / nvec, vq = item - g * nvec;
        int all[8], mine[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) { all[q] = 0; mine[q] = 0; }
        for (int b0 = g; b0 < ncta; b0 += 8 * ngrp) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int b = b0 + u * ngrp;
                v[u] = make_uint4(0, 0, 0, 0);
                if (b < ncta) v[u] = __ldcg(reinterpret_cast<const uint4 *>(counts + (size_t)b * stride) + vq);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const bool before = b0 + u * ngrp < bid;
                const unsigned w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int x = (int)((w[q >> 1] >> (16 * (q & 1))) & 0xffffu);
                    all[q] += x;
                    mine[q] += before ? x : 0;
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            if (all[q]) atomicAdd(&tot[8 * vq + q], all[q]);
            if (mine[q]) atomicAdd(&pre[8 * vq + q], mine[q]);
        }
    }
}

// out[e] = sum over the rows r0 <= r < r1 of src[r * E + e] (fp32, read through L2).  The rows are dealt
// to as many groups of threads as the block has room for, each group a contiguous share with eight loads
// in flight, and the groups' partial sums are added in group order: a fixed association, so the result
// repeats bit for bit, at the cost of a few L2 round trips.  `part` = max(blockDim.x, E) floats of shared
// memory; `out` may be global or shared.  Ends with a block barrier.
__device__ __forceinline__ void fixed_order_sums(const float *src, int r0, int r1, int E, float *part, float *out)
{
    const int nthr = (int)blockDim.x, tid = (int)threadIdx.x;
    const int parts = nthr >= E ? nthr / E : 1;
    const int per = (r1 - r0 + parts - 1) / parts;
    for (int item = tid; item < parts * E; item += nthr) {
        const int g = item / E, e = item - g * E;
        const int a = r0 + g * per, b = a + per < r1 ? a + per : r1;
        float acc = 0.0f;
        for (int r = a; r < b; r += 8) {
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = r + u < b ? __ldcg(src + (size_t)(r + u) * E + e) : 0.0f;
#pragma unroll
            for (int u = 0; u < 8; ++u) acc += v[u];
        }
        part[item] = acc;
    }
    __syncthreads();
    for (int e = tid; e < E; e += nthr) {
        float acc = 0.0f;
        for (int g = 0; g < parts; ++g) acc += part[g * E + e];
        out[e] = acc;
    }
    __syncthreads();
}

// Every block passes here on its way out, whatever happened: the last one puts the barrier words back
// to zero, so the next call starts clean even after a wait that ran out.
__device__ __forceinline__ void leave_grid(int *sync)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(&sync[2], 1) == (int)gridDim.x - 1) {
            sync[0] = 0;
            sync[1] = 0;
            sync[2] = 0;
            __threadfence();
        }
    }
}

// kVar picks what the first phase carries besides the selection, at compile time (the common kernel is
// smaller, and its warps run every piece of code only once): 0 nothing, 1 the softmax work (RR_FR_SOFTMAX's
// key and / or the sums of the load-balance loss, each behind its run-time flag), 2 no selection at all (made
// by the gate projection's epilogue).
// kTma: the rows arrive as swizzled boxes by TMA (E % 32 == 0); else the lanes copy them into padded rows.
template <int KK, int kVar, bool kTma>
__global__ void __launch_bounds__(kMaxWarps * 32, 1)
k_route_fused(const __grid_constant__ CUtensorMap map, const FusedParams p)
{
    constexpr bool kPresel = kVar == 2;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = (int)blockDim.x >> 5, nthr = (int)blockDim.x;
    const int T = p.T, E = p.E, k = p.k, C = p.C, K1 = k + 1, K2 = k + 2;
    const int cols = K1 * E;
    const int NF = route_rec_fields(k);
    const unsigned mode = p.mode;
    const bool soft = kVar == 1 && (mode & RR_FR_SOFTMAX) != 0;
    const bool want_sums = kVar != 0 && p.pre.psum != nullptr;
    const rr_route_tables &t = p.t;

    const int cta_first = (int)blockIdx.x * p.bpc;
    const int cta_end = min(cta_first + p.bpc, p.nblk);
    const int w_first = min(cta_first + warp * p.bpw, cta_end);
    const int w_end = min(w_first + p.bpw, cta_end);
    const int nb_w = w_end - w_first;

    const Plan pl = make_plan(nw, p.ns, p.stage_bytes, E, k, p.rec_smem ? p.bpc * 32 * NF : 0);
    uint8_t *my_stages = sm + pl.stages + (size_t)warp * p.ns * p.stage_bytes;
    uint64_t *bar = reinterpret_cast<uint64_t *>(sm + pl.bars) + warp * p.ns;
    int *wcnt = reinterpret_cast<int *>(sm + pl.wcnt);
    int *wir = reinterpret_cast<int *>(sm + pl.wir);
    int *pre_s = reinterpret_cast<int *>(sm + pl.pre);
    int *tot_s = reinterpret_cast<int *>(sm + pl.tot);
    int *base_s = reinterpret_cast<int *>(sm + pl.base);
    int *kept_s = reinterpret_cast<int *>(sm + pl.kept);
    int *take_s = reinterpret_cast<int *>(sm + pl.take);
    int *nnom_s = reinterpret_cast<int *>(sm + pl.nnom);
    int *loff_s = reinterpret_cast<int *>(sm + pl.loff);
    int *occ_s = reinterpret_cast<int *>(sm + pl.occ);
    int *irpre_s = reinterpret_cast<int *>(sm + pl.irpre);
    int *irtot_s = reinterpret_cast<int *>(sm + pl.irtot);
    int *iro_s = reinterpret_cast<int *>(sm + pl.iro);
    int *row_s = reinterpret_cast<int *>(sm + pl.row);
    SelectShared &selsh = *reinterpret_cast<SelectShared *>(sm + pl.sel);
    int *misc = reinterpret_cast<int *>(sm + pl.misc);  // [0] abort flag of the block, [1] outcome of a grid barrier
    // records: [unit][field][lane]
    int *rec = p.rec_smem ? reinterpret_cast<int *>(sm + pl.rec) : p.s.rec + (size_t)cta_first * 32 * NF;
    auto rec_of = [&](int blk) { return rec + (size_t)(blk - cta_first) * 32 * NF + lane; };

    // ---------------------------------------------------------------- set-up
    if (tid == 0) { misc[0] = 0; misc[1] = 1; }
    if (lane == 0 && kTma) {
        // the warp's first rows are requested before anything else: the counters below are cleared while
        // they are on their way
        for (int s = 0; s < p.ns; ++s) tc::mbar_init(&bar[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // (launched as a programmatic dependent of the kernel before it in the stream: everything up to here
        // may run while that kernel drains; nothing in global memory is touched before it has completed)
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (!kPresel) {
            const int nboxes = E >> 5;
            for (int j = 0; j < nb_w && j < p.ns; ++j) {
                uint8_t *dst = my_stages + (size_t)j * p.stage_bytes;
                tc::mbar_expect_tx(&bar[j], (unsigned)nboxes * 4096u);
                for (int b = 0; b < nboxes; ++b) tc::tma_tile_2d(dst + b * 4096, &map, 32 * b, (w_first + j) * 32, &bar[j]);
            }
        }
    }
    for (int c = tid; c < nw * cols; c += nthr) wcnt[c] = 0;
    for (int c = tid; c < nw * E; c += nthr) wir[c] = 0;
    const int cols8 = (cols + 7) & ~7, E8 = (E + 7) & ~7;  // counts per block in the workspace: multiples of eight
    for (int c = tid; c < cols8; c += nthr) { pre_s[c] = 0; tot_s[c] = 0; }
    for (int c = tid; c < E8; c += nthr) { irpre_s[c] = 0; irtot_s[c] = 0; }
    if (!kTma && (E & 3)) {  // columns E .. of the last piece of a padded row: below every real value
        float *st = reinterpret_cast<float *>(sm + pl.stages);
        const int n = nw * p.ns * (p.stage_bytes >> 2);
        for (int c = tid; c < n; c += nthr) st[c] = -FLT_MAX;
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __syncthreads();
    volatile int *abort_flag = misc;
    int epoch = 0;

    // ---------------------------------------------------------------- phase 1
    {
        const int nboxes = E >> 5;
        auto issue = [&](int j) {
            if (lane == 0) {
                const int s = j % p.ns;
                uint8_t *dst = my_stages + (size_t)s * p.stage_bytes;
                tc::mbar_expect_tx(&bar[s], (unsigned)nboxes * 4096u);
                for (int b = 0; b < nboxes; ++b) tc::tma_tile_2d(dst + b * 4096, &map, 32 * b, (w_first + j) * 32, &bar[s]);
            }
        };
        const int tpg = T / p.G > 0 ? T / p.G : 1, epg = E / p.G;
        const int np = kTma ? (E >> 2) : ((E + 3) >> 2);
        int *wc = wcnt + warp * cols;
        bool bad = false;
        for (int j = 0; j < nb_w; ++j) {
            const int blk = w_first + j;
            const int i = blk * 32 + lane;
            const bool live = i < T;
            uint8_t *st = my_stages + (size_t)(j % p.ns) * p.stage_bytes;
            bool rows_ok = true;
            if (kPresel) {
                // nothing to stage: the gate projection's epilogue has selected (below)
            } else if (kTma) {
                rows_ok = tc::warp_wait(&bar[j % p.ns], (unsigned)(j / p.ns) & 1u, abort_flag, p.s.status);
            } else {
                const int ntok = min(32, T - blk * 32);
                const float *src = p.logits + (size_t)blk * 32 * E;
                if ((E & 3) == 0) {
                    const int c4 = E >> 2;
                    for (int q = lane; q < ntok * c4; q += 32) {
                        const int r = q / c4, c = q - r * c4;
                        *reinterpret_cast<float4 *>(st + ((size_t)r * p.pitch + 4 * c) * 4) = __ldg(reinterpret_cast<const float4 *>(src) + q);
                    }
                } else {
                    for (int q = lane; q < ntok * E; q += 32) {
                        const int r = q / E, c = q - r * E;
                        reinterpret_cast<float *>(st)[(size_t)r * p.pitch + c] = __ldg(src + q);
                    }
                }
                __syncwarp();
            }
            RowView rv;
            if (kTma) { rv.base = st + lane * 128; rv.box_stride = 4096; rv.x = lane & 7; }
            else { rv.base = st + (size_t)lane * p.pitch * 4; rv.box_stride = 128; rv.x = 0; }

            float bv[KK], gv = 0.0f, chk = 0.0f, frk = 0.0f;
            int bj[KK], gj = INT_MAX;
            const int grp = live ? i / tpg : 0;
            const int lo = grp * epg, hi = lo + epg;
            if (kPresel) {
#pragma unroll
                for (int r = 0; r < KK; ++r) {
                    bv[r] = 0.0f;
                    bj[r] = INT_MAX;
                    if (live && r < K1) {
                        const int e = t.topk_expert[(size_t)i * K1 + r];
                        bj[r] = e >= 0 ? e : INT_MAX;
                        bv[r] = p.pre.val[(size_t)i * K1 + r];
                    }
                }
                if (live) { gj = p.pre.h[i]; gv = p.pre.a_h[i]; }
            } else if (live && rows_ok) {
                select_row<KK>(rv, E, np, bv, bj, chk);
                // Section 4.1: the best expert among those of the token's own group (ascending walk,
                // strict ">": the lower index keeps a tie)
                gv = -CUDART_INF_F;
                if ((epg & 3) == 0) {
                    for (int g = lo >> 2; g < (hi >> 2); ++g) {
                        const float4 f = rv.piece(g);
                        const int j0 = 4 * g;
                        if (f.x > gv) { gv = f.x; gj = j0; }
                        if (f.y > gv) { gv = f.y; gj = j0 + 1; }
                        if (f.z > gv) { gv = f.z; gj = j0 + 2; }
                        if (f.w > gv) { gv = f.w; gj = j0 + 3; }
                    }
                } else {
                    for (int c = lo; c < hi; ++c) {
                        const float x = rv.at(c);
                        if (x > gv) { gv = x; gj = c; }
                    }
                }
                if (soft) {
                    // softmax value of the token at its (k+1)-th expert by the fixed recipe: e_j in index
                    // order, one sum, one division (every operation rounds to nearest even)
                    const float mx = bv[0];
                    float Z = 0.0f;
                    for (int c = 0; c < E; ++c) Z = __fadd_rn(Z, exp_fixed(__fsub_rn(rv.at(c), mx)));
                    float vk = bv[0];
#pragma unroll
                    for (int r = 0; r < KK; ++r)
                        if (r == k) vk = bv[r];
                    frk = __fdiv_rn(exp_fixed(__fsub_rn(vk, mx)), Z);
                }
            } else {
#pragma unroll
                for (int r = 0; r < KK; ++r) { bv[r] = 0.0f; bj[r] = INT_MAX; }
            }
            if (kVar == 1 && want_sums) {
                // load-balance loss (Section 5.1): softmax of the token's row, summed per expert over the
                // unit's 32 tokens (hardware exponentials, relative error about 1e-6; tokens beyond T count
                // as zero)
                // (16-byte pieces; the columns beyond E of a padded row hold -FLT_MAX: their exponential is 0)
                float inv = 0.0f;
                const float mx = bv[0];
                if (live && rows_ok) {
                    float Z = 0.0f;
                    for (int g = 0; g < np; ++g) {
                        const float4 f = rv.piece(g);
                        Z += (__expf(f.x - mx) + __expf(f.y - mx)) + (__expf(f.z - mx) + __expf(f.w - mx));
                    }
                    inv = 1.0f / Z;
                }
                for (int g0 = 0; g0 < np; g0 += 8) {
                    float v[32];
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        float4 f = make_float4(-FLT_MAX, -FLT_MAX, -FLT_MAX, -FLT_MAX);
                        if (inv != 0.0f && g0 + q < np) f = rv.piece(g0 + q);
                        v[4 * q] = __expf(f.x - mx) * inv;
                        v[4 * q + 1] = __expf(f.y - mx) * inv;
                        v[4 * q + 2] = __expf(f.z - mx) * inv;
                        v[4 * q + 3] = __expf(f.w - mx) * inv;
                    }
                    warp_transpose_add(v, lane);
                    if (4 * g0 + lane < E) p.pre.psum[(size_t)blk * E + 4 * g0 + lane] = v[0];
                }
            }
            // the stage is free: fetch the unit that will use it next
            if (kTma && !kPresel && j + p.ns < nb_w) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the reads above before the async-proxy write
                __syncwarp();
                issue(j + p.ns);
            }
            if (live && (chk != 0.0f || !rows_ok)) {
                // a NaN or an infinity, or rows that never arrived: the tables are undefined, but every
                // index written must still name an expert
                bad = bad || chk != 0.0f;
#pragma unroll
                for (int r = 0; r < KK; ++r)
                    if ((bj[r] == INT_MAX || bj[r] >= E) && r < E) { bj[r] = r; bv[r] = 0.0f; }
                if (gj == INT_MAX) { gj = lo; gv = 0.0f; }
            }
            if (gj == INT_MAX) gj = lo;

            // position among the warp's tokens with the same (rank, expert), in token order
            int e_r[KK], cnt[KK], rk[KK];
            unsigned mm[KK];
#pragma unroll
            for (int r = 0; r < KK; ++r) {
                if (r < K1) {
                    const int e = (live && bj[r] < E) ? bj[r] : -1;  // INT_MAX / a padded column: none (E == k)
                    e_r[r] = e;
                    mm[r] = __match_any_sync(kFull, e);
                    rk[r] = __popc(mm[r] & ((1u << lane) - 1u));
                    cnt[r] = e >= 0 ? wc[r * E + e] : 0;
                }
            }
            __syncwarp();
#pragma unroll
            for (int r = 0; r < KK; ++r)
                if (r < K1 && e_r[r] >= 0 && rk[r] == 0) wc[r * E + e_r[r]] = cnt[r] + __popc(mm[r]);
            __syncwarp();
            if (live) {
                int *rb = rec_of(blk);
#pragma unroll
                for (int r = 0; r < KK; ++r) {
                    if (r < K1) {
                        if (!kPresel) t.topk_expert[(size_t)i * K1 + r] = e_r[r];
                        rb[r * 32] = __float_as_int(bv[r]);
                        rb[(K1 + r) * 32] = cnt[r] + rk[r];
                        rb[(2 * K1 + r) * 32] = e_r[r];
                    }
                }
                rb[(3 * K1) * 32] = gj;
                rb[(3 * K1 + 1) * 32] = __float_as_int(gv);
                if (soft) p.s.fr_key[i] = frk;
            }
        }
        if (bad) latch_status(p.s.status, RR_ERR_NONFINITE);
    }
    __syncthreads();
    if (misc[0]) {  // a row wait gave up: tell the other blocks, let copies still in flight land, leave
        if (tid == 0) atomicExch(&p.s.sync[1], 1);
        __nanosleep(2000000);
        leave_grid(p.s.sync);
        return;
    }
    if (want_sums) {
        // load-balance loss (Section 5.1): the softmax sums of the block's 32-token units, in unit order
        fixed_order_sums(p.pre.psum, cta_first, cta_end, E, reinterpret_cast<float *>(selsh.hist),
                         p.pre.cta_psum + (size_t)blockIdx.x * E);
    }
    // counts of the block per column; the warps' counts become exclusive prefixes over the warps
    for (int c = tid; c < cols; c += nthr) {
        int run = 0;
        for (int w = 0; w < nw; ++w) {
            const int x = wcnt[w * cols + c];
            wcnt[w * cols + c] = run;
            run += x;
        }
        p.s.agg[(size_t)blockIdx.x * cols8 + c] = (uint16_t)run;
    }
    if (!grid_barrier(p.s.sync, p.s.status, ++epoch, misc + 1, p.wait_limit_ns)) { leave_grid(p.s.sync); return; }

    // ---------------------------------------------------------------- phase 2
    const int ncta = (int)gridDim.x;
    column_sums(p.s.agg, cols8, ncta, pre_s, tot_s, tid, nthr);  // per column: counts of the earlier blocks, of all blocks
    __syncthreads();
    for (int e = tid; e < E; e += nthr) {
        int n = 0;
        for (int r = 0; r < k; ++r) { base_s[r * E + e] = n; n += tot_s[r * E + e]; }
        const int kept = n < C ? n : C;
        const int nn = (mode & RR_FR) ? tot_s[k * E + e] : 0;
        const int tk = nn < C - kept ? nn : C - kept;  // Section 4.2: padding slots go to the best nominees
        kept_s[e] = kept;
        take_s[e] = tk;
        nnom_s[e] = nn;
        occ_s[e] = kept + tk;
        if (blockIdx.x == 0) { t.expert_count[e] = kept + tk; t.n_routed[e] = n; }
    }
    __syncthreads();
    if (want_sums && (int)blockIdx.x == ncta - 1) {
        // L = alpha * E * sum_e f_e P_e: f_e from the first choices of all tokens (before the capacity cut),
        // P_e the mean softmax value; every sum in a fixed order, so the numbers repeat bit for bit
        float *part = reinterpret_cast<float *>(selsh.hist), *term = part + 512;
        const float invT = 1.0f / (float)T;
        fixed_order_sums(p.pre.cta_psum, 0, ncta, E, part, term);
        for (int e = tid; e < E; e += nthr) {
            const float Pe = term[e] * invT, fe = (float)tot_s[e] * invT;
            p.pre.P[e] = Pe;
            p.pre.f[e] = fe;
            term[e] = fe * Pe;
        }
        __syncthreads();
        if (tid == 0) {
            float acc = 0.0f;
            for (int e = 0; e < E; ++e) acc += term[e];
            *p.pre.loss = p.pre.alpha * (float)E * acc;
        }
        __syncthreads();
    }
    if (warp == 0) {  // start of every expert's nominee list
        int carry = 0;
        for (int e0 = 0; e0 < E; e0 += 32) {
            const int e = e0 + lane;
            const int x = e < E ? nnom_s[e] : 0;
            int inc = x;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(kFull, inc, o);
                if (lane >= o) inc += y;
            }
            if (e < E) loff_s[e] = carry + inc - x;
            carry += __shfl_sync(kFull, inc, 31);
        }
        if (lane == 0) loff_s[E] = carry;
    }
    __syncthreads();
    {
        const int *wc = wcnt + warp * cols;
        int *wi = wir + warp * E;
        // The records of the next two units are fetched before the current one is worked on: when they live
        // in the workspace (long token ranges) every unit would otherwise pay an L2 round trip of its own,
        // and one unit ahead leaves too few bytes in flight (sixteen warps an SM) for the memory system.
        struct In2 { int pos[KK], sel[KK], valk, h; float frk; };
        auto fetch = [&](int j, In2 &d) {
            const int blk = w_first + j;
            if (j < nb_w && blk * 32 + lane < T) {
                const int *rb = rec_of(blk);
#pragma unroll
                for (int r = 0; r < KK; ++r)
                    if (r < K1) { d.pos[r] = rb[(K1 + r) * 32]; d.sel[r] = rb[(2 * K1 + r) * 32]; }
                d.valk = rb[k * 32];
                d.h = rb[(3 * K1) * 32];
                d.frk = soft ? p.s.fr_key[blk * 32 + lane] : 0.0f;
            }
        };
        In2 cur, nxt, nx2;
        fetch(0, cur);
        fetch(1, nxt);
        for (int j = 0; j < nb_w; ++j) {
            fetch(j + 2, nx2);
            const int blk = w_first + j;
            const int i = blk * 32 + lane;
            const bool live = i < T;
            int *rb = rec_of(blk);
            int d = 0, h = -1;
            if (live) {
#pragma unroll
                for (int r = 0; r < KK; ++r) {
                    if (r < k) {
                        const int e = cur.sel[r];
                        const int c = r * E + e;
                        const int pos = base_s[c] + pre_s[c] + wc[c] + cur.pos[r];
                        int slot = -1;
                        if (pos < C) {  // Section 3: the position in the expert's queue is below its capacity
                            slot = pos;
                            t.slot_token[(size_t)e * C + pos] = i;
                            t.slot_rank[(size_t)e * C + pos] = (int8_t)r;
                        } else {
                            ++d;
                        }
                        t.route_slot[(size_t)i * K1 + r] = slot;
                        rb[(K1 + r) * 32] = slot;
                    }
                }
                t.route_slot[(size_t)i * K1 + k] = -1;
                if (mode & RR_FR) {  // Section 4.2, stage one: nominate the (k+1)-th expert
                    int e = 0, pk = 0;
#pragma unroll
                    for (int r = 0; r < KK; ++r)
                        if (r == k) { e = cur.sel[r]; pk = cur.pos[r]; }
                    const int c = k * E + e;
                    const int q = loff_s[e] + pre_s[c] + wc[c] + pk;
                    p.s.nom_key[q] = order_key(soft ? cur.frk : __int_as_float(cur.valk));
                    p.s.nom_token[q] = i;
                }
                t.drop_count[i] = d;
                if ((mode & RR_IR) && d > 0) h = cur.h;
            }
            // Section 4.1: tokens with a dropped routing queue at their in-group expert, token order
            const unsigned m = __match_any_sync(kFull, h);
            const int rk = __popc(m & ((1u << lane) - 1u));
            const int cnt = h >= 0 ? wi[h] : 0;
            __syncwarp();
            if (h >= 0 && rk == 0) wi[h] = cnt + __popc(m);
            __syncwarp();
            if (live) rb[(3 * K1 + 2) * 32] = h >= 0 ? cnt + rk : -1;
            cur = nxt;
            nxt = nx2;
        }
    }
    __syncthreads();
    for (int e = tid; e < E; e += nthr) {
        int run = 0;
        for (int w = 0; w < nw; ++w) {
            const int x = wir[w * E + e];
            wir[w * E + e] = run;
            run += x;
        }
        p.s.ir_agg[(size_t)blockIdx.x * E8 + e] = (uint16_t)run;
    }
    if (mode & (RR_IR | RR_FR)) {
        if (!grid_barrier(p.s.sync, p.s.status, ++epoch, misc + 1, p.wait_limit_ns)) { leave_grid(p.s.sync); return; }
    }

    // ---------------------------------------------------------------- phase 3
    // What does not depend on the fill-in -- lengths and starts of the IR lists, the row space -- by the
    // threads t0 .. t0+n-1 of the block (whole warps) on barrier `bar`:
    auto ir_and_rows = [&](int t0, int n, int bar) {
        const int t = tid - t0;
        if (mode & RR_IR) column_sums(p.s.ir_agg, E8, ncta, irpre_s, irtot_s, t, n);
        sub_sync(bar, n);
        if (t < 32) {  // ir_offset and row_offset: exclusive scans over the experts
            int c_ir = 0, c_row = 0;
            for (int e0 = 0; e0 < E; e0 += 32) {
                const int e = e0 + t;
                const int x = e < E ? irtot_s[e] : 0;
                const int y = e < E ? occ_s[e] + x : 0;
                int ix = x, iy = y;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int ux = __shfl_up_sync(kFull, ix, o), uy = __shfl_up_sync(kFull, iy, o);
                    if (t >= o) { ix += ux; iy += uy; }
                }
                if (e < E) { iro_s[e] = c_ir + ix - x; row_s[e] = c_row + iy - y; }
                c_ir += __shfl_sync(kFull, ix, 31);
                c_row += __shfl_sync(kFull, iy, 31);
            }
            if (t == 0) { iro_s[E] = c_ir; row_s[E] = c_row; }
        }
        sub_sync(bar, n);
        if (blockIdx.x == 0)
            for (int e = t; e <= E; e += n) { p.t.row_offset[e] = row_s[e]; p.t.ir_offset[e] = iro_s[e]; }
    };
    bool rows_done = false;
    if (mode & RR_FR) {
        for (int e = (int)blockIdx.x; e < E; e += ncta) {
            const int n = nnom_s[e], tk = take_s[e];
            if (tk == 0) continue;
            // four warps are enough for the sums; the selection is faster the fewer keys a thread holds
            const int need = ((n + 7) / 8 + 31) & ~31;  // the fewest whole warps that hold the list, eight keys per thread
            const int nsel = nthr >= 256 ? (need > nthr - 128 ? need : nthr - 128) : need;
            if (!rows_done && nsel + 64 <= nthr) {
                // a short list: some warps select (their own barrier), the others do the IR sums and the row
                // space meanwhile, instead of one after the other
                if (tid < nsel)
                    select_best_blocked<8>(selsh, p.s.nom_key + loff_s[e], p.s.nom_token + loff_s[e], n, tk, kept_s[e], e, k, K1,
                                           C, t.route_slot, t.slot_token, t.slot_rank, tid, nsel, 1);
                else
                    ir_and_rows(nsel, nthr - nsel, 2);
                rows_done = true;
                __syncthreads();
            } else if (n <= 8 * nthr) {
                select_best_blocked<8>(selsh, p.s.nom_key + loff_s[e], p.s.nom_token + loff_s[e], n, tk, kept_s[e], e, k, K1, C,
                                       t.route_slot, t.slot_token, t.slot_rank, tid, nthr, 0);
            } else {
                select_best_long(selsh, p.s.nom_key + loff_s[e], p.s.nom_token + loff_s[e], n, tk, kept_s[e], e, k, K1, C,
                                 t.route_slot, t.slot_token, t.slot_rank);
            }
        }
    }
    if (!rows_done) {
        ir_and_rows(0, nthr, 0);
        __syncthreads();
    }
    // marks outside the live ranges (E * C + T < 2^31 is an argument rule)
    {
        // (with fill-in, the blocks that had no expert to serve take the marks while the others select)
        const int first_marker = ((mode & RR_FR) && ncta > E) ? E : 0;
        const unsigned stride = (unsigned)(ncta - first_marker) * (unsigned)nthr;
        const unsigned g0 = (int)blockIdx.x >= first_marker ? ((unsigned)blockIdx.x - first_marker) * (unsigned)nthr + tid : 0xffffffffu;
        const unsigned slots = (unsigned)E * (unsigned)C;
        for (unsigned q = g0; q < slots; q += stride) {
            const int e = (int)(q / (unsigned)C), sl = (int)(q - (unsigned)e * (unsigned)C);
            if (sl >= occ_s[e]) { t.slot_token[q] = -1; t.slot_rank[q] = -1; }
        }
        for (unsigned q = g0; q < (unsigned)T; q += stride)
            if ((int)q >= iro_s[E]) t.ir_token[q] = -1;
        for (unsigned q = g0; q < slots + (unsigned)T; q += stride)
            if (q >= (unsigned)row_s[E]) { t.row_token[q] = -1; t.row_weight[q] = 0.0f; }
    }
    if (mode & RR_FR) {
        if (!grid_barrier(p.s.sync, p.s.status, ++epoch, misc + 1, p.wait_limit_ns)) { leave_grid(p.s.sync); return; }
    }

    // ---------------------------------------------------------------- phase 4
    // This block has passed its last barrier: it says so now, and the answer (is it the last to say so?)
    // travels while phase 4 runs instead of costing a round trip at the very end.
    int left_before = -1;
    if (tid == 0) {
        __threadfence();
        left_before = atomicAdd(&p.s.sync[2], 1);
    }
    // A kernel launched as this one's dependent may be made ready now: its blocks find room as these leave and
    // wait for the whole of this grid before they touch memory.  (Signalled at the start of the kernel instead,
    // the same replayed graph ran 5 % slower on 2^20 tokens.)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    {
        const int *wi = wir + warp * E;
        struct In4 { int slot[KK], sel[KK], il, h; float val[KK], a_h; };
        auto fetch = [&](int j, In4 &d) {  // as in phase 2: two units ahead
            const int blk = w_first + j;
            if (j < nb_w && blk * 32 + lane < T) {
                const int *rb = rec_of(blk);
#pragma unroll
                for (int r = 0; r < KK; ++r) {
                    if (r < K1) {
                        d.val[r] = __int_as_float(rb[r * 32]);
                        d.sel[r] = rb[(2 * K1 + r) * 32];
                        d.slot[r] = -1;
                        if (r < k) d.slot[r] = rb[(K1 + r) * 32];
                        else if (mode & RR_FR)  // written by the block that served the expert
                            d.slot[r] = __ldcg(t.route_slot + (size_t)(blk * 32 + lane) * K1 + r);
                    }
                }
                d.il = rb[(3 * K1 + 2) * 32];
                d.h = rb[(3 * K1) * 32];
                d.a_h = __int_as_float(rb[(3 * K1 + 1) * 32]);
            }
        };
        In4 cur, nxt, nx2;
        fetch(0, cur);
        fetch(1, nxt);
        for (int j = 0; j < nb_w; ++j) {
            fetch(j + 2, nx2);
            const int blk = w_first + j;
            const int i = blk * 32 + lane;
            if (i >= T) { cur = nxt; nxt = nx2; continue; }
            int slot_r[kMaxK + 1], exp_r[kMaxK + 1];
            float val_r[kMaxK + 1];
            int drops = 0;
#pragma unroll
            for (int r = 0; r <= kMaxK; ++r) {
                slot_r[r] = -1;
                exp_r[r] = 0;
                val_r[r] = 0.0f;
                if (r < KK && r < K1) {
                    exp_r[r] = cur.sel[r < KK ? r : 0];
                    val_r[r] = cur.val[r < KK ? r : 0];
                    slot_r[r] = cur.slot[r < KK ? r : 0];
                    if (r < k) drops += slot_r[r] < 0;
                }
            }
            const int il = cur.il;
            const int h_i = cur.h;
            const float a_h = cur.a_h;
            cur = nxt;
            nxt = nx2;
            float num[kMaxK + 2];
            int row[kMaxK + 2];
            // Eq. 2 / Eq. 3 are ratios of exponentials: the reference subtracted in the exponents is the
            // largest logit among the token's LIVE routes, so the largest term is 1 and the denominator
            // cannot underflow, however far below the token's best expert its surviving routes lie.
            float m = il >= 0 ? a_h : -CUDART_INF_F;
#pragma unroll
            for (int r = 0; r <= kMaxK; ++r)
                if (slot_r[r] >= 0) m = fmaxf(m, val_r[r]);
            float den = 0.0f;
#pragma unroll
            for (int r = 0; r <= kMaxK; ++r) {
                if (r >= K1) continue;
                num[r] = 0.0f;
                row[r] = -1;
                if (slot_r[r] >= 0) {
                    num[r] = expf(val_r[r] - m);
                    den += num[r];
                    row[r] = row_s[exp_r[r]] + slot_r[r];  // the expert's rows follow slot order
                }
            }
            num[K1] = 0.0f;
            row[K1] = -1;
            int hh = -1, pos = -1;
            if (il >= 0) {
                hh = h_i;
                pos = irpre_s[hh] + wi[hh] + il;
                t.ir_token[iro_s[hh] + pos] = i;
                // Eq. 3: the IR route carries the weight of every dropped routing
                num[K1] = (float)drops * expf(a_h - m);
                den += num[K1];
                row[K1] = row_s[hh] + occ_s[hh] + pos;
            }
            t.ir_expert[i] = hh;
            t.ir_pos[i] = pos;
            const float inv_den = den > 0.0f ? 1.0f / den : 0.0f;  // one division per token
            for (int r = 0; r < K2; ++r) {
                const float w = num[r] * inv_den;
                num[r] = w;
                if (row[r] >= 0) {
                    t.row_token[row[r]] = i;
                    t.row_weight[row[r]] = w;
                }
            }
            if (K2 == 4) {  // top-2: the token's four weights and rows leave as one 16-byte store each
                *reinterpret_cast<float4 *>(t.combine_w + (size_t)i * 4) = make_float4(num[0], num[1], num[2], num[3]);
                *reinterpret_cast<int4 *>(t.token_rows + (size_t)i * 4) = make_int4(row[0], row[1], row[2], row[3]);
            } else {
                for (int r = 0; r < K2; ++r) {
                    t.combine_w[(size_t)i * K2 + r] = num[r];
                    t.token_rows[(size_t)i * K2 + r] = row[r];
                }
            }
        }
    }
    // the last block to have passed its last barrier puts the barrier words back to zero for the next call
    // (the others may still be in phase 4: they do not touch these words any more)
    if (tid == 0 && left_before == ncta - 1) {
        p.s.sync[0] = 0;
        p.s.sync[1] = 0;
        p.s.sync[2] = 0;
    }
}

struct Cfg {
    int ncta, nw, ns, bpc, bpw, nblk, tma, pitch, stage_bytes, rec_smem;
    size_t smem;
};

// Launch shape for a problem on a device with `sms` SMs.
bool choose_cfg(int T, int E, int k, int sms, bool presel, Cfg *c)
{
    const int nblk = (T + 31) / 32;
    const int max_cta = sms < kMaxRouteCtas ? sms : kMaxRouteCtas;
    int bpc = (nblk + max_cta - 1) / max_cta;
    if (bpc < 1) bpc = 1;
    int ncta = (nblk + bpc - 1) / bpc;
    if (ncta < 1) ncta = 1;
    if (bpc * 32 > 65535) return false;  // the per-block counts are 16-bit
    c->nblk = nblk;
    c->bpc = bpc;
    c->ncta = ncta;
    c->tma = (E % 32 == 0) ? 1 : 0;
    if (presel) {  // no rows are staged
        c->tma = 0;
        c->pitch = 0;
        c->stage_bytes = 1024;
    } else if (c->tma) {
        c->pitch = 0;
        c->stage_bytes = (E / 32) * 4096;
    } else {
        int pieces = (E + 3) / 4;
        if ((pieces & 1) == 0) ++pieces;  // an odd number of 16-byte pieces per row: the 32 rows of a warp spread over the banks
        c->pitch = pieces * 4;
        c->stage_bytes = (32 * c->pitch * 4 + 1023) / 1024 * 1024;
    }
    const int NF = route_rec_fields(k);
    const int cand[] = {16, 12, 8, 4, 2, 1};
    for (int nw : cand) {
        const int bpw = (bpc + nw - 1) / nw;
        const int want = c->tma ? (bpw < 2 ? bpw : (nw >= 12 ? 2 : 3)) : 1;
        for (int ns = want; ns >= (bpw > 1 && c->tma ? 2 : 1); --ns) {
            // records in shared memory when they are small; else through the workspace
            for (int rs = 1; rs >= 0; --rs) {
                const size_t rec_words = rs ? (size_t)bpc * 32 * NF : 0;
                if (rs && rec_words * 4 > 64 * 1024) continue;
                const Plan pl = make_plan(nw, ns, c->stage_bytes, E, k, (int)rec_words);
                if (pl.end + 1024 <= (size_t)kSmemBudget) {
                    c->nw = nw; c->ns = ns; c->bpw = bpw; c->rec_smem = rs; c->smem = pl.end + 1024;
                    return true;
                }
            }
        }
    }
    return false;
}

template <int KK, int kVar, bool kTma>
cudaError_t launch_kv(const CUtensorMap &map, const FusedParams &p, const Cfg &c, cudaStream_t st)
{
    cudaError_t err = cudaFuncSetAttribute(k_route_fused<KK, kVar, kTma>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
    if (err != cudaSuccess) return err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(c.ncta);
    cfg.blockDim = dim3(c.nw * 32);
    cfg.dynamicSmemBytes = c.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;  // all blocks resident together: they wait on one another
    attr[0].val.cooperative = 1;
    // the kernel may be set up while its predecessor in the stream drains (it waits for it before it touches memory)
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    static int pdl_ok = 1;  // falls back for good if the driver refuses the combination
    if (pdl_ok) {
        cfg.numAttrs = 2;
        err = cudaLaunchKernelEx(&cfg, k_route_fused<KK, kVar, kTma>, map, p);
        if (err == cudaSuccess) return err;
        (void)cudaGetLastError();
        pdl_ok = 0;
    }
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_route_fused<KK, kVar, kTma>, map, p);
}

template <int KK>
cudaError_t launch_kk(const CUtensorMap &map, const FusedParams &p, const Cfg &c, cudaStream_t st)
{
    if (p.presel) return launch_kv<KK, 2, false>(map, p, c, st);
    if ((p.mode & RR_FR_SOFTMAX) || p.pre.psum)
        return p.tma ? launch_kv<KK, 1, true>(map, p, c, st) : launch_kv<KK, 1, false>(map, p, c, st);
    return p.tma ? launch_kv<KK, 0, true>(map, p, c, st) : launch_kv<KK, 0, false>(map, p, c, st);
}

int device_sms()
{
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev] = n;
    }
    return cached[dev];
}

}  // namespace

cudaError_t launch_route_fused(const float *logits, int T, int E, int k, int C, int G, unsigned mode,
                               const rr_route_tables &t, const RouteScratch &s, cudaStream_t st,
                               const RoutePresel *pre)
{
    const int sms = device_sms();
    if (sms <= 0) return cudaErrorInvalidDevice;
    Cfg c;
    const bool presel = pre && pre->val;  // (`pre` without a selection: only the loss outputs are wanted)
    if (!choose_cfg(T, E, k, sms, presel, &c)) return cudaErrorInvalidConfiguration;
    FusedParams p;
    p.wait_limit_ns = test_wait_limit_ns() ? test_wait_limit_ns() : tc::kWaitLimitNs;
    p.presel = presel ? 1 : 0;
    p.pre = pre ? *pre : RoutePresel{};
    p.logits = logits;
    p.T = T; p.E = E; p.k = k; p.C = C; p.G = G;
    p.mode = mode;
    p.nblk = c.nblk; p.bpc = c.bpc; p.bpw = c.bpw; p.ns = c.ns;
    p.tma = c.tma; p.pitch = c.pitch; p.stage_bytes = c.stage_bytes; p.rec_smem = c.rec_smem;
    p.t = t;
    p.s = s;
    CUtensorMap map;
    memset(&map, 0, sizeof(map));
    if (c.tma && T > 0) {
        // logits [T, E] fp32 as boxes of 32 columns x 32 rows, 128-byte swizzle; rows beyond T read as zeros
        if (!tc::make_map_bytes(&map, logits, (size_t)T, (size_t)E, 4, true, 32, 128)) return cudaErrorUnknown;
    }
    const int K1 = k + 1;
    if (K1 <= 2) return launch_kk<2>(map, p, c, st);
    if (K1 <= 3) return launch_kk<3>(map, p, c, st);
    if (K1 <= 5) return launch_kk<5>(map, p, c, st);
    return launch_kk<kMaxK + 1>(map, p, c, st);
}

}  // namespace rr
