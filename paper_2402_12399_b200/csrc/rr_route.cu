// Routing kernels: top-(k+1) selection, capacity assignment, Intra-GPU
// Rectification, Fill-in Rectification, combine weights and the compact row space
// (arXiv 2402.12399, Section 3 Eq. 1-2, Section 4.1 Eq. 3, Section 4.2).
//
// Five launches per call:
//   k_topk     one pass over logits[T,E] (rows staged in shared memory by bulk copies): per
//              token the k+1 best experts by
//              (logit desc, index asc) and the best expert of its own group; per tile
//              the number of tokens per (rank, expert) and each token's position among them
//   k_scan     exclusive prefix of those counts over tiles and their totals (one block per
//              (rank, expert) column, counts stored column-major so the scan is coalesced)
//   k_assign   slot = base + prefix + local position; kept iff < capacity; nominee lists
//              for FR; per-tile ranking of IR tokens
//   k_fr_ir    one block per expert: choose the v_e best nominees (radix select on an
//              order-preserving key, ties to the lower token) and place them in token
//              order; further blocks (one per expert) scan the IR counts over tiles
//   k_finalize IR lists, combine weights, row space, padding marks
// Every decision is an exact comparison of raw fp32 logits, so the tables are unique.
#include <limits.h>
#include <math_constants.h>

#include "rr_common.cuh"
#include "rr_route_dev.cuh"
#include "rr_tc.cuh"

namespace rr {

namespace {

constexpr int kWarps = kTileTok / 32;

// ---------------------------------------------------------------------------------------
// k_topk.  One thread per token.  The warp's 32 rows of logits are brought into shared
// memory by one bulk copy (TMA, contiguous bytes) and each thread then streams over its own
// row (16-byte shared loads), keeping the best k+1 entries by insertion: no shuffles, and the
// only HBM traffic is the single read of logits[T,E].  Threads walk their rows starting at
// different columns so that the lanes of a warp hit different banks.
// KK >= k+1 is the compile-time length of the insertion list; SOFT adds the softmax value of the
// token at its (k+1)-th expert (RR_FR_SOFTMAX), a second pass over the row.
// ---------------------------------------------------------------------------------------
template <int KK, bool SOFT>
__global__ void __launch_bounds__(kTileTok)
k_topk(const float *__restrict__ logits, int T, int E, int k, int G, int chunk_tok,
       int *__restrict__ topk_expert, float *__restrict__ fr_key, RouteScratch s)
{
    extern __shared__ __align__(128) int smem[];
    const int K1 = k + 1;
    float *rows_s = reinterpret_cast<float *>(smem);                     // [chunk_tok][E]
    int *sel_s = smem + (size_t)chunk_tok * E;                           // [K1][256]
    float *val_s = reinterpret_cast<float *>(sel_s + K1 * kTileTok);     // [K1][256]
    int *pos_s = reinterpret_cast<int *>(val_s + K1 * kTileTok);         // [K1][256]
    int *h_s = pos_s + K1 * kTileTok;                                    // [256]
    float *ah_s = reinterpret_cast<float *>(h_s + kTileTok);             // [256]
    int *wcount = reinterpret_cast<int *>(ah_s + kTileTok);              // [warps][K1][E]
    __shared__ __align__(8) uint64_t bar[kWarps];
    __shared__ int abort_flag;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x;
    const TileToken tt = tile_token(s, tile, tid);
    const int tok0 = tt.i - tid;                                       // first token of the tile
    const int seg_left = s.Tseg - (tile - tt.sg * s.tps) * kTileTok;   // tokens from there to the segment's end
    const int cols = K1 * E;
    if (tid == 0) {
        for (int w = 0; w < kWarps; ++w) tc::mbar_init(&bar[w], 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int c = tid; c < kWarps * cols; c += kTileTok) wcount[c] = 0;
    __syncthreads();

    const int tpg = T / G > 0 ? T / G : 1, epg = E / G;
    const int i = tt.i;
    const bool live = tt.live;
    bool bad = false, rows_ok = true;

    for (int c0 = 0; c0 < kTileTok; c0 += chunk_tok) {
        if (c0) {  // the previous chunk's rows are no longer needed; the next bulk copy writes over them
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // reads before the async-proxy write
            __syncthreads();
        }
        const int w_first = c0 >> 5;
        if (warp >= w_first && warp < ((c0 + chunk_tok) >> 5)) {
            const int first = tok0 + warp * 32;  // first token of this warp
            const int ntok = min(32, seg_left - warp * 32);
            float *dst = rows_s + (size_t)(warp - w_first) * 32 * E;
            if (ntok > 0) {
                const float *src = logits + (size_t)first * E;
                const unsigned bytes = (unsigned)ntok * E * 4u;
                if ((bytes & 15u) == 0 && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
                    if (lane == 0) {
                        tc::mbar_expect_tx(&bar[warp], bytes);
                        asm volatile(
                            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                            ::"r"(tc::smem_u32(dst)), "l"(src), "r"(bytes), "r"(tc::smem_u32(&bar[warp]))
                            : "memory");
                    }
                    // a wait that ran out leaves the rows unfilled: they are not read (below)
                    rows_ok = tc::warp_wait(&bar[warp], 0, &abort_flag, s.status);
                } else {  // ragged tail or segment start: byte count or address not a multiple of 16
                    for (int q = lane; q < ntok * E; q += 32) dst[q] = src[q];
                    __syncwarp();
                }
            }
            // Two insertion lists: A for the columns from this lane's start column to the end of
            // the row, B for the columns before it (visited afterwards, both in ascending order).
            // Inside a list a later column never displaces an equal earlier one (strict >), and
            // every column of B is lower than every column of A, so merging A into B with strict >
            // yields exactly the order (logit desc, index asc) of Eq. 1 without index compares.
            float av[KK], bv[KK], gv = -CUDART_INF_F, chk = 0.0f;
            int aj[KK], bj[KK], gj = INT_MAX;
#pragma unroll
            for (int r = 0; r < KK; ++r) { av[r] = empty_place(); bv[r] = empty_place(); aj[r] = bj[r] = INT_MAX; }
            const int grp = live ? i / tpg : 0;
            const int lo = grp * epg, hi = lo + epg;
            if (live && rows_ok) {
                const float *row = dst + (size_t)lane * E;
                if ((E & 3) == 0 && E >= 8 * KK) {
                    // Two levels.  First the KK best groups of four columns by (group maximum
                    // desc, group index asc), with the same two-list walk; every one of the k+1
                    // best columns lies in one of them (a column outside has, in each chosen
                    // group, that group's maximum ahead of it: larger, or equal at a lower
                    // index).  Then only those groups' columns go through the full insertion,
                    // in ascending column order.
                    const float4 *row4 = reinterpret_cast<const float4 *>(row);
                    const int ng = E >> 2, g0 = lane % ng;
                    for (int g = g0; g < ng; ++g) {
                        const float4 f = row4[g];
                        chk = fmaf(f.x, 0.0f, chk); chk = fmaf(f.y, 0.0f, chk);
                        chk = fmaf(f.z, 0.0f, chk); chk = fmaf(f.w, 0.0f, chk);
                        insert_strict<KK>(fmaxf(fmaxf(f.x, f.y), fmaxf(f.z, f.w)), g, av, aj);
                    }
                    for (int g = 0; g < g0; ++g) {
                        const float4 f = row4[g];
                        chk = fmaf(f.x, 0.0f, chk); chk = fmaf(f.y, 0.0f, chk);
                        chk = fmaf(f.z, 0.0f, chk); chk = fmaf(f.w, 0.0f, chk);
                        insert_strict<KK>(fmaxf(fmaxf(f.x, f.y), fmaxf(f.z, f.w)), g, bv, bj);
                    }
#pragma unroll
                    for (int r = 0; r < KK; ++r) insert_strict<KK>(av[r], aj[r], bv, bj);
                    int gs[KK];  // the chosen groups, ascending
                    // A row of NaNs or of -inf leaves places empty (nothing exceeds -inf, NaN compares
                    // false): such a place takes a group that is certainly there (E >= 8 KK) and not yet
                    // chosen, so every index read or written below names a column of the row.  The row is
                    // reported as non-finite by `chk` in any case.
#pragma unroll
                    for (int r = 0; r < KK; ++r) {
                        if (bj[r] == INT_MAX) {
                            int cand = 0;
#pragma unroll
                            for (int t = 0; t < KK; ++t) {  // smallest group index no earlier place holds
                                bool used = false;
#pragma unroll
                                for (int q = 0; q < KK; ++q) used |= (q < r && bj[q] == cand);
                                cand += used ? 1 : 0;
                            }
                            bj[r] = cand;
                        }
                        gs[r] = bj[r];
                    }
#pragma unroll
                    for (int a = 0; a < KK - 1; ++a)
#pragma unroll
                        for (int b = 0; b < KK - 1 - a; ++b) {
                            const int lo_g = min(gs[b], gs[b + 1]), hi_g = max(gs[b], gs[b + 1]);
                            gs[b] = lo_g;
                            gs[b + 1] = hi_g;
                        }
                    float cv[KK];
                    int cj[KK];
#pragma unroll
                    for (int r = 0; r < KK; ++r) { cv[r] = empty_place(); cj[r] = INT_MAX; }
#pragma unroll
                    for (int r = 0; r < KK; ++r) {  // E >= 8 KK: every entry of gs names a group
                        const float4 f = row4[gs[r]];
                        const int j = 4 * gs[r];
                        insert_strict<KK>(f.x, j, cv, cj); insert_strict<KK>(f.y, j + 1, cv, cj);
                        insert_strict<KK>(f.z, j + 2, cv, cj); insert_strict<KK>(f.w, j + 3, cv, cj);
                    }
#pragma unroll
                    for (int r = 0; r < KK; ++r) { bv[r] = cv[r]; bj[r] = cj[r]; av[r] = empty_place(); aj[r] = INT_MAX; }
                } else if ((E & 3) == 0) {
                    const float4 *row4 = reinterpret_cast<const float4 *>(row);
                    const int ng = E >> 2, g0 = lane % ng;
                    for (int g = g0; g < ng; ++g) {
                        const float4 f = row4[g];
                        chk = fmaf(f.x, 0.0f, chk); chk = fmaf(f.y, 0.0f, chk);
                        chk = fmaf(f.z, 0.0f, chk); chk = fmaf(f.w, 0.0f, chk);
                        insert_strict<KK>(f.x, 4 * g, av, aj); insert_strict<KK>(f.y, 4 * g + 1, av, aj);
                        insert_strict<KK>(f.z, 4 * g + 2, av, aj); insert_strict<KK>(f.w, 4 * g + 3, av, aj);
                    }
                    for (int g = 0; g < g0; ++g) {
                        const float4 f = row4[g];
                        chk = fmaf(f.x, 0.0f, chk); chk = fmaf(f.y, 0.0f, chk);
                        chk = fmaf(f.z, 0.0f, chk); chk = fmaf(f.w, 0.0f, chk);
                        insert_strict<KK>(f.x, 4 * g, bv, bj); insert_strict<KK>(f.y, 4 * g + 1, bv, bj);
                        insert_strict<KK>(f.z, 4 * g + 2, bv, bj); insert_strict<KK>(f.w, 4 * g + 3, bv, bj);
                    }
                } else {
                    const int j0 = lane % E;
                    for (int j = j0; j < E; ++j) { const float x = row[j]; chk = fmaf(x, 0.0f, chk); insert_strict<KK>(x, j, av, aj); }
                    for (int j = 0; j < j0; ++j) { const float x = row[j]; chk = fmaf(x, 0.0f, chk); insert_strict<KK>(x, j, bv, bj); }
                }
#pragma unroll
                for (int r = 0; r < KK; ++r) insert_strict<KK>(av[r], aj[r], bv, bj);
                // Section 4.1: best expert among those of the token's own group (same two-part
                // walk, so that lanes of one group do not all read the same bank)
                {
                    const int s0 = lane % epg;
                    float ga = -CUDART_INF_F, gb = -CUDART_INF_F;
                    int gaj = INT_MAX, gbj = INT_MAX;
                    for (int j = lo + s0; j < hi; ++j) { const float x = row[j]; if (x > ga) { ga = x; gaj = j; } }
                    for (int j = lo; j < lo + s0; ++j) { const float x = row[j]; if (x > gb) { gb = x; gbj = j; } }
                    if (ga > gb) { gv = ga; gj = gaj; } else { gv = gb; gj = gbj; }
                }
            }
            if (live && (chk != 0.0f || !rows_ok)) {
                // a NaN or an infinity (x * 0 is NaN for both), or rows that never arrived: undefined
                // tables, but every index written below must still name an expert
                bad = bad || chk != 0.0f;
#pragma unroll
                for (int r = 0; r < KK; ++r)
                    if (bj[r] == INT_MAX && r < E) { bj[r] = r; bv[r] = 0.0f; }
                if (gj == INT_MAX) { gj = lo; gv = 0.0f; }
            }
#pragma unroll
            for (int r = 0; r < KK; ++r) {
                if (r < K1) {
                    sel_s[r * kTileTok + tid] = (live && bj[r] != INT_MAX) ? bj[r] : -1;
                    val_s[r * kTileTok + tid] = bv[r];
                }
            }
            h_s[tid] = (live && gj != INT_MAX) ? gj : lo;
            ah_s[tid] = gv;
            if (SOFT && live && rows_ok) {
                // Softmax value of the token at its (k+1)-th expert, by the fixed recipe.  The row is no
                // longer needed as logits: e_j = exp_fixed(a_ij - m) replaces it in place (walk from a
                // lane-dependent column: bank spread).  Z adds the e_j in index order; lane l runs l
                // steps behind lane 0 so that the lanes of a warp, whose rows start a multiple of 32
                // words apart when E is one, read different banks.
                float *rw = dst + (size_t)lane * E;
                const float mx = val_s[tid];  // the token's largest logit
                int j = lane % E;
                for (int q = 0; q < E; ++q) {
                    rw[j] = exp_fixed(__fsub_rn(rw[j], mx));
                    if (++j == E) j = 0;
                }
                float Z = 0.0f;
                for (int q = 0; q < E + 31; ++q) {
                    const int c = q - lane;
                    if (c >= 0 && c < E) Z = __fadd_rn(Z, rw[c]);
                }
                const int nj = sel_s[k * kTileTok + tid];  // the nominated expert (FR needs k < E, so it exists)
                fr_key[i] = __fdiv_rn(rw[nj >= 0 ? nj : 0], Z);
            }
        }
    }
    if (bad) latch_status(s.status, RR_ERR_NONFINITE);
    __syncthreads();

    if (live) {
        for (int r = 0; r < K1; ++r) {
            topk_expert[(size_t)i * K1 + r] = sel_s[r * kTileTok + tid];
            s.val[(size_t)i * K1 + r] = val_s[r * kTileTok + tid];
        }
        s.h[i] = h_s[tid];
        s.a_h[i] = ah_s[tid];
    }
    // position of the token among the tile's tokens with the same (rank, expert)
    for (int r = 0; r < K1; ++r) {
        const int e = live ? sel_s[r * kTileTok + tid] : -1;
        const unsigned m = __match_any_sync(kFull, e);
        const int rk = __popc(m & ((1u << lane) - 1u));
        pos_s[r * kTileTok + tid] = rk;
        if (e >= 0 && rk == 0) wcount[(warp * K1 + r) * E + e] = __popc(m);
    }
    __syncthreads();
    for (int c = tid; c < cols; c += kTileTok) {
        int run = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const int t = wcount[w * cols + c];
            wcount[w * cols + c] = run;
            run += t;
        }
        s.hist[(size_t)c * s.tiles + tile] = run;
    }
    __syncthreads();
    if (live) {
        for (int r = 0; r < K1; ++r) {
            const int e = sel_s[r * kTileTok + tid];
            s.pos_local[(size_t)i * K1 + r] = e >= 0 ? wcount[(warp * K1 + r) * E + e] + pos_s[r * kTileTok + tid] : 0;
        }
    }
    if (abort_flag) __nanosleep(2000000);  // a wait gave up: let copies still in flight land before the block's memory is released
}

// ---------------------------------------------------------------------------------------
// k_scan: exclusive prefix over tiles of every column of per-tile counts (column-major:
// hist[c][tile]), in place, and its total.
// ---------------------------------------------------------------------------------------
// One block per (segment, column): the prefix restarts at every capacity segment.  256 tiles per
// step (one per thread), the carry runs from step to step.
__global__ void __launch_bounds__(256)
k_scan(int cols, RouteScratch s)
{
    __shared__ int red[33];
    const int sg = blockIdx.x / cols, c = blockIdx.x - sg * cols;
    int *col = s.hist + (size_t)c * s.tiles + (size_t)sg * s.tps;
    int carry = 0;
    for (int t0 = 0; t0 < s.tps; t0 += 256) {
        const int t = t0 + threadIdx.x;
        const int x = t < s.tps ? col[t] : 0;
        int total;
        const int before = block_excl_scan(x, red, &total);
        if (t < s.tps) col[t] = carry + before;
        carry += total;
    }
    if (threadIdx.x == 0) s.totals[(size_t)sg * cols + c] = carry;
}

// Per-expert quantities every later kernel derives from the totals (E <= 256 values each):
// base[r][e] = slots taken at e by ranks below r, n_e, offsets of the nominee lists.
struct ExpertBases {
    int base[(kMaxK + 1) * kMaxE];
    int list_off[(kMaxK + 1) * (kMaxE + 1)];  // [r][e]: start of the (rank r, expert e) list inside rank r's T entries
    int n_routed[kMaxE];
};

// `first_list` = lowest rank whose candidate lists are needed (k: FR nominees only; 0: every rank,
// for score-priority dropping; k + 1: none).  Every token has one r-th choice, so the lists of rank r
// hold T entries in all and start at r * T in the list arrays.
__device__ __forceinline__ void compute_bases(ExpertBases *b, const int *totals, int E, int k, int first_list)
{
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        int n = 0;
        for (int r = 0; r < k; ++r) { b->base[r * E + e] = n; n += totals[r * E + e]; }
        b->n_routed[e] = n;
    }
    // a warp per rank: exclusive scan of the rank's counts over the experts
    for (int r = first_list + (threadIdx.x >> 5); r <= k; r += blockDim.x >> 5) {
        const int lane = threadIdx.x & 31;
        int carry = 0;
        for (int e0 = 0; e0 < E; e0 += 32) {
            const int e = e0 + lane;
            const int x = e < E ? totals[r * E + e] : 0;
            int inc = x;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(kFull, inc, o);
                if (lane >= o) inc += y;
            }
            if (e < E) b->list_off[r * (kMaxE + 1) + e] = carry + inc - x;
            carry += __shfl_sync(kFull, inc, 31);
        }
        if (lane == 0) b->list_off[r * (kMaxE + 1) + E] = carry;
    }
    __syncthreads();
}

// Section 4.1: tokens with a dropped routing queue at their in-group expert, token order.  `key` is
// that expert or -1; writes the tile's count per expert and the token's position among the tile's.
__device__ __forceinline__ void ir_tile_rank(int key, bool live, int i, int E, int tile, int *wcount, const RouteScratch &s)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned m = __match_any_sync(kFull, key);
    const int rk = __popc(m & ((1u << lane) - 1u));
    if (key >= 0 && rk == 0) wcount[warp * E + key] = __popc(m);
    __syncthreads();
    for (int e = tid; e < E; e += kTileTok) {
        int run = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const int t = wcount[w * E + e];
            wcount[w * E + e] = run;
            run += t;
        }
        s.ir_hist[(size_t)e * s.tiles + tile] = run;
    }
    __syncthreads();
    if (live) s.ir_local[i] = key >= 0 ? wcount[warp * E + key] + rk : -1;
}

// ---------------------------------------------------------------------------------------
// k_assign: one thread per token.  Section 3: a routing keeps its slot iff its position
// in the expert's queue (lower ranks first, token order inside a rank) is below capacity.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTileTok)
k_assign(int T, int E, int k, int C, unsigned mode, const int *__restrict__ topk_expert,
         int *__restrict__ route_slot, int *__restrict__ slot_token, int8_t *__restrict__ slot_rank,
         int *__restrict__ drop_count, RouteScratch s)
{
    extern __shared__ int smem[];
    int *wcount = smem;  // [warps][E]
    __shared__ ExpertBases eb;
    const int K1 = k + 1;
    const int tid = threadIdx.x;
    const int tile = blockIdx.x;
    const TileToken tt = tile_token(s, tile, tid);
    const int i = tt.i, sg = tt.sg;
    const bool live = tt.live;
    const int Cs = C / s.segs, slot0 = sg * Cs;       // the segment's share of every expert's slots
    const size_t seg_list = (size_t)sg * s.Tseg;      // its share of every rank's candidate lists
    for (int c = tid; c < kWarps * E; c += kTileTok) wcount[c] = 0;
    const bool by_score = (mode & RR_SCORE) != 0;
    compute_bases(&eb, s.totals + (size_t)sg * K1 * E, E, k, by_score ? 0 : ((mode & RR_FR) ? k : k + 1));
    if (tile == sg * s.tps)  // the segment's first tile
        for (int e = tid; e < E; e += kTileTok) {
            s.seg_n[sg * E + e] = eb.n_routed[e];
            s.seg_occ[sg * E + e] = eb.n_routed[e] < Cs ? eb.n_routed[e] : Cs;   // kept; the fill-in pass adds its slots
        }

    if (by_score) {
        // who stays is decided per (rank, expert) by k_select_score: hand it every routing as an
        // entry (key, token) of that pair's list, in token order
        if (live) {
            const int last = (mode & RR_FR) ? k : k - 1;
            for (int r = 0; r <= k; ++r) {
                route_slot[(size_t)i * K1 + r] = -1;
                if (r > last) continue;
                const int e = topk_expert[(size_t)i * K1 + r];
                const size_t p = (size_t)r * T + seg_list + eb.list_off[r * (kMaxE + 1) + e] +
                                 s.hist[(size_t)(r * E + e) * s.tiles + tile] + s.pos_local[(size_t)i * K1 + r];
                s.nom_key[p] = order_key((r == k && (mode & RR_FR_SOFTMAX)) ? s.fr_key[i] : s.val[(size_t)i * K1 + r]);
                s.nom_token[p] = i;
            }
        }
        return;
    }

    int d = 0;
    if (live) {
        for (int r = 0; r < k; ++r) {
            const int e = topk_expert[(size_t)i * K1 + r];
            const int p = eb.base[r * E + e] + s.hist[(size_t)(r * E + e) * s.tiles + tile] +
                          s.pos_local[(size_t)i * K1 + r];
            if (p < Cs) {
                route_slot[(size_t)i * K1 + r] = slot0 + p;
                slot_token[(size_t)e * C + slot0 + p] = i;
                slot_rank[(size_t)e * C + slot0 + p] = (int8_t)r;
            } else {
                route_slot[(size_t)i * K1 + r] = -1;
                ++d;
            }
        }
        route_slot[(size_t)i * K1 + k] = -1;
        if (mode & RR_FR) {  // Section 4.2, stage one: nominate the (k+1)-th expert
            const int e = topk_expert[(size_t)i * K1 + k];
            const size_t p = seg_list + eb.list_off[k * (kMaxE + 1) + e] + s.hist[(size_t)(k * E + e) * s.tiles + tile] +
                             s.pos_local[(size_t)i * K1 + k];
            s.nom_key[p] = order_key((mode & RR_FR_SOFTMAX) ? s.fr_key[i] : s.val[(size_t)i * K1 + k]);
            s.nom_token[p] = i;
        }
        drop_count[i] = d;
    }
    const int key = (live && (mode & RR_IR) && d > 0) ? s.h[i] : -1;
    __syncthreads();
    ir_tile_rank(key, live, i, E, tile, wcount, s);
}

// Score-priority dropping, after k_select_score: the dropped routings of a token are those that got no
// slot; then the per-tile ranking of the IR tokens as in k_assign.
__global__ void __launch_bounds__(kTileTok)
k_ir_rank(int T, int E, int k, unsigned mode, const int *__restrict__ route_slot, int *__restrict__ drop_count,
          RouteScratch s)
{
    extern __shared__ int smem[];
    int *wcount = smem;  // [warps][E]
    const int tid = threadIdx.x, K1 = k + 1;
    const int tile = blockIdx.x;
    const TileToken tt = tile_token(s, tile, tid);
    const int i = tt.i;
    const bool live = tt.live;
    for (int c = tid; c < kWarps * E; c += kTileTok) wcount[c] = 0;
    int d = 0;
    if (live) {
        for (int r = 0; r < k; ++r) d += route_slot[(size_t)i * K1 + r] < 0;
        drop_count[i] = d;
    }
    const int key = (live && (mode & RR_IR) && d > 0) ? s.h[i] : -1;
    __syncthreads();
    ir_tile_rank(key, live, i, E, tile, wcount, s);
}


// start of expert e's list among rank r's entries = candidates of all lower experts (one warp)
__device__ __forceinline__ int list_start(const int *__restrict__ totals, int r, int E, int e)
{
    int acc = 0;
    for (int j = threadIdx.x & 31; j < e; j += 32) acc += totals[r * E + j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(kFull, acc, o);
    return acc;
}

// ---------------------------------------------------------------------------------------
// k_fr_ir: blocks 0..E-1 run Fill-in Rectification for one expert each (Section 4.2,
// stage two); block E turns the per-tile IR counts into prefixes and list offsets.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
k_fr_ir(int E, int k, int C, unsigned mode, int *__restrict__ route_slot, int *__restrict__ slot_token,
        int8_t *__restrict__ slot_rank, RouteScratch s)
{
    __shared__ SelectShared sh;
    __shared__ int sh_off, sh_n;
    const int tid = threadIdx.x, K1 = k + 1;

    if ((int)blockIdx.x >= E * s.segs) {  // IR counts: one block per expert (IR lists know no segments)
        const int e = blockIdx.x - E * s.segs;
        int *col = s.ir_hist + (size_t)e * s.tiles;
        int carry = 0;
        for (int t0 = 0; t0 < s.tiles; t0 += blockDim.x) {
            const int t = t0 + tid;
            const int x = t < s.tiles ? col[t] : 0;
            int total;
            const int before = block_excl_scan(x, sh.red, &total);
            if (t < s.tiles) col[t] = carry + before;
            carry += total;
        }
        if (tid == 0) s.ir_totals[e] = carry;
        return;
    }
    if (!(mode & RR_FR)) return;

    // one block per (segment, expert): the segment's padding slots go to the segment's nominees
    const int sg = blockIdx.x / E, e = blockIdx.x - sg * E;
    const int *totals = s.totals + (size_t)sg * K1 * E;
    if (tid < 32) {
        const int off = list_start(totals, k, E, e);
        if (tid == 0) { sh_off = off; sh_n = totals[k * E + e]; }
    }
    __syncthreads();
    const int n = sh_n;
    const int Cs = C / s.segs;
    const int n_top = s.seg_n[sg * E + e];
    const int kept = n_top < Cs ? n_top : Cs;
    const int v = Cs - kept;              // padding slots of this expert in this segment
    const int take = n < v ? n : v;
    if (take == 0) return;
    if (tid == 0) s.seg_occ[sg * E + e] = kept + take;
    const size_t at = (size_t)sg * s.Tseg + sh_off;
    if (n > 4 * (int)blockDim.x)
        select_best_long(sh, s.nom_key + at, s.nom_token + at, n, take, sg * Cs + kept, e, k, K1, C, route_slot,
                         slot_token, slot_rank);
    else
        select_best(sh, s.nom_key + at, s.nom_token + at, n, take, sg * Cs + kept, e, k, K1, C, route_slot, slot_token,
                    slot_rank);
}

// ---------------------------------------------------------------------------------------
// k_select_score: score-priority dropping (the wording of Section 3: a full expert drops the tokens
// with the lowest routing scores).  One block per expert serves rank after rank: the r-th choices
// addressed to it compete for what the lower ranks left of its capacity; with FR the nominees follow
// as one more rank.  The lists were written by k_assign, rank r's at r * T.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024, 1)
k_select_score(int T, int E, int k, int C, unsigned mode, int *__restrict__ route_slot, int *__restrict__ slot_token,
               int8_t *__restrict__ slot_rank, RouteScratch s)
{
    __shared__ SelectShared sh;
    __shared__ int sh_off;
    const int tid = threadIdx.x, K1 = k + 1;
    const int sg = blockIdx.x / E, e = blockIdx.x - sg * E;  // one block per (segment, expert)
    const int *totals = s.totals + (size_t)sg * K1 * E;
    const int Cs = C / s.segs;
    const int last = (mode & RR_FR) ? k : k - 1;
    int used = 0;
    for (int r = 0; r <= last; ++r) {
        __syncthreads();  // the previous rank is done with `sh` and sh_off
        if (tid < 32) {
            const int off = list_start(totals, r, E, e);
            if (tid == 0) sh_off = off;
        }
        __syncthreads();
        const int n = totals[r * E + e];
        const int left = Cs - used;
        const int take = n < left ? n : left;
        if (take > 0) {
            const size_t at = (size_t)r * T + (size_t)sg * s.Tseg + sh_off;
            if (n > 4 * (int)blockDim.x)
                select_best_long(sh, s.nom_key + at, s.nom_token + at, n, take, sg * Cs + used, e, r, K1, C, route_slot,
                                 slot_token, slot_rank);
            else
                select_best(sh, s.nom_key + at, s.nom_token + at, n, take, sg * Cs + used, e, r, K1, C, route_slot,
                            slot_token, slot_rank);
        }
        used += take;
    }
    if (tid == 0) s.seg_occ[sg * E + e] = used;
}

// ---------------------------------------------------------------------------------------
// k_finalize: IR lists, combine weights (Eq. 2 / Eq. 3), row space, padding marks.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTileTok)
k_finalize(int T, int E, int k, int C, rr_route_tables t, RouteScratch s)
{
    __shared__ int cnt_s[kMaxE];   // occupied slots of the expert over all segments
    __shared__ int segb_s[kMaxE];  // of those, the ones in segments below this tile's
    __shared__ int iro_s[kMaxE + 1];
    __shared__ int row_s[kMaxE + 1];
    const int K1 = k + 1, K2 = k + 2;
    const int tid = threadIdx.x, tile = blockIdx.x;
    const TileToken tt = tile_token(s, tile, tid);
    const int i = tt.i;
    const int Cs = C / s.segs;
    // the token's own records first: these loads do not depend on the scans below and overlap them
    int slot_r[kMaxK + 1], exp_r[kMaxK + 1];
    float val_r[kMaxK + 1];
    int il = -1, h_i = 0, drops = 0, ir_before = 0;
    float a_h = 0.0f;
    // (loops of constant length, fully unrolled: the small arrays stay in registers)
#pragma unroll
    for (int r = 0; r <= kMaxK; ++r) {
        slot_r[r] = -1;
        exp_r[r] = 0;
        val_r[r] = 0.0f;
        if (tt.live && r < K1) {
            slot_r[r] = t.route_slot[(size_t)i * K1 + r];
            exp_r[r] = t.topk_expert[(size_t)i * K1 + r];
            val_r[r] = s.val[(size_t)i * K1 + r];
        }
    }
    if (tt.live) {
        il = s.ir_local[i];
        h_i = s.h[i];
        a_h = s.a_h[i];
        drops = t.drop_count[i];
        if (il >= 0) ir_before = s.ir_hist[(size_t)h_i * s.tiles + tile];
    }
    for (int e = tid; e < E; e += kTileTok) {
        int occ = 0, below = 0, n = 0;
        for (int g = 0; g < s.segs; ++g) {
            const int o = s.seg_occ[g * E + e];
            if (g < tt.sg) below += o;
            occ += o;
            n += s.seg_n[g * E + e];
        }
        cnt_s[e] = occ;
        segb_s[e] = below;
        if (tile == 0) { t.expert_count[e] = occ; t.n_routed[e] = n; }
    }
    __syncthreads();
    if (tid < 32) {  // ir_offset and row_offset: exclusive scans over experts by one warp
        int c_ir = 0, c_row = 0;
        for (int e0 = 0; e0 < E; e0 += 32) {
            const int e = e0 + tid;
            const int x = e < E ? s.ir_totals[e] : 0;
            const int y = e < E ? cnt_s[e] + x : 0;
            int ix = x, iy = y;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int ux = __shfl_up_sync(kFull, ix, o), uy = __shfl_up_sync(kFull, iy, o);
                if (tid >= o) { ix += ux; iy += uy; }
            }
            if (e < E) { iro_s[e] = c_ir + ix - x; row_s[e] = c_row + iy - y; }
            c_ir += __shfl_sync(kFull, ix, 31);
            c_row += __shfl_sync(kFull, iy, 31);
        }
        if (tid == 0) { iro_s[E] = c_ir; row_s[E] = c_row; }
    }
    __syncthreads();
    if (tile == 0)
        for (int e = tid; e <= E; e += kTileTok) { t.row_offset[e] = row_s[e]; t.ir_offset[e] = iro_s[e]; }

    if (tt.live) {
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
                // the expert's rows follow slot order: the lower segments' occupied slots come first
                const int e = exp_r[r];
                row[r] = row_s[e] + segb_s[e] + (slot_r[r] - tt.sg * Cs);
            }
        }
        num[K1] = 0.0f;
        row[K1] = -1;
        int hh = -1, pos = -1;
        if (il >= 0) {
            hh = h_i;
            pos = ir_before + il;
            t.ir_token[iro_s[hh] + pos] = i;
            // Eq. 3: the IR route carries the weight of every dropped routing
            num[K1] = (float)drops * expf(a_h - m);
            den += num[K1];
            row[K1] = row_s[hh] + cnt_s[hh] + pos;
        }
        t.ir_expert[i] = hh;
        t.ir_pos[i] = pos;
        const float inv_den = den > 0.0f ? 1.0f / den : 0.0f;  // as the one-kernel path: one division per token
        for (int r = 0; r < K2; ++r) {
            const float w = num[r] * inv_den;
            t.combine_w[(size_t)i * K2 + r] = w;
            t.token_rows[(size_t)i * K2 + r] = row[r];
            if (row[r] >= 0) {
                t.row_token[row[r]] = i;
                t.row_weight[row[r]] = w;
            }
        }
    }

    // marks outside the live ranges
    // (E * C + T < 2^31 is an argument rule, so 32-bit indices and a 32-bit division do)
    const unsigned stride = gridDim.x * kTileTok, g0 = blockIdx.x * kTileTok + tid;
    const unsigned slots = (unsigned)E * (unsigned)C;
    for (unsigned q = g0; q < slots; q += stride) {
        const int e = (int)(q / (unsigned)C), sl = (int)(q - (unsigned)e * (unsigned)C);
        const int g = s.segs == 1 ? 0 : sl / Cs;
        const int occ = s.segs == 1 ? cnt_s[e] : s.seg_occ[g * E + e];
        if (sl - g * Cs >= occ) { t.slot_token[q] = -1; t.slot_rank[q] = -1; }
    }
    for (unsigned q = g0; q < (unsigned)T; q += stride)
        if ((int)q >= iro_s[E]) t.ir_token[q] = -1;
    for (unsigned q = g0; q < slots + (unsigned)T; q += stride)
        if (q >= (unsigned)row_s[E]) { t.row_token[q] = -1; t.row_weight[q] = 0.0f; }
}

// Tokens whose rows are staged in shared memory at a time: at most 64 KB, a multiple of 32.
int topk_chunk_tokens(int E)
{
    int c = (16384 / E) & ~31;
    return c > kTileTok ? kTileTok : (c < 32 ? 32 : c);
}

template <int KK, bool SOFT>
cudaError_t launch_topk(const float *logits, int T, int E, int k, int G, int *topk_expert, float *fr_key,
                        const RouteScratch &s, cudaStream_t st)
{
    const int K1 = k + 1;
    const int chunk = topk_chunk_tokens(E);
    const size_t smem = ((size_t)chunk * E + (size_t)3 * K1 * kTileTok + 2 * kTileTok + (size_t)kWarps * K1 * E) * 4;
    cudaError_t err = cudaFuncSetAttribute(k_topk<KK, SOFT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    k_topk<KK, SOFT><<<s.tiles, kTileTok, smem, st>>>(logits, T, E, k, G, chunk, topk_expert, fr_key, s);
    return cudaGetLastError();
}

}  // namespace

size_t route_scratch_layout(void *ws, int T, int E, int k, RouteScratch *s, unsigned mode, int G)
{
    const int K1 = k + 1;
    const size_t Tn = T > 0 ? T : 1;
    Carver c(ws);
    Header *hdr = c.take<Header>(1);
    *s = RouteScratch{};
    s->status = hdr ? &hdr->status : nullptr;
    s->sync = hdr ? hdr->sync : nullptr;
    s->segs = 1;
    s->Tseg = T;
    if (route_is_fused(mode, T)) {
        s->fused = 1;
        const size_t blocks = (Tn + 31) / 32;
        s->rec = c.take<int>(blocks * 32 * route_rec_fields(k));
        s->agg = c.take<uint16_t>((size_t)((K1 * E + 7) & ~7) * kMaxRouteCtas);
        s->ir_agg = c.take<uint16_t>((size_t)((E + 7) & ~7) * kMaxRouteCtas);
        s->nom_key = c.take<uint32_t>((mode & RR_FR) ? Tn : 0);
        s->nom_token = c.take<int>((mode & RR_FR) ? Tn : 0);
        s->fr_key = c.take<float>((mode & RR_FR_SOFTMAX) ? Tn : 0);
        return align_up(c.off, 256);
    }
    const int segs = (mode & RR_LOCAL_CAP) ? G : 1;
    const int Tseg = T / segs;
    const int tps = Tseg > 0 ? (Tseg + kTileTok - 1) / kTileTok : 1;
    const int tiles = segs * tps;
    s->val = c.take<float>(Tn * K1);
    s->h = c.take<int>(Tn);
    s->a_h = c.take<float>(Tn);
    s->pos_local = c.take<int>(Tn * K1);
    s->hist = c.take<int>((size_t)tiles * K1 * E);
    s->totals = c.take<int>((size_t)segs * K1 * E);
    const size_t lists = (mode & RR_SCORE) ? Tn * K1 : Tn;  // every rank's candidates, or the nominees only
    s->nom_key = c.take<uint32_t>(lists);
    s->nom_token = c.take<int>(lists);
    s->ir_local = c.take<int>(Tn);
    s->ir_hist = c.take<int>((size_t)tiles * E);
    s->ir_totals = c.take<int>(E);
    s->fr_key = c.take<float>((mode & RR_FR_SOFTMAX) ? Tn : 0);
    s->seg_n = c.take<int>((size_t)segs * E);
    s->seg_occ = c.take<int>((size_t)segs * E);
    s->tiles = tiles;
    s->segs = segs;
    s->tps = tps;
    s->Tseg = Tseg;
    return align_up(c.off, 256);
}

cudaError_t launch_route(const float *logits, int T, int E, int k, int C, int G, unsigned mode,
                         const rr_route_tables &t, const RouteScratch &s, cudaStream_t st)
{
    if (s.fused) return launch_route_fused(logits, T, E, k, C, G, mode, t, s, st);
    cudaError_t err;
    const int K1 = k + 1;
    if (mode & RR_FR_SOFTMAX) {
        if (K1 <= 2) err = launch_topk<2, true>(logits, T, E, k, G, t.topk_expert, s.fr_key, s, st);
        else if (K1 <= 3) err = launch_topk<3, true>(logits, T, E, k, G, t.topk_expert, s.fr_key, s, st);
        else if (K1 <= 5) err = launch_topk<5, true>(logits, T, E, k, G, t.topk_expert, s.fr_key, s, st);
        else err = launch_topk<kMaxK + 1, true>(logits, T, E, k, G, t.topk_expert, s.fr_key, s, st);
    } else {
        if (K1 <= 2) err = launch_topk<2, false>(logits, T, E, k, G, t.topk_expert, nullptr, s, st);
        else if (K1 <= 3) err = launch_topk<3, false>(logits, T, E, k, G, t.topk_expert, nullptr, s, st);
        else if (K1 <= 5) err = launch_topk<5, false>(logits, T, E, k, G, t.topk_expert, nullptr, s, st);
        else err = launch_topk<kMaxK + 1, false>(logits, T, E, k, G, t.topk_expert, nullptr, s, st);
    }
    if (err != cudaSuccess) return err;

    const int cols = (k + 1) * E;
    k_scan<<<cols * s.segs, 256, 0, st>>>(cols, s);
    k_assign<<<s.tiles, kTileTok, (size_t)kWarps * E * 4, st>>>(T, E, k, C, mode, t.topk_expert, t.route_slot,
                                                               t.slot_token, t.slot_rank, t.drop_count, s);
    if (mode & RR_SCORE) {
        k_select_score<<<E * s.segs, 1024, 0, st>>>(T, E, k, C, mode, t.route_slot, t.slot_token, t.slot_rank, s);
        k_ir_rank<<<s.tiles, kTileTok, (size_t)kWarps * E * 4, st>>>(T, E, k, mode, t.route_slot, t.drop_count, s);
    }
    // (with score-priority dropping the fill-in pass has run as the last rank above: only the IR counts are left)
    k_fr_ir<<<E * s.segs + E, 1024, 0, st>>>(E, k, C, (mode & RR_SCORE) ? (mode & ~RR_FR) : mode,
                                                         t.route_slot, t.slot_token, t.slot_rank, s);
    k_finalize<<<s.tiles, kTileTok, 0, st>>>(T, E, k, C, t, s);
    return cudaGetLastError();
}

}  // namespace rr
