// Routing kernels: top-(k+1) selection, capacity assignment, Intra-GPU
// Rectification, Fill-in Rectification, combine weights and the compact row space
// (arXiv 2402.12399, Section 3 Eq. 1-2, Section 4.1 Eq. 3, Section 4.2).
//
// Five launches per call:
//   k_topk     one pass over logits[T,E]: per token the k+1 best experts by
//              (logit desc, index asc) and the best expert of its own group; per tile
//              the number of tokens per (rank, expert) and each token's position among them
//   k_scan     exclusive prefix of those counts over tiles, totals, per-expert bases
//   k_assign   slot = base + prefix + local position; kept iff < capacity; nominee lists
//              for FR; per-tile ranking of IR tokens
//   k_fr_ir    one block per expert: choose the v_e best nominees (radix select on an
//              order-preserving key, ties to the lower token) and place them in token
//              order; one more block scans the IR counts over tiles
//   k_finalize IR lists, combine weights, row space, padding marks
// Every decision is an exact comparison of raw fp32 logits, so the tables are unique.
#include <limits.h>
#include <math_constants.h>

#include "rr_common.cuh"

namespace rr {

namespace {

constexpr int kWarps = kTileTok / 32;
constexpr unsigned kFull = 0xffffffffu;

// (logit desc, index asc); float equality, so -0 ties with +0.
__device__ __forceinline__ bool precedes(float a, int ia, float b, int ib)
{
    return a > b || (a == b && ia < ib);
}

// Monotone map float -> uint32 (larger float, larger key); both zeros map to one key.
__device__ __forceinline__ uint32_t order_key(float f)
{
    if (f == 0.0f) f = 0.0f;
    uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Exclusive block scan of one int per thread (blockDim.x multiple of 32, <= 1024).
// `red` is 33 ints of shared memory; returns the exclusive prefix, *total = block sum.
__device__ __forceinline__ int block_excl_scan(int v, int *red, int *total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();  // red may still be read from a previous call
    if (lane == 31) red[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = lane < nw ? red[lane] : 0;
        int winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(kFull, winc, o);
            if (lane >= o) winc += t;
        }
        if (lane < nw) red[lane] = winc - w;
        if (lane == 31) red[32] = winc;
    }
    __syncthreads();
    *total = red[32];
    return red[warp] + inc - v;
}

// ---------------------------------------------------------------------------------------
// k_topk.  L lanes cooperate on one token, each holding V logits in registers
// (element j = (v/4)*128 + sub*4 + v%4, so loads are float4 and coalesced).
// ---------------------------------------------------------------------------------------
template <int L, int V>
__global__ void __launch_bounds__(kTileTok)
k_topk(const float *__restrict__ logits, int T, int E, int k, int G, int *__restrict__ topk_expert,
       RouteScratch s)
{
    extern __shared__ int smem[];
    const int K1 = k + 1;
    int *sel_s = smem;                                                   // [K1][256]
    float *val_s = reinterpret_cast<float *>(sel_s + K1 * kTileTok);     // [K1][256]
    int *pos_s = reinterpret_cast<int *>(val_s + K1 * kTileTok);         // [K1][256]
    int *h_s = pos_s + K1 * kTileTok;                                    // [256]
    float *ah_s = reinterpret_cast<float *>(h_s + kTileTok);             // [256]
    int *wcount = reinterpret_cast<int *>(ah_s + kTileTok);              // [warps][K1][E]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x, tok0 = tile * kTileTok;
    const int cols = K1 * E;
    for (int c = tid; c < kWarps * cols; c += kTileTok) wcount[c] = 0;

    const int tpg = T / G > 0 ? T / G : 1, epg = E / G;
    constexpr int TPP = 32 / L;
    const int sub = lane % L;
    const bool vec = (E & 3) == 0;
    bool bad = false;

    for (int p = 0; p < L; ++p) {
        const int tt = warp * 32 + p * TPP + lane / L;
        const int i = tok0 + tt;
        const bool live = i < T;
        const float *row = logits + (size_t)(live ? i : 0) * E;
        float v[V];
#pragma unroll
        for (int q = 0; q < V / 4; ++q) {
            const int j0 = q * 128 + sub * 4;
            if (live && j0 < E) {
                if (vec) {
                    float4 f = *reinterpret_cast<const float4 *>(row + j0);
                    v[q * 4 + 0] = f.x; v[q * 4 + 1] = f.y; v[q * 4 + 2] = f.z; v[q * 4 + 3] = f.w;
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) v[q * 4 + c] = (j0 + c < E) ? row[j0 + c] : -CUDART_INF_F;
                }
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) v[q * 4 + c] = -CUDART_INF_F;
            }
        }
#pragma unroll
        for (int x = 0; x < V; ++x) {
            const int j = (x >> 2) * 128 + sub * 4 + (x & 3);
            if (live && j < E && !isfinite(v[x])) { bad = true; v[x] = 0.0f; }
        }

        // Eq. 1 extended by one place: k+1 rounds of arg-best over the untaken experts
        unsigned taken = 0;
        for (int r = 0; r < K1; ++r) {
            float bv = -CUDART_INF_F;
            int bj = INT_MAX;
#pragma unroll
            for (int x = 0; x < V; ++x) {
                const int j = (x >> 2) * 128 + sub * 4 + (x & 3);
                if (!((taken >> x) & 1u) && j < E && precedes(v[x], j, bv, bj)) { bv = v[x]; bj = j; }
            }
#pragma unroll
            for (int o = L / 2; o > 0; o >>= 1) {
                float ov = __shfl_xor_sync(kFull, bv, o);
                int oj = __shfl_xor_sync(kFull, bj, o);
                if (precedes(ov, oj, bv, bj)) { bv = ov; bj = oj; }
            }
#pragma unroll
            for (int x = 0; x < V; ++x)
                if ((x >> 2) * 128 + sub * 4 + (x & 3) == bj) taken |= 1u << x;
            if (sub == 0) {
                sel_s[r * kTileTok + tt] = (live && bj != INT_MAX) ? bj : -1;
                val_s[r * kTileTok + tt] = bv;
            }
        }
        // Section 4.1: best expert among those of the token's own group
        {
            const int g = live ? i / tpg : 0;
            const int lo = g * epg, hi = lo + epg;
            float bv = -CUDART_INF_F;
            int bj = INT_MAX;
#pragma unroll
            for (int x = 0; x < V; ++x) {
                const int j = (x >> 2) * 128 + sub * 4 + (x & 3);
                if (j >= lo && j < hi && j < E && precedes(v[x], j, bv, bj)) { bv = v[x]; bj = j; }
            }
#pragma unroll
            for (int o = L / 2; o > 0; o >>= 1) {
                float ov = __shfl_xor_sync(kFull, bv, o);
                int oj = __shfl_xor_sync(kFull, bj, o);
                if (precedes(ov, oj, bv, bj)) { bv = ov; bj = oj; }
            }
            if (sub == 0) {
                h_s[tt] = (live && bj != INT_MAX) ? bj : lo;
                ah_s[tt] = bv;
            }
        }
    }
    if (bad) latch_status(&s.hdr->status, RR_ERR_NONFINITE);
    __syncthreads();

    // thread t now owns token t of the tile
    const int i = tok0 + tid;
    const bool live = i < T;
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
        s.hist[(size_t)tile * cols + c] = run;
    }
    __syncthreads();
    if (live) {
        for (int r = 0; r < K1; ++r) {
            const int e = sel_s[r * kTileTok + tid];
            s.pos_local[(size_t)i * K1 + r] = e >= 0 ? wcount[(warp * K1 + r) * E + e] + pos_s[r * kTileTok + tid] : 0;
        }
    }
}

// ---------------------------------------------------------------------------------------
// k_scan: one block.  hist[tile][c] -> exclusive prefix over tiles; totals; bases.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
k_scan(int E, int k, int C, RouteScratch s, int *__restrict__ n_routed, int *__restrict__ expert_count)
{
    const int K1 = k + 1, cols = K1 * E, tid = threadIdx.x;
    for (int c = tid; c < cols; c += blockDim.x) {
        int run = 0;
        int t = 0;
        for (; t + 8 <= s.tiles; t += 8) {
            int x[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) x[u] = s.hist[(size_t)(t + u) * cols + c];
#pragma unroll
            for (int u = 0; u < 8; ++u) { s.hist[(size_t)(t + u) * cols + c] = run; run += x[u]; }
        }
        for (; t < s.tiles; ++t) {
            const int x = s.hist[(size_t)t * cols + c];
            s.hist[(size_t)t * cols + c] = run;
            run += x;
        }
        s.totals[c] = run;
    }
    __syncthreads();
    for (int e = tid; e < E; e += blockDim.x) {
        int n = 0;
        for (int r = 0; r < k; ++r) { s.base[r * E + e] = n; n += s.totals[r * E + e]; }
        s.base[k * E + e] = n;
        n_routed[e] = n;                  // n_e
        expert_count[e] = n < C ? n : C;  // kept_e; k_fr_ir adds the filled slots
    }
    __syncthreads();
    if (tid == 0) {
        int off = 0;
        for (int e = 0; e < E; ++e) { s.nom_off[e] = off; off += s.totals[k * E + e]; }
        s.nom_off[E] = off;
    }
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
    const int K1 = k + 1, cols = K1 * E;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x, i = tile * kTileTok + tid;
    const bool live = i < T;
    for (int c = tid; c < kWarps * E; c += kTileTok) wcount[c] = 0;

    int d = 0;
    if (live) {
        const int *pre = s.hist + (size_t)tile * cols;
        for (int r = 0; r < k; ++r) {
            const int e = topk_expert[(size_t)i * K1 + r];
            const int p = s.base[r * E + e] + pre[r * E + e] + s.pos_local[(size_t)i * K1 + r];
            if (p < C) {
                route_slot[(size_t)i * K1 + r] = p;
                slot_token[(size_t)e * C + p] = i;
                slot_rank[(size_t)e * C + p] = (int8_t)r;
            } else {
                route_slot[(size_t)i * K1 + r] = -1;
                ++d;
            }
        }
        route_slot[(size_t)i * K1 + k] = -1;
        if (mode & RR_FR) {  // Section 4.2, stage one: nominate the (k+1)-th expert
            const int e = topk_expert[(size_t)i * K1 + k];
            const int p = s.nom_off[e] + pre[k * E + e] + s.pos_local[(size_t)i * K1 + k];
            s.nom_key[p] = order_key(s.val[(size_t)i * K1 + k]);
            s.nom_token[p] = i;
        }
        drop_count[i] = d;
    }
    // Section 4.1: tokens with a dropped routing queue at their in-group expert, token order
    const int key = (live && (mode & RR_IR) && d > 0) ? s.h[i] : -1;
    __syncthreads();
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
        s.ir_hist[(size_t)tile * E + e] = run;
    }
    __syncthreads();
    if (live) s.ir_local[i] = key >= 0 ? wcount[warp * E + key] + rk : -1;
}

// ---------------------------------------------------------------------------------------
// k_fr_ir: blocks 0..E-1 run Fill-in Rectification for one expert each (Section 4.2,
// stage two); block E turns the per-tile IR counts into prefixes and list offsets.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
k_fr_ir(int E, int k, int C, unsigned mode, int *__restrict__ route_slot, int *__restrict__ slot_token,
        int8_t *__restrict__ slot_rank, const int *__restrict__ n_routed, int *__restrict__ expert_count,
        int *__restrict__ ir_offset, RouteScratch s)
{
    __shared__ int hist[256];
    __shared__ int red[33];
    __shared__ int sh_bin, sh_remaining;
    const int tid = threadIdx.x, K1 = k + 1;

    if ((int)blockIdx.x == E) {
        for (int e = tid; e < E; e += blockDim.x) {
            int run = 0;
            for (int t = 0; t < s.tiles; ++t) {
                const int x = s.ir_hist[(size_t)t * E + e];
                s.ir_hist[(size_t)t * E + e] = run;
                run += x;
            }
            hist[e] = run;  // E <= 256
        }
        __syncthreads();
        if (tid == 0) {
            int off = 0;
            for (int e = 0; e < E; ++e) { ir_offset[e] = off; off += hist[e]; }
            ir_offset[E] = off;
        }
        return;
    }
    if (!(mode & RR_FR)) return;

    const int e = blockIdx.x;
    const int n = s.nom_off[e + 1] - s.nom_off[e];
    const uint32_t *key = s.nom_key + s.nom_off[e];
    const int *tok = s.nom_token + s.nom_off[e];
    const int kept = n_routed[e] < C ? n_routed[e] : C;
    const int v = C - kept;               // padding slots of this expert
    const int take = n < v ? n : v;
    if (take == 0) return;
    if (tid == 0) expert_count[e] = kept + take;

    // threshold = take-th largest key (radix select, most significant byte first)
    uint32_t kth = 0;
    int need_eq = 0;
    if (take < n) {
        uint32_t prefix = 0, mask = 0;
        int remaining = take;
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            for (int q = tid; q < n; q += blockDim.x) {
                const uint32_t x = key[q];
                if ((x & mask) == prefix) atomicAdd(&hist[(x >> shift) & 255u], 1);
            }
            __syncthreads();
            if (tid == 0) {
                int cum = 0, b = 255;
                for (; b > 0; --b) {
                    if (cum + hist[b] >= remaining) break;
                    cum += hist[b];
                }
                sh_bin = b;
                sh_remaining = remaining - cum;
            }
            __syncthreads();
            prefix |= (uint32_t)sh_bin << shift;
            mask |= 255u << shift;
            remaining = sh_remaining;
            __syncthreads();
        }
        kth = prefix;
        need_eq = remaining;  // how many of the keys equal to kth are taken (>= 1), lowest tokens first
    }

    // stable compaction in list (= token) order
    int eq_run = 0, ch_run = 0;
    for (int q0 = 0; q0 < n; q0 += blockDim.x) {
        const int q = q0 + tid;
        const bool in = q < n;
        const uint32_t x = in ? key[q] : 0u;
        bool chosen;
        int total;
        if (take < n) {
            const int is_eq = in && x == kth;
            const int eq_before = block_excl_scan(is_eq, red, &total) + eq_run;
            eq_run += total;
            chosen = in && (x > kth || (is_eq && eq_before < need_eq));
        } else {
            chosen = in;
        }
        const int ch_before = block_excl_scan(chosen ? 1 : 0, red, &total) + ch_run;
        ch_run += total;
        if (chosen) {
            const int slot = kept + ch_before;
            const int i = tok[q];
            route_slot[(size_t)i * K1 + k] = slot;
            slot_token[(size_t)e * C + slot] = i;
            slot_rank[(size_t)e * C + slot] = (int8_t)k;
        }
    }
}

// ---------------------------------------------------------------------------------------
// k_finalize: IR lists, combine weights (Eq. 2 / Eq. 3), row space, padding marks.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTileTok)
k_finalize(int T, int E, int k, int C, rr_route_tables t, RouteScratch s)
{
    __shared__ int cnt_s[kMaxE];
    __shared__ int iro_s[kMaxE + 1];
    __shared__ int row_s[kMaxE + 1];
    const int K1 = k + 1, K2 = k + 2;
    const int tid = threadIdx.x, tile = blockIdx.x, i = tile * kTileTok + tid;
    for (int e = tid; e < E; e += kTileTok) cnt_s[e] = t.expert_count[e];
    for (int e = tid; e <= E; e += kTileTok) iro_s[e] = t.ir_offset[e];
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        for (int e = 0; e < E; ++e) { row_s[e] = acc; acc += cnt_s[e] + iro_s[e + 1] - iro_s[e]; }
        row_s[E] = acc;
    }
    __syncthreads();
    if (tile == 0)
        for (int e = tid; e <= E; e += kTileTok) t.row_offset[e] = row_s[e];

    if (i < T) {
        float num[kMaxK + 2];
        int row[kMaxK + 2];
        const float m = s.val[(size_t)i * K1];  // top-1 logit = max over all experts
        float den = 0.0f;
        for (int r = 0; r < K1; ++r) {
            const int slot = t.route_slot[(size_t)i * K1 + r];
            num[r] = 0.0f;
            row[r] = -1;
            if (slot >= 0) {
                num[r] = expf(s.val[(size_t)i * K1 + r] - m);
                den += num[r];
                row[r] = row_s[t.topk_expert[(size_t)i * K1 + r]] + slot;
            }
        }
        num[K1] = 0.0f;
        row[K1] = -1;
        const int il = s.ir_local[i];
        int hh = -1, pos = -1;
        if (il >= 0) {
            hh = s.h[i];
            pos = s.ir_hist[(size_t)tile * E + hh] + il;
            t.ir_token[iro_s[hh] + pos] = i;
            // Eq. 3: the IR route carries the weight of every dropped routing
            num[K1] = (float)t.drop_count[i] * expf(s.a_h[i] - m);
            den += num[K1];
            row[K1] = row_s[hh] + cnt_s[hh] + pos;
        }
        t.ir_expert[i] = hh;
        t.ir_pos[i] = pos;
        for (int r = 0; r < K2; ++r) {
            const float w = den > 0.0f ? num[r] / den : 0.0f;
            t.combine_w[(size_t)i * K2 + r] = w;
            t.token_rows[(size_t)i * K2 + r] = row[r];
            if (row[r] >= 0) {
                t.row_token[row[r]] = i;
                t.row_weight[row[r]] = w;
            }
        }
    }

    // marks outside the live ranges
    const size_t stride = (size_t)gridDim.x * kTileTok, g0 = (size_t)blockIdx.x * kTileTok + tid;
    const size_t slots = (size_t)E * C;
    for (size_t q = g0; q < slots; q += stride) {
        const int e = (int)(q / C), sl = (int)(q % C);
        if (sl >= cnt_s[e]) { t.slot_token[q] = -1; t.slot_rank[q] = -1; }
    }
    for (size_t q = g0; q < (size_t)T; q += stride)
        if ((int)q >= iro_s[E]) t.ir_token[q] = -1;
    for (size_t q = g0; q < slots + T; q += stride)
        if (q >= (size_t)row_s[E]) { t.row_token[q] = -1; t.row_weight[q] = 0.0f; }
}

template <int L, int V>
cudaError_t launch_topk(const float *logits, int T, int E, int k, int G, int *topk_expert,
                        const RouteScratch &s, cudaStream_t st)
{
    const int K1 = k + 1;
    const size_t smem = ((size_t)3 * K1 * kTileTok + 2 * kTileTok + (size_t)kWarps * K1 * E) * 4;
    cudaError_t err = cudaFuncSetAttribute(k_topk<L, V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    k_topk<L, V><<<s.tiles, kTileTok, smem, st>>>(logits, T, E, k, G, topk_expert, s);
    return cudaGetLastError();
}

}  // namespace

size_t route_scratch_layout(void *ws, int T, int E, int k, RouteScratch *s)
{
    const int K1 = k + 1;
    const int tiles = T > 0 ? (T + kTileTok - 1) / kTileTok : 1;
    const size_t Tn = T > 0 ? T : 1;
    Carver c(ws);
    s->hdr = c.take<Header>(1);
    s->val = c.take<float>(Tn * K1);
    s->h = c.take<int>(Tn);
    s->a_h = c.take<float>(Tn);
    s->pos_local = c.take<int>(Tn * K1);
    s->hist = c.take<int>((size_t)tiles * K1 * E);
    s->totals = c.take<int>((size_t)K1 * E);
    s->base = c.take<int>((size_t)K1 * E);
    s->nom_off = c.take<int>(E + 1);
    s->nom_key = c.take<uint32_t>(Tn);
    s->nom_token = c.take<int>(Tn);
    s->ir_local = c.take<int>(Tn);
    s->ir_hist = c.take<int>((size_t)tiles * E);
    s->tiles = tiles;
    return align_up(c.off, 256);
}

cudaError_t launch_route(const float *logits, int T, int E, int k, int C, int G, unsigned mode,
                         const rr_route_tables &t, const RouteScratch &s, cudaStream_t st)
{
    cudaError_t err;
    if (E <= 4) err = launch_topk<1, 4>(logits, T, E, k, G, t.topk_expert, s, st);
    else if (E <= 8) err = launch_topk<2, 4>(logits, T, E, k, G, t.topk_expert, s, st);
    else if (E <= 16) err = launch_topk<4, 4>(logits, T, E, k, G, t.topk_expert, s, st);
    else if (E <= 32) err = launch_topk<8, 4>(logits, T, E, k, G, t.topk_expert, s, st);
    else if (E <= 64) err = launch_topk<16, 4>(logits, T, E, k, G, t.topk_expert, s, st);
    else if (E <= 128) err = launch_topk<32, 4>(logits, T, E, k, G, t.topk_expert, s, st);
    else err = launch_topk<32, 8>(logits, T, E, k, G, t.topk_expert, s, st);
    if (err != cudaSuccess) return err;

    k_scan<<<1, 1024, 0, st>>>(E, k, C, s, t.n_routed, t.expert_count);
    k_assign<<<s.tiles, kTileTok, (size_t)kWarps * E * 4, st>>>(T, E, k, C, mode, t.topk_expert, t.route_slot,
                                                               t.slot_token, t.slot_rank, t.drop_count, s);
    k_fr_ir<<<E + 1, 1024, 0, st>>>(E, k, C, mode, t.route_slot, t.slot_token, t.slot_rank, t.n_routed,
                                    t.expert_count, t.ir_offset, s);
    k_finalize<<<s.tiles, kTileTok, 0, st>>>(T, E, k, C, t, s);
    return cudaGetLastError();
}

}  // namespace rr
