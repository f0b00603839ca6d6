// Device helpers shared by the routing kernels (the multi-launch path in rr_route.cu and the
// single persistent kernel in rr_route_fused.cu): order-preserving keys, the insertion list of the
// top-(k+1) selection, the fixed single-precision exponential, block scans and the per-expert
// selection of the best candidates (Fill-in Rectification, Section 4.2, stage two).
#pragma once
#include <limits.h>
#include <math_constants.h>

#include "rr_common.cuh"

namespace rr {
namespace {

constexpr unsigned kFull = 0xffffffffu;

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

// Barrier among the first `n` threads of a group that agreed on barrier `id` (n a multiple of 32); id 0
// with n = blockDim.x is __syncthreads().
__device__ __forceinline__ void sub_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }

// block_excl_scan for a group of `nthr` threads (indices `tid` = 0 .. nthr-1, whole warps) with its own barrier.
__device__ __forceinline__ int group_excl_scan(int v, int *red, int *total, int tid, int nthr, int bar)
{
    const int lane = tid & 31, warp = tid >> 5, nw = nthr >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += t;
    }
    sub_sync(bar, nthr);  // red may still be read from a previous call
    if (lane == 31) red[warp] = inc;
    sub_sync(bar, nthr);
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
    sub_sync(bar, nthr);
    *total = red[32];
    return red[warp] + inc - v;
}

// 32 x 32 transpose-and-add over a warp: on entry lane l holds v[0..31] (its row), on exit v[0] of lane j
// is the sum over all 32 lanes of their v[j].  After the step with distance `off` a lane holds the half of
// its columns picked by that bit of its index, summed over both lanes of the pair: 31 exchanges, a fixed
// tree (the sums repeat bit for bit).
__device__ __forceinline__ void warp_transpose_add(float (&v)[32], int lane)
{
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < off; ++i) {
            const float send = upper ? v[i] : v[i + off];
            const float recv = __shfl_xor_sync(kFull, send, off);
            v[i] = (upper ? v[i + off] : v[i]) + recv;
        }
    }
}

// -inf that the compiler cannot see through.  The empty places of an insertion list all hold
// -inf; when nvcc 12.9 can prove that (constant initial state reaching the first insertion, e.g.
// after unrolling or peeling), it folds the nested selects of insert_strict on the then identical
// predicates wrongly and the first entry lands in two places.  One volatile asm per place keeps the
// comparisons apart.
__device__ __forceinline__ float empty_place()
{
    float f;
    asm volatile("mov.f32 %0, 0fFF800000;" : "=f"(f));
    return f;
}

// e^t for t <= 0 in single precision with every operation fixed (all round to nearest even): the
// classical two-constant range reduction t = n ln 2 + r, the Taylor polynomial of e^r of degree 7 in
// Horner form, an exact scaling by 2^n.  Arguments below -80 count as -80, so the result is normal.
// Any IEEE-754 machine that follows the same steps obtains the same bits, which lets a value derived
// from it decide who gets a slot (RR_FR_SOFTMAX).
__device__ __forceinline__ float exp_fixed(float t)
{
    t = fmaxf(t, -80.0f);
    const float n = rintf(__fmul_rn(t, 0x1.715476p+0f));  // t * log2(e)
    float r = __fmaf_rn(-n, 0x1.62e4p-1f, t);             // ln 2, leading digits (n * this is exact)
    r = __fmaf_rn(-n, 0x1.7f7d1cp-20f, r);                // ln 2, the rest
    float p = 0x1.a01a02p-13f;                            // 1/7!
    p = __fmaf_rn(p, r, 0x1.6c16c2p-10f);                 // 1/6!
    p = __fmaf_rn(p, r, 0x1.111112p-7f);                  // 1/5!
    p = __fmaf_rn(p, r, 0x1.555556p-5f);                  // 1/4!
    p = __fmaf_rn(p, r, 0x1.555556p-3f);                  // 1/3!
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    return __fmul_rn(p, __int_as_float(((int)n + 127) << 23));
}

// Inserts (x, j) into a list sorted best-first; x enters only ahead of strictly smaller values.
// An empty place holds -inf / INT_MAX and is displaced by any finite value.
template <int KK>
__device__ __forceinline__ void insert_strict(float x, int j, float (&v)[KK], int (&idx)[KK])
{
    bool c[KK];
#pragma unroll
    for (int r = 0; r < KK; ++r) c[r] = x > v[r];
#pragma unroll
    for (int r = KK - 1; r > 0; --r) {
        v[r] = c[r - 1] ? v[r - 1] : (c[r] ? x : v[r]);
        idx[r] = c[r - 1] ? idx[r - 1] : (c[r] ? j : idx[r]);
    }
    v[0] = c[0] ? x : v[0];
    idx[0] = c[0] ? j : idx[0];
}


// ---------------------------------------------------------------------------------------
// One block gives `take` slots of expert e, from slot `first_slot` on, to the best of a list of n
// candidates (keys in list = token order): the take-th largest key by radix select, ties on it to the
// lower tokens, the chosen ones placed in token order.  Section 4.2, stage two, for the nominees;
// the same rule serves every rank when a full expert drops its lowest scores.
// ---------------------------------------------------------------------------------------
// (The candidate lists are read with ld.global.cg: in the persistent routing kernel other blocks of the
// same launch have written them.)
struct SelectShared {
    int hist[4 * 256];  // one histogram per radix pass
    int red[33];
    int bin, remaining;
};

__device__ void select_best(SelectShared &sh, const uint32_t *__restrict__ key, const int *__restrict__ tok, int n,
                            int take, int first_slot, int e, int r, int K1, int C, int *__restrict__ route_slot,
                            int *__restrict__ slot_token, int8_t *__restrict__ slot_rank)
{
    const int tid = threadIdx.x, lane = tid & 31;
    // a list of up to two keys per thread stays in registers, with its tokens
    const int B = (int)blockDim.x;
    const bool in_regs = n <= 2 * B;
    const uint32_t x0 = (in_regs && tid < n) ? __ldcg(key + tid) : 0u;
    const uint32_t x1 = (in_regs && tid + B < n) ? __ldcg(key + tid + B) : 0u;
    const int i0 = (in_regs && tid < n) ? __ldcg(tok + tid) : 0;
    const int i1 = (in_regs && tid + B < n) ? __ldcg(tok + tid + B) : 0;

    // threshold = take-th largest key (most significant byte first).  Two block barriers per pass:
    // the histograms of the four passes are separate and cleared once, and one warp finds the bin.
    uint32_t kth = 0;
    int need_eq = 0;
    if (take < n) {
        __syncthreads();  // an earlier call may still read sh
        for (int c = tid; c < 4 * 256; c += blockDim.x) sh.hist[c] = 0;
        __syncthreads();
        uint32_t prefix = 0, mask = 0;
        int remaining = take;
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            int *hist = sh.hist + 256 * pass;
            if (in_regs) {
                if (tid < n && (x0 & mask) == prefix) atomicAdd(&hist[(x0 >> shift) & 255u], 1);
                if (tid + B < n && (x1 & mask) == prefix) atomicAdd(&hist[(x1 >> shift) & 255u], 1);
            } else {
                for (int q = tid; q < n; q += blockDim.x) {
                    const uint32_t x = __ldcg(key + q);
                    if ((x & mask) == prefix) atomicAdd(&hist[(x >> shift) & 255u], 1);
                }
            }
            __syncthreads();
            if (tid < 32) {
                // bins in descending order, eight per lane: the bin where the running count reaches
                // `remaining`
                int c[8], sum = 0;
#pragma unroll
                for (int u = 0; u < 8; ++u) { c[u] = hist[255 - 8 * lane - u]; sum += c[u]; }
                int inc = sum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int y = __shfl_up_sync(kFull, inc, o);
                    if (lane >= o) inc += y;
                }
                int run = inc - sum;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    if (run < remaining && remaining <= run + c[u]) {
                        sh.bin = 255 - 8 * lane - u;
                        sh.remaining = remaining - run;
                    }
                    run += c[u];
                }
            }
            __syncthreads();
            // (sh.bin is rewritten only after the next pass's first barrier, which every thread reaches
            // after this read)
            prefix |= (uint32_t)sh.bin << shift;
            mask |= 255u << shift;
            remaining = sh.remaining;
        }
        kth = prefix;
        need_eq = remaining;  // how many of the keys equal to kth are taken (>= 1), lowest tokens first
    }

    // stable compaction in list (= token) order; one scan per stretch carries both counts: keys above
    // the threshold in the high half, keys equal to it in the low half (a stretch has <= 1024 entries)
    int eq_run = 0, gt_run = 0;
    for (int q0 = 0; q0 < n; q0 += blockDim.x) {
        const int q = q0 + tid;
        const bool in = q < n;
        const uint32_t x = in_regs ? (q0 == 0 ? x0 : x1) : (in ? __ldcg(key + q) : 0u);
        int before_chosen;
        bool chosen;
        if (take < n) {
            const int is_eq = in && x == kth, is_gt = in && x > kth;
            int total;
            const int b = block_excl_scan(is_eq | (is_gt << 16), sh.red, &total);
            const int eq_before = (b & 0xffff) + eq_run, gt_before = (b >> 16) + gt_run;
            eq_run += total & 0xffff;
            gt_run += total >> 16;
            chosen = is_gt || (is_eq && eq_before < need_eq);
            before_chosen = gt_before + (eq_before < need_eq ? eq_before : need_eq);
        } else {
            chosen = in;
            before_chosen = q;
        }
        if (chosen) {
            const int slot = first_slot + before_chosen;
            const int i = in_regs ? (q0 == 0 ? i0 : i1) : __ldcg(tok + q);
            route_slot[(size_t)i * K1 + r] = slot;
            slot_token[(size_t)e * C + slot] = i;
            slot_rank[(size_t)e * C + slot] = (int8_t)r;
        }
    }
}

// One histogram update per warp and distinct bin, for a digit that takes few values: the keys of one
// expert's candidates mostly share their leading byte (sign and exponent), where one atomic per key
// would serialise on a handful of words.  Every lane of the warp must call it.
__device__ __forceinline__ void hist_add_few_bins(int *hist, bool in, int bin)
{
    const int lane = threadIdx.x & 31;
    unsigned todo = __ballot_sync(kFull, in);
    while (todo) {
        const int leader = __ffs(todo) - 1;
        const int b = __shfl_sync(kFull, bin, leader);
        const unsigned same = __ballot_sync(kFull, in && bin == b);
        if (lane == leader) atomicAdd(&hist[b], __popc(same));
        todo &= ~same;
    }
}

// The same selection for a list of at most KPT keys per thread.  The list is dealt out evenly: with
// kpt = ceil(n / blockDim.x) <= KPT, thread t holds the kpt consecutive keys from t * kpt on (a short
// list keeps every warp busy with one or two keys instead of a few warps with eight).  The keys are
// read once and stay in registers through the four radix passes, the
// histogram updates are aggregated per warp (the keys of one expert share their leading byte, which
// would otherwise serialise the shared-memory atomics), and the stable compaction needs a single block
// scan of the per-thread counts.  n <= KPT * nthr <= 65535.
template <int KPT>
__device__ void select_best_blocked(SelectShared &sh, const uint32_t *__restrict__ key, const int *__restrict__ tok, int n,
                                    int take, int first_slot, int e, int r, int K1, int C, int *__restrict__ route_slot,
                                    int *__restrict__ slot_token, int8_t *__restrict__ slot_rank, int tid, int nthr, int bar)
{
    // run by the `nthr` threads tid = 0 .. nthr-1 of a group of whole warps that synchronises on barrier `bar`
    const int lane = tid & 31;
    const int kpt = (n + nthr - 1) / nthr;  // <= KPT by the caller's choice of nthr
    const int q0 = tid * kpt;
    // key u of this thread exists iff u < kpt and q0 + u < n
#define RR_HAS(u) ((u) < kpt && q0 + (u) < n)
    uint32_t x[KPT];
    int tk[KPT];  // the tokens travel with their keys: one L2 round trip for both
#pragma unroll
    for (int u = 0; u < KPT; ++u) {
        x[u] = RR_HAS(u) ? __ldcg(key + q0 + u) : 0u;
        tk[u] = RR_HAS(u) ? __ldcg(tok + q0 + u) : 0;
    }
    if (take >= n) {  // every candidate fits: list order is slot order
#pragma unroll
        for (int u = 0; u < KPT; ++u) {
            if (RR_HAS(u)) {
                const int i = tk[u], slot = first_slot + q0 + u;
                route_slot[(size_t)i * K1 + r] = slot;
                slot_token[(size_t)e * C + slot] = i;
                slot_rank[(size_t)e * C + slot] = (int8_t)r;
            }
        }
        return;
    }
    sub_sync(bar, nthr);  // an earlier call may still read sh
    for (int c = tid; c < 4 * 256; c += nthr) sh.hist[c] = 0;
    sub_sync(bar, nthr);
    uint32_t prefix = 0, mask = 0;
    int remaining = take;
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        int *hist = sh.hist + 256 * pass;
#pragma unroll
        for (int u = 0; u < KPT; ++u) {
            if (u < kpt) {  // (the same in every thread)
                const bool in = q0 + u < n && (x[u] & mask) == prefix;
                const int bin = (int)((x[u] >> shift) & 255u);
                if (pass == 0) hist_add_few_bins(hist, in, bin);
                else if (in) atomicAdd(&hist[bin], 1);
            }
        }
        sub_sync(bar, nthr);
        if (tid < 32) {
            // bins in descending order, eight per lane: the bin where the running count reaches `remaining`
            int c[8], sum = 0;
#pragma unroll
            for (int u = 0; u < 8; ++u) { c[u] = hist[255 - 8 * lane - u]; sum += c[u]; }
            int inc = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(kFull, inc, o);
                if (lane >= o) inc += y;
            }
            int run = inc - sum;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (run < remaining && remaining <= run + c[u]) {
                    sh.bin = 255 - 8 * lane - u;
                    sh.remaining = remaining - run;
                }
                run += c[u];
            }
        }
        sub_sync(bar, nthr);
        prefix |= (uint32_t)sh.bin << shift;
        mask |= 255u << shift;
        remaining = sh.remaining;
    }
    const uint32_t kth = prefix;   // the take-th largest key
    const int need_eq = remaining; // how many of the keys equal to it are taken (>= 1), lowest tokens first
    int gt = 0, eq = 0;
#pragma unroll
    for (int u = 0; u < KPT; ++u) {
        if (RR_HAS(u)) { gt += x[u] > kth; eq += x[u] == kth; }
    }
    int total;
    const int b = group_excl_scan(eq | (gt << 16), sh.red, &total, tid, nthr, bar);
    int eq_before = b & 0xffff, gt_before = b >> 16;
#pragma unroll
    for (int u = 0; u < KPT; ++u) {
        if (RR_HAS(u)) {
            const bool is_gt = x[u] > kth, is_eq = x[u] == kth;
            if (is_gt || (is_eq && eq_before < need_eq)) {
                const int slot = first_slot + gt_before + (eq_before < need_eq ? eq_before : need_eq);
                const int i = tk[u];
                route_slot[(size_t)i * K1 + r] = slot;
                slot_token[(size_t)e * C + slot] = i;
                slot_rank[(size_t)e * C + slot] = (int8_t)r;
            }
            gt_before += is_gt;
            eq_before += is_eq;
        }
    }
#undef RR_HAS
}

// The same selection for a list of more than four keys per thread (a hot expert's), where the latency
// of the key loads is what counts: eight of them in flight per thread in the histogram passes, the
// next stretch fetched while one is scanned.  (Shorter lists are faster through select_best.)
__device__ void select_best_long(SelectShared &sh, const uint32_t *__restrict__ key, const int *__restrict__ tok, int n,
                            int take, int first_slot, int e, int r, int K1, int C, int *__restrict__ route_slot,
                            int *__restrict__ slot_token, int8_t *__restrict__ slot_rank)
{
    const int tid = threadIdx.x, lane = tid & 31;
    if (take >= n) {  // every nominee gets a slot (Section 4.2 with padding to spare): list order is slot order
        for (int q0 = tid; q0 < n; q0 += 8 * (int)blockDim.x) {  // eight loads in flight per thread
            int is[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int q = q0 + u * (int)blockDim.x;
                is[u] = q < n ? __ldcg(tok + q) : 0;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int q = q0 + u * (int)blockDim.x;
                if (q < n) {
                    const int slot = first_slot + q;
                    route_slot[(size_t)is[u] * K1 + r] = slot;
                    slot_token[(size_t)e * C + slot] = is[u];
                    slot_rank[(size_t)e * C + slot] = (int8_t)r;
                }
            }
        }
        return;
    }
    // a list no longer than the block stays in registers, one key per thread
    const bool in_regs = n <= (int)blockDim.x;
    const uint32_t x0 = (in_regs && tid < n) ? __ldcg(key + tid) : 0u;
    const int i0 = (in_regs && tid < n) ? __ldcg(tok + tid) : 0;  // its token, fetched beside the key

    // threshold = take-th largest key (most significant byte first).  Two block barriers per pass:
    // the histograms of the four passes are separate and cleared once, and one warp finds the bin.
    uint32_t kth = 0;
    int need_eq = 0;
    if (take < n) {
        __syncthreads();  // an earlier call may still read sh
        for (int c = tid; c < 4 * 256; c += blockDim.x) sh.hist[c] = 0;
        __syncthreads();
        uint32_t prefix = 0, mask = 0;
        int remaining = take;
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            int *hist = sh.hist + 256 * pass;
            if (in_regs) {
                if (tid < n && (x0 & mask) == prefix) atomicAdd(&hist[(x0 >> shift) & 255u], 1);
            } else {
                // A long list (a hot expert's) is walked by one block and bound by the latency of its loads:
                // eight 16-byte loads in flight per thread (32 keys; the order of the keys does not matter
                // to a histogram), the up to three keys before the first 16-byte boundary and after the last
                // one by the first lanes of warp 0.
                // First pass: the keys of one expert's candidates mostly share their leading byte (sign and
                // exponent), where one atomic per key would serialise on a handful of words: every thread counts
                // the two values it meets first in registers and adds them up once at the end.
                int b0 = -1, b1 = -1, c0 = 0, c1 = 0;
                auto count = [&](bool in, uint32_t x) {
                    in = in && (x & mask) == prefix;
                    const int bin = (int)((x >> shift) & 255u);
                    if (!in) return;
                    if (pass != 0) { atomicAdd(&hist[bin], 1); return; }
                    if (bin == b0) ++c0;
                    else if (bin == b1) ++c1;
                    else if (b0 < 0) { b0 = bin; c0 = 1; }
                    else if (b1 < 0) { b1 = bin; c1 = 1; }
                    else atomicAdd(&hist[bin], 1);
                };
                const int head = min(n, (int)((4u - (unsigned)((reinterpret_cast<uintptr_t>(key) >> 2) & 3u)) & 3u));
                const int nvec = (n - head) >> 2, tail0 = head + 4 * nvec;
                const uint4 *kv = reinterpret_cast<const uint4 *>(key + head);
                for (int v0 = tid - lane; v0 < nvec; v0 += 8 * (int)blockDim.x) {
                    uint4 xs[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const int v = v0 + lane + u * (int)blockDim.x;
                        xs[u] = v < nvec ? __ldcg(kv + v) : make_uint4(0u, 0u, 0u, 0u);
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const bool in = v0 + lane + u * (int)blockDim.x < nvec;
                        count(in, xs[u].x);
                        count(in, xs[u].y);
                        count(in, xs[u].z);
                        count(in, xs[u].w);
                    }
                }
                if (tid < 32) {  // lanes 0..2: the keys before the first boundary; lanes 3..5: those after the last
                    const int q = lane < 3 ? (lane < head ? lane : -1) : (lane < 6 && tail0 + lane - 3 < n ? tail0 + lane - 3 : -1);
                    const uint32_t x = q >= 0 ? __ldcg(key + q) : 0u;
                    count(q >= 0, x);
                }
                if (c0) atomicAdd(&hist[b0], c0);
                if (c1) atomicAdd(&hist[b1], c1);
            }
            __syncthreads();
            if (tid < 32) {
                // bins in descending order, eight per lane: the bin where the running count reaches
                // `remaining`
                int c[8], sum = 0;
#pragma unroll
                for (int u = 0; u < 8; ++u) { c[u] = hist[255 - 8 * lane - u]; sum += c[u]; }
                int inc = sum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int y = __shfl_up_sync(kFull, inc, o);
                    if (lane >= o) inc += y;
                }
                int run = inc - sum;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    if (run < remaining && remaining <= run + c[u]) {
                        sh.bin = 255 - 8 * lane - u;
                        sh.remaining = remaining - run;
                    }
                    run += c[u];
                }
            }
            __syncthreads();
            // (sh.bin is rewritten only after the next pass's first barrier, which every thread reaches
            // after this read)
            prefix |= (uint32_t)sh.bin << shift;
            mask |= 255u << shift;
            remaining = sh.remaining;
        }
        kth = prefix;
        need_eq = remaining;  // how many of the keys equal to kth are taken (>= 1), lowest tokens first
    }

    if (!in_regs && take < n) {
        // Stable compaction of a long list without a block barrier per stretch: every warp owns a
        // contiguous part of the list (a multiple of 32 entries), counts its keys above / equal to the
        // threshold in a first walk, the warps' counts are added up once, and a second walk places the
        // chosen entries with warp ballots.  Both walks keep eight coalesced loads in flight per thread.
        const int nwp = (int)blockDim.x >> 5, warp = tid >> 5;
        const int seg = ((n + nwp - 1) / nwp + 31) & ~31;
        const int a = warp * seg, bnd = a + seg < n ? a + seg : n;
        const unsigned below = (1u << lane) - 1u;
        int gt_w = 0, eq_w = 0;
        {
            // counting walk: 16-byte loads (the warp's part starts a multiple of four entries into the list, so
            // the keys before the first 16-byte boundary number the same as for the whole list), every lane
            // counts its own keys and the warp adds up once
            const int len = bnd > a ? bnd - a : 0;  // (the last warps of a list that is not that long own nothing)
            const int head = min(len, (int)((4u - (unsigned)((reinterpret_cast<uintptr_t>(key) >> 2) & 3u)) & 3u));
            const int nvec = (len - head) >> 2, tail0 = a + head + 4 * nvec;
            const uint4 *kv = reinterpret_cast<const uint4 *>(key + a + head);
            int gt = 0, eq = 0;
            for (int v0 = 0; v0 < nvec; v0 += 256) {
                uint4 xs[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int v = v0 + 32 * u + lane;
                    xs[u] = v < nvec ? __ldcg(kv + v) : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    if (v0 + 32 * u + lane < nvec) {
                        gt += (xs[u].x > kth) + (xs[u].y > kth) + (xs[u].z > kth) + (xs[u].w > kth);
                        eq += (xs[u].x == kth) + (xs[u].y == kth) + (xs[u].z == kth) + (xs[u].w == kth);
                    }
                }
            }
            const int q = lane < 3 ? (lane < head ? a + lane : -1) : (lane < 6 && tail0 + lane - 3 < a + len ? tail0 + lane - 3 : -1);
            if (q >= 0) {
                const uint32_t x = __ldcg(key + q);
                gt += x > kth;
                eq += x == kth;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                gt += __shfl_xor_sync(kFull, gt, o);
                eq += __shfl_xor_sync(kFull, eq, o);
            }
            gt_w = gt;
            eq_w = eq;
        }
        __syncthreads();  // sh.hist is free: its first words carry the warps' counts
        if (lane == 0) { sh.hist[warp] = gt_w; sh.hist[32 + warp] = eq_w; }
        __syncthreads();
        int gt_run = 0, eq_run = 0;
        for (int w = 0; w < warp; ++w) { gt_run += sh.hist[w]; eq_run += sh.hist[32 + w]; }
        for (int q0 = a; q0 < bnd; q0 += 256) {
            uint32_t xs[8];
            int is[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int q = q0 + 32 * u + lane;
                xs[u] = q < bnd ? __ldcg(key + q) : 0u;
                is[u] = q < bnd ? __ldcg(tok + q) : 0;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const bool in = q0 + 32 * u + lane < bnd;
                const bool is_gt = in && xs[u] > kth, is_eq = in && xs[u] == kth;
                const unsigned m_gt = __ballot_sync(kFull, is_gt), m_eq = __ballot_sync(kFull, is_eq);
                const int eq_before = eq_run + __popc(m_eq & below), gt_before = gt_run + __popc(m_gt & below);
                if (is_gt || (is_eq && eq_before < need_eq)) {
                    const int slot = first_slot + gt_before + (eq_before < need_eq ? eq_before : need_eq);
                    const int i = is[u];
                    route_slot[(size_t)i * K1 + r] = slot;
                    slot_token[(size_t)e * C + slot] = i;
                    slot_rank[(size_t)e * C + slot] = (int8_t)r;
                }
                gt_run += __popc(m_gt);
                eq_run += __popc(m_eq);
            }
        }
        return;
    }

    // stable compaction in list (= token) order; one scan per stretch carries both counts: keys above
    // the threshold in the high half, keys equal to it in the low half (a stretch has <= 1024 entries)
    int eq_run = 0, gt_run = 0;
    // (a long list: the next stretch's key and token are fetched while this one is scanned)
    uint32_t x_next = (!in_regs && tid < n) ? __ldcg(key + tid) : 0u;
    int i_next = (!in_regs && tid < n) ? __ldcg(tok + tid) : 0;
    for (int q0 = 0; q0 < n; q0 += blockDim.x) {
        const int q = q0 + tid;
        const bool in = q < n;
        const uint32_t x = in_regs ? x0 : x_next;
        const int i_here = in_regs ? i0 : i_next;
        if (!in_regs) {
            const int qn = q + (int)blockDim.x;
            x_next = qn < n ? __ldcg(key + qn) : 0u;
            i_next = qn < n ? __ldcg(tok + qn) : 0;
        }
        int before_chosen;
        bool chosen;
        if (take < n) {
            const int is_eq = in && x == kth, is_gt = in && x > kth;
            int total;
            const int b = block_excl_scan(is_eq | (is_gt << 16), sh.red, &total);
            const int eq_before = (b & 0xffff) + eq_run, gt_before = (b >> 16) + gt_run;
            eq_run += total & 0xffff;
            gt_run += total >> 16;
            chosen = is_gt || (is_eq && eq_before < need_eq);
            before_chosen = gt_before + (eq_before < need_eq ? eq_before : need_eq);
        } else {
            chosen = in;
            before_chosen = q;
        }
        if (chosen) {
            const int slot = first_slot + before_chosen;
            const int i = i_here;
            route_slot[(size_t)i * K1 + r] = slot;
            slot_token[(size_t)e * C + slot] = i;
            slot_rank[(size_t)e * C + slot] = (int8_t)r;
        }
    }
}

}  // namespace
}  // namespace rr
