// Shared declarations of the rectified-MoE CUDA library (internal; the public
// interface is include/rr.h).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "rr.h"

namespace rr {

constexpr int kMaxE = 256;         // experts
constexpr int kMaxK = 8;           // top-k
constexpr int kTileTok = 256;      // tokens per routing tile (= threads per routing block)
constexpr int kHeaderBytes = 256;  // workspace header: status word first

// Workspace header, first bytes of every workspace (zero when the workspace is first used).
struct Header {
    int status;    // latched rr_status detected on the device (0 = none)
    int pad0[15];
    // words of the persistent routing kernel's grid barrier: [0] arrivals (monotone inside a call),
    // [1] set when a block gave up waiting, [2] blocks that have left.  The last block to leave puts
    // them back to zero, so a finished call leaves them as it found them.
    int sync[16];
    int pad1[32];
};
static_assert(sizeof(Header) == kHeaderBytes, "the header fills the first 256 bytes of a workspace");

__device__ __forceinline__ void latch_status(int *status, int code) { atomicCAS(status, 0, code); }

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Testing aid (rr_test_set_wait_limit_ns): when non-zero, the time limit of the waits that the tests
// make run out -- the grid barriers of the routing kernel, the accumulator wait of the forward GEMMs'
// epilogue -- instead of the 2 s of production.  Host-side; launches copy it into their parameters.
unsigned long long test_wait_limit_ns();

// Carves aligned sub-buffers out of one workspace allocation (base may be null to size only).
struct Carver {
    char *base;
    size_t off;
    explicit Carver(void *p) : base(static_cast<char *>(p)), off(0) {}
    template <class T>
    T *take(size_t n, size_t align = 256)
    {
        off = align_up(off, align);
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

constexpr int kMaxRouteCtas = 256;  // upper bound on the grid of the persistent routing kernel

// Scratch of the routing kernels (device pointers into the workspace).  Two layouts share the
// struct: the persistent single-launch kernel (`fused`, every mode without RR_SCORE and
// RR_LOCAL_CAP) and the multi-launch path.
struct RouteScratch {
    int *status;        // latched device status word (first word of the workspace header, or the caller's)
    int *sync;          // Header::sync
    int fused;          // 1: layout of the persistent kernel
    // ---- persistent kernel ----
    int *rec;           // [blocks of 32 tokens][fields][32] per-token records carried between the phases
    uint16_t *agg;      // [kMaxRouteCtas][K1*E rounded up to 8] per-block counts of every (rank, expert) column
    uint16_t *ir_agg;   // [kMaxRouteCtas][E rounded up to 8]    per-block counts of IR tokens per expert
    // ---- multi-launch path ----
    float *val;         // [T,K1] logits of the top-(k+1) experts
    int *h;             // [T]    in-group best expert
    float *a_h;         // [T]    its logit
    int *pos_local;     // [T,K1] position among same-(rank,expert) tokens of the tile
    int *hist;          // [K1*E,tiles] per-tile counts (column-major), then exclusive prefix over tiles
    int *totals;        // [segs,K1,E] counts over the tiles of each capacity segment
    int *ir_local;      // [T]    position among the tile's IR tokens of the same expert, -1 none
    int *ir_hist;       // [E,tiles] per-tile IR counts (column-major), then exclusive prefix over tiles
    int *ir_totals;     // [E] IR list lengths
    int *seg_n;         // [segs,E] top-k routings addressed to the expert from the segment's tokens
    int *seg_occ;       // [segs,E] occupied slots of the expert inside the segment (kept, then + filled)
    // ---- both ----
    uint32_t *nom_key;  // [T]    order-preserving keys of nominee logits, expert after expert
                        //        ([K1,T] with RR_SCORE: the candidates of every rank, rank after rank)
    int *nom_token;     // same shape: their tokens
    float *fr_key;      // [T] with RR_FR_SOFTMAX: softmax value of the token at the expert it nominates
    int tiles;          // segs * tps
    // Capacity segments: one over all tokens, or with RR_LOCAL_CAP one per source group.  Segment sg
    // serves tokens [sg*Tseg, (sg+1)*Tseg) with tiles [sg*tps, (sg+1)*tps) (no tile spans two segments)
    // and owns slots [sg*C/segs, (sg+1)*C/segs) of every expert.
    int segs, tps, Tseg;
};

// Words per token of the persistent kernel's records: K1 logits, K1 positions (then slots), K1 experts,
// the in-group expert, its logit, the position in that expert's IR list.
__host__ __device__ inline int route_rec_fields(int k) { return 3 * (k + 1) + 3; }

// Which calls the persistent kernel serves: every mode without RR_SCORE / RR_LOCAL_CAP, up to 2^22
// tokens (its per-block counts are 16-bit: a block's token range must stay below 65536, which holds
// from 65 SMs on).
inline bool route_is_fused(unsigned mode, int T) { return (mode & (RR_SCORE | RR_LOCAL_CAP)) == 0 && T <= (1 << 22); }

// The token a thread of a routing tile works on.
struct TileToken {
    int sg;     // capacity segment of the tile
    int i;      // token index
    bool live;  // false: past the end of the segment
};
__device__ __forceinline__ TileToken tile_token(const RouteScratch &s, int tile, int tid)
{
    const int sg = tile / s.tps;
    const int local = (tile - sg * s.tps) * kTileTok + tid;
    return {sg, sg * s.Tseg + local, local < s.Tseg};
}

size_t route_scratch_layout(void *ws, int T, int E, int k, RouteScratch *s, unsigned mode = 0, int G = 1);

cudaError_t launch_route(const float *logits, int T, int E, int k, int C, int G, unsigned mode,
                         const rr_route_tables &t, const RouteScratch &s, cudaStream_t st);

// What a gate projection that selects in its epilogue (rr_gate_route) hands to the persistent routing
// kernel instead of the logits, and what the kernel returns for the load-balance loss.
struct RoutePresel {
    const float *val;   // [T,K1] scores of the k+1 best experts (their indices are in topk_expert)
    const int *h;       // [T]    best expert of the token's own group
    const float *a_h;   // [T]    its score
    float *psum;        // [ceil(T/32),E] softmax values summed over each 32 tokens, or null (no loss wanted)
    float *cta_psum;    // [kMaxRouteCtas,E] scratch: the same sums per block of the routing kernel
    float alpha;        // L = alpha * E * sum_e f_e P_e
    float *loss, *f, *P;  // [1], [E], [E] outputs (with psum)
};

// The persistent single-launch router (rr_route_fused.cu); `s` must carry the fused layout.  With
// `pre->val` the first phase takes the selection from there and `logits` is not read; with `pre->psum` and
// no selection the first phase also adds up the softmax values itself (rr_route_loss).
cudaError_t launch_route_fused(const float *logits, int T, int E, int k, int C, int G, unsigned mode,
                               const rr_route_tables &t, const RouteScratch &s, cudaStream_t st,
                               const RoutePresel *pre = nullptr);

// Argument rules of rr_route, shared by every entry point that routes.
rr_status check_route_shape(int T, int E, int k, int C, int G, unsigned mode);
rr_status check_route_tables(const rr_route_tables *t);

}  // namespace rr
