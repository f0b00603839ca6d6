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

// Workspace header, first bytes of every workspace.
struct Header {
    int status;  // latched rr_status detected on the device (0 = none)
    int pad[63];
};

__device__ __forceinline__ void latch_status(int *status, int code) { atomicCAS(status, 0, code); }

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

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

// Scratch of the routing kernels (device pointers into the workspace).
struct RouteScratch {
    Header *hdr;
    float *val;         // [T,K1] logits of the top-(k+1) experts
    int *h;             // [T]    in-group best expert
    float *a_h;         // [T]    its logit
    int *pos_local;     // [T,K1] position among same-(rank,expert) tokens of the tile
    int *hist;          // [K1*E,tiles] per-tile counts (column-major), then exclusive prefix over tiles
    int *totals;        // [segs,K1,E] counts over the tiles of each capacity segment
    uint32_t *nom_key;  // [T]    order-preserving keys of nominee logits, expert after expert
                        //        ([K1,T] with RR_SCORE: the candidates of every rank, rank after rank)
    int *nom_token;     // same shape: their tokens
    int *ir_local;      // [T]    position among the tile's IR tokens of the same expert, -1 none
    int *ir_hist;       // [E,tiles] per-tile IR counts (column-major), then exclusive prefix over tiles
    int *ir_totals;     // [E] IR list lengths
    float *fr_key;      // [T] with RR_FR_SOFTMAX: softmax value of the token at the expert it nominates
    int *seg_n;         // [segs,E] top-k routings addressed to the expert from the segment's tokens
    int *seg_occ;       // [segs,E] occupied slots of the expert inside the segment (kept, then + filled)
    int tiles;          // segs * tps
    // Capacity segments: one over all tokens, or with RR_LOCAL_CAP one per source group.  Segment sg
    // serves tokens [sg*Tseg, (sg+1)*Tseg) with tiles [sg*tps, (sg+1)*tps) (no tile spans two segments)
    // and owns slots [sg*C/segs, (sg+1)*C/segs) of every expert.
    int segs, tps, Tseg;
};

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

}  // namespace rr
