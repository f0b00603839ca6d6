/*
 * rr.h -- C ABI of librr: one rectified Mixture-of-Experts layer on one GPU
 * (Rectify-Router, arXiv 2402.12399).
 *
 * Conventions shared by every entry point
 *  - "dev" pointers are CUDA device pointers of the current device, "host"
 *    pointers are ordinary host memory.  All dev pointers must be 16-byte
 *    aligned; hidden / weight / dout tensors must be 128-byte aligned (they are
 *    read through TMA).  Everything is row-major and densely packed.
 *  - The caller owns and allocates every buffer, including the workspace.  The
 *    library allocates no device memory and keeps no state between calls other
 *    than lazily resolved driver entry points.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Work is
 *    enqueued asynchronously; functions return after argument checks and
 *    launches.  Conditions detected on the device (a non-finite logit, a bounded
 *    wait that ran out) are latched in a status word at the start of the
 *    workspace and are read back by rr_check.  Nothing traps, exits or throws.
 *    The first 256 bytes of a workspace must be zero when it is first used
 *    (zero-fill it once after allocating it); the library maintains them afterwards.
 *  - Token i belongs to group i / (T/G); group g owns experts
 *    [g*E/G, (g+1)*E/G) (uniform expert placement, Section 3 "Expert
 *    Parallelism").  Groups stand for the GPUs of the paper on one device.
 *  - Limits: 1 <= k <= 8, k <= E <= 256 (k < E with RR_FR), T % G == 0,
 *    E % G == 0, capacity >= 0, E*capacity + T < 2^31.
 */
#ifndef RR_H_
#define RR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int rr_status;
enum {
    RR_OK = 0,
    RR_ERR_INVALID_ARG = 1,        /* null / misaligned pointer, shape outside the limits   */
    RR_ERR_UNSUPPORTED = 2,        /* valid request this build has no kernel for            */
    RR_ERR_WORKSPACE_TOO_SMALL = 3,
    RR_ERR_CUDA = 4,               /* a CUDA runtime / driver call failed                   */
    RR_ERR_NONFINITE = 5,          /* device: a logit was NaN or Inf (tables are undefined) */
    RR_ERR_TIMEOUT = 6,            /* device: a bounded wait inside a kernel ran out        */
    RR_ERR_STATIC_SCRATCH_EXCEEDED = 7 /* rr_route_noalloc: shape needs more than its fixed scratch */
};

/* mode bits: the four routers of Tables 1-2 (0 = plain top-k) */
#define RR_IR 1u /* Intra-GPU Rectification, Section 4.1 */
#define RR_FR 2u /* Fill-in Rectification, Section 4.2   */
#define RR_SCORE 4u /* a full expert drops its lowest scores, not its latest tokens (Section 3's wording) */
#define RR_LOCAL_CAP 16u /* capacity per (source group, expert): C/G slots each; needs G | capacity */
#define RR_FR_SOFTMAX 8u /* FR ranks nominees by softmax value g_ie, not raw logit (Appendix A's wording); needs RR_FR */

/* flags of rr_moe_shape */
#define RR_GRAD_EXACT 1u /* exact gate gradient instead of the straight-through one (Appendix A) */

/* element type of hidden, W1, W3, W2, dout */
#define RR_BF16 0
#define RR_F32 1

/*
 * Routing tables (all dev, caller-allocated).  With K1 = k+1, K2 = k+2,
 * C = capacity, R = E*C + T:
 *
 *  topk_expert  [T,K1] i32  experts of token i by (logit desc, index asc) (Eq. 1); column k is
 *                           the (k+1)-th expert, FR's nominee (Section 4.2), -1 when E == k
 *  route_slot   [T,K1] i32  slot the routing obtained at that expert, -1 = dropped / not filled
 *  slot_token   [E,C]  i32  token held by each slot of each expert's queue, -1 = padding (Fig. 1)
 *  slot_rank    [E,C]  i8   which routing put it there: 0..k-1, k = fill-in, -1 = padding
 *  drop_count   [T]    i32  d_i = k - |R_i|, the token's dropped top-k routings (Section 3)
 *  ir_expert    [T]    i32  IR expert h_i inside the token's group, -1 if none (Section 4.1)
 *  ir_pos       [T]    i32  position in h_i's IR list (token order), -1 if none
 *  ir_offset    [E+1]  i32  exclusive prefix of the IR list lengths
 *  ir_token     [T]    i32  IR lists back to back; -1 from ir_offset[E] on
 *  expert_count [E]    i32  occupied slots (kept + filled); they are slots 0..count-1
 *  n_routed     [E]    i32  top-k routings addressed to the expert before the capacity cut
 *  row_offset   [E+1]  i32  compact row space: expert e computes rows row_offset[e]..row_offset[e+1]-1,
 *                           its occupied slots in slot order followed by its IR list
 *  row_token    [R]    i32  token of each row, -1 from row_offset[E] on
 *  row_weight   [R]    f32  combine weight of each row, 0 from row_offset[E] on
 *  token_rows   [T,K2] i32  row of each route of token i, -1 if none; columns 0..k-1 top-k,
 *                           k fill-in, k+1 IR
 *  combine_w    [T,K2] f32  combine weights, same columns (Eq. 2, Eq. 3); rows sum to 1 or are 0
 */
typedef struct rr_route_tables {
    int32_t *topk_expert;
    int32_t *route_slot;
    int32_t *slot_token;
    int8_t *slot_rank;
    int32_t *drop_count;
    int32_t *ir_expert;
    int32_t *ir_pos;
    int32_t *ir_offset;
    int32_t *ir_token;
    int32_t *expert_count;
    int32_t *n_routed;
    int32_t *row_offset;
    int32_t *row_token;
    float *row_weight;
    int32_t *token_rows;
    float *combine_w;
} rr_route_tables;

/* Shape of one layer call. */
typedef struct rr_moe_shape {
    int32_t T, E, k, capacity, G; /* as for rr_route                                      */
    int32_t d, d_ff;              /* hidden width, expert FFN width; both multiples of 64 */
    int32_t dtype;                /* RR_BF16 or RR_F32                                    */
    uint32_t mode;                /* RR_IR | RR_FR | RR_SCORE | RR_FR_SOFTMAX | RR_LOCAL_CAP */
    uint32_t flags;               /* RR_GRAD_EXACT                                        */
    void *const *trace;           /* NULL, or host array of 8 cudaEvent_t recorded on `stream`
                                     around the kernels of the call (timing aid):
                                     rr_moe_fwd: [0] start, [1] after gate/up GEMM, [2] after down GEMM
                                     rr_moe_bwd: [0] start, [1] dAct GEMM, [2] dX GEMM, [3] weight
                                     gradients, [4] gate gradient                          */
} rr_moe_shape;

/* Bytes of workspace rr_route needs for this shape (host out-parameter). */
rr_status rr_route_workspace_bytes(int T, int E, int k, int capacity, int G, unsigned mode,
                                   size_t *bytes /* host */);

/*
 * rr_route -- top-k routing under a per-expert capacity with the two rectifications
 * (Section 3 Eq. 1-2 and "Dropped Tokens and Padding"; Section 4.1 Eq. 3; Section 4.2).
 *
 *  logits   [T,E] fp32 dev: a_ij, read only.
 *  capacity slots per expert, applied over all T tokens.  Routings are served first-routing
 *           before second-routing, and in token order inside one routing; what does not fit is
 *           dropped, what stays empty is padding.
 *  mode     RR_IR: a token with >= 1 dropped routing is sent once, without capacity limit, to
 *           the highest-logit expert of its own group, weighted by its number of drops (Eq. 3).
 *           RR_FR: every token nominates its (k+1)-th expert; each expert gives its padding
 *           slots to the nominees with the highest logit (ties: lower token), placed after the
 *           kept tokens in ascending token order.
 *           RR_SCORE: the other reading of Section 3 (overflow costs an expert its lowest-scoring
 *           tokens): ranks are still served one after the other, but when the r-th choices
 *           addressed to an expert exceed what is left of its capacity, those with the highest
 *           logit stay (ties: lower token), in ascending token order from the next free slot on;
 *           IR and FR then apply as above.  Not accepted by rr_route_noalloc.
 *           RR_FR_SOFTMAX (with RR_FR): the other reading of "routing score" in Section 4.2 --
 *           Appendix A gives that name to the softmax values g_ie = e^{a_ie} / sum_j e^{a_ij}.
 *           Each expert ranks its nominees by g_ie instead of a_ie (ties: lower token); all else is
 *           unchanged.  g is computed in single precision by a recipe whose every operation is
 *           fixed, so the tables stay unique: m = max_j a_ij; t_j = max(a_ij - m, -80);
 *           n = rint(t_j * 0x1.715476p+0); r = fma(-n, 0x1.62e4p-1, t_j); r = fma(-n, 0x1.7f7d1cp-20, r);
 *           p = degree-7 Taylor polynomial of e^r in Horner form with fma, coefficients 1/q! rounded
 *           to single precision; e_j = p * 2^n; Z = e_0 + e_1 + ... in index order; g = e_e / Z; every
 *           operation rounds to nearest even.  Not accepted by rr_route_noalloc.
 *           RR_LOCAL_CAP (capacity a multiple of G): the capacity as a device sees it that routes
 *           only its own T/G tokens (Section 3 places the experts on G devices and derives the
 *           capacity from the number of tokens).  Every expert grants each source group capacity/G
 *           slots of its own: slots [g*capacity/G, (g+1)*capacity/G) belong to group g, and queues,
 *           drops, padding, fill-in (and RR_SCORE's selection) are all counted per (group,
 *           expert), as if G routers ran side by side; IR is unchanged.  An expert's occupied slots
 *           are then a prefix of every segment rather than of the whole row; expert_count is their
 *           total and the rows of the compact row space still follow slot order.  Not accepted by
 *           rr_route_noalloc.
 *  Ties everywhere go to the lower expert / token index; comparisons are on raw fp32 logits
 *  (-0 == +0).  The result is unique: two runs give identical tables.
 *
 *  out      host struct of dev pointers; every table is completely overwritten.
 *  workspace dev, >= rr_route_workspace_bytes; scratch, except that its first 256 bytes hold
 *           the status word read by rr_check and the words of the routing kernel's grid barrier
 *           (zero when the workspace is first used; every call leaves them zero again).
 * Returns RR_OK or RR_ERR_INVALID_ARG / RR_ERR_WORKSPACE_TOO_SMALL / RR_ERR_CUDA.  Logits that
 * are not finite (a NaN, an infinity, whole rows of them) make the tables undefined -- but every
 * index stays in range and nothing faults -- and latch RR_ERR_NONFINITE.  T == 0 is accepted.
 * Up to 2^22 tokens and without RR_SCORE / RR_LOCAL_CAP the call is ONE kernel, launched
 * cooperatively with at most one block per SM (the blocks meet at grid-wide barriers, so the device
 * must be able to hold them all at once: do not run it beside kernels that occupy SMs indefinitely).
 * Every wait inside has a time limit; one that runs out latches RR_ERR_TIMEOUT and the tables are
 * undefined.  Calls that share a workspace must not overlap on the GPU.
 */
rr_status rr_route(const float *logits /* dev */, int T, int E, int k, int capacity, int G,
                   unsigned mode, const rr_route_tables *out /* host struct, dev pointers */,
                   void *workspace /* dev */, size_t workspace_bytes, void *stream);

/*
 * rr_route_noalloc -- rr_route without a caller-provided workspace.  (The paper has no
 * counterpart for this entry point; it exists for integration reasons only.)
 *
 * Who needs it: callers that cannot obtain device memory at the time they must route -- code
 * inside a latency-critical or stream-ordered section that must not hit cudaMalloc's implicit
 * synchronisation, extensions that receive buffers but no allocator, or processes whose device
 * memory is already fully handed out.  The scratch rr_route would take from `workspace` lives in
 * a fixed 4 MiB array inside the library image instead (held by every GPU that loads the library
 * until the process ends).  Nothing is allocated or freed by this call.
 *
 * Arguments and results are those of rr_route (same kernels, identical tables), except:
 *  status   dev, 16-byte aligned, at least 4 bytes, zero-filled once by the caller, or NULL.
 *           Device-detected conditions (RR_ERR_NONFINITE, RR_ERR_TIMEOUT) are latched there; pass
 *           the same pointer to rr_check to read them.  With NULL they are latched inside the fixed
 *           array (cleared at the start of every call) and cannot be read back.
 * Limits: shapes whose scratch exceeds the fixed array are refused with
 * RR_ERR_STATIC_SCRATCH_EXCEEDED before anything is launched (T = 65536, E = 64, k = 2 fits;
 * the need grows with T*(k+1) and with T/256 * (k+1) * E).
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress);
 * make that first call outside any stream capture.  The address is kept for the life of the
 * device's primary context; after cudaDeviceReset the library must be reloaded.
 * All calls on a device share the one array: two calls whose kernels overlap on the GPU
 * (different streams, no ordering between them) race on it and corrupt each other's tables.
 * Calls on one stream, or otherwise ordered, are safe.
 */
rr_status rr_route_noalloc(const float *logits /* dev */, int T, int E, int k, int capacity, int G,
                           unsigned mode, const rr_route_tables *out, void *status /* dev or NULL */,
                           void *stream);

/* Workspace bytes of rr_moe_fwd / rr_moe_bwd and bytes of the `saved` buffer (host outs). */
rr_status rr_moe_workspace_bytes(const rr_moe_shape *s /* host */, size_t *fwd_bytes,
                                 size_t *bwd_bytes, size_t *saved_bytes);

/*
 * rr_moe_fwd -- expert computation and combine for tables made by rr_route with the same
 * T, E, k, capacity, G, mode:
 *     out_i = sum over the live routes r of token i of  w_r * E_{e_r}(x_i)      (Eq. 2, Eq. 3)
 *     E_j(x) = W2_j ( silu(W1_j x) * (W3_j x) ),  no biases  (Section 5.1: experts are copies
 *     of the LLaMA2 FFN).
 * Only live rows are computed (padding slots cost nothing); tokens without a live route get 0:
 * their residual connection is outside this layer.
 *
 *  hidden [T,d]; W1, W3 [E,d_ff,d]; W2 [E,d,d_ff]   dev, element type s->dtype, read only
 *  logits [T,E] fp32 dev (unused by the forward pass; kept for symmetry, may be NULL)
 *  out    [T,d] fp32 dev, overwritten
 *  saved  dev, saved_bytes, or NULL for inference: what rr_moe_bwd needs of this pass (the fp32
 *         pre-activations W1_j x, W3_j x of every live row and the token rows in expert order).
 *         RR_BF16 layers only; ignored for RR_F32, which has no backward pass (saved_bytes = 0)
 *  workspace dev, >= fwd_bytes (scratch; its first 256 bytes hold the status word)
 * bf16 inputs are multiplied on the tensor cores with fp32 accumulation; fp32 inputs are
 * multiplied as tf32.  The combine adds rows with floating-point atomics, so the low bits of
 * `out` may differ from run to run.  T == 0 is accepted and does nothing.
 */
rr_status rr_moe_fwd(const rr_moe_shape *s, const void *hidden, const void *W1, const void *W3,
                     const void *W2, const float *logits, const rr_route_tables *tables,
                     float *out, void *saved, void *workspace, size_t workspace_bytes,
                     void *stream);

/*
 * rr_moe_bwd -- gradients of L for given dL/dout (Appendix A for the gate):
 *  dhidden [T,d] fp32   through the experts only (the gate projection is the caller's)
 *  dlogits [T,E] fp32   straight-through by default: the normaliser S_i = sum_r mu_r g_{i,e_r}
 *                       (g = softmax over all E experts) is held constant, so
 *                       dL/dg_ij = sum_{r:e_r=j} mu_r <dout_i, E_j(x_i)> / S_i flows through the
 *                       full softmax (Eq. 6); with RR_GRAD_EXACT the quotient is differentiated
 *                       exactly (zero for single-route tokens).
 *  dW1, dW3 [E,d_ff,d], dW2 [E,d,d_ff] fp32, overwritten (not accumulated)
 *  dout [T,d] element type s->dtype; saved = buffer filled by rr_moe_fwd on the same inputs and tables
 *  (it holds the token rows the pass needs, so `hidden` is checked but not read).
 * T == 0 is accepted: the weight gradients are set to zero, nothing else is touched.
 * RR_BF16 only: with RR_F32 the call returns RR_ERR_UNSUPPORTED before anything is launched, and
 * rr_moe_workspace_bytes reports bwd_bytes = 0 and saved_bytes = 0 for such a shape.
 */
rr_status rr_moe_bwd(const rr_moe_shape *s, const void *dout, const void *hidden, const void *W1,
                     const void *W3, const void *W2, const float *logits,
                     const rr_route_tables *tables, const void *saved, float *dhidden,
                     float *dlogits, float *dW1, float *dW3, float *dW2, void *workspace,
                     size_t workspace_bytes, void *stream);

/*
 * Gate projection (Section 3, Eq. 1): the routing score of token i at expert j is the inner
 * product of the expert's embedding vector with the token's hidden state,
 *     a_ij = w_j^T x_i ,       logits[T,E] = hidden[T,d] . Wg[E,d]^T .
 * rr_gate_fwd writes the fp32 logits that rr_route takes.  bf16 inputs are multiplied exactly
 * and accumulated in fp32 on the tensor cores; fp32 inputs are multiplied as tf32.
 *   hidden [T,d], Wg [E,d]  dev, element type `dtype` (RR_BF16 / RR_F32), 128-byte aligned
 *   logits [T,E] fp32 dev, overwritten
 *   workspace dev, >= fwd_bytes of rr_gate_workspace_bytes; its first 256 bytes hold the status
 *   word (zero them once; rr_check reads it)
 * d must be a multiple of 64, E <= 256.  T == 0 does nothing.
 *
 * rr_gate_bwd, for given dL/da (e.g. the dlogits of rr_moe_bwd):
 *   dWg     [E,d] fp32, overwritten:       dL/dw_j = sum_i dL/da_ij x_i   (summed over slabs of
 *           tokens in a fixed order: the result repeats bit for bit)
 *   dhidden [T,d] fp32, ADDED TO:          dL/dx_i += sum_j dL/da_ij w_j  (pass the dhidden of
 *           rr_moe_bwd to complete it with the path through the gate)
 *   workspace dev, >= bwd_bytes, 256-byte aligned (scratch; its first word is a status word that the call
 *           clears and rr_check reads)
 * bf16 inputs run on the tensor cores: dlogits is split into a bf16 head and a bf16 remainder (16
 * mantissa bits together), dhidden += [head | rem] . [Wg ; Wg] is one GEMM whose 32 x 32 result tiles are
 * added to dhidden by TMA reductions, dWg = head^T hidden + rem^T hidden a GEMM over slabs of tokens
 * whose partial sums are added in slab order.  fp32 inputs use fp32 arithmetic on the CUDA cores.
 */
rr_status rr_gate_workspace_bytes(int T, int E, int d, size_t *fwd_bytes, size_t *bwd_bytes);
rr_status rr_gate_fwd(int T, int E, int d, int dtype, const void *hidden, const void *Wg, float *logits,
                      void *workspace, size_t workspace_bytes, void *stream);
rr_status rr_gate_bwd(int T, int E, int d, int dtype, const float *dlogits, const void *hidden,
                      const void *Wg, float *dWg, float *dhidden, void *workspace,
                      size_t workspace_bytes, void *stream);

/*
 * rr_gate_route -- the gate projection (Eq. 1), the routing of rr_route (Sections 3, 4.1, 4.2) and,
 * if wanted, the load-balance loss (Section 5.1) with the selection made where the scores are
 * produced: the projection's epilogue picks every token's k+1 best experts (score desc, index asc)
 * and the best expert of its group straight from the fp32 accumulators and sums the softmax values
 * per expert, so `logits` is written once (rr_moe_bwd and rr_aux_loss_bwd need it) and never read
 * back; the routing kernel then starts from those records.  Two launches in all.
 *   hidden [T,d], Wg [E,d]  dev, element type `dtype`, 128-byte aligned; d a multiple of 64
 *   logits [T,E] fp32 dev, overwritten: bit for bit what rr_gate_fwd writes
 *   out      routing tables, exactly those of rr_route on `logits`
 *   mode     RR_IR | RR_FR; the other mode bits and T > 2^22 return RR_ERR_UNSUPPORTED (use
 *            rr_gate_fwd + rr_route)
 *   loss [1], f [E], P [E] fp32 dev or all NULL: L = alpha * E * sum_e f_e P_e as rr_aux_loss_fwd defines
 *            it (f from the first choices before the capacity cut, P the mean softmax value; fp32, every
 *            sum in a fixed order)
 *   workspace dev, >= rr_gate_route_workspace_bytes, 256-byte aligned; its first 256 bytes are the header
 *            of rr_route's workspace (zero when first used; rr_check reads the status word)
 * A hidden state or weight that makes a score non-finite latches RR_ERR_NONFINITE.  T == 0 is accepted.
 */
rr_status rr_gate_route_workspace_bytes(int T, int E, int k, int capacity, int G, unsigned mode, int d,
                                        size_t *bytes);
rr_status rr_gate_route(int T, int E, int k, int capacity, int G, unsigned mode, int d, int dtype,
                        const void *hidden, const void *Wg, float *logits, const rr_route_tables *out,
                        float alpha, float *loss, float *f, float *P, void *workspace,
                        size_t workspace_bytes, void *stream);

/*
 * Load-balance loss of the top-k router (Section 5.1 sets its weight to 1e-2; Appendix "Impact of
 * Load-Balance Loss" compares training with and without it).  The paper prints no formula; this is
 * the one of the work it cites there:
 *     f_e = (1/T) #{ i : the first choice of token i is expert e }      (before the capacity cut)
 *     P_e = (1/T) sum_i g_ie,   g_i = softmax(a_i) over all E experts
 *     L   = alpha * E * sum_e f_e P_e            (alpha for uniform scores, alpha*E at collapse)
 * rr_aux_loss_fwd:
 *   logits       [T,E] fp32 dev, 16-byte aligned (finite: rr_route reports others)
 *   first_choice dev i32, element i*stride is the rank-0 expert of token i: pass
 *                tables->topk_expert with stride = k+1; a value outside 0..E-1 latches
 *                RR_ERR_INVALID_ARG in the workspace header
 *   loss [1], f [E], P [E] fp32 dev, overwritten (P may be null)
 *   workspace dev, 256-byte aligned, >= rr_aux_workspace_bytes; first 256 bytes = status word
 *   fp32 arithmetic; the sums over tokens are taken in a fixed order, so results repeat bit for bit.
 *   T == 0 sets loss, f and P to zero.
 * rr_aux_loss_bwd, with the counts f held constant (they are piecewise constant in a):
 *   dL/da_ij = scale * alpha * E / T * g_ij * ( f_j - sum_e f_e g_ie )
 *   f [E] dev as written by rr_aux_loss_fwd; scale = d(total loss)/dL, a host value
 *   dlogits [T,E] fp32 dev, 16-byte aligned: overwritten when accumulate == 0, added to otherwise (e.g. onto the
 *   dlogits of rr_moe_bwd before rr_gate_bwd).  Launches one kernel, needs no workspace.
 */
rr_status rr_aux_workspace_bytes(int T, int E, size_t *bytes);

/*
 * rr_route_loss -- rr_route and rr_aux_loss_fwd in the one routing kernel (Sections 3, 4.1, 4.2 and
 * Section 5.1): the pass that reads logits[T,E] for the selection also adds up the softmax values per
 * expert, and the first-choice counts are the totals the capacity scan needs anyway, so the logits are
 * read once.  Arguments as for rr_route, plus alpha and the outputs loss [1], f [E], P [E] (fp32 dev,
 * all required) as for rr_aux_loss_fwd; workspace >= rr_route_loss_workspace_bytes.  The tables are those
 * of rr_route bit for bit; f, P, L agree with rr_aux_loss_fwd within its tolerances (hardware
 * exponentials here; every sum in a fixed order, so the numbers repeat).  RR_SCORE, RR_LOCAL_CAP and
 * T > 2^22 return RR_ERR_UNSUPPORTED (call rr_route and rr_aux_loss_fwd).
 */
rr_status rr_route_loss_workspace_bytes(int T, int E, int k, int capacity, int G, unsigned mode,
                                        size_t *bytes);
rr_status rr_route_loss(const float *logits, int T, int E, int k, int capacity, int G, unsigned mode,
                        const rr_route_tables *out, float alpha, float *loss, float *f, float *P,
                        void *workspace, size_t workspace_bytes, void *stream);
rr_status rr_aux_loss_fwd(int T, int E, int stride, const float *logits, const int32_t *first_choice,
                          float alpha, float *loss, float *f, float *P, void *workspace,
                          size_t workspace_bytes, void *stream);
rr_status rr_aux_loss_bwd(int T, int E, const float *logits, const float *f, float alpha, float scale,
                          int accumulate, float *dlogits, void *stream);

/*
 * rr_check -- synchronise `stream`, then return the status word latched in `workspace`
 * (RR_OK, RR_ERR_NONFINITE, RR_ERR_TIMEOUT) or RR_ERR_CUDA if the stream reports an error.
 * The first error latched since the last rr_check is kept; rr_check clears it after reporting.
 */
rr_status rr_check(const void *workspace /* dev */, void *stream);

/*
 * rr_test_set_wait_limit_ns -- testing aid (the paper has no counterpart).  Every wait inside the
 * kernels has a time limit (2 s) after which the kernel latches RR_ERR_TIMEOUT, lets go of what it
 * holds and returns, leaving the CUDA context usable.  A non-zero `ns` replaces that limit, for the
 * launches made afterwards by this process, in the waits a test can make run out without breaking
 * anything: the grid barriers of the routing kernel and the accumulator wait in the epilogue of
 * rr_moe_fwd's GEMMs (a limit of a few ns expires while the awaited work is still running).  0 restores
 * the 2 s.  Host-side state, not thread-safe; results of a call that timed out are undefined.
 */
void rr_test_set_wait_limit_ns(unsigned long long ns);

/* Static, NUL-terminated description of a status code. */
const char *rr_status_string(rr_status s);

#ifdef __cplusplus
}
#endif
#endif /* RR_H_ */
