/*
 * pquant.h -- C ABI of the B200 (sm_100a) pQuant decoupled linear layer.
 *
 * The layer (paper Sec. 3.1-3.3) replaces a projection Y = W X by
 *
 *     Y[t,n] = alpha_n * g_t * (B_e A_e x_t)[n]  +  beta_n * (lam / gamma_t) * sum_k S[n,k] q[t,k]
 *
 * with S = Sign(W - mu) (Eq. 3-4), mu = mean W, lam = mean |W| (Eq. 6),
 * q = RoundClip(x * gamma_t) in int8 with gamma_t = 2^7 / max_k |x_tk| (Eq. 7-9),
 * the 1-bit product de-quantised by lam / gamma_t (Eq. 10), the two branches
 * summed under the feature scales alpha, beta (Eq. 11), and the high-precision
 * (HP) branch A_e (r x K), B_e (N x r) chosen per token by a top-1 softmax
 * router, e = argmax_j (Wr x_t)_j, g_t = softmax(Wr x_t)_e (Sec. 3.3).
 * The backward pass is the straight-through estimator of App. B.1.
 *
 * Conventions common to every entry point
 *   - every data pointer is a DEVICE pointer owned by the caller; the library
 *     never allocates or frees device memory and keeps no pointer into the
 *     caller's memory between calls.  What it does keep, per process: a few
 *     small file-scope device variables (a status word, the spin limit, the
 *     64 KiB array of pq_pack_weights_static), and -- unless PQ_OPT_SIDE_STREAM
 *     is 0 -- one helper stream and three events per (device, caller stream)
 *     that has called pq_linear_forward / pq_linear_backward, created on first
 *     use and kept until the process exits;
 *   - work is only enqueued on `stream` (a cudaStream_t passed as void*) and on
 *     that helper stream, which is joined back into `stream` inside the same
 *     call; no call synchronises the device except pq_device_status and
 *     pq_set_option(PQ_OPT_SPIN_CYCLES);
 *   - threads: calls on different streams may come from different host threads;
 *     the helper-stream table is locked.  pq_set_option, pq_profile_events and the
 *     launch counter behind pq_kernel_launches are plain process-wide state without
 *     locks: set options and register events while no other thread is inside the
 *     library, and read the counter as an approximate figure under concurrency;
 *   - the return value is a status: PQ_OK (0) or a negative PQ_ERR_* code.
 *     Nothing is thrown.  After an error the outputs are undefined;
 *   - matrices are dense row-major: X[T,K] bf16, latent W[N,K] fp32,
 *     A[E,r,K] bf16, B[E,N,r] bf16, Wr[E,K] bf16, Y[T,N] bf16.  bf16 is passed
 *     as uint16_t bit patterns.  All base pointers must be 16-byte aligned;
 *   - alpha / beta hold one float (the paper's scalars) or N floats when
 *     PQ_SCALE_VECTOR is set in pq_desc.flags;
 *   - kernels wait on hardware barriers with a bounded spin; if a wait runs
 *     out the kernel records a code in a device status word that
 *     pq_device_status() reads back (PQ_ERR_TIMEOUT).
 */
#ifndef PQUANT_H_
#define PQUANT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  PQ_OK = 0,
  PQ_ERR_NULL = -1,        /* a required pointer is NULL                        */
  PQ_ERR_SHAPE = -2,       /* a size violates the documented constraints        */
  PQ_ERR_ALIGN = -3,       /* a pointer is not 16-byte aligned                  */
  PQ_ERR_WORKSPACE = -4,   /* workspace / saved buffer too small                */
  PQ_ERR_UNSUPPORTED = -5, /* valid request this build does not implement       */
  PQ_ERR_CUDA = -6,        /* a CUDA runtime / driver call failed               */
  PQ_ERR_TIMEOUT = -7,     /* a device-side bounded wait ran out                */
  PQ_ERR_TOO_LARGE = -8    /* problem needs more scratch than a fixed-size buffer holds */
};

enum {
  PQ_SCALE_VECTOR = 1u,    /* pq_desc.flags: alpha, beta have N entries instead of 1                      */
  PQ_DECODE_DUMP_ACC = 2u, /* decode only, test hook: also write the exact int32 sums of the 1-bit product */
  PQ_UNIT_GATES = 4u,      /* with top_k = E: every expert active with gate 1 (test mode, see pq_desc.top_k)     */
  PQ_FUSED_RMSNORM = 8u    /* training path: the layer is called through pq_linear_forward_rms (sizes `saved`) */
};

enum { PQ_PHASE_PACK = 0, PQ_PHASE_FWD = 1, PQ_PHASE_BWD = 2, PQ_PHASE_DECODE = 3 };

/* Shape of one layer.  Constraints: T >= 1; K, N multiples of 32 (bit words,
 * 16-byte rows); r == 0 (pure 1-bit layer, the paper's attention projections,
 * E ignored) or r a multiple of 8 with 8 <= r <= 256 and 1 <= E <= 16;
 * top_k = 1 (the paper's gating).  The training path additionally needs r <= 128.
 * One more value of top_k is taken, as a test mode of the training-size forward (pq_linear_forward with w_s8,
 * pq_saved_bytes, pq_workspace_bytes(PQ_PHASE_FWD)): top_k = E > 1 with PQ_UNIT_GATES in flags and E r <= 128 --
 * every expert is active with weight one and the router is not read (Wr may be NULL), so the layer must equal the
 * dense layer of width E r whose A is the experts' rows stacked and whose B is their columns side by side (the
 * special case in which routing reduces to a dense branch, Sec. 3.3).  `saved` then has the dense layer's layout;
 * pq_linear_backward, the decode path and the other forward variants return PQ_ERR_UNSUPPORTED for such a desc. */
typedef struct pq_desc {
  uint32_t size;  /* sizeof(pq_desc), checked */
  uint32_t flags;
  int32_t T, K, N;
  int32_t r, E, top_k;
} pq_desc;

/* Host-side view into the caller-allocated `saved` buffer that the training
 * forward fills and the backward reads (filled by pq_saved_view; all device
 * pointers into that buffer).  "sorted order": row p holds token perm[p];
 * tokens are sorted by expert, stably (the permutation implied by Sec. 3.3's
 * sparse activation).  With E <= 1 the permutation is the identity. */
typedef struct pq_saved_view {
  int8_t* q;          /* [T,K]  int8 activations, sorted order (Eq. 7)                 */
  uint16_t* xt;       /* [T,K]  bf16 q/gamma, sorted order (backward operand)          */
  uint16_t* xs;       /* [T,K]  bf16 copy of X in sorted order; NULL when E <= 1       */
  float* gamma;       /* [T]    gamma_t, sorted order (Eq. 9)                          */
  float* gate;        /* [T]    g_t, sorted order                                      */
  float* probs;       /* [T,E]  router softmax, sorted order; NULL when E <= 1         */
  int32_t* expert;    /* [T]    e_t, TOKEN order                                       */
  int32_t* perm;      /* [T]    perm[p] = token at sorted position p                   */
  int32_t* pos;       /* [T]    inverse: pos[token] = p                                */
  int32_t* offsets;   /* [E+1]  sorted positions of expert e: offsets[e]..offsets[e+1] */
  uint16_t* h;        /* [2][max_items*128, r] bf16 HP hidden activations as hi/lo planes (h = hi + lo),
                         one 128-row block per item in each plane */
  /* Item table.  An item is the intersection of one 128-row tile of the sorted
   * order with one expert's range; rows of an item's block outside that range
   * are zero.  items[i] = {tile, expert, first row, end row} (rows relative to
   * the tile).  Items are ordered by tile, hence by expert. */
  int32_t* n_items;            /* [1]                                          */
  int32_t* items;              /* [max_items][4]                               */
  int32_t* tile_item_begin;    /* [ceil(T/128)+1] first item of each tile      */
  int32_t* expert_item_begin;  /* [E+1] first item of each expert              */
  int32_t max_items;           /* ceil(T/128) + max(E,1) - 1                   */
} pq_saved_view;

/* Bytes the caller must provide. */
size_t pq_workspace_bytes(const pq_desc* d, int phase);
size_t pq_saved_bytes(const pq_desc* d);
int pq_saved_view_init(const pq_desc* d, void* saved, pq_saved_view* out);

/* Offline / per-step weight quantisation (Eq. 3, 4, 6; storage App. A).
 *   W        [N,K] fp32 latent weights (in)
 *   w_bits   [N,K/32] uint32 (out): bit j of word i of a row <-> k = 32 i + j, 1 <-> +1
 *            (as bytes: the paper's 8 weights per uint8, LSB first)
 *   w_s8     [N,K] int8 +-1 (out), may be NULL for an inference-only pack
 *   w_scales [2] float (out) = { lam, mu }, fp64-accumulated, rounded once
 *   ws       workspace of pq_workspace_bytes(d, PQ_PHASE_PACK) bytes
 * Only d->N and d->K are read. */
int pq_pack_weights(const pq_desc* d, const float* W, uint32_t* w_bits, int8_t* w_s8,
                    float* w_scales, void* ws, size_t ws_bytes, void* stream);

/* Weight quantisation for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of pq_pack_weights.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a serving
 * process whose device memory is handed out once at start-up by another
 * component, a plug-in running inside someone else's memory pool, a section of
 * a program that must not trigger the implicit synchronisation an allocation
 * causes.  Such a caller still owns W and the three outputs, but has nowhere to
 * get the reduction workspace pq_pack_weights asks for.  Here that workspace is a
 * fixed 64 KiB array inside the library (a file-scope device array: every GPU
 * that loads the library holds those 64 KiB until the process exits).
 *
 * Same inputs, outputs and results as pq_pack_weights, minus ws / ws_bytes.
 *   - Limit: N * K <= 67,108,864 elements (4096 slabs of 16384 elements, one
 *     pair of fp64 partial sums each).  Larger matrices get PQ_ERR_TOO_LARGE and
 *     nothing is launched.
 *   - The call makes no cudaMalloc / cudaFree and uses no allocating routine.
 *   - The first call on each device looks up the array's device address (a
 *     one-off host-side query); make that first call outside any stream capture.
 *   - All calls share the one array.  Nothing in it has to start at zero -- each
 *     call overwrites the slots it later reads -- but two calls whose kernels
 *     overlap on the GPU (different streams) would overwrite each other's
 *     partial sums: keep calls on one device in stream order.
 *   - lam and mu are summed slab by slab instead of grid-strided, so they can
 *     differ from pq_pack_weights in the last fp64 bit before the one rounding to
 *     fp32; in practice the outputs are identical. */
int pq_pack_weights_static(const pq_desc* d, const float* W, uint32_t* w_bits, int8_t* w_s8,
                           float* w_scales, void* stream);

/* INT8 high-precision branch (Sec. 3.2: the branch runs at 8-bit precision, its weights quantised the way the
 * 8-bit activations are): Eq. 7-9 applied to each expert matrix as a whole,
 *     gamma = 2^7 / max(max|w|, 1e-5),   code = clamp(rint(w * gamma), -128, 127)   (fp32, round half to even).
 *   A [E,r,K], B [E,N,r] bf16 (in);  A8 [E,r,K], B8 [E,N,r] int8 (out);
 *   hp_scales [E][2] float (out) = { gamma_A_e, gamma_B_e };
 *   ws: workspace of pq_workspace_bytes(d, PQ_PHASE_PACK) bytes.
 * r * K and N * r must be multiples of 8 (they are: r is a multiple of 8). */
int pq_pack_experts(const pq_desc* d, const uint16_t* A, const uint16_t* B, int8_t* A8, int8_t* B8, float* hp_scales, void* ws,
                    size_t ws_bytes, void* stream);

/* Forward of the layer (Eq. 10-11, Sec. 3.3).
 *   training (w_s8 != NULL): tensor-core path; fills `saved` (may be NULL when
 *     no backward follows).  A, B may be NULL iff r == 0; Wr NULL iff E <= 1.
 *   decode (w_s8 == NULL): T <= 16 tokens straight from the packed bits w_bits
 *     (App. A): two kernels bound by the bytes of the weights.  `saved` is ignored,
 *     ws needs pq_workspace_bytes(d, PQ_PHASE_DECODE) bytes.  r <= 256; K and N such
 *     that one SM's share of the bits and expert rows fits its shared memory
 *     (PQ_ERR_UNSUPPORTED otherwise; the 3B-shaped 3200 x 8640 layers fit).  The two
 *     kernels are launched with programmatic stream serialisation, so consecutive
 *     decode calls on one stream overlap their prologues. */
int pq_linear_forward(const pq_desc* d, const uint16_t* X, const uint32_t* w_bits,
                      const int8_t* w_s8, const float* w_scales, const uint16_t* A,
                      const uint16_t* B, const uint16_t* Wr, const float* alpha,
                      const float* beta, uint16_t* Y, void* saved, size_t saved_bytes, void* ws,
                      size_t ws_bytes, void* stream);

/* Training-size forward with RMSNorm fused in front of the activation quantiser (App. A: the norm merges with the
 * quantisation, both being element-wise).  X is the UN-normalised activation; every use of a token -- quantiser, router,
 * HP branch -- sees
 *     bf16( fp32( fp32(x * s_t) * norm_weight_k ) ),   s_t = fp32( 1 / sqrt(mean_k x^2 + norm_eps) )   (mean, root in fp64),
 * the values a separate bf16 norm layer would have handed over, which never exist in memory except as the sorted copy
 * `xs` in `saved`.  d->flags must carry PQ_FUSED_RMSNORM (it sizes `saved` and the workspace: query them with the same
 * desc); norm_weight [K] bf16, norm_eps > 0.  pq_linear_backward with the same desc then takes the layer's input from
 * `saved` (its X argument is not read for the HP gradients) and returns dX with respect to the NORMALISED activation:
 * the norm's own backward belongs to the caller. */
int pq_linear_forward_rms(const pq_desc* d, const uint16_t* X, const uint16_t* norm_weight, float norm_eps, const int8_t* w_s8,
                          const float* w_scales, const uint16_t* A, const uint16_t* B, const uint16_t* Wr, const float* alpha,
                          const float* beta, uint16_t* Y, void* saved, size_t saved_bytes, void* ws, size_t ws_bytes, void* stream);

/* Forward with the paper's INT8 high-precision branch (Sec. 3.2), training-size path (tensor cores), forward only:
 * the branch multiplies the SAME int8 activation codes q the 1-bit branch uses,
 *     h_int = A8_e q_t (int32, exact);   qh, gamma_h = Eq. 7-9 on h_int (gamma_h = 2^7 / max_j |h_int|, from the integers);
 *     z_int = B8_e qh_t (int32, exact);  z = z_int / (gamma_B gamma_h gamma_A gamma_t);
 *     Y = alpha g z + beta (lam / gamma_t) acc                                    (Eq. 10-11)
 * with A8, B8, hp_scales from pq_pack_experts.  Arguments as pq_linear_forward; r must be a multiple of 16
 * (PQ_ERR_SHAPE otherwise), r <= 128.  With `saved` given, its h region holds the codes qh as int8
 * [max_items*128, r] followed (256-byte aligned) by gamma_h as float [max_items*128], rows per item as for h.
 * There is no INT8 backward: pq_linear_backward on a buffer saved by this call is not defined. */
int pq_linear_forward_hp8(const pq_desc* d, const uint16_t* X, const int8_t* w_s8, const float* w_scales, const int8_t* A8,
                          const int8_t* B8, const float* hp_scales, const uint16_t* Wr, const float* alpha, const float* beta,
                          uint16_t* Y, void* saved, size_t saved_bytes, void* ws, size_t ws_bytes, void* stream);

/* FFN-level decoupling, the form the paper trains (Eq. 11, Table 1): two parallel gated FFNs split along the hidden
 * dimension,
 *     Y = alpha * FFN_INT8[:r](x) + beta * FFN_INT1[r:](x),      FFN(x) = down( silu(gate x) * (up x) ),
 * the 1-bit FFN of hidden width F1 = D_ff - r made of three pure 1-bit linears (Eq. 3-10, each output a bf16 tensor,
 * inner feature scale 1), the INT8 FFN of hidden width r on the same int8 codes of x:
 *     g = (G8 q) / (gamma_G gamma_t), u = (U8 q) / (gamma_U gamma_t)   (exact int32 sums, de-quantised in fp32)
 *     m = silu(g) * u, with the logistic factor taken in fp64 and rounded once to fp32;  qm, gamma_m = Eq. 7-9 on m
 *     FFN_INT8 = (D8 qm) / (gamma_D gamma_m).
 * Forward only.  T >= 1; D, F1 multiples of 32; r a multiple of 16, 16 <= r <= 128 (PQ_ERR_SHAPE otherwise).
 *   X [T,D] bf16;  g_s8, u_s8 [F1,D], d_s8 [D,F1] int8 sign matrices and their {lam, mu} from pq_pack_weights;
 *   G8, U8 [r,D], D8 [D,r] int8 and hp_scales [3] = {gamma_G, gamma_U, gamma_D} (pq_pack_experts on (G, D) gives
 *   {gamma_G, gamma_D}, on (U, D) gives gamma_U);  alpha, beta: one float each;  Y [T,D] bf16;
 *   ws: pq_ffn_workspace_bytes(d) bytes.  The 1-bit FFN's hidden activation is bf16(silu(g1) * u1) in fp32. */
typedef struct pq_ffn_desc {
  uint32_t size, flags;   /* sizeof(pq_ffn_desc); flags must be 0 */
  int32_t T, D, F1, r;
} pq_ffn_desc;
size_t pq_ffn_workspace_bytes(const pq_ffn_desc* d);
int pq_ffn_forward(const pq_ffn_desc* d, const uint16_t* X, const int8_t* g_s8, const float* g_scales, const int8_t* u_s8,
                   const float* u_scales, const int8_t* d_s8, const float* d_scales, const int8_t* G8, const int8_t* U8,
                   const int8_t* D8, const float* hp_scales, const float* alpha, const float* beta, uint16_t* Y, void* ws,
                   size_t ws_bytes, void* stream);
/* What pq_ffn_forward leaves in its workspace, for tests: the bf16 outputs G1, U1 [T,F1] of the 1-bit gate and up
 * projections and their gated product M1; the exact sums g_int, u_int [ceil(T/128)*128, r] of the INT8 FFN; the codes
 * qm [.., r] and scales gamma_m of its hidden activation; the codes q_m1 [T,F1] and scales gamma_m1 of M1. */
typedef struct pq_ffn_view {
  uint16_t *G1, *U1, *M1;
  int32_t *g_int, *u_int;
  int8_t* qm;
  float* gamma_m;
  int8_t* q_m1;
  float* gamma_m1;
} pq_ffn_view;
int pq_ffn_view_init(const pq_ffn_desc* d, void* ws, pq_ffn_view* out);

/* What the decode path leaves in its workspace, for tests and diagnostics.  One entry per
 * token: the routed expert, its gate g_t, gamma_t (Eq. 9) and the sum over k of the int8 codes. */
typedef struct pq_decode_token {
  int32_t expert;
  float gate;
  float gamma;
  int32_t code_sum;
} pq_decode_token;
typedef struct pq_decode_view {
  pq_decode_token* tokens; /* [T] (device)                                                        */
  int32_t* acc;            /* [T,N] sum_k S[n,k] q[t,k] when PQ_DECODE_DUMP_ACC is set, else NULL */
  /* INT8 branch on the streaming kernel (pq_decode_item.A8): the exact integers it went through */
  int32_t* hp_h_int;       /* [T,r] h_int = A8_e q                                                 */
  int32_t* hp_z_int;       /* [T,N] z_int = B8_e qh when PQ_DECODE_DUMP_ACC is set, else NULL       */
} pq_decode_view;
int pq_decode_view_init(const pq_desc* d, void* ws, pq_decode_view* out);

/* Decode forward of several INDEPENDENT linears in one launch pair (App. A: at batch size
 * one the weights' bytes are the cost, so linears that do not depend on each other -- the
 * gate and up projections of a block, the q/k/v projections, other sequences -- should
 * stream their weights back to back instead of paying a launch and a pipeline fill each).
 * Each item is what pq_linear_forward takes in its decode form; results are identical to n
 * separate calls.  `items` is a HOST array, read before the call returns.  1 <= n <= 4096
 * (PQ_ERR_SHAPE otherwise; launched in groups of up to 96 consecutive items on the streaming kernel, of 16 on the
 * two-kernel path); every item needs its own ws. */
typedef struct pq_decode_item {
  pq_desc desc;            /* T <= 16 */
  const uint16_t* X;       /* [T,K] bf16 */
  const uint32_t* w_bits;  /* [N,K/32] */
  const float* w_scales;   /* {lam, mu} */
  const uint16_t* A;       /* [E,r,K] */
  const uint16_t* B;       /* [E,N,r] */
  const uint16_t* Wr;      /* [E,K], NULL if E <= 1 */
  const float* alpha;
  const float* beta;
  uint16_t* Y;             /* [T,N] bf16 (out) */
  void* ws;                /* pq_workspace_bytes(&desc, PQ_PHASE_DECODE) bytes */
  size_t ws_bytes;
  /* RMSNorm fused in front of the activation quantiser (App. A, Sec. 4.5: at inference the
   * norm is fused with the quantisation).  norm_weight [K] bf16 (device) or NULL: X arrives
   * normalised.  With it, X is the un-normalised activation and every use of the token (its
   * quantisation, the router, the expert branch) sees
   *   bf16( fp32( fp32(x * s) * norm_weight ) ),   s = fp32( 1 / sqrt(mean_k x^2 + norm_eps) ),
   * the mean and the reciprocal square root taken in fp64.  norm_eps > 0 (PQ_ERR_SHAPE otherwise:
   * an all-zero token would divide by zero). */
  const uint16_t* norm_weight;
  float norm_eps;
  /* The weights in the layout of the streaming decode kernel (pq_pack_decode), or NULL.  When every item of a
   * launch group carries them (w_bits_il, and B_il if r > 0) and the group is large enough for it to pay
   * (PQ_OPT_DECODE_STREAM), the group runs as ONE cooperative kernel that
   * streams each weight byte once with coalesced loads; results: the same integers (codes, routing, sums over k),
   * Y within the tolerance of the float epilogue (the expert product is summed in another order).  Otherwise, and
   * for shapes that kernel does not take (r not a multiple of 8), the two-kernel path is used.  Items of one launch
   * group that read the same X (same pointer, T, K and norm) are quantised once.  w_bits, A and B
   * are needed in both cases (the rows of A_e are read in their natural layout). */
  const uint32_t* w_bits_il;
  const uint16_t* B_il;
  /* The paper's INT8 high-precision branch on the decode path (Sec. 3.2), or NULL for the bf16 branch: A8 [E,r,K] int8 and
   * hp_scales [E][2] from pq_pack_experts, B8_il from pq_pack_decode_hp8.  The branch multiplies the token's int8 codes:
   *   h_int = A8_e q (int32, exact);  qh, gamma_h = Eq. 7-9 on h_int;  z_int = B8_e qh (int32, exact);
   *   z = z_int / (gamma_B gamma_h gamma_A gamma_t)
   * -- the arithmetic of pq_linear_forward_hp8.  It runs on the streaming kernel only, whatever the group's size:
   * w_bits_il is required (PQ_ERR_NULL), r a multiple of 16 (PQ_ERR_SHAPE); A, B and B_il are not read. */
  const int8_t* A8;
  const int8_t* B8_il;
  const float* hp_scales;
} pq_decode_item;
int pq_decode_batch(const pq_decode_item* items, int n, void* stream);

/* Weight layout of the streaming decode kernel (App. A: at batch size one the layer's cost is the bytes of its
 * weights, so they are stored the way the kernel reads them; the paper's CPU kernels permute weights offline in the
 * same spirit).  One-time, per linear:
 *   w_bits_il: [ceil(N/128)][ceil(K/128)][4][32][4] uint32 -- for row group g and chunk c of 128 contraction values,
 *     lane l's j-th feature 128 g + 32 j + l holds its four bit words 4 c .. 4 c + 3 (zero beyond N or K);
 *   B_il: [E][4 ceil(N/128)][r/8][32][8] bf16 -- for a group of 32 features, lane l holds 8 consecutive hidden values
 *     of row 32 group + l of B_e (zero beyond N).
 * pq_decode_pack_bytes gives the two sizes in bytes (b_il_bytes = 0 when r = 0).  r must be a multiple of 8
 * (PQ_ERR_SHAPE).  d->T is not used. */
int pq_decode_pack_bytes(const pq_desc* d, size_t* bits_il_bytes, size_t* b_il_bytes);
int pq_pack_decode(const pq_desc* d, const uint32_t* w_bits, const uint16_t* B, uint32_t* w_bits_il, uint16_t* B_il, void* stream);
/* The int8 codes B8 [E,N,r] of pq_pack_experts in the streaming decode kernel's order:
 * B8_il [E][4 ceil(N/128)][r/16][32][16] int8 (lane l holds 16 consecutive hidden values of row 32 group + l, zero
 * beyond N), pq_decode_pack_hp8_bytes(d) bytes (0 for a shape without this layout: r = 0 or not a multiple of 16). */
size_t pq_decode_pack_hp8_bytes(const pq_desc* d);
int pq_pack_decode_hp8(const pq_desc* d, const int8_t* B8, int8_t* B8_il, size_t b8_il_bytes, void* stream);

/* Straight-through backward (App. B.1): Sign, Round and Clip pass the gradient
 * unchanged; mu, lam, gamma are constants.  Every gradient is OVERWRITTEN.
 *   dY [T,N] bf16 (in);  dX [T,K] bf16;  dW [N,K] fp32 (w.r.t. the latent W);
 *   dA [E,r,K], dB [E,N,r], dWr [E,K] fp32;  dalpha, dbeta fp32 with the same
 *   length as alpha, beta.  dA/dB/dalpha may be NULL iff r == 0; dWr iff E <= 1. */
int pq_linear_backward(const pq_desc* d, const uint16_t* dY, const uint16_t* X,
                       const int8_t* w_s8, const float* w_scales, const uint16_t* A,
                       const uint16_t* B, const uint16_t* Wr, const float* alpha,
                       const float* beta, const void* saved, size_t saved_bytes, uint16_t* dX,
                       float* dW, float* dA, float* dB, float* dWr, float* dalpha, float* dbeta,
                       void* ws, size_t ws_bytes, void* stream);

/* What pq_linear_backward leaves in its workspace, for tests and diagnostics.
 *   dl [T,E] fp32: gradient of the router logits (Sec. 3.3, the router is trained end to end),
 *   dl[p,j] = dg g (delta_{j,e} - p_j) for the token at SORTED position p; NULL when E <= 1. */
typedef struct pq_bwd_view {
  float* dl;
} pq_bwd_view;
int pq_bwd_view_init(const pq_desc* d, void* ws, pq_bwd_view* out);

/* Test hook for the tensor-core engine: D[M,N] = A . B^T-style contraction with
 * raw accumulators written out (int32 for mode 0, fp32 otherwise), so that the
 * integer 1-bit product (Eq. 10) can be checked bit for bit.
 *   mode 0: int8,  A[M,K] and B[N,K] both K-contiguous
 *   mode 1: bf16,  A[M,K], B[N,K] both K-contiguous
 *   mode 2: bf16,  A[M,K] K-contiguous, B[K,N] N-contiguous
 *   mode 3: bf16,  A[K,M] M-contiguous, B[K,N] N-contiguous
 * M, N, K multiples of 8 (bf16) / 16 (int8). */
int pq_debug_gemm(int mode, int M, int N, int K, const void* A, const void* B, void* D,
                  void* stream);
/* Same with the width of the output tiles chosen by the caller (the layer's kernels
 * use 256, or 128 for the two small products of the HP branch): tile_n a multiple of 32
 * (modes 0, 1) or 64 (modes 2, 3), at most 256. */
int pq_debug_gemm_tile(int mode, int M, int N, int K, const void* A, const void* B, void* D,
                       int tile_n, void* stream);

/* Reads the device status word written by a kernel whose bounded wait ran out.
 * Synchronises `stream`.  code = 0 when no wait failed; `where` identifies the
 * waiting role.  The word is cleared by the call. */
int pq_device_status(void* stream, int* code, int* where);

/* Process-wide launch options.
 *   PQ_OPT_DECODE_PDL (default 1): launch the decode kernels with programmatic stream
 *   serialisation, so that a kernel's prologue (barrier set-up, the copy of the sign bits)
 *   overlaps the tail of the kernel before it in the stream.  0 = plain stream order.
 *   PQ_OPT_SIDE_STREAM (default 1): pq_linear_forward (dense layer with an HP branch) and
 *   pq_linear_backward run kernels that do not depend on one another side by side, on a helper
 *   stream the library keeps per caller stream (created on first use, never during a stream
 *   capture); the helper's work is joined back inside the same call, so the caller's stream
 *   order is unchanged and a stream capture records one graph with a fork and a join.  In the
 *   backward pass the weight-gradient tiles that need only dY and q/gamma are one launch
 *   (profile id bwd_dw) and the HP tiles (dB, dA, router) a second one (id hp_db).
 *   0 = every kernel on the caller's stream, the weight gradient as one launch.
 *   PQ_OPT_SPIN_CYCLES: limit of every device-side spin-wait in SM clock cycles (value <= 0 restores
 *   the default of 4e9, about two seconds).  A test hook: with a limit of a few cycles the first wait
 *   that does not succeed at once runs out, the kernel stops issuing work, lets copies and MMAs in
 *   flight finish, releases its TMEM and returns; pq_device_status then reports PQ_ERR_TIMEOUT and the
 *   outputs of that call are undefined.  Applies to the current device; blocks until the device's
 *   earlier work has finished.  Meant for pq_debug_gemm; do not shorten the limit around the decode
 *   entry points, whose later stages read indices an abandoned stage has not delivered.
 *   PQ_OPT_DECODE_STREAM (default 1): which launch groups of pq_decode_batch (up to 96 consecutive items) run on the
 *   streaming kernel when their items carry w_bits_il / B_il.  1 = those for which it is the faster of the two paths
 *   (12 or more linears; 6 or more when no item has more than two tokens); 2 = every group; 0 = none.
 *   PQ_OPT_DECODE_PREFETCH (default 1): the streaming decode kernel asks for the sign bits four chunks ahead of its
 *   bit product to be brought into L2.
 *   PQ_OPT_DECODE_MMA_FROM (default 5): the streaming decode kernel multiplies the sign bits of a group of at least this
 *   many tokens on the tensor cores (mma.sync u8 x s8) and of fewer tokens with dp4a; both are exact.  17 = dp4a only.
 *   PQ_OPT_DECODE_INTERLEAVE (default 1): the streaming decode kernel lets the two halves of a CTA walk the sign bits and
 *   the expert products side by side.  1 = where it measured faster (no linear of the launch has more than eight tokens); 2 = always; 0 = never. */
enum { PQ_OPT_DECODE_PDL = 1, PQ_OPT_SIDE_STREAM = 2, PQ_OPT_SPIN_CYCLES = 3, PQ_OPT_DECODE_STREAM = 4, PQ_OPT_DECODE_PREFETCH = 5,
       PQ_OPT_DECODE_MMA_FROM = 6, PQ_OPT_DECODE_INTERLEAVE = 7 };
int pq_set_option(int option, int value);

/* Cumulative number of kernels this library has launched in this process. */
long long pq_kernel_launches(void);

/* Measurement hook: from now on, every launch of the kernel with this id is
 * bracketed by cudaEventRecord(start_event) / cudaEventRecord(stop_event) on
 * the launching stream (both cudaEvent_t passed as void*; NULL, NULL clears).
 * Ids: 0 weight sums, 1 binarize+pack, 2 router, 3 expert scan, 4 activation
 * quantise, 5 HP up-projection, 6 fused forward tile, 7 row scatter, 8 scaled
 * sign, 9 scaled B, 10 HP dH, 11 dX, 12 dW (with the dB, dA and router-weight
 * tiles), 16 per-feature scale gradients (vector scales), 17 scalar scale gradients (one launch), 18 debug
 * GEMM, 19 decode token preparation, 20 decode main; 13-15, 21, 22 unused. */
int pq_profile_events(int kernel_id, void* start_event, void* stop_event);

const char* pq_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* PQUANT_H_ */
