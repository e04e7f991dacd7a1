/* rom.h — C ABI of the B200 (sm_100a) forward pass of one Routing-Mamba (RoM) layer.
 *
 * Paper notation (Sections 3.1 and 4.2): X in R^{L x D_m} per sequence, D_e = d_inner,
 * D_s = d_state, k = d_conv, d_r = dt_rank, N experts = E, top-K.  T = B*L tokens in (b,t) order,
 * "assignment" a = t*K + k is slot k of token t.
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless marked "host".  The caller owns every buffer; the
 *     library allocates no device memory and keeps no state on the device between calls.  The one
 *     exception is rom_route_noalloc: its scratch is an array resident in the library's device image, so
 *     overlapping calls of it on one GPU must be serialised by the caller (see its own comment).
 *   - All tensors are dense, row-major, channels-last; device pointers must be 16-byte aligned.
 *   - "dtype" tensors are stored as ROM_F32 (float) or ROM_BF16 (bfloat16) as rom_config.dtype says.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream);
 *     they neither synchronise the host nor copy device memory to the host.
 *   - Return value: a rom_status (0 = ok, negative = error).  Argument errors are found on the host
 *     before anything is launched.  Device-side problems (a bounded wait that expired) are latched
 *     in a status word at the head of the workspace and read with rom_get_status.
 *   - Outputs are fully overwritten; inputs are never written; workspace contents are scratch.
 *     Calls that use distinct workspaces and outputs are independent.
 */
#ifndef ROM_H_
#define ROM_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ROM_API __attribute__((visibility("default")))
#else
#define ROM_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { ROM_F32 = 0, ROM_BF16 = 1 } rom_dtype;

typedef enum {
  ROM_OK = 0,
  ROM_ERR_INVALID_ARG = -1,    /* NULL required pointer, bad size, misaligned pointer            */
  ROM_ERR_UNSUPPORTED = -2,    /* a legal problem the library does not cover (e.g. d_state != 16)  */
  ROM_ERR_WORKSPACE = -3,      /* ws_bytes smaller than rom_workspace_size                        */
  ROM_ERR_CUDA = -4,           /* a CUDA runtime/driver call failed (launch, tensor-map encode)   */
  ROM_ERR_ARCH = -5,           /* the current device is not sm_100                                */
  ROM_ERR_DEVICE_TIMEOUT = -6, /* a bounded device-side wait expired (reported by rom_get_status) */
  ROM_ERR_STATIC_SCRATCH = -7, /* the problem does not fit the built-in scratch of rom_route_noalloc */
  ROM_ERR_DEBUG_CHECK = -8     /* ROM_FLAG_DEBUG_CHECKS: a routing-table index out of range or a workspace canary
                                  overwritten (reported by rom_get_status)                          */
} rom_status;

typedef struct {
  int32_t B, L;               /* sequences, tokens per sequence                                   */
  int32_t d_model, d_inner;   /* D_m, D_e : multiples of 64                                       */
  int32_t d_state;            /* D_s : 16                                                         */
  int32_t d_conv;             /* k : 2, 3 or 4                                                    */
  int32_t dt_rank;            /* d_r : multiple of 16 (bf16) / of 4 (f32)                          */
  int32_t E, K;               /* experts (1..64), top-K (1..min(E,8))                             */
  int32_t dtype;              /* rom_dtype                                                        */
  int32_t gate_mode;          /* 0: R_i = P_i * 1[i in TopK] (Section 4.2, routing equation);
                                 1: P_i renormalised over the selected K (the sentence above it)   */
  int32_t disc_mode;          /* 0: zero-order hold B-bar (Section 3.1); 1: B-bar = Delta * B      */
  int32_t flags;              /* ROM_FLAG_* bits                                                  */
  int32_t small_proj_experts; /* 0 or 1: x Proj / dt Proj shared by all experts (Section 4.3, the method as
                                 proposed); E: one x Proj / dt Proj per expert under the same routing
                                 decision (the "(Conv, Gate, dt, x, Out)" ablation row of Section 5.3)      */
} rom_config;

#define ROM_FLAG_SIMT_GEMM 1  /* run every projection on the plain fp32-FMA kernels (bisecting aid;
                                 always the case for ROM_F32) instead of the tcgen05 tensor path   */
#define ROM_FLAG_DEBUG_CHECKS 2 /* rom_layer_forward / rom_layer_step only.  Every gather and scatter of the layer takes
                                 its row index from the routing tables: they are validated on the device before any
                                 kernel uses them (ranges, the two row <-> assignment maps agree, tile -> expert,
                                 padded offsets), and 256-byte canaries between the workspace sub-buffers are written
                                 before the first kernel and compared after the last.  A violation is latched as
                                 ROM_ERR_DEBUG_CHECK.  The workspace is larger with this flag (rom_workspace_size and
                                 rom_workspace_find take it into account); two more small launches per call.      */
#define ROM_FLAG_FUSED_SMALL 8 /* tensor path at top-1 with the shared x Proj / dt Proj: run the short conv, the x Proj and the
                                 dt Proj + softplus as ONE tcgen05 kernel (U written once and never re-read, delta kept on
                                 the SM) instead of three launches.  Same results up to rounding.  Off by default: as
                                 measured it is slower than the three launches (instruction-issue bound on one CTA per
                                 128 tokens); ignored where the sizes do not fit (d_r > 128, d_r + 2 D_s > 160)          */
#define ROM_FLAG_TEST_STALL 4 /* fault injection for tests of the device-side timeout path (tensor path only): the
                                 first grouped projection withholds the copies of one operand stage per CTA and
                                 every device wait gives up after 2^14 polls instead of 2^22, so the call returns
                                 normally, produces no valid output, and rom_get_status reports
                                 ROM_ERR_DEVICE_TIMEOUT.  The workspace stays usable for the next call.          */

typedef struct {                /* all read-only device pointers                                   */
  const void  *W_r;             /* [E, d_model]              dtype  router, W_r of Section 4.2 transposed */
  const float *b_r;             /* [E] or NULL               router bias (not in the paper)        */
  const void  *W_inz;           /* [E, 2*d_inner, d_model]   dtype  rows [0,D_e): Conv Proj W_in,i^T,
                                                                    rows [D_e,2D_e): Gate Proj W_g,i^T */
  const void  *w_conv;          /* [d_conv, d_inner]         dtype  tap d_conv-1 = current token   */
  const float *b_conv;          /* [d_inner] or NULL                                              */
  const void  *W_x;             /* [dt_rank+2*d_state, d_inner] dtype  rows delta | B | C (shared);
                                   [E, dt_rank+2*d_state, d_inner] when small_proj_experts == E      */
  const void  *W_dt;            /* [d_inner, dt_rank]        dtype  (shared); [E, d_inner, dt_rank]
                                   when small_proj_experts == E                                      */
  const float *b_dt;            /* [d_inner] or NULL                                              */
  const float *A;               /* [d_inner, d_state]        fp32, strictly negative              */
  const float *D;               /* [d_inner] or NULL         skip (not in the paper's equations)   */
  const void  *W_out;           /* [E, d_model, d_inner]     dtype  W_out,i^T                      */
} rom_weights;

/* Bytes of workspace rom_layer_forward / rom_route / rom_route_balance / rom_layer_step need for this
 * config (host out).                                                                              */
ROM_API int rom_workspace_size(const rom_config *cfg, size_t *bytes);

/* Bytes of workspace with which rom_scan cuts a long sequence into chunks that run in parallel (host out;
 * a few MB: two states and one sum of Delta per chunk, sequence and channel).  0 when batch x channels
 * already fill the GPU and the sequence is scanned in one pass.  Uses cfg->B, L, d_inner, d_state, dtype. */
ROM_API int rom_scan_workspace_size(const rom_config *cfg, size_t *bytes);

/* Router + top-K + dropless permutation (Section 4.2 routing equation; Section 5.1: no capacity
 * factor, no token dropping).
 *   logit[t,e] = b_r[e] + sum_d x[t,d] W_r[e,d], accumulated in fp64 (exact products; the same summation order
 *   for every expert, so equal weight rows give equal logits);
 *   P = softmax over all E; the K largest logits are selected, ties to the lowest expert id,
 *   slot k = k-th largest; gates per gate_mode.
 *   counts[e] = assignments of expert e; offsets = exclusive prefix sum (offsets[E] = T*K);
 *   inside an expert's segment assignments keep ascending a = t*K+k:
 *   perm[r] = a, inv_perm[a] = r.
 * Outputs: topk_idx[T,K] i32, gates[T,K] f32, counts[E], offsets[E+1], perm[T*K], inv_perm[T*K] i32.
 * Uses cfg->B, L, d_model, E, K, dtype, gate_mode.  Any output pointer may be NULL (not produced). */
ROM_API int rom_route(const rom_config *cfg, const void *x, const void *W_r, const float *b_r,
              int32_t *topk_idx, float *gates, int32_t *counts, int32_t *offsets,
              int32_t *perm, int32_t *inv_perm, void *ws, size_t ws_bytes, void *stream);

/* Load-balance statistic of the router of one layer (Appendix A.3, load balancing loss): runs the router
 * (same logits, top-K and tie rule as rom_route) and returns
 *   F[i]    = fraction of tokens dispatched to expert i = (assignments of i) / (B*L)   (sums to K),
 *   Pbar[i] = mean over tokens of Softmax(X W_r)_i,
 *   loss[0] = alpha * E * sum_i F[i] * Pbar[i]      (this layer's term; the paper uses alpha = 1e-3).
 * F, Pbar [E] and loss [1] are fp32 device outputs; each may be NULL.  Sums over tokens are taken in a fixed
 * order in fp64, so results are reproducible run to run.  Uses cfg->B, L, d_model, E, K, dtype.            */
ROM_API int rom_route_balance(const rom_config *cfg, const void *x, const void *W_r, const float *b_r, float alpha,
                      float *F, float *Pbar, float *loss, void *ws, size_t ws_bytes, void *stream);

/* rom_route for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * is a deployment variant of the routing step above, with identical results.)
 *
 * Who needs it: a host that gives the library a fixed set of buffers and forbids cudaMalloc while
 * it runs -- a serving process whose memory pool belongs to another component, an allocator that
 * is locked after start-up, a latency-critical loop that cannot absorb an allocation's cost or its
 * failure.  Such a caller cannot provide the workspace rom_route asks for, so this entry point keeps
 * its scratch (about 2 MiB at the largest supported size) in a fixed 3 MiB array inside the library's
 * device image.  Every GPU that loads the library holds that array until the process exits.
 *
 * The caller passes inputs and outputs only; arguments, outputs and their meaning are those of
 * rom_route.  Limits: B*L <= 65536 tokens and B*L*K <= 131072 assignments (E <= 64, K <= 8 as
 * elsewhere); anything larger returns ROM_ERR_STATIC_SCRATCH and launches nothing -- use rom_route
 * with a caller-owned workspace instead.  The call itself allocates nothing, on the host or device.
 *
 * The first call on each GPU looks up the array's device address (once per device, with that
 * device current); make that first call before starting any stream capture.
 * All calls on one GPU share the array, and it keeps the previous call's contents.  Each call
 * rewrites what it reads, clears the one table that must start cleared and leaves its blocks-done
 * counter at zero, so back-to-back calls on one stream are safe; calls that overlap on the same GPU (other streams or
 * host threads) race on the scratch and must be serialised by the caller.                          */
ROM_API int rom_route_noalloc(const rom_config *cfg, const void *x, const void *W_r, const float *b_r,
                      int32_t *topk_idx, float *gates, int32_t *counts, int32_t *offsets,
                      int32_t *perm, int32_t *inv_perm, void *stream);

/* Selective scan (Section 3.1, linear recurrence h_t = A-bar h_{t-1} + B-bar U_t, Y_t = C h_t) with
 * A-bar = exp(Delta A), B-bar per disc_mode, optional skip D*U and optional gate y *= SiLU(z)
 * (output equation of Section 3.1).  State and arithmetic are fp32.
 *   u, z, y : [B, L, d_inner] dtype;  delta : [B, L, d_inner] fp32;  A : [d_inner, d_state] fp32;
 *   Bm, Cm : [B, L, d_state] fp32;  D : [d_inner] or NULL;  z NULL = no gate;
 *   h0 : [B, d_inner, d_state] fp32 or NULL (zeros);  h_last : same shape or NULL (not produced).
 *   ws : NULL (one pass per sequence, whatever its length; with few long bf16 sequences a kernel built for one warp per
 *        SM sub-partition is used) or at least rom_scan_workspace_size(cfg) bytes (few long sequences are then cut into
 *        chunks scanned in parallel; a larger buffer, e.g. the layer's workspace, is accepted; only its head is used).
 *        The result does not depend on the choice beyond fp32 rounding order.
 * Uses cfg->B, L, d_inner, d_state, dtype, disc_mode.                                             */
ROM_API int rom_scan(const rom_config *cfg, const void *u, const float *delta, const float *A,
             const float *Bm, const float *Cm, const float *D, const void *z, const float *h0,
             void *y, float *h_last, void *ws, size_t ws_bytes, void *stream);

/* Backward of rom_scan (Section 5.1 trains the layer end to end; the recurrence differentiated is that of Section
 * 3.1): given dy = dLoss/d(output of rom_scan), the gradients of every input of the same call.
 *   forward   h_t = a_t h_{t-1} + b_t u_t,  y_t = C_t h_t + D u_t,  out_t = y_t SiLU(z_t)  (a = exp(Delta A), b per disc_mode)
 *   reverse   g = dLoss/dh_t:  g += C_t e_t (e = dy SiLU(z));  dC_t = sum_c e_t h_t;  da = g h_{t-1};  db = g u_t;  g <- a_t g
 *   dy, u, z : [B, L, d_inner] dtype (z NULL = no gate);  delta : [B, L, d_inner] fp32;  A, Bm, Cm, D, h0 as in rom_scan;
 *   dh_last  : [B, d_inner, d_state] fp32 or NULL: gradient arriving at the final state.
 * Outputs: du, dz [B, L, d_inner] dtype (dz NULL exactly when z is);  ddelta [B, L, d_inner] fp32;  dA [d_inner, d_state],
 *   dBm, dCm [B, L, d_state], dD [d_inner] (NULL exactly when D is) fp32, each the sum over everything that shares the
 *   parameter (dA and dD over sequences and steps; dBm, dCm over channels) -- accumulated with floating-point atomics,
 *   so their last bits vary from run to run;  dh0 [B, d_inner, d_state] fp32 or NULL.
 * ws: rom_scan_backward_workspace_size(cfg) bytes (the state at the start of every 16 steps, plus the chunk states of the chunk-parallel form).  All arithmetic fp32.
 * Uses cfg->B, L, d_inner, d_state, dtype, disc_mode.                                                              */
ROM_API int rom_scan_backward_workspace_size(const rom_config *cfg, size_t *bytes);
ROM_API int rom_scan_backward(const rom_config *cfg, const void *dy, const void *u, const float *delta, const float *A,
                      const float *Bm, const float *Cm, const float *D, const void *z, const float *h0,
                      const float *dh_last, void *du, float *ddelta, float *dA, float *dBm, float *dCm, float *dD,
                      void *dz, float *dh0, void *ws, size_t ws_bytes, void *stream);

/* Forward pass of one RoM layer (Section 4.2 equations for G, H_t, O_t, E_i with the shared
 * Conv1D / x Proj / dt Proj / A / D of Section 4.3):
 *   route -> gather tokens by expert -> per-expert [Conv Proj | Gate Proj] -> un-permute, sum over
 *   the selected experts (indicator only) -> causal depthwise conv + SiLU -> x Proj, dt Proj +
 *   softplus -> selective scan -> * SiLU(gate) -> re-permute with the same routing -> per-expert
 *   Out Proj -> gate-weighted sum over the selected experts.
 *   x, out : [B, L, d_model] dtype.  topk_idx_out [T,K] i32, gates_out [T,K] f32, counts_out [E] i32
 *   may each be NULL.
 * With cfg->small_proj_experts == E the x Proj and dt Proj are per-expert layers under the same
 * routing (the paper prints no equation for this ablation; it is taken in the pattern of H_t and G):
 *   (delta_i, B_i, C_i) = U_t W_x,i;  B_t = sum_i 1_i B_i;  C_t = sum_i 1_i C_i;
 *   Delta_t = softplus(sum_i 1_i delta_i W_dt,i + b_dt)  -- indicator-only sums over the selected
 *   experts in ascending slot order, each expert's delta_i through its own dt Proj, b_dt shared.   */
ROM_API int rom_layer_forward(const rom_config *cfg, const rom_weights *w, const void *x, void *out,
                      int32_t *topk_idx_out, float *gates_out, int32_t *counts_out,
                      void *ws, size_t ws_bytes, void *stream);

/* Backward pass of one RoM layer (Section 5.1: the layer is trained end to end; Appendix A.3: the router is trained
 * through the gate values).  Given dout = dLoss/dO for the forward of rom_layer_forward on the same cfg, weights and
 * x, returns dx = dLoss/dX and the gradient of every weight.  The equations reversed are those of Sections 3.1 and
 * 4.2 as listed at rom_layer_forward.  Readings where the paper is silent: the top-K indicator is piecewise constant
 * and is held fixed, so the router receives gradient only through R_i (gate_mode decides which form), not through the
 * Conv/Gate projections, which carry the indicator alone; jitter noise and SparseMixer (Appendix A.3) are stochastic
 * training-time estimators and are not part of this call.  Only the shared x Proj / dt Proj wiring (Section 4.3) is
 * differentiated: cfg->small_proj_experts == E returns ROM_ERR_UNSUPPORTED.
 * The call recomputes the forward activations it needs from x (it does not read a forward workspace), then walks the
 * steps backwards: data gradients of the projections are the forward grouped GEMMs on transposed weights; weight
 * gradients are sums over the tokens of each expert's segment.
 *   x, dout, dx : [B, L, d_model] dtype.
 *   g           : device pointers, fp32, fully overwritten: the shapes of the corresponding rom_weights fields;
 *                 db_r may be NULL (not produced); dD is NULL exactly when w->D is.
 *   ws          : rom_layer_backward_workspace_size(cfg) bytes.
 * Sums that cross thread blocks use floating-point atomics: the last bits of the gradients vary from run to run.  */
typedef struct {
  float *dW_r;      /* [E, d_model]                    */
  float *db_r;      /* [E] or NULL                     */
  float *dW_inz;    /* [E, 2*d_inner, d_model]         */
  float *dw_conv;   /* [d_conv, d_inner]               */
  float *db_conv;   /* [d_inner]                       */
  float *dW_x;      /* [dt_rank+2*d_state, d_inner]    */
  float *dW_dt;     /* [d_inner, dt_rank]              */
  float *db_dt;     /* [d_inner]                       */
  float *dA;        /* [d_inner, d_state]              */
  float *dD;        /* [d_inner] or NULL               */
  float *dW_out;    /* [E, d_model, d_inner]           */
} rom_grads;
ROM_API int rom_layer_backward_workspace_size(const rom_config *cfg, size_t *bytes);
ROM_API int rom_layer_backward(const rom_config *cfg, const rom_weights *w, const void *x, const void *dout, void *dx,
                       const rom_grads *g, void *ws, size_t ws_bytes, void *stream);

/* rom_layer_forward with HOST input and output: enqueues on `stream` the copy of x_host to x_dev, the
 * forward (x_dev -> out_dev) and the copy of out_dev to out_host, and returns without waiting.
 *   x_host, out_host : HOST pointers, [B, L, d_model] dtype; page-locked memory makes the copies
 *                      asynchronous (pageable memory works but serialises with the host)
 *   x_dev, out_dev   : device staging buffers of the same size, owned by the caller
 * out_host is valid once the stream has been synchronised.  Calls on different streams with their own
 * staging buffers and workspaces overlap one call's copies with another's kernels.               */
ROM_API int rom_layer_forward_host(const rom_config *cfg, const rom_weights *w, const void *x_host, void *out_host,
                           void *x_dev, void *out_dev, void *ws, size_t ws_bytes, void *stream);

/* Single-token step of the layer (recurrent inference; Section 3.1: the state-space model is a linear
 * recurrence, so a generated token costs the same whatever the context length).  Same equations and
 * routing as rom_layer_forward for one new token per sequence, with the state carried by the caller:
 *   x, out     : [B, d_model] dtype (cfg->L must be 1)
 *   conv_state : [B, d_conv-1, d_inner] fp32, in/out: H_t (the summed Conv Proj rows) of the previous
 *                d_conv-1 tokens, oldest first; zeros at the start of a sequence
 *   ssm_state  : [B, d_inner, d_state] fp32, in/out: h_{t-1}; zeros at the start of a sequence
 * Feeding a sequence token by token from zero states reproduces rom_layer_forward on the whole sequence
 * (up to the rounding of the storage dtype).  topk_idx_out [B,K], gates_out [B,K] may be NULL.
 * ws: rom_workspace_size(cfg) bytes.                                                               */
ROM_API int rom_layer_step(const rom_config *cfg, const rom_weights *w, const void *x, float *conv_state,
                   float *ssm_state, void *out, int32_t *topk_idx_out, float *gates_out,
                   void *ws, size_t ws_bytes, void *stream);

/* Feed-forward SwiGLU mixture of experts that shares the routing decision of the preceding RoM layer
 * (Appendix A.2, the two equations of the hybrid RoM + FFN-MoE model):
 *   Y_t = sum_i R_i * 1[i in TopK] * f_i(X_t),   f_i(x) = W_down,i ( SiLU(W_gate,i x) * (W_up,i x) )
 * (the paper names f_i a SwiGLU expert without writing it out; the usual bias-free form is taken).
 * The selected experts and their gates are not recomputed: topk_idx [T,K] i32 and gates [T,K] f32 are
 * the outputs of that layer's rom_route / rom_layer_forward call (device pointers, read only).
 *   d_ff   : hidden width of an expert, a multiple of 128
 *   W_gu   : [E, 2*d_ff, d_model] dtype, rows [0,d_ff) = W_gate,i, rows [d_ff,2*d_ff) = W_up,i
 *   W_down : [E, d_model, d_ff]   dtype
 *   x, out : [B, L, d_model]      dtype (x is this layer's own input)
 *   ws     : rom_ffn_moe_workspace_size(cfg, d_ff) bytes of scratch, independent of the RoM layer's
 * Uses cfg->B, L, d_model, E, K, dtype, flags.  The K experts of a token must be distinct and in
 * [0, E); an index outside that range is clamped (every access stays in bounds, the result for that
 * token is unspecified) and rom_get_status then reports ROM_ERR_INVALID_ARG.                        */
ROM_API int rom_ffn_moe_workspace_size(const rom_config *cfg, int32_t d_ff, size_t *bytes);
ROM_API int rom_ffn_moe_forward(const rom_config *cfg, int32_t d_ff, const void *W_gu, const void *W_down,
                        const void *x, const int32_t *topk_idx, const float *gates, void *out,
                        void *ws, size_t ws_bytes, void *stream);

/* Routing Mamba on a Mamba2-style block (Section 5.2, "RoM on other linear recurrent architectures"; Section 5.4, first
 * insight: for blocks with a unified design all major projection layers become experts under the shared routing;
 * Appendix A.2: the deployment "follows the same logic" as on Mamba).  The paper prints no equations for this variant:
 * the block is the published Mamba2 block with one B/C group, and per token t
 *   [z | x | B | C | dt]_t = sum_i 1_i X_t W_in,i           (indicator only; widths D_e | D_e | N | N | heads)
 *   (x, B, C) <- SiLU(causal depthwise conv(x, B, C) + b_conv);   dt_h = softplus(dt_h + dt_bias_h)
 *   per head h (headdim channels):  H_t = exp(dt_h A_h) H_{t-1} + dt_h x_t (x) B_t,   y_t = C_t H_t + D_h x_t
 *   y^_t = (y_t * SiLU(z_t)) / sqrt(mean_c (y_t * SiLU(z_t))_c^2 + 1e-5) * w_norm
 *   O_t = sum_i R_i(X_t) y^_t W_out,i
 * with the router, top-K, gates and permutation of rom_route.  Shared by all experts: conv, A, D, dt_bias, w_norm.
 *   headdim : channels per head; d_inner / headdim heads, a multiple of 8.  cfg->dt_rank, disc_mode and
 *             small_proj_experts are not used; d_state must be 16, d_conv 2..4.
 *   x, out  : [B, L, d_model] dtype;  ws: rom_mamba2_workspace_size(cfg, headdim) bytes.                            */
typedef struct {                  /* read-only device pointers */
  const void  *W_r;               /* [E, d_model]                               dtype */
  const float *b_r;               /* [E] or NULL */
  const void  *W_in;              /* [E, 2*d_inner + 2*d_state + heads, d_model] dtype  rows z | x | B | C | dt */
  const void  *w_conv;            /* [d_conv, d_inner + 2*d_state]              dtype  tap d_conv-1 = current token */
  const float *b_conv;            /* [d_inner + 2*d_state] or NULL */
  const float *dt_bias;           /* [heads] or NULL */
  const float *A;                 /* [heads], strictly negative */
  const float *D;                 /* [heads] or NULL */
  const float *w_norm;            /* [d_inner] */
  const void  *W_out;             /* [E, d_model, d_inner]                      dtype */
} rom_mamba2_weights;
ROM_API int rom_mamba2_workspace_size(const rom_config *cfg, int32_t headdim, size_t *bytes);
ROM_API int rom_mamba2_layer_forward(const rom_config *cfg, int32_t headdim, const rom_mamba2_weights *w, const void *x,
                             void *out, int32_t *topk_idx_out, float *gates_out, int32_t *counts_out,
                             void *ws, size_t ws_bytes, void *stream);

/* Profiling aid: the same launch sequence as rom_layer_forward with a CUDA event recorded on
 * `stream` between stages; synchronises the stream and writes the device time of each stage in
 * milliseconds to stage_ms (host out, at least rom_num_stages() floats).  Stage i is named
 * rom_stage_name(i): route, gather, in_proj, conv, x_proj, dt_proj, scan, out_proj, combine.      */
ROM_API int rom_layer_forward_profile(const rom_config *cfg, const rom_weights *w, const void *x, void *out,
                              void *ws, size_t ws_bytes, void *stream, float *stage_ms, int n_stage_ms);
ROM_API int rom_num_stages(void);
ROM_API const char *rom_stage_name(int i);

/* Locate a named intermediate of the last rom_layer_forward inside the workspace (host-only
 * arithmetic; for tests and debugging).  Names: "U" [T,D_e] dtype, "delta_r" [T,d_r] dtype,
 * "Bm","Cm" [T,D_s] f32, "Delta" [T,D_e] dtype, "row_of_assign" [T*K] i32 (padded row of each
 * assignment), "XZp" [rows,2*D_e] dtype, "Ygp" [rows,D_e] dtype, "pad_offsets" [E+1] i32.
 * Returns ROM_ERR_INVALID_ARG for an unknown name.                                                */
ROM_API int rom_workspace_find(const rom_config *cfg, const char *name, size_t *offset, size_t *bytes);

/* Re-run the checks of ROM_FLAG_DEBUG_CHECKS on a workspace that the last rom_layer_forward / rom_layer_step call
 * with that flag (same cfg) has filled: routing tables and canaries (a debugging aid; the paper has no counterpart).
 * Asynchronous on `stream`; the verdict is read with rom_get_status.  cfg->flags must carry the flag.  */
ROM_API int rom_debug_check(const rom_config *cfg, void *ws, size_t ws_bytes, void *stream);

/* Read and clear the device status word of a workspace.  `host_code` (host out) receives ROM_OK or the
 * rom_status a kernel latched: ROM_ERR_DEVICE_TIMEOUT (a bounded wait expired) or ROM_ERR_INVALID_ARG
 * (rom_ffn_moe_forward met an expert index out of range) or ROM_ERR_DEBUG_CHECK (ROM_FLAG_DEBUG_CHECKS; the second
 * and third int32 of the workspace then hold which check failed -- 10..15 a routing table, 20 a canary -- and the
 * offending index, until this call clears them).  This call synchronises `stream`.                  */
ROM_API int rom_get_status(void *ws, void *stream, int32_t *host_code);

/* Static string for a rom_status value.                                                           */
ROM_API const char *rom_status_string(int code);

/* Number of kernels the last call of rom_layer_forward launched on this host thread (host-only). */
ROM_API int rom_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* ROM_H_ */
