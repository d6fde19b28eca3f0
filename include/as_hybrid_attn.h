/*
 * as_hybrid_attn.h - C ABI of the hybrid-attention forward pass for NVIDIA B200 (sm_100a).
 *
 * The operator is the hybrid attention of "Attention Surgery" (arXiv 2509.24899), section
 * "Hybrid Attention": for every query i
 *
 *        sum_{j in T_S} exp(q_i.k_j * scale - c_i) v_j  +  lambda_i * phi_q(q_i) S
 *  y_i = -----------------------------------------------------------------------------
 *        sum_{j in T_S} exp(q_i.k_j * scale - c_i)      +  lambda_i * phi_q(q_i) . z
 *
 *  S = sum_{j in T_L} phi_k(k_j)^T v_j   [F x d],      z = sum_{j in T_L} phi_k(k_j)   [F],
 *  c_i = max_{j in T_S} q_i.k_j * scale,
 *
 * where the tokens T = {0..N-1} are split into softmax tokens T_S and linear tokens
 * T_L = T \ T_S by the hybrid rate R (same section: every R-th token is a softmax token), and
 * phi_q, phi_k are the learned polynomial feature maps of "Characterization of phi".
 * Rate 1 is plain softmax attention (Eq. 2); rate 0 is normalised linear attention (the
 * kernelised form in "Preliminaries: Linear Attention").
 *
 * Conventions
 *   - All tensor pointers are DEVICE pointers unless a parameter says "host".
 *   - q, k, v, out: [B, H, N, d] bf16, contiguous, base address 16-byte aligned.
 *   - The caller owns every buffer and the CUDA stream; the library owns only the handle.
 *   - Every function returns a status; nothing aborts, and no kernel traps.  On error the
 *     out-parameters are left untouched.
 *   - `forward` is asynchronous on the given stream, allocates nothing and does not
 *     synchronise.  One handle may be used concurrently only with distinct workspaces.
 */
#ifndef AS_HYBRID_ATTN_H_
#define AS_HYBRID_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define AS_API __attribute__((visibility("default")))
#else
#define AS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct as_hybrid_attn_s* as_hybrid_attn_t;   /* opaque, library-owned */

typedef enum {
  AS_OK = 0,
  AS_ERR_INVALID_ARG = 1,     /* NULL pointer, bad shape, misaligned buffer, inconsistent sizes   */
  AS_ERR_UNSUPPORTED = 2,     /* valid request the library has no kernel for                      */
  AS_ERR_ARCH = 3,            /* current device is not compute capability 10.x                      */
  AS_ERR_ALLOC = 4,           /* host or device allocation failed in create                        */
  AS_ERR_WORKSPACE = 5,       /* workspace NULL, misaligned or smaller than workspace_bytes         */
  AS_ERR_CUDA = 6,            /* a CUDA runtime/driver call failed                                  */
  AS_ERR_DEVICE_TIMEOUT = 7,  /* a bounded wait inside a kernel ran out (see last_status)           */
  AS_ERR_INFEASIBLE = 8       /* block-rate selection: no assignment fits the budget                */
} as_status_t;

/* Stabiliser handling (the paper subtracts c_i only inside the softmax exponentials):
 *   AS_STAB_PAPER  lambda_i = 1            - the equation exactly as printed;
 *   AS_STAB_EXACT  lambda_i = exp(-c_i)    - weights exp(s_ij) beside phi_q.phi_k, independent of c_i. */
enum { AS_STAB_PAPER = 0, AS_STAB_EXACT = 1 };

/* Activation of the feature map's embedding layers. */
enum { AS_ACT_RELU = 0 };

/* Kernel path.  AS_PATH_TENSOR (0, the default) is the library: tcgen05/TMEM/TMA kernels.
 * AS_PATH_SIMT is a TEST AID, not a second backend: plain fp32 CUDA-core kernels of the same steps, kept so
 * that the tests can put an fp32 result beside the tensor-core one on the same inputs.  It is slow, covers
 * one-layer feature maps with F == d and degree <= 2 without bias only, and nothing selects it on its own. */
enum { AS_PATH_TENSOR = 0, AS_PATH_SIMT = 1 };

/* Kernel classes reported by the profiling calls. */
enum { AS_KERNEL_KPASS = 0, AS_KERNEL_REDUCE = 1, AS_KERNEL_QPASS = 2, AS_NUM_KERNELS = 3 };

typedef struct {
  uint32_t struct_size;            /* sizeof(as_hybrid_attn_desc_t), for ABI versioning            */
  int32_t  B, H, N, d;             /* batch, heads, tokens, head dim; d in {64, 128}               */
  int32_t  grid_t, grid_h, grid_w; /* latent grid, product == N; tokens row-major, w fastest       */
  int32_t  blk_t, blk_h, blk_w;    /* spatial block (clipped at the grid border).  Inside each
                                      block the token with 0-based raster index l is a softmax
                                      token iff l mod R == 0.  A block equal to the grid gives the
                                      paper's 1-D rule  T_S = { i : i mod R = 1 }  (1-indexed).     */
  int32_t  rate_den;               /* R: 1 = every token softmax, 0 = none, else rate 1/R          */
  const int32_t* softmax_idx;      /* optional HOST pointer to an explicit sorted, unique T_S;
                                      NULL selects the rule above                                   */
  int32_t  n_softmax;              /* length of softmax_idx (ignored when it is NULL)              */
  int32_t  phi_dim;                /* F == P * D': output width of the feature map.  One layer: d, or a
                                      multiple of 128 up to 512.  Two layers: see phi_hidden.          */
  int32_t  phi_layers;             /* embedding-network depth: 1 or 2                                */
  int32_t  phi_hidden;             /* hidden width when phi_layers == 2 (unused otherwise).  d = 128:
                                      hidden and F each 128 or 256 (the paper's default map is
                                      d -> 2d -> 2d); d = 64: hidden == F == 64                        */
  int32_t  poly_degree;            /* P in 1..4: part p (1-based) of the activation is raised to the
                                      power p; F / P must be a multiple of 32                          */
  int32_t  phi_act;                /* AS_ACT_RELU                                                   */
  float    softmax_scale;          /* 0 selects 1/sqrt(d)                                           */
  int32_t  stab_mode;              /* AS_STAB_PAPER | AS_STAB_EXACT                                 */
  int32_t  kernel_path;            /* AS_PATH_TENSOR; AS_PATH_SIMT only in tests (see above)        */
} as_hybrid_attn_desc_t;

/* Feature-map weights, DEVICE pointers, bf16, row-major with the output feature as the slow
 * index ("Characterization of phi": an embedding network, then the polynomial parts).
 *   phi_layers == 1:  w*1 is [H, F, d], b*1 [H, F];                  a = ReLU(W_1 x + b_1)
 *   phi_layers == 2:  w*1 is [H, hidden, d], b*1 [H, hidden], w*2 is [H, F, hidden], b*2 [H, F];
 *                     a = ReLU(W_2 ReLU(W_1 x + b_1) + b_2)
 * phi(x) = [a_1, a_2^2, ..., a_P^P]: a split into P contiguous parts, part p to the power p.
 * Weight matrices are 16-byte aligned.  Every bias is optional (NULL = none; the paper does not say
 * whether the embedding layers carry one) and 4-byte aligned; w*2 and b*2 must be NULL when
 * phi_layers == 1.  With two layers the hidden activations are rounded to bf16 between the layers. */
typedef struct {
  const void *wq1, *bq1, *wq2, *bq2;
  const void *wk1, *bk1, *wk2, *bk2;
} as_phi_weights_t;

/* Creates a handle for one layer geometry on the CURRENT device: validates the descriptor,
 * builds the token split on the host (section "Hybrid Attention", token rule) and uploads the
 * index tables.  Returns AS_ERR_ARCH when the current device is not sm_100.  The handle belongs to
 * that device: forward, forward_host, linear_state and last_status return AS_ERR_INVALID_ARG when
 * another device is current. */
AS_API as_status_t as_hybrid_attn_create(const as_hybrid_attn_desc_t* desc, as_hybrid_attn_t* out);

/* Frees the handle and its device tables.  NULL is a no-op.  (Utility: no counterpart in the paper.) */
AS_API as_status_t as_hybrid_attn_destroy(as_hybrid_attn_t h);

/* Bytes of scratch `forward` needs (compacted softmax K/V, partial and final linear state, the keys' hidden
 * activations of a two-layer map).  (Utility: no counterpart in the paper.) */
AS_API as_status_t as_hybrid_attn_workspace_bytes(as_hybrid_attn_t h, size_t* bytes);

/* Bytes of scratch `forward_host` needs: the above plus device staging for q, k, v and out.
 * (Utility: no counterpart in the paper.) */
AS_API as_status_t as_hybrid_attn_workspace_bytes_host(as_hybrid_attn_t h, size_t* bytes);

/* The hybrid attention forward pass (equation above; hybrid equation of the paper).
 *   q, k, v   [B,H,N,d] bf16 device, read only
 *   w         feature-map weights (may be NULL only when rate_den == 1)
 *   out       [B,H,N,d] bf16 device, written
 *   aux       optional [B,H,N,3] fp32 device: (c_i, den_S, den_L) with
 *             den_S = sum_{T_S} exp(s_ij - c_i), den_L = phi_q(q_i).z (before lambda_i); NULL to skip
 *   workspace device scratch, 256-byte aligned, >= workspace_bytes; contents are overwritten
 *   cuda_stream  a cudaStream_t (NULL = default stream)
 * Enqueues its kernels and returns; errors found on the host are returned at once, a device
 * time-out is reported later by as_hybrid_attn_last_status.  Calls on one handle must be ordered on the device (one
 * stream, or events between streams): the handle's status word and the arrival counters of the key stage are shared
 * by its calls.  On AS_PATH_TENSOR the key stage's CTAs wait for one another when a head is cut into several token
 * chunks, so that kernel is a cooperative launch (at most one CTA per SM): it needs the whole device, and the launch
 * is refused (AS_ERR_CUDA) where the device cannot hold all of its CTAs at once. */
AS_API as_status_t as_hybrid_attn_forward(as_hybrid_attn_t h, const void* q, const void* k, const void* v,
                                   const as_phi_weights_t* w, void* out, float* aux,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Same operation with HOST q, k, v and out buffers (pinned memory keeps the copies asynchronous).
 * The work is cut into runs of whole heads (about 8 MB of q or more each): the copies in of one run,
 * the kernels of the previous one and the copy out of the one before overlap, on two side streams the
 * handle creates on the first call.  Everything is ordered after the work already in `cuda_stream`,
 * and `cuda_stream` completes only after the last copy out.  The weights stay device pointers.
 * workspace >= workspace_bytes_host.  Not for use by two host threads on one handle at once. */
AS_API as_status_t as_hybrid_attn_forward_host(as_hybrid_attn_t h, const void* q_host, const void* k_host,
                                        const void* v_host, const as_phi_weights_t* w,
                                        void* out_host, void* workspace, size_t workspace_bytes,
                                        void* cuda_stream);

/* Copies the linear state left in `workspace` by the last forward on `cuda_stream`:
 * S_out [B,H,F,d] fp32 and z_out [B,H,F] fp32 (device pointers; either may be NULL).
 * S = sum_{T_L} phi_k(k_j)^T v_j, z = sum_{T_L} phi_k(k_j) ("Preliminaries: Linear Attention":
 * the two sums that do not depend on the query).  AS_ERR_INVALID_ARG when rate_den == 1. */
AS_API as_status_t as_hybrid_attn_linear_state(as_hybrid_attn_t h, const void* workspace,
                                        float* S_out, float* z_out, void* cuda_stream);

/* Number of softmax tokens |T_S| and, optionally, their sorted indices (HOST buffer of
 * `capacity` int32; NULL to skip).  Token rule of section "Hybrid Attention". */
AS_API as_status_t as_hybrid_attn_softmax_tokens(as_hybrid_attn_t h, int32_t* count,
                                          int32_t* idx_host, int32_t capacity);

/* Synchronises `cuda_stream`, then reads and clears the handle's device status word.
 * AS_OK, AS_ERR_DEVICE_TIMEOUT (a bounded barrier wait in a kernel expired; outputs of that
 * forward are undefined but the context stays usable) or AS_ERR_CUDA.  After a time-out the handle is
 * INERT until this call has read and cleared the word: the kernels of every later forward on the handle
 * return at once and leave their outputs untouched, while `forward` itself keeps returning AS_OK.
 * (Utility: no counterpart in the paper.) */
AS_API as_status_t as_hybrid_attn_last_status(as_hybrid_attn_t h, void* cuda_stream);

/* The forward pass in two stages, for a layer whose TOKENS are spread over several GPUs (sequence sharding).
 * The linear state is a sum over keys that does not depend on the query ("Preliminaries: Linear Attention": the two
 * sums can be precomputed), so partial states of token ranges add up, and the softmax tokens of the ranges
 * concatenate; a query then needs only the summed state and the gathered softmax keys (hybrid equation).  Each
 * rank creates a handle for ITS token range (N = tokens of the range, softmax_idx = the range's softmax tokens,
 * counted from the range's start) and runs:
 *   key_pass      k, v [B,H,N,d] of the range -> in `workspace`: the range's softmax keys and values K_S, V_S
 *                 [B*H, n_softmax, d] bf16 and its partial state S [B*H,F,d], z [B*H,F] fp32, at the byte offsets
 *                 `workspace_offsets` returns.  A range without linear tokens is left alone (its keys are k, v
 *                 themselves, its state is zero); a range without softmax tokens leaves no K_S, V_S.
 *   (the caller sums S, z over the ranks and gathers K_S, V_S in rank order, each into local memory)
 *   query_pass    q [B,H,N,d] of the range, the gathered keys ks, vs [B*H, n_keys, d] bf16 (n_keys may be 0), the
 *                 summed S, z (both NULL when no rank has linear tokens) -> out [B,H,N,d] (, aux).  `workspace` is
 *                 scratch of at least workspace_bytes again (it receives S as a bf16 operand); a handle whose own
 *                 range has no linear tokens cannot take a state (AS_ERR_UNSUPPORTED: its workspace has no room).
 * Both are asynchronous on the stream, allocate nothing, and share every rule of `forward`. */
AS_API as_status_t as_hybrid_attn_key_pass(as_hybrid_attn_t h, const void* k, const void* v, const as_phi_weights_t* w,
                                           void* workspace, size_t workspace_bytes, void* cuda_stream);
AS_API as_status_t as_hybrid_attn_workspace_offsets(as_hybrid_attn_t h, size_t* ks, size_t* vs, size_t* S, size_t* z);
AS_API as_status_t as_hybrid_attn_query_pass(as_hybrid_attn_t h, const void* q, const as_phi_weights_t* w, const void* ks,
                                             const void* vs, int32_t n_keys, const float* S, const float* z, void* out,
                                             float* aux, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Gradient of the value-distillation loss w.r.t. the feature-map weights (section "Attention Distillation",
 * value-distillation loss L = || y - y_hat ||_1; Algorithm 1: the student's update touches phi only).  To be
 * called after `forward` with the same q, k, v, w on the same stream:
 *   y_teacher  [B,H,N,d] bf16 device: the teacher block's attention output y
 *   y_hat      [B,H,N,d] bf16 device: `out` of that forward
 *   aux        [B,H,N,3] fp32 device: `aux` of that forward (required: c_i, den_S, den_L)
 *   forward_workspace   the workspace of that forward, untouched since (it holds S and z)
 *   dWq, dWk   [H,F,d] fp32 device, written: dL/dW_q and dL/dW_k, summed over the batch
 *   loss       optional device float, written: L summed over every output element (must be NULL for a layer
 *              without linear tokens, whose gradients are zero)
 *   workspace  device scratch, 256-byte aligned, >= backward_workspace_bytes
 * L = sum |y - y_hat|; q, k, v and y are constants of the step.  lambda_i (AS_STAB_EXACT: exp(-c_i)) and the softmax
 * branch do not depend on the weights.  One-layer feature maps with F == d and no bias; anything else returns
 * AS_ERR_UNSUPPORTED.  With d = F = 128 on AS_PATH_TENSOR the products run on the tensor cores (bf16 operands, fp32
 * accumulation); every other supported shape, and AS_PATH_SIMT, in fp32 on CUDA cores.  Asynchronous on the stream;
 * sums in a fixed order (no float atomics), so results are run-to-run identical. */
AS_API as_status_t as_hybrid_attn_backward_workspace_bytes(as_hybrid_attn_t h, size_t* bytes);
AS_API as_status_t as_hybrid_attn_backward_phi(as_hybrid_attn_t h, const void* q, const void* k, const void* v,
                                               const as_phi_weights_t* w, const void* y_teacher, const void* y_hat,
                                               const float* aux, const void* forward_workspace, float* dWq, float* dWk,
                                               float* loss, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Test aid (no counterpart in the paper): enqueues a one-CTA kernel that waits, with the same bounded wait
 * every kernel of the library uses, on a barrier nobody arrives at; no copy and no tensor-core operation is
 * in flight.  After about `limit_cycles` SM clocks (1 .. 1e8) the wait gives up, the kernel returns and the
 * handle's status word is set exactly as by a time-out inside `forward`: as_hybrid_attn_last_status then
 * returns AS_ERR_DEVICE_TIMEOUT once, and the handle is usable again afterwards. */
AS_API as_status_t as_hybrid_attn_debug_expire_wait(as_hybrid_attn_t h, int64_t limit_cycles, void* cuda_stream);

/* Profiling aid (no counterpart in the paper): after `profile_enable(h, 1)` every kernel launch is bracketed by CUDA events on
 * the launching stream.  `profile_read` synchronises those events, adds the elapsed device time
 * per kernel class into ms[AS_NUM_KERNELS] and the launch counts into launches[AS_NUM_KERNELS],
 * and resets the counters.  At most 1024 launches are kept between two reads. */
AS_API as_status_t as_hybrid_attn_profile_enable(as_hybrid_attn_t h, int32_t enable);
AS_API as_status_t as_hybrid_attn_profile_read(as_hybrid_attn_t h, float* ms, int32_t* launches);

/* Total number of kernels this handle has launched since create.  (Utility: no counterpart in the paper.) */
AS_API as_status_t as_hybrid_attn_launch_count(as_hybrid_attn_t h, uint64_t* count);

/* The linear state S, z of one layer, computed WITHOUT allocating anything.  The paper has no
 * counterpart of this call: it exists for callers that cannot request device memory - a server
 * whose arena already owns all of HBM (cudaMalloc fails or is forbidden there), a plug-in that
 * may only touch the buffers its host framework handed it, a latency-critical loop that must
 * avoid the device-wide synchronisation inside cudaMalloc / cudaFree.  It needs no handle and
 * no workspace: the per-chunk partial sums live in a fixed 8 MiB array inside the library
 * image.  The CUDA driver sets that array up on a device when the library's code is first loaded
 * there - with the default lazy module loading that is this function's first call on the device,
 * with CUDA_MODULE_LOADING=EAGER it is context creation - and keeps it until the process exits.
 * A caller whose arena is about to take all of the device's memory therefore makes one call per
 * device beforehand (or sets CUDA_MODULE_LOADING=EAGER); if the 8 MiB cannot be had any more, that
 * first call returns AS_ERR_CUDA and launches nothing.
 *   k, v      [B,H,N,d] bf16 device, read only          wk  [H,d,d] bf16 device (F == d, one layer)
 *   grid_*, blk_*, rate_den, poly_degree                 as in as_hybrid_attn_desc_t (rule-based T_S)
 *   S_out     [B,H,d,d] fp32 device, written             z_out [B,H,d] fp32 device, written
 *             (one of the two may be NULL)
 * S = sum_{T_L} phi_k(k_j)^T v_j and z = sum_{T_L} phi_k(k_j), in fp32 on CUDA cores.
 * Limits: d in {64, 128}; B*H*d*(d+1)*4 bytes <= 8 MiB (B*H <= 127 at d = 128, <= 504 at d = 64);
 * anything larger returns AS_ERR_UNSUPPORTED and launches nothing.
 * The first call on a device looks up the array's device address and sets kernel attributes;
 * make that first call outside any stream capture.  No cudaMalloc, cudaFree or other allocating
 * routine is called, then or later.  Asynchronous on `cuda_stream`.  All calls share the one
 * array, which keeps the previous call's contents; every slot a call reads it has written first,
 * so nothing needs clearing, but two calls that overlap on the GPU (different streams or
 * threads) race on it - serialise them. */
AS_API as_status_t as_hybrid_attn_linear_state_static(
    const void* k, const void* v, const void* wk, int32_t B, int32_t H, int32_t N, int32_t d,
    int32_t grid_t, int32_t grid_h, int32_t grid_w, int32_t blk_t, int32_t blk_h, int32_t blk_w,
    int32_t rate_den, int32_t poly_degree, float* S_out, float* z_out, void* cuda_stream);

/* Block-rate selection (paragraph "Heterogeneous Block-Rate Optimization"): with n_blocks
 * transformer blocks and n_rates candidate hybrid rates, pick one rate per block so that the summed
 * error is minimal while the summed cost stays within `budget` (a multiple-choice knapsack problem).
 *   cost, err  [n_blocks, n_rates] float64, HOST, row-major, read only: c_ir (FLOPs, latency, ... any
 *              non-negative unit, e.g. per-layer times measured with this library) and e_ir (error
 *              of block i at rate r relative to softmax attention); all finite
 *   budget     beta, in the unit of `cost`; a summed cost equal to it is allowed
 *   choice_out [n_blocks] int32, HOST, written: the chosen rate index per block
 *   total_cost_out, total_err_out   HOST, written when not NULL: the sums over the chosen entries,
 *              added in block order
 * Exact (no cost discretisation): non-dominated partial assignments are carried from block to block.
 * Where several assignments reach the minimal error, one of them is returned.  Host code only; no
 * CUDA call, no stream.  Errors: AS_ERR_INVALID_ARG (NULL, non-positive sizes, NaN/inf or negative
 * cost), AS_ERR_INFEASIBLE (even the cheapest rates exceed the budget; outputs untouched),
 * AS_ERR_UNSUPPORTED (more than 2^22 non-dominated partial assignments), AS_ERR_ALLOC. */
AS_API as_status_t as_select_block_rates(int32_t n_blocks, int32_t n_rates, const double* cost, const double* err,
                                         double budget, int32_t* choice_out, double* total_cost_out,
                                         double* total_err_out);

/* Static description of a status code.  (Utility: no counterpart in the paper.) */
AS_API const char* as_status_string(as_status_t s);

#ifdef __cplusplus
}
#endif
#endif  /* AS_HYBRID_ATTN_H_ */
