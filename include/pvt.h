/*
 * pvt.h -- C ABI of the B200 (sm_100a) library for the discrete "V step" of
 * PV-Tuning on one vector-quantised linear layer.
 *
 * One training step of the method (Algorithm 3) dequantises the model, runs
 * forward/backward passes to accumulate the dense gradient of every linear
 * weight, updates the continuous parameters (P step) and then updates the
 * discrete codes (V step):
 *
 *     update = W - eta * g                  (Eq. 8: y - (1/L_S) Z(grad phi(y)))
 *     S      = choose_subspace(update, tau) (Algorithm 2: top-tau selection; Section
 *                                            3.4: by update size, per matrix)
 *     codes[S] = find_nearest(update[S])    (Appendix C / Appendix J: exhaustive
 *                                            search of one codebook, beam search
 *                                            for additive codebooks; codes
 *                                            outside S stay, Section 3.3)
 *
 * and the next step starts with dequantize_weights (Algorithm 3, first line).
 * This library is those three calls.
 *
 * Conventions
 *   - A layer is `rows x cols`, row-major.  Weight groups are `group_dim` = 8
 *     consecutive elements of a row (input dimension); group j = r * (cols/8) + c
 *     covers W[r, 8c .. 8c+7].  G = rows * cols / 8 groups, G < 2^32.
 *   - Every pointer is DEVICE memory owned by the caller (16-byte aligned where
 *     stated; index, error, move-count and status arrays 4-byte aligned; codes
 *     2-byte aligned when they are two-byte codes or pairs of one-byte codes).
 *     The library allocates nothing.  It keeps no per-layer state between calls; the
 *     only process-wide settings are the ones made through pvt_set_m1_search,
 *     pvt_timing_enable and pvt_test_wait_limit (all off / automatic by default),
 *     and pvt_vstep_select_noalloc remembers the address of its built-in scratch.
 *   - Every call only enqueues work on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and returns without synchronising,
 *     except pvt_status.  Calls on one stream execute in order.
 *   - Return value: PVT_OK (0) = enqueued; negative = rejected before anything
 *     was enqueued (see the error codes).  No C++ exception crosses this ABI.
 *   - Device-side problems never trap: the kernel records a PVT_DEV_* bit in the
 *     status word at the start of the workspace, skips the offending item and
 *     returns.  Read it with pvt_status.
 */
#ifndef PVT_H_
#define PVT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* element types */
#define PVT_F32 0
#define PVT_F16 1
#define PVT_U8 0
#define PVT_U16 1

/* host-side return codes */
#define PVT_OK 0
#define PVT_EINVAL (-1)       /* null / misaligned pointer, k = 0, k > G, cols % 8 != 0, G >= 2^32, bad eta */
#define PVT_EUNSUPPORTED (-2) /* group_dim / M / K / dtype / beam combination the library has no kernel for */
#define PVT_EWORKSPACE (-3)   /* ws_bytes smaller than pvt_workspace_bytes() */
#define PVT_ECUDA (-4)        /* a CUDA runtime call or kernel launch failed; see pvt_last_cuda_error() */
#define PVT_ETOOLARGE (-5)    /* pvt_vstep_select_noalloc only: the layer exceeds the built-in scratch */

/* device-side status bits (pvt_status) */
#define PVT_DEV_BAD_INDEX 1u    /* an entry of idx was >= G; that entry was skipped */
#define PVT_DEV_BAD_CODE 2u     /* a stored code was >= K; treated as code 0 (dequant) or left out of the pool */
#define PVT_DEV_WAIT_EXPIRED 4u /* a bounded wait on an on-chip barrier ran out; results of the call are invalid */
#define PVT_DEV_INTERNAL 8u     /* an internal consistency check failed (selection count mismatch) */

/*
 * One quantised linear layer and the update direction of this step.
 * Representation (Appendix J): M codebooks of K codewords of group_dim values
 * each, one code per group and codebook, per-output-channel scale:
 *     W_hat[r, 8c + i] = scale[r] * sum_m codebooks[m][codes[j][m]][i].
 * Supported: group_dim 8; M = 1 with 2 <= K <= 65536 (codes U8 if K <= 256, else
 * U16; U16 is accepted for any K); M = 2, 3, 4 with 2 <= K <= 256, codes U8, 1 <=
 * beam <= 8.  group_dim 16 (Appendix J's one-codebook representations
 * with groups of 16 weights): M = 1 only; every call but pvt_vstep_refine and
 * pvt_vstep_select_noalloc takes it; read "8" as "16" in the layouts below.
 */
typedef struct pvt_layer {
  int32_t rows, cols;     /* cols % group_dim == 0 */
  int32_t group_dim;      /* 8 (or 16 with one codebook) */
  int32_t num_codebooks;  /* M */
  int32_t codebook_size;  /* K */
  int32_t codebook_dtype; /* PVT_F32 | PVT_F16 */
  int32_t code_dtype;     /* PVT_U8 | PVT_U16 */
  int32_t beam;           /* beam width of the M >= 2 search; ignored for M = 1 */
  float eta;              /* step size 1/L_S of Eq. 8; finite, >= 0 */
  int32_t reserved_;      /* set to 0 */
  const float* W;         /* [rows][cols] current dense weight y (16-byte aligned) */
  const float* g;         /* [rows][cols] update direction: gradient or optimiser update (16-byte aligned) */
  const float* scale;     /* [rows] finite, non-zero (not validated) */
  const void* codebooks;  /* [M][K][group_dim] (16-byte aligned) */
  void* codes;            /* [G][M]; read (previous codes) and overwritten in place by pvt_vstep_encode */
} pvt_layer;

/*
 * Bytes of scratch that pvt_vstep_select / pvt_vstep_encode need for this layer
 * and this k (the larger of the two needs).  Returns 0 if the layer or k is
 * invalid.  The workspace must be 256-byte aligned; its first 256 bytes hold the
 * status word and must be cleared once with pvt_workspace_init before first use.
 */
size_t pvt_workspace_bytes(const pvt_layer* layer, uint64_t k);

/* Clears the status word of a fresh workspace (enqueued on the stream). */
int pvt_workspace_init(void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Subspace choice (the top-tau selection of Algorithm 2; Section 3.4 ranks by the size
 * of the update, separately for every weight matrix; choose_subspace of Algorithm 3).
 *   n_j = ||eta * g_j||^2 per group, in binary32: u_i = eta*g_i rounded once,
 *   acc = fma(u_i, u_i, acc) for i = 0..7 from acc = 0.
 *   idx_out[0..k) = the k groups with the largest n_j, ties at the threshold
 *   resolved towards the lowest group index, written in ascending order.
 * Reads layer->g, rows, cols, eta only.  idx_out: device, k uint32.
 * k is a count (1 <= k <= G); a fraction tau maps to k = max(1, floor(tau*G)).
 */
int pvt_vstep_select(const pvt_layer* layer, uint64_t k, uint32_t* idx_out, void* ws, size_t ws_bytes,
                     void* cuda_stream);

/*
 * pvt_vstep_select for callers that cannot allocate device memory.  (No
 * counterpart in the paper: this is a packaging variant of the call above and
 * computes exactly the same idx_out.)
 *
 * Who needs it: code that has to pick the subspace at a point where no device
 * allocation is possible -- a training process whose memory pool was handed out
 * completely at start-up, a component living inside a host application that
 * owns all device memory, or a thread that must not enter an allocator (a
 * cudaMalloc would also synchronise the device).  Such callers cannot supply the
 * ~5 bytes per group of workspace that pvt_vstep_select asks for.  Here the
 * scratch is a fixed array inside the library image instead; the caller passes
 * only the layer, k and the outputs.
 *
 * Limits and rules
 *   - At most PVT_NOALLOC_MAX_GROUPS groups (2^21, e.g. one 4096 x 4096 layer);
 *     a larger layer is rejected with PVT_ETOOLARGE before anything is enqueued.
 *   - The array (about 10.03 MiB) is held on every GPU on which the library's
 *     device code has been loaded, until the process exits.  The CUDA runtime may
 *     load that code lazily: then it is the first call of this function on a
 *     device that makes the array resident (and that load may synchronise the
 *     device and needs those 10 MiB to be free).
 *   - The first call on each device also looks up the array's device address (a
 *     host-side runtime query; the device must be current).  Make that first
 *     call at start-up -- before the memory is handed out completely and outside
 *     any stream capture; a call on a tiny layer will do.  From the second call
 *     on nothing is loaded or looked up.  The address is kept for the life of
 *     the process: a cudaDeviceReset unloads the array and leaves that address
 *     dangling, so a process that resets a device must not call this
 *     afterwards on that device.
 *   - Every call on a device uses the same array.  Calls whose kernels may
 *     overlap on the GPU (different streams, different host threads) race on it
 *     and give wrong results: issue them on one stream, or order them yourself.
 *     What must start at zero is cleared at the start of every call; nothing
 *     else of a previous call is relied upon.
 *   - The call issues no cudaMalloc / cudaFree and no allocating library routine,
 *     and apart from what the first call on a device may trigger (above) it does
 *     not synchronise.
 * status_out: NULL, or a device uint32 that receives the PVT_DEV_* bits of this
 * call (written by a copy enqueued after the kernels).
 * Other arguments and return codes as pvt_vstep_select.
 */
#define PVT_NOALLOC_MAX_GROUPS (1ull << 21)
int pvt_vstep_select_noalloc(const pvt_layer* layer, uint64_t k, uint32_t* idx_out, uint32_t* status_out,
                             void* cuda_stream);

/*
 * Subspace choice combined with a straight-through buffer (Appendix E: an auxiliary, non-quantised
 * copy of the weights that takes every update, so that updates too small to change a code add up
 * until they do; Section 3.4 and the "PV + STE" rows of Table 1 combine it with the subspace V step).
 * One pass over g does both:
 *   buffer[r, c] = fma(-eta, g[r, c], buffer[r, c])   for every weight (binary32, one fused operation),
 *   idx_out      = exactly what pvt_vstep_select returns (the k groups of largest ||eta g_j||^2).
 * The V step is then completed by pvt_vstep_encode on a descriptor with W = buffer and eta = 0: the
 * chosen groups are re-encoded against buffer / scale.  (Reading of the paper, which does not spell
 * the combination out: the buffer takes the step of every weight, the subspace is chosen by the size
 * of this step's update.)
 * buffer: device, rows x cols floats, 16-byte aligned, updated in place, must not alias g.  With
 * k = G the buffer is still updated.  Other arguments, workspace and return codes as pvt_vstep_select.
 */
int pvt_vstep_select_ste(const pvt_layer* layer, float* buffer, uint64_t k, uint32_t* idx_out, void* ws,
                         size_t ws_bytes, void* cuda_stream);

/*
 * Random subspaces (the small-scale experiments' appendix: instead of the greedy choice, S^k drawn
 * uniformly at random, or at random in proportion to the size of the gradient entries).  Every group
 * j gets the first output word r_j of the counter-based generator Philox-4x32 with 10 rounds (Salmon,
 * Moraes, Dror, Shaw, SC 2011) at counter (j mod 2^32, j div 2^32, 0, 0) and key (seed mod 2^32, seed
 * div 2^32); the k groups with the largest sampling key are returned in ascending order, ties towards
 * the lowest index:
 *   PVT_SAMPLE_UNIFORM       key_j = (float)(r_j >> 8): a uniformly random k-subset; g is not read.
 *   PVT_SAMPLE_PROPORTIONAL  key_j = (float)(n_j / E_j), n_j = ||eta g_j||^2 as in pvt_vstep_select,
 *                            E_j = -ln((r_j + 1/2) 2^-32): k draws without replacement, each in
 *                            proportion to n_j among the groups not yet drawn (exponential clocks);
 *                            groups with n_j = 0 get key 0.  E_j is a fixed sequence of binary64
 *                            operations (x = r + 1/2 = m 2^e, m in [1, 2), halved when above sqrt 2;
 *                            z = (m - 1)/(m + 1); p = 1 + z^2/3 + ... + z^20/21 by Horner's rule with
 *                            one fused operation per coefficient; E = fma(32 - e, ln 2, -(2 z p))),
 *                            the quotient is taken in binary64 and rounded once to binary32.
 * The same seed gives the same subspace on every device and run.  Workspace, idx_out and return
 * codes as pvt_vstep_select; PVT_EINVAL for an unknown rule.
 */
#define PVT_SAMPLE_UNIFORM 0
#define PVT_SAMPLE_PROPORTIONAL 1
int pvt_vstep_sample(const pvt_layer* layer, uint64_t k, int32_t rule, uint64_t seed, uint32_t* idx_out, void* ws,
                     size_t ws_bytes, void* cuda_stream);

/*
 * Re-encode the k groups listed in idx (Eq. 8; Appendix C / Appendix J;
 * Appendix D for the score ||c||^2 - 2 <t, c>).
 *   target (binary32): t_i = fma(-eta, g_i, W_i) / scale[r].
 *   M = 1: codes[j] = argmin over all K codewords of (||t - c||^2, code).
 *   M = 2: greedy residual beam search: the `beam` codewords of codebook 1
 *          nearest to t under (distance, code); each is extended by every
 *          codeword of codebook 2; the pool is those beam*K pairs plus the
 *          previous pair; codes[j] = argmin of (||t - c1 - c2||^2, code1, code2).
 *   M = 3, 4: the same search carried through more stages: after each stage but
 *          the last the `beam` smallest partial tuples under (||t - c1 - ... -
 *          cm||^2, tuple) are kept; the pool is the last stage's beam*K tuples
 *          plus the previous tuple.
 *   A fast binary32 score shortlists candidates; the decision among shortlisted
 *   candidates is taken on binary64 distances sum_i (t_i - c_i)^2 accumulated in
 *   index order, so ties break exactly as stated above.
 *   Groups not in idx keep their codes bit for bit.
 * idx: device, k uint32, each < G, no duplicates (duplicates race benignly: the
 * same value is written twice).  err_out: device, k floats or NULL; receives the
 * new squared error in the scaled space, rounded to binary32.
 */
int pvt_vstep_encode(const pvt_layer* layer, const uint32_t* idx, uint64_t k, float* err_out, void* ws,
                     size_t ws_bytes, void* cuda_stream);

/*
 * V step whose subspace size comes from a trust ratio (Section 4.3 sets tau so that the
 * relative change ||x_new - x_old|| / ||x_old|| of a step stays at one per cent; the
 * hyper-parameter paragraph of Appendix J takes the largest such count, found by
 * re-encoding a hundredth of the weights at a time in the order of decreasing update
 * norm and undoing codes from the end of the last portion, and always lets one weight
 * change).  x is the dequantised matrix W_hat of this layer.
 *
 * What is computed: the k_max groups of largest ||eta*g_j||^2 are ranked by
 * (norm descending, index ascending) and all re-encoded as by pvt_vstep_encode.
 * With d_r the squared change of the dequantised weights of the group at rank r
 * (binary64 sum, in element order, of squared differences of the binary32 values
 * pvt_dequant would write before and after), n is the first rank at which
 * d_0 + ... + d_r < ratio^2 * ||W_hat_old||^2 fails (binary64; k_max if it never
 * fails; at least 1).  Ranks 0 .. n-1 keep their new codes, ranks n .. k_max-1
 * get their previous codes back, every other group is untouched.  This equals
 * the appendix's procedure whenever n < k_max; n == k_max says the cap was
 * reached before the bound.
 *
 * idx_out: device, k_max uint32: group indices in rank order (the first *n_out
 *          are the subspace).  n_out: device uint64.  stats_out: NULL or device
 *          double[2]: ||W_hat_old||^2 and the squared change that was kept.
 * ws: pvt_trust_workspace_bytes(layer, k_max) bytes, 256-byte aligned, header
 *     cleared by pvt_workspace_init; status bits as for the other calls.
 * Two to four codebooks need one-byte codes and 1 <= beam <= 8 (PVT_EUNSUPPORTED).
 * Returns as pvt_vstep_encode; ratio must be finite and >= 0 (PVT_EINVAL).
 */
size_t pvt_trust_workspace_bytes(const pvt_layer* layer, uint64_t k_max);
int pvt_vstep_trust(const pvt_layer* layer, uint64_t k_max, float ratio, uint32_t* idx_out, uint64_t* n_out,
                    double* stats_out, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Local search over single-code changes (Appendix D: the neighbourhood N_1 of
 * assignments that differ in one index, and the search that moves to the best
 * neighbour while the squared error drops) for the groups listed in idx, started
 * from the codes that are stored -- e.g. right after pvt_vstep_encode, whose
 * two-codebook beam search is a heuristic.  The squared error is a sum over
 * groups, so each group is searched on its own:
 *   error(b) = ||t - sum_m C_m[b_m]||^2 with the target t of pvt_vstep_encode, in
 *   binary64 (residual through the codebooks in order, elements in order);
 *   one move: among the M*(K-1) tuples that differ from the current one in one
 *   code, the smallest under (error, tuple); taken only if its error is strictly
 *   below the current error; at most max_moves moves (0 <= max_moves <= 65535).
 * The error never rises; for one codebook a single move reaches the exhaustive
 * optimum.  codes[idx[i]] is rewritten when the group moved.
 * err_out: NULL or device float[k], final error rounded to binary32.  moves_out:
 * NULL or device uint32[k], moves taken.  status: NULL or a device uint32 into
 * which PVT_DEV_BAD_INDEX / PVT_DEV_BAD_CODE are OR-ed (such groups are skipped).
 * No workspace.  Two to four codebooks need one-byte codes (PVT_EUNSUPPORTED).
 */
int pvt_vstep_refine(const pvt_layer* layer, const uint32_t* idx, uint64_t k, int32_t max_moves, float* err_out,
                     uint32_t* moves_out, uint32_t* status, void* cuda_stream);

/*
 * dequantize_weights (Algorithm 3, first line): for every group
 *   W_hat[r, 8c+i] = scale[r] * (C_1[b_1][i] (+ C_2[b_2][i] + ...))   in binary32,
 *   the codebooks added left to right with each sum rounded once, then the product
 *   rounded once; out_dtype PVT_F16 rounds that binary32 value to nearest-even
 *   binary16.
 * W_hat: device, rows x cols of out_dtype, 16-byte aligned.  `status` may be NULL
 * or a device uint32 into which PVT_DEV_BAD_CODE is OR-ed.
 */
int pvt_dequant(const pvt_layer* layer, void* W_hat, int32_t out_dtype, uint32_t* status, void* cuda_stream);

/*
 * The V step over every linear layer of a model block in one call (Algorithm 3, V-step lines: the loop over
 * the quantised weights; the subspace is chosen inside each weight matrix, Section 3.4, so the layers are
 * independent): for i = 0 .. n_layers-1, in order, on the one stream,
 *     pvt_vstep_select(layers[i], k[i]) -> idx_out[i];  pvt_vstep_encode(layers[i], idx_out[i], k[i]);
 *     pvt_dequant(layers[i]) -> W_hat[i]   (skipped when W_hat or W_hat[i] is NULL).
 * A convenience that adds no arithmetic of its own.  layers, k, idx_out, W_hat: HOST arrays of n_layers
 * entries (descriptors, subspace sizes, device pointers to k[i] uint32, device pointers to rows x cols of
 * out_dtype).  ws: one device workspace shared by all layers, at least pvt_block_workspace_bytes (the largest
 * per-layer need), header cleared by pvt_workspace_init; status bits of all layers accumulate in it.
 * Every layer is validated before anything is enqueued; return codes as the three calls.
 */
size_t pvt_block_workspace_bytes(const pvt_layer* layers, const uint64_t* k, int32_t n_layers);
int pvt_vstep_block(const pvt_layer* layers, const uint64_t* k, int32_t n_layers, uint32_t* const* idx_out,
                    void* const* W_hat, int32_t out_dtype, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * P step, the half that shares its inputs with the V step (Algorithm 3, P-step lines:
 * grad_codebooks = backprop(grad_phi)).  Chain rule through dequantize_weights,
 * W_hat[r, 8c+i] = scale[r] * v[j][i], v[j] = sum_m C_m[codes[j][m]] (the binary32 sum
 * pvt_dequant forms):
 *   grad_codebooks[m][kappa][i] = sum over groups j with codes[j][m] == kappa of scale[r(j)] * g[j][i]
 *   grad_scale[r]               = sum over the groups j of row r and over i of g[j][i] * v[j][i]
 * Products are exact in binary64; sums are accumulated in binary64 in an order that
 * is not fixed (atomic adds, or per-block sorted partial sums for small codebooks), so
 * results vary from run to run in the order of binary64 roundings only.
 * Reads layer->g, scale, codes, codebooks, shape.  grad_codebooks: device, M*K*group_dim doubles;
 * grad_scale: device, rows doubles, or NULL.  Both are overwritten.  `status` may be NULL
 * or a device uint32 into which PVT_DEV_BAD_CODE is OR-ed (such groups contribute nothing).
 */
int pvt_pstep_grad(const pvt_layer* layer, double* grad_codebooks, double* grad_scale, uint32_t* status,
                   void* cuda_stream);

/*
 * One Adam update of n binary32 parameters (Algorithm 3: codebooks = adam(grad_codebooks);
 * Section 3.4; Appendix J: beta1 = 0.9, beta2 = 0.95).  The binary64 gradient is rounded
 * once to binary32 (gr); then, in binary32, every operation rounded once:
 *   m = fma(beta1, m, (1 - beta1) * gr)        v = fma(beta2, v, ((1 - beta2) * gr) * gr)
 *   p = p - (lr * (m / bias1)) / (sqrt(v / bias2) + eps)
 * with bias1 = 1 - beta1^t, bias2 = 1 - beta2^t of step t >= 1 supplied by the caller.
 * param, exp_avg, exp_avg_sq: device, n floats, updated in place.  param_f16: NULL, or
 * device n halves that receive the updated parameters rounded to nearest-even (the
 * fp16 codebook the V step reads).  grad: device, n doubles.
 */
int pvt_adam_update(float* param, void* param_f16, const double* grad, float* exp_avg, float* exp_avg_sq, uint64_t n,
                    float lr, float beta1, float beta2, float eps, float bias1, float bias2, void* cuda_stream);

/*
 * Update direction of the V step as the paper runs it (Section 3.4: grad phi(y) of Eq. 8 is
 * replaced by a single Adam update, and the subspace is chosen by the magnitude of that
 * update; the update line of Algorithm 3's V step).  Per weight, binary32,
 * every operation rounded once:
 *   m = fma(beta1, m, (1 - beta1) * g)        v = fma(beta2, v, ((1 - beta2) * g) * g)
 *   dir = (m / bias1) / (sqrt(v / bias2) + eps)
 * The V step then runs with layer->g = dir and layer->eta = the learning rate of the codes.
 * grad, exp_avg, exp_avg_sq, dir: device, n floats, 16-byte aligned, n % 4 == 0 (n = rows *
 * cols of a layer); exp_avg and exp_avg_sq are updated in place; dir may alias grad.
 * bias1 = 1 - beta1^t, bias2 = 1 - beta2^t of step t >= 1.
 */
int pvt_adam_direction(const float* grad, float* exp_avg, float* exp_avg_sq, float* dir, uint64_t n, float beta1,
                       float beta2, float eps, float bias1, float bias2, void* cuda_stream);

/*
 * Bias corrections of Adam's step t >= 1 as the two calls above take them (Section 3.4; Appendix J
 * betas): bias = 1 - beta^t, the power taken in binary64 from the binary32 beta, the difference
 * rounded once to binary32.  Host arithmetic only; bias1_out, bias2_out: host.  PVT_EINVAL for
 * step = 0, a beta outside [0, 1) or a null pointer.
 */
int pvt_adam_bias(uint64_t step, float beta1, float beta2, float* bias1_out, float* bias2_out);

/*
 * Synchronises the stream, returns the PVT_DEV_* bits accumulated in the
 * workspace since the last pvt_status / pvt_workspace_init (>= 0) and clears them;
 * or PVT_ECUDA.
 */
int pvt_status(void* ws, void* cuda_stream);

/* Text for a host-side return code. */
const char* pvt_strerror(int code);

/* Text of the CUDA error behind the most recent PVT_ECUDA on this thread. */
const char* pvt_last_cuda_error(void);

/* Library version: major * 10000 + minor * 100 + patch. */
int pvt_version(void);

/*
 * Engine of the single-codebook search (no counterpart in the paper; both engines
 * compute the same codes).  PVT_M1_AUTO, the default: tensor cores (tcgen05) for
 * fp16 codebooks of at least 1024 codewords, the FP32 pipe otherwise.
 * PVT_M1_FP32: always the FP32 pipe.  PVT_M1_TENSOR: tensor cores for every fp16
 * codebook.  Process-wide; it also changes what pvt_workspace_bytes returns, so
 * set it before sizing workspaces.  Other values are ignored.
 */
#define PVT_M1_AUTO 0
#define PVT_M1_FP32 1
#define PVT_M1_TENSOR 2
void pvt_set_m1_search(int mode);

/*
 * Benchmark instrumentation (no counterpart in the paper).  While enabled, every
 * call brackets its kernels with CUDA events on the caller's stream;
 * pvt_timing_read waits for the recorded events of one kernel class, returns
 * their summed duration and count, and forgets them.
 */
#define PVT_KERNEL_SELECT 0      /* all kernels of pvt_vstep_select */
#define PVT_KERNEL_ENCODE_MAIN 1 /* the search kernel of pvt_vstep_encode */
#define PVT_KERNEL_ENCODE_AUX 2  /* codebook expansion before the M = 1 search */
#define PVT_KERNEL_DEQUANT 3     /* the kernel of pvt_dequant */
#define PVT_KERNEL_ENCODE_RESCORE 4 /* exact rescoring and code write after the M = 1 search */
#define PVT_KERNEL_PSTEP_GRAD 5  /* the kernel of pvt_pstep_grad */
#define PVT_KERNEL_ADAM 6        /* the kernel of pvt_adam_update */
#define PVT_KERNEL_TRUST 7       /* ranking, norm and code saving of pvt_vstep_trust (before its search) */
#define PVT_KERNEL_REFINE 8      /* the kernel of pvt_vstep_refine */
void pvt_timing_enable(int on);
/* FP32 FMA throughput of the current device, measured: a kernel of independent FMA chains on every SM, timed with
 * CUDA events (synchronises).  scratch: device, at least 2048 floats per SM.  tflops_out: host. */
int pvt_probe_fp32_tflops(float* scratch, size_t scratch_floats, float* tflops_out, void* cuda_stream);
/* Kernels this process has launched through the library so far (memsets not counted). */
unsigned long long pvt_launch_count(void);
int pvt_timing_read(int kernel_id, float* total_ms, int* launches);

/*
 * Test hook for the give-up path of the on-chip waits (no counterpart in the paper).  Every wait of
 * the single-codebook search kernels on an on-chip barrier polls a bounded number of times; when
 * the bound is reached the kernel stops, lets the copies and tensor-core work it has issued finish,
 * frees its tensor memory and returns, and pvt_status reports PVT_DEV_WAIT_EXPIRED (the codes of
 * that call are then not written, and PVT_DEV_INTERNAL is set as well).  In normal operation the
 * bound (2^22 polls) is never reached.  This call lowers it to max_polls (0 restores the default)
 * and, if withhold_copy >= 0, makes every thread block leave out the codebook copy with that
 * sequence number, so that a wait provably runs out without anything being left in flight.
 * Process-wide; affects calls enqueued afterwards.  Never use it outside tests.
 */
void pvt_test_wait_limit(uint32_t max_polls, int64_t withhold_copy);

#ifdef __cplusplus
}
#endif
#endif /* PVT_H_ */
