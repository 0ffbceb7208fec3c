/*
 * idkm.h -- C ABI of the IDKM hot path on one CUDA device (sm_100a).
 *
 * IDKM ("Memory Efficient Neural Network Quantization via Implicit, Differentiable k-Means")
 * clusters a layer's m weight-vectors w_i in R^d around k = 2^b codewords c_j with a soft,
 * attention-based k-means (Section 3.2, Algorithm 1), treats the result as the solution of the
 * fixed-point equation C* = F(C*, W) (Section 4.1) and differentiates it either implicitly
 * (Section 4.2) or with Jacobian-free backpropagation (Section 4.3).
 *
 * Shapes and layout.  All tensors are fp32, row-major, in DEVICE memory unless a parameter says
 * "host":  W, Wq, dWq, dW are [m][d];  C0, C, dC are [k][d] ([n_layers][k][d] when batched);
 * A is [m][k].  Every pointer must be 16-byte aligned.  d is 1, 2 or 4; 1 <= k <= 256.
 *
 *   D_ij = ||w_i - c_j||_2,  A_ij = softmax_j(-D_ij / tau)            (Algorithm 1, steps 3-4)
 *   F(C, W)_j = sum_i A_ij w_i / sum_i A_ij                           (Algorithm 1, step 5)
 *   Wq_i = sum_j A_ij c_j                                             (soft quantiser r_tau)
 *
 * Ownership.  The caller owns every buffer, including the workspace; the library borrows them
 * and allocates no device memory in the device-pointer entry points (idkm_create allocates a few
 * bytes of bookkeeping on the host only).  Calls are asynchronous on the given CUDA stream.
 * From idkm_forward* until the matching idkm_backward returns, W, C_out and the workspace must
 * stay valid and unmodified: the backward recomputes the attention matrix from W and C_out and
 * reads the column sums and map values stashed in the workspace by the forward's final pass.
 *
 * Errors.  Every function returns an int status (IDKM_OK = 0, negative = error) and never
 * throws, aborts or traps the device.  Argument and launch errors come back synchronously.
 * Conditions that only the device can see (non-finite values, a diverging adjoint iteration,
 * the iteration cap reached before the tolerance) are reported in idkm_info.status after
 * idkm_get_info.
 */
#ifndef IDKM_H
#define IDKM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define IDKM_MAX_K 256
#define IDKM_MAX_LAYERS 64

/* status codes */
#define IDKM_OK 0
#define IDKM_MAXITER 1           /* advisory: iteration cap reached before the tolerance        */
#define IDKM_ERR_NULL (-1)       /* a required pointer is NULL                                  */
#define IDKM_ERR_ALIGN (-2)      /* a pointer is not 16-byte aligned                            */
#define IDKM_ERR_SHAPE (-3)      /* m < 1, bad layer offsets, n_layers out of range             */
#define IDKM_ERR_UNSUPPORTED (-4)/* d not in {1,2,4} or k not in [1,256]                        */
#define IDKM_ERR_PARAM (-5)      /* tau <= 0, tol < 0, max_iter < 0, alpha not in (0,1], ...    */
#define IDKM_ERR_WORKSPACE (-6)  /* workspace smaller than idkm_workspace_bytes()               */
#define IDKM_ERR_ORDER (-7)      /* idkm_backward without a preceding idkm_forward              */
#define IDKM_ERR_CUDA (-8)       /* a CUDA runtime call failed                                  */
#define IDKM_ERR_NONFINITE (-9)  /* device: NaN/Inf met in W, C or the sums                     */
#define IDKM_ERR_NOALLOC_TOO_LARGE (-11) /* idkm_step_noalloc: the problem needs more than the built-in scratch */
#define IDKM_ERR_TIMEOUT (-12)   /* device: a bounded grid-wide wait of the one-launch forward loop ran out  */
#define IDKM_ERR_DIVERGED (-10)  /* device: adjoint iteration produced non-finite values, its residual
                                    grew 10 steps running, or ||u|| passed 1e6 ||g|| (Section 4.2:
                                    retry with a smaller alpha, see idkm_backward_restart)      */

typedef struct idkm_ctx idkm_ctx; /* opaque; remembers the last forward call for the backward */

typedef enum { IDKM_IMPLICIT = 0, IDKM_JFB = 1 } idkm_mode;

/* One record per layer, filled by idkm_get_info. */
typedef struct {
  int32_t status;         /* IDKM_OK, IDKM_MAXITER or a device-side error                      */
  int32_t fwd_iters;      /* applications of F made by the forward loop                        */
  float   fwd_residual;   /* ||C+ - C||_F / ||C+||_F of the last application                   */
  int32_t dead_clusters;  /* clusters whose column sum fell below 1e-20 in the last step       */
  int32_t adj_iters;      /* adjoint iterations made by the last backward                      */
  float   adj_residual;   /* ||u+ - u||_F / ||u+||_F of the last adjoint iteration             */
} idkm_info;

/* Create / destroy a context bound to the current CUDA device.  Host allocation only. */
int  idkm_create(idkm_ctx** out);
void idkm_destroy(idkm_ctx* ctx);

/* Bytes of device workspace the forward and backward need for a problem of m_total rows in
 * n_layers layers (1 for the single-layer calls).  Returns 0 for unsupported d or k.  Besides the
 * per-layer state and the per-block partial sums it holds, for most codebooks of more than 8
 * centroids, 8 bytes per row: each row's softmax reference and normaliser, which the codebook-
 * gradient pass leaves for the adjoint steps (the iteration of Section 4.2 re-evaluates the same attention
 * rows at every step). */
size_t idkm_workspace_bytes(int64_t m_total, int d, int k, int n_layers);

/*
 * Forward: Algorithm 1 (soft k-means) followed by the soft quantiser (Section 3.2).
 *
 * Starting from C0, applies C <- F(C, W) until the relative change ||C+ - C||_F / ||C+||_F drops
 * below tol, or max_iter applications were made (tol = 0: exactly max_iter applications;
 * max_iter = 0: C_out = C0).  The loop runs on the device: each application is one fused launch
 * that never stores the m x k attention matrix, and the convergence test is made by the device
 * without a host round trip per iteration (launches queued after convergence return at once; with
 * tol > 0 the host queues 16 iterations at a time, peeks at a flag the device sets when every layer
 * has converged and stays at most 32 iterations ahead of the device, so such a call may block the
 * calling thread until the loop is within 32 iterations of its end).  A cluster whose
 * column sum is below 1e-20 keeps its centroid.  Then one final pass at the returned centroids
 * writes Wq = A C (Wq_out, may be NULL), optionally A itself (A_out, may be NULL: m*k floats, the
 * paper's O(m 2^b) term), and stashes S_j = sum_i A_ij and F(C, W)_j in the workspace.
 *
 * C_out receives the last C+ ("return C+", Algorithm 1).  C0 and C_out may alias.
 */
int idkm_forward(idkm_ctx* ctx, const float* W, int64_t m, int d, const float* C0, int k, float tau, float tol,
                 int max_iter, float* C_out, float* A_out, float* Wq_out, void* workspace, size_t workspace_bytes,
                 void* cuda_stream);

/*
 * Batched forward: the same for n_layers independent layers that share d, k, tau, tol and
 * max_iter ("for all layers", Algorithm 2), in the same launches.  W_cat holds the layers' rows
 * back to back; layer l owns rows [layer_offsets[l], layer_offsets[l+1]) (HOST array of
 * n_layers+1 increasing int64, first entry 0); C0 / C_out are [n_layers][k][d]; A_out / Wq_out
 * follow W_cat's row order.  Each layer converges (and stops being touched) on its own.
 * 1 <= n_layers <= IDKM_MAX_LAYERS.
 */
int idkm_forward_batched(idkm_ctx* ctx, const float* W_cat, const int64_t* layer_offsets, int n_layers, int d,
                         const float* C0, int k, float tau, float tol, int max_iter, float* C_out, float* A_out,
                         float* Wq_out, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward of L = <dWq, Wq(W, C*(W))> at the centroids returned by the last forward of this ctx.
 *
 * IDKM_IMPLICIT (Section 4.2): solves u = J_C^T u + g, J_C = dF/dC, by the averaged iteration
 *   u <- alpha (J_C^T u + g) + (1 - alpha) u from u = g, until the relative change of u is below
 *   adj_tol or adj_max_iter steps were made (adj_tol = 0: exactly adj_max_iter steps).  This is
 *   the vector form of the paper's iteration M <- alpha ((dF/dC) M + I) + (1 - alpha) M for
 *   M* = (I - dF/dC)^-1, contracted with g (u* = M*^T g); alpha = 1 is the plain iteration, the
 *   paper uses 0.25.  Each step is one fused vector-Jacobian pass over W; nothing is stored per step.
 * IDKM_JFB (Section 4.3): M* = I, i.e. u = g and no adjoint iterations.
 *
 * g = (dWq/dC)^T dWq is the direct codebook gradient.  Outputs:
 *   dW_out [m][d] = (dWq/dW)^T dWq + (dF/dW)^T u     (may be NULL)
 *   dC_out [k][d] ([n_layers][k][d]) = u             (may be NULL)
 * dWq has W's shape; dW_out must not alias dWq or W.  workspace must be the forward's.
 */
int idkm_backward(idkm_ctx* ctx, const float* dWq, idkm_mode mode, float adj_tol, int adj_max_iter, float alpha,
                  float* dW_out, float* dC_out, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Waits for the ctx's stream and copies one idkm_info per layer of the last forward to the HOST
 * array info_out (n_layers entries; 1 for idkm_forward). */
int idkm_get_info(idkm_ctx* ctx, idkm_info* info_out);

/*
 * Residual history of the last forward (which = 0: relative change of C after each application of F, the quantity
 * of the stop rule of Algorithm 1) or of the last implicit backward (which = 1: relative change of u after each
 * adjoint step) of one layer.  Waits for the ctx's stream, then copies min(iterations run, 1024, capacity) floats to
 * the HOST array host_out, first iteration first, and writes that count to *n_out.  The ratio of successive entries
 * estimates the contraction rate of the iteration (the spectral radius of dF/dC near a fixed point).
 * Returns IDKM_OK, IDKM_ERR_NULL, IDKM_ERR_ORDER (no forward yet), IDKM_ERR_PARAM or IDKM_ERR_CUDA.
 */
int idkm_get_history(idkm_ctx* ctx, int which, int layer, float* host_out, int capacity, int* n_out);

/*
 * Whole hot path on HOST buffers (Algorithm 2's per-layer work: cluster, quantise, differentiate):
 * copies W, C0 and dWq to the device, runs idkm_forward_batched and idkm_backward, and copies
 * C, Wq, dW, dC back; returns after everything has completed.  Device buffers are allocated on
 * first use, kept in the ctx and grown on demand (with idkm_quantize_host_ex the only entry point that
 * allocates device memory); the work runs on two streams of the ctx's own, so that the upload of dWq
 * overlaps the forward loop and the download of C and Wq overlaps the backward (host buffers must be
 * page-locked for the overlap to happen; pageable buffers work, serially).
 * Any of Wq_out, dW_out, dC_out may be NULL; info_out (n_layers entries) too.
 * layer_offsets as in idkm_forward_batched (pass {0, m} and n_layers = 1 for one layer).
 */
int idkm_quantize_host(idkm_ctx* ctx, const float* W_host, const int64_t* layer_offsets, int n_layers, int d,
                       const float* C0_host, int k, float tau, float tol, int max_iter, const float* dWq_host,
                       idkm_mode mode, float adj_tol, int adj_max_iter, float alpha, float* C_out_host,
                       float* Wq_out_host, float* dW_out_host, float* dC_out_host, idkm_info* info_out);

/*
 * The same with both gradients of Sections 4.2 and 4.3 from one forward: when mode is IDKM_IMPLICIT and
 * dW_jfb_out_host or dC_jfb_out_host is given (HOST, shapes of dW_out / dC_out), the Jacobian-free backward
 * (IDKM_JFB) runs as well, after the forward and before the implicit backward, and its results are copied there.
 * With both NULL this is idkm_quantize_host.  info_out describes the implicit backward.
 */
int idkm_quantize_host_ex(idkm_ctx* ctx, const float* W_host, const int64_t* layer_offsets, int n_layers, int d,
                          const float* C0_host, int k, float tau, float tol, int max_iter, const float* dWq_host,
                          idkm_mode mode, float adj_tol, int adj_max_iter, float alpha, float* C_out_host,
                          float* Wq_out_host, float* dW_out_host, float* dC_out_host, float* dW_jfb_out_host,
                          float* dC_jfb_out_host, idkm_info* info_out);

/*
 * Phase timing.  idkm_set_timing(ctx, 1) makes the following forward / backward calls record CUDA
 * events on their stream between phases (a few microseconds per call; events are created on the
 * first enable).  idkm_get_phase_ms waits for the last recorded call and writes six elapsed times in
 * milliseconds to the HOST array ms_out: [0] state initialisation, [1] the loop of fused forward
 * steps (Algorithm 1), [2] the final pass, [3] the direct codebook-gradient pass, [4] the loop of
 * adjoint steps (Section 4.2), [5] the pass that writes dL/dW.  A phase that has not run is -1.
 */
int idkm_set_timing(idkm_ctx* ctx, int enable);
int idkm_get_phase_ms(idkm_ctx* ctx, float* ms_out);

/*
 * One application of the map, C_out = F(C_in, W), that allocates nothing.  (The paper has no
 * counterpart: this exists for callers, not for the method.)
 *
 * For code that cannot obtain device memory at the point of the call: an allocator or memory-pool
 * callback, a server that gave its whole device budget to a fixed arena at start-up, a plug-in that may
 * not touch its host's CUDA allocator.  Such callers cannot supply the workspace the other entry points
 * ask for.  Here the bookkeeping of the fused step (per-block partial sums and the layer's ticket and
 * counters) lives in a fixed array of IDKM_NOALLOC_SCRATCH_BYTES inside the library image; every GPU
 * that loads the library holds those bytes until the process exits.  The call makes no cudaMalloc,
 * cudaFree or other allocating call and needs no idkm_ctx.
 *
 * W [m][d], C_in [k][d], C_out [k][d] are device pointers, 16-byte aligned, owned by the caller; C_in and
 * C_out may alias.  The result is that of idkm_forward with max_iter = 1 (same kernels; the cross-block sums
 * may be grouped differently because this entry point launches at most two blocks per SM).  Asynchronous on
 * cuda_stream.
 *
 * Limits and sharing.  With B = min(2 * SM count, tiles of the layer) blocks and P = padded k * (d+1) doubles
 * per row of partial sums, the call needs 256 + 1024 + (B + 1) * P * 8 + ((B + 1) / 16 + 3) * P * 8 bytes and
 * returns IDKM_ERR_NOALLOC_TOO_LARGE when that exceeds IDKM_NOALLOC_SCRATCH_BYTES.  The largest supported
 * codebook (d = 4, k = 256: P = 1280) needs 3.3 MB on a 148-SM B200, so every supported (d, k) fits there; the
 * check guards parts with more SMs.  All calls on a device share the one array, which still holds the previous
 * call's contents when the next begins: the call clears what must start at zero itself, but two calls that
 * overlap on the GPU (different streams, or different host threads) race on it -- serialise them.
 * The first call on each device looks up the array's device address (with that device current) and the
 * SM count, under a lock, so concurrent first calls from several host threads are safe; make that first call
 * outside any stream capture.
 */
#define IDKM_NOALLOC_SCRATCH_BYTES (4u << 20)
int idkm_step_noalloc(const float* W, int64_t m, int d, const float* C_in, int k, float tau, float* C_out,
                      void* cuda_stream);

/*
 * Device-side status of the last idkm_step_noalloc on the current device (the paper has no counterpart).  The step
 * is asynchronous and has no context to report through: a NaN or Inf in W, C_in or the sums is recorded in the
 * built-in array.  This call copies that one word to *status_host_out (IDKM_OK or IDKM_ERR_NONFINITE) on
 * cuda_stream and waits for the stream; it allocates nothing.  Returns IDKM_OK, IDKM_ERR_NULL or IDKM_ERR_CUDA.
 */
int idkm_step_noalloc_status(int* status_host_out, void* cuda_stream);

/*
 * How IDKM_IMPLICIT runs the adjoint iteration.  0 (default): where k d <= 64 one pass over W forms the k d x k d
 * matrix dF/dC explicitly and the whole iteration u <- alpha (J^T u + g) + (1 - alpha) u then runs on that matrix on
 * the device -- the paper's own formulation (it iterates a k x k matrix, Section 4.2), same iterates, one pass
 * instead of adj_max_iter.  For k d <= 8 always; for 8 < k d <= 64 (the pass costs about ten fused passes) when
 * adj_max_iter >= 16.  Larger codebooks, and shorter iterations, use one fused vector-Jacobian pass per step.
 * 1: always the fused passes.
 * 2: no iteration where the matrix can be formed (k d <= 64): the same pass forms dF/dC and one warp then solves
 * (I - (dF/dC)^T) u = g exactly -- the system behind M* = (I - dF/dC)^-1 of Section 4.2 -- by Gaussian elimination
 * with partial pivoting in fp64; adj_tol, adj_max_iter (> 0) and alpha are ignored, idkm_info reports 0 adjoint
 * iterations, and a singular system (an eigenvalue 1 of dF/dC) or a non-finite solution reads IDKM_ERR_DIVERGED.
 * The result is the limit of the iteration where that converges, and is defined (and returned) also where the
 * iteration would diverge.  Larger codebooks iterate fused passes as with 1.
 */
int idkm_set_adjoint_method(idkm_ctx* ctx, int method);

/*
 * Implicit backward with the safeguard of Section 4.2 ("if we see the iteration diverge, we start over and divide
 * alpha by 2"): runs the codebook gradient and the adjoint iteration of idkm_backward(IDKM_IMPLICIT) with
 * alpha = alpha0, reads the status (this WAITS for the stream after every attempt), and while any layer reports
 * IDKM_ERR_DIVERGED starts over from u = g with half the alpha, at most max_halvings times (0 <= max_halvings <= 30).
 * Then the dL/dW pass and the copy of dC run once, from the last attempt's u.  The alpha of the last attempt and the
 * number of attempts go to the HOST locations alpha_used_out / attempts_out (may be NULL).  Whether the last attempt
 * diverged too is in idkm_info.status, as for idkm_backward.  Halving helps where dF/dC has eigenvalues outside the
 * unit circle whose real part is below 1 (complex pairs occur at centroids that are not yet a fixed point); an
 * eigenvalue above 1 on the real axis defeats every alpha.  Other arguments and return values as idkm_backward.
 */
int idkm_backward_restart(idkm_ctx* ctx, const float* dWq, float adj_tol, int adj_max_iter, float alpha0,
                          int max_halvings, float* dW_out, float* dC_out, void* workspace, size_t workspace_bytes,
                          void* cuda_stream, float* alpha_used_out, int* attempts_out);

/*
 * Which distance the softmax of the E-step takes.  0 (default): the Euclidean norm, D_ij = ||w_i - c_j||_2, as
 * Algorithm 1 (step 3) and the equation for a_j(w_i, C) state it.  1: its square, D_ij = ||w_i - c_j||_2^2, the
 * distance in which the clustering objectives are written (the k-means objective of Section 3.1 and the soft
 * objective of Section 3.2); A_ij is then the posterior of an equal-weight mixture of isotropic Gaussians of variance
 * tau / 2, the gradient dD_ij/dw_i = 2 (w_i - c_j) has no kink at w_i = c_j, and a pair costs one special-function
 * operation (the exponential) instead of two.  Everything else -- F, Wq, the implicit and Jacobian-free gradients,
 * statuses -- is defined as above with that D.  Applies to the following idkm_forward* / idkm_backward /
 * idkm_quantize_host* calls of the ctx; a backward must follow a forward made with the same setting (else
 * IDKM_ERR_ORDER).  In this setting every forward iteration is one launch per iteration of the fused fp32 step
 * (no one-launch loop, no fp64 step for collapsing layers) and the implicit backward always iterates fused passes.
 * A temperature schedule (start warm, end cold, as the paper's closing section suggests) is a sequence of forward
 * calls in which each call's C0 is the previous call's C_out.
 * Returns IDKM_OK, IDKM_ERR_NULL or IDKM_ERR_PARAM.
 */
int idkm_set_distance(idkm_ctx* ctx, int squared);

/*
 * Hard assignment, q(w) = argmin_c ||w - c|| (Section 3.1: the map the soft quantiser r_tau of the forward tends
 * to as tau -> 0) -- the codes and dequantised weights of the trained layer.  For every row i of W [m][d] (DEVICE,
 * fp32) the index of the nearest row of C [k][d] (DEVICE, fp32; squared distances in fp32, ties to the lowest index)
 * is written to codes_out (DEVICE, idkm_codes_bytes(m, k) bytes, or NULL): b = idkm_code_bits(k) bits per weight,
 * b the smallest of 1, 2, 4, 8 with 2^b >= k, at bit offset (i b) mod 8 of byte (i b) / 8 (little-endian within the
 * byte; unused high bits of the last byte are 0).  Wq_out (DEVICE [m][d], or NULL; not W) receives the assigned
 * centroid of every row.  At least one output must be given; W and Wq_out 16-byte aligned.  d in {1,2,4},
 * 1 <= k <= 256, m >= 1; needs no
 * context and no workspace and allocates nothing; asynchronous on cuda_stream.
 * Returns IDKM_OK, IDKM_ERR_NULL, IDKM_ERR_UNSUPPORTED, IDKM_ERR_SHAPE, IDKM_ERR_PARAM, IDKM_ERR_ALIGN or
 * IDKM_ERR_CUDA.
 */
int idkm_assign(const float* W, int64_t m, int d, const float* C, int k, unsigned char* codes_out, float* Wq_out,
                void* cuda_stream);
int idkm_code_bits(int k);                   /* 1, 2, 4 or 8; 0 for k outside [1, 256] */
size_t idkm_codes_bytes(int64_t m, int k);   /* ceil(m * idkm_code_bits(k) / 8); 0 for bad arguments */

/*
 * Measured issue rates of the two pipes that bound the arithmetic-bound passes, for roofline denominators (the
 * paper has no counterpart: this is a measurement utility, nothing on the IDKM path calls it).  Two register-only
 * kernels over all SMs -- eight independent chains per thread of fp32 fused multiply-adds, and of ex2.approx --
 * are timed with CUDA events on cuda_stream (best of five after two warm-up launches, a few milliseconds in all).
 * Writes, to HOST doubles, lane-operations per second: one fused multiply-add (counted as one operation, not two
 * flops) resp. one special-function result, per lane.  The figures are at the clock the GPU ran during the
 * measurement.  Synchronises cuda_stream.  Returns IDKM_OK, IDKM_ERR_NULL or IDKM_ERR_CUDA.
 */
int idkm_measure_pipe_rates(double* fp32_lane_ops_per_s, double* sfu_lane_ops_per_s, void* cuda_stream);

/*
 * How the forward loop (Algorithm 1) is launched.  0 (default): layers with k <= 16 (k <= 8 for d = 4) run the WHOLE
 * loop in one cooperative launch -- a single layer of at most about 9.7 million rows (128 rows per thread of the
 * co-resident grid; half that at d = 4), or a batch of layers (Algorithm 2 clusters every layer of the network before
 * each minibatch: "for all layers") of at most twice that in total and no more layers than the grid has blocks;
 * either way at most 80 MB of weights (they then stay in L2 across the iterations).  The blocks are dealt out to the layers in proportion to their rows, at least one each; per
 * iteration every block publishes one fp64 partial of its layer, all blocks meet at a grid-wide barrier, and every
 * block then adds its layer's partials in the same order and takes the M-step itself, so only the partials cross L2
 * inside the loop.  A layer leaves the loop at the iteration whose stop test passes; a batch leaves at the first
 * barrier at which every layer has.  Layers that collapse on the way step in the fp32 increment form (see
 * idkm_set_collapse_step).  Everything else (larger layers, batches or codebooks, max_iter < 2, the squared
 * distance, the fp64 step for collapsing layers) takes one launch per iteration.  Every barrier wait is bounded
 * (about a second): if one runs out the kernel returns and the status of the layer (of every layer of a batch) is
 * IDKM_ERR_TIMEOUT.  1: always one launch per iteration
 * (for the smallest codebooks -- k <= 4 at d = 1, k <= 2 at d = 2 -- that launch is a kernel that steps the fp32 and
 * the collapsing layers of a batch side by side).  2: as 1, but the fp32 step and the step of the collapsing layers
 * are always two launches, one after the other.  3: as 2, and for codebooks of at most 16 centroids the fp32 step
 * receives its rows through a pipeline of bulk asynchronous copies into shared memory (one copy per trip, issued three
 * trips ahead, completion on a shared-memory barrier with a bounded wait: if a copy never arrives the kernel returns
 * and the layer's status is IDKM_ERR_TIMEOUT) instead of per-thread 128-bit loads; layers whose first row is not
 * 16-byte aligned keep the loads.  All run the same iteration; 0 differs from the others only by the order of the
 * cross-block sums, 1 and 2 give bitwise the same result, and so does 3 when as many blocks are resident with the
 * copy stages in shared memory as without (otherwise the cross-block sums are grouped differently).  Returns
 * IDKM_ERR_PARAM for other values.
 */
int idkm_set_forward_loop(idkm_ctx* ctx, int method);

/*
 * Element type of the soft-quantised weights the forward writes: 0 (default) fp32, 1 bfloat16, 2 IEEE half.  With 1
 * or 2 the Wq_out argument of idkm_forward* points to m * d two-byte elements (still 16-byte aligned, passed through the
 * float* parameter) and receives the fp32 result of Wq = A C rounded to nearest even -- the form in which the
 * quantised layer is fed to a half-precision network in the training loop of Algorithm 2.  Everything else (C, A, the
 * backward) stays fp32; idkm_quantize_host* always exchange fp32.  Returns IDKM_OK, IDKM_ERR_NULL or IDKM_ERR_PARAM.
 */
int idkm_set_wq_dtype(idkm_ctx* ctx, int dtype);

/*
 * How the forward step treats a COLLAPSING layer, i.e. one whose centroids all lie within 0.0625 tau of each other
 * (tau above the spread of the weights: every centroid slides into the mean).  There the update of C is decided by
 * attention differences far below fp32 resolution of w - c_j, so such layers leave the ordinary fp32 step.
 * 0 (default): an fp32 step in the increment form -- with u_i = w_i - c_0 and delta_j = c_j - c_0 the logit
 * differences -(D_ij - D_i0) / tau, the attention increments A_ij - 1/k and the sums of (A_ij - 1/k) and
 * (A_ij - 1/k) u_i are all small quantities evaluated to fp32 relative accuracy; the M-step is completed in fp64 from
 * those sums and sum_i u_i.  1: the same step with fp64 distances, exponentials and sums (about four times slower per
 * row; kept as the reference for the other; launches per iteration only, the one-launch loops are not taken).  Both
 * realise Algorithm 1's steps 3-5 for such layers and agree with
 * the float64 oracle within the stated tolerance.  Returns IDKM_OK, IDKM_ERR_NULL or IDKM_ERR_PARAM.
 */
int idkm_set_collapse_step(idkm_ctx* ctx, int method);

/*
 * Host-side fault injection for tests of the timeout path of the one-launch forward loop (no GPU fault is involved:
 * the waits stay bounded and the kernel returns).  missing_arrivals = n > 0 makes each grid-wide barrier of this
 * ctx's following calls wait for n arrivals that never come; spin_limit_ticks > 0 shortens the bound of every wait
 * to that many SM clock ticks.  (0, 0) restores production behaviour, which is also the state after idkm_create.
 * Returns IDKM_OK, IDKM_ERR_NULL or IDKM_ERR_PARAM (a negative argument).
 */
int idkm_set_test_hooks(idkm_ctx* ctx, int missing_arrivals, int64_t spin_limit_ticks);

/*
 * Consistency self-check: waits for the ctx's stream and counts the arrival counters of the cross-block reductions
 * in the last forward's workspace that are not at rest.  Every counter returns to zero when its reduction
 * completes, so *count_out (HOST) is 0 after any completed call; anything else means a reduction was entered by
 * some blocks and never finished.  Returns IDKM_OK, IDKM_ERR_NULL, IDKM_ERR_ORDER (no forward yet) or IDKM_ERR_CUDA.
 */
int idkm_count_busy_tickets(idkm_ctx* ctx, int* count_out);

/*
 * Which kernels the library picks for a problem shape (for benchmarks that attribute time to kernels).  Writes five
 * ints to the HOST array out: [0], [1] centroids per lane and lanes per weight-vector of the fused forward step
 * (Algorithm 1, steps 3-5); [2], [3] the same of the fused adjoint step (Section 4.2); [4] how an implicit backward
 * of adj_max_iter steps with idkm_set_adjoint_method = adjoint_method runs the iteration: 0 one fused pass per step,
 * 1 explicit k d x k d matrix held in registers (k d <= 8), 2 explicit matrix in tiles (k d <= 64, from 16 steps),
 * 3 exact solve on the explicit matrix (adjoint_method 2, k d <= 64).
 * Returns IDKM_OK, IDKM_ERR_NULL or IDKM_ERR_UNSUPPORTED.  Needs no device.
 */
int idkm_describe_path(int d, int k, int adj_max_iter, int adjoint_method, int* out);

/* Number of kernels this ctx has launched since idkm_create (for accounting in benchmarks). */
int64_t idkm_launch_count(const idkm_ctx* ctx);

/* Static, human-readable text for a status code. */
const char* idkm_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* IDKM_H */
