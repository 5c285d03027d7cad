/*
 * dad.h -- C ABI of libdad: the per-layer hot path of distributed auto-differentiation
 * (dAD) and its rank-reduced form (rank-dAD), as hand-written CUDA for sm_100a.
 *
 * For one linear layer, every site s of S holds its input activations A_s (N x h_in) and
 * the back-propagated errors D_s (N x h_out, the paper's Delta_i).  The site gradient is
 * the product A_s^T D_s (Eq. "local_grad", Sec. 3.1).  dAD ships A_s and D_s and multiplies
 * the concatenated batch (Sec. 3.2); rank-dAD first reduces them to rank-r factors with
 * structured power iterations on the implicit product (Algorithm 2, Sec. 3.3.1), stacks the
 * factors of all sites and reconstructs the gradient from the stacks (Algorithm 1).
 * Sites are slices of one device buffer; nothing here communicates between GPUs.
 *
 * Conventions
 *   - Every matrix is dense row-major.  "DEVICE" pointers are CUDA device memory of the
 *     current device, owned by the caller, who keeps them alive until the work queued on
 *     `cuda_stream` has finished.  "HOST" pointers are ordinary host memory, read or written
 *     before the call returns.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls
 *     only enqueue work; none of them synchronises, allocates device memory or keeps state
 *     between calls (exceptions are stated at the entry point).
 *   - Inputs are never written.  Outputs are overwritten, never accumulated into.
 *   - Every call returns a dad_status.  Errors the host can see (NULL pointers, bad shapes,
 *     ranks, strides, alignment, a workspace that is too small) are returned before anything
 *     is launched.  On error the outputs are unspecified but no write leaves the buffers.
 *   - There is no CPU fallback: without a CUDA device every compute call fails with
 *     DAD_ERR_CUDA.
 */
#ifndef DAD_H_
#define DAD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DAD_OK = 0,
  DAD_ERR_NULL = 1,      /* a required pointer is NULL                                        */
  DAD_ERR_SHAPE = 2,     /* S, N, h_in, h_out, K, iters or a stride is out of range           */
  DAD_ERR_DTYPE = 3,     /* dtype is neither DAD_F32 nor DAD_BF16                             */
  DAD_ERR_RANK = 4,      /* r < 1, r > DAD_MAX_RANK or r > min(h_in, h_out)                   */
  DAD_ERR_WORKSPACE = 5, /* ws is smaller than dad_workspace_bytes() says                     */
  DAD_ERR_ALIGN = 6,     /* a pointer or stride misses the alignment stated below             */
  DAD_ERR_CUDA = 7,      /* the CUDA runtime reported an error (no device, bad launch, ...)   */
  DAD_ERR_TIMEOUT = 8,   /* a bounded device-side wait ran out (reported by dad_check)        */
  DAD_ERR_NUMERIC = 9    /* a NaN/Inf reached the orthonormalisation (reported by dad_check)  */
} dad_status;

typedef enum {
  DAD_F32 = 0,
  DAD_BF16 = 1,
  DAD_BF16_1TERM = 2 /* only as the `math` of a reconstruction: one bf16 product instead of three (see dad_reconstruct) */
} dad_dtype;

#define DAD_MAX_RANK 64

/*
 * One linear layer seen from all S sites.
 *   A: element (s, n, a) at A[s*strideA + n*ldA + a],  0<=n<N, 0<=a<h_in
 *   D: element (s, n, b) at D[s*strideD + n*ldD + b],  0<=b<h_out
 * Strides are in ELEMENTS of `dtype`.  ldA >= h_in, ldD >= h_out; strideA >= N*ldA (when S>1),
 * likewise strideD.  A and D base pointers must be aligned to 16 bytes; for DAD_BF16 the
 * tensor-core kernels are used when, in addition, h_in, h_out, ldA, ldD, strideA and strideD
 * are multiples of 8 elements (16 bytes) -- any other layout takes the slower general kernels,
 * with the same results.  Factors, gradients and start blocks are always fp32, contiguous.
 */
typedef struct {
  int32_t S;            /* number of sites (>= 1)                         */
  int64_t N;            /* rows per site (batch x tokens), >= 1            */
  int64_t h_in, h_out;  /* layer width in / out, >= 1                      */
  dad_dtype dtype;      /* storage type of A and D                        */
  int64_t ldA, ldD;     /* row strides in elements                        */
  int64_t strideA, strideD; /* site strides in elements                   */
} dad_layer;

/*
 * Bytes a site transmits for this layer (host arithmetic, exact, no device work):
 *   dad_bytes_dad : N*(h_in+h_out)*e, both component matrices at their storage width e
 *                   (Sec. 3.1, "m+n against m*n"; Sec. 3.2)
 *   dad_bytes_rank: r*(h_in+h_out)*4, the two rank-r fp32 factors (Sec. 2, the
 *                   Theta(r(h_i+h_{i+1})) bandwidth of rank methods; Sec. 3.3)
 *   dad_bytes_dsgd: h_in*h_out*4, the full fp32 gradient that dSGD ships (Sec. 1)
 * A NULL or invalid layer gives 0.
 */
uint64_t dad_bytes_dad(const dad_layer* layer);
uint64_t dad_bytes_rank(const dad_layer* layer, int r);
uint64_t dad_bytes_dsgd(const dad_layer* layer);

/*
 * Scratch bytes dad_rank_compress / dad_full_grad need for this layer (the larger of the two;
 * 0 if the arguments are invalid).  The caller allocates at least this much DEVICE memory,
 * aligned to 256 bytes, and may reuse it for any later call with the same or smaller needs.
 * Two calls that overlap in time on the GPU must not share a workspace.  The first 256 bytes
 * hold the status words dad_check() reads: they must be zero when the workspace is first handed
 * to the library (one cudaMemset); afterwards the library maintains them.
 */
size_t dad_workspace_bytes(const dad_layer* layer, int r, int iters);

/*
 * Uncompressed dAD gradient (Sec. 3.2; Eq. "local_grad"; Sec. 5.1): the product of the
 * batch-concatenated component matrices,
 *     grad[a][b] = sum_s sum_n A_s[n][a] * D_s[n][b],
 * which equals the gradient of the pooled batch exactly (up to rounding order).
 *   A, D     DEVICE, as laid out by `layer`
 *   grad     DEVICE, h_in x h_out fp32, contiguous, 16-byte aligned
 *   bytes_tx HOST, S entries, or NULL: entry s receives dad_bytes_dad(layer)
 *   ws       DEVICE scratch of ws_bytes >= dad_workspace_bytes(layer, 1, 0)
 * DAD_F32 inputs are multiplied in fp32 (FMA); DAD_BF16 inputs on the tensor cores with fp32
 * accumulation.
 */
dad_status dad_full_grad(const dad_layer* layer, const void* A, const void* D, float* grad,
                         uint64_t* bytes_tx, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The same gradient (Sec. 3.2; Eq. "local_grad") for `groups` layers of one shape in one call: `layer` describes
 * groups * S' slices, layer g owning slices g*S' .. g*S'+S'-1 (S' = layer->S / groups, which must divide), and
 *     grads[g][a][b] = sum over the slices s of layer g and the rows n of  A_s[n][a] * D_s[n][b].
 * One launch then serves all of them where a single layer's output tiles would leave part of the GPU idle (a
 * 1024 x 1024 gradient is 16 tiles of 256 x 256 for 148 SMs).  Arguments as dad_full_grad, with
 *   grads    DEVICE, groups x h_in x h_out fp32, contiguous, 16-byte aligned
 *   bytes_tx HOST, layer->S entries, or NULL
 *   ws       DEVICE scratch of ws_bytes >= dad_full_grad_grouped_workspace_bytes(layer, groups)
 * Shapes the large-tile tensor-core kernel does not take are computed one layer after the other.
 * DAD_ERR_SHAPE if groups < 1 or does not divide layer->S.
 */
size_t dad_full_grad_grouped_workspace_bytes(const dad_layer* layer, int groups);
dad_status dad_full_grad_grouped(const dad_layer* layer, int groups, const void* A, const void* D, float* grads,
                                 uint64_t* bytes_tx, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Structured power iterations, all r vectors of a site advanced together (Algorithm 2;
 * Eq. "nabla_iter" evaluated through A and D as in Eq. "reduced_iter", never forming the
 * h_in x h_out gradient; the peel term of Eq. "peel" realised as orthonormalisation of the
 * r vectors).  Independently for every site s:
 *     G <- Q0_s
 *     repeat iters times:  G <- orth( D_s^T ( A_s ( A_s^T ( D_s G^T ))) )     (rows of G)
 *     Q_s = G,  P_s = ( A_s^T ( D_s G^T ) )^T,  sigma_s[j] = || P_s[j] ||
 * so that P_s^T Q_s is the projection of A_s^T D_s on the span of the r directions found.
 * orth = thin QR with positive diagonal; a vector whose remainder after projection is below
 * 1e-12 (DAD_F32) or 1e-6 (DAD_BF16) of its length is set to exactly zero.
 *   r        1 <= r <= min(h_in, h_out, DAD_MAX_RANK);  iters >= 0
 *   Q0       DEVICE, S x r x h_out fp32: the start vectors g_0 ~ N(0,1), supplied by the caller
 *   P        DEVICE, S x r x h_in  fp32 (out)
 *   Q        DEVICE, S x r x h_out fp32 (out; may alias Q0)
 *   sigma    DEVICE, S x r fp32 (out) or NULL
 *   ws       DEVICE scratch of ws_bytes >= dad_workspace_bytes(layer, r, iters)
 * DAD_F32: all products accumulate in fp64 and intermediates are kept in fp64.
 * DAD_BF16: fp32 accumulation; the fp32 factor operand of each product enters as a
 * two-term bf16 split, so products carry about 16 significant bits of the factor.
 */
dad_status dad_rank_compress(const dad_layer* layer, const void* A, const void* D, int r, int iters,
                             const float* Q0, float* P, float* Q, float* sigma,
                             void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Which of the library's pipelines dad_rank_compress takes for this shape (informational; the paper has no
 * counterpart).  All of them compute the iteration stated above to the same precision contract:
 *   DAD_PATH_GENERAL  any shape: one launch per product and per Cholesky-QR phase (5 * iters + 3 or more launches)
 *   DAD_PATH_TENSOR   bf16 inputs in 16-byte-aligned layouts: the same sequence on tcgen05 tensor cores
 *   DAD_PATH_TENSOR_PAIRED  the tensor-core sequence for calls of few row blocks with each half of the operator of
 *                     Eq. "reduced_iter" (Y = D g then Z = Y^T A; W = A Z^T then W^T D) as one launch in which Y / W
 *                     never leaves the SM (2 * iters + 1 product launches instead of 4 * iters + 2); an option,
 *                     taken only after dad_pair_enable(1)
 *   DAD_PATH_FUSED    small sites: ONE launch, a thread-block cluster of *cluster_size CTAs per site runs every
 *                     application of the operator, the orthonormalisations and the final factor, with Y and W
 *                     in shared memory and Z, G~ and the orthonormal vectors exchanged over distributed shared
 *                     memory (the site's factor buffers fit in the cluster's shared memory).
 *   DAD_PATH_FUSED_L2 the same one launch for sites whose factor buffers do not fit: the CTAs exchange partial
 *                     sums and factors through the workspace (L2) instead.
 * Returns -1 for invalid arguments; cluster_size may be NULL.  dad_fused_enable(0) makes the library skip the
 * one-launch form (process-wide; for timing one pipeline against the other), dad_fused_enable(1) restores it.
 * The workspace size does not depend on that switch.  dad_pair_enable(1 / 0) switches the paired launches of the
 * tensor-core sequence on and off (process-wide; off by default: on B200 they measured no faster than the two
 * streaming kernels they replace); the workspace size does not depend on it either.
 */
#define DAD_PATH_GENERAL 0
#define DAD_PATH_TENSOR 1
#define DAD_PATH_FUSED 2
#define DAD_PATH_FUSED_L2 3
#define DAD_PATH_TENSOR_PAIRED 4
int dad_compress_path(const dad_layer* layer, int r, int iters, int* cluster_size);
void dad_fused_enable(int on);
void dad_pair_enable(int on);

/*
 * The same compression in the form Algorithm 2 prints it, for the regime the paper assumes (batch much smaller
 * than the layer width, N << h; Sec. 3.3.1): C = A A^T (N x N) is precomputed once per site, every application
 * of the operator then touches only D and C,  g <- D^T ( C ( D g ) )  (Eq. "reduced_iter" with B = D^T C), and
 * sigma = sqrt(v^T C v) with v = D g.  A is read twice in all instead of 2*iters + 1 times.  Arguments, results
 * and errors as dad_rank_compress, with two restrictions: dtype must be DAD_F32 (else DAD_ERR_DTYPE) and
 * N <= DAD_MAX_GRAM_ROWS (else DAD_ERR_SHAPE).  Products accumulate in fp64.
 *   ws >= dad_rank_compress_gram_workspace_bytes(layer, r, iters)
 */
#define DAD_MAX_GRAM_ROWS 128
size_t dad_rank_compress_gram_workspace_bytes(const dad_layer* layer, int r, int iters);
dad_status dad_rank_compress_gram(const dad_layer* layer, const void* A, const void* D, int r, int iters,
                                  const float* Q0, float* P, float* Q, float* sigma,
                                  void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The same compression with the components found one after the other, the order in which Algorithm 2 is printed
 * (Sec. 3.3.1): for j = 0 .. r-1, g <- Q0[j] made orthogonal to the components found so far and normalised;
 * iters times  g <- M g - sum_{l<j} sigma_l^2 g_l (g_l . g)  (M = gradW^T gradW applied through D and A, Eq.
 * "reduced_iter"; the subtraction is Eq. "peel"), orthogonalised against the found components again and
 * normalised; then Q[j] = g, P[j] = A^T (D g), sigma_j = ||P[j]||.  A component whose remainder falls to 1e-12 of
 * its length before the projection is set to zero.  It spans the same subspace as dad_rank_compress once both
 * have converged, and costs r times the passes over A and D: provided to compare the two orders, not for speed.
 * Arguments, layouts and errors as dad_rank_compress; both dtypes; products accumulate in fp64.
 *   ws >= dad_rank_compress_sequential_workspace_bytes(layer, r, iters)
 */
size_t dad_rank_compress_sequential_workspace_bytes(const dad_layer* layer, int r, int iters);
dad_status dad_rank_compress_sequential(const dad_layer* layer, const void* A, const void* D, int r, int iters,
                                        const float* Q0, float* P, float* Q, float* sigma,
                                        void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Gather at the aggregator (Algorithm 1, the two vertcat lines): site s's factors become rows
 * s*r .. s*r+r-1 of the stacks, and each site is charged what it sent.
 *   P, Q       DEVICE, S x r x h_in and S x r x h_out fp32 (as written by dad_rank_compress)
 *   Pcat, Qcat DEVICE, (S*r) x h_in and (S*r) x h_out fp32 (out).  Pcat == P and Qcat == Q are
 *              allowed: the stacks then are the factor buffers themselves and nothing is copied.
 *   bytes_tx   HOST, S entries, or NULL: entry s receives dad_bytes_rank(layer, r)
 * Only S, h_in and h_out of `layer` are read.
 */
dad_status dad_gather_factors(const dad_layer* layer, int r, const float* P, const float* Q,
                              float* Pcat, float* Qcat, uint64_t* bytes_tx, void* cuda_stream);

/*
 * Reconstruction (Algorithm 1, the P^T Q step): the sum over the K = S*r stacked rows of the
 * outer products of the factors,
 *     grad[a][b] = sum_k Pcat[k][a] * Qcat[k][b].
 *   Pcat, Qcat DEVICE, K x h_in and K x h_out fp32, contiguous, 16-byte aligned
 *   grad       DEVICE, h_in x h_out fp32 (out)
 *   math       DAD_F32: fp32 FMA.  DAD_BF16: tensor cores with fp32 accumulation; each fp32
 *              factor enters as a two-term bf16 split x = hi + lo and the product is
 *              hi*hi + hi*lo + lo*hi (one contraction of length 3K), so the result carries about
 *              16 significant bits of the factors (the dropped lo*lo term is 2^-16 relative).
 *              DAD_BF16_1TERM: the hi terms only, one contraction of length K -- a third of the
 *              operand traffic and tensor-core work, about 8 significant bits of each factor
 *              (measured 2e-3 to 4e-3 relative on the gradient, inside the 2e-2 bar of bf16 inputs).
 *              Both need h_in and h_out multiples of 8; otherwise they fall back to the
 *              fp32 FMA kernel (still on the device).
 *   ws         DEVICE scratch of ws_bytes >= dad_reconstruct_workspace_bytes(h_in, h_out, K, math),
 *              may be NULL when that is 0
 */
size_t dad_reconstruct_workspace_bytes(int64_t h_in, int64_t h_out, int64_t K, dad_dtype math);
dad_status dad_reconstruct(int64_t h_in, int64_t h_out, int64_t K, const float* Pcat, const float* Qcat,
                           float* grad, dad_dtype math, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The same reconstruction (Algorithm 1, the P^T Q step) for `batch` layers of one shape in one go:
 * entry b owns rows b*K .. b*K+K-1 of the stacks and the b-th h_in x h_out gradient,
 *     grad[b][a][c] = sum_k Pcat[b*K + k][a] * Qcat[b*K + k][c].
 * The entries are independent; batching only saves launches (a single reconstruction is a few
 * microseconds of work).  Arguments, precision and errors as for dad_reconstruct; batch in 1 .. 65535;
 * ws_bytes >= dad_reconstruct_batched_workspace_bytes(h_in, h_out, K, batch, math).  batch = 1 is
 * dad_reconstruct itself, bit for bit.
 */
size_t dad_reconstruct_batched_workspace_bytes(int64_t h_in, int64_t h_out, int64_t K, int batch, dad_dtype math);
dad_status dad_reconstruct_batched(int64_t h_in, int64_t h_out, int64_t K, int batch, const float* Pcat,
                                   const float* Qcat, float* grad, dad_dtype math, void* ws, size_t ws_bytes,
                                   void* cuda_stream);

/*
 * The whole per-layer path from HOST memory (Algorithm 1 with the direct sum of outer products at the
 * aggregator): copies A, D (laid out by `layer`, but in host memory) and Q0 to the device, runs
 * dad_rank_compress -> dad_gather_factors -> dad_reconstruct there, and copies the h_in x h_out fp32 gradient
 * back.  Everything is queued on `cuda_stream`; the call does not synchronise and allocates nothing.
 *   A_host, D_host, Q0_host  HOST (pinned memory for asynchronous copies); strided rows / sites are allowed
 *   grad_host                HOST, h_in x h_out fp32 (out), valid once the stream has drained
 *   bytes_tx                 HOST, S entries or NULL: dad_bytes_rank(layer, r) per site
 *   math                     as for dad_reconstruct
 *   dev_scratch              DEVICE, 256-byte aligned, >= dad_rank_dad_host_scratch_bytes(layer, r, iters, math):
 *                            staging for the inputs, the factors, the gradient, and the workspace
 * Results, precision and errors are those of the three device calls on densely packed copies of the inputs.
 */
size_t dad_rank_dad_host_scratch_bytes(const dad_layer* layer, int r, int iters, dad_dtype math);
dad_status dad_rank_dad_host(const dad_layer* layer, const void* A_host, const void* D_host, const float* Q0_host,
                             int r, int iters, dad_dtype math, float* grad_host, uint64_t* bytes_tx,
                             void* dev_scratch, size_t dev_scratch_bytes, void* cuda_stream);

/*
 * Second structured power iteration, at the aggregator (Algorithm 1: after the vertcat, "SPI(Q_i, G_i)" reduces
 * the stacks of all sites to r rows again, and those r rows are what is broadcast back; Sec. 3.3).  The stacks
 * take the places of the component matrices -- Pcat^T Qcat is "A^T D" with A = Pcat (K x h_in) and D = Qcat
 * (K x h_out) -- so this is dad_rank_compress on one slice of K = S*r fp32 rows, with the same arguments, results,
 * precision (fp64 accumulation) and errors:
 *     Qhat (r x h_out, orthonormal rows), Phat = (Pcat^T (Qcat Qhat^T))^T (r x h_in), sigma (r, or NULL),
 * and Phat^T Qhat is the projection of Pcat^T Qcat on the r directions found.  A site then receives
 * r*(h_in+h_out)*4 bytes (dad_bytes_rank) instead of K*(h_in+h_out)*4.
 *   Q0  DEVICE, r x h_out fp32 start vectors;  ws >= dad_aggregate_workspace_bytes(h_in, h_out, K, r, iters)
 */
size_t dad_aggregate_workspace_bytes(int64_t h_in, int64_t h_out, int64_t K, int r, int iters);
dad_status dad_aggregate_compress(int64_t h_in, int64_t h_out, int64_t K, const float* Pcat, const float* Qcat,
                                  int r, int iters, const float* Q0, float* Phat, float* Qhat, float* sigma,
                                  void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Effective rank (Sec. 3.3.1, last paragraph, and the early stop of Algorithm 2 with theta = 1e-3: components
 * that carry only noise are not computed or sent, so r is an upper limit on what a site transmits).  The paper's
 * stop test compares consecutive, mutually orthogonal vectors and cannot trigger as printed; the reading taken
 * here keeps the leading components of a site while their strength stays above theta times the first one's:
 *     r_eff[s] = min { j : sigma_s[j] <= theta * sigma_s[0] }   (r if there is no such j; 0 if sigma_s[0] == 0),
 * the comparison made in fp32 on the fp32 sigma that dad_rank_compress wrote.  Rows j >= r_eff[s] of P_s and Q_s
 * are set to zero (pass NULL to leave the factors alone), so gather and reconstruct work unchanged and the
 * dropped components add nothing; the site then transmits dad_bytes_rank(layer, r_eff[s]) bytes.
 *   sigma DEVICE S x r fp32;  r_eff DEVICE S x int32 (out);  P, Q DEVICE S x r x h_in / h_out fp32 or NULL
 *   theta in [0, 1].  Only S, h_in, h_out of `layer` are read.
 */
dad_status dad_effective_rank(const dad_layer* layer, int r, float theta, const float* sigma, int32_t* r_eff,
                              float* P, float* Q, void* cuda_stream);

/*
 * Reconstruction without caller scratch (the paper has no counterpart: this is a packaging of
 * dad_reconstruct for hosts that cannot allocate).  Same arguments, results and errors as
 * dad_reconstruct, minus `ws`: the scratch is a fixed array of DAD_STATIC_SCRATCH_BYTES inside the
 * library's device image, present on every GPU that loads the library for the life of the process.
 * It is meant for callers that must not (or cannot) obtain device memory themselves -- a plug-in
 * living inside another program's memory pool, a step running under a fixed device-memory budget,
 * code that cannot afford the device-wide synchronisation an allocation implies.  The call makes no
 * cudaMalloc/cudaFree and calls no allocating library routine.
 *   - Problems whose scratch need (dad_reconstruct_workspace_bytes) exceeds
 *     DAD_STATIC_SCRATCH_BYTES are refused with DAD_ERR_WORKSPACE; nothing is launched.
 *   - The first call on each device resolves the array's device address.  That is also the moment
 *     the CUDA runtime loads the module holding the array, i.e. when its DAD_STATIC_SCRATCH_BYTES
 *     are taken from that device (with the device-wide synchronisation a module load implies, and
 *     DAD_ERR_CUDA if the device has no room left); only the calls after it leave the device's
 *     memory untouched.  Make that first call early, and outside any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the
 *     library clears what has to start at zero.  Two calls that overlap in time on the same GPU
 *     (different streams, different host threads) race on it: serialise them, or use dad_reconstruct
 *     with separate workspaces.  Device-side status is not reported for this entry point.
 */
#define DAD_STATIC_SCRATCH_BYTES (32u << 20)
dad_status dad_reconstruct_static(int64_t h_in, int64_t h_out, int64_t K, const float* Pcat, const float* Qcat,
                                  float* grad, dad_dtype math, void* cuda_stream);

/*
 * Device-side status of the work that used `ws`: synchronises `cuda_stream`, reads the status
 * words at the head of the workspace -- one written by the last dad_rank_compress on it, one by
 * the last dad_full_grad / dad_reconstruct on it -- and returns the first that is not DAD_OK
 * (DAD_ERR_TIMEOUT, DAD_ERR_NUMERIC), or DAD_ERR_CUDA if the stream reports an error.  Each of
 * those calls clears its own word when it starts.  This is the only call that synchronises.
 */
dad_status dad_check(const void* ws, void* cuda_stream);

/*
 * Self-test of the bounded device-side waits (the paper has no counterpart).  Every wait of the tensor-core kernels
 * on a copy or on the tensor cores gives up after a fixed number of polls; the CTA then stops issuing work, waits --
 * again bounded -- for the copies and multiplications it has already issued, frees its tensor memory, records
 * DAD_ERR_TIMEOUT in the workspace's status word and RETURNS.  This call makes that happen on purpose, harmlessly:
 * it launches one small tile whose multiplying role is told to expect one block more than is ever loaded, with a
 * limit of 1024 polls, on zeroed operands inside `ws`.  Nothing hangs and nothing faults; afterwards
 * dad_check(ws) reports DAD_ERR_TIMEOUT, and the context and `ws` remain usable for ordinary calls (each clears the
 * status word when it starts).
 *   ws  DEVICE, 256-byte aligned, ws_bytes >= DAD_SELFTEST_BYTES; its contents are overwritten
 */
#define DAD_SELFTEST_BYTES (64u << 10)
dad_status dad_selftest_bounded_wait(void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Bounds-check build (the paper has no counterpart).  Compiled with -DDAD_BOUNDS_CHECK the library is its own memory
 * checker for the kernels that compute their indices themselves (the general products, the one-launch compress, the
 * fp32 dense product and the small element-wise kernels; the tensor-core kernels address memory through tensor maps,
 * which the hardware clips): dad_rank_compress, dad_full_grad, dad_gather_factors and dad_reconstruct register the
 * address ranges of the buffers they were handed, every access of those kernels is tested against them, and an access
 * outside all of them is NOT made (a load gives zero, a store is dropped) but counted -- nothing traps or faults.
 *   dad_bounds_check_build  1 in such a build, 0 in the ordinary one (where the checks compile to nothing)
 *   dad_bounds_report       synchronises `cuda_stream`, then out[0] = violations so far, out[1..3] = address, size in
 *                           bytes and source line of the first; reset != 0 clears the record.  HOST out.  In the
 *                           ordinary build it reports zeros.
 */
int dad_bounds_check_build(void);
dad_status dad_bounds_report(uint64_t out[4], int reset, void* cuda_stream);

/* Kernels launched by this library in this process so far (all threads); for accounting. */
uint64_t dad_launch_count(void);

const char* dad_status_string(dad_status status);

/*
 * Instrumentation for benchmarks (the paper has no counterpart).  While enabled, every kernel this
 * library launches is bracketed by CUDA events on its own stream, which costs a little time per
 * launch; dad_timing_collect() waits for the recorded events (it synchronises) and adds the elapsed
 * time of each launch to the total of its kernel family, returning the number of families seen.
 * dad_timing_name/ms/launches read family i; dad_timing_reset() clears the totals.
 */
void dad_timing_enable(int on);
int dad_timing_collect(void);
void dad_timing_reset(void);
const char* dad_timing_name(int i);
double dad_timing_ms(int i);
uint64_t dad_timing_launches(int i);

#ifdef __cplusplus
}
#endif
#endif /* DAD_H_ */
