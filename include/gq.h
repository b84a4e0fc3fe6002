/*
 * libgq -- construction of GuidedQuant's end-loss-guided layer objective on one B200 (sm_100a).
 *
 * For one linear layer with input activations X (n tokens x d_in), end-loss gradients of the
 * layer output dl/dZ (n x d_out) and weights W, the library computes
 *
 *   J_k   = { m k, ..., m (k+1) - 1 },  m = d_out / g          (Algorithm 1, grouping step)
 *   s_k   = 1/|J_k| * sum_{j in J_k} (dl/dz_j)^2                (Algorithm 1, saliency step)
 *   H_k   = X^T Diag(s_k) X                                     (Algorithm 1, Hessian step; Section 3.2)
 *   loss  = sum_k sum_{j in J_k} (w_j - what_j)^T H_k (w_j - what_j)          (Eq. 7)
 *
 * Conventions shared by every call
 *   - Plain C ABI.  Unless a parameter is documented as HOST memory, every pointer is a DEVICE
 *     pointer owned by the caller; the library never allocates or frees device memory and never
 *     keeps a pointer after the call returns.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls only
 *     enqueue work; they do not synchronise the host.  Results are in device memory and are
 *     ordered after the call on `stream`.
 *   - Return value: GQ_OK or a negative gq_status.  Invalid arguments are detected on the host
 *     before anything is launched; nothing is written in that case.
 *   - Buffers a call writes (outputs, in/out arguments, workspaces) must not share memory with a buffer
 *     the same call reads, nor with each other: overlapping ranges return GQ_ERR_INVALID_ARG.  Two
 *     read-only arguments may be the same buffer.
 *   - Problems that can only be seen on the device (a pipeline wait that ran out of its time
 *     budget) are recorded in a per-device status word that gq_check() reads.
 *   - Tokens are rows: X is [n, ld_x] and dl/dZ is [n, ld_grad], both bf16, row-major.
 *     Weights are [d_out, d_in] row-major fp32, i.e. row j is the paper's column w_j (Section 2).
 */
#ifndef GQ_H_
#define GQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum gq_status {
    GQ_OK = 0,
    GQ_ERR_INVALID_ARG = -1,       /* null pointer, negative size, g < 1, d_out % g != 0, bad flags, aliasing */
    GQ_ERR_ALIGNMENT = -2,         /* pointer or leading dimension not aligned as documented          */
    GQ_ERR_UNSUPPORTED_SHAPE = -3, /* size outside what the kernels index (see each call)             */
    GQ_ERR_WORKSPACE = -4,         /* workspace missing or smaller than the *_workspace_bytes() value */
    GQ_ERR_CUDA = -5,              /* a CUDA runtime/driver call failed: see gq_last_cuda_error()     */
    GQ_ERR_TIMEOUT = -6            /* a device-side wait gave up (reported by gq_check)               */
} gq_status;

/* Library version, major * 10000 + minor * 100 + patch. */
int gq_version(void);

/* Static, human readable name of a status code (never NULL). */
const char *gq_status_string(int32_t status);

/* The cudaError_t value of the most recent failing CUDA call made by this library on the
 * calling thread (0 if none). */
int32_t gq_last_cuda_error(void);

/*
 * Saliency: Algorithm 1, saliency step, with the gradient scaling of Section 3.2 applied to the gradient
 * before it is squared:
 *     s[k * ld_s + i] = (grad_scale^2 / m) * sum_{j = m k}^{m (k+1) - 1} grad[i * ld_grad + j]^2
 *
 *   grad        bf16 [n, ld_grad], 16-byte aligned, ld_grad >= d_out, ld_grad % 8 == 0
 *   n           tokens in this call, >= 0 (0 is a no-op: sizes are still validated, pointers are not), n * g < 2^31
 *   d_out, g    d_out % g == 0 and (d_out / g) % 8 == 0, 1 <= g <= 1024
 *   grad_scale  finite; the paper uses 1e3, tests use 1
 *   s           fp32 [g, ld_s] (group-major so that each s_k is contiguous), ld_s >= n
 * Squares and sums are fp32.  The result does not depend on the launch shape.
 */
int32_t gq_saliency(const void *grad, int64_t n, int64_t d_out, int64_t ld_grad, int32_t g,
                    float grad_scale, float *s, int64_t ld_s, void *stream);

/*
 * gq_saliency that also leaves s in the packed form the guided-Hessian kernel consumes (Algorithm 1, saliency
 * step; same values, same fp32 s): `hessian_workspace` is the workspace that the NEXT gq_hessian_accumulate call
 * for the same n tokens and the same g will be given, at least gq_hessian_workspace_bytes(n, d_in, g, flags)
 * bytes (the size does not depend on d_in), 1024-byte aligned.  That call is then made with the flag
 * GQ_HESSIAN_S_PREPARED and skips its own preparation kernel: two launches per token chunk instead of three.
 */
int32_t gq_saliency_prepared(const void *grad, int64_t n, int64_t d_out, int64_t ld_grad, int32_t g,
                             float grad_scale, float *s, int64_t ld_s, void *hessian_workspace,
                             size_t workspace_bytes, void *stream);

/*
 * Saliency at the source (Algorithm 1, saliency step; Section 3.2: of the end-loss gradients only the averaged
 * squares are kept, O(n g) numbers per layer): the same reduction for dl/dZ in the dtype and layout a backward
 * pass hands it over, written straight into the caller's calibration-wide s, so that a backward hook keeps nothing
 * but s.
 *
 *   grad        [batch, seq, d_out] with element strides (stride_b, stride_t, 1); token i = b * seq + t.
 *               16-byte aligned; stride_t >= d_out; both strides multiples of 16 bytes (8 elements for the 16-bit
 *               types, 4 for fp32); sequences must not overlap
 *   dtype       GQ_DTYPE_BF16, GQ_DTYPE_FP16 (IEEE half) or GQ_DTYPE_FP32
 *   s           fp32 [g, ld_s], ld_s >= batch * seq; s[k * ld_s + i] is written (pass s + offset of the first token
 *               and the leading dimension of the whole buffer to fill a slice of a larger array)
 * Other rules as for gq_saliency: d_out % g == 0, (d_out / g) % 8 == 0, batch * seq * g < 2^31, grad_scale finite.
 * Values are widened to fp32 exactly; squares and sums are fp32.
 * (There is no accumulating form: squares of partial gradients do not add up to the square of their sum, so
 * the gradient of a token has to be complete when it is reduced.)
 */
enum gq_dtype { GQ_DTYPE_BF16 = 0, GQ_DTYPE_FP16 = 1, GQ_DTYPE_FP32 = 2 };
int32_t gq_saliency_strided(const void *grad, int32_t dtype, int64_t batch, int64_t seq, int64_t d_out,
                            int64_t stride_b, int64_t stride_t, int32_t g, float grad_scale, float *s,
                            int64_t ld_s, void *stream);

/*
 * Guided Hessian, one token chunk: Algorithm 1, Hessian step, streamed,
 *     H[k][a][b] += sum_{i < n} s[k * ld_s + i] * X[i * ld_x + a] * X[i * ld_x + b]
 * for every group k and every a <= b (the upper triangle including the diagonal).  No 1/n factor.
 *
 *   X          bf16 [n, ld_x], 16-byte aligned, ld_x >= d_in, ld_x % 8 == 0
 *   n          tokens in this chunk, >= 0 (0 is a no-op: sizes are still validated, pointers are not)
 *   d_in       d_in % 8 == 0, 8 <= d_in <= 65536
 *   s          fp32 [g, ld_s], s >= 0 (as produced by gq_saliency), ld_s >= n
 *   H          fp32 [g, d_in, d_in] row-major, 128-byte aligned.  The caller zeroes it before the
 *              first chunk and keeps it resident between chunks.  After any number of calls only
 *              entries with a <= b are defined; entries below the diagonal hold unspecified finite
 *              values until gq_hessian_finalize() is called.
 *   flags      0, or GQ_HESSIAN_DETERMINISTIC and / or GQ_HESSIAN_S_PREPARED (see below)
 *   workspace  device scratch of at least gq_hessian_workspace_bytes(n_max, d_in, g, flags) bytes with
 *              n_max >= n, 1024-byte aligned (8 bytes per token and pair of groups: s in the form the
 *              kernel consumes); contents need not be preserved between calls.
 * Arithmetic: the kernel never writes a scaled copy of X to global memory.  A small first kernel rewrites
 * s_k[i] as the sum of two bf16 terms (16 significant bits).  While X is staged for the tensor cores
 * every element is multiplied by that pair with packed bf16 fused multiply-adds and rounded to bf16 once; the products
 * (s_k[i] X[i][a]) * X[i][b] are accumulated in fp32 in tensor memory (two groups per pass over X), and
 * each call adds its fp32 tile sums to H with reduce-add transactions, so H is never read by the SMs.
 * Work is dealt to the SM pairs in whole 256 x 256 tiles of two groups; with flags == 0 the last,
 * incomplete round of tiles is cut along the token axis so that every SM pair gets the same amount of
 * work, and the pieces of such a tile reach H in no fixed order: those entries can differ in the last
 * bit from run to run.  With GQ_HESSIAN_DETERMINISTIC every element of H receives exactly one add per
 * call and results are bit-reproducible run to run, at the price of an idle tail in the last round.
 */
#define GQ_HESSIAN_DETERMINISTIC 1u
/* The workspace already holds s in packed form: it was filled by gq_saliency_prepared for exactly these n tokens
 * and this g, and nothing has written to it since.  (s itself is still validated but not read.) */
#define GQ_HESSIAN_S_PREPARED 2u
int32_t gq_hessian_accumulate(const void *X, int64_t n, int64_t d_in, int64_t ld_x, const float *s,
                              int64_t ld_s, int32_t g, float *H, uint32_t flags, void *workspace,
                              size_t workspace_bytes, void *stream);

/*
 * gq_hessian_accumulate for this chunk and, in the same launch, gq_saliency_prepared for the NEXT chunk
 * (Algorithm 1: the saliency step of a chunk uses nothing that the Hessian step of another chunk writes, so the
 * two are independent).  The Hessian kernel is bound by the tensor cores and leaves two warps per CTA without
 * work; those warps stream the next chunk's gradients meanwhile, so the saliency step costs no time of its own
 * as long as it ends before the Hessian step does (the launch lasts as long as the longer of the two).
 *
 *   X, n, d_in, ld_x, s, ld_s, g, H, flags, workspace, workspace_bytes
 *               exactly as for gq_hessian_accumulate (this chunk)
 *   next_grad, next_n, d_out, ld_grad, grad_scale, next_s, next_ld_s, next_workspace, next_workspace_bytes
 *               exactly as grad, n, d_out, ld_grad, grad_scale, s, ld_s, hessian_workspace, workspace_bytes of
 *               gq_saliency_prepared (the next chunk; same g).  next_workspace is a second scratch block:
 *               neither it nor next_s may share memory with X, s, H or workspace, and next_grad must not share
 *               memory with H or workspace.  (s and next_s may be two disjoint column ranges of one [g, ld]
 *               buffer that holds the saliency of all chunks: with equal leading dimensions the check is exact.)  The next call passes next_workspace as its workspace together
 *               with GQ_HESSIAN_S_PREPARED.
 * next_s and next_workspace receive the same bits as a gq_saliency_prepared call would write.
 * The spare warps of a full launch stream about 1 TB/s.  Where the next chunk's gradients would take longer than
 * this chunk's Hessian work (few groups and d_out large against d_in: roughly 3000 * d_out * next_n > g * d_in^2 * n;
 * or a small d_in, whose launch has few CTAs) the call runs the saliency step as a kernel of its own before the
 * Hessian kernel instead; results are the same.
 * next_n == 0: the call is gq_hessian_accumulate.  n == 0: the call is gq_saliency_prepared for the next chunk
 * (after the arguments of this chunk have been checked).
 * The caller runs the saliency step of the very first chunk with gq_saliency_prepared.
 */
int32_t gq_hessian_accumulate_ahead(const void *X, int64_t n, int64_t d_in, int64_t ld_x, const float *s,
                                    int64_t ld_s, int32_t g, float *H, uint32_t flags, void *workspace,
                                    size_t workspace_bytes, const void *next_grad, int64_t next_n, int64_t d_out,
                                    int64_t ld_grad, float grad_scale, float *next_s, int64_t next_ld_s,
                                    void *next_workspace, size_t next_workspace_bytes, void *stream);

/* Scratch bytes gq_hessian_accumulate needs for chunks of up to n_max tokens (0 on bad arguments). */
size_t gq_hessian_workspace_bytes(int64_t n_max, int64_t d_in, int32_t g, uint32_t flags);

/*
 * Completes H after the last chunk: copies the upper triangle onto the lower one,
 * H[k][b][a] = H[k][a][b] for a < b, so that every H_k is a full, exactly symmetric matrix
 * (H_k is symmetric by definition: Section 3.2).  Idempotent.  H 128-byte aligned.
 */
int32_t gq_hessian_finalize(float *H, int64_t d_in, int32_t g, void *stream);

/*
 * Token-sharded accumulation over several GPUs: H_k is a sum over tokens (Algorithm 1, Hessian step), so every GPU
 * may run gq_hessian_accumulate on its own share of the tokens and the partial matrices are then added.
 * These two calls do that exchange with plain loads from the other GPUs' memory (peer access enabled by the
 * caller, e.g. through CUDA IPC or symmetric memory); no kernel waits for another GPU, the CALLER provides
 * the synchronisation:
 *     every rank:  accumulate its chunks;  barrier (all partial matrices complete)
 *     every rank:  gq_hessian_reduce_share(...);  barrier (all shares reduced)
 *     every rank:  gq_hessian_gather_shares(...); barrier (nobody still reads this rank's H)
 *     every rank:  gq_hessian_finalize(own H, ...)
 * The upper triangle is exchanged in 128 x 128 blocks; rank r owns blocks [r B / R, (r + 1) B / R) of the
 * B = g nb (nb + 1) / 2 blocks (nb = ceil(d_in / 128)), numbered group after group and, inside a group, block
 * column after block column.  reduce_share adds rank r's blocks over all R matrices in rank order (the result
 * does not depend on which GPU forms it) and stores them in H_ranks[rank]; gather_shares copies the other
 * ranks' blocks from their owners' matrices into H_ranks[rank].  Afterwards every rank holds the same upper
 * triangle, bit for bit.
 *
 *   H_ranks    HOST array of `ranks` DEVICE pointers: the [g, d_in, d_in] fp32 matrix of rank 0 .. ranks-1
 *              as addressable from the calling GPU (H_ranks[rank] is the caller's own), 16-byte aligned
 *   ranks      1 <= ranks <= 16 (1: both calls are no-ops)
 *   rank       0 <= rank < ranks
 * The kernels run on `stream` of the current device.  Passing the same set of matrices and every rank in turn
 * from one GPU is valid as well (all "ranks" in one address space).
 */
int32_t gq_hessian_reduce_share(float *const *H_ranks, int32_t ranks, int32_t rank, int64_t d_in, int32_t g,
                                void *stream);
int32_t gq_hessian_gather_shares(float *const *H_ranks, int32_t ranks, int32_t rank, int64_t d_in, int32_t g,
                                 void *stream);

/*
 * Objective, Eq. 7:
 *     loss_out[k] = sum_{j in J_k} (w_j - what_j)^T H_k (w_j - what_j),  k < g
 *     loss_out[g] = sum_k loss_out[k]
 *
 *   W, W_hat   fp32 [d_out, d_in] row-major, 16-byte aligned (row j = output channel j)
 *   H          fp32 [g, d_in, d_in] as left by gq_hessian_accumulate or gq_hessian_finalize, 128-byte aligned:
 *              only entries with a <= b are read
 *   loss_out   fp64 [g + 1] in device memory
 *   workspace  device scratch of at least gq_objective_workspace_bytes(d_in, d_out, g) bytes,
 *              1024-byte aligned
 * Same shape rules as above (d_in % 8 == 0, d_out % g == 0, (d_out / g) % 8 == 0).
 * Arithmetic: delta = W - W_hat in fp32.  A first pass finds max |delta| over the layer, a second writes
 * delta * 2^e to the workspace as ONE fp16 matrix, e chosen so that the largest entry lies in [2^14, 2^15)
 * (11 significant bits for every entry down to 2^-28 of the largest; round to nearest, no bias).  The Gram
 * matrices Delta_k^T Delta_k are formed on the tensor cores (fp16 operands, fp32 accumulation) two 256-column
 * tiles at a time and contracted with H_k (fp32) straight out of tensor memory; partial sums are reduced in
 * fp64 in a fixed order and multiplied by 2^-2e.  Relative error of the result: at most 2^-11 = 4.9e-4 if
 * every rounding error had the same sign and H_k had no negative entries, about 1e-6 for rounding errors of
 * random sign (what is seen on quantisation errors).  Results are bit-reproducible run to run.
 */
int32_t gq_objective(const float *W, const float *W_hat, int64_t d_in, int64_t d_out, const float *H,
                     int32_t g, double *loss_out, void *workspace, size_t workspace_bytes,
                     void *stream);

size_t gq_objective_workspace_bytes(int64_t d_in, int64_t d_out, int32_t g);

/*
 * The whole path for one layer with HOST inputs and outputs (Algorithm 1's grouping, saliency and Hessian steps, and Eq. 7):
 * streams X and dl/dZ from host memory in chunks of `chunk` tokens, builds s and H on the device,
 * finalizes H, evaluates the objective and copies the results back.
 *
 *   X_host, grad_host   HOST bf16 [n, d_in] / [n, d_out], densely packed (pinned memory makes
 *                       the copies asynchronous; pageable memory also works)
 *   W_host, W_hat_host  HOST fp32 [d_out, d_in]
 *   loss_host           HOST fp64 [g + 1], written before the call returns
 *   H_host              HOST fp32 [g, d_in, d_in] or NULL to skip copying H back
 *   arena, arena_bytes  DEVICE scratch of at least gq_layer_host_arena_bytes(...) bytes,
 *                       1024-byte aligned; it holds the chunk buffers, s, H and the workspaces
 * The call synchronises `stream` before returning (it is the only call that does) and also
 * returns device-side errors (as gq_check would).
 */
int32_t gq_layer_objective_host(const void *X_host, const void *grad_host, int64_t n, int64_t chunk,
                                int64_t d_in, int64_t d_out, int32_t g, float grad_scale,
                                const float *W_host, const float *W_hat_host, double *loss_host,
                                float *H_host, void *arena, size_t arena_bytes, void *stream);

size_t gq_layer_host_arena_bytes(int64_t chunk, int64_t d_in, int64_t d_out, int32_t g);

/*
 * The objective for callers that cannot allocate device memory (no counterpart in the paper; it is
 * gq_objective with the scratch supplied by the library instead of the caller).
 *
 * Some users of this library run where cudaMalloc is off limits: inside a region that is being
 * recorded into a CUDA graph, inside a framework callback that must not touch the allocator, in a
 * process whose whole memory budget was handed to another pool at start-up, or in a latency-critical
 * loop where an allocation (and the implicit synchronisation of a free) is not acceptable.  For them
 * this entry point keeps its scratch in a fixed array inside the library's own device image:
 *
 *   - the array is 4 MiB + 256 KiB (two bf16 copies of W - W_hat and the partial sums); every GPU on
 *     which the library is used holds that much from the moment the library is loaded until exit;
 *   - therefore only small layers fit: d_in * d_out <= 1,048,576 weights and
 *     NJ * (NJ + 1) / 2 * g <= 4096 with NJ = ceil(d_in / 256).  Anything larger returns
 *     GQ_ERR_UNSUPPORTED_SHAPE and launches nothing: use gq_objective with your own workspace;
 *   - the call makes no cudaMalloc / cudaFree and no call into an allocating library.  The first
 *     call on each device looks up the array's device address once (cudaGetSymbolAddress) and sets
 *     kernel attributes; make that first call outside any stream capture;
 *   - all calls on a device share the one array.  Two calls that overlap on the GPU (different
 *     streams, or different host threads without ordering) race on it and give wrong results:
 *     order them on one stream or with events.  The array keeps what the last call wrote; every
 *     byte a call reads it has written itself first, so stale contents never leak into a result.
 *
 * Arguments and arithmetic (delta as two bf16 terms, three tensor-core products, fp64 reduction in a
 * fixed order) are those described for gq_objective; W, W_hat, H, loss_out are the caller's device
 * buffers.  The kernel behind this entry point works on one 256 x 256 tile of H at a time, the one behind
 * gq_objective on other units and, since version 0.2, with other operand types, so the two entry
 * points agree to rounding (well inside the 1e-3 relative tolerance of the objective), not bit for bit.
 * Repeated calls of this entry point on the same inputs do return identical bits.
 */
int32_t gq_objective_noalloc(const float *W, const float *W_hat, int64_t d_in, int64_t d_out,
                             const float *H, int32_t g, double *loss_out, void *stream);

/*
 * Cyclic coordinate descent on the objective of Eq. 7 with fixed per-channel codebooks: the assignment
 * step of the layer-wise quantiser (Section 4.2, Eq. 10; Appendix B.2, Algorithm 4).  For every group k and
 * every channel j in J_k, `cycles` times, the coordinates i = 0 .. d_in - 1 are visited in order and set to
 *     W_hat[j][i] = Round_j( W[j][i] - (1 / H_k[i][i]) * sum_{c != i} H_k[i][c] * (W_hat[j][c] - W[j][c]) ),
 * Round_j = the nearest of codebook[j][0 .. m-1] (ties: the smaller index), using the current W_hat of all
 * other coordinates.  Started from a W_hat whose entries are codebook values this never increases a
 * channel's objective (Proposition 1).
 *
 *   W          fp32 [d_out, d_in], 16-byte aligned (row j = output channel j)
 *   W_hat      fp32 [d_out, d_in], in: the starting point, out: the result (every entry a codebook value)
 *   Q          uint8 [d_out, d_in], out: index of W_hat[j][i] in codebook[j]
 *   codebook   fp32 [d_out, m], 1 <= m <= 16 (need not be sorted)
 *   H          fp32 [g, d_in, d_in], FULL symmetric matrices (after gq_hessian_finalize), 16-byte aligned.
 *              A coordinate with H_k[i][i] <= 0 is rounded to the codebook value nearest to W[j][i].
 *   cycles     >= 0 (0 only transposes W_hat through the workspace and back; Q is then all zero)
 *   workspace  device scratch of at least gq_cd_workspace_bytes(d_in, d_out, g) bytes, 1024-byte aligned
 * Same shape rules as gq_objective.
 * Arithmetic: coordinates are processed in blocks of 256.  The contributions of the coordinates outside
 * a block are formed on the tensor cores from bf16 hi + lo splits of H and W_hat - W (three products,
 * fp32 accumulation: about 16 significant bits per factor); everything inside a block, and the rounding
 * decision, is fp32.  Decisions can therefore differ from exact arithmetic only where the rounding
 * target lies within about 1e-5 (relative to the values involved) of the midpoint between two codebook
 * values; from such a coordinate on that channel follows its own, equally valid, descent path.
 * The pieces of a block's tensor-core product are combined with atomic adds in no fixed order, so two runs
 * on the same inputs agree bit for bit only as long as no decision falls within that rounding of a tie.
 */
int32_t gq_cd_cycles(const float *W, float *W_hat, uint8_t *Q, const float *codebook, int32_t m,
                     int64_t d_in, int64_t d_out, const float *H, int32_t g, int32_t cycles,
                     void *workspace, size_t workspace_bytes, void *stream);

size_t gq_cd_workspace_bytes(int64_t d_in, int64_t d_out, int32_t g);

/*
 * Synchronises `stream`, then returns and clears the first device-side error recorded on the
 * current device since the last gq_check (GQ_OK if none).  A pipeline wait inside a kernel that
 * exceeds its time budget (2 s by default; environment variable GQ_WAIT_BUDGET_MS) makes the
 * kernel stop early, leave its outputs incomplete and record GQ_ERR_TIMEOUT here.
 * If `detail` is not NULL it receives 4 words: {status, site id, block index, work-unit index}.
 */
int32_t gq_check(void *stream, uint32_t *detail /* HOST, may be NULL */);

/*
 * Codebook step of the layer-wise quantiser (Section 4.2, Eq. 8; the codebook steps of Algorithm 2): with the
 * assignment matrix P^(j) in {0,1}^{d_in x m} given by the codes of channel j (P_iq = 1 iff Q[j][i] == q),
 *     codebook[j] = (P^T H_k P + lambda I)^-1 P^T H_k w_j          for every channel j of every group k,
 * the minimiser of channel j's objective over its m codebook values for fixed codes (lambda is the small
 * constant the paper adds to the diagonal, 1e-7 there; a level that no coordinate uses gets the value 0).
 *
 *   W          fp32 [d_out, d_in], 16-byte aligned
 *   Q          uint8 [d_out, d_in], codes < m (larger values are read as m - 1)
 *   m          1 <= m <= 16
 *   H          fp32 [g, d_in, d_in], FULL symmetric matrices (after gq_hessian_finalize), 16-byte aligned
 *   lambda     >= 0
 *   codebook   fp32 [d_out, m], out
 *   W_hat      fp32 [d_out, d_in] or NULL; out: W_hat[j][i] = codebook[j][Q[j][i]]
 *   workspace  device scratch of at least gq_codebook_workspace_bytes(d_in, d_out, g, m) bytes, 1024-byte aligned
 * Same shape rules as gq_objective.
 * Arithmetic: H_k W_k^T and H_k [P^(j) ...] are formed on the tensor cores, fp32 accumulation, from bf16
 * hi + lo splits of H and W (16 significant bits per factor; what is dropped is of the size of the fp32
 * accumulation error; the one-hot columns are exact).  The sums over the rows of each level and the m x m
 * Cholesky solves are fp64.
 * Together with gq_cd_cycles and gq_objective this is Algorithm 2: repeat { gq_codebook_update (with W_hat);
 * gq_cd_cycles } T times, then gq_codebook_update once more.
 */
int32_t gq_codebook_update(const float *W, const uint8_t *Q, int32_t m, int64_t d_in, int64_t d_out,
                           const float *H, int32_t g, double lambda, float *codebook, float *W_hat,
                           void *workspace, size_t workspace_bytes, void *stream);

size_t gq_codebook_workspace_bytes(int64_t d_in, int64_t d_out, int32_t g, int32_t m);

/*
 * The layer-wise non-uniform quantiser, Algorithm 2, as one call: starting from the assignment Q,
 *     repeat T times { codebook step (Eq. 8) ; K cycles of coordinate descent (Eq. 10) } ; codebook step
 * i.e. exactly the sequence of gq_codebook_update and gq_cd_cycles calls described above, enqueued on `stream`
 * without any host synchronisation in between.
 *
 *   W          fp32 [d_out, d_in], 16-byte aligned
 *   Q          uint8 [d_out, d_in], in: the initial assignment (codes < m), out: the final one
 *   m          1 <= m <= 16;   T >= 0 rounds;   K >= 0 cycles per round;   lambda >= 0 (the paper: 1e-7)
 *   H          fp32 [g, d_in, d_in], full symmetric matrices (after gq_hessian_finalize), 16-byte aligned
 *   codebook   fp32 [d_out, m], out
 *   W_hat      fp32 [d_out, d_in], out: codebook[j][Q[j][i]], 16-byte aligned
 *   workspace  device scratch of at least gq_lnq_workspace_bytes(d_in, d_out, g, m) bytes, 1024-byte aligned
 * No step increases any channel's objective (Proposition 1 and the optimality of Eq. 8), up to rounding.
 */
int32_t gq_lnq(const float *W, uint8_t *Q, int32_t m, int64_t d_in, int64_t d_out, const float *H, int32_t g,
               int32_t T, int32_t K, double lambda, float *codebook, float *W_hat, void *workspace,
               size_t workspace_bytes, void *stream);

size_t gq_lnq_workspace_bytes(int64_t d_in, int64_t d_out, int32_t g, int32_t m);

/*
 * Self-test of the device-side failure detection (no counterpart in the paper): launches a one-warp kernel
 * that waits, with the pipeline kernels' own bounded wait, on a barrier nothing ever signals.  After
 * `budget_ms` (1 .. 1000) the wait gives up, the kernel returns normally and the next gq_check() reports
 * GQ_ERR_TIMEOUT with site id 99; the CUDA context stays usable.  Nothing is trapped, faulted or hung.
 */
int32_t gq_selftest_wait_timeout(int32_t budget_ms, void *stream);

/* Number of kernels this library has launched from the calling process (for bookkeeping). */
uint64_t gq_launch_count(void);

/*
 * Measurement aid (no counterpart in the paper).  The library's kernels, in launch order of a layer:
 */
enum gq_kernel_id {
    GQ_KERNEL_SALIENCY = 0,    /* Algorithm 1, saliency step                                    */
    GQ_KERNEL_HESSIAN = 1,     /* tensor-core H += X^T Diag(s_k) X, scaling fused (Algorithm 1, Hessian step) */
    GQ_KERNEL_MIRROR = 2,      /* gq_hessian_finalize                                    */
    GQ_KERNEL_SPLIT_DELTA = 3, /* W - W_hat -> fp16 (maximum pass + conversion pass)     */
    GQ_KERNEL_GRAM_DOT = 4,    /* tensor-core Delta_k^T Delta_k contracted with H_k (Eq. 7) */
    GQ_KERNEL_REDUCE = 5,      /* fp64 reduction of the partial sums                     */
    GQ_KERNEL_SPLIT_SALIENCY = 6, /* s -> pairs of bf16 terms for the Hessian kernel's scalers */
    GQ_KERNEL_CD_PANEL = 7,    /* coordinate descent: tensor-core product with the coordinates outside a block */
    GQ_KERNEL_CD_BLOCK = 8,    /* coordinate descent: the 256 coordinates of a block, in order */
    GQ_KERNEL_CD_AUX = 9,      /* coordinate descent: transposes and bf16 splits */
    GQ_KERNEL_CB_GEMM = 10,    /* codebook step: tensor-core products H W^T and H [P ...] */
    GQ_KERNEL_CB_FOLD = 11,    /* codebook step: sums over the rows of each level, m x m solves */
    GQ_KERNEL_CB_AUX = 12,     /* codebook step: splits, transposes, one-hot columns, W_hat */
    GQ_KERNEL_EXCHANGE = 13,   /* token-sharded accumulation: reduce / gather of blocks of H over peer memory */
    GQ_KERNEL_COUNT = 14
};

/*
 * gq_kernel_timing_enable(1) makes every later launch record a CUDA event on its stream directly
 * before and after the kernel; gq_kernel_timing_enable(0) stops that.  Neither call touches what
 * was recorded so far, so a caller can time a sample of its launches (the event pairs cost about 4 % of a
 * step of 52 launches when every launch is timed).  gq_kernel_timing_read() waits for the recorded events and writes, per
 * gq_kernel_id, the summed device time in milliseconds and the number of launches into two HOST
 * arrays of GQ_KERNEL_COUNT entries, then discards them.  Off by default.
 */
int32_t gq_kernel_timing_enable(int32_t enable);
int32_t gq_kernel_timing_read(double *ms_sum, uint64_t *launches);

#ifdef __cplusplus
}
#endif
#endif /* GQ_H_ */
