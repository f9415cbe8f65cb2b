/*
 * tm.h -- C ABI of the transposable N:M mask search for NVIDIA B200 (sm_100a).
 *
 * Method: "Accelerated Sparse Neural Training: A Provable and Efficient Method to Find N:M
 * Transposable Masks" (arXiv 2102.08124), Section 4 "Computing transposable sparsity masks".
 *
 * The operation (Section 4, "Problem formulation", Eq. 1).  A weight matrix W[rows, cols] is tiled
 * into independent M x M blocks anchored at element (0,0).  For every block the search returns a
 * 0/1 mask S with exactly N ones in each block row and each block column -- so that W and its
 * transpose obey the same N:M pattern -- chosen to maximise sum_ij S_ij |W_ij|.
 *
 *   method TM_EXACT         the optimum of Eq. 1 (the paper reaches it through the min-cost flow of
 *                           Fig. 3; for M = 4 it is also reached by enumerating all 90 patterns).
 *   method TM_APPROX        Algorithm 1 (greedy 2-approximation) followed by a deterministic
 *                           completion to exactly N kept entries per line.  Algorithm 1 alone yields a
 *                           cover that may prune more than M-N entries of a line; the paper does not
 *                           say how to finish it, the completion is this library's:
 *                             B. visit the pruned entries heavy -> light, keep an entry again when
 *                                its row and its column both hold fewer than N kept entries;
 *                             C. while a row is short: take the lightest kept entry (r', c') for
 *                                which a short row r with (r, c') free and a short column c with
 *                                (r', c) free exist, un-keep it, keep the heaviest such (r, c') and
 *                                the heaviest such (r', c).
 *   method TM_APPROX_COVER  Algorithm 1 only: at most N kept entries per line (the object the
 *                           paper's Lemma, W(P) <= 2 W*, speaks about).
 *
 * Conventions the paper leaves open
 *   - N counts KEPT entries per block row / column (Eq. 1).  Supported (N, M): (2, 4) and (4, 8) on every
 *     path; (1, 4), (3, 4), (2, 8) and (6, 8) through the generic kernels.
 *   - Order of magnitudes: by the bit pattern of |w| (sign cleared, so -0 == +0), ties broken by the
 *     row-major position p = i*M + j inside the block; the earlier position is the lighter one.
 *     Algorithm 1's degree test is read as "fewer than M-N pruned edges at the node".
 *   - TM_EXACT compares candidate masks by (exact sum of kept |w|, code(S) = sum_p S_p 2^p),
 *     larger wins; the sum is carried in integer arithmetic, never rounded.
 *
 * Layouts
 *   W, masked_w_out   row-major, leading dimension ld (elements; ld == cols in the plain calls),
 *                     fp32 or bf16.  rows and cols must be multiples of M (callers zero-pad).
 *   mask_out          rows * tm_mask_words_per_row(cols) 32-bit words; the bit of element (r, c) is
 *                     bit c % 32 of word r * wpr + c / 32; padding bits of the last word are 0.
 *   masked_w_out      kept entries copied bit for bit, pruned entries +0.  May be NULL (mask only)
 *                     or equal to W (in place).
 *   objective_out     one double: sum over the whole matrix of kept |w| (fp32 adds per thread,
 *                     fp64 across threads and CTAs in a fixed order: same input -> same bits).
 *                     May be NULL.
 *
 * Ownership and execution.  Unless a function says otherwise every data pointer is a DEVICE
 * pointer owned by the caller, calls are asynchronous on the stated stream, and nothing is
 * synchronised.  Host-detectable errors are returned (nothing is launched); conditions only the
 * device can see are OR-ed into a device status word (TM_DEV_* bits) that the caller reads after
 * its own synchronisation -- with TM_DEV_NONFINITE or TM_DEV_BADMASK the outputs are fully written and
 * deterministic; TM_DEV_INTERNAL means the call failed (see the bit's comment).
 * There is no CPU fallback: without a CUDA device every compute entry point returns TM_ERR_CUDA.
 */
#ifndef TM_H_
#define TM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TM_VERSION 100

/* method */
#define TM_EXACT 0
#define TM_APPROX 1
#define TM_APPROX_COVER 2

/* dtype */
#define TM_F32 0
#define TM_BF16 1

/* return codes (host-detected) */
#define TM_OK 0
#define TM_ERR_NULL 1       /* a required pointer is NULL */
#define TM_ERR_SHAPE 2      /* negative size, rows or cols not a multiple of M, ld < cols, count < 0 */
#define TM_ERR_NM 3         /* unsupported (N, M) */
#define TM_ERR_METHOD 4
#define TM_ERR_DTYPE 5
#define TM_ERR_ALIGN 6      /* W / masked_w_out base or row pitch not a multiple of min(16, M * element size) bytes, mask_out not of 4, objective_out not of 8 */
#define TM_ERR_CUDA 7       /* a CUDA runtime call failed (no device, launch error, allocation failure) */
#define TM_ERR_WORKSPACE 8  /* workspace NULL, misaligned (256 bytes) or smaller than tm_workspace_bytes() */
#define TM_ERR_TOO_LARGE 9  /* more matrices than the built-in scratch of tm_find_mask_batched_static() can serve */
#define TM_ERR_CAPTURE 10   /* cuda_stream is being captured and the call would have to copy descriptor tables from host memory */

/* device status bits */
#define TM_DEV_NONFINITE 1  /* an Inf or NaN was met in W (it is ordered by its bit pattern) */
#define TM_DEV_INTERNAL 2   /* a bound inside a kernel was hit (not expected to happen).  An iteration cap of a per-block search leaves
                               that block with the mask reached so far; a bulk copy that did not land within its bounded wait makes
                               the warp stop, and the outputs of its remaining work items stay UNWRITTEN: treat the call as failed */
#define TM_DEV_BADMASK 4    /* tm_compress_2_4: a group of four did not hold exactly two kept entries (zeros were emitted) */

typedef struct tm_problem {
    const void* W;          /* device, dtype, rows x ld */
    int64_t rows, cols, ld; /* ld in elements */
    int32_t dtype;          /* TM_F32 or TM_BF16 */
    uint32_t* mask_out;     /* device, rows * wpr words, required */
    void* masked_w_out;     /* device, same dtype/ld as W; NULL or == W allowed */
    double* objective_out;  /* device, one double; may be NULL */
} tm_problem;

/* Number of 32-bit mask words per matrix row, ceil(cols / 32), and for the whole matrix. */
size_t tm_mask_words_per_row(int64_t cols);
size_t tm_mask_words(int64_t rows, int64_t cols);

/*
 * tm_find_mask / tm_find_mask_bf16 -- Section 4, Eq. 1 (TM_EXACT), Algorithm 1 (TM_APPROX*).
 * One matrix, fp32 resp. bf16, ld == cols, on the legacy default stream (stream 0) of the current
 * device.  All pointers are device pointers.  The first call on a device allocates a small scratch
 * buffer (objective partials, a status word and a count of finished thread blocks) that the library keeps
 * until the process exits; tm_find_mask_batched() never allocates.  For a 16-byte aligned matrix the call is a
 * single kernel launch: the thread block that finishes last adds up the objective partials in a fixed order.  Device status bits of these calls accumulate in that
 * scratch and are fetched with tm_device_status().
 */
int tm_find_mask(const void* W, int64_t rows, int64_t cols, int N, int M, int method,
                 uint32_t* mask_out, void* masked_w_out, double* objective_out);
int tm_find_mask_bf16(const void* W, int64_t rows, int64_t cols, int N, int M, int method,
                      uint32_t* mask_out, void* masked_w_out, double* objective_out);

/* Synchronises stream 0 of the current device, returns the OR of the TM_DEV_* bits raised by the
 * plain calls since the last query in *status_host (host pointer) and clears them. */
int tm_device_status(int* status_host);

/*
 * tm_find_mask_batched -- the same search for `count` matrices (a whole model) in one launch:
 * the from-scratch setting of Section 4.1 re-derives every layer's mask periodically.
 * probs_host: HOST array of descriptors (copied during the call; may be freed on return).
 * workspace_dev: device scratch of at least tm_workspace_bytes(...) bytes, 256-byte aligned, owned
 * by the caller, reusable across calls on the same stream (calls on different streams need
 * different workspaces).  status_dev: device int, OR-ed with TM_DEV_* bits; may be NULL.
 * cuda_stream: a cudaStream_t (NULL = legacy default stream).  Never allocates.  With count == 1 the
 * descriptors travel as kernel arguments and the call only enqueues work; with count > 1 it first copies
 * the descriptor tables from (pageable) host memory into the workspace, and the runtime may hold the
 * calling thread until earlier work of cuda_stream has drained before that copy is staged.  For the same
 * reason only count == 1 calls can be recorded by a stream capture: a count > 1 call on a capturing
 * stream returns TM_ERR_CAPTURE and enqueues nothing -- capture tm_plan_run() instead.
 * All matrices share N, M and method; dtypes may differ.
 */
int tm_find_mask_batched(const tm_problem* probs_host, int count, int N, int M, int method,
                         void* workspace_dev, size_t workspace_bytes, int* status_dev, void* cuda_stream);
size_t tm_workspace_bytes(const tm_problem* probs_host, int count);

/*
 * tm_plan_create / tm_plan_run / tm_plan_destroy -- tm_find_mask_batched() split for training loops that
 * re-derive the masks of the same buffers every few iterations (Section 4.1, "Sparse Training from
 * scratch": the mask is refreshed every 40 iterations).  tm_plan_create validates the descriptors, builds the
 * tensor maps and copies the descriptor tables into the workspace once (synchronising stream 0; it allocates
 * host memory for the plan, nothing on the device).  tm_plan_run then only clears the objective partials and
 * launches the kernels on cuda_stream (the full searches on 16-byte aligned matrices are a single launch that
 * reduces its own objectives and needs no clearing): it touches no host memory asynchronously, so it can be recorded by a stream capture
 * and replayed.  The workspace belongs to the plan until tm_plan_destroy -- its first 256 bytes are cleared at
 * creation and must not be written by anyone else -- and the matrices must stay where they were (same pointers,
 * shapes, pitches).  Masks and masked weights equal tm_find_mask_batched()'s bit for bit; objectives too, except
 * that a launch which reduces its own objectives adds the partial sums in another (fixed) order, i.e. equal
 * up to fp64 rounding.
 */
typedef struct tm_plan tm_plan;
int tm_plan_create(const tm_problem* probs_host, int count, int N, int M, int method, void* workspace_dev, size_t workspace_bytes,
                   tm_plan** plan_out);
int tm_plan_run(const tm_plan* plan, int* status_dev, void* cuda_stream);
void tm_plan_destroy(tm_plan* plan);

/*
 * tm_find_mask_host -- the search on HOST buffers (Eq. 1 / Algorithm 1 as above): copies W to the
 * current device in row strips, runs the kernels and copies mask, masked weights and objective back,
 * overlapping the three on separate streams; returns when the outputs are in host memory.
 * Pinned host buffers make the copies asynchronous; pageable ones work but serialise.
 * masked_w_out_host and objective_out_host may be NULL.  *status_out_host (may be NULL) receives
 * the TM_DEV_* bits.  Allocates device staging buffers on first use and keeps them.
 */
int tm_find_mask_host(const void* W_host, int dtype, int64_t rows, int64_t cols, int N, int M, int method,
                      uint32_t* mask_out_host, void* masked_w_out_host, double* objective_out_host,
                      int* status_out_host);

/*
 * tm_find_mask_batched_static -- no counterpart in the paper: an entry point for callers that must not
 * allocate device memory.  Some hosts of this library (a plug-in running inside another framework's
 * memory pool, a real-time loop that pre-allocates everything, code holding a fixed memory budget)
 * can neither call cudaMalloc themselves nor let a library do it on their behalf, and may have no
 * place to size a workspace up front either.  This call is tm_find_mask_batched() with the workspace
 * replaced by a scratch array built into the library image: TM_STATIC_SCRATCH_BYTES of device memory
 * that every GPU which loads the library holds until the process exits.  It serves at most
 * TM_STATIC_MAX_MATRICES matrices per call (each of any size); a larger count returns
 * TM_ERR_TOO_LARGE and launches nothing -- split the model into several calls.  Inputs and outputs
 * are still the caller's device buffers.
 *
 * The call allocates nothing on the device and frees nothing.  The first call on a device looks the
 * scratch array's device address up (once per device, with that device current); make that first call
 * before any stream capture begins.  Like tm_find_mask_batched(), a call with count > 1 copies its
 * descriptor tables from host memory and is refused (TM_ERR_CAPTURE) on a capturing stream.
 *
 * All calls on one device share the one array, which keeps whatever the previous call left in it; each
 * call clears the objective partials it is about to use.  Calls that can overlap on the GPU (different
 * streams with no dependency between them, or several host threads) MUST be ordered by the caller: the
 * array holds not only the objective partials but, for count > 1, the descriptor table and the tensor
 * maps with the output pointers, at fixed offsets, and every call rewrites them.  A second call can
 * therefore replace the descriptors a running kernel is still reading -- wrong masks and masked weights,
 * and accesses through foreign or half-written descriptors, i.e. memory safety is at stake, not only the
 * objective.  Only count == 1 calls (descriptors passed as kernel arguments) confine such a race to the
 * objective value.  Where calls cannot be ordered use tm_find_mask_batched() with separate workspaces.
 * Results are bit-identical to tm_find_mask_batched() on the same inputs.
 */
#define TM_STATIC_MAX_MATRICES 16
#define TM_STATIC_SCRATCH_BYTES (1064960)
int tm_find_mask_batched_static(const tm_problem* probs_host, int count, int N, int M, int method,
                                int* status_dev, void* cuda_stream);

/*
 * Neighbouring operations.  They share one small device workspace of tm_aux_workspace_bytes() bytes
 * (256-byte aligned, caller-owned, one per stream), run asynchronously on cuda_stream and never allocate.
 *
 * tm_nm_mask_1d -- Section 5, "Structured sparsity without full training": the plain (non-transposable) N:M
 * pattern along rows: in every group of M contiguous weights of a row the M-N of lowest magnitude are pruned
 * (the paper counts the pruned ones; here, as everywhere in this header, N counts the KEPT ones).  Order by
 * (|w|, position), the later of equals being the heavier.  M in {2, 4, 8}, 0 <= N <= M, cols % M == 0.
 * prob_host: one descriptor (host pointer); mask_out, masked_w_out, objective_out as for tm_find_mask.
 * violations_out (device, may be NULL): the paper's "pattern-violations", the number of non-zero weights the
 * pattern removes.  flags & TM_NM1D_ABSORB_MEAN ("mean absorption"): every kept weight receives the mean of
 * its group's pruned weights: mu = (their sum in position order, fp64) / (their number), kept' = kept + mu in
 * fp64, rounded once to fp32 (and from there to bf16, nearest even, for bf16 tensors).  The paper leaves open
 * whether the mean is taken over the pruned or spread over the kept entries; for N = M/2 both agree.
 *
 * tm_mask_violations -- the same count for an arbitrary packed mask (layout of mask_out): weights that are
 * non-zero although their mask bit is 0.
 *
 * tm_compress_2_4 -- Section 1 and Fig. 2: the transposable mask lets the same 2:4 pattern serve Y = W X and
 * dL/dX = W^T dL/dY; this call prepares both operands from one read of W.  values[rows][cols/2]: for every
 * row and every group of four columns the two kept weights in column order; meta[rows][wpr(cols)]: their
 * column indices inside the group as a nibble idx0 | idx1 << 2, group g of the row in bits 4*(g%8) of word g/8.
 * values_t[cols][rows/2], meta_t[cols][wpr(rows)]: the same for W^T (groups of four rows of a column).
 * rows % 4 == cols % 4 == 0; W rows aligned to one block row.  A group without exactly two kept entries gets zeros
 * and raises TM_DEV_BADMASK in *status_dev.  This is this library's plain layout, not a vendor library's.
 *
 * tm_mask_hamming -- number of differing bits of two packed masks of `words` 32-bit words: how much of the
 * mask a refresh changed (Section 4.1 refreshes the mask every 40 iterations; Section 1 recalls that frequent
 * mask changes are what the straight-through training of dense copies has to keep in check).
 */
#define TM_NM1D_ABSORB_MEAN 1
int tm_mask_hamming(const uint32_t* mask_a, const uint32_t* mask_b, int64_t words, unsigned long long* distance_out,
                    void* workspace_dev, size_t workspace_bytes, void* cuda_stream);
size_t tm_aux_workspace_bytes(void);
int tm_nm_mask_1d(const tm_problem* prob_host, int N, int M, int flags, unsigned long long* violations_out,
                  void* workspace_dev, size_t workspace_bytes, int* status_dev, void* cuda_stream);
int tm_mask_violations(const void* W, int dtype, int64_t rows, int64_t cols, int64_t ld, const uint32_t* mask,
                       unsigned long long* violations_out, void* workspace_dev, size_t workspace_bytes, void* cuda_stream);
int tm_compress_2_4(const void* W, int dtype, int64_t rows, int64_t cols, int64_t ld, const uint32_t* mask,
                    void* values, uint32_t* meta, void* values_t, uint32_t* meta_t, int* status_dev, void* cuda_stream);

const char* tm_status_string(int code);
int tm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TM_H_ */
