/*
 * sfda.h -- C ABI of the B200 (sm_100a) Semidirect Fourier Delta Attention library.
 *
 * The library computes the chunkwise constructive chunk-WY forward, the per-chunk
 * factor export and the one-token decode step of the tied SFDA recurrence
 * (Section 3, Eq. "sfda"):
 *
 *     S_t = (I - beta_t k_t k_t^*) Lambda_t S_{t-1} + beta_t k_t v_t^*,
 *     Lambda_t = diag(alpha_t * exp(i theta_t)),        o_t = S_t^* q_t.
 *
 * Storage conventions shared by every entry point
 * -----------------------------------------------
 *  - All tensors are dense, row-major, with the index order written beside them.
 *  - The key space is R^{d_k} ~ C^m, m = d_k / 2: real channel 2j is the real part
 *    and channel 2j+1 the imaginary part of complex coordinate j (the aligned 2x2
 *    rotation-decay blocks of Prop. "Complex phases are real block rotations").
 *    This holds for q, k and for the ROWS of a state S[d_k][d_v].
 *  - v, o and the columns of S are plain real channels (v real, so v^* = v^T).
 *  - alpha, theta are per complex coordinate ([..., m]); beta is one scalar per
 *    token and head.  alpha in (0, 1], beta in [0, 1], |k| <= 1 are preconditions
 *    of the method (Prop. "Basic numerical stability"); they are NOT checked, and
 *    k is not normalised here.
 *  - `dtype` selects the element type of q, k, v, o, o_im: SFDA_F32 (float) or
 *    SFDA_BF16 (bfloat16).  alpha, theta, beta and every state are float.
 *  - o = Re(S_t^* q_t);  o_im = Im(S_t^* q_t) is written when o_im is not NULL.
 *
 * Ownership and execution
 * -----------------------
 *  Unless an argument says "host", pointers are DEVICE pointers owned by the
 *  caller; they must be 16-byte aligned.  The library allocates and frees nothing,
 *  never synchronises, and enqueues all work on `stream` (a cudaStream_t passed as
 *  void*; NULL is the default stream).  Results are ready when the stream reaches
 *  the end of the enqueued work.
 *
 * Errors
 * ------
 *  Every int-returning function returns SFDA_OK (0) or a negative sfda_status.
 *  Arguments are validated on the host before anything is launched; on an error
 *  nothing has been enqueued.  No exceptions, no exit(), no output.
 */
#ifndef SFDA_H
#define SFDA_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define SFDA_API __attribute__((visibility("default")))
#else
#define SFDA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SFDA_OK = 0,
    SFDA_ERR_NULL = -1,        /* a required pointer is NULL                          */
    SFDA_ERR_SHAPE = -2,       /* B, T, H < 1, odd d_k, non-positive chunk            */
    SFDA_ERR_UNSUPPORTED = -3, /* d_k, d_v not in {64,128}; chunk not in {16,...,256}; */
                               /* unknown dtype                                       */
    SFDA_ERR_ALIGN = -4,       /* a pointer is not 16-byte aligned                    */
    SFDA_ERR_WORKSPACE = -5,   /* workspace NULL or smaller than sfda_workspace_bytes */
    SFDA_ERR_CUDA = -6,        /* the CUDA runtime reported an error at launch        */
    SFDA_ERR_TIMEOUT = -7,     /* a bounded device-side wait ran out                  */
    SFDA_ERR_VALUE = -8        /* a scalar argument is out of range (the constants of */
                               /* sfda_frontend; slices / wait_ticks of the diagnostic)*/
} sfda_status;

typedef enum { SFDA_F32 = 0, SFDA_BF16 = 1 } sfda_dtype;

/* Text for a status code (static storage, never NULL). Host only. */
SFDA_API const char *sfda_status_string(int status);

/*
 * Chunk bookkeeping (host only, integer).  Chunks are [j*chunk, (j+1)*chunk); the
 * factors restart at every chunk (Gamma_0 = I, Theorem "Constructive left-to-right
 * chunk-WY recursion").  T need not be a multiple of chunk: the last chunk holds
 * tail_len tokens and is completed with neutral tokens (alpha = 1, theta = 0,
 * beta = 0, k = q = v = 0, for which A_t = I and B_t = 0 by Eq. "AtBt").
 * Writes n_chunks = ceil(T / chunk) and tail_len in [1, chunk].
 */
SFDA_API int sfda_plan(int T, int chunk, int *n_chunks, int *tail_len);

/*
 * Bytes of device scratch sfda_forward should be given for these sizes (0 when it
 * needs none).  The tensor-core path keeps a 256-byte status block there and, when it
 * gets the full size (256 + 4*B*H rounded up to 256 + B*H*d_k*d_v*4 bytes), also the
 * boundary states of the time slices it may cut long sequences into to keep every SM
 * busy; with at least 256 bytes it still runs, one (batch, head) pair per CTA at a time.  Returns 0 for invalid
 * sizes as well; sfda_forward reports those.
 *
 * Concurrency: calls may come from several host threads and streams, each with its own buffers and workspace.
 * When sequences are cut (time slices, or, with at least as many sequences as SMs and a chunk count that does
 * not halve, one contiguous range of chunks per CTA), a CTA of the persistent kernel waits (bounded: about a
 * second, then SFDA_ERR_TIMEOUT through sfda_workspace_status) for the CTA that runs the previous piece of its
 * sequence, so all CTAs of one launch have to
 * be resident together.  Such launches are therefore cooperative launches (at most one CTA per SM): the
 * driver starts such a grid only when all of it fits beside whatever other streams are running, and the call
 * returns the CUDA error instead of launching when the grid can never fit (a context limited to fewer SMs than the
 * device has).
 */
SFDA_API size_t sfda_workspace_bytes(int B, int T, int H, int d_k, int d_v, int chunk, int dtype);

/*
 * How sfda_forward would spread these sizes over a device of n_sm multiprocessors when given workspace_bytes of
 * scratch (host only, integer arithmetic, nothing is launched; Section "chunkwise form": every (batch, head) pair
 * is one serial chain of chunks, so only whole sequences or consecutive pieces of them can be shared out).
 * Writes: slices, the number of equal time slices per sequence (1 = uncut); balanced, 1 when the chunks of
 * all sequences, laid end to end, are instead cut into one contiguous range per CTA (ranges differ by at most one
 * chunk; CTA c starts at chunk c*(N/ctas) + min(c, N%ctas) of the N = B*H*ceil(T/chunk)); ctas, the number of
 * persistent CTAs.  Shapes that the tensor-core path does not take (see sfda_forward) report slices = 1,
 * balanced = 0, ctas = 0.  Returns SFDA_ERR_NULL / SFDA_ERR_SHAPE for bad arguments.
 */
SFDA_API int sfda_forward_partition(int B, int T, int H, int d_k, int d_v, int chunk, int dtype,
                                    size_t workspace_bytes, int n_sm, int *slices, int *balanced, int *ctas);

/*
 * Chunkwise forward: o_t for every token and the final state, by Algorithm 1
 * ("Constructive SFDA-WY chunk summary"), Eq. "apply-transfer" and Theorem "Prefix
 * outputs inside a chunk", scanning boundary states over the chunks of every
 * (batch, head) pair (the "boundary-state scan").
 *
 *  q, k   [B][T][H][d_k]   dtype          v   [B][T][H][d_v]  dtype
 *  alpha, theta [B][T][H][m] float        beta [B][T][H]      float
 *  S0     [B][H][d_k][d_v] float, or NULL for a zero initial state
 *  o      [B][T][H][d_v]   dtype          o_im same shape, or NULL
 *  S_T    [B][H][d_k][d_v] float, or NULL; may alias S0
 *  workspace: device scratch, sfda_workspace_bytes(...) bytes for full speed (may be
 *             NULL when that is 0; the tensor-core path needs at least 256 bytes);
 *             contents are clobbered.
 *
 * Supported: d_k, d_v in {64, 128}; chunk in {16, 32, 64, 128, 256}.  The kernels' tile
 * is at most 64 tokens: chunk = 128 or 256 runs as an exact superchunk of two or four
 * 64-token tiles (Section 6, "superchunks": chunk transfers compose exactly; the state
 * is carried on chip from tile to tile), so outputs and final state are those of the
 * chunk size named (they do not depend on where a sequence is cut) at the cost per
 * token of chunk = 64; workspace, partition and slicing rules are those of chunk = 64.
 * bf16 inputs with d_k = d_v = 128 and chunk >= 64 take the tensor-core path
 * (bf16 operands, fp32 accumulation and state); everything else runs in fp32 on
 * the CUDA cores.  The tensor-core path forms 1/gamma_t inside a chunk and so
 * additionally assumes prod_{t in chunk} alpha_{t,j} >= exp(-80) for every
 * coordinate j; beyond that results lose accuracy but stay finite.
 */
SFDA_API int sfda_forward(const void *q, const void *k, const void *v,
                 const float *alpha, const float *theta, const float *beta,
                 const float *S0, void *o, void *o_im, float *S_T,
                 int B, int T, int H, int d_k, int d_v, int chunk, int dtype,
                 void *workspace, size_t workspace_bytes, void *stream);

/*
 * sfda_forward on the tensor-core shapes (bf16, d_k = d_v = 128, chunk = 64 exactly; SFDA_ERR_UNSUPPORTED otherwise) that
 * also writes the integer bookkeeping of the cumulative phase (Eq. "constructive-Gamma"; App. "Kernel sketch",
 * Stage 1: phases kept as integers):
 *
 *  phase_turns [B][H][NC][m] uint32 (device, 16-byte aligned, NC = ceil(T / chunk)): for every chunk and complex
 *         coordinate the phase the chunk closes with, in 2^-32 turns: the sum, modulo 2^32, over the chunk's tokens of
 *         (uint32)(int64)rint(theta * 683565275.6f), the product taken in single precision (one IEEE multiply,
 *         round to nearest even) and rounded to the nearest integer (ties to even).  Tokens beyond T count as 0.
 *
 * The kernel forms exactly these integers (per group of eight tokens, then summed; integer addition is
 * associative, so the grouping does not show) and takes the chunk's closing rotation and every group's starting
 * angle from them; inside a group of eight tokens gamma_t is a running single-precision complex product.  The
 * conversion differs from sfda_chunk_factors' double-precision one by at most 2^-24 of the angle per token.
 * All other arguments, results and errors as sfda_forward.
 */
SFDA_API int sfda_forward_phase(const void *q, const void *k, const void *v,
                 const float *alpha, const float *theta, const float *beta,
                 const float *S0, void *o, void *o_im, float *S_T, uint32_t *phase_turns,
                 int B, int T, int H, int d_k, int d_v, int chunk, int dtype,
                 void *workspace, size_t workspace_bytes, void *stream);

/*
 * Diagnostic: exercises the kernel's handling of a wait that runs out, without any fault.  Every wait inside the
 * tensor-core forward is bounded (App. "Kernel sketch" leaves the pipeline to the implementation; the boundary-state
 * scan of Section "chunkwise form" is what is being handed over); when one runs out, the CTA raises a flag, all its
 * roles leave their loops, tensor memory is freed, the kernel ends normally and the status word reads
 * SFDA_ERR_TIMEOUT.  This call runs sfda_forward on the tensor-core shapes with every sequence cut into `slices`
 * (2..8, dividing the number of chunks) time slices whose boundary states are written but never announced, and
 * with the wait limit set to `wait_ticks` SM-clock ticks (2^16..2^26): every slice after the first waits for its
 * predecessor until the limit and gives up.  The outputs of first slices are valid, everything else is undefined;
 * sfda_workspace_status(workspace) afterwards returns SFDA_ERR_TIMEOUT, and the context stays usable: a following
 * ordinary call on the same workspace is correct.  Needs the full sfda_workspace_bytes; SFDA_ERR_VALUE for slices
 * or wait_ticks out of range, SFDA_ERR_SHAPE when slices does not divide the chunk count, otherwise the errors of
 * sfda_forward.  Nothing in the library calls this.
 */
SFDA_API int sfda_forward_withheld_handoff(const void *q, const void *k, const void *v,
                 const float *alpha, const float *theta, const float *beta,
                 const float *S0, void *o, void *o_im, float *S_T,
                 int B, int T, int H, int d_k, int d_v, int chunk, int dtype, int slices, unsigned wait_ticks,
                 void *workspace, size_t workspace_bytes, void *stream);

/*
 * sfda_forward for few, long sequences: a two-level scan over the time axis.  A sequence is one serial chain of
 * chunks, so with fewer (batch, head) pairs than SMs most of the GPU idles.  By Theorem "Exact affine chunk
 * transfer" a time slice maps its initial state affinely, S_out = P S_in + B; so every sequence is cut into
 * n_slices slices that run as independent sequences: once from a zero state (B and the outputs o^(0)), once with
 * v = 0 from [I | 0] (P, and g_t = P_t^* q_t in the first d_k / 2 channels of its outputs); a small scan
 * S_{i+1} = P_i S_i + B_i gives every slice its true initial state S_in, and o_t = o_t^(0) + S_in^* g_t is added in
 * place by a tensor-core product.  Two chain passes, each n_slices times as parallel, and a memory-bound epilogue;
 * exact algebra, with P, B, g and S_in carrying the forward's bf16 rounding once more.
 *
 * Arguments, layouts and results as sfda_forward.  n_slices >= 2 must divide T into multiples of chunk;
 * n_slices = 0 lets the library choose (the largest power of two with B H n_slices <= the device's SM count and at
 * least 16 chunks per slice; below 4 slices the call is sfda_forward).  Only the shapes of the tensor-core path
 * (bf16, d_k = d_v = 128, chunk = 64) -> SFDA_ERR_UNSUPPORTED otherwise, also for an n_slices that does not divide.
 * workspace: sfda_forward_two_level_workspace_bytes(...) bytes (the forward's own scratch, five sets of
 * B n_slices H states, a zero v and the two outputs of the second pass, each of the size of v); all of it is
 * required.  sfda_workspace_status on this workspace reports the last of the two chain passes.
 */
SFDA_API size_t sfda_forward_two_level_workspace_bytes(int B, int T, int H, int d_k, int d_v, int chunk, int dtype,
                                                       int n_slices);
SFDA_API int sfda_forward_two_level(const void *q, const void *k, const void *v,
                                    const float *alpha, const float *theta, const float *beta,
                                    const float *S0, void *o, void *o_im, float *S_T,
                                    int B, int T, int H, int d_k, int d_v, int chunk, int dtype, int n_slices,
                                    void *workspace, size_t workspace_bytes, void *stream);

/*
 * After work enqueued by sfda_forward with a non-empty workspace: waits for `stream`
 * and reads the status word the tensor-core kernel keeps at the start of the
 * workspace.  Returns SFDA_OK, or SFDA_ERR_TIMEOUT when a bounded device-side wait
 * (on a TMA copy or a tensor-core commit) ran out, in which case the kernel returned
 * early and o, o_im, S_T of that call are invalid; *detail (host, may be NULL) gets
 * the raw word.  Synchronises the stream.  Host only.
 */
SFDA_API int sfda_workspace_status(const void *workspace, void *stream, uint32_t *detail);

/*
 * sfda_forward for callers that cannot hand the library any scratch memory.  (The paper has no counterpart
 * to this entry point; it exists for deployment reasons only.)
 *
 * Who needs it: programs that give all device memory to their own pool at start-up and must not call the
 * CUDA allocator afterwards -- inference servers with a fixed memory plan, plug-ins running inside another
 * application's memory budget, real-time loops that cannot afford the device-wide synchronisation an
 * allocation or a free may cause.  Such a caller can still pass its inputs and outputs (it owns those), but it
 * has nowhere to take the workspace of sfda_forward from.  Here the workspace is a block of
 * SFDA_STATIC_SCRATCH_BYTES bytes that is part of the library image itself: every GPU that loads the library
 * holds that block until the process exits.  This call allocates and frees nothing, directly or through any
 * library.
 *
 * Same arguments, layouts and results as sfda_forward, without workspace.  Restrictions:
 *  - only the shapes of the tensor-core path (bf16, d_k = d_v = 128, chunk = 64; others need no workspace with
 *    sfda_forward in the first place) -> SFDA_ERR_UNSUPPORTED otherwise;
 *  - it runs on the kernel's minimum scratch (the status block), so without the time slicing sfda_forward does
 *    with a full workspace; a kernel whose minimum exceeded SFDA_STATIC_SCRATCH_BYTES would be refused with
 *    SFDA_ERR_WORKSPACE;
 *  - the first call on each device looks up the block's device address (with that device current); make that
 *    first call before any stream capture begins;
 *  - all calls on a device share the one block, which still holds what the previous call left there: this
 *    call clears the status word on `stream` before the kernel, and two calls whose work overlaps on the GPU
 *    (different streams) race on it.  Calls on one stream are safe.
 * sfda_noalloc_status is the counterpart of sfda_workspace_status for that block (synchronises `stream`).
 */
#define SFDA_STATIC_SCRATCH_BYTES 256
SFDA_API int sfda_forward_noalloc(const void *q, const void *k, const void *v,
                                  const float *alpha, const float *theta, const float *beta,
                                  const float *S0, void *o, void *o_im, float *S_T,
                                  int B, int T, int H, int d_k, int d_v, int chunk, int dtype,
                                  void *stream);
SFDA_API int sfda_noalloc_status(void *stream, uint32_t *detail);

/*
 * Same computation forced onto the fp32 CUDA-core path for any dtype (the
 * reference path of this library; used to cross-check the tensor-core path).
 * Needs no workspace.
 */
SFDA_API int sfda_forward_simt(const void *q, const void *k, const void *v,
                      const float *alpha, const float *theta, const float *beta,
                      const float *S0, void *o, void *o_im, float *S_T,
                      int B, int T, int H, int d_k, int d_v, int chunk, int dtype,
                      void *stream);

/*
 * Per-chunk factors of P = A_C ... A_1 = Gamma - Y M W^* in the convention of
 * Theorem "Constructive left-to-right chunk-WY recursion" with u_t = beta_t k_t,
 * r_t = Lambda_t^* k_t (Cor. "SFDA admits exact constructive block-WY products"):
 *
 *  Gamma [B][H][NC][m][2]       gamma_C = prod_t lambda_t          (Re, Im)
 *  Y     [B][H][NC][m][C][2]    Y[:,t] = (gamma_C / gamma_t) beta_t k_t
 *  M     [B][H][NC][C][C][2]    unit lower triangular
 *  W     [B][H][NC][m][C][2]    W[:,t] = conj(gamma_t) k_t
 *  phase_turns [B][T][H][m] uint32, or NULL: the chunk-local inclusive prefix sum,
 *         modulo 2^32, of  rint((double)theta * 2^32 / (2 pi)).  This kernel and the
 *         fp32 forward derive gamma's angle from these integers; the tensor-core
 *         forward sums a single-precision conversion instead (see sfda_forward_phase).
 *
 * NC = ceil(T / chunk), C = chunk.  Columns (and rows of M) of padded tail tokens
 * are those of neutral tokens (zero columns in Y and W, identity rows in M).
 * Any of Gamma, Y, M, W may be NULL to skip that output.  fp32 arithmetic.
 *
 * chunk in {16, 32, 64, 128, 256}.  The factors of a chunk of 128 or 256 tokens are
 * composed exactly out of those of its 64-token tiles, one tile appended per launch
 * (block form of Eq. "constructive-M": appending tile b to a prefix p gives Gamma =
 * Gamma_b Gamma_p, Y = [Gamma_b Y_p | Y_b], W = [W_p | Gamma_p^* W_b], block row b of
 * M = -M_b (W_b^* Y_p) M_p); the tiles' Gamma wait inside M meanwhile, so with
 * chunk > 64 all of Gamma, Y, M, W are required (SFDA_ERR_NULL otherwise).
 */
SFDA_API int sfda_chunk_factors(const void *k, const float *alpha, const float *theta, const float *beta,
                       float *Gamma, float *Y, float *M, float *W, uint32_t *phase_turns,
                       int B, int T, int H, int d_k, int chunk, int dtype, void *stream);

/*
 * One-token recurrent decode: one application of Eq. "sfda" followed by
 * o = S^* q, for B*H independent states, updating S in place.
 *
 *  q, k [B][H][d_k] dtype     v [B][H][d_v] dtype
 *  alpha, theta [B][H][m] float     beta [B][H] float
 *  S [B][H][d_k][d_v] float, read and overwritten
 *  o [B][H][d_v] dtype;  o_im same shape or NULL
 */
SFDA_API int sfda_step(const void *q, const void *k, const void *v,
              const float *alpha, const float *theta, const float *beta,
              float *S, void *o, void *o_im,
              int B, int H, int d_k, int d_v, int dtype, void *stream);

/*
 * sfda_step on the raw inputs of the stable parameterisation (see sfda_frontend for the map, the scalars'
 * ranges and SFDA_ERR_VALUE): a_raw, b_raw [B][H][m], c_raw [B][H], k_raw [B][H][d_k] take the place of alpha,
 * theta, beta, k; the map is applied inside the decode kernel (accurate exp / tanh / sqrt, fp32), nothing else
 * changes.  With eps = 0 a zero key stays zero.
 */
SFDA_API int sfda_step_fused(const void *q, const void *k_raw, const void *v,
                             const float *a_raw, const float *b_raw, const float *c_raw,
                             float alpha_min, float alpha_max, float theta_max, float eps,
                             float *S, void *o, void *o_im,
                             int B, int H, int d_k, int d_v, int dtype, void *stream);

/*
 * One decode step of the write-decoupled variant (Section 3, paragraph "Write-decoupled variant",
 * Eq. "sfda-decoupled-main"):
 *
 *     S <- (I - eta k k^*) Lambda S + beta r v^*,        o = S^* q,
 *
 * erase direction and strength (k, eta) separate from write direction and strength (r, beta); r = k, eta = beta is
 * sfda_step.  Arguments as sfda_step plus r [B][H][d_k] dtype and eta [B][H] float.
 *
 * sfda_forward_decoupled runs the same variant over whole sequences: arguments, layouts and results as
 * sfda_forward (no chunk, no workspace) plus r [B][T][H][d_k] dtype and eta [B][T][H] float; token by token in
 * fp32 on the CUDA cores, a reference path.  (The chunk-WY kernels of this library compute the tied model only:
 * with a separate write direction a chunk needs a second rotated operand tile, two more Gram blocks and one more
 * product.)
 */
SFDA_API int sfda_forward_decoupled(const void *q, const void *k, const void *r, const void *v,
                                    const float *alpha, const float *theta, const float *eta, const float *beta,
                                    const float *S0, void *o, void *o_im, float *S_T,
                                    int B, int T, int H, int d_k, int d_v, int dtype, void *stream);
SFDA_API int sfda_step_decoupled(const void *q, const void *k, const void *r, const void *v,
                                 const float *alpha, const float *theta, const float *eta, const float *beta,
                                 float *S, void *o, void *o_im,
                                 int B, int H, int d_k, int d_v, int dtype, void *stream);

/*
 * The layer in real coordinates with aligned 2 x 2 orthogonal control blocks (Eq. "intro-sfda-real"; Theorem
 * "Dihedral phase-orientation memory" and the remark after it):
 *
 *     S <- (I - eta P) U D S + beta r v^T,   U D = direct sum of alpha_j R(theta_j) F^{flip_j},   F = diag(1, -1),
 *
 * on the row pairs (2j, 2j+1) of S.  flip [B][T][H][m] (sfda_step_blocks: [B][H][m]) holds one byte per block,
 * zero = rotation only, non-zero = reflect then rotate; NULL means no reflections.  erase selects P:
 * SFDA_ERASE_COMPLEX, the realification k k^T + (Jk)(Jk)^T of the complex k k^* (with flip = NULL this is
 * sfda_forward_decoupled), or SFDA_ERASE_REAL, the real rank-one k k^T on R^{2m} that Eq. "intro-sfda-real"
 * writes.  o = S^T q and o_im = -S^T (Jq), J(x, y) = (-y, x) per pair (Re and Im of S^* q).  Other arguments,
 * layouts, dtypes and errors as sfda_forward_decoupled / sfda_step_decoupled; erase outside the two values gives
 * SFDA_ERR_VALUE.  Token by token in fp32 on the CUDA cores: reference paths, as for the write-decoupled variant.
 */
enum { SFDA_ERASE_COMPLEX = 0, SFDA_ERASE_REAL = 1 };
SFDA_API int sfda_forward_blocks(const void *q, const void *k, const void *r, const void *v,
                                 const float *alpha, const float *theta, const uint8_t *flip,
                                 const float *eta, const float *beta,
                                 const float *S0, void *o, void *o_im, float *S_T,
                                 int B, int T, int H, int d_k, int d_v, int dtype, int erase, void *stream);
SFDA_API int sfda_step_blocks(const void *q, const void *k, const void *r, const void *v,
                              const float *alpha, const float *theta, const uint8_t *flip,
                              const float *eta, const float *beta,
                              float *S, void *o, void *o_im,
                              int B, int H, int d_k, int d_v, int dtype, int erase, void *stream);

/*
 * Host-buffer forward: the call a user with data in host memory makes.  Copies the
 * inputs from HOST memory (pinned for asynchronous copies) into `arena`, runs
 * sfda_forward there and copies o (and o_im, S_T when not NULL) back to HOST
 * memory.  The batch is cut into up to 8 pieces that go up, are computed and come
 * down overlapped: the kernels run on `stream`, the copies on two streams the
 * library creates per device on the first such call (the only resources it ever
 * creates) and chains to `stream` with events; work enqueued on `stream` before the
 * call precedes all of it, and `stream` is finished only when the last download is.
 * Host pointers: q, k, v, alpha, theta, beta,
 * S0, o, o_im, S_T.  Device pointer: arena, at least sfda_forward_host_arena_bytes
 * bytes, 256-byte aligned, clobbered.  bytes_h2d / bytes_d2h (host, may be NULL)
 * receive the bytes copied in each direction.
 */
SFDA_API size_t sfda_forward_host_arena_bytes(int B, int T, int H, int d_k, int d_v, int chunk, int dtype,
                                     int want_o_im, int have_S0, int want_S_T);
SFDA_API int sfda_forward_host(const void *q, const void *k, const void *v,
                      const float *alpha, const float *theta, const float *beta,
                      const float *S0, void *o, void *o_im, float *S_T,
                      int B, int T, int H, int d_k, int d_v, int chunk, int dtype,
                      void *arena, size_t arena_bytes, void *stream,
                      size_t *bytes_h2d, size_t *bytes_d2h);

/*
 * Stable parameterisation (Section 3, paragraph "Stable parameterization", Eqs. "param-alpha", "param-theta",
 * "param-beta", "param-key"): from unconstrained inputs,
 *
 *     alpha = alpha_min + (alpha_max - alpha_min) * sigmoid(a_raw)
 *     theta = theta_max * tanh(b_raw)
 *     beta  = sigmoid(c_raw)
 *     k     = k_raw / (|k_raw|_2 + eps)          (norm over the d_k real channels of a token and head)
 *
 * which gives alpha in [alpha_min, alpha_max], |theta| <= theta_max, beta in [0, 1] and |k| <= 1: the
 * preconditions of Prop. "Basic numerical stability".
 *
 *  a_raw, b_raw [B][T][H][m] float     c_raw [B][T][H] float     k_raw [B][T][H][d_k] dtype
 *  alpha, theta [B][T][H][m] float     beta  [B][T][H] float     k     [B][T][H][d_k] dtype
 *
 * Every output may alias the input it is computed from (in-place use).  d_k in {64, 128}.
 * Scalars: 0 <= alpha_min <= alpha_max <= 1, theta_max >= 0 and finite, eps >= 0 and finite; anything else is
 * SFDA_ERR_VALUE.  With eps = 0 a zero key stays zero (no 0/0).  fp32 arithmetic.
 */
SFDA_API int sfda_frontend(const float *a_raw, const float *b_raw, const float *c_raw, const void *k_raw,
                           float alpha_min, float alpha_max, float theta_max, float eps,
                           float *alpha, float *theta, float *beta, void *k,
                           int B, int T, int H, int d_k, int dtype, void *stream);

/*
 * The derivative of sfda_frontend: with the gradients of a loss with respect to alpha, theta, beta, k (for instance
 * dalpha, dtheta, dbeta, dk of sfda_backward), its gradients with respect to the raw inputs,
 *
 *     da = dalpha (alpha_max - alpha_min) sigmoid(a_raw) (1 - sigmoid(a_raw))
 *     db = dtheta theta_max (1 - tanh(b_raw)^2)
 *     dc = dbeta sigmoid(c_raw) (1 - sigmoid(c_raw))
 *     dk_raw = s dk - s^2 (dk . k_raw) k_raw / |k_raw|,     s = 1 / (|k_raw| + eps)      (a zero key: s dk)
 *
 * Layouts, dtypes, scalars and errors as sfda_frontend; dalpha, dtheta, da, db like alpha; dbeta, dc like beta;
 * dk, dk_raw like k.  Every output may alias the gradient it is computed from.  fp32 arithmetic, one launch.
 */
SFDA_API int sfda_frontend_backward(const float *a_raw, const float *b_raw, const float *c_raw, const void *k_raw,
                                    float alpha_min, float alpha_max, float theta_max, float eps,
                                    const float *dalpha, const float *dtheta, const float *dbeta, const void *dk,
                                    float *da, float *db, float *dc, void *dk_raw,
                                    int B, int T, int H, int d_k, int dtype, void *stream);

/*
 * sfda_forward on the raw inputs: the stable parameterisation above followed by the chunkwise forward, without
 * the caller ever holding alpha, theta, beta or the normalised key.
 *
 * Arguments as sfda_forward, with a_raw, b_raw, c_raw, k_raw in place of alpha, theta, beta, k, and the four
 * scalars of sfda_frontend (same ranges, SFDA_ERR_VALUE otherwise).
 *
 * On the tensor-core path (bf16, d_k = d_v = 128, chunk = 64) the map is applied inside the kernel and the four
 * arrays are never written: alpha, theta and beta are transformed in the operand preparation (fast exponential
 * and reciprocal, 2 ulp each); the key is never divided at all, because the recurrence on k = s k_raw,
 * s = 1 / (|k_raw| + eps), is the recurrence on k_raw with beta s^2 for beta and v / s for v (Eq. "sfda"), and
 * |k_raw|^2 is read off the diagonal of the chunk's Gram matrix, i.e. from the bf16 operands (relative error of
 * s about 2e-4).  |k_raw| + eps below 1e-18 is treated as 1e-18; |k_raw|^2 must be finite in fp32.  The workspace
 * is the one of sfda_forward.  Other shapes run sfda_frontend into the workspace and the CUDA-core forward from
 * there.  sfda_forward_fused_workspace_bytes gives the size for full speed in
 * both cases (the tensor-core path again runs with as little as 256 bytes; the other shapes need it all).
 */
SFDA_API size_t sfda_forward_fused_workspace_bytes(int B, int T, int H, int d_k, int d_v, int chunk, int dtype);
SFDA_API int sfda_forward_fused(const void *q, const void *k_raw, const void *v,
                                const float *a_raw, const float *b_raw, const float *c_raw,
                                float alpha_min, float alpha_max, float theta_max, float eps,
                                const float *S0, void *o, void *o_im, float *S_T,
                                int B, int T, int H, int d_k, int d_v, int chunk, int dtype,
                                void *workspace, size_t workspace_bytes, void *stream);

/*
 * Backward pass: the gradients of a real loss L through the recurrence (Eq. "sfda") and o_t = S_t^* q_t, given
 * the cotangents of the outputs.  (The paper names the backward pass only in its kernel benchmark protocol,
 * App. E; what it computes is the adjoint of Eq. "sfda".)
 *
 *  inputs as sfda_forward:  q, k [B][T][H][d_k] dtype, v [B][T][H][d_v] dtype, alpha, theta [B][T][H][m] float,
 *                           beta [B][T][H] float, S0 [B][H][d_k][d_v] float or NULL
 *  cotangents:  d_o    [B][T][H][d_v] dtype   dL/d Re(S_t^* q_t)
 *               d_o_im same shape or NULL     dL/d Im(S_t^* q_t)  (NULL: zero)
 *               dS_T   [B][H][d_k][d_v] float or NULL (zero): dL/dS_T in the state's paired-row layout
 *  gradients:   dq, dk [B][T][H][d_k] dtype (the (Re, Im) pair of a coordinate gets the gradient with respect
 *               to its two real numbers), dv [B][T][H][d_v] dtype, dalpha, dtheta [B][T][H][m] float,
 *               dbeta [B][T][H] float, dS0 [B][H][d_k][d_v] float.  All are required and overwritten.
 *  workspace:   sfda_backward_workspace_bytes(...) bytes of device scratch (per (batch, head) pair the state at the
 *               start of every 64 tokens and the 64 states of one such segment; with few sequences also fp32
 *               shares of dq, dk, dalpha, dtheta, dbeta per block of value columns); clobbered.
 *
 * d_k, d_v in {64, 128}; no chunk argument (the derivative does not depend on the chunking).  fp32 arithmetic on
 * the CUDA cores, token by token: a first correct path, not a fast one.  One CTA per (batch, head) pair; when
 * B * H is at most half (a quarter) of the 148 SMs of a B200, the value columns -- which never interact -- are split
 * into blocks of 64 (32) with a CTA each, and a second kernel adds the blocks' shares of the sums over the
 * columns in a fixed order.  The result is deterministic either way.
 */
SFDA_API size_t sfda_backward_workspace_bytes(int B, int T, int H, int d_k, int d_v, int dtype);
SFDA_API int sfda_backward(const void *q, const void *k, const void *v,
                           const float *alpha, const float *theta, const float *beta, const float *S0,
                           const void *d_o, const void *d_o_im, const float *dS_T,
                           void *dq, void *dk, void *dv, float *dalpha, float *dtheta, float *dbeta, float *dS0,
                           int B, int T, int H, int d_k, int d_v, int dtype,
                           void *workspace, size_t workspace_bytes, void *stream);

/* Number of kernels the last sfda_forward* / sfda_step / sfda_chunk_factors / sfda_frontend call of
 * this thread enqueued (host only; for launch accounting in benchmarks). */
SFDA_API int sfda_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SFDA_H */
