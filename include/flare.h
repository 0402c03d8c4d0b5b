/*
 * libflare -- C ABI of the FLARE token mixer for NVIDIA B200 (sm_100a).
 *
 * The operator (paper Section 3.2): for every batch item b and head h, M latent queries attend over the N
 * tokens (encode), then the N tokens attend back over the M latents with queries and keys swapped and the
 * latent sequence as values (decode):
 *
 *     Z[b,h]  = softmax_rows(scale * Q[h] K[b,:,h]^T) V[b,:,h]        (encode equation; M x D)
 *     Y[b,:,h] = softmax_rows(scale * K[b,:,h] Q[h]^T) Z[b,h]         (decode equation; N x D)
 *
 * The paper fixes scale = 1 in both stages; it is a parameter here.  No M x N or N x N matrix is ever
 * written to memory.
 *
 * Layouts (all contiguous, row-major, innermost index last):
 *     Q_lat            [H, M, D]      dtype      latent queries, shared by all batch items
 *     K, V, Y, dY, dK, dV [B, N, H, D] dtype      token-major
 *     Z, dZ            [B, H, M, D]   float32    latent sequence
 *     lse_enc          [B, H, M]      float32    log sum_n exp(score) over valid tokens (-inf if none)
 *     lse_dec          [B, N, H]      float32    log sum_m exp(score)
 *     key_mask         [B, N]         uint8      1 = valid token, 0 = padding; NULL = all valid
 *     dQ_lat           [H, M, D]      float32    summed over the batch
 *
 * Padding (not in the paper): a masked token takes no part in the encode softmax; decode is evaluated for
 * every token.  A batch item with no valid token gets Z = 0, lse_enc = -inf.  On the tensor-core path a masked
 * token enters the products with weight exactly 0, so its rows of K and V must still hold finite numbers.
 *
 * Pointers and ownership: unless a function says "host", every pointer is a DEVICE pointer to memory owned
 * by the caller, 16-byte aligned; the library never allocates, frees or keeps them.  Calls enqueue work on
 * `stream` and return without synchronising; outputs are overwritten, never accumulated into.  Two calls may
 * run concurrently on different streams only with different workspaces.  Results are bitwise reproducible
 * for a fixed descriptor and set of requested outputs on a fixed device.
 *
 * Supported shapes: D in {4, 8, 16, 32, 64}; float32: any M >= 1; bfloat16: M a multiple of 16, 16 <= M <= 2048.
 * bfloat16 inputs are multiplied on the tensor cores with float32 accumulation (D = 8 and 4 as part of a 16-wide
 * product whose other columns meet zeros; tensors of fewer than 16 feature columns, or with D = 4 and an odd
 * number of heads, on the CUDA cores).  float16 inputs (the type the paper trains in under autocast; any M >= 1) are
 * accepted by every entry point and run on the CUDA-core kernels with float32 arithmetic: the tensor-core kernels are
 * written for bfloat16 operands, whose wider exponent the forms without a running maximum rely on.
 *
 * Every entry point returns a flare_status_t; nothing is thrown, nothing is printed.
 */
#ifndef FLARE_H_
#define FLARE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st *flare_stream_t; /* a cudaStream_t */

typedef enum {
    FLARE_OK = 0,
    FLARE_ERR_INVALID_ARG = 1,         /* null pointer, non-positive size, misaligned pointer, non-finite scale */
    FLARE_ERR_UNSUPPORTED = 2,         /* shape or dtype outside the supported set */
    FLARE_ERR_WORKSPACE_TOO_SMALL = 3, /* workspace_bytes < flare_workspace_bytes(desc, op) */
    FLARE_ERR_ARCH = 4,                /* current device is not compute capability 10.x */
    FLARE_ERR_CUDA = 5,                /* a CUDA call or launch failed; flare_last_cuda_error() has the text */
    FLARE_ERR_TIMEOUT = 6              /* a bounded device-side wait gave up (reported by flare_check) */
} flare_status_t;

enum { FLARE_DTYPE_F32 = 0, FLARE_DTYPE_BF16 = 1, FLARE_DTYPE_F16 = 2 };
enum { FLARE_OP_ENCODE = 0, FLARE_OP_DECODE = 1, FLARE_OP_FORWARD = 2, FLARE_OP_BACKWARD = 3, FLARE_OP_SPECTRAL = 4 };

typedef struct {
    int32_t B, H, N, M, D; /* batch, heads, tokens, latents per head, head width */
    int32_t dtype;         /* FLARE_DTYPE_* : element type of Q_lat, K, V, Y, dY, dK, dV */
    float scale;           /* multiplies every q.k score; the paper uses 1.0f */
} flare_desc_t;

/* Library version: major * 10000 + minor * 100 + patch. */
int flare_version(void);

/* Static text for a status code (never NULL). */
const char *flare_status_string(int status);

/* Text of the last CUDA error seen by this thread inside the library ("" if none).  Host pointer. */
const char *flare_last_cuda_error(void);

/*
 * Bytes of scratch `workspace` the given operation needs for `desc` on the current device (0 for an invalid
 * or unsupported descriptor).  Encode writes per-split partial results (running maximum, sum and
 * un-normalised latent rows) there: O(splits * B * H * M * (D + 2)) floats, never anything of size N x M.
 * The forward over more than 512 bfloat16 latents decodes them in ranges of 256 and adds one float32 row and
 * one log-sum-exp per token, head and range: ceil(M / 256) * B * N * H * (D + 1) floats.
 */
size_t flare_workspace_bytes(const flare_desc_t *desc, int op);

/* Number of partial results per (b, h, latent) that encode produces and the merge step combines. */
int flare_encode_partials(const flare_desc_t *desc);

/*
 * Number of kernels one call of the given operation launches for `desc` on the current device (0 for an invalid
 * descriptor): e.g. encode, merge and decode for a forward; more where latents are worked off in ranges.
 */
int flare_launch_count(const flare_desc_t *desc, int op);

/*
 * Encode (Section 3.2, encode equation; per-latent sum of the design-principles appendix):
 * Z and, if lse_enc != NULL, lse_enc.  Asking for lse_enc marks a forward whose Z will be differentiated through:
 * for bfloat16 inputs the softmax weights then enter the value contraction as two bfloat16 halves (Z within about
 * 1e-4 of its RMS instead of 4e-3, about a sixth more time in this stage), because the backward magnifies the error
 * of Z several times.  Split over N: every CTA keeps a running maximum and sum per latent
 * (online softmax) over its token range; a second kernel merges the splits by log-sum-exp.
 */
int flare_encode(const flare_desc_t *desc, const void *Q_lat, const void *K, const void *V,
                 const uint8_t *key_mask, float *Z, float *lse_enc, void *workspace, size_t workspace_bytes,
                 flare_stream_t stream);

/*
 * Decode (Section 3.2, decode equation; per-token sum of the design-principles appendix):
 * Y and, if lse_dec != NULL, lse_dec, from K, Q_lat and a latent sequence Z.
 * workspace: flare_workspace_bytes(desc, FLARE_OP_DECODE) bytes, or NULL.  Without a workspace the call still
 * works, but it has nowhere to keep a flag word or partial rows: bfloat16 inputs then always take the exact form
 * of the kernel (see flare_set_path), more than 512 bfloat16 latents run on the CUDA cores, and a bounded wait
 * that gives up is not reported.
 */
int flare_decode(const flare_desc_t *desc, const void *Q_lat, const void *K, const float *Z, void *Y,
                 float *lse_dec, void *workspace, size_t workspace_bytes, flare_stream_t stream);

/*
 * Which form of the bfloat16 tensor-core forward kernels runs (process-wide; the paper has no counterpart).
 * Both stages are softmaxes, and a softmax is usually stabilised by subtracting the row maximum before every
 * exponential (the exact forms: a running maximum in encode, a first pass over the scores in decode).  The fast
 * forms skip that: float32 and bfloat16 hold 2^x for |x| < 126, so exp(score) can be formed as it stands while
 * every |scale * q.k| stays below 96 binades (66.5 in natural units).  They check the sufficient condition
 * |q| |k| scale log2(e) <= 96 on every key row they load, and raise a flag in the workspace header if it fails;
 * the exact form is launched right behind and exits at once unless the flag is up, in which case it redoes the
 * stage.  Results of the two forms agree within the forward's error bound, not bit for bit.
 *   FLARE_PATH_AUTO   (default) fast forms for problems large enough to hide the extra launches
 *   FLARE_PATH_EXACT  always the exact forms
 *   FLARE_PATH_FAST   fast forms wherever the tensor-core kernels run
 */
enum { FLARE_PATH_AUTO = 0, FLARE_PATH_EXACT = 1, FLARE_PATH_FAST = 2 };
int flare_set_path(int path);

/*
 * The whole mixer (the paper's two-call listing in Section 3.2): encode, merge, decode on one stream.
 * Z, lse_enc, lse_dec may each be NULL; a NULL Z lives in the workspace.
 */
int flare_forward(const flare_desc_t *desc, const void *Q_lat, const void *K, const void *V,
                  const uint8_t *key_mask, void *Y, float *Z, float *lse_enc, float *lse_dec, void *workspace,
                  size_t workspace_bytes, flare_stream_t stream);

/*
 * Backward of flare_forward.  The paper times a backward pass but does not write it out; this is the chain
 * rule applied to the two equations above (W_enc, W_dec the two softmax matrices, recomputed tile by tile):
 *     dZ = W_dec^T dY;  dV = W_enc^T dZ;
 *     dS[m,n] = W_dec[n,m] (dY_n.Z_m - dY_n.Y_n) + W_enc[m,n] (dZ_m.V_n - dZ_m.Z_m);
 *     dQ_lat = scale * sum_b dS K;  dK = scale * dS^T Q_lat.
 * Z, lse_enc, lse_dec are the ones flare_forward wrote; Y is its output (part of the saved set; the present
 * kernels rebuild dY_n.Y_n = sum_m W_dec[n,m] (dY_n.Z_m) in float32 instead of reading the rounded Y, which
 * is markedly more accurate where the latent rows a token mixes are nearly equal).
 * bfloat16 inputs run all three passes (dZ; dK, dV; dQ_lat) on the tensor cores (the last two for D <= 32), with
 * every rounded factor of a cancelling sum carried as two bfloat16 halves; float32 inputs run on the CUDA cores.
 * dQ_lat, dK, dV are overwritten.  Workspace: flare_workspace_bytes(desc, FLARE_OP_BACKWARD) bytes holding dZ,
 * per-split partial sums of dZ and dQ_lat, one float per (b, n, h), and, beyond 512 bfloat16 latents (256 at
 * D = 32), float32 sums of the rows of dK and dV; nothing of size N x M.
 */
int flare_backward(const flare_desc_t *desc, const void *Q_lat, const void *K, const void *V,
                   const uint8_t *key_mask, const void *Y, const void *dY, const float *Z, const float *lse_enc,
                   const float *lse_dec, float *dQ_lat, void *dK, void *dV, void *workspace,
                   size_t workspace_bytes, flare_stream_t stream);

/*
 * flare_forward for callers whose tensors live in HOST memory (pinned memory makes the copies asynchronous).
 * Copies Q_lat, K, V (and key_mask if not NULL) from the host pointers into the caller's device staging
 * buffers dQ_lat, dK, dV, dmask, runs flare_forward into dY, and copies Y back to hY, all on `stream`.
 * hQ_lat, hK, hV, hmask, hY are host pointers; everything else is a device pointer.
 */
int flare_forward_host(const flare_desc_t *desc, const void *hQ_lat, const void *hK, const void *hV,
                       const uint8_t *hmask, void *hY, void *dQ_lat, void *dK, void *dV, uint8_t *dmask, void *dY,
                       void *workspace, size_t workspace_bytes, flare_stream_t stream);

/*
 * flare_encode without a caller-provided workspace.  (The paper has no counterpart: this exists for callers
 * that are not allowed to allocate device memory at the point where they need the operator -- code running
 * inside a memory-budgeted plugin or a real-time loop, hosts whose allocator is owned by another runtime and
 * may not be re-entered, or late-bound callers that only hold the input and output tensors they were handed.)
 *
 * The per-split partial results go to a fixed array of FLARE_STATIC_SCRATCH_BYTES that is part of the
 * library's device image: every GPU on which the library is loaded holds that much memory until the process
 * exits, whether or not this function is ever called.  Nothing is allocated or freed by the call.
 *
 * Limits and rules:
 *   - flare_workspace_bytes(desc, FLARE_OP_ENCODE) must not exceed FLARE_STATIC_SCRATCH_BYTES; a larger
 *     problem is refused with FLARE_ERR_WORKSPACE_TOO_SMALL before any work is queued (flare_last_cuda_error()
 *     then names both sizes).  Use flare_encode with your own workspace for those.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left; the function
 *     clears the part that must start at zero itself.  Two calls whose GPU work overlaps in time (different
 *     streams, or different host threads) race on it and produce garbage: serialise them.
 *   - The first call on each device looks up the array's device address (with that device current) and caches
 *     it.  Make that first call outside any stream capture.
 * Arguments, outputs and status codes are otherwise those of flare_encode.
 */
#define FLARE_STATIC_SCRATCH_BYTES (8u << 20)
int flare_encode_static_scratch(const flare_desc_t *desc, const void *Q_lat, const void *K, const void *V,
                                const uint8_t *key_mask, float *Z, float *lse_enc, flare_stream_t stream);

/*
 * Two variants of the mixer that the paper discusses and sets aside (both as entry points of their own; the plain
 * calls above are the method as the paper uses it):
 *   shared_latents != 0   all heads use ONE latent sequence (the "shared vs independent latents" ablation of the
 *                         paper's ablation appendix): Q_enc, Q_dec, dQ_enc, dQ_dec are [M, D] instead of [H, M, D].
 *   Q_dec != NULL         separate latent queries for the two stages (the "asymmetric" remark of the
 *                         design-principles appendix): encode scores are Q_enc K^T, decode scores K Q_dec^T.
 *                         NULL means the symmetric operator (Q_dec = Q_enc); dQ_dec must be NULL exactly then.
 * Both are built from the kernels of the plain calls: a shared sequence is copied out to all heads in the workspace
 * and its gradient summed over the heads; with separate queries the backward runs its two per-token passes twice,
 * once per set of queries, each time with the other stage's weights switched off (its log-sum-exp rows set to
 * +infinity), and adds the two parts of dK.  Workspace: flare_variant_workspace_bytes.  Everything else as in
 * flare_forward / flare_backward.
 */
size_t flare_variant_workspace_bytes(const flare_desc_t *desc, int op, int shared_latents, int separate_decode_queries);
int flare_forward_variant(const flare_desc_t *desc, int shared_latents, const void *Q_enc, const void *Q_dec, const void *K,
                          const void *V, const uint8_t *key_mask, void *Y, float *Z, float *lse_enc, float *lse_dec,
                          void *workspace, size_t workspace_bytes, flare_stream_t stream);
int flare_backward_variant(const flare_desc_t *desc, int shared_latents, const void *Q_enc, const void *Q_dec, const void *K,
                           const void *V, const uint8_t *key_mask, const void *Y, const void *dY, const float *Z,
                           const float *lse_enc, const float *lse_dec, float *dQ_enc, float *dQ_dec, void *dK, void *dV,
                           void *workspace, size_t workspace_bytes, flare_stream_t stream);

/*
 * Spectral analysis of the mixing matrix in O(M^2 N) (spectral-analysis appendix, Algorithm 1).  Per (b, h) the
 * N x N mixing matrix W = W_dec W_enc has rank at most M, and its non-zero eigenvalues are those of the M x M
 * matrix G = J J^T, J = L_M^{1/2} A L_N^{1/2}, A = exp(scale Q K^T), L_M = diag(1 / row sums of A),
 * L_N = diag(1 / column sums of A) (the appendix once writes "J^T J" for the M x M matrix; the algorithm's steps
 * fix it as J J^T).  flare_spectral_gram forms G [B, H, M, M] float32 from Q_lat, K and the two log-sum-exp
 * outputs of flare_forward on the same Q_lat and K (lse_enc = log row sums, lse_dec = log column sums, both of
 * all tokens: no key mask), J[m,n] = exp(score - lse_enc[m]/2 - lse_dec[n]/2): one pass over the tokens, nothing of
 * size M x N is written.  bfloat16 inputs with D in {16, 32} run on the tensor cores: M <= 128 in one pass, larger M
 * (a multiple of 64, up to 1024) as one pass per pair of 64-latent blocks; everything else on the CUDA cores.
 * Workspace: flare_workspace_bytes(desc, FLARE_OP_SPECTRAL).
 */
int flare_spectral_gram(const flare_desc_t *desc, const void *Q_lat, const void *K, const float *lse_enc,
                        const float *lse_dec, float *G, void *workspace, size_t workspace_bytes, flare_stream_t stream);

/*
 * The M x M symmetric eigenproblems of Algorithm 1 (its step "U Sigma^2 U^T = J J^T"), O(M^3) each and off the hot
 * path: cyclic Jacobi rotations, one thread block per matrix.  G [matrices, M, M] float32 is destroyed;
 * eigenvalues [matrices, M] come out in descending order; U [matrices, M, M] (may be NULL) gets the eigenvectors as
 * columns, in the same order.  sweeps <= 0 means the default (12).  M <= 1024.  (The eigenvectors of W itself,
 * L_N^{1/2} J^T U Sigma^{-1}, are N x M and are not formed.)
 */
int flare_spectral_eig(int32_t matrices, int32_t M, float *G, float *eigenvalues, float *U, int32_t sweeps,
                       flare_stream_t stream);

/*
 * Instruction-level measurements behind the kernels' design (the paper has no counterpart), so that the figures the
 * documentation quotes can be re-taken on the GPU at hand.  `which`:
 *   0, 1, 2   exponentials per clock per SM of the softmax loop as the sixteen softmax warps of a forward kernel run it
 *             (32 scores from tensor memory, 16 columns of packed weights back): 0 = with a running maximum and sum,
 *             special-function unit only; 1 = without a maximum, special-function unit only; 2 = without a maximum,
 *             seven pairs of columns in sixteen by the polynomial on the FMA pipe (what the fast forms run);
 *   3, 4      cycles the issuing thread is held by one unit's tensor-core instructions (two value MMAs, one score MMA,
 *             one commit), and cycles from the commit to the flip of its barrier.
 * scratch: at least 4096 bytes of device memory.  *result is a HOST double.  Synchronises the stream.
 */
int flare_microbench(int which, int iters, void *scratch, size_t scratch_bytes, double *result, flare_stream_t stream);

/*
 * After the stream has been synchronised: FLARE_OK, or FLARE_ERR_TIMEOUT if a kernel of the last call that
 * used `workspace` gave up on a bounded wait (its outputs are then undefined).  Reads one word from the
 * workspace with a blocking copy.  workspace = NULL means the built-in scratch array of
 * flare_encode_static_scratch on the current device.
 */
int flare_check(const void *workspace, flare_stream_t stream);

/*
 * Self-test of the bounded device-side waits (the paper has no counterpart).  Every wait inside the kernels
 * (on a TMA load, on a tensor-core result) gives up after a time budget, records a code in the first word of
 * the workspace and lets the kernel finish normally, so that a fault in the pipeline shows up as
 * FLARE_ERR_TIMEOUT from flare_check instead of a hung GPU.  This call runs that mechanism in isolation: a
 * one-block kernel waits for `budget_ns` nanoseconds (clamped to [1 us, 0.1 s]) on a barrier that nothing will
 * ever complete, gives up, and records its code exactly as the other kernels do; flare_check(workspace) must
 * then report FLARE_ERR_TIMEOUT, and the next ordinary call on the same workspace clears it.
 * workspace: at least 256 bytes of device memory.
 */
int flare_selftest_wait(void *workspace, uint64_t budget_ns, flare_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* FLARE_H_ */
