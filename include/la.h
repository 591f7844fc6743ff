/*
 * la.h -- C ABI of the linear-attention library for NVIDIA B200 (sm_100a).
 *
 * The library computes the attention core of "Transformers are RNNs"
 * (Katharopoulos et al., 2020): attention with the kernel feature map
 * phi(x) = elu(x) + 1 in its non-causal form, its causal form with the running
 * state S_i = sum_{j<=i} phi(K_j) V_j^T and normaliser Z_i = sum_{j<=i} phi(K_j),
 * forward and backward, and the one-token recurrent (RNN) step.
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 *  - Every data pointer is DEVICE memory owned by the caller.  The library
 *    allocates and frees nothing; scratch memory is passed in as `ws` and sized
 *    with la_workspace_bytes().  `ws` contents are undefined on return.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *    Every call only enqueues work on it and returns without synchronising.
 *  - Tensors are row-major and contiguous, one (batch, head) pair after another:
 *        Q, K, dQ, dK : [B, H, N, D]        V, O, G, dV : [B, H, N, M]
 *        den          : [B, H, N]  fp32     S : [B, H, D, M] fp32    Z : [B, H, D] fp32
 *    Q, K, V, O, G and the gradients have the I/O type la_problem.dtype (fp32
 *    or bf16, round-to-nearest-even on output); states, normalisers and all
 *    accumulation are fp32.  Data pointers must be 16-byte aligned.
 *  - Outputs must not alias inputs (S and Z of la_recurrent_step are in-out).
 *  - Supported sizes: D and M multiples of 8 in [8, 128]; B, H >= 1; N >= 0
 *    (N == 0 is a successful no-op).  bf16 problems with D = M in {32, 64} run
 *    on the tensor-core kernels (any N: a last chunk of fewer than 128
 *    positions is handled as padding), everything else on the general
 *    fp32-arithmetic kernels; results agree within the rounding of the I/O type.
 *  - Return value: LA_OK (0) or a negative la_status.  All argument checks run
 *    on the host before anything is enqueued; a failed check enqueues nothing.
 *    The library never aborts, throws or traps.  la_last_error() returns a
 *    static, thread-local description of the last failure on this thread.
 */
#ifndef LA_H_
#define LA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LA_OK = 0,
    LA_ERR_INVALID_ARG = -1,    /* NULL pointer, negative size, misaligned pointer, bad enum  */
    LA_ERR_UNSUPPORTED = -2,    /* well-formed problem outside the supported sizes/types      */
    LA_ERR_WORKSPACE = -3,      /* ws is NULL or smaller than la_workspace_bytes()            */
    LA_ERR_CUDA = -4,           /* a CUDA runtime call failed (see la_last_error())           */
    LA_ERR_ARCH = -5,           /* current device is not compute capability 10.x              */
    LA_ERR_DEVICE_TIMEOUT = -6  /* a bounded device-side wait expired (reported by
                                   la_last_device_status())                                   */
} la_status;

typedef enum { LA_F32 = 0, LA_BF16 = 1 } la_dtype;

/* LA_PHI_ELU1: the library applies phi(x) = elu(x) + 1 (Eq. 7) to Q and K and
 * returns gradients with respect to the raw Q, K.  LA_PHI_IDENTITY: Q and K
 * already hold phi(Q), phi(K) (the convention of Algorithm 1); gradients are
 * with respect to those. */
typedef enum { LA_PHI_ELU1 = 0, LA_PHI_IDENTITY = 1 } la_phi;

typedef enum {
    LA_OP_LINEAR_FORWARD = 0,
    LA_OP_LINEAR_BACKWARD = 1,
    LA_OP_CAUSAL_FORWARD = 2,
    LA_OP_CAUSAL_BACKWARD = 3,
    LA_OP_CAUSAL_SAVED = 4,      /* size of the optional `saved` buffer, see la_causal_forward() */
    LA_OP_LINEAR_VARLEN_FORWARD = 5,     /* la_linear_attention_varlen()          */
    LA_OP_LINEAR_VARLEN_BACKWARD = 6,    /* la_linear_attention_varlen_backward() */
    LA_OP_LINEAR_SAVED = 7,              /* size of the optional `saved` buffer, see la_linear_attention_keep() */
    LA_OP_DECODE_LAYER = 8,              /* la_decode_layer_step()                */
    LA_OP_CAUSAL_VARLEN_FORWARD = 9,     /* la_causal_forward_varlen()            */
    LA_OP_CAUSAL_VARLEN_BACKWARD = 10    /* la_causal_backward_varlen()           */
} la_op;

typedef struct {
    int64_t B, H, N, D, M;   /* batch, heads, sequence length, query/key dim, value dim */
    int32_t dtype;           /* la_dtype of Q, K, V, O, G and the gradients             */
    int32_t phi;             /* la_phi                                                  */
    float   eps;             /* added to every denominator; the paper uses none (0)     */
} la_problem;

/*
 * Feature map, Eq. 7:  y[i] = phi(x[i]) = x[i] + 1 (x[i] > 0), exp(x[i]) otherwise;
 * with deriv != 0, y[i] = phi'(x[i]) = 1 (x[i] > 0), exp(x[i]) otherwise.
 * x, y: n elements of `dtype` (device).  y may equal x (in place).
 */
int la_feature_map(const void* x, void* y, int64_t n, int32_t dtype, int32_t deriv, void* stream);

/*
 * Degree-2 polynomial kernel (Section 3.2.1, "Feature Maps and Computational Cost"): the kernel
 * sim(a, b) = (a . b)^2 has the exact feature map phi(x) = vec(x x^T) of dimension D*D,
 *   y[r][i*D + j] = x[r][i] * x[r][j]   (0 <= i, j < D),   y[r][c] = 0 for D*D <= c < C,
 * so that phi(a) . phi(b) = (a . b)^2.  The attention calls take the mapped queries and keys with
 * phi = LA_PHI_IDENTITY and D = C (the cost O(N D^2 M) the paper quotes); the zero padding lets C
 * be the multiple of 8 they ask for.  The paper names the kernel without fixing its form: the
 * homogeneous one is taken, the one whose feature map has exactly D^2 components.
 * x: [rows, D], y: [rows, C] of `dtype` (device, 16-byte aligned; x and y must not overlap).
 * 1 <= D <= 11, D*D <= C <= 128, C a multiple of 8.  Products are formed in fp32 and rounded once.
 * The backward call turns dy = dL/dy [rows, C] into dx[r][i] = sum_j (dy[r][i*D+j] + dy[r][j*D+i]) x[r][j]
 * (fp32 sums; dx: [rows, D], must not alias x; x, dy, dx 16-byte aligned).
 */
int la_feature_map_poly2(const void* x, void* y, int64_t rows, int64_t D, int64_t C, int32_t dtype, void* stream);
int la_feature_map_poly2_backward(const void* x, const void* dy, void* dx, int64_t rows, int64_t D, int64_t C,
                                  int32_t dtype, void* stream);

/*
 * Random Fourier features for the Gaussian kernel (the feature map the paper's conclusion proposes to
 * explore; Section 3.2.1: a feature map of dimension C costs O(N C M)).  The paper gives no formula; the
 * classical paired construction is taken, with the frequencies supplied by the caller:
 *   y[r] = sqrt(2 / C) [cos(W x[r]), sin(W x[r])],   W: [C/2, D] row-major,
 * cosines in columns [0, C/2), sines in [C/2, C), so that y[r] . y[s] = (2 / C) sum_c cos(w_c . (x[r] - x[s])),
 * whose mean over w_c ~ N(0, I) is exp(-|x[r] - x[s]|^2 / 2), and |y[r]| = 1.  Apply it to Q and K and call
 * the attention entry points with phi = LA_PHI_IDENTITY and D = C.  The features have either sign: the
 * weights of Eq. 4 are then not guaranteed positive, which is the caller's concern.
 * x: [rows, D], y: [rows, C], W: [C/2, D], all bf16 (dtype LA_BF16), device, 16-byte aligned, no overlap.
 * D a multiple of 8 in [8, 64]; C = 64 or 128; 1 <= rows < 2^31.  Other shapes or LA_F32: LA_ERR_UNSUPPORTED.
 * The projection runs on the tensor cores (fp32 accumulation), sine and cosine on the special-function unit
 * after a range reduction; one rounding to bf16 on output.
 * The backward call turns dy = dL/dy [rows, C] into
 *   dx[r] = sqrt(2 / C) (-sin(W x[r]) * dy_cos[r] + cos(W x[r]) * dy_sin[r]) W        (dx: [rows, D]),
 * the inner factor being rounded to bf16 before the second product.  W is treated as a constant.
 */
int la_feature_map_rff(const void* x, const void* W, void* y, int64_t rows, int64_t D, int64_t C, int32_t dtype, void* stream);
int la_feature_map_rff_backward(const void* x, const void* W, const void* dy, void* dx, int64_t rows, int64_t D, int64_t C,
                                int32_t dtype, void* stream);

/*
 * Non-causal linear attention, Eq. 5-6:
 *   KV = sum_j phi(K_j) V_j^T,  Zs = sum_j phi(K_j)   (formed once per head),
 *   O_i = phi(Q_i)^T KV / (phi(Q_i)^T Zs + eps).
 * den (optional, may be NULL): phi(Q_i)^T Zs without eps.  KV / Zs (optional): the
 * per-head sums, [B,H,D,M] / [B,H,D] fp32.
 */
int la_linear_attention(const la_problem* p, const void* Q, const void* K, const void* V,
                        void* O, float* den, float* KV, float* Zs,
                        void* ws, size_t ws_bytes, void* stream);

/*
 * Gradient of the non-causal form for an upstream gradient G = dL/dO.  The paper
 * leaves the division to automatic differentiation; here it is absorbed by
 * running the cumulative-sum gradients of Eq. 13-15 (with full, unmasked sums)
 * on the values extended by a constant 1.  O and den are accepted for symmetry
 * with autograd-style callers and may be NULL: everything needed is recomputed.
 */
int la_linear_attention_backward(const la_problem* p, const void* Q, const void* K, const void* V,
                                 const void* O, const float* den, const void* G,
                                 void* dQ, void* dK, void* dV,
                                 void* ws, size_t ws_bytes, void* stream);

/*
 * The non-causal form on a ragged batch: sequences of different lengths padded on the right to
 * the common N of the tensors (a key-padding mask; the paper's speech data are such batches).
 * lengths: [B] int32 on the device, 4-byte aligned; values are clipped to [0, N] on the device.
 * For batch element b only positions i, j < lengths[b] exist:
 *   O_i = phi(Q_i)^T sum_{j < len} phi(K_j) V_j^T / (phi(Q_i)^T sum_{j < len} phi(K_j) + eps),
 * KV / Zs are the sums over the real positions, and O, den (and in the backward pass dQ, dK, dV)
 * are written as zeros on the padding; what Q, K, V, G hold there is never used.  Workspace:
 * la_workspace_bytes(p, LA_OP_LINEAR_VARLEN_FORWARD / _BACKWARD).  The same kernels run as for the
 * full-length calls (splits of a sequence skip the chunks that hold only padding).  Everything
 * else as for la_linear_attention() / la_linear_attention_backward().
 */
int la_linear_attention_varlen(const la_problem* p, const void* Q, const void* K, const void* V,
                               const int32_t* lengths,
                               void* O, float* den, float* KV, float* Zs,
                               void* ws, size_t ws_bytes, void* stream);
int la_linear_attention_varlen_backward(const la_problem* p, const void* Q, const void* K, const void* V,
                                        const int32_t* lengths,
                                        const void* O, const float* den, const void* G,
                                        void* dQ, void* dK, void* dV,
                                        void* ws, size_t ws_bytes, void* stream);

/*
 * The non-causal form for a training step: the forward keeps what it computed once per head, as the
 * paper's "compute KV once and reuse it" does for the queries, so that the backward pass does not form
 * the sums over the keys again.  lengths: NULL (full-length batch) or as for the _varlen calls.
 * saved (device, 16-byte aligned, la_workspace_bytes(p, LA_OP_LINEAR_SAVED) bytes, owned by the caller):
 * written by la_linear_attention_keep() (per-split sums of phi(K_j) [V_j | 1]^T; layout private to the
 * library), valid for la_linear_attention_backward_kept() with the same problem, lengths, K and V until
 * overwritten.  With saved == NULL the calls behave exactly like the plain / _varlen ones; with a saved
 * buffer the forward does not touch its workspace (ws may be NULL) and the results of both calls are the
 * same bit for bit as without.
 */
int la_linear_attention_keep(const la_problem* p, const void* Q, const void* K, const void* V,
                             const int32_t* lengths,
                             void* O, float* den, float* KV, float* Zs,
                             void* saved, size_t saved_bytes,
                             void* ws, size_t ws_bytes, void* stream);
int la_linear_attention_backward_kept(const la_problem* p, const void* Q, const void* K, const void* V,
                                      const int32_t* lengths,
                                      const void* saved, size_t saved_bytes,
                                      const void* O, const float* den, const void* G,
                                      void* dQ, void* dK, void* dV,
                                      void* ws, size_t ws_bytes, void* stream);

/*
 * Causal linear attention, Eq. 9-12 (Algorithm 1, forward, plus the normaliser):
 *   S_i = S_{i-1} + phi(K_i) V_i^T,  Z_i = Z_{i-1} + phi(K_i),  S_0 = 0, Z_0 = 0,
 *   O_i = phi(Q_i)^T S_i / (phi(Q_i)^T Z_i + eps)       (position i sees j <= i).
 * den (optional): phi(Q_i)^T Z_i without eps.  S_out / Z_out (optional): the final
 * state S_N, Z_N, which continues the sequence through la_recurrent_step().
 * saved (optional, device, 128-byte aligned, la_workspace_bytes(p, LA_OP_CAUSAL_SAVED)
 * bytes, owned by the caller): what a training step keeps for the backward pass, as the
 * paper's autograd function keeps phi(Q), phi(K): the mapped queries and keys and the
 * per-segment sums of the forward pre-pass.  Its layout is private to the library; it is
 * valid for la_causal_backward() with the same problem, Q, K and V until overwritten.  The
 * size is 0 for problems that run the general kernels (pass NULL, or any pointer).
 */
int la_causal_forward(const la_problem* p, const void* Q, const void* K, const void* V,
                      void* O, float* den, float* S_out, float* Z_out,
                      void* saved, size_t saved_bytes,
                      void* ws, size_t ws_bytes, void* stream);

/*
 * The causal form continued from a state: the recurrence of Eq. 16-20 run over the N positions of
 * this call from S_0 = S_in, Z_0 = Z_in instead of zero,
 *   O_i = phi(Q_i)^T (S_in + sum_{j<=i} phi(K_j) V_j^T) / (phi(Q_i)^T (Z_in + sum_{j<=i} phi(K_j)) + eps),
 * so that a long sequence can be processed in several calls (chunked prefill) and S_out / Z_out of
 * one call are S_in / Z_in of the next, or the state la_recurrent_step() continues from.
 * S_in [B,H,D,M] and Z_in [B,H,D]: device, fp32, 16-byte aligned, both given or both NULL (NULL:
 * the call is la_causal_forward()); they are only read and must not overlap S_out / Z_out
 * (LA_ERR_INVALID_ARG: the pieces of a sequence run concurrently and all start from S_in).  den
 * includes the Z_in term.  With N = 0 the state is copied to S_out / Z_out.  `saved` as for
 * la_causal_forward(): it is valid for la_causal_backward_from() with the same S_in, Z_in (the
 * state itself is not kept in it).  Everything else as for la_causal_forward().
 */
int la_causal_forward_from(const la_problem* p, const void* Q, const void* K, const void* V,
                           const float* S_in, const float* Z_in,
                           void* O, float* den, float* S_out, float* Z_out,
                           void* saved, size_t saved_bytes,
                           void* ws, size_t ws_bytes, void* stream);

/*
 * Gradient of the causal form in linear time and memory independent of N per
 * head, Eq. 13-15 (Algorithm 1, backward): grad phi(Q_i) uses the forward running
 * sum of phi(K_j)[V_j,1]^T, grad phi(K_i) and grad V_i the reverse running sum of
 * phi(Q_j) Gt_j^T, where Gt_j = [G_j/den_j, -(G_j.O_j)/den_j] carries the division.
 * No per-position state is stored.  G = dL/dO.  O and den may be NULL (recomputed).
 * saved (optional): the buffer a la_causal_forward() call on the same problem and inputs
 * filled.  With it the backward pass reads phi(Q), phi(K) instead of recomputing them from
 * Q and K and skips its forward pre-pass; without it (NULL) everything is recomputed.  The
 * gradients agree with the recomputing path to rounding (phi(Q)/den is rounded from the
 * saved bf16 phi(Q) instead of the fp32 value).
 */
int la_causal_backward(const la_problem* p, const void* Q, const void* K, const void* V,
                       const void* O, const float* den, const void* G,
                       const void* saved, size_t saved_bytes,
                       void* dQ, void* dK, void* dV,
                       void* ws, size_t ws_bytes, void* stream);

/*
 * One recurrent step per (batch, head) stream, Eq. 16-20 (attention part); the
 * state is updated BEFORE it is read:
 *   S += phi(k) v^T,  Z += phi(k),  out = phi(q)^T S / (phi(q)^T Z + eps).
 * q, k: [B,H,D]; v, out: [B,H,M] of p->dtype; S: [B,H,D,M], Z: [B,H,D] fp32, updated
 * in place (zero them to start a sequence).  p->N is ignored.  Needs no workspace.
 */
int la_recurrent_step(const la_problem* p, const void* q, const void* k, const void* v,
                      float* S, float* Z, void* out, void* stream);

/*
 * p->N recurrent steps per (batch, head) stream in one launch, for steps whose inputs are all known
 * beforehand (a prompt continued token by token, scoring a given continuation, several drafted
 * tokens at once): Eq. 18-20 for t = 1..N,
 *   S += phi(k_t) v_t^T,  Z += phi(k_t),  out_t = phi(q_t)^T S / (phi(q_t)^T Z + eps),
 * with the state read from and written to memory once instead of once per step.  q, k: [B,H,N,D];
 * v, out: [B,H,N,M] of p->dtype; S, Z as for la_recurrent_step(), updated in place.  The results
 * are bit-identical to N calls of la_recurrent_step() on the same inputs.  N = 0: no-op.
 * Needs no workspace.
 */
int la_recurrent_steps(const la_problem* p, const void* q, const void* k, const void* v,
                       float* S, float* Z, void* out, void* stream);

/*
 * One decode step of a whole attention sublayer: Eq. 16-20 with the projections of Eq. 2 written
 * out, for B independent streams of model width F = H * D,
 *   q = x W_Q,  k = x W_K,  v = x W_V                     (split into H heads of D = M columns)
 *   S += phi(k) v^T,  Z += phi(k),  a = phi(q)^T S / (phi(q)^T Z + eps)      (per head, update first)
 *   y = a W_O + x                                          (output projection and residual)
 * so that the token produced from y can be fed back as the next x without the caller touching q, k, v.
 * The position-wise feed-forward part f_l of Eq. 20 stays with the caller.  p: B, H, D = M = 64, dtype
 * LA_BF16, phi, eps (N ignored).  x, y: [B, F] bf16.  Wqkv: [3F, F] bf16, row-major "outputs x inputs"
 * (row r < F is column r of W_Q, rows F..2F-1 of W_K, 2F..3F-1 of W_V: the layout of a fused linear
 * layer's weight); Wo: [F, F] likewise.  S [B,H,D,M], Z [B,H,D] fp32, updated in place (zero them for a
 * new sequence).  ws: la_workspace_bytes(p, LA_OP_DECODE_LAYER) bytes (q, k, v, a as bf16: they are
 * rounded to bf16 between the three kernels).  y must not alias x.  Three launches: projection
 * (tensor cores), recurrent step, projection with the residual in its epilogue; asynchronous on
 * `stream`.  Other dtypes or head sizes: LA_ERR_UNSUPPORTED (use la_recurrent_step with your own
 * projections).
 */
int la_decode_layer_step(const la_problem* p, const void* x, const void* Wqkv, const void* Wo,
                         float* S, float* Z, void* y, void* ws, size_t ws_bytes, void* stream);

/*
 * Non-causal forward for callers that cannot allocate device memory (the paper has no
 * counterpart: this is a deployment convenience, not part of the method).
 *
 * Same computation, arguments and results as la_linear_attention(), minus `ws`: the
 * scratch for the per-split partial sums is a fixed array of LA_NOALLOC_SCRATCH_BYTES
 * inside the library's device image.  It is meant for callers that receive only input
 * and output buffers and may not call cudaMalloc or ask their framework for memory at
 * that point: plugin-style integrations, code that runs after a framework has frozen its
 * memory plan, latency-critical loops where an allocation (which can synchronise the
 * device) is not tolerable.  The price: every GPU on which the library is loaded holds
 * those LA_NOALLOC_SCRATCH_BYTES until the process exits, used or not.
 *
 *  - The call itself allocates and frees nothing, on the host or the device, and calls no
 *    allocating library routine.  It always runs the general fp32-arithmetic kernels.
 *    One caveat about the FIRST call on a device: the CUDA runtime loads a library's
 *    device code lazily, and the address look-up of that first call is where the driver
 *    may load this module and place the array in device memory.  That placement is the
 *    driver's, not a cudaMalloc, but it does take device memory at that moment; a caller
 *    under a strict budget should make one warm-up call (any small problem) while it is
 *    still allowed to grow.
 *  - Problems whose scratch need (B*H*splits*D*(M+1)*4 bytes, at most a few splits per
 *    head) exceeds the array are rejected with LA_ERR_WORKSPACE and a message naming
 *    both sizes; nothing is enqueued.
 *  - The first call on each device looks up the array's device address (with that device
 *    current) and caches it; make that first call before starting any stream capture
 *    (it is also the call the caveat above is about).
 *  - All calls on a device share the one array, which keeps the previous call's contents.
 *    Nothing in it needs clearing between calls (each call overwrites what it reads), but
 *    two calls whose kernels overlap on the GPU (different streams) race on it: run them
 *    on one stream or order them with events.
 */
#define LA_NOALLOC_SCRATCH_BYTES (8u << 20)
int la_linear_attention_noalloc(const la_problem* p, const void* Q, const void* K, const void* V,
                                void* O, float* den, float* KV, float* Zs, void* stream);

/*
 * Checked mode (no counterpart in the paper): with the environment variable LA_DEBUG=1 set when the
 * library is first used, the attention, recurrent-step and decode-layer entry points look every
 * tensor argument up with the driver before anything is enqueued (device memory of the current
 * device? does the allocation that holds it reach as far as the call reads or writes, given the
 * sizes in la_problem?) and return LA_ERR_INVALID_ARG otherwise; after enqueueing they synchronise
 * `stream` and report a bounded wait that ran out (LA_ERR_DEVICE_TIMEOUT), a refused saved buffer or
 * a CUDA error from the call itself instead of leaving it to la_last_device_status().  Under a
 * caching allocator the allocation is the allocator's block, so the span check is a lower bound on
 * strictness.  Meant for bring-up on shared GPUs, where an out-of-bounds access must not reach the
 * device; it costs a synchronisation per call and must not be used during stream capture.
 */

/* Bytes of workspace `op` needs for problem p (pure host function; 0 if none).
 * Returns 0 for invalid problems as well: the entry point reports the error. */
size_t la_workspace_bytes(const la_problem* p, int32_t op);

/* Human-readable name of a status code (static string). */
const char* la_status_string(int status);

/* Description of the last failure on the calling thread ("" if none). */
const char* la_last_error(void);

/* Synchronises `stream`, then reports whether any kernel of this library gave up
 * on a bounded wait since the last call (LA_ERR_DEVICE_TIMEOUT), or refused a saved
 * buffer written under another piece plan (LA_ERR_INVALID_ARG, see la_plan_override()),
 * and clears the flag; LA_OK otherwise.  The context stays usable either way. */
int la_last_device_status(void* stream);

/*
 * How the tensor-core causal kernels cut the sequences of problem p (a diagnostic, no counterpart
 * in the paper; host only, nothing is enqueued).  A sequence of N / 128 chunks is cut into pieces,
 * one CTA of a main kernel each, launched in the order the function reports, so that B*H*pieces
 * CTAs keep all SMs busy; every piece is cut into pre-pass parts whose sums give a piece its
 * starting state.  Writes up to `capacity` 32-bit integers to `out` (host memory) and returns how
 * many the full description has, or 0 when p does not run the tensor-core kernels, or a negative
 * status:  out = { pieces, parts,
 *                  piece_begin[0..pieces]  (chunk index; piece_begin[pieces] = N / 128),
 *                  piece_first_part[0..pieces],
 *                  part_begin[0..parts],
 *                  launch_order[0..pieces-1]  (CTA b handles piece launch_order[b / (B*H)] of
 *                                              sequence b % (B*H)) }.
 */
int la_causal_plan(const la_problem* p, int32_t* out, int capacity);

/*
 * Overrides of the automatic plans, for A/B checks and tests (no counterpart in the paper; host only).
 * causal_pieces: equal pieces per sequence in the causal kernels; causal_short: length in chunks of the
 * short middle piece (0: none); linear_splits: splits per sequence in the non-causal kernels.  -1 leaves a
 * choice automatic; la_plan_override(-1, -1, -1) restores the defaults.  The setting is process-wide and
 * read by every later call, la_workspace_bytes() and la_causal_plan() included: change it only between
 * steps, size workspaces and saved buffers after the change, and never between a forward pass that
 * fills a saved buffer and the backward pass that reads it (the backward pass notices: it computes
 * nothing and la_last_device_status() returns LA_ERR_INVALID_ARG).
 */
int la_plan_override(int32_t causal_pieces, int32_t causal_short, int32_t linear_splits);

/*
 * Gradient of the causal form continued from a state, for
 *   L = sum G . O + <dS_out, S_N> + <dZ_out, Z_N>
 * (an upstream gradient on the outputs and, optionally, on the final state: what a sequence
 * processed and differentiated in several calls needs).  Algorithm 1 (backward) with two changes:
 * the forward running sum starts from [S_in | Z_in] and the reverse running sum from
 * [dS_out | dZ_out]; what is left in the reverse sum after the sweep is the gradient of the state
 * the call started from, written to dS_in [B,H,D,M] and dZ_in [B,H,D] (fp32; either may be NULL:
 * not wanted).  S_in / Z_in: both or neither (NULL: zero state).  dS_out / dZ_out: each may be NULL
 * (zero).  All state pointers are device, fp32, 16-byte aligned; dS_in / dZ_in must not overlap
 * dS_out / dZ_out (LA_ERR_INVALID_ARG: the pieces of a sequence run concurrently and all start from
 * the upstream gradient).  With N = 0 the upstream state gradient is copied to dS_in / dZ_in (zeros
 * when it is NULL).  Everything else as for la_causal_backward(), which is this call with every
 * state pointer NULL.
 */
int la_causal_backward_from(const la_problem* p, const void* Q, const void* K, const void* V,
                            const float* S_in, const float* Z_in,
                            const void* O, const float* den, const void* G,
                            const float* dS_out, const float* dZ_out,
                            const void* saved, size_t saved_bytes,
                            void* dQ, void* dK, void* dV, float* dS_in, float* dZ_in,
                            void* ws, size_t ws_bytes, void* stream);

/*
 * The causal form on a right-padded ragged batch (speech-style batches: sequences of different lengths
 * padded to a common N; Eq. 9-12 and 16-20 per sequence on its own length).  lengths: [B] int32 (device),
 * lengths[b] in [0, N] = real positions of batch element b (all its heads); the N - lengths[b] rows behind
 * them are padding whose contents are never used, whatever they hold (Inf and NaN included).  O and den are
 * zero on the padding.  S_out / Z_out (optional) receive the state after each sequence's OWN last position,
 * so that a ragged prefill hands every stream over to la_recurrent_step() at the right place; S_in / Z_in
 * (both or neither) as for la_causal_forward_from().  ws: la_workspace_bytes(p, LA_OP_CAUSAL_VARLEN_FORWARD).
 * Causality alone already keeps right padding out of every real position's output; what this call adds is
 * the state at the true end, zeros instead of garbage on the padding, indifference to non-finite padding,
 * and no time spent on it.  saved / saved_bytes: as for la_causal_forward() (optional; what is kept covers the
 * real positions only, and the backward call must be given the same lengths).
 */
int la_causal_forward_varlen(const la_problem* p, const void* Q, const void* K, const void* V, const int32_t* lengths,
                             const float* S_in, const float* Z_in,
                             void* O, float* den, float* S_out, float* Z_out,
                             void* saved, size_t saved_bytes,
                             void* ws, size_t ws_bytes, void* stream);

/*
 * Gradients of la_causal_forward_varlen() (Eq. 13-15 per sequence on its own length): dQ, dK, dV are zero on
 * the padding, and G is not read there.  The state arguments are those of la_causal_backward_from(): dS_out /
 * dZ_out is the upstream gradient of the state at each sequence's own end, dS_in / dZ_in receive the gradient
 * of the state it started from.  saved / saved_bytes: the buffer la_causal_forward_varlen() filled for the same
 * problem and lengths, or NULL / 0.  ws: la_workspace_bytes(p, LA_OP_CAUSAL_VARLEN_BACKWARD).
 */
int la_causal_backward_varlen(const la_problem* p, const void* Q, const void* K, const void* V, const int32_t* lengths,
                              const float* S_in, const float* Z_in,
                              const void* O, const float* den, const void* G,
                              const float* dS_out, const float* dZ_out,
                              const void* saved, size_t saved_bytes,
                              void* dQ, void* dK, void* dV, float* dS_in, float* dZ_in,
                              void* ws, size_t ws_bytes, void* stream);

/* Number of GPU kernels this library has enqueued in this process so far (all
 * threads, all entry points); a diagnostic for benchmarks. */
long long la_kernel_launches(void);

/*
 * Optional per-kernel timing (a measurement aid, no counterpart in the paper).  While
 * switched on, every launch of the library's main kernels is bracketed by a pair of CUDA
 * events recorded on the launch stream (up to 512 launches per kernel are kept).
 * la_profile_enable(1) creates the events on first use and clears the counts;
 * la_profile_enable(0) stops recording.  la_profile_read() waits for the recorded events and
 * returns the mean duration in milliseconds and the number of launches of one kernel:
 * 0 causal_fwd_kernel, 1 causal_bwd_dq_kernel, 2 causal_bwd_dkv_kernel, 3 segment_sum_kernel,
 * 4 projection_gemm_kernel, 5 linear_sum_kernel, 6 linear_apply_kernel, 7 recurrent_step_kernel.
 * Not thread-safe; meant for a benchmark's single launching thread.
 */
int la_profile_enable(int on);
int la_profile_read(int kernel, double* mean_ms, int* launches);
const char* la_profile_kernel_name(int kernel);

/* Library version, "major.minor". */
const char* la_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LA_H_ */
