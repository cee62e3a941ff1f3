/*
 * linattn — non-causal O(n) linear attention with the Hedgehog feature map, for NVIDIA B200 (sm_100a).
 *
 * The operator (per batch b and head h, all n tokens attend to all n tokens):
 *
 *   phi(x) = softmax(x W) (+) softmax(-x W)            Eq. 6; W is d x d/2, (+) is concatenation,
 *                                                      both softmaxes run over the d/2 features
 *   S = sum_j phi(k_j)^T v_j   (d x d)                 Eq. 5, numerator bracket of the right-hand form
 *   z = sum_j phi(k_j)         (d)                     Eq. 5, denominator bracket
 *   o_i = phi(q_i) S / (phi(q_i) . z)                  Eq. 5, right-hand form
 *
 * with W = W_q for queries and W = W_k for keys.  There is no bias, no temperature, no
 * 1/sqrt(d) factor, no epsilon and no mask inside the operator.
 *
 * Every entry point returns a status and never throws, aborts or prints.  Nothing here falls
 * back to the CPU: an unsupported request is an error.  Unless an entry point says otherwise its
 * pointers are DEVICE pointers on the context's device, work is enqueued on the caller's stream
 * and the call returns without synchronising.
 */
#ifndef LINATTN_H
#define LINATTN_H

#ifdef __cplusplus
extern "C" {
#endif

typedef struct linattn_ctx linattn_ctx; /* opaque: feature-map weights + workspace of one attention layer */

typedef enum {
    LINATTN_OK = 0,
    LINATTN_ERR_INVALID_ARG = 1,    /* null pointer, size out of range, shape differs from create, misaligned pointer */
    LINATTN_ERR_UNSUPPORTED = 2,    /* d not in {64, 128}, unknown dtype, device is not sm_100 */
    LINATTN_ERR_NO_FEATURE_MAP = 3, /* forward before set_feature_map */
    LINATTN_ERR_WORKSPACE = 4,      /* request exceeds what create reserved */
    LINATTN_ERR_CUDA = 5,           /* a CUDA call failed; text via linattn_last_error */
    LINATTN_ERR_TIMEOUT = 6         /* a bounded device-side wait gave up (reported by linattn_check) */
} linattn_status;

typedef enum { LINATTN_F32 = 0, LINATTN_BF16 = 1 } linattn_dtype;

/* Options for linattn_set_option. */
typedef enum {
    LINATTN_OPT_SPLITS = 0, /* number of key-side partial reductions per (b,h); 0 = automatic (default) */
    LINATTN_OPT_PATH = 1,   /* 0 = automatic (default), 1 = CUDA-core kernels, 2 = tensor-core (tcgen05 + TMA) kernels */
    LINATTN_OPT_FUSE = 3,   /* tensor-core path: 1 = one cooperative kernel for the whole forward (default, used when the
                               device allows it), 0 = three launches (key side, combine, query side) */
    LINATTN_OPT_LAYOUT = 4, /* memory order of q, k, v, out (and o_softmax): 0 = [B][H][n][d] (default), 1 = [B][n][H][d],
                               the order in which a DiT's projection layers leave them (no transposes around the call);
                               d is contiguous in both */
    LINATTN_OPT_KERNEL_FUNCTION = 5, /* the map phi of Eq. 5: 0 = the Hedgehog feature map of Eq. 6 (default); 1 = the ReLU
                               kernel function of the paper's comparison across kernel functions, phi(x) = max(x, 0)
                               element by element on the d features of the head: no weights (set_feature_map is not
                               needed), no epsilon (a query whose phi is orthogonal to every key's gives a non-finite
                               row).  Applies to every entry point; the gradients (linattn_backward, _backward_mixed) then
                               run on the CUDA-core kernels, have no weight gradients (dWq, dWk are ignored and may be
                               NULL), and take d phi / d x = 1 where x > 0, else 0 */
    LINATTN_OPT_REUSE_STATE = 6, /* 1 = linattn_backward (tensor-core path) takes S and z from the workspace instead of
                               recomputing them when the most recent state-producing call on this context was a forward
                               (or backward) on the same k and v POINTERS, B, n and layout, with the same feature map.
                               The caller promises that the contents of k and v have not changed in between (the
                               forward -> backward order of a training step).  0 = always recompute (default) */
    LINATTN_OPT_WAIT_LIMIT_US = 7, /* bound, in microseconds, of every wait inside the tensor-core kernels, forward and
                               backward (on a shared-memory barrier or on another CTA): default 2,000,000.  A wait that
                               runs out makes the kernel record a code, unwind and return; linattn_check then reports
                               LINATTN_ERR_TIMEOUT */
    LINATTN_OPT_TEST_UNMET_ARRIVAL = 8, /* for tests of the time-out path only.  1 = the single-kernel forward waits, at the
                               points where the CTAs that share a head meet, for one arrival more than will ever come;
                               2 / 3 = in the query-side / key-side kernel of the tensor-core backward one warp of every
                               CTA leaves out one arrival that the warp issuing the tensor-core products waits for.  The
                               bounded wait runs out (nothing faults or hangs: the kernel gives up after the wait limit,
                               its output is not produced, linattn_check reports TIMEOUT).  0 = off (default) */
    LINATTN_OPT_PROFILE = 2 /* 1 = record CUDA events around every kernel of each forward (see linattn_profile_get);
                               switching it on clears the accumulated figures; 0 = off (default) */
} linattn_option;

/*
 * Create a context for one attention layer with H heads of dimension d (Eq. 5-6 are per head;
 * the paper writes a single head).  Allocates, on `device`, room for the feature-map weights and
 * the workspace that holds the partial and final S and z (Eq. 5) for up to max_B * H (b,h) pairs.
 * max_n bounds the sequence length later calls may use.  *ctx is written only on success.
 * Errors: INVALID_ARG (null ctx, H/max_B/max_n < 1), UNSUPPORTED (d not 64 or 128, device not
 * compute capability 10.x), CUDA (allocation failed).
 */
linattn_status linattn_create(linattn_ctx** ctx, int device, int H, int d, long long max_B, long long max_n);

/*
 * Set W_q and W_k of Eq. 6.  Wq, Wk: device pointers, row-major [H][d][d/2] when per_head != 0, or
 * [d][d/2] shared by all heads when per_head == 0, of type wdtype.  The values are COPIED (and
 * converted) into the context on `stream`; the caller may free its buffers once that stream has
 * passed this point.  Errors: INVALID_ARG, UNSUPPORTED (wdtype), CUDA.
 */
linattn_status linattn_set_feature_map(linattn_ctx* ctx, const void* Wq, const void* Wk, int per_head,
                                       linattn_dtype wdtype, void* stream);

/*
 * Eq. 5 (right-hand form) with the feature map of Eq. 6, for all B*H (b,h) pairs.
 *   q, k, v : device, contiguous [B][H][n][d] (or [B][n][H][d], see LINATTN_OPT_LAYOUT) of `dtype`, 16-byte aligned,
 *             read-only
 *   out     : device, same shape and type, written in full; must not overlap q, k or v
 *   H, d    : must equal the values given to create;  1 <= B <= max_B;  1 <= n <= max_n
 *   dtype   : LINATTN_BF16 (bf16 in, bf16 out, round-to-nearest-even) or LINATTN_F32
 *   stream  : a cudaStream_t of the context's device (NULL = default stream)
 * All accumulation (S, z, numerator, denominator) is fp32.  The call allocates nothing, does not
 * synchronise, and is deterministic: the same inputs give bit-identical outputs.  Calls on one
 * context must be stream-ordered (they share the context's workspace).  Nothing about a launch
 * depends on earlier launches (the single cooperative kernel of the tensor-core path leaves its
 * synchronisation counters cleared), so the call may be recorded into a CUDA graph and replayed.
 * Errors: INVALID_ARG, UNSUPPORTED, NO_FEATURE_MAP, WORKSPACE, CUDA (launch failure).
 */
linattn_status linattn_forward(linattn_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                               int B, int H, int n, int d, linattn_dtype dtype, void* stream);

/*
 * Mixed attention, Eq. 8: the layer's output while softmax attention is being transferred to linear attention,
 *   out = r^ * o_softmax + (1 - r^) * [Eq. 5 applied to q, k, v],    r^ = min(max(r, 0), 1)
 * (the footnote to Eq. 8 clips the learnable score r into [0, 1] before use).  o_softmax is the output of the
 * softmax-attention branch of the same layer, computed by the caller with whatever attention kernel and
 * scale it uses (the paper prints 1/sqrt(d) under Eq. 4 and 1/d inside Eq. 8); the blend is fused into the
 * query side's epilogue: fp32, rounded once to the output type.  r^ = 0 gives linattn_forward's result bit
 * for bit, r^ = 1 returns o_softmax.
 *   o_softmax : device, [B][H][n][d] of `dtype`, 16-byte aligned, read-only; it may be the SAME buffer as `out`
 *               (in place); any other overlap with `out` is an error
 *   r         : the layer's score (host value); NaN is an error
 * Everything else as for linattn_forward.  Errors: as linattn_forward, plus INVALID_ARG for the above.
 */
linattn_status linattn_forward_mixed(linattn_ctx* ctx, const void* q, const void* k, const void* v,
                                     const void* o_softmax, float r, void* out, int B, int H, int n, int d,
                                     linattn_dtype dtype, void* stream);

/*
 * Gradients of linattn_forward: what the training objective (Eq. 14) back-propagates through a layer that uses
 * Eq. 5 with the feature map of Eq. 6.  Given dout = dL/d(out), writes dL/dq, dL/dk, dL/dv and the gradients of
 * the two feature-map weight matrices.  S and z are recomputed from k, v (no forward needs to precede the call;
 * see LINATTN_OPT_REUSE_STATE for taking them over from the forward).
 *   q, k, v, dout : device, as q, k, v of linattn_forward (same layout option), read-only
 *   dq, dk, dv    : device, same shape, type and layout; written in full; must not overlap any input or each other
 *   dWq, dWk      : device, fp32, 16-byte aligned, written in full: [H][d][d/2] when per_head != 0 (each head's
 *                   gradient summed over the batch), [d][d/2] when per_head == 0 (one shared matrix: summed over
 *                   batch and heads).  The weights differentiated are the ones given to set_feature_map.
 * Two sets of kernels, chosen like the forward's (LINATTN_OPT_PATH): for bf16 activations with d = 128 and bf16
 * feature-map weights the products run on the tensor cores (bf16 operands, fp32 accumulation; S and dS enter as
 * bf16 hi + lo pairs and dO itself, exact in bf16, is the operand where dO / den is needed, so that gradients stay
 * accurate when V has a large mean; relative L2 error about 3e-3 per gradient); everything else, or path 1, runs in
 * fp32 on the CUDA cores (the stored q, k, v, dout are then the only rounded quantities).  dq, dk, dv are
 * rounded once to `dtype`.  All sums have a fixed order: the same inputs give bit-identical gradients.  The first
 * call allocates the backward workspace (it synchronises the device once); later calls allocate nothing.  After
 * the call the context holds the S, z of these k, v (linattn_read_state returns them).
 * Errors: INVALID_ARG, UNSUPPORTED, NO_FEATURE_MAP, WORKSPACE, CUDA.
 */
linattn_status linattn_backward(linattn_ctx* ctx, const void* q, const void* k, const void* v, const void* dout,
                                void* dq, void* dk, void* dv, float* dWq, float* dWk, int per_head,
                                int B, int H, int n, int d, linattn_dtype dtype, void* stream);

/*
 * Gradients through mixed attention, Eq. 8: out = r^ * o_softmax + (1 - r^) * [Eq. 5 applied to q, k, v], r^ = clip(r, 0, 1),
 * the layer that the objective of Eq. 14 is back-propagated through while softmax attention is being transferred to
 * linear attention.  Given dout = dL/d(out):
 *   dq, dk, dv, dWq, dWk : the gradients of linattn_backward for the incoming gradient (1 - r^) * dout (the factor is
 *                          applied inside the kernels, to the fp32 accumulators: nothing is rounded twice)
 *   d_o_softmax          : r^ * dout, the gradient that reaches the softmax branch (device, shape and type of dout;
 *                          may be NULL: not computed); must not overlap any other argument
 *   dr                   : device, ONE float, 4-byte aligned: dL/dr = sum dout * (o_softmax - linear attention) if
 *                          0 <= r <= 1, else 0.  (The paper clips r and says nothing of the clip's derivative; it is taken
 *                          as 1 on the closed interval: every r starts at 1, and with a zero derivative there it could
 *                          never move.)  Summed in a fixed order: bit-reproducible.
 *   o_softmax            : the softmax branch's output as given to linattn_forward_mixed (read-only)
 * Everything else (layouts, the two sets of kernels, workspace, errors) as for linattn_backward; r = NaN is INVALID_ARG.
 */
linattn_status linattn_backward_mixed(linattn_ctx* ctx, const void* q, const void* k, const void* v,
                                      const void* o_softmax, float r, const void* dout,
                                      void* dq, void* dk, void* dv, float* dWq, float* dWk, int per_head,
                                      void* d_o_softmax, float* dr,
                                      int B, int H, int n, int d, linattn_dtype dtype, void* stream);

/*
 * The same operation on HOST buffers (pageable or pinned; pinned buffers let the copies overlap).  For the
 * default [B][H][n][d] layout the (b,h) pairs, which are independent and contiguous, go through a three-stage
 * pipeline inside the call: copies to the device on one internal stream, the forward of one pair on `stream`,
 * copies of finished pairs back on a second internal stream, so that both copy directions and the compute
 * overlap; the call returns when `out` is complete.  For the token-major layout the problem goes in one piece.
 * The staging buffers (four of the problem's size) are allocated, or grown, on the first call that needs them
 * and released by destroy.  Same argument rules and errors as linattn_forward, except that the pointers are
 * host pointers with no alignment requirement.  Each pair is reduced with the split of a one-pair problem, so
 * the result agrees with linattn_forward's to rounding (not bit for bit); it is deterministic like every entry
 * point.  linattn_read_state afterwards returns the S, z of all pairs as usual.
 */
linattn_status linattn_forward_host(linattn_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                                    int B, int H, int n, int d, linattn_dtype dtype, void* stream);

/*
 * Copy the S and z (Eq. 5) left in the workspace by the most recent forward to HOST memory:
 * S_host [B][H][d][d] floats with S[f][c] = sum_j phi(k_j)[f] v_j[c], z_host [B][H][d] floats.
 * Waits for `stream`.  Either pointer may be NULL.  For tests and debugging.
 */
linattn_status linattn_read_state(linattn_ctx* ctx, float* S_host, float* z_host, int B, void* stream);

/*
 * The forward for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * is a property of the library, not of the method.)  Typical cases: a plug-in that is handed
 * pointers and a stream by a framework whose memory pool it may not touch; a latency-critical
 * serving thread, where cudaMalloc / cudaFree would synchronise the whole device; code that must
 * not fail for lack of memory at call time.  It needs no context: the feature-map weights are
 * passed in, and the scratch for the partial and combined S, z of Eq. 5 is a fixed array inside
 * the library's device image (about 5.3 MB, held by every GPU that loads the library until the
 * process exits).  It calls no allocator of any kind and computes the same operation as
 * linattn_forward with the CUDA-core kernels.
 *   q, k, v, out : as for linattn_forward (device, [B][H][n][d] of `dtype`, 16-byte aligned)
 *   Wq, Wk       : device, fp32, 16-byte aligned, [H][d][d/2] (per_head != 0) or [d][d/2]; read, not copied
 *   limits       : B * H <= 16 and d in {64, 128}; any n >= 1.  A larger B * H returns
 *                  LINATTN_ERR_WORKSPACE ("request exceeds the workspace ...") and launches nothing.
 *   out          : must not overlap q, k or v (INVALID_ARG)
 * Runs on the CURRENT device, which must be of compute capability 10.x (else UNSUPPORTED).  The first
 * call on each device looks up the device address of the scratch array and raises the kernels'
 * shared-memory limit; make that first call before any stream capture begins, and from ONE host
 * thread (the set-up results are cached in unsynchronised host variables; later calls may come
 * from any thread).  All calls on a device share the one scratch array: it keeps the previous
 * call's contents, every element a call reads is first written by that same call (nothing needs
 * clearing), and two calls whose kernels overlap on the GPU (different streams, no ordering) race
 * on it and give wrong results -- keep calls on one device stream-ordered.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA.
 */
linattn_status linattn_forward_noalloc(const void* q, const void* k, const void* v, void* out,
                                       const float* Wq, const float* Wk, int per_head,
                                       int B, int H, int n, int d, linattn_dtype dtype, void* stream);

/* Tuning and test knobs; see linattn_option.  Errors: INVALID_ARG (unknown option or value). */
linattn_status linattn_set_option(linattn_ctx* ctx, linattn_option opt, long long value);

/*
 * Wait for `stream` and report whether any kernel of this context gave up a bounded wait
 * (TIMEOUT) or the stream hit a CUDA error (CUDA); clears the device-side error word.
 */
linattn_status linattn_check(linattn_ctx* ctx, void* stream);

/*
 * Per-kernel timing gathered while LINATTN_OPT_PROFILE is on.  index = position of the kernel in the
 * forward's launch order.  Returns 1 and fills the outputs (any may be NULL) if that kernel has been
 * timed at least once, else 0: *name (static string), *mean_ms (mean duration between the CUDA events
 * around its launches), *launches, *algorithmic_bytes (bytes of q/k/v/out one launch must move:
 * K+V for the key side, Q+O for the query side).  Waits for the last profiled forward to finish.
 */
int linattn_profile_get(linattn_ctx* ctx, int index, const char** name, double* mean_ms, long long* launches,
                        double* algorithmic_bytes);

/* Number of kernels the most recent linattn_forward or linattn_backward on this context launched (0 before any). */
int linattn_last_launch_count(const linattn_ctx* ctx);

/* Text of the last CUDA error seen by this context ("" if none).  Valid until the next call on ctx. */
const char* linattn_last_error(const linattn_ctx* ctx);

/* Release everything the context owns.  Waits for the device.  NULL is accepted. */
linattn_status linattn_destroy(linattn_ctx* ctx);

/* Static text for a status code. */
const char* linattn_status_string(linattn_status s);

#ifdef __cplusplus
}
#endif
#endif /* LINATTN_H */
