/*
 * fq.h -- C ABI of the B200 (sm_100a) folded quantized linear layer.
 *
 * One projection site of the method runs as
 *   offline : W~ = W S R^T, round to nearest per output channel, pack   (Alg. 1, offline half; Eq. 3)
 *   runtime : z_t = R S^-1 x_t, per-token symmetric quantization         (Alg. 1 runtime half; Eq. 5)
 *             c = q^W q^A (int32), y = delta_t (s^W (.) c) + b           (Eq. 8)
 * with R the normalised block Hadamard transform applied as an FWHT.
 *
 * Conventions that hold for every entry point
 *   - "device" pointers are CUDA global-memory addresses on the current device,
 *     "host" pointers are ordinary process memory.  The kind is stated per argument.
 *   - Matrices are row-major; a leading dimension (ld*) counts ELEMENTS between rows.
 *     Activations are [M tokens, K channels]; weights are [N output channels, K].
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     All work is enqueued on it; no entry point synchronises unless it says so.
 *   - The caller owns every buffer except the memory inside an fq_weights handle.
 *     Inputs are never written.  Output rows >= M and bytes outside the stated
 *     shapes are never touched.
 *   - Errors are return codes.  Nothing aborts, throws or traps.  Argument checks run
 *     on the host before any launch; a failed check launches nothing.
 *   - Inputs must be finite; NaN/Inf give unspecified codes (never a fault).
 *   - Supported sizes: hadamard_block a power of two in [1, 256] dividing K (1 = identity rotation);
 *     K a multiple of 32 and <= 131072 (int32 accumulator bound; the prologue and the fold
 *     keep a whole token in one thread block and accept K <= 32768); N a multiple of 8;
 *     bits 4 or 8; clip_ratio in (0, 1].  M = 0 or N = 0 succeeds and does nothing.
 *   - Device pointers must be 16-byte aligned and ld* a multiple of 8 elements.
 *   - Arithmetic of the transform and quantizer is IEEE binary32, round to nearest
 *     even, no fused multiply-add, ascending butterfly strides; ties in round() go
 *     to even.  4-bit codes are two's-complement nibbles, even channel in the low
 *     nibble, row pitch K/2 bytes; 8-bit codes are int8, row pitch K bytes.
 */
#ifndef FQ_H_
#define FQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FQ_OK = 0,
    FQ_ERR_INVALID_ARG = 1, /* NULL where data is required, negative size, bits not 4/8, bad clip ratio */
    FQ_ERR_UNSUPPORTED = 2, /* size or block outside the supported set, handle/call bit width mismatch */
    FQ_ERR_ALIGNMENT = 3,   /* pointer not 16-byte aligned or leading dimension not a multiple of 8 */
    FQ_ERR_ARCH = 4,        /* current device is not compute capability 10.x */
    FQ_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed */
    FQ_ERR_NOMEM = 6,       /* allocation failed, or caller workspace too small */
    FQ_ERR_TIMEOUT = 7      /* a bounded device-side wait expired (see fq_device_status) */
} fq_status;

typedef enum { FQ_F32 = 0, FQ_BF16 = 1 } fq_dtype;

/* Opaque folded-weight pack of one consumer projection (or several consumers of one
 * site concatenated along N).  Owns device memory; changed only by the offline calls
 * fq_weights_set_multiplier / fq_weights_scale_outputs. */
typedef struct fq_weights fq_weights;

const char* fq_status_string(fq_status s);

/* ---- offline: fold + round + pack (Alg. 1 offline half, Eq. 3 fold-before, RTN) ----------
 * W      device, [N, K] of dtype wt, leading dimension ldw.
 * smooth device float[K] SmoothQuant scales s_c, or NULL for S = I.
 * bias   device float[N] or NULL (= 0); copied into the handle unchanged (output transform is I).
 * Creates *out holding: packed codes [N, K*bits/8], s^W[N], bias[N] and the runtime multiplier
 * g[K] = (1/s_c) * block^-1/2.  Allocates with cudaMalloc (this call only); work is async on stream.
 * Row j of W~ is FWHT(s (.) w_j * block^-1/2); s^W_j = max|W~_j| / q; no weight clipping.
 * hadamard_block is a power of two in [1, 256] dividing K; 1 is the identity rotation (R = I: a site that is
 * only scaled, or -- with smooth = NULL -- plain RTN of W, the identity transform of a graph boundary). */
fq_status fq_fold_weights(const void* W, fq_dtype wt, int64_t N, int64_t K, int64_t ldw,
                          const float* smooth, const float* bias, int hadamard_block, int bits,
                          void* stream, fq_weights** out);

/* ---- offline, fold-after variant (section "Transforms supported by the runtime", Eq. 2 with
 * (D^i, D^o) = (I, P^-1)): W~ = W R^T P, row j = (R w_j) (.) p, then RTN and packing as above.
 * post_scale device float[K], the positive diagonal P calibrated AFTER rotation (statistics of R x and
 * of W R^T; fq_col_absmax / fq_smooth_scale work on such rotated tensors like on any other).
 * The handle's runtime multiplier is 1/p_c and is applied behind the rotation: z = P^-1 R x, with the
 * constant block^-1/2 ahead of it (the paper's "extra pass" costs one multiply per element in the same
 * kernel).  Every other call takes such a handle like a fold-before one. */
fq_status fq_fold_weights_after(const void* W, fq_dtype wt, int64_t N, int64_t K, int64_t ldw,
                                const float* post_scale, const float* bias, int hadamard_block, int bits,
                                void* stream, fq_weights** out);

/* 1 if the handle was folded after the rotation (its multiplier is the post-rotation 1/p), else 0. */
int fq_weights_fold_after(const fq_weights* w);

/* Frees the handle's device memory (cudaFree synchronises the device). NULL is accepted. */
fq_status fq_weights_destroy(fq_weights* w);

/* Shape query (host). Any out pointer may be NULL. */
fq_status fq_weights_info(const fq_weights* w, int64_t* N, int64_t* K, int* hadamard_block, int* bits);

/* Device pointer to the handle's runtime multiplier g[K] (valid until destroy). */
const float* fq_weights_multiplier(const fq_weights* w);

/* Copy the canonical pack out of / into a handle.  All pointers are device pointers with
 * the shapes listed for fq_fold_weights; any destination may be NULL to skip it.
 * Import allocates a new handle; bias may be NULL (= 0). */
fq_status fq_weights_export(const fq_weights* w, void* codes, float* w_scale, float* mult_g, float* bias,
                            void* stream);
fq_status fq_weights_import(const void* codes, const float* w_scale, const float* mult_g,
                            const float* bias, int64_t N, int64_t K, int hadamard_block, int bits,
                            void* stream, fq_weights** out);

/* ---- exact folds into neighbouring operators (section "Normalization gains", Eq. 4) --------------
 * fq_weights_set_multiplier replaces the handle's runtime multiplier (offline; the stream is synchronised).
 *   mult device float[K]: e.g. gamma_c * (1/s_c) * block^-1/2 for a projection that follows an RMS
 *   normalisation whose learned gain gamma is absorbed here (the product D^i Gamma of Eq. 4: the input is
 *   then the gain-free normalised activation), or NULL: the constant block^-1/2, for a site whose diagonal
 *   1/s has been absorbed by its producer.
 * fq_weights_scale_outputs multiplies output channels [first, first + count) of a handle by d_j > 0
 *   (d device float[count]): s^W_j *= d_j and b_j *= d_j, one binary32 multiply each; codes unchanged.  This
 *   is how a diagonal 1/s ahead of down_proj is absorbed into the linear up branch of a gated MLP (d = 1/s on
 *   the up rows of the gate/up handle) without crossing the gate non-linearity. */
fq_status fq_weights_set_multiplier(fq_weights* w, const float* mult, void* stream);
fq_status fq_weights_scale_outputs(fq_weights* w, int64_t first, int64_t count, const float* d, void* stream);

/* Import of a fold-after pack: mult_post device float[K] = 1/p (required). */
fq_status fq_weights_import_after(const void* codes, const float* w_scale, const float* mult_post,
                                  const float* bias, int64_t N, int64_t K, int hadamard_block, int bits,
                                  void* stream, fq_weights** out);

/* ---- offline fold with GPTQ rounding in transformed coordinates (section "Rounding and native execution",
 * Eq. 7: min_Q ||(W~ - Q) Z||_F^2 with G = Z Z^T and diagonal damping; the paper's rounding at four bits) ------
 * As fq_fold_weights (fold-before), but the codes come from the GPTQ sweep instead of round-to-nearest:
 *   calib  device [Mc, K] of dtype ct, leading dimension ldc: calibration tokens of the site in ORIGINAL
 *          coordinates; they are transformed with the handle's own runtime multiplier, Z = T calib;
 *   damp   lambda = damp * mean(diag G) is added to the diagonal (0.01 is customary); a channel that is never
 *          active in calibration (G_cc = 0) gets zero codes;
 *   the per-output-channel steps are those of the round-to-nearest fold (max|W~_j| / q).
 * Channels are rounded in index order; each rounding error (w - q s)/U_ii is spread over the channels still to
 * come along row i of the upper Cholesky factor U of (G + lambda I)^-1.  All of it runs in binary32 in a fixed
 * order, so the codes are reproducible bit for bit.  K <= 16384 (FQ_ERR_UNSUPPORTED beyond; the factorisation is
 * column-sequential and cubic in K: 0.2 s at K = 2048, minutes at K = 16384); FQ_ERR_INVALID_ARG if
 * the damped second moment is not positive definite in binary32.  Offline: allocates (about 3 K^2 + (N + Mc) K
 * floats of temporaries) and synchronises the stream. */
fq_status fq_fold_weights_gptq(const void* W, fq_dtype wt, int64_t N, int64_t K, int64_t ldw, const float* smooth,
                               const float* bias, const void* calib, fq_dtype ct, int64_t Mc, int64_t ldc,
                               int hadamard_block, int bits, float damp, void* stream, fq_weights** out);

/* ---- stored composite rotation (section "Transforms supported by the runtime": optional for the action
 * expert; the design ablation "butterfly vs. composite rotation") ------------------------------------------
 * R = blockdiag(B_0 .. B_{K/block-1}) Pi: a channel permutation, then one stored dense block x block matrix per
 * block of channels.   z[b*block + i] = sum_j B_b[i][j] * v[perm[b*block + j]],  v = x (.) (1/s).
 *   perm   device int32[K]: perm[c] = source channel of position c (a permutation of 0..K-1);
 *   blocks device float[K/block][block][block], row-major; orthogonal matrices that carry their own
 *          normalisation (e.g. block^-1/2 H U^T of an SVD basis U) -- the library does not check orthogonality:
 *          the fold W~ = W S R^T computed here is row j = R (s (.) w_j), which equals W S R^-1 only if R^T R = I;
 *   block  in {16, 32, 64, 128, 256}.
 * Arithmetic: binary32, one multiply for the diagonal, then one fused multiply-add per term in ascending j.
 * fq_fold_weights_composite: as fq_fold_weights (RTN per output channel, packing, allocation, offline
 *   synchronisation); FQ_ERR_INVALID_ARG if perm has an entry outside [0, K).  The handle's runtime multiplier is
 *   1/s_c (ones without smoothing).  The handle does not keep perm and blocks.
 * fq_quantize_act_composite: the runtime prologue of such a site (rotation, then Eq. 5); workspace device, at least
 *   4*M*K bytes, 16-byte aligned (the rotated rows in binary32; two kernels).  Entries of perm outside [0, K) are
 *   clamped.  Then fq_gemm_w4a4 / fq_gemm_w8a8 per consumer; the one-call fq_linear_* entry points return
 *   FQ_ERR_UNSUPPORTED for a composite handle. */
fq_status fq_fold_weights_composite(const void* W, fq_dtype wt, int64_t N, int64_t K, int64_t ldw, const float* smooth,
                                    const float* bias, const int32_t* perm, const float* blocks, int block, int bits,
                                    void* stream, fq_weights** out);
fq_status fq_quantize_act_composite(const void* x, fq_dtype xt, int64_t M, int64_t K, int64_t ldx, const float* mult_g,
                                    const int32_t* perm, const float* blocks, int block, int bits, float clip_ratio,
                                    void* codes_out, float* delta_out, void* workspace, size_t ws_bytes, void* stream);
/* 1 if the handle was folded with a stored composite rotation, else 0. */
int fq_weights_composite(const fq_weights* w);

/* ---- calibration support (section "Transforms supported by the runtime", SmoothQuant scale) --
 * fq_col_absmax: out[c] = max(out[c] if accumulate else 0, max_t |x[t][c]|); x device [M, K].
 * fq_smooth_scale: s_c = clamp(max(a_c,1e-5)^alpha / max(w_c,1e-5)^(1-alpha), 1e-5, 1e5) in
 * binary64 on the device; a, w, s device float[K]; alpha in [0, 1]. */
fq_status fq_col_absmax(const void* x, fq_dtype xt, int64_t M, int64_t K, int64_t ldx, int accumulate,
                        float* out, void* stream);
fq_status fq_smooth_scale(const float* a, const float* w, int64_t K, double alpha, float* s, void* stream);

/* ---- runtime prologue (Alg. 1 runtime half lines 1-2; Eq. 5) ----------------------------------
 * x       device [M, K] of dtype xt, leading dimension ldx.
 * mult_g  device float[K] (fq_weights_multiplier of any consumer of the site) or NULL (S = I).
 * codes_out device, [M, K*bits/8] bytes, canonical packing, pitch K*bits/8.
 * delta_out device float[M]: delta_t = (clip_ratio * max_c|z_tc|) / q, 0 for a zero token
 * (a token whose step would be below FLT_MIN), whose codes are all 0. */
fq_status fq_quantize_act(const void* x, fq_dtype xt, int64_t M, int64_t K, int64_t ldx,
                          const float* mult_g, int hadamard_block, int bits, float clip_ratio,
                          void* codes_out, float* delta_out, void* stream);

/* Runtime prologue of a fold-after site: z = P^-1 R x (mult_post = fq_weights_multiplier of a consumer
 * folded with fq_fold_weights_after), then Eq. 5 as above. */
fq_status fq_quantize_act_after(const void* x, fq_dtype xt, int64_t M, int64_t K, int64_t ldx,
                                const float* mult_post, int hadamard_block, int bits, float clip_ratio,
                                void* codes_out, float* delta_out, void* stream);

/* ---- integer GEMM + rescale/bias epilogue on pre-quantized activations (Eq. 8) -----------------
 * a_codes device, canonical codes from fq_quantize_act with the same bit width as W.
 * a_delta device float[M]; any 4-byte aligned address is accepted (a slice delta + t0 of a longer vector is
 * fine: the epilogue then reads the steps one by one instead of four at a time).
 * y device [M, N] of dtype yt, leading dimension ldy.
 * workspace device, at least fq_workspace_bytes(M, K, N, bits) bytes, 256-byte aligned; contents
 * are scratch (calls sharing a workspace must be stream-ordered).
 * Shared sites: quantize once, then call this once per consumer handle. */
fq_status fq_gemm_w4a4(const void* a_codes, const float* a_delta, int64_t M, const fq_weights* W,
                       void* y, fq_dtype yt, int64_t ldy, void* workspace, size_t ws_bytes, void* stream);
fq_status fq_gemm_w8a8(const void* a_codes, const float* a_delta, int64_t M, const fq_weights* W,
                       void* y, fq_dtype yt, int64_t ldy, void* workspace, size_t ws_bytes, void* stream);

/* ---- whole runtime path of one consumer: prologue + GEMM + epilogue (Alg. 1 runtime half) ------
 * Equivalent to fq_quantize_act (codes and delta kept in the workspace) followed by fq_gemm_*.
 * K, N, block and bits come from the handle; the handle's bit width must match the entry point. */
fq_status fq_linear_w4a4(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const fq_weights* W,
                         float clip_ratio, void* y, fq_dtype yt, int64_t ldy, void* workspace,
                         size_t ws_bytes, void* stream);
fq_status fq_linear_w8a8(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const fq_weights* W,
                         float clip_ratio, void* y, fq_dtype yt, int64_t ldy, void* workspace,
                         size_t ws_bytes, void* stream);

/* ---- weight-only 4-bit projection with floating-point activations ------------------------------
 * (Section "Problem statement": in the W4A4 engines the adaptive layer-normalisation modulation keeps
 * floating-point activations and only its weights are INT4.)  With the reconstruction W^_jc = s^W_j qW_jc
 * of Eq. 8:   y[t][j] = s^W_j * sum_c qW[j][c] * x[t][c] + b_j.
 * W is any 4-bit handle; its codes multiply x as given, so a handle meant for this call is made with the
 * identity transform (fq_fold_weights with hadamard_block = 1 and smooth = NULL: plain per-output-channel
 * RTN of W), or x must already be in the handle's transformed coordinates.  No quantization of x, no
 * workspace.  x device [M, K] of dtype xt (FQ_F32 or FQ_BF16); binary32 accumulation (the products are exact; the
 * expanded codes carry an offset that a second MMA removes sixteen channels at a time, so the sums' rounding does not
 * depend on the activations' mean).
 * These projections see
 * one conditioning vector per sample: the kernel streams the weights once per eight tokens and is meant for
 * short batches (any M is accepted).  Errors as for fq_linear_w4a4; FQ_ERR_UNSUPPORTED for 8-bit handles. */
fq_status fq_linear_w4a16(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const fq_weights* W, void* y,
                          fq_dtype yt, int64_t ldy, void* stream);

/* ---- the site behind a gated MLP: gate product fused into down_proj's prologue -------------------------
 * (Section "Normalization gains" names the gated MLP and its gate non-linearity; the paper fixes neither the
 * function nor a fused kernel -- this removes the round trip of the widest activation of a layer through HBM.)
 * gate_up device [M, 2K] of dtype xt, leading dimension ld >= 2K: gate in columns [0, K), up in [K, 2K), as a fused
 * gate/up projection writes them.  The quantizer's input is h = act(gate) (.) up, never stored:
 *   act(x) = x * sigmoid(k),  k = x (FQ_GATE_SILU)  or  k = 2 sqrt(2/pi) (x + 0.044715 x^3) (FQ_GATE_GELU_TANH),
 * in fixed binary32 arithmetic (the exponential is a range reduction, a degree-6 polynomial in Horner form with
 * fused multiply-adds and a scaling by exponent bits: h decides integer codes, so the oracle and the device take
 * the same steps).  Then as fq_quantize_act / fq_linear_* with K = the handle's (intermediate) width.
 * fq_linear_gated dispatches on the handle's bit width; fold-after handles work, composite ones do not. */
typedef enum { FQ_GATE_SILU = 0, FQ_GATE_GELU_TANH = 1 } fq_gate_act;
fq_status fq_quantize_act_gated(const void* gate_up, fq_dtype xt, int64_t M, int64_t K, int64_t ld, fq_gate_act act,
                                const float* mult_g, int hadamard_block, int bits, float clip_ratio, void* codes_out,
                                float* delta_out, void* stream);
fq_status fq_linear_gated(const void* gate_up, fq_dtype xt, int64_t M, int64_t ld, fq_gate_act act, const fq_weights* W,
                          float clip_ratio, void* y, fq_dtype yt, int64_t ldy, void* workspace, size_t ws_bytes,
                          void* stream);

/* ---- fused W4A4 linear without a workspace, for callers that cannot allocate ------------------
 * (The paper has no counterpart: this is a deployment convenience of this library.)
 * Same result as fq_linear_w4a4, but the quantized activations and per-token steps that sit
 * between the two kernels live in a scratch area built into the library image instead of a
 * caller workspace.  It is meant for code that has no way to obtain device memory at call time:
 * plugin enqueue callbacks that are forbidden to call cudaMalloc, control loops that cannot
 * tolerate the device-wide synchronisation an allocation can imply, processes whose device
 * memory was all handed out at start-up.  The call performs no cudaMalloc/cudaFree and calls no
 * allocating library routine; the caller still provides x and y.
 *   Limits: M * K <= FQ_STATIC_MAX_CODE_BYTES (4 MiB) and M <= FQ_STATIC_MAX_TOKENS (16384);
 *   anything larger returns FQ_ERR_NOMEM and launches nothing.  The scratch (4 MiB + 64 KiB) is
 *   held by every GPU that loads the library until the process exits.
 *   The first call on each device looks up the scratch's device address (once, with that device
 *   current).  That look-up is also what makes the CUDA runtime load the part of the library image
 *   that holds the scratch onto the device, so this ONE call may itself reserve device memory, may
 *   synchronise, and can fail with FQ_ERR_CUDA on a device that has no room left: make it at
 *   start-up, before any stream capture and before the phase in which allocation is forbidden.  A
 *   call with M = 0 performs just this set-up and launches nothing, so it serves as the warm-up.
 *   All calls on a device share the one scratch.  Nothing in it needs clearing -- each call
 *   rewrites every row it later reads -- but it keeps the previous call's contents, and two calls
 *   whose kernels may overlap on the GPU (different streams without an ordering between them)
 *   race on it: keep calls to this entry point stream-ordered per device. */
#define FQ_STATIC_MAX_CODE_BYTES (4ll << 20)
#define FQ_STATIC_MAX_TOKENS 16384ll
fq_status fq_linear_w4a4_static(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const fq_weights* W,
                                float clip_ratio, void* y, fq_dtype yt, int64_t ldy, void* stream);

/* Bytes of workspace that fq_gemm_* / fq_linear_* want for this shape (host computation): the int8
 * activation codes and steps (M*K + 4*M bytes, each rounded up to 256), plus scratch for int32 partial
 * tiles on shapes with few output tiles and a long K, which the GEMM then splits along K.  A workspace
 * that holds only the first part is accepted; the GEMM then runs without the split.  Everything a call
 * scribbles on lives in the workspace it was given (the split's tile counters included, cleared by a
 * memset node at the head of the call): a weight handle is read-only at run time, so calls on the same
 * handle may run concurrently on different streams as long as each has its own workspace. */
size_t fq_workspace_bytes(int64_t M, int64_t K, int64_t N, int bits);

/* Parity/debug: raw int32 accumulators acc[M, N] (device, pitch N) of Eq. 8's integer sum. */
fq_status fq_gemm_acc_i32(const void* a_codes, int64_t M, const fq_weights* W, int32_t* acc,
                          void* workspace, size_t ws_bytes, void* stream);

/* On-device second witness (Eq. 8 with CUDA-core dp4a arithmetic, untuned): same arguments as
 * fq_gemm_*; if acc != NULL it receives raw int32 accumulators [M, N] and y is ignored.  Used by the
 * tests to cross-check the tensor-core kernel at sizes where the CPU oracle can only sample. */
fq_status fq_gemm_simt(const void* a_codes, const float* a_delta, int64_t M, const fq_weights* W, void* y,
                       fq_dtype yt, int64_t ldy, int32_t* acc, void* workspace, size_t ws_bytes, void* stream);

/* Profiling hook (process-global, not thread-safe; benchmarks only).  While `event` -- a
 * cudaEvent_t passed as void* -- is non-NULL, every fq_linear_* call records it on its stream
 * between the prologue kernel and the GEMM kernel, so a caller that brackets the call with two
 * events of its own obtains the two kernel durations of that very launch.  During a stream capture
 * the mark becomes an external event-record node of the graph.  NULL switches it off. */
fq_status fq_profile_mark(void* event);

/* Self-test of the watchdog below: enqueues a one-warp kernel whose only action is a bounded wait, with the
 * library's own wait routine and a limit of limit_ns nanoseconds (clamped to [1 us, 100 ms]), on a barrier that
 * nothing ever signals.  The wait gives up, the kernel ends normally, and the next fq_device_status() returns
 * FQ_ERR_TIMEOUT (detail bit 0x400) and clears the record; the device stays fully usable.  Lets a deployment
 * (and this library's tests) check the time-out plumbing without any faulting or hanging kernel. */
fq_status fq_watchdog_selftest(uint64_t limit_ns, void* stream);

/* Device-side wait watchdog.  Every spin on an mbarrier inside the kernels is bounded; a wait
 * that expires records a code in a device word and the kernel winds down normally.  This call
 * SYNCHRONISES the device, returns FQ_ERR_TIMEOUT if any kernel recorded an expiry since the
 * last call (and clears the record), else FQ_OK.  *detail (host, may be NULL) gets the raw word. */
fq_status fq_device_status(uint32_t* detail);

#ifdef __cplusplus
}
#endif
#endif /* FQ_H_ */
