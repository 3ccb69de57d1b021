/*
 * FoldQuant linear layer -- CPU ORACLE (test infrastructure, not product code).
 *
 * A plain, slow, step-by-step restatement of the folded quantized linear layer:
 *   offline : fold  W~ = W S R^T  (fold-before transform family, Eq. 3),
 *             round to nearest per output channel, nibble-pack        (Alg. 1 offline half)
 *   runtime : z_t = R S^-1 x_t, per-token symmetric quantization      (Eq. 5)
 *             integer product with int32 accumulation, rescale + bias (Eq. 8, Alg. 1 runtime half)
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call
 * this file.  It shares no code, header, table or helper with the CUDA path.
 *
 * Arithmetic contract (so that integer stages can be compared bit for bit):
 *   - every floating-point step of the transform and the quantizer is one
 *     IEEE-754 binary32 operation, round-to-nearest-even, no fused
 *     multiply-add (build with -ffp-contract=off), denormals preserved;
 *   - butterflies run with ascending stride h = 1, 2, ..., beta/2; the lower
 *     index receives a+b, the upper a-b (natural / Sylvester ordering);
 *   - the epilogue is evaluated in binary64 and rounded once.
 *
 * Readings the paper leaves open (fixed here, "parity unpinned" by the paper
 * itself): ties in round() go to even; two 4-bit codes share a byte with the
 * even channel in the low nibble, two's complement; smoothing-scale floors
 * 1e-5 and bounds [1e-5, 1e5].
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define FQO_F32 0
#define FQO_BF16 1

int fqo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* bfloat16 <-> float. Widening is exact; narrowing rounds to nearest even. */
static float bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static uint16_t f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40u); /* NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

static float load_elem(const void* base, int dtype, int64_t idx) {
    if (dtype == FQO_BF16) return bf16_to_f32(((const uint16_t*)base)[idx]);
    return ((const float*)base)[idx];
}

/* beta = 1 is the identity rotation (R = I: sites that are only scaled, and the identity transforms at
 * graph and engine boundaries); the butterfly loops below then have no stage and beta^(-1/2) = 1. */
static int valid_block(int beta, int64_t K) {
    if (beta < 1 || beta > 256 || (beta & (beta - 1)) != 0) return 0;
    return K > 0 && K % beta == 0;
}

static float qmax_of(int bits) { return bits == 4 ? 7.0f : 127.0f; }

/* Section "Transforms supported by the runtime": unnormalised Sylvester
 * Hadamard product of one block of beta values, in place, by butterflies. */
void fqo_fwht_block(float* v, int beta) {
    for (int h = 1; h < beta; h <<= 1) {
        for (int i = 0; i < beta; ++i) {
            if ((i & h) == 0) {
                float a = v[i];
                float b = v[i + h];
                v[i] = a + b;
                v[i + h] = a - b;
            }
        }
    }
}

/* u = (I (x) H_beta) v over a row of K channels, unnormalised. */
void fqo_fwht_row(float* v, int64_t K, int beta) {
    for (int64_t c0 = 0; c0 < K; c0 += beta) fqo_fwht_block(v + c0, beta);
}

/* Per-channel multiplier that carries both the diagonal factor of the
 * fold-before transform and the beta^(-1/2) normalisation of R.
 *   for_weights = 0 : g_c = (1/s_c) * beta^(-1/2)   (runtime side, S^-1)
 *   for_weights = 1 : g_c =    s_c  * beta^(-1/2)   (offline side, S)
 * smooth == NULL means S = I. */
int fqo_multiplier(const float* smooth, int64_t K, int beta, int for_weights, float* g) {
    if (!valid_block(beta, K) || !g) return 1;
    float c = (float)(1.0 / sqrt((double)beta));
    for (int64_t i = 0; i < K; ++i) {
        if (!smooth) {
            g[i] = c;
        } else if (for_weights) {
            g[i] = smooth[i] * c;
        } else {
            float inv = 1.0f / smooth[i];
            g[i] = inv * c;
        }
    }
    return 0;
}

/* SmoothQuant channel scale s_c = a_c^alpha / w_c^(1-alpha) with floors and
 * bounds (section "Transforms supported by the runtime").  a = calibrated
 * activation max-abs per channel, w = largest weight magnitude per input
 * channel over all consumers of the site.  binary64, cast once. */
int fqo_smooth_scale(const float* a, const float* w, int64_t K, double alpha, float* s) {
    if (!a || !w || !s || alpha < 0.0 || alpha > 1.0) return 1;
    for (int64_t i = 0; i < K; ++i) {
        double ac = a[i] > 1e-5 ? (double)a[i] : 1e-5;
        double wc = w[i] > 1e-5 ? (double)w[i] : 1e-5;
        double v = pow(ac, alpha) / pow(wc, 1.0 - alpha);
        if (v < 1e-5) v = 1e-5;
        if (v > 1e5) v = 1e5;
        s[i] = (float)v;
    }
    return 0;
}

/* Column-wise max |x| over the rows of a [M, K] matrix (calibration statistic). */
int fqo_col_absmax(const void* x, int dtype, int64_t M, int64_t K, int64_t ldx, float* out) {
    if (!x || !out) return 1;
    for (int64_t c = 0; c < K; ++c) out[c] = 0.0f;
    for (int64_t t = 0; t < M; ++t)
        for (int64_t c = 0; c < K; ++c) {
            float v = fabsf(load_elem(x, dtype, t * ldx + c));
            if (v > out[c]) out[c] = v;
        }
    return 0;
}

/* Store one row of signed codes.  4 bits: byte i = code[2i] in the low nibble,
 * code[2i+1] in the high nibble, two's complement.  8 bits: one int8 each. */
static void pack_row(const int* code, int64_t K, int bits, uint8_t* out) {
    if (bits == 4) {
        for (int64_t i = 0; i < K / 2; ++i)
            out[i] = (uint8_t)((code[2 * i] & 0xF) | ((code[2 * i + 1] & 0xF) << 4));
    } else {
        for (int64_t i = 0; i < K; ++i) out[i] = (uint8_t)(int8_t)code[i];
    }
}

static int code_at(const uint8_t* row, int64_t c, int bits) {
    if (bits == 8) return (int)(int8_t)row[c];
    int nib = (row[c >> 1] >> ((c & 1) * 4)) & 0xF;
    return nib >= 8 ? nib - 16 : nib;
}

int fqo_pack(const int32_t* codes, int64_t rows, int64_t K, int bits, uint8_t* out) {
    if ((bits != 4 && bits != 8) || (bits == 4 && (K & 1))) return 1;
    int64_t pitch = K * bits / 8;
    int* tmp = (int*)malloc(sizeof(int) * (size_t)(K > 0 ? K : 1));
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t c = 0; c < K; ++c) tmp[c] = codes[r * K + c];
        pack_row(tmp, K, bits, out + r * pitch);
    }
    free(tmp);
    return 0;
}

int fqo_unpack(const uint8_t* packed, int64_t rows, int64_t K, int bits, int32_t* codes) {
    if ((bits != 4 && bits != 8) || (bits == 4 && (K & 1))) return 1;
    int64_t pitch = K * bits / 8;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < K; ++c) codes[r * K + c] = code_at(packed + r * pitch, c, bits);
    return 0;
}

/* Eq. 5 applied to one already-transformed row u: per-row step
 * delta = (r * max|u|) / q, codes = clip(round(u * (1/delta)), -q, q).
 * A row whose step would fall below the smallest normal float is the zero
 * token: (codes, delta) = (0, 0). */
static float quantize_row(const float* u, int64_t K, int bits, float clip_ratio, int* code) {
    float qf = qmax_of(bits);
    int q = (int)qf;
    float m = 0.0f;
    for (int64_t c = 0; c < K; ++c) {
        float a = fabsf(u[c]);
        if (a > m) m = a;
    }
    float rm = clip_ratio * m;
    float delta = rm / qf;
    if (!(delta >= FLT_MIN)) {
        for (int64_t c = 0; c < K; ++c) code[c] = 0;
        return 0.0f;
    }
    float inv = 1.0f / delta;
    for (int64_t c = 0; c < K; ++c) {
        float scaled = u[c] * inv;
        int v = (int)rintf(scaled); /* default rounding mode: ties to even */
        if (v > q) v = q;
        if (v < -q) v = -q;
        code[c] = v;
    }
    return delta;
}

/* Runtime prologue (Alg. 1, runtime half, first two lines): for each token
 * z_t = R S^-1 x_t then Eq. 5.  g is the runtime multiplier of
 * fqo_multiplier(for_weights = 0), or NULL for S = I.
 * If z_out != NULL it receives the transformed rows [M, K] (for tests). */
int fqo_quantize_act(const void* x, int dtype, int64_t M, int64_t K, int64_t ldx, const float* g,
                     int beta, int bits, float clip_ratio, uint8_t* codes, float* delta,
                     float* z_out) {
    if (!valid_block(beta, K) || (bits != 4 && bits != 8)) return 1;
    if (!(clip_ratio > 0.0f && clip_ratio <= 1.0f)) return 1;
    if (M < 0 || ldx < K || (M > 0 && (!x || !codes || !delta))) return 1;
    float c = (float)(1.0 / sqrt((double)beta));
    int64_t pitch = K * bits / 8;
#pragma omp parallel
    {
        float* v = (float*)malloc(sizeof(float) * (size_t)K);
        int* code = (int*)malloc(sizeof(int) * (size_t)K);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < M; ++t) {
            for (int64_t i = 0; i < K; ++i) {
                float xv = load_elem(x, dtype, t * ldx + i);
                float gi = g ? g[i] : c;
                v[i] = xv * gi;
            }
            fqo_fwht_row(v, K, beta);
            if (z_out) memcpy(z_out + t * K, v, sizeof(float) * (size_t)K);
            delta[t] = quantize_row(v, K, bits, clip_ratio, code);
            pack_row(code, K, bits, codes + t * pitch);
        }
        free(v);
        free(code);
    }
    return 0;
}

/* The whole transform family of the section "Transforms supported by the runtime":
 * T = D^o R D^i with positive diagonals, z = D^o (R (D^i x)), followed by Eq. 5.
 *   pre  (optional) = d^i_c * beta^(-1/2) per channel, applied before the butterflies
 *                     (NULL: the constant beta^(-1/2), i.e. D^i = I);
 *   post (optional) = d^o_c per channel, applied after them (NULL: D^o = I).
 * Fold-before is (pre, NULL), fold-after is (NULL, post).  With post == NULL this is
 * fqo_quantize_act operation for operation.  z_out (optional) receives z [M, K]. */
int fqo_transform_quantize(const void* x, int dtype, int64_t M, int64_t K, int64_t ldx, const float* pre,
                           const float* post, int beta, int bits, float clip_ratio, uint8_t* codes,
                           float* delta, float* z_out) {
    if (!valid_block(beta, K) || (bits != 4 && bits != 8)) return 1;
    if (!(clip_ratio > 0.0f && clip_ratio <= 1.0f)) return 1;
    if (M < 0 || ldx < K || (M > 0 && (!x || !codes || !delta))) return 1;
    float c = (float)(1.0 / sqrt((double)beta));
    int64_t pitch = K * bits / 8;
#pragma omp parallel
    {
        float* v = (float*)malloc(sizeof(float) * (size_t)K);
        int* code = (int*)malloc(sizeof(int) * (size_t)K);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < M; ++t) {
            for (int64_t i = 0; i < K; ++i) {
                float xv = load_elem(x, dtype, t * ldx + i);
                float gi = pre ? pre[i] : c;
                v[i] = xv * gi;
            }
            fqo_fwht_row(v, K, beta);
            if (post)
                for (int64_t i = 0; i < K; ++i) v[i] = v[i] * post[i];
            if (z_out) memcpy(z_out + t * K, v, sizeof(float) * (size_t)K);
            delta[t] = quantize_row(v, K, bits, clip_ratio, code);
            pack_row(code, K, bits, codes + t * pitch);
        }
        free(v);
        free(code);
    }
    return 0;
}

/* Stored composite rotation (section "Transforms supported by the runtime": optional for the action
 * expert -- a channel permutation followed by one stored dense matrix per block of beta channels):
 *   R = blockdiag(B_0 .. B_{K/beta-1}) Pi,   z = R (d (.) x),   then Eq. 5.
 *   pre  (optional) = the input diagonal d (1/s at run time, s when folding weights); NULL = 1;
 *   perm[c]         = source channel of position c: p_c = v[perm[c]];
 *   blocks          = [K/beta][beta][beta] row-major, u[b*beta + i] = sum_j B_b[i][j] * p[b*beta + j].
 * The normalisation lives inside the stored matrices (no beta^(-1/2) factor here).  binary32: one
 * multiply for the diagonal, then one fused multiply-add per term in ascending j, starting from 0.
 * Applied to weight rows with pre = s this is the offline fold: row j of W~ = W S R^T is R (s (.) w_j)
 * for any real R.  z_out (optional) receives z [M, K]. */
int fqo_composite_quantize(const void* x, int dtype, int64_t M, int64_t K, int64_t ldx, const float* pre,
                           const int32_t* perm, const float* blocks, int beta, int bits, float clip_ratio,
                           uint8_t* codes, float* delta, float* z_out) {
    if (beta < 1 || beta > 256 || K <= 0 || K % beta != 0 || (bits != 4 && bits != 8)) return 1;
    if (!(clip_ratio > 0.0f && clip_ratio <= 1.0f) || !perm || !blocks) return 1;
    if (M < 0 || ldx < K || (M > 0 && (!x || !codes || !delta))) return 1;
    for (int64_t c = 0; c < K; ++c)
        if (perm[c] < 0 || perm[c] >= K) return 1;
    int64_t pitch = K * bits / 8;
#pragma omp parallel
    {
        float* v = (float*)malloc(sizeof(float) * (size_t)K);
        float* u = (float*)malloc(sizeof(float) * (size_t)K);
        int* code = (int*)malloc(sizeof(int) * (size_t)K);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < M; ++t) {
            for (int64_t c = 0; c < K; ++c) {
                float xv = load_elem(x, dtype, t * ldx + c);
                v[c] = pre ? xv * pre[c] : xv;
            }
            for (int64_t b = 0; b < K / beta; ++b) {
                const float* B = blocks + b * (int64_t)beta * beta;
                for (int i = 0; i < beta; ++i) {
                    float acc = 0.0f;
                    for (int j = 0; j < beta; ++j) acc = fmaf(B[i * beta + j], v[perm[b * beta + j]], acc);
                    u[b * beta + i] = acc;
                }
            }
            if (z_out) memcpy(z_out + t * K, u, sizeof(float) * (size_t)K);
            delta[t] = quantize_row(u, K, bits, clip_ratio, code);
            pack_row(code, K, bits, codes + t * pitch);
        }
        free(v);
        free(u);
        free(code);
    }
    return 0;
}

/* Fold-after, offline half: W~ = W R^T P, row j = (R w_j) (.) p (the block Hadamard matrix is
 * symmetric), then RTN as in fqo_fold_weights.  mult_post (optional) receives the RUNTIME
 * post-rotation multiplier 1/p_c (one binary32 division per channel); at run time the
 * pre-rotation factor is the constant beta^(-1/2).  wt_out (optional) receives W~. */
int fqo_fold_weights_after(const void* W, int dtype, int64_t N, int64_t K, int64_t ldw, const float* p,
                           int beta, int bits, uint8_t* codes, float* w_scale, float* mult_post,
                           float* wt_out) {
    if (!p) return 1;
    if (mult_post)
        for (int64_t i = 0; i < K; ++i) mult_post[i] = 1.0f / p[i];
    return fqo_transform_quantize(W, dtype, N, K, ldw, NULL, p, beta, bits, 1.0f, codes, w_scale, wt_out);
}

/* Offline half of Alg. 1 for one consumer with round-to-nearest:
 * row j of W~ = W S R^T is R (s (.) w_j) because the block Hadamard matrix is
 * symmetric.  Per-output-channel step s^W_j = max|W~_j| / q, no clipping.
 * mult_g (optional) receives the matching RUNTIME multiplier (1/s)*beta^-1/2.
 * wt_out (optional) receives W~ [N, K] in float (for tests). */
int fqo_fold_weights(const void* W, int dtype, int64_t N, int64_t K, int64_t ldw,
                     const float* smooth, int beta, int bits, uint8_t* codes, float* w_scale,
                     float* mult_g, float* wt_out) {
    if (!valid_block(beta, K) || (bits != 4 && bits != 8)) return 1;
    if (N < 0 || ldw < K || (N > 0 && (!W || !codes || !w_scale))) return 1;
    float* gw = (float*)malloc(sizeof(float) * (size_t)K);
    fqo_multiplier(smooth, K, beta, 1, gw);
    if (mult_g) fqo_multiplier(smooth, K, beta, 0, mult_g);
    int64_t pitch = K * bits / 8;
#pragma omp parallel
    {
        float* v = (float*)malloc(sizeof(float) * (size_t)K);
        int* code = (int*)malloc(sizeof(int) * (size_t)K);
#pragma omp for schedule(static)
        for (int64_t j = 0; j < N; ++j) {
            for (int64_t i = 0; i < K; ++i) v[i] = load_elem(W, dtype, j * ldw + i) * gw[i];
            fqo_fwht_row(v, K, beta);
            if (wt_out) memcpy(wt_out + j * K, v, sizeof(float) * (size_t)K);
            w_scale[j] = quantize_row(v, K, bits, 1.0f, code);
            pack_row(code, K, bits, codes + j * pitch);
        }
        free(v);
        free(code);
    }
    free(gw);
    return 0;
}

/* Integer product of Eq. 8: acc[t][j] = sum_c qA[t][c] * qW[j][c], summed in
 * 64 bits and required to fit 32.  Returns 2 if any sum does not fit. */
int fqo_gemm_i32(const uint8_t* a_codes, const uint8_t* w_codes, int64_t M, int64_t N, int64_t K,
                 int bits, int32_t* acc) {
    if ((bits != 4 && bits != 8) || (K & 1)) return 1;
    int64_t pitch = K * bits / 8;
    int overflow = 0;
#pragma omp parallel
    {
        int* arow = (int*)malloc(sizeof(int) * (size_t)(K > 0 ? K : 1));
#pragma omp for schedule(static) reduction(| : overflow)
        for (int64_t t = 0; t < M; ++t) {
            for (int64_t c = 0; c < K; ++c) arow[c] = code_at(a_codes + t * pitch, c, bits);
            for (int64_t j = 0; j < N; ++j) {
                const uint8_t* wrow = w_codes + j * pitch;
                int64_t s = 0;
                for (int64_t c = 0; c < K; ++c) s += (int64_t)arow[c] * (int64_t)code_at(wrow, c, bits);
                if (s > INT32_MAX || s < INT32_MIN) overflow = 1;
                acc[t * N + j] = (int32_t)s;
            }
        }
        free(arow);
    }
    return overflow ? 2 : 0;
}

/* Rescale + bias of Eq. 8: y[t][j] = s^W_j * delta_t * acc[t][j] + b_j in
 * binary64, rounded once to the output type.  bias == NULL means b = 0. */
int fqo_epilogue(const int32_t* acc, const float* delta, const float* w_scale, const float* bias,
                 int64_t M, int64_t N, void* y, int ydtype, int64_t ldy) {
    if (ldy < N) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < M; ++t) {
        for (int64_t j = 0; j < N; ++j) {
            double v = (double)w_scale[j] * (double)delta[t] * (double)acc[t * N + j] +
                       (bias ? (double)bias[j] : 0.0);
            float f = (float)v;
            if (ydtype == FQO_BF16)
                ((uint16_t*)y)[t * ldy + j] = f32_to_bf16(f);
            else
                ((float*)y)[t * ldy + j] = f;
        }
    }
    return 0;
}

/* Weight-only low-bit projection with floating-point activations (section "Problem statement": in
 * the W4A4 engines the adaptive layer-normalisation modulation keeps its activations in floating
 * point and only its weights are 4-bit).  With the weight reconstruction W^_jc = s^W_j qW_jc of Eq. 8:
 *   y[t][j] = s^W_j * sum_c qW[j][c] * x[t][c] + b_j,
 * products and sum in binary64 in channel order, rounded once to the output type. */
int fqo_linear_wonly(const void* x, int xdtype, int64_t M, int64_t K, int64_t ldx, const uint8_t* w_codes,
                     const float* w_scale, const float* bias, int64_t N, int bits, void* y, int ydtype,
                     int64_t ldy) {
    if ((bits != 4 && bits != 8) || (K & 1) || ldx < K || ldy < N) return 1;
    int64_t pitch = K * bits / 8;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < M; ++t) {
        for (int64_t j = 0; j < N; ++j) {
            const uint8_t* wrow = w_codes + j * pitch;
            double s = 0.0;
            for (int64_t c = 0; c < K; ++c)
                s += (double)code_at(wrow, c, bits) * (double)load_elem(x, xdtype, t * ldx + c);
            double v = (double)w_scale[j] * s + (bias ? (double)bias[j] : 0.0);
            float f = (float)v;
            if (ydtype == FQO_BF16)
                ((uint16_t*)y)[t * ldy + j] = f32_to_bf16(f);
            else
                ((float*)y)[t * ldy + j] = f;
        }
    }
    return 0;
}

/* ---- gated-MLP product ahead of down_proj's quantizer ---------------------------------------------
 * The site feeding down_proj holds h = act(gate) (.) up (section "Normalization gains" names the gated
 * MLP and its gate non-linearity without fixing it; the two in use by the policies' language models are
 * SiLU and the tanh form of GELU).  Both are x * sigmoid(k): k = x for SiLU, k = 2 sqrt(2/pi) (x + 0.044715 x^3)
 * for GELU-tanh (0.5 (1 + tanh u) = sigmoid(2u)).  Because h feeds a quantizer, its arithmetic is fixed in
 * binary32 and the device takes the same steps:
 *   e = exp(-k): argument clamped to [-87, 88]; n = rint(a * log2e); r = fma(n, -ln2_hi, a); r = fma(n, -ln2_lo, r);
 *       degree-6 Taylor polynomial in Horner form with fused multiply-adds; times 2^n built from its exponent bits;
 *   act = x / (1 + e);   h = act * up.
 * gate_up [M][2K]: gate in columns [0, K), up in [K, 2K) (the layout of a fused gate/up projection). */
static float exp_fixed(float a) {
    if (a < -87.0f) a = -87.0f;
    if (a > 88.0f) a = 88.0f;
    float n = rintf(a * 1.44269504f);
    float r = fmaf(n, -0.693145752f, a);
    r = fmaf(n, -1.42860677e-06f, r);
    float p = 1.38888892e-03f;
    p = fmaf(p, r, 8.33333377e-03f);
    p = fmaf(p, r, 4.16666679e-02f);
    p = fmaf(p, r, 1.66666672e-01f);
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    int32_t bits = ((int32_t)n + 127) << 23;
    float s;
    memcpy(&s, &bits, 4);
    return p * s;
}

float fqo_gate_act(float x, int act) {
    float k = x;
    if (act == 1) {                                  /* GELU, tanh form */
        float x2 = x * x;
        float x3 = x2 * x;
        float inner = fmaf(0.044715f, x3, x);
        k = 1.59576917f * inner;
    }
    float e = exp_fixed(-k);
    return x / (1.0f + e);
}

int fqo_gated_product(const void* gate_up, int dtype, int64_t M, int64_t K, int64_t ld, int act, float* h) {
    if (!gate_up || !h || M < 0 || K <= 0 || ld < 2 * K || (act != 0 && act != 1)) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < M; ++t)
        for (int64_t c = 0; c < K; ++c) {
            float g = load_elem(gate_up, dtype, t * ld + c);
            float u = load_elem(gate_up, dtype, t * ld + K + c);
            h[t * K + c] = fqo_gate_act(g, act) * u;
        }
    return 0;
}

/* ---- GPTQ rounding in transformed coordinates (section "Rounding and native execution", Eq. 7) ----
 * min_Q ||(W~ - Q) Z||_F^2 with G = Z Z^T (Z: transformed calibration tokens as columns; here the tokens
 * are the ROWS of z[Mc][K]) and diagonal damping, solved approximately by the published GPTQ sweep:
 * channels are rounded one after the other and each rounding error is spread over the channels not yet
 * rounded, along the rows of the upper Cholesky factor U of H^-1 (H^-1 = U^T U), H = G + lambda I.
 * All arithmetic is binary32 in a fixed order (fused multiply-add chains in ascending index), because it
 * decides integer codes: the device path takes the same steps in the same order.
 *
 * fqo_gptq_factor:  G[a][b] = sum_t z[t][a] z[t][b];  lambda = damp * mean(diag G);
 *   a channel with G[a][a] = 0 is dead (never active in calibration): H[a][a] = 1, reported in dead[a];
 *   H = M M^T with M upper triangular (columns from the last to the first), U = M^-1 (upper triangular),
 *   so that H^-1 = U^T U.  U is written row-major [K][K] (zeros below the diagonal).  Returns 3 if H is
 *   not positive definite in binary32. */
int fqo_gptq_factor(const float* z, int64_t Mc, int64_t K, float damp, float* U, uint8_t* dead) {
    if (!z || !U || !dead || Mc < 0 || K <= 0 || !(damp >= 0.0f)) return 1;
    float* H = (float*)malloc(sizeof(float) * (size_t)K * (size_t)K);
    float* Mu = (float*)malloc(sizeof(float) * (size_t)K * (size_t)K);   /* Mu[i][k], k >= i */
    if (!H || !Mu) { free(H); free(Mu); return 1; }
#pragma omp parallel for schedule(static)
    for (int64_t a = 0; a < K; ++a)
        for (int64_t b = 0; b < K; ++b) {
            float acc = 0.0f;
            for (int64_t t = 0; t < Mc; ++t) acc = fmaf(z[t * K + a], z[t * K + b], acc);
            H[a * K + b] = acc;
        }
    float sum = 0.0f;
    for (int64_t a = 0; a < K; ++a) sum = sum + H[a * K + a];
    float lambda = damp * (sum / (float)K);
    for (int64_t a = 0; a < K; ++a) {
        dead[a] = H[a * K + a] == 0.0f;
        if (dead[a]) H[a * K + a] = 1.0f;
        H[a * K + a] = H[a * K + a] + lambda;
    }
    memset(Mu, 0, sizeof(float) * (size_t)K * (size_t)K);
    int bad = 0;
    for (int64_t j = K - 1; j >= 0; --j) {
        float acc = H[j * K + j];
        for (int64_t k = j + 1; k < K; ++k) acc = fmaf(-Mu[j * K + k], Mu[j * K + k], acc);
        if (!(acc > 0.0f)) { bad = 1; break; }
        float d = sqrtf(acc);
        Mu[j * K + j] = d;
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < j; ++i) {
            float a2 = H[i * K + j];
            for (int64_t k = j + 1; k < K; ++k) a2 = fmaf(-Mu[i * K + k], Mu[j * K + k], a2);
            Mu[i * K + j] = a2 / d;
        }
    }
    if (!bad) {
        memset(U, 0, sizeof(float) * (size_t)K * (size_t)K);
#pragma omp parallel for schedule(dynamic, 8)
        for (int64_t c = 0; c < K; ++c) {           /* column c of U: M U = I, from row c upwards */
            U[c * K + c] = 1.0f / Mu[c * K + c];
            for (int64_t i = c - 1; i >= 0; --i) {
                float acc = 0.0f;
                for (int64_t k = i + 1; k <= c; ++k) acc = fmaf(Mu[i * K + k], U[k * K + c], acc);
                U[i * K + c] = -acc / Mu[i * K + i];
            }
        }
    }
    free(H);
    free(Mu);
    return bad ? 3 : 0;
}

/* fqo_gptq_round: the sweep.  Wt [N][K] (modified in place), per-output-channel steps w_scale[N] taken
 * from the unmodified W~ (max|row| / q), codes[N][K] as ints.  For channel i = 0 .. K-1 and every row r:
 *   w = Wt[r][i] (0 if the channel is dead);  code = clip(rint(w * (1 / s_r)), -q, q);  e = (w - code * s_r) / U[i][i];
 *   Wt[r][j] = fma(-e, U[i][j], Wt[r][j]) for j > i.        A row with s_r = 0 gets zero codes. */
int fqo_gptq_round(float* Wt, int64_t N, int64_t K, const float* U, const uint8_t* dead, const float* w_scale,
                   int q, int* codes) {
    if (!Wt || !U || !dead || !w_scale || !codes || N < 0 || K <= 0) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N; ++r) {
        float s = w_scale[r];
        float inv = s >= FLT_MIN ? 1.0f / s : 0.0f;
        float* w = Wt + r * K;
        for (int64_t i = 0; i < K; ++i) {
            float wi = dead[i] ? 0.0f : w[i];
            int v = (int)rintf(wi * inv);
            if (v > q) v = q;
            if (v < -q) v = -q;
            codes[r * K + i] = v;
            float e = (wi - (float)v * s) / U[i * K + i];
            for (int64_t j = i + 1; j < K; ++j) w[j] = fmaf(-e, U[i * K + j], w[j]);
        }
    }
    return 0;
}

/* Whole runtime path for one consumer: prologue, integer product, epilogue.
 * rows_sel (optional, n_sel entries) restricts the integer product and the
 * epilogue to those token rows (output then has n_sel rows); the prologue
 * always runs on all M rows. acc_out is optional. */
int fqo_linear(const void* x, int xdtype, int64_t M, int64_t K, int64_t ldx, const float* g, int beta,
               int bits, float clip_ratio, const uint8_t* w_codes, const float* w_scale,
               const float* bias, int64_t N, const int64_t* rows_sel, int64_t n_sel, void* y,
               int ydtype, int64_t ldy, uint8_t* a_codes_out, float* delta_out, int32_t* acc_out) {
    int64_t pitch = K * bits / 8;
    uint8_t* codes = a_codes_out ? a_codes_out : (uint8_t*)malloc((size_t)(M * pitch + 1));
    float* delta = delta_out ? delta_out : (float*)malloc(sizeof(float) * (size_t)(M + 1));
    int rc = fqo_quantize_act(x, xdtype, M, K, ldx, g, beta, bits, clip_ratio, codes, delta, NULL);
    if (rc == 0) {
        int64_t Ms = rows_sel ? n_sel : M;
        uint8_t* ca = codes;
        float* da = delta;
        if (rows_sel) {
            ca = (uint8_t*)malloc((size_t)(Ms * pitch + 1));
            da = (float*)malloc(sizeof(float) * (size_t)(Ms + 1));
            for (int64_t i = 0; i < Ms; ++i) {
                memcpy(ca + i * pitch, codes + rows_sel[i] * pitch, (size_t)pitch);
                da[i] = delta[rows_sel[i]];
            }
        }
        int32_t* acc = acc_out ? acc_out : (int32_t*)malloc(sizeof(int32_t) * (size_t)(Ms * N + 1));
        rc = fqo_gemm_i32(ca, w_codes, Ms, N, K, bits, acc);
        if (rc == 0) rc = fqo_epilogue(acc, da, w_scale, bias, Ms, N, y, ydtype, ldy);
        if (!acc_out) free(acc);
        if (rows_sel) {
            free(ca);
            free(da);
        }
    }
    if (!a_codes_out) free(codes);
    if (!delta_out) free(delta);
    return rc;
}
