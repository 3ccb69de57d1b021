// Runtime prologue of a projection site (Alg. 1 runtime half, lines 1-2):
//   v = x (.) g            per-channel multiplier (S^-1 and block^-1/2 folded together)
//   u = (I (x) H_block) v  block Hadamard by FWHT, ascending strides
//   delta = (r max|u|)/q   per-token step (Eq. 5)
//   code = clip(round(u * (1/delta)), -q, q), packed
// The same kernel performs the offline fold of a weight row (row j of W S R^T is
// R (s (.) w_j)), so folded weights and runtime activations share one butterfly
// network bit for bit.
//
// Every floating-point step is a single IEEE binary32 operation issued through
// the __f*_rn intrinsics, which the compiler never contracts into FMAs; the one
// FMA used (own * (+-1) + partner) is exact in its product and therefore rounds
// exactly like the add/sub it replaces.
//
// Work decomposition: a thread owns E consecutive channels of one token, a row
// of K channels is spread over K/E threads (rounded up to whole warps), strides
// below E run in registers, strides E..block/2 by warp shuffles.  The whole
// token stays in registers between the absmax reduction and the quantizer, so x
// is read once and nothing but codes and steps is written.
#include <cuda_bf16.h>
#include <float.h>

#include "fq_common.cuh"
#include "ptx_sm100.cuh"
#include "act_common.cuh"

namespace fq {
namespace {

constexpr int kMaxThreads = 1024;

template <typename XT, int E>
struct RawRow;

template <int E>
struct RawRow<float, E> {
    float4 q[E / 4];
    __device__ __forceinline__ void load(const float* p, bool pred) {
#pragma unroll
        for (int i = 0; i < E / 4; ++i)
            q[i] = pred ? __ldg(reinterpret_cast<const float4*>(p) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    __device__ __forceinline__ void widen(float* v) const {
#pragma unroll
        for (int i = 0; i < E / 4; ++i) {
            v[4 * i + 0] = q[i].x;
            v[4 * i + 1] = q[i].y;
            v[4 * i + 2] = q[i].z;
            v[4 * i + 3] = q[i].w;
        }
    }
};

template <int E>
struct RawRow<__nv_bfloat16, E> {
    uint4 q[E / 8];
    __device__ __forceinline__ void load(const __nv_bfloat16* p, bool pred) {
#pragma unroll
        for (int i = 0; i < E / 8; ++i)
            q[i] = pred ? __ldg(reinterpret_cast<const uint4*>(p) + i) : make_uint4(0u, 0u, 0u, 0u);
    }
    __device__ __forceinline__ void widen(float* v) const {
#pragma unroll
        for (int i = 0; i < E / 8; ++i) {
            const uint32_t w[4] = {q[i].x, q[i].y, q[i].z, q[i].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[8 * i + 2 * j + 0] = __uint_as_float(w[j] << 16);          // bf16 -> f32 is exact
                v[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
            }
        }
    }
};

// Gate non-linearity of a gated MLP in fixed binary32 arithmetic: act(x) = x * sigmoid(k), k = x (SiLU) or
// k = 2 sqrt(2/pi) (x + 0.044715 x^3) (GELU, tanh form).  exp(-k): argument clamped to [-87, 88], n = rint(a log2e),
// two-step reduction by ln2, degree-6 Taylor polynomial in Horner form, times 2^n from its exponent bits.  The
// product act(gate) * up feeds a quantizer, so every operation and its order are part of the definition.
__device__ __forceinline__ float exp_fixed(float a) {
    a = fminf(fmaxf(a, -87.0f), 88.0f);
    const float n = rintf(__fmul_rn(a, 1.44269504f));
    float r = __fmaf_rn(n, -0.693145752f, a);
    r = __fmaf_rn(n, -1.42860677e-06f, r);
    float p = 1.38888892e-03f;
    p = __fmaf_rn(p, r, 8.33333377e-03f);
    p = __fmaf_rn(p, r, 4.16666679e-02f);
    p = __fmaf_rn(p, r, 1.66666672e-01f);
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    return __fmul_rn(p, __int_as_float(((int)n + 127) << 23));
}
__device__ __forceinline__ float gate_act(float x, int kind) {
    float k = x;
    if (kind == 1) {
        const float x3 = __fmul_rn(__fmul_rn(x, x), x);
        k = __fmul_rn(1.59576917f, __fmaf_rn(0.044715f, x3, x));
    }
    return __fdiv_rn(x, __fadd_rn(1.0f, exp_fixed(-k)));
}

// FMT: 0 = two 4-bit codes per byte, 1 = one int8 per code.  CLAMP: clip_ratio < 1.
// GATED (lean variant only): the row is [gate | up] with 2K columns and the kernel's input is
// act(gate) * up (the site behind a gated MLP), gate_kind 0 = SiLU, 1 = GELU-tanh.
// CACHE: keep the multiplier slice in registers across tokens and prefetch the next
// token (thread blocks of at most 512 threads); otherwise a lean variant for up to
// 1024 threads that re-reads the multiplier (L1/L2 resident) for every token.
template <typename XT, int E, int FMT, bool CLAMP, bool CACHE, bool GATED = false>
__global__ void __launch_bounds__(CACHE ? 512 : kMaxThreads)
transform_quantize_kernel(const XT* __restrict__ x, int64_t rows, int K, int64_t ldx,
                          const float* __restrict__ mult, float cnorm, int block, float qmax,
                          float clip_ratio, uint8_t* __restrict__ codes, float* __restrict__ delta,
                          int tpr, int rpc, int mult_after, int gate_kind) {
    __shared__ float s_part[2][32];   // per-warp partial maxima, double buffered

    griddep_wait();                   // launched with programmatic serialization: see launch_pdl
    griddep_launch_dependents();
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int r_in_cta = tid / tpr;
    const int t_in_row = tid - r_in_cta * tpr;
    const int wpr = tpr >> 5;                       // warps per row
    const int col0 = t_in_row * E;
    const bool col_ok = col0 < K;

    float g[CACHE ? E : 1];
    if (CACHE) {
        if (mult != nullptr && col_ok) {
#pragma unroll
            for (int i = 0; i < E / 4; ++i) {
                float4 t = __ldg(reinterpret_cast<const float4*>(mult + col0) + i);
                g[(4 * i + 0) % (CACHE ? E : 1)] = t.x; g[(4 * i + 1) % (CACHE ? E : 1)] = t.y;
                g[(4 * i + 2) % (CACHE ? E : 1)] = t.z; g[(4 * i + 3) % (CACHE ? E : 1)] = t.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < (CACHE ? E : 1); ++i) g[i] = cnorm;
        }
    }

    const int64_t row_step = (int64_t)gridDim.x * rpc;
    int64_t row = (int64_t)blockIdx.x * rpc + r_in_cta;
    RawRow<XT, E> raw;
    if (CACHE) raw.load(x + row * ldx + col0, col_ok && row < rows);

    int buf = 0;
    for (int64_t rb = (int64_t)blockIdx.x * rpc; rb < rows; rb += row_step, row += row_step, buf ^= 1) {
        float v[E];
        const bool row_ok = col_ok && row < rows;
        if (CACHE) {
            raw.widen(v);
            // prefetch the next token while this one is transformed
            const int64_t nrow = row + row_step;
            raw.load(x + nrow * ldx + col0, col_ok && nrow < rows);
#pragma unroll
            for (int i = 0; i < E; ++i) v[i] = __fmul_rn(v[i], mult_after ? cnorm : g[i % (CACHE ? E : 1)]);
        } else {
            raw.load(x + row * ldx + col0, row_ok);
            raw.widen(v);
            if (GATED) {
                RawRow<XT, E> up;
                up.load(x + row * ldx + K + col0, row_ok);
                float u[E];
                up.widen(u);
#pragma unroll
                for (int i = 0; i < E; ++i) v[i] = __fmul_rn(gate_act(v[i], gate_kind), u[i]);
            }
            if (mult != nullptr && col_ok && !mult_after) {
#pragma unroll
                for (int i = 0; i < E / 4; ++i) {
                    const float4 t = __ldg(reinterpret_cast<const float4*>(mult + col0) + i);
                    v[4 * i + 0] = __fmul_rn(v[4 * i + 0], t.x);
                    v[4 * i + 1] = __fmul_rn(v[4 * i + 1], t.y);
                    v[4 * i + 2] = __fmul_rn(v[4 * i + 2], t.z);
                    v[4 * i + 3] = __fmul_rn(v[4 * i + 3], t.w);
                }
            } else {
#pragma unroll
                for (int i = 0; i < E; ++i) v[i] = __fmul_rn(v[i], cnorm);
            }
        }

        // strides 1 .. E/2: registers
#pragma unroll
        for (int h = 1; h < E; h <<= 1) {
            if (h < block) {
#pragma unroll
                for (int i = 0; i < E; ++i) {
                    if ((i & h) == 0) {
                        const float a = v[i], b = v[i + h];
                        v[i] = __fadd_rn(a, b);
                        v[i + h] = __fsub_rn(a, b);
                    }
                }
            }
        }
        // strides E .. block/2: partner lane = lane ^ (h / E); upper lane keeps partner - own
        for (int h = E; h < block; h <<= 1) {
            const int lm = h / E;
            const float sgn = (lane & lm) ? -1.0f : 1.0f;
#pragma unroll
            for (int i = 0; i < E; ++i) {
                const float p = __shfl_xor_sync(0xffffffffu, v[i], lm);
                v[i] = __fmaf_rn(v[i], sgn, p);
            }
        }
        // fold-after sites: the diagonal sits behind the rotation (z = D^o R x)
        if (mult_after) {
            if (CACHE) {
#pragma unroll
                for (int i = 0; i < E; ++i) v[i] = __fmul_rn(v[i], g[i % (CACHE ? E : 1)]);
            } else if (col_ok) {
#pragma unroll
                for (int i = 0; i < E / 4; ++i) {
                    const float4 t = __ldg(reinterpret_cast<const float4*>(mult + col0) + i);
                    v[4 * i + 0] = __fmul_rn(v[4 * i + 0], t.x);
                    v[4 * i + 1] = __fmul_rn(v[4 * i + 1], t.y);
                    v[4 * i + 2] = __fmul_rn(v[4 * i + 2], t.z);
                    v[4 * i + 3] = __fmul_rn(v[4 * i + 3], t.w);
                }
            }
        }

        // per-token max |u|
        float m = 0.0f;
#pragma unroll
        for (int i = 0; i < E; ++i) m = fmaxf(m, fabsf(v[i]));
        m = warp_max_nonneg(m);
        if (wpr > 1) {
            if (lane == 0) s_part[buf][warp] = m;
            __syncthreads();
            const int w0 = r_in_cta * wpr;
            m = (lane < wpr) ? s_part[buf][w0 + lane] : 0.0f;
            m = warp_max_nonneg(m);
        }

        // Eq. 5 step; a token whose step is below the smallest normal float is the zero token
        float d = __fdiv_rn(__fmul_rn(clip_ratio, m), qmax);
        float inv;
        if (d >= FLT_MIN) {
            inv = __fdiv_rn(1.0f, d);
        } else {
            d = 0.0f;
            inv = 0.0f;
        }

        // round to nearest even through the 1.5*2^23 trick: the low mantissa bits of
        // (t + 12582912) hold the two's-complement integer rint(t) for |t| < 2^22
        constexpr int kPer = FMT == 0 ? 8 : 4;               // codes per 32-bit word
        uint32_t w[E / kPer];
#pragma unroll
        for (int j = 0; j < E / kPer; ++j) {
            uint32_t b[kPer];
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                float t = __fmul_rn(v[code_index<FMT>(j, i)], inv);
                if (CLAMP) t = fminf(fmaxf(t, -qmax), qmax);
                b[i] = __float_as_uint(__fadd_rn(t, 12582912.0f));
            }
            w[j] = pack_word<FMT>(b);
        }
        if (row_ok) {
            if (FMT == 0) {
                uint8_t* dst = codes + row * (int64_t)(K / 2) + col0 / 2;
                if (E == 8) {
                    *reinterpret_cast<uint32_t*>(dst) = w[0];
                } else {
#pragma unroll
                    for (int i = 0; i < E / 16; ++i)
                        reinterpret_cast<uint2*>(dst)[i] = make_uint2(w[2 * i], w[2 * i + 1]);
                }
            } else {
                uint8_t* dst = codes + row * (int64_t)K + col0;
                if (E == 8) {
                    *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
                } else {
#pragma unroll
                    for (int i = 0; i < E / 16; ++i)
                        reinterpret_cast<uint4*>(dst)[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
                }
            }
            if (t_in_row == 0) delta[row] = d;
        }
    }
}

template <typename XT, int E, int FMT>
cudaError_t launch_e(const XT* x, int64_t rows, int K, int64_t ldx, const float* mult, float cnorm, int mult_after,
                     int block, int qmax, float clip_ratio, void* codes, float* delta, cudaStream_t stream, int gate = -1) {
    const int tpr = ((K / E) + 31) / 32 * 32;
    if (tpr > kMaxThreads) return cudaErrorInvalidConfiguration;
    int rpc = 256 / tpr;
    if (rpc < 1) rpc = 1;
    const int threads = tpr * rpc;
    const int sms = device_sm_count();
    const int64_t iters = (rows + rpc - 1) / rpc;
    auto args = [&](auto kern) {
        const int resident = max_resident_blocks(reinterpret_cast<const void*>(kern), threads);
        int64_t grid = iters < (int64_t)sms * resident ? iters : (int64_t)sms * resident;
        if (grid < 1) grid = 1;
        launch_pdl(kern, (unsigned)grid, (unsigned)threads, 0, stream, 1u, x, rows, K, ldx, mult, cnorm, block, (float)qmax,
                   clip_ratio, static_cast<uint8_t*>(codes), delta, tpr, rpc, mult_after, gate);
    };
    const bool clamp = clip_ratio < 1.0f;
    if (gate >= 0) {
        if (clamp) args(transform_quantize_kernel<XT, E, FMT, true, false, true>);
        else args(transform_quantize_kernel<XT, E, FMT, false, false, true>);
    } else if (threads <= 512) {
        if (clamp) args(transform_quantize_kernel<XT, E, FMT, true, true>);
        else args(transform_quantize_kernel<XT, E, FMT, false, true>);
    } else {
        if (clamp) args(transform_quantize_kernel<XT, E, FMT, true, false>);
        else args(transform_quantize_kernel<XT, E, FMT, false, false>);
    }
    return cudaGetLastError();
}

template <typename XT, int FMT>
cudaError_t launch_t(const XT* x, int64_t rows, int K, int64_t ldx, const float* mult, float cnorm, int mult_after,
                     int block, int qmax, float clip_ratio, void* codes, float* delta, cudaStream_t stream, int gate = -1) {
    // E = 8 keeps short rows spread over a full warp; E = 16 is the streaming default;
    // E = 32 holds K = 16384 in 512 threads (cached variant) and reaches K = 32768 in 1024.
    if (K % 16 != 0 || K <= 256)
        return launch_e<XT, 8, FMT>(x, rows, K, ldx, mult, cnorm, mult_after, block, qmax, clip_ratio, codes, delta, stream, gate);
    if (K <= 8192)
        return launch_e<XT, 16, FMT>(x, rows, K, ldx, mult, cnorm, mult_after, block, qmax, clip_ratio, codes, delta, stream, gate);
    return launch_e<XT, 32, FMT>(x, rows, K, ldx, mult, cnorm, mult_after, block, qmax, clip_ratio, codes, delta, stream, gate);
}

__global__ void multipliers_kernel(const float* __restrict__ smooth, int K, float cnorm,
                                   float* __restrict__ mult_w, float* __restrict__ mult_g) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K) return;
    float mw = cnorm, mg = cnorm;
    if (smooth != nullptr) {
        const float s = smooth[i];
        mw = __fmul_rn(s, cnorm);
        mg = __fmul_rn(__fdiv_rn(1.0f, s), cnorm);
    }
    if (mult_w) mult_w[i] = mw;
    if (mult_g) mult_g[i] = mg;
}

// s^W_j *= d_j, b_j *= d_j for a run of output channels (one binary32 multiply each).
__global__ void scale_outputs_kernel(float* __restrict__ w_scale, float* __restrict__ bias,
                                     const float* __restrict__ d, int64_t count) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= count) return;
    w_scale[j] = __fmul_rn(w_scale[j], d[j]);
    bias[j] = __fmul_rn(bias[j], d[j]);
}

template <typename XT>
__global__ void col_absmax_kernel(const XT* __restrict__ x, int64_t M, int K, int64_t ldx, int accumulate,
                                  float* __restrict__ out, int rows_per_block) {
    // grid.x tiles columns, grid.y tiles rows; float max of non-negative values == unsigned max of bits
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= K) return;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_block;
    int64_t r1 = r0 + rows_per_block;
    if (r1 > M) r1 = M;
    float m = 0.0f;
    for (int64_t r = r0; r < r1; ++r) {
        float v;
        if (sizeof(XT) == 2)
            v = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(x)[r * ldx + c]);
        else
            v = reinterpret_cast<const float*>(x)[r * ldx + c];
        m = fmaxf(m, fabsf(v));
    }
    atomicMax(reinterpret_cast<unsigned int*>(out) + c, __float_as_uint(m));
}

__global__ void smooth_scale_kernel(const float* __restrict__ a, const float* __restrict__ w, int K,
                                    double alpha, float* __restrict__ s) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K) return;
    const double ac = a[i] > 1e-5f ? (double)a[i] : 1e-5;
    const double wc = w[i] > 1e-5f ? (double)w[i] : 1e-5;
    double v = pow(ac, alpha) / pow(wc, 1.0 - alpha);
    v = v < 1e-5 ? 1e-5 : (v > 1e5 ? 1e5 : v);
    s[i] = (float)v;
}

// 16 packed bytes (32 codes) per thread -> 32 int8 holding 16*code, each group of 8 channels in the
// (even channels, odd channels) order of StoreFmt::Int8Perm.
__global__ void expand_nibbles_kernel(const uint4* __restrict__ packed, int64_t n_vec, uint4* __restrict__ out) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_vec) return;
    const uint4 p = __ldg(packed + i);
    const uint32_t w[4] = {p.x, p.y, p.z, p.w};
    uint32_t o[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t lo = (w[j] << 4) & 0xF0F0F0F0u;   // even channels, code in the high nibble of each byte
        const uint32_t hi = w[j] & 0xF0F0F0F0u;          // odd channels
        o[2 * j + 0] = lo;     // channels 0,2,4,6 of the group of 8
        o[2 * j + 1] = hi;     // channels 1,3,5,7
    }
    out[2 * i + 0] = make_uint4(o[0], o[1], o[2], o[3]);
    out[2 * i + 1] = make_uint4(o[4], o[5], o[6], o[7]);
}

}  // namespace

cudaError_t launch_transform_quantize(const void* x, fq_dtype xt, int64_t rows, int64_t K, int64_t ldx,
                                      const float* mult, float cnorm, bool mult_after_rotation, int block, int qmax,
                                      float clip_ratio, StoreFmt fmt, void* codes, float* delta, cudaStream_t stream) {
    if (rows == 0) return cudaSuccess;
    const int mult_after = (mult != nullptr && mult_after_rotation) ? 1 : 0;
    {   // long batches stream through the TMA-fed ring; everything else stays in registers
        const cudaError_t e = launch_transform_quantize_ring(x, xt, rows, K, ldx, mult, cnorm, mult_after != 0, block, qmax,
                                                             clip_ratio, fmt, codes, delta, stream);
        if (e != cudaErrorNotSupported) return e;
    }
    const int k = (int)K;
    if (xt == FQ_F32) {
        const float* p = static_cast<const float*>(x);
            if (fmt == StoreFmt::Nibble) return launch_t<float, 0>(p, rows, k, ldx, mult, cnorm, mult_after, block, qmax, clip_ratio, codes, delta, stream);
        if (fmt == StoreFmt::Int8) return launch_t<float, 1>(p, rows, k, ldx, mult, cnorm, mult_after, block, qmax, clip_ratio, codes, delta, stream);
        return launch_t<float, 2>(p, rows, k, ldx, mult, cnorm, mult_after, block, qmax, clip_ratio, codes, delta, stream);
    }
    const __nv_bfloat16* p = static_cast<const __nv_bfloat16*>(x);
    if (fmt == StoreFmt::Nibble) return launch_t<__nv_bfloat16, 0>(p, rows, k, ldx, mult, cnorm, mult_after, block, qmax, clip_ratio, codes, delta, stream);
    if (fmt == StoreFmt::Int8) return launch_t<__nv_bfloat16, 1>(p, rows, k, ldx, mult, cnorm, mult_after, block, qmax, clip_ratio, codes, delta, stream);
    return launch_t<__nv_bfloat16, 2>(p, rows, k, ldx, mult, cnorm, mult_after, block, qmax, clip_ratio, codes, delta, stream);
}

// The site behind a gated MLP: x is [rows, 2K] = [gate | up], the quantizer's input is act(gate) * up.
// Always the register kernel's lean variant (the streaming kernel has no gated form).
cudaError_t launch_gated_transform_quantize(const void* x, fq_dtype xt, int64_t rows, int64_t K, int64_t ldx, int gate_kind,
                                            const float* mult, float cnorm, bool mult_after_rotation, int block, int qmax,
                                            float clip_ratio, StoreFmt fmt, void* codes, float* delta, cudaStream_t stream) {
    if (rows == 0) return cudaSuccess;
    const int k = (int)K;
    const int after = mult_after_rotation ? 1 : 0;
    if (xt == FQ_F32) {
        const float* p = static_cast<const float*>(x);
        if (fmt == StoreFmt::Nibble) return launch_t<float, 0>(p, rows, k, ldx, mult, cnorm, after, block, qmax, clip_ratio, codes, delta, stream, gate_kind);
        if (fmt == StoreFmt::Int8) return launch_t<float, 1>(p, rows, k, ldx, mult, cnorm, after, block, qmax, clip_ratio, codes, delta, stream, gate_kind);
        return launch_t<float, 2>(p, rows, k, ldx, mult, cnorm, after, block, qmax, clip_ratio, codes, delta, stream, gate_kind);
    }
    const __nv_bfloat16* p = static_cast<const __nv_bfloat16*>(x);
    if (fmt == StoreFmt::Nibble) return launch_t<__nv_bfloat16, 0>(p, rows, k, ldx, mult, cnorm, after, block, qmax, clip_ratio, codes, delta, stream, gate_kind);
    if (fmt == StoreFmt::Int8) return launch_t<__nv_bfloat16, 1>(p, rows, k, ldx, mult, cnorm, after, block, qmax, clip_ratio, codes, delta, stream, gate_kind);
    return launch_t<__nv_bfloat16, 2>(p, rows, k, ldx, mult, cnorm, after, block, qmax, clip_ratio, codes, delta, stream, gate_kind);
}

cudaError_t launch_multipliers(const float* smooth, int64_t K, float cnorm, float* mult_w, float* mult_g,
                               cudaStream_t stream) {
    multipliers_kernel<<<(unsigned)((K + 255) / 256), 256, 0, stream>>>(smooth, (int)K, cnorm, mult_w, mult_g);
    return cudaGetLastError();
}

cudaError_t launch_scale_outputs(float* w_scale, float* bias, const float* d, int64_t count, cudaStream_t stream) {
    if (count == 0) return cudaSuccess;
    scale_outputs_kernel<<<(unsigned)((count + 255) / 256), 256, 0, stream>>>(w_scale, bias, d, count);
    return cudaGetLastError();
}

cudaError_t launch_col_absmax(const void* x, fq_dtype xt, int64_t M, int64_t K, int64_t ldx, int accumulate,
                              float* out, cudaStream_t stream) {
    if (!accumulate) {
        cudaError_t e = cudaMemsetAsync(out, 0, sizeof(float) * (size_t)K, stream);
        if (e != cudaSuccess) return e;
    }
    if (M == 0) return cudaSuccess;
    const int rows_per_block = 64;
    dim3 grid((unsigned)((K + 127) / 128), (unsigned)((M + rows_per_block - 1) / rows_per_block));
    if (xt == FQ_F32)
        col_absmax_kernel<float><<<grid, 128, 0, stream>>>(static_cast<const float*>(x), M, (int)K, ldx, accumulate,
                                                           out, rows_per_block);
    else
        col_absmax_kernel<__nv_bfloat16><<<grid, 128, 0, stream>>>(static_cast<const __nv_bfloat16*>(x), M, (int)K,
                                                                   ldx, accumulate, out, rows_per_block);
    return cudaGetLastError();
}

cudaError_t launch_smooth_scale(const float* a, const float* w, int64_t K, double alpha, float* s,
                                cudaStream_t stream) {
    smooth_scale_kernel<<<(unsigned)((K + 255) / 256), 256, 0, stream>>>(a, w, (int)K, alpha, s);
    return cudaGetLastError();
}

cudaError_t launch_expand_nibbles(const void* packed, int64_t rows, int64_t K, void* out, cudaStream_t stream) {
    const int64_t n_vec = rows * K / 32;
    if (n_vec == 0) return cudaSuccess;
    expand_nibbles_kernel<<<(unsigned)((n_vec + 255) / 256), 256, 0, stream>>>(
        static_cast<const uint4*>(packed), n_vec, static_cast<uint4*>(out));
    return cudaGetLastError();
}

}  // namespace fq
