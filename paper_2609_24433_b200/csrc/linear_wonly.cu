// Weight-only 4-bit projection with floating-point activations (the adaptive layer-normalisation
// modulation of the W4A4 engines keeps its activations in floating point):
//   y[t][j] = s^W_j * sum_c qW[j][c] * x[t][c] + b_j
// These projections see one conditioning vector per sample (M = batch, a handful of tokens), so the
// operation is a matrix-vector product bound by the weight bytes: CUDA cores, each warp streaming
// eight weight rows with 8-byte loads per lane while the activations of its 16 channels stay in
// registers; binary32 accumulation, one fused multiply-add for the rescale and bias.
#include <cuda_bf16.h>

#include "fq_common.cuh"
#include "ptx_sm100.cuh"

namespace fq {
namespace {

constexpr int kRows = 8;          // weight rows per warp
constexpr int kWarps = 8;
constexpr int kChunk = 16;        // channels per lane and step (one 8-byte load of packed weights)

// Eight 4-bit two's-complement codes of a word -> binary32, exactly: (n & 15) ^ 8 = n + 8, placed in
// the mantissa of 2^23, minus (2^23 + 8).
__device__ __forceinline__ void decode8(uint32_t w, float* q) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
        q[i] = __uint_as_float(((w >> (4 * i)) & 0xFu) ^ 0x4B000008u) - 8388616.0f;
}

template <typename XT>
__device__ __forceinline__ void load_x16(const XT* p, bool ok, float* v);
template <>
__device__ __forceinline__ void load_x16<float>(const float* p, bool ok, float* v) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float4 t = ok ? __ldg(reinterpret_cast<const float4*>(p) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        v[4 * i + 0] = t.x; v[4 * i + 1] = t.y; v[4 * i + 2] = t.z; v[4 * i + 3] = t.w;
    }
}
template <>
__device__ __forceinline__ void load_x16<__nv_bfloat16>(const __nv_bfloat16* p, bool ok, float* v) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const uint4 t = ok ? __ldg(reinterpret_cast<const uint4*>(p) + i) : make_uint4(0u, 0u, 0u, 0u);
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            v[8 * i + 2 * k + 0] = __uint_as_float(w[k] << 16);
            v[8 * i + 2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
        }
    }
}

// MT tokens per pass over the weights (their activations live in registers).
template <typename XT, int MT>
__global__ void __launch_bounds__(kWarps * 32)
linear_wonly4_kernel(const XT* __restrict__ x, int64_t M, int K, int64_t ldx, const uint8_t* __restrict__ wcodes,
                     const float* __restrict__ w_scale, const float* __restrict__ bias, int64_t N, void* __restrict__ y,
                     fq_dtype yt, int64_t ldy) {
    griddep_wait();                   // launched with programmatic serialization
    griddep_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int64_t j0 = ((int64_t)blockIdx.x * kWarps + (threadIdx.x >> 5)) * kRows;
    if (j0 >= N) return;              // N is a multiple of 8: a warp has all of its rows or none
    const int64_t pitch = K / 2;
    for (int64_t t0 = (int64_t)blockIdx.y * MT; t0 < M; t0 += (int64_t)gridDim.y * MT) {
        float acc[kRows][MT];
#pragma unroll
        for (int r = 0; r < kRows; ++r)
#pragma unroll
            for (int t = 0; t < MT; ++t) acc[r][t] = 0.0f;
        for (int c0 = lane * kChunk; c0 < K; c0 += 32 * kChunk) {
            float xv[MT][kChunk];
#pragma unroll
            for (int t = 0; t < MT; ++t) load_x16<XT>(x + (t0 + t) * ldx + c0, t0 + t < M, xv[t]);
            uint2 w[kRows];
#pragma unroll
            for (int r = 0; r < kRows; ++r) w[r] = __ldg(reinterpret_cast<const uint2*>(wcodes + (j0 + r) * pitch + c0 / 2));
#pragma unroll
            for (int r = 0; r < kRows; ++r) {
                float q[kChunk];
                decode8(w[r].x, q);
                decode8(w[r].y, q + 8);
#pragma unroll
                for (int t = 0; t < MT; ++t)
#pragma unroll
                    for (int i = 0; i < kChunk; ++i) acc[r][t] = fmaf(q[i], xv[t][i], acc[r][t]);
            }
        }
        // lanes hold partial sums over their channels: butterfly reduction, then lane r*MT + t stores
        float mine = 0.0f;
#pragma unroll
        for (int r = 0; r < kRows; ++r)
#pragma unroll
            for (int t = 0; t < MT; ++t) {
                float v = acc[r][t];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (lane == r * MT + t) mine = v;
            }
        if (lane < kRows * MT) {
            const int r = lane / MT, t = lane % MT;
            const int64_t j = j0 + r, tt = t0 + t;
            if (tt < M) {
                const float v = fmaf(mine, __ldg(w_scale + j), __ldg(bias + j));
                if (yt == FQ_F32) static_cast<float*>(y)[tt * ldy + j] = v;
                else static_cast<__nv_bfloat16*>(y)[tt * ldy + j] = __float2bfloat16_rn(v);
            }
        }
    }
}

template <typename XT>
cudaError_t launch_xt(const XT* x, int64_t M, const Weights& W, int64_t ldx, void* y, fq_dtype yt, int64_t ldy,
                      cudaStream_t stream) {
    const unsigned gx = (unsigned)((W.N / kRows + kWarps - 1) / kWarps);
    const int K = (int)W.K;
    auto go = [&](auto kern, int mt) {
        int64_t groups = (M + mt - 1) / mt;
        if (groups > 64) groups = 64;               // beyond that a CTA walks several token groups
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(gx, (unsigned)groups, 1);
        cfg.blockDim = dim3(kWarps * 32, 1, 1);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kern, x, M, K, ldx, (const uint8_t*)W.codes, (const float*)W.w_scale,
                                  (const float*)W.bias, W.N, y, yt, ldy);
    };
    if (M == 1) return go(linear_wonly4_kernel<XT, 1>, 1);
    if (M == 2) return go(linear_wonly4_kernel<XT, 2>, 2);
    return go(linear_wonly4_kernel<XT, 4>, 4);
}

}  // namespace

cudaError_t launch_linear_wonly4(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const Weights& W, void* y,
                                 fq_dtype yt, int64_t ldy, cudaStream_t stream) {
    if (M == 0 || W.N == 0) return cudaSuccess;
    if (xt == FQ_F32) return launch_xt(static_cast<const float*>(x), M, W, ldx, y, yt, ldy, stream);
    return launch_xt(static_cast<const __nv_bfloat16*>(x), M, W, ldx, y, yt, ldy, stream);
}

}  // namespace fq
