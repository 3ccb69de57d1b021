// CUDA-core integer GEMM (dp4a), one output per thread.  It is the on-device
// second witness for the tensor-core kernel at sizes the CPU oracle can only
// sample, and the bring-up path; it is not tuned.
//   acc[t][j] = sum_c qA[t][c] * qW[j][c]           (Eq. 8, integer sum)
//   y[t][j]   = delta_t * s^W_j * acc + b_j         (Eq. 8, rescale + bias)
#include <cuda_bf16.h>

#include "fq_common.cuh"

namespace fq {
namespace {

template <int BITS>
__global__ void gemm_simt_kernel(const int8_t* __restrict__ a8, int64_t M, int64_t N, int64_t K,
                                 const uint8_t* __restrict__ wcodes, const float* __restrict__ w_scale,
                                 const float* __restrict__ bias, int acc_shift, GemmOut out) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t t = blockIdx.y;
    if (j >= N || t >= M) return;
    const uint4* arow = reinterpret_cast<const uint4*>(a8 + t * K);
    int acc = 0;
    if (BITS == 8) {
        const uint4* wrow = reinterpret_cast<const uint4*>(wcodes + j * K);
        for (int64_t k = 0; k < K / 16; ++k) {
            const uint4 a = __ldg(arow + k), w = __ldg(wrow + k);
            acc = __dp4a((int)a.x, (int)w.x, acc);
            acc = __dp4a((int)a.y, (int)w.y, acc);
            acc = __dp4a((int)a.z, (int)w.z, acc);
            acc = __dp4a((int)a.w, (int)w.w, acc);
        }
    } else {
        const uint2* wrow = reinterpret_cast<const uint2*>(wcodes + j * (K / 2));
        for (int64_t k = 0; k < K / 16; ++k) {
            const uint4 a = __ldg(arow + k);
            const uint2 w = __ldg(wrow + k);
            const uint32_t lo0 = (w.x << 4) & 0xF0F0F0F0u, hi0 = w.x & 0xF0F0F0F0u;
            const uint32_t lo1 = (w.y << 4) & 0xF0F0F0F0u, hi1 = w.y & 0xF0F0F0F0u;
            // 4-bit activations arrive as int8 with each group of 8 channels in (even, odd) order
            acc = __dp4a((int)a.x, (int)lo0, acc);
            acc = __dp4a((int)a.y, (int)hi0, acc);
            acc = __dp4a((int)a.z, (int)lo1, acc);
            acc = __dp4a((int)a.w, (int)hi1, acc);
        }
    }
    acc >>= acc_shift;   // exact: the scaled operands make acc a multiple of 2^acc_shift
    if (out.acc != nullptr) {
        out.acc[t * N + j] = acc;
    } else {
        const float v = fmaf((float)acc, out.a_delta[t] * w_scale[j], bias[j]);
        if (out.yt == FQ_F32)
            static_cast<float*>(out.y)[t * out.ldy + j] = v;
        else
            static_cast<__nv_bfloat16*>(out.y)[t * out.ldy + j] = __float2bfloat16_rn(v);
    }
}

}  // namespace

cudaError_t launch_gemm_simt(const int8_t* a8, int64_t M, const Weights& W, int acc_shift, const GemmOut& out,
                             cudaStream_t stream) {
    if (M == 0 || W.N == 0) return cudaSuccess;
    if (M > 65535) return cudaErrorInvalidConfiguration;
    dim3 grid((unsigned)((W.N + 127) / 128), (unsigned)M);
    if (W.bits == 8)
        gemm_simt_kernel<8><<<grid, 128, 0, stream>>>(a8, M, W.N, W.K, W.codes, W.w_scale, W.bias, acc_shift, out);
    else
        gemm_simt_kernel<4><<<grid, 128, 0, stream>>>(a8, M, W.N, W.K, W.codes, W.w_scale, W.bias, acc_shift, out);
    return cudaGetLastError();
}

}  // namespace fq
