// Stored composite rotation (optional transform of the action expert): a channel permutation followed
// by one stored dense matrix per block of `beta` channels,
//   R = blockdiag(B_0 .. B_{K/beta-1}) Pi,      u[t][b*beta + i] = sum_j B_b[i][j] * v[t][perm[b*beta + j]],
//   v = x (.) d  (d = 1/s at run time, s when folding weights).
// This kernel produces u in binary32 (one multiply for the diagonal, then one fused multiply-add per
// term in ascending j, starting from 0 -- the order the results are defined in); the per-token step and
// the codes of Eq. 5 are then taken by the ordinary prologue kernel run with the identity rotation.
// The contraction is 2*beta flops per element against 6 for the butterflies; it is dense but tiny per
// block (beta x beta), the sums must keep their order, and the path is optional and used on short
// batches: CUDA cores, one CTA per (block, tile of tokens), the block's matrix staged through shared
// memory in transposed chunks so that both its global reads and its shared reads are conflict-free.
#include <cuda_bf16.h>

#include "fq_common.cuh"
#include "ptx_sm100.cuh"

namespace fq {
namespace {

constexpr int kThreads = 256;
constexpr int kChunkJ = 32;          // columns of B staged at a time

template <typename XT>
__device__ __forceinline__ float load_as_float(const XT* p);
template <>
__device__ __forceinline__ float load_as_float<float>(const float* p) { return __ldg(p); }
template <>
__device__ __forceinline__ float load_as_float<__nv_bfloat16>(const __nv_bfloat16* p) {
    return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}

// BETA in {16, 32, 64, 128, 256}.  Thread (group = tid / BETA, i = tid % BETA) computes output i of
// R = 8 tokens (one shared-memory read of the matrix entry and two 16-byte reads of the inputs feed eight
// multiply-adds); a CTA covers (256 / BETA) * 8 tokens of one block.
template <typename XT, int BETA>
__global__ void __launch_bounds__(kThreads)
composite_rotate_kernel(const XT* __restrict__ x, int64_t rows, int K, int64_t ldx, const float* __restrict__ diag,
                        const int32_t* __restrict__ perm, const float* __restrict__ blocks, float* __restrict__ u) {
    constexpr int G = kThreads / BETA;
    constexpr int R = 8;
    constexpr int TOK = G * R;
    __shared__ __align__(16) float s_p[BETA][TOK];   // permuted, scaled inputs of the tile, token-minor
    __shared__ float s_b[kChunkJ][BETA + 1];         // B_b[.][j0 .. j0+31], transposed: s_b[jj][i]
    griddep_wait();
    griddep_launch_dependents();
    const int tid = threadIdx.x;
    const int b = blockIdx.x;
    const int64_t tile0 = (int64_t)blockIdx.y * TOK;
    // gather: p[tok][j] = x[tok][perm[b*BETA + j]] * d[perm[...]]   (an index outside [0, K) is clamped)
    for (int o = tid; o < TOK * BETA; o += kThreads) {
        const int tok = o / BETA, j = o % BETA;
        int src = __ldg(perm + b * BETA + j);
        src = src < 0 ? 0 : (src >= K ? K - 1 : src);
        float v = 0.0f;
        if (tile0 + tok < rows) {
            v = load_as_float<XT>(x + (tile0 + tok) * ldx + src);
            if (diag != nullptr) v = __fmul_rn(v, __ldg(diag + src));
        }
        s_p[j][tok] = v;
    }
    const int grp = tid / BETA, i = tid % BETA;
    float acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.0f;
    const float* B = blocks + (size_t)b * BETA * BETA;
    for (int j0 = 0; j0 < BETA; j0 += kChunkJ) {
        __syncthreads();                             // s_p written (first pass) / previous chunk consumed
        constexpr int CJ = BETA < kChunkJ ? BETA : kChunkJ;
        for (int o = tid; o < BETA * CJ; o += kThreads) {
            const int row = o / CJ, jj = o % CJ;     // consecutive threads: consecutive columns of one row
            s_b[jj][row] = __ldg(B + (size_t)row * BETA + j0 + jj);
        }
        __syncthreads();
#pragma unroll 8
        for (int jj = 0; jj < CJ; ++jj) {
            const float bv = s_b[jj][i];
            const float4 pa = *reinterpret_cast<const float4*>(&s_p[j0 + jj][grp * R]);
            const float4 pb = *reinterpret_cast<const float4*>(&s_p[j0 + jj][grp * R + 4]);
            acc[0] = __fmaf_rn(bv, pa.x, acc[0]); acc[1] = __fmaf_rn(bv, pa.y, acc[1]);
            acc[2] = __fmaf_rn(bv, pa.z, acc[2]); acc[3] = __fmaf_rn(bv, pa.w, acc[3]);
            acc[4] = __fmaf_rn(bv, pb.x, acc[4]); acc[5] = __fmaf_rn(bv, pb.y, acc[5]);
            acc[6] = __fmaf_rn(bv, pb.z, acc[6]); acc[7] = __fmaf_rn(bv, pb.w, acc[7]);
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int64_t t = tile0 + grp * R + r;
        if (t < rows) u[t * K + b * BETA + i] = acc[r];
    }
}

template <typename XT, int BETA>
cudaError_t launch_beta(const XT* x, int64_t rows, int K, int64_t ldx, const float* diag, const int32_t* perm,
                        const float* blocks, float* u, cudaStream_t stream) {
    constexpr int TOK = (kThreads / BETA) * 8;
    const int64_t tiles = (rows + TOK - 1) / TOK;
    if (tiles > 65535) return cudaErrorInvalidConfiguration;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(K / BETA), (unsigned)tiles, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, composite_rotate_kernel<XT, BETA>, x, rows, K, ldx, diag, perm, blocks, u);
}

template <typename XT>
cudaError_t launch_xt(const XT* x, int64_t rows, int K, int64_t ldx, const float* diag, const int32_t* perm,
                      const float* blocks, int beta, float* u, cudaStream_t stream) {
    switch (beta) {
        case 16: return launch_beta<XT, 16>(x, rows, K, ldx, diag, perm, blocks, u, stream);
        case 32: return launch_beta<XT, 32>(x, rows, K, ldx, diag, perm, blocks, u, stream);
        case 64: return launch_beta<XT, 64>(x, rows, K, ldx, diag, perm, blocks, u, stream);
        case 128: return launch_beta<XT, 128>(x, rows, K, ldx, diag, perm, blocks, u, stream);
        case 256: return launch_beta<XT, 256>(x, rows, K, ldx, diag, perm, blocks, u, stream);
        default: return cudaErrorNotSupported;
    }
}

__global__ void perm_check_kernel(const int32_t* __restrict__ perm, int K, int* __restrict__ bad) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < K && (perm[c] < 0 || perm[c] >= K)) *bad = 1;
}

}  // namespace

cudaError_t launch_composite_rotate(const void* x, fq_dtype xt, int64_t rows, int64_t K, int64_t ldx, const float* diag,
                                    const int32_t* perm, const float* blocks, int beta, float* u, cudaStream_t stream) {
    if (rows == 0) return cudaSuccess;
    if (xt == FQ_F32)
        return launch_xt(static_cast<const float*>(x), rows, (int)K, ldx, diag, perm, blocks, beta, u, stream);
    return launch_xt(static_cast<const __nv_bfloat16*>(x), rows, (int)K, ldx, diag, perm, blocks, beta, u, stream);
}

cudaError_t launch_perm_check(const int32_t* perm, int64_t K, int* bad_flag, cudaStream_t stream) {
    perm_check_kernel<<<(unsigned)((K + 255) / 256), 256, 0, stream>>>(perm, (int)K, bad_flag);
    return cudaGetLastError();
}

}  // namespace fq
