// GPTQ rounding in transformed coordinates (offline; section "Rounding and native execution", Eq. 7):
//   min_Q ||(W~ - Q) Z||_F^2,  G = Z Z^T, H = G + lambda I,  H^-1 = U^T U (U upper triangular),
// channels rounded one after the other, each rounding error spread along the row of U over the channels
// still to come.  Everything here decides integer codes, so all arithmetic is binary32 in a fixed order
// (fused multiply-add chains in ascending index): results do not depend on how the work is split over
// threads, only on these definitions.
//   transform_rows    z = (I (x) H_beta)(x (.) mult): the prologue's transform without its quantizer
//   gram              G[a][b] = sum_t z[t][a] z[t][b], t ascending
//   damp              lambda = damp * (sum_a G[a][a]) / K (sum in ascending a); dead channels (G[a][a] = 0) get 1
//   rev_chol_col      column j of the upper factor M of H = M M^T, j = K-1 .. 0 (stored transposed: Mt[k][i] = M[i][k])
//   tri_inverse       U = M^-1, one thread per column, rows from the diagonal upwards
//   sweep             per weight row, channels i = 0 .. K-1: code, error, update of the channels j > i
#include <cuda_bf16.h>
#include <float.h>

#include "fq_common.cuh"

namespace fq {
namespace {

template <typename XT>
__device__ __forceinline__ float ld_f32(const XT* p);
template <>
__device__ __forceinline__ float ld_f32<float>(const float* p) { return __ldg(p); }
template <>
__device__ __forceinline__ float ld_f32<__nv_bfloat16>(const __nv_bfloat16* p) {
    return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}

// One CTA per row; the row lives in shared memory (K floats) while the butterflies run.
template <typename XT>
__global__ void __launch_bounds__(256)
transform_rows_kernel(const XT* __restrict__ x, int K, int64_t ldx, const float* __restrict__ mult, float cnorm,
                      int block, float* __restrict__ z) {
    extern __shared__ float s_v[];
    const int64_t r = blockIdx.x;
    for (int c = threadIdx.x; c < K; c += blockDim.x)
        s_v[c] = __fmul_rn(ld_f32<XT>(x + r * ldx + c), mult ? __ldg(mult + c) : cnorm);
    for (int h = 1; h < block; h <<= 1) {
        __syncthreads();
        for (int p = threadIdx.x; p < K / 2; p += blockDim.x) {
            const int i = ((p / h) * 2 * h) + (p % h);        // the pair (i, i + h), i & h == 0
            const float a = s_v[i], b = s_v[i + h];
            s_v[i] = __fadd_rn(a, b);
            s_v[i + h] = __fsub_rn(a, b);
        }
    }
    __syncthreads();
    for (int c = threadIdx.x; c < K; c += blockDim.x) z[r * K + c] = s_v[c];
}

// 16 x 16 outputs per CTA, tokens staged 16 at a time.
__global__ void __launch_bounds__(256)
gram_kernel(const float* __restrict__ z, int64_t Mc, int K, float* __restrict__ G) {
    __shared__ float s_a[16][17], s_b[16][17];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int a0 = blockIdx.y * 16, b0 = blockIdx.x * 16;
    float acc = 0.0f;
    for (int64_t t0 = 0; t0 < Mc; t0 += 16) {
        const int64_t t = t0 + ty;
        s_a[ty][tx] = (t < Mc && a0 + tx < K) ? z[t * K + a0 + tx] : 0.0f;
        s_b[ty][tx] = (t < Mc && b0 + tx < K) ? z[t * K + b0 + tx] : 0.0f;
        __syncthreads();
        const int n = (int)((Mc - t0) < 16 ? (Mc - t0) : 16);
        for (int k = 0; k < n; ++k) acc = __fmaf_rn(s_a[k][ty], s_b[k][tx], acc);
        __syncthreads();
    }
    if (a0 + ty < K && b0 + tx < K) G[(int64_t)(a0 + ty) * K + b0 + tx] = acc;
}

__global__ void damp_kernel(float* __restrict__ H, int K, float damp, uint8_t* __restrict__ dead) {
    __shared__ float s_lambda;
    if (threadIdx.x == 0) {
        float sum = 0.0f;
        for (int a = 0; a < K; ++a) sum = __fadd_rn(sum, H[(int64_t)a * K + a]);
        s_lambda = __fmul_rn(damp, __fdiv_rn(sum, (float)K));
    }
    __syncthreads();
    for (int a = threadIdx.x; a < K; a += blockDim.x) {
        float d = H[(int64_t)a * K + a];
        const bool is_dead = d == 0.0f;
        dead[a] = is_dead ? 1 : 0;
        if (is_dead) d = 1.0f;
        H[(int64_t)a * K + a] = __fadd_rn(d, s_lambda);
    }
}

// Column j of M (H = M M^T, M upper triangular), stored as row j of Mt.  Every CTA first copies the
// finished entries M[j][k], k > j, into shared memory (all threads load, so the strided reads overlap),
// then recomputes the diagonal entry from them (one chain of at most K terms) instead of waiting for
// another CTA to publish it; the off-diagonal chains read the same copy.
__global__ void __launch_bounds__(256)
rev_chol_col_kernel(const float* __restrict__ H, float* __restrict__ Mt, int K, int j, int* __restrict__ bad) {
    extern __shared__ float s_mj[];                  // K floats: s_mj[k - j - 1] = M[j][k]
    __shared__ float s_d;
    const int n = K - 1 - j;
    for (int o = threadIdx.x; o < n; o += blockDim.x) s_mj[o] = Mt[(int64_t)(j + 1 + o) * K + j];
    __syncthreads();
    if (threadIdx.x == 0) {
        float acc = H[(int64_t)j * K + j];
        for (int o = 0; o < n; ++o) acc = __fmaf_rn(-s_mj[o], s_mj[o], acc);
        if (!(acc > 0.0f)) { *bad = 1; acc = 1.0f; }
        s_d = __fsqrt_rn(acc);
    }
    __syncthreads();
    const float d = s_d;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == j) Mt[(int64_t)j * K + j] = d;
    if (i < j) {
        // sixteen loads in flight ahead of the (sequential) chain: the loop is bound by their latency otherwise
        float acc = H[(int64_t)i * K + j];
        const float* col = Mt + (int64_t)(j + 1) * K + i;
        int o = 0;
        if (n >= 32) {
            float cur[32], nxt[32];
#pragma unroll
            for (int q = 0; q < 32; ++q) cur[q] = col[(int64_t)q * K];
            for (; o + 64 <= n; o += 32) {           // the next batch is requested before this one is consumed
#pragma unroll
                for (int q = 0; q < 32; ++q) nxt[q] = col[(int64_t)(o + 32 + q) * K];
#pragma unroll
                for (int q = 0; q < 32; ++q) acc = __fmaf_rn(-cur[q], s_mj[o + q], acc);
#pragma unroll
                for (int q = 0; q < 32; ++q) cur[q] = nxt[q];
            }
#pragma unroll
            for (int q = 0; q < 32; ++q) acc = __fmaf_rn(-cur[q], s_mj[o + q], acc);
            o += 32;
        }
        for (; o < n; ++o) acc = __fmaf_rn(-col[(int64_t)o * K], s_mj[o], acc);
        Mt[(int64_t)j * K + i] = __fdiv_rn(acc, d);
    }
}

// U = M^-1: column c from row c upwards; U row-major [K][K], zeros below the diagonal.
__global__ void __launch_bounds__(128)
tri_inverse_kernel(const float* __restrict__ Mt, float* __restrict__ U, int K) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= K) return;
    for (int i = K - 1; i > c; --i) U[(int64_t)i * K + c] = 0.0f;
    U[(int64_t)c * K + c] = __fdiv_rn(1.0f, Mt[(int64_t)c * K + c]);
    for (int i = c - 1; i >= 0; --i) {
        float acc = 0.0f;
        int k = i + 1;
        for (; k + 8 <= c + 1; k += 8) {             // eight pairs of loads in flight ahead of the chain
            float m[8], u[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) { m[q] = Mt[(int64_t)(k + q) * K + i]; u[q] = U[(int64_t)(k + q) * K + c]; }
#pragma unroll
            for (int q = 0; q < 8; ++q) acc = __fmaf_rn(m[q], u[q], acc);
        }
        for (; k <= c; ++k) acc = __fmaf_rn(Mt[(int64_t)k * K + i], U[(int64_t)k * K + c], acc);
        U[(int64_t)i * K + c] = __fdiv_rn(-acc, Mt[(int64_t)i * K + i]);
    }
}

// The sweep is independent per weight row: a CTA keeps kSweepRows rows in shared memory (four; two of the longest
// rows, which would not fit otherwise) and walks the channels.
template <int BITS, int kSweepRows>
__global__ void __launch_bounds__(256)
gptq_sweep_kernel(const float* __restrict__ Wt, int64_t N, int K, const float* __restrict__ U,
                  const uint8_t* __restrict__ dead, const float* __restrict__ w_scale, uint8_t* __restrict__ codes) {
    extern __shared__ float s_w[];                   // [kSweepRows][K]
    __shared__ float s_e[kSweepRows];
    const int64_t r0 = (int64_t)blockIdx.x * kSweepRows;
    for (int o = threadIdx.x; o < kSweepRows * K; o += blockDim.x) {
        const int r = o / K, c = o - r * K;
        s_w[o] = r0 + r < N ? Wt[(r0 + r) * K + c] : 0.0f;
    }
    const float qmax = BITS == 4 ? 7.0f : 127.0f;
    // threads 0 .. kSweepRows-1 each own a row's quantizer (and its pending low nibble)
    float s = 0.0f, inv = 0.0f;
    int low = 0;
    if (threadIdx.x < kSweepRows && r0 + threadIdx.x < N) {
        s = w_scale[r0 + threadIdx.x];
        inv = s >= FLT_MIN ? __fdiv_rn(1.0f, s) : 0.0f;
    }
    __syncthreads();
    for (int i = 0; i < K; ++i) {
        if (threadIdx.x < kSweepRows) {
            const int r = threadIdx.x;
            const float wi = dead[i] ? 0.0f : s_w[r * K + i];
            float t = rintf(__fmul_rn(wi, inv));
            t = fminf(fmaxf(t, -qmax), qmax);
            const int v = (int)t;
            s_e[r] = __fdiv_rn(__fsub_rn(wi, __fmul_rn(t, s)), U[(int64_t)i * K + i]);
            if (r0 + r < N) {
                if (BITS == 8) {
                    codes[(r0 + r) * (int64_t)K + i] = (uint8_t)(int8_t)v;
                } else if (i & 1) {
                    codes[(r0 + r) * (int64_t)(K / 2) + (i >> 1)] = (uint8_t)((low & 15) | ((v & 15) << 4));
                } else {
                    low = v;
                }
            }
        }
        __syncthreads();
        float e[kSweepRows];
#pragma unroll
        for (int r = 0; r < kSweepRows; ++r) e[r] = -s_e[r];
        for (int j = i + 1 + threadIdx.x; j < K; j += blockDim.x) {
            const float u = __ldg(U + (int64_t)i * K + j);
#pragma unroll
            for (int r = 0; r < kSweepRows; ++r) s_w[r * K + j] = __fmaf_rn(e[r], u, s_w[r * K + j]);
        }
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_transform_rows(const void* x, fq_dtype xt, int64_t rows, int64_t K, int64_t ldx, const float* mult,
                                  float cnorm, int block, float* z, cudaStream_t stream) {
    if (rows == 0) return cudaSuccess;
    const size_t smem = sizeof(float) * (size_t)K;
    if (xt == FQ_F32) {
        cudaError_t e = cudaFuncSetAttribute(transform_rows_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        transform_rows_kernel<float><<<(unsigned)rows, 256, smem, stream>>>(static_cast<const float*>(x), (int)K, ldx, mult,
                                                                           cnorm, block, z);
    } else {
        cudaError_t e = cudaFuncSetAttribute(transform_rows_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        transform_rows_kernel<__nv_bfloat16><<<(unsigned)rows, 256, smem, stream>>>(static_cast<const __nv_bfloat16*>(x),
                                                                                   (int)K, ldx, mult, cnorm, block, z);
    }
    return cudaGetLastError();
}

// H (K x K) from Z, damped; U = upper factor of H^-1; *bad (device int, zeroed by the caller) is set if H is
// not positive definite in binary32.  Mt and H are K x K scratch.
cudaError_t launch_gptq_factor(const float* z, int64_t Mc, int64_t K, float damp, float* H, float* Mt, float* U,
                               uint8_t* dead, int* bad, cudaStream_t stream) {
    const dim3 g((unsigned)((K + 15) / 16), (unsigned)((K + 15) / 16));
    gram_kernel<<<g, 256, 0, stream>>>(z, Mc, (int)K, H);
    damp_kernel<<<1, 256, 0, stream>>>(H, (int)K, damp, dead);
    cudaError_t e = cudaMemsetAsync(Mt, 0, sizeof(float) * (size_t)K * (size_t)K, stream);
    if (e != cudaSuccess) return e;
    const size_t col_smem = sizeof(float) * (size_t)K;
    e = ensure_dynamic_smem(reinterpret_cast<const void*>(rev_chol_col_kernel), col_smem);
    if (e != cudaSuccess) return e;
    for (int j = (int)K - 1; j >= 0; --j)
        rev_chol_col_kernel<<<(unsigned)(j / 256 + 1), 256, col_smem, stream>>>(H, Mt, (int)K, j, bad);
    tri_inverse_kernel<<<(unsigned)((K + 127) / 128), 128, 0, stream>>>(Mt, U, (int)K);
    return cudaGetLastError();
}

namespace {
template <int BITS, int ROWS>
cudaError_t launch_sweep_variant(const float* Wt, int64_t N, int64_t K, const float* U, const uint8_t* dead,
                                 const float* w_scale, uint8_t* codes, cudaStream_t stream) {
    const size_t smem = sizeof(float) * (size_t)ROWS * (size_t)K;
    const unsigned grid = (unsigned)((N + ROWS - 1) / ROWS);
    auto kern = gptq_sweep_kernel<BITS, ROWS>;
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, 256, smem, stream>>>(Wt, N, (int)K, U, dead, w_scale, codes);
    return cudaGetLastError();
}
}  // namespace

cudaError_t launch_gptq_sweep(const float* Wt, int64_t N, int64_t K, const float* U, const uint8_t* dead,
                              const float* w_scale, int bits, uint8_t* codes, cudaStream_t stream) {
    if (N == 0) return cudaSuccess;
    // four rows of K floats per CTA up to K = 8192 (128 KB), two beyond (K <= 16384: 128 KB)
    if (K <= 8192)
        return bits == 4 ? launch_sweep_variant<4, 4>(Wt, N, K, U, dead, w_scale, codes, stream)
                         : launch_sweep_variant<8, 4>(Wt, N, K, U, dead, w_scale, codes, stream);
    return bits == 4 ? launch_sweep_variant<4, 2>(Wt, N, K, U, dead, w_scale, codes, stream)
                     : launch_sweep_variant<8, 2>(Wt, N, K, U, dead, w_scale, codes, stream);
}

}  // namespace fq
