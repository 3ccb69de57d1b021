// Internal declarations shared by the translation units of the library
// (never installed; the public boundary is include/fq.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>

#include "fq.h"

namespace fq {

// Folded-weight pack of one projection (Alg. 1, offline half: packed codes,
// output-channel scales, bias) plus the constants the runtime prologue needs.
struct Weights {
    int64_t N = 0, K = 0;
    int block = 0, bits = 0;
    int device = 0;
    uint8_t* codes = nullptr;   // [N, K*bits/8], canonical packing
    float* w_scale = nullptr;   // [N]
    float* bias = nullptr;      // [N]
    float* mult_g = nullptr;    // [K] runtime multiplier (1/s_c) * block^-1/2
    bool fold_after = false;    // mult_g is the post-rotation multiplier 1/p (T = P^-1 R) instead of (1/s) block^-1/2
    bool composite = false;     // folded with a stored composite rotation: the prologue is fq_quantize_act_composite
    bool mult_const = false;    // mult_g holds the constant block^-1/2 in every entry (no smoothing, or the diagonal absorbed
                                // upstream): the fused calls then run the prologue without the per-channel vector
    CUtensorMap tmap;           // TMA view of `codes` for the GEMM's weight operand
    bool tmap_valid = false;
    CUtensorMap tmap_stream;    // 4-bit weights: view for the short-batch streaming kernel (32 rows x 128 bytes)
    bool tmap_stream_valid = false;
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Facts about the current device and per-kernel launch set-up, looked up once and remembered (an eager call
// otherwise pays several runtime queries per launch).
int device_sm_count();                                              // multiprocessors of the current device
int device_cc_major();                                              // compute-capability major, -1 on error
cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes);  // opt a kernel in to `bytes` of dynamic shared memory
int max_resident_blocks(const void* kernel, int threads);           // thread blocks of a kernel one SM holds (no dynamic smem)

// Launch with programmatic stream serialization (the kernel must call griddep_wait() before its first
// global-memory access) and, optionally, a thread-block cluster along x.
template <typename Kern, typename... Args>
inline cudaError_t launch_pdl(Kern kern, unsigned grid, unsigned block, size_t smem, cudaStream_t stream,
                              unsigned cluster_x, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    unsigned n = 0;
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster_x > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster_x;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

// ---- launchers (host side, defined next to their kernels) -------------------
// Int8Perm: one int8 per code, but every group of 8 channels stored as (c0,c2,c4,c6,c1,c3,c5,c7) --
// the order in which the GEMM's nibble unpack produces the 4-bit weights without a byte permute.
enum class StoreFmt : int { Nibble = 0, Int8 = 1, Int8Perm = 2 };

// Runtime prologue / offline fold share one kernel: multiply by mult[K] (or the
// constant `cnorm` if mult == nullptr), block FWHT, per-row absmax, quantize to
// +-qmax, store codes in `fmt`, store per-row step to delta.
// mult_after_rotation (fold-after sites, T = D^o R): multiply by `cnorm` before the butterflies
// and by mult[K] after them instead.
cudaError_t launch_transform_quantize(const void* x, fq_dtype xt, int64_t rows, int64_t K, int64_t ldx,
                                      const float* mult, float cnorm, bool mult_after_rotation, int block,
                                      int qmax, float clip_ratio, StoreFmt fmt, void* codes, float* delta,
                                      cudaStream_t stream);

// Same, for the site behind a gated MLP: x is [rows, 2K] = [gate | up] and the input is act(gate) * up
// (gate_kind 0 = SiLU, 1 = GELU-tanh, fixed binary32 arithmetic).
cudaError_t launch_gated_transform_quantize(const void* x, fq_dtype xt, int64_t rows, int64_t K, int64_t ldx, int gate_kind,
                                            const float* mult, float cnorm, bool mult_after_rotation, int block, int qmax,
                                            float clip_ratio, StoreFmt fmt, void* codes, float* delta, cudaStream_t stream);

// mult_w[c] = s_c * cnorm, mult_g[c] = (1/s_c) * cnorm (smooth == nullptr: both = cnorm).
cudaError_t launch_multipliers(const float* smooth, int64_t K, float cnorm, float* mult_w, float* mult_g,
                               cudaStream_t stream);

// w_scale[j] *= d[j], bias[j] *= d[j] for j < count (pointers already offset to the first channel).
cudaError_t launch_scale_outputs(float* w_scale, float* bias, const float* d, int64_t count, cudaStream_t stream);

cudaError_t launch_col_absmax(const void* x, fq_dtype xt, int64_t M, int64_t K, int64_t ldx, int accumulate,
                              float* out, cudaStream_t stream);
cudaError_t launch_smooth_scale(const float* a, const float* w, int64_t K, double alpha, float* s,
                                cudaStream_t stream);

// packed nibbles [rows, K/2] -> int8 [rows, K] holding 16*code (natural channel order).
cudaError_t launch_expand_nibbles(const void* packed, int64_t rows, int64_t K, void* out, cudaStream_t stream);

// Epilogue selector of the GEMM kernels.
struct GemmOut {
    void* y = nullptr;          // [M, N] of yt, leading dimension ldy   (nullptr when acc is used)
    fq_dtype yt = FQ_F32;
    int64_t ldy = 0;
    int32_t* acc = nullptr;     // raw accumulators [M, N] (debug/parity)
    const float* a_delta = nullptr;
};

// Reference-grade CUDA-core integer GEMM (dp4a); a8 = int8 activations [M, K].
cudaError_t launch_gemm_simt(const int8_t* a8, int64_t M, const Weights& W, int acc_shift, const GemmOut& out,
                             cudaStream_t stream);

// Short-batch weight streaming (4-bit weights, warp-level MMAs fed by a TMA ring).
//  - launch_linear_wonly4: weight-only projection of float activations, y = s^W (qW x) + b;
//  - launch_gemm_stream: the integer product + epilogue of the GEMM for batches gemm_stream_applies() accepts.
bool build_stream_tmap(Weights& W);
bool gemm_stream_applies(int64_t M, const Weights& W);
cudaError_t launch_gemm_stream(const int8_t* a8, int64_t M, const Weights& W, int acc_shift, const GemmOut& out,
                               cudaStream_t stream);
cudaError_t launch_linear_wonly4(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const Weights& W, void* y,
                                 fq_dtype yt, int64_t ldy, cudaStream_t stream);

// tcgen05 integer GEMM; a8 = int8 activations [M, K] (pitch K), 16-byte aligned.  `scratch` (device,
// 256-byte aligned, may be null) holds int32 partial tiles when the launch splits K over a cluster;
// gemm_scratch_bytes() is what the split the planner would pick for this shape needs.
fq_status launch_gemm_tcgen05(const int8_t* a8, int64_t M, const Weights& W, int acc_shift, const GemmOut& out,
                              void* scratch, size_t scratch_bytes, cudaStream_t stream);
// The GEMM of the runtime path: the streaming kernel for short batches on 4-bit weights, else the tcgen05 kernel.
fq_status launch_gemm(const int8_t* a8, int64_t M, const Weights& W, int acc_shift, const GemmOut& out,
                      void* scratch, size_t scratch_bytes, cudaStream_t stream);
size_t gemm_scratch_bytes(int64_t M, int64_t N, int64_t K, int bits);
// Enqueue whatever the GEMM of this shape needs cleared in `scratch` (the K split's tile counters).  Called by every
// entry point ahead of the call's first kernel; a launch_gemm on the same scratch must follow on the same stream.
fq_status gemm_prepare(int64_t M, const Weights& W, void* scratch, size_t scratch_bytes, cudaStream_t stream);

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link-time libcuda dependency).
// dims/box innermost first; strides_bytes has rank-1 entries (dimension 0 is contiguous).
bool encode_tiled(CUtensorMap* map, CUtensorMapDataType dt, uint32_t rank, const void* ptr, const uint64_t* dims,
                  const uint64_t* strides_bytes, const uint32_t* box, bool swizzle128);

// Streaming variant of the prologue (TMA-fed shared-memory ring). Returns cudaErrorNotSupported
// when the shape does not fit it; the caller then uses the register-only kernel.
cudaError_t launch_transform_quantize_ring(const void* x, fq_dtype xt, int64_t rows, int64_t K, int64_t ldx,
                                           const float* mult, float cnorm, bool mult_after_rotation, int block,
                                           int qmax, float clip_ratio, StoreFmt fmt, void* codes, float* delta,
                                           cudaStream_t stream);

// Stored composite rotation: u[t][b*beta + i] = sum_j B_b[i][j] * (x (.) diag)[t][perm[b*beta + j]] in binary32,
// u [rows, K] (pitch K).  beta in {16, 32, 64, 128, 256}; diag may be null.
cudaError_t launch_composite_rotate(const void* x, fq_dtype xt, int64_t rows, int64_t K, int64_t ldx, const float* diag,
                                    const int32_t* perm, const float* blocks, int beta, float* u, cudaStream_t stream);
// *bad_flag (device int) is set to 1 if an entry of perm[K] lies outside [0, K).
cudaError_t launch_perm_check(const int32_t* perm, int64_t K, int* bad_flag, cudaStream_t stream);

// GPTQ rounding (offline): the transform without its quantizer, the damped second moment and the upper factor U
// of its inverse (H, Mt: K x K scratch; *bad set if not positive definite), and the sweep that writes the codes.
cudaError_t launch_transform_rows(const void* x, fq_dtype xt, int64_t rows, int64_t K, int64_t ldx, const float* mult,
                                  float cnorm, int block, float* z, cudaStream_t stream);
cudaError_t launch_gptq_factor(const float* z, int64_t Mc, int64_t K, float damp, float* H, float* Mt, float* U,
                               uint8_t* dead, int* bad, cudaStream_t stream);
cudaError_t launch_gptq_sweep(const float* Wt, int64_t N, int64_t K, const float* U, const uint8_t* dead,
                              const float* w_scale, int bits, uint8_t* codes, cudaStream_t stream);

// Builds the weight-operand tensor map of a handle (after `codes` is allocated).
fq_status build_weight_tmap(Weights& W);

// Device watchdog word (see fq_device_status).
cudaError_t read_and_clear_watchdog(uint32_t* word);
uint32_t* watchdog_device_ptr();
// One-warp kernel whose bounded wait is certain to expire after limit_ns (see fq_watchdog_selftest).
cudaError_t launch_watchdog_selftest(uint64_t limit_ns, cudaStream_t stream);

}  // namespace fq
