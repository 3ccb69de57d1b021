// C ABI of the library (see include/fq.h): host-side argument checks, handle
// management and stream-ordered dispatch.  No entry point below touches data on
// the host; every step of the path runs in the kernels of this library.
#include <math.h>
#include <mutex>
#include <new>
#include <unordered_map>

#include "fq_common.cuh"

using namespace fq;

namespace fq {

namespace {
constexpr int kMaxDevices = 64;
struct DeviceFacts { int sms = 0, major = -1; };
std::mutex g_facts_mutex;
DeviceFacts g_facts[kMaxDevices];
std::unordered_map<const void*, size_t> g_smem_opt_in[kMaxDevices];
std::unordered_map<const void*, std::unordered_map<int, int>> g_resident[kMaxDevices];

DeviceFacts device_facts() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return DeviceFacts(); }
    const bool cached = dev >= 0 && dev < kMaxDevices;
    std::lock_guard<std::mutex> lock(g_facts_mutex);
    if (cached && g_facts[dev].sms > 0) return g_facts[dev];
    DeviceFacts f;
    if (cudaDeviceGetAttribute(&f.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&f.major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return DeviceFacts();
    }
    if (cached) g_facts[dev] = f;
    return f;
}
}  // namespace

int device_sm_count() {
    const int sms = device_facts().sms;
    return sms > 0 ? sms : 148;
}

int device_cc_major() { return device_facts().major; }

cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaGetLastError();
    const bool cached = dev >= 0 && dev < kMaxDevices;
    if (cached) {
        std::lock_guard<std::mutex> lock(g_facts_mutex);
        auto it = g_smem_opt_in[dev].find(kernel);
        if (it != g_smem_opt_in[dev].end() && it->second >= bytes) return cudaSuccess;
    }
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess && cached) {
        std::lock_guard<std::mutex> lock(g_facts_mutex);
        g_smem_opt_in[dev][kernel] = bytes;
    }
    return e;
}

int max_resident_blocks(const void* kernel, int threads) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return 1; }
    const bool cached = dev >= 0 && dev < kMaxDevices;
    if (cached) {
        std::lock_guard<std::mutex> lock(g_facts_mutex);
        auto it = g_resident[dev].find(kernel);
        if (it != g_resident[dev].end()) {
            auto jt = it->second.find(threads);
            if (jt != it->second.end()) return jt->second;
        }
    }
    int resident = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kernel, threads, 0) != cudaSuccess || resident < 1) {
        (void)cudaGetLastError();
        return 1;
    }
    if (cached) {
        std::lock_guard<std::mutex> lock(g_facts_mutex);
        g_resident[dev][kernel][threads] = resident;
    }
    return resident;
}

}  // namespace fq

namespace {

constexpr int64_t kMaxK = 131072;       // 127^2 * K and 256 * 49 * K stay below 2^31
constexpr int64_t kMaxPrologueK = 32768; // one token must fit the registers of one CTA

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool valid_block(int block, int64_t K) {
    // block 1 is the identity rotation (R = I: scale-only sites, weight-only handles)
    return block >= 1 && block <= 256 && (block & (block - 1)) == 0 && K > 0 && K % block == 0;
}

float block_norm(int block) { return (float)(1.0 / sqrt((double)block)); }

fq_status check_arch() {
    const int major = device_cc_major();
    if (major < 0) return FQ_ERR_CUDA;
    return major == 10 ? FQ_OK : FQ_ERR_ARCH;
}

fq_status check_shape(int64_t N, int64_t K, int block, int bits) {
    if (N < 0 || K <= 0) return FQ_ERR_INVALID_ARG;
    if (bits != 4 && bits != 8) return FQ_ERR_INVALID_ARG;
    if (!valid_block(block, K) || K % 32 != 0 || K > kMaxK || N % 8 != 0) return FQ_ERR_UNSUPPORTED;
    return FQ_OK;
}

fq_status alloc_handle(int64_t N, int64_t K, int block, int bits, Weights** out) {
    Weights* w = new (std::nothrow) Weights();
    if (!w) return FQ_ERR_NOMEM;
    w->N = N; w->K = K; w->block = block; w->bits = bits;
    cudaGetDevice(&w->device);
    const size_t code_bytes = (size_t)N * (size_t)K * bits / 8;
    bool ok = true;
    ok = ok && cudaMalloc(&w->codes, code_bytes > 0 ? code_bytes : 16) == cudaSuccess;
    ok = ok && cudaMalloc(&w->w_scale, sizeof(float) * (size_t)(N > 0 ? N : 4)) == cudaSuccess;
    ok = ok && cudaMalloc(&w->bias, sizeof(float) * (size_t)(N > 0 ? N : 4)) == cudaSuccess;
    ok = ok && cudaMalloc(&w->mult_g, sizeof(float) * (size_t)K) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        cudaFree(w->codes); cudaFree(w->w_scale); cudaFree(w->bias); cudaFree(w->mult_g);
        delete w;
        return FQ_ERR_NOMEM;
    }
    *out = w;
    return FQ_OK;
}

cudaEvent_t g_profile_mark = nullptr;   // see fq_profile_mark

struct Workspace {
    int8_t* a8;
    float* delta;
};

size_t ws_bytes_needed(int64_t M, int64_t K) {
    return align_up((size_t)M * (size_t)K, 256) + align_up(sizeof(float) * (size_t)M, 256);
}

fq_status carve(void* workspace, size_t ws_bytes, int64_t M, int64_t K, Workspace* ws) {
    if (!workspace) return FQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return FQ_ERR_ALIGNMENT;
    if (ws_bytes < ws_bytes_needed(M, K)) return FQ_ERR_NOMEM;
    ws->a8 = static_cast<int8_t*>(workspace);
    ws->delta = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + align_up((size_t)M * (size_t)K, 256));
    return FQ_OK;
}

// Whatever the caller's workspace holds beyond the activation codes and steps serves the GEMM as
// scratch for partial tiles (K split); without it the GEMM simply does not split.
void* scratch_of(void* workspace, size_t ws_bytes, int64_t M, int64_t K, size_t* avail) {
    const size_t base = ws_bytes_needed(M, K);
    *avail = 0;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 || ws_bytes <= base) return nullptr;
    *avail = ws_bytes - base;
    return static_cast<uint8_t*>(workspace) + base;
}

fq_status check_y(const void* y, fq_dtype yt, int64_t ldy, int64_t N) {
    if (!y) return FQ_ERR_INVALID_ARG;
    if (yt != FQ_F32 && yt != FQ_BF16) return FQ_ERR_INVALID_ARG;
    if (ldy < N) return FQ_ERR_INVALID_ARG;
    if (!aligned16(y) || ldy % 8 != 0) return FQ_ERR_ALIGNMENT;
    return FQ_OK;
}

// a_codes: canonical codes of width W->bits.  Produces the int8 operand of the GEMM.
fq_status gemm_from_codes(const void* a_codes, const float* a_delta, int64_t M, const fq_weights* Wp, int bits,
                          const GemmOut& out, void* workspace, size_t ws_bytes, cudaStream_t stream, bool simt) {
    const Weights* W = reinterpret_cast<const Weights*>(Wp);
    if (!W || M < 0) return FQ_ERR_INVALID_ARG;
    if (W->bits != bits) return FQ_ERR_UNSUPPORTED;
    if (M == 0 || W->N == 0) return FQ_OK;
    if (!a_codes || (!a_delta && !out.acc)) return FQ_ERR_INVALID_ARG;
    if (!aligned16(a_codes)) return FQ_ERR_ALIGNMENT;
    fq_status st = check_arch();
    if (st != FQ_OK) return st;
    const int8_t* a8 = static_cast<const int8_t*>(a_codes);
    int shift = 0;
    size_t scratch_bytes = 0;
    void* scratch = scratch_of(workspace, ws_bytes, M, W->K, &scratch_bytes);
    if (!simt) {
        st = gemm_prepare(M, *W, scratch, scratch_bytes, stream);
        if (st != FQ_OK) return st;
    }
    if (bits == 4) {
        Workspace ws;
        st = carve(workspace, ws_bytes, M, W->K, &ws);
        if (st != FQ_OK) return st;
        if (launch_expand_nibbles(a_codes, M, W->K, ws.a8, stream) != cudaSuccess) return FQ_ERR_CUDA;
        a8 = ws.a8;
        shift = 8;   // both operands carry 16*code
    }
    if (simt) return launch_gemm_simt(a8, M, *W, shift, out, stream) == cudaSuccess ? FQ_OK : FQ_ERR_CUDA;
    return launch_gemm(a8, M, *W, shift, out, scratch, scratch_bytes, stream);
}

fq_status linear_impl(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const fq_weights* Wp, int bits,
                      float clip_ratio, void* y, fq_dtype yt, int64_t ldy, void* workspace, size_t ws_bytes,
                      void* stream, int gate = -1) {
    const Weights* W = reinterpret_cast<const Weights*>(Wp);
    if (!W || M < 0) return FQ_ERR_INVALID_ARG;
    if (W->bits != bits) return FQ_ERR_UNSUPPORTED;
    if (W->composite) return FQ_ERR_UNSUPPORTED;   // two calls: fq_quantize_act_composite, then fq_gemm_*
    if (!(clip_ratio > 0.0f && clip_ratio <= 1.0f)) return FQ_ERR_INVALID_ARG;
    if (xt != FQ_F32 && xt != FQ_BF16) return FQ_ERR_INVALID_ARG;
    if (M == 0 || W->N == 0) return FQ_OK;
    if (!x || ldx < (gate >= 0 ? 2 * W->K : W->K)) return FQ_ERR_INVALID_ARG;
    if (!aligned16(x) || ldx % 8 != 0) return FQ_ERR_ALIGNMENT;
    if (W->K > kMaxPrologueK) return FQ_ERR_UNSUPPORTED;
    fq_status st = check_y(y, yt, ldy, W->N);
    if (st != FQ_OK) return st;
    st = check_arch();
    if (st != FQ_OK) return st;
    Workspace ws;
    st = carve(workspace, ws_bytes, M, W->K, &ws);
    if (st != FQ_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    size_t scratch_bytes = 0;
    void* scratch = scratch_of(workspace, ws_bytes, M, W->K, &scratch_bytes);
    st = gemm_prepare(M, *W, scratch, scratch_bytes, s);       // ahead of the prologue: see gemm_prepare
    if (st != FQ_OK) return st;
    // Prologue writes one int8 per code into the workspace (4-bit codes stay in [-7, 7] and are laid
    // out in the channel order the GEMM's nibble unpack gives the weights).
    const int qmax = bits == 4 ? 7 : 127;
    const StoreFmt fmt = bits == 4 ? StoreFmt::Int8Perm : StoreFmt::Int8;
    // a multiplier that is block^-1/2 in every channel is passed as "none": same products, no vector to stage
    const float* mult = W->mult_const ? nullptr : W->mult_g;
    const cudaError_t pe =
        gate >= 0 ? launch_gated_transform_quantize(x, xt, M, W->K, ldx, gate, mult, block_norm(W->block), W->fold_after,
                                                    W->block, qmax, clip_ratio, fmt, ws.a8, ws.delta, s)
                  : launch_transform_quantize(x, xt, M, W->K, ldx, mult, block_norm(W->block), W->fold_after, W->block,
                                              qmax, clip_ratio, fmt, ws.a8, ws.delta, s);
    if (pe != cudaSuccess) return FQ_ERR_CUDA;
    if (g_profile_mark != nullptr) {
        // Inside a stream capture the mark must be an external event-record node to stay readable.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) return FQ_ERR_CUDA;
        const unsigned flags = cap == cudaStreamCaptureStatusActive ? cudaEventRecordExternal : cudaEventRecordDefault;
        if (cudaEventRecordWithFlags(g_profile_mark, s, flags) != cudaSuccess) return FQ_ERR_CUDA;
    }
    GemmOut out;
    out.y = y; out.yt = yt; out.ldy = ldy; out.a_delta = ws.delta;
    // 4-bit weights are expanded to 16*code on chip: accumulator = 16 * integer sum.
    return launch_gemm(ws.a8, M, *W, bits == 4 ? 4 : 0, out, scratch, scratch_bytes, s);
}

}  // namespace

extern "C" {

const char* fq_status_string(fq_status s) {
    switch (s) {
        case FQ_OK: return "ok";
        case FQ_ERR_INVALID_ARG: return "invalid argument";
        case FQ_ERR_UNSUPPORTED: return "unsupported size or configuration";
        case FQ_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
        case FQ_ERR_ARCH: return "device is not sm_100";
        case FQ_ERR_CUDA: return "CUDA call failed";
        case FQ_ERR_NOMEM: return "out of memory or workspace too small";
        case FQ_ERR_TIMEOUT: return "bounded device wait expired";
    }
    return "unknown status";
}

namespace {
// fold-before (after == false): diag = s, W~ = W S R^T, runtime multiplier (1/s) * block^-1/2 ahead of the rotation.
// fold-after  (after == true):  diag = p, W~ = W R^T P, runtime multiplier 1/p behind the rotation.
fq_status fold_impl(const void* Wsrc, fq_dtype wt, int64_t N, int64_t K, int64_t ldw, const float* smooth, bool after,
                    const float* bias, int hadamard_block, int bits, void* stream, fq_weights** out) {
    if (!out) return FQ_ERR_INVALID_ARG;
    *out = nullptr;
    fq_status st = check_shape(N, K, hadamard_block, bits);
    if (st != FQ_OK) return st;
    if (wt != FQ_F32 && wt != FQ_BF16) return FQ_ERR_INVALID_ARG;
    if (K > kMaxPrologueK) return FQ_ERR_UNSUPPORTED;
    if (N > 0 && (!Wsrc || ldw < K)) return FQ_ERR_INVALID_ARG;
    if (N > 0 && (!aligned16(Wsrc) || ldw % 8 != 0)) return FQ_ERR_ALIGNMENT;
    if ((smooth && !aligned16(smooth)) || (bias && !aligned16(bias))) return FQ_ERR_ALIGNMENT;
    st = check_arch();
    if (st != FQ_OK) return st;
    Weights* w = nullptr;
    st = alloc_handle(N, K, hadamard_block, bits, &w);
    if (st != FQ_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float* mult_w = nullptr;   // s_c * block^-1/2, only needed while folding
    if (cudaMalloc(&mult_w, sizeof(float) * (size_t)K) != cudaSuccess) {
        fq_weights_destroy(reinterpret_cast<fq_weights*>(w));
        return FQ_ERR_NOMEM;
    }
    const float cn = block_norm(hadamard_block);
    w->fold_after = after;
    w->mult_const = smooth == nullptr;
    // fold-after: the two vectors are p itself (offline side) and 1/p (runtime side), without the block norm
    bool ok = launch_multipliers(smooth, K, after ? 1.0f : cn, mult_w, w->mult_g, s) == cudaSuccess;
    ok = ok && launch_transform_quantize(Wsrc, wt, N, K, ldw, mult_w, cn, after, hadamard_block, bits == 4 ? 7 : 127,
                                         1.0f, bits == 4 ? StoreFmt::Nibble : StoreFmt::Int8, w->codes, w->w_scale,
                                         s) == cudaSuccess;
    if (N > 0) {
        if (bias)
            ok = ok && cudaMemcpyAsync(w->bias, bias, sizeof(float) * (size_t)N, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
        else
            ok = ok && cudaMemsetAsync(w->bias, 0, sizeof(float) * (size_t)N, s) == cudaSuccess;
    }
    ok = ok && cudaStreamSynchronize(s) == cudaSuccess;   // mult_w is freed below; folding is offline
    cudaFree(mult_w);
    if (ok) ok = build_weight_tmap(*w) == FQ_OK;
    if (!ok) {
        fq_weights_destroy(reinterpret_cast<fq_weights*>(w));
        return FQ_ERR_CUDA;
    }
    *out = reinterpret_cast<fq_weights*>(w);
    return FQ_OK;
}

}  // namespace

fq_status fq_fold_weights(const void* Wsrc, fq_dtype wt, int64_t N, int64_t K, int64_t ldw, const float* smooth,
                          const float* bias, int hadamard_block, int bits, void* stream, fq_weights** out) {
    return fold_impl(Wsrc, wt, N, K, ldw, smooth, false, bias, hadamard_block, bits, stream, out);
}

fq_status fq_fold_weights_after(const void* Wsrc, fq_dtype wt, int64_t N, int64_t K, int64_t ldw, const float* post_scale,
                                const float* bias, int hadamard_block, int bits, void* stream, fq_weights** out) {
    if (!post_scale) return FQ_ERR_INVALID_ARG;
    return fold_impl(Wsrc, wt, N, K, ldw, post_scale, true, bias, hadamard_block, bits, stream, out);
}

fq_status fq_fold_weights_composite(const void* Wsrc, fq_dtype wt, int64_t N, int64_t K, int64_t ldw, const float* smooth,
                                    const float* bias, const int32_t* perm, const float* blocks, int block, int bits,
                                    void* stream, fq_weights** out) {
    if (!out) return FQ_ERR_INVALID_ARG;
    *out = nullptr;
    fq_status st = check_shape(N, K, block, bits);
    if (st != FQ_OK) return st;
    if (block < 16) return FQ_ERR_UNSUPPORTED;
    if (wt != FQ_F32 && wt != FQ_BF16) return FQ_ERR_INVALID_ARG;
    if (!perm || !blocks || K > kMaxPrologueK) return !perm || !blocks ? FQ_ERR_INVALID_ARG : FQ_ERR_UNSUPPORTED;
    if (N > 0 && (!Wsrc || ldw < K)) return FQ_ERR_INVALID_ARG;
    if ((smooth && !aligned16(smooth)) || (bias && !aligned16(bias))) return FQ_ERR_ALIGNMENT;
    st = check_arch();
    if (st != FQ_OK) return st;
    Weights* w = nullptr;
    st = alloc_handle(N, K, block, bits, &w);
    if (st != FQ_OK) return st;
    w->composite = true;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float* mult_w = nullptr;   // s_c, only needed while folding
    float* u = nullptr;        // rotated rows before rounding
    int* bad = nullptr;
    bool ok = cudaMalloc(&mult_w, sizeof(float) * (size_t)K) == cudaSuccess &&
              cudaMalloc(&u, sizeof(float) * (size_t)(N > 0 ? N : 1) * (size_t)K) == cudaSuccess &&
              cudaMalloc(&bad, sizeof(int)) == cudaSuccess;
    if (!ok) {
        cudaFree(mult_w); cudaFree(u); cudaFree(bad);
        fq_weights_destroy(reinterpret_cast<fq_weights*>(w));
        return FQ_ERR_NOMEM;
    }
    // the normalisation lives in the stored matrices: both vectors carry the diagonal only (s and 1/s)
    ok = cudaMemsetAsync(bad, 0, sizeof(int), s) == cudaSuccess;
    ok = ok && launch_perm_check(perm, K, bad, s) == cudaSuccess;
    ok = ok && launch_multipliers(smooth, K, 1.0f, mult_w, w->mult_g, s) == cudaSuccess;
    ok = ok && launch_composite_rotate(Wsrc, wt, N, K, ldw, smooth ? mult_w : nullptr, perm, blocks, block, u, s) == cudaSuccess;
    ok = ok && launch_transform_quantize(u, FQ_F32, N, K, K, nullptr, 1.0f, false, 1, bits == 4 ? 7 : 127, 1.0f,
                                         bits == 4 ? StoreFmt::Nibble : StoreFmt::Int8, w->codes, w->w_scale, s) == cudaSuccess;
    if (N > 0) {
        if (bias)
            ok = ok && cudaMemcpyAsync(w->bias, bias, sizeof(float) * (size_t)N, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
        else
            ok = ok && cudaMemsetAsync(w->bias, 0, sizeof(float) * (size_t)N, s) == cudaSuccess;
    }
    int bad_host = 0;
    ok = ok && cudaMemcpyAsync(&bad_host, bad, sizeof(int), cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(s) == cudaSuccess;   // the temporaries are freed below; folding is offline
    cudaFree(mult_w); cudaFree(u); cudaFree(bad);
    if (ok && !bad_host) ok = build_weight_tmap(*w) == FQ_OK;
    if (!ok || bad_host) {
        fq_weights_destroy(reinterpret_cast<fq_weights*>(w));
        return bad_host ? FQ_ERR_INVALID_ARG : FQ_ERR_CUDA;
    }
    *out = reinterpret_cast<fq_weights*>(w);
    return FQ_OK;
}

fq_status fq_fold_weights_gptq(const void* Wsrc, fq_dtype wt, int64_t N, int64_t K, int64_t ldw, const float* smooth,
                               const float* bias, const void* calib, fq_dtype ct, int64_t Mc, int64_t ldc,
                               int hadamard_block, int bits, float damp, void* stream, fq_weights** out) {
    if (!out) return FQ_ERR_INVALID_ARG;
    *out = nullptr;
    fq_status st = check_shape(N, K, hadamard_block, bits);
    if (st != FQ_OK) return st;
    if (K > 16384) return FQ_ERR_UNSUPPORTED;         // three K x K binary32 matrices; a row of K floats per CTA in shared memory
    if ((wt != FQ_F32 && wt != FQ_BF16) || (ct != FQ_F32 && ct != FQ_BF16)) return FQ_ERR_INVALID_ARG;
    if (!calib || Mc < 1 || ldc < K || !(damp >= 0.0f)) return FQ_ERR_INVALID_ARG;
    if (N > 0 && (!Wsrc || ldw < K)) return FQ_ERR_INVALID_ARG;
    if (N > 0 && (!aligned16(Wsrc) || ldw % 8 != 0)) return FQ_ERR_ALIGNMENT;
    if ((smooth && !aligned16(smooth)) || (bias && !aligned16(bias))) return FQ_ERR_ALIGNMENT;
    st = check_arch();
    if (st != FQ_OK) return st;
    Weights* w = nullptr;
    st = alloc_handle(N, K, hadamard_block, bits, &w);
    if (st != FQ_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t kk = sizeof(float) * (size_t)K * (size_t)K;
    float *mult_w = nullptr, *Wt = nullptr, *Z = nullptr, *H = nullptr, *Mt = nullptr, *U = nullptr;
    uint8_t* dead = nullptr;
    int* bad = nullptr;
    bool ok = cudaMalloc(&mult_w, sizeof(float) * (size_t)K) == cudaSuccess &&
              cudaMalloc(&Wt, sizeof(float) * (size_t)(N > 0 ? N : 1) * (size_t)K) == cudaSuccess &&
              cudaMalloc(&Z, sizeof(float) * (size_t)Mc * (size_t)K) == cudaSuccess &&
              cudaMalloc(&H, kk) == cudaSuccess && cudaMalloc(&Mt, kk) == cudaSuccess && cudaMalloc(&U, kk) == cudaSuccess &&
              cudaMalloc(&dead, (size_t)K) == cudaSuccess && cudaMalloc(&bad, sizeof(int)) == cudaSuccess;
    auto release = [&]() {
        cudaFree(mult_w); cudaFree(Wt); cudaFree(Z); cudaFree(H); cudaFree(Mt); cudaFree(U); cudaFree(dead); cudaFree(bad);
    };
    if (!ok) {
        release();
        fq_weights_destroy(reinterpret_cast<fq_weights*>(w));
        return FQ_ERR_NOMEM;
    }
    const float cn = block_norm(hadamard_block);
    const int qmax = bits == 4 ? 7 : 127;
    w->mult_const = smooth == nullptr;
    ok = cudaMemsetAsync(bad, 0, sizeof(int), s) == cudaSuccess;
    ok = ok && launch_multipliers(smooth, K, cn, mult_w, w->mult_g, s) == cudaSuccess;
    // per-output-channel steps: those of the round-to-nearest fold (its codes are overwritten by the sweep)
    ok = ok && launch_transform_quantize(Wsrc, wt, N, K, ldw, mult_w, cn, false, hadamard_block, qmax, 1.0f,
                                         bits == 4 ? StoreFmt::Nibble : StoreFmt::Int8, w->codes, w->w_scale, s) == cudaSuccess;
    ok = ok && launch_transform_rows(Wsrc, wt, N, K, ldw, mult_w, cn, hadamard_block, Wt, s) == cudaSuccess;
    ok = ok && launch_transform_rows(calib, ct, Mc, K, ldc, w->mult_g, cn, hadamard_block, Z, s) == cudaSuccess;
    ok = ok && launch_gptq_factor(Z, Mc, K, damp, H, Mt, U, dead, bad, s) == cudaSuccess;
    ok = ok && launch_gptq_sweep(Wt, N, K, U, dead, w->w_scale, bits, w->codes, s) == cudaSuccess;
    if (N > 0) {
        if (bias)
            ok = ok && cudaMemcpyAsync(w->bias, bias, sizeof(float) * (size_t)N, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
        else
            ok = ok && cudaMemsetAsync(w->bias, 0, sizeof(float) * (size_t)N, s) == cudaSuccess;
    }
    int bad_host = 0;
    ok = ok && cudaMemcpyAsync(&bad_host, bad, sizeof(int), cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(s) == cudaSuccess;   // offline: the temporaries are freed below
    release();
    if (ok && !bad_host) ok = build_weight_tmap(*w) == FQ_OK;
    if (!ok || bad_host) {
        fq_weights_destroy(reinterpret_cast<fq_weights*>(w));
        return bad_host ? FQ_ERR_INVALID_ARG : FQ_ERR_CUDA;
    }
    *out = reinterpret_cast<fq_weights*>(w);
    return FQ_OK;
}

fq_status fq_quantize_act_gated(const void* gate_up, fq_dtype xt, int64_t M, int64_t K, int64_t ld, fq_gate_act act,
                                const float* mult_g, int hadamard_block, int bits, float clip_ratio, void* codes_out,
                                float* delta_out, void* stream) {
    if (M < 0 || (bits != 4 && bits != 8)) return FQ_ERR_INVALID_ARG;
    if (xt != FQ_F32 && xt != FQ_BF16) return FQ_ERR_INVALID_ARG;
    if (act != FQ_GATE_SILU && act != FQ_GATE_GELU_TANH) return FQ_ERR_INVALID_ARG;
    if (!(clip_ratio > 0.0f && clip_ratio <= 1.0f)) return FQ_ERR_INVALID_ARG;
    if (!valid_block(hadamard_block, K) || K % 32 != 0 || K > kMaxPrologueK) return FQ_ERR_UNSUPPORTED;
    if (M == 0) return FQ_OK;
    if (!gate_up || !codes_out || !delta_out || ld < 2 * K) return FQ_ERR_INVALID_ARG;
    if (!aligned16(gate_up) || !aligned16(codes_out) || ld % 8 != 0 || (mult_g && !aligned16(mult_g)))
        return FQ_ERR_ALIGNMENT;
    fq_status st = check_arch();
    if (st != FQ_OK) return st;
    return launch_gated_transform_quantize(gate_up, xt, M, K, ld, (int)act, mult_g, block_norm(hadamard_block), false,
                                           hadamard_block, bits == 4 ? 7 : 127, clip_ratio,
                                           bits == 4 ? StoreFmt::Nibble : StoreFmt::Int8, codes_out, delta_out,
                                           static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? FQ_OK : FQ_ERR_CUDA;
}

fq_status fq_linear_gated(const void* gate_up, fq_dtype xt, int64_t M, int64_t ld, fq_gate_act act, const fq_weights* W,
                          float clip_ratio, void* y, fq_dtype yt, int64_t ldy, void* workspace, size_t ws_bytes,
                          void* stream) {
    const Weights* w = reinterpret_cast<const Weights*>(W);
    if (!w) return FQ_ERR_INVALID_ARG;
    if (act != FQ_GATE_SILU && act != FQ_GATE_GELU_TANH) return FQ_ERR_INVALID_ARG;
    return linear_impl(gate_up, xt, M, ld, W, w->bits, clip_ratio, y, yt, ldy, workspace, ws_bytes, stream, (int)act);
}

int fq_weights_composite(const fq_weights* wp) {
    const Weights* w = reinterpret_cast<const Weights*>(wp);
    return (w && w->composite) ? 1 : 0;
}

fq_status fq_quantize_act_composite(const void* x, fq_dtype xt, int64_t M, int64_t K, int64_t ldx, const float* mult_g,
                                    const int32_t* perm, const float* blocks, int block, int bits, float clip_ratio,
                                    void* codes_out, float* delta_out, void* workspace, size_t ws_bytes, void* stream) {
    if (M < 0 || (bits != 4 && bits != 8)) return FQ_ERR_INVALID_ARG;
    if (xt != FQ_F32 && xt != FQ_BF16) return FQ_ERR_INVALID_ARG;
    if (!(clip_ratio > 0.0f && clip_ratio <= 1.0f)) return FQ_ERR_INVALID_ARG;
    if (!valid_block(block, K) || block < 16 || K % 32 != 0 || K > kMaxPrologueK) return FQ_ERR_UNSUPPORTED;
    if (M == 0) return FQ_OK;
    if (!x || !codes_out || !delta_out || !perm || !blocks || ldx < K) return FQ_ERR_INVALID_ARG;
    if (!aligned16(codes_out) || (mult_g && !aligned16(mult_g))) return FQ_ERR_ALIGNMENT;
    if (!workspace || ws_bytes < sizeof(float) * (size_t)M * (size_t)K) return FQ_ERR_NOMEM;
    if (!aligned16(workspace)) return FQ_ERR_ALIGNMENT;
    fq_status st = check_arch();
    if (st != FQ_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float* u = static_cast<float*>(workspace);
    if (launch_composite_rotate(x, xt, M, K, ldx, mult_g, perm, blocks, block, u, s) != cudaSuccess) return FQ_ERR_CUDA;
    return launch_transform_quantize(u, FQ_F32, M, K, K, nullptr, 1.0f, false, 1, bits == 4 ? 7 : 127, clip_ratio,
                                     bits == 4 ? StoreFmt::Nibble : StoreFmt::Int8, codes_out, delta_out, s) == cudaSuccess
               ? FQ_OK : FQ_ERR_CUDA;
}

int fq_weights_fold_after(const fq_weights* wp) {
    const Weights* w = reinterpret_cast<const Weights*>(wp);
    return (w && w->fold_after) ? 1 : 0;
}

fq_status fq_weights_destroy(fq_weights* wp) {
    Weights* w = reinterpret_cast<Weights*>(wp);
    if (!w) return FQ_OK;
    cudaFree(w->codes); cudaFree(w->w_scale); cudaFree(w->bias); cudaFree(w->mult_g);
    delete w;
    return FQ_OK;
}

fq_status fq_weights_info(const fq_weights* wp, int64_t* N, int64_t* K, int* hadamard_block, int* bits) {
    const Weights* w = reinterpret_cast<const Weights*>(wp);
    if (!w) return FQ_ERR_INVALID_ARG;
    if (N) *N = w->N;
    if (K) *K = w->K;
    if (hadamard_block) *hadamard_block = w->block;
    if (bits) *bits = w->bits;
    return FQ_OK;
}

const float* fq_weights_multiplier(const fq_weights* wp) {
    const Weights* w = reinterpret_cast<const Weights*>(wp);
    return w ? w->mult_g : nullptr;
}

fq_status fq_weights_export(const fq_weights* wp, void* codes, float* w_scale, float* mult_g, float* bias,
                            void* stream) {
    const Weights* w = reinterpret_cast<const Weights*>(wp);
    if (!w) return FQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t code_bytes = (size_t)w->N * (size_t)w->K * w->bits / 8;
    bool ok = true;
    if (codes && code_bytes) ok = ok && cudaMemcpyAsync(codes, w->codes, code_bytes, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    if (w_scale && w->N) ok = ok && cudaMemcpyAsync(w_scale, w->w_scale, sizeof(float) * (size_t)w->N, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    if (bias && w->N) ok = ok && cudaMemcpyAsync(bias, w->bias, sizeof(float) * (size_t)w->N, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    if (mult_g) ok = ok && cudaMemcpyAsync(mult_g, w->mult_g, sizeof(float) * (size_t)w->K, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    return ok ? FQ_OK : FQ_ERR_CUDA;
}

namespace {
fq_status import_impl(const void* codes, const float* w_scale, const float* mult_g, bool after, const float* bias,
                      int64_t N, int64_t K, int hadamard_block, int bits, void* stream, fq_weights** out) {
    if (!out) return FQ_ERR_INVALID_ARG;
    *out = nullptr;
    fq_status st = check_shape(N, K, hadamard_block, bits);
    if (st != FQ_OK) return st;
    if (N > 0 && (!codes || !w_scale)) return FQ_ERR_INVALID_ARG;
    st = check_arch();
    if (st != FQ_OK) return st;
    Weights* w = nullptr;
    st = alloc_handle(N, K, hadamard_block, bits, &w);
    if (st != FQ_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t code_bytes = (size_t)N * (size_t)K * bits / 8;
    w->fold_after = after && mult_g != nullptr;
    w->mult_const = mult_g == nullptr;
    bool ok = true;
    if (N > 0) {
        ok = ok && cudaMemcpyAsync(w->codes, codes, code_bytes, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(w->w_scale, w_scale, sizeof(float) * (size_t)N, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
        if (bias)
            ok = ok && cudaMemcpyAsync(w->bias, bias, sizeof(float) * (size_t)N, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
        else
            ok = ok && cudaMemsetAsync(w->bias, 0, sizeof(float) * (size_t)N, s) == cudaSuccess;
    }
    if (mult_g)
        ok = ok && cudaMemcpyAsync(w->mult_g, mult_g, sizeof(float) * (size_t)K, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    else
        ok = ok && launch_multipliers(nullptr, K, block_norm(hadamard_block), nullptr, w->mult_g, s) == cudaSuccess;
    // A handle is complete when it is returned (as after fq_fold_weights): the GEMM's weight
    // producers start reading it before the kernels ahead of them in the stream have finished.
    ok = ok && cudaStreamSynchronize(s) == cudaSuccess;
    if (ok) ok = build_weight_tmap(*w) == FQ_OK;
    if (!ok) {
        fq_weights_destroy(reinterpret_cast<fq_weights*>(w));
        return FQ_ERR_CUDA;
    }
    *out = reinterpret_cast<fq_weights*>(w);
    return FQ_OK;
}
}  // namespace

fq_status fq_weights_import(const void* codes, const float* w_scale, const float* mult_g, const float* bias,
                            int64_t N, int64_t K, int hadamard_block, int bits, void* stream, fq_weights** out) {
    return import_impl(codes, w_scale, mult_g, false, bias, N, K, hadamard_block, bits, stream, out);
}

fq_status fq_weights_import_after(const void* codes, const float* w_scale, const float* mult_post, const float* bias,
                                  int64_t N, int64_t K, int hadamard_block, int bits, void* stream, fq_weights** out) {
    if (!mult_post) return FQ_ERR_INVALID_ARG;
    return import_impl(codes, w_scale, mult_post, true, bias, N, K, hadamard_block, bits, stream, out);
}

fq_status fq_weights_set_multiplier(fq_weights* wp, const float* mult, void* stream) {
    Weights* w = reinterpret_cast<Weights*>(wp);
    if (!w) return FQ_ERR_INVALID_ARG;
    if (mult && !aligned16(mult)) return FQ_ERR_ALIGNMENT;
    if (w->fold_after && !mult) return FQ_ERR_INVALID_ARG;     // a fold-after handle keeps a post-rotation vector
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    bool ok;
    if (mult)
        ok = cudaMemcpyAsync(w->mult_g, mult, sizeof(float) * (size_t)w->K, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    else
        ok = launch_multipliers(nullptr, w->K, block_norm(w->block), nullptr, w->mult_g, s) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(s) == cudaSuccess;        // the handle is complete when the call returns
    if (ok) w->mult_const = mult == nullptr;
    return ok ? FQ_OK : FQ_ERR_CUDA;
}

fq_status fq_weights_scale_outputs(fq_weights* wp, int64_t first, int64_t count, const float* d, void* stream) {
    Weights* w = reinterpret_cast<Weights*>(wp);
    if (!w || !d || first < 0 || count < 0 || first + count > w->N) return FQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    bool ok = launch_scale_outputs(w->w_scale + first, w->bias + first, d, count, s) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(s) == cudaSuccess;
    return ok ? FQ_OK : FQ_ERR_CUDA;
}

fq_status fq_col_absmax(const void* x, fq_dtype xt, int64_t M, int64_t K, int64_t ldx, int accumulate, float* out,
                        void* stream) {
    if (M < 0 || K <= 0 || !out || (M > 0 && (!x || ldx < K))) return FQ_ERR_INVALID_ARG;
    if (xt != FQ_F32 && xt != FQ_BF16) return FQ_ERR_INVALID_ARG;
    return launch_col_absmax(x, xt, M, K, ldx, accumulate, out, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? FQ_OK : FQ_ERR_CUDA;
}

fq_status fq_smooth_scale(const float* a, const float* w, int64_t K, double alpha, float* s, void* stream) {
    if (!a || !w || !s || K <= 0 || !(alpha >= 0.0 && alpha <= 1.0)) return FQ_ERR_INVALID_ARG;
    return launch_smooth_scale(a, w, K, alpha, s, static_cast<cudaStream_t>(stream)) == cudaSuccess ? FQ_OK
                                                                                                     : FQ_ERR_CUDA;
}

namespace {
fq_status quantize_impl(const void* x, fq_dtype xt, int64_t M, int64_t K, int64_t ldx, const float* mult_g, bool after,
                        int hadamard_block, int bits, float clip_ratio, void* codes_out, float* delta_out,
                        void* stream) {
    if (M < 0 || K <= 0) return FQ_ERR_INVALID_ARG;
    if (bits != 4 && bits != 8) return FQ_ERR_INVALID_ARG;
    if (!(clip_ratio > 0.0f && clip_ratio <= 1.0f)) return FQ_ERR_INVALID_ARG;
    if (xt != FQ_F32 && xt != FQ_BF16) return FQ_ERR_INVALID_ARG;
    if (!valid_block(hadamard_block, K) || K % 32 != 0 || K > kMaxPrologueK) return FQ_ERR_UNSUPPORTED;
    if (M == 0) return FQ_OK;
    if (!x || !codes_out || !delta_out || ldx < K) return FQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(codes_out) || ldx % 8 != 0 || (mult_g && !aligned16(mult_g)))
        return FQ_ERR_ALIGNMENT;
    fq_status st = check_arch();
    if (st != FQ_OK) return st;
    cudaError_t e = launch_transform_quantize(x, xt, M, K, ldx, mult_g, block_norm(hadamard_block), after,
                                              hadamard_block, bits == 4 ? 7 : 127, clip_ratio,
                                              bits == 4 ? StoreFmt::Nibble : StoreFmt::Int8, codes_out, delta_out,
                                              static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? FQ_OK : FQ_ERR_CUDA;
}
}  // namespace

fq_status fq_quantize_act(const void* x, fq_dtype xt, int64_t M, int64_t K, int64_t ldx, const float* mult_g,
                          int hadamard_block, int bits, float clip_ratio, void* codes_out, float* delta_out,
                          void* stream) {
    return quantize_impl(x, xt, M, K, ldx, mult_g, false, hadamard_block, bits, clip_ratio, codes_out, delta_out, stream);
}

fq_status fq_quantize_act_after(const void* x, fq_dtype xt, int64_t M, int64_t K, int64_t ldx, const float* mult_post,
                                int hadamard_block, int bits, float clip_ratio, void* codes_out, float* delta_out,
                                void* stream) {
    if (!mult_post) return FQ_ERR_INVALID_ARG;
    return quantize_impl(x, xt, M, K, ldx, mult_post, true, hadamard_block, bits, clip_ratio, codes_out, delta_out, stream);
}

fq_status fq_gemm_w4a4(const void* a_codes, const float* a_delta, int64_t M, const fq_weights* W, void* y,
                       fq_dtype yt, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    if (!W) return FQ_ERR_INVALID_ARG;
    if (M > 0 && reinterpret_cast<const Weights*>(W)->N > 0) {
        fq_status st = check_y(y, yt, ldy, reinterpret_cast<const Weights*>(W)->N);
        if (st != FQ_OK) return st;
    }
    GemmOut out;
    out.y = y; out.yt = yt; out.ldy = ldy; out.a_delta = a_delta;
    return gemm_from_codes(a_codes, a_delta, M, W, 4, out, workspace, ws_bytes, static_cast<cudaStream_t>(stream), false);
}

fq_status fq_gemm_w8a8(const void* a_codes, const float* a_delta, int64_t M, const fq_weights* W, void* y,
                       fq_dtype yt, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    if (!W) return FQ_ERR_INVALID_ARG;
    if (M > 0 && reinterpret_cast<const Weights*>(W)->N > 0) {
        fq_status st = check_y(y, yt, ldy, reinterpret_cast<const Weights*>(W)->N);
        if (st != FQ_OK) return st;
    }
    GemmOut out;
    out.y = y; out.yt = yt; out.ldy = ldy; out.a_delta = a_delta;
    return gemm_from_codes(a_codes, a_delta, M, W, 8, out, workspace, ws_bytes, static_cast<cudaStream_t>(stream), false);
}

fq_status fq_linear_w4a4(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const fq_weights* W, float clip_ratio,
                         void* y, fq_dtype yt, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    return linear_impl(x, xt, M, ldx, W, 4, clip_ratio, y, yt, ldy, workspace, ws_bytes, stream);
}

fq_status fq_linear_w8a8(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const fq_weights* W, float clip_ratio,
                         void* y, fq_dtype yt, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    return linear_impl(x, xt, M, ldx, W, 8, clip_ratio, y, yt, ldy, workspace, ws_bytes, stream);
}

fq_status fq_linear_w4a16(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const fq_weights* Wp, void* y,
                          fq_dtype yt, int64_t ldy, void* stream) {
    const Weights* W = reinterpret_cast<const Weights*>(Wp);
    if (!W || M < 0) return FQ_ERR_INVALID_ARG;
    if (W->bits != 4) return FQ_ERR_UNSUPPORTED;
    if (xt != FQ_F32 && xt != FQ_BF16) return FQ_ERR_INVALID_ARG;
    if (M == 0 || W->N == 0) return FQ_OK;
    if (!x || ldx < W->K) return FQ_ERR_INVALID_ARG;
    if (!aligned16(x) || ldx % 8 != 0) return FQ_ERR_ALIGNMENT;
    fq_status st = check_y(y, yt, ldy, W->N);
    if (st != FQ_OK) return st;
    st = check_arch();
    if (st != FQ_OK) return st;
    return launch_linear_wonly4(x, xt, M, ldx, *W, y, yt, ldy, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? FQ_OK : FQ_ERR_CUDA;
}

size_t fq_workspace_bytes(int64_t M, int64_t K, int64_t N, int bits) {
    if (M <= 0 || K <= 0) return 256;
    return ws_bytes_needed(M, K) + align_up(gemm_scratch_bytes(M, N, K, bits == 4 ? 4 : 8), 256);
}

fq_status fq_gemm_acc_i32(const void* a_codes, int64_t M, const fq_weights* W, int32_t* acc, void* workspace,
                          size_t ws_bytes, void* stream) {
    if (!W) return FQ_ERR_INVALID_ARG;
    const Weights* w = reinterpret_cast<const Weights*>(W);
    if (M > 0 && w->N > 0 && !acc) return FQ_ERR_INVALID_ARG;
    GemmOut out;
    out.acc = acc;
    return gemm_from_codes(a_codes, nullptr, M, W, w->bits, out, workspace, ws_bytes, static_cast<cudaStream_t>(stream), false);
}

fq_status fq_gemm_simt(const void* a_codes, const float* a_delta, int64_t M, const fq_weights* W, void* y,
                       fq_dtype yt, int64_t ldy, int32_t* acc, void* workspace, size_t ws_bytes, void* stream) {
    if (!W) return FQ_ERR_INVALID_ARG;
    const Weights* w = reinterpret_cast<const Weights*>(W);
    GemmOut out;
    if (acc) {
        out.acc = acc;
    } else {
        if (M > 0 && w->N > 0) {
            fq_status st = check_y(y, yt, ldy, w->N);
            if (st != FQ_OK) return st;
        }
        out.y = y; out.yt = yt; out.ldy = ldy; out.a_delta = a_delta;
    }
    return gemm_from_codes(a_codes, a_delta, M, W, w->bits, out, workspace, ws_bytes, static_cast<cudaStream_t>(stream), true);
}

fq_status fq_profile_mark(void* event) {
    g_profile_mark = static_cast<cudaEvent_t>(event);
    return FQ_OK;
}

fq_status fq_watchdog_selftest(uint64_t limit_ns, void* stream) {
    fq_status st = check_arch();
    if (st != FQ_OK) return st;
    if (limit_ns < 1000ull) limit_ns = 1000ull;
    if (limit_ns > 100000000ull) limit_ns = 100000000ull;
    return launch_watchdog_selftest(limit_ns, static_cast<cudaStream_t>(stream)) == cudaSuccess ? FQ_OK : FQ_ERR_CUDA;
}

fq_status fq_device_status(uint32_t* detail) {
    uint32_t word = 0;
    if (read_and_clear_watchdog(&word) != cudaSuccess) return FQ_ERR_CUDA;
    if (detail) *detail = word;
    return word ? FQ_ERR_TIMEOUT : FQ_OK;
}

}  // extern "C"
