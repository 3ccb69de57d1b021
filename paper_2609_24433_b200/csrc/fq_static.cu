// fq_linear_w4a4_static: the fused W4A4 linear for callers that must not allocate.
//
// fq_linear_w4a4 keeps the quantized activations (one int8 per code) and the
// per-token steps in a caller-supplied workspace between its two kernels.  Some
// callers have nowhere to get that workspace from: an enqueue callback of an
// inference-engine plugin may not call cudaMalloc, a robot's control loop cannot
// afford the device-wide synchronisation an allocation may imply, and a process
// whose device memory was handed out once at start-up has no allocator to ask.
// For them the same two kernels run here on a fixed scratch area that lives in
// the library image itself.
//
// The scratch is a file-scope __device__ array.  In host code that name is only
// a host-side stand-in for the symbol, not an address a kernel may use, so the
// device address is looked up with cudaGetSymbolAddress -- once per device, with
// that device current -- and it is that pointer which the kernels receive.
#include <mutex>

#include "fq_common.cuh"

#define FQ_STATIC_MAX_CODE_BYTES_ (4ll << 20)
#define FQ_STATIC_MAX_TOKENS_ 16384ll

namespace {

constexpr size_t kCodeBytes = (size_t)FQ_STATIC_MAX_CODE_BYTES_;
constexpr size_t kDeltaBytes = sizeof(float) * (size_t)FQ_STATIC_MAX_TOKENS_;

// Held by every GPU that loads the library, until the process exits: 4 MiB + 64 KiB.
static __device__ __align__(256) unsigned char g_static_scratch[kCodeBytes + kDeltaBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
unsigned char* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch on the CURRENT device (looked up on first use).
fq_status scratch_on_current_device(unsigned char** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FQ_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return FQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        unsigned char* ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return FQ_ERR_CUDA;
        }
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return FQ_OK;
}

}  // namespace

extern "C" fq_status fq_linear_w4a4_static(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const fq_weights* Wp,
                                           float clip_ratio, void* y, fq_dtype yt, int64_t ldy, void* stream) {
    using namespace fq;
    const Weights* W = reinterpret_cast<const Weights*>(Wp);
    if (!W || M < 0) return FQ_ERR_INVALID_ARG;
    if (W->bits != 4 || W->composite) return FQ_ERR_UNSUPPORTED;
    if (!(clip_ratio > 0.0f && clip_ratio <= 1.0f)) return FQ_ERR_INVALID_ARG;
    if ((xt != FQ_F32 && xt != FQ_BF16) || (yt != FQ_F32 && yt != FQ_BF16)) return FQ_ERR_INVALID_ARG;
    if (M == 0 || W->N == 0) {
        // A call without tokens still performs the one-time set-up for the current device (it loads the
        // module that holds the scratch and looks the address up), so it can serve as the start-up call.
        unsigned char* warm = nullptr;
        return device_cc_major() == 10 ? scratch_on_current_device(&warm) : FQ_OK;
    }
    // The built-in scratch is fixed: refuse anything that does not fit instead of overrunning it.
    if (M > FQ_STATIC_MAX_TOKENS_ || (size_t)M * (size_t)W->K > kCodeBytes) return FQ_ERR_NOMEM;
    if (!x || !y || ldx < W->K || ldy < W->N) return FQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) & 15u) || (reinterpret_cast<uintptr_t>(y) & 15u) || ldx % 8 != 0 || ldy % 8 != 0)
        return FQ_ERR_ALIGNMENT;
    if (W->K > 32768) return FQ_ERR_UNSUPPORTED;
    const int major = device_cc_major();
    if (major < 0) return FQ_ERR_CUDA;
    if (major != 10) return FQ_ERR_ARCH;

    unsigned char* scratch = nullptr;
    fq_status st = scratch_on_current_device(&scratch);
    if (st != FQ_OK) return st;
    int8_t* a8 = reinterpret_cast<int8_t*>(scratch);                 // [M, K] codes, rows < M rewritten below
    float* delta = reinterpret_cast<float*>(scratch + kCodeBytes);   // [M] steps,    rows < M rewritten below
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float cnorm = (float)(1.0 / sqrt((double)W->block));
    if (launch_transform_quantize(x, xt, M, W->K, ldx, W->mult_const ? nullptr : W->mult_g, cnorm, W->fold_after, W->block, 7, clip_ratio, StoreFmt::Int8Perm, a8,
                                  delta, s) != cudaSuccess)
        return FQ_ERR_CUDA;
    GemmOut out;
    out.y = y; out.yt = yt; out.ldy = ldy; out.a_delta = delta;
    return launch_gemm(a8, M, *W, 4, out, nullptr, 0, s);   // no scratch: the GEMM does not split K
}
