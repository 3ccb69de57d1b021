// Streaming variant of the runtime prologue (Alg. 1 runtime half lines 1-2, Eq. 5) for long
// batches: same arithmetic, bit for bit, as transform_quantize_kernel, but tokens reach the
// SM through a TMA-fed shared-memory ring so that many rows are in flight per SM regardless
// of register pressure.
//
//   - One persistent CTA of 1024 threads per SM, split into row groups of `gw` warps; a
//     group owns one token at a time, a thread owns E = 32 consecutive channels of it.
//   - A token row is fetched as a 3-D tiled TMA box {128 bytes, K*e/128, 1} with the 128-byte
//     swizzle, which makes the per-thread 64/128-byte reads bank-conflict free.  The per-
//     channel multiplier is staged once in shared memory with the same swizzle.
//   - Each group runs `depth` slots: the group barrier that exchanges the per-warp maxima also
//     proves that every warp has finished reading the slot, so the group's leader refills it
//     right there -- no separate "empty" barrier.
//   - Strides 1..16 run in registers, strides 32..block/2 by warp shuffles (2 or 3 stages for
//     blocks of 128 / 256 channels instead of the 3 or 4 a 16-channel thread needs).
#include <cuda_bf16.h>
#include <float.h>

#include "fq_common.cuh"
#include "ptx_sm100.cuh"
#include "act_common.cuh"

namespace fq {
namespace {

constexpr int E = 32;
constexpr int kThreads = 512;
constexpr int kMaxSlots = 128;

// 128-byte swizzle of a byte offset inside a 1024-byte aligned region.
__device__ __forceinline__ uint32_t swz128(uint32_t off) { return off ^ (((off >> 7) & 7u) << 4); }

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
// Group barrier that also ANDs a predicate over the group (ids 1..15, count a multiple of 32).
__device__ __forceinline__ bool group_barrier_and(int id, int count, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %3, 0;\n\t"
        "bar.red.and.pred p, %1, %2, q;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(id), "r"(count), "r"((uint32_t)pred)
        : "memory");
    return r != 0;
}

struct RingParams {
    int64_t rows;
    int K;
    int block;
    float cnorm, qmax, clip_ratio;
    const float* mult;
    uint8_t* codes;
    float* delta;
    int gw;            // warps per row group (power of two)
    int depth;         // ring slots per group
    uint32_t slot_bytes;
    uint32_t g_bytes;  // bytes of the multiplier stage (0 if no multiplier)
    uint32_t* watchdog;
};

template <typename XT, int FMT, bool CLAMP>
__global__ void __launch_bounds__(kThreads, 1)
transform_quantize_ring_kernel(const __grid_constant__ CUtensorMap map_x, const RingParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[kMaxSlots];
    __shared__ float s_part[2][32];
    __shared__ int s_abort;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ngroups = (kThreads / 32) / p.gw;
    const int group = warp / p.gw;
    const int wg = warp - group * p.gw;
    const int col0 = (wg * 32 + lane) * E;
    const bool col_ok = col0 < p.K;
    const bool leader = wg == 0 && lane == 0;
    volatile int* abort_flag = &s_abort;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t slots_off = (p.g_bytes + 1023u) & ~1023u;

    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < ngroups * p.depth; ++s) mbar_init(smem_u32(&s_full[s]), 1);
        fence_mbarrier_init();
        fence_proxy_async_smem();
    }
    if (p.mult != nullptr) {   // stage the multiplier, swizzled like the rows
        for (int i = tid * 4; i < p.K; i += kThreads * 4) {
            const float4 g4 = __ldg(reinterpret_cast<const float4*>(p.mult + i));
            *reinterpret_cast<float4*>(gen + swz128((uint32_t)i * 4u)) = g4;
        }
    }
    __syncthreads();

    const int first = (int)blockIdx.x * ngroups + group;     // rows < 2^31 (checked by the launcher)
    const int step = (int)gridDim.x * ngroups;
    const int rows = (int)p.rows;
    const uint32_t tx = (uint32_t)p.K * (uint32_t)sizeof(XT);
    const uint32_t slot0 = base + slots_off + (uint32_t)(group * p.depth) * p.slot_bytes;
    uint64_t* full0 = &s_full[group * p.depth];

    int issued = 0;          // rows requested by this group's leader
    if (leader) {
        for (int d = 0; d < p.depth; ++d) {
            const int r = first + d * step;
            if (r < rows) {
                mbar_arrive_expect_tx(smem_u32(&full0[d]), tx);
                tma_load_3d(slot0 + d * p.slot_bytes, &map_x, 0, 0, (int)r, smem_u32(&full0[d]));
                ++issued;
            }
        }
    }

    // A thread's 16-byte pieces lie in one 128-byte line, so their swizzled offsets are
    // swz(first) ^ (i << 4): one register per operand instead of one per piece.
    constexpr int kPieces = E * (int)sizeof(XT) / 16;      // 4 (bf16) or 8 (fp32)
    const uint32_t xoff0 = swz128((uint32_t)col0 * (uint32_t)sizeof(XT));
    const uint8_t* gptr = gen + swz128((uint32_t)col0 * 4u);

    int n = 0, d = 0;
    uint32_t ph = 0;
    for (int row = first; row < rows; row += step, ++n) {
        bool ok = mbar_wait_warp(smem_u32(&full0[d]), ph, abort_flag, p.watchdog, 0x100u);

        float v[E];
        const uint8_t* slot = gen + slots_off + (size_t)(group * p.depth + d) * p.slot_bytes + xoff0;
        if (col_ok) {
            if (sizeof(XT) == 2) {
#pragma unroll
                for (int i = 0; i < kPieces; ++i) {
                    const uint4 q = *reinterpret_cast<const uint4*>(
                        reinterpret_cast<const uint8_t*>(reinterpret_cast<uintptr_t>(slot) ^ (uintptr_t)(i << 4)));
                    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        v[8 * i + 2 * j + 0] = __uint_as_float(w[j] << 16);
                        v[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < kPieces; ++i) {
                    const float4 q = *reinterpret_cast<const float4*>(
                        reinterpret_cast<const uint8_t*>(reinterpret_cast<uintptr_t>(slot) ^ (uintptr_t)(i << 4)));
                    v[4 * i + 0] = q.x; v[4 * i + 1] = q.y; v[4 * i + 2] = q.z; v[4 * i + 3] = q.w;
                }
            }
            if (p.mult != nullptr) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 g4 = *reinterpret_cast<const float4*>(
                        reinterpret_cast<const uint8_t*>(reinterpret_cast<uintptr_t>(gptr) ^ (uintptr_t)(i << 4)));
                    v[4 * i + 0] = __fmul_rn(v[4 * i + 0], g4.x);
                    v[4 * i + 1] = __fmul_rn(v[4 * i + 1], g4.y);
                    v[4 * i + 2] = __fmul_rn(v[4 * i + 2], g4.z);
                    v[4 * i + 3] = __fmul_rn(v[4 * i + 3], g4.w);
                }
            } else {
#pragma unroll
                for (int i = 0; i < E; ++i) v[i] = __fmul_rn(v[i], p.cnorm);
            }
        } else {
#pragma unroll
            for (int i = 0; i < E; ++i) v[i] = 0.0f;
        }

        // strides 1..16 in registers, 32..block/2 across lanes (same network as the register-only kernel)
#pragma unroll
        for (int h = 1; h < E; h <<= 1) {
            if (h < p.block) {
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
        for (int h = E; h < p.block; h <<= 1) {
            const int lm = h / E;
            const float sgn = (lane & lm) ? -1.0f : 1.0f;
#pragma unroll
            for (int i = 0; i < E; ++i) {
                const float q = __shfl_xor_sync(0xffffffffu, v[i], lm);
                v[i] = __fmaf_rn(v[i], sgn, q);
            }
        }

        float m = 0.0f;
#pragma unroll
        for (int i = 0; i < E; ++i) m = fmaxf(m, fabsf(v[i]));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (p.gw > 1) {
            if (lane == 0) s_part[n & 1][warp] = m;
            ok = group_barrier_and(1 + group, p.gw * 32, ok);
            m = (lane < p.gw) ? s_part[n & 1][group * p.gw + lane] : 0.0f;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        } else {
            ok = __all_sync(0xffffffffu, ok);
        }
        if (!ok) break;

        // every warp of the group has read the slot: refill it with the row `depth` steps ahead
        if (leader) {
            const int nr = row + p.depth * step;
            if (nr < rows) {
                fence_proxy_async_smem();
                mbar_arrive_expect_tx(smem_u32(&full0[d]), tx);
                tma_load_3d(slot0 + d * p.slot_bytes, &map_x, 0, 0, (int)nr, smem_u32(&full0[d]));
                ++issued;
            }
        }

        float dl = __fdiv_rn(__fmul_rn(p.clip_ratio, m), p.qmax);
        float inv;
        if (dl >= FLT_MIN) {
            inv = __fdiv_rn(1.0f, dl);
        } else {
            dl = 0.0f;
            inv = 0.0f;
        }
        constexpr int kPer = FMT == 0 ? 8 : 4;               // codes per 32-bit word
        uint32_t w[E / kPer];
#pragma unroll
        for (int j = 0; j < E / kPer; ++j) {
            uint32_t b[kPer];
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                float t = __fmul_rn(v[j * kPer + i], inv);
                if (CLAMP) t = fminf(fmaxf(t, -p.qmax), p.qmax);
                b[i] = __float_as_uint(__fadd_rn(t, 12582912.0f));
            }
            w[j] = pack_word<FMT>(b);
        }
        if (col_ok) {
            if (FMT == 0) {
                uint4* dst = reinterpret_cast<uint4*>(p.codes + (int64_t)row * (p.K / 2) + col0 / 2);
                dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
            } else {
                uint4* dst = reinterpret_cast<uint4*>(p.codes + (int64_t)row * p.K + col0);
                dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                dst[1] = make_uint4(w[FMT == 0 ? 0 : 4], w[FMT == 0 ? 1 : 5], w[FMT == 0 ? 2 : 6], w[FMT == 0 ? 3 : 7]);
            }
            if (wg == 0 && lane == 0) p.delta[row] = dl;
        }
        if (++d == p.depth) { d = 0; ph ^= 1u; }
    }

    // Winding down after an expired wait: let the copies this group still has in flight land.
    if (leader && *abort_flag) {
        for (int k = n; k < issued; ++k) {
            const int dk = k % p.depth;
            const uint32_t phk = (uint32_t)((k / p.depth) & 1);
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&full0[dk]), phk)) {
                if (global_timer_ns() - t0 > kWaitLimitNs) { atomicOr(p.watchdog, 0x200u); break; }
            }
        }
    }
}

template <typename XT, int FMT>
cudaError_t launch_ring(const CUtensorMap& map, const RingParams& p, int grid, size_t smem, cudaStream_t stream) {
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<grid, kThreads, smem, stream>>>(map, p);
        return cudaGetLastError();
    };
    if (p.clip_ratio < 1.0f) return go(transform_quantize_ring_kernel<XT, FMT, true>);
    return go(transform_quantize_ring_kernel<XT, FMT, false>);
}

}  // namespace

cudaError_t launch_transform_quantize_ring(const void* x, fq_dtype xt, int64_t rows, int64_t K, int64_t ldx,
                                           const float* mult, float cnorm, int block, int qmax, float clip_ratio,
                                           StoreFmt fmt, void* codes, float* delta, cudaStream_t stream) {
    const size_t esz = xt == FQ_BF16 ? 2 : 4;
    const size_t row_bytes = (size_t)K * esz;
    // shape gate: whole 128-byte lines, at most 256 of them per box, a full warp of 32-channel threads
    if (K < 1024 || row_bytes % 128 != 0 || row_bytes / 128 > 256 || rows > 0x7fffffffll) return cudaErrorNotSupported;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (rows < 2 * (int64_t)sms) return cudaErrorNotSupported;     // short batches: latency-bound, register kernel

    int gw = 1;
    while ((int64_t)gw * 32 * E < K) gw <<= 1;
    if (gw > 32) return cudaErrorNotSupported;
    if (gw > kThreads / 32) return cudaErrorNotSupported;
    int ngroups = (kThreads / 32) / gw;
    const size_t slot = (row_bytes + 1023) / 1024 * 1024;
    const size_t g_bytes = mult ? ((size_t)K * 4 + 1023) / 1024 * 1024 : 0;
    const size_t budget = 227 * 1024 - 2048 - 1024;
    if (g_bytes + 2 * slot > budget) return cudaErrorNotSupported;
    int depth = (int)((budget - g_bytes) / (slot * ngroups));
    if (depth > 4) depth = 4;
    if (depth < 2) return cudaErrorNotSupported;
    if (ngroups * depth > kMaxSlots) return cudaErrorNotSupported;

    CUtensorMap map;
    const uint64_t dims[3] = {128 / esz, row_bytes / 128, (uint64_t)rows};
    const uint64_t strides[2] = {128, (uint64_t)ldx * esz};
    const uint32_t box[3] = {(uint32_t)(128 / esz), (uint32_t)(row_bytes / 128), 1};
    if (!encode_tiled(&map, xt == FQ_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, x,
                      dims, strides, box, true))
        return cudaErrorNotSupported;

    RingParams p{};
    p.rows = rows; p.K = (int)K; p.block = block; p.cnorm = cnorm; p.qmax = (float)qmax; p.clip_ratio = clip_ratio;
    p.mult = mult; p.codes = static_cast<uint8_t*>(codes); p.delta = delta; p.gw = gw; p.depth = depth;
    p.slot_bytes = (uint32_t)slot; p.g_bytes = (uint32_t)g_bytes;
    p.watchdog = watchdog_device_ptr();
    if (!p.watchdog) return cudaErrorUnknown;
    const size_t smem = g_bytes + slot * ngroups * depth + 1024;
    int64_t need = (rows + ngroups - 1) / ngroups;
    const int grid = (int)(need < sms ? need : sms);
    if (xt == FQ_BF16)
        return fmt == StoreFmt::Nibble ? launch_ring<__nv_bfloat16, 0>(map, p, grid, smem, stream)
                                       : launch_ring<__nv_bfloat16, 1>(map, p, grid, smem, stream);
    return fmt == StoreFmt::Nibble ? launch_ring<float, 0>(map, p, grid, smem, stream)
                                   : launch_ring<float, 1>(map, p, grid, smem, stream);
}

}  // namespace fq
