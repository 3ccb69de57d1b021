// Streaming variant of the runtime prologue (Alg. 1 runtime half lines 1-2, Eq. 5) for long
// batches: same arithmetic, bit for bit, as transform_quantize_kernel, but tokens reach the
// SM through a TMA-fed shared-memory ring so that many rows are in flight per SM regardless
// of register pressure, and the floating-point work is issued as packed f32x2 instructions.
//
//   - One persistent CTA of 512 threads per SM, split into row groups of `gw` warps; a
//     group owns one token at a time, a thread owns E = 64 (or 32) consecutive channels.
//   - A token row is fetched as a 3-D tiled TMA box {128 bytes, K*e/128, 1} with the 128-byte
//     swizzle, which makes the per-thread 64..256-byte reads bank-conflict free.  The per-
//     channel multiplier is staged once in shared memory with the same swizzle.
//   - Each group runs `depth` slots: the group barrier that exchanges the per-warp maxima also
//     proves that every warp has finished reading the slot, so the group's leader refills it
//     right there -- no separate "empty" barrier.
//   - Register layout: float2 v[p] = (channel p, channel p + E/2).  Butterflies with stride
//     below E/2 then act on both halves at once (fadd2 / ffma2 by -1: each lane of a packed
//     instruction is one IEEE binary32 operation, so the rounding is that of the scalar
//     network); the stride-E/2 stage works inside the pairs; strides E..block/2 go across
//     lanes (one shuffle per value, one packed FMA per pair).
#include <cuda_bf16.h>
#include <float.h>

#include "fq_common.cuh"
#include "ptx_sm100.cuh"
#include "act_common.cuh"

namespace fq {
namespace {

constexpr int kThreads = 512;
// Threads of a CTA by channels per thread.  (1024 threads of 32 channels -- twice the warps at 64 registers -- measured
// slower than 512 threads of 64 channels for 4-bit output: 0.65 against 0.75 of the copy rate at K = 8192, block 128;
// the extra cross-lane butterfly stage costs more than the occupancy returns.)
constexpr int threads_for(int) { return kThreads; }
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
// max(m, |x|, |y|) in one instruction (3-input max of sm_100).
__device__ __forceinline__ float max3_abs(float m, float x, float y) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(m), "f"(fabsf(x)), "f"(fabsf(y)));
    return r;
}
// A thread's slice is 64, 128 or 256 contiguous bytes of a swizzled, 1024-byte aligned region.
// Inside one 128-byte line the swizzled address of 16-byte piece i is (address of piece 0) ^ (i << 4),
// so one address per line (line0, line1 = swizzled starts of the slice's lines) is all a thread keeps.
// Addresses are 32-bit shared-window addresses and the loads explicit ld.shared: through generic
// pointers the same reads cost 64-bit address arithmetic (about one extra instruction per element).
__device__ __forceinline__ uint32_t piece(uint32_t line0, uint32_t line1, int i) {
    return (i < 8 ? line0 : line1) ^ (uint32_t)((i & 7) << 4);
}
// (Not volatile, so that the compiler may batch and hoist them; the caller pins their addresses
// behind the barrier wait that makes the data valid, see `pin_after_wait`.)
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
// An empty volatile statement that "rewrites" an address: loads through that address cannot be
// moved above it, and it cannot be moved above the (volatile) barrier wait before it.
__device__ __forceinline__ void pin_after_wait(uint32_t& addr) { asm volatile("" : "+r"(addr) : : "memory"); }
// Volatile variant for the multiplier: kept in program order, interleaved with the multiplies that
// consume it (hoisting all of them too would not fit the register file).
__device__ __forceinline__ float4 lds128f_ordered(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ float4 lds128f(uint32_t addr) {
    float4 v;
    asm("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

struct RingParams {
    int64_t rows;
    int K;
    float cnorm, qmax, clip_ratio;
    const float* mult;
    int mult_after;    // 1: multiply by cnorm before the butterflies and by mult after them (fold-after sites)
    uint8_t* codes;
    float* delta;
    int gw;            // warps per row group (power of two)
    int depth;         // ring slots per group
    uint32_t slot_bytes;
    uint32_t g_bytes;  // bytes of the multiplier stage (0 if no multiplier)
    uint32_t* watchdog;
};

template <typename XT, int FMT, bool CLAMP, int E, int BLOCK, bool AFTER, int THREADS = kThreads>
__global__ void __launch_bounds__(THREADS, 1)
transform_quantize_ring_kernel(const __grid_constant__ CUtensorMap map_x, const RingParams p) {
    constexpr int H = E / 2;                       // channels per half: v[i] = (channel i, channel i + H)
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[kMaxSlots];
    __shared__ float s_part[2][32];
    __shared__ int s_abort;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ngroups = (THREADS / 32) / p.gw;
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
    __syncthreads();                 // barriers initialised before any copy is issued
    griddep_wait();                  // the kernel before this one may still be writing x (or reading codes)
    griddep_launch_dependents();

    const int first = group * (int)gridDim.x + (int)blockIdx.x;   // rows < 2^31 (checked by the launcher)
    const int step = (int)gridDim.x * ngroups;
    const int rows = (int)p.rows;
    const uint32_t tx = (uint32_t)p.K * (uint32_t)sizeof(XT);
    const uint32_t slot0 = base + slots_off + (uint32_t)(group * p.depth) * p.slot_bytes;
    uint64_t* full0 = &s_full[group * p.depth];

    // The first rows are requested before the multiplier is staged, so that their flight time
    // overlaps the staging loop.
    int issued = 0;          // rows requested by this group's leader
    if (leader) {
        for (int d = 0; d < p.depth; ++d) {
            const int r = first + d * step;
            if (r < rows) {
                mbar_arrive_expect_tx(smem_u32(&full0[d]), tx);
                tma_load_3d(slot0 + d * p.slot_bytes, &map_x, 0, 0, r, smem_u32(&full0[d]));
                ++issued;
            }
        }
    }
    if (p.mult != nullptr) {
        // Stage the multiplier in the order the registers hold a slice: inside every thread slice (E floats)
        // the entries are interleaved as (g[q], g[q + H]) pairs, so that one 16-byte read yields two ready
        // operands of the packed multiply (no register moves to pair them up), and the 16-byte pieces are
        // XOR-swizzled by the slice index, so that the slice-per-thread reads are bank-conflict free.
        for (int i = tid * 4; i < p.K; i += THREADS * 4) {
            const float4 g4 = __ldg(reinterpret_cast<const float4*>(p.mult + i));
            const float gv[4] = {g4.x, g4.y, g4.z, g4.w};
            const uint32_t slice = (uint32_t)i / E;
            const uint32_t key = (slice & 7u) << 4;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t q = ((uint32_t)i % E) + k;                       // position inside the slice
                const uint32_t off = q < H ? q * 8u : (q - H) * 8u + 4u;         // pair q (low half) or q - H (high half)
                *reinterpret_cast<float*>(gen + ((slice * (E * 4u) + off) ^ key)) = gv[k];
            }
        }
    }
    __syncthreads();

    // swizzled starts of the (up to two) 128-byte lines of this thread's slices
    const uint32_t xs0 = swz128((uint32_t)col0 * (uint32_t)sizeof(XT));
    const uint32_t xs1 = swz128((uint32_t)col0 * (uint32_t)sizeof(XT) + 128u);
    const uint32_t gkey = (uint32_t)((col0 / E) & 7) << 4;
    const uint32_t g0 = base + (((uint32_t)col0 * 4u) ^ gkey);
    const uint32_t g1 = base + (((uint32_t)col0 * 4u + 128u) ^ gkey);
    const bool warp_ok = __all_sync(0xffffffffu, col_ok);   // the usual case: no lane of the warp is past K
    const float2 neg1 = make_float2(-1.0f, -1.0f);

    int n = 0, d = 0;
    uint32_t ph = 0;
    for (int row = first; row < rows; row += step, ++n) {
        bool ok = mbar_wait_all(smem_u32(&full0[d]), ph, abort_flag, p.watchdog, 0x100u);   // every lane polls: cheaper than one lane + broadcast

        float2 v[H];
        const uint32_t slot = base + slots_off + (uint32_t)(group * p.depth + d) * p.slot_bytes;
        uint32_t x0 = slot + xs0, x1 = slot + xs1;
        pin_after_wait(x0);
        pin_after_wait(x1);
        auto load_row = [&]() {
            if (sizeof(XT) == 2) {
                // bf16: 8 channels per 16-byte piece; pieces [0, H/8) are the low half, the rest the high half
#pragma unroll
                for (int i = 0; i < H / 8; ++i) {
                    const uint4 lo = lds128(piece(x0, x1, i));
                    const uint4 hi = lds128(piece(x0, x1, i + H / 8));
                    const uint32_t wl[4] = {lo.x, lo.y, lo.z, lo.w}, wh[4] = {hi.x, hi.y, hi.z, hi.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        v[8 * i + 2 * j + 0] = make_float2(__uint_as_float(wl[j] << 16), __uint_as_float(wh[j] << 16));
                        v[8 * i + 2 * j + 1] = make_float2(__uint_as_float(wl[j] & 0xffff0000u),
                                                           __uint_as_float(wh[j] & 0xffff0000u));
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < H / 4; ++i) {
                    const float4 lo = lds128f(piece(x0, x1, i));
                    const float4 hi = lds128f(piece(x0, x1, i + H / 4));
                    v[4 * i + 0] = make_float2(lo.x, hi.x);
                    v[4 * i + 1] = make_float2(lo.y, hi.y);
                    v[4 * i + 2] = make_float2(lo.z, hi.z);
                    v[4 * i + 3] = make_float2(lo.w, hi.w);
                }
            }
            if (!AFTER && p.mult != nullptr) {
#pragma unroll
                for (int i = 0; i < H / 2; ++i) {           // one piece = the multipliers of pairs 2i and 2i + 1
                    const float4 q = lds128f_ordered(piece(g0, g1, i));
                    v[2 * i + 0] = f2_mul(v[2 * i + 0], make_float2(q.x, q.y));
                    v[2 * i + 1] = f2_mul(v[2 * i + 1], make_float2(q.z, q.w));
                }
            } else {
                const float2 c2 = make_float2(p.cnorm, p.cnorm);
#pragma unroll
                for (int i = 0; i < H; ++i) v[i] = f2_mul(v[i], c2);
            }
        };
        // Warp-uniform fast path: with a per-lane `col_ok` the zero fill below is compiled into
        // predicated instructions that every row pays for (half an instruction per element).
        if (warp_ok) {
            load_row();
        } else if (col_ok) {
            load_row();
        } else {
#pragma unroll
            for (int i = 0; i < H; ++i) v[i] = make_float2(0.0f, 0.0f);
        }

        // strides 1 .. H/2: both halves at once
#pragma unroll
        for (int h = 1; h < H; h <<= 1) {
            if (h < BLOCK) {
#pragma unroll
                for (int i = 0; i < H; ++i) {
                    if ((i & h) == 0) {
                        const float2 a = v[i], b = v[i + h];
                        v[i] = f2_add(a, b);
                        v[i + h] = f2_fma(b, neg1, a);       // a - b, exact product
                    }
                }
            }
        }
        // stride H: inside each pair
        if (H < BLOCK) {
#pragma unroll
            for (int i = 0; i < H; ++i) {
                const float a = v[i].x, b = v[i].y;
                v[i] = make_float2(__fadd_rn(a, b), __fsub_rn(a, b));
            }
        }
        // strides E .. BLOCK/2: partner lane = lane ^ (h / E); upper lane keeps partner - own
#pragma unroll
        for (int h = E; h < BLOCK; h <<= 1) {
            const int lm = h / E;
            const float s = (lane & lm) ? -1.0f : 1.0f;
            const float2 s2 = make_float2(s, s);
#pragma unroll
            for (int i = 0; i < H; ++i) {
                const float2 q = make_float2(__shfl_xor_sync(0xffffffffu, v[i].x, lm),
                                             __shfl_xor_sync(0xffffffffu, v[i].y, lm));
                v[i] = f2_fma(v[i], s2, q);
            }
        }

        // fold-after sites: the diagonal sits behind the rotation (z = D^o R x)
        if (AFTER && col_ok) {
#pragma unroll
            for (int i = 0; i < H / 2; ++i) {
                const float4 q = lds128f_ordered(piece(g0, g1, i));
                v[2 * i + 0] = f2_mul(v[2 * i + 0], make_float2(q.x, q.y));
                v[2 * i + 1] = f2_mul(v[2 * i + 1], make_float2(q.z, q.w));
            }
        }

        float m = 0.0f;
#pragma unroll
        for (int i = 0; i < H; ++i) m = max3_abs(m, v[i].x, v[i].y);
        m = warp_max_nonneg(m);
        if (p.gw > 1) {
            if (lane == 0) s_part[n & 1][warp] = m;
            ok = group_barrier_and(1 + group, p.gw * 32, ok);
            m = (lane < p.gw) ? s_part[n & 1][group * p.gw + lane] : 0.0f;
            m = warp_max_nonneg(m);
        }
        if (!ok) break;

        // every warp of the group has read the slot: refill it with the row `depth` steps ahead
        if (leader) {
            const int nr = row + p.depth * step;
            if (nr < rows) {
                fence_proxy_async_smem();
                mbar_arrive_expect_tx(smem_u32(&full0[d]), tx);
                tma_load_3d(slot0 + d * p.slot_bytes, &map_x, 0, 0, nr, smem_u32(&full0[d]));
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
        // codes: channel i from .x, channel i + H from .y
        constexpr int kPer = FMT == 0 ? 8 : 4;               // codes per 32-bit word
        constexpr int kWords = H / kPer;                     // words per half
        const float2 inv2 = make_float2(inv, inv);
        uint32_t wlo[kWords], whi[kWords];
#pragma unroll
        for (int j = 0; j < kWords; ++j) {
            uint32_t bl[kPer], bh[kPer];
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                float2 t = f2_mul(v[code_index<FMT>(j, i)], inv2);
                if (CLAMP) {
                    t.x = fminf(fmaxf(t.x, -p.qmax), p.qmax);
                    t.y = fminf(fmaxf(t.y, -p.qmax), p.qmax);
                }
                // t * 1 + magic as an explicit packed FMA (exact product, so it rounds like the add).  A
                // packed multiply feeding a packed ADD was observed to be fused into one packed FMA by the
                // assembler, which rounds exact ties differently.
                t = f2_fma(t, make_float2(1.0f, 1.0f), make_float2(12582912.0f, 12582912.0f));
                bl[i] = __float_as_uint(t.x);
                bh[i] = __float_as_uint(t.y);
            }
            wlo[j] = pack_word<FMT>(bl);
            whi[j] = pack_word<FMT>(bh);
        }
        if (col_ok) {
            // low-half words then high-half words are consecutive channels: one contiguous store run
            uint32_t w[2 * kWords];
#pragma unroll
            for (int j = 0; j < kWords; ++j) { w[j] = wlo[j]; w[kWords + j] = whi[j]; }
            const int64_t pitch = FMT == 0 ? p.K / 2 : p.K;
            uint4* dst = reinterpret_cast<uint4*>(p.codes + (int64_t)row * pitch + (FMT == 0 ? col0 / 2 : col0));
#pragma unroll
            for (int j = 0; j < 2 * kWords / 4; ++j) dst[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
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

template <typename XT, int FMT, int E, int BLOCK>
cudaError_t launch_ring(const CUtensorMap& map, const RingParams& p, int grid, size_t smem, cudaStream_t stream) {
    constexpr int THREADS = threads_for(E);
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem);
        if (e != cudaSuccess) return e;
        return launch_pdl(kern, (unsigned)grid, (unsigned)THREADS, smem, stream, 1u, map, p);
    };
    // (the fold-after variant is its own instantiation: as a run-time branch it cost the default
    // path registers, and spills, in the 64-channels-per-thread kernels)
    if (p.mult_after) {
        if (p.clip_ratio < 1.0f) return go(transform_quantize_ring_kernel<XT, FMT, true, E, BLOCK, true, THREADS>);
        return go(transform_quantize_ring_kernel<XT, FMT, false, E, BLOCK, true, THREADS>);
    }
    if (p.clip_ratio < 1.0f) return go(transform_quantize_ring_kernel<XT, FMT, true, E, BLOCK, false, THREADS>);
    return go(transform_quantize_ring_kernel<XT, FMT, false, E, BLOCK, false, THREADS>);
}

template <typename XT, int FMT, int E>
cudaError_t launch_ring_block(int block, const CUtensorMap& map, const RingParams& p, int grid, size_t smem,
                              cudaStream_t stream) {
    switch (block) {
        case 32: return launch_ring<XT, FMT, E, 32>(map, p, grid, smem, stream);
        case 64: return launch_ring<XT, FMT, E, 64>(map, p, grid, smem, stream);
        case 128: return launch_ring<XT, FMT, E, 128>(map, p, grid, smem, stream);
        case 256: return launch_ring<XT, FMT, E, 256>(map, p, grid, smem, stream);
        default: return cudaErrorNotSupported;
    }
}

template <typename XT, int FMT>
cudaError_t launch_ring_e(int e, int block, const CUtensorMap& map, const RingParams& p, int grid, size_t smem,
                          cudaStream_t stream) {
    return e == 64 ? launch_ring_block<XT, FMT, 64>(block, map, p, grid, smem, stream)
                   : launch_ring_block<XT, FMT, 32>(block, map, p, grid, smem, stream);
}

}  // namespace

cudaError_t launch_transform_quantize_ring(const void* x, fq_dtype xt, int64_t rows, int64_t K, int64_t ldx,
                                           const float* mult, float cnorm, bool mult_after_rotation, int block,
                                           int qmax, float clip_ratio, StoreFmt fmt, void* codes, float* delta,
                                           cudaStream_t stream) {
    const size_t esz = xt == FQ_BF16 ? 2 : 4;
    const size_t row_bytes = (size_t)K * esz;
    // shape gate: whole 128-byte lines, at most 256 of them per box, blocks of 32..256 channels
    if (K < 1024 || row_bytes % 128 != 0 || row_bytes / 128 > 256 || rows > 0x7fffffffll || block < 32)
        return cudaErrorNotSupported;
    const int sms = device_sm_count();
    // Short batches are latency-bound and go to the register kernel, which spreads a row over more threads: fewer
    // than 8 rows per SM, unless the rows are long (measured at M = 816: K = 2048 6.4 us there against 7.1-7.9 us
    // here, K = 16384 24.3 us there against 21.2 us here).
    if (rows < 2 * (int64_t)sms || (rows < 8 * (int64_t)sms && K < 8192)) return cudaErrorNotSupported;

    // channels per thread (the fold-after variant with shuffle stages does not fit 64 without spills)
    const int e = (K >= 2048 && K % 64 == 0 && !(mult != nullptr && mult_after_rotation && block >= 128)) ? 64 : 32;
    const int threads = threads_for(e);
    int gw = 1;
    while ((int64_t)gw * 32 * e < K) gw <<= 1;
    if (gw > threads / 32) return cudaErrorNotSupported;
    const int ngroups = (threads / 32) / gw;
    if (gw > 1 && ngroups > 15) return cudaErrorNotSupported;      // one named barrier per group
    const size_t slot = (row_bytes + 1023) / 1024 * 1024;
    const size_t g_bytes = mult ? ((size_t)K * 4 + 1023) / 1024 * 1024 : 0;
    const size_t budget = 227 * 1024 - 2048 - 1024;
    if (g_bytes + 2 * slot * ngroups > budget) return cudaErrorNotSupported;
    int depth = (int)((budget - g_bytes) / (slot * ngroups));
    if (depth > 4) depth = 4;
    if (depth < 2 || ngroups * depth > kMaxSlots) return cudaErrorNotSupported;

    CUtensorMap map;
    const uint64_t dims[3] = {128 / esz, row_bytes / 128, (uint64_t)rows};
    const uint64_t strides[2] = {128, (uint64_t)ldx * esz};
    const uint32_t box[3] = {(uint32_t)(128 / esz), (uint32_t)(row_bytes / 128), 1};
    if (!encode_tiled(&map, xt == FQ_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, x,
                      dims, strides, box, true))
        return cudaErrorNotSupported;

    RingParams p{};
    p.rows = rows; p.K = (int)K; p.cnorm = cnorm; p.qmax = (float)qmax; p.clip_ratio = clip_ratio;
    p.mult = mult; p.mult_after = (mult != nullptr && mult_after_rotation) ? 1 : 0; p.codes = static_cast<uint8_t*>(codes); p.delta = delta; p.gw = gw; p.depth = depth;
    p.slot_bytes = (uint32_t)slot; p.g_bytes = (uint32_t)g_bytes;
    p.watchdog = watchdog_device_ptr();
    if (!p.watchdog) return cudaErrorUnknown;
    const size_t smem = g_bytes + slot * ngroups * depth + 1024;
    // Rows are dealt to the CTAs first and to a CTA's row groups second (row r -> CTA r % grid),
    // so that a short batch spreads over all SMs instead of filling every group of a few CTAs.
    const int grid = (int)(rows < sms ? rows : sms);
    if (xt == FQ_BF16)
    {
        if (fmt == StoreFmt::Nibble) return launch_ring_e<__nv_bfloat16, 0>(e, block, map, p, grid, smem, stream);
        if (fmt == StoreFmt::Int8) return launch_ring_e<__nv_bfloat16, 1>(e, block, map, p, grid, smem, stream);
        return launch_ring_e<__nv_bfloat16, 2>(e, block, map, p, grid, smem, stream);
    }
    if (fmt == StoreFmt::Nibble) return launch_ring_e<float, 0>(e, block, map, p, grid, smem, stream);
    if (fmt == StoreFmt::Int8) return launch_ring_e<float, 1>(e, block, map, p, grid, smem, stream);
    return launch_ring_e<float, 2>(e, block, map, p, grid, smem, stream);
}

}  // namespace fq
