// Short-batch weight streaming for 4-bit weights: the projection of a handful of tokens is a
// matrix-vector product bound by the weight bytes, which must cross HBM once.  Two users:
//   * the W4A4 and W8A8 integer products of Eq. 8 for batches of at most 16 tokens where it measured faster than
//     the TMA/TMEM pipeline of the big GEMM (see gemm_stream_applies), whose per-k-block hand-overs cannot be fed
//     at HBM rate by so thin a tile (8-bit weights: a line is 128 channels, the bytes enter the MMAs as they are);
//   * the weight-only projection with floating-point activations (the adaptive layer-normalisation
//     modulation of the W4A4 engines):  y[t][j] = s^W_j * sum_c qW[j][c] * x[t][c] + b_j.
// One persistent CTA per SM walks groups of 32 weight rows.  A producer warp streams the packed rows
// through a ring of 32 KB stages (32 rows x 2048 channels, ONE 128-byte-swizzled TMA box each: an
// issuing warp gets out one tensor copy per ~260 cycles whatever its size, so a stage must not be
// several) that holds ~190 KB in flight per SM.  Each of the 16 consumer warps takes, of every stage, one
// 256-channel line of all 32 rows and in it every other 32-channel unit: both 16-row MMA tiles share one B
// fragment, so a token's activations are fetched and permuted once per 32 rows.  The codes are expanded in
// registers and multiplied with warp-level MMAs (m16n8k32 s8 -> s32, or m16n8k16 bf16 -> f32); tokens ride
// along 8 per MMA at no extra weight traffic.  The warps' partial sums meet in shared memory, are added in a
// fixed order, rescaled and stored.  binary32 activations are split into three bf16 terms (exactly), so both
// float input types see exact products and binary32 sums.
//
// Operand layout.  Lane (g = lane / 4, t = lane % 4) reads 16 bytes = 32 codes of rows g, g + 8, g + 16 and
// g + 24 at unit 2t + h of the warp's line, and the activations of token g at the same channels.  A sum over
// channels may run in any order as long as both operands agree on it, so the k index of the MMA is
// mapped to channels the way the codes unpack cheapest:
//   int8:  (w << 4) & 0xF0F0F0F0 holds 16 x the codes of channels 0,2,4,6 of a word and w & 0xF0F0F0F0
//          those of channels 1,3,5,7 -- the order in which the prologue stores its int8 codes;
//   bf16:  one mask of the word shifted by 4 j isolates the codes of channels j and j + 4 in the two
//          halves of a register, and the B fragment pairs the activations of those channels.
// What bounds the float path is the integer pipe (shift + mask per pair of codes, half the rate of the
// other pipes): the codes enter the MMAs 136 too large (see codes_plus136_bf16x2) because taking the offset
// off each pair cost another instruction, and the activations' loads are issued a stage ahead of the byte
// permutes that consume them.
#include <cuda_bf16.h>
#include <stdlib.h>

#include "fq_common.cuh"
#include "ptx_sm100.cuh"

namespace fq {
namespace {

constexpr int kConsumers = 16;                  // consumer warps: (row tile, 128-channel slot of a stage)
constexpr int kThreads = 32 * (kConsumers + 1); // + one producer warp
constexpr int kRowsCta = 32;                    // two 16-row MMA tiles
constexpr int kLines = 8;                       // 128-byte lines per row and stage
constexpr int kStageBytes = kRowsCta * kLines * 128;   // one TMA box: 32 rows x 8 lines of 128 bytes (32 KB)
constexpr int kMaxDepth = 6;
// kModeInt: 4-bit weights x int8 activations; kModeBf16 / kModeF32: 4-bit weights x float activations;
// kModeInt8: 8-bit weights x int8 activations (a line is 128 channels then, a 16-byte unit 16 channels, and the
// bytes go into the MMAs as they are)
enum : int { kModeInt = 0, kModeBf16 = 1, kModeF32 = 2, kModeInt8 = 3 };
template <int MODE>
struct Geometry {
    static constexpr bool kIntegers = MODE == kModeInt || MODE == kModeInt8;
    static constexpr int kLineCh = MODE == kModeInt8 ? 128 : 256;     // channels of a 128-byte line
    static constexpr int kUnitCh = kLineCh / 8;                       // channels of a 16-byte unit
    static constexpr int kStageCh = kLines * kLineCh;                 // channels per stage
};

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void mma_bf16(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_s8(int* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

// Codes of channels j and j + 4 of a packed word (eight two's-complement nibbles, channel i at bits
// 4 i) as two bf16, each 136 too large: (n & 15) ^ 8 = n + 8 goes into the mantissa of 128 (0x4300).
// The exact value 136 + n is what the product MMA multiplies; a second MMA of the constant -136 against the same
// activations takes the offset off again at once, sixteen channels at a time, so the accumulator never carries more
// than one MMA's worth of it.  (Taking 136 off every pair with a packed subtract cost a third of the kernel's
// integer instructions -- the pipe that bounds it; the tensor pipe has room for twice the MMAs.)
__device__ __forceinline__ uint32_t codes_plus136_bf16x2(uint32_t w, int j) {
    return ((w >> (4 * j)) & 0x000F000Fu) ^ 0x43084308u;
}

// The activations of one token at a lane's 32 channels: fetch() issues the loads into raw registers, permute() --
// called a stage later, when they have long arrived -- forms the B-fragment registers.  (With the byte permutes right
// behind the loads a warp sat out the loads' latency in every stage.)
template <int MODE>
struct XFrag;
// int8 codes as the prologue stores them: 8 channels = (c0,c2,c4,c6) (c1,c3,c5,c7); word w -> b[2w], b[2w+1]
template <>
struct XFrag<kModeInt> {
    typedef int8_t elem;
    static constexpr int kTerms = 1;
    uint4 raw[2];
    uint32_t b[1][8];
    __device__ __forceinline__ void fetch(const int8_t* p, bool ok) {
#pragma unroll
        for (int h = 0; h < 2; ++h) raw[h] = ok ? __ldg(reinterpret_cast<const uint4*>(p) + h) : make_uint4(0u, 0u, 0u, 0u);
    }
    __device__ __forceinline__ void permute() {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            b[0][4 * h + 0] = raw[h].x; b[0][4 * h + 1] = raw[h].y; b[0][4 * h + 2] = raw[h].z; b[0][4 * h + 3] = raw[h].w;
        }
    }
};
// int8 codes in channel order against 8-bit weights: the unit's 16 channels, four per register, as they are
template <>
struct XFrag<kModeInt8> {
    typedef int8_t elem;
    static constexpr int kTerms = 1;
    uint4 raw[1];
    uint32_t b[1][4];
    __device__ __forceinline__ void fetch(const int8_t* p, bool ok) {
        raw[0] = ok ? __ldg(reinterpret_cast<const uint4*>(p)) : make_uint4(0u, 0u, 0u, 0u);
    }
    __device__ __forceinline__ void permute() { b[0][0] = raw[0].x; b[0][1] = raw[0].y; b[0][2] = raw[0].z; b[0][3] = raw[0].w; }
};
// bf16: for word w, b[4w + j] = (channel j, channel j + 4), j = 0..3
template <>
struct XFrag<kModeBf16> {
    typedef __nv_bfloat16 elem;
    static constexpr int kTerms = 1;
    uint4 raw[4];
    uint32_t b[1][16];
    __device__ __forceinline__ void fetch(const __nv_bfloat16* p, bool ok) {
#pragma unroll
        for (int w = 0; w < 4; ++w) raw[w] = ok ? __ldg(reinterpret_cast<const uint4*>(p) + w) : make_uint4(0u, 0u, 0u, 0u);
    }
    __device__ __forceinline__ void permute() {
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const uint4 n = raw[w];
            b[0][4 * w + 0] = __byte_perm(n.x, n.z, 0x5410);   // (c0, c4)
            b[0][4 * w + 1] = __byte_perm(n.x, n.z, 0x7632);   // (c1, c5)
            b[0][4 * w + 2] = __byte_perm(n.y, n.w, 0x5410);   // (c2, c6)
            b[0][4 * w + 3] = __byte_perm(n.y, n.w, 0x7632);   // (c3, c7)
        }
    }
};
// binary32, split into three bf16 terms that add up to it exactly (8 + 8 + 8 significant bits, by truncation)
template <>
struct XFrag<kModeF32> {
    typedef float elem;
    static constexpr int kTerms = 3;
    float4 raw[8];
    uint32_t b[3][16];
    __device__ __forceinline__ void fetch(const float* p, bool ok) {
#pragma unroll
        for (int i = 0; i < 8; ++i) raw[i] = ok ? __ldg(reinterpret_cast<const float4*>(p) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    __device__ __forceinline__ void permute() {
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float4 lo4 = raw[2 * w], hi4 = raw[2 * w + 1];
            float r[8] = {lo4.x, lo4.y, lo4.z, lo4.w, hi4.x, hi4.y, hi4.z, hi4.w};
#pragma unroll
            for (int s = 0; s < 3; ++s) {
                uint32_t top[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    top[i] = __float_as_uint(r[i]) & 0xFFFF0000u;            // leading 8 significant bits
                    r[i] = __fsub_rn(r[i], __uint_as_float(top[i]));        // exact remainder
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) b[s][4 * w + j] = __byte_perm(top[j], top[j + 4], 0x7632);
            }
        }
    }
};

struct StreamParams {
    const void* x;            // activations [M, K]: int8 codes (pitch K) or bf16 / binary32 (pitch ldx)
    int64_t ldx;
    int64_t M, N;
    int K;
    int depth;                // ring stages
    int acc_shift;            // int8: the integer sum carries a factor 2^acc_shift
    const float* a_delta;     // int8: per-token steps
    const float* w_scale;
    const float* bias;
    void* y;
    fq_dtype yt;
    int64_t ldy;
    int32_t* acc_out;         // int8: raw sums instead of y (parity/debug)
    uint32_t* watchdog;
    uint32_t zero;            // 0, as a run-time value (see the consumers' release of a stage)
};

enum : uint32_t { kWdStreamFull = 0x400u, kWdStreamEmpty = 0x800u, kWdStreamSync = 0x1000u };

// GROUPS token groups of 8 per pass over the weights.
template <int MODE, int GROUPS>
__global__ void __launch_bounds__(kThreads, 1)
weight_stream_kernel(const __grid_constant__ CUtensorMap map_w, const StreamParams p) {
    extern __shared__ uint8_t smem_raw[];
    typedef typename XFrag<MODE>::elem XT;
    typedef typename std::conditional<Geometry<MODE>::kIntegers, int, float>::type AccT;
    constexpr int kTerms = XFrag<MODE>::kTerms;
    constexpr int kTok = 8 * GROUPS;
    constexpr bool kIntegers = Geometry<MODE>::kIntegers;
    constexpr int kStageCh = Geometry<MODE>::kStageCh, kLineCh = Geometry<MODE>::kLineCh, kUnitCh = Geometry<MODE>::kUnitCh;
    __shared__ uint64_t s_full[kMaxDepth], s_empty[kMaxDepth];
    __shared__ uint64_t s_sync;                       // rendezvous of the consumer warps (bounded, unlike bar.sync)
    __shared__ int s_abort;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    volatile int* abort_flag = &s_abort;
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    AccT* s_part = reinterpret_cast<AccT*>(smem_raw + (ring - smem_u32(smem_raw)) + (size_t)p.depth * kStageBytes);
    // s_part[consumer warp][row 0..31][token, padded to kTok + 1]

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < p.depth; ++s) {
            mbar_init(smem_u32(&s_full[s]), 1);
            mbar_init(smem_u32(&s_empty[s]), kConsumers);
        }
        mbar_init(smem_u32(&s_sync), kConsumers);
        fence_mbarrier_init();
        fence_proxy_async_smem();
    }
    __syncthreads();
    const int row_groups = (int)((p.N + kRowsCta - 1) / kRowsCta);
    const int stages_k = (p.K + kStageCh - 1) / kStageCh;
    const int passes = (int)((p.M + kTok - 1) / kTok);

    if (warp == kConsumers) {
        // ------------------------------------------------------------------ producer
        // The weights are complete before any call that uses them is enqueued: no need to wait for
        // the kernel ahead in the stream.
        griddep_launch_dependents();
        int slot = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int rg = blockIdx.x; rg < row_groups && ok; rg += gridDim.x)
            for (int pass = 0; pass < passes && ok; ++pass)
                for (int s = 0; s < stages_k; ++s) {
                    ok = mbar_wait_all(smem_u32(&s_empty[slot]), ph ^ 1u, abort_flag, p.watchdog, kWdStreamEmpty);
                    if (!ok) break;
                    if (elect_one()) {
                        // the weights as [row][128-byte line][byte]: lines past the row's end and rows past N
                        // are out of bounds and arrive as zeros (the whole box always counts as transferred)
                        const uint32_t bar = smem_u32(&s_full[slot]);
                        mbar_arrive_expect_tx(bar, (uint32_t)kStageBytes);
                        tma_load_3d(ring + slot * kStageBytes, &map_w, 0, s * kLines, rg * kRowsCta, bar);
                    }
                    __syncwarp();
                    if (++slot == p.depth) { slot = 0; ph ^= 1u; }
                }
        if (!ok && lane == 0) {               // let the copies already issued land before the CTA gives its memory back
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 100000ull) __nanosleep(1000);
        }
    } else {
        // ----------------------------------------------------------------- consumers
        griddep_wait();                       // activations come from the kernel ahead in the stream
        griddep_launch_dependents();
        const int g = lane >> 2, t = lane & 3;
        const int h = warp & 1, kq = warp >> 1;            // unit parity, 256-channel line of the stage
        // Stage layout: [row 0..31][line 0..7][128 bytes], line = 256 channels; the 128-byte swizzle XORs the
        // 16-byte unit index with the low three bits of (8 row + line) = line.  This warp reads line kq of all 32
        // rows -- lane (g, t): rows g, g + 8, g + 16, g + 24 -- and of each row the 16-byte unit 2t + h (32 channels):
        // both 16-row MMA tiles of the stage share one B fragment, so the activations are fetched and permuted
        // once per 32 rows.  (All rows of an MMA must use the same channels for a given lane t, so the two rows that
        // share a shared-memory phase read the same unit: a two-way bank conflict that cannot be swizzled away here.)
        const int line = kq;
        const uint32_t unit_off = (uint32_t)(((2 * t + h) ^ line) << 4);
        int slot = 0;
        uint32_t ph = 0, sync_ph = 0;
        bool ok = true;
        const XT* xp = static_cast<const XT*>(p.x);
        for (int rg = blockIdx.x; rg < row_groups && ok; rg += gridDim.x) {
            const int64_t j0 = (int64_t)rg * kRowsCta;
            for (int pass = 0; pass < passes && ok; ++pass) {
                const int64_t t0 = (int64_t)pass * kTok;
                AccT acc[2][GROUPS][4];                      // [row tile][token group][C fragment]
#pragma unroll
                for (int r = 0; r < 2; ++r)
#pragma unroll
                    for (int q = 0; q < GROUPS; ++q)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc[r][q][i] = 0;
                [[maybe_unused]] const uint32_t minus136[4] = {0xC308C308u, 0xC308C308u, 0xC308C308u, 0xC308C308u};   // bf16 -136
                XFrag<MODE> xf[GROUPS];
                // the lane's 32 channels of stage s
                auto load_x = [&](int s) {
                    const int c = s * kStageCh + kq * kLineCh + kUnitCh * (2 * t + h);
#pragma unroll
                    for (int q = 0; q < GROUPS; ++q) {
                        const int64_t tok = t0 + 8 * q + g;
                        xf[q].fetch(xp + tok * p.ldx + c, tok < p.M && c < p.K);
                    }
                };
                load_x(0);
                for (int s = 0; s < stages_k; ++s) {
                    ok = mbar_wait_all(smem_u32(&s_full[slot]), ph, abort_flag, p.watchdog, kWdStreamFull);
                    if (!ok) break;
                    const uint32_t row0 = ring + slot * kStageBytes + (uint32_t)((g * kLines + line) * 128) + unit_off;
                    uint4 wq[4];                             // rows g, g + 8, g + 16, g + 24
#pragma unroll
                    for (int r = 0; r < 4; ++r) wq[r] = lds128(row0 + (uint32_t)(r * 8 * kLines * 128));
                    const int slot_used = slot;              // given back only after the stage's MMAs, see below
                    if (++slot == p.depth) { slot = 0; ph ^= 1u; }
                    const bool exists = s * kStageCh + kq * kLineCh < p.K;     // (warp-uniform) the line is inside the row
                    // this stage's activations arrived a stage ago: form the fragments, then put the next stage's loads in
                    // flight behind this stage's MMAs (after them for binary32 activations, whose three fragments per token
                    // leave no registers for both)
                    constexpr bool kAhead = MODE != kModeF32;
#pragma unroll
                    for (int q = 0; q < GROUPS; ++q) xf[q].permute();
                    if (kAhead && s + 1 < stages_k) load_x(s + 1);
                    XFrag<MODE>* xc = xf;
                    if (exists) {
#pragma unroll
                        for (int r = 0; r < 2; ++r) {
                            const uint32_t w0[4] = {wq[2 * r].x, wq[2 * r].y, wq[2 * r].z, wq[2 * r].w};                   // row 16 r + g
                            const uint32_t w1[4] = {wq[2 * r + 1].x, wq[2 * r + 1].y, wq[2 * r + 1].z, wq[2 * r + 1].w};   // row 16 r + g + 8
                            if constexpr (MODE == kModeInt8) {
#pragma unroll
                                for (int w = 0; w < 2; ++w) {      // two MMAs: the unit's bytes 0-7 and 8-15
                                    const uint32_t a[4] = {w0[2 * w], w1[2 * w], w0[2 * w + 1], w1[2 * w + 1]};
#pragma unroll
                                    for (int q = 0; q < GROUPS; ++q)
                                        mma_s8(reinterpret_cast<int*>(acc[r][q]), a, xc[q].b[0][2 * w], xc[q].b[0][2 * w + 1]);
                                }
                            } else if constexpr (MODE == kModeInt) {
#pragma unroll
                                for (int w = 0; w < 4; ++w) {
                                    const uint32_t a[4] = {(w0[w] << 4) & 0xF0F0F0F0u, (w1[w] << 4) & 0xF0F0F0F0u,
                                                           w0[w] & 0xF0F0F0F0u, w1[w] & 0xF0F0F0F0u};
#pragma unroll
                                    for (int q = 0; q < GROUPS; ++q)
                                        mma_s8(reinterpret_cast<int*>(acc[r][q]), a, xc[q].b[0][2 * w], xc[q].b[0][2 * w + 1]);
                                }
                            } else {
#pragma unroll
                                for (int w = 0; w < 4; ++w)
#pragma unroll
                                    for (int m = 0; m < 2; ++m) {      // channels (2m, 2m+4 | 2m+1, 2m+5) of the word
                                        const uint32_t a[4] = {codes_plus136_bf16x2(w0[w], 2 * m), codes_plus136_bf16x2(w1[w], 2 * m),
                                                               codes_plus136_bf16x2(w0[w], 2 * m + 1), codes_plus136_bf16x2(w1[w], 2 * m + 1)};
#pragma unroll
                                        for (int q = 0; q < GROUPS; ++q)
#pragma unroll
                                            for (int tm = 0; tm < kTerms; ++tm)
                                            {
                                                mma_bf16(reinterpret_cast<float*>(acc[r][q]), a, xc[q].b[tm][4 * w + 2 * m],
                                                         xc[q].b[tm][4 * w + 2 * m + 1]);
                                                mma_bf16(reinterpret_cast<float*>(acc[r][q]), minus136, xc[q].b[tm][4 * w + 2 * m],
                                                         xc[q].b[tm][4 * w + 2 * m + 1]);
                                            }
                                    }
                            }
                        }
                    }
                    if (!kAhead && s + 1 < stages_k) load_x(s + 1);
                    // The stage goes back to the producer only now, behind the MMAs that consumed what was loaded from it:
                    // released right after the loads had been issued (and a __syncwarp), the float path -- the one slow
                    // enough to keep the ring full, so that a freed stage is overwritten at once -- returned wrong sums in
                    // about one launch in a thousand once a row had more stages than the ring (K >= 16384): the loads had
                    // not all been performed when the producer's copy landed.
                    // (and its barrier's address is formed from an accumulator and a run-time zero: a true dependence)
                    uint32_t dep;
                    if constexpr (kIntegers) dep = (uint32_t)(acc[0][0][0] ^ acc[1][0][0]) & p.zero;
                    else dep = (__float_as_uint(acc[0][0][0]) ^ __float_as_uint(acc[1][0][0])) & p.zero;
                    __syncwarp();
                    if (elect_one()) mbar_arrive(smem_u32(&s_empty[slot_used]) + dep);
                }
                if (!ok) break;
                // C fragment: [0..1] = row g, tokens 2t, 2t+1; [2..3] = row g + 8
                AccT* part = s_part + (size_t)warp * kRowsCta * (kTok + 1);
#pragma unroll
                for (int r = 0; r < 2; ++r)
#pragma unroll
                    for (int q = 0; q < GROUPS; ++q) {
                        part[(16 * r + g) * (kTok + 1) + 8 * q + 2 * t] = acc[r][q][0];
                        part[(16 * r + g) * (kTok + 1) + 8 * q + 2 * t + 1] = acc[r][q][1];
                        part[(16 * r + g + 8) * (kTok + 1) + 8 * q + 2 * t] = acc[r][q][2];
                        part[(16 * r + g + 8) * (kTok + 1) + 8 * q + 2 * t + 1] = acc[r][q][3];
                    }
                __syncwarp();
                if (elect_one()) mbar_arrive(smem_u32(&s_sync));
                ok = mbar_wait_all(smem_u32(&s_sync), sync_ph, abort_flag, p.watchdog, kWdStreamSync);
                sync_ph ^= 1u;
                if (!ok) break;
                for (int o = threadIdx.x; o < kRowsCta * kTok; o += kConsumers * 32) {
                    const int row = o % kRowsCta, tok = o / kRowsCta;    // consecutive threads: consecutive channels
                    AccT sum = 0;
#pragma unroll
                    for (int k = 0; k < kConsumers; ++k) sum += s_part[((size_t)k * kRowsCta + row) * (kTok + 1) + tok];
                    const int64_t j = j0 + row, tt = t0 + tok;
                    if (j < p.N && tt < p.M) {
                        if (kIntegers && p.acc_out != nullptr) {
                            p.acc_out[tt * p.N + j] = (int)sum >> p.acc_shift;
                        } else {
                            float v;
                            if (kIntegers) {
                                // (float)sum * 2^-shift is exact: the shift is folded into the channel scale
                                const float sw = __ldg(p.w_scale + j) * (1.0f / (float)(1 << p.acc_shift));
                                v = fmaf((float)sum, __ldg(p.a_delta + tt) * sw, __ldg(p.bias + j));
                            } else {
                                v = fmaf((float)sum, __ldg(p.w_scale + j), __ldg(p.bias + j));
                            }
                            if (p.yt == FQ_F32) static_cast<float*>(p.y)[tt * p.ldy + j] = v;
                            else static_cast<__nv_bfloat16*>(p.y)[tt * p.ldy + j] = __float2bfloat16_rn(v);
                        }
                    }
                }
                // the partial sums are rewritten by the next pass / row group
                __syncwarp();
                if (elect_one()) mbar_arrive(smem_u32(&s_sync));
                ok = mbar_wait_all(smem_u32(&s_sync), sync_ph, abort_flag, p.watchdog, kWdStreamSync);
                sync_ph ^= 1u;
            }
        }
    }
    __syncthreads();
}

template <int MODE, int GROUPS>
cudaError_t launch_stream(const CUtensorMap& map, StreamParams p, cudaStream_t stream) {
    typedef typename std::conditional<Geometry<MODE>::kIntegers, int, float>::type AccT;
    const int sms = device_sm_count();
    const size_t part_bytes = (size_t)kConsumers * kRowsCta * (8 * GROUPS + 1) * sizeof(AccT);
    const size_t budget = 227 * 1024 - 1024 /*alignment*/ - 1024 /*static*/ - part_bytes;
    int depth = (int)(budget / kStageBytes);
    if (depth > kMaxDepth) depth = kMaxDepth;
    if (depth < 2) return cudaErrorInvalidConfiguration;
    p.depth = depth;
    p.watchdog = watchdog_device_ptr();
    if (!p.watchdog) return cudaErrorUnknown;
    const size_t smem = (size_t)depth * kStageBytes + part_bytes + 1024;
    auto kern = weight_stream_kernel<MODE, GROUPS>;
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem);
    if (e != cudaSuccess) return e;
    const int64_t row_groups = (p.N + kRowsCta - 1) / kRowsCta;
    const unsigned grid = (unsigned)(row_groups < sms ? row_groups : sms);
    return launch_pdl(kern, grid, (unsigned)kThreads, smem, stream, 1u, map, p);
}

// Rows shorter than one TMA box (K < 256): one thread per output, plain loops.  Such projections are a
// few kilobytes; nothing about them is worth tuning.
template <typename XT>
__global__ void linear_wonly4_small_kernel(const XT* __restrict__ x, int64_t M, int K, int64_t ldx,
                                           const uint8_t* __restrict__ wcodes, const float* __restrict__ w_scale,
                                           const float* __restrict__ bias, int64_t N, void* __restrict__ y, fq_dtype yt,
                                           int64_t ldy) {
    griddep_wait();
    griddep_launch_dependents();
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, t = blockIdx.y;
    if (j >= N || t >= M) return;
    const uint8_t* wrow = wcodes + j * (K / 2);
    float acc = 0.0f;
    for (int c = 0; c < K; c += 2) {
        const int byte = wrow[c / 2];
        const float q0 = (float)(((byte & 15) ^ 8) - 8), q1 = (float)(((byte >> 4) ^ 8) - 8);
        float x0, x1;
        if (sizeof(XT) == 4) {
            x0 = reinterpret_cast<const float*>(x)[t * ldx + c];
            x1 = reinterpret_cast<const float*>(x)[t * ldx + c + 1];
        } else {
            x0 = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(x)[t * ldx + c]);
            x1 = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(x)[t * ldx + c + 1]);
        }
        acc = fmaf(q0, x0, acc);
        acc = fmaf(q1, x1, acc);
    }
    const float v = fmaf(acc, w_scale[j], bias[j]);
    if (yt == FQ_F32) static_cast<float*>(y)[t * ldy + j] = v;
    else static_cast<__nv_bfloat16*>(y)[t * ldy + j] = __float2bfloat16_rn(v);
}

}  // namespace

bool build_stream_tmap(Weights& W) {
    W.tmap_stream_valid = false;
    // rows of whole 128-byte lines only (K a multiple of 256 at 4 bits, of 128 at 8); other widths take the general kernels
    const int64_t row_bytes = W.bits == 4 ? W.K / 2 : W.K;
    if (W.N == 0 || W.K % (W.bits == 4 ? 256 : 128) != 0) return true;
    const uint64_t dims[3] = {128, (uint64_t)row_bytes / 128, (uint64_t)W.N};
    const uint64_t strides[2] = {128, (uint64_t)row_bytes};
    const uint32_t box[3] = {128, (uint32_t)kLines, (uint32_t)kRowsCta};
    W.tmap_stream_valid = encode_tiled(&W.tmap_stream, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, W.codes, dims, strides, box, true);
    return W.tmap_stream_valid;
}

bool gemm_stream_applies(int64_t M, const Weights& W) {
    // Measured against the tcgen05 kernel over M in {1, 8, 16} x K, N in {4096, 8192, 16384}, operands from HBM: ahead wherever the
    // row groups make at most two rounds over the SMs (N <= 64 x SMs: 4096 and 8192 rows) -- every row group ends with a
    // rendezvous and a reduction, which four rounds of short rows (K = 4096, N = 16384: 19 us against 10 us) do not amortise --
    // up to 128 Mi weights for at most 8 tokens and 64 Mi for at most 16 (16 x 16384 x 8192: 23 us against 21 us).
    if (!W.tmap_stream_valid || M < 1 || M > 16) return false;
    // 8-bit weights (twice the bytes per row): ahead where the row groups make ONE round over the SMs, up to 64 Mi
    // weights (16 tokens, K = 8192, N = 4096: 12.8 us against 17.5 us; K = 4096, N = 8192: 14.0 against 11.5 us)
    if (W.bits == 8) return W.N <= 32ll * device_sm_count() && W.N * W.K <= (1ll << 26);
    if (W.N > 64ll * device_sm_count()) return false;
    return W.N * W.K <= (M <= 8 ? (1ll << 27) : (1ll << 26));
}

cudaError_t launch_gemm_stream(const int8_t* a8, int64_t M, const Weights& W, int acc_shift, const GemmOut& out,
                               cudaStream_t stream) {
    StreamParams p{};
    p.x = a8; p.ldx = W.K; p.M = M; p.N = W.N; p.K = (int)W.K; p.acc_shift = acc_shift;
    p.a_delta = out.a_delta; p.w_scale = W.w_scale; p.bias = W.bias;
    p.y = out.y; p.yt = out.yt; p.ldy = out.ldy; p.acc_out = out.acc;
    if (W.bits == 8)
        return M <= 8 ? launch_stream<kModeInt8, 1>(W.tmap_stream, p, stream) : launch_stream<kModeInt8, 2>(W.tmap_stream, p, stream);
    if (M <= 8) return launch_stream<kModeInt, 1>(W.tmap_stream, p, stream);
    return launch_stream<kModeInt, 2>(W.tmap_stream, p, stream);
}

cudaError_t launch_linear_wonly4(const void* x, fq_dtype xt, int64_t M, int64_t ldx, const Weights& W, void* y,
                                 fq_dtype yt, int64_t ldy, cudaStream_t stream) {
    if (M == 0 || W.N == 0) return cudaSuccess;
    if (!W.tmap_stream_valid) {
        if (M > 65535) return cudaErrorInvalidConfiguration;
        const dim3 grid((unsigned)((W.N + 127) / 128), (unsigned)M);
        if (xt == FQ_F32)
            linear_wonly4_small_kernel<float><<<grid, 128, 0, stream>>>(static_cast<const float*>(x), M, (int)W.K, ldx, W.codes,
                                                                        W.w_scale, W.bias, W.N, y, yt, ldy);
        else
            linear_wonly4_small_kernel<__nv_bfloat16><<<grid, 128, 0, stream>>>(static_cast<const __nv_bfloat16*>(x), M,
                                                                                (int)W.K, ldx, W.codes, W.w_scale, W.bias,
                                                                                W.N, y, yt, ldy);
        return cudaGetLastError();
    }
    StreamParams p{};
    p.x = x; p.ldx = ldx; p.M = M; p.N = W.N; p.K = (int)W.K;
    p.w_scale = W.w_scale; p.bias = W.bias; p.y = y; p.yt = yt; p.ldy = ldy;
    // eight tokens per pass over the weights: two token groups at a time need more registers than a thread has
    // (16 tokens measured 130 us against 2 x 59 us at 16384 x 16384)
    if (xt == FQ_F32) return launch_stream<kModeF32, 1>(W.tmap_stream, p, stream);
    return launch_stream<kModeBf16, 1>(W.tmap_stream, p, stream);
}

}  // namespace fq
