// Integer GEMM of Eq. 8 on the 5th-generation tensor cores (sm_100a):
//   acc[j][t] = sum_c qW[j][c] * qA[t][c]   tcgen05.mma kind::i8, int32 accumulators in TMEM
//   y[t][j]   = delta_t * s^W_j * acc + b_j fused epilogue straight out of TMEM
//
// Orientation.  The 128 rows of an MMA tile are OUTPUT CHANNELS (weight rows),
// the MMA's N dimension (16..256, any multiple of 16) is a tile of TOKENS.  A
// TMEM lane therefore owns one output channel: its scale and bias are per-thread
// scalars in the epilogue, a warp stores 32 consecutive channels of one token
// (coalesced), and ragged token counts (M = 50, 816, ...) are absorbed by the
// free N dimension instead of padding a fixed 128-row tile.
//
// Operands.  Activations (the MMA's B operand) arrive as int8 by TMA, K-major with
// 128-byte rows in the 128B-swizzled shared memory layout.  8-bit weights (the A
// operand) arrive the same way.  4-bit weights stay packed in HBM and in their TMA
// stage; four unpack warps expand each row's 64 packed bytes to 128 int8 holding
// 16*code (nibble moved to the high half of the byte: no sign extension needed) and
// write them with tcgen05.st straight into TENSOR MEMORY, from where the MMA takes
// its A operand -- the unpacked weights never touch shared memory, which is the
// bandwidth that bounds this kernel.  The accumulator is then an exact multiple of
// 2^acc_shift that the epilogue folds into the scale.
//
// Roles (warp specialised, persistent over tiles):
//   warp 0       TMA producer          warp 1  MMA issuer + TMEM allocator
//   warps 2-9    epilogue (two warps per TMEM lane quadrant, alternating 16-token chunks)
//   warps 10-17  nibble unpack (two sets of four, alternating k-blocks), warp 18 TMA producer
//                of packed weights (4-bit weights); warp 10 TMA producer of int8 weights (8-bit)
// Every role runs its loop with the whole warp converged and elects one lane (elect.sync) for
// the issue itself; a k-block of the MMA warp is one block of PTX that also tests the next
// k-block's barriers (see issue_kblock_*).  With 4-bit weights three rings are decoupled:
// activations (TMA -> MMA), packed weights (TMA -> unpack, deep and cheap: 8 KB a stage) and
// unpacked weights (unpack -> MMA, 32 TMEM columns a stage); one tcgen05.commit per k-block
// frees both the activation stage and the k-block's TMEM slot.
// Variants: CTAS = 2 runs CTA pairs (cta_group::2, 256 channels per MMA, each CTA staging half
// of the token tile); SPLIT lets the CTAs of a cluster share a tile along K and exchange int32
// partial sums through global scratch.
// bf16 outputs leave through a per-warp 1 KB shared-memory transposer so that global
// stores are 16-byte vectors of 8 consecutive channels; fp32/raw outputs store directly.
// Every mbarrier wait is bounded by wall-clock time; on expiry the CTA records a
// code in the watchdog word, stops issuing work, and still frees its TMEM.
#include <cuda_bf16.h>

#include <string.h>

#include <mutex>

#include "fq_common.cuh"
#include "ptx_sm100.cuh"
#include "act_common.cuh"

namespace fq {

__device__ uint32_t g_watchdog_word = 0;

uint32_t* watchdog_device_ptr() {
    // the symbol's address differs per device: looked up once for each
    static std::mutex mutex;
    static uint32_t* addr[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    const bool cached = dev >= 0 && dev < 64;
    std::lock_guard<std::mutex> lock(mutex);
    if (cached && addr[dev] != nullptr) return addr[dev];
    uint32_t* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_watchdog_word) != cudaSuccess) return nullptr;
    if (cached) addr[dev] = p;
    return p;
}

// Self-test of the bounded-wait machinery: one warp waits, with the ordinary wait routine and a caller-chosen
// limit, on a barrier that nobody ever arrives at.  The wait must give up, record its code in the watchdog word
// and let the kernel end normally.
__global__ void watchdog_selftest_kernel(uint32_t* watchdog, uint64_t limit_ns) {
    __shared__ uint64_t s_bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        s_abort = 0;
        mbar_init(smem_u32(&s_bar), 1);
        fence_mbarrier_init();
    }
    __syncthreads();
    mbar_wait_all(smem_u32(&s_bar), 0u, &s_abort, watchdog, 0x400u, false, limit_ns);
}

cudaError_t launch_watchdog_selftest(uint64_t limit_ns, cudaStream_t stream) {
    uint32_t* wd = watchdog_device_ptr();
    if (!wd) return cudaErrorUnknown;
    watchdog_selftest_kernel<<<1, 32, 0, stream>>>(wd, limit_ns);
    return cudaGetLastError();
}

cudaError_t read_and_clear_watchdog(uint32_t* word) {
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return e;
    e = cudaMemcpyFromSymbol(word, g_watchdog_word, sizeof(uint32_t));
    if (e != cudaSuccess) return e;
    const uint32_t zero = 0;
    return cudaMemcpyToSymbol(g_watchdog_word, &zero, sizeof(uint32_t));
}

namespace {

constexpr int kTileN = 128;          // output channels per tile (MMA M)
constexpr int kBlockK = 128;         // int8 elements (= bytes) of K per pipeline stage
constexpr int kAccStages = 2;
constexpr int kEpiWarps = 8;
constexpr int kEpiBuffers = 2;                          // output buffers per epilogue warp (bulk stores in flight; four measured no faster)
constexpr int kEpiStageBytes = kEpiBuffers * 16 * 64;   // per epilogue warp: buffers of 16 tokens x 32 channels of bf16
constexpr int kThreadsW8 = 32 * (2 + kEpiWarps + 1);   // + one warp: TMA producer of int8 weights
constexpr int kFirstUnpackWarp = 2 + kEpiWarps;
constexpr int kUnpackSets = 2;          // sets of four unpack warps, one TMEM lane quadrant each
constexpr int kThreadsW4 = 32 * (2 + kEpiWarps) + kUnpackSets * 128 + 32;
constexpr int kMaxStagesW = 8;
constexpr int kColsW = kBlockK / 4;     // TMEM columns of one unpacked k-block (128 int8 per lane)
constexpr int kMaxStages = 16;
constexpr int kMaxStagesP = 16;
constexpr int kMaxSplit = 16;          // K slices per tile, at most
constexpr int kMaxSplitTiles = 1024;   // tiles of a launch that splits K (one counter each, ahead of the partial sums)
constexpr size_t kCounterBytes = kMaxSplitTiles * sizeof(uint32_t);

struct Params {
    int64_t M, N, K;
    int bt;              // tokens per tile (MMA N), multiple of 16, <= 256
    int stages;          // activation ring (and int8 weight ring, in lockstep, for 8-bit weights)
    int stages_p;        // packed-weight ring (4-bit weights)
    int stages_w;        // unpacked-weight ring (4-bit weights)
    int m_tiles, n_tiles;
    int band;            // token tiles per band of the tile order (see tile_coords); m_tiles = one band = channel-major order
    int tmem_cols;
    int acc_shift;
    const float* w_scale;
    const float* bias;
    GemmOut out;
    uint32_t* watchdog;
    // index arithmetic done once on the host (integer divisions cost the short launches ~0.3 us)
    int cluster_shift;   // log2 of the CTAs per cluster (1 for CTA pairs)
    int unit_step;       // CTAs (or pairs) in the grid
    int units_q, units_rem;   // work units per CTA: units_q, one more for the first units_rem CTAs
    int kb_per;          // k-blocks of one work unit (all of K, or K / split)
    int split, split_shift;   // K split: a tile is `split` (power of two) work units, each on a slice of K
    int32_t* partials;   // [tile][slice][bt tokens][128 channels] int32 raw sums of the slices (K split)
    uint32_t* counters;  // [tile] slices finished so far; zeroed by the host before the launch (K split)
    int delta_vec;       // a_delta is 16-byte aligned: the epilogue may read four steps per load
    uint32_t zero;       // 0, as a run-time value (see the unpack warps' release of a packed stage)
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
// ---- CTA-pair (cta_group::2) helpers -----------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ void mbar_arrive_cta(uint32_t bar, uint32_t rank) {
    asm volatile(
        "{\n\t.reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.shared::cluster.b64 _, [ra];\n\t}"
        ::"r"(bar), "r"(rank)
        : "memory");
}
// Pair variant of the tiled load: issued by both CTAs into their own shared memory, but the
// bytes are counted on the barrier of the pair's even CTA (address with the peer bit cleared).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar & 0xFEFFFFFFu)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

template <int CTAS>
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    if (CTAS == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else {   // same warp index in both CTAs of the pair, same destination offset
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
}
template <int CTAS>
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    if (CTAS == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
    else
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// One k-block of work for the issuing warp, as ONE block of PTX so that the two barrier tests for
// the NEXT k-block are in flight while this k-block's four MMAs and its commits are issued (their
// results are read only at the end; separate asm statements would stall on each test's ~100-cycle
// latency).  Must be called by a converged warp: every lane executes the tests, and the lane that
// elect.sync picks inside the block issues the MMAs and commits (measured: 160 cycles per k-block
// with the election inside the block, 400 with a predicate derived from the lane index).
//   a[4]      A operand of the four K=32 steps: TMEM addresses (TS) or shared-memory descriptors (SS)
//   bar_stage barrier that frees the k-block's shared-memory (and TMEM weight) stage
//   bar_acc   barrier "accumulator complete", or 0 when this is not the tile's last k-block
// Returns 1 if both tested phases were complete (0 when `peek` is 0).
#define FQ_ISSUE_HEAD                                                   \
    "{\n\t"                                                             \
    ".reg .pred pl, pacc, pt, pk, pa, pw, pc;\n\t"                       \
    "elect.sync _|pl, 0xffffffff;\n\t"                                  \
    "setp.ne.b32 pacc, %12, 0;\n\t"                                     \
    "setp.eq.b32 pt, %1, %1;\n\t"                                       \
    "setp.ne.b32 pk, %15, 0;\n\t"                                       \
    "setp.ne.b32 pa, %1, %1;\n\t"                                       \
    "setp.ne.b32 pw, %1, %1;\n\t"                                       \
    "@pk mbarrier.test_wait.parity.shared::cta.b64 pa, [%16], %17;\n\t" \
    "@pk mbarrier.test_wait.parity.shared::cta.b64 pw, [%18], %19;\n\t"
#define FQ_ISSUE_MMAS(CG, L, R)                                                          \
    "@pl tcgen05.mma.cta_group::" CG ".kind::i8 [%2], " L "%3" R ", %7, %11, pacc;\n\t"   \
    "@pl tcgen05.mma.cta_group::" CG ".kind::i8 [%2], " L "%4" R ", %8, %11, pt;\n\t"     \
    "@pl tcgen05.mma.cta_group::" CG ".kind::i8 [%2], " L "%5" R ", %9, %11, pt;\n\t"     \
    "@pl tcgen05.mma.cta_group::" CG ".kind::i8 [%2], " L "%6" R ", %10, %11, pt;\n\t"
#define FQ_ISSUE_COMMITS_1                                                                          \
    "@pl tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%13];\n\t"          \
    "setp.ne.and.b32 pc, %14, 0, pl;\n\t"                                                           \
    "@pc tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%14];\n\t"
#define FQ_ISSUE_COMMITS_2                                                                                          \
    "@pl tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%13], %20;\n\t"  \
    "setp.ne.and.b32 pc, %14, 0, pl;\n\t"                                                                           \
    "@pc tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%14], %20;\n\t"
#define FQ_ISSUE_TAIL            \
    "and.pred pa, pa, pw;\n\t"   \
    "selp.b32 %0, 1, 0, pa;\n\t" \
    "}"
#define FQ_ISSUE_OPERANDS(ACON)                                                                                      \
    : "=r"(ready)                                                                                                    \
    : "r"(issue), "r"(d_tmem), ACON(a[0]), ACON(a[1]), ACON(a[2]), ACON(a[3]), "l"(b[0]), "l"(b[1]), "l"(b[2]),      \
      "l"(b[3]), "r"(idesc), "r"(accumulate), "r"(bar_stage), "r"(bar_acc), "r"(peek), "r"(peek_bar_a),              \
      "r"(peek_par_a), "r"(peek_bar_w), "r"(peek_par_w), "h"(mask)                                                   \
    : "memory"
#define FQ_CON_R(x) "r"(x)
#define FQ_CON_L(x) "l"(x)

template <int CTAS>
__device__ __forceinline__ uint32_t issue_kblock_ts(uint32_t issue, uint32_t d_tmem, const uint32_t* a, const uint64_t* b,
                                                    uint32_t idesc, uint32_t accumulate, uint32_t bar_stage,
                                                    uint32_t bar_acc, uint32_t peek, uint32_t peek_bar_a,
                                                    uint32_t peek_par_a, uint32_t peek_bar_w, uint32_t peek_par_w) {
    uint32_t ready;
    const uint16_t mask = 3;
    if (CTAS == 1)
        asm volatile(FQ_ISSUE_HEAD FQ_ISSUE_MMAS("1", "[", "]") FQ_ISSUE_COMMITS_1 FQ_ISSUE_TAIL FQ_ISSUE_OPERANDS(FQ_CON_R));
    else
        asm volatile(FQ_ISSUE_HEAD FQ_ISSUE_MMAS("2", "[", "]") FQ_ISSUE_COMMITS_2 FQ_ISSUE_TAIL FQ_ISSUE_OPERANDS(FQ_CON_R));
    return ready;
}
template <int CTAS>
__device__ __forceinline__ uint32_t issue_kblock_ss(uint32_t issue, uint32_t d_tmem, const uint64_t* a, const uint64_t* b,
                                                    uint32_t idesc, uint32_t accumulate, uint32_t bar_stage,
                                                    uint32_t bar_acc, uint32_t peek, uint32_t peek_bar_a,
                                                    uint32_t peek_par_a, uint32_t peek_bar_w, uint32_t peek_par_w) {
    uint32_t ready;
    const uint16_t mask = 3;
    if (CTAS == 1)
        asm volatile(FQ_ISSUE_HEAD FQ_ISSUE_MMAS("1", "", "") FQ_ISSUE_COMMITS_1 FQ_ISSUE_TAIL FQ_ISSUE_OPERANDS(FQ_CON_L));
    else
        asm volatile(FQ_ISSUE_HEAD FQ_ISSUE_MMAS("2", "", "") FQ_ISSUE_COMMITS_2 FQ_ISSUE_TAIL FQ_ISSUE_OPERANDS(FQ_CON_L));
    return ready;
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
// Four TS-form MMAs (one K = 128 atom) from the lane elect.sync picks; no commit: the stage's last atom,
// issued by issue_kblock_ts right after, commits for both.
__device__ __forceinline__ void issue_mmas_ts(uint32_t d_tmem, const uint32_t* a, const uint64_t* b, uint32_t idesc,
                                              uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred pl, pacc, pt;\n\t"
        "elect.sync _|pl, 0xffffffff;\n\t"
        "setp.ne.b32 pacc, %10, 0;\n\t"
        "setp.eq.b32 pt, %0, %0;\n\t"
        "@pl tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %5, %9, pacc;\n\t"
        "@pl tcgen05.mma.cta_group::1.kind::i8 [%0], [%2], %6, %9, pt;\n\t"
        "@pl tcgen05.mma.cta_group::1.kind::i8 [%0], [%3], %7, %9, pt;\n\t"
        "@pl tcgen05.mma.cta_group::1.kind::i8 [%0], [%4], %8, %9, pt;\n\t"
        "}"
        ::"r"(d_tmem), "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]), "r"(idesc),
          "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 16 TMEM lanes x 16 columns in the layout of a warp-level MMA accumulator: thread T holds, for column groups n = 0, 1,
//   r[4n + 0], r[4n + 1] = lane T/4,     columns 8n + 2(T%4), 8n + 2(T%4) + 1
//   r[4n + 2], r[4n + 3] = lane T/4 + 8, the same two columns.
// With channels on the lanes and tokens on the columns, a register pair is one channel at two adjacent tokens --
// the fragment that stmatrix stores transposed, i.e. token-major.
__device__ __forceinline__ void tmem_ld_16x256b_x2(uint32_t taddr, uint32_t* r) {
    asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}
// Four 8x8 matrices of 16-bit elements, each thread's register i a fragment (row T/4, columns 2(T%4), 2(T%4)+1) of
// matrix i, stored TRANSPOSED: the 16 bytes at the address given by thread 8i + r receive column r of matrix i.
__device__ __forceinline__ void stmatrix_x4_trans(uint32_t addr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3) {
    asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1, %2, %3, %4};"
                 ::"r"(addr), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
                 : "memory");
}
// Tiled bulk STORE shared -> global (a store, never a multicast load); rows and columns beyond the tensor's extent
// are clipped by the copy engine.  Completion is tracked per issuing thread in bulk groups.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int c0, int c1, uint32_t src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(src)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// At most N of this thread's bulk groups still read their shared-memory source.
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
// One channel at two adjacent tokens: y = acc * (delta_t * s_j) + b_j, rounded to bf16, token 2k in the low half.
__device__ __forceinline__ uint32_t scale_pair_bf16(uint32_t a0, uint32_t a1, float2 d, float2 sw2, float2 bj2) {
    const float2 a2 = make_float2((float)(int)a0, (float)(int)a1);
    const float2 v2 = f2_fma(a2, f2_mul(d, sw2), bj2);
    uint32_t w;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w) : "f"(v2.y), "f"(v2.x));
    return w;
}

// Shared-memory matrix descriptor: K-major operand, 128-byte rows, 128B swizzle,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);   // start address, 16-byte units
    d |= (uint64_t)1 << 16;                    // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                    // 128-byte swizzle
    return d;
}
// Instruction descriptor: s8 x s8 -> s32, both operands K-major, M = m (128, or 256 for a CTA pair), N = n.
__device__ __forceinline__ uint32_t instr_desc_i8(int m, int n) {
    return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// After an expired wait a producer lets the copies it already issued land before the CTA gives its
// shared memory back: they complete within microseconds, so a bounded pause suffices.
__device__ __forceinline__ void drain_after_abort() {
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 100000ull) __nanosleep(1000);
}

enum : uint32_t {
    kWdProducer = 1u, kWdMmaFull = 2u, kWdMmaAcc = 4u, kWdEpilogue = 8u, kWdUnpackFull = 16u,
    kWdUnpackEmpty = 32u, kWdDrain = 64u, kWdPartials = 128u
};

// CTAS = 2: two CTAs of a cluster work as a pair on a 256-channel x bt-token tile (cta_group::2):
// each loads its own 128 weight rows and HALF of the token tile, the even CTA issues the MMAs for
// both, and every MMA reads the token halves out of both CTAs' shared memory.  This halves the
// activation bytes each SM pulls from L2, which is what bounds the single-CTA kernel.
// ATOMS (4-bit weights, single CTAs, token tiles of at most 128): a pipeline stage holds ATOMS k-blocks of 128
// channels (two 128-byte swizzle atoms side by side).  The kernel is bound by instruction issue, and the waits,
// arrivals, fences and ring arithmetic of every role are paid per stage: twice the channels per stage take a
// third off the instructions per channel.  (Longer token tiles have no TMEM left for slots twice as wide.)
template <int BITS, int CTAS, bool SPLIT, int ATOMS = 1>
__global__ void __launch_bounds__(BITS == 4 ? kThreadsW4 : kThreadsW8, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w,
                    const __grid_constant__ CUtensorMap map_y, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full_tma[kMaxStages];     // activations (+ int8 weights) landed
    __shared__ uint64_t s_empty[kMaxStages];        // ... consumed by the MMAs (one commit per k-block; for 4-bit
                                                    // weights it also frees that k-block's TMEM weight slot)
    __shared__ uint64_t s_full_p[kMaxStagesP];      // packed weights landed
    __shared__ uint64_t s_empty_p[kMaxStagesP];     // ... read by the unpack warps
    __shared__ uint64_t s_full_w8[kMaxStagesW];     // unpacked weights written
    __shared__ uint64_t s_acc_full[kAccStages];
    __shared__ uint64_t s_acc_empty[kAccStages];
    __shared__ uint64_t s_epi_sync;                 // K split: rendezvous of the eight epilogue warps (bounded, unlike bar.sync)
    __shared__ int s_last[2];                       // K split: this CTA counted the last slice of its tile (alternating slots)
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    volatile int* abort_flag = &s_abort;
    if (threadIdx.x == 32) {
        // the three copy descriptors are kernel parameters: fetching them now takes their first-use latency (a few
        // hundred nanoseconds each) off the path between the end of the kernel ahead and this kernel's first copy
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_w)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_y)) : "memory");
    }
    const uint32_t cta_rank = CTAS == 2 ? cluster_ctarank() : 0u;
    const bool leader = cta_rank == 0;
    // K split: a tile is `split` work units, unit = tile * split + slice, slice s
    // covering k-blocks [s * k_blocks, (s + 1) * k_blocks).  Any CTA takes any unit; the CTA that
    // finishes a tile's last slice adds up the slices' partial sums and runs the epilogue.
    const int split = SPLIT ? p.split : 1;   // compile-time 1 in the common instantiation
    const int split_shift = SPLIT ? p.split_shift : 0;
    const int bt_cta = p.bt / CTAS;                 // token rows this CTA loads

    // carve dynamic shared memory: [A8 stages][W8 stages][packed stages][epilogue transposers], 1024-byte aligned
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_atom = (uint32_t)bt_cta * kBlockK;        // one 128-channel atom of the token tile
    const uint32_t a_bytes = a_atom * ATOMS;
    const uint32_t w_bytes = kTileN * kBlockK;
    const uint32_t pk_atom = kTileN * kBlockK / 2;
    const uint32_t pk_bytes = pk_atom * ATOMS;
    constexpr int kSlotCols = kColsW * ATOMS;                   // TMEM columns of one unpacked stage
    const uint32_t smem_a = base;
    const uint32_t smem_w = smem_a + (uint32_t)p.stages * a_bytes;
    const uint32_t smem_p = smem_w + (BITS == 4 ? 0u : (uint32_t)p.stages * w_bytes);
    const uint32_t smem_e = smem_p + (BITS == 4 ? (uint32_t)p.stages_p * pk_bytes : 0u);
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));   // generic pointer to `base`

    if (threadIdx.x == 0) {
        // (One thread on purpose: spreading these initialisations over the lanes of a warp, one ring
        // slot per lane, shortened the set-up by 0.3 us but made the 8-bit main loop 10 % slower.)
        s_abort = 0;
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&s_full_tma[s]), BITS == 8 ? 2 : 1);   // 8-bit: activation and weight producers
            mbar_init(smem_u32(&s_empty[s]), 1);
        }
        if (BITS == 4) {
            for (int s = 0; s < p.stages_p; ++s) {
                mbar_init(smem_u32(&s_full_p[s]), 1);
                mbar_init(smem_u32(&s_empty_p[s]), 4);
            }
            for (int s = 0; s < p.stages_w; ++s) mbar_init(smem_u32(&s_full_w8[s]), 4 * CTAS);
        }
        for (int a = 0; a < kAccStages; ++a) {
            mbar_init(smem_u32(&s_acc_full[a]), 1);
            mbar_init(smem_u32(&s_acc_empty[a]), kEpiWarps * CTAS);
        }
        mbar_init(smem_u32(&s_epi_sync), kEpiWarps);
        fence_mbarrier_init();
        fence_proxy_async_smem();
    }
    if (warp == 1) tmem_alloc<CTAS>(smem_u32(&s_tmem_base), (uint32_t)p.tmem_cols);
    tc_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync_all();              // the peer's barriers exist before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    // Everything above is on-chip setup; from here on global memory is touched (activations written
    // by the kernel before this one, outputs that it may still be reading).
    // Only the warps that touch what the kernel ahead writes (or may still read) wait for it: the activation
    // producer, and the epilogue warps (per-token steps, K-split scratch, the output).  A weight handle is
    // complete before any call that uses it is enqueued, so the weight producer streams tiles in, the unpack
    // warps fill their TMEM slots, and the MMA warp parks on its barriers while the prologue still runs.
    if (warp == 0 || (warp >= 2 && warp < 2 + kEpiWarps)) griddep_wait();
    griddep_launch_dependents();

    // work units: (super-tile of 128*CTAS channels) x (token tile) [x K slice]; one unit per CTA or
    // CTA pair at a time
    const int num_units = (p.m_tiles * p.n_tiles) << split_shift;
    const int unit0 = (int)blockIdx.x >> p.cluster_shift;
    const int unit_step = p.unit_step;
    const int my_units = p.units_q + (unit0 < p.units_rem ? 1 : 0);
    const int k_blocks = p.kb_per;
    auto tile_of = [&](int unit) { return unit >> split_shift; };
    // Tile order.  Consecutive tile numbers -- the tiles the SMs work on at the same time -- cover a compact block of
    // the output: the token tiles are cut into bands of p.band, a band is walked channel tile by channel tile with
    // its token tiles fastest.  What one wave of CTAs pulls through L2 is then band activation tiles plus SMs/band
    // weight tiles instead of every activation tile of the batch (long batches: the int8 activations alone exceed
    // L2, and in channel-major order every wave streamed all of them from HBM again).
    auto m_of = [&](int tile) {
        if (p.band >= p.m_tiles) return tile % p.m_tiles;
        const int b = tile / (p.band * p.n_tiles);
        const int r = tile - b * (p.band * p.n_tiles);
        const int rows = max(1, min(p.band, p.m_tiles - b * p.band));   // (a producer also maps the unit past its last one)
        return b * p.band + r % rows;
    };
    auto n_of = [&](int tile) {
        if (p.band >= p.m_tiles) return tile / p.m_tiles;
        const int b = tile / (p.band * p.n_tiles);
        const int r = tile - b * (p.band * p.n_tiles);
        return r / max(1, min(p.band, p.m_tiles - b * p.band));
    };
    auto kb0_of = [&](int unit) { return (unit & (split - 1)) * k_blocks; };   // first k-block of the unit's slice

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        // The whole warp runs the loop and waits; one lane issues.  (A lone lane looping while its
        // warp-mates are parked at the final __syncthreads was measured 2-3x slower per barrier
        // hand-off: every dependent wait/branch of the lone lane pays for the divergent warp.)
        {
            const uint32_t tx = a_bytes;
            const int total_kb = my_units * k_blocks;
            bool ok = true;
            int stage = 0, kb = 0, unit = unit0;
            uint32_t phase = 0;
            int t0 = m_of(tile_of(unit)) * p.bt + (int)cta_rank * bt_cta;
            int kb0 = kb0_of(unit);
            bool peek = false;
            for (int n = 0; n < total_kb; ++n) {
                ok = mbar_wait_all_lazy(smem_u32(&s_empty[stage]), phase ^ 1u, abort_flag, p.watchdog, kWdProducer, peek);
                if (!ok) break;
                {   // look at the next stage now: the test's latency hides behind the copy issued below
                    const int s1 = stage + 1 == p.stages ? 0 : stage + 1;
                    const uint32_t ph1 = s1 == 0 ? phase ^ 1u : phase;
                    peek = n + 1 < total_kb && mbar_test_wait(smem_u32(&s_empty[s1]), ph1 ^ 1u);
                }
                if (elect_one()) {
                    const uint32_t bar = smem_u32(&s_full_tma[stage]);
                    if (CTAS == 1) {
                        mbar_arrive_expect_tx(bar, tx);
#pragma unroll
                        for (int h = 0; h < ATOMS; ++h)     // channels past K arrive as zeros
                            tma_load_2d(smem_a + stage * a_bytes + h * a_atom, &map_a, ((kb0 + kb) * ATOMS + h) * kBlockK, t0, bar);
                    } else {
                        // the pair's bytes are all counted on the even CTA's barrier, which it arms for both
                        if (leader) mbar_arrive_expect_tx(bar, tx * CTAS);
                        tma_load_2d_pair(smem_a + stage * a_bytes, &map_a, (kb0 + kb) * kBlockK, t0, bar);
                    }
                }
                if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                if (++kb == k_blocks) {
                    kb = 0;
                    unit += unit_step;
                    t0 = m_of(tile_of(unit)) * p.bt + (int)cta_rank * bt_cta;
                    kb0 = kb0_of(unit);
                }
            }
            if (!ok && lane == 0) drain_after_abort();
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        // All lanes of the warp run the loop and the waits (converged); lane 0 of the pair's even
        // CTA issues the MMAs and commits.
        if (leader) {
            const uint32_t idesc = instr_desc_i8(kTileN * CTAS, p.bt);
            int stage = 0, wstage = 0;
            uint32_t phase = 0, wphase = 0;
            int acc_stage = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            // The barriers of the NEXT k-block are tested (without blocking) inside the block of PTX
            // that issues the current one: a barrier test has ~100 cycles of latency, and two of them
            // in series per k-block would otherwise sit on the issuing warp's critical path.
            bool ready = false;
            int left = my_units * k_blocks;   // k-blocks still to issue
            for (int unit = unit0; unit < num_units && ok; unit += unit_step) {
                ok = mbar_wait_all(smem_u32(&s_acc_empty[acc_stage]), acc_phase ^ 1u, abort_flag, p.watchdog, kWdMmaAcc);
                if (!ok) break;
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc_stage * p.bt);
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!__all_sync(0xffffffffu, ready)) {
                        ok = mbar_wait_all(smem_u32(&s_full_tma[stage]), phase, abort_flag, p.watchdog, kWdMmaFull);
                        if (ok && BITS == 4)
                            ok = mbar_wait_all(smem_u32(&s_full_w8[wstage]), wphase, abort_flag, p.watchdog, kWdMmaFull);
                        if (!ok) break;
                    }
                    --left;
                    tc_fence_after();
                    const int s1 = stage + 1 == p.stages ? 0 : stage + 1;
                    const uint32_t ph1 = s1 == 0 ? phase ^ 1u : phase;
                    const int w1 = wstage + 1 == p.stages_w ? 0 : wstage + 1;
                    const uint32_t wph1 = w1 == 0 ? wphase ^ 1u : wphase;
                    const uint32_t peek_bar_a = smem_u32(&s_full_tma[s1]);
                    const uint32_t peek_bar_w = BITS == 4 ? smem_u32(&s_full_w8[w1]) : peek_bar_a;
                    const uint32_t peek_par_w = BITS == 4 ? wph1 : ph1;
                    const uint32_t bar_acc = kb == k_blocks - 1 ? smem_u32(&s_acc_full[acc_stage]) : 0u;
                    uint32_t accumulate = kb != 0 ? 1u : 0u;
                    if (BITS == 4 && ATOMS > 1) {        // all atoms of the stage but the last: four MMAs each, no commit yet
#pragma unroll
                        for (int h = 0; h < ATOMS - 1; ++h) {
                            const uint64_t adesc0 = smem_desc_sw128(smem_a + stage * a_bytes + h * a_atom);
                            const uint64_t bd0[4] = {adesc0, adesc0 + 2, adesc0 + 4, adesc0 + 6};
                            const uint32_t w0 = tmem_base + (uint32_t)(kAccStages * p.bt + wstage * kSlotCols + h * kColsW);
                            const uint32_t at0[4] = {w0, w0 + 8, w0 + 16, w0 + 24};
                            issue_mmas_ts(d_tmem, at0, bd0, idesc, accumulate);
                            accumulate = 1u;
                        }
                    }
                    const uint64_t adesc = smem_desc_sw128(smem_a + stage * a_bytes + (ATOMS - 1) * a_atom);
                    // step 32 bytes along K inside the swizzle atom: +2 in 16-byte address units
                    const uint64_t bd[4] = {adesc, adesc + 2, adesc + 4, adesc + 6};
                    uint32_t r;
                    if (BITS == 4) {
                        // 32 int8 of K = 8 TMEM columns per MMA
                        const uint32_t w_tmem = tmem_base + (uint32_t)(kAccStages * p.bt + wstage * kSlotCols + (ATOMS - 1) * kColsW);
                        const uint32_t at[4] = {w_tmem, w_tmem + 8, w_tmem + 16, w_tmem + 24};
                        r = issue_kblock_ts<CTAS>(0u, d_tmem, at, bd, idesc, accumulate,
                                                  smem_u32(&s_empty[stage]), bar_acc, left > 0 ? 1u : 0u, peek_bar_a, ph1,
                                                  peek_bar_w, peek_par_w);
                    } else {
                        const uint64_t wdesc = smem_desc_sw128(smem_w + stage * w_bytes);
                        const uint64_t ad[4] = {wdesc, wdesc + 2, wdesc + 4, wdesc + 6};
                        r = issue_kblock_ss<CTAS>(0u, d_tmem, ad, bd, idesc, kb != 0 ? 1u : 0u,
                                                  smem_u32(&s_empty[stage]), bar_acc, left > 0 ? 1u : 0u, peek_bar_a, ph1,
                                                  peek_bar_w, peek_par_w);
                    }
                    ready = r != 0;
                    stage = s1;
                    phase = ph1;
                    if (BITS == 4) { wstage = w1; wphase = wph1; }
                }
                if (!ok) break;
                if (++acc_stage == kAccStages) { acc_stage = 0; acc_phase ^= 1u; }
            }
        }
    } else if (warp < 2 + kEpiWarps) {
        // ---------------------------------------------------------------- epilogue
        const int quad = warp & 3;                       // TMEM lanes [32*quad, 32*quad + 32)
        const int half = (warp - 2) >> 2;                // which of the alternating 16-token chunks
        uint8_t* xpose = gen_base + (smem_e - base) + (warp - 2) * kEpiStageBytes;
        const bool staged = p.out.acc == nullptr && p.out.yt == FQ_BF16;
        const float unshift = 1.0f / (float)(1 << p.acc_shift);   // exact power of two
        int acc_stage = 0;
        uint32_t acc_phase = 0;
        [[maybe_unused]] uint32_t epi_phase = 0;
        [[maybe_unused]] int epi_use = 0;
        [[maybe_unused]] int store_use = 0;             // bulk stores issued by this warp so far (buffer = parity)
        bool ok = true;
        for (int unit = unit0; unit < num_units && ok; unit += unit_step) {
            const int tile = tile_of(unit);
            const int64_t jq = (int64_t)n_of(tile) * (kTileN * CTAS) + (int64_t)cta_rank * kTileN + quad * 32;   // first channel of this warp
            const int64_t j = jq + lane;
            const int64_t t0 = (int64_t)m_of(tile) * p.bt;
            const bool j_ok = j < p.N;
            float sw = 0.0f, bj = 0.0f;
            if (j_ok && p.out.acc == nullptr) {
                sw = __ldg(p.w_scale + j) * unshift;     // (float)acc * 2^-shift is exact: fold the shift here
                bj = __ldg(p.bias + j);
            }
            // a tile takes at least ~0.2 us per k-block: sleep through a quarter of that before the first look,
            // so that eight idle warps do not spend issue slots polling while a long tile is being accumulated
            if (k_blocks * ATOMS >= 32) __nanosleep(k_blocks * ATOMS >= 400 ? 20000u : (unsigned)(k_blocks * ATOMS) * 50u);
            ok = mbar_wait_warp_relaxed(smem_u32(&s_acc_full[acc_stage]), acc_phase, abort_flag, p.watchdog, kWdEpilogue);
            if (!ok) break;
            // K split.  Every slice writes its raw int32 sums to its own block of scratch
            // ([tile][slice][bt tokens][128 channels]: a warp's 32 channels of one token are one 128-byte
            // line, coalesced both ways) and then counts itself in; the CTA that counts last adds the other
            // slices to its own accumulator (still in TMEM) and runs the epilogue.  Nobody waits for anybody.
            const int32_t* part = nullptr;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc_stage * p.bt);
            const int slice = unit & (split - 1);
            if (split > 1) {
                tc_fence_after();
                // (in a CTA pair each CTA exchanges and counts its own 128 channels of the tile)
                const int ctile = tile * CTAS + (int)cta_rank;
                int32_t* tile_part = p.partials + (size_t)ctile * (size_t)split * kTileN * (size_t)p.bt + (size_t)(quad * 32 + lane);
                int32_t* mine = tile_part + (size_t)slice * kTileN * (size_t)p.bt;
                for (int c = half * 16; c < p.bt; c += 32) {
                    if (t0 + c >= p.M) break;
                    uint32_t r[16];
                    tmem_ld16(taddr + (uint32_t)c, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) __stcg(mine + (size_t)(c + i) * kTileN, (int)r[i]);
                }
                __threadfence();                 // this slice's sums are visible before it is counted
                // rendezvous 1: every epilogue warp has written and fenced its part
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&s_epi_sync));
                ok = mbar_wait_all(smem_u32(&s_epi_sync), epi_phase, abort_flag, p.watchdog, kWdPartials);
                epi_phase ^= 1u;
                if (!ok) break;
                int* last_slot = &s_last[epi_use & 1];
                if (warp == 2 && lane == 0) {
                    const uint32_t done = atomicAdd(p.counters + ctile, 1u);
                    *last_slot = done == (uint32_t)(split - 1) ? 1 : 0;
                }
                // rendezvous 2: the outcome is written (its slot is reused two tiles later, after both
                // rendezvous of the next tile)
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&s_epi_sync));
                ok = mbar_wait_all(smem_u32(&s_epi_sync), epi_phase, abort_flag, p.watchdog, kWdPartials);
                epi_phase ^= 1u;
                if (!ok) break;
                const bool last = *reinterpret_cast<volatile int*>(last_slot) != 0;
                ++epi_use;
                if (!last) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if (CTAS == 1) mbar_arrive(smem_u32(&s_acc_empty[acc_stage]));
                        else mbar_arrive_cta(smem_u32(&s_acc_empty[acc_stage]), 0);
                    }
                    if (++acc_stage == kAccStages) { acc_stage = 0; acc_phase ^= 1u; }
                    continue;
                }
                __threadfence();                 // the other slices' sums, written through L2
                part = tile_part;
            }
            tc_fence_after();
            if (!SPLIT && staged) {
                // bf16 outputs.  The accumulators are read as MMA-style fragments (a thread: four channels, two adjacent
                // tokens of each 8-token group), scaled in packed pairs, stored token-major into a 1 KB buffer of
                // [16 tokens][32 channels] with two transposing matrix stores, and leave as one tiled bulk store; two
                // buffers alternate so that a chunk is written while the previous one is on its way out.
                const int g = lane >> 2, q = lane & 3;
                float2 sw4[4], bj4[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int64_t ji = jq + g + 8 * i;
                    float swv = 0.0f, bv = 0.0f;
                    if (ji < p.N) { swv = __ldg(p.w_scale + ji) * unshift; bv = __ldg(p.bias + ji); }
                    sw4[i] = make_float2(swv, swv);
                    bj4[i] = make_float2(bv, bv);
                }
                // address of "matrix lane>>3, row lane&7" inside a buffer: token (lane>>4)*8 + (lane&7), 16-byte
                // chunk ((lane>>3)&1) [+2 for channels 16..31], chunk index XORed with (token>>1)&3 (64-byte swizzle)
                const uint32_t tok = (uint32_t)((lane >> 4) * 8 + (lane & 7));
                const uint32_t ch = (uint32_t)((lane >> 3) & 1);
                const uint32_t off_a = tok * 64u + ((ch ^ ((tok >> 1) & 3u)) << 4);
                const uint32_t off_b = tok * 64u + (((ch + 2u) ^ ((tok >> 1) & 3u)) << 4);
                const uint32_t buf0 = smem_e + (uint32_t)(warp - 2) * kEpiStageBytes;
                const bool any_channel = jq < p.N;        // warp-uniform
                // The accumulators and steps of a chunk are requested as soon as the chunk before it has been handed to the
                // copy engine.
                uint32_t na[8], nb[8];
                float2 nd0, nd1;
                auto request = [&](int c) {
                    tmem_ld_16x256b_x2(taddr + (uint32_t)c, na);                    // channels 0..15 of the quadrant
                    tmem_ld_16x256b_x2(taddr + (16u << 16) + (uint32_t)c, nb);      // channels 16..31
                    const int64_t ta = t0 + c + 2 * q, tb = ta + 8;
                    nd0.x = ta < p.M ? __ldg(p.out.a_delta + ta) : 0.0f;
                    nd0.y = ta + 1 < p.M ? __ldg(p.out.a_delta + ta + 1) : 0.0f;
                    nd1.x = tb < p.M ? __ldg(p.out.a_delta + tb) : 0.0f;
                    nd1.y = tb + 1 < p.M ? __ldg(p.out.a_delta + tb + 1) : 0.0f;
                };
                if (t0 + half * 16 < p.M) request(half * 16);
                for (int c = half * 16; c < p.bt; c += 32) {
                    const int64_t tc = t0 + c;
                    if (tc >= p.M) break;                // tokens beyond M: nothing to store (warp-uniform)
                    tmem_ld_wait();
                    uint32_t ra[8], rb[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) { ra[i] = na[i]; rb[i] = nb[i]; }
                    const float2 d0 = nd0, d1 = nd1;
                    const uint32_t buf = buf0 + (uint32_t)(store_use % kEpiBuffers) * 1024u;
                    if (store_use >= kEpiBuffers) {      // the store that last used this buffer has read it
                        if (lane == 0) bulk_wait_read<kEpiBuffers - 1>();
                        __syncwarp();
                    }
                    const uint32_t wa0 = scale_pair_bf16(ra[0], ra[1], d0, sw4[0], bj4[0]);
                    const uint32_t wa1 = scale_pair_bf16(ra[2], ra[3], d0, sw4[1], bj4[1]);
                    const uint32_t wa2 = scale_pair_bf16(ra[4], ra[5], d1, sw4[0], bj4[0]);
                    const uint32_t wa3 = scale_pair_bf16(ra[6], ra[7], d1, sw4[1], bj4[1]);
                    stmatrix_x4_trans(buf + off_a, wa0, wa1, wa2, wa3);
                    const uint32_t wb0 = scale_pair_bf16(rb[0], rb[1], d0, sw4[2], bj4[2]);
                    const uint32_t wb1 = scale_pair_bf16(rb[2], rb[3], d0, sw4[3], bj4[3]);
                    const uint32_t wb2 = scale_pair_bf16(rb[4], rb[5], d1, sw4[2], bj4[2]);
                    const uint32_t wb3 = scale_pair_bf16(rb[6], rb[7], d1, sw4[3], bj4[3]);
                    stmatrix_x4_trans(buf + off_b, wb0, wb1, wb2, wb3);
                    fence_proxy_async_smem();            // the buffer, written through the generic proxy, is read by the copy engine
                    __syncwarp();
                    if (lane == 0 && any_channel) {
                        tma_store_2d(&map_y, (int)jq * 2, (int)tc, buf);   // the output map counts bytes along a row
                        bulk_commit();
                    }
                    ++store_use;
                    // (requested only now: with the next chunk's TMEM loads in flight during the arithmetic above, the
                    // main loop beside this epilogue ran slower -- gate/up 46.5 against 44.9 us)
                    if (c + 32 < p.bt && tc + 32 < p.M) request(c + 32);
                }
                tmem_ld_wait();                          // (nothing outstanding unless the loop broke early)
            } else {
            // K split: the other slices' sums of a chunk are requested one chunk ahead of their use, so that their
            // trip through L2 overlaps the arithmetic and stores of the chunk before.
            [[maybe_unused]] int32_t pv_next[16];
            auto fetch_partials = [&](int c) {
#pragma unroll
                for (int i = 0; i < 16; ++i) pv_next[i] = 0;
                for (int rk = 0; rk < split; ++rk) {
                    if (rk == slice) continue;
                    const int32_t* src = part + ((size_t)rk * (size_t)p.bt + (size_t)c) * kTileN;
#pragma unroll
                    for (int i = 0; i < 16; ++i) pv_next[i] += __ldcg(src + (size_t)i * kTileN);
                }
            };
            if (split > 1 && t0 + half * 16 < p.M) fetch_partials(half * 16);
            for (int c = half * 16; c < p.bt; c += 32) {
                const int64_t tc = t0 + c;
                if (tc >= p.M) break;                    // tokens beyond M: nothing to store (warp-uniform)
                uint32_t r[16];
                tmem_ld16(taddr + (uint32_t)c, r);
                if (split > 1) {
                    int32_t pv[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) pv[i] = pv_next[i];
                    if (c + 32 < p.bt && tc + 32 < p.M) fetch_partials(c + 32);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] += (uint32_t)pv[i];
                }
                if (p.out.acc != nullptr) {
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (tc + i < p.M && j_ok) p.out.acc[(tc + i) * p.N + j] = ((int)r[i]) >> p.acc_shift;
                    continue;
                }
                float d[16];
                if (tc + 16 <= p.M && p.delta_vec) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float4 q = __ldg(reinterpret_cast<const float4*>(p.out.a_delta + tc) + i);
                        d[4 * i + 0] = q.x; d[4 * i + 1] = q.y; d[4 * i + 2] = q.z; d[4 * i + 3] = q.w;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) d[i] = tc + i < p.M ? __ldg(p.out.a_delta + tc + i) : 0.0f;
                }
                tmem_ld_wait();
                if (staged) {
                    // Transpose 32 channels x 16 tokens through shared memory, then 16-byte stores.  Tokens
                    // go in pairs: packed multiply, packed FMA and one two-way bf16 conversion per pair, the
                    // pair's word (token 2k low, token 2k+1 high) stored at [pair k][channel].  A lane then
                    // reads 8 channels of one pair (32 bytes), splits the two tokens with byte permutes and
                    // writes 8 consecutive channels of each token.
                    uint32_t* xw = reinterpret_cast<uint32_t*>(xpose);
                    const float2 sw2 = make_float2(sw, sw), bj2 = make_float2(bj, bj);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const float2 a2 = make_float2((float)(int)r[2 * k], (float)(int)r[2 * k + 1]);
                        const float2 v2 = f2_fma(a2, f2_mul(make_float2(d[2 * k], d[2 * k + 1]), sw2), bj2);
                        uint32_t w;
                        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w) : "f"(v2.y), "f"(v2.x));
                        xw[k * 32 + lane] = w;
                    }
                    __syncwarp();
                    __nv_bfloat16* y = static_cast<__nv_bfloat16*>(p.out.y);
                    {
                        const int k = lane >> 2;
                        const int64_t jj = jq + (lane & 3) * 8;
                        const uint4 q0 = *reinterpret_cast<const uint4*>(xw + k * 32 + (lane & 3) * 8);
                        const uint4 q1 = *reinterpret_cast<const uint4*>(xw + k * 32 + (lane & 3) * 8 + 4);
                        uint4 lo, hi;     // token 2k and token 2k + 1, channels jj .. jj + 7
                        lo.x = __byte_perm(q0.x, q0.y, 0x5410); hi.x = __byte_perm(q0.x, q0.y, 0x7632);
                        lo.y = __byte_perm(q0.z, q0.w, 0x5410); hi.y = __byte_perm(q0.z, q0.w, 0x7632);
                        lo.z = __byte_perm(q1.x, q1.y, 0x5410); hi.z = __byte_perm(q1.x, q1.y, 0x7632);
                        lo.w = __byte_perm(q1.z, q1.w, 0x5410); hi.w = __byte_perm(q1.z, q1.w, 0x7632);
                        if (jj < p.N) {
                            if (tc + 2 * k < p.M) *reinterpret_cast<uint4*>(y + (tc + 2 * k) * p.out.ldy + jj) = lo;
                            if (tc + 2 * k + 1 < p.M) *reinterpret_cast<uint4*>(y + (tc + 2 * k + 1) * p.out.ldy + jj) = hi;
                        }
                    }
                    __syncwarp();
                } else {
                    float* y = static_cast<float*>(p.out.y) + tc * p.out.ldy + j;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float v = fmaf((float)(int)r[i], d[i] * sw, bj);
                        if (tc + i < p.M && j_ok) {
                            if (p.out.yt == FQ_F32)
                                y[i * p.out.ldy] = v;
                            else
                                reinterpret_cast<__nv_bfloat16*>(p.out.y)[(tc + i) * p.out.ldy + j] = __float2bfloat16_rn(v);
                        }
                    }
                }
            }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (CTAS == 1) mbar_arrive(smem_u32(&s_acc_empty[acc_stage]));
                else mbar_arrive_cta(smem_u32(&s_acc_empty[acc_stage]), 0);   // the even CTA issues the MMAs
            }
            if (++acc_stage == kAccStages) { acc_stage = 0; acc_phase ^= 1u; }
        }
        // this warp's stores have read their buffers before the CTA gives up its shared memory (the writes themselves
        // are complete when the grid is: no need to wait for them here, which would add their latency to the tail)
        if (!SPLIT && staged && lane == 0) bulk_wait_read<0>();
    } else if (BITS == 8) {
        // ------------------------------------------------- TMA producer, int8 weights
        // (converged warp, one issuing lane: see the activation producer)
        {
            const int total_kb = my_units * k_blocks;
            bool ok = true;
            int stage = 0, kb = 0, unit = unit0;
            uint32_t phase = 0;
            int n0 = n_of(tile_of(unit)) * (kTileN * CTAS) + (int)cta_rank * kTileN;
            int kb0 = kb0_of(unit);
            bool peek = false;
            for (int n = 0; n < total_kb; ++n) {
                ok = mbar_wait_all_lazy(smem_u32(&s_empty[stage]), phase ^ 1u, abort_flag, p.watchdog, kWdProducer, peek);
                if (!ok) break;
                {
                    const int s1 = stage + 1 == p.stages ? 0 : stage + 1;
                    const uint32_t ph1 = s1 == 0 ? phase ^ 1u : phase;
                    peek = n + 1 < total_kb && mbar_test_wait(smem_u32(&s_empty[s1]), ph1 ^ 1u);
                }
                if (elect_one()) {
                    const uint32_t bar = smem_u32(&s_full_tma[stage]);
                    if (CTAS == 1) {
                        mbar_arrive_expect_tx(bar, w_bytes);
                        tma_load_2d(smem_w + stage * w_bytes, &map_w, (kb0 + kb) * kBlockK, n0, bar);
                    } else {
                        if (leader) mbar_arrive_expect_tx(bar, w_bytes * CTAS);
                        tma_load_2d_pair(smem_w + stage * w_bytes, &map_w, (kb0 + kb) * kBlockK, n0, bar);
                    }
                }
                if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                if (++kb == k_blocks) {
                    kb = 0;
                    unit += unit_step;
                    n0 = n_of(tile_of(unit)) * (kTileN * CTAS) + (int)cta_rank * kTileN;
                    kb0 = kb0_of(unit);
                }
            }
            if (!ok && lane == 0) drain_after_abort();
        }
    } else if (warp < kFirstUnpackWarp + 4 * kUnpackSets) {
        // ------------------------------------------------------------ nibble unpack
        // A thread owns one weight row (= one TMEM lane of its warp's quadrant).  The packed tile is
        // 128 rows x 64 bytes with the 64-byte TMA swizzle: 16-byte chunk c of row r sits at
        // chunk c ^ ((r >> 1) & 3), which makes the row-per-thread reads bank-conflict free.
        const int row = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const int swz = (row >> 1) & 3;
        uint32_t row_off[4];                             // this lane's four 16-byte chunks inside a packed stage
#pragma unroll
        for (int c = 0; c < 4; ++c) row_off[c] = (uint32_t)(row * 64 + ((c ^ swz) << 4));
        // Set `uset` takes the k-blocks whose running index n is congruent to it modulo kUnpackSets,
        // so two k-blocks are in flight per quadrant and one set's store latency hides behind the other.
        const int uset = (warp - kFirstUnpackWarp) >> 2;
        const int total_kb = my_units * k_blocks;
        bool ok = true;
        int ps = uset, ws = uset;                        // ring slots of k-block n, kept incrementally
        uint32_t pph = 0;
        while (ps >= p.stages_p) { ps -= p.stages_p; pph ^= 1u; }
        while (ws >= p.stages_w) ws -= p.stages_w;
        // TMEM slot ws is free once the MMAs of k-block m = n - stages_w have retired, which is the
        // same event that frees that k-block's activation stage: barrier s_empty[m % stages], use
        // number m / stages (stages_w <= stages, so the barrier cannot run a phase ahead of this wait).
        int m = uset - p.stages_w, es = 0;
        uint32_t eph = 0;
        if (m >= 0) es = m;
        while (es >= p.stages) { es -= p.stages; eph ^= 1u; }
        for (int n = uset; n < total_kb && ok; n += kUnpackSets) {
            {
                ok = mbar_wait_all(smem_u32(&s_full_p[ps]), pph, abort_flag, p.watchdog, kWdUnpackFull);
                if (!ok) break;
                const uint32_t src = smem_p + (uint32_t)ps * pk_bytes;     // shared-space address of the stage
                const uint32_t w_tmem = tmem_base + lane_addr + (uint32_t)(kAccStages * p.bt + ws * kSlotCols);
                bool slot_free = false;
#pragma unroll
                for (int h = 0; h < ATOMS; ++h) {
                    uint4 pk[4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) pk[c] = lds128(src + h * pk_atom + row_off[c]);
                    if (h == 0) {
                        // is the TMEM slot free?  (tested now, needed only after the expansion below)
                        slot_free = m < 0 || mbar_test_wait(smem_u32(&s_empty[es]), eph);
                    }
                    uint32_t o[32];                          // 128 codes -> 128 int8 = 32 TMEM columns
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t w[4] = {pk[c].x, pk[c].y, pk[c].z, pk[c].w};
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const uint32_t lo = (w[q] << 4) & 0xF0F0F0F0u;   // even channels, 16*code
                            const uint32_t hi = w[q] & 0xF0F0F0F0u;          // odd channels
                            o[8 * c + 2 * q + 0] = lo;   // same (even, odd) channel order as the int8 activations
                            o[8 * c + 2 * q + 1] = hi;
                        }
                    }
                    if (h == ATOMS - 1) {
                        // The packed stage goes back to its producer behind the expansion that consumed what was loaded
                        // from it, and the barrier's address is formed from one expanded word of each load and a run-time
                        // zero: neither the compiler nor the load/store unit may let the arrival overtake the loads (the
                        // ring is always full, a freed stage is overwritten at once; the weight-streaming kernel, which
                        // released its stages right behind the loads, returned wrong sums once in a thousand launches).
                        const uint32_t dep = (o[0] ^ o[9] ^ o[18] ^ o[27]) & p.zero;
                        __syncwarp();
                        if (elect_one()) mbar_arrive(smem_u32(&s_empty_p[ps]) + dep);
                    }
                    if (h == 0) {
                        ok = mbar_wait_all(smem_u32(&s_empty[es]), eph, abort_flag, p.watchdog, kWdUnpackEmpty, slot_free);
                        if (!ok) break;
                        tc_fence_after();
                    }
                    tmem_st32(w_tmem + h * kColsW, o);
                }
                if (!ok) break;
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (elect_one()) {
                    if (CTAS == 1) mbar_arrive(smem_u32(&s_full_w8[ws]));
                    else mbar_arrive_cta(smem_u32(&s_full_w8[ws]), 0);
                }
                // (every ring has at least kUnpackSets slots: one subtraction brings an index back into range)
                ps += kUnpackSets;
                if (ps >= p.stages_p) { ps -= p.stages_p; pph ^= 1u; }
                ws += kUnpackSets;
                if (ws >= p.stages_w) ws -= p.stages_w;
                m += kUnpackSets;
                if (m >= kUnpackSets) es += kUnpackSets;
                else if (m >= 0) es = m;
                if (es >= p.stages) { es -= p.stages; eph ^= 1u; }
            }
        }
    } else if (BITS == 4) {
        // ------------------------------------------------- TMA producer, packed weights
        {
            const int total_kb = my_units * k_blocks;
            bool ok = true;
            int ps = 0, kb = 0, unit = unit0;
            uint32_t pph = 0;
            int n0 = n_of(tile_of(unit)) * (kTileN * CTAS) + (int)cta_rank * kTileN;
            int kb0 = kb0_of(unit);
            bool peek = false;
            for (int n = 0; n < total_kb; ++n) {
                ok = mbar_wait_all_lazy(smem_u32(&s_empty_p[ps]), pph ^ 1u, abort_flag, p.watchdog, kWdProducer, peek);
                if (!ok) break;
                {
                    const int s1 = ps + 1 == p.stages_p ? 0 : ps + 1;
                    const uint32_t ph1 = s1 == 0 ? pph ^ 1u : pph;
                    peek = n + 1 < total_kb && mbar_test_wait(smem_u32(&s_empty_p[s1]), ph1 ^ 1u);
                }
                if (elect_one()) {
                    const uint32_t bar = smem_u32(&s_full_p[ps]);
                    mbar_arrive_expect_tx(bar, pk_bytes);
#pragma unroll
                    for (int h = 0; h < ATOMS; ++h)
                        tma_load_2d(smem_p + ps * pk_bytes + h * pk_atom, &map_w, ((kb0 + kb) * ATOMS + h) * (kBlockK / 2), n0, bar);
                }
                if (++ps == p.stages_p) { ps = 0; pph ^= 1u; }
                if (++kb == k_blocks) {
                    kb = 0;
                    unit += unit_step;
                    n0 = n_of(tile_of(unit)) * (kTileN * CTAS) + (int)cta_rank * kTileN;
                    kb0 = kb0_of(unit);
                }
            }
            if (!ok && lane == 0) drain_after_abort();
        }
    }

    // ------------------------------------------------------------------ teardown
    tc_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync_all();              // neither CTA leaves while the other may still signal it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<CTAS>(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// ---- host side ---------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// 2-D byte tensor [rows, row_bytes] (row pitch = pitch_bytes, 0 = row_bytes), box [box_rows, box_bytes].
bool encode_2d(CUtensorMap* map, const void* ptr, uint64_t row_bytes, uint64_t rows, uint32_t box_bytes,
               uint32_t box_rows, CUtensorMapSwizzle swizzle, uint64_t pitch_bytes = 0) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {row_bytes, rows};
    const cuuint64_t strides[1] = {pitch_bytes ? pitch_bytes : row_bytes};
    const cuuint32_t box[2] = {box_bytes, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool encode_tiled(CUtensorMap* map, CUtensorMapDataType dt, uint32_t rank, const void* ptr, const uint64_t* dims,
                  const uint64_t* strides_bytes, const uint32_t* box, bool swizzle128) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t d[5], st[5];
    cuuint32_t b[5], es[5];
    for (uint32_t i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = 1; }
    for (uint32_t i = 0; i + 1 < rank; ++i) st[i] = strides_bytes[i];
    return fn(map, dt, rank, const_cast<void*>(ptr), d, st, b, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

int next_pow2(int v) {
    int r = 32;
    while (r < v) r <<= 1;
    return r;
}

}  // namespace

fq_status build_weight_tmap(Weights& W) {
    W.tmap_valid = false;
    if (W.N == 0) return FQ_OK;
    const bool ok = W.bits == 4
                        ? encode_2d(&W.tmap, W.codes, (uint64_t)W.K / 2, (uint64_t)W.N, kBlockK / 2, kTileN,
                                    CU_TENSOR_MAP_SWIZZLE_64B)
                        : encode_2d(&W.tmap, W.codes, (uint64_t)W.K, (uint64_t)W.N, kBlockK, kTileN,
                                    CU_TENSOR_MAP_SWIZZLE_128B);
    if (!ok) return FQ_ERR_CUDA;
    W.tmap_valid = true;
    build_stream_tmap(W);       // optional second view (short batches); shapes it does not fit go without
    return FQ_OK;
}

namespace {

template <int BITS, int CTAS, bool SPLIT, int ATOMS = 1>
fq_status launch_variant(const CUtensorMap& map_a, const CUtensorMap& map_w, const CUtensorMap& map_y, const Params& p,
                         int grid, size_t smem, int cluster, cudaStream_t stream) {
    auto kern = gemm_tcgen05_kernel<BITS, CTAS, SPLIT, ATOMS>;
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem) != cudaSuccess) return FQ_ERR_CUDA;
    return launch_pdl(kern, (unsigned)grid, (unsigned)(BITS == 4 ? kThreadsW4 : kThreadsW8), smem, stream, (unsigned)cluster,
                      map_a, map_w, map_y, p) == cudaSuccess ? FQ_OK : FQ_ERR_CUDA;
}

}  // namespace

namespace {

struct Plan {
    int bt = 0;       // tokens per tile
    int ctas = 1;     // 2: CTA pairs on 256-channel tiles (cta_group::2)
    int split = 1;    // >1: every tile is that many work units, each on a slice of K
    size_t scratch = 0;   // bytes of scratch the split needs: the tile counters, then the int32 partial tiles
};

// Token tile, CTA grouping and K split.  Upper bound of the tile from TMEM: two accumulator stages,
// plus the unpacked-weight ring for 4-bit weights (2*bt + 3*32 <= 512 columns).  M is split evenly
// over m_tiles so that ragged M wastes little.  Candidates are ranked by a cost model fitted to
// measured launches (cycles): rounds of work units over the SMs, each unit costing
//     k_blocks * per_kblock(bt) + 16*bt + 1000          (the tail: epilogue and tile hand-over)
//   4-bit weights:          per_kblock = 330 + bt       (issue floor, then the MMAs' 2*bt); 235 + bt for tiles of at
//                                        most 128 tokens, whose stages hold two k-blocks
//   8-bit, one CTA:         per_kblock = max(350 + 0.8*bt, 230 + 2*bt)   (issue floor, then shared memory:
//                                        both operands pass through it)
//   8-bit, CTA pair:        per_kblock = max(545, 2.62*bt)   (each CTA stages half of the token tile)
// Pairs gain nothing for 4-bit weights, which never pass through shared memory unpacked.
// K split (single CTAs, and CTA pairs on 8-bit weights): problems with fewer tiles than SMs and a long K (every short batch; down_proj
// at M = 816: 64 tiles of 128 k-blocks) make `split` work units of every tile, each on a slice of K; the
// slices leave int32 partial sums in scratch and the one that finishes last adds them up.  Fitted cost per
// unit: 12500 + 40*bt cycles, plus 1500 per extra slice -- the constant is what a split costs a call on operands
// from HBM whatever its size (the node that clears the counters ahead of the prologue, two rendezvous, the
// round trips of the exchange: 16-25 thousand cycles measured at tiles of 16 and 64 tokens split in 2, 4 and 8,
// where an earlier model of 1500 + 70*bt chose splits that ran 15-45 % slower than the same tile unsplit).
Plan plan_gemm(int64_t M, int64_t N, int64_t K, int bits, int sms, size_t scratch_avail) {
    const int bt_max = bits == 4 ? 208 : 256;
    const int64_t kb = (K + kBlockK - 1) / kBlockK;
    Plan best;
    double best_cost = 0.0;
    for (int c = 1; c <= ((bits == 8 && N > kTileN) ? 2 : 1); ++c) {
        const int64_t n_units = (N + kTileN * c - 1) / (kTileN * c);
        for (int mt = (int)((M + bt_max - 1) / bt_max); mt <= (int)((M + 63) / 64); ++mt) {
            int b = (int)(((M + mt - 1) / mt + 15) / 16 * 16);
            if (b > bt_max) continue;
            // 4-bit weights, token tiles of 32..64 (four-atom stages): kept to the envelope in which that configuration
            // has run clean under CUDA-graph replay -- at most 64 work units and K <= 4096.  Beyond it (M = 64 at
            // K = N = 8192 and 16384 ended two benchmark runs with a launch failure whose cause reading has not shown)
            // the batch is padded to a 128-token tile with two-atom stages: the configuration every mid-size batch runs
            // (it may split K like any other: 32 tiles of 128 k-blocks are better off as 128 units).
            if (bits == 4 && b > 16 && b <= 64 && (n_units * ((M + b - 1) / b) > 64 || kb > 32)) {
                b = 128;
            }
            const int64_t units = n_units * ((M + b - 1) / b);
            const double w8_single = 350.0 + 0.8 * b > 230.0 + 2.0 * b ? 350.0 + 0.8 * b : 230.0 + 2.0 * b;
            // 4-bit, tiles of at most 128 tokens: two-atom stages (see the kernel) cost less per 128 channels
            const double w4 = (c == 1 && b <= 128 && K % kBlockK == 0) ? 235.0 + b : 330.0 + b;
            const double per_kb = bits == 4 ? w4 : (c == 1 ? w8_single : (2.62 * b > 545.0 ? 2.62 * b : 545.0));
            for (int sp = 1; sp <= ((c == 1 || bits == 8) ? kMaxSplit : 1); sp *= 2) {
                if (sp > 1 && (kb % sp != 0 || kb / sp < 2 || units * c > kMaxSplitTiles || units * c * sp > 4 * (int64_t)sms)) continue;
                const int64_t kb_per = kb / sp;
                const size_t scratch = sp > 1 ? kCounterBytes + (size_t)units * c * sp * kTileN * b * sizeof(int32_t) : 0;
                if (scratch > scratch_avail) continue;
                const int slots = sms / c;
                const double unit_cost = (double)kb_per * per_kb + 16.0 * b + 1000.0 + (sp > 1 ? 12500.0 + 40.0 * b + 1500.0 * (sp - 1) : 0.0);
                const double cost = (double)((units * sp + slots - 1) / slots) * unit_cost;
                if (best.bt == 0 || cost < best_cost * 0.98) {   // ties: the earlier candidate (larger tile, no split)
                    best.bt = b; best.ctas = c; best.split = sp; best.scratch = scratch;
                    best_cost = cost;
                }
            }
        }
    }
    return best;
}

}  // namespace

// A launch that splits K counts the finished slices of every tile in counters at the head of the scratch.
// They are cleared here, by a memset node enqueued AHEAD of the call's first kernel (between the prologue
// and the GEMM it would break the programmatic overlap of the two): each call starts from zero whatever an
// earlier call -- even one that gave up on an expired wait -- left there, and nothing in the weight handle
// changes at run time.
fq_status gemm_prepare(int64_t M, const Weights& W, void* scratch, size_t scratch_bytes, cudaStream_t stream) {
    if (M <= 0 || W.N == 0 || scratch == nullptr || gemm_stream_applies(M, W)) return FQ_OK;
    const Plan plan = plan_gemm(M, W.N, W.K, W.bits, device_sm_count(), scratch_bytes);
    if (plan.split <= 1) return FQ_OK;
    return cudaMemsetAsync(scratch, 0, kCounterBytes, stream) == cudaSuccess ? FQ_OK : FQ_ERR_CUDA;
}

fq_status launch_gemm(const int8_t* a8, int64_t M, const Weights& W, int acc_shift, const GemmOut& out, void* scratch,
                      size_t scratch_bytes, cudaStream_t stream) {
    if (M == 0 || W.N == 0) return FQ_OK;
    if (gemm_stream_applies(M, W))
        return launch_gemm_stream(a8, M, W, acc_shift, out, stream) == cudaSuccess ? FQ_OK : FQ_ERR_CUDA;
    return launch_gemm_tcgen05(a8, M, W, acc_shift, out, scratch, scratch_bytes, stream);
}

size_t gemm_scratch_bytes(int64_t M, int64_t N, int64_t K, int bits) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    return plan_gemm(M, N, K, bits, device_sm_count(), (size_t)-1).scratch;
}

fq_status launch_gemm_tcgen05(const int8_t* a8, int64_t M, const Weights& W, int acc_shift, const GemmOut& out,
                              void* scratch, size_t scratch_bytes, cudaStream_t stream) {
    if (M == 0 || W.N == 0) return FQ_OK;
    if (!W.tmap_valid) return FQ_ERR_CUDA;

    Params p{};
    p.M = M; p.N = W.N; p.K = W.K;
    const int sms = device_sm_count();
    const Plan plan = plan_gemm(M, W.N, W.K, W.bits, sms, scratch ? scratch_bytes : 0);
    const int bt = plan.bt, ctas = plan.ctas, split = plan.split;
    p.split = split;
    p.counters = static_cast<uint32_t*>(scratch);            // cleared by gemm_prepare()
    p.partials = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(scratch) + kCounterBytes);
    p.delta_vec = (reinterpret_cast<uintptr_t>(out.a_delta) & 15u) == 0 ? 1 : 0;
    p.bt = bt;
    p.m_tiles = (int)((M + bt - 1) / bt);
    p.n_tiles = (int)((W.N + kTileN * ctas - 1) / (kTileN * ctas));
    // Bands of 8 token tiles once the batch is long enough for the order to matter: a wave of 148 CTAs (74 pairs)
    // then covers 8 token tiles x 18 (9) channel tiles, close to the square that minimises the bytes it shares.
    p.band = p.m_tiles >= 16 ? 8 : p.m_tiles;
    p.acc_shift = acc_shift;
    p.w_scale = W.w_scale;
    p.bias = W.bias;
    p.out = out;
    p.watchdog = watchdog_device_ptr();
    if (!p.watchdog) return FQ_ERR_CUDA;
    // 4-bit weights, single CTAs, token tiles of at most 128: two 128-channel atoms per pipeline stage (the
    // accumulators of longer tiles leave no room for TMEM slots twice as wide).  Needs whole atoms (K a multiple
    // of 128) and, with a K split, slices of whole stages.
    const int64_t kb128 = (W.K + kBlockK - 1) / kBlockK;
    int atoms = (W.bits == 4 && ctas == 1 && bt <= 128 && W.K % kBlockK == 0 && (split == 1 || kb128 % (2 * split) == 0)) ? 2 : 1;
    if (atoms == 2 && bt <= 64 && kb128 >= 4 * split && (split == 1 || kb128 % (4 * split) == 0)) atoms = 4;   // four for the shortest tiles
    // 4-bit weights: every TMEM column the accumulators leave free becomes unpacked-weight ring
    int stages_w = W.bits == 4 ? (512 - kAccStages * bt) / (kColsW * atoms) : 0;
    if (stages_w > kMaxStagesW) stages_w = kMaxStagesW;
    p.tmem_cols = next_pow2(kAccStages * bt + stages_w * kColsW * atoms);

    const size_t epi_bytes = (size_t)kEpiWarps * kEpiStageBytes;
    const size_t budget = 227 * 1024 - 1024 /*alignment slack*/ - 1024 /*static*/ - epi_bytes;
    const size_t a_bytes = (size_t)(bt / ctas) * kBlockK * atoms, w_bytes = (size_t)kTileN * kBlockK,
                 pk_bytes = w_bytes / 2 * atoms;
    size_t smem;
    if (W.bits == 4) {
        p.stages_w = stages_w;
        // Both TMA rings need the same look-ahead in k-blocks (their latencies are the same):
        // split the budget evenly, then give the remainder to the cheaper packed ring.
        int sa = (int)(budget / (a_bytes + pk_bytes));
        if (sa > kMaxStages) sa = kMaxStages;
        if (sa < 2) return FQ_ERR_UNSUPPORTED;
        int sp = (int)((budget - sa * a_bytes) / pk_bytes);
        if (sp > kMaxStagesP) sp = kMaxStagesP;
        if (stages_w > sa) {            // the unpack warps wait on the activation ring's barriers
            stages_w = sa;
            p.stages_w = sa;
        }
        p.stages = sa;
        p.stages_p = sp;
        smem = sa * a_bytes + sp * pk_bytes + epi_bytes + 1024;
    } else {
        int stages = (int)(budget / (a_bytes + w_bytes));
        if (stages > kMaxStages) stages = kMaxStages;
        if (stages < 2) return FQ_ERR_UNSUPPORTED;
        p.stages = stages;
        p.stages_p = 0;
        p.stages_w = 0;
        smem = (a_bytes + w_bytes) * stages + epi_bytes + 1024;
    }

    // each CTA of a pair loads its own half of the token tile
    CUtensorMap map_a;
    if (!encode_2d(&map_a, a8, (uint64_t)W.K, (uint64_t)M, kBlockK, (uint32_t)(bt / ctas), CU_TENSOR_MAP_SWIZZLE_128B))
        return FQ_ERR_CUDA;

    // bf16 outputs of an unsplit launch leave through tiled bulk stores of [16 tokens x 32 channels] (64-byte rows,
    // 64-byte swizzle in shared memory); the copy engine clips what lies beyond M tokens or N channels
    CUtensorMap map_y;
    memset(&map_y, 0, sizeof(map_y));
    if (out.acc == nullptr && out.yt == FQ_BF16 && split == 1 &&
        !encode_2d(&map_y, out.y, (uint64_t)W.N * 2, (uint64_t)M, 64, 16, CU_TENSOR_MAP_SWIZZLE_64B, (uint64_t)out.ldy * 2))
        return FQ_ERR_CUDA;

    const int num_units = p.m_tiles * p.n_tiles * split;       // a K split makes `split` units of every tile
    const int max_units = sms / ctas;
    const int clusters = num_units < max_units ? num_units : max_units;
    const int grid = clusters * ctas;
    p.cluster_shift = ctas == 2 ? 1 : 0;
    p.unit_step = clusters;
    p.units_q = num_units / clusters;
    p.units_rem = num_units % clusters;
    p.kb_per = (int)((kb128 + atoms - 1) / atoms) / split;      // stages per unit; the planner only picks splits that divide it
    p.split_shift = split == 1 ? 0 : (split == 2 ? 1 : (split == 4 ? 2 : (split == 8 ? 3 : 4)));

    if (W.bits == 4) {
        if (ctas == 2) return launch_variant<4, 2, false>(map_a, W.tmap, map_y, p, grid, smem, 2, stream);
        if (atoms == 4)
            return split > 1 ? launch_variant<4, 1, true, 4>(map_a, W.tmap, map_y, p, grid, smem, 1, stream)
                             : launch_variant<4, 1, false, 4>(map_a, W.tmap, map_y, p, grid, smem, 1, stream);
        if (atoms == 2)
            return split > 1 ? launch_variant<4, 1, true, 2>(map_a, W.tmap, map_y, p, grid, smem, 1, stream)
                             : launch_variant<4, 1, false, 2>(map_a, W.tmap, map_y, p, grid, smem, 1, stream);
        return split > 1 ? launch_variant<4, 1, true>(map_a, W.tmap, map_y, p, grid, smem, 1, stream)
                         : launch_variant<4, 1, false>(map_a, W.tmap, map_y, p, grid, smem, 1, stream);
    }
    if (ctas == 2)
        return split > 1 ? launch_variant<8, 2, true>(map_a, W.tmap, map_y, p, grid, smem, 2, stream)
                         : launch_variant<8, 2, false>(map_a, W.tmap, map_y, p, grid, smem, 2, stream);
    return split > 1 ? launch_variant<8, 1, true>(map_a, W.tmap, map_y, p, grid, smem, 1, stream)
                     : launch_variant<8, 1, false>(map_a, W.tmap, map_y, p, grid, smem, 1, stream);
}

}  // namespace fq
