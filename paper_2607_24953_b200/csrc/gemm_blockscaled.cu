// Block-scaled tcgen05 GEMMs for sm_100a: C[M,N] = A[M,K] * B[N,K]^T with both operands
// contraction-contiguous ("K-major"), FP32 accumulation in tensor memory.
//
//   kind::mxf4      E2M1 payload, 2 codes per byte, one UE8M0 scale per 32x32 block of the source tensor
//                   (the 2D-block format): the hardware's per-row, per-32-element scale for row r and
//                   contraction block kb is scale[r/32][kb] or, for a transposed view, scale[kb][r/32].
//   kind::mxf8f6f4  E4M3 payload, one UE8M0 scale per row and 32 contraction elements (MXFP8).
//
// Persistent kernel, one CTA per SM, 12 warps.  Dense FP4 products run as clusters of two CTAs that share a 256x256
// tile through cta_group::2 MMAs (each CTA holds 128 rows of the accumulator, loads its own 128 A rows and half of
// the B rows); grouped products and MXFP8 use one CTA per 128x256 tile.
//   warp 0      TMA producer: per stage the A tile (128 rows x 128 B) and the B tile (256 or 128 rows x 128 B),
//               128B swizzle; polls all free slots first, then issues their loads back to back
//   warp 1      MMA issuer: stays converged, one elected lane issues per stage 6 tcgen05.cp (scale images -> TMEM),
//               4 tcgen05.mma and the tcgen05.commit that frees the slot; it never reads shared memory in the loop
//   warp 2      watcher: polls the slots' "full" barriers (several at a time), the scale images and the
//               accumulator's "empty" barrier and meets the MMA warp at a named barrier per stage
//   warp 3      scale image builder: per unit of 16 (FP4) or 8 (MXFP8) stages gathers the scale bytes and writes the
//               images tcgen05.cp reads in place (double-buffered); 2D-block scales as replicated 8-row images,
//               per-row scales as real 32-row images
//   warps 4-11  epilogue: tcgen05.ld of the 128x256 FP32 accumulator (each warp 32 lanes x 128 columns),
//               release of the accumulator as soon as it sits in registers, then convert and store (pair kernel:
//               through staging rows and TMA stores; one CTA: 256-bit stores)
// A ring of four (one CTA: 48 KB of operands per stage) or five (pair: 32 KB) shared-memory stages is guarded by
// mbarriers; the scale columns in TMEM form a ring of the same depth.  Every mbarrier wait is bounded: when a limit
// is hit the CTA records FP4Q_ERR_TIMEOUT in the workspace, releases the MMA warp from its named barriers, stops
// issuing work and leaves through the normal exit (TMEM is freed).
#include <cstdlib>
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "quant_device.cuh"

namespace fp4q {

constexpr int BM = 128, BN = 256;            // per-CTA accumulator: 128 rows x 256 columns (a CTA pair covers 256 x 256)
constexpr int kMaxStages = 6;
constexpr int kAStageBytes = BM * 128;
constexpr int kMaxGroupsShared = 1023;       // grouped contraction: boundaries kept in shared memory up to this many groups
constexpr int kMaxRowTilesShared = 2048;     // grouped rows: group of each 128-row tile kept in shared memory up to this many tiles
constexpr int kSmemTail = 512;               // barriers, TMEM base, abort flag, scale scratch (one per loader warp)
// 2D-block scales: the scale images of a whole unit (up to 16 stages = 4096 contraction elements of one tile) are
// built once, ahead of time, and tcgen05.cp reads them in place.  Per 128-element chunk the compact form is one
// 16-byte row for A [row tile 0..3][block 0..3] and two for B (row tiles 0..3, 4..7); an image is such a row
// replicated over the 8 rows of one core matrix (128 B), which a descriptor with a zero stride between 8-row
// groups presents as the 32 identical rows tcgen05.cp.32x128b expects.  Per stage: 6 images = 768 B.
constexpr int kCacheChunks = 32;             // chunks per unit
constexpr int kUnitStagesMxf4 = kCacheChunks / 2;
// Per-row scales (MXFP8): a stage covers 4 contraction blocks; its three images (A rows, B rows 0..127, B rows
// 128..255) are real 32-row x 16-byte images (512 B each), row l holding rows l, l+32, l+64, l+96 of the operand.
// A unit is 8 stages, so that a buffer has the same size as for 2D-block scales.
constexpr int kUnitStagesMxf8 = 8;
constexpr int kImageStageBytesMxf8 = 1536;
constexpr int kCompactBytes = kCacheChunks * 48;
constexpr int kImageStageBytes = 768;        // A chunk 0, A chunk 1, B chunk 0 (rows 0..127, 128..255), B chunk 1 (same)
constexpr int kCacheBufBytes = kUnitStagesMxf4 * kImageStageBytes;
static_assert(kUnitStagesMxf8 * kImageStageBytesMxf8 == kCacheBufBytes, "both kinds share the image buffers");
// mxf4 with per-row scales: a stage has two chunks of four blocks; A 2 x 512 B, B (256 rows) 4 x 512 B per stage
constexpr int kUnitStagesMxf4R = 4;
constexpr int kImageStageBytesMxf4R = 3072;
static_assert(kUnitStagesMxf4R * kImageStageBytesMxf4R == kCacheBufBytes, "all kinds share the image buffers");
// mxf4nvf4 with 16-element scale vectors (tensors quantized in 16 x 16 blocks): every MMA (64 contraction elements)
// has its own image per 128 operand rows - four scale bytes per row - so a stage holds A 4 x 512 B and B 8 x 512 B
constexpr int kUnitStagesMxf4B16 = 2;
constexpr int kImageStageBytesMxf4B16 = 6144;
static_assert(kUnitStagesMxf4B16 * kImageStageBytesMxf4B16 == kCacheBufBytes, "all kinds share the image buffers");
// Epilogue staging of the pair kernel: each of the 8 epilogue warps owns 32 rows x 128 bytes, written from registers
// (128-byte swizzle: the 16-byte pieces of 8 rows fall into different banks) and drained by a TMA store, which keeps
// the output off the load/store unit that the MMA warp's instructions also pass through.
constexpr int kStagingWarpBytes = 32 * 128;

// CTAS = 1: one CTA per 128x256 tile, it loads all 256 B rows.  CTAS = 2: a cluster of two CTAs shares a 256x256
// tile through cta_group::2 MMAs; each CTA loads its own 128 A rows and half of the B rows, which halves the
// B-operand shared-memory and L2 traffic per CTA and leaves room for two more ring stages.
// KIND_MXF4: FP4 payloads, 2D-block scales on both operands (replicated scale images).  KIND_MXF8: E4M3 payloads,
// per-row scales.  KIND_MXF4R: FP4 payloads with per-row scale images - an operand quantized in 1D blocks (the
// paper's activation layout) next to a 2D-block operand, whose tile scale is then expanded to its 32 rows.
// KIND_MXF4B16: FP4 payloads of tensors quantized in 16 x 16 blocks (block-size study): 16-element scale vectors
// (kind::mxf4nvf4, scale_vec::4X, UE8M0 scales), real images built like the per-row kinds' (row_shift 4).
enum { KIND_MXF4 = 0, KIND_MXF8 = 1, KIND_MXF4R = 2, KIND_MXF4B16 = 3 };
__host__ __device__ constexpr bool kind_fp4(int kind) { return kind != KIND_MXF8; }

// Per-row scale images are rebuilt every 4 (FP4) or 8 (MXFP8) stages from 12 KB of scale bytes, whose global-memory
// latency under the operand traffic (about 3000 cycles) exceeds the time such a unit runs.  The kernels for those
// kinds therefore fetch the bytes two units ahead with cp.async into raw buffers (no registers are held meanwhile)
// and pay for the buffers with one ring stage; the pair kernel also keeps a third image buffer, because the way
// from "the MMAs have finished with a buffer" to "the leader may copy the next unit out of it" (commit to both
// CTAs, build, report to the leader) is longer than one unit as well.
template <int KIND, int CTAS>
struct Cfg {
    static constexpr bool kRowImages = KIND != KIND_MXF4;
    static constexpr int kImageBufs = (CTAS == 2 && kRowImages) ? 3 : 2;
    static constexpr int kRawBufs = kRowImages ? 2 : 0;
    // The output leaves through staging rows and TMA stores wherever shared memory allows (everything but the
    // one-CTA kernel of the per-row kinds).  In the one-CTA kernel of the 2D kind - grouped products with short
    // contractions - plain stores of the 64 KB tile filled the SM's path to L2 and the TMA loads issued meanwhile
    // took 6500-8000 cycles instead of 3000; the staging costs that kernel its fourth ring stage.
    static constexpr bool kTmaStores = CTAS == 2 || !kRowImages;
    // One-CTA kernel of the 2D kind (grouped products): its 48 KB stages keep the TMA unit busy ~740 of every ~800 cycles,
    // so a producer that also polls (a poll queues behind the loads the same warp has just issued) leaves gaps.  There
    // the producer is split: warp 2 waits for free slots and arms their barriers, warp 0 only issues loads; the MMA warp
    // waits on its barriers itself (measured: MoE expert layer 1.95 -> 2.07 PFLOP/s; no gain for the pair kernel).
    static constexpr bool kSplitProducer = KIND == KIND_MXF4 && CTAS == 1;
    static constexpr int kStages = (CTAS == 2 ? 5 : (kTmaStores ? 3 : 4)) - (kRowImages ? 1 : 0);
    static constexpr int kSmemCache = kCompactBytes + (kImageBufs + kRawBufs) * kCacheBufBytes;
    static constexpr int kBRows = CTAS == 2 ? 128 : 256;
    static constexpr int kBStageBytes = kBRows * 128;
    static constexpr int kSmemOperands = kStages * (kAStageBytes + kBStageBytes);
    static constexpr int kSmemScales = (kSmemCache + 1023) / 1024 * 1024;
    static constexpr int kSmemStaging = kTmaStores ? 8 * kStagingWarpBytes : 0;
    static constexpr int kSmemGroups = (CTAS == 1 || KIND == KIND_MXF4) ? (kMaxGroupsShared + 1) * 4 : 0;   // grouped products: group table
    static_assert(kSmemGroups == 0 || kSmemGroups >= kMaxRowTilesShared * 2, "group table");
    static constexpr int kSmemBytes = 1024 + kSmemOperands + kSmemScales + kSmemStaging + kSmemTail + kSmemGroups;
    static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
};
constexpr int kRasterM = 16;                 // dense products: row tiles per rasterisation group
constexpr int kThreads = 384;
constexpr int kTmemCols = 512;
constexpr int kTmemSfBase = 256;
// scale columns per ring stage: SFA at +0 (+4 per chunk), SFB at +8 (+8 per chunk); with 16-element scale vectors
// SFA at +0 (+4 per MMA), SFB at +16 (+8 per MMA)
template <int KIND> struct SfCols { static constexpr int kStride = KIND == KIND_MXF4B16 ? 48 : 32; };
static_assert(kTmemSfBase + 5 * SfCols<KIND_MXF4>::kStride <= kTmemCols && kTmemSfBase + 4 * SfCols<KIND_MXF4B16>::kStride <= kTmemCols,
              "tensor memory budget: 256 accumulator columns + one scale slot per ring stage");
constexpr uint32_t kWaitLimit = 1u << 22;       // default number of polls after which a wait gives up (workspace word 2 overrides it)
constexpr int kRelaxedNs = 64, kLazyNs = 256;   // back-off between polls of roles with slack
// Developer diagnostic (off by default): -DFP4Q_TRACE makes CTA 0 add up clock64() intervals of its roles in
// registers and leave them in the workspace's padding words (status[16 + 2*slot], 64-bit each).
#ifdef FP4Q_TRACE
#define TRACE_DECL(n) long long n = 0
#define TRACE_T0(t) long long t = clock64()
#define TRACE_ADD(acc, t) do { long long t_now = clock64(); acc += t_now - t; t = t_now; } while (0)
#define TRACE_OUT(p, slot, v) do { if (blockIdx.x == 0) reinterpret_cast<long long *>(p.status + 16)[slot] = (v); } while (0)
#ifdef FP4Q_TRACE_EVENTS
__device__ long long g_trace_events[2][8][512][2];   // [CTA 0/1][kind][stream index][clock64, globaltimer]
#define TRACE_EV(kind, idx) do { if (blockIdx.x < 2 && (idx) < 512) { long long gt; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt)); \
    g_trace_events[blockIdx.x][kind][idx][0] = clock64(); g_trace_events[blockIdx.x][kind][idx][1] = gt; } } while (0)
extern "C" int fp4q_debug_events(void *host) { return (int)cudaMemcpyFromSymbol(host, g_trace_events, sizeof(g_trace_events)); }
#else
#define TRACE_EV(kind, idx)
#endif
#else
#define TRACE_EV(kind, idx)
#define TRACE_DECL(n)
#define TRACE_T0(t)
#define TRACE_ADD(acc, t)
#define TRACE_OUT(p, slot, v)
#endif
constexpr uint8_t kScalePad = 127;           // UE8M0 code of 1.0 for scale slots beyond the tensor (their payload is 0)

enum { MODE_DENSE = 0, MODE_GROUPED_ROWS = 1, MODE_GROUPED_K = 2 };

struct ScaleView {
    const uint8_t *ptr;
    int64_t stride_row;   // mxf4: bytes between consecutive 32-row tiles; mxf8: bytes between consecutive rows
    int64_t stride_kb;    // bytes between consecutive contraction blocks of 32
    int32_t n_row;        // mxf4: number of row tiles; mxf8: number of rows
    int32_t n_kb;         // number of contraction blocks
    int32_t row_shift;    // per-row images only: operand row r reads scale row r >> row_shift (5: a 2D-block operand, n_row counts tiles)
};

struct GemmParams {
    ScaleView sfa, sfb;
    void *C;
    int64_t ldc;
    int32_t M, N, K;                 // per-problem output rows, output columns, contraction length (elements)
    int32_t m_tiles, n_tiles, n_tile_total;   // m_tiles counts rows of 128 * ctas
    int32_t ctas;                    // CTAs per tile (1, or 2 for cta_group::2 pairs)
    int32_t raster_m;                // tile order: groups of raster_m row tiles, within a group row tile fastest
    int32_t out_f32, accumulate;
    int32_t wide_stores;             // output base and row pitch are 32-byte aligned: 256-bit stores (whole sectors)
    int32_t mode, n_groups;
    int32_t rows_pair_aligned;       // grouped rows: every group starts on a multiple of 256 rows (caller's statement)
    const int64_t *row_offsets;
    int32_t b_rows_per_group;        // grouped rows: B row offset per group (forward)
    int32_t b_k_per_group;           // grouped rows: B contraction offset per group (dgrad)
    uint32_t *status;
    // quantizing epilogue (EPI_QUANT): the output leaves as a 2D-block FP4 tensor instead of BF16/FP32
    uint8_t *q_rm, *q_t, *q_scale;
    int64_t q_ld_rm, q_ld_t, q_ld_s;
    int32_t q_mode;                  // FP4Q_ROUND_NEAREST or FP4Q_ROUND_STOCHASTIC
    uint32_t q_tensor_id;
    PhiloxRoundKeys q_keys;
};

enum { EPI_STORE = 0, EPI_QUANT = 1 };

struct Tile {
    int32_t a_row0, b_row0, b_load_row0, a_k0, b_k0, k_len, c_row0, c_col0, m_valid, n_valid;
};

// ---------------------------------------------------------------------------------------- PTX helpers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Non-blocking probe of a barrier phase (the try_wait form may suspend the thread for a while).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// One lane of a converged warp.
__device__ __forceinline__ bool elect_one()
{
    uint32_t p;
    asm volatile("{\n .reg .pred P;\n elect.sync _|P, 0xFFFFFFFF;\n selp.b32 %0, 1, 0, P;\n}" : "=r"(p));
    return p != 0;
}
// Named barrier on which the MMA warp and the warp that watches a ring slot for it meet (64 threads).  Both sides
// use the waiting form: with a non-waiting arrival a watcher that releases stages unseen (after a timeout) could
// complete a barrier phase on its own and leave the MMA warp without a partner.
__device__ __forceinline__ void named_sync(uint32_t id) { asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory"); }

// Bounded wait.  Returns false when the limit ran out (the timeout is then recorded) or when another
// role of this CTA has already given up.  Every poll of an mbarrier is a shared-memory transaction that
// competes with the tensor core's operand reads and with the MMA thread's own waits, so roles that have
// slack (everything but the MMA issuer) sleep between polls.
template <int BACKOFF_NS, bool PROBE = false>
__device__ __forceinline__ bool mbar_wait_impl(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *status,
                                               uint64_t limit, uint32_t where)
{
    for (uint64_t it = 0; it < limit; it++) {
        if (PROBE ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity)) return true;
        if (BACKOFF_NS > 0) __nanosleep(BACKOFF_NS);
        if (((uint32_t)it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1u;
    if (atomicCAS(status, 0u, (uint32_t)FP4Q_ERR_TIMEOUT) == 0u) status[1] = where;
    return false;
}
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *status, uint64_t limit,
                                       uint32_t where)
{
    return mbar_wait_impl<0>(bar, parity, abort_flag, status, limit, where);
}
__device__ __noinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *status,
                                               uint64_t limit, uint32_t where)
{
    return mbar_wait_impl<kRelaxedNs>(bar, parity, abort_flag, status, limit, where);
}
__device__ __noinline__ bool mbar_wait_lazy(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *status,
                                            uint64_t limit, uint32_t where)
{
    return mbar_wait_impl<kLazyNs>(bar, parity, abort_flag, status, limit, where);
}
// For barriers that another CTA of the cluster completes (a multicast tcgen05.commit): probe instead of try_wait,
// whose suspended thread is not reliably woken early by a remote arrival.
__device__ __noinline__ bool mbar_poll(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *status, uint64_t limit,
                                       uint32_t where)
{
    return mbar_wait_impl<0, true>(bar, parity, abort_flag, status, limit, where);
}
__device__ __noinline__ bool mbar_poll_relaxed(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *status,
                                               uint64_t limit, uint32_t where)
{
    return mbar_wait_impl<kRelaxedNs, true>(bar, parity, abort_flag, status, limit, where);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// The same load issued by either CTA of a pair: the bytes are counted on the barrier at this address in the
// pair's leader CTA (cta_group::2 permits the barrier to live in the peer).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, uint32_t leader_bar)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(leader_bar) : "memory");
}
// shared::cluster address of this CTA's shared-memory location `addr` as seen in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_addr(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster_release(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// TMA stores out of shared memory (bulk async-group completion).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, int32_t x, int32_t y, uint32_t src)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap *map, int32_t x, int32_t y, uint32_t src)
{
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }

template <int CTAS>
__device__ __forceinline__ void tcgen05_commit(uint32_t bar)
{
    if (CTAS == 1) {
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    } else {   // arrives on the barrier at this offset in both CTAs of the pair
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(bar), "h"((uint16_t)3) : "memory");
    }
}
template <int CTAS>
__device__ __forceinline__ void tcgen05_cp_32x128b_warpx4(uint32_t taddr, uint64_t sdesc)
{
    if (CTAS == 1) asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
    else asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}

template <int KIND, int CTAS>
__device__ __forceinline__ void tcgen05_mma_block_scaled(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                         uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate)
{
    if (KIND == KIND_MXF4B16 && CTAS == 2) {
        asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                     " tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%5], [%6], p;\n}"
                     ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
                     : "memory");
    } else if (KIND == KIND_MXF4B16) {
        asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                     " tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%5], [%6], p;\n}"
                     ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
                     : "memory");
    } else if (kind_fp4(KIND) && CTAS == 2) {
        asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                     " tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%6], p;\n}"
                     ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
                     : "memory");
    } else if (kind_fp4(KIND)) {
        asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                     " tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%6], p;\n}"
                     ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
                     : "memory");
    } else if (CTAS == 2) {
        asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                     " tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%5], [%6], p;\n}"
                     ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
                     : "memory");
    } else {
        asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                     " tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%5], [%6], p;\n}"
                     ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
                     : "memory");
    }
}

// Shared-memory matrix descriptor, K-major operand tile stored as rows of 128 B with the 128-byte swizzle
// (8-row groups 1024 B apart).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Descriptor of a replicated scale image: 8 rows of 16 B; the stride between 8-row groups is zero, so the 32 rows
// tcgen05.cp reads are four passes over the same 128 bytes.
__device__ __forceinline__ uint64_t smem_desc_scale_image_rep(uint32_t addr)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 46);
}
// Descriptor of a scale image: 32 rows of 16 B, contiguous (no swizzle; 8-row groups 128 B apart).
__device__ __forceinline__ uint64_t smem_desc_scale_image(uint32_t addr)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(128 >> 4) << 32) | (1ull << 46);
}

// Instruction descriptor of the block-scaled MMA: formats, K-major operands, N, UE8M0 scales, M, scale byte ids.
template <int KIND, int CTAS>
__device__ __forceinline__ uint32_t instr_desc(uint32_t a_sf_id, uint32_t b_sf_id)
{
    const uint32_t fmt = kind_fp4(KIND) ? 1u : 0u;   // mxf4: E2M1 = 1; mxf8f6f4: E4M3 = 0
    return (b_sf_id << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(BN >> 3) << 17) | (1u << 23) |
           ((uint32_t)((BM * CTAS) >> 4) << 24) | (a_sf_id << 29);
}

#define FP4Q_TMEM_LD_X32(taddr, v)                                                                              \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                      \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                      \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                     \
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), \
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),      \
                   "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),    \
                   "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),    \
                   "=r"(v[29]), "=r"(v[30]), "=r"(v[31])                                                         \
                 : "r"(taddr))

// ---------------------------------------------------------------------------------------- tile decoding

// Grouped products need their group once per tile.  Searching the boundaries is a chain of dependent loads (seven
// for 128 groups), and in the TMA producer every load queues behind the copies it has just issued (about 500 cycles
// each): 4000 cycles per tile, more than a tile with a short contraction runs.  So the CTA fills a table in shared
// memory before its roles start (`goffs`, 4 KB, null when the problem is too large for it or the kernel's
// configuration has no room): with grouped rows the group of every 128-row tile as 16 bits (one load per tile),
// with a grouped contraction a 32-bit copy of the boundaries.

__device__ __forceinline__ int find_group(const int64_t *offs, const int32_t *goffs, int n_groups, int64_t row)
{
    int lo = 0, hi = n_groups;      // largest g with offs[g] <= row
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        const int64_t v = goffs ? (int64_t)goffs[mid] : __ldg(offs + mid);
        if (v <= row) lo = mid; else hi = mid;
    }
    return lo;
}

// need_b = false leaves out the B operand's position: with grouped rows that is the group lookup, which only the
// producer and the scale builder need - the MMA issuer, the watcher and the epilogue use the contraction length and
// the output position alone, and a lookup in the MMA warp (shared-memory reads behind its pending MMAs) costs
// about 1900 cycles per tile.
__device__ __forceinline__ void decode_tile(const GemmParams &p, int tile, int rank, Tile &t, const int32_t *goffs, bool need_b = true)
{
    const int per_problem = p.m_tiles * p.n_tiles;
    const int g = p.mode == MODE_GROUPED_K ? tile / per_problem : 0;
    const int local = tile - g * per_problem;
    // Tiles that run at the same time (consecutive indices) cover raster_m row tiles x a few column tiles, and
    // the sweep over column tiles finishes before the next group of row tiles starts: the group's A rows stay
    // in L2 for the whole sweep instead of the whole A operand being streamed once per wave.
    const int per_group = p.raster_m * p.n_tiles;
    const int grp_m = local / per_group, in_grp = local - grp_m * per_group;
    const int m0 = grp_m * p.raster_m, gsz = min(p.raster_m, p.m_tiles - m0);
    const int n_blk = in_grp / gsz, m_blk = m0 + (in_grp - n_blk * gsz);
    t.a_row0 = (m_blk * p.ctas + rank) * BM;
    t.b_row0 = n_blk * BN;
    t.b_load_row0 = t.b_row0 + (p.ctas == 2 ? rank * 128 : 0);
    t.a_k0 = t.b_k0 = 0;
    t.k_len = p.K;
    t.c_row0 = t.a_row0;
    t.c_col0 = t.b_row0;
    t.m_valid = min(BM, p.M - t.a_row0);
    t.n_valid = min(BN, p.N - t.b_row0);
    if (p.mode == MODE_GROUPED_ROWS) {
        if (!need_b) return;
        const int grp = goffs ? (int)reinterpret_cast<const uint16_t *>(goffs)[t.a_row0 / BM]
                              : find_group(p.row_offsets, nullptr, p.n_groups, (int64_t)t.a_row0);
        t.b_row0 += grp * p.b_rows_per_group;
        t.b_load_row0 += grp * p.b_rows_per_group;
        t.b_k0 = grp * p.b_k_per_group;
    } else if (p.mode == MODE_GROUPED_K) {
        const int64_t k0 = goffs ? (int64_t)goffs[g] : __ldg(p.row_offsets + g), k1 = goffs ? (int64_t)goffs[g + 1] : __ldg(p.row_offsets + g + 1);
        t.a_k0 = t.b_k0 = (int32_t)k0;
        t.k_len = (int32_t)(k1 - k0);
        t.c_row0 = g * p.M + t.a_row0;
    }
}

// ---------------------------------------------------------------------------------------- scale images

// Scale slots beyond the tensor read this byte instead (their payload is zero, any finite scale will do).
__device__ const uint8_t g_scale_pad[4] = {kScalePad, kScalePad, kScalePad, kScalePad};

// One compact scale byte.  The bounds check selects the ADDRESS, not the value, so that nothing depends on
// the loaded byte until it is written into the image several stages later (an in-order warp stalls at the
// first use of a pending load).
__device__ __forceinline__ void load_scale(const ScaleView &v, int row, int kb, uint32_t &dst)
{
    const uint8_t *ptr = (row < v.n_row && kb < v.n_kb) ? v.ptr + (int64_t)row * v.stride_row + (int64_t)kb * v.stride_kb
                                                        : g_scale_pad;
    asm volatile("ld.global.nc.u8 %0, [%1];" : "=r"(dst) : "l"(ptr));
}

// The stream of ring stages one CTA works through: its tiles in order, each with its contraction stages.
struct StageIter {
    int tile, step, rank, it, n_it;
    const int32_t *goffs;
    bool need_b;
    Tile t;
    __device__ __forceinline__ void seek(const GemmParams &p, int stage_elems)
    {
        while (tile < p.n_tile_total) {
            decode_tile(p, tile, rank, t, goffs, need_b);
            n_it = (t.k_len + stage_elems - 1) / stage_elems;
            if (n_it > 0) { it = 0; return; }
            tile += step;
        }
        n_it = 0;
    }
    __device__ __forceinline__ void init(const GemmParams &p, int first, int step_, int rank_, int stage_elems, const int32_t *goffs_,
                                         bool need_b_)
    {
        tile = first; step = step_; rank = rank_; it = 0; goffs = goffs_; need_b = need_b_;
        seek(p, stage_elems);
    }
    __device__ __forceinline__ bool valid(const GemmParams &p) const { return tile < p.n_tile_total; }
    __device__ __forceinline__ void next(const GemmParams &p, int stage_elems)
    {
        if (++it >= n_it) { tile += step; seek(p, stage_elems); }
    }
};

__device__ __forceinline__ void ldg_b32(const uint8_t *ptr, uint32_t &w)
{
    asm volatile("ld.global.nc.b32 %0, [%1];" : "=r"(w) : "l"(ptr));
}

// Rows of a 4x4 byte matrix given by its columns: w[k] holds byte rt of column k in byte lane rt.
__device__ __forceinline__ uint4 transpose4x4_bytes(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3)
{
    const uint32_t t0 = __byte_perm(w0, w1, 0x5140), t1 = __byte_perm(w2, w3, 0x5140);
    const uint32_t t2 = __byte_perm(w0, w1, 0x7362), t3 = __byte_perm(w2, w3, 0x7362);
    return make_uint4(__byte_perm(t0, t1, 0x5410), __byte_perm(t0, t1, 0x7632), __byte_perm(t2, t3, 0x5410),
                      __byte_perm(t2, t3, 0x7632));
}

// mxf4 / 2D blocks: a stage covers 8 contraction blocks (two chunks of 4).  For 128 operand rows and one chunk the
// scale image is 32 identical rows of 16 bytes [row tile 0..3][block 0..3]; A needs 2 such rows per stage (one per
// chunk), B (256 rows) 4.
// Gathers the scale bytes of n_chunks contraction chunks (4 blocks each) for 2^log2_rt consecutive row tiles into
// dst[(chunk << log2_rt) + rt] as 32-bit words (byte k = block 4*chunk + k): the 16-byte image rows of the chunk.
// One warp; each lane takes items lane, lane + 32, ...  Slots beyond the tensor read the pad byte.
__device__ __forceinline__ void build_scale_cache(const ScaleView &v, int rt0, int kb0, int n_chunks, int log2_rt,
                                                  uint32_t *dst, int lane)
{
    const bool aligned4 = (reinterpret_cast<uintptr_t>(v.ptr) & 3) == 0;
    if (v.stride_row == 1 && v.stride_kb != 1 && aligned4 && (v.stride_kb & 3) == 0 && (rt0 & 3) == 0) {
        // transposed view: the row-tile bytes of one block are contiguous.  An item is a chunk and a group of four
        // row tiles: four 32-bit loads (one per block) and a 4x4 byte transpose give the group's four words.
        const int log2_g = log2_rt - 2, n_items = n_chunks << log2_g;
        for (int base = 0; base < n_items; base += 32 * 2) {
            uint32_t w[2][4];
#pragma unroll
            for (int j = 0; j < 2; j++) {
                const int q = base + 32 * j + lane;
                const int chunk = q >> log2_g, rg = q & ((1 << log2_g) - 1);
                const int row = rt0 + 4 * rg, kb = kb0 + 4 * chunk;
#pragma unroll
                for (int k = 0; k < 4; k++) {
                    w[j][k] = kScalePad * 0x01010101u;
                    if (q < n_items) {
                        if (row + 4 <= v.n_row && kb + k < v.n_kb) {
                            ldg_b32(v.ptr + (int64_t)(kb + k) * v.stride_kb + row, w[j][k]);
                        } else {
                            uint32_t b0, b1, b2, b3;
                            load_scale(v, row, kb + k, b0);
                            load_scale(v, row + 1, kb + k, b1);
                            load_scale(v, row + 2, kb + k, b2);
                            load_scale(v, row + 3, kb + k, b3);
                            w[j][k] = b0 | (b1 << 8) | (b2 << 16) | (b3 << 24);
                        }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < 2; j++) {
                const int q = base + 32 * j + lane;
                if (q < n_items) reinterpret_cast<uint4 *>(dst)[q] = transpose4x4_bytes(w[j][0], w[j][1], w[j][2], w[j][3]);
            }
        }
        return;
    }
    const int n_items = n_chunks << log2_rt;
    const bool along_k = v.stride_kb == 1 && aligned4 && (v.stride_row & 3) == 0 && (kb0 & 3) == 0;
    for (int base = 0; base < n_items; base += 32 * 4) {
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; j++) {   // loads of four items in flight before anything is used
            const int q = base + 32 * j + lane;
            const int chunk = q >> log2_rt, rt = q & ((1 << log2_rt) - 1);
            const int row = rt0 + rt, kb = kb0 + 4 * chunk;
            w[j] = 0;
            if (q < n_items) {
                if (along_k && row < v.n_row && kb + 4 <= v.n_kb) {
                    ldg_b32(v.ptr + (int64_t)row * v.stride_row + kb, w[j]);
                } else {
                    uint32_t b0, b1, b2, b3;
                    load_scale(v, row, kb, b0);
                    load_scale(v, row, kb + 1, b1);
                    load_scale(v, row, kb + 2, b2);
                    load_scale(v, row, kb + 3, b3);
                    w[j] = b0 | (b1 << 8) | (b2 << 16) | (b3 << 24);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const int q = base + 32 * j + lane;
            if (q < n_items) dst[q] = w[j];
        }
    }
}

// Per-row scales (MXFP8): one 32-bit word = the four scale bytes of one row and one stage.
__device__ __forceinline__ void load_scale_word(const ScaleView &v, int row, int kb0, uint32_t &dst)
{
    const uint8_t *ptr = v.ptr + (int64_t)row * v.stride_row + kb0;
    if (row < v.n_row && kb0 + 4 <= v.n_kb && v.stride_kb == 1 && (reinterpret_cast<uintptr_t>(ptr) & 3) == 0) {
        asm volatile("ld.global.nc.b32 %0, [%1];" : "=r"(dst) : "l"(ptr));   // the common case: nothing depends on it yet
        return;
    }
    uint32_t word = 0;
#pragma unroll
    for (int kb = 0; kb < 4; kb++) {
        uint32_t b;
        load_scale(v, row, kb0 + kb, b);
        word |= b << (8 * kb);
    }
    dst = word;
}

__device__ __forceinline__ void ldg_v4(const uint8_t *ptr, uint32_t *w)
{
    asm volatile("ld.global.nc.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "l"(ptr));
}

template <int KIND>
__device__ __forceinline__ void store_row_scale_images(const uint32_t (&w)[12][8], int n_stages, uint8_t *images, int lane)
{
    if (KIND == KIND_MXF8) {
#pragma unroll
        for (int st = 0; st < 8; st++) {
            if (st < n_stages) {
                uint4 *img = reinterpret_cast<uint4 *>(images + st * kImageStageBytesMxf8);
                img[lane] = make_uint4(w[0][st], w[1][st], w[2][st], w[3][st]);           // A
                img[32 + lane] = make_uint4(w[4][st], w[5][st], w[6][st], w[7][st]);      // B rows 0..127
                img[64 + lane] = make_uint4(w[8][st], w[9][st], w[10][st], w[11][st]);    // B rows 128..255
            }
        }
    } else if (KIND == KIND_MXF4B16) {
        // word j of a row = the four scale bytes of MMA j of the unit (stage j / 4, MMA j % 4)
#pragma unroll
        for (int st = 0; st < 2; st++) {
            if (st < n_stages) {
                uint4 *img = reinterpret_cast<uint4 *>(images + st * kImageStageBytesMxf4B16);
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    const int j = 4 * st + i;
                    img[32 * i + lane] = make_uint4(w[0][j], w[1][j], w[2][j], w[3][j]);                  // A, MMA i
                    img[128 + 64 * i + lane] = make_uint4(w[4][j], w[5][j], w[6][j], w[7][j]);            // B rows 0..127
                    img[160 + 64 * i + lane] = make_uint4(w[8][j], w[9][j], w[10][j], w[11][j]);          // B rows 128..255
                }
            }
        }
    } else {
#pragma unroll
        for (int st = 0; st < 4; st++) {
            if (st < n_stages) {
                uint4 *img = reinterpret_cast<uint4 *>(images + st * kImageStageBytesMxf4R);
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    const int j = 2 * st + c;
                    img[32 * c + lane] = make_uint4(w[0][j], w[1][j], w[2][j], w[3][j]);                 // A, chunk c
                    img[64 + 64 * c + lane] = make_uint4(w[4][j], w[5][j], w[6][j], w[7][j]);            // B rows 0..127
                    img[96 + 64 * c + lane] = make_uint4(w[8][j], w[9][j], w[10][j], w[11][j]);          // B rows 128..255
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------- epilogue store

// Transpose of a 32x32 matrix of nibbles held one row per lane (W[w] nibble n = column 8w + n of the lane's row): on
// return lane c holds column c (W[w] nibble n = row 8w + n).  Five exchange steps, one per index bit: lanes that
// differ in bit b swap the elements whose position bit b differs from their own lane bit b (whole words for the
// two word-index bits, masked and shifted nibble groups for the three nibble-index bits).
__device__ __forceinline__ void transpose32x32_nibbles(uint32_t W[4], int lane)
{
    {   // position bit 4 = word bit 1: words {2,3} <-> {0,1} between lanes 16 apart
        const bool up = lane & 16;
        const uint32_t r0 = __shfl_xor_sync(0xFFFFFFFFu, up ? W[0] : W[2], 16);
        const uint32_t r1 = __shfl_xor_sync(0xFFFFFFFFu, up ? W[1] : W[3], 16);
        if (up) { W[0] = r0; W[1] = r1; } else { W[2] = r0; W[3] = r1; }
    }
    {   // position bit 3 = word bit 0: words {1,3} <-> {0,2} between lanes 8 apart
        const bool up = lane & 8;
        const uint32_t r0 = __shfl_xor_sync(0xFFFFFFFFu, up ? W[0] : W[1], 8);
        const uint32_t r1 = __shfl_xor_sync(0xFFFFFFFFu, up ? W[2] : W[3], 8);
        if (up) { W[0] = r0; W[2] = r1; } else { W[1] = r0; W[3] = r1; }
    }
#pragma unroll
    for (int b = 2; b >= 0; b--) {   // nibble-index bits: groups of 4, 2, 1 nibbles between lanes 4, 2, 1 apart
        const uint32_t lo = b == 2 ? 0x0000FFFFu : b == 1 ? 0x00FF00FFu : 0x0F0F0F0Fu;
        const int sh = 4 << b;
        const bool up = lane & (1 << b);
#pragma unroll
        for (int w = 0; w < 4; w++) {
            const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, W[w], 1 << b);
            W[w] = up ? ((W[w] & ~lo) | ((other & ~lo) >> sh)) : ((W[w] & lo) | ((other & lo) << sh));
        }
    }
}

// One round of the pair kernel's epilogue: 32 words per lane (this lane's row, 128 bytes) into the warp's swizzled
// staging rows, then one TMA store (kind 0: BF16 bytes, 1: FP32 bytes, 2: FP32 add-reduction) of the 32 x 128 B box.
__device__ __forceinline__ void stage_and_store(const CUtensorMap *map, const uint32_t *w, uint32_t stg_row, uint32_t swz,
                                                uint32_t stg, int col, int32_t y, int kind, int lane)
{
    if (lane == 0) bulk_wait_read_all();   // the previous round's store has read the staging rows
    __syncwarp();
#pragma unroll
    for (int c = 0; c < 8; c++)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg_row + ((c ^ swz) << 4)), "r"(w[4 * c]), "r"(w[4 * c + 1]),
                     "r"(w[4 * c + 2]), "r"(w[4 * c + 3]) : "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> TMA store
    __syncwarp();
    if (lane == 0) {
        if (kind == 2) tma_reduce_add_2d(map, col, y, stg);                 // x in FP32 elements
        else tma_store_2d(map, col * (kind == 1 ? 4 : 2), y, stg);          // x in bytes
        bulk_commit();
    }
}

// One whole 32-byte sector per lane (a 16-byte store leaves half a sector to a second transaction).
__device__ __forceinline__ void st_global_v8(void *dst, const uint32_t *w)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                 "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
}

__device__ __forceinline__ void store_row_chunk(const GemmParams &p, int64_t row, int col0, int n_cols_valid,
                                                const uint32_t v[32])
{
    // 32 consecutive accumulator columns of one output row, starting at column col0
    if (n_cols_valid <= 0) return;
    if (p.out_f32) {
        float *dst = static_cast<float *>(p.C) + row * p.ldc + col0;
        if (n_cols_valid >= 32 && p.wide_stores && !p.accumulate) {
#pragma unroll
            for (int q = 0; q < 4; q++) st_global_v8(dst + 8 * q, v + 8 * q);
        } else if (n_cols_valid >= 32) {
#pragma unroll
            for (int q = 0; q < 8; q++) {
                float4 o = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                       __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                if (p.accumulate) {
                    const float4 old = *reinterpret_cast<const float4 *>(dst + 4 * q);
                    o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                }
                *reinterpret_cast<float4 *>(dst + 4 * q) = o;
            }
        } else {
#pragma unroll
            for (int q = 0; q < 32; q++)
                if (q < n_cols_valid) dst[q] = __uint_as_float(v[q]) + (p.accumulate ? dst[q] : 0.0f);
        }
    } else {
        __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.C) + row * p.ldc + col0;
        if (n_cols_valid >= 32 && p.wide_stores) {
            uint32_t w[16];
#pragma unroll
            for (int e = 0; e < 16; e++) {
                const __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
                w[e] = *reinterpret_cast<const uint32_t *>(&b);
            }
            st_global_v8(dst, w);
            st_global_v8(dst + 16, w + 8);
        } else if (n_cols_valid >= 32) {
#pragma unroll
            for (int q = 0; q < 4; q++) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; e++) {
                    const __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(v[8 * q + 2 * e]),
                                                                   __uint_as_float(v[8 * q + 2 * e + 1]));
                    w[e] = *reinterpret_cast<const uint32_t *>(&b);
                }
                *reinterpret_cast<uint4 *>(dst + 8 * q) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        } else {
#pragma unroll
            for (int q = 0; q < 32; q++)
                if (q < n_cols_valid) dst[q] = __float2bfloat16_rn(__uint_as_float(v[q]));
        }
    }
}

// Position in a ring of image buffers: buffer index and the parity of the barrier phase that goes with it.
struct BufRing {
    uint32_t buf = 0, phase = 0;
    __device__ __forceinline__ void next(uint32_t n) { if (++buf == n) { buf = 0; phase ^= 1u; } }
};

// The stream of scale units (kUnitStages stages of one tile) a CTA works through.
struct UnitIter {
    int tile, step, rank, k0;
    const int32_t *goffs;
    Tile t;
    __device__ __forceinline__ void seek(const GemmParams &p)
    {
        while (tile < p.n_tile_total) {
            decode_tile(p, tile, rank, t, goffs);
            if (k0 < t.k_len) return;
            tile += step;
            k0 = 0;
        }
    }
    __device__ __forceinline__ void init(const GemmParams &p, int first, int step_, int rank_, const int32_t *goffs_)
    {
        tile = first; step = step_; rank = rank_; k0 = 0; goffs = goffs_;
        seek(p);
    }
    __device__ __forceinline__ bool valid(const GemmParams &p) const { return tile < p.n_tile_total; }
    __device__ __forceinline__ void next(const GemmParams &p, int unit_elems) { k0 += unit_elems; seek(p); }
};

__device__ __forceinline__ void cp_async(uint32_t dst, const void *src, int bytes, int src_bytes)
{
    if (bytes == 16) asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
    else if (bytes == 8) asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
    else asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

// Raw scale bytes of one unit (32 contraction blocks from k0), asynchronously into `raw` (12 KB): slot q (1 KB,
// q < 4: A rows 32q.., q >= 4: B rows 32(q-4)..) holds 32 bytes per lane, the scale bytes of the lane's operand row.
// A 2D-block operand (row_shift 5) needs only 32 bytes per row tile: they are packed at the start of the operand's
// first slot; if its view is transposed (blocks stride_kb apart, row tiles contiguous) lane l fetches block l's
// bytes for the operand's 4 or 8 row tiles into the first 8 bytes of its entry of that slot.  With 16 x 16 blocks
// (row_shift 4, KB_SHIFT 4: a block is 16 contraction elements and a row tile 16 rows) the unit still has 32 blocks but
// the operand has 8 or 16 row tiles.  Bytes beyond the tensor arrive as zero.  Every lane commits exactly one
// cp.async group per call.
template <int KB_SHIFT>
__device__ __forceinline__ void issue_raw_scales(const GemmParams &p, const Tile &t, int k0, uint8_t *raw, int lane)
{
#pragma unroll
    for (int op = 0; op < 2; op++) {
        const ScaleView &v = op == 0 ? p.sfa : p.sfb;
        const int nq = op == 0 ? 4 : 8, q0 = op == 0 ? 0 : 4;
        const int row0 = op == 0 ? t.a_row0 : t.b_row0;
        const int kb0 = ((op == 0 ? t.a_k0 : t.b_k0) + k0) >> KB_SHIFT;
        const int n_tiles = v.row_shift != 0 ? nq << (5 - v.row_shift) : 0;   // row tiles of a 2D-block operand
        if (v.row_shift != 0 && v.stride_kb != 1) {
            const int rt0 = row0 >> v.row_shift, kb = kb0 + lane, nbytes = n_tiles;   // 4 .. 16 row tiles, one byte each
            uint8_t *dst = raw + q0 * 1024 + lane * 32;
            const uint8_t *src = v.ptr + (int64_t)kb * v.stride_kb + rt0;
            const int valid = kb < v.n_kb ? max(0, min(nbytes, v.n_row - rt0)) : 0;
            if (v.stride_row == 1 && (reinterpret_cast<uintptr_t>(src) & (nbytes - 1)) == 0) {
                cp_async(smem_u32(dst), valid > 0 ? src : v.ptr - (reinterpret_cast<uintptr_t>(v.ptr) & 15), nbytes, valid);
            } else {
                for (int r = 0; r < nbytes; r++) {
                    uint32_t b;
                    load_scale(v, rt0 + r, kb, b);
                    dst[r] = (uint8_t)b;
                }
            }
            continue;
        }
        if (v.row_shift != 0) {
            // 2D-block operand, blocks contiguous: the 32 bytes of each of the operand's row tiles once (two lanes
            // per row tile copy 16 bytes each), packed at the start of the operand's first slot
            if (lane < 2 * n_tiles) {
                const int rt = (row0 >> v.row_shift) + (lane >> 1), kb = kb0 + 16 * (lane & 1);
                uint8_t *dst = raw + q0 * 1024 + lane * 16;
                const uint8_t *src = v.ptr + (int64_t)rt * v.stride_row + kb;
                if ((reinterpret_cast<uintptr_t>(src) & 15) == 0) {
                    const int valid = rt < v.n_row ? max(0, min(16, v.n_kb - kb)) : 0;
                    cp_async(smem_u32(dst), valid > 0 ? src : v.ptr - (reinterpret_cast<uintptr_t>(v.ptr) & 15), 16, valid);
                } else {
#pragma unroll
                    for (int st = 0; st < 4; st++) {
                        uint32_t word;
                        load_scale_word(v, rt, kb + 4 * st, word);
                        reinterpret_cast<uint32_t *>(dst)[st] = word;
                    }
                }
            }
            continue;
        }
#pragma unroll
        for (int q = 0; q < nq; q++) {
            const int row = row0 + lane + 32 * q;
            uint8_t *dst = raw + (q0 + q) * 1024 + lane * 32;
            const uint8_t *src = v.ptr + (int64_t)row * v.stride_row + kb0;
            if (v.stride_kb == 1 && (reinterpret_cast<uintptr_t>(src) & 15) == 0) {
                const int valid = row < v.n_row ? max(0, min(32, v.n_kb - kb0)) : 0;
                const uint8_t *safe = v.ptr - (reinterpret_cast<uintptr_t>(v.ptr) & 15);
                cp_async(smem_u32(dst), valid > 0 ? src : safe, 16, min(valid, 16));
                cp_async(smem_u32(dst + 16), valid > 16 ? src + 16 : safe, 16, max(valid - 16, 0));
            } else {
#pragma unroll
                for (int st = 0; st < 8; st++) {
                    uint32_t word;
                    load_scale_word(v, row, kb0 + 4 * st, word);
                    reinterpret_cast<uint32_t *>(dst)[st] = word;
                }
            }
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// The unit's scale words from a raw buffer whose copies have completed: w[q][j] = the four scale bytes of the
// lane's row of slot q for blocks 4j..4j+3.  Lanes read bytes other lanes copied: the caller synchronizes the warp
// after its cp.async wait.
__device__ __forceinline__ void read_raw_scales(const GemmParams &p, const uint8_t *raw, int lane, uint32_t (&w)[12][8])
{
#pragma unroll
    for (int op = 0; op < 2; op++) {
        const ScaleView &v = op == 0 ? p.sfa : p.sfb;
        const int nq = op == 0 ? 4 : 8, q0 = op == 0 ? 0 : 4;
        if (v.row_shift != 0 && v.stride_kb != 1) {
            // lane l holds block l's bytes [row tile 0..]: words of four consecutive lanes, transposed as 4x4 bytes,
            // are the four row tiles' words of one chunk
            if (v.row_shift == 4) {
                // 16-row tiles: 8 (A) or 16 (B) bytes per lane; operand rows l + 32 q of image row l lie in row tile
                // 2 q + (l >> 4), so the two halves of the warp pick different tiles of each transposed word
                const uint4 mine4 = *reinterpret_cast<const uint4 *>(raw + q0 * 1024 + lane * 32);
                const bool hi = lane >= 16;
#pragma unroll
                for (int h = 0; h < (op == 0 ? 2 : 4); h++) {
                    const uint32_t m = h == 0 ? mine4.x : h == 1 ? mine4.y : h == 2 ? mine4.z : mine4.w;
#pragma unroll
                    for (int j = 0; j < 8; j++) {
                        const uint4 tr = transpose4x4_bytes(__shfl_sync(0xFFFFFFFFu, m, 4 * j), __shfl_sync(0xFFFFFFFFu, m, 4 * j + 1),
                                                            __shfl_sync(0xFFFFFFFFu, m, 4 * j + 2), __shfl_sync(0xFFFFFFFFu, m, 4 * j + 3));
                        w[q0 + 2 * h][j] = hi ? tr.y : tr.x;
                        w[q0 + 2 * h + 1][j] = hi ? tr.w : tr.z;
                    }
                }
                continue;
            }
            const uint2 mine = *reinterpret_cast<const uint2 *>(raw + q0 * 1024 + lane * 32);
#pragma unroll
            for (int h = 0; h < (op == 0 ? 1 : 2); h++) {
                const uint32_t m = h == 0 ? mine.x : mine.y;
#pragma unroll
                for (int j = 0; j < 8; j++) {
                    const uint4 tr = transpose4x4_bytes(__shfl_sync(0xFFFFFFFFu, m, 4 * j), __shfl_sync(0xFFFFFFFFu, m, 4 * j + 1),
                                                        __shfl_sync(0xFFFFFFFFu, m, 4 * j + 2), __shfl_sync(0xFFFFFFFFu, m, 4 * j + 3));
                    w[q0 + 4 * h + 0][j] = tr.x; w[q0 + 4 * h + 1][j] = tr.y; w[q0 + 4 * h + 2][j] = tr.z; w[q0 + 4 * h + 3][j] = tr.w;
                }
            }
            continue;
        }
#pragma unroll
        for (int q = 0; q < nq; q++) {
            const int tile = v.row_shift == 4 ? 2 * q + (lane >> 4) : q;   // row tile of operand row lane + 32 q
            const uint4 *src = reinterpret_cast<const uint4 *>(v.row_shift != 0 ? raw + q0 * 1024 + tile * 32 : raw + (q0 + q) * 1024 + lane * 32);
            const uint4 lo = src[0], hi = src[1];
            w[q0 + q][0] = lo.x; w[q0 + q][1] = lo.y; w[q0 + q][2] = lo.z; w[q0 + q][3] = lo.w;
            w[q0 + q][4] = hi.x; w[q0 + q][5] = hi.y; w[q0 + q][6] = hi.z; w[q0 + q][7] = hi.w;
        }
    }
}

// ---------------------------------------------------------------------------------------- kernel

template <int KIND, int CTAS, int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm_block_scaled_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                         const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmD,
                         const __grid_constant__ GemmParams p)
{
    constexpr int kStageElems = kind_fp4(KIND) ? 256 : 128;   // contraction elements per stage (128 B per row)
    constexpr int kMmaK = kind_fp4(KIND) ? 64 : 32;           // contraction elements per MMA (32 B per row)
    constexpr int kElemsPerByte = kind_fp4(KIND) ? 2 : 1;
    constexpr int kStages = Cfg<KIND, CTAS>::kStages;
    constexpr int kBStageBytes = Cfg<KIND, CTAS>::kBStageBytes;
    constexpr int kUnitStages = KIND == KIND_MXF4 ? kUnitStagesMxf4 : KIND == KIND_MXF8 ? kUnitStagesMxf8
                                : KIND == KIND_MXF4R ? kUnitStagesMxf4R : kUnitStagesMxf4B16;   // stages whose scale images are built together
    constexpr int kKbShift = KIND == KIND_MXF4B16 ? 4 : 5;    // log2 of the scale vector's length (contraction elements per scale byte)

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *smem_a = smem;
    uint8_t *smem_b = smem + kStages * kAStageBytes;
    uint8_t *smem_compact = smem + Cfg<KIND, CTAS>::kSmemOperands;   // 2D blocks: compact scale rows of the unit being built ...
    uint8_t *smem_images = smem_compact + kCompactBytes;        // ... and the buffers of ready scale images (any kind)
    uint8_t *smem_raw_scales = smem_images + Cfg<KIND, CTAS>::kImageBufs * kCacheBufBytes;   // per-row scales: bytes in flight
    uint8_t *smem_staging = smem_compact + Cfg<KIND, CTAS>::kSmemScales;   // 1024-byte aligned (pair kernel only)
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_staging + Cfg<KIND, CTAS>::kSmemStaging);
    // bars[0..5] full, bars[6..11] empty, bars[12] accumulator full, bars[13] accumulator empty,
    // bars[18] tensor pipe drained (abort path), bars[24..27] scale images full, bars[28..31] scale images empty,
    // bars[32..35] (leader of a pair) the second CTA's scale images full - one of each per image buffer
    uint32_t *tmem_base_slot = reinterpret_cast<uint32_t *>(bars + 21);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(bars + 21) + 1;
    int32_t *goffs_smem = reinterpret_cast<int32_t *>(reinterpret_cast<uint8_t *>(bars) + kSmemTail);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Poll limit of every bounded wait (workspace word 2; 0 = the default) and the development hook of word 3 (n > 0:
    // the producer of CTA 0 leaves out its n-th stage load, so that a test can watch a wait run out and the kernel
    // leave through its timeout path without anything faulting or spinning for long).
    const uint32_t wait_limit_word = __ldg(p.status + 2), withhold_load = blockIdx.x == 0 ? __ldg(p.status + 3) : 0u;
    const uint64_t wait_limit = wait_limit_word != 0u ? wait_limit_word : kWaitLimit;
    const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + kMaxStages);
    const uint32_t bar_acc_full = smem_u32(bars + 12), bar_acc_empty = smem_u32(bars + 13);
    const uint32_t bar_cache_full = smem_u32(bars + 24), bar_cache_empty = smem_u32(bars + 28);
    const uint32_t bar_drain = smem_u32(bars + 18), bar_peer_cache_full = smem_u32(bars + 32);
    constexpr int kImageBufs = Cfg<KIND, CTAS>::kImageBufs;

    // In a pair, rank 0 leads: it owns the "full" and "accumulator empty" barriers and issues every tcgen05.mma.
    const int rank = CTAS == 2 ? (int)cluster_ctarank() : 0;
    const bool leader = rank == 0;
    const int first_tile = blockIdx.x / CTAS, tile_step = gridDim.x / CTAS;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; s++) {
            // The producer's expect_tx arrival (in a pair the leader's, which announces both CTAs' bytes: the second
            // CTA's loads complete on the leader's barrier).  The watcher of the stage waits on it.
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);    // tcgen05.commit
        }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_drain, 1);
        mbar_init(bar_acc_empty, 8 * CTAS);     // one arrival per epilogue warp (of both CTAs of a pair)
        for (int b = 0; b < Cfg<KIND, CTAS>::kImageBufs; b++) {
            mbar_init(bar_cache_full + 8 * b, 1);
            mbar_init(bar_cache_empty + 8 * b, 1);
            mbar_init(bar_peer_cache_full + 8 * b, 1);
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
        if (Cfg<KIND, CTAS>::kTmaStores) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmC) : "memory");
        if (EPI == EPI_QUANT) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmD) : "memory");
    }
    if (warp == 1) {
        if (CTAS == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_slot)),
                         "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_slot)),
                         "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        }
    }
    // grouped products: a 32-bit copy of the group boundaries for the per-tile lookups of every role
    const int n_row_tiles = (p.M + BM - 1) / BM;
    const bool goffs_ok = Cfg<KIND, CTAS>::kSmemGroups > 0 &&
                          ((p.mode == MODE_GROUPED_K && p.n_groups <= kMaxGroupsShared) ||
                           (p.mode == MODE_GROUPED_ROWS && n_row_tiles <= kMaxRowTilesShared && p.n_groups <= 65535));
    if (goffs_ok && p.mode == MODE_GROUPED_K)
        for (int g = threadIdx.x; g <= p.n_groups; g += kThreads) goffs_smem[g] = (int32_t)__ldg(p.row_offsets + g);
    if (goffs_ok && p.mode == MODE_GROUPED_ROWS)
        for (int i = threadIdx.x; i < n_row_tiles; i += kThreads)
            reinterpret_cast<uint16_t *>(goffs_smem)[i] = (uint16_t)find_group(p.row_offsets, nullptr, p.n_groups, (int64_t)i * BM);
    const int32_t *goffs = goffs_ok ? goffs_smem : nullptr;
    tcgen05_fence_before();
    __syncwarp();
    if (CTAS == 2) cluster_sync_all();   // the peer's barriers must exist before anything is signalled across CTAs
    else __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_base_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // A shared-memory access of this warp (the poll of the next "empty" barrier) queues behind the TMA
        // instructions it has just issued and waits ~450 cycles, which would limit one warp to a stage per
        // ~900 cycles.  So every round first polls - it waits for the next slot and then probes up to two
        // more - and only then issues the loads of all slots found free, back to back.
        constexpr int kBatch = 3;
        StageIter pr;
        pr.init(p, first_tile, tile_step, rank, kStageElems, goffs, true);
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        const bool issuer = elect_one();
        TRACE_DECL(c_empty); TRACE_DECL(c_issue); TRACE_DECL(c_rounds);
        TRACE_T0(tt);
        int ev_j = 0;
        while (Cfg<KIND, CTAS>::kSplitProducer && pr.valid(p)) {
            asm volatile("bar.sync %0, 64;" ::"r"(8 + stage) : "memory");   // the poller (warp 2) has seen the slot free and armed its barrier
            if (issuer && !(withhold_load != 0u && (uint32_t)ev_j + 1u == withhold_load)) {
                const Tile &t = pr.t;
                const int xa = (t.a_k0 + pr.it * kStageElems) / kElemsPerByte, xb = (t.b_k0 + pr.it * kStageElems) / kElemsPerByte;
                tma_load_2d(smem_u32(smem_a + stage * kAStageBytes), &tmA, xa, t.a_row0, bar_full + 8 * stage);
                tma_load_2d(smem_u32(smem_b + stage * kBStageBytes), &tmB, xb, t.b_load_row0, bar_full + 8 * stage);
            }
            ev_j++;
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
            pr.next(p, kStageElems);
        }
        while (ok && pr.valid(p)) {
            int n_free = 0;
#ifdef FP4Q_TRACE
            c_rounds++;
#endif
            if (lane == 0) {
                ok = mbar_wait_impl<0, true>(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status, wait_limit, 0x100u + stage);
                if (ok) {
                    n_free = 1;
                    uint32_t s2 = stage, ph2 = phase;
                    while (n_free < kBatch) {
                        if (++s2 == kStages) { s2 = 0; ph2 ^= 1u; }
                        if (!mbar_test_wait(bar_empty + 8 * s2, ph2 ^ 1u)) break;
                        n_free++;
                    }
                }
            }
            n_free = __shfl_sync(0xFFFFFFFFu, n_free, 0);
            ok = n_free > 0;
            TRACE_ADD(c_empty, tt);
            for (int b = 0; b < n_free && pr.valid(p); b++) {
                if (lane == 0) TRACE_EV(0, ev_j);
                if (issuer && !(withhold_load != 0u && (uint32_t)ev_j + 1u == withhold_load)) {
                    const Tile &t = pr.t;
                    const int xa = (t.a_k0 + pr.it * kStageElems) / kElemsPerByte, xb = (t.b_k0 + pr.it * kStageElems) / kElemsPerByte;
                    if (CTAS == 1) {
                        mbar_arrive_expect_tx(bar_full + 8 * stage, kAStageBytes + kBStageBytes);
                        tma_load_2d(smem_u32(smem_a + stage * kAStageBytes), &tmA, xa, t.a_row0, bar_full + 8 * stage);
                        tma_load_2d(smem_u32(smem_b + stage * kBStageBytes), &tmB, xb, t.b_load_row0, bar_full + 8 * stage);
                    } else {
                        // Both CTAs' bytes are counted on the leader's barrier, which the leader arms for all of them.
                        // (A remote mbarrier.arrive per stage by a thread of the second CTA costs ~1200 cycles each
                        // and cannot be pipelined; letting the TMA unit signal the remote barrier costs nothing.)
                        if (leader) mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * (kAStageBytes + kBStageBytes));
                        const uint32_t lbar = cluster_addr(bar_full + 8 * stage, 0);
                        tma_load_2d_pair(smem_u32(smem_a + stage * kAStageBytes), &tmA, xa, t.a_row0, lbar);
                        tma_load_2d_pair(smem_u32(smem_b + stage * kBStageBytes), &tmB, xb, t.b_load_row0, lbar);
                    }
                }
                if (lane == 0) TRACE_EV(1, ev_j);
                ev_j++;
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
                pr.next(p, kStageElems);
            }
            TRACE_ADD(c_issue, tt);
        }
        if (!ok) {   // give copies already in flight time to land before the CTA's shared memory is released
            for (int i = 0; i < 200; i++) __nanosleep(1000);
        }
        if (lane == 0) { TRACE_OUT(p, 0, c_empty); TRACE_OUT(p, 1, c_issue); TRACE_OUT(p, 5, c_rounds); }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (the leader CTA of a pair)
        // The warp stays converged and one elected lane issues the tcgen05 instructions: their descriptors then live
        // in uniform registers, and a scale copy costs about ten cycles of the issuing thread instead of fifty.  The
        // warp never reads shared memory inside the loop: a shared-memory access of this warp queues behind its own
        // pending MMAs and stalls the tensor pipe for ~200 cycles per poll.  A watcher warp polls the stage's "full"
        // barrier (and, for 2D scales, the accumulator's "empty" barrier) and hands over through a named barrier.
        uint32_t stage = 0, full_phase = 0, acc_empty_phase = 0;
        bool mma_ok = true;   // split producer only: this warp's own waits have not run out
        BufRing ring;   // image buffer of the current unit
        const bool issuer = elect_one();
        int ev_j = 0;
        TRACE_DECL(c_acc); TRACE_DECL(c_sync); TRACE_DECL(c_issue);
        TRACE_T0(tt);
        for (int tile = first_tile; leader && tile < p.n_tile_total; tile += tile_step) {
            Tile t;
            decode_tile(p, tile, rank, t, goffs, false);
            const int n_it = (t.k_len + kStageElems - 1) / kStageElems;
            if (n_it == 0) continue;
            TRACE_ADD(c_acc, tt);
            for (int it = 0; it < n_it; it++) {
                if (Cfg<KIND, CTAS>::kSplitProducer) {
                    // no watcher: the elected lane waits for the accumulator, the unit's scale images and the operands itself
                    if (lane == 0 && mma_ok) {
                        if (it == 0) mma_ok = mbar_wait_impl<0, true>(bar_acc_empty, acc_empty_phase ^ 1u, abort_flag, p.status, wait_limit, 0x200u);
                        if (mma_ok && (it & (kUnitStages - 1)) == 0)
                            mma_ok = mbar_wait_impl<0, true>(bar_cache_full + 8 * ring.buf, ring.phase, abort_flag, p.status, wait_limit, 0x510u + ring.buf);
                        if (mma_ok) mma_ok = mbar_wait_impl<0, true>(bar_full + 8 * stage, full_phase, abort_flag, p.status, wait_limit, 0x300u + stage);
                    }
                    if (it == 0) acc_empty_phase ^= 1u;
                    __syncwarp();
                } else {
                    named_sync(1 + stage);   // the watcher has seen the operands and both scale images of this stage
                }
                tcgen05_fence_after();
                TRACE_ADD(c_sync, tt);
                if (lane == 0) TRACE_EV(2, ev_j);
                if (issuer) {
                    const uint32_t sf_tmem = tmem_base + kTmemSfBase + stage * SfCols<KIND>::kStride;
                    if (KIND == KIND_MXF4) {
                        const uint32_t img = smem_u32(smem_images + ring.buf * kCacheBufBytes + (it & (kUnitStages - 1)) * kImageStageBytes);
#pragma unroll
                        for (int c = 0; c < 2; c++) {
                            tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem + 4 * c, smem_desc_scale_image_rep(img + 128 * c));
                            tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem + 8 + 8 * c, smem_desc_scale_image_rep(img + 256 + 256 * c));
                            tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem + 12 + 8 * c, smem_desc_scale_image_rep(img + 384 + 256 * c));
                        }
                    } else if (KIND == KIND_MXF4B16) {
                        const uint32_t img = smem_u32(smem_images + ring.buf * kCacheBufBytes + (it & (kUnitStages - 1)) * kImageStageBytesMxf4B16);
#pragma unroll
                        for (int i = 0; i < 4; i++) {
                            tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem + 4 * i, smem_desc_scale_image(img + 512 * i));
                            tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem + 16 + 8 * i, smem_desc_scale_image(img + 2048 + 1024 * i));
                            tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem + 20 + 8 * i, smem_desc_scale_image(img + 2560 + 1024 * i));
                        }
                    } else if (KIND == KIND_MXF4R) {
                        const uint32_t img = smem_u32(smem_images + ring.buf * kCacheBufBytes + (it & (kUnitStages - 1)) * kImageStageBytesMxf4R);
#pragma unroll
                        for (int c = 0; c < 2; c++) {
                            tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem + 4 * c, smem_desc_scale_image(img + 512 * c));
                            tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem + 8 + 8 * c, smem_desc_scale_image(img + 1024 + 1024 * c));
                            tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem + 12 + 8 * c, smem_desc_scale_image(img + 1536 + 1024 * c));
                        }
                    } else {
                        const uint32_t img = smem_u32(smem_images + ring.buf * kCacheBufBytes + (it & (kUnitStages - 1)) * kImageStageBytesMxf8);
                        tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem, smem_desc_scale_image(img));
                        tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem + 8, smem_desc_scale_image(img + 512));
                        tcgen05_cp_32x128b_warpx4<CTAS>(sf_tmem + 12, smem_desc_scale_image(img + 1024));
                    }
                    const uint64_t adesc = smem_desc_sw128(smem_u32(smem_a + stage * kAStageBytes));
                    const uint64_t bdesc = smem_desc_sw128(smem_u32(smem_b + stage * kBStageBytes));
                    const int k_left = t.k_len - it * kStageElems;
                    const int n_mma = min(4, (k_left + kMmaK - 1) / kMmaK);
#pragma unroll
                    for (int i = 0; i < 4; i++) {
                        if (i < n_mma) {
                            if (KIND == KIND_MXF4B16) {   // one 32-bit scale column entry per row and MMA: all four bytes are used
                                tcgen05_mma_block_scaled<KIND, CTAS>(tmem_base, adesc + 2 * i, bdesc + 2 * i, instr_desc<KIND, CTAS>(0u, 0u),
                                                                     sf_tmem + 4 * i, sf_tmem + 16 + 8 * i, (it > 0 || i > 0) ? 1u : 0u);
                                continue;
                            }
                            const int chunk = kind_fp4(KIND) ? (i >> 1) : 0;
                            const uint32_t sf_id = kind_fp4(KIND) ? 2u * (i & 1) : (uint32_t)i;
                            tcgen05_mma_block_scaled<KIND, CTAS>(tmem_base, adesc + 2 * i, bdesc + 2 * i,
                                                                 instr_desc<KIND, CTAS>(sf_id, sf_id), sf_tmem + 4 * chunk,
                                                                 sf_tmem + 8 + 8 * chunk, (it > 0 || i > 0) ? 1u : 0u);
                        }
                    }
                    tcgen05_commit<CTAS>(bar_empty + 8 * stage);
                    if (it == n_it - 1) tcgen05_commit<CTAS>(bar_acc_full);
                    if ((it & (kUnitStages - 1)) == kUnitStages - 1 || it == n_it - 1)
                        tcgen05_commit<CTAS>(bar_cache_empty + 8 * ring.buf);   // the unit's images have been copied
                }
                if ((it & (kUnitStages - 1)) == kUnitStages - 1 || it == n_it - 1) ring.next(kImageBufs);
                TRACE_ADD(c_issue, tt);
                if (lane == 0) TRACE_EV(3, ev_j);
                ev_j++;
                if (++stage == kStages) { stage = 0; full_phase ^= 1u; }
            }
        }
        if (leader && *abort_flag) {
            // Some role gave up: the watchers then release every remaining stage unseen, and this warp has run
            // through them.  Wait (bounded) until the tensor pipe is idle before tensor memory is freed.
            if (issuer) tcgen05_commit<CTAS>(bar_drain);
            __syncwarp();
            if (lane == 0) mbar_wait_lazy(bar_drain, 0u, abort_flag, p.status, wait_limit, 0x220u);   // gives up after 256 polls (abort is set)
            __syncwarp();
            // After an abort the stages were consumed without waiting for their operands, so loads of either CTA may
            // still be on their way: hold the pair (the other roles wait at the final barrier) until they have landed.
            for (int i = 0; i < 200; i++) __nanosleep(1000);
        }
        if (lane == 0) { TRACE_OUT(p, 2, c_acc); TRACE_OUT(p, 3, c_sync); TRACE_OUT(p, 4, c_issue); }
    } else if (warp == 3) {
        // ------------------------------------------------------------------ scale image builder
        // 2D-block scales: per unit (up to 16 stages of one tile) gathers the compact scale bytes from global memory
        // into 16-byte rows and replicates each row into its image; per-row scales: loads the unit's scale words and
        // writes the 32-row images directly.  Two image buffers alternate, so the next unit is built while
        // the current one runs: all global-memory latency of the scale path is paid here, off the per-stage
        // critical path, and nothing has to be written per stage.  A buffer is free again once the MMA warp's
        // commit reports that the last scale copy out of it has completed.  In a pair each CTA builds the images
        // of its own 128 A rows and of all 256 B rows.
        BufRing ring;
        bool ok = true;
        if (KIND != KIND_MXF4) {
            // per-row scales: the raw bytes of the next kRawBufs units are in flight (cp.async) while a unit is
            // turned into images.  In a pair an image buffer is released by the leader's multicast commit: probe
            // (a suspended try_wait is not reliably woken early by a remote arrival).
            constexpr int kRawBufs = Cfg<KIND, CTAS>::kRawBufs > 0 ? Cfg<KIND, CTAS>::kRawBufs : 1;
            UnitIter ahead, cur;
            ahead.init(p, first_tile, tile_step, rank, goffs);
            cur.init(p, first_tile, tile_step, rank, goffs);
            uint32_t raw_fill = 0, raw_read = 0;
            for (int i = 0; i < kRawBufs; i++) {
                if (ahead.valid(p)) {
                    issue_raw_scales<kKbShift>(p, ahead.t, ahead.k0, smem_raw_scales + raw_fill * kCacheBufBytes, lane);
                    ahead.next(p, kUnitStages * kStageElems);
                } else {
                    asm volatile("cp.async.commit_group;" ::: "memory");
                }
                if (++raw_fill == kRawBufs) raw_fill = 0;
            }
            while (cur.valid(p)) {
                asm volatile("cp.async.wait_group %0;" ::"n"(kRawBufs - 1) : "memory");   // this unit's bytes have landed
                __syncwarp();
                uint32_t w[12][8];
                read_raw_scales(p, smem_raw_scales + raw_read * kCacheBufBytes, lane, w);
                if (lane == 0)
                    ok = mbar_wait_impl<kRelaxedNs, CTAS == 2>(bar_cache_empty + 8 * ring.buf, ring.phase ^ 1u, abort_flag, p.status, wait_limit, 0x500u + ring.buf);
                ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
                if (!ok) break;
                store_row_scale_images<KIND>(w, min(kUnitStages, (cur.t.k_len - cur.k0 + kStageElems - 1) / kStageElems),
                                             smem_images + ring.buf * kCacheBufBytes, lane);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> tcgen05.cp
                __syncwarp();
                // In the second CTA of a pair the arrival is forwarded to the leader by warp 2: the remote arrival
                // stalls its issuing thread for about a thousand cycles, which this warp spends on the next unit.
                if (lane == 0) mbar_arrive(bar_cache_full + 8 * ring.buf);
                ring.next(kImageBufs);
                cur.next(p, kUnitStages * kStageElems);
                // the raw buffer just read is free: fetch the unit kRawBufs ahead into it
                if (ahead.valid(p)) {
                    issue_raw_scales<kKbShift>(p, ahead.t, ahead.k0, smem_raw_scales + raw_read * kCacheBufBytes, lane);
                    ahead.next(p, kUnitStages * kStageElems);
                } else {
                    asm volatile("cp.async.commit_group;" ::: "memory");
                }
                if (++raw_read == kRawBufs) raw_read = 0;
            }
            asm volatile("cp.async.wait_all;" ::: "memory");
        }
        for (int tile = first_tile; KIND == KIND_MXF4 && ok && tile < p.n_tile_total; tile += tile_step) {
            Tile t;
            decode_tile(p, tile, rank, t, goffs);
            for (int k0 = 0; ok && k0 < t.k_len; k0 += kUnitStages * kStageElems, ring.next(kImageBufs)) {
                const int buf = ring.buf;
                uint8_t *images = smem_images + buf * kCacheBufBytes;
                {
                    const int n_chunks = min(kCacheChunks, (((t.k_len - k0 + 127) >> 7) + 1) & ~1);   // whole stages; pad rows beyond the tensor
                    uint32_t *compact = reinterpret_cast<uint32_t *>(smem_compact);
                    build_scale_cache(p.sfa, t.a_row0 >> 5, ((t.a_k0 + k0) >> 5), n_chunks, 2, compact, lane);
                    build_scale_cache(p.sfb, t.b_row0 >> 5, ((t.b_k0 + k0) >> 5), n_chunks, 3, compact + kCacheChunks * 4, lane);
                    __syncwarp();
                    if (lane == 0)
                        ok = CTAS == 2 ? mbar_poll_relaxed(bar_cache_empty + 8 * buf, ring.phase ^ 1u, abort_flag, p.status, wait_limit, 0x500u + buf)
                                       : mbar_wait_relaxed(bar_cache_empty + 8 * buf, ring.phase ^ 1u, abort_flag, p.status, wait_limit, 0x500u + buf);
                    ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
                    if (!ok) break;
                    const uint4 *rows = reinterpret_cast<const uint4 *>(smem_compact);
                    for (int q = lane; q < 3 * n_chunks; q += 32) {
                        uint4 row;
                        uint8_t *dst;
                        if (q < n_chunks) {                       // A, chunk q
                            row = rows[q];
                            dst = images + (q >> 1) * kImageStageBytes + (q & 1) * 128;
                        } else {                                  // B, chunk (q - n_chunks) / 2, rows 0..127 or 128..255
                            const int qb = q - n_chunks, chunk = qb >> 1;
                            row = rows[kCacheChunks + qb];
                            dst = images + (chunk >> 1) * kImageStageBytes + 256 + (chunk & 1) * 256 + (qb & 1) * 128;
                        }
#pragma unroll
                        for (int r = 0; r < 8; r++) reinterpret_cast<uint4 *>(dst)[r] = row;
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> tcgen05.cp
                __syncwarp();
                if (lane == 0) {   // 16-stage units leave time for the second CTA's own (slow) remote arrival
                    if (CTAS == 1 || leader) mbar_arrive(bar_cache_full + 8 * buf);
                    else mbar_arrive_cluster_release(cluster_addr(bar_peer_cache_full + 8 * buf, 0));
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ watcher
        // Follows the stream of stages (one CTA, or the leader of a pair; the second CTA's warp idles).  For each
        // it waits for the ring slot's "full" barrier (the operand bytes of both CTAs), at the first stage of a
        // unit for the unit's scale images (of both CTAs), and at the first stage of a tile for the accumulator
        // to be drained; then it meets the MMA warp at the slot's named barrier.  After a timeout every remaining
        // stage is released unseen, so that the MMA warp, which cannot time out on a named barrier, always runs
        // to its end.
        StageIter sg;
        sg.init(p, first_tile, tile_step, rank, kStageElems, goffs, false);
        uint32_t stage = 0, phase = 0, acc_phase = 0;
        BufRing ring;   // image buffer of the current unit
        bool ok = true;
        TRACE_DECL(c_meet); TRACE_DECL(c_poll);
        TRACE_T0(tt);
        int ev_j = 0;
        bool unit_seen = false;   // lane 0: the next unit's scale images have been seen complete
        uint32_t ahead = 0;   // stages after the current one whose "full" barrier is already known to be complete
        if (Cfg<KIND, CTAS>::kSplitProducer) {
            // poller half of the split producer: waits for each slot to be free, arms its barrier for the stage's bytes and
            // releases the issuing warp; after a timeout it keeps releasing, so that warp 0 always reaches its end
            while (sg.valid(p)) {
                if (lane == 0) {
                    if (ok) ok = mbar_wait_impl<0, true>(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status, wait_limit, 0x100u + stage);
                    mbar_arrive_expect_tx(bar_full + 8 * stage, kAStageBytes + kBStageBytes);
                }
                __syncwarp();
                asm volatile("bar.sync %0, 64;" ::"r"(8 + stage) : "memory");
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
                sg.next(p, kStageElems);
            }
        }
        while (!Cfg<KIND, CTAS>::kSplitProducer && leader && sg.valid(p)) {
            if (lane == 0) TRACE_EV(4, ev_j);
            if (ahead > 0) {
                ahead--;
            } else {
                if (ok && lane == 0) {
                    if ((sg.it & (kUnitStages - 1)) == 0 && !unit_seen) {
                        // both CTAs' images of this unit: the two barriers probed together (the latencies overlap)
                        const uint32_t b0 = bar_cache_full + 8 * ring.buf, b1 = (CTAS == 2 ? bar_peer_cache_full : bar_cache_full) + 8 * ring.buf;
                        for (uint32_t spin = 0; ; spin++) {
                            uint32_t q0, q1;
                            asm volatile("{\n .reg .pred p0, p1;\n"
                                         " mbarrier.test_wait.parity.shared::cta.b64 p0, [%2], %4;\n"
                                         " mbarrier.test_wait.parity.shared::cta.b64 p1, [%3], %4;\n"
                                         " selp.b32 %0, 1, 0, p0;\n selp.b32 %1, 1, 0, p1;\n}"
                                         : "=r"(q0), "=r"(q1) : "r"(b0), "r"(b1), "r"(ring.phase) : "memory");
                            if (q0 && q1) break;
                            if (spin >= wait_limit) {
                                ok = false;
                                *abort_flag = 1u;
                                if (atomicCAS(p.status, 0u, (uint32_t)FP4Q_ERR_TIMEOUT) == 0u) p.status[1] = (q0 ? 0x520u : 0x510u) + ring.buf;
                                break;
                            }
                            if ((spin & 255u) == 255u && *abort_flag) { ok = false; break; }
                        }
                    }
                    if ((sg.it & (kUnitStages - 1)) == 0) unit_seen = false;
                    // Whether the next unit's images are in place is looked up ahead of time, so that a unit boundary
                    // costs no extra probe on the critical path: with short units (per-row scales) the two barriers
                    // ride along with every probe of the ring slots below; with 16-stage units one look in the second
                    // half of the unit is enough, and the slot probes stay as light as they can be.
                    BufRing nu = ring;
                    nu.next(kImageBufs);
                    const uint32_t nb0 = bar_cache_full + 8 * nu.buf, nb1 = (CTAS == 2 ? bar_peer_cache_full : bar_cache_full) + 8 * nu.buf;
                    if (KIND == KIND_MXF4 && ok && (sg.it & (kUnitStages - 1)) >= kUnitStages / 2 && !unit_seen)
                        unit_seen = mbar_test_wait(nb0, nu.phase) && (CTAS == 1 || mbar_test_wait(nb1, nu.phase));
                    if (ok && sg.it == 0) ok = mbar_wait_impl<0, true>(bar_acc_empty, acc_phase ^ 1u, abort_flag, p.status, wait_limit, 0x200u);
                    if (ok) {
                        // A probe of an mbarrier takes this warp a few hundred cycles even when the phase is long
                        // complete, more than the MMA warp needs per stage.  So the slot's "full" barrier and those of
                        // the next three slots are probed in one go (the latencies overlap); slots found complete are
                        // handed over later without another look.  Only stages of the same unit qualify: they need
                        // nothing but their "full" barrier.
                        const int left = min(kUnitStages - 1 - (sg.it & (kUnitStages - 1)), sg.n_it - 1 - sg.it);
                        uint32_t sl[4], ph[4];
                        sl[0] = stage; ph[0] = phase;
#pragma unroll
                        for (int q = 1; q < 4; q++) {
                            sl[q] = sl[q - 1] + 1 == kStages ? 0u : sl[q - 1] + 1;
                            ph[q] = sl[q] == 0 ? ph[q - 1] ^ 1u : ph[q - 1];
                        }
                        uint32_t r0 = 0, r1 = 0, r2 = 0, r3 = 0, r4 = 0, r5 = 0;
                        for (uint32_t spin = 0; ; spin++) {
                            if (KIND == KIND_MXF4)
                                asm volatile("{\n .reg .pred p0, p1, p2, p3;\n"
                                             " mbarrier.test_wait.parity.shared::cta.b64 p0, [%4], %5;\n"
                                             " mbarrier.test_wait.parity.shared::cta.b64 p1, [%6], %7;\n"
                                             " mbarrier.test_wait.parity.shared::cta.b64 p2, [%8], %9;\n"
                                             " mbarrier.test_wait.parity.shared::cta.b64 p3, [%10], %11;\n"
                                             " selp.b32 %0, 1, 0, p0;\n selp.b32 %1, 1, 0, p1;\n selp.b32 %2, 1, 0, p2;\n selp.b32 %3, 1, 0, p3;\n}"
                                             : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                                             : "r"(bar_full + 8 * sl[0]), "r"(ph[0]), "r"(bar_full + 8 * sl[1]), "r"(ph[1]),
                                               "r"(bar_full + 8 * sl[2]), "r"(ph[2]), "r"(bar_full + 8 * sl[3]), "r"(ph[3]) : "memory");
                            else
                            asm volatile("{\n .reg .pred p0, p1, p2, p3, p4, p5;\n"
                                         " mbarrier.test_wait.parity.shared::cta.b64 p0, [%6], %7;\n"
                                         " mbarrier.test_wait.parity.shared::cta.b64 p1, [%8], %9;\n"
                                         " mbarrier.test_wait.parity.shared::cta.b64 p2, [%10], %11;\n"
                                         " mbarrier.test_wait.parity.shared::cta.b64 p3, [%12], %13;\n"
                                         " mbarrier.test_wait.parity.shared::cta.b64 p4, [%14], %16;\n"
                                         " mbarrier.test_wait.parity.shared::cta.b64 p5, [%15], %16;\n"
                                         " selp.b32 %0, 1, 0, p0;\n selp.b32 %1, 1, 0, p1;\n selp.b32 %2, 1, 0, p2;\n selp.b32 %3, 1, 0, p3;\n"
                                         " selp.b32 %4, 1, 0, p4;\n selp.b32 %5, 1, 0, p5;\n}"
                                         : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3), "=r"(r4), "=r"(r5)
                                         : "r"(bar_full + 8 * sl[0]), "r"(ph[0]), "r"(bar_full + 8 * sl[1]), "r"(ph[1]),
                                           "r"(bar_full + 8 * sl[2]), "r"(ph[2]), "r"(bar_full + 8 * sl[3]), "r"(ph[3]),
                                           "r"(nb0), "r"(nb1), "r"(nu.phase) : "memory");
                            if (r0) break;
                            if (spin >= wait_limit) {
                                ok = false;
                                *abort_flag = 1u;
                                if (atomicCAS(p.status, 0u, (uint32_t)FP4Q_ERR_TIMEOUT) == 0u) p.status[1] = 0x300u + stage;
                                break;
                            }
                            if ((spin & 255u) == 255u && *abort_flag) { ok = false; break; }
                        }
                        ahead = !ok ? 0u : (left >= 1 && r1) ? ((left >= 2 && r2) ? ((left >= 3 && r3) ? 3u : 2u) : 1u) : 0u;
                        if (r4 && r5) unit_seen = true;
                    }
                }
                ahead = __shfl_sync(0xFFFFFFFFu, ahead, 0);
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
            TRACE_ADD(c_poll, tt);
            if (lane == 0) TRACE_EV(6, ev_j);
            ev_j++;
            named_sync(1 + stage);   // rendezvous: the MMA warp is at most one stage behind
            TRACE_ADD(c_meet, tt);
            if (sg.it == 0) acc_phase ^= 1u;
            if ((sg.it & (kUnitStages - 1)) == kUnitStages - 1 || sg.it == sg.n_it - 1) ring.next(kImageBufs);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
            sg.next(p, kStageElems);
        }
        if (KIND != KIND_MXF4 && CTAS == 2 && !leader && lane == 0) {
            // Per-row scales, second CTA of a pair: report each unit of scale images the builder has finished to the
            // leader, which issues the scale copies of both CTAs.
            bool fwd_ok = true;
            BufRing fr;
            UnitIter un;
            for (un.init(p, first_tile, tile_step, rank, goffs); fwd_ok && un.valid(p); un.next(p, kUnitStages * kStageElems), fr.next(kImageBufs)) {
                fwd_ok = mbar_wait_impl<kRelaxedNs>(bar_cache_full + 8 * fr.buf, fr.phase, abort_flag, p.status, wait_limit, 0x530u + fr.buf);
                if (fwd_ok) mbar_arrive_cluster_release(cluster_addr(bar_peer_cache_full + 8 * fr.buf, 0));
            }
        }
        __syncwarp();
        if (lane == 0) { TRACE_OUT(p, 6, c_meet); TRACE_OUT(p, 7, c_poll); }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue
        const int quarter = warp & 3;            // TMEM lanes 32*quarter .. +31 (hardware: warp id mod 4)
        const int half = (warp - 4) >> 2;        // accumulator columns 128*half .. +127
        uint32_t acc_phase = 0;
        bool ok = true;
        int ev_t = 0;
        TRACE_DECL(c_wait); TRACE_DECL(c_ld); TRACE_DECL(c_store);
        TRACE_T0(tt);
        for (int tile = first_tile; ok && tile < p.n_tile_total; tile += tile_step) {
            Tile t;
            decode_tile(p, tile, rank, t, goffs, false);
            const int row_in_tile = 32 * quarter + lane;
            const int64_t row = (int64_t)t.c_row0 + row_in_tile;
            const bool row_ok = row_in_tile < t.m_valid;
            uint32_t v[4][32];
            if (t.k_len > 0) {
                // this wait spans a whole tile (every other one spans a few stages at most): its limit grows with the
                // tile's contraction length, so that a very long contraction cannot run into it on a healthy run
                const uint64_t tile_limit = wait_limit * (uint64_t)(1 + (t.k_len >> 12));
                if (lane == 0)
                    ok = CTAS == 2 ? mbar_poll(bar_acc_full, acc_phase, abort_flag, p.status, tile_limit, 0x400u + warp)
                                   : mbar_wait_relaxed(bar_acc_full, acc_phase, abort_flag, p.status, tile_limit, 0x400u + warp);
                ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
                TRACE_ADD(c_wait, tt);
                if (lane == 0) TRACE_EV(7, 16 * ev_t + 2 * (warp - 4));
                if (!ok) break;
                acc_phase ^= 1u;
                tcgen05_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(32 * quarter) << 16) + 128u * half;
                FP4Q_TMEM_LD_X32(taddr, v[0]);
                FP4Q_TMEM_LD_X32(taddr + 32, v[1]);
                FP4Q_TMEM_LD_X32(taddr + 64, v[2]);
                FP4Q_TMEM_LD_X32(taddr + 96, v[3]);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) {   // the accumulator now lives in registers; the leader's MMA thread waits for both CTAs
                    if (CTAS == 1 || leader) mbar_arrive(bar_acc_empty);
                    else mbar_arrive_cluster(cluster_addr(bar_acc_empty, 0));
                }
                TRACE_ADD(c_ld, tt);
                if (lane == 0) TRACE_EV(7, 16 * ev_t + 2 * (warp - 4) + 1);
                ev_t++;
            } else {
#pragma unroll
                for (int j = 0; j < 4; j++)
#pragma unroll
                    for (int q = 0; q < 32; q++) v[j][q] = 0u;
            }
            if (EPI == EPI_QUANT) {
                // The output tile leaves as 2D-block FP4: each warp owns four 32x32 blocks (its 32 rows x 32 columns
                // per chunk).  The accumulator is rounded to BF16 first, so the result equals fp4q_quantize2d applied
                // to the BF16 output of the plain product: block maximum over the warp, truncation-free scale, E2M1
                // codes by the same converts, row-major payload from the lane's own row, transposed payload by a
                // 32x32 nibble transpose across the warp's lanes; both leave through the staging rows and TMA stores.
                const int64_t row_g = (int64_t)t.c_row0 + row_in_tile;
                const int row0_blk = t.c_row0 + 32 * quarter;
                // staging: 32 rows x 64 B of row-major payload (64-byte swizzle) and 128 rows x 16 B of transposed payload
                uint8_t *stg = smem_staging + (warp - 4) * kStagingWarpBytes;
                const uint32_t stg_rm = smem_u32(stg) + lane * 64, swz = (uint32_t)((lane >> 1) & 3);
                const uint32_t stg_t = smem_u32(stg) + 2048 + lane * 16;
                const bool any = row0_blk < p.M && t.c_col0 + 128 * half < p.N;   // warp-uniform: something to write
                if (any) {
                    if (lane == 0) bulk_wait_read_all();   // the previous tile's stores have read the staging rows
                    __syncwarp();
                }
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const int col0 = t.c_col0 + 128 * half + 32 * j;
                    if (col0 >= p.N || row0_blk >= p.M) continue;   // warp-uniform
                    uint32_t raw[16], mx = 0;
                    bool nonfinite = false;
#pragma unroll
                    for (int e = 0; e < 16; e++) {
                        const __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(v[j][2 * e]), __uint_as_float(v[j][2 * e + 1]));
                        raw[e] = *reinterpret_cast<const uint32_t *>(&b);
                        const uint32_t m0 = raw[e] & 0x7FFFu, m1 = (raw[e] >> 16) & 0x7FFFu;
                        nonfinite |= m0 >= 0x7F80u || m1 >= 0x7F80u;
                        mx = max(mx, max(m0 >= 0x7F80u ? 0u : m0, m1 >= 0x7F80u ? 0u : m1));
                    }
                    mx = __reduce_max_sync(0xFFFFFFFFu, mx);
                    nonfinite = __any_sync(0xFFFFFFFFu, nonfinite);
                    const int code = scale_code_from_max(mx);
                    uint32_t W[4];
#pragma unroll
                    for (int sg = 0; sg < 2; sg++) {
                        uint32_t R[4] = {0u, 0u, 0u, 0u};
                        if (p.q_mode == FP4Q_ROUND_STOCHASTIC) {
                            const uint64_t blk = (uint64_t)(row_g * p.N + col0 + 16 * sg) >> 4;   // N % 16 == 0
                            philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), p.q_tensor_id, 0u, p.q_keys, R);
                        }
                        if (nonfinite) {
                            const uint4 lo = make_uint4(raw[8 * sg], raw[8 * sg + 1], raw[8 * sg + 2], raw[8 * sg + 3]);
                            const uint4 hi = make_uint4(raw[8 * sg + 4], raw[8 * sg + 5], raw[8 * sg + 6], raw[8 * sg + 7]);
                            const uint4 rn = make_uint4(R[0], R[1], R[2], R[3]);
                            const uint2 w = p.q_mode == FP4Q_ROUND_STOCHASTIC
                                                ? round_segment_scalar<FP4Q_ROUND_STOCHASTIC>(lo, hi, rn, inv_scale_f16_aligned(code))
                                                : round_segment_scalar<FP4Q_ROUND_NEAREST>(lo, hi, rn, inv_scale_f16_aligned(code));
                            W[2 * sg] = w.x;
                            W[2 * sg + 1] = w.y;
                        } else if (p.q_mode == FP4Q_ROUND_STOCHASTIC) {
                            round_segment<FP4Q_ROUND_STOCHASTIC>(raw + 8 * sg, inv_scale(code), R, W + 2 * sg);
                        } else {
                            round_segment<FP4Q_ROUND_NEAREST>(raw + 8 * sg, inv_scale(code), R, W + 2 * sg);
                        }
                    }
                    if (lane == 0) p.q_scale[(int64_t)(row0_blk >> 5) * p.q_ld_s + (col0 >> 5)] = (uint8_t)code;
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg_rm + (((uint32_t)j ^ swz) << 4)), "r"(W[0]), "r"(W[1]),
                                 "r"(W[2]), "r"(W[3]) : "memory");
                    if (p.q_t != nullptr) {
                        transpose32x32_nibbles(W, lane);   // lane c now holds column c: nibble r = row r of the block
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg_t + 512u * j), "r"(W[0]), "r"(W[1]), "r"(W[2]),
                                     "r"(W[3]) : "memory");
                    }
                }
                if (any) {
                    // both payloads leave by TMA stores, which clip at the tensors' edges (rows past T, columns past N)
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tmC, (t.c_col0 + 128 * half) >> 1, row0_blk, smem_u32(stg));
                        if (p.q_t != nullptr) tma_store_2d(&tmD, row0_blk >> 1, t.c_col0 + 128 * half, smem_u32(stg) + 2048);
                        bulk_commit();
                    }
                }
            } else if (Cfg<KIND, CTAS>::kTmaStores) {
                // 128 bytes per row and round - 64 BF16 or 32 FP32 columns - go
                // through this warp's staging rows and leave by a TMA store, which clips rows and columns past the
                // output's edge.  With accumulation the store is the TMA's FP32 add-reduction.
                if (t.m_valid > 32 * quarter) {
                    uint8_t *stg = smem_staging + (warp - 4) * kStagingWarpBytes;
                    const uint32_t stg_row = smem_u32(stg) + lane * 128, swz = (uint32_t)(lane & 7);
                    const int32_t y = t.c_row0 + 32 * quarter;
                    if (p.out_f32) {
#pragma unroll
                        for (int h = 0; h < 4; h++) {
                            const int col_in_tile = 128 * half + 32 * h;
                            if (col_in_tile < t.n_valid)
                                stage_and_store(&tmC, v[h], stg_row, swz, smem_u32(stg), t.c_col0 + col_in_tile, y, p.accumulate ? 2 : 1, lane);
                        }
                    } else {
#pragma unroll
                        for (int h = 0; h < 2; h++) {
                            const int col_in_tile = 128 * half + 64 * h;
                            if (col_in_tile >= t.n_valid) continue;
                            uint32_t w[32];
#pragma unroll
                            for (int e = 0; e < 32; e++) {
                                const __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(v[2 * h + (e >> 4)][(2 * e) & 31]),
                                                                               __uint_as_float(v[2 * h + (e >> 4)][(2 * e + 1) & 31]));
                                w[e] = *reinterpret_cast<const uint32_t *>(&b);
                            }
                            stage_and_store(&tmC, w, stg_row, swz, smem_u32(stg), t.c_col0 + col_in_tile, y, 0, lane);
                        }
                    }
                }
            } else if (row_ok) {
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const int col_in_tile = 128 * half + 32 * j;
                    store_row_chunk(p, row, t.c_col0 + col_in_tile, t.n_valid - col_in_tile, v[j]);
                }
            }
            TRACE_ADD(c_store, tt);
        }
        if ((Cfg<KIND, CTAS>::kTmaStores || EPI == EPI_QUANT) && lane == 0) bulk_wait_all();   // every store of this warp is complete before the CTA ends
        if (warp == 4 && lane == 0) { TRACE_OUT(p, 10, c_wait); TRACE_OUT(p, 11, c_ld); TRACE_OUT(p, 12, c_store); }
    }

    tcgen05_fence_before();
    __syncwarp();
    if (CTAS == 2) cluster_sync_all();   // the peer's shared memory and tensor memory stay alive until the pair is done
    else __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        if (CTAS == 1)
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// Operand tile map: a [rows, row_bytes] byte matrix with pitch ld_bytes, box = 128 B x box_rows, 128B swizzle.
static bool make_operand_map(CUtensorMap *map, const void *base, int64_t rows, int64_t row_bytes, int64_t ld_bytes,
                             int box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld_bytes};
    const cuuint32_t box[2] = {128u, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Output map for the pair kernel's TMA stores: box = 128 bytes x 32 rows, 128-byte swizzle.  Plain stores address the
// output as bytes; accumulation uses the TMA add-reduction, which needs the element type (FP32, 32 per box row).
static bool make_output_map(CUtensorMap *map, void *base, int64_t rows, int64_t cols, int64_t ld, bool f32, bool reduce)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const int64_t esize = f32 ? 4 : 2;
    const cuuint64_t dims[2] = {(cuuint64_t)(reduce ? cols : cols * esize), (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)(ld * esize)};
    const cuuint32_t box[2] = {reduce ? 32u : 128u, 32u};
    const cuuint32_t estr[2] = {1u, 1u};
    return fn(map, reduce ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Plain byte matrix [rows, row_bytes] with pitch ld_bytes as a store target.
static bool make_byte_map(CUtensorMap *map, void *base, int64_t rows, int64_t row_bytes, int64_t ld_bytes, int box_bytes,
                          int box_rows, CUtensorMapSwizzle swizzle)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)box_bytes, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
              CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Operand {
    const uint8_t *payload;
    int64_t rows, row_bytes, ld_bytes;
    ScaleView sf;
};

constexpr int kMaxDevices = 64;   // per-device host state (attributes set, SM counts, static workspace address)

static int current_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

static int sm_count(int dev)
{
    static int n[kMaxDevices];
    if (n[dev] == 0 && (cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n[dev] <= 0)) n[dev] = 148;
    return n[dev];
}

template <int KIND, int CTAS, int EPI = EPI_STORE>
static fp4q_status launch_gemm_impl(const Operand &A, const Operand &B, GemmParams &p, void *stream)
{
    CUtensorMap tmA, tmB, tmC;
    const int64_t out_rows = p.mode == MODE_GROUPED_K ? (int64_t)p.n_groups * p.M : p.M;
    if (!make_operand_map(&tmA, A.payload, A.rows, A.row_bytes, A.ld_bytes, BM)) return FP4Q_ERR_CUDA;
    CUtensorMap tmD = tmA;   // second output map: only the quantizing epilogue has one
    if (EPI == EPI_QUANT) {
        // row-major payload [T, ceil32(N)/2] bytes, box 64 B x 32 rows (64-byte swizzle); transposed payload
        // [N, ceil32(T)/2] bytes, box 16 B x 128 rows
        if (!make_byte_map(&tmC, p.q_rm, p.M, round_up(p.N, 32) / 2, p.q_ld_rm, 64, 32, CU_TENSOR_MAP_SWIZZLE_64B)) return FP4Q_ERR_CUDA;
        if (p.q_t && !make_byte_map(&tmD, p.q_t, p.N, round_up(p.M, 32) / 2, p.q_ld_t, 16, 128, CU_TENSOR_MAP_SWIZZLE_NONE)) return FP4Q_ERR_CUDA;
    } else if (!make_output_map(&tmC, p.C, out_rows, p.N, p.ldc, p.out_f32 != 0, p.accumulate != 0)) return FP4Q_ERR_CUDA;
    if (!make_operand_map(&tmB, B.payload, B.rows, B.row_bytes, B.ld_bytes, Cfg<KIND, CTAS>::kBRows)) return FP4Q_ERR_CUDA;
    p.ctas = CTAS;
    p.m_tiles = (int32_t)ceil_div(p.M, BM * CTAS);
    p.n_tile_total = p.m_tiles * p.n_tiles * (p.mode == MODE_GROUPED_K ? p.n_groups : 1);
    p.raster_m = p.mode == MODE_DENSE ? (p.m_tiles < kRasterM ? p.m_tiles : kRasterM) : p.m_tiles;
#ifdef FP4Q_TRACE
    if (const char *g = getenv("FP4Q_DEBUG_RASTER")) { p.raster_m = atoi(g); if (p.raster_m > p.m_tiles) p.raster_m = p.m_tiles; }
#endif

    const int dev = current_device();
    if (dev < 0) return FP4Q_ERR_CUDA;
    static bool attr_set[kMaxDevices];   // the attribute is a property of (kernel, device): one flag per device and instantiation
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(gemm_block_scaled_kernel<KIND, CTAS, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 Cfg<KIND, CTAS>::kSmemBytes) != cudaSuccess)
            return FP4Q_ERR_CUDA;
        attr_set[dev] = true;
    }
    int slots = sm_count(dev) / CTAS;
#ifdef FP4Q_TRACE
    if (const char *g = getenv("FP4Q_DEBUG_SLOTS")) slots = atoi(g);   // development only: use fewer SMs
#endif
    const int grid = CTAS * (p.n_tile_total < slots ? p.n_tile_total : slots);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = Cfg<KIND, CTAS>::kSmemBytes;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CTAS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = CTAS == 2 ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, gemm_block_scaled_kernel<KIND, CTAS, EPI>, tmA, tmB, tmC, tmD, p) == cudaSuccess ? FP4Q_OK : FP4Q_ERR_CUDA;
}

// Argument checks common to every product: everything that can be refused is refused here, before any work is enqueued.
static fp4q_status check_gemm_args(const Operand &A, const Operand &B, const GemmParams &p, const void *ws, size_t ws_bytes)
{
    if (!ws || ws_bytes < sizeof(Workspace)) return FP4Q_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return FP4Q_ERR_ALIGN;
    if (!aligned(A.payload, 16) || !aligned(B.payload, 16) || A.ld_bytes % 16 || B.ld_bytes % 16) return FP4Q_ERR_ALIGN;
    const size_t esize = p.out_f32 ? 4 : 2;
    if (!aligned(p.C, 16) || (p.ldc * esize) % 16) return FP4Q_ERR_ALIGN;
    return FP4Q_OK;
}

template <int KIND>
static fp4q_status launch_gemm(const Operand &A, const Operand &B, GemmParams &p, void *ws, size_t ws_bytes, void *stream)
{
    if (fp4q_status s = check_gemm_args(A, B, p, ws, ws_bytes)) return s;
    const size_t esize = p.out_f32 ? 4 : 2;
    if (p.n_tile_total <= 0) return FP4Q_OK;
    p.wide_stores = aligned(p.C, 32) && (p.ldc * esize) % 32 == 0;
    p.sfa = A.sf;
    p.sfb = B.sf;
    p.status = reinterpret_cast<uint32_t *>(ws);
    // Dense products (FP4 and MXFP8) with more than one row tile run as cta_group::2 pairs: 256x256 tiles, each CTA
    // loads half of the B rows; so does the grouped weight gradient, whose groups cut the contraction axis, not the
    // output rows of a tile.  FP4Q_CTA_PAIRS=0 in the environment (read once, before the first GEMM call) selects
    // the one-CTA kernel instead; grouped forward / input-gradient products use one CTA per 128x256 tile unless the
    // caller states that every token group starts on a multiple of 256 rows.
    static const bool use_pairs = [] { const char *e = getenv("FP4Q_CTA_PAIRS"); return !(e && e[0] == '0'); }();
    const bool pair_mode = p.mode == MODE_DENSE || p.mode == MODE_GROUPED_K || (p.mode == MODE_GROUPED_ROWS && p.rows_pair_aligned);
    if (use_pairs && pair_mode && p.M > BM) return launch_gemm_impl<KIND, 2>(A, B, p, stream);
    return launch_gemm_impl<KIND, 1>(A, B, p, stream);
}

static bool tensor_ok(const fp4q_tensor *t) { return t && t->rows >= 0 && t->cols >= 0; }

static fp4q_status check_groups(const fp4q_groups *g)
{
    if (!g) return FP4Q_OK;
    if (g->n_groups <= 0) return FP4Q_ERR_SHAPE;
    if (g->row_alignment != 0 && g->row_alignment != 128 && g->row_alignment != 256) return FP4Q_ERR_UNSUPPORTED;
    if (!g->row_offsets) return FP4Q_ERR_NULL;
    return FP4Q_OK;
}

// Row-major payload of a tensor [rows, cols] as an operand whose rows are the tensor's rows.
static Operand operand_rm(const fp4q_tensor *t)
{
    Operand o;
    o.payload = t->q_rm;
    o.rows = t->rows;
    o.row_bytes = round_up(t->cols, 32) / 2;
    o.ld_bytes = t->ld_rm;
    o.sf = ScaleView{t->scale, t->ld_s, 1, (int32_t)ceil_div(t->rows, 32), (int32_t)ceil_div(t->cols, 32)};
    return o;
}
// Transposed payload: operand rows are the tensor's columns, contraction runs over the tensor's rows.
static Operand operand_t(const fp4q_tensor *t)
{
    Operand o;
    o.payload = t->q_t;
    o.rows = t->cols;
    o.row_bytes = round_up(t->rows, 32) / 2;
    o.ld_bytes = t->ld_t;
    o.sf = ScaleView{t->scale, 1, t->ld_s, (int32_t)ceil_div(t->cols, 32), (int32_t)ceil_div(t->rows, 32)};
    return o;
}

static void dense_tiles(GemmParams &p)
{
    p.m_tiles = (int32_t)ceil_div(p.M, BM);
    p.n_tiles = (int32_t)ceil_div(p.N, BN);
    p.n_tile_total = p.m_tiles * p.n_tiles;
}

}  // namespace fp4q

using namespace fp4q;

static const int64_t kMaxDim = 0x7FFFFFFF - 4096;

// The forward product's arguments turned into kernel parameters.  *noop is set when there is nothing to compute.
static fp4q_status prepare_fwd(const fp4q_tensor *X, const fp4q_tensor *W, void *Y, int64_t ldy, fp4q_out dt, const fp4q_groups *g,
                               GemmParams &p, bool *noop)
{
    *noop = false;
    if (!tensor_ok(X) || !tensor_ok(W)) return X && W ? FP4Q_ERR_SHAPE : FP4Q_ERR_NULL;
    if (fp4q_status s = check_groups(g)) return s;
    if (dt != FP4Q_OUT_BF16 && dt != FP4Q_OUT_F32) return FP4Q_ERR_UNSUPPORTED;
    if (X->cols != W->cols) return FP4Q_ERR_SHAPE;
    const int64_t T = X->rows, K = X->cols;
    const int64_t N = g ? W->rows / g->n_groups : W->rows;
    if (g && (W->rows % g->n_groups || N % 32)) return FP4Q_ERR_SHAPE;   // expert blocks must start on a 32-row tile
    if (T > kMaxDim || N > kMaxDim || K > kMaxDim || W->rows > kMaxDim) return FP4Q_ERR_UNSUPPORTED;
    if (T == 0 || N == 0) { *noop = true; return FP4Q_OK; }
    if (!Y || !X->q_rm || !W->q_rm || !X->scale || !W->scale) return FP4Q_ERR_NULL;
    if (ldy < N) return FP4Q_ERR_SHAPE;
    p = GemmParams{};
    p.C = Y; p.ldc = ldy; p.M = (int32_t)T; p.N = (int32_t)N; p.K = (int32_t)K;
    p.out_f32 = dt == FP4Q_OUT_F32; p.accumulate = 0;
    dense_tiles(p);
    if (g) {
        p.mode = MODE_GROUPED_ROWS; p.n_groups = g->n_groups; p.row_offsets = g->row_offsets;
        p.rows_pair_aligned = g->row_alignment == 256;
        p.b_rows_per_group = (int32_t)N; p.b_k_per_group = 0;
    }
    return FP4Q_OK;
}

extern "C" fp4q_status fp4q_gemm_fwd(const fp4q_tensor *X, const fp4q_tensor *W, void *Y, int64_t ldy, fp4q_out dt,
                                     const fp4q_groups *g, void *ws, size_t ws_bytes, void *stream)
{
    GemmParams p;
    bool noop;
    if (fp4q_status s = prepare_fwd(X, W, Y, ldy, dt, g, p, &noop)) return s;
    if (noop) return FP4Q_OK;
    return launch_gemm<KIND_MXF4>(operand_rm(X), operand_rm(W), p, ws, ws_bytes, stream);
}

// C[M, N] = A B^T with the output leaving as the 2D-block FP4 tensor Cq (dense, pair kernel).
// Grouped form (g != NULL): b_rows_per_group / b_k_per_group as in the plain grouped products; the pair tiles need
// every group to start on a multiple of 256 rows.
static fp4q_status launch_gemm_quantized(const Operand &A, const Operand &B, int64_t M, int64_t N, int64_t K, const fp4q_tensor *Cq,
                                         fp4q_round mode, uint64_t seed, uint32_t tensor_id, const fp4q_groups *g,
                                         int32_t b_rows_per_group, int32_t b_k_per_group, void *ws, size_t ws_bytes, void *stream)
{
    if (mode != FP4Q_ROUND_NEAREST && mode != FP4Q_ROUND_STOCHASTIC) return FP4Q_ERR_UNSUPPORTED;
    if (fp4q_status s = check_groups(g)) return s;
    if (g && g->row_alignment != 256) return FP4Q_ERR_UNSUPPORTED;
    if (Cq->rows != M || Cq->cols != N) return FP4Q_ERR_SHAPE;
    if (M > kMaxDim || N > kMaxDim || K > kMaxDim) return FP4Q_ERR_UNSUPPORTED;
    if (N % 16 != 0) return FP4Q_ERR_UNSUPPORTED;   // one Philox block per 16-element row segment of the output
    if (M == 0 || N == 0) return FP4Q_OK;
    if (!A.payload || !B.payload || !A.sf.ptr || !B.sf.ptr || !Cq->q_rm || !Cq->scale) return FP4Q_ERR_NULL;
    if (Cq->ld_rm < round_up(N, 32) / 2 || Cq->ld_s < ceil_div(N, 32)) return FP4Q_ERR_SHAPE;
    if (Cq->q_t && Cq->ld_t < round_up(M, 32) / 2) return FP4Q_ERR_SHAPE;
    if (!aligned(Cq->q_rm, 16) || Cq->ld_rm % 16 != 0) return FP4Q_ERR_ALIGN;
    if (Cq->q_t && (!aligned(Cq->q_t, 16) || Cq->ld_t % 16 != 0)) return FP4Q_ERR_ALIGN;
    if (!ws || ws_bytes < sizeof(Workspace)) return FP4Q_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return FP4Q_ERR_ALIGN;
    if (!aligned(A.payload, 16) || !aligned(B.payload, 16) || A.ld_bytes % 16 || B.ld_bytes % 16) return FP4Q_ERR_ALIGN;
    GemmParams p = {};
    p.M = (int32_t)M; p.N = (int32_t)N; p.K = (int32_t)K;
    dense_tiles(p);
    p.sfa = A.sf; p.sfb = B.sf;
    p.status = reinterpret_cast<uint32_t *>(ws);
    p.q_rm = Cq->q_rm; p.q_ld_rm = Cq->ld_rm;
    p.q_t = Cq->q_t; p.q_ld_t = Cq->ld_t;
    p.q_scale = Cq->scale; p.q_ld_s = Cq->ld_s;
    p.q_mode = (int32_t)mode; p.q_tensor_id = tensor_id;
    philox_round_keys(seed, p.q_keys);
    if (g) {
        p.mode = MODE_GROUPED_ROWS; p.n_groups = g->n_groups; p.row_offsets = g->row_offsets;
        p.rows_pair_aligned = 1;
        p.b_rows_per_group = b_rows_per_group; p.b_k_per_group = b_k_per_group;
    }
    return launch_gemm_impl<KIND_MXF4, 2, EPI_QUANT>(A, B, p, stream);
}

extern "C" fp4q_status fp4q_gemm_fwd_quantized(const fp4q_tensor *X, const fp4q_tensor *W, const fp4q_tensor *Yq, fp4q_round mode,
                                               uint64_t seed, uint32_t tensor_id, const fp4q_groups *g, void *ws, size_t ws_bytes,
                                               void *stream)
{
    if (!tensor_ok(X) || !tensor_ok(W) || !tensor_ok(Yq)) return X && W && Yq ? FP4Q_ERR_SHAPE : FP4Q_ERR_NULL;
    if (X->cols != W->cols) return FP4Q_ERR_SHAPE;
    if (g && g->n_groups > 0 && (W->rows % g->n_groups || (W->rows / g->n_groups) % 32)) return FP4Q_ERR_SHAPE;
    const int64_t N = g && g->n_groups > 0 ? W->rows / g->n_groups : W->rows;
    return launch_gemm_quantized(operand_rm(X), operand_rm(W), X->rows, N, X->cols, Yq, mode, seed, tensor_id, g, (int32_t)N, 0, ws,
                                 ws_bytes, stream);
}

extern "C" fp4q_status fp4q_gemm_dgrad_quantized(const fp4q_tensor *dY, const fp4q_tensor *W, const fp4q_tensor *dXq, fp4q_round mode,
                                                 uint64_t seed, uint32_t tensor_id, const fp4q_groups *g, void *ws, size_t ws_bytes,
                                                 void *stream)
{
    if (!tensor_ok(dY) || !tensor_ok(W) || !tensor_ok(dXq)) return dY && W && dXq ? FP4Q_ERR_SHAPE : FP4Q_ERR_NULL;
    const int64_t N = dY->cols;
    if (g && g->n_groups > 0 ? (W->rows != N * g->n_groups || N % 64) : (W->rows != N)) return FP4Q_ERR_SHAPE;
    return launch_gemm_quantized(operand_rm(dY), operand_t(W), dY->rows, W->cols, N, dXq, mode, seed, tensor_id, g, 0, (int32_t)N, ws,
                                 ws_bytes, stream);
}

extern "C" fp4q_status fp4q_gemm_dgrad(const fp4q_tensor *dY, const fp4q_tensor *W, void *dX, int64_t ldx, fp4q_out dt,
                                       const fp4q_groups *g, void *ws, size_t ws_bytes, void *stream)
{
    if (!tensor_ok(dY) || !tensor_ok(W)) return dY && W ? FP4Q_ERR_SHAPE : FP4Q_ERR_NULL;
    if (fp4q_status s = check_groups(g)) return s;
    if (dt != FP4Q_OUT_BF16 && dt != FP4Q_OUT_F32) return FP4Q_ERR_UNSUPPORTED;
    const int64_t T = dY->rows, N = dY->cols, K = W->cols;
    if (g ? (W->rows != N * g->n_groups) : (W->rows != N)) return FP4Q_ERR_SHAPE;
    if (g && N % 64) return FP4Q_ERR_UNSUPPORTED;   // a group's contraction range must end on an MMA boundary
    if (T > kMaxDim || N > kMaxDim || K > kMaxDim || W->rows > kMaxDim) return FP4Q_ERR_UNSUPPORTED;
    if (T == 0 || K == 0) return FP4Q_OK;
    if (!dX || !dY->q_rm || !W->q_t || !dY->scale || !W->scale) return FP4Q_ERR_NULL;
    if (ldx < K) return FP4Q_ERR_SHAPE;
    GemmParams p = {};
    p.C = dX; p.ldc = ldx; p.M = (int32_t)T; p.N = (int32_t)K; p.K = (int32_t)N;
    p.out_f32 = dt == FP4Q_OUT_F32; p.accumulate = 0;
    dense_tiles(p);
    if (g) {
        p.mode = MODE_GROUPED_ROWS; p.n_groups = g->n_groups; p.row_offsets = g->row_offsets;
        p.rows_pair_aligned = g->row_alignment == 256;
        p.b_rows_per_group = 0; p.b_k_per_group = (int32_t)N;
    }
    return launch_gemm<KIND_MXF4>(operand_rm(dY), operand_t(W), p, ws, ws_bytes, stream);
}

extern "C" fp4q_status fp4q_gemm_wgrad(const fp4q_tensor *dY, const fp4q_tensor *X, void *dW, int64_t ldw, fp4q_out dt,
                                       int accumulate, const fp4q_groups *g, void *ws, size_t ws_bytes, void *stream)
{
    if (!tensor_ok(dY) || !tensor_ok(X)) return dY && X ? FP4Q_ERR_SHAPE : FP4Q_ERR_NULL;
    if (fp4q_status s = check_groups(g)) return s;
    if (dt != FP4Q_OUT_BF16 && dt != FP4Q_OUT_F32) return FP4Q_ERR_UNSUPPORTED;
    if (accumulate && dt != FP4Q_OUT_F32) return FP4Q_ERR_UNSUPPORTED;
    if (dY->rows != X->rows) return FP4Q_ERR_SHAPE;
    const int64_t T = dY->rows, N = dY->cols, K = X->cols;
    if (T > kMaxDim || N > kMaxDim || K > kMaxDim) return FP4Q_ERR_UNSUPPORTED;
    if (g && N * g->n_groups > kMaxDim) return FP4Q_ERR_UNSUPPORTED;
    if (N == 0 || K == 0) return FP4Q_OK;
    if (!dW || !dY->q_t || !X->q_t || !dY->scale || !X->scale) return FP4Q_ERR_NULL;
    if (ldw < K) return FP4Q_ERR_SHAPE;
    GemmParams p = {};
    p.C = dW; p.ldc = ldw; p.M = (int32_t)N; p.N = (int32_t)K; p.K = (int32_t)T;
    p.out_f32 = dt == FP4Q_OUT_F32; p.accumulate = accumulate ? 1 : 0;
    dense_tiles(p);
    if (g) {
        p.mode = MODE_GROUPED_K; p.n_groups = g->n_groups; p.row_offsets = g->row_offsets;
        p.n_tile_total *= g->n_groups;
    }
    return launch_gemm<KIND_MXF4>(operand_t(dY), operand_t(X), p, ws, ws_bytes, stream);
}

extern "C" fp4q_status fp4q_mxfp8_qk(const uint8_t *xq, int64_t ld_xq, const uint8_t *xs, int64_t ld_xs, int64_t T,
                                     int64_t Kdim, const uint8_t *wq_q, const uint8_t *wq_s, const uint8_t *wk_q,
                                     const uint8_t *wk_s, int64_t ld_wq, int64_t ld_ws, int64_t N, void *Q_out,
                                     void *K_out, int64_t ldo, fp4q_out dt, void *ws, size_t ws_bytes, void *stream)
{
    if (T < 0 || N < 0 || Kdim < 0) return FP4Q_ERR_SHAPE;
    if (dt != FP4Q_OUT_BF16 && dt != FP4Q_OUT_F32) return FP4Q_ERR_UNSUPPORTED;
    if (T > kMaxDim || N > kMaxDim || Kdim > kMaxDim) return FP4Q_ERR_UNSUPPORTED;
    if (T == 0 || N == 0) return FP4Q_OK;
    if (!xq || !xs) return FP4Q_ERR_NULL;
    if ((wq_q && (!wq_s || !Q_out)) || (wk_q && (!wk_s || !K_out))) return FP4Q_ERR_NULL;
    const int64_t kpad = round_up(Kdim, 32), nkb = ceil_div(Kdim, 32);
    if (ld_xq < kpad || ld_wq < kpad || ld_xs < nkb || ld_ws < nkb || ldo < N) return FP4Q_ERR_SHAPE;
    Operand A;
    A.payload = xq; A.rows = T; A.row_bytes = kpad; A.ld_bytes = ld_xq;
    A.sf = ScaleView{xs, ld_xs, 1, (int32_t)T, (int32_t)nkb};
    const uint8_t *wq[2] = {wq_q, wk_q};
    const uint8_t *wsf[2] = {wq_s, wk_s};
    void *out[2] = {Q_out, K_out};
    for (int i = 0; i < 2; i++) {
        if (!wq[i]) continue;
        Operand B;
        B.payload = wq[i]; B.rows = N; B.row_bytes = kpad; B.ld_bytes = ld_wq;
        B.sf = ScaleView{wsf[i], ld_ws, 1, (int32_t)N, (int32_t)nkb};
        GemmParams p = {};
        p.C = out[i]; p.ldc = ldo; p.M = (int32_t)T; p.N = (int32_t)N; p.K = (int32_t)Kdim;
        p.out_f32 = dt == FP4Q_OUT_F32;
        dense_tiles(p);
        if (fp4q_status s = launch_gemm<KIND_MXF8>(A, B, p, ws, ws_bytes, stream)) return s;
    }
    return FP4Q_OK;
}

extern "C" fp4q_status fp4q_mxfp8_gemm(const uint8_t *aq, int64_t ld_aq, const uint8_t *as, int64_t ld_as, int64_t M,
                                       const uint8_t *bq, int64_t ld_bq, const uint8_t *bs, int64_t ld_bs, int64_t N,
                                       int64_t Kdim, void *C, int64_t ldc, fp4q_out dt, void *ws, size_t ws_bytes,
                                       void *stream)
{
    if (M < 0 || N < 0 || Kdim < 0) return FP4Q_ERR_SHAPE;
    if (dt != FP4Q_OUT_BF16 && dt != FP4Q_OUT_F32) return FP4Q_ERR_UNSUPPORTED;
    if (M > kMaxDim || N > kMaxDim || Kdim > kMaxDim) return FP4Q_ERR_UNSUPPORTED;
    if (M == 0 || N == 0) return FP4Q_OK;
    if (!aq || !as || !bq || !bs || !C) return FP4Q_ERR_NULL;
    const int64_t kpad = round_up(Kdim, 32), nkb = ceil_div(Kdim, 32);
    if (ld_aq < kpad || ld_bq < kpad || ld_as < nkb || ld_bs < nkb || ldc < N) return FP4Q_ERR_SHAPE;
    Operand A, B;
    A.payload = aq; A.rows = M; A.row_bytes = kpad; A.ld_bytes = ld_aq;
    A.sf = ScaleView{as, ld_as, 1, (int32_t)M, (int32_t)nkb};
    B.payload = bq; B.rows = N; B.row_bytes = kpad; B.ld_bytes = ld_bq;
    B.sf = ScaleView{bs, ld_bs, 1, (int32_t)N, (int32_t)nkb};
    GemmParams p = {};
    p.C = C; p.ldc = ldc; p.M = (int32_t)M; p.N = (int32_t)N; p.K = (int32_t)Kdim;
    p.out_f32 = dt == FP4Q_OUT_F32;
    dense_tiles(p);
    return launch_gemm<KIND_MXF8>(A, B, p, ws, ws_bytes, stream);
}

extern "C" fp4q_status fp4q_gemm_fwd_act1d(const uint8_t *xq, int64_t ld_xq, const uint8_t *xs, int64_t ld_xs, int64_t T,
                                           const fp4q_tensor *W, void *Y, int64_t ldy, fp4q_out dt, void *ws, size_t ws_bytes,
                                           void *stream)
{
    if (!tensor_ok(W)) return W ? FP4Q_ERR_SHAPE : FP4Q_ERR_NULL;
    if (T < 0) return FP4Q_ERR_SHAPE;
    if (dt != FP4Q_OUT_BF16 && dt != FP4Q_OUT_F32) return FP4Q_ERR_UNSUPPORTED;
    const int64_t N = W->rows, K = W->cols;
    if (T > kMaxDim || N > kMaxDim || K > kMaxDim) return FP4Q_ERR_UNSUPPORTED;
    if (T == 0 || N == 0) return FP4Q_OK;
    if (!Y || !xq || !xs || !W->q_rm || !W->scale) return FP4Q_ERR_NULL;
    if (ldy < N || ld_xq < round_up(K, 32) / 2 || ld_xs < ceil_div(K, 32)) return FP4Q_ERR_SHAPE;
    Operand A, B = operand_rm(W);
    A.payload = xq; A.rows = T; A.row_bytes = round_up(K, 32) / 2; A.ld_bytes = ld_xq;
    A.sf = ScaleView{xs, ld_xs, 1, (int32_t)T, (int32_t)ceil_div(K, 32), 0};
    B.sf.row_shift = 5;
    GemmParams p = {};
    p.C = Y; p.ldc = ldy; p.M = (int32_t)T; p.N = (int32_t)N; p.K = (int32_t)K;
    p.out_f32 = dt == FP4Q_OUT_F32;
    dense_tiles(p);
    return launch_gemm<KIND_MXF4R>(A, B, p, ws, ws_bytes, stream);
}

extern "C" fp4q_status fp4q_gemm_wgrad_act1d(const fp4q_tensor *dY, const uint8_t *xtq, int64_t ld_xtq, const uint8_t *xts,
                                             int64_t ld_xts, int64_t K, void *dW, int64_t ldw, fp4q_out dt, int accumulate,
                                             void *ws, size_t ws_bytes, void *stream)
{
    if (!tensor_ok(dY)) return dY ? FP4Q_ERR_SHAPE : FP4Q_ERR_NULL;
    if (K < 0) return FP4Q_ERR_SHAPE;
    if (dt != FP4Q_OUT_BF16 && dt != FP4Q_OUT_F32) return FP4Q_ERR_UNSUPPORTED;
    if (accumulate && dt != FP4Q_OUT_F32) return FP4Q_ERR_UNSUPPORTED;
    const int64_t T = dY->rows, N = dY->cols;
    if (T > kMaxDim || N > kMaxDim || K > kMaxDim) return FP4Q_ERR_UNSUPPORTED;
    if (N == 0 || K == 0) return FP4Q_OK;
    if (!dW || !dY->q_t || !dY->scale || !xtq || !xts) return FP4Q_ERR_NULL;
    if (ldw < K || ld_xtq < round_up(T, 32) / 2 || ld_xts < ceil_div(T, 32)) return FP4Q_ERR_SHAPE;
    Operand A = operand_t(dY), B;
    A.sf.row_shift = 5;
    B.payload = xtq; B.rows = K; B.row_bytes = round_up(T, 32) / 2; B.ld_bytes = ld_xtq;
    B.sf = ScaleView{xts, ld_xts, 1, (int32_t)K, (int32_t)ceil_div(T, 32), 0};
    GemmParams p = {};
    p.C = dW; p.ldc = ldw; p.M = (int32_t)N; p.N = (int32_t)K; p.K = (int32_t)T;
    p.out_f32 = dt == FP4Q_OUT_F32; p.accumulate = accumulate ? 1 : 0;
    dense_tiles(p);
    return launch_gemm<KIND_MXF4R>(A, B, p, ws, ws_bytes, stream);
}

// ------------------------------------------------------------------------------------------------------
// Products on tensors quantized in 16 x 16 blocks (block-size study): same payloads, scale matrix
// [ceil(rows/16), ceil(cols/16)], 16-element scale vectors in the MMA.  Dense only.
namespace fp4q {

static Operand operand_rm16(const fp4q_tensor *t)
{
    Operand o = operand_rm(t);
    o.sf = ScaleView{t->scale, t->ld_s, 1, (int32_t)ceil_div(t->rows, 16), (int32_t)ceil_div(t->cols, 16), 4};
    return o;
}
static Operand operand_t16(const fp4q_tensor *t)
{
    Operand o = operand_t(t);
    o.sf = ScaleView{t->scale, 1, t->ld_s, (int32_t)ceil_div(t->cols, 16), (int32_t)ceil_div(t->rows, 16), 4};
    return o;
}

// which: 0 forward (A = a.q_rm [M,K], B = b.q_rm [N,K]), 1 input gradient (A = a.q_rm [M,K'], B = b.q_t), 2 weight
// gradient (A = a.q_t, B = b.q_t)
static fp4q_status gemm_b16(int which, const fp4q_tensor *a, const fp4q_tensor *b, void *C, int64_t ldc, fp4q_out dt, int accumulate,
                            void *ws, size_t ws_bytes, void *stream)
{
    if (!tensor_ok(a) || !tensor_ok(b)) return a && b ? FP4Q_ERR_SHAPE : FP4Q_ERR_NULL;
    if (dt != FP4Q_OUT_BF16 && dt != FP4Q_OUT_F32) return FP4Q_ERR_UNSUPPORTED;
    if (accumulate && dt != FP4Q_OUT_F32) return FP4Q_ERR_UNSUPPORTED;
    int64_t M, N, K;
    if (which == 0) { if (a->cols != b->cols) return FP4Q_ERR_SHAPE; M = a->rows; N = b->rows; K = a->cols; }
    else if (which == 1) { if (a->cols != b->rows) return FP4Q_ERR_SHAPE; M = a->rows; N = b->cols; K = a->cols; }
    else { if (a->rows != b->rows) return FP4Q_ERR_SHAPE; M = a->cols; N = b->cols; K = a->rows; }
    if (M > kMaxDim || N > kMaxDim || K > kMaxDim) return FP4Q_ERR_UNSUPPORTED;
    if (M == 0 || N == 0) return FP4Q_OK;
    const uint8_t *pa = which == 2 ? a->q_t : a->q_rm, *pb = which == 0 ? b->q_rm : b->q_t;
    if (!C || !pa || !pb || !a->scale || !b->scale) return FP4Q_ERR_NULL;
    if (ldc < N) return FP4Q_ERR_SHAPE;
    GemmParams p = {};
    p.C = C; p.ldc = ldc; p.M = (int32_t)M; p.N = (int32_t)N; p.K = (int32_t)K;
    p.out_f32 = dt == FP4Q_OUT_F32; p.accumulate = accumulate ? 1 : 0;
    dense_tiles(p);
    return launch_gemm<KIND_MXF4B16>(which == 2 ? operand_t16(a) : operand_rm16(a), which == 0 ? operand_rm16(b) : operand_t16(b), p, ws,
                                     ws_bytes, stream);
}

}  // namespace fp4q

extern "C" fp4q_status fp4q_gemm_fwd_b16(const fp4q_tensor *X, const fp4q_tensor *W, void *Y, int64_t ldy, fp4q_out dt, void *ws,
                                         size_t ws_bytes, void *stream)
{
    return gemm_b16(0, X, W, Y, ldy, dt, 0, ws, ws_bytes, stream);
}

extern "C" fp4q_status fp4q_gemm_dgrad_b16(const fp4q_tensor *dY, const fp4q_tensor *W, void *dX, int64_t ldx, fp4q_out dt, void *ws,
                                           size_t ws_bytes, void *stream)
{
    return gemm_b16(1, dY, W, dX, ldx, dt, 0, ws, ws_bytes, stream);
}

extern "C" fp4q_status fp4q_gemm_wgrad_b16(const fp4q_tensor *dY, const fp4q_tensor *X, void *dW, int64_t ldw, fp4q_out dt,
                                           int accumulate, void *ws, size_t ws_bytes, void *stream)
{
    return gemm_b16(2, dY, X, dW, ldw, dt, accumulate, ws, ws_bytes, stream);
}

// ------------------------------------------------------------------------------------------------------
// Forward product for callers that cannot allocate device memory.
//
// The GEMM kernel records device-side anomalies in a small workspace that the regular entry points take
// from the caller.  Code that runs where cudaMalloc is off limits -- a plug-in inside a host application
// that owns the device heap, a real-time loop that must not enter the allocator, a sandbox that only hands
// out pre-registered buffers -- has no way to supply one.  For those callers the workspace lives in the
// fixed array below, which every GPU that loads this library holds until the process exits.
namespace fp4q {

constexpr size_t kStaticWorkspaceBytes = 1024;   // stated maximum; the kernel's workspace must fit in it
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

static void *g_static_workspace_addr[kMaxDevices];   // device address of the array, per device

// In host code the array's name is only a handle: the device address has to be asked for, once per device,
// with that device current.
static fp4q_status static_workspace_address(void **out)
{
    const int dev = current_device();
    if (dev < 0) return FP4Q_ERR_CUDA;
    if (g_static_workspace_addr[dev] == nullptr) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || ptr == nullptr) return FP4Q_ERR_CUDA;
        g_static_workspace_addr[dev] = ptr;
    }
    *out = g_static_workspace_addr[dev];
    return FP4Q_OK;
}

}  // namespace fp4q

extern "C" fp4q_status fp4q_gemm_fwd_static_workspace(const fp4q_tensor *X, const fp4q_tensor *W, void *Y, int64_t ldy,
                                                      fp4q_out dt, uint32_t *status_out, void *stream)
{
    if (fp4q_workspace_bytes() > kStaticWorkspaceBytes) return FP4Q_ERR_WORKSPACE;   // layout outgrew the array
    // every argument error is reported before anything is put on the stream
    GemmParams p;
    bool noop;
    if (fp4q_status s = prepare_fwd(X, W, Y, ldy, dt, nullptr, p, &noop)) return s;
    void *ws = nullptr;
    if (fp4q_status s = static_workspace_address(&ws)) return s;
    if (!noop)
        if (fp4q_status s = check_gemm_args(operand_rm(X), operand_rm(W), p, ws, kStaticWorkspaceBytes)) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: the status words must start at zero
    if (cudaMemsetAsync(ws, 0, sizeof(Workspace), st) != cudaSuccess) return FP4Q_ERR_CUDA;
    if (!noop)
        if (fp4q_status s = launch_gemm<KIND_MXF4>(operand_rm(X), operand_rm(W), p, ws, kStaticWorkspaceBytes, stream)) return s;
    if (status_out &&
        cudaMemcpyAsync(status_out, ws, sizeof(uint32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return FP4Q_ERR_CUDA;
    return FP4Q_OK;
}
