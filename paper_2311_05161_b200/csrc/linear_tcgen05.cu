// Tensor-core kernel of the W4A8-dINT linear layer (Eq. 1 contraction with the Eq. 6
// dequantization folded into an integer lookup), sm_100a.
//
// Orientation: the 128 output features of a tile are the M side of the MMA (operand A,
// decoded weights), the tokens are the N side (operand B, INT8 activations), so the
// accumulator in tensor memory has one feature per lane and one token per column.  Per
// 128-wide k-block:
//   producer thread   TMA tile load of TOK x 128 INT8 activations (128-byte swizzle) into the
//                     stage; for weight-streaming shapes also L2 prefetches of the code tiles
//   decode warps      teams of four warps take k-blocks in turn, one thread per feature row:
//                     64 bytes of 4-bit codes straight from global memory into registers (one
//                     of the team's k-blocks ahead), 4-bit codes -> INT8 through a 16-entry
//                     byte table held in four registers (byte permute), written into the stage
//                     in the 128-byte-swizzled K-major layout the MMA reads
//   MMA thread        4 x tcgen05.mma kind::i8 (128 x TOK x 32) into tensor memory, INT32
//   epilogue warps    tcgen05.ld, FP32 rescale (token step x weight step / 2), bias, BF16
// Per-channel weights accumulate over the whole K slice in tensor memory; group-128
// weights hand every k-block's INT32 partial to the epilogue warps, which scale it by the
// group's step and add it to FP32 registers, while the next k-block accumulates into the
// other tensor-memory buffer.  Split-K slices leave partial tiles in the workspace and the
// last slice to finish a tile (an atomic counter, no spinning) reduces them in slice order.
//
// Every wait is bounded: a wait that runs out records a status, raises a flag that all
// roles poll, and the CTA drains its copies, frees tensor memory and returns.
#include <cuda.h>

#include <atomic>

#include "common.cuh"
#include "decode.cuh"

namespace w4a8 {

namespace {

constexpr int kFirstDecodeWarp = 2;
constexpr int kSwigluVariant = 5;
constexpr int kAsymGroupVariant = 6;
constexpr int kMaxDevices = 64;
constexpr int kABytes = kTileN * kTileK;            // decoded INT8 tile, 16 KiB
constexpr int kDefaultTeamWarps = 4;               // warps per decode team
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
// how long a waiting thread may stay suspended in hardware before it polls again (it is woken
// at once when the barrier phase completes); keeps waiting warps out of the issue slots
constexpr uint32_t kSuspendHintNs = 20000u;
constexpr unsigned long long kDrainLimitNs = 200000000ull;

template <int TOK, bool GROUPED, int DW, int CL>
struct Cfg {
    // warps in a row: producer, MMA issuer, DW decode warps, epilogue warps
    static constexpr int kFirstEpiWarp = kFirstDecodeWarp + DW;
    // epilogue warpgroups: group mode spreads the per-k-block FP32 accumulation over
    // 32 columns per thread (more warps in flight, fewer registers each)
    static constexpr int kEpiGroups = !GROUPED ? 1 : (TOK >= 128 ? 4 : TOK >= 64 ? 2 : 1);
    // output staging buffers per group (one where the token ring needs the room)
    static constexpr int kStageBufs = (GROUPED || (TOK >= 256 && CL != 3 && CL != 5)) ? 1 : 2;
    static constexpr int kAStagesWanted = CL == 4 ? 5 : CL == 5 ? 6 : CL == 3 ? 4 : GROUPED ? 5 : TOK >= 256 ? 3 : 4;
    static constexpr int kEpiWarps = 4 * kEpiGroups;
    static constexpr int kThreads = 32 * (kFirstEpiWarp + kEpiWarps);
    static constexpr int kColsPerThread = TOK / kEpiGroups;
    static constexpr int kChunk = kColsPerThread >= 32 ? 32 : 16;
    // CL = 1: one CTA.  CL = 2 (kShare): two CTAs on the same row tile, each on its own token
    // tile, share the expansion of the codes.  CL = 3 (kPair): two CTAs on two row tiles and the
    // same token tile run as one MMA pair (cta_group::2): every MMA instruction covers both row
    // tiles, CTA r holds (and loads) tokens 128 r .. 128 r + 127 of the tile, and the leader's one
    // issuing thread serves both, so the token bytes per SM and the issue cost per CTA halve.
    // CL = 4 (kDual): one CTA on two row tiles and one token tile: the two tiles' MMAs read the same
    // token buffer, so the token bytes per MAC halve as in the MMA pair, without any traffic
    // between CTAs; the two accumulators fill tensor memory, so the epilogue of a unit no longer
    // overlaps the next unit's main loop.
    // CL = 5: the MMA pair with three k-blocks per barrier round (for k-block counts that are
    // multiples of three: twelve MMA instructions per wait and commit).
    static constexpr bool kShare = CL == 2, kPair = CL == 3 || CL == 5, kDual = CL == 4;
    static constexpr int kCtas = (kShare || kPair) ? 2 : 1;
    static constexpr int kTiles = kDual ? 2 : 1;               // row tiles of a unit in this CTA
    // k-blocks per barrier round.  The issuing thread's loop (wait, MMAs, commit) is the serial
    // spine of the kernel, and its fixed part per round (wait, commit, bookkeeping: some 300
    // cycles) is what keeps an MMA pair from outrunning one CTA; with two k-blocks per round the
    // pair pays it once per eight MMA instructions.  Operand buffers stay one k-block each.
    static constexpr int kSub = CL == 5 ? 3 : kPair ? 2 : 1;
    static constexpr int kPerRound = kTiles * kSub;            // weight buffers filled per round
    static constexpr int kTokRows = kPair ? TOK / 2 : TOK;     // token rows this CTA loads per k-block
    static constexpr int kTokBytes = kTokRows * kTileK;
    // Codes go from global memory straight into the decode threads' registers (shared-memory
    // bandwidth and capacity are the scarce resources); for weight-streaming shapes the
    // producer thread runs ahead with L2 prefetches of the code tiles.
    // Decode warps work in teams that take k-blocks in turn; a team of kTeamWarps warps splits
    // the 128 x 128 tile into kTeamWarps / 4 column slices (a thread expands 64, 32 or 16 bytes
    // of codes of one row).  Wider teams fill a stage sooner (the stage ring is short), narrower
    // teams pay the per-k-block bookkeeping less often.
    static constexpr int kTeamWarps = (DW % kDefaultTeamWarps == 0) ? kDefaultTeamWarps : 4;
    static constexpr int kTeams = DW / kTeamWarps;
    // The CTAs of a cluster (CL = 1 or 2) work on the same row tile and k-block at the same time,
    // each on its own token tile.  With CL = 2 each expands 64 of the tile's 128 rows into its own
    // stage and sends them to its peer's stage with a bulk copy through distributed shared memory
    // that completes on the peer's barrier, so the table lookups per MMA halve.
    static constexpr int kRowsPerCta = kShare ? kTileN / 2 : kTileN;
    static constexpr int kQuartersPerThread = kShare ? 2 : 4;   // 32-k quarters of a row per thread
    static_assert(CL >= 1 && CL <= 5, "one CTA, a sharing pair, an MMA pair (two forms) or two row tiles per CTA");
    static_assert(!kDual || (TOK == 256 && !GROUPED), "two row tiles per CTA: 256 tokens, per-channel weights");
    static_assert(!kPair || (TOK == 256 && !GROUPED), "the MMA pair: 256 tokens, per-channel weights");
    static_assert(DW % kTeamWarps == 0 && kTeamWarps == 4, "decode warps form whole teams of four");
    // Two rings of operand buffers, one set of barriers.  Ring A holds decoded INT8 weights of a
    // k-block (16 KiB, written by the decode warps), ring B the tokens of a k-block (written by
    // TMA).  K-block number `it` uses A buffer it % kAStages, B buffer it % kStages and the barrier
    // pair it % kStages (with two row tiles per unit: weight buffer (2 it + h) % kAStages for
    // tile h).  The rings differ in depth because they hide different latencies: a
    // token tile comes from L2 and is on its way for a few thousand cycles when all SMs pull
    // tiles at once (the bytes in flight bound the rate), decoded weights come from registers.
    // (Keeping operand A in tensor memory instead was measured slower at every token tile.)
    static constexpr int kPrefetchAhead = 16;          // k-blocks of codes requested into L2
    // output staging: kStageBufs buffers of kChunk tokens x 128 features BF16 per epilogue group
    static constexpr int kStagingBytes = kEpiGroups * kStageBufs * kChunk * kTileN * 2;
    static constexpr int kTailBytes =
        kStagingBytes + 3072 /* token steps, zero-points, offset sums */ + 1024 /* barriers */;
    static constexpr int kRingBytes = 232448 - 1024 - kTailBytes;
    static constexpr int kAStages = kAStagesWanted;
    static constexpr int kMaxStages = (kRingBytes - kAStages * kABytes) / kTokBytes;
    static constexpr int kStages = kMaxStages > 12 ? 12 : kMaxStages;
    static constexpr int kOffTokRing = kAStages * kABytes;
    // accumulator buffers in tensor memory: two for per-channel weights (epilogue of one unit
    // overlaps the main loop of the next); group mode hands over every k-block, and a hand-over
    // costs several hundred cycles of latency, so it rotates over as many buffers as fit
    static constexpr int kAccBufs = !GROUPED ? 2 : (512 / TOK > 8 ? 8 : 512 / TOK);
    static constexpr int kTmemNeed = kAccBufs * TOK;
    static constexpr int kTmemCols = kTmemNeed <= 32 ? 32 : kTmemNeed <= 64 ? 64 : kTmemNeed <= 128 ? 128
                                     : kTmemNeed <= 256 ? 256 : 512;
    static constexpr int kOffStaging = kOffTokRing + kStages * kTokBytes;
    static constexpr int kOffTok = kOffStaging + kStagingBytes;
    static constexpr int kOffBarriers = kOffTok + 3072;
    static constexpr int kSmemBytes = kOffBarriers + 1024 + 1024 /* alignment slack */;
    // (a barrier slot must not be reused while a decode thread may still wait on its last phase:
    // the weight buffers span at most as many rounds as there are slots)
    static_assert(kStages * kPerRound >= kAStages && kAStages >= 2 && kStages >= 3, "pipeline depth");
    static_assert(kTmemNeed <= 512, "tensor memory budget");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
    static_assert(!GROUPED || TOK <= 128, "group mode keeps its FP32 sums in registers");
};

struct Params {
    const uint8_t *blob;
    const uint8_t *codes;
    const float *scales;
    const uint8_t *zeros;
    const float *tok_scale;
    const float *bias;
    __nv_bfloat16 *Y;
    int32_t *acc_out;
    StatusBlock *sb;
    int *counters;
    void *partials;
    BlobLayout L;
    int M, tok_tiles, m_pad, split_k, kb_per_split, total_units, prefetch_codes;
    int tok_groups, tok_run;   // token-tile groups of the unit list, and how many form a run (unit_tiles)
    ZeroPoint zp;
    LevelTables lt;
    float unit;          // level unit as a factor of the step: 2^-shift
    unsigned long long wait_ns, drain_ns;   // limits of the bounded waits
    int offset;          // 0, or 13 * 2^shift: the decode warps use the offset tables (decode.cuh)
                         // and the epilogue subtracts tok_offsum[m] = offset * (sum of token m)
    const int32_t *tok_offsum;
    int swiglu;          // gated-unit epilogue: Y is [M][N / 2] binary16, silu(row 2i) * row 2i + 1
    int batch_rows;      // 0, or M when every 128-row tile has its own [M][K] block of tokens (and
                         // token steps), stacked in tile order: the attention P*V form
    int skip_load;       // test hook: every producer leaves out the token load of its k-block
                         // number skip_load - 1 (0 = none), so that a wait runs out
};

// --------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Copy `bytes` (a multiple of 16) of this CTA's shared memory into a peer CTA's shared memory;
// the bytes count towards the transaction count of the peer's barrier `bar_in_cluster`.
__device__ __forceinline__ void bulk_copy_to_cta(uint32_t dst_in_cluster, uint32_t src, uint32_t bytes,
                                                 uint32_t bar_in_cluster)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
            "r"(dst_in_cluster),
        "r"(src), "r"(bytes), "r"(bar_in_cluster)
        : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_in_cluster)
{
    // (default semantics, as for a local arrival: asking for a cluster-scope release here was
    // measured to cost the arriving thread more than half a microsecond per arrival)
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_in_cluster) : "memory");
}
// wait with cluster-scope acquire: what a peer CTA released by its arrival is visible afterwards
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
        : "memory");
    return ok != 0;
}
// Tile load of a CTA of an MMA pair: the bytes land in this CTA, the completion counts on the
// barrier `bar_in_cluster`, which may belong to the pair's other CTA (no multicast: one copy).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y,
                                                 uint32_t bar_in_cluster)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar_in_cluster), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::
                     "l"(map),
                 "r"(src), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::
                     "r"(bar)
                 : "memory");
}
// The same arrival on the barrier at this offset in every CTA of `mask`.
__device__ __forceinline__ void tc_commit_multicast(uint32_t bar, uint16_t mask)
{
    asm volatile(
        "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::
            "r"(bar),
        "h"(mask)
        : "memory");
}
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The pair forms: one instruction of the leader CTA drives the tensor cores of both CTAs.
__device__ __forceinline__ void tc_mma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                               uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, uint16_t mask)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::
            "r"(bar),
        "h"(mask)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
          "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),
          "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Two FP32 values in one 64-bit register for the packed FP32 instructions.
__device__ __forceinline__ uint64_t pack_f32x2(uint32_t lo, uint32_t hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi)
{
    uint32_t a, b;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
    lo = __uint_as_float(a);
    hi = __uint_as_float(b);
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
// A group's INT32 partial sum is below 2^22 in magnitude (128 products of at most 127 * 104), so
// adding it, as an integer, to the bit pattern of 1.5 * 2^23 gives the FP32 number 1.5 * 2^23 + sum:
// no conversion instruction (an eighth of the FP32 rate).  The add is written as a multiply-add
// by a register that holds 1, which runs on the FMA pipe: the 16-lane logic pipe is what the
// decode warps need.  Subtracting 1.5 * 2^23 afterwards is exact.  (Accumulators that start from
// that bit pattern, refilled with tcgen05.st after every read, were measured slower: the refill
// sits in the hand-over chain.)
constexpr uint32_t kMagicBits = 0x4B400000u;          // 1.5 * 2^23 = 12582912.0f
__device__ __forceinline__ uint32_t biased_float_bits(uint32_t acc, uint32_t one)
{
    uint32_t r;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(acc), "r"(one), "r"(kMagicBits));
    return r;
}
__device__ __forceinline__ void named_bar_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// Barrier over `threads` threads that also ANDs a predicate: every caller gets the same answer.
__device__ __forceinline__ bool named_bar_and(int id, int threads, bool pred)
{
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %3, 0;\n\t"
        "bar.red.and.pred q, %1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out)
        : "r"(id), "r"(threads), "r"((uint32_t)pred)
        : "memory");
    return out != 0;
}

// Shared-memory matrix descriptors (built in the MMA thread): K-major operand tile with 128-byte
// rows and 128-byte swizzle, 8-row groups 1024 bytes apart; the start address advances by 32
// bytes per 32-deep MMA step inside the swizzle span.
// Instruction descriptor: signed 8-bit A and B, both K-major, INT32 accumulate, M = 128.
__host__ __device__ constexpr uint32_t instr_desc_i8(int n, int m = 128)
{
    return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// --------------------------------------------------------------------------- bounded wait
struct Ctl {
    volatile int abort;
    int is_last;
    uint32_t tmem_base;
    unsigned long long wait_ns, drain_ns;      // limits of an ordinary wait and of a drain wait
};

// `draining`: the CTA has given up and only waits for what it has in flight (copies, MMAs):
// such a wait does not end because of the abort flag, and it has the shorter limit.
template <bool CLUSTER_ACQUIRE = false>
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, Ctl *ctl,
                                             StatusBlock *sb, int where, bool draining = false)
{
    auto test = [&]() {
        return CLUSTER_ACQUIRE ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity);
    };
    if (test()) return true;
    // the timer is slow to read: it is only consulted after many failed polls
    unsigned long long t0 = 0;
    for (uint32_t i = 1;; ++i) {
        if (test()) return true;
        if ((i & 63u) == 0u) {
            if (ctl->abort && !draining) return false;
            if (t0 == 0) {
                t0 = global_ns();
            } else if (global_ns() - t0 > (draining ? ctl->drain_ns : ctl->wait_ns)) {
                ctl->abort = 1;
                report_failure(sb, W4A8_ERR_TIMEOUT, where);
                return false;
            }
        }
    }
}

// The same wait for the roles with many threads (decode, epilogue): between polls the thread
// sleeps, so that its warp leaves the issue slots to the producer and MMA threads, whose
// per-k-block loops are the serial part of the pipeline.
__device__ __forceinline__ bool wait_bounded_idle(uint32_t bar, uint32_t parity, Ctl *ctl,
                                                  StatusBlock *sb, int where)
{
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = 0;
    for (uint32_t i = 1;; ++i) {
        __nanosleep(64);
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 1023u) == 0u) {
            if (ctl->abort) return false;
            if (t0 == 0) {
                t0 = global_ns();
            } else if (global_ns() - t0 > ctl->wait_ns) {
                ctl->abort = 1;
                report_failure(sb, W4A8_ERR_TIMEOUT, where);
                return false;
            }
        }
    }
}

// Order of the units.  Unit number `rest` (K slices taken out) belongs to a run of `tok_run`
// consecutive token tiles; inside a run the token tile changes fastest, then the row tile, and the
// runs follow one another.  CTAs work on consecutive units at the same time, so with a run of one
// token tile they share the tokens and walk through the whole weight matrix once per token tile
// (right when the packed weights stay in L2), and with longer runs tok_run CTAs read the same code
// tile at about the same time (one DRAM read, the others hit L2) while the run's tokens stay in L2:
// the host picks the run so that whichever operand does not fit in L2 is streamed once.
// RUNS = false: the kernel instance has only the one-tile form (the host then never asks for longer
// runs).  The general form costs the instances that never need it - group mode and 3-bit codes
// measured 15-20 % slower with it compiled in, as a call that is not inlined it cost all of them -
// so only the wide per-channel 4-bit instances, the ones that meet code matrices larger than L2
// with many token tiles, carry it.
template <bool RUNS>
__device__ __forceinline__ void unit_tiles(int rest, int row_groups, int tok_groups, int tok_run,
                                           int &row_group, int &tok_group)
{
    if (!RUNS || tok_run == 1) {        // the row group changes fastest
        tok_group = rest / row_groups;
        row_group = rest - tok_group * row_groups;
        return;
    }
    const int per_run = tok_run * row_groups;
    const int run = rest / per_run, r = rest - run * per_run;
    const int first = run * tok_run;
    const int width = min(tok_run, tok_groups - first);
    row_group = r / width;
    tok_group = first + (r - row_group * width);
}

// What does not change while a cursor walks: kept apart from the cursor, so that a copy of the
// cursor (the decode warps hold the current and the next position) copies six registers, not fifteen.
struct CursorEnv {
    int step, total_units, split_k, kb_per_split, k_blocks, row_groups, tok_groups, tok_run, tiles;
};
template <bool RUNS>
struct KbCursor {
    int u, kb, kb1;
    int nt;                    // row-tile group of the unit (integer divisions happen once per unit)
    int h;                     // row tile inside the unit
    uint32_t it;               // counts (k-block, tile) items
    __device__ __forceinline__ void open_unit(const CursorEnv &e)
    {
        if (u < e.total_units) {
            const int rest = u / e.split_k;
            const int s = u - rest * e.split_k;
            int tg;
            unit_tiles<RUNS>(rest, e.row_groups, e.tok_groups, e.tok_run, nt, tg);
            kb = s * e.kb_per_split;
            kb1 = min(e.k_blocks, kb + e.kb_per_split);
        }
    }
    __device__ __forceinline__ void start(int first, const CursorEnv &e)
    {
        u = first; it = 0; kb = kb1 = 0; nt = 0; h = 0;
        open_unit(e);
    }
    __device__ __forceinline__ bool valid(const CursorEnv &e) const { return u < e.total_units; }
    __device__ __forceinline__ void advance(int n, const CursorEnv &e)
    {
        // the usual case in one step: the n items ahead lie inside the current unit
        // (the decode warps call this once per item, in the serial part of their cycle)
        if (valid(e)) {
            const int ahead = h + n;
            const int kb_new = kb + ahead / e.tiles;
            if (kb_new < kb1) {
                kb = kb_new;
                h = ahead % e.tiles;
                it += (uint32_t)n;
                return;
            }
        }
        for (int i = 0; i < n && valid(e); ++i) {
            ++it;
            if (++h < e.tiles) continue;
            h = 0;
            if (++kb >= kb1) {
                u += e.step;
                open_unit(e);
            }
        }
    }
};

// Ask for `bytes` (a multiple of 16) at `p` to be brought into L2; nothing waits for it.
__device__ __forceinline__ void prefetch_l2(const void *p, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

// --------------------------------------------------------------------------- token sums
// out[m] = offset * sum_k Xq[m][k]: what the offset form of the decode tables adds to every
// accumulator of token m.  One CTA per token; launched in front of the main kernel.
__global__ void __launch_bounds__(256)
token_offsum_kernel(const int8_t *__restrict__ Xq, int K, int offset, int32_t *__restrict__ out)
{
    __shared__ int red[8];
    allow_dependents();
    dependent_wait();                      // Xq may be the output of the kernel before
    const int4 *row = reinterpret_cast<const int4 *>(Xq + (size_t)blockIdx.x * K);
    int s = 0;
    const int n16 = K / 16;
    // four independent 16-byte loads per thread and round: the kernel is a pure read of Xq
    for (int i0 = threadIdx.x; i0 < n16; i0 += 4 * 256) {
        int4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = i0 + j * 256;
            v[j] = i < n16 ? __ldg(row + i) : make_int4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            s = __dp4a(v[j].x, 0x01010101, s);
            s = __dp4a(v[j].y, 0x01010101, s);
            s = __dp4a(v[j].z, 0x01010101, s);
            s = __dp4a(v[j].w, 0x01010101, s);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int w = 0; w < 8; ++w) t += red[w];
        out[blockIdx.x] = t * offset;
    }
}

// --------------------------------------------------------------------------- the kernel
// VARIANT: 4 = 4-bit codes, 3 = 3-bit codes, kAsymGroupVariant = 4-bit codes in groups with
// asymmetric activations (a kernel of its own: the zero-point correction in the loop over the
// groups, even as an untaken branch, was measured to cost the symmetric path a quarter of its
// throughput through register pressure), kSwigluVariant = 4-bit codes with the gated-unit
// epilogue (rows 2i / 2i + 1 of the weight matrix are feature i of the gate / up projection;
// the output is silu(gate) * up in binary16, half as wide as the weight matrix is tall)
template <int TOK, bool GROUPED, int DW, int CL, int VARIANT>
__global__ void __launch_bounds__(Cfg<TOK, GROUPED, DW, CL>::kThreads, 1)
linear_tcgen05_kernel(const __grid_constant__ CUtensorMap tok_map,
                      const __grid_constant__ CUtensorMap y_map, const Params P)
{
    using C = Cfg<TOK, GROUPED, DW, CL>;
    constexpr int BITS = VARIANT == 3 ? 3 : 4;
    constexpr bool SWIGLU = VARIANT == kSwigluVariant;
    constexpr bool ASYM_GROUP = VARIANT == kAsymGroupVariant;
    constexpr bool kRuns = !GROUPED && TOK >= 128 && VARIANT == 4;   // see unit_tiles
    static_assert(!ASYM_GROUP || GROUPED, "the asymmetric group variant is a group-mode kernel");
    constexpr int kFirstEpiWarp = C::kFirstEpiWarp;
    constexpr int S = C::kStages;
    extern __shared__ uint8_t smem_raw[];

    allow_dependents();

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar_base = base + C::kOffBarriers;
    const uint32_t bar_dec = bar_base;                   // S: operands of the stage in place
    const uint32_t bar_empty = bar_base + 8 * S;         // S: MMAs of the stage retired
    constexpr int NB = C::kAccBufs;
    const uint32_t bar_acc_full = bar_base + 16 * S;          // NB
    const uint32_t bar_acc_empty = bar_acc_full + 8 * NB;     // NB
    const uint32_t bar_drain = bar_acc_empty + 8 * NB;        // 1
    Ctl *ctl = reinterpret_cast<Ctl *>(gen_base + C::kOffBarriers + 16 * S + 16 * NB + 16);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // role of this warp and its index inside the role
    enum { kProducer, kMma, kDecode, kEpilogue };
    int role, role_idx = 0;
    if (warp == 0) role = kProducer;
    else if (warp == 1) role = kMma;
    else if (warp < kFirstEpiWarp) { role = kDecode; role_idx = warp - kFirstDecodeWarp; }
    else { role = kEpilogue; role_idx = warp - kFirstEpiWarp; }
    // Units (token-tile group, row-tile group, K slice) are dealt round-robin to the clusters.
    // Sharing pair: CTA `rank` takes token tile 2 * group + rank of the unit.  MMA pair: CTA
    // `rank` takes row tile 2 * group + rank.
    constexpr bool kShare = C::kShare, kPair = C::kPair, kDual = C::kDual;
    constexpr int kTiles = C::kTiles, kSub = C::kSub;
    const uint32_t rank = C::kCtas > 1 ? cluster_ctarank() : 0u;
    const int unit0 = (int)blockIdx.x / C::kCtas, unit_step = (int)gridDim.x / C::kCtas;
    // row-tile groups of the unit list, and this CTA's row / token tile inside a unit
    const int nt_groups = (kPair || kDual) ? P.L.n_tiles / 2 : P.L.n_tiles;
    auto row_tile = [&](int g, int h = 0) { return kPair ? 2 * g + (int)rank : kDual ? 2 * g + h : g; };
    auto tok_tile_of = [&](int g) { return kShare ? 2 * g + (int)rank : g; };
    // the barriers the MMA thread waits on live in the leader CTA of an MMA pair
    const bool leader = !kPair || rank == 0u;
    auto at_leader = [&](uint32_t bar) { return kPair ? map_to_cta(bar, 0u) : bar; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            // the warps of a decode team and the producer's arrival; the token copy and, in a
            // cluster, the peer's half of the expanded rows complete on it too
            // (MMA pair: the leader's barrier collects both CTAs' arrivals)
            // (MMA pair: the leader's barrier collects the decode warps of both CTAs)
            // (two row tiles per CTA: the teams of both tiles)
            mbar_init(bar_dec + 8 * s, C::kPerRound * C::kTeamWarps * (kPair ? 2 : 1) + 1);
            // sharing pair: the MMA threads of both CTAs, which all read rows this CTA wrote
            mbar_init(bar_empty + 8 * s, kShare ? 2 : 1);
        }
        for (int b = 0; b < NB; ++b) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, C::kEpiWarps * (kPair ? 2 : 1));
        }
        mbar_init(bar_drain, 1);
        ctl->abort = 0;
        ctl->is_last = 0;
        ctl->wait_ns = P.wait_ns;
        ctl->drain_ns = P.drain_ns;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    if (role == kMma) {
        if (kPair) {
            // the MMA warps of both CTAs allocate the same columns together
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                             smem_u32(&ctl->tmem_base)),
                         "r"((uint32_t)C::kTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                             smem_u32(&ctl->tmem_base)),
                         "r"((uint32_t)C::kTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    // no CTA may touch a peer's barriers or stages before the peer has set them up
    if (C::kCtas > 1) cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    // Set-up is done; earlier work in the stream (the activation quantizer, a previous call's
    // use of the workspace, the packing) is complete and visible from here on.
    dependent_wait();
    const bool blob_ok = header_matches(P.blob, P.L);

    const int n_tiles = P.L.n_tiles, k_blocks = P.L.k_blocks;
    const CursorEnv env = {unit_step, P.total_units, P.split_k, P.kb_per_split, k_blocks, nt_groups,
                           P.tok_groups, P.tok_run, kTiles};

    if (!blob_ok) {
        // not the blob the caller described: nothing is read or written, only the status
        if (threadIdx.x == 0) report_failure(P.sb, W4A8_ERR_BAD_BLOB, 2);
    } else if (role == kProducer) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            KbCursor<kRuns> pf;
            pf.start(unit0, env);
            for (int u = unit0; u < P.total_units && ok; u += unit_step) {
                const int s = u % P.split_k, rest = u / P.split_k;
                int row_group, tok_group;
                unit_tiles<kRuns>(rest, nt_groups, P.tok_groups, P.tok_run, row_group, tok_group);
                const int tt = tok_tile_of(tok_group);
                const int nt_of_unit = row_tile(row_group);
                const int kb0 = s * P.kb_per_split;
                const int kb1 = min(k_blocks, kb0 + P.kb_per_split);
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    // token buffer it % S, last used by k-block it - S: free once the round of
                    // that k-block has retired; the copy completes on the barrier of its own round
                    const int st = it % S;
                    if (it >= (uint32_t)S) {
                        const uint32_t r = (it - (uint32_t)S) / kSub;
                        if (!wait_bounded(bar_empty + 8 * (r % S), (r / S) & 1u, ctl, P.sb, 10)) {
                            ok = false;
                            break;
                        }
                    }
                    if (P.skip_load != 0 && it == (uint32_t)(P.skip_load - 1)) continue;
                    const uint32_t tok_dst = base + C::kOffTokRing + st * C::kTokBytes;
                    const uint32_t tok_bar = bar_dec + 8 * ((it / kSub) % S);
                    if (kPair) {
                        // this CTA's 128 of the tile's 256 tokens; completion counts at the leader
                        // (the leader's copy thread announces both CTAs' bytes with its own
                        // arrival; the other CTA only issues its copy: a release-arrival on a
                        // remote barrier was measured to cost that thread about a microsecond)
                        const uint32_t lead_bar = at_leader(tok_bar);
                        // (once per round: the bytes of both its k-blocks)
                        if (rank == 0u && it % kSub == 0) mbar_arrive_expect_tx(tok_bar, 2 * kSub * C::kTokBytes);
                        tma_load_2d_pair(tok_dst, &tok_map, kb * kTileK,
                                         tt * TOK + (int)rank * C::kTokRows, lead_bar);
                    } else {
                        mbar_arrive_expect_tx(tok_bar, C::kTokBytes + (kShare ? kABytes / 2 : 0));
                        tma_load_2d(tok_dst, &tok_map, kb * kTileK,
                                    nt_of_unit * P.batch_rows + tt * TOK, tok_bar);
                    }
                    if (P.prefetch_codes) {
                        // keep the code stream kPrefetchAhead k-blocks ahead of the decode warps
                        while (pf.valid(env) && pf.it < (it + C::kPrefetchAhead) * kTiles) {
                            const int pnt = row_tile(pf.nt, pf.h);
                            prefetch_l2(P.codes + ((size_t)pnt * k_blocks + pf.kb) * (BITS == 3 ? kTileBytes3 : kTileBytes),
                                        BITS == 3 ? kTileBytes3 : kTileBytes);
                            pf.advance(1, env);
                        }
                    }
                }
            }
            if (!ok && leader) {
                // copies already issued must land before the CTA gives its memory back (in an MMA
                // pair the leader's barriers count both CTAs' copies, and the other CTA stays
                // until the leader is through: the cluster barrier at the end)
                // (a round of which only a part was issued never completes: that wait runs out)
                const uint32_t first = (it > (uint32_t)S ? it - S : 0u) / kSub;
                for (uint32_t j = first; j < (it + kSub - 1) / kSub; ++j)
                    wait_bounded(bar_dec + 8 * (j % S), (j / S) & 1u, ctl, P.sb, 11, true);
            }
        }
        __syncwarp();
    } else if (role == kMma) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && leader) {
            // This loop is the serial spine of the kernel (one thread, once per k-block): all
            // counters are kept incrementally and the descriptors are an add away.
            constexpr uint32_t idesc = instr_desc_i8(TOK, kPair ? 256 : 128);
            constexpr uint16_t kBoth = 3;                // both CTAs of the cluster
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
            const uint32_t a_lo0 = ((base & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t b_lo0 = (((base + C::kOffTokRing) & 0x3FFFFu) >> 4) | (1u << 16);
            uint32_t st = 0, st_par = 0;                 // barrier slot of the round and its parity
            uint32_t sa = 0, tb = 0;                     // weight buffer, token buffer
            uint32_t buf = 0, buf_par = 0;               // accumulator buffer and its parity
            bool ok = true;
            for (int u = unit0; u < P.total_units && ok; u += unit_step) {
                const int s = u % P.split_k;
                const int kb0 = s * P.kb_per_split;
                const int nkb = min(k_blocks, kb0 + P.kb_per_split) - kb0;
                for (int i = 0; i < nkb; i += C::kSub) {
                    const bool first = GROUPED || i == 0;
                    const bool last = GROUPED || i + C::kSub >= nkb;
                    if (!kDual && first &&
                        !wait_bounded<kPair>(bar_acc_empty + 8 * buf, buf_par ^ 1u, ctl, P.sb, 20)) {
                        ok = false;
                        break;
                    }
                    // decoded weights and tokens of the round
                    if (!wait_bounded<kPair>(bar_dec + 8 * st, st_par, ctl, P.sb, 21)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    if constexpr (kDual) {
                        // both row tiles of the unit against the same tokens; accumulator h belongs
                        // to tile h, and the epilogue hands the two back one after the other
                        const uint64_t b_desc = ((uint64_t)kDescHi << 32) | (b_lo0 + tb * (C::kTokBytes >> 4));
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if (first &&
                                !wait_bounded(bar_acc_empty + 8 * h, buf_par ^ 1u, ctl, P.sb, 20)) {
                                ok = false;
                                break;
                            }
                            if (first) tc_fence_after();
                            const uint64_t a_desc = ((uint64_t)kDescHi << 32) | (a_lo0 + sa * (kABytes >> 4));
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)
                                tc_mma_i8(tmem_base + h * TOK, a_desc + (uint64_t)(ks * 2),
                                          b_desc + (uint64_t)(ks * 2), idesc, (!first || ks > 0) ? 1u : 0u);
                            if (++sa == (uint32_t)C::kAStages) sa = 0;
                        }
                        if (!ok) break;
                        if (++tb == (uint32_t)S) tb = 0;
                        tc_commit(bar_empty + 8 * st);
                        if (last) {
                            tc_commit(bar_acc_full);
                            tc_commit(bar_acc_full + 8);
                            buf_par ^= 1u;
                        }
                    } else {
                        const uint32_t d = tmem_base + buf * TOK;
#pragma unroll
                        for (int h = 0; h < C::kSub; ++h) {
                            // (the k-blocks of a round: one weight and one token buffer each)
                            const uint64_t a_desc = ((uint64_t)kDescHi << 32) | (a_lo0 + sa * (kABytes >> 4));
                            const uint64_t b_desc = ((uint64_t)kDescHi << 32) | (b_lo0 + tb * (C::kTokBytes >> 4));
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks) {
                                const uint32_t acc_flag = (!first || h > 0 || ks > 0) ? 1u : 0u;
                                if (kPair)
                                    tc_mma_i8_pair(d, a_desc + (uint64_t)(ks * 2), b_desc + (uint64_t)(ks * 2),
                                                   idesc, acc_flag);
                                else
                                    tc_mma_i8(d, a_desc + (uint64_t)(ks * 2), b_desc + (uint64_t)(ks * 2), idesc,
                                              acc_flag);
                            }
                            if (++sa == (uint32_t)C::kAStages) sa = 0;
                            if (++tb == (uint32_t)S) tb = 0;
                        }
                        if (kPair) tc_commit_pair(bar_empty + 8 * st, kBoth);
                        else if (kShare) tc_commit_multicast(bar_empty + 8 * st, kBoth);
                        else tc_commit(bar_empty + 8 * st);
                        if (last) {
                            if (kPair) tc_commit_pair(bar_acc_full + 8 * buf, kBoth);
                            else tc_commit(bar_acc_full + 8 * buf);
                            if (++buf == (uint32_t)NB) { buf = 0; buf_par ^= 1u; }
                        }
                    }
                    if (++st == (uint32_t)S) { st = 0; st_par ^= 1u; }
                }
            }
            // nothing issued may still be running when tensor memory is freed
            if (kPair) tc_commit_pair(bar_drain, 1); else tc_commit(bar_drain);
            wait_bounded(bar_drain, 0u, ctl, P.sb, 22, !ok);
        }
        __syncwarp();
    } else if (role == kDecode) {
        // ------------------------------------------------------------------ decode warps
        // The warps of a team share a k-block (a thread takes one feature row and one column
        // slice of it); teams take k-blocks in turn, so the fixed latency of one k-block (barrier
        // wait, loads, proxy fence, arrive) overlaps the table lookups of the other teams.
        const int dt = role_idx * 32 + lane;
        constexpr int QT = C::kQuartersPerThread;
        // One thread per row of the tile; in a cluster this CTA takes 64 of the rows, a warp 16 of
        // them, and a thread half a row, so that a warp's rows are one contiguous 2 KiB piece of
        // the stage.
        const int r = !kShare ? (dt & 127)
                              : (int)rank * C::kRowsPerCta + ((dt >> 5) & 3) * 16 + (lane & 15);
        const int q0 = !kShare ? 0 : (lane >> 4) * QT;       // first 32-k quarter of this thread
        const int team = dt / (32 * C::kTeamWarps);
        constexpr int T = C::kTeams;
        // the same stage and barrier in the peer CTA
        const uint32_t peer = rank ^ 1u;
        KbCursor<kRuns> cur;
        cur.start(unit0, env);
        cur.advance(team, env);
        // Items (k-block, row tile of the unit) are numbered in the order the MMAs use them.  The
        // weight buffer of item `it` is free once the MMAs of item it - kAStages, its last user,
        // have retired (their commit completed a phase of that item's k-block's barrier slot).
        auto wait_a_free = [&](uint32_t it) -> bool {
            if (it < (uint32_t)C::kAStages) return true;
            const uint32_t j = (it - (uint32_t)C::kAStages) / C::kPerRound;
            return wait_bounded(bar_empty + 8 * (j % S), (j / S) & 1u, ctl, P.sb, 31);
        };
        if constexpr (BITS == 3) {
            // 3-bit codes: twelve words per row and k-block (three per 32-k quarter, each read
            // as 128 contiguous bytes by a warp); the selector nibbles of eight codes are the
            // words with their top bits cleared, the fourth selector of a quarter is put
            // together from those top bits; one byte permute on the two table words yields four
            // levels.  One thread per row (no clusters in this mode).
            static_assert(CL == 1, "3-bit codes: one CTA per cluster");
            uint32_t w3[12];
            int z3 = 0;
            auto fetch3 = [&](const KbCursor<kRuns> &c, uint32_t (&dst)[12], int &zz) {
                const int n = c.nt * kTileN + r;
                zz = GROUPED ? P.zeros[(size_t)c.kb * P.L.n_pad + n] : P.zeros[n];
                const uint32_t *src = reinterpret_cast<const uint32_t *>(
                    P.codes + ((size_t)c.nt * k_blocks + c.kb) * kTileBytes3 + r * 4);
#pragma unroll
                for (int i = 0; i < 12; ++i) {
                    uint32_t v;
                    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(src + i * 128));
                    dst[i] = v;
                }
            };
            if (cur.valid(env)) fetch3(cur, w3, z3);
            bool ok3 = true;
            while (cur.valid(env) && ok3) {
                KbCursor<kRuns> nxt = cur;
                nxt.advance(C::kTeams, env);
                uint32_t wn3[12];
                int zn3 = 0;
                if (nxt.valid(env)) fetch3(nxt, wn3, zn3);
                const int st = (cur.it / C::kPerRound) % S, sa = cur.it % C::kAStages;
                uint32_t t3[2];
                build_level_tables3(z3, P.L.shift, t3);
                ok3 = wait_a_free(cur.it);
                ok3 = __all_sync(0xffffffffu, ok3);
                if (!ok3) break;
                uint8_t *arow = gen_base + sa * kABytes + r * 128;
                const int sw = r & 7;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint32_t a = w3[3 * q], b = w3[3 * q + 1], c = w3[3 * q + 2];
                    const uint32_t s0 = a & 0x77777777u, s1 = b & 0x77777777u, s2 = c & 0x77777777u;
                    const uint32_t s3 = ((a >> 3) & 0x11111111u) | ((b >> 2) & 0x22222222u) |
                                        ((c >> 1) & 0x44444444u);
                    uint4 c0, c1;
                    c0.x = prmt(t3[0], t3[1], s0); c0.y = prmt(t3[0], t3[1], s0 >> 16);
                    c0.z = prmt(t3[0], t3[1], s1); c0.w = prmt(t3[0], t3[1], s1 >> 16);
                    c1.x = prmt(t3[0], t3[1], s2); c1.y = prmt(t3[0], t3[1], s2 >> 16);
                    c1.z = prmt(t3[0], t3[1], s3); c1.w = prmt(t3[0], t3[1], s3 >> 16);
                    *reinterpret_cast<uint4 *>(arow + (((2 * q) ^ sw) << 4)) = c0;
                    *reinterpret_cast<uint4 *>(arow + (((2 * q + 1) ^ sw) << 4)) = c1;
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_dec + 8 * st);
#pragma unroll
                for (int i = 0; i < 12; ++i) w3[i] = wn3[i];
                z3 = zn3;
                cur = nxt;
            }
        } else {
        uint4 w[QT];
        int z = 0;
        auto fetch = [&](const KbCursor<kRuns> &c, uint4 (&dst)[QT], int &zz) {
            const int nt = row_tile(c.nt, c.h);
            const int n = nt * kTileN + r;
            zz = GROUPED ? P.zeros[(size_t)c.kb * P.L.n_pad + n] : P.zeros[n];
            const uint4 *src = reinterpret_cast<const uint4 *>(
                P.codes + ((size_t)nt * k_blocks + c.kb) * kTileBytes + r * 16);
#pragma unroll
            for (int q = 0; q < QT; ++q) dst[q] = ld_stream(src + (q0 + q) * (kQuarterBytes / 16));
        };
        if (cur.valid(env)) fetch(cur, w, z);
        bool ok = true;
        const bool use_offset = !GROUPED && P.offset != 0;   // (per-channel weights only)
        uint32_t one = 1u;                       // opaque to the compiler: see decode8_offset
        asm volatile("" : "+r"(one));
        while (cur.valid(env) && ok) {
            KbCursor<kRuns> nxt = cur;
            nxt.advance(T, env);
            const int st = (cur.it / C::kPerRound) % S, sa = cur.it % C::kAStages;
            uint32_t t[4];
            if (use_offset) build_offset_tables(z, P.lt, P.L.shift, t);
            else build_level_tables(z, P.lt, t);
            uint4 lv[2 * QT];                    // the thread's INT8 levels, 16 per register quad
            auto expand = [&]() {
                if (use_offset) {
#pragma unroll
                    for (int q = 0; q < QT; ++q) {
                        const uint4 wq = w[q];
                        decode8_offset(wq.x, t, one, lv[2 * q].x, lv[2 * q].y);
                        decode8_offset(wq.y, t, one, lv[2 * q].z, lv[2 * q].w);
                        decode8_offset(wq.z, t, one, lv[2 * q + 1].x, lv[2 * q + 1].y);
                        decode8_offset(wq.w, t, one, lv[2 * q + 1].z, lv[2 * q + 1].w);
                    }
                    return;
                }
#pragma unroll
                for (int q = 0; q < QT; ++q) {
                    const uint4 wq = w[q];
                    decode8(wq.x, t, lv[2 * q].x, lv[2 * q].y);
                    decode8(wq.y, t, lv[2 * q].z, lv[2 * q].w);
                    decode8(wq.z, t, lv[2 * q + 1].x, lv[2 * q + 1].y);
                    decode8(wq.w, t, lv[2 * q + 1].z, lv[2 * q + 1].w);
                }
            };
            // The levels are ready in registers before the buffer is: only the stores stand between
            // the moment the buffer is free and the moment its operand is in place (the expansion
            // of a tile takes a team a few thousand cycles while all teams work, more than the
            // ring of weight buffers can hide).  The codes of the team's next item are requested
            // only now, into the registers the expansion has just read, so a thread holds raw
            // codes and levels of one item at a time; the wait and the stores cover the loads.
            // (Group mode measured the same with either order.)
            int zn = 0;
            expand();
#pragma unroll
            for (int q = 0; q < 2 * QT; ++q)
                asm volatile("" : "+r"(lv[q].x), "+r"(lv[q].y), "+r"(lv[q].z), "+r"(lv[q].w));
            if (nxt.valid(env)) fetch(nxt, w, zn);
            {
                // (all lanes poll: one polling lane per warp was measured a quarter slower)
                ok = wait_a_free(cur.it);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                uint8_t *arow = gen_base + sa * kABytes + r * 128;
                const int sw = r & 7;
#pragma unroll
                for (int q = 0; q < QT; ++q) {
                    *reinterpret_cast<uint4 *>(arow + (((2 * (q0 + q)) ^ sw) << 4)) = lv[2 * q];
                    *reinterpret_cast<uint4 *>(arow + (((2 * (q0 + q) + 1) ^ sw) << 4)) = lv[2 * q + 1];
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    if (kPair && rank != 0u) mbar_arrive_cluster(at_leader(bar_dec + 8 * st));
                    else mbar_arrive(bar_dec + 8 * st);
                    if (kShare) {
                        // this warp's 16 rows, now complete in the local stage, go to the peer
                        const uint32_t piece = base + sa * kABytes + (uint32_t)(r * 128);
                        bulk_copy_to_cta(map_to_cta(piece, peer), piece, 16 * 128,
                                         map_to_cta(bar_dec + 8 * st, peer));
                    }
                }
            }
            z = zn;
            cur = nxt;
        }
        }   // 4-bit codes
    } else if (role == kEpilogue) {
        // ------------------------------------------------------------------ epilogue warps
        const int ew = role_idx;
        const int quarter = warp & 3;                     // tensor-memory lane quarter
        const int col_group = ew >> 2;                    // which share of the columns
        const int col0 = col_group * C::kColsPerThread;
        const int f = quarter * 32 + lane;                // feature row inside the tile
        constexpr int kEpiThreads = 32 * C::kEpiWarps;
        const int et = ew * 32 + lane;
        const bool elected = et == col_group * 128;       // issues this group's bulk stores
        const int group_bar = 2 + col_group;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        float *s_tok = reinterpret_cast<float *>(gen_base + C::kOffTok);
        int *s_tz = reinterpret_cast<int *>(gen_base + C::kOffTok + 1024);   // tokens' zero-points
        int *s_off = reinterpret_cast<int *>(gen_base + C::kOffTok + 2048);  // offset * token sum
        __nv_bfloat16 *stg =
            reinterpret_cast<__nv_bfloat16 *>(gen_base + C::kOffStaging) +
            col_group * C::kStageBufs * C::kChunk * kTileN;
        // Outputs leave through shared memory: the accumulator has one feature per thread,
        // the output row is one token, so a chunk of kChunk tokens x 128 features is
        // transposed into a staging buffer and written by one bulk tensor store.
        const bool bulk_out = P.Y != nullptr && P.split_k == 1;
        uint32_t phase = 0, stores = 0;
        bool ok = true;

        auto emit = [&](const float (&tv)[32], int nt, int tok_row) {
            const uint32_t sbuf = stores % C::kStageBufs;
            if (elected) bulk_wait_read<C::kStageBufs - 1>();   // the buffer's last store has been read
            named_bar_sync(group_bar, 128);
            if constexpr (SWIGLU) {
                // lanes 2i and 2i + 1 hold the gate and the up value of feature i: the even
                // lane takes its neighbour's value and writes silu(gate) * up, 64 features per
                // token in the staging buffer
                __half *dst = reinterpret_cast<__half *>(stg + sbuf * (C::kChunk * kTileN)) + (f >> 1);
#pragma unroll
                for (int j = 0; j < C::kChunk; ++j) {
                    const float up = __shfl_xor_sync(0xffffffffu, tv[j], 1);
                    const float gate = tv[j];
                    const float h = __fmul_rn(__fdiv_rn(gate, __fadd_rn(1.0f, __expf(-gate))), up);
                    if ((lane & 1) == 0) dst[j * (kTileN / 2)] = __float2half_rn(h);
                }
            } else {
                __nv_bfloat16 *dst = stg + sbuf * (C::kChunk * kTileN) + f;
#pragma unroll
                for (int j = 0; j < C::kChunk; ++j) dst[j * kTileN] = __float2bfloat16_rn(tv[j]);
            }
            fence_proxy_async();
            named_bar_sync(group_bar, 128);
            if (elected) {
                tma_store_2d(&y_map, smem_u32(stg + sbuf * (C::kChunk * kTileN)),
                             SWIGLU ? nt * (kTileN / 2) : nt * kTileN, tok_row);
                bulk_commit();
            }
            ++stores;
        };

        for (int uh = unit0 * kTiles; uh < P.total_units * kTiles && ok;
             uh += ((uh + 1) % kTiles == 0 ? (unit_step - 1) * kTiles + 1 : 1)) {
            // (two row tiles per unit: tile 0 from accumulator 0, then tile 1 from accumulator 1)
            const int u = uh / kTiles, h = uh % kTiles;
            const int s = u % P.split_k, rest = u / P.split_k;
            int row_group, tok_group;
            unit_tiles<kRuns>(rest, nt_groups, P.tok_groups, P.tok_run, row_group, tok_group);
            const int nt = row_tile(row_group, h), tt = tok_tile_of(tok_group);
            const int kb0 = s * P.kb_per_split;
            const int kb1 = min(k_blocks, kb0 + P.kb_per_split);
            const int n = nt * kTileN + f;
            const bool n_ok = n < P.L.N;
            const int tok0 = tt * TOK + col0;
            int valid = P.M - tok0;                       // columns of this thread that are tokens
            valid = valid < 0 ? 0 : (valid > C::kColsPerThread ? C::kColsPerThread : valid);
            const float bias_n = (P.bias && n_ok) ? P.bias[n] : 0.0f;

            if (P.Y || P.zp.tok_zero || P.offset) {
                // token step sizes (and zero-points) of this tile, shared by all epilogue threads
                named_bar_sync(1, kEpiThreads);
                for (int i = et; i < TOK; i += kEpiThreads) {
                    const bool in = tt * TOK + i < P.M;
                    s_tok[i] = (in && P.tok_scale) ? __ldg(P.tok_scale + nt * P.batch_rows + tt * TOK + i) : 0.0f;
                    s_tz[i] = (in && P.zp.tok_zero) ? __ldg(P.zp.tok_zero + tt * TOK + i) : 0;
                    s_off[i] = (in && P.offset) ? __ldcg(P.tok_offsum + nt * P.batch_rows + tt * TOK + i) : 0;
                }
                named_bar_sync(1, kEpiThreads);
            }

            if (!GROUPED) {
                const float half_step = __fmul_rn(P.unit, P.scales[n]);
                // asymmetric activations: the token's zero-point times this row's level sum
                // leaves the accumulator before the rescale (zero for the symmetric path)
                const int row_sum = (P.zp.rowsum && n_ok) ? __ldg(P.zp.rowsum + n) : 0;
                const uint32_t buf = phase % NB;
                ok = wait_bounded_idle(bar_acc_full + 8 * buf, (phase / NB) & 1u, ctl, P.sb, 40);
                ok = named_bar_and(1, kEpiThreads, ok);
                if (!ok) break;
                tc_fence_after();
                ++phase;
                int32_t *part = reinterpret_cast<int32_t *>(P.partials);
#pragma unroll 1
                for (int c = 0; c < C::kColsPerThread; c += C::kChunk) {
                    uint32_t v[32];
                    const uint32_t taddr = tmem_base + lane_base + buf * TOK + col0 + c;
                    if (C::kChunk == 32) tc_ld32(taddr, v); else tc_ld16(taddr, v);
                    tc_wait_ld();
                    if (c + C::kChunk >= C::kColsPerThread) {
                        // the accumulator is in registers: hand the buffer back
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            if (kPair && rank != 0u) mbar_arrive_cluster(at_leader(bar_acc_empty + 8 * buf));
                            else mbar_arrive(bar_acc_empty + 8 * buf);
                        }
                    }
                    if (c >= valid) continue;             // uniform over the column group
                    if ((P.zp.tok_zero || P.offset) && P.split_k == 1) {
                        // the token's zero-point times the row's level sum, and the offset of the
                        // decode tables times the token's own sum, leave the accumulator
#pragma unroll
                        for (int j = 0; j < C::kChunk; ++j)
                            v[j] = (uint32_t)((int)v[j] - s_tz[col0 + c + j] * row_sum - s_off[col0 + c + j]);   // (both staged: zero when unused)
                    }
                    if (P.acc_out && P.split_k == 1 && n_ok) {
#pragma unroll
                        for (int j = 0; j < C::kChunk; ++j)
                            if (c + j < valid)
                                P.acc_out[(size_t)(tok0 + c + j) * P.L.N + n] = (int)v[j];
                    }
                    if (bulk_out) {
                        float tv[32];
#pragma unroll
                        for (int j = 0; j < C::kChunk; ++j) {
                            float x = rescale_channel((int)v[j], s_tok[col0 + c + j], half_step);
                            if (P.bias) x = __fadd_rn(x, bias_n);
                            tv[j] = x;
                        }
                        emit(tv, nt, tok0 + c);
                    } else if (P.split_k > 1) {
#pragma unroll
                        for (int j = 0; j < C::kChunk; ++j) {
                            if (c + j < valid) {
                                const int m = tok0 + c + j;
                                part[((size_t)s * P.m_pad + m) * P.L.n_pad + n] = (int)v[j];
                            }
                        }
                    }
                }
                if (P.split_k > 1) {
                    __threadfence();
                    named_bar_sync(1, kEpiThreads);
                    if (et == 0) {
                        const int old = atomicAdd(P.counters + (size_t)tt * n_tiles + nt, 1);
                        const int last = old == P.split_k - 1;
                        if (last) P.counters[(size_t)tt * n_tiles + nt] = 0;
                        ctl->is_last = last;
                    }
                    named_bar_sync(1, kEpiThreads);
                    const bool is_last = ctl->is_last != 0;
                    named_bar_sync(1, kEpiThreads);
                    if (is_last && n_ok) {
                        __threadfence();
                        // eight tokens at a time, so that many independent loads are in flight
                        // (rows past the last token exist in the padded buffer and are ignored)
                        for (int j0 = 0; j0 < valid; j0 += 8) {
                            int acc[8];
#pragma unroll
                            for (int t = 0; t < 8; ++t) acc[t] = 0;
#pragma unroll 2
                            for (int ss = 0; ss < P.split_k; ++ss) {
                                const int32_t *row =
                                    part + ((size_t)ss * P.m_pad + tok0 + j0) * P.L.n_pad + n;
#pragma unroll
                                for (int t = 0; t < 8; ++t)
                                    if (j0 + t < C::kColsPerThread)
                                        acc[t] += __ldcg(row + (size_t)t * P.L.n_pad);
                            }
#pragma unroll
                            for (int t = 0; t < 8; ++t) {
                                const int j = j0 + t;
                                if (j >= valid) break;
                                const int m = tok0 + j;
                                if (P.zp.tok_zero) acc[t] -= s_tz[col0 + j] * row_sum;
                                if (P.offset) acc[t] -= s_off[col0 + j];
                                if (P.acc_out) P.acc_out[(size_t)m * P.L.N + n] = acc[t];
                                if (P.Y) {
                                    float x = rescale_channel(acc[t], s_tok[col0 + j], half_step);
                                    if (P.bias) x = __fadd_rn(x, bias_n);
                                    P.Y[(size_t)m * P.L.N + n] = __float2bfloat16_rn(x);
                                }
                            }
                        }
                    }
                }
            } else {
                // FP32 sums over the groups, two tokens per 64-bit register: each k-block adds
                // float(partial) * step/2 with one packed add and one packed fused multiply-add
                // per pair (same roundings as the scalar fmaf)
                uint64_t usum2[C::kColsPerThread / 2];
#pragma unroll
                for (int j = 0; j < C::kColsPerThread / 2; ++j) usum2[j] = 0ull;
                uint32_t one = 1u;                       // opaque to the compiler: see biased_float_bits
                asm volatile("" : "+r"(one));
                const uint32_t neg_magic = __float_as_uint(-12582912.0f);
                const uint64_t neg_magic2 = pack_f32x2(neg_magic, neg_magic);
                constexpr int kAcc = 16;          // columns per tensor-memory load while accumulating
                {
                    constexpr bool ASYM = ASYM_GROUP;
                    // the next group's step is loaded one k-block ahead and only touched when
                    // used, so the warp never stalls on that load; the group's level sum of this
                    // row (asymmetric activations) likewise
                    float step_next = P.scales[(size_t)kb0 * P.L.n_pad + n];
                    int rs_next = 0;
                    if (ASYM) rs_next = n_ok ? __ldg(P.zp.rowsum + (size_t)kb0 * P.L.N + n) : 0;
                    for (int kb = kb0; kb < kb1; ++kb) {
                        const uint32_t h_bits = __float_as_uint(__fmul_rn(P.unit, step_next));
                        const uint64_t h2 = pack_f32x2(h_bits, h_bits);
                        const int rs = rs_next;
                        if (kb + 1 < kb1) {
                            step_next = P.scales[(size_t)(kb + 1) * P.L.n_pad + n];
                            if (ASYM && n_ok) rs_next = __ldg(P.zp.rowsum + (size_t)(kb + 1) * P.L.N + n);
                        }
                        const uint32_t buf = phase % NB;
                        ok = wait_bounded(bar_acc_full + 8 * buf, (phase / NB) & 1u, ctl, P.sb, 41);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        tc_fence_after();
                        ++phase;
#pragma unroll
                        for (int c = 0; c < C::kColsPerThread; c += kAcc) {
                            uint32_t v[32];
                            const uint32_t taddr = tmem_base + lane_base + buf * TOK + col0 + c;
                            tc_ld16(taddr, v);
                            tc_wait_ld();
                            if (c + kAcc >= C::kColsPerThread) {
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(bar_acc_empty + 8 * buf);
                            }
                            if (ASYM) {
                                // the token's zero-point times the group's level sum leaves the
                                // integer partial before it is scaled
#pragma unroll
                                for (int j = 0; j < kAcc; ++j)
                                    v[j] = (uint32_t)((int)v[j] - s_tz[col0 + c + j] * rs);
                            }
#pragma unroll
                            for (int j = 0; j < kAcc; j += 2) {
                                const uint64_t biased =
                                    pack_f32x2(biased_float_bits(v[j], one), biased_float_bits(v[j + 1], one));
                                usum2[(c + j) >> 1] =
                                    fma_f32x2(add_f32x2(biased, neg_magic2), h2, usum2[(c + j) >> 1]);
                            }
                            if (P.acc_out && n_ok) {
#pragma unroll
                                for (int j = 0; j < kAcc; ++j)
                                    if (c + j < valid)
                                        P.acc_out[((size_t)kb * P.M + tok0 + c + j) * P.L.N + n] =
                                            (int)v[j];
                            }
                        }
                    }
                }
                ok = named_bar_and(1, kEpiThreads, ok);
                if (!ok) break;
                float usum[C::kColsPerThread];
#pragma unroll
                for (int j = 0; j < C::kColsPerThread / 2; ++j)
                    unpack_f32x2(usum2[j], usum[2 * j], usum[2 * j + 1]);
                if (bulk_out) {
#pragma unroll
                    for (int c = 0; c < C::kColsPerThread; c += C::kChunk) {
                        if (c < valid) {
                            float tv[32];
#pragma unroll
                            for (int j = 0; j < C::kChunk; ++j) {
                                float x = __fmul_rn(usum[c + j], s_tok[col0 + c + j]);
                                if (P.bias) x = __fadd_rn(x, bias_n);
                                tv[j] = x;
                            }
                            emit(tv, nt, tok0 + c);
                        }
                    }
                } else if (P.split_k > 1) {
                    float *part = reinterpret_cast<float *>(P.partials);
#pragma unroll
                    for (int j = 0; j < C::kColsPerThread; ++j)
                        if (j < valid)
                            part[((size_t)s * P.m_pad + tok0 + j) * P.L.n_pad + n] = usum[j];
                    __threadfence();
                    named_bar_sync(1, kEpiThreads);
                    if (et == 0) {
                        const int old = atomicAdd(P.counters + (size_t)tt * n_tiles + nt, 1);
                        const int last = old == P.split_k - 1;
                        if (last) P.counters[(size_t)tt * n_tiles + nt] = 0;
                        ctl->is_last = last;
                    }
                    named_bar_sync(1, kEpiThreads);
                    const bool is_last = ctl->is_last != 0;
                    named_bar_sync(1, kEpiThreads);
                    if (is_last && n_ok && P.Y) {
                        __threadfence();
                        // eight tokens at a time (independent loads in flight); every token's
                        // slices are still added in slice order
                        for (int j0 = 0; j0 < valid; j0 += 8) {
                            float usm[8];
#pragma unroll
                            for (int t = 0; t < 8; ++t) usm[t] = 0.0f;
#pragma unroll 2
                            for (int ss = 0; ss < P.split_k; ++ss) {
                                const float *row =
                                    part + ((size_t)ss * P.m_pad + tok0 + j0) * P.L.n_pad + n;
#pragma unroll
                                for (int t = 0; t < 8; ++t)
                                    if (j0 + t < C::kColsPerThread)
                                        usm[t] = __fadd_rn(usm[t], __ldcg(row + (size_t)t * P.L.n_pad));
                            }
#pragma unroll
                            for (int t = 0; t < 8; ++t) {
                                const int j = j0 + t;
                                if (j >= valid) break;
                                float x = __fmul_rn(usm[t], s_tok[col0 + j]);
                                if (P.bias) x = __fadd_rn(x, bias_n);
                                P.Y[(size_t)(tok0 + j) * P.L.N + n] = __float2bfloat16_rn(x);
                            }
                        }
                    }
                }
            }
        }
        // the staging buffers must have been read before the CTA gives its memory back
        if (elected) bulk_wait_read<0>();
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    // a peer may still write this CTA's stages or arrive on its barriers until it is done too
    if (CL > 1) cluster_sync_all();
    if (role == kMma) {
        tc_fence_after();
        if (kPair)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                         "r"((uint32_t)C::kTmemCols)
                         : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                         "r"((uint32_t)C::kTmemCols)
                         : "memory");
    }
}

// --------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) ==
                cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

struct Maps {
    CUtensorMap tok, y16, y32;      // activations; output with 16- and 32-token boxes
};

// Tensor maps of a two-dimensional row-major tensor, kept per host thread: a serving loop calls
// with the same pointers and shapes over and over, and a map depends on nothing else (addresses
// are unique across the devices of a process).  Eight entries, replaced in turn.
struct MapKey {
    const void *base;
    unsigned long long dim0, dim1, stride;
    unsigned box0, box1;
    int dtype, swizzle, promotion;
    bool operator==(const MapKey &o) const
    {
        return base == o.base && dim0 == o.dim0 && dim1 == o.dim1 && stride == o.stride && box0 == o.box0 &&
               box1 == o.box1 && dtype == o.dtype && swizzle == o.swizzle && promotion == o.promotion;
    }
};
bool encode_2d(EncodeTiledFn enc, CUtensorMap *out, CUtensorMapDataType dtype, const void *base,
               cuuint64_t dim0, cuuint64_t dim1, cuuint64_t stride_bytes, cuuint32_t box0, cuuint32_t box1,
               CUtensorMapSwizzle swizzle, CUtensorMapL2promotion promotion)
{
    constexpr int kEntries = 8;
    thread_local MapKey keys[kEntries] = {};
    thread_local CUtensorMap maps[kEntries];
    thread_local int next = 0;
    const MapKey key = {base, dim0, dim1, stride_bytes, box0, box1, (int)dtype, (int)swizzle, (int)promotion};
    for (int i = 0; i < kEntries; ++i) {
        if (keys[i].base != nullptr && keys[i] == key) {
            *out = maps[i];
            return true;
        }
    }
    const cuuint64_t dims[2] = {dim0, dim1};
    const cuuint64_t strides[1] = {stride_bytes};
    const cuuint32_t box[2] = {box0, box1};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(out, dtype, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            swizzle, promotion, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    keys[next] = key;
    maps[next] = *out;
    next = (next + 1) % kEntries;
    return true;
}

// Clusters of CL CTAs of this kernel that the current device can hold at once (one CTA per
// SM); asked once per kernel instance and device.
template <int TOK, bool GROUPED, int DW, int CL, int VARIANT>
int resident_clusters()
{
    using C = Cfg<TOK, GROUPED, DW, CL>;
    static std::atomic<int> cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    int n = cached[dev].load(std::memory_order_acquire);
    if (n > 0) return n;
    auto kern = linear_tcgen05_kernel<TOK, GROUPED, DW, CL, VARIANT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) !=
        cudaSuccess)
        return 0;
    if (CL == 1) {
        n = device_sms();
    } else {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(C::kCtas * device_sms());
        cfg.blockDim = dim3(C::kThreads);
        cfg.dynamicSmemBytes = C::kSmemBytes;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = C::kCtas;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n < 1) {
            cudaGetLastError();
            return 0;
        }
    }
    cached[dev].store(n, std::memory_order_release);
    return n;
}

template <int TOK, bool GROUPED, int DW, int CL, int VARIANT = 4>
w4a8_status launch_cl(const Maps &maps, const Params &P, cudaStream_t st)
{
    using C = Cfg<TOK, GROUPED, DW, CL>;
    auto kern = linear_tcgen05_kernel<TOK, GROUPED, DW, CL, VARIANT>;
    const int resident = resident_clusters<TOK, GROUPED, DW, CL, VARIANT>();   // also sizes the kernel's shared memory
    if (resident < 1) return W4A8_ERR_CUDA;
    const int clusters = P.total_units < resident ? P.total_units : resident;
    const cudaError_t e =
        launch_overlapped_cluster(kern, dim3(clusters * C::kCtas), dim3(C::kThreads), (size_t)C::kSmemBytes, st, C::kCtas,
                          maps.tok, C::kChunk == 32 ? maps.y32 : maps.y16, P);
    return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

template <int TOK, bool GROUPED, int DW>
w4a8_status launch_dw(const Maps &maps, const Params &P, int cluster, cudaStream_t st)
{
    // two-CTA clusters exist for the wide token tiles: narrow ones serve few tokens
    if constexpr (TOK >= 128) {
        if (cluster == 2) return launch_cl<TOK, GROUPED, DW, 2>(maps, P, st);
    }
    if constexpr (TOK == 256 && !GROUPED && (DW == 8 || DW == 16)) {
        if (cluster == 3) return launch_cl<TOK, false, DW, 3>(maps, P, st);
        if constexpr (DW == 16) {
            if (cluster == 5) return launch_cl<TOK, false, 16, 5>(maps, P, st);
        }
    }
    if constexpr (TOK == 256 && !GROUPED && DW == 16) {
        if (cluster == 4) return P.batch_rows == 0 ? launch_cl<TOK, false, 16, 4>(maps, P, st) : W4A8_ERR_SHAPE;
    }
    if (cluster == 1) return launch_cl<TOK, GROUPED, DW, 1>(maps, P, st);
    return W4A8_ERR_SHAPE;
}

template <int TOK, bool GROUPED>
w4a8_status launch_one(const Maps &maps, const Params &P, int dw, int cluster, cudaStream_t st)
{
    // 3-bit codes: eight decode warps, no clusters (make_plan picks nothing else)
    if (P.L.bits == 3) return dw == 8 && cluster == 1 ? launch_cl<TOK, GROUPED, 8, 1, 3>(maps, P, st) : W4A8_ERR_SHAPE;
    // gated-unit epilogue: the default warps, no clusters, no K split (make_plan picks nothing else)
    if (P.swiglu) {
        if (cluster != 1 || P.split_k != 1 || dw != (GROUPED ? 8 : 16)) return W4A8_ERR_SHAPE;
        return launch_cl<TOK, GROUPED, GROUPED ? 8 : 16, 1, kSwigluVariant>(maps, P, st);
    }
    if constexpr (GROUPED) {
        // asymmetric activations with group steps: a kernel variant of its own, one CTA per cluster
        if (P.zp.tok_zero) {
            if (cluster != 1) return W4A8_ERR_SHAPE;
            if (dw == 4) return launch_cl<TOK, true, 4, 1, kAsymGroupVariant>(maps, P, st);
            if (dw == 8) return launch_cl<TOK, true, 8, 1, kAsymGroupVariant>(maps, P, st);
            return W4A8_ERR_SHAPE;
        }
    }
    if (dw == 4) return launch_dw<TOK, GROUPED, 4>(maps, P, cluster, st);
    if (dw == 8) return launch_dw<TOK, GROUPED, 8>(maps, P, cluster, st);
    if (dw == 12 && !GROUPED) return launch_dw<TOK, false, 12>(maps, P, cluster, st);
    if (dw == 16 && !GROUPED) return launch_dw<TOK, false, 16>(maps, P, cluster, st);
    return W4A8_ERR_SHAPE;
}

}  // namespace

bool make_plan(int M, const BlobLayout &L, const w4a8_opts *opts, LinearPlan *plan, bool auto_pair)
{
    const bool grouped = L.group != 0;
    const int cap = grouped ? 128 : 256;
    int tok = opts ? opts->tok_tile : 0;
    int split = opts ? opts->split_k : 0;
    if (tok == 0 || split == 0) {
        // Pick the token tile and the K split by a small cost model, in units of one k-block of
        // one CTA (about 800 cycles whatever the token tile: the decode of the 128 x 128 weight
        // tile dominates it).  Units are dealt round-robin to one persistent CTA per SM, so the
        // job takes ceil(units / SMs) rounds of (k-blocks per unit + a fixed cost per unit for
        // pipeline fill and epilogue); a split adds the partial tile's round trip per unit and,
        // once at the end, the last slice's reduction (its loads go sixteen at a time).
        const int sms = device_sms();
        int tok_max = 16;
        while (tok_max < M && tok_max < cap) tok_max *= 2;
        double best = 0.0;
        int best_tok = 0, best_split = 0;
        const int t_first = tok ? tok : tok_max, t_last = tok ? tok : 16;
        for (int t = t_first; t >= t_last; t /= 2) {
            const long long tiles_t = (long long)((M + t - 1) / t) * L.n_tiles;
            const int tokens = M < t ? M : t;
            const int max_split = L.k_blocks / 2 > 16 ? 16 : (L.k_blocks / 2 > 0 ? L.k_blocks / 2 : 1);
            for (int sp = 1; sp <= max_split; ++sp) {
                if (split && sp != split) continue;
                const int per = (L.k_blocks + sp - 1) / sp;
                const int slices = (L.k_blocks + per - 1) / per;
                if (slices != sp) continue;                  // the same plan as a smaller split
                const long long units = tiles_t * slices;
                const double rounds = (double)((units + sms - 1) / sms);
                // a k-block costs a little more with a wide token tile (the MMAs), a unit costs
                // its epilogue (by tile width) plus pipeline fill, a split unit its partial
                // tile's round trip; constants fitted to measured mid-size shapes
                const double kb_cost = 1.0 + 0.1 * t / 256.0;
                double cost = rounds * (per * kb_cost + 2.0 + t / 64.0 + (slices > 1 ? 6.0 : 0.0));
                if (slices > 1) cost += 1.5 * tokens * slices / 16.0;
                if (best_tok == 0 || cost < best * 0.999) {
                    best = cost;
                    best_tok = t;
                    best_split = slices;
                }
            }
        }
        if (tok == 0) tok = best_tok ? best_tok : tok_max;
        if (split == 0) split = best_split ? best_split : 1;
    }
    if (tok != 16 && tok != 32 && tok != 64 && tok != 128 && tok != 192 && tok != 256) return false;
    if (tok > cap) return false;
    const int tok_tiles = (M + tok - 1) / tok;
    // Cluster forms.  The sharing pair (2) halves the table lookups per CTA, but the hand-over
    // between the two CTAs lengthens the per-k-block chain by more than that gains: on request only.
    // The MMA pair (3) halves the token bytes per SM and, with two k-blocks per barrier round, the
    // issuing thread's fixed cost per MMA; together with the offset form of the decode tables
    // it is the most energy-efficient form, and a long job runs at the power cap, where that
    // decides (OPT-66B block at 2048 tokens, sustained: 2430 against 2360 TOPS).  The automatic
    // plan takes it for 1024 tokens and more on layers of at least 8192 x 8192: the token sums of
    // the offset tables cost a launch whose time goes with M x K while the layer's goes with
    // M x N x K, and with few k-blocks per unit the pair's longer rounds do not pay (4096 -> 4096
    // at 2048 tokens: 39.6 against 31.5 us, 16384 -> 4096: 112 against 103 us).
    int cluster = opts ? opts->cluster : 0;
    const int off = 13 << L.shift;
    const bool offset_fits = !grouped && L.bits == 4 && L.shift <= 2 &&
                             (long long)L.K * 127 * (2 * off) < (1LL << 31);
    bool auto_offset = false;
    if (cluster == 0) {
        cluster = 1;
        if (auto_pair && M >= 1024 && L.N >= 8192 && L.K >= 8192 && tok == 256 && split == 1 &&
            offset_fits && L.n_tiles % 2 == 0 &&
            L.k_blocks % 2 == 0 && (!opts || (opts->decode_warps == 0 && opts->offset_tables == 0))) {
            // (very long K: two row tiles per CTA instead - no traffic between CTAs, and the
            // epilogue that this form cannot overlap is small against 256 and more k-blocks;
            // 36864 -> 9216 at 2048 tokens, sustained: 2660 against 2460 TOPS)
            // (k-block counts that are multiples of three: the pair with three k-blocks per
            // round, twelve MMA instructions per wait and commit; OPT-66B block, the three
            // 9216-deep layers, sustained: 2560 / 2305 / 2600 against 2455 / 2235 / 2510 TOPS)
            cluster = L.k_blocks >= 256 ? 4 : L.k_blocks % 3 == 0 ? 5 : 3;
            auto_offset = true;
        }
    }
    // (3: the MMA pair - 256-token tiles, per-channel 4-bit weights, an even number of row tiles)
    // (4: two row tiles per CTA - the same conditions, sixteen decode warps)
    const bool pair = cluster == 3 || cluster == 4 || cluster == 5;
    if (pair && !(tok == 256 && !grouped && L.bits == 4 && L.n_tiles % 2 == 0)) return false;
    if (cluster != 1 && !pair && !(cluster == 2 && tok >= 128)) return false;
    const int share = cluster == 2 ? 2 : 1;
    const int tok_groups = (tok_tiles + share - 1) / share;
    // one counter per (token tile, row tile), empty partner tiles included
    const long long tiles = (long long)tok_groups * share * L.n_tiles;
    if (split < 1 || split > L.k_blocks) return false;
    const int kb_per = (L.k_blocks + split - 1) / split;
    split = (L.k_blocks + kb_per - 1) / kb_per;              // no empty slice
    if (tiles * split > 0x7fffffffLL) return false;
    // the MMA pair takes k-blocks two at a time: every K slice has an even number of them
    if (cluster == 3 && (kb_per % 2 != 0 || L.k_blocks % 2 != 0)) return false;
    if (cluster == 5 && (kb_per % 3 != 0 || L.k_blocks % 3 != 0)) return false;
    int dw = opts ? opts->decode_warps : 0;
    if (dw == 0) dw = (grouped || L.bits == 3) ? 8 : 16;
    if (L.bits == 3 && (dw != 8 || cluster != 1)) return false;
    if ((cluster == 4 || cluster == 5) && dw != 16) return false;
    if (dw != 4 && dw != 8 && !((dw == 12 || dw == 16) && !grouped)) return false;
    plan->decode_warps = dw;
    plan->cluster = cluster;
    plan->batched = 0;
    plan->tok_run = opts ? opts->tok_run : 0;
    plan->swiglu = 0;
    plan->debug_wait_ms = opts ? opts->debug_wait_ms : 0;
    plan->debug_skip_load = opts ? opts->debug_skip_load : 0;
    plan->tok_tile = tok;
    plan->tok_tiles = tok_tiles;
    plan->split_k = split;
    plan->kb_per_split = kb_per;
    plan->off_counters = sizeof(StatusBlock);
    plan->off_partials = align_up(plan->off_counters + (size_t)tiles * sizeof(int), 256);
    const size_t m_pad = (size_t)tok_tiles * tok;
    plan->off_toksum = align_up(plan->off_partials + (split > 1 ? (size_t)split * m_pad * L.n_pad * 4 : 0), 256);
    // Offset form of the decode tables (decode.cuh): per-channel 4-bit weights whose special
    // value is step/2 or step/4, and a K short enough for the offset sums to stay inside INT32.
    // It needs offset * (sum of each token), computed by a small kernel in front into the
    // workspace (one INT32 per token and row tile in the P*V form, so the slot is sized for the
    // padded rows).  Seven instead of eleven logic-pipe instructions per eight codes: the time per
    // k-block does not follow the logic pipe, but the energy does, so the form pays where the
    // power cap sets the clock (long prefill jobs) and costs its extra launch elsewhere.  On
    // request, and with the automatic MMA pair.
    const bool want = auto_offset || (opts && opts->offset_tables == 1);
    if (want && !offset_fits) return false;
    plan->offset = want ? off : 0;
    plan->toksum_slots = (size_t)L.n_tiles * M;
    plan->workspace_bytes = plan->off_toksum + (plan->offset ? plan->toksum_slots * 4 : 0);
    return true;
}

w4a8_status launch_linear_tcgen05(const int8_t *Xq, const float *tok_scale, const uint8_t *blob,
                                  const BlobLayout &L, const float *bias, int M,
                                  __nv_bfloat16 *Y, int32_t *acc, uint8_t *workspace,
                                  const LinearPlan &plan, cudaStream_t st, ZeroPoint zp)
{
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return W4A8_ERR_CUDA;
    Maps maps;
    memset(&maps, 0, sizeof(maps));
    // (P*V form: the token blocks of all row tiles are stacked, one after the other; an MMA
    // pair: each CTA loads half of the token tile)
    if (!encode_2d(enc, &maps.tok, CU_TENSOR_MAP_DATA_TYPE_UINT8, Xq, (cuuint64_t)L.K,
                   (cuuint64_t)M * (plan.batched ? L.n_tiles : 1), (cuuint64_t)L.K, (cuuint32_t)kTileK,
                   (cuuint32_t)((plan.cluster == 3 || plan.cluster == 5) ? plan.tok_tile / 2 : plan.tok_tile),
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B))
        return W4A8_ERR_CUDA;
    if (Y && plan.split_k == 1) {
        // output tiles of 128 features x 16 or 32 tokens; parts beyond N or M are clipped
        // (gated-unit epilogue: half as many features per tile and per row, binary16)
        const int width = plan.swiglu ? L.N / 2 : L.N, tile_w = plan.swiglu ? kTileN / 2 : kTileN;
        for (int rows = 16; rows <= 32; rows += 16) {
            if (!encode_2d(enc, rows == 16 ? &maps.y16 : &maps.y32,
                           plan.swiglu ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Y,
                           (cuuint64_t)width, (cuuint64_t)M, (cuuint64_t)width * 2, (cuuint32_t)tile_w,
                           (cuuint32_t)rows, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE))
                return W4A8_ERR_CUDA;
        }
    }

    Params P;
    P.blob = blob;
    P.codes = blob + L.off_codes;
    P.scales = reinterpret_cast<const float *>(blob + L.off_scales);
    P.zeros = blob + L.off_zeros;
    P.tok_scale = tok_scale;
    P.bias = bias;
    P.Y = Y;
    P.acc_out = acc;
    P.sb = reinterpret_cast<StatusBlock *>(workspace);
    P.counters = reinterpret_cast<int *>(workspace + plan.off_counters);
    P.partials = workspace + plan.off_partials;
    P.L = L;
    P.M = M;
    P.tok_tiles = plan.tok_tiles;
    P.m_pad = plan.tok_tiles * plan.tok_tile;
    P.split_k = plan.split_k;
    P.kb_per_split = plan.kb_per_split;
    // units: (token-tile group, row-tile group, K slice); a sharing pair groups two token tiles,
    // an MMA pair two row tiles
    P.total_units = plan.cluster == 2 ? (plan.tok_tiles + 1) / 2 * L.n_tiles * plan.split_k
                  : (plan.cluster == 3 || plan.cluster == 4 || plan.cluster == 5) ? plan.tok_tiles * (L.n_tiles / 2) * plan.split_k
                                      : plan.tok_tiles * L.n_tiles * plan.split_k;
    // Order of the units (unit_tiles): packed weights that stay in L2 are walked once per token
    // tile; larger ones are read by a run of token tiles at the same time, the run as long as its
    // tokens fit in a third of L2 (the codes of the row tiles in flight and the outputs take the rest).
    {
        const int share = plan.cluster == 2 ? 2 : 1;
        P.tok_groups = (plan.tok_tiles + share - 1) / share;
        const long long l2 = device_l2_bytes();
        const long long code_bytes = (long long)L.n_tiles * L.k_blocks * L.tile_bytes;
        const long long run_bytes = (long long)plan.tok_tile * share * L.K;      // tokens of one group
        long long run = code_bytes <= l2 / 3 ? 1 : (l2 / 3) / run_bytes;
        if (plan.tok_run > 0) run = plan.tok_run;
        if (plan.batched) run = 1;                      // every row tile has its own tokens
        // only the wide per-channel 4-bit instances of the kernel know longer runs
        if (L.group != 0 || plan.tok_tile < 128 || L.bits != 4 || plan.swiglu) run = 1;
        P.tok_run = (int)(run < 1 ? 1 : run > P.tok_groups ? P.tok_groups : run);
    }
    P.prefetch_codes = plan.tok_tiles == 1 ? 1 : 0;   // every code tile is read exactly once
    P.zp = zp;
    P.lt = make_level_tables(L.shift);
    P.unit = level_unit(L.shift);
    P.wait_ns = plan.debug_wait_ms > 0 ? (unsigned long long)plan.debug_wait_ms * 1000000ull : kWaitLimitNs;
    P.drain_ns = plan.debug_wait_ms > 0 ? P.wait_ns : kDrainLimitNs;
    P.skip_load = plan.debug_skip_load;
    P.batch_rows = plan.batched ? M : 0;
    P.swiglu = plan.swiglu;
    P.offset = plan.offset;
    P.tok_offsum = reinterpret_cast<const int32_t *>(workspace + plan.off_toksum);
    if (plan.offset) {
        const int rows = plan.batched ? M * L.n_tiles : M;
        if (launch_overlapped(token_offsum_kernel, dim3(rows), dim3(256), 0, st, Xq, L.K, plan.offset,
                              reinterpret_cast<int32_t *>(workspace + plan.off_toksum)) != cudaSuccess)
            return W4A8_ERR_CUDA;
    }

    const bool g = L.group != 0;
    switch (plan.tok_tile) {
    case 16: return g ? launch_one<16, true>(maps, P, plan.decode_warps, plan.cluster, st) : launch_one<16, false>(maps, P, plan.decode_warps, plan.cluster, st);
    case 32: return g ? launch_one<32, true>(maps, P, plan.decode_warps, plan.cluster, st) : launch_one<32, false>(maps, P, plan.decode_warps, plan.cluster, st);
    case 64: return g ? launch_one<64, true>(maps, P, plan.decode_warps, plan.cluster, st) : launch_one<64, false>(maps, P, plan.decode_warps, plan.cluster, st);
    case 128: return g ? launch_one<128, true>(maps, P, plan.decode_warps, plan.cluster, st) : launch_one<128, false>(maps, P, plan.decode_warps, plan.cluster, st);
    case 192: return g ? W4A8_ERR_SHAPE : launch_one<192, false>(maps, P, plan.decode_warps, plan.cluster, st);
    case 256: return g ? W4A8_ERR_SHAPE : launch_one<256, false>(maps, P, plan.decode_warps, plan.cluster, st);
    }
    return W4A8_ERR_SHAPE;
}

}  // namespace w4a8
