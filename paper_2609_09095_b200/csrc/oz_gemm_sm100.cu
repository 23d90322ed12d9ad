// Residue GEMMs on the 5th-generation tensor cores (Algorithm 1, the loop over moduli; Sec. 2
// "FP8 variant"; Eq. 8), with the per-modulus combination and `mod m_i` fused into the epilogue.
//
// For every modulus the product of two centred residues is rebuilt from exact plane products:
//   square m = s^2 (planes d0,d1):        d e = d0 e0 + s (d1 e0 + d0 e1)              (mod m)
//   non-square (planes d0,d1,dS=d0+d1):   d e = -15 d0 e0 + 16 dS eS + 240 d1 e1       (Eq. 8)
// so one (modulus, output tile) work item is a short list of "accumulator jobs", each a K-loop
// of tcgen05.mma instructions into one TMEM accumulator:
//   square:      job 0 = D0.E0 (weight 1);  job 1 = [D1|D0].[E0|E1] (two K-loops, weight s)
//   non-square:  job 0 = D0.E0 (-15);  job 1 = DS.ES (16);  job 2 = D1.E1 (240)
//   non-square, merged accumulators (FP8): job 0 = [D0|-16 D1].[E0|E1] (-15); job 1 = DS.ES (16)
//                -- the regrouping discussed under Table "tuples" (N_acc = 2); one TMEM drain
//                fewer per modulus, and the drains are what the epilogue pays for at small k
// Three MMA K-loops per modulus either way (p_mma = 3r).
//
// Split-K inside the kernel: a job whose K range exceeds the exact depth of its accumulator (4097
// or 15420 for the merged job 0, 32768 for every other FP32 accumulator, 2^31 / term size in
// INT32) is cut into segments of whole K chunks; each segment has an accumulator of its own that
// is reduced modulo m_i before it is weighted and added, so the residues are those of the whole K.
//
// The tile is computed transposed: the MMA's M dimension (128 TMEM lanes) runs over 128 columns
// j of C (planes of B), its N dimension (256 TMEM columns) over 256 rows i of C (planes of A).
// An epilogue thread therefore owns one column j and a run of 64 consecutive rows, which is
// contiguous in the column-major residue array; a warp transposes its 32 x 64 block through a
// small swizzled shared-memory buffer so that each store instruction writes whole lines.
//
// Kernel structure (one persistent CTA per SM, 576 threads, up to 112 registers each; launched as
// clusters of two CTAs that share one tcgen05.mma.cta_group::2 unless n pads badly to 256):
//   warp 0       TMA producer: 128-byte-swizzled K-major tiles of B (128 lines) and A (256 lines,
//                or this CTA's half of them in a pair) into a shared-memory ring of 192 KiB
//                (4 stages of 48 KiB, or 6 of 32 KiB in a pair), no multicast
//   warp 1       MMA issuer: one lane issues tcgen05.mma (M=128 or 256 across the pair, N=256,
//                K=32); accumulators live in TMEM, two slots of 256 columns used alternately per job
//   warps 2..17  epilogue (4 per TMEM lane quarter, 64 columns each): tcgen05.ld the finished slot,
//                reduce each accumulator modulo m_i in FP32 (all values are integers below 2^24,
//                every step exact), fold it with the job's weight into a per-thread running
//                combination held in registers, release the slot; after the last job reduce once
//                more and store the residues (uint16, or uint8 for the all-byte set)
// so the epilogue of one job overlaps the K-loop of the next, and TMEM never needs the three
// accumulators of a non-square modulus at once.
//
// Exactness: the FP8 route relies on integer-valued partial sums below 2^24 being accumulated
// without rounding (accumulation invariant of Algorithm 2, Lemma 1) and its epilogue works in
// exact FP32; the INT8 routes accumulate in INT32 and their epilogue is integer arithmetic
// (weights by IMAD, `mod m` by a multiply-high division on a biased, non-negative value).
//
// Native INT8 route (all-byte set A only): the centred residue itself is the operand, so a modulus
// is ONE job -- one plane, one K-loop, weight 1 -- and the schedule has r = 15 products; its
// accumulator is loaded straight into the combination registers and the slot released at once.
//
// Every barrier wait is bounded: on expiry the CTA records OZ_ERR_TIMEOUT in the device status
// word, every role leaves its loops, in-flight copies are given a bounded time to land, TMEM is
// freed and the kernel returns.
#include <cuda.h>
#include <atomic>
#include <cstdlib>

#include "oz_internal.h"
#include "oz_convert.cuh"

namespace oz {
namespace {

constexpr int BLOCK_M = 128;                       // MMA M: columns j of C (lines of B)
constexpr int BLOCK_N = 256;                       // MMA N: rows i of C (lines of A)
constexpr int BLOCK_K = 128;                       // bytes = elements (8-bit operands)
constexpr int UMMA_K = 32;                         // 8-bit operands: 32 elements per instruction
constexpr int A_BYTES = BLOCK_M * BLOCK_K;         // 16 KiB: MMA operand a = 128 lines of B's planes per CTA

// CG = 1: one CTA per tile of 128 columns x 256 rows of C.
// CG = 2: a pair of CTAs (cluster of 2) shares one tcgen05.mma.cta_group::2 of M = 256: the tile is
//         256 columns x 256 rows; each CTA loads its own 128 lines of B's planes (operand a) and HALF
//         of the 256 lines of A's planes (operand b), the tensor core reads both halves, and each
//         CTA's TMEM holds the accumulators of its own 128 columns.  Per CTA this halves the
//         shared-memory traffic of operand b and the TMA bytes per MMA.
template <int CG>
struct Tile {
    static constexpr int B_LINES = BLOCK_N / CG;                 // lines of A's planes loaded per CTA
    static constexpr int B_BYTES = B_LINES * BLOCK_K;            // 32 KiB / 16 KiB
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;        // 48 KiB / 32 KiB
    static constexpr int STAGES = CG == 1 ? 4 : 6;               // 192 KiB ring either way
    static constexpr int TILE_J = BLOCK_M * CG;                  // columns of C per work item
};
constexpr int TMEM_COLS = 512;                     // two accumulator slots of BLOCK_N columns
constexpr int NUM_THREADS = 576;                   // 18 warps: 112 registers each fit the register file
constexpr int FIRST_EPI_WARP = 2;                  // warp 0: producer, warp 1: MMA issuer
constexpr int EPI_WARPS = 16;
constexpr int COLS_PER_WARP = BLOCK_N / 4;         // four warps share a TMEM lane quarter
#ifndef OZ_DRAIN_W
#define OZ_DRAIN_W 16
#endif
constexpr int DRAIN_W = OZ_DRAIN_W;                // accumulator columns per tcgen05.ld of a drain: 64 running
                                                   // values + 16 loaded ones stay inside the 96 registers
constexpr int XPOSE_BYTES = 16 * 128;                // per epilogue warp: 16 lines x 128 bytes
constexpr size_t SMEM_BYTES = 4 * 49152 + EPI_WARPS * XPOSE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
static_assert(Tile<1>::STAGES * Tile<1>::STAGE_BYTES == 4 * 49152 && Tile<2>::STAGES * Tile<2>::STAGE_BYTES == 4 * 49152, "ring size");

struct ModInfo {
    float m, inv_m;
    float w[3];           // weight of each job
    int reduce[3];        // reduce the accumulator modulo m before weighting (0: the exact FP32 range allows skipping it)
    int njobs;            // 2 (square), 3, 1 (native INT8 residues) or 2 (non-square, merged accumulators)
    int kind;             // 0 square, 1 non-square separate, 2 native, 3 non-square merged
    int planeA0, planeB0; // first stored plane of this modulus in A's and in B's plane arrays
    // Split-K inside the kernel: the K range of a job is cut into segments of whole chunks, each with
    // an accumulator of its own that is reduced before the next is added, so that every accumulator
    // stays exact.  nseg / seg_len: job 0 of the merged schedule (depth 4097 or 15420);
    // nseg_all / seg_len_all: every other job (depth 32768 in FP32; 2^31 / term size in INT32).
    int nseg, seg_len;
    int nseg_all, seg_len_all;
    // integer epilogue of the INT8 routes (INT32 accumulators):
    int iw[3];            // weights as integers
    uint32_t mi;          // the modulus
    uint32_t magic;       // floor(2^32 / m)
    uint32_t bias;        // a multiple of m just above 2^31: makes a signed combination non-negative
    // native INT8 residues, one accumulator of at most 2^30 in magnitude (k <= 65536): exact division
    uint32_t magic39;     // ceil(2^39 / m): floor(u / m) = (u * magic39) >> 39 exactly for u < 2^31 + 256, m in (128, 256]
    uint32_t bias30;      // the multiple of m just above 2^30
};

struct GemmParams {
    int64_t m, n, k;
    int tiles_m, tiles_n, nk;       // tiles of 256 rows / 128 columns of C; nk = K chunks of BLOCK_K
    int vec_store;                  // R rows 16-byte aligned: use vector stores
    int stall_producer;             // test hook: the producer issues no copy, so every wait runs out
    int r;
    int64_t total_items;
    void *R;                        // residues: uint16 (RB = 2) or uint8 (RB = 1, byte moduli)
    int64_t ldr, mod_stride;
    unsigned int *rowmax, *colmax;  // bound product only: one word per row / column, word stride 2
    unsigned int *status;
    ModInfo mod[kMaxR];
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

// cluster-scope acquire: the barriers of the CTA-pair variant are also signalled by the peer CTA
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}

// Arrivals that hand a drained accumulator back to the MMA issuer.  The TMEM reads they follow have
// already completed (tcgen05.wait::ld) and no memory written by this thread is read by the waiter,
// so the arrive carries no release: a release would first wait for the residue stores in flight.
__device__ __forceinline__ void mbar_arrive_relaxed(uint32_t bar)
{
    asm volatile("mbarrier.arrive.relaxed.cta.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_cluster_relaxed(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

// all threads of both CTAs of the pair (no time limit: every thread reaches it on every path)
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s per wait

// Bounded wait.  Returns false when the wait ran out or another role already gave up.
// The timer is read only after a long run of failed polls: the common path never touches it.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          unsigned int *status)
{
#pragma unroll 1
    for (int it = 0; it < 4096; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    unsigned long long start = global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int it = 0; it < 256; ++it)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - start > kWaitLimitNs) {
            *abort_flag = 1;
            atomicOr(status, 1u << OZ_ERR_TIMEOUT);
            return false;
        }
    }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                            int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// CTA-pair copy: same as tma_load_3d, but the mbarrier may live in the peer CTA (cluster address)
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar_cluster,
                                                 int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// In the CTA-pair variant the same warp of BOTH CTAs executes the allocation / release.
template <int CG>
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols)
{
    if (CG == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
}

template <int CG>
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    if (CG == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
    else
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

template <int SUB, int CG>
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc,
                                     uint32_t accumulate)
{
#define OZ_UMMA(GROUP, KIND)                                                                      \
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"                              \
                 "tcgen05.mma.cta_group::" GROUP ".kind::" KIND " [%0], %1, %2, %3, p;\n\t}"      \
                 ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory")
    if (SUB == 0 && CG == 1) OZ_UMMA("1", "f8f6f4");
    if (SUB == 0 && CG == 2) OZ_UMMA("2", "f8f6f4");
    if (SUB == 1 && CG == 1) OZ_UMMA("1", "i8");
    if (SUB == 1 && CG == 2) OZ_UMMA("2", "i8");
#undef OZ_UMMA
}

// mbarrier arrives once every MMA issued so far by this thread has completed
// (CTA pair: the arrive is delivered to the barrier at this offset in BOTH CTAs)
template <int CG>
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    if (CG == 1) {
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    } else {
        const uint16_t both = 3;
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(bar), "h"(both) : "memory");
    }
}

template <int N>
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[N])
{
    static_assert(N == 32, "32 columns");
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]),
          "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
          "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 16 columns of the warp's 32 lanes, with the wait
template <int N>
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[N])
{
    static_assert(N == 16, "16 columns");
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// same load without the wait, into v[OFF .. OFF+31]
template <int OFF>
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&v)[64])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[OFF + 0]), "=r"(v[OFF + 1]), "=r"(v[OFF + 2]), "=r"(v[OFF + 3]), "=r"(v[OFF + 4]),
          "=r"(v[OFF + 5]), "=r"(v[OFF + 6]), "=r"(v[OFF + 7]), "=r"(v[OFF + 8]), "=r"(v[OFF + 9]),
          "=r"(v[OFF + 10]), "=r"(v[OFF + 11]), "=r"(v[OFF + 12]), "=r"(v[OFF + 13]), "=r"(v[OFF + 14]),
          "=r"(v[OFF + 15]), "=r"(v[OFF + 16]), "=r"(v[OFF + 17]), "=r"(v[OFF + 18]), "=r"(v[OFF + 19]),
          "=r"(v[OFF + 20]), "=r"(v[OFF + 21]), "=r"(v[OFF + 22]), "=r"(v[OFF + 23]), "=r"(v[OFF + 24]),
          "=r"(v[OFF + 25]), "=r"(v[OFF + 26]), "=r"(v[OFF + 27]), "=r"(v[OFF + 28]), "=r"(v[OFF + 29]),
          "=r"(v[OFF + 30]), "=r"(v[OFF + 31])
        : "r"(taddr)
        : "memory");
}

// shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 B apart
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr >> 4) & 0x3FFFu);   // start address / 16
    d |= static_cast<uint64_t>(1) << 16;                 // leading byte offset (unused here) / 16
    d |= static_cast<uint64_t>(1024 >> 4) << 32;         // stride byte offset / 16
    d |= static_cast<uint64_t>(1) << 46;                 // descriptor version of sm_100
    d |= static_cast<uint64_t>(2) << 61;                 // 128-byte swizzle
    return d;
}

// instruction descriptor: D format, A/B formats, K-major both, N/8 at bit 17, M/16 at bit 24
template <int SUB, int CG>
__host__ __device__ constexpr uint32_t instr_desc()
{
    uint32_t cfmt = SUB == 0 ? 1u /*f32*/ : 2u /*s32*/;
    uint32_t abfmt = SUB == 0 ? 0u /*e4m3*/ : 1u /*s8*/;
    return (cfmt << 4) | (abfmt << 7) | (abfmt << 10) | (static_cast<uint32_t>(BLOCK_N >> 3) << 17) |
           (static_cast<uint32_t>((BLOCK_M * CG) >> 4) << 24);
}

// work item -> (modulus, tile_m, tile_n): modulus-major so that one modulus' planes stay in L2;
// inside a modulus, bands of 16 tile rows are swept column by column.
struct Item { int mod, tm, tn; };

__device__ __forceinline__ Item decode_item(int64_t item64, const GemmParams &p)
{
    // the host refuses launches with 2^31 or more items: 32-bit divisions are enough
    constexpr uint32_t BAND = 16;
    const uint32_t item = static_cast<uint32_t>(item64);
    const uint32_t tiles_m = static_cast<uint32_t>(p.tiles_m), tiles_n = static_cast<uint32_t>(p.tiles_n);
    const uint32_t per_mod = tiles_m * tiles_n;
    Item it;
    const uint32_t mod = item / per_mod;
    const uint32_t t = item - mod * per_mod;
    const uint32_t band_size = BAND * tiles_n;
    const uint32_t band = t / band_size;
    const uint32_t in_band = t - band * band_size;
    const uint32_t rows = tiles_m - band * BAND < BAND ? tiles_m - band * BAND : BAND;
    const uint32_t tn = in_band / rows;
    it.mod = static_cast<int>(mod);
    it.tn = static_cast<int>(tn);
    it.tm = static_cast<int>(band * BAND + (in_band - tn * rows));
    return it;
}

// plane pair (A plane, B plane) of K-loop `pair` of job `job`
__device__ __forceinline__ void job_planes(const ModInfo &mi, int job, int pair, int *pa, int *pb)
{
    int oa, ob;
    if (mi.kind == 1) {
        // non-square, stored order d0, d1, dS; jobs d0 e0, dS eS, d1 e1
        oa = ob = job == 0 ? 0 : (job == 1 ? 2 : 1);
    } else if (mi.kind == 3) {
        // non-square merged (A stores d0, -16 d1, dS): job 0 = [d0 | -16 d1] . [e0 | e1] (two K-loops),
        // job 1 = dS eS
        oa = ob = job == 0 ? pair : 2;
    } else if (mi.kind == 0 && job == 1) {
        // square: job 1 = [d1 | d0] . [e0 | e1]
        oa = pair == 0 ? 1 : 0;
        ob = pair == 0 ? 0 : 1;
    } else {
        oa = ob = 0;            // square job 0, native
    }
    *pa = mi.planeA0 + oa;
    *pb = mi.planeB0 + ob;
}

__device__ __forceinline__ int job_pairs(const ModInfo &mi, int job)
{
    return ((mi.kind == 0 && job == 1) || (mi.kind == 3 && job == 0)) ? 2 : 1;
}

// accumulators (K segments) of job `job`
__device__ __forceinline__ int job_segments(const ModInfo &mi, int job)
{
    return (mi.kind == 3 && job == 0) ? mi.nseg : mi.nseg_all;
}

// chunk range [kc0, kc1) of segment `seg`
__device__ __forceinline__ void segment_range(const ModInfo &mi, int job, int seg, int nk, int *kc0, int *kc1)
{
    const int len = (mi.kind == 3 && job == 0) ? mi.seg_len : mi.seg_len_all;
    *kc0 = seg * len;
    *kc1 = min(nk, *kc0 + len);
}

// acc - m * rint(acc / m) for a pair of integer-valued floats below 2^24 (exact): rint through the
// 1.5 * 2^23 constant, then one fused multiply-add
__device__ __forceinline__ float2 mod_balanced2(float2 acc, float2 inv_m2, float2 neg_m2)
{
    const float2 big = make_float2(12582912.0f, 12582912.0f), neg_big = make_float2(-12582912.0f, -12582912.0f);
    const float2 quot = __fadd2_rn(__ffma2_rn(acc, inv_m2, big), neg_big);
    return __ffma2_rn(quot, neg_m2, acc);
}

// RB: bytes of one stored residue (2: uint16, 1: uint8 for the all-byte modulus set)
// DIRECT: native INT8 residues -- one accumulator per modulus, loaded straight into the registers
//         that otherwise hold the running combination of several accumulators
// LOOSE: the stored residue is some representative in [0, 2 m_i) instead of the canonical one in
//         [0, m_i) (two-byte residues only).  The reconstruction is indifferent to it -- the CRT
//         weight of m_i is a multiple of M -- and the epilogue saves the canonicalisation; used for
//         the residues that stay inside the whole-method calls.
// TILED: the residue array is the private, tile-ordered one of the whole-method calls (see
//         residue_tiling() below): the 32 columns x 64 rows that an epilogue warp owns form one
//         contiguous block, [16-byte chunk][lane], so that every store instruction of a warp writes
//         512 consecutive bytes straight from registers -- no transposition through shared memory,
//         which the tensor pipe and the TMA writes need for themselves.  The reconstruction reads
//         the same order.  Without it the public layout R[mod][j][ldr] is written.
// BOUND: not a residue product but the magnitude-bound product of the accurate mode (Sec. 2 "The FP8
//         variant", the "+1" pass): one plane per operand, one accumulator per tile, and instead of
//         residues the epilogue reduces the row and column maxima of the tile into p.rowmax / p.colmax.
template <int SUB, int CG, int RB, bool DIRECT, bool LOOSE, bool TILED, bool BOUND = false>
__global__ void __launch_bounds__(NUM_THREADS, 1)
residue_gemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                    const __grid_constant__ GemmParams p)
{
    constexpr int STAGES = Tile<CG>::STAGES;
    constexpr int STAGE_BYTES = Tile<CG>::STAGE_BYTES;
    // CTA pair: rank 0 leads (issues the MMAs, owns the `full` and `tmem-empty` barriers that both
    // CTAs signal); work items are dealt to pairs, so both CTAs walk the same item sequence.
    const uint32_t rank = CG == 2 ? cluster_ctarank() : 0u;
    const int64_t first_item = CG == 2 ? (blockIdx.x >> 1) : blockIdx.x;
    const int64_t item_step = CG == 2 ? (gridDim.x >> 1) : gridDim.x;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;                     // 1024-byte aligned ring
    const uint32_t bars = tiles + STAGES * STAGE_BYTES + EPI_WARPS * XPOSE_BYTES;
    const uint32_t full_bar = bars;                                   // STAGES x 8 bytes
    const uint32_t empty_bar = bars + 8 * STAGES;
    const uint32_t tfull_bar = bars + 16 * STAGES;                    // 2 x 8
    const uint32_t tempty_bar = tfull_bar + 16;                       // 2 x 8
    const uint32_t tmem_slot = tempty_bar + 16;                       // 4 bytes: TMEM base address
    unsigned char *xpose_base = smem_raw + (tiles - raw) + STAGES * STAGE_BYTES;
    unsigned char *gen = xpose_base + EPI_WARPS * XPOSE_BYTES;
    volatile uint32_t *tmem_base_ptr = reinterpret_cast<volatile uint32_t *>(gen + 16 * STAGES + 32);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gen + 16 * STAGES + 40);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(tfull_bar + 8 * s, 1);
            mbar_init(tempty_bar + 8 * s, EPI_WARPS * CG);   // pair: the peer's epilogue warps arrive too
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc<CG>(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();      // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_ptr;

    if (warp < FIRST_EPI_WARP) {
        if (warp == 0 && lane == 0) {
            // -------------------------------------------------------- TMA producer
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int64_t item = first_item; ok && !p.stall_producer && item < p.total_items; item += item_step) {
                Item it = decode_item(item, p);
                const ModInfo &mi = p.mod[it.mod];
                for (int job = 0; ok && job < mi.njobs; ++job)
                for (int seg = 0, nseg = job_segments(mi, job); ok && seg < nseg; ++seg) {
                    int npairs = job_pairs(mi, job), kc0, kc1;
                    segment_range(mi, job, seg, p.nk, &kc0, &kc1);
                    for (int pair = 0; ok && pair < npairs; ++pair) {
                        int pa, pb;
                        job_planes(mi, job, pair, &pa, &pb);
                        for (int kc = kc0; kc < kc1; ++kc) {
                            ok = mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.status);
                            if (!ok) break;
                            uint32_t fb = full_bar + 8 * stage;
                            uint32_t sa = tiles + stage * STAGE_BYTES;
                            if (CG == 1) {
                                mbar_expect_tx(fb, STAGE_BYTES);
                                tma_load_3d(sa, &mapB, fb, kc * BLOCK_K, it.tn * BLOCK_M, pb);
                                tma_load_3d(sa + A_BYTES, &mapA, fb, kc * BLOCK_K, it.tm * BLOCK_N, pa);
                            } else {
                                // both CTAs' copies complete on the leader's barrier
                                if (rank == 0) mbar_expect_tx(fb, 2 * STAGE_BYTES);
                                const uint32_t fb_leader = map_to_cta(fb, 0);
                                tma_load_3d_pair(sa, &mapB, fb_leader, kc * BLOCK_K,
                                                 it.tn * Tile<CG>::TILE_J + static_cast<int>(rank) * BLOCK_M, pb);
                                tma_load_3d_pair(sa + A_BYTES, &mapA, fb_leader, kc * BLOCK_K,
                                                 it.tm * BLOCK_N + static_cast<int>(rank) * Tile<CG>::B_LINES, pa);
                            }
                            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                        }
                    }
                }
            }
            if (!ok) {
                // give copies already in flight a bounded time to land before the CTA exits
                unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 2000000ull) { }
            }
        } else if (warp == 1 && lane == 0 && rank == 0) {
            // -------------------------------------------------------- MMA issuer (pair: leader CTA only)
            constexpr uint32_t idesc = instr_desc<SUB, CG>();
            int stage = 0;
            uint32_t phase = 0;
            int slot = 0;
            uint32_t slot_phase = 0;   // bit s = phase of slot s
            bool ok = true;
            for (int64_t item = first_item; ok && item < p.total_items; item += item_step) {
                Item it = decode_item(item, p);
                const ModInfo &mi = p.mod[it.mod];
                for (int job = 0; ok && job < mi.njobs; ++job)
                for (int seg = 0, nseg = job_segments(mi, job); ok && seg < nseg; ++seg) {
                    ok = mbar_wait(tempty_bar + 8 * slot, ((slot_phase >> slot) & 1u) ^ 1u, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(slot * BLOCK_N);
                    uint32_t accumulate = 0;
                    int kc0, kc1;
                    segment_range(mi, job, seg, p.nk, &kc0, &kc1);
                    int steps = job_pairs(mi, job) * (kc1 - kc0);
                    for (int st = 0; st < steps; ++st) {
                        ok = mbar_wait(full_bar + 8 * stage, phase, abort_flag, p.status);
                        if (!ok) break;
                        tc_fence_after();
                        uint32_t sa = tiles + stage * STAGE_BYTES;
                        uint64_t da = smem_desc(sa), db = smem_desc(sa + A_BYTES);
#pragma unroll
                        for (int ks = 0; ks < BLOCK_K / UMMA_K; ++ks) {
                            // advancing K inside the 128-byte swizzle atom: +32 bytes = +2 in the address field
                            umma<SUB, CG>(d_tmem, da + static_cast<uint64_t>(ks * (UMMA_K >> 4)),
                                      db + static_cast<uint64_t>(ks * (UMMA_K >> 4)), idesc, accumulate);
                            accumulate = 1;
                        }
                        umma_commit<CG>(empty_bar + 8 * stage);     // frees the stage when these MMAs finish
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    umma_commit<CG>(tfull_bar + 8 * slot);           // accumulator complete
                    slot_phase ^= 1u << slot;
                    slot ^= 1;
                }
            }
            if (!ok) {
                unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 2000000ull) { }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int q = warp & 3;                              // TMEM lane quarter this warp may read
        const int part = (warp - FIRST_EPI_WARP) >> 2;       // which 64 of the tile's 256 TMEM columns (any four
                                                             // consecutive warps cover the four lane quarters)
        int slot = 0;
        uint32_t slot_phase = 0;   // bit s = phase of slot s
        bool ok = true;
        for (int64_t item = first_item; ok && item < p.total_items; item += item_step) {
            Item it = decode_item(item, p);
            const ModInfo &mi = p.mod[it.mod];
            const float mm = mi.m, inv_m = mi.inv_m;
            const float loose_offset = mm + 8388608.0f;          // exact: m < 2^11
            const float2 inv_m2 = make_float2(inv_m, inv_m), neg_m2 = make_float2(-mm, -mm);
            const uint32_t im = mi.mi, imagic = mi.magic, ibias = mi.bias;
            // running combination per element: FP32 (FP8 route) or INT32 (INT8 routes), as raw bits
            uint32_t comb[COLS_PER_WARP];
            if constexpr (!DIRECT) {
#pragma unroll
                for (int c = 0; c < COLS_PER_WARP; ++c) comb[c] = 0u;
            }
            for (int job = 0; ok && job < mi.njobs; ++job)
            for (int seg = 0, nseg = job_segments(mi, job); ok && seg < nseg; ++seg) {
                // every lane polls for itself; the outcome is made warp-uniform before anything that
                // contains a warp barrier depends on it
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(tfull_bar + 8 * slot, (slot_phase >> slot) & 1u, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
                const float wj = mi.w[job];
                const bool reduce_first = mi.reduce[job] != 0;
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                       static_cast<uint32_t>(slot * BLOCK_N + part * COLS_PER_WARP);
                if constexpr (DIRECT) {
                    // the only accumulator of this modulus lands in the combination registers as it is
                    tmem_ld32_issue<0>(taddr, comb);
                    tmem_ld32_issue<32>(taddr + 32, comb);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                } else
#pragma unroll
                for (int c0 = 0; c0 < COLS_PER_WARP; c0 += DRAIN_W) {
                    uint32_t v[DRAIN_W];
                    if constexpr (DRAIN_W == 32) tmem_ld32(taddr + c0, v);
                    else tmem_ld16(taddr + c0, v);
                    if constexpr (SUB == 0) {
                        // two values per instruction (packed FP32 pairs): half the issue slots
                        const float2 wj2 = make_float2(wj, wj);
                        if (reduce_first) {
#pragma unroll
                            for (int e = 0; e < DRAIN_W; e += 2) {
                                const float2 acc = make_float2(__uint_as_float(v[e]), __uint_as_float(v[e + 1]));
                                const float2 res = mod_balanced2(acc, inv_m2, neg_m2);       // exact, |res| <= ~m/2
                                const float2 cur = make_float2(__uint_as_float(comb[c0 + e]), __uint_as_float(comb[c0 + e + 1]));
                                const float2 nxt = __ffma2_rn(res, wj2, cur);
                                comb[c0 + e] = __float_as_uint(nxt.x);
                                comb[c0 + e + 1] = __float_as_uint(nxt.y);
                            }
                        } else {
                            // the host has checked that w * acc stays below 2^24 for this k
#pragma unroll
                            for (int e = 0; e < DRAIN_W; e += 2) {
                                const float2 acc = make_float2(__uint_as_float(v[e]), __uint_as_float(v[e + 1]));
                                const float2 cur = make_float2(__uint_as_float(comb[c0 + e]), __uint_as_float(comb[c0 + e + 1]));
                                const float2 nxt = __ffma2_rn(acc, wj2, cur);
                                comb[c0 + e] = __float_as_uint(nxt.x);
                                comb[c0 + e + 1] = __float_as_uint(nxt.y);
                            }
                        }
                    } else {
                        // INT32 accumulators: exact integer arithmetic, no conversions
                        const int iwj = mi.iw[job];
                        if (reduce_first) {
#pragma unroll
                            for (int e = 0; e < DRAIN_W; ++e) {
                                uint32_t u = v[e] + ibias;                       // non-negative, same residue
                                uint32_t r = u - __umulhi(u, imagic) * im;       // in [0, 2m)
                                r = min(r, r - im);
                                comb[c0 + e] = static_cast<uint32_t>(static_cast<int>(r) * iwj + static_cast<int>(comb[c0 + e]));
                            }
                        } else {
                            // the host has checked that the weighted sum stays inside INT32 for this k
#pragma unroll
                            for (int e = 0; e < DRAIN_W; ++e)
                                comb[c0 + e] = static_cast<uint32_t>(static_cast<int>(v[e]) * iwj + static_cast<int>(comb[c0 + e]));
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (CG == 1) mbar_arrive_relaxed(tempty_bar + 8 * slot);
                    else mbar_arrive_cluster_relaxed(map_to_cta(tempty_bar + 8 * slot, 0));   // the leader's barrier
                }
                slot_phase ^= 1u << slot;
                slot ^= 1;
            }
            if (!ok) break;
            // this thread: column j of C, rows i0 .. i0+63 (contiguous in the residue array)
            const int64_t jw = static_cast<int64_t>(it.tn) * Tile<CG>::TILE_J + rank * BLOCK_M + q * 32;   // first column of the warp
            const int64_t j = jw + lane;
            const int64_t i0 = static_cast<int64_t>(it.tm) * BLOCK_N + part * COLS_PER_WARP;
            if (i0 >= p.m || jw >= p.n) continue;                                 // warp-uniform
            if constexpr (BOUND) {
                // The accumulators are non-negative integers held exactly in FP32: their bit patterns
                // order like their values, so the maxima are taken on the raw words.
                uint32_t colv = 0u, keep0 = 0u, keep1 = 0u;
#pragma unroll
                for (int c = 0; c < COLS_PER_WARP; ++c) {
                    colv = max(colv, comb[c]);
                    const uint32_t rowv = __reduce_max_sync(0xFFFFFFFFu, comb[c]);   // over the warp's 32 columns
                    if ((c & 31) == lane) { if (c < 32) keep0 = rowv; else keep1 = rowv; }
                }
                if (j < p.n && colv) atomicMax(p.colmax + 2 * j, colv);
                if (i0 + lane < p.m && keep0) atomicMax(p.rowmax + 2 * (i0 + lane), keep0);
                if (i0 + 32 + lane < p.m && keep1) atomicMax(p.rowmax + 2 * (i0 + 32 + lane), keep1);
            }
            if constexpr (!BOUND) {
            // last reduction of one combination value: the stored residue in the low bits of a word
            auto final_bits = [&](uint32_t cv) -> uint32_t {
                if constexpr (SUB == 0) {
                    float t = __uint_as_float(cv);
                    float quot = fmaf(t, inv_m, 12582912.0f) - 12582912.0f;
                    float res = fmaf(-quot, mm, t);                      // |res| <= ~m/2
                    if constexpr (LOOSE) {
                        return __float_as_uint(res + loose_offset);      // res + m in (0, 2m), low mantissa bits
                    } else {
                        res = res < 0.0f ? res + mm : res;               // canonical [0, m)
                        return __float_as_uint(res + 8388608.0f);        // integer in the low mantissa bits
                    }
                } else if constexpr (DIRECT) {
                    uint32_t u = cv + mi.bias30;                          // in (0, 2^31 + 256)
                    return u - (__umulhi(u, mi.magic39) >> 7) * im;      // exact quotient: canonical [0, m)
                } else {
                    uint32_t u = cv + ibias;
                    uint32_t r = u - __umulhi(u, imagic) * im;           // in [0, 2m)
                    return LOOSE ? r : min(r, r - im);                   // canonical [0, m) unless LOOSE
                }
            };
            // same for two values at once; the loose FP32 form is done with packed pairs
            auto final_bits2 = [&](uint32_t c0v, uint32_t c1v, uint32_t &b0, uint32_t &b1) {
                if constexpr (SUB == 0 && LOOSE) {
                    const float2 res = mod_balanced2(make_float2(__uint_as_float(c0v), __uint_as_float(c1v)), inv_m2, neg_m2);
                    const float2 out = __fadd2_rn(res, make_float2(loose_offset, loose_offset));
                    b0 = __float_as_uint(out.x);
                    b1 = __float_as_uint(out.y);
                } else {
                    b0 = final_bits(c0v);
                    b1 = final_bits(c1v);
                }
            };
            // four consecutive rows starting at combination value c -> one (RB = 1) or two (RB = 2) words
            auto pack4 = [&](int c, uint32_t &w0, uint32_t &w1) {
                uint32_t b0, b1, b2, b3;
                final_bits2(comb[c], comb[c + 1], b0, b1);
                final_bits2(comb[c + 2], comb[c + 3], b2, b3);
                if constexpr (RB == 2) {
                    w0 = __byte_perm(b0, b1, 0x5410);
                    w1 = __byte_perm(b2, b3, 0x5410);
                } else {
                    w0 = __byte_perm(__byte_perm(b0, b1, 0x0040), __byte_perm(b2, b3, 0x0040), 0x5410);
                    w1 = 0u;
                }
            };
            constexpr int NCH = COLS_PER_WARP * RB / 16;     // 16-byte chunks of a thread's run of rows
            if constexpr (TILED) {
                // block (tile, CTA rank, warp), then modulus: the r residue blocks of one 32 x 64 patch of
                // the output lie next to one another, which is how the reconstruction reads them
                unsigned char *blk = static_cast<unsigned char *>(p.R) +
                    (((((static_cast<int64_t>(it.tm) * p.tiles_n + it.tn) * CG + rank) * EPI_WARPS + (part * 4 + q)) * p.r +
                      it.mod) * static_cast<int64_t>(NCH * 512)) + lane * 16;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    uint4 val;
                    if constexpr (RB == 2) {
                        pack4(8 * c, val.x, val.y);
                        pack4(8 * c + 4, val.z, val.w);
                    } else {
                        uint32_t unused;
                        pack4(16 * c, val.x, unused);
                        pack4(16 * c + 4, val.y, unused);
                        pack4(16 * c + 8, val.z, unused);
                        pack4(16 * c + 12, val.w, unused);
                    }
                    *reinterpret_cast<uint4 *>(blk + c * 512) = val;
                }
            } else {
            // residues packed 4 / RB to a word in row order
            uint32_t packed[COLS_PER_WARP * RB / 4];
#pragma unroll
            for (int c = 0; c < COLS_PER_WARP; c += 4) {
                if constexpr (RB == 2) pack4(c, packed[c >> 1], packed[(c >> 1) + 1]);
                else {
                    uint32_t unused;
                    pack4(c, packed[c >> 2], unused);
                }
            }
            unsigned char *rbase = static_cast<unsigned char *>(p.R) + it.mod * p.mod_stride * RB;
            if (p.vec_store && i0 + COLS_PER_WARP <= p.m) {
                // Transpose through a per-warp shared buffer so that one store instruction writes
                // whole lines of the residue array (128 bytes per column for uint16, 64 for uint8)
                // instead of 32 separate 16-byte pieces.  Chunks are XOR-swizzled by the line
                // number: both the writes and the reads are free of bank conflicts.
                unsigned char *xp = xpose_base + (warp - FIRST_EPI_WARP) * XPOSE_BYTES;
                if constexpr (RB == 2) {
                    // 16 lines x 128 bytes per pass; lane -> line lane/8 + 4t, 16-byte chunk lane%8
#pragma unroll
                    for (int rho = 0; rho < 2; ++rho) {
                        if ((lane >> 4) == rho) {
                            const int lr = lane & 15;
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                *reinterpret_cast<uint4 *>(xp + lr * 128 + ((c ^ (lr & 7)) << 4)) =
                                    make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
                        }
                        __syncwarp();
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            const int lr = (lane >> 3) + 4 * t, c = lane & 7;
                            uint4 val = *reinterpret_cast<const uint4 *>(xp + lr * 128 + ((c ^ (lr & 7)) << 4));
                            const int64_t jg = jw + 16 * rho + lr;
                            if (jg < p.n) *reinterpret_cast<uint4 *>(rbase + (jg * p.ldr + i0 + 8 * c) * 2) = val;
                        }
                        __syncwarp();
                    }
                } else {
                    // 32 lines x 64 bytes in one pass; lane -> line lane/4 + 8t, 16-byte chunk lane%4
#pragma unroll
                    for (int c = 0; c < NCH; ++c)
                        *reinterpret_cast<uint4 *>(xp + lane * 64 + (((c ^ (lane >> 1)) & 3) << 4)) =
                            make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
                    __syncwarp();
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int lr = (lane >> 2) + 8 * t, c = lane & 3;
                        uint4 val = *reinterpret_cast<const uint4 *>(xp + lr * 64 + (((c ^ (lr >> 1)) & 3) << 4));
                        const int64_t jg = jw + lr;
                        if (jg < p.n) *reinterpret_cast<uint4 *>(rbase + jg * p.ldr + i0 + 16 * c) = val;
                    }
                    __syncwarp();
                }
            } else if (j < p.n) {
                unsigned char *dst = rbase + (j * p.ldr + i0) * RB;
#pragma unroll
                for (int c = 0; c < COLS_PER_WARP; ++c)
                    if (i0 + c < p.m) {
                        if constexpr (RB == 2)
                            reinterpret_cast<uint16_t *>(dst)[c] = static_cast<uint16_t>((packed[c >> 1] >> (16 * (c & 1))) & 0xFFFFu);
                        else
                            dst[c] = static_cast<unsigned char>((packed[c >> 2] >> (8 * (c & 3))) & 0xFFu);
                    }
            }
            }   // public layout
            }   // residues
        }
    }

    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();      // neither CTA leaves while the other may still touch it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<CG>(tmem_base, TMEM_COLS);
    }
}

#include "oz_gemm_fused.cuh"

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// 3-D map over planes[plane][line][kbyte]; box = 128 bytes x box_lines lines x 1 plane,
// 128-byte swizzle, out-of-range elements read as zero.
bool make_plane_map(CUtensorMap *map, const uint8_t *base, int64_t lines, int64_t pitch,
                    int64_t plane_stride, int planes, int box_lines)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(pitch), static_cast<cuuint64_t>(lines),
                          static_cast<cuuint64_t>(planes)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(pitch), static_cast<cuuint64_t>(plane_stride)};
    cuuint32_t box[3] = {static_cast<cuuint32_t>(BLOCK_K), static_cast<cuuint32_t>(box_lines), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<uint8_t *>(base), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

// 3-D map over planes[plane][line][kbyte] for the fused kernel: box = 16 bytes x 128 lines x 1 plane,
// no swizzle (8 rows x 16 bytes land as one contiguous core matrix), out-of-range elements read as zero.
bool make_core_matrix_map(CUtensorMap *map, const uint8_t *base, int64_t lines, int64_t pitch,
                          int64_t plane_stride, int planes)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(pitch), static_cast<cuuint64_t>(lines),
                          static_cast<cuuint64_t>(planes)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(pitch), static_cast<cuuint64_t>(plane_stride)};
    cuuint32_t box[3] = {16, 128, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<uint8_t *>(base), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

template <int SUB, int SET>
oz_status_t launch_fused_variant(const CUtensorMap &mapB, const GemmParams &p, const FusedGemmParams &f, int sms,
                                 cudaStream_t stream)
{
    constexpr int LAYOUT_A = SUB == 0 ? kLayoutMerged : kLayoutMergedI8A;
    auto kernel = fused_gemm_kernel<SUB, SET, LAYOUT_A>;
    constexpr size_t smem = fused_gemm_smem(SET);
    OZ_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    const int grid = f.tiles < sms ? f.tiles : sms;
    kernel<<<grid, F_THREADS, smem, stream>>>(mapB, p, f);
    count_launch();
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

template <int SUB, int CG, int RB, bool DIRECT = false, bool LOOSE = false, bool TILED = false, bool BOUND = false>
oz_status_t launch_variant(const CUtensorMap &mapA, const CUtensorMap &mapB, const GemmParams &p, int sms,
                           cudaStream_t stream)
{
    static_assert(!LOOSE || RB == 2, "a representative below 2m needs the two-byte element");
    auto kernel = residue_gemm_kernel<SUB, CG, RB, DIRECT, LOOSE, TILED, BOUND>;
    OZ_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(SMEM_BYTES)));
    int64_t groups = sms / CG;                                    // CTAs, or CTA pairs
    if (p.total_items < groups) groups = p.total_items;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(groups * CG));
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    OZ_CUDA_CHECK(cudaLaunchKernelEx(&cfg, kernel, mapA, mapB, p));
    count_launch();
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

}  // namespace

// Which variant runs: CTA pairs (tcgen05 cta_group::2, tiles of 256 columns) unless that would pad
// the column count noticeably more than 128-column tiles do (n = 128: one half-empty pair tile).
static int cta_group_choice(int64_t n)
{
    const int64_t pad1 = round_up(n, BLOCK_M), pad2 = round_up(n, 2 * BLOCK_M);
    return (pad2 * 20 <= pad1 * 21) ? 2 : 1;
}

// Test hook for the bounded waits, read once when the library is loaded: with
// OZ_TEST_STALL_PRODUCER=once in the environment the first residue-GEMM launch of the process loads
// no operand, every role's wait runs into its time limit, the kernel sets OZ_ERR_TIMEOUT and
// returns cleanly; later launches are normal.  ("1": every launch.)
static std::atomic<int> g_stall_producer{[] {
    const char *env = getenv("OZ_TEST_STALL_PRODUCER");
    if (!env) return 0;
    return env[0] == '1' ? 1 : (env[0] == 'o' ? 2 : 0);
}()};

static int take_stall_flag()
{
    int v = g_stall_producer.load();
    if (v == 2) {
        g_stall_producer.store(0);
        return 1;
    }
    return v;
}

// Per-modulus constants of the epilogue and the accumulator schedule (jobs, weights, which
// accumulators are reduced before they are weighted, K segments) for inner dimension k; p.r and p.nk
// (chunks of BLOCK_K) are set by the caller.
static void fill_mod_info(GemmParams &p, int set, const Route &rt, int64_t k)
{
    for (int i = 0; i < p.r; ++i) {
        int mi = modulus(set, i), s = square_root(mi);
        p.mod[i].m = static_cast<float>(mi);
        p.mod[i].inv_m = 1.0f / static_cast<float>(mi);
        // Exact range of the running combination.  Digits are bounded by |d0| <= 14 (16 for
        // squares), |d1| <= 16, |d0+d1| <= 22 (Lemma 1), a reduced accumulator by (m+1)/2 <= 545
        // (FP32 path, balanced) or m-1 <= 1088 (integer path, canonical).  A job's accumulator may
        // be weighted without reducing it first while the worst-case sum stays inside the exact
        // range: 2^24 for the FP32 epilogue, 2^31 (minus headroom for the bias) for the integer one.
        const bool integer = rt.substrate != 0;
        const int64_t lim = integer ? (1ll << 31) - 8192 : (1ll << 24) - 1, kk = k > 0 ? k : 1;
        const int64_t red = integer ? 1088 : 545;
        ModInfo &mo = p.mod[i];
        mo.mi = static_cast<uint32_t>(mi);
        mo.magic = barrett_magic(static_cast<uint32_t>(mi));
        mo.bias = static_cast<uint32_t>((((1ull << 31) + mi - 1) / mi) * mi);
        mo.magic39 = mi > 128 ? static_cast<uint32_t>(((1ull << 39) + mi - 1) / mi) : 0u;
        mo.bias30 = static_cast<uint32_t>((((1ull << 30) + mi - 1) / mi) * mi);
        mo.planeA0 = first_plane(set, i, rt.layout(0));
        mo.planeB0 = first_plane(set, i, rt.layout(1));
        mo.nseg = 1;
        mo.seg_len = p.nk;
        // exact depth of one accumulator, in chunks of BLOCK_K: the largest term is 2 * 16 * 16 (the
        // two-product job of a square), 128 * 128 for native residues
        const int seg_max_all = !integer ? (1 << 24) / 512 / BLOCK_K
                                         : static_cast<int>(((1ll << 31) - 1) / (rt.native() ? 16384 : 512) / BLOCK_K);
        mo.nseg_all = (p.nk + seg_max_all - 1) / seg_max_all;
        mo.seg_len_all = (p.nk + mo.nseg_all - 1) / mo.nseg_all;
        const bool split = mo.nseg_all > 1;       // then every accumulator is reduced before it is weighted
        if (rt.native()) {
            mo.njobs = 1;
            mo.kind = 2;
            mo.w[0] = 1.0f; mo.w[1] = mo.w[2] = 0.0f;
            mo.reduce[0] = split ? 1 : 0;
            mo.reduce[1] = mo.reduce[2] = 1;
        } else if (s) {
            mo.njobs = 2;
            mo.kind = 0;
            mo.w[0] = 1.0f; mo.w[1] = static_cast<float>(s); mo.w[2] = 0.0f;
            const bool skip_all = !split && integer && (256 + 512 * static_cast<int64_t>(s)) * kk <= lim;
            mo.reduce[0] = (skip_all || (!split && 256 * kk + static_cast<int64_t>(s) * red <= lim)) ? 0 : 1;
            mo.reduce[1] = skip_all ? 0 : 1;
            mo.reduce[2] = 1;
        } else if (rt.merged()) {
            // d e = -15 [d0 e0 - 16 d1 e1] + 16 dS eS; merged term <= 4095 (9-bit tail) or 1088 (bytes).
            // INT8 planes hold -d0 and 4*d1, so the accumulator is the NEGATIVE of the bracket (weight
            // +15) and its term is bounded by 4292 for every modulus up to 1089.
            mo.njobs = 2;
            mo.kind = 3;
            mo.w[0] = integer ? 15.0f : -15.0f; mo.w[1] = 16.0f; mo.w[2] = 0.0f;
            // K longer than the exact range of one merged accumulator is cut into equal segments,
            // each drained and reduced on its own (the residues add modulo m).
            const int64_t merged_term = integer ? 4292 : (mi > 256 ? 4095 : 1088);
            const int seg_max = integer ? static_cast<int>(((1ll << 31) - 1) / merged_term / BLOCK_K)
                                        : static_cast<int>(merged_k_limit(set) / BLOCK_K);
            mo.nseg = (p.nk + seg_max - 1) / seg_max;
            if (mo.nseg < 1) mo.nseg = 1;
            mo.seg_len = (p.nk + mo.nseg - 1) / mo.nseg;
            const bool skip_all = !split && mo.nseg == 1 && (15 * merged_term + 16 * 484) * kk <= lim;
            mo.reduce[0] = skip_all ? 0 : 1;
            mo.reduce[1] = (skip_all || (!split && 16 * 484 * kk + 15 * red * mo.nseg <= lim)) ? 0 : 1;
            mo.reduce[2] = 1;
        } else {
            mo.njobs = 3;
            mo.kind = 1;
            mo.w[0] = -15.0f; mo.w[1] = 16.0f; mo.w[2] = 240.0f;
            const bool skip_all = !split && integer && (15 * 196 + 16 * 484 + 240 * 256) * kk <= lim;
            const bool skip01 = skip_all || (!split && (15 * 196 + 16 * 484) * kk + 240 * red <= lim);
            mo.reduce[0] = skip01 ? 0 : 1;
            mo.reduce[1] = skip01 ? 0 : 1;
            mo.reduce[2] = skip_all ? 0 : 1;
        }
        for (int j = 0; j < 3; ++j) mo.iw[j] = static_cast<int>(mo.w[j]);
    }
}

ResidueTiling residue_tiling(int64_t m, int64_t n, int set)
{
    ResidueTiling t;
    t.cg = cta_group_choice(n);
    t.tile_cols = BLOCK_M * t.cg;
    t.tiles_m = static_cast<int>((m + BLOCK_N - 1) / BLOCK_N);
    t.tiles_n = static_cast<int>((n + t.tile_cols - 1) / t.tile_cols);
    t.mod_stride = static_cast<int64_t>(t.tiles_m) * t.tiles_n * t.tile_cols * BLOCK_N;
    (void)set;
    return t;
}

oz_status_t launch_residue_gemm(int64_t m, int64_t n, int64_t k, const uint8_t *PA, int64_t strideA,
                                int64_t pitchA, const uint8_t *PB, int64_t strideB, int64_t pitchB,
                                int set, const Route &rt, void *R, int64_t ldr,
                                int64_t mod_stride, bool loose, bool tiled, cudaStream_t stream)
{
    const int cg = cta_group_choice(n);
    GemmParams p{};
    p.m = m; p.n = n; p.k = k;
    p.tiles_m = static_cast<int>((m + BLOCK_N - 1) / BLOCK_N);             // 256 rows of C per tile
    p.tiles_n = static_cast<int>((n + BLOCK_M * cg - 1) / (BLOCK_M * cg)); // 128 (256) columns of C per tile
    const int rb = residue_bytes(set);
    p.vec_store = ((ldr * rb) % 16 == 0 && (mod_stride * rb) % 16 == 0 && (reinterpret_cast<uintptr_t>(R) & 15u) == 0) ? 1 : 0;
    p.nk = static_cast<int>((k + BLOCK_K - 1) / BLOCK_K);
    if (k == 0) p.nk = 1;   // one all-zero chunk (the planes' padding) gives residues 0
    p.r = set_r(set);
    p.total_items = static_cast<int64_t>(p.r) * p.tiles_m * p.tiles_n;
    if (p.total_items >= 0x7FFFFFFFll) return OZ_ERR_UNSUPPORTED;        // item numbers are 32-bit in the kernel
    p.R = R; p.ldr = ldr; p.mod_stride = mod_stride;
    p.stall_producer = take_stall_flag();
    p.status = device_status_word();
    fill_mod_info(p, set, rt, k);

    CUtensorMap mapA, mapB;
    if (!make_plane_map(&mapA, PA, m, pitchA, strideA, p_store(set, rt.layout(0)), BLOCK_N / cg) ||
        !make_plane_map(&mapB, PB, n, pitchB, strideB, p_store(set, rt.layout(1)), BLOCK_M))
        return OZ_ERR_CUDA;

    int dev = 0, sms = 148;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    OZ_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    // substrate 0: FP8 planes; otherwise INT8 planes (two-limb digits or native residues)
#define OZ_LAUNCH(SUB, RB, DIRECT, LOOSE, TILED)                                                    \
    (cg == 2 ? launch_variant<SUB, 2, RB, DIRECT, LOOSE, TILED>(mapA, mapB, p, sms, stream)        \
             : launch_variant<SUB, 1, RB, DIRECT, LOOSE, TILED>(mapA, mapB, p, sms, stream))
#define OZ_LAUNCH_SUB(RB, LOOSE, TILED)                                                             \
    (rt.substrate == 0 ? OZ_LAUNCH(0, RB, false, LOOSE, TILED) : OZ_LAUNCH(1, RB, false, LOOSE, TILED))
    // one accumulator per modulus of at most 128 * 128 * k <= 2^30: the direct drain with the exact division
    if (rt.native() && p.mod[0].nseg_all == 1 && k <= 65536)
        return tiled ? OZ_LAUNCH(1, 1, true, false, true) : OZ_LAUNCH(1, 1, true, false, false);
    if (rb == 1) return tiled ? OZ_LAUNCH_SUB(1, false, true) : OZ_LAUNCH_SUB(1, false, false);
    // the tile-ordered array is private to the whole-method calls, which also take the loose residues
    if (tiled) return OZ_LAUNCH_SUB(2, true, true);
    if (loose) return OZ_LAUNCH_SUB(2, true, false);
    return OZ_LAUNCH_SUB(2, false, false);
#undef OZ_LAUNCH_SUB
#undef OZ_LAUNCH
}

// Whether the fused mode applies: merged schedule on digit planes, all of B in one 128-lane tile, and
// an inner dimension that every accumulator holds exactly without K segments.
bool fused_gemm_applies(int64_t m, int64_t n, int64_t k, int set, const Route &rt)
{
    if (rt.native() || !rt.merged() || n < 1 || n > BLOCK_M || m < 1 || k < 1) return false;
    if ((m + F_LINES - 1) / F_LINES >= 0x7FFFFFFFll) return false;
    // one accumulator per job over all of k: FP32 holds the merged term (4095 on the 9-bit tail of S,
    // 1088 on byte moduli) exactly to 2^24, INT32 the term 4292 far beyond any k taken here; where the
    // epilogue reduces an accumulator before weighting it is decided for this k by fill_mod_info
    const int64_t kmax = rt.substrate == 0 ? merged_k_limit(set) : 262144;
    return k <= kmax;
}

// Residue products with A converted on the fly (storage mode F): A in FP64 with the shifts of its rows,
// B's planes materialised in the layout of side 1 of the route; canonical residues in the public layout
// R[mod][j][ldr], ldr a multiple of 64 and at least m rounded up to 64 (the last tile stores whole).
oz_status_t launch_fused_gemm(int64_t m, int64_t n, int64_t k, const double *A, int64_t lda, const int32_t *shiftA,
                              const uint8_t *PB, int64_t strideB, int64_t pitchB, int set, const Route &rt,
                              void *R, int64_t ldr, int64_t mod_stride, cudaStream_t stream)
{
    if (!fused_gemm_applies(m, n, k, set, rt)) return OZ_ERR_UNSUPPORTED;
    if (ldr % F_LINES != 0 || ldr < round_up(m, F_LINES) || (reinterpret_cast<uintptr_t>(R) & 15u)) return OZ_ERR_INVALID_ARG;
    GemmParams p{};
    p.m = m; p.n = n; p.k = k;
    p.r = set_r(set);
    p.nk = static_cast<int>((k + BLOCK_K - 1) / BLOCK_K);
    p.R = R; p.ldr = ldr; p.mod_stride = mod_stride;
    p.stall_producer = 0;
    p.status = device_status_word();
    fill_mod_info(p, set, rt, k);
    FusedGemmParams f{};
    f.A = A; f.lda = lda; f.shiftA = shiftA;
    f.lut_global = device_lut(set, rt.substrate);
    f.tz = rt.quant;
    f.tiles = static_cast<int>((m + F_LINES - 1) / F_LINES);
    f.passes = (p.r + F_GROUP - 1) / F_GROUP;
    f.nks = static_cast<int>((k + F_K - 1) / F_K);
    CUtensorMap mapB;
    if (!make_core_matrix_map(&mapB, PB, n, pitchB, strideB, p_store(set, rt.layout(1)))) return OZ_ERR_CUDA;
    int dev = 0, sms = 148;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    OZ_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
#define OZ_FUSED_GEMM(SET_) \
    (rt.substrate == 0 ? launch_fused_variant<0, SET_>(mapB, p, f, sms, stream) : launch_fused_variant<1, SET_>(mapB, p, f, sms, stream))
    if (set == 0) return OZ_FUSED_GEMM(0);
    if (set == 1) return OZ_FUSED_GEMM(1);
    return OZ_FUSED_GEMM(2);
#undef OZ_FUSED_GEMM
}

// The magnitude-bound product of the accurate mode: one E4M3 plane per operand (digits <= 32, terms
// <= 1024, so one FP32 accumulator is exact for k <= 16384), the same tiles, TMA ring and tcgen05
// instructions as the residue products, and an epilogue that keeps only the row and column maxima.
oz_status_t launch_bound_gemm(int64_t m, int64_t n, int64_t k, const uint8_t *GA, int64_t pitchA,
                              const uint8_t *GB, int64_t pitchB, unsigned int *rowmax,
                              unsigned int *colmax, cudaStream_t stream)
{
    if (k > kBoundKMax) return OZ_ERR_UNSUPPORTED;
    const int cg = cta_group_choice(n);
    GemmParams p{};
    p.m = m; p.n = n; p.k = k;
    p.tiles_m = static_cast<int>((m + BLOCK_N - 1) / BLOCK_N);
    p.tiles_n = static_cast<int>((n + BLOCK_M * cg - 1) / (BLOCK_M * cg));
    p.nk = static_cast<int>((k + BLOCK_K - 1) / BLOCK_K);
    if (k == 0) p.nk = 1;
    p.r = 1;
    p.total_items = static_cast<int64_t>(p.tiles_m) * p.tiles_n;
    if (p.total_items >= 0x7FFFFFFFll) return OZ_ERR_UNSUPPORTED;
    p.stall_producer = 0;
    p.status = device_status_word();
    p.rowmax = rowmax;
    p.colmax = colmax;
    ModInfo &mo = p.mod[0];
    mo.m = 1.0f; mo.inv_m = 1.0f; mo.mi = 1u;
    mo.njobs = 1;
    mo.kind = 2;                       // one plane, one K-loop
    mo.w[0] = 1.0f;
    mo.iw[0] = 1;
    mo.reduce[0] = 0;
    mo.planeA0 = mo.planeB0 = 0;
    mo.nseg = mo.nseg_all = 1;
    mo.seg_len = mo.seg_len_all = p.nk;
    CUtensorMap mapA, mapB;
    if (!make_plane_map(&mapA, GA, m, pitchA, m * pitchA, 1, BLOCK_N / cg) ||
        !make_plane_map(&mapB, GB, n, pitchB, n * pitchB, 1, BLOCK_M))
        return OZ_ERR_CUDA;
    int dev = 0, sms = 148;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    OZ_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    return cg == 2 ? launch_variant<0, 2, 2, true, false, false, true>(mapA, mapB, p, sms, stream)
                   : launch_variant<0, 1, 2, true, false, false, true>(mapA, mapB, p, sms, stream);
}

}  // namespace oz
