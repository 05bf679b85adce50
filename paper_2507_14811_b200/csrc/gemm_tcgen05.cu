// W8A8 GEMM + dequantizing epilogue for sm_100a (Sec. 4.2.2 segment-wise products, Sec. 4.3.2 dual
// path recombination, App. A symmetric recovery).
//
// Persistent kernel, one CTA per SM, 384 threads.  With CG = 2 two neighbouring CTAs (a cluster of
// two) work on one 256-row output tile with tcgen05 cta_group::2: each CTA loads its own 128
// activation rows and HALF of the weight tile, the pair's leader issues every MMA, and each CTA
// holds the accumulators of its own 128 rows in its tensor memory (TMEM).  CG = 1 is the same
// kernel with one CTA per 128-row tile (used when M <= 128).
//   warp 0      TMA producer (one lane): per 128-byte K-block, one tile of each activation code
//               matrix and this CTA's part of ONE weight tile into a shared-memory ring
//   warp 1      tcgen05.mma issuer (one lane, leader CTA only): for every 32-byte K-step one MMA of the
//               positive (or only) code matrix against the weight tile; every (K-segment, polarity) has
//               its own accumulator in TMEM
//   warp 2      dual layers: the same for the negative code matrix, against the SAME weight tile
//   warp 3      idle: it fills the first warpgroup, which hands most of its registers to the others
//   warps 4..11 epilogue: tcgen05.ld of the accumulators of a 32-column slab, y = bias + sum over
//               (segment, polarity) of factor * accumulator in fp32, -> bf16 (32 x 32 blocks staged in
//               shared memory and written by TMA stores) or fp32 / unaligned output (plain stores)
// Registers: the kernel starts with 168 per thread; warps 0..3 drop to 56 (setmaxnreg.dec) and the epilogue
// warps rise to 224 (setmaxnreg.inc): 128 x 56 + 256 x 224 = 384 x 168, the CTA's allocation.  The
// epilogue uses them to hold up to six 32-column accumulator loads at once, so that a tile's accumulators
// are back with the MMA issuer early in the epilogue.
// One K-segment: the npol accumulators (128 lanes x TILE_N columns each) of a tile stay in TMEM until the
// tile's epilogue; if they use at most half of TMEM there are two sets, and the epilogue of one tile
// overlaps the main loop of the next.  A dual 256-wide tile fills TMEM: its two polarities are handed back
// to their issuing threads separately.  Single-scale layers may use 256 x 512 tiles built the same way
// (WIDE below).  Several K-segments: see SEQ below.
// Every wait on an mbarrier is bounded (SM cycle counter, about 2 s); on expiry the CTA records
// which wait gave up in the status word, stops issuing work, lets its own copies land and leaves
// normally.  No load uses cluster multicast.
// Host side: prepare_gemm works out everything a launch needs (tile plan, kernel instantiation, tensor maps,
// shared-memory size, grid) without launching; run_gemm is one cudaLaunchKernelExC from that.
#include <atomic>
#include <mutex>
#include <vector>
#include <cuda_bf16.h>
#include "sq_common.cuh"

namespace sq {
namespace {

constexpr int TILE_M = 128;           // rows per CTA (TMEM lanes)
constexpr int BLOCK_K = 128;          // bytes (= codes) per K-block: one 128B swizzle row
constexpr int MMA_K = 32;             // codes per tcgen05.mma of an 8-bit kind
constexpr int kEpiWarps = 8;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kFrontThreads = 128;     // warpgroup 0: producer, MMA issuer, two idle warps
constexpr int kThreads = kFrontThreads + kEpiThreads;
constexpr int kLaunchRegs = 168;      // per thread at launch: 65536 / 384, rounded down to a multiple of 8
constexpr int kFrontRegs = 56, kEpiRegs = 224;     // per-thread register counts after the role split
// setmaxnreg.inc waits, without limit, until the CTA's OWN register allocation (made at launch) has that many
// registers free, so the new counts must fit in what the launch gave the CTA
static_assert(kFrontThreads * kFrontRegs + kEpiThreads * kEpiRegs <= kThreads * kLaunchRegs,
              "register counts after the role split exceed the CTA's allocation");
static_assert(kFrontRegs % 8 == 0 && kEpiRegs % 8 == 0 && kFrontRegs >= 24 && kEpiRegs <= 256, "setmaxnreg operand");
constexpr int kEpiBufRegs = 192;      // of kEpiRegs: accumulator load buffers plus running sums (SEQ)
constexpr int kResidentBufs = 4;      // accumulator load buffers of the resident epilogue
constexpr int kMaxStages = 8;
constexpr int kTmemCols = 512;
constexpr uint32_t kSmemBudget = 227 * 1024;
constexpr long long kWaitLimitCycles = 4000000000ll;   // about 2 s
constexpr uint32_t kStageBytesPerWarp = 32 * 64;       // one 32 x 32 bf16 output block per epilogue warp
constexpr uint32_t kStageBytes = kEpiWarps * kStageBytesPerWarp;
constexpr int kMaxTokenSegments = 32;                  // per-token layers: channel scales of up to 32 K-segments (32 KiB at 256 columns) are staged per tile
constexpr int kMaxFactorTable = 2048;                  // (K-segments x polarities) x N-segments factors in shared memory

// ----------------------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Programmatic dependent launch: the kernel may start while the previous kernel of the stream is still
// finishing.  grid_dependency_wait() returns once that kernel has completed and its writes are visible;
// every thread calls it before its first access to global memory.  grid_launch_dependents() lets the
// next kernel of the stream (if launched the same way) be scheduled as this one winds down.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// arrive on a barrier given by a shared::cluster address (possibly in the peer CTA)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait.  Returns false if the wait expired or another role already gave up.  The limit is
// counted on the SM cycle counter; kWaitLimitCycles is about 2 s at the maximum SM clock.
__device__ __forceinline__ uint32_t ld_shared_volatile_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.volatile.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void st_shared_volatile_u32(uint32_t addr, uint32_t v)
{
    asm volatile("st.volatile.shared::cta.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
// abort_flag: shared-memory address of the CTA's abort word
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t abort_flag,
                                          uint32_t *status, uint32_t where)
{
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = 0;
    uint32_t polls = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 63u) == 0) {
            if (ld_shared_volatile_u32(abort_flag)) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            if (now - t0 > kWaitLimitCycles) {
                st_shared_volatile_u32(abort_flag, 1u);
                atomicCAS(status, 0u, where);
                return false;
            }
        }
    }
    return true;
}

// 2-D tiled TMA load into this CTA's shared memory; completion bytes go to `bar`, which for CG = 2
// is a shared::cluster address (the leader CTA's barrier).
template <int CG>
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    if (CG == 1)
        asm volatile(
            "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
            ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
    else
        asm volatile(
            "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
            ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}

__device__ __forceinline__ void ld_shared_2x64(uint32_t addr, uint64_t &a, uint64_t &b)
{
    asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "r"(addr));
}
__device__ __forceinline__ float ld_shared_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t ld_shared_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
// packed fp32 pairs (two outputs per instruction)
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ uint64_t pack_b32x2(uint32_t lo, uint32_t hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// 16- and 32-byte global stores
__device__ __forceinline__ void st_global_16(void *p, uint4 v)
{
    asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void st_global_32(void *p, uint4 a, uint4 b)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Arrives on `bar` once every MMA issued so far by this thread has retired.  CG = 2: the arrival is
// delivered to the barrier at the same shared-memory offset in both CTAs of the pair.
template <int CG>
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    if (CG == 1)
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    else
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(bar), "h"(uint16_t(3)) : "memory");
}

template <int KIND, int CG>   // KIND 0: kind::i8, 1: kind::f8f6f4
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate)
{
    if (KIND == 0 && CG == 1)
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    else if (KIND == 0)
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    else if (CG == 1)
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp receives lane (base_lane + t).
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile stored as 128-byte rows with the 128B swizzle
// (the layout a 2-D TMA load with CU_TENSOR_MAP_SWIZZLE_128B writes): start address >> 4 in bits
// 0-13, stride between 8-row groups (1024 B) >> 4 in bits 32-45, descriptor version 1 in bits 46-47,
// swizzle mode 2 (128B) in bits 61-63.  The leading-dimension offset is unused for this layout.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= uint64_t((smem_addr & 0x3FFFFu) >> 4);
    d |= uint64_t(1024u >> 4) << 32;
    d |= uint64_t(1) << 46;
    d |= uint64_t(2) << 61;
    return d;
}

// Instruction descriptor: D format bits 4-5 (1 = f32, 2 = s32), A format bits 7-9, B format bits
// 10-12 (kind::i8: 1 = signed 8-bit; kind::f8f6f4: 0 = e4m3), A and B K-major (bits 15, 16 = 0),
// N >> 3 in bits 17-22, M >> 4 in bits 24-28 (M = 128 per CTA, 256 for a CTA pair).
__host__ __device__ constexpr uint32_t make_idesc(int kind, int tile_n, int mma_m)
{
    return (kind == 0 ? (2u << 4) | (1u << 7) | (1u << 10) : (1u << 4)) |
           (uint32_t(tile_n >> 3) << 17) | (uint32_t(mma_m >> 4) << 24);
}

// ----------------------------------------------------------------------------- the kernel

// bytes of the epilogue's tables between the ring and the header (multiple of 16)
__host__ __device__ constexpr uint32_t epi_table_bytes(int nacc, int Q, int tile_n)
{
    return ((uint32_t(tile_n) + uint32_t(nacc) * Q + uint32_t(Q) + 1u) * 4u + 15u) & ~15u;
}

struct SharedHeader {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t sk_flag;            // (split tiles) the arrival count the CTA's thread 0 read, for the other epilogue threads
};

// Split tiles (SK variants): the work of a launch is the sequence of all (tile, K-block) units, tile-major, cut
// into one contiguous range per CTA pair: pair c takes units [c U / C, (c + 1) U / C).  A range is walked as
// segments (tile, K-blocks k0 .. k1 - 1); a segment that is not a whole tile is a PARTIAL one.  Every role of a
// CTA walks the same sequence.
struct SkWalk {
    int u, u_begin, u_end, kblocks;
};
__device__ __forceinline__ int sk_bound(int c, int total_units, int pairs)
{
    return int((long long)c * total_units / pairs);
}
__device__ __forceinline__ SkWalk sk_range(int pair, int pairs, int num_tiles, int kblocks)
{
    const int total = num_tiles * kblocks;
    SkWalk w;
    w.u_begin = sk_bound(pair, total, pairs);
    w.u_end = sk_bound(pair + 1, total, pairs);
    w.u = w.u_begin;
    w.kblocks = kblocks;
    return w;
}
__device__ __forceinline__ bool sk_next(SkWalk &w, int &tile, int &k0, int &k1)
{
    if (w.u >= w.u_end) return false;
    tile = w.u / w.kblocks;
    k0 = w.u - tile * w.kblocks;
    const int rem = w.u_end - w.u;
    k1 = k0 + rem < w.kblocks ? k0 + rem : w.kblocks;
    w.u += k1 - k0;
    return true;
}
// the pair whose range holds unit x: the largest c with c U / C <= x
__device__ __forceinline__ int sk_owner(int x, int total_units, int pairs)
{
    return int((((long long)x + 1) * pairs - 1) / total_units);
}
// barrier 1 of the 256 epilogue threads, returning the AND of their predicates
__device__ __forceinline__ bool epilogue_all(bool pred)
{
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %1, 0;\n\tbar.red.and.pred q, 1, 256, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                 : "=r"(r) : "r"(uint32_t(pred)) : "memory");
    return r != 0;
}
__device__ __forceinline__ uint4 ld_global_cg_16(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

// where-codes written to the status word when a wait expires
enum : uint32_t { kWhereProducer = 0x100, kWhereMmaFull = 0x200, kWhereMmaTmem = 0x300, kWhereEpilogue = 0x400 };

// A whole K-block (four K-steps of 32 codes, each against every activation tile) issued from one block
// of PTX.  The issuing thread is the only one feeding the tensor pipe, so its instruction count per
// MMA matters when MMAs are short (narrow tiles): descriptors differ only in the 14-bit address field
// of their low word, so each one costs a 32-bit add with an immediate; the accumulate predicate is set
// once.  %0 TMEM address, %1 / %2 low words of the A / B descriptors of the stage, %3 their common high
// word, %4 instruction descriptor, %5 accumulate flag of the first K-step, %6 TILE_N (second
// polarity's accumulator).  Offsets: +2 per K-step (32 bytes >> 4), +1024 to the second activation tile.
#define SQ_KBLOCK_1(OP)                                                                                   \
    "{\n\t.reg .pred pf, pt;\n\t.reg .b64 da, db;\n\t.reg .b32 la, lb;\n\t"                              \
    "setp.ne.b32 pf, %5, 0;\n\tsetp.eq.b32 pt, %5, %5;\n\t"                                               \
    "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t" OP " [%0], da, db, %4, pf;\n\t"                  \
    "add.u32 la, %1, 2;\n\tadd.u32 lb, %2, 2;\n\tmov.b64 da, {la, %3};\n\tmov.b64 db, {lb, %3};\n\t"      \
    OP " [%0], da, db, %4, pt;\n\t"                                                                       \
    "add.u32 la, %1, 4;\n\tadd.u32 lb, %2, 4;\n\tmov.b64 da, {la, %3};\n\tmov.b64 db, {lb, %3};\n\t"      \
    OP " [%0], da, db, %4, pt;\n\t"                                                                       \
    "add.u32 la, %1, 6;\n\tadd.u32 lb, %2, 6;\n\tmov.b64 da, {la, %3};\n\tmov.b64 db, {lb, %3};\n\t"      \
    OP " [%0], da, db, %4, pt;\n\t}"
#define SQ_KBLOCK_2(OP)                                                                                   \
    "{\n\t.reg .pred pf, pt;\n\t.reg .b64 da, db;\n\t.reg .b32 la, lb, td;\n\t"                          \
    "setp.ne.b32 pf, %5, 0;\n\tsetp.eq.b32 pt, %5, %5;\n\tadd.u32 td, %0, %6;\n\t"                        \
    "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t" OP " [%0], da, db, %4, pf;\n\t"                  \
    "add.u32 la, %1, 1024;\n\tmov.b64 da, {la, %3};\n\t" OP " [td], da, db, %4, pf;\n\t"                  \
    "add.u32 la, %1, 2;\n\tadd.u32 lb, %2, 2;\n\tmov.b64 da, {la, %3};\n\tmov.b64 db, {lb, %3};\n\t"      \
    OP " [%0], da, db, %4, pt;\n\t"                                                                       \
    "add.u32 la, %1, 1026;\n\tmov.b64 da, {la, %3};\n\t" OP " [td], da, db, %4, pt;\n\t"                  \
    "add.u32 la, %1, 4;\n\tadd.u32 lb, %2, 4;\n\tmov.b64 da, {la, %3};\n\tmov.b64 db, {lb, %3};\n\t"      \
    OP " [%0], da, db, %4, pt;\n\t"                                                                       \
    "add.u32 la, %1, 1028;\n\tmov.b64 da, {la, %3};\n\t" OP " [td], da, db, %4, pt;\n\t"                  \
    "add.u32 la, %1, 6;\n\tadd.u32 lb, %2, 6;\n\tmov.b64 da, {la, %3};\n\tmov.b64 db, {lb, %3};\n\t"      \
    OP " [%0], da, db, %4, pt;\n\t"                                                                       \
    "add.u32 la, %1, 1030;\n\tmov.b64 da, {la, %3};\n\t" OP " [td], da, db, %4, pt;\n\t}"
#define SQ_KBLOCK_ARGS ::"r"(d0), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate), "n"(TILE_N) : "memory"

template <int KIND, int NPOL, int TILE_N, int CG>
__device__ __forceinline__ void issue_full_kblock(uint32_t d0, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                                  uint32_t accumulate)
{
    static_assert(BLOCK_K / MMA_K == 4 && ((TILE_M * BLOCK_K) >> 4) == 1024, "offsets are written into the PTX");
    if (NPOL == 1) {
        if (KIND == 0 && CG == 1) asm volatile(SQ_KBLOCK_1("tcgen05.mma.cta_group::1.kind::i8") SQ_KBLOCK_ARGS);
        else if (KIND == 0) asm volatile(SQ_KBLOCK_1("tcgen05.mma.cta_group::2.kind::i8") SQ_KBLOCK_ARGS);
        else if (CG == 1) asm volatile(SQ_KBLOCK_1("tcgen05.mma.cta_group::1.kind::f8f6f4") SQ_KBLOCK_ARGS);
        else asm volatile(SQ_KBLOCK_1("tcgen05.mma.cta_group::2.kind::f8f6f4") SQ_KBLOCK_ARGS);
    } else {
        if (KIND == 0 && CG == 1) asm volatile(SQ_KBLOCK_2("tcgen05.mma.cta_group::1.kind::i8") SQ_KBLOCK_ARGS);
        else if (KIND == 0) asm volatile(SQ_KBLOCK_2("tcgen05.mma.cta_group::2.kind::i8") SQ_KBLOCK_ARGS);
        else if (CG == 1) asm volatile(SQ_KBLOCK_2("tcgen05.mma.cta_group::1.kind::f8f6f4") SQ_KBLOCK_ARGS);
        else asm volatile(SQ_KBLOCK_2("tcgen05.mma.cta_group::2.kind::f8f6f4") SQ_KBLOCK_ARGS);
    }
}

// One K-block worth of MMAs: nk K-steps of 32 codes, each against every activation tile.
template <int KIND, int NPOL, int TILE_N, int CG>
__device__ __forceinline__ void issue_kblock(uint32_t d0, uint64_t da, uint64_t db, uint32_t idesc, int nk,
                                             uint32_t accumulate)
{
    constexpr uint64_t kATileDesc = uint64_t(TILE_M * BLOCK_K) >> 4;   // next activation tile in the stage
    if (nk == BLOCK_K / MMA_K) {
        issue_full_kblock<KIND, NPOL, TILE_N, CG>(d0, uint32_t(da), uint32_t(db), uint32_t(da >> 32), idesc, accumulate);
    } else {
        for (int kk = 0; kk < nk; kk++) {
            const uint64_t koff = uint64_t((kk * MMA_K) >> 4);
#pragma unroll
            for (int pol = 0; pol < NPOL; pol++)
                tc_mma<KIND, CG>(d0 + pol * TILE_N, da + pol * kATileDesc + koff, db + koff, idesc,
                                 kk == 0 ? accumulate : 1u);
        }
    }
}

// ----------------------------------------------------------------------------- epilogue pieces

// N-segment of column n: the number of interior bounds nb[1..Q-1] that are <= n, counted warp-wide
// (all 32 lanes call it together).
__device__ __forceinline__ int seg_of_column(int n, int Q, uint32_t nb_addr, int lane)
{
    int cnt = 0;
    for (int base = 1; base < Q; base += 32) {
        const int i = base + lane;
        const bool le = i < Q && n >= int(ld_shared_u32(nb_addr + 4u * uint32_t(i < Q ? i : 0)));
        cnt += __popc(__ballot_sync(0xFFFFFFFFu, le));
    }
    return cnt;
}

// y += c[a][q(column)] * acc for the 32 columns nf .. nf + 31 of one row; y holds 16 packed fp32 pairs, r the
// raw accumulator words of one TMEM load.  A slab that lies in one N-segment (q_lo == q_hi; always so in the
// production variant) takes one factor; otherwise the factor is looked up per column.
// INIT: y starts from the bias slice at shared address bias_slab (32 floats) instead of its old value.
// Per-token x per-channel factors (4-bit weights with per-channel scales, activations with per-token scales):
// the factor of column n is row_factor * col_scale[n * col_stride], row_factor being the token's scale for this
// accumulator.  col_scale == nullptr: factors come from the table.  Only the checking variant carries this.
struct TokenScale {
    float row_factor;
    const float *col_scale;      // already offset to the accumulator's K-segment
    int col_stride, N;
    uint32_t col_smem;           // nonzero: shared address such that col_smem + 4 n holds column n's scale (this tile)
};
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t ld_shared_64(uint32_t addr)
{
    uint64_t v;
    asm volatile("ld.shared.b64 %0, [%1];" : "=l"(v) : "r"(addr));
    return v;
}

template <int KIND, bool GENERIC, bool INIT = false, bool PT = false>
__device__ __forceinline__ void scale_add_unit(uint64_t (&y2)[16], const uint32_t (&r)[32], int a, int Q, int q_lo,
                                               int q_hi, int nf, uint32_t tab_addr, uint32_t nb_addr,
                                               uint32_t bias_slab = 0, const TokenScale *ts = nullptr)
{
    if (GENERIC && ts && ts->col_scale) {
        if (INIT) {
#pragma unroll
            for (int j4 = 0; j4 < 8; j4++) ld_shared_2x64(bias_slab + uint32_t(16 * j4), y2[2 * j4], y2[2 * j4 + 1]);
        }
        const uint64_t rf2 = pack_f32x2(ts->row_factor, ts->row_factor);
#pragma unroll
        for (int j = 0; j < 16; j++) {
            uint64_t c2;
            if (ts->col_smem) {                       // the tile's channel scales are staged in shared memory
                c2 = mul_f32x2(rf2, ld_shared_64(ts->col_smem + uint32_t(nf + 2 * j) * 4u));
            } else {
                float cc[2];
#pragma unroll
                for (int t = 0; t < 2; t++) {
                    const int n = nf + 2 * j + t;
                    cc[t] = n < ts->N ? __fmul_rn(ts->row_factor, __ldg(ts->col_scale + size_t(n) * ts->col_stride)) : 0.0f;
                }
                c2 = pack_f32x2(cc[0], cc[1]);
            }
            const uint64_t v2 = KIND == 0 ? pack_f32x2(__int2float_rn(int(r[2 * j])), __int2float_rn(int(r[2 * j + 1])))
                                          : pack_b32x2(r[2 * j], r[2 * j + 1]);
            y2[j] = fma_f32x2(c2, v2, y2[j]);
        }
        return;
    }
    if (!GENERIC || q_lo == q_hi) {
        // PT (production variant of the per-token layer): the token's scale times the staged channel scales
        const float c = PT ? ts->row_factor : ld_shared_f32(tab_addr + uint32_t(a * Q + q_lo) * 4u);
        uint64_t c2 = pack_f32x2(c, c);
        const uint64_t rf2 = c2;
#pragma unroll
        for (int j4 = 0; j4 < 8; j4++) {
            uint64_t b0 = y2[2 * j4], b1 = y2[2 * j4 + 1];
            if (INIT) ld_shared_2x64(bias_slab + uint32_t(16 * j4), b0, b1);
#pragma unroll
            for (int t = 0; t < 2; t++) {
                const int j = 2 * j4 + t;
                if (PT) c2 = mul_f32x2(rf2, ld_shared_64(ts->col_smem + uint32_t(nf + 2 * j) * 4u));
                const uint64_t v2 = KIND == 0 ? pack_f32x2(__int2float_rn(int(r[2 * j])), __int2float_rn(int(r[2 * j + 1])))
                                              : pack_b32x2(r[2 * j], r[2 * j + 1]);
                y2[j] = fma_f32x2(c2, v2, t == 0 ? b0 : b1);
            }
        }
    } else {
        if (INIT) {
#pragma unroll
            for (int j4 = 0; j4 < 8; j4++) ld_shared_2x64(bias_slab + uint32_t(16 * j4), y2[2 * j4], y2[2 * j4 + 1]);
        }
        int q = q_lo;
#pragma unroll
        for (int j = 0; j < 16; j++) {
            float cc[2];
#pragma unroll
            for (int t = 0; t < 2; t++) {
                while (q < q_hi && nf + 2 * j + t >= int(ld_shared_u32(nb_addr + 4u * uint32_t(q + 1)))) q++;
                cc[t] = ld_shared_f32(tab_addr + uint32_t(a * Q + q) * 4u);
            }
            const uint64_t v2 = KIND == 0 ? pack_f32x2(__int2float_rn(int(r[2 * j])), __int2float_rn(int(r[2 * j + 1])))
                                          : pack_b32x2(r[2 * j], r[2 * j + 1]);
            y2[j] = fma_f32x2(pack_f32x2(cc[0], cc[1]), v2, y2[j]);
        }
    }
}

// raw accumulator words of one unit -> dump[a][row][nf .. nf + 31] (parity tests)
__device__ __forceinline__ void dump_unit(void *acc_dump, const uint32_t (&r)[32], int a, int row, int nf, int M, int N)
{
    uint32_t *dump = static_cast<uint32_t *>(acc_dump) + (size_t(a) * M + row) * size_t(N) + nf;
#pragma unroll
    for (int j = 0; j < 32; j++)
        if (nf + j < N) dump[j] = r[j];
}

// 32 fp32 outputs (16 packed pairs) -> 32 bf16 (16 words), round to nearest even
__device__ __forceinline__ void pack_bf16(const uint64_t (&y2)[16], uint32_t (&h)[16])
{
#pragma unroll
    for (int j = 0; j < 16; j++) {
        float lo, hi;
        unpack_f32x2(y2[j], lo, hi);
        __nv_bfloat162 v2 = __floats2bfloat162_rn(lo, hi);
        h[j] = *reinterpret_cast<uint32_t *>(&v2);
    }
}

// Where the production variant's output goes: the warp's 32 x 32 bf16 block is staged in shared memory and
// written by one TMA store (whole 64-byte row pieces per request instead of one request per lane and piece).
struct YOut {
    const CUtensorMap *tm;   // Y as [M, N] bf16, box 32 x 32, 64-byte swizzle
    uint32_t stage;          // this warp's 2 KiB staging buffer (shared address, 1 KiB aligned)
    int lane;
    int row0;                // first row of the warp's 32-row block
};

// Lane l holds row row0 + l of the block as 16 words h (32 bf16, columns col .. col + 31).  Rows beyond M and
// columns beyond N are clipped by the tensor map; a block entirely outside is skipped.  The previous store of
// this warp must have finished READING the staging buffer before it is overwritten; lane 0 issued it, so lane 0
// waits for it.
__device__ __forceinline__ void tma_store_block(const uint32_t (&h)[16], const YOut &yo, int col, int M, int N)
{
    if (yo.row0 >= M || col >= N) return;               // warp-uniform
    if (yo.lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    __syncwarp();
    const uint32_t row_addr = yo.stage + uint32_t(yo.lane) * 64u;
    const uint32_t sw = (uint32_t(yo.lane) >> 1) & 3u;  // 64-byte swizzle: 16-byte piece index ^ bits 7-8 of the address
#pragma unroll
    for (int c = 0; c < 4; c++)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_addr + ((uint32_t(c) ^ sw) << 4)),
                     "r"(h[4 * c]), "r"(h[4 * c + 1]), "r"(h[4 * c + 2]), "r"(h[4 * c + 3]) : "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (yo.lane == 0) {
        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                     ::"l"(reinterpret_cast<uint64_t>(yo.tm)), "r"(col), "r"(yo.row0), "r"(yo.stage) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
}
// before the CTA's shared memory goes away (all lanes may call; lane 0 issued the stores)
__device__ __forceinline__ void tma_store_drain(const YOut &yo)
{
    if (yo.lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    __syncwarp();
}

// Converts and stores the 32 outputs y of row `row`, columns nf .. nf + 31, in 16-byte chunks (8 bf16 or
// 4 fp32).  N is a multiple of 8, so a chunk is entirely inside or outside the matrix; two adjacent chunks go
// out as one 32-byte store when the rows of Y are 32-byte aligned.
// The production variant (GENERIC = false) is called by all 32 lanes of the warp together and writes through
// yo; the generic one writes row `row` (< M) from registers.
template <bool GENERIC, typename Params>
__device__ __forceinline__ void store_slab(const uint64_t (&y2)[16], const Params &prm, int row, int nf, const YOut &yo)
{
    const int nvalid = prm.N - nf;                       // valid columns of this slab, may exceed 32
    if (!GENERIC) {
        uint32_t h[16];
        pack_bf16(y2, h);
        tma_store_block(h, yo, nf, prm.M, prm.N);
    } else if (prm.y_is_f32) {
        float *dst = static_cast<float *>(prm.Y) + size_t(row) * prm.ldy + nf;
#pragma unroll
        for (int c = 0; c < 4; c++) {                    // 8 columns = 32 bytes
            if (8 * c < nvalid) {
                const uint4 lo = make_uint4(uint32_t(y2[4 * c]), uint32_t(y2[4 * c] >> 32),
                                            uint32_t(y2[4 * c + 1]), uint32_t(y2[4 * c + 1] >> 32));
                const uint4 hi = make_uint4(uint32_t(y2[4 * c + 2]), uint32_t(y2[4 * c + 2] >> 32),
                                            uint32_t(y2[4 * c + 3]), uint32_t(y2[4 * c + 3] >> 32));
                if (prm.y_wide) st_global_32(dst + 8 * c, lo, hi);
                else { st_global_16(dst + 8 * c, lo); st_global_16(dst + 8 * c + 4, hi); }
            }
        }
    } else {
        __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(prm.Y) + size_t(row) * prm.ldy + nf;
        uint32_t h[16];
#pragma unroll
        for (int j = 0; j < 16; j++) {
            float lo, hi;
            unpack_f32x2(y2[j], lo, hi);
            __nv_bfloat162 v2 = __floats2bfloat162_rn(lo, hi);
            h[j] = *reinterpret_cast<uint32_t *>(&v2);
        }
#pragma unroll
        for (int c = 0; c < 2; c++) {                    // 16 columns = 32 bytes
            const uint4 w0 = make_uint4(h[8 * c], h[8 * c + 1], h[8 * c + 2], h[8 * c + 3]);
            const uint4 w1 = make_uint4(h[8 * c + 4], h[8 * c + 5], h[8 * c + 6], h[8 * c + 7]);
            if (16 * c + 8 < nvalid && prm.y_wide) {
                st_global_32(dst + 16 * c, w0, w1);
            } else {
                if (16 * c < nvalid) st_global_16(dst + 16 * c, w0);
                if (16 * c + 8 < nvalid) st_global_16(dst + 16 * c + 8, w1);
            }
        }
    }
}

// GENERIC = false is the production variant: bf16 output, no accumulator dump, every interior N-bound
// a multiple of 32 (so that each 32-column slab of the output lies in one N-segment and takes ONE
// dequantization factor per accumulator).  Its epilogue loop is small enough for the instruction
// cache.  GENERIC = true adds the fp32 output, the accumulator dump for the parity tests and a
// per-column factor lookup for slabs that straddle an N-bound.
// SEQ = true (layers with more than one K-segment): TMEM holds the accumulators of ONE K-segment at a time,
// in two alternating sets.  The MMA issuer fills a set with segment p while the epilogue warps drain the set
// of segment p - 1, scale it and add it to fp32 running sums kept in registers for the whole tile; the sums
// are converted and stored after the last segment.  Any number of K-segments fits, tiles stay wide, and the
// drain of every segment but the last overlaps tensor work.  SEQ = false keeps every (segment, polarity)
// accumulator of a tile resident in TMEM and drains once per tile.
// WIDE = true (single-scale layers, one K-segment, CTA pairs): the tile is 256 rows x 512 columns, two 256-column
// halves that share ONE activation tile per K-block, the mirror image of a dual tile (two activation tiles, one
// weight tile).  A single-scale 256 x 256 tile asks for 64 bytes of operands per SM cycle, which is all the L2
// path delivers; the wide tile asks for 48.  Each half has its own weight tile in the ring stage, its own
// issuing thread and accumulator, and is released to its thread separately, like the polarities of a dual tile.
// PT = true: the production variant for layers with per-token and per-channel scales (W4A8): the tile's channel
// scales are staged in shared memory and every factor is the token's scale times the channel's.
// SK = true (one K-segment, CTA pairs, layers whose tile count fills the machine badly): the K loops of the tiles
// are cut so that every CTA pair gets the same number of K-blocks (SkWalk above).  A CTA that has worked on part
// of a tile's K range writes its raw accumulators (exact int32 sums, or fp32 ones) to a slot of the caller's
// workspace and counts itself in on the tile's counter; the CTA whose count completes the tile adds the slots up,
// in the order of the K ranges, and runs the tile's epilogue.  Nobody waits for anybody.
template <int KIND, int NPOL, int TILE_N, int CG, bool GENERIC, bool SEQ, bool WIDE = false, bool PT = false, bool SK = false>
// 384 threads = 12 warps, 3 on each SM sub-partition with 16 K registers: 168 registers per thread at launch
__global__ void __launch_bounds__(kThreads, 1)
segquant_gemm_kernel(const __grid_constant__ CUtensorMap tm_a_pos, const __grid_constant__ CUtensorMap tm_a_neg,
                     const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_y,
                     const KernelParams prm)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // layout: [ring: stages x (NPOL A tiles of 16 KiB, B part of B_ROWS*128 B)] [output staging] [scales] [header]
    constexpr int B_ROWS = TILE_N / CG;                  // weight rows this CTA loads per K-block
    constexpr uint32_t a_bytes = TILE_M * BLOCK_K;
    constexpr uint32_t b_bytes = B_ROWS * BLOCK_K;
    constexpr int kHalves = WIDE ? 2 : 1;                // weight tiles per stage
    constexpr int kTileCols = TILE_N * kHalves;          // output columns of a tile
    constexpr int kIssuers = (NPOL == 2 || WIDE) ? 2 : 1;
    static_assert(!WIDE || (NPOL == 1 && TILE_N == 256 && CG == 2 && !GENERIC && !SEQ), "wide single-scale tile");
    static_assert(!SK || (CG == 2 && !GENERIC && !SEQ && !WIDE && !PT && NPOL * TILE_N == 256), "split tiles");
    constexpr uint32_t stage_bytes = NPOL * a_bytes + kHalves * b_bytes;
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sh_stage = smem + size_t(prm.stages) * stage_bytes;      // 1 KiB aligned: stages are multiples of 1 KiB
    float *sh_bias = reinterpret_cast<float *>(sh_stage + (GENERIC ? 0 : kStageBytes));     // [TILE_N], per tile
    float *sh_tab = sh_bias + kTileCols;                                                    // [nacc][Q], per launch
    int *sh_nb = reinterpret_cast<int *>(sh_tab + prm.nacc * prm.sb.Q);                     // [Q + 1]
    // (per-token mode, few K-segments) the tile's channel scales [P][kTileCols], refreshed per tile
    float *sh_col = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(sh_bias) +
                                              epi_table_bytes(prm.nacc, prm.sb.Q, kTileCols));
    SharedHeader *hdr = reinterpret_cast<SharedHeader *>(reinterpret_cast<uint8_t *>(sh_col) + prm.col_tab_bytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = CG == 2 ? cluster_rank() : 0u;       // 0 = leader of the pair
    const int unit = blockIdx.x / CG, num_units = gridDim.x / CG;
    const int num_tiles = prm.num_m_tiles * prm.num_n_tiles;
    const uint32_t abort_flag = smem_u32(&hdr->abort_flag);

    if (threadIdx.x == 32 * 0 + 1) {     // descriptor fetches overlap the set-up below
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_a_pos)) : "memory");
        if (NPOL == 2) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_a_neg)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_b)) : "memory");
        if (!GENERIC) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_y)) : "memory");
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < prm.stages; s++) {
            mbar_init(smem_u32(&hdr->full[s]), 1);
            mbar_init(smem_u32(&hdr->empty[s]), kIssuers);      // one arrival per MMA-issuing thread
        }
        for (int s = 0; s < 2; s++) {
            mbar_init(smem_u32(&hdr->tmem_full[s]), kIssuers);
            mbar_init(smem_u32(&hdr->tmem_empty[s]), CG * kEpiWarps);
        }
        hdr->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // Every thread arrives at the cluster barrier now (thread 0 after its barrier initialisation) and waits for it
    // only after the TMEM allocation below, so the barrier's latency overlaps the allocation.
    __syncwarp();
    if (CG == 2) asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    if (warp == 1) {
        if (CG == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&hdr->tmem_base)), "r"(uint32_t(kTmemCols)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&hdr->tmem_base)), "r"(uint32_t(kTmemCols)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (CG == 2) asm volatile("barrier.cluster.wait.acquire;" ::: "memory");   // the peer's barriers are initialised
    tc_fence_after();
    const uint32_t tmem_base = hdr->tmem_base;
    const int acc_cols = (SEQ ? NPOL : prm.nacc) * kTileCols;  // TMEM columns of one accumulator set
    // A dual 256-wide tile (one K-segment) fills TMEM, so there is one accumulator set and the tensor pipe would
    // idle during the epilogue up to the set's release.  Instead the two polarities are released SEPARATELY
    // (barrier tmem_empty[0] = positive accumulator free, tmem_empty[1] = negative one): the epilogue reads all
    // positive columns first, and the thread that issues the positive MMAs starts the next tile as soon as they
    // are in registers, ahead of the negative thread by at most the depth of the ring.
    constexpr bool kSplitRel = (NPOL == 2 && TILE_N == 256 && !SEQ && !GENERIC && !SK) || WIDE;
    const int sk_pairs = min(num_units, num_tiles * prm.sk_kblocks);    // (SK) pairs that have a range

    // The producer and the MMA issuer are single threads: their loops are kept to a few dozen
    // instructions per K-block (ring slot and phase advance incrementally, descriptors by addition).
    if (warp < kFrontThreads / 32) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kFrontRegs));
      if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint32_t stages = prm.stages, P = prm.sb.P;
            const uint32_t full0 = smem_u32(&hdr->full[0]), empty0 = smem_u32(&hdr->empty[0]);
            grid_dependency_wait();                 // the code matrices come from the previous kernel
            // completion bytes of both CTAs' loads are counted on the leader's barrier
            const uint32_t full0_sig = CG == 2 ? map_to_cta(full0, 0) : full0;
            const uint32_t ring0 = smem_u32(smem);
            uint32_t s = 0, ph = 0, issued = 0;
            bool ok = true;
            if constexpr (SK) {
                SkWalk w = sk_range(unit, sk_pairs, num_tiles, prm.sk_kblocks);
                int tile = 0, k0 = 0, k1 = 0;
                while (ok && unit < sk_pairs && sk_next(w, tile, k0, k1)) {
                    const int m0 = (tile / prm.num_n_tiles) * (TILE_M * CG) + int(rank) * TILE_M;
                    const int n0 = (tile % prm.num_n_tiles) * kTileCols + int(rank) * B_ROWS;
                    for (int kbi = k0; kbi < k1; kbi++) {
                        if (!mbar_wait(empty0 + 8 * s, ph ^ 1, abort_flag, prm.status, kWhereProducer)) {
                            ok = false;
                            break;
                        }
                        const uint32_t dst = ring0 + s * stage_bytes;
                        if (rank == 0) mbar_expect_tx(full0 + 8 * s, CG * stage_bytes);
                        const uint32_t bar = full0_sig + 8 * s;
                        tma_load_2d<CG>(dst, &tm_a_pos, bar, kbi * BLOCK_K, m0);
                        if (NPOL == 2) tma_load_2d<CG>(dst + a_bytes, &tm_a_neg, bar, kbi * BLOCK_K, m0);
                        tma_load_2d<CG>(dst + NPOL * a_bytes, &tm_b, bar, kbi * BLOCK_K, n0);
                        issued++;
                        if (++s == stages) { s = 0; ph ^= 1; }
                    }
                }
            }
            for (int tile = unit; !SK && tile < num_tiles && ok; tile += num_units) {
                const int m0 = (tile / prm.num_n_tiles) * (TILE_M * CG) + int(rank) * TILE_M;
                const int n0 = (tile % prm.num_n_tiles) * kTileCols + int(rank) * B_ROWS;
                for (uint32_t p = 0; p < P && ok; p++) {
                    const int k_end = prm.sb.kb[p + 1];
                    for (int k = prm.sb.kb[p]; k < k_end; k += BLOCK_K) {
                        if (!mbar_wait(empty0 + 8 * s, ph ^ 1, abort_flag, prm.status, kWhereProducer)) {
                            ok = false;
                            break;
                        }
                        const uint32_t dst = ring0 + s * stage_bytes;
                        if (rank == 0) mbar_expect_tx(full0 + 8 * s, CG * stage_bytes);
                        const uint32_t bar = full0_sig + 8 * s;
                        tma_load_2d<CG>(dst, &tm_a_pos, bar, k, m0);
                        if (NPOL == 2) tma_load_2d<CG>(dst + a_bytes, &tm_a_neg, bar, k, m0);
                        tma_load_2d<CG>(dst + NPOL * a_bytes, &tm_b, bar, k, n0);
                        if (WIDE) tma_load_2d<CG>(dst + NPOL * a_bytes + b_bytes, &tm_b, bar, k, n0 + TILE_N);
                        issued++;
                        if (++s == stages) { s = 0; ph ^= 1; }
                    }
                }
            }
            grid_launch_dependents();               // all of this CTA's loads are issued: the tail begins
            if (!ok && rank == 0) {
                // let the copies this thread issued land before the CTA's shared memory goes away
                const uint32_t pending = issued < stages ? issued : stages;
                for (uint32_t j = 0; j < pending; j++) {
                    if (s == 0) { s = stages; ph ^= 1; }
                    s--;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(full0 + 8 * s, ph) && clock64() - t0 < 200000000ll) {}
                }
            }
        }
      } else if (warp == 1 || (kIssuers == 2 && warp == 2)) {
        // ------------------------------------------------------------------ MMA issuers (leader CTA)
        // One thread per polarity: warp 1 issues the MMAs of the positive code matrix, warp 2 (dual layers)
        // those of the negative one, each into its own accumulators.  A tcgen05.mma keeps its issuing thread
        // busy for about 70 cycles, more than a 128-column MMA occupies the tensor pipe, so one thread cannot
        // feed the pipe for narrow dual tiles.  Ring slots and accumulator sets are handed on when BOTH
        // threads' MMAs have retired (barrier counts NPOL).  With the per-polarity release of a dual 256-wide
        // tile each thread waits for its own accumulator only, so the positive thread starts the next tile
        // while the negative accumulator is still being read (it can run ahead by the depth of the ring).
        if (lane == 0 && rank == 0) {
            const uint32_t pol = uint32_t(warp - 1);
            constexpr uint32_t idesc = make_idesc(KIND, TILE_N, TILE_M * CG);
            const uint32_t stages = prm.stages, P = prm.sb.P, acc_stages = prm.acc_stages;
            const uint32_t full0 = smem_u32(&hdr->full[0]), empty0 = smem_u32(&hdr->empty[0]);
            // dual: thread `pol` takes activation tile `pol`; wide: thread `pol` takes weight tile (half) `pol`
            const uint64_t desc0 = make_smem_desc(smem_u32(smem)) + (WIDE ? 0u : pol) * (uint64_t(a_bytes) >> 4);
            constexpr uint64_t kStageDesc = uint64_t(stage_bytes) >> 4;
            const uint64_t b_off = WIDE ? (uint64_t(a_bytes) >> 4) + pol * (uint64_t(b_bytes) >> 4)
                                        : (uint64_t(NPOL * a_bytes) >> 4) - pol * (uint64_t(a_bytes) >> 4);
            uint32_t s = 0, ph = 0, as = 0, aph = 0;
            bool ok = true;
            if constexpr (SK) {
                SkWalk w = sk_range(unit, sk_pairs, num_tiles, prm.sk_kblocks);
                int tile = 0, k0 = 0, k1 = 0;
                while (ok && unit < sk_pairs && sk_next(w, tile, k0, k1)) {
                    if (!mbar_wait(smem_u32(&hdr->tmem_empty[as]), aph ^ 1, abort_flag, prm.status, kWhereMmaTmem)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t d0 = tmem_base + as * acc_cols + pol * TILE_N;
                    uint32_t accumulate = 0;                       // a segment starts from zero wherever it begins in K
                    for (int kbi = k0; kbi < k1; kbi++) {
                        if (!mbar_wait(full0 + 8 * s, ph, abort_flag, prm.status, kWhereMmaFull)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint64_t da = desc0 + s * kStageDesc;
                        const int rem = prm.K - kbi * BLOCK_K;
                        const int nk = rem >= BLOCK_K ? BLOCK_K / MMA_K : (rem + MMA_K - 1) / MMA_K;
                        issue_kblock<KIND, 1, TILE_N, CG>(d0, da, da + b_off, idesc, nk, accumulate);
                        accumulate = 1;
                        tc_commit<CG>(empty0 + 8 * s);
                        if (++s == stages) { s = 0; ph ^= 1; }
                    }
                    if (ok) tc_commit<CG>(smem_u32(&hdr->tmem_full[as]));
                    if (++as == acc_stages) { as = 0; aph ^= 1; }
                }
            }
            for (int tile = unit; !SK && tile < num_tiles && ok; tile += num_units) {
                if (!SEQ) {
                    const uint32_t bar = smem_u32(&hdr->tmem_empty[kSplitRel ? pol : as]);
                    if (!mbar_wait(bar, aph ^ 1, abort_flag, prm.status, kWhereMmaTmem)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                }
                for (uint32_t p = 0; p < P && ok; p++) {
                    if (SEQ) {                                     // one accumulator set per K-segment
                        if (!mbar_wait(smem_u32(&hdr->tmem_empty[as]), aph ^ 1, abort_flag, prm.status, kWhereMmaTmem)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                    }
                    const uint32_t d0 = tmem_base + as * acc_cols + (SEQ ? 0u : p * (NPOL * TILE_N)) + pol * TILE_N;
                    const int k_end = prm.sb.kb[p + 1];
                    uint32_t accumulate = 0;
                    for (int k = prm.sb.kb[p]; k < k_end; k += BLOCK_K) {
                        if (!mbar_wait(full0 + 8 * s, ph, abort_flag, prm.status, kWhereMmaFull)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint64_t da = desc0 + s * kStageDesc;
                        const int rem = k_end - k;
                        const int nk = rem >= BLOCK_K ? BLOCK_K / MMA_K : (rem + MMA_K - 1) / MMA_K;
                        issue_kblock<KIND, 1, TILE_N, CG>(d0, da, da + b_off, idesc, nk, accumulate);
                        accumulate = 1;
                        tc_commit<CG>(empty0 + 8 * s);             // the slot is free when both threads' MMAs have retired
                        if (++s == stages) { s = 0; ph ^= 1; }
                    }
                    if (SEQ) {
                        if (ok) tc_commit<CG>(smem_u32(&hdr->tmem_full[as]));  // accumulators of this segment complete
                        if (++as == acc_stages) { as = 0; aph ^= 1; }
                    }
                }
                if (!SEQ) {
                    if (ok) tc_commit<CG>(smem_u32(&hdr->tmem_full[as]));  // accumulators of this tile complete
                    if (++as == acc_stages) { as = 0; aph ^= 1; }
                }
            }
        }
      }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        // Warp w may read TMEM lanes 32 * (w % 4) .. + 31; the two warps of one lane group take one half
        // of the tile's 32-column slabs each.  Per output: y = bias, then y = fma(c[a][q], acc[a], y) over
        // a = (p, polarity) ascending, two outputs per instruction on packed fp32 pairs.
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kEpiRegs));
        const int et = threadIdx.x - kFrontThreads;
        const int ew = warp - kFrontThreads / 32;
        const int lane_grp = warp & 3;
        constexpr int kColGroups = kEpiWarps / 4;
        constexpr int kSlabs = TILE_N / 32;
        constexpr int kSlabsPerWarp = (kSlabs + kColGroups - 1) / kColGroups;
        const int slab0 = (ew >> 2) * kSlabsPerWarp;
        const int nacc = prm.nacc;
        const int P = prm.sb.P, Q = prm.sb.Q;
        const uint32_t tmem_empty_sig0 = CG == 2 ? map_to_cta(smem_u32(&hdr->tmem_empty[0]), 0)
                                                 : smem_u32(&hdr->tmem_empty[0]);
        const uint32_t tab_addr = smem_u32(sh_tab), nb_addr = smem_u32(sh_nb), bias_addr = smem_u32(sh_bias);
        auto release = [&](uint32_t set) {             // accumulator set `set` is in registers: hand it back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (CG == 2) mbar_arrive_cluster(tmem_empty_sig0 + 8 * set);
                else mbar_arrive(tmem_empty_sig0 + 8 * set);
            }
        };
        // bias slice of a tile, one column per thread, fetched one tile ahead into a register
        auto fetch_bias = [&](int tile, int half = 0) -> float {
            if (tile >= num_tiles || et >= TILE_N || !prm.bias) return 0.0f;
            const int n = (tile % prm.num_n_tiles) * kTileCols + half * TILE_N + et;
            return n < prm.N ? __ldg(prm.bias + n) : 0.0f;
        };
        grid_dependency_wait();                     // scales, bias and Y may belong to the previous kernel
        SkWalk skw = sk_range(SK ? unit : 0, SK ? max(sk_pairs, 1) : 1, SK ? num_tiles : 0, SK ? prm.sk_kblocks : 1);
        float bias_next = fetch_bias(SK ? (unit < sk_pairs ? skw.u_begin / max(prm.sk_kblocks, 1) : num_tiles) : unit);
        float bias_next1 = WIDE ? fetch_bias(unit, 1) : 0.0f;   // second half of a wide tile
        // dequantization factors c[a][q] = s_act[p][pol] * s_w[p][q], a = p * NPOL + pol (one fp32 multiply);
        // built here, off the producer's and the MMA issuer's path, and published by the first tile's barrier
        const bool per_token = PT || (GENERIC && prm.col_scale != nullptr);      // factors per (token, channel), no table
        for (int i = et; i < nacc * Q && !per_token; i += kEpiThreads) {
            const int a = i / Q, q = i - a * Q, p = a / NPOL;
            const float s_act = (NPOL == 2 && (a & 1)) ? prm.s_neg[p] : prm.s_pos[p];
            sh_tab[i] = s_act * prm.s_w[p * Q + q];
        }
        // (per-token mode) this thread's token scale for accumulator a = p * NPOL + pol, and the channel scales of p
        const bool col_staged = per_token && prm.col_tab_bytes != 0;
        const uint32_t col_addr = smem_u32(sh_col);
        int tile_n0 = 0;                                                 // first column of the current tile
        auto token_scale = [&](int a, int row_) -> TokenScale {
            TokenScale t{0.0f, nullptr, 0, prm.N, 0u};
            if (per_token) {
                const int p = a / NPOL;
                const float *rs = (NPOL == 2 && (a & 1)) ? prm.row_neg : prm.row_pos;
                t.row_factor = row_ < prm.M ? __ldg(rs + size_t(row_) * P + p) : 0.0f;
                t.col_scale = prm.col_scale + p;
                t.col_stride = P;
                if (col_staged) t.col_smem = col_addr + uint32_t(p * kTileCols - tile_n0) * 4u;
            }
            return t;
        };
        for (int i = et; i <= Q; i += kEpiThreads) sh_nb[i] = prm.sb.nb[i];

        YOut yo{&tm_y, smem_u32(sh_stage) + uint32_t(ew) * kStageBytesPerWarp, lane, 0};
        uint32_t as = 0, aph = 0;
        bool ok = true;
        int tile = unit - num_units;
        while (true) {
            int sk_k0 = 0, sk_k1 = 0, next_tile = 0;          // (SK) this segment's K-blocks; the tile after this one
            if constexpr (SK) {
                if (unit >= sk_pairs || !sk_next(skw, tile, sk_k0, sk_k1)) break;
                SkWalk peek = skw;
                int pk0, pk1;
                if (!sk_next(peek, next_tile, pk0, pk1)) next_tile = num_tiles;
            } else {
                tile += num_units;
                if (tile >= num_tiles) break;
                next_tile = tile + num_units;
            }
            const int m0 = (tile / prm.num_n_tiles) * (TILE_M * CG) + int(rank) * TILE_M;
            const int n0 = (tile % prm.num_n_tiles) * kTileCols;
            const int row = m0 + lane_grp * 32 + lane;
            yo.row0 = m0 + lane_grp * 32;

            asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");   // previous tile's readers are done
            if (et < TILE_N) sh_bias[et] = bias_next;
            if ((GENERIC || PT) && col_staged) {                              // this tile's channel scales, all K-segments
                tile_n0 = n0;
                for (int i = et; i < P * kTileCols; i += kEpiThreads) {
                    const int pp = i / kTileCols, c = i - pp * kTileCols;
                    sh_col[i] = n0 + c < prm.N ? __ldg(prm.col_scale + size_t(n0 + c) * P + pp) : 0.0f;
                }
            }
            bias_next = fetch_bias(next_tile);                               // lands during this tile's work
            if (WIDE) {
                sh_bias[TILE_N + et] = bias_next1;                           // et < 256 = TILE_N for every epilogue thread
                bias_next1 = fetch_bias(next_tile, 1);
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");

            // A warp's share of one accumulator set is kUnits TMEM loads (unit u = slab u / NPOL, polarity
            // u % NPOL).  Up to NB of them are in registers at once: NB loads go out at the start, and the
            // buffer freed by unit u - 1 takes the load of unit u - 1 + NB while unit u is scaled.  Once the last
            // load has landed the set goes back to the MMA issuer.  (With one resident set per tile that moment
            // is on the critical path, so there the last load goes out AHEAD of the wait that precedes unit u.)
            if constexpr (SEQ) {
                // ---- one accumulator set per K-segment: running sums of the whole tile stay in registers
                static_assert(!SEQ || kSlabsPerWarp * kColGroups == kSlabs, "SEQ needs TILE_N >= 64");
                constexpr int kUnits = kSlabsPerWarp * NPOL;                // TMEM loads per segment and warp
                constexpr int kBufMax = GENERIC ? 2 : (kEpiBufRegs - 32 * kSlabsPerWarp) / 32;
                constexpr int NB = kUnits < kBufMax ? kUnits : kBufMax;
                constexpr int kRel = kUnits <= NB ? 0 : kUnits - NB + 1;    // unit before which the set is released
                static_assert(NB >= 2 || kUnits == 1, "needs two load buffers");
                uint64_t y2[kSlabsPerWarp][16];
                int q_lo[kSlabsPerWarp], q_hi[kSlabsPerWarp];
#pragma unroll
                for (int sl = 0; sl < kSlabsPerWarp; sl++) {
                    const int c0 = (slab0 + sl) * 32;
                    q_lo[sl] = seg_of_column(n0 + c0, Q, nb_addr, lane);
                    q_hi[sl] = GENERIC ? seg_of_column(min(n0 + c0 + 31, prm.N - 1), Q, nb_addr, lane) : q_lo[sl];
#pragma unroll
                    for (int j4 = 0; j4 < 8; j4++)
                        ld_shared_2x64(bias_addr + uint32_t(c0 + 4 * j4) * 4u, y2[sl][2 * j4], y2[sl][2 * j4 + 1]);
                }
                for (int p = 0; p < P; p++) {
                    const uint32_t cur_as = as, cur_aph = aph;
                    if (++as == 2u) { as = 0; aph ^= 1; }
                    if (ok) ok = mbar_wait(smem_u32(&hdr->tmem_full[cur_as]), cur_aph, abort_flag, prm.status, kWhereEpilogue);
                    if (!ok) continue;
                    tc_fence_after();
                    const uint32_t t_row = tmem_base + (uint32_t(lane_grp * 32) << 16) + cur_as * acc_cols +
                                           uint32_t(slab0 * 32);
                    uint32_t buf[NB][32];
#pragma unroll
                    for (int u = 0; u < NB; u++) tc_ld32(t_row + uint32_t((u % NPOL) * TILE_N + (u / NPOL) * 32), buf[u]);
#pragma unroll
                    for (int u = 0; u < kUnits; u++) {
                        const int sl = u / NPOL, pol = u % NPOL;
                        tc_wait_ld();
                        if (u == kRel) release(cur_as);
                        if (u >= 1 && u - 1 + NB < kUnits)                           // buffer of unit u - 1 is free
                            tc_ld32(t_row + uint32_t(((u - 1 + NB) % NPOL) * TILE_N + ((u - 1 + NB) / NPOL) * 32),
                                    buf[(u - 1) % NB]);
                        const int a = p * NPOL + pol;
                        const int nf = n0 + (slab0 + sl) * 32;
                        const TokenScale tk = token_scale(a, row);
                        scale_add_unit<KIND, GENERIC, false, PT>(y2[sl], buf[u % NB], a, Q, q_lo[sl], q_hi[sl], nf, tab_addr, nb_addr, 0, &tk);
                        if (GENERIC && prm.acc_dump && row < prm.M)
                            dump_unit(prm.acc_dump, buf[u % NB], a, row, nf, prm.M, prm.N);
                    }
                }
                if (ok && (!GENERIC || row < prm.M)) {
#pragma unroll
                    for (int sl = 0; sl < kSlabsPerWarp; sl++)
                        store_slab<GENERIC>(y2[sl], prm, row, n0 + (slab0 + sl) * 32, yo);
                }
            } else {
                // ---- all accumulators of the tile resident
                const uint32_t cur_as = as, cur_aph = aph;
                if (++as == uint32_t(prm.acc_stages)) { as = 0; aph ^= 1; }
                if (ok) ok = mbar_wait(smem_u32(&hdr->tmem_full[cur_as]), cur_aph, abort_flag, prm.status, kWhereEpilogue);
                if constexpr (SK) ok = epilogue_all(ok);    // the barriers below need all 256 threads or none
                if (!ok) continue;                  // keep the named barriers balanced, do no more work
                tc_fence_after();
                const uint32_t t_row = tmem_base + (uint32_t(lane_grp * 32) << 16) + cur_as * acc_cols;
                constexpr bool kEvenSplit = kSlabsPerWarp * kColGroups == kSlabs;
                if constexpr (SK) {
                    const int kbt = prm.sk_kblocks;
                    if (!(sk_k0 == 0 && sk_k1 == kbt)) {
                        // ---- part of a tile's K range.  n pairs share the tile; the one that holds its first K-blocks
                        // (the OWNER; that segment is the last of its range, the others' segments the first of theirs)
                        // normally finds the other n - 1 partial sums waiting and finishes the tile from its own
                        // accumulators in TMEM plus their slots.  Counter protocol, without any waiting: a non-owner
                        // writes its slot, then adds 1; the owner adds 1 first, and if that did not read n - 1 it
                        // writes its slot too and adds 1 again.  Whoever brings the count to n + 1 (or the owner
                        // reading n - 1) finishes the tile, from the slots alone in the first case.
                        static_assert(!SK || kEvenSplit, "split tiles: every warp has the same number of slabs");
                        constexpr int kUnits = kSlabsPerWarp * NPOL;
                        constexpr size_t kSlotBytes = size_t(NPOL) * TILE_M * TILE_N * 4;   // one CTA's accumulators
                        const int total = num_tiles * kbt, tile_u0 = tile * kbt;
                        // slot 0 of a pair: the segment that starts the pair's range; slot 1: its other partial one
                        auto slot_of = [&](int pair, int seg_u0) {
                            const int sl = seg_u0 == sk_bound(pair, total, sk_pairs) ? 0 : 1;
                            return reinterpret_cast<uint4 *>(prm.sk_slots + size_t((pair * 2 + sl) * 2 + int(rank)) * kSlotBytes) + et;
                        };
                        const uint32_t t_warp = t_row + uint32_t(slab0 * 32);
                        uint32_t *cnt = prm.sk_counters + tile * 2 + int(rank);
                        const int c_first = sk_owner(tile_u0, total, sk_pairs), c_last = sk_owner(tile_u0 + kbt - 1, total, sk_pairs);
                        const int sharers = c_last - c_first + 1;
                        auto count_in = [&]() -> int {             // all 256 threads; returns the count before this arrival
                            asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
                            if (et == 0) {
                                const uint32_t before = atomicAdd(cnt, 1u);
                                __threadfence();
                                st_shared_volatile_u32(smem_u32(&hdr->sk_flag), before);
                            }
                            asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
                            return int(ld_shared_volatile_u32(smem_u32(&hdr->sk_flag)));
                        };
                        bool from_tmem = false;                    // finishing with this CTA's own sums still in TMEM
                        bool finish = false;
                        if (sk_k0 == 0) {
                            from_tmem = finish = count_in() == sharers - 1;
                        }
                        if (!from_tmem) {
                            uint4 *mine = slot_of(unit, tile_u0 + sk_k0);
                            uint32_t buf[2][32];
                            tc_ld32(t_warp, buf[0]);
#pragma unroll
                            for (int u = 0; u < kUnits; u++) {
                                tc_wait_ld();
                                if (u + 1 < kUnits)
                                    tc_ld32(t_warp + uint32_t(((u + 1) % NPOL) * TILE_N + ((u + 1) / NPOL) * 32), buf[(u + 1) & 1]);
                                else
                                    release(cur_as);
#pragma unroll
                                for (int j = 0; j < 8; j++)          // 512 consecutive bytes per warp and store
                                    st_global_16(mine + (u * 8 + j) * kEpiThreads,
                                                 make_uint4(buf[u & 1][4 * j], buf[u & 1][4 * j + 1], buf[u & 1][4 * j + 2], buf[u & 1][4 * j + 3]));
                            }
                            __threadfence();
                            finish = count_in() == sharers;         // n + 1 arrivals with this one
                        }
                        if (!finish) continue;
                        // ---- this CTA completes the tile: the sums of the K ranges in ascending order, then the usual
                        // epilogue.  The counter goes back to zero for the next launch.
                        if (et == 0) *cnt = 0u;
#pragma unroll 1
                        for (int sl = 0; sl < kSlabsPerWarp; sl++) {
                            const int c0 = (slab0 + sl) * 32, nf = n0 + c0;
                            const int q = seg_of_column(nf, Q, nb_addr, lane);
                            uint64_t y2[16];
#pragma unroll
                            for (int pol = 0; pol < NPOL; pol++) {
                                const int u = sl * NPOL + pol;
                                uint32_t acc[32];
                                if (from_tmem) {                   // the owner's range is the first in K (c_first == unit)
                                    tc_ld32(t_warp + uint32_t(pol * TILE_N + sl * 32), acc);
                                    tc_wait_ld();
                                } else {
#pragma unroll
                                    for (int j = 0; j < 32; j++) acc[j] = 0u;
                                }
                                // two slots' loads (16 of 16 bytes) are in flight before the first add
                                for (int c = c_first + (from_tmem ? 1 : 0); c <= c_last; c += 2) {
                                    const bool two = c + 1 <= c_last;
                                    const uint4 *src0 = slot_of(c, max(sk_bound(c, total, sk_pairs), tile_u0)) + u * 8 * kEpiThreads;
                                    const uint4 *src1 = two ? slot_of(c + 1, max(sk_bound(c + 1, total, sk_pairs), tile_u0)) + u * 8 * kEpiThreads
                                                            : src0;
                                    uint4 v[2][8];
#pragma unroll
                                    for (int j = 0; j < 8; j++) v[0][j] = ld_global_cg_16(src0 + j * kEpiThreads);
                                    if (two) {
#pragma unroll
                                        for (int j = 0; j < 8; j++) v[1][j] = ld_global_cg_16(src1 + j * kEpiThreads);
                                    }
#pragma unroll
                                    for (int h = 0; h < 2; h++) {
                                        if (h == 1 && !two) break;
#pragma unroll
                                        for (int j = 0; j < 8; j++) {
                                            const uint32_t w[4] = {v[h][j].x, v[h][j].y, v[h][j].z, v[h][j].w};
#pragma unroll
                                            for (int t = 0; t < 4; t++)
                                                acc[4 * j + t] = KIND == 0 ? acc[4 * j + t] + w[t]
                                                                           : __float_as_uint(__uint_as_float(acc[4 * j + t]) + __uint_as_float(w[t]));
                                        }
                                    }
                                }
                                const TokenScale tk = token_scale(pol, row);
                                if (pol == 0)
                                    scale_add_unit<KIND, false, true, false>(y2, acc, 0, Q, q, q, nf, tab_addr, nb_addr,
                                                                             bias_addr + uint32_t(c0) * 4u, &tk);
                                else
                                    scale_add_unit<KIND, false, false, false>(y2, acc, pol, Q, q, q, nf, tab_addr, nb_addr, 0, &tk);
                            }
                            store_slab<GENERIC>(y2, prm, row, nf, yo);
                        }
                        if (from_tmem) release(cur_as);
                        continue;
                    }
                }
                if constexpr (WIDE) {
                    // two independent 256-column halves, four slabs of each per warp: all units of half 0 first
                    // (then its accumulator goes back), two of half 1, and the last two of half 1 into the
                    // registers of the first two finished slabs (then the second accumulator goes back)
                    const uint32_t t_h0 = t_row + uint32_t(slab0 * 32), t_h1 = t_h0 + uint32_t(TILE_N);
                    uint32_t hb[2][4][32];
                    uint64_t y2[16];
#pragma unroll
                    for (int sl = 0; sl < 4; sl++) tc_ld32(t_h0 + uint32_t(sl * 32), hb[0][sl]);
                    tc_wait_ld();
                    release(0);
                    tc_ld32(t_h1, hb[1][0]);
                    tc_ld32(t_h1 + 32u, hb[1][1]);
#pragma unroll
                    for (int u = 0; u < 8; u++) {
                        const int h = u >> 2, sl = u & 3;
                        const int c0 = h * TILE_N + (slab0 + sl) * 32, nf = n0 + c0;
                        const int q = seg_of_column(min(nf, prm.N - 1), Q, nb_addr, lane);
                        const TokenScale tk = token_scale(0, row);
                        scale_add_unit<KIND, false, true, PT>(y2, hb[h][sl], 0, Q, q, q, nf, tab_addr, nb_addr,
                                                              bias_addr + uint32_t(c0) * 4u, &tk);
                        store_slab<GENERIC>(y2, prm, row, nf, yo);
                        if (u == 1) {
                            tc_ld32(t_h1 + 64u, hb[1][2]);
                            tc_ld32(t_h1 + 96u, hb[1][3]);
                            tc_wait_ld();
                            release(1);
                        }
                    }
                    continue;
                }
                if constexpr (kSplitRel && !WIDE) {
                    // four slabs per warp: all positive units first (then the positive accumulator goes back),
                    // negative units as registers come free (then the negative one); five units live at most
                    static_assert(!kSplitRel || kSlabsPerWarp == 4, "split release: 256-wide tile, 8 epilogue warps");
                    const uint32_t t_pos = t_row + uint32_t(slab0 * 32), t_neg = t_pos + uint32_t(TILE_N);
                    uint32_t pb[4][32], nbuf[4][32];
                    uint64_t y2[16];
#pragma unroll
                    for (int sl = 0; sl < 4; sl++) tc_ld32(t_pos + uint32_t(sl * 32), pb[sl]);
                    tc_wait_ld();
                    release(0);
                    tc_ld32(t_neg, nbuf[0]);
                    tc_ld32(t_neg + 32u, nbuf[1]);
#pragma unroll
                    for (int sl = 0; sl < 4; sl++) {
                        const int c0 = (slab0 + sl) * 32, nf = n0 + c0;
                        const int q = seg_of_column(nf, Q, nb_addr, lane);
                        const TokenScale tk0 = token_scale(0, row), tk1 = token_scale(1, row);
                        scale_add_unit<KIND, false, true, PT>(y2, pb[sl], 0, Q, q, q, nf, tab_addr, nb_addr,
                                                              bias_addr + uint32_t(c0) * 4u, &tk0);
                        if (sl == 0) tc_wait_ld();
                        scale_add_unit<KIND, false, false, PT>(y2, nbuf[sl], 1, Q, q, q, nf, tab_addr, nb_addr, 0, &tk1);
                        store_slab<GENERIC>(y2, prm, row, nf, yo);
                        if (sl == 0) {                        // registers of slab 0 are free: the last two negative units
                            tc_ld32(t_neg + 64u, nbuf[2]);
                            tc_ld32(t_neg + 96u, nbuf[3]);
                            tc_wait_ld();
                            release(1);
                        }
                    }
                    continue;
                }
                if (kEvenSplit && nacc == NPOL) {
                    // one K-segment (the usual case): the unit count is a compile-time constant, outputs slab by slab
                    constexpr int kUnits = kSlabsPerWarp * NPOL;
                    constexpr int kBufMax = GENERIC ? 2 : kResidentBufs;
                    constexpr int NB = kUnits < kBufMax ? kUnits : kBufMax;
                    constexpr int kRel = kUnits <= NB ? 0 : kUnits - NB;
                    static_assert(NB >= 2 || kUnits == 1, "needs two load buffers");
                    const uint32_t t_warp = t_row + uint32_t(slab0 * 32);
                    uint32_t buf[NB][32];
#pragma unroll
                    for (int u = 0; u < NB; u++) tc_ld32(t_warp + uint32_t((u % NPOL) * TILE_N + (u / NPOL) * 32), buf[u]);
                    uint64_t y2[16];
                    int q_lo = 0, q_hi = 0;
#pragma unroll
                    for (int u = 0; u < kUnits; u++) {
                        const int sl = u / NPOL, pol = u % NPOL;
                        const int c0 = (slab0 + sl) * 32, nf = n0 + c0;
                        const bool refill = u >= 1 && u - 1 + NB < kUnits;
                        const bool last_load = u - 1 + NB == kUnits - 1;
                        if (refill && last_load)
                            tc_ld32(t_warp + uint32_t(((u - 1 + NB) % NPOL) * TILE_N + ((u - 1 + NB) / NPOL) * 32),
                                    buf[(u - 1) % NB]);
                        tc_wait_ld();
                        if (u == kRel) release(cur_as);
                        if (refill && !last_load)
                            tc_ld32(t_warp + uint32_t(((u - 1 + NB) % NPOL) * TILE_N + ((u - 1 + NB) / NPOL) * 32),
                                    buf[(u - 1) % NB]);
                        if (pol == 0) {
                            q_lo = seg_of_column(nf, Q, nb_addr, lane);
                            q_hi = GENERIC ? seg_of_column(min(nf + 31, prm.N - 1), Q, nb_addr, lane) : q_lo;
                            const TokenScale tk = token_scale(pol, row);
                            scale_add_unit<KIND, GENERIC, true, PT>(y2, buf[u % NB], pol, Q, q_lo, q_hi, nf, tab_addr, nb_addr,
                                                                    bias_addr + uint32_t(c0) * 4u, &tk);
                        } else {
                            const TokenScale tk = token_scale(pol, row);
                            scale_add_unit<KIND, GENERIC, false, PT>(y2, buf[u % NB], pol, Q, q_lo, q_hi, nf, tab_addr, nb_addr, 0, &tk);
                        }
                        if (GENERIC && prm.acc_dump && row < prm.M)
                            dump_unit(prm.acc_dump, buf[u % NB], pol, row, nf, prm.M, prm.N);
                        if (pol == NPOL - 1 && (!GENERIC || row < prm.M)) store_slab<GENERIC>(y2, prm, row, nf, yo);
                    }
                    continue;
                }
                // several K-segments kept resident, or a tile narrower than the warps' column split: the unit
                // count is a run-time value; loads run one unit ahead of the arithmetic
                const int my_slabs = max(0, min(kSlabsPerWarp, kSlabs - slab0));
                const int units = my_slabs * nacc;                          // (slab, accumulator) pairs of this warp

                uint64_t y2[16];
                uint32_t ra[32], rb[32];
                int i_sl = 0, i_a = 0;              // next unit to load
                int c_sl = 0, c_a = 0;              // next unit to consume
                int q_lo = 0, q_hi = 0;             // N-segments of the first and last column of the slab
                auto issue = [&](uint32_t (&r)[32]) {
                    tc_ld32(t_row + uint32_t(i_a * TILE_N + (slab0 + i_sl) * 32), r);
                    if (++i_a == nacc) { i_a = 0; i_sl++; }
                };
                auto consume = [&](const uint32_t (&r)[32]) {
                    const int c0 = (slab0 + c_sl) * 32;
                    const int nf = n0 + c0;                          // first column of the slab
                    if (c_a == 0) {
                        q_lo = seg_of_column(nf, Q, nb_addr, lane);
                        q_hi = GENERIC ? seg_of_column(min(nf + 31, prm.N - 1), Q, nb_addr, lane) : q_lo;
#pragma unroll
                        for (int j4 = 0; j4 < 8; j4++)
                            ld_shared_2x64(bias_addr + uint32_t(c0 + 4 * j4) * 4u, y2[2 * j4], y2[2 * j4 + 1]);
                    }
                    const TokenScale tk = token_scale(c_a, row);
                    scale_add_unit<KIND, GENERIC, false, PT>(y2, r, c_a, Q, q_lo, q_hi, nf, tab_addr, nb_addr, 0, &tk);
                    if (GENERIC && prm.acc_dump && row < prm.M) dump_unit(prm.acc_dump, r, c_a, row, nf, prm.M, prm.N);
                    if (++c_a < nacc) return;
                    c_a = 0;
                    c_sl++;
                    if (!GENERIC || row < prm.M) store_slab<GENERIC>(y2, prm, row, nf, yo);   // last accumulator of the slab
                };
                if (units == 0) {
                    release(cur_as);
                } else {
                    issue(ra);
#pragma unroll 1
                    for (int u = 0; u < units; u += 2) {
                        tc_wait_ld();
                        if (u + 1 < units) issue(rb); else release(cur_as);
                        consume(ra);
                        if (u + 1 < units) {
                            tc_wait_ld();
                            if (u + 2 < units) issue(ra); else release(cur_as);
                            consume(rb);
                        }
                    }
                }
            }
        }
        if (!GENERIC) tma_store_drain(yo);          // the staging buffers are read before the CTA may exit
    }

    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();                // neither CTA leaves while the other may still signal it
    if (warp == 1) {
        tc_fence_after();
        if (CG == 1)
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(uint32_t(kTmemCols)) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(uint32_t(kTmemCols)) : "memory");
    }
}

// ----------------------------------------------------------------------------- host side

using EncodeFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                              const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up once per process.
EncodeFn get_encode_fn()
{
    static std::once_flag once;
    static EncodeFn fn = nullptr;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeFn>(p);
    });
    return fn;
}

// 2-D map over a row-major byte matrix [rows, cols] with row pitch ld: box = 128 bytes x box_rows,
// 128B swizzle, out-of-range elements read as zero.
bool make_map(CUtensorMap *map, const void *base, int64_t rows, int64_t cols, int64_t ld, int box_rows)
{
    EncodeFn enc = get_encode_fn();
    if (!enc) return false;
    cuuint64_t dims[2] = {cuuint64_t(cols), cuuint64_t(rows)};
    cuuint64_t strides[1] = {cuuint64_t(ld)};
    cuuint32_t box[2] = {cuuint32_t(BLOCK_K), cuuint32_t(box_rows)};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// 2-D map over the bf16 output [M, N] with row pitch ldy (elements): box = 32 columns x 32 rows, 64-byte
// swizzle (the layout tma_store_block writes).  Needs a 16-byte aligned base and pitch.
bool make_map_y(CUtensorMap *map, void *base, int64_t M, int64_t N, int64_t ldy)
{
    EncodeFn enc = get_encode_fn();
    if (!enc) return false;
    cuuint64_t dims[2] = {cuuint64_t(N), cuuint64_t(M)};
    cuuint64_t strides[1] = {cuuint64_t(ldy) * 2};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Tile-plan overrides for benchmarking sweeps and tests (segquant_set_tuning); 0 = automatic.
std::atomic<int> g_tune_tile_n{0}, g_tune_stages{0}, g_tune_cta_group{0}, g_tune_seq{0};

// What has been found out per (device, kernel instantiation, dynamic shared-memory size): how many CTA pairs can
// be resident; and per (device, kernel instantiation) the largest dynamic shared-memory size the kernel's
// attribute has been raised to (it is only ever raised, so that earlier plans stay launchable).  Guarded by a
// mutex; a handful of entries.
struct KernelFacts { int device; const void *kernel; size_t smem; int clusters; };
struct KernelSmem { int device; const void *kernel; size_t max_smem; };
std::mutex g_facts_mu;
std::vector<KernelFacts> g_facts;
std::vector<KernelSmem> g_smem;

template <typename Kern>
sq_status kernel_facts(int device, Kern kern, size_t smem, int cg, const cudaLaunchConfig_t &cfg, int *clusters)
{
    const void *key = reinterpret_cast<const void *>(kern);
    std::lock_guard<std::mutex> lock(g_facts_mu);
    KernelSmem *ks = nullptr;
    for (KernelSmem &e : g_smem)
        if (e.device == device && e.kernel == key) ks = &e;
    if (!ks || ks->max_smem < smem) {
        const cudaError_t ea = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (ea != cudaSuccess) { note_cuda_error(ea); return SQ_ERR_CUDA; }
        if (ks) ks->max_smem = smem;
        else g_smem.push_back({device, key, smem});
    }
    for (const KernelFacts &f : g_facts)
        if (f.device == device && f.kernel == key && f.smem == smem) { *clusters = f.clusters; return SQ_OK; }
    int n = 0;
    if (cg == 2) {
        const cudaError_t eo = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (eo != cudaSuccess || n <= 0) { note_cuda_error(eo != cudaSuccess ? eo : cudaErrorLaunchOutOfResources); return SQ_ERR_CUDA; }
    }
    g_facts.push_back({device, key, smem, n});
    *clusters = n;
    return SQ_OK;
}

// Split tiles hold 256 accumulator columns per CTA (two sets fit in TMEM, and a CTA's partial sums are 128 KiB):
// 256-column tiles for single-scale layers, 128-column tiles for dual ones.  (256-column dual tiles were measured
// too: twice the partial sums to exchange, one accumulator set, slower on every shape tried.)
constexpr int sk_tile_n(int npol) { return npol == 2 ? 128 : 256; }
constexpr size_t kSkSlotBytes = size_t(TILE_M) * 256 * 4;                  // one CTA's accumulators of such a tile
inline size_t sk_counter_bytes(int64_t tiles) { return size_t((tiles * 2 * 4 + 255) / 256 * 256); }

template <int KIND, int NPOL, int TILE_N, int CG, bool GENERIC, bool SEQ, bool WIDE = false, bool PT = false, bool SK = false>
sq_status prepare_variant(const GemmArgs &g, GemmLaunch &L, int device, int sm_count)
{
    constexpr int kTileCols = TILE_N * (WIDE ? 2 : 1);
    constexpr int B_ROWS = TILE_N / CG;
    KernelParams &prm = L.prm;
    if (GENERIC) L.ty = CUtensorMap{};                // unused by the generic variant
    else if (!make_map_y(&L.ty, g.Y, g.M, g.N, g.ldy)) return SQ_ERR_CUDA;
    if (!make_map(&L.ta, g.a_pos, g.M, g.K, g.lda, TILE_M)) return SQ_ERR_CUDA;
    if (!make_map(&L.tn, g.a_neg ? g.a_neg : g.a_pos, g.M, g.K, g.lda, TILE_M)) return SQ_ERR_CUDA;
    if (!make_map(&L.tb, g.b, g.N, g.K, g.ldb, B_ROWS)) return SQ_ERR_CUDA;

    const uint32_t stage_bytes = NPOL * TILE_M * BLOCK_K + (WIDE ? 2 : 1) * B_ROWS * BLOCK_K;
    // per-token mode: the tile's channel scales are staged in shared memory when there are few K-segments
    prm.col_tab_bytes = ((GENERIC || PT) && prm.col_scale && prm.sb.P <= kMaxTokenSegments) ? uint32_t(prm.sb.P) * kTileCols * 4u : 0u;
    const uint32_t tail = (GENERIC ? 0u : kStageBytes) + epi_table_bytes(prm.nacc, prm.sb.Q, kTileCols) + prm.col_tab_bytes +
                          sizeof(SharedHeader);
    int stages = int((kSmemBudget - 1024 - tail) / stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    const int tune_stages = g_tune_stages.load(std::memory_order_relaxed);
    if (tune_stages >= 2 && tune_stages < stages) stages = tune_stages;
    if (stages < 2) return SQ_ERR_UNSUPPORTED;
    prm.stages = stages;
    prm.num_m_tiles = int((g.M + TILE_M * CG - 1) / (TILE_M * CG));
    prm.num_n_tiles = int((g.N + kTileCols - 1) / kTileCols);
    const size_t smem = 1024 + size_t(stages) * stage_bytes + tail;

    auto kern = segquant_gemm_kernel<KIND, NPOL, TILE_N, CG, GENERIC, SEQ, WIDE, PT, SK>;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(sm_count / CG * CG));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = CG == 2 ? 1 : 0;

    // persistent grid: one CTA (pair) per SM (pair) that can be resident at the same time
    int units = sm_count / CG, clusters = 0;
    const sq_status fs = kernel_facts(device, kern, smem, CG, cfg, &clusters);
    if (fs != SQ_OK) return fs;
    if (CG == 2 && clusters < units) units = clusters;
    const int tiles = prm.num_m_tiles * prm.num_n_tiles;
    L.kernel = reinterpret_cast<const void *>(kern);
    L.grid = unsigned((tiles < units ? tiles : units) * CG);
    if (SK) {
        // every pair gets the same share of all (tile, K-block) units; two slots per pair and CTA for its partial
        // segments, one counter per tile and CTA of the pair
        static_assert(!SK || size_t(NPOL) * TILE_M * TILE_N * 4 == kSkSlotBytes, "slot size");
        const int64_t kblocks = (g.K + BLOCK_K - 1) / BLOCK_K, total = int64_t(tiles) * kblocks;
        if (total > 0x3FFFFFFF) return SQ_ERR_UNSUPPORTED;
        const int pairs = int(total < units ? total : units);
        const size_t need = sk_counter_bytes(tiles) + size_t(pairs) * 4 * kSkSlotBytes;
        if (!g.sk_scratch || g.sk_bytes < need) return SQ_ERR_WORKSPACE;
        prm.sk_counters = static_cast<uint32_t *>(g.sk_scratch);
        prm.sk_slots = static_cast<uint8_t *>(g.sk_scratch) + sk_counter_bytes(tiles);
        prm.sk_kblocks = int(kblocks);
        L.grid = unsigned(pairs * CG);
    }
    L.cluster = CG;
    L.smem = smem;
    L.device = device;
    return SQ_OK;
}

template <int KIND, int NPOL, int CG>
sq_status prepare_tile(const GemmArgs &g, GemmLaunch &L, int tile_n, bool seq, int device, int sm_count)
{
    KernelParams &prm = L.prm;
    bool dbg = prm.y_is_f32 || prm.acc_dump != nullptr;
    // the production variant writes Y with TMA stores: 16-byte aligned base and row pitch
    dbg = dbg || reinterpret_cast<uintptr_t>(g.Y) % 16 != 0 || (size_t(g.ldy) * 2) % 16 != 0;
    for (int q = 1; q < prm.sb.Q; q++) dbg = dbg || (prm.sb.nb[q] % 32 != 0);
    // per-token x per-channel scales: the production variant stages a tile's channel scales in shared memory, which
    // it does for up to 32 K-segments, int8 codes and CTA pairs; anything else runs the checking variant
    const bool pt = prm.col_scale != nullptr;
    if (pt && !(KIND == 0 && CG == 2 && prm.sb.P <= kMaxTokenSegments)) dbg = true;
    if (seq) {      // sequential K-segments: one tile width per polarity count
        constexpr int TN = NPOL == 1 ? 256 : 128;
        if (dbg) return prepare_variant<KIND, NPOL, TN, CG, true, true>(g, L, device, sm_count);
        if constexpr (KIND == 0 && CG == 2)
            if (pt) return prepare_variant<KIND, NPOL, TN, CG, false, true, false, true>(g, L, device, sm_count);
        return prepare_variant<KIND, NPOL, TN, CG, false, true>(g, L, device, sm_count);
    }
    if constexpr (KIND == 0 && CG == 2) {
        if (pt && !dbg) {     // 256- and 128-column tiles only (the automatic choice never goes below for these layers)
            if constexpr (NPOL == 1) {      // single-scale, one K-segment: 256 x 512 tiles under the rule given further down
                const int tune = g_tune_seq.load(std::memory_order_relaxed);
                const int64_t n256w = (g.N + 255) / 256, mp = (g.M + 2 * TILE_M - 1) / (2 * TILE_M), un = sm_count / 2;
                const int64_t w256 = (mp * n256w + un - 1) / un, wwide = (mp * ((n256w + 1) / 2) + un - 1) / un;
                if (tile_n == 256 && prm.sb.P == 1 && tune != 4 && (n256w % 2 == 0 || n256w >= 9) &&
                    (tune == 5 || 2 * wwide * 94 < w256 * 100)) {
                    prm.acc_stages = 1;
                    return prepare_variant<KIND, 1, 256, 2, false, false, true, true>(g, L, device, sm_count);
                }
            }
            if (tile_n == 256) return prepare_variant<KIND, NPOL, 256, CG, false, false, false, true>(g, L, device, sm_count);
            if (tile_n == 128) return prepare_variant<KIND, NPOL, 128, CG, false, false, false, true>(g, L, device, sm_count);
            dbg = true;
        }
    }
    // single-scale layer, one K-segment, CTA pairs, at least two 256-column tiles: 256 x 512 tiles whose halves
    // share the activation tile; an odd number of 256-column tiles leaves one half idle, so then only when there
    // are many of them; and a wide tile is two tiles' work, so it must not cost more waves than it saves time
    // (measured gain per unit of work: 5-6 %)
    const int tune_seq = g_tune_seq.load(std::memory_order_relaxed);
    const int64_t n256 = (g.N + 255) / 256, m_pairs = (g.M + 2 * TILE_M - 1) / (2 * TILE_M), units = sm_count / 2;
    const int64_t waves_256 = (m_pairs * n256 + units - 1) / units;
    const int64_t waves_wide = (m_pairs * ((n256 + 1) / 2) + units - 1) / units;
    const bool wide = NPOL == 1 && CG == 2 && !dbg && tile_n == 256 && prm.sb.P == 1 && tune_seq != 4 &&
                      (n256 % 2 == 0 || n256 >= 9) && (tune_seq == 5 || 2 * waves_wide * 94 < waves_256 * 100);
    // Split tiles: one K-segment, CTA pairs, production output, and a tile count that leaves a good part of the
    // last wave idle.  Time in K-blocks of 256 accumulator columns: whole tiles take waves x K-blocks; split
    // tiles take their even share plus the exchange of partial sums (a fixed part and one slot read per pair
    // that shares a tile, in K-block times; measured).  segment_mode 6 forces the split where it is possible, 7 forbids it.
    if constexpr (CG == 2) {
        if (!dbg && !pt && prm.sb.P == 1 && g.sk_scratch && tune_seq != 7) {
            constexpr int TN = sk_tile_n(NPOL);
            constexpr double kSkFixup = 30.0, kSkPerSharer = 10.0;
            const int64_t pairs = sm_count / 2, m_tiles = (g.M + 2 * TILE_M - 1) / (2 * TILE_M);
            const int64_t kblocks = (g.K + BLOCK_K - 1) / BLOCK_K;
            const int64_t tiles_sk = m_tiles * ((g.N + TN - 1) / TN), tiles_dp = m_tiles * ((g.N + tile_n - 1) / tile_n);
            double t_dp = double((tiles_dp + pairs - 1) / pairs) * double(kblocks) * (double(tile_n * NPOL) / 256.0);
            if (wide) t_dp = double(2 * waves_wide) * 0.94 * double(kblocks);
            // the CTA that completes a tile reads one slot per pair that worked on it
            const double sharers = double(pairs) / double(tiles_sk) + 1.0;
            const double t_sk = double(tiles_sk * kblocks) / double(pairs) + kSkFixup + kSkPerSharer * (sharers < 2.0 ? 2.0 : sharers);
            const size_t need = sk_counter_bytes(tiles_sk) + size_t(pairs) * 4 * kSkSlotBytes;
            if (g.sk_bytes >= need && tiles_sk * kblocks >= 2 && (tune_seq == 6 || t_sk < 0.9 * t_dp)) {
                prm.acc_stages = 2;
                return prepare_variant<KIND, NPOL, TN, 2, false, false, false, false, true>(g, L, device, sm_count);
            }
        }
    }
    if (wide) {
        prm.acc_stages = 1;
        return prepare_variant<KIND, 1, 256, 2, false, false, true>(g, L, device, sm_count);
    }
    switch (tile_n) {
        case 256: return dbg ? prepare_variant<KIND, NPOL, 256, CG, true, false>(g, L, device, sm_count)
                             : prepare_variant<KIND, NPOL, 256, CG, false, false>(g, L, device, sm_count);
        case 128: return dbg ? prepare_variant<KIND, NPOL, 128, CG, true, false>(g, L, device, sm_count)
                             : prepare_variant<KIND, NPOL, 128, CG, false, false>(g, L, device, sm_count);
        case 64: return dbg ? prepare_variant<KIND, NPOL, 64, CG, true, false>(g, L, device, sm_count)
                            : prepare_variant<KIND, NPOL, 64, CG, false, false>(g, L, device, sm_count);
        case 32: return dbg ? prepare_variant<KIND, NPOL, 32, CG, true, false>(g, L, device, sm_count)
                            : prepare_variant<KIND, NPOL, 32, CG, false, false>(g, L, device, sm_count);
    }
    return SQ_ERR_UNSUPPORTED;
}

template <int KIND>
sq_status prepare_kind(const GemmArgs &g, GemmLaunch &L, int npol, int cg, int tile_n, bool seq, int device, int sm_count)
{
    if (npol == 2)
        return cg == 2 ? prepare_tile<KIND, 2, 2>(g, L, tile_n, seq, device, sm_count)
                       : prepare_tile<KIND, 2, 1>(g, L, tile_n, seq, device, sm_count);
    return cg == 2 ? prepare_tile<KIND, 1, 2>(g, L, tile_n, seq, device, sm_count)
                   : prepare_tile<KIND, 1, 1>(g, L, tile_n, seq, device, sm_count);
}

}  // namespace

size_t gemm_split_scratch_bytes(int64_t M, int64_t N, int dual)
{
    int dev = 0, sm_count = 0;
    if (M <= 0 || N <= 0 || cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count < 2)
        return 0;
    const int64_t tiles = ((M + 2 * TILE_M - 1) / (2 * TILE_M)) * ((N + sk_tile_n(dual ? 2 : 1) - 1) / sk_tile_n(dual ? 2 : 1));
    return sk_counter_bytes(tiles) + size_t(sm_count / 2) * 4 * kSkSlotBytes;
}

void set_gemm_tuning(int tile_n, int stages, int cta_group, int segment_mode)
{
    g_tune_tile_n.store(tile_n, std::memory_order_relaxed);
    g_tune_stages.store(stages, std::memory_order_relaxed);
    g_tune_cta_group.store(cta_group, std::memory_order_relaxed);
    g_tune_seq.store(segment_mode, std::memory_order_relaxed);
}

// Everything a GEMM launch needs that can be worked out ahead of it: tile plan, kernel instantiation, tensor
// maps, shared-memory size and grid.  Launches nothing.
sq_status prepare_gemm(const GemmArgs &g, GemmLaunch *out)
{
    GemmLaunch &L = *out;
    KernelParams &prm = L.prm;
    prm = KernelParams{};
    prm.M = int(g.M); prm.N = int(g.N); prm.K = int(g.K);
    const int npol = g.a_neg ? 2 : 1;
    prm.nacc = g.sb.P * npol;
    prm.sb = g.sb;
    prm.s_pos = g.s_pos; prm.s_neg = g.s_neg; prm.s_w = g.s_w; prm.bias = g.bias;
    prm.row_pos = g.row_pos; prm.row_neg = g.row_neg; prm.col_scale = g.col_scale;
    prm.Y = g.Y; prm.ldy = g.ldy;
    prm.y_is_f32 = g.y_dtype == SQ_F32;
    prm.y_wide = (reinterpret_cast<uintptr_t>(g.Y) % 32 == 0) && ((size_t(g.ldy) * (prm.y_is_f32 ? 4 : 2)) % 32 == 0);
    prm.acc_dump = g.acc_dump;
    prm.status = g.status;

    int dev = 0, sm_count = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SQ_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count <= 0)
        return SQ_ERR_CUDA;
    const int tune_tile_n = g_tune_tile_n.load(std::memory_order_relaxed);
    const int tune_cta_group = g_tune_cta_group.load(std::memory_order_relaxed);
    const int tune_seq = g_tune_seq.load(std::memory_order_relaxed);

    // CTA pairs whenever a tile has more than 128 rows to work on
    int cg = g.M > TILE_M ? 2 : 1;
    if (tune_cta_group == 1 || tune_cta_group == 2) cg = tune_cta_group;
    if (sm_count < 2) cg = 1;

    // More than one K-segment: segments go through TMEM one after the other (SEQ) unless the caller asks for
    // all accumulators of a tile to stay resident, which needs 32 columns for each of them.
    bool seq = g.sb.P > 1;
    if (tune_seq == 1 && prm.nacc * 32 <= kTmemCols) seq = false;
    if (tune_seq == 2) seq = true;
    if (prm.nacc * g.sb.Q > kMaxFactorTable) return SQ_ERR_UNSUPPORTED;
    if (seq) {
        prm.acc_stages = 2;
        return g.code == SQ_CODE_INT8 ? prepare_kind<0>(g, L, npol, cg, 0, true, dev, sm_count)
                                      : prepare_kind<1>(g, L, npol, cg, 0, true, dev, sm_count);
    }

    // Tile width: the widest tile whose accumulators fit the 512 TMEM columns, unless half that width
    // fills the machine so much better that it outweighs the narrower tile's higher operand traffic
    // per MMA (weights 1 : 0.75; a double-buffered accumulator set counts 10 % extra).
    int tile_max = 256;
    while (tile_max * prm.nacc > kTmemCols) tile_max >>= 1;
    if (tile_max < 32) return SQ_ERR_UNSUPPORTED;
    int tile_n = tile_max;
    if (tile_max >= 128) {
        const int64_t units = sm_count / cg;
        auto score = [&](int tn, double weight) {
            const int64_t tiles = ((g.M + TILE_M * cg - 1) / (TILE_M * cg)) * ((g.N + tn - 1) / tn);
            const int64_t waves = (tiles + units - 1) / units;
            const double dbuf = (2 * tn * prm.nacc <= kTmemCols) ? 1.1 : 1.0;
            return weight * dbuf * double(tiles) / double(waves * units);
        };
        if (score(tile_max / 2, 0.75) > score(tile_max, 1.0)) tile_n = tile_max / 2;
    }
    // per-(token, channel) factors run in the checking variant, whose epilogue releases a full-TMEM accumulator set
    // only at its end: keep two sets so that it overlaps the next tile's main loop
    const bool pt_generic = g.col_scale && (prm.y_is_f32 || prm.acc_dump || g.code != SQ_CODE_INT8 || cg != 2 || g.sb.P > kMaxTokenSegments);
    if (pt_generic && 2 * tile_n * prm.nacc > kTmemCols && tile_n >= 64) tile_n >>= 1;
    if (tune_tile_n >= 32 && tune_tile_n <= tile_max && (tune_tile_n & (tune_tile_n - 1)) == 0)
        tile_n = tune_tile_n;
    prm.acc_stages = (2 * tile_n * prm.nacc <= kTmemCols) ? 2 : 1;

    return g.code == SQ_CODE_INT8 ? prepare_kind<0>(g, L, npol, cg, tile_n, false, dev, sm_count)
                                  : prepare_kind<1>(g, L, npol, cg, tile_n, false, dev, sm_count);
}

// One launch from a prepared plan: no queries, no encoding.
sq_status run_gemm(const GemmLaunch &L, cudaStream_t st)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(L.grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = L.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = L.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = L.cluster == 2 ? attr : attr + 1;          // the cluster attribute only for CTA pairs
    cfg.numAttrs = L.cluster == 2 ? 2 : 1;
    void *args[5] = {const_cast<CUtensorMap *>(&L.ta), const_cast<CUtensorMap *>(&L.tn), const_cast<CUtensorMap *>(&L.tb),
                     const_cast<CUtensorMap *>(&L.ty), const_cast<KernelParams *>(&L.prm)};
    const cudaError_t e = cudaLaunchKernelExC(&cfg, L.kernel, args);
    count_launch();
    if (e != cudaSuccess) { note_cuda_error(e); return SQ_ERR_CUDA; }
    return SQ_OK;
}

sq_status launch_gemm(const GemmArgs &g, cudaStream_t st)
{
    GemmLaunch L;
    const sq_status s = prepare_gemm(g, &L);
    return s == SQ_OK ? run_gemm(L, st) : s;
}

}  // namespace sq
