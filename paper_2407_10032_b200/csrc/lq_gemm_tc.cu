// bf16 x bf16 -> fp32 (or 8-bit integer x 8-bit integer -> int32) "NT" GEMM on the sm_100a tensor cores.
//
//   D[M x N] (+)= alpha * sum_p A_p[M x K] * B_p[N x K]^T        (all row-major, K contiguous)
//
// Used by stage 1 (H += 2 X X^T, Algorithm 1 line 3) and by the lazy trailing update of
// the column loop (Algorithm 1 line 20).  fp32 operands are fed as several bf16 passes
// (hi/mid/lo terms), which is what n_pass > 1 is for.
//
// One persistent CTA per SM, K consumed 64 at a time; K may be cut into a few parts so that the
// schedule's last round is short (see next_piece).  Two forms of the same kernel:
//   CTAS = 1 : one CTA computes a 128 x 256 tile (tcgen05 cta_group::1);
//   CTAS = 2 : a cluster of two CTAs computes a 256 x 256 tile with the two-SM MMA form
//              (cta_group::2): each CTA loads its own 128 rows of A and only its half of B, so
//              the shared-memory traffic per flop drops by a third; the even CTA of the pair
//              issues the MMAs for both, each CTA drains its own 128 x 256 accumulator.
//   warp 0      : TMA producer (cp.async.bulk.tensor, 128-byte swizzle, ring of stages)
//   warp 1      : issues tcgen05.mma (one thread), accumulators in TMEM (2 x 256 columns,
//                 so the epilogue of one segment overlaps the main loop of the next); in the
//                 odd CTA of a pair it idles (both CTAs' loads complete on the even CTA's barrier)
//   warps 2..9  : epilogue.  The tensor core adds into its fp32 accumulator with truncation,
//                 which over a long K biases every sum low; so K is consumed in short
//                 segments, and after each one these warps tcgen05.ld the partial sum and
//                 add it (round-to-nearest) to running sums held in registers.  After the
//                 piece's last segment: scale -> swizzled smem slab -> TMA store, or a TMA
//                 reduce-add when accumulating into D (no read of D by the SM).
// With 8-bit integer operands (the digit slices of stage 2's deferred updates) the same pipeline runs tcgen05.mma
// kind::i8: a k-step is still 128 bytes (128 digits instead of 64 bf16), the accumulator holds int32 sums, which
// are exact, and the epilogue converts each partial sum to fp32 and scales it by its level's power of two.
// Every wait on an mbarrier is bounded: when the time limit passes the CTA records
// LQ_ERR_TIMEOUT in the handle's status word, stops issuing work and leaves.
#include <cuda.h>

#include "lq_common.cuh"

namespace {

constexpr int BM = 128;                // rows of A (and of the accumulator) per CTA
constexpr int BN = 256;                // tile width
constexpr int BK = 64;                 // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int EPI_COLS = 32;           // 32 fp32 = 128 bytes = one swizzle row
constexpr int EPI_BUF_BYTES = BM * EPI_COLS * 4;
constexpr int EPI_BUFS = 2;
constexpr int NUM_THREADS = 320;
constexpr int TMEM_COLS = 512;
constexpr int MAX_STAGES = 6;

template <int CTAS> struct Cfg {
    static constexpr int B_ROWS = BN / CTAS;                     // rows of B a CTA loads
    static constexpr int B_STAGE_BYTES = B_ROWS * BK * 2;
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    static constexpr int STAGES = CTAS == 1 ? 4 : 6;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BUFS * EPI_BUF_BYTES + 1024;
    static constexpr int TILE_M = BM * CTAS;
    // Instruction descriptor: D fp32, A and B bf16, both K-major, M = TILE_M, N = 256.
    static constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(BN >> 3) << 17) | (uint32_t(TILE_M >> 4) << 24);
    // The same for kind::i8: D int32 (2 in bits 4-5), A and B unsigned (0) or signed (1) 8-bit integers in bits 7-9 / 10-12.
    static constexpr uint32_t idesc_i8(bool a_signed, bool b_signed) {
        return (2u << 4) | ((a_signed ? 1u : 0u) << 7) | ((b_signed ? 1u : 0u) << 10) | (uint32_t(BN >> 3) << 17) |
               (uint32_t(TILE_M >> 4) << 24);
    }
};

struct KParams {
    int M, N, K;
    int n_pass;
    int a_off[LQ_TC_MAX_PASS];
    int b_off[LQ_TC_MAX_PASS];
    float alpha;
    int accumulate;
    int upper_only;
    int tile_m;               // rows of a tile: 128 or 256
    int tiles_m, tiles_n;
    int band;                 // tile rows per band of the schedule (see tile_coords)
    int num_tiles;
    int seg_iters;            // k-iterations accumulated in TMEM before the partial sum is flushed to D
    int segs_per_tile;        // ceil(k_iters / seg_iters), or n_lvl * n_chunks with levels
    // Level-major order (n_lvl > 0): the passes form groups ("levels"); a segment is one level over one chunk of
    // chunk_kb 64-wide k-blocks, and the segments run level by level.  See lq_tc_gemm_args::n_lvl.
    int n_lvl;
    int lvl_pass0[LQ_TC_MAX_LVL];
    int lvl_npass[LQ_TC_MAX_LVL];
    int chunk_kb;
    int n_chunks;
    int k_parts;              // K is cut into this many parts (<= segs_per_tile)
    long long total_units;    // num_tiles * k_parts work units, dealt round-robin to the CTAs (or CTA pairs)
    lq_dev_status* status;
    unsigned long long timeout_ns;
    int stall_bytes;          // test hook: bytes a load barrier expects on top of what its loads deliver (0 in normal use)
    // 8-bit integer operands: elements per 128-byte k-step, one instruction descriptor per pass (its operands may be
    // signed or unsigned), and the factor each level's int32 partial sums are scaled by on their way into the fp32 sum
    int int8_ops;
    int bk_elems;
    uint32_t idesc_pass[LQ_TC_MAX_PASS];
    float lvl_scale[LQ_TC_MAX_LVL];
    int first_out;            // the first level's sum is stored through the second output map and leaves the running sum
};

// ---------------------------------------------------------------- PTX wrappers ----
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long global_timer() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Arrive on the barrier at the same shared-memory offset in CTA `rank` of this cluster.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(bar), "r"(rank));
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          const KParams& p, int where) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer();
    uint32_t spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer() - t0 > p.timeout_ns) {
                *abort_flag = 1;
                lq_report(p.status, LQ_ERR_TIMEOUT, where);
                return false;
            }
        }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// The same load issued by either CTA of a pair, completing on a barrier given as a cluster address
// (the even CTA's): the two-CTA form of the instruction allows the barrier to live in the peer.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ uint32_t cluster_addr(uint32_t addr, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(addr), "r"(rank));
    return remote;
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N> __device__ __forceinline__ void bulk_wait() {
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
template <int CTAS> __device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    if (CTAS == 1) asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    else asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
template <int CTAS> __device__ __forceinline__ void tmem_relinquish() {
    if (CTAS == 1) asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    else asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
template <int CTAS> __device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    if (CTAS == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
template <int CTAS>
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t acc) {
    if (CTAS == 1)
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(acc) : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(acc) : "memory");
}
template <int CTAS>
__device__ __forceinline__ void umma_i8(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t acc) {
    if (CTAS == 1)
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(acc) : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(acc) : "memory");
}
// The barrier is signalled when all MMAs issued so far by this thread have completed; with two
// CTAs the signal goes to the barrier at this offset in both CTAs of the pair.
template <int CTAS> __device__ __forceinline__ void umma_commit(uint32_t bar) {
    if (CTAS == 1) {
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    } else {
        const uint16_t mask = 3;
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(bar), "h"(mask) : "memory");
    }
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void group_bar_sync(uint32_t id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }
// Barrier over the 128 threads of an epilogue group that also tells every thread whether any of them passed `v`.
__device__ __forceinline__ bool group_bar_or(uint32_t id, bool v) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %2, 0;\n\t"
        "bar.red.or.pred p, %1, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out) : "r"(id), "r"(static_cast<uint32_t>(v)) : "memory");
    return out != 0;
}

// Shared-memory matrix descriptor for a K-major bf16 tile stored by TMA with the 128-byte
// swizzle: rows of 128 bytes, groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t make_desc_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);       // start address / 16
    d |= static_cast<uint64_t>(1) << 16;                        // leading byte offset / 16 (fixed for swizzled K-major)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;                // stride byte offset / 16
    d |= static_cast<uint64_t>(1) << 46;                        // descriptor version of this architecture
    d |= static_cast<uint64_t>(2) << 61;                        // 128-byte swizzle
    return d;
}

// Map the idx-th scheduled tile to (tile row, tile column).  With upper_only, row tm keeps
// the columns tn with (tn + 1) * BN > tm * tile_m.  The tiles are ordered in bands of `band`
// tile rows, column by column inside a band: the CTAs of one scheduling round then work on a
// roughly square patch of the output and share a few panels of each operand through the L2
// (in plain row-major order a round shares one panel of A and reads as many panels of B as it
// has tiles, which makes wide symmetric products HBM-bound).
__device__ __forceinline__ void tile_coords(const KParams& p, int idx, int& tm, int& tn) {
    const int G = p.band;
    if (!p.upper_only) {
        const int per_band = G * p.tiles_n;
        const int m0 = (idx / per_band) * G;
        const int rows = (m0 + G < p.tiles_m) ? G : p.tiles_m - m0;      // the last band may be lower
        const int in_band = idx - (m0 / G) * per_band;
        tn = in_band / rows;
        tm = m0 + in_band - tn * rows;
        return;
    }
    for (int m0 = 0;; m0 += G) {
        const int m1 = (m0 + G < p.tiles_m) ? m0 + G : p.tiles_m;
        int band_cnt = 0;
        for (int m = m0; m < m1; ++m) {
            const int cnt = p.tiles_n - (m * p.tile_m) / BN;
            band_cnt += cnt > 0 ? cnt : 0;
        }
        if (idx >= band_cnt && m1 < p.tiles_m) { idx -= band_cnt; continue; }
        // inside the band: the first columns are met by some of its rows only (first column of a row never decreases)
        const int rows_all = m1 - m0;
        const int full_from = ((m1 - 1) * p.tile_m) / BN;            // from this column on every row of the band is present
        for (int c = (m0 * p.tile_m) / BN; c < full_from && c < p.tiles_n; ++c) {
            int rows = 0;
            for (int m = m0; m < m1; ++m) rows += ((m * p.tile_m) / BN <= c) ? 1 : 0;
            if (idx < rows) { tm = m0 + idx; tn = c; return; }
            idx -= rows;
        }
        tn = full_from + idx / rows_all;
        tm = m0 + idx % rows_all;
        return;
    }
}

// When the tile count is not a multiple of the CTA count, whole tiles leave some SMs idle in the
// last round.  K is therefore cut into k_parts equal parts and the launch's work becomes the
// list of (part, tile) units in part-major order, dealt round-robin to the CTAs (CTA pairs):
// rounds are 1 / k_parts of a tile long, so the idle tail shrinks with them, and at any moment
// all CTAs still read about the same columns of the operands (they share them through the L2).
// A unit leaves a partial sum over its part of K, which is fine because results are added into D.
struct Piece { int tile, s0, s1; };       // segments [s0, s1) of a tile
__device__ __forceinline__ bool next_piece(const KParams& p, long long& u, long long stride, Piece& pc) {
    if (u >= p.total_units) return false;
    const int part = static_cast<int>(u / p.num_tiles);
    pc.tile = static_cast<int>(u - static_cast<long long>(part) * p.num_tiles);
    pc.s0 = static_cast<int>(static_cast<long long>(p.segs_per_tile) * part / p.k_parts);
    pc.s1 = static_cast<int>(static_cast<long long>(p.segs_per_tile) * (part + 1) / p.k_parts);
    u += stride;
    return true;
}

// Segment s of a tile: how many (pass, k-block) items it has and which they are.
struct Seg { int len, kit0, pass0, kb0, kbn; };
__device__ __forceinline__ Seg seg_of(const KParams& p, int k_blocks, int k_iters, int s) {
    Seg g;
    if (p.n_lvl == 0) {
        g.kit0 = s * p.seg_iters;
        g.len = min(p.seg_iters, k_iters - g.kit0);
        g.pass0 = 0; g.kb0 = 0; g.kbn = k_blocks;
    } else {
        const int lvl = s / p.n_chunks, ch = s - lvl * p.n_chunks;
        g.kit0 = 0;
        g.pass0 = p.lvl_pass0[lvl];
        g.kb0 = ch * p.chunk_kb;
        g.kbn = min(p.chunk_kb, k_blocks - g.kb0);
        g.len = p.lvl_npass[lvl] * g.kbn;
    }
    return g;
}
__device__ __forceinline__ void seg_item(const Seg& g, int q, int& pass, int& kb) {
    const int kit = g.kit0 + q;
    const int ps = kit / g.kbn;
    pass = g.pass0 + ps;
    kb = g.kb0 + kit - ps * g.kbn;
}

// I8: the instantiation for 8-bit integer operands; the bf16 instantiation carries none of that code.
template <int CTAS, bool I8>
__global__ void __launch_bounds__(NUM_THREADS, 1)
lq_tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_d1,
                  const __grid_constant__ KParams p) {
    typedef Cfg<CTAS> C;
    constexpr int STAGES = C::STAGES;
    constexpr bool PAIR = CTAS == 2;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[3 * MAX_STAGES + 4];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t warp_idx = threadIdx.x >> 5;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;      // 0: issues the MMAs; 1: its peer
    const bool mma_cta = rank == 0;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t epi_base = smem_base + STAGES * C::STAGE_BYTES;
    uint8_t* epi_gen = smem_gen + STAGES * C::STAGE_BYTES;

    const uint32_t bar_full = smem_u32(&bars[0]);                      // the TMA loads of a stage have landed (pair: both CTAs', on the even CTA)
    const uint32_t bar_empty = smem_u32(&bars[MAX_STAGES]);            // the MMAs that read a stage have completed
    const uint32_t bar_tfull = smem_u32(&bars[3 * MAX_STAGES]);        // an accumulator holds a finished segment
    const uint32_t bar_tempty = smem_u32(&bars[3 * MAX_STAGES + 2]);   // (even CTA) an accumulator has been drained

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);
            mbar_init(bar_tempty + 8 * a, 8 * CTAS);          // one arrival per epilogue warp of the pair
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp_idx == 1) {
        tmem_alloc<CTAS>(smem_u32(&tmem_base_slot), TMEM_COLS);
        tmem_relinquish<CTAS>();
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();           // the peer's barriers are initialised before anything arrives on them
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_base_slot);
    volatile int* abortp = &abort_flag;

    const int k_blocks = (p.K + p.bk_elems - 1) / p.bk_elems;
    const int k_iters = k_blocks * p.n_pass;
    const long long u_begin = blockIdx.x / CTAS;
    const long long u_stride = gridDim.x / CTAS;

    if (warp_idx == 0) {
        // ------------------------------------------------------------ TMA producer
        uint32_t stage = 0, phase = 0;
        bool alive = true;
        long long u = u_begin;
        Piece pc;
        while (alive && next_piece(p, u, u_stride, pc)) {
            int tm, tn;
            tile_coords(p, pc.tile, tm, tn);
            const int m0 = tm * C::TILE_M + static_cast<int>(rank) * BM;
            const int n0 = tn * BN + static_cast<int>(rank) * C::B_ROWS;
            for (int sg = pc.s0; sg < pc.s1 && alive; ++sg) {
              const Seg g = seg_of(p, k_blocks, k_iters, sg);
              for (int q = 0; q < g.len; ++q) {
                if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abortp, p, 1)) { alive = false; break; }
                if (lane == 0) {
                    int pass, kb;
                    seg_item(g, q, pass, kb);
                    const int k0 = kb * p.bk_elems;
                    const uint32_t sa = smem_base + stage * C::STAGE_BYTES;
                    const uint32_t sb = sa + A_STAGE_BYTES;
                    if (!PAIR) {
                        mbar_arrive_expect_tx(bar_full + 8 * stage, C::STAGE_BYTES + p.stall_bytes);
                        tma_load_2d(sa, &map_a, bar_full + 8 * stage, k0, p.a_off[pass] + m0);
                        tma_load_2d(sb, &map_b, bar_full + 8 * stage, k0, p.b_off[pass] + n0);
                    } else {
                        // both CTAs' loads of a stage complete on the even CTA's barrier, which expects the bytes of both
                        if (mma_cta) mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * C::STAGE_BYTES + p.stall_bytes);
                        const uint32_t full0 = cluster_addr(bar_full + 8 * stage, 0);
                        tma_load_2d_pair(sa, &map_a, full0, k0, p.a_off[pass] + m0);
                        tma_load_2d_pair(sb, &map_b, full0, k0, p.b_off[pass] + n0);
                    }
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
              }
            }
        }
    } else if (warp_idx == 1 && mma_cta) {
        // ------------------------------------------------------------ MMA issuer
        uint32_t stage = 0, phase = 0;
        int it = 0;                                  // counts segments: one TMEM accumulator each
        bool alive = true;
        long long u = u_begin;
        Piece pc;
        while (alive && next_piece(p, u, u_stride, pc)) {
            for (int sg = pc.s0; sg < pc.s1 && alive; ++sg, ++it) {
                const Seg seg = seg_of(p, k_blocks, k_iters, sg);
                const int seg_len = seg.len;
                const uint32_t acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abortp, p, 2)) { alive = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + acc * BN;
                for (int q = 0; q < seg_len; ++q) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abortp, p, 3)) { alive = false; break; }
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t sa = smem_base + stage * C::STAGE_BYTES;
                        const uint64_t da = make_desc_sw128(sa);
                        const uint64_t db = make_desc_sw128(sa + A_STAGE_BYTES);
#pragma unroll
                        if (I8) {
                            int pass, kb;
                            seg_item(seg, q, pass, kb);
                            const uint32_t idesc = p.idesc_pass[pass];
#pragma unroll
                            for (int kk = 0; kk < BK / UMMA_K; ++kk)      // 32 digits = 32 bytes per instruction: the same +2
                                umma_i8<CTAS>(tmem_d, da + 2 * kk, db + 2 * kk, idesc, (q > 0 || kk > 0) ? 1u : 0u);
                        } else {
#pragma unroll
                            for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                                // advancing 16 bf16 = 32 bytes inside the swizzle row: +2 in the address field
                                umma_bf16<CTAS>(tmem_d, da + 2 * kk, db + 2 * kk, C::IDESC, (q > 0 || kk > 0) ? 1u : 0u);
                            }
                        }
                        umma_commit<CTAS>(bar_empty + 8 * stage);
                    }
                    __syncwarp();
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!alive) break;
                if (lane == 0) umma_commit<CTAS>(bar_tfull + 8 * acc);
                __syncwarp();
            }
        }
    } else if (warp_idx == 1) {
        // the odd CTA's warp 1 has nothing to issue: the even CTA drives the MMAs of the pair
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..9)
        // Two groups of four warps; group hf owns columns [128*hf, 128*hf + 128) of the tile.
        // Each thread keeps its row's 128 running sums in registers: after every segment
        // the TMEM partial sum is added in with round-to-nearest, and the piece is written
        // to D once, after its last segment.
        const uint32_t q = warp_idx & 3;              // TMEM lane quarter this warp may read
        const uint32_t hf = (warp_idx - 2) >> 2;
        const uint32_t row = q * 32 + lane;           // row inside this CTA's 128 rows
        const bool leader = (lane == 0) && (warp_idx == 2 + 4 * hf);
        uint8_t* my_buf = epi_gen + hf * EPI_BUF_BYTES;
        const uint32_t my_buf_s = epi_base + hf * EPI_BUF_BYTES;
        float accr[BN / 2];
        int it = 0;
        bool alive = true;
        long long u = u_begin;
        Piece pc;
        while (alive && next_piece(p, u, u_stride, pc)) {
            int tm, tn;
            tile_coords(p, pc.tile, tm, tn);
            const int m0 = tm * C::TILE_M + static_cast<int>(rank) * BM, n0 = tn * BN;
            // the running sums of this thread's row go to D: scale -> swizzled slab -> TMA store or reduce-add
            auto store_tile = [&](const CUtensorMap* md, bool reduce) {
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    const int col0 = n0 + hf * (BN / 2) + ch * EPI_COLS;
                    if (col0 < p.N && m0 < p.M) {
                        if (leader) bulk_wait_read<0>();          // the slab buffer has been read out
                        group_bar_sync(1 + hf);
                        uint8_t* rowp = my_buf + row * 128u;
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            float4 o;
                            o.x = p.alpha * accr[ch * 32 + 4 * j + 0];
                            o.y = p.alpha * accr[ch * 32 + 4 * j + 1];
                            o.z = p.alpha * accr[ch * 32 + 4 * j + 2];
                            o.w = p.alpha * accr[ch * 32 + 4 * j + 3];
                            *reinterpret_cast<float4*>(rowp + ((j ^ (row & 7u)) << 4)) = o;
                        }
                        fence_async_smem();
                        group_bar_sync(1 + hf);
                        if (leader) {
                            if (reduce) tma_reduce_add_2d(md, my_buf_s, col0, m0);
                            else tma_store_2d(md, my_buf_s, col0, m0);
                            bulk_commit();
                        }
                    }
                }
            };
            const bool first_out = I8 && p.first_out != 0;
            bool voted_out = false;
            for (int sg = pc.s0; sg < pc.s1; ++sg, ++it) {
                const uint32_t acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                if (!mbar_wait(bar_tfull + 8 * acc, acc_phase, abortp, p, 4)) { alive = false; break; }
                tc_fence_after();
                const bool fresh = sg == pc.s0 || (first_out && sg == pc.s0 + 1);       // this segment starts the running sum
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t v[32];
                    tmem_ld32(tmem_base + ((q * 32u) << 16) + acc * BN + hf * (BN / 2) + ch * EPI_COLS, v);
                    tmem_wait_ld();
                    if (I8) {
                        // int32 partial sums (exact) -> fp32, scaled by the level's power of two
                        const float sc = p.lvl_scale[p.n_lvl > 0 ? sg / p.n_chunks : 0];
                        if (fresh) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) accr[ch * 32 + i] = static_cast<float>(static_cast<int>(v[i])) * sc;
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i) accr[ch * 32 + i] = fmaf(static_cast<float>(static_cast<int>(v[i])), sc, accr[ch * 32 + i]);
                        }
                    } else if (fresh) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) accr[ch * 32 + i] = __uint_as_float(v[i]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) accr[ch * 32 + i] += __uint_as_float(v[i]);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (mma_cta) mbar_arrive(bar_tempty + 8 * acc);
                    else mbar_arrive_remote(bar_tempty + 8 * acc, 0);
                }
                if (first_out && sg == pc.s0) {
                    // The first level on its own goes out now, while the tensor core works on the next level.  The vote is
                    // the same barrier as the one behind the loop: a warp whose wait ran out above meets this one there.
                    if (group_bar_or(1 + hf, false)) { voted_out = true; break; }
                    store_tile(&map_d1, false);
                }
            }
            if (voted_out) { alive = false; break; }
            // A wait may have run out in some warps of the group and not in others: the group leaves together, or
            // the warps that went on would wait at the slab barriers below for warps that never come.
            if (group_bar_or(1 + hf, !alive)) { alive = false; break; }
            store_tile(&map_d, p.accumulate != 0);
        }
        if (leader) bulk_wait<0>();
    }

    if (*abortp) {
        // give copies that were already issued time to land before the smem is released
        const unsigned long long t0 = global_timer();
        while (global_timer() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();           // neither CTA frees its TMEM or leaves while the other may still use it
    if (warp_idx == 1) {
        tc_fence_after();
        __syncwarp();
        tmem_dealloc<CTAS>(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------- host side ----
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode_fn() {
    static encode_tiled_fn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<encode_tiled_fn>(ptr);
    }
    return fn;
}

bool make_map_2d(CUtensorMap* map, CUtensorMapDataType dt, int elem_bytes, const void* base, uint64_t inner,
                 uint64_t outer, uint64_t ld_elems, uint32_t box_inner, uint32_t box_outer) {
    encode_tiled_fn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {ld_elems * static_cast<uint64_t>(elem_bytes)};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Number of CTA pairs that can be resident at once (0 when the pair form cannot be launched).
int max_pairs(int sm_count) {
    static int cached_per_device[64];
    static lq_once_per_device once;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    int& cached = cached_per_device[dev];
    if (!once.first()) return cached;
    cached = 0;
    if (cudaFuncSetAttribute(lq_tc_gemm_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<2>::SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(lq_tc_gemm_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<2>::SMEM_BYTES) != cudaSuccess) {
        cudaGetLastError();
        return cached;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(sm_count / 2 * 2));
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = Cfg<2>::SMEM_BYTES;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, lq_tc_gemm_kernel<2, false>, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return cached;
    }
    cached = n < sm_count / 2 ? n : sm_count / 2;
    return cached;
}

}  // namespace

int lq_tc_gemm(lq_handle* h, cudaStream_t stream, const lq_tc_gemm_args& a) {
    if (a.M <= 0 || a.N <= 0) return LQ_OK;
    if (a.K <= 0) return LQ_OK;
    if (a.n_pass < 1 || a.n_pass > LQ_TC_MAX_PASS) return LQ_ERR_INVALID_ARG;
    if (a.n_lvl < 0 || a.n_lvl > LQ_TC_MAX_LVL || (a.n_lvl > 0 && a.chunk_kb < 1)) return LQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(a.A_all) & 15) || (reinterpret_cast<uintptr_t>(a.B_all) & 15) ||
        (reinterpret_cast<uintptr_t>(a.D) & 15) || (a.lda % (a.int8_ops ? 16 : 8)) || (a.ldb % (a.int8_ops ? 16 : 8)) || (a.ldd % 4))
        return LQ_ERR_INVALID_ARG;
    if (a.a_rows > 0x7fffffffLL || a.b_rows > 0x7fffffffLL || a.K > 0x7fffffffLL || a.M > 0x7fffffffLL ||
        a.N > 0x7fffffffLL)
        return LQ_ERR_UNSUPPORTED;

    static lq_once_per_device attr_set;
    if (attr_set.first()) {
        LQ_CUDA_TRY(cudaFuncSetAttribute(lq_tc_gemm_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<1>::SMEM_BYTES));
        LQ_CUDA_TRY(cudaFuncSetAttribute(lq_tc_gemm_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<1>::SMEM_BYTES));
    }
    // The pair form pays off once there are at least a few 256-row tiles; below that one CTA per tile.
    const int pairs = (a.M > BM) ? max_pairs(h->sm_count) : 0;
    const int ctas_per_tile = pairs > 0 ? 2 : 1;
    const int b_rows_box = BN / ctas_per_tile;

    CUtensorMap map_a, map_b, map_d, map_d1;
    const bool i8 = a.int8_ops != 0;
    const int bk_elems = i8 ? 2 * BK : BK;                 // a k-step is one 128-byte swizzle row of either type
    const CUtensorMapDataType op_dt = i8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const int op_bytes = i8 ? 1 : 2;
    if (!make_map_2d(&map_a, op_dt, op_bytes, a.A_all, a.K, a.a_rows, a.lda, bk_elems, BM) ||
        !make_map_2d(&map_b, op_dt, op_bytes, a.B_all, a.K, a.b_rows, a.ldb, bk_elems, b_rows_box) ||
        !make_map_2d(&map_d, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.D, a.N, a.M, a.ldd, EPI_COLS, BM))
        return LQ_ERR_CUDA;
    map_d1 = map_d;
    if (a.D_first) {
        // the first level's sum on its own: integer operands, at least two levels, one segment per level, nothing added to D
        if (!i8 || a.n_lvl < 2 || a.accumulate || (reinterpret_cast<uintptr_t>(a.D_first) & 15) ||
            a.chunk_kb < lq_ceil_div(a.K, bk_elems))
            return LQ_ERR_INVALID_ARG;
        if (!make_map_2d(&map_d1, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.D_first, a.N, a.M, a.ldd, EPI_COLS, BM)) return LQ_ERR_CUDA;
    }

    KParams p;
    p.M = static_cast<int>(a.M);
    p.N = static_cast<int>(a.N);
    p.K = static_cast<int>(a.K);
    p.n_pass = a.n_pass;
    for (int i = 0; i < LQ_TC_MAX_PASS; ++i) {
        p.a_off[i] = static_cast<int>(a.a_row_off[i]);
        p.b_off[i] = static_cast<int>(a.b_row_off[i]);
    }
    p.alpha = a.alpha;
    p.accumulate = a.accumulate;
    p.upper_only = a.upper_only;
    p.band = 8;
    p.tile_m = BM * ctas_per_tile;
    p.tiles_m = static_cast<int>(lq_ceil_div(a.M, p.tile_m));
    p.tiles_n = static_cast<int>(lq_ceil_div(a.N, BN));
    if (a.upper_only) {
        int cnt = 0;
        for (int m = 0; m < p.tiles_m; ++m) {
            int c = p.tiles_n - (m * p.tile_m) / BN;
            if (c > 0) cnt += c;
        }
        p.num_tiles = cnt;
    } else {
        p.num_tiles = p.tiles_m * p.tiles_n;
    }
    p.status = h->dstatus;
    p.timeout_ns = h->wait_limit_ns;
    p.stall_bytes = h->inject_stall ? 16 : 0;
    p.int8_ops = i8 ? 1 : 0;
    p.bk_elems = bk_elems;
    for (int i = 0; i < LQ_TC_MAX_PASS; ++i)
        p.idesc_pass[i] = ctas_per_tile == 2 ? Cfg<2>::idesc_i8(a.a_signed[i] != 0, a.b_signed[i] != 0)
                                             : Cfg<1>::idesc_i8(a.a_signed[i] != 0, a.b_signed[i] != 0);
    for (int i = 0; i < LQ_TC_MAX_LVL; ++i) p.lvl_scale[i] = a.lvl_scale[i];
    p.first_out = a.D_first ? 1 : 0;
    if (p.num_tiles == 0) return LQ_OK;
    {
        const int k_blocks = static_cast<int>(lq_ceil_div(a.K, bk_elems));
        const int k_iters = k_blocks * a.n_pass;
        p.seg_iters = (a.seg_iters > 0 && a.seg_iters < k_iters) ? a.seg_iters : k_iters;
        p.segs_per_tile = static_cast<int>(lq_ceil_div(k_iters, p.seg_iters));
        p.n_lvl = a.n_lvl;
        p.chunk_kb = a.chunk_kb > 0 ? a.chunk_kb : k_blocks;
        p.n_chunks = static_cast<int>(lq_ceil_div(k_blocks, p.chunk_kb));
        for (int i = 0; i < LQ_TC_MAX_LVL; ++i) { p.lvl_pass0[i] = 0; p.lvl_npass[i] = 0; }
        if (a.n_lvl > 0) {
            int next = 0;
            for (int i = 0; i < a.n_lvl; ++i) {
                if (a.lvl_npass[i] < 1) return LQ_ERR_INVALID_ARG;
                p.lvl_pass0[i] = next;
                p.lvl_npass[i] = a.lvl_npass[i];
                next += a.lvl_npass[i];
            }
            if (next != a.n_pass) return LQ_ERR_INVALID_ARG;
            p.segs_per_tile = a.n_lvl * p.n_chunks;
        }
    }
    // number of K parts: the one that leaves the shortest schedule, ceil(tiles * q / workers) / q
    const int workers = ctas_per_tile == 2 ? pairs : h->sm_count;
    p.k_parts = 1;
    if (a.accumulate && p.segs_per_tile >= 16) {          // long K only: every unit pays one epilogue
        double best = static_cast<double>(lq_ceil_div(p.num_tiles, workers));
        for (int q = 2; q <= 8 && q <= p.segs_per_tile; ++q) {
            const double t = static_cast<double>(lq_ceil_div(static_cast<int64_t>(p.num_tiles) * q, workers)) / q;
            if (t < best * 0.98) { best = t; p.k_parts = q; }
        }
    }
    p.total_units = static_cast<long long>(p.num_tiles) * p.k_parts;
    const int active = p.total_units < workers ? static_cast<int>(p.total_units) : workers;

    if (ctas_per_tile == 2) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(2 * active));
        cfg.blockDim = dim3(NUM_THREADS);
        cfg.dynamicSmemBytes = Cfg<2>::SMEM_BYTES;
        cfg.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        const cudaError_t le = i8 ? cudaLaunchKernelEx(&cfg, lq_tc_gemm_kernel<2, true>, map_a, map_b, map_d, map_d1, p)
                                  : cudaLaunchKernelEx(&cfg, lq_tc_gemm_kernel<2, false>, map_a, map_b, map_d, map_d1, p);
        if (le != cudaSuccess) {
            cudaGetLastError();
            return LQ_ERR_CUDA;
        }
        lq_launches_total.fetch_add(1, std::memory_order_relaxed);
    } else {
        if (i8) lq_tc_gemm_kernel<1, true><<<active, NUM_THREADS, Cfg<1>::SMEM_BYTES, stream>>>(map_a, map_b, map_d, map_d1, p);
        else lq_tc_gemm_kernel<1, false><<<active, NUM_THREADS, Cfg<1>::SMEM_BYTES, stream>>>(map_a, map_b, map_d, map_d1, p);
        LQ_LAUNCH_CHECK();
    }
    return LQ_OK;
}
