// Fused decode + prune + dense product on the 5th-generation tensor cores (sm_100a).
//
// Orientation.  Y[b][o] = sum_i X[b][i] * (W .* Ia)[o][i] is issued as D = A * B^T with
//   A = masked W tile   [128 rows of W      x 64 columns], K-major, 128-byte swizzle
//   B = X tile          [BN  rows of X      x 64 columns], K-major, 128-byte swizzle
//   D = fp32 accumulator in tensor memory: lane = row of W (output feature), column = batch row.
// W is the operand that must be masked, and it is the M operand so that one masked 128 x 64
// block feeds a 128 x BN x 64 MMA: with BN = 256 every decoded index bit is amortised over 256
// multiply-accumulates, which keeps the integer work of the decode under the MMA time.
//
// Warp roles in a 448-thread block:
//   warp 0      lane 0 issues the TMA loads (cp.async.bulk.tensor, 128B swizzle, zero fill outside
//               the matrix) of the X tile into the B stage and of the raw W tile into the A stage.
//   warp 1      allocates tensor memory; lane 0 issues tcgen05.mma for each filled stage and
//               commits the stage's "empty" barrier; finally commits the accumulator barrier.
//   warps 10-13 index decoders, one panel (PW*32 columns, all inside one tile) ahead of the pruning
//               warps.  They transpose the panel's column words of Iz into k bit-planes (plane l =
//               row l of Iz, 32 columns per word; a warp-wide 32x32 bit transpose, i.e. what 32
//               __ballot_sync votes would give), then each thread ORs, for one of the 128 rows, the
//               planes selected by the set bits of that row's Ip word.  That is Eq. 3 evaluated 32
//               columns per bitwise instruction; the result, the decoded index of the 128 x panel
//               block, stays bit-packed in shared memory (double buffered) and goes nowhere else.
//   warps 2-9   pruning warps, two sets of four that take alternate K blocks.  A thread owns one row (eight
//               16-byte chunks) of the 128 x 64 block.  When the stage's copies have landed it reads its chunks
//               from the A stage, expands its 64 index bits to bf16 AND-masks (a shift puts four bits on the sign
//               positions of the four bytes, prmt replicates each sign over a 16-bit half), zeroes pruned
//               weights and writes the chunks back in place.  The writes are made visible to the
//               tensor core with fence.proxy.async before the stage's "masked" barrier is signalled.
//               No pruning warp ever waits on global memory.  After the last K block the same warps
//               run the epilogue: tcgen05.ld of their 32-lane quadrant, conversion, transposition
//               through shared memory, and 16-byte row-contiguous stores to Y (or fp32 partial sums
//               when K is split).
//
// Every barrier wait is bounded by a wall-clock limit.  A wait that runs out records a code in
// the device status word and raises a block-wide abort flag; every role then leaves its loop, the
// TMA thread drains (bounded) the copies it has in flight, and tensor memory is freed before exit.
#include <mutex>

#include "lrbi_common.cuh"
#include "pipeline_ptx.cuh"

namespace lrbi {

constexpr int TC_THREADS = 448;               // with one group of decoder warps; a second group adds 128
constexpr int TC_BM = 128;                 // rows of W per block (MMA M)
constexpr int TC_BK = 64;                  // columns per stage: 64 bf16 = one 128-byte swizzle row
constexpr int TC_A_STAGE_BYTES = TC_BM * TC_BK * 2;
constexpr int TC_MASK_WARPS = 8;           // warps 2-9: prune the W tile of each stage, then run the epilogue
constexpr int TC_DECODE_WARPS = 4;         // warps 10-13: decode the index one panel ahead
// Two-accumulator blocks (BN = 512) and the 192-column pairs run a second group of decoder warps (14-17): group g decodes the panels
// with P % 2 == g into index buffer g, so a panel may take two panels' worth of pruning time.
__host__ __device__ constexpr int tc_decode_groups(int bn) { return (bn > 256 || bn == 192) ? 2 : 1; }
__host__ __device__ constexpr int tc_threads(int bn) { return TC_THREADS + (tc_decode_groups(bn) - 1) * TC_DECODE_WARPS * 32; }
__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// ---- CTA-pair (cta_group::2) variants: one MMA spans the tensor cores and shared memory of two
// CTAs of a cluster; the accumulator rows are split between their tensor memories.
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync_all()
{
    cluster_arrive();
    cluster_wait();
}
__device__ __forceinline__ void tmem_alloc2(uint32_t *dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma2_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are done.
__device__ __forceinline__ void umma2_commit_both(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((uint16_t)3) : "memory");
}
// Arrive on the barrier at the same offset in the shared memory of CTA `rank` of the cluster.
__device__ __forceinline__ void mbar_arrive_remote(uint64_t *bar, uint32_t rank)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(bar)), "r"(rank));
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows 128 bytes apart,
// 8-row groups 1024 bytes apart (PTX ISA, tcgen05 matrix descriptor).
__device__ __forceinline__ uint64_t make_sw128_desc(uint32_t saddr)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);           // start address
    d |= (uint64_t)1 << 16;                             // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                   // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                             // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                             // 128-byte swizzle
    return d;
}
// The same for an MN-major operand (the M or N index runs along memory, K across rows), 128-byte swizzle: an atom is
// 64 values of M/N (128 bytes) x 8 values of K (rows 128 bytes apart); atoms along M/N lie `mn_atom_bytes` apart
// (the leading byte offset), groups of 8 values of K 1024 bytes apart (the stride byte offset).
__device__ __forceinline__ uint64_t make_sw128_mn_desc(uint32_t saddr, uint32_t mn_atom_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(mn_atom_bytes >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = bn.
__host__ __device__ constexpr uint32_t make_idesc(int bn, int m = TC_BM)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// 16-byte asynchronous copy global -> shared; bytes beyond `valid` (0..16) are written as zero.
__device__ __forceinline__ void cp_async_16(void *dst_smem, const void *src, int valid)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst_smem)), "l"(src), "r"(valid) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// Rank and words per row/column of the tile that holds rows o0.. and columns c0.. (one rank per tile when `rk`
// carries arrays, else the layout's rank), and the first factor words of that tile.
__device__ __forceinline__ void panel_tile(const Geo &g, const TileRanks &rk, const uint32_t *ip, const uint32_t *iz,
                                           int c0, int o0, int &k, int &kw, const uint32_t *&ipt, const uint32_t *&izt)
{
    const int tr = min(o0, g.rows - 1) / g.tm, tc = min(c0, g.cols - 1) / g.tn;
    const size_t tile = (size_t)tr * g.ts_r + (size_t)tc * g.ts_c;
    if (rk.ranks) {
        k = __ldg(rk.ranks + tile);
        kw = (k + 31) >> 5;
        ipt = ip + __ldg(rk.ip_offset + tile);
        izt = iz + __ldg(rk.iz_offset + tile);
    } else {
        k = g.k;
        kw = g.kw;
        ipt = ip + tile * g.tm * g.kw;
        izt = iz + tile * g.tn * g.kw;
    }
}

// Stage the factor words of one panel: the Iz words of its `pw32` columns (first column c0, tile row tr)
// and the Ip words of the block's 128 rows (first row o0), kw words each (the rank of the panel's tile).
// Words outside the tile are written as zero.
// Asynchronous copies (one commit group); the caller waits for them.  dt = 0 .. nthreads-1.
__device__ __forceinline__ void stage_panel_factors(const Geo &g, const TileRanks &rk, const uint32_t *__restrict__ ip,
                                                    const uint32_t *__restrict__ iz, uint32_t *iz_stage,
                                                    uint32_t *ip_stage, int pw32, int c0, int o0, int dt, int nthreads)
{
    int k, kw;
    const uint32_t *ipt, *izt;
    panel_tile(g, rk, ip, iz, c0, o0, k, kw, ipt, izt);
    const int zwords = pw32 * kw, xwords = TC_BM * kw;
    if (o0 >= g.rows) {                                  // a block without rows of W (second CTA of a ragged pair)
        for (int q = dt; q < zwords; q += nthreads) iz_stage[q] = 0u;
        for (int q = dt; q < xwords; q += nthreads) ip_stage[q] = 0u;
        cp_async_commit();
        return;
    }
    const int i0 = o0 - (o0 / g.tm) * g.tm;              // first row of the block inside its tile
    const int j0 = c0 - (c0 / g.tn) * g.tn;              // first column of the panel inside its tile
    const uint32_t *zsrc = izt + (size_t)j0 * kw;
    const uint32_t *xsrc = ipt + (size_t)i0 * kw;
    // 16-byte copies need 16-byte aligned sources (tile bases of a ranked layout need not be)
    const bool z_vec = (reinterpret_cast<uintptr_t>(zsrc) & 15u) == 0, x_vec = (reinterpret_cast<uintptr_t>(xsrc) & 15u) == 0;
    const int zvalid = (g.tn - j0) * kw, xvalid = (g.tm - i0) * kw;   // words that exist in the tile
    for (int q = dt * 4; q < zwords; q += nthreads * 4) {
        const int n = min(4, max(0, zvalid - q));
        if (z_vec) cp_async_16(iz_stage + q, zsrc + (n > 0 ? q : 0), n * 4);
        else for (int e = 0; e < 4; ++e) iz_stage[q + e] = e < n ? __ldg(zsrc + q + e) : 0u;
    }
    for (int q = dt * 4; q < xwords; q += nthreads * 4) {
        const int n = min(4, max(0, xvalid - q));
        if (x_vec) cp_async_16(ip_stage + q, xsrc + (n > 0 ? q : 0), n * 4);
        else for (int e = 0; e < 4; ++e) ip_stage[q + e] = e < n ? __ldg(xsrc + q + e) : 0u;
    }
    cp_async_commit();
}

// Shared-memory bookkeeping that follows the operand stages.
struct TcCtl {
    uint64_t full[8];        // TMA copies of a stage have landed
    uint64_t masked[8];      // ... and its W tile has been pruned in place (leader of a pair: in both CTAs)
    uint64_t empty[8];       // the MMAs that read the stage have completed
    uint64_t accum;
    uint64_t tmem_free;      // PERSIST: tensor memory may be overwritten by the next tile's MMAs
    uint64_t bits_ready[2];  // decoders -> pruners: the index bits of a panel are in buffer b
    uint64_t bits_free[2];   // pruners -> decoders: buffer b may be overwritten
    uint64_t dsync[2];       // the four warps of a decoder group meet here twice per panel
    uint32_t tmem_base;
    int abort_flag;
};

// --------------------------------------------------------------------------------------
// kernel
// --------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Bit position of column e (0..31) inside a plane / index word.  Column e = 4g + i sits at bit
// 8i + 7 - g, so that `word << g` leaves the four bits of group g on the sign positions of the
// four bytes.  column_of_bit is the inverse (which column a ballot lane stands for).
__device__ __forceinline__ int column_of_bit(int bit) { return 4 * (7 - (bit & 7)) + (bit >> 3); }

// Zero the pruned halves of the eight bf16 values of one 16-byte chunk.  `bits` holds the index
// bits of the row's 32 columns in the permuted order above; chunk j uses groups 2j and 2j+1.
__device__ __forceinline__ uint4 prune_chunk(uint4 w, uint32_t bits, int j)
{
    const uint32_t t0 = bits << (2 * j), t1 = bits << (2 * j + 1);
    w.x &= prmt(t0, t0, 0x9988u);       // sign of byte 0 -> low half, sign of byte 1 -> high half
    w.y &= prmt(t0, t0, 0xBBAAu);       // bytes 2 and 3
    w.z &= prmt(t1, t1, 0x9988u);
    w.w &= prmt(t1, t1, 0xBBAAu);
    return w;
}

// Decoder group of a thread (0 for every thread that is not in the second group).
__device__ __forceinline__ int warp_of_thread_decoder_group(unsigned tid)
{
    return tid >= (unsigned)TC_THREADS ? 1 : 0;
}

// grid = (batch tiles, row tiles of 128, K splits).  When gridDim.z > 1 the block writes fp32
// partial sums to `partials` [split][batch][rows]; a second kernel adds them up.
// PW = 32-bit index words per row of a panel (8: 256-column panels, 2: 64-column panels).
// PAIR: two CTAs of a cluster (neighbours along grid x) share one 256-row x BN-column
// output tile.  Each loads and prunes its own 128 rows of W and loads its own half of the X tile; the
// leader CTA (cluster rank 0) issues tcgen05.mma.cta_group::2, which reads the operands of both CTAs
// and leaves each CTA's 128 accumulator rows in its own tensor memory.  Every X tile is then fetched
// once per 256 rows of W instead of once per 128, and each byte of it is read from shared memory by
// one tensor core pass instead of two.  Two such blocks are resident per SM (three stages each), so
// one block's epilogue and panel hand-overs overlap the other's MMAs.
// PERSIST (two-accumulator pairs, K not split): the grid is one pair per two SMs and a pair walks output tiles
// (pair p takes tiles p, p + pairs, ...).  Stage, panel and barrier state run on across tiles, so while the pruning
// warps drain tensor memory of tile n (through warp-private staging, the operand stages are no longer free), the
// copies, the factor words and the first index panels of tile n + 1 are already on their way; the first MMA of a
// tile waits until both CTAs have emptied tensor memory.
// DW (persistent pairs only): the product of the masked layer's weight gradient, dW = (dY^T X) .* Ia.  Nothing is
// pruned inside the contraction (the pruning warps only pass the stages on); `gi` is the layout of the index as the
// output sees it (rows = rows of the output tile, columns = its batch axis), the decoders decode the two 256-column
// panels of each output tile from it, and the epilogue zeroes the pruned outputs as it stores them.
template <int BN, int PW, bool PAIR, bool PERSIST, bool DW, bool MNM>
__global__ void __launch_bounds__(tc_threads(BN), (BN > 256 || BN == 192) ? 1 : 2)
gemm_tc_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap w_map, Geo g, Geo gi, TileRanks rk,
               const uint32_t *__restrict__ ip, const uint32_t *__restrict__ iz, int batch,
               void *__restrict__ Y, int y_dtype, float *__restrict__ partials, int kb_per_split,
               int stages, int *status)
{
    extern __shared__ __align__(1024) uint8_t smem[];    // swizzled operand stages need 1024-byte alignment
    constexpr int B_ROWS = PAIR ? BN / 2 : BN;          // rows of X this CTA loads per stage
    constexpr int B_STAGE_BYTES = B_ROWS * TC_BK * 2;
    constexpr int TMEM_COLS = BN < 32 ? 32 : BN == 192 ? 256 : BN;   // a power of two
    // Pair mode, BN = 512: two accumulators of 256 batch columns fill the 512 columns of tensor memory.
    // A pruned W stage then feeds two MMAs, so decode and pruning are amortised over twice the tensor work.
    // Accumulator a covers batch rows b0 + 256 a ...; CTA `rank` loads the 128 rows b0 + 256 a + 128 rank ...
    // of it as box a of its B stage.
    // BN = 192: one accumulator of 192 columns, 96 rows of X per CTA (a tile width that puts layers with few rows
    // and a long batch on more of the chip's SMs: 12544 batch rows make 66 tiles of 192 against 25 of 512).
    constexpr int NACC = PAIR && BN > 256 ? BN / 256 : 1;
    constexpr int XBOX_ROWS = PAIR ? (BN < 256 ? BN / 2 : 128) : BN;   // rows of one TMA box of X
    constexpr int MMA_N = PAIR ? (BN < 256 ? BN : 256) : BN;
    static_assert(!PAIR || BN == 192 || BN == 256 || BN == 512, "pair mode: one accumulator of 192 or 256 columns, or two of 256");
    static_assert(!PERSIST || BN == 512, "the persistent epilogue walks two 256-column accumulators");
    static_assert(!MNM || (DW && PERSIST && PAIR), "MN-major operands: the weight-gradient product only");
    constexpr int KBP = PW / 2;                          // K blocks per panel
    uint8_t *a_base = smem;
    uint8_t *b_base = smem + (size_t)stages * TC_A_STAGE_BYTES;
    constexpr int PWS = PW == 8 ? 12 : PW;               // words between planes (padded: conflict-free 16-byte reads)
    uint32_t *row_bits = reinterpret_cast<uint32_t *>(b_base + (size_t)stages * B_STAGE_BYTES);   // [2][128][PW]
    constexpr int NDG = tc_decode_groups(BN);            // groups of decoder warps
    // per decoder group: planes [kw*32][PWS], iz_stage [PW*32][kw], ip_stage [128][kw]
    const int ikw = DW ? gi.kw : g.kw;                   // index words per factor row / column
    const int dgroup_words = ikw * 32 * PWS + PW * 32 * ikw + TC_BM * ikw;
    const int dgrp = warp_of_thread_decoder_group(threadIdx.x);
    uint32_t *planes = row_bits + 2 * TC_BM * PW + dgrp * dgroup_words;
    uint32_t *iz_stage = planes + ikw * 32 * PWS;
    uint32_t *ip_stage = iz_stage + PW * 32 * ikw;
    uint8_t *epi_stage = reinterpret_cast<uint8_t *>(row_bits + 2 * TC_BM * PW + NDG * dgroup_words);   // PERSIST: 1 KB per pruning warp
    TcCtl *ctl = reinterpret_cast<TcCtl *>(epi_stage + (PERSIST ? TC_MASK_WARPS * 1024 : 0));
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if ((smem_u32(smem) & 1023u) != 0) {                 // never expected; refuse rather than compute garbage
        if (threadIdx.x == 0) atomicCAS(status, 0, DEV_BAD_SMEM_ALIGN);
        return;
    }
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u; // 0 = leader of the pair
    // grid.x runs fastest over blocks that share rows of W, so W streams from HBM once and X stays in L2.
    // Pair mode: the two CTAs of a cluster are neighbours along x (x = 2 * batch tile + rank), y = 256-row pair.
    // PERSIST: the block's n-th tile is tile t = (pair index) + n * (pairs in the grid).  t runs fastest over the tiles of
    // the smaller operand (batch tiles when X is the smaller matrix, row pairs when W is), so that the pairs at work
    // at any time share all of the small operand, which stays in L2, and the large one streams from memory once.
    const int nbt = (batch + BN - 1) / BN;
    const int nrp = (g.rows + 2 * TC_BM - 1) / (2 * TC_BM);
    const bool rows_fast = g.rows < batch;
    const int tile_first = PERSIST ? (int)(blockIdx.x >> 1) : 0, tile_step = PERSIST ? (int)(gridDim.x >> 1) : 1;
    const int my_tiles = PERSIST ? (nbt * nrp - tile_first + tile_step - 1) / tile_step : 1;
    auto tile_b0 = [&](int n) {                          // first batch row of the block's n-th tile
        const int t = tile_first + n * tile_step;
        return PERSIST ? (rows_fast ? t / nrp : t % nbt) * BN : (int)(PAIR ? (blockIdx.x >> 1) : blockIdx.x) * BN;
    };
    auto tile_o0 = [&](int n) {                          // first row of W of this block in its n-th tile
        const int t = tile_first + n * tile_step;
        return PERSIST ? ((rows_fast ? t % nrp : t / nbt) * 2 + (int)rank) * TC_BM
                       : (int)(PAIR ? (blockIdx.y * 2 + rank) : blockIdx.y) * TC_BM;
    };
    const int b0 = tile_b0(0), o0 = tile_o0(0);
    const int nkb_total = (g.cols + TC_BK - 1) / TC_BK;
    const int kb_begin = blockIdx.z * kb_per_split;      // a multiple of KBP
    const int kb_end = min(nkb_total, kb_begin + kb_per_split);
    const int nkb = kb_end - kb_begin;                   // >= 1 by construction of the grid

    // Long-latency requests first: the decoder warps ask for the factor words of their first panel, one
    // thread warms the TMA descriptors; both overlap the barrier and tensor-memory set-up below.
    {
        const int npanels0 = DW ? BN / 256 : (nkb + KBP - 1) / KBP;   // group g starts with panel g (of the block's first tiles)
        if (warp >= 2 + TC_MASK_WARPS && dgrp < my_tiles * npanels0)
            stage_panel_factors(DW ? gi : g, rk, ip, iz, iz_stage, ip_stage, PW * 32,
                                DW ? tile_b0(dgrp / npanels0) + (dgrp % npanels0) * 256 : (kb_begin + (dgrp % npanels0) * KBP) * TC_BK,
                                tile_o0(dgrp / npanels0),
                                (threadIdx.x - (2 + TC_MASK_WARPS) * 32) & (TC_DECODE_WARPS * 32 - 1), TC_DECODE_WARPS * 32);
    }
    if (threadIdx.x == 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&x_map) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&w_map) : "memory");
    }
    if (warp == 0) {                                     // one lane per stage, three more for the rest
        if (lane < stages) {
            mbar_init(&ctl->full[lane], 1);
            // leader of a pair: its stage is ready when its own four pruning warps of the K block's set and the other CTA's relay have arrived
            mbar_init(&ctl->masked[lane], TC_MASK_WARPS / 2 + ((PAIR && rank == 0) ? 1 : 0));   // one set of pruning warps per K block
            mbar_init(&ctl->empty[lane], 1);
        } else if (lane == 8) {
            mbar_init(&ctl->accum, 1);
            mbar_init(&ctl->tmem_free, 2 * TC_MASK_WARPS);   // PERSIST, leader: the pruning warps of both CTAs have drained tensor memory
            ctl->abort_flag = 0;
        } else if (lane == 9 || lane == 10) {
            const int b = lane - 9;
            mbar_init(&ctl->bits_ready[b], TC_DECODE_WARPS);
            mbar_init(&ctl->bits_free[b], TC_MASK_WARPS);
            mbar_init(&ctl->dsync[b], TC_DECODE_WARPS);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        if (PAIR) tmem_alloc2(&ctl->tmem_base, TMEM_COLS);
        else tmem_alloc(&ctl->tmem_base, TMEM_COLS);
    }
    tc_fence_before();
    __syncthreads();
    // Both CTAs' barriers must exist before anyone signals across.  Everybody arrives at the cluster barrier now; the
    // warp of the TMA producer waits only after its first round of copies is on its way (they touch this CTA alone).
    __syncwarp();                                        // (the cluster barrier is a warp-wide instruction)
    if (PAIR) {
        cluster_arrive();
        if (warp != 0) cluster_wait();
    }
    tc_fence_after();
    const uint32_t tmem_d = ctl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------- TMA producer (X tiles)
        bool issued = false;
        int s = 0;
        uint32_t parity = 1;                            // a fresh barrier reports its "previous" phase complete
        bool go = true;
        const long long total = (long long)my_tiles * nkb;
        auto issue = [&](long long q0, long long q1) {  // K blocks q0 .. q1-1, counted across the block's tiles
            for (long long q = q0; q < q1 && go; ++q) {
                const int n = (int)(q / nkb), it = (int)(q - (long long)n * nkb);
                const int b0 = tile_b0(n), o0 = tile_o0(n);
                if (!mbar_wait(&ctl->empty[s], parity, abort_flag, status, DEV_TIMEOUT_EMPTY)) { go = false; break; }
                mbar_arrive_expect_tx(&ctl->full[s], B_STAGE_BYTES + TC_A_STAGE_BYTES);
                if (MNM) {
                    // MN-major operands: boxes of 64 values of M (or N) x 64 values of K, 8 KB each; this CTA's 128
                    // rows of A are two boxes, its 128 columns of accumulator a two more
#pragma unroll
                    for (int h = 0; h < 2; ++h)
                        tma_load_2d(a_base + s * TC_A_STAGE_BYTES + h * 8192, &w_map, &ctl->full[s], o0 + 64 * h, (kb_begin + it) * TC_BK);
#pragma unroll
                    for (int a = 0; a < NACC; ++a)
#pragma unroll
                        for (int h = 0; h < 2; ++h)
                            tma_load_2d(b_base + s * B_STAGE_BYTES + a * 16384 + h * 8192, &x_map, &ctl->full[s],
                                        b0 + a * 256 + (int)rank * 128 + 64 * h, (kb_begin + it) * TC_BK);
                } else {
                tma_load_2d(a_base + s * TC_A_STAGE_BYTES, &w_map, &ctl->full[s], (kb_begin + it) * TC_BK, o0);
#pragma unroll
                for (int a = 0; a < NACC; ++a)
                    tma_load_2d(b_base + s * B_STAGE_BYTES + a * (XBOX_ROWS * TC_BK * 2), &x_map, &ctl->full[s],
                                (kb_begin + it) * TC_BK, b0 + a * 256 + (int)rank * XBOX_ROWS);
                }
                issued = true;
                if (++s == stages) { s = 0; parity ^= 1; }
            }
        };
        const long long first = total < stages ? total : stages;   // the ring's first round needs nobody else
        if (lane == 0) issue(0, first);
        __syncwarp();
        if (PAIR) cluster_wait();
        if (lane == 0) {
            issue(first, total);
            if (*abort_flag && issued) {
                // Abort path: copies already issued must land before this block's shared memory is
                // given up.  Wait on elapsed cycles alone (bounded): about 2 ms, far beyond any copy
                // in flight.
                const long long t0 = clock64();
                while (clock64() - t0 < 4000000ll) { }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------- MMA issuer
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = (PAIR ? make_idesc(MMA_N, 2 * TC_BM) : make_idesc(MMA_N)) | (MNM ? (1u << 15) | (1u << 16) : 0u);   // bits 15, 16: A, B MN-major
            bool ok = true;
            int s = 0;
            uint32_t parity = 0;
            uint32_t tfree_parity = 1;                  // a fresh barrier reports its "previous" phase complete
            for (int n = 0; n < my_tiles && ok; ++n) {
            if (PERSIST) {                              // both CTAs have read the previous tile's accumulators
                ok = mbar_wait(&ctl->tmem_free, tfree_parity, abort_flag, status, DEV_TIMEOUT_ACCUM);
                tfree_parity ^= 1;
                if (!ok) break;
                tc_fence_after();
            }
            for (int it = 0; it < nkb && ok; ++it) {
                ok = mbar_wait(&ctl->masked[s], parity, abort_flag, status, DEV_TIMEOUT_FULL);
                if (!ok) break;
                tc_fence_after();
                const uint64_t da = MNM ? make_sw128_mn_desc(smem_u32(a_base + s * TC_A_STAGE_BYTES), 8192)
                                        : make_sw128_desc(smem_u32(a_base + s * TC_A_STAGE_BYTES));
                const uint64_t db = MNM ? make_sw128_mn_desc(smem_u32(b_base + s * B_STAGE_BYTES), 8192)
                                        : make_sw128_desc(smem_u32(b_base + s * B_STAGE_BYTES));
#pragma unroll
                for (int k4 = 0; k4 < TC_BK / 16; ++k4) {
                    // 16 bf16 = 32 bytes further along K inside the swizzled row: +2 in address units
                    if (MNM) {                           // 16 values of K further: 16 rows of 128 bytes
#pragma unroll
                        for (int a = 0; a < NACC; ++a)
                            umma2_bf16(tmem_d + (uint32_t)(a * 256), da + (uint64_t)(128 * k4),
                                       db + (uint64_t)(a * (16384 >> 4) + 128 * k4), idesc, (it | k4) ? 1u : 0u);
                    } else if (PAIR) {
#pragma unroll
                        for (int a = 0; a < NACC; ++a)   // box a of the B stage -> accumulator a (256 columns further)
                            umma2_bf16(tmem_d + (uint32_t)(a * 256), da + (uint64_t)(2 * k4),
                                       db + (uint64_t)(a * ((XBOX_ROWS * TC_BK * 2) >> 4) + 2 * k4), idesc, (it | k4) ? 1u : 0u);
                    } else {
                        umma_bf16(tmem_d, da + (uint64_t)(2 * k4), db + (uint64_t)(2 * k4), idesc, (it | k4) ? 1u : 0u);
                    }
                }
                // frees the stage (in both CTAs of a pair) when these MMAs have read it
                if (PAIR) umma2_commit_both(&ctl->empty[s]); else umma_commit(&ctl->empty[s]);
                if (++s == stages) { s = 0; parity ^= 1; }
            }
            if (ok) {                                   // accumulator complete
                if (PAIR) umma2_commit_both(&ctl->accum); else umma_commit(&ctl->accum);
            }
            }
        } else if (lane == 0) {
            // ------------------------------------------------------------- relay (second CTA of a pair)
            // tells the leader when this CTA's half of a stage is loaded and pruned
            bool ok = true;
            int s = 0;
            uint32_t parity = 0;
            for (long long it = 0; it < (long long)my_tiles * nkb && ok; ++it) {
                ok = mbar_wait(&ctl->masked[s], parity, abort_flag, status, DEV_TIMEOUT_FULL);
                if (!ok) break;
                mbar_arrive_remote(&ctl->masked[s], 0);
                if (++s == stages) { s = 0; parity ^= 1; }
            }
        }
    } else if (warp >= 2 + TC_MASK_WARPS) {
        // ------------------------------------------------------------- index decoders
        const int dt = (threadIdx.x - (2 + TC_MASK_WARPS) * 32) & (TC_DECODE_WARPS * 32 - 1);   // 0..127: row of the block this thread decodes
        const int dw = dt >> 5;                         // decoder warp 0..3
        const int bit_col = column_of_bit(lane);        // column (0..31) this lane stands for in a transpose
        const Geo &gx = DW ? gi : g;                   // the layout the index is decoded from
        const int npanels = DW ? BN / 256 : (nkb + KBP - 1) / KBP;

        // panels are counted across the block's tiles: panel PG is panel PG % npanels of tile PG / npanels
        auto stage_factors = [&](int PG) {
            if (PG < my_tiles * npanels) {
                const int n2 = PG / npanels, P2 = PG - n2 * npanels;
                stage_panel_factors(gx, rk, ip, iz, iz_stage, ip_stage, PW * 32, DW ? tile_b0(n2) + P2 * 256 : (kb_begin + P2 * KBP) * TC_BK, tile_o0(n2), dt, TC_DECODE_WARPS * 32);
            }
        };

        uint32_t dsync_parity = 0;
        bool ok = true;
        auto dsync = [&]() {                            // the four decoder warps meet (bounded wait)
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->dsync[dgrp]);
            ok = mbar_wait(&ctl->dsync[dgrp], dsync_parity, abort_flag, status, DEV_TIMEOUT_EMPTY);
            dsync_parity ^= 1;
        };

        // (the group's first panel was requested at kernel entry)
        for (int PG = dgrp; PG < my_tiles * npanels && ok; PG += NDG) {
            const int tile_n = PG / npanels, P = PG - tile_n * npanels;
            const int o0 = tile_o0(tile_n);
            const int tr = o0 / gx.tm;                   // the 128 rows lie in one tile row
            const int i0 = o0 - tr * gx.tm;              // first row of the block inside its tile
            const bool row_ok = o0 + dt < gx.rows && i0 + dt < gx.tm;
            const int buf = PG & 1;
            uint32_t *rb_buf = row_bits + buf * (TC_BM * PW);
            const int c0 = DW ? tile_b0(tile_n) + P * 256 : (kb_begin + P * KBP) * TC_BK;
            // rank of the panel's tile (the layout's, or the tile's own in a ranked layout)
            int kp = gx.k, kwp = gx.kw;
            if (rk.ranks) {
                kp = __ldg(rk.ranks + (size_t)min(tr, gx.gr - 1) * gx.ts_r + (size_t)(min(c0, gx.cols - 1) / gx.tn) * gx.ts_c);
                kwp = (kp + 31) >> 5;
            }
            const uint32_t tail = tail_mask(kp);
            const int npairs = kwp * PW;                 // (32-plane block, index word) pairs of the panel
            cp_async_wait_all();                         // this thread's copies for panel P have landed
            dsync();                                     // ... and everybody else's
            if (!ok) break;
            // (a) bit-planes of Iz: each lane brings the k-bit word of one column, a warp-wide transpose
            //     turns 32 column words into 32 plane words (lane l keeps plane lb*32 + l)
            for (int n0 = 0; dw + TC_DECODE_WARPS * n0 < npairs; n0 += 4) {
                uint32_t z[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int pi = dw + TC_DECODE_WARPS * (n0 + t);
                    const int lb = pi / PW, col = (pi % PW) * 32 + bit_col;
                    z[t] = (pi < npairs && c0 + col < gx.cols) ? iz_stage[col * kwp + lb] : 0u;
                    if (lb == kwp - 1) z[t] &= tail;
                }
                warp_transpose32_x4(z, lane);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int pi = dw + TC_DECODE_WARPS * (n0 + t);
                    if (pi < npairs) planes[((pi / PW) * 32 + lane) * PWS + (pi % PW)] = z[t];
                }
            }
            // this thread's row words of Ip, into registers (k <= 256: at most eight)
            uint32_t xw[8];
#pragma unroll
            for (int lb = 0; lb < 8; ++lb) {
                xw[lb] = (row_ok && lb < kwp) ? ip_stage[dt * kwp + lb] : 0u;
                if (lb == kwp - 1) xw[lb] &= tail;
            }
            dsync();                                     // planes complete, factor staging consumed
            if (!ok) break;
            stage_factors(PG + NDG);                     // the group's next panel: its factor words start their trip now
            // the pruning warps must be done with the panel that used this buffer two panels ago
            ok = mbar_wait(&ctl->bits_free[buf], ((PG >> 1) & 1) ^ 1, abort_flag, status, DEV_TIMEOUT_EMPTY);
            if (!ok) break;
            // (b) Eq. 3 for one row: OR of the planes its Ip bits select
            uint32_t acc[PW];
#pragma unroll
            for (int q = 0; q < PW; ++q) acc[q] = 0;
#pragma unroll
            for (int lb = 0; lb < 8; ++lb) {
                uint32_t x = xw[lb];
                while (x) {
                    const int l = lb * 32 + __ffs(x) - 1;
                    x &= x - 1;
                    const uint32_t *src = planes + l * PWS;
                    if (PW == 8) {
                        const uint4 v0 = reinterpret_cast<const uint4 *>(src)[0], v1 = reinterpret_cast<const uint4 *>(src)[1];
                        acc[0] |= v0.x; acc[1] |= v0.y; acc[2 % PW] |= v0.z; acc[3 % PW] |= v0.w;
                        acc[4 % PW] |= v1.x; acc[5 % PW] |= v1.y; acc[6 % PW] |= v1.z; acc[7 % PW] |= v1.w;
                    } else {
#pragma unroll
                        for (int q = 0; q < PW; ++q) acc[q] |= src[q];
                    }
                }
            }
            if (PW == 8) {
                reinterpret_cast<uint4 *>(rb_buf + dt * PW)[0] = make_uint4(acc[0], acc[1], acc[2 % PW], acc[3 % PW]);
                reinterpret_cast<uint4 *>(rb_buf + dt * PW)[1] = make_uint4(acc[4 % PW], acc[5 % PW], acc[6 % PW], acc[7 % PW]);
            } else {
#pragma unroll
                for (int q = 0; q < PW; ++q) rb_buf[dt * PW + q] = acc[q];
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->bits_ready[buf]);
        }
        cp_async_wait_all();
    } else {
        // ------------------------------------------------------------- pruning warps
        const int mt = threadIdx.x - 64;                // 0..255
        const int mw = mt >> 5;                         // pruning warp 0..7
        // The warps form two sets of four; set q takes the K blocks that land in the stages with s mod 2 == q, so the
        // wait - load - prune - store - fence - arrive chain of one K block overlaps the next block's (the chain is
        // latency, not work).  The split goes by stage, not by K block, on purpose: a stage's barriers are then waited
        // on by the same warps in every phase.  A warp that skipped a phase of a barrier would ask for a parity that
        // the barrier's previous phase also has, and pass before the copies it waits for were even issued (with an
        // odd number of stages and sets by K block that happened about once in two hundred launches).
        // Inside a set a thread owns one row of the 128 (eight 16-byte chunks; the eight lanes of one access phase
        // fall on eight different swizzled chunk positions).
        const int set = mw >> 2;
        const int r = (mw & 3) * 32 + lane;             // row of the 128-row block

        bool ok = true;
        int s = 0;                                       // stage of the current K block
        uint32_t full_parity = 0;
        int kp = 0;                                      // K block inside its panel
        int P = 0;                                       // panel index, counted across the block's tiles
        int P_seen = -1;                                 // last panel whose index bits this warp has waited for
        auto panel_bits_ready = [&]() {                  // (every warp waits for every panel, also one it takes no block of:
            if (P_seen != P) {                           //  its arrival below must not run ahead of the decoders)
                ok = mbar_wait(&ctl->bits_ready[P & 1], (P >> 1) & 1, abort_flag, status, DEV_TIMEOUT_FULL);
                P_seen = P;
            }
        };
        for (int tile_n = 0; tile_n < my_tiles && ok; ++tile_n) {
        const int b0 = tile_b0(tile_n), o0 = tile_o0(tile_n);
        for (int it = 0; it < nkb && ok; ++it) {
            const bool mine = (s & 1) == set;
            if (DW) {                                    // nothing is pruned inside this contraction: pass the stage on
                if (mine) {
                    ok = mbar_wait(&ctl->full[s], full_parity, abort_flag, status, DEV_TIMEOUT_FULL);
                    if (!ok) break;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->masked[s]);
                }
                if (++s == stages) { s = 0; full_parity ^= 1; }
                continue;
            }
            const int buf = P & 1;
            if (mine) {
                panel_bits_ready();
                if (!ok) break;
                const uint2 bits = *reinterpret_cast<const uint2 *>(row_bits + buf * (TC_BM * PW) + r * PW + kp * 2);
                // ---------------- prune the 64 weights of one row of the A stage, in place
                ok = mbar_wait(&ctl->full[s], full_parity, abort_flag, status, DEV_TIMEOUT_FULL);
                if (!ok) break;
                uint8_t *a_row = a_base + s * TC_A_STAGE_BYTES + r * 128;
                uint4 wv[8];
#pragma unroll
                for (int c = 0; c < 8; ++c)              // 128-byte swizzle: 16-byte chunk c of row r lives at chunk position c ^ (r % 8)
                    wv[c] = *reinterpret_cast<const uint4 *>(a_row + ((c ^ (r & 7)) << 4));
#pragma unroll
                for (int c = 0; c < 8; ++c) {            // chunk c: index word c / 4, chunk-in-word c % 4
                    wv[c] = prune_chunk(wv[c], (c < 4) ? bits.x : bits.y, c & 3);
                    *reinterpret_cast<uint4 *>(a_row + ((c ^ (r & 7)) << 4)) = wv[c];
                }
                fence_async_proxy();                     // generic-proxy stores -> visible to the MMA
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->masked[s]);
            }
            if (kp == KBP - 1 || it == nkb - 1) {        // the panel ends: hand its buffer back to the decoders
                panel_bits_ready();
                if (!ok) break;
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->bits_free[buf]);
            }
            if (++s == stages) { s = 0; full_parity ^= 1; }
            if (++kp == KBP) { kp = 0; ++P; }
        }
        if (!DW && kp != 0) { kp = 0; ++P; }             // a tile's last panel may be short

        // ------------------------------------------------------------- epilogue (same warps)
        if (ok) ok = mbar_wait(&ctl->accum, (uint32_t)(tile_n & 1), abort_flag, status, DEV_TIMEOUT_ACCUM);
        if (ok && DW) {                                  // the index bits of the tile's two 256-column panels
            ok = mbar_wait(&ctl->bits_ready[0], (P >> 1) & 1, abort_flag, status, DEV_TIMEOUT_FULL);
            if (ok) ok = mbar_wait(&ctl->bits_ready[1], (P >> 1) & 1, abort_flag, status, DEV_TIMEOUT_FULL);
        }
        // The lanes of a warp leave a barrier wait one by one (each polls for itself); the tensor-memory loads of the
        // epilogue are warp-wide instructions and need the warp back together, with one verdict for all its lanes: a
        // lane whose wait failed has raised the block's abort flag before, and the lanes read the flag together.
        // (A vote instead of the flag was measured 8 us slower on the 35 us convolution layer.)
        __syncwarp();
        const bool epi_ok = ok && *abort_flag == 0;
        if (epi_ok && PERSIST) {
            // The operand stages already belong to the next tile: every warp moves its 32 output features x 16
            // (fp32: 8) batch columns through 1 KB of its own and stores 16-byte pieces, 64 (128) bytes of a row of Y
            // per four (eight) lanes.
            tc_fence_after();
            const bool out32 = y_dtype == LRBI_Y_F32;
            const int quad = warp & 3, half = mw >> 2;   // tensor-memory lanes this warp may read; its half of the columns
            uint8_t *st = epi_stage + mw * 1024;
            const int f0 = o0 + quad * 32;               // first output feature of the warp
            const bool vec_ok = (g.rows % (out32 ? 4 : 8)) == 0;
            for (int ch = 0; ch < BN / 32; ++ch) {
                const int cl = half * (BN / 2) + ch * 16;            // first batch column of the chunk inside the tile
                uint32_t v[16];
                tmem_ld16(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)cl, v);
                tmem_ld_wait();
                if (DW) {
                    // row quad*32+lane of the block, columns cl .. cl+15: panel cl/256, word (cl%256)/32; column e of a
                    // word sits at bit 8 (e%4) + 7 - e/4 (the order the decoders write)
                    const uint32_t wbits = row_bits[(cl >> 8) * (TC_BM * PW) + (quad * 32 + lane) * PW + ((cl & 255) >> 5)];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int e = (cl & 31) + j;
                        if (!((wbits >> (8 * (e & 3) + 7 - (e >> 2))) & 1u)) v[j] = 0u;
                    }
                }
                if (!out32) {
                    uint16_t *s16 = reinterpret_cast<uint16_t *>(st);
#pragma unroll
                    for (int j = 0; j < 16; ++j) s16[j * 32 + lane] = f32_to_bf16_rne(__uint_as_float(v[j]));
                    __syncwarp();
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int idx = lane + 32 * u, col = idx >> 2, part = idx & 3;
                        const int bb = b0 + cl + col, ff = f0 + part * 8;
                        if (bb < batch && ff < g.rows) {
                            uint16_t *dst = reinterpret_cast<uint16_t *>(Y) + (size_t)bb * g.rows + ff;
                            if (vec_ok && ff + 8 <= g.rows) *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(st + col * 64 + part * 16);
                            else for (int e = 0; e < min(8, g.rows - ff); ++e) dst[e] = s16[col * 32 + part * 8 + e];
                        }
                    }
                    __syncwarp();
                } else {
                    float *s32 = reinterpret_cast<float *>(st);
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) s32[j * 32 + lane] = __uint_as_float(v[hh * 8 + j]);
                        __syncwarp();
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int idx = lane + 32 * u, col = idx >> 3, part = idx & 7;
                            const int bb = b0 + cl + hh * 8 + col, ff = f0 + part * 4;
                            if (bb < batch && ff < g.rows) {
                                float *dst = reinterpret_cast<float *>(Y) + (size_t)bb * g.rows + ff;
                                if (vec_ok && ff + 4 <= g.rows) *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(st + col * 128 + part * 16);
                                else for (int e = 0; e < min(4, g.rows - ff); ++e) dst[e] = s32[col * 32 + part * 4 + e];
                            }
                        }
                        __syncwarp();
                    }
                }
            }
            // this warp has read its part of tensor memory: tell the leader's MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (rank == 0) mbar_arrive(&ctl->tmem_free);
                else mbar_arrive_remote(&ctl->tmem_free, 0);
                if (DW) { mbar_arrive(&ctl->bits_free[0]); mbar_arrive(&ctl->bits_free[1]); }   // both index panels are used up
            }
            if (DW) P += 2;
        }
        if (epi_ok && !PERSIST) {
            // K split: the kernel that adds the partial sums up may be set up from here on (it waits for this grid's end)
            if (partials != nullptr && mt == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
            tc_fence_after();
            // All MMAs have completed.  In tensor memory a lane is an output feature and a column a batch row, so the 32
            // lanes of a warp hold 32 consecutive outputs of one row of Y: every column goes out as one 64-byte (fp32:
            // 128-byte) warp store straight from the registers, whole sectors, no staging and no meeting of the warps.
            const bool out32 = partials != nullptr || y_dtype == LRBI_Y_F32;
            const int quad = warp & 3;                   // tensor-memory lanes this warp may read
            const int half = mw >> 2;                    // which half of the tile's columns
            constexpr int HC = BN >= 32 ? BN / 2 : BN;   // columns per warp (a 16-column tile: the first four warps only)
            const int o = o0 + quad * 32 + lane;         // this lane's output feature
            const bool o_ok = o < g.rows;
            uint8_t *dst_base = partials ? reinterpret_cast<uint8_t *>(partials + (long long)blockIdx.z * batch * g.rows)
                                         : reinterpret_cast<uint8_t *>(Y);
            if (BN >= 32 || half == 0) {
#pragma unroll 1
                for (int ch = 0; ch < HC / 16; ++ch) {
                    const int cl = half * HC + ch * 16;  // first batch column of the chunk inside the tile
                    if (b0 + cl >= batch) break;         // (the whole warp) the rest of the tile lies outside the batch
                    uint32_t v[16];
                    tmem_ld16(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)cl, v);
                    tmem_ld_wait();
                    const long long row0 = (long long)(b0 + cl) * g.rows + o;
                    if (out32) {
                        float *dst = reinterpret_cast<float *>(dst_base) + row0;
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (o_ok && b0 + cl + j < batch) dst[(long long)j * g.rows] = __uint_as_float(v[j]);
                    } else {
                        uint16_t *dst = reinterpret_cast<uint16_t *>(dst_base) + row0;
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (o_ok && b0 + cl + j < batch) dst[(long long)j * g.rows] = f32_to_bf16_rne(__uint_as_float(v[j]));
                    }
                }
            }
        }
        }                                                // the block's tiles
    }

    tc_fence_before();
    __syncthreads();
    __syncwarp();                    // (warp-wide instructions follow; a warp's lanes may have come here on different paths)
    if (PAIR) cluster_sync_all();    // neither CTA frees tensor memory or leaves while the other may still touch it
    if (warp == 1) {
        tc_fence_after();
        if (PAIR) tmem_dealloc2(tmem_d, TMEM_COLS);
        else tmem_dealloc(tmem_d, TMEM_COLS);
    }
}

// The give-up path of the pipeline's bounded wait, exercised on its own: one thread waits, with a short
// limit, on a barrier that nothing arrives at.  The wait runs out, the code lands in the status word and
// the kernel returns normally.
__global__ void bounded_wait_selftest_kernel(long long limit_cycles, int *status)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(&bar, 0, &abort_flag, status, DEV_TIMEOUT_SELFTEST, limit_cycles);
    }
}

lrbi_status launch_bounded_wait_selftest(unsigned limit_us, cudaStream_t s)
{
    int *status = device_status_ptr();
    if (!status) return LRBI_ERR_CUDA;
    if (limit_us > 100000u) limit_us = 100000u;          // a tenth of a second at most
    bounded_wait_selftest_kernel<<<1, 32, 0, s>>>((long long)limit_us * 2000ll, status);   // about 2 cycles per ns
    count_launch();
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

// Sum of the K-split partial results: Y[b][o] = sum_z partials[z][b][o].
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float *__restrict__ partials, int splits, long long n, void *__restrict__ Y, int y_dtype)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    // launched while the product kernel is still draining (programmatic dependent launch): its writes are
    // visible only after this wait
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (idx >= n) return;
    float acc = 0.f;
    for (int z = 0; z < splits; ++z) acc += partials[(long long)z * n + idx];
    if (y_dtype == LRBI_Y_F32) reinterpret_cast<float *>(Y)[idx] = acc;
    else reinterpret_cast<uint16_t *>(Y)[idx] = f32_to_bf16_rne(acc);
}

// --------------------------------------------------------------------------------------
// host side
// --------------------------------------------------------------------------------------
constexpr int TC_MAX_RANK = 256;

bool gemm_tc_supported(const Geo &g, int batch)
{
    if (batch < 1 || g.k > TC_MAX_RANK) return false;
    if ((g.cols % 8) != 0) return false;                                   // 16-byte rows for TMA and vector loads
    if (!(g.gr == 1 || (g.tm % TC_BM) == 0)) return false;                 // 128 rows inside one tile row
    if (!(g.gc == 1 || (g.tn % TC_BK) == 0)) return false;                 // a K block inside one tile column
    return true;
}

// Library-owned buffer for K-split partial sums, one per device, grown on demand (under the library lock).
struct Workspace {
    float *ptr = nullptr;
    size_t bytes = 0;
};
static Workspace g_ws[LRBI_MAX_DEVICES];

static float *workspace(int dev, size_t bytes)
{
    std::lock_guard<std::mutex> lock(lib_mutex());
    Workspace &w = g_ws[dev];
    if (w.bytes < bytes) {
        if (w.ptr) cudaFree(w.ptr);
        w.ptr = nullptr; w.bytes = 0;
        if (cudaMalloc(&w.ptr, bytes) != cudaSuccess) { w.ptr = nullptr; return nullptr; }
        w.bytes = bytes;
    }
    return w.ptr;
}

// Everything the host decides about one launch of the tensor-core kernel: which instantiation runs, how
// the reduction over K is cut, how many operand stages fit.  One function, so that the launcher, the
// scratch-size query and the plan query of the C ABI cannot disagree.
struct TcPlan {
    int bn;              // batch columns per output tile
    int pw;              // index words per panel row (8: 256-column panels, 2: 64-column panels)
    bool pair;           // CTA pairs (cta_group::2)
    int row_blocks;      // 128-row blocks along grid y (pair mode: an even number, two per cluster)
    int splits;          // blocks along the reduction (grid z)
    int kb_per_split;    // K blocks per split (a multiple of 4: splits start on panel boundaries)
    int stages;          // operand stages in shared memory
    size_t smem;         // dynamic shared memory per block
    size_t scratch;      // bytes of fp32 partial sums (0 when K is not split)
    bool persist;        // one pair per two SMs walks the output tiles (two-accumulator pairs, K not split)
    int pairs;           // persist: pairs in the grid
};

// `force`: 0 = choose by shape; 1 = CTA pairs with one accumulator (256 batch columns per pair);
// 2 = CTA pairs with two accumulators (512 batch columns per pair); 3 = CTA pairs with one accumulator of 192 columns.
static bool make_tc_plan(const Geo &g, int batch, int sm_count, int force, TcPlan *out)
{
    if (!gemm_tc_supported(g, batch)) return false;
    TcPlan p;
    // Measured on B200 (K = 4096, microseconds; single CTAs with 128-column tiles / pairs with one / with two
    // accumulators): 1024 x 4096 outputs 88 / 68 / 64; 4096 x 4096 283 / 174 / 125; 16384 x 4096 (the FFN
    // layer) - / 568 / 408.  So: pairs whenever there are two 128-row blocks to pair and more than 128
    // batch rows, two accumulators whenever the batch has more than 256 rows.
    p.pair = force ? true : (batch > 128 && g.rows > TC_BM);
    p.bn = batch <= 16 ? 16 : batch <= 32 ? 32 : batch <= 64 ? 64 : 128;
    if (p.pair) p.bn = force == 1 ? 256 : force == 2 ? 512 : force == 3 ? 192 : (batch > 256 ? 512 : 256);
    // Few rows and a long batch (a lowered convolution): tiles of 512 batch rows leave most SMs idle.  When the
    // 192-row tiles fit the chip in one wave of pairs they win (measured, 256 x 2304 weights: 12544 batch rows
    // 33.9 us against 48.1, 3136 rows 25.6 against 31.7; 300 x 1000 weights, 777 rows 19.4 against 25.4).
    if (p.pair && force == 0 && batch > 256 &&
        (long long)((batch + 191) / 192) * ((g.rows + 2 * TC_BM - 1) / (2 * TC_BM)) <= sm_count / 2) p.bn = 192;
    // index words per panel row: 256-column panels when every panel then lies inside one tile
    p.pw = (g.gc == 1 || (g.tn % 256) == 0) ? 8 : 2;
    const int nkb = (g.cols + TC_BK - 1) / TC_BK;
    p.row_blocks = p.pair ? 2 * ((g.rows + 2 * TC_BM - 1) / (2 * TC_BM)) : (g.rows + TC_BM - 1) / TC_BM;
    const long long tiles = (long long)((batch + p.bn - 1) / p.bn) * p.row_blocks;
    // Split K when the output tiles alone cannot occupy the chip.
    int splits = 1;
    if (!p.pair) {
        if (batch <= p.bn && tiles < 2 * sm_count) {  // one batch tile: the small-batch, bandwidth-bound case
            splits = (int)((2 * sm_count + tiles - 1) / tiles);
            splits = splits > nkb / 4 ? (nkb / 4 > 0 ? nkb / 4 : 1) : splits;   // at least 4 K blocks per split
            if (splits > 32) splits = 32;
        }
    } else {
        // A lone block advances about one K block per microsecond (its ring of stages is bound by latency, not
        // by the tensor pipe), so cutting K pays when blocks are few -- as long as writing and re-reading the
        // fp32 partial sums (about 5 bytes per nanosecond) costs less than half of the time it saves.
        const long long slots = (long long)sm_count * ((p.bn == 512 || p.bn == 192) ? 1 : 2);   // blocks resident at once
        if (tiles < slots) {
            int sp = (int)(slots / tiles);
            if (sp > nkb / 8) sp = nkb / 8;           // at least 8 K blocks per split
            if (sp > 32) sp = 32;
            while (sp > 1) {
                const double partial_us = (double)sp * batch * g.rows * 8.0 / 5.0e6;
                const double saved_us = (double)(nkb - (nkb + sp - 1) / sp);
                if (partial_us <= 0.5 * saved_us) break;
                --sp;
            }
            splits = sp < 1 ? 1 : sp;
        }
    }
    int kb_per_split = (nkb + splits - 1) / splits;
    kb_per_split = (kb_per_split + 3) / 4 * 4;                               // splits start on panel boundaries
    p.splits = (nkb + kb_per_split - 1) / kb_per_split;                      // no empty split
    p.kb_per_split = kb_per_split;
    p.scratch = p.splits > 1 ? (size_t)p.splits * batch * g.rows * sizeof(float) : 0;

    // As many stages as let two blocks share an SM (at least three); if two cannot fit (large ranks need
    // more room for planes and factor staging), one block with up to six stages.  Two resident blocks
    // overlap one's epilogue and hand-overs with the other's MMAs and double the copies in flight.
    // (an SM has 228 KB of shared memory; each resident block also reserves 1 KB)
    const size_t b_stage = (size_t)(p.pair ? p.bn / 2 : p.bn) * TC_BK * 2;
    const size_t dgroup_words = (size_t)g.kw * 32 * (p.pw == 8 ? 12 : p.pw) + (size_t)p.pw * 32 * g.kw + (size_t)TC_BM * g.kw;
    p.persist = p.pair && p.bn == 512 && p.splits == 1;
    p.pairs = 0;
    if (p.persist) {
        const long long tiles2 = (long long)((batch + 511) / 512) * (p.row_blocks / 2);
        p.pairs = (int)(tiles2 < sm_count / 2 ? tiles2 : sm_count / 2);
        if (p.pairs < 1) p.persist = false;
    }
    const size_t extras = ((size_t)2 * TC_BM * p.pw + tc_decode_groups(p.bn) * dgroup_words) * 4 + sizeof(TcCtl) +
                          (p.persist ? TC_MASK_WARPS * 1024 : 0);
    const size_t per_stage = TC_A_STAGE_BYTES + b_stage;
    const size_t half_sm = 113 * 1024, whole_sm = 224 * 1024;
    int stages = (int)((half_sm - extras) / per_stage);
    // (a grid of no more blocks than SMs has an SM per block anyway: deeper rings for those)
    if (extras > half_sm || stages < 3 || tiles * p.splits <= sm_count || p.bn == 192) stages = (int)((whole_sm - extras) / per_stage);
    if (stages > 6) stages = 6;
    if (stages < 2) return false;
    p.stages = stages;
    p.smem = (size_t)stages * per_stage + extras;
    const unsigned nbt = (unsigned)((batch + p.bn - 1) / p.bn);
    if ((p.pair ? p.row_blocks / 2 : p.row_blocks) > 65535 || p.splits > 65535 || nbt > 0x3FFFFFFFu) return false;
    *out = p;
    return true;
}

static int device_sm_count(int *dev_out)
{
    int dev = 0, sm_count = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= LRBI_MAX_DEVICES) { *dev_out = -1; return sm_count; }
    cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
    *dev_out = dev;
    return sm_count;
}

template <int BN, int PW, bool PAIR, bool PERSIST, bool DW = false, bool MNM = false>
static lrbi_status launch_tc(const Geo &g, const TcPlan &plan, int dev, const uint16_t *W, const uint32_t *ip,
                             const uint32_t *iz, const uint16_t *X, int batch, void *Y, int y_dtype,
                             cudaStream_t s, float *partials, const TileRanks &rk, const Geo *index_geo = nullptr)
{
    const Geo gi = index_geo ? *index_geo : g;
    EncodeTiledFn encode = get_encode_fn();
    if (!encode) { note_cuda_error(-1); return LRBI_ERR_CUDA; }
    CUtensorMap map;
    // K-major operands: [rows of the operand][K]; MN-major (MNM): [K][rows of the operand], boxes of 64 x 64
    const cuuint64_t dims[2] = {(cuuint64_t)(MNM ? batch : g.cols), (cuuint64_t)(MNM ? g.cols : batch)};
    const cuuint64_t strides[1] = {(cuuint64_t)(MNM ? batch : g.cols) * 2};
    const cuuint32_t box[2] = {TC_BK, MNM ? TC_BK : PAIR ? (BN < 256 ? BN / 2 : 128) : BN};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<uint16_t *>(X), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { note_cuda_error((int)r); return LRBI_ERR_CUDA; }
    CUtensorMap wmap;
    const cuuint64_t wdims[2] = {(cuuint64_t)(MNM ? g.rows : g.cols), (cuuint64_t)(MNM ? g.cols : g.rows)};
    const cuuint64_t wstrides[1] = {(cuuint64_t)(MNM ? g.rows : g.cols) * 2};
    const cuuint32_t wbox[2] = {TC_BK, MNM ? TC_BK : TC_BM};
    r = encode(&wmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<uint16_t *>(W), wdims, wstrides, wbox, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { note_cuda_error((int)r); return LRBI_ERR_CUDA; }

    auto kern = gemm_tc_kernel<BN, PW, PAIR, PERSIST, DW, MNM>;
    {
        // the opt-in to more than 48 KB of dynamic shared memory is a per-device attribute of the function
        static bool attr_done[LRBI_MAX_DEVICES] = {false};
        std::lock_guard<std::mutex> lock(lib_mutex());
        if (!attr_done[dev]) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024);
            if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
            attr_done[dev] = true;
        }
    }
    const unsigned nbt = (unsigned)((batch + BN - 1) / BN);
    dim3 grid(PAIR ? 2 * nbt : nbt, (unsigned)(PAIR ? plan.row_blocks / 2 : plan.row_blocks), (unsigned)plan.splits);
    if (PERSIST) grid = dim3(2u * (unsigned)plan.pairs, 1, 1);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(tc_threads(BN));
    cfg.dynamicSmemBytes = plan.smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;      // the pair must lie along x: other shapes are refused
    attr[0].val.clusterDim.x = PAIR ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int *status = device_status_ptr();
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, map, wmap, g, gi, rk, ip, iz, batch, Y, y_dtype, partials, plan.kb_per_split, plan.stages, status);
    count_launch();
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    if (plan.splits > 1) {
        const long long n = (long long)batch * g.rows;
        // the reduction's blocks may be set up while the product kernel's last blocks finish; they wait for its
        // completion before they read (griddepcontrol.wait)
        cudaLaunchConfig_t rcfg = {};
        rcfg.gridDim = dim3((unsigned)((n + 255) / 256));
        rcfg.blockDim = dim3(256);
        rcfg.stream = s;
        cudaLaunchAttribute rattr[1];
        rattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        rattr[0].val.programmaticStreamSerializationAllowed = 1;
        rcfg.attrs = rattr;
        rcfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&rcfg, splitk_reduce_kernel, (const float *)partials, (int)plan.splits, n, Y, y_dtype);
        count_launch();
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    }
    return LRBI_OK;
}

// `fixed_scratch` != nullptr: the caller forbids allocation, partial sums go there (fixed_bytes) or nowhere.
static lrbi_status run_tc(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                          const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s,
                          float *fixed_scratch, size_t fixed_bytes, int force = 0, const TileRanks *ranks = nullptr)
{
    const TileRanks rk = ranks ? *ranks : TileRanks{nullptr, nullptr, nullptr};
    if (!gemm_tc_supported(g, batch)) return LRBI_ERR_UNSUPPORTED;    // shape errors come before device errors
    int dev = -1;
    const int sm_count = device_sm_count(&dev);
    if (dev < 0) return LRBI_ERR_CUDA;
    TcPlan plan;
    if (!make_tc_plan(g, batch, sm_count, force, &plan)) return LRBI_ERR_UNSUPPORTED;
    if (fixed_scratch && plan.scratch > fixed_bytes) return LRBI_ERR_TOO_LARGE;   // before any launch
    if (!device_status_ptr()) return LRBI_ERR_CUDA;
    float *partials = nullptr;
    if (plan.scratch) {
        partials = fixed_scratch ? fixed_scratch : workspace(dev, plan.scratch);
        if (!partials) { note_cuda_error((int)cudaErrorMemoryAllocation); return LRBI_ERR_CUDA; }
    }
#define LRBI_TC_CASE(BN_, PW_, PAIR_) \
    if (plan.bn == BN_ && plan.pw == PW_ && plan.pair == PAIR_ && !plan.persist) \
        return launch_tc<BN_, PW_, PAIR_, false>(g, plan, dev, W, ip, iz, X, batch, Y, y_dtype, s, partials, rk);
    LRBI_TC_CASE(16, 8, false) LRBI_TC_CASE(16, 2, false)
    LRBI_TC_CASE(32, 8, false) LRBI_TC_CASE(32, 2, false)
    LRBI_TC_CASE(64, 8, false) LRBI_TC_CASE(64, 2, false)
    LRBI_TC_CASE(128, 8, false) LRBI_TC_CASE(128, 2, false)
    LRBI_TC_CASE(192, 8, true) LRBI_TC_CASE(192, 2, true)
    LRBI_TC_CASE(256, 8, true) LRBI_TC_CASE(256, 2, true)
    LRBI_TC_CASE(512, 8, true) LRBI_TC_CASE(512, 2, true)
    if (plan.persist && plan.pw == 8) return launch_tc<512, 8, true, true>(g, plan, dev, W, ip, iz, X, batch, Y, y_dtype, s, partials, rk);
    if (plan.persist && plan.pw == 2) return launch_tc<512, 2, true, true>(g, plan, dev, W, ip, iz, X, batch, Y, y_dtype, s, partials, rk);
#undef LRBI_TC_CASE
    return LRBI_ERR_UNSUPPORTED;
}

lrbi_status launch_gemm_tc(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                           const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s, int force, const TileRanks *ranks)
{
    return run_tc(g, W, ip, iz, X, batch, Y, y_dtype, s, nullptr, 0, force, ranks);
}

// dW = (dY^T X) .* Ia on the persistent pair kernel: `g` describes the contraction (rows = cols of the layer, read from
// Xt [layer cols][batch]; reduction over the batch; "batch" = rows of the layer, read from dYt [layer rows][batch]), `gi`
// the index as the output tile sees it (the layer's layout transposed).  Returns LRBI_ERR_UNSUPPORTED when the shape
// does not run on that kernel (the caller then takes another route).
// mn_major: the operands are X [batch][layer cols] and dY [batch][layer rows] as the layer has them (the M and the N
// index run along memory, K across rows); no transposed copies are needed.  Needs layer rows % 8 == 0.
lrbi_status launch_gemm_tc_dw(const Geo &g, const Geo &gi, const uint16_t *Xt, const uint32_t *ip_t, const uint32_t *iz_t,
                              const uint16_t *dYt, int out_rows, void *dW, int dtype, cudaStream_t s, bool mn_major)
{
    if (mn_major && ((out_rows % 8) != 0 || (g.rows % 8) != 0)) return LRBI_ERR_UNSUPPORTED;   // 16-byte rows for the copies
    if (!gemm_tc_supported(g, out_rows) || gi.k > TC_MAX_RANK) return LRBI_ERR_UNSUPPORTED;
    if (!(gi.gr == 1 || (gi.tm % TC_BM) == 0) || !(gi.gc == 1 || (gi.tn % 256) == 0)) return LRBI_ERR_UNSUPPORTED;
    int dev = -1;
    const int sm_count = device_sm_count(&dev);
    if (dev < 0) return LRBI_ERR_CUDA;
    Geo gs = g;                                          // shared memory is sized for the index's rank
    gs.k = gi.k; gs.kw = gi.kw;
    TcPlan plan;
    if (!make_tc_plan(gs, out_rows, sm_count, 2, &plan) || !plan.persist || plan.pw != 8) return LRBI_ERR_UNSUPPORTED;
    if (!device_status_ptr()) return LRBI_ERR_CUDA;
    const TileRanks none = {nullptr, nullptr, nullptr};
    if (mn_major) return launch_tc<512, 8, true, true, true, true>(gs, plan, dev, Xt, ip_t, iz_t, dYt, out_rows, dW, dtype, s, nullptr, none, &gi);
    return launch_tc<512, 8, true, true, true>(gs, plan, dev, Xt, ip_t, iz_t, dYt, out_rows, dW, dtype, s, nullptr, none, &gi);
}

bool gemm_tc_plan(const Geo &g, int batch, int force, lrbi_gemm_plan *out)
{
    int dev = -1;
    const int sm_count = device_sm_count(&dev);
    TcPlan p;
    if (!make_tc_plan(g, batch, sm_count, force, &p)) return false;
    out->batch_tile = p.bn;
    out->cta_pair = p.pair ? 1 : 0;
    out->panel_columns = p.pw * 32;
    out->k_splits = p.splits;
    out->stages = p.stages;
    out->scratch_bytes = (uint64_t)p.scratch;
    return true;
}

// --------------------------------------------------------------------------------------
// No-allocation variant: K-split partial sums live in a fixed array inside the library image.
// --------------------------------------------------------------------------------------
// The array belongs to the module: each GPU that loads the library carries its own copy until the
// process ends.  In host code this name is only a handle for the runtime, never a device address;
// the address a kernel may use comes from cudaGetSymbolAddress, asked once per device.
static __device__ __align__(256) float g_static_scratch[LRBI_STATIC_SCRATCH_BYTES / sizeof(float)];
static float *g_static_scratch_ptr[LRBI_MAX_DEVICES] = {nullptr};

static float *static_scratch_ptr()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= LRBI_MAX_DEVICES) return nullptr;
    std::lock_guard<std::mutex> lock(lib_mutex());
    if (!g_static_scratch_ptr[dev]) {                    // first call on this device (it is the current one)
        void *p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) { note_cuda_error((int)e); return nullptr; }
        g_static_scratch_ptr[dev] = static_cast<float *>(p);
    }
    return g_static_scratch_ptr[dev];
}

size_t gemm_tc_scratch_bytes(const Geo &g, int batch)
{
    int dev = -1;
    const int sm_count = device_sm_count(&dev);
    TcPlan p;
    return make_tc_plan(g, batch, sm_count, 0, &p) ? p.scratch : 0;
}

lrbi_status launch_gemm_tc_static(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                                  const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s)
{
    if (!gemm_tc_supported(g, batch)) return LRBI_ERR_UNSUPPORTED;
    if (gemm_tc_scratch_bytes(g, batch) > LRBI_STATIC_SCRATCH_BYTES) return LRBI_ERR_TOO_LARGE;   // before any launch
    float *scratch = static_scratch_ptr();
    if (!scratch) return LRBI_ERR_CUDA;
    return run_tc(g, W, ip, iz, X, batch, Y, y_dtype, s, scratch, LRBI_STATIC_SCRATCH_BYTES);
}

}  // namespace lrbi
