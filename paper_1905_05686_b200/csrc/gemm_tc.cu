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
// Warp roles in a 320-thread block:
//   warp 0      lane 0 issues the TMA loads of X (cp.async.bulk.tensor, 128B swizzle, zero fill
//               outside the matrix) into the B stages.
//   warp 1      allocates tensor memory; lane 0 issues tcgen05.mma for each filled stage and
//               commits the stage's "empty" barrier; finally commits the accumulator barrier.
//   warps 2-9   mask producers.  Each thread owns one 16-byte chunk column (8 weights) and four
//               rows of the 128 x 64 block: it loads W with coalesced 16-byte loads, one K block
//               ahead, decodes the eight index bits per row from the row words of Ip and the
//               column words of Iz ((ip & iz) != 0, Eq. 3), zeroes pruned bf16 values and stores
//               the chunk at its swizzled position in the A stage.  Writes are made visible to
//               the tensor core with fence.proxy.async before the stage barrier is signalled.
//               After the last K block the same warps run the epilogue: tcgen05.ld of their
//               32-lane quadrant, conversion, stores to Y (or fp32 partial sums when K is split).
//
// Every barrier wait is bounded by a wall-clock limit.  A wait that runs out records a code in
// the device status word and raises a block-wide abort flag; every role then leaves its loop, the
// TMA thread drains (bounded) the copies it has in flight, and tensor memory is freed before exit.
#include <cuda.h>

#include "lrbi_common.cuh"

namespace lrbi {

constexpr int TC_THREADS = 320;
constexpr int TC_BM = 128;                 // rows of W per block (MMA M)
constexpr int TC_BK = 64;                  // columns per stage: 64 bf16 = one 128-byte swizzle row
constexpr int TC_A_STAGE_BYTES = TC_BM * TC_BK * 2;
constexpr int TC_MASK_WARPS = 8;
constexpr unsigned long long TC_WAIT_LIMIT_NS = 2000000000ull;   // 2 s

// ------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false if the block is aborting or the limit ran out (then it records
// `code` and raises the abort flag).
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                          int *status, int code)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    int spins = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((++spins & 255) == 0 && global_ns() - t0 > TC_WAIT_LIMIT_NS) {
            atomicCAS(status, 0, code);
            *abort_flag = 1;
            __threadfence_block();
            return false;
        }
    }
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}

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
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = bn.
__host__ __device__ constexpr uint32_t make_idesc(int bn)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
}

__device__ __forceinline__ uint4 ldg_w(const uint16_t *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Shared-memory bookkeeping that follows the operand stages.
struct TcCtl {
    uint64_t full[8];
    uint64_t empty[8];
    uint64_t accum;
    uint32_t tmem_base;
    int abort_flag;
};

// --------------------------------------------------------------------------------------
// kernel
// --------------------------------------------------------------------------------------
// grid = (batch tiles, row tiles of 128, K splits).  When gridDim.z > 1 the block writes fp32
// partial sums to `partials` [split][batch][rows]; a second kernel adds them up.
template <int BN, int KW>
__global__ void __launch_bounds__(TC_THREADS)
gemm_tc_kernel(const __grid_constant__ CUtensorMap x_map, Geo g, const uint16_t *__restrict__ W,
               const uint32_t *__restrict__ ip, const uint32_t *__restrict__ iz, int batch,
               void *__restrict__ Y, int y_dtype, float *__restrict__ partials, int kb_per_split,
               int stages, int *status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int B_STAGE_BYTES = BN * TC_BK * 2;
    constexpr int TMEM_COLS = BN < 32 ? 32 : BN;
    uint8_t *a_base = smem;
    uint8_t *b_base = smem + (size_t)stages * TC_A_STAGE_BYTES;
    TcCtl *ctl = reinterpret_cast<TcCtl *>(b_base + (size_t)stages * B_STAGE_BYTES);
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b0 = blockIdx.x * BN;                      // first batch row of this block
    const int o0 = blockIdx.y * TC_BM;                   // first row of W of this block
    const int nkb_total = (g.cols + TC_BK - 1) / TC_BK;
    const int kb_begin = blockIdx.z * kb_per_split;
    const int kb_end = min(nkb_total, kb_begin + kb_per_split);
    const int nkb = kb_end - kb_begin;                   // >= 1 by construction of the grid

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&ctl->full[s], 1 + TC_MASK_WARPS);
            mbar_init(&ctl->empty[s], 1);
        }
        mbar_init(&ctl->accum, 1);
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&ctl->tmem_base, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = ctl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------- TMA producer (X tiles)
        if (lane == 0) {
            int armed = 0;
            for (int it = 0; it < nkb; ++it) {
                const int s = it % stages, round = it / stages;
                if (round > 0 && !mbar_wait(&ctl->empty[s], (round - 1) & 1, abort_flag, status, DEV_TIMEOUT_EMPTY)) break;
                mbar_arrive_expect_tx(&ctl->full[s], B_STAGE_BYTES);
                tma_load_2d(b_base + (size_t)s * B_STAGE_BYTES, &x_map, &ctl->full[s], (kb_begin + it) * TC_BK, b0);
                armed = it + 1;
            }
            if (*abort_flag) {
                // drain: copies already issued must land before this block's shared memory goes away.
                // A full barrier also needs the mask warps' arrivals, which may never come now, so
                // the wait is on elapsed time only (bounded), long enough for any copy in flight.
                const unsigned long long t0 = global_ns();
                while (armed > 0 && global_ns() - t0 < 2000000ull) { }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(BN);
            bool ok = true;
            for (int it = 0; it < nkb && ok; ++it) {
                const int s = it % stages, round = it / stages;
                ok = mbar_wait(&ctl->full[s], round & 1, abort_flag, status, DEV_TIMEOUT_FULL);
                if (!ok) break;
                tc_fence_after();
                const uint64_t da = make_sw128_desc(smem_u32(a_base + (size_t)s * TC_A_STAGE_BYTES));
                const uint64_t db = make_sw128_desc(smem_u32(b_base + (size_t)s * B_STAGE_BYTES));
#pragma unroll
                for (int k4 = 0; k4 < TC_BK / 16; ++k4) {
                    // 16 bf16 = 32 bytes further along K inside the swizzled row: +2 in address units
                    umma_bf16(tmem_d, da + (uint64_t)(2 * k4), db + (uint64_t)(2 * k4), idesc, (it | k4) ? 1u : 0u);
                }
                umma_commit(&ctl->empty[s]);            // frees the stage when these MMAs have read it
            }
            if (ok) umma_commit(&ctl->accum);           // accumulator complete
        }
    } else {
        // ------------------------------------------------------------- mask producers
        const int mt = threadIdx.x - 64;                // 0..255
        const int cc = mt & 7;                          // 16-byte chunk column inside the 128-byte row
        const int rb = mt >> 3;                         // rows rb, rb+32, rb+64, rb+96
        const uint32_t tail = tail_mask(g.k);
        const int tr = o0 / g.tm;                       // the 128 rows lie in one tile row
        const int i0 = o0 - tr * g.tm;

        uint32_t ipv[4][KW];
        int tc_prev = -1;
        uint4 wnext[4];
        uint4 znext[2 * KW];

        auto fetch = [&](int it, uint4 (&wv)[4], uint4 (&zv)[2 * KW]) {
            const int c = (kb_begin + it) * TC_BK + cc * 8;          // first of this thread's 8 columns
            const bool colok = it < nkb && c < g.cols;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int o = o0 + rb + 32 * q;
                wv[q] = (colok && o < g.rows) ? ldg_w(W + (long long)o * g.cols + c) : make_uint4(0, 0, 0, 0);
            }
            if (colok) {
                const int tc = c / g.tn, j = c - tc * g.tn;
                const uint4 *zp = reinterpret_cast<const uint4 *>(iz + (((long long)tr * g.gc + tc) * g.tn + j) * KW);
#pragma unroll
                for (int v = 0; v < 2 * KW; ++v) zv[v] = __ldg(zp + v);
            } else {
#pragma unroll
                for (int v = 0; v < 2 * KW; ++v) zv[v] = make_uint4(0, 0, 0, 0);
            }
        };
        fetch(0, wnext, znext);

        bool ok = true;
        for (int it = 0; it < nkb && ok; ++it) {
            const int s = it % stages, round = it / stages;
            uint4 wcur[4], zcur[2 * KW];
#pragma unroll
            for (int q = 0; q < 4; ++q) wcur[q] = wnext[q];
#pragma unroll
            for (int v = 0; v < 2 * KW; ++v) zcur[v] = znext[v];
            fetch(it + 1, wnext, znext);                 // next K block in flight while this one is masked

            const int c = (kb_begin + it) * TC_BK + cc * 8;
            const int tc = min(c, g.cols - 1) / g.tn;
            if (tc != tc_prev) {                         // row words of Ip change with the tile column
                tc_prev = tc;
                const long long tile = (long long)tr * g.gc + tc;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int i = i0 + rb + 32 * q;
#pragma unroll
                    for (int w = 0; w < KW; ++w) {
                        uint32_t v = (i < g.tm) ? __ldg(ip + (tile * g.tm + i) * KW + w) : 0u;
                        if (w == KW - 1) v &= tail;
                        ipv[q][w] = v;
                    }
                }
            }
            uint32_t izv[8][KW];
#pragma unroll
            for (int v = 0; v < 2 * KW; ++v) {
                const uint32_t zz[4] = {zcur[v].x, zcur[v].y, zcur[v].z, zcur[v].w};
#pragma unroll
                for (int t = 0; t < 4; ++t) izv[(v * 4 + t) / KW][(v * 4 + t) % KW] = zz[t];
            }

            if (round > 0) ok = mbar_wait(&ctl->empty[s], (round - 1) & 1, abort_flag, status, DEV_TIMEOUT_EMPTY);
            if (!ok) break;

            uint8_t *a_stage = a_base + (size_t)s * TC_A_STAGE_BYTES;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = rb + 32 * q;
                uint32_t ww[4] = {wcur[q].x, wcur[q].y, wcur[q].z, wcur[q].w};
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    uint32_t lo = 0, hi = 0;
#pragma unroll
                    for (int w = 0; w < KW; ++w) {
                        lo |= ipv[q][w] & izv[2 * h][w];
                        hi |= ipv[q][w] & izv[2 * h + 1][w];
                    }
                    const uint32_t keep = (lo ? 0x0000FFFFu : 0u) | (hi ? 0xFFFF0000u : 0u);
                    ww[h] &= keep;                       // pruned weights become +0
                }
                // 128-byte swizzle: 16-byte chunk cc of row r lives at chunk position cc ^ (r % 8)
                uint4 *dst = reinterpret_cast<uint4 *>(a_stage + r * 128 + ((cc ^ (r & 7)) << 4));
                *dst = make_uint4(ww[0], ww[1], ww[2], ww[3]);
            }
            fence_async_proxy();                         // generic-proxy stores -> visible to the MMA
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->full[s]);
        }

        // ------------------------------------------------------------- epilogue (same warps)
        if (ok) ok = mbar_wait(&ctl->accum, 0, abort_flag, status, DEV_TIMEOUT_ACCUM);
        if (ok) {
            tc_fence_after();
            const int quad = warp & 3;                   // tensor-memory lanes this warp may read
            const int half = (warp - 2) >> 2;            // which half of the accumulator columns
            const int o = o0 + quad * 32 + lane;
            constexpr int COLS_PER_WARP = BN / 2 < 16 ? 16 : BN / 2;
            constexpr int NCHUNK = COLS_PER_WARP / 16;
            const bool active = (BN >= 32) || half == 0;
            if (active) {
#pragma unroll 1
                for (int ch = 0; ch < NCHUNK; ++ch) {
                    const int col0 = half * COLS_PER_WARP + ch * 16;
                    uint32_t v[16];
                    tmem_ld16(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)col0, v);
                    tmem_ld_wait();
                    if (o < g.rows) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int b = b0 + col0 + j;
                            if (b < batch) {
                                const float f = __uint_as_float(v[j]);
                                if (partials) {
                                    partials[((long long)blockIdx.z * batch + b) * g.rows + o] = f;
                                } else if (y_dtype == LRBI_Y_F32) {
                                    reinterpret_cast<float *>(Y)[(long long)b * g.rows + o] = f;
                                } else {
                                    reinterpret_cast<uint16_t *>(Y)[(long long)b * g.rows + o] = f32_to_bf16_rne(f);
                                }
                            }
                        }
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_d, TMEM_COLS);
    }
}

// Sum of the K-split partial results: Y[b][o] = sum_z partials[z][b][o].
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float *__restrict__ partials, int splits, long long n, void *__restrict__ Y, int y_dtype)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n) return;
    float acc = 0.f;
    for (int z = 0; z < splits; ++z) acc += partials[(long long)z * n + idx];
    if (y_dtype == LRBI_Y_F32) reinterpret_cast<float *>(Y)[idx] = acc;
    else reinterpret_cast<uint16_t *>(Y)[idx] = f32_to_bf16_rne(acc);
}

// --------------------------------------------------------------------------------------
// host side
// --------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

bool gemm_tc_supported(const Geo &g, int batch)
{
    if (batch < 1 || g.kw > 2) return false;
    if ((g.cols % 8) != 0) return false;                                   // 16-byte rows for TMA and vector loads
    if (!(g.gr == 1 || (g.tm % TC_BM) == 0)) return false;                 // 128 rows inside one tile row
    if (!(g.gc == 1 ? (g.tn % 8) == 0 : (g.tn % TC_BK) == 0)) return false; // a K block inside one tile column
    return true;
}

struct Workspace {
    float *ptr = nullptr;
    size_t bytes = 0;
};
static Workspace g_ws[64];

static float *workspace(size_t bytes)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    Workspace &w = g_ws[dev];
    if (w.bytes < bytes) {
        if (w.ptr) cudaFree(w.ptr);
        w.ptr = nullptr; w.bytes = 0;
        if (cudaMalloc(&w.ptr, bytes) != cudaSuccess) { w.ptr = nullptr; return nullptr; }
        w.bytes = bytes;
    }
    return w.ptr;
}

template <int BN, int KW>
static lrbi_status launch_tc(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                             const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s, int sm_count)
{
    EncodeTiledFn encode = get_encode_fn();
    if (!encode) { note_cuda_error(-1); return LRBI_ERR_CUDA; }
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)g.cols, (cuuint64_t)batch};
    const cuuint64_t strides[1] = {(cuuint64_t)g.cols * 2};
    const cuuint32_t box[2] = {TC_BK, BN};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<uint16_t *>(X), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { note_cuda_error((int)r); return LRBI_ERR_CUDA; }

    constexpr int B_STAGE = BN * TC_BK * 2;
    const int nkb = (g.cols + TC_BK - 1) / TC_BK;
    const int tiles = ((batch + BN - 1) / BN) * ((g.rows + TC_BM - 1) / TC_BM);
    // split K when the output tiles alone cannot occupy the chip (small batch: bandwidth-bound)
    int splits = 1;
    if (batch <= BN && tiles < 2 * sm_count) {        // one batch tile: the small-batch, bandwidth-bound case
        splits = (2 * sm_count + tiles - 1) / tiles;
        splits = splits > nkb / 4 ? (nkb / 4 > 0 ? nkb / 4 : 1) : splits;   // at least 4 K blocks per split
        if (splits > 32) splits = 32;
    }
    int kb_per_split = (nkb + splits - 1) / splits;
    splits = (nkb + kb_per_split - 1) / kb_per_split;                        // no empty split

    int stages = BN >= 256 ? 4 : (BN >= 128 ? 4 : 6);
    if (stages > 8) stages = 8;
    const size_t smem = 1024 + (size_t)stages * (TC_A_STAGE_BYTES + B_STAGE) + sizeof(TcCtl);

    float *partials = nullptr;
    if (splits > 1) {
        partials = workspace((size_t)splits * batch * g.rows * sizeof(float));
        if (!partials) { note_cuda_error((int)cudaErrorMemoryAllocation); return LRBI_ERR_CUDA; }
    }
    auto kern = gemm_tc_kernel<BN, KW>;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
        attr_done = true;
    }
    dim3 grid((unsigned)((batch + BN - 1) / BN), (unsigned)((g.rows + TC_BM - 1) / TC_BM), (unsigned)splits);
    if (grid.y > 65535 || grid.z > 65535) return LRBI_ERR_UNSUPPORTED;
    kern<<<grid, TC_THREADS, smem, s>>>(map, g, W, ip, iz, batch, Y, y_dtype, partials, kb_per_split, stages,
                                         device_status_ptr());
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    if (splits > 1) {
        const long long n = (long long)batch * g.rows;
        splitk_reduce_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(partials, splits, n, Y, y_dtype);
        count_launch();
        e = cudaGetLastError();
        if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    }
    return LRBI_OK;
}

template <int BN>
static lrbi_status launch_tc_kw(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                                const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s, int sm_count)
{
    return g.kw == 1 ? launch_tc<BN, 1>(g, W, ip, iz, X, batch, Y, y_dtype, s, sm_count)
                     : launch_tc<BN, 2>(g, W, ip, iz, X, batch, Y, y_dtype, s, sm_count);
}

lrbi_status launch_gemm_tc(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                           const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s)
{
    if (!gemm_tc_supported(g, batch)) return LRBI_ERR_UNSUPPORTED;
    if (!device_status_ptr()) return LRBI_ERR_CUDA;
    int dev = 0, sm_count = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (batch <= 16) return launch_tc_kw<16>(g, W, ip, iz, X, batch, Y, y_dtype, s, sm_count);
    if (batch <= 32) return launch_tc_kw<32>(g, W, ip, iz, X, batch, Y, y_dtype, s, sm_count);
    if (batch <= 64) return launch_tc_kw<64>(g, W, ip, iz, X, batch, Y, y_dtype, s, sm_count);
    if (batch <= 128) return launch_tc_kw<128>(g, W, ip, iz, X, batch, Y, y_dtype, s, sm_count);
    return launch_tc_kw<256>(g, W, ip, iz, X, batch, Y, y_dtype, s, sm_count);
}

}  // namespace lrbi
