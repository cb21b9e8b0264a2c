// Small-batch fused decode + prune + product on CUDA cores, and the any-shape fallback.
//
//   gemm_generic   one thread per output element; decodes every index bit from the packed
//                  factors as it goes.  Covers every legal shape; slow.
//   stream_mma     batch <= 32.  The same streaming idea with warp-level tensor-core MMAs (mma.sync): a
//                  block owns 16 rows, its 16 warps split K, pruned weights go straight from registers
//                  into the MMAs.  Chosen for batch 2..8.
//   gemv           batch <= 8.  Streams W exactly once with 16-byte loads (the dominant HBM
//                  traffic), decodes the index bits in registers from the row words of Ip and
//                  the column words of Iz, and accumulates in fp32.  A warp owns RW rows and a
//                  contiguous range of 256-column chunks, so the column words and the
//                  activations it loads are reused RW times from registers.
#include "lrbi_common.cuh"

namespace lrbi {

__device__ __forceinline__ void store_y(void *Y, int y_dtype, long long idx, float v)
{
    if (y_dtype == LRBI_Y_F32) reinterpret_cast<float *>(Y)[idx] = v;
    else reinterpret_cast<uint16_t *>(Y)[idx] = f32_to_bf16_rne(v);
}

// --------------------------------------------------------------------------------------
// gemm_generic
// --------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
gemm_generic_kernel(Geo g, const uint16_t *__restrict__ W, const uint32_t *__restrict__ ip,
                    const uint32_t *__restrict__ iz, const uint16_t *__restrict__ X, int batch,
                    void *__restrict__ Y, int y_dtype)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)batch * g.rows) return;
    const int o = (int)(idx % g.rows), b = (int)(idx / g.rows);
    const int tr = o / g.tm, i = o - tr * g.tm;
    const uint32_t tail = tail_mask(g.k);
    float acc = 0.f;
    for (int tc = 0; tc < g.gc; ++tc) {
        const long long tile = (long long)tr * g.gc + tc;
        const uint32_t *ipw = ip + (tile * g.tm + i) * g.kw;
        const int c_end = min(g.tn, g.cols - tc * g.tn);
        for (int j = 0; j < c_end; ++j) {
            const uint32_t *izw = iz + (tile * g.tn + j) * g.kw;
            uint32_t any = 0;
            for (int w = 0; w < g.kw; ++w) {
                uint32_t t = __ldg(ipw + w) & __ldg(izw + w);
                if (w == g.kw - 1) t &= tail;
                any |= t;
            }
            if (any) {
                const int c = tc * g.tn + j;
                const float wv = __uint_as_float((uint32_t)W[(long long)o * g.cols + c] << 16);
                const float xv = __uint_as_float((uint32_t)X[(long long)b * g.cols + c] << 16);
                acc = fmaf(wv, xv, acc);
            }
        }
    }
    store_y(Y, y_dtype, idx, acc);
}

lrbi_status launch_gemm_generic(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                                const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s)
{
    const long long total = (long long)batch * g.rows;
    const long long blocks = (total + 255) / 256;
    if (blocks > 0x7FFFFFFFLL) return LRBI_ERR_UNSUPPORTED;
    gemm_generic_kernel<<<(unsigned)blocks, 256, 0, s>>>(g, W, ip, iz, X, batch, Y, y_dtype);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

// --------------------------------------------------------------------------------------
// gemv
// --------------------------------------------------------------------------------------
constexpr int GEMV_WARPS = 4;
constexpr int GEMV_CHUNK = 256;       // columns per warp step: 32 lanes x 8 bf16 (16 bytes)

__device__ __forceinline__ uint4 ldg_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

template <int BATCH, int RW, int KW>
__global__ void __launch_bounds__(GEMV_WARPS * 32)
gemv_kernel(Geo g, const uint16_t *__restrict__ W, const uint32_t *__restrict__ ip,
            const uint32_t *__restrict__ iz, const uint16_t *__restrict__ X, int batch,
            void *__restrict__ Y, int y_dtype)
{
    __shared__ float part[GEMV_WARPS][RW][BATCH];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int o0 = blockIdx.x * RW;                     // first row of this block's row group
    const int tr = o0 / g.tm;                           // the whole group lies in one tile row
    const int i0 = o0 - tr * g.tm;
    const uint32_t tail = tail_mask(g.k);

    float acc[RW][BATCH];
#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
        for (int b = 0; b < BATCH; ++b) acc[r][b] = 0.f;

    // contiguous range of chunks for this warp
    const int nchunks = (g.cols + GEMV_CHUNK - 1) / GEMV_CHUNK;
    const int per = (nchunks + GEMV_WARPS - 1) / GEMV_WARPS;
    const int ch_begin = warp * per, ch_end = min(nchunks, ch_begin + per);

    uint32_t ipv[RW][KW];
    int tc_prev = -1;

    uint4 wnext[RW];
    auto load_w = [&](int ch, uint4 (&dst)[RW]) {
        const int c0 = ch * GEMV_CHUNK + lane * 8;
#pragma unroll
        for (int r = 0; r < RW; ++r) {
            const int o = o0 + r;
            dst[r] = (ch < ch_end && c0 < g.cols && o < g.rows)
                         ? ldg_stream(reinterpret_cast<const uint4 *>(W + (long long)o * g.cols + c0))
                         : make_uint4(0, 0, 0, 0);
        }
    };
    load_w(ch_begin, wnext);

    for (int ch = ch_begin; ch < ch_end; ++ch) {
        uint4 wcur[RW];
#pragma unroll
        for (int r = 0; r < RW; ++r) wcur[r] = wnext[r];
        load_w(ch + 1, wnext);                          // keep the next chunk of W in flight

        const int c0 = ch * GEMV_CHUNK + lane * 8;
        if (c0 >= g.cols) continue;                     // cols % 8 == 0: a lane's 8 columns exist or not
        const int tc = c0 / g.tn, j0 = c0 - tc * g.tn;  // tn % 8 == 0: all 8 in one tile
        const long long tile = (long long)tr * g.gc + tc;
        if (tc != tc_prev) {
            tc_prev = tc;
#pragma unroll
            for (int r = 0; r < RW; ++r)
#pragma unroll
                for (int w = 0; w < KW; ++w) {
                    uint32_t v = (i0 + r < g.tm) ? __ldg(ip + (tile * g.tm + i0 + r) * KW + w) : 0u;
                    if (w == KW - 1) v &= tail;
                    ipv[r][w] = v;
                }
        }
        // column words of the 8 columns: 8*KW consecutive words
        uint32_t izv[8][KW];
        {
            const uint4 *zp = reinterpret_cast<const uint4 *>(iz + (tile * g.tn + j0) * KW);
#pragma unroll
            for (int v = 0; v < 2 * KW; ++v) {
                const uint4 z = __ldg(zp + v);
                const uint32_t zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
                for (int t = 0; t < 4; ++t) izv[(v * 4 + t) / KW][(v * 4 + t) % KW] = zz[t];
            }
        }
        // activations of the 8 columns
        float xf[BATCH][8];
#pragma unroll
        for (int b = 0; b < BATCH; ++b) {
            uint4 xv = make_uint4(0, 0, 0, 0);
            if (b < batch) xv = __ldg(reinterpret_cast<const uint4 *>(X + (long long)b * g.cols + c0));
            xf[b][0] = bf16_lo(xv.x); xf[b][1] = bf16_hi(xv.x);
            xf[b][2] = bf16_lo(xv.y); xf[b][3] = bf16_hi(xv.y);
            xf[b][4] = bf16_lo(xv.z); xf[b][5] = bf16_hi(xv.z);
            xf[b][6] = bf16_lo(xv.w); xf[b][7] = bf16_hi(xv.w);
        }
#pragma unroll
        for (int r = 0; r < RW; ++r) {
            const uint32_t ww[4] = {wcur[r].x, wcur[r].y, wcur[r].z, wcur[r].w};
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                uint32_t any = 0;
#pragma unroll
                for (int w = 0; w < KW; ++w) any |= ipv[r][w] & izv[e][w];
                if (any) {                               // Eq. 3: kept weight
                    const float wf = (e & 1) ? bf16_hi(ww[e >> 1]) : bf16_lo(ww[e >> 1]);
#pragma unroll
                    for (int b = 0; b < BATCH; ++b) acc[r][b] = fmaf(wf, xf[b][e], acc[r][b]);
                }
            }
        }
    }

    // reduce over lanes, then over warps
#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
        for (int b = 0; b < BATCH; ++b) {
            float v = acc[r][b];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
            if (lane == 0) part[warp][r][b] = v;
        }
    __syncthreads();
    for (int t = threadIdx.x; t < RW * BATCH; t += GEMV_WARPS * 32) {
        const int r = t / BATCH, b = t - r * BATCH;
        const int o = o0 + r;
        if (o < g.rows && b < batch) {
            float v = 0.f;
#pragma unroll
            for (int wp = 0; wp < GEMV_WARPS; ++wp) v += part[wp][r][b];
            store_y(Y, y_dtype, (long long)b * g.rows + o, v);
        }
    }
}

// --------------------------------------------------------------------------------------
// stream_mma: batch <= 32, bandwidth-bound, warp-level tensor-core MMAs
// --------------------------------------------------------------------------------------
// A block owns 16 rows of W (one m16 tile); its warps split K into contiguous ranges and add their
// partial tiles up through shared memory, so no scratch memory and no second kernel are needed.  Per
// step a warp covers 32 columns: lane (g, t) = (lane / 4, lane % 4) loads the 8 consecutive weights
// W[g][k0 + 8t ..] and W[g + 8][k0 + 8t ..] (two 16-byte loads), the column words of Iz of those 8
// columns and 16 bytes of X per 8 batch rows, decodes its 16 index bits from the row words of Ip
// ((ip & iz) != 0, Eq. 3), zeroes pruned weights with AND-masks and issues two m16n8k16 MMAs per 8 batch
// rows.  The K index inside an MMA is a summation index, so the 32 columns are handed to the MMAs in the
// order in which they sit in the registers (both operands use the same order): no shuffles, no staging.
// The kernel keeps few registers so that many warps are resident: latency is hidden by occupancy
// (loading two steps ahead of the MMAs was measured: the registers it costs halve the occupancy and the
// kernel gets slower).
constexpr int SM_WARPS = 16;

__device__ __forceinline__ void mma_bf16_16x8x16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                 uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int NT, int KW>       // NT = batch tiles of 8 rows
__global__ void __launch_bounds__(SM_WARPS * 32)
stream_mma_kernel(Geo g, const uint16_t *__restrict__ W, const uint32_t *__restrict__ ip,
                  const uint32_t *__restrict__ iz, const uint16_t *__restrict__ X, int batch,
                  void *__restrict__ Y, int y_dtype)
{
    __shared__ float part[SM_WARPS][16][NT * 8 + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane >> 2, t = lane & 3;
    const int o0 = blockIdx.x * 16;                     // first row of this block
    const int tr = o0 / g.tm;                           // the 16 rows lie in one tile row
    const int i0 = o0 - tr * g.tm;
    const uint32_t tail = tail_mask(g.k);
    const bool row_lo = o0 + gq < g.rows && i0 + gq < g.tm, row_hi = o0 + gq + 8 < g.rows && i0 + gq + 8 < g.tm;

    float acc[NT][4];
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[n][e] = 0.f;

    const int nsteps = (g.cols + 31) / 32;
    const int per = (nsteps + SM_WARPS - 1) / SM_WARPS;
    const int st_begin = warp * per, st_end = min(nsteps, st_begin + per);

    uint32_t ip_lo[KW], ip_hi[KW];
    int tc_prev = -1;
    for (int st = st_begin; st < st_end; ++st) {
        const int c0 = st * 32 + t * 8;                 // this lane's 8 columns
        // cols % 8 == 0: the 8 columns exist or not.  A lane without columns feeds zeros: every lane of the
        // warp has to take part in the MMAs.
        const bool live = c0 < g.cols;
        const int cc0 = live ? c0 : 0;
        const int tc = cc0 / g.tn, j0 = cc0 - tc * g.tn;  // tn % 8 == 0: all 8 in one tile
        const long long tile = (long long)tr * g.gc + tc;
        const uint4 zero = make_uint4(0, 0, 0, 0);
        const uint4 wlo = (live && row_lo) ? ldg_stream(reinterpret_cast<const uint4 *>(W + (long long)(o0 + gq) * g.cols + cc0)) : zero;
        const uint4 whi = (live && row_hi) ? ldg_stream(reinterpret_cast<const uint4 *>(W + (long long)(o0 + gq + 8) * g.cols + cc0)) : zero;
        uint4 xv[NT];
#pragma unroll
        for (int n = 0; n < NT; ++n)
            xv[n] = (live && n * 8 + gq < batch) ? __ldg(reinterpret_cast<const uint4 *>(X + (long long)(n * 8 + gq) * g.cols + cc0)) : zero;
        uint32_t izv[8][KW];
        {
            const uint4 *zp = reinterpret_cast<const uint4 *>(iz + (tile * g.tn + j0) * KW);
#pragma unroll
            for (int v = 0; v < 2 * KW; ++v) {
                const uint4 z = __ldg(zp + v);
                const uint32_t zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) izv[(v * 4 + q) / KW][(v * 4 + q) % KW] = zz[q];
            }
        }
        if (tc != tc_prev) {                            // row words of Ip change with the tile column
            tc_prev = tc;
#pragma unroll
            for (int w = 0; w < KW; ++w) {
                uint32_t lo = row_lo ? __ldg(ip + (tile * g.tm + i0 + gq) * KW + w) : 0u;
                uint32_t hi = row_hi ? __ldg(ip + (tile * g.tm + i0 + gq + 8) * KW + w) : 0u;
                if (w == KW - 1) { lo &= tail; hi &= tail; }
                ip_lo[w] = lo; ip_hi[w] = hi;
            }
        }
        // prune: 16-bit AND-masks from the Boolean product of Eq. 3
        uint32_t alo[4] = {wlo.x, wlo.y, wlo.z, wlo.w}, ahi[4] = {whi.x, whi.y, whi.z, whi.w};
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            uint32_t l0 = 0, l1 = 0, h0 = 0, h1 = 0;
#pragma unroll
            for (int w = 0; w < KW; ++w) {
                l0 |= ip_lo[w] & izv[2 * p][w];  l1 |= ip_lo[w] & izv[2 * p + 1][w];
                h0 |= ip_hi[w] & izv[2 * p][w];  h1 |= ip_hi[w] & izv[2 * p + 1][w];
            }
            alo[p] &= (l0 ? 0x0000FFFFu : 0u) | (l1 ? 0xFFFF0000u : 0u);
            ahi[p] &= (h0 ? 0x0000FFFFu : 0u) | (h1 ? 0xFFFF0000u : 0u);
        }
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            mma_bf16_16x8x16(acc[n], alo[0], ahi[0], alo[1], ahi[1], xv[n].x, xv[n].y);
            mma_bf16_16x8x16(acc[n], alo[2], ahi[2], alo[3], ahi[3], xv[n].z, xv[n].w);
        }
    }

    // accumulator layout: c0,c1 = (row g, batch 2t, 2t+1), c2,c3 = (row g+8, same)
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        part[warp][gq][n * 8 + 2 * t] = acc[n][0];
        part[warp][gq][n * 8 + 2 * t + 1] = acc[n][1];
        part[warp][gq + 8][n * 8 + 2 * t] = acc[n][2];
        part[warp][gq + 8][n * 8 + 2 * t + 1] = acc[n][3];
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < 16 * NT * 8; idx += SM_WARPS * 32) {
        const int b = idx / 16, r = idx - b * 16;       // consecutive threads -> consecutive output features
        if (b < batch && o0 + r < g.rows) {
            float v = 0.f;
#pragma unroll
            for (int wp = 0; wp < SM_WARPS; ++wp) v += part[wp][r][b];
            store_y(Y, y_dtype, (long long)b * g.rows + o0 + r, v);
        }
    }
}

bool stream_mma_supported(const Geo &g, int batch)
{
    if (batch < 1 || batch > 32 || g.kw > 2) return false;
    if ((g.cols % 8) != 0 || (g.tn % 8) != 0) return false;
    return g.gr == 1 || (g.tm % 16) == 0;
}

template <int NT>
static void stream_mma_dispatch(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                                const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s)
{
    const unsigned blocks = (unsigned)((g.rows + 15) / 16);
    if (g.kw == 1) stream_mma_kernel<NT, 1><<<blocks, SM_WARPS * 32, 0, s>>>(g, W, ip, iz, X, batch, Y, y_dtype);
    else stream_mma_kernel<NT, 2><<<blocks, SM_WARPS * 32, 0, s>>>(g, W, ip, iz, X, batch, Y, y_dtype);
}

lrbi_status launch_stream_mma(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                              const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s)
{
    if (!stream_mma_supported(g, batch)) return LRBI_ERR_UNSUPPORTED;
    if (batch <= 8) stream_mma_dispatch<1>(g, W, ip, iz, X, batch, Y, y_dtype, s);
    else if (batch <= 16) stream_mma_dispatch<2>(g, W, ip, iz, X, batch, Y, y_dtype, s);
    else stream_mma_dispatch<4>(g, W, ip, iz, X, batch, Y, y_dtype, s);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

static int gemv_rows_per_block(int batch) { return batch <= 2 ? 8 : 4; }

bool gemv_supported(const Geo &g, int batch)
{
    if (batch < 1 || batch > 8 || g.kw > 2) return false;
    if ((g.cols % 8) != 0 || (g.tn % 8) != 0) return false;
    const int rw = gemv_rows_per_block(batch);
    return g.gr == 1 || (g.tm % rw) == 0;
}

template <int BATCH, int RW>
static void gemv_dispatch_kw(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                             const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s)
{
    const unsigned blocks = (unsigned)((g.rows + RW - 1) / RW);
    if (g.kw == 1) gemv_kernel<BATCH, RW, 1><<<blocks, GEMV_WARPS * 32, 0, s>>>(g, W, ip, iz, X, batch, Y, y_dtype);
    else gemv_kernel<BATCH, RW, 2><<<blocks, GEMV_WARPS * 32, 0, s>>>(g, W, ip, iz, X, batch, Y, y_dtype);
}

lrbi_status launch_gemv(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                        const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s)
{
    if (!gemv_supported(g, batch)) return LRBI_ERR_UNSUPPORTED;
    if (batch == 1) gemv_dispatch_kw<1, 8>(g, W, ip, iz, X, batch, Y, y_dtype, s);
    else if (batch == 2) gemv_dispatch_kw<2, 8>(g, W, ip, iz, X, batch, Y, y_dtype, s);
    else if (batch <= 4) gemv_dispatch_kw<4, 4>(g, W, ip, iz, X, batch, Y, y_dtype, s);
    else gemv_dispatch_kw<8, 4>(g, W, ip, iz, X, batch, Y, y_dtype, s);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

}  // namespace lrbi
