// Generalised layouts (Section 3.1, last paragraph: every submatrix may choose its own rank) and decoding
// several layers in one launch.
//
// Ranked layout.  Tile t has rank k_t (0 <= k_t <= the layout's rank, which is only the upper bound) and its
// factors are packed with KW_t = ceil(k_t / 32) words per row of Ip / per column of Iz, so a low-rank tile costs
// less storage:  ip[ip_offset[t] + i * KW_t + w],  iz[iz_offset[t] + j * KW_t + w].
//
//   decode_any        any shape, any ranks, up to 32 layers per launch: one __ballot_sync per mask word
//                     ((ip & iz) != 0 over the tile's own words), rows written as 16-byte vectors.
//   gemm_ranked       any shape, any ranks: one thread per output element (the tensor-core kernel covers the
//                     aligned shapes, see gemm_tc.cu).
#include "lrbi_common.cuh"

namespace lrbi {

constexpr int RK_THREADS = 256;
constexpr int RK_WORDS = 8;            // mask words (256 columns) per block column
constexpr int RK_PITCH = 12;           // words per staged row (8 + pad, keeps 16-byte alignment)
constexpr int RK_MAX_LAYERS = 32;      // layers per launch of the batched decode

struct DecodeJob {
    Geo g;
    TileRanks rk;                      // null pointers: one rank for every tile
    const uint32_t *ip, *iz;
    uint32_t *mask;
    unsigned first_block, blocks_x;    // this layer's blocks start here; blocks per row band
};
struct DecodeTable {
    int n;
    DecodeJob job[RK_MAX_LAYERS];
};

// Rank, words per row/column and first factor words of tile `tile`.
__device__ __forceinline__ void tile_factors(const Geo &g, const TileRanks &rk, long long tile, int &k, int &kw,
                                             const uint32_t *ip, const uint32_t *iz, const uint32_t *&ipt, const uint32_t *&izt)
{
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

__global__ void __launch_bounds__(RK_THREADS)
decode_any_kernel(const __grid_constant__ DecodeTable tab)
{
    __shared__ __align__(16) uint32_t stage[RK_THREADS / 32][32][RK_PITCH];
    int li = 0;
    while (li + 1 < tab.n && blockIdx.x >= tab.job[li + 1].first_block) ++li;     // block-uniform
    const DecodeJob &jb = tab.job[li];
    const Geo &g = jb.g;
    const unsigned local = blockIdx.x - jb.first_block;
    const int bx = (int)(local % jb.blocks_x), by = (int)(local / jb.blocks_x);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int word0 = bx * RK_WORDS;
    const int row0 = (by * (RK_THREADS / 32) + warp) * 32;
    if (row0 >= g.rows) return;                                // whole warp leaves together

    for (int rr = 0; rr < 32; ++rr) {
        const int r = row0 + rr;
        if (r >= g.rows) break;                                // warp-uniform
        const int tr = r / g.tm, i = r - tr * g.tm;
#pragma unroll
        for (int q = 0; q < RK_WORDS; ++q) {
            const int c = (word0 + q) * 32 + lane;
            uint32_t any = 0;
            if (c < g.cols) {
                const int tc = c / g.tn, j = c - tc * g.tn;
                int k, kw;
                const uint32_t *ipt, *izt;
                tile_factors(g, jb.rk, (long long)tr * g.gc + tc, k, kw, jb.ip, jb.iz, ipt, izt);
                const uint32_t tail = tail_mask(k);
                for (int w = 0; w < kw; ++w) {
                    uint32_t t = __ldg(ipt + (long long)i * kw + w) & __ldg(izt + (long long)j * kw + w);
                    if (w == kw - 1) t &= tail;
                    any |= t;
                }
            }
            const uint32_t word = __ballot_sync(0xFFFFFFFFu, any != 0);
            if (lane == q) stage[warp][rr][q] = word;
        }
    }
    __syncwarp();
    const int r = row0 + lane;                                 // lane <-> staged row
    if (r < g.rows) {
        uint32_t *dst = jb.mask + (long long)r * g.pitch + word0;
        const int nw = min(RK_WORDS, g.pitch - word0);
        if (nw == RK_WORDS && (g.pitch & 3) == 0) {
            const uint4 *src = reinterpret_cast<const uint4 *>(&stage[warp][lane][0]);
            reinterpret_cast<uint4 *>(dst)[0] = src[0];
            reinterpret_cast<uint4 *>(dst)[1] = src[1];
        } else {
            for (int q = 0; q < nw; ++q) dst[q] = stage[warp][lane][q];
        }
    }
}

static lrbi_status launch_table(const DecodeTable &tab, unsigned blocks, cudaStream_t s)
{
    decode_any_kernel<<<blocks, RK_THREADS, 0, s>>>(tab);
    count_launch();
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

static bool add_job(DecodeTable &tab, unsigned &blocks, const Geo &g, const TileRanks &rk, const uint32_t *ip,
                    const uint32_t *iz, uint32_t *mask)
{
    const unsigned long long bx = (unsigned long long)((g.pitch + RK_WORDS - 1) / RK_WORDS);
    const unsigned long long by = (unsigned long long)((g.rows + RK_THREADS - 1) / RK_THREADS);
    if ((unsigned long long)blocks + bx * by > 0x7FFFFFFFull) return false;
    DecodeJob &j = tab.job[tab.n++];
    j.g = g; j.rk = rk; j.ip = ip; j.iz = iz; j.mask = mask;
    j.first_block = blocks; j.blocks_x = (unsigned)bx;
    blocks += (unsigned)(bx * by);
    return true;
}

lrbi_status launch_decode_ranked(const Geo &g, const TileRanks &rk, const uint32_t *ip, const uint32_t *iz,
                                 uint32_t *mask, cudaStream_t s)
{
    DecodeTable tab;
    tab.n = 0;
    unsigned blocks = 0;
    if (!add_job(tab, blocks, g, rk, ip, iz, mask)) return LRBI_ERR_UNSUPPORTED;
    return launch_table(tab, blocks, s);
}

lrbi_status launch_decode_batch(int n, const Geo *g, const uint32_t *const *ip, const uint32_t *const *iz,
                                uint32_t *const *mask, cudaStream_t s)
{
    const TileRanks none = {nullptr, nullptr, nullptr};
    for (int first = 0; first < n; first += RK_MAX_LAYERS) {   // one launch per 32 layers
        DecodeTable tab;
        tab.n = 0;
        unsigned blocks = 0;
        for (int l = first; l < n && l < first + RK_MAX_LAYERS; ++l)
            if (!add_job(tab, blocks, g[l], none, ip[l], iz[l], mask[l])) return LRBI_ERR_UNSUPPORTED;
        const lrbi_status st = launch_table(tab, blocks, s);
        if (st != LRBI_OK) return st;
    }
    return LRBI_OK;
}

// --------------------------------------------------------------------------------------
// gemm_ranked: any shape, any ranks
// --------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
gemm_ranked_kernel(Geo g, TileRanks rk, const uint16_t *__restrict__ W, const uint32_t *__restrict__ ip,
                   const uint32_t *__restrict__ iz, const uint16_t *__restrict__ X, int batch,
                   void *__restrict__ Y, int y_dtype)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)batch * g.rows) return;
    const int o = (int)(idx % g.rows), b = (int)(idx / g.rows);
    const int tr = o / g.tm, i = o - tr * g.tm;
    float acc = 0.f;
    for (int tc = 0; tc < g.gc; ++tc) {
        int k, kw;
        const uint32_t *ipt, *izt;
        tile_factors(g, rk, (long long)tr * g.ts_r + (long long)tc * g.ts_c, k, kw, ip, iz, ipt, izt);
        const uint32_t tail = tail_mask(k);
        const uint32_t *ipw = ipt + (long long)i * kw;
        const int c_end = min(g.tn, g.cols - tc * g.tn);
        for (int j = 0; j < c_end; ++j) {
            const uint32_t *izw = izt + (long long)j * kw;
            uint32_t any = 0;
            for (int w = 0; w < kw; ++w) {
                uint32_t t = __ldg(ipw + w) & __ldg(izw + w);
                if (w == kw - 1) t &= tail;
                any |= t;
            }
            if (any) {                                         // Eq. 3 with the tile's own rank: kept weight
                const int c = tc * g.tn + j;
                const float wv = __uint_as_float((uint32_t)W[(long long)o * g.cols + c] << 16);
                const float xv = __uint_as_float((uint32_t)X[(long long)b * g.cols + c] << 16);
                acc = fmaf(wv, xv, acc);
            }
        }
    }
    if (y_dtype == LRBI_Y_F32) reinterpret_cast<float *>(Y)[idx] = acc;
    else reinterpret_cast<uint16_t *>(Y)[idx] = f32_to_bf16_rne(acc);
}

lrbi_status launch_gemm_ranked_generic(const Geo &g, const TileRanks &rk, const uint16_t *W, const uint32_t *ip,
                                       const uint32_t *iz, const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s)
{
    const long long total = (long long)batch * g.rows;
    const long long blocks = (total + 255) / 256;
    if (blocks > 0x7FFFFFFFLL) return LRBI_ERR_UNSUPPORTED;
    gemm_ranked_kernel<<<(unsigned)blocks, 256, 0, s>>>(g, rk, W, ip, iz, X, batch, Y, y_dtype);
    count_launch();
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

}  // namespace lrbi
