// Inner loop of Algorithm 1 (Section 2.1 of the paper) on the GPU:
//   threshold_pack   binary conversion of the NMF factors: bit = (value >= T), one threshold pair per tile, written
//                    straight into the packed factor format of this library (one __ballot_sync per row word of Ip;
//                    a thread gathers the k bits of a column word of Iz from coalesced loads);
//   index_cost       per tile: the ones of the magnitude index I = (|W| >= theta), the ones of the decoded index
//                    Ia = Ip (x) Iz (Eq. 3), the positions with I = 1 and Ia = 0 and Cost = the sum of |W| over them.
//                    W is streamed once; Ia is decoded on the fly from bit-planes in shared memory (the same
//                    transposition as in the decode kernels) and never stored.
#include "lrbi_common.cuh"

namespace lrbi {

constexpr int A1_THREADS = 256;

// ---------------------------------------------------------------------------------------- threshold_pack
// One warp per (tile, row, word) of Ip: lane l tests bit 32 w + l.
__global__ void __launch_bounds__(A1_THREADS)
threshold_pack_ip_kernel(Geo g, const float *__restrict__ mp, const float *__restrict__ tp, uint32_t *__restrict__ ip)
{
    const int lane = threadIdx.x & 31;
    const long long warps = (long long)gridDim.x * (A1_THREADS / 32);
    const long long total = (long long)g.gr * g.gc * g.tm * g.kw;          // row words
    for (long long q = (long long)blockIdx.x * (A1_THREADS / 32) + (threadIdx.x >> 5); q < total; q += warps) {
        const long long row = q / g.kw;                                     // tile * tm + i
        const int w = (int)(q - row * g.kw);
        const long long tile = row / g.tm;
        const int b = w * 32 + lane;
        const bool one = b < g.k && __ldg(mp + row * g.k + b) >= __ldg(tp + tile);
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, one);
        if (lane == 0) ip[q] = word;
    }
}

// One thread per (tile, column) of Iz: consecutive threads read consecutive columns of a row of Mz.
__global__ void __launch_bounds__(A1_THREADS)
threshold_pack_iz_kernel(Geo g, const float *__restrict__ mz, const float *__restrict__ tz, uint32_t *__restrict__ iz)
{
    const long long total = (long long)g.gr * g.gc * g.tn;                  // columns of all tiles
    for (long long q = (long long)blockIdx.x * A1_THREADS + threadIdx.x; q < total; q += (long long)gridDim.x * A1_THREADS) {
        const long long tile = q / g.tn;
        const int j = (int)(q - tile * g.tn);
        const float t = __ldg(tz + tile);
        const float *src = mz + tile * g.k * g.tn + j;
        for (int w = 0; w < g.kw; ++w) {
            uint32_t word = 0;
            for (int l = 0; l < 32 && w * 32 + l < g.k; ++l)
                if (__ldg(src + (long long)(w * 32 + l) * g.tn) >= t) word |= 1u << l;
            iz[q * g.kw + w] = word;
        }
    }
}

lrbi_status launch_threshold_pack(const Geo &g, const float *mp, const float *mz, const float *tp, const float *tz,
                                  uint32_t *ip, uint32_t *iz, cudaStream_t s)
{
    const long long row_words = (long long)g.gr * g.gc * g.tm * g.kw, cols = (long long)g.gr * g.gc * g.tn;
    long long b1 = (row_words + A1_THREADS / 32 - 1) / (A1_THREADS / 32), b2 = (cols + A1_THREADS - 1) / A1_THREADS;
    if (b1 > 148 * 32) b1 = 148 * 32;                                       // grid-stride loops
    if (b2 > 148 * 32) b2 = 148 * 32;
    threshold_pack_ip_kernel<<<(unsigned)b1, A1_THREADS, 0, s>>>(g, mp, tp, ip);
    threshold_pack_iz_kernel<<<(unsigned)b2, A1_THREADS, 0, s>>>(g, mz, tz, iz);
    count_launch(2);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

// ---------------------------------------------------------------------------------------- index_cost
constexpr int A1_BAND = 64;            // rows of a tile per block

struct CostAcc {
    unsigned long long kept_i, kept_a, lost;
    double cost;
};

// Eight consecutive weights (16 bytes) and the eight index bits of Ia that go with them: counts by popcount,
// cost as a select-and-add in fp32 (eight terms; the caller carries it on in fp64).
__device__ __forceinline__ void cost_chunk(const uint4 &v, uint32_t ia8, float theta, uint32_t &kept_i, uint32_t &kept_a,
                                           uint32_t &lost, float &cost_f)
{
    const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
    uint32_t i8 = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const float m = __uint_as_float(((e & 1) ? ww[e >> 1] : (ww[e >> 1] << 16)) & 0x7FFF0000u);   // M = |W|
        const bool i = m >= theta;                                          // I (false for NaN)
        i8 |= i ? (1u << e) : 0u;
        cost_f += (i && !((ia8 >> e) & 1u)) ? m : 0.f;
    }
    ia8 &= 0xFFu;
    kept_i += __popc(i8);
    kept_a += __popc(ia8);
    lost += __popc(i8 & ~ia8);
}

__device__ __forceinline__ void cost_element(uint32_t wbits, bool ia, float theta, CostAcc &a, float &cost_f)
{
    const float m = fabsf(__uint_as_float(wbits << 16));                     // M = |W|
    const bool i = m >= theta;                                              // I (false for NaN)
    a.kept_i += i;
    a.kept_a += ia;
    if (i && !ia) { a.lost += 1; cost_f += m; }
}

// FAST: cols % 8 == 0, tn % 32 == 0 (or one tile column with cols % 32 == 0 handled by zero planes), planes fit shared memory.
// grid = (bands per tile, tiles).  Shared memory: planes[kw*32][tnw] (FAST only).
// U: 256-column chunks of a row that a warp takes at a time (a tile of 512 columns has two: four would leave half
// of every step idle).
template <bool FAST, int U>
__global__ void __launch_bounds__(A1_THREADS)
index_cost_kernel(Geo g, const uint16_t *__restrict__ W, float theta, const uint32_t *__restrict__ ip,
                  const uint32_t *__restrict__ iz, lrbi_tile_cost *__restrict__ out)
{
    extern __shared__ __align__(16) uint32_t a1_planes[];
    __shared__ CostAcc red[A1_THREADS / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int tile = blockIdx.y, tr = tile / g.gc, tc = tile - tr * g.gc;
    const int i_begin = blockIdx.x * A1_BAND;
    const int i_end = min(min(g.tm, g.rows - tr * g.tm), i_begin + A1_BAND);
    const int ncols = min(g.tn, g.cols - tc * g.tn);                        // columns of the tile inside the matrix
    const uint32_t tail = tail_mask(g.k);
    const int tnw = (g.tn + 31) >> 5;
    CostAcc acc = {0ull, 0ull, 0ull, 0.0};

    if (FAST) {
        // bit-planes of the tile's Iz: plane l, word w = bits of row l of Iz over columns 32 w .. 32 w + 31
        for (int pi = warp; pi < g.kw * tnw; pi += A1_THREADS / 32) {
            const int lb = pi / tnw, w = pi - lb * tnw;
            const int j = w * 32 + lane;
            uint32_t z = j < ncols ? __ldg(iz + ((size_t)tile * g.tn + j) * g.kw + lb) : 0u;
            if (lb == g.kw - 1) z &= tail;
            a1_planes[(lb * 32 + lane) * tnw + w] = warp_transpose32(z, lane);
        }
        __syncthreads();
        // A warp walks (row, 256-column chunk) pairs; a lane owns 8 consecutive columns of a chunk.  The weights
        // of the next pair are requested before the current one is evaluated.
        const int nch = (ncols + 255) >> 8;
        const int nrows_w = i_begin + warp < i_end ? (i_end - i_begin - warp + A1_THREADS / 32 - 1) / (A1_THREADS / 32) : 0;
        const uint16_t *wtile = W + (size_t)(tr * g.tm) * g.cols + (size_t)tc * g.tn;
        auto load_w = [&](int j, int ch) {
            const int c = ch * 256 + lane * 8;                              // cols % 8 == 0 and tn % 8 == 0: all 8 exist or none
            return (j < nrows_w && ch < nch && c < ncols)
                       ? __ldg(reinterpret_cast<const uint4 *>(wtile + (size_t)(i_begin + warp + j * (A1_THREADS / 32)) * g.cols + c))
                       : make_uint4(0, 0, 0, 0);
        };
        uint32_t n_i = 0, n_a = 0, n_l = 0;
        // groups of U chunks (U * 256 columns of a row): a warp keeps U * 512 bytes requested ahead of what it evaluates
        const int ngr = (nch + U - 1) / U;
        uint4 wnext[U];
#pragma unroll
        for (int u = 0; u < U; ++u) wnext[u] = load_w(0, u);
        for (int j = 0; j < nrows_w; ++j) {
            const int i = i_begin + warp + j * (A1_THREADS / 32);
            const uint32_t *ipw = ip + ((size_t)tile * g.tm + i) * g.kw;
            for (int gr4 = 0; gr4 < ngr; ++gr4) {
                uint4 v[U];
#pragma unroll
                for (int u = 0; u < U; ++u) v[u] = wnext[u];
                const int jn = gr4 + 1 < ngr ? j : j + 1, gn = gr4 + 1 < ngr ? gr4 + 1 : 0;
#pragma unroll
                for (int u = 0; u < U; ++u) wnext[u] = load_w(jn, gn * U + u);
                uint32_t bits[U];                                           // index bits of the words that hold this lane's columns
#pragma unroll
                for (int u = 0; u < U; ++u) bits[u] = 0u;
                const int word0 = gr4 * (8 * U) + (lane >> 2);              // chunk u: word0 + 8 u
                for (int lb = 0; lb < g.kw; ++lb) {
                    uint32_t x = __ldg(ipw + lb);                           // warp-uniform: no divergence below
                    if (lb == g.kw - 1) x &= tail;
                    while (x) {
                        const uint32_t *pl = a1_planes + (lb * 32 + __ffs(x) - 1) * tnw;
                        x &= x - 1;
#pragma unroll
                        for (int u = 0; u < U; ++u) bits[u] |= pl[min(word0 + 8 * u, tnw - 1)];
                    }
                }
                float cf = 0.f;                                             // fp32 over the group's 8 U weights, fp64 beyond
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int c = (gr4 * U + u) * 256 + lane * 8;
                    if (c < ncols) cost_chunk(v[u], bits[u] >> (c & 31), theta, n_i, n_a, n_l, cf);
                }
                acc.cost += (double)cf;
            }
        }
        acc.kept_i = n_i; acc.kept_a = n_a; acc.lost = n_l;
    } else {
        // any shape: one column per lane, Eq. 3 evaluated per element from the packed words
        for (int i = i_begin + warp; i < i_end; i += A1_THREADS / 32) {
            const uint32_t *ipw = ip + ((size_t)tile * g.tm + i) * g.kw;
            const uint16_t *wrow = W + (size_t)(tr * g.tm + i) * g.cols + (size_t)tc * g.tn;
            for (int c = lane; c < ncols; c += 32) {
                const uint32_t *izw = iz + ((size_t)tile * g.tn + c) * g.kw;
                uint32_t any = 0;
                for (int lb = 0; lb < g.kw; ++lb) {
                    uint32_t t = __ldg(ipw + lb) & __ldg(izw + lb);
                    if (lb == g.kw - 1) t &= tail;
                    any |= t;
                }
                float cf = 0.f;
                cost_element(wrow[c], any != 0, theta, acc, cf);
                acc.cost += (double)cf;
            }
        }
    }

    // block reduction, then one atomic update of the tile's record per block
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        acc.kept_i += __shfl_xor_sync(0xFFFFFFFFu, acc.kept_i, off);
        acc.kept_a += __shfl_xor_sync(0xFFFFFFFFu, acc.kept_a, off);
        acc.lost += __shfl_xor_sync(0xFFFFFFFFu, acc.lost, off);
        acc.cost += __shfl_xor_sync(0xFFFFFFFFu, acc.cost, off);
    }
    if (lane == 0) red[warp] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        CostAcc t = red[0];
        for (int w = 1; w < A1_THREADS / 32; ++w) {
            t.kept_i += red[w].kept_i; t.kept_a += red[w].kept_a; t.lost += red[w].lost; t.cost += red[w].cost;
        }
        lrbi_tile_cost *o = out + tile;
        atomicAdd(reinterpret_cast<unsigned long long *>(&o->kept_i), t.kept_i);
        atomicAdd(reinterpret_cast<unsigned long long *>(&o->kept_a), t.kept_a);
        atomicAdd(reinterpret_cast<unsigned long long *>(&o->lost), t.lost);
        atomicAdd(&o->cost, t.cost);
    }
}

lrbi_status launch_index_cost(const Geo &g, const uint16_t *W, float theta, const uint32_t *ip, const uint32_t *iz,
                              lrbi_tile_cost *out, cudaStream_t s)
{
    const long long tiles = (long long)g.gr * g.gc;
    if (tiles > 65535) return LRBI_ERR_UNSUPPORTED;
    cudaError_t e = cudaMemsetAsync(out, 0, (size_t)tiles * sizeof(lrbi_tile_cost), s);   // every count starts at zero
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    const int tnw = (g.tn + 31) / 32;
    const size_t smem = (size_t)g.kw * 32 * tnw * sizeof(uint32_t);
    const bool fast = (g.cols % 8) == 0 && (g.tn % 8) == 0 && smem <= 48 * 1024;
    dim3 grid((unsigned)((g.tm + A1_BAND - 1) / A1_BAND), (unsigned)tiles);
    const int nch = (g.tn + 255) / 256;                  // 256-column chunks of a tile row
    if (fast && nch <= 1) index_cost_kernel<true, 1><<<grid, A1_THREADS, smem, s>>>(g, W, theta, ip, iz, out);
    else if (fast && nch == 2) index_cost_kernel<true, 2><<<grid, A1_THREADS, smem, s>>>(g, W, theta, ip, iz, out);
    else if (fast) index_cost_kernel<true, 4><<<grid, A1_THREADS, smem, s>>>(g, W, theta, ip, iz, out);
    else index_cost_kernel<false, 1><<<grid, A1_THREADS, 0, s>>>(g, W, theta, ip, iz, out);
    count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

}  // namespace lrbi
