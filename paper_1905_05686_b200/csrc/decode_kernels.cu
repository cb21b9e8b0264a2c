// Decode of the tiled low-rank binary index into a bit-packed mask (Eq. 3 per tile).
//
// Two kernels:
//   decode_ballot  any shape.  A lane owns one column word of Iz, the row word of Ip is
//                  warp-uniform, the test is (ip & iz) != 0 and __ballot_sync builds one
//                  32-bit mask word per vote.  ~3 warp instructions per output word.
//   decode_planes  tile_cols % 32 == 0.  Iz of a block of columns is first transposed into k
//                  bit-planes (plane l = the bits of row l of Iz); a thread then owns one mask row
//                  and ORs the planes selected by the set bits of its Ip word: 32 mask bits per
//                  bitwise instruction instead of one per lane.  Two variants: 256-column blocks
//                  transposed with __ballot_sync (any tile_cols % 32 == 0), and, for
//                  tile_cols % 128 == 0 and k <= 256, 1024-column blocks transposed with warp
//                  shuffles, where a thread writes whole 128-byte lines of its mask row.
#include "lrbi_common.cuh"

namespace lrbi {

constexpr int DEC_THREADS = 256;
constexpr int DEC_WORDS = 8;          // mask words (256 columns) per block column
constexpr int STAGE_PITCH = 12;       // words per staged row (8 + pad, keeps 16-byte alignment)

// --------------------------------------------------------------------------------------
// decode_ballot
// --------------------------------------------------------------------------------------
// KWREG > 0: the lane keeps its KWREG column words of Iz in registers for all rows (kw <= KWREG).
// KWREG == 0: any kw, column words are re-read (L1) for every row.
template <int KWREG>
__global__ void __launch_bounds__(DEC_THREADS)
decode_ballot_kernel(Geo g, const uint32_t *__restrict__ ip, const uint32_t *__restrict__ iz,
                     uint32_t *__restrict__ mask)
{
    __shared__ __align__(16) uint32_t stage[DEC_THREADS / 32][32][STAGE_PITCH];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int word0 = blockIdx.x * DEC_WORDS;                  // first mask word of this block column
    const int row0 = (blockIdx.y * (DEC_THREADS / 32) + warp) * 32;
    if (row0 >= g.rows) return;                                // whole warp leaves together
    const uint32_t tail = tail_mask(g.k);

    // per lane: tile column and offset of its column in each of the 8 words
    int tc[DEC_WORDS];
    int joff[DEC_WORDS];
    bool colok[DEC_WORDS];
    uint32_t zreg[DEC_WORDS][KWREG > 0 ? KWREG : 1];
#pragma unroll
    for (int q = 0; q < DEC_WORDS; ++q) {
        const int c = (word0 + q) * 32 + lane;
        colok[q] = c < g.cols;
        const int cc = colok[q] ? c : 0;
        tc[q] = cc / g.tn;
        joff[q] = cc - tc[q] * g.tn;                           // column inside its tile
    }

    for (int rr = 0; rr < 32; ++rr) {
        const int r = row0 + rr;
        if (r >= g.rows) break;                                // warp-uniform
        const int tr = r / g.tm, i = r - tr * g.tm;
        const bool new_tile_row = (rr == 0) || (i == 0);       // column words change with the tile row
#pragma unroll
        for (int q = 0; q < DEC_WORDS; ++q) {
            const long long tile = (long long)tr * g.gc + tc[q];
            const uint32_t *ipw = ip + (tile * g.tm + i) * g.kw;            // warp-uniform when tn % 32 == 0
            const uint32_t *izw = iz + (tile * g.tn + joff[q]) * g.kw;
            uint32_t any = 0;
            if (KWREG > 0) {
                if (new_tile_row) {
#pragma unroll
                    for (int w = 0; w < KWREG; ++w) {
                        uint32_t z = (colok[q] && w < g.kw) ? __ldg(izw + w) : 0u;
                        if (w == g.kw - 1) z &= tail;
                        zreg[q][w] = z;
                    }
                }
#pragma unroll
                for (int w = 0; w < KWREG; ++w)
                    if (w < g.kw) any |= __ldg(ipw + w) & zreg[q][w];
            } else if (colok[q]) {
                for (int w = 0; w < g.kw; ++w) {
                    uint32_t t = __ldg(ipw + w) & __ldg(izw + w);
                    if (w == g.kw - 1) t &= tail;
                    any |= t;
                }
            }
            const uint32_t word = __ballot_sync(0xFFFFFFFFu, any != 0);
            if (lane == q) stage[warp][rr][q] = word;
        }
    }
    __syncwarp();

    // vectorised, row-contiguous stores: lane <-> staged row
    const int r = row0 + lane;
    if (r < g.rows) {
        uint32_t *dst = mask + (long long)r * g.pitch + word0;
        const int nw = min(DEC_WORDS, g.pitch - word0);
        if (nw == DEC_WORDS && (g.pitch & 3) == 0) {
            const uint4 *src = reinterpret_cast<const uint4 *>(&stage[warp][lane][0]);
            reinterpret_cast<uint4 *>(dst)[0] = src[0];
            reinterpret_cast<uint4 *>(dst)[1] = src[1];
        } else {
            for (int q = 0; q < nw; ++q) dst[q] = stage[warp][lane][q];
        }
    }
}

lrbi_status launch_decode_ballot(const Geo &g, const uint32_t *ip, const uint32_t *iz, uint32_t *mask,
                                 cudaStream_t s)
{
    dim3 grid((g.pitch + DEC_WORDS - 1) / DEC_WORDS, (g.rows + DEC_THREADS - 1) / DEC_THREADS);
    if (grid.y > 65535) return LRBI_ERR_UNSUPPORTED;
    if (g.kw == 1) decode_ballot_kernel<1><<<grid, DEC_THREADS, 0, s>>>(g, ip, iz, mask);
    else if (g.kw == 2) decode_ballot_kernel<2><<<grid, DEC_THREADS, 0, s>>>(g, ip, iz, mask);
    else decode_ballot_kernel<0><<<grid, DEC_THREADS, 0, s>>>(g, ip, iz, mask);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

// --------------------------------------------------------------------------------------
// decode_planes
// --------------------------------------------------------------------------------------
constexpr int PLANES_MAX_RANK = 1024;
constexpr int PLANES_ROWS_PER_BLOCK = 1024;    // up to 4 rows per thread share one plane build

bool decode_planes_supported(const Geo &g) { return (g.tn % 32) == 0 && g.k <= PLANES_MAX_RANK; }

__global__ void __launch_bounds__(DEC_THREADS)
decode_planes_kernel(Geo g, int col_blocks_per_tile, int row_bands_per_tile,
                     const uint32_t *__restrict__ ip, const uint32_t *__restrict__ iz,
                     uint32_t *__restrict__ mask)
{
    extern __shared__ __align__(16) uint32_t planes[];         // [k][DEC_WORDS]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int tc = blockIdx.x / col_blocks_per_tile, cb = blockIdx.x - tc * col_blocks_per_tile;
    const int tr = blockIdx.y / row_bands_per_tile, band = blockIdx.y - tr * row_bands_per_tile;
    const long long tile = (long long)tr * g.gc + tc;
    const int words_in_tile = g.tn >> 5;
    const int tword0 = cb * DEC_WORDS;                          // first word of this block inside the tile
    const int nw_tile = min(DEC_WORDS, words_in_tile - tword0); // words of this block that exist in the tile
    const int gword0 = tc * words_in_tile + tword0;             // first word in the mask row
    const uint32_t tail = tail_mask(g.k);

    // ---- build the bit-planes: warp q transposes the 32 column words of mask word q
    {
        const int q = warp;
        const int j = (tword0 + q) * 32 + lane;                 // column inside the tile
        const bool ok = q < nw_tile && (long long)tc * g.tn + j < g.cols;
        const uint32_t *izw = iz + (tile * g.tn + (ok ? j : 0)) * g.kw;
        for (int w = 0; w < g.kw; ++w) {
            uint32_t z = ok ? __ldg(izw + w) : 0u;
            if (w == g.kw - 1) z &= tail;
            uint32_t keep = 0;
#pragma unroll
            for (int b = 0; b < 32; ++b) {
                const uint32_t v = __ballot_sync(0xFFFFFFFFu, (z >> b) & 1u);
                if (lane == b) keep = v;
            }
            const int l = w * 32 + lane;
            if (l < g.k) planes[l * DEC_WORDS + q] = keep;
        }
    }
    __syncthreads();

    // ---- one thread per mask row: OR the planes its Ip word selects
    const int i_end = min(g.tm, g.rows - tr * g.tm);
    const int nw = min(nw_tile, g.pitch - gword0);
    for (int i = band * PLANES_ROWS_PER_BLOCK + threadIdx.x;
         i < min(i_end, (band + 1) * PLANES_ROWS_PER_BLOCK); i += DEC_THREADS) {
        uint4 m0 = make_uint4(0, 0, 0, 0), m1 = make_uint4(0, 0, 0, 0);
        const uint32_t *ipw = ip + (tile * g.tm + i) * g.kw;
        for (int w = 0; w < g.kw; ++w) {
            uint32_t x = __ldg(ipw + w);
            if (w == g.kw - 1) x &= tail;
            while (x) {
                const int l = w * 32 + __ffs(x) - 1;
                x &= x - 1;
                const uint4 *p = reinterpret_cast<const uint4 *>(planes + l * DEC_WORDS);
                const uint4 a = p[0], b = p[1];
                m0.x |= a.x; m0.y |= a.y; m0.z |= a.z; m0.w |= a.w;
                m1.x |= b.x; m1.y |= b.y; m1.z |= b.z; m1.w |= b.w;
            }
        }
        uint32_t *dst = mask + (long long)(tr * g.tm + i) * g.pitch + gword0;
        if (nw == DEC_WORDS && (g.pitch & 3) == 0 && (gword0 & 3) == 0) {
            reinterpret_cast<uint4 *>(dst)[0] = m0;
            reinterpret_cast<uint4 *>(dst)[1] = m1;
        } else {
            const uint32_t v[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
#pragma unroll
            for (int q = 0; q < DEC_WORDS; ++q)
                if (q < nw) dst[q] = v[q];
        }
    }
}

// --------------------------------------------------------------------------------------
// decode_planes, wide variant: a block decodes up to 1024 rows x 1024 columns
// --------------------------------------------------------------------------------------
constexpr int WIDE_WORDS = 32;          // mask words (1024 columns = one 128-byte line) per row and block
constexpr int WIDE_PITCH = 36;          // words between planes in shared memory (16-byte aligned, spreads banks)
constexpr int WIDE_MAX_RANK = 256;

// SEGQ = 128-column quads per run of columns that lies inside one tile (8: the whole block).
template <int SEGQ>
__global__ void __launch_bounds__(DEC_THREADS, SEGQ <= 2 ? 8 : 4)
decode_planes_wide_kernel(Geo g, int row_bands_per_tile, int rows_per_block,
                          const uint32_t *__restrict__ ip, const uint32_t *__restrict__ iz,
                          uint32_t *__restrict__ mask)
{
    extern __shared__ __align__(16) uint32_t planes[];         // [kw*32][WIDE_PITCH]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gw0 = blockIdx.x * WIDE_WORDS;                    // first mask word of this block's columns
    const int tr = blockIdx.y / row_bands_per_tile, band = blockIdx.y - tr * row_bands_per_tile;
    const int words_in_tile = g.tn >> 5;
    const uint32_t tail = tail_mask(g.k);
    const int i_end = min(g.tm, g.rows - tr * g.tm);
    const int i_first = band * rows_per_block + threadIdx.x;

    // Row words of Ip for this thread's first row, requested before the planes are built so that their
    // trip from memory overlaps the trip of the column words (k <= 64; larger ranks load them later).
    constexpr int NSEG = 8 / SEGQ;
    uint32_t xpre[NSEG][2];
    const bool pre = g.kw <= 2;
#pragma unroll
    for (int seg = 0; seg < NSEG; ++seg) {
        const int gw = gw0 + seg * SEGQ * 4;
        const bool live = pre && gw < g.pitch && i_first < i_end;
        const uint32_t *ipw = ip + (((long long)tr * g.gc + (live ? gw / words_in_tile : 0)) * g.tm + (live ? i_first : 0)) * g.kw;
#pragma unroll
        for (int lb = 0; lb < 2; ++lb) xpre[seg][lb] = (live && lb < g.kw) ? __ldg(ipw + lb) : 0u;
    }

    // ---- bit-planes of the block's 1024 columns: one warp transpose per (32 planes, mask word)
    for (int pi = warp; pi < g.kw * WIDE_WORDS; pi += DEC_THREADS / 32) {
        const int lb = pi / WIDE_WORDS, w = pi - lb * WIDE_WORDS;
        const int c = (gw0 + w) * 32 + lane;                    // column of this lane
        uint32_t z = 0;
        if (c < g.cols) {
            const int tc = c / g.tn, j = c - tc * g.tn;
            z = __ldg(iz + (((long long)tr * g.gc + tc) * g.tn + j) * g.kw + lb);
            if (lb == g.kw - 1) z &= tail;
        }
        planes[(lb * 32 + lane) * WIDE_PITCH + w] = warp_transpose32(z, lane);   // lane l keeps plane lb*32 + l
    }
    __syncthreads();

    // ---- one thread per mask row; per run of quads inside one tile, OR the planes its Ip word selects
    const bool vec = (g.pitch & 3) == 0;
    for (int i = i_first; i < min(i_end, (band + 1) * rows_per_block); i += DEC_THREADS) {
        uint32_t *dst = mask + (long long)(tr * g.tm + i) * g.pitch + gw0;
#pragma unroll
        for (int seg = 0; seg < 8 / SEGQ; ++seg) {
            const int gw = gw0 + seg * SEGQ * 4;                // first mask word of the run
            if (gw >= g.pitch) break;
            uint4 acc[SEGQ];                                    // the run's index bits of this row
#pragma unroll
            for (int q = 0; q < SEGQ; ++q) acc[q] = make_uint4(0, 0, 0, 0);
            const int tc = gw / words_in_tile;
            const uint32_t *ipw = ip + (((long long)tr * g.gc + tc) * g.tm + i) * g.kw;
            auto or_planes = [&](uint32_t x, int lb) {
                if (lb == g.kw - 1) x &= tail;
                while (x) {
                    const int l = lb * 32 + __ffs(x) - 1;
                    x &= x - 1;
                    const uint4 *src = reinterpret_cast<const uint4 *>(planes + l * WIDE_PITCH + seg * SEGQ * 4);
#pragma unroll
                    for (int q = 0; q < SEGQ; ++q) {
                        const uint4 v = src[q];
                        uint4 &a = acc[q];
                        a.x |= v.x; a.y |= v.y; a.z |= v.z; a.w |= v.w;
                    }
                }
            };
            if (pre && i == i_first) {                   // statically indexed: the prefetched words stay in registers
                or_planes(xpre[seg][0], 0);
                if (g.kw > 1) or_planes(xpre[seg][1], 1);
            } else {
                for (int lb = 0; lb < g.kw; ++lb) or_planes(__ldg(ipw + lb), lb);
            }
            // store the run; the thread's runs together fill one 128-byte line of its mask row
#pragma unroll
            for (int q = 0; q < SEGQ; ++q) {
                const int w = seg * SEGQ * 4 + q * 4;           // word inside the block
                const int nw = g.pitch - gw0 - w;               // words of this quad that exist in the row
                if (nw >= 4 && vec) {
                    *reinterpret_cast<uint4 *>(dst + w) = acc[q];
                } else if (nw > 0) {
                    const uint32_t v[4] = {acc[q].x, acc[q].y, acc[q].z, acc[q].w};
                    for (int e = 0; e < min(nw, 4); ++e) dst[w + e] = v[e];
                }
            }
        }
    }
}

static bool decode_planes_wide_supported(const Geo &g) { return (g.tn % 128) == 0 && g.k <= WIDE_MAX_RANK; }

lrbi_status launch_decode_planes_wide(const Geo &g, const uint32_t *ip, const uint32_t *iz, uint32_t *mask,
                                      cudaStream_t s)
{
    if (!decode_planes_wide_supported(g)) return LRBI_ERR_UNSUPPORTED;
    const int rows_per_block = g.tm >= 1024 ? 1024 : (g.tm + DEC_THREADS - 1) / DEC_THREADS * DEC_THREADS;
    const int rbpt = (g.tm + rows_per_block - 1) / rows_per_block;
    dim3 grid((unsigned)((g.pitch + WIDE_WORDS - 1) / WIDE_WORDS), (unsigned)(g.gr * rbpt));
    if (grid.y > 65535) return LRBI_ERR_UNSUPPORTED;
    const size_t smem = (size_t)g.kw * 32 * WIDE_PITCH * sizeof(uint32_t);       // <= 36 KB
    const int segq = (g.tn % 1024) == 0 || g.gc == 1 ? 8 : (g.tn % 512) == 0 ? 4 : (g.tn % 256) == 0 ? 2 : 1;
    if (segq == 8) decode_planes_wide_kernel<8><<<grid, DEC_THREADS, smem, s>>>(g, rbpt, rows_per_block, ip, iz, mask);
    else if (segq == 4) decode_planes_wide_kernel<4><<<grid, DEC_THREADS, smem, s>>>(g, rbpt, rows_per_block, ip, iz, mask);
    else if (segq == 2) decode_planes_wide_kernel<2><<<grid, DEC_THREADS, smem, s>>>(g, rbpt, rows_per_block, ip, iz, mask);
    else decode_planes_wide_kernel<1><<<grid, DEC_THREADS, smem, s>>>(g, rbpt, rows_per_block, ip, iz, mask);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

lrbi_status launch_decode_planes(const Geo &g, const uint32_t *ip, const uint32_t *iz, uint32_t *mask,
                                 cudaStream_t s)
{
    if (!decode_planes_supported(g)) return LRBI_ERR_UNSUPPORTED;
    // the wide variant wants enough 1024-column blocks to fill the chip; a small mask is better served by
    // the many small blocks of the 256-column variant
    const long long wide_blocks = (long long)((g.pitch + WIDE_WORDS - 1) / WIDE_WORDS) * g.gr * ((g.tm + 1023) / 1024);
    if (decode_planes_wide_supported(g) && wide_blocks >= 256) return launch_decode_planes_wide(g, ip, iz, mask, s);
    const int cbpt = ((g.tn >> 5) + DEC_WORDS - 1) / DEC_WORDS;
    const int rbpt = (g.tm + PLANES_ROWS_PER_BLOCK - 1) / PLANES_ROWS_PER_BLOCK;
    dim3 grid((unsigned)(g.gc * cbpt), (unsigned)(g.gr * rbpt));
    if (grid.y > 65535) return LRBI_ERR_UNSUPPORTED;
    const size_t smem = (size_t)g.k * DEC_WORDS * sizeof(uint32_t);
    decode_planes_kernel<<<grid, DEC_THREADS, smem, s>>>(g, cbpt, rbpt, ip, iz, mask);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

}  // namespace lrbi
