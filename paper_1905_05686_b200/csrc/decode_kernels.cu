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
#include <mutex>

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

// SEGQ = 128-column quads per run of columns that lies inside one tile: the tile is SEGQ * 128 columns wide
// (SEGQ = 1, 2, 4), or a multiple of 1024 columns / the only tile column (SEGQ = 8: the whole item is one run).
// An item therefore starts on a tile boundary and run `seg` lies in tile column tc0 + seg: no division per row.
// TABLES (rank <= 8): instead of walking the set bits of a row word, the block first ORs the planes into two
// 16-entry tables (one per nibble of the row word: entry e = OR of the planes whose bits are set in e), and a row
// is then two look-ups and one OR per 128 columns, with no data-dependent loop.
// The grid is persistent: a block walks work items (1024 columns x up to rows_per_block rows of one tile row) and
// requests the factor words of its next item (cp.async into a second buffer) before it decodes the current one, so
// the trip of those words from HBM is waited for only once.
__device__ __forceinline__ void cp_async_4(void *dst_smem, const void *src, bool valid)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src), "r"(valid ? 4 : 0) : "memory");
}

template <int SEGQ, bool TABLES>
__global__ void __launch_bounds__(DEC_THREADS, 4)
decode_planes_wide_kernel(Geo g, int row_bands_per_tile, int rows_per_block, int items_x, int items,
                          const uint32_t *__restrict__ ip, const uint32_t *__restrict__ iz,
                          uint32_t *__restrict__ mask)
{
    extern __shared__ __align__(16) uint32_t planes[];         // [kw*32][WIDE_PITCH], then tables, staging, factor buffers
    constexpr int NSEG = 8 / SEGQ;                              // runs per item
    constexpr int RUN_WORDS = SEGQ * 4;                         // mask words per run
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t tail = tail_mask(g.k);
    const int kw = g.kw;
    const size_t iz_tile = (size_t)g.tn * kw, ip_tile = (size_t)g.tm * kw;
    uint32_t *tables = planes + kw * 32 * WIDE_PITCH;          // [2][16][WIDE_PITCH], TABLES only (kw == 1)
    uint32_t *stage_all = tables + (TABLES ? 32 : 0) * WIDE_PITCH;                 // [DEC_THREADS][WIDE_PITCH]
    uint32_t *zbuf = stage_all + DEC_THREADS * WIDE_PITCH;      // [2][1024 * kw]  column words of the item's 1024 columns
    uint32_t *xbuf = zbuf + 2 * 1024 * kw;                      // [2][DEC_THREADS][NSEG * kw]  row words of its first 256 rows
    uint32_t *stage = stage_all + warp * 32 * WIDE_PITCH;       // [32 rows][WIDE_PITCH]

    struct Item { int gw0, tr, band, tc0, j00, i_limit; };     // geometry of a work item
    auto item_of = [&](int it) {
        Item m;
        const int bx = it % items_x, by = it / items_x;
        m.gw0 = bx * WIDE_WORDS;                                // first mask word of the item's columns
        m.tr = by / row_bands_per_tile;
        m.band = by - m.tr * row_bands_per_tile;
        m.tc0 = (m.gw0 * 32) / g.tn;                            // tile column of run 0
        m.j00 = m.gw0 * 32 - m.tc0 * g.tn;                      // first column of the item inside that tile (SEGQ = 8)
        m.i_limit = min(min(g.tm, g.rows - m.tr * g.tm), (m.band + 1) * rows_per_block);
        return m;
    };
    // column word (col, lb) of the item lands at zbuf[buf][col * kw + lb]; row word (thread, seg, lb) at
    // xbuf[buf][(thread * NSEG + seg) * kw + lb]; what falls outside the matrix is filled with zero
    auto request = [&](int it, int buf) {
        if (it < items) {
            const Item m = item_of(it);
            const uint32_t *iz0 = iz + ((size_t)m.tr * g.gc + m.tc0) * g.tn * kw;
            const uint32_t *ip0 = ip + ((size_t)m.tr * g.gc + m.tc0) * g.tm * kw;
#pragma unroll
            for (int col = threadIdx.x; col < 1024; col += DEC_THREADS) {
                const int seg = col / (SEGQ * 128);
                const int j = NSEG > 1 ? col - seg * SEGQ * 128 : m.j00 + col;
                const bool ok = m.gw0 * 32 + col < g.cols;
                const uint32_t *src = iz0 + (NSEG > 1 ? seg * iz_tile : 0) + (size_t)(ok ? j : 0) * kw;
                for (int lb = 0; lb < kw; ++lb) cp_async_4(zbuf + buf * 1024 * kw + col * kw + lb, src + lb, ok);
            }
            const int i = m.band * rows_per_block + threadIdx.x;
#pragma unroll
            for (int seg = 0; seg < NSEG; ++seg) {
                const bool ok = i < m.i_limit && m.gw0 + seg * RUN_WORDS < g.pitch;
                for (int lb = 0; lb < kw; ++lb)
                    cp_async_4(xbuf + buf * DEC_THREADS * NSEG * kw + (threadIdx.x * NSEG + seg) * kw + lb,
                               ip0 + seg * ip_tile + (size_t)(ok ? i : 0) * kw + lb, ok);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    int buf = 0;
    request(blockIdx.x, 0);
    for (int item = blockIdx.x; item < items; item += gridDim.x, buf ^= 1) {
        request(item + gridDim.x, buf ^ 1);                     // next item's factor words start their trip now
        asm volatile("cp.async.wait_group 1;" ::: "memory");    // this item's have landed (this thread's requests)
        __syncthreads();                                        // ... and everybody else's
        const Item m = item_of(item);
        const int gw0 = m.gw0, tr = m.tr;
        const uint32_t *ip0 = ip + ((size_t)tr * g.gc + m.tc0) * g.tm * kw;
        const uint32_t *zb = zbuf + buf * 1024 * kw;
        const uint32_t *xb = xbuf + buf * DEC_THREADS * NSEG * kw + threadIdx.x * NSEG * kw;

        // ---- bit-planes of the item's 1024 columns: one warp transpose per (32 planes, mask word), four at a time
        for (int p0 = warp; p0 < kw * WIDE_WORDS; p0 += 4 * (DEC_THREADS / 32)) {
            uint32_t z[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int pi = p0 + u * (DEC_THREADS / 32);
                const int lb = pi >> 5, w = pi & 31;            // WIDE_WORDS == 32
                z[u] = pi < kw * WIDE_WORDS ? zb[(w * 32 + lane) * kw + lb] : 0u;
                if (lb == kw - 1) z[u] &= tail;
            }
            warp_transpose32_x4(z, lane);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int pi = p0 + u * (DEC_THREADS / 32);
                if (pi < kw * WIDE_WORDS) planes[((pi >> 5) * 32 + lane) * WIDE_PITCH + (pi & 31)] = z[u];   // lane l keeps plane lb*32 + l
            }
        }
        __syncthreads();
        if (TABLES) {
            const int e = threadIdx.x >> 3, q = threadIdx.x & 7;    // table entry 0..31 (nibble h = e / 16), quad of words
            uint4 v = make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int b = 0; b < 4; ++b)
                if ((e >> b) & 1) {
                    const uint4 pl = *reinterpret_cast<const uint4 *>(planes + ((e >> 4) * 4 + b) * WIDE_PITCH + q * 4);
                    v.x |= pl.x; v.y |= pl.y; v.z |= pl.z; v.w |= pl.w;
                }
            *reinterpret_cast<uint4 *>(tables + e * WIDE_PITCH + q * 4) = v;
            __syncthreads();
        }

        // ---- one thread per mask row; per run, OR the planes its Ip word selects
        const bool vec = (g.pitch & 3) == 0;
        // Whole 128-byte lines (the usual case): a warp stages the lines of its 32 rows in shared memory and writes
        // them out four lines per store instruction, instead of 32 separate 16-byte pieces.
        const bool staged = vec && g.pitch - gw0 >= WIDE_WORDS;
        const int ib0 = m.band * rows_per_block + warp * 32;
        for (int ib = ib0; ib < m.i_limit; ib += DEC_THREADS) {   // warp-uniform
            const int i = ib + lane;
            const bool first = ib == ib0;                       // the rows whose words were requested ahead
            uint32_t *row0 = mask + ((size_t)tr * g.tm + ib) * g.pitch + gw0;   // the warp's first row, this item's columns
            if (i < m.i_limit) {
                uint32_t *dst = staged ? stage + lane * WIDE_PITCH : row0 + (size_t)lane * g.pitch;
#pragma unroll
                for (int seg = 0; seg < NSEG; ++seg) {
                    if (gw0 + seg * RUN_WORDS >= g.pitch) break;
                    uint4 acc[SEGQ];                            // the run's index bits of this row
#pragma unroll
                    for (int q = 0; q < SEGQ; ++q) acc[q] = make_uint4(0, 0, 0, 0);
                    const uint32_t *ipw = ip0 + seg * ip_tile + (size_t)i * kw;
                    if (TABLES) {
                        const uint32_t x = (first ? xb[seg] : __ldg(ipw)) & tail;
                        const uint4 *lo = reinterpret_cast<const uint4 *>(tables + (x & 15u) * WIDE_PITCH + seg * RUN_WORDS);
                        const uint4 *hi = reinterpret_cast<const uint4 *>(tables + (16u + (x >> 4)) * WIDE_PITCH + seg * RUN_WORDS);
#pragma unroll
                        for (int q = 0; q < SEGQ; ++q) {
                            const uint4 a = lo[q], b = hi[q];
                            acc[q] = make_uint4(a.x | b.x, a.y | b.y, a.z | b.z, a.w | b.w);
                        }
                    } else {
                        for (int lb = 0; lb < kw; ++lb) {
                            uint32_t x = first ? xb[seg * kw + lb] : __ldg(ipw + lb);
                            if (lb == kw - 1) x &= tail;
                            while (x) {
                                const int l = lb * 32 + __ffs(x) - 1;
                                x &= x - 1;
                                const uint4 *src = reinterpret_cast<const uint4 *>(planes + l * WIDE_PITCH + seg * RUN_WORDS);
#pragma unroll
                                for (int q = 0; q < SEGQ; ++q) {
                                    const uint4 v = src[q];
                                    uint4 &a = acc[q];
                                    a.x |= v.x; a.y |= v.y; a.z |= v.z; a.w |= v.w;
                                }
                            }
                        }
                    }
                    // store the run; the thread's runs together fill one 128-byte line of its mask row
#pragma unroll
                    for (int q = 0; q < SEGQ; ++q) {
                        const int w = seg * RUN_WORDS + q * 4;  // word inside the item
                        const int nw = g.pitch - gw0 - w;       // words of this quad that exist in the row
                        if (staged || (nw >= 4 && vec)) {
                            *reinterpret_cast<uint4 *>(dst + w) = acc[q];
                        } else if (nw > 0) {
                            const uint32_t v[4] = {acc[q].x, acc[q].y, acc[q].z, acc[q].w};
                            for (int e = 0; e < min(nw, 4); ++e) dst[w + e] = v[e];
                        }
                    }
                }
            }
            if (staged) {
                __syncwarp();
                const int nr = min(32, m.i_limit - ib);
                const int q = lane & 7;                         // eight lanes write one row's line
                uint32_t *out = row0 + (size_t)(lane >> 3) * g.pitch + q * 4;
                const uint32_t *in = stage + (lane >> 3) * WIDE_PITCH + q * 4;
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    if (it * 4 + (lane >> 3) < nr)
                        *reinterpret_cast<uint4 *>(out + (size_t)it * 4 * g.pitch) = *reinterpret_cast<const uint4 *>(in + it * 4 * WIDE_PITCH);
                }
                __syncwarp();
            }
        }
        __syncthreads();                                        // planes, tables and this buffer may be overwritten
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

template <int SEGQ, bool TABLES>
static cudaError_t wide_launch(int items_x, int items, int blocks, size_t smem, cudaStream_t s, int dev, const Geo &g, int rbpt,
                               int rows_per_block, const uint32_t *ip, const uint32_t *iz, uint32_t *mask)
{
    auto kern = decode_planes_wide_kernel<SEGQ, TABLES>;
    {
        static bool attr_done[LRBI_MAX_DEVICES] = {false};   // the opt-in above 48 KB is per function and device
        std::lock_guard<std::mutex> lock(lib_mutex());
        if (!attr_done[dev]) {
            const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
            if (e != cudaSuccess) return e;
            attr_done[dev] = true;
        }
    }
    kern<<<(unsigned)blocks, DEC_THREADS, smem, s>>>(g, rbpt, rows_per_block, items_x, items, ip, iz, mask);
    return cudaSuccess;
}

// tiles of 128, 256 or 512 columns, or of a multiple of 1024 columns (or a single tile column whose width is a multiple of 128)
static bool decode_planes_wide_supported(const Geo &g)
{
    if (g.k > WIDE_MAX_RANK || (g.tn % 128) != 0) return false;
    return g.gc == 1 || (g.tn % 1024) == 0 || g.tn == 512 || g.tn == 256 || g.tn == 128;
}

lrbi_status launch_decode_planes_wide(const Geo &g, const uint32_t *ip, const uint32_t *iz, uint32_t *mask,
                                      cudaStream_t s)
{
    if (!decode_planes_wide_supported(g)) return LRBI_ERR_UNSUPPORTED;
    const int rows_per_block = g.tm >= 1024 ? 1024 : (g.tm + DEC_THREADS - 1) / DEC_THREADS * DEC_THREADS;
    const int rbpt = (g.tm + rows_per_block - 1) / rows_per_block;
    const long long items_x = (g.pitch + WIDE_WORDS - 1) / WIDE_WORDS, items = items_x * g.gr * rbpt;
    if (items > 0x7FFFFFFFLL) return LRBI_ERR_UNSUPPORTED;
    const bool tables = g.k <= 8;                                                // two nibble tables follow the planes
    const int segq = (g.tn % 1024) == 0 || g.gc == 1 ? 8 : g.tn / 128;
    // planes, tables, a staging line per thread, and two buffers of factor words (1024 column words, 256 x runs row words)
    const size_t smem = ((size_t)(g.kw * 32 + (tables ? 32 : 0) + DEC_THREADS) * WIDE_PITCH +
                         2 * (size_t)g.kw * (1024 + DEC_THREADS * (8 / segq))) * sizeof(uint32_t);
    int dev = 0, sm_count = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= LRBI_MAX_DEVICES) return LRBI_ERR_CUDA;
    cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
    int per_sm = (int)((220 * 1024) / (smem + 1024));
    if (per_sm > 4) per_sm = 4;
    if (per_sm < 1) return LRBI_ERR_UNSUPPORTED;
    const int blocks = (int)(items < (long long)sm_count * per_sm ? items : (long long)sm_count * per_sm);
    cudaError_t e0 = cudaSuccess;
#define LRBI_WIDE_CASE(Q) \
    if (segq == Q) { \
        if (tables) e0 = wide_launch<Q, true>((int)items_x, (int)items, blocks, smem, s, dev, g, rbpt, rows_per_block, ip, iz, mask); \
        else e0 = wide_launch<Q, false>((int)items_x, (int)items, blocks, smem, s, dev, g, rbpt, rows_per_block, ip, iz, mask); \
    }
    LRBI_WIDE_CASE(8) LRBI_WIDE_CASE(4) LRBI_WIDE_CASE(2) LRBI_WIDE_CASE(1)
#undef LRBI_WIDE_CASE
    count_launch();
    const cudaError_t e = e0 != cudaSuccess ? e0 : cudaGetLastError();
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
