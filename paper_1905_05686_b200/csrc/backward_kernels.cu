// Backward pass of the masked layer (Section 2.2 of the paper: the pruned network is retrained with the decoded
// index Ia as its masking layer).  With Y = X (W .* Ia)^T and dY = dL/dY:
//     dX = dY (W .* Ia)           dW = (dY^T X) .* Ia
// Both contractions run on the forward tensor-core kernel (gemm_tc.cu):
//   dX   is the forward product of the TRANSPOSED layer: weights W^T (the caller keeps that copy), factors swapped
//        (the row words of Ip are the column words of Ip^T and the other way round, so the packed arrays are used as
//        they are, with the tile grid walked column-major);
//   dW   is the product with X^T in the place of the weights and dY^T as the activations, on the persistent pair
//        kernel in its DW mode: X and dY are read as they are (MN-major operands of the MMA), nothing is pruned inside
//        the contraction, the index of every output tile is decoded from the layer's factors (seen through the
//        transposed layout) while the tile accumulates, and the epilogue writes zeros where Ia = 0.  Layers whose row
//        count is not a multiple of 8 run the same kernel on transposed copies; shapes that kernel does not take run
//        the product with an index of rank one whose bits are all set, followed by apply_index on dW in place.
// This file holds the helper kernels: the bf16 transpose, the in-place application of the index, a filler, and a
// slow any-shape dW.
#include "lrbi_common.cuh"

namespace lrbi {

// ---------------------------------------------------------------------------------------- transpose
// dst[c][r] = src[r][c]; 64 x 64 tiles through shared memory, 256 threads.
__global__ void __launch_bounds__(256)
transpose_bf16_kernel(const uint16_t *__restrict__ src, int rows, int cols, uint16_t *__restrict__ dst)
{
    __shared__ uint16_t tile[64][66];
    const int c0 = blockIdx.x * 64, r0 = blockIdx.y * 64;
    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;       // 64 x 4
    for (int r = ty; r < 64; r += 4)
        if (r0 + r < rows && c0 + tx < cols) tile[r][tx] = src[(size_t)(r0 + r) * cols + c0 + tx];
    __syncthreads();
    for (int c = ty; c < 64; c += 4)
        if (c0 + c < cols && r0 + tx < rows) dst[(size_t)(c0 + c) * rows + r0 + tx] = tile[tx][c];
}

// The same with 16-byte accesses on both sides (rows % 8 == 0, cols % 8 == 0): a thread reads 8 consecutive values of
// a row, and writes 8 consecutive values of a row of the result gathered from a column of the tile.
__global__ void __launch_bounds__(256)
transpose_bf16_vec_kernel(const uint16_t *__restrict__ src, int rows, int cols, uint16_t *__restrict__ dst)
{
    __shared__ uint16_t tile[64][64 + 2];
    const int c0 = blockIdx.x * 64, r0 = blockIdx.y * 64;
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int idx = threadIdx.x + 256 * u, r = idx >> 3, cs = (idx & 7) * 8;     // 64 rows x 8 pieces of 8
        uint4 v = make_uint4(0, 0, 0, 0);
        if (r0 + r < rows && c0 + cs < cols) v = *reinterpret_cast<const uint4 *>(src + (size_t)(r0 + r) * cols + c0 + cs);
        uint32_t *t32 = reinterpret_cast<uint32_t *>(&tile[r][cs]);                   // row pitch 132 bytes: 4-byte aligned
        t32[0] = v.x; t32[1] = v.y; t32[2] = v.z; t32[3] = v.w;
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int idx = threadIdx.x + 256 * u, c = idx >> 3, rs = (idx & 7) * 8;      // 64 result rows x 8 pieces of 8
        if (c0 + c < cols && r0 + rs < rows) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) w[e] = (uint32_t)tile[rs + 2 * e][c] | ((uint32_t)tile[rs + 2 * e + 1][c] << 16);
            *reinterpret_cast<uint4 *>(dst + (size_t)(c0 + c) * rows + r0 + rs) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

lrbi_status launch_transpose_bf16(const uint16_t *src, int rows, int cols, uint16_t *dst, cudaStream_t s)
{
    dim3 grid((unsigned)((cols + 63) / 64), (unsigned)((rows + 63) / 64));
    if (grid.y > 65535) return LRBI_ERR_UNSUPPORTED;
    const bool vec = (rows % 8) == 0 && (cols % 8) == 0 && ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15u) == 0;
    if (vec) transpose_bf16_vec_kernel<<<grid, 256, 0, s>>>(src, rows, cols, dst);
    else transpose_bf16_kernel<<<grid, 256, 0, s>>>(src, rows, cols, dst);
    count_launch();
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

__global__ void fill_words_kernel(uint32_t *dst, size_t n, uint32_t value)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) dst[i] = value;
}
lrbi_status launch_fill_words(uint32_t *dst, size_t n, uint32_t value, cudaStream_t s)
{
    size_t blocks = (n + 255) / 256;
    if (blocks > 1024) blocks = 1024;
    if (blocks == 0) return LRBI_OK;
    fill_words_kernel<<<(unsigned)blocks, 256, 0, s>>>(dst, n, value);
    count_launch();
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

// ---------------------------------------------------------------------------------------- apply_index
// data[o][i] = Ia[o][i] ? data[o][i] : 0, in place; data is [rows][cols] of bf16 (ESZ = 2) or fp32 (ESZ = 4).
// A block owns a 64-row band of one tile: the tile's Iz goes into bit-planes in shared memory, a warp walks rows,
// a lane owns 8 consecutive elements of each 256-column chunk (FAST: cols % 8 == 0, tile_cols % 8 == 0).
constexpr int AP_THREADS = 256;
constexpr int AP_BAND = 64;

template <int ESZ, bool FAST>
__global__ void __launch_bounds__(AP_THREADS)
apply_index_kernel(Geo g, const uint32_t *__restrict__ ip, const uint32_t *__restrict__ iz, uint8_t *__restrict__ data)
{
    extern __shared__ __align__(16) uint32_t ap_planes[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int tile = blockIdx.y, tr = tile / g.gc, tc = tile - tr * g.gc;
    const int i_begin = blockIdx.x * AP_BAND;
    const int i_end = min(min(g.tm, g.rows - tr * g.tm), i_begin + AP_BAND);
    const int ncols = min(g.tn, g.cols - tc * g.tn);
    const uint32_t tail = tail_mask(g.k);
    const int tnw = (g.tn + 31) >> 5;
    if (FAST) {
        for (int pi = warp; pi < g.kw * tnw; pi += AP_THREADS / 32) {
            const int lb = pi / tnw, w = pi - lb * tnw;
            const int j = w * 32 + lane;
            uint32_t z = j < ncols ? __ldg(iz + ((size_t)tile * g.tn + j) * g.kw + lb) : 0u;
            if (lb == g.kw - 1) z &= tail;
            ap_planes[(lb * 32 + lane) * tnw + w] = warp_transpose32(z, lane);
        }
        __syncthreads();
        for (int i = i_begin + warp; i < i_end; i += AP_THREADS / 32) {
            const uint32_t *ipw = ip + ((size_t)tile * g.tm + i) * g.kw;
            uint8_t *row = data + ((size_t)(tr * g.tm + i) * g.cols + (size_t)tc * g.tn) * ESZ;
            for (int c0 = 0; c0 < ncols; c0 += 256) {
                const int c = c0 + lane * 8;
                const int word = min(c >> 5, tnw - 1);
                uint32_t bits = 0;
                for (int lb = 0; lb < g.kw; ++lb) {
                    uint32_t x = __ldg(ipw + lb);                           // warp-uniform
                    if (lb == g.kw - 1) x &= tail;
                    while (x) {
                        bits |= ap_planes[(lb * 32 + __ffs(x) - 1) * tnw + word];
                        x &= x - 1;
                    }
                }
                if (c < ncols) {
                    const uint32_t b8 = (bits >> (c & 31)) & 0xFFu;
                    if (b8 != 0xFFu) {                                      // something to prune among the eight
                        if (ESZ == 2) {
                            uint4 v = *reinterpret_cast<uint4 *>(row + (size_t)c * 2);
                            uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                w4[e] &= ((b8 >> (2 * e)) & 1u ? 0x0000FFFFu : 0u) | ((b8 >> (2 * e + 1)) & 1u ? 0xFFFF0000u : 0u);
                            *reinterpret_cast<uint4 *>(row + (size_t)c * 2) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                        } else {
                            uint4 *p = reinterpret_cast<uint4 *>(row + (size_t)c * 4);
                            uint4 a = p[0], b = p[1];
                            if (!(b8 & 1u)) a.x = 0;  if (!(b8 & 2u)) a.y = 0;  if (!(b8 & 4u)) a.z = 0;  if (!(b8 & 8u)) a.w = 0;
                            if (!(b8 & 16u)) b.x = 0; if (!(b8 & 32u)) b.y = 0; if (!(b8 & 64u)) b.z = 0; if (!(b8 & 128u)) b.w = 0;
                            p[0] = a; p[1] = b;
                        }
                    }
                }
            }
        }
    } else {
        for (int i = i_begin + warp; i < i_end; i += AP_THREADS / 32) {
            const uint32_t *ipw = ip + ((size_t)tile * g.tm + i) * g.kw;
            uint8_t *row = data + ((size_t)(tr * g.tm + i) * g.cols + (size_t)tc * g.tn) * ESZ;
            for (int c = lane; c < ncols; c += 32) {
                const uint32_t *izw = iz + ((size_t)tile * g.tn + c) * g.kw;
                uint32_t any = 0;
                for (int lb = 0; lb < g.kw; ++lb) {
                    uint32_t t = __ldg(ipw + lb) & __ldg(izw + lb);
                    if (lb == g.kw - 1) t &= tail;
                    any |= t;
                }
                if (!any) {
                    if (ESZ == 2) reinterpret_cast<uint16_t *>(row)[c] = 0;
                    else reinterpret_cast<uint32_t *>(row)[c] = 0;
                }
            }
        }
    }
}

lrbi_status launch_apply_index(const Geo &g, const uint32_t *ip, const uint32_t *iz, void *data, int dtype, cudaStream_t s)
{
    const long long tiles = (long long)g.gr * g.gc;
    if (tiles > 65535) return LRBI_ERR_UNSUPPORTED;
    const int tnw = (g.tn + 31) / 32;
    const size_t smem = (size_t)g.kw * 32 * tnw * sizeof(uint32_t);
    const bool fast = (g.cols % 8) == 0 && (g.tn % 8) == 0 && smem <= 48 * 1024;
    dim3 grid((unsigned)((g.tm + AP_BAND - 1) / AP_BAND), (unsigned)tiles);
    uint8_t *d = static_cast<uint8_t *>(data);
    if (dtype == LRBI_Y_F32) {
        if (fast) apply_index_kernel<4, true><<<grid, AP_THREADS, smem, s>>>(g, ip, iz, d);
        else apply_index_kernel<4, false><<<grid, AP_THREADS, 0, s>>>(g, ip, iz, d);
    } else {
        if (fast) apply_index_kernel<2, true><<<grid, AP_THREADS, smem, s>>>(g, ip, iz, d);
        else apply_index_kernel<2, false><<<grid, AP_THREADS, 0, s>>>(g, ip, iz, d);
    }
    count_launch();
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

// ---------------------------------------------------------------------------------------- dW, any shape
// One thread per weight: Eq. 3 for its index bit, then the sum over the batch for a kept weight.  Slow.
__global__ void __launch_bounds__(256)
dw_generic_kernel(Geo g, const uint16_t *__restrict__ dY, const uint16_t *__restrict__ X, int batch,
                  const uint32_t *__restrict__ ip, const uint32_t *__restrict__ iz, void *__restrict__ dW, int dtype)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)g.rows * g.cols) return;
    const int o = (int)(idx / g.cols), c = (int)(idx - (long long)o * g.cols);
    const int tr = o / g.tm, i = o - tr * g.tm, tc = c / g.tn, j = c - tc * g.tn;
    const long long tile = (long long)tr * g.gc + tc;
    const uint32_t tail = tail_mask(g.k);
    uint32_t any = 0;
    for (int w = 0; w < g.kw; ++w) {
        uint32_t t = __ldg(ip + (tile * g.tm + i) * g.kw + w) & __ldg(iz + (tile * g.tn + j) * g.kw + w);
        if (w == g.kw - 1) t &= tail;
        any |= t;
    }
    float acc = 0.f;
    if (any)
        for (int b = 0; b < batch; ++b)
            acc = fmaf(__uint_as_float((uint32_t)dY[(long long)b * g.rows + o] << 16),
                       __uint_as_float((uint32_t)X[(long long)b * g.cols + c] << 16), acc);
    if (dtype == LRBI_Y_F32) reinterpret_cast<float *>(dW)[idx] = acc;
    else reinterpret_cast<uint16_t *>(dW)[idx] = f32_to_bf16_rne(acc);
}

lrbi_status launch_dw_generic(const Geo &g, const uint16_t *dY, const uint16_t *X, int batch, const uint32_t *ip,
                              const uint32_t *iz, void *dW, int dtype, cudaStream_t s)
{
    const long long total = (long long)g.rows * g.cols, blocks = (total + 255) / 256;
    if (blocks > 0x7FFFFFFFLL) return LRBI_ERR_UNSUPPORTED;
    dw_generic_kernel<<<(unsigned)blocks, 256, 0, s>>>(g, dY, X, batch, ip, iz, dW, dtype);
    count_launch();
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

}  // namespace lrbi
