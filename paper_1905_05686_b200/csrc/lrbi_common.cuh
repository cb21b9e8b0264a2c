// Shared declarations of the lrbi CUDA library (device geometry, status word, launch helpers).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "lrbi.h"

namespace lrbi {

// Geometry handed to every kernel by value.
struct Geo {
    int rows, cols;   // N_out, K_in
    int tm, tn;       // tile rows / cols
    int k, kw;        // rank, words per packed row/column
    int gr, gc;       // tile grid
    int pitch;        // mask words per row = ceil(cols / 32)
    int ts_r, ts_c;   // tile (tr, tc) is tile number tr * ts_r + tc * ts_c of the factor arrays: (gc, 1), or (1, gr) when the
                      // layer is used transposed (backward pass); only the kernels that serve that pass look at them
};

inline Geo make_geo(const lrbi_layout &l)
{
    Geo g;
    g.rows = l.rows; g.cols = l.cols; g.tm = l.tile_rows; g.tn = l.tile_cols;
    g.k = l.rank; g.kw = (l.rank + 31) / 32;
    g.gr = (l.rows + l.tile_rows - 1) / l.tile_rows;
    g.gc = (l.cols + l.tile_cols - 1) / l.tile_cols;
    g.pitch = (l.cols + 31) / 32;
    g.ts_r = g.gc; g.ts_c = 1;
    return g;
}

// One rank per tile (null pointers: the layout's rank for every tile).  Offsets count 32-bit words.
struct TileRanks {
    const int32_t *ranks;
    const long long *ip_offset;
    const long long *iz_offset;
};

// Codes a kernel leaves in the device status word when a bounded wait runs out.
enum : int {
    DEV_OK = 0,
    DEV_TIMEOUT_FULL = 0x100,   // MMA issuer waited for a filled stage
    DEV_TIMEOUT_EMPTY = 0x200,  // a producer waited for a free stage
    DEV_TIMEOUT_ACCUM = 0x300,  // epilogue waited for the accumulator
    DEV_TIMEOUT_DRAIN = 0x400,  // drain of in-flight bulk copies on the abort path
    DEV_BAD_SMEM_ALIGN = 0x500, // dynamic shared memory did not start on a 1024-byte boundary
    DEV_TIMEOUT_SELFTEST = 0x600 // the self-test's wait on a barrier nobody signals (expected to run out)
};

constexpr int LRBI_MAX_DEVICES = 64;       // size of the per-device tables

// One lock for the library's lazily initialised host state (per-device tables, the driver entry point,
// the K-split buffer, function attributes).  Entry points may be called from several host threads.
std::mutex &lib_mutex();

// Device status word (one per device that loads the module) and the host-side accessors.
int *device_status_ptr();                  // device address, resolved once per device
bool device_timeout_seen();                // a synchronising call has seen a non-zero status word on the current device
void count_launch(int n = 1);
void note_cuda_error(int code);

// Last word of a packed k-bit row/column: bits >= k are ignored.
__host__ __device__ inline uint32_t tail_mask(int k)
{
    return (k & 31) ? ((1u << (k & 31)) - 1u) : 0xFFFFFFFFu;
}

// bf16 helpers on raw bit patterns.
__device__ __forceinline__ float bf16_lo(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t pair) { return __uint_as_float(pair & 0xFFFF0000u); }
__device__ __forceinline__ uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);  // quiet NaN
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

#ifdef __CUDACC__
// 32 x 32 bit-matrix transpose across a warp: lane L gives the word x_L, lane l receives the word
// whose bit L is bit l of x_L.  Five butterfly stages of one shuffle each.  It yields the same
// 32 words as 32 __ballot_sync votes on ((x >> l) & 1), l = 0..31, at a sixth of the instructions.
__device__ __forceinline__ uint32_t warp_transpose32(uint32_t x, int lane)
{
#pragma unroll
    for (int stage = 0; stage < 5; ++stage) {
        const int j = 16 >> stage;
        const uint32_t m = stage == 0 ? 0x0000FFFFu : stage == 1 ? 0x00FF00FFu : stage == 2 ? 0x0F0F0F0Fu
                         : stage == 3 ? 0x33333333u : 0x55555555u;
        const uint32_t y = __shfl_xor_sync(0xFFFFFFFFu, x, j);
        const bool upper = (lane & j) != 0;
        const uint32_t sh = upper ? (y >> j) : (y << j);
        const uint32_t keep = upper ? ~m : m;
        x = (x & keep) | (sh & ~keep);
    }
    return x;
}

// Four independent transposes with their shuffles interleaved (latency of one, work of four).
__device__ __forceinline__ void warp_transpose32_x4(uint32_t (&x)[4], int lane)
{
#pragma unroll
    for (int stage = 0; stage < 5; ++stage) {
        const int j = 16 >> stage;
        const uint32_t m = stage == 0 ? 0x0000FFFFu : stage == 1 ? 0x00FF00FFu : stage == 2 ? 0x0F0F0F0Fu
                         : stage == 3 ? 0x33333333u : 0x55555555u;
        const bool upper = (lane & j) != 0;
        const uint32_t keep = upper ? ~m : m;
        uint32_t y[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) y[t] = __shfl_xor_sync(0xFFFFFFFFu, x[t], j);
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const uint32_t sh = upper ? (y[t] >> j) : (y[t] << j);
            x[t] = (x[t] & keep) | (sh & ~keep);
        }
    }
}
#endif

// Kernel launchers (one translation unit each).
lrbi_status launch_decode_ballot(const Geo &g, const uint32_t *ip, const uint32_t *iz, uint32_t *mask, cudaStream_t s);
lrbi_status launch_decode_planes(const Geo &g, const uint32_t *ip, const uint32_t *iz, uint32_t *mask, cudaStream_t s);
bool decode_planes_supported(const Geo &g);
lrbi_status launch_decode_planes_wide(const Geo &g, const uint32_t *ip, const uint32_t *iz, uint32_t *mask, cudaStream_t s);

lrbi_status launch_gemm_generic(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                                const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s);
bool gemv_supported(const Geo &g, int batch);
lrbi_status launch_gemv(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                        const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s);
bool stream_mma_supported(const Geo &g, int batch);
lrbi_status launch_stream_mma(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                              const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s);
bool gemm_tc_supported(const Geo &g, int batch);
// When it splits K the launcher keeps fp32 partial sums in the library-owned buffer of the device.
// force: 0 = instantiation chosen by shape, 1 = CTA pairs (one accumulator), 2 = CTA pairs (two accumulators)
lrbi_status launch_gemm_tc(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                           const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s, int force = 0,
                           const TileRanks *ranks = nullptr);   // ranks: one rank per tile (a ranked layout), or null

lrbi_status launch_gemm_tc_dw(const Geo &g, const Geo &gi, const uint16_t *Xt, const uint32_t *ip_t, const uint32_t *iz_t,
                              const uint16_t *dYt, int out_rows, void *dW, int dtype, cudaStream_t s, bool mn_major = false);

// Variant that keeps K-split partial sums in the library's fixed device array; allocates nothing.
lrbi_status launch_gemm_tc_static(const Geo &g, const uint16_t *W, const uint32_t *ip, const uint32_t *iz,
                                  const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s);
size_t gemm_tc_scratch_bytes(const Geo &g, int batch);   // fp32 partial sums the tensor-core path would keep
lrbi_status launch_bounded_wait_selftest(unsigned limit_us, cudaStream_t s);
bool gemm_tc_plan(const Geo &g, int batch, int force, lrbi_gemm_plan *out);   // fills the tensor-core fields of the plan


// Generalised layouts: one rank per tile, several layers per launch.
lrbi_status launch_decode_ranked(const Geo &g, const TileRanks &rk, const uint32_t *ip, const uint32_t *iz,
                                 uint32_t *mask, cudaStream_t s);
lrbi_status launch_decode_batch(int n, const Geo *g, const uint32_t *const *ip, const uint32_t *const *iz,
                                uint32_t *const *mask, cudaStream_t s);
lrbi_status launch_gemm_ranked_generic(const Geo &g, const TileRanks &rk, const uint16_t *W, const uint32_t *ip,
                                       const uint32_t *iz, const uint16_t *X, int batch, void *Y, int y_dtype, cudaStream_t s);

// Backward pass of the masked layer.
lrbi_status launch_transpose_bf16(const uint16_t *src, int rows, int cols, uint16_t *dst, cudaStream_t s);
lrbi_status launch_apply_index(const Geo &g, const uint32_t *ip, const uint32_t *iz, void *data, int dtype, cudaStream_t s);
lrbi_status launch_fill_words(uint32_t *dst, size_t n, uint32_t value, cudaStream_t s);
lrbi_status launch_dw_generic(const Geo &g, const uint16_t *dY, const uint16_t *X, int batch, const uint32_t *ip,
                              const uint32_t *iz, void *dW, int dtype, cudaStream_t s);

// NMF of |W| per tile (multiplicative updates).
size_t nmf_workspace_bytes(const Geo &g);
lrbi_status launch_nmf(const Geo &g, const uint16_t *W, float *mp, float *mz, int iterations, float eps, float *ws, cudaStream_t s);

// Inner loop of Algorithm 1.
lrbi_status launch_threshold_pack(const Geo &g, const float *mp, const float *mz, const float *tp, const float *tz,
                                  uint32_t *ip, uint32_t *iz, cudaStream_t s);
lrbi_status launch_index_cost(const Geo &g, const uint16_t *W, float theta, const uint32_t *ip, const uint32_t *iz,
                              lrbi_tile_cost *out, cudaStream_t s);

}  // namespace lrbi
