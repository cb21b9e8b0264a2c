// C ABI of the lrbi library: argument checks, kernel choice, host-buffer layer handle.
#include <atomic>
#include <cstring>
#include <mutex>
#include <new>

#include "lrbi_common.cuh"

namespace lrbi {

__device__ int g_device_status = 0;

static std::atomic<uint64_t> g_launches{0};
static std::atomic<int> g_last_cuda_error{0};
static std::mutex g_mutex;
static int *g_status_ptr[LRBI_MAX_DEVICES] = {nullptr};
static std::atomic<int> g_timeout_seen[LRBI_MAX_DEVICES];   // sticky: set when a synchronising call reads a non-zero status word

std::mutex &lib_mutex() { return g_mutex; }

void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
void note_cuda_error(int code) { g_last_cuda_error.store(code, std::memory_order_relaxed); }

int *device_status_ptr()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= LRBI_MAX_DEVICES) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_status_ptr[dev]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_device_status);
        if (e != cudaSuccess) { note_cuda_error((int)e); return nullptr; }
        g_status_ptr[dev] = static_cast<int *>(p);
    }
    return g_status_ptr[dev];
}

bool device_timeout_seen()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= LRBI_MAX_DEVICES) return false;
    return g_timeout_seen[dev].load(std::memory_order_relaxed) != 0;
}

// Reads the status word of the current device; the caller has synchronised whatever it cares about.
// A non-zero word makes every later compute call on the device return LRBI_ERR_TIMEOUT until it is cleared.
static int read_status_word(bool clear)
{
    int *p = device_status_ptr();
    if (!p) return -1;
    int dev = 0;
    cudaGetDevice(&dev);
    int v = 0;
    cudaError_t e = cudaMemcpy(&v, p, sizeof v, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { note_cuda_error((int)e); return -1; }
    if (v != 0) g_timeout_seen[dev].store(1, std::memory_order_relaxed);
    if (clear) {
        if (v != 0) {
            const int zero = 0;
            cudaMemcpy(p, &zero, sizeof zero, cudaMemcpyHostToDevice);
        }
        g_timeout_seen[dev].store(0, std::memory_order_relaxed);
    }
    return v;
}

static bool layout_ok(const lrbi_layout *l)
{
    if (!l) return false;
    if (l->rows < 1 || l->cols < 1 || l->tile_rows < 1 || l->tile_cols < 1 || l->rank < 1) return false;
    return true;
}
static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int choose_gemm(const Geo &g, int batch)
{
    // measured on B200 (4096 x 9216 layer, microseconds, CUDA-core GEMV / warp-MMA stream / tcgen05):
    // batch 1: 22 / 28 / 30; batch 2: 31 / 28 / 30; batch 4: 29 / 27 / 30; batch 8: 64 / 29 / 30; batch 16: - / 31 / 30
    if (batch == 1 && gemv_supported(g, batch)) return LRBI_ALGO_GEMV;
    if (batch <= 8 && stream_mma_supported(g, batch)) return LRBI_ALGO_STREAM;
    if (batch <= 4 && gemv_supported(g, batch)) return LRBI_ALGO_GEMV;
    if (gemm_tc_supported(g, batch)) return LRBI_ALGO_TENSOR;
    return LRBI_ALGO_GENERIC;
}

}  // namespace lrbi

using namespace lrbi;

extern "C" {

size_t lrbi_packed_ip_words(const lrbi_layout *l)
{
    if (!layout_ok(l)) return 0;
    Geo g = make_geo(*l);
    return (size_t)g.gr * g.gc * g.tm * g.kw;
}
size_t lrbi_packed_iz_words(const lrbi_layout *l)
{
    if (!layout_ok(l)) return 0;
    Geo g = make_geo(*l);
    return (size_t)g.gr * g.gc * g.tn * g.kw;
}
size_t lrbi_mask_words(const lrbi_layout *l)
{
    if (!layout_ok(l)) return 0;
    Geo g = make_geo(*l);
    return (size_t)g.rows * g.pitch;
}

lrbi_status lrbi_decode_mask(const lrbi_layout *layout, const uint32_t *ip, const uint32_t *iz,
                             uint32_t *mask_out, int32_t algo, void *stream)
{
    if (!layout_ok(layout) || !ip || !iz || !mask_out) return LRBI_ERR_INVALID_ARG;
    if (!aligned16(ip) || !aligned16(iz) || !aligned16(mask_out)) return LRBI_ERR_INVALID_ARG;
    if (device_timeout_seen()) return LRBI_ERR_TIMEOUT;
    const Geo g = make_geo(*layout);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (algo) {
    case LRBI_ALGO_AUTO:
        return decode_planes_supported(g) ? launch_decode_planes(g, ip, iz, mask_out, s)
                                          : launch_decode_ballot(g, ip, iz, mask_out, s);
    case LRBI_ALGO_DECODE_BALLOT: return launch_decode_ballot(g, ip, iz, mask_out, s);
    case LRBI_ALGO_DECODE_PLANES: return launch_decode_planes(g, ip, iz, mask_out, s);
    case LRBI_ALGO_DECODE_PLANES_WIDE: return launch_decode_planes_wide(g, ip, iz, mask_out, s);
    default: return LRBI_ERR_INVALID_ARG;
    }
}

int32_t lrbi_masked_gemm_choice(const lrbi_layout *layout, int32_t batch)
{
    if (!layout_ok(layout) || batch < 1) return -1;
    return choose_gemm(make_geo(*layout), batch);
}

lrbi_status lrbi_masked_gemm(const lrbi_layout *layout, const uint16_t *W, const uint32_t *ip,
                             const uint32_t *iz, const uint16_t *X, int32_t batch, void *Y,
                             int32_t y_dtype, int32_t algo, void *stream)
{
    if (!layout_ok(layout) || !W || !ip || !iz || !X || !Y || batch < 1) return LRBI_ERR_INVALID_ARG;
    if (y_dtype != LRBI_Y_BF16 && y_dtype != LRBI_Y_F32) return LRBI_ERR_INVALID_ARG;
    if (!aligned16(W) || !aligned16(ip) || !aligned16(iz) || !aligned16(X) || !aligned16(Y)) return LRBI_ERR_INVALID_ARG;
    if (device_timeout_seen()) return LRBI_ERR_TIMEOUT;
    const Geo g = make_geo(*layout);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (algo == LRBI_ALGO_AUTO) algo = choose_gemm(g, batch);
    switch (algo) {
    case LRBI_ALGO_GENERIC: return launch_gemm_generic(g, W, ip, iz, X, batch, Y, y_dtype, s);
    case LRBI_ALGO_GEMV: return launch_gemv(g, W, ip, iz, X, batch, Y, y_dtype, s);
    case LRBI_ALGO_STREAM: return launch_stream_mma(g, W, ip, iz, X, batch, Y, y_dtype, s);
    case LRBI_ALGO_TENSOR: return launch_gemm_tc(g, W, ip, iz, X, batch, Y, y_dtype, s);
    case LRBI_ALGO_TENSOR_PAIR: return launch_gemm_tc(g, W, ip, iz, X, batch, Y, y_dtype, s, 1);
    case LRBI_ALGO_TENSOR_PAIR2: return launch_gemm_tc(g, W, ip, iz, X, batch, Y, y_dtype, s, 2);
    case LRBI_ALGO_TENSOR_PAIR192: return launch_gemm_tc(g, W, ip, iz, X, batch, Y, y_dtype, s, 3);
    default: return LRBI_ERR_INVALID_ARG;
    }
}

lrbi_status lrbi_masked_gemm_static(const lrbi_layout *layout, const uint16_t *W, const uint32_t *ip,
                                    const uint32_t *iz, const uint16_t *X, int32_t batch, void *Y,
                                    int32_t y_dtype, void *stream)
{
    if (!layout_ok(layout) || !W || !ip || !iz || !X || !Y || batch < 1) return LRBI_ERR_INVALID_ARG;
    if (y_dtype != LRBI_Y_BF16 && y_dtype != LRBI_Y_F32) return LRBI_ERR_INVALID_ARG;
    if (!aligned16(W) || !aligned16(ip) || !aligned16(iz) || !aligned16(X) || !aligned16(Y)) return LRBI_ERR_INVALID_ARG;
    if (device_timeout_seen()) return LRBI_ERR_TIMEOUT;
    return launch_gemm_tc_static(make_geo(*layout), W, ip, iz, X, batch, Y, y_dtype, static_cast<cudaStream_t>(stream));
}

size_t lrbi_masked_gemm_static_bytes(const lrbi_layout *layout, int32_t batch)
{
    if (!layout_ok(layout) || batch < 1) return 0;
    const Geo g = make_geo(*layout);
    return gemm_tc_supported(g, batch) ? gemm_tc_scratch_bytes(g, batch) : 0;
}

lrbi_status lrbi_threshold_pack(const lrbi_layout *layout, const float *mp, const float *mz, const float *tp,
                                const float *tz, uint32_t *ip_out, uint32_t *iz_out, void *stream)
{
    if (!layout_ok(layout) || !mp || !mz || !tp || !tz || !ip_out || !iz_out) return LRBI_ERR_INVALID_ARG;
    if (!aligned16(ip_out) || !aligned16(iz_out)) return LRBI_ERR_INVALID_ARG;
    if (device_timeout_seen()) return LRBI_ERR_TIMEOUT;
    return launch_threshold_pack(make_geo(*layout), mp, mz, tp, tz, ip_out, iz_out, static_cast<cudaStream_t>(stream));
}

lrbi_status lrbi_index_cost(const lrbi_layout *layout, const uint16_t *W, float theta, const uint32_t *ip,
                            const uint32_t *iz, lrbi_tile_cost *out, void *stream)
{
    if (!layout_ok(layout) || !W || !ip || !iz || !out) return LRBI_ERR_INVALID_ARG;
    if (!aligned16(W) || !aligned16(ip) || !aligned16(iz) || (reinterpret_cast<uintptr_t>(out) & 7u)) return LRBI_ERR_INVALID_ARG;
    if (device_timeout_seen()) return LRBI_ERR_TIMEOUT;
    return launch_index_cost(make_geo(*layout), W, theta, ip, iz, out, static_cast<cudaStream_t>(stream));
}

static bool ranks_ok(const lrbi_tile_ranks *r) { return r && r->ranks && r->ip_offset && r->iz_offset; }
static TileRanks to_ranks(const lrbi_tile_ranks *r)
{
    TileRanks t = {r->ranks, reinterpret_cast<const long long *>(r->ip_offset), reinterpret_cast<const long long *>(r->iz_offset)};
    return t;
}

lrbi_status lrbi_decode_mask_ranked(const lrbi_layout *layout, const lrbi_tile_ranks *ranks, const uint32_t *ip,
                                    const uint32_t *iz, uint32_t *mask_out, void *stream)
{
    if (!layout_ok(layout) || !ranks_ok(ranks) || !ip || !iz || !mask_out || !aligned16(mask_out)) return LRBI_ERR_INVALID_ARG;
    if (device_timeout_seen()) return LRBI_ERR_TIMEOUT;
    return launch_decode_ranked(make_geo(*layout), to_ranks(ranks), ip, iz, mask_out, static_cast<cudaStream_t>(stream));
}

lrbi_status lrbi_masked_gemm_ranked(const lrbi_layout *layout, const lrbi_tile_ranks *ranks, const uint16_t *W,
                                    const uint32_t *ip, const uint32_t *iz, const uint16_t *X, int32_t batch, void *Y,
                                    int32_t y_dtype, int32_t algo, void *stream)
{
    if (!layout_ok(layout) || !ranks_ok(ranks) || !W || !ip || !iz || !X || !Y || batch < 1) return LRBI_ERR_INVALID_ARG;
    if (y_dtype != LRBI_Y_BF16 && y_dtype != LRBI_Y_F32) return LRBI_ERR_INVALID_ARG;
    if (!aligned16(W) || !aligned16(X) || !aligned16(Y)) return LRBI_ERR_INVALID_ARG;
    if (device_timeout_seen()) return LRBI_ERR_TIMEOUT;
    const Geo g = make_geo(*layout);
    const TileRanks rk = to_ranks(ranks);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (algo == LRBI_ALGO_AUTO) algo = gemm_tc_supported(g, batch) ? LRBI_ALGO_TENSOR : LRBI_ALGO_GENERIC;
    switch (algo) {
    case LRBI_ALGO_GENERIC: return launch_gemm_ranked_generic(g, rk, W, ip, iz, X, batch, Y, y_dtype, s);
    case LRBI_ALGO_TENSOR: return launch_gemm_tc(g, W, ip, iz, X, batch, Y, y_dtype, s, 0, &rk);
    case LRBI_ALGO_TENSOR_PAIR: return launch_gemm_tc(g, W, ip, iz, X, batch, Y, y_dtype, s, 1, &rk);
    case LRBI_ALGO_TENSOR_PAIR2: return launch_gemm_tc(g, W, ip, iz, X, batch, Y, y_dtype, s, 2, &rk);
    case LRBI_ALGO_TENSOR_PAIR192: return launch_gemm_tc(g, W, ip, iz, X, batch, Y, y_dtype, s, 3, &rk);
    default: return LRBI_ERR_INVALID_ARG;
    }
}

lrbi_status lrbi_decode_mask_batch(int32_t n, const lrbi_layout *layouts, const uint32_t *const *ip,
                                   const uint32_t *const *iz, uint32_t *const *mask_out, void *stream)
{
    if (n < 1 || n > 4096 || !layouts || !ip || !iz || !mask_out) return LRBI_ERR_INVALID_ARG;
    Geo *g = new (std::nothrow) Geo[n];
    if (!g) return LRBI_ERR_CUDA;
    lrbi_status st = LRBI_OK;
    for (int l = 0; l < n && st == LRBI_OK; ++l) {
        if (!layout_ok(&layouts[l]) || !ip[l] || !iz[l] || !mask_out[l] || !aligned16(mask_out[l])) st = LRBI_ERR_INVALID_ARG;
        else g[l] = make_geo(layouts[l]);
    }
    if (st == LRBI_OK && device_timeout_seen()) st = LRBI_ERR_TIMEOUT;
    if (st == LRBI_OK) st = launch_decode_batch(n, g, ip, iz, mask_out, static_cast<cudaStream_t>(stream));
    delete[] g;
    return st;
}

lrbi_status lrbi_transpose_bf16(const uint16_t *src, int32_t rows, int32_t cols, uint16_t *dst, void *stream)
{
    if (!src || !dst || rows < 1 || cols < 1) return LRBI_ERR_INVALID_ARG;
    return launch_transpose_bf16(src, rows, cols, dst, static_cast<cudaStream_t>(stream));
}

// Geometry of the transposed layer: rows and columns, tile sides and grid swapped; tile (tr', tc') of it is tile
// (tc', tr') of the layer, i.e. number tc' * GC + tr' of the factor arrays.
static Geo transposed_geo(const Geo &g)
{
    Geo t = g;
    t.rows = g.cols; t.cols = g.rows; t.tm = g.tn; t.tn = g.tm; t.gr = g.gc; t.gc = g.gr;
    t.pitch = (t.cols + 31) / 32;
    t.ts_r = 1; t.ts_c = g.gc;
    return t;
}

lrbi_status lrbi_masked_gemm_dx(const lrbi_layout *layout, const uint16_t *Wt, const uint32_t *ip, const uint32_t *iz,
                                const uint16_t *dY, int32_t batch, void *dX, int32_t dx_dtype, int32_t algo, void *stream)
{
    if (!layout_ok(layout) || !Wt || !ip || !iz || !dY || !dX || batch < 1) return LRBI_ERR_INVALID_ARG;
    if (dx_dtype != LRBI_Y_BF16 && dx_dtype != LRBI_Y_F32) return LRBI_ERR_INVALID_ARG;
    if (!aligned16(Wt) || !aligned16(ip) || !aligned16(iz) || !aligned16(dY) || !aligned16(dX)) return LRBI_ERR_INVALID_ARG;
    if (device_timeout_seen()) return LRBI_ERR_TIMEOUT;
    const Geo t = transposed_geo(make_geo(*layout));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const TileRanks none = {nullptr, nullptr, nullptr};
    if (algo == LRBI_ALGO_AUTO) algo = gemm_tc_supported(t, batch) ? LRBI_ALGO_TENSOR : LRBI_ALGO_GENERIC;
    // the transposed layer's "Ip" is Iz (its rows are the layer's columns) and the other way round
    switch (algo) {
    case LRBI_ALGO_GENERIC: return launch_gemm_ranked_generic(t, none, Wt, iz, ip, dY, batch, dX, dx_dtype, s);
    case LRBI_ALGO_TENSOR: return launch_gemm_tc(t, Wt, iz, ip, dY, batch, dX, dx_dtype, s, 0);
    case LRBI_ALGO_TENSOR_PAIR: return launch_gemm_tc(t, Wt, iz, ip, dY, batch, dX, dx_dtype, s, 1);
    case LRBI_ALGO_TENSOR_PAIR2: return launch_gemm_tc(t, Wt, iz, ip, dY, batch, dX, dx_dtype, s, 2);
    case LRBI_ALGO_TENSOR_PAIR192: return launch_gemm_tc(t, Wt, iz, ip, dY, batch, dX, dx_dtype, s, 3);
    default: return LRBI_ERR_INVALID_ARG;
    }
}

static size_t round16(size_t b) { return (b + 15) & ~(size_t)15; }

size_t lrbi_masked_gemm_dw_workspace(const lrbi_layout *layout, int32_t batch)
{
    if (!layout_ok(layout) || batch < 1) return 0;
    // dY^T, X^T, and the two all-ones factors of the rank-one index the contraction runs with
    return round16((size_t)layout->rows * batch * 2) + round16((size_t)layout->cols * batch * 2) +
           round16((size_t)layout->cols * 4) + round16((size_t)batch * 4);
}

lrbi_status lrbi_masked_gemm_dw(const lrbi_layout *layout, const uint16_t *dY, const uint16_t *X, int32_t batch,
                                const uint32_t *ip, const uint32_t *iz, void *dW, int32_t dw_dtype, void *workspace,
                                size_t workspace_bytes, void *stream)
{
    if (!layout_ok(layout) || !dY || !X || !ip || !iz || !dW || batch < 1) return LRBI_ERR_INVALID_ARG;
    if (dw_dtype != LRBI_Y_BF16 && dw_dtype != LRBI_Y_F32) return LRBI_ERR_INVALID_ARG;
    if (!aligned16(dY) || !aligned16(X) || !aligned16(ip) || !aligned16(iz) || !aligned16(dW) || !aligned16(workspace)) return LRBI_ERR_INVALID_ARG;
    if (workspace && workspace_bytes < lrbi_masked_gemm_dw_workspace(layout, batch)) return LRBI_ERR_INVALID_ARG;
    if (device_timeout_seen()) return LRBI_ERR_TIMEOUT;
    const Geo g = make_geo(*layout);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the contraction as a forward product: "weights" X^T [cols][batch], "activations" dY^T [rows][batch], one tile of rank one
    lrbi_layout one = {layout->cols, batch, layout->cols, batch, 1};
    const Geo g1 = make_geo(one);
    // First choice: the persistent pair kernel on X and dY as they are (MN-major operands), nothing pruned inside the
    // contraction, the index (seen transposed: rows = layer columns) applied as the output tile is stored.
    if ((batch % 8) == 0 && gemm_tc_supported(g1, layout->rows)) {
        const lrbi_status st0 = launch_gemm_tc_dw(g1, transposed_geo(g), X, iz, ip, dY, layout->rows, dW, dw_dtype, s, true);
        if (st0 != LRBI_ERR_UNSUPPORTED) return st0;
    }
    if (!workspace || (batch % 8) != 0 || !gemm_tc_supported(g1, layout->rows))
        return launch_dw_generic(g, dY, X, batch, ip, iz, dW, dw_dtype, s);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    uint16_t *dYt = reinterpret_cast<uint16_t *>(ws);
    uint16_t *Xt = reinterpret_cast<uint16_t *>(ws + round16((size_t)layout->rows * batch * 2));
    uint32_t *ones_ip = reinterpret_cast<uint32_t *>(reinterpret_cast<uint8_t *>(Xt) + round16((size_t)layout->cols * batch * 2));
    uint32_t *ones_iz = reinterpret_cast<uint32_t *>(reinterpret_cast<uint8_t *>(ones_ip) + round16((size_t)layout->cols * 4));
    lrbi_status st = launch_transpose_bf16(dY, batch, layout->rows, dYt, s);
    if (st == LRBI_OK) st = launch_transpose_bf16(X, batch, layout->cols, Xt, s);
    if (st != LRBI_OK) return st;
    // (kept for layers whose row count is not a multiple of 8) the same kernel on transposed copies
    st = launch_gemm_tc_dw(g1, transposed_geo(g), Xt, iz, ip, dYt, layout->rows, dW, dw_dtype, s);
    if (st != LRBI_ERR_UNSUPPORTED) return st;
    // Otherwise: the forward kernel with an all-ones index of rank one, then the index applied to dW in place.
    st = launch_fill_words(ones_ip, (size_t)layout->cols, 1u, s);
    if (st == LRBI_OK) st = launch_fill_words(ones_iz, (size_t)batch, 1u, s);
    if (st == LRBI_OK) st = launch_gemm_tc(g1, Xt, ones_ip, ones_iz, dYt, layout->rows, dW, dw_dtype, s);
    if (st == LRBI_OK) st = launch_apply_index(g, ip, iz, dW, dw_dtype, s);
    return st;
}

size_t lrbi_nmf_workspace(const lrbi_layout *layout)
{
    return layout_ok(layout) ? nmf_workspace_bytes(make_geo(*layout)) : 0;
}

lrbi_status lrbi_nmf_update(const lrbi_layout *layout, const uint16_t *W, float *mp, float *mz, int32_t iterations, float eps,
                            void *workspace, size_t workspace_bytes, void *stream)
{
    if (!layout_ok(layout) || !W || !mp || !mz || !workspace || iterations < 0 || !(eps >= 0.f)) return LRBI_ERR_INVALID_ARG;
    if (!aligned16(workspace) || workspace_bytes < lrbi_nmf_workspace(layout)) return LRBI_ERR_INVALID_ARG;
    if (device_timeout_seen()) return LRBI_ERR_TIMEOUT;
    return launch_nmf(make_geo(*layout), W, mp, mz, iterations, eps, static_cast<float *>(workspace), static_cast<cudaStream_t>(stream));
}

uint64_t lrbi_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int32_t lrbi_device_status(int32_t clear)
{
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { note_cuda_error((int)e); return -1; }
    return read_status_word(clear != 0);
}

int32_t lrbi_last_device_error(void) { return lrbi_device_status(0); }

lrbi_status lrbi_selftest_bounded_wait(uint32_t limit_us, void *stream)
{
    return launch_bounded_wait_selftest(limit_us, static_cast<cudaStream_t>(stream));
}

lrbi_status lrbi_masked_gemm_plan(const lrbi_layout *layout, int32_t batch, int32_t algo, lrbi_gemm_plan *plan)
{
    if (!layout_ok(layout) || batch < 1 || !plan) return LRBI_ERR_INVALID_ARG;
    const Geo g = make_geo(*layout);
    if (algo == LRBI_ALGO_AUTO) algo = choose_gemm(g, batch);
    std::memset(plan, 0, sizeof *plan);
    plan->algo = algo;
    plan->k_splits = 1;
    switch (algo) {
    case LRBI_ALGO_GENERIC: return LRBI_OK;
    case LRBI_ALGO_GEMV: return gemv_supported(g, batch) ? LRBI_OK : LRBI_ERR_UNSUPPORTED;
    case LRBI_ALGO_STREAM: return stream_mma_supported(g, batch) ? LRBI_OK : LRBI_ERR_UNSUPPORTED;
    case LRBI_ALGO_TENSOR: return gemm_tc_plan(g, batch, 0, plan) ? LRBI_OK : LRBI_ERR_UNSUPPORTED;
    case LRBI_ALGO_TENSOR_PAIR: return gemm_tc_plan(g, batch, 1, plan) ? LRBI_OK : LRBI_ERR_UNSUPPORTED;
    case LRBI_ALGO_TENSOR_PAIR2: return gemm_tc_plan(g, batch, 2, plan) ? LRBI_OK : LRBI_ERR_UNSUPPORTED;
    case LRBI_ALGO_TENSOR_PAIR192: return gemm_tc_plan(g, batch, 3, plan) ? LRBI_OK : LRBI_ERR_UNSUPPORTED;
    default: return LRBI_ERR_INVALID_ARG;
    }
}

const char *lrbi_status_string(lrbi_status s)
{
    switch (s) {
    case LRBI_OK: return "ok";
    case LRBI_ERR_INVALID_ARG: return "invalid argument";
    case LRBI_ERR_UNSUPPORTED: return "unsupported shape or kernel choice";
    case LRBI_ERR_CUDA: return "CUDA call failed";
    case LRBI_ERR_TIMEOUT: return "device-side wait timed out";
    case LRBI_ERR_TOO_LARGE: return "needs more scratch than the fixed array holds";
    default: return "unknown status";
    }
}

int32_t lrbi_last_cuda_error(void) { return g_last_cuda_error.load(std::memory_order_relaxed); }

// ---------------------------------------------------------------------------------------------
// Host-buffer layer handle
// ---------------------------------------------------------------------------------------------
struct lrbi_layer {
    lrbi_layout layout;
    Geo g;
    int max_batch;
    uint16_t *W = nullptr;
    uint32_t *ip = nullptr, *iz = nullptr;
    uint16_t *X = nullptr;
    void *Y = nullptr;                 // max_batch x rows x 4 bytes
    cudaStream_t s_in = nullptr, s_run = nullptr, s_out = nullptr;
    static constexpr int kSlots = 64;
    cudaEvent_t ev_in[kSlots] = {}, ev_run[kSlots] = {};
};

static void layer_free(lrbi_layer *L)
{
    if (!L) return;
    cudaFree(L->W); cudaFree(L->ip); cudaFree(L->iz); cudaFree(L->X); cudaFree(L->Y);
    for (int i = 0; i < lrbi_layer::kSlots; ++i) {
        if (L->ev_in[i]) cudaEventDestroy(L->ev_in[i]);
        if (L->ev_run[i]) cudaEventDestroy(L->ev_run[i]);
    }
    if (L->s_in) cudaStreamDestroy(L->s_in);
    if (L->s_run) cudaStreamDestroy(L->s_run);
    if (L->s_out) cudaStreamDestroy(L->s_out);
    delete L;
}

lrbi_status lrbi_layer_create(const lrbi_layout *layout, const uint16_t *W_host, const uint32_t *ip_host,
                              const uint32_t *iz_host, int32_t max_batch, lrbi_layer **out)
{
    if (!layout_ok(layout) || !W_host || !ip_host || !iz_host || !out || max_batch < 1) return LRBI_ERR_INVALID_ARG;
    lrbi_layer *L = new (std::nothrow) lrbi_layer;
    if (!L) return LRBI_ERR_CUDA;
    L->layout = *layout;
    L->g = make_geo(*layout);
    L->max_batch = max_batch;
    const size_t wb = (size_t)layout->rows * layout->cols * 2;
    const size_t ipb = lrbi_packed_ip_words(layout) * 4, izb = lrbi_packed_iz_words(layout) * 4;
    cudaError_t e = cudaSuccess;
    auto step = [&](cudaError_t r) { if (e == cudaSuccess) e = r; };
    step(cudaMalloc(&L->W, wb));
    step(cudaMalloc(&L->ip, ipb));
    step(cudaMalloc(&L->iz, izb));
    step(cudaMalloc(&L->X, (size_t)max_batch * layout->cols * 2));
    step(cudaMalloc(&L->Y, (size_t)max_batch * layout->rows * 4));
    step(cudaStreamCreateWithFlags(&L->s_in, cudaStreamNonBlocking));
    step(cudaStreamCreateWithFlags(&L->s_run, cudaStreamNonBlocking));
    step(cudaStreamCreateWithFlags(&L->s_out, cudaStreamNonBlocking));
    for (int i = 0; i < lrbi_layer::kSlots; ++i) {
        step(cudaEventCreateWithFlags(&L->ev_in[i], cudaEventDisableTiming));
        step(cudaEventCreateWithFlags(&L->ev_run[i], cudaEventDisableTiming));
    }
    if (e == cudaSuccess) {
        step(cudaMemcpy(L->W, W_host, wb, cudaMemcpyHostToDevice));
        step(cudaMemcpy(L->ip, ip_host, ipb, cudaMemcpyHostToDevice));
        step(cudaMemcpy(L->iz, iz_host, izb, cudaMemcpyHostToDevice));
    }
    if (e != cudaSuccess) { note_cuda_error((int)e); layer_free(L); return LRBI_ERR_CUDA; }
    *out = L;
    return LRBI_OK;
}

lrbi_status lrbi_layer_forward_host(lrbi_layer *L, const uint16_t *X_host, int32_t batch, void *Y_host,
                                    int32_t y_dtype, int32_t algo)
{
    if (!L || !X_host || !Y_host || batch < 1 || batch > L->max_batch) return LRBI_ERR_INVALID_ARG;
    if (y_dtype != LRBI_Y_BF16 && y_dtype != LRBI_Y_F32) return LRBI_ERR_INVALID_ARG;
    const int cols = L->layout.cols, rows = L->layout.rows;
    const size_t ysz = y_dtype == LRBI_Y_F32 ? 4 : 2;
    // Chunks of the batch flow through three streams: copy in, compute, copy out.  With pinned
    // host buffers the three overlap; with pageable ones the copies serialise but stay correct.
    int chunk = batch;
    if (batch >= 1024) chunk = 512;
    int nchunks = (batch + chunk - 1) / chunk;
    if (nchunks > lrbi_layer::kSlots) { chunk = (batch + lrbi_layer::kSlots - 1) / lrbi_layer::kSlots; chunk = (chunk + 255) / 256 * 256; nchunks = (batch + chunk - 1) / chunk; }
    cudaError_t e = cudaSuccess;
    auto step = [&](cudaError_t r) { if (e == cudaSuccess) e = r; };
    lrbi_status st = LRBI_OK;
    for (int c = 0; c < nchunks && e == cudaSuccess && st == LRBI_OK; ++c) {
        const int b0 = c * chunk, nb = (batch - b0 < chunk) ? batch - b0 : chunk;
        uint16_t *xd = L->X + (size_t)b0 * cols;
        uint8_t *yd = static_cast<uint8_t *>(L->Y) + (size_t)b0 * rows * ysz;
        step(cudaMemcpyAsync(xd, X_host + (size_t)b0 * cols, (size_t)nb * cols * 2, cudaMemcpyHostToDevice, L->s_in));
        step(cudaEventRecord(L->ev_in[c], L->s_in));
        step(cudaStreamWaitEvent(L->s_run, L->ev_in[c], 0));
        if (e != cudaSuccess) break;
        st = lrbi_masked_gemm(&L->layout, L->W, L->ip, L->iz, xd, nb, yd, y_dtype, algo, L->s_run);
        if (st != LRBI_OK) break;
        step(cudaEventRecord(L->ev_run[c], L->s_run));
        step(cudaStreamWaitEvent(L->s_out, L->ev_run[c], 0));
        step(cudaMemcpyAsync(static_cast<uint8_t *>(Y_host) + (size_t)b0 * rows * ysz, yd, (size_t)nb * rows * ysz,
                             cudaMemcpyDeviceToHost, L->s_out));
    }
    cudaError_t e2 = cudaStreamSynchronize(L->s_in);
    cudaError_t e3 = cudaStreamSynchronize(L->s_run);
    cudaError_t e4 = cudaStreamSynchronize(L->s_out);
    if (e == cudaSuccess) e = e2 != cudaSuccess ? e2 : (e3 != cudaSuccess ? e3 : e4);
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    // every kernel of this call has finished: a bounded wait that gave up left its code in the status word,
    // and Y_host is then incomplete
    if (st == LRBI_OK && read_status_word(false) != 0) return LRBI_ERR_TIMEOUT;
    return st;
}

lrbi_status lrbi_layer_destroy(lrbi_layer *L)
{
    if (!L) return LRBI_ERR_INVALID_ARG;
    cudaDeviceSynchronize();
    layer_free(L);
    return LRBI_OK;
}

}  // extern "C"
