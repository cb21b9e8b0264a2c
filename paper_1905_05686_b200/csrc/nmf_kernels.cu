// NMF of the magnitude matrix M = |W| (Section 2.1, Eq. 4; first steps of Algorithm 1), every tile on its own
// (Section 3.1), by multiplicative updates for the Frobenius objective ||M - Mp Mz||^2:
//     Mz <- Mz * (Mp^T M) / (Mp^T Mp Mz + eps)        then        Mp <- Mp * (M Mz^T) / (Mp Mz Mz^T + eps).
// The paper leaves the solver to "an NMF library"; this is the update rule of the NMF reference it cites.
// All arithmetic is fp32 on CUDA cores (the factors are real-valued and the iteration is sensitive to rounding; the
// two large products per iteration are 4 k tm tn flops per tile, small against the layer's own GEMMs).
//   nmf_gemm<0>   N1 = Mp^T |W|   (k x tn per tile)         nmf_gemm<1>   N2 = |W| Mz^T   (tm x k per tile)
//   nmf_gram      G  = Mp^T Mp  or  Mz Mz^T   (k x k per tile)
//   nmf_update_z / nmf_update_p   the element-wise update with the k-term denominator
#include "lrbi_common.cuh"

namespace lrbi {

constexpr int NG_T = 64;               // output tile of the product kernels
constexpr int NG_K = 16;               // reduction step

__device__ __forceinline__ float abs_bf16(uint16_t h) { return __uint_as_float(((uint32_t)h << 16) & 0x7FFF0000u); }

// MODE 0: C[l][j] = sum_i P[i][l] |W[i][j]|   (rows of C: k, columns: tn, reduction: tm)
// MODE 1: C[i][l] = sum_j |W[i][j]| Z[l][j]   (rows of C: tm, columns: k, reduction: tn)
// grid = (column tiles, row tiles, layer tiles); 256 threads, 4 x 4 outputs each.
template <int MODE>
__global__ void __launch_bounds__(256)
nmf_gemm_kernel(Geo g, const uint16_t *__restrict__ W, const float *__restrict__ F, float *__restrict__ C)
{
    __shared__ float As[NG_K][NG_T + 4], Bs[NG_K][NG_T + 4];
    const int tile = blockIdx.z, tr = tile / g.gc, tc = tile - tr * g.gc;
    const int k = g.k;
    const int CM = MODE == 0 ? k : g.tm, CN = MODE == 0 ? g.tn : k, KR = MODE == 0 ? g.tm : g.tn;
    const int m0 = blockIdx.y * NG_T, n0 = blockIdx.x * NG_T;
    const uint16_t *Wt = W + (size_t)tr * g.tm * g.cols + (size_t)tc * g.tn;
    const int wrows = min(g.tm, g.rows - tr * g.tm), wcols = min(g.tn, g.cols - tc * g.tn);   // part of the tile inside the matrix
    const float *Ft = F + (size_t)tile * (MODE == 0 ? (size_t)g.tm * k : (size_t)k * g.tn);
    float *Ct = C + (size_t)tile * CM * CN;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4] = {};
    for (int r0 = 0; r0 < KR; r0 += NG_K) {
        for (int e = threadIdx.x; e < NG_K * NG_T; e += 256) {
            if (MODE == 0) {
                const int kk = e / NG_T, m = e - kk * NG_T;             // consecutive threads: consecutive l (contiguous in P)
                const int i = r0 + kk, l = m0 + m;
                As[kk][m] = (i < g.tm && l < k) ? Ft[(size_t)i * k + l] : 0.f;
                const int j = n0 + m;                                    // and consecutive j (contiguous in W)
                Bs[kk][m] = (i < wrows && j < wcols) ? abs_bf16(Wt[(size_t)i * g.cols + j]) : 0.f;
            } else {
                const int m = e / NG_K, kk = e - m * NG_K;              // consecutive threads: consecutive j (contiguous in W and Z)
                const int j = r0 + kk;
                const int i = m0 + m;
                As[kk][m] = (i < wrows && j < wcols) ? abs_bf16(Wt[(size_t)i * g.cols + j]) : 0.f;
                const int l = n0 + m;
                Bs[kk][m] = (l < k && j < g.tn) ? Ft[(size_t)l * g.tn + j] : 0.f;
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < NG_K; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) { a[u] = As[kk][ty * 4 + u]; b[u] = Bs[kk][tx * 4 + u]; }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(a[u], b[v], acc[u][v]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int m = m0 + ty * 4 + u, n = n0 + tx * 4 + v;
            if (m < CM && n < CN) Ct[(size_t)m * CN + n] = acc[u][v];
        }
}

// G[a][b] = sum_r F(r, a) F(r, b): ZMODE 0: F = Mp [tm][k] (r = row), ZMODE 1: F = Mz [k][tn] (r = column).
// grid = (k*k / 256, layer tiles, slices of the reduction): a block sums its slice of r and adds it to G (zeroed
// before the launch) with one atomic per entry; a lone thread per entry over the whole reduction was measured at
// 200-280 us per launch on the AlexNet layer, as much as the large products.
constexpr int NMF_GRAM_SLICE = 32;
template <int ZMODE>
__global__ void __launch_bounds__(256)
nmf_gram_kernel(Geo g, const float *__restrict__ F, float *__restrict__ G)
{
    const int tile = blockIdx.y, k = g.k;
    const int e = blockIdx.x * 256 + threadIdx.x;
    if (e >= k * k) return;
    const int a = e / k, b = e - a * k;
    const float *Ft = F + (size_t)tile * (ZMODE == 0 ? (size_t)g.tm * k : (size_t)k * g.tn);
    const int R = ZMODE == 0 ? g.tm : g.tn;
    const int r0 = blockIdx.z * NMF_GRAM_SLICE, r1 = min(R, r0 + NMF_GRAM_SLICE);
    float s = 0.f;
    for (int r = r0; r < r1; ++r)
        s = ZMODE == 0 ? fmaf(Ft[(size_t)r * k + a], Ft[(size_t)r * k + b], s) : fmaf(Ft[(size_t)a * g.tn + r], Ft[(size_t)b * g.tn + r], s);
    atomicAdd(G + (size_t)tile * k * k + e, s);
}

constexpr int NMF_MAX_RANK = 256;

// Mz[l][j] *= N1[l][j] / (sum_m G1[l][m] Mz[m][j] + eps): a thread owns column j (the old column is read before any write).
__global__ void __launch_bounds__(128)
nmf_update_z_kernel(Geo g, const float *__restrict__ N1, const float *__restrict__ G1, float *__restrict__ Z, float eps)
{
    const int tile = blockIdx.y, k = g.k, j = blockIdx.x * 128 + threadIdx.x;
    if (j >= g.tn) return;
    float *Zt = Z + (size_t)tile * k * g.tn;
    const float *Nt = N1 + (size_t)tile * k * g.tn, *Gt = G1 + (size_t)tile * k * k;
    float z[NMF_MAX_RANK];
    for (int m = 0; m < k; ++m) z[m] = Zt[(size_t)m * g.tn + j];
    for (int l = 0; l < k; ++l) {
        float den = 0.f;
        for (int m = 0; m < k; ++m) den = fmaf(__ldg(Gt + l * k + m), z[m], den);
        Zt[(size_t)l * g.tn + j] = z[l] * Nt[(size_t)l * g.tn + j] / (den + eps);
    }
}

// Mp[i][l] *= N2[i][l] / (sum_m Mp[i][m] G2[m][l] + eps): a thread owns row i.
__global__ void __launch_bounds__(128)
nmf_update_p_kernel(Geo g, const float *__restrict__ N2, const float *__restrict__ G2, float *__restrict__ P, float eps)
{
    const int tile = blockIdx.y, k = g.k, i = blockIdx.x * 128 + threadIdx.x;
    if (i >= g.tm) return;
    float *Pt = P + ((size_t)tile * g.tm + i) * k;
    const float *Nt = N2 + ((size_t)tile * g.tm + i) * k, *Gt = G2 + (size_t)tile * k * k;
    float p[NMF_MAX_RANK];
    for (int m = 0; m < k; ++m) p[m] = Pt[m];
    for (int l = 0; l < k; ++l) {
        float den = 0.f;
        for (int m = 0; m < k; ++m) den = fmaf(p[m], __ldg(Gt + m * k + l), den);
        Pt[l] = p[l] * Nt[l] / (den + eps);
    }
}

size_t nmf_workspace_bytes(const Geo &g)
{
    const size_t tiles = (size_t)g.gr * g.gc;
    return tiles * ((size_t)g.k * (g.tm > g.tn ? g.tm : g.tn) + (size_t)g.k * g.k) * sizeof(float);
}

lrbi_status launch_nmf(const Geo &g, const uint16_t *W, float *mp, float *mz, int iterations, float eps, float *ws, cudaStream_t s)
{
    if (g.k > NMF_MAX_RANK) return LRBI_ERR_UNSUPPORTED;
    const long long tiles = (long long)g.gr * g.gc;
    if (tiles > 65535) return LRBI_ERR_UNSUPPORTED;
    float *N = ws, *G = ws + (size_t)tiles * g.k * (g.tm > g.tn ? g.tm : g.tn);
    const unsigned kt = (unsigned)((g.k + NG_T - 1) / NG_T), gk2 = (unsigned)((g.k * g.k + 255) / 256);
    for (int it = 0; it < iterations; ++it) {
        nmf_gemm_kernel<0><<<dim3((unsigned)((g.tn + NG_T - 1) / NG_T), kt, (unsigned)tiles), 256, 0, s>>>(g, W, mp, N);
        cudaMemsetAsync(G, 0, (size_t)tiles * g.k * g.k * sizeof(float), s);
        nmf_gram_kernel<0><<<dim3(gk2, (unsigned)tiles, (unsigned)((g.tm + NMF_GRAM_SLICE - 1) / NMF_GRAM_SLICE)), 256, 0, s>>>(g, mp, G);
        nmf_update_z_kernel<<<dim3((unsigned)((g.tn + 127) / 128), (unsigned)tiles), 128, 0, s>>>(g, N, G, mz, eps);
        nmf_gemm_kernel<1><<<dim3(kt, (unsigned)((g.tm + NG_T - 1) / NG_T), (unsigned)tiles), 256, 0, s>>>(g, W, mz, N);
        cudaMemsetAsync(G, 0, (size_t)tiles * g.k * g.k * sizeof(float), s);
        nmf_gram_kernel<1><<<dim3(gk2, (unsigned)tiles, (unsigned)((g.tn + NMF_GRAM_SLICE - 1) / NMF_GRAM_SLICE)), 256, 0, s>>>(g, mz, G);
        nmf_update_p_kernel<<<dim3((unsigned)((g.tm + 127) / 128), (unsigned)tiles), 128, 0, s>>>(g, N, G, mp, eps);
        count_launch(6);
    }
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

}  // namespace lrbi
