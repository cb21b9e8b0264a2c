// NMF of the magnitude matrix M = |W| (Section 2.1, Eq. 4; first steps of Algorithm 1), every tile on its own
// (Section 3.1), by multiplicative updates for the Frobenius objective ||M - Mp Mz||^2:
//     Mz <- Mz * (Mp^T M) / (Mp^T Mp Mz + eps)        then        Mp <- Mp * (M Mz^T) / (Mp Mz Mz^T + eps).
// The paper leaves the solver to "an NMF library"; this is the update rule of the NMF reference it cites.
// All arithmetic is fp32 on CUDA cores (the factors are real-valued and the iteration is sensitive to rounding; the
// two large products per iteration are 4 k tm tn flops per tile, small against the layer's own GEMMs).
//   nmf_prod_z    N1 = Mp^T |W|   (k x tn per tile)         nmf_prod_p    N2 = |W| Mz^T   (tm x k per tile)
//                 (a thread owns one output column / row and 32 rank values; |W| is read once per 32 rank values)
//   nmf_gram      G  = Mp^T Mp  or  Mz Mz^T   (k x k per tile)
//   nmf_update_z / nmf_update_p   the element-wise update with the k-term denominator
#include <mutex>

#include "lrbi_common.cuh"

namespace lrbi {

constexpr int NP_THREADS = 128;        // outputs of a product block: one column (prod_z) or row (prod_p) per thread.x
constexpr int NP_GROUPS = 4;           // threads per output (thread.y): each takes a quarter of every slab of the reduction
constexpr int NP_KC = 32;              // rank values per block: a thread keeps that many running sums in registers
constexpr int NP_SLAB0 = 32;           // rows of the reduction staged per step, prod_z
constexpr int NP_SLAB1 = 64;           // columns of the reduction staged per step, prod_p

__device__ __forceinline__ float abs_bf16(uint16_t h) { return __uint_as_float(((uint32_t)h << 16) & 0x7FFF0000u); }

// N1[l][j] = sum_i P[i][l] |W[i][j]|   (k x tn per tile; the reduction runs over the tile's rows).
// grid = (ceil(tn / 128), layer tiles, ceil(k / 32)).  A thread owns column j and 32 values of l: |W[i][j]| comes
// straight from device memory (consecutive threads, consecutive columns), the 32 values P[i][l] of a row are read
// from shared memory by every thread alike (broadcast), 32 multiply-adds per weight.  Four threads share a column
// (each takes a quarter of a slab's rows) and add their sums up through shared memory at the end.
__device__ __forceinline__ void nmf_fold_groups(float (&acc)[NP_KC], float *red, int t, int q)
{
    for (int qq = 1; qq < NP_GROUPS; ++qq) {
        __syncthreads();
        if (q == qq) {
#pragma unroll
            for (int c = 0; c < NP_KC; ++c) red[c * NP_THREADS + t] = acc[c];
        }
        __syncthreads();
        if (q == 0) {
#pragma unroll
            for (int c = 0; c < NP_KC; ++c) acc[c] += red[c * NP_THREADS + t];
        }
    }
}

__global__ void __launch_bounds__(NP_THREADS * NP_GROUPS, 2)
nmf_prod_z_kernel(Geo g, const uint16_t *__restrict__ W, const float *__restrict__ P, float *__restrict__ N1)
{
    __shared__ __align__(16) float Ps[NP_SLAB0][NP_KC];
    __shared__ float red[NP_KC * NP_THREADS];
    const int tile = blockIdx.y, tr = tile / g.gc, tc = tile - tr * g.gc, k = g.k, t = threadIdx.x, q = threadIdx.y;
    const int tid = q * NP_THREADS + t;
    constexpr int RQ = NP_SLAB0 / NP_GROUPS;            // rows of a slab per thread
    const int j = blockIdx.x * NP_THREADS + t, l0 = blockIdx.z * NP_KC, kc = min(NP_KC, k - l0);
    const int wrows = min(g.tm, g.rows - tr * g.tm), wcols = min(g.tn, g.cols - tc * g.tn);   // part of the tile inside the matrix
    const uint16_t *Wt = W + (size_t)tr * g.tm * g.cols + (size_t)tc * g.tn;
    const float *Pt = P + (size_t)tile * g.tm * k;
    float acc[NP_KC];
#pragma unroll
    for (int c = 0; c < NP_KC; ++c) acc[c] = 0.f;
    for (int i0 = 0; i0 < wrows; i0 += NP_SLAB0) {      // rows outside the matrix hold |W| = 0: nothing to add
        uint16_t wv[RQ];
#pragma unroll
        for (int r = 0; r < RQ; ++r) wv[r] = (i0 + q * RQ + r < wrows && j < wcols) ? Wt[(size_t)(i0 + q * RQ + r) * g.cols + j] : (uint16_t)0;
#pragma unroll
        for (int u = 0; u < NP_SLAB0 * NP_KC / (NP_THREADS * NP_GROUPS); ++u) {
            const int e = tid + NP_THREADS * NP_GROUPS * u, r = e / NP_KC, c = e - r * NP_KC;
            Ps[r][c] = (i0 + r < g.tm && c < kc) ? Pt[(size_t)(i0 + r) * k + l0 + c] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int rr = 0; rr < RQ; ++rr) {
            const int r = q * RQ + rr;
            const float w = abs_bf16(wv[rr]);
#pragma unroll
            for (int c4 = 0; c4 < NP_KC / 4; ++c4) {
                const float4 p = *reinterpret_cast<const float4 *>(&Ps[r][c4 * 4]);
                acc[c4 * 4 + 0] = fmaf(p.x, w, acc[c4 * 4 + 0]);
                acc[c4 * 4 + 1] = fmaf(p.y, w, acc[c4 * 4 + 1]);
                acc[c4 * 4 + 2] = fmaf(p.z, w, acc[c4 * 4 + 2]);
                acc[c4 * 4 + 3] = fmaf(p.w, w, acc[c4 * 4 + 3]);
            }
        }
        __syncthreads();
    }
    nmf_fold_groups(acc, red, t, q);
    if (q == 0 && j < g.tn) {
        float *Nt = N1 + (size_t)tile * k * g.tn;
#pragma unroll
        for (int c = 0; c < NP_KC; ++c)
            if (c < kc) Nt[(size_t)(l0 + c) * g.tn + j] = acc[c];
    }
}

// The same product for aligned layers (cols % 8 == 0, tn % 8 == 0, k % 4 == 0): the slabs of |W| (32 rows x 128
// columns) and of Mp (32 rows x 32 rank values) travel through a ring of four shared-memory buffers filled by
// cp.async three slabs ahead, so nobody waits on device memory inside the loop.
constexpr int NP_RING = 4;
constexpr int NP_RING_BYTES = NP_SLAB0 * NP_THREADS * 2 + NP_SLAB0 * NP_KC * 4;      // 8 KB of W + 4 KB of Mp per buffer
__device__ __forceinline__ void nmf_cp_async_16(void *dst_smem, const void *src, int valid)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src), "r"(valid) : "memory");
}
__global__ void __launch_bounds__(NP_THREADS * NP_GROUPS, 2)
nmf_prod_z_ring_kernel(Geo g, const uint16_t *__restrict__ W, const float *__restrict__ P, float *__restrict__ N1)
{
    extern __shared__ __align__(16) uint8_t nmf_ring[];
    const int tile = blockIdx.y, tr = tile / g.gc, tc = tile - tr * g.gc, k = g.k, t = threadIdx.x, q = threadIdx.y;
    const int tid = q * NP_THREADS + t;
    constexpr int RQ = NP_SLAB0 / NP_GROUPS;
    const int l0 = blockIdx.z * NP_KC, kc = min(NP_KC, k - l0);
    // a thread owns 4 columns x 8 rank values (lane = group of 4 columns, warp = group of 8 rank values): per row of
    // the slab it reads 8 bytes of |W| and 32 bytes of Mp for its 32 multiply-adds; with 1 column x 32 rank values it
    // read 2 + 128 bytes, and the delivery of shared memory to the registers was the limit
    const int cg = t & 31, lg = t >> 5;
    const int wrows = min(g.tm, g.rows - tr * g.tm), wcols = min(g.tn, g.cols - tc * g.tn);
    const uint16_t *Wt = W + (size_t)tr * g.tm * g.cols + (size_t)tc * g.tn;
    const float *Pt = P + (size_t)tile * g.tm * k;
    const int nslab = (wrows + NP_SLAB0 - 1) / NP_SLAB0;
    auto issue = [&](int sl) {                           // (a group is committed even when it is empty: the count stays uniform)
        if (sl < nslab) {
            uint8_t *buf = nmf_ring + (sl % NP_RING) * NP_RING_BYTES;
            const int i0 = sl * NP_SLAB0;
            {
                const int r = tid >> 4, c8 = (tid & 15) * 8, jj = blockIdx.x * NP_THREADS + c8;   // 8 columns: all inside the matrix or none
                const bool in = i0 + r < wrows && jj < wcols;
                nmf_cp_async_16(reinterpret_cast<uint16_t *>(buf) + r * NP_THREADS + c8, in ? Wt + (size_t)(i0 + r) * g.cols + jj : Wt, in ? 16 : 0);
            }
            if (tid < NP_SLAB0 * NP_KC / 4) {
                const int r = tid >> 3, c4 = (tid & 7) * 4;
                const bool in = i0 + r < g.tm && c4 < kc;                                         // k % 4 == 0: four values or none
                nmf_cp_async_16(reinterpret_cast<float *>(buf + NP_SLAB0 * NP_THREADS * 2) + r * NP_KC + c4, in ? Pt + (size_t)(i0 + r) * k + l0 + c4 : Pt, in ? 16 : 0);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    float acc[NP_KC];
#pragma unroll
    for (int c = 0; c < NP_KC; ++c) acc[c] = 0.f;
    for (int sl = 0; sl < NP_RING - 1; ++sl) issue(sl);
    for (int sl = 0; sl < nslab; ++sl) {
        asm volatile("cp.async.wait_group %0;" ::"n"(NP_RING - 2) : "memory");   // this thread's part of slab sl has landed
        __syncthreads();                                 // ... everybody's; and everybody is done with the buffer refilled next
        issue(sl + NP_RING - 1);
        const uint8_t *buf = nmf_ring + (sl % NP_RING) * NP_RING_BYTES;
        const uint16_t *Ws = reinterpret_cast<const uint16_t *>(buf);
        const float *Ps = reinterpret_cast<const float *>(buf + NP_SLAB0 * NP_THREADS * 2);
#pragma unroll
        for (int rr = 0; rr < RQ; ++rr) {
            const int r = q * RQ + rr;
            const uint2 wv = *reinterpret_cast<const uint2 *>(Ws + r * NP_THREADS + cg * 4);
            const float w[4] = {abs_bf16((uint16_t)wv.x), abs_bf16((uint16_t)(wv.x >> 16)), abs_bf16((uint16_t)wv.y), abs_bf16((uint16_t)(wv.y >> 16))};
            const float4 pa = *reinterpret_cast<const float4 *>(Ps + r * NP_KC + lg * 8);
            const float4 pb = *reinterpret_cast<const float4 *>(Ps + r * NP_KC + lg * 8 + 4);
            const float pv[8] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
#pragma unroll
            for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                for (int ll = 0; ll < 8; ++ll) acc[cc * 8 + ll] = fmaf(pv[ll], w[cc], acc[cc * 8 + ll]);
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    nmf_fold_groups(acc, reinterpret_cast<float *>(nmf_ring), t, q);    // (its first barrier comes before the ring is reused)
    const int j4 = blockIdx.x * NP_THREADS + cg * 4;    // tn % 8 == 0: the four columns are inside the tile or none is
    if (q == 0 && j4 < g.tn) {
        float *Nt = N1 + (size_t)tile * k * g.tn;
#pragma unroll
        for (int ll = 0; ll < 8; ++ll) {
            const int l = l0 + lg * 8 + ll;
            if (l < k) *reinterpret_cast<float4 *>(Nt + (size_t)l * g.tn + j4) = make_float4(acc[ll], acc[8 + ll], acc[16 + ll], acc[24 + ll]);
        }
    }
}

// N2[i][l] = sum_j |W[i][j]| Z[l][j]   (tm x k per tile; the reduction runs over the tile's columns).
// grid = (ceil(tm / 128), layer tiles, ceil(k / 32)).  A thread owns row i and 32 values of l.  A slab of 128 rows x 64
// columns of W goes through shared memory (read along the rows, used along the columns), the slab of Z is stored
// [column][l] so that a thread reads the 32 values of one column as eight 16-byte broadcasts.
__global__ void __launch_bounds__(NP_THREADS * NP_GROUPS, 2)
nmf_prod_p_kernel(Geo g, const uint16_t *__restrict__ W, const float *__restrict__ Z, float *__restrict__ N2)
{
    constexpr int WP = NP_SLAB1 + 2;                     // 33 words per row: a column is read without bank conflicts
    constexpr int ZP = NP_KC + 4;                        // keeps rows 16-byte aligned
    __shared__ uint16_t Ws[NP_THREADS * WP];
    __shared__ __align__(16) float Zs[NP_SLAB1 * ZP];
    __shared__ float red[NP_KC * NP_THREADS];
    const int tile = blockIdx.y, tr = tile / g.gc, tc = tile - tr * g.gc, k = g.k, t = threadIdx.x, q = threadIdx.y;
    const int tid = q * NP_THREADS + t;
    constexpr int JQ = NP_SLAB1 / NP_GROUPS;            // columns of a slab per thread
    const int ib = blockIdx.x * NP_THREADS, l0 = blockIdx.z * NP_KC, kc = min(NP_KC, k - l0);
    const int wrows = min(g.tm, g.rows - tr * g.tm), wcols = min(g.tn, g.cols - tc * g.tn);
    const uint16_t *Wt = W + (size_t)tr * g.tm * g.cols + (size_t)tc * g.tn;
    const float *Zt = Z + (size_t)tile * k * g.tn;
    float acc[NP_KC];
#pragma unroll
    for (int c = 0; c < NP_KC; ++c) acc[c] = 0.f;
    for (int j0 = 0; j0 < wcols; j0 += NP_SLAB1) {      // columns outside the matrix hold |W| = 0
        // (all requests of a thread go out before the first value is used: the slab costs one trip to memory, not sixteen)
        constexpr int NW = NP_THREADS * NP_SLAB1 / (NP_THREADS * NP_GROUPS), NZ = NP_KC * NP_SLAB1 / (NP_THREADS * NP_GROUPS);
        uint16_t wl[NW];
        float zl[NZ];
#pragma unroll
        for (int u = 0; u < NW; ++u) {
            const int e = tid + NP_THREADS * NP_GROUPS * u, r = e / NP_SLAB1, jj = e - r * NP_SLAB1;
            wl[u] = (ib + r < wrows && j0 + jj < wcols) ? Wt[(size_t)(ib + r) * g.cols + j0 + jj] : (uint16_t)0;
        }
#pragma unroll
        for (int u = 0; u < NZ; ++u) {
            const int e = tid + NP_THREADS * NP_GROUPS * u, c = e / NP_SLAB1, jj = e - c * NP_SLAB1;
            zl[u] = (c < kc && j0 + jj < g.tn) ? Zt[(size_t)(l0 + c) * g.tn + j0 + jj] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < NW; ++u) {
            const int e = tid + NP_THREADS * NP_GROUPS * u, r = e / NP_SLAB1, jj = e - r * NP_SLAB1;
            Ws[r * WP + jj] = wl[u];
        }
#pragma unroll
        for (int u = 0; u < NZ; ++u) {
            const int e = tid + NP_THREADS * NP_GROUPS * u, c = e / NP_SLAB1, jj = e - c * NP_SLAB1;
            Zs[jj * ZP + c] = zl[u];
        }
        __syncthreads();
#pragma unroll 8
        for (int jj = q * JQ; jj < (q + 1) * JQ; ++jj) {
            const float w = abs_bf16(Ws[t * WP + jj]);
#pragma unroll
            for (int c4 = 0; c4 < NP_KC / 4; ++c4) {
                const float4 z = *reinterpret_cast<const float4 *>(&Zs[jj * ZP + c4 * 4]);
                acc[c4 * 4 + 0] = fmaf(w, z.x, acc[c4 * 4 + 0]);
                acc[c4 * 4 + 1] = fmaf(w, z.y, acc[c4 * 4 + 1]);
                acc[c4 * 4 + 2] = fmaf(w, z.z, acc[c4 * 4 + 2]);
                acc[c4 * 4 + 3] = fmaf(w, z.w, acc[c4 * 4 + 3]);
            }
        }
        __syncthreads();
    }
    nmf_fold_groups(acc, red, t, q);
    const int i = ib + t;
    if (q == 0 && i < g.tm) {
        float *Nt = N2 + ((size_t)tile * g.tm + i) * k + l0;
#pragma unroll
        for (int c = 0; c < NP_KC; ++c)
            if (c < kc) Nt[c] = acc[c];
    }
}

// The ring version of the second product (same conditions as nmf_prod_z_ring_kernel): slabs of 128 rows x 64 columns of
// |W| (rows 144 bytes apart) and of 64 columns x 32 rank values of Mz (stored [column][rank value], filled by 4-byte
// cp.async), three buffers.  A thread owns rows rg, rg + 32, rg + 64, rg + 96 and 8 rank values.
constexpr int NP_RING1 = 3;
constexpr int NP_WPITCH = NP_SLAB1 + 8;                  // bf16 per staged row of W: 144 bytes
constexpr int NP_ZPITCH = NP_KC + 4;                     // floats per staged column of Mz: the 4-byte copies of 32 columns spread over 8 banks, not 1
constexpr int NP_RING1_BYTES = NP_THREADS * NP_WPITCH * 2 + NP_SLAB1 * NP_ZPITCH * 4;
__global__ void __launch_bounds__(NP_THREADS * NP_GROUPS, 2)
nmf_prod_p_ring_kernel(Geo g, const uint16_t *__restrict__ W, const float *__restrict__ Z, float *__restrict__ N2)
{
    extern __shared__ __align__(16) uint8_t nmf_ring[];
    const int tile = blockIdx.y, tr = tile / g.gc, tc = tile - tr * g.gc, k = g.k, t = threadIdx.x, q = threadIdx.y;
    const int tid = q * NP_THREADS + t;
    const int ib = blockIdx.x * NP_THREADS, l0 = blockIdx.z * NP_KC, kc = min(NP_KC, k - l0);
    const int rg = t & 31, lg = t >> 5;
    const int wrows = min(g.tm, g.rows - tr * g.tm), wcols = min(g.tn, g.cols - tc * g.tn);
    const uint16_t *Wt = W + (size_t)tr * g.tm * g.cols + (size_t)tc * g.tn;
    const float *Zt = Z + (size_t)tile * k * g.tn;
    const int nslab = (wcols + NP_SLAB1 - 1) / NP_SLAB1;
    auto issue = [&](int sl) {
        if (sl < nslab) {
            uint8_t *buf = nmf_ring + (sl % NP_RING1) * NP_RING1_BYTES;
            const int j0 = sl * NP_SLAB1;
#pragma unroll
            for (int u = 0; u < 2; ++u) {                // 128 rows x 8 pieces of 8 columns
                const int e = tid + NP_THREADS * NP_GROUPS * u, r = e >> 3, c8 = (e & 7) * 8;
                const bool in = ib + r < wrows && j0 + c8 < wcols;
                nmf_cp_async_16(reinterpret_cast<uint16_t *>(buf) + r * NP_WPITCH + c8, in ? Wt + (size_t)(ib + r) * g.cols + j0 + c8 : Wt, in ? 16 : 0);
            }
            float *Zs = reinterpret_cast<float *>(buf + NP_THREADS * NP_WPITCH * 2);
#pragma unroll
            for (int u = 0; u < NP_KC * NP_SLAB1 / (NP_THREADS * NP_GROUPS); ++u) {
                const int e = tid + NP_THREADS * NP_GROUPS * u, c = e / NP_SLAB1, jj = e - c * NP_SLAB1;
                const bool in = c < kc && j0 + jj < g.tn;
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(Zs + jj * NP_ZPITCH + c)),
                             "l"(in ? Zt + (size_t)(l0 + c) * g.tn + j0 + jj : Zt), "r"(in ? 4 : 0) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    float acc[NP_KC];
#pragma unroll
    for (int c = 0; c < NP_KC; ++c) acc[c] = 0.f;
    for (int sl = 0; sl < NP_RING1 - 1; ++sl) issue(sl);
    constexpr int JQ = NP_SLAB1 / NP_GROUPS;            // columns of a slab per thread: 16, two pieces of 8
    for (int sl = 0; sl < nslab; ++sl) {
        asm volatile("cp.async.wait_group %0;" ::"n"(NP_RING1 - 2) : "memory");
        __syncthreads();
        issue(sl + NP_RING1 - 1);
        const uint8_t *buf = nmf_ring + (sl % NP_RING1) * NP_RING1_BYTES;
        const uint16_t *Ws = reinterpret_cast<const uint16_t *>(buf);
        const float *Zs = reinterpret_cast<const float *>(buf + NP_THREADS * NP_WPITCH * 2);
#pragma unroll
        for (int pc = 0; pc < JQ / 8; ++pc) {
            const int jb = q * JQ + pc * 8;
            uint4 wv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) wv[u] = *reinterpret_cast<const uint4 *>(Ws + (rg + 32 * u) * NP_WPITCH + jb);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float4 za = *reinterpret_cast<const float4 *>(Zs + (jb + e) * NP_ZPITCH + lg * 8);
                const float4 zb = *reinterpret_cast<const float4 *>(Zs + (jb + e) * NP_ZPITCH + lg * 8 + 4);
                const float zv[8] = {za.x, za.y, za.z, za.w, zb.x, zb.y, zb.z, zb.w};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t word = e < 2 ? wv[u].x : e < 4 ? wv[u].y : e < 6 ? wv[u].z : wv[u].w;
                    const float w = abs_bf16((uint16_t)((e & 1) ? word >> 16 : word));
#pragma unroll
                    for (int ll = 0; ll < 8; ++ll) acc[u * 8 + ll] = fmaf(w, zv[ll], acc[u * 8 + ll]);
                }
            }
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    nmf_fold_groups(acc, reinterpret_cast<float *>(nmf_ring), t, q);
    if (q == 0) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = ib + rg + 32 * u;
            if (i < g.tm) {
                float *Nt = N2 + ((size_t)tile * g.tm + i) * k + l0 + lg * 8;      // k % 4 == 0: 16-byte aligned
                if (lg * 8 < kc) *reinterpret_cast<float4 *>(Nt) = make_float4(acc[u * 8], acc[u * 8 + 1], acc[u * 8 + 2], acc[u * 8 + 3]);
                if (lg * 8 + 4 < kc) *reinterpret_cast<float4 *>(Nt + 4) = make_float4(acc[u * 8 + 4], acc[u * 8 + 5], acc[u * 8 + 6], acc[u * 8 + 7]);
            }
        }
    }
}

// G[a][b] = sum_r F(r, a) F(r, b): ZMODE 0: F = Mp [tm][k] (r = row), ZMODE 1: F = Mz [k][tn] (r = column).
// grid = (blocks of 32 x 32 entries, layer tiles, slices of 64 values of r): a block stages its slice of the two
// 32-wide strips of F in shared memory, a thread sums four entries and adds them to G (zeroed before the launch)
// with one atomic each.
constexpr int NMF_GRAM_SLICE = 64;
template <int ZMODE>
__global__ void __launch_bounds__(256)
nmf_gram_kernel(Geo g, const float *__restrict__ F, float *__restrict__ G)
{
    constexpr int GP = 33;                               // words per staged row
    __shared__ float As[NMF_GRAM_SLICE * GP], Bs[NMF_GRAM_SLICE * GP];
    const int tile = blockIdx.y, k = g.k, t = threadIdx.x;
    const int kb = (k + 31) / 32;
    const int a0 = (blockIdx.x / kb) * 32, b0 = (blockIdx.x % kb) * 32;
    const int R = ZMODE == 0 ? g.tm : g.tn;
    const int r0 = blockIdx.z * NMF_GRAM_SLICE;
    const float *Ft = F + (size_t)tile * (ZMODE == 0 ? (size_t)g.tm * k : (size_t)k * g.tn);
    for (int e = t; e < NMF_GRAM_SLICE * 32; e += 256) {
        int r, c;
        if (ZMODE == 0) { r = e >> 5; c = e & 31; }      // consecutive threads: consecutive rank values (contiguous in Mp)
        else { c = e / NMF_GRAM_SLICE; r = e - c * NMF_GRAM_SLICE; }   // consecutive columns (contiguous in Mz)
        const bool rin = r0 + r < R;
        As[r * GP + c] = (rin && a0 + c < k) ? (ZMODE == 0 ? Ft[(size_t)(r0 + r) * k + a0 + c] : Ft[(size_t)(a0 + c) * g.tn + r0 + r]) : 0.f;
        Bs[r * GP + c] = (rin && b0 + c < k) ? (ZMODE == 0 ? Ft[(size_t)(r0 + r) * k + b0 + c] : Ft[(size_t)(b0 + c) * g.tn + r0 + r]) : 0.f;
    }
    __syncthreads();
    const int a = t >> 3, b4 = (t & 7) * 4;
    float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
    for (int r = 0; r < NMF_GRAM_SLICE; ++r) {
        const float av = As[r * GP + a];
#pragma unroll
        for (int u = 0; u < 4; ++u) s[u] = fmaf(av, Bs[r * GP + b4 + u], s[u]);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
        if (a0 + a < k && b0 + b4 + u < k) atomicAdd(G + (size_t)tile * k * k + (size_t)(a0 + a) * k + b0 + b4 + u, s[u]);
}

constexpr int NMF_MAX_RANK = 256;

// Mz[l][j] *= N1[l][j] / (sum_m G1[l][m] Mz[m][j] + eps).  A block holds the old values of its columns of Mz in shared
// memory ([k][columns]); a thread owns column j and forms four denominators at a time, reading row m of the
// (symmetric) Gram matrix as G1[m][l .. l+3].
__global__ void
nmf_update_z_kernel(Geo g, const float *__restrict__ N1, const float *__restrict__ G1, float *__restrict__ Z, float eps, int gram_in_smem)
{
    extern __shared__ __align__(16) float nmf_old[];    // [k][blockDim.x], then (gram_in_smem) the tile's Gram matrix [k][k]
    const int tile = blockIdx.y, k = g.k, t = threadIdx.x, nb = blockDim.x, j = blockIdx.x * nb + t;
    float *Zt = Z + (size_t)tile * k * g.tn;
    const float *Nt = N1 + (size_t)tile * k * g.tn, *Gt = G1 + (size_t)tile * k * k;
    if (gram_in_smem) {                                  // the sums below then wait on shared memory, not on L1 / L2
        float *Gs = nmf_old + k * nb;
        for (int e = t; e < k * k; e += nb) Gs[e] = Gt[e];
        Gt = Gs;
    }
    for (int m0 = 0; m0 < k; m0 += 8) {                  // eight requests in flight per thread
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = (m0 + u < k && j < g.tn) ? Zt[(size_t)(m0 + u) * g.tn + j] : 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (m0 + u < k) nmf_old[(m0 + u) * nb + t] = v[u];
    }
    __syncthreads();
    if (j >= g.tn) return;
    const bool vec = (k & 3) == 0;
    for (int l0 = 0; l0 < k; l0 += 4) {
        float nv[4];                                     // the numerators are asked for before the sums they divide
#pragma unroll
        for (int u = 0; u < 4; ++u) nv[u] = l0 + u < k ? Nt[(size_t)(l0 + u) * g.tn + j] : 0.f;
        float den[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
        for (int m = 0; m < k; ++m) {
            const float z = nmf_old[m * nb + t];
            if (vec) {
                const float4 gv = *reinterpret_cast<const float4 *>(Gt + (size_t)m * k + l0);
                den[0] = fmaf(gv.x, z, den[0]); den[1] = fmaf(gv.y, z, den[1]);
                den[2] = fmaf(gv.z, z, den[2]); den[3] = fmaf(gv.w, z, den[3]);
            } else {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (l0 + u < k) den[u] = fmaf(Gt[(size_t)(l0 + u) * k + m], z, den[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (l0 + u < k) Zt[(size_t)(l0 + u) * g.tn + j] = nmf_old[(l0 + u) * nb + t] * nv[u] / (den[u] + eps);
    }
}

// Mp[i][l] *= N2[i][l] / (sum_m Mp[i][m] G2[m][l] + eps).  The block's rows of Mp (contiguous in memory) are staged in
// shared memory, k + 1 words apart; a thread owns row i.
__global__ void
nmf_update_p_kernel(Geo g, const float *__restrict__ N2, const float *__restrict__ G2, float *__restrict__ P, float eps, int gram_in_smem)
{
    extern __shared__ __align__(16) float nmf_old[];    // [blockDim.x][k + 1], then (gram_in_smem) the Gram matrix [k][k], 16-byte aligned
    const int tile = blockIdx.y, k = g.k, t = threadIdx.x, nb = blockDim.x, ib = blockIdx.x * nb, i = ib + t;
    float *Pt = P + (size_t)tile * g.tm * k;
    const float *Nt = N2 + (size_t)tile * g.tm * k, *Gt = G2 + (size_t)tile * k * k;
    if (gram_in_smem) {
        float *Gs = nmf_old + ((nb * (k + 1) + 3) & ~3);
        for (int e = t; e < k * k; e += nb) Gs[e] = Gt[e];
        Gt = Gs;
    }
    const int nrows = min(nb, g.tm - ib);
    for (int e = t; e < nrows * k; e += nb) {
        const int r = e / k, c = e - r * k;
        nmf_old[r * (k + 1) + c] = Pt[(size_t)ib * k + e];
    }
    __syncthreads();
    if (i >= g.tm) return;
    const float *mine = nmf_old + t * (k + 1);
    const bool vec = (k & 3) == 0;
    for (int l0 = 0; l0 < k; l0 += 4) {
        float nv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) nv[u] = l0 + u < k ? Nt[(size_t)i * k + l0 + u] : 0.f;
        float den[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
        for (int m = 0; m < k; ++m) {
            const float p = mine[m];
            if (vec) {
                const float4 gv = *reinterpret_cast<const float4 *>(Gt + (size_t)m * k + l0);
                den[0] = fmaf(p, gv.x, den[0]); den[1] = fmaf(p, gv.y, den[1]);
                den[2] = fmaf(p, gv.z, den[2]); den[3] = fmaf(p, gv.w, den[3]);
            } else {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (l0 + u < k) den[u] = fmaf(p, Gt[(size_t)m * k + l0 + u], den[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (l0 + u < k) Pt[(size_t)i * k + l0 + u] = mine[l0 + u] * nv[u] / (den[u] + eps);
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
    const unsigned kc = (unsigned)((g.k + NP_KC - 1) / NP_KC), kb = (unsigned)((g.k + 31) / 32);
    // the update kernels keep k x (threads) old values in shared memory: 128 threads up to rank 64, 32 above
    const unsigned ut = g.k <= 64 ? 128u : 32u;
    // the Gram matrix of a tile beside the old values in shared memory, where both fit the 48 KB a launch gets without opt-in
    const int gsm = ((((size_t)ut * (g.k + 1) + 3) & ~(size_t)3) + (size_t)g.k * g.k) * sizeof(float) <= 48 * 1024 ? 1 : 0;
    const size_t gbytes = gsm ? (size_t)g.k * g.k * sizeof(float) : 0;
    const size_t smem_z = (size_t)g.k * ut * sizeof(float) + gbytes, smem_p = (((size_t)ut * (g.k + 1) + 3) & ~(size_t)3) * sizeof(float) + gbytes;
    // aligned layers: the product kernels that stream their slabs through a cp.async ring
    const bool ring = (g.cols % 8) == 0 && (g.tn % 8) == 0 && (g.k % 4) == 0 &&
                      ((reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(mp) | reinterpret_cast<uintptr_t>(mz)) & 15u) == 0;
    if (ring) {
        int dev = 0;
        static bool attr_done[LRBI_MAX_DEVICES] = {false};
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= LRBI_MAX_DEVICES) return LRBI_ERR_CUDA;
        std::lock_guard<std::mutex> lock(lib_mutex());
        if (!attr_done[dev]) {                           // more than 48 KB of dynamic shared memory: a per-device opt-in
            const cudaError_t ea = cudaFuncSetAttribute(nmf_prod_p_ring_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, NP_RING1 * NP_RING1_BYTES);
            if (ea != cudaSuccess) { note_cuda_error((int)ea); return LRBI_ERR_CUDA; }
            attr_done[dev] = true;
        }
    }
    for (int it = 0; it < iterations; ++it) {
        if (ring) nmf_prod_z_ring_kernel<<<dim3((unsigned)((g.tn + NP_THREADS - 1) / NP_THREADS), (unsigned)tiles, kc), dim3(NP_THREADS, NP_GROUPS), NP_RING * NP_RING_BYTES, s>>>(g, W, mp, N);
        else nmf_prod_z_kernel<<<dim3((unsigned)((g.tn + NP_THREADS - 1) / NP_THREADS), (unsigned)tiles, kc), dim3(NP_THREADS, NP_GROUPS), 0, s>>>(g, W, mp, N);
        cudaMemsetAsync(G, 0, (size_t)tiles * g.k * g.k * sizeof(float), s);
        nmf_gram_kernel<0><<<dim3(kb * kb, (unsigned)tiles, (unsigned)((g.tm + NMF_GRAM_SLICE - 1) / NMF_GRAM_SLICE)), 256, 0, s>>>(g, mp, G);
        nmf_update_z_kernel<<<dim3((unsigned)((g.tn + ut - 1) / ut), (unsigned)tiles), ut, smem_z, s>>>(g, N, G, mz, eps, gsm);
        if (ring) nmf_prod_p_ring_kernel<<<dim3((unsigned)((g.tm + NP_THREADS - 1) / NP_THREADS), (unsigned)tiles, kc), dim3(NP_THREADS, NP_GROUPS), NP_RING1 * NP_RING1_BYTES, s>>>(g, W, mz, N);
        else nmf_prod_p_kernel<<<dim3((unsigned)((g.tm + NP_THREADS - 1) / NP_THREADS), (unsigned)tiles, kc), dim3(NP_THREADS, NP_GROUPS), 0, s>>>(g, W, mz, N);
        cudaMemsetAsync(G, 0, (size_t)tiles * g.k * g.k * sizeof(float), s);
        nmf_gram_kernel<1><<<dim3(kb * kb, (unsigned)tiles, (unsigned)((g.tn + NMF_GRAM_SLICE - 1) / NMF_GRAM_SLICE)), 256, 0, s>>>(g, mz, G);
        nmf_update_p_kernel<<<dim3((unsigned)((g.tm + ut - 1) / ut), (unsigned)tiles), ut, smem_p, s>>>(g, N, G, mp, eps, gsm);
        count_launch(6);
    }
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error((int)e); return LRBI_ERR_CUDA; }
    return LRBI_OK;
}

}  // namespace lrbi
