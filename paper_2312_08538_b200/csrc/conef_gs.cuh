// P-reduce + orthonormalisation of P_bar on a thread-block cluster.
//
// One cluster per compressed tensor: CTA k of the cluster keeps rows
// [k * rows_per_cta, ...) of P_bar in registers (up to 8 rows per thread), so
// nothing goes back to memory between the sum over workers and P_hat.
// P_hat is the orthonormal factor of the QR factorisation with a positive
// diagonal, the one left-to-right (modified) Gram-Schmidt produces.  It is
// computed through the Gram matrix: G = P_bar^T P_bar needs ONE reduction
// over the tensor (fp64 across threads: per warp by shuffles, per CTA through
// shared memory, across the cluster by reading the other CTAs' shared memory
// in rank order, so the result does not depend on scheduling), its Cholesky
// factor L is formed in fp64 by one thread, and every row solves
// P_hat L^T = P_bar in fp64.  Against Gram-Schmidt column by column (r
// reductions, kept below as the alternative) the GPT-2-small list went from
// 0.20 to 0.06 ms and P_hat agrees with the oracle's Gram-Schmidt to 4e-6
// (relative Frobenius).
#pragma once
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <float.h>

#include "conef_internal.h"
#include "conef_kernels.cuh"

namespace conef {

namespace cg = cooperative_groups;

constexpr int kGsThreads = 512;
// rows per thread: 8 rows of rank up to 8 fit the 128 registers a 512-thread CTA may use
__host__ __device__ constexpr int gs_rows(int R) { return R <= 8 ? 8 : 4; }
__host__ __device__ constexpr int gs_rows_per_cta(int R) { return kGsThreads * gs_rows(R); }

#ifndef CONEF_GS_CHOLESKY
#define CONEF_GS_CHOLESKY 1
#endif

template <int R>
__global__ void __launch_bounds__(kGsThreads, 1)
k_gs_cluster(const __grid_constant__ DevView V, const int32_t *__restrict__ pfx, float *__restrict__ out_sum)
{
    constexpr int kGsRows = gs_rows(R);
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned csize = cluster.num_blocks();
    const unsigned crank = cluster.block_rank();
#if !CONEF_GS_CHOLESKY
    __shared__ double warp_part[32][R];
    __shared__ double cta_part[2][R];            // double-buffered by column parity
#endif
    const int tile = blockIdx.x / csize;         // one cluster per tensor of this launch
    const int li = find_layer(pfx, V.n_layers, tile);
    const LayerDesc *Lp = V.layers + li;
    const int64_t n = Lp->rows;
    const int r = Lp->rank;                      // r <= R
    const int64_t off = Lp->msgp_off;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t rows_per_cta = (n + csize - 1) / csize;
    const int64_t row_lo = crank * rows_per_cta;
    const int64_t row_hi = min(n, row_lo + rows_per_cta);

    // P_bar = ((P_0 + P_1) + P_2) + ... in worker order.  All of a worker's values are loaded
    // before any is used and nothing is stored until the sum is complete, so that the loads of a
    // round are in flight together (one round trip to L2 per worker instead of one per value).
    float v[kGsRows][R];
#pragma unroll
    for (int k = 0; k < kGsRows; ++k)
#pragma unroll
        for (int c = 0; c < R; ++c)
            v[k][c] = 0.f;
    constexpr int KB = R > 4 ? 2 : 8;   // rows loaded per round (registers)
    for (int i = 0; i < V.n_workers; ++i) {
        const float *__restrict__ src = V.msgp + i * V.msgp_stride + off;
#pragma unroll
        for (int k0 = 0; k0 < kGsRows; k0 += KB) {
            float x[KB][R];
            if (r == R && (off & 3) == 0 && (V.msgp_stride & 3) == 0) {
                // full rank: a row is R contiguous, 16-byte aligned floats
#pragma unroll
                for (int k = 0; k < KB; ++k) {
                    const int64_t a = row_lo + (int64_t)(k0 + k) * kGsThreads + tid;
#pragma unroll
                    for (int c = 0; c < R; c += 4) {
                        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (a < row_hi)
                            t = __ldg((const float4 *)(src + a * R + c));
                        x[k][c] = t.x; x[k][c + 1] = t.y; x[k][c + 2] = t.z; x[k][c + 3] = t.w;
                    }
                }
            } else {
#pragma unroll
                for (int k = 0; k < KB; ++k) {
                    const int64_t a = row_lo + (int64_t)(k0 + k) * kGsThreads + tid;
#pragma unroll
                    for (int c = 0; c < R; ++c)
                        x[k][c] = (a < row_hi && c < r) ? __ldg(src + a * r + c) : 0.f;
                }
            }
#pragma unroll
            for (int k = 0; k < KB; ++k)
#pragma unroll
                for (int c = 0; c < R; ++c)
                    v[k0 + k][c] = i == 0 ? x[k][c] : __fadd_rn(v[k0 + k][c], x[k][c]);
        }
    }
    const bool vec = r == R && (off & 3) == 0;
#pragma unroll
    for (int k = 0; k < kGsRows; ++k) {
        const int64_t a = row_lo + (int64_t)k * kGsThreads + tid;
        if (a < row_hi) {
            if (vec) {
#pragma unroll
                for (int c = 0; c < R; c += 4) {
                    const float4 t = make_float4(v[k][c], v[k][c + 1], v[k][c + 2], v[k][c + 3]);
                    *(float4 *)(V.pbar + off + a * R + c) = t;
                    if (out_sum) {
                        if (((uintptr_t)out_sum & 15) == 0)
                            *(float4 *)(out_sum + off + a * R + c) = t;
                        else {
                            out_sum[off + a * R + c] = t.x; out_sum[off + a * R + c + 1] = t.y;
                            out_sum[off + a * R + c + 2] = t.z; out_sum[off + a * R + c + 3] = t.w;
                        }
                    }
                }
            } else {
#pragma unroll
                for (int c = 0; c < R; ++c)
                    if (c < r) {
                        V.pbar[off + a * r + c] = v[k][c];
                        if (out_sum)
                            out_sum[off + a * r + c] = v[k][c];
                    }
            }
        }
    }

#if CONEF_GS_CHOLESKY
    // The orthonormal factor through the Gram matrix: P_bar = P_hat L^T with L the Cholesky factor of
    // G = P_bar^T P_bar, which is the same P_hat as left-to-right Gram-Schmidt gives (both are the
    // QR factorisation with a positive diagonal), but needs ONE reduction over the tensor instead of
    // one per column.  G is accumulated in fp64 throughout (Cholesky-QR squares the condition
    // number: fp32 partial sums lost a 4 x 4 P_bar of condition 2e3), factored in fp64 by one
    // thread, and every row is solved in fp64.  A column whose
    // pivot is not >= FLT_MIN as a float is dead: it becomes zero and takes no part afterwards.
    {
        constexpr int NG = R * (R + 1) / 2;          // entries (j, c), c <= j, at j (j + 1) / 2 + c
        __shared__ double warp_g[kGsThreads / 32][NG];
        __shared__ double cta_g[NG];
        __shared__ double Ls[NG];
        __shared__ double invd[R];
#pragma unroll
        for (int j = 0; j < R; ++j)
#pragma unroll
            for (int c = 0; c <= j; ++c) {
                double td = 0.0;   // products of two floats are exact in fp64
#pragma unroll
                for (int k = 0; k < kGsRows; ++k)
                    td = fma((double)v[k][c], (double)v[k][j], td);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1)
                    td += __shfl_xor_sync(0xffffffffu, td, o);
                if (lane == 0)
                    warp_g[warp][j * (j + 1) / 2 + c] = td;
            }
        __syncthreads();
        if (tid < NG) {
            double t = 0.0;
            for (int w = 0; w < kGsThreads / 32; ++w)
                t += warp_g[w][tid];
            cta_g[tid] = t;
        }
        cluster.sync();   // every CTA's partial Gram matrix is in its shared memory
        if (tid < NG) {
            double t = 0.0;
            for (unsigned k = 0; k < csize; ++k)   // rank order
                t += *cluster.map_shared_rank(&cta_g[tid], k);
            Ls[tid] = t;
        }
        __syncthreads();
        if (tid == 0) {
            for (int c = 0; c < R; ++c) {
                double d = Ls[c * (c + 1) / 2 + c];
                for (int k = 0; k < c; ++k)
                    d -= Ls[c * (c + 1) / 2 + k] * Ls[c * (c + 1) / 2 + k];
                const double sd = sqrt(d);
                const bool dead = !((float)sd >= FLT_MIN);   // also a negative or NaN pivot
                Ls[c * (c + 1) / 2 + c] = dead ? 0.0 : sd;
                invd[c] = dead ? 0.0 : 1.0 / sd;
                for (int j = c + 1; j < R; ++j) {
                    double t = Ls[j * (j + 1) / 2 + c];
                    for (int k = 0; k < c; ++k)
                        t -= Ls[j * (j + 1) / 2 + k] * Ls[c * (c + 1) / 2 + k];
                    Ls[j * (j + 1) / 2 + c] = dead ? 0.0 : t * invd[c];
                }
            }
        }
        __syncthreads();
        // P_hat[a][c] = (P_bar[a][c] - sum_{k<c} L[c][k] P_hat[a][k]) / L[c][c]
#pragma unroll
        for (int k = 0; k < kGsRows; ++k) {
            double x[R];
#pragma unroll
            for (int c = 0; c < R; ++c) {
                double t = (double)v[k][c];
#pragma unroll
                for (int kk = 0; kk < c; ++kk)
                    t -= Ls[c * (c + 1) / 2 + kk] * x[kk];
                x[c] = t * invd[c];
                v[k][c] = (float)x[c];
            }
        }
    }
#else
#pragma unroll
    for (int c = 0; c < R; ++c) {
        if (c >= r)
            break;   // r is the same in every thread of the cluster
        // d[j] = sum_a v[a][c] * v[a][j], j = c .. r-1, over the whole tensor
        // a thread's few rows are summed in fp32; everything across threads is fp64
#pragma unroll
        for (int j = 0; j < R; ++j) {
            float t = 0.f;
            if (j >= c && j < r) {
#pragma unroll
                for (int k = 0; k < kGsRows; ++k)
                    t = __fmaf_rn(v[k][c], v[k][j], t);
            }
            double td = (double)t;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
                td += __shfl_xor_sync(0xffffffffu, td, o);
            if (lane == 0)
                warp_part[warp][j] = td;
        }
        __syncthreads();
        if (warp == 0) {
#pragma unroll
            for (int j = 0; j < R; ++j) {
                double t = lane < kGsThreads / 32 ? warp_part[lane][j] : 0.0;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1)
                    t += __shfl_xor_sync(0xffffffffu, t, o);
                if (lane == 0)
                    cta_part[c & 1][j] = t;
            }
        }
        cluster.sync();   // every CTA's partial is in its shared memory
        // sum over the cluster: lane k of every warp reads CTA k's partial (one remote round trip
        // for all of them), a butterfly over the lanes adds them in a fixed tree
        double d[R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            double t = (unsigned)lane < csize ? *cluster.map_shared_rank(&cta_part[c & 1][j], lane) : 0.0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
                t += __shfl_xor_sync(0xffffffffu, t, o);
            d[j] = t;
        }
        // (the buffer of the other parity is rewritten only after the next cluster.sync)
        const float nu = (float)sqrt(d[c]);
        const bool dead = !(nu >= FLT_MIN);
        // P_hat[:,c] . v[:,j]: lane j divides, the others take its result
        float coef[R];
        {
            double mine = 0.0;
#pragma unroll
            for (int j = 0; j < R; ++j)
                mine = lane == j ? d[j] : mine;
            const float cj = dead ? 0.f : (float)(mine / (double)nu);
#pragma unroll
            for (int j = 0; j < R; ++j)
                coef[j] = __shfl_sync(0xffffffffu, cj, j);
        }
#pragma unroll
        for (int k = 0; k < kGsRows; ++k) {
            const float ph = dead ? 0.f : __fdiv_rn(v[k][c], nu);
            v[k][c] = ph;
#pragma unroll
            for (int j = 0; j < R; ++j)
                if (j > c && j < r)
                    v[k][j] = __fmaf_rn(-coef[j], ph, v[k][j]);
        }
    }
#endif
    cluster.sync();       // no CTA leaves while its shared memory may still be read
#pragma unroll
    for (int k = 0; k < kGsRows; ++k) {
        const int64_t a = row_lo + (int64_t)k * kGsThreads + tid;
        if (a < row_hi) {
            if (vec) {
#pragma unroll
                for (int c = 0; c < R; c += 4)
                    *(float4 *)(V.phat + off + a * R + c) = make_float4(v[k][c], v[k][c + 1], v[k][c + 2], v[k][c + 3]);
            } else {
#pragma unroll
                for (int c = 0; c < R; ++c)
                    if (c < r)
                        V.phat[off + a * r + c] = v[k][c];
            }
        }
    }
}

// Launch over `tiles` tensors (prefix table pfx) with the given cluster size.
template <int R>
inline cudaError_t gs_launch(const DevView &V, const int32_t *pfx, int tiles, int cluster_size, float *out_sum,
                             cudaStream_t s)
{
    if (tiles <= 0)
        return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles * cluster_size), 1, 1);
    cfg.blockDim = dim3(kGsThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    if (cluster_size > 8) {   // above the portable limit: opt in once
        static bool allowed[64] = {};   // per device: function attributes are set per device
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess)
            return e;
        if (dev < 0 || dev >= 64 || !allowed[dev]) {
            e = cudaFuncSetAttribute(k_gs_cluster<R>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
            if (e != cudaSuccess)
                return e;
            if (dev >= 0 && dev < 64)
                allowed[dev] = true;
        }
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster_size;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_gs_cluster<R>, V, pfx, out_sum);
}

}  // namespace conef
