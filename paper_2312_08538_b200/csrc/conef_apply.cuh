// Model update from the summed messages (Alg. 2 lines 7-8): x <- x - Delta_t, Delta_t the mean
// over workers of Q's outputs.  HBM-bound: x is read and written once (8 B per parameter; the
// random-k case touches only the k shared coordinates).
#pragma once
#include "conef_kernels.cuh"

namespace conef {

constexpr int kApplyTile = 4096;      // elements (or message values) per CTA, dense and sparse cases
constexpr int kApplyRows = 16;        // low-rank: rows per CTA, one column per thread

// tiles per tensor, in the order the kernel decodes them
__host__ __device__ inline int64_t apply_tiles(const LayerDesc &L, int qkind)
{
    if (!L.compressed || qkind == CONEF_Q_IDENTITY)
        return (L.d + kApplyTile - 1) / kApplyTile;
    if (qkind == CONEF_Q_RANDK || qkind == CONEF_Q_RANDBLOCK)
        return (L.k + kApplyTile - 1) / kApplyTile;
    return ((L.rows + kApplyRows - 1) / kApplyRows) * ((L.cols + 255) / 256);
}

__global__ void __launch_bounds__(256) k_apply(const __grid_constant__ DevView V, const int32_t *__restrict__ pfx,
                                               float *__restrict__ x, const float *__restrict__ sum_values,
                                               const float *__restrict__ sum_dense1d)
{
    const int li = find_layer(pfx, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int64_t tile = blockIdx.x - pfx[li];
    float *__restrict__ xs = x + L.g_off;
    const float nw = V.n_workers_f;
    if (!L.compressed || V.qkind == CONEF_Q_IDENTITY) {
        const float *__restrict__ sum = L.compressed ? sum_values + L.msgv_off : sum_dense1d + L.msg1d_off;
        for (int q = threadIdx.x; q < kApplyTile; q += 256) {
            const int64_t j = tile * kApplyTile + q;
            if (j < L.d)
                xs[j] = __fsub_rn(xs[j], __fdiv_rn(sum[j], nw));
        }
    } else if (V.qkind == CONEF_Q_RANDK || V.qkind == CONEF_Q_RANDBLOCK) {
        const float *__restrict__ sum = sum_values + L.msgv_off;
        const uint32_t *__restrict__ idx = V.idx + L.idx_off;
        for (int q = threadIdx.x; q < kApplyTile; q += 256) {
            const int64_t s = tile * kApplyTile + q;
            if (s < L.k) {
                const uint32_t j = idx[s];
                xs[j] = __fsub_rn(xs[j], __fdiv_rn(sum[s], nw));   // indices are distinct: no race
            }
        }
    } else {
        // Delta = P_hat Qmean^T, Qmean = the warm start left by the reduction of the Q messages
        const int r = L.rank;
        const int64_t ctiles = (L.cols + 255) / 256;
        const int64_t b = (tile % ctiles) * 256 + threadIdx.x;
        const int64_t a0 = (tile / ctiles) * kApplyRows;
        if (b >= L.cols)
            return;
        const float *__restrict__ phat = V.phat + L.msgp_off;
        const float *__restrict__ qm = V.qprev + L.msgq_off + b * r;
        float qreg[CONEF_MAX_RANK];
#pragma unroll
        for (int c = 0; c < CONEF_MAX_RANK; ++c)
            qreg[c] = c < r ? qm[c] : 0.f;
        for (int64_t a = a0; a < min(L.rows, a0 + kApplyRows); ++a) {
            float dl = 0.f;
#pragma unroll
            for (int c = 0; c < CONEF_MAX_RANK; ++c)
                if (c < r)
                    dl = __fmaf_rn(phat[a * r + c], qreg[c], dl);
            xs[a * L.cols + b] = __fsub_rn(xs[a * L.cols + b], dl);
        }
    }
}

// the same for sketches stored in binary16: fp32 sum of the workers' values, one division, stored
// like an update (saturated, nearest even)
__global__ void __launch_bounds__(256) k_error_reset_half(uint8_t *__restrict__ state, int64_t stride_bytes, int n_workers,
                                                          float nw, int64_t halves)
{
    for (int64_t j = (int64_t)blockIdx.x * 256 + threadIdx.x; j < halves; j += (int64_t)gridDim.x * 256) {
        float acc = __half2float(((const __half *)state)[j]);
        for (int i = 1; i < n_workers; ++i)
            acc = __fadd_rn(acc, __half2float(((const __half *)(state + i * stride_bytes))[j]));
        const unsigned short h = rs_to_half(__fdiv_rn(acc, nw));
        for (int i = 0; i < n_workers; ++i)
            ((unsigned short *)(state + i * stride_bytes))[j] = h;
    }
}

}  // namespace conef

namespace conef {

// Error reset for a linear C: every worker's state becomes the mean over workers (sum in worker
// order, one division).  `words` floats per worker.
__global__ void __launch_bounds__(256) k_error_reset(uint8_t *__restrict__ state, int64_t stride_bytes, int n_workers,
                                                     float nw, int64_t words)
{
    for (int64_t j = (int64_t)blockIdx.x * 256 + threadIdx.x; j < words; j += (int64_t)gridDim.x * 256) {
        float acc = ((const float *)state)[j];
        for (int i = 1; i < n_workers; ++i)
            acc = __fadd_rn(acc, ((const float *)(state + i * stride_bytes))[j]);
        acc = __fdiv_rn(acc, nw);
        for (int i = 0; i < n_workers; ++i)
            ((float *)(state + i * stride_bytes))[j] = acc;
    }
}

}  // namespace conef
