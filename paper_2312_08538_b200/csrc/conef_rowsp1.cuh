// Low-rank pass 1 (Sec. 5.2: P_i = M_i Q_{t-1}, with M_i = eta G + decode(e) formed on the fly)
// with one matrix row per lane, for rank 4 on an int4 / 128 / fp16 error state and matrices whose
// width is a multiple of 64.  A CTA owns 128 rows and walks the columns 64 at a time: the 128 x 64
// gradient tile and its codes are staged in shared memory by 16-byte asynchronous copies (two
// stages), each of the 8 warps takes 8 of the 64 columns, and a lane accumulates the 4 dot products
// of its 4 rows (lane, lane + 32, ...) over the whole width in registers.  No shuffles and no
// partial rows: the 8 warps' sums are added through shared memory once per tile and P_i is
// written directly.  About 75 instructions per 8 elements against 170 for the column-per-thread
// kernel, whose times follow the instruction count.
#pragma once
#include "conef_fast.cuh"

namespace conef {

constexpr int kRpRows = 128;            // rows per CTA
constexpr int kRpCols = 64;             // columns per stage: inside one 128-element block whenever cols % 64 == 0
constexpr int kRpGPitch = kRpCols + 4;  // floats; pitch / 4 odd: conflict-free 16-byte reads down a column of rows
constexpr int kRpCPitch = kRpCols / 8 + 1;   // words of codes per row, odd
constexpr int kRpThreads = 256;
struct alignas(16) RpStage {
    float g[kRpRows * kRpGPitch];
    uint32_t c[kRpRows * kRpCPitch];
};
static_assert(sizeof(RpStage) % 16 == 0, "stages stay 16-byte aligned");
constexpr size_t kRpSmem = 2 * sizeof(RpStage);

__global__ void __launch_bounds__(kRpThreads, 2) k_rows_p1(const __grid_constant__ DevView V,
                                                           const int32_t *__restrict__ pfx)
{
    extern __shared__ __align__(16) unsigned char rp_smem[];
    RpStage *st = (RpStage *)rp_smem;
    const int li = find_layer(pfx, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int worker = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = (int)L.rows, m = (int)L.cols;
    const int row0 = (blockIdx.x - pfx[li]) * kRpRows;
    const float *__restrict__ gt = V.grads[worker] + L.g_off;
    const uint8_t *__restrict__ sw = V.state + worker * V.state_stride;
    const uint8_t *__restrict__ ct = sw + L.a_off;
    const __half *__restrict__ sct = (const __half *)(sw + L.b_off);
    const float4 *__restrict__ Qt = (const float4 *)(V.qprev + L.msgq_off);
    const float lr = V.lr;
    const int nst = m / kRpCols;

    auto issue = [&](int s, int buf) {
        const int col0 = s * kRpCols;
        for (int x = tid; x < kRpRows * (kRpCols / 4); x += kRpThreads) {
            const int r = x / (kRpCols / 4), pc = x % (kRpCols / 4);
            const int row = min(row0 + r, n - 1);   // rows past the end repeat the last one and are not stored
            cp_async16(&st[buf].g[r * kRpGPitch + pc * 4], gt + (int64_t)row * m + col0 + pc * 4);
        }
        for (int x = tid; x < kRpRows * (kRpCols / 8); x += kRpThreads) {
            const int r = x / (kRpCols / 8), pc = x % (kRpCols / 8);
            const int row = min(row0 + r, n - 1);
            cp_async_small<4>(&st[buf].c[r * kRpCPitch + pc], ct + ((int64_t)row * m + col0) / 2 + pc * 4);
        }
        cp_async_commit();
    };

    float acc[4][4];
#pragma unroll
    for (int rr = 0; rr < 4; ++rr)
#pragma unroll
        for (int c = 0; c < 4; ++c)
            acc[rr][c] = 0.f;

    issue(0, 0);
    for (int s = 0; s < nst; ++s) {
        const int buf = s & 1;
        if (s + 1 < nst)
            issue(s + 1, buf ^ 1);
        else
            cp_async_commit();
        const int col0 = s * kRpCols + warp * 8;
        // this warp's 8 rows of Q_{t-1} (one address for all lanes) and its rows' block scales
        float4 q[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
            q[k] = __ldg(Qt + col0 + k);
        float sc[4];
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) {
            const int row = min(row0 + lane + 32 * rr, n - 1);
            sc[rr] = __half2float(sct[((int64_t)row * m + col0) >> 7]);
        }
        cp_async_wait<1>();
        __syncthreads();
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) {
            const int r = lane + 32 * rr;
            const float4 g0 = *(const float4 *)&st[buf].g[r * kRpGPitch + warp * 8];
            const float4 g1 = *(const float4 *)&st[buf].g[r * kRpGPitch + warp * 8 + 4];
            const uint32_t w0 = st[buf].c[r * kRpCPitch + warp];
            const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            float e[8];
            decode8<CONEF_C_INT4, true>(w0, 0u, scale_const<CONEF_C_INT4, true>(sc[rr]), e);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const float p = __fmaf_rn(lr, gv[k], e[k]);   // Alg. 2 line 5
                acc[rr][0] = __fmaf_rn(p, q[k].x, acc[rr][0]);
                acc[rr][1] = __fmaf_rn(p, q[k].y, acc[rr][1]);
                acc[rr][2] = __fmaf_rn(p, q[k].z, acc[rr][2]);
                acc[rr][3] = __fmaf_rn(p, q[k].w, acc[rr][3]);
            }
        }
        __syncthreads();   // the next iteration's copies refill this buffer
    }
    // the 8 warps hold the sums over their column slices: add them in warp order
    float4 *red = (float4 *)rp_smem;   // [8][kRpRows]
#pragma unroll
    for (int rr = 0; rr < 4; ++rr)
        red[warp * kRpRows + lane + 32 * rr] = make_float4(acc[rr][0], acc[rr][1], acc[rr][2], acc[rr][3]);
    __syncthreads();
    if (tid < kRpRows && row0 + tid < n) {
        float4 a = red[tid];
        for (int w = 1; w < 8; ++w) {
            const float4 b = red[w * kRpRows + tid];
            a.x = __fadd_rn(a.x, b.x);
            a.y = __fadd_rn(a.y, b.y);
            a.z = __fadd_rn(a.z, b.z);
            a.w = __fadd_rn(a.w, b.w);
        }
        float *out = V.msgp + worker * V.msgp_stride + L.msgp_off;
        *(float4 *)(out + (int64_t)(row0 + tid) * 4) = a;
    }
}

// which tensors the kernel takes (the caller has checked rank 4, int4, fp16 scales, blocks of 128)
inline bool rows_p1_takes(const LayerDesc &L)
{
    return L.rank == 4 && L.cols % kRpCols == 0 && L.g_off % 4 == 0 && L.msgq_off % 4 == 0 && L.msgp_off % 4 == 0 &&
           L.rows >= 32;
}

inline cudaError_t rows_p1_launch(const DevView &V, const int32_t *pfx, int tiles, cudaStream_t s)
{
    if (tiles <= 0)
        return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(k_rows_p1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRpSmem);
    if (e != cudaSuccess)
        return e;
    k_rows_p1<<<dim3(tiles, V.n_workers), kRpThreads, kRpSmem, s>>>(V, pfx);
    return cudaSuccess;
}

}  // namespace conef
