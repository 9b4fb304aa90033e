// Low-rank pass 1 (Sec. 5.2: P_i = M_i Q_{t-1}, with M_i = eta G + decode(e) formed on the fly)
// with one matrix row per lane, for rank 4 or 8 on an int4 / 128 / fp16 error state and matrices
// whose width is a multiple of 64.  A CTA owns 64 rows and walks the columns 64 at a time: the
// gradient tile, its codes, the 64 rows of Q_{t-1} and the rows' block scales are staged in shared
// memory by asynchronous copies (two stages), each of the 8 warps takes 8 of the 64 columns, and a
// lane accumulates the dot products of its 2 rows (lane, lane + 32) over the whole width in
// registers.  No shuffles, no partial rows and no global load in the loop: the 8 warps' sums are
// added through shared memory once per tile and P_i is written directly.  Three CTAs share an SM.
#pragma once
#include "conef_fast.cuh"

namespace conef {

constexpr int kRpCols = 64;             // columns per stage: inside one 128-element block whenever cols % 64 == 0
constexpr int kRpGPitch = kRpCols + 4;  // floats; pitch / 4 odd: conflict-free 16-byte reads down a column of rows
constexpr int kRpCPitch = kRpCols / 8 + 1;   // words of codes per row, odd
constexpr int kRpThreads = 256;
#ifndef CONEF_RP_STAGES
#define CONEF_RP_STAGES 2
#endif
constexpr int kRpStages = CONEF_RP_STAGES;
template <int ROWS, int R>
struct alignas(16) RpStage {
    float g[ROWS * kRpGPitch];
    uint32_t c[ROWS * kRpCPitch];
    float4 q[kRpCols * (R / 4)];   // rows s * 64 ... of Q_{t-1}
    uint32_t sc[ROWS];             // per row: the aligned pair of binary16 scales that holds this stage's
};
#ifndef CONEF_RP_ROWS
#define CONEF_RP_ROWS 64
#endif
#ifndef CONEF_RP_MINB
#define CONEF_RP_MINB 3
#endif
__host__ __device__ constexpr int rp_rows(int) { return CONEF_RP_ROWS; }   // rows per CTA: two per lane

template <int R, bool PARTIAL>
__global__ void __launch_bounds__(kRpThreads, CONEF_RP_MINB) k_rows_p1(const __grid_constant__ DevView V,
                                                           const int32_t *__restrict__ pfx)
{
    constexpr int kRpRows = rp_rows(R), RL = kRpRows / 32;   // rows per CTA, rows per lane
    using Stage = RpStage<kRpRows, R>;
    static_assert(sizeof(Stage) % 16 == 0, "stages stay 16-byte aligned");
    extern __shared__ __align__(16) unsigned char rp_smem[];
    Stage *st = (Stage *)rp_smem;
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
    const float4 *__restrict__ Qt = (const float4 *)(V.qprev + L.msgq_off);   // R / 4 of them per column
    const float lr = V.lr;
    const float omb = V.omb;   // PARTIAL (Alg. 4): p = eta g + (1 - beta) e, the product rounded first
    const int nst = m / kRpCols;

    // A thread copies the same pieces of every stage: 16-byte pieces of the gradient tile in rows
    // r0 + 16 k, 4-byte pieces of the codes in rows rc + 32 k.  Rows past the end of the matrix
    // repeat the last one and are not stored.
    constexpr int GK = kRpRows * (kRpCols / 4) / kRpThreads, CKN = kRpRows * (kRpCols / 8) / kRpThreads;
    const int r0 = tid >> 4, pg = tid & 15, rc = tid >> 3, pcw = tid & 7;
    uint32_t goff[GK], coff[CKN];   // element / byte offsets of the pieces in stage 0 (d < 2^32)
#pragma unroll
    for (int k = 0; k < GK; ++k)
        goff[k] = (uint32_t)min(row0 + r0 + 16 * k, n - 1) * (uint32_t)m + pg * 4;
#pragma unroll
    for (int k = 0; k < CKN; ++k)
        coff[k] = ((uint32_t)min(row0 + rc + 32 * k, n - 1) * (uint32_t)m) / 2 + pcw * 4;
    const uint32_t srow = (uint32_t)min(row0 + (tid < kRpRows ? tid : 0), n - 1) * (uint32_t)m;   // the row whose scale this thread copies
    auto issue = [&](int s, int buf) {
#pragma unroll
        for (int k = 0; k < GK; ++k)
            cp_async16(&st[buf].g[(r0 + 16 * k) * kRpGPitch + pg * 4], gt + goff[k] + s * kRpCols);
#pragma unroll
        for (int k = 0; k < CKN; ++k)
            cp_async_small<4>(&st[buf].c[(rc + 32 * k) * kRpCPitch + pcw], ct + coff[k] + s * (kRpCols / 2));
        // the stage's 64 rows of Q_{t-1} and the rows' block scales ride along (loaded from L2 by every
        // lane at the top of a stage they left the warps waiting for the round trip)
        if (tid < kRpCols * (R / 4))
            cp_async16(&st[buf].q[tid], Qt + s * (kRpCols * (R / 4)) + tid);
        if (tid < kRpRows)
            cp_async_small<4>(&st[buf].sc[tid], (const uint8_t *)sct + (((srow + (uint32_t)(s * kRpCols)) >> 7 << 1) & ~3u));
        cp_async_commit();
    };
    uint32_t spar[RL];   // first element of each of this lane's rows (its block's parity picks the scale of the pair)
#pragma unroll
    for (int rr = 0; rr < RL; ++rr)
        spar[rr] = (uint32_t)min(row0 + lane + 32 * rr, n - 1) * (uint32_t)m;

    float acc[RL][R];
#pragma unroll
    for (int rr = 0; rr < RL; ++rr)
#pragma unroll
        for (int c = 0; c < R; ++c)
            acc[rr][c] = 0.f;

    // kRpStages buffers, one barrier per stage.  The first kRpStages stages are issued up front; from
    // stage 1 on, stage s + kRpStages - 1 is issued while stage s is worked on, into the buffer of
    // stage s - 1, which every warp left before the barrier of this iteration.  One group of copies
    // is committed per issue point (an empty one past the end), so that at stage s >= 1 all but the
    // newest kRpStages - 2 groups having landed means stage s has.
#pragma unroll
    for (int i = 0; i < kRpStages; ++i) {
        if (i < nst)
            issue(i, i);
        else
            cp_async_commit();
    }
    int buf = 0, nbuf = kRpStages - 1;
    for (int s = 0; s < nst; ++s) {
        // this warp's 8 rows of Q_{t-1} (one address for all lanes) come in groups of KQ columns, so
        // that rank 8 keeps 32 registers of them at a time like rank 4
        constexpr int KQ = R <= 4 ? 8 : 4;
        if (s == 0)
            cp_async_wait<kRpStages - 1>();
        else
            cp_async_wait<kRpStages - 2>();
        __syncthreads();
        if (s >= 1) {
            if (s + kRpStages - 1 < nst)
                issue(s + kRpStages - 1, nbuf);
            else
                cp_async_commit();
        }
        float sc[RL];
#pragma unroll
        for (int rr = 0; rr < RL; ++rr) {
            const uint32_t pair = st[buf].sc[lane + 32 * rr];
            const uint32_t odd = ((spar[rr] + (uint32_t)(s * kRpCols)) >> 7) & 1u;
            sc[rr] = __half2float(__ushort_as_half((unsigned short)(odd ? pair >> 16 : pair & 0xFFFFu)));
        }
        float4 q[KQ][R / 4];
#pragma unroll
        for (int k = 0; k < KQ; ++k)
#pragma unroll
            for (int h = 0; h < R / 4; ++h)
                q[k][h] = st[buf].q[(warp * 8 + k) * (R / 4) + h];
        float p[RL][8];
#pragma unroll
        for (int rr = 0; rr < RL; ++rr) {
            const int r = lane + 32 * rr;
            const float4 g0 = *(const float4 *)&st[buf].g[r * kRpGPitch + warp * 8];
            const float4 g1 = *(const float4 *)&st[buf].g[r * kRpGPitch + warp * 8 + 4];
            const uint32_t w0 = st[buf].c[r * kRpCPitch + warp];
            const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            float e[8];
            decode8<CONEF_C_INT4, true>(w0, 0u, scale_const<CONEF_C_INT4, true>(sc[rr]), e);
            if (PARTIAL) {
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    e[k] = __fmul_rn(omb, e[k]);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k)
                p[rr][k] = __fmaf_rn(lr, gv[k], e[k]);   // Alg. 2 line 5 (Alg. 4 line 5 with beta)
        }
#pragma unroll
        for (int kq = 0; kq < 8; kq += KQ) {
            if (kq > 0) {
#pragma unroll
                for (int k = 0; k < KQ; ++k)
#pragma unroll
                    for (int h = 0; h < R / 4; ++h)
                        q[k][h] = st[buf].q[(warp * 8 + kq + k) * (R / 4) + h];
            }
#pragma unroll
            for (int rr = 0; rr < RL; ++rr)
#pragma unroll
                for (int k = 0; k < KQ; ++k)
#pragma unroll
                    for (int h = 0; h < R / 4; ++h) {
                        acc[rr][4 * h + 0] = __fmaf_rn(p[rr][kq + k], q[k][h].x, acc[rr][4 * h + 0]);
                        acc[rr][4 * h + 1] = __fmaf_rn(p[rr][kq + k], q[k][h].y, acc[rr][4 * h + 1]);
                        acc[rr][4 * h + 2] = __fmaf_rn(p[rr][kq + k], q[k][h].z, acc[rr][4 * h + 2]);
                        acc[rr][4 * h + 3] = __fmaf_rn(p[rr][kq + k], q[k][h].w, acc[rr][4 * h + 3]);
                    }
        }
        nbuf = buf;
        buf = buf + 1 == kRpStages ? 0 : buf + 1;
    }
    cp_async_wait<0>();
    __syncthreads();   // every warp is done with the stages: their memory now takes the warps' sums
    // the 8 warps hold the sums over their column slices: add them in warp order
    float4 *red = (float4 *)rp_smem;   // [8 warps][kRpRows][R / 4]
#pragma unroll
    for (int rr = 0; rr < RL; ++rr)
#pragma unroll
        for (int h = 0; h < R / 4; ++h)
            red[(warp * kRpRows + lane + 32 * rr) * (R / 4) + h] =
                make_float4(acc[rr][4 * h], acc[rr][4 * h + 1], acc[rr][4 * h + 2], acc[rr][4 * h + 3]);
    __syncthreads();
    for (int x = tid; x < kRpRows * (R / 4); x += kRpThreads) {
        const int r = x / (R / 4);
        if (row0 + r >= n)
            continue;
        float4 a = red[x];
        for (int w = 1; w < 8; ++w) {
            const float4 b = red[w * kRpRows * (R / 4) + x];
            a.x = __fadd_rn(a.x, b.x);
            a.y = __fadd_rn(a.y, b.y);
            a.z = __fadd_rn(a.z, b.z);
            a.w = __fadd_rn(a.w, b.w);
        }
        float *out = V.msgp + worker * V.msgp_stride + L.msgp_off;
        *(float4 *)(out + (int64_t)row0 * R + 4 * x) = a;
    }
}

// Which tensors the kernel takes (the caller has checked int4, fp16 scales, blocks of 128).  Rank 8
// loads its rows of Q in two groups of four columns, so that it keeps as many of them in registers
// at a time as rank 4.
inline bool rows_p1_takes(const LayerDesc &L)
{
    return (L.rank == 4 || L.rank == 8) && L.cols % kRpCols == 0 && L.g_off % 4 == 0 && L.msgq_off % 4 == 0 &&
           L.msgp_off % 4 == 0 && L.rows >= 32;
}

template <int R>
inline cudaError_t rows_p1_launch(const DevView &V, const int32_t *pfx, int tiles, cudaStream_t s)
{
    if (tiles <= 0)
        return cudaSuccess;
    constexpr size_t smem = kRpStages * sizeof(RpStage<rp_rows(R), R>);
    static int done_partial[64], done_plain[64];
    if (V.beta != 0.f) {
        const cudaError_t e = opt_in_smem(k_rows_p1<R, true>, smem, done_partial);
        if (e != cudaSuccess)
            return e;
        k_rows_p1<R, true><<<dim3(tiles, V.n_workers), kRpThreads, smem, s>>>(V, pfx);
        return cudaSuccess;
    }
    const cudaError_t e = opt_in_smem(k_rows_p1<R, false>, smem, done_plain);
    if (e != cudaSuccess)
        return e;
    k_rows_p1<R, false><<<dim3(tiles, V.n_workers), kRpThreads, smem, s>>>(V, pfx);
    return cudaSuccess;
}

}  // namespace conef
