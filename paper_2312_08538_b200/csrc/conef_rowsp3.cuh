// Low-rank pass 3 (Alg. 2 lines 5 and 9 with the rank-r Q of Sec. 5.2: r = p - P_hat Q_i^T, then
// C(r) stored in place) with one run of whole quantisation blocks per lane, for rank 4 on an
// int4 / 128 / fp16 error state.  A "span" is lcm(cols, 128) consecutive elements of the row-major
// matrix: one row when cols is a multiple of 128, two rows when it is an odd multiple of 64, so
// that a span is a whole number of 128-element blocks.  A CTA owns 64 spans (lane, lane + 32) and
// walks them one block at a time: the 64 x 128 gradient tile and its codes are staged in shared
// memory (two stages of asynchronous copies); each of the 8 warps takes 16 of the block's 128
// elements and keeps their residuals in registers, the warps' maxima meet in shared memory, and a
// second sweep quantises the residuals against the block's scale, packs the codes and stores its 8
// bytes of the block (the 8 warps fill the block's 64 bytes; L2 merges them).  No shuffles; the factor rows of Q_i
// come from L1 by one-address loads and the lane's rows of P_hat sit in registers.
#pragma once
#include <cstdlib>
#include "conef_fast.cuh"

namespace conef {

constexpr int kR3Spans = 64;             // spans per CTA: two per lane
constexpr int kR3GPitch = 128 + 4;       // floats per tile row; pitch / 4 odd: conflict-free 16-byte accesses
constexpr int kR3CPitch = 16 + 1;        // words of codes per tile row (64 bytes), odd
constexpr int kR3Threads = 256;
struct alignas(16) R3Stage {
    float g[kR3Spans * kR3GPitch];
    uint32_t c[kR3Spans * kR3CPitch];
};
static_assert(sizeof(R3Stage) % 16 == 0, "stages stay 16-byte aligned");
struct R3Smem {
    R3Stage st[2];
    float amax[2][kR3Spans][8];   // per stage parity, span and warp: maximum of the warp's 16 residuals
};

__global__ void __launch_bounds__(kR3Threads, 2) k_rows_p3(const __grid_constant__ DevView V,
                                                           const int32_t *__restrict__ pfx)
{
    constexpr int R = 4;
    extern __shared__ __align__(16) unsigned char r3_smem[];
    R3Smem &S = *(R3Smem *)r3_smem;
    const int li = find_layer(pfx, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int worker = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t m = (uint32_t)L.cols;
    const uint32_t span = (m % 128u == 0) ? m : 2u * m;   // elements per span
    const int rps = (int)(span / m);                      // matrix rows per span: 1 or 2
    const int nspans = (int)(L.rows / rps);
    const int span0 = (blockIdx.x - pfx[li]) * kR3Spans;
    const float *__restrict__ gt = V.grads[worker] + L.g_off;
    uint8_t *sw = V.state + worker * V.state_stride;
    uint8_t *ct = sw + L.a_off;
    unsigned short *sct = (unsigned short *)(sw + L.b_off);
    const float4 *__restrict__ Qi = (const float4 *)(V.msgq + worker * V.msgq_stride + L.msgq_off);
    const float lr = V.lr;
    const int nst = (int)(span / 128u);

    // a thread copies the same pieces of every stage: 16-byte pieces of the gradient tile in rows
    // r0 + 8 k (32 pieces per row), one 16-byte piece of the codes (4 per row)
    const int r0 = tid >> 5, pg = tid & 31, rc = tid >> 2, pcw = tid & 3;
    uint32_t goff[8];
#pragma unroll
    for (int k = 0; k < 8; ++k)
        goff[k] = (uint32_t)min(span0 + r0 + 8 * k, nspans - 1) * span + pg * 4;
    const uint32_t coff = ((uint32_t)min(span0 + rc, nspans - 1) * span) / 2 + pcw * 16;   // bytes
    auto issue = [&](int s, int buf) {
#pragma unroll
        for (int k = 0; k < 8; ++k)
            cp_async16(&S.st[buf].g[(r0 + 8 * k) * kR3GPitch + pg * 4], gt + goff[k] + s * 128);
        // the code tile has an odd pitch in words: four 4-byte copies
#pragma unroll
        for (int x = 0; x < 4; ++x)
            cp_async_small<4>(&S.st[buf].c[rc * kR3CPitch + pcw * 4 + x], ct + coff + s * 64 + 4 * x);
        cp_async_commit();
    };

    // the lane's rows of P_hat (one or two matrix rows per span) and the first block of each span
    float ph[2][2][R];
    uint32_t blk0[2];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
        const int sp = min(span0 + lane + 32 * rr, nspans - 1);
        blk0[rr] = (uint32_t)sp * (span / 128u);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const float4 t = *(const float4 *)(V.phat + L.msgp_off + ((int64_t)sp * rps + (h < rps ? h : 0)) * R);
            ph[rr][h][0] = t.x;
            ph[rr][h][1] = t.y;
            ph[rr][h][2] = t.z;
            ph[rr][h][3] = t.w;
        }
    }

    // One barrier per block: before it a thread waits for its copies of the next stage, so the
    // barrier both publishes the warps' maxima of this block and hands over the next stage; the
    // buffer of this block is refilled right after it (no warp reads the tile in the second sweep).
    issue(0, 0);
    cp_async_wait<0>();
    __syncthreads();
    if (nst > 1)
        issue(1, 1);
    for (int s = 0; s < nst; ++s) {
        const int buf = s & 1;
        R3Stage &T = S.st[buf];
        // ---- sweep 1: residuals of this warp's 16 elements of the block
        float am[2] = {0.f, 0.f};
        float res[2][2][8];   // [h][span of the lane][element]: kept in registers for the second sweep
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t o = (uint32_t)s * 128u + (uint32_t)warp * 16u + (uint32_t)h * 8u;   // offset in the span
            const bool second = o >= m;            // (uniform) the span's second matrix row
            const uint32_t col = second ? o - m : o;
            float4 q[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
                q[k] = __ldg(Qi + col + k);
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                const int r = lane + 32 * rr;
                const float *gp = &T.g[r * kR3GPitch + warp * 16 + h * 8];
                const float4 g0 = *(const float4 *)gp;
                const float4 g1 = *(const float4 *)(gp + 4);
                const uint32_t w0 = T.c[r * kR3CPitch + warp * 2 + h];
                const float sc = __half2float(__ushort_as_half(sct[blk0[rr] + s]));
                const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
                float e[8];
                decode8<CONEF_C_INT4, true>(w0, 0u, scale_const<CONEF_C_INT4, true>(sc), e);
                const float p0 = second ? ph[rr][1][0] : ph[rr][0][0], p1 = second ? ph[rr][1][1] : ph[rr][0][1];
                const float p2 = second ? ph[rr][1][2] : ph[rr][0][2], p3 = second ? ph[rr][1][3] : ph[rr][0][3];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    float acc = __fmaf_rn(lr, gv[k], e[k]);   // Alg. 2 line 5
                    acc = __fmaf_rn(-p0, q[k].x, acc);        // r = p - P_hat Q_i^T, ascending rank index
                    acc = __fmaf_rn(-p1, q[k].y, acc);
                    acc = __fmaf_rn(-p2, q[k].z, acc);
                    acc = __fmaf_rn(-p3, q[k].w, acc);
                    res[h][rr][k] = acc;
                    am[rr] = fmaxf(am[rr], fabsf(acc));
                }
            }
        }
#pragma unroll
        for (int rr = 0; rr < 2; ++rr)
            S.amax[buf][lane + 32 * rr][warp] = am[rr];
        cp_async_wait<0>();   // this thread's pieces of stage s + 1
        __syncthreads();
        if (s + 2 < nst)
            issue(s + 2, buf);
        // ---- the block's scale (every warp computes it for its lanes' spans), sweep 2: quantise and pack
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
            const int r = lane + 32 * rr;
            const float4 a0 = *(const float4 *)&S.amax[buf][r][0], a1 = *(const float4 *)&S.amax[buf][r][4];
            const float amax = fmaxf(fmaxf(fmaxf(a0.x, a0.y), fmaxf(a0.z, a0.w)), fmaxf(fmaxf(a1.x, a1.y), fmaxf(a1.z, a1.w)));
            float sc, inv;
            unsigned short hb;
            block_scale<CONEF_C_INT4, true>(amax, sc, inv, hb);
            if (warp == 0 && span0 + r < nspans)
                sct[blk0[rr] + s] = hb;
            if (span0 + r < nspans) {
                // this lane's 16 codes of the block: two words, 8 bytes at (block, warp)
                uint32_t c0, c1, d0, d1;
                // |r * inv| <= amax * inv for the whole block: the clamp is needed only where a
                // binary16 scale was rounded down by a lot
                if (__fmul_rn(amax, inv) < 7.49f) {
                    quant_pack8<CONEF_C_INT4, false>(res[0][rr], inv, c0, c1);
                    quant_pack8<CONEF_C_INT4, false>(res[1][rr], inv, d0, d1);
                } else {
                    quant_pack8<CONEF_C_INT4, true>(res[0][rr], inv, c0, c1);
                    quant_pack8<CONEF_C_INT4, true>(res[1][rr], inv, d0, d1);
                }
                *(uint2 *)(ct + ((size_t)(blk0[rr] + s) * 64 + warp * 8)) = make_uint2(c0, d0);
            }
        }
    }
}

// which tensors the kernel takes (the caller has checked rank 4, int4, fp16 scales, blocks of 128)
// Off unless the environment says CONEF_ROWS_P3=1 when the context is planned: on the GPT-2-XL list
// this kernel ties with the column-per-thread pass 3 under the power cap (18.7 ms both) and is the
// slower one in a cold single-kernel capture (828 us against 758 us on the two-block slice), with
// 187 against 214 instructions per 256 elements at 24 % of the warp slots.
inline bool rows_p3_takes(const LayerDesc &L)
{
    const char *env = getenv("CONEF_ROWS_P3");
    if (!env || env[0] != '1')
        return false;
    if (L.rank != 4 || L.cols % 64 != 0 || L.g_off % 4 != 0 || L.msgq_off % 4 != 0 || L.msgp_off % 4 != 0)
        return false;
    const int64_t rps = L.cols % 128 == 0 ? 1 : 2;
    return L.rows % rps == 0 && L.rows / rps >= 32;
}
inline int64_t rows_p3_spans(const LayerDesc &L) { return L.rows / (L.cols % 128 == 0 ? 1 : 2); }

inline cudaError_t rows_p3_launch(const DevView &V, const int32_t *pfx, int tiles, cudaStream_t s)
{
    if (tiles <= 0)
        return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(k_rows_p3, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(R3Smem));
    if (e != cudaSuccess)
        return e;
    k_rows_p3<<<dim3(tiles, V.n_workers), kR3Threads, sizeof(R3Smem), s>>>(V, pfx);
    return cudaSuccess;
}

}  // namespace conef
