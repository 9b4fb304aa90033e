// Tuned sm_100a kernels for the low-rank path on large, aligned tensors
// (cols % 8 == 0, int8/int4 error state).  HBM-bound streaming kernels:
// 256-bit global loads of the gradient, packed code words, per-block scales,
// factor fragments kept in registers, warp-shuffle absmax.  CUDA-core fp32 on
// purpose: 2r flop per element is far left of the tensor-core ridge, and the
// residual chain has to be reproducible bit for bit.
//
//   pass 1  P_i = M_i Q_{t-1}   a warp owns 4 rows and sweeps the columns
//   pass 2  Q_i = M_i^T P_hat   a thread owns 8 fixed columns and runs down the rows
//   pass 3  r = p - P_hat Q_i^T, absmax, requantise, store  (same ownership)
//
// Passes 2 and 3 tile the flat index space periodically: with L = lcm(cols,
// block) a CTA covers a segment of CW elements (a multiple of the quantisation
// block that divides L) of every "super-row" of L elements in its tile.  A
// thread's 8 elements then keep the same columns from iteration to iteration
// (factor fragment stays in registers) and every quantisation block lies
// inside one aligned group of block/8 lanes, also when blocks straddle rows.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <vector>

#include "conef_internal.h"

namespace conef {

constexpr int kFastE = 8;            // elements per thread per iteration
constexpr int kFastIt2 = 256;        // iterations per tile, pass 2
constexpr int kFastIt3 = 64;         // iterations per tile, pass 3
constexpr int kFastP1Rows = 4;       // rows per warp, pass 1
constexpr int kFastP1Warps = 8;

inline int64_t gcd64(int64_t a, int64_t b)
{
    while (b) {
        int64_t t = a % b;
        a = b;
        b = t;
    }
    return a;
}

// Decide whether the tuned kernels apply to a tensor and with which geometry.
inline void fast_classify(LayerDesc &L, int ckind, int unit, int cfg_rank)
{
    L.fast = 0;
    if (!(ckind == CONEF_C_INT8 || ckind == CONEF_C_INT4))
        return;
    if (L.cols % 8 != 0 || L.g_off % 8 != 0 || unit % kFastE != 0)
        return;
    if (L.rank != cfg_rank || !(cfg_rank == 4 || cfg_rank == 8))
        return;
    if (L.msgp_off % 4 != 0 || L.msgq_off % 4 != 0)
        return;   // float4 loads of the factors
    const int64_t lcm = L.cols / gcd64(L.cols, unit) * unit;   // super-row
    if (lcm > (1 << 20))
        return;
    const int64_t nblk = lcm / unit;                           // blocks per super-row
    // column segment: the largest divisor of nblk whose thread count is <= 256
    int64_t best = 0;
    for (int64_t u = 1; u <= nblk; ++u)
        if (nblk % u == 0 && u * unit / kFastE <= 256)
            best = u;
    if (best == 0)
        return;
    L.fast = 1;
    L.f_lcm = (int32_t)lcm;
    L.f_cw = (int32_t)(best * unit);
    L.f_threads = (int32_t)(best * unit / kFastE);
    L.f_ncg = (int32_t)(nblk / best);
    L.f_subs = (int32_t)(lcm / L.cols);
    L.f_niter = (L.d + lcm - 1) / lcm;
    L.f_rt2 = (int32_t)((L.f_niter + kFastIt2 - 1) / kFastIt2);
    L.f_rt3 = (int32_t)((L.f_niter + kFastIt3 - 1) / kFastIt3);
}

// ------------------------------------------------------------------ loads
__device__ __forceinline__ void ldg8(const float *p, float (&v)[8])
{
    asm volatile("ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]),
                   "=f"(v[7])
                 : "l"(p));
}

// raw stored state of 8 consecutive elements: code word(s) and the block scale
template <int CK>
struct Raw8 {
    uint32_t w0, w1;   // int4: w0 holds 8 nibbles; int8: w0,w1 hold 8 bytes
    float scale;
};

template <int CK>
__device__ __forceinline__ void load_raw8(const uint8_t *__restrict__ codes,
                                          const uint8_t *__restrict__ scales, uint32_t j,
                                          int unit_shift, int half, Raw8<CK> &r)
{
    if (CK == CONEF_C_INT4) {
        r.w0 = __ldg((const uint32_t *)(codes + (j >> 1)));
        r.w1 = 0;
    } else {
        const uint2 t = __ldg((const uint2 *)(codes + j));
        r.w0 = t.x;
        r.w1 = t.y;
    }
    const uint32_t blk = j >> unit_shift;
    if (half)
        r.scale = __half2float(__ushort_as_half(__ldg((const unsigned short *)scales + blk)));
    else
        r.scale = __ldg((const float *)scales + blk);
}

// e_j = float(code_j) * scale.  The integer-to-float conversion goes through
// the 2^23 trick (exact), then one rounded multiply: the same value as
// __fmul_rn((float)code, scale).
template <int CK>
__device__ __forceinline__ void decode8(const Raw8<CK> &r, float (&e)[8])
{
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        uint32_t bits;
        float off;
        if (CK == CONEF_C_INT4) {
            bits = (((r.w0 >> (4 * q)) & 0xFu) ^ 0x8u) | 0x4B000000u;   // 2^23 + (nibble ^ 8)
            off = 8388616.0f;                                          // 2^23 + 8
        } else {
            const uint32_t w = q < 4 ? r.w0 : r.w1;
            bits = (((w >> (8 * (q & 3))) & 0xFFu) ^ 0x80u) | 0x4B000000u;
            off = 8388736.0f;                                          // 2^23 + 128
        }
        e[q] = __fmul_rn(__fadd_rn(__uint_as_float(bits), -off), r.scale);
    }
}

// code = clamp(rint(x), -qmax, qmax) as a two's complement field, through the
// 1.5 * 2^23 trick (round to nearest even in the adder); NaN -> 0.
__device__ __forceinline__ uint32_t quant_bits(float r, float inv, float qmaxf)
{
    float x = __fmul_rn(r, inv);
    x = (x != x) ? 0.f : x;
    x = fminf(fmaxf(x, -qmaxf), qmaxf);
    return __float_as_uint(__fadd_rn(x, 12582912.0f));
}

// sum over the 32 lanes of NV values per lane; on return lane l holds the
// total of value index (l % NV) ... arranged so that v[0] of lane l is the sum
// of input value  idx(l) = bit-reversed selection; see the caller.
template <int NV>
__device__ __forceinline__ float warp_reduce_many(float (&v)[NV], int lane)
{
    // halving butterfly: after the step with offset o, a lane keeps half of its values
    int n = NV;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        if (n > 1) {
            const int h = n >> 1;
            const bool up = (lane & o) != 0;
#pragma unroll
            for (int i = 0; i < NV / 2; ++i)
                if (i < h) {
                    const float send = up ? v[i] : v[i + h];
                    const float keep = up ? v[i + h] : v[i];
                    v[i] = __fadd_rn(keep, __shfl_xor_sync(0xffffffffu, send, o));
                }
            n = h;
        } else {
            v[0] = __fadd_rn(v[0], __shfl_xor_sync(0xffffffffu, v[0], o));
        }
    }
    return v[0];
}

// ------------------------------------------------------------------ pass 1
// P_i[row][c] = sum_col p[row][col] * Q[col][c].  A warp owns 4 consecutive
// rows; a lane takes 8 consecutive columns of each row per sweep step, so one
// fragment of Q (8 x R, read through L1) serves 32 multiply-adds per column.
template <int CK, int R>
__global__ void __launch_bounds__(kFastP1Warps * 32)
k_fast_pass1(const __grid_constant__ DevView V, const int32_t *__restrict__ pfx)
{
    const int li = find_layer(pfx, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int worker = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t m = (uint32_t)L.cols, n = (uint32_t)L.rows;
    const uint8_t *st = V.state + worker * V.state_stride;
    const uint8_t *__restrict__ codes = st + L.a_off;
    const uint8_t *__restrict__ scales = st + L.b_off;
    const float *__restrict__ g = V.grads[worker] + L.g_off;
    const float *__restrict__ Q = V.qprev + L.msgq_off;
    float *__restrict__ P = V.msgp + worker * V.msgp_stride + L.msgp_off;
    const int unit_shift = 31 - __clz(L.unit);
    const uint32_t row0 = (uint32_t)(blockIdx.x - pfx[li]) * (kFastP1Warps * kFastP1Rows) + warp * kFastP1Rows;
    if (row0 >= n)
        return;
    float acc[kFastP1Rows * R];
#pragma unroll
    for (int i = 0; i < kFastP1Rows * R; ++i)
        acc[i] = 0.f;
    for (uint32_t col = lane * 8; col < m; col += 256) {
        float gv[kFastP1Rows][8];
        Raw8<CK> raw[kFastP1Rows];
#pragma unroll
        for (int rr = 0; rr < kFastP1Rows; ++rr) {
            const uint32_t row = min(row0 + rr, n - 1);   // clamp: a short last group re-reads a valid row
            const uint32_t j = row * m + col;
            ldg8(g + j, gv[rr]);
            load_raw8<CK>(codes, scales, j, unit_shift, V.scale_half, raw[rr]);
        }
        float qf[8][R];
#pragma unroll
        for (int q = 0; q < 8; ++q)
#pragma unroll
            for (int c = 0; c < R; c += 4) {
                const float4 t = __ldg((const float4 *)(Q + (size_t)(col + q) * R + c));
                qf[q][c] = t.x; qf[q][c + 1] = t.y; qf[q][c + 2] = t.z; qf[q][c + 3] = t.w;
            }
#pragma unroll
        for (int rr = 0; rr < kFastP1Rows; ++rr) {
            float e[8];
            decode8<CK>(raw[rr], e);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float p = __fmaf_rn(V.lr, gv[rr][q], e[q]);
#pragma unroll
                for (int c = 0; c < R; ++c)
                    acc[rr * R + c] = __fmaf_rn(p, qf[q][c], acc[rr * R + c]);
            }
        }
    }
    // reduce the 4*R per-lane sums over the warp: after the butterfly lane l
    // holds the total of one (row, c) pair
    constexpr int NV = kFastP1Rows * R;   // 16 or 32
    warp_reduce_many<NV>(acc, lane);
    // which value ended up in this lane: the butterfly keeps the upper half
    // where the lane bit is set, offsets 16, 8, 4, ... in that order
    int idx = 0, h = NV;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1)
        if (h > 1) {
            h >>= 1;
            if (lane & o)
                idx += h;
        }
    // with NV = 16 the last step (offset 1) is a plain sum: lanes 2k and 2k+1 agree
    const bool writer = (NV == 32) || ((lane & 1) == 0);
    const int rr = idx / R, c = idx % R;
    if (writer && row0 + rr < n)
        P[(size_t)(row0 + rr) * R + c] = acc[0];
}

// ------------------------------------------------------------------ passes 2 and 3
// what one thread holds of one iteration while its loads are in flight
template <int CK, int R>
struct Stage {
    float gv[8];
    Raw8<CK> raw;
    float phr[R];
};

// plain (coherent) loads for state that the same kernel rewrites in place
template <int CK>
__device__ __forceinline__ void load_raw8_rw(const uint8_t *codes, const uint8_t *scales, uint32_t j,
                                             int unit_shift, int half, Raw8<CK> &r)
{
    if (CK == CONEF_C_INT4) {
        r.w0 = *(const volatile uint32_t *)(codes + (j >> 1));
        r.w1 = 0;
    } else {
        r.w0 = *(const volatile uint32_t *)(codes + j);
        r.w1 = *(const volatile uint32_t *)(codes + j + 4);
    }
    const uint32_t blk = j >> unit_shift;
    if (half)
        r.scale = __half2float(__ushort_as_half(*((const volatile unsigned short *)scales + blk)));
    else
        r.scale = *((const volatile float *)scales + blk);
}

template <int PASS, int CK, int R>
__global__ void __launch_bounds__(256)
k_fast_pass23(const __grid_constant__ DevView V, const int32_t *__restrict__ pfx)
{
    const int li = find_layer(pfx, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int nthreads = L.f_threads;
    if ((int)threadIdx.x >= nthreads)
        return;
    const int worker = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31;
    const uint32_t m = (uint32_t)L.cols, d = (uint32_t)L.d;
    uint8_t *st = V.state + worker * V.state_stride;
    uint8_t *codes = st + L.a_off;
    uint8_t *scales = st + L.b_off;
    const float *__restrict__ g = V.grads[worker] + L.g_off;
    const float *__restrict__ ph = V.phat + L.msgp_off;
    const int unit_shift = 31 - __clz(L.unit);
    const int half = V.scale_half;
    const float lr = V.lr;
    constexpr int IT = PASS == 2 ? kFastIt2 : kFastIt3;
    const int local = blockIdx.x - pfx[li];
    const int cg = local % L.f_ncg, rt = local / L.f_ncg;
    const uint32_t lcm = (uint32_t)L.f_lcm;
    const uint32_t off = (uint32_t)cg * (uint32_t)L.f_cw + (uint32_t)tid * kFastE;   // within the super-row
    const uint32_t sub = off / m, col = off - sub * m;
    const uint32_t subs = (uint32_t)L.f_subs;
    const uint32_t it0 = (uint32_t)rt * IT;
    const uint32_t it1 = (uint32_t)min((int64_t)L.f_niter, (int64_t)it0 + IT);
    // lanes of this warp that exist (the last warp of a CTA may be partial)
    const int wbase = tid & ~31;
    const unsigned wmask = (nthreads - wbase >= 32) ? 0xffffffffu : ((1u << (nthreads - wbase)) - 1u);

    float frag[8][R];   // pass 2: accumulators of Q_i[col..col+7][:]; pass 3: Q_i[col..col+7][:]
    if (PASS == 2) {
#pragma unroll
        for (int q = 0; q < 8; ++q)
#pragma unroll
            for (int c = 0; c < R; ++c)
                frag[q][c] = 0.f;
    } else {
        const float *__restrict__ qi = V.msgq + worker * V.msgq_stride + L.msgq_off;
#pragma unroll
        for (int q = 0; q < 8; ++q)
#pragma unroll
            for (int c = 0; c < R; c += 4) {
                const float4 t = __ldg((const float4 *)(qi + (size_t)(col + q) * R + c));
                frag[q][c] = t.x; frag[q][c + 1] = t.y; frag[q][c + 2] = t.z; frag[q][c + 3] = t.w;
            }
    }
    constexpr int qmax = (CK == CONEF_C_INT8) ? 127 : 7;
    const int lanes_per_block = L.unit / kFastE;

    auto issue = [&](uint32_t it, Stage<CK, R> &S) {
        const uint32_t base = it * lcm + off;
        if (it < it1 && base < d) {
            ldg8(g + base, S.gv);
            if (PASS == 2)
                load_raw8<CK>(codes, scales, base, unit_shift, half, S.raw);
            else
                load_raw8_rw<CK>(codes, scales, base, unit_shift, half, S.raw);
            const uint32_t row = it * subs + sub;
#pragma unroll
            for (int c = 0; c < R; c += 4) {
                const float4 t = __ldg((const float4 *)(ph + (size_t)row * R + c));
                S.phr[c] = t.x; S.phr[c + 1] = t.y; S.phr[c + 2] = t.z; S.phr[c + 3] = t.w;
            }
        } else {
#pragma unroll
            for (int q = 0; q < 8; ++q)
                S.gv[q] = 0.f;
            S.raw.w0 = 0u;
            S.raw.w1 = 0u;
            S.raw.scale = 0.f;
            if (CK == CONEF_C_INT8) {   // code byte 0 decodes to 0 only through a zero scale: keep it zero
                S.raw.w0 = 0u;
            }
#pragma unroll
            for (int c = 0; c < R; ++c)
                S.phr[c] = 0.f;
        }
    };
    auto compute = [&](uint32_t it, const Stage<CK, R> &S) {
        const uint32_t base = it * lcm + off;
        const bool valid = it < it1 && base < d;
        float e[8];
        decode8<CK>(S.raw, e);
        float p[8];
#pragma unroll
        for (int q = 0; q < 8; ++q)
            p[q] = __fmaf_rn(lr, S.gv[q], e[q]);   // Alg. 2 line 5 (zero where not valid)
        if (PASS == 2) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
#pragma unroll
                for (int c = 0; c < R; ++c)
                    frag[q][c] = __fmaf_rn(p[q], S.phr[c], frag[q][c]);
        } else {
            float amax = 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                float acc = p[q];
#pragma unroll
                for (int c = 0; c < R; ++c)
                    acc = __fmaf_rn(-S.phr[c], frag[q][c], acc);   // r = p - P_hat Q_i^T
                p[q] = acc;
                amax = fmaxf(amax, fabsf(acc));
            }
            for (int o = lanes_per_block >> 1; o > 0; o >>= 1)
                amax = fmaxf(amax, __shfl_xor_sync(wmask, amax, o));
            float s, inv;
            unsigned short hb;
            quant_scale(amax, qmax, half, s, inv, hb);
            if (valid) {
                if ((lane & (lanes_per_block - 1)) == 0) {
                    const uint32_t blk = base >> unit_shift;
                    if (half)
                        ((unsigned short *)scales)[blk] = hb;
                    else
                        ((float *)scales)[blk] = s;
                }
                if (CK == CONEF_C_INT4) {
                    uint32_t w = 0;
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        w |= (quant_bits(p[q], inv, 7.0f) & 0xFu) << (4 * q);
                    *(uint32_t *)(codes + (base >> 1)) = w;
                } else {
                    uint32_t w0 = 0, w1 = 0;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        w0 |= (quant_bits(p[q], inv, 127.0f) & 0xFFu) << (8 * q);
                        w1 |= (quant_bits(p[q + 4], inv, 127.0f) & 0xFFu) << (8 * q);
                    }
                    *(uint2 *)(codes + base) = make_uint2(w0, w1);
                }
            }
        }
    };

    // two-stage software pipeline: the loads of the next iteration are issued
    // before the arithmetic of the current one
    Stage<CK, R> A, B;
    issue(it0, A);
    for (uint32_t it = it0; it < it1; it += 2) {
        issue(it + 1, B);
        compute(it, A);
        issue(it + 2, A);
        compute(it + 1, B);
    }
    if (PASS == 2) {
        // partial sums of this (row tile, sub-row): rows are summed in order by k_lr_pass2_reduce
        float *__restrict__ part = V.part + worker * V.part_stride + L.part_off +
                                   ((size_t)((size_t)rt * subs + sub) * m + col) * R;
#pragma unroll
        for (int q = 0; q < 8; ++q)
#pragma unroll
            for (int c = 0; c < R; c += 4)
                *(float4 *)(part + q * R + c) = make_float4(frag[q][c], frag[q][c + 1], frag[q][c + 2], frag[q][c + 3]);
    }
}

// ------------------------------------------------------------------ launch helpers
template <int CK, int R>
inline void fast_launch_pass1(const DevView &V, const int32_t *pfx, int tiles, cudaStream_t s)
{
    dim3 grid(tiles, V.n_workers);
    k_fast_pass1<CK, R><<<grid, kFastP1Warps * 32, 0, s>>>(V, pfx);
}
template <int PASS, int CK, int R>
inline void fast_launch_pass23(const DevView &V, const int32_t *pfx, int tiles, int threads, cudaStream_t s)
{
    dim3 grid(tiles, V.n_workers);
    k_fast_pass23<PASS, CK, R><<<grid, threads, 0, s>>>(V, pfx);
}

// PASS: 1, 2 or 3.  Returns false for a configuration that has no tuned kernel.
inline bool fast_launch(int pass, int ckind, int rank, const DevView &V, const int32_t *pfx, int tiles,
                        int threads, cudaStream_t s)
{
    if (tiles <= 0)
        return true;
#define CONEF_FAST_CASE(CKV, RV)                                                        \
    if (ckind == CKV && rank == RV) {                                                   \
        if (pass == 1) fast_launch_pass1<CKV, RV>(V, pfx, tiles, s);                    \
        else if (pass == 2) fast_launch_pass23<2, CKV, RV>(V, pfx, tiles, threads, s);  \
        else fast_launch_pass23<3, CKV, RV>(V, pfx, tiles, threads, s);                 \
        return true;                                                                    \
    }
    CONEF_FAST_CASE(CONEF_C_INT4, 4)
    CONEF_FAST_CASE(CONEF_C_INT4, 8)
    CONEF_FAST_CASE(CONEF_C_INT8, 4)
    CONEF_FAST_CASE(CONEF_C_INT8, 8)
#undef CONEF_FAST_CASE
    return false;
}

}  // namespace conef
