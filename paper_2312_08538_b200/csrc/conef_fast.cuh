// Tuned sm_100a kernels for the low-rank path on large, aligned tensors
// (cols % 32 == 0, int8/int4 error state).  HBM-bound streaming kernels: every
// thread runs its own ring of asynchronous copies (cp.async, 16 bytes each,
// L2 -> shared memory) that stages its gradient and code words several
// iterations ahead, so memory-level parallelism does not depend on registers
// or occupancy and needs no barrier (a thread only ever reads what it copied);
// factor fragments stay in registers, the block scales and the rows of P_hat
// of 64 iterations at a time are staged in shared memory by the CTA, absmax
// is a warp shuffle.  CUDA-core fp32 on purpose: 2r flop per element is far left
// of the tensor-core ridge, and the residual chain has to be reproducible bit
// for bit.  (A ring of TMA bulk copies per warp was measured first: at 1 KB
// per request it was slower than plain loads.)
//
//   pass 1  P_i = M_i Q_{t-1}   a thread owns 8 fixed columns; row sums by warp shuffles, one partial row per warp
//   pass 2  Q_i = M_i^T P_hat   a thread owns 8 fixed columns and runs down the rows
//   pass 3  r = p - P_hat Q_i^T, absmax, requantise, store  (same ownership)
//
// Passes 2 and 3 tile the flat index space periodically: with the period
// L = lcm(cols, 256) a CTA of w warps covers a segment of 256 w elements of
// every period in its tile (w divides L / 256).  A thread's 8 elements then
// keep the same columns from iteration to iteration (factor fragment stays in
// registers), every warp is full, and every quantisation block lies inside one
// aligned group of block/8 lanes, also when blocks straddle rows.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <vector>

#include "conef_internal.h"
#include "conef_codec.cuh"

namespace conef {

constexpr int kFastE = 8;            // elements per thread per iteration
constexpr int kFastIt1 = 64;         // iterations per tile, pass 1 (upper limits: small models get shorter tiles, see fast_tile_iters)
constexpr int kFastIt2 = 256;        // iterations per tile, pass 2
constexpr int kFastIt3 = 128;        // iterations per tile, pass 3
// Compile-time tunables (-D overrides serve experiments): iterations a thread works on at once
// for rank 8 / for rank 4 in pass 3, the register cap of rank-4 pass 3 as CTAs per SM, the ring
// depths, and whether the loop is unrolled over the ring.  Rank 4: pass 2 runs a ring of 4 stages,
// passes 1 and 3 of 2; rank 8: 4 stages and two iterations at once in passes 2 and 3.  Scalar
// fp32 instructions throughout (packed pairs cost registers under the 64-register cap).
#ifndef CONEF_NI8
#define CONEF_NI8 2
#endif
#ifndef CONEF_NI4
#define CONEF_NI4 1
#endif
#ifndef CONEF_MB4
#define CONEF_MB4 4
#endif
#ifndef CONEF_NI8_P2
#define CONEF_NI8_P2 1
#endif
#ifndef CONEF_MB8
#define CONEF_MB8 2
#endif
#ifndef CONEF_RING8
#define CONEF_RING8 4
#endif
#ifndef CONEF_RING4_P1
#define CONEF_RING4_P1 2
#endif
#ifndef CONEF_RING4_P3
#define CONEF_RING4_P3 2
#endif
#ifndef CONEF_UNROLL4
#define CONEF_UNROLL4 1
#endif
__host__ __device__ constexpr int ring_depth(int pass, int rank)
{
    return rank > 4 ? CONEF_RING8 : (pass == 2) ? 4 : (pass == 3 && CONEF_NI4 > 1) ? 4 : pass == 1 ? CONEF_RING4_P1 : CONEF_RING4_P3;
}
// Rank 4 unrolls the loop once per ring stage (constant slot addresses); rank 8, whose body is twice
// as large, keeps one copy of it and a running slot index.
#ifndef CONEF_UNROLL8
#define CONEF_UNROLL8 0   // bit p-1: unroll pass p of rank 8 over the ring (185-213 registers: slower)
#endif
__host__ __device__ constexpr bool ring_unrolled(int pass, int rank)
{
    return rank <= 4 ? !(pass == 3 && CONEF_NI4 > 1) && (pass == 2 || CONEF_UNROLL4 != 0) : (CONEF_UNROLL8 >> (pass - 1)) & 1;
}
// Rank 8 keeps a 64-register factor fragment per thread, so few warps fit on an SM; a thread
// then works on two consecutive iterations (two rows of its 8 columns) at once, which gives the
// scheduler two independent dependency chains per warp.
__host__ __device__ constexpr int iters_per_step(int pass, int rank)
{
    return rank <= 4 ? (pass == 3 ? CONEF_NI4 : 1) : (pass == 1 ? 1 : pass == 2 ? CONEF_NI8_P2 : CONEF_NI8);
}
// minimum CTAs of 256 threads per SM the compiler must allow for (caps the registers)
__host__ __device__ constexpr int min_ctas(int pass, int rank)
{
    return rank <= 4 ? (pass == 3 ? CONEF_MB4 : 4) : (pass == 1 ? 2 : CONEF_MB8);
}
constexpr int kFastMaxWarps = 8;     // warps per CTA, passes 2 and 3
// The passes stage the rows of P_hat and the block scales of kFastStageIt iterations at a time in
// shared memory, CTA-wide, between two barriers: loaded from L2 by each thread in every iteration,
// even an iteration ahead, they held the warp for an L2 round trip per iteration (a wait on the
// scoreboard such a load shares ends only when the youngest load on it has returned).
constexpr int kFastStageIt = 64;
#ifndef CONEF_PAIRS
#define CONEF_PAIRS 1
#endif
__host__ __device__ constexpr bool pairs_pass(int pass) { return CONEF_PAIRS != 0 && pass == 3; }
// bytes of that stage: per iteration `subs` rows of P_hat (passes 2, 3) and threads * 8 / unit scales
inline size_t fast_stage_bytes(int pass, int rank, int it, int subs, int threads, int unit, int scale_bytes)
{
    const size_t ph = pass == 1 ? 0 : (size_t)subs * rank * 4 * (pairs_pass(pass) ? 2 : 1);
    return (size_t)std::min(it, kFastStageIt) * (ph + (size_t)(threads * kFastE / unit) * scale_bytes) + 16;
}

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
// Iterations per tile for a model with `cta_iters` CTA-iterations per step over all workers: the
// limits above for large models; shorter tiles where those would leave the SMs with fewer than
// about 16 CTAs each per pass (a launch of few long tiles takes the time of its longest tile).  Powers of two from 8 up (matrix heights are mostly powers of two times small
// factors, so such tiles leave no ragged tail).
inline int fast_tile_iters(int limit, int64_t cta_iters)
{
    const int64_t want = cta_iters / (kPlanSMs * 16);
    int it = 8;
    while (it * 2 <= limit && it * 8 <= want * 5)   // up to 25 % above the wanted length
        it *= 2;
    return it;
}

inline void fast_classify(LayerDesc &L, int ckind, int unit, int cfg_rank, int it1 = kFastIt1, int it2 = kFastIt2,
                          int it3 = kFastIt3)
{
    L.fast = 0;
    if (!(ckind == CONEF_C_INT8 || ckind == CONEF_C_INT4))
        return;
    if (L.cols % 32 != 0 || L.g_off % 8 != 0 || unit < 32 || 256 % unit != 0)
        return;   // 16-byte copies of gradient and codes; blocks must tile a warp's 256 elements
    if (L.d >= (1ll << 31))
        return;   // 32-bit element offsets with a period of slack
    if (L.rank != cfg_rank || !(cfg_rank == 4 || cfg_rank == 8))
        return;
    if (L.msgp_off % 4 != 0 || L.msgq_off % 4 != 0)
        return;   // float4 loads of the factors
    const int64_t lcm = L.cols / gcd64(L.cols, 256) * 256;   // period
    if (lcm > (1 << 22) || lcm >= (1ll << 31) / 8)
        return;
    const int64_t nw = lcm / 256;                            // warps per period
    int64_t best = 1;
    for (int64_t w = 1; w <= kFastMaxWarps; ++w)
        if (nw % w == 0)
            best = w;
    L.fast = 1;
    L.f_lcm = (int32_t)lcm;
    L.f_cw = (int32_t)(best * 256);
    L.f_threads = (int32_t)(best * 32);
    L.f_ncg = (int32_t)(nw / best);
    L.f_subs = (int32_t)(lcm / L.cols);
    L.f_niter = (L.d + lcm - 1) / lcm;
    L.f_it1 = it1;
    L.f_it2 = it2;
    L.f_it3 = it3;
    L.f_rt1 = (int32_t)((L.f_niter + it1 - 1) / it1);
    // a row meets at most this many warps (256 elements each)
    L.f_j = (int32_t)((L.cols + 255) / 256 + 1);
    L.f_rt2 = (int32_t)((L.f_niter + it2 - 1) / it2);
    L.f_rt3 = (int32_t)((L.f_niter + it3 - 1) / it3);
}

// ------------------------------------------------------------------ asynchronous copies
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
// 16 bytes, global -> shared.  A thread copies the two halves of a 32-byte
// sector with two of these; caching in L1 (.ca) makes the second one hit
// there, so that every sector crosses the L2 -> SM crossbar once (with .cg it
// was measured to cross twice).
__device__ __forceinline__ void cp_async16(void *dst, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
template <int BYTES>   // 4 or 8
__device__ __forceinline__ void cp_async_small(void *dst, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2;" ::"r"(smem_u32(dst)), "l"(src), "n"(BYTES) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }


// sum over the 32 lanes of NV values per lane by a halving butterfly: after
// the step with offset o a lane keeps half of its values; see the caller for
// which total ends up in which lane.
template <int NV>
__device__ __forceinline__ float warp_reduce_many(float (&v)[NV], int lane)
{
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

// ------------------------------------------------------------------ the three passes
template <int N>
struct IntC {
    static constexpr int value = N;
    __device__ constexpr operator int() const { return N; }
};
struct IntR {   // a run-time value where IntC gives a constant
    int v;
    __device__ operator int() const { return v; }
};
// f(IntC<0>()), f(IntC<1>()), ..., f(IntC<N-1>())
template <int N, class F>
__device__ __forceinline__ void static_for(F &&f)
{
    if constexpr (N > 0) {
        static_for<N - 1>(f);
        f(IntC<N - 1>());
    }
}

// PASS 1, 2 or 3.  Rank 4 is capped at 64 registers (a few spilled words), which lets six of the
// usual 160-thread CTAs share an SM; rank 8 keeps its 128 registers.
// PARTIAL: partial error feedback, Alg. 4: p = eta g + (1 - beta) e with the product rounded first,
// and the stored error is C(beta e + r).  A template parameter so that Alg. 2 pays nothing for it.
template <int PASS, int CK, int R, bool HALF, bool SHORT, bool NARROW, bool PARTIAL = false>
__global__ void __launch_bounds__(kFastMaxWarps * 32, min_ctas(PASS, R))
k_fast_pass(const __grid_constant__ DevView V, const int32_t *__restrict__ pfx)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const int li = find_layer(pfx, V.n_layers, blockIdx.x);
    const LayerDesc *Lp = V.layers + li;
    // everything the loop needs goes to registers first
    const uint32_t m = (uint32_t)Lp->cols, d = (uint32_t)Lp->d, P = (uint32_t)Lp->f_lcm;
    const uint32_t subs = (uint32_t)Lp->f_subs, ncg = (uint32_t)Lp->f_ncg;
    const uint32_t niter = (uint32_t)Lp->f_niter;
    const int unit_shift = 31 - __clz(Lp->unit);
    const int lpb = Lp->unit >> 3;   // lanes per quantisation block
    const int worker = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31;
    const int bd = blockDim.x;
    // tile length: a constant for large models (faster than the same value read from the table),
    // the table's value for small ones
    const uint32_t IT = SHORT ? (uint32_t)(PASS == 1 ? Lp->f_it1 : PASS == 2 ? Lp->f_it2 : Lp->f_it3)
                              : (uint32_t)(PASS == 1 ? kFastIt1 : PASS == 2 ? kFastIt2 : kFastIt3);
    constexpr int kRing23 = ring_depth(PASS, R);
    constexpr int NI = iters_per_step(PASS, R);                   // iterations a thread works on at once
    constexpr int CW = (CK == CONEF_C_INT4) ? 1 : 2;        // code words per thread and iteration
    constexpr int SB = HALF ? 2 : 4;                        // bytes per scale
    const uint32_t local = blockIdx.x - pfx[li];
    const uint32_t cg = local % ncg, rt = local / ncg;
    const uint32_t off = cg * (uint32_t)Lp->f_cw + (uint32_t)tid * kFastE;   // within the period
    const uint32_t sub = off / m, col = off - sub * m;
    const uint32_t it0 = rt * IT;
    const uint32_t it1 = min(niter, it0 + IT);
    const uint32_t it_full = min(it1, d / P);                           // iterations wholly inside the tensor
    const uint32_t it_mine = off < d ? min(it1, (d - off + P - 1) / P) : it0;   // this thread's elements exist below it

    uint8_t *st = V.state + worker * V.state_stride;
    const uint32_t base0 = it0 * P + off;
    const float *gp_iss = V.grads[worker] + Lp->g_off + base0;          // copy source, 3 iterations ahead
    const uint8_t *cp_iss = st + Lp->a_off + (size_t)base0 * CW / 2;
    uint8_t *cp_st = st + Lp->a_off + (size_t)base0 * CW / 2;           // where this iteration's codes go back
    uint8_t *sp = st + Lp->b_off + (size_t)(base0 >> unit_shift) * SB;  // scale of the current iteration
    const uint32_t sp_step = (P >> unit_shift) * SB;
    const float lr = V.lr;
    const float omb = V.omb, beta = V.beta;   // (used with PARTIAL only)

    // ring stage s: lo[s][thread], hi[s][thread] (float4 each), cw[s][thread] (code words)
    float4 *ring_lo = (float4 *)smem_raw + tid;
    float4 *ring_hi = ring_lo + kRing23 * bd;
    uint32_t *ring_cw = (uint32_t *)((float4 *)smem_raw + 2 * kRing23 * bd) + tid * CW;
    // pass 3 of Alg. 2 computes on pairs of elements (packed fp32 instructions); its rows of P_hat
    // are staged negated and doubled, (-P_hat[c], -P_hat[c]) for each c, so that a 16-byte load
    // yields two ready operands
    constexpr bool PAIR = pairs_pass(PASS) && !PARTIAL && HALF;   // (fp32 scales: the two-step decode made it slower)
    constexpr int PHW = PAIR ? 2 : 1;   // staged floats per element of a row of P_hat
    // the rows of P_hat and the block scales of kFastStageIt iterations at a time, staged by the CTA behind the ring
    const uint32_t st_nb = ((uint32_t)bd * kFastE) >> unit_shift;               // blocks a CTA covers per iteration
    float *st_ph = (float *)(smem_raw + (size_t)kRing23 * bd * (32 + 4 * CW));
    uint8_t *st_sc = (uint8_t *)(st_ph + (PASS == 1 ? 0 : (size_t)min(IT, (uint32_t)kFastStageIt) * subs * R * PHW));

    // pass 1: where this warp's row sums go.  rowA = the row (within the period) of the warp's first
    // lane; a warp straddles when its last lane is in the next row.  The totals of warp_reduce_many
    // end up in the lanes whose bits below p1_plain are zero, column p1_idx each.
    const int64_t n_rows = Lp->rows;
    const uint32_t woff = off - (uint32_t)lane * kFastE;                  // first element of the warp within the period
    const uint32_t rowA = woff / m;
    const bool p1_straddle = PASS == 1 && (woff + 255) / m != rowA;
    const bool p1_first = sub == rowA;                                    // this lane belongs to the first of the two rows
    int p1_idx = 0, p1_plain = 32;
    {
        int hh = R;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1)
            if (hh > 1) {
                hh >>= 1;
                if (lane & o)
                    p1_idx += hh;
                p1_plain = o;
            }
    }
    // rows narrower than a warp's 256 elements: several rows per warp, summed by a segmented
    // shuffle reduction; p1_same bit k: lane + 2^k is in the same row; heads write
    constexpr bool p1_narrow = PASS == 1 && NARROW;   // (a launch holds tensors of one kind: kept out of the wide kernel, where it cost 9 %)
    uint32_t p1_same = 0;
    bool p1_head = false;
    if (p1_narrow) {
#pragma unroll
        for (int k = 0; k < 5; ++k) {
            const uint32_t other = __shfl_down_sync(0xffffffffu, sub, 1 << k);
            if (lane + (1 << k) < 32 && other == sub)
                p1_same |= 1u << k;
        }
        const uint32_t prev = __shfl_up_sync(0xffffffffu, sub, 1);
        p1_head = lane == 0 || prev != sub;
    }
    const int64_t p1_rowA_off = rowA;                                     // matrix row of rowA at iteration 0
    float *p1_dstA = nullptr, *p1_dstB = nullptr;
    if (PASS == 1) {
        float *ppart = V.ppart + worker * V.ppart_stride + Lp->pp_off;
        const uint32_t wg = woff >> 8;                                    // warp index within the period
        const uint32_t jA = wg - ((rowA * m) >> 8), jB = wg - (((rowA + 1) * m) >> 8);   // which of the row's warps this is
        p1_dstA = ppart + ((size_t)jA * n_rows + rowA) * R + p1_idx;
        p1_dstB = ppart + ((size_t)jB * n_rows + rowA + 1) * R + p1_idx;
        if (p1_narrow)   // this lane's own row; used by the heads only
            p1_dstA = ppart + ((size_t)(wg - ((sub * m) >> 8)) * n_rows + sub) * R;
    }

    float frag[8][R];   // pass 1: Q_{t-1}[col..col+7][:]; pass 2: accumulators of Q_i[col..col+7][:]; pass 3: Q_i[...]
    if (PASS == 1) {
        const float *qp = V.qprev + Lp->msgq_off;
#pragma unroll
        for (int q = 0; q < 8; ++q)
#pragma unroll
            for (int c = 0; c < R; c += 4) {
                const float4 t = __ldg((const float4 *)(qp + (size_t)(col + q) * R + c));
                frag[q][c] = t.x; frag[q][c + 1] = t.y; frag[q][c + 2] = t.z; frag[q][c + 3] = t.w;
            }
    } else if (PASS == 2) {
#pragma unroll
        for (int q = 0; q < 8; ++q)
#pragma unroll
            for (int c = 0; c < R; ++c)
                frag[q][c] = 0.f;
    } else {
        const float *qi = V.msgq + worker * V.msgq_stride + Lp->msgq_off;
#pragma unroll
        for (int q = 0; q < 8; ++q)
#pragma unroll
            for (int c = 0; c < R; c += 4) {
                const float4 t = __ldg((const float4 *)(qi + (size_t)(col + q) * R + c));
                frag[q][c] = t.x; frag[q][c + 1] = t.y; frag[q][c + 2] = t.z; frag[q][c + 3] = t.w;
            }
    }
    f32x2 frag2[PAIR ? 4 : 1][R];   // PAIR: (Q_i[col + 2k][c], Q_i[col + 2k + 1][c])
    if constexpr (PAIR) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
            for (int c = 0; c < R; ++c)
                frag2[k][c] = pk2(frag[2 * k][c], frag[2 * k + 1][c]);
    }
    const f32x2 lr2 = pk2(V.lr, V.lr);

    const uint8_t *st_scp = st_sc;   // this thread's block scale of iteration it
    const float *st_php = st_ph;     // its row of P_hat of iteration it
    const uint32_t st_sc_step = st_nb * SB, st_ph_step = subs * R * PHW;
    uint32_t it = it0;
    // copies of iteration j into a slot; the source pointers advance in any case
    auto issue = [&](uint32_t j, int slot) {
        if (j < it_mine) {
            cp_async16(ring_lo + slot * bd, gp_iss);
            cp_async16(ring_hi + slot * bd, gp_iss + 4);
            cp_async_small<4 * CW>(ring_cw + slot * bd * CW, cp_iss);
        }
        cp_async_commit();
        gp_iss += P;
        cp_iss += P * CW / 2;
    };
    // NI consecutive iterations at once (their instruction streams interleave): SLOT is the ring
    // slot the first one reads; CHECK is false where every thread of the CTA is known to hold
    // existing elements in all of them
    auto step = [&](auto slot_c, auto check_c) {
        const int SLOT = slot_c;
        constexpr bool CHECK = decltype(check_c)::value != 0;
#pragma unroll
        for (int u = 0; u < NI; ++u)   // refill the slots read one step ago
            issue(it + kRing23 - NI + u, (SLOT + kRing23 - NI + u) % kRing23);
        float sc[NI], phr[NI][R];
        bool valid[NI];
#pragma unroll
        for (int u = 0; u < NI; ++u) {
            sc[u] = HALF ? __half2float(__ushort_as_half(*(const unsigned short *)(st_scp + u * st_sc_step)))
                         : *(const float *)(st_scp + u * st_sc_step);
#pragma unroll
            for (int c = 0; c < (PASS == 1 || PAIR ? 0 : R); c += 4) {
                const float4 t = *(const float4 *)(st_php + u * st_ph_step + c);
                phr[u][c] = t.x; phr[u][c + 1] = t.y; phr[u][c + 2] = t.z; phr[u][c + 3] = t.w;
            }
            valid[u] = !CHECK || it + u < it_mine;
        }
        cp_async_wait<kRing23 - NI>();   // these iterations' copies have landed
        float p[NI][8];
        [[maybe_unused]] float ek[PARTIAL && PASS == 3 ? NI : 1][8];   // the decoded error, kept for the store of Alg. 4
        [[maybe_unused]] f32x2 r2[PAIR ? NI : 1][4];                   // PAIR: the residuals as pairs
        if constexpr (PAIR) {
            constexpr float span = (CK == CONEF_C_INT4) ? 16.f : 256.f;
            constexpr float off = (CK == CONEF_C_INT4) ? 24.f : 384.f;
#pragma unroll
            for (int u = 0; u < NI; ++u) {
                const int sl = (SLOT + u) % kRing23;
                const ulonglong2 ga = *(const ulonglong2 *)(ring_lo + sl * bd);
                const ulonglong2 gb = *(const ulonglong2 *)(ring_hi + sl * bd);
                const f32x2 g2[4] = {ga.x, ga.y, gb.x, gb.y};
                const uint32_t w0 = ring_cw[sl * bd * CW];
                const uint32_t w1 = CW == 2 ? ring_cw[sl * bd * CW + CW - 1] : 0u;
                uint32_t tb[8];
                decode8_bits<CK>(w0, w1, tb);
                const ScaleConst<CK> k = scale_const<CK, HALF>(sc[u]);
                const f32x2 a2 = pk2(k.a, k.a), b2 = HALF ? pk2(k.b, k.b) : pk2(-off, -off);
                f32x2 nph[R];
#pragma unroll
                for (int c = 0; c < R; c += 2) {
                    const ulonglong2 t = *(const ulonglong2 *)(st_php + u * st_ph_step + 2 * c);
                    nph[c] = t.x;
                    nph[c + 1] = t.y;
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const f32x2 f2 = pk2u(tb[2 * kk], tb[2 * kk + 1]);
                    const f32x2 e2 = HALF ? fma2(f2, a2, b2) : mul2(fma2(f2, pk2(span, span), b2), a2);
                    f32x2 acc = fma2(lr2, g2[kk], e2);   // Alg. 2 line 5
                    if (CHECK)
                        acc = valid[u] ? acc : 0ull;     // a slot that was not filled holds stale data
#pragma unroll
                    for (int c = 0; c < R; ++c)
                        acc = fma2(nph[c], frag2[kk][c], acc);   // r = p - P_hat Q_i^T
                    if (CHECK)
                        acc = valid[u] ? acc : 0ull;     // lanes past the end of the tensor add nothing to the block's absmax
                    r2[u][kk] = acc;
                    upk2(acc, p[u][2 * kk], p[u][2 * kk + 1]);
                }
            }
        } else {
#pragma unroll
        for (int u = 0; u < NI; ++u) {
            const int sl = (SLOT + u) % kRing23;
            const float4 g0 = ring_lo[sl * bd];
            const float4 g1 = ring_hi[sl * bd];
            const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            const uint32_t w0 = ring_cw[sl * bd * CW];
            const uint32_t w1 = CW == 2 ? ring_cw[sl * bd * CW + CW - 1] : 0u;
            float e[8];
            decode8<CK, HALF>(w0, w1, scale_const<CK, HALF>(sc[u]), e);
            if (PARTIAL) {
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (PASS == 3)
                        ek[PARTIAL && PASS == 3 ? u : 0][q] = e[q];
                    e[q] = __fmul_rn(omb, e[q]);
                }
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                p[u][q] = __fmaf_rn(lr, gv[q], e[q]);   // Alg. 2 line 5 (Alg. 4 line 5 with beta)
                if (CHECK)
                    p[u][q] = valid[u] ? p[u][q] : 0.f;   // a slot that was not filled holds stale data
            }
        }
        }
        if (PASS == 1) {
            // this thread's share of P_i[row][:]
#pragma unroll
            for (int u = 0; u < NI; ++u) {
                float pr[R];
#pragma unroll
                for (int c = 0; c < R; ++c)
                    pr[c] = 0.f;
#pragma unroll
                for (int q = 0; q < 8; ++q)
#pragma unroll
                    for (int c = 0; c < R; ++c)
                        pr[c] = __fmaf_rn(p[u][q], frag[q][c], pr[c]);
                // sum over the warp's lanes of the same matrix row (a warp's 256 elements lie in one
                // row, or in two when a row ends inside it) and write one partial row per
                // (row, warp); k_fast_p1_combine adds the warps of a row in order
                if constexpr (p1_narrow) {
#pragma unroll
                    for (int k = 0; k < 5; ++k) {
#pragma unroll
                        for (int c = 0; c < R; ++c) {
                            const float o = __shfl_down_sync(0xffffffffu, pr[c], 1 << k);
                            pr[c] = (p1_same >> k) & 1u ? __fadd_rn(pr[c], o) : pr[c];
                        }
                    }
                    if (p1_head && (int64_t)(it + u) * subs + sub < n_rows) {
                        float *dst = p1_dstA + (size_t)(it + u) * subs * R;
#pragma unroll
                        for (int c = 0; c < R; c += 4)
                            *(float4 *)(dst + c) = make_float4(pr[c], pr[c + 1], pr[c + 2], pr[c + 3]);
                    }
                } else {
                    float t0[R];
                    if (p1_straddle) {   // (uniform over the warp) only the lanes of the first row
#pragma unroll
                        for (int c = 0; c < R; ++c)
                            t0[c] = p1_first ? pr[c] : 0.f;
                    } else {
#pragma unroll
                        for (int c = 0; c < R; ++c)
                            t0[c] = pr[c];
                    }
                    warp_reduce_many<R>(t0, lane);
                    if ((lane & (p1_plain - 1)) == 0 && p1_rowA_off + (int64_t)(it + u) * subs < n_rows && p1_idx < R)
                        p1_dstA[(size_t)(it + u) * subs * R] = t0[0];
                    if (p1_straddle) {   // the lanes of the second row
                        float t1[R];
#pragma unroll
                        for (int c = 0; c < R; ++c)
                            t1[c] = p1_first ? 0.f : pr[c];
                        warp_reduce_many<R>(t1, lane);
                        if ((lane & (p1_plain - 1)) == 0 && p1_rowA_off + 1 + (int64_t)(it + u) * subs < n_rows && p1_idx < R)
                            p1_dstB[(size_t)(it + u) * subs * R] = t1[0];
                    }
                }
            }
        } else if (PASS == 2) {
#pragma unroll
            for (int u = 0; u < NI; ++u)   // rows in ascending order
#pragma unroll
                for (int q = 0; q < 8; ++q)
#pragma unroll
                    for (int c = 0; c < R; ++c)
                        frag[q][c] = __fmaf_rn(p[u][q], phr[u][c], frag[q][c]);
        } else {
            float amax[NI];
#pragma unroll
            for (int u = 0; u < NI; ++u) {
                amax[u] = 0.f;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    float acc = p[u][q];
                    if constexpr (!PAIR) {
#pragma unroll
                        for (int c = 0; c < R; ++c)
                            acc = __fmaf_rn(-phr[u][c], frag[q][c], acc);   // r = p - P_hat Q_i^T
                        if (PARTIAL)
                            acc = __fmaf_rn(beta, ek[PARTIAL && PASS == 3 ? u : 0][q], acc);   // what is stored: beta e + r (Alg. 4 line 9)
                        if (CHECK)
                            acc = valid[u] ? acc : 0.f;   // lanes past the end of the tensor add nothing to the block's absmax
                        p[u][q] = acc;
                    }
                    amax[u] = fmaxf(amax[u], fabsf(acc));
                }
            }
            // absmax over the block/8 lanes of the quantisation block
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1)
                if (o <= 2 || lpb > o)
#pragma unroll
                    for (int u = 0; u < NI; ++u)
                        amax[u] = fmaxf(amax[u], __shfl_xor_sync(0xffffffffu, amax[u], o));
            float s[NI], inv[NI];
            unsigned short hb[NI];
            bool clamp = false;
            // |r * inv| <= amax * inv for every element of the block (rounding is monotone), so
            // when that bound rounds to at most qmax no element needs the clamp.  It is needed
            // only where a binary16 scale was rounded down by a lot (subnormal scales).
            constexpr float qlim = (CK == CONEF_C_INT8 ? 127.f : 7.f) + 0.49f;
#pragma unroll
            for (int u = 0; u < NI; ++u) {
                block_scale<CK, HALF>(amax[u], s[u], inv[u], hb[u]);
                clamp = clamp || !(__fmul_rn(amax[u], inv[u]) < qlim);
            }
            uint32_t c0[NI], c1[NI];
            if (__any_sync(0xffffffffu, clamp)) {
#pragma unroll
                for (int u = 0; u < NI; ++u)
                    quant_pack8<CK, true>(p[u], inv[u], c0[u], c1[u]);
            } else if constexpr (PAIR) {
#pragma unroll
                for (int u = 0; u < NI; ++u) {
                    const f32x2 inv2 = pk2(inv[u], inv[u]);
                    uint32_t tq[8];
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        // The multiply packed, the additions scalar: a packed multiply followed by a
                        // packed add of the rounding constant gave codes that differed from the
                        // two-rounding result in about one element in 10^5 (what one fused operation,
                        // which rounds once, would give).
                        float x0, x1;
                        upk2(mul2(r2[u][kk], inv2), x0, x1);
                        tq[2 * kk] = __float_as_uint(__fadd_rn(x0, 12582912.0f));
                        tq[2 * kk + 1] = __float_as_uint(__fadd_rn(x1, 12582912.0f));
                    }
                    pack_fields8<CK>(tq, c0[u], c1[u]);
                }
            } else {
#pragma unroll
                for (int u = 0; u < NI; ++u)
                    quant_pack8<CK, false>(p[u], inv[u], c0[u], c1[u]);
            }
#pragma unroll
            for (int u = 0; u < NI; ++u) {
                if (valid[u]) {
                    if ((lane & (lpb - 1)) == 0) {
                        if (HALF)
                            *(unsigned short *)(sp + u * sp_step) = hb[u];
                        else
                            *(float *)(sp + u * sp_step) = s[u];
                    }
                    if (CK == CONEF_C_INT4)
                        *(uint32_t *)cp_st = c0[u];
                    else
                        *(uint2 *)cp_st = make_uint2(c0[u], c1[u]);
                }
                cp_st += P * CW / 2;
            }
        }
        sp += NI * sp_step;
        st_scp += NI * st_sc_step;
        st_php += NI * st_ph_step;
        it += NI;
    };

#pragma unroll
    for (int s = 0; s < kRing23 - NI; ++s)
        issue(it0 + s, s);
    static_assert(kRing23 % NI == 0 && kRing23 > NI - 1, "steps tile the ring");
    static_assert(kFastStageIt % kRing23 == 0, "chunks end on a ring boundary");
    // iterations [c0, c1) of the tile: their rows of P_hat (contiguous; rows past the matrix read as
    // zero) and their st_nb block scales each (blocks past the tensor read as zero).  A step of NI
    // iterations may reach past c1 at the end of the tile: those iterations are staged as zeros
    // (pass 2 multiplies its zero p by them).
    auto stage = [&](uint32_t c0, uint32_t c1) {
        __syncthreads();   // every thread is done with the previous chunk
        const uint32_t cpad = (c1 - c0 + NI - 1) / NI * NI;
        if (PASS != 1) {
            const uint32_t n4 = (c1 - c0) * subs * (R / 4), n4pad = cpad * subs * (R / 4);
            const int64_t have4 = (n_rows - (int64_t)c0 * subs) * (R / 4);
            const float4 *src = (const float4 *)(V.phat + Lp->msgp_off + (size_t)c0 * subs * R);
            for (uint32_t i = tid; i < n4pad; i += bd) {
                const float4 v = (i < n4 && (int64_t)i < have4) ? __ldg(src + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                if (PAIR) {
                    ((float4 *)st_ph)[2 * i] = make_float4(-v.x, -v.x, -v.y, -v.y);
                    ((float4 *)st_ph)[2 * i + 1] = make_float4(-v.z, -v.z, -v.w, -v.w);
                } else {
                    ((float4 *)st_ph)[i] = v;
                }
            }
        }
        const uint32_t nblk = (d + (uint32_t)Lp->unit - 1) >> unit_shift;
        const uint32_t blk0 = (c0 * P + cg * (uint32_t)Lp->f_cw) >> unit_shift, blk_step = P >> unit_shift;
        const uint8_t *sbase = st + Lp->b_off;   // (plain loads: pass 3 stores new scales to this array, each CTA to the blocks it staged)
        const uint32_t ns = (c1 - c0) * st_nb, nspad = cpad * st_nb;
        for (uint32_t i = tid; i < nspad; i += bd) {
            const uint32_t j = i / st_nb, b = i - j * st_nb;
            const uint32_t blk = blk0 + j * blk_step + b;
            const bool have = i < ns && blk < nblk;
            if (HALF)
                ((unsigned short *)st_sc)[i] = have ? ((const unsigned short *)sbase)[blk] : (unsigned short)0;
            else
                ((float *)st_sc)[i] = have ? ((const float *)sbase)[blk] : 0.f;
        }
        __syncthreads();
        st_scp = st_sc + (((uint32_t)tid * kFastE) >> unit_shift) * SB;
        st_php = st_ph + sub * R * PHW;
    };
    int slot = 0;   // (the loop that is not unrolled over the ring)
    uint32_t cend = it0;
    do {
        const uint32_t c0 = cend;
        cend = min(c0 + (uint32_t)kFastStageIt, it1);
        stage(c0, cend);
        const uint32_t lim = min(it_full, cend);
        if constexpr (ring_unrolled(PASS, R)) {
            // the loop is unrolled over the ring so that every slot index is a constant
            while (it + kRing23 <= lim) {
                static_for<kRing23 / NI>([&](auto i) { step(IntC<decltype(i)::value * NI>(), IntC<0>()); });
            }
        } else {
            static_assert((kRing23 & (kRing23 - 1)) == 0, "slot arithmetic by masking");
            while (it + NI <= lim) {
                step(IntR{slot}, IntC<0>());
                slot = (slot + NI) & (kRing23 - 1);
            }
        }
    } while (it == cend && cend < it1);   // (a chunk left early holds the end of the tensor, and with it the end of the tile)
    if constexpr (ring_unrolled(PASS, R)) {
        // fewer than kRing23 whole iterations and at most one partial one remain
        static_for<kRing23 / NI>([&](auto i) {
            if (it < it1)
                step(IntC<decltype(i)::value * NI>(), IntC<1>());
        });
    } else {
        while (it < it1) {
            step(IntR{slot}, IntC<1>());
            slot = (slot + NI) & (kRing23 - 1);
        }
    }
    if (PASS == 2) {
        // partial sums of this (row tile, sub-row): rows are summed in order by k_lr_pass2_reduce
        float *part = V.part + worker * V.part_stride + Lp->part_off + ((size_t)((size_t)rt * subs + sub) * m + col) * R;
#pragma unroll
        for (int q = 0; q < 8; ++q)
#pragma unroll
            for (int c = 0; c < R; c += 4)
                *(float4 *)(part + q * R + c) = make_float4(frag[q][c], frag[q][c + 1], frag[q][c + 2], frag[q][c + 3]);
    }
}

// P_i[row][c] = sum over the warps that meet the row, in warp order
template <int R>
__global__ void __launch_bounds__(256) k_fast_p1_combine(const __grid_constant__ DevView V, const int32_t *__restrict__ pfx)
{
    const int li = find_layer(pfx, V.n_layers, blockIdx.x);
    const LayerDesc *Lp = V.layers + li;
    const int worker = blockIdx.y;
    const int64_t n = Lp->rows;
    const int64_t q = (int64_t)(blockIdx.x - pfx[li]) * 256 + threadIdx.x;   // (row, c) pair
    if (q >= n * R)
        return;
    const int64_t a = q / R;
    const uint32_t m = (uint32_t)Lp->cols, subs = (uint32_t)Lp->f_subs;
    const uint32_t rr = (uint32_t)(a % subs);
    const uint32_t first = (rr * m) >> 8, last = ((rr + 1) * m - 1) >> 8;   // the warps that meet the row
    const float *ppart = V.ppart + worker * V.ppart_stride + Lp->pp_off;
    float acc = ppart[q];
    for (uint32_t j = 1; j <= last - first; ++j)
        acc = __fadd_rn(acc, ppart[(size_t)j * n * R + q]);
    V.msgp[worker * V.msgp_stride + Lp->msgp_off + q] = acc;
}

// ------------------------------------------------------------------ launch helpers
template <int PASS, int CK, int R, bool HALF, bool SHORT, bool NARROW = false, bool PARTIAL = false>
inline cudaError_t fast_launch_pass23(const DevView &V, const int32_t *pfx, int tiles, int threads, cudaStream_t s,
                                      size_t stage)
{
    const size_t smem = (size_t)ring_depth(PASS, R) * threads * (32 + (CK == CONEF_C_INT4 ? 4 : 8)) + stage;
    static int done[64];
    const cudaError_t e = opt_in_smem(k_fast_pass<PASS, CK, R, HALF, SHORT, NARROW, PARTIAL>, smem, done);
    if (e != cudaSuccess)
        return e;
    dim3 grid(tiles, V.n_workers);
    k_fast_pass<PASS, CK, R, HALF, SHORT, NARROW, PARTIAL><<<grid, threads, smem, s>>>(V, pfx);
    return cudaSuccess;
}

// PASS: 1, 2 or 3.  Returns cudaErrorNotSupported for a configuration that has no tuned kernel.
// short_tiles: the plan's tile lengths are below the limits (small models); narrow: the launch's
// tensors have rows shorter than a warp's 256 elements (pass 1 sums several rows per warp)
inline cudaError_t fast_launch(int pass, int ckind, int rank, int half, const DevView &V, const int32_t *pfx,
                               int tiles, int threads, cudaStream_t s, bool short_tiles, bool narrow, size_t stage)
{
    if (tiles <= 0)
        return cudaSuccess;
#define CONEF_FAST_CASE_P(CKV, RV, HV, PV)                                                                \
    if (ckind == CKV && rank == RV && (half != 0) == HV && (V.beta != 0.f) == PV) {                       \
        if (pass == 1 && narrow) {                                                                        \
            if (short_tiles) return fast_launch_pass23<1, CKV, RV, HV, true, true, PV>(V, pfx, tiles, threads, s, stage);  \
            return fast_launch_pass23<1, CKV, RV, HV, false, true, PV>(V, pfx, tiles, threads, s, stage);        \
        }                                                                                                 \
        if (short_tiles) {                                                                                \
            if (pass == 1) return fast_launch_pass23<1, CKV, RV, HV, true, false, PV>(V, pfx, tiles, threads, s, stage);    \
            if (pass == 2) return fast_launch_pass23<2, CKV, RV, HV, true, false, PV>(V, pfx, tiles, threads, s, stage);    \
            return fast_launch_pass23<3, CKV, RV, HV, true, false, PV>(V, pfx, tiles, threads, s, stage);        \
        }                                                                                                 \
        if (pass == 1) return fast_launch_pass23<1, CKV, RV, HV, false, false, PV>(V, pfx, tiles, threads, s, stage);       \
        if (pass == 2) return fast_launch_pass23<2, CKV, RV, HV, false, false, PV>(V, pfx, tiles, threads, s, stage);       \
        return fast_launch_pass23<3, CKV, RV, HV, false, false, PV>(V, pfx, tiles, threads, s, stage);           \
    }
#define CONEF_FAST_CASE(CKV, RV, HV) CONEF_FAST_CASE_P(CKV, RV, HV, false) CONEF_FAST_CASE_P(CKV, RV, HV, true)
    CONEF_FAST_CASE(CONEF_C_INT4, 4, true)
    CONEF_FAST_CASE(CONEF_C_INT4, 8, true)
    CONEF_FAST_CASE(CONEF_C_INT8, 4, true)
    CONEF_FAST_CASE(CONEF_C_INT8, 8, true)
    CONEF_FAST_CASE(CONEF_C_INT4, 4, false)
    CONEF_FAST_CASE(CONEF_C_INT4, 8, false)
    CONEF_FAST_CASE(CONEF_C_INT8, 4, false)
    CONEF_FAST_CASE(CONEF_C_INT8, 8, false)
#undef CONEF_FAST_CASE
#undef CONEF_FAST_CASE_P
    return cudaErrorNotSupported;
}

inline cudaError_t fast_launch_p1_combine(int rank, const DevView &V, const int32_t *pfx, int tiles, cudaStream_t s)
{
    if (tiles <= 0)
        return cudaSuccess;
    dim3 grid(tiles, V.n_workers);
    if (rank == 4)
        k_fast_p1_combine<4><<<grid, 256, 0, s>>>(V, pfx);
    else
        k_fast_p1_combine<8><<<grid, 256, 0, s>>>(V, pfx);
    return cudaSuccess;
}

}  // namespace conef
