// Low-rank passes 2 and 3 in one persistent kernel that keeps p on the chip (Sec. 5.2:
// Q_i = M_i^T P_hat, Delta_i = P_hat Q_i^T; Alg. 2 line 9: state = C(p - Delta_i), with
// M_i = eta G + decode(e) formed on the fly, Alg. 2 line 5).
//
// The residual needs all of Q_i, and Q_i is a sum over all rows of the tensor, so the tensor has
// to be walked twice.  Two separate kernels read the gradient and the codes twice from HBM and
// decode them twice.  Here a (worker, tensor) unit is given to a gang of CTAs; in phase A every
// warp streams its share of the unit through shared memory by bulk asynchronous copies (TMA,
// one mbarrier per slot), forms p, adds its columns' share of Q_i and writes p back over the
// gradient in the slot it arrived in; the gang then meets at a barrier in global memory, sums the
// per-CTA partial Q_i in a fixed order, meets again, and in phase B every warp turns the p it
// kept into the residual, block maxima, codes and scales.  What does not fit into a warp's slots
// is streamed a second time in phase B through a small ring of slots (it was read last in phase A,
// so most of it is still in L2).  Several gangs are resident at once (two CTAs per SM, from
// different gangs), so that one gang's barrier and its compute-only phase B overlap the other
// gang's streaming phase A.
//
// Tiling: with the period L = lcm(cols, 256) a warp-iteration covers segment cg (256 consecutive
// elements) of one period; a lane owns elements 4 lane .. 4 lane + 3 and 128 + 4 lane .. + 3 of
// it (two conflict-free 16-byte shared-memory accesses; a quantisation block of 128 elements is
// one 16-byte piece of every lane, so its maximum is one warp reduction), hence the same 8 columns
// in every period.  A CTA owns a contiguous range of (segment, period) pairs, segment-major, split
// evenly over the gang; its 8 warps take the periods of a segment round-robin and add their
// partial Q_i through shared memory in warp order, so the result does not depend on timing.
//
// CUDA-core fp32 on purpose: 2 r flop per element is far left of the tensor-core ridge and the
// residual chain has to be reproducible bit for bit.
#include <cuda_runtime.h>

#include <algorithm>

#include "conef_codec.cuh"

namespace conef {

namespace {

constexpr int kFuWarps = kFuWarpsPerCta;
constexpr int kFuThreads = kFuWarps * 32;
constexpr uint32_t kFuMbarTries = 1u << 20;   // bounded waits: a kernel that gives up sets ST_FUSED_TIMEOUT and returns
constexpr uint32_t kFuGangPolls = 1u << 21;

__device__ __forceinline__ uint32_t fu_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t tx)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(tx) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// global -> shared bulk copy (no multicast; the CTA is its own cluster), completion counted on `bar`
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// e_j = float(code_j) * scale for the 4 codes of one 16-byte piece (see decode8)
template <int CK, bool HALF>
__device__ __forceinline__ void decode4(uint32_t w, const ScaleConst<CK> &k, float *e)
{
    constexpr float span = (CK == CONEF_C_INT4) ? 16.f : 256.f;
    constexpr float off = (CK == CONEF_C_INT4) ? 24.f : 384.f;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint32_t t;
        if (CK == CONEF_C_INT4) {
            t = ((w << (19 - 4 * q)) & 0x00780000u) ^ 0x3FC00000u;
        } else {
            const uint32_t sh = q == 0 ? (w << 15) : q == 1 ? (w << 7) : q == 2 ? (w >> 1) : (w >> 9);
            t = (sh & 0x007F8000u) ^ 0x3FC00000u;
        }
        const float f = __uint_as_float(t);
        e[q] = HALF ? __fmaf_rn(f, k.a, k.b) : __fmul_rn(__fmaf_rn(f, span, -off), k.a);
    }
}

// two's complement codes of 4 residuals: 16 bits (int4) or 32 bits (int8); see quant_pack8
template <int CK, bool CLAMP>
__device__ __forceinline__ uint32_t quant_pack4(const float *r, float inv)
{
    constexpr float qm = (CK == CONEF_C_INT4) ? 7.f : 127.f;
    uint32_t t[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        float x = __fmul_rn(r[q], inv);
        if (CLAMP)
            x = fminf(fmaxf(x, -qm), qm);
        t[q] = __float_as_uint(__fadd_rn(x, 12582912.0f));
    }
    if (CK == CONEF_C_INT4) {
        uint32_t acc = t[3];
#pragma unroll
        for (int q = 2; q >= 0; --q)
            acc = (acc << 4) + t[q];
        // the patterns' constant part 0x4B400000 has no bits in the low half-word
        return ((acc + 0x8888u) ^ 0x8888u) & 0xFFFFu;
    }
    uint32_t acc = t[3];
#pragma unroll
    for (int q = 2; q >= 0; --q)
        acc = (acc << 8) + t[q];
    constexpr uint32_t K = 0x4B400000u * 0x01010101u;
    return (acc - K + 0x80808080u) ^ 0x80808080u;
}

template <int R, int CK, bool HALF>
struct FuLayout {
    static constexpr int UNIT = (CK == CONEF_C_INT4) ? 128 : 256;   // quantisation block
    static constexpr int NBLK = 256 / UNIT;                         // blocks per warp-iteration
    static constexpr int SB = HALF ? 2 : 4;                         // bytes per scale
    static constexpr int CB = (CK == CONEF_C_INT4) ? 128 : 256;     // code bytes per warp-iteration
    static constexpr int OFF_C = 1024;                              // slot: gradient / p, codes,
    static constexpr int OFF_S = OFF_C + CB;                        // a 16-byte window of the scales,
    static constexpr int OFF_P = OFF_S + 16;                        // the (at most two) rows of P_hat
    static constexpr int SLOT = OFF_P + 2 * R * 4;
};

template <int R, int CK, bool HALF>
__global__ void __launch_bounds__(kFuThreads, 2) k_fused23(const __grid_constant__ FusedParams P)
{
    using Lay = FuLayout<R, CK, HALF>;
    constexpr int UNIT = Lay::UNIT, NBLK = Lay::NBLK, SB = Lay::SB, SLOT = Lay::SLOT;
    constexpr int OFF_C = Lay::OFF_C, OFF_S = Lay::OFF_S, OFF_P = Lay::OFF_P;
    constexpr int USH = (UNIT == 128) ? 7 : 8;
    constexpr float qlim = (CK == CONEF_C_INT8 ? 127.f : 7.f) + 0.49f;
    extern __shared__ __align__(128) uint8_t fu_smem[];
    __shared__ int s_abort;
    const DevView &V = P.V;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int NS = P.n_slots, G = P.gang_size;
    const int gang = blockIdx.x / G, cta = blockIdx.x - gang * G;
    uint8_t *wslots = fu_smem + (size_t)warp * NS * SLOT;
    float *qacc = (float *)(fu_smem + (size_t)kFuWarps * NS * SLOT);   // 256 x R floats
    uint64_t *bars = (uint64_t *)(qacc + 256 * R) + warp * NS;
    const uint32_t slots_u32 = fu_smem_u32(wslots), bars_u32 = fu_smem_u32(bars);
    uint32_t *gctr = P.gang_ctr + gang * 32;   // one counter per 128 bytes
    float *partial = P.partial + (size_t)gang * P.partial_gang_stride;
    const int KMAX = P.kmax;
    const float lr = V.lr;

    if (tid == 0)
        s_abort = 0;
    if (lane == 0)
        for (int s = 0; s < NS; ++s)
            mbar_init(bars_u32 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
    __syncthreads();

    uint32_t par = 0;    // bit s: parity of the phase slot s completes next
    uint32_t pend = 0;   // bit s: copies into slot s are in flight
    uint32_t epoch = 0;  // value of the gang counter after the last barrier
    auto aborted = [&]() { return *(volatile int *)&s_abort != 0; };
    auto give_up = [&]() {
        s_abort = 1;
        atomicOr(V.status, ST_FUSED_TIMEOUT);
    };
    auto wait_slot = [&](int slot) {
        const uint32_t bar = bars_u32 + 8 * slot, ph = (par >> slot) & 1u;
        uint32_t tries = 0;
        while (!mbar_try_wait(bar, ph)) {
            if (++tries > kFuMbarTries) {
                give_up();
                return false;
            }
        }
        par ^= 1u << slot;
        pend &= ~(1u << slot);
        return true;
    };
    // all CTAs of the gang have arrived; their global writes before it are visible after it
    auto gang_sync = [&]() {
        epoch += (uint32_t)G;
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            atomicAdd(gctr, 1u);
            uint32_t polls = 0;
            while (ld_acquire_u32(gctr) < epoch) {
                ++polls;
                if (polls > kFuGangPolls || ((polls & 63u) == 0 && (*(volatile int *)V.status & ST_FUSED_TIMEOUT))) {
                    give_up();
                    break;
                }
                __nanosleep(40);
            }
            __threadfence();
        }
        __syncthreads();
    };

    for (int ui = 0;; ++ui) {
        const int2 un = P.sched[(size_t)gang * P.sched_pitch + ui];
        if (un.x < 0)
            break;
        const LayerDesc &L = V.layers[un.x];
        const int worker = un.y;
        const uint32_t m = (uint32_t)L.cols, d = (uint32_t)L.d, n = (uint32_t)L.rows, Lp = (uint32_t)L.f_lcm;
        const uint32_t subs = (uint32_t)L.f_subs, niter = (uint32_t)L.f_niter, ncg = Lp >> 8;
        const uint32_t T = ncg * niter, chunk = (T + G - 1) / G;
        const uint32_t lo = min(T, (uint32_t)cta * chunk), hi = min(T, lo + chunk);
        const uint32_t cg0 = lo / niter;
        const int K = hi > lo ? (int)((hi - 1) / niter - cg0) + 1 : 0;
        const float *gp = V.grads[worker] + L.g_off;
        uint8_t *st = V.state + worker * V.state_stride;
        uint8_t *codes = st + L.a_off, *scales = st + L.b_off;
        const float *phat = V.phat + L.msgp_off;
        float *q_out = P.q_out + worker * P.q_out_stride + L.msgq_off;
        const float *q_res = P.q_res + worker * P.q_res_stride + L.msgq_off;

        auto sub_p0 = [&](int k) { return k == 0 ? lo - cg0 * niter : 0u; };
        auto sub_p1 = [&](int k) { return min(niter, hi - (cg0 + (uint32_t)k) * niter); };
        // this warp's iterations: sub-range k = 0 .. K-1 (one segment each), periods p0 + warp, p0 + warp + 8, ...
        auto cur_fix = [&](int &k, uint32_t &p) {
            while (k < K && p >= sub_p1(k)) {
                ++k;
                p = (uint32_t)warp;   // sub_p0(k) == 0 for k > 0
            }
        };
        uint32_t nw = 0;
        for (int k = 0; k < K; ++k) {
            const uint32_t a = sub_p0(k) + warp, b = sub_p1(k);
            nw += b > a ? (b - a + 7) >> 3 : 0u;
        }
        const uint32_t nres = nw <= (uint32_t)NS ? nw : (uint32_t)(NS - P.n_ring);   // iterations whose p stays
        const uint32_t ring = (uint32_t)NS - nres;                                    // slots the rest cycles through
        auto slot_of = [&](uint32_t j) { return j < nres ? (int)j : (int)(nres + (j - nres) % ring); };

        // copies of iteration (k, p) into `slot`: gradient, codes, scale window, rows of P_hat
        auto issue = [&](int k, uint32_t p, int slot) {
            const uint32_t cg = cg0 + (uint32_t)k;
            const uint32_t e0w = p * Lp + (cg << 8);
            const uint32_t nv = e0w < d ? min(256u, d - e0w) : 0u;
            const uint32_t subf = (cg << 8) / m, subl = ((cg << 8) + 255u) / m;
            const uint32_t row0 = p * subs + subf;
            const uint32_t nrows = nv ? min(subl - subf + 1u, n - row0) : 0u;
            const uint32_t gb = nv * 4u, cb = CK == CONEF_C_INT4 ? nv >> 1 : nv, sb = nv ? 16u : 0u, pb = nrows * (R * 4u);
            const uint32_t dst = slots_u32 + (uint32_t)slot * SLOT, bar = bars_u32 + 8u * (uint32_t)slot;
            if (lane == 0)
                mbar_expect_tx(bar, gb + cb + sb + pb);
            __syncwarp();
            const void *src = lane == 0   ? (const void *)(gp + e0w)
                              : lane == 1 ? (const void *)(codes + (CK == CONEF_C_INT4 ? e0w >> 1 : e0w))
                              : lane == 2 ? (const void *)(scales + (((e0w >> USH) * SB) & ~15u))
                                          : (const void *)(phat + (size_t)row0 * R);
            const uint32_t dd = dst + (lane == 0 ? 0u : lane == 1 ? (uint32_t)OFF_C : lane == 2 ? (uint32_t)OFF_S : (uint32_t)OFF_P);
            const uint32_t nb = lane == 0 ? gb : lane == 1 ? cb : lane == 2 ? sb : pb;
            if (lane < 4 && nb)
                bulk_g2s(dd, src, nb, bar);
            pend |= 1u << slot;
        };

        // per sub-range: where this lane's two pieces sit
        uint32_t col[2], rsel[2];
        auto set_subrange = [&](int k) {
            const uint32_t cg = cg0 + (uint32_t)k, subf = (cg << 8) / m;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                const uint32_t off = (cg << 8) + 128u * x + 4u * lane, sub = off / m;
                col[x] = off - sub * m;
                rsel[x] = sub - subf;
            }
        };
        // p (Alg. 2 line 5) of this lane's 8 elements of the iteration in `sl`, from gradient and codes
        auto form_p = [&](const uint8_t *sl, uint32_t e0w, float *p) {
            const float4 g0 = *(const float4 *)(sl + lane * 16), g1 = *(const float4 *)(sl + 512 + lane * 16);
            const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            const uint32_t soff = ((e0w >> USH) * SB) & 15u;
            float sc[2];
            if (NBLK == 2) {
                if (HALF) {
                    const uint32_t sw = *(const uint32_t *)(sl + OFF_S + soff);
                    sc[0] = __half2float(__ushort_as_half((unsigned short)(sw & 0xFFFFu)));
                    sc[1] = __half2float(__ushort_as_half((unsigned short)(sw >> 16)));
                } else {
                    const float2 sw = *(const float2 *)(sl + OFF_S + soff);
                    sc[0] = sw.x;
                    sc[1] = sw.y;
                }
            } else {
                sc[0] = HALF ? __half2float(__ushort_as_half(*(const unsigned short *)(sl + OFF_S + soff)))
                             : *(const float *)(sl + OFF_S + soff);
                sc[1] = sc[0];
            }
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                const uint32_t w = CK == CONEF_C_INT4 ? (uint32_t) * (const unsigned short *)(sl + OFF_C + 64 * x + lane * 2)
                                                      : *(const uint32_t *)(sl + OFF_C + 128 * x + lane * 4);
                float e[4];
                decode4<CK, HALF>(w, scale_const<CK, HALF>(sc[x]), e);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    p[4 * x + q] = __fmaf_rn(lr, gv[4 * x + q], e[q]);
            }
        };
        auto load_ph = [&](const uint8_t *sl, float (*ph)[R]) {
#pragma unroll
            for (int x = 0; x < 2; ++x)
#pragma unroll
                for (int c = 0; c < R; c += 4) {
                    const float4 t = *(const float4 *)(sl + OFF_P + rsel[x] * (R * 4) + c * 4);
                    ph[x][c] = t.x; ph[x][c + 1] = t.y; ph[x][c + 2] = t.z; ph[x][c + 3] = t.w;
                }
        };

        // ------------------------------------------------------------------ phase A
        int ik = 0;
        uint32_t ip = sub_p0(0) + warp, ij = 0;   // issue cursor
        cur_fix(ik, ip);
        int bk = 0;
        uint32_t bp = 0;                           // issue cursor at the first iteration that is streamed again in phase B
        if (!aborted()) {
            __syncwarp();
            fence_proxy_async();   // the slots were read and written through the generic proxy in the last unit
            while (ij < nw && ij < (uint32_t)NS) {
                if (ij == nres) {
                    bk = ik;
                    bp = ip;
                }
                issue(ik, ip, slot_of(ij));
                ++ij;
                ip += 8;
                cur_fix(ik, ip);
            }
            if (ij == nres) {
                bk = ik;
                bp = ip;
            }
        }
        uint32_t j = 0;   // iterations consumed
        for (int k = 0; k < K; ++k) {
            float frag[8][R];
#pragma unroll
            for (int q = 0; q < 8; ++q)
#pragma unroll
                for (int c = 0; c < R; ++c)
                    frag[q][c] = 0.f;
            set_subrange(k);
            const uint32_t cgoff = (cg0 + (uint32_t)k) << 8;
            for (uint32_t p_ = sub_p0(k) + warp; p_ < sub_p1(k); p_ += 8, ++j) {
                if (aborted())
                    break;
                const int slot = slot_of(j);
                if (!wait_slot(slot))
                    break;
                uint8_t *sl = wslots + (size_t)slot * SLOT;
                const uint32_t e0w = p_ * Lp + cgoff;
                float p[8], ph[2][R];
                form_p(sl, e0w, p);
                load_ph(sl, ph);
                if (e0w + 256u > d) {   // the last period: lanes past the end hold stale data
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        const bool ok = e0w + 128u * x + 4u * lane < d;
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            p[4 * x + q] = ok ? p[4 * x + q] : 0.f;
#pragma unroll
                        for (int c = 0; c < R; ++c)
                            ph[x][c] = ok ? ph[x][c] : 0.f;
                    }
                }
                if (j < nres) {   // p stays in the slot for phase B
                    *(float4 *)(sl + lane * 16) = make_float4(p[0], p[1], p[2], p[3]);
                    *(float4 *)(sl + 512 + lane * 16) = make_float4(p[4], p[5], p[6], p[7]);
                } else if (j + ring < nw) {   // the slot is free: fetch the iteration that takes it next
                    __syncwarp();
                    fence_proxy_async();
                    issue(ik, ip, slot);
                    ++ij;
                    ip += 8;
                    cur_fix(ik, ip);
                }
#pragma unroll
                for (int x = 0; x < 2; ++x)
#pragma unroll
                    for (int q = 0; q < 4; ++q)
#pragma unroll
                        for (int c = 0; c < R; ++c)
                            frag[4 * x + q][c] = __fmaf_rn(p[4 * x + q], ph[x][c], frag[4 * x + q][c]);
            }
            // the 8 warps' sums, added in warp order; the CTA's partial of this segment
            for (int w = 0; w < kFuWarps; ++w) {
                if (warp == w) {
#pragma unroll
                    for (int x = 0; x < 2; ++x)
#pragma unroll
                        for (int q = 0; q < 4; ++q)
#pragma unroll
                            for (int c = 0; c < R; c += 4) {
                                float4 *dst = (float4 *)(qacc + (size_t)(128 * x + 4 * lane + q) * R + c);
                                float4 a = make_float4(frag[4 * x + q][c], frag[4 * x + q][c + 1], frag[4 * x + q][c + 2],
                                                       frag[4 * x + q][c + 3]);
                                if (w > 0) {
                                    const float4 o = *dst;
                                    a.x = __fadd_rn(o.x, a.x); a.y = __fadd_rn(o.y, a.y);
                                    a.z = __fadd_rn(o.z, a.z); a.w = __fadd_rn(o.w, a.w);
                                }
                                *dst = a;
                            }
                }
                __syncthreads();
            }
            {
                float4 *dst = (float4 *)(partial + ((size_t)cta * KMAX + k) * 256 * R);
                for (int x = tid; x < 256 * R / 4; x += kFuThreads)
                    dst[x] = ((const float4 *)qacc)[x];
            }
            __syncthreads();
        }
        gang_sync();
        // ------------------------------------------------------------------ Q_i = sum of the partials, in a fixed order
        if (!aborted()) {
            const uint32_t items = m * (R / 4);
            for (uint32_t i = (uint32_t)cta * kFuThreads + tid; i < items; i += (uint32_t)G * kFuThreads) {
                const uint32_t c = i / (R / 4), h = i - c * (R / 4);
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (uint32_t s = 0; s < subs; ++s) {
                    const uint32_t pos = s * m + c, cgp = pos >> 8, off = pos & 255u;
                    const uint32_t a = cgp * niter, cf = a / chunk, cl = (a + niter - 1) / chunk;
                    for (uint32_t cc = cf; cc <= cl; ++cc) {
                        const uint32_t kk = cgp - (cc * chunk) / niter;
                        const float4 v = __ldcg((const float4 *)(partial + (((size_t)cc * KMAX + kk) * 256 + off) * R) + h);
                        acc.x = __fadd_rn(acc.x, v.x); acc.y = __fadd_rn(acc.y, v.y);
                        acc.z = __fadd_rn(acc.z, v.z); acc.w = __fadd_rn(acc.w, v.w);
                    }
                }
                *((float4 *)(q_out + (size_t)c * R) + h) = acc;
            }
        }
        gang_sync();
        // ------------------------------------------------------------------ phase B
        ik = bk;
        ip = bp;
        ij = nres;
        if (!aborted()) {
            __syncwarp();
            fence_proxy_async();
            while (ij < nw && ij < nres + ring) {
                issue(ik, ip, slot_of(ij));
                ++ij;
                ip += 8;
                cur_fix(ik, ip);
            }
        }
        j = 0;
        for (int k = 0; k < K; ++k) {
            if (aborted())
                break;
            set_subrange(k);
            float frag[8][R];   // Q_i of this lane's columns
#pragma unroll
            for (int x = 0; x < 2; ++x)
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int c = 0; c < R; c += 4) {
                        const float4 t = __ldcg((const float4 *)(q_res + (size_t)(col[x] + q) * R + c));
                        frag[4 * x + q][c] = t.x; frag[4 * x + q][c + 1] = t.y;
                        frag[4 * x + q][c + 2] = t.z; frag[4 * x + q][c + 3] = t.w;
                    }
            const uint32_t cgoff = (cg0 + (uint32_t)k) << 8;
            for (uint32_t p_ = sub_p0(k) + warp; p_ < sub_p1(k); p_ += 8, ++j) {
                if (aborted())
                    break;
                const int slot = slot_of(j);
                uint8_t *sl = wslots + (size_t)slot * SLOT;
                const uint32_t e0w = p_ * Lp + cgoff;
                float p[8], ph[2][R];
                if (j < nres) {
                    const float4 a = *(const float4 *)(sl + lane * 16), b = *(const float4 *)(sl + 512 + lane * 16);
                    p[0] = a.x; p[1] = a.y; p[2] = a.z; p[3] = a.w;
                    p[4] = b.x; p[5] = b.y; p[6] = b.z; p[7] = b.w;
                    load_ph(sl, ph);
                } else {
                    if (!wait_slot(slot))
                        break;
                    form_p(sl, e0w, p);
                    load_ph(sl, ph);
                    if (j + ring < nw) {
                        __syncwarp();
                        fence_proxy_async();
                        issue(ik, ip, slot);
                        ++ij;
                        ip += 8;
                        cur_fix(ik, ip);
                    }
                }
                const bool tail = e0w + 256u > d;
                bool ok[2] = {true, true};
                if (tail) {
                    ok[0] = e0w + 4u * lane < d;
                    ok[1] = e0w + 128u + 4u * lane < d;
                }
                float am[2];
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    am[x] = 0.f;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float acc = p[4 * x + q];
#pragma unroll
                        for (int c = 0; c < R; ++c)
                            acc = __fmaf_rn(-ph[x][c], frag[4 * x + q][c], acc);   // r = p - P_hat Q_i^T (Alg. 2 line 9)
                        if (tail)
                            acc = ok[x] ? acc : 0.f;
                        p[4 * x + q] = acc;
                        am[x] = fmaxf(am[x], fabsf(acc));
                    }
                }
                // block maxima: bit patterns of non-negative floats order like integers
                float bm[2];
                if (NBLK == 2) {
                    bm[0] = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(am[0])));
                    bm[1] = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(am[1])));
                } else {
                    bm[0] = bm[1] = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(fmaxf(am[0], am[1]))));
                }
                float s[2], inv[2];
                unsigned short hb[2];
                bool clamp = false;
#pragma unroll
                for (int x = 0; x < NBLK; ++x) {
                    block_scale<CK, HALF>(bm[x], s[x], inv[x], hb[x]);
                    clamp = clamp || !(__fmul_rn(bm[x], inv[x]) < qlim);
                }
                if (NBLK == 1) {
                    s[1] = s[0];
                    inv[1] = inv[0];
                    hb[1] = hb[0];
                }
                uint32_t cw[2];
                if (clamp) {   // (the same for every lane: the maxima are the warp's)
                    cw[0] = quant_pack4<CK, true>(p, inv[0]);
                    cw[1] = quant_pack4<CK, true>(p + 4, inv[1]);
                } else {
                    cw[0] = quant_pack4<CK, false>(p, inv[0]);
                    cw[1] = quant_pack4<CK, false>(p + 4, inv[1]);
                }
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    const uint32_t e = e0w + 128u * x + 4u * lane;
                    if (ok[x]) {
                        if (CK == CONEF_C_INT4)
                            *(unsigned short *)(codes + (e >> 1)) = (unsigned short)cw[x];
                        else
                            *(uint32_t *)(codes + e) = cw[x];
                    }
                }
                if (lane == 0) {
#pragma unroll
                    for (int x = 0; x < NBLK; ++x)
                        if (e0w + (uint32_t)UNIT * x < d) {
                            if (HALF)
                                *(unsigned short *)(scales + (size_t)((e0w >> USH) + x) * 2) = hb[x];
                            else
                                *(float *)(scales + (size_t)((e0w >> USH) + x) * 4) = s[x];
                        }
                }
            }
        }
        __syncthreads();
        if (aborted())
            break;
    }
    // copies still in flight (only after a wait gave up) must land before the CTA's memory goes away
    for (int s = 0; s < NS; ++s)
        if ((pend >> s) & 1u) {
            const uint32_t bar = bars_u32 + 8 * s, ph = (par >> s) & 1u;
            for (uint32_t t = 0; t < kFuMbarTries && !mbar_try_wait(bar, ph); ++t) {
            }
        }
}

template <int R, int CK, bool HALF>
cudaError_t fused_config_t(int n_sms, FusedConfig *out)
{
    using Lay = FuLayout<R, CK, HALF>;
    int dev = 0, max_smem = 0, max_sm = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess)
        return e;
    if ((e = cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess)
        return e;
    if ((e = cudaDeviceGetAttribute(&max_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev)) != cudaSuccess)
        return e;
    const int fixed = 256 * R * 4 + 128;   // partial Q_i, alignment slack
    // two CTAs per SM (1 KB of each SM's shared memory is reserved per CTA)
    const int per_cta = std::min(max_smem, max_sm / 2 - 1024);
    int ns = (per_cta - fixed) / (kFuWarps * (Lay::SLOT + 8));
    ns = std::min(ns, 32);
    if (ns < 6)
        return cudaErrorInvalidConfiguration;
    out->n_slots = ns;
    out->n_ring = 4;
    out->smem = (size_t)kFuWarps * ns * (Lay::SLOT + 8) + fixed;
    out->threads = kFuThreads;
    out->slot_elems = 256;
    if ((e = cudaFuncSetAttribute(k_fused23<R, CK, HALF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)out->smem)) !=
        cudaSuccess)
        return e;
    int occ = 0;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_fused23<R, CK, HALF>, kFuThreads, out->smem)) != cudaSuccess)
        return e;
    if (occ < 1)
        return cudaErrorInvalidConfiguration;
    out->ctas = std::min(occ, 2) * n_sms;
    return cudaSuccess;
}

template <int R, int CK, bool HALF>
cudaError_t fused_launch_t(const FusedParams &P, int n_ctas, size_t smem, cudaStream_t s)
{
    void *args[] = {(void *)&P};
    return cudaLaunchCooperativeKernel((const void *)k_fused23<R, CK, HALF>, dim3(n_ctas), dim3(kFuThreads), args, smem, s);
}

}  // namespace

#define CONEF_FUSED_DISPATCH(FN, ...)                                                                  \
    if (ckind == CONEF_C_INT4 && rank == 4 && half) return FN<4, CONEF_C_INT4, true>(__VA_ARGS__);     \
    if (ckind == CONEF_C_INT4 && rank == 8 && half) return FN<8, CONEF_C_INT4, true>(__VA_ARGS__);     \
    if (ckind == CONEF_C_INT4 && rank == 4 && !half) return FN<4, CONEF_C_INT4, false>(__VA_ARGS__);   \
    if (ckind == CONEF_C_INT4 && rank == 8 && !half) return FN<8, CONEF_C_INT4, false>(__VA_ARGS__);   \
    if (ckind == CONEF_C_INT8 && rank == 4 && half) return FN<4, CONEF_C_INT8, true>(__VA_ARGS__);     \
    if (ckind == CONEF_C_INT8 && rank == 8 && half) return FN<8, CONEF_C_INT8, true>(__VA_ARGS__);     \
    if (ckind == CONEF_C_INT8 && rank == 4 && !half) return FN<4, CONEF_C_INT8, false>(__VA_ARGS__);   \
    if (ckind == CONEF_C_INT8 && rank == 8 && !half) return FN<8, CONEF_C_INT8, false>(__VA_ARGS__);   \
    return cudaErrorNotSupported;

cudaError_t fused_config(int ckind, int rank, int half, int n_sms, FusedConfig *out)
{
    CONEF_FUSED_DISPATCH(fused_config_t, n_sms, out)
}

cudaError_t fused_launch(int ckind, int rank, int half, const FusedParams &P, int n_ctas, size_t smem, cudaStream_t s)
{
    CONEF_FUSED_DISPATCH(fused_launch_t, P, n_ctas, smem, s)
}

}  // namespace conef
