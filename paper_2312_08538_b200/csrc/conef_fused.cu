// Low-rank passes 2 and 3 in one persistent kernel (Sec. 5.2: Q_i = M_i^T P_hat,
// Delta_i = P_hat Q_i^T; Alg. 2 line 9: state = C(p - Delta_i), with M_i = eta G + decode(e)
// formed on the fly, Alg. 2 line 5).
//
// The residual needs all of Q_i, and Q_i is a sum over all rows of the tensor, so the tensor has
// to be walked twice.  As two grids over the whole model the second walk finds nothing of the
// first in L2.  Here both walks are cut into tiles (one 256-element segment of the period, a run
// of periods) and all tiles of the step form ONE list of tasks that resident CTAs take in order
// from a counter: the Q_i tiles of a (worker, tensor) unit, then, about one wave of tasks later,
// its residual tiles, interleaved with the Q_i tiles of the units that follow.  A residual tile
// therefore reads a gradient and codes that crossed L2 a moment ago.  No barrier over CTAs: a
// Q_i tile writes its partial sums, counts itself in, and the tile that arrives last at a
// segment adds that segment's partials in tile order; the segment that finishes last adds the
// segments that share columns (a period may hold several rows) and raises the unit's flag, on
// which the unit's residual tiles wait (bounded; by the order of the list the flag is almost
// always up before they look).  Sums are taken in a fixed order whoever does them, so results
// do not depend on timing.
//
// Tiling: with the period L = lcm(cols, 256) a warp-iteration covers segment cg (256 consecutive
// elements) of one period; a lane owns elements 4 lane .. 4 lane + 3 and 128 + 4 lane .. + 3 of
// it (two conflict-free 16-byte shared-memory accesses; a quantisation block of 128 elements is
// one 16-byte piece of every lane, so its maximum is one warp reduction), hence the same 8 columns
// in every period.  The 8 warps of a CTA take the periods of a tile round-robin; each streams its
// iterations through a private ring of shared-memory slots filled by bulk asynchronous copies
// (TMA, one mbarrier per slot: gradient, codes, a window of the scales, the rows of P_hat).
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
constexpr uint32_t kFuFlagPolls = 1u << 21;

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
// global -> shared bulk copy (one destination CTA: the CTA is its own cluster), completion counted on `bar`
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

template <int N>
struct IntC {
    static constexpr int value = N;
};

template <int R, int CK, bool HALF>
struct FuLayout {
    static constexpr int UNIT = (CK == CONEF_C_INT4) ? 128 : 256;   // quantisation block
    static constexpr int NBLK = 256 / UNIT;                         // blocks per warp-iteration
    static constexpr int SB = HALF ? 2 : 4;                         // bytes per scale
    static constexpr int CB = (CK == CONEF_C_INT4) ? 128 : 256;     // code bytes per warp-iteration
    static constexpr int OFF_C = 1024;                              // slot: gradient, codes
    static constexpr int SLOT = OFF_C + CB;
};

// a value the compiler can keep in a uniform register: the same in every lane by construction
__device__ __forceinline__ uint32_t uni(uint32_t v) { return __shfl_sync(0xffffffffu, v, 0); }
__device__ __forceinline__ int uni(int v) { return __shfl_sync(0xffffffffu, v, 0); }
__device__ __forceinline__ int64_t uni(int64_t v) { return (int64_t)__shfl_sync(0xffffffffu, (long long)v, 0); }
__device__ __forceinline__ uint32_t elect_one()
{
    uint32_t pred;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "elect.sync _|p, 0xffffffff;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(pred));
    return pred;
}

// the block scales of one warp-iteration as they sit in memory: two binary16 (one word), two
// floats, or one of either
template <int NBLK, bool HALF>
struct ScaleWord {
    uint32_t a, b;
};
template <int NBLK, bool HALF>
__device__ __forceinline__ ScaleWord<NBLK, HALF> load_scales(const uint8_t *p)
{
    ScaleWord<NBLK, HALF> w;
    w.b = 0;
    if (NBLK == 2 && HALF)
        w.a = __ldg((const uint32_t *)p);
    else if (NBLK == 2) {
        const uint2 t = __ldg((const uint2 *)p);
        w.a = t.x;
        w.b = t.y;
    } else if (HALF)
        w.a = __ldg((const unsigned short *)p);
    else
        w.a = __ldg((const uint32_t *)p);
    return w;
}
template <int NBLK, bool HALF>
__device__ __forceinline__ void scales_of(const ScaleWord<NBLK, HALF> &w, float (&sc)[2])
{
    if (NBLK == 2 && HALF) {
        sc[0] = __half2float(__ushort_as_half((unsigned short)(w.a & 0xFFFFu)));
        sc[1] = __half2float(__ushort_as_half((unsigned short)(w.a >> 16)));
    } else if (NBLK == 2) {
        sc[0] = __uint_as_float(w.a);
        sc[1] = __uint_as_float(w.b);
    } else {
        sc[0] = HALF ? __half2float(__ushort_as_half((unsigned short)w.a)) : __uint_as_float(w.a);
        sc[1] = sc[0];
    }
}

// What one lane holds of one warp-iteration: p (Alg. 2 line 5) of its 8 elements, formed from the
// gradient and the codes in the slot and the scales, and the rows of P_hat its two pieces lie in.
template <int R, int CK, bool HALF>
__device__ __forceinline__ void read_iteration(const uint8_t *sl, const uint8_t *phl0, const uint8_t *phl1, int lane,
                                               const float (&sc)[2], float lr, float (&p)[8], float (&ph)[2][R])
{
    using Lay = FuLayout<R, CK, HALF>;
    const float4 g0 = *(const float4 *)(sl + lane * 16), g1 = *(const float4 *)(sl + 512 + lane * 16);
    uint32_t w[2];
    if (CK == CONEF_C_INT4) {
        w[0] = *(const unsigned short *)(sl + Lay::OFF_C + lane * 2);
        w[1] = *(const unsigned short *)(sl + Lay::OFF_C + 64 + lane * 2);
    } else {
        w[0] = *(const uint32_t *)(sl + Lay::OFF_C + lane * 4);
        w[1] = *(const uint32_t *)(sl + Lay::OFF_C + 128 + lane * 4);
    }
#pragma unroll
    for (int c = 0; c < R; c += 4) {
        const float4 t0 = *(const float4 *)(phl0 + c * 4), t1 = *(const float4 *)(phl1 + c * 4);
        ph[0][c] = t0.x; ph[0][c + 1] = t0.y; ph[0][c + 2] = t0.z; ph[0][c + 3] = t0.w;
        ph[1][c] = t1.x; ph[1][c + 1] = t1.y; ph[1][c + 2] = t1.z; ph[1][c + 3] = t1.w;
    }
    const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        float e[4];
        decode4<CK, HALF>(w[x], scale_const<CK, HALF>(sc[x]), e);
#pragma unroll
        for (int q = 0; q < 4; ++q)
            p[4 * x + q] = __fmaf_rn(lr, gv[4 * x + q], e[q]);
    }
}

template <int R, int CK, bool HALF, int MINB>
__global__ void __launch_bounds__(kFuThreads, MINB) k_fused23(const __grid_constant__ FusedParams P)
{
    using Lay = FuLayout<R, CK, HALF>;
    constexpr int UNIT = Lay::UNIT, NBLK = Lay::NBLK, SB = Lay::SB, SLOT = Lay::SLOT, CB = Lay::CB, OFF_C = Lay::OFF_C;
    constexpr int USH = (UNIT == 128) ? 7 : 8;
    constexpr float qlim = (CK == CONEF_C_INT8 ? 127.f : 7.f) + 0.49f;
    extern __shared__ __align__(128) uint8_t fu_smem[];
    __shared__ int s_abort, s_last;
    __shared__ uint32_t s_task[2];   // this task and the next one, with their groups
    __shared__ int s_group[2];
    const DevView &V = P.V;
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = uni(tid >> 5);
    const int RS = P.ring;
    const uint32_t ring_bytes = (uint32_t)RS * SLOT;
    uint8_t *wslots = fu_smem + (size_t)warp * ring_bytes;
    uint8_t *phbuf = fu_smem + (size_t)kFuWarps * ring_bytes;           // the tile's rows of P_hat
    uint64_t *bars = (uint64_t *)(phbuf + kFuPhBytes);                   // [warp][slot], then the one of phbuf
    const uint32_t slots_u32 = fu_smem_u32(wslots), bars_u32 = fu_smem_u32(bars + warp * RS);
    const uint32_t phbuf_u32 = fu_smem_u32(phbuf), phbar_u32 = fu_smem_u32(bars + kFuWarps * RS);
    const float lr = V.lr;

    // take the next task from the counter and find its group: the table entry of the task's
    // 32-block names a group at or before it
    auto fetch_task = [&](int slot) {
        const uint32_t task = atomicAdd(P.next_task, 1u);
        int g = 0;
        if (task < (uint32_t)P.n_tasks) {
            g = (int)__ldg(P.hint + (task >> 5));
            while (g + 1 < P.n_groups && (uint32_t)__ldg(&P.groups[g + 1].first) <= task)
                ++g;
        }
        s_task[slot] = task;
        s_group[slot] = g;
    };
    if (tid == 0) {
        s_abort = 0;
        fetch_task(0);
        mbar_init(phbar_u32, 1);
    }
    if (lane == 0)
        for (int s = 0; s < RS; ++s)
            mbar_init(bars_u32 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
    __syncthreads();

    uint32_t par = 0;      // bit s: parity of the phase slot s completes next
    uint32_t phpar = 0;    // ... of the phase the buffer of P_hat completes next
    auto aborted = [&]() { return *(volatile int *)&s_abort != 0; };
    auto give_up = [&]() {
        s_abort = 1;
        atomicOr(V.status, ST_FUSED_TIMEOUT);
    };
    auto wait_bar = [&](uint32_t bar, uint32_t parity) {
        uint32_t tries = 0;
        while (!mbar_try_wait(bar, parity)) {
            if (++tries > kFuMbarTries) {
                give_up();
                return false;
            }
        }
        return true;
    };
    // thread 0 waits (bounded) until *flag is set; every thread continues after it
    auto wait_flag = [&](const uint32_t *flag) {
        if (tid == 0) {
            uint32_t polls = 0;
            while (ld_acquire_u32(flag) == 0u) {
                ++polls;
                if (polls > kFuFlagPolls || ((polls & 63u) == 0 && (*(volatile int *)V.status & ST_FUSED_TIMEOUT))) {
                    give_up();
                    break;
                }
                __nanosleep(64);
            }
            __threadfence();
        }
        __syncthreads();
    };

    int tb = 0;
    uint32_t in_flight = 0;   // iterations of this warp whose copies were issued and not yet waited for
    int cpos = 0;             // ring slot of the next iteration to work on
    for (;;) {
        const uint32_t task = uni(s_task[tb]);
        if (task >= (uint32_t)P.n_tasks)
            break;
        // ---- the task: one phase of one unit, one tile (every value the same in all lanes)
        const FusedGroup *gp_ = P.groups + uni(s_group[tb]);
        const uint32_t gunit = uni((uint32_t)gp_->unit);
        const int phase = (int)(gunit >> 31);
        const uint32_t tile = task - uni((uint32_t)gp_->first) + uni((uint32_t)gp_->tile0);
        const FusedUnit *up = P.units + (gunit & 0x7fffffffu);
        const LayerDesc *Lp_ = V.layers + uni(up->layer);
        const int worker = uni(up->worker);
        const uint32_t ntp = uni((uint32_t)up->ntp), TP = uni((uint32_t)up->tp);
        uint32_t *ctr = P.ctr + uni(up->ctr_off);   // [ncg] arrivals per segment, [ncg] arrived segments, [ncg + 1] done
        const uint32_t m = (uint32_t)uni((int)Lp_->cols), d = (uint32_t)uni((int)Lp_->d), n = (uint32_t)uni((int)Lp_->rows);
        const uint32_t Lp = (uint32_t)uni(Lp_->f_lcm), subs = (uint32_t)uni(Lp_->f_subs), niter = (uint32_t)uni((int)Lp_->f_niter);
        const uint32_t ncg = Lp >> 8;
        const uint32_t t = tile / ncg, cg = tile - t * ncg;   // segments of one run of periods are neighbours in the list
        const uint32_t pt0 = t * TP, p0 = pt0 + (uint32_t)warp, p1 = min(niter, pt0 + TP);
        const uint32_t cnt = p1 > p0 ? (p1 - p0 + 7u) >> 3 : 0u;   // this warp's iterations: periods p0, p0 + 8, ...
        const uint32_t last_e = (niter - 1) * Lp + (cg << 8);   // this segment in the last period, the only one that may be short
        const uint32_t last_nv = last_e < d ? min(256u, d - last_e) : 0u;
        // the warp's last iteration is short: it is the last period and the segment is not whole there
        const bool short_last = cnt > 0 && p0 + 8u * (cnt - 1u) == niter - 1u && last_nv < 256u;
        const uint32_t cnt_full = short_last ? cnt - 1u : cnt;
        uint8_t *st = V.state + (int64_t)worker * V.state_stride;
        uint8_t *codes = st + uni(Lp_->a_off), *scales = st + uni(Lp_->b_off);
        const int64_t msgq_off = uni(Lp_->msgq_off);
        const uint32_t subf = (cg << 8) / m, nrows = ((cg << 8) + 255u) / m - subf + 1u;
        // first iteration's sources and the step to the next (8 periods on); all warp-uniform
        const uint64_t a_g = (uint64_t)(V.grads[worker] + uni(Lp_->g_off) + (cg << 8)) + (uint64_t)p0 * (Lp * 4u);
        const uint64_t a_c = (uint64_t)(codes + cg * (uint32_t)CB) + (uint64_t)p0 * (CK == CONEF_C_INT4 ? Lp >> 1 : Lp);
        const uint32_t d_g = Lp * 32u, d_c = CK == CONEF_C_INT4 ? Lp * 4u : Lp * 8u;
        uint32_t i_k = 0;   // iterations of this task whose copies have been issued
        auto issue_next = [&]() {
            int ipos = cpos + (int)in_flight;
            ipos = ipos >= RS ? ipos - RS : ipos;
            const uint32_t dst = slots_u32 + (uint32_t)ipos * SLOT, bar = bars_u32 + 8u * (uint32_t)ipos;
            if (elect_one()) {
                const uint64_t g_ = a_g + (uint64_t)i_k * d_g, c_ = a_c + (uint64_t)i_k * d_c;
                fence_proxy_async();
                if (i_k < cnt_full) {
                    mbar_expect_tx(bar, 1024u + CB);
                    bulk_g2s(dst, (const void *)g_, 1024u, bar);
                    bulk_g2s(dst + OFF_C, (const void *)c_, (uint32_t)CB, bar);
                } else {   // the short last period: copy what exists
                    const uint32_t gb = last_nv * 4u, cb = CK == CONEF_C_INT4 ? last_nv >> 1 : last_nv;
                    mbar_expect_tx(bar, gb + cb);
                    if (last_nv) {
                        bulk_g2s(dst, (const void *)g_, gb, bar);
                        bulk_g2s(dst + OFF_C, (const void *)c_, cb, bar);
                    }
                }
            }
            ++in_flight;
            ++i_k;
        };
        if (!aborted()) {
            __syncwarp();
            if (warp == 0 && elect_one()) {
                // the rows of P_hat the tile's periods meet, one run
                const uint32_t r0 = pt0 * subs + subf, r1 = min(n, (p1 - 1u) * subs + subf + nrows);
                const uint32_t nb = r1 > r0 ? (r1 - r0) * (R * 4u) : 0u;   // (nothing where the segment ends before this tile)
                fence_proxy_async();
                mbar_expect_tx(phbar_u32, nb);
                if (nb)
                    bulk_g2s(phbuf_u32, V.phat + Lp_->msgp_off + (size_t)r0 * R, nb, phbar_u32);
            }
            for (int s = 0; s < RS && i_k < cnt; ++s)
                issue_next();
        }
        if (tid == 0)
            fetch_task(tb ^ 1);   // while the first copies are under way; read after the barrier that ends this task

        // ---- where this lane's two pieces sit
        uint32_t col[2];
        const uint8_t *phl[2];   // this lane's rows of P_hat in the buffer, current iteration
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const uint32_t off = (cg << 8) + 128u * x + 4u * lane, sub = off / m;
            col[x] = off - sub * m;
            phl[x] = phbuf + ((uint32_t)warp * subs + sub - subf) * (R * 4u);
        }
        const uint32_t ph_step = 8u * subs * (R * 4u);
        uint32_t c_e0w = p0 * Lp + (cg << 8);
        const uint8_t *sptr = scales + (size_t)(c_e0w >> USH) * SB;   // the scales of the current iteration
        const uint32_t sstep = ((8u * Lp) >> USH) * SB;
        ScaleWord<NBLK, HALF> sw_next{};
        if (cnt > 0 && c_e0w < d)
            sw_next = load_scales<NBLK, HALF>(sptr);
        // wait for the next iteration's slot and read it; pass the slot on to the stream; false: the wait gave up
        auto next_iteration = [&](float (&p)[8], float (&ph)[2][R], bool more) -> bool {
            if (!wait_bar(bars_u32 + 8u * (uint32_t)cpos, (par >> cpos) & 1u))
                return false;
            par ^= 1u << cpos;
            float sc[2];
            scales_of<NBLK, HALF>(sw_next, sc);
            if (more && c_e0w + 8u * Lp < d)
                sw_next = load_scales<NBLK, HALF>(sptr + sstep);
            read_iteration<R, CK, HALF>(wslots + (size_t)cpos * SLOT, phl[0], phl[1], lane, sc, lr, p, ph);
            cpos = cpos + 1 == RS ? 0 : cpos + 1;
            --in_flight;
            if (i_k < cnt) {   // the slot is free: fetch the iteration that takes it next
                __syncwarp();
                issue_next();
            }
            return true;
        };
        auto advance = [&]() {
            c_e0w += 8u * Lp;
            sptr += sstep;
            phl[0] += ph_step;
            phl[1] += ph_step;
        };
        bool ok_run = !aborted();
        if (phase == 0) {
            // ------------------------------------------------------------------ Q_i partials of this tile
            float frag[8][R];
#pragma unroll
            for (int q = 0; q < 8; ++q)
#pragma unroll
                for (int c = 0; c < R; ++c)
                    frag[q][c] = 0.f;
            if (ok_run && cnt > 0)
                ok_run = wait_bar(phbar_u32, phpar);
            uint32_t i = 0;
            for (; ok_run && i < cnt_full; ++i) {
                float p[8], ph[2][R];
                if (!next_iteration(p, ph, i + 1 < cnt)) {
                    ok_run = false;
                    break;
                }
#pragma unroll
                for (int x = 0; x < 2; ++x)
#pragma unroll
                    for (int q = 0; q < 4; ++q)
#pragma unroll
                        for (int c = 0; c < R; ++c)
                            frag[4 * x + q][c] = __fmaf_rn(p[4 * x + q], ph[x][c], frag[4 * x + q][c]);
                advance();
            }
            if (ok_run && short_last) {   // lanes past the end of the tensor hold stale data
                float p[8], ph[2][R];
                if (next_iteration(p, ph, false)) {
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        const bool ok = c_e0w + 128u * x + 4u * lane < d;
#pragma unroll
                        for (int q = 0; q < 4; ++q)
#pragma unroll
                            for (int c = 0; c < R; ++c)
                                frag[4 * x + q][c] = ok ? __fmaf_rn(p[4 * x + q], ph[x][c], frag[4 * x + q][c]) : frag[4 * x + q][c];
                    }
                }
            }
            // the 8 warps' sums, added in warp order: every warp leaves its sums in its own ring
            // (all its copies have been consumed), 4 factor columns at a time, as [piece 4x + q][lane]
            // (no bank conflicts); thread tid then adds position tid of the 8 warps.  Partial sums and
            // segment sums keep that order; the last step below maps it back to columns.
            float *part = P.scratch + uni(up->scratch_off);              // [ncg][ntp][R / 4][256] float4
            float *qseg = part + (size_t)ncg * ntp * 256 * R;            // [ncg][R / 4][256] float4
            bool guards_done = false;
#pragma unroll
            for (int c = 0; c < R; c += 4) {
                if (c > 0)
                    __syncthreads();
#pragma unroll
                for (int x = 0; x < 2; ++x)
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        ((float4 *)wslots)[(4 * x + q) * 32 + lane] =
                            make_float4(frag[4 * x + q][c], frag[4 * x + q][c + 1], frag[4 * x + q][c + 2], frag[4 * x + q][c + 3]);
                __syncthreads();
                float4 acc = ((const float4 *)fu_smem)[tid];
#pragma unroll
                for (int w = 1; w < kFuWarps; ++w) {
                    const float4 v = *((const float4 *)(fu_smem + (size_t)w * ring_bytes) + tid);
                    acc.x = __fadd_rn(acc.x, v.x); acc.y = __fadd_rn(acc.y, v.y);
                    acc.z = __fadd_rn(acc.z, v.z); acc.w = __fadd_rn(acc.w, v.w);
                }
                if (!guards_done) {
                    // the scratch of this unit may still belong to earlier units (it cycles): wait for those
                    const int guard_lo = uni(up->guard_lo), guard_hi = uni(up->guard_hi);
                    for (int gu = guard_lo; gu <= guard_hi; ++gu)
                        wait_flag(P.ctr + P.units[gu].flag_off);
                    guards_done = true;
                }
                ((float4 *)(part + ((size_t)cg * ntp + t) * 256 * R))[(c / 4) * 256 + tid] = acc;
            }
            __syncthreads();   // every thread's partial sums are written: thread 0's fence below covers them
            if (tid == 0) {
                __threadfence();
                s_last = !aborted() && atomicAdd(ctr + cg, 1u) == ntp - 1u;
            }
            __syncthreads();
            if (s_last) {
                // last tile of this segment: the segment's sums, tiles in order
                __threadfence();
                for (int x = tid; x < 256 * R / 4; x += kFuThreads) {
                    const float4 *src = (const float4 *)(part + (size_t)cg * ntp * 256 * R) + x;
                    float4 acc = __ldcg(src);
                    for (uint32_t tt = 1; tt < ntp; ++tt) {
                        const float4 v = __ldcg(src + (size_t)tt * (256 * R / 4));
                        acc.x = __fadd_rn(acc.x, v.x); acc.y = __fadd_rn(acc.y, v.y);
                        acc.z = __fadd_rn(acc.z, v.z); acc.w = __fadd_rn(acc.w, v.w);
                    }
                    ((float4 *)(qseg + (size_t)cg * 256 * R))[x] = acc;
                }
                __syncthreads();
                if (tid == 0) {
                    __threadfence();
                    s_last = atomicAdd(ctr + ncg, 1u) == ncg - 1u;
                }
                __syncthreads();
                if (s_last) {
                    // last segment of the unit: Q_i of a column = its positions in the period's rows, in order
                    __threadfence();
                    float *q_out = P.q_out + (int64_t)worker * P.q_out_stride + msgq_off;
                    const uint32_t items = m * (R / 4);
                    for (uint32_t it = tid; it < items; it += kFuThreads) {
                        const uint32_t c = it / (R / 4), h = it - c * (R / 4);
                        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                        for (uint32_t s = 0; s < subs; ++s) {
                            const uint32_t pos = s * m + c, off = pos & 255u;
                            const uint32_t sp = (((off >> 7) * 4u + (off & 3u)) << 5) + ((off >> 2) & 31u);
                            const float4 v = __ldcg((const float4 *)(qseg + (size_t)(pos >> 8) * 256 * R) + h * 256 + sp);
                            if (s == 0) {
                                acc = v;
                            } else {
                                acc.x = __fadd_rn(acc.x, v.x); acc.y = __fadd_rn(acc.y, v.y);
                                acc.z = __fadd_rn(acc.z, v.z); acc.w = __fadd_rn(acc.w, v.w);
                            }
                        }
                        *((float4 *)(q_out + (size_t)c * R) + h) = acc;
                    }
                    __syncthreads();
                    if (tid == 0) {
                        __threadfence();
                        atomicExch(ctr + ncg + 1, 1u);
                    }
                }
            }
        } else {
            // ------------------------------------------------------------------ residual, block maxima, codes and scales
            wait_flag(ctr + ncg + 1);
            const float *q_res = P.q_res + (int64_t)worker * P.q_res_stride + msgq_off;
            float frag[8][R];   // Q_i of this lane's columns
#pragma unroll
            for (int x = 0; x < 2; ++x)
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int c = 0; c < R; c += 4) {
                        const float4 t4 = __ldcg((const float4 *)(q_res + (size_t)(col[x] + q) * R + c));
                        frag[4 * x + q][c] = t4.x; frag[4 * x + q][c + 1] = t4.y;
                        frag[4 * x + q][c + 2] = t4.z; frag[4 * x + q][c + 3] = t4.w;
                    }
            // where this lane's codes of the current iteration go
            uint8_t *cptr = codes + (CK == CONEF_C_INT4 ? (c_e0w + 4u * lane) >> 1 : c_e0w + 4u * lane);
            const uint32_t cstep = CK == CONEF_C_INT4 ? Lp * 4u : Lp * 8u;
            auto finish = [&](float (&p)[8], const float (&ph)[2][R], auto tail_c) {
                constexpr bool TAIL = decltype(tail_c)::value != 0;
                bool ok[2] = {true, true};
                if (TAIL) {
                    ok[0] = c_e0w + 4u * lane < d;
                    ok[1] = c_e0w + 128u + 4u * lane < d;
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
                        if (TAIL)
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
                    cw[0] = quant_pack4<CK, true>(&p[0], inv[0]);
                    cw[1] = quant_pack4<CK, true>(&p[4], inv[1]);
                } else {
                    cw[0] = quant_pack4<CK, false>(&p[0], inv[0]);
                    cw[1] = quant_pack4<CK, false>(&p[4], inv[1]);
                }
#pragma unroll
                for (int x = 0; x < 2; ++x)
                    if (ok[x]) {
                        if (CK == CONEF_C_INT4)
                            *(unsigned short *)(cptr + 64 * x) = (unsigned short)cw[x];
                        else
                            *(uint32_t *)(cptr + 128 * x) = cw[x];
                    }
                if (lane == 0) {
                    uint8_t *sout = scales + (size_t)(c_e0w >> USH) * SB;
#pragma unroll
                    for (int x = 0; x < NBLK; ++x)
                        if (!TAIL || c_e0w + (uint32_t)UNIT * x < d) {
                            if (HALF)
                                *(unsigned short *)(sout + 2 * x) = hb[x];
                            else
                                *(float *)(sout + 4 * x) = s[x];
                        }
                }
            };
            if (ok_run && cnt > 0)
                ok_run = wait_bar(phbar_u32, phpar);
            uint32_t i = 0;
            for (; ok_run && i < cnt_full; ++i) {
                float p[8], ph[2][R];
                if (!next_iteration(p, ph, i + 1 < cnt)) {
                    ok_run = false;
                    break;
                }
                finish(p, ph, IntC<0>());
                advance();
                cptr += cstep;
            }
            if (ok_run && short_last) {
                float p[8], ph[2][R];
                if (next_iteration(p, ph, false))
                    finish(p, ph, IntC<1>());
            }
        }
        phpar ^= 1u;   // (every warp tracks the buffer's phase, whether it waited or not)
        __syncthreads();
        if (aborted())
            break;
        tb ^= 1;
    }
    // copies still in flight (only after a wait gave up) must land before the CTA's memory goes away
    for (; in_flight; --in_flight) {
        const uint32_t bar = bars_u32 + 8u * (uint32_t)cpos, ph = (par >> cpos) & 1u;
        for (uint32_t tt = 0; tt < kFuMbarTries && !mbar_try_wait(bar, ph); ++tt) {
        }
        cpos = cpos + 1 == RS ? 0 : cpos + 1;
    }
    if (aborted() && warp == 0)
        for (uint32_t tt = 0; tt < kFuMbarTries && !mbar_try_wait(phbar_u32, phpar); ++tt) {
        }
}

template <int R, int CK, bool HALF, int MINB>
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
    const int fixed = kFuPhBytes + 8 + 128;   // the tile's rows of P_hat and their barrier, alignment slack
    // MINB CTAs per SM (1 KB of each SM's shared memory is reserved per CTA)
    const int per_cta = std::min(max_smem, max_sm / MINB - 1024);
    int ring = (per_cta - fixed) / (kFuWarps * (Lay::SLOT + 8));
    ring = std::min(ring, 8);
    if (ring * Lay::SLOT < 4096)   // a warp's ring also takes its 256 x 4 partial sums at the end of a tile
        return cudaErrorInvalidConfiguration;
    out->ring = ring;
    out->smem = (size_t)kFuWarps * ring * (Lay::SLOT + 8) + fixed;
    out->threads = kFuThreads;
    out->ctas_per_sm = MINB;
    if ((e = cudaFuncSetAttribute(k_fused23<R, CK, HALF, MINB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)out->smem)) !=
        cudaSuccess)
        return e;
    int occ = 0;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_fused23<R, CK, HALF, MINB>, kFuThreads, out->smem)) !=
        cudaSuccess)
        return e;
    if (occ < 1)
        return cudaErrorInvalidConfiguration;
    out->ctas = std::min(occ, MINB) * n_sms;
    return cudaSuccess;
}

template <int R, int CK, bool HALF, int MINB>
cudaError_t fused_launch_t(const FusedParams &P, int n_ctas, size_t smem, cudaStream_t s)
{
    void *args[] = {(void *)&P};
    return cudaLaunchCooperativeKernel((const void *)k_fused23<R, CK, HALF, MINB>, dim3(n_ctas), dim3(kFuThreads), args, smem, s);
}

}  // namespace

#define CONEF_FUSED_CASE(FN, RV, CKV, HV, ...)                                                        \
    if (ckind == CKV && rank == RV && (half != 0) == HV) {                                             \
        if (minb == 2) return FN<RV, CKV, HV, 2>(__VA_ARGS__);                                         \
        if (minb == 3) return FN<RV, CKV, HV, 3>(__VA_ARGS__);                                         \
        if (minb == 4) return FN<RV, CKV, HV, 4>(__VA_ARGS__);                                         \
        return cudaErrorNotSupported;                                                                  \
    }
#define CONEF_FUSED_DISPATCH(FN, ...)                                \
    CONEF_FUSED_CASE(FN, 4, CONEF_C_INT4, true, __VA_ARGS__)         \
    CONEF_FUSED_CASE(FN, 8, CONEF_C_INT4, true, __VA_ARGS__)         \
    CONEF_FUSED_CASE(FN, 4, CONEF_C_INT4, false, __VA_ARGS__)        \
    CONEF_FUSED_CASE(FN, 8, CONEF_C_INT4, false, __VA_ARGS__)        \
    CONEF_FUSED_CASE(FN, 4, CONEF_C_INT8, true, __VA_ARGS__)         \
    CONEF_FUSED_CASE(FN, 8, CONEF_C_INT8, true, __VA_ARGS__)         \
    CONEF_FUSED_CASE(FN, 4, CONEF_C_INT8, false, __VA_ARGS__)        \
    CONEF_FUSED_CASE(FN, 8, CONEF_C_INT8, false, __VA_ARGS__)        \
    return cudaErrorNotSupported;

cudaError_t fused_config(int ckind, int rank, int half, int minb, int n_sms, FusedConfig *out)
{
    CONEF_FUSED_DISPATCH(fused_config_t, n_sms, out)
}

cudaError_t fused_launch(int ckind, int rank, int half, int minb, const FusedParams &P, int n_ctas, size_t smem, cudaStream_t s)
{
    CONEF_FUSED_DISPATCH(fused_launch_t, P, n_ctas, smem, s)
}

}  // namespace conef
