// Tuned fused step for Q in {identity, random-k, random-block-k} with an int8 / int4 error state,
// or the stochastic quantiser of Eq. 6 with at most 127 levels (signed levels in one byte, fp32 scale)
// (Alg. 2 lines 5, 6, 9 in one kernel): decode, p = eta g + e, message, residual, block absmax,
// requantise, store in place.  A thread owns 8 consecutive elements (two 16-byte copies of the
// gradient, one 8- or 4-byte copy of the codes, through a ring of asynchronous copies), a warp 256, so that every
// quantisation block (32..256 elements) is an aligned group of lanes and its absmax a few
// shuffles.  Membership in the shared random-k index set comes from the bitmap that the
// selection kernels leave (one byte per thread), not from hashing every element again for every
// worker; message slots are tile offset + block offset + a prefix over the block's lanes.
// ICO = 1 is iConEF-v1 (Alg. 3) on an int8 / int4 state: a second state q of the same kind is decoded
// beside the first, p = (eta g + e~) + q, and the store has a second round, q = C(r - decode(e~)).
// ICO = 2 is iConEF-v2 (Alg. 3 line 12) with a sparsifying Q: e~ is the k values a second draw of Q
// kept at the step that stored them (gathered through that draw's bitmap and slot offsets), the
// stored state is q, p = (eta g + e~) + q; this step's second draw takes its members' residuals as
// the next e~ and the rest is stored as q = C(r - e~).
// Takes tensors with d % 8 == 0 and 16-byte aligned gradients; the generic kernel does the rest.
#pragma once
#include "conef_fast.cuh"
#include "conef_kernels.cuh"

namespace conef {

constexpr int kFvThreads = 256;
constexpr int kFvChunks = kHistTile / (kFvThreads * 8);   // 256-element chunks per warp and selection tile (4)
constexpr int kFvRing = 3;                                // stages of the per-thread copy ring
constexpr int kFvTiles = 4;                               // selection tiles (8192 elements) per CTA for large models (V.fv_tiles; 1 for small ones)

template <int QK, int CK, bool HALF, int ICO = 0>
__global__ void __launch_bounds__(kFvThreads, ICO ? 3 : 4) k_flat_vec(const __grid_constant__ DevView V, const int32_t *__restrict__ pfx)
{
    const int li = find_layer(pfx, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int worker = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t d = (uint32_t)L.d;
    const uint32_t tile0 = (blockIdx.x - pfx[li]) * (uint32_t)V.fv_tiles;   // first selection tile of this CTA
    const int unit_shift = 31 - __clz(L.unit);
    const int lpb = L.unit >> 3;                       // lanes per quantisation block
    constexpr int CW = (CK == CONEF_C_INT4) ? 1 : 2;   // code words per thread
    // signed levels of the stochastic quantiser decode like int8 codes with an fp32 scale
    constexpr int DK = (CK == CONEF_C_STOCHQUANT) ? CONEF_C_INT8 : CK;
    uint8_t *st = V.state + worker * V.state_stride;
    const float *__restrict__ g = V.grads[worker] + L.g_off;
    uint8_t *codes = st + L.a_off;
    uint8_t *scales = st + L.b_off;
    uint8_t *codes2 = st + L.a2_off, *scales2 = st + L.b2_off;   // the second state (ICO)
    float *__restrict__ msg = V.msgv + worker * V.msgv_stride + L.msgv_off;
    const uint8_t *__restrict__ bits = (const uint8_t *)(V.selbits + L.selbits_off);
    const uint32_t *__restrict__ tileoff = V.tileoff + L.tileoff_off;
    uint32_t blk_start = 0;
    if (QK == CONEF_Q_RANDBLOCK)
        blk_start = randblock_start(stream_key(V.seed_q, (uint64_t)li, (uint64_t)V.step), d, (uint32_t)L.k);
    // iConEF-v2: the draw that stored e~ (A) and this step's second draw (B)
    const uint8_t *__restrict__ bitsA = (const uint8_t *)(V.selbitsA + L.selbits_off);
    const uint8_t *__restrict__ bitsB = (const uint8_t *)(V.selbitsB + L.selbits_off);
    const float *__restrict__ ev_old = V.ev_old + worker * V.msgv_stride + L.msgv_off;
    float *__restrict__ ev_new = V.ev_new + worker * V.msgv_stride + L.msgv_off;
    uint32_t blk_startA = 0, blk_startB = 0;
    if (ICO == 2 && QK == CONEF_Q_RANDBLOCK) {
        blk_startA = randblock_start(stream_key(V.seed_q, (uint64_t)li, (uint64_t)(V.ev_step + kSecondDraw)), d, (uint32_t)L.k);
        blk_startB = randblock_start(stream_key(V.seed_q, (uint64_t)li, (uint64_t)(V.step + kSecondDraw)), d, (uint32_t)L.k);
    }
    const float lr = V.lr;

    // within a selection tile the warp's chunks are consecutive: 1024 elements per warp and tile;
    // step i of the warp is chunk i % 4 of tile i / 4
    const uint32_t e0 = tile0 * (uint32_t)kHistTile + (uint32_t)warp * (kFvChunks * 256) + (uint32_t)lane * 8;
    const int kSteps = V.fv_tiles * kFvChunks;
    auto elem = [&](int i) { return e0 + (uint32_t)(i / kFvChunks) * kHistTile + (uint32_t)(i % kFvChunks) * 256; };
    // A ring of kFvRing stages of asynchronous copies per thread (a thread only reads what it
    // copied, so no barrier): the gradient, the code words, and 4-byte words that hold the block's
    // scale and the thread's membership byte(s).  Stage s of thread t: lo[s][t], hi[s][t] (16 bytes
    // each), then 4-byte arrays [s][t] in the order codes, scale, membership, and with Alg. 3 the
    // second state's codes and scale (version 1) or the two second draws' membership (version 2).
    extern __shared__ __align__(128) uint8_t fv_smem[];
    constexpr int D = kFvRing, T = kFvThreads;
    constexpr int SB = HALF ? 2 : 4;
    const int tid = threadIdx.x;
    float4 *r_lo = (float4 *)fv_smem + tid, *r_hi = r_lo + D * T;
    uint32_t *r32 = (uint32_t *)((float4 *)fv_smem + 2 * D * T);
    uint32_t *r_cw = r32 + tid * CW, *r_sc = r32 + D * T * CW + tid, *r_sel = r32 + D * T * (CW + 1) + tid;
    uint32_t *r_cv = r32 + D * T * (CW + 2) + tid * CW, *r_sc2 = r32 + D * T * (2 * CW + 2) + tid;   // ICO = 1
    uint32_t *r_selA = r32 + D * T * (CW + 2) + tid, *r_selB = r32 + D * T * (CW + 3) + tid;         // ICO = 2
    auto word_of = [](const void *p) { return (const void *)((uintptr_t)p & ~(uintptr_t)3); };   // the aligned 4 bytes that hold *p
    auto issue = [&](int c, int slot) {
        const uint32_t j = elem(c);
        if (c < kSteps && j < d) {
            cp_async16(r_lo + slot * T, g + j);
            cp_async16(r_hi + slot * T, g + j + 4);
            cp_async_small<4 * CW>(r_cw + slot * T * CW, codes + (CW == 1 ? (j >> 1) : j));
            cp_async_small<4>(r_sc + slot * T, word_of(scales + (size_t)(j >> unit_shift) * SB));
            if (QK == CONEF_Q_RANDK)
                cp_async_small<4>(r_sel + slot * T, word_of(bits + (j >> 3)));
            if (ICO == 1) {
                cp_async_small<4 * CW>(r_cv + slot * T * CW, codes2 + (CW == 1 ? (j >> 1) : j));
                cp_async_small<4>(r_sc2 + slot * T, word_of(scales2 + (size_t)(j >> unit_shift) * SB));
            }
            if (ICO == 2 && QK == CONEF_Q_RANDK) {
                if (V.ev_valid)
                    cp_async_small<4>(r_selA + slot * T, word_of(bitsA + (j >> 3)));
                cp_async_small<4>(r_selB + slot * T, word_of(bitsB + (j >> 3)));
            }
        }
        cp_async_commit();
    };
    auto scale_in = [&](uint32_t word, uint32_t blk) {   // the block's scale out of its 4-byte word
        if (HALF)
            return __half2float(__ushort_as_half((unsigned short)((blk & 1u) ? word >> 16 : word & 0xFFFFu)));
        return __uint_as_float(word);
    };
    auto byte_in = [](uint32_t word, const uint8_t *p) { return (word >> (8 * (uint32_t)((uintptr_t)p & 3))) & 0xFFu; };
#pragma unroll
    for (int s = 0; s < D - 1; ++s)
        issue(s, s);
    uint32_t toff = 0;
    int rs = 0;
    // one chunk; CHECK is false where the warp's 256 elements all exist (no selects on `valid`)
    auto chunk = [&](int c, auto check_c) {
        constexpr bool CHECK = decltype(check_c)::value != 0;
        issue(c + D - 1, rs == 0 ? D - 1 : rs - 1);   // the stage read one iteration ago
        cp_async_wait<D - 1>();                          // this chunk's copies have landed
        constexpr int buf = 0;
        float4 g0[1], g1[1];
        uint32_t w0[1], w1[1], v0[1], v1[1], sel[1], selA[1], selB[1];
        float sc[1], sc2[1];
        {
            const uint32_t jj = elem(c);
            const bool have = !CHECK || jj < d;   // a stage that was not filled holds stale data
            const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
            g0[0] = have ? r_lo[rs * T] : z4;
            g1[0] = have ? r_hi[rs * T] : z4;
            w0[0] = have ? r_cw[rs * T * CW] : 0u;
            w1[0] = (have && CW == 2) ? r_cw[rs * T * CW + CW - 1] : 0u;
            sc[0] = have ? scale_in(r_sc[rs * T], jj >> unit_shift) : 0.f;
            sel[0] = (have && QK == CONEF_Q_RANDK) ? byte_in(r_sel[rs * T], bits + (jj >> 3)) : 0u;
            v0[0] = v1[0] = 0u;
            sc2[0] = 0.f;
            selA[0] = selB[0] = 0u;
            if (ICO == 1) {
                v0[0] = have ? r_cv[rs * T * CW] : 0u;
                v1[0] = (have && CW == 2) ? r_cv[rs * T * CW + CW - 1] : 0u;
                sc2[0] = have ? scale_in(r_sc2[rs * T], jj >> unit_shift) : 0.f;
            }
            if (ICO == 2 && QK == CONEF_Q_RANDK) {
                selA[0] = (have && V.ev_valid) ? byte_in(r_selA[rs * T], bitsA + (jj >> 3)) : 0u;
                selB[0] = have ? byte_in(r_selB[rs * T], bitsB + (jj >> 3)) : 0u;
            }
        }
        rs = rs + 1 == D ? 0 : rs + 1;
        const uint32_t j = elem(c);
        const bool valid = !CHECK || j < d;
        if (QK == CONEF_Q_RANDK && c % kFvChunks == 0)
            toff = tileoff[tile0 + c / kFvChunks];
        const float gv[8] = {g0[buf].x, g0[buf].y, g0[buf].z, g0[buf].w, g1[buf].x, g1[buf].y, g1[buf].z, g1[buf].w};
        float e[8], r[8];
        decode8<DK, HALF>(w0[buf], w1[buf], scale_const<DK, HALF>(sc[buf]), e);
        float qv[8];
        if (ICO == 1)
            decode8<DK, HALF>(v0[buf], v1[buf], scale_const<DK, HALF>(sc2[buf]), qv);
        uint32_t mybits = sel[buf];
        // iConEF-v2: the stored state is q; e~ comes from the values draw A kept
        uint32_t mA = 0, mB = 0, slotA = 0, slotB = 0;
        if (ICO == 2) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
                qv[q] = e[q];
            if (QK == CONEF_Q_RANDK) {
                mA = selA[buf];
                mB = selB[buf];
                const int cA = __popc(mA), cB = __popc(mB);
                int incA = cA, incB = cB;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int tA = __shfl_up_sync(0xffffffffu, incA, o), tB = __shfl_up_sync(0xffffffffu, incB, o);
                    if (o < lpb && (lane & (lpb - 1)) >= o) {
                        incA += tA;
                        incB += tB;
                    }
                }
                const uint32_t tile = tile0 + (uint32_t)(c / kFvChunks), unit = j >> unit_shift;
                if (cA)
                    slotA = V.tileoffA[L.tileoff_off + tile] + V.unitoffA[L.unitoff_off + unit] + (uint32_t)(incA - cA);
                if (cB)
                    slotB = V.tileoffB[L.tileoff_off + tile] + V.unitoffB[L.unitoff_off + unit] + (uint32_t)(incB - cB);
            } else {
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    mA |= (uint32_t)(V.ev_valid && (j + q - blk_startA) < (uint32_t)L.k) << q;
                    mB |= (uint32_t)((j + q - blk_startB) < (uint32_t)L.k) << q;
                }
                mA = valid ? mA : 0u;
                mB = valid ? mB : 0u;
                slotA = j - blk_startA + (uint32_t)__ffs(mA) - 1u;   // the blocks are contiguous: first member
                slotB = j - blk_startB + (uint32_t)__ffs(mB) - 1u;
            }
#pragma unroll
            for (int q = 0; q < 8; ++q)
                e[q] = 0.f;
            for (uint32_t mm = mA; mm; mm &= mm - 1) {   // the few members of A among this thread's elements
                const int q = __ffs(mm) - 1;
                const float v = ev_old[slotA++];
#pragma unroll
                for (int x = 0; x < 8; ++x)
                    e[x] = q == x ? v : e[x];
            }
        }
        if (QK == CONEF_Q_RANDBLOCK) {
            mybits = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                mybits |= (uint32_t)((j + q - blk_start) < (uint32_t)L.k) << q;
            mybits = valid ? mybits : 0u;
        }
        // message slot of this thread's first selected element
        uint32_t slot = 0;
        if (QK == CONEF_Q_RANDK) {
            const int cnt = __popc(mybits);
            int inc = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, inc, o);
                if (o < lpb && (lane & (lpb - 1)) >= o)
                    inc += t;
            }
            if (cnt)
                slot = toff + V.unitoff[L.unitoff_off + (j >> unit_shift)] + (uint32_t)(inc - cnt);   // (a copy of this word in the ring cost more than the load)
        } else if (QK == CONEF_Q_RANDBLOCK) {
            slot = j - blk_start + (uint32_t)__ffs(mybits) - 1u;   // the block is contiguous: first selected element
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            float p = __fmaf_rn(lr, gv[q], e[q]);   // Alg. 2 line 5
            if (ICO)
                p = __fadd_rn(p, qv[q]);                  // Alg. 3 line 5: + q (the second state, or with version 2 the stored one)
            e[q] = p;   // kept for the message stores below
            r[q] = (QK == CONEF_Q_IDENTITY || ((mybits >> q) & 1u) || !valid) ? 0.f : p;   // r = p - Delta
        }
        if (QK != CONEF_Q_IDENTITY) {
            // the few selected elements of this thread, in ascending index order
            for (uint32_t m = mybits; m; m &= m - 1) {
                const int q = __ffs(m) - 1;
                float p = e[0];
#pragma unroll
                for (int x = 1; x < 8; ++x)
                    p = q == x ? e[x] : p;
                msg[slot] = p;
                if (worker == 0)
                    V.idx[L.idx_off + slot] = j + q;
                ++slot;
            }
        }
        if (QK == CONEF_Q_IDENTITY && valid) {
            *(float4 *)(msg + j) = make_float4(e[0], e[1], e[2], e[3]);
            *(float4 *)(msg + j + 4) = make_float4(e[4], e[5], e[6], e[7]);
        }
        if (ICO == 2) {
            // Alg. 3 line 12: e~ = Q(r) by the second draw; r - e~ is exactly zero where e~ keeps the value
            for (uint32_t mm = mB; mm; mm &= mm - 1) {
                const int q = __ffs(mm) - 1;
                float v = r[0];
#pragma unroll
                for (int x = 1; x < 8; ++x)
                    v = q == x ? r[x] : v;
                ev_new[slotB++] = v;
#pragma unroll
                for (int x = 0; x < 8; ++x)
                    r[x] = q == x ? 0.f : r[x];
            }
        }
        // store r through C (Alg. 2 line 9)
        float amax = 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q)
            amax = fmaxf(amax, fabsf(r[q]));
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1)
            if (o <= 2 || lpb > o)
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        float s, inv;
        unsigned short hb = 0;
        uint32_t c0 = 0, c1 = 0;
        if constexpr (CK == CONEF_C_STOCHQUANT) {
            // Eq. 6 with the block's max-norm: level floor(u) or floor(u) + 1, up with probability
            // u - floor(u); the variate of (worker, tensor, step, element) from a counter-based stream
            const float lv = (float)V.levels;
            s = __fdiv_rn(amax, lv);
            const bool zero = !(s >= FLT_MIN);
            s = zero ? 0.f : s;
            inv = zero ? 0.f : __fdiv_rn(1.0f, s);
            if (!zero) {
                const uint64_t stc = stream_key(mix64(V.seed_c + (uint64_t)worker + 1u), (uint64_t)li, (uint64_t)V.step);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    float u = __fmul_rn(fabsf(r[q]), inv);
                    u = !(u <= lv) ? lv : u;
                    const float l = floorf(u);
                    const float frac = __fsub_rn(u, l);
                    const float rnd = __fmul_rn((float)(uint32_t)(h64(stc, j + q) >> 40), 1.0f / 16777216.0f);
                    int lev = (int)l + (rnd < frac ? 1 : 0);
                    lev = min(lev, V.levels);
                    const uint32_t byte = (uint32_t)(r[q] < 0.f ? -lev : lev) & 0xFFu;
                    if (q < 4)
                        c0 |= byte << (8 * q);
                    else
                        c1 |= byte << (8 * (q - 4));
                }
            }
        } else {
            block_scale<DK, HALF>(amax, s, inv, hb);
            constexpr float qlim = (CK == CONEF_C_INT8 ? 127.f : 7.f) + 0.49f;
            if (__any_sync(0xffffffffu, !(__fmul_rn(amax, inv) < qlim)))
                quant_pack8<DK, true>(r, inv, c0, c1);
            else
                quant_pack8<DK, false>(r, inv, c0, c1);
        }
        if (valid) {
            if ((lane & (lpb - 1)) == 0) {
                if (HALF)
                    ((unsigned short *)scales)[j >> unit_shift] = hb;
                else
                    ((float *)scales)[j >> unit_shift] = s;
            }
            if (CW == 1)
                *(uint32_t *)(codes + (j >> 1)) = c0;
            else
                *(uint2 *)(codes + j) = make_uint2(c0, c1);
        }
        if constexpr (ICO == 1 && CK != CONEF_C_STOCHQUANT) {
            // Alg. 3 lines 10, 14: e~ = C(r) was just formed; q = C(r - decode(e~)), what the first state misses
            float e1[8];
            decode8<DK, HALF>(c0, c1, scale_const<DK, HALF>(s), e1);
            float amax2 = 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                r[q] = __fsub_rn(r[q], e1[q]);
                amax2 = fmaxf(amax2, fabsf(r[q]));
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1)
                if (o <= 2 || lpb > o)
                    amax2 = fmaxf(amax2, __shfl_xor_sync(0xffffffffu, amax2, o));
            float s2, inv2;
            unsigned short hb2 = 0;
            uint32_t d0 = 0, d1 = 0;
            block_scale<DK, HALF>(amax2, s2, inv2, hb2);
            constexpr float qlim2 = (CK == CONEF_C_INT8 ? 127.f : 7.f) + 0.49f;
            if (__any_sync(0xffffffffu, !(__fmul_rn(amax2, inv2) < qlim2)))
                quant_pack8<DK, true>(r, inv2, d0, d1);
            else
                quant_pack8<DK, false>(r, inv2, d0, d1);
            if (valid) {
                if ((lane & (lpb - 1)) == 0) {
                    if (HALF)
                        ((unsigned short *)scales2)[j >> unit_shift] = hb2;
                    else
                        ((float *)scales2)[j >> unit_shift] = s2;
                }
                if (CW == 1)
                    *(uint32_t *)(codes2 + (j >> 1)) = d0;
                else
                    *(uint2 *)(codes2 + j) = make_uint2(d0, d1);
            }
        }
    };
    for (int c = 0; c < kSteps; ++c) {
        const uint32_t jw = elem(c) - (uint32_t)lane * 8;   // the warp's first element of this chunk
        if (jw >= d)
            break;              // past the end of the tensor
        if (jw + 256 <= d)
            chunk(c, IntC<0>());
        else
            chunk(c, IntC<1>());
    }
    cp_async_wait<0>();   // (a warp that left the loop early still has copies in flight)
}

// bytes of the copy ring (below the 48 KB that need no opt-in)
inline size_t fv_smem_bytes(int ckind, int ico)
{
    const int cw = ckind == CONEF_C_INT4 ? 1 : 2;
    return (size_t)kFvRing * kFvThreads * (32 + 4 * (cw + 2) + (ico == 1 ? 4 * (cw + 1) : ico == 2 ? 8 : 0));
}

inline cudaError_t flatvec_launch(int qkind, int ckind, int half, const DevView &V, const int32_t *pfx, int tiles,
                                  cudaStream_t s)
{
    if (tiles <= 0)
        return cudaSuccess;
    dim3 grid(tiles, V.n_workers);
    const int ico = V.iconef;
    if (V.iconef) {   // iConEF-v1: the variants with a second state; -v2: with e~ as the values of a second draw
#define CONEF_FV_ICO(QV, CKV, HV)                                               \
    if (qkind == QV && ckind == CKV && (half != 0) == HV) {                     \
        if (V.iconef == 1)                                                      \
            k_flat_vec<QV, CKV, HV, 1><<<grid, kFvThreads, fv_smem_bytes(CKV, ico), s>>>(V, pfx);     \
        else if (QV != CONEF_Q_IDENTITY)                                        \
            k_flat_vec<QV == CONEF_Q_IDENTITY ? CONEF_Q_RANDK : QV, CKV, HV, 2><<<grid, kFvThreads, fv_smem_bytes(CKV, ico), s>>>(V, pfx); \
        else                                                                    \
            return cudaErrorNotSupported;                                       \
        return cudaSuccess;                                                     \
    }
#define CONEF_FV_ICO_Q(QV)                  \
    CONEF_FV_ICO(QV, CONEF_C_INT8, false)   \
    CONEF_FV_ICO(QV, CONEF_C_INT8, true)    \
    CONEF_FV_ICO(QV, CONEF_C_INT4, false)   \
    CONEF_FV_ICO(QV, CONEF_C_INT4, true)
        CONEF_FV_ICO_Q(CONEF_Q_IDENTITY)
        CONEF_FV_ICO_Q(CONEF_Q_RANDK)
        CONEF_FV_ICO_Q(CONEF_Q_RANDBLOCK)
#undef CONEF_FV_ICO_Q
#undef CONEF_FV_ICO
        return cudaErrorNotSupported;
    }
#define CONEF_FV_CASE(QV, CKV, HV)                                              \
    if (qkind == QV && ckind == CKV && (half != 0) == HV) {                     \
        k_flat_vec<QV, CKV, HV><<<grid, kFvThreads, fv_smem_bytes(CKV, ico), s>>>(V, pfx);            \
        return cudaSuccess;                                                     \
    }
#define CONEF_FV_Q(QV)                       \
    CONEF_FV_CASE(QV, CONEF_C_INT8, false)   \
    CONEF_FV_CASE(QV, CONEF_C_INT8, true)    \
    CONEF_FV_CASE(QV, CONEF_C_INT4, false)   \
    CONEF_FV_CASE(QV, CONEF_C_INT4, true)    \
    CONEF_FV_CASE(QV, CONEF_C_STOCHQUANT, false)
    CONEF_FV_Q(CONEF_Q_IDENTITY)
    CONEF_FV_Q(CONEF_Q_RANDK)
    CONEF_FV_Q(CONEF_Q_RANDBLOCK)
#undef CONEF_FV_Q
#undef CONEF_FV_CASE
    return cudaErrorNotSupported;
}

}  // namespace conef
