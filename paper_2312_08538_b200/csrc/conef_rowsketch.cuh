// Error state kept as a count sketch over matrix rows (Sec. 4.2.2, the tensor
// trick; the form the experiments of Sec. 5.4 run) with partial error feedback
// (Alg. 4).  One fused kernel per step does, for one worker:
//
//   e = decode(T)                       median over sketch rows of s_i(a) T_i[h_i(a)][b]
//   p = eta g + (1 - beta) e            Alg. 4 line 5 (beta = 0: Alg. 2 line 5)
//   Delta = Q(p), message               identity / shared random-k / rank-r residual
//   T' = beta T + sketch(p - Delta)     Alg. 4 line 9 in its linear form: no re-decode
//
// A scatter (one atomic per element and sketch row) is turned into a gather:
// the buckets of the matrix rows do not depend on the step, so the rows of
// every bucket are listed once when the context is created, and a CTA owns
// whole buckets: thread = one column, loop over the bucket's rows in ascending
// order, accumulate in a register (fp64, the old term first, rounded once), one
// store.  All loads of the gradient are row-contiguous and coalesced, every
// sketch entry is read and written once, and the result does not depend on
// scheduling.  HBM-bound: 4 B of gradient per element plus 8 v w / rows bytes
// of sketch.
#pragma once
#include "conef_kernels.cuh"
#include "conef_fast.cuh"

namespace conef {

#ifndef CONEF_RS_ROWS
#define CONEF_RS_ROWS 2
#endif
// Rows of a bucket whose loads are issued together.  Measured on the two-block GPT-2-XL list with a
// low-rank Q (pass 3 on the row sketch), on an earlier version of the loop body: 2 rows 1.05 ms,
// 4 rows 1.16 ms, 8 rows 1.24 ms (registers against occupancy); the current body with 2 rows takes
// 0.87 ms.  A per-thread ring of asynchronous copies 8 rows deep over the concatenated row lists,
// without and with the lists in shared memory, was also built: 0.86 and 0.96 ms with almost twice
// the instructions, so the simple form stays.
constexpr int kRsRows = CONEF_RS_ROWS;

// VEC columns per thread (4: 16-byte loads; needs cols % 4 == 0, for random-k cols % 32 == 0, and
// 16-byte aligned gradients; 1: any shape).  The CTA covers kRsThreads * VEC columns of kRsBuckets
// buckets of one sketch row.
// RK: 4 when the tensor's rank is exactly 4 (one 16-byte load per row of P_hat), else 8 (any rank).
template <int QK, int VEC, bool V1, int RK>
__device__ __forceinline__ void rs_body(const DevView &V, const LayerDesc &L, const int li, uint32_t local)
{
    const int worker = blockIdx.y;
    const uint32_t m = (uint32_t)L.cols, n = (uint32_t)L.rows, w = (uint32_t)L.w, d = (uint32_t)L.d;
    const int v = V.cs_rows;
    constexpr uint32_t CW = kRsThreads * VEC;               // columns per CTA
    const uint32_t slabs = (m + CW - 1) / CW;
    const uint32_t groups = (w + kRsBuckets - 1) / kRsBuckets;
    const uint32_t slab = local % slabs;
    local /= slabs;
    const uint32_t grp = local % groups;
    const uint32_t i = local / groups;                      // sketch row this CTA builds
    const int lane = threadIdx.x & 31;
    const uint32_t b = slab * CW + threadIdx.x * VEC;       // this thread's first column
    const bool colok = b < m;                               // VEC divides cols: all or none of the thread's columns exist

    const uint32_t *__restrict__ info = V.rs + L.rs_info_off;
    const uint32_t *__restrict__ bptr = V.rs + L.rs_ptr_off + (size_t)i * (w + 1);
    const uint32_t *__restrict__ brow = V.rs + L.rs_row_off + (size_t)i * n;
    const void *__restrict__ Told = V.state + worker * V.state_stride + L.a_off;
    void *__restrict__ Tnew = V.state_new + worker * V.state_stride + L.a_off;
    const bool th = V.scale_half != 0;   // the sketch is stored in binary16
    const float *__restrict__ g = V.grads[worker] + L.g_off;
    float *__restrict__ msg = V.msgv + worker * V.msgv_stride + L.msgv_off;

    const uint32_t *__restrict__ selbits = V.selbits + L.selbits_off;
    const uint32_t *__restrict__ uoff = V.unitoff + L.unitoff_off;
    const uint32_t *__restrict__ toff = V.tileoff + L.tileoff_off;   // slot = toff[tile] + uoff[unit] + rank
    uint32_t blk_start = 0;
    if (QK == CONEF_Q_RANDBLOCK)
        blk_start = randblock_start(stream_key(V.seed_q, (uint64_t)li, (uint64_t)V.step), d, (uint32_t)L.k);
    const int r = L.rank;
    float qreg[VEC][RK];   // Q_i[b..b+VEC-1][:], fixed for the thread
    const float *__restrict__ phat = V.phat + L.msgp_off;
    if (QK == CONEF_Q_LOWRANK) {
        const float *qi = V.msgq + worker * V.msgq_stride + L.msgq_off;
#pragma unroll
        for (int x = 0; x < VEC; ++x)
#pragma unroll
            for (int c = 0; c < RK; ++c)
                qreg[x][c] = (c < r && colok) ? qi[(size_t)(b + x) * r + c] : 0.f;
    }

    auto load_vec = [&](const float *p, float (&out)[VEC]) {
        if (VEC == 4) {
            const float4 t = *(const float4 *)p;
            out[0] = t.x; out[1 % VEC] = t.y; out[2 % VEC] = t.z; out[3 % VEC] = t.w;
        } else {
            out[0] = *p;
        }
    };
    auto load_t = [&](size_t idx, float (&out)[VEC]) {   // VEC entries of the old sketch
        if (VEC == 4) {
            float t4[4];
            rs_load4(Told, idx, th, t4);
            out[0] = t4[0]; out[1 % VEC] = t4[1]; out[2 % VEC] = t4[2]; out[3 % VEC] = t4[3];
        } else {
            out[0] = rs_load1(Told, idx, th);
        }
    };

    const uint32_t h_end = min(w, (grp + 1) * kRsBuckets);
    for (uint32_t h = grp * kRsBuckets; h < h_end; ++h) {
        const uint32_t lo = bptr[h], hi = bptr[h + 1];
        float told[VEC];
#pragma unroll
        for (int x = 0; x < VEC; ++x)
            told[x] = 0.f;
        if (colok)
            load_t(((size_t)i * w + h) * m + b, told);
        double acc[VEC];
#pragma unroll
        for (int x = 0; x < VEC; ++x)
            acc[x] = (double)__fmul_rn(V.beta, told[x]);
        for (uint32_t k0 = lo; k0 < hi; k0 += kRsRows) {
            uint32_t ent[kRsRows];
            float gv[kRsRows][VEC];
#pragma unroll
            for (int u = 0; u < kRsRows; ++u) {   // the loads of several rows are in flight together
                ent[u] = k0 + u < hi ? brow[k0 + u] : 0u;
#pragma unroll
                for (int x = 0; x < VEC; ++x)
                    gv[u][x] = 0.f;
                if (k0 + u < hi && colok)
                    load_vec(g + ((ent[u] & 0x7FFFFFFFu) * m + b), gv[u]);
            }
#pragma unroll
            for (int u = 0; u < kRsRows; ++u) {
                if (k0 + u >= hi)
                    break;
                const uint32_t a = ent[u] & 0x7FFFFFFFu;
                const uint32_t sgn = ent[u] & 0x80000000u;   // the sign bit of s_i(a)
                const uint32_t j = a * m + b;   // first element of the thread in this row
                // decode: with one sketch row the estimate is this bucket's own entry
                float e[VEC];
                if (V1) {
#pragma unroll
                    for (int x = 0; x < VEC; ++x)
                        e[x] = __uint_as_float(__float_as_uint(told[x]) ^ sgn);
                } else {
                    float est[VEC][7];
#pragma unroll
                    for (int y = 0; y < 7; ++y) {
                        float t[VEC];
#pragma unroll
                        for (int x = 0; x < VEC; ++x)
                            t[x] = 0.f;
                        uint32_t in = 0;
                        if (y < v) {
                            in = info[(size_t)y * n + a];
                            if (colok)
                                load_t(((size_t)y * w + (in & 0x7FFFFFFFu)) * m + b, t);
                        }
#pragma unroll
                        for (int x = 0; x < VEC; ++x)
                            est[x][y] = (in >> 31) ? -t[x] : t[x];
                    }
#pragma unroll
                    for (int x = 0; x < VEC; ++x)
                        e[x] = median_small(est[x], v);
                }
                float p[VEC], res[VEC];
#pragma unroll
                for (int x = 0; x < VEC; ++x)
                    p[x] = form_p(V, gv[u][x], e[x]);
                if (QK == CONEF_Q_IDENTITY) {
#pragma unroll
                    for (int x = 0; x < VEC; ++x) {
                        if (i == 0 && colok)
                            msg[j + x] = p[x];
                        res[x] = 0.f;
                    }
                } else if (QK == CONEF_Q_RANDBLOCK) {
#pragma unroll
                    for (int x = 0; x < VEC; ++x) {
                        const uint32_t slot = j + x - blk_start;
                        const bool sel = colok && slot < (uint32_t)L.k;
                        res[x] = sel ? 0.f : p[x];
                        if (i == 0 && sel) {
                            msg[slot] = p[x];
                            if (worker == 0)
                                V.idx[L.idx_off + slot] = j + x;
                        }
                    }
                } else if (QK == CONEF_Q_RANDK) {
                    // membership from the bitmap the selection left (bit i of word w: element 32 w + i);
                    // the thread's VEC elements lie in one word (VEC = 4: j is a multiple of 4)
                    const uint32_t word = colok ? selbits[j >> 5] : 0u;
                    bool sel[VEC];
                    int nsel = 0;
#pragma unroll
                    for (int x = 0; x < VEC; ++x) {
                        sel[x] = (word >> ((j + x) & 31u)) & 1u;
                        res[x] = sel[x] ? 0.f : p[x];
                        nsel += sel[x];
                    }
                    if (i == 0) {   // the CTAs of sketch row 0 meet every matrix row once: they write the message
                        uint32_t slot = 0;
                        if (VEC == 4) {
                            // cols % 32 == 0: a message unit is 8 consecutive lanes; exclusive prefix within them
                            int inc = nsel;
#pragma unroll
                            for (int o = 1; o < 8; o <<= 1) {
                                const int t = __shfl_up_sync(0xffffffffu, inc, o, 8);
                                if ((lane & 7) >= o)
                                    inc += t;
                            }
                            if (nsel)
                                slot = toff[j / kHistTile] + uoff[j >> 5] + (uint32_t)(inc - nsel);
                        } else {
                            // one element per thread: its rank within the unit from the unit's bitmap word
                            if (sel[0])
                                slot = toff[j / kHistTile] + uoff[j >> 5] + __popc(word & ((1u << (j & 31u)) - 1u));
                        }
#pragma unroll
                        for (int x = 0; x < VEC; ++x)
                            if (sel[x]) {
                                msg[slot] = p[x];   // message value, ascending index order
                                if (worker == 0)
                                    V.idx[L.idx_off + slot] = j + x;
                                ++slot;
                            }
                    }
                } else {
                    float ph[RK];
                    if (RK == 4) {
                        const float4 t = __ldg((const float4 *)(phat + (size_t)a * 4));
                        ph[0] = t.x; ph[1] = t.y; ph[2] = t.z; ph[3] = t.w;
                    } else {
#pragma unroll
                        for (int c = 0; c < RK; ++c)
                            ph[c] = c < r ? phat[(size_t)a * r + c] : 0.f;
                    }
#pragma unroll
                    for (int x = 0; x < VEC; ++x) {
                        res[x] = p[x];
#pragma unroll
                        for (int c = 0; c < RK; ++c)
                            if (RK == 4 || c < r)
                                res[x] = __fmaf_rn(-ph[c], qreg[x][c], res[x]);   // r = p - P_hat Q_i^T
                    }
                }
#pragma unroll
                for (int x = 0; x < VEC; ++x)
                    acc[x] += (double)__uint_as_float(__float_as_uint(res[x]) ^ sgn);   // s_i(a) * r, exact
            }
        }
        if (colok) {
            const size_t dst = ((size_t)i * w + h) * m + b;
            if (VEC == 4)
                rs_store4(Tnew, dst, th, (float)acc[0], (float)acc[1 % VEC], (float)acc[2 % VEC], (float)acc[3 % VEC]);
            else
                rs_store1(Tnew, dst, th, (float)acc[0]);
        }
    }
}

// rs_vec of a tensor chooses the body; both live in one kernel so that one launch covers the model
template <int QK, bool V1>   // V1: one sketch row (the usual setting), no median
__global__ void __launch_bounds__(kRsThreads) k_rowsketch(const __grid_constant__ DevView V)
{
    const int li = find_layer(V.pfx_rs, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const uint32_t local = blockIdx.x - V.pfx_rs[li];
    constexpr int RKG = QK == CONEF_Q_LOWRANK ? 8 : 4;   // the rank only matters to the low-rank Q
    if (L.rs_vec == 4 && V.rs_vec_ok) {
        if (QK == CONEF_Q_LOWRANK && L.rank == 4 && (L.msgp_off & 3) == 0)
            rs_body<QK, 4, V1, 4>(V, L, li, local);
        else
            rs_body<QK, 4, V1, RKG>(V, L, li, local);
    }
    else if (L.rs_vec == 4) {
        // 16-byte loads are not possible with this call's gradient pointers: the same tiles,
        // four scalar slabs per vector slab
        const uint32_t slabs4 = (uint32_t)((L.cols + kRsThreads * 4 - 1) / (kRsThreads * 4));
        const uint32_t slabs1 = (uint32_t)((L.cols + kRsThreads - 1) / kRsThreads);
        const uint32_t slab = local % slabs4, rest = local / slabs4;
        for (uint32_t s = slab * 4; s < min(slabs1, slab * 4 + 4); ++s)
            rs_body<QK, 1, V1, RKG>(V, L, li, rest * slabs1 + s);
    } else
        rs_body<QK, 1, V1, RKG>(V, L, li, local);
}

// ------------------------------------------------------------------ low-rank passes 1 and 2 on a row-sketch state
// The same bucket-major walk (one sketch row, four columns per thread), for tensors whose
// gradients allow 16-byte loads: every matrix row lies in exactly one bucket of sketch row 0, so
// the CTAs of (bucket group, column slab) meet every element once.
//   PASS 1: P_i[a][:] = sum_b p[a][b] Q_{t-1}[b][:]; a warp reduces its 128 columns by shuffles and
//           writes one partial row per (column slab, warp); k_rs_p1_combine adds them in order.
//   PASS 2: Q_i[b][:] = sum_a p[a][b] P_hat[a][:]; a thread accumulates its columns over the rows
//           of the group's buckets and writes one partial row per bucket group, summed in group
//           order by k_lr_pass2_reduce.
// Sums over rows and columns run in bucket order, not index order: like the other factor kernels
// they match the oracle to rounding (fp32, fixed order), not bit for bit.
template <int PASS, int RK>
__device__ __forceinline__ void rs12_body(const DevView &V, const int32_t *__restrict__ pfx, const int li, const LayerDesc &L)
{
    constexpr int VEC = 4;
    const int worker = blockIdx.y;
    const uint32_t m = (uint32_t)L.cols, n = (uint32_t)L.rows, w = (uint32_t)L.w;
    constexpr uint32_t CW = kRsThreads * VEC;
    const uint32_t slabs = (m + CW - 1) / CW;
    const uint32_t local = blockIdx.x - pfx[li];
    const uint32_t slab = local % slabs, grp = local / slabs;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t b = slab * CW + threadIdx.x * VEC;
    const bool colok = b < m;
    const uint32_t *__restrict__ bptr = V.rs + L.rs_ptr_off;    // sketch row 0
    const uint32_t *__restrict__ brow = V.rs + L.rs_row_off;
    const void *__restrict__ T = V.state + worker * V.state_stride + L.a_off;
    const bool th = V.scale_half != 0;
    const float *__restrict__ g = V.grads[worker] + L.g_off;
    const float *__restrict__ phat = V.phat + L.msgp_off;
    const int r = L.rank;

    float q[VEC][RK];   // pass 1: Q_{t-1}[b..b+3][:]; pass 2: accumulators of Q_i[b..b+3][:]
#pragma unroll
    for (int x = 0; x < VEC; ++x)
#pragma unroll
        for (int c = 0; c < RK; ++c)
            q[x][c] = (PASS == 1 && colok && c < r) ? V.qprev[L.msgq_off + (size_t)(b + x) * r + c] : 0.f;
    float *__restrict__ ppart = V.ppart + worker * V.ppart_stride + L.pp_off +
                                (size_t)(slab * (kRsThreads / 32) + warp) * n * r;

    const uint32_t h_end = min(w, (grp + 1) * kRsBuckets);
    for (uint32_t h = grp * kRsBuckets; h < h_end; ++h) {
        const uint32_t lo = bptr[h], hi = bptr[h + 1];
        float4 told = make_float4(0.f, 0.f, 0.f, 0.f);
        if (colok) {
            float t4[4];
            rs_load4(T, (size_t)h * m + b, th, t4);
            told = make_float4(t4[0], t4[1], t4[2], t4[3]);
        }
        for (uint32_t k0 = lo; k0 < hi; k0 += kRsRows) {
            uint32_t ent[kRsRows];
            float4 gv[kRsRows];
#pragma unroll
            for (int u = 0; u < kRsRows; ++u) {
                ent[u] = k0 + u < hi ? brow[k0 + u] : 0u;
                gv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (k0 + u < hi && colok)
                    gv[u] = *(const float4 *)(g + ((ent[u] & 0x7FFFFFFFu) * m + b));
            }
#pragma unroll
            for (int u = 0; u < kRsRows; ++u) {
                if (k0 + u >= hi)
                    break;
                const uint32_t a = ent[u] & 0x7FFFFFFFu, sgn = ent[u] & 0x80000000u;
                const float tv[VEC] = {told.x, told.y, told.z, told.w};
                const float gq[VEC] = {gv[u].x, gv[u].y, gv[u].z, gv[u].w};
                float p[VEC];
#pragma unroll
                for (int x = 0; x < VEC; ++x)
                    p[x] = form_p(V, gq[x], __uint_as_float(__float_as_uint(tv[x]) ^ sgn));
                if (PASS == 2) {
                    float ph[RK];
                    if (RK == 4) {
                        const float4 t = __ldg((const float4 *)(phat + (size_t)a * 4));
                        ph[0] = t.x; ph[1] = t.y; ph[2] = t.z; ph[3] = t.w;
                    } else {
#pragma unroll
                        for (int c = 0; c < RK; ++c)
                            ph[c] = c < r ? phat[(size_t)a * r + c] : 0.f;
                    }
#pragma unroll
                    for (int x = 0; x < VEC; ++x)
#pragma unroll
                        for (int c = 0; c < RK; ++c)
                            q[x][c] = __fmaf_rn(p[x], ph[c], q[x][c]);
                } else {
                    float pr[RK];
#pragma unroll
                    for (int c = 0; c < RK; ++c) {
                        pr[c] = 0.f;
#pragma unroll
                        for (int x = 0; x < VEC; ++x)
                            pr[c] = __fmaf_rn(p[x], q[x][c], pr[c]);
                    }
                    warp_reduce_many<RK>(pr, lane);
                    // total of column idx sits in the lanes whose bits below `plain` are zero
                    int idx = 0, hh = RK, plain = 32;
#pragma unroll
                    for (int o = 16; o >= 1; o >>= 1)
                        if (hh > 1) {
                            hh >>= 1;
                            if (lane & o)
                                idx += hh;
                            plain = o;
                        }
                    if ((lane & (plain - 1)) == 0 && idx < r)
                        ppart[(size_t)a * r + idx] = pr[0];
                }
            }
        }
    }
    if (PASS == 2 && colok) {
        float *__restrict__ part = V.part + worker * V.part_stride + L.part_off + ((size_t)grp * m + b) * r;
#pragma unroll
        for (int x = 0; x < VEC; ++x)
#pragma unroll
            for (int c = 0; c < RK; ++c)
                if (c < r)
                    part[(size_t)x * r + c] = q[x][c];
    }
}

template <int PASS>
__global__ void __launch_bounds__(kRsThreads) k_rs_pass12(const __grid_constant__ DevView V, const int32_t *__restrict__ pfx)
{
    const int li = find_layer(pfx, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    if (L.rank == 4 && (L.msgp_off & 3) == 0)
        rs12_body<PASS, 4>(V, pfx, li, L);
    else
        rs12_body<PASS, 8>(V, pfx, li, L);
}

// P_i[a][c] = sum over the (column slab, warp) partials of pass 1, in slab-major order
__global__ void __launch_bounds__(256) k_rs_p1_combine(const __grid_constant__ DevView V, const int32_t *__restrict__ pfx)
{
    const int li = find_layer(pfx, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int worker = blockIdx.y;
    const int64_t nr = L.rows * L.rank;
    const int64_t qi = (int64_t)(blockIdx.x - pfx[li]) * 256 + threadIdx.x;
    if (qi >= nr)
        return;
    const float *__restrict__ ppart = V.ppart + worker * V.ppart_stride + L.pp_off;
    float acc = ppart[qi];
    for (int j = 1; j < L.f_j; ++j)
        acc = __fadd_rn(acc, ppart[(size_t)j * nr + qi]);
    V.msgp[worker * V.msgp_stride + L.msgp_off + qi] = acc;
}

}  // namespace conef
