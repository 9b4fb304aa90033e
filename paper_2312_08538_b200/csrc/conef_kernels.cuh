// Generic sm_100a kernels of the ConEF step.  They are correct for every
// tensor shape and alignment (scalar global accesses only); the tuned kernels
// in conef_fast.cuh take over for the large, aligned tensors.
//
// Arithmetic contract (what makes codes and indices reproducible bit for bit):
// fp32 with explicit __fmaf_rn / __fmul_rn / __fdiv_rn, no fast-math, no
// flush-to-zero; the file is compiled with -fmad=false so that the compiler
// fuses nothing by itself.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <float.h>

#include "conef_internal.h"
#include "conef_hash.cuh"

namespace conef {

// last tensor l with pfx[l] <= bid (prefix tables have n + 1 entries)
__device__ __forceinline__ int find_layer(const int32_t *__restrict__ pfx, int n, int bid)
{
    int lo = 0, hi = n;  // invariant: pfx[lo] <= bid < pfx[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (__ldg(pfx + mid) <= bid)
            lo = mid;
        else
            hi = mid;
    }
    return lo;
}

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        v = __fadd_rn(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// ------------------------------------------------------------------ decode (S1)
__device__ __forceinline__ float load_scale(const uint8_t *__restrict__ b, int64_t blk, int half)
{
    if (half)
        return __half2float(__ushort_as_half(((const unsigned short *)b)[blk]));
    return ((const float *)b)[blk];
}

__device__ __forceinline__ float median_small(float *x, int v)
{
    if (v == 1)
        return x[0];
    if (v == 3)
        return fmaxf(fminf(x[0], x[1]), fminf(fmaxf(x[0], x[1]), x[2]));
    if (v == 5) {
        // median of five by a fixed exchange network
        float a = fminf(x[0], x[1]), b = fmaxf(x[0], x[1]);
        float c = fminf(x[2], x[3]), d = fmaxf(x[2], x[3]);
        float lo = fmaxf(a, c);   // the smaller of the two minima cannot be the median
        float hi = fminf(b, d);   // nor the larger of the two maxima
        float e = x[4];
        // median of {lo, hi, e} together with the leftover middle pair
        float m1 = fminf(lo, hi), m2 = fmaxf(lo, hi);
        return fmaxf(m1, fminf(m2, e));
    }
    // v == 7: insertion sort
    for (int a = 1; a < v; ++a) {
        float val = x[a];
        int b = a - 1;
        while (b >= 0 && x[b] > val) {
            x[b + 1] = x[b];
            --b;
        }
        x[b + 1] = val;
    }
    return x[v / 2];
}

struct SketchKeys {
    uint64_t st[7];
};
__device__ __forceinline__ SketchKeys sketch_keys(uint64_t seed, int tensor, int v)
{
    SketchKeys k;
#pragma unroll
    for (int i = 0; i < 7; ++i)
        k.st[i] = i < v ? stream_key(seed, (uint64_t)tensor, (uint64_t)i) : 0;
    return k;
}

// Count sketch applied run by run (cs_chunk > 0): the window [lo, lo + width) of every sketch row
// that the run of element j owns.  Runs are cs_chunk consecutive elements, the last one also takes
// the remainder; windows are cut in proportion to the elements.  One run: the whole row.
__device__ __forceinline__ void sketch_window_of_run(uint32_t c, uint32_t nc, uint32_t chunk, uint32_t d, uint32_t w,
                                                     uint32_t &lo, uint32_t &width)
{
    const uint64_t b0 = c == 0 ? 0ull : (uint64_t)w * ((uint64_t)c * chunk) / d;          // w c E <= w d < 2^64
    const uint64_t b1 = c == nc - 1 ? (uint64_t)w : (uint64_t)w * ((uint64_t)(c + 1) * chunk) / d;
    lo = (uint32_t)b0;
    width = (uint32_t)(b1 - b0);
}
__device__ __forceinline__ void sketch_window(const DevView &V, const LayerDesc &L, uint32_t j, uint32_t &lo,
                                              uint32_t &width)
{
    lo = 0;
    width = (uint32_t)L.w;
    if (V.cs_chunk > 0) {
        const uint32_t chunk = (uint32_t)V.cs_chunk, d = (uint32_t)L.d;
        uint32_t nc = d / chunk;
        nc = nc < 1 ? 1 : nc;
        uint32_t c = j / chunk;
        c = c > nc - 1 ? nc - 1 : c;
        if (nc > 1)
            sketch_window_of_run(c, nc, chunk, d, (uint32_t)L.w, lo, width);
    }
}

// Alg. 2 line 5, p = eta g + e; with partial error feedback (Alg. 4 line 5) p = eta g + (1-beta) e,
// the product rounded first.  V.omb is 1 for beta = 0, and 1 * e is e.
__device__ __forceinline__ float form_p(const DevView &V, float g, float e)
{
    return __fmaf_rn(V.lr, g, __fmul_rn(V.omb, e));
}
// whether this codec keeps the second state of iConEF-v1 (Alg. 3)
template <int CK>
__device__ __forceinline__ bool has_second(const DevView &V)
{
    return (CK == CONEF_C_IDENTITY || CK == CONEF_C_INT8 || CK == CONEF_C_INT4) && V.iconef == 1;
}

// iConEF-v2: the second application of Q in a step draws from the stream of step t + 2^62
constexpr int64_t kSecondDraw = 1ll << 62;
// Whether element j belongs to a stored draw of Q (membership bitmap, unit and tile offsets as the
// selection kernels leave them; or the block of random-block-k), and its slot among the k values.
template <int QK>
__device__ __forceinline__ bool draw_member(const LayerDesc &L, const uint32_t *__restrict__ selbits,
                                            const uint32_t *__restrict__ unitoff,
                                            const uint32_t *__restrict__ tileoff, uint32_t blk_start, uint32_t j,
                                            uint32_t &slot)
{
    if (QK == CONEF_Q_RANDBLOCK) {
        slot = j - blk_start;   // wraps to a large value below the block
        return slot < (uint32_t)L.k;
    }
    const uint32_t wi = j >> 5, word = selbits[L.selbits_off + wi];
    if (!((word >> (j & 31u)) & 1u))
        return false;
    const int unit_shift = 31 - __clz(L.unit);
    const uint32_t first = (j >> unit_shift) << (unit_shift - 5);   // first bitmap word of the unit
    uint32_t before = __popc(word & ((1u << (j & 31u)) - 1u));
    for (uint32_t x = first; x < wi; ++x)
        before += __popc(selbits[L.selbits_off + x]);
    slot = tileoff[L.tileoff_off + j / kHistTile] + unitoff[L.unitoff_off + (j >> unit_shift)] + before;
    return true;
}

// e_j of one element from a worker's stored state (Alg. 2 line 5, decode).
// Row-sketch entries are fp32 or, with a binary16 sketch, halves (stored saturated to the finite
// half range, rounded to nearest even).  idx counts entries.
__device__ __forceinline__ float rs_load1(const void *T, size_t idx, bool half)
{
    return half ? __half2float(((const __half *)T)[idx]) : ((const float *)T)[idx];
}
__device__ __forceinline__ void rs_load4(const void *T, size_t idx, bool half, float (&out)[4])
{
    if (half) {
        const uint2 raw = *(const uint2 *)((const __half *)T + idx);
        const float2 a = __half22float2(*(const __half2 *)&raw.x), b = __half22float2(*(const __half2 *)&raw.y);
        out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
    } else {
        const float4 t = *(const float4 *)((const float *)T + idx);
        out[0] = t.x; out[1] = t.y; out[2] = t.z; out[3] = t.w;
    }
}
__device__ __forceinline__ unsigned short rs_to_half(float f)
{
    f = f > 65504.0f ? 65504.0f : f;
    f = f < -65504.0f ? -65504.0f : f;
    return __half_as_ushort(__float2half_rn(f));
}
__device__ __forceinline__ void rs_store1(void *T, size_t idx, bool half, float f)
{
    if (half)
        ((unsigned short *)T)[idx] = rs_to_half(f);
    else
        ((float *)T)[idx] = f;
}
__device__ __forceinline__ void rs_store4(void *T, size_t idx, bool half, float a, float b, float c, float d)
{
    if (half) {
        uint2 raw;
        raw.x = (uint32_t)rs_to_half(a) | ((uint32_t)rs_to_half(b) << 16);
        raw.y = (uint32_t)rs_to_half(c) | ((uint32_t)rs_to_half(d) << 16);
        *(uint2 *)((unsigned short *)T + idx) = raw;
    } else {
        *(float4 *)((float *)T + idx) = make_float4(a, b, c, d);
    }
}

// second: the state q of iConEF (Alg. 3) instead of the first one.
template <int CK>
__device__ __forceinline__ float decode_elem(const DevView &V, const LayerDesc &L,
                                             const uint8_t *__restrict__ st, uint32_t j,
                                             const SketchKeys &keys, bool second = false)
{
    const int64_t aoff = second ? L.a2_off : L.a_off, boff = second ? L.b2_off : L.b_off;
    if (CK == CONEF_C_IDENTITY)
        return ((const float *)(st + aoff))[j];
    if (CK == CONEF_C_INT8) {
        int c = ((const signed char *)(st + aoff))[j];
        return __fmul_rn((float)c, load_scale(st + boff, j / (uint32_t)L.unit, V.scale_half));
    }
    if (CK == CONEF_C_INT4) {
        unsigned byte = (st + aoff)[j >> 1];
        int nib = (j & 1) ? (byte >> 4) : (byte & 0xF);
        int c = (nib ^ 8) - 8;
        return __fmul_rn((float)c, load_scale(st + boff, j / (uint32_t)L.unit, V.scale_half));
    }
    if (CK == CONEF_C_STOCHQUANT) {
        const int c = V.sq_wide ? (int)((const short *)(st + L.a_off))[j] : (int)((const signed char *)(st + L.a_off))[j];
        return __fmul_rn((float)c, ((const float *)(st + L.b_off))[j / (uint32_t)L.unit]);
    }
    if (CK == CONEF_C_ROWSKETCH) {
        // row sketch: median over sketch rows of s_i(a) * T_i[h_i(a)][b]; buckets and signs of
        // the matrix rows come from the table built when the context was created
        const void *T = st + L.a_off;
        const bool th = V.scale_half != 0;
        const uint32_t m = (uint32_t)L.cols, a = j / m, b = j - a * m;
        const uint32_t *info = V.rs + L.rs_info_off;
        float est[7];
#pragma unroll
        for (int i = 0; i < 7; ++i) {
            if (i < V.cs_rows) {
                const uint32_t in = info[(int64_t)i * L.rows + a];
                const float t = rs_load1(T, (size_t)(((int64_t)i * L.w + (in & 0x7FFFFFFFu)) * m + b), th);
                est[i] = (in >> 31) ? -t : t;
            } else
                est[i] = 0.f;
        }
        return median_small(est, V.cs_rows);
    }
    // count sketch: median over rows of s_i(j) * S[i][h_i(j)]
    const float *S = (const float *)(st + L.a_off);
    float est[7];
    uint32_t lo, width;
    sketch_window(V, L, j, lo, width);
#pragma unroll
    for (int i = 0; i < 7; ++i) {
        if (i < V.cs_rows) {
            uint64_t u = h64(keys.st[i], j);
            uint64_t b = lo + (((u >> 32) * (uint64_t)width) >> 32);
            float s = S[(int64_t)i * L.w + (int64_t)b];
            est[i] = (u & 1) ? -s : s;
        } else
            est[i] = 0.f;
    }
    return median_small(est, V.cs_rows);
}

// ------------------------------------------------------------------ 1-D pass-through
__global__ void __launch_bounds__(256) k_passthrough(const __grid_constant__ DevView V)
{
    const int li = find_layer(V.pfx_pass, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int worker = blockIdx.y;
    const int64_t j0 = (int64_t)(blockIdx.x - V.pfx_pass[li]) * kPassTile;
    const float *__restrict__ g = V.grads[worker] + L.g_off;
    float *__restrict__ out = V.msg1d + worker * V.msg1d_stride + L.msg1d_off;
    for (int q = threadIdx.x; q < kPassTile; q += 256) {
        int64_t j = j0 + q;
        if (j < L.d)
            out[j] = __fmul_rn(V.lr, g[j]);
    }
}

// ------------------------------------------------------------------ random-k selection (S3a)
// The index set S_t = the k smallest keys (hash32(j) << 32 | j).  Membership
// is "key(j) <= tau"; tau is found by a three-level radix select on the hash
// (11 + 11 + 10 bits) followed by a tie-break on the index among the few
// elements that share the threshold's hash.  No memory traffic: hashes are
// recomputed.  All of it depends on (seed, tensor, step) only and is shared
// by the N workers.

template <int LEVEL>
__global__ void __launch_bounds__(256) k_rk_hist(const __grid_constant__ DevView V)
{
    __shared__ uint32_t hist[kHistBins];
    const int li = find_layer(V.pfx_hist, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    uint32_t *sel = V.sel + L.sel_off;
    const uint32_t prefix = sel[3 * kHistBins + SEL_PREFIX];
    for (int b = threadIdx.x; b < kHistBins; b += 256)
        hist[b] = 0;
    __syncthreads();
    const uint64_t st = stream_key(V.seed_q, (uint64_t)li, (uint64_t)V.step);
    const int64_t j0 = (int64_t)(blockIdx.x - V.pfx_hist[li]) * kHistTile;
    uint32_t *stw = sel + 3 * kHistBins;
    uint32_t *cand = V.cand + 2 * L.cand_off;
    auto visit = [&](uint32_t h, uint32_t j) {
        if (LEVEL == 0)
            atomicAdd(&hist[h >> 21], 1u);
        else if (LEVEL == 1) {
            if ((h >> 21) == prefix) {
                atomicAdd(&hist[(h >> 10) & 2047u], 1u);
                // the later levels only look at these elements (one in 2048): keep them
                const uint32_t pos = atomicAdd(&stw[SEL_NCAND], 1u);
                if (pos < (uint32_t)L.cand_cap) {
                    cand[2 * pos] = h;
                    cand[2 * pos + 1] = j;
                }
            }
        } else if (LEVEL == 2) {
            if ((h >> 10) == prefix)
                atomicAdd(&hist[h & 1023u], 1u);
        } else {  // LEVEL 3: collect the elements whose hash equals the threshold's
            if (h == stw[SEL_TAU_HI]) {
                uint32_t pos = atomicAdd(&stw[SEL_NTIES], 1u);
                if (pos < (uint32_t)kMaxTies)
                    stw[16 + pos] = j;
            }
        }
    };
    // levels 2 and 3 read the candidate list where it held everything, and hash all elements again
    // where it overflowed
    const uint32_t ncand = LEVEL >= 2 ? stw[SEL_NCAND] : 0u;
    if (LEVEL >= 2 && ncand <= (uint32_t)L.cand_cap) {
        for (int q = threadIdx.x; q < kHistTile; q += 256) {
            const int64_t x = j0 + q;
            if (x >= (int64_t)ncand)
                break;
            visit(cand[2 * x], cand[2 * x + 1]);
        }
    } else {
        for (int q = threadIdx.x; q < kHistTile; q += 256) {
            int64_t j = j0 + q;
            if (j >= L.d)
                break;
            visit(hash32(st, (uint64_t)j), (uint32_t)j);
        }
    }
    if (LEVEL < 3) {
        __syncthreads();
        uint32_t *gh = sel + LEVEL * kHistBins;
        for (int b = threadIdx.x; b < kHistBins; b += 256)
            if (hist[b])
                atomicAdd(&gh[b], hist[b]);
    }
}

// one CTA of 1024 threads per random-k tensor: pick the bin that holds the
// wanted rank, or (LEVEL 3) the tie-breaking index
template <int LEVEL>
__global__ void __launch_bounds__(1024) k_rk_pick(const __grid_constant__ DevView V)
{
    __shared__ uint32_t wsum[32];
    __shared__ uint32_t ties[kMaxTies];
    const int li = find_layer(V.pfx_gs, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    uint32_t *sel = V.sel + L.sel_off;
    uint32_t *stw = sel + 3 * kHistBins;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (LEVEL < 3) {
        const uint32_t remain = (LEVEL == 0) ? (uint32_t)L.k : stw[SEL_REMAIN];
        const uint32_t *gh = sel + LEVEL * kHistBins;
        // each thread owns two adjacent bins; inclusive scan over threads
        uint32_t c0 = gh[2 * tid], c1 = gh[2 * tid + 1];
        uint32_t mine = c0 + c1, inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o)
                inc += n;
        }
        if (lane == 31)
            wsum[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            uint32_t w = wsum[lane], winc = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                uint32_t n = __shfl_up_sync(0xffffffffu, winc, o);
                if (lane >= o)
                    winc += n;
            }
            wsum[lane] = winc - w;  // exclusive
        }
        __syncthreads();
        const uint32_t before = wsum[warp] + inc - mine;  // elements in bins below 2*tid
        __syncthreads();
        if (tid == 0)
            wsum[0] = 0xffffffffu;
        __syncthreads();
        // the wanted rank (1-based "remain") lies in the first bin whose inclusive count reaches it
        if (before < remain && remain <= before + mine) {
            uint32_t bin, rem;
            if (remain <= before + c0) {
                bin = 2 * tid;
                rem = remain - before;
            } else {
                bin = 2 * tid + 1;
                rem = remain - before - c0;
            }
            const uint32_t prefix = (LEVEL == 0) ? 0u : stw[SEL_PREFIX];
            if (LEVEL == 0)
                stw[SEL_PREFIX] = bin;
            else if (LEVEL == 1)
                stw[SEL_PREFIX] = (prefix << 11) | bin;
            else
                stw[SEL_TAU_HI] = (prefix << 10) | bin;
            stw[SEL_REMAIN] = rem;
            wsum[0] = 0;
        }
        __syncthreads();
        if (tid == 0 && wsum[0] != 0)
            atomicOr(V.status, ST_SELECT_FAILED);
    } else {
        const uint32_t n = stw[SEL_NTIES], remain = stw[SEL_REMAIN];
        if (n > (uint32_t)kMaxTies || remain > n || remain == 0) {
            if (tid == 0) {
                atomicOr(V.status, ST_TIE_OVERFLOW);
                stw[SEL_TAU_LO] = 0xffffffffu;
            }
            return;
        }
        if ((uint32_t)tid < n)
            ties[tid] = stw[16 + tid];
        __syncthreads();
        if ((uint32_t)tid < n) {
            uint32_t me = ties[tid], rank = 0;
            for (uint32_t q = 0; q < n; ++q)
                rank += ties[q] < me;
            if (rank == remain - 1)
                stw[SEL_TAU_LO] = me;  // the remain-th smallest index among the ties
        }
    }
}


// count the selected coordinates of every work unit; the exclusive prefix within the CTA's tile of
// kHistTile elements goes to unitoff, the tile's total to tileoff (scanned by k_rk_scan):
// message slot of an element = tileoff[tile] + unitoff[unit] + its rank within the unit
__global__ void __launch_bounds__(256) k_rk_count(const __grid_constant__ DevView V)
{
    __shared__ uint32_t cnts[kHistTile / 32];
    const int li = find_layer(V.pfx_hist, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const uint32_t *stw = V.sel + L.sel_off + 3 * kHistBins;
    const uint32_t tau_hi = stw[SEL_TAU_HI], tau_lo = stw[SEL_TAU_LO];
    const uint64_t st = stream_key(V.seed_q, (uint64_t)li, (uint64_t)V.step);
    const int64_t tile = blockIdx.x - V.pfx_hist[li];
    const int64_t j0 = tile * kHistTile;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int U = L.unit, nu = kHistTile / U;   // units per tile: 32 .. 256
    for (int u = warp; u < nu; u += 8) {
        const int64_t base = j0 + (int64_t)u * U;
        int cnt = 0;
        if (base < L.d)
            for (int q = lane; q < U; q += 32) {
                const int64_t j = base + q;
                const bool in = j < L.d && rk_selected(hash32(st, (uint64_t)j), (uint32_t)j, tau_hi, tau_lo);
                // membership bitmap, read by the step kernels of all workers instead of hashing again
                const uint32_t word = __ballot_sync(0xffffffffu, in);
                if (lane == 0)
                    V.selbits[L.selbits_off + ((base + q) >> 5)] = word;
                cnt += in;
            }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
            cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        if (lane == 0)
            cnts[u] = (uint32_t)cnt;
    }
    __syncthreads();
    if (warp == 0) {
        // exclusive scan of up to 256 counts: 8 per lane, then across lanes
        const int per = nu / 32;   // 1 .. 8
        uint32_t loc[8], sum = 0;
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            loc[x] = x < per ? cnts[lane * per + x] : 0u;
            sum += loc[x];
        }
        uint32_t inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o)
                inc += t;
        }
        uint32_t run = inc - sum;
        const int64_t unit0 = j0 / U;
#pragma unroll
        for (int x = 0; x < 8; ++x)
            if (x < per) {
                if (unit0 + lane * per + x < L.nunits)
                    V.unitoff[L.unitoff_off + unit0 + lane * per + x] = run;
                run += loc[x];
            }
        if (lane == 31)
            V.tileoff[L.tileoff_off + tile] = inc;
    }
}

// exclusive scan of the per-tile totals, in place; one CTA per tensor
__global__ void __launch_bounds__(1024) k_rk_scan(const __grid_constant__ DevView V)
{
    __shared__ uint32_t wsum[32];
    __shared__ uint32_t carry_s;
    const int li = find_layer(V.pfx_gs, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    if (!L.compressed)
        return;
    uint32_t *cnt = V.tileoff + L.tileoff_off;
    const int64_t ntiles = (L.d + kHistTile - 1) / kHistTile;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0)
        carry_s = 0;
    __syncthreads();
    for (int64_t base = 0; base < ntiles; base += 1024) {
        int64_t u = base + tid;
        uint32_t v = u < ntiles ? cnt[u] : 0u, inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o)
                inc += n;
        }
        if (lane == 31)
            wsum[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            uint32_t w = wsum[lane], winc = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                uint32_t n = __shfl_up_sync(0xffffffffu, winc, o);
                if (lane >= o)
                    winc += n;
            }
            wsum[lane] = winc - w;
        }
        __syncthreads();
        const uint32_t carry = carry_s;
        if (u < ntiles)
            cnt[u] = carry + wsum[warp] + inc - v;
        __syncthreads();
        if (tid == 1023)
            carry_s = carry + wsum[31] + inc;
        __syncthreads();
    }
    if (tid == 0 && carry_s != (uint32_t)L.k)
        atomicOr(V.status, ST_COUNT_MISMATCH);
}

// ------------------------------------------------------------------ quantiser (S5, C1)
// scale and reciprocal of one block from its absmax; zero block when the
// stored scale is not >= FLT_MIN
__device__ __forceinline__ void quant_scale(float amax, int qmax, int half, float &s, float &inv,
                                            unsigned short &hbits)
{
    s = __fdiv_rn(amax, (float)qmax);
    hbits = 0;
    if (half) {
        s = fminf(s, 65504.0f);
        __half h = __float2half_rn(s);
        hbits = __half_as_ushort(h);
        s = __half2float(h);
    }
    if (!(s >= FLT_MIN)) {
        s = 0.f;
        inv = 0.f;
        hbits = 0;
    } else
        inv = __fdiv_rn(1.0f, s);
}
__device__ __forceinline__ int quant_code(float r, float inv, int qmax)
{
    int c = __float2int_rn(__fmul_rn(r, inv));  // NaN -> 0, out of range saturates
    return max(-qmax, min(qmax, c));
}

// ------------------------------------------------------------------ fused flat step
// One warp per work unit (= quantisation block of 32..256 elements); a lane
// owns unit/32 consecutive elements.  Covers S1+S2+S3+S4+S5 for Q = identity
// and Q = random-k, and S1+S2+S4+S5 ("pass 3") for the low-rank Q.
template <int QK, int CK>
__global__ void __launch_bounds__(kFlatThreads) k_flat(const __grid_constant__ DevView V)
{
    const int li = find_layer(V.pfx_flat, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int worker = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int U = L.unit, E = U >> 5;
    const uint32_t d = (uint32_t)L.d, m = (uint32_t)L.cols;
    uint8_t *st = V.state + worker * V.state_stride;
    const float *__restrict__ g = V.grads[worker] + L.g_off;
    const int64_t unit0 = (int64_t)(blockIdx.x - V.pfx_flat[li]) * kFlatUnitsPerCta;
    const int qmax = (CK == CONEF_C_INT8) ? 127 : 7;

    SketchKeys keys = {};
    if (CK == CONEF_C_COUNTSKETCH)
        keys = sketch_keys(V.seed_c, li, V.cs_rows);
    uint32_t blk_start = 0;
    if (QK == CONEF_Q_RANDBLOCK)
        blk_start = randblock_start(stream_key(V.seed_q, (uint64_t)li, (uint64_t)V.step), d, (uint32_t)L.k);
    float *__restrict__ msg = V.msgv + worker * V.msgv_stride + L.msgv_off;
    // iConEF-v2: e~ is the k values that the second draw of Q kept; the stored state is q
    constexpr int QD = QK == CONEF_Q_RANDBLOCK ? CONEF_Q_RANDBLOCK : CONEF_Q_RANDK;
    const bool v2 = (QK == CONEF_Q_RANDK || QK == CONEF_Q_RANDBLOCK) && V.iconef == 2;
    const float *__restrict__ ev_old = V.ev_old + worker * V.msgv_stride + L.msgv_off;
    float *__restrict__ ev_new = V.ev_new + worker * V.msgv_stride + L.msgv_off;
    uint32_t blk_startA = 0, blk_startB = 0;
    if (QK == CONEF_Q_RANDBLOCK && v2) {
        blk_startA = randblock_start(stream_key(V.seed_q, (uint64_t)li, (uint64_t)(V.ev_step + kSecondDraw)), d, (uint32_t)L.k);
        blk_startB = randblock_start(stream_key(V.seed_q, (uint64_t)li, (uint64_t)(V.step + kSecondDraw)), d, (uint32_t)L.k);
    }
    const int r = L.rank;
    const float *__restrict__ phat = V.phat + L.msgp_off;
    const float *__restrict__ qi = V.msgq + worker * V.msgq_stride + L.msgq_off;

    for (int u = warp; u < kFlatUnitsPerCta; u += kFlatThreads / 32) {
        const int64_t unit = unit0 + u;
        if (unit >= L.nunits)
            break;
        const uint32_t base = (uint32_t)(unit * U) + lane * E;
        // iConEF-v2 with random-k: membership bits of this thread's elements in the two second draws
        // (a thread's E <= 8 elements share one bitmap word) and the slot of its first member, by
        // the same prefix over the unit's lanes as the message slots below
        uint32_t bitsA = 0, bitsB = 0, slotA = 0, slotB = 0;
        if (QK == CONEF_Q_RANDK && v2) {
            if (base < d) {
                const uint32_t emask = (1u << E) - 1u, wi = L.selbits_off + (base >> 5), sh = base & 31u;
                bitsA = V.ev_valid ? (V.selbitsA[wi] >> sh) & emask : 0u;
                bitsB = (V.selbitsB[wi] >> sh) & emask;
            }
            const int cA = __popc(bitsA), cB = __popc(bitsB);
            int incA = cA, incB = cB;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int nA = __shfl_up_sync(0xffffffffu, incA, o), nB = __shfl_up_sync(0xffffffffu, incB, o);
                if (lane >= o) {
                    incA += nA;
                    incB += nB;
                }
            }
            const int64_t tile = (unit * U) / kHistTile;
            if (V.ev_valid)
                slotA = V.tileoffA[L.tileoff_off + tile] + V.unitoffA[L.unitoff_off + unit] + (uint32_t)(incA - cA);
            slotB = V.tileoffB[L.tileoff_off + tile] + V.unitoffB[L.unitoff_off + unit] + (uint32_t)(incB - cB);
        }
        float val[8], ekeep[8];
        bool selq[8];
        int nsel = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            val[q] = 0.f;
            ekeep[q] = 0.f;
            selq[q] = false;
            const uint32_t j = base + q;
            if (q < E && j < d) {
                float e;
                if (v2) {
                    e = 0.f;
                    if (QK == CONEF_Q_RANDK) {
                        if ((bitsA >> q) & 1u)
                            e = ev_old[slotA + (uint32_t)__popc(bitsA & ((1u << q) - 1u))];
                    } else {
                        uint32_t sl;
                        if (V.ev_valid && draw_member<QD>(L, V.selbitsA, V.unitoffA, V.tileoffA, blk_startA, j, sl))
                            e = ev_old[sl];
                    }
                } else
                    e = decode_elem<CK>(V, L, st, j, keys);
                float p = form_p(V, g[j], e);  // Alg. 2 line 5
                if (has_second<CK>(V))
                    p = __fadd_rn(p, decode_elem<CK>(V, L, st, j, keys, true));  // Alg. 3 line 5: + q
                else if (v2)
                    p = __fadd_rn(p, decode_elem<CK>(V, L, st, j, keys));        // the same line; q is the stored state
                ekeep[q] = e;
                if (QK == CONEF_Q_IDENTITY) {
                    msg[j] = p;
                    val[q] = 0.f;
                } else if (QK == CONEF_Q_RANDK) {
                    selq[q] = (V.selbits[L.selbits_off + (j >> 5)] >> (j & 31u)) & 1u;   // bitmap left by the selection
                    nsel += selq[q];
                    val[q] = p;
                } else if (QK == CONEF_Q_RANDBLOCK) {
                    const uint32_t slot = j - blk_start;   // wraps to a large value below the block
                    if (slot < (uint32_t)L.k) {
                        msg[slot] = p;
                        if (worker == 0)
                            V.idx[L.idx_off + slot] = j;
                        val[q] = 0.f;   // r = p - Delta is zero on a transmitted coordinate
                    } else
                        val[q] = p;
                } else {
                    const uint32_t row = j / m, col = j - row * m;
                    float acc = p;
                    for (int c = 0; c < r; ++c)
                        acc = __fmaf_rn(-phat[(int64_t)row * r + c], qi[(int64_t)col * r + c], acc);
                    val[q] = acc;  // r = p - P_hat Q_i^T
                }
            }
        }
        if (QK == CONEF_Q_RANDK) {
            int inc = nsel;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int n = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o)
                    inc += n;
            }
            uint32_t slot = V.tileoff[L.tileoff_off + (unit * U) / kHistTile] + V.unitoff[L.unitoff_off + unit] +
                            (uint32_t)(inc - nsel);
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (selq[q]) {
                    msg[slot] = val[q];  // message value, ascending index order
                    if (worker == 0)
                        V.idx[L.idx_off + slot] = base + q;
                    ++slot;
                    val[q] = 0.f;  // r = p - Delta is zero on a transmitted coordinate
                }
        }
        if (v2) {
            // Alg. 3 line 12: e~ = Q(r) by a second draw; line 14 then stores q = C(r - e~), and
            // r - e~ is exactly zero where e~ keeps the value
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const uint32_t j = base + q;
                uint32_t sl;
                if (QK == CONEF_Q_RANDK) {
                    if ((bitsB >> q) & 1u) {
                        ev_new[slotB + (uint32_t)__popc(bitsB & ((1u << q) - 1u))] = val[q];
                        val[q] = 0.f;
                    }
                } else if (q < E && j < d && draw_member<QD>(L, V.selbitsB, V.unitoffB, V.tileoffB, blk_startB, j, sl)) {
                    ev_new[sl] = val[q];
                    val[q] = 0.f;
                }
            }
        }
        // ---- store r through C (Alg. 2 line 9); Alg. 4 line 9 stores C(beta e + r)
        if (V.beta != 0.f) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
                val[q] = __fmaf_rn(V.beta, ekeep[q], val[q]);
        }
        if (CK == CONEF_C_IDENTITY) {
            float *e = (float *)(st + L.a_off);
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (q < E && base + q < d)
                    e[base + q] = val[q];
            if (has_second<CK>(V)) {   // e~ = r exactly: nothing is left for q
                float *e2 = (float *)(st + L.a2_off);
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (q < E && base + q < d)
                        e2[base + q] = __fsub_rn(val[q], val[q]);
            }
        } else if (CK == CONEF_C_STOCHQUANT) {
            // Eq. 6 with the block's max-norm: level floor(u) or floor(u) + 1, up with probability u - floor(u)
            float amax = 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                amax = fmaxf(amax, fabsf(val[q]));
            amax = warp_max(amax);
            const float lv = (float)V.levels;
            float s = __fdiv_rn(amax, lv);
            const bool zero = !(s >= FLT_MIN);
            s = zero ? 0.f : s;
            const float inv = zero ? 0.f : __fdiv_rn(1.0f, s);
            if (lane == 0)
                ((float *)(st + L.b_off))[unit] = s;
            // this worker's variates for this tensor and step: a counter-based stream
            const uint64_t stc = stream_key(mix64(V.seed_c + (uint64_t)worker + 1u), (uint64_t)li, (uint64_t)V.step);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const uint32_t j = base + q;
                if (q < E && j < d) {
                    int c = 0;
                    if (!zero) {
                        float u = __fmul_rn(fabsf(val[q]), inv);
                        u = !(u <= lv) ? lv : u;
                        const float l = floorf(u);
                        const float frac = __fsub_rn(u, l);
                        const float rnd = __fmul_rn((float)(uint32_t)(h64(stc, j) >> 40), 1.0f / 16777216.0f);
                        int lev = (int)l + (rnd < frac ? 1 : 0);
                        lev = min(lev, V.levels);
                        c = val[q] < 0.f ? -lev : lev;
                    }
                    if (V.sq_wide)
                        ((short *)(st + L.a_off))[j] = (short)c;
                    else
                        ((signed char *)(st + L.a_off))[j] = (signed char)c;
                }
            }
        } else if (CK == CONEF_C_COUNTSKETCH) {
            float *S = (float *)(V.state_new + worker * V.state_stride + L.a_off);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const uint32_t j = base + q;
                if (q < E && j < d && val[q] != 0.f) {
                    uint32_t lo, width;
                    sketch_window(V, L, j, lo, width);
#pragma unroll
                    for (int i = 0; i < 7; ++i)
                        if (i < V.cs_rows) {
                            uint64_t h = h64(keys.st[i], j);
                            uint64_t b = lo + (((h >> 32) * (uint64_t)width) >> 32);
                            atomicAdd(&S[(int64_t)i * L.w + (int64_t)b], (h & 1) ? -val[q] : val[q]);
                        }
                }
            }
        } else {
            // e~ = C(r); with iConEF-v1 a second round stores q = C(r - e~) (Alg. 3 lines 10, 14)
            const int rounds = has_second<CK>(V) ? 2 : 1;
            for (int lev = 0; lev < rounds; ++lev) {
                const int64_t aoff = lev ? L.a2_off : L.a_off, boff = lev ? L.b2_off : L.b_off;
                float amax = 0.f;
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    amax = fmaxf(amax, fabsf(val[q]));
                amax = warp_max(amax);
                float s, inv;
                unsigned short hb;
                quant_scale(amax, qmax, V.scale_half, s, inv, hb);
                if (lane == 0) {
                    if (V.scale_half)
                        ((unsigned short *)(st + boff))[unit] = hb;
                    else
                        ((float *)(st + boff))[unit] = s;
                }
                int cq[8];
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    cq[q] = quant_code(val[q], inv, qmax);
                if (CK == CONEF_C_INT8) {
                    signed char *codes = (signed char *)(st + aoff);
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        if (q < E && base + q < d)
                            codes[base + q] = (signed char)cq[q];
                } else {
                    uint8_t *codes = st + aoff;
#pragma unroll
                    for (int q = 0; q < 8; q += 2)
                        if (q < E && base + q < d) {
                            int lo = cq[q] & 0xF;
                            int hi = (base + q + 1 < d) ? (cq[q + 1] & 0xF) : 0;
                            codes[(base + q) >> 1] = (uint8_t)(lo | (hi << 4));
                        }
                }
                if (lev + 1 < rounds) {
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        val[q] = __fsub_rn(val[q], __fmul_rn((float)cq[q], s));   // what the first state misses
                }
            }
        }
    }
}

// ------------------------------------------------------------------ low-rank pass 1 (generic)
// P_i = M_i Q_{t-1}: one warp per row, lanes stride over the columns.
template <int CK>
__global__ void __launch_bounds__(256) k_lr_pass1(const __grid_constant__ DevView V)
{
    const int li = find_layer(V.pfx_p1, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int worker = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t m = (uint32_t)L.cols;
    const int r = L.rank;
    const uint8_t *st = V.state + worker * V.state_stride;
    const float *__restrict__ g = V.grads[worker] + L.g_off;
    const float *__restrict__ Q = V.qprev + L.msgq_off;
    float *__restrict__ P = V.msgp + worker * V.msgp_stride + L.msgp_off;
    SketchKeys keys = {};
    if (CK == CONEF_C_COUNTSKETCH)
        keys = sketch_keys(V.seed_c, li, V.cs_rows);
    const int64_t row0 = (int64_t)(blockIdx.x - V.pfx_p1[li]) * kP1RowsPerCta;
    for (int rr = 0; rr < kP1RowsPerCta / 8; ++rr) {
        const int64_t row = row0 + warp * (kP1RowsPerCta / 8) + rr;
        if (row >= L.rows)
            break;
        float acc[CONEF_MAX_RANK];
#pragma unroll
        for (int c = 0; c < CONEF_MAX_RANK; ++c)
            acc[c] = 0.f;
        for (uint32_t col = lane; col < m; col += 32) {
            const uint32_t j = (uint32_t)row * m + col;
            float p = form_p(V, g[j], decode_elem<CK>(V, L, st, j, keys));
            if (has_second<CK>(V))
                p = __fadd_rn(p, decode_elem<CK>(V, L, st, j, keys, true));
#pragma unroll
            for (int c = 0; c < CONEF_MAX_RANK; ++c)
                if (c < r)
                    acc[c] = __fmaf_rn(p, Q[(int64_t)col * r + c], acc[c]);
        }
#pragma unroll
        for (int c = 0; c < CONEF_MAX_RANK; ++c)
            if (c < r) {
                float s = warp_sum(acc[c]);
                if (lane == 0)
                    P[row * r + c] = s;
            }
    }
}

// ------------------------------------------------------------------ P-reduce + Gram-Schmidt
__device__ __forceinline__ double block_sum_double(double v, double *sh)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();  // sh may still be read from the previous call
    if (lane == 0)
        sh[warp] = v;
    __syncthreads();
    double t = (lane < (int)(blockDim.x >> 5)) ? sh[lane] : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        t += __shfl_xor_sync(0xffffffffu, t, o);
    return t;  // the same value in every thread
}

// One CTA per compressed tensor: P_bar = sum over workers (worker order);
// modified Gram-Schmidt on its columns, left to right, dot products and norms
// accumulated in fp64 and rounded once.
__global__ void __launch_bounds__(1024) k_gram_schmidt(const __grid_constant__ DevView V,
                                                       float *__restrict__ out_sum)
{
    __shared__ double sh[32];
    const int li = find_layer(V.pfx_gs, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int64_t n = L.rows;
    const int r = L.rank;
    float *__restrict__ pbar = V.pbar + L.msgp_off;
    float *__restrict__ ph = V.phat + L.msgp_off;
    for (int64_t q = threadIdx.x; q < n * r; q += blockDim.x) {
        float acc = V.msgp[L.msgp_off + q];
        for (int i = 1; i < V.n_workers; ++i)
            acc = __fadd_rn(acc, V.msgp[i * V.msgp_stride + L.msgp_off + q]);
        pbar[q] = acc;
        ph[q] = acc;
        if (out_sum)
            out_sum[L.msgp_off + q] = acc;
    }
    __syncthreads();
    for (int c = 0; c < r; ++c) {
        for (int cp = 0; cp < c; ++cp) {
            double part = 0.0;
            for (int64_t a = threadIdx.x; a < n; a += blockDim.x)
                part += (double)ph[a * r + cp] * (double)ph[a * r + c];
            const float dotf = (float)block_sum_double(part, sh);
            for (int64_t a = threadIdx.x; a < n; a += blockDim.x)
                ph[a * r + c] = __fmaf_rn(-dotf, ph[a * r + cp], ph[a * r + c]);
            __syncthreads();
        }
        double part = 0.0;
        for (int64_t a = threadIdx.x; a < n; a += blockDim.x)
            part += (double)ph[a * r + c] * (double)ph[a * r + c];
        const float nu = (float)sqrt(block_sum_double(part, sh));
        const bool dead = !(nu >= FLT_MIN);
        for (int64_t a = threadIdx.x; a < n; a += blockDim.x)
            ph[a * r + c] = dead ? 0.f : __fdiv_rn(ph[a * r + c], nu);
        __syncthreads();
    }
}

// ------------------------------------------------------------------ low-rank pass 2 (generic)
// Q_i = M_i^T P_hat: a thread owns one column and runs down a tile of rows;
// the per-tile partials are summed in tile order by k_lr_pass2_reduce, so the
// result does not depend on scheduling.
template <int CK>
__global__ void __launch_bounds__(kP2ColsPerCta) k_lr_pass2(const __grid_constant__ DevView V)
{
    const int li = find_layer(V.pfx_p2, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int worker = blockIdx.y;
    const uint32_t m = (uint32_t)L.cols;
    const int r = L.rank;
    const int local = blockIdx.x - V.pfx_p2[li];
    const int ncoltiles = (int)((m + kP2ColsPerCta - 1) / kP2ColsPerCta);
    const int rt = local / ncoltiles, ct = local - rt * ncoltiles;
    const uint32_t col = ct * kP2ColsPerCta + threadIdx.x;
    if (col >= m)
        return;
    const uint8_t *st = V.state + worker * V.state_stride;
    const float *__restrict__ g = V.grads[worker] + L.g_off;
    const float *__restrict__ ph = V.phat + L.msgp_off;
    SketchKeys keys = {};
    if (CK == CONEF_C_COUNTSKETCH)
        keys = sketch_keys(V.seed_c, li, V.cs_rows);
    float acc[CONEF_MAX_RANK];
#pragma unroll
    for (int c = 0; c < CONEF_MAX_RANK; ++c)
        acc[c] = 0.f;
    const int64_t rend = min((int64_t)L.rows, (int64_t)(rt + 1) * kP2RowsPerTile);
    for (int64_t row = (int64_t)rt * kP2RowsPerTile; row < rend; ++row) {
        const uint32_t j = (uint32_t)row * m + col;
        float p = form_p(V, g[j], decode_elem<CK>(V, L, st, j, keys));
        if (has_second<CK>(V))
            p = __fadd_rn(p, decode_elem<CK>(V, L, st, j, keys, true));
#pragma unroll
        for (int c = 0; c < CONEF_MAX_RANK; ++c)
            if (c < r)
                acc[c] = __fmaf_rn(p, ph[row * r + c], acc[c]);
    }
    float *__restrict__ part = V.part + worker * V.part_stride + L.part_off;
#pragma unroll
    for (int c = 0; c < CONEF_MAX_RANK; ++c)
        if (c < r)
            part[((int64_t)rt * m + col) * r + c] = acc[c];
}

// Q_i = sum over the row tiles' partials, in tile order: four consecutive (column, c) entries per
// thread, 16-byte loads where the tensor's offsets allow, the loads of four tiles in flight
constexpr int kQ2PerCta = 1024;
__global__ void __launch_bounds__(256) k_lr_pass2_reduce(const __grid_constant__ DevView V)
{
    const int li = find_layer(V.pfx_q2, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int worker = blockIdx.y;
    const int64_t mr = L.cols * L.rank;
    const int64_t q = ((int64_t)(blockIdx.x - V.pfx_q2[li]) * 256 + threadIdx.x) * 4;
    if (q >= mr)
        return;
    const int64_t ntiles = (V.fast_on && L.fast) ? L.p2_rows_fast : L.p2_rows_generic;
    const float *__restrict__ part = V.part + worker * V.part_stride + L.part_off;
    float *out = V.msgq + worker * V.msgq_stride + L.msgq_off;
    if (mr % 4 == 0 && ((V.part_stride | L.part_off | V.msgq_stride | L.msgq_off) & 3) == 0) {
        const float4 *p4 = (const float4 *)(part + q);
        const int64_t step = mr / 4;
        float4 acc = p4[0];
        int64_t t = 1;
        for (; t + 4 <= ntiles; t += 4) {
            const float4 a = p4[t * step], b = p4[(t + 1) * step], c = p4[(t + 2) * step], d = p4[(t + 3) * step];
            acc.x = __fadd_rn(__fadd_rn(__fadd_rn(__fadd_rn(acc.x, a.x), b.x), c.x), d.x);
            acc.y = __fadd_rn(__fadd_rn(__fadd_rn(__fadd_rn(acc.y, a.y), b.y), c.y), d.y);
            acc.z = __fadd_rn(__fadd_rn(__fadd_rn(__fadd_rn(acc.z, a.z), b.z), c.z), d.z);
            acc.w = __fadd_rn(__fadd_rn(__fadd_rn(__fadd_rn(acc.w, a.w), b.w), c.w), d.w);
        }
        for (; t < ntiles; ++t) {
            const float4 a = p4[t * step];
            acc.x = __fadd_rn(acc.x, a.x);
            acc.y = __fadd_rn(acc.y, a.y);
            acc.z = __fadd_rn(acc.z, a.z);
            acc.w = __fadd_rn(acc.w, a.w);
        }
        *(float4 *)(out + q) = acc;
        return;
    }
    for (int64_t j = q; j < min(q + 4, mr); ++j) {
        float acc = part[j];
        for (int64_t t = 1; t < ntiles; ++t)
            acc = __fadd_rn(acc, part[t * mr + j]);
        out[j] = acc;
    }
}

// ------------------------------------------------------------------ aggregate (S6)
// out[j] = ((m_0[j] + m_1[j]) + ...) in worker order; optionally also the mean
__global__ void __launch_bounds__(256) k_reduce_workers(const float *__restrict__ base,
                                                        int64_t stride, int n_workers, int64_t len,
                                                        float *__restrict__ out,
                                                        float *__restrict__ mean_out, float nf)
{
    for (int64_t j = (int64_t)blockIdx.x * 256 + threadIdx.x; j < len; j += (int64_t)gridDim.x * 256) {
        float acc = base[j];
        for (int i = 1; i < n_workers; ++i)
            acc = __fadd_rn(acc, base[i * stride + j]);
        if (out)
            out[j] = acc;
        if (mean_out)
            mean_out[j] = __fdiv_rn(acc, nf);
    }
}

// ------------------------------------------------------------------ decode alone
template <int CK>
__global__ void __launch_bounds__(256) k_decompress(const __grid_constant__ DevView V, int worker,
                                                    float *__restrict__ out)
{
    const int li = find_layer(V.pfx_flat, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const uint8_t *st = V.state + worker * V.state_stride;
    SketchKeys keys = {};
    if (CK == CONEF_C_COUNTSKETCH)
        keys = sketch_keys(V.seed_c, li, V.cs_rows);
    const int64_t j0 = (int64_t)(blockIdx.x - V.pfx_flat[li]) * kFlatUnitsPerCta * L.unit;
    const int64_t j1 = min(L.d, j0 + (int64_t)kFlatUnitsPerCta * L.unit);
    for (int64_t j = j0 + threadIdx.x; j < j1; j += 256)
    {
        float e = decode_elem<CK>(V, L, st, (uint32_t)j, keys);
        if (has_second<CK>(V))
            e = __fadd_rn(e, decode_elem<CK>(V, L, st, (uint32_t)j, keys, true));   // e~ + q
        if (V.iconef == 2) {   // e~ (the k values of the draw that stored them) + q
            float ev = 0.f;
            uint32_t sl;
            if (V.ev_valid) {
                const float *evp = V.ev_old + worker * V.msgv_stride + L.msgv_off;
                if (V.qkind == CONEF_Q_RANDBLOCK) {
                    const uint32_t bs = randblock_start(stream_key(V.seed_q, (uint64_t)li, (uint64_t)(V.ev_step + kSecondDraw)),
                                                        (uint32_t)L.d, (uint32_t)L.k);
                    if (draw_member<CONEF_Q_RANDBLOCK>(L, V.selbitsA, V.unitoffA, V.tileoffA, bs, (uint32_t)j, sl))
                        ev = evp[sl];
                } else if (draw_member<CONEF_Q_RANDK>(L, V.selbitsA, V.unitoffA, V.tileoffA, 0u, (uint32_t)j, sl))
                    ev = evp[sl];
            }
            e = __fadd_rn(ev, e);
        }
        out[L.e_off + j] = e;
    }
}

}  // namespace conef
