// Fused step for the count sketch applied run by run (Alg. 2 lines 5, 6, 9 with C = count sketch,
// Sec. 4.2.2; cs_chunk > 0) and Q in {identity, random-k, random-block-k}.  One CTA owns one run of
// a tensor for one worker: the run's window of the stored sketch (v rows of a few thousand
// buckets) is copied to shared memory with coalesced loads, every element of the run is decoded
// from it (v hashes, v shared-memory reads, the median), p = eta g + e is formed, the message is
// written, and the residual is added into a second window in shared memory, which is then
// written out with coalesced stores.  The sketch moves through HBM once in each direction and
// the v gathers and v atomic adds per element stay inside the SM, where the whole-tensor hash
// needs them in L2.
#pragma once
#include "conef_kernels.cuh"

namespace conef {

#ifndef CONEF_CS_THREADS
#define CONEF_CS_THREADS 256
#endif
constexpr int kCsThreads = CONEF_CS_THREADS;

template <int QK, int VR>
__global__ void __launch_bounds__(kCsThreads) k_sketch_chunk(const __grid_constant__ DevView V,
                                                             const int32_t *__restrict__ pfx)
{
    extern __shared__ float cs_smem[];
    const int li = find_layer(pfx, V.n_layers, blockIdx.x);
    const LayerDesc &L = V.layers[li];
    const int worker = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int v = VR ? VR : V.cs_rows;
    const uint32_t d = (uint32_t)L.d, w = (uint32_t)L.w, chunk = (uint32_t)V.cs_chunk;
    const uint32_t c = blockIdx.x - pfx[li];
    uint32_t nc = d / chunk;
    nc = nc < 1 ? 1 : nc;
    const uint32_t j_lo = c * chunk, j_hi = (c == nc - 1) ? d : j_lo + chunk;
    uint32_t lo = 0, width = w;
    if (nc > 1)
        sketch_window_of_run(c, nc, chunk, d, w, lo, width);

    float *olds = cs_smem;                 // v x width: the stored window
    float *news = cs_smem + v * width;     // v x width: the window being built
    const float *__restrict__ S = (const float *)(V.state + worker * V.state_stride + L.a_off);
    float *__restrict__ Sn = (float *)(V.state_new + worker * V.state_stride + L.a_off);
    for (int i = 0; i < v; ++i)
        for (uint32_t b = threadIdx.x; b < width; b += kCsThreads) {
            olds[i * width + b] = S[(int64_t)i * w + lo + b];
            news[i * width + b] = 0.f;
        }
    __syncthreads();

    const SketchKeys keys = sketch_keys(V.seed_c, li, V.cs_rows);
    const float *__restrict__ g = V.grads[worker] + L.g_off;
    float *__restrict__ msg = V.msgv + worker * V.msgv_stride + L.msgv_off;
    uint32_t blk_start = 0;
    if (QK == CONEF_Q_RANDBLOCK)
        blk_start = randblock_start(stream_key(V.seed_q, (uint64_t)li, (uint64_t)V.step), d, (uint32_t)L.k);
    const int unit_shift = 31 - __clz(L.unit);          // message slots are handed out per unit of 32..256 elements
    const uint32_t words_per_unit = (uint32_t)L.unit >> 5;

    // a warp takes 32 consecutive elements at a time (one word of the membership bitmap)
    for (uint32_t base = j_lo + warp * 32; base < j_hi; base += kCsThreads) {
        const uint32_t j = base + lane;
        const bool valid = j < j_hi;
        uint32_t word = 0;
        if (QK == CONEF_Q_RANDK)
            word = V.selbits[L.selbits_off + (base >> 5)];
        float p = 0.f, e = 0.f;
        uint32_t bi[VR ? VR : 7];   // bucket of this element in each row; bit 31: negative sign
        if (valid) {
            float est[VR ? VR : 7];
#pragma unroll
            for (int i = 0; i < (VR ? VR : 7); ++i) {
                est[i] = 0.f;
                bi[i] = 0;
                if (i < v) {
                    const uint64_t u = h64(keys.st[i], j);
                    const uint32_t b = (uint32_t)i * width + (uint32_t)(((u >> 32) * (uint64_t)width) >> 32);
                    const float s = olds[b];
                    est[i] = (u & 1) ? -s : s;
                    bi[i] = b | ((uint32_t)(u & 1) << 31);
                }
            }
            e = median_small(est, v);
            p = form_p(V, g[j], e);   // Alg. 2 line 5 (Alg. 4 line 5 with beta)
        }
        bool sel = false;
        if (QK == CONEF_Q_IDENTITY) {
            sel = valid;
            if (valid)
                msg[j] = p;
        } else if (QK == CONEF_Q_RANDBLOCK) {
            const uint32_t slot = j - blk_start;   // wraps to a large value below the block
            sel = valid && slot < (uint32_t)L.k;
            if (sel) {
                msg[slot] = p;
                if (worker == 0)
                    V.idx[L.idx_off + slot] = j;
            }
        } else {
            sel = valid && ((word >> lane) & 1u);
            if (word != 0) {   // (uniform over the warp)
                // slot = tile offset + unit offset + selected elements before this one in its unit
                const uint32_t wi = base >> 5, first = wi & ~(words_per_unit - 1);
                uint32_t before = 0;
                for (uint32_t x = first; x < wi; ++x)
                    before += __popc(V.selbits[L.selbits_off + x]);
                if (sel) {
                    const uint32_t slot = V.tileoff[L.tileoff_off + base / kHistTile] +
                                          V.unitoff[L.unitoff_off + (base >> unit_shift)] + before +
                                          __popc(word & ((1u << lane) - 1u));
                    msg[slot] = p;
                    if (worker == 0)
                        V.idx[L.idx_off + slot] = j;
                }
            }
        }
        // r = p - Delta (zero on a transmitted coordinate); Alg. 4 line 9 keeps beta e as well
        float val = sel ? 0.f : p;
        if (V.beta != 0.f)
            val = __fmaf_rn(V.beta, e, val);
        if (valid && val != 0.f) {
#pragma unroll
            for (int i = 0; i < (VR ? VR : 7); ++i)
                if (i < v)
                    atomicAdd(&news[bi[i] & 0x7FFFFFFFu], (bi[i] >> 31) ? -val : val);
        }
    }
    __syncthreads();
    for (int i = 0; i < v; ++i)
        for (uint32_t b = threadIdx.x; b < width; b += kCsThreads)
            Sn[(int64_t)i * w + lo + b] = news[i * width + b];
}

// whether the two windows of the widest run of a tensor fit a CTA's shared memory
inline int64_t chunk_window_max(int64_t d, int64_t w, int64_t chunk)
{
    int64_t nc = d / chunk;
    if (nc < 1)
        nc = 1;
    if (nc == 1)
        return w;
    // full runs get at most ceil(w chunk / d) buckets; the last run what is left after nc - 1 of them
    const int64_t full = (int64_t)(((unsigned __int128)w * (unsigned __int128)chunk) / (unsigned __int128)d) + 1;
    const int64_t last = w - (int64_t)(((unsigned __int128)w * (unsigned __int128)(nc - 1) * (unsigned __int128)chunk) / (unsigned __int128)d);
    return full > last ? full : last;
}

inline cudaError_t chunksketch_launch(int qkind, int v, const DevView &V, const int32_t *pfx, int tiles,
                                      size_t smem_bytes, cudaStream_t s)
{
    if (tiles <= 0)
        return cudaSuccess;
    dim3 grid(tiles, V.n_workers);
#define CONEF_CSK_CASE(QV, VRV)                                                                             \
    if (qkind == QV && (VRV == 0 || v == VRV)) {                                                            \
        static int done[64];                                                                                \
        const cudaError_t e = opt_in_smem(k_sketch_chunk<QV, VRV>, smem_bytes, done);                       \
        if (e != cudaSuccess)                                                                               \
            return e;                                                                                       \
        k_sketch_chunk<QV, VRV><<<grid, kCsThreads, smem_bytes, s>>>(V, pfx);                               \
        return cudaSuccess;                                                                                 \
    }
#define CONEF_CSK_Q(QV)    \
    CONEF_CSK_CASE(QV, 1)  \
    CONEF_CSK_CASE(QV, 3)  \
    CONEF_CSK_CASE(QV, 5)  \
    CONEF_CSK_CASE(QV, 0)
    CONEF_CSK_Q(CONEF_Q_IDENTITY)
    CONEF_CSK_Q(CONEF_Q_RANDK)
    CONEF_CSK_Q(CONEF_Q_RANDBLOCK)
#undef CONEF_CSK_Q
#undef CONEF_CSK_CASE
    return cudaErrorNotSupported;
}

}  // namespace conef
