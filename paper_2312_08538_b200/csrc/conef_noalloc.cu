// Allocation-free variant of the random-k index selection.
//
// Who needs it: the side that RECEIVES a random-k message.  To scatter the k
// values back into a dense update it must know the index set S_t, which
// depends only on (seed, tensor, step).  Such a receiver (a parameter server,
// a rank that only applies updates, a hook called from inside another
// framework's step) often holds no ConEF context and is not allowed to touch
// the device allocator: its memory pool is fixed up front, and a cudaMalloc in
// the middle of a step would synchronise the device or fail under memory
// pressure.  The selection needs scratch (radix histograms, per-block counts);
// here that scratch is a fixed array that lives in the library's device image.
#include <cuda_runtime.h>

#include <mutex>

#include "conef_hash.cuh"
#include "conef_internal.h"

using namespace conef;

namespace {

constexpr int kNaUnit = 256;                                        // elements per counted block
constexpr int64_t kNaMaxElems = CONEF_NOALLOC_MAX_ELEMS;
constexpr int kNaSelWords = kSelWords;                              // histograms, state, tie list
constexpr int64_t kNaWords = kNaSelWords + kNaMaxElems / kNaUnit;   // + one count per block

// The scratch itself.  Every GPU that loads the library holds these ~290 KB
// until the process exits.  In host code the name below is only a handle for
// cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) uint32_t g_noalloc_scratch[kNaWords];

struct NaArgs {
    uint32_t *sel;     // selection scratch (kNaSelWords words)
    uint32_t *cnt;     // per-block counts, then offsets
    uint64_t stream;   // hash stream key of (seed, tensor, step)
    uint32_t d, k;
};

template <int LEVEL>
__global__ void __launch_bounds__(256) k_na_hist(NaArgs a)
{
    __shared__ uint32_t hist[kHistBins];
    uint32_t *stw = a.sel + 3 * kHistBins;
    const uint32_t prefix = stw[SEL_PREFIX];
    for (int b = threadIdx.x; b < kHistBins; b += 256)
        hist[b] = 0;
    __syncthreads();
    const int64_t j0 = (int64_t)blockIdx.x * kHistTile;
    for (int q = threadIdx.x; q < kHistTile; q += 256) {
        const int64_t j = j0 + q;
        if (j >= a.d)
            break;
        const uint32_t h = hash32(a.stream, (uint64_t)j);
        if (LEVEL == 0)
            atomicAdd(&hist[h >> 21], 1u);
        else if (LEVEL == 1) {
            if ((h >> 21) == prefix)
                atomicAdd(&hist[(h >> 10) & 2047u], 1u);
        } else if (LEVEL == 2) {
            if ((h >> 10) == prefix)
                atomicAdd(&hist[h & 1023u], 1u);
        } else if (h == stw[SEL_TAU_HI]) {
            const uint32_t pos = atomicAdd(&stw[SEL_NTIES], 1u);
            if (pos < (uint32_t)kMaxTies)
                stw[16 + pos] = (uint32_t)j;
        }
    }
    if (LEVEL < 3) {
        __syncthreads();
        uint32_t *gh = a.sel + LEVEL * kHistBins;
        for (int b = threadIdx.x; b < kHistBins; b += 256)
            if (hist[b])
                atomicAdd(&gh[b], hist[b]);
    }
}

// one CTA: the bin that holds the wanted rank (levels 0-2), the tie-breaking index (level 3)
template <int LEVEL>
__global__ void __launch_bounds__(1024) k_na_pick(NaArgs a, int32_t *status)
{
    __shared__ uint32_t wsum[32];
    __shared__ uint32_t ties[kMaxTies];
    uint32_t *stw = a.sel + 3 * kHistBins;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (LEVEL < 3) {
        const uint32_t remain = (LEVEL == 0) ? a.k : stw[SEL_REMAIN];
        const uint32_t *gh = a.sel + LEVEL * kHistBins;
        const uint32_t c0 = gh[2 * tid], c1 = gh[2 * tid + 1];
        const uint32_t mine = c0 + c1;
        uint32_t inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o)
                inc += n;
        }
        if (lane == 31)
            wsum[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const uint32_t w = wsum[lane];
            uint32_t winc = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t n = __shfl_up_sync(0xffffffffu, winc, o);
                if (lane >= o)
                    winc += n;
            }
            wsum[lane] = winc - w;
        }
        __syncthreads();
        const uint32_t before = wsum[warp] + inc - mine;
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
            atomicOr(&stw[SEL_FOUND], 1u << LEVEL);
        }
    } else {
        const uint32_t n = stw[SEL_NTIES], remain = stw[SEL_REMAIN];
        if (n > (uint32_t)kMaxTies || remain > n || remain == 0) {
            if (tid == 0) {
                if (status)
                    atomicOr(status, ST_TIE_OVERFLOW);
                stw[SEL_TAU_LO] = 0xffffffffu;
                stw[SEL_FAILED] = 1u;
            }
            return;
        }
        if ((uint32_t)tid < n)
            ties[tid] = stw[16 + tid];
        __syncthreads();
        if ((uint32_t)tid < n) {
            const uint32_t me = ties[tid];
            uint32_t rank = 0;
            for (uint32_t q = 0; q < n; ++q)
                rank += ties[q] < me;
            if (rank == remain - 1)
                stw[SEL_TAU_LO] = me;
        }
    }
}

// WRITE == 0: count the selected coordinates of each block of 256 elements;
// WRITE == 1: write them, in ascending order, at the block's offset
template <int WRITE>
__global__ void __launch_bounds__(256) k_na_count(NaArgs a, uint32_t *__restrict__ idx_out)
{
    const uint32_t *stw = a.sel + 3 * kHistBins;
    const uint32_t tau_hi = stw[SEL_TAU_HI], tau_lo = stw[SEL_TAU_LO];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t nblocks = ((int64_t)a.d + kNaUnit - 1) / kNaUnit;
    for (int64_t blk = (int64_t)blockIdx.x * 8 + warp; blk < nblocks; blk += (int64_t)gridDim.x * 8) {
        const uint32_t base = (uint32_t)blk * kNaUnit + lane * 8;   // a lane owns 8 consecutive elements
        bool sel[8];
        int n = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t j = base + q;
            sel[q] = j < a.d && rk_selected(hash32(a.stream, j), j, tau_hi, tau_lo);
            n += sel[q];
        }
        int inc = n;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o)
                inc += t;
        }
        if (!WRITE) {
            if (lane == 31)
                a.cnt[blk] = (uint32_t)inc;
        } else {
            uint32_t slot = a.cnt[blk] + (uint32_t)(inc - n);
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (sel[q]) {
                    if (slot < a.k)   // never past the caller's k entries, whatever went wrong before
                        idx_out[slot] = base + q;
                    ++slot;
                }
        }
    }
}

// exclusive scan of the block counts, in place (one CTA)
__global__ void __launch_bounds__(1024) k_na_scan(NaArgs a)
{
    __shared__ uint32_t wsum[32];
    __shared__ uint32_t carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t nblocks = ((int64_t)a.d + kNaUnit - 1) / kNaUnit;
    if (tid == 0)
        carry_s = 0;
    __syncthreads();
    for (int64_t base = 0; base < nblocks; base += 1024) {
        const int64_t u = base + tid;
        const uint32_t v = u < nblocks ? a.cnt[u] : 0u;
        uint32_t inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o)
                inc += n;
        }
        if (lane == 31)
            wsum[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const uint32_t w = wsum[lane];
            uint32_t winc = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t n = __shfl_up_sync(0xffffffffu, winc, o);
                if (lane >= o)
                    winc += n;
            }
            wsum[lane] = winc - w;
        }
        __syncthreads();
        const uint32_t carry = carry_s;
        if (u < nblocks)
            a.cnt[u] = carry + wsum[warp] + inc - v;
        __syncthreads();
        if (tid == 1023)
            carry_s = carry + wsum[31] + inc;
        __syncthreads();
    }
    if (tid == 0)
        a.sel[3 * kHistBins + SEL_TOTAL] = carry_s;   // coordinates selected in all
}

// A selection that did not come out as exactly k coordinates (a radix level without its bin, more
// ties on the threshold hash than the tie list holds, a count other than k) is made visible in
// the output itself, since this entry point neither synchronises nor owns a status buffer:
// idx_out[0] = 0xFFFFFFFF, a value no index can take.
__global__ void k_na_finish(NaArgs a, uint32_t *__restrict__ idx_out)
{
    const uint32_t *stw = a.sel + 3 * kHistBins;
    if (threadIdx.x == 0 && (stw[SEL_FOUND] != 7u || stw[SEL_FAILED] != 0u || stw[SEL_TOTAL] != a.k))
        idx_out[0] = 0xFFFFFFFFu;
}

// device address of the scratch on each device, resolved once per device
std::mutex g_mu;
uint32_t *g_scratch_ptr[64] = {nullptr};
int g_sm_count[64] = {0};

}  // namespace

extern "C" int conef_randk_indices_noalloc(uint64_t seed, int64_t tensor, int64_t step, int64_t d, int64_t k,
                                           uint32_t *idx_out, conef_stream stream)
{
    if (d <= 0 || k <= 0 || k > d || tensor < 0 || step < 0 || !idx_out)
        return CONEF_ERR_INVALID_ARG;
    if (d > kNaMaxElems)
        return CONEF_ERR_TOO_LARGE;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return CONEF_ERR_CUDA;
    uint32_t *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_scratch_ptr[dev]) {
            // set-up, with this device current: turn the symbol into its device address
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p)
                return CONEF_ERR_CUDA;
            int sms = 0;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
                return CONEF_ERR_CUDA;
            g_sm_count[dev] = sms;
            g_scratch_ptr[dev] = (uint32_t *)p;
        }
        scratch = g_scratch_ptr[dev];
    }
    if (cudaPeekAtLastError() != cudaSuccess)
        return CONEF_ERR_CUDA;   // an error from before this call is pending: nothing is launched on top of it
    cudaStream_t s = (cudaStream_t)stream;
    NaArgs a;
    a.sel = scratch;
    a.cnt = scratch + kNaSelWords;
    a.stream = stream_key(seed, (uint64_t)tensor, (uint64_t)step);
    a.d = (uint32_t)d;
    a.k = (uint32_t)k;
    // the array keeps the previous call's contents: histograms and state must start at zero
    if (cudaMemsetAsync(a.sel, 0, sizeof(uint32_t) * kNaSelWords, s) != cudaSuccess)
        return CONEF_ERR_CUDA;
    const int nh = (int)((d + kHistTile - 1) / kHistTile);
    const int64_t nblocks = (d + kNaUnit - 1) / kNaUnit;
    const int64_t nc_cap = (int64_t)g_sm_count[dev] * 8;
    const int nc = (int)((nblocks + 7) / 8 < nc_cap ? (nblocks + 7) / 8 : nc_cap);
    k_na_hist<0><<<nh, 256, 0, s>>>(a);
    k_na_pick<0><<<1, 1024, 0, s>>>(a, nullptr);
    k_na_hist<1><<<nh, 256, 0, s>>>(a);
    k_na_pick<1><<<1, 1024, 0, s>>>(a, nullptr);
    k_na_hist<2><<<nh, 256, 0, s>>>(a);
    k_na_pick<2><<<1, 1024, 0, s>>>(a, nullptr);
    k_na_hist<3><<<nh, 256, 0, s>>>(a);
    k_na_pick<3><<<1, 1024, 0, s>>>(a, nullptr);
    k_na_count<0><<<nc, 256, 0, s>>>(a, idx_out);
    k_na_scan<<<1, 1024, 0, s>>>(a);
    k_na_count<1><<<nc, 256, 0, s>>>(a, idx_out);
    k_na_finish<<<1, 32, 0, s>>>(a, idx_out);
    return cudaGetLastError() == cudaSuccess ? CONEF_OK : CONEF_ERR_CUDA;
}
