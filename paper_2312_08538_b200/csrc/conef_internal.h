// Internal structures of libconef shared by the host dispatch code and the
// kernels.  Nothing here is part of the public ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/conef.h"

namespace conef {

// The plan (tile lengths, workspace layout) is made without a device, so that the workspace size
// can be asked for anywhere: where it weighs tiles against SMs it takes the SM count of the part
// this library is written for.  Grids that are capped at run time use the count read in conef_init.
constexpr int kPlanSMs = 148;

// Work-unit sizes of the generic kernels
constexpr int kFlatThreads = 256;       // 8 warps; one quantisation block per warp at a time
constexpr int kFlatUnitsPerCta = 32;    // units handled by one CTA of the flat kernel
constexpr int kPassTile = 2048;         // elements of a pass-through tensor per CTA
constexpr int kP1RowsPerCta = 32;       // pass 1 (generic): rows per CTA (8 warps x 4 rows)
constexpr int kP2ColsPerCta = 256;      // pass 2 (generic): one column per thread
constexpr int kP2RowsPerTile = 256;     // pass 2: rows reduced by one CTA before the second stage
constexpr int kRsThreads = 128;         // row sketch: threads per CTA (four columns each where 16-byte loads line up, else one)
constexpr int kRsBuckets = 8;           // row sketch: buckets handled by one CTA
constexpr int kHistTile = 8192;         // random-k selection: elements hashed per CTA
constexpr int kHistBins = 2048;         // radix levels: 11 + 11 + 10 bits of the 32-bit hash
constexpr int kMaxTies = 1024;          // elements that may share the threshold's 32-bit hash
constexpr int kSelWords = 3 * kHistBins + 16 + kMaxTies;  // uint32 words of selection scratch per tensor

// selection state words (after the three histograms)
enum { SEL_PREFIX = 0, SEL_REMAIN = 1, SEL_TAU_HI = 2, SEL_TAU_LO = 3, SEL_NTIES = 4, SEL_NCAND = 5,
       // used by the allocation-free selection only: radix levels that found their bin (bits 0-2),
       // a failed tie-break, the number of coordinates counted
       SEL_FOUND = 6, SEL_FAILED = 7, SEL_TOTAL = 8 };

// status bits written by kernels (sticky, OR-ed)
enum {
    ST_TIE_OVERFLOW = 1,    // more elements share the threshold hash than the tie list holds
    ST_COUNT_MISMATCH = 2,  // the number of selected coordinates differs from k
    ST_SELECT_FAILED = 4,   // a radix level found no bin holding the wanted rank
    ST_FUSED_TIMEOUT = 8    // a bounded wait of the fused low-rank kernel ran out (a copy or a gang member never arrived)
};

struct LayerDesc {
    int64_t rows, cols, d;
    int64_t g_off;       // element offset of this tensor in a worker's flat gradient
    int32_t compressed;  // 1: 2-D and compressed; 0: pass-through
    int32_t rank;        // r_l (low-rank)
    int32_t unit;        // elements per work unit of the flat kernel (= quantisation block)
    int32_t cidx;        // index among the compressed tensors, -1 otherwise
    int64_t nunits;      // ceil(d / unit)
    int64_t k;           // random-k: number of coordinates kept (d for Q = identity)
    int64_t w;           // count sketch: buckets per row
    int64_t a_off;       // bytes, within one worker's state region: codes / dense e / sketch
    int64_t a_bytes;
    int64_t b_off;       // bytes: scales
    int64_t b_bytes;
    int64_t a2_off, b2_off;   // iConEF-v1: the second state q, same sizes
    int64_t e_off;       // floats: position in the concatenated error vector
    int64_t msgv_off;    // floats, within a worker's VALUES message
    int64_t msgp_off;    // floats, within a worker's P message
    int64_t msgq_off;    // floats, within a worker's Q message
    int64_t msg1d_off;   // floats, within a worker's DENSE1D message
    int64_t idx_off;     // uint32 words in the shared index buffer
    int64_t unitoff_off; // uint32 words in the shared per-unit slot-offset buffer
    int64_t tileoff_off; // uint32 words in the shared per-tile (kHistTile elements) slot-offset buffer
    int64_t selbits_off; // uint32 words in the shared membership bitmap (bit i of word w: element 32 w + i is in S_t)
    int64_t part_off;    // floats, within a worker's pass-2 partial buffer
    int64_t sel_off;     // uint32 words in the selection scratch
    int64_t cand_off;    // uint32 words in the candidate list (pairs: hash, index)
    int64_t cand_cap;    // pairs the list of this tensor holds
    int64_t p2_rows_generic;  // partial rows written by the generic pass 2
    int64_t p2_rows_fast;     // ... by the tuned pass 2
    // geometry of the tuned low-rank kernels (conef_fast.cuh); fast == 0: generic only
    int32_t fast;
    int32_t f_lcm;       // super-row: lcm(cols, block) elements
    int32_t f_cw;        // elements of a super-row covered by one CTA
    int32_t f_threads;   // f_cw / 8
    int32_t f_ncg;       // column groups = f_lcm / f_cw
    int32_t f_subs;      // rows per super-row
    int32_t f_rt1, f_rt2, f_rt3;  // row tiles of the three passes
    int32_t f_it1, f_it2, f_it3;  // iterations per tile of the three passes
    int32_t f_fused;     // the fused passes 2 + 3 (conef_fused.cu) take this tensor
    int32_t f_j;         // pass 1: partial rows per row (column segments a row can meet)
    int64_t pp_off;      // floats, within a worker's pass-1 partial buffer
    int64_t f_niter;     // super-rows in the tensor
    // row sketch: uint32 words in the bucket tables (see DevView::rs)
    int64_t rs_info_off; // [v][rows]: bucket of a row | sign << 31
    int64_t rs_ptr_off;  // [v][w + 1]: start of each bucket's row list
    int64_t rs_row_off;  // [v][rows]: rows by bucket, ascending within a bucket, | sign << 31
    int32_t rs_vec;      // columns per thread of the row-sketch kernel (4 or 1)
    int32_t rs_pad;
};

// Device-side view of a context; passed to kernels by value.
struct DevView {
    const LayerDesc *layers;
    int32_t n_layers, n_workers;
    int32_t qkind, ckind, bits, scale_half, cs_rows, block;
    float lr, lr_pad;
    float beta, omb;     // partial error feedback (Alg. 4): beta and 1 - beta (fp32)
    int32_t iconef, cs_chunk;   // 1, 2: iConEF-v1, -v2 (Alg. 3); count sketch: elements per run (0: one run)
    int32_t levels, sq_wide;   // stochastic quantiser: s; levels stored as int16 (else int8)
    float n_workers_f;
    uint64_t seed_q, seed_c;
    int64_t step;
    // per-worker regions: base + worker * stride
    uint8_t *state;      int64_t state_stride;    // bytes (sketch: the buffer decoded this step)
    uint8_t *state_new;                           // sketch only: the buffer being built
    float *msgv;         int64_t msgv_stride;     // floats
    float *msgp;         int64_t msgp_stride;
    float *msgq;         int64_t msgq_stride;
    float *msg1d;        int64_t msg1d_stride;
    float *part;         int64_t part_stride;
    float *ppart;        int64_t ppart_stride;    // pass-1 partial rows per column segment
    // shared by all workers
    float *pbar, *phat, *qprev;                   // indexed by msgp_off / msgq_off
    uint32_t *idx, *unitoff, *tileoff, *sel, *selbits;
    uint32_t *cand;      // random-k selection: elements of the threshold's first-level bin, as (hash, index)
    // iConEF-v2 (Alg. 3 line 12): e~ = Q(p - Delta) kept as the k values of a second draw of Q.
    // Set A is the draw that stored the values being read (step ev_step), set B this step's.
    uint32_t *unitoffA, *tileoffA, *selbitsA, *unitoffB, *tileoffB, *selbitsB;
    float *ev_old, *ev_new;      // per worker (msgv_stride apart), per tensor at msgv_off
    int64_t ev_step;
    int32_t ev_valid, ev_pad;    // 0: no e~ stored yet (e~_0 = 0)
    int32_t *status;
    const uint32_t *rs;  // row sketch: bucket tables of all tensors (hashes do not depend on the step)
    const int32_t *pfx_rs;
    int32_t rs_vec_ok;   // this call's gradient pointers allow 16-byte loads
    int32_t fv_tiles;    // tuned fused step: selection tiles per CTA
    // tile -> tensor prefix tables (n_layers + 1 entries each)
    const int32_t *pfx_flat, *pfx_pass, *pfx_p1, *pfx_p2, *pfx_q2, *pfx_hist, *pfx_gs;
    int32_t fast_on;     // the tuned kernels produced this step's pass-2 partials
    const float *grads[CONEF_MAX_WORKERS];
};

// ---- fused low-rank passes 2 + 3 (conef_fused.cu) ----
constexpr int kFuWarpsPerCta = 8;
constexpr int kFuMaxSeg = 128;          // segments (256 elements) per period of a tensor the kernel takes
constexpr int kFuTilePeriods = 128;     // periods of one segment per tile (default upper limit)
constexpr int kFuRun = 16;              // consecutive tiles of one phase in the task list while two phases alternate
constexpr int kFuPhBytes = 8192 + 128;  // rows of P_hat a tile keeps in shared memory

// one (tensor, worker) pair
struct FusedUnit {
    int32_t layer, worker;
    int32_t ntp;           // tiles per segment
    int32_t tp;            // periods per tile
    int32_t guard_lo, guard_hi;   // earlier units whose scratch this unit's overlaps: they must be finished first (none: hi < lo)
    int32_t ctr_off;       // uint32 words: arrivals per segment [ncg], arrived segments, done flag
    int32_t flag_off;      // ... the done flag
    int64_t scratch_off;   // floats: tile partials [segment][tile][256][r], then segment sums [segment][256][r]
};
// a run of consecutive tasks: tiles tile0, tile0 + 1, ... of one phase of one unit
struct FusedGroup {
    int32_t unit;          // bit 31: phase (0: Q_i partials, pass 2; 1: residual and store, pass 3)
    int32_t first;         // number of its first task
    int32_t tile0;         // tile of the unit that task works on
    int32_t pad;
};

struct FusedParams {
    DevView V;
    const FusedUnit *units;
    const FusedGroup *groups;
    const uint32_t *hint;           // [task / 32]: a group at or before the one that holds task 32 * (task / 32)
    int32_t n_groups, n_tasks;
    int32_t ring, pad;              // slots per warp
    uint32_t *next_task;            // task counter, zero at launch
    uint32_t *ctr;                  // per-unit counters, zero at launch
    float *scratch;
    float *q_out;                   // where the reduced Q_i goes (per worker: + worker * q_out_stride + msgq_off)
    int64_t q_out_stride;
    const float *q_res;             // the Q_i the residual is formed with (the same buffer unless a test injects its own)
    int64_t q_res_stride;
};

struct FusedConfig {
    int ring, threads, ctas, ctas_per_sm;
    size_t smem;
};

// shared-memory budget, occupancy and grid of the kernel on the current device (also opts the
// kernel in to that much dynamic shared memory)
cudaError_t fused_config(int ckind, int rank, int half, int ctas_per_sm, int n_sms, FusedConfig *out);
// cooperative launch (all CTAs co-resident: tasks wait on results of earlier tasks)
cudaError_t fused_launch(int ckind, int rank, int half, int ctas_per_sm, const FusedParams &P, int n_ctas, size_t smem, cudaStream_t s);

// Opt a kernel in to `bytes` of dynamic shared memory, once per device and kernel: `done` is the
// caller's per-kernel record (largest size set so far on each device).  Sizes up to the default
// 48 KB need no call.
template <class K>
inline cudaError_t opt_in_smem(K *kernel, size_t bytes, int (&done)[64])
{
    if (bytes <= 48 * 1024)
        return cudaSuccess;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        dev = 0;
    if ((size_t)done[dev] >= bytes)
        return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess)
        done[dev] = (int)bytes;
    return e;
}

}  // namespace conef
