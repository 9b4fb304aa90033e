// Host side of libconef: argument validation, workspace carving, work tables
// and kernel dispatch behind the C ABI of include/conef.h.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <algorithm>
#include <type_traits>
#include <vector>

#include "conef_internal.h"
#include "conef_kernels.cuh"
#include "conef_hash.cuh"
#include "conef_rowsketch.cuh"
#include "conef_apply.cuh"
#include "conef_fast.cuh"
#include "conef_gs.cuh"
#include "conef_flatvec.cuh"
#include "conef_chunksketch.cuh"
#include "conef_rowsp1.cuh"

using namespace conef;

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxFastClasses = 8;
constexpr int kNumTables = 26 + 5 * kMaxFastClasses;
enum { T_FLAT = 0, T_PASS, T_P1, T_P2, T_Q2, T_HIST, T_GS, T_SLOW_FLAT, T_SLOW_P1, T_SLOW_P2, T_FAST_P1,
       T_GS_ONE, T_GS_CLUSTER, T_GS_CLUSTER16, T_GS_REST,   // Gram-Schmidt: one CTA / clusters of 8, 16 / generic
       T_RS,                                                // row sketch: (sketch row, bucket group, column slab)
       T_APPLY,                                             // model update
       T_RS_P12, T_RS_P1C,                                  // low-rank passes 1, 2 on a row-sketch state; pass-1 combine
       T_FV, T_NOFV,                                        // tuned fused step (identity / random-k Q, int8 / int4 C) and the rest
       T_CSK,                                               // count sketch applied run by run: one tile per run
       T_RP1, T_RP1_R8,                                     // low-rank pass 1 with a matrix row per lane (rank 4, rank 8)
       T_Q2_NF,                                             // pass-2 reduce over the tensors the fused passes 2 + 3 do not take
       T_FAST_CLASS0,                                       // + 3 c + {0, 1, 2}: tuned passes 1, 2, 3 of CTA-size class c
       T_FASTNF_CLASS0 = T_FAST_CLASS0 + 3 * kMaxFastClasses };   // + 2 c + {0, 1}: passes 2, 3 without the fused kernel's tensors
// periods per tile of the fused passes 2 + 3: the wanted length, as far as the tile's rows of
// P_hat fit their shared-memory buffer
inline int64_t fused_tile_periods(int rank, int64_t subs, int64_t want)
{
    const int64_t rows_cap = kFuPhBytes / (rank * 4) - 2;
    return std::max<int64_t>(1, std::min<int64_t>(want, rows_cap / subs));
}
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

thread_local std::string g_last_cuda_error;

// everything that follows from the configuration alone
struct Plan {
    std::vector<LayerDesc> layers;
    // tile -> tensor prefix tables.  0..6: all tensors (flat, pass-through, pass 1, pass 2,
    // pass-2 reduce, selection, one-per-tensor); 7..9: flat / pass 1 / pass 2 over the tensors
    // the tuned kernels do not take; 10: tuned pass 1; 11..14: Gram-Schmidt by tensor height;
    // 15: row-sketch step; 16: model update; 17, 18: bucket-major low-rank passes and their combine;
    // 19, 20: tuned fused step of the single-phase compressors and its complement; 21: runs of the
    // chunk-wise count sketch; 22, 23: tiles of the row-per-lane pass 1 (rank 4, rank 8); 24: pass-2 reduce
    // without the fused kernel's tensors; then 3c + {0,1,2}: tuned passes 1, 2, 3 of CTA-size class c, and
    // 2c + {0,1}: passes 2, 3 over the tensors the fused kernel leaves; table 10 (tuned pass 1)
    // counts the tiles of the kernel that adds up the row partials of pass 1
    std::vector<int32_t> pfx[kNumTables];
    std::vector<int> fast_threads;  // CTA size of each class
    std::vector<char> fast_narrow;  // ... and whether its tensors' rows are shorter than 256 elements
    std::vector<int> fast_subs;     // ... and the most rows a period of its tensors spans
    int fast_it[3] = {kFastIt1, kFastIt2, kFastIt3};   // iterations per tile of the tuned passes
    int fast_unit = 256;            // elements per quantisation block
    bool any_fast = false, any_slow = false, any_rs12 = false;
    bool short_tiles = false;   // tile lengths of the tuned passes below their limits
    bool any_fv = false;        // some tensor takes the tuned fused step (conef_flatvec.cuh)
    int fv_tiles = 1;           // ... with this many selection tiles per CTA
    bool any_fused = false;     // some tensor takes the fused passes 2 + 3 (conef_fused.cu)
    int n_fused = 0;
    bool any_csk = false;       // some tensor takes the shared-memory step of the chunk-wise count sketch
    size_t csk_smem = 0;        // ... with this much shared memory per CTA (two windows of the widest run)
    int64_t msg_elems[4] = {0, 0, 0, 0};
    int64_t err_elems = 0;
    int64_t state_stride = 0;  // bytes per worker
    int64_t part_stride = 0;   // floats per worker
    int64_t ppart_stride = 0;  // floats per worker: pass-1 partial rows
    int64_t idx_words = 0, unitoff_words = 0, tileoff_words = 0, sel_words = 0, selbits_words = 0;
    int64_t rs_words = 0;      // row sketch: uint32 words of bucket tables
    int64_t cand_pairs = 0;    // random-k selection: (hash, index) pairs of all candidate lists
    int n_comp = 0;
    // byte offsets in the workspace
    size_t off_layers = 0, off_pfx = 0, off_status = 0, off_sel = 0, off_idx = 0, off_unitoff = 0, off_tileoff = 0, off_selbits = 0,
           off_pbar = 0, off_phat = 0, off_qprev = 0, off_state = 0, off_state_new = 0,
           off_msgv = 0, off_msgp = 0, off_msgq = 0, off_msg1d = 0, off_part = 0, off_ppart = 0, off_rs = 0, off_cand = 0,
           off_ev[2] = {0, 0}, off_unitoff2[2] = {0, 0}, off_tileoff2[2] = {0, 0}, off_selbits2[2] = {0, 0},   // iConEF-v2
           off_fu_units = 0, off_fu_groups = 0, off_fu_hint = 0, off_fu_ctr = 0, off_fu_scratch = 0, off_fu_q = 0,   // fused passes 2 + 3
           total = 0;
    int64_t fu_units = 0;          // (tensor, worker) units of the fused kernel
    int64_t fu_ctr_words = 0;      // the task counter and the units' counters
    int64_t fu_hint_words = 0;     // task block -> group table
    int64_t fu_group_cap = 0;      // entries of the group table
    int64_t fu_scratch_floats = 0; // capacity of the cyclic scratch for tile partials and segment sums
    // strides in floats, padded so that each worker's buffer stays 256-byte aligned
    int64_t msg_stride[4] = {0, 0, 0, 0};
};

inline int64_t pad_floats(int64_t n) { return (int64_t)(align_up((size_t)n * 4) / 4); }

int make_plan(const conef_tensor *tensors, int n_tensors, int n_workers, const conef_q_cfg *q,
              const conef_c_cfg *c, Plan &P)
{
    if (!tensors || !q || !c || n_tensors <= 0 || n_workers <= 0)
        return CONEF_ERR_INVALID_ARG;
    if (n_workers > CONEF_MAX_WORKERS)
        return CONEF_ERR_UNSUPPORTED;
    if (q->kind < CONEF_Q_IDENTITY || q->kind > CONEF_Q_RANDBLOCK)
        return CONEF_ERR_INVALID_ARG;
    if (c->kind < CONEF_C_IDENTITY || c->kind > CONEF_C_STOCHQUANT)
        return CONEF_ERR_INVALID_ARG;
    if (!(c->beta >= 0.f && c->beta < 1.f) || c->iconef < 0 || c->iconef > 2)
        return CONEF_ERR_INVALID_ARG;
    if (c->iconef && (!(c->kind == CONEF_C_IDENTITY || c->kind == CONEF_C_INT8 || c->kind == CONEF_C_INT4) ||
                      c->beta != 0.f))
        return CONEF_ERR_UNSUPPORTED;
    if (c->iconef == 2 && q->kind != CONEF_Q_RANDK && q->kind != CONEF_Q_RANDBLOCK)
        return CONEF_ERR_UNSUPPORTED;   // version 2 keeps e~ = Q(r) as the k values of a second draw
    if ((q->kind == CONEF_Q_RANDK || q->kind == CONEF_Q_RANDBLOCK) && (q->k_num <= 0 || q->k_den <= 0 || q->k_num > q->k_den))
        return CONEF_ERR_INVALID_ARG;
    if (q->kind == CONEF_Q_LOWRANK && (q->rank < 1 || q->rank > CONEF_MAX_RANK))
        return q->rank < 1 ? CONEF_ERR_INVALID_ARG : CONEF_ERR_UNSUPPORTED;
    int unit = 256;
    if (c->kind == CONEF_C_INT8 || c->kind == CONEF_C_INT4) {
        const int b = c->block;
        if (!(b == 32 || b == 64 || b == 128 || b == 256) || (c->kind == CONEF_C_INT4 && b < 64))
            return CONEF_ERR_INVALID_ARG;
        if (c->scale_dtype != CONEF_SCALE_FP32 && c->scale_dtype != CONEF_SCALE_FP16)
            return CONEF_ERR_INVALID_ARG;
        unit = b;
    }
    if (c->kind == CONEF_C_COUNTSKETCH || c->kind == CONEF_C_ROWSKETCH) {
        if (c->cs_rows < 1 || c->cs_rows > 7 || (c->cs_rows % 2) == 0 || c->cs_col_div < 1)
            return CONEF_ERR_INVALID_ARG;
    }
    if (c->kind == CONEF_C_COUNTSKETCH && c->cs_chunk != 0) {
        if (c->cs_chunk < 0 || c->cs_chunk % 256 != 0 || (int64_t)c->cs_chunk < 4 * c->cs_col_div)
            return CONEF_ERR_INVALID_ARG;
    }
    if (c->kind == CONEF_C_STOCHQUANT) {
        const int b = c->block;
        if (!(b == 32 || b == 64 || b == 128 || b == 256) || c->levels < 1 || c->levels > 32767)
            return CONEF_ERR_INVALID_ARG;
        unit = b;
    }
    if (c->kind == CONEF_C_ROWSKETCH) {
        if (c->scale_dtype != CONEF_SCALE_FP32 && c->scale_dtype != CONEF_SCALE_FP16)
            return CONEF_ERR_INVALID_ARG;
        unit = 32;
    }   // message slots are handed out per aligned group of 32 elements
    const int scale_bytes = (c->scale_dtype == CONEF_SCALE_FP16) ? 2 : 4;

    P.layers.assign(n_tensors, LayerDesc{});
    for (auto &v : P.pfx)
        v.assign(n_tensors + 1, 0);
    {   // the tuned fused step gives a CTA four selection tiles where that still leaves about 16 CTAs per SM
        int64_t total = 0;
        for (int l = 0; l < n_tensors; ++l)
            if (tensors[l].rows > 0 && tensors[l].cols > 0 && tensors[l].rows <= 0xFFFFFFFFLL / tensors[l].cols)
                total += tensors[l].rows * tensors[l].cols;
        P.fv_tiles = total * n_workers / (kHistTile * kFvTiles) >= kPlanSMs * 16 ? kFvTiles : 1;
    }
    // tile lengths of the tuned low-rank passes from the model's size
    int it1 = kFastIt1, it2 = kFastIt2, it3 = kFastIt3;
    if (q->kind == CONEF_Q_LOWRANK) {
        int64_t cta_iters = 0;
        for (int l = 0; l < n_tensors; ++l) {
            LayerDesc T{};
            T.rows = tensors[l].rows;
            T.cols = tensors[l].cols;
            if (T.rows <= 0 || T.cols <= 1 || !tensors[l].compress || T.rows > 0xFFFFFFFFLL / T.cols)
                continue;
            T.d = T.rows * T.cols;
            T.rank = (int)std::min<int64_t>(q->rank, std::min(T.rows, T.cols));
            fast_classify(T, c->kind, unit, q->rank);   // offsets are zero here: only the geometry matters
            if (T.fast)
                cta_iters += T.f_niter * T.f_ncg;
        }
        cta_iters *= n_workers;
        it1 = fast_tile_iters(kFastIt1, cta_iters);
        it2 = fast_tile_iters(kFastIt2, cta_iters);
        it3 = fast_tile_iters(kFastIt3, cta_iters);
        if (it1 != kFastIt1 || it2 != kFastIt2 || it3 != kFastIt3)
            P.short_tiles = true;
        else
            it1 = kFastIt1, it2 = kFastIt2, it3 = kFastIt3;
    }
    P.fast_it[0] = it1, P.fast_it[1] = it2, P.fast_it[2] = it3;
    P.fast_unit = unit;
    int64_t g_off = 0, state_off = 0;
    for (int l = 0; l < n_tensors; ++l) {
        const conef_tensor &t = tensors[l];
        if (t.rows <= 0 || t.cols <= 0)
            return CONEF_ERR_INVALID_ARG;
        if (t.rows > 0xFFFFFFFFLL / t.cols)
            return CONEF_ERR_UNSUPPORTED;  // indices are 32-bit
        LayerDesc &L = P.layers[l];
        L.rows = t.rows;
        L.cols = t.cols;
        L.d = t.rows * t.cols;
        L.g_off = g_off;
        g_off += L.d;
        L.compressed = (t.compress != 0 && t.cols > 1) ? 1 : 0;
        L.cidx = -1;
        int tiles[kNumTables] = {0};
        if (!L.compressed) {
            L.msg1d_off = P.msg_elems[CONEF_MSG_DENSE1D];
            P.msg_elems[CONEF_MSG_DENSE1D] += L.d;
            tiles[T_PASS] = (int)ceil_div(L.d, kPassTile);
        } else {
            L.cidx = P.n_comp++;
            L.unit = unit;
            L.nunits = ceil_div(L.d, unit);
            L.e_off = P.err_elems;
            P.err_elems += L.d;
            // error state of one worker
            L.a_off = state_off;
            switch (c->kind) {
            case CONEF_C_IDENTITY: L.a_bytes = L.d * 4; break;
            case CONEF_C_INT8: L.a_bytes = L.d; break;
            case CONEF_C_INT4: L.a_bytes = (L.d + 1) / 2; break;
            case CONEF_C_STOCHQUANT: L.a_bytes = L.d * (c->levels > 127 ? 2 : 1); break;
            case CONEF_C_ROWSKETCH:
                L.w = L.rows / c->cs_col_div < 1 ? 1 : L.rows / c->cs_col_div;
                L.a_bytes = (int64_t)c->cs_rows * L.w * L.cols * (c->scale_dtype == CONEF_SCALE_FP16 ? 2 : 4);
                L.rs_info_off = P.rs_words;
                L.rs_ptr_off = L.rs_info_off + (int64_t)c->cs_rows * L.rows;
                L.rs_row_off = L.rs_ptr_off + (int64_t)c->cs_rows * (L.w + 1);
                P.rs_words = L.rs_row_off + (int64_t)c->cs_rows * L.rows;
                // four columns per thread where 16-byte accesses line up (random-k also needs message
                // units that do not straddle rows)
                L.rs_vec = (L.cols % 4 == 0 && L.g_off % 4 == 0 && (q->kind != CONEF_Q_RANDK || L.cols % 32 == 0)) ? 4 : 1;
                tiles[T_RS] = (int)(c->cs_rows * ceil_div(L.w, kRsBuckets) * ceil_div(L.cols, kRsThreads * L.rs_vec));
                break;
            default:
                L.w = L.d / c->cs_col_div < 1 ? 1 : L.d / c->cs_col_div;
                L.a_bytes = (int64_t)c->cs_rows * L.w * 4;
            }
            state_off += (int64_t)align_up((size_t)L.a_bytes);
            if (c->kind == CONEF_C_INT8 || c->kind == CONEF_C_INT4 || c->kind == CONEF_C_STOCHQUANT) {
                L.b_off = state_off;
                L.b_bytes = L.nunits * (c->kind == CONEF_C_STOCHQUANT ? 4 : scale_bytes);
                state_off += (int64_t)align_up((size_t)L.b_bytes);
            }
            if (c->iconef == 1) {   // the second state q (Alg. 3), laid out like the first
                L.a2_off = state_off;
                state_off += (int64_t)align_up((size_t)L.a_bytes);
                L.b2_off = state_off;
                state_off += (int64_t)align_up((size_t)L.b_bytes);
            }
            tiles[T_FLAT] = (int)ceil_div(L.nunits, kFlatUnitsPerCta);
            tiles[T_GS] = 1;
            if (q->kind == CONEF_Q_IDENTITY) {
                L.k = L.d;
            } else if (q->kind == CONEF_Q_RANDBLOCK) {
                unsigned __int128 kk = (unsigned __int128)L.d * (unsigned __int128)q->k_num /
                                       (unsigned __int128)q->k_den;
                L.k = kk < 1 ? 1 : (int64_t)kk;
                L.idx_off = P.idx_words;
                P.idx_words += L.k;
            } else if (q->kind == CONEF_Q_RANDK) {
                // k = max(1, floor(d * k_num / k_den)) without overflow: d < 2^32
                unsigned __int128 kk = (unsigned __int128)L.d * (unsigned __int128)q->k_num /
                                       (unsigned __int128)q->k_den;
                L.k = kk < 1 ? 1 : (int64_t)kk;
                L.idx_off = P.idx_words;
                P.idx_words += L.k;
                L.unitoff_off = P.unitoff_words;
                P.unitoff_words += L.nunits;
                L.tileoff_off = P.tileoff_words;
                P.tileoff_words += ceil_div(L.d, kHistTile);
                L.selbits_off = P.selbits_words;
                P.selbits_words += ceil_div(L.d, 32) + 8;   // whole 256-element groups may be read
                L.sel_off = P.sel_words;
                P.sel_words += kSelWords;
                // candidates of the second selection level: d / 2048 expected; room for twice that and a margin
                L.cand_off = P.cand_pairs;
                L.cand_cap = L.d / 1024 + 1024;
                P.cand_pairs += L.cand_cap;
                tiles[T_HIST] = (int)ceil_div(L.d, kHistTile);
            }
            if (q->kind != CONEF_Q_LOWRANK) {
                L.msgv_off = P.msg_elems[CONEF_MSG_VALUES];
                P.msg_elems[CONEF_MSG_VALUES] += L.k;
                // the tuned fused step: whole 8-element groups, 16-byte accesses, Alg. 2 proper
                const bool fv = (c->kind == CONEF_C_INT8 || c->kind == CONEF_C_INT4 ||
                                 (c->kind == CONEF_C_STOCHQUANT && c->levels <= 127)) && c->beta == 0.f &&
                                (c->iconef == 0 || c->kind != CONEF_C_STOCHQUANT) &&
                                L.d % 8 == 0 && L.g_off % 4 == 0 && L.d < (1ll << 31) &&
                                (q->kind != CONEF_Q_IDENTITY || L.msgv_off % 4 == 0);
                // the chunk-wise count sketch: a run's two windows in shared memory
                const int64_t csk_floats = c->kind == CONEF_C_COUNTSKETCH && c->cs_chunk > 0
                                               ? 2 * c->cs_rows * chunk_window_max(L.d, L.w, c->cs_chunk) : 0;
                if (fv) {
                    P.any_fv = true;
                    tiles[T_FV] = (int)ceil_div(L.d, (int64_t)kHistTile * P.fv_tiles);
                } else if (csk_floats > 0 && csk_floats * 4 <= 200 * 1024) {
                    P.any_csk = true;
                    P.csk_smem = std::max(P.csk_smem, (size_t)csk_floats * 4);
                    tiles[T_CSK] = (int)std::max<int64_t>(1, L.d / c->cs_chunk);
                } else {
                    tiles[T_NOFV] = tiles[T_FLAT];
                }
            } else {
                int64_t r = q->rank;
                if (r > L.rows) r = L.rows;
                if (r > L.cols) r = L.cols;
                L.rank = (int)r;
                L.msgp_off = P.msg_elems[CONEF_MSG_P];
                P.msg_elems[CONEF_MSG_P] += L.rows * r;
                L.msgq_off = P.msg_elems[CONEF_MSG_Q];
                P.msg_elems[CONEF_MSG_Q] += L.cols * r;
                const int64_t rtiles = ceil_div(L.rows, kP2RowsPerTile);
                L.p2_rows_generic = rtiles;
                tiles[T_P1] = (int)ceil_div(L.rows, kP1RowsPerCta);
                tiles[T_P2] = (int)(rtiles * ceil_div(L.cols, kP2ColsPerCta));
                tiles[T_Q2] = (int)ceil_div(L.cols * r, kQ2PerCta);
                const int64_t gs_cta = gs_rows_per_cta(q->rank <= 4 ? 4 : 8);
                if (L.rows <= gs_cta)
                    tiles[T_GS_ONE] = 1;
                else if (L.rows <= 8 * gs_cta)
                    tiles[T_GS_CLUSTER] = 1;
                else if (L.rows <= 16 * gs_cta)
                    tiles[T_GS_CLUSTER16] = 1;
                else
                    tiles[T_GS_REST] = 1;
                fast_classify(L, c->kind, unit, q->rank, it1, it2, it3);
                if (c->iconef)
                    L.fast = 0;   // the tuned kernels implement Alg. 2 and Alg. 4, not Alg. 3
                int cls = -1;
                if (L.fast) {
                    const char narrow = L.cols < 256;
                    for (size_t k = 0; k < P.fast_threads.size(); ++k)
                        if (P.fast_threads[k] == L.f_threads && P.fast_narrow[k] == narrow)
                            cls = (int)k;
                    if (cls < 0 && (int)P.fast_threads.size() < kMaxFastClasses) {
                        cls = (int)P.fast_threads.size();
                        P.fast_threads.push_back(L.f_threads);
                        P.fast_narrow.push_back(narrow);
                        P.fast_subs.push_back(0);
                    }
                    if (cls < 0)
                        L.fast = 0;
                    else
                        P.fast_subs[cls] = std::max(P.fast_subs[cls], (int)L.f_subs);
                }
                if (c->kind == CONEF_C_ROWSKETCH && c->cs_rows == 1 && L.rs_vec == 4 && c->beta >= 0.f) {
                    // bucket-major passes 1 and 2 (conef_rowsketch.cuh)
                    L.fast = 2;
                    P.any_rs12 = true;
                    const int64_t groups = ceil_div(L.w, kRsBuckets), slabs = ceil_div(L.cols, kRsThreads * 4);
                    L.p2_rows_fast = groups;
                    L.f_j = (int32_t)(slabs * (kRsThreads / 32));
                    tiles[T_RS_P12] = (int)(groups * slabs);
                    tiles[T_RS_P1C] = (int)ceil_div(L.rows * r, 256);
                    L.pp_off = P.ppart_stride;
                    P.ppart_stride += (int64_t)L.f_j * L.rows * r;
                } else if (L.fast) {
                    P.any_fast = true;
                    L.p2_rows_fast = (int64_t)L.f_rt2 * L.f_subs;
                    // pass 1 with a row per lane where the configuration and the shape allow it
                    if (c->kind == CONEF_C_INT4 && c->scale_dtype == CONEF_SCALE_FP16 && c->block == 128 &&
                        rows_p1_takes(L)) {
                        tiles[L.rank == 4 ? T_RP1 : T_RP1_R8] = (int)ceil_div(L.rows, rp_rows(L.rank));
                    } else {
                        tiles[T_FAST_P1] = (int)ceil_div(L.rows * r, 256);
                        tiles[T_FAST_CLASS0 + 3 * cls] = L.f_rt1 * L.f_ncg;
                    }
                    tiles[T_FAST_CLASS0 + 3 * cls + 1] = L.f_rt2 * L.f_ncg;
                    tiles[T_FAST_CLASS0 + 3 * cls + 2] = L.f_rt3 * L.f_ncg;
                    // the fused passes 2 + 3: rows at least a warp-iteration wide, the block size of
                    // the kernel's layout, few enough segments per period
                    L.f_fused = (c->beta == 0.f && L.cols >= 256 && L.f_lcm / 256 <= kFuMaxSeg &&
                                 unit == (c->kind == CONEF_C_INT4 ? 128 : 256)) ? 1 : 0;
                    if (L.f_fused) {
                        P.any_fused = true;
                        ++P.n_fused;
                    } else {
                        tiles[T_FASTNF_CLASS0 + 2 * cls] = L.f_rt2 * L.f_ncg;
                        tiles[T_FASTNF_CLASS0 + 2 * cls + 1] = L.f_rt3 * L.f_ncg;
                    }
                    L.pp_off = P.ppart_stride;
                    P.ppart_stride += (int64_t)L.f_j * L.rows * r;
                } else {
                    P.any_slow = true;
                    tiles[T_SLOW_FLAT] = tiles[T_FLAT];
                    tiles[T_SLOW_P1] = tiles[T_P1];
                    tiles[T_SLOW_P2] = tiles[T_P2];
                }
                if (!L.f_fused)
                    tiles[T_Q2_NF] = tiles[T_Q2];
                L.part_off = P.part_stride;
                P.part_stride += std::max(L.p2_rows_generic, L.p2_rows_fast) * L.cols * r;
            }
        }
        tiles[T_APPLY] = (int)apply_tiles(L, q->kind);
        for (int k = 0; k < kNumTables; ++k)
            P.pfx[k][l + 1] = P.pfx[k][l] + tiles[k];
    }
    P.state_stride = state_off;
    for (int k = 0; k < 4; ++k)
        P.msg_stride[k] = pad_floats(P.msg_elems[k]);
    P.part_stride = pad_floats(P.part_stride);
    P.ppart_stride = pad_floats(P.ppart_stride);

    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t at = off;
        off += align_up(bytes);
        return at;
    };
    P.off_layers = take(sizeof(LayerDesc) * n_tensors);
    P.off_pfx = take(sizeof(int32_t) * kNumTables * (n_tensors + 1));
    P.off_status = take(256);
    P.off_sel = take((size_t)P.sel_words * 4);
    P.off_idx = take((size_t)P.idx_words * 4);
    P.off_unitoff = take((size_t)P.unitoff_words * 4);
    P.off_tileoff = take((size_t)P.tileoff_words * 4);
    P.off_selbits = take((size_t)P.selbits_words * 4);
    P.off_pbar = take((size_t)P.msg_elems[CONEF_MSG_P] * 4);
    P.off_phat = take((size_t)P.msg_elems[CONEF_MSG_P] * 4);
    P.off_qprev = take((size_t)P.msg_elems[CONEF_MSG_Q] * 4);
    P.off_state = take((size_t)P.state_stride * n_workers);
    P.off_state_new = (c->kind == CONEF_C_COUNTSKETCH || c->kind == CONEF_C_ROWSKETCH)
                          ? take((size_t)P.state_stride * n_workers)
                          : P.off_state;
    P.off_msgv = take((size_t)P.msg_stride[CONEF_MSG_VALUES] * 4 * n_workers);
    P.off_msgp = take((size_t)P.msg_stride[CONEF_MSG_P] * 4 * n_workers);
    P.off_msgq = take((size_t)P.msg_stride[CONEF_MSG_Q] * 4 * n_workers);
    P.off_msg1d = take((size_t)P.msg_stride[CONEF_MSG_DENSE1D] * 4 * n_workers);
    P.off_part = take((size_t)P.part_stride * 4 * n_workers);
    P.off_ppart = take((size_t)P.ppart_stride * 4 * n_workers);
    P.off_rs = take((size_t)P.rs_words * 4);
    P.off_cand = take((size_t)P.cand_pairs * 8);
    if (c->iconef == 2)   // two value buffers per worker and the structures of two more draws of Q
        for (int x = 0; x < 2; ++x) {
            P.off_ev[x] = take((size_t)P.msg_stride[CONEF_MSG_VALUES] * 4 * n_workers);
            P.off_unitoff2[x] = take((size_t)P.unitoff_words * 4);
            P.off_tileoff2[x] = take((size_t)P.tileoff_words * 4);
            P.off_selbits2[x] = take((size_t)P.selbits_words * 4);
        }
    if (P.any_fused) {
        // unit and task-group tables, the task counter and the units' counters, a cyclic scratch for
        // the tiles' partial Q_i and the segments' sums (at least twice the largest unit at the default
        // tile length), and a second Q_i buffer that takes the kernel's own Q_i when a caller injects
        // the Q_i of the residual
        P.fu_units = (int64_t)P.n_fused * n_workers;
        int64_t largest = 0, words = 64, tasks = 0;
        for (const LayerDesc &L : P.layers)
            if (L.compressed && L.f_fused) {
                const int64_t ncg = L.f_lcm / 256, ntp = ceil_div(L.f_niter, fused_tile_periods(q->rank, L.f_subs, kFuTilePeriods));
                largest = std::max(largest, ncg * (ntp + 1) * 256 * q->rank);
                words += (ncg + 2) * n_workers;
                tasks += 2 * ncg * ntp * n_workers;
            }
        P.fu_hint_words = std::max<int64_t>(65536, tasks / 4 + 64);   // room for tiles an eighth as long as the default
        P.fu_group_cap = std::max<int64_t>(65536, tasks + 4 * P.fu_units);
        P.fu_ctr_words = words;
        P.fu_scratch_floats = std::max<int64_t>(2 * largest, (int64_t)16 << 20);
        P.off_fu_units = take((size_t)P.fu_units * sizeof(FusedUnit));
        P.off_fu_groups = take((size_t)P.fu_group_cap * sizeof(FusedGroup));
        P.off_fu_hint = take((size_t)P.fu_hint_words * 4);
        P.off_fu_ctr = take((size_t)P.fu_ctr_words * 4);
        P.off_fu_scratch = take((size_t)P.fu_scratch_floats * 4);
        P.off_fu_q = take((size_t)P.msg_stride[CONEF_MSG_Q] * 4 * n_workers);
    }
    P.total = off;
    return CONEF_OK;
}

}  // namespace

struct conef_ctx {
    Plan plan;
    conef_q_cfg q;
    conef_c_cfg c;
    int n_layers = 0, n_workers = 0;
    uint8_t *ws = nullptr;
    DevView view;
    int64_t last_step = -1;
    int expect = 0;        // low-rank call order: 0 idle, 1 after phase 0, 2 after reduce P,
                           // 3 after phase 2, 4 after phase 1/3
    bool stepped = false;  // a step has run (messages exist)
    int sketch_cur = 0;
    int ev_cur = 0;            // iConEF-v2: which value buffer holds e~
    int64_t ev_step = -1;      // ... and the step whose second draw of Q stored it (-1: e~ = 0)
    int64_t draw_step[2] = {-1, -1};   // the step whose second draw each set of selection structures holds
    int fast = 1;
    int sm_count = kPlanSMs;   // of the device the context was created on (read in conef_init)
    int64_t launches = 0;
    // fused passes 2 + 3 (conef_fused.cu): on by default where the device allows
    int fused = 0, fused_tile_periods = kFuTilePeriods, fused_ctas_per_sm = 2;
    bool fused_ready = false;       // configuration and task list exist for this device
    bool fused_dirty = false;       // the tables on the device are older than the host's
    FusedConfig fcfg{};
    std::vector<FusedUnit> fu_units;
    std::vector<FusedGroup> fu_groups;
    std::vector<uint32_t> fu_hint;
    int fu_tasks = 0;
    // side streams on which the CTA-size classes of a tuned pass run next to one another
    cudaStream_t aux[kMaxFastClasses] = {};
    cudaEvent_t ev_fork = nullptr, ev_join[kMaxFastClasses] = {};
    int n_aux = 0;
    ~conef_ctx()
    {
        for (int k = 0; k < n_aux; ++k) {
            cudaEventDestroy(ev_join[k]);
            cudaStreamDestroy(aux[k]);
        }
        if (ev_fork)
            cudaEventDestroy(ev_fork);
    }
};

namespace {

#define CK_CUDA(expr)                                                     \
    do {                                                                  \
        cudaError_t e_ = (expr);                                          \
        if (e_ != cudaSuccess) {                                          \
            g_last_cuda_error = std::string(#expr) + ": " + cudaGetErrorString(e_); \
            return CONEF_ERR_CUDA;                                        \
        }                                                                 \
    } while (0)

#define LAUNCH_CHECK(ctx)                       \
    do {                                        \
        (ctx)->launches++;                      \
        CK_CUDA(cudaGetLastError());            \
    } while (0)

inline const int32_t *table_ptr(const conef_ctx *ctx, int which)
{
    return (const int32_t *)(ctx->ws + ctx->plan.off_pfx) + (size_t)which * (ctx->n_layers + 1);
}

void fill_view(conef_ctx *ctx)
{
    const Plan &P = ctx->plan;
    DevView &V = ctx->view;
    memset(&V, 0, sizeof(V));
    uint8_t *ws = ctx->ws;
    V.layers = (const LayerDesc *)(ws + P.off_layers);
    V.n_layers = ctx->n_layers;
    V.n_workers = ctx->n_workers;
    V.qkind = ctx->q.kind;
    V.ckind = ctx->c.kind;
    V.bits = ctx->c.kind == CONEF_C_INT8 ? 8 : 4;
    V.scale_half = ctx->c.scale_dtype == CONEF_SCALE_FP16;
    V.cs_rows = ctx->c.cs_rows;
    V.block = ctx->c.block;
    V.n_workers_f = (float)ctx->n_workers;
    V.seed_q = ctx->q.seed;
    V.seed_c = ctx->c.seed;
    V.state = ws + P.off_state;
    V.state_new = ws + P.off_state_new;
    V.state_stride = P.state_stride;
    V.msgv = (float *)(ws + P.off_msgv);
    V.msgv_stride = P.msg_stride[CONEF_MSG_VALUES];
    V.msgp = (float *)(ws + P.off_msgp);
    V.msgp_stride = P.msg_stride[CONEF_MSG_P];
    V.msgq = (float *)(ws + P.off_msgq);
    V.msgq_stride = P.msg_stride[CONEF_MSG_Q];
    V.msg1d = (float *)(ws + P.off_msg1d);
    V.msg1d_stride = P.msg_stride[CONEF_MSG_DENSE1D];
    V.part = (float *)(ws + P.off_part);
    V.part_stride = P.part_stride;
    V.ppart = (float *)(ws + P.off_ppart);
    V.ppart_stride = P.ppart_stride;
    V.pbar = (float *)(ws + P.off_pbar);
    V.phat = (float *)(ws + P.off_phat);
    V.qprev = (float *)(ws + P.off_qprev);
    V.idx = (uint32_t *)(ws + P.off_idx);
    V.unitoff = (uint32_t *)(ws + P.off_unitoff);
    V.tileoff = (uint32_t *)(ws + P.off_tileoff);
    V.selbits = (uint32_t *)(ws + P.off_selbits);
    V.fv_tiles = P.fv_tiles;
    V.sel = (uint32_t *)(ws + P.off_sel);
    V.cand = (uint32_t *)(ws + P.off_cand);
    V.status = (int32_t *)(ws + P.off_status);
    V.rs = (const uint32_t *)(ws + P.off_rs);
    V.pfx_rs = table_ptr(ctx, T_RS);
    V.iconef = ctx->c.iconef;
    V.unitoffA = (uint32_t *)(ws + P.off_unitoff2[0]);
    V.tileoffA = (uint32_t *)(ws + P.off_tileoff2[0]);
    V.selbitsA = (uint32_t *)(ws + P.off_selbits2[0]);
    V.unitoffB = (uint32_t *)(ws + P.off_unitoff2[1]);
    V.tileoffB = (uint32_t *)(ws + P.off_tileoff2[1]);
    V.selbitsB = (uint32_t *)(ws + P.off_selbits2[1]);
    V.ev_old = V.ev_new = nullptr;
    V.ev_step = -1;
    V.ev_valid = 0;
    V.ev_pad = 0;
    V.cs_chunk = ctx->c.kind == CONEF_C_COUNTSKETCH ? ctx->c.cs_chunk : 0;
    V.levels = ctx->c.levels;
    V.sq_wide = ctx->c.levels > 127;
    V.beta = ctx->c.beta;
    V.omb = 1.0f - ctx->c.beta;
    V.pfx_flat = table_ptr(ctx, T_FLAT);
    V.pfx_pass = table_ptr(ctx, T_PASS);
    V.pfx_p1 = table_ptr(ctx, T_P1);
    V.pfx_p2 = table_ptr(ctx, T_P2);
    V.pfx_q2 = table_ptr(ctx, T_Q2);
    V.pfx_hist = table_ptr(ctx, T_HIST);
    V.pfx_gs = table_ptr(ctx, T_GS);
}

inline int tiles_of(const conef_ctx *ctx, int which) { return ctx->plan.pfx[which][ctx->n_layers]; }

// the view for this call: sketch buffers in their current roles
DevView current_view(const conef_ctx *ctx)
{
    DevView V = ctx->view;
    if ((ctx->c.kind == CONEF_C_COUNTSKETCH || ctx->c.kind == CONEF_C_ROWSKETCH) && ctx->sketch_cur) {
        uint8_t *t = V.state;
        V.state = V.state_new;
        V.state_new = t;
    }
    if (ctx->c.iconef == 2) {
        V.ev_old = (float *)(ctx->ws + ctx->plan.off_ev[ctx->ev_cur]);
        V.ev_new = (float *)(ctx->ws + ctx->plan.off_ev[ctx->ev_cur ^ 1]);
        V.ev_step = ctx->ev_step;
        V.ev_valid = ctx->ev_step >= 0;
        // the structures of a draw live beside the values it stored
        const Plan &P = ctx->plan;
        const int a = ctx->ev_cur, b = ctx->ev_cur ^ 1;
        V.unitoffA = (uint32_t *)(ctx->ws + P.off_unitoff2[a]);
        V.tileoffA = (uint32_t *)(ctx->ws + P.off_tileoff2[a]);
        V.selbitsA = (uint32_t *)(ctx->ws + P.off_selbits2[a]);
        V.unitoffB = (uint32_t *)(ctx->ws + P.off_unitoff2[b]);
        V.tileoffB = (uint32_t *)(ctx->ws + P.off_tileoff2[b]);
        V.selbitsB = (uint32_t *)(ctx->ws + P.off_selbits2[b]);
    }
    return V;
}

// the fused step on a row-sketch error state (all of decode, p, Q's message or residual, update)
template <int QK>
int launch_rowsketch(conef_ctx *ctx, const DevView &V, cudaStream_t s)
{
    const int n = tiles_of(ctx, T_RS);
    if (n == 0)
        return CONEF_OK;
    dim3 grid(n, ctx->n_workers);
    if (ctx->c.cs_rows == 1)
        k_rowsketch<QK, true><<<grid, kRsThreads, 0, s>>>(V);
    else
        k_rowsketch<QK, false><<<grid, kRsThreads, 0, s>>>(V);
    LAUNCH_CHECK(ctx);
    return CONEF_OK;
}

template <int QK>
int launch_flat(conef_ctx *ctx, DevView V, cudaStream_t s, int table = T_FLAT)
{
    if (ctx->c.kind == CONEF_C_ROWSKETCH)
        return launch_rowsketch<QK>(ctx, V, s);
    const int n = tiles_of(ctx, table);
    V.pfx_flat = table_ptr(ctx, table);
    if (n == 0)
        return CONEF_OK;
    dim3 grid(n, ctx->n_workers);
    switch (ctx->c.kind) {
    case CONEF_C_IDENTITY: k_flat<QK, CONEF_C_IDENTITY><<<grid, kFlatThreads, 0, s>>>(V); break;
    case CONEF_C_INT8: k_flat<QK, CONEF_C_INT8><<<grid, kFlatThreads, 0, s>>>(V); break;
    case CONEF_C_INT4: k_flat<QK, CONEF_C_INT4><<<grid, kFlatThreads, 0, s>>>(V); break;
    case CONEF_C_STOCHQUANT: k_flat<QK, CONEF_C_STOCHQUANT><<<grid, kFlatThreads, 0, s>>>(V); break;
    default: k_flat<QK, CONEF_C_COUNTSKETCH><<<grid, kFlatThreads, 0, s>>>(V); break;
    }
    LAUNCH_CHECK(ctx);
    return CONEF_OK;
}

int launch_pass1(conef_ctx *ctx, DevView V, cudaStream_t s, int table = T_P1)
{
    const int n = tiles_of(ctx, table);
    V.pfx_p1 = table_ptr(ctx, table);
    if (n == 0)
        return CONEF_OK;
    dim3 grid(n, ctx->n_workers);
    switch (ctx->c.kind) {
    case CONEF_C_IDENTITY: k_lr_pass1<CONEF_C_IDENTITY><<<grid, 256, 0, s>>>(V); break;
    case CONEF_C_INT8: k_lr_pass1<CONEF_C_INT8><<<grid, 256, 0, s>>>(V); break;
    case CONEF_C_INT4: k_lr_pass1<CONEF_C_INT4><<<grid, 256, 0, s>>>(V); break;
    case CONEF_C_ROWSKETCH: k_lr_pass1<CONEF_C_ROWSKETCH><<<grid, 256, 0, s>>>(V); break;
    case CONEF_C_STOCHQUANT: k_lr_pass1<CONEF_C_STOCHQUANT><<<grid, 256, 0, s>>>(V); break;
    default: k_lr_pass1<CONEF_C_COUNTSKETCH><<<grid, 256, 0, s>>>(V); break;
    }
    LAUNCH_CHECK(ctx);
    return CONEF_OK;
}

int launch_pass2(conef_ctx *ctx, DevView V, cudaStream_t s, int table = T_P2)
{
    const int n = tiles_of(ctx, table);
    if (n == 0)
        return CONEF_OK;
    V.pfx_p2 = table_ptr(ctx, table);
    dim3 grid(n, ctx->n_workers);
    switch (ctx->c.kind) {
    case CONEF_C_IDENTITY: k_lr_pass2<CONEF_C_IDENTITY><<<grid, kP2ColsPerCta, 0, s>>>(V); break;
    case CONEF_C_INT8: k_lr_pass2<CONEF_C_INT8><<<grid, kP2ColsPerCta, 0, s>>>(V); break;
    case CONEF_C_INT4: k_lr_pass2<CONEF_C_INT4><<<grid, kP2ColsPerCta, 0, s>>>(V); break;
    case CONEF_C_ROWSKETCH: k_lr_pass2<CONEF_C_ROWSKETCH><<<grid, kP2ColsPerCta, 0, s>>>(V); break;
    case CONEF_C_STOCHQUANT: k_lr_pass2<CONEF_C_STOCHQUANT><<<grid, kP2ColsPerCta, 0, s>>>(V); break;
    default: k_lr_pass2<CONEF_C_COUNTSKETCH><<<grid, kP2ColsPerCta, 0, s>>>(V); break;
    }
    LAUNCH_CHECK(ctx);
    return CONEF_OK;
}

// second stage of pass 2: sums the per-tile partials of every tensor in tile order
int launch_pass2_reduce(conef_ctx *ctx, DevView V, cudaStream_t s, bool skip_fused = false)
{
    const int table = skip_fused ? T_Q2_NF : T_Q2;
    if (tiles_of(ctx, table) == 0)
        return CONEF_OK;
    V.pfx_q2 = table_ptr(ctx, table);
    dim3 grid2(tiles_of(ctx, table), ctx->n_workers);
    k_lr_pass2_reduce<<<grid2, 256, 0, s>>>(V);
    LAUNCH_CHECK(ctx);
    return CONEF_OK;
}

// the tuned kernels on the tensors they take (pass 1: one launch; passes 2, 3: one per CTA size)
int launch_fast(conef_ctx *ctx, int pass, const DevView &V, cudaStream_t s, bool skip_fused = false)
{
    const Plan &P = ctx->plan;
    // The classes touch different tensors: all but the first go to side streams that fork from
    // and join back into the caller's stream, so that their (often small) grids share the GPU.
    const bool side = ctx->n_aux > 0 && P.fast_threads.size() > 1;
    if (side)
        CK_CUDA(cudaEventRecord(ctx->ev_fork, s));
    int used = 0;
    for (size_t k = 0; k < P.fast_threads.size(); ++k) {
        const int table = skip_fused && pass >= 2 ? T_FASTNF_CLASS0 + 2 * (int)k + (pass - 2) : T_FAST_CLASS0 + 3 * (int)k + (pass - 1);
        const int n = tiles_of(ctx, table);
        if (n == 0)
            continue;
        cudaStream_t sk = s;
        const bool off_main = side && k > 0 && used < ctx->n_aux;
        if (off_main) {
            sk = ctx->aux[used];
            CK_CUDA(cudaStreamWaitEvent(sk, ctx->ev_fork, 0));
        }
        const size_t stage = fast_stage_bytes(pass, ctx->q.rank, P.fast_it[pass - 1], P.fast_subs[k], P.fast_threads[k],
                                              P.fast_unit, V.scale_half ? 2 : 4);
        CK_CUDA(fast_launch(pass, ctx->c.kind, ctx->q.rank, V.scale_half, V, table_ptr(ctx, table), n, P.fast_threads[k], sk,
                            P.short_tiles, P.fast_narrow[k] != 0, stage));
        LAUNCH_CHECK(ctx);
        if (off_main) {
            CK_CUDA(cudaEventRecord(ctx->ev_join[used], sk));
            ++used;
        }
    }
    for (int k = 0; k < used; ++k)
        CK_CUDA(cudaStreamWaitEvent(s, ctx->ev_join[k], 0));
    if (pass == 1 && tiles_of(ctx, T_RP1) > 0) {
        CK_CUDA(rows_p1_launch<4>(V, table_ptr(ctx, T_RP1), tiles_of(ctx, T_RP1), s));
        LAUNCH_CHECK(ctx);
    }
    if (pass == 1 && tiles_of(ctx, T_RP1_R8) > 0) {
        CK_CUDA(rows_p1_launch<8>(V, table_ptr(ctx, T_RP1_R8), tiles_of(ctx, T_RP1_R8), s));
        LAUNCH_CHECK(ctx);
    }
    if (pass == 1 && tiles_of(ctx, T_FAST_P1) > 0) {
        // P_i = sum of the per-segment row partials
        CK_CUDA(fast_launch_p1_combine(ctx->q.rank, V, table_ptr(ctx, T_FAST_P1), tiles_of(ctx, T_FAST_P1), s));
        LAUNCH_CHECK(ctx);
    }
    return CONEF_OK;
}

// zero the sketch being built, run `body`, then swap the two sketch buffers
template <class F>
int with_new_sketch(conef_ctx *ctx, const DevView &V, cudaStream_t s, F body)
{
    const bool sk = ctx->c.kind == CONEF_C_COUNTSKETCH || ctx->c.kind == CONEF_C_ROWSKETCH;
    // built by atomic adds; the row sketch, and the run-by-run step where it takes every tensor, write
    // every entry themselves
    const bool all_csk = ctx->fast && ctx->plan.any_csk && tiles_of(ctx, T_NOFV) == 0 && ctx->q.kind != CONEF_Q_LOWRANK;
    if (ctx->c.kind == CONEF_C_COUNTSKETCH && !all_csk)
        CK_CUDA(cudaMemsetAsync(V.state_new, 0, (size_t)ctx->plan.state_stride * ctx->n_workers, s));
    int rc = body();
    if (rc == CONEF_OK && sk)
        ctx->sketch_cur ^= 1;
    return rc;
}

// ---- fused passes 2 + 3 (conef_fused.cu)
// The task list for the device the context lives on: units in table order, workers of a tensor
// next to one another (they share P_hat); the Q_i tiles of a unit, and its residual tiles once
// about one and a half tasks per resident CTA have been listed after them (so that the Q_i tiles
// are done when the first residual tile looks, and the unit's data is still in L2).  Scratch for
// the partial sums cycles through a fixed region; a unit records which earlier units' scratch it
// overwrites and waits for them.  Returns CONEF_ERR_UNSUPPORTED where a unit's scratch does not
// fit (tiles far shorter than the default on a large tensor).
int fused_schedule(conef_ctx *ctx)
{
    const Plan &P = ctx->plan;
    const int64_t lag = (int64_t)ctx->fcfg.ctas;
    ctx->fu_units.clear();
    ctx->fu_groups.clear();
    int64_t cursor = 0, ctr = 64;   // word 0 of the counters is the task counter
    std::vector<int64_t> tiles;
    struct Live { int64_t lo, hi; int unit; };
    std::vector<Live> live;
    for (int l = 0; l < ctx->n_layers; ++l) {
        const LayerDesc &L = P.layers[l];
        if (!(L.compressed && L.f_fused))
            continue;
        const int64_t TP = fused_tile_periods(ctx->q.rank, L.f_subs, ctx->fused_tile_periods);
        const int64_t ncg = L.f_lcm / 256, ntp = ceil_div(L.f_niter, TP);
        const int64_t size = ncg * (ntp + 1) * 256 * ctx->q.rank;
        if (size > P.fu_scratch_floats)
            return CONEF_ERR_UNSUPPORTED;
        for (int w = 0; w < ctx->n_workers; ++w) {
            FusedUnit U{};
            U.layer = l;
            U.worker = w;
            U.ntp = (int32_t)ntp;
            U.tp = (int32_t)TP;
            if (cursor + size > P.fu_scratch_floats)
                cursor = 0;
            U.scratch_off = cursor;
            U.guard_lo = 0;
            U.guard_hi = -1;
            std::vector<Live> keep;
            for (const Live &v : live) {
                if (v.lo < cursor + size && cursor < v.hi) {
                    if (U.guard_hi < U.guard_lo)
                        U.guard_lo = U.guard_hi = v.unit;
                    U.guard_lo = std::min(U.guard_lo, v.unit);
                    U.guard_hi = std::max(U.guard_hi, v.unit);
                } else {
                    keep.push_back(v);
                }
            }
            live.swap(keep);
            live.push_back({cursor, cursor + size, (int)ctx->fu_units.size()});
            cursor += size;
            U.ctr_off = (int32_t)ctr;
            U.flag_off = (int32_t)(ctr + ncg + 1);
            ctr += ncg + 2;
            ctx->fu_units.push_back(U);
            tiles.push_back(ncg * ntp);
        }
    }
    // Two streams of tiles, both in unit order: the Q_i tiles (A) and the residual tiles (B).  The
    // list takes runs of kFuRun tiles from A; once `lag` A tiles have been listed after the last
    // A tile of the unit at the head of B (so that they are done when a CTA gets there), runs of
    // B alternate with them: the residual tiles of a unit then run next to the Q_i tiles of the
    // unit that follows it, and two units' data share L2.
    const size_t nu = ctx->fu_units.size();
    std::vector<int64_t> a_end(nu, 0);   // A tiles listed when the unit's last one was
    int64_t pos = 0, a_listed = 0;
    size_t ua = 0, ub = 0;
    int64_t ta = 0, tb2 = 0;   // next tile of the unit at the head of A / B
    auto emit = [&](size_t unit, int phase, int64_t tile0, int64_t count) {
        ctx->fu_groups.push_back(FusedGroup{(int32_t)(unit | (phase ? 0x80000000u : 0u)), (int32_t)pos, (int32_t)tile0, 0});
        pos += count;
    };
    while (ua < nu || ub < nu) {
        if (ua < nu) {
            const int64_t c = std::min<int64_t>(kFuRun, tiles[ua] - ta);
            emit(ua, 0, ta, c);
            ta += c;
            a_listed += c;
            if (ta == tiles[ua]) {
                a_end[ua] = a_listed;
                ++ua;
                ta = 0;
            }
        }
        if (ub < ua && (ua == nu || a_listed >= a_end[ub] + lag)) {
            const int64_t c = std::min<int64_t>(kFuRun, tiles[ub] - tb2);
            emit(ub, 1, tb2, c);
            tb2 += c;
            if (tb2 == tiles[ub]) {
                ++ub;
                tb2 = 0;
            }
        }
    }
    if (pos >= (1ll << 31) || ctr > P.fu_ctr_words || (pos + 31) / 32 > P.fu_hint_words ||
        (int64_t)ctx->fu_groups.size() > P.fu_group_cap)
        return CONEF_ERR_UNSUPPORTED;
    ctx->fu_hint.assign((size_t)((pos + 31) / 32), 0u);
    for (size_t g = 0, b = 0; b < ctx->fu_hint.size(); ++b) {
        while (g + 1 < ctx->fu_groups.size() && (int64_t)ctx->fu_groups[g + 1].first <= (int64_t)b * 32)
            ++g;
        ctx->fu_hint[b] = (uint32_t)g;
    }
    ctx->fu_tasks = (int)pos;
    ctx->fused_dirty = true;
    return CONEF_OK;
}

int fused_upload(conef_ctx *ctx, cudaStream_t s)
{
    const Plan &P = ctx->plan;
    CK_CUDA(cudaMemcpyAsync(ctx->ws + P.off_fu_units, ctx->fu_units.data(), ctx->fu_units.size() * sizeof(FusedUnit),
                            cudaMemcpyHostToDevice, s));
    CK_CUDA(cudaMemcpyAsync(ctx->ws + P.off_fu_groups, ctx->fu_groups.data(), ctx->fu_groups.size() * sizeof(FusedGroup),
                            cudaMemcpyHostToDevice, s));
    CK_CUDA(cudaMemcpyAsync(ctx->ws + P.off_fu_hint, ctx->fu_hint.data(), ctx->fu_hint.size() * 4, cudaMemcpyHostToDevice, s));
    ctx->fused_dirty = false;
    return CONEF_OK;
}

// configuration of the fused kernel on the current device; leaves fused_ready false (the separate
// passes run) where the device cannot co-schedule the grid
int fused_setup(conef_ctx *ctx)
{
    ctx->fused_ready = false;
    if (!ctx->plan.any_fused)
        return CONEF_OK;
    int dev = 0, sms = 0, coop = 0;
    CK_CUDA(cudaGetDevice(&dev));
    CK_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CK_CUDA(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
    if (!coop || sms <= 0)
        return CONEF_OK;
    const cudaError_t e = fused_config(ctx->c.kind, ctx->q.rank, ctx->c.scale_dtype == CONEF_SCALE_FP16,
                                       ctx->fused_ctas_per_sm, sms, &ctx->fcfg);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return CONEF_OK;
    }
    const int rc = fused_schedule(ctx);
    if (rc != CONEF_OK)
        return rc;
    ctx->fused_ready = true;
    return CONEF_OK;
}

// passes 2 + 3 of the tensors the fused kernel takes.  own_q: the kernel's Q_i goes to the second
// buffer and the residual is formed with the Q_i found in the message buffer.
int launch_fused(conef_ctx *ctx, const DevView &V, cudaStream_t s, bool own_q)
{
    const Plan &P = ctx->plan;
    if (ctx->fu_tasks == 0)
        return CONEF_OK;
    if (ctx->fused_dirty) {
        int rc = fused_upload(ctx, s);
        if (rc != CONEF_OK)
            return rc;
    }
    CK_CUDA(cudaMemsetAsync(ctx->ws + P.off_fu_ctr, 0, (size_t)P.fu_ctr_words * 4, s));
    FusedParams A;
    A.V = V;
    A.units = (const FusedUnit *)(ctx->ws + P.off_fu_units);
    A.groups = (const FusedGroup *)(ctx->ws + P.off_fu_groups);
    A.hint = (const uint32_t *)(ctx->ws + P.off_fu_hint);
    A.n_groups = (int32_t)ctx->fu_groups.size();
    A.n_tasks = ctx->fu_tasks;
    A.ring = ctx->fcfg.ring;
    A.pad = 0;
    A.next_task = (uint32_t *)(ctx->ws + P.off_fu_ctr);
    A.ctr = (uint32_t *)(ctx->ws + P.off_fu_ctr);
    A.scratch = (float *)(ctx->ws + P.off_fu_scratch);
    A.q_out = own_q ? (float *)(ctx->ws + P.off_fu_q) : V.msgq;
    A.q_out_stride = V.msgq_stride;
    A.q_res = V.msgq;
    A.q_res_stride = V.msgq_stride;
    CK_CUDA(fused_launch(ctx->c.kind, ctx->q.rank, V.scale_half, ctx->fcfg.ctas_per_sm, A,
                         std::min(ctx->fcfg.ctas, ctx->fu_tasks), ctx->fcfg.smem, s));
    LAUNCH_CHECK(ctx);
    return CONEF_OK;
}

int launch_randk_select(conef_ctx *ctx, const DevView &V, cudaStream_t s)
{
    const int nh = tiles_of(ctx, T_HIST), nc = tiles_of(ctx, T_GS);
    if (nh == 0)
        return CONEF_OK;
    CK_CUDA(cudaMemsetAsync(V.sel, 0, (size_t)ctx->plan.sel_words * 4, s));
    k_rk_hist<0><<<nh, 256, 0, s>>>(V); LAUNCH_CHECK(ctx);
    k_rk_pick<0><<<nc, 1024, 0, s>>>(V); LAUNCH_CHECK(ctx);
    k_rk_hist<1><<<nh, 256, 0, s>>>(V); LAUNCH_CHECK(ctx);
    k_rk_pick<1><<<nc, 1024, 0, s>>>(V); LAUNCH_CHECK(ctx);
    k_rk_hist<2><<<nh, 256, 0, s>>>(V); LAUNCH_CHECK(ctx);
    k_rk_pick<2><<<nc, 1024, 0, s>>>(V); LAUNCH_CHECK(ctx);
    k_rk_hist<3><<<nh, 256, 0, s>>>(V); LAUNCH_CHECK(ctx);
    k_rk_pick<3><<<nc, 1024, 0, s>>>(V); LAUNCH_CHECK(ctx);
    k_rk_count<<<nh, 256, 0, s>>>(V); LAUNCH_CHECK(ctx);
    k_rk_scan<<<nc, 1024, 0, s>>>(V); LAUNCH_CHECK(ctx);
    return CONEF_OK;
}

}  // namespace

extern "C" {

int conef_workspace_bytes(const conef_tensor *tensors, int n_tensors, int n_workers,
                          const conef_q_cfg *q, const conef_c_cfg *c, size_t *out_bytes)
{
    if (!out_bytes)
        return CONEF_ERR_INVALID_ARG;
    Plan P;
    int rc = make_plan(tensors, n_tensors, n_workers, q, c, P);
    if (rc != CONEF_OK)
        return rc;
    *out_bytes = P.total;
    return CONEF_OK;
}

int conef_init(conef_ctx **out, const conef_tensor *tensors, int n_tensors, int n_workers,
               const conef_q_cfg *q, const conef_c_cfg *c, float lr, void *workspace,
               size_t workspace_bytes, conef_stream stream)
{
    if (!out)
        return CONEF_ERR_INVALID_ARG;
    *out = nullptr;
    conef_ctx *ctx = new (std::nothrow) conef_ctx();
    if (!ctx)
        return CONEF_ERR_INVALID_ARG;
    int rc = make_plan(tensors, n_tensors, n_workers, q, c, ctx->plan);
    if (rc == CONEF_OK && (!workspace || ((uintptr_t)workspace % kAlign) != 0))
        rc = CONEF_ERR_INVALID_ARG;
    if (rc == CONEF_OK && workspace_bytes < ctx->plan.total)
        rc = CONEF_ERR_WORKSPACE_TOO_SMALL;
    if (rc == CONEF_OK && q->kind == CONEF_Q_LOWRANK && !q->q_init && ctx->plan.msg_elems[CONEF_MSG_Q] > 0)
        rc = CONEF_ERR_INVALID_ARG;
    if (rc == CONEF_OK && !(lr == lr))
        rc = CONEF_ERR_INVALID_ARG;
    if (rc != CONEF_OK) {
        delete ctx;
        return rc;
    }
    ctx->q = *q;
    ctx->c = *c;
    ctx->n_layers = n_tensors;
    ctx->n_workers = n_workers;
    ctx->ws = (uint8_t *)workspace;
    fill_view(ctx);
    ctx->view.lr = lr;
    const Plan &P = ctx->plan;
    cudaStream_t s = (cudaStream_t)stream;
    auto fail = [&](cudaError_t e, const char *what) {
        g_last_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
        delete ctx;
        return CONEF_ERR_CUDA;
    };
    cudaError_t e;
    // everything past the tables starts at zero: status, selection scratch,
    // factors, error state (e_0 = 0, Alg. 2 line 1), messages
    if ((e = cudaMemsetAsync(ctx->ws + P.off_status, 0, P.total - P.off_status, s)) != cudaSuccess)
        return fail(e, "cudaMemsetAsync(workspace)");
    if ((e = cudaMemcpyAsync(ctx->ws + P.off_layers, P.layers.data(), sizeof(LayerDesc) * n_tensors,
                             cudaMemcpyHostToDevice, s)) != cudaSuccess)
        return fail(e, "cudaMemcpyAsync(layer table)");
    std::vector<int32_t> pf;
    for (auto &v : P.pfx)
        pf.insert(pf.end(), v.begin(), v.end());
    if ((e = cudaMemcpyAsync(ctx->ws + P.off_pfx, pf.data(), pf.size() * 4, cudaMemcpyHostToDevice, s)) != cudaSuccess)
        return fail(e, "cudaMemcpyAsync(prefix tables)");
    std::vector<uint32_t> rs;
    if (c->kind == CONEF_C_ROWSKETCH && P.rs_words > 0) {
        // buckets and signs of the matrix rows (Sec. 4.2.2): h_i(a), s_i(a) from the stream
        // (seed, tensor, i) evaluated at the row index; they do not depend on the step
        rs.assign((size_t)P.rs_words, 0u);
        for (int l = 0; l < n_tensors; ++l) {
            const LayerDesc &L = P.layers[l];
            if (!L.compressed)
                continue;
            for (int i = 0; i < c->cs_rows; ++i) {
                uint32_t *info = rs.data() + L.rs_info_off + (size_t)i * L.rows;
                uint32_t *ptr = rs.data() + L.rs_ptr_off + (size_t)i * (L.w + 1);
                uint32_t *row = rs.data() + L.rs_row_off + (size_t)i * L.rows;
                const uint64_t st = stream_key(c->seed, (uint64_t)l, (uint64_t)i);
                for (int64_t a = 0; a < L.rows; ++a) {
                    const uint64_t u = h64(st, (uint64_t)a);
                    const uint32_t h = (uint32_t)(((u >> 32) * (uint64_t)L.w) >> 32);
                    info[a] = h | ((uint32_t)(u & 1) << 31);
                    ptr[h + 1]++;
                }
                for (int64_t h = 0; h < L.w; ++h)
                    ptr[h + 1] += ptr[h];
                std::vector<uint32_t> fill(ptr, ptr + L.w);
                for (int64_t a = 0; a < L.rows; ++a)   // ascending a within every bucket
                    row[fill[info[a] & 0x7FFFFFFFu]++] = (uint32_t)a | (info[a] & 0x80000000u);
            }
        }
        if ((e = cudaMemcpyAsync(ctx->ws + P.off_rs, rs.data(), rs.size() * 4, cudaMemcpyHostToDevice, s)) != cudaSuccess)
            return fail(e, "cudaMemcpyAsync(row-sketch tables)");
    }
    // pageable sources are staged before the call returns, but be explicit
    if ((e = cudaStreamSynchronize(s)) != cudaSuccess)
        return fail(e, "cudaStreamSynchronize(init)");
    if (q->kind == CONEF_Q_LOWRANK) {
        // side streams: one per further CTA-size class of the tuned passes, at least three for the
        // Gram-Schmidt launches by tensor height
        const size_t want = std::max<size_t>(P.fast_threads.size(), 4);
        if ((e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming)) != cudaSuccess)
            return fail(e, "cudaEventCreateWithFlags");
        for (size_t k = 1; k < want && k < (size_t)kMaxFastClasses; ++k) {
            cudaStream_t st = nullptr;
            cudaEvent_t ev = nullptr;
            if ((e = cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking)) != cudaSuccess)
                return fail(e, "cudaStreamCreateWithFlags");
            if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) {
                cudaStreamDestroy(st);
                return fail(e, "cudaEventCreateWithFlags");
            }
            ctx->aux[ctx->n_aux] = st;
            ctx->ev_join[ctx->n_aux] = ev;
            ++ctx->n_aux;
        }
    }
    {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
            ctx->sm_count = sms;
    }
    if (q->kind == CONEF_Q_LOWRANK) {
        int rc2 = fused_setup(ctx);
        if (rc2 != CONEF_OK) {
            delete ctx;
            return rc2;
        }
    }
    if (q->kind == CONEF_Q_LOWRANK && P.msg_elems[CONEF_MSG_Q] > 0) {
        ctx->q.q_init = nullptr;
        if ((e = cudaMemcpyAsync(ctx->ws + P.off_qprev, q->q_init, (size_t)P.msg_elems[CONEF_MSG_Q] * 4,
                                 cudaMemcpyDeviceToDevice, s)) != cudaSuccess)
            return fail(e, "cudaMemcpyAsync(q_init)");
    }
    *out = ctx;
    return CONEF_OK;
}

int conef_step(conef_ctx *ctx, int64_t step, const float *const *grads, int phase,
               conef_stream stream)
{
    if (!ctx || !grads || step < 0)
        return CONEF_ERR_INVALID_ARG;
    for (int i = 0; i < ctx->n_workers; ++i)
        if (!grads[i] || ((uintptr_t)grads[i] & 3))
            return CONEF_ERR_INVALID_ARG;
    const bool lowrank = ctx->q.kind == CONEF_Q_LOWRANK;
    if (!lowrank) {
        if (phase != 0)
            return CONEF_ERR_BAD_PHASE;
        if (step <= ctx->last_step)
            return CONEF_ERR_BAD_PHASE;
    } else {
        if (phase < 0 || phase > 4)
            return CONEF_ERR_BAD_PHASE;
        if (phase == 0 && (ctx->expect != 0 || step <= ctx->last_step))
            return CONEF_ERR_BAD_PHASE;
        if ((phase == 1 || phase == 2) && (ctx->expect != 2 || step != ctx->last_step))
            return CONEF_ERR_BAD_PHASE;
        if ((phase == 3 || phase == 4) && (ctx->expect != 3 || step != ctx->last_step))
            return CONEF_ERR_BAD_PHASE;
    }
    cudaStream_t s = (cudaStream_t)stream;
    DevView V = current_view(ctx);
    V.step = step;
    bool aligned32 = true;   // the tuned kernels use 256-bit loads
    for (int i = 0; i < ctx->n_workers; ++i) {
        V.grads[i] = grads[i];
        aligned32 = aligned32 && (((uintptr_t)grads[i] & 31) == 0);
    }
    V.rs_vec_ok = 1;
    for (int i = 0; i < ctx->n_workers; ++i)
        if ((uintptr_t)grads[i] & 15)
            V.rs_vec_ok = 0;
    // tuned kernels for this call: the int8/int4 streaming passes, or the bucket-major passes on a row sketch
    const bool rs12 = ctx->fast && V.rs_vec_ok && ctx->plan.any_rs12;
    const bool fast = (ctx->fast && aligned32 && ctx->plan.any_fast) || rs12;
    int rc = CONEF_OK;

    if (phase == 0 && tiles_of(ctx, T_PASS) > 0) {
        dim3 grid(tiles_of(ctx, T_PASS), ctx->n_workers);
        k_passthrough<<<grid, 256, 0, s>>>(V);
        LAUNCH_CHECK(ctx);
    }
    // single-phase compressors: the tuned fused step where a tensor allows it, the generic kernel elsewhere
    const bool fv = ctx->fast && V.rs_vec_ok && ctx->plan.any_fv;
    const bool csk = ctx->fast && ctx->plan.any_csk;
    auto flat_step = [&](auto qk) -> int {
        constexpr int QK = decltype(qk)::value;
        if (!fv && !csk)
            return launch_flat<QK>(ctx, V, s);
        if (fv) {
            CK_CUDA(flatvec_launch(QK, ctx->c.kind, ctx->c.kind == CONEF_C_STOCHQUANT ? 0 : V.scale_half, V,
                                   table_ptr(ctx, T_FV), tiles_of(ctx, T_FV), s));
            LAUNCH_CHECK(ctx);
        }
        if (csk) {
            CK_CUDA(chunksketch_launch(QK, ctx->c.cs_rows, V, table_ptr(ctx, T_CSK), tiles_of(ctx, T_CSK),
                                       ctx->plan.csk_smem, s));
            LAUNCH_CHECK(ctx);
        }
        return launch_flat<QK>(ctx, V, s, T_NOFV);
    };
    // iConEF-v2 with random-k: the index sets of the draw that stored e~ (A) and of this step's
    // second draw (B), by the same selection kernels on the stream of step + 2^62
    auto second_draws = [&]() -> int {
        if (ctx->c.iconef != 2 || ctx->q.kind != CONEF_Q_RANDK)
            return CONEF_OK;
        for (int x = V.ev_valid ? 0 : 1; x < 2; ++x) {
            const int set = x == 0 ? ctx->ev_cur : ctx->ev_cur ^ 1;
            const int64_t draw = x == 0 ? V.ev_step : step;
            if (ctx->draw_step[set] == draw)
                continue;   // last step's draw B is this step's draw A
            DevView D = V;
            D.step = draw + kSecondDraw;
            D.unitoff = x == 0 ? V.unitoffA : V.unitoffB;
            D.tileoff = x == 0 ? V.tileoffA : V.tileoffB;
            D.selbits = x == 0 ? V.selbitsA : V.selbitsB;
            ctx->draw_step[set] = -1;
            int rc2 = launch_randk_select(ctx, D, s);
            if (rc2 != CONEF_OK)
                return rc2;
            ctx->draw_step[set] = draw;
        }
        return CONEF_OK;
    };
    if (ctx->q.kind == CONEF_Q_IDENTITY) {
        rc = with_new_sketch(ctx, V, s, [&] { return flat_step(std::integral_constant<int, CONEF_Q_IDENTITY>()); });
    } else if (ctx->q.kind == CONEF_Q_RANDBLOCK) {
        rc = with_new_sketch(ctx, V, s, [&] { return flat_step(std::integral_constant<int, CONEF_Q_RANDBLOCK>()); });
    } else if (ctx->q.kind == CONEF_Q_RANDK) {
        rc = launch_randk_select(ctx, V, s);
        if (rc == CONEF_OK)
            rc = second_draws();
        if (rc == CONEF_OK)
            rc = with_new_sketch(ctx, V, s, [&] { return flat_step(std::integral_constant<int, CONEF_Q_RANDK>()); });
    } else {
        // tensors the tuned kernels take go to them, the rest to the generic kernels
        V.fast_on = fast ? 1 : 0;
        const bool slow_left = !fast || ctx->plan.any_slow;
        // passes 2 and 3 in one kernel where the call asks for both (phase 1), or for pass 3 by that
        // kernel (phase 4: its own Q_i goes to a second buffer)
        const bool fused = fast && !rs12 && ctx->fused && ctx->fused_ready && ctx->plan.any_fused && (phase == 1 || phase == 4);
        if (rc == CONEF_OK && fused)
            rc = launch_fused(ctx, V, s, phase == 4);
        auto launch_rs12 = [&](int pass) -> int {
            const int n = tiles_of(ctx, T_RS_P12);
            if (n == 0)
                return CONEF_OK;
            dim3 grid(n, ctx->n_workers);
            if (pass == 1) {
                k_rs_pass12<1><<<grid, kRsThreads, 0, s>>>(V, table_ptr(ctx, T_RS_P12));
                LAUNCH_CHECK(ctx);
                dim3 gridc(tiles_of(ctx, T_RS_P1C), ctx->n_workers);
                k_rs_p1_combine<<<gridc, 256, 0, s>>>(V, table_ptr(ctx, T_RS_P1C));
            } else {
                k_rs_pass12<2><<<grid, kRsThreads, 0, s>>>(V, table_ptr(ctx, T_RS_P12));
            }
            LAUNCH_CHECK(ctx);
            return CONEF_OK;
        };
        if (phase == 0) {
            if (rs12)
                rc = launch_rs12(1);
            else if (fast)
                rc = launch_fast(ctx, 1, V, s);
            if (rc == CONEF_OK && slow_left)
                rc = launch_pass1(ctx, V, s, fast ? T_SLOW_P1 : T_P1);
        }
        if (rc == CONEF_OK && (phase == 1 || phase == 2)) {
            if (rs12)
                rc = launch_rs12(2);
            else if (fast)
                rc = launch_fast(ctx, 2, V, s, fused);
            if (rc == CONEF_OK && slow_left)
                rc = launch_pass2(ctx, V, s, fast ? T_SLOW_P2 : T_P2);
            if (rc == CONEF_OK)
                rc = launch_pass2_reduce(ctx, V, s, fused);
        }
        if (rc == CONEF_OK && (phase == 1 || phase == 3 || phase == 4)) {
            rc = with_new_sketch(ctx, V, s, [&] {
                if (ctx->c.kind == CONEF_C_ROWSKETCH)
                    return launch_rowsketch<CONEF_Q_LOWRANK>(ctx, V, s);
                int r2 = fast ? launch_fast(ctx, 3, V, s, fused) : CONEF_OK;
                if (r2 == CONEF_OK && slow_left)
                    r2 = launch_flat<CONEF_Q_LOWRANK>(ctx, V, s, fast ? T_SLOW_FLAT : T_FLAT);
                return r2;
            });
        }
    }
    if (rc != CONEF_OK) {
        if (rc == CONEF_ERR_CUDA && g_last_cuda_error.empty())
            g_last_cuda_error = cudaGetErrorString(cudaGetLastError());
        return rc;
    }
    ctx->last_step = step;
    ctx->stepped = true;
    if (ctx->c.iconef == 2) {   // the values just written are e~ from now on
        ctx->ev_cur ^= 1;
        ctx->ev_step = step;
    }
    if (lowrank)
        ctx->expect = phase == 0 ? 1 : (phase == 2 ? 3 : 4);   // (phases 1, 3 and 4 complete the step)
    return CONEF_OK;
}

int conef_reduce_messages(conef_ctx *ctx, int which, float *out_sum, conef_stream stream)
{
    if (!ctx || which < CONEF_MSG_VALUES || which > CONEF_MSG_DENSE1D)
        return CONEF_ERR_INVALID_ARG;
    if (!ctx->stepped)
        return CONEF_ERR_BAD_PHASE;
    const bool lowrank = ctx->q.kind == CONEF_Q_LOWRANK;
    cudaStream_t s = (cudaStream_t)stream;
    const Plan &P = ctx->plan;
    const DevView V = current_view(ctx);
    const int64_t len = P.msg_elems[which];
    auto plain = [&](const float *base, int64_t stride, float *mean_out) -> int {
        if (len == 0)
            return CONEF_OK;
        int64_t blocks = ceil_div(len, 256);
        if (blocks > (int64_t)ctx->sm_count * 16)
            blocks = (int64_t)ctx->sm_count * 16;
        k_reduce_workers<<<(int)blocks, 256, 0, s>>>(base, stride, ctx->n_workers, len, out_sum,
                                                     mean_out, V.n_workers_f);
        LAUNCH_CHECK(ctx);
        return CONEF_OK;
    };
    switch (which) {
    case CONEF_MSG_VALUES:
        if (lowrank)
            return CONEF_ERR_INVALID_ARG;
        if (!out_sum && len > 0)
            return CONEF_ERR_INVALID_ARG;
        return plain(V.msgv, V.msgv_stride, nullptr);
    case CONEF_MSG_DENSE1D:
        if (!out_sum && len > 0)
            return CONEF_ERR_INVALID_ARG;
        return plain(V.msg1d, V.msg1d_stride, nullptr);
    case CONEF_MSG_P: {
        if (!lowrank)
            return CONEF_ERR_INVALID_ARG;
        if (ctx->expect != 1)
            return CONEF_ERR_BAD_PHASE;
        if (ctx->fast) {
            // by height: one CTA, a cluster of 8 CTAs, a cluster of 16, and the generic kernel beyond
            // the launches work on different tensors: all but the first run on side streams
            const int tabs[3] = {T_GS_ONE, T_GS_CLUSTER, T_GS_CLUSTER16};
            const int csz[3] = {1, 8, 16};
            int used = 0, launched = 0;
            if (ctx->n_aux > 0)
                CK_CUDA(cudaEventRecord(ctx->ev_fork, s));
            auto pick = [&]() -> cudaStream_t {
                if (launched++ == 0 || used >= ctx->n_aux)
                    return s;
                cudaStream_t sk = ctx->aux[used];
                cudaStreamWaitEvent(sk, ctx->ev_fork, 0);
                return sk;
            };
            auto done = [&](cudaStream_t sk) {
                if (sk != s) {
                    cudaEventRecord(ctx->ev_join[used], sk);
                    ++used;
                }
            };
            for (int k = 0; k < 3; ++k) {
                const int n = tiles_of(ctx, tabs[k]);
                if (n == 0)
                    continue;
                cudaStream_t sk = pick();
                if (ctx->q.rank <= 4)
                    CK_CUDA(gs_launch<4>(V, table_ptr(ctx, tabs[k]), n, csz[k], out_sum, sk));
                else
                    CK_CUDA(gs_launch<8>(V, table_ptr(ctx, tabs[k]), n, csz[k], out_sum, sk));
                LAUNCH_CHECK(ctx);
                done(sk);
            }
            if (tiles_of(ctx, T_GS_REST) > 0) {
                DevView V2 = V;
                V2.pfx_gs = table_ptr(ctx, T_GS_REST);
                cudaStream_t sk = pick();
                k_gram_schmidt<<<tiles_of(ctx, T_GS_REST), 1024, 0, sk>>>(V2, out_sum);
                LAUNCH_CHECK(ctx);
                done(sk);
            }
            for (int k = 0; k < used; ++k)
                CK_CUDA(cudaStreamWaitEvent(s, ctx->ev_join[k], 0));
        } else if (tiles_of(ctx, T_GS) > 0) {
            k_gram_schmidt<<<tiles_of(ctx, T_GS), 1024, 0, s>>>(V, out_sum);
            LAUNCH_CHECK(ctx);
        }
        ctx->expect = 2;
        return CONEF_OK;
    }
    default: {
        if (!lowrank)
            return CONEF_ERR_INVALID_ARG;
        if (ctx->expect != 4)
            return CONEF_ERR_BAD_PHASE;
        int rc = plain(V.msgq, V.msgq_stride, V.qprev);
        if (rc == CONEF_OK)
            ctx->expect = 0;
        return rc;
    }
    }
}

int conef_apply_update(conef_ctx *ctx, float *x, const float *sum_values, const float *sum_dense1d,
                       conef_stream stream)
{
    if (!ctx || !x)
        return CONEF_ERR_INVALID_ARG;
    if (!ctx->stepped)
        return CONEF_ERR_BAD_PHASE;
    const Plan &P = ctx->plan;
    const bool lowrank = ctx->q.kind == CONEF_Q_LOWRANK;
    if (lowrank && ctx->expect != 0)
        return CONEF_ERR_BAD_PHASE;   // Qmean exists only after reduce(MSG_Q)
    if ((!lowrank && P.msg_elems[CONEF_MSG_VALUES] > 0 && !sum_values) ||
        (P.msg_elems[CONEF_MSG_DENSE1D] > 0 && !sum_dense1d))
        return CONEF_ERR_INVALID_ARG;
    const int n = tiles_of(ctx, T_APPLY);
    if (n == 0)
        return CONEF_OK;
    const DevView V = current_view(ctx);
    k_apply<<<n, 256, 0, (cudaStream_t)stream>>>(V, table_ptr(ctx, T_APPLY), x, sum_values, sum_dense1d);
    LAUNCH_CHECK(ctx);
    return CONEF_OK;
}

int conef_error_reset(conef_ctx *ctx, conef_stream stream)
{
    if (!ctx)
        return CONEF_ERR_INVALID_ARG;
    const int k = ctx->c.kind;
    if (k != CONEF_C_IDENTITY && k != CONEF_C_COUNTSKETCH && k != CONEF_C_ROWSKETCH)
        return CONEF_ERR_UNSUPPORTED;
    if (ctx->c.iconef == 2)   // e~ lives outside the state that is averaged here
        return CONEF_ERR_UNSUPPORTED;
    if (ctx->q.kind == CONEF_Q_LOWRANK && ctx->expect != 0)
        return CONEF_ERR_BAD_PHASE;
    // every region of a linear state has one element type (padding is zero): fp32, or binary16 for a half row sketch
    const bool half = k == CONEF_C_ROWSKETCH && ctx->c.scale_dtype == CONEF_SCALE_FP16;
    const int64_t words = ctx->plan.state_stride / (half ? 2 : 4);
    if (words == 0)
        return CONEF_OK;
    const DevView V = current_view(ctx);
    int64_t blocks = ceil_div(words, 256);
    if (blocks > (int64_t)ctx->sm_count * 16)
        blocks = (int64_t)ctx->sm_count * 16;
    if (half)
        k_error_reset_half<<<(int)blocks, 256, 0, (cudaStream_t)stream>>>(V.state, V.state_stride, ctx->n_workers,
                                                                          V.n_workers_f, words);
    else
        k_error_reset<<<(int)blocks, 256, 0, (cudaStream_t)stream>>>(V.state, V.state_stride, ctx->n_workers, V.n_workers_f, words);
    LAUNCH_CHECK(ctx);
    return CONEF_OK;
}

int conef_decompress_error(conef_ctx *ctx, int worker, float *out, conef_stream stream)
{
    if (!ctx || worker < 0 || worker >= ctx->n_workers || (!out && ctx->plan.err_elems > 0))
        return CONEF_ERR_INVALID_ARG;
    const int n = tiles_of(ctx, T_FLAT);
    if (n == 0)
        return CONEF_OK;
    cudaStream_t s = (cudaStream_t)stream;
    const DevView V = current_view(ctx);
    if (ctx->c.iconef == 2 && ctx->q.kind == CONEF_Q_RANDK && V.ev_valid && ctx->draw_step[ctx->ev_cur] != V.ev_step) {
        // the index set of the draw that stored e~
        DevView D = V;
        D.step = V.ev_step + kSecondDraw;
        D.unitoff = V.unitoffA;
        D.tileoff = V.tileoffA;
        D.selbits = V.selbitsA;
        ctx->draw_step[ctx->ev_cur] = -1;
        int rc = launch_randk_select(ctx, D, s);
        if (rc != CONEF_OK)
            return rc;
        ctx->draw_step[ctx->ev_cur] = V.ev_step;
    }
    switch (ctx->c.kind) {
    case CONEF_C_IDENTITY: k_decompress<CONEF_C_IDENTITY><<<n, 256, 0, s>>>(V, worker, out); break;
    case CONEF_C_INT8: k_decompress<CONEF_C_INT8><<<n, 256, 0, s>>>(V, worker, out); break;
    case CONEF_C_INT4: k_decompress<CONEF_C_INT4><<<n, 256, 0, s>>>(V, worker, out); break;
    case CONEF_C_ROWSKETCH: k_decompress<CONEF_C_ROWSKETCH><<<n, 256, 0, s>>>(V, worker, out); break;
    case CONEF_C_STOCHQUANT: k_decompress<CONEF_C_STOCHQUANT><<<n, 256, 0, s>>>(V, worker, out); break;
    default: k_decompress<CONEF_C_COUNTSKETCH><<<n, 256, 0, s>>>(V, worker, out); break;
    }
    LAUNCH_CHECK(ctx);
    return CONEF_OK;
}

void conef_destroy(conef_ctx *ctx) { delete ctx; }

int64_t conef_message_elems(const conef_ctx *ctx, int which)
{
    if (!ctx || which < 0 || which > 3)
        return -1;
    return ctx->plan.msg_elems[which];
}
int64_t conef_error_elems(const conef_ctx *ctx) { return ctx ? ctx->plan.err_elems : -1; }
int64_t conef_state_bytes_per_worker(const conef_ctx *ctx)
{
    if (!ctx)
        return -1;
    int64_t b = 0;
    for (const LayerDesc &L : ctx->plan.layers)
        if (L.compressed)
            b += (L.a_bytes + L.b_bytes) * (ctx->c.iconef == 1 ? 2 : 1) + (ctx->c.iconef == 2 ? L.k * 4 : 0);
    return b;
}

int conef_get_message(const conef_ctx *ctx, int which, int worker, float **ptr)
{
    if (!ctx || !ptr || which < 0 || which > 3 || worker < 0 || worker >= ctx->n_workers)
        return CONEF_ERR_INVALID_ARG;
    const DevView &V = ctx->view;
    float *base[4] = {V.msgv, V.msgp, V.msgq, V.msg1d};
    int64_t stride[4] = {V.msgv_stride, V.msgp_stride, V.msgq_stride, V.msg1d_stride};
    *ptr = base[which] + worker * stride[which];
    return CONEF_OK;
}

int conef_get_state(const conef_ctx *ctx, int worker, int tensor, void **a, size_t *a_bytes,
                    void **b, size_t *b_bytes)
{
    if (!ctx || worker < 0 || worker >= ctx->n_workers || tensor < 0 || tensor >= ctx->n_layers)
        return CONEF_ERR_INVALID_ARG;
    const LayerDesc &L = ctx->plan.layers[tensor];
    if (!L.compressed)
        return CONEF_ERR_INVALID_ARG;
    const DevView V = current_view(ctx);
    uint8_t *st = V.state + worker * V.state_stride;
    if (a) *a = st + L.a_off;
    if (a_bytes) *a_bytes = (size_t)L.a_bytes;
    if (b) *b = L.b_bytes ? st + L.b_off : nullptr;
    if (b_bytes) *b_bytes = (size_t)L.b_bytes;
    return CONEF_OK;
}

int conef_get_state2(const conef_ctx *ctx, int worker, int tensor, void **a, size_t *a_bytes,
                     void **b, size_t *b_bytes)
{
    if (!ctx || worker < 0 || worker >= ctx->n_workers || tensor < 0 || tensor >= ctx->n_layers || !ctx->c.iconef)
        return CONEF_ERR_INVALID_ARG;
    const LayerDesc &L = ctx->plan.layers[tensor];
    if (!L.compressed)
        return CONEF_ERR_INVALID_ARG;
    const DevView V = current_view(ctx);
    if (ctx->c.iconef == 2) {   // e~: the k values of the second draw, in index order
        if (a) *a = V.ev_old + worker * V.msgv_stride + L.msgv_off;
        if (a_bytes) *a_bytes = (size_t)L.k * 4;
        if (b) *b = nullptr;
        if (b_bytes) *b_bytes = 0;
        return CONEF_OK;
    }
    uint8_t *st = V.state + worker * V.state_stride;
    if (a) *a = st + L.a2_off;
    if (a_bytes) *a_bytes = (size_t)L.a_bytes;
    if (b) *b = L.b_bytes ? st + L.b2_off : nullptr;
    if (b_bytes) *b_bytes = (size_t)L.b_bytes;
    return CONEF_OK;
}

int64_t conef_get_error_step(const conef_ctx *ctx) { return ctx && ctx->c.iconef == 2 ? ctx->ev_step : -1; }

int conef_set_error_step(conef_ctx *ctx, int64_t step)
{
    if (!ctx || ctx->c.iconef != 2 || step < -1 || step >= kSecondDraw)
        return CONEF_ERR_INVALID_ARG;
    ctx->ev_step = step;
    return CONEF_OK;
}

int conef_get_indices(const conef_ctx *ctx, int tensor, uint32_t **idx, int64_t *k)
{
    if (!ctx || tensor < 0 || tensor >= ctx->n_layers ||
        (ctx->q.kind != CONEF_Q_RANDK && ctx->q.kind != CONEF_Q_RANDBLOCK))
        return CONEF_ERR_INVALID_ARG;
    const LayerDesc &L = ctx->plan.layers[tensor];
    if (!L.compressed)
        return CONEF_ERR_INVALID_ARG;
    if (idx) *idx = ctx->view.idx + L.idx_off;
    if (k) *k = L.k;
    return CONEF_OK;
}

int conef_get_factors(const conef_ctx *ctx, int tensor, int worker, float **p_hat, float **q_prev,
                      float **q_i, float **p_i, int *rank)
{
    if (!ctx || tensor < 0 || tensor >= ctx->n_layers || worker < 0 || worker >= ctx->n_workers ||
        ctx->q.kind != CONEF_Q_LOWRANK)
        return CONEF_ERR_INVALID_ARG;
    const LayerDesc &L = ctx->plan.layers[tensor];
    if (!L.compressed)
        return CONEF_ERR_INVALID_ARG;
    const DevView &V = ctx->view;
    if (p_hat) *p_hat = V.phat + L.msgp_off;
    if (q_prev) *q_prev = V.qprev + L.msgq_off;
    if (q_i) *q_i = V.msgq + worker * V.msgq_stride + L.msgq_off;
    if (p_i) *p_i = V.msgp + worker * V.msgp_stride + L.msgp_off;
    if (rank) *rank = L.rank;
    return CONEF_OK;
}

int conef_last_status(conef_ctx *ctx, conef_stream stream, int *status)
{
    if (!ctx || !status)
        return CONEF_ERR_INVALID_ARG;
    int32_t v = 0;
    CK_CUDA(cudaMemcpyAsync(&v, ctx->view.status, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    CK_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    *status = v;
    return v ? CONEF_ERR_DEVICE_STATUS : CONEF_OK;
}

int64_t conef_launch_count(const conef_ctx *ctx) { return ctx ? ctx->launches : -1; }

int conef_set_total_workers(conef_ctx *ctx, int total)
{
    if (!ctx || total < ctx->n_workers)
        return CONEF_ERR_INVALID_ARG;
    ctx->view.n_workers_f = (float)total;
    return CONEF_OK;
}

int conef_set_fused(conef_ctx *ctx, int enable, int tile_periods, int ctas_per_sm)
{
    if (!ctx || tile_periods < 0 || tile_periods > (1 << 20) || !(ctas_per_sm == 0 || (ctas_per_sm >= 2 && ctas_per_sm <= 4)))
        return CONEF_ERR_INVALID_ARG;
    if (tile_periods == 0)
        tile_periods = kFuTilePeriods;
    if (ctas_per_sm == 0)
        ctas_per_sm = 2;
    if (ctx->q.kind == CONEF_Q_LOWRANK && (tile_periods != ctx->fused_tile_periods || ctas_per_sm != ctx->fused_ctas_per_sm)) {
        const int old_tp = ctx->fused_tile_periods, old_c = ctx->fused_ctas_per_sm;
        ctx->fused_tile_periods = tile_periods;
        ctx->fused_ctas_per_sm = ctas_per_sm;
        int rc = fused_setup(ctx);
        if (rc != CONEF_OK) {   // keep what worked
            ctx->fused_tile_periods = old_tp;
            ctx->fused_ctas_per_sm = old_c;
            fused_setup(ctx);
            return rc;
        }
    }
    ctx->fused = enable ? 1 : 0;
    return CONEF_OK;
}

int conef_fused_info(const conef_ctx *ctx, int *active, int *ctas, int *tile_periods, int *ring, int *tasks)
{
    if (!ctx)
        return CONEF_ERR_INVALID_ARG;
    const bool on = ctx->fast && ctx->fused && ctx->fused_ready;
    if (active) *active = on ? 1 : 0;
    if (ctas) *ctas = ctx->fused_ready ? ctx->fcfg.ctas : 0;
    if (tile_periods) *tile_periods = ctx->fused_tile_periods;
    if (ring) *ring = ctx->fused_ready ? ctx->fcfg.ring : 0;
    if (tasks) *tasks = ctx->fused_ready ? ctx->fu_tasks : 0;
    return CONEF_OK;
}

int conef_get_fused_q(const conef_ctx *ctx, int tensor, int worker, float **q_i)
{
    if (!ctx || !q_i || tensor < 0 || tensor >= ctx->n_layers || worker < 0 || worker >= ctx->n_workers ||
        ctx->q.kind != CONEF_Q_LOWRANK)
        return CONEF_ERR_INVALID_ARG;
    const LayerDesc &L = ctx->plan.layers[tensor];
    if (!L.compressed || !L.f_fused || !ctx->plan.any_fused)
        return CONEF_ERR_INVALID_ARG;
    *q_i = (float *)(ctx->ws + ctx->plan.off_fu_q) + worker * ctx->view.msgq_stride + L.msgq_off;
    return CONEF_OK;
}

int conef_set_fast_path(conef_ctx *ctx, int enable)
{
    if (!ctx)
        return CONEF_ERR_INVALID_ARG;
    ctx->fast = enable ? 1 : 0;
    return CONEF_OK;
}

const char *conef_error_string(int code)
{
    switch (code) {
    case CONEF_OK: return "ok";
    case CONEF_ERR_INVALID_ARG: return "invalid argument";
    case CONEF_ERR_BAD_PHASE: return "calls out of order or step index not increasing";
    case CONEF_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case CONEF_ERR_UNSUPPORTED: return "unsupported configuration";
    case CONEF_ERR_CUDA: return g_last_cuda_error.empty() ? "CUDA error" : g_last_cuda_error.c_str();
    case CONEF_ERR_DEVICE_STATUS: return "a kernel recorded a consistency error";
    case CONEF_ERR_TOO_LARGE: return "size exceeds the fixed scratch of the allocation-free entry point";
    default: return "unknown error";
    }
}

}  // extern "C"
