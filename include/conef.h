/*
 * libconef — one step of contractive error feedback (ConEF) on one GPU.
 *
 * C ABI.  Every pointer is either a HOST pointer or a DEVICE pointer and each
 * argument says which.  The library allocates no device memory: the caller
 * owns one device workspace whose size conef_workspace_bytes() reports, the
 * gradients and every output buffer.  All device work is enqueued on the
 * stream the caller passes (a cudaStream_t, typed void* here so that this
 * header needs no CUDA include); no call synchronises the device except
 * conef_last_status() and the copy helpers that say so.
 *
 * Every function returns CONEF_OK (0) or a negative CONEF_ERR_* code.  An
 * argument error is detected on the host before anything is launched and
 * leaves the context unchanged.
 *
 * What one step computes (Algorithm 2 of the paper, lines 5-9), for each of N
 * simulated workers i and each tensor of d = rows*cols elements:
 *     e   = decode(state_i)                       (line 5; e_0 = 0, line 1)
 *     p   = eta * g_i + e                          (line 5)
 *     D_i = Q(p)      -> all-reducible message     (line 6)
 *     r   = p - D_i                                (line 9)
 *     state_i = C(r)                               (line 9)
 * and conef_reduce_messages() forms the sum over workers of the messages
 * (line 7, "aggregate", before the division by N).  Algorithm 1 (EFSGD) is the
 * case C = identity.  Tensors with cols == 1 or compress == 0 pass through:
 * their message is eta*g and they keep no error state.
 */
#ifndef CONEF_H
#define CONEF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct conef_ctx conef_ctx;
typedef void *conef_stream; /* cudaStream_t */

enum {
    CONEF_OK = 0,
    CONEF_ERR_INVALID_ARG = -1,
    CONEF_ERR_BAD_PHASE = -2,           /* calls out of order, or a step index that does not advance */
    CONEF_ERR_WORKSPACE_TOO_SMALL = -3,
    CONEF_ERR_UNSUPPORTED = -4,
    CONEF_ERR_CUDA = -5,                /* a CUDA runtime call failed; see conef_error_string */
    CONEF_ERR_DEVICE_STATUS = -6,       /* a kernel recorded a consistency error (see conef_last_status) */
    CONEF_ERR_TOO_LARGE = -7            /* a size exceeds the fixed scratch of an allocation-free entry point */
};

/* gradient compressor Q (Alg. 2 line 6) */
enum { CONEF_Q_IDENTITY = 0, CONEF_Q_RANDK = 1, CONEF_Q_LOWRANK = 2, CONEF_Q_RANDBLOCK = 3 };
/* error compressor C (Alg. 2 line 9; Sec. 4.2) */
enum { CONEF_C_IDENTITY = 0, CONEF_C_INT8 = 1, CONEF_C_INT4 = 2, CONEF_C_COUNTSKETCH = 3,
       CONEF_C_ROWSKETCH = 4, CONEF_C_STOCHQUANT = 5 };
enum { CONEF_SCALE_FP32 = 0, CONEF_SCALE_FP16 = 1 };
/* message kinds */
enum { CONEF_MSG_VALUES = 0, CONEF_MSG_P = 1, CONEF_MSG_Q = 2, CONEF_MSG_DENSE1D = 3 };

#define CONEF_MAX_WORKERS 64
#define CONEF_MAX_RANK 8

/* One parameter tensor, viewed as a rows x cols row-major matrix (a conv
 * weight as out x (in*kh*kw)).  rows*cols must be below 2^32. */
typedef struct {
    int64_t rows;
    int64_t cols;
    int32_t compress; /* 0: pass through */
    int32_t reserved;
} conef_tensor;

/* Q.  random-k (Sec. 1; remark after Assumption 4; Sec. 5.3): keep
 * k = max(1, floor(d*k_num/k_den)) coordinates, the same on every worker and
 * new at every step, no d/k rescaling.  random-block-k (Sec. 5.3): the k kept
 * coordinates are one contiguous block whose start is uniform on [0, d-k],
 * drawn from the shared (seed, tensor, step) stream.  low-rank (Sec. 5.2): rank
 * r = min(rank, rows, cols), one power iteration, warm-started. */
typedef struct {
    int32_t kind;
    int32_t rank;        /* low-rank: 1..CONEF_MAX_RANK */
    int64_t k_num, k_den;
    const float *q_init; /* DEVICE, low-rank only: concatenation over the compressed tensors,
                            in table order, of the cols x r row-major warm starts Q_0.
                            Copied during conef_init; the caller may free it afterwards
                            (after the stream has run). */
    uint64_t seed;       /* random-k, random-block-k: the seed shared by all workers */
} conef_q_cfg;

/* C.  int8/int4 (Sec. 4.2.1): symmetric absmax quantisation of blocks of
 * `block` consecutive elements of the row-major flattening (block in
 * {32,64,128,256}; int4 needs block >= 64), round to nearest even, one fp32
 * or fp16 scale per block; int4 packs element 2q in the low nibble of byte q.
 * count sketch (Sec. 4.2.2): cs_rows (odd, <= 7) rows of
 * w = max(1, floor(d/cs_col_div)) fp32 buckets, median decode.
 * row sketch (Sec. 4.2.2, the tensor trick; the form Sec. 5.4 runs): the
 * matrix view is hashed one row at a time, sketch row i is a w x cols fp32
 * matrix with w = max(1, floor(rows/cs_col_div)), T_i[h_i(a)][:] += s_i(a) R[a][:];
 * state per worker and tensor: cs_rows x w x cols floats, row-major; with
 * scale_dtype = CONEF_SCALE_FP16 the sketch itself is kept in binary16 (each
 * updated entry clamped to +-65504 and rounded to nearest even).
 * beta (Alg. 4, partial error feedback, 0 <= beta < 1; 0 is Alg. 2):
 * p = eta g + (1-beta) e and the stored error is C(beta e + p - Delta); the
 * row sketch, being linear, is updated as T <- beta T + sketch(p - Delta)
 * without decoding.
 * iconef = 1 (Alg. 3, version 1; identity, int8, int4 with beta = 0 only): a
 * second state q of the same kind and size is kept, p = (eta g + e~) + q,
 * e~ <- C(r), q <- C(r - decode(e~)) with r = p - Delta; conef_get_state2
 * reads it, conef_decompress_error returns e~ + q.  The tuned low-rank
 * kernels are switched off.
 * iconef = 2 (Alg. 3, version 2; Q random-k or random-block-k, C identity,
 * int8 or int4, beta = 0): e~ <- Q(r) by a second application of Q in the same
 * step, which draws its index set from the stream of step t + 2^62 (the first
 * draw would return zeros: r vanishes there); e~ is kept as its k fp32 values
 * in index order (conef_get_state2), the index set is recomputed when needed.
 * The stored state is q <- C(r - e~), and r - e~ is exactly 0 where e~ keeps a
 * value.  Next step p = (eta g + e~) + q.  conef_decompress_error returns
 * e~ + q.  A checkpoint also needs the step that stored e~
 * (conef_get_error_step / conef_set_error_step).
 * stochastic quantiser (Eq. 6 with the max-norm of Sec. 5.1, block-wise):
 * `levels` = s in 1..32767; per block a = max|r|, scale = a/s (fp32), the
 * stored level of r_j is floor(u) or floor(u)+1 with u = |r_j|/scale, up with
 * probability u - floor(u), signed; E[level * scale] = r_j.  Levels are kept
 * as int8 when s <= 127, else int16.  The uniform variate of (worker i, tensor,
 * step t, element j) is the top 24 bits of the library's 64-bit hash of j in
 * the stream (mix64(seed + i + 1), tensor, t), times 2^-24.
 * cs_chunk (count sketch only; 0 = off): the sketch of Sec. 4.2.2 applied to
 * runs of a tensor, one level below the paper's layer-wise use.  A tensor of
 * d elements is cut into nc = max(1, floor(d / cs_chunk)) runs of cs_chunk
 * consecutive elements (the last run also takes the remainder); run c owns
 * the buckets [b(c), b(c+1)) of every sketch row, b(c) = floor(w c cs_chunk / d),
 * b(nc) = w, and element j of run c goes to bucket
 * b(c) + (((u >> 32) * (b(c+1) - b(c))) >> 32) with the hash u of j as before.
 * State size and layout are unchanged.  Runs never share a bucket, so the
 * library keeps a run's window in shared memory: coalesced reads and writes of
 * the sketch instead of gathers and atomic adds in L2.  Must be a multiple of
 * 256 and at least 4 cs_col_div, else CONEF_ERR_INVALID_ARG. */
typedef struct {
    int32_t kind;
    int32_t block;
    int32_t scale_dtype;
    int32_t cs_rows;
    int64_t cs_col_div;
    uint64_t seed; /* sketches: seed of the hash and sign functions */
    float beta;
    int32_t levels; /* stochastic quantiser: s */
    int32_t iconef; /* 1: iConEF-v1 (Alg. 3), see above; 0: off */
    int32_t cs_chunk; /* count sketch: elements per run, see above; 0: one run per tensor */
} conef_c_cfg;

/* Size in bytes of the device workspace for this configuration (HOST out). */
int conef_workspace_bytes(const conef_tensor *tensors /* HOST */, int n_tensors, int n_workers,
                          const conef_q_cfg *q /* HOST */, const conef_c_cfg *c /* HOST */,
                          size_t *out_bytes /* HOST */);

/* Create a context.  `workspace` is DEVICE memory, 256-byte aligned, of at
 * least conef_workspace_bytes() bytes; it stays the caller's and must outlive
 * the context.  Enqueues on `stream` the zeroing of all error state
 * (e_0 = 0, Alg. 2 line 1) and the copy of q_init.  `lr` is eta. */
int conef_init(conef_ctx **out /* HOST */, const conef_tensor *tensors /* HOST */, int n_tensors,
               int n_workers, const conef_q_cfg *q /* HOST */, const conef_c_cfg *c /* HOST */,
               float lr, void *workspace /* DEVICE */, size_t workspace_bytes,
               conef_stream stream);

/* Alg. 2 lines 5, 6, 9 for every worker and tensor.  grads is a HOST array of
 * n_workers DEVICE pointers; each points at one worker's gradient, the flat
 * fp32 concatenation of all tensors in table order (borrowed, read only,
 * 4-byte aligned; 32-byte alignment enables the vectorised kernels).
 * `step` is t; it must increase from call to call.  Identity and random-k Q
 * take phase 0 only.  Low-rank Q takes two phases because two reductions sit
 * inside Q: step(t,0) [P_i = M_i Q_{t-1}] -> reduce(MSG_P) [P_hat] ->
 * step(t,1) [Q_i = M_i^T P_hat; r; state = C(r)] -> reduce(MSG_Q) [Q_t].
 * Phase 1 may be given as phase 2 (Q_i only) followed by phase 3 (residual
 * and store only), which lets a caller read or replace the factors in
 * between; phase 4 is phase 3 computed by the fused kernel (conef_set_fused).
 * Another order returns CONEF_ERR_BAD_PHASE and launches nothing.
 * Non-finite gradients or states are not trapped and set no status: they
 * propagate IEEE-wise into p, the messages and the factors; a block maximum
 * skips NaN entries, and the stored code of a non-finite residual is
 * unspecified. */
int conef_step(conef_ctx *ctx, int64_t step, const float *const *grads, int phase,
               conef_stream stream);

/* Alg. 2 line 7 without the division by N: out_sum[j] = ((m_0[j] + m_1[j]) +
 * m_2[j]) + ... in fp32, worker order.  out_sum is DEVICE memory of
 * conef_message_elems(which) floats, concatenated over tensors in table
 * order; it may be NULL for MSG_P and MSG_Q, whose results (the
 * orthonormalised P_hat, the warm start Q_t = sum/N) also stay inside the
 * context.  MSG_VALUES: the k selected values per compressed tensor in
 * ascending index order (all d values for Q = identity).  MSG_DENSE1D: the
 * pass-through tensors. */
int conef_reduce_messages(conef_ctx *ctx, int which, float *out_sum /* DEVICE */,
                          conef_stream stream);

/* Alg. 2 lines 7-8, x <- x - Delta_t with Delta_t the mean over workers of
 * Q's outputs.  x is DEVICE memory laid out like one worker's gradient (all
 * tensors, table order), read and written in place.  sum_values and
 * sum_dense1d are the DEVICE buffers conef_reduce_messages filled for this
 * step (MSG_VALUES; MSG_DENSE1D); either may be NULL when that message kind
 * is empty.  Identity Q and pass-through tensors: x[j] -= sum[j]/N.  Random-k:
 * x[idx[s]] -= sum[s]/N for the k shared indices of this step.  Low-rank:
 * x[a][b] -= fma-chain over c of P_hat[a][c] * Qmean[b][c], Qmean = (sum_i
 * Q_i)/N as left in the context by reduce(MSG_Q); the call must follow that
 * reduction (else CONEF_ERR_BAD_PHASE). */
int conef_apply_update(conef_ctx *ctx, float *x /* DEVICE */, const float *sum_values /* DEVICE */,
                       const float *sum_dense1d /* DEVICE */, conef_stream stream);

/* Error reset for a linear error compressor (Sec. 4.2.2 (ii); identity, count
 * sketch, row sketch): every worker's stored error becomes the mean over
 * workers, S_i <- (S_0 + S_1 + ...)/N (sum in worker order, one fp32
 * division).  Other compressors, and iconef = 2 (whose e~ is kept outside that
 * state), return CONEF_ERR_UNSUPPORTED.  Call it between steps. */
int conef_error_reset(conef_ctx *ctx, conef_stream stream);

/* Alg. 2 line 5's decode alone: the error e of one worker, concatenated over
 * the compressed tensors in table order, written to out (DEVICE,
 * conef_error_elems() floats). */
int conef_decompress_error(conef_ctx *ctx, int worker, float *out /* DEVICE */,
                           conef_stream stream);

/* Frees the host-side context and the side streams it created (the tuned low-rank passes run their
 * CTA-size classes on side streams that fork from and join into the caller's stream); the
 * workspace stays the caller's. */
void conef_destroy(conef_ctx *ctx);

/* ---- sizes ---- */
int64_t conef_message_elems(const conef_ctx *ctx, int which); /* floats per worker */
int64_t conef_error_elems(const conef_ctx *ctx);              /* sum of d over compressed tensors */
int64_t conef_state_bytes_per_worker(const conef_ctx *ctx);   /* compressed error state */

/* ---- inspection (tests, checkpoints); none is on the hot path ---- */

/* DEVICE pointer to worker's message buffer of the given kind. */
int conef_get_message(const conef_ctx *ctx, int which, int worker, float **ptr /* HOST out */);
/* DEVICE pointers to the stored error of (worker, tensor): a = codes (int8 or
 * packed int4), dense e (identity) or the sketch; b = scales (fp32 or fp16) or
 * NULL.  Sizes in bytes. */
int conef_get_state(const conef_ctx *ctx, int worker, int tensor, void **a, size_t *a_bytes,
                    void **b, size_t *b_bytes);
/* The same for the second state q of iConEF-v1, or for e~ of iConEF-v2 (a = k fp32 values, b =
 * NULL); CONEF_ERR_INVALID_ARG when iconef is 0. */
int conef_get_state2(const conef_ctx *ctx, int worker, int tensor, void **a, size_t *a_bytes,
                     void **b, size_t *b_bytes);
/* iConEF-v2: the step whose second draw of Q stored the current e~ (-1: none yet, e~ = 0), and a
 * setter for a context that resumes from a checkpoint (host only, nothing is launched;
 * CONEF_ERR_INVALID_ARG unless iconef = 2 and -1 <= step < 2^62). */
int64_t conef_get_error_step(const conef_ctx *ctx);
int conef_set_error_step(conef_ctx *ctx, int64_t step);
/* DEVICE pointer to this step's sorted random-k indices of a tensor (uint32[k]). */
int conef_get_indices(const conef_ctx *ctx, int tensor, uint32_t **idx, int64_t *k);
/* DEVICE pointers to the low-rank factors of a tensor: P_hat (rows x r), the
 * warm start Q (cols x r), and worker's local Q_i (cols x r) / P_i (rows x r). */
int conef_get_factors(const conef_ctx *ctx, int tensor, int worker, float **p_hat, float **q_prev,
                      float **q_i, float **p_i, int *rank);
/* Most recent consistency status written by the kernels (0 = none).
 * Synchronises `stream`. */
int conef_last_status(conef_ctx *ctx, conef_stream stream, int *status /* HOST out */);
/* Kernels launched by this context so far. */
int64_t conef_launch_count(const conef_ctx *ctx);
/* Rank-sharded runs (one process per GPU, the messages all-reduced across processes between
 * conef_step and conef_reduce_messages, Alg. 2 line 7): the N of the means (the warm start
 * Q_t = sum/N left by reduce(MSG_Q), the update x -= sum/N of conef_apply_update) is then the
 * number of workers of the whole job, not of this context.  total >= n_workers; the default is
 * n_workers. */
int conef_set_total_workers(conef_ctx *ctx, int total);
/* Choose kernels: 0 = generic kernels only, 1 = tuned kernels where the
 * tensor's shape and alignment allow (default). */
int conef_set_fast_path(conef_ctx *ctx, int enable);
/* Low-rank Q, phase 1 (Sec. 5.2; Alg. 2 line 9): on tensors whose shape allows it (rank 4 or 8,
 * cols a multiple of 32 and at least 256, int4 blocks of 128 or int8 blocks of 256) the two
 * halves of phase 1, Q_i = M_i^T P_hat and state = C(p - P_hat Q_i^T), run in ONE persistent
 * kernel whose CTAs take tiles of both halves from one list, ordered so that the second
 * half of a (worker, tensor) pair follows its first half while the gradient and the codes are
 * still in L2.  The kernel is launched cooperatively (all its CTAs resident) because a tile of
 * the second half waits for the tiles of the first; every wait is bounded, and one that runs
 * out is reported by conef_last_status.  enable = 0 (the default) keeps the separate kernels
 * (what phases 2 and 3 always run).  tile_periods = 0 takes the default tile length; a smaller number makes
 * small tensors span many tiles (tests) and is refused with CONEF_ERR_UNSUPPORTED where the
 * partial sums of a tensor would not fit the scratch.  ctas_per_sm (0 = default, or 2..4):
 * resident CTAs per SM the kernel is built for.  Nothing is launched. */
int conef_set_fused(conef_ctx *ctx, int enable, int tile_periods, int ctas_per_sm);
/* Whether phase 1 currently uses that kernel (HOST outs, any may be NULL): active, CTAs of the
 * launch, periods per tile, shared-memory slots per warp, tiles per step. */
int conef_fused_info(const conef_ctx *ctx, int *active, int *ctas, int *tile_periods, int *ring, int *tasks);
/* For tests: phase 4 of conef_step is phase 3 computed by that kernel: the residual is formed
 * with the Q_i found in the message buffer (which a caller may have replaced after phase 2),
 * and the Q_i the kernel itself computes on the way is left in a second buffer, to which this
 * returns the DEVICE pointer for (tensor, worker).  CONEF_ERR_INVALID_ARG for a tensor the
 * kernel does not take. */
int conef_get_fused_q(const conef_ctx *ctx, int tensor, int worker, float **q_i /* HOST out */);
const char *conef_error_string(int code);

/* ---- for callers that cannot allocate ----
 *
 * (The paper has no counterpart to this call: it is a packaging of step S3a,
 * the shared random-k index set, for a caller without a context.)
 *
 * The side that receives a random-k message has to know the index set S_t to
 * scatter the k values back into a dense update; S_t depends on (seed, tensor,
 * step) only.  A receiver of that kind (a parameter server, a rank that only
 * applies updates, a hook run inside another framework's step) often has no
 * ConEF context and may not use the device allocator: its memory pool is fixed
 * up front, and an allocation in the middle of a step would synchronise the
 * device or fail under memory pressure.  This call writes S_t (k indices,
 * ascending, bit-identical to what conef_step produces for the same seed,
 * tensor index and step) into idx_out (DEVICE, k uint32, caller-owned) and
 * allocates nothing: no cudaMalloc, no cudaFree, no allocating library call.
 *
 * Its scratch (radix histograms and one counter per 256 elements, about
 * 290 KB) is a fixed array in the library's device image; every GPU that loads
 * the library holds it until the process exits.  Hence the limit
 * d <= CONEF_NOALLOC_MAX_ELEMS; a larger d returns CONEF_ERR_TOO_LARGE and
 * launches nothing.  The first call on a device looks up the array's device
 * address (cudaGetSymbolAddress); make that first call before any stream
 * capture.  All calls share the one array and it keeps the last call's
 * contents (each call clears what it needs zeroed), so two calls whose work
 * overlaps on the GPU -- different streams, or different host threads -- race:
 * issue them on one stream, or order them yourself.  Work is enqueued on
 * `stream`; the call does not synchronise, so a selection that fails on the
 * device (more than 1024 elements sharing the threshold's 32-bit hash: not
 * observed, and excluded for practical purposes at d <= 2^24) cannot be
 * returned as a code: it is reported in the output instead, idx_out[0] =
 * 0xFFFFFFFF, a value no index can take, and no write ever goes past
 * idx_out[k-1].  A CUDA error pending from before the call makes it return
 * CONEF_ERR_CUDA without launching anything. */
#define CONEF_NOALLOC_MAX_ELEMS (1 << 24)
int conef_randk_indices_noalloc(uint64_t seed, int64_t tensor, int64_t step, int64_t d, int64_t k,
                                uint32_t *idx_out /* DEVICE */, conef_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* CONEF_H */
