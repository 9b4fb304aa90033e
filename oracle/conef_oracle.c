/*
 * CPU oracle for one step of contractive error feedback (ConEF).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
 * CUDA library is compared with.  Nothing on the product path may include,
 * link or call it, and it shares no code, table or constant generator with
 * the CUDA sources.  Every function is a direct transcription of one line of
 * the paper's algorithms (or of the reading of a silent point that the design
 * notes list), written as scalar loops so it can be checked by eye.
 *
 * Numerical convention (the paper fixes fp32 storage and says nothing else):
 *   - stored values are fp32; elementwise operations are fp32, in exactly the
 *     order written here, with a fused multiply-add only where fmaf() is
 *     written (compile with -ffp-contract=off);
 *   - every long reduction (dot product, norm, sketch bucket) accumulates in
 *     fp64 in ascending index order and is rounded to fp32 once;
 *   - the sum over workers is the exception: fp32 adds in worker order, so
 *     that it equals what an in-order all-reduce would give.
 *   A quantisation code is an integer decided by floating point, so the
 *   decision is taken here in fp32, the precision the kernels use.
 *
 * Pins (tests/test_oracle_*.py): Q(p) + r = p; reduction to Alg. 1 when C is
 * the identity; zero error when Q is the identity; contraction bounds of
 * Assumptions 3 and 4; numpy.rint / numpy.median / numpy.linalg.qr / svd on
 * the library-routine steps; brute force on tiny inputs.  No function in
 * this file is "parity unpinned".
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ hashing
 * The paper leaves the shared random seed (Sec. 5.3, "same random seed among
 * GPUs") and the sketch's hash and sign functions h_i, s_i (Sec. 4.2.2)
 * abstract.  Reading: one 64-bit finalising mixer (the splitmix64 finaliser)
 * keyed by (seed, a, b) and evaluated at element j.                         */

#define ORC_GOLDEN 0x9E3779B97F4A7C15ULL

uint64_t orc_mix64(uint64_t z)
{
    z ^= z >> 30;
    z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27;
    z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}

/* key of the stream (seed, a, b): a = tensor index, b = step (random-k) or
 * sketch row (count sketch) */
uint64_t orc_stream(uint64_t seed, uint64_t a, uint64_t b)
{
    uint64_t s = orc_mix64(seed + ORC_GOLDEN * (a + 1));
    return orc_mix64(s + ORC_GOLDEN * (b + 1));
}

uint64_t orc_h64(uint64_t stream, uint64_t j)
{
    return orc_mix64(stream + ORC_GOLDEN * (j + 1));
}

/* ------------------------------------------------------------------- fp16
 * IEEE binary16 <-> binary32, round to nearest even, subnormals kept.      */

uint16_t orc_f32_to_f16(float f)
{
    uint32_t x;
    memcpy(&x, &f, 4);
    uint32_t sign = (x >> 16) & 0x8000u;
    uint32_t mag = x & 0x7FFFFFFFu;
    if (mag >= 0x7F800000u) /* inf or nan */
        return (uint16_t)(sign | 0x7C00u | ((mag > 0x7F800000u) ? 0x0200u : 0u));
    if (mag >= 0x477FF000u) /* rounds to >= 65520: overflow to inf */
        return (uint16_t)(sign | 0x7C00u);
    if (mag < 0x33000001u) /* <= 2^-25: rounds to zero (tie at 2^-25 goes to even = 0) */
        return (uint16_t)sign;
    int32_t e = (int32_t)(mag >> 23) - 127; /* unbiased exponent */
    uint32_t man = (mag & 0x007FFFFFu) | 0x00800000u; /* 24-bit significand */
    int shift; /* bits of the significand to drop */
    uint32_t base;
    if (e >= -14) { /* normal half */
        shift = 13;
        base = (uint32_t)(e + 15) << 10;
        man &= 0x007FFFFFu;
    } else { /* subnormal half: value = man * 2^(e-23), unit 2^-24 */
        shift = 13 + (-14 - e);
        base = 0;
    }
    uint32_t q = man >> shift;
    uint32_t rem = man & ((1u << shift) - 1u);
    uint32_t half = 1u << (shift - 1);
    if (rem > half || (rem == half && (q & 1u)))
        q += 1; /* a carry out of the mantissa bumps the exponent correctly */
    return (uint16_t)(sign | (base + q));
}

float orc_f16_to_f32(uint16_t h)
{
    uint32_t sign = ((uint32_t)h & 0x8000u) << 16;
    uint32_t e = (h >> 10) & 0x1Fu;
    uint32_t man = h & 0x3FFu;
    float mag;
    if (e == 0)
        mag = ldexpf((float)man, -24);
    else if (e == 31)
        mag = man ? NAN : INFINITY;
    else
        mag = ldexpf((float)(man | 0x400u), (int)e - 25);
    uint32_t bits;
    memcpy(&bits, &mag, 4);
    bits |= sign;
    memcpy(&mag, &bits, 4);
    return mag;
}

/* ------------------------------------------------ Alg. 2 line 5: p = eta g + e */

void orc_form_p(float lr, const float *g, const float *e, int64_t d, float *p)
{
    for (int64_t j = 0; j < d; ++j)
        p[j] = fmaf(lr, g[j], e[j]);
}

/* 1-D tensors are not compressed: the message is p = eta g (no error state). */
void orc_passthrough(float lr, const float *g, int64_t d, float *msg)
{
    for (int64_t j = 0; j < d; ++j)
        msg[j] = lr * g[j];
}

/* --------------------------------------- Q = unscaled random-k, shared seed
 * (Sec. 1 "(unscaled) random-k"; remark after Assumption 4).  The index set
 * S_t holds the k indices with the smallest 64-bit keys
 *     key(j) = (high 32 bits of h64(seed, tensor, step, j)) << 32 | j .
 * The index in the low half makes the keys distinct, so exactly k are taken;
 * they depend on (seed, tensor, step) only, hence are identical on all
 * workers.  idx receives S_t in ascending index order.                     */

static int cmp_u64(const void *a, const void *b)
{
    uint64_t x = *(const uint64_t *)a, y = *(const uint64_t *)b;
    return (x > y) - (x < y);
}
static int cmp_u32(const void *a, const void *b)
{
    uint32_t x = *(const uint32_t *)a, y = *(const uint32_t *)b;
    return (x > y) - (x < y);
}

int orc_randk_indices(uint64_t seed, int64_t tensor, int64_t step, int64_t d, int64_t k,
                      uint32_t *idx)
{
    if (d <= 0 || d > 0xFFFFFFFFLL || k < 0 || k > d)
        return -1;
    uint64_t *keys = (uint64_t *)malloc((size_t)d * sizeof(uint64_t));
    if (!keys)
        return -2;
    uint64_t st = orc_stream(seed, (uint64_t)tensor, (uint64_t)step);
    for (int64_t j = 0; j < d; ++j)
        keys[j] = ((orc_h64(st, (uint64_t)j) >> 32) << 32) | (uint64_t)j;
    qsort(keys, (size_t)d, sizeof(uint64_t), cmp_u64);
    for (int64_t q = 0; q < k; ++q)
        idx[q] = (uint32_t)(keys[q] & 0xFFFFFFFFu);
    qsort(idx, (size_t)k, sizeof(uint32_t), cmp_u32);
    free(keys);
    return 0;
}

/* Delta = Q(p): message m[q] = p[idx[q]] (no d/k rescaling); residual
 * r = p - Delta, i.e. r[j] = 0 on S_t and p[j] elsewhere (Alg. 2 line 9,
 * the argument of C).                                                      */
void orc_randk_apply(const float *p, int64_t d, const uint32_t *idx, int64_t k, float *msg,
                     float *r)
{
    for (int64_t j = 0; j < d; ++j)
        r[j] = p[j];
    for (int64_t q = 0; q < k; ++q) {
        msg[q] = p[idx[q]];
        r[idx[q]] = p[idx[q]] - p[idx[q]]; /* p - Delta on a transmitted entry */
    }
}

/* ------------------------- C = block-wise symmetric absmax integer quantiser
 * (Sec. 4.2.1 "int-quantization", max-norm scaling as in Sec. 5.1).  The
 * tensor is flattened row-major and cut into blocks of `block` elements (the
 * last one may be short).  Per block: a = max |r_j|; s = a / qmax, rounded to
 * binary16 (saturating at 65504) when scale_half; a block whose stored scale
 * is not >= FLT_MIN stores scale 0 and codes 0.  Otherwise inv = 1 / s and
 * code_j = clamp(rint(r_j * inv), -qmax, qmax), ties to even.  bits = 8:
 * one signed byte per element.  bits = 4: two's-complement nibbles, element
 * 2q in the low nibble of byte q and element 2q+1 in the high nibble.
 * scales_f32 always receives the decoded scale; scales_f16 (may be NULL)
 * receives the binary16 bits.                                              */

static int orc_quant_code(float x, int qmax)
{
    if (isnan(x))
        return 0;
    if (x >= (float)qmax)
        return qmax;
    if (x <= -(float)qmax)
        return -qmax;
    return (int)rintf(x); /* default rounding mode: nearest, ties to even */
}

void orc_quant_encode(const float *r, int64_t d, int block, int bits, int scale_half,
                      uint8_t *codes, float *scales_f32, uint16_t *scales_f16)
{
    const int qmax = (bits == 8) ? 127 : 7;
    int64_t nblocks = (d + block - 1) / block;
    if (bits == 4)
        memset(codes, 0, (size_t)((d + 1) / 2));
    for (int64_t b = 0; b < nblocks; ++b) {
        int64_t lo = b * block, hi = lo + block < d ? lo + block : d;
        float a = 0.0f;
        for (int64_t j = lo; j < hi; ++j) {
            float v = fabsf(r[j]);
            if (v > a) /* false for a NaN entry: it is skipped, and its code is 0 */
                a = v;
        }
        float s = a / (float)qmax;
        uint16_t hb = 0;
        if (scale_half) {
            if (s > 65504.0f)
                s = 65504.0f;
            hb = orc_f32_to_f16(s);
            s = orc_f16_to_f32(hb);
        }
        int zero_block = !(s >= FLT_MIN);
        if (zero_block) {
            s = 0.0f;
            hb = 0;
        }
        scales_f32[b] = s;
        if (scales_f16)
            scales_f16[b] = hb;
        float inv = zero_block ? 0.0f : 1.0f / s;
        for (int64_t j = lo; j < hi; ++j) {
            int c = zero_block ? 0 : orc_quant_code(r[j] * inv, qmax);
            if (bits == 8)
                codes[j] = (uint8_t)(int8_t)c;
            else if (j & 1)
                codes[j >> 1] |= (uint8_t)((c & 0xF) << 4);
            else
                codes[j >> 1] |= (uint8_t)(c & 0xF);
        }
    }
}

/* Alg. 2 line 5, the decode of the stored e: e_j = (float)code_j * scale_b. */
void orc_quant_decode(const uint8_t *codes, const float *scales_f32, int64_t d, int block,
                      int bits, float *e)
{
    for (int64_t j = 0; j < d; ++j) {
        int c;
        if (bits == 8)
            c = (int8_t)codes[j];
        else {
            int nib = (j & 1) ? (codes[j >> 1] >> 4) : (codes[j >> 1] & 0xF);
            c = (nib & 0x8) ? nib - 16 : nib;
        }
        e[j] = (float)c * scales_f32[j / block];
    }
}

/* ------------------------------------------- C = count sketch (Sec. 4.2.2)
 * S is v x w, row-major.  Row i uses the stream (seed, tensor, i):
 *   u = h64(stream_i, j);  h_i(j) = ((u >> 32) * w) >> 32  (0-based bucket);
 *   s_i(j) = -1 if (u & 1) else +1.
 * Hashes do not depend on the step: next step's decode needs the same ones.
 * Encode: S[i][h_i(j)] += s_i(j) * r_j for every j, each bucket accumulated
 * in fp64 in ascending j and rounded once.  Decode: e_j = median over i of
 * s_i(j) * S[i][h_i(j)]  (v odd: the middle order statistic).              */

void orc_sketch_bucket(uint64_t seed, int64_t tensor, int row, int64_t j, int64_t w,
                       int64_t *bucket, int *sign)
{
    uint64_t st = orc_stream(seed, (uint64_t)tensor, (uint64_t)row);
    uint64_t u = orc_h64(st, (uint64_t)j);
    *bucket = (int64_t)(((u >> 32) * (uint64_t)w) >> 32);
    *sign = (u & 1) ? -1 : 1;
}

int orc_sketch_encode(const float *r, int64_t d, int v, int64_t w, uint64_t seed, int64_t tensor,
                      float *S)
{
    double *acc = (double *)calloc((size_t)w, sizeof(double));
    if (!acc)
        return -2;
    for (int i = 0; i < v; ++i) {
        memset(acc, 0, (size_t)w * sizeof(double));
        for (int64_t j = 0; j < d; ++j) {
            int64_t h;
            int sg;
            orc_sketch_bucket(seed, tensor, i, j, w, &h, &sg);
            acc[h] += (double)sg * (double)r[j];
        }
        for (int64_t c = 0; c < w; ++c)
            S[(int64_t)i * w + c] = (float)acc[c];
    }
    free(acc);
    return 0;
}

void orc_sketch_decode(const float *S, int64_t d, int v, int64_t w, uint64_t seed, int64_t tensor,
                       float *e)
{
    float est[16] = {0};
    for (int64_t j = 0; j < d; ++j) {
        for (int i = 0; i < v; ++i) {
            int64_t h;
            int sg;
            orc_sketch_bucket(seed, tensor, i, j, w, &h, &sg);
            est[i] = (float)sg * S[(int64_t)i * w + h];
        }
        for (int a = 1; a < v; ++a) { /* insertion sort, v <= 15 */
            float x = est[a];
            int b = a - 1;
            while (b >= 0 && est[b] > x) {
                est[b + 1] = est[b];
                --b;
            }
            est[b + 1] = x;
        }
        e[j] = est[v / 2];
    }
}

/* --------------------- Q = rank-r approximation, one power iteration (Sec. 5.2)
 * M is the n x m row-major matrix view of p.  The paper gives one sentence;
 * the steps below are the reading the design notes list: P_i = M_i Q_prev;
 * P_bar = sum over workers; P_hat = Gram-Schmidt(P_bar); Q_i = M_i^T P_hat;
 * Delta_i = P_hat Q_i^T.                                                   */

/* P = M Q  (n x m times m x r) */
void orc_lowrank_project_rows(const float *M, int64_t n, int64_t m, const float *Q, int r, float *P)
{
    for (int64_t a = 0; a < n; ++a)
        for (int c = 0; c < r; ++c) {
            double acc = 0.0;
            for (int64_t b = 0; b < m; ++b)
                acc += (double)M[a * m + b] * (double)Q[b * r + c];
            P[a * r + c] = (float)acc;
        }
}

/* Modified Gram-Schmidt on the columns of P (n x r, row-major), left to
 * right, in place.  A column whose norm is not >= FLT_MIN becomes 0.       */
void orc_gram_schmidt(float *P, int64_t n, int r)
{
    for (int c = 0; c < r; ++c) {
        for (int cp = 0; cp < c; ++cp) {
            double dot = 0.0;
            for (int64_t a = 0; a < n; ++a)
                dot += (double)P[a * r + cp] * (double)P[a * r + c];
            float dotf = (float)dot;
            for (int64_t a = 0; a < n; ++a)
                P[a * r + c] = fmaf(-dotf, P[a * r + cp], P[a * r + c]);
        }
        double ss = 0.0;
        for (int64_t a = 0; a < n; ++a)
            ss += (double)P[a * r + c] * (double)P[a * r + c];
        float nu = (float)sqrt(ss);
        if (!(nu >= FLT_MIN)) {
            for (int64_t a = 0; a < n; ++a)
                P[a * r + c] = 0.0f;
        } else {
            for (int64_t a = 0; a < n; ++a)
                P[a * r + c] = P[a * r + c] / nu;
        }
    }
}

/* Q = M^T P_hat  (m x n times n x r) */
void orc_lowrank_project_cols(const float *M, int64_t n, int64_t m, const float *Phat, int r,
                              float *Qi)
{
    for (int64_t b = 0; b < m; ++b)
        for (int c = 0; c < r; ++c) {
            double acc = 0.0;
            for (int64_t a = 0; a < n; ++a)
                acc += (double)M[a * m + b] * (double)Phat[a * r + c];
            Qi[b * r + c] = (float)acc;
        }
}

/* Residual r = p - Delta with Delta = P_hat Q_i^T, formed as a chain of fused
 * multiply-adds in ascending c (Alg. 2 line 9, the argument of C).  delta
 * (may be NULL) receives Delta = p - r's counterpart computed directly.    */
void orc_lowrank_residual(const float *M, int64_t n, int64_t m, const float *Phat, const float *Qi,
                          int r, float *res, float *delta)
{
    for (int64_t a = 0; a < n; ++a)
        for (int64_t b = 0; b < m; ++b) {
            float acc = M[a * m + b];
            for (int c = 0; c < r; ++c)
                acc = fmaf(-Phat[a * r + c], Qi[b * r + c], acc);
            res[a * m + b] = acc;
            if (delta) {
                double dl = 0.0;
                for (int c = 0; c < r; ++c)
                    dl += (double)Phat[a * r + c] * (double)Qi[b * r + c];
                delta[a * m + b] = (float)dl;
            }
        }
}

/* ------------------------------------------------ Alg. 2 line 7: aggregate
 * out = ((m_0 + m_1) + m_2) + ...  in fp32, worker order.  The caller
 * divides by N where the mean of Sec. 2 is wanted.                          */
void orc_sum_workers(const float *const *msgs, int n_workers, int64_t len, float *out)
{
    for (int64_t j = 0; j < len; ++j) {
        float acc = msgs[0][j];
        for (int i = 1; i < n_workers; ++i)
            acc = acc + msgs[i][j];
        out[j] = acc;
    }
}

void orc_divide(const float *x, float denom, int64_t len, float *out)
{
    for (int64_t j = 0; j < len; ++j)
        out[j] = x[j] / denom;
}

/* ------------------------------------------- partial error feedback (Alg. 4)
 * Line 5: p = eta g + (1 - beta) e.  (1 - beta) is passed in as an fp32
 * value so that both sides of a comparison use the same constant; the
 * product is rounded to fp32 before the fused multiply-add.  With beta = 0
 * this is orc_form_p bit for bit.                                           */
void orc_form_p_partial(float lr, float one_minus_beta, const float *g, const float *e, int64_t d,
                        float *p)
{
    for (int64_t j = 0; j < d; ++j)
        p[j] = fmaf(lr, g[j], one_minus_beta * e[j]);
}

/* Line 9, the argument of C for a compressor that is not linear:
 * x = beta e + (p - Delta), one fused multiply-add.                         */
void orc_partial_keep(float beta, const float *e, const float *r, int64_t d, float *x)
{
    for (int64_t j = 0; j < d; ++j)
        x[j] = fmaf(beta, e[j], r[j]);
}

/* ------------------------- count sketch applied chunk by chunk (Sec. 4.2.2)
 * The paper leaves h_i abstract and applies every compressor layer-wise
 * (Sec. 5); this variant goes one level finer.  With chunk length E > 0 a
 * tensor of d elements is cut into nc = max(1, floor(d / E)) runs of E
 * consecutive elements (the last run also takes the remainder, so it holds
 * E .. 2E-1 elements), and run c owns the buckets [b(c), b(c+1)) of every
 * sketch row, b(c) = floor(w c E / d) for c < nc and b(nc) = w: widths in
 * proportion to the elements, all w buckets used.  Inside its window an
 * element is hashed as before, from its index in the whole tensor:
 *   h_i(j) = b(c) + (((u >> 32) * width_c) >> 32),  u = h64(stream_i, j).
 * One run (E >= d, or E = 0) is the plain count sketch above.  Elements of
 * different runs never collide, so a run and its window can be handled on
 * their own (in a GPU's shared memory, as Sec. 4.2.2 suggests).            */
void orc_chunk_window(int64_t d, int64_t w, int64_t chunk, int64_t j, int64_t *lo, int64_t *width)
{
    int64_t nc = chunk > 0 ? d / chunk : 1;
    if (nc < 1)
        nc = 1;
    int64_t c = chunk > 0 ? j / chunk : 0;
    if (c > nc - 1)
        c = nc - 1;
    /* w c E <= w d < 2^62 for every size the library accepts */
    int64_t b0 = c == 0 ? 0 : (int64_t)(((unsigned __int128)w * (unsigned __int128)c * (unsigned __int128)chunk) / (unsigned __int128)d);
    int64_t b1 = c == nc - 1 ? w : (int64_t)(((unsigned __int128)w * (unsigned __int128)(c + 1) * (unsigned __int128)chunk) / (unsigned __int128)d);
    *lo = b0;
    *width = b1 - b0;
}

static void chunk_bucket(uint64_t seed, int64_t tensor, int row, int64_t j, int64_t d, int64_t w,
                         int64_t chunk, int64_t *bucket, int *sign)
{
    int64_t lo, width, h;
    orc_chunk_window(d, w, chunk, j, &lo, &width);
    orc_sketch_bucket(seed, tensor, row, j, width, &h, sign);
    *bucket = lo + h;
}

int orc_sketch_encode_chunked(const float *r, int64_t d, int v, int64_t w, int64_t chunk, uint64_t seed,
                              int64_t tensor, float *S)
{
    double *acc = (double *)calloc((size_t)w, sizeof(double));
    if (!acc)
        return -2;
    for (int i = 0; i < v; ++i) {
        memset(acc, 0, (size_t)w * sizeof(double));
        for (int64_t j = 0; j < d; ++j) {
            int64_t h;
            int sg;
            chunk_bucket(seed, tensor, i, j, d, w, chunk, &h, &sg);
            acc[h] += (double)sg * (double)r[j];
        }
        for (int64_t c = 0; c < w; ++c)
            S[(int64_t)i * w + c] = (float)acc[c];
    }
    free(acc);
    return 0;
}

void orc_sketch_decode_chunked(const float *S, int64_t d, int v, int64_t w, int64_t chunk, uint64_t seed,
                               int64_t tensor, float *e)
{
    float est[16] = {0};
    for (int64_t j = 0; j < d; ++j) {
        for (int i = 0; i < v; ++i) {
            int64_t h;
            int sg;
            chunk_bucket(seed, tensor, i, j, d, w, chunk, &h, &sg);
            est[i] = (float)sg * S[(int64_t)i * w + h];
        }
        for (int a = 1; a < v; ++a) {
            float x = est[a];
            int b = a - 1;
            while (b >= 0 && est[b] > x) {
                est[b + 1] = est[b];
                --b;
            }
            est[b + 1] = x;
        }
        e[j] = est[v / 2];
    }
}

/* ------------------------------- count sketch over matrix rows (Sec. 4.2.2,
 * "tensor trick"; Sec. 5.4 uses it throughout).  The n x m matrix view is
 * hashed one ROW at a time: sketch row i is a w x m matrix T_i and
 * T_i[h_i(a)][:] += s_i(a) R[a][:], so only n hashes per sketch row are
 * needed and whole matrix rows move together.  h_i, s_i are orc_sketch_bucket
 * evaluated at the row index a.  T is v x w x m, row-major.
 *
 * The sketch is linear, so Alg. 4 line 9 needs no decode of e:
 *     T <- beta T + sketch(p - Delta).
 * Per entry: the old term beta * T (an fp32 product) first, then the rows of
 * the bucket in ascending a, accumulated in fp64 and rounded once.
 * beta = 0 gives Alg. 2 line 9 (a fresh sketch of the residual).           */
int orc_rowsketch_update(float beta, const float *R, int64_t n, int64_t m, int v, int64_t w,
                         uint64_t seed, int64_t tensor, float *T)
{
    double *acc = (double *)malloc((size_t)(w * m) * sizeof(double));
    if (!acc)
        return -2;
    for (int i = 0; i < v; ++i) {
        float *Ti = T + (int64_t)i * w * m;
        for (int64_t q = 0; q < w * m; ++q)
            acc[q] = (double)(beta * Ti[q]);
        for (int64_t a = 0; a < n; ++a) {
            int64_t h;
            int sg;
            orc_sketch_bucket(seed, tensor, i, a, w, &h, &sg);
            for (int64_t b = 0; b < m; ++b)
                acc[h * m + b] += (double)sg * (double)R[a * m + b];
        }
        for (int64_t q = 0; q < w * m; ++q)
            Ti[q] = (float)acc[q];
    }
    free(acc);
    return 0;
}

/* e[a][b] = median over i of s_i(a) * T_i[h_i(a)][b]  (v odd) */
void orc_rowsketch_decode(const float *T, int64_t n, int64_t m, int v, int64_t w, uint64_t seed,
                          int64_t tensor, float *e)
{
    float est[16];
    int64_t h[16];
    int sg[16];
    for (int64_t a = 0; a < n; ++a) {
        for (int i = 0; i < v; ++i)
            orc_sketch_bucket(seed, tensor, i, a, w, &h[i], &sg[i]);
        for (int64_t b = 0; b < m; ++b) {
            for (int i = 0; i < v; ++i)
                est[i] = (float)sg[i] * T[((int64_t)i * w + h[i]) * m + b];
            for (int x = 1; x < v; ++x) {
                float val = est[x];
                int y = x - 1;
                while (y >= 0 && est[y] > val) {
                    est[y + 1] = est[y];
                    --y;
                }
                est[y + 1] = val;
            }
            e[a * m + b] = est[v / 2];
        }
    }
}

/* ---------------- C = unbiased stochastic s-level quantiser (Eq. 6, Sec. 4.2.1)
 * with the max-norm in place of the l2 norm (Sec. 5.1), block-wise like the
 * integer quantiser.  Per block a = max|r_j|; u_j = |r_j| / a * s lies in
 * [0, s]; l = floor(u_j); the level is l+1 with probability u_j - l, else l,
 * so that E[level] = u_j.  The uniform variate rnd[j] in [0,1) is supplied by
 * the caller: up iff rnd[j] < u_j - l.  Stored: the signed level in [-s, s]
 * and the block scale a / s, so that decode is level * scale.
 * fp32 steps: scale = a / s; a block whose scale is not >= FLT_MIN is stored
 * as zeros; inv = 1 / scale; u = |r| * inv, clamped to s.                    */
void orc_stochquant_encode(const float *r, const float *rnd, int64_t d, int block, int levels,
                           int16_t *codes, float *scales_f32)
{
    int64_t nblocks = (d + block - 1) / block;
    for (int64_t b = 0; b < nblocks; ++b) {
        int64_t lo = b * block, hi = lo + block < d ? lo + block : d;
        float a = 0.0f;
        for (int64_t j = lo; j < hi; ++j) {
            float v = fabsf(r[j]);
            if (v > a)
                a = v;
        }
        float s = a / (float)levels;
        int zero_block = !(s >= FLT_MIN);
        scales_f32[b] = zero_block ? 0.0f : s;
        float inv = zero_block ? 0.0f : 1.0f / s;
        for (int64_t j = lo; j < hi; ++j) {
            int c = 0;
            if (!zero_block) {
                float u = fabsf(r[j]) * inv;
                if (!(u <= (float)levels)) /* also catches NaN */
                    u = (float)levels;
                float l = floorf(u);
                float frac = u - l; /* exact: both below 2^24 and l <= u < l + 1 */
                int lev = (int)l + ((rnd[j] < frac) ? 1 : 0);
                if (lev > levels)
                    lev = levels;
                c = (r[j] < 0.0f) ? -lev : lev;
            }
            codes[j] = (int16_t)c;
        }
    }
}

void orc_stochquant_decode(const int16_t *codes, const float *scales_f32, int64_t d, int block,
                           float *e)
{
    for (int64_t j = 0; j < d; ++j)
        e[j] = (float)codes[j] * scales_f32[j / block];
}

/* The uniform variates of the stochastic quantiser: a counter-based generator,
 * so that worker i's draw for element j of a tensor at step t is a pure
 * function of (seed, i, tensor, t, j): the top 24 bits of
 * h64(stream(mix64(seed + i + 1), tensor, t), j), scaled by 2^-24.          */
void orc_uniform24(uint64_t seed, int worker, int64_t tensor, int64_t step, int64_t d, float *out)
{
    uint64_t st = orc_stream(orc_mix64(seed + (uint64_t)worker + 1u), (uint64_t)tensor, (uint64_t)step);
    for (int64_t j = 0; j < d; ++j)
        out[j] = (float)(orc_h64(st, (uint64_t)j) >> 40) * (1.0f / 16777216.0f);
}

/* ------------------------------------- Alg. 2 lines 7-8: x <- x - Delta_t,
 * Delta_t the mean over workers of Q's outputs.  The messages arrive summed
 * (orc_sum_workers); the division by N is one fp32 division per value.     */

/* Q = identity and the pass-through tensors: Delta = sum / N, dense */
void orc_apply_dense(float *x, const float *sum, float n_workers, int64_t len)
{
    for (int64_t j = 0; j < len; ++j)
        x[j] = x[j] - sum[j] / n_workers;
}

/* Q = random-k: only the k shared coordinates move */
void orc_apply_sparse(float *x, const uint32_t *idx, const float *sum, float n_workers, int64_t k)
{
    for (int64_t s = 0; s < k; ++s)
        x[idx[s]] = x[idx[s]] - sum[s] / n_workers;
}

/* Q = rank-r: mean_i P_hat Q_i^T = P_hat Qmean^T with Qmean = (sum_i Q_i) / N
 * (the warm start of the next step).  Delta[a][b] is the fp32 chain
 * d = fma(P_hat[a][c], Qmean[b][c], d) over ascending c from d = 0.        */
void orc_apply_lowrank(float *x, int64_t n, int64_t m, const float *Phat, const float *Qmean, int r)
{
    for (int64_t a = 0; a < n; ++a)
        for (int64_t b = 0; b < m; ++b) {
            float dl = 0.0f;
            for (int c = 0; c < r; ++c)
                dl = fmaf(Phat[a * r + c], Qmean[b * r + c], dl);
            x[a * m + b] = x[a * m + b] - dl;
        }
}

/* ---------------- Q = unscaled random-block-k (Sec. 5.3, Table 2's set-up):
 * one contiguous block of k coordinates whose start is uniform on [0, d-k],
 * drawn from the shared (seed, tensor, step) stream so that every worker
 * keeps the same block: start = floor(u * (d - k + 1) / 2^32) with u the top
 * 32 bits of the stream's hash of 0.                                        */
int64_t orc_randblock_start(uint64_t seed, int64_t tensor, int64_t step, int64_t d, int64_t k)
{
    uint64_t st = orc_stream(seed, (uint64_t)tensor, (uint64_t)step);
    uint64_t u = orc_h64(st, 0) >> 32;
    uint64_t span = (uint64_t)(d - k) + 1;
    return (int64_t)((u * span) >> 32);
}

/* ------------------------------ error reset for a linear C (Sec. 4.2.2 (ii);
 * the appendix runs it every 512 steps): the workers' compressed errors are
 * all-reduced.  Reading taken here: "synchronises the local errors" = every
 * worker continues with the mean, S_i <- (S_0 + S_1 + ...) / N, the sum in
 * worker order and one fp32 division.  len = values of one worker's state.  */
void orc_error_reset(float *const *states, int n_workers, int64_t len)
{
    for (int64_t j = 0; j < len; ++j) {
        float acc = states[0][j];
        for (int i = 1; i < n_workers; ++i)
            acc = acc + states[i][j];
        acc = acc / (float)n_workers;
        for (int i = 0; i < n_workers; ++i)
            states[i][j] = acc;
    }
}

/* ---------------- the row sketch kept in binary16 (halves its memory again):
 * every entry of T is stored as fp16.  Update: the old term beta * float(T)
 * (an fp32 product) first, then the bucket's rows in ascending order, in fp64;
 * the sum is rounded to fp32, clamped to the finite half range +-65504 and
 * rounded to fp16 (nearest even).  Decode reads float(T).                    */
static uint16_t orc_store_f16(double acc)
{
    float f = (float)acc;
    if (f > 65504.0f)
        f = 65504.0f;
    if (f < -65504.0f)
        f = -65504.0f;
    return orc_f32_to_f16(f);
}

int orc_rowsketch_update_f16(float beta, const float *R, int64_t n, int64_t m, int v, int64_t w,
                             uint64_t seed, int64_t tensor, uint16_t *T)
{
    double *acc = (double *)malloc((size_t)(w * m) * sizeof(double));
    if (!acc)
        return -2;
    for (int i = 0; i < v; ++i) {
        uint16_t *Ti = T + (int64_t)i * w * m;
        for (int64_t q = 0; q < w * m; ++q)
            acc[q] = (double)(beta * orc_f16_to_f32(Ti[q]));
        for (int64_t a = 0; a < n; ++a) {
            int64_t h;
            int sg;
            orc_sketch_bucket(seed, tensor, i, a, w, &h, &sg);
            for (int64_t b = 0; b < m; ++b)
                acc[h * m + b] += (double)sg * (double)R[a * m + b];
        }
        for (int64_t q = 0; q < w * m; ++q)
            Ti[q] = orc_store_f16(acc[q]);
    }
    free(acc);
    return 0;
}

void orc_rowsketch_decode_f16(const uint16_t *T, int64_t n, int64_t m, int v, int64_t w, uint64_t seed,
                              int64_t tensor, float *e)
{
    float *Tf = (float *)malloc((size_t)(v * w * m) * sizeof(float));
    for (int64_t q = 0; q < v * w * m; ++q)
        Tf[q] = orc_f16_to_f32(T[q]);
    orc_rowsketch_decode(Tf, n, m, v, w, seed, tensor, e);
    free(Tf);
}

/* error reset of fp16 sketches: fp32 sum of the workers' values in worker order, one division,
 * stored like an update */
void orc_error_reset_f16(uint16_t *const *states, int n_workers, int64_t len)
{
    for (int64_t j = 0; j < len; ++j) {
        float acc = orc_f16_to_f32(states[0][j]);
        for (int i = 1; i < n_workers; ++i)
            acc = acc + orc_f16_to_f32(states[i][j]);
        acc = acc / (float)n_workers;
        uint16_t h = orc_store_f16((double)acc);
        for (int i = 0; i < n_workers; ++i)
            states[i][j] = h;
    }
}
