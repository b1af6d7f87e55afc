/*
 * CPU oracle for the outlier-aware W4A16 decode matmul.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct
 * statement of what the method computes.  Only the test-suite, the smoke check
 * and the benchmark's cpu_baseline / reference arm may build or call it.  It
 * shares no code, header, table or helper with the CUDA library; the format
 * decoders below are written from the packed-format description alone.
 *
 * What it states (paper passage for each):
 *   - affine 4-bit group quantiser            Eq. 2 (q = round(w/s) + z) and the
 *                                             formulas for s and z given with Eq. 3
 *   - dequantisation  w^ = s (q - z)          Eq. 3
 *   - result  Y = X deq(W_Q) + X W_O          Eq. 1
 *   - Tile-COO arrays (tile_indptr, bucket_info, packed_outliers; four
 *     outliers per 16-byte packet, each a 32-bit slot: BF16 value, row inside
 *     the tile, column number inside the bucket)
 *                                             Section 3.2.1, Table 1
 *
 * Readings taken where the paper is silent (each also listed in the design
 * notes): round = round-half-to-even; q and z clamped to [0,15]; the quantiser
 * runs in IEEE binary32 with the BF16-rounded scale; the group range always
 * contains 0; a degenerate group gets s = 1, z = 0, q = 0; an outlier slot holds
 * q = z so that it dequantises to exactly 0 and W_O carries the full BF16
 * weight; groups run along K.
 *
 * Floating point: everything after the quantiser is binary64, k ascending,
 * no blocking, no reordering.  Build with -ffp-contract=off and without
 * -ffast-math.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ BF16 */

/* binary32 -> bfloat16, round to nearest even; NaN stays NaN. */
uint16_t orc_f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

float orc_bf16_to_f32(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------ quantiser */

static int clamp_i(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

/*
 * Eq. 2 with b = 4, per (group of g rows along K, column n), over the weights
 * that are not outliers.  W is K x N row-major binary32; mask is K x N (1 =
 * outlier) or NULL.  Outputs: q K x N (one code per byte), scale and zero
 * (K/g) x N as BF16 bit patterns.  Returns 0, or -1 on bad sizes.
 */
int orc_quantize(const float* W, const uint8_t* mask, uint32_t K, uint32_t N, uint32_t g,
                 uint8_t* q, uint16_t* scale, uint16_t* zero) {
    if (g == 0 || K % g != 0) return -1;
    const uint32_t G = K / g;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < (int64_t)N; ++n) {
        for (uint32_t gi = 0; gi < G; ++gi) {
            float wmin = 0.0f, wmax = 0.0f; /* the range always contains 0 */
            for (uint32_t k = gi * g; k < (gi + 1) * g; ++k) {
                size_t idx = (size_t)k * N + (size_t)n;
                if (mask && mask[idx]) continue;
                float w = W[idx];
                if (w < wmin) wmin = w;
                if (w > wmax) wmax = w;
            }
            float s32 = (wmax - wmin) / 15.0f; /* s = (wmax - wmin) / (2^b - 1) */
            uint16_t sb = orc_f32_to_bf16(s32);
            float sf = orc_bf16_to_f32(sb);
            int z;
            if (!(sf > 0.0f)) { /* degenerate group */
                sb = orc_f32_to_bf16(1.0f);
                sf = 1.0f;
                z = 0;
                for (uint32_t k = gi * g; k < (gi + 1) * g; ++k) q[(size_t)k * N + (size_t)n] = 0;
            } else {
                z = clamp_i((int)nearbyintf(-wmin / sf), 0, 15); /* z = round(-wmin / s) */
                for (uint32_t k = gi * g; k < (gi + 1) * g; ++k) {
                    size_t idx = (size_t)k * N + (size_t)n;
                    if (mask && mask[idx]) {
                        q[idx] = (uint8_t)z; /* dequantises to exactly 0 */
                    } else {
                        int qi = (int)nearbyintf(W[idx] / sf) + z; /* q = round(w / s) + z */
                        q[idx] = (uint8_t)clamp_i(qi, 0, 15);
                    }
                }
            }
            scale[(size_t)gi * N + (size_t)n] = sb;
            zero[(size_t)gi * N + (size_t)n] = orc_f32_to_bf16((float)z);
        }
    }
    return 0;
}

/* Eq. 3: What[k][n] = s[k/g][n] * (q[k][n] - z[k/g][n]), in binary64. */
void orc_dequant(const uint8_t* q, const uint16_t* scale, const uint16_t* zero, uint32_t K,
                 uint32_t N, uint32_t g, double* What) {
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < (int64_t)K; ++k) {
        const size_t gi = (size_t)k / g;
        for (uint32_t n = 0; n < N; ++n) {
            double s = (double)orc_bf16_to_f32(scale[gi * N + n]);
            double z = (double)orc_bf16_to_f32(zero[gi * N + n]);
            What[(size_t)k * N + n] = s * ((double)q[(size_t)k * N + n] - z);
        }
    }
}

/* --------------------------------------------------------------- result */

/*
 * Eq. 1 on a list of output columns (cols == NULL: all N columns, ncols == N).
 *   Y[m][j]    = sum_k X[m][k] * s (q - z)  +  sum over outliers in column
 *                cols[j] of X[m][k] * W_O[k][n]
 *   Yabs[m][j] = the same sums with every product replaced by its magnitude
 *                (NULL to skip); used only for condition-aware reporting.
 * X is M x K BF16 bits, row-major.  Outliers come as COO (k, n, value bits);
 * value_type 0: the bits are BF16, 1: IEEE binary16 (Table 1's value field
 * allows either).
 * Y and Yabs are M x ncols binary64, row-major.
 */
/* IEEE binary16 -> binary64, from the definition: 1 sign, 5 exponent (bias 15),
 * 10 fraction bits; exponent 0 is subnormal (fraction * 2^-24), 31 is inf/NaN. */
double orc_f16_to_f64(uint16_t h) {
    const int sign = h >> 15, e = (h >> 10) & 31, f = h & 1023;
    double mag;
    if (e == 0) mag = ldexp((double)f, -24);
    else if (e == 31) mag = f ? NAN : INFINITY;
    else mag = ldexp(1.0 + (double)f / 1024.0, e - 15);
    return sign ? -mag : mag;
}

void orc_fused_matmul(const uint16_t* X, uint32_t M, uint32_t K, uint32_t N, uint32_t g,
                      const uint8_t* q, const uint16_t* scale, const uint16_t* zero,
                      const uint32_t* coo_k, const uint32_t* coo_n, const uint16_t* coo_v,
                      uint32_t value_type, size_t nnz, const uint32_t* cols, uint32_t ncols, double* Y,
                      double* Yabs) {
    /* dense part: X * dequant(W_Q) */
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < (int64_t)ncols; ++j) {
        const uint32_t n = cols ? cols[j] : (uint32_t)j;
        for (uint32_t m = 0; m < M; ++m) {
            double acc = 0.0, accabs = 0.0;
            for (uint32_t k = 0; k < K; ++k) {
                const size_t gi = (size_t)k / g;
                double s = (double)orc_bf16_to_f32(scale[gi * N + n]);
                double z = (double)orc_bf16_to_f32(zero[gi * N + n]);
                double w = s * ((double)q[(size_t)k * N + n] - z);
                double x = (double)orc_bf16_to_f32(X[(size_t)m * K + k]);
                acc += x * w;
                accabs += fabs(x * w);
            }
            Y[(size_t)m * ncols + (size_t)j] = acc;
            if (Yabs) Yabs[(size_t)m * ncols + (size_t)j] = accabs;
        }
    }
    /* sparse part: X * W_O, one COO entry at a time */
    int64_t* slot = NULL;
    if (cols) {
        slot = (int64_t*)malloc(sizeof(int64_t) * (size_t)N);
        for (uint32_t n = 0; n < N; ++n) slot[n] = -1;
        for (uint32_t j = 0; j < ncols; ++j) slot[cols[j]] = (int64_t)j;
    }
    for (size_t e = 0; e < nnz; ++e) {
        int64_t j = cols ? slot[coo_n[e]] : (int64_t)coo_n[e];
        if (j < 0) continue;
        double v = value_type == 1 ? orc_f16_to_f64(coo_v[e]) : (double)orc_bf16_to_f32(coo_v[e]);
        for (uint32_t m = 0; m < M; ++m) {
            double x = (double)orc_bf16_to_f32(X[(size_t)m * K + coo_k[e]]);
            Y[(size_t)m * ncols + (size_t)j] += x * v;
            if (Yabs) Yabs[(size_t)m * ncols + (size_t)j] += fabs(x * v);
        }
    }
    free(slot);
}

/* ------------------------------------------- pad-slot repurposing */

/*
 * Section 3.2.1, last remark: padding slots of the packed outliers can hold
 * original weight values.  In the column-slotted packets a bucket (four
 * columns of a 128 x BN tile: tile column c belongs to bucket 8*(c/32) + c%8)
 * is as deep as its longest column; every other column has depth - count
 * padding slots that cost their bytes anyway.  This function names the
 * weights that go there.  For every tile, bucket and column, taken on their
 * own:
 *   count = the column's outliers inside the tile (mask = 1, BF16 value not 0);
 *   depth = the largest count of the bucket's four columns; a bucket with a
 *           count above 32 is left alone (its packets are laid out otherwise);
 *   the depth - count non-outlier weights of the column inside the tile with
 *   the largest error |w - s (q - z)| of the quantisation under `mask`
 *   (Eq. 2, Eq. 3; binary64 difference), larger error first, lower row first
 *   among equals, error 0 or BF16 value 0 never, become outliers as well.
 * mask_out = mask plus those.  Quantising again under mask_out and encoding
 * gives the same packet count as under mask.  q, scale, zero: the result of
 * orc_quantize under `mask`.  Returns the number of weights added, or -1.
 */
int64_t orc_repurpose_pads(const float* W, const uint8_t* mask, uint32_t K, uint32_t N, uint32_t g,
                           uint32_t BN, const uint8_t* q, const uint16_t* scale, const uint16_t* zero,
                           uint8_t* mask_out) {
    if (K % 128 != 0 || N % BN != 0 || g == 0 || K % g != 0) return -1;
    memcpy(mask_out, mask, (size_t)K * N);
    int64_t added = 0;
    for (uint32_t tn = 0; tn < N / BN; ++tn)
        for (uint32_t kt = 0; kt < K / 128; ++kt)
            for (uint32_t b = 0; b < BN / 4; ++b) {
                uint32_t count[4], depth = 0;
                for (uint32_t j = 0; j < 4; ++j) {
                    const uint32_t n = tn * BN + 32 * (b / 8) + b % 8 + 8 * j;
                    count[j] = 0;
                    for (uint32_t r = 0; r < 128; ++r) {
                        const size_t idx = (size_t)(kt * 128 + r) * N + n;
                        if (mask[idx] && (orc_f32_to_bf16(W[idx]) & 0x7fffu) != 0) ++count[j];
                    }
                    if (count[j] > depth) depth = count[j];
                }
                if (depth > 32) continue;
                for (uint32_t j = 0; j < 4; ++j) {
                    const uint32_t n = tn * BN + 32 * (b / 8) + b % 8 + 8 * j;
                    for (uint32_t pick = count[j]; pick < depth; ++pick) {
                        double best = 0.0;
                        int64_t best_r = -1;
                        for (uint32_t r = 0; r < 128; ++r) {
                            const uint32_t k = kt * 128 + r;
                            const size_t idx = (size_t)k * N + n;
                            if (mask_out[idx] || (orc_f32_to_bf16(W[idx]) & 0x7fffu) == 0) continue;
                            const double s = (double)orc_bf16_to_f32(scale[(size_t)(k / g) * N + n]);
                            const double z = (double)orc_bf16_to_f32(zero[(size_t)(k / g) * N + n]);
                            const double err = fabs((double)W[idx] - s * ((double)q[idx] - z));
                            if (err > best) best = err, best_r = (int64_t)r;   /* strict: the lowest row wins a tie */
                        }
                        if (best_r < 0) break;
                        mask_out[(size_t)(kt * 128 + (uint32_t)best_r) * N + n] = 1;
                        ++added;
                    }
                }
            }
    return added;
}

/* ------------------------------------------------------ format decoders */

/*
 * Packed INT4 weight buffer -> q[K][N], from the format description:
 *
 *   The buffer is a sequence of chunks, one per (column tile tn, row tile kt),
 *   ordered tn-major (chunk index tn * (K/128) + kt).  A chunk covers 128 rows
 *   by BN columns and holds 16 * BN little-endian 32-bit words.  Word index
 *   inside the chunk, with j = 0..3, t = 0..BN-1, w = 0..3:
 *        (j * BN + t) * 4 + w .
 *   Nibble p (bits 4p .. 4p+3) of that word, p = i + 4h with i = 0..3, h = 0..1, is the code of
 *        column  tn*BN + t
 *        row     kt*128 + 32*j + 8*w + 2*i + h
 */
int orc_decode_wq(const uint32_t* wq, uint32_t K, uint32_t N, uint32_t BN, uint8_t* q) {
    if (K % 128 != 0 || BN == 0 || N % BN != 0) return -1;
    const uint32_t KT = K / 128, NT = N / BN;
    const size_t chunk_words = (size_t)16 * BN;
    for (uint32_t tn = 0; tn < NT; ++tn)
        for (uint32_t kt = 0; kt < KT; ++kt) {
            const uint32_t* chunk = wq + ((size_t)tn * KT + kt) * chunk_words;
            for (uint32_t j = 0; j < 4; ++j)
                for (uint32_t t = 0; t < BN; ++t)
                    for (uint32_t w = 0; w < 4; ++w) {
                        uint32_t word = chunk[(j * BN + t) * 4 + w];
                        for (uint32_t p = 0; p < 8; ++p) {
                            uint32_t i = p & 3, h = p >> 2;
                            uint32_t col = tn * BN + t;
                            uint32_t row = kt * 128 + 32 * j + 8 * w + 2 * i + h;
                            q[(size_t)row * N + col] = (uint8_t)((word >> (4 * p)) & 0xfu);
                        }
                    }
        }
    return 0;
}

/*
 * Tile-COO arrays -> COO list, from the format description:
 *
 *   Tiles are 128 rows by BN columns, tile index tn * (K/128) + kt.
 *   tile_indptr[t] .. tile_indptr[t+1] is the tile's range of 16-byte packets
 *   in packed_outliers.  bucket_info[t * NB + b] = offset | (depth << 16) |
 *   (tail << 24), offset 16 bits, depth and tail 8 bits each: bucket b of
 *   tile t owns packets [tile_indptr[t] + offset, + depth + tail).  Bucket b
 *   holds the tile columns 32 * (b / 8) + b % 8 + 8 * j, j = 0..3.
 *   A packet is four little-endian 32-bit slots.  A slot: bits 13-31 the
 *   value (an FP32 number cut to ten explicit significand bits; for a BF16
 *   value bits 13-15 are 0 and bits 16-31 are its bit pattern), bits 5-11 the
 *   row inside the tile, bits 3-4 the column number j, all other bits 0.  A
 *   slot whose value bits are all 0 is padding.  In the first `depth` packets
 *   of a bucket, slot number i names column number i.  out_v receives the
 *   19 value bits (bits 13-31 of the slot, shifted down).
 *
 * out_* must have room for 4 * (number of packets) entries; *count receives the
 * number of real entries.  Returns 0, or a negative code for a structural
 * error (-2 indptr not monotone, -3 bucket range outside its tile, -4 a slot
 * with stray bits, or a column-slotted slot that names another column).
 */
int orc_decode_tilecoo(const uint32_t* tile_indptr, const uint32_t* bucket_info,
                       const uint8_t* packed, uint32_t K, uint32_t N, uint32_t BN, uint32_t NB,
                       uint32_t* out_k, uint32_t* out_n, uint32_t* out_v, uint32_t* out_bucket,
                       size_t* count) {
    if (K % 128 != 0 || N % BN != 0) return -1;
    const uint32_t KT = K / 128, NT = N / BN;
    size_t c = 0;
    for (uint32_t tn = 0; tn < NT; ++tn)
        for (uint32_t kt = 0; kt < KT; ++kt) {
            const size_t t = (size_t)tn * KT + kt;
            const uint32_t p0 = tile_indptr[t], p1 = tile_indptr[t + 1];
            if (p1 < p0) return -2;
            for (uint32_t b = 0; b < NB; ++b) {
                uint32_t info = bucket_info[t * NB + b];
                uint32_t off = info & 0xffffu, depth = (info >> 16) & 0xffu, tail = info >> 24;
                if ((size_t)p0 + off + depth + tail > (size_t)p1) return -3;
                for (uint32_t i = 0; i < depth + tail; ++i) {
                    const uint8_t* pk = packed + ((size_t)p0 + off + i) * 16;
                    for (uint32_t sidx = 0; sidx < 4; ++sidx) {
                        uint32_t slot = (uint32_t)pk[4 * sidx] | ((uint32_t)pk[4 * sidx + 1] << 8) |
                                        ((uint32_t)pk[4 * sidx + 2] << 16) | ((uint32_t)pk[4 * sidx + 3] << 24);
                        uint32_t kk = (slot >> 5) & 127u, j = (slot >> 3) & 3u;
                        uint32_t v = slot >> 13;
                        if ((slot & 0x1007u) != 0) return -4;
                        if (i < depth && j != sidx) return -4;
                        if (v == 0) continue;
                        out_k[c] = kt * 128 + kk;
                        out_n[c] = tn * BN + 32 * (b / 8) + b % 8 + 8 * j;
                        out_v[c] = v;
                        if (out_bucket) out_bucket[c] = (uint32_t)(t * NB + b);
                        ++c;
                    }
                }
            }
        }
    *count = c;
    return 0;
}
