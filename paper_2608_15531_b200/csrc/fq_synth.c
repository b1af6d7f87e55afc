/*
 * Seeded synthetic inputs for the W4A16 + outlier decode matmul.
 *
 * This file only draws numbers.  It holds none of the method's arithmetic (no
 * quantiser, no packing, no matmul); both the CUDA library's callers and the
 * CPU oracle's callers feed on the same arrays it writes.
 *
 * Generator: counter based.  Every value is a SplitMix64 finaliser applied to
 * (seed, stream, index), so any element can be drawn without drawing the ones
 * before it and results do not depend on thread count.  Normals are
 * Box-Muller in binary64.
 *
 * Streams: 0 dense weights, 1 activations, 2 outlier positions, 3 outlier
 * magnitudes and signs.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline uint64_t syn_mix(uint64_t seed, uint64_t stream, uint64_t idx) {
    uint64_t z = seed ^ (stream * 0xD1B54A32D192ED03ull);
    z += (idx + 1) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline double syn_u01(uint64_t seed, uint64_t stream, uint64_t idx) {
    return ((double)(syn_mix(seed, stream, idx) >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}

static inline double syn_normal(uint64_t seed, uint64_t stream, uint64_t idx) {
    double u1 = syn_u01(seed, stream, 2 * idx);
    double u2 = syn_u01(seed, stream, 2 * idx + 1);
    return sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925286766559 * u2);
}

static inline uint16_t syn_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static inline float syn_bf16_f32(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* W[i] = (float)(sigma * N(0,1)), i over K*N row-major. */
void syn_dense_weights(uint64_t seed, uint64_t count, double sigma, float* W) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)count; ++i) W[i] = (float)(sigma * syn_normal(seed, 0, (uint64_t)i));
}

/* X[i] = bf16(N(0,1)), i over M*K row-major. */
void syn_activations(uint64_t seed, uint64_t count, uint16_t* X) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)count; ++i) X[i] = syn_bf16((float)syn_normal(seed, 1, (uint64_t)i));
}

/*
 * Place `nnz` distinct outlier positions into mask (K x N, must arrive zeroed).
 *   layout 0  uniform over the matrix
 *   layout 1  mixed: floor(nnz/2) uniform, the rest uniform inside
 *             ceil(0.01 K) hot rows (input channels)
 *   layout 2  clustered: floor(0.005 K) hot rows and floor(0.005 N) hot
 *             columns; 80 % of nnz goes into their union, but never more than
 *             75 % of the union's slots; the rest is uniform
 * Returns the number placed inside the hot region (0 for layout 0).
 */
uint64_t syn_outlier_positions(uint64_t seed, uint32_t K, uint32_t N, uint64_t nnz, int layout,
                               uint8_t* mask) {
    const uint64_t total = (uint64_t)K * N;
    uint64_t ctr = 0, placed = 0, in_hot = 0;
    if (nnz > total) nnz = total;
    uint64_t n_uniform = nnz;
    if (layout == 1) {
        uint32_t H = (uint32_t)ceil(0.01 * (double)K);
        if (H < 1) H = 1;
        uint64_t n_hot = nnz - nnz / 2;
        if (n_hot > (uint64_t)H * N / 2) n_hot = (uint64_t)H * N / 2;
        n_uniform = nnz - n_hot;
        /* uniform half first */
        while (placed < n_uniform) {
            uint64_t i = syn_mix(seed, 2, ctr++) % total;
            if (!mask[i]) { mask[i] = 1; ++placed; }
        }
        uint32_t* rows = (uint32_t*)malloc(sizeof(uint32_t) * H);
        uint8_t* is_hot = (uint8_t*)calloc(K, 1);
        for (uint32_t h = 0; h < H;) {
            uint32_t r = (uint32_t)(syn_mix(seed, 2, ctr++) % K);
            if (!is_hot[r]) { is_hot[r] = 1; rows[h++] = r; }
        }
        while (in_hot < n_hot) {
            uint64_t d = syn_mix(seed, 2, ctr++);
            uint64_t i = (uint64_t)rows[(d >> 32) % H] * N + (d & 0xffffffffull) % N;
            if (!mask[i]) { mask[i] = 1; ++in_hot; }
        }
        free(rows);
        free(is_hot);
        return in_hot;
    }
    if (layout == 2) {
        uint32_t HR = (uint32_t)floor(0.005 * (double)K), HC = (uint32_t)floor(0.005 * (double)N);
        if (HR < 1) HR = 1;
        if (HC < 1) HC = 1;
        uint64_t cap = (uint64_t)HR * N + (uint64_t)HC * K - (uint64_t)HR * HC;
        uint64_t want = (uint64_t)llround(0.8 * (double)nnz);
        uint64_t lim = (uint64_t)floor(0.75 * (double)cap);
        uint64_t n_hot = want < lim ? want : lim;
        if (n_hot > nnz) n_hot = nnz;
        uint32_t* rows = (uint32_t*)malloc(sizeof(uint32_t) * HR);
        uint32_t* cols = (uint32_t*)malloc(sizeof(uint32_t) * HC);
        uint8_t* hot_r = (uint8_t*)calloc(K, 1);
        uint8_t* hot_c = (uint8_t*)calloc(N, 1);
        for (uint32_t h = 0; h < HR;) {
            uint32_t r = (uint32_t)(syn_mix(seed, 2, ctr++) % K);
            if (!hot_r[r]) { hot_r[r] = 1; rows[h++] = r; }
        }
        for (uint32_t h = 0; h < HC;) {
            uint32_t c = (uint32_t)(syn_mix(seed, 2, ctr++) % N);
            if (!hot_c[c]) { hot_c[c] = 1; cols[h++] = c; }
        }
        const uint64_t region_a = (uint64_t)HR * N, region_b = (uint64_t)HC * K;
        while (in_hot < n_hot) {
            uint64_t d = syn_mix(seed, 2, ctr++) % (region_a + region_b);
            uint64_t i;
            if (d < region_a) {
                i = (uint64_t)rows[d / N] * N + d % N;
            } else {
                d -= region_a;
                uint32_t r = (uint32_t)(d % K);
                if (hot_r[r]) continue; /* already covered by region a: keeps the union uniform */
                i = (uint64_t)r * N + cols[d / K];
            }
            if (!mask[i]) { mask[i] = 1; ++in_hot; }
        }
        free(rows); free(cols); free(hot_r); free(hot_c);
        n_uniform = nnz - n_hot;
    }
    while (placed < n_uniform) {
        uint64_t i = syn_mix(seed, 2, ctr++) % total;
        if (!mask[i]) { mask[i] = 1; ++placed; }
    }
    return in_hot;
}

/*
 * For every marked position (index order): magnitude sigma * U(6, 20), random
 * sign, rounded to BF16; the dense weight is overwritten with that value so the
 * "original" matrix contains its outliers.  Writes the COO list; returns its
 * length.
 */
uint64_t syn_outlier_values(uint64_t seed, uint32_t K, uint32_t N, double sigma, const uint8_t* mask,
                            float* W, uint32_t* coo_k, uint32_t* coo_n, uint16_t* coo_v) {
    uint64_t c = 0;
    const uint64_t total = (uint64_t)K * N;
    for (uint64_t i = 0; i < total; ++i) {
        if (!mask[i]) continue;
        double mag = sigma * (6.0 + 14.0 * syn_u01(seed, 3, 2 * i));
        if (syn_mix(seed, 3, 2 * i + 1) & 1ull) mag = -mag;
        uint16_t b = syn_bf16((float)mag);
        W[i] = syn_bf16_f32(b);
        coo_k[c] = (uint32_t)(i / N);
        coo_n[c] = (uint32_t)(i % N);
        coo_v[c] = b;
        ++c;
    }
    return c;
}
