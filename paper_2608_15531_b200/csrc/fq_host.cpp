// Host side of the library: layout choice, INT4 group quantiser + packer (Eq. 2, Eq. 3),
// Tile-COO encoder / decoder / validator (Section 3.2).  Plain C++, no CUDA.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

#include "fq_internal.h"

namespace fq {
char* error_buffer() {
    static thread_local char buf[512] = {0};
    return buf;
}

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40u);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}
static inline float bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

// Position of the code of (row kr, column cr) inside a 128 x BN chunk: word index and nibble.
static inline void wq_slot(uint32_t kr, uint32_t cr, uint32_t BN, uint32_t& word, uint32_t& nib) {
    const uint32_t j = kr >> 5, w = (kr >> 3) & 3, i = (kr >> 1) & 3, h = kr & 1;
    word = (j * BN + cr) * 4 + w;
    nib = i + 4 * h;
}
}  // namespace fq

using namespace fq;

extern "C" {

const char* fq_last_error(void) { return error_buffer(); }

fq_status_t fq_get_layout(uint32_t K, uint32_t N, uint32_t group, uint32_t bn_hint, uint32_t nb_hint,
                          fq_layout_t* out) {
    if (!out) return fail(FQ_ERR_INVALID_ARG, "fq_get_layout: null output");
    if (group != 64 && group != 128) return fail(FQ_ERR_UNSUPPORTED_SHAPE, "group must be 64 or 128, got %u", group);
    if (K == 0 || K % FQ_BK != 0) return fail(FQ_ERR_UNSUPPORTED_SHAPE, "K = %u is not a multiple of 128", K);
    uint32_t BN = bn_hint;
    if (BN == 0) BN = (N % 256 == 0) ? 256 : 128;
    if (BN != 128 && BN != 256) return fail(FQ_ERR_UNSUPPORTED_SHAPE, "BN must be 128 or 256, got %u", BN);
    if (N == 0 || N % BN != 0) return fail(FQ_ERR_UNSUPPORTED_SHAPE, "N = %u is not a multiple of BN = %u", N, BN);
    if (N / BN > kMaxTilesN) return fail(FQ_ERR_UNSUPPORTED_SHAPE, "N = %u has too many column tiles", N);
    // one bucket per group of four columns {g, g + 8, g + 16, g + 24} of a 32-column block
    const uint32_t NB = BN / 4;
    if (nb_hint != 0 && nb_hint != NB) return fail(FQ_ERR_UNSUPPORTED_SHAPE, "buckets per tile must be BN / 4 = %u, got %u", NB, nb_hint);
    std::memset(out, 0, sizeof(*out));
    out->abi = FQ_ABI_VERSION;
    out->K = K;
    out->N = N;
    out->group = group;
    out->BK = FQ_BK;
    out->BN = BN;
    out->buckets_per_tile = NB;
    out->wq_interleave = 3;
    out->coo_unit_bytes = 16;
    return FQ_OK;
}

// Tile column of column number j of bucket b (buckets are static: 8 * (c / 32) + c % 8).
static inline uint32_t column_of_bucket(uint32_t b, uint32_t j) { return ((b >> 3) << 5) | (b & 7u) | (j << 3); }

fq_status_t fq_pack_int4_sizes(const fq_layout_t* L, size_t* wq_bytes, size_t* scale_bytes, size_t* zero_bytes) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if (wq_bytes) *wq_bytes = (size_t)L->K * L->N / 2;
    if (scale_bytes) *scale_bytes = (size_t)(L->K / L->group) * L->N * 2;
    if (zero_bytes) *zero_bytes = (size_t)(L->K / L->group) * L->N * 2;
    return FQ_OK;
}

fq_status_t fq_pack_int4(const fq_layout_t* L, const float* W, const uint8_t* mask, void* wq_out,
                         uint16_t* scale, uint16_t* zero) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if (!W || !wq_out || !scale || !zero) return fail(FQ_ERR_INVALID_ARG, "fq_pack_int4: null pointer");
    const uint32_t K = L->K, N = L->N, g = L->group, BN = L->BN;
    const uint32_t KT = K / FQ_BK, NT = N / BN, gpc = FQ_BK / g;  // groups per chunk
    uint32_t* wq = (uint32_t*)wq_out;
    const size_t chunk_words = (size_t)16 * BN;
#pragma omp parallel
    {
        std::vector<float> wmin(BN), wmax(BN), sf(BN);
        std::vector<int> zz(BN);
#pragma omp for schedule(dynamic, 4)
        for (int64_t ch = 0; ch < (int64_t)NT * KT; ++ch) {
            const uint32_t tn = (uint32_t)(ch / KT), kt = (uint32_t)(ch % KT);
            uint32_t* chunk = wq + (size_t)ch * chunk_words;
            std::memset(chunk, 0, chunk_words * 4);
            const size_t n0 = (size_t)tn * BN;
            for (uint32_t gi = 0; gi < gpc; ++gi) {
                const uint32_t k0 = kt * FQ_BK + gi * g;
                const size_t grow = (size_t)(k0 / g);
                std::fill(wmin.begin(), wmin.end(), 0.0f);  // the range always contains 0
                std::fill(wmax.begin(), wmax.end(), 0.0f);
                for (uint32_t k = k0; k < k0 + g; ++k) {
                    const float* wr = W + (size_t)k * N + n0;
                    const uint8_t* mr = mask ? mask + (size_t)k * N + n0 : nullptr;
                    for (uint32_t c = 0; c < BN; ++c) {
                        if (mr && mr[c]) continue;
                        float w = wr[c];
                        if (w < wmin[c]) wmin[c] = w;
                        if (w > wmax[c]) wmax[c] = w;
                    }
                }
                for (uint32_t c = 0; c < BN; ++c) {
                    float s32 = (wmax[c] - wmin[c]) / 15.0f;
                    uint16_t sb = f32_to_bf16_rne(s32);
                    float s = bf16_to_f32(sb);
                    int z = 0;
                    if (!(s > 0.0f)) {  // degenerate group
                        sb = f32_to_bf16_rne(1.0f);
                        s = 0.0f;       // marks "all codes 0" below
                    } else {
                        z = (int)nearbyintf(-wmin[c] / s);
                        z = z < 0 ? 0 : (z > 15 ? 15 : z);
                    }
                    sf[c] = s;
                    zz[c] = z;
                    scale[grow * N + n0 + c] = sb;
                    zero[grow * N + n0 + c] = f32_to_bf16_rne((float)z);
                }
                for (uint32_t k = k0; k < k0 + g; ++k) {
                    const float* wr = W + (size_t)k * N + n0;
                    const uint8_t* mr = mask ? mask + (size_t)k * N + n0 : nullptr;
                    const uint32_t kr = k - kt * FQ_BK;
                    for (uint32_t c = 0; c < BN; ++c) {
                        int q;
                        if (sf[c] == 0.0f) {
                            q = 0;
                        } else if (mr && mr[c]) {
                            q = zz[c];
                        } else {
                            q = (int)nearbyintf(wr[c] / sf[c]) + zz[c];
                            q = q < 0 ? 0 : (q > 15 ? 15 : q);
                        }
                        uint32_t word, nib;
                        wq_slot(kr, c, BN, word, nib);
                        chunk[word] |= (uint32_t)q << (4 * nib);
                    }
                }
            }
        }
    }
    return FQ_OK;
}

fq_status_t fq_repurpose_pad_slots(const fq_layout_t* L, const float* W, const uint8_t* mask, uint8_t* mask_out,
                                   uint64_t* added_out) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if (!W || !mask || !mask_out) return fail(FQ_ERR_INVALID_ARG, "fq_repurpose_pad_slots: null pointer");
    const uint32_t K = L->K, N = L->N, g = L->group, BN = L->BN, NB = L->buckets_per_tile;
    const uint32_t KT = K / FQ_BK, NT = N / BN, gpc = FQ_BK / g;
    std::memcpy(mask_out, mask, (size_t)K * N);
    uint64_t added = 0;
#pragma omp parallel reduction(+ : added)
    {
        std::vector<double> err((size_t)FQ_BK * BN);          // quantisation error of every weight of the tile; < 0: not a candidate
        std::vector<uint32_t> count(BN);
        std::vector<std::pair<double, uint32_t>> cand;
#pragma omp for schedule(dynamic, 4)
        for (int64_t ch = 0; ch < (int64_t)NT * KT; ++ch) {
            const uint32_t tn = (uint32_t)(ch / KT), kt = (uint32_t)(ch % KT);
            const size_t n0 = (size_t)tn * BN;
            std::fill(count.begin(), count.end(), 0u);
            for (uint32_t gi = 0; gi < gpc; ++gi) {
                const uint32_t k0 = kt * FQ_BK + gi * g;
                for (uint32_t c = 0; c < BN; ++c) {
                    // Eq. 2 for this group and column under `mask`, as in fq_pack_int4
                    float wmin = 0.0f, wmax = 0.0f;
                    for (uint32_t k = k0; k < k0 + g; ++k) {
                        if (mask[(size_t)k * N + n0 + c]) continue;
                        const float w = W[(size_t)k * N + n0 + c];
                        wmin = std::min(wmin, w), wmax = std::max(wmax, w);
                    }
                    float s = bf16_to_f32(f32_to_bf16_rne((wmax - wmin) / 15.0f));
                    int z = 0;
                    const bool degenerate = !(s > 0.0f);
                    if (!degenerate) {
                        z = (int)nearbyintf(-wmin / s);
                        z = z < 0 ? 0 : (z > 15 ? 15 : z);
                    }
                    for (uint32_t k = k0; k < k0 + g; ++k) {
                        const size_t idx = (size_t)k * N + n0 + c;
                        const float w = W[idx];
                        const bool nonzero = (f32_to_bf16_rne(w) & 0x7fffu) != 0;
                        double e = -1.0;
                        if (mask[idx]) {
                            if (nonzero) ++count[c];
                        } else if (nonzero) {
                            int q = 0;
                            if (!degenerate) {
                                q = (int)nearbyintf(w / s) + z;
                                q = q < 0 ? 0 : (q > 15 ? 15 : q);
                            }
                            const double what = degenerate ? 0.0 : (double)s * ((double)q - (double)z);   // Eq. 3
                            e = std::fabs((double)w - what);
                        }
                        err[(size_t)(k - kt * FQ_BK) * BN + c] = e;
                    }
                }
            }
            for (uint32_t b = 0; b < NB; ++b) {
                uint32_t depth = 0;
                for (uint32_t j = 0; j < 4; ++j) depth = std::max(depth, count[column_of_bucket(b, j)]);
                if (depth > 32) continue;                      // a bucket with a tail keeps its padding
                for (uint32_t j = 0; j < 4; ++j) {
                    const uint32_t c = column_of_bucket(b, j), free_slots = depth - count[c];
                    if (!free_slots) continue;
                    cand.clear();
                    for (uint32_t r = 0; r < FQ_BK; ++r)
                        if (err[(size_t)r * BN + c] > 0.0) cand.emplace_back(err[(size_t)r * BN + c], r);
                    const size_t take = std::min<size_t>(free_slots, cand.size());
                    // larger error first, lower row first among equals
                    std::partial_sort(cand.begin(), cand.begin() + take, cand.end(),
                                      [](const std::pair<double, uint32_t>& x, const std::pair<double, uint32_t>& y) {
                                          return x.first != y.first ? x.first > y.first : x.second < y.second;
                                      });
                    for (size_t i = 0; i < take; ++i) mask_out[(size_t)(kt * FQ_BK + cand[i].second) * N + n0 + c] = 1;
                    added += take;
                }
            }
        }
    }
    if (added_out) *added_out = added;
    return FQ_OK;
}

fq_status_t fq_unpack_int4(const fq_layout_t* L, const void* wq_in, uint8_t* q) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if (!wq_in || !q) return fail(FQ_ERR_INVALID_ARG, "fq_unpack_int4: null pointer");
    const uint32_t K = L->K, N = L->N, BN = L->BN, KT = K / FQ_BK, NT = N / BN;
    const uint32_t* wq = (const uint32_t*)wq_in;
#pragma omp parallel for schedule(static)
    for (int64_t ch = 0; ch < (int64_t)NT * KT; ++ch) {
        const uint32_t tn = (uint32_t)(ch / KT), kt = (uint32_t)(ch % KT);
        const uint32_t* chunk = wq + (size_t)ch * 16 * BN;
        for (uint32_t kr = 0; kr < FQ_BK; ++kr)
            for (uint32_t c = 0; c < BN; ++c) {
                uint32_t word, nib;
                wq_slot(kr, c, BN, word, nib);
                q[(size_t)(kt * FQ_BK + kr) * N + (size_t)tn * BN + c] = (uint8_t)((chunk[word] >> (4 * nib)) & 0xf);
            }
    }
    return FQ_OK;
}

}  // extern "C"

// ------------------------------------------------------------------ Tile-COO encoder

namespace {

struct Entry {
    uint8_t k, c;
    uint32_t v;      // the slot's 19 value bits
};

struct Encoded {
    std::vector<uint32_t> indptr;   // N_tile + 1
    std::vector<uint32_t> info;     // N_tile * NB
    std::vector<uint32_t> words;    // 4 * n_packets
    uint32_t max_tile_packets = 0;
    uint32_t max_bucket_packets = 0;
    uint32_t max_tail_packets = 0;
};

// Bucket of a tile column: the four columns {g, g + 8, g + 16, g + 24} of a 32-column block share
// bucket 8 * (c / 32) + c % 8.  These are the columns whose accumulators one group of four lanes
// holds in the kernels, so a bucket's outliers are applied in registers.
inline uint32_t bucket_of(uint32_t c) { return ((c >> 5) << 3) | (c & 7u); }
// Number of a column inside its bucket, and the way back.
inline uint32_t number_in_bucket(uint32_t c) { return (c >> 3) & 3u; }
inline uint32_t column_of(uint32_t b, uint32_t j) { return ((b >> 3) << 5) | (b & 7u) | (j << 3); }

// One outlier as a 32-bit word: the 19 value bits from bit 13 up, row * 32 in bits 5-11, the column's number
// inside the bucket in bits 3-4.
inline uint32_t entry_word(uint32_t k, uint32_t j, uint32_t v19) { return (v19 << fq::kSlotValueShift) | (j << fq::kSlotColShift) | (k << 5); }

// IEEE binary16 bits -> the FP32 number's bits (every binary16 number is an FP32 number with at most ten fraction
// bits), and back (exact for such numbers; `ok` says whether it was one).
inline uint32_t f16_to_f32_bits(uint16_t h) {
    const uint32_t sign = (uint32_t)(h & 0x8000u) << 16, e = (h >> 10) & 31u, f = h & 1023u;
    if (e == 31) return sign | 0x7f800000u | (f << 13);
    if (e != 0) return sign | ((e + 112u) << 23) | (f << 13);
    if (f == 0) return sign;
    int shift = 0;
    uint32_t m = f;
    while (!(m & 1024u)) m <<= 1, ++shift;                 // normalise the subnormal
    return sign | ((uint32_t)(113 - shift) << 23) | ((m & 1023u) << 13);
}
inline uint16_t f32_bits_to_f16(uint32_t u, bool* ok) {
    const uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    const int e = (int)((u >> 23) & 255u) - 127;
    const uint32_t f = u & 0x7fffffu;
    uint16_t h;
    if (((u >> 23) & 255u) == 255u) h = (uint16_t)(sign | 0x7c00u | (f >> 13));
    else if ((u & 0x7fffffffu) == 0) h = sign;
    else if (e >= -14 && e <= 15) h = (uint16_t)(sign | ((uint32_t)(e + 15) << 10) | (f >> 13));
    else if (e >= -24 && e < -14) h = (uint16_t)(sign | ((0x800000u | f) >> (13 + (-14 - e))));
    else h = (uint16_t)(sign | 0x7c00u);                   // out of range
    *ok = f16_to_f32_bits(h) == u;
    return h;
}
// The caller's 16 value bits as the slot's 19 value bits, and back.
inline uint32_t value_field(uint16_t v, uint32_t value_type) {
    return value_type == FQ_VALUE_FP16 ? f16_to_f32_bits(v) >> fq::kSlotValueShift : (uint32_t)v << 3;
}

// A column with more entries than this in one tile gives its bucket a tail.
constexpr uint32_t kSlottedMax = 32;
// Column-slotted packets of a bucket that has a tail.
constexpr uint32_t kSlottedWithTail = 4;

fq_status_t encode_impl(const fq_layout_t* L, const uint32_t* k, const uint32_t* n, const uint16_t* v,
                        size_t nnz, Encoded& E) {
    const uint32_t K = L->K, N = L->N, BN = L->BN, NB = L->buckets_per_tile;
    const uint32_t KT = K / FQ_BK, NT = N / BN;
    const size_t ntile = (size_t)KT * NT;
    // counting sort of the entries by tile
    std::vector<size_t> tstart(ntile + 1, 0);
    for (size_t e = 0; e < nnz; ++e) {
        if (k[e] >= K || n[e] >= N) return fq::fail(FQ_ERR_INVALID_ARG, "outlier %zu at (%u, %u) is outside the %u x %u matrix", e, k[e], n[e], K, N);
        if ((v[e] & 0x7fffu) == 0) continue;  // +-0 is not an outlier
        size_t t = (size_t)(n[e] / BN) * KT + k[e] / FQ_BK;
        ++tstart[t + 1];
    }
    for (size_t t = 0; t < ntile; ++t) tstart[t + 1] += tstart[t];
    std::vector<Entry> sorted(tstart[ntile]);
    {
        std::vector<size_t> fill(tstart.begin(), tstart.end() - 1);
        for (size_t e = 0; e < nnz; ++e) {
            if ((v[e] & 0x7fffu) == 0) continue;
            size_t t = (size_t)(n[e] / BN) * KT + k[e] / FQ_BK;
            sorted[fill[t]++] = Entry{(uint8_t)(k[e] % FQ_BK), (uint8_t)(n[e] % BN), value_field(v[e], L->value_type)};
        }
    }
    // pass 1: per tile and bucket, the column-slotted packets (packet i = entry i of each of the
    // four columns, by row) and, for a bucket with a long column, the tail (the entries beyond each
    // column's first kSlottedWithTail, by (row, column), four to a packet)
    E.indptr.assign(ntile + 1, 0);
    E.info.assign(ntile * NB, 0);
    std::vector<std::vector<uint32_t>> tile_words(ntile);
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t t = 0; t < (int64_t)ntile; ++t) {
        std::vector<std::vector<Entry>> per(NB * 4);      // by (bucket, number in bucket)
        for (size_t e = tstart[t]; e < tstart[t + 1]; ++e)
            per[bucket_of(sorted[e].c) * 4 + number_in_bucket(sorted[e].c)].push_back(sorted[e]);
        std::vector<uint32_t>& tw = tile_words[t];
        // depth of every bucket: its longest column, or kSlottedWithTail when that column is too long
        std::vector<uint32_t> depths(NB);
        for (uint32_t b = 0; b < NB; ++b) {
            size_t longest = 0;
            for (uint32_t j = 0; j < 4; ++j) {
                std::vector<Entry>& col = per[b * 4 + j];
                std::sort(col.begin(), col.end(), [](const Entry& x, const Entry& y) { return x.k < y.k; });
                longest = std::max(longest, col.size());
            }
            depths[b] = longest > kSlottedMax ? kSlottedWithTail : (uint32_t)longest;
        }
        // Which of its column-slotted packets holds which of a column's outliers is free (the sum is
        // order-independent up to rounding).  By row: packet i holds the column's i-th.  Bank-aware (Section
        // 3.2.2's element reordering, restated for a k-major FP32 copy of eight activation rows, 32 B per row,
        // where rows with equal k mod 4 share banks): one load instruction of a warp reads slot j of packet d of
        // its eight buckets and is served half a warp, i.e. four neighbouring buckets, at a time, in as many
        // passes as the fullest bank group has different rows.  So for every four neighbouring buckets, slot j
        // and packet number d in turn, the rows are chosen among what the four columns still have to place (or
        // padding, row 0, where a column has places to spare) such that the passes are fewest.
        std::vector<std::vector<uint32_t>> place(NB * 4);          // [bucket * 4 + j][d] -> index into the column + 1, 0 = padding
        for (uint32_t b = 0; b < NB; ++b)
            for (uint32_t j = 0; j < 4; ++j) place[b * 4 + j].assign(depths[b], 0);
        if (L->slot_order == 1) {
            for (uint32_t c = 0; c < NB * 4; ++c)
                for (uint32_t d = 0; d < std::min<size_t>(per[c].size(), place[c].size()); ++d) place[c][d] = d + 1;
        } else {
            for (uint32_t b0 = 0; b0 < NB; b0 += 4)
                for (uint32_t j = 0; j < 4; ++j) {
                    uint32_t dmax = 0;
                    std::vector<uint8_t> used[4];
                    uint32_t todo[4];
                    for (uint32_t q = 0; q < 4; ++q) {
                        const uint32_t c = (b0 + q) * 4 + j;
                        todo[q] = (uint32_t)std::min<size_t>(per[c].size(), depths[b0 + q]);
                        used[q].assign(todo[q], 0);
                        dmax = std::max(dmax, depths[b0 + q]);
                    }
                    for (uint32_t d = 0; d < dmax; ++d) {
                        // candidates per bucket: up to four unplaced outliers (lowest rows first), padding if the
                        // column has a place to spare; a bucket whose list has ended reads row 0 whatever happens
                        int cand[4][5], ncand[4];
                        for (uint32_t q = 0; q < 4; ++q) {
                            ncand[q] = 0;
                            if (d >= depths[b0 + q]) { cand[q][ncand[q]++] = -1; continue; }
                            for (uint32_t e = 0; e < used[q].size() && ncand[q] < 4; ++e)
                                if (!used[q][e]) cand[q][ncand[q]++] = (int)e;
                            if (todo[q] < depths[b0 + q] - d) cand[q][ncand[q]++] = -1;
                        }
                        int best[4] = {cand[0][0], cand[1][0], cand[2][0], cand[3][0]};
                        uint32_t best_cost = 1u << 30;
                        int pick[4];
                        for (int i0 = 0; i0 < ncand[0]; ++i0)
                            for (int i1 = 0; i1 < ncand[1]; ++i1)
                                for (int i2 = 0; i2 < ncand[2]; ++i2)
                                    for (int i3 = 0; i3 < ncand[3]; ++i3) {
                                        pick[0] = cand[0][i0], pick[1] = cand[1][i1], pick[2] = cand[2][i2], pick[3] = cand[3][i3];
                                        uint32_t rows[4], passes = 0, pads = 0;
                                        for (uint32_t q = 0; q < 4; ++q) {
                                            rows[q] = pick[q] < 0 ? 0u : per[(b0 + q) * 4 + j][pick[q]].k;
                                            pads += pick[q] < 0 && d < depths[b0 + q];
                                        }
                                        for (uint32_t cls = 0; cls < 4; ++cls) {
                                            uint32_t n = 0;
                                            for (uint32_t q = 0; q < 4; ++q) {
                                                if ((rows[q] & 3u) != cls) continue;
                                                bool seen = false;
                                                for (uint32_t r = 0; r < q; ++r) seen |= rows[r] == rows[q];
                                                n += !seen;
                                            }
                                            passes = std::max(passes, n);
                                        }
                                        // fewest passes; then fewest paddings (outliers placed early leave later
                                        // packets more freedom); then the first combination found (lowest rows)
                                        const uint32_t cost = passes * 16 + pads;
                                        if (cost < best_cost) { best_cost = cost; for (int q = 0; q < 4; ++q) best[q] = pick[q]; }
                                    }
                        for (uint32_t q = 0; q < 4; ++q)
                            if (best[q] >= 0) { place[(b0 + q) * 4 + j][d] = (uint32_t)best[q] + 1; used[q][best[q]] = 1; --todo[q]; }
                    }
                }
        }
        uint32_t off = 0;
        for (uint32_t b = 0; b < NB; ++b) {
            const uint32_t depth = depths[b];
            for (uint32_t d = 0; d < depth; ++d)
                for (uint32_t j = 0; j < 4; ++j) {
                    const std::vector<Entry>& col = per[b * 4 + j];
                    const uint32_t e = place[b * 4 + j][d];
                    tw.push_back(e ? entry_word(col[e - 1].k, j, col[e - 1].v) : entry_word(0, j, 0));
                }
            std::vector<Entry> rest;
            for (uint32_t j = 0; j < 4; ++j) {
                const std::vector<Entry>& col = per[b * 4 + j];
                if (col.size() > depth) rest.insert(rest.end(), col.begin() + depth, col.end());
            }
            std::sort(rest.begin(), rest.end(), [](const Entry& x, const Entry& y) {
                return x.k != y.k ? x.k < y.k : x.c < y.c;
            });
            const uint32_t tail = (uint32_t)((rest.size() + 3) / 4);
            for (const Entry& e : rest) tw.push_back(entry_word(e.k, number_in_bucket(e.c), e.v));
            for (size_t i = rest.size(); i < (size_t)tail * 4; ++i) tw.push_back(0);
            if (off > 0xffffu || depth > 0xffu || tail > 0xffu) {
#pragma omp atomic write
                bad = 1;
            }
            E.info[(size_t)t * NB + b] = (off & 0xffffu) | (depth << 16) | (tail << 24);
            off += depth + tail;
        }
        E.indptr[t + 1] = off;
    }
    if (bad) return fq::fail(FQ_ERR_UNSUPPORTED_SHAPE, "a bucket exceeds the packet offset/count range of its descriptor");
    for (size_t i = 0; i < E.info.size(); ++i) {
        const uint32_t depth = (E.info[i] >> 16) & 0xffu, tail = E.info[i] >> 24;
        E.max_bucket_packets = std::max(E.max_bucket_packets, depth + tail);
        E.max_tail_packets = std::max(E.max_tail_packets, tail);
    }
    uint64_t total = 0;
    for (size_t t = 0; t < ntile; ++t) {
        uint32_t c = E.indptr[t + 1];
        E.max_tile_packets = std::max(E.max_tile_packets, c);
        total += c;
        if (total > 0xffffffffull) return fq::fail(FQ_ERR_UNSUPPORTED_SHAPE, "more than 2^32 packets");
        E.indptr[t + 1] = (uint32_t)total;
    }
    E.words.assign((size_t)total * 4, 0);
    // pass 2: the tiles' packets one after the other
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t t = 0; t < (int64_t)ntile; ++t)
        if (!tile_words[t].empty())
            std::memcpy(&E.words[(size_t)E.indptr[t] * 4], tile_words[t].data(), tile_words[t].size() * 4);
    return FQ_OK;
}

}  // namespace

extern "C" {

fq_status_t fq_encode_tilecoo_sizes(const fq_layout_t* L, const uint32_t* k, const uint32_t* n,
                                    const uint16_t* v, size_t nnz, size_t* n_indptr, size_t* n_bucket_info,
                                    size_t* n_packets, uint32_t* max_tile_packets) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if (nnz && (!k || !n || !v)) return fail(FQ_ERR_INVALID_ARG, "fq_encode_tilecoo_sizes: null pointer");
    Encoded E;
    fq_status_t st = encode_impl(L, k, n, v, nnz, E);
    if (st != FQ_OK) return st;
    if (n_indptr) *n_indptr = E.indptr.size();
    if (n_bucket_info) *n_bucket_info = E.info.size();
    if (n_packets) *n_packets = E.words.size() / 4;
    if (max_tile_packets) *max_tile_packets = E.max_tile_packets;
    return FQ_OK;
}

fq_status_t fq_encode_tilecoo(fq_layout_t* L, const uint32_t* k, const uint32_t* n, const uint16_t* v,
                              size_t nnz, uint32_t* tile_indptr, uint32_t* bucket_info, void* packed,
                              size_t n_packets) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if ((nnz && (!k || !n || !v)) || !tile_indptr || !bucket_info) return fail(FQ_ERR_INVALID_ARG, "fq_encode_tilecoo: null pointer");
    Encoded E;
    fq_status_t st = encode_impl(L, k, n, v, nnz, E);
    if (st != FQ_OK) return st;
    if (E.words.size() / 4 > n_packets) return fail(FQ_ERR_BUFFER_TOO_SMALL, "packed_outliers holds %zu packets, %zu needed", n_packets, E.words.size() / 4);
    if (!E.words.empty() && !packed) return fail(FQ_ERR_INVALID_ARG, "fq_encode_tilecoo: null packet buffer");
    std::memcpy(tile_indptr, E.indptr.data(), E.indptr.size() * 4);
    std::memcpy(bucket_info, E.info.data(), E.info.size() * 4);
    if (!E.words.empty()) std::memcpy(packed, E.words.data(), E.words.size() * 4);
    L->max_tile_packets = E.max_tile_packets;
    L->max_bucket_packets = E.max_bucket_packets;
    L->max_tail_packets = E.max_tail_packets;
    L->tilecoo_encoded = 1;
    return FQ_OK;
}

fq_status_t fq_decode_tilecoo(const fq_layout_t* L, const uint32_t* indptr, const uint32_t* info,
                              const void* packed, uint32_t* k, uint32_t* n, uint16_t* v, size_t* nnz_inout) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if (!indptr || !info || !nnz_inout) return fail(FQ_ERR_INVALID_ARG, "fq_decode_tilecoo: null pointer");
    const uint32_t BN = L->BN, NB = L->buckets_per_tile, KT = L->K / FQ_BK, NT = L->N / BN;
    const uint32_t* pw = (const uint32_t*)packed;
    const size_t cap = *nnz_inout;
    size_t c = 0;
    for (uint32_t tn = 0; tn < NT; ++tn)
        for (uint32_t kt = 0; kt < KT; ++kt) {
            size_t t = (size_t)tn * KT + kt;
            for (uint32_t b = 0; b < NB; ++b) {
                const uint32_t inf = info[t * NB + b];
                const size_t i0 = (size_t)indptr[t] + (inf & 0xffffu), cnt = ((inf >> 16) & 0xffu) + (inf >> 24);
                for (size_t i = 0; i < cnt * 4; ++i) {
                    const uint32_t w = pw[i0 * 4 + i];
                    if ((w & fq::kSlotValueMask) == 0) continue;
                    if (c >= cap) return fail(FQ_ERR_BUFFER_TOO_SMALL, "decode buffer holds %zu entries", cap);
                    k[c] = kt * FQ_BK + ((w >> 5) & 127u);
                    n[c] = tn * BN + column_of(b, (w >> fq::kSlotColShift) & 3u);
                    if (L->value_type == FQ_VALUE_FP16) {
                        bool ok = true;
                        v[c] = f32_bits_to_f16(w & fq::kSlotValueMask, &ok);
                        if (!ok) return fail(FQ_ERR_FORMAT, "a value of tile %zu is not an IEEE binary16 number", t);
                    } else {
                        if (w & 0xe000u) return fail(FQ_ERR_FORMAT, "a value of tile %zu is not a BF16 number", t);
                        v[c] = (uint16_t)(w >> 16);
                    }
                    ++c;
                }
            }
        }
    *nnz_inout = c;
    return FQ_OK;
}

fq_status_t fq_validate_tilecoo(const fq_layout_t* L, const uint32_t* indptr, const uint32_t* info,
                                const void* packed, size_t n_packets) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if (!indptr || !info || (n_packets && !packed)) return fail(FQ_ERR_INVALID_ARG, "fq_validate_tilecoo: null pointer");
    const uint32_t BN = L->BN, NB = L->buckets_per_tile;
    const size_t ntile = (size_t)(L->K / FQ_BK) * (L->N / BN);
    const uint32_t* pw = (const uint32_t*)packed;
    if (indptr[0] != 0) return fail(FQ_ERR_FORMAT, "tile_indptr[0] = %u, expected 0", indptr[0]);
    for (size_t t = 0; t < ntile; ++t) {
        if (indptr[t + 1] < indptr[t]) return fail(FQ_ERR_FORMAT, "tile_indptr decreases at tile %zu", t);
        const uint32_t tile_pk = indptr[t + 1] - indptr[t];
        if ((size_t)indptr[t + 1] > n_packets) return fail(FQ_ERR_FORMAT, "tile %zu ends at packet %u of %zu", t, indptr[t + 1], n_packets);
        for (uint32_t b = 0; b < NB; ++b) {
            const uint32_t inf = info[t * NB + b];
            const uint32_t off = inf & 0xffffu, depth = (inf >> 16) & 0xffu, tail = inf >> 24;
            if (off + depth + tail > tile_pk) return fail(FQ_ERR_FORMAT, "bucket %u of tile %zu covers packets [%u, %u) of %u", b, t, off, off + depth + tail, tile_pk);
            if (depth > kSlottedMax) return fail(FQ_ERR_FORMAT, "bucket %u of tile %zu has %u column-slotted packets, at most %u allowed", b, t, depth, kSlottedMax);
            for (uint32_t i = 0; i < (depth + tail) * 4; ++i) {
                const uint32_t w = pw[((size_t)indptr[t] + off) * 4 + i];
                if (L->value_type == FQ_VALUE_FP16) {
                    bool ok = true;
                    f32_bits_to_f16(w & fq::kSlotValueMask, &ok);
                    if (!ok) return fail(FQ_ERR_FORMAT, "a value in bucket %u of tile %zu is not an IEEE binary16 number", b, t);
                } else if (w & 0xe000u) {
                    return fail(FQ_ERR_FORMAT, "a value in bucket %u of tile %zu is not a BF16 number", b, t);
                }
                if (w & fq::kSlotStrayMask) return fail(FQ_ERR_FORMAT, "bits outside the fields are set in a slot of bucket %u, tile %zu", b, t);
                if (i < depth * 4 && ((w >> fq::kSlotColShift) & 3u) != (i & 3u))
                    return fail(FQ_ERR_FORMAT, "slot %u of a column-slotted packet of bucket %u, tile %zu, names column number %u", i & 3u, b, t, (w >> fq::kSlotColShift) & 3u);
            }
        }
    }
    if ((size_t)indptr[ntile] != n_packets) return fail(FQ_ERR_FORMAT, "tile_indptr ends at %u, %zu packets given", indptr[ntile], n_packets);
    return FQ_OK;
}

}  // extern "C"
