// The fused operator for short jobs: one CTA per strip of 32 output columns, the k-steps of the strip dealt
// out over the CTA's warps, the weights read straight from global memory into registers.
// Included by fq_kernels.cu inside namespace fq, after fq_mma_kernel.cuh (same MMA helper, same packed formats).
//
// A layer whose column tiles are few is a short job for every CTA of the streaming kernel: three or four
// units, then a round trip through the scratch (or a cluster barrier) to add up the parts of a split tile.
// Here no tile is split over CTAs: warp w of the strip's CTA takes k-steps w, w + W, ..., and the W partial
// sums of the strip meet in shared memory at the end (Section 3.1.1's split-K, kept inside the CTA).  There is
// no ring, no barrier object and no producer: a warp requests the 2 KB of codes, the scales, zero-points, bucket
// descriptor and its slots of the first eight packets of its k-step before it waits for the grid before it (all
// weights), then copies its block of activations into shared memory (cp.async), and the other warps' requests
// keep the memory system busy while it computes.
//   dense:    lane (g, t) holds word t (rows 8t..8t+7 of each 32-row block) of columns g, g+8, g+16, g+24 of
//             the strip; exact integers 128 + q as BF16 into mma.sync m16n8k16, the batch on the N side, the
//             activations as 16-byte fragments from the warp's shared-memory rows; per group
//             acc += s * (sum_k x (128+q) - (128+z) sum_k x)                     (Eq. 3 inside Eq. 1)
//             with sum_k x from one more MMA whose weight operand is all ones.
//   outliers: the lane's four columns are one Tile-COO bucket (Section 4.2 without the shared-memory scatter).
//             Up to 8 rows (MS = 1, 4, 8 rows kept): lane (g, t) takes slot t of every packet, i.e. column
//             g + 8t, for all rows, from a k-major copy of the warp's activations, into sums of its own that move
//             into the MMA fragment layout once, after the last k-step.  16 rows (MS = 16): the lane takes all four
//             slots for its own fragment rows.  Tail packets (slots name their column) are read when met.
struct DirectParams {
    const uint16_t* X;
    const uint8_t* wq;
    const uint16_t* scale;
    const uint16_t* zero;
    const uint32_t* indptr;
    const uint32_t* info;
    const uint4* packed;
    uint16_t* Y;
    uint32_t* status;
    uint32_t M, K, N, KT, BN, NB;
};

__device__ __forceinline__ void cp_async_16(uint32_t dst_smem, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_4(uint32_t dst_smem, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

constexpr int kDirectSlots = 8;     // packets of a bucket that are requested with the weights
// bytes of shared memory a warp of the direct kernel owns: rows of X, k-major copy, scale and zero rows, packets
constexpr int kDirectWarpBytes = 16 * 256 + 256 + 8 * kDirectSlots * 16;

template <int MO, int MS, int GROUP, bool SPARSE, int WARPS>
__global__ void __launch_bounds__(32 * WARPS, (MO == 1 && WARPS == 16) ? 2 : 1) fq_direct_kernel(const DirectParams p) {
    constexpr int CG = 2, GPS = kBK / GROUP, NV = MO * CG * 4;
    // Shared memory, per warp: its block of activations, 8 MO rows of 256 B (16-byte chunk c of an odd row at
    // c ^ 4, so that the fragment loads of a quarter warp touch every bank once); (MS = 4, 8) the k-major BF16
    // copy [k][8]; the strip's scale and zero-point rows of the k-step (64 B each per group); the first eight
    // packets of the warp's eight buckets (packet d of bucket g at position d ^ g, so that the eight lane groups
    // read different banks).  After the last k-step the same bytes hold the warps' sums, [WARPS][NV + R][32] FP32.
    extern __shared__ __align__(16) float red[];
    constexpr bool kMajor = SPARSE && (MS == 4 || MS == 8);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    uint8_t* xrow_s = reinterpret_cast<uint8_t*>(red) + warp * kDirectWarpBytes;
    uint8_t* xk8 = xrow_s + 8 * 256;                                // MO == 1 only (two octets of rows fill these bytes)
    uint8_t* szs = xrow_s + 16 * 256;
    uint8_t* pks = szs + 256;
    const uint32_t strip = blockIdx.x, spt = p.BN / 32, tn = strip / spt, dw = strip - tn * spt;
    const uint32_t KT = p.KT, BN = p.BN;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    float accf[MO][CG][4];
#pragma unroll
    for (int o = 0; o < MO; ++o)
#pragma unroll
        for (int cg = 0; cg < CG; ++cg)
#pragma unroll
            for (int i = 0; i < 4; ++i) accf[o][cg][i] = 0.0f;
    constexpr int R = MS == 16 ? 1 : MS;
    float sacc[R];                                                  // column-per-lane outlier sums
#pragma unroll
    for (int r = 0; r < R; ++r) sacc[r] = 0.0f;

    bool waited = false;
    for (uint32_t kt = warp; kt < KT; kt += WARPS) {
        const size_t u = (size_t)tn * KT + kt;
        // ---- weights of the k-step, all requested before the first is used (the bucket descriptor first: the
        // packets can only be requested once it is here)
        uint32_t inf = 0, a = 0, b = 0;
        if (SPARSE) {
            inf = __ldg(p.info + u * p.NB + dw * 8 + g);
            a = __ldg(p.indptr + u), b = __ldg(p.indptr + u + 1);
        }
        const uint32_t* wp = reinterpret_cast<const uint32_t*>(p.wq + u * (size_t)(16 * BN * 4)) + (dw * 32 + g) * 4 + t;
        uint32_t wr[4][4];                                          // [block j][column g + 8 i]
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int i = 0; i < 4; ++i) wr[j][i] = __ldg(wp + j * BN * 4 + i * 32);
        __syncwarp();                                               // the previous k-step's readers are done
#pragma unroll
        for (int gi = 0; gi < GPS; ++gi) {
            // lanes 0-15: the strip's 32 scales of this group, two per lane; lanes 16-31: its zero-points
            const uint16_t* row = (lane < 16 ? p.scale : p.zero) + (size_t)(kt * GPS + gi) * p.N + (size_t)strip * 32 + 2 * (lane & 15);
            cp_async_4(smem_u32(szs + gi * 128 + lane * 4), row);
        }
        // outliers: packets t and t + 4 of the lane group's bucket, as far as it has them
        uint32_t sp_first = 0, sp_depth = 0, sp_tail = 0;
        if (SPARSE) {
            sp_first = a + (inf & 0xffffu), sp_depth = (inf >> 16) & 0xffu, sp_tail = inf >> 24;
            if (sp_first + sp_depth + sp_tail > b) {
                // a descriptor that does not belong to these packets: report it and skip the bucket
                atomicExch(p.status, (uint32_t)FQ_ERR_FORMAT);
                sp_depth = 0, sp_tail = 0;
            }
            const uint32_t n = sp_depth + sp_tail;
#pragma unroll
            for (int h = 0; h < kDirectSlots / 4; ++h) {
                const uint32_t d = t + 4 * h;
                if (d < n) cp_async_16(smem_u32(pks + g * (kDirectSlots * 16) + ((d ^ g) & (kDirectSlots - 1)) * 16), p.packed + sp_first + d);
            }
        }
        if (!waited) {
            // everything above is weights; the activations may come from the grid before this one
            asm volatile("griddepcontrol.wait;" ::: "memory");
            waited = true;
        }
        // ---- this k-step's block of X into the warp's rows (rows beyond M are zero)
#pragma unroll
        for (int o = 0; o < MO; ++o)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t m = 8 * o + g, chunk = (4 * j + t) ^ ((g & 1) << 2);
                uint8_t* dst = xrow_s + m * 256 + chunk * 16;
                if (m < p.M) cp_async_16(smem_u32(dst), p.X + (size_t)m * p.K + (size_t)kt * kBK + 32 * j + 8 * t);
                else *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
            }
        cp_async_wait_all();
        __syncwarp();
        // ---- dense
        const uint8_t* xfrag = xrow_s + g * 256 + t * 16;           // chunk 4j + t of row g: 64 B on for even j, back for odd
        const uint8_t* xf_e = xfrag + ((g & 1) << 6);
        const uint8_t* xf_o = xfrag - ((g & 1) << 6);
#pragma unroll
        for (int gi = 0; gi < GPS; ++gi) {
            float accg[MO][CG][4], ones[MO][4];
#pragma unroll
            for (int o = 0; o < MO; ++o) {
#pragma unroll
                for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                    for (int i = 0; i < 4; ++i) accg[o][cg][i] = 0.0f;
#pragma unroll
                for (int i = 0; i < 4; ++i) ones[o][i] = 0.0f;
            }
#pragma unroll
            for (int j = gi * (4 / GPS); j < (gi + 1) * (4 / GPS); ++j) {
                uint4 xb[MO];
#pragma unroll
                for (int o = 0; o < MO; ++o) xb[o] = *reinterpret_cast<const uint4*>(((j & 1) ? xf_o : xf_e) + o * 8 * 256 + j * 64);
#pragma unroll
                for (int cg = 0; cg < CG; ++cg) {
                    const uint32_t wa = wr[j][2 * cg], wb = wr[j][2 * cg + 1];
                    const uint32_t a0 = codes_to_bf16x2(wa), a1 = codes_to_bf16x2(wa >> 4);
                    const uint32_t a2 = codes_to_bf16x2(wa >> 8), a3 = codes_to_bf16x2(wa >> 12);
                    const uint32_t b0 = codes_to_bf16x2(wb), b1 = codes_to_bf16x2(wb >> 4);
                    const uint32_t b2 = codes_to_bf16x2(wb >> 8), b3 = codes_to_bf16x2(wb >> 12);
#pragma unroll
                    for (int o = 0; o < MO; ++o) {
                        mma_bf16(accg[o][cg], a0, b0, a1, b1, xb[o].x, xb[o].y);
                        mma_bf16(accg[o][cg], a2, b2, a3, b3, xb[o].z, xb[o].w);
                    }
                }
                constexpr uint32_t kOne = 0x3f803f80u;              // BF16 1.0 twice: the MMA then sums the activations
#pragma unroll
                for (int o = 0; o < MO; ++o) {
                    mma_bf16(ones[o], kOne, kOne, kOne, kOne, xb[o].x, xb[o].y);
                    mma_bf16(ones[o], kOne, kOne, kOne, kOne, xb[o].z, xb[o].w);
                }
            }
#pragma unroll
            for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint16_t* szr = reinterpret_cast<const uint16_t*>(szs) + gi * 64 + g + 16 * cg + 8 * h;
                    const float sv = bf16_bits_to_float(szr[0]);
                    const float zc = -(128.0f + bf16_bits_to_float(szr[32]));
#pragma unroll
                    for (int o = 0; o < MO; ++o) {
                        accf[o][cg][2 * h + 0] = fmaf(sv, fmaf(zc, ones[o][0], accg[o][cg][2 * h + 0]), accf[o][cg][2 * h + 0]);
                        accf[o][cg][2 * h + 1] = fmaf(sv, fmaf(zc, ones[o][1], accg[o][cg][2 * h + 1]), accf[o][cg][2 * h + 1]);
                    }
                }
        }
        // ---- outliers of the lane group's bucket
        if constexpr (SPARSE && MS != 16) {
            if constexpr (kMajor) {
                // k-major copy [k][8] of the eight rows (BF16), by 8 x 8 transposes: thread T of a transpose
                // holds rows 2 (T % 4), 2 (T % 4) + 1 of column k = 8 block + T / 4
#pragma unroll
                for (int kb = 0; kb < 4; ++kb) {
                    uint32_t r4[4];
                    const uint32_t chunk = (kb * 4 + (lane >> 3)) ^ (((uint32_t)lane & 1u) << 2);
                    ldmatrix_x4_trans(smem_u32(xrow_s) + (lane & 7) * 256 + chunk * 16, r4[0], r4[1], r4[2], r4[3]);
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        *reinterpret_cast<uint32_t*>(xk8 + (kb * 32 + i * 8 + (lane >> 2)) * 16 + (lane & 3) * 4) = r4[i];
                }
                __syncwarp();
            }
            auto add_mine = [&](const uint32_t w) {
                const float v = __uint_as_float(w & kSlotValueMask);
                const uint32_t k = (w >> 5) & 127u;
                if constexpr (MS == 1) {
                    sacc[0] = fmaf(v, bf16_bits_to_float(reinterpret_cast<const uint16_t*>(xrow_s)[k]), sacc[0]);
                } else if constexpr (MS == 4) {
                    const uint2 q = *reinterpret_cast<const uint2*>(xk8 + k * 16);
                    sacc[0] = fmaf(v, bf16lo(q.x), sacc[0]); sacc[1] = fmaf(v, bf16hi(q.x), sacc[1]);
                    sacc[2] = fmaf(v, bf16lo(q.y), sacc[2]); sacc[3] = fmaf(v, bf16hi(q.y), sacc[3]);
                } else {
                    const uint4 q = *reinterpret_cast<const uint4*>(xk8 + k * 16);
                    sacc[0] = fmaf(v, bf16lo(q.x), sacc[0]); sacc[1] = fmaf(v, bf16hi(q.x), sacc[1]);
                    sacc[2] = fmaf(v, bf16lo(q.y), sacc[2]); sacc[3] = fmaf(v, bf16hi(q.y), sacc[3]);
                    sacc[4] = fmaf(v, bf16lo(q.z), sacc[4]); sacc[5] = fmaf(v, bf16hi(q.z), sacc[5]);
                    sacc[6] = fmaf(v, bf16lo(q.w), sacc[6]); sacc[7] = fmaf(v, bf16hi(q.w), sacc[7]);
                }
            };
            // the lane's slot of the staged packets, as far as the longest list of the warp goes (a lane past its
            // own list adds padding: value 0, k = 0), then the rare rest from global memory
            const uint32_t dmax = __reduce_max_sync(0xffffffffu, sp_depth);
            const uint8_t* myp = pks + g * (kDirectSlots * 16) + t * 4;
#pragma unroll
            for (int d = 0; d < kDirectSlots; ++d)
                if ((uint32_t)d < dmax) add_mine((uint32_t)d < sp_depth ? *reinterpret_cast<const uint32_t*>(myp + ((d ^ g) & (kDirectSlots - 1)) * 16) : 0u);
            const uint32_t* slot = reinterpret_cast<const uint32_t*>(p.packed + sp_first) + t;
            for (uint32_t d = kDirectSlots; d < sp_depth; ++d) add_mine(__ldg(slot + 4 * d));
            for (uint32_t d = sp_depth; d < sp_depth + sp_tail; ++d) {      // tail: every slot that names this lane's column
                const uint4 q = d < (uint32_t)kDirectSlots ? *reinterpret_cast<const uint4*>(pks + g * (kDirectSlots * 16) + ((d ^ g) & (kDirectSlots - 1)) * 16)
                                                           : __ldg(p.packed + sp_first + d);
                const uint32_t wd[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (((wd[e] >> kSlotColShift) & 3u) == (uint32_t)t) add_mine(wd[e]);
            }
        }
        if constexpr (SPARSE && MS == 16) {
            auto add_slot = [&](const uint32_t w, const int i) {
                const float v = __uint_as_float(w & kSlotValueMask);
                const uint32_t k = (w >> 5) & 127u;
#pragma unroll
                for (int o = 0; o < MO; ++o)
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        const uint32_t m = 8 * o + 2 * t + r;       // the row's parity is r: chunk k / 8 sits at (k / 8) ^ 4 r
                        const uint16_t xbits = *reinterpret_cast<const uint16_t*>(xrow_s + m * 256 + (((k >> 3) ^ (r << 2)) << 4) + (k & 7) * 2);
                        accf[o][i >> 1][2 * (i & 1) + r] = fmaf(v, bf16_bits_to_float(xbits), accf[o][i >> 1][2 * (i & 1) + r]);
                    }
            };
            // staged packets first, later ones (rare) from global memory; past its own list a lane group adds padding
            const uint32_t n = sp_depth + sp_tail;
            const uint32_t nmax = __reduce_max_sync(0xffffffffu, n);
            for (uint32_t d = 0; d < nmax; ++d) {
                uint4 pk = make_uint4(0, 0, 0, 0);
                if (d < n) pk = d < (uint32_t)kDirectSlots ? *reinterpret_cast<const uint4*>(pks + g * (kDirectSlots * 16) + ((d ^ g) & (kDirectSlots - 1)) * 16)
                                                           : __ldg(p.packed + sp_first + d);
                if (d >= sp_depth && d < n) {
                    // tail: a slot names its column; in the others it counts as padding
                    const uint32_t wd[4] = {pk.x, pk.y, pk.z, pk.w};
                    pk = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const uint32_t col = (wd[e] >> kSlotColShift) & 3u, w = wd[e];
                        add_slot(col == 0 ? w : 0u, 0); add_slot(col == 1 ? w : 0u, 1);
                        add_slot(col == 2 ? w : 0u, 2); add_slot(col == 3 ? w : 0u, 3);
                    }
                }
                add_slot(pk.x, 0); add_slot(pk.y, 1); add_slot(pk.z, 2); add_slot(pk.w, 3);
            }
        }
    }
    if (!waited) asm volatile("griddepcontrol.wait;" ::: "memory");     // a warp without a k-step still writes below
    // ---- the W partial sums of the strip, added in warp order; then Y
    __syncthreads();                                                    // the staging bytes become the sums
#pragma unroll
    for (int o = 0; o < MO; ++o)
#pragma unroll
        for (int cg = 0; cg < CG; ++cg)
#pragma unroll
            for (int i = 0; i < 4; ++i) red[(warp * NV + (o * CG + cg) * 4 + i) * 32 + lane] = accf[o][cg][i];
    // the column-per-lane outlier sums go beside them as they are, [WARPS][R][32]: lane (g, i) holds column g + 8i
    float* sred = red + WARPS * NV * 32;
    if constexpr (SPARSE && MS != 16) {
#pragma unroll
        for (int r = 0; r < R; ++r) sred[(warp * R + r) * 32 + lane] = sacc[r];
    }
    __syncthreads();
    if (tid < NV * 32) {
        const int e = tid >> 5;                                     // (o, cg, h, r) of this thread's element; lane = (g, t)
        const int o = e / (CG * 4), cg = (e >> 2) % CG, h = (e >> 1) & 1, r = e & 1;
        const uint32_t m = 8 * o + 2 * t + r;
        float sum = 0.0f;
#pragma unroll 8
        for (int w = 0; w < WARPS; ++w) sum += red[(w * NV + e) * 32 + lane];
        if constexpr (SPARSE && MS != 16) {
            if (m < (uint32_t)R) {
                // column g + 16 cg + 8 h is column number 2 cg + h of bucket g: its sums sit in lane 4 g + 2 cg + h
                float osum = 0.0f;
#pragma unroll 8
                for (int w = 0; w < WARPS; ++w) osum += sred[(w * R + m) * 32 + 4 * g + 2 * cg + h];
                sum += osum;
            }
        }
        if (m < p.M) p.Y[(size_t)m * p.N + (size_t)strip * 32 + g + 16 * cg + 8 * h] = float_to_bf16_bits(sum);
    }
}
