// The fused operator with warp-level MMAs (mma.sync m16n8k16), for launches of up to 16 batch rows.
// Included by fq_kernels.cu inside namespace fq, after the PTX helpers.
//
// Persistent, warp-specialised, one CTA per SM; (tile, k-step) units of 128 rows x BN columns stream through a
// ring of shared-memory stages (cp.async.bulk + mbarrier expect_tx).  The tensor cores get the exact integers
// 128 + q as BF16, and scale and zero-point are applied once per group in FP32:
//     acc[m] += s * (sum_k x (128+q) - (128+z) sum_k x)                 (Eq. 3 inside Eq. 1)

struct MmaParams {
    const uint16_t* X;
    const uint8_t* wq;
    const uint16_t* scale;
    const uint16_t* zero;
    const uint32_t* indptr;
    const uint32_t* info;
    const uint4* packed;
    uint16_t* Y;
    uint32_t* status;
    uint32_t* counters;
    float* partials;
    uint32_t M, K, N, KT, NT;
    uint32_t NB, coo_cap, stages;
    uint32_t split;   // 0 = units dealt out as one contiguous range per CTA (stream-K);
                      // c > 0 = every column tile belongs to c CTAs, CTA b takes part b mod c of tile b / c
    // shared-memory offsets (bytes); the first five are relative to a stage
    uint32_t stage_bytes, off_sz, off_xcan, off_xsum, off_info, off_coo;
    uint32_t off_shc, off_xt, off_bar;
};

// Transpose one octet of BF16 activation rows into the FP32 k-major copy xt[k][8] (32 B per k).
// `row0` is the shared-memory address of row 0 / 16-byte chunk 0 of the octet, rows `row_step`
// bytes apart, consecutive 16-byte chunks (8 k each) `chunk_step` bytes apart.  Whole warp.
// SWZ: odd rows keep chunk c at position c ^ 4.  PAIRS < 4: only the first PAIRS pairs of rows are
// kept, 2 * PAIRS floats per k.
template <bool SWZ = false, int PAIRS = 4>
__device__ __forceinline__ void transpose_octet_f32(uint32_t row0, uint32_t row_step, uint32_t chunk_step, float* xt, int lane) {
#pragma unroll
    for (int kb = 0; kb < 4; ++kb) {
        uint32_t r[4];
        const uint32_t chunk = (kb * 4 + (lane >> 3)) ^ (SWZ ? ((uint32_t)lane & 1u) << 2 : 0u);
        ldmatrix_x4_trans(row0 + (lane & 7) * row_step + chunk * chunk_step, r[0], r[1], r[2], r[3]);
        // thread T holds rows m = 2(T%4), 2(T%4)+1 of column k = 8*block + T/4
        float* dst = xt + ((kb * 32) + (lane >> 2)) * (2 * PAIRS) + (lane & 3) * 2;
        if (PAIRS == 4 || (lane & 3) < PAIRS) {
#pragma unroll
            for (int i = 0; i < 4; ++i) *reinterpret_cast<float2*>(dst + i * 16 * PAIRS) = make_float2(bf16lo(r[i]), bf16hi(r[i]));
        }
    }
}


__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

constexpr int kActWarps = 2;   // activation warps of the streaming kernel
// Activation row in shared memory: 256 B, its sixteen 16-byte chunks stored at chunk ^ 4 in odd rows.
// The fragment loads of a quarter warp (rows g and g + 1, four consecutive chunks each) then touch
// all 32 banks once.
constexpr int kXPitch = 256;

// The same operator for M <= 8 per octet (MO octets of batch rows): every dense warp runs the same
// short loop (one 32-column strip per warp, warp-level m16n8k16 MMAs with the weights on the M side
// and the batch on the N side), so the instruction stream of the CTA's dense warps is shared and
// stays in the instruction cache.  Same packed formats, same producer, same split-tile protocol as
// the tcgen05 kernel; the dense engine differs, and the outliers need no warps of their own:
//   warp 0            producer: bulk copies of the packed weights and the scales (and the
//                     zero-points in kernels with outliers)
//   warps 1..2        activations (alternate units): X block -> row-major shared-memory rows +
//                     per-group row sums + an FP32 k-major copy for the outlier step; bulk copies of
//                     the unit's bucket descriptors and packets (or of its zero-points)
//   then NGRP x BN/32 dense + outliers.  Lane (g, t) of warp w holds the accumulators of columns
//                     32w + {g, g+8, g+16, g+24}, batch rows 2t, 2t+1 (+8 per octet).  Dense: the
//                     lane loads, as one 16-byte word group, word t of its four columns of each
//                     32-row block: 8 codes per column = its share of two k16 steps (the k order
//                     inside a block follows the 16-byte activation loads of the lanes).  Outliers:
//                     those four columns are one Tile-COO bucket, so the four lanes of group g walk
//                     that bucket's packets and add v * x[row][k] straight into their accumulators,
//                     slot j into column number j (Section 4.2 without the shared-memory scatter:
//                     no atomics, no read-modify-write, no merge step).
template <int BN, int MO, int GROUP, bool SPARSE, int MS, int NGRP, bool HOT>
__global__ void __launch_bounds__(32 * (1 + kActWarps + NGRP * (BN / 32)), 1) fq_mma_kernel(const MmaParams p) {
    constexpr int NDW = BN / 32;
    constexpr int NA = kActWarps;                           // activation warps: warp a takes the units it with it mod NA == a
    // (the number of stages is a multiple of NA and of NGRP, so that a stage always returns to the same
    // activation warp and dense group: each of them then sees every phase of the stage's barriers)
    constexpr int DW0 = 1 + NA;                             // first dense warp
    // NGRP dense warp groups: group r takes the units it with it mod NGRP == r
    constexpr int CG = 2;                                   // 16-column MMA strips per warp
    // two groups of 16-row warps share the register file, and 32-row warps fill it alone: one packet
    // requested ahead instead of two and its activation rows, two contributors in flight when a split
    // tile is settled
    constexpr bool kTight = (MO == 2 && NGRP == 2) || MO == 4;
    constexpr int GPS = kBK / GROUP;
    constexpr int W_BYTES = 16 * BN * 4;
    constexpr int SZ_ROW = BN * 2;
    constexpr bool kActZero = !SPARSE;                      // who requests the zero-points: see the producer
    constexpr int LDC = 8 * MO;
    extern __shared__ __align__(128) uint8_t smem[];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t S = p.stages;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * S;
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 2 * S + 4);
    // hand-over of group 1's partial sums to group 0 at the end of a piece: one pair of barriers per strip
    const uint32_t bar_xfull = bar_empty + 8 * S + 64, bar_xempty = bar_xfull + 8 * NDW;

    // one barrier per thread of warp 0: S full, S empty (then the hand-over pairs)
    if ((uint32_t)tid < S) mbar_init(bar_full + 8 * tid, 2);                 // producer's expect_tx arrival + activation warp
    else if ((uint32_t)tid < 2 * S) mbar_init(bar_empty + 8 * (tid - S), NDW);   // the dense warps of one group
    else if ((uint32_t)tid < 2 * S + 2 * NDW) mbar_init(bar_xfull + 8 * (tid - 2 * S), 1);
    if (tid == 0) *abort_flag = 0;
    if (tid < 32) asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    // The grid after this one in the stream may start now (it takes SMs as this grid's CTAs leave).
    // Every warp but the producer waits for the grid before this one to finish: the producer reads
    // only weights, which no kernel writes while calls are in flight.  (The activation warps first
    // request the other weight arrays of their first units, see there.)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (warp >= DW0) asm volatile("griddepcontrol.wait;" ::: "memory");

    const uint32_t KT = p.KT;
    const uint32_t U = p.NT * KT, P = gridDim.x, q = U / P, r = U % P;
    uint32_t u_begin, u_end;
    if (p.split) {
        // tile-aligned split: no CTA works on two tiles, so none settles two split tiles one after the other
        const uint32_t tile = blockIdx.x / p.split, part = blockIdx.x - tile * p.split;
        u_begin = tile * KT + part * KT / p.split;
        u_end = tile * KT + (part + 1) * KT / p.split;
    } else {
        u_begin = unit_begin_of(blockIdx.x, q, r);
        u_end = u_begin + q + (blockIdx.x < r ? 1u : 0u);
    }

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        // Packed weights and scales of every unit; its zero-points too in a kernel with outliers, where
        // the unit's activation warp requests the outlier arrays (without outliers it requests the
        // zero-points).  A bulk copy costs its issuing warp a few hundred cycles next to the dense
        // warps' shared-memory traffic: five of them per unit made this warp the bottleneck of the
        // kernels with one octet of rows, and this split measured best.
        uint32_t issued = 0;
        bool ok = true;
        for (UnitIter w(u_begin, KT); w.u < u_end; w.next(S, KT)) {
            const uint32_t u = w.u, it = w.it, s = w.s, ph = w.ph;
            if (!warp_wait(bar_empty + 8 * s, ph ^ 1, abort_flag, p.status)) { ok = false; break; }
            const uint32_t full = bar_full + 8 * s;
            const uint32_t st = smem_u32(smem) + s * p.stage_bytes;
            if (lane == 0) {
                mbar_arrive_expect_tx(full, W_BYTES + (kActZero ? 1 : 2) * GPS * SZ_ROW);
                bulk_g2s(st, p.wq + (size_t)u * W_BYTES, W_BYTES, full);
#pragma unroll
                for (int gi = 0; gi < GPS; ++gi) {
                    const size_t row = (size_t)(w.kt * GPS + gi) * p.N + (size_t)w.tn * BN;
                    bulk_g2s(st + p.off_sz + gi * SZ_ROW, p.scale + row, SZ_ROW, full);
                    if (!kActZero) bulk_g2s(st + p.off_sz + (GPS + gi) * SZ_ROW, p.zero + row, SZ_ROW, full);
                }
            }
            issued = it + 1;
        }
        if (!ok) {
            for (uint32_t j = (issued > S ? issued - S : 0); j < issued; ++j)
                for (uint32_t spin = 0; spin < (1u << 20) && !mbar_try_wait(bar_full + 8 * (j % S), (j / S) & 1); ++spin) {}
        }
    } else if (warp < DW0) {
        // ------------------------------------------------------------------ activation warps
        const uint32_t aw = warp - 1;
        // lane -> (row m, part): 16-byte chunks of that row; rows beyond M are zero
        constexpr int ROWS = 8 * MO;
        constexpr int LPR = 32 / ROWS;                       // lanes per row: 4 (8 rows), 2 (16 rows) or 1 (32 rows)
        constexpr int CPL = 16 / LPR;                        // chunks per lane
        const int m = lane % ROWS, part = lane / ROWS;
        const bool real = (uint32_t)m < p.M;
        const uint8_t* xrow = reinterpret_cast<const uint8_t*>(p.X) + ((size_t)m * p.K) * 2 + part * CPL * 16;
        uint4 nxt[CPL];
        auto load = [&](uint32_t kt) {
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                nxt[c] = make_uint4(0, 0, 0, 0);
                if (real) nxt[c] = __ldg(reinterpret_cast<const uint4*>(xrow + (size_t)kt * 256 + c * 16));
            }
        };
        // the unit's range of outlier packets (lane 0), read one unit ahead like the activations
        uint32_t ip_nxt = 0, ip_nxt_end = 0, last_bar = 0, last_ph = 0;
        bool ok = true;
        auto load_ip = [&](uint32_t u) {
            if (SPARSE && lane == 0) { ip_nxt = __ldg(p.indptr + u); ip_nxt_end = __ldg(p.indptr + u + 1); }
        };
        // this warp's share of the weight arrays of unit u (k-step kt of column tile tn): bucket
        // descriptors and packets, or the zero-points; into the stage at shared-memory address sta,
        // counted on its barrier before this warp's arrival
        auto request = [&](uint32_t u, uint32_t tn, uint32_t kt, uint32_t sta, uint32_t full, uint32_t ip, uint32_t npk) {
            mbar_expect_tx(full, kActZero ? GPS * SZ_ROW : p.NB * 4 + npk * 16);
            if (kActZero) {
#pragma unroll
                for (int gi = 0; gi < GPS; ++gi)
                    bulk_g2s(sta + p.off_sz + (GPS + gi) * SZ_ROW, p.zero + (size_t)(kt * GPS + gi) * p.N + (size_t)tn * BN, SZ_ROW, full);
            }
            if (SPARSE) {
                bulk_g2s(sta + p.off_info, p.info + (size_t)u * p.NB, p.NB * 4, full);
                if (npk) bulk_g2s(sta + p.off_coo, p.packed + ip, npk * 16, full);
            }
        };
        {
            // The first pass over the ring finds every stage empty, and these arrays are weights:
            // lane l requests those of this warp's l-th unit before the wait for the previous grid.
            const uint32_t it0 = aw + NA * lane;
            if (it0 < min(S, u_end - u_begin)) {
                const uint32_t u = u_begin + it0, tn = u / KT;
                uint32_t a = 0, npk = 0;
                if (SPARSE) { a = __ldg(p.indptr + u); npk = min(__ldg(p.indptr + u + 1) - a, p.coo_cap); }
                request(u, tn, u - tn * KT, smem_u32(smem) + it0 * p.stage_bytes, bar_full + 8 * it0, a, npk);
            }
            __syncwarp();
            asm volatile("griddepcontrol.wait;" ::: "memory");
        }
        if (u_begin + aw < u_end) { load((u_begin + aw) % KT); load_ip(u_begin + aw); }
        for (UnitIter w(u_begin, KT); w.u < u_end; w.next(S, KT)) {
            if (w.it % NA != aw) continue;
            const uint32_t s = w.s, ph = w.ph;
            uint8_t* st = smem + s * p.stage_bytes;
            uint4 xv[CPL];
#pragma unroll
            for (int c = 0; c < CPL; ++c) xv[c] = nxt[c];
            const uint32_t ip = ip_nxt, npk = min(ip_nxt_end - ip_nxt, p.coo_cap);
            if (w.u + NA < u_end) { uint32_t kn = w.kt + NA; load(kn >= KT ? kn % KT : kn); load_ip(w.u + NA); }   // this warp's next unit
            if (!warp_wait(bar_empty + 8 * s, ph ^ 1, abort_flag, p.status)) { ok = false; break; }
            last_bar = bar_full + 8 * s, last_ph = ph;
            if (lane == 0 && w.it >= S) request(w.u, w.tn, w.kt, smem_u32(st), bar_full + 8 * s, ip, npk);
            uint8_t* dst = st + p.off_xcan + m * kXPitch;
            const int swz = (m & 1) << 2;
            float sum = 0.0f, sum_lo = 0.0f;          // sum_lo: chunks 0-7 where a lane holds a whole row
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                const uint4 v = xv[c];
                *reinterpret_cast<uint4*>(dst + ((part * CPL + c) ^ swz) * 16) = v;
                if (LPR == 1 && c == 8) sum_lo = sum, sum = 0.0f;
                sum += (bf16lo(v.x) + bf16hi(v.x)) + (bf16lo(v.y) + bf16hi(v.y)) + (bf16lo(v.z) + bf16hi(v.z)) +
                       (bf16lo(v.w) + bf16hi(v.w));
            }
            // per-group sums of each row: lanes with the same m hold consecutive quarters / halves of the row
            float* xsum = reinterpret_cast<float*>(st + p.off_xsum);
            if (LPR == 4) {
                const float s1 = sum + __shfl_xor_sync(0xffffffffu, sum, 8);       // parts {0,1} and {2,3}
                const float s2 = s1 + __shfl_xor_sync(0xffffffffu, s1, 16);
                if (GPS == 2) { if ((part & 1) == 0) xsum[(part >> 1) * ROWS + m] = s1; }
                else if (part == 0) xsum[m] = s2;
            } else if (LPR == 2) {
                const float s1 = sum + __shfl_xor_sync(0xffffffffu, sum, 16);
                if (GPS == 2) xsum[part * ROWS + m] = sum;
                else if (part == 0) xsum[m] = s1;
            } else {
                if (GPS == 2) xsum[m] = sum_lo, xsum[ROWS + m] = sum;
                else xsum[m] = sum_lo + sum;
            }
            __syncwarp();
            if (SPARSE && MS == 1) {
                // FP32 copy of the single batch row for the outlier step: xt[k]
                if (m == 0) {
                    float4* xt4 = reinterpret_cast<float4*>(st + p.off_xt) + part * CPL * 2;
#pragma unroll
                    for (int c = 0; c < CPL; ++c) {
                        xt4[2 * c] = make_float4(bf16lo(xv[c].x), bf16hi(xv[c].x), bf16lo(xv[c].y), bf16hi(xv[c].y));
                        xt4[2 * c + 1] = make_float4(bf16lo(xv[c].z), bf16hi(xv[c].z), bf16lo(xv[c].w), bf16hi(xv[c].w));
                    }
                }
                __syncwarp();
            } else if (SPARSE && MS == 4) {
                // FP32 k-major copy of the first four batch rows for the outlier step: xt[k][4]
                transpose_octet_f32<true, 2>(smem_u32(st + p.off_xcan), kXPitch, 16, reinterpret_cast<float*>(st + p.off_xt), lane);
                __syncwarp();
            } else if (SPARSE) {
                // FP32 k-major copy [octet][k][8] for the outlier step
#pragma unroll
                for (int o = 0; o < MO; ++o)
                    transpose_octet_f32<true>(smem_u32(st + p.off_xcan) + o * 8 * kXPitch, kXPitch, 16,
                                        reinterpret_cast<float*>(st + p.off_xt) + o * 1024, lane);
                __syncwarp();
            }
            if (lane == 0) mbar_arrive(bar_full + 8 * s);
        }
        if (!ok && last_bar)                // gave up: let this warp's last copies land before the CTA exits
            for (uint32_t spin = 0; spin < (1u << 20) && !mbar_try_wait(last_bar, last_ph); ++spin) {}
    } else if (warp >= DW0 && warp < DW0 + NGRP * NDW) {
        // ------------------------------------------------------------------ dense warps (all alike)
        // Two groups of NDW warps take alternate units, each with accumulators of its own: twice the
        // warps to hide latencies with, and no warp does less work per unit it takes.  At the end of
        // a piece group 1 hands its sums to group 0 through shared memory.
        const int dwi = warp - DW0, grp = dwi / NDW, dw = dwi % NDW, g = lane >> 2, t = lane & 3;
        float* xch = reinterpret_cast<float*>(smem + p.off_shc) + dw * (MO * CG * 4 * 32) + lane;
        const int c0 = dw * 32 + g;                           // this lane's columns: c0 + 8 * {0, 1, 2, 3}
        float accf[MO][CG][4];
#pragma unroll
        for (int o = 0; o < MO; ++o)
#pragma unroll
            for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                for (int i = 0; i < 4; ++i) accf[o][cg][i] = 0.0f;
        // Outlier sums of the column-per-lane forms (MS == 1: one batch row, MS == 4: up to four): there
        // lane (g, t) owns ONE column, 32 dw + 8 t + g (the bucket's column number t), and takes slot t
        // of every packet; the sums are moved into the MMA fragment layout above (four columns x two
        // rows per lane) once per piece.
        constexpr int R = MS == 4 ? 4 : 1;
        float sacc[R];
#pragma unroll
        for (int ri = 0; ri < R; ++ri) sacc[ri] = 0.0f;
        uint32_t piece = 0;
        bool ok = true;
        // outer loop: the pieces of this CTA's range (a piece = its units of one column tile); inner loop:
        // this group's units of the piece (every NGRP-th unit of the range; the ring length is a multiple
        // of NGRP).  The end-of-piece code stays out of the inner loop's body.
        uint32_t u = u_begin + grp, s = grp, ph = 0;                    // this group's next unit, its stage and parity
        uint32_t tn = u_begin / KT;
        for (uint32_t piece_first = u_begin; piece_first < u_end && ok; ++tn) {
          const uint32_t piece_stop = min(u_end, (tn + 1) * KT);        // one past the piece's last unit
          piece_first = piece_stop;
          for (; u < piece_stop; u += NGRP, s = (s + NGRP >= S ? s + NGRP - S : s + NGRP), ph ^= (s < (uint32_t)NGRP ? 1u : 0u)) {
            const uint8_t* st = smem + s * p.stage_bytes;
            {
            if (!warp_wait(bar_full + 8 * s, ph, abort_flag, p.status)) { ok = false; break; }
            const uint32_t* wp = reinterpret_cast<const uint32_t*>(st) + (dw * 32 + g) * 4 + t;   // word t of column c0; the others 8 columns on
            // chunk 4j + t of row g (+ 8 per octet): at (4j + t) ^ 4 in odd rows, i.e. 64 B further for
            // even j and 64 B back for odd j
            const uint8_t* xrow = st + p.off_xcan + g * kXPitch + t * 16;
            const uint8_t* xrow_e = xrow + ((g & 1) << 6);
            const uint8_t* xrow_o = xrow - ((g & 1) << 6);
            const uint16_t* sc = reinterpret_cast<const uint16_t*>(st + p.off_sz);
            const float* xsum = reinterpret_cast<const float*>(st + p.off_xsum);
            // outliers: the bucket descriptor and the first two packets are requested now and used
            // after the dense math of the unit.  A bucket's packets are column-slotted: slot j of a packet
            // belongs to column number j of the bucket, so a slot's accumulators are known at compile time.
            // PKT is what a lane reads of a packet: its own slot (MS == 1, lane t keeps column number t) or
            // all four (MS == 8, lane t keeps batch rows 2t, 2t + 1 of all four columns).
            // HOT is the general form of the outlier step, chosen by the host for layers that need it:
            //  - buckets with a tail (a very long column): the tail's packets, whose slots name their
            //    column, are shared out over the eight lane groups, which add into sums of their own that
            //    are added up over the groups afterwards;
            //  - tiles with more packets than a stage holds: the rest is read from global memory.
            // Kernels for layers that need neither are compiled without that code: the presence of either
            // costs the common path 3-4 %.
            using PKT = typename std::conditional<MS != 8, uint32_t, uint4>::type;
            uint32_t sp_off = 0, sp_cnt = 0, sp_tail = 0, cmax = 0;
            const uint4* pk_s = reinterpret_cast<const uint4*>(st + p.off_coo);
            const uint4* pk_g = nullptr;
            const char* xtb = reinterpret_cast<const char*>(st + p.off_xt);
            const uint32_t x_lane = MS != 8 ? 0u : 8u * t;    // byte offset of the lane's batch rows in a row of xt
            auto load_packet = [&](uint32_t idx) -> PKT {
                const uint4* src = (!HOT || idx < p.coo_cap) ? pk_s + idx : pk_g + idx;
                if constexpr (MS != 8) return reinterpret_cast<const uint32_t*>(src)[t];
                else return *src;
            };
            auto packet = [&](uint32_t i) -> PKT {
                PKT pk = PKT();                               // beyond the bucket's list: padding
                if (i < sp_cnt) pk = load_packet(sp_off + i);
                return pk;
            };
            // activation rows 2t, 2t + 1 of every octet for the row of one slot (slot & 0xfe0 = 32 * row)
            auto slot_x = [&](const uint32_t w, float2 (&x2)[MO]) {
#pragma unroll
                for (int o = 0; o < MO; ++o) x2[o] = *reinterpret_cast<const float2*>(xtb + ((w & 0xfe0u) | x_lane) + o * 4096);
            };
            auto fetch_x = [&](const uint4 pk, float2 (&x2)[4][MO]) {
                slot_x(pk.x, x2[0]); slot_x(pk.y, x2[1]); slot_x(pk.z, x2[2]); slot_x(pk.w, x2[3]);
            };
            PKT pk0 = PKT(), pk1 = PKT();
            float2 xa[4][MO];
            if (SPARSE) {
                const uint32_t info = reinterpret_cast<const uint32_t*>(st + p.off_info)[dw * 8 + g];
                sp_off = info & 0xffffu;
                sp_cnt = (info >> 16) & 0xffu;
                if (HOT) sp_tail = info >> 24;
                if (!HOT && __any_sync(0xffffffffu, sp_off + sp_cnt > p.coo_cap)) {
                    // a descriptor that does not belong to the staged packets (layout struct and arrays out of
                    // step): report it and skip the unit's outliers instead of reading past the stage
                    if (lane == 0) atomicExch(p.status, (uint32_t)FQ_ERR_FORMAT);
                    sp_cnt = 0;
                }
                cmax = __reduce_max_sync(0xffffffffu, sp_cnt);
                if (HOT && __reduce_max_sync(0xffffffffu, sp_off + sp_cnt + sp_tail) > p.coo_cap)
                    pk_g = p.packed + __ldg(p.indptr + u);           // packets beyond the staged part
                pk0 = packet(0);
                if constexpr (!kTight) pk1 = packet(1);
                if constexpr (MS == 8 && !kTight) fetch_x(pk0, xa);
            }
#pragma unroll
            for (int gi = 0; gi < GPS; ++gi) {
                float accg[MO][CG][4];
#pragma unroll
                for (int o = 0; o < MO; ++o)
#pragma unroll
                    for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                        for (int i = 0; i < 4; ++i) accg[o][cg][i] = 0.0f;
#pragma unroll
                for (int j = gi * (4 / GPS); j < (gi + 1) * (4 / GPS); ++j) {
                    uint4 xb[MO];
#pragma unroll
                    for (int o = 0; o < MO; ++o) xb[o] = *reinterpret_cast<const uint4*>(((j & 1) ? xrow_o : xrow_e) + o * 8 * kXPitch + j * 64);
                    const uint4 w4 = make_uint4(wp[j * BN * 4], wp[j * BN * 4 + 32], wp[j * BN * 4 + 64], wp[j * BN * 4 + 96]);   // columns +0, +8, +16, +24
#pragma unroll
                    for (int cg = 0; cg < CG; ++cg) {
                        const uint32_t wa = cg ? w4.z : w4.x, wb = cg ? w4.w : w4.y;
                        const uint32_t a0 = codes_to_bf16x2(wa), a1 = codes_to_bf16x2(wa >> 4);
                        const uint32_t a2 = codes_to_bf16x2(wa >> 8), a3 = codes_to_bf16x2(wa >> 12);
                        const uint32_t b0 = codes_to_bf16x2(wb), b1 = codes_to_bf16x2(wb >> 4);
                        const uint32_t b2 = codes_to_bf16x2(wb >> 8), b3 = codes_to_bf16x2(wb >> 12);
#pragma unroll
                        for (int o = 0; o < MO; ++o) {
                            mma_bf16(accg[o][cg], a0, b0, a1, b1, xb[o].x, xb[o].y);   // rows 8t+0..3 of the block
                            mma_bf16(accg[o][cg], a2, b2, a3, b3, xb[o].z, xb[o].w);   // rows 8t+4..7
                        }
                    }
                }
                // once per group: acc += s * (sum x (128+q) - (128+z) sum x)     (Eq. 3 inside Eq. 1)
                float2 xs[MO];
#pragma unroll
                for (int o = 0; o < MO; ++o) xs[o] = *reinterpret_cast<const float2*>(xsum + gi * LDC + o * 8 + 2 * t);
#pragma unroll
                for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int col = c0 + 16 * cg + 8 * h;
                        const float sv = bf16_bits_to_float(sc[gi * BN + col]);
                        const float zc = -(128.0f + bf16_bits_to_float(sc[(GPS + gi) * BN + col]));
#pragma unroll
                        for (int o = 0; o < MO; ++o) {
                            accf[o][cg][2 * h + 0] = fmaf(sv, fmaf(zc, xs[o].x, accg[o][cg][2 * h + 0]), accf[o][cg][2 * h + 0]);
                            accf[o][cg][2 * h + 1] = fmaf(sv, fmaf(zc, xs[o].y, accg[o][cg][2 * h + 1]), accf[o][cg][2 * h + 1]);
                        }
                    }
            }
            if (SPARSE) {
                // ---- outliers of this unit in the lane group's bucket (padding slots have value 0: they
                // add 0)
                if constexpr (MS != 8) {
                    // column per lane: lane t keeps the slots of column number t of the bucket; a row of xt
                    // holds the R batch rows of one k (slot & 0xfe0 = 32 * row)
                    auto add = [&](float (&acc)[R], const float v, const uint32_t w) {
                        if constexpr (R == 1) {
                            acc[0] = fmaf(v, *reinterpret_cast<const float*>(xtb + ((w >> 3) & 0x1fcu)), acc[0]);
                        } else {
                            const float4 x = *reinterpret_cast<const float4*>(xtb + ((w >> 1) & 0x7f0u));
                            acc[0] = fmaf(v, x.x, acc[0]);
                            acc[1] = fmaf(v, x.y, acc[1]);
                            acc[2] = fmaf(v, x.z, acc[2]);
                            acc[R - 1] = fmaf(v, x.w, acc[R - 1]);
                        }
                    };
                    auto apply = [&](const uint32_t w) { add(sacc, __uint_as_float(w & kSlotValueMask), w); };
                    if (cmax > 0) apply(pk0);
                    if (cmax > 1) {
                        apply(pk1);
                        for (uint32_t i = 2; i < cmax; ++i) apply(packet(i));
                    }
                    if (HOT) {
                        for (uint32_t hot = __ballot_sync(0xffffffffu, sp_tail != 0); hot; ) {     // warp-uniform
                            const uint32_t hot_lane = __ffs(hot) - 1;
                            hot &= ~(0xfu << (hot_lane & ~3u));
                            const uint32_t hot_off = __shfl_sync(0xffffffffu, sp_off + sp_cnt, hot_lane);
                            const uint32_t hot_cnt = __shfl_sync(0xffffffffu, sp_tail, hot_lane);
                            float hacc[R];
#pragma unroll
                            for (int ri = 0; ri < R; ++ri) hacc[ri] = 0.0f;
                            for (uint32_t i = g; i < hot_cnt; i += 8) {
                                const uint32_t idx = hot_off + i;
                                const uint4 pk = (idx < p.coo_cap) ? pk_s[idx] : __ldg(pk_g + idx);
                                const uint32_t w[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e)     // a tail slot names its column
                                    add(hacc, ((w[e] >> kSlotColShift) & 3u) == (uint32_t)t ? __uint_as_float(w[e] & kSlotValueMask) : 0.0f, w[e]);
                            }
#pragma unroll
                            for (int ri = 0; ri < R; ++ri) {
                                float v = hacc[ri];
                                v += __shfl_xor_sync(0xffffffffu, v, 4);
                                v += __shfl_xor_sync(0xffffffffu, v, 8);
                                v += __shfl_xor_sync(0xffffffffu, v, 16);
                                if ((uint32_t)g == (hot_lane >> 2)) sacc[ri] += v;
                            }
                        }
                    }
                } else {
                    // several batch rows: lane t keeps rows 2t, 2t+1 (+8) of all four columns, in the
                    // MMA fragment registers themselves; slot j goes to column number j
                    auto apply = [&](const uint4 pk, const float2 (&x2)[4][MO]) {
                        const uint32_t w[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float v = __uint_as_float(w[e] & kSlotValueMask);
#pragma unroll
                            for (int o = 0; o < MO; ++o) {
                                accf[o][e >> 1][2 * (e & 1) + 0] = fmaf(v, x2[e][o].x, accf[o][e >> 1][2 * (e & 1) + 0]);
                                accf[o][e >> 1][2 * (e & 1) + 1] = fmaf(v, x2[e][o].y, accf[o][e >> 1][2 * (e & 1) + 1]);
                            }
                        }
                    };
                    if constexpr (kTight) {
                        if (cmax > 0) { fetch_x(pk0, xa); apply(pk0, xa); }
                        for (uint32_t i = 1; i < cmax; ++i) {
                            const uint4 pk = packet(i);
                            fetch_x(pk, xa);
                            apply(pk, xa);
                        }
                    } else {
                    if (cmax > 0) apply(pk0, xa);
                    if (cmax > 1) {
                        float2 xb2[4][MO];
                        fetch_x(pk1, xb2);
                        apply(pk1, xb2);
                        for (uint32_t i = 2; i < cmax; ++i) {
                            const uint4 pk = packet(i);
                            fetch_x(pk, xb2);
                            apply(pk, xb2);
                        }
                    }
                    }
                    if (HOT) {
                        for (uint32_t hot = __ballot_sync(0xffffffffu, sp_tail != 0); hot; ) {     // warp-uniform
                            const uint32_t hot_lane = __ffs(hot) - 1;
                            hot &= ~(0xfu << (hot_lane & ~3u));
                            const uint32_t hot_off = __shfl_sync(0xffffffffu, sp_off + sp_cnt, hot_lane);
                            const uint32_t hot_cnt = __shfl_sync(0xffffffffu, sp_tail, hot_lane);
                            float hacc[MO][CG][4];
#pragma unroll
                            for (int o = 0; o < MO; ++o)
#pragma unroll
                                for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                                    for (int i = 0; i < 4; ++i) hacc[o][cg][i] = 0.0f;
                            for (uint32_t i = g; i < hot_cnt; i += 8) {
                                const uint32_t idx = hot_off + i;
                                const uint4 pk = (idx < p.coo_cap) ? pk_s[idx] : __ldg(pk_g + idx);
                                float2 xh[4][MO];
                                fetch_x(pk, xh);
                                const uint32_t w[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const uint32_t cls = (w[e] >> kSlotColShift) & 3u;
                                    const float v = __uint_as_float(w[e] & kSlotValueMask);
#pragma unroll
                                    for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                                        for (int h = 0; h < 2; ++h) {
                                            // a select, not a branch: the lanes of a warp hold different columns
                                            const float vv = (cls == (uint32_t)(2 * cg + h)) ? v : 0.0f;
#pragma unroll
                                            for (int o = 0; o < MO; ++o) {
                                                hacc[o][cg][2 * h + 0] = fmaf(vv, xh[e][o].x, hacc[o][cg][2 * h + 0]);
                                                hacc[o][cg][2 * h + 1] = fmaf(vv, xh[e][o].y, hacc[o][cg][2 * h + 1]);
                                            }
                                        }
                                }
                            }
#pragma unroll
                            for (int o = 0; o < MO; ++o)
#pragma unroll
                                for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                                    for (int i = 0; i < 4; ++i) {
                                        float v = hacc[o][cg][i];
                                        v += __shfl_xor_sync(0xffffffffu, v, 4);
                                        v += __shfl_xor_sync(0xffffffffu, v, 8);
                                        v += __shfl_xor_sync(0xffffffffu, v, 16);
                                        if ((uint32_t)g == (hot_lane >> 2)) accf[o][cg][i] += v;
                                    }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive_relaxed(bar_empty + 8 * s);
            }

          }
          if (!ok) break;
          {
                const uint32_t kt = piece_stop - 1 - tn * KT;               // k-step of the piece's last unit
                // ---------------------------------------------------------- end of a piece
                if (SPARSE && MS == 1) {
                    // single-row outlier sums -> fragment layout: column number c of the group comes
                    // from lane (g, c); batch row 0 lives in lane t = 0
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const float v = __shfl_sync(0xffffffffu, sacc[0], (lane & ~3) | c);
                        if (t == 0) accf[0][c >> 1][2 * (c & 1)] += v;
                    }
                    sacc[0] = 0.0f;
                }
                if constexpr (SPARSE && MS == 4) {
                    // four rows of outlier sums -> fragment layout: column number c comes from lane (g, c);
                    // rows 0, 1 live in lane t = 0, rows 2, 3 in lane t = 1
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            const float v0 = __shfl_sync(0xffffffffu, sacc[j], (lane & ~3) | c);
                            const float v1 = __shfl_sync(0xffffffffu, sacc[R - 2 + j], (lane & ~3) | c);
                            accf[0][c >> 1][2 * (c & 1) + j] += t == 0 ? v0 : (t == 1 ? v1 : 0.0f);
                        }
#pragma unroll
                    for (int ri = 0; ri < R; ++ri) sacc[ri] = 0.0f;
                }
                if (NGRP > 1) {
                    if (grp == 1) {
                        // hand the sums over (after group 0 has taken the previous piece's) and start afresh
                        if (piece > 0 && !warp_wait(bar_xempty + 8 * dw, (piece - 1) & 1, abort_flag, p.status)) { ok = false; break; }
#pragma unroll
                        for (int o = 0; o < MO; ++o)
#pragma unroll
                            for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    xch[((o * CG + cg) * 4 + i) * 32] = accf[o][cg][i];
                                    accf[o][cg][i] = 0.0f;
                                }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_xfull + 8 * dw);
                        ++piece;
                        continue;
                    }
                    if (!warp_wait(bar_xfull + 8 * dw, piece & 1, abort_flag, p.status)) { ok = false; break; }
#pragma unroll
                    for (int o = 0; o < MO; ++o)
#pragma unroll
                        for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                            for (int i = 0; i < 4; ++i) accf[o][cg][i] += xch[((o * CG + cg) * 4 + i) * 32];
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_xempty + 8 * dw);
                }
                const uint32_t u_tile0 = tn * KT;
                const uint32_t piece_k0 = max(u_tile0, u_begin) - u_tile0;
                const bool full_piece = (piece_k0 == 0) && (kt == KT - 1);
                bool write_y = full_piece;
                if (!full_piece) {
                    // Split tile.  Every warp settles its own 32-column strip, without CTA-wide
                    // barriers: FP32 partial in fragment order, then one arrival per (tile, strip);
                    // the last warp to arrive adds the partials in CTA order (the same order in
                    // every run) and writes Y.
                    const uint32_t which = (p.split || u_begin / KT == tn) ? 0u : 1u;
                    float* slot = p.partials + ((size_t)blockIdx.x * 2 + which) * (size_t)(BN * LDC) + dw * (32 * LDC) + lane;
#pragma unroll
                    for (int o = 0; o < MO; ++o)
#pragma unroll
                        for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                            for (int i = 0; i < 4; ++i) __stcg(slot + ((o * CG + cg) * 4 + i) * 32, accf[o][cg][i]);
                    __syncwarp();
                    const uint32_t c_first = p.split ? tn * p.split : cta_of_unit(u_tile0, q, r);
                    const uint32_t c_last = p.split ? c_first + p.split - 1 : cta_of_unit(u_tile0 + KT - 1, q, r);
                    uint32_t last = 0;
                    if (lane == 0) {
                        // one arrival, release and acquire at GPU scope: the warp's stores (ordered before
                        // this lane by the __syncwarp above) precede it, and the warp that finds itself last
                        // sees the stores of all contributors that arrived before
                        uint32_t old;
                        asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(old) : "l"(p.counters + tn * NDW + dw) : "memory");
                        last = (old == c_last - c_first) ? 1u : 0u;
                    }
                    last = __shfl_sync(0xffffffffu, last, 0);
                    __syncwarp();
                    if (last) {
                        write_y = true;
#pragma unroll
                        for (int o = 0; o < MO; ++o)
#pragma unroll
                            for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                                for (int i = 0; i < 4; ++i) accf[o][cg][i] = 0.0f;
                        // ND contributors' loads in flight at a time (more where the registers allow it:
                        // the short jobs, whose time is mostly such round trips); the additions keep CTA order
                        constexpr int ND = (MO == 1 && NGRP == 1) ? 8 : (kTight ? 2 : 4);
                        for (uint32_t c = c_first; c <= c_last; c += ND) {
                            float v[ND][MO * CG * 4];
#pragma unroll
                            for (int d = 0; d < ND; ++d) {
                                const uint32_t cc = min(c + d, c_last);
                                const uint32_t wch = (p.split || unit_begin_of(cc, q, r) / KT == tn) ? 0u : 1u;
                                const float* sl = p.partials + ((size_t)cc * 2 + wch) * (size_t)(BN * LDC) + dw * (32 * LDC) + lane;
#pragma unroll
                                for (int e = 0; e < MO * CG * 4; ++e) v[d][e] = __ldcg(sl + e * 32);
                            }
#pragma unroll
                            for (int d = 0; d < ND; ++d)
                                if (c + d <= c_last) {
#pragma unroll
                                    for (int o = 0; o < MO; ++o)
#pragma unroll
                                        for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                                            for (int i = 0; i < 4; ++i) accf[o][cg][i] += v[d][(o * CG + cg) * 4 + i];
                                }
                        }
                        if (lane == 0) p.counters[tn * NDW + dw] = 0;  // ready for the next call
                    }
                }
                if (write_y) {
#pragma unroll
                    for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                        for (int h = 0; h < 2; ++h)
#pragma unroll
                            for (int o = 0; o < MO; ++o)
#pragma unroll
                                for (int j = 0; j < 2; ++j) {
                                    const uint32_t m = o * 8 + 2 * t + j;
                                    if (m < p.M)
                                        p.Y[(size_t)m * p.N + (size_t)tn * BN + c0 + 16 * cg + 8 * h] = float_to_bf16_bits(accf[o][cg][2 * h + j]);
                                }
                }
#pragma unroll
                for (int o = 0; o < MO; ++o)
#pragma unroll
                    for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                        for (int i = 0; i < 4; ++i) accf[o][cg][i] = 0.0f;
                ++piece;
          }
        }
    }
}
