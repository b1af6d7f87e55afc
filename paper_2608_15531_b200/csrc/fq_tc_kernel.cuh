// The fused operator on the fifth-generation tensor cores (tcgen05.mma, operands in tensor memory).
// Included by fq_kernels.cu inside namespace fq, after the PTX helpers.
//
// A unit is one (column tile, 128-row k-step): 128 x BN INT4 codes with their scales, zero-points and
// Tile-COO slice.  One persistent CTA per SM walks a range of units through a ring of shared-memory
// stages (cp.async.bulk + mbarrier expect_tx, Section 4.1).  Thread = output column throughout: tensor
// memory lane c of a 128-column half holds row c of the A operand (the column's 128 dequantised
// codes) and row c of the accumulator D (the column's batch rows).
//
//   warp 0          producer: bulk copies of codes and scales (and zero-points in kernels with outliers)
//   warp 1          tensor: owns the tensor-memory allocation; per unit 8 x BN/128 tcgen05.mma
//                   (M = 128 columns, N = NMMA batch rows, K = 16; A from tensor memory, B = activations
//                   from shared memory, D = FP32 in tensor memory), tcgen05.commit to mbarriers
//   warps 2..3      activations (alternate units): the unit's block of X from global memory (L2) as the
//                   K-major MMA operand + per-group row sums + a k-major FP32 copy for the outlier step;
//                   they also request the unit's bucket descriptors and packets (or its zero-points)
//   unpack warps    BN/32: per 32 rows one 128-bit load of 32 codes, lop3/shift to 16 BF16 pairs 128 + q
//                   (exact integers), tcgen05.st into the A operand
//   epilogue warps  BN/32: tcgen05.ld of the group sums, acc += s * (sum x (128+q) - (128+z) sum x) in
//                   FP32 (Eq. 3 inside Eq. 1), then the unit's outliers of the thread's own column
//                   straight into the same registers (Section 4.2 without the shared-memory scatter:
//                   no atomics, no read-modify-write), and at the end of a piece the split-tile
//                   settlement and the BF16 store of Y
//
// Lane l of an epilogue warp owns column 32 * strip + l = 8 t + g with g = l % 8, t = l / 8: bucket g of
// the strip, column number t of that bucket, so it takes slot t of every column-slotted packet of the
// bucket.  The k-major FP32 copy xt[k][RR] is stored with its 16-byte chunks XOR-swizzled by k
// (Section 3.2.2's concern, shared-memory bank conflicts of the sparse step, met on the activation side:
// the rows a warp's lanes pick are random, and the swizzle spreads them over all eight 16-byte bank groups).

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// N consecutive FP32 cells of this thread's tensor-memory lane (N = 1, 4, 8, 16 or 32)
template <int N>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, float (&d)[N]) {
    uint32_t r[N];
    if constexpr (N == 1) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r[0]) : "r"(taddr) : "memory");
    } else if constexpr (N == 4) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
    } else if constexpr (N == 8) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                     : "r"(taddr) : "memory");
    } else if constexpr (N == 16) {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
              "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
            : "r"(taddr) : "memory");
    } else {
        static_assert(N == 32, "unsupported tcgen05.ld width");
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
            "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
              "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
              "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
              "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
            : "r"(taddr) : "memory");
    }
    tmem_wait_ld();
#pragma unroll
    for (int i = 0; i < N; ++i) d[i] = __uint_as_float(r[i]);
}

// XOR applied to the 16-byte chunk index of row k of the k-major FP32 copy (RR floats per row): with C
// chunks per row, 8 / C consecutive rows share a 128-byte line, and the swizzle makes the chunk a lane
// reads in one load instruction depend on k, so that lanes with random k cover all eight bank groups.
template <int RR>
__device__ __forceinline__ uint32_t xt_swizzle(uint32_t k) {
    constexpr uint32_t C = RR / 4;
    if constexpr (C <= 1) return 0u;
    else return ((k * C) >> 3) & (C - 1);
}

// acc[0..RR) += v * x[0..RR)[k] for NP outliers of the thread's column, each a slot word (BF16 value in the
// upper half, row k of the unit in bits 5-11; a padding slot has value 0 and adds 0).  The activation rows
// of all NP are requested before the first multiply-add, so that their shared-memory latencies overlap.
template <int RR, int NP>
__device__ __forceinline__ void add_outliers(float (&acc)[RR], const uint32_t (&wd)[NP], const char* xtb) {
    if constexpr (RR == 1) {
        float x[NP];
#pragma unroll
        for (int j = 0; j < NP; ++j) x[j] = *reinterpret_cast<const float*>(xtb + ((wd[j] >> 3) & 0x1fcu));
#pragma unroll
        for (int j = 0; j < NP; ++j) acc[0] = fmaf(__uint_as_float(wd[j] & 0xffff0000u), x[j], acc[0]);
    } else {
        float4 x[NP][RR / 4];
#pragma unroll
        for (int j = 0; j < NP; ++j) {
            const uint32_t k = (wd[j] >> 5) & 127u;
            const char* row = xtb + k * (4 * RR);
            const uint32_t sw = xt_swizzle<RR>(k) << 4;
#pragma unroll
            for (int c = 0; c < RR / 4; ++c) x[j][c] = *reinterpret_cast<const float4*>(row + (((uint32_t)c << 4) ^ sw));
        }
#pragma unroll
        for (int j = 0; j < NP; ++j) {
            const float v = __uint_as_float(wd[j] & 0xffff0000u);
#pragma unroll
            for (int c = 0; c < RR / 4; ++c) {
                acc[4 * c + 0] = fmaf(v, x[j][c].x, acc[4 * c + 0]);
                acc[4 * c + 1] = fmaf(v, x[j][c].y, acc[4 * c + 1]);
                acc[4 * c + 2] = fmaf(v, x[j][c].z, acc[4 * c + 2]);
                acc[4 * c + 3] = fmaf(v, x[j][c].w, acc[4 * c + 3]);
            }
        }
    }
}

// The k-major FP32 copy xt[k][RR] (swizzled, see xt_swizzle) of the first RR batch rows of a unit, built
// from the K-major MMA operand in shared memory (8-row x 16-byte core matrices; core matrix (chunk c,
// octet o) at (c * nmma8 + o) * 128).  RR >= 4; whole warp.
template <int RR>
__device__ __forceinline__ void build_xt(uint32_t xb_addr, uint32_t nmma8, char* xt, int lane) {
    constexpr int NO = RR >= 8 ? RR / 8 : 1;
    const uint32_t pr = lane & 3;
#pragma unroll
    for (int o = 0; o < NO; ++o) {
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
            uint32_t r[4];
            const uint32_t chunk = kb * 4 + (lane >> 3);
            ldmatrix_x4_trans(xb_addr + (chunk * nmma8 + o) * 128 + (lane & 7) * 16, r[0], r[1], r[2], r[3]);
            // this thread now holds rows m = 8 o + 2 pr, 2 pr + 1 of k = 8 (4 kb + i) + lane / 4, i = 0..3
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t k = (kb * 4 + i) * 8 + (lane >> 2);
                if constexpr (RR == 4) {
                    if (pr < 2) *reinterpret_cast<float2*>(xt + k * 16 + pr * 8) = make_float2(bf16lo(r[i]), bf16hi(r[i]));
                } else {
                    const uint32_t cl = 2 * o + (pr >> 1);
                    *reinterpret_cast<float2*>(xt + k * (4 * RR) + ((cl ^ xt_swizzle<RR>(k)) << 4) + (pr & 1) * 8) =
                        make_float2(bf16lo(r[i]), bf16hi(r[i]));
                }
            }
        }
    }
}

constexpr int kTcActWarps = 4;

// BN: tile columns (128 or 256).  NMMA: batch columns of the MMA (16 or 32).  RR: batch rows kept per
// epilogue thread (1, 4, 8, 16, 32; M <= RR <= NMMA).  HOT: general form of the outlier step (buckets
// with a tail, tiles with more packets than a stage holds).
template <int BN, int NMMA, int RR, int GROUP, bool SPARSE, bool HOT>
__global__ void __launch_bounds__(32 * (2 + kTcActWarps + 2 * (BN / 32)), 1) fq_tc_kernel(const Params p) {
    constexpr int NDW = BN / 32;              // unpack warps = epilogue warps = 32-column strips
    constexpr int NT128 = BN / 128;           // 128-column halves per unit
    constexpr int NAW = kTcActWarps;         // activation warps launched; the first p.nact of them work
    constexpr int UW0 = 2 + NAW, EW0 = UW0 + NDW;
    constexpr int GPS = kBK / GROUP;          // groups per k-step
    constexpr int DCOLS = GPS * NMMA;         // accumulator columns per half and buffer
    constexpr uint32_t D_BASE = 2 * NT128 * 64;
    constexpr int W_BYTES = 16 * BN * 4;
    constexpr int SZ_ROW = BN * 2;
    constexpr int NMMA8 = NMMA / 8;
    constexpr bool kActZero = !SPARSE;        // who requests the zero-points: the activation warp, if it has no outlier arrays to request
    constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NMMA >> 3) << 17) | (8u << 24);
    static_assert(D_BASE + 2 * NT128 * DCOLS <= 512, "tensor memory: two A buffers and two D buffers must fit");
    static_assert(RR <= NMMA && (RR == 1 || RR % 4 == 0), "rows per thread");
    static_assert(RR > 8 || NMMA == 16, "up to eight rows: the MMA's second octet of rows is zero padding");
    extern __shared__ __align__(128) uint8_t smem[];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t S = p.stages;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * S;
    const uint32_t bar_go = bar_empty + 8 * S;           // [2] A buffer written (unpack warps) and D buffer free (epilogue warps)
    const uint32_t bar_d_ready = bar_go + 16;            // [2] MMAs of a unit complete (D written, A read)
    const uint32_t bar_final = bar_d_ready + 16;
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 2 * S + 5);
    volatile uint32_t* tmem_slot = abort_flag + 1;

    if (tid == 0) {
        for (uint32_t s = 0; s < S; ++s) {
            mbar_init(bar_full + 8 * s, 2);                    // producer's expect_tx arrival + activation warp
            mbar_init(bar_empty + 8 * s, 2 * NDW + 1);         // unpack warps, epilogue warps, the MMAs' commit
        }
        for (uint32_t b = 0; b < 2; ++b) {
            mbar_init(bar_go + 8 * b, 2 * NDW);                // unpack warps (A of this unit), epilogue warps (D of the unit two before)
            mbar_init(bar_d_ready + 8 * b, 1);
        }
        mbar_init(bar_final, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (RR <= 8) {
        // batch rows 8..15 of the MMA operand are never written by the activation warps: zero them once
        for (uint32_t i = tid; i < S * 16 * 8; i += blockDim.x) {
            const uint32_t s = i >> 7, c = (i >> 3) & 15, r = i & 7;
            *reinterpret_cast<uint4*>(smem + s * p.stage_bytes + p.off_xcan + (c * NMMA8 + 1) * 128 + r * 16) = make_uint4(0, 0, 0, 0);
        }
    }
    if (warp == 1) {
        tmem_alloc(smem_u32((const void*)tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // The grid after this one in the stream may start now (it takes SMs as this grid's CTAs leave).  The
    // warps that touch X, Y or the scratch wait for the grid before this one; the producer reads only
    // weights, which no kernel writes while calls are in flight.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (warp >= EW0) asm volatile("griddepcontrol.wait;" ::: "memory");

    const uint32_t KT = p.KT;
    const uint32_t U = p.NT * KT, P = gridDim.x, q = U / P, r = U % P;
    uint32_t u_begin, u_end;
    if (p.split) {
        const uint32_t tile = blockIdx.x / p.split, part = blockIdx.x - tile * p.split;
        u_begin = tile * KT + part * KT / p.split;
        u_end = tile * KT + (part + 1) * KT / p.split;
    } else {
        u_begin = unit_begin_of(blockIdx.x, q, r);
        u_end = u_begin + q + (blockIdx.x < r ? 1u : 0u);
    }

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        uint32_t issued = 0;
        bool ok = true;
        for (UnitIter w(u_begin, KT); w.u < u_end; w.next(S, KT)) {
            const uint32_t s = w.s;
            if (!warp_wait(bar_empty + 8 * s, w.ph ^ 1, abort_flag, p.status)) { ok = false; break; }
            const uint32_t full = bar_full + 8 * s;
            const uint32_t st = smem_u32(smem) + s * p.stage_bytes;
            if (lane == 0) mbar_arrive_expect_tx(full, W_BYTES + (kActZero ? 1 : 2) * GPS * SZ_ROW);
            __syncwarp();
            // one copy per lane: issuing a bulk copy occupies its thread for a few hundred cycles
            if (lane == 0) {
                bulk_g2s(st, p.wq + (size_t)w.u * W_BYTES, W_BYTES, full);
            } else if (lane <= GPS) {
                const int gi = lane - 1;
                bulk_g2s(st + p.off_sz + gi * SZ_ROW, p.scale + (size_t)(w.kt * GPS + gi) * p.N + (size_t)w.tn * BN, SZ_ROW, full);
            } else if (!kActZero && lane <= 2 * GPS) {
                const int gi = lane - 1 - GPS;
                bulk_g2s(st + p.off_sz + (GPS + gi) * SZ_ROW, p.zero + (size_t)(w.kt * GPS + gi) * p.N + (size_t)w.tn * BN, SZ_ROW, full);
            }
            issued = w.it + 1;
        }
        if (!ok) {   // giving up: let the copies already issued land before the CTA's shared memory goes away
            for (uint32_t j = (issued > S ? issued - S : 0); j < issued; ++j)
                for (uint32_t spin = 0; spin < (1u << 20) && !mbar_try_wait(bar_full + 8 * (j % S), (j / S) & 1); ++spin) {}
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ tensor warp
        // The whole warp runs the loop with warp-uniform operands; one elected lane issues each instruction.
        // The first MMA of a CTA takes microseconds to start (the tensor pipe wakes up): issue a throw-away
        // one now, while the first loads are in flight.  It reads whatever A buffer 0 and stage 0 hold and
        // writes D buffer 1, which the first real MMA into that buffer overwrites.
        umma_ts(tmem_base + D_BASE + NT128 * DCOLS, tmem_base, make_b_desc(smem_u32(smem) + p.off_xcan, NMMA8 * 128, 128), IDESC, 0);
        for (UnitIter w(u_begin, KT); w.u < u_end; w.next(S, KT)) {
            const uint32_t it = w.it, s = w.s, b = w.it & 1;
            if (!warp_wait(bar_full + 8 * s, w.ph, abort_flag, p.status)) break;       // the activation operand
            if (!warp_wait(bar_go + 8 * b, (it >> 1) & 1, abort_flag, p.status)) break;
            tc_fence_after();
            const uint64_t bd0 = make_b_desc(smem_u32(smem) + s * p.stage_bytes + p.off_xcan, NMMA8 * 128, 128);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const int gi = ks / (8 / GPS);
#pragma unroll
                for (int h = 0; h < NT128; ++h) {
                    const uint32_t d = tmem_base + D_BASE + (b * NT128 + h) * DCOLS + gi * NMMA;
                    const uint32_t a = tmem_base + (b * NT128 + h) * 64 + ks * 8;
                    umma_ts(d, a, bd0 + (uint64_t)((ks * 2 * NMMA8 * 128) >> 4), IDESC, (ks % (8 / GPS)) != 0);
                }
            }
            umma_commit(bar_d_ready + 8 * b);   // this unit's sums are complete and its A buffer has been read
            umma_commit(bar_empty + 8 * s);     // and so has the stage's activation operand
        }
        __syncwarp();
        umma_commit(bar_final);                 // fires when every MMA this warp issued has retired
    } else if (warp < UW0) {
        // ------------------------------------------------------------------ activation warps
        const uint32_t aw = warp - 2, NA = p.nact;           // the ring length is a multiple of NA: a stage always returns to the same warp
        constexpr int ROWS = RR <= 8 ? 8 : NMMA;             // rows this warp lays out (rows 8..15 stay zero if RR <= 8)
        constexpr int LPR = 32 / ROWS;                       // lanes per row: 4, 2 or 1
        constexpr int CPL = 16 / LPR;                        // 16-byte chunks per lane
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
        uint32_t ip_nxt = 0, ip_nxt_end = 0, last_bar = 0, last_ph = 0;
        bool ok = true;
        auto load_ip = [&](uint32_t u) {
            if (SPARSE && lane == 0) { ip_nxt = __ldg(p.indptr + u); ip_nxt_end = __ldg(p.indptr + u + 1); }
        };
        // this warp's share of the weight arrays of unit u: bucket descriptors and packets, or the zero-points
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
            // The first pass over the ring finds every stage empty, and these arrays are weights: lane l
            // requests those of this warp's l-th unit before the wait for the previous grid.
            const uint32_t it0 = aw + NA * lane;
            if (aw < NA && it0 < min(S, u_end - u_begin)) {
                const uint32_t u = u_begin + it0, tn = u / KT;
                uint32_t a = 0, npk = 0;
                if (SPARSE) { a = __ldg(p.indptr + u); npk = min(__ldg(p.indptr + u + 1) - a, p.coo_cap); }
                request(u, tn, u - tn * KT, smem_u32(smem) + it0 * p.stage_bytes, bar_full + 8 * it0, a, npk);
            }
            __syncwarp();
            asm volatile("griddepcontrol.wait;" ::: "memory");
        }
        if (aw < NA && u_begin + aw < u_end) { load((u_begin + aw) % KT); load_ip(u_begin + aw); }
        for (UnitIter w(u_begin, KT); aw < NA && w.u < u_end; w.next(S, KT)) {
            if (w.it % NA != aw) continue;
            const uint32_t s = w.s, ph = w.ph;
            uint8_t* st = smem + s * p.stage_bytes;
            uint4 xv[CPL];
#pragma unroll
            for (int c = 0; c < CPL; ++c) xv[c] = nxt[c];
            const uint32_t ip = ip_nxt, npk = min(ip_nxt_end - ip_nxt, p.coo_cap);
            if (w.u + NA < u_end) { uint32_t kn = w.kt + NA; load(kn >= KT ? kn % KT : kn); load_ip(w.u + NA); }
            if (!warp_wait(bar_empty + 8 * s, ph ^ 1, abort_flag, p.status)) { ok = false; break; }
            last_bar = bar_full + 8 * s, last_ph = ph;
            if (lane == 0 && w.it >= S) request(w.u, w.tn, w.kt, smem_u32(st), bar_full + 8 * s, ip, npk);
            // K-major MMA operand: core matrix (chunk c, octet o) at (c * NMMA8 + o) * 128, row m % 8 at + 16 (m % 8)
            uint8_t* dst = st + p.off_xcan + ((part * CPL) * NMMA8 + (m >> 3)) * 128 + (m & 7) * 16;
            float sum = 0.0f, sum_lo = 0.0f;          // sum_lo: chunks 0-7 where a lane holds a whole row
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                const uint4 v = xv[c];
                *reinterpret_cast<uint4*>(dst + c * NMMA8 * 128) = v;
                if (LPR == 1 && c == 8) sum_lo = sum, sum = 0.0f;
                sum += (bf16lo(v.x) + bf16hi(v.x)) + (bf16lo(v.y) + bf16hi(v.y)) + (bf16lo(v.z) + bf16hi(v.z)) +
                       (bf16lo(v.w) + bf16hi(v.w));
            }
            // per-group sums of each row -> xsum[group][NMMA]
            float* xsum = reinterpret_cast<float*>(st + p.off_xsum);
            if (LPR == 4) {
                const float s1 = sum + __shfl_xor_sync(0xffffffffu, sum, 8);       // parts {0,1} and {2,3}
                const float s2 = s1 + __shfl_xor_sync(0xffffffffu, s1, 16);
                if (GPS == 2) { if ((part & 1) == 0) xsum[(part >> 1) * NMMA + m] = s1; }
                else if (part == 0) xsum[m] = s2;
            } else if (LPR == 2) {
                const float s1 = sum + __shfl_xor_sync(0xffffffffu, sum, 16);
                if (GPS == 2) xsum[part * NMMA + m] = sum;
                else if (part == 0) xsum[m] = s1;
            } else {
                if (GPS == 2) xsum[m] = sum_lo, xsum[NMMA + m] = sum;
                else xsum[m] = sum_lo + sum;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the operand is read by the tensor core
            __syncwarp();
            if (SPARSE) {
                char* xt = reinterpret_cast<char*>(st + p.off_xt);
                if constexpr (RR == 1) {
                    if (m == 0) {
                        float4* xt4 = reinterpret_cast<float4*>(xt) + part * CPL * 2;
#pragma unroll
                        for (int c = 0; c < CPL; ++c) {
                            xt4[2 * c] = make_float4(bf16lo(xv[c].x), bf16hi(xv[c].x), bf16lo(xv[c].y), bf16hi(xv[c].y));
                            xt4[2 * c + 1] = make_float4(bf16lo(xv[c].z), bf16hi(xv[c].z), bf16lo(xv[c].w), bf16hi(xv[c].w));
                        }
                    }
                } else {
                    build_xt<RR>(smem_u32(st + p.off_xcan), NMMA8, xt, lane);
                }
                __syncwarp();
            }
            if (lane == 0) mbar_arrive(bar_full + 8 * s);
        }
        if (!ok && last_bar)                // gave up: let this warp's last copies land before the CTA exits
            for (uint32_t spin = 0; spin < (1u << 20) && !mbar_try_wait(last_bar, last_ph); ++spin) {}
    } else if (warp < EW0) {
        // ------------------------------------------------------------------ unpack warps: thread = column
        const int dw = warp - UW0;
        const uint32_t t_lane = ((uint32_t)((dw & 3) * 32)) << 16;
        const uint32_t t_a = tmem_base + t_lane + (uint32_t)(dw >> 2) * 64;
        for (UnitIter w(u_begin, KT); w.u < u_end; w.next(S, KT)) {
            const uint32_t it = w.it, s = w.s, b = w.it & 1;
            if (!warp_wait(bar_full + 8 * s, w.ph, abort_flag, p.status)) break;
            // the A buffer of this parity was last read by the MMAs of unit it - 2
            if (it >= 2 && !warp_wait(bar_d_ready + 8 * b, ((it - 2) >> 1) & 1, abort_flag, p.status)) break;
            tc_fence_after();
            // the column's 128 codes: four 16-byte loads (32 rows each), lanes contiguous
            const uint4* wp = reinterpret_cast<const uint4*>(smem + s * p.stage_bytes) + dw * 32 + lane;
            uint4 w4 = wp[0];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint4 cur = w4;
                if (j < 3) w4 = wp[(j + 1) * BN];
                const uint32_t ww[4] = {cur.x, cur.y, cur.z, cur.w};
                uint32_t a[16];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    a[4 * x + 0] = codes_to_bf16x2(ww[x]);
                    a[4 * x + 1] = codes_to_bf16x2(ww[x] >> 4);
                    a[4 * x + 2] = codes_to_bf16x2(ww[x] >> 8);
                    a[4 * x + 3] = codes_to_bf16x2(ww[x] >> 12);
                }
                tmem_st16(t_a + b * (NT128 * 64) + j * 16, a);
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive_relaxed(bar_go + 8 * b);
                mbar_arrive_relaxed(bar_empty + 8 * s);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps: thread = column
        const int dw = warp - EW0;
        const int col = dw * 32 + lane;
        const uint32_t g = lane & 7, t = lane >> 3;          // bucket of the strip, column number in the bucket
        const uint32_t t_lane = ((uint32_t)((dw & 3) * 32)) << 16;
        const uint32_t t_d = tmem_base + t_lane + D_BASE + (uint32_t)(dw >> 2) * DCOLS;
        float accf[RR];
#pragma unroll
        for (int i = 0; i < RR; ++i) accf[i] = 0.0f;
        bool ok = true;
        // both D buffers start free: this warp's share of the first two units' go-ahead
        if (lane == 0) { mbar_arrive_relaxed(bar_go); mbar_arrive_relaxed(bar_go + 8); }
        for (UnitIter w(u_begin, KT); w.u < u_end && ok; w.next(S, KT)) {
            const uint32_t u = w.u, it = w.it, s = w.s, b = w.it & 1;
            const uint32_t tn = w.tn, kt = w.kt;
            const uint8_t* st = smem + s * p.stage_bytes;
            if (!warp_wait(bar_full + 8 * s, w.ph, abort_flag, p.status)) { ok = false; break; }
            // outliers: the bucket descriptor and this lane's slot of the first packet are requested now
            uint32_t sp_off = 0, sp_cnt = 0, sp_tail = 0, cmax = 0;
            constexpr int NP = RR <= 16 ? 2 : 1;                     // packet rounds in flight
            uint32_t pk[NP];
            const uint32_t* pk_s = reinterpret_cast<const uint32_t*>(st + p.off_coo);
            const uint32_t* pk_g = nullptr;
            const char* xtb = reinterpret_cast<const char*>(st + p.off_xt);
            if (SPARSE) {
                const uint32_t info = reinterpret_cast<const uint32_t*>(st + p.off_info)[dw * 8 + g];
                sp_off = info & 0xffffu;
                sp_cnt = (info >> 16) & 0xffu;
                if (HOT) {
                    sp_tail = info >> 24;
                    if (__reduce_max_sync(0xffffffffu, sp_off + sp_cnt + sp_tail) > p.coo_cap)
                        pk_g = reinterpret_cast<const uint32_t*>(p.packed + __ldg(p.indptr + u));   // packets beyond the staged part
                } else if (__any_sync(0xffffffffu, sp_off + sp_cnt > p.coo_cap)) {
                    // a descriptor that does not belong to the staged packets (layout struct and arrays
                    // out of step): report it and skip the unit's outliers instead of reading past the stage
                    if (lane == 0) atomicExch(p.status, (uint32_t)FQ_ERR_FORMAT);
                    sp_cnt = 0;
                }
                cmax = __reduce_max_sync(0xffffffffu, sp_cnt);
            }
            auto slot_word = [&](uint32_t idx) -> uint32_t {           // word t of packet idx of the tile
                if (!HOT || idx < p.coo_cap) return pk_s[idx * 4 + t];
                return __ldg(pk_g + idx * 4 + t);
            };
#pragma unroll
            for (int j = 0; j < NP; ++j) pk[j] = (SPARSE && (uint32_t)j < sp_cnt) ? slot_word(sp_off + j) : 0u;
            // the unit's sums, once its MMAs are complete
            if (!warp_wait(bar_d_ready + 8 * b, (it >> 1) & 1, abort_flag, p.status)) { ok = false; break; }
            tc_fence_after();
            const uint16_t* sc = reinterpret_cast<const uint16_t*>(st + p.off_sz);
            const float* xsum = reinterpret_cast<const float*>(st + p.off_xsum);
#pragma unroll
            for (int gi = 0; gi < GPS; ++gi) {
                const float sv = bf16_bits_to_float(sc[gi * BN + col]);
                const float zc = -(128.0f + bf16_bits_to_float(sc[(GPS + gi) * BN + col]));
                float d[RR];
                tmem_ld<RR>(t_d + b * (NT128 * DCOLS) + gi * NMMA, d);
                if constexpr (RR == 1) {
                    accf[0] = fmaf(sv, fmaf(zc, xsum[gi * NMMA], d[0]), accf[0]);
                } else {
#pragma unroll
                    for (int i = 0; i < RR / 4; ++i) {
                        const float4 xs = *reinterpret_cast<const float4*>(xsum + gi * NMMA + 4 * i);
                        accf[4 * i + 0] = fmaf(sv, fmaf(zc, xs.x, d[4 * i + 0]), accf[4 * i + 0]);
                        accf[4 * i + 1] = fmaf(sv, fmaf(zc, xs.y, d[4 * i + 1]), accf[4 * i + 1]);
                        accf[4 * i + 2] = fmaf(sv, fmaf(zc, xs.z, d[4 * i + 2]), accf[4 * i + 2]);
                        accf[4 * i + 3] = fmaf(sv, fmaf(zc, xs.w, d[4 * i + 3]), accf[4 * i + 3]);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_relaxed(bar_go + 8 * b);         // the MMAs of unit it + 2 may overwrite this D buffer
            if (SPARSE) {
                // ---- the unit's outliers of this thread's column (padding slots have value 0: they add 0)
                for (uint32_t i = 0; i < cmax; i += NP) {
                    uint32_t nx[NP];                               // the next rounds' slots, requested before this round's math
#pragma unroll
                    for (int j = 0; j < NP; ++j) nx[j] = (i + NP + j < sp_cnt) ? slot_word(sp_off + i + NP + j) : 0u;
                    add_outliers<RR, NP>(accf, pk, xtb);
#pragma unroll
                    for (int j = 0; j < NP; ++j) pk[j] = nx[j];
                }
                if (HOT) {
                    // a bucket with a tail: its packets (slots name their column) are shared out over the eight
                    // lane groups g, each adding into sums of its own that are added up over g afterwards
                    for (uint32_t hot = __ballot_sync(0xffffffffu, sp_tail != 0); hot; ) {     // warp-uniform
                        const uint32_t hot_lane = __ffs(hot) - 1;
                        hot &= ~(0x01010101u << (hot_lane & 7u));
                        const uint32_t hot_off = __shfl_sync(0xffffffffu, sp_off + sp_cnt, hot_lane);
                        const uint32_t hot_cnt = __shfl_sync(0xffffffffu, sp_tail, hot_lane);
                        float hacc[RR];
#pragma unroll
                        for (int ri = 0; ri < RR; ++ri) hacc[ri] = 0.0f;
                        for (uint32_t i = g; i < hot_cnt; i += 8) {
                            const uint32_t idx = hot_off + i;
                            const uint4 pk = (idx < p.coo_cap) ? reinterpret_cast<const uint4*>(pk_s)[idx]
                                                               : __ldg(reinterpret_cast<const uint4*>(pk_g) + idx);
                            const uint32_t wd[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                // a tail slot names its column: slots of other columns count as padding (value 0)
                                const uint32_t mine[1] = {((wd[e] >> 12) & 3u) == t ? wd[e] : (wd[e] & 0xffffu)};
                                add_outliers<RR, 1>(hacc, mine, xtb);
                            }
                        }
#pragma unroll
                        for (int ri = 0; ri < RR; ++ri) {
                            float v = hacc[ri];
                            v += __shfl_xor_sync(0xffffffffu, v, 1);
                            v += __shfl_xor_sync(0xffffffffu, v, 2);
                            v += __shfl_xor_sync(0xffffffffu, v, 4);
                            if (g == (hot_lane & 7u)) accf[ri] += v;
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive_relaxed(bar_empty + 8 * s);

            if (kt == KT - 1 || u == u_end - 1) {
                // ---------------------------------------------------------- end of a piece
                const uint32_t u_tile0 = tn * KT;
                const uint32_t piece_k0 = max(u_tile0, u_begin) - u_tile0;
                const bool full_piece = (piece_k0 == 0) && (kt == KT - 1);
                bool write_y = full_piece;
                if (!full_piece) {
                    // Split tile.  Every warp settles its own 32-column strip, without CTA-wide barriers: FP32
                    // partial [row][column], then one arrival per (tile, strip); the last warp to arrive adds
                    // the partials in CTA order (the same order in every run) and writes Y.
                    const uint32_t which = (p.split || u_begin / KT == tn) ? 0u : 1u;
                    float* slot = p.partials + ((size_t)blockIdx.x * 2 + which) * (size_t)(BN * RR) + col;
#pragma unroll
                    for (int mm = 0; mm < RR; ++mm) __stcg(slot + mm * BN, accf[mm]);
                    __syncwarp();
                    const uint32_t c_first = p.split ? tn * p.split : cta_of_unit(u_tile0, q, r);
                    const uint32_t c_last = p.split ? c_first + p.split - 1 : cta_of_unit(u_tile0 + KT - 1, q, r);
                    uint32_t last = 0;
                    if (lane == 0) {
                        // one arrival, release and acquire at GPU scope: the warp's stores (ordered before this
                        // lane by the __syncwarp above) precede it, and the warp that finds itself last sees the
                        // stores of all contributors that arrived before
                        uint32_t old;
                        asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(old) : "l"(p.counters + tn * NDW + dw) : "memory");
                        last = (old == c_last - c_first) ? 1u : 0u;
                    }
                    last = __shfl_sync(0xffffffffu, last, 0);
                    __syncwarp();
                    if (last) {
                        write_y = true;
#pragma unroll
                        for (int mm = 0; mm < RR; ++mm) accf[mm] = 0.0f;
                        constexpr int ND = RR <= 4 ? 8 : (RR <= 8 ? 4 : 2);       // contributors' loads in flight
                        for (uint32_t c = c_first; c <= c_last; c += ND) {
                            float v[ND][RR];
#pragma unroll
                            for (int dd = 0; dd < ND; ++dd) {
                                const uint32_t cc = min(c + dd, c_last);
                                const uint32_t wch = (p.split || unit_begin_of(cc, q, r) / KT == tn) ? 0u : 1u;
                                const float* sl = p.partials + ((size_t)cc * 2 + wch) * (size_t)(BN * RR) + col;
#pragma unroll
                                for (int mm = 0; mm < RR; ++mm) v[dd][mm] = __ldcg(sl + mm * BN);
                            }
#pragma unroll
                            for (int dd = 0; dd < ND; ++dd)
                                if (c + dd <= c_last) {
#pragma unroll
                                    for (int mm = 0; mm < RR; ++mm) accf[mm] += v[dd][mm];
                                }
                        }
                        if (lane == 0) p.counters[tn * NDW + dw] = 0;  // ready for the next call
                    }
                }
                if (write_y) {
#pragma unroll
                    for (int mm = 0; mm < RR; ++mm)
                        if ((uint32_t)mm < p.M) p.Y[(size_t)mm * p.N + (size_t)tn * BN + col] = float_to_bf16_bits(accf[mm]);
                }
#pragma unroll
                for (int mm = 0; mm < RR; ++mm) accf[mm] = 0.0f;
            }
        }
    }

    // ---------------------------------------------------------------------- common exit
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        // every tcgen05 operation of this CTA must have retired before its tensor memory is released
        for (uint32_t spin = 0; spin < (1u << 24) && !mbar_try_wait(bar_final, 0); ++spin) {}
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}
