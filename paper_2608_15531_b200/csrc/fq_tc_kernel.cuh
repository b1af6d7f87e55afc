// The fused operator on the fifth-generation tensor cores (tcgen05.mma kind::i8, operands in tensor memory).
// Included by fq_kernels.cu inside namespace fq, after the PTX helpers.
//
// Arithmetic.  The tensor core multiplies 8-bit integers exactly: the INT4 codes q go in as they are, and the
// BF16 activations go in as block fixed point.  For every batch row and quantisation group (64 or 128 k) a
// small kernel (fq_prep_x_kernel) writes x as an integer x_int = round(x * 2^(21-E)) (E = exponent of the
// group's largest |x|, so |x_int| < 2^22: exact for every element within 2^14 of the largest, rounded to 2^-22
// of the largest below that), split into three signed 8-bit limbs x_int = l0 + 2^8 l1 + 2^16 l2, together with
// 2^(E-21), sum_k x_int and a k-major FP32 copy of x for the outlier step.  Then
//     sum_k x (q - z)  =  2^(E-21) * ( sum_j 2^(8j) sum_k q l_j  -  z sum_k x_int )            (Eq. 3 inside Eq. 1)
// with the inner sums exact INT32 results of the MMA, and the scale s applied once per group in FP32.
//
// A unit is one (column tile, 128-row k-step): 128 x BN INT4 codes with their scales, zero-points and
// Tile-COO slice.  One persistent CTA per SM walks a range of units through a ring of shared-memory
// stages (bulk copies + mbarrier expect_tx, Section 4.1).  Thread = output column throughout: tensor
// memory lane c of a 128-column half holds row c of the A operand (the column's 128 codes) and row c of
// the accumulator D (the column's batch rows, one column of D per limb and row).
//
//   warps 0, 2      producers (cp.async.bulk): warp 0 copies a unit's codes, scales and zero-points, warp 2
//                   its bucket descriptors, its outlier packets and the k-step's activation block, which the
//                   preparation kernel wrote in the stage's own layout (limbs as the K-major MMA operand of
//                   8-row x 16-byte core matrices, then scales and sums, then the FP32 copy).  Issuing a bulk
//                   copy occupies its warp for about 120 ns, whichever lane issues it: one warp with all six
//                   to eight copies of a unit bounded the kernel
//   warp 1          tensor: per unit 4 x BN/128 tcgen05.mma (M = 128 columns, N = NMMA limb rows, K = 32;
//                   A from tensor memory, B from shared memory, D = INT32 in tensor memory), tcgen05.commit
//                   to mbarriers.  An MMA occupies the tensor pipe for 55-66 cycles whatever N <= 128 and
//                   the operand type are, which is why the 8-bit type (K = 32 per instruction instead of
//                   16) matters: with BF16 operands the tensor pipe, not HBM, bounds the kernel
//   unpack warps    BN/32: per 32 rows one 128-bit load of 32 codes, two masks and a shift per 8 codes,
//                   tcgen05.st into the A operand
//   epilogue warps  BN/32: tcgen05.ld of the limb sums, the FP32 combination above, then the unit's outliers
//                   of the thread's own column straight into the same registers (Section 4.2 without the
//                   shared-memory scatter: no atomics, no read-modify-write), and at the end of a piece the
//                   split-tile settlement and the BF16 store of Y
//
// Lane l of an epilogue warp owns column 32 * strip + l = 8 t + g with g = l % 8, t = l / 8: bucket g of
// the strip, column number t of that bucket, so it takes slot t of every column-slotted packet of the
// bucket.  The k-major FP32 copy xt[k][RR] is stored with its 16-byte chunks XOR-swizzled by k
// (Section 3.2.2's concern, shared-memory bank conflicts of the sparse step, met on the activation side:
// the rows a warp's lanes pick are random, and the swizzle spreads them over all eight 16-byte bank groups).

constexpr int kLimbs = 3;

__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]), "r"(r[1]),
                 "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}

// N consecutive 32-bit cells of this thread's tensor-memory lane (N = 1, 4, 8, 16 or 32)
template <int N>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t (&r)[N]) {
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
}

// (float)v for |v| < 2^22 without a conversion instruction (those issue at a quarter of the ALU rate, and an
// epilogue thread needs three per batch row and group): v + 1.5 * 2^23 as an integer bit pattern is the float
// 1.5 * 2^23 + v exactly.
__device__ __forceinline__ float small_int_to_float(uint32_t v) { return __uint_as_float(v + 0x4B400000u) - 12582912.0f; }

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
        for (int j = 0; j < NP; ++j) acc[0] = fmaf(__uint_as_float(wd[j] & kSlotValueMask), x[j], acc[0]);
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
            const float v = __uint_as_float(wd[j] & kSlotValueMask);
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

// D[128 x N] (+)= A[128 x 32] (tensor memory) * B[32 x N] (shared-memory descriptor), signed 8-bit in, INT32 out.
// Called by the whole (converged) warp with warp-uniform operands; one elected lane issues.
__device__ __forceinline__ void umma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p, e;\n setp.ne.b32 p, %4, 0;\n elect.sync _|e, 0xffffffff;\n"
        " @e tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

// Rows of the activation arrays kept per unit for RR batch rows (at least four, so that every copy is a
// multiple of 16 bytes).
__host__ __device__ constexpr int meta_rows(int rr) { return rr < 4 ? 4 : rr; }

// ----------------------------------------------------------------------------- activation preparation

// Bytes of the activation block of one k-step for RR batch rows: the limb operand (NMMA rows x 128 k, one byte
// each), scales and sums (padded to 128 bytes), the FP32 copy.
__host__ __device__ constexpr int nmma_rows(int rr) { return (kLimbs * rr + 15) / 16 * 16; }
__host__ __device__ constexpr int blob_meta_off(int rr) { return nmma_rows(rr) * 128; }
__host__ __device__ constexpr int blob_xt_off(int rr, int gps) { return blob_meta_off(rr) + (gps * 2 * meta_rows(rr) * 4 + 127) / 128 * 128; }
__host__ __device__ constexpr int blob_bytes(int rr, int gps) { return blob_xt_off(rr, gps) + kBK * rr * 4; }

// One warp per (batch row m < RR, k-step kt): the row's 128 activations of the k-step -> limbs, scale,
// integer sum and FP32 copy, per quantisation group (GROUP = 64: lanes 0-15 and 16-31; 128: the warp), into
// the k-step's block xb + kt * blob_bytes, laid out as a stage of the fused kernel holds it:
//   limbs  [16-k block c = 0..7][row n = j * RR + m][16 bytes]: limb j of batch row m, the K-major MMA operand
//          (8-row x 16-byte core matrices); rows n >= 3 RR are zero
//   meta   [128 / GROUP][2][meta_rows(RR)] floats: 2^(E-21), then sum_k x_int (as a float)
//   xt     [128][RR] floats, 16-byte chunks XOR-swizzled by k (xt_swizzle)
// Rows m >= M are written as zeros.  A group with a non-finite activation gets the scale NaN.
template <int RR, int GROUP>
__global__ void __launch_bounds__(128) fq_prep_x_kernel(const uint16_t* __restrict__ X, uint32_t M, uint32_t K, uint8_t* __restrict__ xb) {
    constexpr int GPS = kBK / GROUP, RM = meta_rows(RR), NMMA = nmma_rows(RR);
    // the grid after this one (the fused kernel) may start streaming weights; this one reads X and writes
    // scratch that the grid before it may still be using
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t lane = threadIdx.x & 31, wg = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const uint32_t KT = K / kBK;
    if (wg >= RR * KT) return;
    const uint32_t m = wg / KT, kt = wg - m * KT, k0 = kt * kBK + 4 * lane;
    uint8_t* blob = xb + (size_t)kt * blob_bytes(RR, GPS);
    uint2 raw = make_uint2(0, 0);
    if (m < M) raw = __ldg(reinterpret_cast<const uint2*>(X + (size_t)m * K + k0));
    const uint32_t bits[4] = {raw.x & 0xffffu, raw.x >> 16, raw.y & 0xffffu, raw.y >> 16};
    float x[4];
    uint32_t amax = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) { x[i] = __uint_as_float(bits[i] << 16); amax = max(amax, bits[i] & 0x7fffu); }
#pragma unroll
    for (int d = 1; d < 32 / GPS; d <<= 1) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, d));
    const uint32_t ef_raw = amax >> 7;                        // biased exponent of the group's largest |x|
    const uint32_t ef = max(ef_raw, 22u);                     // keeps 2^(E-21) a normal number; tinier groups lose nothing that matters
    const float up = __uint_as_float((275u - ef) << 23);      // 2^(21-E)
    int xi[4], sum = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) { xi[i] = __float2int_rn(x[i] * up); sum += xi[i]; }
#pragma unroll
    for (int d = 1; d < 32 / GPS; d <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
    // signed limbs: x_int = l0 + 256 l1 + 65536 l2
    uint32_t w[kLimbs] = {0, 0, 0};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int l0 = (xi[i] << 24) >> 24;
        const int r1 = (xi[i] - l0) >> 8;
        const int l1 = (r1 << 24) >> 24;
        const int l2 = (r1 - l1) >> 8;
        w[0] |= (uint32_t)(l0 & 0xff) << (8 * i);
        w[1] |= (uint32_t)(l1 & 0xff) << (8 * i);
        w[2] |= (uint32_t)(l2 & 0xff) << (8 * i);
    }
    // Byte position of k inside its 16-k block: the unpack's two masks put row r of an 8-row word at position
    // 2 (r % 4) + r / 4 of the word's eight (rows 0, 4, 1, 5, 2, 6, 3, 7), and the MMA pairs operand bytes by
    // position.  This lane's four k are rows 4 (lane % 2) .. of 8-row word lane / 2.
    uint8_t* lrow = blob + (lane >> 2) * (NMMA * 16) + ((lane >> 1) & 1) * 8 + (lane & 1);
#pragma unroll
    for (int j = 0; j < kLimbs; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) lrow[(j * RR + m) * 16 + 2 * i] = (uint8_t)(w[j] >> (8 * i));
    if (m == 0) {
#pragma unroll
        for (int n = kLimbs * RR; n < NMMA; ++n)
#pragma unroll
            for (int i = 0; i < 4; ++i) lrow[n * 16 + 2 * i] = 0;          // padding rows of the operand
    }
    if ((lane & (32 / GPS - 1)) == 0) {
        const uint32_t gi = lane / (32 / GPS);
        float* mt = reinterpret_cast<float*>(blob + blob_meta_off(RR)) + gi * 2 * RM;
        mt[m] = ef_raw == 0xffu ? __uint_as_float(0x7fc00000u) : __uint_as_float((ef - 21u) << 23);     // 2^(E-21)
        mt[RM + m] = (float)sum;
    }
    uint8_t* xtu = blob + blob_xt_off(RR, GPS);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t k = 4 * lane + i;
        *reinterpret_cast<float*>(xtu + k * (4 * RR) + ((((m >> 2) ^ xt_swizzle<RR>(k)) << 4) | ((m & 3) << 2))) = x[i];
    }
}

// ----------------------------------------------------------------------------- the fused kernel

// Sets of epilogue warps; with two, the sets take alternate units (set e the units in D buffer e) and set 1
// hands its sums to set 0 through shared memory at the end of a piece.  An epilogue thread's work on a unit is
// a chain of latencies (barrier, tensor-memory load, packet, activation row, multiply-add) of 0.6-1.2 us;
// two warps per strip keep two such chains in flight.
__host__ __device__ constexpr int epilogue_sets(int rr) { return rr <= 16 ? 2 : 1; }

constexpr int kTcFirstUnpack = 4;  // a warp reaches the tensor-memory lanes 32 * (warp % 4) ..., so strips start at a multiple of 4

// BN: tile columns (128 or 256).  RR: batch rows kept per epilogue thread (1, 4, 8, 16, 32; M <= RR).  The
// MMA's N is NMMA = kLimbs * RR rounded up to 16.  HOT: general form of the outlier step (buckets with a tail,
// tiles with more packets than a stage holds).
template <int BN, int RR, int GROUP, bool SPARSE, bool HOT>
__global__ void __launch_bounds__(32 * (kTcFirstUnpack + (1 + epilogue_sets(RR)) * (BN / 32)), 1) fq_tc_kernel(const Params p) {
    constexpr int NDW = BN / 32;              // unpack warps = epilogue warps = 32-column strips
    constexpr int NT128 = BN / 128;           // 128-column halves per unit
    constexpr int UW0 = kTcFirstUnpack, EW0 = UW0 + NDW;
    constexpr int NEPI = epilogue_sets(RR);
    constexpr int GPS = kBK / GROUP;          // groups per k-step
    constexpr int NMMA = nmma_rows(RR);
    constexpr int RM = meta_rows(RR);
    constexpr int DCOLS = GPS * NMMA;         // accumulator columns per half and buffer
    // A buffers (one unit's codes each): four if tensor memory has room beside the two D buffers, so that the
    // unpack warps run up to three units ahead of the MMAs; else two
    constexpr int NAB = (4 * NT128 * 32 + 2 * NT128 * DCOLS <= 512) ? 4 : 2;
    constexpr uint32_t D_BASE = NAB * NT128 * 32;
    constexpr int W_BYTES = 16 * BN * 4;
    constexpr int SZ_ROW = BN * 2;
    // what a stage takes of the k-step's activation block: without outliers, not the FP32 copy at its end
    constexpr int XB_BYTES = SPARSE ? blob_bytes(RR, GPS) : blob_xt_off(RR, GPS);
    constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NMMA >> 3) << 17) | (8u << 24);
    static_assert(D_BASE + 2 * NT128 * DCOLS <= 512, "tensor memory: the A buffers and two D buffers must fit");
    static_assert(RR == 1 || RR % 4 == 0, "rows per thread");
    extern __shared__ __align__(128) uint8_t smem[];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t S = p.stages;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * S;
    const uint32_t bar_a_full = bar_empty + 8 * S;       // [4] A buffer written (unpack warps)
    const uint32_t bar_a_empty = bar_a_full + 32;        // [4] the MMAs that read the A buffer are complete
    const uint32_t bar_d_free = bar_a_empty + 32;        // [2] D buffer read (epilogue warps)
    const uint32_t bar_d_ready = bar_d_free + 16;        // [2] MMAs of a unit complete: D written
    const uint32_t bar_final = bar_d_ready + 16;
    const uint32_t bar_xfull = bar_final + 8, bar_xempty = bar_xfull + 8 * NDW;   // [NDW] each: hand-over of set 1's sums, per strip
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 2 * S + 13 + 2 * NDW);
    volatile uint32_t* tmem_slot = abort_flag + 1;

    if (tid == 0) {
        for (uint32_t s = 0; s < S; ++s) {
            mbar_init(bar_full + 8 * s, 2);                    // the two producers' expect_tx arrivals
            mbar_init(bar_empty + 8 * s, 2 * NDW + 1);         // unpack warps, epilogue warps, the MMAs' commit
        }
        for (uint32_t b = 0; b < 2; ++b) {
            mbar_init(bar_d_free + 8 * b, NDW);                // the epilogue warps of the unit two before
            mbar_init(bar_d_ready + 8 * b, 1);
        }
        for (uint32_t a = 0; a < 4; ++a) {
            mbar_init(bar_a_full + 8 * a, NDW);
            mbar_init(bar_a_empty + 8 * a, 1);
        }
        mbar_init(bar_final, 1);
        for (uint32_t i = 0; i < 2 * NDW; ++i) mbar_init(bar_xfull + 8 * i, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
    // warps that write Y or touch the scratch wait for the grids before this one, and so does the producer
    // before its first copy of the activation arrays; the weight arrays are read before: no kernel writes
    // them while calls are in flight.
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
        // ------------------------------------------------------------------ producer of the dense arrays
        // codes, scales and zero-points of every unit: weights, which no kernel writes while calls are in
        // flight, so this warp never waits for the grids before this one
        uint32_t issued = 0;
        bool ok = true;
        for (UnitIter w(u_begin, KT); w.u < u_end; w.next(S, KT)) {
            const uint32_t s = w.s, full = bar_full + 8 * s;
            if (!warp_wait(bar_empty + 8 * s, w.ph ^ 1, abort_flag, p.status)) { ok = false; break; }
            const uint32_t st = smem_u32(smem) + s * p.stage_bytes;
            if (lane == 0) {
                mbar_arrive_expect_tx(full, W_BYTES + 2 * GPS * SZ_ROW);
                bulk_g2s(st, p.wq + (size_t)w.u * W_BYTES, W_BYTES, full);
#pragma unroll
                for (int gi = 0; gi < GPS; ++gi) {
                    const size_t row = (size_t)(w.kt * GPS + gi) * p.N + (size_t)w.tn * BN;
                    bulk_g2s(st + p.off_sz + gi * SZ_ROW, p.scale + row, SZ_ROW, full);
                    bulk_g2s(st + p.off_sz + (GPS + gi) * SZ_ROW, p.zero + row, SZ_ROW, full);
                }
            }
            issued = w.it + 1;
        }
        if (!ok) {   // giving up: let the copies already issued land before the CTA's shared memory goes away
            for (uint32_t j = (issued > S ? issued - S : 0); j < issued; ++j)
                for (uint32_t spin = 0; spin < (1u << 20) && !mbar_try_wait(bar_full + 8 * (j % S), (j / S) & 1); ++spin) {}
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ producer of the outlier arrays and the activations
        uint32_t ip_a = 0, ip_b = 0;                                   // packet ranges of the next 32 units, read 32 at a time
        uint32_t last_bar = 0, last_ph = 0;
        bool ok = true;
        auto outliers = [&](const UnitIter& w, uint32_t extra) {       // arrival with the byte count of this warp's copies
            const uint32_t s = w.s, full = bar_full + 8 * s;
            const uint32_t st = smem_u32(smem) + s * p.stage_bytes;
            if (SPARSE && (w.it & 31) == 0) {
                const uint32_t i = w.u + lane;
                ip_a = (i <= U) ? __ldg(p.indptr + i) : 0;
                ip_b = (i + 1 <= U) ? __ldg(p.indptr + i + 1) : 0;
            }
            uint32_t pk0 = 0, npk = 0;
            if (SPARSE) {
                pk0 = __shfl_sync(0xffffffffu, ip_a, w.it & 31);
                npk = min(__shfl_sync(0xffffffffu, ip_b, w.it & 31) - pk0, p.coo_cap);
            }
            if (lane == 0) {
                mbar_arrive_expect_tx(full, extra + (SPARSE ? p.NB * 4 + npk * 16 : 0));
                if (SPARSE) {
                    bulk_g2s(st + p.off_info, p.info + (size_t)w.u * p.NB, p.NB * 4, full);
                    if (npk) bulk_g2s(st + p.off_coo, p.packed + pk0, npk * 16, full);
                }
            }
            last_bar = full, last_ph = w.ph;
        };
        auto activations = [&](const UnitIter& w) {                    // the k-step's block, as the preparation kernel laid it out
            if (lane == 0)
                bulk_g2s(smem_u32(smem) + w.s * p.stage_bytes + p.off_xcan, p.xblob + (size_t)w.kt * blob_bytes(RR, GPS), XB_BYTES, bar_full + 8 * w.s);
        };
        // the first pass over the ring finds every stage empty: its outlier arrays (weights) are requested
        // before the wait for the grids before this one, its activation blocks after
        const uint32_t n_first = min(S, u_end - u_begin);
        {
            UnitIter w(u_begin, KT);
            for (uint32_t i = 0; i < n_first; ++i, w.next(S, KT)) outliers(w, XB_BYTES);
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
        {
            UnitIter w(u_begin, KT);
            for (uint32_t i = 0; i < n_first; ++i, w.next(S, KT)) activations(w);
            for (; w.u < u_end; w.next(S, KT)) {
                if (!warp_wait(bar_empty + 8 * w.s, w.ph ^ 1, abort_flag, p.status)) { ok = false; break; }
                outliers(w, XB_BYTES);
                activations(w);
            }
        }
        if (!ok && last_bar)                // gave up: let this warp's last copies land before the CTA exits
            for (uint32_t spin = 0; spin < (1u << 20) && !mbar_try_wait(last_bar, last_ph); ++spin) {}
    } else if (warp == 1) {
        // ------------------------------------------------------------------ tensor warp
        // One warp issues every MMA of the CTA (issued from two warps in turn, MMAs run several times slower).
        // The first MMA of a CTA takes microseconds to start (the tensor pipe wakes up): issue a throw-away
        // one now, while the first loads are in flight.  It reads whatever A buffer 0 and stage 0 hold and
        // writes D buffer 1, which the first real MMA into that buffer overwrites.
        umma_i8_ts(tmem_base + D_BASE + NT128 * DCOLS, tmem_base, make_b_desc(smem_u32(smem) + p.off_xcan, NMMA * 16, 128), IDESC, 0);
        // The tensor pipe should never wait for this warp: the completion signals of a unit go out after the
        // first MMA of the next one has been issued (they then fire one MMA, about 30 ns, later), and the next
        // unit's barriers are tested while the last MMAs of this one run.
        uint32_t ready = 0, pending = 0, pv_b = 0, pv_a = 0, pv_s = 0;
        auto signal = [&]() {                                  // completion of the unit before: D written, A and stage read
            if (pending) {
                umma_commit(bar_d_ready + 8 * pv_b);
                umma_commit(bar_a_empty + 8 * pv_a);
                umma_commit(bar_empty + 8 * pv_s);
                pending = 0;
            }
        };
        for (UnitIter w(u_begin, KT); w.u < u_end; w.next(S, KT)) {
            const uint32_t it = w.it, s = w.s, b = w.it & 1;    // D buffer b, A buffer it % NAB
            if (!ready) {
                // the stage's activation operand, the unit's A buffer, and the D buffer's last reader
                signal();
                if (!warp_wait(bar_full + 8 * s, w.ph, abort_flag, p.status)) break;
                if (!warp_wait(bar_a_full + 8 * (it % NAB), (it / NAB) & 1, abort_flag, p.status)) break;
                if (it >= 2 && !warp_wait(bar_d_free + 8 * b, ((it - 2) >> 1) & 1, abort_flag, p.status)) break;
            }
            tc_fence_after();
            UnitIter nx = w;
            nx.next(S, KT);
            uint32_t seen = 0;
            const uint64_t bd0 = make_b_desc(smem_u32(smem) + s * p.stage_bytes + p.off_xcan, NMMA * 16, 128);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {             // 32 k per MMA: 16-k blocks 2 ks, 2 ks + 1 of the operand
                const int gi = ks / (4 / GPS);
#pragma unroll
                for (int h = 0; h < NT128; ++h) {
                    const uint32_t d = tmem_base + D_BASE + (b * NT128 + h) * DCOLS + gi * NMMA;
                    const uint32_t a = tmem_base + ((it % NAB) * NT128 + h) * 32 + ks * 8;
                    umma_i8_ts(d, a, bd0 + (uint64_t)((ks * 2 * NMMA * 16) >> 4), IDESC, (ks % (4 / GPS)) != 0);
                    if (ks == 0 && h == 0) signal();
                }
                if (ks == 2 && nx.u < u_end && lane == 0)   // one lane, three tests whose latencies overlap
                    seen = mbar_test_wait(bar_full + 8 * nx.s, nx.ph) & mbar_test_wait(bar_a_full + 8 * (nx.it % NAB), (nx.it / NAB) & 1) &
                           (nx.it < 2 ? 1u : mbar_test_wait(bar_d_free + 8 * (nx.it & 1), ((nx.it - 2) >> 1) & 1));
            }
            pending = 1, pv_b = b, pv_a = it % NAB, pv_s = s;
            ready = __shfl_sync(0xffffffffu, seen, 0);
        }
        signal();
        __syncwarp();
        umma_commit(bar_final);                 // fires when every MMA this warp issued has retired
    } else if (warp < UW0) {
        // idle: keeps the strips' warps at a multiple of four
    } else if (warp < EW0) {
        // ------------------------------------------------------------------ unpack warps: thread = column
        const int dw = warp - UW0;
        const int col = dw * 32 + lane;
        const uint32_t t_lane = ((uint32_t)((dw & 3) * 32)) << 16;
        const uint32_t t_a = tmem_base + t_lane + (uint32_t)(dw >> 2) * 32;
        for (UnitIter w(u_begin, KT); w.u < u_end; w.next(S, KT)) {
            const uint32_t it = w.it, s = w.s, b = w.it & 1;
            const uint8_t* st = smem + s * p.stage_bytes;
            if (!warp_wait(bar_full + 8 * s, w.ph, abort_flag, p.status)) break;
            // the column's 128 codes: four 16-byte loads (32 rows each), lanes contiguous
            const uint4* wp = reinterpret_cast<const uint4*>(st) + col;
            uint4 w4[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) w4[j] = wp[j * BN];
            // this A buffer was last read by the MMAs of unit it - NAB
            if (it >= NAB && !warp_wait(bar_a_empty + 8 * (it % NAB), ((it - NAB) / NAB) & 1, abort_flag, p.status)) break;
            tc_fence_after();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t ww[4] = {w4[j].x, w4[j].y, w4[j].z, w4[j].w};
                uint32_t a[8];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    // nibble i + 4h of a word is row 2i + h of its eight: the even nibbles are rows 0, 4, 1, 5 and the
                    // odd ones rows 2, 6, 3, 7, two cells of four bytes; the limb operand is stored in the same k order
                    a[2 * x + 0] = ww[x] & 0x0f0f0f0fu;
                    a[2 * x + 1] = (ww[x] >> 4) & 0x0f0f0f0fu;
                }
                tmem_st8(t_a + (it % NAB) * (NT128 * 32) + j * 8, a);
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive_relaxed(bar_a_full + 8 * (it % NAB));
                mbar_arrive_relaxed(bar_empty + 8 * s);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps: thread = column
        const int ew = warp - EW0, es = ew / NDW, dw = ew % NDW;     // set es (its units: it % NEPI == es), strip dw
        const int col = dw * 32 + lane;
        const uint32_t g = lane & 7, t = lane >> 3;          // bucket of the strip, column number in the bucket
        const uint32_t t_lane = ((uint32_t)((dw & 3) * 32)) << 16;
        const uint32_t t_d = tmem_base + t_lane + D_BASE + (uint32_t)(dw >> 2) * DCOLS;
        float* xch = reinterpret_cast<float*>(smem + p.off_xch) + dw * (RR * 32) + lane;     // hand-over slot of this column
        float accf[RR];
#pragma unroll
        for (int i = 0; i < RR; ++i) accf[i] = 0.0f;
        bool ok = true;
        // outer loop: the pieces of this CTA's range (a piece = its units of one column tile); inner loop: this
        // set's units of the piece
        UnitIter w(u_begin, KT);
        if (es == 1) w.next(S, KT);
        uint32_t tn = u_begin / KT, piece = 0;
        for (uint32_t piece_first = u_begin; piece_first < u_end && ok; ++tn, ++piece) {
          const uint32_t piece_stop = min(u_end, (tn + 1) * KT);        // one past the piece's last unit
          piece_first = piece_stop;
          for (; w.u < piece_stop; w.next(S, KT), (NEPI == 2 ? w.next(S, KT) : (void)0)) {
            const uint32_t u = w.u, it = w.it, s = w.s, b = w.it & 1;
            const uint8_t* st = smem + s * p.stage_bytes;
            if (!warp_wait(bar_full + 8 * s, w.ph, abort_flag, p.status)) { ok = false; break; }
            // outliers: the bucket descriptor and this lane's slots of the first packets are requested now
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
            float sv[GPS], zv[GPS];
#pragma unroll
            for (int gi = 0; gi < GPS; ++gi) {
                sv[gi] = bf16_bits_to_float(reinterpret_cast<const uint16_t*>(st + p.off_sz)[gi * BN + col]);
                zv[gi] = -bf16_bits_to_float(reinterpret_cast<const uint16_t*>(st + p.off_sz)[(GPS + gi) * BN + col]);
            }
            const float* meta = reinterpret_cast<const float*>(st + p.off_xmeta);
            // the unit's sums, once its MMAs are complete
            if (!warp_wait(bar_d_ready + 8 * b, (it >> 1) & 1, abort_flag, p.status)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int gi = 0; gi < GPS; ++gi) {
                // sum_k x (q - z) = 2^(E-21) * (D0 + 2^8 D1 + 2^16 D2 - z sum_k x_int), D_j = sum_k q l_j exact in INT32
                if constexpr (RR == 1) {
                    uint32_t c[4];                                  // one load of four cells covers the three limbs of the single row
                    tmem_ld<4>(t_d + b * (NT128 * DCOLS) + gi * NMMA, c);
                    tmem_wait_ld();
                    const float f = fmaf(zv[gi], meta[gi * 2 * RM + RM],
                                         fmaf(small_int_to_float(c[2]), 65536.0f, fmaf(small_int_to_float(c[1]), 256.0f, small_int_to_float(c[0]))));
                    accf[0] = fmaf(sv[gi] * meta[gi * 2 * RM], f, accf[0]);
                } else {
#pragma unroll
                    for (int i0 = 0; i0 < RR; i0 += 8 < RR ? 8 : RR) {     // eight rows at a time (four with RR = 4)
                        constexpr int CH = 8 < RR ? 8 : RR;
                        uint32_t c[kLimbs][CH];
#pragma unroll
                        for (int j = 0; j < kLimbs; ++j) tmem_ld<CH>(t_d + b * (NT128 * DCOLS) + gi * NMMA + j * RR + i0, c[j]);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < CH; ++i) {
                            const float xs = meta[gi * 2 * RM + i0 + i], sx = meta[gi * 2 * RM + RM + i0 + i];
                            const float f = fmaf(zv[gi], sx, fmaf(small_int_to_float(c[2][i]), 65536.0f, fmaf(small_int_to_float(c[1][i]), 256.0f, small_int_to_float(c[0][i]))));
                            accf[i0 + i] = fmaf(sv[gi] * xs, f, accf[i0 + i]);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_relaxed(bar_d_free + 8 * b);     // the MMAs of unit it + 2 may overwrite this D buffer
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
                            const uint4 pkt = (idx < p.coo_cap) ? reinterpret_cast<const uint4*>(pk_s)[idx]
                                                                : __ldg(reinterpret_cast<const uint4*>(pk_g) + idx);
                            const uint32_t wd[4] = {pkt.x, pkt.y, pkt.z, pkt.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                // a tail slot names its column: slots of other columns count as padding (value 0)
                                const uint32_t mine[1] = {((wd[e] >> kSlotColShift) & 3u) == t ? wd[e] : (wd[e] & ~kSlotValueMask)};
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
          }
          if (!ok) break;
          {
                // ---------------------------------------------------------- end of a piece
                if (NEPI == 2) {
                    if (es == 1) {
                        // hand the sums over (after set 0 has taken the previous piece's) and start afresh
                        if (piece > 0 && !warp_wait(bar_xempty + 8 * dw, (piece - 1) & 1, abort_flag, p.status)) { ok = false; break; }
#pragma unroll
                        for (int mm = 0; mm < RR; ++mm) { xch[mm * 32] = accf[mm]; accf[mm] = 0.0f; }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_xfull + 8 * dw);
                        continue;
                    }
                    if (!warp_wait(bar_xfull + 8 * dw, piece & 1, abort_flag, p.status)) { ok = false; break; }
#pragma unroll
                    for (int mm = 0; mm < RR; ++mm) accf[mm] += xch[mm * 32];
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_xempty + 8 * dw);
                }
                const uint32_t kt = piece_stop - 1 - tn * KT;               // k-step of the piece's last unit
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
