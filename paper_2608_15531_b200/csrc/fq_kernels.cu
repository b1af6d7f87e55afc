// CUDA side of the library (sm_100a): the fused W4A16 + Tile-COO outlier decode matmul
// (Eq. 1; Sections 3.1, 4.1, 4.2), its two unfused baselines and the launchers behind the C ABI.
//
// Two kernels compute the fused operator.  Both are persistent (one CTA per SM) and warp-specialised,
// work on (tile, k-step) units of 128 rows x BN columns, stream them through the same ring of
// shared-memory stages (cp.async.bulk + mbarrier expect_tx), feed the tensor cores
// the exact integers 128 + q as BF16 and apply scale and zero-point once per group in FP32:
//     acc[m] += s * (sum_k x (128+q) - (128+z) sum_k x)                 (Eq. 3 inside Eq. 1)
//
//   fq_mma_kernel    the default (16 batch rows per launch).  Dense warps own 32-column strips: lop3
//                    unpack in registers, mma.sync m16n8k16 with the weights on the M side, and the
//                    unit's outliers added straight into the MMA accumulators (a Tile-COO bucket is
//                    the four columns a group of four lanes holds, and slot j of a packet belongs
//                    to the j-th of them).  Activation warps lay out X and its row sums per unit and
//                    issue part of the unit's bulk copies.  Described in detail above the kernel.
//   fq_fused_kernel  the tcgen05 kernel (FQ_ENGINE=tc; 32 batch rows per launch):
//     warp 0        producer
//     warp 1 (+3)   tensor: own the TMEM allocation and issue tcgen05.mma (A = dequantised weights
//                   in TMEM, B = activations in shared memory, D = FP32 in TMEM); completion is
//                   signalled with tcgen05.commit
//     warp 2        activations: the unit's M x 128 block of X from global memory (it stays in L2) as
//                   the canonical K-major MMA operand in the stage, plus the per-group row sums
//     unpack warps  thread = output column: its 128 codes of the unit -> BF16 (128 + q) -> TMEM A
//                   operand (tcgen05.st)
//     epilogue      thread = output column: reads the FP32 group sums back (tcgen05.ld), applies scale
//                   and zero-point, at the end of a piece adds the outlier tile and writes Y
//     sparse warps  lane = bucket; per packet slot adds v * x[0..7][k] into the FP32 tile sh_c[col][m]
//                   in shared memory (buckets own disjoint columns, so no atomics)
//
// Units are split over CTAs as contiguous ranges (stream-K) or, for layers with few column tiles, as
// tile-aligned parts.  A tile whose k-range is shared by several CTAs is finished by the last to
// arrive, which adds the FP32 partials in CTA order; no CTA waits for another.  Every wait on a barrier
// is bounded: on expiry the CTA raises the scratch status word, drains and leaves (the tcgen05 kernel
// through the common exit that frees its TMEM).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <type_traits>

#include "fq_internal.h"

namespace fq {

constexpr int kBK = 128;
constexpr int kSmemBudget = 232448;    // 227 KB per CTA on sm_100
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
constexpr uint32_t kTmemCols = 512;


struct Params {
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
    uint32_t NB, coo_cap, stages, nsw;
    uint32_t nact;    // tcgen05 kernel: activation warps at work (the ring length is a multiple of it)
    uint32_t split;   // small-batch kernel: 0 = units dealt out as one contiguous range per CTA (stream-K);
                      // c > 0 = every column tile belongs to c CTAs, CTA b takes part b mod c of tile b / c
    // shared-memory offsets (bytes); the first five are relative to a stage
    uint32_t stage_bytes, off_sz, off_xcan, off_xsum, off_info, off_coo;
    uint32_t off_shc, off_xt, off_bar;
};

// ----------------------------------------------------------------------------- PTX helpers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.shared::cta.b64 st, [%0];\n}" ::"r"(bar) : "memory");
}
// For arrivals that publish nothing through the generic proxy (a consumer that only read a stage,
// or a thread whose stores were tcgen05 operations already fenced): no release fence needed.
__device__ __forceinline__ void mbar_arrive_relaxed(uint32_t bar) {
    asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.relaxed.cta.shared::cta.b64 st, [%0];\n}" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}" ::"r"(bar), "r"(bytes)
                 : "memory");
}
// more bytes for the barrier's current phase, without arriving
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// The time hint lets a waiting thread sleep in hardware (up to about 20 us per attempt) instead of
// spinning on the issue slots that the working warps of the CTA need.
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(20000u)
        : "memory");
    return ok;
}
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait, slow part.  Inlined: a call in the pipeline loops constrains the register allocation of
// the code around it (measured: 3 % on the dense-only kernel).
__device__ __forceinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t* status) {
    uint32_t spins = 0;
    unsigned long long t0 = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0xf) == 0) {
            if (*abort_flag) return false;
            unsigned long long now = globaltimer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                atomicExch(status, (uint32_t)FQ_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}
// Bounded wait: false if this CTA is giving up (its own limit expired, or another warp's did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status) {
    if (mbar_test_wait(bar, parity)) return true;   // already complete
    return mbar_wait_slow(bar, parity, abort_flag, status);
}
// Warp-uniform form: every lane waits, and the warp gives up together.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t* status) {
    uint32_t ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag, status) ? 1u : 0u;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// (w & 0x000f000f) | 0x43004300: two codes -> two BF16 values 128 + q
__device__ __forceinline__ uint32_t codes_to_bf16x2(uint32_t w) {
    uint32_t r;
    asm("lop3.b32 %0, %1, 0x000f000f, 0x43004300, 0xea;" : "=r"(r) : "r"(w));
    return r;
}
__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
__device__ __forceinline__ float bf16_bits_to_float(uint16_t v) { return __uint_as_float((uint32_t)v << 16); }
__device__ __forceinline__ uint16_t float_to_bf16_bits(float f) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

// ---- tcgen05 / tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]), "r"(r[1]),
                 "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&d)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    tmem_wait_ld();
#pragma unroll
    for (int i = 0; i < 16; ++i) d[i] = __uint_as_float(r[i]);
}
// D[128 x N] (+)= A[128 x 16] (TMEM) * B[16 x N] (shared-memory descriptor), BF16 in, FP32 out
// Called by the whole (converged) warp with warp-uniform operands; one elected lane issues.
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p, e;\n setp.ne.b32 p, %4, 0;\n elect.sync _|e, 0xffffffff;\n"
        " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile(
        "{\n .reg .pred e;\n elect.sync _|e, 0xffffffff;\n"
        " @e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}" ::"r"(bar)
        : "memory");
}
// K-major, no swizzle: 8 rows x 16 B core matrices; LBO = step between the two K halves of one MMA,
// SBO = step between 8-row groups.
__device__ __forceinline__ uint64_t make_b_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((saddr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46);
}

// Which CTA owns unit u when U units are dealt out as contiguous ranges, the first r CTAs one longer.
__device__ __forceinline__ uint32_t cta_of_unit(uint32_t u, uint32_t q, uint32_t r) {
    const uint32_t big = r * (q + 1);
    return u < big ? u / (q + 1) : r + (u - big) / q;
}
__device__ __forceinline__ uint32_t unit_begin_of(uint32_t c, uint32_t q, uint32_t r) { return c * q + min(c, r); }

// Walks a CTA's units without integer division: ring slot s with its parity, tile tn, k-step kt.
struct UnitIter {
    uint32_t u, it, s, ph, tn, kt;
    __device__ __forceinline__ UnitIter(uint32_t u_begin, uint32_t KT) : u(u_begin), it(0), s(0), ph(0) {
        tn = u_begin / KT;
        kt = u_begin - tn * KT;
    }
    __device__ __forceinline__ void next(uint32_t S, uint32_t KT) {
        ++u;
        ++it;
        if (++s == S) { s = 0; ph ^= 1; }
        if (++kt == KT) { kt = 0; ++tn; }
    }
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

#include "fq_tc_kernel.cuh"

// ----------------------------------------------------------------------------- small-batch kernel

__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

constexpr int kActWarps = 2;   // activation warps of the small-batch kernel
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
__global__ void __launch_bounds__(32 * (1 + kActWarps + NGRP * (BN / 32)), 1) fq_mma_kernel(const Params p) {
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
                    auto apply = [&](const uint32_t w) { add(sacc, __uint_as_float(w & 0xffff0000u), w); };
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
                                    add(hacc, ((w[e] >> 12) & 3u) == (uint32_t)t ? __uint_as_float(w[e] & 0xffff0000u) : 0.0f, w[e]);
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
                            const float v = __uint_as_float(w[e] & 0xffff0000u);
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
                                    const uint32_t cls = (w[e] >> 12) & 3u;
                                    const float v = __uint_as_float(w[e] & 0xffff0000u);
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

// ----------------------------------------------------------------------------- unfused SpMM

// Y += X * W_O as its own launch (the sparse half of the two-kernel baseline).  One warp per bucket of
// a column tile (four columns): its lanes take the row tiles kt = lane, lane + 32, ..., read the
// bucket's packets and the activations x[m][k] from global memory (L2-resident) and add into registers
// (4 columns x 8 batch rows per lane); a butterfly sum over the lanes and one read-modify-write of the
// BF16 Y per element finish it.  No shared memory, no atomics: a bucket's columns belong to one warp.
__global__ void __launch_bounds__(256) fq_spmm_kernel(const uint16_t* __restrict__ X, const uint32_t* __restrict__ indptr,
                                                    const uint32_t* __restrict__ info, const uint4* __restrict__ packed,
                                                    uint16_t* __restrict__ Y, uint32_t M, uint32_t K, uint32_t N,
                                                    uint32_t BN, uint32_t NB) {
    constexpr int MB = 8;
    const int lane = threadIdx.x & 31;
    const uint32_t wg = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wg >= (N / BN) * NB) return;
    const uint32_t tn = wg / NB, b = wg - tn * NB, KT = K / kBK;
    const uint32_t first_col = tn * BN + (((b >> 3) << 5) | (b & 7u));      // column number c of the bucket: + 8 c
    for (uint32_t m0 = 0; m0 < M; m0 += MB) {
        float acc[4][MB];
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int m = 0; m < MB; ++m) acc[c][m] = 0.0f;
        for (uint32_t kt = lane; kt < KT; kt += 32) {
            const size_t t = (size_t)tn * KT + kt;
            const uint32_t inf = __ldg(info + t * NB + b);
            const uint4* pk = packed + __ldg(indptr + t) + (inf & 0xffffu);
            const uint32_t depth = (inf >> 16) & 0xffu, tail = inf >> 24;
            for (uint32_t i = 0; i < depth; ++i) {              // column-slotted: slot e is column number e
                const uint4 q = __ldg(pk + i);
                const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if ((w[e] >> 16) == 0) continue;            // padding: no activation loads for it
                    const float v = __uint_as_float(w[e] & 0xffff0000u);
                    const uint16_t* xp = X + (size_t)m0 * K + kt * kBK + ((w[e] >> 5) & 127u);
#pragma unroll
                    for (int m = 0; m < MB; ++m)
                        acc[e][m] = fmaf(v, (m0 + m < M) ? bf16_bits_to_float(__ldg(xp + (size_t)m * K)) : 0.0f, acc[e][m]);
                }
            }
            for (uint32_t i = depth; i < depth + tail; ++i) {   // tail: a slot names its column
                const uint4 q = __ldg(pk + i);
                const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t cls = (w[e] >> 12) & 3u;
                    const float v = __uint_as_float(w[e] & 0xffff0000u);
                    const uint16_t* xp = X + (size_t)m0 * K + kt * kBK + ((w[e] >> 5) & 127u);
#pragma unroll
                    for (int m = 0; m < MB; ++m) {
                        const float x = (m0 + m < M) ? bf16_bits_to_float(__ldg(xp + (size_t)m * K)) : 0.0f;
#pragma unroll
                        for (int c = 0; c < 4; ++c) acc[c][m] = fmaf(cls == (uint32_t)c ? v : 0.0f, x, acc[c][m]);
                    }
                }
            }
        }
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int m = 0; m < MB; ++m) {
                float a = acc[c][m];
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) a += __shfl_xor_sync(0xffffffffu, a, d);
                if (lane == c * MB + m && m0 + m < M) {
                    uint16_t* y = Y + (size_t)(m0 + m) * N + first_col + 8 * c;
                    *y = float_to_bf16_bits(bf16_bits_to_float(*y) + a);
                }
            }
    }
}

// ----------------------------------------------------------------------------- launch plumbing

struct Plan {
    Params p;
    uint32_t threads, smem, grid;
    uint32_t ngrp;   // small-batch kernel: groups of dense warps
    bool general;    // small-batch kernel: the layer needs the general form of the outlier step
};

static inline uint32_t round_up(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }

static int sm_count_cached() {
    static int cached[64];
    static std::once_flag once;
    std::call_once(once, [] { std::memset(cached, 0, sizeof(cached)); });
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
        cached[dev] = n;
    }
    return cached[dev];
}

static inline uint32_t nb16_of(uint32_t m) { return m <= 16 ? 1u : 2u; }

// Rows kept per epilogue thread of the tcgen05 kernel, and the MMA's batch columns, for a launch of M rows.
static inline uint32_t rr_of(uint32_t m) { return m <= 1 ? 1u : (m <= 4 ? 4u : (m <= 8 ? 8u : (m <= 16 ? 16u : 32u))); }
static inline uint32_t nmma_of(uint32_t m) { return m <= 16 ? 16u : 32u; }

// Plan of the tcgen05 kernel (fq_tc_kernel): up to 32 rows per launch.
static fq_status_t make_plan(const fq_layout_t* L, uint32_t M, bool sparse, Plan& pl) {
    const uint32_t BN = L->BN, NB = L->buckets_per_tile, GPS = kBK / L->group;
    const uint32_t NMMA = nmma_of(M), RR = rr_of(M);
    Params& p = pl.p;
    std::memset(&p, 0, sizeof(p));
    p.M = M; p.K = L->K; p.N = L->N; p.KT = L->K / kBK; p.NT = L->N / BN; p.NB = NB; p.nsw = 0;
    const int sms = sm_count_cached();
    if (sms <= 0) return fail(FQ_ERR_CUDA, "no CUDA device: %s", cudaGetErrorString(cudaGetLastError()));
    const uint32_t NT = p.NT, KT = p.KT;
    uint32_t grid = std::min<uint32_t>({(uint32_t)sms, kMaxCtas, NT * KT});
    uint32_t units_per_cta = (NT * KT + grid - 1) / grid;
    // Tile-aligned split instead of one contiguous range per CTA when it costs at most one more unit
    // per CTA: then no CTA has to settle two split tiles in a row.
    uint32_t split = 0;
    if (NT <= grid) {
        const uint32_t c = std::min<uint32_t>(grid / NT, KT);
        if (c >= 2 && (KT + c - 1) / c <= units_per_cta + 1) {
            split = c;
            grid = NT * c;
            units_per_cta = (KT + c - 1) / c;
        }
    }
    p.split = split;
    const uint32_t w_bytes = 16 * BN * 4, sz_bytes = 2 * GPS * BN * 2;
    const uint32_t xt_bytes = sparse ? kBK * RR * 4 : 0;                 // FP32 k-major copy [k][RR]
    uint32_t cap = 0;
    if (sparse) {
        cap = L->tilecoo_encoded ? std::max<uint32_t>(8, round_up(L->max_tile_packets, 8)) : 256;
        cap = std::min<uint32_t>(cap, 1024);
    }
    uint32_t stage = 0, S = 0;
    for (;;) {
        p.off_sz = w_bytes;
        p.off_xcan = p.off_sz + round_up(sz_bytes, 128);
        p.off_xsum = p.off_xcan + NMMA * 256;
        p.off_xt = p.off_xsum + round_up(GPS * NMMA * 4, 128);
        p.off_info = p.off_xt + xt_bytes;
        p.off_coo = p.off_info + (sparse ? round_up(NB * 4, 128) : 0);
        stage = round_up(p.off_coo + cap * 16, 128);
        S = std::min<uint32_t>(8, (kSmemBudget - 1024) / stage);
        if (S >= 4 || cap <= 64) break;
        cap = std::max<uint32_t>(64, cap / 2);  // oversized tiles read their tail from global memory
    }
    if (S < 2) return fail(FQ_ERR_UNSUPPORTED_SHAPE, "shared-memory stages do not fit");
    // The activation warps take the units in turn, and the ring length is a multiple of their number, so
    // that a stage always returns to the same warp (which then meets every phase of the stage's barriers).
    p.nact = S >= 8 ? 4 : (S >= 6 ? 3 : (S >= 4 ? 4 : 2));
    S = S / p.nact * p.nact;
    p.coo_cap = cap; p.stages = S; p.stage_bytes = stage;
    // hot columns, tiles larger than the staged part, or an encoding whose sizes were not recorded
    pl.general = sparse && (L->max_tail_packets > 0 || L->max_tile_packets > cap || !L->tilecoo_encoded);
    p.off_shc = S * stage;
    p.off_bar = p.off_shc;
    pl.smem = p.off_bar + 1024;
    pl.threads = 32 * (2 + kTcActWarps + 2 * (BN / 32));
    pl.grid = grid;
    pl.ngrp = 1;
    return FQ_OK;
}

// Plan of the small-batch kernel (fq_mma_kernel): M <= 16 per launch.
static fq_status_t make_plan_mma(const fq_layout_t* L, uint32_t M, bool sparse, Plan& pl) {
    const uint32_t BN = L->BN, NB = L->buckets_per_tile, GPS = kBK / L->group;
    const uint32_t MO = M <= 8 ? 1 : (M <= 16 ? 2 : 4), ROWS = 8 * MO;
    const uint32_t NDW = BN / 32;
    Params& p = pl.p;
    std::memset(&p, 0, sizeof(p));
    p.M = M; p.K = L->K; p.N = L->N; p.KT = L->K / kBK; p.NT = L->N / BN; p.NB = NB; p.nsw = 0;
    const uint32_t w_bytes = 16 * BN * 4, sz_bytes = 2 * GPS * BN * 2;
    const uint32_t xt_bytes = sparse ? (M == 1 ? 512 : (M <= 4 ? 2048 : MO * 4096)) : 0;     // FP32 [k], [k][4] or [octet][k][8]
    // Two groups of dense warps (each takes every other unit) pay off when a CTA has enough units to
    // stream; short jobs keep one group.  With two octets of rows the second group fits only because
    // the outlier step of that variant prefetches less (96 registers per thread).
    const int sms = sm_count_cached();
    if (sms <= 0) return fail(FQ_ERR_CUDA, "no CUDA device: %s", cudaGetErrorString(cudaGetLastError()));
    const uint32_t NT = L->N / BN, KT = L->K / kBK;
    uint32_t grid = std::min<uint32_t>({(uint32_t)sms, kMaxCtas, NT * KT});
    uint32_t units_per_cta = (NT * KT + grid - 1) / grid;
    // Tile-aligned split instead of one contiguous range per CTA when it costs at most one more unit
    // per CTA: then no CTA has to settle two split tiles in a row.
    uint32_t split = 0;
    if (NT <= grid) {
        const uint32_t c = std::min<uint32_t>(grid / NT, KT);
        if (c >= 2 && (KT + c - 1) / c <= units_per_cta + 1) {
            split = c;
            grid = NT * c;
            units_per_cta = (KT + c - 1) / c;
        }
    }
    p.split = split;
    pl.ngrp = (units_per_cta >= 8 && MO <= 2) ? 2 : 1;    // four octets of rows: the accumulators leave no room
    const uint32_t xch_bytes = pl.ngrp > 1 ? BN * ROWS * 4 : 0;   // hand-over of a group's partial sums
    const uint32_t fixed = 1024 + xch_bytes;
    const uint32_t budget = kSmemBudget;
    uint32_t cap = 0;
    if (sparse) {
        cap = L->tilecoo_encoded ? std::max<uint32_t>(8, round_up(L->max_tile_packets, 8)) : 256;
        cap = std::min<uint32_t>(cap, 1024);
    }
    uint32_t stage = 0, S = 0;
    for (;;) {
        p.off_sz = w_bytes;
        p.off_xcan = p.off_sz + round_up(sz_bytes, 128);
        p.off_xsum = p.off_xcan + round_up(ROWS * kXPitch, 128);
        p.off_xt = p.off_xsum + round_up(GPS * ROWS * 4, 128);          // stage-relative in this kernel
        p.off_info = p.off_xt + xt_bytes;
        p.off_coo = p.off_info + (sparse ? round_up(NB * 4, 128) : 0);
        stage = round_up(p.off_coo + cap * 16, 128);
        // An even number of stages: the activation warps and the dense groups take alternate units, and
        // a parity wait is only valid for a waiter that meets every phase of the barrier.  With S even a
        // stage always comes back to the same activation warp and the same dense group.
        S = std::min<uint32_t>(8, (budget - fixed) / stage) & ~1u;
        if (S >= 4 || cap <= 64) break;
        cap = std::max<uint32_t>(64, cap / 2);
    }
    if (S < 4) return fail(FQ_ERR_UNSUPPORTED_SHAPE, "shared-memory stages do not fit");
    p.coo_cap = cap; p.stages = S; p.stage_bytes = stage;
    // hot columns, tiles larger than the staged part, or an encoding whose sizes were not recorded
    pl.general = sparse && (L->max_tail_packets > 0 || L->max_tile_packets > cap || !L->tilecoo_encoded);
    p.off_shc = S * stage;
    p.off_bar = p.off_shc + xch_bytes;
    pl.smem = p.off_bar + 1024;
    pl.threads = 32 * (1 + kActWarps + pl.ngrp * NDW);
    pl.grid = grid;
    return FQ_OK;
}

typedef void (*KernelFn)(const Params);

// MS: form of the outlier step (1: single batch row, one column per lane; 8: rows split over the lanes);
// NGRP: groups of dense warps; HOT: general form of the outlier step
// (long bucket lists shared out, packets beyond the staged part of a tile)
template <int BN, int MO, int G, bool HOT>
static KernelFn pick_mma_sparse(bool sparse, uint32_t ms, uint32_t ngrp) {
    if constexpr (MO == 1) {
        if (ngrp == 2) {
            if (!sparse) return (KernelFn)fq_mma_kernel<BN, MO, G, false, 8, 2, false>;
            if (ms == 1) return (KernelFn)fq_mma_kernel<BN, MO, G, true, 1, 2, HOT>;
            if (ms == 4) return (KernelFn)fq_mma_kernel<BN, MO, G, true, 4, 2, HOT>;
            return (KernelFn)fq_mma_kernel<BN, MO, G, true, 8, 2, HOT>;
        }
        if (sparse && ms == 1) return (KernelFn)fq_mma_kernel<BN, MO, G, true, 1, 1, HOT>;
        if (sparse && ms == 4) return (KernelFn)fq_mma_kernel<BN, MO, G, true, 4, 1, HOT>;
    }
    if constexpr (MO == 2) {
        if (ngrp == 2) return sparse ? (KernelFn)fq_mma_kernel<BN, MO, G, true, 8, 2, HOT> : (KernelFn)fq_mma_kernel<BN, MO, G, false, 8, 2, false>;
    }
    if (!sparse) return (KernelFn)fq_mma_kernel<BN, MO, G, false, 8, 1, false>;
    return (KernelFn)fq_mma_kernel<BN, MO, G, true, 8, 1, HOT>;
}
template <int BN, int MO>
static KernelFn pick_mma_group(uint32_t g, bool sparse, uint32_t ms, uint32_t ngrp, bool hot) {
    if (g == 64) return hot ? pick_mma_sparse<BN, MO, 64, true>(sparse, ms, ngrp) : pick_mma_sparse<BN, MO, 64, false>(sparse, ms, ngrp);
    return hot ? pick_mma_sparse<BN, MO, 128, true>(sparse, ms, ngrp) : pick_mma_sparse<BN, MO, 128, false>(sparse, ms, ngrp);
}
static KernelFn pick_mma_kernel(uint32_t bn, uint32_t M, uint32_t g, bool sparse, uint32_t ngrp, bool hot) {
    const uint32_t mo = M <= 8 ? 1 : (M <= 16 ? 2 : 4), ms = M <= 1 ? 1 : (M <= 4 ? 4 : 8);
    if (bn == 128) return mo == 1 ? pick_mma_group<128, 1>(g, sparse, ms, ngrp, hot) : mo == 2 ? pick_mma_group<128, 2>(g, sparse, ms, ngrp, hot) : pick_mma_group<128, 4>(g, sparse, ms, ngrp, hot);
    return mo == 1 ? pick_mma_group<256, 1>(g, sparse, ms, ngrp, hot) : mo == 2 ? pick_mma_group<256, 2>(g, sparse, ms, ngrp, hot) : pick_mma_group<256, 4>(g, sparse, ms, ngrp, hot);
}

// Which kernel serves a call: the tcgen05 kernel.  The warp-level MMA kernel stays reachable through an
// internal switch for comparison runs.
static int g_engine = 0;   // 0: tcgen05 kernel, 1: warp-level MMA kernel

template <int BN, int NMMA, int RR, int G>
static KernelFn pick_tc_sparse(bool sparse, bool hot) {
    if (!sparse) return (KernelFn)fq_tc_kernel<BN, NMMA, RR, G, false, false>;
    return hot ? (KernelFn)fq_tc_kernel<BN, NMMA, RR, G, true, true> : (KernelFn)fq_tc_kernel<BN, NMMA, RR, G, true, false>;
}
template <int BN, int G>
static KernelFn pick_tc_rows(uint32_t rr, bool sparse, bool hot) {
    switch (rr) {
        case 1: return pick_tc_sparse<BN, 16, 1, G>(sparse, hot);
        case 4: return pick_tc_sparse<BN, 16, 4, G>(sparse, hot);
        case 8: return pick_tc_sparse<BN, 16, 8, G>(sparse, hot);
        case 16: return pick_tc_sparse<BN, 16, 16, G>(sparse, hot);
        default: return pick_tc_sparse<BN, 32, 32, G>(sparse, hot);
    }
}
static KernelFn pick_kernel(uint32_t bn, uint32_t M, uint32_t g, bool sparse, bool hot) {
    const uint32_t rr = rr_of(M);
    if (bn == 128) return g == 64 ? pick_tc_rows<128, 64>(rr, sparse, hot) : pick_tc_rows<128, 128>(rr, sparse, hot);
    return g == 64 ? pick_tc_rows<256, 64>(rr, sparse, hot) : pick_tc_rows<256, 128>(rr, sparse, hot);
}

// cudaFuncSetAttribute costs several microseconds: do it once per (kernel, device).
static cudaError_t ensure_smem_attr(const void* fn, int bytes) {
    struct Seen { const void* fn; int dev; };
    static Seen seen[256];
    static int nseen = 0;
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < nseen; ++i)
        if (seen[i].fn == fn && seen[i].dev == dev) return cudaSuccess;
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && nseen < 256) seen[nseen++] = Seen{fn, dev};
    return e;
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

static fq_status_t launch_gemm(const fq_layout_t* L, const void* X, uint32_t M, const void* wq, const void* scale,
                               const void* zero, const void* indptr, const void* info, const void* packed, void* Y,
                               void* workspace, size_t workspace_bytes, void* stream, bool sparse) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if (M < 1 || M > FQ_MAX_M) return fail(FQ_ERR_INVALID_ARG, "M = %u outside [1, %u]", M, FQ_MAX_M);
    if (!X || !wq || !scale || !zero || !Y || !workspace) return fail(FQ_ERR_INVALID_ARG, "null device pointer");
    if (sparse && (!indptr || !info)) return fail(FQ_ERR_INVALID_ARG, "null Tile-COO pointer");
    if (sparse && !packed && (L->max_tile_packets || !L->tilecoo_encoded)) return fail(FQ_ERR_INVALID_ARG, "null packet pointer");
    if (!aligned(X, 16) || !aligned(Y, 16) || !aligned(wq, 128) || !aligned(scale, 128) || !aligned(zero, 128) ||
        !aligned(workspace, 128) || (sparse && (!aligned(indptr, 4) || !aligned(info, 128) || !aligned(packed, 128))))
        return fail(FQ_ERR_INVALID_ARG, "misaligned device pointer");
    size_t need = 0;
    fq_status_t st = fq_workspace_bytes(L, M, &need);
    if (st != FQ_OK) return st;
    if (workspace_bytes < need) return fail(FQ_ERR_BUFFER_TOO_SMALL, "workspace holds %zu bytes, %zu needed", workspace_bytes, need);
    const bool use_mma = g_engine == 1;
    // the small-batch kernel takes up to 32 rows per launch; a remainder of at most 16 rows gets the cheaper variants
    const uint32_t rows_per_launch = 32;
    for (uint32_t m0 = 0; m0 < M; m0 += rows_per_launch) {
        const uint32_t mb = std::min<uint32_t>(rows_per_launch, M - m0);
        Plan pl;
        st = use_mma ? make_plan_mma(L, mb, sparse, pl) : make_plan(L, mb, sparse, pl);
        if (st != FQ_OK) return st;
        Params& p = pl.p;
        p.X = (const uint16_t*)X + (size_t)m0 * L->K;
        p.Y = (uint16_t*)Y + (size_t)m0 * L->N;
        p.wq = (const uint8_t*)wq; p.scale = (const uint16_t*)scale; p.zero = (const uint16_t*)zero;
        p.indptr = (const uint32_t*)indptr; p.info = (const uint32_t*)info; p.packed = (const uint4*)packed;
        p.status = (uint32_t*)workspace;
        p.counters = (uint32_t*)((uint8_t*)workspace + kWsHeaderBytes);
        p.partials = (float*)((uint8_t*)workspace + kWsHeaderBytes + kWsCounterBytes);
        KernelFn fn = use_mma ? pick_mma_kernel(L->BN, mb, L->group, sparse, pl.ngrp, pl.general)
                              : pick_kernel(L->BN, mb, L->group, sparse, pl.general);
        cudaError_t e = ensure_smem_attr((const void*)fn, (int)kSmemBudget);
        if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        {
            // Programmatic dependent launch: this grid may become resident while the kernel before it
            // in the stream drains.  Its producer warp then already streams weights (which no kernel
            // writes); the warps that touch X, Y or the scratch first execute griddepcontrol.wait, after
            // which all memory operations of the earlier grid are complete and visible.
            cudaLaunchConfig_t cfg;
            std::memset(&cfg, 0, sizeof(cfg));
            cfg.gridDim = dim3(pl.grid);
            cfg.blockDim = dim3(pl.threads);
            cfg.dynamicSmemBytes = pl.smem;
            cfg.stream = (cudaStream_t)stream;
            cudaLaunchAttribute attr[1];
            std::memset(attr, 0, sizeof(attr));
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            e = cudaLaunchKernelEx(&cfg, fn, p);
            if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
        }
        e = cudaGetLastError();
        if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
    }
    return FQ_OK;
}

}  // namespace fq

using namespace fq;

extern "C" {

// Comparison runs only (not declared in fq.h): 0 = the tcgen05 kernel (default), 1 = the warp-level MMA kernel.
void fq_internal_select_engine(int e) { fq::g_engine = e == 1 ? 1 : 0; }

fq_status_t fq_workspace_bytes(const fq_layout_t* L, uint32_t M, size_t* bytes) {
    if (!layout_ok(L) || !bytes) return fail(FQ_ERR_INVALID_ARG, "bad layout or null output");
    if (M < 1 || M > FQ_MAX_M) return fail(FQ_ERR_INVALID_ARG, "M = %u outside [1, %u]", M, FQ_MAX_M);
    const uint32_t mb = std::min<uint32_t>(M, 32);
    *bytes = kWsHeaderBytes + kWsCounterBytes + (size_t)kMaxCtas * 2 * L->BN * 16 * nb16_of(mb) * 4;
    return FQ_OK;
}

fq_status_t fq_fused_w4a16_outlier_gemm(const fq_layout_t* L, const void* X, uint32_t M, const void* wq,
                                        const void* scale, const void* zero, const void* tile_indptr,
                                        const void* bucket_info, const void* packed_outliers, void* Y,
                                        void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return launch_gemm(L, X, M, wq, scale, zero, tile_indptr, bucket_info, packed_outliers, Y, workspace,
                       workspace_bytes, cuda_stream, true);
}

// ---- the entry point that allocates nothing -------------------------------------------------
// Scratch for callers that cannot allocate device memory: lives in the library's own image on
// every GPU that loads it, for the life of the process.
static __device__ __align__(256) unsigned char g_static_scratch[FQ_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device.  In host code the array's name is only
// a handle; the address a kernel can use comes from cudaGetSymbolAddress, asked once per device
// with that device current.
static fq_status_t static_scratch_address(void** out) {
    static void* addr[64] = {nullptr};
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= 64) return fail(FQ_ERR_CUDA, "device ordinal %d is outside the supported range", dev);
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) return fail(FQ_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        addr[dev] = ptr;
    }
    *out = addr[dev];
    return FQ_OK;
}

fq_status_t fq_fused_w4a16_outlier_gemm_noalloc(const fq_layout_t* L, const void* X, uint32_t M, const void* wq,
                                                const void* scale, const void* zero, const void* tile_indptr,
                                                const void* bucket_info, const void* packed_outliers, void* Y,
                                                void* cuda_stream) {
    size_t need = 0;
    fq_status_t st = fq_workspace_bytes(L, M, &need);
    if (st != FQ_OK) return st;
    if (need > (size_t)FQ_STATIC_SCRATCH_BYTES)
        return fail(FQ_ERR_BUFFER_TOO_SMALL,
                    "this call needs %zu bytes of scratch but the built-in scratch holds %zu (M <= %u fits); "
                    "use fq_fused_w4a16_outlier_gemm with caller-allocated scratch",
                    need, (size_t)FQ_STATIC_SCRATCH_BYTES, (unsigned)FQ_STATIC_SCRATCH_MAX_M);
    void* scratch = nullptr;
    st = static_scratch_address(&scratch);
    if (st != FQ_OK) return st;
    // the status word and the tile-arrival counters must start at zero; the previous user of the
    // shared array may have been interrupted
    cudaError_t e = cudaMemsetAsync(scratch, 0, kWsHeaderBytes + kWsCounterBytes, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "clearing the built-in scratch: %s", cudaGetErrorString(e));
    return launch_gemm(L, X, M, wq, scale, zero, tile_indptr, bucket_info, packed_outliers, Y, scratch,
                       (size_t)FQ_STATIC_SCRATCH_BYTES, cuda_stream, true);
}

fq_status_t fq_unfused_gemm(const fq_layout_t* L, const void* X, uint32_t M, const void* wq, const void* scale,
                            const void* zero, void* Y, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return launch_gemm(L, X, M, wq, scale, zero, nullptr, nullptr, nullptr, Y, workspace, workspace_bytes,
                       cuda_stream, false);
}

fq_status_t fq_unfused_spmm(const fq_layout_t* L, const void* X, uint32_t M, const void* tile_indptr,
                            const void* bucket_info, const void* packed_outliers, void* Y, void* cuda_stream) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if (M < 1 || M > FQ_MAX_M) return fail(FQ_ERR_INVALID_ARG, "M = %u outside [1, %u]", M, FQ_MAX_M);
    if (!X || !tile_indptr || !bucket_info || !Y) return fail(FQ_ERR_INVALID_ARG, "null device pointer");
    if (!packed_outliers && (L->max_tile_packets || !L->tilecoo_encoded)) return fail(FQ_ERR_INVALID_ARG, "null packet pointer");
    const uint32_t buckets = (L->N / L->BN) * L->buckets_per_tile;   // one warp each
    fq_spmm_kernel<<<(buckets + 7) / 8, 256, 0, (cudaStream_t)cuda_stream>>>(
        (const uint16_t*)X, (const uint32_t*)tile_indptr, (const uint32_t*)bucket_info, (const uint4*)packed_outliers,
        (uint16_t*)Y, M, L->K, L->N, L->BN, L->buckets_per_tile);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "spmm launch: %s", cudaGetErrorString(e));
    return FQ_OK;
}

fq_status_t fq_fused_host_io_async(const fq_layout_t* L, const void* X_host, uint32_t M, void* x_dev, const void* wq,
                                   const void* scale, const void* zero, const void* tile_indptr,
                                   const void* bucket_info, const void* packed_outliers, void* y_dev, void* Y_host,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if (!X_host || !Y_host || !x_dev || !y_dev) return fail(FQ_ERR_INVALID_ARG, "null pointer");
    if (M < 1 || M > FQ_MAX_M) return fail(FQ_ERR_INVALID_ARG, "M = %u outside [1, %u]", M, FQ_MAX_M);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemcpyAsync(x_dev, X_host, (size_t)M * L->K * 2, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "copy of X: %s", cudaGetErrorString(e));
    fq_status_t st = fq_fused_w4a16_outlier_gemm(L, x_dev, M, wq, scale, zero, tile_indptr, bucket_info,
                                                 packed_outliers, y_dev, workspace, workspace_bytes, cuda_stream);
    if (st != FQ_OK) return st;
    e = cudaMemcpyAsync(Y_host, y_dev, (size_t)M * L->N * 2, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "copy of Y: %s", cudaGetErrorString(e));
    return FQ_OK;
}

fq_status_t fq_fused_host_io(const fq_layout_t* L, const void* X_host, uint32_t M, void* x_dev, const void* wq,
                             const void* scale, const void* zero, const void* tile_indptr, const void* bucket_info,
                             const void* packed_outliers, void* y_dev, void* Y_host, void* workspace,
                             size_t workspace_bytes, void* cuda_stream) {
    fq_status_t st = fq_fused_host_io_async(L, X_host, M, x_dev, wq, scale, zero, tile_indptr, bucket_info,
                                            packed_outliers, y_dev, Y_host, workspace, workspace_bytes, cuda_stream);
    if (st != FQ_OK) return st;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "stream synchronisation: %s", cudaGetErrorString(e));
    return FQ_OK;
}

fq_status_t fq_check_status(void* workspace, void* cuda_stream) {
    if (!workspace) return fail(FQ_ERR_INVALID_ARG, "null workspace");
    cudaStream_t s = (cudaStream_t)cuda_stream;
    uint32_t word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, workspace, 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "status read: %s", cudaGetErrorString(e));
    if (word != 0) {
        cudaMemsetAsync(workspace, 0, 4, s);
        cudaStreamSynchronize(s);
        return fail((fq_status_t)(int32_t)word, "a device-side wait expired (status word %d)", (int32_t)word);
    }
    return FQ_OK;
}

}  // extern "C"
