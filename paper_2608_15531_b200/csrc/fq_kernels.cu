// CUDA side of the library (sm_100a): the fused W4A16 + Tile-COO outlier decode matmul
// (Eq. 1; Sections 3.1, 4.1, 4.2), its two unfused baselines and the launchers behind the C ABI.
//
// The fused operator is one persistent, warp-specialised kernel (one CTA per SM), fq_tc_kernel in
// fq_tc_kernel.cuh: (tile, k-step) units of 128 rows x BN columns stream through a ring of shared-memory
// stages (bulk copies + mbarrier expect_tx); the codes are unpacked to the exact integers q - z in BF16
// and written to tensor memory as the A operand of tcgen05.mma, the activations are the B operand, and
// the scale is applied once per group in FP32:
//     acc[m] += s * sum_k x (q - z)                                     (Eq. 3 inside Eq. 1)
// The unit's Tile-COO outliers are added in the registers of the epilogue threads, one thread per
// output column.
//
// Units are split over CTAs as contiguous ranges (stream-K) or, for layers with few column tiles, as
// tile-aligned parts.  A tile whose k-range is shared by several CTAs is finished by the last to
// arrive, which adds the FP32 partials in CTA order; no CTA waits for another.  Every wait on a barrier
// is bounded: on expiry the CTA raises the scratch status word, drains and leaves through the common
// exit that frees its tensor memory.
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <mutex>

#include "fq_internal.h"

namespace cg = cooperative_groups;
namespace fq {

constexpr int kBK = 128;
constexpr int kSmemBudget = 232448;    // 227 KB per CTA on sm_100
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
constexpr uint32_t kTmemCols = 512;


struct Params {
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
    const uint8_t* xblob; // per k-step: the activation block fq_prep_x_kernel wrote (limbs, scales and sums, FP32 copy)
    uint32_t M, K, N, KT, NT;
    uint32_t NB, coo_cap, stages;
    uint32_t split;   // 0 = units dealt out as one contiguous range per CTA (stream-K);
                      // c > 0 = every column tile belongs to c CTAs, CTA b takes part b mod c of tile b / c
    // shared-memory offsets (bytes); all but the last are relative to a stage
    uint32_t stage_bytes, off_sz, off_xcan, off_xmeta, off_xt, off_info, off_coo;
    uint32_t off_xch;     // hand-over of the second epilogue set's sums (BN x RR floats), if there are two sets
    uint32_t off_bar;
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
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
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

#include "fq_tc_kernel.cuh"
#include "fq_mma_kernel.cuh"
#include "fq_direct_kernel.cuh"

// ----------------------------------------------------------------------------- unfused SpMM

// Y += X * W_O as its own launch (the sparse half of the two-kernel baseline, Section 2.2).  One CTA per
// (column tile, slab of k-steps); the slabs of a tile form one thread-block cluster.  A warp owns a strip of
// 32 columns (lane = column = slot t of bucket g) and every second (fourth, for tiles of 128 columns) k-step of the slab.  The CTA stages the
// activations of eight k-steps at a time as a k-major BF16 tile in shared memory; while those loads are in
// flight every warp fetches the bucket descriptors and the first four packet slots of its k-steps, so one
// chunk costs three global-memory latencies whatever its length.  A lane multiplies-adds the slots of its
// column into RR FP32 registers (a padding slot has value 0 and reads row 0: a broadcast).  The warps of
// a strip add up in shared memory, the slabs of a tile through distributed shared memory (plain loads from
// the peers' tiles, each CTA taking its share of the elements in slab order: a fixed order, so the result
// is the same from run to run), and each element of Y is read, added to and written once.
constexpr int kSpmmChunk = 8;     // k-steps of activations staged at a time
constexpr int kSpmmThreads = 512; // 16 warps: 8 strips x 2 (tiles of 256 columns) or 4 strips x 4 (tiles of 128)
constexpr int kSpmmPer = 4;       // k-steps per warp and chunk, at most

template <int RR>
__device__ __forceinline__ void spmm_add(float (&acc)[RR], uint32_t w, const uint8_t* xrow) {
    const uint32_t k = (w >> 5) & 127u;
    const float v = __uint_as_float(w & kSlotValueMask);
    if constexpr (RR == 1) {
        acc[0] = fmaf(v, __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(xrow)[k] << 16), acc[0]);
    } else {
#pragma unroll
        for (int c = 0; c < RR / 8; ++c) {
            const uint4 q = *reinterpret_cast<const uint4*>(xrow + k * (2 * RR) + 16 * c);
            const uint32_t x[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                acc[8 * c + 2 * i] = fmaf(v, bf16lo(x[i]), acc[8 * c + 2 * i]);
                acc[8 * c + 2 * i + 1] = fmaf(v, bf16hi(x[i]), acc[8 * c + 2 * i + 1]);
            }
        }
    }
}

template <int RR>
__global__ void __launch_bounds__(kSpmmThreads, 2) fq_spmm_kernel(const uint16_t* __restrict__ X, const uint32_t* __restrict__ indptr,
                                                    const uint32_t* __restrict__ info, const uint4* __restrict__ packed,
                                                    uint16_t* __restrict__ Y, uint32_t M, uint32_t K, uint32_t N,
                                                    uint32_t BN, uint32_t slabs) {
    extern __shared__ __align__(16) uint8_t spmm_smem[];
    const uint32_t NB = BN / 4, NS = BN / 32, KW = kSpmmThreads / 32 / NS, KT = K / kBK;
    float* red = reinterpret_cast<float*>(spmm_smem);                 // [RR][BN] sums of this slab
    uint8_t* xs = spmm_smem + (size_t)RR * BN * 4;                    // [kSpmmChunk * 128][RR] BF16, k-major
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t strip = warp % NS, kw = warp / NS, g = lane & 7, t = lane >> 3;
    const uint32_t tile = blockIdx.x / slabs, slab = blockIdx.x - tile * slabs;
    const uint32_t kt0 = slab * KT / slabs, kt1 = (slab + 1) * KT / slabs;
    float acc[RR];
#pragma unroll
    for (int i = 0; i < RR; ++i) acc[i] = 0.0f;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (kt0 >= kt1) asm volatile("griddepcontrol.wait;" ::: "memory");     // a slab without k-steps still adds to Y below

    for (uint32_t c0 = kt0; c0 < kt1; c0 += kSpmmChunk) {
        const uint32_t nk = min((uint32_t)kSpmmChunk, kt1 - c0);
        uint32_t inf[kSpmmPer], base[kSpmmPer];
#pragma unroll
        for (int j = 0; j < kSpmmPer; ++j) {
            const uint32_t kl = kw + j * KW;
            inf[j] = 0, base[j] = 0;
            if (kl < nk) {
                const size_t u = (size_t)tile * KT + c0 + kl;
                inf[j] = __ldg(info + u * NB + strip * 8 + g);
                base[j] = __ldg(indptr + u);
            }
        }
        uint32_t w[kSpmmPer][4];
        const uint32_t* pk[kSpmmPer];
#pragma unroll
        for (int j = 0; j < kSpmmPer; ++j) {
            pk[j] = reinterpret_cast<const uint32_t*>(packed + base[j] + (inf[j] & 0xffffu));
            const uint32_t depth = (inf[j] >> 16) & 0xffu;
#pragma unroll
            for (int d = 0; d < 4; ++d) w[j][d] = (uint32_t)d < depth ? __ldg(pk[j] + d * 4 + t) : 0u;
        }
        // descriptors and packets are weights; X and Y may come from the grid before this one in the stream
        if (c0 == kt0) asm volatile("griddepcontrol.wait;" ::: "memory");
        // the chunk's activations: a thread takes eight consecutive k of one batch row at a time
        constexpr int XU = RR == 1 ? 1 : RR * 16 * kSpmmChunk / kSpmmThreads;
        uint4 xr[XU];
#pragma unroll
        for (int j = 0; j < XU; ++j) {
            const uint32_t e = tid + j * kSpmmThreads, m = e % RR, o = e / RR;
            xr[j] = make_uint4(0, 0, 0, 0);
            if (o < 16 * nk && m < M) xr[j] = __ldg(reinterpret_cast<const uint4*>(X + (size_t)m * K + (size_t)c0 * kBK) + o);
        }
#pragma unroll
        for (int j = 0; j < XU; ++j) {
            const uint32_t e = tid + j * kSpmmThreads, m = e % RR, o = e / RR;
            if (o < 16 * kSpmmChunk) {
                if constexpr (RR == 1) {
                    *reinterpret_cast<uint4*>(xs + 16 * o) = xr[j];
                } else {
                    // value i of the eight goes to row 8 o + i; the lanes of a warp that hold other octets
                    // start at other i, so that one store instruction never hits a bank twice
                    const uint32_t v[4] = {xr[j].x, xr[j].y, xr[j].z, xr[j].w};
                    const uint32_t rot = (lane / RR) & 7u;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t ii = (i + rot) & 7u;
                        const uint32_t word = ii & 4 ? (ii & 2 ? v[3] : v[2]) : (ii & 2 ? v[1] : v[0]);
                        *reinterpret_cast<uint16_t*>(xs + (size_t)(8 * o + ii) * (2 * RR) + 2 * m) =
                            (uint16_t)(ii & 1 ? word >> 16 : word);
                    }
                }
            }
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < kSpmmPer; ++j) {
            const uint8_t* xrow = xs + (size_t)(kw + j * KW) * kBK * (2 * RR);
            const uint32_t depth = (inf[j] >> 16) & 0xffu, tail = inf[j] >> 24;
            const uint32_t dmax = __reduce_max_sync(0xffffffffu, depth);
#pragma unroll
            for (int d = 0; d < 4; ++d)
                if ((uint32_t)d < dmax) spmm_add<RR>(acc, w[j][d], xrow);
            for (uint32_t d = 4; d < depth; ++d) spmm_add<RR>(acc, __ldg(pk[j] + d * 4 + t), xrow);
            for (uint32_t d = depth; d < depth + tail; ++d) {             // tail: a slot names its column
                const uint4 q4 = __ldg(reinterpret_cast<const uint4*>(pk[j]) + d);
                const uint32_t wd[4] = {q4.x, q4.y, q4.z, q4.w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (((wd[e] >> kSlotColShift) & 3u) == t) spmm_add<RR>(acc, wd[e], xrow);
            }
        }
        __syncthreads();                                                  // the tile is overwritten by the next chunk
    }

    // the warps of a strip, then the slabs of the tile
    const uint32_t col = strip * 32 + lane;
    for (uint32_t r = 0; r < KW; ++r) {
        if (kw == r) {
#pragma unroll
            for (int m = 0; m < RR; ++m) red[m * BN + col] = r ? red[m * BN + col] + acc[m] : acc[m];
        }
        __syncthreads();
    }
    cg::cluster_group cluster = cg::this_cluster();
    if (slabs > 1) cluster.sync(); else __syncthreads();
    const uint32_t E = M * BN, e0 = slab * E / slabs, e1 = (slab + 1) * E / slabs;
    for (uint32_t e = e0 + tid; e < e1; e += kSpmmThreads) {
        float sum = 0.0f;
        for (uint32_t s2 = 0; s2 < slabs; ++s2) sum += slabs > 1 ? cluster.map_shared_rank(red, s2)[e] : red[e];
        uint16_t* y = Y + (size_t)(e / BN) * N + (size_t)tile * BN + (e % BN);
        *y = float_to_bf16_bits(bf16_bits_to_float(*y) + sum);
    }
    if (slabs > 1) cluster.sync();                                        // peers may still be reading this tile
}

// ----------------------------------------------------------------------------- launch plumbing

struct Plan {
    Params p;
    uint32_t threads, smem, grid;
    bool general;    // the layer needs the general form of the outlier step
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

// Rows kept per epilogue thread of the tcgen05 kernel, and the MMA's batch columns, for a launch of M rows.
static inline uint32_t rr_of(uint32_t m) { return m <= 1 ? 1u : (m <= 4 ? 4u : (m <= 8 ? 8u : (m <= 16 ? 16u : 32u))); }
static inline uint32_t nmma_of(uint32_t m) { return (uint32_t)nmma_rows((int)rr_of(m)); }      // limb rows of the MMA operand

// Plan of a launch of up to 32 rows (16 with groups of 64: the accumulators of both groups must fit in tensor memory).
static fq_status_t make_plan(const fq_layout_t* L, uint32_t M, bool sparse, Plan& pl) {
    const uint32_t BN = L->BN, NB = L->buckets_per_tile, GPS = kBK / L->group;
    const uint32_t NMMA = nmma_of(M), RR = rr_of(M);
    Params& p = pl.p;
    std::memset(&p, 0, sizeof(p));
    p.M = M; p.K = L->K; p.N = L->N; p.KT = L->K / kBK; p.NT = L->N / BN; p.NB = NB;
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
    const uint32_t xch_bytes = epilogue_sets((int)RR) == 2 ? BN * RR * 4 : 0;
    uint32_t stage = 0, S = 0;
    for (;;) {
        p.off_sz = w_bytes;
        p.off_xcan = p.off_sz + round_up(sz_bytes, 128);
        // the k-step's activation block lands here as one copy: limbs (NMMA rows x 128 k, one byte each),
        // scales and sums, FP32 copy (kernels with outliers only)
        p.off_xmeta = p.off_xcan + blob_meta_off((int)RR);
        p.off_xt = p.off_xcan + blob_xt_off((int)RR, (int)GPS);
        p.off_info = p.off_xt + xt_bytes;
        p.off_coo = p.off_info + (sparse ? round_up(NB * 4, 128) : 0);
        stage = round_up(p.off_coo + cap * 16, 128);
        S = std::min<uint32_t>(8, (kSmemBudget - 1024 - xch_bytes) / stage);
        if (S >= 4 || cap <= 64) break;
        cap = std::max<uint32_t>(64, cap / 2);  // oversized tiles read their tail from global memory
    }
    if (S < 2) return fail(FQ_ERR_UNSUPPORTED_SHAPE, "shared-memory stages do not fit");
    p.coo_cap = cap; p.stages = S; p.stage_bytes = stage;
    // hot columns, tiles larger than the staged part, or an encoding whose sizes were not recorded
    pl.general = sparse && (L->max_tail_packets > 0 || L->max_tile_packets > cap || !L->tilecoo_encoded);
    p.off_xch = S * stage;
    p.off_bar = p.off_xch + xch_bytes;
    pl.smem = p.off_bar + 1024;
    pl.threads = 32 * (kTcFirstUnpack + (1 + epilogue_sets((int)RR)) * (BN / 32));
    pl.grid = grid;
    return FQ_OK;
}

// Short jobs go to fq_direct_kernel: launches of up to 16 rows on layers with so few strips of 32 columns and
// so few k-steps that a CTA of the streaming kernel would get only a handful of units, and its fixed costs
// (ring start-up, settlement of split tiles) would be most of the call.  Returns the warps per CTA of the
// direct kernel, 0 = not a short job.  The bounds are where it measured faster than the streaming kernel
// on B200: every strip a CTA of its own on its own SM and at most two k-steps to a warp (32 warps up to 8 rows,
// 16 warps with twice the accumulators for 9-16 rows); for a single row also up to two CTAs of 16 warps to an SM.
typedef void (*DirectFn)(const DirectParams);
static inline uint32_t direct_warps(const fq_layout_t* L, uint32_t rows) {
    const int sms = sm_count_cached();
    if (sms <= 0 || rows > 16 || L->kernel_hint == 1) return 0;
    const uint32_t strips = L->N / 32, KT = L->K / kBK;
    if (strips <= (uint32_t)sms) {
        if (rows <= 8) return KT <= 64 ? 32u : 0u;
        return KT <= 32 ? 16u : 0u;
    }
    return (rows == 1 && strips <= 2u * (uint32_t)sms && KT <= 32) ? 16u : 0u;
}
template <int MO, int MS, int W>
static DirectFn pick_direct_group(uint32_t g, bool sparse) {
    if (!sparse) return g == 64 ? (DirectFn)fq_direct_kernel<MO, 8 * MO, 64, false, W> : (DirectFn)fq_direct_kernel<MO, 8 * MO, 128, false, W>;
    return g == 64 ? (DirectFn)fq_direct_kernel<MO, MS, 64, true, W> : (DirectFn)fq_direct_kernel<MO, MS, 128, true, W>;
}
template <int W>
static DirectFn pick_direct_rows(uint32_t rows, uint32_t g, bool sparse) {
    if (rows == 1) return pick_direct_group<1, 1, W>(g, sparse);
    if (rows <= 4) return pick_direct_group<1, 4, W>(g, sparse);
    return pick_direct_group<1, 8, W>(g, sparse);
}
static DirectFn pick_direct(uint32_t rows, uint32_t warps, uint32_t g, bool sparse) {
    if (rows > 8) return pick_direct_group<2, 16, 16>(g, sparse);
    return warps == 32 ? pick_direct_rows<32>(rows, g, sparse) : pick_direct_rows<16>(rows, g, sparse);
}

// Scratch layout: status word and header, tile-arrival counters, FP32 partial slots, then the activation
// blocks fq_prep_x_kernel writes for the launch in flight (one per k-step).
struct Scratch {
    size_t off_partials, off_xb, total;
};
// Which kernel serves a launch is decided by its rows alone: up to 16 rows the warp-level MMA kernel, 17 to 32
// rows the tcgen05 kernel (its MMAs cost the same for any number of batch rows up to 42; with groups of 64 its
// two accumulators per unit fit in tensor memory only up to 16 rows, so such layers stay with the first).
static inline bool tc_serves(const fq_layout_t* L, uint32_t rows) { return rows > 16 && L->group == 128; }
static inline uint32_t rows_per_launch(const fq_layout_t* L, uint32_t rows_left) { return tc_serves(L, rows_left) ? std::min<uint32_t>(rows_left, 32u) : std::min<uint32_t>(rows_left, 16u); }
static Scratch scratch_layout(const fq_layout_t* L, uint32_t rows) {
    const bool tc = tc_serves(L, rows);
    const size_t prow = tc ? 32 : 16;                     // batch rows of an FP32 partial slot
    Scratch sc;
    sc.off_partials = kWsHeaderBytes + kWsCounterBytes;
    sc.off_xb = sc.off_partials + (size_t)kMaxCtas * 2 * L->BN * prow * 4;
    sc.total = sc.off_xb + (tc ? (size_t)(L->K / kBK) * blob_bytes(32, (int)(kBK / L->group)) : 0);
    return sc;
}

typedef void (*PrepFn)(const uint16_t*, uint32_t, uint32_t, uint8_t*);
static PrepFn pick_prep() { return fq_prep_x_kernel<32, 128>; }      // 17 to 32 rows, groups of 128: one variant

typedef void (*KernelFn)(const Params);

struct MmaPlan {
    MmaParams p;
    uint32_t threads, smem, grid;
    uint32_t ngrp;   // groups of dense warps
    bool general;    // the layer needs the general form of the outlier step
};
typedef void (*MmaKernelFn)(const MmaParams);

// Plan of the streaming kernel (fq_mma_kernel): M <= 16 per launch.
static fq_status_t make_plan_mma(const fq_layout_t* L, uint32_t M, bool sparse, MmaPlan& pl) {
    const uint32_t BN = L->BN, NB = L->buckets_per_tile, GPS = kBK / L->group;
    const uint32_t MO = M <= 8 ? 1 : 2, ROWS = 8 * MO;
    const uint32_t NDW = BN / 32;
    MmaParams& p = pl.p;
    std::memset(&p, 0, sizeof(p));
    p.M = M; p.K = L->K; p.N = L->N; p.KT = L->K / kBK; p.NT = L->N / BN; p.NB = NB;
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

// MS: form of the outlier step (1: single batch row, one column per lane; 8: rows split over the lanes);
// NGRP: groups of dense warps; HOT: general form of the outlier step
// (long bucket lists shared out, packets beyond the staged part of a tile)
template <int BN, int MO, int G, bool HOT>
static MmaKernelFn pick_mma_sparse(bool sparse, uint32_t ms, uint32_t ngrp) {
    if constexpr (MO == 1) {
        if (ngrp == 2) {
            if (!sparse) return (MmaKernelFn)fq_mma_kernel<BN, MO, G, false, 8, 2, false>;
            if (ms == 1) return (MmaKernelFn)fq_mma_kernel<BN, MO, G, true, 1, 2, HOT>;
            if (ms == 4) return (MmaKernelFn)fq_mma_kernel<BN, MO, G, true, 4, 2, HOT>;
            return (MmaKernelFn)fq_mma_kernel<BN, MO, G, true, 8, 2, HOT>;
        }
        if (sparse && ms == 1) return (MmaKernelFn)fq_mma_kernel<BN, MO, G, true, 1, 1, HOT>;
        if (sparse && ms == 4) return (MmaKernelFn)fq_mma_kernel<BN, MO, G, true, 4, 1, HOT>;
    }
    if constexpr (MO == 2) {
        if (ngrp == 2) return sparse ? (MmaKernelFn)fq_mma_kernel<BN, MO, G, true, 8, 2, HOT> : (MmaKernelFn)fq_mma_kernel<BN, MO, G, false, 8, 2, false>;
    }
    if (!sparse) return (MmaKernelFn)fq_mma_kernel<BN, MO, G, false, 8, 1, false>;
    return (MmaKernelFn)fq_mma_kernel<BN, MO, G, true, 8, 1, HOT>;
}
template <int BN, int MO>
static MmaKernelFn pick_mma_group(uint32_t g, bool sparse, uint32_t ms, uint32_t ngrp, bool hot) {
    if (g == 64) return hot ? pick_mma_sparse<BN, MO, 64, true>(sparse, ms, ngrp) : pick_mma_sparse<BN, MO, 64, false>(sparse, ms, ngrp);
    return hot ? pick_mma_sparse<BN, MO, 128, true>(sparse, ms, ngrp) : pick_mma_sparse<BN, MO, 128, false>(sparse, ms, ngrp);
}
static MmaKernelFn pick_mma_kernel(uint32_t bn, uint32_t M, uint32_t g, bool sparse, uint32_t ngrp, bool hot) {
    const uint32_t mo = M <= 8 ? 1 : 2, ms = M <= 1 ? 1 : (M <= 4 ? 4 : 8);
    if (bn == 128) return mo == 1 ? pick_mma_group<128, 1>(g, sparse, ms, ngrp, hot) : pick_mma_group<128, 2>(g, sparse, ms, ngrp, hot);
    return mo == 1 ? pick_mma_group<256, 1>(g, sparse, ms, ngrp, hot) : pick_mma_group<256, 2>(g, sparse, ms, ngrp, hot);
}

template <int BN, int RR, int G>
static KernelFn pick_tc_sparse(bool sparse, bool hot) {
    if (!sparse) return (KernelFn)fq_tc_kernel<BN, RR, G, false, false>;
    return hot ? (KernelFn)fq_tc_kernel<BN, RR, G, true, true> : (KernelFn)fq_tc_kernel<BN, RR, G, true, false>;
}
static KernelFn pick_kernel(uint32_t bn, bool sparse, bool hot) {      // 17 to 32 rows, groups of 128: one variant per tile width
    return bn == 128 ? pick_tc_sparse<128, 32, 128>(sparse, hot) : pick_tc_sparse<256, 32, 128>(sparse, hot);
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

// Argument checks of the device entry points: nothing is enqueued when one fails.
static fq_status_t check_gemm_args(const fq_layout_t* L, const void* X, uint32_t M, const void* wq, const void* scale,
                                   const void* zero, const void* indptr, const void* info, const void* packed, void* Y,
                                   void* workspace, bool sparse) {
    if (!layout_ok(L)) return fail(FQ_ERR_INVALID_ARG, "bad layout");
    if (M < 1 || M > FQ_MAX_M) return fail(FQ_ERR_INVALID_ARG, "M = %u outside [1, %u]", M, FQ_MAX_M);
    if (!X || !wq || !scale || !zero || !Y || !workspace) return fail(FQ_ERR_INVALID_ARG, "null device pointer");
    if (sparse && (!indptr || !info)) return fail(FQ_ERR_INVALID_ARG, "null Tile-COO pointer");
    if (sparse && !packed && (L->max_tile_packets || !L->tilecoo_encoded)) return fail(FQ_ERR_INVALID_ARG, "null packet pointer");
    if (!aligned(X, 16) || !aligned(Y, 16) || !aligned(wq, 128) || !aligned(scale, 128) || !aligned(zero, 128) ||
        !aligned(workspace, 128) || (sparse && (!aligned(indptr, 4) || !aligned(info, 128) || !aligned(packed, 128))))
        return fail(FQ_ERR_INVALID_ARG, "misaligned device pointer");
    return FQ_OK;
}

static fq_status_t launch_gemm(const fq_layout_t* L, const void* X, uint32_t M, const void* wq, const void* scale,
                               const void* zero, const void* indptr, const void* info, const void* packed, void* Y,
                               void* workspace, size_t workspace_bytes, void* stream, bool sparse) {
    fq_status_t st = check_gemm_args(L, X, M, wq, scale, zero, indptr, info, packed, Y, workspace, sparse);
    if (st != FQ_OK) return st;
    const size_t need = scratch_layout(L, M).total;
    if (workspace_bytes < need) return fail(FQ_ERR_BUFFER_TOO_SMALL, "workspace holds %zu bytes, %zu needed", workspace_bytes, need);
    const Scratch sc = scratch_layout(L, M);
    cudaLaunchAttribute attr[1];
    std::memset(attr, 0, sizeof(attr));
    // Programmatic dependent launch: a grid may become resident while the kernel before it in the stream
    // drains.  Its producer warps then already stream weights (which no kernel writes); everything that touches
    // X, Y or the scratch first executes griddepcontrol.wait, after which all memory operations of the earlier
    // grids are complete and visible.
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    for (uint32_t m0 = 0; m0 < M;) {
        const uint32_t mb = rows_per_launch(L, M - m0);
        const uint16_t* Xm = (const uint16_t*)X + (size_t)m0 * L->K;
        uint16_t* Ym = (uint16_t*)Y + (size_t)m0 * L->N;
        cudaLaunchConfig_t cfg;
        std::memset(&cfg, 0, sizeof(cfg));
        cfg.stream = (cudaStream_t)stream;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e;
        if (tc_serves(L, mb)) {
            Plan pl;
            st = make_plan(L, mb, sparse, pl);
            if (st != FQ_OK) return st;
            Params& p = pl.p;
            const uint32_t rr = rr_of(mb);
            uint8_t* xb = (uint8_t*)workspace + sc.off_xb;
            p.Y = Ym;
            p.wq = (const uint8_t*)wq; p.scale = (const uint16_t*)scale; p.zero = (const uint16_t*)zero;
            p.indptr = (const uint32_t*)indptr; p.info = (const uint32_t*)info; p.packed = (const uint4*)packed;
            p.status = (uint32_t*)workspace;
            p.counters = (uint32_t*)((uint8_t*)workspace + kWsHeaderBytes);
            p.partials = (float*)((uint8_t*)workspace + sc.off_partials);
            p.xblob = xb;
            KernelFn fn = pick_kernel(L->BN, sparse, pl.general);
            e = ensure_smem_attr((const void*)fn, (int)kSmemBudget);
            if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
            // the activation blocks of these rows, then the fused kernel
            const uint32_t warps = rr * (L->K / kBK);
            cfg.gridDim = dim3((warps + 3) / 4);
            cfg.blockDim = dim3(128);
            cfg.dynamicSmemBytes = 0;
            e = cudaLaunchKernelEx(&cfg, pick_prep(), Xm, mb, L->K, xb);
            if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "activation preparation launch: %s", cudaGetErrorString(e));
            cfg.gridDim = dim3(pl.grid);
            cfg.blockDim = dim3(pl.threads);
            cfg.dynamicSmemBytes = pl.smem;
            e = cudaLaunchKernelEx(&cfg, fn, p);
        } else if (direct_warps(L, mb)) {
            DirectParams p;
            std::memset(&p, 0, sizeof(p));
            p.X = Xm; p.Y = Ym;
            p.wq = (const uint8_t*)wq; p.scale = (const uint16_t*)scale; p.zero = (const uint16_t*)zero;
            p.indptr = (const uint32_t*)indptr; p.info = (const uint32_t*)info; p.packed = (const uint4*)packed;
            p.status = (uint32_t*)workspace;
            p.M = mb; p.K = L->K; p.N = L->N; p.KT = L->K / kBK; p.BN = L->BN; p.NB = L->buckets_per_tile;
            const uint32_t warps = direct_warps(L, mb);
            cfg.gridDim = dim3(L->N / 32);
            cfg.blockDim = dim3(32 * warps);
            // per warp: rows of activations, their k-major copy, scale and zero rows, staged packets; the warps'
            // sums reuse those bytes
            cfg.dynamicSmemBytes = warps * kDirectWarpBytes;
            DirectFn dfn = pick_direct(mb, warps, L->group, sparse);
            e = ensure_smem_attr((const void*)dfn, 32 * kDirectWarpBytes);
            if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
            e = cudaLaunchKernelEx(&cfg, dfn, p);
        } else {
            MmaPlan pl;
            st = make_plan_mma(L, mb, sparse, pl);
            if (st != FQ_OK) return st;
            MmaParams& p = pl.p;
            p.X = Xm; p.Y = Ym;
            p.wq = (const uint8_t*)wq; p.scale = (const uint16_t*)scale; p.zero = (const uint16_t*)zero;
            p.indptr = (const uint32_t*)indptr; p.info = (const uint32_t*)info; p.packed = (const uint4*)packed;
            p.status = (uint32_t*)workspace;
            p.counters = (uint32_t*)((uint8_t*)workspace + kWsHeaderBytes);
            p.partials = (float*)((uint8_t*)workspace + sc.off_partials);
            MmaKernelFn fn = pick_mma_kernel(L->BN, mb, L->group, sparse, pl.ngrp, pl.general);
            e = ensure_smem_attr((const void*)fn, (int)kSmemBudget);
            if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
            cfg.gridDim = dim3(pl.grid);
            cfg.blockDim = dim3(pl.threads);
            cfg.dynamicSmemBytes = pl.smem;
            e = cudaLaunchKernelEx(&cfg, fn, p);
        }
        if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
        m0 += mb;
    }
    return FQ_OK;
}

template <int RR>
static cudaError_t launch_spmm(const fq_layout_t* L, const uint16_t* X, uint32_t M, const void* indptr, const void* info,
                               const void* packed, uint16_t* Y, uint32_t slabs, cudaStream_t stream) {
    const uint32_t smem = (uint32_t)RR * L->BN * 4 + kSpmmChunk * kBK * RR * 2;
    cudaError_t e = ensure_smem_attr((const void*)fq_spmm_kernel<RR>, 64 * 1024);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(L->N / L->BN * slabs);
    cfg.blockDim = dim3(kSpmmThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute at[2];
    std::memset(at, 0, sizeof(at));
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = slabs, at[0].val.clusterDim.y = 1, at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;        // as the fused launches: the descriptors
    at[1].val.programmaticStreamSerializationAllowed = 1;                 // and first slots load during the tail of
    cfg.attrs = at, cfg.numAttrs = 2;                                     // the kernel before (the dense half)
    return cudaLaunchKernelEx(&cfg, fq_spmm_kernel<RR>, X, (const uint32_t*)indptr, (const uint32_t*)info,
                              (const uint4*)packed, Y, M, L->K, L->N, L->BN, slabs);
}

}  // namespace fq

using namespace fq;

extern "C" {

fq_status_t fq_workspace_bytes(const fq_layout_t* L, uint32_t M, size_t* bytes) {
    if (!layout_ok(L) || !bytes) return fail(FQ_ERR_INVALID_ARG, "bad layout or null output");
    if (M < 1 || M > FQ_MAX_M) return fail(FQ_ERR_INVALID_ARG, "M = %u outside [1, %u]", M, FQ_MAX_M);
    *bytes = scratch_layout(L, M).total;
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
    // every argument error is reported before anything is put on the stream (the scratch pointer stands in for itself)
    fq_status_t st = check_gemm_args(L, X, M, wq, scale, zero, tile_indptr, bucket_info, packed_outliers, Y, (void*)256, true);
    if (st != FQ_OK) return st;
    const size_t need = scratch_layout(L, M).total;
    if (need > (size_t)FQ_STATIC_SCRATCH_BYTES)
        return fail(FQ_ERR_BUFFER_TOO_SMALL,
                    "this call needs %zu bytes of scratch but the built-in scratch holds %zu (M <= %u always fits); "
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
    if (!aligned(X, 16) || !aligned(Y, 16) || !aligned(packed_outliers, 16))
        return fail(FQ_ERR_INVALID_ARG, "misaligned device pointer");
    const int sms = sm_count_cached();
    if (sms <= 0) return fail(FQ_ERR_CUDA, "no CUDA device: %s", cudaGetErrorString(cudaGetLastError()));
    const uint32_t NT = L->N / L->BN, KT = L->K / kBK;
    // slabs of a tile = one cluster (at most eight CTAs): as many as it takes to put about two CTAs on every SM
    const uint32_t slabs = std::max<uint32_t>(1, std::min<uint32_t>(std::min<uint32_t>(8, KT), (uint32_t)(2 * sms) / NT));
    for (uint32_t m0 = 0; m0 < M; m0 += 16) {
        const uint32_t mb = std::min<uint32_t>(16, M - m0);
        const uint16_t* Xm = (const uint16_t*)X + (size_t)m0 * L->K;
        uint16_t* Ym = (uint16_t*)Y + (size_t)m0 * L->N;
        cudaStream_t st = (cudaStream_t)cuda_stream;
        cudaError_t e = mb == 1 ? launch_spmm<1>(L, Xm, mb, tile_indptr, bucket_info, packed_outliers, Ym, slabs, st)
                      : mb <= 8 ? launch_spmm<8>(L, Xm, mb, tile_indptr, bucket_info, packed_outliers, Ym, slabs, st)
                                : launch_spmm<16>(L, Xm, mb, tile_indptr, bucket_info, packed_outliers, Ym, slabs, st);
        if (e != cudaSuccess) return fail(FQ_ERR_CUDA, "spmm launch: %s", cudaGetErrorString(e));
    }
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
        // A call that gave up left some tile-arrival counters short: clear the status word and all of them, so
        // that the next call on this scratch starts from a clean state (Y of the failed call is undefined).
        cudaMemsetAsync(workspace, 0, kWsHeaderBytes + kWsCounterBytes, s);
        cudaStreamSynchronize(s);
        return fail((fq_status_t)(int32_t)word, "the device reported status %d (-5: a bounded wait expired, -6: Tile-COO descriptors do not match the staged packets)", (int32_t)word);
    }
    return FQ_OK;
}

}  // extern "C"
