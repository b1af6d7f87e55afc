/*
 * fq.h -- C ABI of the fused outlier-aware W4A16 decode matmul for NVIDIA B200
 * (sm_100a).
 *
 *      Y = X * dequant(W_Q) + X * W_O                                  (Eq. 1)
 *
 * X is a small-M BF16 activation block (M x K, row-major), W_Q is K x N
 * group-quantised asymmetric INT4 (Eq. 2, Eq. 3; groups of 64 or 128 rows along
 * K, BF16 scale and BF16-held integer zero-point per group and column) and W_O
 * is a sparse BF16 outlier matrix in the Tile-COO encoding (Section 3.2.1,
 * Table 1).  Y is M x N BF16, row-major, accumulated in FP32 and rounded once.
 *
 * Conventions
 *   - Every function returns an fq_status_t; nothing throws across the ABI.
 *     fq_last_error() gives a thread-local text for the last failure.
 *   - "host" pointers are ordinary memory, "device" pointers are CUDA global
 *     memory of the current device.  The caller owns every buffer; the library
 *     allocates nothing that outlives a call.
 *   - Device entry points only enqueue work on `cuda_stream` (a cudaStream_t
 *     passed as void*; NULL = the legacy default stream) and return.  Argument
 *     errors are reported synchronously and nothing is launched.  A device-side
 *     wait that gave up is reported by fq_check_status().
 *   - Device arrays must be 128-byte aligned (16 bytes for X and Y rows, which
 *     follows from K % 8 == 0 and N % 8 == 0).
 *
 * Packed formats (the kernel's choice; the paper leaves them open)
 *
 *   INT4 weights.  BK = 128 rows, BN = 128 or 256 columns per tile.  The buffer
 *   is a sequence of chunks, one per (column tile tn, row tile kt), chunk index
 *   tn * (K/128) + kt, each 16 * BN little-endian 32-bit words.  Word index
 *   inside a chunk is
 *       (j*BN + t)*4 + w
 *   (j = 0..3: 32-row block, t = column inside the tile, w = 0..3: 8-row
 *   block).  Nibble p = i + 4h (i = 0..3, h = 0..1; bits 4p..4p+3) of that
 *   word is the code of
 *       column tn*BN + t
 *       row    kt*128 + 32j + 8w + 2i + h .
 *   (The four words of a column's 32-row block are 16 contiguous bytes, and
 *   consecutive columns follow each other: a thread that owns a column fetches
 *   them with one 128-bit load, a warp without bank conflicts.  One
 *   shift-and-mask turns nibbles i and i+4 of a word into a BF16 pair of
 *   consecutive rows, the operand order of the warp-level MMA; one mask each
 *   turns the even and the odd nibbles into four bytes, the operand of the
 *   integer MMA.)
 *
 *   Scale, zero.  (K/group) x N row-major BF16.  zero holds the integer 0..15.
 *
 *   Tile-COO.  Tiles are BK x BN, tile index t = tn * (K/128) + kt.
 *   tile_indptr[t] .. tile_indptr[t+1]: the tile's range of 16-byte packets in
 *   packed_outliers (N_tile + 1 entries, uint32).  NB = BN/4 buckets per tile,
 *   and the bucket of tile column c is fixed: 8*(c/32) + c%8, i.e. the four
 *   columns {g, g+8, g+16, g+24} of a 32-column block share a bucket; column
 *   g + 8j is column number j of its bucket.  (These are the columns whose
 *   accumulators one group of four lanes holds after the m16n8k16 MMAs of the
 *   kernels, so a bucket is applied in registers; the paper's
 *   load-balancing column permutation, Section 3.2.2, is replaced by this
 *   static assignment.)
 *     bucket_info[t*NB + b] = offset | depth << 16 | tail << 24  (uint16, uint8,
 *   uint8): bucket b of tile t owns depth + tail packets starting `offset`
 *   packets after the tile's first.
 *     A packet is four little-endian 32-bit slots; a slot holds one outlier:
 *   bits 13-31 the value — an FP32 number cut to ten explicit significand
 *   bits, which holds every BF16 and every FP16 number exactly (for a BF16
 *   value, bits 16-31 are its bit pattern and bits 13-15 are 0); slot &
 *   0xffffe000 is the value as FP32 —, bits 5-11 the row inside the tile (so
 *   that slot & 0xfe0 is the row times 32), bits 3-4 the column number j, all
 *   other bits 0.  A padding slot has value bits 0 and row 0.
 *     The first `depth` packets of a bucket are column-slotted (padding per
 *   column as in Section 4.2, with the column given by the slot's position
 *   instead of a column index per packet): slot j of packet i is one of the
 *   outliers of column number j (which one is the encoder's choice, see
 *   slot_order below), or a padding slot that still names j.  If no column of
 *   the bucket has more than 32 outliers in the tile, depth is the longest
 *   column's count and tail is 0.  Otherwise depth is 4, and the outliers
 *   beyond the first 4 of each column follow in `tail` packets by (row,
 *   column), four to a packet in any slot, the last one filled with all-zero
 *   padding slots.  Storage: (N_tile+1)*4 + N_tile*NB*4 + 16*packets bytes.
 */
#ifndef FQ_H_
#define FQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t fq_status_t;
#define FQ_OK 0
#define FQ_ERR_INVALID_ARG (-1)       /* null or misaligned pointer, M out of range, bad layout */
#define FQ_ERR_UNSUPPORTED_SHAPE (-2) /* K % 128, N % BN, group not 64/128, bucket count */
#define FQ_ERR_BUFFER_TOO_SMALL (-3)
#define FQ_ERR_CUDA (-4)              /* a CUDA runtime call failed; text in fq_last_error() */
#define FQ_ERR_TIMEOUT (-5)           /* a bounded device-side wait expired */
#define FQ_ERR_FORMAT (-6)            /* Tile-COO validator: bad indptr / offset / index */

#define FQ_ABI_VERSION 2u
#define FQ_VALUE_BF16 0u
#define FQ_VALUE_FP16 1u
#define FQ_MAX_M 128u
#define FQ_BK 128u

/* Plain data, caller-owned.  Filled by fq_get_layout(); fq_encode_tilecoo()
 * writes max_tile_packets, max_bucket_packets and max_tail_packets (the kernels
 * size their staging by the first and choose their outlier path by the third).  Pass the same
 * struct to every later call. */
typedef struct fq_layout {
    uint32_t abi;
    uint32_t K, N;
    uint32_t group;            /* 64 or 128, along K */
    uint32_t BK;               /* 128 */
    uint32_t BN;               /* 128 or 256 */
    uint32_t buckets_per_tile; /* NB = BN / 4 */
    uint32_t wq_interleave;    /* 3: the word order described above */
    uint32_t coo_unit_bytes;   /* 16 */
    uint32_t max_tile_packets; /* largest tile of the encoded W_O, in packets */
    uint32_t max_bucket_packets; /* longest packet list (depth + tail) of one bucket in one tile */
    uint32_t max_tail_packets; /* longest tail; 0 = every packet is column-slotted */
    uint32_t tilecoo_encoded;  /* 1 = the three maxima above describe the arrays in use (set by
                                  fq_encode_tilecoo); 0 = unknown: the kernels assume the worst */
    uint32_t kernel_hint;      /* 0 = the library chooses the kernel of a launch from its rows and the layer's
                                  shape; 1 = never the short-job kernel (one CTA per strip of 32 columns), so
                                  that tests reach the streaming kernels on small layers too */
    uint32_t slot_order;       /* read by fq_encode_tilecoo: 0 = bank-aware order of a column's outliers over its
                                  column-slotted packets (Section 3.2.2, restated for this library's kernels:
                                  packet d of bucket g prefers a row with k mod 4 = (g + d) mod 4); 1 = by row.
                                  Every kernel accepts either; the arrays decode to the same set */
    uint32_t value_type;       /* type of the outlier values handed to fq_encode_tilecoo and returned by
                                  fq_decode_tilecoo, 16 bits each: FQ_VALUE_BF16 (default) or FQ_VALUE_FP16 (IEEE
                                  binary16; Table 1's value field).  The packed slots hold either exactly, and the
                                  kernels read them the same way */
} fq_layout_t;

/* Choose tile sizes for a K x N layer.  bn_hint: 0 = library default (256 when
 * N is a multiple of 256), otherwise 128 or 256.  nb_hint: 0, or BN/4 (the only
 * bucket count there is).  Errors: FQ_ERR_UNSUPPORTED_SHAPE for shapes the
 * kernels cannot tile (K % 128, N % BN, group not 64 or 128, more than 1024
 * column tiles). */
fq_status_t fq_get_layout(uint32_t K, uint32_t N, uint32_t group, uint32_t bn_hint, uint32_t nb_hint,
                          fq_layout_t* out);

/* ---------------------------------------------------------------- host, offline */

/* Byte sizes of the three arrays fq_pack_int4 writes. */
fq_status_t fq_pack_int4_sizes(const fq_layout_t* L, size_t* wq_bytes, size_t* scale_bytes,
                               size_t* zero_bytes);

/*
 * Quantise and pack (Eq. 2 with b = 4, the formulas for s and z that follow
 * Eq. 3).  W: host, K x N row-major binary32.  outlier_mask: host, K x N bytes,
 * 1 = outlier (excluded from the group range, stored with code = zero-point so
 * that it dequantises to 0), may be NULL.  Outputs (host): wq in the chunked
 * order above, scale and zero as (K/group) x N BF16 bit patterns.  Readings
 * where the paper is silent: round-half-to-even, codes and zero-point clamped to
 * 0..15, binary32 arithmetic with the BF16-rounded scale, the group range always
 * contains 0, a degenerate group gets scale 1 and zero 0.
 */
fq_status_t fq_pack_int4(const fq_layout_t* L, const float* W, const uint8_t* outlier_mask, void* wq,
                         uint16_t* scale_bf16, uint16_t* zero_bf16);

/* Section 3.2.1, last remark: padding slots of the packed outliers can hold original weight values.  In the
 * column-slotted packets a bucket is as deep as its longest column, so every other column of the bucket has
 * (depth - count) slots that cost their bytes anyway.  This host function names the weights that go there: for
 * every tile, bucket and column, the (depth - count) non-outlier weights of the column inside the tile with the
 * largest quantisation error |w - s (q - z)| under `mask` (larger first, lower row first among equals; never a
 * weight whose error or whose BF16 value is 0); buckets with a column of more than 32 outliers are left alone.
 * mask_out (K x N bytes, may not alias mask) = mask plus those; *added (may be NULL) = how many.  Packing and
 * encoding under mask_out gives exactly as many packets as under mask.  W: K x N binary32 row-major. */
fq_status_t fq_repurpose_pad_slots(const fq_layout_t* L, const float* W, const uint8_t* mask, uint8_t* mask_out,
                                   uint64_t* added);

/* Inverse of the nibble interleave: wq (host) -> q_canon (host, K x N, one code per byte). */
fq_status_t fq_unpack_int4(const fq_layout_t* L, const void* wq, uint8_t* q_canon);

/*
 * Tile-COO encoder (Section 3.2.1).  Input: COO triplets on the host (k, n,
 * 16 value bits of the type L->value_type names), any order; entries whose
 * value is +-0 are dropped.  Every entry goes to the bucket of its column and
 * is stored as "Tile-COO" above says: column-slotted packets with per-column
 * padding (Section 4.2), and a tail for a bucket with a very long column.  Of
 * the two reorderings of Section 3.2.2 the element order is applied, restated
 * for the kernels' shared-memory reads (L->slot_order); the column-to-bucket
 * assignment is static (see "Tile-COO" above), so the column permutation is
 * not.
 *
 * fq_encode_tilecoo_sizes: element counts of the three arrays (tile_indptr in
 * uint32, bucket_info in uint32, packets in 16-byte units) and the largest
 * tile.  fq_encode_tilecoo: writes them and stores max_tile_packets,
 * max_bucket_packets and max_tail_packets in *L.
 */
fq_status_t fq_encode_tilecoo_sizes(const fq_layout_t* L, const uint32_t* k, const uint32_t* n,
                                    const uint16_t* val_bf16, size_t nnz, size_t* n_indptr,
                                    size_t* n_bucket_info, size_t* n_packets,
                                    uint32_t* max_tile_packets);
fq_status_t fq_encode_tilecoo(fq_layout_t* L, const uint32_t* k, const uint32_t* n,
                              const uint16_t* val_bf16, size_t nnz, uint32_t* tile_indptr,
                              uint32_t* bucket_info, void* packed_outliers, size_t n_packets);

/* Tile-COO -> COO (host).  *nnz_inout: capacity on entry, count on return. */
fq_status_t fq_decode_tilecoo(const fq_layout_t* L, const uint32_t* tile_indptr,
                              const uint32_t* bucket_info, const void* packed_outliers, uint32_t* k,
                              uint32_t* n, uint16_t* val_bf16, size_t* nnz_inout);

/* Structural check of host Tile-COO arrays before they are given to a kernel:
 * monotone indptr ending at n_packets, bucket ranges inside their tile, every
 * slot's indices inside the tile, every outlier in the bucket of its column.
 * FQ_ERR_FORMAT on violation. */
fq_status_t fq_validate_tilecoo(const fq_layout_t* L, const uint32_t* tile_indptr,
                                const uint32_t* bucket_info, const void* packed_outliers,
                                size_t n_packets);

/* --------------------------------------------------------------------- device */

/* Bytes of caller-allocated device scratch for calls with this layout and M.
 * The scratch must be zeroed once before its first use; every completed call
 * leaves it ready for the next one on the same stream.  Calls that may overlap
 * on the GPU need distinct scratch. */
fq_status_t fq_workspace_bytes(const fq_layout_t* L, uint32_t M, size_t* bytes);

/*
 * The fused operator (Eq. 1; Sections 3.1 and 4.1): a launch reads X, W_Q and
 * the Tile-COO tiles, dequantises in registers into tensor-core operands (exact
 * integers, scale and zero-point applied per group in FP32), adds the tile's
 * outliers into the accumulators of their columns, and writes Y once.  Which
 * kernel serves a launch is decided from its rows and the layer's shape alone:
 *   - up to 16 rows: warp-level MMAs (128 + q as BF16).  Layers with so few
 *     32-column strips and k-steps that every CTA's job would be short get one
 *     CTA per strip, whose warps split K among themselves and read the weights
 *     straight into registers; every other layer streams (tile, k-step) units
 *     through a bulk-copy/mbarrier ring on persistent CTAs;
 *   - 17 to 32 rows (a larger M is cut into such launches), groups of 128: a
 *     kernel built on tcgen05.mma with 8-bit integer operands.  Its
 *     activations are block fixed point, 22 bits plus sign relative to the
 *     largest |x| of each row and group, so activations more than 2^14 below
 *     that maximum are rounded (to 2^-22 of it).  Groups of 64 stay with
 *     launches of 16 rows.
 * L->kernel_hint = 1 keeps the one-CTA-per-strip kernel out (for tests).
 * X: device, M x K BF16.  M in [1, FQ_MAX_M].  Y: device, M x N BF16,
 * overwritten.  All other arrays: device copies of the host packer/encoder
 * output.  Partial sums of one output, whether of the warps of a CTA or of
 * several CTAs that share a tile, are added in a fixed order, so results are
 * run-to-run reproducible.
 *
 * Ordering.  Every kernel is launched so that it may become resident while the
 * kernel before it in the stream is still draining (programmatic dependent
 * launch): it then already streams the weight arrays (wq, scale, zero,
 * tile_indptr, bucket_info, packed_outliers), and touches X, Y and the scratch
 * only after that earlier kernel has completed.  So the weight arrays must not
 * be written by a kernel that can still be running when this call is made
 * (they are constants of the layer in any real use); every other dependency
 * through the stream is honoured as usual.
 */
fq_status_t fq_fused_w4a16_outlier_gemm(const fq_layout_t* L, const void* X, uint32_t M,
                                        const void* wq, const void* scale, const void* zero,
                                        const void* tile_indptr, const void* bucket_info,
                                        const void* packed_outliers, void* Y, void* workspace,
                                        size_t workspace_bytes, void* cuda_stream);

/*
 * The same operator for callers that cannot allocate device memory.  (The paper
 * has no counterpart: this is a convenience of the library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a
 * framework's allocator-managed region, in a plug-in that is handed device
 * buffers but may not create any, or in a process whose device-memory budget
 * was handed out completely at start-up.  Such callers still pass X, the packed
 * layer and Y; only the scratch is missing.
 *
 * Instead of a caller-provided workspace, the kernel uses an array that is part
 * of the library image: FQ_STATIC_SCRATCH_BYTES of device memory on every GPU
 * that loads the library, held until the process exits.  That fixes the limit:
 * calls whose fq_workspace_bytes() exceeds it (M > FQ_STATIC_SCRATCH_MAX_M) are
 * refused with FQ_ERR_BUFFER_TOO_SMALL and nothing is launched.  The function calls no cudaMalloc / cudaFree and no allocating
 * library routine; per call it enqueues one small memset (status word and tile
 * counters, which must start at zero) and the kernel.
 *
 * The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress, with that device current); make that first call
 * outside any stream capture.  There is one array per device: every call
 * shares it and finds the previous call's contents, so calls that may overlap
 * on the GPU (different streams) race -- serialise them, or use the entry
 * point above with separate scratch.  Errors otherwise as above; a wait that
 * gave up is not retrievable through fq_check_status() here (the array is not
 * visible to the caller) and shows as undefined Y.
 */
#define FQ_STATIC_SCRATCH_BYTES 6356992u /* 6 MiB + 64 KiB */
#define FQ_STATIC_SCRATCH_MAX_M 16u
fq_status_t fq_fused_w4a16_outlier_gemm_noalloc(const fq_layout_t* L, const void* X, uint32_t M,
                                                const void* wq, const void* scale, const void* zero,
                                                const void* tile_indptr, const void* bucket_info,
                                                const void* packed_outliers, void* Y,
                                                void* cuda_stream);

/* Unfused baseline, dense half: Y = X * dequant(W_Q) (same kernel, sparse path
 * compiled out). */
fq_status_t fq_unfused_gemm(const fq_layout_t* L, const void* X, uint32_t M, const void* wq,
                            const void* scale, const void* zero, void* Y, void* workspace,
                            size_t workspace_bytes, void* cuda_stream);

/* Unfused baseline, sparse half: Y += X * W_O as a separate launch (one per 16
 * rows) that re-reads X and reads, adds to and writes each BF16 element of Y
 * once (the two-kernel scheme the paper compares against, Section 2.2).  A
 * column tile's row tiles are split into at most eight slabs, one CTA each,
 * that form a thread-block cluster and add their FP32 sums through
 * distributed shared memory in slab order (the same bits every run).  Needs no
 * scratch.  Device pointers, same alignment as the fused call; the layout and
 * the descriptors are trusted (a baseline: no format guard). */
fq_status_t fq_unfused_spmm(const fq_layout_t* L, const void* X, uint32_t M, const void* tile_indptr,
                            const void* bucket_info, const void* packed_outliers, void* Y,
                            void* cuda_stream);

/* Same operator as fq_fused_w4a16_outlier_gemm, called with HOST X and HOST Y:
 * copies X to x_dev, runs the kernel, copies Y back from y_dev and waits for
 * the stream.  x_dev / y_dev are caller-allocated device staging buffers of
 * M*K*2 and M*N*2 bytes. */
fq_status_t fq_fused_host_io(const fq_layout_t* L, const void* X_host, uint32_t M, void* x_dev,
                             const void* wq, const void* scale, const void* zero,
                             const void* tile_indptr, const void* bucket_info,
                             const void* packed_outliers, void* y_dev, void* Y_host, void* workspace,
                             size_t workspace_bytes, void* cuda_stream);

/* The same without the final wait: enqueues the copy of X, the kernel and the
 * copy of Y on `cuda_stream` and returns.  X_host must stay valid and Y_host
 * must not be read until the caller has synchronised the stream (use pinned
 * host memory, or the copies are not asynchronous).  Several calls may be
 * enqueued before one synchronisation if each has staging buffers of its own;
 * they may share the scratch, since they run in stream order. */
fq_status_t fq_fused_host_io_async(const fq_layout_t* L, const void* X_host, uint32_t M, void* x_dev,
                                   const void* wq, const void* scale, const void* zero,
                                   const void* tile_indptr, const void* bucket_info,
                                   const void* packed_outliers, void* y_dev, void* Y_host,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Synchronise the stream and return the scratch's status word: FQ_OK,
 * FQ_ERR_TIMEOUT if a bounded wait expired in a kernel, or FQ_ERR_FORMAT if a
 * kernel found bucket descriptors that point outside the packets staged for
 * their tile (a layout struct that does not belong to the uploaded arrays).  Y
 * of such a call is undefined.  A call that gave up leaves tile-arrival
 * counters short, so on an error this function clears the status word and all
 * counters: the scratch is then ready for the next call. */
fq_status_t fq_check_status(void* workspace, void* cuda_stream);

/* Thread-local description of the most recent error; valid until the next call. */
const char* fq_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FQ_H_ */
