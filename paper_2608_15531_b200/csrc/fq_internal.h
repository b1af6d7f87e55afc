// Internal declarations shared by the host packer/encoder and the CUDA launchers.
#pragma once
#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "fq.h"

namespace fq {

// thread-local error text returned by fq_last_error()
char* error_buffer();
inline fq_status_t fail(fq_status_t code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(error_buffer(), 512, fmt, ap);
    va_end(ap);
    return code;
}

inline bool layout_ok(const fq_layout_t* L) {
    if (!L || L->abi != FQ_ABI_VERSION) return false;
    if (L->BK != FQ_BK || (L->BN != 128 && L->BN != 256)) return false;
    if (L->group != 64 && L->group != 128) return false;
    if (L->K == 0 || L->N == 0 || L->K % FQ_BK != 0 || L->N % L->BN != 0) return false;
    if (L->buckets_per_tile != L->BN / 4) return false;      // a bucket is four columns, in every kernel
    if (L->wq_interleave != 3 || L->coo_unit_bytes != 16) return false;
    if (L->value_type > FQ_VALUE_FP16 || L->slot_order > 1 || L->kernel_hint > 1) return false;
    return true;
}

// A Tile-COO slot (32 bits): bits 13-31 the value, an FP32 number cut to ten explicit significand bits (holds
// every BF16 and every FP16 number exactly); bits 5-11 the row inside the tile; bits 3-4 the column number
// inside the bucket; bits 0-2 and 12 zero.  A slot whose value bits are zero is padding.
constexpr uint32_t kSlotValueMask = 0xffffe000u;
constexpr uint32_t kSlotValueShift = 13;
constexpr uint32_t kSlotColShift = 3;
constexpr uint32_t kSlotStrayMask = 0x00001007u;

// Upper bound on persistent CTAs per launch; sizes the scratch independently of the device.
constexpr uint32_t kMaxCtas = 192;
constexpr uint32_t kMaxTilesN = 1024;       // column tiles; the scratch holds 8 arrival counters for each
constexpr size_t kWsHeaderBytes = 256;      // status word lives at offset 0
constexpr size_t kWsCounterBytes = kMaxTilesN * 8 * 4;

}  // namespace fq
