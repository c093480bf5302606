// Internal declarations shared by the host codec and the device entry points.
#pragma once
#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "huffllm.h"

static_assert(sizeof(huffllm_desc) == 256, "the descriptor is the 256-byte blob header");

namespace huffllm {

constexpr uint32_t kTileRows = 16;      // rows of a chunk tile
constexpr uint32_t kBlockCols = 32;     // columns of one block (16 weights per lane)
constexpr uint32_t kLagBits = 7;        // zero bits in front of every bit sequence
constexpr uint32_t kSeqs = 64;          // bit sequences per chunk: two per lane (rows g and g + 8)
constexpr uint32_t kDefaultBudget = 8;  // default joint code-length bound
constexpr uint32_t kMinBudget = 8, kMaxBudget = 12;
constexpr uint32_t kRecordUnit = 128;   // record offsets are counted in this many bytes

huffllm_status fail(huffllm_status st, const char *fmt, ...);
void clear_error();

// Geometry checks common to host and device calls; returns OK or sets the error.
huffllm_status check_desc(const huffllm_desc *d);

inline uint32_t blocks_in_chunk(const huffllm_desc &d, uint32_t kc) {
    uint64_t left = d.cols - (uint64_t)kc * d.chunk_cols;
    uint64_t c = left < d.chunk_cols ? left : d.chunk_cols;
    return (uint32_t)((c + kBlockCols - 1) / kBlockCols);
}

}  // namespace huffllm
