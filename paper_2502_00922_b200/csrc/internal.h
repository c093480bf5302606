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
// Zero bits in front of every bit sequence: they put the table index where the device forms a table address from the
// shifted window with one logic operation (BF16: one table, 128 bytes per entry; FP16: 64 bytes per entry).
inline uint32_t lag_bits_for(uint32_t dtype) { return dtype == HUFFLLM_FP16 ? 6u : 7u; }
constexpr uint32_t kSeqs = 64;          // bit sequences per chunk: two per lane (rows g and g + 8)
constexpr uint32_t kDefaultBudget = 8;  // default joint code-length bound
constexpr uint32_t kMinBudget = 8, kMaxBudget = 12;
// FP16 fields are limited one by one and have 32 symbols each: 7 bits are allowed there as well (128-entry tables, which
// the device keeps once per lane: lookups without bank conflicts)
inline uint32_t min_budget_for(uint32_t dtype) { return dtype == HUFFLLM_FP16 ? 7u : kMinBudget; }
constexpr uint32_t kRecordUnit = 128;   // record offsets are counted in this many bytes
// Zero bytes behind the payload, part of the blob: the product kernel's requests into L2 run up to 2 KB past the record
// they are issued in, and with this slack they never leave the blob.
constexpr uint64_t kTailSlack = 4096;

huffllm_status fail(huffllm_status st, const char *fmt, ...);
void clear_error();

// Geometry checks common to host and device calls; returns OK or sets the error.
huffllm_status check_desc(const huffllm_desc *d);

// Bytes of the raw part of a record with nkb blocks: BF16 one byte per weight; FP16 one sign bit per weight
// ([block][lane] uint16), padded to the record unit.
inline uint32_t raw_part_bytes(uint32_t dtype, uint32_t nkb) {
    return dtype == HUFFLLM_FP16 ? (nkb * 64u + kRecordUnit - 1) / kRecordUnit * kRecordUnit : nkb * 512u;
}

// BF16 raw bytes: the four weights i = 4 q + j of a group share a 32-bit word; weight j's seven mantissa bits go to the
// low bits of byte kRawMantByte[j] of the word and its sign to bit 7 of byte kRawSignByte[j].
constexpr uint32_t kRawMantByte[4] = {0, 2, 1, 3};
constexpr uint32_t kRawSignByte[4] = {1, 3, 2, 0};

// Pieces of the host encoder that the device encoder shares (defined with the codebook, in the host codec).
void fill_desc_fixed(const huffllm_codebook *cb, uint64_t rows, uint64_t cols, uint32_t chunk_elems, uint32_t Kc, uint32_t RG,
                     uint32_t KC, huffllm_desc *out);
void write_fixed_sections(const huffllm_codebook *cb, const huffllm_desc &d, uint8_t *base);
void encoder_tables(const huffllm_codebook *cb, uint8_t len[256], uint32_t bits[256]);
uint32_t codebook_dtype(const huffllm_codebook *cb);

inline uint32_t blocks_in_chunk(const huffllm_desc &d, uint32_t kc) {
    uint64_t left = d.cols - (uint64_t)kc * d.chunk_cols;
    uint64_t c = left < d.chunk_cols ? left : d.chunk_cols;
    return (uint32_t)((c + kBlockCols - 1) / kBlockCols);
}

}  // namespace huffllm
