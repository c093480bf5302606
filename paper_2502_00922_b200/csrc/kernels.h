// Launch interface between the C-ABI entry points (api.cu) and the kernels (kernels.cu).
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace huffllm {

constexpr uint32_t kMaxMats = 8;   // matrices one launch can work through

// One matrix of a launch.
struct MatArgs {
    const uint8_t *blob;       // device
    uint64_t off_lut, off_index, off_payload;
    uint64_t rows, cols;
    uint32_t payload_units;    // payload size in 128-byte units
    uint32_t n_chunks, chunk_cols, col_chunks;
    uint32_t cta_first, cta_count;   // the CTAs of the launch that work on this matrix (each at least one chunk)
    uint32_t cta_chunks, cta_extra;  // n_chunks / cta_count and n_chunks % cta_count: the first cta_extra CTAs take one chunk more
    const uint16_t *x;         // [batch][cols]
    float *y;                  // [batch][rows]
    float *ws_partial;         // [cta_count * 2][16 * batch]
    float *ws_warp_pieces;     // batch 9..16 only: [cta_count][2 * 32][16 * batch], the pieces warps of one CTA exchange
    unsigned int *ws_ticket;   // [cta_count] arrival counters, zero between calls
    uint16_t *out;             // decode output
};

struct KernelArgs {
    uint32_t n_mats, total_chunks, lut_bits;
    uint32_t fmt;              // 0: BF16 blobs (one table), 1: FP16 blobs (three tables)
    uint32_t lut_align, lut_size;   // shared-memory window of the table(s): a power-of-two alignment above the index bits, and its bytes
    uint32_t slot_bytes;       // shared-memory bytes of one slot: largest max_words * 256
    uint32_t pair_recip;       // floor(2^32 / (slots * slot_bytes)): umulhi(x, pair_recip) is x / (slots * slot_bytes) or one less
    uint32_t guard_bytes;      // readable bytes kept free behind the last slot
    uint32_t part_bytes;       // bytes at the end of dynamic shared memory for the CTA's partial sums (tensor-core path: the stages of activations)
    uint32_t dyn_smem_bytes;
    uint32_t batch;            // 1..8 (register path), 9..16 (register path with two tiles of activations)
    int32_t *err;              // may be null
    // tensor-core small-batch path only
    uint32_t tc_npad;          // batch rounded up to 16, 32 or 64
    uint32_t tc_tiles;         // 128-row tiles a CTA decodes side by side (8 warps each): 1..4
    uint32_t tc_reserved[2];   // (the per-matrix values of that path live in TcArgs; these words keep the fields behind
    void *tc_reserved_p[2];    //  them where the register-path kernels were measured with them)
    MatArgs m[kMaxMats];
    // (behind the matrices, so that the fields the hot loops read keep their places)
    uint32_t slots;            // slots per decoder warp: 2 (the next record lands while this one is decoded), or 1 where two would
                               // leave too few warps a slot (large records: the feeder then waits for a slot before every copy).
                               // Kernels with single slots exist for FP16 blobs and for BF16 blobs with 8-bit tables.
    uint32_t fp16_flat;        // FP16 blobs: both mantissa halves of every matrix of the launch carry the flat 5-bit code
};

// Arguments of the tensor-core kernel: the launch description plus, per matrix, its work items and where their pieces meet.
// (The CTAs of a launch are dealt to the matrices as in the other kernels: m[i].cta_first / cta_count.)
struct TcArgs {
    KernelArgs k;
    uint32_t m_tiles[kMaxMats];        // row tiles (of the decoder warps' row groups) of matrix i
    uint32_t ksplit[kMaxMats];         // ranges its column chunks are cut into; work items = m_tiles * ksplit
    float *partial[kMaxMats];          // [m_tiles * ksplit][32 warps][npad / 2][32]
    unsigned int *ticket[kMaxMats];    // [m_tiles][32], zero between calls
};

cudaError_t launch_decode(const KernelArgs &k, uint32_t grid, cudaStream_t stream);
cudaError_t launch_gemm(const KernelArgs &k, uint32_t grid, cudaStream_t stream);
cudaError_t launch_gemm_tc(const TcArgs &t, uint32_t grid, cudaStream_t stream);
cudaError_t launch_stage_copy(void *dst, const void *src, uint64_t bytes, uint32_t sms, cudaStream_t stream);
// The dense bf16 comparison product: up to kMaxMats matrices per launch, rows dealt to the warps round-robin.
struct PlainMat {
    const uint16_t *w;         // [rows][cols] bf16, device
    const uint16_t *x;         // [cols]
    float *y;                  // [rows]
    uint64_t rows, cols;
    uint32_t row_first;        // number of the matrix's first row among the launch's rows
};
struct PlainArgs {
    uint32_t n_mats, total_rows;
    PlainMat m[kMaxMats];
};
cudaError_t launch_plain_gemv(const PlainArgs &a, uint32_t sms, cudaStream_t stream);

}  // namespace huffllm
