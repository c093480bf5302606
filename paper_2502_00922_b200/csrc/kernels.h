// Launch interface between the C-ABI entry points (api.cu) and the kernels (kernels.cu).
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace huffllm {

struct KernelArgs {
    const uint8_t *blob;       // device
    uint64_t off_lut, off_index, off_payload;
    uint32_t payload_units;    // payload size in 128-byte units
    uint64_t rows, cols, n_chunks;
    uint32_t chunk_cols, col_chunks, lut_bits;
    uint32_t slot_bytes;       // shared-memory bytes of one slot: (max_words + 1) * 256
    uint32_t guard_bytes;      // readable bytes kept free behind the last slot
    uint32_t part_bytes;       // bytes at the end of dynamic shared memory for the CTA's partial sums
    uint32_t dyn_smem_bytes;
    const uint16_t *x;         // [batch][cols]
    float *y;                  // [batch][rows]
    uint32_t batch;            // 1..8
    float *ws_partial;         // [grid * 2][16 * batch]
    unsigned int *ws_ticket;   // [grid] arrival counters, zero between calls
    uint16_t *out;             // decode output
    int32_t *err;              // may be null
};

cudaError_t launch_decode(const KernelArgs &k, uint32_t grid, cudaStream_t stream);
cudaError_t launch_gemm(const KernelArgs &k, uint32_t grid, cudaStream_t stream);
cudaError_t launch_plain_gemv(const uint16_t *w, uint64_t rows, uint64_t cols, const uint16_t *x, float *y, uint32_t sms,
                              cudaStream_t stream);

}  // namespace huffllm
