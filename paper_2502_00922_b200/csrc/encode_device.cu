// Device-side encoder: builds the same blob as huffllm_encode, byte for byte, from weights that already sit in
// device memory.  Compression is an offline, one-time step (Section 3.1); on the host it takes seconds per decoder
// layer, here it is three short passes over the tensor, so a model can be compressed while it is being loaded.
//
// One thread per bit sequence (64 per chunk), as in the format: thread q of a chunk owns lane q / 2 and row half q % 2,
// so neighbouring threads write neighbouring raw bytes and the two halves of a lane sit in one warp.
//   pass 1  code lengths only -> words per sequence of every chunk, coded bits
//   scan    record offsets (the index section), payload size, largest record
//   pass 2  raw part and coded part of every record
//   pass 3  the checksum term of every record
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <vector>

#include "internal.h"

namespace huffllm {

struct EncTotals {
    unsigned long long payload_units, coded_bits, checksum;
    uint32_t max_words, bad;     // bad: 1 = a symbol without codeword, 2 = payload beyond the 32-bit record index
};

struct EncArgs {
    const uint16_t *w;
    uint64_t rows, cols, n_chunks;
    uint32_t Kc, KC, fp16, lag_bits, pad, vec_ok;
    uint32_t *words, *chunk_bits, *index;
    uint8_t *payload;
    EncTotals *totals;
    uint8_t len[256];
    uint32_t bits[256];
};

constexpr uint32_t kEncThreads = 256, kEncChunks = kEncThreads / 64;

// byte of a group's 32-bit word that takes weight j's mantissa bits, and the one that takes its sign (the raw-byte layout)
__host__ __device__ constexpr uint32_t raw_mant_byte(uint32_t j) { return ((j & 1u) << 1) | (j >> 1); }
__host__ __device__ constexpr uint32_t raw_sign_byte(uint32_t j) { return (raw_mant_byte(j) + 1u) & 3u; }
static_assert(raw_mant_byte(0) == kRawMantByte[0] && raw_mant_byte(1) == kRawMantByte[1] && raw_mant_byte(2) == kRawMantByte[2] &&
              raw_mant_byte(3) == kRawMantByte[3], "raw-byte layout");
static_assert(raw_sign_byte(0) == kRawSignByte[0] && raw_sign_byte(1) == kRawSignByte[1] && raw_sign_byte(2) == kRawSignByte[2] &&
              raw_sign_byte(3) == kRawSignByte[3], "raw-byte layout");

__device__ __forceinline__ uint32_t enc_blocks_of(const EncArgs &A, uint32_t kc) {
    uint64_t left = A.cols - (uint64_t)kc * A.Kc;
    return (uint32_t)(((left < A.Kc ? left : A.Kc) + 31) / 32);
}
__device__ __forceinline__ uint32_t enc_raw_bytes(const EncArgs &A, uint32_t nkb) {
    return A.fp16 ? (nkb * 64u + 127u) & ~127u : nkb * 512u;
}

// The eight weights of (row r, columns c .. c + 7), pad words outside the tensor.
__device__ __forceinline__ void enc_load8(const EncArgs &A, uint64_t r, uint64_t c, uint32_t (&v)[8]) {
    if (r < A.rows && c + 8 <= A.cols && A.vec_ok) {
        const uint4 q = __ldg((const uint4 *)(A.w + r * A.cols + c));
        const uint32_t x[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = (x[i >> 1] >> (16 * (i & 1))) & 0xFFFFu;
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = (r < A.rows && c + i < A.cols) ? A.w[r * A.cols + c + i] : A.pad;
    }
}

struct EncThread {
    uint32_t sub, q, lane, half, seq;
    uint64_t c, r, col0;
    uint32_t kc, nkb;
    bool active;
};
__device__ __forceinline__ EncThread enc_thread(const EncArgs &A) {
    EncThread T;
    T.sub = threadIdx.x >> 6;
    T.q = threadIdx.x & 63;
    T.lane = T.q >> 1;
    T.half = T.q & 1;
    T.seq = T.lane + 32 * T.half;
    T.c = (uint64_t)blockIdx.x * kEncChunks + T.sub;
    T.active = T.c < A.n_chunks;
    const uint64_t cc = T.active ? T.c : 0;
    const uint32_t rg = (uint32_t)(cc / A.KC);
    T.kc = (uint32_t)(cc % A.KC);
    T.nkb = enc_blocks_of(A, T.kc);
    T.r = (uint64_t)rg * 16 + (T.lane >> 2) + 8 * T.half;
    T.col0 = (uint64_t)T.kc * A.Kc + (T.lane & 3) * 8;
    return T;
}

__global__ void __launch_bounds__(kEncThreads) encode_size_kernel(const __grid_constant__ EncArgs A) {
    __shared__ uint32_t s_max[kEncChunks], s_sum[kEncChunks], s_bad;
    __shared__ uint8_t s_len[256];
    s_len[threadIdx.x] = A.len[threadIdx.x];
    if (threadIdx.x < kEncChunks) s_max[threadIdx.x] = s_sum[threadIdx.x] = 0;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    const EncThread T = enc_thread(A);
    if (T.active) {
        uint32_t bits = 0, bad = 0;
        for (uint32_t kb = 0; kb < T.nkb; ++kb) {
            uint32_t v[8];
            enc_load8(A, T.r, T.col0 + kb * 32, v);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (A.fp16) {
                    const uint32_t l0 = s_len[(v[i] >> 10) & 31], l1 = s_len[32 + ((v[i] >> 5) & 31)], l2 = s_len[64 + (v[i] & 31)];
                    bad |= (!l0 || !l1 || !l2) ? 1u : 0u;
                    bits += l0 + l1 + l2;
                } else {
                    const uint32_t l = s_len[(v[i] >> 7) & 0xFF];
                    bad |= l ? 0u : 1u;
                    bits += l;
                }
            }
        }
        atomicMax(&s_max[T.sub], bits + A.lag_bits);
        atomicAdd(&s_sum[T.sub], bits);
        if (bad) s_bad = 1;
    }
    __syncthreads();
    if (T.active && T.q == 0) {
        A.words[T.c] = max(1u, (s_max[T.sub] + 31) / 32);
        A.chunk_bits[T.c] = s_sum[T.sub];
    }
    if (threadIdx.x == 0 && s_bad) atomicOr(&A.totals->bad, 1u);
}

// Record offsets: an exclusive prefix sum of the record sizes (in 128-byte units), by a single CTA.
__global__ void __launch_bounds__(1024) encode_scan_kernel(const __grid_constant__ EncArgs A) {
    __shared__ unsigned long long s_warp[32], s_carry, s_bits[32];
    __shared__ uint32_t s_maxw[32];
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) s_carry = 0;
    unsigned long long bits = 0;
    uint32_t maxw = 0, over = 0;
    __syncthreads();
    for (uint64_t base = 0; base < A.n_chunks; base += 1024) {
        const uint64_t c = base + tid;
        unsigned long long units = 0;
        if (c < A.n_chunks) {
            const uint32_t W = A.words[c];
            units = (enc_raw_bytes(A, enc_blocks_of(A, (uint32_t)(c % A.KC))) + (unsigned long long)W * 256ull) / kRecordUnit;
            bits += A.chunk_bits[c];
            maxw = max(maxw, W);
        }
        unsigned long long incl = units;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            unsigned long long n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= (uint32_t)o) incl += n;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        unsigned long long before = s_carry;
        for (uint32_t w2 = 0; w2 < warp; ++w2) before += s_warp[w2];
        const unsigned long long excl = before + incl - units;
        if (c < A.n_chunks) {
            A.index[c] = (uint32_t)excl;
            if (excl + units > 0xFFFFFFFFull) over = 1;
        }
        __syncthreads();
        if (tid == 1023) s_carry = before + incl;
        __syncthreads();
    }
    // totals
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        bits += __shfl_xor_sync(0xFFFFFFFFu, bits, o);
        maxw = max(maxw, __shfl_xor_sync(0xFFFFFFFFu, maxw, o));
        over |= __shfl_xor_sync(0xFFFFFFFFu, over, o);
    }
    if (lane == 0) {
        s_bits[warp] = bits;
        s_maxw[warp] = maxw;
        if (over) atomicOr(&A.totals->bad, 2u);
    }
    __syncthreads();
    if (tid == 0) {
        unsigned long long b = 0;
        uint32_t m = 0;
        for (int i = 0; i < 32; ++i) {
            b += s_bits[i];
            m = max(m, s_maxw[i]);
        }
        A.index[A.n_chunks] = (uint32_t)s_carry;
        A.totals->payload_units = s_carry;
        A.totals->coded_bits = b;
        A.totals->max_words = m;
    }
}

__global__ void __launch_bounds__(kEncThreads) encode_write_kernel(const __grid_constant__ EncArgs A) {
    __shared__ uint8_t s_len[256];
    __shared__ uint32_t s_bits[256];
    s_len[threadIdx.x] = A.len[threadIdx.x];
    s_bits[threadIdx.x] = A.bits[threadIdx.x];
    __syncthreads();
    const EncThread T = enc_thread(A);
    if (!T.active) return;          // whole 64-thread groups leave together: the shuffles below stay inside a group's warps
    const uint32_t W = A.words[T.c], raw_bytes = enc_raw_bytes(A, T.nkb);
    uint8_t *raw = A.payload + (uint64_t)A.index[T.c] * kRecordUnit;
    uint32_t *coded = (uint32_t *)(raw + raw_bytes) + T.seq;      // word j of this sequence at coded[64 j]
    unsigned long long acc = 0;
    uint32_t nacc = A.lag_bits, j = 0;
    auto append = [&](uint32_t b, uint32_t len) {                 // len <= 16, nacc < 32
        acc |= (unsigned long long)b << nacc;
        nacc += len;
        if (nacc >= 32) {
            coded[(size_t)64 * j++] = (uint32_t)acc;
            acc >>= 32;
            nacc -= 32;
        }
    };
    for (uint32_t kb = 0; kb < T.nkb; ++kb) {
        uint32_t v[8];
        enc_load8(A, T.r, T.col0 + kb * 32, v);
        if (A.fp16) {
            // sign bit of weight i: pair p = i / 2 (+ 4 for the row g + 8 sequence), bit p (+ 8 if i is odd)
            uint32_t sg = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                sg |= (v[i] >> 15) << ((i >> 1) + 4 * T.half + 8 * (i & 1));
                append(s_bits[(v[i] >> 10) & 31], s_len[(v[i] >> 10) & 31]);
                append(s_bits[32 + ((v[i] >> 5) & 31)], s_len[32 + ((v[i] >> 5) & 31)]);
                append(s_bits[64 + (v[i] & 31)], s_len[64 + (v[i] & 31)]);
            }
            sg |= __shfl_xor_sync(0xFFFFFFFFu, sg, 1);
            if (T.half == 0) *(uint16_t *)(raw + kb * 64 + T.lane * 2) = (uint16_t)sg;
        } else {
            uint32_t word[2] = {0, 0};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                word[i >> 2] |= (v[i] & 0x7Fu) << (8 * raw_mant_byte(i & 3));
                word[i >> 2] |= ((v[i] >> 8) & 0x80u) << (8 * raw_sign_byte(i & 3));
                const uint32_t e = (v[i] >> 7) & 0xFF;
                append(s_bits[e], s_len[e]);
            }
            *(uint2 *)(raw + kb * 512 + T.lane * 16 + T.half * 8) = make_uint2(word[0], word[1]);
        }
    }
    if (nacc) coded[(size_t)64 * j++] = (uint32_t)acc;
    for (; j < W; ++j) coded[(size_t)64 * j] = 0;
    if (A.fp16 && (T.nkb & 1u) && T.q < 32) *(uint16_t *)(raw + T.nkb * 64 + T.q * 2) = 0;   // padding of the sign plane
}

// Checksum term of every record: the same byte-serial hash the host encoder and the validator use, one thread per
// record (the records were just written and mostly still sit in L2).
__global__ void __launch_bounds__(128) encode_checksum_kernel(const __grid_constant__ EncArgs A) {
    const uint64_t c = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned long long term = 0;
    if (c < A.n_chunks) {
        const uint32_t r0 = A.index[c], r1 = A.index[c + 1];
        const uint4 *p = (const uint4 *)(A.payload + (uint64_t)r0 * kRecordUnit);
        unsigned long long h = 1469598103934665603ull;
        for (uint64_t i = 0; i < (uint64_t)(r1 - r0) * (kRecordUnit / 16); ++i) {
            const uint4 q = __ldcg(p + i);
            const uint32_t x[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int k = 0; k < 16; ++k) h = (h ^ ((x[k >> 2] >> (8 * (k & 3))) & 0xFFu)) * 1099511628211ull;
        }
        term = h * (2 * c + 1);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) term += __shfl_xor_sync(0xFFFFFFFFu, term, o);
    if ((threadIdx.x & 31) == 0 && term) atomicAdd(&A.totals->checksum, term);
}

}  // namespace huffllm

using namespace huffllm;

extern "C" huffllm_status huffllm_encode_device_scratch_bytes(uint64_t rows, uint64_t cols, uint32_t chunk_elems, size_t *bytes) {
    clear_error();
    if (!bytes) return fail(HUFFLLM_ERR_INVALID_ARG, "null output");
    if (rows == 0 || cols == 0 || rows > (1ull << 31) || cols > (1ull << 31) || chunk_elems % 512 || chunk_elems < 512 || chunk_elems > 16384)
        return fail(HUFFLLM_ERR_INVALID_ARG, "bad shape or chunk_elems");
    const uint64_t Kc = chunk_elems / kTileRows, n_chunks = ((rows + 15) / 16) * ((cols + Kc - 1) / Kc);
    *bytes = (size_t)(256 + 8 * n_chunks);
    return HUFFLLM_OK;
}

extern "C" huffllm_status huffllm_encode_device(const huffllm_codebook *cb, const uint16_t *w_dev, uint64_t rows, uint64_t cols,
                                                uint32_t chunk_elems, void *blob_dev, size_t blob_cap, void *scratch_dev,
                                                size_t scratch_bytes, huffllm_desc *desc, huffllm_stream stream) {
    clear_error();
    if (!cb || !w_dev || !blob_dev || !scratch_dev || !desc) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer");
    size_t need = 0;
    huffllm_status st = huffllm_encode_device_scratch_bytes(rows, cols, chunk_elems, &need);
    if (st != HUFFLLM_OK) return st;
    if (scratch_bytes < need) return fail(HUFFLLM_ERR_BUFFER_TOO_SMALL, "scratch needs %llu bytes", (unsigned long long)need);
    if (((uintptr_t)w_dev & 1u) || ((uintptr_t)blob_dev & 255u) || ((uintptr_t)scratch_dev & 255u))
        return fail(HUFFLLM_ERR_INVALID_ARG, "blob and scratch must be 256-byte aligned");
    const uint32_t Kc = chunk_elems / kTileRows, RG = (uint32_t)((rows + 15) / 16), KC = (uint32_t)((cols + Kc - 1) / Kc);
    huffllm_desc d;
    fill_desc_fixed(cb, rows, cols, chunk_elems, Kc, RG, KC, &d);
    if (blob_cap < d.off_payload) return fail(HUFFLLM_ERR_BUFFER_TOO_SMALL, "blob capacity below the fixed sections");
    if (d.n_chunks > 0x7FFFFFFFull * kEncChunks) return fail(HUFFLLM_ERR_UNSUPPORTED, "too many chunks");

    cudaStream_t s = (cudaStream_t)stream;
    uint8_t *blob = (uint8_t *)blob_dev, *scr = (uint8_t *)scratch_dev;
    EncArgs A = {};
    A.w = w_dev;
    A.rows = rows;
    A.cols = cols;
    A.n_chunks = d.n_chunks;
    A.Kc = Kc;
    A.KC = KC;
    A.fp16 = d.dtype == HUFFLLM_FP16 ? 1u : 0u;
    A.lag_bits = d.lag_bits;
    A.pad = d.pad_word;
    A.vec_ok = (cols % 8 == 0 && ((uintptr_t)w_dev & 15u) == 0) ? 1u : 0u;
    A.totals = (EncTotals *)scr;
    A.words = (uint32_t *)(scr + 256);
    A.chunk_bits = A.words + d.n_chunks;
    A.index = (uint32_t *)(blob + d.off_index);
    A.payload = blob + d.off_payload;
    encoder_tables(cb, A.len, A.bits);

    cudaError_t e;
    auto cuda_fail = [&](const char *what) { return fail(HUFFLLM_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e)); };
    if ((e = cudaMemsetAsync(scr, 0, 256, s)) != cudaSuccess) return cuda_fail("cudaMemsetAsync");
    if ((e = cudaMemsetAsync(blob, 0, d.off_payload, s)) != cudaSuccess) return cuda_fail("cudaMemsetAsync");
    const uint32_t grid = (uint32_t)((d.n_chunks + kEncChunks - 1) / kEncChunks);
    encode_size_kernel<<<grid, kEncThreads, 0, s>>>(A);
    encode_scan_kernel<<<1, 1024, 0, s>>>(A);
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail("encode size pass");
    EncTotals tot;
    if ((e = cudaMemcpyAsync(&tot, scr, sizeof(tot), cudaMemcpyDeviceToHost, s)) != cudaSuccess || (e = cudaStreamSynchronize(s)) != cudaSuccess)
        return cuda_fail("encode size pass");
    if (tot.bad & 1u) return fail(HUFFLLM_ERR_INVALID_ARG, "a weight uses a symbol the codebook has no codeword for");
    if (tot.bad & 2u) return fail(HUFFLLM_ERR_UNSUPPORTED, "payload exceeds the 32-bit record index");
    d.max_words = tot.max_words;
    d.payload_bytes = tot.payload_units * kRecordUnit;
    d.blob_bytes = d.off_payload + d.payload_bytes + kTailSlack;
    d.coded_bits = tot.coded_bits;
    if (blob_cap < d.blob_bytes)
        return fail(HUFFLLM_ERR_BUFFER_TOO_SMALL, "blob needs %llu bytes, capacity is %llu", (unsigned long long)d.blob_bytes, (unsigned long long)blob_cap);

    if ((e = cudaMemsetAsync((uint8_t *)blob + d.off_payload + d.payload_bytes, 0, kTailSlack, s)) != cudaSuccess) return cuda_fail("clearing the tail");
    encode_write_kernel<<<grid, kEncThreads, 0, s>>>(A);
    encode_checksum_kernel<<<(uint32_t)((d.n_chunks + 127) / 128), 128, 0, s>>>(A);
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail("encode write pass");
    if ((e = cudaMemcpyAsync(&tot, scr, sizeof(tot), cudaMemcpyDeviceToHost, s)) != cudaSuccess || (e = cudaStreamSynchronize(s)) != cudaSuccess)
        return cuda_fail("encode write pass");
    d.payload_checksum = tot.checksum;

    // header, code lengths and table: bytes [0, off_index), assembled on the host
    std::vector<uint8_t> fixed((size_t)d.off_index, 0);
    write_fixed_sections(cb, d, fixed.data());
    if ((e = cudaMemcpyAsync(blob, fixed.data(), fixed.size(), cudaMemcpyHostToDevice, s)) != cudaSuccess || (e = cudaStreamSynchronize(s)) != cudaSuccess)
        return cuda_fail("header copy");
    *desc = d;
    return HUFFLLM_OK;
}
