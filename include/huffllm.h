/*
 * huffllm — Huffman-compressed 16-bit LLM weights that stay compressed in GPU memory and are
 * decoded on the fly inside the matrix-vector / small-batch matrix products that consume them.
 *
 * The method is Huff-LLM's: each weight is split into bit fields, the sign (and, for BF16, the
 * seven mantissa bits) stay raw, the exponent fields are Huffman coded (BF16 {1,4,4,7}:
 * Section 5.1; FP16 {1,5,5,5}: Section 3.1), compression happens once, offline, on the CPU
 * (Section 3.1), weights stay compressed everywhere and are decompressed only to be multiplied
 * with activations (Section 1, contributions), and the decoder knows a fixed bound L_max on the
 * codeword length (Section 3.2).
 *
 * Conventions for every call
 *   - C ABI, plain pointers and sizes.  "host" / "device" on a pointer says where it must live.
 *   - The caller owns every buffer.  The only object the library allocates is the codebook
 *     (create with huffllm_build_codebook, release with huffllm_codebook_free).
 *   - Weights are row-major [rows = out_features][cols = in_features], as 16-bit patterns.
 *   - Device calls are asynchronous on `stream`, never synchronise, never allocate.
 *   - The decode and product kernels are launched so that their set-up may overlap the tail of the kernel in
 *     front of them on the stream: they read the BLOB (table, record index, first records) before that kernel
 *     has finished, and everything else (x, workspace, y, out) only after it has.  A blob must therefore be
 *     complete in device memory before the kernel that precedes the call on the stream starts; a blob written
 *     by that very kernel (a device-side copy or encoder right in front of the call) needs a stream
 *     synchronisation or an event in between.
 *   - Every call returns a huffllm_status; huffllm_last_error() gives a thread-local message.
 *     Nothing aborts, throws, or traps on the device.
 */
#ifndef HUFFLLM_H
#define HUFFLLM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HUFFLLM_OK = 0,
    HUFFLLM_ERR_INVALID_ARG = 1,      /* null pointer, zero size, misaligned device pointer, bad enum        */
    HUFFLLM_ERR_UNSUPPORTED = 2,      /* valid request this build does not implement (nothing was launched)  */
    HUFFLLM_ERR_BUFFER_TOO_SMALL = 3, /* blob / workspace capacity below what the call needs                 */
    HUFFLLM_ERR_CORRUPT = 4,          /* blob fails validation                                               */
    HUFFLLM_ERR_CUDA = 5,             /* a CUDA runtime call failed; message holds cudaGetErrorString        */
    HUFFLLM_ERR_NOMEM = 6             /* host allocation failed                                              */
} huffllm_status;

typedef enum { HUFFLLM_BF16 = 0, HUFFLLM_FP16 = 1 } huffllm_dtype;

/* How a weight's bits are grouped into coded fields.
 *   HUFFLLM_SPLIT_PAPER           the paper's hardware-friendly splits: BF16 {1,4,4,7} (Section 5.1)
 *   HUFFLLM_SPLIT_WHOLE_EXPONENT  BF16 {1,8,7}: the 8-bit exponent is one symbol of a 256-symbol code.  The
 *                                 paper's entropy table lists this split and Section 3.1 sets it aside because a
 *                                 256-entry CAM is too costly in its hardware decoder; a lookup table in GPU
 *                                 shared memory has no such cost, so the split is offered here.  The device
 *                                 kernels are the same: they see only the table.                              */
typedef enum { HUFFLLM_SPLIT_PAPER = 0, HUFFLLM_SPLIT_WHOLE_EXPONENT = 1 } huffllm_split;

/* A CUDA stream handle (cudaStream_t), spelled without the CUDA headers. */
typedef struct CUstream_st *huffllm_stream;

/* Opaque host object: per-field symbol counts, code lengths, canonical codewords, decode table. */
typedef struct huffllm_codebook huffllm_codebook;

/*
 * Descriptor of an encoded tensor.  It is also, byte for byte, the first 256 bytes of the blob,
 * so a blob saved to disk describes itself (huffllm_validate_blob re-reads it).  Little endian.
 *
 * Blob layout (every section starts on a 256-byte boundary):
 *   header    this struct
 *   codebook  n_fields == 2: uint8 lengths[3][32] (hi-nibble code, lo-nibble code, zeros);
 *             n_fields == 1: uint8 lengths[256] of the whole-exponent code;
 *             n_fields == 3 (FP16): uint8 lengths[3][32] (exponent, upper five, lower five mantissa bits).
 *             0 = symbol unused; codewords are canonical: symbols ordered by
 *             (length, symbol), first codeword 0, next = (previous + 1) << (length growth); a
 *             codeword's most significant bit comes first in the stream
 *   LUT       uint32[1 << lut_bits], indexed by the next lut_bits stream bits (first bit = bit 0);
 *             BF16 entry = (code length of the weight: hi-nibble + lo-nibble code, or the whole-exponent
 *             code) << 16 | exponent << 7, i.e. the exponent already sits where a bf16 word has it.
 *             FP16: three such tables back to back, one per field, indexed by the next lut_bits bits at that
 *             field's position; entry = code length << 16 | symbol << (10, 5, 0): the three entries of a
 *             weight OR-ed together give its 15 low bits
 *   index     uint32[n_chunks + 1]: record offsets from off_payload, in units of 128 bytes
 *   payload   one record per chunk, chunk id = row_group * col_chunks + col_chunk
 *
 * A chunk is a tile of 16 rows x chunk_cols (= chunk_elems / 16) columns, cut into blocks of 32
 * columns (the last column chunk may hold fewer blocks).  It is decoded by 32 lanes; lane
 * l = 4 g + t (g < 8, t < 4) owns rows g and g + 8 of the tile and columns 8t .. 8t+7 of every
 * block, as two independent bit sequences: sequence l holds row g's weights, sequence 32 + l
 * holds row g + 8's, block after block (eight weights per block each).  Positions outside the
 * tensor hold `pad_word`.  Record = raw bytes [block][lane][16] (a lane's 16 bytes are row g's eight
 * weights, then row g + 8's, in groups of four weights per little-endian 32-bit word: weight j of a
 * group has its seven mantissa bits in the low bits of byte (0, 2, 1, 3)[j] of the word and its sign in
 * bit 7 of byte (1, 3, 2, 0)[j], which puts the first pair's bits, and after a rotation by one byte the
 * second pair's, where a packed pair of bf16 words has them), then W rows of 64
 * little-endian uint32 (row j, sequence s): the sequence's bits, bit i in word i / 32 at bit
 * i % 32.  A sequence starts with `lag_bits` zero bits, then for every weight
 * code(exponent >> 4) code(exponent & 15) (n_fields == 2) or code(exponent) (n_fields == 1); bits after
 * the last codeword are zero.
 * FP16 blobs: per weight code(exponent) code(mantissa >> 5) code(mantissa & 31); the raw part of a record is
 * [block][lane] uint16 (padded to a multiple of 128 bytes) holding the signs of the lane's 16 weights of the block:
 * the lane's weights form eight pairs (row g: columns (0,1) (2,3) (4,5) (6,7) of its eight, then row g + 8 likewise);
 * bit p is the sign of the first weight of pair p, bit 8 + p the sign of its second weight.  W is the
 * longest sequence of the chunk in words (all 64 are padded to it).
 * Behind the last record the blob holds 4096 zero bytes (part of blob_bytes): the product kernels ask the cache for
 * bytes up to 2 KB past the record they work on, and with this slack such a request never leaves the blob.
 */
typedef struct huffllm_desc {
    char     magic[4];        /* "HFLM"                                                    */
    uint32_t version;         /* 1                                                         */
    uint32_t dtype;           /* huffllm_dtype                                             */
    uint32_t chunk_elems;     /* weights per chunk: a multiple of 512 in [512, 16384]      */
    uint64_t rows, cols;
    uint32_t tile_rows;       /* 16                                                        */
    uint32_t chunk_cols;      /* chunk_elems / 16                                          */
    uint32_t row_groups;      /* ceil(rows / 16)                                           */
    uint32_t col_chunks;      /* ceil(cols / chunk_cols)                                   */
    uint64_t n_chunks;        /* row_groups * col_chunks                                   */
    uint32_t lut_bits;        /* L_max: BF16: of one weight's coded fields together (8 .. 12); FP16: of each field (7 .. 12) */
    uint32_t lag_bits;        /* 7 (BF16 blobs), 6 (FP16 blobs)                            */
    uint32_t n_fields;        /* coded fields per weight: 2 (BF16 {1,4,4,7}), 1 ({1,8,7}), 3 (FP16 {1,5,5,5}) */
    uint8_t  caps[4];         /* per-field maximum code length chosen under lut_bits       */
    uint16_t pad_word;        /* weight stored at positions outside the tensor            */
    uint16_t flat_fields;     /* FP16 blobs: bit f set = coded field f carries the flat code (all 32 symbols, 5 bits each, the
                                 codeword of symbol s is s): the decoders then read that field without its table.  Written
                                 by the encoders; 0 is always valid (every field is decoded through its table)       */
    uint32_t max_words;       /* largest W over all chunks                                 */
    uint64_t off_codebook, off_lut, off_index, off_payload;   /* byte offsets in the blob */
    uint64_t payload_bytes;   /* 128 * index[n_chunks]                                     */
    uint64_t blob_bytes;      /* total size: off_payload + payload_bytes + 4096 zero bytes  */
    uint64_t coded_bits;      /* sum of codeword lengths over all stored weights           */
    uint64_t raw_bits;        /* raw bits of the rows*cols real weights                    */
    uint64_t payload_checksum;/* sum over chunks of (2 id + 1) * FNV-1a-64(record bytes)   */
    uint8_t  reserved[104];
} huffllm_desc;

/* ------------------------------------------------------------------ host: compress once, offline */

/*
 * Count the coded fields of `w` (host, rows*cols 16-bit words) and build one Huffman code per
 * field for this tensor (Sections 3.1 and 5.1).  `max_code_len` is L_max (Section 3.2) for the
 * coded fields of one weight taken together: for BF16 the hi- and lo-nibble code lengths are
 * capped at (c0, c1) with c0 + c1 <= max_code_len, chosen to minimise the coded size, each code
 * being the optimal length-limited prefix code for its cap; where plain Huffman already fits,
 * the result is plain Huffman.  0 selects the default (8); supported range 8..12.
 * (FP16 also takes 7: its fields have 32 symbols each, and the device keeps 128-entry tables once per lane.)
 * A field with a single used symbol gets a 1-bit code.  An empty tensor is INVALID_ARG.
 * HUFFLLM_FP16 is the paper's {1,5,5,5} split (Section 3.1): sign raw, exponent and the two mantissa halves each
 * with its own code, each limited to max_code_len on its own (Section 3.2 quotes 12 for these 5-bit fields).
 * The device kernels decode every limit from 8 to 12: up to 8 bits per field (FP16) or 9 bits per weight (BF16)
 * with one table lookup per codeword, longer codes with a second lookup for the codewords that exceed 8 bits
 * (slower by the extra instructions; small batches above 8 vectors then run as passes of 8).
 * On success *out owns a new codebook.
 */
huffllm_status huffllm_build_codebook(const uint16_t *w_host, uint64_t rows, uint64_t cols, huffllm_dtype dtype,
                                      uint32_t max_code_len, huffllm_codebook **out);

/*
 * The same for a chosen field split.  HUFFLLM_SPLIT_PAPER is huffllm_build_codebook.  With
 * HUFFLLM_SPLIT_WHOLE_EXPONENT (BF16 only) the exponent byte is coded by one Huffman code of at most
 * max_code_len bits (0 = 8; range 8..12; the optimal length-limited code when plain Huffman is longer);
 * blobs encoded with it have n_fields == 1 and run through the same device calls.
 */
huffllm_status huffllm_build_codebook_split(const uint16_t *w_host, uint64_t rows, uint64_t cols, huffllm_dtype dtype,
                                            huffllm_split split, uint32_t max_code_len, huffllm_codebook **out);

/* Read the code of a whole-exponent codebook: per exponent value its count, code length (0 = unused) and
 * canonical codeword.  Arrays hold 256 entries.  INVALID_ARG for a codebook of another split.        */
huffllm_status huffllm_codebook_get_exponent(const huffllm_codebook *cb, uint64_t counts[256], uint8_t lengths[256],
                                             uint32_t codes[256]);

/* Read one field of a codebook: number of symbols of the field's alphabet, and per symbol its
 * count, code length (0 = unused) and canonical codeword.  Arrays hold 32 entries.            */
huffllm_status huffllm_codebook_get(const huffllm_codebook *cb, uint32_t field, uint32_t *n_symbols,
                                    uint64_t counts[32], uint8_t lengths[32], uint32_t codes[32]);

void huffllm_codebook_free(huffllm_codebook *cb);

/* Upper bound, in bytes, of the blob huffllm_encode can produce for this shape (any codebook).  */
huffllm_status huffllm_encode_bound(uint64_t rows, uint64_t cols, huffllm_dtype dtype, uint32_t chunk_elems,
                                    size_t *max_bytes);

/*
 * Encode `w` (host) with `cb` into `blob` (host, capacity blob_cap, 256-byte aligned recommended):
 * chunked bitstreams with a per-chunk offset index so that chunks decode in parallel.  Every
 * weight must use only symbols the codebook has codewords for (always true for the tensor the
 * codebook was built from), else INVALID_ARG.  *desc receives the descriptor (= blob header).
 */
huffllm_status huffllm_encode(const huffllm_codebook *cb, const uint16_t *w_host, uint64_t rows, uint64_t cols,
                              uint32_t chunk_elems, void *blob_host, size_t blob_cap, huffllm_desc *desc);

/*
 * The same steps for weights that already sit in DEVICE memory (a model being loaded): count on the device, build the
 * codebook from the counts, encode on the device.  The blob is, byte for byte, the one huffllm_encode writes.
 *
 * huffllm_build_codebook_from_counts: counts (host) = BF16: the 256 counters of the exponent byte, i.e. field 1 of
 *   huffllm_split_histogram with widths {1,8,7}; FP16: the 96 counters of exponent, upper and lower mantissa half,
 *   i.e. fields 1..3 of widths {1,5,5,5}.  Same result as huffllm_build_codebook_split on the tensor itself.
 * huffllm_encode_device: w_dev (device, row-major; the fast path wants 16-byte alignment and cols % 8 == 0, anything
 *   else works too), blob_dev and scratch_dev (device, 256-byte aligned; capacities as for huffllm_encode /
 *   huffllm_encode_device_scratch_bytes).  Launches on `stream` and WAITS for it (the descriptor depends on the
 *   payload size and checksum, which only the device knows): this is an offline call, not part of the decode path.
 *   Errors as huffllm_encode; on error the blob's content is unspecified.
 */
huffllm_status huffllm_build_codebook_from_counts(const uint64_t *counts_host, huffllm_dtype dtype, huffllm_split split,
                                                  uint32_t max_code_len, huffllm_codebook **out);
huffllm_status huffllm_encode_device_scratch_bytes(uint64_t rows, uint64_t cols, uint32_t chunk_elems, size_t *bytes);
huffllm_status huffllm_encode_device(const huffllm_codebook *cb, const uint16_t *w_dev, uint64_t rows, uint64_t cols,
                                     uint32_t chunk_elems, void *blob_dev, size_t blob_cap, void *scratch_dev,
                                     size_t scratch_bytes, huffllm_desc *desc, huffllm_stream stream);

/*
 * Check a blob held in host memory before it is uploaded: header fields and geometry, section
 * bounds, Kraft sums of the stored code lengths, the LUT against the codebook, a monotone record
 * index, record sizes, and a walk over every lane's bits (each lane must hold exactly its number
 * of codewords inside its W words, with zero lag and tail bits) and the payload checksum.  Returns CORRUPT on any
 * failure.  On success *desc_out (optional) receives the descriptor.
 */
huffllm_status huffllm_validate_blob(const void *blob_host, size_t bytes, huffllm_desc *desc_out);

/* --------------------------------------------------------- device: decode, and decode fused with products */

/*
 * Scratch bytes the fused products need for this matrix and `batch` activation vectors.  The workspace must be
 * zero-filled once after allocation.  Its first huffllm_workspace_control_bytes(desc) bytes are arrival counters:
 * every call that completes leaves them zero again; the rest holds partial sums and is overwritten freely.
 * After a call that set the error flag, clear those leading bytes before the workspace is used again.
 * Calls that share a workspace must not overlap on the GPU.
 */
huffllm_status huffllm_workspace_bytes(const huffllm_desc *desc, uint32_t batch, size_t *bytes);
huffllm_status huffllm_workspace_control_bytes(const huffllm_desc *desc, size_t *bytes);

/*
 * Decompress a blob (device, 256-byte aligned) to its original 16-bit weights, bit for bit
 * (Section 3.2: sign, exponent and mantissa are concatenated back into the 16-bit weight).
 * `out` (device) receives rows*cols words, row-major.  `err_flag` (device int32, may be null; the same in the
 * product calls) is left alone by a sound blob and otherwise set to: c + 1 if chunk c's record offsets point outside
 * the payload or do not fit (that chunk is skipped, nothing is read through them); 0x40000000 + c + 1 if chunk c's bits
 * made the decoder run past the end of its record (a damaged coded part: the chunk's output is wrong, but no read left
 * the CTA's shared memory: a sequence moves on by at most one row per refill check, and room for that is kept, see
 * huffllm_decode_smem_plan); -1 if a copy never arrived within the wait limit.  A damaged coded part that still ends
 * inside its record is not detectable here: huffllm_validate_blob (host, checksum) is the check for that.
 */
huffllm_status huffllm_decode(const huffllm_desc *desc, const void *blob_dev, uint16_t *out_dev,
                              int32_t *err_flag_dev, huffllm_stream stream);

/*
 * The shared-memory budget a decoder CTA keeps for this blob (host call, no device needed; any pointer may be null):
 * bytes of the decode table(s), bytes of one slot (the coded rows of the largest record: max_words * 256), the number
 * of refill checks per bit sequence and block of 32 columns, and the readable bytes kept behind the last slot,
 * 256 * (3 + checks * blocks per chunk): the furthest row any stream, sound or not, can make the decoder touch.
 */
huffllm_status huffllm_decode_smem_plan(const huffllm_desc *desc, uint32_t *table_bytes, uint32_t *slot_bytes,
                                        uint32_t *refill_checks_per_block, uint32_t *guard_bytes);

/*
 * How a CTA of huffllm_decode (batch 0) or of the products of 1 to 8 vectors is laid out for this blob (host call, no device
 * needed; any pointer may be null).  `smem_bytes_per_cta`: the GPU's opt-in shared memory per CTA, 0 = the B200's 232448.
 * slots_per_warp: 2 where every decoder warp can keep two records in shared memory (the next one lands while this one is
 * decoded), 1 where records are so large that pairs would leave fewer than 31 warps a place and single slots serve at
 * least a quarter more of them.  decoder_warps: how many of a CTA's 31 decoder warps get a place, at least.
 * HUFFLLM_ERR_UNSUPPORTED if not even one record fits.
 */
huffllm_status huffllm_decode_launch_plan(const huffllm_desc *desc, uint32_t batch, uint32_t smem_bytes_per_cta,
                                          uint32_t *slots_per_warp, uint32_t *decoder_warps);

/*
 * y = W x with W taken straight from the compressed blob: weights are decoded in registers and
 * multiplied at once, so only compressed bytes cross the memory bus (Section 1: weights are
 * decompressed only when needed, to multiply with activations).  x: device, cols words of the
 * blob's dtype.  y: rows floats in device memory, or in pinned host memory the device can address (the results
 * then go to the host as the kernels produce them; y is only ever written).  cols must be a multiple of 32 (UNSUPPORTED otherwise;
 * huffllm_decode takes any shape).  Products are exact, sums are accumulated in fp32.
 * Results are bitwise reproducible from run to run.
 */
huffllm_status huffllm_decode_gemv(const huffllm_desc *desc, const void *blob_dev, const uint16_t *x_dev, float *y_dev,
                                   void *workspace_dev, size_t workspace_bytes, int32_t *err_flag_dev,
                                   huffllm_stream stream);

/*
 * Small-batch version: x is [batch][cols] row-major (device), y is [batch][rows] floats (device).
 * batch 1..64.  Which kernel runs is the library's choice and does not change the result's meaning (sums are fp32, their
 * order is fixed for a given call): one vector, 2..8 vectors and 9..16 vectors of BF16 blobs with 8-bit tables multiply from
 * the decoded registers; 17..64 vectors (and 9..16 where that is faster for the matrix's shape, or the only way) go through
 * the tensor core; blobs neither takes at that batch are done in passes of 8 vectors.
 */
huffllm_status huffllm_decode_gemm(const huffllm_desc *desc, const void *blob_dev, const uint16_t *x_dev, uint32_t batch,
                                   float *y_dev, void *workspace_dev, size_t workspace_bytes, int32_t *err_flag_dev,
                                   huffllm_stream stream);

/*
 * Several products in ONE launch: y_i = W_i x_i for i < n (n <= 8; batch <= 8 for every blob, 9..16 for BF16 blobs of
 * max_code_len 8, 17..64 for BF16 blobs of max_code_len 8 or 9 and FP16 blobs of max_code_len 8: UNSUPPORTED otherwise), e.g. the q, k and v
 * projections of a decoder layer, or gate and up.  The chunks of all matrices are spread over the GPU
 * together, so small matrices do not pay a launch, a set-up and a tail each.  Arrays are host arrays
 * of n pointers; every matrix needs its own workspace (each at least workspace_bytes_each long, which must
 * cover huffllm_workspace_bytes of every matrix of the call), its own x_i ([batch][cols_i]) and y_i
 * ([batch][rows_i]).  All blobs must have been encoded with the same max_code_len.
 */
huffllm_status huffllm_decode_gemm_multi(uint32_t n, const huffllm_desc *const *descs, const void *const *blobs_dev,
                                         const uint16_t *const *xs_dev, uint32_t batch, float *const *ys_dev,
                                         void *const *workspaces_dev, size_t workspace_bytes_each, int32_t *err_flag_dev,
                                         huffllm_stream stream);

/*
 * The same product called with HOST activations and a HOST result: copies x to `x_stage_dev`
 * (device, batch*cols words), runs huffllm_decode_gemm, copies y from `y_stage_dev` (device,
 * batch*rows floats) to y_host and waits for the stream.  x_host / y_host should be pinned.
 */
huffllm_status huffllm_decode_gemm_host(const huffllm_desc *desc, const void *blob_dev, const uint16_t *x_host,
                                        uint32_t batch, float *y_host, uint16_t *x_stage_dev, float *y_stage_dev,
                                        void *workspace_dev, size_t workspace_bytes, int32_t *err_flag_dev,
                                        huffllm_stream stream);

/*
 * huffllm_decode_gemm_multi with HOST activations and HOST results: copies every x_i to its staging
 * buffer, runs the one launch, copies every y_i back and waits for the stream once.
 */
huffllm_status huffllm_decode_gemm_multi_host(uint32_t n, const huffllm_desc *const *descs, const void *const *blobs_dev,
                                              const uint16_t *const *xs_host, uint32_t batch, float *const *ys_host,
                                              uint16_t *const *x_stages_dev, float *const *y_stages_dev,
                                              void *const *workspaces_dev, size_t workspace_bytes_each,
                                              int32_t *err_flag_dev, huffllm_stream stream);

/*
 * The same without the wait: copies, launch and copies back are only enqueued on `stream`; the caller waits for the
 * stream before it reads ys_host.  Lets the launches of one decoder layer follow each other without a host round trip.
 */
huffllm_status huffllm_decode_gemm_multi_host_async(uint32_t n, const huffllm_desc *const *descs, const void *const *blobs_dev,
                                                    const uint16_t *const *xs_host, uint32_t batch, float *const *ys_host,
                                                    uint16_t *const *x_stages_dev, float *const *y_stages_dev,
                                                    void *const *workspaces_dev, size_t workspace_bytes_each,
                                                    int32_t *err_flag_dev, huffllm_stream stream);

/*
 * (No counterpart in the paper: an engineering addition for callers that cannot allocate.)
 *
 * huffllm_decode_gemm for callers that have no device scratch buffer to hand over and no way to get
 * one: code that runs inside a host application which has already claimed all of the GPU's memory
 * for its own pools (a serving engine that reserved HBM for its KV cache, a plug-in that must not
 * call cudaMalloc), or a latency-critical loop where an allocation, which synchronises the whole
 * device, is not acceptable.  The call allocates nothing: its scratch is a fixed array inside the
 * library's device image, HUFFLLM_STATIC_SCRATCH_BYTES long, which every GPU that loads the library
 * holds until the process exits.
 *
 * Inputs and outputs are the caller's, exactly as in huffllm_decode_gemm; batch may be at most
 * HUFFLLM_STATIC_MAX_BATCH, and huffllm_workspace_bytes(desc, batch) at most HUFFLLM_STATIC_SCRATCH_BYTES
 * (true for any matrix of up to about half a million rows) — anything larger is refused with
 * HUFFLLM_ERR_BUFFER_TOO_SMALL.  A call that is refused, for this or any other reason, enqueues nothing and
 * leaves the array untouched.  The first call on each device looks up the array's device address (with that device
 * current) and remembers it; make that first call outside any stream capture.  Every call clears
 * the scratch's control words on `stream` before the kernel runs, so a call never depends on what an
 * earlier call left behind.  All calls on one GPU share the one array: two calls that can overlap on
 * the GPU (different streams without an ordering between them) race on it and give wrong sums.
 */
#define HUFFLLM_STATIC_MAX_BATCH 8u
#define HUFFLLM_STATIC_SCRATCH_BYTES (1u << 20)
huffllm_status huffllm_decode_gemm_static(const huffllm_desc *desc, const void *blob_dev, const uint16_t *x_dev,
                                          uint32_t batch, float *y_dev, int32_t *err_flag_dev, huffllm_stream stream);

/*
 * Reference point for the compressed path: y = W x for an UNCOMPRESSED bf16 matrix (device,
 * row-major, 16-byte aligned rows, cols a multiple of 8), same fp32 accumulation, written as a
 * streaming kernel (many independent 16-byte loads in flight per lane).  This is the dense product
 * whose memory traffic the compression removes (Section 6: compression pays while weight movement
 * binds).  huffllm_plain_gemv_multi runs up to 8 such products (host arrays of n pointers / sizes)
 * in one launch, so that the dense layer can be timed in the same launch groups as the compressed one.
 */
huffllm_status huffllm_plain_gemv(const uint16_t *w_dev, uint64_t rows, uint64_t cols, const uint16_t *x_dev,
                                  float *y_dev, huffllm_stream stream);
huffllm_status huffllm_plain_gemv_multi(uint32_t n, const uint16_t *const *ws_dev, const uint64_t *rows, const uint64_t *cols,
                                        const uint16_t *const *xs_dev, float *const *ys_dev, huffllm_stream stream);

/*
 * Bit-field split explorer (Section 3.1, entropy table): what would it cost, in bits per parameter, to cut the
 * 16-bit weights into fields some other way and code each field on its own?
 *
 * A split is a list of field widths from the most significant bit down: {1,5,5,5} = sign, exponent, upper and lower
 * mantissa half of an FP16 number; {8,8}; {4,4,4,4}; {16} (the whole word as one symbol).  1 <= n_fields <=
 * HUFFLLM_MAX_FIELDS, every width 1..16, the widths add up to 16.
 *
 * huffllm_split_counts_size: number of counters of a split = sum over the fields of 2^width.
 * huffllm_split_histogram: one streaming pass (two for a 16-bit field) over n_weights 16-bit words in DEVICE memory
 *   (16-byte aligned) that counts, per field, how often each value occurs.  counts_dev (device, 8-byte aligned,
 *   huffllm_split_counts_size entries) is overwritten: field 0's 2^width counters first, then field 1's, ...
 *   Asynchronous on `stream`; no allocation; at most 2^38 weights per call.
 * huffllm_split_entropy (host only): from such counters (HOST memory) the Shannon entropy of each field in bits per
 *   parameter (entropy_bits[n_fields]); their sum is the split's "Total Bits/Param" of the table.  If huffman_bits
 *   is not NULL it receives, per field, the average codeword length of an unrestricted Huffman code for the counts
 *   (a field with a single value in use costs 1 bit, as in the blob format).
 */
#define HUFFLLM_MAX_FIELDS 16
huffllm_status huffllm_split_counts_size(const uint8_t *widths, uint32_t n_fields, size_t *n_counts);
huffllm_status huffllm_split_histogram(const uint16_t *w_dev, uint64_t n_weights, const uint8_t *widths, uint32_t n_fields,
                                       uint64_t *counts_dev, huffllm_stream stream);
huffllm_status huffllm_split_entropy(const uint64_t *counts_host, const uint8_t *widths, uint32_t n_fields,
                                     double *entropy_bits, double *huffman_bits);

/*
 * Copy `bytes` (a multiple of 16; both pointers 16-byte aligned) between two buffers the device can address —
 * device memory, or pinned host memory (cudaHostAlloc / cudaHostRegister: with unified addressing the device reaches
 * it through the same pointer) — with a small kernel on `stream`.  Meant for the activations and results of a decode
 * step (tens of kilobytes per token, Section 1: end-to-end latency): between kernels, and above all inside a CUDA graph,
 * a kernel copy costs a few microseconds where a DMA copy costs about ten.  The product calls also accept such pinned host
 * memory as their y, in which case the results are written to the host by the kernels themselves (x should be
 * staged into device memory: every CTA reads it).  Asynchronous; wait for the stream before reading a host destination.
 */
huffllm_status huffllm_stage_copy(void *dst, const void *src, size_t bytes, huffllm_stream stream);

/* Message of the last failing call on this thread ("" if none). */
const char *huffllm_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* HUFFLLM_H */
