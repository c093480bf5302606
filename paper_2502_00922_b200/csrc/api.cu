// C-ABI entry points that run on the device: argument checks, launch geometry, launches.
// No allocation and no synchronisation here (huffllm_decode_gemm_host, which exists to be timed
// end to end with host buffers, is the one call that waits for its stream).
#include <cuda_runtime.h>
#include <atomic>
#include <cstdlib>
#include <cstring>

#include "internal.h"
#include "kernels.h"

using namespace huffllm;

namespace {

constexpr uint32_t kMaxGrid = 512;        // CTAs the scratch layout provides for
constexpr uint32_t kKernelBatch = 8;      // activation vectors one launch multiplies
constexpr uint32_t kStaticSmem = 2048;    // barriers and tables the kernel declares statically (rounded up)

// Per-device facts, looked up once.  Threads may race to fill an entry: they write the same values, and `known` is
// published last.
struct DeviceSlot {
    std::atomic<bool> known{false};
    std::atomic<int> sms{0}, smem_optin{0};
};
DeviceSlot g_dev[64];
struct DeviceInfo {
    int sms = 0, smem_optin = 0;
};

huffllm_status device_info(DeviceInfo *out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= 64) return fail(HUFFLLM_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
    DeviceSlot &d = g_dev[dev];
    if (!d.known.load(std::memory_order_acquire)) {
        int sms = 0, smem = 0;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess)
            return fail(HUFFLLM_ERR_CUDA, "cudaDeviceGetAttribute: %s", cudaGetErrorString(e));
        d.sms.store(sms, std::memory_order_relaxed);
        d.smem_optin.store(smem, std::memory_order_relaxed);
        d.known.store(true, std::memory_order_release);
    }
    out->sms = d.sms.load(std::memory_order_relaxed);
    out->smem_optin = d.smem_optin.load(std::memory_order_relaxed);
    return HUFFLLM_OK;
}

// Scratch layout of one matrix's workspace:
//   [0, 4096)            arrival counters of the register-path kernel (one per CTA)
//   [4096, partial_off)  arrival counters of the tensor-core kernel, sized for its smallest tile
//   [partial_off, ...)   partial sums: of the register path's CTAs, or of the tensor-core path's work items
// Everything in front of partial_off is zero between calls; what lies behind it is overwritten freely by either path.
size_t ws_ctrl_bytes(const huffllm_desc *) { return 4096; }
size_t ws_partial_offset(const huffllm_desc *d) {
    const size_t max_m_tiles = (d->row_groups + 7) / 8;      // tensor-core row tiles at their smallest (128 rows)
    return ws_ctrl_bytes(d) + (max_m_tiles * 32 * 4 + 255) / 256 * 256;
}
// Partial sums of the register path: [kMaxGrid * 2][16 * b] CTA pieces, and, with two tiles of activations (batch
// 9..16), [kMaxGrid][2 * 32][16 * b] pieces that the warps of one CTA exchange (shared memory has no room for them).
constexpr uint32_t kTwoTileBatch = 16;    // most activation vectors of the register path with two tiles
bool two_tile_blob(const huffllm_desc *d) { return d->dtype == HUFFLLM_BF16 && d->lut_bits == 8; }
// blobs the tensor-core kernel takes: tables of up to 9 bits (FP16: field codes of up to 8 bits)
bool tc_blob(const huffllm_desc *d) { return d->dtype == HUFFLLM_FP16 ? d->lut_bits == 8u : d->lut_bits <= 9u; }
size_t ws_cta_pieces_bytes(uint32_t b) { return (size_t)kMaxGrid * 2 * 16 * b * sizeof(float); }
// (a workspace sized for `batch` vectors serves every smaller batch too)
size_t ws_bytes_for(const huffllm_desc *d, uint32_t batch) {
    size_t need = ws_cta_pieces_bytes(batch < kKernelBatch ? batch : kKernelBatch);
    if (batch > kKernelBatch && two_tile_blob(d)) {
        const uint32_t b = batch < kTwoTileBatch ? batch : kTwoTileBatch;
        need = ws_cta_pieces_bytes(b) + (size_t)kMaxGrid * 2 * 32 * 16 * b * sizeof(float);
    }
    return ws_partial_offset(d) + need;
}

// What a blob asks of a decoder CTA's shared memory.
struct SmemNeeds {
    uint32_t table_align, table_bytes;   // window of the decode table(s)
    uint32_t slot_bytes;                 // one slot: the W rows of the largest record
    uint32_t checks_per_block;           // refill checks per bit sequence and block of 32 columns
    uint32_t guard_bytes;                // readable bytes kept behind the last slot
};
SmemNeeds smem_needs(const huffllm_desc *desc) {
    SmemNeeds n;
    const bool fmt = desc->dtype == HUFFLLM_FP16;
    // BF16 tables of up to 9 bits are replicated per lane; longer ones are looked up in two levels: a per-lane table of the
    // first 8 bits, then one copy of the whole table behind it
    // (FP16: three sixteen-fold tables of 8 bits; fields of 9 bits and more take the second level too)
    const bool two_level = desc->lut_bits > (fmt ? 8u : 9u);
    // (FP16 blobs whose mantissa codes are flat need the exponent's table only; a launch over several matrices of which
    // some are not marked takes all three, see fp16_table_bytes)
    n.table_align = fmt ? 16384u : 128u << (two_level ? 8u : desc->lut_bits);
    const bool flat = fmt && desc->lut_bits == 8 && (desc->flat_fields & 6u) == 6u;
    n.table_bytes = fmt ? (flat ? 16384u : 49152u) + (two_level ? 3u * (4u << desc->lut_bits) : 0u)
                        : (two_level ? (128u << 8) + (4u << desc->lut_bits) : 128u << desc->lut_bits);
    // a slot holds the W rows of a record; the window runs one row ahead of what it consumes, and that look-ahead
    // past the last row lands in the next slot, the table or the guard area and is never used
    n.slot_bytes = desc->max_words * 256;
    // A stream can move its read pointer by one row per refill check and no further, whatever its bits and whatever the
    // table says: a sequence opens on rows 0 and 1, and every check loads at most the next row.  The furthest row a
    // chunk's decoder can touch is therefore 1 + checks, counted from the slot's first row, and the bytes kept readable
    // behind the last slot cover that for a slot of any size.
    n.checks_per_block = fmt ? (two_level ? 24 : 8) : (desc->lut_bits == 8 ? 3 : 4);
    n.guard_bytes = 256 * (3 + n.checks_per_block * (desc->chunk_cols / kBlockCols));
    return n;
}

// How many decoder warps get their slots: the kernels' own shared-memory plan (plan_smem in decode_common.cuh) worked out
// on the host.  Slots lie in front of and behind the decode table, which sits on a boundary of `lut_align` bytes, so up to a
// slot pair's bytes are lost on either side; where the dynamic window starts depends on the kernel's static shared memory,
// which the host does not know exactly: the smallest count over every 128-byte start within kStaticSmem + 1 KB is taken.
uint32_t planned_warps(uint32_t lut_align, uint32_t lut_size, uint64_t pair_bytes, uint32_t dyn_smem, uint32_t part_bytes,
                       uint32_t guard_bytes) {
    const uint64_t guard_extra = guard_bytes > part_bytes ? guard_bytes - part_bytes : 0;
    uint64_t least = ~0ull;
    for (uint64_t base = 0; base <= kStaticSmem + 1024; base += 128) {
        const uint64_t lut = (base + lut_align - 1) / lut_align * lut_align;
        const uint64_t n_a = lut > base ? (lut - base) / pair_bytes : 0;
        const uint64_t slot_b = lut + lut_size, end = base + dyn_smem - part_bytes;
        const uint64_t n_b = end > slot_b + guard_extra ? (end - slot_b - guard_extra) / pair_bytes : 0;
        if (n_a + n_b < least) least = n_a + n_b;
    }
    return (uint32_t)(least > 64 ? 64 : least);
}

// Geometry of the tensor-core small-batch path (batch 9..64): row tiles of 512 rows, column chunks cut into
// `ksplit` ranges so that the work items fill the GPU's SMs in whole waves as well as they can.
struct TcPlan {
    uint32_t npad, tiles, m_tiles, ksplit, items;
    size_t ticket_off, partial_off, bytes;
};
// Shared memory the tensor-core kernel needs with `tiles` 128-row tiles per CTA.
// Stages of the tensor-core kernel: four, two at the widest batch padding, where shared memory is short.
uint32_t tc_stages(uint32_t npad) { return npad == 64 ? 2u : 3u; }
// (`flat`: every matrix of the launch has flat FP16 mantissa codes: the exponent's table alone is kept)
bool flat_fp16(const huffllm_desc *d) { return d->dtype == HUFFLLM_FP16 && d->lut_bits == 8 && (d->flat_fields & 6u) == 6u; }
// Do the slot pairs of `tiles` tiles' decoder warps fit beside the tables and the stages of activations?
bool tc_fits(const huffllm_desc *d, uint32_t npad, uint32_t tiles, bool flat, uint32_t dyn_smem) {
    SmemNeeds n = smem_needs(d);
    if (d->dtype == HUFFLLM_FP16 && d->lut_bits == 8) n.table_bytes = flat ? 16384u : 49152u;   // (a launch-wide choice)
    const uint32_t b_stages = tc_stages(npad) * npad * 128;          // the guard area may lie over them
    const uint32_t n_dec = 8 * tiles < 31 ? 8 * tiles : 31;
    return planned_warps(n.table_align, n.table_bytes, 2ull * n.slot_bytes, dyn_smem, b_stages, n.guard_bytes) >= n_dec;
}
// `sms`: the CTAs this matrix can have (all SMs, or its share of a launch over several matrices); `tiles_cap`: the tiles
// the launch's other matrices leave room for; `max_bytes`: the workspace at hand (column ranges whose pieces would not
// fit are not considered: a share of the SMs can favour more ranges than the whole GPU, for which workspaces are sized).
TcPlan tc_plan(const huffllm_desc *d, uint32_t batch, uint32_t sms, uint32_t dyn_smem, bool flat, uint32_t tiles_cap = 4,
               size_t max_bytes = ~(size_t)0) {
    TcPlan p;
    p.npad = batch <= 16 ? 16 : (batch <= 32 ? 32 : 64);
    p.tiles = tiles_cap;                            // as many 8-warp tiles as the chunk slots leave room for
    while (p.tiles > 1 && !tc_fits(d, p.npad, p.tiles, flat, dyn_smem)) --p.tiles;
    const uint32_t n_dec = 8 * p.tiles < 31 ? 8 * p.tiles : 31;      // the CTA's last warp issues the MMAs and never decodes
    p.m_tiles = (d->row_groups + n_dec - 1) / n_dec;
    // Column ranges: the one with the shortest finish time.  A CTA takes items b, b + grid, ... in turn; an item costs its
    // blocks of 32 columns (ranges of one matrix differ by a chunk when ksplit does not divide the chunk count) plus a start
    // and an epilogue worth a few blocks.  Counting whole waves alone would pick many short, unequal ranges.
    // (measured on the 70B-FFN shapes at 64 vectors: a block of 32 columns takes 1.25 us of an item, the item's start and
    // epilogue together 5 to 8 us)
    constexpr uint64_t kItemBlocks = 5;
    uint32_t best = 1;
    uint64_t best_span = ~0ull;
    for (uint32_t ks = 1; ks <= 16 && ks <= d->col_chunks; ++ks) {
        const uint64_t items = (uint64_t)p.m_tiles * ks, grid = items < sms ? items : sms;
        if (ks > 1 && ws_partial_offset(d) + (size_t)items * 32 * (p.npad / 2) * 32 * sizeof(float) > max_bytes) break;
        uint64_t span = 0;
        for (uint64_t b = 0; b < grid; ++b) {
            uint64_t t = 0;
            for (uint64_t it = b; it < items; it += grid) {
                const uint32_t r = (uint32_t)(it % ks);
                const uint32_t len = (uint32_t)((uint64_t)d->col_chunks * (r + 1) / ks) - (uint32_t)((uint64_t)d->col_chunks * r / ks);
                t += (uint64_t)len * (d->chunk_cols / kBlockCols) + kItemBlocks;
            }
            if (t > span) span = t;
        }
        if (span < best_span) { best_span = span; best = ks; }
    }
    p.ksplit = best;
    p.items = p.m_tiles * best;
    // the counters' region is sized for the smallest tile (most row tiles), so that plans for different batch sizes
    // sharing one workspace never put partial sums where another plan keeps counters
    p.ticket_off = ws_ctrl_bytes(d);
    p.partial_off = ws_partial_offset(d);
    p.bytes = p.partial_off + (best > 1 ? (size_t)p.items * 32 * (p.npad / 2) * 32 * sizeof(float) : 0);
    return p;
}

// Bytes of the FP16 tables a launch keeps in shared memory: three sixteen-fold tables of 8-bit codes, or the exponent's
// alone where every matrix of the launch has flat mantissa codes (those are read without tables).
uint32_t fp16_table_bytes(const KernelArgs *k) { return k->lut_bits == 8 && k->fp16_flat ? 16384u : 49152u; }

// Start a launch description.
void begin_args(KernelArgs *k, uint32_t batch, const DeviceInfo &dev) {
    memset(k, 0, sizeof(*k));
    k->batch = batch;
    k->dyn_smem_bytes = (uint32_t)dev.smem_optin - kStaticSmem;
}

// Append one matrix to a launch description (checks the descriptor and the blob pointer).
huffllm_status add_matrix(KernelArgs *k, const huffllm_desc *desc, const void *blob) {
    huffllm_status st = check_desc(desc);
    if (st != HUFFLLM_OK) return st;
    if (!blob || ((uintptr_t)blob & 255)) return fail(HUFFLLM_ERR_INVALID_ARG, "blob must be a 256-byte aligned device pointer");
    const uint32_t fmt = desc->dtype == HUFFLLM_FP16 ? 1u : 0u;

    if (k->n_mats && k->fmt != fmt) return fail(HUFFLLM_ERR_UNSUPPORTED, "matrices of one call must share the dtype");
    k->fmt = fmt;
    if (k->n_mats == kMaxMats) return fail(HUFFLLM_ERR_UNSUPPORTED, "at most %u matrices per call", kMaxMats);
    if (k->n_mats && k->lut_bits != desc->lut_bits)
        return fail(HUFFLLM_ERR_UNSUPPORTED, "matrices of one call must share max_code_len");
    if (desc->n_chunks + k->total_chunks >= (1ull << 31)) return fail(HUFFLLM_ERR_UNSUPPORTED, "too many chunks for one launch");
    MatArgs &m = k->m[k->n_mats++];
    m.blob = (const uint8_t *)blob;
    m.off_lut = desc->off_lut;
    m.off_index = desc->off_index;
    m.off_payload = desc->off_payload;
    m.payload_units = (uint32_t)(desc->payload_bytes / kRecordUnit);
    m.rows = desc->rows;
    m.cols = desc->cols;
    m.n_chunks = (uint32_t)desc->n_chunks;
    m.chunk_cols = desc->chunk_cols;
    m.col_chunks = desc->col_chunks;
    k->total_chunks += m.n_chunks;
    k->lut_bits = desc->lut_bits;
    // (flat mantissa codes: only if every matrix of the launch has them)
    const uint32_t flat = fmt && (desc->flat_fields & 6u) == 6u ? 1u : 0u;
    k->fp16_flat = k->n_mats == 1 ? flat : (k->fp16_flat & flat);
    const SmemNeeds need = smem_needs(desc);
    k->lut_align = need.table_align;
    k->lut_size = need.table_bytes;
    if (need.slot_bytes > k->slot_bytes) k->slot_bytes = need.slot_bytes;
    if (need.guard_bytes > k->guard_bytes) k->guard_bytes = need.guard_bytes;
    return HUFFLLM_OK;
}

// Close a launch description: shared-memory budget and grid size.
huffllm_status finish_args(KernelArgs *k, bool product, const DeviceInfo &dev, uint32_t *grid, uint32_t *warps_at_least = nullptr) {
    // (pieces that warps of a CTA exchange: in shared memory up to 8 vectors, in the workspace above)
    k->part_bytes = product && k->batch <= kKernelBatch ? 2 * 32 * 16 * k->batch * (uint32_t)sizeof(float) : 0;
    if (k->fmt && k->lut_bits <= 8) k->lut_size = fp16_table_bytes(k);
    // Two slots per decoder warp, so that a warp's next record lands while it decodes this one.  Where records are so large
    // that this would leave fewer than 31 warps a slot pair, and single slots serve at least a quarter more warps, every
    // warp gets one slot: more decoders at work outweigh the wait for a copy at every chunk start.
    const uint64_t max_w = 31;                                       // decoder warps of a CTA of 1024 threads
    uint64_t w2 = planned_warps(k->lut_align, k->lut_size, 2ull * k->slot_bytes, k->dyn_smem_bytes, k->part_bytes, k->guard_bytes);
    uint64_t w1 = planned_warps(k->lut_align, k->lut_size, k->slot_bytes, k->dyn_smem_bytes, k->part_bytes, k->guard_bytes);
    if (w2 > max_w) w2 = max_w;
    if (w1 > max_w) w1 = max_w;
    const bool single_ok = k->fmt || k->lut_bits == 8;                // (the kernels that exist with single slots)
    k->slots = single_ok && w2 < max_w && 4 * w1 >= 5 * w2 ? 1u : 2u;
    if ((k->slots == 2 ? w2 : w1) == 0)
        return fail(HUFFLLM_ERR_UNSUPPORTED, "chunk records too large for shared memory (slot %u bytes)", k->slot_bytes);
    if (warps_at_least) *warps_at_least = (uint32_t)(k->slots == 1 ? w1 : w2);
    k->pair_recip = (uint32_t)(0x100000000ull / ((uint64_t)k->slots * k->slot_bytes));
    uint64_t g = k->total_chunks < (uint64_t)dev.sms ? k->total_chunks : (uint64_t)dev.sms;
    *grid = (uint32_t)(g < kMaxGrid ? g : kMaxGrid);
    // deal the CTAs out to the matrices: one each, then always to the matrix with the most chunks per CTA, so that
    // the largest piece is as small as it can be and no CTA works in two matrices
    if (*grid < k->n_mats) return fail(HUFFLLM_ERR_UNSUPPORTED, "more matrices than SMs");
    uint32_t cnt[kMaxMats];
    for (uint32_t i = 0; i < k->n_mats; ++i) cnt[i] = 1;
    for (uint32_t left = *grid - k->n_mats; left; --left) {
        uint32_t best = k->n_mats;
        for (uint32_t i = 0; i < k->n_mats; ++i) {
            if (cnt[i] >= k->m[i].n_chunks) continue;
            if (best == k->n_mats || (uint64_t)k->m[i].n_chunks * cnt[best] > (uint64_t)k->m[best].n_chunks * cnt[i]) best = i;
        }
        if (best == k->n_mats) break;
        ++cnt[best];
    }
    uint32_t first = 0;
    for (uint32_t i = 0; i < k->n_mats; ++i) {
        k->m[i].cta_first = first;
        k->m[i].cta_count = cnt[i];
        k->m[i].cta_chunks = k->m[i].n_chunks / cnt[i];
        k->m[i].cta_extra = k->m[i].n_chunks % cnt[i];
        first += cnt[i];
    }
    *grid = first;
    return HUFFLLM_OK;
}

}  // namespace

extern "C" {

huffllm_status huffllm_workspace_bytes(const huffllm_desc *desc, uint32_t batch, size_t *bytes) {
    clear_error();
    if (!bytes) return fail(HUFFLLM_ERR_INVALID_ARG, "bytes is null");
    huffllm_status st = check_desc(desc);
    if (st != HUFFLLM_OK) return st;
    if (batch == 0 || batch > 64) return fail(HUFFLLM_ERR_INVALID_ARG, "batch must be in [1, 64]");
    *bytes = ws_bytes_for(desc, batch);     // (above 8 vectors: what passes of 8 need, should the tensor-core kernel not fit)
    if (batch > kKernelBatch) {      // the tensor-core path keeps partial tiles of its column ranges here
        DeviceInfo dev;       // without a device (a host-only caller sizing buffers): the B200's figures
        const bool have = device_info(&dev) == HUFFLLM_OK;
        clear_error();
        const int sms = have ? dev.sms : 148;
        const uint32_t dyn = (have ? (uint32_t)dev.smem_optin : 232448u) - kStaticSmem;
        size_t tc = tc_plan(desc, batch, (uint32_t)sms, dyn, false).bytes;     // (with all three FP16 tables: the larger plan)
        if (tc > *bytes) *bytes = tc;
    }
    return HUFFLLM_OK;
}

huffllm_status huffllm_workspace_control_bytes(const huffllm_desc *desc, size_t *bytes) {
    clear_error();
    if (!bytes) return fail(HUFFLLM_ERR_INVALID_ARG, "bytes is null");
    huffllm_status st = check_desc(desc);
    if (st != HUFFLLM_OK) return st;
    *bytes = ws_partial_offset(desc);
    return HUFFLLM_OK;
}

huffllm_status huffllm_decode_smem_plan(const huffllm_desc *desc, uint32_t *table_bytes, uint32_t *slot_bytes,
                                        uint32_t *refill_checks_per_block, uint32_t *guard_bytes) {
    clear_error();
    huffllm_status st = check_desc(desc);
    if (st != HUFFLLM_OK) return st;
    const SmemNeeds n = smem_needs(desc);
    if (table_bytes) *table_bytes = n.table_bytes;
    if (slot_bytes) *slot_bytes = n.slot_bytes;
    if (refill_checks_per_block) *refill_checks_per_block = n.checks_per_block;
    if (guard_bytes) *guard_bytes = n.guard_bytes;
    return HUFFLLM_OK;
}

huffllm_status huffllm_decode_launch_plan(const huffllm_desc *desc, uint32_t batch, uint32_t smem_bytes_per_cta,
                                          uint32_t *slots_per_warp, uint32_t *decoder_warps) {
    clear_error();
    huffllm_status st = check_desc(desc);
    if (st != HUFFLLM_OK) return st;
    if (batch > kKernelBatch) return fail(HUFFLLM_ERR_INVALID_ARG, "the plan is that of the register path: batch 0 (decode) to %u", kKernelBatch);
    DeviceInfo dev = {};
    dev.sms = 148;
    dev.smem_optin = smem_bytes_per_cta ? smem_bytes_per_cta : 232448;
    KernelArgs k;
    uint32_t grid = 0, warps = 0;
    begin_args(&k, batch ? batch : 1, dev);
    if ((st = add_matrix(&k, desc, (const void *)256)) != HUFFLLM_OK) return st;     // (the pointer is only checked for alignment)
    if ((st = finish_args(&k, batch != 0, dev, &grid, &warps)) != HUFFLLM_OK) return st;
    if (slots_per_warp) *slots_per_warp = k.slots;
    if (decoder_warps) *decoder_warps = warps;
    return HUFFLLM_OK;
}

huffllm_status huffllm_decode(const huffllm_desc *desc, const void *blob, uint16_t *out, int32_t *err_flag, huffllm_stream stream) {
    clear_error();
    DeviceInfo dev;
    huffllm_status st = device_info(&dev);
    if (st != HUFFLLM_OK) return st;
    if (!out || ((uintptr_t)out & 15)) return fail(HUFFLLM_ERR_INVALID_ARG, "out must be a 16-byte aligned device pointer");
    KernelArgs k;
    uint32_t grid;
    begin_args(&k, 1, dev);
    if ((st = add_matrix(&k, desc, blob)) != HUFFLLM_OK) return st;
    if ((st = finish_args(&k, false, dev, &grid)) != HUFFLLM_OK) return st;
    k.m[0].out = out;
    k.err = err_flag;
    cudaError_t e = launch_decode(k, grid, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "decode launch: %s", cudaGetErrorString(e));
    return HUFFLLM_OK;
}

// Checks shared by the product entry points for one matrix of a call.
static huffllm_status check_product_args(const huffllm_desc *desc, const uint16_t *x, const float *y, const void *workspace,
                                         size_t workspace_bytes, uint32_t batch) {
    if (!x || !y || !workspace) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer");
    if (((uintptr_t)x & 15) || ((uintptr_t)y & 3) || ((uintptr_t)workspace & 255))
        return fail(HUFFLLM_ERR_INVALID_ARG, "x must be 16-byte, y 4-byte, workspace 256-byte aligned");
    huffllm_status st = check_desc(desc);
    if (st != HUFFLLM_OK) return st;
    if (workspace_bytes < ws_bytes_for(desc, batch)) return fail(HUFFLLM_ERR_BUFFER_TOO_SMALL, "workspace too small");
    if (desc->cols % kBlockCols) return fail(HUFFLLM_ERR_UNSUPPORTED, "fused products need cols to be a multiple of 32");
    return HUFFLLM_OK;
}

huffllm_status huffllm_decode_gemm_multi(uint32_t n, const huffllm_desc *const *descs, const void *const *blobs,
                                         const uint16_t *const *xs, uint32_t batch, float *const *ys, void *const *workspaces,
                                         size_t workspace_bytes_each, int32_t *err_flag, huffllm_stream stream) {
    clear_error();
    DeviceInfo dev;
    huffllm_status st = device_info(&dev);
    if (st != HUFFLLM_OK) return st;
    if (!descs || !blobs || !xs || !ys || !workspaces) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer");
    if (n == 0 || n > kMaxMats) return fail(HUFFLLM_ERR_INVALID_ARG, "between 1 and %u matrices per call", kMaxMats);
    if (batch == 0 || batch > 64) return fail(HUFFLLM_ERR_INVALID_ARG, "batch must be in [1, 64]");
    if (batch > kTwoTileBatch) {
        // 17..64 vectors: the tensor-core kernel, its CTAs dealt to the matrices like the other kernels'
        TcArgs t;
        memset(&t, 0, sizeof(t));
        KernelArgs &k = t.k;
        uint32_t grid;
        begin_args(&k, batch, dev);
        for (uint32_t i = 0; i < n; ++i) {
            if ((st = check_product_args(descs[i], xs[i], ys[i], workspaces[i], workspace_bytes_each, batch)) != HUFFLLM_OK) return st;
            if (!tc_blob(descs[i]))
                return fail(HUFFLLM_ERR_UNSUPPORTED, "more than %u vectors per call over several matrices take tables of up to 9 bits (FP16: 8)", kTwoTileBatch);
            for (uint32_t j = 0; j < i; ++j)
                if (workspaces[j] == workspaces[i]) return fail(HUFFLLM_ERR_INVALID_ARG, "matrices %u and %u share a workspace", j, i);
            if ((st = add_matrix(&k, descs[i], blobs[i])) != HUFFLLM_OK) return st;
            k.m[i].x = xs[i];
            k.m[i].y = ys[i];
        }
        if ((st = finish_args(&k, true, dev, &grid)) != HUFFLLM_OK) return st;      // (deals the CTAs to the matrices by their chunks)
        const uint32_t npad = batch <= 32 ? 32 : 64;
        uint32_t tiles = 4;                             // what the matrix with the largest records leaves room for
        for (uint32_t i = 0; i < n; ++i) {
            const TcPlan tp = tc_plan(descs[i], batch, (uint32_t)dev.sms, k.dyn_smem_bytes, k.fp16_flat != 0);
            if (!tc_fits(descs[i], tp.npad, tp.tiles, k.fp16_flat != 0, k.dyn_smem_bytes))
                return fail(HUFFLLM_ERR_UNSUPPORTED, "chunk records of matrix %u too large for the tensor-core kernel's slots", i);
            if (tp.tiles < tiles) tiles = tp.tiles;
        }
        k.part_bytes = tc_stages(npad) * npad * 128;
        k.slots = 2;
        k.pair_recip = (uint32_t)(0x100000000ull / (2ull * k.slot_bytes));
        k.tc_npad = npad;
        k.tc_tiles = tiles;
        uint32_t first = 0;
        for (uint32_t i = 0; i < n; ++i) {
            const TcPlan tp = tc_plan(descs[i], batch, k.m[i].cta_count, k.dyn_smem_bytes, k.fp16_flat != 0, tiles, workspace_bytes_each);
            if (workspace_bytes_each < tp.bytes) return fail(HUFFLLM_ERR_BUFFER_TOO_SMALL, "workspace of matrix %u too small for batch %u", i, batch);
            t.m_tiles[i] = tp.m_tiles;
            t.ksplit[i] = tp.ksplit;
            t.ticket[i] = (unsigned int *)((uint8_t *)workspaces[i] + tp.ticket_off);
            t.partial[i] = (float *)((uint8_t *)workspaces[i] + tp.partial_off);
            k.m[i].cta_first = first;
            if (tp.items < k.m[i].cta_count) k.m[i].cta_count = tp.items;
            first += k.m[i].cta_count;
        }
        k.err = err_flag;
        cudaError_t e = launch_gemm_tc(t, first, (cudaStream_t)stream);
        if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "tensor-core product launch: %s", cudaGetErrorString(e));
        return HUFFLLM_OK;
    }
    KernelArgs k;
    uint32_t grid;
    begin_args(&k, batch, dev);
    for (uint32_t i = 0; i < n; ++i) {
        if ((st = check_product_args(descs[i], xs[i], ys[i], workspaces[i], workspace_bytes_each, batch)) != HUFFLLM_OK) return st;
        if (batch > kKernelBatch && !two_tile_blob(descs[i]))
            return fail(HUFFLLM_ERR_UNSUPPORTED, "more than %u vectors per call take BF16 blobs of max_code_len 8", kKernelBatch);
        for (uint32_t j = 0; j < i; ++j)
            if (workspaces[j] == workspaces[i]) return fail(HUFFLLM_ERR_INVALID_ARG, "matrices %u and %u share a workspace", j, i);
        if ((st = add_matrix(&k, descs[i], blobs[i])) != HUFFLLM_OK) return st;
        MatArgs &m = k.m[i];
        m.x = xs[i];
        m.y = ys[i];
        m.ws_ticket = (unsigned int *)workspaces[i];
        m.ws_partial = (float *)((uint8_t *)workspaces[i] + ws_partial_offset(descs[i]));
        m.ws_warp_pieces = (float *)((uint8_t *)workspaces[i] + ws_partial_offset(descs[i]) + ws_cta_pieces_bytes(batch));   // (used above 8 vectors)
    }
    if ((st = finish_args(&k, true, dev, &grid)) != HUFFLLM_OK) return st;
    k.err = err_flag;
    cudaError_t e = launch_gemm(k, grid, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "product launch: %s", cudaGetErrorString(e));
    return HUFFLLM_OK;
}

huffllm_status huffllm_decode_gemm(const huffllm_desc *desc, const void *blob, const uint16_t *x, uint32_t batch, float *y,
                                   void *workspace, size_t workspace_bytes, int32_t *err_flag, huffllm_stream stream) {
    clear_error();
    DeviceInfo dev;
    huffllm_status st = device_info(&dev);
    if (st != HUFFLLM_OK) return st;
    if (batch == 0 || batch > 64) return fail(HUFFLLM_ERR_INVALID_ARG, "batch must be in [1, 64]");
    if ((st = check_product_args(desc, x, y, workspace, workspace_bytes, batch)) != HUFFLLM_OK) return st;
    // Paths for more than 8 vectors.  Each returns HUFFLLM_OK with `done` set if it launched, HUFFLLM_OK without if it does
    // not apply here (the next path decides), or an error.
    bool done = false;
    auto two_tiles = [&]() -> huffllm_status {
        // 9..16 vectors on the default BF16 blobs: the register path with two tiles of activations per decoded block
        if (batch > kTwoTileBatch || !two_tile_blob(desc)) return HUFFLLM_OK;
        KernelArgs k;
        uint32_t grid;
        begin_args(&k, batch, dev);
        huffllm_status s2 = add_matrix(&k, desc, blob);
        if (s2 != HUFFLLM_OK) return s2;
        if (finish_args(&k, true, dev, &grid) != HUFFLLM_OK) {
            clear_error();      // records too large for shared memory: another path decides
            return HUFFLLM_OK;
        }
        k.m[0].x = x;
        k.m[0].y = y;
        k.m[0].ws_ticket = (unsigned int *)workspace;
        k.m[0].ws_partial = (float *)((uint8_t *)workspace + ws_partial_offset(desc));
        k.m[0].ws_warp_pieces = (float *)((uint8_t *)workspace + ws_partial_offset(desc) + ws_cta_pieces_bytes(batch));
        k.err = err_flag;
        cudaError_t e = launch_gemm(k, grid, (cudaStream_t)stream);
        if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "product launch: %s", cudaGetErrorString(e));
        done = true;
        return HUFFLLM_OK;
    };
    auto tensor_core = [&](bool other_path_left) -> huffllm_status {
        // one pass over the compressed weights for the whole batch (tables of up to 9 bits; longer codes take passes of 8
        // vectors through the register-path kernel and its two-level lookup)
        if (!tc_blob(desc)) return HUFFLLM_OK;
        // (column ranges are planned within the workspace at hand)
        const TcPlan tp = tc_plan(desc, batch, (uint32_t)dev.sms, (uint32_t)dev.smem_optin - kStaticSmem, flat_fp16(desc), 4, workspace_bytes);
        TcArgs t;
        memset(&t, 0, sizeof(t));
        KernelArgs &k = t.k;
        begin_args(&k, batch, dev);
        huffllm_status s2 = add_matrix(&k, desc, blob);
        if (s2 != HUFFLLM_OK) return s2;
        k.part_bytes = tc_stages(tp.npad) * tp.npad * 128;      // the stages of activations
        k.slots = 2;
        k.pair_recip = (uint32_t)(0x100000000ull / (2ull * k.slot_bytes));
        if (!tc_fits(desc, tp.npad, tp.tiles, flat_fp16(desc), k.dyn_smem_bytes)) return HUFFLLM_OK;   // records too large for this kernel's slots
        if (workspace_bytes < tp.bytes) {
            if (other_path_left) return HUFFLLM_OK;     // (the register path needs less)
            return fail(HUFFLLM_ERR_BUFFER_TOO_SMALL, "workspace too small for batch %u", batch);
        }
        k.m[0].x = x;
        k.m[0].y = y;
        k.tc_npad = tp.npad;
        k.tc_tiles = tp.tiles;
        t.m_tiles[0] = tp.m_tiles;
        t.ksplit[0] = tp.ksplit;
        t.ticket[0] = (unsigned int *)((uint8_t *)workspace + tp.ticket_off);
        t.partial[0] = (float *)((uint8_t *)workspace + tp.partial_off);
        k.err = err_flag;
        const uint32_t grid = tp.items < (uint32_t)dev.sms ? tp.items : (uint32_t)dev.sms;
        k.m[0].cta_first = 0;
        k.m[0].cta_count = grid;
        cudaError_t e = launch_gemm_tc(t, grid, (cudaStream_t)stream);
        if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "tensor-core product launch: %s", cudaGetErrorString(e));
        done = true;
        return HUFFLLM_OK;
    };
    if (batch > kKernelBatch) {
        // 9..16 vectors: the tensor-core kernel, whose time does not grow with the batch below its padding of 16, is the
        // faster one for matrices that are at least as wide as tall (few row groups per SM make the register path's
        // cross-CTA sums of 16-vector pieces expensive), unless they have so few rows that it gets few row tiles; measured
        // at 12 and 16 vectors on seven shapes from 1024 x 8192 to 28672 x 8192.  Above 16 vectors it is the only one.
        const bool wide = desc->cols >= desc->rows && desc->rows >= 2048;
        if (!wide && (st = two_tiles()) != HUFFLLM_OK) return st;
        if (!done && (st = tensor_core(wide && batch <= kTwoTileBatch && two_tile_blob(desc))) != HUFFLLM_OK) return st;
        if (!done && wide && (st = two_tiles()) != HUFFLLM_OK) return st;
        if (done) return HUFFLLM_OK;
        // neither applies (long codes, or chunk records too large for the slots): passes of 8 vectors
    }
    for (uint32_t b0 = 0; b0 < batch; b0 += kKernelBatch) {
        uint32_t nb = batch - b0 < kKernelBatch ? batch - b0 : kKernelBatch;
        KernelArgs k;
        uint32_t grid;
        begin_args(&k, nb, dev);
        if ((st = add_matrix(&k, desc, blob)) != HUFFLLM_OK) return st;
        if ((st = finish_args(&k, true, dev, &grid)) != HUFFLLM_OK) return st;
        k.m[0].x = x + (uint64_t)b0 * desc->cols;
        k.m[0].y = y + (uint64_t)b0 * desc->rows;
        k.m[0].ws_ticket = (unsigned int *)workspace;
        k.m[0].ws_partial = (float *)((uint8_t *)workspace + ws_partial_offset(desc));
        k.err = err_flag;
        cudaError_t e = launch_gemm(k, grid, (cudaStream_t)stream);
        if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "product launch: %s", cudaGetErrorString(e));
    }
    return HUFFLLM_OK;
}

huffllm_status huffllm_decode_gemv(const huffllm_desc *desc, const void *blob, const uint16_t *x, float *y, void *workspace,
                                   size_t workspace_bytes, int32_t *err_flag, huffllm_stream stream) {
    return huffllm_decode_gemm(desc, blob, x, 1, y, workspace, workspace_bytes, err_flag, stream);
}

huffllm_status huffllm_decode_gemm_multi_host_async(uint32_t n, const huffllm_desc *const *descs, const void *const *blobs,
                                                    const uint16_t *const *xs_host, uint32_t batch, float *const *ys_host,
                                                    uint16_t *const *x_stages, float *const *y_stages, void *const *workspaces,
                                                    size_t workspace_bytes_each, int32_t *err_flag, huffllm_stream stream) {
    clear_error();
    if (!descs || !xs_host || !ys_host || !x_stages || !y_stages) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer");
    if (n == 0 || n > kMaxMats) return fail(HUFFLLM_ERR_INVALID_ARG, "between 1 and %u matrices per call", kMaxMats);
    if (batch == 0 || batch > 64) return fail(HUFFLLM_ERR_INVALID_ARG, "batch must be in [1, 64]");
    cudaStream_t s = (cudaStream_t)stream;
    for (uint32_t i = 0; i < n; ++i) {     // nothing is enqueued before every argument has been looked at
        if (!descs[i] || !xs_host[i] || !ys_host[i] || !x_stages[i] || !y_stages[i]) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer");
        huffllm_status st = check_product_args(descs[i], x_stages[i], y_stages[i], workspaces ? workspaces[i] : nullptr,
                                               workspace_bytes_each, batch);
        if (st != HUFFLLM_OK) return st;
        if (!blobs || !blobs[i] || ((uintptr_t)blobs[i] & 255))
            return fail(HUFFLLM_ERR_INVALID_ARG, "blob must be a 256-byte aligned device pointer");
        if (batch > kKernelBatch && batch <= kTwoTileBatch && !two_tile_blob(descs[i]))
            return fail(HUFFLLM_ERR_UNSUPPORTED, "9 to %u vectors per call over several matrices take BF16 blobs of max_code_len 8", kTwoTileBatch);
        if (batch > kTwoTileBatch && !tc_blob(descs[i]))
            return fail(HUFFLLM_ERR_UNSUPPORTED, "more than %u vectors per call over several matrices take tables of up to 9 bits (FP16: 8)", kTwoTileBatch);
    }
    for (uint32_t i = 0; i < n; ++i) {
        cudaError_t e = cudaMemcpyAsync(x_stages[i], xs_host[i], (size_t)batch * descs[i]->cols * 2, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "copy of x: %s", cudaGetErrorString(e));
    }
    huffllm_status st = huffllm_decode_gemm_multi(n, descs, blobs, (const uint16_t *const *)x_stages, batch, y_stages, workspaces,
                                                  workspace_bytes_each, err_flag, stream);
    if (st != HUFFLLM_OK) return st;
    for (uint32_t i = 0; i < n; ++i) {
        cudaError_t e = cudaMemcpyAsync(ys_host[i], y_stages[i], (size_t)batch * descs[i]->rows * 4, cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "copy of y: %s", cudaGetErrorString(e));
    }
    return HUFFLLM_OK;
}

huffllm_status huffllm_decode_gemm_multi_host(uint32_t n, const huffllm_desc *const *descs, const void *const *blobs,
                                              const uint16_t *const *xs_host, uint32_t batch, float *const *ys_host,
                                              uint16_t *const *x_stages, float *const *y_stages, void *const *workspaces,
                                              size_t workspace_bytes_each, int32_t *err_flag, huffllm_stream stream) {
    huffllm_status st = huffllm_decode_gemm_multi_host_async(n, descs, blobs, xs_host, batch, ys_host, x_stages, y_stages, workspaces,
                                                             workspace_bytes_each, err_flag, stream);
    if (st != HUFFLLM_OK) return st;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "waiting for the stream: %s", cudaGetErrorString(e));
    return HUFFLLM_OK;
}

huffllm_status huffllm_decode_gemm_host(const huffllm_desc *desc, const void *blob, const uint16_t *x_host, uint32_t batch,
                                        float *y_host, uint16_t *x_stage, float *y_stage, void *workspace,
                                        size_t workspace_bytes, int32_t *err_flag, huffllm_stream stream) {
    clear_error();
    if (!desc || !x_host || !y_host || !x_stage || !y_stage) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer");
    if (batch == 0 || batch > 64) return fail(HUFFLLM_ERR_INVALID_ARG, "batch must be in [1, 64]");
    huffllm_status st0 = check_product_args(desc, x_stage, y_stage, workspace, workspace_bytes, batch);
    if (st0 != HUFFLLM_OK) return st0;       // nothing is enqueued for a call that will be refused
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyAsync(x_stage, x_host, (size_t)batch * desc->cols * 2, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "copy of x: %s", cudaGetErrorString(e));
    huffllm_status st = huffllm_decode_gemm(desc, blob, x_stage, batch, y_stage, workspace, workspace_bytes, err_flag, stream);
    if (st != HUFFLLM_OK) return st;
    e = cudaMemcpyAsync(y_host, y_stage, (size_t)batch * desc->rows * 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "copy of y: %s", cudaGetErrorString(e));
    return HUFFLLM_OK;
}

}  // extern "C"

// Scratch of huffllm_decode_gemm_static.  In host code this name is only a handle for the runtime, not a
// device address: the address the kernels get comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_static_scratch[HUFFLLM_STATIC_SCRATCH_BYTES];
static std::atomic<void *> g_static_scratch_addr[64];

extern "C" {

huffllm_status huffllm_decode_gemm_static(const huffllm_desc *desc, const void *blob, const uint16_t *x, uint32_t batch,
                                          float *y, int32_t *err_flag, huffllm_stream stream) {
    clear_error();
    if (batch == 0) return fail(HUFFLLM_ERR_INVALID_ARG, "batch must be at least 1");
    huffllm_status st = check_desc(desc);
    if (st != HUFFLLM_OK) return st;
    if (batch > HUFFLLM_STATIC_MAX_BATCH || ws_bytes_for(desc, batch) > sizeof(g_static_scratch))
        return fail(HUFFLLM_ERR_BUFFER_TOO_SMALL,
                    "this matrix with %u vectors needs %zu bytes of scratch; the built-in array has %u (and takes at most %u vectors)",
                    batch, ws_bytes_for(desc, batch), (unsigned)HUFFLLM_STATIC_SCRATCH_BYTES, (unsigned)HUFFLLM_STATIC_MAX_BATCH);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= 64) return fail(HUFFLLM_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
    void *ws = g_static_scratch_addr[dev].load(std::memory_order_acquire);
    if (!ws) {   // set-up, once per device, with that device current (racing threads look up the same address)
        e = cudaGetSymbolAddress(&ws, g_static_scratch);
        if (e != cudaSuccess || !ws) return fail(HUFFLLM_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        g_static_scratch_addr[dev].store(ws, std::memory_order_release);
    }
    // Everything that can refuse the call is checked before anything is enqueued: a refused call leaves the array alone.
    DeviceInfo info;
    if ((st = device_info(&info)) != HUFFLLM_OK) return st;
    if ((st = check_product_args(desc, x, y, ws, sizeof(g_static_scratch), batch)) != HUFFLLM_OK) return st;
    {
        KernelArgs k;
        uint32_t grid;
        begin_args(&k, batch, info);
        if ((st = add_matrix(&k, desc, blob)) != HUFFLLM_OK) return st;
        if ((st = finish_args(&k, true, info, &grid)) != HUFFLLM_OK) return st;
    }
    // the array keeps whatever the last call (finished or not) left: the control words must start at zero
    e = cudaMemsetAsync(ws, 0, ws_partial_offset(desc), (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "clearing the built-in scratch: %s", cudaGetErrorString(e));
    return huffllm_decode_gemm(desc, blob, x, batch, y, ws, sizeof(g_static_scratch), err_flag, stream);
}

huffllm_status huffllm_stage_copy(void *dst, const void *src, size_t bytes, huffllm_stream stream) {
    clear_error();
    DeviceInfo dev;
    huffllm_status st = device_info(&dev);
    if (st != HUFFLLM_OK) return st;
    if (!dst || !src) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer");
    if (bytes % 16 || ((uintptr_t)dst & 15) || ((uintptr_t)src & 15)) return fail(HUFFLLM_ERR_INVALID_ARG, "size and pointers must be multiples of 16 bytes");
    cudaError_t e = launch_stage_copy(dst, src, bytes, (uint32_t)dev.sms, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "copy launch: %s", cudaGetErrorString(e));
    return HUFFLLM_OK;
}

huffllm_status huffllm_plain_gemv_multi(uint32_t n, const uint16_t *const *ws, const uint64_t *rows, const uint64_t *cols,
                                        const uint16_t *const *xs, float *const *ys, huffllm_stream stream) {
    clear_error();
    DeviceInfo dev;
    huffllm_status st = device_info(&dev);
    if (st != HUFFLLM_OK) return st;
    if (!ws || !rows || !cols || !xs || !ys) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer");
    if (n == 0 || n > kMaxMats) return fail(HUFFLLM_ERR_INVALID_ARG, "between 1 and %u matrices per call", kMaxMats);
    PlainArgs a;
    memset(&a, 0, sizeof(a));
    a.n_mats = n;
    uint64_t total = 0;
    for (uint32_t i = 0; i < n; ++i) {
        if (!ws[i] || !xs[i] || !ys[i] || rows[i] == 0 || cols[i] == 0) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer or empty matrix");
        if (cols[i] % 8 || ((uintptr_t)ws[i] & 15) || ((uintptr_t)xs[i] & 15))
            return fail(HUFFLLM_ERR_UNSUPPORTED, "cols must be a multiple of 8 and pointers 16-byte aligned");
        a.m[i].w = ws[i];
        a.m[i].x = xs[i];
        a.m[i].y = ys[i];
        a.m[i].rows = rows[i];
        a.m[i].cols = cols[i];
        a.m[i].row_first = (uint32_t)total;
        total += rows[i];
        if (total >= (1ull << 31)) return fail(HUFFLLM_ERR_UNSUPPORTED, "too many rows for one launch");
    }
    a.total_rows = (uint32_t)total;
    cudaError_t e = launch_plain_gemv(a, (uint32_t)dev.sms, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "plain gemv launch: %s", cudaGetErrorString(e));
    return HUFFLLM_OK;
}

huffllm_status huffllm_plain_gemv(const uint16_t *w, uint64_t rows, uint64_t cols, const uint16_t *x, float *y, huffllm_stream stream) {
    return huffllm_plain_gemv_multi(1, &w, &rows, &cols, &x, &y, stream);
}

}  // extern "C"
