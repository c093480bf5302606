// Small-batch product on the 5th-generation tensor cores (tcgen05), batch 9..64.
//
// Same decoder as the matrix-vector kernel (one table lookup per weight, two bit sequences per lane), but the
// decoded 16-bit weights are not multiplied from registers: every warp stores its 16 rows x 32 columns of a
// block into TENSOR MEMORY as the A operand of a 128-row tile, the activations of the same 32 columns go to
// shared memory as the B operand, and one thread issues tcgen05.mma (M = 128, N = padded batch, K = 16)
// whose fp32 accumulator also lives in tensor memory.  The decoded weights are consumed where they are
// produced (Section 1 of the paper: decompress only to multiply) and one pass over the compressed bytes
// serves the whole batch; the tensor pipe only takes the batch-fold of multiply-adds off the issue slots.
//
// Geometry of a CTA: 4 tiles of 8 warps; a tile is 128 rows (8 row groups of 16), warp (q = warp % 4, h = warp / 4 % 2)
// of a tile owns tensor-memory lanes 32 q + 16 h .. + 15, which is what the 16x256b store shape of a warp can reach.
// The CTA's LAST warp does not decode: it issues the MMAs (so a CTA decodes 31 row groups at a time, and the last 16 rows
// of the fourth tile are never read).  Tensor memory (512 columns): 4 accumulators of N columns, then 4 tiles x S stages
// x 32 columns of A (a stage = two blocks of 32 weight columns = four K = 16 steps; a chunk's odd last block makes a
// stage of one block).
// A work item is (31 row groups) x (a range of column chunks); partial results of the ranges of one row tile are
// added in a fixed order by whoever finishes last (per-warp arrival counters, nobody waits).
//
// Stage protocol: a decoder warp fills its share of stage s (A rows, a slice of B; each block into its half of the stage
// as soon as it is decoded), arrives on the stage's "full" mbarrier and goes on decoding; no warp waits for another one except through the depth of the stage ring.  The issuer
// warp waits for a stage to be full, issues its 16 MMAs and a tcgen05.commit onto the stage's "empty" mbarrier, which the
// decoders wait on (with a limit) before they reuse the stage.  (With the issue taking turns among the decoder warps and a
// barrier after every block, each block cost the CTA its decode time plus the 2000 cycles one warp needs to issue the
// MMAs: that warp had to decode its next block before the next barrier could open.)
// BF16 and FP16 {1,5,5,5} blobs share the kernel (template parameter FMT): tables, raw part and operand format differ.
#include <atomic>

#include "decode_common.cuh"

namespace huffllm {

constexpr int kTcStages = 3;
constexpr int kTcTiles = 4;

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
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 16 lanes x 512 bits: thread (g = lane / 4, t = lane % 4) supplies, for rows g and g + 8, the 32-bit columns
// 2t, 2t+1 (r0, r1 | r2, r3) and 8 + 2t, 8 + 2t + 1 (r4, r5 | r6, r7).
__device__ __forceinline__ void tc_st_16x256b_x2(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.16x256b.x2.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr), "r"(r[0]),
                 "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tc_mma_f16_tmem_a(uint32_t d, uint32_t a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d),
        "r"(a), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
template <int N>
__device__ __forceinline__ void tc_ld_32x32b(uint32_t taddr, uint32_t (&v)[N]);
template <>
__device__ __forceinline__ void tc_ld_32x32b<8>(uint32_t taddr, uint32_t (&v)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "r"(taddr)
                 : "memory");
}
template <>
__device__ __forceinline__ void tc_ld_32x32b<16>(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
          "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
template <>
__device__ __forceinline__ void tc_ld_32x32b<32>(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, "
        "%18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
          "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]),
          "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
          "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

// Shared-memory matrix descriptor of a K-major operand without swizzle: 8-row x 16-byte core matrices,
// `lbo` bytes between core matrices along K, `sbo` bytes between 8-row groups.
__device__ __forceinline__ uint64_t smem_desc_kmajor(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46);
}

// LB = table index bits; NPAD = batch rounded up to 16, 32 or 64 (the MMA's N); FMT = 0: BF16 blobs, 1: FP16 {1,5,5,5} blobs, 2: FP16 blobs with flat mantissa codes
// (three tables, sign words as the raw part, f16 operands).
// MULTI: the launch works through several matrices (a launch over one matrix reads its arguments without an index).
template <int LB, int NPAD, int FMT, bool MULTI>
__global__ void __launch_bounds__(1024, 1) huff_gemm_tc_kernel(const __grid_constant__ TcArgs T) {
    const KernelArgs &A = T.k;
    constexpr uint32_t kRawBlock = FMT ? 64u : 512u;          // raw bytes of one block of a record
    constexpr uint32_t kRawLane = FMT ? 2u : 16u;             // of which one lane's share
    auto raw_part = [](uint32_t nkb) -> uint32_t { return FMT ? (nkb * 64u + 127u) & ~127u : nkb * 512u; };
    auto load_raw = [](const uint8_t *p) -> uint4 {
        if (FMT) return make_uint4(ldg_stream2(p), 0, 0, 0);
        return ldg_stream16(p);
    };
    // the decoder that starts behind the leading zero bits and takes four codewords at a time (see huff_kernel)
    constexpr bool SKIP = LB == 8 && FMT == 0;
    // FP16 (8-bit tables only here): three codewords at a time with in-place shifts; FMT = 2: flat codes for both mantissa halves
    constexpr int SKIP16 = FMT ? (FMT == 2 ? 3 : 1) : 0;
    constexpr int R = SKIP ? 4 : LB == 8 ? 3 : 2;
    constexpr uint32_t kIdxMask = ((1u << LB) - 1u) << 7;
    constexpr int S = NPAD == 64 ? 2 : kTcStages;          // the host's tc_stages(): shared memory is short at the widest padding
    constexpr uint32_t kBStage = NPAD * 128;                // bytes of B per stage: NPAD rows x 64 columns (two blocks) of bf16
    constexpr uint32_t kLbo = 128, kSbo = 1024;             // core matrices: 8 along K side by side, then the next 8 rows
    constexpr uint32_t kACol0 = kTcTiles * NPAD;            // first tensor-memory column of the A stages
    // instruction descriptor: fp32 accumulate, bf16 x bf16, both K-major, N = NPAD, M = 128
    constexpr uint32_t kIdesc = (1u << 4) | (FMT ? 0u : (1u << 7) | (1u << 10)) | ((uint32_t)(NPAD >> 3) << 17) | ((128u >> 4) << 24);

    extern __shared__ __align__(128) uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t bars[kMaxWarps * 2];   // per warp: its two coded-copy barriers
    __shared__ __align__(8) uint64_t empty_bar[S];          // stage may be refilled (arrived on by tcgen05.commit)
    __shared__ __align__(8) uint64_t full_bar[S];           // every decoder warp's share of the stage is in place
    __shared__ uint32_t s_tmem_base;

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_launch_dependents();   // the next kernel in the stream may be scheduled early; it waits for this one before it reads results
    // the matrix this CTA works in (the launch's CTAs are dealt to its matrices; a CTA builds one table), and the CTA's
    // number among that matrix's CTAs: it takes the matrix's work items J, J + n_cta, ...
    uint32_t mi = 0;
    if (MULTI)
        while (mi + 1 < A.n_mats && blockIdx.x >= A.m[mi + 1].cta_first) ++mi;
    const MatArgs &k = A.m[MULTI ? mi : 0];
    const uint32_t J = blockIdx.x - k.cta_first, n_cta = k.cta_count;
    const uint32_t smem_base = smem_u32(dyn_smem);
    // decoder warps: eight per tile, except that the CTA's last warp never decodes: it issues the MMAs (with four tiles the
    // last tile has seven row groups; its last 16 rows are never read).  Warps between the decoders and the issuer leave at once.
    const uint32_t n_tiles = A.tc_tiles, n_dec = min(n_tiles * 8u, 31u), issuer = 31u;
    const SmemPlan plan = plan_smem(smem_base, A, n_dec);
    if (plan.warps < n_dec) {                                   // the entry point sizes shared memory so that this cannot happen
        if (tid == 0 && A.err) atomicExch(A.err, -3);
        return;
    }
    const uint32_t b_base = smem_base + A.dyn_smem_bytes - A.part_bytes;   // S stages of B behind everything else
    uint32_t lut_lane = plan.lut | ((FMT ? lane & 15u : lane) << 2);
    asm volatile("mov.u32 %0, %0;" : "+r"(lut_lane));
    const uint32_t bar0 = smem_u32(&bars[warp * 2]);
    const uint32_t slot0 = slot_addr(plan, warp, 0, A.slot_bytes);    // (this kernel always runs with two slots per warp)

    // ---- set-up: table, barriers, tensor memory
    {
        const uint32_t *lut_g = (const uint32_t *)(k.blob + k.off_lut);
        uint32_t *lut_s = (uint32_t *)(dyn_smem + (plan.lut - smem_base));
        // (FP16: three tables of 256 entries, sixteen copies each: word j holds entry j / 16)
        constexpr uint32_t kLutWords = FMT == 2 ? 16u * 256u : FMT ? 3u * 16u * 256u : 32u << LB;   // (flat mantissa codes: the exponent's table alone)
        for (uint32_t i = tid; i < kLutWords; i += 1024) {
            const uint32_t v = __ldg(lut_g + (i >> (FMT ? 4 : 5)));
            lut_s[i] = SKIP ? lut_entry_inplace(v) : SKIP16 ? fp16_entry_inplace(v) : v;
        }
    }
    if (lane == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
    }
    if (tid < S) {
        mbar_init(smem_u32(&empty_bar[tid]), 1);
        mbar_init(smem_u32(&full_bar[tid]), n_dec);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (warp == 0) {
        tmem_alloc(smem_u32(&s_tmem_base), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    if (warp >= n_dec && warp != issuer) {   // neither decoder nor issuer in this configuration: only the teardown barrier is left
        tc_fence_before();
        __syncthreads();
        return;
    }

    // the table is built and tensor memory allocated: from here on activations are read and results written, which the
    // kernel in front of this one in the stream may still be producing
    pdl_wait_prior_grid();

    // ---- roles
    const uint32_t tile = warp >> 3, q = warp & 3, h = (warp >> 2) & 1;
    const uint32_t rgi = tile * 8 + q * 2 + h;                              // row group of the CTA's 32 that this warp decodes
    const uint32_t a_lane = (32u * q + 16u * h) << 16;
    const uint32_t KC = k.col_chunks, RG = (uint32_t)((k.rows + 15) / 16);
    const uint32_t *index = (const uint32_t *)(k.blob + k.off_index);
    const uint8_t *payload = k.blob + k.off_payload;
    const uint32_t ksplit = T.ksplit[MULTI ? mi : 0], n_items = T.m_tiles[MULTI ? mi : 0] * ksplit;
    float *const tc_partial = T.partial[MULTI ? mi : 0];
    unsigned int *const tc_ticket = T.ticket[MULTI ? mi : 0];
    uint32_t phase = 0, gb = 0;          // coded-copy barrier parities; blocks this CTA has gone through so far
    bool failed = false;                 // a wait ran out: stop waiting, keep moving, report

    auto blocks_of = [&](uint32_t kc) -> uint32_t {
        uint32_t left = (uint32_t)k.cols - kc * k.chunk_cols;
        return (min(left, k.chunk_cols) + 31u) >> 5;
    };
    auto record_ok = [&](uint32_t r0, uint32_t r1, uint32_t nkb) -> bool {
        return r1 > r0 && r1 <= k.payload_units && (r1 - r0) * 128u > raw_part(nkb) &&
               (r1 - r0) * 128u - raw_part(nkb) <= A.slot_bytes;
    };
    auto issue = [&](uint32_t c, uint32_t which) {
        uint32_t nkb = blocks_of(c % KC), r0 = __ldg(index + c), r1 = __ldg(index + c + 1);
        uint32_t bar = bar0 + which * 8;
        if (record_ok(r0, r1, nkb)) {
            uint32_t bytes = (r1 - r0) * 128u - raw_part(nkb);
            mbar_expect_tx(bar, bytes);
            bulk_g2s(slot0 + which * A.slot_bytes, payload + (uint64_t)r0 * 128u + raw_part(nkb), bytes, bar);
        } else {
            mbar_expect_tx(bar, 0);
        }
    };
    auto bounded_wait = [&](uint32_t bar, uint32_t parity) {
        if (failed) return;
        uint32_t spins = 0;
        bool done = mbar_try_wait(bar, parity);
        while (!__all_sync(0xFFFFFFFFu, done)) {
            if (++spins > kWaitLimit) {
                failed = true;
                if (A.err && lane == 0) atomicExch(A.err, -2);
                return;
            }
            done = mbar_try_wait(bar, parity);
        }
    };

    // The activations of a block are NPAD * 4 pieces of 16 bytes, 32 per warp, carried by the first warps.  A warp's
    // piece u = 32 warp + lane belongs to vector n = u / 4 and K positions 8 kap .. 8 kap + 7 (kap = u % 4) of the
    // tile, which hold columns base .. base + 3 and base + 8 .. base + 11 of the block, base = 16 (kap & 1) + 4 (kap >> 1).
    const bool x_carrier = warp * 32 + lane < NPAD * 4;
    const bool x_carrier_warp = warp * 32 < NPAD * 4;            // (NPAD * 4 is a multiple of 32: whole warps carry)
    const uint32_t x_n = (warp * 32 + lane) >> 2, x_kap = lane & 3;
    const uint16_t *x_src = k.x + (uint64_t)x_n * k.cols + (x_kap & 1) * 16 + (x_kap >> 1) * 4;
    const bool x_loads = x_carrier && x_n < A.batch;         // carriers of padding vectors stage zeros
    auto load_x = [&](uint4 &v, const uint16_t *p) {         // fetched one block ahead of its use
        if (x_loads) {
            uint2 lo = __ldg((const uint2 *)p), hi = __ldg((const uint2 *)(p + 8));
            v = make_uint4(lo.x, lo.y, hi.x, hi.y);
        }
    };
    // addresses that change only with the stage: this warp's rows of the A operand, its piece of the B slice
    const uint32_t a_dst0 = tmem + a_lane + kACol0 + tile * S * 32;
    const uint32_t x_dst0 = b_base + (x_n >> 3) * kSbo + x_kap * kLbo + (x_n & 7) * 16;

    // One block of the stage protocol, decoder side.  `a` = this warp's decoded 16 rows x 32 columns (null if the warp has
    // no rows).  The warp stores its share, says so on the stage's "full" barrier and goes on decoding: nobody waits for
    // the other warps here.  A warp can run ahead of the slowest one by the depth of the stage ring and no further (it
    // needs the stage back, which the issuer's tcgen05.commit announces on the "empty" barrier).
    auto stage_block = [&](const uint32_t *a, const uint4 &xv, uint32_t half, bool publish) {
        const uint32_t s = gb % S, use = gb / S;
        if (half == 0) {
            if (use > 0) bounded_wait(smem_u32(&empty_bar[s]), (use - 1) & 1u);
            tc_fence_after();
        }
        if (a) {
            // lane (g, t): row g's weights 0..3 -> 32-bit columns 2t, 2t+1; weights 4..7 -> columns 8 + 2t, 8 + 2t + 1
            const uint32_t r[8] = {a[0], a[1], a[4], a[5], a[2], a[3], a[6], a[7]};
            tc_st_16x256b_x2(a_dst0 + s * 32 + half * 16, r);
        }
        if (x_carrier)
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(x_dst0 + s * kBStage + half * 4 * kLbo), "r"(xv.x), "r"(xv.y), "r"(xv.z), "r"(xv.w) : "memory");
        if (!publish) return;
        tc_wait_st();
        if (x_carrier_warp) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the B slice must be visible to the tensor core's reads
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&full_bar[s]));
        ++gb;
    };
    // The same block, issuer side: when every decoder warp has arrived, one lane issues the block's MMAs for every tile
    // and commits them onto the stage's "empty" barrier.  (After a wait that ran out the commit still goes out: the
    // stage ring keeps moving and the kernel ends with its error flag set.)
    auto issue_block = [&](bool first_of_item, uint32_t halves) {
        const uint32_t s = gb % S, use = gb / S;
        bounded_wait(smem_u32(&full_bar[s]), use & 1u);
        if (lane == 0) {
            tc_fence_after();
            const uint32_t bst = b_base + s * kBStage;
            if (!failed) {
                for (uint32_t tl = 0; tl < n_tiles; ++tl) {
#pragma unroll
                    for (uint32_t j = 0; j < 4; ++j)      // four K = 16 steps per full stage, two for the odd last block of a chunk
                        if (j < 2 * halves)
                            tc_mma_f16_tmem_a(tmem + tl * NPAD, tmem + kACol0 + (tl * S + s) * 32 + j * 8,
                                              smem_desc_kmajor(bst + j * 2 * kLbo, kLbo, kSbo), kIdesc, (first_of_item && j == 0) ? 0u : 1u);
                }
            }
            tc_commit(smem_u32(&empty_bar[s]));
        }
        __syncwarp();
        ++gb;
    };

    // first and last chunk of this warp's row group in a work item (false: the row group lies outside the matrix)
    auto item_chunks = [&](uint32_t it, uint32_t &cb, uint32_t &ce) -> bool {
        const uint32_t mt_i = it / ksplit, ks_i = it % ksplit, rg_i = mt_i * n_dec + rgi;
        cb = rg_i * KC + (uint32_t)((uint64_t)KC * ks_i / ksplit);
        ce = rg_i * KC + (uint32_t)((uint64_t)KC * (ks_i + 1) / ksplit);
        return rg_i < RG;
    };
    bool primed = false;                 // the item's first two record copies were started at the end of the item before

#pragma unroll 1
    for (uint32_t item = J; item < n_items; item += n_cta) {
        const uint32_t mt = item / ksplit, ks = item % ksplit;
        const uint32_t rg = mt * n_dec + rgi;
        const bool active = rg < RG;
        const uint32_t kc0 = (uint32_t)((uint64_t)KC * ks / ksplit), kc1 = (uint32_t)((uint64_t)KC * (ks + 1) / ksplit);
        const uint32_t gb_item = gb;
        // the item's blocks are consecutive 32-column blocks of the matrix, from col_lo up to col_hi
        const uint32_t col_lo = kc0 * k.chunk_cols, col_hi = min(kc1 * k.chunk_cols, (uint32_t)k.cols);
        // activations: x_a holds the current block's piece at the top of every chunk; the pointer names the block after it
        const uint16_t *x_p = x_src + col_lo + 32, *const x_end = x_src + col_hi;
        uint4 x_a = make_uint4(0, 0, 0, 0), x_b = make_uint4(0, 0, 0, 0);
        load_x(x_a, x_src + col_lo);

        if (warp == issuer) {
            for (uint32_t kc = kc0; kc < kc1; ++kc) {       // stages are cut like the decoders': pairs of blocks inside a chunk
                const uint32_t nkb = blocks_of(kc);
                for (uint32_t kb = 0; kb < nkb; kb += 2) issue_block(gb == gb_item, min(nkb - kb, 2u));
            }
        } else if (active) {
            const uint32_t c_beg = rg * KC + kc0, c_end = rg * KC + kc1;
            if (lane == 0 && !primed) {
                issue(c_beg, 0);
                if (c_beg + 1 < c_end) issue(c_beg + 1, 1);
            }
            uint32_t kc = kc0;
            uint32_t r0 = __ldg(index + c_beg), r1 = __ldg(index + c_beg + 1);
#pragma unroll 1
            for (uint32_t c = c_beg; c < c_end; ++c, ++kc) {
                const uint32_t which = (c - c_beg) & 1u;
                const uint32_t nkb = blocks_of(kc);
                const bool ok = record_ok(r0, r1, nkb);
                const uint32_t r2 = c + 1 < c_end ? __ldg(index + c + 2) : r1;
                const uint8_t *raw_p = payload + (uint64_t)r0 * 128u + lane * kRawLane;
                uint4 raw_cur = make_uint4(0, 0, 0, 0);
                if (ok) raw_cur = load_raw(raw_p);
                bounded_wait(bar0 + which * 8, (phase >> which) & 1u);
                phase ^= 1u << which;
                if (!ok && A.err && lane == 0) atomicExch(A.err, (int32_t)min(c + 1, 0x7FFFFFFFu));
                if (!ok) {
                    // record offsets out of range (reported above): nothing of the record is touched, zeros go to the stages
                    const uint32_t zero[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
                    for (uint32_t kb = 0; kb < nkb; ++kb) {
                        if (x_p < x_end) load_x(x_b, x_p);
                        x_p += 32;
                        stage_block(zero, x_a, kb & 1u, (kb & 1u) || kb + 1 == nkb);
                        x_a = x_b;
                    }
                    __syncwarp();
                    if (lane == 0 && c + 2 < c_end) issue(c + 2, which);
                    r0 = r1;
                    r1 = r2;
                    continue;
                }
                LaneStream sa, sb;
                stream_open(sa, slot0 + which * A.slot_bytes + (lane << 2), SKIP ? 7u : SKIP16 ? 6u : 0u);
                stream_open(sb, slot0 + which * A.slot_bytes + 128u + (lane << 2), SKIP ? 7u : SKIP16 ? 6u : 0u);
                // one block: fetch the next block's raw bytes and activations into the other register set, decode
                // this one, hand it to the tensor core
                auto block = [&](const uint4 &raw_c, uint4 &raw_n, const uint4 &x_c, uint4 &x_n2, bool more, uint32_t half, bool publish) {
                    raw_p += kRawBlock;
                    if (more) raw_n = load_raw(raw_p);
                    if (x_p < x_end) load_x(x_n2, x_p);
                    x_p += 32;
                    uint32_t a[8];
                    if (FMT) decode_block_fp16<false, SKIP16>(sa, sb, lut_lane, raw_c.x, a);
                    else decode_block<R, SKIP>(sa, sb, kIdxMask, lut_lane, raw_c, a);
                    stage_block(a, x_c, half, publish);
                };
                uint4 raw_b = make_uint4(0, 0, 0, 0);
                uint32_t kb = 0;
#pragma unroll 1
                for (; kb + 2 <= nkb; kb += 2) {                  // the usual case: pairs of blocks, two register sets in turn
                    block(raw_cur, raw_b, x_a, x_b, true, 0, false);
                    block(raw_b, raw_cur, x_b, x_a, kb + 2 < nkb, 1, true);
                }
                if (kb < nkb) {                                   // odd block count (a ragged last chunk): a stage of one block
                    block(raw_cur, raw_b, x_a, x_b, false, 0, true);
                    x_a = x_b;
                }
                __syncwarp();
                if (lane == 0 && c + 2 < c_end) issue(c + 2, which);
                r0 = r1;
                r1 = r2;
            }
        } else {
            // no rows of the matrix for this warp: it still carries its slice of the activations and its arrivals
            for (uint32_t kc = kc0; kc < kc1; ++kc) {
                const uint32_t nkb = blocks_of(kc);
                for (uint32_t kb = 0; kb < nkb; ++kb) {
                    if (x_p < x_end) load_x(x_b, x_p);
                    x_p += 32;
                    stage_block(nullptr, x_a, kb & 1u, (kb & 1u) || kb + 1 == nkb);
                    x_a = x_b;
                }
            }
        }

        // both slots are free again: the next item's first records are asked for now, so that they arrive behind the epilogue
        primed = false;
        if (warp < n_dec && item + n_cta < n_items) {
            uint32_t nb, ne;
            if (item_chunks(item + n_cta, nb, ne)) {
                if (lane == 0) {
                    issue(nb, 0);
                    if (nb + 1 < ne) issue(nb + 1, 1);
                }
                primed = true;
            }
        }

        // ---- epilogue of the item: wait for the last stage's MMAs, read this warp's 32 rows x NPAD/2 columns
        // (the issuer has a share like every warp of a tile; with fewer than four tiles its tile does not exist)
        if (tile < n_tiles) {
            const uint32_t gl = gb - 1;
            bounded_wait(smem_u32(&empty_bar[gl % S]), (gl / S) & 1u);
            tc_fence_after();
            uint32_t v[NPAD / 2];
            tc_ld_32x32b<NPAD / 2>(tmem + ((32u * q) << 16) + tile * NPAD + h * (NPAD / 2), v);
            tc_wait_ld();
            tc_fence_before();
            // thread `lane` holds row 32 q + lane of the tile, columns n = h * NPAD/2 + i
            const uint64_t row = (uint64_t)(mt * n_dec + tile * 8) * 16 + 32u * q + lane;
            const bool row_ok = row < k.rows && tile * 8 + 2 * q + (lane >> 4) < n_dec;   // (the last tile's last row group belongs to the next item)
            const uint32_t n0 = h * (NPAD / 2);
            if (ksplit == 1) {
#pragma unroll
                for (int i = 0; i < NPAD / 2; ++i)
                    if (n0 + i < A.batch && row_ok) k.y[(uint64_t)(n0 + i) * k.rows + row] = __uint_as_float(v[i]);
            } else {
                // piece of (item, warp): [NPAD/2][32] floats; the last range to arrive adds the pieces in range order
                float *piece = tc_partial + ((size_t)item * 32 + warp) * (NPAD / 2) * 32;   // 32 piece slots per item, n_dec used
#pragma unroll
                for (int i = 0; i < NPAD / 2; ++i) piece[i * 32 + lane] = __uint_as_float(v[i]);
                __syncwarp();
                uint32_t last = 0;
                if (lane == 0) {
                    unsigned int *ctr = tc_ticket + mt * 32 + warp;
                    last = arrive_acq_rel(ctr) == ksplit - 1 ? 1u : 0u;
                    if (last) *ctr = 0;
                }
                if (__shfl_sync(0xFFFFFFFFu, last, 0)) {
                    // range after range, NPAD/2 independent loads in flight each time; every output adds its pieces in range order
                    float sum[NPAD / 2];
#pragma unroll
                    for (int i = 0; i < NPAD / 2; ++i) sum[i] = 0.f;
                    for (uint32_t s2 = 0; s2 < ksplit; ++s2) {
                        const float *pc = tc_partial + ((size_t)(mt * ksplit + s2) * 32 + warp) * (NPAD / 2) * 32 + lane;
#pragma unroll
                        for (int i = 0; i < NPAD / 2; ++i) sum[i] += __ldcg(pc + i * 32);
                    }
#pragma unroll
                    for (int i = 0; i < NPAD / 2; ++i)
                        if (n0 + i < A.batch && row_ok) k.y[(uint64_t)(n0 + i) * k.rows + row] = sum[i];
                }
            }
        }
    }

    // ---- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

template <int LB, int NPAD, int FMT, bool MULTI>
static cudaError_t launch_tc_m(const TcArgs &t, uint32_t grid, cudaStream_t stream) {
    const KernelArgs &k = t.k;
    auto fn = huff_gemm_tc_kernel<LB, NPAD, FMT, MULTI>;
    static std::atomic<bool> attr_set[64];   // set twice by racing threads at worst: the call is idempotent
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)k.dyn_smem_bytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev].store(true, std::memory_order_release);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(1024);
    cfg.dynamicSmemBytes = k.dyn_smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set-up overlaps the previous kernel's tail
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fn, t);
}

template <int LB, int NPAD, int FMT>
static cudaError_t launch_tc_one(const TcArgs &t, uint32_t grid, cudaStream_t stream) {
    if (t.k.n_mats > 1) return launch_tc_m<LB, NPAD, FMT, true>(t, grid, stream);
    return launch_tc_m<LB, NPAD, FMT, false>(t, grid, stream);
}

cudaError_t launch_gemm_tc(const TcArgs &t, uint32_t grid, cudaStream_t stream) {
    const KernelArgs &k = t.k;
    if (k.fmt && k.fp16_flat) {
        if (k.tc_npad == 16) return launch_tc_one<8, 16, 2>(t, grid, stream);
        if (k.tc_npad == 32) return launch_tc_one<8, 32, 2>(t, grid, stream);
        return launch_tc_one<8, 64, 2>(t, grid, stream);
    }
    if (k.fmt) {
        if (k.tc_npad == 16) return launch_tc_one<8, 16, 1>(t, grid, stream);
        if (k.tc_npad == 32) return launch_tc_one<8, 32, 1>(t, grid, stream);
        return launch_tc_one<8, 64, 1>(t, grid, stream);
    }
    if (k.lut_bits == 8) {
        if (k.tc_npad == 16) return launch_tc_one<8, 16, 0>(t, grid, stream);
        if (k.tc_npad == 32) return launch_tc_one<8, 32, 0>(t, grid, stream);
        return launch_tc_one<8, 64, 0>(t, grid, stream);
    }
    if (k.tc_npad == 16) return launch_tc_one<9, 16, 0>(t, grid, stream);
    if (k.tc_npad == 32) return launch_tc_one<9, 32, 0>(t, grid, stream);
    return launch_tc_one<9, 64, 0>(t, grid, stream);
}

}  // namespace huffllm
