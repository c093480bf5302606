// Device kernels (sm_100a): Huffman decode of the chunked blob, alone and fused into the
// matrix-vector / small-batch matrix product.
//
// What one decoder step does is the paper's (Section 3.2): look at the next L_max bits at the start
// pointer, find the codeword they begin with, emit its symbol, advance the pointer by its length.
// The CAM of the hardware decoder becomes a lookup table in shared memory; because the two 4-bit
// exponent codes of one BF16 weight (Section 5.1) are adjacent in the stream and their joint length
// is bounded, one lookup resolves both.  The decoded exponent is merged with the raw sign and
// mantissa into the 16-bit weight (Section 3.2) in registers and consumed at once, so decompressed
// weights never touch memory (Section 1).
//
// Mapping to the GPU
//   * one warp decodes one chunk; lane l owns the two bit sequences l and 32 + l of the chunk record
//     and steps through them alternately, which gives every lane two independent dependency chains
//   * one warp of the CTA (the feeder) does the bookkeeping of all the others: per decoder warp it reads the
//     record index, checks the offsets and starts one bulk-async copy per chunk (no multicast) of the coded
//     part into one of the warp's two shared-memory slots, completion on an mbarrier; a second mbarrier per
//     slot brings the slot back.  It also asks L2 for the raw part of a record with one bulk prefetch
//   * the raw sign/mantissa bytes go straight from global memory to the decoders' registers, 16 bytes per
//     lane per block of 32 columns, one block ahead
//   * the LUT is replicated per lane in shared memory (entry i of lane l at word 32 i + l), so a
//     warp-wide lookup never has a bank conflict
//   * a lane's 16 weights of a block are exactly its share of two m16n8k16 tensor-core operand
//     tiles, so the product needs no shuffles: decode, pack to bf16x2, mma
//   * partial sums of a row group that is split over warps or CTAs are combined in a fixed order
//     (shared memory inside a CTA, arrival counters and a scratch buffer across CTAs); nobody waits for anybody
#include <cuda_runtime.h>
#include <atomic>
#include <cstdint>
#include <type_traits>

#include "decode_common.cuh"

namespace huffllm {

// ------------------------------------------------------------------------------ the fused kernel

// MODE 0: write the decoded weights.  MODE 1: y = W x for up to 8 activation vectors.
// LB = table index bits (the blobs' lut_bits): 8 or 9; LB = 12 stands for every longer limit up to 12 (BF16: 10..12,
// FP16: 9..12): two-level lookup, the number of bits is A.lut_bits.
// FMT = 0: BF16 blobs; FMT = 1: FP16 {1,5,5,5} blobs (three lookups per weight, sign bits as the raw part); FMT = 2: the same
// where both mantissa halves carry the flat 5-bit code (8-bit tables only: one lookup and a bit reversal per weight).
//
// One launch works through a LIST of matrices (A.n_mats, usually the matrices of one decoder layer that
// may run together).  The CTAs are dealt out to the matrices in proportion to their chunks, so every CTA
// lies inside a single matrix, builds a single table and meets no CTA-wide barrier after set-up.
//
// Roles.  The last warp of the CTA is the FEEDER: lane w looks after decoder warp w.  It reads the record index,
// checks the offsets, starts the bulk copy of a chunk's coded part into one of the warp's two slots and leaves
// a two-word note (the record's offsets) beside it; the copy's barrier carries the note to the decoder.  When a
// decoder has finished with a slot it says so on a second barrier, which the feeder polls.  All bookkeeping of a
// chunk is thus one lane's work instead of a whole warp's: the decoder warps, whose issue slots bound the kernel,
// spend theirs on decoding.
// NT = 8-column tiles of activations per product: 1 (batch 1..8) or 2 (batch 9..16: twice the multiply-adds on the same
// decoded registers; the pieces that warps of a CTA exchange then live in the workspace, shared memory has no room for them).
// NT = 0 (BF16 blobs, batch 1): no tensor core at all.  The two mma.sync of a block cost the decoders more issue time
// than the sixteen mixed-precision multiply-adds (bf16 x bf16 + f32, `fma.rn.f32.bf16`) that a lane needs for its 16
// weights and one vector: those run on the FMA pipe, which the decoder leaves idle.
// SLOTS = shared-memory slots per decoder warp: 2 (a warp's next record lands while it decodes this one), or 1 for records
// so large that pairs would leave too few warps a place (the feeder then waits for the slot before every copy).
template <int MODE, int LB, int THREADS, int FMT, int NT = 1, int SLOTS = 2>
__global__ void __launch_bounds__(THREADS, 1) huff_kernel(const __grid_constant__ KernelArgs A) {
    constexpr int kV = NT == 2 ? 8 : 4;                       // values a lane holds of a row group's 16 x batch outputs
    constexpr uint32_t kRawBlock = FMT ? 64u : 512u;          // raw bytes of one block of a record
    constexpr uint32_t kRawLane = FMT ? 2u : 16u;             // of which one lane's share
    // raw part of a record with nkb blocks, in record units of 128 bytes (FP16: rounded up to whole units)
    auto raw_units = [](uint32_t nkb) -> uint32_t { return FMT ? (nkb + 1u) >> 1 : nkb * 4u; };
    // 8-bit BF16 tables: the decoder starts behind the sequences' leading zero bits and works on four codewords at a
    // time (stream_step4x2)
    constexpr bool SKIP = LB == 8 && FMT == 0;
    constexpr int SKIP16 = FMT ? (LB == 8 ? (FMT == 2 ? 3 : 1) : LB == 7 ? 2 : 0) : 0;   // the same scheme for FP16: three codewords (one weight) at a
                                                             // time; 2 = field codes of 7 bits, tables once per lane
    constexpr bool LONG = LB > 9;                            // first level of 8 bits, then the whole table (FP16: lut_bits 9..12)
    constexpr uint32_t kLB1 = LONG ? 8u : (uint32_t)LB;      // index bits of the per-lane table
    constexpr int R = SKIP ? 4 : LB == 8 ? 3 : 2;            // decoder steps between two refill checks
    constexpr uint32_t kIdxMask = ((1u << kLB1) - 1u) << 7;
    extern __shared__ __align__(128) uint8_t dyn_smem[];
    // per decoder warp: "full" barriers of its two slots (the copy has landed), then the two "empty" ones (the decoder is done)
    __shared__ __align__(16) uint64_t bars[kMaxWarps * 4];
    __shared__ __align__(16) uint2 notes[kMaxWarps * 2];       // per slot: the record's first and last offset, or kBadRecord
    __shared__ uint32_t s_arrive[kMaxWarps];   // arrival counters of row groups shared by several warps
    __shared__ uint32_t s_stop;                // a decoder gave up waiting: the feeder stops too
    constexpr uint32_t kBadRecord = 0xFFFFFFFFu;

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps_launched = blockDim.x >> 5;
    pdl_launch_dependents();   // the next kernel's set-up may overlap this kernel's tail
    const uint32_t smem_base = smem_u32(dyn_smem);
    const uint32_t feeder = nwarps_launched - 1;
    const SmemPlan plan = plan_smem(smem_base, A, feeder, SLOTS);
    const uint32_t nw = plan.warps;                            // decoder warps
    const uint32_t vals = 16 * A.batch;
    // the pieces of row groups that several warps of the CTA share: [2 * warps][16 * batch], in shared memory (NT = 1)
    float *part_val = (float *)(dyn_smem + A.dyn_smem_bytes - A.part_bytes);

    // the matrix this CTA works in, and the CTA's piece of that matrix's chunks
    uint32_t mi = 0;
    while (mi + 1 < A.n_mats && blockIdx.x >= A.m[mi + 1].cta_first) ++mi;
    const MatArgs &k = A.m[mi];
    const uint32_t J = blockIdx.x - k.cta_first;                        // this CTA's number among the CTAs of its matrix
    auto cta_cut = [&](uint32_t j) -> uint32_t { return j * k.cta_chunks + min(j, k.cta_extra); };   // first chunk of the matrix's CTA j
    const uint32_t cta_beg = cta_cut(J), cta_end = cta_cut(J + 1);
    const uint32_t KC = k.col_chunks;
    // the CTA's chunks are dealt to its decoder warps: wq each, and wr warps in the MIDDLE of the range one more.  The
    // warps with the extra chunk finish last; in the middle their row groups belong to this CTA alone, so what runs at
    // the very end of the launch is a reduction in shared memory, not the one across CTAs with its global round trips
    const uint32_t cta_len = cta_end - cta_beg, wq = nw == 31 ? cta_len / 31u : cta_len / nw, wr = cta_len - wq * nw;
    const uint32_t w_mid = (nw - wr) >> 1;
    auto warp_beg = [&](uint32_t w) -> uint32_t { return cta_beg + w * wq + min(w > w_mid ? w - w_mid : 0u, wr); };
    const uint32_t *index = (const uint32_t *)(k.blob + k.off_index);
    const uint8_t *payload = k.blob + k.off_payload;
    // blocks of 32 columns in column chunk kc: every chunk is full except, possibly, the last one of a row
    const uint32_t nkb_full = k.chunk_cols >> 5, nkb_tail = ((uint32_t)k.cols - (KC - 1) * k.chunk_cols + 31u) >> 5;

    const uint32_t bar_w = smem_u32(&bars[(warp == feeder ? lane : warp) * 4]);   // the four barriers of "my" decoder warp
    constexpr uint32_t kSetupBarrier = 1;       // hardware barrier of the set-up: the decoders wait at it, the feeder only arrives

    if (warp == feeder) {
        // ================================================================== the feeder
        // lane w: next chunk and end of decoder warp w's range, that chunk's column chunk, chunks issued so far, and the
        // offsets of the record to issue next
        uint32_t f_ci = 0, f_ce = 0, f_issued = 0, f_ra = 0, f_rb = 0;
        if (lane < nw) {
            f_ci = warp_beg(lane);
            f_ce = warp_beg(lane + 1);
            if (f_ci < f_ce) {                       // asked for first: the set-up below runs while the answers are under way
                f_ra = __ldg(index + f_ci);
                f_rb = __ldg(index + f_ci + 1);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) mbar_init(bar_w + 8 * i, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        if (lane == 0) *(volatile uint32_t *)&s_stop = 0;
        __syncwarp();
        // the barriers exist: the decoders may go on as soon as their table is built; the feeder does not wait for them
        asm volatile("bar.arrive %0, %1;" ::"r"(kSetupBarrier), "r"(THREADS) : "memory");
        uint32_t f_kc = f_ci % KC;
        const uint32_t slot_units = A.slot_bytes >> 7, slot_w = SLOTS == 2 ? slot_addr(plan, lane < nw ? lane : 0u, 0, A.slot_bytes)
                                                                                : slot_addr_single(plan, lane < nw ? lane : 0u, A.slot_bytes);
        const uint32_t note_w = smem_u32(&notes[lane * 2]);
        uint32_t idle = 0;
        while (__any_sync(0xFFFFFFFFu, f_ci < f_ce)) {
            const uint32_t which = f_issued & 1u;
            // a slot is free for its first chunk, and later once the decoder has handed it back: with two slots that is the
            // chunk before the last one issued, with one slot the last one (barriers and notes alternate either way)
            const bool ready = f_ci < f_ce &&
                               (SLOTS == 2 ? f_issued < 2 || mbar_test_wait(bar_w + 16 + 8 * which, ((f_issued >> 1) - 1u) & 1u)
                                           : f_issued < 1 || mbar_test_wait(bar_w + 16 + 8 * (which ^ 1u), ((f_issued - 1u) >> 1) & 1u));
            if (ready) {
                const uint32_t full = bar_w + 8 * which, nkb = f_kc + 1 == KC ? nkb_tail : nkb_full;
                // a record is usable if it lies inside the payload, is longer than its raw part and its coded part fits a slot
                const bool ok = f_rb <= k.payload_units && f_rb - f_ra - raw_units(nkb) - 1u < slot_units;
                asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(note_w + 8 * which), "r"(ok ? f_ra : kBadRecord), "r"(f_rb) : "memory");
                if (ok) {
                    const uint32_t bytes = (f_rb - f_ra - raw_units(nkb)) << 7;
                    mbar_expect_tx(full, bytes);
                    bulk_g2s(slot_w + (SLOTS == 2 ? which * A.slot_bytes : 0u), payload + ((uint64_t)(f_ra + raw_units(nkb)) << 7), bytes, full);
                    // the raw part of the record is asked into L2 with one request (not for a warp's first two chunks: at the
                    // start of a launch every warp's copies are under way at once, and only the decoders' own loads matter)
                    if (f_issued >= 2)
                        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(payload + ((uint64_t)f_ra << 7)), "r"(raw_units(nkb) << 7) : "memory");
                } else {
                    mbar_expect_tx(full, 0);  // completes the phase with nothing to wait for; the decoder skips the chunk
                }
                ++f_ci;
                ++f_issued;
                f_kc = f_kc + 1 == KC ? 0u : f_kc + 1;
                f_ra = f_rb;
                if (f_ci < f_ce) f_rb = __ldg(index + f_ci + 1);
            }
            if (__any_sync(0xFFFFFFFFu, ready)) {
                idle = 0;
            } else {
                __nanosleep(100);
                if (++idle > kFeederIdleLimit || *(volatile uint32_t *)&s_stop) break;   // (a decoder that stopped never hands slots back)
            }
        }
        return;
    }

    // ====================================================================== the decoder warps
    // ---- set-up: the table loads are started first, then this warp's own values are worked out, then the table is
    // written to shared memory (by the decoder warps alone: the feeder is already asking for records)
    // (FP16: three tables of 256 entries, sixteen copies each: word j holds entry j / 16 of its table)
    // The table goes to shared memory in 16-byte pieces: four neighbouring copies of one entry per piece.
    // (FP16, 7 bits: 3 x 32 x 128, the same; flat mantissa codes: the exponent's table alone)
    constexpr uint32_t kLutWords = FMT == 2 ? 16u * 256u : FMT ? 3u * 16u * 256u : 32u << kLB1;
    constexpr uint32_t kLutRep = FMT && LB != 7 ? 4u : 5u; // log2 of the copies per entry
    constexpr uint32_t kLutVecs = kLutWords / 4;
    constexpr uint32_t kLutThreads = THREADS - 32;
    constexpr int kLutLoads = (kLutVecs + kLutThreads - 1) / kLutThreads;
    uint32_t lut_v[kLutLoads];
    {
        const uint32_t *lut_g = (const uint32_t *)(k.blob + k.off_lut);
#pragma unroll
        for (int i = 0; i < kLutLoads; ++i) {
            uint32_t v = tid + i * kLutThreads;
            // (entry of vector v: BF16 v / 8; FP16 field v / 1024, entry v / 4 % 256 of that field's table of 1 << lut_bits)
            const uint32_t src = FMT ? ((v >> 10) << A.lut_bits) + (LB == 7 ? (v >> 3) & 127u : (v >> 2) & 255u) : v >> (kLutRep - 2);
            lut_v[i] = v < kLutVecs ? __ldg(lut_g + src) : 0u;
            if (SKIP) lut_v[i] = lut_entry_inplace(lut_v[i]);   // the length once more, where an in-place shift reads it
            if (SKIP16) lut_v[i] = fp16_entry_inplace(lut_v[i]);
            if (LONG && (lut_v[i] >> 16) > 8u) lut_v[i] |= kLongMark;   // a codeword longer than the first level resolves
        }
    }
    // two-level lookup: the whole table (1 << lut_bits entries, one copy) sits behind the per-lane first level
    const uint32_t full_base = plan.lut + (FMT ? 49152u : 128u << kLB1), full_mask = ((1u << A.lut_bits) - 1u) << 2;
    uint32_t lut_lane = plan.lut | ((FMT && LB != 7 ? lane & 15u : lane) << 2);
    asm volatile("mov.u32 %0, %0;" : "+r"(lut_lane));  // keep it in a register: it is an operand of every lookup
    const uint32_t g = lane >> 2, t = lane & 3;
    uint32_t c_beg = 0, c_end = 0;
    if (warp < nw) {
        c_beg = warp_beg(warp);
        c_end = warp_beg(warp + 1);
    }
    // the warp's first record: its raw bytes are asked for before the table is finished
    uint32_t r_first = c_beg < c_end ? __ldg(index + c_beg) : 0xFFFFFFFFu;
    // raw sign/mantissa bytes travel one block ahead of the decoder, in two register sets used in turn
    uint4 raw_a = make_uint4(0, 0, 0, 0), raw_b = make_uint4(0, 0, 0, 0);
    bool primed = false;
    auto load_raw = [](const uint8_t *p) -> uint4 {
        if (FMT) return make_uint4(ldg_stream2(p), 0, 0, 0);
        return ldg_stream16(p);
    };
    const uint8_t *raw_p = payload;
    {
        uint4 *lut_s = (uint4 *)(dyn_smem + (plan.lut - smem_base));
#pragma unroll
        for (int i = 0; i < kLutLoads; ++i) {
            uint32_t v = tid + i * kLutThreads;
            if (v < kLutVecs) lut_s[v] = make_uint4(lut_v[i], lut_v[i], lut_v[i], lut_v[i]);
        }
        if (tid < kMaxWarps) s_arrive[tid] = 0;
        if (LONG) {
            const uint32_t *lut_g = (const uint32_t *)(k.blob + k.off_lut);
            uint32_t *full_s = (uint32_t *)(dyn_smem + (full_base - smem_base));
            for (uint32_t i = tid; i < (FMT ? 3u : 1u) << A.lut_bits; i += kLutThreads) full_s[i] = __ldg(lut_g + i);
        }
    }
    if (r_first < k.payload_units) {        // (the blob keeps 4 KB behind the payload: a block's read stays inside it)
        raw_p = payload + ((uint64_t)r_first << 7) + lane * kRawLane;
        raw_a = load_raw(raw_p);
        primed = true;
    }
    asm volatile("bar.sync %0, %1;" ::"r"(kSetupBarrier), "r"(THREADS) : "memory");
    if (warp >= nw) return;

    bool waited_prior = false, failed = false;

    float acc[kV];
#pragma unroll
    for (int j = 0; j < kV; ++j) acc[j] = 0.f;
    int cur_rg = -1;
    if (NT == 2) part_val = k.ws_warp_pieces + (size_t)J * (2 * kMaxWarps) * vals;   // (same-SM traffic: it stays in L1 / L2)

    // ---- reduction of a finished row group, without any CTA-wide barrier.
    // A row group whose chunks this warp decoded alone goes straight to y.  Otherwise the warp parks its
    // piece in shared memory and bumps an arrival counter (indexed by the first warp that holds a piece);
    // the warp that arrives last adds the pieces in warp order.  If other CTAs hold pieces too, the CTA's
    // sum goes to the scratch buffer and the same game is played across CTAs with a counter in global
    // memory.  Sums are always taken in the same order, and nobody waits for anybody.
    auto cta_of_chunk = [&](uint32_t ch) -> uint32_t {     // which of the matrix's CTAs works on chunk ch
        const uint32_t big = k.cta_extra * (k.cta_chunks + 1);
        return ch < big ? ch / (k.cta_chunks + 1) : k.cta_extra + (ch - big) / k.cta_chunks;
    };
    // lanes 0..vals-1 (looping if vals > 32) hold or produce the value of output o = column * 16 + row
    auto finish_cta_sum = [&](int rg, float (&v)[kV]) {      // v[i] = value of output o = lane + 32 i
        const uint32_t g_lo = (uint32_t)rg * KC, g_hi = g_lo + KC;
        if (cta_beg <= g_lo && cta_end >= g_hi) {             // the CTA held the whole row group
#pragma unroll
            for (int i = 0; i < kV; ++i) {
                uint32_t o = lane + 32 * i;
                uint64_t r = (uint64_t)rg * 16 + (o & 15);
                if (o < vals && r < k.rows) k.y[(uint64_t)(o >> 4) * k.rows + r] = v[i];
            }
            return;
        }
        // slot 0 holds the piece of the CTA's first row group in this matrix, slot 1 the piece of its last one
        const uint32_t my_slot = (uint32_t)rg == cta_beg / KC ? 0u : 1u;
#pragma unroll
        for (int i = 0; i < kV; ++i) {
            uint32_t o = lane + 32 * i;
            if (o < vals) k.ws_partial[((size_t)J * 2 + my_slot) * vals + o] = v[i];
        }
        __syncwarp();
        const uint32_t c0 = cta_of_chunk(g_lo), c1 = cta_of_chunk(g_hi - 1);
        uint32_t last = 0;
        if (lane == 0) {
            last = arrive_acq_rel(k.ws_ticket + c0) == c1 - c0 ? 1u : 0u;
            if (last) k.ws_ticket[c0] = 0;                    // leave the counter as it was found
        }
        if (!__shfl_sync(0xFFFFFFFFu, last, 0)) return;       // somebody else will arrive later and add us in
#pragma unroll
        for (int i = 0; i < kV; ++i) {
            uint32_t o = lane + 32 * i;
            if (o >= vals) continue;
            float sum = 0.f;
            for (uint32_t c = c0; c <= c1; ++c) {
                uint32_t slot = cta_cut(c) / KC == (uint32_t)rg ? 0u : 1u;
                sum += __ldcg(k.ws_partial + ((size_t)c * 2 + slot) * vals + o);
            }
            uint64_t r = (uint64_t)rg * 16 + (o & 15);
            if (r < k.rows) k.y[(uint64_t)(o >> 4) * k.rows + r] = sum;
        }
    };
    auto flush = [&](int rg, uint32_t first_c, uint32_t last_c_excl) {
        if (rg < 0) return;
        const uint32_t g_lo = max((uint32_t)rg * KC, cta_beg), g_hi = min((uint32_t)(rg + 1) * KC, cta_end);  // this CTA's part
        const bool alone = first_c <= g_lo && last_c_excl >= g_hi;   // no other warp of this CTA holds a piece
        // D fragment -> output order (o = column * 16 + row) through this warp's shared-memory entry
        const uint32_t ent = warp * 2 + ((uint32_t)rg == c_beg / KC ? 0u : 1u);
        float *mine = part_val + (size_t)ent * vals;
        if (NT == 0) {
            // acc[0]: this lane's eight columns of row g; acc[2]: of row g + 8.  The four lanes of a row add theirs
            // (always in this order), and lane t = 0 then holds what the D fragment's column 0 would hold.
            float s_lo = acc[0], s_hi = acc[2];
            s_lo += __shfl_xor_sync(0xFFFFFFFFu, s_lo, 1);
            s_hi += __shfl_xor_sync(0xFFFFFFFFu, s_hi, 1);
            s_lo += __shfl_xor_sync(0xFFFFFFFFu, s_lo, 2);
            s_hi += __shfl_xor_sync(0xFFFFFFFFu, s_hi, 2);
            acc[0] = s_lo;
            acc[2] = s_hi;
        }
#pragma unroll
        for (int j = 0; j < kV; ++j) {      // (tile j / 4 of the activations: columns 8 (j / 4) + 2 t, + 1)
            uint32_t col = 8 * (j >> 2) + 2 * t + (j & 1), row = g + 8 * ((j >> 1) & 1);
            if (col < A.batch) mine[col * 16 + row] = acc[j];
        }
#pragma unroll
        for (int j = 0; j < kV; ++j) acc[j] = 0.f;
        __syncwarp();
        float v[kV];
        if (alone) {
#pragma unroll
            for (int i = 0; i < kV; ++i) v[i] = lane + 32 * i < vals ? mine[lane + 32 * i] : 0.f;
            __syncwarp();
            finish_cta_sum(rg, v);
            return;
        }
        // which warps of this CTA hold a piece of this row group (lane l answers for warp l)
        const uint32_t wb = warp_beg(lane), we = warp_beg(lane + 1);
        const bool holds = lane < nw && wb < we && wb < g_hi && we > g_lo;
        const uint32_t mask = __ballot_sync(0xFFFFFFFFu, holds);
        const uint32_t w_first = __ffs(mask) - 1, n_hold = __popc(mask);
        const uint32_t slot_of_lane = (uint32_t)rg == wb / KC ? 0u : 1u;
        uint32_t last = 0;
        if (lane == 0) {
            __threadfence_block();
            last = atomicAdd(&s_arrive[w_first], 1u) == n_hold - 1 ? 1u : 0u;
            if (last) __threadfence_block();
        }
        if (!__shfl_sync(0xFFFFFFFFu, last, 0)) return;
#pragma unroll
        for (int i = 0; i < kV; ++i) v[i] = 0.f;
        for (uint32_t m = mask; m; m &= m - 1) {              // pieces in warp order
            const uint32_t w = __ffs(m) - 1;
            const float *piece = part_val + (size_t)(w * 2 + __shfl_sync(0xFFFFFFFFu, slot_of_lane, w)) * vals;
#pragma unroll
            for (int i = 0; i < kV; ++i)
                if (lane + 32 * i < vals) v[i] += piece[lane + 32 * i];
        }
        finish_cta_sum(rg, v);
    };

    if (c_beg < c_end) {
        uint32_t rg = c_beg / KC, kc = c_beg - rg * KC;               // tracked incrementally from here on
        // The activation pointer runs on from chunk to chunk: the columns of a row group's chunks follow each other.
        const uint16_t *xq = k.x + (MODE == 1 ? (uint64_t)min(g, A.batch - 1) * k.cols + kc * k.chunk_cols + t * 8u : 0);
        // (second tile of activations, vectors 8 .. 15: lane g's vector 8 + g lies this many elements further on)
        const uint64_t x_tile2 = NT == 2 ? (uint64_t)(min(g + 8u, A.batch - 1) - min(g, A.batch - 1)) * k.cols : 0;
        // this chunk's slot (the lane's column of it), its barrier and its note, toggled by XOR from chunk to chunk; parity
        // of the barrier's next completion (each of the two "full" barriers completes every second chunk)
        // (With two tiles of activations, where registers are shortest, the five are worked out from the chunk's number at
        // every chunk instead of being carried along: 4 % faster there, 3 % slower in the other kernels.)
        constexpr bool kDerive = NT == 2;
        uint32_t slot_cur = (SLOTS == 2 ? slot_addr(plan, warp, 0, A.slot_bytes) : slot_addr_single(plan, warp, A.slot_bytes)) + (lane << 2);
        uint32_t bar_cur = bar_w, par = 0, which = 0;
        const uint32_t slot_tog = SLOTS == 2 ? slot_cur ^ (slot_cur + A.slot_bytes) : 0u;   // (one slot: every chunk lands in the same place)
        uint32_t note_cur = smem_u32(&notes[warp * 2]);
        const uint32_t slot0 = slot_cur, note0 = note_cur;      // (used where the five are worked out anew)

#pragma unroll 1
        for (uint32_t c = c_beg; c < c_end; ++c) {
            const uint32_t nkb = kc + 1 == KC ? nkb_tail : nkb_full;
            if (kDerive) {
                const uint32_t ci = c - c_beg;
                which = ci & 1u;
                par = (ci >> 1) & 1u;
                bar_cur = bar_w + 8u * which;
                note_cur = note0 + 8u * which;
                slot_cur = slot0 + (SLOTS == 2 ? which * A.slot_bytes : 0u);
            }
            if (MODE == 1 && (int)rg != cur_rg) {
                flush(cur_rg, c_beg, c);  // the previous row group ended with chunk c - 1
                cur_rg = (int)rg;
            }

            // wait, with a limit, for the coded part; the outcome is made uniform across the warp
            if (!failed) {
                uint32_t spins = 0;
                bool done = mbar_try_wait(bar_cur, par);
                while (!__all_sync(0xFFFFFFFFu, done)) {
                    if (++spins > kWaitLimit) {
                        failed = true;      // this chunk and the warp's later ones add nothing; the row groups are still closed
                        if (lane == 0) {
                            if (A.err) atomicExch(A.err, -1);
                            *(volatile uint32_t *)&s_stop = 1;
                        }
                        break;
                    }
                    done = mbar_try_wait(bar_cur, par);
                }
            }
            if (!waited_prior) {
                pdl_wait_prior_grid();   // from here on this warp reads x and writes results: the previous kernel must be done
                waited_prior = true;
            }
            uint32_t r0, r1;            // the feeder's note: the record's first and last offset
            asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(note_cur));
            if (failed || r0 == kBadRecord) {  // record offsets out of range: report, produce nothing for this chunk, touch no memory
                if (!failed && A.err && lane == 0) atomicExch(A.err, (int32_t)min(c + 1, 0x7FFFFFFFu));
                primed = false;
                if (MODE == 1) xq += nkb * 32u;
            } else {
                if (!primed) {
                    raw_p = payload + ((uint64_t)r0 << 7) + lane * kRawLane;
                    raw_a = load_raw(raw_p);
                }
                // the record behind this one is the next chunk's: its first raw block is fetched from inside this chunk's last
                // block (the address lies inside the blob whatever that record's offsets turn out to be)
                const bool has_next = c + 1 < c_end;
                const uint32_t coded_bytes = (r1 - r0 - raw_units(nkb)) << 7;
                // from the end of the record's last raw block to the next record: the coded part and, in FP16 records with an
                // odd number of blocks, the 64 bytes that pad the raw part to a whole unit
                const uint32_t to_next = FMT ? ((r1 - r0) << 7) - nkb * kRawBlock : coded_bytes;
                LaneStream sa, sb;
                stream_open(sa, slot_cur, SKIP ? 7u : SKIP16 ? 6u : 0u);
                stream_open(sb, slot_cur + 128u, SKIP ? 7u : SKIP16 ? 6u : 0u);
                const uint32_t col0 = kc * k.chunk_cols + t * 8u;
                // (activations: lanes of unused output columns repeat the last vector; cols is a multiple of 32
                // here, so every block of the chunk lies inside the row and xq ends the chunk where the next begins)
                uint16_t *out0 = MODE == 0 ? k.out + ((uint64_t)rg * 16 + g) * k.cols + col0 : nullptr;
                const uint32_t last = nkb - 1;

                // one block: start the fetch of the next block's raw bytes into `nxt`, decode with `cur`
                // (may_be_last = false: the caller knows that another block of this chunk follows)
                // Every block asks L2 for the 16 bytes per lane that lie four blocks further on in the record stream (the
                // loads that bring raw bytes to registers run one block ahead of the decoder, too short for a miss in
                // DRAM).  In a record's first half that is the raw part of its second half; in the second half it is the
                // coded part and, at its end, the start of the next record.  The request ends at most 2 KB behind the
                // record it is issued in: inside the blob, whose format keeps 4 KB of zero bytes behind the payload for this.
                // (products of BF16 blobs only: the decode-only kernel has no register to spare for it, and an FP16 record's
                // raw part is a sixteenth of its bytes)
                constexpr bool kPrefetchRaw = false;
                auto block = [&](uint32_t kb, const uint4 &cur, uint4 &nxt, auto may_be_last) {
                    raw_p += kRawBlock;
                    if (kPrefetchRaw) asm volatile("prefetch.global.L2 [%0];" ::"l"(raw_p + 3u * kRawBlock));
                    if (decltype(may_be_last)::value) {
                        if (kb == last) raw_p += to_next;           // the next record's first block
                        if (kb != last || has_next) nxt = load_raw(raw_p);
                    } else {
                        nxt = load_raw(raw_p);
                    }
                    uint4 xv;
                    if (MODE == 1) {
                        if (NT <= 1) xv = __ldg((const uint4 *)xq);   // (two tiles: both are fetched behind the decoder, registers are short)
                        xq += 32;
                    }

                    uint32_t a[8];
                    if (FMT) decode_block_fp16<LONG, SKIP16>(sa, sb, lut_lane, cur.x, a, full_base, full_mask);
                    else decode_block<R, SKIP, LONG>(sa, sb, kIdxMask, lut_lane, cur, a, full_base, full_mask);

                    if (MODE == 1) {
                        uint4 xw;
                        if (NT == 2) {
                            xv = __ldg((const uint4 *)(xq - 32));
                            xw = __ldg((const uint4 *)(xq - 32 + x_tile2));
                        }
                        float (&acc0)[4] = *reinterpret_cast<float (*)[4]>(&acc[0]);
                        if (NT == 0) {
                            // the lane's weights a[i] (row g) and a[4 + i] (row g + 8) stand in columns 2 i, 2 i + 1 of its
                            // eight, and xv holds the vector's entries of the same columns
                            const uint32_t xs[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                if (FMT) {
                                    fma2_f16(acc[0], a[i], xs[i]);
                                    fma2_f16(acc[2], a[4 + i], xs[i]);
                                } else {
                                    fma2_bf16(acc[0], a[i], xs[i]);
                                    fma2_bf16(acc[2], a[4 + i], xs[i]);
                                }
                            }
                        } else if (FMT) {
                            mma_f16_16816(acc0, a[0], a[4], a[1], a[5], xv.x, xv.y);
                            mma_f16_16816(acc0, a[2], a[6], a[3], a[7], xv.z, xv.w);
                        } else {
                            mma_bf16_16816(acc0, a[0], a[4], a[1], a[5], xv.x, xv.y);
                            mma_bf16_16816(acc0, a[2], a[6], a[3], a[7], xv.z, xv.w);
                        }
                        if (NT == 2) {
                            float (&acc1)[4] = *reinterpret_cast<float (*)[4]>(&acc[NT == 2 ? 4 : 0]);
                            if (FMT) {
                                mma_f16_16816(acc1, a[0], a[4], a[1], a[5], xw.x, xw.y);
                                mma_f16_16816(acc1, a[2], a[6], a[3], a[7], xw.z, xw.w);
                            } else {
                                mma_bf16_16816(acc1, a[0], a[4], a[1], a[5], xw.x, xw.y);
                                mma_bf16_16816(acc1, a[2], a[6], a[3], a[7], xw.z, xw.w);
                            }
                        }
                    } else {
                        const uint32_t col = col0 + kb * 32u;
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if ((uint64_t)rg * 16 + g + 8 * h >= k.rows || col >= (uint32_t)k.cols) continue;
                            uint16_t *dst = out0 + (uint64_t)(8 * h) * k.cols + kb * 32u;
                            if (k.cols % 8 == 0) {
                                *(uint4 *)dst = make_uint4(a[4 * h], a[4 * h + 1], a[4 * h + 2], a[4 * h + 3]);
                            } else {
#pragma unroll
                                for (int i = 0; i < 8; ++i)
                                    if (col + i < (uint32_t)k.cols) dst[i] = (uint16_t)(a[4 * h + (i >> 1)] >> (16 * (i & 1)));
                            }
                        }
                    }
                };
                constexpr std::integral_constant<bool, false> inner{};
                constexpr std::integral_constant<bool, true> maybe_last{};
                uint32_t kb = 0;
#pragma unroll 1
                for (; kb + 4 <= nkb; kb += 4) {                    // the usual case: groups of four blocks
                    block(kb, raw_a, raw_b, inner);
                    block(kb + 1, raw_b, raw_a, inner);
                    block(kb + 2, raw_a, raw_b, inner);
                    block(kb + 3, raw_b, raw_a, maybe_last);
                }
#pragma unroll 1
                for (; kb < nkb; kb += 2) {
                    block(kb, raw_a, raw_b, maybe_last);
                    if (kb + 1 < nkb) block(kb + 1, raw_b, raw_a, maybe_last);
                }
                if (nkb & 1u) raw_a = raw_b;     // the next chunk's first block always starts in raw_a
                primed = has_next;
                // A sequence of a sound record ends inside the record's W rows, so its next-row pointer stands at most two
                // rows behind them.  Bits that made the decoder run further (a damaged coded part) are reported; what was
                // decoded from them is wrong, but every read stayed inside shared memory (one row per refill check at most).
                const uint32_t row_limit = slot_cur + 512u + coded_bytes;
                if (__any_sync(0xFFFFFFFFu, sa.nxt > row_limit || sb.nxt > row_limit + 128u)) {
                    if (A.err && lane == 0) atomicExch(A.err, (int32_t)(kErrOverrun | min(c + 1, kErrOverrun - 1u)));
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_cur + 16);                 // the slot goes back to the feeder
            if (!kDerive) {
                par ^= which;                                     // 0, 0, 1, 1, 0, 0, ...
                which ^= 1u;
                if (SLOTS == 2) slot_cur ^= slot_tog;
                bar_cur ^= 8u;
                note_cur ^= 8u;
            }
            kc = kc + 1 == KC ? 0u : kc + 1;
            if (kc == 0) {                                        // the next chunk starts the next row group: back to column 0
                ++rg;
                if (MODE == 1) xq -= k.cols;
            }
        }
        if (MODE == 1) flush(cur_rg, c_beg, c_end);
    }
}

// ------------------------------------------------------------------------------ plain bf16 GEMV

// The dense product the compressed path competes with: y = W x for uncompressed bf16 matrices, written as a streaming
// kernel so that it is a fair opponent.  One launch takes a list of matrices (the same launch groups as the compressed
// path).  A warp takes one row at a time and walks it 4 KB per step: eight independent 16-byte loads per lane are in
// flight before the first is used (32 warps per SM: 128 KB per SM on its way, several times what the memory latency
// times an SM's share of the bandwidth asks for); x comes from L1; products in fp32, shuffle reduction.  Rows are dealt
// round-robin to the warps of the grid, so every SM keeps loads in flight until the launch ends.
__device__ __forceinline__ void fma_bf16x8(float &lo, float &hi, const uint4 &w, const uint4 &x) {
    const uint32_t wv[4] = {w.x, w.y, w.z, w.w}, xv[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        lo = fmaf(__uint_as_float(wv[j] << 16), __uint_as_float(xv[j] << 16), lo);
        hi = fmaf(__uint_as_float(wv[j] & 0xFFFF0000u), __uint_as_float(xv[j] & 0xFFFF0000u), hi);
    }
}

__global__ void __launch_bounds__(256, 4) plain_gemv_kernel(const __grid_constant__ PlainArgs A) {
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    // launched like the compressed path: the next launch may start early, and this one asks for its first weights before
    // the launch in front of it has finished; x is read only after that
    pdl_launch_dependents();
    bool waited_prior = false;
    uint32_t mi = 0;
    for (uint32_t u = warp; u < A.total_rows; u += nwarps) {
        while (mi + 1 < A.n_mats && u >= A.m[mi + 1].row_first) ++mi;
        const PlainMat &m = A.m[mi];
        const uint64_t r = u - m.row_first;
        const uint32_t nv = (uint32_t)(m.cols >> 3);                       // 16-byte pieces of a row
        const uint4 *wr = (const uint4 *)(m.w + r * m.cols), *xr = (const uint4 *)m.x;
        float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;
        for (uint32_t i = lane; i < nv; i += 256) {                        // eight pieces per lane and step
            uint4 p[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) p[j] = i + 32 * j < nv ? ldg_stream16(wr + i + 32 * j) : make_uint4(0, 0, 0, 0);
            if (!waited_prior) {
                pdl_wait_prior_grid();
                waited_prior = true;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint4 xv = i + 32 * j < nv ? __ldg(xr + i + 32 * j) : make_uint4(0, 0, 0, 0);
                if (j & 1) fma_bf16x8(b0, b1, p[j], xv);
                else fma_bf16x8(a0, a1, p[j], xv);
            }
        }
        float sum = (a0 + a1) + (b0 + b1);
#pragma unroll
        for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
        if (lane == 0) m.y[r] = sum;
    }
}

// ------------------------------------------------------------------------------ small copies by a kernel

// Copies 16-byte pieces between device-accessible buffers (device memory, or pinned host memory that the device can
// address).  For the tens of kilobytes of activations and results of a decode step this is cheaper than a DMA copy:
// inside a CUDA graph a copy node between kernel nodes costs about 10 microseconds, this kernel about 3.
__global__ void __launch_bounds__(512) stage_copy_kernel(uint4 *__restrict__ dst, const uint4 *__restrict__ src, uint64_t n16) {
    pdl_launch_dependents();   // a product kernel behind this copy may do its set-up meanwhile: it waits for the copy before it reads x
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (uint64_t)gridDim.x * blockDim.x) dst[i] = src[i];
}

cudaError_t launch_stage_copy(void *dst, const void *src, uint64_t bytes, uint32_t sms, cudaStream_t stream) {
    const uint64_t n16 = bytes / 16;
    uint64_t grid = (n16 + 511) / 512;
    if (grid > sms) grid = sms;
    if (grid == 0) return cudaSuccess;
    stage_copy_kernel<<<(uint32_t)grid, 512, 0, stream>>>((uint4 *)dst, (const uint4 *)src, n16);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------ launchers

template <int MODE, int LB, int THREADS, int FMT, int NT = 1, int SLOTS = 2>
static cudaError_t launch_one(const KernelArgs &k, uint32_t grid, cudaStream_t stream) {
    auto fn = huff_kernel<MODE, LB, THREADS, FMT, NT, SLOTS>;
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
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = k.dyn_smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set-up overlaps the previous kernel's tail
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fn, k);
}

// One or two slots per decoder warp (the host decides; kernels.h says for which kernels single slots exist).
template <int MODE, int LB, int FMT, int NT = 1>
static cudaError_t launch_slots(const KernelArgs &k, uint32_t grid, cudaStream_t stream) {
    if (k.slots == 1) return launch_one<MODE, LB, kThreads, FMT, NT, 1>(k, grid, stream);
    return launch_one<MODE, LB, kThreads, FMT, NT, 2>(k, grid, stream);
}

cudaError_t launch_decode(const KernelArgs &k, uint32_t grid, cudaStream_t stream) {
    if (k.fmt && k.lut_bits == 7) return launch_slots<0, 7, 1>(k, grid, stream);
    if (k.fmt && k.lut_bits == 8 && k.fp16_flat) return launch_slots<0, 8, 2>(k, grid, stream);
    if (k.fmt) return k.lut_bits > 8 ? launch_slots<0, 12, 1>(k, grid, stream) : launch_slots<0, 8, 1>(k, grid, stream);
    if (k.lut_bits > 9) return launch_one<0, 12, kThreads, 0>(k, grid, stream);
    return k.lut_bits == 8 ? launch_slots<0, 8, 0>(k, grid, stream) : launch_one<0, 9, kThreads, 0>(k, grid, stream);
}

cudaError_t launch_gemm(const KernelArgs &k, uint32_t grid, cudaStream_t stream) {
    if (k.batch == 1 && k.fmt) {                  // one vector: multiply-adds on the FMA pipe
        if (k.lut_bits == 7) return launch_slots<1, 7, 1, 0>(k, grid, stream);
        if (k.lut_bits == 8 && k.fp16_flat) return launch_slots<1, 8, 2, 0>(k, grid, stream);
        return k.lut_bits > 8 ? launch_slots<1, 12, 1, 0>(k, grid, stream) : launch_slots<1, 8, 1, 0>(k, grid, stream);
    }
    if (k.batch == 1) {
        if (k.lut_bits > 9) return launch_one<1, 12, kThreads, 0, 0>(k, grid, stream);
        return k.lut_bits == 8 ? launch_slots<1, 8, 0, 0>(k, grid, stream) : launch_one<1, 9, kThreads, 0, 0>(k, grid, stream);
    }
    if (k.batch > 8) return launch_slots<1, 8, 0, 2>(k, grid, stream);   // (the entry point sends only BF16 blobs of 8-bit tables here)
    if (k.fmt && k.lut_bits == 7) return launch_slots<1, 7, 1>(k, grid, stream);
    if (k.fmt && k.lut_bits == 8 && k.fp16_flat) return launch_slots<1, 8, 2>(k, grid, stream);
    if (k.fmt) return k.lut_bits > 8 ? launch_slots<1, 12, 1>(k, grid, stream) : launch_slots<1, 8, 1>(k, grid, stream);
    if (k.lut_bits > 9) return launch_one<1, 12, kThreads, 0>(k, grid, stream);
    return k.lut_bits == 8 ? launch_slots<1, 8, 0>(k, grid, stream) : launch_one<1, 9, kThreads, 0>(k, grid, stream);
}

cudaError_t launch_plain_gemv(const PlainArgs &a, uint32_t sms, cudaStream_t stream) {
    const uint64_t blocks = ((uint64_t)a.total_rows + 7) / 8;               // 8 warps per CTA, a row per warp and turn
    const uint32_t grid = (uint32_t)(blocks < (uint64_t)sms * 4 ? blocks : (uint64_t)sms * 4);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, plain_gemv_kernel, a);
}

}  // namespace huffllm
