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
//   * the coded part of a record is brought into shared memory by one bulk-async copy per chunk
//     (no multicast), completion on an mbarrier; two slots per warp, so the next chunk is in
//     flight while this one is decoded
//   * the raw sign/mantissa bytes go straight from global memory to registers, 16 bytes per lane
//     per block of 32 columns, one block ahead
//   * the LUT is replicated per lane in shared memory (entry i of lane l at word 32 i + l), so a
//     warp-wide lookup never has a bank conflict; it is placed on an address boundary that lets
//     the lookup address be formed with a single logic operation
//   * a lane's 16 weights of a block are exactly its share of two m16n8k16 tensor-core operand
//     tiles, so the product needs no shuffles: decode, pack to bf16x2, mma
//   * partial sums of a row group that is split over warps or CTAs are combined in a fixed order
//     (shared memory inside a CTA, a scratch buffer plus a last-CTA pass across CTAs)
#include <cuda_runtime.h>
#include <cstdint>

#include "kernels.h"

namespace huffllm {

// ------------------------------------------------------------------------------ PTX helpers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t lds_stream(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
// LUT reads: the table is constant once built, so the compiler may schedule these freely.
__device__ __forceinline__ uint32_t lds_lut(uint32_t addr) {
    uint32_t v;
    asm("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bulk asynchronous copy global -> this CTA's shared memory, completion counted on `bar`.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint4 ldg_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Arrival counter bump that publishes this warp's earlier stores and acquires the other arrivals' stores.
__device__ __forceinline__ uint32_t arrive_acq_rel(unsigned int *counter) {
    uint32_t old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(counter) : "memory");
    return old;
}
// Programmatic dependent launch: let the next kernel in the stream be scheduled early / wait for the previous one.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_prior_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ------------------------------------------------------------------------------ lane decoder

// State of the decoder of one bit sequence.  (hi:lo) holds 64 stream bits; the current codeword starts
// at bit pos + 7 of that window (the 7 bits in front are the lag that makes the table address fall out
// of a single AND/OR); nxt is the shared-memory address of the sequence's next 32-bit word.  Words of
// one sequence are 256 bytes apart (a row of the record holds one word of each of the 64 sequences).
struct LaneStream {
    uint32_t lo, hi, pos, nxt;
};

__device__ __forceinline__ void stream_open(LaneStream &s, uint32_t lane_word0) {
    s.lo = lds_stream(lane_word0);
    s.hi = lds_stream(lane_word0 + 256);
    s.nxt = lane_word0 + 512;
    s.pos = 0;
}

// One decoder step: returns the table entry (length << 16 | exponent << 7) and advances the start pointer.
// The window is shifted as a 64-bit value, so the pointer may run past bit 32 between two refill
// checks.  The table address is (window & index mask) | (table base + 4 * lane): one logic operation,
// because the table sits on a boundary above the index bits.  Only byte 2 of the entry (the length)
// is added to the pointer: dp4a with that byte selected does it in one instruction off the ALU pipe.
__device__ __forceinline__ uint32_t stream_step(LaneStream &s, uint32_t idx_mask, uint32_t lut_lane) {
    uint64_t win = ((uint64_t)s.hi << 32) | s.lo;
    uint32_t t = (uint32_t)(win >> s.pos), addr;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(addr) : "r"(t), "r"(idx_mask), "r"(lut_lane));
    uint32_t e = lds_lut(addr);
    s.pos = __dp4a(e, 0x00010000u, s.pos);
    return e;
}

// Refill: once 32 bits have been consumed, slide the window by one word.  Written with predicated
// instructions so that lanes which need a word and lanes which do not stay converged.
// The two additions are written as multiply-adds by a register holding 1 so that they run on the FMA pipe:
// the 16-lane integer ALU pipe is the busiest unit of this kernel.
__device__ __forceinline__ void stream_refill(LaneStream &s, uint32_t one) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ge.u32 p, %2, 32;\n\t"
        "@p mov.u32 %0, %1;\n\t"
        "@p ld.shared.u32 %1, [%3];\n\t"
        "@p mad.lo.u32 %3, %4, 256, %3;\n\t"
        "@p mad.lo.u32 %2, %4, 0xFFFFFFE0, %2;\n\t}"
        : "+r"(s.lo), "+r"(s.hi), "+r"(s.pos), "+r"(s.nxt)
        : "r"(one));
}

// Two table entries + two raw bytes -> two bf16 weights packed in one register.
// SEL picks raw bytes (i, i+1) of `raw` as (byte, sign-replicated byte) pairs.  The exponent of the
// even weight is already in place (bits 7..14); the odd entry times 65536 puts its exponent at bits
// 23..30 and pushes its length out of the word, so one multiply-add (FMA pipe) merges the two.
template <uint32_t SEL>
__device__ __forceinline__ uint32_t pack_pair(uint32_t e_even, uint32_t e_odd, uint32_t raw) {
    uint32_t sm = prmt(raw, 0u, SEL);   // [sign1*0xFF, raw1, sign0*0xFF, raw0]
    uint32_t ex;
    asm("mad.lo.u32 %0, %1, 65536, %2;" : "=r"(ex) : "r"(e_odd), "r"(e_even));
    uint32_t w;   // sign and mantissa bits from sm, exponent bits from ex
    asm("lop3.b32 %0, %1, %2, 0x807F807F, 0xE4;" : "=r"(w) : "r"(sm), "r"(ex));
    return w;
}

// Decode one block (16 weights of this lane) into 8 packed registers:
// a[0..3] = row g, columns (0,1) (2,3) (4,5) (6,7);  a[4..7] = row g+8, same columns.
// The lane's two sequences are stepped alternately.  Each window is checked for a refill before every
// R-th step: after a check at least 26 bits are valid in front of the start pointer, enough for R
// codewords of at most 26/R bits.
template <int R>
__device__ __forceinline__ void decode_block(LaneStream &sa, LaneStream &sb, uint32_t idx_mask, uint32_t lut_lane, uint32_t one,
                                             const uint4 &raw, uint32_t (&a)[8]) {
    uint32_t e[16];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (i % R == 0) {
            stream_refill(sa, one);
            stream_refill(sb, one);
        }
        e[i] = stream_step(sa, idx_mask, lut_lane);
        e[8 + i] = stream_step(sb, idx_mask, lut_lane);
    }
    a[0] = pack_pair<0x9180u>(e[0], e[1], raw.x);
    a[1] = pack_pair<0xB3A2u>(e[2], e[3], raw.x);
    a[2] = pack_pair<0x9180u>(e[4], e[5], raw.y);
    a[3] = pack_pair<0xB3A2u>(e[6], e[7], raw.y);
    a[4] = pack_pair<0x9180u>(e[8], e[9], raw.z);
    a[5] = pack_pair<0xB3A2u>(e[10], e[11], raw.z);
    a[6] = pack_pair<0x9180u>(e[12], e[13], raw.w);
    a[7] = pack_pair<0xB3A2u>(e[14], e[15], raw.w);
}

// ------------------------------------------------------------------------------ shared memory plan

// Dynamic shared memory, laid out at run time from the window's real start address:
//   [base, lut)            slot pairs (as many as fit)
//   [lut, lut + LUTSZ)     per-lane LUT; lut = base rounded up to a multiple of LUTSZ, so that the
//                          index bits of a lookup address never overlap the table's base bits
//   [lut + LUTSZ, ...)     more slot pairs, then a guard area no valid stream ever reads
//   [end - part_bytes, end) the CTA's table of partial sums (fused product only)
struct SmemPlan {
    uint32_t lut;    // shared address of the table
    uint32_t warps;  // warps that own a slot pair
    uint32_t slotA;  // first slot pair before the table
    uint32_t nA;     // slot pairs before the table
    uint32_t slotB;  // first slot pair after it
};

__device__ __forceinline__ SmemPlan plan_smem(uint32_t base, const KernelArgs &k, uint32_t max_warps) {   // k: launch-wide fields only
    SmemPlan p;
    const uint32_t lut_bytes = 128u << k.lut_bits;
    uint32_t a0 = (base + 127u) & ~127u;
    p.lut = (base + lut_bytes - 1) / lut_bytes * lut_bytes;
    p.slotA = a0;
    p.nA = p.lut > a0 ? (p.lut - a0) / (2 * k.slot_bytes) : 0;  // a stream that overruns here reads the table: harmless
    p.slotB = p.lut + lut_bytes;
    uint32_t end = base + k.dyn_smem_bytes - k.part_bytes;
    uint32_t roomB = end > p.slotB + k.guard_bytes ? end - p.slotB - k.guard_bytes : 0;
    p.warps = min(max_warps, p.nA + roomB / (2 * k.slot_bytes));
    return p;
}

__device__ __forceinline__ uint32_t slot_addr(const SmemPlan &p, uint32_t warp, uint32_t which, uint32_t slot_bytes) {
    uint32_t pair = warp < p.nA ? p.slotA + warp * 2 * slot_bytes : p.slotB + (warp - p.nA) * 2 * slot_bytes;
    return pair + which * slot_bytes;
}

constexpr int kMaxWarps = 32;
// Experiment build only (-DHUFFLLM_TIMING): every warp writes nanosecond stamps of its phases into the
// buffer passed as the error flag, [cta][warp][8].
#ifdef HUFFLLM_TIMING
__device__ __forceinline__ unsigned long long gtime() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define STAMP(i) do { if (lane == 0) ((unsigned long long *)A.err)[((size_t)blockIdx.x * 32 + warp) * 8 + (i)] = gtime(); } while (0)
#define BLOCKSTAMP(n, phase) do { if (lane == 0 && blockIdx.x == 3 && (n) < 64) ((unsigned long long *)A.err)[148 * 32 * 8 + (warp * 64 + (n)) * 4 + (phase)] = clock64(); } while (0)
#else
#define STAMP(i) do {} while (0)
#define BLOCKSTAMP(n, phase) do {} while (0)
#endif
#ifndef HUFFLLM_THREADS
#define HUFFLLM_THREADS 1024
#endif
constexpr int kThreads = HUFFLLM_THREADS;   // threads per CTA of the decode kernels (one CTA per SM)
constexpr uint32_t kWaitLimit = 1u << 22;

// ------------------------------------------------------------------------------ the fused kernel

// MODE 0: write the decoded weights.  MODE 1: y = W x for up to 8 activation vectors.
// LB = table index bits (the blobs' lut_bits): 8 or 9.
//
// One launch works through a LIST of matrices (A.n_mats, usually the matrices of one decoder layer that
// may run together).  The chunks of all matrices form one long list that is cut into equal pieces, one
// per CTA, so almost every CTA lies inside a single matrix and builds a single table; the few CTAs whose
// piece crosses from one matrix into the next rebuild the table once, behind a CTA-wide barrier.
template <int MODE, int LB, int THREADS>
__global__ void __launch_bounds__(THREADS, 1) huff_kernel(const __grid_constant__ KernelArgs A) {
    constexpr int R = LB == 8 ? 3 : 2;                       // decoder steps between two refill checks
    constexpr uint32_t kIdxMask = ((1u << LB) - 1u) << 7;
    extern __shared__ __align__(128) uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t bars[kMaxWarps * 2];
    __shared__ uint32_t s_arrive[kMaxWarps];   // arrival counters of row groups shared by several warps

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps_launched = blockDim.x >> 5;
    STAMP(0);
    pdl_launch_dependents();   // the next kernel's set-up may overlap this kernel's tail
    const uint32_t smem_base = smem_u32(dyn_smem);
    const SmemPlan plan = plan_smem(smem_base, A, nwarps_launched);
    const uint32_t nw = plan.warps;
    const uint32_t vals = 16 * A.batch;
    float *part_val = (float *)(dyn_smem + A.dyn_smem_bytes - A.part_bytes);  // [2 * warps][16 * batch]

    uint32_t lut_lane = plan.lut | (lane << 2);
    asm volatile("mov.u32 %0, %0;" : "+r"(lut_lane));  // keep it in a register: it is an operand of every lookup
    uint32_t one = 1;
    asm volatile("mov.u32 %0, %0;" : "+r"(one));       // a 1 the compiler cannot see through (see stream_refill)
    const uint32_t g = lane >> 2, t = lane & 3;
    const uint32_t bar0 = smem_u32(&bars[warp * 2]);
    const uint32_t slot0 = slot_addr(plan, warp, 0, A.slot_bytes);
    if (lane == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    uint32_t phase = 0;            // bit s = parity of the next completion of this warp's barrier s
    bool waited_prior = false, failed = false;

    // this CTA's piece of the list of all chunks
    const uint32_t G = gridDim.x, TT = A.total_chunks;
    auto cta_cut = [&](uint32_t c) -> uint32_t { return (uint32_t)((uint64_t)TT * c / G); };
    const uint32_t piece_beg = cta_cut(blockIdx.x), piece_end = cta_cut(blockIdx.x + 1);
    bool first_segment = true;

#pragma unroll 1
    for (uint32_t mi = 0; mi < A.n_mats; ++mi) {
        const MatArgs &k = A.m[mi];
        if (piece_end <= k.chunk_base || piece_beg >= k.chunk_base + k.n_chunks) continue;
        // ---- the part of matrix mi that this CTA works on, in the matrix's own chunk numbers
        const uint32_t cta_beg = max(piece_beg, k.chunk_base) - k.chunk_base;
        const uint32_t cta_end = min(piece_end, k.chunk_base + k.n_chunks) - k.chunk_base;
        const uint32_t KC = k.col_chunks;
        uint32_t c_beg = cta_beg, c_end = cta_beg;
        if (warp < nw) {
            c_beg = cta_beg + (cta_end - cta_beg) * warp / nw;
            c_end = cta_beg + (cta_end - cta_beg) * (warp + 1) / nw;
        }
        const uint32_t *index = (const uint32_t *)(k.blob + k.off_index);
        const uint8_t *payload = k.blob + k.off_payload;

        // blocks of 32 columns in column chunk kc
        auto blocks_of = [&](uint32_t kc) -> uint32_t {
            uint32_t left = (uint32_t)k.cols - kc * k.chunk_cols;
            return (min(left, k.chunk_cols) + 31u) >> 5;
        };
        // a record is usable if it lies inside the payload and its coded part fits a slot
        auto record_ok = [&](uint32_t r0, uint32_t r1, uint32_t nkb) -> bool {
            return r1 > r0 && r1 <= k.payload_units && (r1 - r0) * 128u > nkb * 512u &&
                   (r1 - r0) * 128u - nkb * 512u + 256u <= A.slot_bytes;
        };
        // lane 0: start the bulk copy of a chunk's coded part into slot `which`
        auto issue = [&](uint32_t c, uint32_t which) {
            uint32_t nkb = blocks_of(c % KC), r0 = __ldg(index + c), r1 = __ldg(index + c + 1);
            uint32_t bar = bar0 + which * 8;
            if (record_ok(r0, r1, nkb)) {
                uint32_t bytes = (r1 - r0) * 128u - nkb * 512u;
                mbar_expect_tx(bar, bytes);
                bulk_g2s(slot0 + which * A.slot_bytes, payload + (uint64_t)r0 * 128u + nkb * 512u, bytes, bar);
            } else {
                mbar_expect_tx(bar, 0);  // completes the phase with nothing to wait for; the chunk is skipped below
            }
        };

        // ---- set-up of a segment.  The table loads are started first, then every warp starts its first
        // copies, then the table is written to shared memory: the cold misses on the table, on the record
        // index and on the first records overlap instead of following each other.
        constexpr int kLutLoads = ((32 << LB) + THREADS - 1) / THREADS;
        uint32_t lut_v[kLutLoads];
        {
            const uint32_t *lut_g = (const uint32_t *)(k.blob + k.off_lut);
#pragma unroll
            for (int i = 0; i < kLutLoads; ++i) {
                uint32_t j = tid + i * THREADS;
                lut_v[i] = j < (32u << LB) ? __ldg(lut_g + (j >> 5)) : 0u;
            }
        }
        if (lane == 0 && c_beg < c_end) {
            issue(c_beg, 0);
            if (c_beg + 1 < c_end) issue(c_beg + 1, 1);
        }
        if (!first_segment) __syncthreads();      // everybody is done with the previous matrix's table and counters
        first_segment = false;
        {
            uint32_t *lut_s = (uint32_t *)(dyn_smem + (plan.lut - smem_base));
#pragma unroll
            for (int i = 0; i < kLutLoads; ++i) {
                uint32_t j = tid + i * THREADS;
                if (j < (32u << LB)) lut_s[j] = lut_v[i];
            }
            if (tid < kMaxWarps) s_arrive[tid] = 0;
        }
        STAMP(1);
        __syncthreads();
        STAMP(2);

        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        int cur_rg = -1;

        // ---- reduction of a finished row group, without any CTA-wide barrier.
        // A row group whose chunks this warp decoded alone goes straight to y.  Otherwise the warp parks its
        // piece in shared memory and bumps an arrival counter (indexed by the first warp that holds a piece);
        // the warp that arrives last adds the pieces in warp order.  If other CTAs hold pieces too, the CTA's
        // sum goes to the scratch buffer and the same game is played across CTAs with a counter in global
        // memory.  Sums are always taken in the same order, and nobody waits for anybody.
        const uint32_t cta_len = cta_end - cta_beg;
        auto warp_beg = [&](uint32_t w) -> uint32_t { return cta_beg + cta_len * w / nw; };
        auto cta_of_chunk = [&](uint32_t ch) -> uint32_t {     // ch = chunk number inside this matrix
            const uint32_t gch = ch + k.chunk_base;
            uint32_t c = (uint32_t)((uint64_t)gch * G / TT);
            while (c + 1 < G && cta_cut(c + 1) <= gch) ++c;
            while (c > 0 && cta_cut(c) > gch) --c;
            return c;
        };
        // first chunk of this matrix that CTA c works on
        auto cta_first_chunk = [&](uint32_t c) -> uint32_t { return max(cta_cut(c), k.chunk_base) - k.chunk_base; };
        // lanes 0..vals-1 (looping if vals > 32) hold or produce the value of output o = column * 16 + row
        auto finish_cta_sum = [&](int rg, float (&v)[4]) {       // v[i] = value of output o = lane + 32 i
            const uint32_t g_lo = (uint32_t)rg * KC, g_hi = g_lo + KC;
            if (cta_beg <= g_lo && cta_end >= g_hi) {             // the CTA held the whole row group
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t o = lane + 32 * i;
                    uint64_t r = (uint64_t)rg * 16 + (o & 15);
                    if (o < vals && r < k.rows) k.y[(uint64_t)(o >> 4) * k.rows + r] = v[i];
                }
                return;
            }
            // slot 0 holds the piece of the CTA's first row group in this matrix, slot 1 the piece of its last one
            const uint32_t my_slot = (uint32_t)rg == cta_beg / KC ? 0u : 1u;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t o = lane + 32 * i;
                if (o < vals) k.ws_partial[((size_t)blockIdx.x * 2 + my_slot) * vals + o] = v[i];
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
            for (int i = 0; i < 4; ++i) {
                uint32_t o = lane + 32 * i;
                if (o >= vals) continue;
                float sum = 0.f;
                for (uint32_t c = c0; c <= c1; ++c) {
                    uint32_t slot = cta_first_chunk(c) / KC == (uint32_t)rg ? 0u : 1u;
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
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint32_t col = 2 * t + (j & 1), row = g + 8 * (j >> 1);
                if (col < A.batch) mine[col * 16 + row] = acc[j];
            }
            acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
            __syncwarp();
            float v[4];
            if (alone) {
#pragma unroll
                for (int i = 0; i < 4; ++i) v[i] = lane + 32 * i < vals ? mine[lane + 32 * i] : 0.f;
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
            for (int i = 0; i < 4; ++i) v[i] = 0.f;
            for (uint32_t m = mask; m; m &= m - 1) {              // pieces in warp order
                const uint32_t w = __ffs(m) - 1;
                const float *piece = part_val + (size_t)(w * 2 + __shfl_sync(0xFFFFFFFFu, slot_of_lane, w)) * vals;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (lane + 32 * i < vals) v[i] += piece[lane + 32 * i];
            }
            finish_cta_sum(rg, v);
        };

        if (c_beg < c_end && !failed) {
            uint32_t rg = c_beg / KC, kc = c_beg - rg * KC;            // tracked incrementally from here on
            uint32_t r0 = __ldg(index + c_beg), r1 = __ldg(index + c_beg + 1);
            // raw sign/mantissa bytes travel one block ahead of the decoder, in two register sets used in turn
            uint4 raw_a = make_uint4(0, 0, 0, 0), raw_b = make_uint4(0, 0, 0, 0);
            bool primed = false;

#pragma unroll 1
            for (uint32_t c = c_beg; c < c_end; ++c) {
                const uint32_t which = (c - c_beg) & 1u;
                const uint32_t nkb = blocks_of(kc);
                const bool ok = record_ok(r0, r1, nkb);
                // the chunk after this one: its first raw block is fetched from inside this chunk's loop
                const bool has_next = c + 1 < c_end;
                const uint32_t kc1 = kc + 1 == KC ? 0u : kc + 1;
                const uint32_t r2 = has_next ? __ldg(index + c + 2) : r1;
                const bool next_ok = has_next && record_ok(r1, r2, blocks_of(kc1));

                if (MODE == 1 && (int)rg != cur_rg) {
                    flush(cur_rg, c_beg, c);  // the previous row group ended with chunk c - 1
                    cur_rg = (int)rg;
                }

                // records follow each other in memory: the block after this chunk's last one is the first block
                // of the next record, `coded_bytes` further on
                const uint8_t *raw_p = payload + (uint64_t)r0 * 128u + lane * 16u;   // raw bytes of block 0
                const uint32_t coded_bytes = (r1 - r0) * 128u - nkb * 512u;
                if (ok && !primed) raw_a = ldg_stream16(raw_p);

                // wait, with a limit, for the coded part; the outcome is made uniform across the warp
                {
                    const uint32_t bar = bar0 + which * 8, parity = (phase >> which) & 1u;
                    uint32_t spins = 0;
                    bool done = mbar_try_wait(bar, parity);
                    while (!__all_sync(0xFFFFFFFFu, done)) {
                        if (++spins > kWaitLimit) { failed = true; break; }
                        done = mbar_try_wait(bar, parity);
                    }
                    if (failed) {
                        if (A.err && lane == 0) atomicExch(A.err, -1);
                        break;
                    }
                    phase ^= 1u << which;
                }

                if (!waited_prior) {
                    STAMP(3);
                    pdl_wait_prior_grid();   // from here on this warp reads x and writes results: the previous kernel must be done
                    waited_prior = true;
                }
                if (!ok) {  // record offsets out of range: report, produce nothing for this chunk, touch no memory
                    if (A.err && lane == 0) atomicExch(A.err, (int32_t)min(c + 1, 0x7FFFFFFFu));
                    primed = false;
                } else {
                    LaneStream sa, sb;
                    stream_open(sa, slot0 + which * A.slot_bytes + (lane << 2));
                    stream_open(sb, slot0 + which * A.slot_bytes + 128u + (lane << 2));
                    const uint32_t col0 = kc * k.chunk_cols + t * 8u;
                    // activations: lanes of unused output columns repeat the last vector (cols is a multiple of 32
                    // here, so every block of the chunk lies inside the row)
                    const uint16_t *xq = k.x + (MODE == 1 ? (uint64_t)min(g, A.batch - 1) * k.cols + col0 : 0);
                    uint16_t *out0 = MODE == 0 ? k.out + ((uint64_t)rg * 16 + g) * k.cols + col0 : nullptr;
                    const uint32_t last = nkb - 1;

                    // one block: start the fetch of the next block's raw bytes into `nxt`, decode with `cur`
                    auto block = [&](uint32_t kb, const uint4 &cur, uint4 &nxt) {
                        BLOCKSTAMP((c - c_beg) * 8 + kb, 0);
                        raw_p += 512;
                        if (kb == last) raw_p += coded_bytes;           // the next record's first block
                        if (kb != last || next_ok) nxt = ldg_stream16(raw_p);
                        uint4 xv;
                        if (MODE == 1) {
                            xv = __ldg((const uint4 *)xq);
                            xq += 32;
                        }

                        uint32_t a[8];
                        decode_block<R>(sa, sb, kIdxMask, lut_lane, one, cur, a);
                        BLOCKSTAMP((c - c_beg) * 8 + kb, 1);

                        if (MODE == 1) {
                            mma_bf16_16816(acc, a[0], a[4], a[1], a[5], xv.x, xv.y);
                            mma_bf16_16816(acc, a[2], a[6], a[3], a[7], xv.z, xv.w);
                            BLOCKSTAMP((c - c_beg) * 8 + kb, 2);
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
#pragma unroll 1
                    for (uint32_t kb = 0; kb < nkb; kb += 2) {
                        block(kb, raw_a, raw_b);
                        if (kb + 1 < nkb) block(kb + 1, raw_b, raw_a);
                    }
                    if (nkb & 1u) raw_a = raw_b;     // the next chunk's first block always starts in raw_a
                    primed = next_ok;
                }
                __syncwarp();
                if (lane == 0 && c + 2 < c_end) issue(c + 2, which);
                r0 = r1;
                r1 = r2;
                kc = kc1;
                rg += kc1 == 0 ? 1u : 0u;
            }
            if (MODE == 1 && !failed) flush(cur_rg, c_beg, c_end);
        }
        STAMP(4);
    }
    STAMP(7);
}

// ------------------------------------------------------------------------------ plain bf16 GEMV

// One warp per row, 16-byte loads, fp32 accumulation, shuffle reduction.
__global__ void __launch_bounds__(256) plain_gemv_kernel(const uint16_t *__restrict__ w, uint64_t rows, uint64_t cols,
                                                         const uint16_t *__restrict__ x, float *__restrict__ y) {
    const uint32_t lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    for (uint64_t r = warp; r < rows; r += nwarps) {
        const uint4 *wr = (const uint4 *)(w + r * cols);
        const uint4 *xr = (const uint4 *)x;
        float acc0 = 0.f, acc1 = 0.f;
        for (uint64_t i = lane; i < cols / 8; i += 32) {
            uint4 a = ldg_stream16(wr + i);
            uint4 b = __ldg(xr + i);
            const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc0 = fmaf(__uint_as_float(av[j] << 16), __uint_as_float(bv[j] << 16), acc0);
                acc1 = fmaf(__uint_as_float(av[j] & 0xFFFF0000u), __uint_as_float(bv[j] & 0xFFFF0000u), acc1);
            }
        }
        float acc = acc0 + acc1;
#pragma unroll
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) y[r] = acc;
    }
}

// ------------------------------------------------------------------------------ launchers

template <int MODE, int LB, int THREADS>
static cudaError_t launch_one(const KernelArgs &k, uint32_t grid, cudaStream_t stream) {
    auto fn = huff_kernel<MODE, LB, THREADS>;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)k.dyn_smem_bytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
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

cudaError_t launch_decode(const KernelArgs &k, uint32_t grid, cudaStream_t stream) {
    return k.lut_bits == 8 ? launch_one<0, 8, kThreads>(k, grid, stream) : launch_one<0, 9, kThreads>(k, grid, stream);
}

cudaError_t launch_gemm(const KernelArgs &k, uint32_t grid, cudaStream_t stream) {
    return k.lut_bits == 8 ? launch_one<1, 8, kThreads>(k, grid, stream) : launch_one<1, 9, kThreads>(k, grid, stream);
}

cudaError_t launch_plain_gemv(const uint16_t *w, uint64_t rows, uint64_t cols, const uint16_t *x, float *y, uint32_t sms,
                              cudaStream_t stream) {
    uint64_t blocks = (rows + 7) / 8;
    uint32_t grid = (uint32_t)(blocks < (uint64_t)sms * 8 ? blocks : (uint64_t)sms * 8);
    plain_gemv_kernel<<<grid, 256, 0, stream>>>(w, rows, cols, x, y);
    return cudaGetLastError();
}

}  // namespace huffllm
