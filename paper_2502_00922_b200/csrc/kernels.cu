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
//   * one warp decodes one chunk; lane l owns the bit sequence of lane l in the chunk record
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

// ------------------------------------------------------------------------------ lane decoder

// State of one lane's decoder.  (hi:lo) holds 64 stream bits; the current codeword starts at bit
// pos + 7 of that window (the 7 bits in front are the lag that makes the table address fall out of
// a single AND/OR); nxt is the shared-memory address of the lane's next 32-bit word.
struct LaneStream {
    uint32_t lo, hi, pos, nxt;
};

__device__ __forceinline__ void stream_open(LaneStream &s, uint32_t lane_word0) {
    s.lo = lds_stream(lane_word0);
    s.hi = lds_stream(lane_word0 + 128);
    s.nxt = lane_word0 + 256;
    s.pos = 0;
}

// One decoder step: returns the table entry (exponent << 23 | length) and advances the start pointer.
// The window is shifted as a 64-bit value, so the pointer may run past bit 32 between two refill
// checks.  Only the entry's low byte (the length) is added to the pointer: dp4a with the byte
// selector 1 does "pos += e & 0xFF" in one instruction, off the integer ALU pipe.
__device__ __forceinline__ uint32_t stream_step(LaneStream &s, uint32_t idx_mask, uint32_t lut_lane) {
    uint64_t win = ((uint64_t)s.hi << 32) | s.lo;
    uint32_t t = (uint32_t)(win >> s.pos);
    uint32_t e = lds_lut((t & idx_mask) | lut_lane);
    s.pos = __dp4a(e, 1u, s.pos);
    return e;
}

// Refill: once 32 bits have been consumed, slide the window by one word.
__device__ __forceinline__ void stream_refill(LaneStream &s) {
    if (s.pos & 32u) {
        s.lo = s.hi;
        s.hi = lds_stream(s.nxt);
        s.nxt += 128;
    }
    s.pos &= 31u;
}

// Two table entries + two raw bytes -> two bf16 weights packed in one register.
// SEL picks raw bytes (i, i+1) of `raw` as (byte, sign-replicated byte) pairs.
template <uint32_t SEL>
__device__ __forceinline__ uint32_t pack_pair(uint32_t e_even, uint32_t e_odd, uint32_t raw) {
    uint32_t sm = prmt(raw, 0u, SEL);             // [sign1*0xFF, raw1, sign0*0xFF, raw0]
    uint32_t ex = prmt(e_even, e_odd, 0x7632u);   // [E1 << 7 | E0 << 7] in the two halves
    return (sm & 0x807F807Fu) | (ex & 0x7F807F80u);
}

// Decode one block (16 weights of this lane) into 8 packed registers:
// a[0..3] = row g, columns (0,1) (2,3) (4,5) (6,7);  a[4..7] = row g+8, same columns.
// The window is checked for a refill before every R-th step: after a check at least 26 bits are
// valid in front of the start pointer, enough for R codewords of at most 26/R bits.
template <int R>
__device__ __forceinline__ void decode_block(LaneStream &s, uint32_t idx_mask, uint32_t lut_lane, const uint4 &raw,
                                             uint32_t (&a)[8]) {
    uint32_t e[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        if (i % R == 0) stream_refill(s);
        e[i] = stream_step(s, idx_mask, lut_lane);
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

__device__ __forceinline__ SmemPlan plan_smem(uint32_t base, const KernelArgs &k, uint32_t max_warps) {
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
constexpr uint32_t kWaitLimit = 1u << 22;

// ------------------------------------------------------------------------------ the fused kernel

// MODE 0: write the decoded weights.  MODE 1: y = W x for up to 8 activation vectors.
// R = decoder steps between two refill checks (3 when codewords are at most 8 bits, else 2).
template <int MODE, int R>
__global__ void __launch_bounds__(1024, 1) huff_kernel(const KernelArgs k) {
    extern __shared__ __align__(128) uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t bars[kMaxWarps * 2];
    __shared__ int part_rg[kMaxWarps * 2];
    __shared__ uint32_t s_last;

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps_launched = blockDim.x >> 5;
    const uint32_t smem_base = smem_u32(dyn_smem);
    const SmemPlan plan = plan_smem(smem_base, k, nwarps_launched);
    const uint32_t nw = plan.warps;
    const uint32_t vals = 16 * k.batch;
    float *part_val = (float *)(dyn_smem + k.dyn_smem_bytes - k.part_bytes);  // [2 * warps][16 * batch]

    // ---- set-up: per-lane table, barriers
    {
        const uint32_t *lut_g = (const uint32_t *)(k.blob + k.off_lut);
        uint32_t *lut_s = (uint32_t *)(dyn_smem + (plan.lut - smem_base));
        for (uint32_t i = tid; i < (32u << k.lut_bits); i += blockDim.x) lut_s[i] = __ldg(lut_g + (i >> 5));
        if (tid < kMaxWarps * 2) {
            mbar_init(smem_u32(&bars[tid]), 1);
            part_rg[tid] = -1;
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // ---- this warp's contiguous range of chunks
    const uint64_t T = k.n_chunks;
    const uint64_t cta_beg = T * blockIdx.x / gridDim.x, cta_end = T * (blockIdx.x + 1) / gridDim.x;
    uint64_t c_beg = cta_beg, c_end = cta_beg;
    if (warp < nw) {
        c_beg = cta_beg + (cta_end - cta_beg) * warp / nw;
        c_end = cta_beg + (cta_end - cta_beg) * (warp + 1) / nw;
    }

    const uint32_t *index = (const uint32_t *)(k.blob + k.off_index);
    const uint8_t *payload = k.blob + k.off_payload;
    const uint32_t idx_mask = ((1u << k.lut_bits) - 1u) << 7;
    const uint32_t lut_lane = plan.lut | (lane << 2);
    const uint32_t g = lane >> 2, t = lane & 3;

    auto blocks_of = [&](uint64_t c) -> uint32_t {
        uint32_t kc = (uint32_t)(c % k.col_chunks);
        uint32_t left = (uint32_t)(k.cols - (uint64_t)kc * k.chunk_cols);
        return (min(left, k.chunk_cols) + 31u) >> 5;
    };
    // a record is usable if it lies inside the payload and its coded part fits a slot
    auto record_ok = [&](uint32_t r0, uint32_t r1, uint32_t nkb) -> bool {
        return r1 > r0 && r1 <= k.payload_units && (r1 - r0) * 128u > nkb * 512u &&
               (r1 - r0) * 128u - nkb * 512u + 128u <= k.slot_bytes;
    };
    // lane 0: start the bulk copy of chunk c's coded part into slot `which`
    auto issue = [&](uint64_t c, uint32_t which) {
        uint32_t nkb = blocks_of(c), r0 = __ldg(index + c), r1 = __ldg(index + c + 1);
        uint32_t bar = smem_u32(&bars[warp * 2 + which]);
        if (record_ok(r0, r1, nkb)) {
            uint32_t bytes = (r1 - r0) * 128u - nkb * 512u;
            mbar_expect_tx(bar, bytes);
            bulk_g2s(slot_addr(plan, warp, which, k.slot_bytes), payload + (uint64_t)r0 * 128u + nkb * 512u, bytes, bar);
        } else {
            mbar_expect_tx(bar, 0);  // completes the phase with nothing to wait for; the chunk is skipped below
        }
    };

    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    int64_t cur_rg = -1;
    uint32_t n_partial = 0;

    // hand a finished row group to y (if this warp saw all of its chunks) or to the CTA's partial table
    auto flush = [&](int64_t rg, uint64_t first_c, uint64_t last_c_excl) {
        if (rg < 0) return;
        bool complete = first_c <= (uint64_t)rg * k.col_chunks && last_c_excl >= (uint64_t)(rg + 1) * k.col_chunks;
        uint32_t ent = warp * 2 + min(n_partial, 1u);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t col = 2 * t + (j & 1), row = g + 8 * (j >> 1);
            if (col >= k.batch) continue;
            if (complete) {
                uint64_t r = (uint64_t)rg * 16 + row;
                if (r < k.rows) k.y[(uint64_t)col * k.rows + r] = acc[j];
            } else {
                part_val[(size_t)ent * vals + col * 16 + row] = acc[j];
            }
        }
        if (!complete) {
            if (lane == 0) part_rg[ent] = (int)rg;
            ++n_partial;
        }
        acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
    };

    if (c_beg < c_end) {
        if (lane == 0) {
            issue(c_beg, 0);
            if (c_beg + 1 < c_end) issue(c_beg + 1, 1);
        }
        uint4 raw_next = make_uint4(0, 0, 0, 0);
        {
            uint32_t r0 = __ldg(index + c_beg);
            if (r0 + 4u <= k.payload_units) raw_next = ldg_stream16(payload + (uint64_t)r0 * 128u + lane * 16u);
        }
        bool failed = false;

        for (uint64_t c = c_beg; c < c_end; ++c) {
            const uint32_t which = (uint32_t)(c - c_beg) & 1u, parity = (uint32_t)((c - c_beg) >> 1) & 1u;
            const uint32_t rg = (uint32_t)(c / k.col_chunks), kc = (uint32_t)(c % k.col_chunks);
            const uint32_t nkb = blocks_of(c);
            const uint32_t r0 = __ldg(index + c), r1 = __ldg(index + c + 1);
            const bool ok = record_ok(r0, r1, nkb);
            const uint8_t *raw_g = payload + (uint64_t)r0 * 128u + lane * 16u;
            const bool next_ok = c + 1 < c_end && r1 + 4u <= k.payload_units;
            const uint8_t *raw_g_next = payload + (uint64_t)r1 * 128u + lane * 16u;

            if (MODE == 1 && (int64_t)rg != cur_rg) {
                flush(cur_rg, c_beg, c);  // the previous row group ended with chunk c - 1
                cur_rg = rg;
            }

            // wait, with a limit, for the coded part; the outcome is made uniform across the warp
            {
                uint32_t bar = smem_u32(&bars[warp * 2 + which]), spins = 0;
                bool done = mbar_try_wait(bar, parity);
                while (!__all_sync(0xFFFFFFFFu, done)) {
                    if (++spins > kWaitLimit) { failed = true; break; }
                    done = mbar_try_wait(bar, parity);
                }
                if (failed) {
                    if (k.err && lane == 0) atomicExch(k.err, -1);
                    break;
                }
            }

            if (!ok) {  // record offsets out of range: report, produce nothing for this chunk, touch no memory
                if (k.err && lane == 0) atomicExch(k.err, (int32_t)min(c + 1, (uint64_t)0x7FFFFFFF));
                raw_next = next_ok ? ldg_stream16(raw_g_next) : make_uint4(0, 0, 0, 0);
            } else {
                LaneStream s;
                stream_open(s, slot_addr(plan, warp, which, k.slot_bytes) + (lane << 2));
                const uint64_t col0 = (uint64_t)kc * k.chunk_cols + t * 8u;

                for (uint32_t kb = 0; kb < nkb; ++kb) {
                    const uint4 raw = raw_next;
                    if (kb + 1 < nkb) raw_next = ldg_stream16(raw_g + (size_t)(kb + 1) * 512u);
                    else if (next_ok) raw_next = ldg_stream16(raw_g_next);

                    const uint64_t col = col0 + (uint64_t)kb * 32u;
                    uint4 xv = make_uint4(0, 0, 0, 0);
                    if (MODE == 1 && col < k.cols)  // lanes of unused output columns repeat the last vector
                        xv = __ldg((const uint4 *)(k.x + (uint64_t)min(g, k.batch - 1) * k.cols + col));

                    uint32_t a[8];
                    decode_block<R>(s, idx_mask, lut_lane, raw, a);

                    if (MODE == 1) {
                        mma_bf16_16816(acc, a[0], a[4], a[1], a[5], xv.x, xv.y);
                        mma_bf16_16816(acc, a[2], a[6], a[3], a[7], xv.z, xv.w);
                    } else {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            uint64_t r = (uint64_t)rg * 16 + g + 8 * h;
                            if (r >= k.rows || col >= k.cols) continue;
                            uint16_t *dst = k.out + r * k.cols + col;
                            if (k.cols % 8 == 0) {
                                *(uint4 *)dst = make_uint4(a[4 * h], a[4 * h + 1], a[4 * h + 2], a[4 * h + 3]);
                            } else {
#pragma unroll
                                for (int i = 0; i < 8; ++i)
                                    if (col + i < k.cols) dst[i] = (uint16_t)(a[4 * h + (i >> 1)] >> (16 * (i & 1)));
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0 && c + 2 < c_end) issue(c + 2, which);
        }
        if (MODE == 1 && !failed) flush(cur_rg, c_beg, c_end);
    }

    if (MODE != 1) return;

    // ---- combine inside the CTA, in warp order
    __syncthreads();
    float *ws_val = k.ws_partial + (size_t)blockIdx.x * 2 * vals;
    int *ws_rg = k.ws_rg + blockIdx.x * 2;
    if (tid < vals) {
        int cur = -1, n_out = 0;
        float sum = 0.f;
        auto emit = [&](int rg) {
            bool complete = cta_beg <= (uint64_t)rg * k.col_chunks && cta_end >= (uint64_t)(rg + 1) * k.col_chunks;
            if (complete) {
                uint64_t r = (uint64_t)rg * 16 + (tid & 15);
                if (r < k.rows) k.y[(uint64_t)(tid >> 4) * k.rows + r] = sum;
            } else {
                int slot = min(n_out, 1);
                ws_val[(size_t)slot * vals + tid] = sum;
                if (tid == 0) ws_rg[slot] = rg;
                ++n_out;
            }
        };
        for (uint32_t e = 0; e < nw * 2; ++e) {
            int rg = part_rg[e];
            if (rg < 0) continue;
            if (rg != cur) {
                if (cur >= 0) emit(cur);
                cur = rg;
                sum = 0.f;
            }
            sum += part_val[(size_t)e * vals + tid];
        }
        if (cur >= 0) emit(cur);
        if (tid == 0)
            for (int sl = n_out; sl < 2; ++sl) ws_rg[sl] = -1;
    }

    // ---- combine across CTAs: the last CTA to arrive adds the boundary partials in CTA order
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(k.ws_ticket, 1u) == gridDim.x - 1) ? 1u : 0u;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const uint32_t n_ent = gridDim.x * 2;
    for (uint32_t e = warp; e < n_ent; e += nwarps_launched) {
        int rg = __ldcg(k.ws_rg + e);
        if (rg < 0) continue;
        bool first = true;  // first valid entry of its row group?
        for (int q = (int)e - 1; q >= 0; --q) {
            int tag = __ldcg(k.ws_rg + q);
            if (tag < 0) continue;
            first = tag != rg;
            break;
        }
        if (!first) continue;
        for (uint32_t o = lane; o < vals; o += 32) {
            float sum = 0.f;
            for (uint32_t q = e; q < n_ent; ++q) {
                int tag = __ldcg(k.ws_rg + q);
                if (tag < 0) continue;
                if (tag != rg) break;
                sum += __ldcg(k.ws_partial + (size_t)q * vals + o);
            }
            uint64_t r = (uint64_t)rg * 16 + (o & 15);
            if (r < k.rows) k.y[(uint64_t)(o >> 4) * k.rows + r] = sum;
        }
    }
    __syncthreads();
    // leave the scratch as it was found: all zero
    for (uint32_t e = tid; e < n_ent; e += blockDim.x) k.ws_rg[e] = 0;
    if (tid == 0) *k.ws_ticket = 0;
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

template <int MODE, int R>
static cudaError_t launch_one(const KernelArgs &k, uint32_t grid, cudaStream_t stream) {
    auto fn = huff_kernel<MODE, R>;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)k.dyn_smem_bytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    fn<<<grid, 1024, k.dyn_smem_bytes, stream>>>(k);
    return cudaGetLastError();
}

cudaError_t launch_decode(const KernelArgs &k, uint32_t grid, cudaStream_t stream) {
    return k.lut_bits == 8 ? launch_one<0, 3>(k, grid, stream) : launch_one<0, 2>(k, grid, stream);
}

cudaError_t launch_gemm(const KernelArgs &k, uint32_t grid, cudaStream_t stream) {
    return k.lut_bits == 8 ? launch_one<1, 3>(k, grid, stream) : launch_one<1, 2>(k, grid, stream);
}

cudaError_t launch_plain_gemv(const uint16_t *w, uint64_t rows, uint64_t cols, const uint16_t *x, float *y, uint32_t sms,
                              cudaStream_t stream) {
    uint64_t blocks = (rows + 7) / 8;
    uint32_t grid = (uint32_t)(blocks < (uint64_t)sms * 8 ? blocks : (uint64_t)sms * 8);
    plain_gemv_kernel<<<grid, 256, 0, stream>>>(w, rows, cols, x, y);
    return cudaGetLastError();
}

}  // namespace huffllm
