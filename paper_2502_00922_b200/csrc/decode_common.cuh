// Device code shared by the decode kernels: PTX helpers, the per-sequence decoder, the shared-memory plan.
#pragma once
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
// Arrival without a transaction count (a consumer hands a slot back).
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One look at a barrier's phase, without waiting.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
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
__device__ __forceinline__ uint32_t ldg_stream2(const void *p) {
    uint16_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void mma_f16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                              uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Two mixed-precision multiply-adds: acc += w.lo * x.lo, then acc += w.hi * x.hi (bf16 halves of the two words).
// The products are exact in f32; each addition rounds once.
__device__ __forceinline__ void fma2_bf16(float &acc, uint32_t w, uint32_t x) {
    asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\t"
        "mov.b32 {wl, wh}, %1;\n\t"
        "mov.b32 {xl, xh}, %2;\n\t"
        "fma.rn.f32.bf16 %0, wl, xl, %0;\n\t"
        "fma.rn.f32.bf16 %0, wh, xh, %0;\n\t}"
        : "+f"(acc)
        : "r"(w), "r"(x));
}

__device__ __forceinline__ void fma2_f16(float &acc, uint32_t w, uint32_t x) {
    asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\t"
        "mov.b32 {wl, wh}, %1;\n\t"
        "mov.b32 {xl, xh}, %2;\n\t"
        "fma.rn.f32.f16 %0, wl, xl, %0;\n\t"
        "fma.rn.f32.f16 %0, wh, xh, %0;\n\t}"
        : "+f"(acc)
        : "r"(w), "r"(x));
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

__device__ __forceinline__ void stream_open(LaneStream &s, uint32_t lane_word0, uint32_t pos0 = 0) {
    s.lo = lds_stream(lane_word0);
    s.hi = lds_stream(lane_word0 + 256);
    s.nxt = lane_word0 + 512;
    s.pos = pos0;
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

// Tables of 10 to 12 index bits (Section 3.2 quotes L_max = 12) are looked up in two levels.  The first level is the
// 256-entry table of the first 8 stream bits, replicated per lane like the 8-bit table; an entry whose codeword is longer
// than 8 bits carries a mark (bit 31) instead of a result, and the lane then reads the entry from the whole table
// (one copy in shared memory, indexed by all lut_bits bits; bank conflicts there do not matter: long codewords are
// rare).  full_mask = ((1 << lut_bits) - 1) << 2 turns the shifted window into that table's byte offset.
constexpr uint32_t kLongMark = 0x80000000u;
__device__ __forceinline__ uint32_t stream_step_long(LaneStream &s, uint32_t lut_lane, uint32_t full_base, uint32_t full_mask) {
    uint64_t win = ((uint64_t)s.hi << 32) | s.lo;
    uint32_t t = (uint32_t)(win >> s.pos), addr;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(addr) : "r"(t), "r"(0xFFu << 7), "r"(lut_lane));
    uint32_t e = lds_lut(addr);
    if (e & kLongMark) e = lds_lut(full_base + ((t >> 5) & full_mask));   // (t >> 7) is the index: times 4 bytes
    s.pos = __dp4a(e, 0x00010000u, s.pos);
    return e;
}

// The decoder of 8-bit BF16 tables works on four codewords at a time.  Its pointer stands on the codeword itself (the
// sequence's leading zero bits are skipped when the sequence is opened), so after a refill check, with the pointer
// below 32, the low 32 bits of the shifted window are all valid: room for four codewords of at most 8 bits.
//   * The 32 bits are taken out of the window once (one 64-bit shift) and then shifted in place by each codeword's
//     length: the shared-memory copy of the table repeats the length in an entry's low 5 bits (lut_entry_inplace), and a
//     wrapping shift reads just those.  The pointer is not on the chain from one lookup to the next.
//   * The table index is byte 0 of that word, and index * 128 + table base is one byte dot product.
//   * The pointer is advanced once per four codewords by two three-input additions of the whole entries.  Only its low
//     6 bits mean anything (pointer + lengths <= 31 + 32; bits 5 and 6 of an entry are zero, the exponent starts at
//     bit 7, so nothing carries into them and bit 6 stays zero); whatever piles up above bit 6 is never read: the
//     refill check tests bit 5 and the funnel shift reads bits 0..4.
__device__ __forceinline__ uint32_t lut_entry_inplace(uint32_t e) { return e | (e >> 16); }

template <bool RELOAD = true>      // false: the low word is copied from the high one (where shared-memory bandwidth is the scarcer resource)
__device__ __forceinline__ void stream_refill4(LaneStream &s) {
    if (RELOAD) {
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t.reg .b32 b;\n\t"
            "setp.ne.u32 q, 0, 0;\n\t"
            "lop3.or.b32 b|p, %2, 32, 0, 0xC0, q;\n\t"          // p = bit 5 of the pointer: 32 or more bits consumed
            "@p ld.shared.u32 %0, [%3+-256];\n\t"
            "@p ld.shared.u32 %1, [%3];\n\t"
            "@p add.u32 %3, %3, 256;\n\t"
            "@p add.u32 %2, %2, 0xFFFFFFE0;\n\t}"
            : "+r"(s.lo), "+r"(s.hi), "+r"(s.pos), "+r"(s.nxt));
    } else {
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t.reg .b32 b;\n\t"
            "setp.ne.u32 q, 0, 0;\n\t"
            "lop3.or.b32 b|p, %2, 32, 0, 0xC0, q;\n\t"
            "@p mov.u32 %0, %1;\n\t"
            "@p ld.shared.u32 %1, [%3];\n\t"
            "@p add.u32 %3, %3, 256;\n\t"
            "@p add.u32 %2, %2, 0xFFFFFFE0;\n\t}"
            : "+r"(s.lo), "+r"(s.hi), "+r"(s.pos), "+r"(s.nxt));
    }
}
// The 32 window bits at the pointer, right after a refill check (pointer below 32: a 32-bit funnel shift is enough,
// and it reads only the pointer's low 5 bits).
__device__ __forceinline__ uint32_t window_at(const LaneStream &s) {
    uint32_t t;
    asm("shf.r.wrap.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(s.lo), "r"(s.hi), "r"(s.pos));
    return t;
}
__device__ __forceinline__ uint32_t lookup_byte0(uint32_t t, uint32_t lut_lane) { return lds_lut(__dp4a(t, 0x00000080u, lut_lane)); }
__device__ __forceinline__ uint32_t shift_by_entry(uint32_t t, uint32_t e) {
    uint32_t d;
    asm("shf.r.wrap.b32 %0, %1, 0, %2;" : "=r"(d) : "r"(t), "r"(e));
    return d;
}
// Four codewords of each of a lane's two sequences, the two chains interleaved.
__device__ __forceinline__ void stream_step4x2(LaneStream &sa, LaneStream &sb, uint32_t lut_lane, uint32_t *ea, uint32_t *eb) {
    stream_refill4(sa);
    stream_refill4(sb);
    uint32_t ta = window_at(sa), tb = window_at(sb);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        ea[k] = lookup_byte0(ta, lut_lane);
        eb[k] = lookup_byte0(tb, lut_lane);
        if (k < 3) {
            ta = shift_by_entry(ta, ea[k]);
            tb = shift_by_entry(tb, eb[k]);
        }
    }
    sa.pos = (sa.pos + ea[0] + ea[1]) + (ea[2] + ea[3]);
    sb.pos = (sb.pos + eb[0] + eb[1]) + (eb[2] + eb[3]);
}

// Refill: once 32 bits have been consumed, slide the window by one word.  Written with predicated
// instructions so that lanes which need a word and lanes which do not stay converged.  The low word is
// reloaded from shared memory rather than copied from the high word: a load is not an integer
// instruction, and 32-bit integer issue is what bounds this kernel.
// (A plain 32-bit addition costs one dispatch cycle; logic, shift, compare, select and byte-permute instructions two.
// Adding the entry's length by multiply-high with a register holding 65536 is cheap in isolation, 1.35 cycles, but
// made this kernel 20 % slower: the pointer advance sits on the decoder's dependency chain.)
template <bool RELOAD = true>
__device__ __forceinline__ void stream_refill(LaneStream &s) {
    if (RELOAD) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ge.u32 p, %2, 32;\n\t"
            "@p ld.shared.u32 %0, [%3+-256];\n\t"
            "@p ld.shared.u32 %1, [%3];\n\t"
            "@p add.u32 %3, %3, 256;\n\t"
            "@p add.u32 %2, %2, 0xFFFFFFE0;\n\t}"
            : "+r"(s.lo), "+r"(s.hi), "+r"(s.pos), "+r"(s.nxt));
    } else {   // where shared-memory bandwidth is the scarcer resource (FP16 blobs): copy the register instead
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ge.u32 p, %2, 32;\n\t"
            "@p mov.u32 %0, %1;\n\t"
            "@p ld.shared.u32 %1, [%3];\n\t"
            "@p add.u32 %3, %3, 256;\n\t"
            "@p add.u32 %2, %2, 0xFFFFFFE0;\n\t}"
            : "+r"(s.lo), "+r"(s.hi), "+r"(s.pos), "+r"(s.nxt));
    }
}

// Two table entries + the raw word of their group -> two bf16 weights packed in one register.
// A raw word holds the sign and mantissa bits of four consecutive weights of a row, laid out so that the first pair's
// bits already sit where a packed pair of bf16 words has them (mantissas at bits 0..6 and 16..22, signs at 15 and 31)
// and the second pair's do after a rotation by one byte; the other pair's bits lie in the exponent positions, which
// the select below takes from the table entries.  The exponent of the even weight is already in place (bits 7..14);
// the odd entry times 65536 puts its exponent at bits 23..30 and pushes its length out of the word, so one
// multiply-add merges the two.
__device__ __forceinline__ uint32_t pack_pair(uint32_t e_even, uint32_t e_odd, uint32_t sm) {
    uint32_t ex;
    asm("mad.lo.u32 %0, %1, 65536, %2;" : "=r"(ex) : "r"(e_odd), "r"(e_even));
    uint32_t w;   // sign and mantissa bits from sm, exponent bits from ex
    asm("lop3.b32 %0, %1, %2, 0x807F807F, 0xE4;" : "=r"(w) : "r"(sm), "r"(ex));
    return w;
}
__device__ __forceinline__ uint32_t rotr8(uint32_t v) { return prmt(v, v, 0x0321u); }

// Decode one block (16 weights of this lane) into 8 packed registers:
// a[0..3] = row g, columns (0,1) (2,3) (4,5) (6,7);  a[4..7] = row g+8, same columns.
// The lane's two sequences are stepped alternately.  Each window is checked for a refill before every
// R-th step: after a check at least 26 bits are valid in front of the start pointer, enough for R
// codewords of at most 26/R bits.
template <int R, bool SKIP = false, bool LONG = false>
__device__ __forceinline__ void decode_block(LaneStream &sa, LaneStream &sb, uint32_t idx_mask, uint32_t lut_lane,
                                             const uint4 &raw, uint32_t (&a)[8], uint32_t full_base = 0, uint32_t full_mask = 0) {
    uint32_t e[16];
    if (SKIP) {
        stream_step4x2(sa, sb, lut_lane, e, e + 8);
        stream_step4x2(sa, sb, lut_lane, e + 4, e + 12);
    } else
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (i % R == 0) {
            stream_refill(sa);
            stream_refill(sb);
        }
        if (LONG) {
            e[i] = stream_step_long(sa, lut_lane, full_base, full_mask);
            e[8 + i] = stream_step_long(sb, lut_lane, full_base, full_mask);
        } else {
            e[i] = stream_step(sa, idx_mask, lut_lane);
            e[8 + i] = stream_step(sb, idx_mask, lut_lane);
        }
    }
    a[0] = pack_pair(e[0], e[1], raw.x);
    a[1] = pack_pair(e[2], e[3], rotr8(raw.x));
    a[2] = pack_pair(e[4], e[5], raw.y);
    a[3] = pack_pair(e[6], e[7], rotr8(raw.y));
    a[4] = pack_pair(e[8], e[9], raw.z);
    a[5] = pack_pair(e[10], e[11], rotr8(raw.z));
    a[6] = pack_pair(e[12], e[13], raw.w);
    a[7] = pack_pair(e[14], e[15], rotr8(raw.w));
}

// ------------------------------------------------------------------------------ FP16 {1,5,5,5}

// FP16 blobs code three fields per weight (exponent, upper and lower mantissa half: Section 3.1), each with its own
// 256-entry table.  The tables sit 16 KB apart, each replicated sixteen times (entry i of copy c at word 16 i + c; a
// lane uses copy lane % 16: two lanes share a copy and collide when their entries fall into the same bank, which the
// measured 86 % shared-memory pipe load of an eight-fold version made worth halving), so the index bits of a lookup
// address are bits 6..13 and the lag of the stream is 6 bits.
// A table entry is length << 16 | symbol << (10, 5, 0): the three entries of a weight OR-ed together are its low
// 15 bits.  One refill check per weight: after it the pointer is below 32, three codewords of at most 8 bits and the
// lag of the last lookup end at bit 31 + 16 + 14 = 61 of the 64-bit window.
__device__ __forceinline__ uint32_t fp16_field(LaneStream &s, uint32_t lut_lane, uint32_t table_off) {
    uint64_t win = ((uint64_t)s.hi << 32) | s.lo;
    uint32_t t = (uint32_t)(win >> s.pos), addr, e;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(addr) : "r"(t), "r"(0xFFu << 6), "r"(lut_lane));
    asm("ld.shared.u32 %0, [%1];" : "=r"(e) : "r"(addr + table_off));
    s.pos = __dp4a(e, 0x00010000u, s.pos);
    return e;
}
__device__ __forceinline__ uint32_t fp16_weight(LaneStream &s, uint32_t lut_lane) {
    uint32_t e0 = fp16_field(s, lut_lane, 0), e1 = fp16_field(s, lut_lane, 16384), e2 = fp16_field(s, lut_lane, 32768), w;
    asm("lop3.b32 %0, %1, %2, %3, 0xFE;" : "=r"(w) : "r"(e0), "r"(e1), "r"(e2));
    return w;                                      // low 16 bits: exponent and mantissa; above: the three lengths mixed
}
// Field codes of 9 to 12 bits (Section 3.2: L_max = 12 for the 5-bit fields): two levels, as for BF16.  The first level is
// the field's sixteen-fold table of the first 8 bits; a marked entry sends the lane to the field's whole table
// (1 << lut_bits entries, one copy; the three follow each other from full_base).  A codeword may now take 12 bits, so the
// window is checked before every field (pointer below 32: lag 6 + 12 bits end inside the 64-bit window).
__device__ __forceinline__ uint32_t fp16_field_long(LaneStream &s, uint32_t lut_lane, uint32_t table_off, uint32_t full_addr,
                                                    uint32_t full_mask) {
    stream_refill<false>(s);
    uint64_t win = ((uint64_t)s.hi << 32) | s.lo;
    uint32_t t = (uint32_t)(win >> s.pos), addr, e;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(addr) : "r"(t), "r"(0xFFu << 6), "r"(lut_lane));
    asm("ld.shared.u32 %0, [%1];" : "=r"(e) : "r"(addr + table_off));
    if (e & kLongMark) e = lds_lut(full_addr + ((t >> 4) & full_mask));     // (t >> 6) is the index: times 4 bytes
    s.pos = __dp4a(e, 0x00010000u, s.pos);
    return e;
}
__device__ __forceinline__ uint32_t fp16_weight_long(LaneStream &s, uint32_t lut_lane, uint32_t full_base, uint32_t full_mask) {
    const uint32_t table_bytes = full_mask + 4u;                            // bytes of one field's whole table
    uint32_t e0 = fp16_field_long(s, lut_lane, 0, full_base, full_mask);
    uint32_t e1 = fp16_field_long(s, lut_lane, 16384, full_base + table_bytes, full_mask);
    uint32_t e2 = fp16_field_long(s, lut_lane, 32768, full_base + 2u * table_bytes, full_mask), w;
    asm("lop3.b32 %0, %1, %2, %3, 0xFE;" : "=r"(w) : "r"(e0), "r"(e1), "r"(e2));
    return w;
}
// Field codes of at most 8 bits, three codewords at a time (the scheme of the 8-bit BF16 decoder): the pointer stands on the
// codeword (the sequence's 6 leading zero bits are skipped when it is opened); after one check per weight it is below 32,
// so the low 32 bits of the shifted window hold the weight's three codewords (at most 24 bits).  They are taken out of
// the window once and shifted in place by each codeword's length, which the shared-memory copy of the tables keeps in an
// entry's low byte: entry = symbol bits << 8 | length (fp16_entry_inplace), so the OR of a weight's three entries has the
// weight's low 15 bits at bits 8..22.  The table address is byte 0 of the window times 64 plus the lane's column of the
// field's table: one byte dot product.  The pointer is advanced once per weight by the sum of the three entries; only its
// low 6 bits mean anything (lengths add up to at most 24, bits 4..7 of an entry are zero) and nothing reads above them.
__device__ __forceinline__ uint32_t fp16_entry_inplace(uint32_t e) { return ((e & 0x7FFFu) << 8) | (e >> 16); }
__device__ __forceinline__ uint32_t fp16_weight_inplace(LaneStream &s, uint32_t lut_lane) {
    stream_refill4<false>(s);
    uint32_t t = window_at(s);
    const uint32_t e0 = lds_lut(__dp4a(t, 0x00000040u, lut_lane));
    t = shift_by_entry(t, e0);
    const uint32_t e1 = lds_lut(__dp4a(t, 0x00000040u, lut_lane) + 16384u);
    t = shift_by_entry(t, e1);
    const uint32_t e2 = lds_lut(__dp4a(t, 0x00000040u, lut_lane) + 32768u);
    s.pos = (s.pos + e0) + (e1 + e2);
    uint32_t w;
    asm("lop3.b32 %0, %1, %2, %3, 0xFE;" : "=r"(w) : "r"(e0), "r"(e1), "r"(e2));
    return w;                                      // bits 8..22: exponent and mantissa
}
// Both mantissa halves carry the FLAT code (all 32 symbols, 5 bits each: the canonical codeword of symbol s is s, written
// first bit first), which is what fp16-trained weights give: their mantissa bits are incompressible.  The ten stream bits
// behind the exponent's codeword are then the weight's ten mantissa bits in reverse order: one bit reversal replaces two
// table lookups.  (The exponent's table and everything else is as in fp16_weight_inplace; bits 0..7 of the result hold
// the exponent's length and later stream bits, which the packing step never looks at.)
__device__ __forceinline__ uint32_t fp16_weight_flat(LaneStream &s, uint32_t lut_lane) {
    stream_refill4<false>(s);
    uint32_t t = window_at(s);
    const uint32_t e0 = lds_lut(__dp4a(t, 0x00000040u, lut_lane));
    t = shift_by_entry(t, e0);
    s.pos = s.pos + e0 + 10u;
    return e0 | (__brev(t) >> 14);                 // bits 8..17: the mantissa, bits 18..22: the exponent
}
// Field codes of at most 7 bits: the same three-at-a-time scheme on tables of 128 entries, which are small enough to keep
// once per LANE (entry i of lane l at word 32 i + l, 16 KB per field: the footprint of the sixteen-fold 256-entry tables),
// so that a warp-wide lookup never has a bank conflict.  Seven index bits are not a byte, so the window is moved up by 7
// bits once per weight and the table address is (window & index mask) | lane column, one logic operation; the in-place
// shifts keep the next codeword at bit 7 (25 window bits are valid there: three codewords take at most 21).
__device__ __forceinline__ uint32_t fp16_weight_lane(LaneStream &s, uint32_t lut_lane) {
    stream_refill4<false>(s);
    uint32_t t = window_at(s) << 7, a0, a1, a2;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(a0) : "r"(t), "r"(0x7Fu << 7), "r"(lut_lane));
    const uint32_t e0 = lds_lut(a0);
    t = shift_by_entry(t, e0);
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(a1) : "r"(t), "r"(0x7Fu << 7), "r"(lut_lane));
    const uint32_t e1 = lds_lut(a1 + 16384u);
    t = shift_by_entry(t, e1);
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(a2) : "r"(t), "r"(0x7Fu << 7), "r"(lut_lane));
    const uint32_t e2 = lds_lut(a2 + 32768u);
    s.pos = (s.pos + e0) + (e1 + e2);
    uint32_t w;
    asm("lop3.b32 %0, %1, %2, %3, 0xFE;" : "=r"(w) : "r"(e0), "r"(e1), "r"(e2));
    return w;                                      // bits 8..22: exponent and mantissa
}
// Decode one block of an FP16 chunk into 8 packed registers (same order as decode_block).  `signs` is the lane's
// uint16 of the block: bit p = sign of the first weight of pair p, bit 8 + p = sign of its second weight.
// INPLACE: the three-at-a-time decoders above: 1 = tables of 8 bits (sixteen-fold), 2 = tables of 7 bits (per lane),
// 3 = tables of 8 bits with flat codes for both mantissa halves.
template <bool LONG = false, int INPLACE = 0>
__device__ __forceinline__ void decode_block_fp16(LaneStream &sa, LaneStream &sb, uint32_t lut_lane, uint32_t signs,
                                                  uint32_t (&a)[8], uint32_t full_base = 0, uint32_t full_mask = 0) {
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (INPLACE == 3) {
            w[i] = fp16_weight_flat(sa, lut_lane);
            w[8 + i] = fp16_weight_flat(sb, lut_lane);
        } else if (INPLACE == 2) {
            w[i] = fp16_weight_lane(sa, lut_lane);
            w[8 + i] = fp16_weight_lane(sb, lut_lane);
        } else if (INPLACE == 1) {
            w[i] = fp16_weight_inplace(sa, lut_lane);
            w[8 + i] = fp16_weight_inplace(sb, lut_lane);
        } else if (LONG) {
            w[i] = fp16_weight_long(sa, lut_lane, full_base, full_mask);
            w[8 + i] = fp16_weight_long(sb, lut_lane, full_base, full_mask);
        } else {
            stream_refill<false>(sa);
            stream_refill<false>(sb);
            w[i] = fp16_weight(sa, lut_lane);
            w[8 + i] = fp16_weight(sb, lut_lane);
        }
    }
    const uint32_t s32 = prmt(signs, 0u, 0x4140u);     // first-weight signs in bits 0..7, second-weight signs in bits 16..23
#pragma unroll
    for (int p = 0; p < 8; ++p) {
        uint32_t pair = prmt(w[2 * p], w[2 * p + 1], INPLACE ? 0x6521u : 0x5410u);   // the two weights' 15 bits (in place: from bits 8..22)
        uint32_t sh = s32 << (15 - p);                            // their sign bits at bits 15 and 31
        asm("lop3.b32 %0, %1, %2, 0x7FFF7FFF, 0xE4;" : "=r"(a[p]) : "r"(pair), "r"(sh));   // mask bit set: pair, else sign
    }
}

// ------------------------------------------------------------------------------ shared memory plan

// Dynamic shared memory, laid out at run time from the window's real start address:
//   [base, lut)            slot pairs (single slots where the launch says so), as many as fit
//   [lut, lut + LUTSZ)     per-lane LUT; lut = base rounded up to a multiple of LUTSZ, so that the
//                          index bits of a lookup address never overlap the table's base bits
//   [lut + LUTSZ, ...)     more slot pairs, then a guard area no valid stream ever reads (it may overlap the next area)
//   [end - part_bytes, end) the CTA's table of partial sums (fused product only)
struct SmemPlan {
    uint32_t lut;    // shared address of the table
    uint32_t warps;  // warps that own a slot pair
    uint32_t slotA;  // first slot pair before the table
    uint32_t nA;     // slot pairs before the table
    uint32_t slotB;  // first slot pair after it
};

__device__ __forceinline__ SmemPlan plan_smem(uint32_t base, const KernelArgs &k, uint32_t max_warps, uint32_t slots = 2) {   // k: launch-wide fields only
    SmemPlan p;
    const uint32_t lut_bytes = k.lut_align;
    uint32_t a0 = (base + 127u) & ~127u;
    p.lut = (base + lut_bytes - 1) & ~(lut_bytes - 1);        // lut_align is a power of two
    p.slotA = a0;
    // (divisions by the slot pair's size as a multiplication by its rounded-down reciprocal and one correction: this
    // runs in every warp of a launch's set-up, which is bound by instruction issue)
    const uint32_t pair = slots == 2 ? 2 * k.slot_bytes : k.slot_bytes;
    auto div_pair = [&](uint32_t x) -> uint32_t {
        uint32_t q = __umulhi(x, k.pair_recip);
        return x - q * pair >= pair ? q + 1 : q;
    };
    p.nA = p.lut > a0 ? div_pair(p.lut - a0) : 0;  // a stream that overruns here reads the table: harmless
    p.slotB = p.lut + k.lut_size;
    uint32_t end = base + k.dyn_smem_bytes - k.part_bytes;
    // the guard area (read only, and only by a corrupt stream) may lie over what follows the slots; what it needs beyond that stays free
    const uint32_t guard_extra = k.guard_bytes > k.part_bytes ? k.guard_bytes - k.part_bytes : 0;
    uint32_t roomB = end > p.slotB + guard_extra ? end - p.slotB - guard_extra : 0;
    p.warps = min(max_warps, p.nA + div_pair(roomB));
    return p;
}

// Slot `which` of a decoder warp (two slots per warp).
__device__ __forceinline__ uint32_t slot_addr(const SmemPlan &p, uint32_t warp, uint32_t which, uint32_t slot_bytes) {
    uint32_t pair = warp < p.nA ? p.slotA + warp * 2 * slot_bytes : p.slotB + (warp - p.nA) * 2 * slot_bytes;
    return pair + which * slot_bytes;
}
// The one slot of a decoder warp where warps have single slots.
__device__ __forceinline__ uint32_t slot_addr_single(const SmemPlan &p, uint32_t warp, uint32_t slot_bytes) {
    return warp < p.nA ? p.slotA + warp * slot_bytes : p.slotB + (warp - p.nA) * slot_bytes;
}

constexpr int kMaxWarps = 32;
constexpr int kThreads = 1024;   // threads per CTA of the decode kernels (one CTA per SM)
constexpr uint32_t kWaitLimit = 1u << 22;
constexpr uint32_t kErrOverrun = 0x40000000u;     // error flag: this bit + (chunk + 1): the chunk's bits ran past its record
constexpr uint32_t kFeederIdleLimit = 1u << 22;   // polls of 100 ns without any slot coming back before the feeder gives up

}  // namespace huffllm
