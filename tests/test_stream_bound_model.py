"""How far can damaged bits drive the device decoders?  (CPU only.)

The kernels read a chunk's coded rows from a shared-memory slot and never check a bit sequence against its length
inside the hot loop; what keeps a damaged blob from reading outside the CTA's shared memory is structural: a sequence
opens on rows 0 and 1 of its slot and every refill check moves its row pointer by at most one row, whatever the window
holds and whatever the decode table returns.  The library therefore keeps 256 * (3 + checks * blocks) readable bytes
behind the last slot (huffllm_decode_smem_plan).

This file restates the pointer arithmetic of the four decoders (window, position, refill rule, position advance) in
plain Python, drives it with random and with adversarial windows and tables, and asserts that the furthest row ever
addressed stays inside slot + guard as the library computes them, for every format, table size and chunk size, and
that every table address stays inside the table.  It models addresses only: the decoded values are not its subject.
"""
import numpy as np
import pytest

import workloads as wl

M32 = 0xFFFFFFFF


class Rows:
    """A slot's column of one sequence: row j of the record is word j of the sequence.  Rows beyond the record read as
    whatever lies there (random); the furthest row asked for is remembered."""

    def __init__(self, rng, mode):
        self.rng, self.mode, self.furthest = rng, mode, -1

    def read(self, row):
        assert row >= 0
        self.furthest = max(self.furthest, row)
        if self.mode == "ones":
            return M32
        if self.mode == "zeros":
            return 0
        return int(self.rng.integers(0, 1 << 32))


class Table:
    """A decode table of `entries` 32-bit words, sound or damaged; every index is checked against its size."""

    def __init__(self, rng, entries, mode):
        self.entries, self.mode, self.rng = entries, mode, rng
        self.words = rng.integers(0, 1 << 32, size=entries, dtype=np.uint64)

    def get(self, idx):
        assert 0 <= idx < self.entries, "table address outside the table"
        if self.mode == "max":
            return M32
        if self.mode == "adv":       # every entry drives the pointer over a word boundary before the next check
            return (64 << 16) | 8
        if self.mode == "zero":
            return 0
        return int(self.words[idx])


def run_bf16_four_at_a_time(rows, tab, blocks):
    """8-bit BF16 tables: the pointer starts behind the 7 leading bits; per round of four codewords one check of bit 5
    of the pointer; lookups by the window's low byte, in-place shifts by an entry's low 5 bits, the pointer advanced by
    the sum of the four whole entries (wrapping)."""
    lo, hi, nxt, pos, checks = rows.read(0), rows.read(1), 2, 7, 0
    for _ in range(blocks * 2):                      # two rounds of four codewords per block and sequence
        checks += 1
        if pos & 32:
            lo, hi = rows.read(nxt - 1), rows.read(nxt)
            nxt += 1
            pos = (pos - 32) & M32
        t = (((hi << 32) | lo) >> (pos & 31)) & M32
        total = 0
        for _ in range(4):
            e = tab.get(t & 0xFF)
            total += e
            t >>= e & 31
        pos = (pos + total) & M32
    return checks


def run_pointer_based(rows, tab, blocks, steps_per_check, index_bits, long_bits=0, long_tab=None):
    """Tables of 9 bits, and of 10..12 bits through two levels: a 64-bit window shifted by the pointer, a check
    (pointer >= 32) before every `steps_per_check`-th codeword, the pointer advanced by byte 2 of the entry."""
    lo, hi, nxt, pos, checks = rows.read(0), rows.read(1), 2, 0, 0
    for i in range(blocks * 8):
        if i % steps_per_check == 0:
            checks += 1
            if pos >= 32:
                lo, hi = rows.read(nxt - 1), rows.read(nxt)
                nxt += 1
                pos = (pos - 32) & M32
        t = (((hi << 32) | lo) >> pos) & M32 if pos < 64 else 0
        e = tab.get((t >> 7) & ((1 << index_bits) - 1))
        if long_bits and e & 0x80000000:
            e = long_tab.get((t >> 7) & ((1 << long_bits) - 1))
        pos = (pos + ((e >> 16) & 0xFF)) & M32
    return checks


def run_fp16(rows, tabs, blocks, long_bits=0, long_tabs=None):
    """FP16 {1,5,5,5}: three lookups per weight (index = 8 window bits behind a lag of 6); one check per weight, or,
    with field codes above 8 bits, one before every field; a refill keeps the high word and loads one new row."""
    lo, hi, nxt, pos, checks = rows.read(0), rows.read(1), 2, 0, 0
    for _ in range(blocks * 8):
        for f in range(3):
            if long_bits or f == 0:
                checks += 1
                if pos >= 32:
                    lo, hi = hi, rows.read(nxt)
                    nxt += 1
                    pos = (pos - 32) & M32
            t = (((hi << 32) | lo) >> pos) & M32 if pos < 64 else 0
            e = tabs[f].get((t >> 6) & 0xFF)
            if long_bits and e & 0x80000000:
                e = long_tabs[f].get((t >> 6) & ((1 << long_bits) - 1))
            pos = (pos + ((e >> 16) & 0xFF)) & M32
    return checks


CASES = [(dtype, bits, ce) for dtype in ("bf16", "fp16") for bits in (8, 9, 10, 12) for ce in (512, 1024, 4096, 16384)]


@pytest.mark.parametrize("dtype,bits,chunk_elems", CASES)
def test_no_stream_and_no_table_can_drive_a_decoder_past_the_guard(dtype, bits, chunk_elems):
    import paper_2502_00922_b200 as hl
    w = (wl.gaussian_weights(16, chunk_elems // 16, 0.02, 3, "fp16") if dtype == "fp16"
         else wl.skewed_exponent_weights(16, chunk_elems // 16, 3))
    cb = hl.build_codebook(w, hl.FP16 if dtype == "fp16" else hl.BF16, bits)
    _, desc = hl.encode(cb, w, chunk_elems)
    cb.free()
    assert desc.lut_bits == bits
    plan = hl.decode_smem_plan(desc)
    blocks = desc.chunk_cols // 32
    assert plan["slot_bytes"] == desc.max_words * 256
    assert plan["guard_bytes"] == 256 * (3 + plan["refill_checks_per_block"] * blocks)
    rng = np.random.default_rng(bits * 1000 + chunk_elems)
    worst = 0
    for stream_mode in ("random", "ones", "zeros"):
        for table_mode in ("random", "max", "zero", "adv"):
            for trial in range(3 if stream_mode == table_mode == "random" else 1):
                rows = Rows(rng, stream_mode)
                if dtype == "bf16" and bits == 8:
                    checks = run_bf16_four_at_a_time(rows, Table(rng, 256, table_mode), blocks)
                elif dtype == "bf16" and bits == 9:
                    checks = run_pointer_based(rows, Table(rng, 512, table_mode), blocks, 2, 9)
                elif dtype == "bf16":
                    checks = run_pointer_based(rows, Table(rng, 256, table_mode), blocks, 2, 8, bits, Table(rng, 1 << bits, table_mode))
                elif bits == 8:
                    checks = run_fp16(rows, [Table(rng, 256, table_mode) for _ in range(3)], blocks)
                else:
                    checks = run_fp16(rows, [Table(rng, 256, table_mode) for _ in range(3)], blocks, bits,
                                      [Table(rng, 1 << bits, table_mode) for _ in range(3)])
                # what the restated arithmetic does per block is what the library budgets for, or less
                assert checks <= plan["refill_checks_per_block"] * blocks
                # one row per check, from rows 0 and 1
                assert rows.furthest <= 1 + checks
                worst = max(worst, rows.furthest)
    # the furthest row lies inside slot + guard even for the smallest slot a record can have (one row), and for the last
    # slot of the CTA, behind which only the guard bytes are promised
    assert (worst + 1) * 256 <= 256 + plan["guard_bytes"]
    assert (worst + 1) * 256 <= plan["slot_bytes"] + plan["guard_bytes"]
    # the adversarial cases do reach the bound's order of magnitude: the budget is not idle
    assert worst >= blocks
