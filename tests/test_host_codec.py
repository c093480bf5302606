"""Host side of the library (codebook, encoder, validator) against the CPU oracle.  No GPU needed."""
import ctypes
import os

import numpy as np
import pytest

import paper_2502_00922_b200 as hl
import workloads as wl
from oracle import oracle as orc


def kraft_ok(lens):
    used = [int(l) for l in lens if l]
    return sum(1 << (16 - l) for l in used) == 1 << 16 or used == [1]


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(os.path.dirname(hl.__file__), "..", "include", "huffllm.h")).read()
    import re
    declared = set(re.findall(r"\b(huffllm_[a-z_]+)\s*\(", header))
    assert declared == set(hl.exported_symbols())
    so = ctypes.CDLL(os.path.join(os.path.dirname(hl.__file__), "libhuffllm.so"))
    for name in declared:
        assert getattr(so, name) is not None


DATASETS = {
    "gauss": lambda: wl.gaussian_weights(64, 2048, 0.02, 21),
    "gauss015": lambda: wl.gaussian_weights(64, 2048, 0.015, 22),
    "student": lambda: wl.student_t_weights(128, 1024, 23),
    "uniform": lambda: wl.uniform_exponent_weights(64, 1024, 24),
    "patterns": lambda: wl.all_patterns_weights(64, 2048, 25),
    "constant": lambda: np.full((16, 512), 0x3C12, dtype=np.uint16),
}


@pytest.mark.parametrize("name", sorted(DATASETS))
@pytest.mark.parametrize("budget", [0, 8, 9, 10, 12])
def test_codebook_cost_matches_oracle(name, budget):
    w = DATASETS[name]()
    cb = hl.build_codebook(w, hl.BF16, budget)
    counts = orc.histogram(w)
    olens, ocaps = orc.build_lengths(counts, orc.BF16, budget or 8)
    total = 0
    for f in range(2):
        n, c, lens, codes = cb.get(f)
        assert n == 16 and np.array_equal(c[:16], counts[f][:16])
        assert kraft_ok(lens) and max(lens) <= (budget or 8)
        assert np.array_equal(codes, orc.canonical_codes(lens))           # same canonical rule on both sides
        total += orc.code_cost(c, lens)
    assert total == orc.code_cost(counts[0], olens[0]) + orc.code_cost(counts[1], olens[1])
    cb.free()


@pytest.mark.parametrize("name", sorted(DATASETS))
@pytest.mark.parametrize("budget", [0, 8, 9, 12])
def test_whole_exponent_codebook_cost_matches_oracle(name, budget):
    w = DATASETS[name]()
    cb = hl.build_codebook(w, hl.BF16, budget, hl.SPLIT_WHOLE_EXPONENT)
    counts = orc.histogram(w, orc.BF16_E8)
    olens, ocaps = orc.build_lengths(counts, orc.BF16_E8, budget or 8)
    c, lens, codes = cb.get_exponent()
    assert np.array_equal(c, counts[0])
    assert kraft_ok(lens) and max(lens) <= (budget or 8)
    assert np.array_equal(codes, orc.canonical_codes(lens))
    assert orc.code_cost(c, lens) == orc.code_cost(counts[0], olens[0])
    with pytest.raises(hl.HuffllmError):
        cb.get(0)                                       # the nibble accessor does not apply
    cb.free()
    cb2 = hl.build_codebook(w, hl.BF16, budget)
    with pytest.raises(hl.HuffllmError):
        cb2.get_exponent()
    cb2.free()


@pytest.mark.parametrize("rows,cols,ce,budget,gen,split", [
    (48, 1056, 4096, 8, "gauss", 0), (37, 300, 1024, 8, "student", 0), (16, 256, 4096, 9, "gauss", 0),
    (5, 31, 512, 8, "patterns", 0), (33, 2080, 16384, 8, "gauss", 0), (64, 1024, 4096, 12, "uniform", 0),
    (20, 520, 1024, 10, "patterns", 0), (1, 8, 512, 8, "gauss", 0),
    (48, 1056, 4096, 8, "gauss", 1), (37, 300, 1024, 9, "student", 1), (5, 31, 512, 8, "patterns", 1),
    (64, 1024, 4096, 12, "uniform", 1), (33, 2080, 16384, 8, "gauss", 1)])
def test_blob_decodes_with_oracle_and_bits_match(rows, cols, ce, budget, gen, split):
    w = {"gauss": lambda: wl.gaussian_weights(rows, cols, 0.02, 31),
         "student": lambda: wl.student_t_weights(rows, cols, 32),
         "uniform": lambda: wl.uniform_exponent_weights(rows, cols, 33),
         "patterns": lambda: wl.all_patterns_weights(rows, cols, 34)}[gen]()
    cb = hl.build_codebook(w, hl.BF16, budget, split)
    blob, d = hl.encode(cb, w, ce)
    assert d.n_fields == (2 if split == 0 else 1)
    assert d.blob_bytes == blob.size <= hl.encode_bound(rows, cols, hl.BF16, ce)
    hl.validate_blob(blob)
    back, used = orc.decode_blob(blob)                  # slow reader + bit-serial decoder; checks lag/tail/pad bits
    assert np.array_equal(back, w)
    # the oracle's own encoding with the blob's code lengths gives the same bits, lane by lane
    parsed = orc.parse_blob(blob)
    lens, codes, scheme = parsed["lens"], parsed["codes"], parsed["dtype"]
    assert scheme == (orc.BF16 if split == 0 else orc.BF16_E8)
    flat = np.append(w.ravel(), np.uint16(d.pad_word))
    assert d.pad_word == orc.pad_word(lens, scheme)
    for chunk_ids, idx in orc.element_map(rows, cols, ce):
        n, _, steps = idx.shape
        S = orc.SEQS
        bits, off, raw = orc.encode_sequences(flat[idx.reshape(n * S, steps)], lens, codes, scheme)
        for a, cid in enumerate(chunk_ids):
            pbits, poff, praw = parsed["chunks"][int(cid)]
            per = pbits.reshape(S, -1)
            for l in range(S):
                lo, hi = int(off[a * S + l]), int(off[a * S + l + 1])
                assert int(used[int(cid)][l]) == hi - lo
                assert np.array_equal(per[l, :hi - lo], bits[lo:hi])
            assert np.array_equal(praw, raw[a * S:a * S + S])
    # the LUT is what a bit-serial decode of every index gives
    assert np.array_equal(parsed["lut"], orc.lut_from_code(lens, codes, d.lut_bits, scheme))
    # accounting
    assert d.coded_bits == sum(int(u.sum()) for u in used.values()) and d.raw_bits == 8 * rows * cols
    cb.free()


@pytest.mark.parametrize("split", [0, 1])
def test_validator_rejects_damaged_blobs(split):
    w = wl.gaussian_weights(48, 1056, 0.02, 41)
    cb = hl.build_codebook(w, hl.BF16, 0, split)
    blob, d = hl.encode(cb, w, 4096)
    hl.validate_blob(blob)

    def damaged(offset, xor=0xFF):
        b = blob.copy()
        b[offset] ^= xor
        with pytest.raises(hl.HuffllmError) as e:
            hl.validate_blob(b)
        assert e.value.status_name in ("CORRUPT", "UNSUPPORTED")

    damaged(0)                                   # magic
    damaged(16, 1)                               # rows
    damaged(56, 1)                               # lut_bits
    damaged(76, 1)                               # max_words
    damaged(d.off_codebook + (6 if split == 0 else int(np.argmax(blob[d.off_codebook:d.off_codebook + 256] > 0))), 1)   # a code length
    damaged(d.off_lut + 40, 1)                   # a LUT entry
    damaged(d.off_index + 4, 1)                  # record index
    damaged(d.off_payload + 8 * 512 + 0, 1)      # lag bit of chunk 0 lane 0
    damaged(d.off_payload + 8 * 512 + 200)       # coded bits
    damaged(d.off_payload + d.payload_bytes - 1, 0x80)  # tail padding of the last record
    with pytest.raises(hl.HuffllmError):
        hl.validate_blob(blob[:-128])            # truncated


def test_argument_errors():
    w = wl.gaussian_weights(16, 64, 0.02, 51)
    with pytest.raises(hl.HuffllmError) as e:
        hl.build_codebook(w, 7)
    assert e.value.status_name == "INVALID_ARG"
    with pytest.raises(hl.HuffllmError) as e:
        hl.build_codebook(w, hl.FP16, 0, hl.SPLIT_WHOLE_EXPONENT)
    assert e.value.status_name == "UNSUPPORTED"
    with pytest.raises(hl.HuffllmError) as e:
        hl.build_codebook(w, hl.BF16, 5)
    assert e.value.status_name == "UNSUPPORTED"
    cb = hl.build_codebook(w)
    with pytest.raises(hl.HuffllmError) as e:
        hl.encode(cb, w, 1000)
    assert e.value.status_name == "INVALID_ARG"
    other = wl.uniform_exponent_weights(16, 64, 52, 1, 250)     # uses exponents the codebook never saw
    with pytest.raises(hl.HuffllmError) as e:
        hl.encode(cb, other, 512)
    assert e.value.status_name == "INVALID_ARG" and "codeword" in str(e.value)
    blob, d = hl.encode(cb, w, 512)
    assert hl.workspace_bytes(d, 1) > 0
    with pytest.raises(hl.HuffllmError):
        hl.workspace_bytes(d, 65)


FP16_SETS = {
    "fp16": lambda r, c: wl.gaussian_weights(r, c, 0.02, 71, "fp16"),
    "fp16_from_bf16": lambda r, c: wl.gaussian_weights(r, c, 0.02, 72, "fp16_from_bf16"),
    "patterns": lambda r, c: wl.all_patterns_weights(r, c, 73),
    "constant": lambda r, c: np.full((r, c), 0x2E66, dtype=np.uint16),
}


@pytest.mark.parametrize("name", sorted(FP16_SETS))
@pytest.mark.parametrize("budget", [0, 7, 8, 12])
def test_fp16_codebook_cost_matches_oracle(name, budget):
    """FP16 {1,5,5,5}: three codes, each limited on its own."""
    w = FP16_SETS[name](64, 1024)
    cb = hl.build_codebook(w, hl.FP16, budget)
    counts = orc.histogram(w, orc.FP16)
    olens, ocaps = orc.build_lengths(counts, orc.FP16, budget or 8)
    for f in range(3):
        n, c, lens, codes = cb.get(f)
        assert n == 32 and np.array_equal(c, counts[f][:32])
        assert kraft_ok(lens) and max(lens) <= (budget or 8)
        assert np.array_equal(codes, orc.canonical_codes(lens))
        assert orc.code_cost(c, lens) == orc.code_cost(counts[f], olens[f])
    cb.free()


@pytest.mark.parametrize("rows,cols,ce,budget,gen", [
    (48, 1056, 1024, 8, "fp16"), (37, 300, 1024, 8, "fp16_from_bf16"), (5, 31, 512, 8, "patterns"),
    (33, 2080, 4096, 12, "fp16"), (16, 512, 512, 8, "constant"), (64, 1024, 2048, 9, "fp16_from_bf16"),
    (48, 1056, 1024, 7, "fp16"), (37, 300, 512, 7, "patterns")])
def test_fp16_blob_decodes_with_oracle_and_bits_match(rows, cols, ce, budget, gen):
    w = FP16_SETS[gen](rows, cols)
    cb = hl.build_codebook(w, hl.FP16, budget)
    blob, d = hl.encode(cb, w, ce)
    assert (d.dtype, d.n_fields, d.lag_bits) == (hl.FP16, 3, 6)
    assert d.blob_bytes == blob.size <= hl.encode_bound(rows, cols, hl.FP16, ce)
    hl.validate_blob(blob)
    back, used = orc.decode_blob(blob)
    assert np.array_equal(back, w)
    parsed = orc.parse_blob(blob)
    lens, codes = parsed["lens"], parsed["codes"]
    assert parsed["dtype"] == orc.FP16 and d.pad_word == orc.pad_word(lens, orc.FP16)
    flat = np.append(w.ravel(), np.uint16(d.pad_word))
    for chunk_ids, idx in orc.element_map(rows, cols, ce):
        n, _, steps = idx.shape
        S = orc.SEQS
        bits, off, raw = orc.encode_sequences(flat[idx.reshape(n * S, steps)], lens, codes, orc.FP16)
        for a, cid in enumerate(chunk_ids):
            pbits, poff, praw = parsed["chunks"][int(cid)]
            per = pbits.reshape(S, -1)
            for l in range(S):
                lo, hi = int(off[a * S + l]), int(off[a * S + l + 1])
                assert int(used[int(cid)][l]) == hi - lo
                assert np.array_equal(per[l, :hi - lo], bits[lo:hi])
            assert np.array_equal(praw, raw[a * S:a * S + S])          # sign bits, sequence by sequence
    assert np.array_equal(parsed["lut"], orc.lut_from_code(lens, codes, d.lut_bits, orc.FP16))
    assert d.coded_bits == sum(int(u.sum()) for u in used.values()) and d.raw_bits == rows * cols
    cb.free()


def test_fp16_validator_rejects_damaged_blobs():
    w = wl.gaussian_weights(48, 1056, 0.02, 74, "fp16")
    cb = hl.build_codebook(w, hl.FP16)
    blob, d = hl.encode(cb, w, 1024)
    hl.validate_blob(blob)
    first = int(np.frombuffer(blob.tobytes(), dtype="<u4", count=2, offset=d.off_index)[1]) * 128   # size of record 0

    def damaged(offset, xor=0xFF):
        b = blob.copy()
        b[offset] ^= xor
        with pytest.raises(hl.HuffllmError):
            hl.validate_blob(b)

    damaged(8, 3)                                # dtype
    damaged(60, 2)                               # lag_bits
    damaged(d.off_codebook + 40, 1)              # a code length of the second field
    damaged(d.off_lut + 4 * 300, 1)              # an entry of the second table
    damaged(d.off_payload + 128, 0x01)           # a lag bit of record 0 (its raw part is 2 blocks * 64 bytes)
    damaged(d.off_payload + 128 + 300)           # coded bits
    damaged(d.off_payload + first - 1, 0x80)     # tail padding of record 0


def test_fp16_lands_on_the_papers_bits_per_param():
    # entropy table and Section 5: true fp16 weights ~13.7 bits/param, bf16-origin weights stored as fp16 ~10.96
    for gen, lo, hi in (("fp16", 13.55, 13.9), ("fp16_from_bf16", 10.8, 11.15)):
        w = wl.gaussian_weights(256, 4096, 0.02, 75, gen)
        cb = hl.build_codebook(w, hl.FP16)
        blob, d = hl.encode(cb, w, 4096)
        assert lo <= (d.coded_bits + d.raw_bits) / w.size <= hi
        cb.free()


def test_compression_accounting_on_paper_shaped_weights():
    # Section 5.1: BF16 lands at 11.59-11.68 bits/param on real checkpoints; the synthetic stand-in gives ~11.7-11.8
    w = wl.gaussian_weights(256, 4096, 0.02, 61)
    cb = hl.build_codebook(w)
    blob, d = hl.encode(cb, w, 4096)
    n = w.size
    payload_bits = (d.coded_bits + d.raw_bits) / n
    assert 11.6 <= payload_bits <= 11.9
    total_ratio = 2.0 * n / d.blob_bytes
    assert 1.25 <= total_ratio <= 1.37          # lane padding and side tables cost a few percent


def test_device_call_sizes_are_consistent():
    """Host-only size queries of the device calls: a workspace sized for `batch` vectors serves every smaller batch, its
    control words come first, the static entry point's limits are what the header says, and the shared-memory plan is the
    formula the header states."""
    w = wl.gaussian_weights(528, 4096, 0.02, 91)
    cb = hl.build_codebook(w)
    _, d = hl.encode(cb, w, 4096)
    cb.free()
    sizes = [hl.workspace_bytes(d, b) for b in range(1, 65)]
    assert all(a <= b for a, b in zip(sizes, sizes[1:]))
    ctrl = hl.workspace_control_bytes(d)
    assert 4096 <= ctrl < sizes[0] and ctrl % 256 == 0
    assert sizes[hl.STATIC_MAX_BATCH - 1] <= 1 << 20                # fits the static entry point's built-in array
    plan = hl.decode_smem_plan(d)
    assert plan["slot_bytes"] == d.max_words * 256
    assert plan["guard_bytes"] == 256 * (3 + plan["refill_checks_per_block"] * (d.chunk_cols // 32))
    assert plan["table_bytes"] == 128 << 8
    with pytest.raises(hl.HuffllmError):
        hl.workspace_bytes(d, 65)


def test_launch_plan_slots_per_warp():
    """Two slots per decoder warp where 31 pairs fit, one where records are large: the plan of a decoder CTA as the library
    reports it (host only), checked against the shared-memory arithmetic of the header."""
    smem = 232448
    for dtype, name, ce, slots in ((hl.BF16, "bf16", 4096, 2), (hl.BF16, "bf16", 8192, 1), (hl.FP16, "fp16", 1024, 2),
                                   (hl.FP16, "fp16", 4096, 1), (hl.FP16, "fp16", 16384, 1)):
        w = wl.gaussian_weights(64, 4096, 0.02, 94, name)
        cb = hl.build_codebook(w, dtype)
        _, d = hl.encode(cb, w, ce)
        cb.free()
        sp = hl.decode_smem_plan(d)
        for batch in (0, 1, 8):
            plan = hl.decode_launch_plan(d, batch)
            assert plan["slots_per_warp"] == slots, (name, ce, batch, plan)
            assert 1 <= plan["decoder_warps"] <= 31
            # the reported warps fit: their slots, the table(s) and the guard area lie inside a CTA's shared memory
            assert plan["decoder_warps"] * slots * sp["slot_bytes"] + sp["table_bytes"] + sp["guard_bytes"] <= smem
            if slots == 2:
                assert plan["decoder_warps"] == 31
            else:   # single slots serve more warps than pairs would
                assert plan["decoder_warps"] > (smem - sp["table_bytes"] - sp["guard_bytes"]) // (2 * sp["slot_bytes"]) or plan["decoder_warps"] == 31
        try:     # less shared memory: fewer warps, or no launch at all
            assert hl.decode_launch_plan(d, 1, 100 * 1024)["decoder_warps"] <= hl.decode_launch_plan(d, 1)["decoder_warps"]
        except hl.HuffllmError as e:
            assert "too large for shared memory" in str(e)
        with pytest.raises(hl.HuffllmError):
            hl.decode_launch_plan(d, 9)


def test_flat_fields_mark_exactly_the_flat_codes():
    """FP16 blobs: the descriptor marks the fields whose code is the flat one (all 32 symbols at 5 bits, codeword = symbol):
    both mantissa halves of fp16-trained weights, only the upper half of bf16-trained weights stored as fp16, none of
    skewed data; BF16 blobs never.  A mark on a field whose code is not flat is refused by the validator, no mark at all
    is always accepted (the decoders then use the tables)."""
    cases = [("fp16", 0b110), ("fp16_from_bf16", 0b010)]
    for name, want in cases:
        w = wl.gaussian_weights(64, 4096, 0.02, 95, name)
        cb = hl.build_codebook(w, hl.FP16)
        lens = [cb.get(f)[2] for f in range(3)]
        blob, d = hl.encode(cb, w, 1024)
        cb.free()
        flat = sum(1 << f for f in range(3) if all(int(l) == 5 for l in lens[f][:32]))
        assert d.flat_fields == flat == want, (name, d.flat_fields, flat)
        # the codewords of a flat field are the symbols themselves (canonical code), which is what lets a decoder skip its table
        parsed = orc.parse_blob(blob)
        assert parsed["header"]["_r"] == want
        hl.validate_blob(blob)
        unmarked = blob.copy()
        unmarked[74:76] = 0
        assert hl.validate_blob(unmarked).flat_fields == 0
        wrong = blob.copy()
        wrong[74] = 0b111                      # the exponent's code is never flat on these weights
        with pytest.raises(hl.HuffllmError):
            hl.validate_blob(wrong)
    w = wl.skewed_exponent_weights(64, 1024, 96, dtype="fp16")
    cb = hl.build_codebook(w, hl.FP16)
    _, d = hl.encode(cb, w, 1024)
    cb.free()
    assert d.flat_fields == 0
    w = wl.gaussian_weights(64, 1024, 0.02, 97)
    cb = hl.build_codebook(w)
    blob, d = hl.encode(cb, w, 1024)
    cb.free()
    assert d.flat_fields == 0
    bad = blob.copy()
    bad[74] = 2
    with pytest.raises(hl.HuffllmError):
        hl.validate_blob(bad)


def test_code_length_limits_accepted_per_format():
    """BF16 budgets 8..12 (the two nibble codes of a weight together); FP16 field limits 7..12."""
    wb = wl.gaussian_weights(16, 512, 0.02, 92)
    wh = wl.gaussian_weights(16, 512, 0.02, 93, "fp16")
    for b in (8, 9, 10, 11, 12):
        hl.build_codebook(wb, hl.BF16, b).free()
    for b in (7, 8, 12):
        hl.build_codebook(wh, hl.FP16, b).free()
    for dt, w, b in ((hl.BF16, wb, 7), (hl.BF16, wb, 13), (hl.FP16, wh, 6), (hl.FP16, wh, 13)):
        with pytest.raises(hl.HuffllmError) as e:
            hl.build_codebook(w, dt, b)
        assert e.value.status_name == "UNSUPPORTED"
