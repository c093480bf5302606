"""Pins for the CPU oracle: every check compares it with something fixed by the paper or by
mathematics (closed forms, brute force, invariants), never with itself or with the CUDA path."""
import itertools
import math
import os

import numpy as np
import pytest

import workloads as wl
from oracle import oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def kraft_num(lens, L=32):
    return sum(1 << (L - int(l)) for l in lens if l)


def brute_force_cost(counts, cap):
    """Minimum of sum(count*len) over all length vectors with Kraft sum <= 1 and len <= cap."""
    used = [int(c) for c in counts if c > 0]
    best = None
    for lens in itertools.product(range(1, cap + 1), repeat=len(used)):
        if sum(2.0 ** -l for l in lens) <= 1.0 + 1e-12:
            c = sum(a * b for a, b in zip(used, lens))
            best = c if best is None or c < best else best
    return best


def entropy_bits(counts):
    c = np.asarray([x for x in counts if x > 0], dtype=np.float64)
    p = c / c.sum()
    return float(-(p * np.log2(p)).sum())


# ------------------------------------------------------------------ lengths

def test_kraft_equality_random_counts():
    rng = np.random.default_rng(1)
    for trial in range(200):
        n = int(rng.integers(2, 33))
        counts = np.zeros(32, dtype=np.uint64)
        counts[rng.choice(32, n, replace=False)] = rng.integers(1, 10 ** int(rng.integers(1, 8)), n)
        lens = orc.huffman_lengths(counts)
        assert kraft_num(lens) == 1 << 32
        assert all((l > 0) == (c > 0) for l, c in zip(lens, counts))
        cap = max(int(math.ceil(math.log2(n))), int(rng.integers(3, 13)))
        lim = orc.limited_lengths(counts, cap)
        assert kraft_num(lim) == 1 << 32 and max(lim) <= cap


@pytest.mark.parametrize("n", [2, 3, 4, 5, 6, 7])
def test_lengths_are_brute_force_optimal(n):
    rng = np.random.default_rng(10 + n)
    for trial in range(12 if n < 7 else 3):
        counts = np.zeros(16, dtype=np.uint64)
        hi = [3, 20, 1000][trial % 3]
        counts[rng.choice(16, n, replace=False)] = rng.integers(1, hi, n)
        lens = orc.huffman_lengths(counts)
        assert orc.code_cost(counts, lens) == brute_force_cost(counts, n)       # depth never exceeds n-1
        for cap in range(max(1, math.ceil(math.log2(n))), n + 1):
            lim = orc.limited_lengths(counts, cap)
            assert max(lim) <= cap
            assert orc.code_cost(counts, lim) == brute_force_cost(counts, cap)


def test_closed_forms():
    # dyadic counts: length = log2(total / count), average length equals the entropy exactly
    counts = np.zeros(16, dtype=np.uint64)
    counts[[3, 5, 7, 9, 11]] = [8, 4, 2, 1, 1]
    lens = orc.huffman_lengths(counts)
    assert [int(lens[s]) for s in (3, 5, 7, 9, 11)] == [1, 2, 3, 4, 4]
    assert orc.code_cost(counts, lens) / 16 == pytest.approx(entropy_bits(counts), abs=1e-12)
    # uniform over 16 symbols: every length 4, with or without a cap of 4
    u = np.full(16, 5, dtype=np.uint64)
    assert list(orc.huffman_lengths(u)) == [4] * 16 and list(orc.limited_lengths(u, 4)) == [4] * 16
    # Fibonacci counts: the deepest possible tree
    f = np.zeros(16, dtype=np.uint64)
    f[:8] = [1, 1, 2, 3, 5, 8, 13, 21]
    assert list(orc.huffman_lengths(f)[:8]) == [7, 7, 6, 5, 4, 3, 2, 1]
    # two symbols, one symbol, none
    t = np.zeros(16, dtype=np.uint64); t[[2, 9]] = [1, 1000]
    assert [int(x) for x in orc.huffman_lengths(t)[[2, 9]]] == [1, 1]
    o = np.zeros(16, dtype=np.uint64); o[4] = 7
    assert int(orc.huffman_lengths(o)[4]) == 1 and int(orc.huffman_lengths(o).sum()) == 1
    assert int(orc.huffman_lengths(np.zeros(16, dtype=np.uint64)).sum()) == 0
    assert orc.limited_lengths(u, 3) is None                                    # 16 symbols need 4 bits


def test_entropy_bounds_and_cap_monotone():
    rng = np.random.default_rng(3)
    for trial in range(50):
        counts = rng.integers(0, 10 ** int(rng.integers(1, 7)), 32).astype(np.uint64)
        if (counts > 0).sum() < 2:
            continue
        n = int(counts.sum())
        lens = orc.huffman_lengths(counts)
        avg, H = orc.code_cost(counts, lens) / n, entropy_bits(counts)
        assert H - 1e-9 <= avg < H + 1
        prev = None
        for cap in range(5, int(max(lens)) + 3):
            c = orc.code_cost(counts, orc.limited_lengths(counts, cap))
            assert c >= orc.code_cost(counts, lens)
            assert prev is None or c <= prev
            if cap >= max(lens):
                assert c == orc.code_cost(counts, lens)
            prev = c


def test_canonical_codes_prefix_free_and_ordered():
    rng = np.random.default_rng(4)
    for trial in range(40):
        counts = rng.integers(0, 1000, 32).astype(np.uint64)
        counts[rng.integers(0, 32)] += 1
        counts[(rng.integers(0, 31) + 1)] += 1
        lens = orc.huffman_lengths(counts)
        codes = orc.canonical_codes(lens)
        words = {s: format(int(codes[s]), "0{}b".format(int(lens[s]))) for s in range(32) if lens[s]}
        assert all(len(v) == lens[s] for s, v in words.items())                 # code fits its length
        for a, b in itertools.permutations(words.values(), 2):
            assert not b.startswith(a)
        order = sorted(words, key=lambda s: (int(lens[s]), s))
        vals = [int(words[s].ljust(32, "0"), 2) for s in order]                 # left-justified values increase
        assert vals == sorted(vals) and len(set(vals)) == len(vals)
        assert int(codes[order[0]]) == 0


def test_joint_budget_is_best_split_bf16():
    rng = np.random.default_rng(5)
    for trial in range(10):
        counts = np.zeros((3, orc.MAXSYM), dtype=np.uint64)
        n0, n1 = int(rng.integers(1, 5)), int(rng.integers(2, 7))
        counts[0, rng.choice(16, n0, replace=False)] = rng.integers(1, 50, n0)
        counts[1, rng.choice(16, n1, replace=False)] = rng.integers(1, 50, n1)
        for budget in (4, 5, 6, 8):
            best = None
            for c0 in range(1, budget):
                c1 = budget - c0
                if (n0 > 1 and 2 ** c0 < n0) or (n1 > 1 and 2 ** c1 < n1):
                    continue
                a = brute_force_cost(counts[0], c0) if n0 > 1 else int(counts[0].sum())
                b = brute_force_cost(counts[1], c1) if n1 > 1 else int(counts[1].sum())
                best = a + b if best is None else min(best, a + b)
            if best is None:
                with pytest.raises(ValueError):
                    orc.build_lengths(counts, orc.BF16, budget)
                continue
            lens, caps = orc.build_lengths(counts, orc.BF16, budget)
            assert caps[0] + caps[1] <= budget and max(lens[0]) <= caps[0] and max(lens[1]) <= caps[1]
            assert orc.code_cost(counts[0], lens[0]) + orc.code_cost(counts[1], lens[1]) == best
        nat, _ = orc.build_lengths(counts, orc.BF16, 0)
        assert list(nat[0]) == list(orc.huffman_lengths(counts[0])) and list(nat[1]) == list(orc.huffman_lengths(counts[1]))


# ------------------------------------------------------------ worked example

def read_golden(name):
    out = {}
    for line in open(os.path.join(GOLD, name)):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        out[k] = v
    return out


def test_worked_example_bf16():
    g = read_golden("worked_example_bf16.txt")
    w = np.array([int(x, 16) for x in g["weights_hex"]], dtype=np.uint16)
    counts = orc.histogram(w)
    lens, _ = orc.build_lengths(counts, orc.BF16, 0)
    codes = orc.codes_for(lens)
    for field, key in ((0, "hi"), (1, "lo")):
        syms = [int(s, 16) for s in g[key + "_symbols"]]
        assert [int(lens[field][s]) for s in syms] == [int(x) for x in g[key + "_lengths"]]
        assert [format(int(codes[field][s]), "0{}b".format(int(lens[field][s]))) for s in syms] == g[key + "_codes"]
        assert int((lens[field] > 0).sum()) == len(syms)
    bits, off, raw = orc.encode_sequences(w[None, :], lens, codes)
    assert "".join(map(str, bits)) == g["bitstream"][0]
    assert [int(x) for x in raw[0]] == [int(x, 16) for x in g["raw_hex"]]
    assert len(bits) + 8 * 8 == int(g["payload_bits"][0])
    back, used = orc.decode_sequences(bits, off, raw, lens, codes)
    assert np.array_equal(back[0], w) and int(used[0]) == len(bits)
    y, d = orc.matmul(w[None, :], np.full((1, 8), 0x3F80, dtype=np.uint16))
    assert y[0, 0] == float(g["y"][0]) and d[0, 0] == float(g["abs_sum"][0])


def test_worked_example_fp16():
    g = read_golden("worked_example_fp16.txt")
    w = np.array([int(x, 16) for x in g["weights_hex"]], dtype=np.uint16)
    counts = orc.histogram(w, orc.FP16)
    lens, _ = orc.build_lengths(counts, orc.FP16, 0)
    codes = orc.codes_for(lens)
    for field, key in ((0, "exp"), (1, "mhi"), (2, "mlo")):
        syms = [int(s, 16) for s in g[key + "_symbols"]]
        assert [int(lens[field][s]) for s in syms] == [int(x) for x in g[key + "_lengths"]]
        assert [format(int(codes[field][s]), "0{}b".format(int(lens[field][s]))) for s in syms] == g[key + "_codes"]
        assert int((lens[field] > 0).sum()) == len(syms)
    bits, off, raw = orc.encode_sequences(w[None, :], lens, codes, orc.FP16)
    assert "".join(map(str, bits)) == g["bitstream"][0]
    assert [int(x) for x in raw[0]] == [int(x) for x in g["raw_bits"]]
    assert len(bits) + 8 == int(g["payload_bits"][0])
    back, used = orc.decode_sequences(bits, off, raw, lens, codes, orc.FP16)
    assert np.array_equal(back[0], w) and int(used[0]) == len(bits)
    y, d = orc.matmul(w[None, :], np.full((1, 8), 0x3C00, dtype=np.uint16), orc.FP16)
    assert y[0, 0] == float(g["y"][0]) and d[0, 0] == float(g["abs_sum"][0])


def test_worked_example_bf16_whole_exponent():
    g = read_golden("worked_example_bf16_whole_exponent.txt")
    w = np.array([int(x, 16) for x in g["weights_hex"]], dtype=np.uint16)
    counts = orc.histogram(w, orc.BF16_E8)
    lens, _ = orc.build_lengths(counts, orc.BF16_E8, 0)
    codes = orc.codes_for(lens)
    syms = [int(s, 16) for s in g["exp_symbols"]]
    assert [int(lens[0][s]) for s in syms] == [int(x) for x in g["exp_lengths"]]
    assert [format(int(codes[0][s]), "0{}b".format(int(lens[0][s]))) for s in syms] == g["exp_codes"]
    assert int((lens[0] > 0).sum()) == len(syms) and not lens[1:].any()
    bits, off, raw = orc.encode_sequences(w[None, :], lens, codes, orc.BF16_E8)
    assert "".join(map(str, bits)) == g["bitstream"][0]
    assert [int(x) for x in raw[0]] == [int(x, 16) for x in g["raw_hex"]]
    assert len(bits) + 8 * 8 == int(g["payload_bits"][0])
    back, used = orc.decode_sequences(bits, off, raw, lens, codes, orc.BF16_E8)
    assert np.array_equal(back[0], w) and int(used[0]) == len(bits)


def test_whole_exponent_split_against_the_nibble_split():
    """{1,8,7} codes the same exponent byte as {1,4,4,7}: same raw bytes, same decoded words, and its entropy is at
    most the sum of the nibble entropies, so its Huffman cost is below the nibble cost + 1 bit per weight."""
    w = wl.gaussian_weights(256, 1024, 0.02, 11)
    c2, c1 = orc.histogram(w, orc.BF16), orc.histogram(w, orc.BF16_E8)
    assert int(c1[0].sum()) == w.size and not c1[1:].any()
    # the byte histogram folds into the two nibble histograms
    assert np.array_equal(c1[0].reshape(16, 16).sum(axis=1), c2[0][:16])
    assert np.array_equal(c1[0].reshape(16, 16).sum(axis=0), c2[1][:16])
    l2, _ = orc.build_lengths(c2, orc.BF16, 0)
    l1, _ = orc.build_lengths(c1, orc.BF16_E8, 0)
    p = c1[0][c1[0] > 0].astype(np.float64) / w.size
    H = float(-(p * np.log2(p)).sum())
    avg1 = orc.code_cost(c1[0], l1[0]) / w.size
    avg2 = (orc.code_cost(c2[0], l2[0]) + orc.code_cost(c2[1], l2[1])) / w.size
    assert H <= avg1 < H + 1 and avg1 < avg2
    assert abs((8 + avg1) - 10.7) < 0.2                    # about one bit per weight below the nibble split's 11.7
    for budget in (8, 9, 12):
        lb, caps = orc.build_lengths(c1, orc.BF16_E8, budget)
        assert max(lb[0]) <= budget and caps[0] == budget and kraft_num(lb[0]) == 1 << 32
        assert orc.code_cost(c1[0], lb[0]) >= orc.code_cost(c1[0], l1[0])
    bits, off, raw = orc.encode_sequences(w.reshape(64, -1), l1, orc.codes_for(l1), orc.BF16_E8)
    _, _, raw2 = orc.encode_sequences(w.reshape(64, -1), l2, orc.codes_for(l2), orc.BF16)
    assert np.array_equal(raw, raw2)


# ----------------------------------------------------------------- lossless

@pytest.mark.parametrize("dtype", [orc.BF16, orc.FP16, orc.BF16_E8])
def test_every_pattern_round_trips(dtype):
    w = wl.all_patterns_weights(64, 2048, seed=7)                                # 2 x all 65536 patterns
    counts = orc.histogram(w, dtype)
    for budget in (0, 12) if dtype != orc.BF16 else (0, 8, 10, 12):
        lens, caps = orc.build_lengths(counts, dtype, budget)
        codes = orc.codes_for(lens)
        bits, off, raw = orc.encode_sequences(w.reshape(16, -1), lens, codes, dtype)
        back, used = orc.decode_sequences(bits, off, raw, lens, codes, dtype)
        assert np.array_equal(back.reshape(w.shape), w)
        assert np.array_equal(used, np.diff(off))
        nf = orc.num_fields(dtype)
        assert len(bits) == sum(orc.code_cost(counts[k], lens[k]) for k in range(nf))


def test_field_split_definitions():
    # BF16 1-8-7 and FP16 1-5-10 bit positions (Section 2.1), nibble / 5-bit groups (Sections 3.1, 5.1)
    c = orc.histogram(np.array([0xC0FF], dtype=np.uint16), orc.BF16)             # s=1 E=0x81 m=0x7F
    assert c[0][8] == 1 and c[1][1] == 1 and c.sum() == 2
    _, _, raw = orc.encode_sequences(np.array([[0xC0FF, 0x3F80]], dtype=np.uint16), *one_bit_code(c, [0x3F80]))
    assert list(raw[0]) == [0xFF, 0x00]
    c = orc.histogram(np.array([0xB6B5], dtype=np.uint16), orc.FP16)             # s=1 E=01101 M=10101 10101
    assert c[0][0b01101] == 1 and c[1][0b10101] == 1 and c[2][0b10101] == 1 and c.sum() == 3


def one_bit_code(c, extra):
    counts = orc.histogram(np.array([0xC0FF] + extra, dtype=np.uint16))
    lens, _ = orc.build_lengths(counts, orc.BF16, 0)
    return lens, orc.codes_for(lens)


@pytest.mark.parametrize("rows,cols,ce", [(16, 256, 4096), (37, 300, 1024), (48, 1056, 4096), (5, 31, 512), (33, 2080, 16384)])
def test_element_map_is_a_bijection(rows, cols, ce):
    seen = np.zeros(rows * cols, dtype=np.int32)
    geo = orc.geometry(rows, cols, ce)
    n_chunks = 0
    for chunk_ids, idx in orc.element_map(rows, cols, ce):
        n_chunks += len(chunk_ids)
        np.add.at(seen, idx[idx >= 0], 1)
        # a sequence's 8 steps of one block are 8 consecutive columns of one row
        a = idx[0].reshape(orc.SEQS, -1, 8)
        ok = a[..., 0] >= 0
        full = ok & (a[..., 7] >= 0)
        assert np.all((a[..., 7] - a[..., 0])[full] == 7)
    assert np.all(seen == 1) and n_chunks == geo["RG"] * geo["KC"]


@pytest.mark.parametrize("gen", ["gauss", "student", "uniform", "patterns", "constant", "two"])
def test_tensor_round_trip(gen):
    rows, cols = 40, 1100                                                       # ragged in both directions
    w = {"gauss": lambda: wl.gaussian_weights(rows, cols, 0.02, 1),
         "student": lambda: wl.student_t_weights(rows, cols, 2),
         "uniform": lambda: wl.uniform_exponent_weights(rows, cols, 3),
         "patterns": lambda: wl.all_patterns_weights(rows, cols, 4),
         "constant": lambda: np.full((rows, cols), 0x3C12, dtype=np.uint16),
         "two": lambda: np.where(np.arange(rows * cols).reshape(rows, cols) % 3 == 0, 0x3F80, 0xBB00).astype(np.uint16)}[gen]()
    for ce, budget in ((1024, 8), (4096, 10)):
        enc = orc.encode_tensor(w, ce, budget)
        assert np.array_equal(orc.decode_tensor(enc), w)


# ----------------------------------------------------------- paper's numbers

def bits_per_param(w, dtype):
    counts = orc.histogram(w, dtype)
    lens, _ = orc.build_lengths(counts, dtype, 0)
    nf = orc.num_fields(dtype)
    coded = [orc.code_cost(counts[k], lens[k]) / w.size for k in range(nf)]
    ent = [entropy_bits(counts[k]) for k in range(nf)]
    return orc.lib().orc_raw_bits(dtype) + sum(coded), coded, ent


def test_synthetic_weights_land_on_the_papers_table():
    # Section 5.1 compression table: BF16 11.59-11.68 bits/param for every family; FP16 10.88-10.96 for
    # bf16-origin families and 13.68-13.78 for the others.  Section 3.1 entropy table (1-5-5-5 row):
    # 2.60 / 4.97 / 2.04.  Real checkpoints are unavailable, so these are soft pins on synthetic stand-ins.
    w = wl.gaussian_weights(1024, 4096, 0.02, 11, "bf16")
    total, coded, ent = bits_per_param(w, orc.BF16)
    assert 11.55 <= total <= 11.85 and coded[0] < 1.05 and 2.6 < coded[1] < 2.85
    w = wl.gaussian_weights(1024, 4096, 0.02, 11, "fp16_from_bf16")
    total, coded, ent = bits_per_param(w, orc.FP16)
    assert 10.8 <= total <= 11.1
    assert abs(ent[0] - 2.60) < 0.15 and abs(ent[1] - 4.97) < 0.05 and abs(ent[2] - 2.04) < 0.1
    w = wl.gaussian_weights(1024, 4096, 0.02, 11, "fp16")
    total, _, _ = bits_per_param(w, orc.FP16)
    assert 13.6 <= total <= 13.85


# ------------------------------------------------------------------ products

def test_values_of_special_patterns():
    assert orc.value(0x3F80) == 1.0 and orc.value(0xC000) == -2.0 and orc.value(0x0000) == 0.0
    assert orc.value(0x0001) == 2.0 ** -133 and orc.value(0x0080) == 2.0 ** -126
    assert orc.value(0x7F80) == math.inf and orc.value(0xFF80) == -math.inf and math.isnan(orc.value(0x7FC1))
    assert orc.value(0x3C00, orc.FP16) == 1.0 and orc.value(0x0001, orc.FP16) == 2.0 ** -24
    assert orc.value(0x7BFF, orc.FP16) == 65504.0 and orc.value(0xFC00, orc.FP16) == -math.inf
    # every finite bf16 pattern against an independent widening (bit shift into float32)
    allb = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    with np.errstate(invalid="ignore"):
        f = wl.bf16_bits_to_f32(allb).astype(np.float64)
    mine = np.array([orc.value(int(b)) for b in allb[::97]])
    ref = f[::97]
    assert np.array_equal(np.isnan(mine), np.isnan(ref)) and np.array_equal(mine[~np.isnan(ref)], ref[~np.isnan(ref)])
    h = allb.view(np.float16).astype(np.float64)[::97]
    mine = np.array([orc.value(int(b), orc.FP16) for b in allb[::97]])
    assert np.array_equal(mine[~np.isnan(h)], h[~np.isnan(h)])


def test_matmul_closed_forms():
    rows, cols = 24, 352
    one = np.full((rows, cols), 0x3F80, dtype=np.uint16)
    y, d = orc.matmul(one, np.full((1, cols), 0x3F80, dtype=np.uint16))
    assert np.all(y == cols) and np.all(d == cols)
    w = wl.gaussian_weights(rows, cols, 0.02, 5)
    wf = wl.bf16_bits_to_f32(w).astype(np.float64)
    for k in (0, 17, cols - 1):                                                 # one-hot x picks a column
        x = np.zeros((1, cols), dtype=np.uint16); x[0, k] = 0x3F80
        y, _ = orc.matmul(w, x)
        assert np.array_equal(y[0], wf[:, k])
    x = wl.activations(3, cols, 6)
    xf = wl.bf16_bits_to_f32(x).astype(np.float64)
    y, d = orc.matmul(w, x)
    assert np.allclose(y, xf @ wf.T, rtol=0, atol=1e-12) and np.allclose(d, np.abs(xf) @ np.abs(wf).T, rtol=1e-12)
    yn, _ = orc.matmul(w, x ^ np.uint16(0x8000))                                # y(-x) = -y
    assert np.array_equal(yn, -y)
    # a transposed operand would fail this: non-square, distinct rows
    assert y.shape == (3, rows) and not np.allclose(y[0], y[1])
    # powers of two: exact small sums
    p = np.array([[0x4000, 0x3F00, 0x3E80, 0xBF80]], dtype=np.uint16)           # 2, .5, .25, -1
    y, d = orc.matmul(p, np.array([[0x3F80, 0x4000, 0x4080, 0x3F80]], dtype=np.uint16))  # 1 2 4 1
    assert y[0, 0] == 2 + 1 + 1 - 1 and d[0, 0] == 5


# ------------------------------------------------------------------ bit-field splits (Section 3.1 entropy table)

def test_split_entropy_hand_sample():
    g = read_golden("entropy_table_section3_1.txt")
    w = np.array([int(x, 16) for x in g["sample_hex"]], dtype=np.uint16)
    widths = [int(x) for x in g["sample_widths"]]
    per_field, total = orc.split_entropy(w, widths)
    want = [float(x) for x in g["sample_entropy"]]
    assert per_field == pytest.approx(want, abs=1e-12) and total == pytest.approx(sum(want), abs=1e-12)
    h = orc.split_histograms(w, widths)
    assert [int(h[0][1]), int(h[0][2]), int(h[1][2]), int(h[1][3])] == [6, 2, 4, 4]
    assert [int(x) for x in h[2][:4]] == [4, 2, 1, 1] and all(int(x.sum()) == 8 for x in h)


def test_split_entropy_closed_forms():
    every = np.arange(65536, dtype=np.uint16)                 # each 16-bit pattern once: every field is uniform
    for widths in ([16], [8, 8], [1, 5, 5, 5], [4, 4, 4, 4], [1, 4, 4, 7], [3, 13], [1] * 16):
        per_field, total = orc.split_entropy(every, widths)
        assert per_field == pytest.approx([float(x) for x in widths], abs=1e-12) and total == pytest.approx(16.0, abs=1e-12)
    assert orc.split_entropy(np.full(1000, 0x3C00, dtype=np.uint16), [1, 5, 5, 5]) == ([0.0] * 4, 0.0)
    # a product set (each combination of a field-0 value and a field-1 value exactly once): the fields are
    # independent, so the sum of the field entropies equals the entropy of the whole word
    a, b = np.array([3, 77, 200], dtype=np.uint16), np.array([0, 1, 2, 3, 250], dtype=np.uint16)
    w = ((a[:, None] << 8) | b[None, :]).ravel()
    per_field, total = orc.split_entropy(w, [8, 8])
    assert per_field == pytest.approx([math.log2(3), math.log2(5)], abs=1e-12)
    assert total == pytest.approx(orc.split_entropy(w, [16])[1], abs=1e-12)


def test_split_field_order_is_most_significant_first():
    w = np.array([0x8000, 0x7C00, 0x03E0, 0x001F], dtype=np.uint16)      # one field of {1,5,5,5} all ones, in turn
    f = orc.split_fields(w, [1, 5, 5, 5])
    assert [list(map(int, x)) for x in f] == [[1, 0, 0, 0], [0, 31, 0, 0], [0, 0, 31, 0], [0, 0, 0, 31]]
    with pytest.raises(ValueError):
        orc.split_fields(w, [8, 7])


def test_refining_a_split_never_lowers_its_total():
    # entropy is subadditive: cutting a field in two can only raise the sum, and no split beats the whole word
    w = wl.gaussian_weights(256, 4096, 0.02, 5, "fp16_from_bf16")
    t16 = orc.split_entropy(w, [16])[1]
    t88 = orc.split_entropy(w, [8, 8])[1]
    t4444 = orc.split_entropy(w, [4, 4, 4, 4])[1]
    t1555 = orc.split_entropy(w, [1, 5, 5, 5])[1]
    t1x16 = orc.split_entropy(w, [1] * 16)[1]
    assert t16 <= t88 + 1e-9 <= t4444 + 2e-9 <= t1x16 + 3e-9 and t16 <= t1555 + 1e-9 <= t1x16 + 2e-9
    # and the field histogram of {1,5,5,5} is the one the codebook builder counts
    counts = orc.histogram(w, orc.FP16)
    h = orc.split_histograms(w, [1, 5, 5, 5])
    for k in range(3):
        assert np.array_equal(h[k + 1], counts[k][:32])
    # a Huffman code of a field spends between H and H + 1 bits per symbol
    for k in range(3):
        lens = orc.huffman_lengths(counts[k][:32])
        avg = orc.code_cost(counts[k][:32], lens) / w.size
        H = orc.shannon_entropy(h[k + 1])
        assert H - 1e-9 <= avg < H + 1


def test_synthetic_fp16_weights_land_on_the_papers_entropy_table():
    # Real checkpoints are unavailable: a soft pin of the synthetic stand-in against the printed rows.
    g = read_golden("entropy_table_section3_1.txt")
    w = wl.gaussian_weights(1024, 4096, 0.02, 11, "fp16_from_bf16")
    for name, widths, tol in (("16", [16], 0.15), ("8_8", [8, 8], 0.15), ("1_5_5_5", [1, 5, 5, 5], 0.15), ("4_4_4_4", [4, 4, 4, 4], 0.35)):
        per_field, total = orc.split_entropy(w, widths)
        want = [float(x) for x in g["split_" + name]]
        assert np.abs(np.array(per_field) - np.array(want)).max() < tol, (name, per_field)
        if name != "4_4_4_4":
            assert abs(total - float(g["total_" + name][0])) < tol
    # the ordering the section argues from: 16 < 8-8 < 1-5-5-5 < 4-4-4-4
    tot = [orc.split_entropy(w, s)[1] for s in ([16], [8, 8], [1, 5, 5, 5], [4, 4, 4, 4])]
    assert tot == sorted(tot)
