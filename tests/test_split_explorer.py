"""Bit-field split explorer (Section 3.1, entropy table): the library's counters and entropies against the oracle's."""
import numpy as np
import pytest

import workloads as wl
from oracle import oracle as orc

SPLITS = [[16], [8, 8], [1, 5, 5, 5], [4, 4, 4, 4], [1, 4, 4, 7], [1, 8, 7], [3, 13], [2, 14], [1, 15], [1] * 16, [9, 7], [12, 4]]


@pytest.fixture(scope="module")
def hl():
    import paper_2502_00922_b200 as m
    m.lib()
    return m


# ------------------------------------------------------------------ host part

@pytest.mark.parametrize("widths", [[8, 8], [1, 5, 5, 5], [4, 4, 4, 4], [16], [1, 4, 4, 7]])
def test_entropy_of_counters_matches_oracle(hl, widths):
    w = wl.gaussian_weights(64, 4096, 0.02, 3, "fp16_from_bf16")
    hist = orc.split_histograms(w, widths)
    counts = np.concatenate(hist)
    assert counts.size == hl.split_counts_size(widths)
    ent, huf = hl.split_entropy(counts, widths)
    want, total = orc.split_entropy(w, widths)
    assert ent == pytest.approx(want, abs=1e-9) and float(ent.sum()) == pytest.approx(total, abs=1e-9)
    for k, width in enumerate(widths):
        if width <= 8:                                    # the oracle's Huffman routine takes up to 256 symbols
            lens = orc.huffman_lengths(hist[k])
            assert huf[k] == pytest.approx(orc.code_cost(hist[k], lens) / w.size, abs=1e-9)
        assert ent[k] - 1e-9 <= huf[k] < ent[k] + 1 or (ent[k] == 0 and huf[k] == 1.0)


def test_entropy_special_cases(hl):
    counts = np.zeros(2 + 32 * 3, dtype=np.uint64)
    counts[[1, 2 + 15, 34 + 0, 66 + 0]] = 1000           # one value per field: entropy 0, the format's 1-bit code
    ent, huf = hl.split_entropy(counts, [1, 5, 5, 5])
    assert list(ent) == [0.0] * 4 and list(huf) == [1.0] * 4
    ent, huf = hl.split_entropy(np.zeros(512, dtype=np.uint64), [8, 8])     # nothing counted
    assert list(ent) == [0.0, 0.0] and list(huf) == [0.0, 0.0]
    ent, huf = hl.split_entropy(np.ones(65536, dtype=np.uint64), [16])      # uniform: 16 bits either way
    assert ent[0] == pytest.approx(16.0, abs=1e-12) and huf[0] == pytest.approx(16.0, abs=1e-12)


def test_bad_splits_are_refused(hl):
    for widths in ([8, 7], [8, 9], [0, 16], [17], [1] * 17, []):
        with pytest.raises((hl.HuffllmError, ValueError)):
            hl.split_counts_size(widths)
    with pytest.raises(ValueError):
        hl.split_entropy(np.zeros(10, dtype=np.uint64), [8, 8])


# ------------------------------------------------------------------ device part

def device_counts(hl, torch, w, widths):
    w_dev = torch.from_numpy(np.ascontiguousarray(w).view(np.int16).ravel()).cuda() if w.size else torch.zeros(8, dtype=torch.int16, device="cuda")
    n = hl.split_counts_size(widths)
    counts = torch.full((n + 4,), 77, dtype=torch.int64, device="cuda")      # stale values in front, a canary behind
    hl.split_histogram(w_dev, int(w.size), widths, counts)
    torch.cuda.synchronize()
    res = counts.cpu().numpy().view(np.uint64)
    assert np.all(res[n:] == 77)
    return res[:n]


@pytest.mark.gpu
@pytest.mark.parametrize("widths", SPLITS)
def test_device_counters_are_exact(hl, widths):
    import torch
    for gen, shape in (("fp16_from_bf16", (256, 4096)), ("bf16", (33, 1000 + 3))):   # the second: a ragged tail of 3 weights
        w = wl.gaussian_weights(shape[0], shape[1], 0.02, 9, gen)
        got = device_counts(hl, torch, w, widths)
        assert np.array_equal(got, np.concatenate(orc.split_histograms(w, widths)))


@pytest.mark.gpu
def test_device_counters_edge_sizes(hl):
    import torch
    for n in (0, 1, 7, 8, 9):
        w = (np.arange(n, dtype=np.uint16) * 4099 + 0x3C00).astype(np.uint16)
        for widths in ([1, 5, 5, 5], [16]):
            got = device_counts(hl, torch, w, widths)
            want = np.concatenate(orc.split_histograms(w, widths)) if n else np.zeros(hl.split_counts_size(widths), dtype=np.uint64)
            assert np.array_equal(got, want)
    # every lane on the same value (the worst case for counters that are not replicated), and all 65536 patterns
    w = np.full(1 << 20, 0x3C00, dtype=np.uint16)
    for widths in ([1, 5, 5, 5], [16], [2, 14]):
        assert np.array_equal(device_counts(hl, torch, w, widths), np.concatenate(orc.split_histograms(w, widths)))
    every = np.tile(np.arange(65536, dtype=np.uint16), 4)
    got = device_counts(hl, torch, every, [16])
    assert np.all(got == 4)
    with pytest.raises(hl.HuffllmError):                   # misaligned weights are refused before any launch
        t = torch.zeros(64, dtype=torch.int16, device="cuda")
        hl.split_histogram(t.data_ptr() + 2, 16, [8, 8], torch.zeros(512, dtype=torch.int64, device="cuda"))


@pytest.mark.gpu
def test_full_size_matrix_reproduces_the_tables_rows(hl):
    """A full-size FFN matrix of the benchmark's layer, every split of the entropy table, counters exact."""
    import torch
    w = wl.gaussian_weights(11008, 4096, 0.02, 21, "fp16_from_bf16")
    totals = []
    for widths in ([16], [8, 8], [1, 5, 5, 5], [4, 4, 4, 4]):
        got = device_counts(hl, torch, w, widths)
        assert np.array_equal(got, np.concatenate(orc.split_histograms(w, widths)))
        ent, _ = hl.split_entropy(got, widths)
        assert float(ent.sum()) == pytest.approx(orc.split_entropy(w, widths)[1], abs=1e-9)
        totals.append(float(ent.sum()))
    assert totals == sorted(totals)                        # 16 < 8-8 < 1-5-5-5 < 4-4-4-4, as in the table
