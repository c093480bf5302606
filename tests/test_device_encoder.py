"""Compression of weights that sit in device memory: counts on the device, codebook from the counts, encoder on the
device.  The blob must be the host encoder's byte for byte, and the oracle's slow reader must get the tensor back."""
import numpy as np
import pytest

import workloads as wl
from oracle import oracle as orc


@pytest.fixture(scope="module")
def hl():
    import paper_2502_00922_b200 as m
    m.lib()
    return m


def gen(kind, rows, cols, seed):
    return {"gauss": lambda: wl.gaussian_weights(rows, cols, 0.02, seed),
            "fp16": lambda: wl.gaussian_weights(rows, cols, 0.02, seed, "fp16"),
            "fp16_from_bf16": lambda: wl.gaussian_weights(rows, cols, 0.02, seed, "fp16_from_bf16"),
            "student": lambda: wl.student_t_weights(rows, cols, seed),
            "patterns": lambda: wl.all_patterns_weights(rows, cols, seed),
            "constant": lambda: np.full((rows, cols), 0xBD33, dtype=np.uint16)}[kind]()


def counts_for_codebook(w, dtype):
    """The counters huffllm_build_codebook_from_counts wants, taken from the oracle's field histograms."""
    if dtype == 1:
        return np.concatenate(orc.split_histograms(w, [1, 5, 5, 5])[1:])
    return orc.split_histograms(w, [1, 8, 7])[1]


# ------------------------------------------------------------------ host part: codebook from counts

@pytest.mark.parametrize("kind,dtype,split,budget", [("gauss", 0, 0, 0), ("gauss", 0, 1, 0), ("student", 0, 0, 9), ("fp16", 1, 0, 0),
                                                     ("fp16_from_bf16", 1, 0, 0), ("constant", 0, 0, 0), ("patterns", 0, 1, 9)])
def test_codebook_from_counts_is_the_codebook_of_the_tensor(hl, kind, dtype, split, budget):
    w = gen(kind, 48, 640, 4)
    cb_a = hl.build_codebook(w, dtype, budget, split)
    cb_b = hl.build_codebook_from_counts(counts_for_codebook(w, dtype), dtype, budget, split)
    blob_a, desc_a = hl.encode(cb_a, w, 1024)
    blob_b, desc_b = hl.encode(cb_b, w, 1024)
    assert np.array_equal(blob_a, blob_b) and bytes(desc_a) == bytes(desc_b)
    cb_a.free()
    cb_b.free()


def test_codebook_from_counts_refuses_nonsense(hl):
    with pytest.raises(hl.HuffllmError):
        hl.build_codebook_from_counts(np.zeros(256, dtype=np.uint64), 0)           # nothing counted
    with pytest.raises(hl.HuffllmError):
        hl.build_codebook_from_counts(np.ones(96, dtype=np.uint64), 1, 0, 1)       # whole-exponent split is for bf16
    with pytest.raises(ValueError):
        hl.build_codebook_from_counts(np.ones(96, dtype=np.uint64), 0)


# ------------------------------------------------------------------ device part

CASES = [  # rows, cols, chunk_elems, kind, dtype, split, budget
    (64, 1024, 4096, "gauss", 0, 0, 0),
    (100, 1000, 2048, "gauss", 0, 0, 0),            # ragged rows, columns a multiple of 8 but not of 32
    (37, 333, 512, "student", 0, 0, 9),             # nothing aligned: scalar loads, pad words
    (16, 32, 512, "constant", 0, 0, 0),             # a single block, a single symbol
    (48, 2080, 1024, "patterns", 0, 1, 9),          # whole-exponent code, every exponent in use
    (64, 1024, 1024, "fp16", 1, 0, 0),
    (50, 1096, 2048, "fp16_from_bf16", 1, 0, 0),    # FP16, odd block count in the last chunk (sign plane padding)
    (33, 100, 512, "fp16", 1, 0, 0),
    (512, 4096, 4096, "gauss", 0, 0, 0),
]


@pytest.mark.gpu
@pytest.mark.parametrize("rows,cols,ce,kind,dtype,split,budget", CASES)
def test_device_encoder_writes_the_host_encoders_blob(hl, rows, cols, ce, kind, dtype, split, budget):
    import torch
    w = gen(kind, rows, cols, 12)
    w_dev = torch.from_numpy(w.view(np.int16)).cuda()
    # counts on the device -> codebook
    widths = [1, 5, 5, 5] if dtype == 1 else [1, 8, 7]
    counts = torch.zeros(hl.split_counts_size(widths), dtype=torch.int64, device="cuda")
    hl.split_histogram(w_dev, rows * cols, widths, counts)
    c = counts.cpu().numpy().view(np.uint64)
    cb = hl.build_codebook_from_counts(c[2:98] if dtype == 1 else c[2:258], dtype, budget, split)
    # encode on the device
    cap = hl.encode_bound(rows, cols, dtype, ce)
    blob_dev = torch.full((cap + 256,), 0xA5, dtype=torch.uint8, device="cuda")
    n_scr = hl.encode_device_scratch_bytes(rows, cols, ce)
    scratch = torch.full((n_scr,), 0x5A, dtype=torch.uint8, device="cuda")
    desc = hl.encode_device(cb, w_dev, rows, cols, ce, blob_dev, cap, scratch, n_scr)
    got = blob_dev.cpu().numpy()
    assert np.all(got[desc.blob_bytes:] == 0xA5), "wrote behind the blob"
    got = got[:desc.blob_bytes]
    # the host encoder's blob, byte for byte
    cb_host = hl.build_codebook(w, dtype, budget, split)
    want, desc_host = hl.encode(cb_host, w, ce)
    assert bytes(desc) == bytes(desc_host)
    assert np.array_equal(got, want)
    hl.validate_blob(got)
    # and, independently of the host encoder, the oracle's reader gets the tensor back
    if rows * cols <= 1 << 17:
        back, _ = orc.decode_blob(got)
        assert np.array_equal(back, w)
    cb.free()
    cb_host.free()


@pytest.mark.gpu
def test_full_size_matrix_on_the_device_equals_the_host_blob(hl):
    """A full-size FFN matrix of the benchmark's layer (45 M weights, 11008 chunks)."""
    import torch
    rows, cols, ce = 11008, 4096, 4096
    w = wl.gaussian_weights(rows, cols, 0.02, 1003)
    w_dev = torch.from_numpy(w.view(np.int16)).cuda()
    counts = torch.zeros(hl.split_counts_size([1, 8, 7]), dtype=torch.int64, device="cuda")
    hl.split_histogram(w_dev, rows * cols, [1, 8, 7], counts)
    cb = hl.build_codebook_from_counts(counts.cpu().numpy().view(np.uint64)[2:258], 0)
    cap = hl.encode_bound(rows, cols, 0, ce)
    blob_dev = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    n_scr = hl.encode_device_scratch_bytes(rows, cols, ce)
    desc = hl.encode_device(cb, w_dev, rows, cols, ce, blob_dev, cap, torch.zeros(n_scr, dtype=torch.uint8, device="cuda"), n_scr)
    cb_host = hl.build_codebook(w, 0)
    want, desc_host = hl.encode(cb_host, w, ce)
    assert bytes(desc) == bytes(desc_host)
    assert np.array_equal(blob_dev[:desc.blob_bytes].cpu().numpy(), want)
    cb.free()
    cb_host.free()


@pytest.mark.gpu
def test_device_encoded_blob_feeds_the_product_kernel(hl):
    import torch
    rows, cols = 256, 2048
    w = wl.gaussian_weights(rows, cols, 0.02, 33)
    w_dev = torch.from_numpy(w.view(np.int16)).cuda()
    counts = torch.zeros(hl.split_counts_size([1, 8, 7]), dtype=torch.int64, device="cuda")
    hl.split_histogram(w_dev, rows * cols, [1, 8, 7], counts)
    cb = hl.build_codebook_from_counts(counts.cpu().numpy().view(np.uint64)[2:258], 0)
    cap = hl.encode_bound(rows, cols, 0, 4096)
    blob_dev = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    n_scr = hl.encode_device_scratch_bytes(rows, cols, 4096)
    desc = hl.encode_device(cb, w_dev, rows, cols, 4096, blob_dev, cap, torch.zeros(n_scr, dtype=torch.uint8, device="cuda"), n_scr)
    x = wl.activations(1, cols, 5)
    x_dev = torch.from_numpy(x.view(np.int16).reshape(-1)).cuda()
    y = torch.zeros(rows, dtype=torch.float32, device="cuda")
    ws_bytes = hl.workspace_bytes(desc, 1)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    hl.decode_gemv(desc, blob_dev, x_dev, y, ws, ws_bytes, err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    y_ref, y_abs = orc.matmul(w, x)
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - y_ref[0]) <= 2e-3 * y_abs[0] + 1e-30)
    cb.free()


@pytest.mark.gpu
def test_device_encoder_errors(hl):
    import torch
    w = wl.gaussian_weights(32, 256, 0.02, 1)
    w_dev = torch.from_numpy(w.view(np.int16)).cuda()
    cb = hl.build_codebook(w, 0)
    cap = hl.encode_bound(32, 256, 0, 512)
    blob = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    n_scr = hl.encode_device_scratch_bytes(32, 256, 512)
    scr = torch.zeros(n_scr, dtype=torch.uint8, device="cuda")
    with pytest.raises(hl.HuffllmError) as e:
        hl.encode_device(cb, w_dev, 32, 256, 512, blob, 1024, scr, n_scr)            # capacity below the payload
    assert e.value.status_name == "BUFFER_TOO_SMALL"
    with pytest.raises(hl.HuffllmError) as e:
        hl.encode_device(cb, w_dev, 32, 256, 512, blob, cap, scr, 16)                # scratch too small
    assert e.value.status_name == "BUFFER_TOO_SMALL"
    # a weight whose exponent the codebook has never seen
    other = torch.from_numpy(np.full((32, 256), 0x7F00, dtype=np.uint16).view(np.int16)).cuda()
    with pytest.raises(hl.HuffllmError) as e:
        hl.encode_device(cb, other, 32, 256, 512, blob, cap, scr, n_scr)
    assert e.value.status_name == "INVALID_ARG"
    hl.encode_device(cb, w_dev, 32, 256, 512, blob, cap, scr, n_scr)                 # and the context is still fine
    cb.free()
