"""Parity of the CUDA path against the CPU oracle, through the C-ABI.  Needs a GPU."""
import numpy as np
import pytest

import workloads as wl
from oracle import oracle as orc

pytestmark = pytest.mark.gpu

TOL = 2e-3   # |y_gpu - y_oracle| <= TOL * sum_k |w x|, per output


@pytest.fixture(scope="module")
def hl():
    import paper_2502_00922_b200 as m
    m.lib()
    return m


@pytest.fixture(scope="module")
def torch():
    import torch as t
    assert t.cuda.is_available()
    return t


class Uploaded:
    """A tensor encoded on the host and resident on the device, with its scratch buffers."""

    def __init__(self, hl, torch, w, chunk_elems=4096, budget=0, batch=1, split=0, dtype=0):
        self.w = w
        cb = hl.build_codebook(w, dtype, budget, split)
        self.blob, self.desc = hl.encode(cb, w, chunk_elems)
        cb.free()
        hl.validate_blob(self.blob)
        self.blob_dev = torch.from_numpy(self.blob).cuda()
        assert self.blob_dev.data_ptr() % 256 == 0
        self.ws_bytes = hl.workspace_bytes(self.desc, batch)
        self.ws = torch.zeros(self.ws_bytes, dtype=torch.uint8, device="cuda")
        self.err = torch.zeros(1, dtype=torch.int32, device="cuda")


def gpu_decode(hl, torch, up):
    rows, cols = up.w.shape
    out = torch.full((rows * cols + 64,), 0x5A5A, dtype=torch.int16, device="cuda")   # canary behind the output
    hl.decode(up.desc, up.blob_dev, out, up.err)
    torch.cuda.synchronize()
    assert int(up.err.item()) == 0
    res = out.cpu().numpy().view(np.uint16)
    assert np.all(res[rows * cols:] == 0x5A5A)
    return res[:rows * cols].reshape(rows, cols)


def gpu_gemm(hl, torch, up, x):
    rows, cols = up.w.shape
    batch = x.shape[0]
    x_dev = torch.from_numpy(x.view(np.int16)).cuda()
    y = torch.full((batch * rows + 16,), float("nan"), dtype=torch.float32, device="cuda")
    if batch == 1:
        hl.decode_gemv(up.desc, up.blob_dev, x_dev, y, up.ws, up.ws_bytes, up.err)
    else:
        hl.decode_gemm(up.desc, up.blob_dev, x_dev, batch, y, up.ws, up.ws_bytes, up.err)
    torch.cuda.synchronize()
    assert int(up.err.item()) == 0
    assert int(up.ws[:hl.workspace_control_bytes(up.desc)].count_nonzero().item()) == 0, "the scratch control words must be left zero"
    res = y.cpu().numpy()
    assert np.all(np.isnan(res[batch * rows:]))
    return res[:batch * rows].reshape(batch, rows)


def check_product(y_gpu, w, x, dtype=orc.BF16):
    y, d = orc.matmul(w, x, dtype)
    err = np.abs(y_gpu.astype(np.float64) - y)
    assert np.all(err <= TOL * d + 1e-30), f"max err/bound = {np.max(err / (TOL * d + 1e-30))}"
    assert np.all(y_gpu[d == 0] == 0)
    return float(np.max(err / np.maximum(d, 1e-300)))


DECODE_CASES = [
    # rows, cols, chunk_elems, budget, generator
    (1024, 1024, 4096, 0, "gauss"),        # the small benchmark configuration
    (16, 256, 4096, 0, "gauss"),           # exactly one chunk
    (37, 300, 1024, 0, "student"),         # ragged rows and columns, scalar stores
    (48, 1056, 4096, 0, "gauss"),          # ragged last column chunk
    (5, 31, 512, 0, "patterns"),           # smaller than one tile
    (272, 2080, 16384, 0, "gauss"),        # largest chunk size
    (64, 8192, 1024, 0, "uniform"),        # worst-case exponents, smallest benchmark chunk size
    (256, 2048, 4096, 0, "patterns"),      # every bit pattern incl. NaN / Inf / denormals
    (96, 4096, 4096, 9, "student"),        # the other table size
    (2368, 512, 512, 0, "gauss"),          # more chunks than warps, many per warp
    (16, 512, 512, 0, "constant"),         # single-symbol codes
]


def make(gen, rows, cols, seed):
    return {"gauss": lambda: wl.gaussian_weights(rows, cols, 0.02, seed),
            "student": lambda: wl.student_t_weights(rows, cols, seed),
            "uniform": lambda: wl.uniform_exponent_weights(rows, cols, seed),
            "patterns": lambda: wl.all_patterns_weights(rows, cols, seed),
            "skewed": lambda: wl.skewed_exponent_weights(rows, cols, seed),
            "constant": lambda: np.full((rows, cols), 0xBD33, dtype=np.uint16)}[gen]()


@pytest.mark.parametrize("rows,cols,ce,budget,gen", DECODE_CASES)
def test_decode_is_bit_exact(hl, torch, rows, cols, ce, budget, gen):
    w = make(gen, rows, cols, 100 + rows)
    up = Uploaded(hl, torch, w, ce, budget)
    got = gpu_decode(hl, torch, up)
    if rows * cols <= 300_000:
        ref, _ = orc.decode_blob(up.blob)          # the oracle's bit-serial decode of the same blob
        assert np.array_equal(ref, w)
    assert np.array_equal(got, w)                  # lossless: the oracle's result is the original tensor


@pytest.mark.parametrize("rows,cols,ce,budget,gen,batch", [
    (1024, 1024, 4096, 0, "gauss", 1), (37, 300, 1024, 0, "student", 0), (256, 2048, 4096, 0, "patterns", 0),
    (512, 4096, 4096, 9, "student", 5), (272, 2080, 16384, 0, "gauss", 4), (16, 512, 512, 0, "constant", 2),
    (1040, 4096, 4096, 0, "gauss", 33), (256, 2048, 4096, 0, "uniform", 8)])
def test_whole_exponent_split_decode_and_product(hl, torch, rows, cols, ce, budget, gen, batch):
    """Blobs of the {1,8,7} split (one 256-symbol exponent code) run through the same kernels: only the table differs."""
    w = make(gen, rows, cols, 700 + rows)
    up = Uploaded(hl, torch, w, ce, budget, max(batch, 1), split=hl.SPLIT_WHOLE_EXPONENT)
    assert up.desc.n_fields == 1
    assert np.array_equal(gpu_decode(hl, torch, up), w)
    if rows * cols <= 300_000:
        ref, _ = orc.decode_blob(up.blob)
        assert np.array_equal(ref, w)
    if batch:
        x = wl.activations(batch, cols, 800 + cols)
        check_product(gpu_gemm(hl, torch, up, x), w, x)


FP16_GENS = {"fp16": lambda r, c, seed: wl.gaussian_weights(r, c, 0.02, seed, "fp16"),
             "fp16_from_bf16": lambda r, c, seed: wl.gaussian_weights(r, c, 0.02, seed, "fp16_from_bf16"),
             "patterns": lambda r, c, seed: wl.all_patterns_weights(r, c, seed),
             "constant": lambda r, c, seed: np.full((r, c), 0xAE66, dtype=np.uint16),
             "skewed": lambda r, c, seed: wl.skewed_exponent_weights(r, c, seed, dtype="fp16")}


@pytest.mark.parametrize("rows,cols,ce,gen,batch", [
    (1024, 1024, 1024, "fp16", 1),                # true fp16 weights: 13.7 bits per weight
    (37, 300, 512, "fp16_from_bf16", 0),          # ragged rows and columns (decode only)
    (256, 2048, 1024, "patterns", 0),             # every bit pattern incl. NaN / Inf / denormals (decode only)
    (5, 31, 512, "patterns", 0),
    (16, 512, 512, "constant", 2),                # single-symbol codes in all three fields
    (40, 2080, 1024, "fp16_from_bf16", 3),        # ragged rows, odd number of blocks in the last column chunk
    (512, 4096, 2048, "fp16_from_bf16", 8),       # larger chunks fit when the weights came from bf16 (10.9 bits per weight)
    (2368, 512, 512, "fp16", 5),                  # many chunks per warp
    (272, 2048, 1024, "fp16", 16),                # batch above 8: the tensor-core path with f16 operands
    (1000, 4096, 1024, "fp16", 33),               # ragged row tiles, batch padded to 64, several column ranges
    (600, 2080, 1024, "fp16_from_bf16", 9),       # odd block count in the last chunk, batch padded to 16
    (64, 4096, 4096, "fp16", 12),                 # records too large for the tensor-core kernel's slots: passes of 8 vectors
])
def test_fp16_decode_and_product(hl, torch, rows, cols, ce, gen, batch):
    """FP16 {1,5,5,5} blobs: bit-exact decode and products within the tolerance, against the oracle."""
    w = FP16_GENS[gen](rows, cols, 900 + rows)
    up = Uploaded(hl, torch, w, ce, 0, max(batch, 1), dtype=hl.FP16)
    assert (up.desc.dtype, up.desc.n_fields) == (hl.FP16, 3)
    assert np.array_equal(gpu_decode(hl, torch, up), w)
    if rows * cols <= 300_000:
        ref, _ = orc.decode_blob(up.blob)
        assert np.array_equal(ref, w)
    if batch:
        x = wl.activations(batch, cols, 950 + cols, "fp16")
        check_product(gpu_gemm(hl, torch, up, x), w, x, orc.FP16)


@pytest.mark.parametrize("rows,cols,ce,budget,gen,batch", [
    (256, 1024, 1024, 12, "skewed", 1),           # Section 3.2's L_max = 12: geometric laws in all three fields, long codewords occur
    (128, 2048, 512, 10, "skewed", 5),
    (1024, 1024, 1024, 12, "fp16", 3),            # true fp16 weights under the longer limit
    (37, 300, 512, 9, "skewed", 0),               # ragged, 9 bits (decode only)
    (256, 2048, 1024, 12, "patterns", 0),         # every bit pattern (decode only)
    (64, 1024, 1024, 12, "skewed", 16),           # batch above 8: passes of 8 vectors
])
def test_fp16_long_field_codes_decode_and_product(hl, torch, rows, cols, ce, budget, gen, batch):
    """FP16 {1,5,5,5} blobs whose field codes are limited to 9..12 bits: two-level lookup on the device."""
    w = FP16_GENS[gen](rows, cols, 1400 + rows + budget)
    up = Uploaded(hl, torch, w, ce, budget, max(batch, 1), dtype=hl.FP16)
    assert (up.desc.dtype, up.desc.lut_bits) == (hl.FP16, budget)
    if gen == "skewed":
        lut = up.blob[up.desc.off_lut:up.desc.off_lut + 3 * (4 << budget)].view(np.uint32)
        assert int(((lut >> 16) > 8).sum()) > 0, "the case should contain codewords longer than the first level"
    assert np.array_equal(gpu_decode(hl, torch, up), w)
    if rows * cols <= 600_000:
        ref, _ = orc.decode_blob(up.blob)
        assert np.array_equal(ref, w)
    if batch:
        x = wl.activations(batch, cols, 1450 + cols, "fp16")
        check_product(gpu_gemm(hl, torch, up, x), w, x, orc.FP16)


@pytest.mark.parametrize("rows,cols,ce,gen,batch", [
    (1024, 1024, 1024, "fp16", 1),                # true fp16 weights
    (512, 4096, 2048, "fp16_from_bf16", 8),
    (256, 1024, 1024, "skewed", 3),               # geometric laws: the 7-bit limit bites in all three fields
    (37, 300, 512, "skewed", 0),                  # ragged rows and columns (decode only)
    (256, 2048, 1024, "patterns", 0),             # every bit pattern (decode only)
    (16, 512, 512, "constant", 2),                # single-symbol codes
    (128, 1024, 1024, "fp16", 16),                # batch above 8: passes of 8 vectors
])
def test_fp16_seven_bit_field_codes(hl, torch, rows, cols, ce, gen, batch):
    """FP16 {1,5,5,5} blobs whose field codes are limited to 7 bits: 128-entry tables that the device keeps once per lane."""
    w = FP16_GENS[gen](rows, cols, 1500 + rows)
    up = Uploaded(hl, torch, w, ce, 7, max(batch, 1), dtype=hl.FP16)
    assert (up.desc.dtype, up.desc.lut_bits) == (hl.FP16, 7)
    assert np.array_equal(gpu_decode(hl, torch, up), w)
    if rows * cols <= 600_000:
        ref, _ = orc.decode_blob(up.blob)
        assert np.array_equal(ref, w)
    if batch:
        x = wl.activations(batch, cols, 1550 + cols, "fp16")
        check_product(gpu_gemm(hl, torch, up, x), w, x, orc.FP16)


def test_fp16_large_chunks_run_on_single_slots(hl, torch):
    """Records too large for 31 pairs of shared-memory slots: every decoder warp gets one slot instead of a pair
    (4096-element FP16 chunks keep 22 of 31 warps that way, against 11); still larger ones are decoded by as many warps as have room."""
    w = wl.gaussian_weights(64, 4096, 0.02, 990, "fp16")
    up = Uploaded(hl, torch, w, 16384, 0, 1, dtype=hl.FP16)
    assert up.desc.max_words > 64
    plan = hl.decode_launch_plan(up.desc, 1)
    assert plan["slots_per_warp"] == 1 and 2 <= plan["decoder_warps"] < 31
    assert np.array_equal(gpu_decode(hl, torch, up), w)
    x = wl.activations(1, 4096, 991, "fp16")
    check_product(gpu_gemm(hl, torch, up, x), w, x, orc.FP16)
    # the benchmark chunk size: single slots for two thirds of the warps; many chunks per warp, so that slots are reused
    w = wl.gaussian_weights(1040, 4096, 0.02, 992, "fp16")
    up = Uploaded(hl, torch, w, 4096, 0, 3, dtype=hl.FP16)
    plan = hl.decode_launch_plan(up.desc, 1)
    assert plan["slots_per_warp"] == 1 and plan["decoder_warps"] >= 20
    assert np.array_equal(gpu_decode(hl, torch, up), w)
    for batch in (1, 3):
        x = wl.activations(batch, 4096, 993 + batch, "fp16")
        check_product(gpu_gemm(hl, torch, up, x), w, x, orc.FP16)


GEMM_CASES = [
    (1024, 1024, 4096, 0, "gauss", 1),
    (16, 256, 4096, 0, "gauss", 1),
    (48, 1056, 4096, 0, "gauss", 1),
    (40, 2080, 1024, 0, "student", 3),            # ragged rows, last column chunk holds a single block
    (40, 2080, 1024, 0, "student", 1),            # the same as a matrix-vector product (multiply-adds on the FMA pipe)
    (512, 4096, 4096, 9, "student", 1),           # ... with a 512-entry table
    (16, 65536, 4096, 0, "gauss", 1),             # one row group split over every CTA
    (32, 32768, 4096, 0, "gauss", 8),
    (2368, 512, 512, 0, "gauss", 2),
    (272, 2080, 16384, 0, "gauss", 4),
    (512, 4096, 4096, 9, "student", 5),
    (256, 2048, 4096, 0, "uniform", 8),
    (128, 1024, 1024, 0, "gauss", 16),            # 9..16 vectors, few rows: the register path with two tiles of activations
    (2048, 2048, 4096, 0, "gauss", 13),           # 9..16 vectors, as wide as tall: the tcgen05 path at its smallest padding
    (2064, 4096, 4096, 0, "student", 16),         # ... ragged rows (129 row groups: five row tiles, the last nearly empty)
    (4096, 1024, 4096, 0, "gauss", 12),           # 9..16 vectors, tall: two tiles
    (64, 1024, 4096, 0, "gauss", 23),
    (40, 2080, 1024, 0, "student", 9),            # ragged rows, padded batch
    (1040, 4096, 4096, 0, "gauss", 64),           # three row tiles, column chunks cut into ranges
    (16, 65536, 4096, 0, "gauss", 16),            # one row group, 16 column ranges
    (2368, 512, 512, 0, "uniform", 48),           # several work items per CTA
    (528, 2048, 4096, 9, "student", 32),          # 512-entry table
    (69, 2496, 4096, 9, "student", 9),            # ... and records of 18 rows: two tiles is all that fits beside a 64 KB table
]


@pytest.mark.parametrize("rows,cols,ce,budget,gen,batch", GEMM_CASES)
def test_fused_product_matches_oracle(hl, torch, rows, cols, ce, budget, gen, batch):
    w = make(gen, rows, cols, 200 + rows)
    x = wl.activations(batch, cols, 300 + cols)
    up = Uploaded(hl, torch, w, ce, budget, batch)
    y1 = gpu_gemm(hl, torch, up, x)
    check_product(y1, w, x)
    y2 = gpu_gemm(hl, torch, up, x)
    assert np.array_equal(y1, y2), "results must be bitwise reproducible"


@pytest.mark.parametrize("rows,cols,ce,budget,gen,batch,split", [
    (1024, 1024, 4096, 12, "gauss", 1, 0),        # the small benchmark configuration with the paper's L_max
    (256, 2048, 4096, 10, "skewed", 5, 0),        # geometric exponents: codewords of 9 and 10 bits do occur
    (256, 2048, 4096, 12, "skewed", 1, 0),        # ... and of 11 and 12
    (96, 4096, 4096, 11, "student", 3, 0),
    (256, 2048, 4096, 12, "patterns", 0, 0),      # every bit pattern (decode only)
    (37, 300, 1024, 12, "skewed", 0, 0),          # ragged rows and columns (decode only)
    (272, 2080, 16384, 12, "skewed", 8, 0),       # largest chunks, ragged last column chunk
    (512, 4096, 4096, 12, "skewed", 4, 1),        # one 256-symbol exponent code of up to 12 bits
    (128, 1024, 1024, 12, "skewed", 16, 0),       # batch above 8: passes of 8 vectors through the two-level kernel
])
def test_long_code_tables_decode_and_product(hl, torch, rows, cols, ce, budget, gen, batch, split):
    """max_code_len 10..12 (Section 3.2 quotes L_max = 12): the device looks codewords up in two levels.  Decode is
    bit-exact and products stay within the tolerance, against the oracle."""
    w = make(gen, rows, cols, 1200 + rows + budget)
    up = Uploaded(hl, torch, w, ce, budget, max(batch, 1), split=split)
    assert up.desc.lut_bits == budget
    if gen == "skewed":                            # the case is only worth its name if long codewords are really there
        lut = up.blob[up.desc.off_lut:up.desc.off_lut + (4 << budget)].view(np.uint32)
        assert int(((lut >> 16) > 8).sum()) > 0
    assert np.array_equal(gpu_decode(hl, torch, up), w)
    if rows * cols <= 600_000:
        ref, _ = orc.decode_blob(up.blob)
        assert np.array_equal(ref, w)
    if batch:
        x = wl.activations(batch, cols, 1300 + cols)
        y1 = gpu_gemm(hl, torch, up, x)
        check_product(y1, w, x)
        assert np.array_equal(y1, gpu_gemm(hl, torch, up, x)), "results must be bitwise reproducible"


@pytest.mark.parametrize("batch", [1, 3, 13, 33, 64])
def test_several_matrices_in_one_launch(hl, torch, batch):
    """Matrices of different shapes and chunk sizes through huffllm_decode_gemm_multi (one vector, one tile, two tiles,
    tensor core): every result against the oracle, and the launch must leave every workspace's control words zero."""
    shapes = [(256, 1024, 4096, "gauss"), (48, 2080, 1024, "student"), (1040, 512, 512, "gauss"), (16, 8192, 4096, "gauss"),
              (2368, 256, 4096, "uniform")]
    ups, xs, x_devs, ys = [], [], [], []
    for i, (rows, cols, ce, gen) in enumerate(shapes):
        w = make(gen, rows, cols, 900 + i)
        ups.append(Uploaded(hl, torch, w, ce, 0, batch))
        x = wl.activations(batch, cols, 950 + i)
        xs.append(x)
        x_devs.append(torch.from_numpy(x.view(np.int16)).cuda())
        ys.append(torch.full((batch * rows,), float("nan"), dtype=torch.float32, device="cuda"))
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws_each = max(u.ws_bytes for u in ups)         # every workspace of a call has at least the largest matrix's size
    for u in ups:
        u.ws = torch.zeros(ws_each, dtype=torch.uint8, device="cuda")
    for rep in range(2):
        hl.decode_gemm_multi([u.desc for u in ups], [u.blob_dev for u in ups], x_devs, batch, ys, [u.ws for u in ups],
                             ws_each, err)
        torch.cuda.synchronize()
        assert int(err.item()) == 0
        for u, x, y in zip(ups, xs, ys):
            check_product(y.cpu().numpy().reshape(batch, -1), u.w, x)
            assert int(u.ws[:hl.workspace_control_bytes(u.desc)].count_nonzero().item()) == 0
    # the same call with host buffers
    xh = [torch.from_numpy(x.view(np.int16).reshape(-1)).pin_memory() for x in xs]
    yh = [torch.zeros(batch * u.w.shape[0], dtype=torch.float32).pin_memory() for u in ups]
    hl.decode_gemm_multi_host([u.desc for u in ups], [u.blob_dev for u in ups], xh, batch, yh, x_devs, ys, [u.ws for u in ups],
                              ws_each, err)
    for u, x, y in zip(ups, xs, yh):
        check_product(y.numpy().reshape(batch, -1), u.w, x)
    # and enqueued only, through the prepared call: the caller waits for the stream
    for y in yh:
        y.fill_(float("nan"))
    prep = hl.PreparedMulti([u.desc for u in ups], [u.blob_dev for u in ups], x_devs, batch, ys, [u.ws for u in ups],
                            ws_each, err, xh, yh)
    prep.run_host_async(torch.cuda.current_stream().cuda_stream)
    torch.cuda.current_stream().synchronize()
    for u, x, y in zip(ups, xs, yh):
        check_product(y.numpy().reshape(batch, -1), u.w, x)


def test_product_closed_forms(hl, torch):
    rows, cols = 64, 1024
    ones = np.full((rows, cols), 0x3F80, dtype=np.uint16)
    up = Uploaded(hl, torch, ones)
    y = gpu_gemm(hl, torch, up, np.full((1, cols), 0x3F80, dtype=np.uint16))
    assert np.all(y == cols)
    w = wl.gaussian_weights(rows, cols, 0.02, 7)
    up = Uploaded(hl, torch, w)
    for k in (0, 519, cols - 1):                   # one-hot x returns column k exactly
        x = np.zeros((1, cols), dtype=np.uint16)
        x[0, k] = 0x3F80
        assert np.array_equal(gpu_gemm(hl, torch, up, x)[0], wl.bf16_bits_to_f32(w[:, k]))


def test_plain_gemv_matches_oracle(hl, torch):
    rows, cols = 520, 4096
    w = wl.gaussian_weights(rows, cols, 0.02, 9)
    x = wl.activations(1, cols, 10)
    y = torch.zeros(rows, dtype=torch.float32, device="cuda")
    hl.plain_gemv(torch.from_numpy(w.view(np.int16)).cuda(), rows, cols, torch.from_numpy(x.view(np.int16)).cuda(), y)
    torch.cuda.synchronize()
    check_product(y.cpu().numpy()[None, :], w, x)


def test_host_buffer_call(hl, torch):
    rows, cols, batch = 256, 2048, 4
    w = wl.gaussian_weights(rows, cols, 0.02, 11)
    x = wl.activations(batch, cols, 12)
    up = Uploaded(hl, torch, w, batch=batch)
    x_host = torch.from_numpy(x.view(np.int16)).pin_memory()
    y_host = torch.zeros(batch * rows, dtype=torch.float32).pin_memory()
    x_stage = torch.zeros(batch * cols, dtype=torch.int16, device="cuda")
    y_stage = torch.zeros(batch * rows, dtype=torch.float32, device="cuda")
    hl.decode_gemm_host(up.desc, up.blob_dev, x_host, batch, y_host, x_stage, y_stage, up.ws, up.ws_bytes, up.err)
    check_product(y_host.numpy().reshape(batch, rows), w, x)


def test_bad_record_offsets_are_reported_not_followed(hl, torch):
    """A record index pointing outside the payload (made on the host) sets the error flag; the kernel
    skips that chunk, touches nothing out of range, and every other chunk still decodes."""
    rows, cols = 64, 1024
    w = wl.gaussian_weights(rows, cols, 0.02, 13)
    up = Uploaded(hl, torch, w)
    blob = up.blob.copy()
    idx = blob[up.desc.off_index:up.desc.off_index + 4 * (up.desc.n_chunks + 1)].view(np.uint32)
    idx[5] = 0x7FFFFFF0                            # chunk 4 ends / chunk 5 starts far outside
    with pytest.raises(hl.HuffllmError):
        hl.validate_blob(blob)                     # the host check refuses it
    dev = torch.from_numpy(blob).cuda()
    out = torch.zeros(rows * cols, dtype=torch.int16, device="cuda")
    hl.decode(up.desc, dev, out, up.err)
    torch.cuda.synchronize()
    assert int(up.err.item()) != 0
    got = out.cpu().numpy().view(np.uint16).reshape(rows, cols)
    good = np.ones((rows, cols), dtype=bool)
    kc_cols = up.desc.chunk_cols
    for c in (4, 5):
        rg, kc = divmod(c, up.desc.col_chunks)
        good[rg * 16:(rg + 1) * 16, kc * kc_cols:(kc + 1) * kc_cols] = False
    assert np.array_equal(got[good], w[good])
    # the products, on every consume path (one vector, one tile, two tiles, tensor core): the two chunks add nothing
    w_skipped = np.where(good, w, np.uint16(0))
    for batch in (1, 4, 13, 32):
        x = wl.activations(batch, cols, 50 + batch)
        x_dev = torch.from_numpy(x.view(np.int16)).cuda()
        ws_bytes = hl.workspace_bytes(up.desc, batch)
        ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
        y = torch.full((batch * rows,), float("nan"), dtype=torch.float32, device="cuda")
        up.err.zero_()
        hl.decode_gemm(up.desc, dev, x_dev, batch, y, ws, ws_bytes, up.err)
        torch.cuda.synchronize()
        assert int(up.err.item()) != 0
        check_product(y.cpu().numpy().reshape(batch, rows), w_skipped, x)


def test_damaged_coded_part_is_reported_and_contained(hl, torch):
    """The coded rows of one chunk are overwritten (on the host) with the longest codeword over and over, so that the
    chunk's sequences run far past their record.  The kernels must say so in the error flag, stay inside their shared
    memory (the read pointer moves one row per refill check at most, and room for that is kept), and decode every
    other chunk as before."""
    rows, cols = 64, 2048
    w = wl.gaussian_weights(rows, cols, 0.02, 21)
    up = Uploaded(hl, torch, w)
    d = up.desc
    blob = up.blob.copy()
    lut = blob[d.off_lut:d.off_lut + (4 << d.lut_bits)].view(np.uint32)
    longest = int(((lut >> 16) & 0xFF).max())
    q = int(np.argmax((lut >> 16) & 0xFF))                       # eight stream bits that start a longest codeword
    assert longest == 8                                            # (so the same byte follows it again)
    idx = blob[d.off_index:d.off_index + 4 * (d.n_chunks + 1)].view(np.uint32)
    victim = 5
    nkb = d.chunk_cols // 32
    beg, end = d.off_payload + 128 * int(idx[victim]) + 512 * nkb, d.off_payload + 128 * int(idx[victim + 1])
    n_words = (end - beg) // 256                                   # W rows of 64 words
    bits = np.zeros(32 * n_words, dtype=np.uint64)
    i = np.arange(7, bits.size)
    bits[7:] = (q >> ((i - 7) % 8)) & 1                            # 7 leading zero bits, then the byte for ever
    words = (bits.reshape(n_words, 32) << np.arange(32, dtype=np.uint64)).sum(axis=1).astype(np.uint32)
    blob[beg:end].view(np.uint32).reshape(n_words, 64)[:] = words[:, None]
    with pytest.raises(hl.HuffllmError):
        hl.validate_blob(blob)                                     # the host check (checksum, bit walk) refuses it
    dev = torch.from_numpy(blob).cuda()
    out = torch.zeros(rows * cols, dtype=torch.int16, device="cuda")
    hl.decode(d, dev, out, up.err)
    torch.cuda.synchronize()
    assert int(up.err.item()) == 0x40000000 + victim + 1
    got = out.cpu().numpy().view(np.uint16).reshape(rows, cols)
    good = np.ones((rows, cols), dtype=bool)
    rg, kc = divmod(victim, d.col_chunks)
    good[rg * 16:(rg + 1) * 16, kc * d.chunk_cols:(kc + 1) * d.chunk_cols] = False
    assert np.array_equal(got[good], w[good])
    # the fused product reports it too and leaves its workspace usable
    up.err.zero_()
    x_dev = torch.from_numpy(wl.activations(1, cols, 22).view(np.int16)).cuda()
    y = torch.zeros(rows, dtype=torch.float32, device="cuda")
    hl.decode_gemv(d, dev, x_dev, y, up.ws, up.ws_bytes, up.err)
    torch.cuda.synchronize()
    assert int(up.err.item()) == 0x40000000 + victim + 1
    assert int(up.ws[:hl.workspace_control_bytes(d)].count_nonzero().item()) == 0


def test_unsupported_requests_fail_before_launch(hl, torch):
    w = wl.gaussian_weights(16, 520, 0.02, 14)     # cols not a multiple of 32
    up = Uploaded(hl, torch, w, 512)
    x = torch.zeros(520, dtype=torch.int16, device="cuda")
    y = torch.zeros(16, dtype=torch.float32, device="cuda")
    with pytest.raises(hl.HuffllmError) as e:
        hl.decode_gemv(up.desc, up.blob_dev, x, y, up.ws, up.ws_bytes, up.err)
    assert e.value.status_name == "UNSUPPORTED"
    w = wl.gaussian_weights(16, 512, 0.02, 15)
    up = Uploaded(hl, torch, w, 512)
    with pytest.raises(hl.HuffllmError) as e:      # misaligned blob pointer
        hl.decode(up.desc, up.blob_dev.data_ptr() + 8, torch.zeros(16 * 512, dtype=torch.int16, device="cuda"), up.err)
    assert e.value.status_name == "INVALID_ARG"


def test_full_size_layer_matrix_sampled(hl, torch):
    """gate/up projection of the Llama-7B-shaped layer at full size, in the launch configuration the
    benchmark times: decode compared everywhere with the original tensor, the product on sampled rows."""
    rows, cols = 11008, 4096
    w = wl.gaussian_weights(rows, cols, 0.02, 2004)
    x = wl.activations(1, cols, 2504)
    up = Uploaded(hl, torch, w)
    got = gpu_decode(hl, torch, up)
    assert np.array_equal(got, w)
    y = gpu_gemm(hl, torch, up, x)
    rs = np.random.default_rng(0).choice(rows, 64, replace=False)
    yo, d = orc.matmul(w[rs], x)
    assert np.all(np.abs(y[0, rs] - yo[0]) <= TOL * d[0])
    # a property that holds at any size: y(-x) = -y exactly (sign flips commute with every rounding)
    yn = gpu_gemm(hl, torch, up, x ^ np.uint16(0x8000))
    assert np.array_equal(yn, -y)


@pytest.mark.parametrize("fuse", ["deps", "all"])
def test_full_layer_in_the_benchmarks_launch_groups_sampled(hl, torch, fuse):
    """The whole Llama-7B-shaped layer exactly as bench.py runs it (same generators, same launch groups, the prepared
    multi-matrix call): sampled rows of all seven products against the oracle, twice (results are reproducible)."""
    import bench
    dev = torch.device("cuda", 0)
    mats = bench.prepare("llama7b_layer", 4096, hl, torch, dev, cpu_sample_mats=7)
    groups = bench.launch_groups(wl.LAYER_LLAMA7B, fuse)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    preps = [hl.PreparedMulti([mats[i]["desc"] for i in g], [mats[i]["blob_dev"] for i in g], [mats[i]["x_dev"] for i in g], 1,
                              [mats[i]["y_dev"] for i in g], [mats[i]["ws"] for i in g], max(m["ws_bytes"] for m in mats), err) for g in groups]
    first = None
    for rep in range(2):
        for m in mats:
            m["y_dev"].fill_(float("nan"))
        for p in preps:
            p.run(stream)
        torch.cuda.synchronize()
        assert int(err.item()) == 0
        ys = [m["y_dev"].cpu().numpy() for m in mats]
        if first is None:
            first = ys
        else:
            assert all(np.array_equal(a, b) for a, b in zip(first, ys))
    rng = np.random.default_rng(5)
    for m, y in zip(mats, first):
        rs = rng.choice(m["rows"], 32, replace=False)
        yo, d = orc.matmul(m["w_sample"][rs], m["x_np"])
        assert np.all(np.abs(y[rs] - yo[0]) <= TOL * d[0]), m["name"]
        assert int(m["ws"][:hl.workspace_control_bytes(m["desc"])].count_nonzero().item()) == 0


def test_launches_can_be_captured_in_a_cuda_graph(hl, torch):
    """The device calls only enqueue work on the stream they are given (no allocation, no synchronisation), so a
    step can be captured once and replayed; replays with new activations give the oracle's products."""
    rows, cols = 512, 4096
    w = wl.gaussian_weights(rows, cols, 0.02, 77)
    up = Uploaded(hl, torch, w)
    x0 = wl.activations(1, cols, 78)
    x_dev = torch.from_numpy(x0.view(np.int16).reshape(-1)).cuda()
    y_dev = torch.zeros(rows, dtype=torch.float32, device="cuda")
    hl.decode_gemv(up.desc, up.blob_dev, x_dev, y_dev, up.ws, up.ws_bytes, up.err)      # first call outside the capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.graph(graph, stream=side):
            hl.decode_gemv(up.desc, up.blob_dev, x_dev, y_dev, up.ws, up.ws_bytes, up.err, side)
            hl.decode_gemv(up.desc, up.blob_dev, x_dev, y_dev, up.ws, up.ws_bytes, up.err, side)
    for seed in (79, 80):
        x = wl.activations(1, cols, seed)
        x_dev.copy_(torch.from_numpy(x.view(np.int16).reshape(-1)))
        y_dev.fill_(float("nan"))
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert int(up.err.item()) == 0
        check_product(y_dev.cpu().numpy()[None, :], w, x)
        assert int(up.ws[:hl.workspace_control_bytes(up.desc)].count_nonzero().item()) == 0


STRESS = [
    # generator, chunk_elems — the distribution stress configuration at 4096 x 14336
    ("student", 4096), ("uniform", 4096), ("patterns", 4096), ("gauss", 1024), ("gauss", 16384),
]


@pytest.mark.parametrize("gen,ce", STRESS)
def test_distribution_stress_full_size(hl, torch, gen, ce):
    """4096 x 14336 bf16: heavy tails with outlier rows, uniform exponents (worst compression), every bit pattern,
    and the smallest / largest benchmark chunk sizes.  Decode is compared everywhere with the original tensor;
    the fused product (finite inputs only) on sampled rows with the oracle."""
    rows, cols = 4096, 14336
    w = make(gen, rows, cols, 3000 + ce)
    up = Uploaded(hl, torch, w, ce)
    got = gpu_decode(hl, torch, up)
    assert np.array_equal(got, w)
    del got
    if gen == "patterns":
        return                                     # NaN / Inf weights: decode only
    x = wl.activations(1, cols, 3500)
    y = gpu_gemm(hl, torch, up, x)
    rs = np.random.default_rng(1).choice(rows, 48, replace=False)
    yo, d = orc.matmul(w[rs], x)
    assert np.all(np.abs(y[0, rs] - yo[0]) <= TOL * d[0])


@pytest.mark.parametrize("seed", [1, 3])
def test_random_shapes_formats_and_batches(hl, torch, seed):
    """Seeded random configurations (shape, chunk size, format, code-length limit, split, batch, distribution): decode
    against the original tensor, the product against the oracle.  Two of the cases such a run first met are kept above
    as tests of their own (FP16 records with an odd number of blocks; long records with 512-entry tables on the tensor core)."""
    rng = np.random.default_rng(seed)
    ran = 0
    for case in range(70):
        dtype = rng.choice(["bf16", "bf16", "fp16", "fp16_from_bf16"])
        rows = int(rng.choice([rng.integers(1, 80), rng.integers(80, 700), rng.integers(700, 2600)]))
        cols = int(rng.integers(1, 160)) * 32
        ce = int(rng.choice([512, 1024, 2048, 4096, 8192, 16384]))
        batch = int(rng.choice([1, 1, 2, 5, 8, 9, 13, 16, 17, 32, 33, 64]))
        if dtype == "bf16":
            gen = str(rng.choice(["gauss", "student", "uniform", "skewed"]))
            budget, split = int(rng.choice([0, 0, 9, 10, 12])), int(rng.choice([0, 0, 1]))
            w = make(gen, rows, cols, 7000 + case)
            hd, od = hl.BF16, orc.BF16
        else:
            budget, split = int(rng.choice([0, 0, 7, 9, 12])), 0
            w = (wl.gaussian_weights(rows, cols, 0.02, 7000 + case, str(dtype)) if rng.random() < 0.8
                 else wl.skewed_exponent_weights(rows, cols, 7000 + case, dtype="fp16"))
            hd, od = hl.FP16, orc.FP16
        what = (case, str(dtype), rows, cols, ce, batch, budget, split)
        up = Uploaded(hl, torch, w, ce, budget, batch, split=split, dtype=hd)
        try:
            got = gpu_decode(hl, torch, up)
        except hl.HuffllmError as e:          # records of the largest chunks may not fit shared memory: refused before any launch
            assert "too large" in str(e), what
            continue
        assert np.array_equal(got, w), what
        x = wl.activations(batch, cols, 7500 + case, "bf16" if dtype == "bf16" else "fp16")
        check_product(gpu_gemm(hl, torch, up, x), w, x, od)
        ran += 1
    assert ran >= 55


@pytest.mark.parametrize("rows,cols,ce,gen", [
    (586, 4032, 512, "fp16_from_bf16"),      # one block per chunk, several chunks per warp
    (586, 4032, 512, "fp16"),                # ... through the flat-code decoder
    (2400, 2080, 1024, "fp16"),              # two blocks per chunk, one in each row's last chunk, more chunks than warps
])
def test_fp16_records_with_an_odd_number_of_blocks_in_a_row(hl, torch, rows, cols, ce, gen):
    """An FP16 record's raw part (64 bytes of signs per block) is padded to a whole 128-byte unit when its chunk has an
    odd number of blocks; a warp that goes from such a record straight to its next one must step over the padding.
    (Found by a randomised run: with at most one chunk per warp, as in the smaller cases, the step is never taken.)"""
    w = wl.gaussian_weights(rows, cols, 0.02, 7002, gen)
    up = Uploaded(hl, torch, w, ce, 0, 3, dtype=hl.FP16)
    assert np.array_equal(gpu_decode(hl, torch, up), w)
    for batch in (1, 3):
        x = wl.activations(batch, cols, 7100 + batch, "fp16")
        check_product(gpu_gemm(hl, torch, up, x), w, x, orc.FP16)


@pytest.mark.parametrize("dtype,ce", [("fp16", 4096), ("bf16", 8192)])
def test_single_slots_reused_full_size(hl, torch, dtype, ce):
    """Records that get one shared-memory slot per decoder warp, on a matrix large enough that every warp goes through
    its slot several times (4096 x 8192: 8192 or 4096 chunks for at most 148 x 31 warps at FP16, 8192 x 8192 at BF16):
    decode against the original tensor, products on sampled rows against the oracle."""
    rows, cols = (4096, 8192) if dtype == "fp16" else (8192, 8192)
    w = wl.gaussian_weights(rows, cols, 0.02, 3100 + ce, dtype)
    up = Uploaded(hl, torch, w, ce, 0, 3, dtype=hl.FP16 if dtype == "fp16" else hl.BF16)
    assert hl.decode_launch_plan(up.desc, 1)["slots_per_warp"] == 1
    assert np.array_equal(gpu_decode(hl, torch, up), w)
    rs = np.random.default_rng(2).choice(rows, 32, replace=False)
    for batch in (1, 3):
        x = wl.activations(batch, cols, 3600 + batch, dtype)
        y = gpu_gemm(hl, torch, up, x)
        yo, d = orc.matmul(w[rs], x, orc.FP16 if dtype == "fp16" else orc.BF16)
        assert np.all(np.abs(y[:, rs] - yo) <= TOL * d)


@pytest.mark.parametrize("rows,cols", [(28672, 8192), (8192, 28672)])
def test_ffn70b_shapes_small_batch_sampled(hl, torch, rows, cols):
    """70B-FFN shapes at full size, batch 1 / 4 (register path) and 16 / 64 (tensor-core path), sampled rows."""
    w = wl.gaussian_weights(rows, cols, 0.015, 4000 + rows)
    rs = np.random.default_rng(2).choice(rows, 24, replace=False)
    up = Uploaded(hl, torch, w, 4096, 0, 64)
    for batch in (1, 4, 16, 64):
        x = wl.activations(batch, cols, 4500 + batch)
        y = gpu_gemm(hl, torch, up, x)
        yo, d = orc.matmul(w[rs], x)
        assert np.all(np.abs(y[:, rs] - yo) <= TOL * d), f"batch {batch}"


def test_results_straight_to_pinned_host_memory_and_kernel_copy(hl, torch):
    """y may be pinned host memory (the kernels write the results to the host themselves), and huffllm_stage_copy moves
    small buffers between pinned host memory and the device with a kernel."""
    rows, cols = 1040, 2048
    w = wl.gaussian_weights(rows, cols, 0.02, 77)
    up = Uploaded(hl, torch, w, 4096, 0, 3)
    x = wl.activations(3, cols, 78)
    x_host = torch.from_numpy(x.view(np.int16).reshape(-1).copy()).pin_memory()
    x_dev = torch.zeros(x_host.numel() + 8, dtype=torch.int16, device="cuda")
    y_host = torch.full((3 * rows + 4,), float("nan"), dtype=torch.float32).pin_memory()
    hl.stage_copy(x_dev, x_host, x_host.numel() * 2)
    hl.decode_gemm(up.desc, up.blob_dev, x_dev, 3, y_host, up.ws, up.ws_bytes, up.err)
    torch.cuda.synchronize()
    assert int(up.err.item()) == 0
    assert np.array_equal(x_dev.cpu().numpy()[:x_host.numel()], x_host.numpy()) and not x_dev[x_host.numel():].any()
    y = y_host.numpy()
    assert np.all(np.isnan(y[3 * rows:]))
    check_product(y[:3 * rows].reshape(3, rows), w, x)
    # the same results as through device memory, bit for bit
    assert np.array_equal(gpu_gemm(hl, torch, up, x), y[:3 * rows].reshape(3, rows))
    with pytest.raises(hl.HuffllmError):
        hl.stage_copy(x_dev, x_host, 24)                      # not a multiple of 16
