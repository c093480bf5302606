"""ctypes binding of include/huffllm.h: same names, argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

BF16, FP16 = 0, 1
SPLIT_PAPER, SPLIT_WHOLE_EXPONENT = 0, 1
_SO = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libhuffllm.so")
_lib = None

STATUS = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "BUFFER_TOO_SMALL", 4: "CORRUPT", 5: "CUDA", 6: "NOMEM"}


class HuffllmError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"huffllm: {STATUS.get(status, status)}: {message}")
        self.status = status
        self.status_name = STATUS.get(status, str(status))


class Desc(C.Structure):
    """huffllm_desc: descriptor of an encoded tensor = first 256 bytes of the blob."""
    _fields_ = [("magic", C.c_char * 4), ("version", C.c_uint32), ("dtype", C.c_uint32), ("chunk_elems", C.c_uint32),
                ("rows", C.c_uint64), ("cols", C.c_uint64), ("tile_rows", C.c_uint32), ("chunk_cols", C.c_uint32),
                ("row_groups", C.c_uint32), ("col_chunks", C.c_uint32), ("n_chunks", C.c_uint64),
                ("lut_bits", C.c_uint32), ("lag_bits", C.c_uint32), ("n_fields", C.c_uint32), ("caps", C.c_uint8 * 4),
                ("pad_word", C.c_uint16), ("flat_fields", C.c_uint16), ("max_words", C.c_uint32),
                ("off_codebook", C.c_uint64), ("off_lut", C.c_uint64), ("off_index", C.c_uint64),
                ("off_payload", C.c_uint64), ("payload_bytes", C.c_uint64), ("blob_bytes", C.c_uint64),
                ("coded_bits", C.c_uint64), ("raw_bits", C.c_uint64), ("payload_checksum", C.c_uint64),
                ("reserved", C.c_uint8 * 104)]


assert C.sizeof(Desc) == 256

_SIGNATURES = {
    "huffllm_build_codebook": [C.c_void_p, C.c_uint64, C.c_uint64, C.c_int, C.c_uint32, C.POINTER(C.c_void_p)],
    "huffllm_build_codebook_split": [C.c_void_p, C.c_uint64, C.c_uint64, C.c_int, C.c_int, C.c_uint32, C.POINTER(C.c_void_p)],
    "huffllm_codebook_get_exponent": [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p],
    "huffllm_codebook_get": [C.c_void_p, C.c_uint32, C.POINTER(C.c_uint32), C.c_void_p, C.c_void_p, C.c_void_p],
    "huffllm_codebook_free": [C.c_void_p],
    "huffllm_encode_bound": [C.c_uint64, C.c_uint64, C.c_int, C.c_uint32, C.POINTER(C.c_size_t)],
    "huffllm_encode": [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint32, C.c_void_p, C.c_size_t, C.POINTER(Desc)],
    "huffllm_validate_blob": [C.c_void_p, C.c_size_t, C.POINTER(Desc)],
    "huffllm_workspace_bytes": [C.POINTER(Desc), C.c_uint32, C.POINTER(C.c_size_t)],
    "huffllm_workspace_control_bytes": [C.POINTER(Desc), C.POINTER(C.c_size_t)],
    "huffllm_decode_smem_plan": [C.POINTER(Desc), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)],
    "huffllm_decode_launch_plan": [C.POINTER(Desc), C.c_uint32, C.c_uint32, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)],
    "huffllm_decode": [C.POINTER(Desc), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p],
    "huffllm_decode_gemv": [C.POINTER(Desc), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p],
    "huffllm_decode_gemm": [C.POINTER(Desc), C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p],
    "huffllm_decode_gemm_multi_host_async": [C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p],
    "huffllm_decode_gemm_multi": [C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_size_t,
                                  C.c_void_p, C.c_void_p],
    "huffllm_decode_gemm_multi_host": [C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p],
    "huffllm_decode_gemm_host": [C.POINTER(Desc), C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p,
                                 C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p],
    "huffllm_decode_gemm_static": [C.POINTER(Desc), C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p],
    "huffllm_stage_copy": [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p],
    "huffllm_plain_gemv": [C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p],
    "huffllm_plain_gemv_multi": [C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p],
    "huffllm_build_codebook_from_counts": [C.c_void_p, C.c_int, C.c_int, C.c_uint32, C.POINTER(C.c_void_p)],
    "huffllm_encode_device_scratch_bytes": [C.c_uint64, C.c_uint64, C.c_uint32, C.POINTER(C.c_size_t)],
    "huffllm_encode_device": [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint32, C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t,
                              C.POINTER(Desc), C.c_void_p],
    "huffllm_split_counts_size": [C.c_void_p, C.c_uint32, C.POINTER(C.c_size_t)],
    "huffllm_split_histogram": [C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p],
    "huffllm_split_entropy": [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p],
    "huffllm_last_error": [],
}


def exported_symbols():
    """Names include/huffllm.h declares; the library must export every one of them."""
    return sorted(_SIGNATURES)


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(_SO):
            raise ImportError(f"{_SO} is missing: build it with `python -m paper_2502_00922_b200.build` "
                              "(there is no fallback implementation)")
        L = C.CDLL(_SO)
        for name, args in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.argtypes = args
            fn.restype = C.c_int
        L.huffllm_codebook_free.restype = None
        L.huffllm_last_error.restype = C.c_char_p
        _lib = L
    return _lib


def last_error() -> str:
    return lib().huffllm_last_error().decode()


def _check(status: int):
    if status != 0:
        raise HuffllmError(status, last_error())


def _ptr(t):
    """Address of a torch tensor, a numpy array, an int, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


class Codebook:
    """Owner of a huffllm_codebook*."""

    def __init__(self, handle, dtype: int = BF16):
        self._h = handle
        self.dtype = dtype

    def get(self, field: int):
        n = C.c_uint32()
        counts = np.zeros(32, np.uint64)
        lengths = np.zeros(32, np.uint8)
        codes = np.zeros(32, np.uint32)
        _check(lib().huffllm_codebook_get(self._h, field, C.byref(n), counts.ctypes.data, lengths.ctypes.data, codes.ctypes.data))
        return n.value, counts, lengths, codes

    def get_exponent(self):
        """Whole-exponent codebooks: (counts, lengths, codes), 256 entries each."""
        counts = np.zeros(256, np.uint64)
        lengths = np.zeros(256, np.uint8)
        codes = np.zeros(256, np.uint32)
        _check(lib().huffllm_codebook_get_exponent(self._h, counts.ctypes.data, lengths.ctypes.data, codes.ctypes.data))
        return counts, lengths, codes

    def free(self):
        if self._h:
            lib().huffllm_codebook_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def build_codebook(w: np.ndarray, dtype: int = BF16, max_code_len: int = 0, split: int = SPLIT_PAPER) -> Codebook:
    w = np.ascontiguousarray(w, dtype=np.uint16)
    rows, cols = w.shape if w.ndim == 2 else (1, w.size)
    h = C.c_void_p()
    if split == SPLIT_PAPER:
        _check(lib().huffllm_build_codebook(w.ctypes.data, rows, cols, dtype, max_code_len, C.byref(h)))
    else:
        _check(lib().huffllm_build_codebook_split(w.ctypes.data, rows, cols, dtype, split, max_code_len, C.byref(h)))
    return Codebook(h, dtype)


def encode_bound(rows: int, cols: int, dtype: int = BF16, chunk_elems: int = 4096) -> int:
    n = C.c_size_t()
    _check(lib().huffllm_encode_bound(rows, cols, dtype, chunk_elems, C.byref(n)))
    return n.value


def encode(cb: Codebook, w: np.ndarray, chunk_elems: int = 4096):
    """Returns (blob as a numpy uint8 array trimmed to its size, Desc)."""
    w = np.ascontiguousarray(w, dtype=np.uint16)
    rows, cols = w.shape
    cap = encode_bound(rows, cols, cb.dtype, chunk_elems)
    buf = np.empty(cap, dtype=np.uint8)
    d = Desc()
    _check(lib().huffllm_encode(cb._h, w.ctypes.data, rows, cols, chunk_elems, buf.ctypes.data, cap, C.byref(d)))
    return buf[:d.blob_bytes].copy(), d


def validate_blob(blob: np.ndarray) -> Desc:
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    d = Desc()
    _check(lib().huffllm_validate_blob(blob.ctypes.data, blob.size, C.byref(d)))
    return d


def workspace_bytes(desc: Desc, batch: int = 1) -> int:
    n = C.c_size_t()
    _check(lib().huffllm_workspace_bytes(C.byref(desc), batch, C.byref(n)))
    return n.value


def workspace_control_bytes(desc: Desc) -> int:
    """huffllm_workspace_control_bytes: the leading bytes of a workspace that are zero between calls."""
    n = C.c_size_t()
    _check(lib().huffllm_workspace_control_bytes(C.byref(desc), C.byref(n)))
    return n.value


def decode_smem_plan(desc: Desc) -> dict:
    """huffllm_decode_smem_plan: table bytes, slot bytes, refill checks per block and guard bytes of a decoder CTA."""
    t, sl, ch, g = C.c_uint32(), C.c_uint32(), C.c_uint32(), C.c_uint32()
    _check(lib().huffllm_decode_smem_plan(C.byref(desc), C.byref(t), C.byref(sl), C.byref(ch), C.byref(g)))
    return {"table_bytes": t.value, "slot_bytes": sl.value, "refill_checks_per_block": ch.value, "guard_bytes": g.value}


def decode_launch_plan(desc: Desc, batch: int = 1, smem_bytes_per_cta: int = 0) -> dict:
    """huffllm_decode_launch_plan: slots per decoder warp (2, or 1 for large records) and the decoder warps that get a place."""
    s, w = C.c_uint32(), C.c_uint32()
    _check(lib().huffllm_decode_launch_plan(C.byref(desc), batch, smem_bytes_per_cta, C.byref(s), C.byref(w)))
    return {"slots_per_warp": s.value, "decoder_warps": w.value}


def decode(desc: Desc, blob_dev, out_dev, err_flag_dev=None, stream=None):
    _check(lib().huffllm_decode(C.byref(desc), _ptr(blob_dev), _ptr(out_dev), _ptr(err_flag_dev), _stream(stream)))


def decode_gemv(desc: Desc, blob_dev, x_dev, y_dev, workspace_dev, workspace_bytes_: int, err_flag_dev=None, stream=None):
    _check(lib().huffllm_decode_gemv(C.byref(desc), _ptr(blob_dev), _ptr(x_dev), _ptr(y_dev), _ptr(workspace_dev),
                                     workspace_bytes_, _ptr(err_flag_dev), _stream(stream)))


def decode_gemm(desc: Desc, blob_dev, x_dev, batch: int, y_dev, workspace_dev, workspace_bytes_: int, err_flag_dev=None,
                stream=None):
    _check(lib().huffllm_decode_gemm(C.byref(desc), _ptr(blob_dev), _ptr(x_dev), batch, _ptr(y_dev), _ptr(workspace_dev),
                                     workspace_bytes_, _ptr(err_flag_dev), _stream(stream)))


def decode_gemm_multi(descs, blobs_dev, xs_dev, batch: int, ys_dev, workspaces_dev, workspace_bytes_each: int,
                      err_flag_dev=None, stream=None):
    """huffllm_decode_gemm_multi: lists of equal length, one entry per matrix."""
    n = len(descs)
    desc_arr = (C.POINTER(Desc) * n)(*[C.pointer(d) for d in descs])
    ptrs = lambda seq: (C.c_void_p * n)(*[_ptr(t) for t in seq])
    _check(lib().huffllm_decode_gemm_multi(n, desc_arr, ptrs(blobs_dev), ptrs(xs_dev), batch, ptrs(ys_dev), ptrs(workspaces_dev),
                                           workspace_bytes_each, _ptr(err_flag_dev), _stream(stream)))


def decode_gemm_multi_host(descs, blobs_dev, xs_host, batch: int, ys_host, x_stages_dev, y_stages_dev, workspaces_dev,
                           workspace_bytes_each: int, err_flag_dev=None, stream=None):
    """huffllm_decode_gemm_multi_host: host activations in, host results out, one wait for the stream."""
    n = len(descs)
    desc_arr = (C.POINTER(Desc) * n)(*[C.pointer(d) for d in descs])
    ptrs = lambda seq: (C.c_void_p * n)(*[_ptr(t) for t in seq])
    _check(lib().huffllm_decode_gemm_multi_host(n, desc_arr, ptrs(blobs_dev), ptrs(xs_host), batch, ptrs(ys_host),
                                                ptrs(x_stages_dev), ptrs(y_stages_dev), ptrs(workspaces_dev),
                                                workspace_bytes_each, _ptr(err_flag_dev), _stream(stream)))


class PreparedMulti:
    """The argument arrays of a huffllm_decode_gemm_multi / _multi_host call, marshalled once.  A caller that issues
    the same launch every step (a decoder layer) pays one foreign call per step instead of rebuilding the arrays.
    The tensors must stay alive and in place for as long as the object is used."""

    def __init__(self, descs, blobs_dev, xs_dev, batch: int, ys_dev, workspaces_dev, workspace_bytes_each: int,
                 err_flag_dev=None, xs_host=None, ys_host=None):
        n = self.n = len(descs)
        self._keep = (descs, blobs_dev, xs_dev, ys_dev, workspaces_dev, err_flag_dev, xs_host, ys_host)
        self.descs = (C.POINTER(Desc) * n)(*[C.pointer(d) for d in descs])
        ptrs = lambda seq: (C.c_void_p * n)(*[_ptr(t) for t in seq])
        self.blobs, self.xs, self.ys, self.wss = ptrs(blobs_dev), ptrs(xs_dev), ptrs(ys_dev), ptrs(workspaces_dev)
        self.xh = ptrs(xs_host) if xs_host is not None else None
        self.yh = ptrs(ys_host) if ys_host is not None else None
        self.batch, self.ws_each, self.err = batch, workspace_bytes_each, _ptr(err_flag_dev)
        self._fn, self._fn_host = lib().huffllm_decode_gemm_multi, lib().huffllm_decode_gemm_multi_host
        self._fn_host_async = lib().huffllm_decode_gemm_multi_host_async

    def run(self, stream: int):
        """Device-resident activations and results; `stream` is the raw cudaStream_t value."""
        st = self._fn(self.n, self.descs, self.blobs, self.xs, self.batch, self.ys, self.wss, self.ws_each, self.err, stream)
        if st:
            _check(st)

    def run_host_async(self, stream: int):
        """Host activations in, host results out, enqueued only: wait for the stream before reading the results."""
        st = self._fn_host_async(self.n, self.descs, self.blobs, self.xh, self.batch, self.yh, self.xs, self.ys, self.wss,
                                 self.ws_each, self.err, stream)
        if st:
            _check(st)

    def run_host(self, stream: int):
        """Host activations in, host results out (returns when the results are on the host)."""
        st = self._fn_host(self.n, self.descs, self.blobs, self.xh, self.batch, self.yh, self.xs, self.ys, self.wss,
                           self.ws_each, self.err, stream)
        if st:
            _check(st)


def decode_gemm_host(desc: Desc, blob_dev, x_host, batch: int, y_host, x_stage_dev, y_stage_dev, workspace_dev,
                     workspace_bytes_: int, err_flag_dev=None, stream=None):
    _check(lib().huffllm_decode_gemm_host(C.byref(desc), _ptr(blob_dev), _ptr(x_host), batch, _ptr(y_host),
                                          _ptr(x_stage_dev), _ptr(y_stage_dev), _ptr(workspace_dev), workspace_bytes_,
                                          _ptr(err_flag_dev), _stream(stream)))


STATIC_MAX_BATCH = 8


def decode_gemm_static(desc: Desc, blob_dev, x_dev, batch: int, y_dev, err_flag_dev=None, stream=None):
    """huffllm_decode_gemm_static: the product with the library's built-in scratch (no workspace argument)."""
    _check(lib().huffllm_decode_gemm_static(C.byref(desc), _ptr(blob_dev), _ptr(x_dev), batch, _ptr(y_dev),
                                            _ptr(err_flag_dev), _stream(stream)))


def plain_gemv(w_dev, rows: int, cols: int, x_dev, y_dev, stream=None):
    _check(lib().huffllm_plain_gemv(_ptr(w_dev), rows, cols, _ptr(x_dev), _ptr(y_dev), _stream(stream)))


class PreparedPlainMulti:
    """The argument arrays of a huffllm_plain_gemv_multi call, marshalled once (the tensors must stay alive and in place)."""

    def __init__(self, ws_dev, rows, cols, xs_dev, ys_dev):
        n = self.n = len(ws_dev)
        self._keep = (ws_dev, xs_dev, ys_dev)
        ptrs = lambda seq: (C.c_void_p * n)(*[_ptr(t) for t in seq])
        self.ws, self.xs, self.ys = ptrs(ws_dev), ptrs(xs_dev), ptrs(ys_dev)
        self.rows, self.cols = (C.c_uint64 * n)(*rows), (C.c_uint64 * n)(*cols)
        self._fn = lib().huffllm_plain_gemv_multi

    def run(self, stream: int):
        st = self._fn(self.n, self.ws, self.rows, self.cols, self.xs, self.ys, stream)
        if st:
            _check(st)


def plain_gemv_multi(ws_dev, rows, cols, xs_dev, ys_dev, stream=None):
    """huffllm_plain_gemv_multi: several dense bf16 products in one launch (lists of equal length)."""
    PreparedPlainMulti(ws_dev, rows, cols, xs_dev, ys_dev).run(_stream(stream))


def _widths(widths) -> np.ndarray:
    return np.ascontiguousarray(list(widths), dtype=np.uint8)


def split_counts_size(widths) -> int:
    """huffllm_split_counts_size: counters of a split (sum of 2^width over its fields)."""
    wd, n = _widths(widths), C.c_size_t(0)
    _check(lib().huffllm_split_counts_size(wd.ctypes.data, wd.size, C.byref(n)))
    return n.value


def split_histogram(w_dev, n_weights: int, widths, counts_dev, stream=None):
    """huffllm_split_histogram: per-field value counts of 16-bit words in device memory (counts_dev: uint64, device)."""
    wd = _widths(widths)
    _check(lib().huffllm_split_histogram(_ptr(w_dev), n_weights, wd.ctypes.data, wd.size, _ptr(counts_dev), _stream(stream)))


def split_entropy(counts_host: np.ndarray, widths, huffman: bool = True):
    """huffllm_split_entropy: (entropy per field, Huffman bits per field or None) from host counters."""
    wd = _widths(widths)
    counts = np.ascontiguousarray(counts_host, dtype=np.uint64)
    if counts.size != sum(1 << int(x) for x in wd):
        raise ValueError("counter array does not match the split")
    ent = np.zeros(wd.size, dtype=np.float64)
    huf = np.zeros(wd.size, dtype=np.float64) if huffman else None
    _check(lib().huffllm_split_entropy(counts.ctypes.data, wd.ctypes.data, wd.size, ent.ctypes.data, _ptr(huf)))
    return ent, huf


def build_codebook_from_counts(counts_host: np.ndarray, dtype: int = BF16, max_code_len: int = 0, split: int = SPLIT_PAPER) -> Codebook:
    """huffllm_build_codebook_from_counts: BF16: 256 exponent-byte counters; FP16: 96 counters (exponent, upper, lower mantissa half)."""
    counts = np.ascontiguousarray(counts_host, dtype=np.uint64)
    if counts.size != (96 if dtype == FP16 else 256):
        raise ValueError("counter array does not match the dtype")
    h = C.c_void_p()
    _check(lib().huffllm_build_codebook_from_counts(counts.ctypes.data, dtype, split, max_code_len, C.byref(h)))
    return Codebook(h, dtype)


def encode_device_scratch_bytes(rows: int, cols: int, chunk_elems: int = 4096) -> int:
    n = C.c_size_t(0)
    _check(lib().huffllm_encode_device_scratch_bytes(rows, cols, chunk_elems, C.byref(n)))
    return n.value


def encode_device(cb: Codebook, w_dev, rows: int, cols: int, chunk_elems, blob_dev, blob_cap: int, scratch_dev, scratch_bytes: int,
                  stream=None) -> Desc:
    """huffllm_encode_device: encode weights resident on the device into blob_dev; returns the descriptor."""
    desc = Desc()
    _check(lib().huffllm_encode_device(cb._h, _ptr(w_dev), rows, cols, chunk_elems, _ptr(blob_dev), blob_cap, _ptr(scratch_dev),
                                       scratch_bytes, C.byref(desc), _stream(stream)))
    return desc


def stage_copy(dst, src, nbytes: int, stream=None):
    """huffllm_stage_copy: a small copy by a kernel between device-accessible buffers (device or pinned host memory)."""
    _check(lib().huffllm_stage_copy(_ptr(dst), _ptr(src), nbytes, _stream(stream)))
