"""Python face of the CPU oracle (TEST INFRASTRUCTURE — never imported by the library).

Three parts:

1. ctypes wrappers around ``huffllm_oracle.c`` (field split, histogram, Huffman and
   length-limited code lengths, canonical codes, bit-serial encode/decode of
   sequences, double-precision matrix product).
2. The element map of the blob format — which weight of a ``[rows][cols]`` tensor
   sits at which (chunk, lane, step) — written here from the format description,
   with numpy index arithmetic, independently of the library's encoder.
3. A slow reader for blobs produced by the library: it pulls every lane's bits out
   of the byte buffer, hands them to the oracle's bit-serial decoder and checks
   every structural promise of the format on the way.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg use this.
"""
from __future__ import annotations

import ctypes as C
import os
import struct
import subprocess

import numpy as np

BF16, FP16, BF16_E8 = 0, 1, 2     # BF16_E8: bf16 numbers with the exponent coded whole (one 256-symbol field)
MAXSYM = 256
_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "huffllm_oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-Wall", "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"])
    return _SO


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u8p, u16p, u32p, u64p, f64p = (C.POINTER(t) for t in (C.c_uint8, C.c_uint16, C.c_uint32, C.c_uint64, C.c_double))
        L.orc_histogram.argtypes = [C.c_int, u16p, C.c_size_t, u64p]
        L.orc_huffman_lengths.argtypes = [u64p, C.c_int, u8p]
        L.orc_limited_lengths.argtypes = [u64p, C.c_int, C.c_int, u8p]
        L.orc_code_cost.argtypes = [u64p, u8p, C.c_int]
        L.orc_code_cost.restype = C.c_uint64
        L.orc_build_lengths.argtypes = [C.c_int, u64p, C.c_int, u8p, C.POINTER(C.c_int)]
        L.orc_canonical_codes.argtypes = [u8p, C.c_int, u32p]
        L.orc_encode_sequences.argtypes = [C.c_int, u16p, C.c_size_t, C.c_size_t, u8p, u32p, u8p, u64p, u8p]
        L.orc_encode_sequences.restype = C.c_uint64
        L.orc_decode_sequences.argtypes = [C.c_int, u8p, u64p, C.c_size_t, C.c_size_t, u8p, u32p, u8p, u16p, u64p]
        L.orc_decode_sequences.restype = C.c_int64
        L.orc_value.argtypes = [C.c_int, C.c_uint16]
        L.orc_value.restype = C.c_double
        L.orc_matmul.argtypes = [C.c_int, u16p, C.c_size_t, C.c_size_t, u16p, C.c_size_t, f64p, f64p]
        _lib = L
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t)) if a is not None else None


# ----------------------------------------------------------------- codebooks

def num_fields(dtype):
    return {BF16: 2, FP16: 3, BF16_E8: 1}[dtype]


def field_symbols(dtype):
    return {BF16: 16, FP16: 32, BF16_E8: 256}[dtype]


def histogram(w: np.ndarray, dtype=BF16) -> np.ndarray:
    w = np.ascontiguousarray(w, dtype=np.uint16).ravel()
    counts = np.zeros((3, MAXSYM), dtype=np.uint64)
    lib().orc_histogram(dtype, _p(w, C.c_uint16), w.size, _p(counts, C.c_uint64))
    return counts


def huffman_lengths(counts) -> np.ndarray:
    counts = np.ascontiguousarray(counts, dtype=np.uint64)
    out = np.zeros(counts.size, dtype=np.uint8)
    lib().orc_huffman_lengths(_p(counts, C.c_uint64), counts.size, _p(out, C.c_uint8))
    return out


def limited_lengths(counts, cap: int):
    counts = np.ascontiguousarray(counts, dtype=np.uint64)
    out = np.zeros(counts.size, dtype=np.uint8)
    r = lib().orc_limited_lengths(_p(counts, C.c_uint64), counts.size, cap, _p(out, C.c_uint8))
    return out if r >= 0 else None


def code_cost(counts, lengths) -> int:
    return int(sum(int(c) * int(l) for c, l in zip(counts, lengths)))


def build_lengths(counts: np.ndarray, dtype=BF16, budget: int = 0):
    """Code lengths [3][MAXSYM] and the per-field caps chosen under `budget` (0 = unrestricted)."""
    counts = np.ascontiguousarray(counts, dtype=np.uint64)
    lens = np.zeros((3, MAXSYM), dtype=np.uint8)
    caps = (C.c_int * 3)()
    r = lib().orc_build_lengths(dtype, _p(counts, C.c_uint64), budget, _p(lens, C.c_uint8), caps)
    if r != 0:
        raise ValueError("no code fits the budget")
    return lens, list(caps)


def canonical_codes(lengths) -> np.ndarray:
    lengths = np.ascontiguousarray(lengths, dtype=np.uint8)
    out = np.zeros(lengths.size, dtype=np.uint32)
    lib().orc_canonical_codes(_p(lengths, C.c_uint8), lengths.size, _p(out, C.c_uint32))
    return out


def codes_for(lens: np.ndarray) -> np.ndarray:
    return np.stack([canonical_codes(lens[k]) for k in range(3)])


# ----------------------------------------------------- sequences of weights

def encode_sequences(w_seq: np.ndarray, lens, codes, dtype=BF16):
    """w_seq is [n_seq][seq_len] of 16-bit words.  Returns (bits, bit_off, raw): `bits` holds one bit per
    byte, sequence q occupies bits[bit_off[q]:bit_off[q+1]], raw is [n_seq][seq_len] bytes."""
    w_seq = np.ascontiguousarray(w_seq, dtype=np.uint16)
    n_seq, seq_len = w_seq.shape
    lens = np.ascontiguousarray(lens, dtype=np.uint8)
    codes = np.ascontiguousarray(codes, dtype=np.uint32)
    total = lib().orc_encode_sequences(dtype, _p(w_seq, C.c_uint16), n_seq, seq_len, _p(lens, C.c_uint8),
                                       _p(codes, C.c_uint32), None, None, None)
    if total == 2**64 - 1:
        raise ValueError("a weight uses a symbol that has no codeword")
    bits = np.zeros(total, dtype=np.uint8)
    off = np.zeros(n_seq + 1, dtype=np.uint64)
    raw = np.zeros((n_seq, seq_len), dtype=np.uint8)
    lib().orc_encode_sequences(dtype, _p(w_seq, C.c_uint16), n_seq, seq_len, _p(lens, C.c_uint8),
                               _p(codes, C.c_uint32), _p(bits, C.c_uint8), _p(off, C.c_uint64), _p(raw, C.c_uint8))
    return bits, off, raw


def decode_sequences(bits, bit_off, raw, lens, codes, dtype=BF16):
    """Inverse of encode_sequences.  Returns (w_seq, bits_used per sequence)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    bit_off = np.ascontiguousarray(bit_off, dtype=np.uint64)
    raw = np.ascontiguousarray(raw, dtype=np.uint8)
    n_seq, seq_len = raw.shape
    lens = np.ascontiguousarray(lens, dtype=np.uint8)
    codes = np.ascontiguousarray(codes, dtype=np.uint32)
    out = np.zeros((n_seq, seq_len), dtype=np.uint16)
    used = np.zeros(n_seq, dtype=np.uint64)
    r = lib().orc_decode_sequences(dtype, _p(bits, C.c_uint8), _p(bit_off, C.c_uint64), n_seq, seq_len,
                                   _p(lens, C.c_uint8), _p(codes, C.c_uint32), _p(raw, C.c_uint8),
                                   _p(out, C.c_uint16), _p(used, C.c_uint64))
    if r != 0:
        raise ValueError(f"sequence {-r - 1} does not decode")
    return out, used


def value(b: int, dtype=BF16) -> float:
    return float(lib().orc_value(dtype, int(b)))


def matmul(w: np.ndarray, x: np.ndarray, dtype=BF16):
    """y[j][r] = sum_k W[r][k] x[j][k] in double precision, and d = sum_k |W x| per output."""
    w = np.ascontiguousarray(w, dtype=np.uint16)
    x = np.ascontiguousarray(x, dtype=np.uint16)
    if x.ndim == 1:
        x = x[None, :]
    rows, cols = w.shape
    batch = x.shape[0]
    assert x.shape[1] == cols
    y = np.zeros((batch, rows), dtype=np.float64)
    d = np.zeros((batch, rows), dtype=np.float64)
    lib().orc_matmul(dtype, _p(w, C.c_uint16), rows, cols, _p(x, C.c_uint16), batch, _p(y, C.c_double), _p(d, C.c_double))
    return y, d


# ------------------------------------------------------- blob element map
# A chunk is a tile of 16 rows by Kc = chunk_elems/16 columns, cut into blocks of 32 columns.
# Lane l = 4*g + t (g = 0..7, t = 0..3) owns rows g and g+8 of the tile and, in every 32-column
# block, the 8 columns 8t..8t+7.  Each lane carries TWO independent bit sequences: sequence l holds
# row g's weights, sequence 32 + l holds row g+8's, block after block (8 steps per block each).

TILE_ROWS = 16
BLOCK_COLS = 32
def lag_bits(dtype: int) -> int:
    """Zero bits in front of every bit sequence of a blob: 7 for bf16 blobs, 6 for fp16 blobs."""
    return 6 if dtype == FP16 else 7

SEQS = 64          # bit sequences per chunk


def geometry(rows: int, cols: int, chunk_elems: int):
    if chunk_elems % (TILE_ROWS * BLOCK_COLS) or not (512 <= chunk_elems <= 16384):
        raise ValueError("chunk_elems must be a multiple of 512 in [512, 16384]")
    kc = chunk_elems // TILE_ROWS
    return dict(Kc=kc, RG=-(-rows // TILE_ROWS), KC=-(-cols // kc))


def blocks_in_chunk(cols: int, Kc: int, kc: int) -> int:
    return -(-min(Kc, cols - kc * Kc) // BLOCK_COLS)


def element_map(rows: int, cols: int, chunk_elems: int):
    """Yield groups (chunk_ids[n], idx[n][64][steps]): flat tensor index of every (chunk, sequence, step),
    -1 where the position lies outside the tensor (a pad weight).  Chunks are numbered rg*KC + kc; the
    chunks of the last column-chunk form their own group when they hold fewer blocks."""
    geo = geometry(rows, cols, chunk_elems)
    Kc, RG, KC = geo["Kc"], geo["RG"], geo["KC"]
    seq = np.arange(SEQS)
    half, lane = seq // 32, seq % 32
    g, t = lane // 4, lane % 4
    groups = {}
    for kc in range(KC):
        groups.setdefault(blocks_in_chunk(cols, Kc, kc), []).append(kc)
    for nkb, kcs in groups.items():
        steps = np.arange(nkb * 8)
        kb, i = steps // 8, steps % 8
        rg = np.arange(RG)
        kcs = np.asarray(kcs)
        row = rg[:, None, None, None] * 16 + (g + 8 * half)[None, None, :, None] + 0 * steps[None, None, None, :]
        col = kcs[None, :, None, None] * Kc + kb[None, None, None, :] * 32 + t[None, None, :, None] * 8 + i[None, None, None, :]
        row, col = np.broadcast_arrays(row, col)
        idx = np.where((row < rows) & (col < cols), row.astype(np.int64) * cols + col, -1)
        chunk_ids = (rg[:, None] * KC + kcs[None, :]).ravel()
        yield chunk_ids, idx.reshape(len(chunk_ids), SEQS, nkb * 8)


def pad_word(lens: np.ndarray, dtype=BF16) -> int:
    """The weight written at positions outside the tensor: every coded field takes its shortest codeword
    (ties: smallest symbol), raw bits zero."""
    f = []
    for k in range(num_fields(dtype)):
        used = [(int(lens[k][s]), s) for s in range(field_symbols(dtype)) if lens[k][s]]
        f.append(min(used)[1])
    if dtype == FP16:
        return (f[0] << 10 | f[1] << 5 | f[2]) & 0xFFFF
    e = (f[0] << 4 | f[1]) if dtype == BF16 else f[0]
    return (e << 7) & 0xFFFF


def encode_tensor(w: np.ndarray, chunk_elems: int = 4096, budget: int = 8, dtype=BF16):
    """Oracle-side encoding of a whole tensor in the blob's sequence order.  Returns a dict with the code
    (lens, codes, caps), and per chunk id: (bits, bit_off, raw) of its 64 sequences."""
    w = np.ascontiguousarray(w, dtype=np.uint16)
    rows, cols = w.shape
    counts = histogram(w, dtype)
    lens, caps = build_lengths(counts, dtype, budget)
    codes = codes_for(lens)
    pad = pad_word(lens, dtype)
    flat = np.append(w.ravel(), np.uint16(pad))        # index -1 -> pad word
    chunks = {}
    for chunk_ids, idx in element_map(rows, cols, chunk_elems):
        n, _, steps = idx.shape
        seq = flat[idx.reshape(n * SEQS, steps)]
        bits, off, raw = encode_sequences(seq, lens, codes, dtype)
        for a, cid in enumerate(chunk_ids):
            lo, hi = off[a * SEQS], off[a * SEQS + SEQS]
            chunks[int(cid)] = (bits[lo:hi], (off[a * SEQS:a * SEQS + SEQS + 1] - lo).copy(), raw[a * SEQS:a * SEQS + SEQS])
    return dict(rows=rows, cols=cols, chunk_elems=chunk_elems, dtype=dtype, counts=counts, lens=lens,
                codes=codes, caps=caps, pad=pad, chunks=chunks)


def decode_tensor(enc) -> np.ndarray:
    """Decode an encode_tensor() result (or a parsed blob) back to the [rows][cols] tensor."""
    rows, cols, dtype = enc["rows"], enc["cols"], enc["dtype"]
    out = np.zeros(rows * cols + 1, dtype=np.uint16)
    for chunk_ids, idx in element_map(rows, cols, enc["chunk_elems"]):
        for a, cid in enumerate(chunk_ids):
            bits, off, raw = enc["chunks"][int(cid)]
            seq, _ = decode_sequences(bits, off, raw, enc["lens"], enc["codes"], dtype)
            out[idx[a]] = seq                          # index -1 lands in the spare slot
    return out[:-1].reshape(rows, cols)


# ------------------------------------------------------------- blob reader
# Layout (little endian).  Header, 256 bytes:
#   0 magic "HFLM" | 4 u32 version | 8 u32 dtype | 12 u32 chunk_elems | 16 u64 rows | 24 u64 cols
#   32 u32 tile_rows | 36 u32 chunk_cols | 40 u32 row_groups | 44 u32 col_chunks | 48 u64 n_chunks
#   56 u32 lut_bits | 60 u32 lag_bits | 64 u32 n_fields | 68 u8 caps[4] | 72 u16 pad_word | 74 u16 flat_fields (a hint to the device decoders; not used here)
#   76 u32 max_words | 80 u64 off_codebook | 88 u64 off_lut | 96 u64 off_index | 104 u64 off_payload
#   112 u64 payload_bytes | 120 u64 blob_bytes | 128 u64 coded_bits | 136 u64 raw_bits | 144 u64 checksum
# codebook: n_fields == 2: u8 lengths[3][32] (two nibble codes, third row zero); n_fields == 1: u8 lengths[256]
# of the whole-exponent code.  LUT: u32[1 << lut_bits], entry = (code length of the weight) << 16 | E << 7,
# indexed by the next lut_bits stream bits (first bit = bit 0).  index: u32[n_chunks + 1], record offsets in 128-byte
# units from off_payload.  Record of a chunk with nkb blocks: raw bytes [nkb][32 lanes][16] (a lane's 16
# bytes: row g's eight weights, then row g+8's), then W rows of 64 little-endian u32 (row j, sequence s):
# the sequence's bits, bit i in word i // 32 at bit i % 32, starting with lag_bits zero bits (7 for bf16 blobs, 6 for fp16); unused bits
# after the last codeword are zero.

HEADER = struct.Struct("<4sIIIQQIIIIQIII4sHHIQQQQQQQQ")


def parse_header(blob: bytes) -> dict:
    f = HEADER.unpack_from(blob, 0)
    keys = ["magic", "version", "dtype", "chunk_elems", "rows", "cols", "tile_rows", "chunk_cols", "row_groups",
            "col_chunks", "n_chunks", "lut_bits", "lag_bits", "n_fields", "caps", "pad_word", "_r", "max_words",
            "off_codebook", "off_lut", "off_index", "off_payload", "payload_bytes", "blob_bytes", "coded_bits",
            "raw_bits"]
    h = dict(zip(keys, f))
    assert h["magic"] == b"HFLM" and h["version"] == 1, "bad magic/version"
    return h


def parse_blob(blob) -> dict:
    """Read a library blob into the same structure encode_tensor() returns, checking the format's
    promises: geometry fields, monotone record index, zero lag bits, zero tail bits."""
    blob = bytes(blob)
    h = parse_header(blob)
    rows, cols, ce, dtype = h["rows"], h["cols"], h["chunk_elems"], h["dtype"]
    assert (dtype, h["n_fields"]) in ((BF16, 1), (BF16, 2), (FP16, 3))
    scheme = FP16 if dtype == FP16 else (BF16 if h["n_fields"] == 2 else BF16_E8)      # which fields are coded
    geo = geometry(rows, cols, ce)
    assert (h["tile_rows"], h["chunk_cols"], h["row_groups"], h["col_chunks"]) == (16, geo["Kc"], geo["RG"], geo["KC"])
    assert h["n_chunks"] == geo["RG"] * geo["KC"] and h["lag_bits"] == lag_bits(dtype)
    assert h["blob_bytes"] == len(blob)
    for k in ("off_codebook", "off_lut", "off_index", "off_payload"):
        assert h[k] % 256 == 0
    lens = np.zeros((3, MAXSYM), dtype=np.uint8)
    if scheme in (BF16, FP16):
        lens[:, :32] = np.frombuffer(blob, dtype=np.uint8, count=96, offset=h["off_codebook"]).reshape(3, 32)
    else:
        lens[0] = np.frombuffer(blob, dtype=np.uint8, count=256, offset=h["off_codebook"])
    codes = codes_for(lens)
    n_tables = 3 if scheme == FP16 else 1
    lut = np.frombuffer(blob, dtype=np.uint32, count=n_tables << h["lut_bits"], offset=h["off_lut"]).copy()
    index = np.frombuffer(blob, dtype=np.uint32, count=h["n_chunks"] + 1, offset=h["off_index"]).astype(np.int64)
    assert index[0] == 0 and np.all(np.diff(index) > 0) and index[-1] * 128 == h["payload_bytes"]
    assert h["off_payload"] + h["payload_bytes"] <= len(blob)
    chunks, max_words = {}, 0
    for chunk_ids, idx in element_map(rows, cols, ce):
        steps = idx.shape[2]
        nkb = steps // 8
        for a, cid in enumerate(chunk_ids):
            beg = h["off_payload"] + int(index[cid]) * 128
            size = int(index[cid + 1] - index[cid]) * 128
            raw_bytes = nkb * 512 if scheme != FP16 else -(-nkb * 64 // 128) * 128
            W = (size - raw_bytes) // 256
            assert W >= 1 and raw_bytes + W * 256 == size
            max_words = max(max_words, W)
            if scheme != FP16:
                # a lane's 16 bytes: row g's eight weights, then row g+8's, in groups of four weights per 32-bit word:
                # weight j of a group has its mantissa in the low 7 bits of byte (0, 2, 1, 3)[j] and its sign in bit 7
                # of byte (1, 3, 2, 0)[j]
                by = np.frombuffer(blob, dtype=np.uint8, count=nkb * 512, offset=beg).reshape(nkb, 32, 2, 2, 4)
                mant = by[..., [0, 2, 1, 3]] & np.uint8(0x7F)
                sign = by[..., [1, 3, 2, 0]] & np.uint8(0x80)
                raw = (mant | sign).reshape(nkb, 32, 2, 8)
                raw = raw.transpose(2, 1, 0, 3).reshape(SEQS, steps).copy()        # [half][lane] -> sequence
            else:
                # one uint16 per (block, lane): bit p = sign of the first weight of pair p, bit 8 + p of its second;
                # pairs 0..3 are row g's weights (0,1) (2,3) (4,5) (6,7), pairs 4..7 row g+8's
                sg = np.frombuffer(blob, dtype="<u2", count=nkb * 32, offset=beg).reshape(nkb, 32)
                assert not np.frombuffer(blob, dtype=np.uint8, count=raw_bytes - nkb * 64, offset=beg + nkb * 64).any()
                raw = np.zeros((SEQS, steps), dtype=np.uint8)
                for half in range(2):
                    for i in range(8):
                        bit = (i // 2 + 4 * half) + 8 * (i % 2)
                        raw[half * 32:half * 32 + 32, i::8] = ((sg >> bit) & 1).T
            words = np.frombuffer(blob, dtype="<u4", count=W * SEQS, offset=beg + raw_bytes).reshape(W, SEQS)
            seq_bits = ((words.T[:, :, None] >> np.arange(32, dtype=np.uint32)) & 1).astype(np.uint8).reshape(SEQS, W * 32)
            lag = h["lag_bits"]
            assert not seq_bits[:, :lag].any(), "lag bits must be zero"
            body = np.ascontiguousarray(seq_bits[:, lag:])
            off = (np.arange(SEQS + 1, dtype=np.uint64) * np.uint64(body.shape[1]))
            chunks[int(cid)] = (body.ravel(), off, raw)
    enc = dict(rows=rows, cols=cols, chunk_elems=ce, dtype=scheme, lens=lens, codes=codes, caps=list(h["caps"][:3]),
               pad=h["pad_word"], chunks=chunks, header=h, lut=lut)
    assert max_words == h["max_words"]
    return enc


def decode_blob(blob):
    """Full slow decode of a library blob: (tensor, per-chunk per-sequence bits used).  Also checks that
    every bit after a sequence's last codeword is zero and that pad positions hold the pad word."""
    enc = parse_blob(blob)
    rows, cols, dtype = enc["rows"], enc["cols"], enc["dtype"]
    out = np.zeros(rows * cols + 1, dtype=np.uint16)
    used_all = {}
    total = 0
    for chunk_ids, idx in element_map(rows, cols, enc["chunk_elems"]):
        for a, cid in enumerate(chunk_ids):
            bits, off, raw = enc["chunks"][int(cid)]
            seq, used = decode_sequences(bits, off, raw, enc["lens"], enc["codes"], dtype)
            per = bits.reshape(SEQS, -1)
            for l in range(SEQS):
                assert not per[l, int(used[l]):].any(), "non-zero bits after the last codeword"
            assert np.all(seq[idx[a] < 0] == enc["pad"]), "pad positions must hold the pad word"
            out[idx[a]] = seq
            used_all[int(cid)] = used
            total += int(used.sum())
    assert total == enc["header"]["coded_bits"]
    return out[:-1].reshape(rows, cols), used_all


def lut_from_code(lens, codes, lut_bits: int, dtype=BF16) -> np.ndarray:
    """What the blob's LUT must contain, found the slow way: for every index, write its bits out as a
    stream and run one bit-serial decode of a single weight (all its coded fields) on it.
    FP16 blobs hold one table per field: entry = length << 16 | symbol << (10, 5, 0); each is found by decoding
    a single symbol of that field alone (the one-field scheme's decoder, given that field's code)."""
    if dtype == FP16:
        tables = []
        for k in range(3):
            l1, c1 = np.zeros_like(lens), np.zeros_like(codes)
            l1[0], c1[0] = lens[k], codes[k]
            t = lut_from_code(l1, c1, lut_bits, BF16_E8)           # entry = length << 16 | symbol << 7
            tables.append((t & np.uint32(0xFFFF0000)) | (((t >> np.uint32(7)) & np.uint32(0xFF)) << np.uint32(10 - 5 * k)))
        return np.concatenate(tables)
    n = 1 << lut_bits
    idx_bits = ((np.arange(n, dtype=np.uint32)[:, None] >> np.arange(lut_bits, dtype=np.uint32)) & 1).astype(np.uint8)
    out = np.zeros(n, dtype=np.uint32)
    raw = np.zeros((1, 1), dtype=np.uint8)
    for i in range(n):
        off = np.array([0, lut_bits], dtype=np.uint64)
        try:
            seq, used = decode_sequences(idx_bits[i], off, raw, lens, codes, dtype)
        except ValueError:
            continue                                   # no codeword pair is a prefix of this index
        out[i] = (int(used[0]) << 16) | (((int(seq[0, 0]) >> 7) & 0xFF) << 7)
    return out


# ----------------------------------------------------------------- bit-field splits (Section 3.1, entropy table)

def split_fields(w: np.ndarray, widths) -> list:
    """The fields of every 16-bit word under a split: ``widths`` lists the field widths from the most significant
    bit down (the table's "1-5-5-5" is [1, 5, 5, 5], "8-8" is [8, 8], "16" is [16]) and must add up to 16."""
    widths = [int(x) for x in widths]
    if sum(widths) != 16 or any(x < 1 for x in widths):
        raise ValueError("field widths must be positive and add up to 16")
    w = np.ascontiguousarray(w, dtype=np.uint16).ravel().astype(np.uint32)
    out, hi = [], 16
    for width in widths:
        lo = hi - width
        out.append((w >> np.uint32(lo)) & np.uint32((1 << width) - 1))
        hi = lo
    return out


def split_histograms(w: np.ndarray, widths) -> list:
    """Per field, how often each of its 2^width values occurs."""
    return [np.bincount(f, minlength=1 << int(width)).astype(np.uint64) for f, width in zip(split_fields(w, widths), widths)]


def shannon_entropy(counts) -> float:
    """- sum p log2 p over the symbols that occur, in double precision (bits per symbol)."""
    c = np.asarray(counts, dtype=np.float64)
    total = c.sum()
    if total == 0:
        return 0.0
    p = c[c > 0] / total
    return float(-(p * np.log2(p)).sum())


def split_entropy(w: np.ndarray, widths):
    """One row of the entropy table: the entropy of each field, and their sum = bits per parameter of the split."""
    per_field = [shannon_entropy(h) for h in split_histograms(w, widths)]
    return per_field, float(sum(per_field))
