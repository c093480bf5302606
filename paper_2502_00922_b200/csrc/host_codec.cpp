// Host side of the library: codebook construction, encoder, blob validator.
//
// Compression runs once, offline, on the CPU (Section 3.1).  The field split is the paper's
// BF16 {1,4,4,7} scheme (Section 5.1): sign and mantissa stay raw, the exponent is coded as two
// 4-bit groups, each with its own Huffman code.  Code lengths are bounded by a fixed L_max
// (Section 3.2) — here a joint bound on the two nibble codes of one weight, so that the device
// can resolve both with a single table lookup.
#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <new>
#include <thread>
#include <vector>

#include "internal.h"

namespace huffllm {

static thread_local char g_err[512] = "";

huffllm_status fail(huffllm_status st, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return st;
}
void clear_error() { g_err[0] = 0; }

static inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

// Order-independent checksum term of one chunk record.
static inline uint64_t record_checksum(const uint8_t *p, uint64_t n, uint64_t chunk_id) {
    uint64_t h = 1469598103934665603ull;
    for (uint64_t i = 0; i < n; ++i) h = (h ^ p[i]) * 1099511628211ull;
    return h * (2 * chunk_id + 1);
}

huffllm_status check_desc(const huffllm_desc *d) {
    if (!d) return fail(HUFFLLM_ERR_INVALID_ARG, "descriptor is null");
    if (memcmp(d->magic, "HFLM", 4) != 0 || d->version != 1) return fail(HUFFLLM_ERR_CORRUPT, "bad magic or version");
    if (d->dtype != HUFFLLM_BF16 && d->dtype != HUFFLLM_FP16) return fail(HUFFLLM_ERR_CORRUPT, "bad dtype");
    if (d->rows == 0 || d->cols == 0 || d->rows > (1ull << 31) || d->cols > (1ull << 31))
        return fail(HUFFLLM_ERR_CORRUPT, "bad shape");
    if (d->chunk_elems % (kTileRows * kBlockCols) || d->chunk_elems < 512 || d->chunk_elems > 16384)
        return fail(HUFFLLM_ERR_CORRUPT, "bad chunk_elems");
    if (d->tile_rows != kTileRows || d->chunk_cols != d->chunk_elems / kTileRows || d->lag_bits != lag_bits_for(d->dtype) ||
        (d->dtype == HUFFLLM_BF16 && d->n_fields != 2 && d->n_fields != 1) || (d->dtype == HUFFLLM_FP16 && d->n_fields != 3))
        return fail(HUFFLLM_ERR_CORRUPT, "bad tile geometry");
    if (d->flat_fields & ~7u) return fail(HUFFLLM_ERR_CORRUPT, "bad flat_fields");
    if (d->flat_fields && (d->dtype != HUFFLLM_FP16 || d->lut_bits < 5))
        return fail(HUFFLLM_ERR_CORRUPT, "flat_fields set where no field can carry the flat code");
    if (d->row_groups != (d->rows + kTileRows - 1) / kTileRows ||
        d->col_chunks != (d->cols + d->chunk_cols - 1) / d->chunk_cols ||
        d->n_chunks != (uint64_t)d->row_groups * d->col_chunks)
        return fail(HUFFLLM_ERR_CORRUPT, "chunk counts do not match the shape");
    if (d->lut_bits < min_budget_for(d->dtype) || d->lut_bits > kMaxBudget) return fail(HUFFLLM_ERR_CORRUPT, "bad lut_bits");
    uint32_t max_steps = d->chunk_cols / kBlockCols * 8;   // per bit sequence
    uint32_t w_bound = (d->lag_bits + max_steps * d->lut_bits * (d->dtype == HUFFLLM_FP16 ? 3 : 1) + 31) / 32;
    if (d->max_words == 0 || d->max_words > w_bound) return fail(HUFFLLM_ERR_CORRUPT, "bad max_words");
    if (d->off_codebook % 256 || d->off_lut % 256 || d->off_index % 256 || d->off_payload % 256 ||
        d->off_codebook < 256 || d->off_lut < d->off_codebook + (d->n_fields == 1 ? 256u : 96u) ||
        d->off_index < d->off_lut + (d->dtype == HUFFLLM_FP16 ? 3 : 1) * (4ull << d->lut_bits) || d->off_payload < d->off_index + 4 * (d->n_chunks + 1) ||
        d->payload_bytes % kRecordUnit || d->blob_bytes < d->off_payload + d->payload_bytes + kTailSlack ||
        d->payload_bytes / kRecordUnit > 0xFFFFFFFFull)
        return fail(HUFFLLM_ERR_CORRUPT, "bad section offsets");
    return HUFFLLM_OK;
}

// ------------------------------------------------------------------ code construction

// Optimal prefix-code lengths with every length <= cap, by exhaustive dynamic programming over
// the Kraft budget: state = (symbols placed, budget spent in units of 2^-cap).
static bool limited_lengths(const uint64_t *counts, int nsym, int cap, uint8_t *len) {
    std::vector<int> used;
    for (int s = 0; s < nsym; ++s) {
        len[s] = 0;
        if (counts[s]) used.push_back(s);
    }
    int n = (int)used.size();
    if (n == 0) return false;
    if (n == 1) { len[used[0]] = 1; return true; }
    if (cap < 1 || cap > 15 || (1 << cap) < n) return false;
    std::stable_sort(used.begin(), used.end(), [&](int a, int b) { return counts[a] > counts[b]; });
    const int U = 1 << cap;
    const uint64_t INF = ~0ull;
    std::vector<uint64_t> cost((size_t)(n + 1) * (U + 1), INF);
    std::vector<uint8_t> choice((size_t)(n + 1) * (U + 1), 0);
    cost[0] = 0;
    for (int i = 0; i < n; ++i)
        for (int b = 0; b <= U; ++b) {
            uint64_t c = cost[(size_t)i * (U + 1) + b];
            if (c == INF) continue;
            for (int l = 1; l <= cap; ++l) {
                int nb = b + (U >> l);
                if (nb > U) continue;
                uint64_t v = c + counts[used[i]] * (uint64_t)l;
                size_t k = (size_t)(i + 1) * (U + 1) + nb;
                if (v < cost[k]) { cost[k] = v; choice[k] = (uint8_t)l; }
            }
        }
    int best_b = -1;
    for (int b = 0; b <= U; ++b)
        if (cost[(size_t)n * (U + 1) + b] != INF &&
            (best_b < 0 || cost[(size_t)n * (U + 1) + b] < cost[(size_t)n * (U + 1) + best_b]))
            best_b = b;
    if (best_b < 0) return false;
    for (int i = n, b = best_b; i > 0; --i) {
        int l = choice[(size_t)i * (U + 1) + b];
        len[used[i - 1]] = (uint8_t)l;
        b -= U >> l;
    }
    return true;
}

static uint64_t code_cost(const uint64_t *counts, const uint8_t *len, int nsym) {
    uint64_t c = 0;
    for (int s = 0; s < nsym; ++s) c += counts[s] * len[s];
    return c;
}

static void canonical_codes(const uint8_t *len, int nsym, uint32_t *code) {
    std::vector<int> order;
    for (int s = 0; s < nsym; ++s) {
        code[s] = 0;
        if (len[s]) order.push_back(s);
    }
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return len[a] < len[b]; });
    uint32_t next = 0;
    for (size_t i = 0; i < order.size(); ++i) {
        if (i) next = (next + 1) << (len[order[i]] - len[order[i - 1]]);
        code[order[i]] = next;
    }
}

static uint32_t reverse_bits(uint32_t v, int n) {
    uint32_t r = 0;
    for (int i = 0; i < n; ++i) r |= ((v >> i) & 1u) << (n - 1 - i);
    return r;
}

}  // namespace huffllm

using namespace huffllm;

struct huffllm_codebook {
    uint32_t dtype, budget;
    uint32_t n_fields;       // 2: hi/lo nibble codes (len, code);  1: one code for the exponent byte (len_e, code_e)
    uint64_t counts[3][32];
    uint8_t len[3][32];
    uint32_t code[3][32];
    uint64_t counts_e[256];
    uint8_t len_e[256];
    uint32_t code_e[256];
    uint32_t bits5[3][32];   // FP16: stream bits of a field's codeword, first bit in bit 0
    uint8_t caps[4];
    uint16_t pad_word;
    uint8_t len8[256];    // code length of a whole exponent byte (hi + lo), 0 = no codeword
    uint32_t bits8[256];  // its stream bits, first bit in bit 0
    std::vector<uint32_t> lut;
};

// Fill len8 / bits8 / lut / pad_word from len[] and code[].
static void finish_codebook(huffllm_codebook *cb) {
    if (cb->dtype == HUFFLLM_FP16) {
        // three tables, one per field; entry = length << 16 | symbol << (10, 5, 0)
        const uint32_t n = 1u << cb->budget;
        cb->lut.assign((size_t)3 * n, 0u);
        uint32_t pad = 0;
        for (int k = 0; k < 3; ++k) {
            const int shift = 10 - 5 * k;
            int best = -1;
            for (int s = 0; s < 32; ++s) {
                int L = cb->len[k][s];
                cb->bits5[k][s] = 0;
                if (!L) continue;
                if (best < 0 || L < cb->len[k][best]) best = s;
                uint32_t seq = reverse_bits(cb->code[k][s], L);
                cb->bits5[k][s] = seq;
                for (uint32_t hi = 0; hi < (1u << (cb->budget - L)); ++hi)
                    cb->lut[(size_t)k * n + (seq | (hi << L))] = ((uint32_t)L << 16) | ((uint32_t)s << shift);
            }
            pad |= (uint32_t)best << shift;
        }
        cb->pad_word = (uint16_t)pad;
        return;
    }
    memset(cb->len8, 0, sizeof(cb->len8));
    memset(cb->bits8, 0, sizeof(cb->bits8));
    cb->lut.assign((size_t)1 << cb->budget, 0u);
    for (int e = 0; e < 256; ++e) {
        uint32_t seq;
        int L;
        if (cb->n_fields == 2) {
            int h = e >> 4, l = e & 15;
            int lh = cb->len[0][h], ll = cb->len[1][l];
            if (!lh || !ll) continue;
            seq = reverse_bits(cb->code[0][h], lh) | (reverse_bits(cb->code[1][l], ll) << lh);
            L = lh + ll;
        } else {
            L = cb->len_e[e];
            if (!L) continue;
            seq = reverse_bits(cb->code_e[e], L);
        }
        cb->len8[e] = (uint8_t)L;
        cb->bits8[e] = seq;
        for (uint32_t hi = 0; hi < (1u << (cb->budget - L)); ++hi)
            cb->lut[seq | (hi << L)] = ((uint32_t)L << 16) | ((uint32_t)e << 7);
    }
    // pad word: every coded field takes its shortest codeword (ties: the smallest symbol)
    if (cb->n_fields == 2) {
        int f[2];
        for (int k = 0; k < 2; ++k) {
            int best = -1;
            for (int s = 0; s < 16; ++s)
                if (cb->len[k][s] && (best < 0 || cb->len[k][s] < cb->len[k][best])) best = s;
            f[k] = best;
        }
        cb->pad_word = (uint16_t)(((f[0] << 4) | f[1]) << 7);
    } else {
        int best = -1;
        for (int e = 0; e < 256; ++e)
            if (cb->len_e[e] && (best < 0 || cb->len_e[e] < cb->len_e[best])) best = e;
        cb->pad_word = (uint16_t)(best << 7);
    }
}

// Histogram of the exponent byte of a bf16 tensor, threaded over slices.
static void exponent_histogram(const uint16_t *w, uint64_t n, uint64_t hist[256]) {
    unsigned nt = std::max(1u, std::min(16u, std::thread::hardware_concurrency()));
    if (n < (1u << 20)) nt = 1;
    std::vector<std::vector<uint64_t>> part(nt, std::vector<uint64_t>(256, 0));
    std::vector<std::thread> th;
    for (unsigned t = 0; t < nt; ++t)
        th.emplace_back([&, t] {
            uint64_t a = n * t / nt, b = n * (t + 1) / nt;
            uint64_t *h = part[t].data();
            for (uint64_t i = a; i < b; ++i) h[(w[i] >> 7) & 0xFF]++;
        });
    for (auto &x : th) x.join();
    memset(hist, 0, 256 * sizeof(uint64_t));
    for (unsigned t = 0; t < nt; ++t)
        for (int e = 0; e < 256; ++e) hist[e] += part[t][e];
}

extern "C" {

const char *huffllm_last_error(void) { return g_err; }

// The codebook of a tensor from its symbol counts.  FP16: counts3 = the 3 x 32 counters of exponent, upper and lower
// mantissa half.  BF16: counts_e = the 256 counters of the exponent byte (both BF16 splits start from them).
static huffllm_status codebook_from_counts(huffllm_dtype dtype, huffllm_split split, uint32_t max_code_len, const uint64_t *counts3,
                                           const uint64_t *counts_e, huffllm_codebook **out) {
    if (dtype != HUFFLLM_BF16 && dtype != HUFFLLM_FP16) return fail(HUFFLLM_ERR_INVALID_ARG, "bad dtype");
    if (split != HUFFLLM_SPLIT_PAPER && split != HUFFLLM_SPLIT_WHOLE_EXPONENT) return fail(HUFFLLM_ERR_INVALID_ARG, "bad split");
    if (split == HUFFLLM_SPLIT_WHOLE_EXPONENT && dtype != HUFFLLM_BF16) return fail(HUFFLLM_ERR_UNSUPPORTED, "the whole-exponent split is for bf16");
    uint32_t budget = max_code_len ? max_code_len : kDefaultBudget;
    if (budget < min_budget_for(dtype) || budget > kMaxBudget)
        return fail(HUFFLLM_ERR_UNSUPPORTED, "max_code_len must be 0 or in [%u, %u]", min_budget_for(dtype), kMaxBudget);
    huffllm_codebook *cb = new (std::nothrow) huffllm_codebook();
    if (!cb) return fail(HUFFLLM_ERR_NOMEM, "out of host memory");
    cb->dtype = dtype;
    cb->budget = budget;
    memset(cb->counts, 0, sizeof(cb->counts));
    memset(cb->counts_e, 0, sizeof(cb->counts_e));
    memset(cb->len, 0, sizeof(cb->len));
    memset(cb->code, 0, sizeof(cb->code));
    memset(cb->caps, 0, sizeof(cb->caps));

    if (dtype == HUFFLLM_FP16) {
        // {1,5,5,5}: exponent, upper and lower mantissa half, each with its own code limited to `budget`
        cb->n_fields = 3;
        for (int k = 0; k < 3; ++k) {
            memcpy(cb->counts[k], counts3 + 32 * k, 32 * sizeof(uint64_t));
            if (!limited_lengths(cb->counts[k], 32, (int)budget, cb->len[k])) {
                delete cb;
                return fail(HUFFLLM_ERR_INVALID_ARG, "no code fits max_code_len");
            }
            cb->caps[k] = (uint8_t)budget;
            canonical_codes(cb->len[k], 32, cb->code[k]);
        }
        finish_codebook(cb);
        *out = cb;
        return HUFFLLM_OK;
    }
    memcpy(cb->counts_e, counts_e, sizeof(cb->counts_e));
    if (split == HUFFLLM_SPLIT_WHOLE_EXPONENT) {
        cb->n_fields = 1;
        if (!limited_lengths(cb->counts_e, 256, (int)budget, cb->len_e)) {
            delete cb;
            return fail(HUFFLLM_ERR_INVALID_ARG, "no code fits max_code_len");
        }
        cb->caps[0] = (uint8_t)budget;
        canonical_codes(cb->len_e, 256, cb->code_e);
        finish_codebook(cb);
        *out = cb;
        return HUFFLLM_OK;
    }
    // histogram of the exponent byte, folded into the two nibble fields
    cb->n_fields = 2;
    for (int e = 0; e < 256; ++e) {
        cb->counts[0][e >> 4] += cb->counts_e[e];
        cb->counts[1][e & 15] += cb->counts_e[e];
    }

    bool have = false;
    uint64_t best = 0;
    uint8_t l0[32], l1[32];
    for (uint32_t c0 = 1; c0 < budget; ++c0) {
        uint32_t c1 = budget - c0;
        if (!limited_lengths(cb->counts[0], 16, (int)c0, l0) || !limited_lengths(cb->counts[1], 16, (int)c1, l1)) continue;
        uint64_t cost = code_cost(cb->counts[0], l0, 16) + code_cost(cb->counts[1], l1, 16);
        if (!have || cost < best) {
            have = true;
            best = cost;
            cb->caps[0] = (uint8_t)c0;
            cb->caps[1] = (uint8_t)c1;
            memcpy(cb->len[0], l0, 16);
            memcpy(cb->len[1], l1, 16);
        }
    }
    if (!have) {
        delete cb;
        return fail(HUFFLLM_ERR_INVALID_ARG, "no code fits max_code_len");
    }
    canonical_codes(cb->len[0], 16, cb->code[0]);
    canonical_codes(cb->len[1], 16, cb->code[1]);
    finish_codebook(cb);
    *out = cb;
    return HUFFLLM_OK;
}

huffllm_status huffllm_build_codebook_split(const uint16_t *w, uint64_t rows, uint64_t cols, huffllm_dtype dtype,
                                            huffllm_split split, uint32_t max_code_len, huffllm_codebook **out) {
    clear_error();
    if (!w || !out || rows == 0 || cols == 0) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer or empty tensor");
    if (dtype == HUFFLLM_FP16) {
        uint64_t counts3[3 * 32] = {};
        const uint64_t n = rows * cols;
        for (uint64_t i = 0; i < n; ++i) {
            uint16_t v = w[i];
            counts3[(v >> 10) & 31]++;
            counts3[32 + ((v >> 5) & 31)]++;
            counts3[64 + (v & 31)]++;
        }
        return codebook_from_counts(dtype, split, max_code_len, counts3, nullptr, out);
    }
    uint64_t counts_e[256];
    exponent_histogram(w, rows * cols, counts_e);
    return codebook_from_counts(dtype, split, max_code_len, nullptr, counts_e, out);
}

huffllm_status huffllm_build_codebook(const uint16_t *w, uint64_t rows, uint64_t cols, huffllm_dtype dtype,
                                      uint32_t max_code_len, huffllm_codebook **out) {
    return huffllm_build_codebook_split(w, rows, cols, dtype, HUFFLLM_SPLIT_PAPER, max_code_len, out);
}

huffllm_status huffllm_build_codebook_from_counts(const uint64_t *counts, huffllm_dtype dtype, huffllm_split split,
                                                  uint32_t max_code_len, huffllm_codebook **out) {
    clear_error();
    if (!counts || !out) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer");
    uint64_t total = 0;
    for (int i = 0; i < (dtype == HUFFLLM_FP16 ? 32 : 256); ++i) total += counts[i];
    if (total == 0) return fail(HUFFLLM_ERR_INVALID_ARG, "empty tensor");
    return codebook_from_counts(dtype, split, max_code_len, counts, counts, out);
}

huffllm_status huffllm_codebook_get_exponent(const huffllm_codebook *cb, uint64_t counts[256], uint8_t lengths[256],
                                             uint32_t codes[256]) {
    clear_error();
    if (!cb || cb->n_fields != 1) return fail(HUFFLLM_ERR_INVALID_ARG, "not a whole-exponent codebook");
    for (int e = 0; e < 256; ++e) {
        if (counts) counts[e] = cb->counts_e[e];
        if (lengths) lengths[e] = cb->len_e[e];
        if (codes) codes[e] = cb->code_e[e];
    }
    return HUFFLLM_OK;
}

huffllm_status huffllm_codebook_get(const huffllm_codebook *cb, uint32_t field, uint32_t *n_symbols, uint64_t counts[32],
                                    uint8_t lengths[32], uint32_t codes[32]) {
    clear_error();
    if (!cb || cb->n_fields < 2 || field >= cb->n_fields) return fail(HUFFLLM_ERR_INVALID_ARG, "bad codebook or field");
    if (n_symbols) *n_symbols = cb->n_fields == 2 ? 16 : 32;
    for (int s = 0; s < 32; ++s) {
        if (counts) counts[s] = cb->counts[field][s];
        if (lengths) lengths[s] = cb->len[field][s];
        if (codes) codes[s] = cb->code[field][s];
    }
    return HUFFLLM_OK;
}

void huffllm_codebook_free(huffllm_codebook *cb) { delete cb; }

}  // extern "C"

// ------------------------------------------------------------------------------ encoder

namespace {

struct Geometry {
    uint64_t rows, cols;
    uint32_t Kc, RG, KC;
};

bool make_geometry(uint64_t rows, uint64_t cols, uint32_t chunk_elems, Geometry *g) {
    if (chunk_elems % (kTileRows * kBlockCols) || chunk_elems < 512 || chunk_elems > 16384) return false;
    if (rows == 0 || cols == 0 || rows > (1ull << 31) || cols > (1ull << 31)) return false;
    g->rows = rows;
    g->cols = cols;
    g->Kc = chunk_elems / kTileRows;
    g->RG = (uint32_t)((rows + kTileRows - 1) / kTileRows);
    g->KC = (uint32_t)((cols + g->Kc - 1) / g->Kc);
    return true;
}

inline uint32_t blocks_of(const Geometry &g, uint32_t kc) {
    uint64_t left = g.cols - (uint64_t)kc * g.Kc;
    return (uint32_t)((std::min<uint64_t>(left, g.Kc) + kBlockCols - 1) / kBlockCols);
}

// The weight at (chunk, sequence, step) of the element map, or the pad word outside the tensor.
// Sequence s belongs to lane s % 32 and holds row g (s < 32) or row g + 8 (s >= 32) of the tile.
inline uint16_t weight_at(const uint16_t *w, const Geometry &g, uint32_t rg, uint32_t kc, uint32_t seq, uint32_t step,
                          uint16_t pad) {
    uint32_t lane = seq & 31, half = seq >> 5, gg = lane >> 2, t = lane & 3, kb = step >> 3, i = step & 7;
    uint64_t r = (uint64_t)rg * 16 + gg + 8 * half;
    uint64_t c = (uint64_t)kc * g.Kc + (uint64_t)kb * 32 + t * 8 + i;
    return (r < g.rows && c < g.cols) ? w[r * g.cols + c] : pad;
}

template <class F>
void parallel_chunks(uint64_t n, F f) {
    unsigned nt = std::max(1u, std::min(16u, std::thread::hardware_concurrency()));
    if (n < 64) nt = 1;
    std::atomic<uint64_t> next{0};
    std::vector<std::thread> th;
    for (unsigned t = 0; t < nt; ++t)
        th.emplace_back([&] {
            for (;;) {
                uint64_t a = next.fetch_add(16);
                if (a >= n) break;
                for (uint64_t c = a; c < std::min(n, a + 16); ++c) f(c);
            }
        });
    for (auto &x : th) x.join();
}

}  // namespace

namespace huffllm {

// Everything of a blob's descriptor that does not depend on the payload.
void fill_desc_fixed(const huffllm_codebook *cb, uint64_t rows, uint64_t cols, uint32_t chunk_elems, uint32_t Kc, uint32_t RG,
                     uint32_t KC, huffllm_desc *out) {
    huffllm_desc d;
    memset(&d, 0, sizeof(d));
    memcpy(d.magic, "HFLM", 4);
    d.version = 1;
    d.dtype = cb->dtype;
    d.chunk_elems = chunk_elems;
    d.rows = rows;
    d.cols = cols;
    d.tile_rows = kTileRows;
    d.chunk_cols = Kc;
    d.row_groups = RG;
    d.col_chunks = KC;
    d.n_chunks = (uint64_t)RG * KC;
    d.lut_bits = cb->budget;
    d.lag_bits = lag_bits_for(cb->dtype);
    d.n_fields = cb->n_fields;
    memcpy(d.caps, cb->caps, 4);
    d.pad_word = cb->pad_word;
    if (cb->dtype == HUFFLLM_FP16)
        for (int k = 0; k < 3; ++k) {      // flat code: all 32 symbols at 5 bits (canonical codes are then the symbols themselves)
            bool flat = true;
            for (int s = 0; s < 32; ++s) flat = flat && cb->len[k][s] == 5;
            if (flat) d.flat_fields |= (uint16_t)(1u << k);
        }
    d.off_codebook = 256;
    d.off_lut = 512;
    d.off_index = d.off_lut + align_up((cb->dtype == HUFFLLM_FP16 ? 3 : 1) * (4ull << cb->budget), 256);
    d.off_payload = d.off_index + align_up(4 * (d.n_chunks + 1), 256);
    d.raw_bits = (cb->dtype == HUFFLLM_FP16 ? 1 : 8) * rows * cols;
    *out = d;
}

// Header, code lengths and decode table: bytes [0, off_index) of the blob (the caller has zeroed them).
void write_fixed_sections(const huffllm_codebook *cb, const huffllm_desc &d, uint8_t *base) {
    memcpy(base, &d, sizeof(d));
    if (cb->n_fields >= 2) {
        for (int k = 0; k < 3; ++k) memcpy(base + d.off_codebook + 32 * k, cb->len[k], 32);
    } else {
        memcpy(base + d.off_codebook, cb->len_e, 256);
    }
    memcpy(base + d.off_lut, cb->lut.data(), cb->lut.size() * sizeof(uint32_t));
}

// The encoder's view of a codebook: per symbol the code length (0 = no codeword) and the stream bits, first bit in
// bit 0.  BF16: indexed by the exponent byte.  FP16: field k's symbol s at index 32 k + s.
void encoder_tables(const huffllm_codebook *cb, uint8_t len[256], uint32_t bits[256]) {
    memset(len, 0, 256);
    memset(bits, 0, 256 * sizeof(uint32_t));
    if (cb->dtype == HUFFLLM_FP16) {
        for (int k = 0; k < 3; ++k)
            for (int s = 0; s < 32; ++s) {
                len[32 * k + s] = cb->len[k][s];
                bits[32 * k + s] = cb->bits5[k][s];
            }
    } else {
        memcpy(len, cb->len8, 256);
        memcpy(bits, cb->bits8, 256 * sizeof(uint32_t));
    }
}

uint32_t codebook_dtype(const huffllm_codebook *cb) { return cb->dtype; }

}  // namespace huffllm

extern "C" {

huffllm_status huffllm_encode_bound(uint64_t rows, uint64_t cols, huffllm_dtype dtype, uint32_t chunk_elems,
                                    size_t *max_bytes) {
    clear_error();
    Geometry g;
    if (!max_bytes) return fail(HUFFLLM_ERR_INVALID_ARG, "max_bytes is null");
    if (dtype != HUFFLLM_BF16 && dtype != HUFFLLM_FP16) return fail(HUFFLLM_ERR_INVALID_ARG, "bad dtype");
    if (!make_geometry(rows, cols, chunk_elems, &g)) return fail(HUFFLLM_ERR_INVALID_ARG, "bad shape or chunk_elems");
    const uint64_t fields = dtype == HUFFLLM_FP16 ? 3 : 1;
    uint64_t payload = 0;
    for (uint32_t kc = 0; kc < g.KC; ++kc) {
        uint32_t nkb = blocks_of(g, kc);
        uint64_t w = (lag_bits_for(dtype) + (uint64_t)nkb * 8 * kMaxBudget * fields + 31) / 32;
        payload += (uint64_t)g.RG * (raw_part_bytes(dtype, nkb) + w * 256ull);
    }
    uint64_t n_chunks = (uint64_t)g.RG * g.KC;
    *max_bytes = (size_t)(256 + 256 + align_up(fields * (4ull << kMaxBudget), 256) + align_up(4 * (n_chunks + 1), 256) + payload + 256 + kTailSlack);
    return HUFFLLM_OK;
}

huffllm_status huffllm_encode(const huffllm_codebook *cb, const uint16_t *w, uint64_t rows, uint64_t cols,
                              uint32_t chunk_elems, void *blob, size_t blob_cap, huffllm_desc *desc) {
    clear_error();
    if (!cb || !w || !blob || !desc) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer");
    Geometry g;
    if (!make_geometry(rows, cols, chunk_elems, &g)) return fail(HUFFLLM_ERR_INVALID_ARG, "bad shape or chunk_elems");
    const uint64_t n_chunks = (uint64_t)g.RG * g.KC;

    huffllm_desc d;
    fill_desc_fixed(cb, rows, cols, chunk_elems, g.Kc, g.RG, g.KC, &d);
    const bool fp16 = cb->dtype == HUFFLLM_FP16;
    if (blob_cap < d.off_payload) return fail(HUFFLLM_ERR_BUFFER_TOO_SMALL, "blob capacity below the fixed sections");

    // pass 1: words per sequence (W) of every chunk, from the code lengths alone
    std::vector<uint32_t> words(n_chunks);
    std::vector<uint64_t> chunk_bits(n_chunks);
    std::atomic<int> bad{0};
    const uint8_t *len8 = cb->len8;
    const uint16_t pad = cb->pad_word;
    parallel_chunks(n_chunks, [&](uint64_t c) {
        uint32_t rg = (uint32_t)(c / g.KC), kc = (uint32_t)(c % g.KC), steps = blocks_of(g, kc) * 8;
        uint32_t max_bits = 0;
        uint64_t sum = 0;
        for (uint32_t lane = 0; lane < kSeqs; ++lane) {
            uint32_t bits = 0;
            for (uint32_t s = 0; s < steps; ++s) {
                const uint16_t v = weight_at(w, g, rg, kc, lane, s, pad);
                if (fp16) {
                    uint32_t l0 = cb->len[0][(v >> 10) & 31], l1 = cb->len[1][(v >> 5) & 31], l2 = cb->len[2][v & 31];
                    if (!l0 || !l1 || !l2) bad.store(1);
                    bits += l0 + l1 + l2;
                } else {
                    uint32_t l = len8[(v >> 7) & 0xFF];
                    if (!l) bad.store(1);
                    bits += l;
                }
            }
            sum += bits;
            max_bits = std::max(max_bits, bits + d.lag_bits);
        }
        words[c] = std::max(1u, (max_bits + 31) / 32);
        chunk_bits[c] = sum;
    });
    if (bad.load()) return fail(HUFFLLM_ERR_INVALID_ARG, "a weight uses a symbol the codebook has no codeword for");

    uint8_t *base = (uint8_t *)blob;
    std::vector<uint64_t> rec(n_chunks + 1, 0);
    uint32_t max_words = 0;
    uint64_t coded_bits = 0;
    for (uint64_t c = 0; c < n_chunks; ++c) {
        uint32_t nkb = blocks_of(g, (uint32_t)(c % g.KC));
        rec[c + 1] = rec[c] + (raw_part_bytes(cb->dtype, nkb) + words[c] * 256ull) / kRecordUnit;
        max_words = std::max(max_words, words[c]);
        coded_bits += chunk_bits[c];
    }
    d.max_words = max_words;
    d.payload_bytes = rec[n_chunks] * kRecordUnit;
    d.blob_bytes = d.off_payload + d.payload_bytes + kTailSlack;
    d.coded_bits = coded_bits;
    d.raw_bits = (fp16 ? 1 : 8) * rows * cols;
    if (rec[n_chunks] > 0xFFFFFFFFull) return fail(HUFFLLM_ERR_UNSUPPORTED, "payload exceeds the 32-bit record index");
    if (blob_cap < d.blob_bytes)
        return fail(HUFFLLM_ERR_BUFFER_TOO_SMALL, "blob needs %llu bytes, capacity is %llu", (unsigned long long)d.blob_bytes,
                    (unsigned long long)blob_cap);

    memset(base, 0, d.off_payload);
    memset(base + d.off_payload + d.payload_bytes, 0, kTailSlack);
    write_fixed_sections(cb, d, base);
    uint32_t *index = (uint32_t *)(base + d.off_index);
    for (uint64_t c = 0; c <= n_chunks; ++c) index[c] = (uint32_t)rec[c];

    // pass 2: write the records
    const uint32_t *bits8 = cb->bits8;
    std::atomic<uint64_t> checksum{0};
    parallel_chunks(n_chunks, [&](uint64_t c) {
        uint32_t rg = (uint32_t)(c / g.KC), kc = (uint32_t)(c % g.KC), nkb = blocks_of(g, kc), steps = nkb * 8;
        uint32_t W = words[c];
        uint8_t *raw = base + d.off_payload + rec[c] * kRecordUnit;
        const uint32_t raw_bytes = raw_part_bytes(cb->dtype, nkb);
        uint32_t *coded = (uint32_t *)(raw + raw_bytes);
        memset(coded, 0, (size_t)W * 256);
        memset(raw, 0, raw_bytes);
        for (uint32_t lane = 0; lane < kSeqs; ++lane) {
            uint64_t acc = 0;
            uint32_t nacc = d.lag_bits, j = 0;
            auto append = [&](uint32_t bits, uint32_t len) {      // len <= 16, nacc < 32
                acc |= (uint64_t)bits << nacc;
                nacc += len;
                if (nacc >= 32) {
                    coded[(size_t)j++ * kSeqs + lane] = (uint32_t)acc;
                    acc >>= 32;
                    nacc -= 32;
                }
            };
            for (uint32_t s = 0; s < steps; ++s) {
                uint16_t v = weight_at(w, g, rg, kc, lane, s, pad);
                if (fp16) {
                    // sign bit of weight i of the sequence: pair p = i / 2 (+ 4 for the row g + 8 sequence), bit p (+ 8 if odd)
                    uint32_t i = s & 7, p = (i >> 1) + 4 * (lane >> 5), bit = p + 8 * (i & 1);
                    uint16_t *sg = (uint16_t *)(raw + (s >> 3) * 64 + (lane & 31) * 2);
                    *sg = (uint16_t)(*sg | ((v >> 15) << bit));
                    uint32_t f[3] = {(uint32_t)(v >> 10) & 31, (uint32_t)(v >> 5) & 31, (uint32_t)v & 31};
                    for (int k = 0; k < 3; ++k) append(cb->bits5[k][f[k]], cb->len[k][f[k]]);
                } else {
                    uint8_t *grp = raw + (s >> 3) * 512 + (lane & 31) * 16 + (lane >> 5) * 8 + (s & 4);    // the weight's group of four
                    grp[kRawMantByte[s & 3]] |= (uint8_t)(v & 0x7F);
                    grp[kRawSignByte[s & 3]] |= (uint8_t)((v >> 8) & 0x80);
                    uint32_t e = (v >> 7) & 0xFF;
                    append(bits8[e], len8[e]);
                }
            }
            if (nacc) coded[(size_t)j * kSeqs + lane] = (uint32_t)acc;
        }
        checksum.fetch_add(record_checksum(raw, raw_bytes + (uint64_t)W * 256, c));
    });
    d.payload_checksum = checksum.load();
    memcpy(base, &d, sizeof(d));
    *desc = d;
    return HUFFLLM_OK;
}

huffllm_status huffllm_validate_blob(const void *blob, size_t bytes, huffllm_desc *desc_out) {
    clear_error();
    if (!blob || bytes < 256) return fail(HUFFLLM_ERR_CORRUPT, "blob shorter than its header");
    huffllm_desc d;
    memcpy(&d, blob, sizeof(d));
    huffllm_status st = check_desc(&d);
    if (st != HUFFLLM_OK) return st == HUFFLLM_ERR_UNSUPPORTED ? st : HUFFLLM_ERR_CORRUPT;
    if (d.blob_bytes != bytes) return fail(HUFFLLM_ERR_CORRUPT, "blob_bytes does not match the buffer size");
    const uint8_t *base = (const uint8_t *)blob;

    // codebook: used symbols must form a complete prefix code (a single 1-bit code is the one exception)
    huffllm_codebook cb;
    memset(cb.counts, 0, sizeof(cb.counts));
    memset(cb.code, 0, sizeof(cb.code));
    cb.dtype = d.dtype;
    cb.budget = d.lut_bits;
    cb.n_fields = d.n_fields;
    memset(cb.len, 0, sizeof(cb.len));
    memset(cb.len_e, 0, sizeof(cb.len_e));
    memset(cb.code_e, 0, sizeof(cb.code_e));
    // Kraft sum of one stored code: complete, or the single 1-bit code
    auto check_code = [&](const uint8_t *len, int slots, int nsym, int cap, int k) -> bool {
        uint64_t kraft = 0;
        int used = 0, mx = 0;
        for (int s = 0; s < slots; ++s) {
            int l = len[s];
            if (!l) continue;
            if (s >= nsym || l > 15) { fail(HUFFLLM_ERR_CORRUPT, "code length out of range"); return false; }
            kraft += 1ull << (16 - l);
            ++used;
            mx = std::max(mx, l);
        }
        if (used == 0) { fail(HUFFLLM_ERR_CORRUPT, "field %d has no codewords", k); return false; }
        if (!(kraft == (1ull << 16) || (used == 1 && mx == 1))) { fail(HUFFLLM_ERR_CORRUPT, "field %d is not a complete prefix code", k); return false; }
        if (mx > cap) { fail(HUFFLLM_ERR_CORRUPT, "field %d exceeds its cap", k); return false; }
        return true;
    };
    const bool fp16 = d.dtype == HUFFLLM_FP16;
    if (fp16) {
        for (int k = 0; k < 3; ++k) {
            memcpy(cb.len[k], base + d.off_codebook + 32 * k, 32);
            if (!check_code(cb.len[k], 32, 32, d.caps[k], k)) return HUFFLLM_ERR_CORRUPT;
            if (d.caps[k] > d.lut_bits) return fail(HUFFLLM_ERR_CORRUPT, "caps exceed lut_bits");
            if (d.flat_fields >> k & 1u)
                for (int s = 0; s < 32; ++s)
                    if (cb.len[k][s] != 5) return fail(HUFFLLM_ERR_CORRUPT, "flat_fields names a field whose code is not flat");
            canonical_codes(cb.len[k], 32, cb.code[k]);
        }
    } else if (d.n_fields == 2) {
        for (int k = 0; k < 3; ++k) memcpy(cb.len[k], base + d.off_codebook + 32 * k, 32);
        for (int k = 0; k < 2; ++k)
            if (!check_code(cb.len[k], 32, 16, d.caps[k], k)) return HUFFLLM_ERR_CORRUPT;
        for (int s = 0; s < 32; ++s)
            if (cb.len[2][s]) return fail(HUFFLLM_ERR_CORRUPT, "unexpected third field");
        if (d.caps[0] + d.caps[1] > (int)d.lut_bits) return fail(HUFFLLM_ERR_CORRUPT, "caps exceed lut_bits");
        canonical_codes(cb.len[0], 16, cb.code[0]);
        canonical_codes(cb.len[1], 16, cb.code[1]);
    } else {
        memcpy(cb.len_e, base + d.off_codebook, 256);
        if (!check_code(cb.len_e, 256, 256, d.caps[0], 0)) return HUFFLLM_ERR_CORRUPT;
        if (d.caps[0] > d.lut_bits || d.caps[1]) return fail(HUFFLLM_ERR_CORRUPT, "caps exceed lut_bits");
        canonical_codes(cb.len_e, 256, cb.code_e);
    }
    finish_codebook(&cb);
    if (memcmp(cb.lut.data(), base + d.off_lut, cb.lut.size() * sizeof(uint32_t)) != 0) return fail(HUFFLLM_ERR_CORRUPT, "LUT does not match the codebook");
    if (cb.pad_word != d.pad_word) return fail(HUFFLLM_ERR_CORRUPT, "pad_word does not match the codebook");

    Geometry g;
    make_geometry(d.rows, d.cols, d.chunk_elems, &g);
    const uint32_t *index = (const uint32_t *)(base + d.off_index);
    if (index[0] != 0 || (uint64_t)index[d.n_chunks] * kRecordUnit != d.payload_bytes)
        return fail(HUFFLLM_ERR_CORRUPT, "record index does not span the payload");
    std::atomic<int> bad{0};
    std::atomic<uint64_t> total_bits{0}, checksum{0};
    std::atomic<uint32_t> max_words{0};
    const uint32_t mask = (1u << d.lut_bits) - 1;
    parallel_chunks(d.n_chunks, [&](uint64_t c) {
        uint32_t kc = (uint32_t)(c % g.KC), rg = (uint32_t)(c / g.KC), nkb = blocks_of(g, kc), steps = nkb * 8;
        if (index[c + 1] <= index[c]) { bad.store(1); return; }
        uint64_t size = (uint64_t)(index[c + 1] - index[c]) * kRecordUnit;
        const uint64_t raw_bytes = raw_part_bytes(d.dtype, nkb);
        if (size <= raw_bytes) { bad.store(2); return; }
        if ((size - raw_bytes) % 256) { bad.store(9); return; }
        uint32_t W = (uint32_t)((size - raw_bytes) / 256);
        if (W > d.max_words) { bad.store(3); return; }
        uint32_t seen = max_words.load();
        while (W > seen && !max_words.compare_exchange_weak(seen, W)) {}
        const uint8_t *raw = base + d.off_payload + (uint64_t)index[c] * kRecordUnit;
        const uint32_t *coded = (const uint32_t *)(raw + raw_bytes);
        uint64_t sum = 0;
        if (fp16)
            for (uint64_t b = nkb * 64ull; b < raw_bytes; ++b)
                if (raw[b]) { bad.store(10); return; }          // padding behind the sign bits
        for (uint32_t lane = 0; lane < kSeqs; ++lane) {
            auto word = [&](uint32_t j) -> uint64_t { return j < W ? coded[(size_t)j * kSeqs + lane] : 0; };
            if (word(0) & ((1u << d.lag_bits) - 1)) { bad.store(4); return; }
            uint32_t pos = d.lag_bits;
            for (uint32_t s = 0; s < steps; ++s) {
                uint32_t ln = lane & 31, half = lane >> 5, gg = ln >> 2, t = ln & 3, kb = s >> 3, i = s & 7;
                uint64_t r = (uint64_t)rg * 16 + gg + 8 * half, col = (uint64_t)kc * g.Kc + kb * 32ull + t * 8 + i;
                const bool outside = r >= g.rows || col >= g.cols;
                if (fp16) {
                    uint32_t word15 = 0;
                    for (uint32_t k = 0; k < 3; ++k) {
                        uint64_t win = (word(pos >> 5) | (word((pos >> 5) + 1) << 32)) >> (pos & 31);
                        uint32_t e = cb.lut[((size_t)k << d.lut_bits) + ((uint32_t)win & mask)];
                        uint32_t l = e >> 16;
                        if (!l) { bad.store(5); return; }
                        word15 |= e & 0x7FFFu;
                        pos += l;
                        sum += l;
                    }
                    if (outside) {
                        uint32_t bit = ((i >> 1) + 4 * half) + 8 * (i & 1);
                        uint16_t sg = *(const uint16_t *)(raw + kb * 64 + ln * 2);
                        if (((sg >> bit) & 1) || word15 != d.pad_word) { bad.store(6); return; }
                    }
                    continue;
                }
                uint64_t win = (word(pos >> 5) | (word((pos >> 5) + 1) << 32)) >> (pos & 31);
                uint32_t e = cb.lut[(uint32_t)win & mask];
                uint32_t l = e >> 16;
                if (!l) { bad.store(5); return; }
                if (outside) {
                    const uint8_t *grp = raw + (s >> 3) * 512 + ln * 16 + half * 8 + (s & 4);
                    uint8_t rb = (uint8_t)((grp[kRawMantByte[s & 3]] & 0x7F) | (grp[kRawSignByte[s & 3]] & 0x80));
                    if (rb != 0 || ((e >> 7) & 0xFFu) != ((d.pad_word >> 7) & 0xFFu)) { bad.store(6); return; }
                }
                pos += l;
                sum += l;
            }
            if (pos > W * 32) { bad.store(7); return; }
            for (uint32_t p = pos; p < W * 32; ++p)
                if ((word(p >> 5) >> (p & 31)) & 1) { bad.store(8); return; }
        }
        total_bits.fetch_add(sum);
        checksum.fetch_add(record_checksum(raw, size, c));
    });
    if (bad.load()) return fail(HUFFLLM_ERR_CORRUPT, "payload check %d failed", bad.load());
    if (total_bits.load() != d.coded_bits) return fail(HUFFLLM_ERR_CORRUPT, "coded_bits does not match the payload");
    if (max_words.load() != d.max_words) return fail(HUFFLLM_ERR_CORRUPT, "max_words does not match the payload");
    if (checksum.load() != d.payload_checksum) return fail(HUFFLLM_ERR_CORRUPT, "payload checksum mismatch");
    if (d.raw_bits != (fp16 ? 1 : 8) * d.rows * d.cols) return fail(HUFFLLM_ERR_CORRUPT, "raw_bits does not match the shape");
    if (desc_out) *desc_out = d;
    return HUFFLLM_OK;
}

}  // extern "C"
