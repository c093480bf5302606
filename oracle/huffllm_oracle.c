/*
 * CPU oracle for field-split Huffman compression of 16-bit floating-point weights
 * and for the matrix products that consume the decoded weights.
 *
 * THIS IS TEST INFRASTRUCTURE.  It is deliberately plain and slow: one bit per
 * byte in its bitstreams, linear searches where hardware would use a CAM, double
 * precision sums in index order.  It shares no code, header, table or constant
 * with the CUDA library and is only ever called from the tests, the smoke check
 * and the CPU-baseline leg of the benchmark.
 *
 * What follows the paper, by passage:
 *   - field split FP16 {1,5,5,5}: sign raw; exponent, upper five and lower five
 *     mantissa bits each coded by its own Huffman code      (Section 3.1)
 *   - field split BF16 {1,4,4,7}: sign and the seven mantissa bits raw; the
 *     8-bit exponent is coded as two 4-bit groups            (Section 5.1)
 *   - BF16 with the exponent coded whole, {1,8,7}: one 256-symbol code; the
 *     split the paper's entropy table lists and sets aside because a 256-entry
 *     CAM is too large for its hardware decoder              (Section 3.1, entropy table)
 *   - decoder: compare the bits at the start pointer with every stored codeword,
 *     emit the matching symbol, advance the pointer by that codeword's length
 *                                                           (Section 3.2, decoder figure)
 *   - L_max is a fixed, known bound on the codeword length   (Section 3.2)
 *   - the decoded weight is sign | exponent | mantissa put back together, and it
 *     is used only to be multiplied with activations        (Sections 1, 3.2)
 *
 * Readings where the paper is silent are listed in the repository's design notes;
 * the ones that matter here: ties in the Huffman merge are broken by
 * (weight, node id) with leaves numbered by symbol and merged nodes numbered
 * 1000, 1001, ... in creation order; a field with one used symbol gets a 1-bit
 * code; length limits use package-merge (optimal length-limited prefix code).
 *
 * Parity pins (tests/test_oracle_pins.py): Kraft equality, brute-force optimal
 * lengths on small alphabets (free and length-limited), dyadic and Fibonacci
 * closed forms, entropy bounds, prefix-freeness, a hand-worked 8-weight example,
 * round trips over every 16-bit pattern, closed-form matrix products.
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

#define ORC_MAXSYM 256
#define ORC_BF16 0      /* {1,4,4,7} */
#define ORC_FP16 1      /* {1,5,5,5} */
#define ORC_BF16_E8 2   /* {1,8,7}: BF16 numbers, exponent coded as one 8-bit symbol */

/* ------------------------------------------------------------------ fields */

int orc_num_fields(int dtype) { return dtype == ORC_BF16 ? 2 : dtype == ORC_FP16 ? 3 : 1; }
int orc_field_symbols(int dtype) { return dtype == ORC_BF16 ? 16 : dtype == ORC_FP16 ? 32 : 256; }
int orc_raw_bits(int dtype) { return dtype == ORC_FP16 ? 1 : 8; }

/* Split one 16-bit word into its coded fields f[] and its raw (uncoded) bits.
 * BF16: word = s(1) E(8) m(7);  f0 = E>>4, f1 = E&15, raw = s<<7 | m.
 * FP16: word = s(1) E(5) M(10); f0 = E, f1 = M>>5, f2 = M&31, raw = s.
 * BF16 whole exponent: f0 = E, raw = s<<7 | m.                               */
void orc_split(int dtype, uint16_t b, uint8_t f[3], uint8_t *raw)
{
    if (dtype == ORC_BF16) {
        unsigned s = b >> 15, e = (b >> 7) & 0xFF, m = b & 0x7F;
        f[0] = (uint8_t)(e >> 4); f[1] = (uint8_t)(e & 15); f[2] = 0;
        *raw = (uint8_t)((s << 7) | m);
    } else if (dtype == ORC_BF16_E8) {
        unsigned s = b >> 15, e = (b >> 7) & 0xFF, m = b & 0x7F;
        f[0] = (uint8_t)e; f[1] = 0; f[2] = 0;
        *raw = (uint8_t)((s << 7) | m);
    } else {
        unsigned s = b >> 15, e = (b >> 10) & 31, m = b & 0x3FF;
        f[0] = (uint8_t)e; f[1] = (uint8_t)(m >> 5); f[2] = (uint8_t)(m & 31);
        *raw = (uint8_t)s;
    }
}

uint16_t orc_join(int dtype, const uint8_t f[3], uint8_t raw)
{
    if (dtype == ORC_BF16) {
        unsigned s = raw >> 7, m = raw & 0x7F, e = ((unsigned)f[0] << 4) | f[1];
        return (uint16_t)((s << 15) | (e << 7) | m);
    } else if (dtype == ORC_BF16_E8) {
        unsigned s = raw >> 7, m = raw & 0x7F;
        return (uint16_t)((s << 15) | ((unsigned)f[0] << 7) | m);
    } else {
        unsigned s = raw & 1, m = ((unsigned)f[1] << 5) | f[2];
        return (uint16_t)((s << 15) | ((unsigned)f[0] << 10) | m);
    }
}

/* counts[field][symbol] over the whole tensor (one codebook set per tensor). */
void orc_histogram(int dtype, const uint16_t *w, size_t n, uint64_t counts[3][ORC_MAXSYM])
{
    memset(counts, 0, 3 * ORC_MAXSYM * sizeof(uint64_t));
    int nf = orc_num_fields(dtype);
    for (size_t i = 0; i < n; ++i) {
        uint8_t f[3], raw;
        orc_split(dtype, w[i], f, &raw);
        for (int k = 0; k < nf; ++k) counts[k][f[k]]++;
    }
}

/* --------------------------------------------------------- Huffman lengths */

/* Classic Huffman: repeatedly merge the two smallest nodes; a symbol's length is
 * its depth.  Node order is (weight, id).  Returns the number of used symbols. */
int orc_huffman_lengths(const uint64_t *counts, int nsym, uint8_t *len)
{
    uint64_t wt[2 * ORC_MAXSYM]; int id[2 * ORC_MAXSYM], parent[2 * ORC_MAXSYM], alive[2 * ORC_MAXSYM];
    int nn = 0, used = 0;
    for (int s = 0; s < nsym; ++s) {
        len[s] = 0;
        if (counts[s] > 0) { wt[nn] = counts[s]; id[nn] = s; parent[nn] = -1; alive[nn] = 1; ++nn; ++used; }
    }
    if (used == 0) return 0;
    if (used == 1) { len[id[0]] = 1; return 1; }
    int created = 0, remaining = used;
    while (remaining > 1) {
        int a = -1, b = -1;
        for (int i = 0; i < nn; ++i) {             /* smallest (weight, id) */
            if (!alive[i]) continue;
            if (a < 0 || wt[i] < wt[a] || (wt[i] == wt[a] && id[i] < id[a])) a = i;
        }
        alive[a] = 0;
        for (int i = 0; i < nn; ++i) {             /* second smallest */
            if (!alive[i]) continue;
            if (b < 0 || wt[i] < wt[b] || (wt[i] == wt[b] && id[i] < id[b])) b = i;
        }
        alive[b] = 0;
        wt[nn] = wt[a] + wt[b]; id[nn] = 1000 + created++; parent[nn] = -1; alive[nn] = 1;
        parent[a] = nn; parent[b] = nn; ++nn; --remaining;
    }
    for (int i = 0; i < nn; ++i) {
        if (id[i] >= 1000) continue;
        int d = 0;
        for (int p = parent[i]; p >= 0; p = parent[p]) ++d;
        len[id[i]] = (uint8_t)d;
    }
    return used;
}

/* Optimal prefix code with every length <= cap, by package-merge: at each of
 * `cap` levels the leaf "coins" are merged with the pairs packaged on the level
 * below; the 2n-2 cheapest items of the top level are bought, and a symbol's
 * length is the number of bought items that contain it.
 * Returns used symbols, or -1 if 2^cap < used.                                */
typedef struct { uint64_t w; int is_pkg; uint8_t cnt[ORC_MAXSYM]; } orc_item;

static int orc_item_cmp(const void *pa, const void *pb)
{
    const orc_item *a = (const orc_item *)pa, *b = (const orc_item *)pb;
    if (a->w != b->w) return a->w < b->w ? -1 : 1;
    return a->is_pkg - b->is_pkg;                  /* at equal weight, leaves first */
}

int orc_limited_lengths(const uint64_t *counts, int nsym, int cap, uint8_t *len)
{
    int used = 0, sym[ORC_MAXSYM];
    for (int s = 0; s < nsym; ++s) { len[s] = 0; if (counts[s] > 0) sym[used++] = s; }
    if (used == 0) return 0;
    if (used == 1) { len[sym[0]] = 1; return 1; }
    if (cap < 1 || cap > 31 || (cap < 31 && (1 << cap) < used)) return -1;

    orc_item *cur = (orc_item *)malloc(sizeof(orc_item) * 4 * ORC_MAXSYM);
    orc_item *pkg = (orc_item *)malloc(sizeof(orc_item) * 2 * ORC_MAXSYM);
    int npkg = 0, ncur = 0;
    for (int level = cap; level >= 1; --level) {
        ncur = 0;
        for (int i = 0; i < used; ++i) {           /* one coin per symbol on this level */
            cur[ncur].w = counts[sym[i]]; cur[ncur].is_pkg = 0;
            memset(cur[ncur].cnt, 0, ORC_MAXSYM); cur[ncur].cnt[sym[i]] = 1; ++ncur;
        }
        for (int i = 0; i < npkg; ++i) cur[ncur++] = pkg[i];
        /* stable enough: qsort with a total order on (weight, kind); equal items are interchangeable in cost */
        qsort(cur, ncur, sizeof(orc_item), orc_item_cmp);
        if (level > 1) {
            npkg = 0;
            for (int i = 0; i + 1 < ncur; i += 2) {
                pkg[npkg].w = cur[i].w + cur[i + 1].w; pkg[npkg].is_pkg = 1;
                for (int s = 0; s < ORC_MAXSYM; ++s) pkg[npkg].cnt[s] = (uint8_t)(cur[i].cnt[s] + cur[i + 1].cnt[s]);
                ++npkg;
            }
        }
    }
    for (int i = 0; i < 2 * used - 2; ++i)
        for (int s = 0; s < nsym; ++s) len[s] = (uint8_t)(len[s] + cur[i].cnt[s]);
    free(cur); free(pkg);
    return used;
}

/* Sum over symbols of count * length. */
uint64_t orc_code_cost(const uint64_t *counts, const uint8_t *len, int nsym)
{
    uint64_t c = 0;
    for (int s = 0; s < nsym; ++s) c += counts[s] * (uint64_t)len[s];
    return c;
}

/* Code lengths for all coded fields of a tensor under a length budget.
 * budget == 0: unrestricted Huffman for every field.
 * FP16 and BF16 whole exponent: every field is limited to `budget` on its own.
 * BF16: the two exponent nibbles of one weight are decoded together, so the
 *       budget bounds the SUM of the two fields' maximum lengths: choose caps
 *       (c0, c1), c0 + c1 <= budget, minimising the total coded bits; ties go to
 *       the smaller c0.  If plain Huffman already fits, this is plain Huffman.
 * Returns 0, or -1 if the budget cannot hold the used symbols.                 */
int orc_build_lengths(int dtype, const uint64_t counts[3][ORC_MAXSYM], int budget,
                      uint8_t len[3][ORC_MAXSYM], int caps[3])
{
    int nf = orc_num_fields(dtype), ns = orc_field_symbols(dtype);
    memset(len, 0, 3 * ORC_MAXSYM);
    caps[0] = caps[1] = caps[2] = 0;
    if (budget == 0) {
        for (int k = 0; k < nf; ++k) if (orc_huffman_lengths(counts[k], ns, len[k]) == 0) return -1;
        return 0;
    }
    if (dtype != ORC_BF16) {
        for (int k = 0; k < nf; ++k) {
            if (orc_limited_lengths(counts[k], ns, budget, len[k]) <= 0) return -1;
            caps[k] = budget;
        }
        return 0;
    }
    int have = 0; uint64_t best = 0; uint8_t l0[ORC_MAXSYM] = {0}, l1[ORC_MAXSYM] = {0};
    for (int c0 = 1; c0 < budget; ++c0) {
        int c1 = budget - c0;
        if (orc_limited_lengths(counts[0], ns, c0, l0) <= 0) continue;
        if (orc_limited_lengths(counts[1], ns, c1, l1) <= 0) continue;
        uint64_t cost = orc_code_cost(counts[0], l0, ns) + orc_code_cost(counts[1], l1, ns);
        if (!have || cost < best) {
            have = 1; best = cost; caps[0] = c0; caps[1] = c1;
            memcpy(len[0], l0, ORC_MAXSYM); memcpy(len[1], l1, ORC_MAXSYM);
        }
    }
    return have ? 0 : -1;
}

/* Canonical codewords: symbols ordered by (length, symbol); the first gets 0,
 * each next one gets previous+1, shifted left when the length grows.  The
 * codeword's most significant bit is the first bit in the stream.             */
void orc_canonical_codes(const uint8_t *len, int nsym, uint32_t *code)
{
    uint32_t next = 0; int prev_len = 0, first = 1;
    for (int s = 0; s < nsym; ++s) code[s] = 0;
    for (int l = 1; l <= 31; ++l)
        for (int s = 0; s < nsym; ++s) {
            if (len[s] != l) continue;
            if (!first) next = (next + 1) << (l - prev_len);
            code[s] = next; prev_len = l; first = 0;
        }
}

/* ------------------------------------------------------- encode and decode */

/* Encode `n_seq` independent sequences of `seq_len` weights each (w is
 * [n_seq][seq_len]).  For every weight, in order, append code(f0) code(f1)
 * [code(f2)] to the sequence's bit list and the raw bits to raw[].  Bits are
 * stored one per byte (0/1) in `bits`; bit_off[i] .. bit_off[i+1] delimit
 * sequence i.  Pass bits == NULL to only count.  Returns total bits, or
 * (uint64_t)-1 if a weight uses a symbol without a codeword.                  */
uint64_t orc_encode_sequences(int dtype, const uint16_t *w, size_t n_seq, size_t seq_len,
                              const uint8_t len[3][ORC_MAXSYM], const uint32_t code[3][ORC_MAXSYM],
                              uint8_t *bits, uint64_t *bit_off, uint8_t *raw)
{
    int nf = orc_num_fields(dtype);
    uint64_t pos = 0;
    for (size_t q = 0; q < n_seq; ++q) {
        if (bit_off) bit_off[q] = pos;
        for (size_t i = 0; i < seq_len; ++i) {
            uint8_t f[3], r;
            orc_split(dtype, w[q * seq_len + i], f, &r);
            if (raw) raw[q * seq_len + i] = r;
            for (int k = 0; k < nf; ++k) {
                int l = len[k][f[k]];
                if (l == 0) return (uint64_t)-1;
                for (int b = l - 1; b >= 0; --b) {      /* most significant codeword bit first */
                    if (bits) bits[pos] = (uint8_t)((code[k][f[k]] >> b) & 1);
                    ++pos;
                }
            }
        }
    }
    if (bit_off) bit_off[n_seq] = pos;
    return pos;
}

/* One decoder step for one field: starting at bits[*pos], grow the candidate one
 * bit at a time and compare it with every stored codeword of that length (the
 * CAM lookup); on a match return the symbol and advance *pos by its length.   */
static int orc_decode_symbol(const uint8_t *bits, uint64_t nbits, uint64_t *pos,
                             const uint8_t *len, const uint32_t *code, int nsym)
{
    uint32_t cand = 0;
    for (int l = 1; l <= 31; ++l) {
        if (*pos + (uint64_t)l > nbits) return -1;
        cand = (cand << 1) | bits[*pos + l - 1];
        for (int s = 0; s < nsym; ++s)
            if (len[s] == l && code[s] == cand) { *pos += (uint64_t)l; return s; }
    }
    return -1;
}

/* Decode sequence by sequence: exactly seq_len weights from the bits between
 * bit_off[q] and bit_off[q+1]; bits_used[q] (optional) receives the number of
 * bits consumed.  Returns 0, or -(q+1) if sequence q does not decode.          */
int64_t orc_decode_sequences(int dtype, const uint8_t *bits, const uint64_t *bit_off, size_t n_seq, size_t seq_len,
                             const uint8_t len[3][ORC_MAXSYM], const uint32_t code[3][ORC_MAXSYM],
                             const uint8_t *raw, uint16_t *w_out, uint64_t *bits_used)
{
    int nf = orc_num_fields(dtype), ns = orc_field_symbols(dtype);
    for (size_t q = 0; q < n_seq; ++q) {
        uint64_t pos = bit_off[q], end = bit_off[q + 1];
        for (size_t i = 0; i < seq_len; ++i) {
            uint8_t f[3] = {0, 0, 0};
            for (int k = 0; k < nf; ++k) {
                int s = orc_decode_symbol(bits, end, &pos, len[k], code[k], ns);
                if (s < 0) return -(int64_t)(q + 1);
                f[k] = (uint8_t)s;
            }
            w_out[q * seq_len + i] = orc_join(dtype, f, raw[q * seq_len + i]);
        }
        if (bits_used) bits_used[q] = pos - bit_off[q];
    }
    return 0;
}

/* ------------------------------------------------------ values and products */

/* Exact value of a 16-bit pattern as a double (Section 2.1: (-1)^S 2^(E-B) (1.M),
 * with the IEEE conventions for E == 0 and E == all ones).                    */
double orc_value(int dtype, uint16_t b)
{
    int ebits = dtype == ORC_FP16 ? 5 : 8, mbits = dtype == ORC_FP16 ? 10 : 7;
    int bias = (1 << (ebits - 1)) - 1, emax = (1 << ebits) - 1;
    int s = b >> 15, e = (b >> mbits) & emax, m = b & ((1 << mbits) - 1);
    double sign = s ? -1.0 : 1.0, frac = (double)m / (double)(1 << mbits);
    if (e == emax) return m ? NAN : sign * INFINITY;
    if (e == 0) return sign * ldexp(frac, 1 - bias);
    return sign * ldexp(1.0 + frac, e - bias);
}

/* y[j][r] = sum_k value(W[r][k]) * value(x[j][k]) in k order, double precision;
 * d[j][r] = sum_k |value(W[r][k]) * value(x[j][k])| (the error-bound scale).   */
void orc_matmul(int dtype, const uint16_t *W, size_t rows, size_t cols,
                const uint16_t *x, size_t batch, double *y, double *d)
{
    double *xv = (double *)malloc(sizeof(double) * cols);
    for (size_t j = 0; j < batch; ++j) {
        for (size_t k = 0; k < cols; ++k) xv[k] = orc_value(dtype, x[j * cols + k]);
        for (size_t r = 0; r < rows; ++r) {
            double acc = 0.0, mag = 0.0;
            for (size_t k = 0; k < cols; ++k) {
                double p = orc_value(dtype, W[r * cols + k]) * xv[k];
                acc += p; mag += fabs(p);
            }
            y[j * rows + r] = acc; if (d) d[j * rows + r] = mag;
        }
    }
    free(xv);
}
