// Bit-field split explorer (Section 3.1, entropy table): how many bits per parameter would each way of cutting a
// 16-bit weight into separately coded fields cost?  The device part counts, for every field of a split, how often
// each of its values occurs in a weight tensor that already sits in device memory; the host part turns counts into
// entropies and Huffman code costs.
//
// Counting is one streaming pass over the weights (2 bytes per weight from HBM).  Every CTA keeps private counters in
// shared memory and adds them to the global 64-bit counters at the end.  LLM weights are very skewed (a handful of
// exponent values cover almost all weights), so a narrow field's counters are replicated 32 times, one copy per
// lane: the lanes of a warp never touch the same address or the same bank, whatever the data.  Wider fields get
// fewer copies; a field whose counters do not fit is counted in several launches, each owning a range of values.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <vector>

#include "internal.h"

namespace huffllm {

constexpr uint32_t kHistThreads = 1024;
constexpr uint32_t kHistBudgetWords = 48u * 1024u;   // shared-memory counters of one launch (192 KB)
constexpr uint32_t kFieldWords = 8u * 1024u;         // target size of one field's counters, copies included

struct FieldPlan {
    uint32_t shift, mask;        // value of the field = (word >> shift) & mask
    uint32_t bin_lo, bin_n;      // values counted by this launch: bin_lo .. bin_lo + bin_n - 1
    uint32_t smem_off;           // first counter, in 32-bit words
    uint32_t rep_log2;           // log2 of the copies per value
    uint32_t out_off;            // index of the field's value 0 in the output counters
    uint32_t ranged;             // 1 if the launch covers only a part of the field's values
};
struct HistArgs {
    const uint16_t *w;
    uint64_t n;
    unsigned long long *counts;
    uint32_t n_fields, smem_words;
    FieldPlan f[HUFFLLM_MAX_FIELDS];
};

__device__ __forceinline__ void red_shared_inc(uint32_t addr) {
    asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(addr) : "memory");
}

__global__ void __launch_bounds__(kHistThreads) split_histogram_kernel(const __grid_constant__ HistArgs A) {
    extern __shared__ __align__(16) uint32_t hist[];
    const uint32_t tid = threadIdx.x, lane = tid & 31;
    for (uint32_t i = tid; i < A.smem_words; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    const uint32_t base = (uint32_t)__cvta_generic_to_shared(hist);

    // 16-byte vectors of eight weights, dealt to the grid's threads in turn; the last n % 8 weights go to one thread
    const uint64_t n_vec = A.n / 8, stride = (uint64_t)gridDim.x * blockDim.x;
    const uint4 *src = (const uint4 *)A.w;
    auto count_word = [&](uint32_t word, uint32_t n_in_word) {     // one or two weights of a 32-bit word
#pragma unroll 1
        for (uint32_t fi = 0; fi < A.n_fields; ++fi) {
            const FieldPlan &f = A.f[fi];
            const uint32_t lane_off = base + ((f.smem_off + (lane & ((1u << f.rep_log2) - 1u))) << 2);
            const uint32_t step = 4u << f.rep_log2;
#pragma unroll
            for (uint32_t j = 0; j < 2; ++j) {
                if (j >= n_in_word) break;
                uint32_t b = ((word >> (f.shift + 16 * j)) & f.mask) - f.bin_lo;
                if (!f.ranged || b < f.bin_n) red_shared_inc(lane_off + b * step);
            }
        }
    };
    for (uint64_t v = (uint64_t)blockIdx.x * blockDim.x + tid; v < n_vec; v += stride) {
        const uint4 q = __ldg(src + v);
        const uint32_t word[4] = {q.x, q.y, q.z, q.w};
#pragma unroll 1
        for (uint32_t fi = 0; fi < A.n_fields; ++fi) {
            const FieldPlan &f = A.f[fi];
            const uint32_t lane_off = base + ((f.smem_off + (lane & ((1u << f.rep_log2) - 1u))) << 2);
            const uint32_t step = 4u << f.rep_log2, sh = f.shift, mask = f.mask, lo = f.bin_lo, nb = f.bin_n;
            if (!f.ranged) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    red_shared_inc(lane_off + ((word[i] >> sh) & mask) * step);
                    red_shared_inc(lane_off + ((word[i] >> (sh + 16)) & mask) * step);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t b0 = ((word[i] >> sh) & mask) - lo, b1 = ((word[i] >> (sh + 16)) & mask) - lo;
                    if (b0 < nb) red_shared_inc(lane_off + b0 * step);
                    if (b1 < nb) red_shared_inc(lane_off + b1 * step);
                }
            }
        }
    }
    if (blockIdx.x == 0 && tid == 0)
        for (uint64_t i = n_vec * 8; i < A.n; ++i) count_word(A.w[i], 1);
    __syncthreads();

    // add the CTA's counters to the global ones (copies of a value summed first; zero sums are skipped)
    for (uint32_t fi = 0; fi < A.n_fields; ++fi) {
        const FieldPlan &f = A.f[fi];
        const uint32_t reps = 1u << f.rep_log2;
        for (uint32_t b = tid; b < f.bin_n; b += blockDim.x) {
            unsigned long long s = 0;
            for (uint32_t r = 0; r < reps; ++r) s += hist[f.smem_off + (b << f.rep_log2) + ((r + tid) & (reps - 1u))];
            if (s) atomicAdd(A.counts + f.out_off + f.bin_lo + b, s);
        }
    }
}

static huffllm_status check_widths(const uint8_t *widths, uint32_t n_fields, size_t *total_bins) {
    if (!widths || n_fields == 0 || n_fields > HUFFLLM_MAX_FIELDS) return fail(HUFFLLM_ERR_INVALID_ARG, "a split has 1..%d fields", HUFFLLM_MAX_FIELDS);
    uint32_t sum = 0;
    size_t bins = 0;
    for (uint32_t i = 0; i < n_fields; ++i) {
        if (widths[i] < 1 || widths[i] > 16) return fail(HUFFLLM_ERR_INVALID_ARG, "field %u has width %u", i, (unsigned)widths[i]);
        sum += widths[i];
        bins += (size_t)1 << widths[i];
    }
    if (sum != 16) return fail(HUFFLLM_ERR_INVALID_ARG, "the field widths add up to %u, not 16", sum);
    if (total_bins) *total_bins = bins;
    return HUFFLLM_OK;
}

}  // namespace huffllm

using namespace huffllm;

extern "C" huffllm_status huffllm_split_counts_size(const uint8_t *widths, uint32_t n_fields, size_t *n_counts) {
    clear_error();
    if (!n_counts) return fail(HUFFLLM_ERR_INVALID_ARG, "null output");
    return check_widths(widths, n_fields, n_counts);
}

extern "C" huffllm_status huffllm_split_histogram(const uint16_t *w_dev, uint64_t n_weights, const uint8_t *widths,
                                                  uint32_t n_fields, uint64_t *counts_dev, huffllm_stream stream) {
    clear_error();
    size_t bins = 0;
    huffllm_status st = check_widths(widths, n_fields, &bins);
    if (st != HUFFLLM_OK) return st;
    if (!w_dev || !counts_dev) return fail(HUFFLLM_ERR_INVALID_ARG, "null device pointer");
    if (((uintptr_t)w_dev & 15u) || ((uintptr_t)counts_dev & 7u)) return fail(HUFFLLM_ERR_INVALID_ARG, "weights must be 16-byte aligned, counters 8-byte aligned");
    if (n_weights >> 38) return fail(HUFFLLM_ERR_UNSUPPORTED, "more than 2^38 weights in one call");   // a CTA's 32-bit counters cannot overflow below that
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemsetAsync(counts_dev, 0, bins * sizeof(uint64_t), s);
    if (e != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    if (n_weights == 0) return HUFFLLM_OK;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess || (e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
        return fail(HUFFLLM_ERR_CUDA, "device query: %s", cudaGetErrorString(e));

    // the pieces to count: a field, or a range of values of a wide field, each with its counters' size
    std::vector<FieldPlan> pieces;
    uint32_t hi = 16, out_off = 0;
    for (uint32_t i = 0; i < n_fields; ++i) {
        const uint32_t wd = widths[i], n_bins = 1u << wd;
        FieldPlan f = {};
        f.shift = hi - wd;
        f.mask = n_bins - 1u;
        f.out_off = out_off;
        while (f.rep_log2 < 5u && (n_bins << (f.rep_log2 + 1u)) <= kFieldWords) ++f.rep_log2;
        const uint32_t per_piece = std::min(n_bins, kHistBudgetWords / 2u >= n_bins ? n_bins : 32u * 1024u);
        for (uint32_t lo = 0; lo < n_bins; lo += per_piece) {
            f.bin_lo = lo;
            f.bin_n = per_piece;
            f.ranged = per_piece < n_bins ? 1u : 0u;
            pieces.push_back(f);
        }
        hi -= wd;
        out_off += n_bins;
    }
    // launches: pieces in order, as many as fit the shared-memory budget
    size_t p = 0;
    while (p < pieces.size()) {
        HistArgs A = {};
        A.w = w_dev;
        A.n = n_weights;
        A.counts = (unsigned long long *)counts_dev;
        uint32_t words = 0;
        while (p < pieces.size() && A.n_fields < HUFFLLM_MAX_FIELDS) {
            FieldPlan f = pieces[p];
            const uint32_t need = f.bin_n << f.rep_log2;
            if (A.n_fields && words + need > kHistBudgetWords) break;
            f.smem_off = words;
            words += need;
            A.f[A.n_fields++] = f;
            ++p;
        }
        A.smem_words = words;
        const size_t smem = (size_t)words * 4u;
        if ((e = cudaFuncSetAttribute(split_histogram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kHistBudgetWords * 4u))) != cudaSuccess)
            return fail(HUFFLLM_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        const uint64_t n_vec = n_weights / 8;
        uint32_t grid = (uint32_t)sms * (smem <= 100u * 1024u ? 2u : 1u);
        grid = (uint32_t)std::max<uint64_t>(1, std::min<uint64_t>(grid, (n_vec + kHistThreads - 1) / kHistThreads));
        split_histogram_kernel<<<grid, kHistThreads, smem, s>>>(A);
        if ((e = cudaGetLastError()) != cudaSuccess) return fail(HUFFLLM_ERR_CUDA, "split_histogram_kernel: %s", cudaGetErrorString(e));
    }
    return HUFFLLM_OK;
}

extern "C" huffllm_status huffllm_split_entropy(const uint64_t *counts_host, const uint8_t *widths, uint32_t n_fields,
                                                double *entropy_bits, double *huffman_bits) {
    clear_error();
    huffllm_status st = check_widths(widths, n_fields, nullptr);
    if (st != HUFFLLM_OK) return st;
    if (!counts_host || !entropy_bits) return fail(HUFFLLM_ERR_INVALID_ARG, "null pointer");
    const uint64_t *c = counts_host;
    for (uint32_t i = 0; i < n_fields; ++i) {
        const size_t n_bins = (size_t)1 << widths[i];
        long double total = 0;
        for (size_t b = 0; b < n_bins; ++b) total += (long double)c[b];
        double H = 0;
        if (total > 0)
            for (size_t b = 0; b < n_bins; ++b)
                if (c[b]) {
                    const double pr = (double)((long double)c[b] / total);
                    H -= pr * std::log2(pr);
                }
        entropy_bits[i] = H;
        if (huffman_bits) {
            // cost of a Huffman code = sum of the weights of the internal nodes of its tree (two-queue merge of the
            // sorted counts); a field with a single value in use is given the 1-bit code the blob format gives it
            std::vector<uint64_t> leaf;
            for (size_t b = 0; b < n_bins; ++b)
                if (c[b]) leaf.push_back(c[b]);
            std::sort(leaf.begin(), leaf.end());
            double bits = 0;
            if (leaf.size() == 1) {
                bits = 1.0;
            } else if (leaf.size() > 1) {
                std::vector<uint64_t> node;
                node.reserve(leaf.size());
                size_t li = 0, ni = 0;
                long double cost = 0;
                auto take = [&]() -> uint64_t {
                    if (li < leaf.size() && (ni >= node.size() || leaf[li] <= node[ni])) return leaf[li++];
                    return node[ni++];
                };
                for (size_t m = 0; m + 1 < leaf.size(); ++m) {
                    const uint64_t a = take(), b2 = take();
                    node.push_back(a + b2);
                    cost += (long double)(a + b2);
                }
                bits = (double)(cost / total);
            }
            huffman_bits[i] = bits;
        }
        c += n_bins;
    }
    return HUFFLLM_OK;
}
