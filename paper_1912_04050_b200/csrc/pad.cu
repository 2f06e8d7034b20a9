// Sizes that are not a power of two: a permutation of [0, n_elems) is extended
// to N = 2^log2n by fixed points (pi[j] = j for j >= n_elems), which leaves
// the routing of the first n_elems positions unchanged; payloads are copied
// into and out of rows of N elements.
#include "common.cuh"

namespace benes {
namespace {

constexpr int kThreads = 256;

inline unsigned grid_for(size_t items) {
    size_t blocks = (items + kThreads - 1) / kThreads;
    size_t cap = size_t(sm_count()) * 16;
    return unsigned(blocks < cap ? (blocks ? blocks : 1) : cap);
}

// dst[b][j] = src[b][j] for j < n_elems, j for n_elems <= j < N
__global__ void __launch_bounds__(kThreads)
k_pad_perm(const uint32_t *__restrict__ src, uint32_t *__restrict__ dst, size_t n_elems, int log2n,
           size_t total) {
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    const size_t nmask = (size_t(1) << log2n) - 1;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const size_t b = i >> log2n, j = i & nmask;
        dst[i] = j < n_elems ? src[b * n_elems + j] : uint32_t(j);
    }
}

// rows of n_elems elements <-> rows of N elements (the tail of a padded row is zero)
template <typename E, bool PAD>
__global__ void __launch_bounds__(kThreads)
k_pad_rows(const E *__restrict__ src, E *__restrict__ dst, size_t n_elems, int log2n, size_t total) {
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    const size_t nmask = (size_t(1) << log2n) - 1;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const size_t b = i >> log2n, j = i & nmask;
        if (PAD) dst[i] = j < n_elems ? src[b * n_elems + j] : E(0);
        else if (j < n_elems) dst[b * n_elems + j] = src[i];
    }
}

}  // namespace

int launch_pad_perm(const uint32_t *src, uint32_t *dst, size_t n_elems, int log2n, size_t batch,
                    cudaStream_t s) {
    const size_t total = batch << log2n;
    k_pad_perm<<<grid_for(total), kThreads, 0, s>>>(src, dst, n_elems, log2n, total);
    return launch_status();
}

int launch_pad_rows(const void *src, void *dst, int elem_bytes, bool pad, size_t n_elems, int log2n,
                    size_t batch, cudaStream_t s) {
    const size_t total = batch << log2n;
    const unsigned grid = grid_for(total);
    if (elem_bytes == 4) {
        if (pad) k_pad_rows<uint32_t, true><<<grid, kThreads, 0, s>>>(
            static_cast<const uint32_t *>(src), static_cast<uint32_t *>(dst), n_elems, log2n, total);
        else k_pad_rows<uint32_t, false><<<grid, kThreads, 0, s>>>(
            static_cast<const uint32_t *>(src), static_cast<uint32_t *>(dst), n_elems, log2n, total);
    } else if (elem_bytes == 8) {
        if (pad) k_pad_rows<unsigned long long, true><<<grid, kThreads, 0, s>>>(
            static_cast<const unsigned long long *>(src), static_cast<unsigned long long *>(dst), n_elems,
            log2n, total);
        else k_pad_rows<unsigned long long, false><<<grid, kThreads, 0, s>>>(
            static_cast<const unsigned long long *>(src), static_cast<unsigned long long *>(dst), n_elems,
            log2n, total);
    } else {
        return BENES_ERR_BADARG;
    }
    return launch_status();
}

}  // namespace benes

// ---- in-place ("butterfly") form of the switch settings ------------------------
//
// The same network drawn without wires between stages: data stays in place,
// stage row r pairs positions u and u | 2^i that differ in bit i (i = r for the
// n rows up to the middle, i = 2n-2-r after it) and a set bit swaps them.
// Position u then holds, in its low bits, the outputs the element took at the
// earlier stages, so the switch of the recursive layout that acts on the pair is
//     (low i bits of u, reversed) << (n-1-i)  +  (u >> (i+1)).
// Pair p of row r (u with bit i removed) is bit p of the row, same packing.
namespace benes {
namespace {

__global__ void __launch_bounds__(256)
k_export_butterfly(const uint32_t *__restrict__ bits, uint32_t *__restrict__ out, int n, size_t rows,
                   uint32_t words_per_row) {
    const uint32_t half = 1u << (n - 1);                       // switches per row
    const size_t lanes_per_row = size_t(words_per_row) * 32;
    const size_t total = rows * lanes_per_row;
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t idx = size_t(blockIdx.x) * blockDim.x + threadIdx.x; idx < total; idx += stride) {
        const size_t row = idx / lanes_per_row;                // permutation * (2n-1) + stage row
        const uint32_t p = uint32_t(idx - row * lanes_per_row);
        const int r = int(row % size_t(2 * n - 1));
        const int i = r <= n - 1 ? r : 2 * n - 2 - r;
        uint32_t bit = 0;
        if (p < half) {
            const uint32_t lowmask = (1u << i) - 1u;
            const uint32_t low = p & lowmask, high = p >> i;   // u = high << (i+1) | low
            const uint32_t rev = i ? (__brev(low) >> (32 - i)) : 0u;
            const uint32_t sw = (rev << (n - 1 - i)) + high;
            bit = (__ldg(bits + row * words_per_row + (sw >> 5)) >> (sw & 31u)) & 1u;
        }
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, bit);
        if ((threadIdx.x & 31) == 0) out[row * words_per_row + (p >> 5)] = word;
    }
}

}  // namespace

int launch_export_butterfly(const uint32_t *bits, uint32_t *out, int log2n, size_t batch, cudaStream_t s) {
    const uint32_t words = log2n >= 6 ? (1u << (log2n - 6)) : 1u;
    const size_t rows = batch * size_t(2 * log2n - 1);
    const size_t total = rows * words * 32;
    size_t blocks = (total + 255) / 256;
    if (blocks > size_t(sm_count()) * 16) blocks = size_t(sm_count()) * 16;
    k_export_butterfly<<<unsigned(blocks), 256, 0, s>>>(bits, out, log2n, rows, words);
    return launch_status();
}

}  // namespace benes
