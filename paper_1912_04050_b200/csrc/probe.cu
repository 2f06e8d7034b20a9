// Measurement aid, not a step of the routing method: independent random 4-byte
// gathers from a caller's array.  The ruler walks of the loop labelling are
// chains of random accesses, so the rate this kernel reaches on the same GPU,
// on an array of the same size, is the ceiling their access rate is compared
// with.  The caller times the launch with CUDA events on its stream.
#include "common.cuh"

namespace benes {
namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbePerThread = 8;          // all of a thread's gathers are in flight together

__device__ __forceinline__ uint32_t probe_hash(uint32_t x) {
    x ^= x >> 16; x *= 0x7FEB352Du;
    x ^= x >> 15; x *= 0x846CA68Bu;
    x ^= x >> 16;
    return x;
}

__global__ void __launch_bounds__(kProbeThreads)
k_probe_gather(const uint32_t *__restrict__ table, uint32_t word_mask, size_t gathers,
               uint32_t *__restrict__ sink) {
    const size_t first = (size_t(blockIdx.x) * kProbeThreads + threadIdx.x) * kProbePerThread;
    uint32_t v[kProbePerThread];
#pragma unroll
    for (int i = 0; i < kProbePerThread; ++i)
        v[i] = first + i < gathers ? __ldg(table + (probe_hash(uint32_t(first) + uint32_t(i)) & word_mask)) : 0u;
    uint32_t x = 0;
#pragma unroll
    for (int i = 0; i < kProbePerThread; ++i) x ^= v[i];
    // keeps the loads alive: the store depends on what was read (and happens about once in 2^32 threads)
    if (x == 0x9E3779B9u) *sink = x;
}

}  // namespace
}  // namespace benes

using namespace benes;

extern "C" int benes_probe_gather(const uint32_t *table, int log2_words, size_t gathers, uint32_t *sink,
                                  benes_stream_t stream) {
    if (!table || !sink || log2_words < 1 || log2_words > 31 || gathers == 0 || gathers > (size_t(1) << 32))
        return BENES_ERR_BADARG;
    const size_t threads = (gathers + kProbePerThread - 1) / kProbePerThread;
    const unsigned grid = unsigned((threads + kProbeThreads - 1) / kProbeThreads);
    k_probe_gather<<<grid, kProbeThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        table, (1u << log2_words) - 1u, gathers, sink);
    return launch_status();
}

extern "C" int benes_shard_batch(int batch, int world, int rank, int *first, int *count) {
    if (batch < 1 || world < 1 || rank < 0 || rank >= world || !first || !count) return BENES_ERR_BADARG;
    // contiguous slices whose sizes differ by at most one; the first batch % world ranks take the larger ones
    const int q = batch / world, r = batch % world;
    *first = rank * q + (rank < r ? rank : r);
    *count = q + (rank < r ? 1 : 0);
    return BENES_OK;
}
