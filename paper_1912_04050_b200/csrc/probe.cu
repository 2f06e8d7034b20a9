// Measurement aid, not a step of the routing method: random accesses to a
// caller's array, every one to a different pseudo-randomly placed record.  The
// ruler walks of the loop labelling are chains of such accesses, so the rates and
// the DRAM traffic these kernels reach on the same GPU, on an array of the same
// size, are what the walks are compared with.  The caller times the launch with
// CUDA events on its stream (and counts DRAM bytes with a profiler).
#include "common.cuh"

namespace benes {
namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbePer = 2;                 // a thread's accesses are in flight together (more would overflow the L2 between a load and its claim)

// i -> a record index: an odd multiplier permutes [0, 2^32), the mask keeps the
// low bits, so ops <= records touch distinct records
__device__ __forceinline__ uint32_t probe_index(uint32_t i, uint32_t mask) {
    return (i * 0x9E3779B1u + 12345u) & mask;
}

// MODE 0: 4-byte load of a record's first word; 1: 16-byte load; 2: 16-byte load, then
// compare-and-swap on the record's third word (the claim of a wide switch record);
// 3: 64-bit atomic AND on a record's first half (the claim of a packed record);
// 4: 4-byte store to the record's third word.  Records are `stride` bytes apart.
template <int MODE>
__global__ void __launch_bounds__(kProbeThreads)
k_probe(unsigned char *__restrict__ table, uint32_t mask, uint32_t stride, size_t ops, uint32_t *__restrict__ sink) {
    const size_t first = (size_t(blockIdx.x) * kProbeThreads + threadIdx.x) * kProbePer;
    uint32_t x = 0;
    uint4 v[kProbePer];
#pragma unroll
    for (int k = 0; k < kProbePer; ++k) {
        v[k] = make_uint4(0, 0, 0, 0);
        if (first + k >= ops) continue;
        unsigned char *rec = table + size_t(probe_index(uint32_t(first) + k, mask)) * stride;
        if (MODE == 0) v[k].x = __ldcg(reinterpret_cast<const uint32_t *>(rec));
        if (MODE == 1 || MODE == 2) v[k] = __ldcg(reinterpret_cast<const uint4 *>(rec));
        if (MODE == 3) {
            const unsigned long long old = atomicAnd(reinterpret_cast<unsigned long long *>(rec),
                                                     ((unsigned long long)(uint32_t(first) + k) << 40) | ((1ull << 40) - 1ull));
            v[k].x = uint32_t(old) ^ uint32_t(old >> 32);
        }
        if (MODE == 4) reinterpret_cast<uint32_t *>(rec)[2] = uint32_t(first) + k;
    }
    if (MODE == 2) {
#pragma unroll
        for (int k = 0; k < kProbePer; ++k) {
            if (first + k >= ops) continue;
            unsigned char *rec = table + size_t(probe_index(uint32_t(first) + k, mask)) * stride;
            v[k].z = atomicCAS(reinterpret_cast<uint32_t *>(rec) + 2, v[k].z, uint32_t(first) + k);
        }
    }
#pragma unroll
    for (int k = 0; k < kProbePer; ++k) x ^= v[k].x ^ v[k].y ^ v[k].z;
    // keeps the accesses alive: the store depends on what was read (about once in 2^32 threads)
    if (MODE != 4 && x == 0x9E3779B9u) *sink = x;
}

}  // namespace
}  // namespace benes

using namespace benes;

extern "C" int benes_probe_random_access(void *table, int log2_records, int record_bytes, int mode, size_t ops,
                                         uint32_t *sink, benes_stream_t stream) {
    if (!table || !sink || log2_records < 1 || log2_records > 31 || ops == 0 || ops > (size_t(1) << 32))
        return BENES_ERR_BADARG;
    if (mode < 0 || mode > 4) return BENES_ERR_BADARG;
    // a record must hold what the mode touches, aligned to it
    const int need = mode == 0 ? 4 : (mode == 3 ? 8 : 16);
    if (record_bytes < need || record_bytes % need || record_bytes > 4096) return BENES_ERR_BADARG;
    const size_t threads = (ops + kProbePer - 1) / kProbePer;
    const unsigned grid = unsigned((threads + kProbeThreads - 1) / kProbeThreads);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    unsigned char *t = static_cast<unsigned char *>(table);
    const uint32_t mask = (1u << log2_records) - 1u, stride = uint32_t(record_bytes);
    switch (mode) {
        case 0: k_probe<0><<<grid, kProbeThreads, 0, s>>>(t, mask, stride, ops, sink); break;
        case 1: k_probe<1><<<grid, kProbeThreads, 0, s>>>(t, mask, stride, ops, sink); break;
        case 2: k_probe<2><<<grid, kProbeThreads, 0, s>>>(t, mask, stride, ops, sink); break;
        case 3: k_probe<3><<<grid, kProbeThreads, 0, s>>>(t, mask, stride, ops, sink); break;
        default: k_probe<4><<<grid, kProbeThreads, 0, s>>>(t, mask, stride, ops, sink); break;
    }
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
