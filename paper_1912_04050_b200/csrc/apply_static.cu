// benes_apply_static: payload apply for callers that must not allocate.
//
// The per-stage apply ping-pongs between `out` and one scratch buffer.  The
// regular entry point takes that buffer from the library workspace, which the
// library cudaMallocs the first time it is too small.  Some callers cannot
// live with that: a service whose device memory has been handed over in full
// to another allocator (a late cudaMalloc then simply fails), or a
// latency-critical loop that cannot afford the device-wide stall a cudaMalloc
// or cudaFree causes.  For them the scratch lives in the fixed array below,
// which is part of the library image: every GPU that loads the library holds
// these 4 MiB until the process exits.
#include "common.cuh"

#include <mutex>

namespace benes {
namespace {

// Scratch for the odd-numbered intermediate stages.  Nothing in it has to
// start at zero: every stage writes all batch*N elements before the next
// stage reads them.  All calls share it, so it always holds the leftovers of
// the last call.
static __device__ __align__(256) unsigned char g_static_scratch[BENES_STATIC_SCRATCH_BYTES];

constexpr int kMaxDev = 64;
void *g_scratch_addr[kMaxDev] = {};   // device address of the array, per device
std::mutex g_static_mu;

// `g_static_scratch` in host code is only a handle for the runtime, not a
// device address; the address each device gave the array has to be asked for,
// once per device, while that device is current.
int scratch_for_current_device(void **out) {
    int dev = 0;
    BENES_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDev) return BENES_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return BENES_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return BENES_OK;
}

}  // namespace
}  // namespace benes

using namespace benes;

extern "C" int benes_apply_static(const uint32_t *switch_bits, const void *in, void *out,
                                  int elem_bytes, int log2n, int batch, benes_stream_t stream) {
    if (!switch_bits || !in || !out || in == out) return BENES_ERR_BADARG;
    if (log2n < 1 || log2n > BENES_MAX_LOG2N || batch < 1) return BENES_ERR_BADARG;
    if (elem_bytes != 4 && elem_bytes != 8) return BENES_ERR_BADARG;
    // size check in a form that cannot overflow
    const size_t cap_elems = size_t(BENES_STATIC_SCRATCH_BYTES) / size_t(elem_bytes);
    if (log2n > 40 || (size_t(1) << log2n) > cap_elems || size_t(batch) > (cap_elems >> log2n))
        return BENES_ERR_TOO_LARGE;
    void *scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc) return rc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int stages = 2 * log2n - 1;
    const void *src = in;
    for (int st = 0; st < stages; ++st) {
        // the last stage must land in `out`, so stages alternate backwards from there
        void *dst = ((stages - 1 - st) % 2 == 0) ? out : scratch;
        rc = launch_apply_stage(switch_bits, src, dst, elem_bytes, st, log2n, size_t(batch), s);
        if (rc) return rc;
        src = dst;
    }
    return BENES_OK;
}
