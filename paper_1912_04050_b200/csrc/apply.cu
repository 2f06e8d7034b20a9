// Payload apply: one streaming kernel per stage.  A thread owns one switch:
// it reads the switch's two inputs, swaps them if the switch is crossed and
// writes them where the wiring to the next stage puts them.
//   input side of level l  : reads the adjacent pair (2s, 2s+1) of its block,
//                            writes position s of the upper and lower half;
//   middle                 : adjacent pair in, adjacent pair out;
//   output side of level l : reads position t of the upper and lower half,
//                            writes the adjacent pair (2t, 2t+1).
#include "common.cuh"

namespace benes {
namespace {

constexpr int kThreads = 256;

template <typename E> struct Pair;
template <> struct Pair<uint32_t> { using type = uint2; };
template <> struct Pair<unsigned long long> { using type = ulonglong2; };

// side: 0 = input side (incl. middle when log2m == 1), 1 = output side
template <typename E, int SIDE>
__global__ void __launch_bounds__(kThreads)
k_apply_stage(const uint32_t *__restrict__ bits, const E *__restrict__ x, E *__restrict__ y,
              size_t switches, int log2m, int stage, int log2n) {
    using P2 = typename Pair<E>::type;
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    const size_t half_n = size_t(1) << (log2n - 1);
    const size_t stage_w = log2n >= 6 ? (size_t(1) << (log2n - 6)) : 1;
    const size_t per_perm = size_t(2 * log2n - 1) * stage_w;
    const size_t H = size_t(1) << (log2m - 1);
    for (size_t t = size_t(blockIdx.x) * blockDim.x + threadIdx.x; t < switches; t += stride) {
        size_t perm = t >> (log2n - 1);
        size_t tl = t & (half_n - 1);
        uint32_t cross = (__ldg(bits + perm * per_perm + size_t(stage) * stage_w + (tl >> 5)) >> (tl & 31)) & 1u;
        size_t base = (2 * t) & ~((size_t(2) << (log2m - 1)) - 1);
        size_t s = t - base / 2;
        if (SIDE == 0) {
            P2 v = reinterpret_cast<const P2 *>(x)[t];
            E a = cross ? v.y : v.x, b = cross ? v.x : v.y;
            if (log2m == 1) {
                v.x = a; v.y = b;
                reinterpret_cast<P2 *>(y)[t] = v;
            } else {
                y[base + s] = a;
                y[base + H + s] = b;
            }
        } else {
            E u = x[base + s], l = x[base + H + s];
            P2 v;
            v.x = cross ? l : u;
            v.y = cross ? u : l;
            reinterpret_cast<P2 *>(y)[t] = v;
        }
    }
}

template <typename E>
int launch_typed(const uint32_t *bits, const void *x, void *y, int stage, int log2n, size_t batch,
                 cudaStream_t s) {
    size_t switches = batch << (log2n - 1);
    int level = stage <= log2n - 1 ? stage : 2 * log2n - 2 - stage;
    int log2m = log2n - level;
    size_t blocks = (switches + kThreads - 1) / kThreads;
    size_t cap = size_t(sm_count()) * 16;
    int grid = int(blocks < cap ? blocks : cap);
    if (stage <= log2n - 1)
        k_apply_stage<E, 0><<<grid, kThreads, 0, s>>>(bits, static_cast<const E *>(x),
                                                      static_cast<E *>(y), switches, log2m, stage, log2n);
    else
        k_apply_stage<E, 1><<<grid, kThreads, 0, s>>>(bits, static_cast<const E *>(x),
                                                      static_cast<E *>(y), switches, log2m, stage, log2n);
    return launch_status();
}

}  // namespace

int launch_apply_stage(const uint32_t *bits, const void *x, void *y, int elem_bytes, int stage,
                       int log2n, size_t batch, cudaStream_t s) {
    if (elem_bytes == 4) return launch_typed<uint32_t>(bits, x, y, stage, log2n, batch, s);
    if (elem_bytes == 8) return launch_typed<unsigned long long>(bits, x, y, stage, log2n, batch, s);
    return BENES_ERR_BADARG;
}

}  // namespace benes
