// Work-efficient loop labelling for the HBM levels: ruler sampling.
//
// Pointer jumping over all outputs costs O(M log M) random accesses per level.
// Here only a sample of the outputs (the "rulers") is labelled by pointer
// jumping; everything else is reached by one sequential walk per ruler:
//
//   1. Switches are cut into groups of k = 2^kappa consecutive switches; a hash
//      of the group number picks one RULER switch per group.  Both outputs of
//      a ruler switch are ruler outputs; ruler output rho = 2*group + (j & 1).
//   2. k_walk: one thread per ruler output follows the successor
//      g(j) = base + Q[base + (P[j^1] ^ 1)] until it meets the next ruler
//      output.  It records (next ruler, smallest index seen) as one 64-bit
//      word of the contracted list and stamps its id on every even output it
//      passes ("owner" of the switch).  Every output lies on exactly one such
//      segment, so the walks cost O(M) in total.
//   3. The contracted list (T/k words, cache resident) is labelled by the
//      ordinary in-place pointer-jumping pass: afterwards a ruler's word holds
//      the minimum of its whole g-cycle.
//   4. k_colour: colour of output 2t = parity of the cycle minimum of its
//      owner.  A switch nobody stamped lies on a loop without ruler; such
//      loops are short (probability (1-1/k)^length) and the thread walks the
//      cycle itself.
//
// Both walks give up after `cap` hops and raise a per-level flag; the flag
// gates the full pointer-jumping kernels of route_levels.cu, which then
// relabel the level.  So the result never depends on the sampling.
#include "common.cuh"

namespace benes {
namespace {

constexpr int kThreads = 256;
constexpr int kSMs = 148;
constexpr uint32_t kUnowned = 0xFFFFFFFFu;

__device__ __forceinline__ uint32_t ruler_slot(uint32_t group, uint32_t salt, uint32_t kmask) {
    uint32_t h = group * 0x9E3779B1u + salt;
    h ^= h >> 15;
    h *= 0x85EBCA6Bu;
    h ^= h >> 13;
    return h & kmask;
}

__device__ __forceinline__ unsigned long long make_word(uint32_t nxt, uint32_t mn) {
    return (static_cast<unsigned long long>(mn) << 32) | nxt;
}

// Step 2.  rulers = T / k threads, launched in index order so that the blocks
// being walked at any moment are neighbours in memory.
__global__ void __launch_bounds__(kThreads)
k_walk(const uint32_t *__restrict__ P, const uint32_t *__restrict__ Q, uint32_t *__restrict__ owner,
       unsigned long long *__restrict__ Wc, uint32_t rulers, uint32_t mmask, int kappa,
       uint32_t salt, uint32_t cap, uint32_t *__restrict__ gate) {
    const uint32_t rho = blockIdx.x * kThreads + threadIdx.x;
    if (rho >= rulers) return;
    const uint32_t kmask = (1u << kappa) - 1u;
    const uint32_t group = rho >> 1;
    const uint32_t t0 = (group << kappa) | ruler_slot(group, salt, kmask);
    uint32_t j = 2u * t0 + (rho & 1u);
    const uint32_t base = j & ~mmask;
    uint32_t mn = j, nxt = rho, hops = 0;
    if (!(rho & 1u)) owner[t0] = rho;
    for (;;) {
        uint32_t p = __ldg(P + (j ^ 1u)) & mmask;
        j = base + (__ldg(Q + base + (p ^ 1u)) & mmask);
        uint32_t t = j >> 1, g = t >> kappa;
        if ((t & kmask) == ruler_slot(g, salt, kmask)) {
            nxt = 2u * g + (j & 1u);
            break;
        }
        if (++hops > cap) {         // give up: the word stays a self loop
            *gate = 1u;
            break;
        }
        // somebody else gave up: the level is relabelled anyway
        if ((hops & 63u) == 0u && *reinterpret_cast<volatile uint32_t *>(gate)) break;
        mn = min(mn, j);
        if (!(j & 1u)) owner[t] = rho;
    }
    Wc[rho] = make_word(nxt, mn);
}

// Step 4 + output side of the level's switches.
__global__ void __launch_bounds__(kThreads)
k_colour(const uint32_t *__restrict__ P, const uint32_t *__restrict__ Q,
         const uint32_t *__restrict__ owner, const unsigned long long *__restrict__ Wc,
         size_t switches, uint32_t mmask, BitsLayout L, int out_stage, uint32_t cap,
         uint32_t *__restrict__ gate) {
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t t = size_t(blockIdx.x) * blockDim.x + threadIdx.x; t < switches; t += stride) {
        uint32_t o = __ldcs(owner + t);
        uint32_t mn;
        if (o != kUnowned) {
            mn = uint32_t(__ldg(Wc + o) >> 32);
        } else {
            // loop without ruler: walk the g-cycle of output 2t
            const uint32_t j0 = uint32_t(2 * t);
            const uint32_t base = j0 & ~mmask;
            uint32_t j = j0, hops = 0;
            mn = j0;
            for (;;) {
                uint32_t p = __ldg(P + (j ^ 1u)) & mmask;
                j = base + (__ldg(Q + base + (p ^ 1u)) & mmask);
                if (j == j0) break;
                if (++hops > cap) {
                    *gate = 1u;
                    break;
                }
                if ((hops & 63u) == 0u && *reinterpret_cast<volatile uint32_t *>(gate)) break;
                mn = min(mn, j);
            }
        }
        uint32_t word = __ballot_sync(0xFFFFFFFFu, mn & 1u);
        if ((threadIdx.x & 31) == 0) L.bits[L.word(out_stage, t >> 5)] = word;
    }
}

}  // namespace

int launch_walk(const uint32_t *P, const uint32_t *Q, uint32_t *owner, unsigned long long *Wc,
                size_t total, int log2m, int kappa, uint32_t salt, uint32_t cap, uint32_t *gate,
                cudaStream_t s) {
    const size_t rulers = total >> kappa;
    const unsigned grid = unsigned((rulers + kThreads - 1) / kThreads);
    k_walk<<<grid, kThreads, 0, s>>>(P, Q, owner, Wc, uint32_t(rulers), (1u << log2m) - 1u, kappa,
                                     salt, cap, gate);
    return launch_status();
}

int launch_colour(const uint32_t *P, const uint32_t *Q, const uint32_t *owner,
                  const unsigned long long *Wc, size_t total, int log2m, BitsLayout L,
                  int out_stage, uint32_t cap, uint32_t *gate, cudaStream_t s) {
    const size_t switches = total / 2;
    size_t blocks = (switches + kThreads - 1) / kThreads;
    const size_t capb = size_t(kSMs) * 8;
    k_colour<<<unsigned(blocks < capb ? blocks : capb), kThreads, 0, s>>>(
        P, Q, owner, Wc, switches, (1u << log2m) - 1u, L, out_stage, cap, gate);
    return launch_status();
}

}  // namespace benes
