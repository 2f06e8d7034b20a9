// Work-efficient loop labelling for the HBM levels: ruler sampling.
//
// Pointer jumping over all outputs costs O(M log M) random accesses per level.
// Here every output switch is visited ONCE per level:
//
//   1. Switches are cut into groups of k = 2^kappa consecutive switches; a hash
//      of the group number picks one RULER switch per group.  Both outputs of
//      a ruler switch are ruler outputs; ruler output rho = 2*group + (j & 1).
//   2. k_walk: one thread per ruler output follows the successor
//      g(j) = base + Q[base + (P[j^1] ^ 1)].  The g-cycle through output j
//      and the g-cycle through j^1 are mirror images (g(g(j)^1) = j^1), so the
//      walker that leaves ruler switch T forwards and the walker that leaves
//      the next ruler switch T' backwards run over the same switches from the
//      two ends.  Each claims the switches it reaches with a compare-and-swap
//      on the record's owner field and stops at the first switch the other one
//      owns: together they touch every switch of the segment once.  A walker
//      keeps the smallest output index on its own side of the switches it
//      claimed (fwd), the smallest on the far side (part), and its partner
//      (peer).  The claim stores (walker, side of arrival).  At the levels with
//      packed records and enough rulers to fill the GPU a thread advances the
//      two walkers of one ruler switch together (k_walk_multi).
//   3. k_combine: the segment of walker rho ends at ruler output peer^1 and
//      its minimum is min(fwd[rho], part[peer]): one 64-bit (next, min) word
//      per ruler output -- the contracted list.
//   4. The contracted list is labelled with the minimum of every cycle:
//      lists of up to 2^14 words per block in one CTA's shared memory, longer
//      ones by sampling again: the list is mirror symmetric like the loops, so
//      it is sampled the same way (one ruler pair per 16 pairs of words, walks
//      that meet in the middle, k_combine again).
//   5. k_colour: output 2t lies on its owner's cycle if the owner arrived on
//      the even side, else on the mirror cycle, which has the other colour:
//      colour = (cycle minimum of the owner & 1) ^ side.  A switch nobody
//      claimed lies on a loop without ruler; such loops are short
//      (probability (1-1/k)^length) and the thread walks the cycle itself.
//
// Every walk gives up after `cap` hops and raises the level's gate; the gate
// opens the full pointer-jumping kernel of route_levels.cu, which relabels the
// level.  So the result never depends on the sampling.
#include "common.cuh"

BENES_GUARD_TU("route_sampled.cu")

namespace benes {


namespace {

constexpr int kThreads = 256;
constexpr int kWalkThreads = 128;             // a CTA's slots are free again when its longest walk ends
constexpr int kListThreads = 1024;

__device__ __forceinline__ uint32_t ruler_slot(uint32_t group, uint32_t salt, uint32_t kmask) {
    uint32_t h = group * 0x9E3779B1u + salt;
    h ^= h >> 15;
    h *= 0x85EBCA6Bu;
    h ^= h >> 13;
    return h & kmask;
}

__device__ __forceinline__ bool gate_raised(const uint32_t *gate) {
    return *reinterpret_cast<const volatile uint32_t *>(gate) != 0u;
}

// Step 2.  rulers = T / k threads, launched in index order so that the blocks
// being walked at any moment are neighbours in memory.
//
// Wide records: the walker loads the record (16 B) and claims its owner word
// with a compare-and-swap.  Packed records: one 64-bit atomic AND with
// (my code << 2m | ones) returns the two P values and the previous owner and,
// if the switch was free (owner all ones), leaves my code there; if it was
// taken, the AND has mangled the other walker's code, and since nobody but the
// two of us ever touches this switch, writing the old word back repairs it.
template <bool PACKED>
__global__ void __launch_bounds__(kWalkThreads)
k_walk(void *__restrict__ Sv, const uint32_t *__restrict__ Q, uint4 *__restrict__ rec,
       uint32_t rulers, int m, int kappa, uint32_t salt, uint32_t cap,
       uint32_t *__restrict__ gate) {
    const uint32_t rho = blockIdx.x * kWalkThreads + threadIdx.x;
    if (rho >= rulers) return;
    const uint32_t mmask = (1u << m) - 1u;
    const uint32_t kmask = (1u << kappa) - 1u;
    const uint32_t group = rho >> 1, side0 = rho & 1u;
    const uint32_t t0 = (group << kappa) | ruler_slot(group, salt, kmask);
    uint32_t j = 2u * t0 + side0;
    const uint32_t base = j & ~mmask;
    uint32_t fwd = j, part = kUnowned, peer = rho ^ 1u, hops = 0;
    uint4 *S16 = static_cast<uint4 *>(Sv);
    unsigned long long *S8 = static_cast<unsigned long long *>(Sv);
    // packed owners are local to the block: its first ruler output is base >> kappa
    const uint32_t rho_base = base >> kappa;
    const int cshift = 2 * m;
    const unsigned long long low_ones = PACKED ? ((1ull << cshift) - 1ull) : 0ull;
    const uint32_t none8 = PACKED ? uint32_t(~0ull >> cshift) : 0u;

    uint32_t p;                                                   // P[j^1]
    if (PACKED) {
        unsigned long long w;
        // the ruler switch belongs to its even-side walker (nobody else claims it)
        if (!side0) w = atomicAnd(S8 + t0, ((unsigned long long)((rho - rho_base) << 1) << cshift) | low_ones);
        else w = __ldcg(S8 + t0);
        p = uint32_t(w >> (side0 ? 0 : m)) & mmask;
    } else {
        const uint4 r = __ldcg(S16 + t0);
        if (!side0) reinterpret_cast<uint32_t *>(S16 + t0)[2] = rho << 1;
        p = BENES_GUARD(side0 ? r.x : r.y, mmask);
    }
    uint32_t q = BENES_GUARD(__ldcg(Q + base + (p ^ 1u)), mmask);
    for (;;) {
        j = base + q;
        const uint32_t t = j >> 1, side = j & 1u, g = t >> kappa;
        if ((t & kmask) == ruler_slot(g, salt, kmask)) {          // reached the next ruler
            peer = (2u * g + side) ^ 1u;
            break;
        }
        if (++hops > cap) {
            *gate = 1u;
            break;
        }
        if ((hops & 63u) == 0u && gate_raised(gate)) break;       // the level is relabelled anyway
        uint32_t qn;
        bool met;
        if (PACKED) {
            const unsigned long long mine = (unsigned long long)(((rho - rho_base) << 1) | side) << cshift;
            const unsigned long long w = atomicAnd(S8 + t, mine | low_ones);
            p = uint32_t(w >> (side ? 0 : m)) & mmask;
            // next hop's gather, issued before the claim is looked at (harmless if we stop)
            qn = BENES_GUARD(__ldcg(Q + base + (p ^ 1u)), mmask);
            const uint32_t prev = uint32_t(w >> cshift);
            met = prev != none8;
            if (met) {
                __stcg(S8 + t, w);                                // put the other walker's code back
                peer = rho_base + (prev >> 1);
            }
        } else {
            const uint4 r = __ldcg(S16 + t);
            p = BENES_GUARD(side ? r.x : r.y, mmask);
            qn = BENES_GUARD(__ldcg(Q + base + (p ^ 1u)), mmask);
            uint32_t prev = r.z;
            if (prev == kUnowned)
                prev = atomicCAS(reinterpret_cast<uint32_t *>(S16 + t) + 2, kUnowned, (rho << 1) | side);
            met = prev != kUnowned;
            if (met) peer = prev >> 1;
        }
        if (met) break;                                           // met the walker from the other end
        fwd = min(fwd, j);
        part = min(part, j ^ 1u);
        q = qn;
    }
    rec[rho] = make_uint4(fwd, part, peer, 0u);
}

// Step 2, packed records, 2 G walkers per thread: the two ruler outputs of each of G
// neighbouring ruler switches (the two walks of a switch leave it in opposite
// directions).  A hop is a chain of two dependent L2 accesses and most lanes of a
// warp are idle while its longest walk lasts; advancing a thread's walks together,
// one hop each per round, overlaps their chains.  Same claims and records as
// k_walk<true>.  The hop limit counts rounds.
template <int G>
__global__ void __launch_bounds__(kWalkThreads)
k_walk_multi(unsigned long long *__restrict__ S8, const uint32_t *__restrict__ Q, uint4 *__restrict__ rec,
             uint32_t groups, int m, int kappa, uint32_t salt, uint32_t cap, uint32_t *__restrict__ gate) {
    constexpr int W = 2 * G;
    const uint32_t group0 = (blockIdx.x * kWalkThreads + threadIdx.x) * G;     // groups is a multiple of G
    if (group0 >= groups) return;
    const uint32_t mmask = (1u << m) - 1u;
    const uint32_t kmask = (1u << kappa) - 1u;
    const int cshift = 2 * m;
    const unsigned long long low_ones = (1ull << cshift) - 1ull;
    const uint32_t none8 = uint32_t(~0ull >> cshift);
    const uint32_t rho0 = 2u * group0;                               // walker i is ruler output rho0 + i
    // G neighbouring groups lie in one block (a block has at least 2^7 ruler outputs)
    const uint32_t base = (2u * (group0 << kappa)) & ~mmask;
    const uint32_t rho_base = base >> kappa;
    uint32_t q[W], fwd[W], part[W], peer[W];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const uint32_t group = group0 + g;
        const uint32_t t0 = (group << kappa) | ruler_slot(group, salt, kmask);
        // the ruler switch belongs to its even-side walker; the claim returns both P values
        const unsigned long long w0 = atomicAnd(S8 + t0, ((unsigned long long)((2u * group - rho_base) << 1) << cshift) | low_ones);
        q[2 * g] = BENES_GUARD(__ldcg(Q + base + ((uint32_t(w0 >> m) & mmask) ^ 1u)), mmask);     // needs P[2 t0 + 1]
        q[2 * g + 1] = BENES_GUARD(__ldcg(Q + base + ((uint32_t(w0) & mmask) ^ 1u)), mmask);      // needs P[2 t0]
        fwd[2 * g] = 2u * t0; fwd[2 * g + 1] = 2u * t0 + 1u;
        part[2 * g] = part[2 * g + 1] = kUnowned;
        peer[2 * g] = (2u * group) ^ 1u; peer[2 * g + 1] = 2u * group;
    }
    uint32_t active = (1u << W) - 1u, hops = 0;
    while (active) {
        if (++hops > cap) {
            *gate = 1u;
            break;
        }
        if ((hops & 63u) == 0u && gate_raised(gate)) break;         // the level is relabelled anyway
        unsigned long long w[W];
#pragma unroll
        for (int i = 0; i < W; ++i) {
            w[i] = 0ull;
            if (!((active >> i) & 1u)) continue;
            const uint32_t j = base + q[i], t = j >> 1, side = j & 1u, g = t >> kappa;
            if ((t & kmask) == ruler_slot(g, salt, kmask)) {        // reached the next ruler
                peer[i] = (2u * g + side) ^ 1u;
                active &= ~(1u << i);
            } else {
                w[i] = atomicAnd(S8 + t, ((unsigned long long)((((rho0 + i) - rho_base) << 1) | side) << cshift) | low_ones);
            }
        }
        uint32_t qn[W];
#pragma unroll
        for (int i = 0; i < W; ++i) {
            qn[i] = 0u;
            if (!((active >> i) & 1u)) continue;
            const uint32_t side = q[i] & 1u;                        // base is even
            const uint32_t p = uint32_t(w[i] >> (side ? 0 : m)) & mmask;
            qn[i] = BENES_GUARD(__ldcg(Q + base + (p ^ 1u)), mmask);
        }
#pragma unroll
        for (int i = 0; i < W; ++i) {
            if (!((active >> i) & 1u)) continue;
            const uint32_t j = base + q[i];
            const uint32_t prev = uint32_t(w[i] >> cshift);
            if (prev != none8) {                                    // met the walker from the other end
                __stcg(S8 + (j >> 1), w[i]);                        // put its code back
                peer[i] = rho_base + (prev >> 1);
                active &= ~(1u << i);
            } else {
                fwd[i] = min(fwd[i], j);
                part[i] = min(part[i], j ^ 1u);
                q[i] = qn[i];
            }
        }
    }
#pragma unroll
    for (int i = 0; i < W; ++i) rec[rho0 + i] = make_uint4(fwd[i], part[i], peer[i], 0u);
}

// Step 3.
__global__ void __launch_bounds__(kThreads)
k_combine(const uint4 *__restrict__ rec, unsigned long long *__restrict__ W, uint32_t rulers) {
    const uint32_t rho = blockIdx.x * kThreads + threadIdx.x;
    if (rho >= rulers) return;
    const uint4 a = rec[rho];
    const uint32_t peer = BENES_GUARD_BELOW(a.z, rulers, rho);
    const uint4 b = __ldg(rec + peer);
    W[rho] = make_word(peer ^ 1u, min(a.x, b.y));
}

// Step 4, sampling a list.  The contracted list inherits the mirror symmetry
// of the loops (next[rho] = sigma implies next[sigma ^ 1] = rho ^ 1), and so does
// every list sampled from it this way: a list is sampled the way the switches are.  Words 2q and 2q+1 form a pair; one pair per 16
// pairs is a ruler pair, both of its words start a walker; the walker from the
// even word runs along its cycle, the walker from the odd word of the NEXT
// ruler pair runs along the mirror cycle, i.e. over the same pairs from the
// other end; each claims pairs (owner[q] = walker, side of arrival) and stops
// where the other one has been.  The longest walk of a launch is half as long
// as with one-directional walks.  A walker keeps the minimum over the words it
// passed (fwd), over their partners (part) and whom it met (peer): the same
// record as in step 2, turned into the 16 times shorter list by k_combine.
constexpr int kPairGroupLog2 = kListKappa;          // pairs per ruler pair (log2)

__global__ void __launch_bounds__(kWalkThreads)
k_list_walk_pairs(const ulonglong2 *__restrict__ W2p, uint32_t *__restrict__ owner, uint4 *__restrict__ rec,
                  uint32_t rulers, uint32_t pairs, uint32_t salt, uint32_t cap, uint32_t *__restrict__ gate) {
    const uint32_t sigma = blockIdx.x * kWalkThreads + threadIdx.x;
    if (sigma >= rulers) return;
    constexpr uint32_t kmask = (1u << kPairGroupLog2) - 1u;
    const uint32_t group = sigma >> 1, side0 = sigma & 1u;
    const uint32_t q0 = (group << kPairGroupLog2) | ruler_slot(group, salt, kmask);
    ulonglong2 w = __ldcg(W2p + q0);
    if (!side0) owner[q0] = sigma << 1;                            // the ruler pair belongs to its even walker
    unsigned long long own = side0 ? w.y : w.x;
    uint32_t fwd = uint32_t(own >> 32), part = kUnowned, peer = sigma ^ 1u, hops = 0;
    for (;;) {
        // (a batch need not be a power of two: an index a raised gate left undefined is clamped, not masked)
        const uint32_t e = uint32_t(own), q = BENES_GUARD_BELOW(e >> 1, pairs, 0u), side = e & 1u, g = q >> kPairGroupLog2;
        if ((q & kmask) == ruler_slot(g, salt, kmask)) {           // reached the next ruler pair
            peer = (2u * g + side) ^ 1u;
            break;
        }
        if (++hops > cap) {
            *gate = 1u;
            break;
        }
        if ((hops & 63u) == 0u && gate_raised(gate)) break;
        w = __ldcg(W2p + q);
        const uint32_t prev = atomicCAS(owner + q, kUnowned, (sigma << 1) | side);
        if (prev != kUnowned) {                                    // met the walker from the other end
            peer = prev >> 1;
            break;
        }
        own = side ? w.y : w.x;
        const unsigned long long far = side ? w.x : w.y;
        fwd = min(fwd, uint32_t(own >> 32));
        part = min(part, uint32_t(far >> 32));
    }
    rec[sigma] = make_uint4(fwd, part, peer, 0u);
}

// Back from a sampled list: a thread takes the pair 2q, 2q+1 (and hands the
// owner slot back as kUnowned).  Word 2q + b lies on its owner's cycle if the
// owner arrived on side b, else on the mirror cycle, which is the cycle of the
// owner's partner walker and whose minimum has the other parity.  A pair nobody
// claimed lies on a cycle without ruler pair: the thread walks the cycle of
// word 2q (and that of word 2q+1 if the minima themselves are needed).
// Of the first list (the rulers of the level) only the parity of the minima is
// needed afterwards: with `cb` one bit per word goes there, so that the colouring
// kernel gathers from an array 64 times smaller than the list (it stays in
// L1/L2 next to the streaming traffic); without, the words take their minima.
__device__ __forceinline__ uint32_t list_cycle_min(const unsigned long long *W, uint32_t e0, uint32_t words,
                                                   uint32_t cap, uint32_t *gate) {
    unsigned long long v = __ldcg(W + e0);
    uint32_t mn = uint32_t(v >> 32), e = BENES_GUARD_BELOW(uint32_t(v), words, 0u), hops = 0;
    while (e != e0) {
        if (++hops > cap) {
            *gate = 1u;
            break;
        }
        v = __ldcg(W + e);
        mn = min(mn, uint32_t(v >> 32));       // words rewritten meanwhile hold the minimum of this same cycle
        e = BENES_GUARD_BELOW(uint32_t(v), words, 0u);
    }
    return mn;
}

__global__ void __launch_bounds__(kThreads)
k_list_resolve_pairs(unsigned long long *__restrict__ W, uint32_t *__restrict__ owner,
                     const unsigned long long *__restrict__ W2, uint32_t pairs, uint32_t words,
                     uint32_t cap, uint32_t *__restrict__ gate, uint32_t *__restrict__ cb) {
    const uint32_t q = blockIdx.x * kThreads + threadIdx.x;       // pairs is a multiple of 32
    if (q >= pairs) return;
    const uint32_t code = owner[q];
    if (!cb) {
        uint32_t mn0, mn1;
        if (code != kUnowned) {
            const uint32_t a = uint32_t(__ldcg(W2 + (code >> 1)) >> 32), b = uint32_t(__ldcg(W2 + ((code >> 1) ^ 1u)) >> 32);
            mn0 = (code & 1u) ? b : a;
            mn1 = (code & 1u) ? a : b;
            owner[q] = kUnowned;
        } else {
            mn0 = list_cycle_min(W, 2u * q, words, cap, gate);
            mn1 = list_cycle_min(W, 2u * q + 1u, words, cap, gate);
        }
        ulonglong2 *Wp = reinterpret_cast<ulonglong2 *>(W) + q;
        ulonglong2 w = *Wp;
        w.x = make_word(uint32_t(w.x), mn0);
        w.y = make_word(uint32_t(w.y), mn1);
        *Wp = w;
        return;
    }
    uint32_t bit0;
    if (code != kUnowned) {
        bit0 = (uint32_t(__ldcg(W2 + (code >> 1)) >> 32) ^ code) & 1u;
        owner[q] = kUnowned;
    } else {
        bit0 = list_cycle_min(W, 2u * q, words, cap, gate) & 1u;
    }
    // a warp covers 64 words: two words of cb
    store_stage_bits64(cb + ((q - (threadIdx.x & 31u)) >> 4), bit0, bit0 ^ 1u);
}

// Step 4, the end of the recursion: one CTA labels one block's list of
// 2^log2b words in shared memory by synchronous pointer jumping (new words are
// held in registers across the barrier; PER words per thread, blockDim =
// 2^log2b / PER).  A cycle and its mirror image have the same number of words
// and lie in the same block, so a cycle has at most 2^(log2b-1) words: log2b - 1
// passes.
// With `cb` (first list of a level) the parities of the minima go there, one bit
// per word, instead of the words back to W.
template <int PER>
__global__ void __launch_bounds__(kListThreads)
k_list_label(unsigned long long *__restrict__ W, int log2b, uint32_t *__restrict__ cb) {
    extern __shared__ unsigned long long sm[];
    const uint32_t B = 1u << log2b, bmask = B - 1u;
    const size_t base = size_t(blockIdx.x) << log2b;
    const uint32_t T = blockDim.x, tid = threadIdx.x;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const uint32_t e = tid + uint32_t(i) * T;
        unsigned long long w = __ldcs(W + base + e);
        sm[e] = make_word(uint32_t(w) & bmask, uint32_t(w >> 32));
    }
    __syncthreads();
    unsigned long long v[PER];
    for (int pass = 0; pass < log2b - 1; ++pass) {
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const unsigned long long w = sm[tid + uint32_t(i) * T];
            const unsigned long long t = sm[uint32_t(w)];
            v[i] = make_word(uint32_t(t), min(uint32_t(w >> 32), uint32_t(t >> 32)));
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < PER; ++i) sm[tid + uint32_t(i) * T] = v[i];
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const uint32_t e = tid + uint32_t(i) * T;
        const unsigned long long w = sm[e];
        if (cb) {
            const uint32_t word = __ballot_sync(0xFFFFFFFFu, uint32_t(w >> 32) & 1u);
            if ((tid & 31u) == 0u) cb[(base + e) >> 5] = word;
        } else {
            W[base + e] = make_word(uint32_t(base) + uint32_t(w), uint32_t(w >> 32));
        }
    }
}

template <int PER>
int launch_list_label(unsigned long long *W, uint32_t count, int beta, uint32_t *cb, cudaStream_t s) {
    static OncePerDevice configured;
    const size_t smem = (size_t(1) << beta) * 8;
    {
        const int rc = configured.run([]() -> int {
            BENES_CUDA_TRY(cudaFuncSetAttribute(k_list_label<PER>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (1 << kListSmemLog2) * 8));
            return BENES_OK;
        });
        if (rc) return rc;
    }
    k_list_label<PER><<<count >> beta, (1u << beta) / PER, smem, s>>>(W, beta, cb);
    return launch_status();
}

// Steps 3 and 4 in one kernel for a level whose blocks have at most 2^18 outputs
// and lists that fit one CTA (no sampling of the list): the CTA forms its
// block's list words from the walk records, (next, min) = (peer ^ 1,
// min(fwd[rho], part[peer])), as 14 + 18 bit, both local to the block, labels
// them by synchronous pointer jumping and writes the parity bits.  Indices a
// raised gate may have left undefined are masked into the block.
template <int PER>
__global__ void __launch_bounds__(kListThreads)
k_list_label_rec(const uint4 *__restrict__ rec, uint32_t *__restrict__ cb, int log2b, int m) {
    extern __shared__ uint32_t sw[];
    constexpr uint32_t kNext = (1u << kListSmemLog2) - 1u;
    const uint32_t B = 1u << log2b, bmask = B - 1u, mmask = (1u << m) - 1u;
    const uint32_t base = blockIdx.x << log2b;                    // first ruler output of the block
    const uint32_t T = blockDim.x, tid = threadIdx.x;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const uint32_t e = tid + uint32_t(i) * T;
        const uint4 a = __ldcs(rec + base + e);
        const uint32_t peer = a.z & bmask;
        const uint4 b = __ldg(rec + base + peer);
        sw[e] = (peer ^ 1u) | ((min(a.x, b.y) & mmask) << kListSmemLog2);
    }
    __syncthreads();
    uint32_t v[PER];
    for (int pass = 0; pass < log2b - 1; ++pass) {
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t w = sw[tid + uint32_t(i) * T];
            const uint32_t t = sw[w & kNext];
            v[i] = (t & kNext) | min(w & ~kNext, t & ~kNext);
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < PER; ++i) sw[tid + uint32_t(i) * T] = v[i];
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const uint32_t e = tid + uint32_t(i) * T;
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, (sw[e] >> kListSmemLog2) & 1u);
        if ((tid & 31u) == 0u) cb[(base + e) >> 5] = word;
    }
}

template <int PER>
int launch_list_label_rec(const uint4 *rec, uint32_t *cb, uint32_t count, int beta, int m, cudaStream_t s) {
    static OncePerDevice configured;
    {
        const int rc = configured.run([]() -> int {
            BENES_CUDA_TRY(cudaFuncSetAttribute(k_list_label_rec<PER>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (1 << kListSmemLog2) * 4));
            return BENES_OK;
        });
        if (rc) return rc;
    }
    k_list_label_rec<PER><<<count >> beta, (1u << beta) / PER, (size_t(1) << beta) * 4, s>>>(rec, cb, beta, m);
    return launch_status();
}

// Step 5 for a switch on a loop without ruler: the minimum of the g-cycle C of
// output 2t, walked from both ends.  The cycle of output 2t+1 is the mirror
// image of C (g(g(j)^1) = j^1), so g(b^1)^1 is the predecessor of b on C: one
// chain follows C forwards, the other backwards, their gathers overlap, and
// they stop where they meet.  p_even / p_odd = P[2t] / P[2t+1], which the
// caller holds already, start the two chains.
template <bool PACKED>
__device__ __forceinline__ uint32_t loop_colour(const void *S, const uint32_t *Q, uint32_t t, uint32_t base,
                                                uint32_t p_even, uint32_t p_odd, int m, uint32_t mmask,
                                                uint32_t cap, uint32_t *gate) {
    const uint32_t j0 = 2u * t;
    uint32_t f = j0, bk = j0, mn = j0, hops = 0;
    uint32_t pf = p_odd;                 // P[f ^ 1]
    uint32_t pb = p_even;                // P[bk]
    for (;;) {
        const uint32_t qf = BENES_GUARD(__ldg(Q + base + (pf ^ 1u)), mmask);        // g(f)
        const uint32_t qb = BENES_GUARD(__ldg(Q + base + (pb ^ 1u)), mmask);        // g(bk ^ 1)
        f = base + qf;
        if (f == bk) break;                                             // forwards reached the part walked backwards
        mn = min(mn, f);
        bk = (base + qb) ^ 1u;
        if (bk == f) break;                                             // both ends on the same output
        mn = min(mn, bk);
        if (++hops > cap) {
            *gate = 1u;
            break;
        }
        if ((hops & 63u) == 0u && gate_raised(gate)) break;
        pf = rec_p<PACKED>(S, f ^ 1u, m);
        pb = rec_p<PACKED>(S, bk, m);
    }
    return mn & 1u;
}

// colour of output 2t from the owner of switch t
__device__ __forceinline__ uint32_t owner_colour(const uint32_t *cb, uint32_t code, uint32_t rulers) {
    const uint32_t rho = BENES_GUARD_BELOW(code >> 1, rulers, 0u);
    return ((__ldg(cb + (rho >> 5)) >> (rho & 31u)) ^ code) & 1u;
}

// Step 5 + output side of the level's switches + the next level's records
// (owner reset).  A thread owns the neighbouring switches 2i and 2i+1: their
// colour-0 outputs are neighbours in the upper half-block of the next level and
// their colour-1 outputs in the lower one, i.e. the thread writes one whole
// record of each.  If the gate is raised afterwards, the split kernel redoes
// the records from the relabelled stage.
template <bool PACKED, bool NEXT_PACKED>
__global__ void __launch_bounds__(kThreads)
k_colour(const void *__restrict__ S, const uint32_t *__restrict__ Q,
         const uint32_t *__restrict__ cb, void *__restrict__ Sn, uint32_t pairs,
         uint32_t rulers, int m, int kappa, BitsLayout L, int out_stage, uint32_t cap,
         uint32_t *__restrict__ gate, uint32_t rounds) {
    // a CTA takes `rounds` consecutive groups of blockDim.x pairs: the ruler bits
    // it gathers belong to one block of the level for a long time (L1 hits)
    const uint32_t stride = blockDim.x;
    const uint32_t last = min(pairs, (blockIdx.x + 1u) * rounds * stride);
    const uint32_t mmask = (1u << m) - 1u;
    const uint32_t H = (mmask + 1) >> 1;
    const uint32_t none = PACKED ? uint32_t(~0ull >> (2 * m)) : kUnowned;
    // packed fields with 32-bit operations (m < 32): the owner starts at bit 2m of
    // the word, the next level's owner (all ones) at bit 2(m-1)
    const int s_own = 2 * m, s_next = 2 * (m - 1);
    const uint32_t ones_lo = s_next < 32 ? ~0u << s_next : 0u;
    const uint32_t ones_hi = s_next < 32 ? ~0u : ~0u << (s_next - 32);
    // the records of the next round are on their way while this one is coloured
    // (pairs is a multiple of 32: a warp stays together)
    uint32_t i = blockIdx.x * rounds * stride + threadIdx.x;
    ulonglong2 w = make_ulonglong2(0, 0);
    uint4 r0 = make_uint4(0, 0, 0, 0), r1 = r0;
    if (i < last) {
        if (PACKED) w = __ldcs(static_cast<const ulonglong2 *>(S) + i);
        else { r0 = __ldcs(static_cast<const uint4 *>(S) + 2 * size_t(i)); r1 = __ldcs(static_cast<const uint4 *>(S) + 2 * size_t(i) + 1); }
    }
    while (i < last) {
        const uint32_t inext = i + stride;
        ulonglong2 wn = make_ulonglong2(0, 0);
        uint4 r0n = make_uint4(0, 0, 0, 0), r1n = r0n;
        if (inext < last) {
            if (PACKED) wn = __ldcs(static_cast<const ulonglong2 *>(S) + inext);
            else { r0n = __ldcs(static_cast<const uint4 *>(S) + 2 * size_t(inext)); r1n = __ldcs(static_cast<const uint4 *>(S) + 2 * size_t(inext) + 1); }
        }
        const uint32_t t = 2u * i;                              // first switch of the pair
        const uint32_t base = (2u * t) & ~mmask;
        uint32_t px0, py0, px1, py1, code0, code1;
        bool own0, own1;
        if (PACKED) {
            const uint32_t rb = (base >> kappa) << 1;
            const uint32_t lo0 = uint32_t(w.x), hi0 = uint32_t(w.x >> 32);
            const uint32_t lo1 = uint32_t(w.y), hi1 = uint32_t(w.y >> 32);
            px0 = lo0 & mmask; py0 = __funnelshift_r(lo0, hi0, m) & mmask;
            px1 = lo1 & mmask; py1 = __funnelshift_r(lo1, hi1, m) & mmask;
            const uint32_t l0 = s_own >= 32 ? hi0 >> (s_own - 32) : __funnelshift_r(lo0, hi0, s_own);
            const uint32_t l1 = s_own >= 32 ? hi1 >> (s_own - 32) : __funnelshift_r(lo1, hi1, s_own);
            own0 = l0 != none; own1 = l1 != none;
            code0 = rb + l0; code1 = rb + l1;                    // owner local to the block -> global
        } else {
            px0 = BENES_GUARD(r0.x, mmask); py0 = BENES_GUARD(r0.y, mmask); code0 = r0.z; own0 = code0 != none;
            px1 = BENES_GUARD(r1.x, mmask); py1 = BENES_GUARD(r1.y, mmask); code1 = r1.z; own1 = code1 != none;
        }
        // all but the switches of loops without ruler are owned
        const uint32_t c0 = own0 ? owner_colour(cb, code0, rulers)
                                 : loop_colour<PACKED>(S, Q, t, base, px0, py0, m, mmask, cap, gate);
        const uint32_t c1 = own1 ? owner_colour(cb, code1, rulers)
                                 : loop_colour<PACKED>(S, Q, t + 1u, base, px1, py1, m, mmask, cap, gate);
        // a warp covers 64 switches: two words of the output-side stage
        store_stage_bits64(L.bits + L.word32(out_stage, (t - 2u * (threadIdx.x & 31u)) >> 5), c0, c1);
        const uint32_t r = (base >> 1) + (((t - (base >> 1)) >> 1));   // record of the upper half
        const uint32_t u0 = (c0 ? py0 : px0) >> 1, u1 = (c1 ? py1 : px1) >> 1;     // upper half-block
        const uint32_t d0 = (c0 ? px0 : py0) >> 1, d1 = (c1 ? px1 : py1) >> 1;     // lower half-block
        if (NEXT_PACKED) {
            uint2 *Sn8 = static_cast<uint2 *>(Sn);
            Sn8[r] = make_uint2(u0 | (u1 << (m - 1)) | ones_lo, (u1 >> (33 - m)) | ones_hi);
            Sn8[r + (H >> 1)] = make_uint2(d0 | (d1 << (m - 1)) | ones_lo, (d1 >> (33 - m)) | ones_hi);
        } else {
            rec_write<false>(Sn, r, m - 1, u0, u1);
            rec_write<false>(Sn, r + (H >> 1), m - 1, d0, d1);
        }
        w = wn; r0 = r0n; r1 = r1n;
        i = inext;
    }
}

inline size_t align256(size_t v) { return (v + 255) & ~size_t(255); }
constexpr int kMaxLists = 5;

// Number of times the list of a block with 2^beta words is sampled again.
inline int list_depth(int beta) {
    int d = 0;
    while (beta > kListSmemLog2 && d < kMaxLists - 1) {
        beta -= kListKappa;
        ++d;
    }
    return d;
}

}  // namespace

// Scratch: walk records, the contracted lists and the owners of every list
// that may be sampled again.  Sized for the largest level (log2m = 30).
size_t sampled_scratch_bytes(size_t total, int kappa) {
    size_t R = total >> kappa, bytes = align256(R * 16) + align256(R / 8 + 4);
    for (int i = 0; i < kMaxLists; ++i) {
        size_t c = R >> (kListKappa * i);
        if (c < 4) c = 4;
        bytes += align256(c * 8) + align256(c * 4);
    }
    return bytes;
}

void sampled_scratch_carve(char *base, size_t total, int kappa, SampledScratch *out) {
    size_t R = total >> kappa, off = 0;
    out->rec = reinterpret_cast<uint4 *>(base);
    off += align256(R * 16);
    out->ruler_bits = reinterpret_cast<uint32_t *>(base + off);
    off += align256(R / 8 + 4);
    for (int i = 0; i < kMaxLists; ++i) {
        size_t c = R >> (kListKappa * i);
        if (c < 4) c = 4;
        out->list[i] = reinterpret_cast<unsigned long long *>(base + off);
        off += align256(c * 8);
        out->owner[i] = reinterpret_cast<uint32_t *>(base + off);
        off += align256(c * 4);
    }
}

int sampled_scratch_reset(const SampledScratch &sc, size_t total, int kappa, cudaStream_t s) {
    size_t R = total >> kappa;
    for (int i = 0; i < kMaxLists - 1; ++i) {
        size_t c = R >> (kListKappa * i);
        if (c < 4) c = 4;
        BENES_CUDA_TRY(cudaMemsetAsync(sc.owner[i], 0xFF, c * 4, s));
    }
    return BENES_OK;
}

int sampled_label(void *S, bool packed, const uint32_t *Q, void *Sn, bool next_packed,
                  const SampledScratch &sc, size_t total, int log2m, int kappa, uint32_t salt,
                  uint32_t cap, int walk_pairs, BitsLayout L, int out_stage, uint32_t *gate, cudaStream_t s) {
    const uint32_t R = uint32_t(total >> kappa);
    const unsigned rgrid = (R + kThreads - 1) / kThreads;
    {
        ProfileScope ps(kWalk, s);
        const unsigned wgrid = (R + kWalkThreads - 1) / kWalkThreads;
        // Two walkers per thread pay once the halved number of threads still fills the GPU
        // (C4, cache-resident levels: 0.52-0.57 instead of 0.55-0.63 ms); below that the launch
        // lasts as long as its longest thread and one walker per thread is faster.  Four and
        // eight walkers per thread measured slower (0.60 and 0.90 ms).
        const bool pair = walk_pairs == 2 || (walk_pairs == 1 && size_t(R >> 1) >= size_t(sm_count()) * 2048);
        if (packed && pair)
            k_walk_multi<1><<<((R >> 1) + kWalkThreads - 1) / kWalkThreads, kWalkThreads, 0, s>>>(
                static_cast<unsigned long long *>(S), Q, sc.rec, R >> 1, log2m, kappa, salt, cap, gate);
        else if (packed) k_walk<true><<<wgrid, kWalkThreads, 0, s>>>(S, Q, sc.rec, R, log2m, kappa, salt, cap, gate);
        else k_walk<false><<<wgrid, kWalkThreads, 0, s>>>(S, Q, sc.rec, R, log2m, kappa, salt, cap, gate);
        int rc = launch_status();
        if (rc) return rc;
    }
    uint32_t *cb = sc.ruler_bits;
    // label the contracted list: sample it until a block's list fits one CTA
    int beta = log2m - kappa;
    const int depth = list_depth(beta);
    uint32_t count = R;
    // (the kernels that write the parity bits ballot: whole warps, i.e. lists of 2^7 words at least)
    if (depth == 0 && beta < 7) return BENES_ERR_BADARG;
    const bool from_records = depth == 0 && log2m <= 32 - kListSmemLog2;
    if (from_records) {
        ProfileScope ps(kListLabel, s);
        int rc = beta <= 12 ? launch_list_label_rec<4>(sc.rec, cb, count, beta, log2m, s)
               : beta == 13 ? launch_list_label_rec<8>(sc.rec, cb, count, beta, log2m, s)
                            : launch_list_label_rec<16>(sc.rec, cb, count, beta, log2m, s);
        if (rc) return rc;
    } else {
        ProfileScope ps(kCombine, s);
        k_combine<<<rgrid, kThreads, 0, s>>>(sc.rec, sc.list[0], R);
        int rc = launch_status();
        if (rc) return rc;
    }
    for (int d = 0; d < depth; ++d) {
        // walks from both ends; the walk records of the previous stage (switches,
        // or the list before) are dead, their memory takes the new ones
        const uint32_t next = count >> kListKappa;
        {
            ProfileScope ps(kListWalk, s);
            k_list_walk_pairs<<<(next + kWalkThreads - 1) / kWalkThreads, kWalkThreads, 0, s>>>(
                reinterpret_cast<const ulonglong2 *>(sc.list[d]), sc.owner[d], sc.rec, next, count >> 1,
                salt * 7u + uint32_t(d) + 1u, cap, gate);
            int rc = launch_status();
            if (rc) return rc;
        }
        {
            ProfileScope ps(kCombine, s);
            k_combine<<<(next + kThreads - 1) / kThreads, kThreads, 0, s>>>(sc.rec, sc.list[d + 1], next);
            int rc = launch_status();
            if (rc) return rc;
        }
        count = next;
        beta -= kListKappa;
    }
    if (!from_records) {
        ProfileScope ps(kListLabel, s);
        if (beta > kListSmemLog2 || beta < 5) return BENES_ERR_BADARG;
        // 4 words per thread up to 2^12 words, then 1024 threads
        uint32_t *bits_out = depth == 0 ? cb : nullptr;
        int rc = beta <= 12 ? launch_list_label<4>(sc.list[depth], count, beta, bits_out, s)
               : beta == 13 ? launch_list_label<8>(sc.list[depth], count, beta, bits_out, s)
                            : launch_list_label<16>(sc.list[depth], count, beta, bits_out, s);
        if (rc) return rc;
    }
    for (int d = depth - 1; d >= 0; --d) {
        ProfileScope ps(kListResolve, s);
        const uint32_t c = R >> (kListKappa * d);
        k_list_resolve_pairs<<<(c / 2 + kThreads - 1) / kThreads, kThreads, 0, s>>>(
            sc.list[d], sc.owner[d], sc.list[d + 1], c / 2, c, cap, gate, d == 0 ? cb : nullptr);
        int rc = launch_status();
        if (rc) return rc;
    }
    {
        ProfileScope ps(kColour, s);
        const uint32_t switches = uint32_t(total / 4);           // pairs of switches, one per thread
        const uint32_t rounds = stream_rounds(switches, kThreads);
        const unsigned grid = unsigned((size_t(switches) + size_t(kThreads) * rounds - 1) / (size_t(kThreads) * rounds));
        if (packed)          // a packed level is followed by packed levels only
            k_colour<true, true><<<grid, kThreads, 0, s>>>(S, Q, cb, Sn, switches, R, log2m, kappa, L,
                                                            out_stage, cap, gate, rounds);
        else if (next_packed)
            k_colour<false, true><<<grid, kThreads, 0, s>>>(S, Q, cb, Sn, switches, R, log2m, kappa, L,
                                                             out_stage, cap, gate, rounds);
        else
            k_colour<false, false><<<grid, kThreads, 0, s>>>(S, Q, cb, Sn, switches, R, log2m, kappa, L,
                                                              out_stage, cap, gate, rounds);
        return launch_status();
    }
}

}  // namespace benes
