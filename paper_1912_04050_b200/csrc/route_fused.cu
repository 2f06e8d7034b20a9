// Fused path: one CTA finishes every remaining level of one block of size
// M = 2^LOGM entirely in shared memory (inverse scatter, successor pairing,
// pointer jumping, colouring, stage bits, compaction, middle stage).  It serves
// both the tail of a large permutation (the flat level-(n-LOGM) array holds
// N/M blocks) and a batch of small permutations (N = M, one CTA each).
//
// Shared-memory words are 32 bit: low 16 = nxt, high 16 = mn, both indices
// local to the CTA's block (M <= 2^16).  Passes are separated by a CTA barrier,
// updates inside a pass are in place: a 32-bit shared-memory access is atomic,
// and a word read at any time satisfies "mn = min over the path from j up to,
// excluding, nxt", so every pass at least doubles the shortest window.
#include "common.cuh"

namespace benes {
namespace {

template <int LOGM>
struct FusedCfg {
    static constexpr int M = 1 << LOGM;
    static constexpr int kPairs = M / 2;
    static constexpr int kThreads = kPairs >= 1024 ? 1024 : (kPairs >= 32 ? kPairs : 32);
    static constexpr int kColourWords = M >= 64 ? M / 64 : 1;
    // Pa, Pb, Q: uint16[M] each; Wd: uint32[M]; colour words
    static constexpr size_t kSmemBytes = size_t(M) * (2 + 2 + 2 + 4) + size_t(kColourWords) * 4;
};

template <int LOGM>
__global__ void __launch_bounds__(FusedCfg<LOGM>::kThreads)
k_route_fused(const uint32_t *__restrict__ P, int records, uint32_t *__restrict__ bits, int log2n) {
    using C = FusedCfg<LOGM>;
    constexpr int M = C::M;
    constexpr int T = C::kThreads;
    // pair loops run over a multiple of 32 so that every lane reaches the ballots
    constexpr int kPairsPadded = C::kPairs >= 32 ? C::kPairs : 32;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint16_t *Pa = reinterpret_cast<uint16_t *>(smem_raw);
    uint16_t *Pb = Pa + M;
    uint16_t *Q = Pb + M;
    uint32_t *Wd = reinterpret_cast<uint32_t *>(Q + M);
    uint32_t *cw = Wd + M;

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int n = log2n;
    const int level0 = n - LOGM;               // recursion level of this CTA's block
    const size_t flat0 = size_t(blockIdx.x) << LOGM;
    // where this CTA's words of a stage start
    const size_t N = size_t(1) << n;
    const size_t stage_w = N >= 64 ? N / 64 : 1;
    const size_t perm = flat0 >> n;
    const size_t local_first_switch = (flat0 & (N - 1)) >> 1;
    uint32_t *my_bits = bits + perm * size_t(2 * n - 1) * stage_w + (local_first_switch >> 5);

    // plain array, or 16-byte switch records {P[2t], P[2t+1], -, -}
    for (int j = tid; j < M; j += T) {
        size_t f = flat0 + j;
        uint32_t v = records ? P[((f >> 1) << 2) | (f & 1)] : P[f];
        Pa[j] = uint16_t(v & uint32_t(M - 1));
    }
    __syncthreads();

#pragma unroll 1
    for (int k = 0; k < LOGM; ++k) {
        const int logS = LOGM - k;
        const uint32_t S = 1u << logS;
        const uint32_t smask = S - 1u;
        const int level = level0 + k;

        if (logS == 1) {
            // a7: middle stage, crossed iff output 0 of the 2-block takes input 1
            for (int t = tid; t < kPairsPadded; t += T) {
                uint32_t b = (t < C::kPairs) ? (Pa[2 * t] & 1u) : 0u;
                uint32_t word = __ballot_sync(0xFFFFFFFFu, b);
                if (lane == 0) my_bits[size_t(n - 1) * stage_w + (t >> 5)] = word;
            }
            break;
        }

        // a1: block-local inverse
        for (int j = tid; j < M; j += T) {
            uint32_t sb = uint32_t(j) & ~smask;
            Q[sb + (Pa[j] & smask)] = uint16_t(uint32_t(j) & smask);
        }
        __syncthreads();

        // a2: successor and initial word
        for (int t = tid; t < C::kPairs; t += T) {
            uint32_t j = 2u * t;
            uint32_t sb = j & ~smask;
            uint32_t p0 = Pa[j] & smask, p1 = Pa[j + 1] & smask;
            uint32_t g0 = sb + (Q[sb + (p1 ^ 1u)] & smask);
            uint32_t g1 = sb + (Q[sb + (p0 ^ 1u)] & smask);
            Wd[j] = g0 | (j << 16);
            Wd[j + 1] = g1 | ((j + 1u) << 16);
        }
        __syncthreads();

        // a3: at most logS-1 passes; the last one only for even outputs.  A pass
        // that changes no word has reached the fixed point (every successor's
        // window then spans its whole cycle), and in-place updates usually get
        // there early.
        for (int r = 1; r < logS - 1; ++r) {
            int changed = 0;
            for (int j = tid; j < M; j += T) {
                uint32_t w = Wd[j];
                uint32_t v = Wd[w & 0xFFFFu];
                uint32_t hw = w & 0xFFFF0000u, hv = v & 0xFFFF0000u;
                uint32_t nw = (hw < hv ? hw : hv) | (v & 0xFFFFu);
                changed |= (nw != w);
                Wd[j] = nw;
            }
            if (!__syncthreads_or(changed)) break;
        }
        // last pass + a4 + output side of a5
        for (int t = tid; t < kPairsPadded; t += T) {
            uint32_t c = 0;
            if (t < C::kPairs) {
                uint32_t w = Wd[2 * t];
                uint32_t v = Wd[w & 0xFFFFu];
                uint32_t mn = (w >> 16) < (v >> 16) ? (w >> 16) : (v >> 16);
                c = mn & 1u;
            }
            uint32_t word = __ballot_sync(0xFFFFFFFFu, c);
            if (lane == 0) {
                cw[t >> 5] = word;
                my_bits[size_t(2 * n - 2 - level) * stage_w + (t >> 5)] = word;
            }
        }
        __syncthreads();

        // input side of a5 + a6 (only P' is kept; Q is re-scattered next level)
        const uint32_t H = S >> 1;
        for (int t = tid; t < kPairsPadded; t += T) {
            uint32_t cin = 0;
            if (t < C::kPairs) {
                uint32_t j = 2u * t;
                uint32_t sb = j & ~smask;
                uint32_t tl = (j & smask) >> 1;
                uint32_t c = (cw[t >> 5] >> (t & 31)) & 1u;
                Pb[sb + c * H + tl] = uint16_t((Pa[j] & smask) >> 1);
                Pb[sb + (1u - c) * H + tl] = uint16_t((Pa[j + 1] & smask) >> 1);
                uint32_t q0 = Q[j] & smask;
                uint32_t o = sb + q0;
                cin = ((cw[o >> 6] >> ((o >> 1) & 31)) & 1u) ^ (q0 & 1u);
            }
            uint32_t word = __ballot_sync(0xFFFFFFFFu, cin);
            if (lane == 0) my_bits[size_t(level) * stage_w + (t >> 5)] = word;
        }
        __syncthreads();
        uint16_t *tmp = Pa; Pa = Pb; Pb = tmp;
    }
}

template <int LOGM>
int launch_one(const uint32_t *P, int records, size_t total, uint32_t *bits, int log2n, cudaStream_t s) {
    using C = FusedCfg<LOGM>;
    static bool configured = false;
    if (!configured && C::kSmemBytes > 48 * 1024) {
        BENES_CUDA_TRY(cudaFuncSetAttribute(k_route_fused<LOGM>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            int(C::kSmemBytes)));
        configured = true;
    }
    size_t blocks = total >> LOGM;
    k_route_fused<LOGM><<<unsigned(blocks), C::kThreads, C::kSmemBytes, s>>>(P, records, bits, log2n);
    return launch_status();
}

}  // namespace

int launch_fused(const void *Pv, int records, size_t total, int log2m, uint32_t *bits, int log2n,
                 cudaStream_t s) {
    const uint32_t *P = static_cast<const uint32_t *>(Pv);
    switch (log2m) {
        case 1: return launch_one<1>(P, records, total, bits, log2n, s);
        case 2: return launch_one<2>(P, records, total, bits, log2n, s);
        case 3: return launch_one<3>(P, records, total, bits, log2n, s);
        case 4: return launch_one<4>(P, records, total, bits, log2n, s);
        case 5: return launch_one<5>(P, records, total, bits, log2n, s);
        case 6: return launch_one<6>(P, records, total, bits, log2n, s);
        case 7: return launch_one<7>(P, records, total, bits, log2n, s);
        case 8: return launch_one<8>(P, records, total, bits, log2n, s);
        case 9: return launch_one<9>(P, records, total, bits, log2n, s);
        case 10: return launch_one<10>(P, records, total, bits, log2n, s);
        case 11: return launch_one<11>(P, records, total, bits, log2n, s);
        case 12: return launch_one<12>(P, records, total, bits, log2n, s);
        case 13: return launch_one<13>(P, records, total, bits, log2n, s);
        case 14: return launch_one<14>(P, records, total, bits, log2n, s);
        default: return BENES_ERR_BADARG;
    }
}

}  // namespace benes
