// Fused path: one CTA finishes every remaining level of one block of size
// M = 2^LOGM entirely in shared memory (inverse scatter, loop labelling,
// colouring, stage bits, compaction, middle stage).  It serves both the tail of
// a large permutation (the flat level-(n-LOGM) array holds N/M blocks) and a
// batch of small permutations (N = M, one CTA each).
//
// All indices are local to the CTA's block and 16 bit (M <= 2^15).  A level
// works on sub-blocks of size S; its loops are labelled the same way as at the
// HBM levels, with shared-memory latencies:
//   - sub-blocks of S >= 512: one ruler switch per 8 switches; a walker per
//     ruler output follows g, claims switches with a 16-bit compare-and-swap
//     and stops where it meets the walker from the other end; the contracted
//     list (M/8 words of (next, min), 16 + 16 bit) is labelled by in-place
//     pointer jumping; a switch takes (minimum of its owner & 1) ^ side;
//   - switches nobody claimed (loops without ruler) walk their own cycle;
//   - sub-blocks of S = 256 and 128 are labelled by in-place pointer jumping over
//     all outputs with 16-bit words (next, min: 8 + 8 bit, local to the sub-block),
//     which costs fewer instructions than walks once cycles are this short;
//   - sub-blocks of S <= 64 never leave a warp: it labels a sub-block of 64 in
//     registers (a switch per lane, jumps by shuffle) and both halves of it, down
//     to the middle stage, one output per lane.
// The scratch of the labelling (owners, walk records, list) lives where the
// next level's P' is written afterwards.
#include "common.cuh"

#include <cooperative_groups.h>

BENES_GUARD_TU("route_fused.cu")

namespace benes {
namespace {

constexpr int kFKappa = 3;                     // ruler spacing (log2) inside a CTA
constexpr int kFMinLogS = 9;                   // smallest sub-block that is sampled; below: 8+8-bit pointer jumping
constexpr uint32_t kNone16 = 0xFFFFu;

template <int LOGM>
struct FusedCfg {
    static constexpr int M = 1 << LOGM;
    static constexpr int kPairs = M / 2;
    // 16 entries per thread (at least two warps, at most 1024 threads): with fewer
    // entries per thread the barriers of a level cost more than its work
    // (4096 x 2^12: 1.58 ms with 1024 threads per CTA, 0.88 ms with 256)
    static constexpr int kThreads = M / 16 >= 1024 ? 1024 : (M / 16 >= 64 ? M / 16 : (kPairs >= 64 ? 64 : (kPairs >= 32 ? kPairs : 32)));
    static constexpr int kColourWords = M >= 64 ? M / 64 : 1;
    static constexpr int kRulers = M >> kFKappa;                 // ruler outputs (0 if M < 8)
    // Pa, Pb, Q: uint16[M]; colour words; scratch beyond Pb: see carve-up in the kernel
    static constexpr size_t kScratchBytes = size_t(M) + size_t(kRulers) * (4 + 2 + 4);   // owners, records, list
    static constexpr size_t kExtra = kScratchBytes > size_t(2 * M) ? kScratchBytes - size_t(2 * M) : 0;
    static constexpr size_t kSmemBytes = size_t(M) * 6 + size_t(kColourWords) * 4 + kExtra + 16;
};

__device__ __forceinline__ uint32_t fused_slot(uint32_t group, uint32_t salt) {
    // top bits of a multiplicative hash: two instructions on the walk's critical path
    return ((group + salt * 0x632BE5ABu) * 0x9E3779B1u) >> (32 - kFKappa);
}

// The last five levels of one group of 32 outputs (sub-blocks of 32 and less stay
// inside it): a warp finishes the group in registers, one output per lane, p = the
// lane's entry of the group's sub-permutation, gathers done with shuffles (the
// inverse goes through the group's 32 entries of Q, which only this warp touches).
// grp = index of the group in the CTA's block, g0 = 32 grp.
template <int LOGM>
__device__ __forceinline__ void fused_tail32(uint32_t p, int grp, int g0, int lane, uint16_t *Q, uint32_t *my_bits,
                                             int n, int level0, size_t stage_w) {
    constexpr int M = 1 << LOGM;
    uint16_t *half = reinterpret_cast<uint16_t *>(my_bits);     // 16 switches = one half word
    const size_t half_stride = stage_w * 2;
#pragma unroll
    for (int ls = 5; ls >= 2; --ls) {
        const uint32_t sm_ = (1u << ls) - 1u, sbl = uint32_t(lane) & ~sm_;
        const int lvl = level0 + (LOGM - ls);
        p &= sm_;
        // a1: inverse inside the sub-block
        Q[g0 + sbl + p] = uint16_t(uint32_t(lane) & sm_);
        __syncwarp();
        const uint32_t q = Q[g0 + lane];
        __syncwarp();
        // a2: successor
        const uint32_t p1 = __shfl_xor_sync(0xFFFFFFFFu, p, 1);
        uint32_t nxt = sbl + __shfl_sync(0xFFFFFFFFu, q, int(sbl + (p1 ^ 1u)));
        uint32_t mn = uint32_t(lane);
        // a3: synchronous pointer jumping, ls-1 passes cover cycles of 2^(ls-1)
#pragma unroll
        for (int r = 0; r < ls - 1; ++r) {
            const uint32_t mm = __shfl_sync(0xFFFFFFFFu, mn, int(nxt));
            nxt = __shfl_sync(0xFFFFFFFFu, nxt, int(nxt));
            mn = min(mn, mm);
        }
        const uint32_t c = mn & 1u;                          // a4, every output
        // output side of a5: switch t = lane (< 16) takes the colour of output 2t
        const uint32_t ce = __shfl_sync(0xFFFFFFFFu, c, (lane & 15) * 2);
        const uint32_t outw = __ballot_sync(0xFFFFFFFFu, ce) & 0xFFFFu;
        // input side of a5: colour of the output fed by input 2t
        const uint32_t qe = __shfl_sync(0xFFFFFFFFu, q, (lane & 15) * 2);
        const uint32_t sbe = uint32_t((lane & 15) * 2) & ~sm_;
        const uint32_t ci = __shfl_sync(0xFFFFFFFFu, c, int(sbe + qe));
        const uint32_t inw = __ballot_sync(0xFFFFFFFFu, ci) & 0xFFFFu;
        if (lane == 0) {
            if (M == 32) {
                my_bits[size_t(2 * n - 2 - lvl) * stage_w] = outw;
                my_bits[size_t(lvl) * stage_w] = inw;
            } else {
                half[size_t(2 * n - 2 - lvl) * half_stride + grp] = uint16_t(outw);
                half[size_t(lvl) * half_stride + grp] = uint16_t(inw);
            }
        }
        // a6: position dl of the upper (lower) half takes the colour-0 (1) output of switch tl
        const uint32_t H = 1u << (ls - 1), dl = uint32_t(lane) & sm_;
        const uint32_t tl = dl & (H - 1u), lower = dl >> (ls - 1);
        const uint32_t c2 = __shfl_sync(0xFFFFFFFFu, c, int(sbl + 2u * tl));
        p = __shfl_sync(0xFFFFFFFFu, p, int(sbl + 2u * tl + (c2 ^ lower))) >> 1;
    }
    // a7: middle stage
    const uint32_t pm = __shfl_sync(0xFFFFFFFFu, p, (lane & 15) * 2) & 1u;
    const uint32_t midw = __ballot_sync(0xFFFFFFFFu, pm) & 0xFFFFu;
    if (lane == 0) {
        if (M == 32) my_bits[size_t(n - 1) * stage_w] = midw;
        else half[size_t(n - 1) * half_stride + grp] = uint16_t(midw);
    }
}

// Levels level0 .. level0 + LOGM - 1 of the block of M = 2^LOGM outputs whose
// sub-permutation (16-bit, local) is in Pcur.  Pnext is the other buffer of M
// entries; `tail` = the extra scratch bytes (FusedCfg::kExtra); my_bits = where the
// block's words of a stage start (stage_w words per stage).
template <int LOGM>
__device__ __forceinline__ void fused_levels(uint16_t *Pcur, uint16_t *Pnext, uint16_t *Q, uint32_t *cw,
                                             unsigned char *tail, uint32_t *my_bits, int n, int level0,
                                             size_t stage_w) {
    using C = FusedCfg<LOGM>;
    constexpr int M = C::M;
    constexpr int T = C::kThreads;
    constexpr int R = C::kRulers;
    // pair loops run over a multiple of 32 so that every lane reaches the ballots
    constexpr int kPairsPadded = C::kPairs >= 32 ? C::kPairs : 32;
    const int tid = threadIdx.x;
    const int lane = tid & 31;

#pragma unroll 1
    for (int k = 0; k < LOGM; ++k) {
        const int logS = LOGM - k;
        const uint32_t S = 1u << logS;
        const uint32_t smask = S - 1u;
        const int level = level0 + k;

        if (logS == 6 && LOGM >= 6) {
            // Sub-blocks of 64: a warp takes one, a lane one of its 32 switches (two outputs),
            // and labels it in registers: the (next, min) words of a lane's two outputs share
            // one register (8 + 8 bits each), a jump is one shuffle per output, five passes
            // cover cycles of 32 outputs.  The two half-blocks then stay in the warp for the
            // remaining levels (fused_tail32), so nothing of these six levels but the inverse
            // goes through shared memory and no CTA-wide barrier is needed any more.
            for (int g64 = tid >> 5; g64 < M / 64; g64 += T / 32) {
                const int g0 = g64 * 64;
                const uint32_t pp = *reinterpret_cast<const uint32_t *>(Pcur + g0 + 2 * lane);
                const uint32_t p0 = BENES_GUARD16(pp, 63u), p1 = BENES_GUARD(pp >> 16, 63u);
                // a1: inverse inside the sub-block
                Q[g0 + p0] = uint16_t(2 * lane);
                Q[g0 + p1] = uint16_t(2 * lane + 1);
                __syncwarp();
                const uint32_t q0 = BENES_GUARD(uint32_t(Q[g0 + 2 * lane]), 63u);   // output fed by input 2 lane
                // a2: successors of the lane's two outputs
                const uint32_t nx0 = BENES_GUARD(uint32_t(Q[g0 + (p1 ^ 1u)]), 63u);
                const uint32_t nx1 = BENES_GUARD(uint32_t(Q[g0 + (p0 ^ 1u)]), 63u);
                __syncwarp();                                            // the tails below reuse these entries of Q
                uint32_t w = (nx0 | (uint32_t(2 * lane) << 8)) | ((nx1 | (uint32_t(2 * lane + 1) << 8)) << 16);
                // a3: synchronous pointer jumping
#pragma unroll
                for (int r = 0; r < 5; ++r) {
                    const uint32_t a0 = w & 0xFFu, a1 = (w >> 16) & 0xFFu;
                    const uint32_t v0 = (__shfl_sync(0xFFFFFFFFu, w, int(a0 >> 1)) >> ((a0 & 1u) * 16u)) & 0xFFFFu;
                    const uint32_t v1 = (__shfl_sync(0xFFFFFFFFu, w, int(a1 >> 1)) >> ((a1 & 1u) * 16u)) & 0xFFFFu;
                    const uint32_t n0 = (v0 & 0xFFu) | min(w & 0xFF00u, v0 & 0xFF00u);
                    const uint32_t n1 = (v1 & 0xFFu) | min((w >> 16) & 0xFF00u, v1 & 0xFF00u);
                    w = n0 | (n1 << 16);
                }
                const uint32_t c0 = (w >> 8) & 1u;                       // a4: colour of output 2 lane (2 lane + 1 has the other)
                // a5: output side, switch = lane; input side, the colour of the output fed by input 2 lane
                const uint32_t outw = __ballot_sync(0xFFFFFFFFu, c0);
                const uint32_t ci = (__shfl_sync(0xFFFFFFFFu, c0, int(q0 >> 1)) ^ q0) & 1u;
                const uint32_t inw = __ballot_sync(0xFFFFFFFFu, ci);
                if (lane == 0) {
                    my_bits[size_t(2 * n - 2 - level) * stage_w + g64] = outw;
                    my_bits[size_t(level) * stage_w + g64] = inw;
                }
                // a6: position `lane` of the upper (lower) half takes the colour-0 (1) output of switch `lane`
                fused_tail32<LOGM>((c0 ? p1 : p0) >> 1, 2 * g64, g0, lane, Q, my_bits, n, level0, stage_w);
                fused_tail32<LOGM>((c0 ? p0 : p1) >> 1, 2 * g64 + 1, g0 + 32, lane, Q, my_bits, n, level0, stage_w);
            }
            break;
        }

        if (logS == 5 && LOGM >= 5) {
            for (int grp = tid >> 5; grp < M / 32; grp += T / 32)
                fused_tail32<LOGM>(BENES_GUARD(uint32_t(Pcur[grp * 32 + lane]), 31u), grp, grp * 32, lane, Q, my_bits, n,
                                   level0, stage_w);
            break;
        }

        if (logS == 1) {
            // a7: middle stage, crossed iff output 0 of the 2-block takes input 1
            for (int t = tid; t < kPairsPadded; t += T) {
                uint32_t b = (t < C::kPairs) ? (Pcur[2 * t] & 1u) : 0u;
                uint32_t word = __ballot_sync(0xFFFFFFFFu, b);
                if (lane == 0) my_bits[size_t(n - 1) * stage_w + (t >> 5)] = word;
            }
            break;
        }

        // scratch of this level's labelling: first 2M bytes = the buffer P' goes to, rest = tail
        // owners: uint16 per switch (M bytes); records (own min | far min << 16): uint32 per ruler
        // output; peers: uint16 per ruler output; list words (next | min << 16): uint32 per ruler
        uint16_t *own = Pnext;
        uint32_t *recm = reinterpret_cast<uint32_t *>(reinterpret_cast<unsigned char *>(Pnext) + M);
        uint32_t *list = recm + R;                       // recm and list fill the second M bytes
        uint16_t *peer = (size_t(M) + size_t(R) * 10 <= size_t(2 * M))
                             ? reinterpret_cast<uint16_t *>(list + R)      // still inside that buffer
                             : reinterpret_cast<uint16_t *>(tail);
        const bool sampled = LOGM >= kFMinLogS && logS >= kFMinLogS;

        // a1: block-local inverse; owners reset
        for (int j = tid; j < M; j += T) {
            uint32_t sb = uint32_t(j) & ~smask;
            Q[sb + BENES_GUARD(uint32_t(Pcur[j]), smask)] = uint16_t(uint32_t(j) & smask);
        }
        if (sampled)
            for (int t = tid; t < C::kPairs; t += T) own[t] = uint16_t(kNone16);
        __syncthreads();

        if (sampled) {
            // walks from the ruler outputs; they meet in the middle of a segment
            for (int rho = tid; rho < R; rho += T) {
                const uint32_t group = uint32_t(rho) >> 1, side0 = uint32_t(rho) & 1u;
                const uint32_t t0 = (group << kFKappa) | fused_slot(group, uint32_t(level));
                uint32_t j = 2u * t0 + side0;
                const uint32_t sb = j & ~smask;
                uint32_t fwd = j, part = kNone16, pr = uint32_t(rho) ^ 1u;
                if (!side0) own[t0] = uint16_t(rho << 1);
                uint32_t pp = *reinterpret_cast<const uint32_t *>(Pcur + 2u * t0);
                uint32_t p = BENES_GUARD16(side0 ? pp : (pp >> 16), smask);       // P[j^1]
                uint32_t q = BENES_GUARD(uint32_t(Q[sb + (p ^ 1u)]), smask);
                for (uint32_t hops = 0; hops < S; ++hops) {                // a walk claims < S/2 switches
                    j = sb + q;
                    const uint32_t t = j >> 1, side = j & 1u, g = t >> kFKappa;
                    if ((t & ((1u << kFKappa) - 1u)) == fused_slot(g, uint32_t(level))) {
                        pr = (2u * g + side) ^ 1u;                          // reached the next ruler
                        break;
                    }
                    pp = *reinterpret_cast<const uint32_t *>(Pcur + 2u * t);
                    p = BENES_GUARD16(side ? pp : (pp >> 16), smask);
                    const uint32_t qn = BENES_GUARD(uint32_t(Q[sb + (p ^ 1u)]), smask);
                    // The claim needs no atomic.  Only the two walkers of this segment ever reach
                    // switch t, from opposite ends.  If both find it free at the same moment, both
                    // write (either code is a valid owner: the two stand for mirror cycles and
                    // arrive on opposite sides, so the colour comes out the same), both go on, and
                    // each stops at the next switch, which the other has claimed; minima are taken
                    // over one switch more, which changes nothing.
                    const uint32_t prev = reinterpret_cast<volatile uint16_t *>(own)[t];
                    if (prev == kNone16) reinterpret_cast<volatile uint16_t *>(own)[t] = uint16_t((uint32_t(rho) << 1) | side);
                    if (prev != kNone16) {                                  // met the other walker
                        pr = prev >> 1;
                        break;
                    }
                    fwd = min(fwd, j);
                    part = min(part, j ^ 1u);
                    q = qn;
                }
                recm[rho] = fwd | (part << 16);
                peer[rho] = uint16_t(pr < uint32_t(R > 0 ? R : 1) ? pr : uint32_t(rho));
            }
            __syncthreads();
            // contracted list: next = peer ^ 1, minimum = own side of mine, far side of the peer's
            for (int rho = tid; rho < R; rho += T) {
                const uint32_t pr = peer[rho];
                const uint32_t mn = min(recm[rho] & 0xFFFFu, recm[pr] >> 16);
                list[rho] = (pr ^ 1u) | (mn << 16);
            }
            __syncthreads();
            // in-place pointer jumping over the list; a cycle of the list has at most
            // S/16 words (half of the ruler outputs of its sub-block)
            for (int r = 0; r < logS - kFKappa - 1; ++r) {
                int changed = 0;
                for (int e = tid; e < R; e += T) {
                    uint32_t w = list[e];
                    uint32_t v = list[w & 0xFFFFu];
                    uint32_t hw = w & 0xFFFF0000u, hv = v & 0xFFFF0000u;
                    uint32_t nw = (hw < hv ? hw : hv) | (v & 0xFFFFu);
                    changed |= (nw != w);
                    list[e] = nw;
                }
                if (!__syncthreads_or(changed)) break;
            }
        }

        if (sampled) {
            // a4 + output side of a5: colour of output 2t from its owner
            for (int t = tid; t < kPairsPadded; t += T) {
                uint32_t c = 0;
                if (t < C::kPairs) {
                    const uint32_t code = own[t];
                    if (code != kNone16) {
                        c = ((list[code >> 1] >> 16) ^ code) & 1u;
                    } else {
                        // no owner: walk the g-cycle of output 2t (at most S/2 outputs) from
                        // both ends; g(b ^ 1) ^ 1 is the predecessor of b on the cycle (the
                        // cycle of 2t+1 is its mirror image), and the two chains overlap
                        const uint32_t j0 = 2u * uint32_t(t), sb = j0 & ~smask;
                        uint32_t f = j0, bk = j0, mn = j0;
                        for (uint32_t hops = 0; hops < S; ++hops) {
                            const uint32_t pf = BENES_GUARD(uint32_t(Pcur[f ^ 1u]), smask), pb = BENES_GUARD(uint32_t(Pcur[bk]), smask);
                            const uint32_t qf = BENES_GUARD(uint32_t(Q[sb + (pf ^ 1u)]), smask), qb = BENES_GUARD(uint32_t(Q[sb + (pb ^ 1u)]), smask);
                            f = sb + qf;
                            if (f == bk) break;
                            mn = min(mn, f);
                            bk = (sb + qb) ^ 1u;
                            if (bk == f) break;
                            mn = min(mn, bk);
                        }
                        c = mn & 1u;
                    }
                }
                uint32_t word = __ballot_sync(0xFFFFFFFFu, c);
                if (lane == 0) {
                    cw[t >> 5] = word;
                    my_bits[size_t(2 * n - 2 - level) * stage_w + (t >> 5)] = word;
                }
            }
        } else {
            // a2: successor and initial word (next | min << 8), indices local to the sub-block
            uint16_t *Wd = Pnext;
            for (int t = tid; t < C::kPairs; t += T) {
                const uint32_t j = 2u * t, sb = j & ~smask, jl = j & smask;
                const uint32_t pp = *reinterpret_cast<const uint32_t *>(Pcur + j);
                const uint32_t p0 = BENES_GUARD16(pp, smask), p1 = BENES_GUARD(pp >> 16, smask);
                const uint32_t g0 = BENES_GUARD(uint32_t(Q[sb + (p1 ^ 1u)]), smask), g1 = BENES_GUARD(uint32_t(Q[sb + (p0 ^ 1u)]), smask);
                *reinterpret_cast<uint32_t *>(Wd + j) = (g0 | (jl << 8)) | ((g1 | ((jl + 1u) << 8)) << 16);
            }
            __syncthreads();
            // a3: at most logS-1 passes, in place; the last one only for even outputs
            for (int r = 1; r < logS - 1; ++r) {
                int changed = 0;
                for (int j = tid; j < M; j += T) {
                    const uint32_t sb = uint32_t(j) & ~smask;
                    const uint32_t w = Wd[j];
                    const uint32_t v = Wd[sb + (w & 0xFFu)];
                    const uint32_t nw = min(w & 0xFF00u, v & 0xFF00u) | (v & 0xFFu);
                    changed |= (nw != w);
                    Wd[j] = uint16_t(nw);
                }
                if (!__syncthreads_or(changed)) break;
            }
            for (int t = tid; t < kPairsPadded; t += T) {
                uint32_t c = 0;
                if (t < C::kPairs) {
                    const uint32_t j = 2u * t, sb = j & ~smask;
                    const uint32_t w = Wd[j];
                    const uint32_t v = Wd[sb + (w & 0xFFu)];
                    c = (min(w, v) >> 8) & 1u;
                }
                uint32_t word = __ballot_sync(0xFFFFFFFFu, c);
                if (lane == 0) {
                    cw[t >> 5] = word;
                    my_bits[size_t(2 * n - 2 - level) * stage_w + (t >> 5)] = word;
                }
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
                Pnext[sb + c * H + tl] = uint16_t(BENES_GUARD(uint32_t(Pcur[j]), smask) >> 1);
                Pnext[sb + (1u - c) * H + tl] = uint16_t(BENES_GUARD(uint32_t(Pcur[j + 1]), smask) >> 1);
                uint32_t q0 = BENES_GUARD(uint32_t(Q[j]), smask);
                uint32_t o = sb + q0;
                cin = ((cw[o >> 6] >> ((o >> 1) & 31)) & 1u) ^ (q0 & 1u);
            }
            uint32_t word = __ballot_sync(0xFFFFFFFFu, cin);
            if (lane == 0) my_bits[size_t(level) * stage_w + (t >> 5)] = word;
        }
        __syncthreads();
        uint16_t *tmp = Pcur; Pcur = Pnext; Pnext = tmp;
    }
}

// (a block of 2^15 fills the shared memory of an SM: saying that one CTA per SM is
// enough lets the compiler use all 64 registers a thread of a 1024-thread CTA can
// have; left to itself it settles for 32 and spills inside the walks)
template <int LOGM>
__global__ void __launch_bounds__(FusedCfg<LOGM>::kThreads, (LOGM >= 15 ? 1 : 0))
k_route_fused(const uint32_t *__restrict__ P, int records, uint32_t *__restrict__ bits, int log2n,
              uint32_t block0) {
    using C = FusedCfg<LOGM>;
    constexpr int M = C::M;
    constexpr int T = C::kThreads;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint16_t *Pa = reinterpret_cast<uint16_t *>(smem_raw);
    uint16_t *Q = Pa + M;
    uint32_t *cw = reinterpret_cast<uint32_t *>(Q + M);
    uint16_t *Pb = reinterpret_cast<uint16_t *>(cw + C::kColourWords);   // + scratch tail
    // Pa and Pb swap roles every level, the labelling scratch always overlays
    // the buffer P' is written to next; it starts at that buffer's first byte.
    // Since only Pb is followed by the extra bytes, the scratch that does not
    // fit into 2M bytes is taken from the tail behind Pb in both cases.
    unsigned char *tail = reinterpret_cast<unsigned char *>(Pb + M);

    const int tid = threadIdx.x;
    const int n = log2n;
    const size_t flat0 = size_t(blockIdx.x + block0) << LOGM;    // a launch may cover a range of the blocks
    // where this CTA's words of a stage start
    const size_t N = size_t(1) << n;
    const size_t stage_w = N >= 64 ? N / 64 : 1;
    const size_t perm = flat0 >> n;
    const size_t local_first_switch = (flat0 & (N - 1)) >> 1;
    uint32_t *my_bits = bits + perm * size_t(2 * n - 1) * stage_w + (local_first_switch >> 5);

    // plain array (0), wide switch records {P[2t], P[2t+1], -, -} (1), or packed
    // records P[2t] | P[2t+1] << LOGM | ... (2)
    for (int j = tid; j < M; j += T) {
        size_t f = flat0 + j;
        uint32_t v;
        if (records == 2) {
            const unsigned long long w = reinterpret_cast<const unsigned long long *>(P)[f >> 1];
            v = uint32_t(w >> ((f & 1) ? LOGM : 0));
        } else {
            v = records ? P[((f >> 1) << 2) | (f & 1)] : P[f];
        }
        Pa[j] = uint16_t(records == 2 ? (v & uint32_t(M - 1)) : BENES_GUARD(v, uint32_t(M - 1)));
    }
    __syncthreads();
    fused_levels<LOGM>(Pa, Pb, Q, cw, tail, my_bits, n, n - LOGM, stage_w);
}

// ---- a block of 2^16 outputs in a thread-block cluster of two CTAs ----------------
// The level whose sub-block spans both CTAs runs on distributed shared memory:
// CTA r keeps outputs / inputs [r 2^15, (r+1) 2^15) of P and Q, the owners of
// switches [r 2^14, (r+1) 2^14), the records of ruler outputs [r 2^12, (r+1) 2^12)
// and colour words [512 r, 512 (r+1)), in the same layout the one-CTA kernel uses
// for a block of 2^15; an index picks the CTA with its top bit.  Walkers hop
// between the two shared memories with ordinary loads and a 16-bit
// compare-and-swap on the owner (no multicast, no bulk copies).  The compaction
// sends the upper half-block to CTA 0 and the lower one to CTA 1, after which
// each CTA finishes its half exactly like the one-CTA kernel.  All values of this
// level fit 16 bits (indices < 2^16, owner codes < 2^14, 0xFFFF = none).
constexpr int kClusterLog2M = kFusedLog2M + 1;

template <class Tp>
struct Pair2 {                       // the same array in the two CTAs of the cluster
    Tp *a, *b;
    __device__ __forceinline__ Tp *of(uint32_t rank) const { return rank ? b : a; }
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(FusedCfg<kFusedLog2M>::kThreads)
k_route_cluster2(const uint32_t *__restrict__ P, int records, uint32_t *__restrict__ bits, int log2n,
                 uint32_t block0) {
    constexpr int LOGM = kFusedLog2M;           // per CTA
    using C = FusedCfg<LOGM>;
    constexpr int M = C::M;                      // outputs per CTA
    constexpr int T = C::kThreads;
    constexpr int R = C::kRulers;                // ruler outputs per CTA
    constexpr int LOGR = LOGM - kFKappa;
    constexpr uint32_t kInCta = uint32_t(M) - 1u, kSwInCta = uint32_t(M / 2) - 1u, kRInCta = uint32_t(R) - 1u;
    constexpr uint32_t kWordsPerCta = M / 64;    // colour words per CTA
    constexpr uint32_t kBoth = 2u * uint32_t(M) - 1u;
    static_assert(size_t(M) + size_t(R) * 10 > size_t(2 * M), "peers live in the tail");

    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t rank = cluster.block_rank();

    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint16_t *Pa = reinterpret_cast<uint16_t *>(smem_raw);
    uint16_t *Q = Pa + M;
    uint32_t *cw = reinterpret_cast<uint32_t *>(Q + M);
    uint16_t *Pb = reinterpret_cast<uint16_t *>(cw + C::kColourWords);
    unsigned char *tail = reinterpret_cast<unsigned char *>(Pb + M);
    // scratch of the labelling, over the buffer the next level's P' goes to
    uint16_t *own = Pb;
    uint32_t *recm = reinterpret_cast<uint32_t *>(reinterpret_cast<unsigned char *>(Pb) + M);
    uint32_t *list = recm + R;
    uint16_t *peer = reinterpret_cast<uint16_t *>(tail);

    const Pair2<uint16_t> Pa2{cluster.map_shared_rank(Pa, 0), cluster.map_shared_rank(Pa, 1)};
    const Pair2<uint16_t> Q2{cluster.map_shared_rank(Q, 0), cluster.map_shared_rank(Q, 1)};
    const Pair2<uint16_t> Pb2{cluster.map_shared_rank(Pb, 0), cluster.map_shared_rank(Pb, 1)};
    const Pair2<uint16_t> own2{cluster.map_shared_rank(own, 0), cluster.map_shared_rank(own, 1)};
    const Pair2<uint32_t> recm2{cluster.map_shared_rank(recm, 0), cluster.map_shared_rank(recm, 1)};
    const Pair2<uint32_t> list2{cluster.map_shared_rank(list, 0), cluster.map_shared_rank(list, 1)};
    const Pair2<uint32_t> cw2{cluster.map_shared_rank(cw, 0), cluster.map_shared_rank(cw, 1)};

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int n = log2n;
    const int level = n - kClusterLog2M;         // recursion level of the cluster's block
    const size_t flat0 = size_t((blockIdx.x >> 1) + block0) << kClusterLog2M;
    const size_t N = size_t(1) << n;
    const size_t stage_w = N / 64;
    const size_t perm = flat0 >> n;
    const size_t local_first_switch = (flat0 & (N - 1)) >> 1;
    // this CTA's half of the block's words of a stage
    uint32_t *my_bits = bits + perm * size_t(2 * n - 1) * stage_w + (local_first_switch >> 5) + rank * kWordsPerCta;

    for (int j = tid; j < M; j += T) {
        const size_t f = flat0 + rank * uint32_t(M) + j;
        uint32_t v;
        if (records == 2) {
            const unsigned long long w = reinterpret_cast<const unsigned long long *>(P)[f >> 1];
            v = uint32_t(w >> ((f & 1) ? kClusterLog2M : 0));
        } else {
            v = records ? P[((f >> 1) << 2) | (f & 1)] : P[f];
        }
        Pa[j] = uint16_t(records == 2 ? (v & kBoth) : BENES_GUARD(v, kBoth));
    }
    for (int t = tid; t < M / 2; t += T) own[t] = uint16_t(kNone16);
    cluster.sync();           // both CTAs are running (and loaded) before either touches the other's memory
    // a1: the inverse goes to the CTA that keeps that input
    for (int j = tid; j < M; j += T) {
        const uint32_t v = Pa[j];
        Q2.of(v >> LOGM)[v & kInCta] = uint16_t(rank * uint32_t(M) + j);
    }
    cluster.sync();

    // walks from this CTA's ruler outputs (its ruler switches are its own); about half of
    // the switches and inverse entries a walker reaches are in the other CTA
    for (int rl = tid; rl < R; rl += T) {
        const uint32_t rho = rank * uint32_t(R) + rl;
        const uint32_t group = rho >> 1, side0 = rho & 1u;
        const uint32_t t0 = (group << kFKappa) | fused_slot(group, uint32_t(level));
        uint32_t j = 2u * t0 + side0;
        uint32_t fwd = j, part = kNone16, pr = rho ^ 1u;
        if (!side0) own[t0 & kSwInCta] = uint16_t(rho << 1);
        uint32_t pp = *reinterpret_cast<const uint32_t *>(Pa + 2u * (t0 & kSwInCta));
        uint32_t p = (side0 ? pp : (pp >> 16)) & kBoth;                // P[j^1]
        uint32_t q = Q2.of((p ^ 1u) >> LOGM)[(p ^ 1u) & kInCta];
        for (uint32_t hops = 0; hops <= kBoth; ++hops) {                 // a walk claims < 2^15 switches
            j = q;
            const uint32_t t = j >> 1, side = j & 1u, g = t >> kFKappa;
            if ((t & ((1u << kFKappa) - 1u)) == fused_slot(g, uint32_t(level))) {
                pr = (2u * g + side) ^ 1u;                               // reached the next ruler
                break;
            }
            const uint32_t c = t >> (LOGM - 1), tl = t & kSwInCta;
            pp = *reinterpret_cast<const uint32_t *>(Pa2.of(c) + 2u * tl);
            p = (side ? pp : (pp >> 16)) & kBoth;
            const uint32_t qn = Q2.of((p ^ 1u) >> LOGM)[(p ^ 1u) & kInCta];
            const uint32_t prev = atomicCAS(reinterpret_cast<unsigned short *>(own2.of(c) + tl),
                                            static_cast<unsigned short>(kNone16),
                                            static_cast<unsigned short>((rho << 1) | side));
            if (prev != kNone16) {                                       // met the other walker
                pr = prev >> 1;
                break;
            }
            fwd = min(fwd, j);
            part = min(part, j ^ 1u);
            q = qn;
        }
        recm[rl] = fwd | (part << 16);
        peer[rl] = uint16_t(pr < 2u * uint32_t(R) ? pr : rho);
    }
    cluster.sync();
    // contracted list: next = peer ^ 1, minimum = own side of mine, far side of the peer's
    for (int rl = tid; rl < R; rl += T) {
        const uint32_t pr = peer[rl];
        const uint32_t mn = min(recm[rl] & 0xFFFFu, recm2.of(pr >> LOGR)[pr & kRInCta] >> 16);
        list[rl] = (pr ^ 1u) | (mn << 16);
    }
    cluster.sync();
    // in-place pointer jumping; a cycle of the list has at most 2^12 words (half of the ruler outputs)
    for (int r = 0; r < kClusterLog2M - kFKappa - 1; ++r) {
        for (int e = tid; e < R; e += T) {
            const uint32_t w = list[e], nx = w & 0xFFFFu;
            const uint32_t v = list2.of((nx >> LOGR) & 1u)[nx & kRInCta];
            const uint32_t hw = w & 0xFFFF0000u, hv = v & 0xFFFF0000u;
            list[e] = (hw < hv ? hw : hv) | (v & 0xFFFFu);
        }
        cluster.sync();
    }
    // a4 + output side of a5 for this CTA's switches
    for (int tl = tid; tl < M / 2; tl += T) {
        uint32_t c;
        const uint32_t code = own[tl];
        if (code != kNone16) {
            const uint32_t rr = code >> 1;
            c = ((list2.of((rr >> LOGR) & 1u)[rr & kRInCta] >> 16) ^ code) & 1u;
        } else {
            // loop without ruler: walk the cycle of output 2t from both ends
            const uint32_t j0 = 2u * (rank * uint32_t(M / 2) + tl);
            uint32_t f = j0, bk = j0, mn = j0;
            for (uint32_t hops = 0; hops <= kBoth; ++hops) {
                const uint32_t pf = Pa2.of((f ^ 1u) >> LOGM)[(f ^ 1u) & kInCta], pb = Pa2.of(bk >> LOGM)[bk & kInCta];
                const uint32_t qf = Q2.of((pf ^ 1u) >> LOGM)[(pf ^ 1u) & kInCta];
                const uint32_t qb = Q2.of((pb ^ 1u) >> LOGM)[(pb ^ 1u) & kInCta];
                f = qf;
                if (f == bk) break;
                mn = min(mn, f);
                bk = qb ^ 1u;
                if (bk == f) break;
                mn = min(mn, bk);
            }
            c = mn & 1u;
        }
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, c);
        if (lane == 0) {
            cw[tl >> 5] = word;
            my_bits[size_t(2 * n - 2 - level) * stage_w + (tl >> 5)] = word;
        }
    }
    cluster.sync();
    // input side of a5 + a6: the upper half-block goes to CTA 0, the lower one to CTA 1
    for (int tl = tid; tl < M / 2; tl += T) {
        const uint32_t t = rank * uint32_t(M / 2) + tl;                  // position of the switch in either half-block
        const uint32_t c = (cw[tl >> 5] >> (tl & 31)) & 1u;
        const uint32_t pp = *reinterpret_cast<const uint32_t *>(Pa + 2 * tl);
        Pb2.of(c)[t] = uint16_t((pp & 0xFFFFu) >> 1);
        Pb2.of(c ^ 1u)[t] = uint16_t(pp >> 17);
        const uint32_t q0 = Q[2 * tl];                                   // output fed by input 2t of the block
        const uint32_t wq = q0 >> 6;
        const uint32_t cin = ((cw2.of(wq / kWordsPerCta)[wq % kWordsPerCta] >> ((q0 >> 1) & 31u)) ^ q0) & 1u;
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, cin);
        if (lane == 0) my_bits[size_t(level) * stage_w + (tl >> 5)] = word;
    }
    cluster.sync();
    // from here on nothing leaves the CTA
    fused_levels<LOGM>(Pb, Pa, Q, cw, tail, my_bits, n, level + 1, stage_w);
}

template <int LOGM>
int launch_one(const uint32_t *P, int records, size_t first_block, size_t blocks, uint32_t *bits, int log2n,
               cudaStream_t s) {
    using C = FusedCfg<LOGM>;
    static OncePerDevice configured;
    if (C::kSmemBytes > 48 * 1024) {
        const int rc = configured.run([]() -> int {
            BENES_CUDA_TRY(cudaFuncSetAttribute(k_route_fused<LOGM>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                int(C::kSmemBytes)));
            BENES_CUDA_TRY(cudaFuncSetAttribute(k_route_fused<LOGM>,
                                                cudaFuncAttributePreferredSharedMemoryCarveout,
                                                cudaSharedmemCarveoutMaxShared));
            return BENES_OK;
        });
        if (rc) return rc;
    }
    k_route_fused<LOGM><<<unsigned(blocks), C::kThreads, C::kSmemBytes, s>>>(P, records, bits, log2n,
                                                                             uint32_t(first_block));
    return launch_status();
}

int launch_cluster2(const uint32_t *P, int records, size_t first_block, size_t blocks, uint32_t *bits,
                    int log2n, cudaStream_t s) {
    using C = FusedCfg<kFusedLog2M>;
    static OncePerDevice configured;
    const int rc = configured.run([]() -> int {
        BENES_CUDA_TRY(cudaFuncSetAttribute(k_route_cluster2, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            int(C::kSmemBytes)));
        BENES_CUDA_TRY(cudaFuncSetAttribute(k_route_cluster2, cudaFuncAttributePreferredSharedMemoryCarveout,
                                            cudaSharedmemCarveoutMaxShared));
        return BENES_OK;
    });
    if (rc) return rc;
    // two CTAs per block (the cluster size is part of the kernel)
    k_route_cluster2<<<unsigned(2 * blocks), C::kThreads, C::kSmemBytes, s>>>(P, records, bits, log2n,
                                                                               uint32_t(first_block));
    return launch_status();
}

}  // namespace

int launch_fused(const void *Pv, int records, size_t total, int log2m, uint32_t *bits, int log2n,
                 cudaStream_t s, size_t first_block, size_t blocks) {
    const uint32_t *P = static_cast<const uint32_t *>(Pv);
    if (log2m < 1 || log2m > kClusterLog2M) return BENES_ERR_BADARG;
    if (blocks == 0) blocks = (total >> log2m) - first_block;        // all the rest
    if (first_block + blocks > (total >> log2m)) return BENES_ERR_BADARG;
    if (log2m == kClusterLog2M) return launch_cluster2(P, records, first_block, blocks, bits, log2n, s);
    switch (log2m) {
        case 1: return launch_one<1>(P, records, first_block, blocks, bits, log2n, s);
        case 2: return launch_one<2>(P, records, first_block, blocks, bits, log2n, s);
        case 3: return launch_one<3>(P, records, first_block, blocks, bits, log2n, s);
        case 4: return launch_one<4>(P, records, first_block, blocks, bits, log2n, s);
        case 5: return launch_one<5>(P, records, first_block, blocks, bits, log2n, s);
        case 6: return launch_one<6>(P, records, first_block, blocks, bits, log2n, s);
        case 7: return launch_one<7>(P, records, first_block, blocks, bits, log2n, s);
        case 8: return launch_one<8>(P, records, first_block, blocks, bits, log2n, s);
        case 9: return launch_one<9>(P, records, first_block, blocks, bits, log2n, s);
        case 10: return launch_one<10>(P, records, first_block, blocks, bits, log2n, s);
        case 11: return launch_one<11>(P, records, first_block, blocks, bits, log2n, s);
        case 12: return launch_one<12>(P, records, first_block, blocks, bits, log2n, s);
        case 13: return launch_one<13>(P, records, first_block, blocks, bits, log2n, s);
        case 14: return launch_one<14>(P, records, first_block, blocks, bits, log2n, s);
        case 15: return launch_one<15>(P, records, first_block, blocks, bits, log2n, s);
        default: return BENES_ERR_BADARG;
    }
}

}  // namespace benes
