// Payload apply over several stages per pass.
//
// One stage per kernel moves the whole payload through HBM 2n-1 times.  Here a
// CTA keeps 2^13 elements in shared memory and runs many stages on them:
//
//   inner kernel : every block of 2^b elements (b = min(n, 13)) of level n-b
//                  is closed under the 2b-1 innermost stages (input side of
//                  levels n-b .. n-2, middle, output side back up to n-b);
//   outer kernels: k <= 7 consecutive input-side stages of levels l0..l0+k-1
//                  send a contiguous chunk of 2^k * T elements of a level-l0
//                  block to 2^k runs of T consecutive positions (one run per
//                  path through the k switches), so a CTA reads one chunk,
//                  runs k stages and writes 2^k coalesced runs; the
//                  output-side kernel is the mirror image.
//
// In shared memory nothing moves except through the switches.  Element "slot"
// u of a chunk keeps, in its low bits, the outcomes of the stages done so far
// (bit i = 1 if the element left stage l0+i through the lower output) and in
// its high bits the part of its position the remaining stages still act on:
// stage l0+i pairs slots u and u | (1 << i), and a crossed switch swaps them.
// The true position after i stages is
//     (bit-reversed low i bits of u) << (m0 - i)  +  (X0 >> i) + (u >> i),
// m0 = log2 of the level-l0 block size, X0 = offset of the chunk in that
// block; this gives both the switch index of a pair and where a slot is
// written at the end.  The output side reads the same relation backwards.
//
// A thread holds 8 slots (3 slot bits) in registers and runs 3 stages between
// two barriers; the switch words of all stages of the pass are staged in
// shared memory first.
#include "common.cuh"

namespace benes {
namespace {

constexpr int kChunkLog2 = 13;               // elements per CTA
constexpr int kChunk = 1 << kChunkLog2;
constexpr int kRound = 3;                    // stages between barriers
constexpr int kApplyThreads = 512;           // two 8-slot groups per thread and round

// Slot u lives at shared-memory index phys(u): an XOR swizzle of the low bits,
// chosen so that every access pattern of the kernels (consecutive slots; the
// 8-slot groups of each round; columns of the 2^k x T transposition of the
// outer kernels) spreads a warp over all banks.
__device__ __forceinline__ uint32_t phys(uint32_t u) { return u ^ ((u >> 3) & 31u) ^ ((u >> 7) & 31u); }
constexpr int kSmemElems = kChunk;

__device__ __forceinline__ uint32_t rev_bits(uint32_t v, int i) {
    return i ? (__brev(v) >> (32 - i)) : 0u;
}

struct Geometry {
    const uint32_t *bits_p;   // switch words of this permutation
    uint32_t stage_w;         // words per stage
    uint32_t first_sw;        // first switch of the level-l0 block (within the permutation)
    uint32_t x0;              // offset of the chunk inside that block
    int m0;                   // log2 of the level-l0 block size
    int n;
};

// The switch words a CTA needs are copied to shared memory first: kBitWords
// words per stage, the stage's runs (one run per path through the earlier
// stages of the pass) one after the other.  Stage l0+i of a chunk of 2^cbits
// slots has 2^i runs of 2^(cbits-1-i) switches; run c starts at switch
//     first_sw + (c << (m0-1-i)) + (x0 >> (i+1)).
// In the inner kernel (x0 = 0, m0 = cbits) the runs of a stage are contiguous,
// so the stage is one piece of 2^(cbits-1) bits.
constexpr int kBitWords = kChunk / 64;

template <bool OUT>
__device__ __forceinline__ void stage_bits_to_smem(uint32_t *sb, const Geometry &g, int l0, int cbits,
                                                   int i_count, int slot0) {
    const int wbits = cbits > 6 ? cbits - 6 : 0;          // log2(words per stage), at least one word
    for (uint32_t idx = threadIdx.x; idx < uint32_t(i_count) << wbits; idx += blockDim.x) {
        const int i = int(idx >> wbits);
        const uint32_t r = idx & ((1u << wbits) - 1u);
        const int rw = wbits - i;                         // log2(words per run); < 0: runs inside a word
        const int stage = OUT ? (2 * g.n - 2 - (l0 + i)) : (l0 + i);
        const uint32_t *src = g.bits_p + size_t(stage) * g.stage_w;
        uint32_t word;
        if (rw >= 0) {
            const uint32_t c = r >> rw, w = r & ((1u << rw) - 1u);
            const uint32_t sw = g.first_sw + (c << (g.m0 - 1 - i)) + (g.x0 >> (i + 1));
            word = __ldg(src + (sw >> 5) + w);
        } else {
            word = __ldg(src + (g.first_sw >> 5) + r);    // inner kernel only: contiguous
        }
        sb[(slot0 + i) * kBitWords + r] = word;
    }
}

// R stages on slot bits [ilo, ilo + R) of a chunk of 2^cbits slots: ascending
// on the input side, descending on the output side.  sb + (slot_of_i0 + i) *
// kBitWords = words of the stage on slot bit i.  A thread holds the 2^R slots
// u0 | (q << ilo).  The switch of the pair (q, q | 1 << j) of stage i = ilo+j
// is bit  (rev_i(low i bits of the slot) << (cbits-1-i)) + (slot >> (i+1))  of
// the stage: the bits of q below j move the run, the bits above j are
// neighbouring switches of one word.
template <typename E, bool OUT, int R>
__device__ __forceinline__ void run_round(E *sm, const uint32_t *sb, int slot_of_i0, int cbits, int ilo) {
    const uint32_t groups = 1u << (cbits - R);
    // phys is linear over XOR and the slots of a group differ from u0 in bits u0 lacks
    uint32_t dq[1 << R];
#pragma unroll
    for (int q = 0; q < (1 << R); ++q) dq[q] = phys(uint32_t(q) << ilo);
    for (uint32_t gi = threadIdx.x; gi < groups; gi += blockDim.x) {
        const uint32_t u0 = ((gi >> ilo) << (ilo + R)) | (gi & ((1u << ilo) - 1u));
        const uint32_t p0 = phys(u0);
        E e[1 << R];
#pragma unroll
        for (int q = 0; q < (1 << R); ++q) e[q] = sm[p0 ^ dq[q]];
#pragma unroll
        for (int jj = 0; jj < R; ++jj) {
            const int j = OUT ? (R - 1 - jj) : jj;
            const int i = ilo + j, sh = cbits - 1 - i;
            const uint32_t idx0 = (rev_bits(u0 & ((1u << i) - 1u), i) << sh) + (u0 >> (i + 1));
            const uint32_t *words = sb + (slot_of_i0 + i) * kBitWords;
#pragma unroll
            for (int lo = 0; lo < (1 << j); ++lo) {
                uint32_t crev = 0;                        // lo with its j bits reversed
#pragma unroll
                for (int t = 0; t < j; ++t) crev |= ((uint32_t(lo) >> t) & 1u) << (j - 1 - t);
                const uint32_t idx = idx0 + (crev << sh);
                const uint32_t w = words[idx >> 5] >> (idx & 31u);
#pragma unroll
                for (int hi = 0; hi < (1 << (R - 1 - j)); ++hi) {
                    const int q = lo | (hi << (j + 1));
                    const bool cross = (w >> hi) & 1u;
                    const E a = e[q], b = e[q | (1 << j)];
                    e[q] = cross ? b : a;
                    e[q | (1 << j)] = cross ? a : b;
                }
            }
        }
#pragma unroll
        for (int q = 0; q < (1 << R); ++q) sm[p0 ^ dq[q]] = e[q];
    }
}

template <typename E, bool OUT>
__device__ __forceinline__ void run_round_r(E *sm, const uint32_t *sb, int slot_of_i0, int cbits, int ilo,
                                            int r) {
    if (r == 3) run_round<E, OUT, 3>(sm, sb, slot_of_i0, cbits, ilo);
    else if (r == 2) run_round<E, OUT, 2>(sm, sb, slot_of_i0, cbits, ilo);
    else run_round<E, OUT, 1>(sm, sb, slot_of_i0, cbits, ilo);
}

__device__ __forceinline__ Geometry geometry(const uint32_t *bits, size_t flat, int n, int m0) {
    Geometry g;
    const size_t N = size_t(1) << n;
    g.stage_w = n >= 6 ? (1u << (n - 6)) : 1u;
    g.bits_p = bits + (flat >> n) * size_t(2 * n - 1) * g.stage_w;
    const uint32_t local = uint32_t(flat & (N - 1));
    const uint32_t block = local & ~((1u << m0) - 1u);
    g.first_sw = block >> 1;
    g.x0 = local - block;
    g.m0 = m0;
    g.n = n;
    return g;
}

// Inner kernel: all 2b-1 stages of one block of 2^b elements of level n-b.
template <typename E>
__global__ void __launch_bounds__(kApplyThreads, 2)
k_apply_inner(const uint32_t *__restrict__ bits, const E *__restrict__ x, E *__restrict__ y, int n, int b,
              uint32_t cta0) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    E *sm = reinterpret_cast<E *>(smem_raw);
    const size_t flat0 = size_t(blockIdx.x + cta0) << b;
    const Geometry g = geometry(bits, flat0, n, b);
    const int l0 = n - b;
    const uint32_t B = 1u << b;
    // words of the b input-side + middle stages in slots 0..b-1, of the b-1
    // output-side stages in slots b..2b-2 (slot b+i for slot bit i)
    uint32_t *sb = reinterpret_cast<uint32_t *>(sm + kSmemElems);
    stage_bits_to_smem<false>(sb, g, l0, b, b, 0);
    stage_bits_to_smem<true>(sb, g, l0, b, b - 1, b);
    for (uint32_t u = threadIdx.x; u < B; u += blockDim.x) sm[phys(u)] = x[flat0 + u];
    __syncthreads();
    for (int ilo = 0; ilo < b; ilo += kRound) {                     // input side and middle
        run_round_r<E, false>(sm, sb, 0, b, ilo, min(kRound, b - ilo));
        __syncthreads();
    }
    for (int ihi = b - 2; ihi >= 0; ihi -= kRound) {                // output side
        const int r = min(kRound, ihi + 1);
        run_round_r<E, true>(sm, sb, b, b, ihi - r + 1, r);
        __syncthreads();
    }
    for (uint32_t u = threadIdx.x; u < B; u += blockDim.x) y[flat0 + u] = sm[phys(u)];
}

// Outer kernel, input side (OUT = false): stages l0 .. l0+k-1 on a contiguous
// chunk; output side (OUT = true): stages 2n-2-(l0+k-1) .. 2n-2-l0, chunk
// gathered from its 2^k runs and written contiguously.
template <typename E, bool OUT>
__global__ void __launch_bounds__(kApplyThreads, 3)
k_apply_outer(const uint32_t *__restrict__ bits, const E *__restrict__ x, E *__restrict__ y, int n,
              int l0, int k, uint32_t cta0) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    E *sm = reinterpret_cast<E *>(smem_raw);
    const size_t flat0 = size_t(blockIdx.x + cta0) << kChunkLog2;
    const int m0 = n - l0;
    const Geometry g = geometry(bits, flat0, n, m0);
    const int tbits = kChunkLog2 - k;                               // log2 of the run length T
    const uint32_t tmask = (1u << tbits) - 1u;
    // flat start of the level-l0 block, and the first position of the runs inside it
    const size_t block0 = flat0 - g.x0;
    const uint32_t y0 = g.x0 >> k;
    uint32_t *sb = reinterpret_cast<uint32_t *>(sm + kSmemElems);
    stage_bits_to_smem<OUT>(sb, g, l0, kChunkLog2, k, 0);
    if (!OUT) {
        for (uint32_t u = threadIdx.x; u < uint32_t(kChunk); u += blockDim.x) sm[phys(u)] = x[flat0 + u];
    } else {
        for (uint32_t idx = threadIdx.x; idx < uint32_t(kChunk); idx += blockDim.x) {
            const uint32_t c = idx >> tbits, yy = idx & tmask;
            sm[phys((yy << k) | c)] = x[block0 + (size_t(rev_bits(c, k)) << (m0 - k)) + y0 + yy];
        }
    }
    __syncthreads();
    if (!OUT) {
        for (int ilo = 0; ilo < k; ilo += kRound) {
            run_round_r<E, false>(sm, sb, 0, kChunkLog2, ilo, min(kRound, k - ilo));
            __syncthreads();
        }
        for (uint32_t idx = threadIdx.x; idx < uint32_t(kChunk); idx += blockDim.x) {
            const uint32_t c = idx >> tbits, yy = idx & tmask;
            y[block0 + (size_t(rev_bits(c, k)) << (m0 - k)) + y0 + yy] = sm[phys((yy << k) | c)];
        }
    } else {
        for (int ihi = k - 1; ihi >= 0; ihi -= kRound) {
            const int r = min(kRound, ihi + 1);
            run_round_r<E, true>(sm, sb, 0, kChunkLog2, ihi - r + 1, r);
            __syncthreads();
        }
        for (uint32_t u = threadIdx.x; u < uint32_t(kChunk); u += blockDim.x) y[flat0 + u] = sm[phys(u)];
    }
}

template <typename K>
int opt_in_smem(K kernel, size_t bytes) {
    if (bytes > 48 * 1024)
        BENES_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bytes)));
    // room for two CTAs per SM
    BENES_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                        cudaSharedmemCarveoutMaxShared));
    return BENES_OK;
}

template <typename E>
int apply_fused_typed(const uint32_t *bits, const E *in, E *out, E *scratch, int n, size_t batch,
                      cudaStream_t s, const ApplyHostPipe *pipe) {
    const size_t total = batch << n;
    // payload slots + the switch words of up to 2*13-1 stages
    const size_t smem = size_t(kSmemElems) * sizeof(E) + size_t(2 * kChunkLog2 - 1) * kBitWords * 4;
    // an outer pass stages the words of at most 7 stages: three CTAs of 8-byte
    // elements fit one SM, so that one CTA's copies overlap the others' stages
    const size_t smem_outer = size_t(kSmemElems) * sizeof(E) + size_t(7) * kBitWords * 4;
    static OncePerDevice configured;
    {
        const int rc0 = configured.run([&]() -> int {
            int rc;
            if ((rc = opt_in_smem(k_apply_inner<E>, smem))) return rc;
            if ((rc = opt_in_smem(k_apply_outer<E, false>, smem))) return rc;
            return opt_in_smem(k_apply_outer<E, true>, smem);
        });
        if (rc0) return rc0;
    }
    const int b = n < kChunkLog2 ? n : kChunkLog2;
    const int outer = n - b;                       // levels handled by the outer kernels, per side
    const int per_side = (outer + 6) / 7;          // passes per side, at most 7 stages each
    const int passes = 2 * per_side + 1;
    // split `outer` levels evenly over the passes of a side
    int ks[8] = {0};
    for (int i = 0; i < per_side; ++i) ks[i] = outer / per_side + (i < outer % per_side ? 1 : 0);

    // ping-pong between `out` and the scratch buffer so that the last pass lands in `out`
    const E *src = in;
    int pass = 0;
    auto next_dst = [&]() { ++pass; return ((passes - pass) % 2 == 0) ? out : scratch; };
    const unsigned chunks = unsigned(total >> kChunkLog2);
    // A pass is one launch, or `parts` launches over equal ranges of CTAs: the
    // first pass of a piped call waits for each part of `in`, its last pass
    // hands each finished part of `out` to the side stream.  CTA c of the first
    // (last) pass reads (writes) elements [c, c+1) * 2^13 (2^b in the inner pass).
    const int total_passes = passes;
    auto run_pass = [&](int index, unsigned ctas, size_t elems_per_cta, auto &&launch) -> int {
        const bool first = pipe && index == 0, last = pipe && index == total_passes - 1;
        const unsigned parts = (first || last) ? unsigned(pipe->parts) : 1u;
        const unsigned per = ctas / parts;
        for (unsigned p = 0; p < parts; ++p) {
            if (first) BENES_CUDA_TRY(cudaStreamWaitEvent(s, pipe->in_ready[p], 0));
            launch(per, p * per);
            int rc = launch_status();
            if (rc) return rc;
            if (last) {
                BENES_CUDA_TRY(cudaEventRecord(pipe->out_done[p], s));
                BENES_CUDA_TRY(cudaStreamWaitEvent(pipe->side, pipe->out_done[p], 0));
                const size_t off = size_t(p) * per * elems_per_cta * sizeof(E), bytes = size_t(per) * elems_per_cta * sizeof(E);
                BENES_CUDA_TRY(cudaMemcpyAsync(static_cast<char *>(pipe->out_host) + off,
                                               reinterpret_cast<const char *>(out) + off, bytes,
                                               cudaMemcpyDeviceToHost, pipe->side));
            }
        }
        return BENES_OK;
    };
    int l0 = 0, index = 0, rc;
    for (int i = 0; i < per_side; ++i) {
        E *dst = next_dst();
        const int k = ks[i], lvl = l0;
        if ((rc = run_pass(index++, chunks, size_t(kChunk), [&](unsigned ctas, unsigned cta0) {
                 k_apply_outer<E, false><<<ctas, kApplyThreads, smem_outer, s>>>(bits, src, dst, n, lvl, k, cta0);
             })))
            return rc;
        src = dst;
        l0 += ks[i];
    }
    {
        E *dst = next_dst();
        const unsigned blocks = unsigned(total >> b);
        unsigned threads = (1u << b) >> kRound;
        threads = threads < 32u ? 32u : (threads > unsigned(kApplyThreads) ? unsigned(kApplyThreads) : threads);
        if ((rc = run_pass(index++, blocks, size_t(1) << b, [&](unsigned ctas, unsigned cta0) {
                 k_apply_inner<E><<<ctas, threads, smem, s>>>(bits, src, dst, n, b, cta0);
             })))
            return rc;
        src = dst;
    }
    for (int i = per_side - 1; i >= 0; --i) {
        E *dst = next_dst();
        l0 -= ks[i];
        const int k = ks[i], lvl = l0;
        if ((rc = run_pass(index++, chunks, size_t(kChunk), [&](unsigned ctas, unsigned cta0) {
                 k_apply_outer<E, true><<<ctas, kApplyThreads, smem_outer, s>>>(bits, src, dst, n, lvl, k, cta0);
             })))
            return rc;
        src = dst;
    }
    return BENES_OK;
}

}  // namespace

int apply_fused_passes(int log2n) {
    const int b = log2n < kChunkLog2 ? log2n : kChunkLog2;
    return 2 * ((log2n - b + 6) / 7) + 1;
}

size_t apply_fused_chunks(int log2n, size_t batch) {
    return log2n > kChunkLog2 ? (batch << log2n) >> kChunkLog2 : 0;
}

int launch_apply_fused(const uint32_t *bits, const void *in, void *out, void *scratch, int elem_bytes,
                       int log2n, size_t batch, cudaStream_t s, const ApplyHostPipe *pipe) {
    if (pipe && (pipe->parts < 1 || pipe->parts > kApplyMaxParts ||
                 apply_fused_chunks(log2n, batch) % size_t(pipe->parts) != 0 || apply_fused_chunks(log2n, batch) == 0))
        return BENES_ERR_BADARG;
    if (elem_bytes == 4)
        return apply_fused_typed<uint32_t>(bits, static_cast<const uint32_t *>(in),
                                           static_cast<uint32_t *>(out), static_cast<uint32_t *>(scratch),
                                           log2n, batch, s, pipe);
    if (elem_bytes == 8)
        return apply_fused_typed<unsigned long long>(bits, static_cast<const unsigned long long *>(in),
                                                     static_cast<unsigned long long *>(out),
                                                     static_cast<unsigned long long *>(scratch), log2n,
                                                     batch, s, pipe);
    return BENES_ERR_BADARG;
}

}  // namespace benes
