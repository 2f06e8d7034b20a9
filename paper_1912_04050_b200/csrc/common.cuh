// Shared declarations of the Benes routing library (CUDA side only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include <atomic>
#include <mutex>

#include "benes.h"

namespace benes {

// Largest block finished inside one CTA (log2).  Blocks above it go through
// the per-level HBM kernels.
constexpr int kFusedLog2M = 15;

// Largest list (log2 of its 64-bit words) that one CTA labels in shared memory.
constexpr int kListSmemLog2 = 14;
// Ruler spacing (log2) used when a contracted list is itself sampled.
constexpr int kListKappa = 4;

constexpr uint32_t kUnowned = 0xFFFFFFFFu;

// Every kernel launch of the library goes through this counter.
extern unsigned long long g_launches;

#define BENES_CUDA_TRY(expr)                                   \
    do {                                                       \
        cudaError_t e_ = (expr);                               \
        if (e_ != cudaSuccess) {                               \
            cudaGetLastError(); /* reported here, not by a later launch */ \
            return BENES_ERR_CUDA;                             \
        }                                                      \
    } while (0)

// Result of the launch just issued; a launch error is taken off the runtime's
// error state so that it is reported once, by the call that caused it.
inline int launch_status() {
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? BENES_OK : BENES_ERR_CUDA;
}

// Kernel attributes (opt-in shared memory) belong to a device: a launcher sets
// them the first time it runs on each device of the process.
constexpr int kMaxDevices = 64;
struct OncePerDevice {
    std::mutex mu;
    bool done[kMaxDevices] = {};
    // Runs `configure` (returns a status) the first time on each device; a second
    // thread that arrives meanwhile waits until the attributes are set.
    template <class F>
    int run(F &&configure) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return BENES_ERR_CUDA; }
        std::lock_guard<std::mutex> lk(mu);
        if (done[dev]) return BENES_OK;
        const int rc = configure();
        if (rc == BENES_OK) done[dev] = true;
        return rc;
    }
};

// ---- index guards ---------------------------------------------------------------
// Every index a kernel forms from data is forced into range with a mask or a
// clamp, so that an input that is not a permutation cannot cause an access out
// of bounds.  On a permutation no guard ever changes the value it is given.  A
// build with -DBENES_DEBUG checks exactly that: a guard that has to change its
// value counts the event in a device word of its translation unit and keeps the
// source line (no trap, no printf; the access itself is still the guarded one).
// benes_debug_guard_hits adds the words up.  It stands in for a memory checker
// where none can be run.
//   BENES_GUARD(v, mask)          v & mask, v expected to be <= mask already
//   BENES_GUARD16(v, mask)        the same for the low 16 bits of v (the rest is other data)
//   BENES_GUARD_BELOW(v, n, alt)  v < n ? v : alt, v expected to be < n
#ifdef BENES_DEBUG
static __device__ unsigned int t_guard_words[2];         // hits, line of the last one
__device__ __forceinline__ uint32_t guard_mask(uint32_t v, uint32_t mask, unsigned line) {
    if (v & ~mask) {
        atomicAdd(&t_guard_words[0], 1u);
        t_guard_words[1] = line;
    }
    return v & mask;
}
__device__ __forceinline__ uint32_t guard_below(uint32_t v, uint32_t n, uint32_t alt, unsigned line) {
    if (v >= n) {
        atomicAdd(&t_guard_words[0], 1u);
        t_guard_words[1] = line;
        return alt;
    }
    return v;
}
#define BENES_GUARD(v, mask) ::benes::guard_mask((v), (mask), __LINE__)
#define BENES_GUARD16(v, mask) ::benes::guard_mask((v) & 0xFFFFu, (mask), __LINE__)
#define BENES_GUARD_BELOW(v, n, alt) ::benes::guard_below((v), (n), (alt), __LINE__)
// Every translation unit with kernels registers a reader of its own words.
using GuardReader = int (*)(unsigned int out[2], int clear);
void guard_register(GuardReader reader, const char *file);
#define BENES_GUARD_TU(name)                                                                     \
    namespace {                                                                                  \
    int guard_read_tu(unsigned int out[2], int clear) {                                          \
        if (cudaMemcpyFromSymbol(out, ::benes::t_guard_words, 8) != cudaSuccess) { cudaGetLastError(); return BENES_ERR_CUDA; } \
        if (clear) {                                                                             \
            const unsigned int zero[2] = {0u, 0u};                                               \
            if (cudaMemcpyToSymbol(::benes::t_guard_words, zero, 8) != cudaSuccess) { cudaGetLastError(); return BENES_ERR_CUDA; } \
        }                                                                                        \
        return BENES_OK;                                                                         \
    }                                                                                            \
    struct GuardRegistrar { GuardRegistrar() { ::benes::guard_register(&guard_read_tu, name); } } t_guard_registrar; \
    }
#else
#define BENES_GUARD(v, mask) ((v) & (mask))
#define BENES_GUARD16(v, mask) ((v) & (mask))
#define BENES_GUARD_BELOW(v, n, alt) ((v) < (n) ? (v) : (alt))
#define BENES_GUARD_TU(name)
#endif

// Multiprocessors of the current device (read once per device).
int sm_count();

// Optional event timing of a group of launches of one kind (see benes.h).
enum ProfileKind {
    kInverse = 0, kFullLabel, kSplit, kFused, kApply, kWalk, kCombine, kListWalk, kListLabel,
    kListResolve, kColour, kApplyFused
};
struct ProfileScope {
    ProfileScope(int kind, cudaStream_t s);
    ~ProfileScope();
    int kind_;
    cudaStream_t s_;
    int slot_;
    unsigned long long launches0_;
};

// Where the words of one stage live.  T = flat switch-word index over the
// whole batch (flat switch index >> 5); valid when N >= 64, so that a word
// never straddles two permutations.
struct BitsLayout {
    uint32_t *bits;        // batch x (2n-1) x W words
    int log2n;             // n
    int log2w;             // log2(W), W = N/64
    __host__ __device__ size_t word(int stage, size_t flat_word) const {
        size_t perm = flat_word >> log2w;
        size_t lw = flat_word & ((size_t(1) << log2w) - 1);
        return ((perm * size_t(2 * log2n - 1) + size_t(stage)) << log2w) + lw;
    }
    // the same in 32 bits: a chunk has at most 2^30 elements, i.e. fewer than
    // 2^24 * (2n-1) < 2^30 words
    __host__ __device__ uint32_t word32(int stage, uint32_t flat_word) const {
        const uint32_t perm = flat_word >> log2w;
        const uint32_t lw = flat_word & ((1u << log2w) - 1u);
        return ((perm * uint32_t(2 * log2n - 1) + uint32_t(stage)) << log2w) + lw;
    }
};

// ---- layout of a level in HBM ------------------------------------------------
// A level of the per-level path keeps its sub-permutations as one record per
// output switch t of the flat array, and the inverses Q as a plain uint32
// array (read at random, never claimed).  Two record formats:
//
//   wide   (16 B)  { P[2t], P[2t+1], owner, 0 }, P block-local; owner is
//                  kUnowned until a walk of the sampled labelling claims the
//                  switch with a compare-and-swap.  It sits in the record so
//                  that claiming hits the sector the walker has just fetched.
//   packed (8 B)   P[2t] | P[2t+1] << m | owner << 2m for blocks of 2^m outputs,
//                  owner local to the block, all ones = unowned.  One 64-bit
//                  atomic AND both returns the two P values and claims the
//                  switch, i.e. one memory operation instead of two.  Used
//                  when the owner fits with room for the all-ones value:
//                  2m + (m - kappa + 1) < 64.
//
// Owner = (ruler output that claimed the switch) << 1 | side of arrival.
__host__ __device__ inline bool rec_is_packed(int m, int kappa) {
    return kappa != 0 && 3 * m - kappa + 1 < 64;
}

template <bool PACKED>
__device__ __forceinline__ void rec_read(const void *S, size_t t, int m, uint32_t &p0, uint32_t &p1) {
    if (PACKED) {
        const unsigned long long w = __ldcs(static_cast<const unsigned long long *>(S) + t);
        const uint32_t mask = (1u << m) - 1u;
        p0 = uint32_t(w) & mask;
        p1 = uint32_t(w >> m) & mask;
    } else {
        const uint4 r = __ldcs(static_cast<const uint4 *>(S) + t);
        const uint32_t mask = (1u << m) - 1u;
        p0 = BENES_GUARD(r.x, mask);
        p1 = BENES_GUARD(r.y, mask);
    }
}

// one P value, P[j], read at random
template <bool PACKED>
__device__ __forceinline__ uint32_t rec_p(const void *S, uint32_t j, int m) {
    if (PACKED) {
        const unsigned long long w = __ldg(static_cast<const unsigned long long *>(S) + (j >> 1));
        return uint32_t(w >> ((j & 1u) ? m : 0)) & ((1u << m) - 1u);
    }
    return BENES_GUARD(static_cast<const uint32_t *>(S)[(size_t(j >> 1) << 2) | (j & 1u)], (1u << m) - 1u);
}

// A thread of the streaming kernels owns the two neighbouring switches 2i and
// 2i+1; a warp therefore covers 64 switches = two stage words.  c0 / c1 = the
// bit of the thread's first / second switch.  Lane l fetches the bits of
// switches l and 32 + l (held by threads l/2 and 16 + l/2), so that two
// ballots give the two words.
__device__ __forceinline__ void store_stage_bits64(uint32_t *row_words, uint32_t c0, uint32_t c1) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t both = c0 | (c1 << 1);
    const uint32_t lo = __shfl_sync(0xFFFFFFFFu, both, int(lane >> 1));
    const uint32_t hi = __shfl_sync(0xFFFFFFFFu, both, int(16u + (lane >> 1)));
    const uint32_t w0 = __ballot_sync(0xFFFFFFFFu, (lo >> (lane & 1u)) & 1u);
    const uint32_t w1 = __ballot_sync(0xFFFFFFFFu, (hi >> (lane & 1u)) & 1u);
    if (lane < 2) row_words[lane] = lane ? w1 : w0;
}

// an unowned record of a level with blocks of 2^m outputs
template <bool PACKED>
__device__ __forceinline__ void rec_write(void *S, size_t t, int m, uint32_t p0, uint32_t p1) {
    if (PACKED)
        static_cast<unsigned long long *>(S)[t] =
            (unsigned long long)p0 | ((unsigned long long)p1 << m) | (~0ull << (2 * m));
    else
        static_cast<uint4 *>(S)[t] = make_uint4(p0, p1, kUnowned, 0u);
}

__device__ __forceinline__ unsigned long long make_word(uint32_t nxt, uint32_t mn) {
    return (static_cast<unsigned long long>(mn) << 32) | nxt;
}

// The streaming kernels of a level give every CTA `rounds` consecutive groups of
// `threads` items: as many as keep 8 CTAs per SM busy, at most 16.
inline uint32_t stream_rounds(size_t items, int threads) {
    const size_t r = items / (size_t(threads) * size_t(sm_count()) * 8);
    return uint32_t(r < 1 ? 1 : (r > 16 ? 16 : r));
}

// ---- per-level HBM path (route_levels.cu) ----------------------------------
// total = batch * N flat elements (<= 2^30), all blocks of one level per launch.
// Level 0: S records from the caller's permutation, and Q[P[j]] = j.
int launch_inverse(const uint32_t *perm, void *S, bool packed, uint32_t *Q, size_t total, int log2m,
                   cudaStream_t s);
// The same for total >= 2^kInversePartitionMinLog2 in two streaming passes:
// `pairs` = total x 8 bytes of scratch, `fill` = total >> 18 zero-initialised
// counters (at most kInverseMaxBuckets).
constexpr int kInversePartitionMinLog2 = 22;
constexpr int kInverseMaxBuckets = 4096;
int launch_inverse_partitioned(const uint32_t *perm, void *S, bool packed, uint32_t *Q, void *pairs,
                               uint32_t *fill, size_t total, int log2m, cudaStream_t s);
int launch_inverse_clear(uint32_t *fill, size_t total, cudaStream_t s);
int launch_inverse_partition_piece(const uint32_t *perm, void *S, bool packed, void *pairs, uint32_t *fill,
                                   size_t total, size_t j_first, size_t count, int log2m,
                                   cudaStream_t s);
int launch_inverse_scatter(const void *pairs, uint32_t *Q, size_t total, int log2m, cudaStream_t s);
// Pointer jumping over all outputs (successor build, log2m-2 in-place passes,
// last pass + output-side bits) in ONE cooperative launch; `gate` (may be
// null) is a device word: the kernel returns at once while it is 0.
int launch_full_label(const void *S, bool packed, const uint32_t *Q, unsigned long long *Wd, size_t total,
                      int log2m, BitsLayout L, int out_stage, const uint32_t *gate, cudaStream_t s);
// Input-side bits + next level's inverses; also the next level's records
// (owner reset) if `gate` is null or *gate != 0 (otherwise the colouring kernel
// of the sampled labelling has written them already).
int launch_split(const void *S, bool packed, const uint32_t *Q, void *Sn, bool next_packed, uint32_t *Qn,
                 size_t total, int log2m, BitsLayout L, int in_stage, int out_stage, const uint32_t *gate,
                 cudaStream_t s);

// ---- ruler-sampled loop labelling (route_sampled.cu) --------------------------
struct SampledScratch {
    uint4 *rec;                  // total >> kappa walk records
    uint32_t *ruler_bits;        // parity of every ruler's cycle minimum, one bit each
    unsigned long long *list[5]; // contracted lists: total >> (kappa + 4 i) words
    uint32_t *owner[5];          // owners of the words of list[i] (all kUnowned between uses)
};
size_t sampled_scratch_bytes(size_t total, int kappa);
void sampled_scratch_carve(char *base, size_t total, int kappa, SampledScratch *out);
// Labels every loop of the level, writes the output-side stage and the next
// level's records Sn; raises *gate if some walk exceeded `cap` hops (the level
// must then be relabelled and Sn rewritten).
int sampled_label(void *S, bool packed, const uint32_t *Q, void *Sn, bool next_packed,
                  const SampledScratch &sc, size_t total, int log2m, int kappa, uint32_t salt, uint32_t cap,
                  int walk_pairs, BitsLayout L, int out_stage, uint32_t *gate, cudaStream_t s);
// owner[0] and owner[1] must be all kUnowned before the first sampled_label.
int sampled_scratch_reset(const SampledScratch &sc, size_t total, int kappa, cudaStream_t s);

// ---- fused path (route_fused.cu) -------------------------------------------
// Finishes levels (n - log2m) .. n-1 of every block of size 2^log2m of the flat
// level array (total elements), one CTA per block for log2m <= kFusedLog2M, one
// cluster of two CTAs per block for log2m = kFusedLog2M + 1.
// P is a plain uint32 array if records == 0, wide records if 1, packed records if 2.
// `blocks` blocks from `first_block` on (blocks = 0: all from first_block).
int launch_fused(const void *P, int records, size_t total, int log2m, uint32_t *bits, int log2n,
                 cudaStream_t s, size_t first_block = 0, size_t blocks = 0);

// ---- payload apply (apply.cu) ----------------------------------------------
int launch_apply_stage(const uint32_t *bits, const void *x, void *y, int elem_bytes, int stage,
                       int log2n, size_t batch, cudaStream_t s);

// ---- payload apply, several stages per pass (apply_fused.cu) -----------------
// `scratch` (batch * N elements) is needed when apply_fused_passes(log2n) > 1.
int apply_fused_passes(int log2n);
// With a pipe the first pass runs part by part as the parts of `in` arrive
// (in_ready[i], recorded on another stream), and the parts of `out` the last
// pass has finished are copied to out_host on the side stream.
constexpr int kApplyMaxParts = 8;
struct ApplyHostPipe {
    int parts;                              // divides the number of 2^13-element chunks
    cudaEvent_t in_ready[kApplyMaxParts];
    cudaEvent_t out_done[kApplyMaxParts];
    cudaStream_t side;
    void *out_host;
};
int launch_apply_fused(const uint32_t *bits, const void *in, void *out, void *scratch, int elem_bytes,
                       int log2n, size_t batch, cudaStream_t s, const ApplyHostPipe *pipe = nullptr);
// chunks (CTAs) of the first and of the last pass, 0 if the size is too small to pipe
size_t apply_fused_chunks(int log2n, size_t batch);

// ---- sizes that are not a power of two (pad.cu) ------------------------------
int launch_pad_perm(const uint32_t *src, uint32_t *dst, size_t n_elems, int log2n, size_t batch,
                    cudaStream_t s);
int launch_pad_rows(const void *src, void *dst, int elem_bytes, bool pad, size_t n_elems, int log2n,
                    size_t batch, cudaStream_t s);

int launch_export_butterfly(const uint32_t *bits, uint32_t *out, int log2n, size_t batch, cudaStream_t s);

// ---- validation (route_levels.cu) -------------------------------------------
int launch_validate(const uint32_t *perm, size_t total, int log2n, uint32_t *seen_words,
                    uint32_t *flag, cudaStream_t s);

}  // namespace benes
