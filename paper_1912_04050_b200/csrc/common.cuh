// Shared declarations of the Benes routing library (CUDA side only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "benes.h"

namespace benes {

// Largest block finished inside one CTA (log2).  Blocks above it go through
// the per-level HBM kernels.
constexpr int kFusedLog2M = 13;

// Every kernel launch of the library goes through this counter.
extern unsigned long long g_launches;

#define BENES_CUDA_TRY(expr)                                   \
    do {                                                       \
        cudaError_t e_ = (expr);                               \
        if (e_ != cudaSuccess) return BENES_ERR_CUDA;          \
    } while (0)

inline int launch_status() {
    ++g_launches;
    return cudaPeekAtLastError() == cudaSuccess ? BENES_OK : BENES_ERR_CUDA;
}

// Optional event timing of a group of launches of one kind (see benes.h).
enum ProfileKind { kInverse = 0, kBuild, kJump, kJumpLast, kSplit, kFused, kApply, kWalk, kRulerJump, kColour };
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
};

// ---- per-level HBM path (route_levels.cu) ----------------------------------
// total = batch * N flat elements (<= 2^31), all blocks of one level per launch.
int launch_inverse(const uint32_t *P, uint32_t *Q, size_t total, int log2m, cudaStream_t s);
// `gate` (may be null): device word; the kernel does nothing while it is 0.
int launch_build(const uint32_t *P, const uint32_t *Q, unsigned long long *Wd, size_t total,
                 int log2m, const uint32_t *gate, cudaStream_t s);
int launch_jump(unsigned long long *Wd, size_t total, const uint32_t *gate, cudaStream_t s);
int launch_jump_last(const unsigned long long *Wd, size_t total, BitsLayout L, int out_stage,
                     const uint32_t *gate, cudaStream_t s);
int launch_split(const uint32_t *P, const uint32_t *Q, uint32_t *Pn, uint32_t *Qn, size_t total,
                 int log2m, BitsLayout L, int in_stage, int out_stage, cudaStream_t s);

// ---- ruler-sampled loop labelling (route_sampled.cu) --------------------------
// One ruler switch per group of 2^kappa switches.  owner: total/2 words, preset
// to 0xFFFFFFFF; Wc: total >> kappa contracted words; gate: raised when a walk
// exceeds `cap` hops.
int launch_walk(const uint32_t *P, const uint32_t *Q, uint32_t *owner, unsigned long long *Wc,
                size_t total, int log2m, int kappa, uint32_t salt, uint32_t cap, uint32_t *gate,
                cudaStream_t s);
int launch_colour(const uint32_t *P, const uint32_t *Q, const uint32_t *owner,
                  const unsigned long long *Wc, size_t total, int log2m, BitsLayout L,
                  int out_stage, uint32_t cap, uint32_t *gate, cudaStream_t s);

// ---- fused path (route_fused.cu) -------------------------------------------
// Finishes levels (n - log2m) .. n-1 of every block of size 2^log2m of the flat
// array P (total elements), one CTA per block.  log2m <= kFusedLog2M.
int launch_fused(const uint32_t *P, size_t total, int log2m, uint32_t *bits, int log2n,
                 cudaStream_t s);

// ---- payload apply (apply.cu) ----------------------------------------------
int launch_apply_stage(const uint32_t *bits, const void *x, void *y, int elem_bytes, int stage,
                       int log2n, size_t batch, cudaStream_t s);

// ---- validation (route_levels.cu) -------------------------------------------
int launch_validate(const uint32_t *perm, size_t total, int log2n, uint32_t *seen_words,
                    uint32_t *flag, cudaStream_t s);

}  // namespace benes
