// Per-level kernels of the switch-setting computation for blocks that do not
// fit one CTA's shared memory.  One launch covers all 2^l blocks of a level
// (and all permutations of a batch): arrays are flat, a block of size
// M = 2^log2m owns flat indices [bM, (b+1)M), and P / Q hold block-local
// values.
//
// Words of the pointer-jumping array: one 64-bit word per output,
//   low 32 bits  = nxt (flat index of the current successor),
//   high 32 bits = mn  (smallest flat index seen on the path so far),
// read and written only as whole aligned 8-byte accesses, which is what makes
// the in-place update safe: whenever a word is read it satisfies
// "mn = min over the g-path from j up to, but excluding, nxt".
#include "common.cuh"

namespace benes {

unsigned long long g_launches = 0;

namespace {

constexpr int kThreads = 256;
constexpr int kSMs = 148;

inline int grid_for(size_t work_items, int per_sm = 8) {
    size_t blocks = (work_items + kThreads - 1) / kThreads;
    size_t cap = size_t(kSMs) * per_sm;
    return int(blocks < cap ? (blocks ? blocks : 1) : cap);
}

__device__ __forceinline__ unsigned long long make_word(uint32_t nxt, uint32_t mn) {
    return (static_cast<unsigned long long>(mn) << 32) | nxt;
}

// a1: Q[base + P[j]] = j - base.  Four elements per thread, 16-byte loads.
__global__ void __launch_bounds__(kThreads)
k_inverse(const uint4 *__restrict__ P4, uint32_t *__restrict__ Q, size_t quads, uint32_t mmask) {
    size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < quads; i += stride) {
        uint4 p = __ldg(P4 + i);
        size_t j = i * 4;
        size_t base = j & ~size_t(mmask);
        uint32_t jl = uint32_t(j) & mmask;
        Q[base + (p.x & mmask)] = jl;
        Q[base + (p.y & mmask)] = jl + 1;
        Q[base + (p.z & mmask)] = jl + 2;
        Q[base + (p.w & mmask)] = jl + 3;
    }
}

// a2: successor g(j) = base + Q[base + (P[j^1] ^ 1)], word = (g(j), j).
// Two output switches (four outputs) per thread.
__global__ void __launch_bounds__(kThreads)
k_build(const uint4 *__restrict__ P4, const uint32_t *__restrict__ Q,
        ulonglong2 *__restrict__ W2, size_t quads, uint32_t mmask, const uint32_t *__restrict__ gate) {
    if (gate && *gate == 0u) return;
    size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < quads; i += stride) {
        uint4 p = __ldg(P4 + i);
        size_t j = i * 4;
        size_t base = j & ~size_t(mmask);
        uint32_t b32 = uint32_t(base);
        uint32_t g0 = b32 + (__ldg(Q + base + ((p.y & mmask) ^ 1u)) & mmask);
        uint32_t g1 = b32 + (__ldg(Q + base + ((p.x & mmask) ^ 1u)) & mmask);
        uint32_t g2 = b32 + (__ldg(Q + base + ((p.w & mmask) ^ 1u)) & mmask);
        uint32_t g3 = b32 + (__ldg(Q + base + ((p.z & mmask) ^ 1u)) & mmask);
        uint32_t j32 = uint32_t(j);
        ulonglong2 a, b;
        a.x = make_word(g0, j32);
        a.y = make_word(g1, j32 + 1);
        b.x = make_word(g2, j32 + 2);
        b.y = make_word(g3, j32 + 3);
        W2[2 * i] = a;
        W2[2 * i + 1] = b;
    }
}

__device__ __forceinline__ unsigned long long jump(unsigned long long w, unsigned long long t) {
    // new nxt = t.nxt, new mn = min(w.mn, t.mn): compare the high halves.
    unsigned long long hi = (w >> 32) < (t >> 32) ? (w >> 32) : (t >> 32);
    return (hi << 32) | (t & 0xFFFFFFFFull);
}

// a3: one in-place pointer-jumping pass.  Four words per thread: two 16-byte
// loads of the thread's own words, four independent 8-byte gathers.
__global__ void __launch_bounds__(kThreads)
k_jump(unsigned long long *__restrict__ Wd, size_t quads, const uint32_t *__restrict__ gate) {
    if (gate && *gate == 0u) return;
    size_t stride = size_t(gridDim.x) * blockDim.x;
    ulonglong2 *W2 = reinterpret_cast<ulonglong2 *>(Wd);
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < quads; i += stride) {
        ulonglong2 a = __ldcg(W2 + 2 * i);
        ulonglong2 b = __ldcg(W2 + 2 * i + 1);
        unsigned long long t0 = __ldcg(Wd + uint32_t(a.x));
        unsigned long long t1 = __ldcg(Wd + uint32_t(a.y));
        unsigned long long t2 = __ldcg(Wd + uint32_t(b.x));
        unsigned long long t3 = __ldcg(Wd + uint32_t(b.y));
        a.x = jump(a.x, t0);
        a.y = jump(a.y, t1);
        b.x = jump(b.x, t2);
        b.y = jump(b.y, t3);
        __stcg(W2 + 2 * i, a);
        __stcg(W2 + 2 * i + 1, b);
    }
}

// a3 (last pass) + a4 + out-side half of a5: only the even outputs are
// needed; colour = leader & 1 goes straight into the output-side stage word.
__global__ void __launch_bounds__(kThreads)
k_jump_last(const unsigned long long *__restrict__ Wd, size_t switches, BitsLayout L, int out_stage,
            const uint32_t *__restrict__ gate) {
    if (gate && *gate == 0u) return;
    size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t t = size_t(blockIdx.x) * blockDim.x + threadIdx.x; t < switches; t += stride) {
        unsigned long long w = __ldcg(Wd + 2 * t);
        unsigned long long v = __ldcg(Wd + uint32_t(w));
        uint32_t mn = uint32_t(jump(w, v) >> 32);
        uint32_t word = __ballot_sync(0xFFFFFFFFu, mn & 1u);
        if ((threadIdx.x & 31) == 0) L.bits[L.word(out_stage, t >> 5)] = word;
    }
}

// in-side half of a5 + a6: input-side stage word, P' and Q'.
__global__ void __launch_bounds__(kThreads)
k_split(const uint2 *__restrict__ P2, const uint2 *__restrict__ Q2, uint32_t *__restrict__ Pn,
        uint32_t *__restrict__ Qn, size_t switches, uint32_t mmask, BitsLayout L, int in_stage,
        int out_stage) {
    size_t stride = size_t(gridDim.x) * blockDim.x;
    const uint32_t H = (mmask + 1) >> 1;
    for (size_t t = size_t(blockIdx.x) * blockDim.x + threadIdx.x; t < switches; t += stride) {
        size_t base = (2 * t) & ~size_t(mmask);
        uint32_t tl = uint32_t(t - base / 2);
        uint2 p = __ldg(P2 + t);
        uint2 q = __ldg(Q2 + t);
        p.x &= mmask; p.y &= mmask; q.x &= mmask; q.y &= mmask;
        // colour of output 2t
        uint32_t c = (L.bits[L.word(out_stage, t >> 5)] >> (t & 31)) & 1u;
        Pn[base + c * H + tl] = p.x >> 1;
        Pn[base + (1u - c) * H + tl] = p.y >> 1;
        // colour of the output fed by input 2t
        size_t o = base + q.x;
        uint32_t cin = ((L.bits[L.word(out_stage, o >> 6)] >> ((o >> 1) & 31)) & 1u) ^ (q.x & 1u);
        uint32_t word = __ballot_sync(0xFFFFFFFFu, cin);
        if ((threadIdx.x & 31) == 0) L.bits[L.word(in_stage, t >> 5)] = word;
        Qn[base + cin * H + tl] = q.x >> 1;
        Qn[base + (1u - cin) * H + tl] = q.y >> 1;
    }
}

// Marks every value in a bit set; a value out of range or seen twice raises the flag.
__global__ void __launch_bounds__(kThreads)
k_validate(const uint32_t *__restrict__ perm, size_t total, uint32_t nmask,
           uint32_t *__restrict__ seen, uint32_t *__restrict__ flag) {
    size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t j = size_t(blockIdx.x) * blockDim.x + threadIdx.x; j < total; j += stride) {
        uint32_t v = perm[j];
        if (v > nmask) { *flag = 1u; continue; }
        size_t pos = (j & ~size_t(nmask)) + v;
        uint32_t bit = 1u << (pos & 31);
        if (atomicOr(seen + (pos >> 5), bit) & bit) *flag = 1u;
    }
}

}  // namespace

int launch_inverse(const uint32_t *P, uint32_t *Q, size_t total, int log2m, cudaStream_t s) {
    size_t quads = total / 4;
    k_inverse<<<grid_for(quads), kThreads, 0, s>>>(reinterpret_cast<const uint4 *>(P), Q, quads,
                                                   (1u << log2m) - 1u);
    return launch_status();
}

int launch_build(const uint32_t *P, const uint32_t *Q, unsigned long long *Wd, size_t total,
                 int log2m, const uint32_t *gate, cudaStream_t s) {
    size_t quads = total / 4;
    k_build<<<grid_for(quads), kThreads, 0, s>>>(reinterpret_cast<const uint4 *>(P), Q,
                                                 reinterpret_cast<ulonglong2 *>(Wd), quads,
                                                 (1u << log2m) - 1u, gate);
    return launch_status();
}

int launch_jump(unsigned long long *Wd, size_t total, const uint32_t *gate, cudaStream_t s) {
    size_t quads = total / 4;
    k_jump<<<grid_for(quads), kThreads, 0, s>>>(Wd, quads, gate);
    return launch_status();
}

int launch_jump_last(const unsigned long long *Wd, size_t total, BitsLayout L, int out_stage,
                     const uint32_t *gate, cudaStream_t s) {
    size_t switches = total / 2;
    k_jump_last<<<grid_for(switches), kThreads, 0, s>>>(Wd, switches, L, out_stage, gate);
    return launch_status();
}

int launch_split(const uint32_t *P, const uint32_t *Q, uint32_t *Pn, uint32_t *Qn, size_t total,
                 int log2m, BitsLayout L, int in_stage, int out_stage, cudaStream_t s) {
    size_t switches = total / 2;
    k_split<<<grid_for(switches), kThreads, 0, s>>>(reinterpret_cast<const uint2 *>(P),
                                                    reinterpret_cast<const uint2 *>(Q), Pn, Qn,
                                                    switches, (1u << log2m) - 1u, L, in_stage,
                                                    out_stage);
    return launch_status();
}

int launch_validate(const uint32_t *perm, size_t total, int log2n, uint32_t *seen_words,
                    uint32_t *flag, cudaStream_t s) {
    k_validate<<<grid_for(total), kThreads, 0, s>>>(perm, total, (1u << log2n) - 1u, seen_words, flag);
    return launch_status();
}

}  // namespace benes
