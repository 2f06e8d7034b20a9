// Per-level kernels of the switch-setting computation for blocks that do not
// fit one CTA's shared memory.  One launch covers all 2^l blocks of a level
// (and all permutations of a batch): arrays are flat, a block of size
// M = 2^log2m owns flat indices [bM, (b+1)M), and P / Q hold block-local
// values.  P lives in 16-byte switch records (see common.cuh).
//
// This file: the level-0 inverse scatter, the compaction that forms the next
// level, and pointer jumping over ALL outputs (one cooperative kernel), which
// is the labelling when sampling is switched off and the fallback when a walk
// of the sampled labelling gives up.
//
// Words of the pointer-jumping array: one 64-bit word per output,
//   low 32 bits  = nxt (flat index of the current successor),
//   high 32 bits = mn  (smallest flat index seen on the path so far),
// read and written only as whole aligned 8-byte accesses, which is what makes
// the in-place update safe: whenever a word is read it satisfies
// "mn = min over the g-path from j up to, but excluding, nxt".
#include "common.cuh"

#include <cooperative_groups.h>

#include <atomic>

namespace cg = cooperative_groups;

BENES_GUARD_TU("route_levels.cu")

namespace benes {

unsigned long long g_launches = 0;

int sm_count() {
    static std::atomic<int> cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
    int v = cached[dev].load(std::memory_order_relaxed);
    if (v == 0) {
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1) {
            cudaGetLastError();
            v = 148;
        }
        cached[dev].store(v, std::memory_order_relaxed);
    }
    return v;
}

namespace {

constexpr int kThreads = 256;

inline int grid_for(size_t work_items, int per_sm = 8) {
    size_t blocks = (work_items + kThreads - 1) / kThreads;
    size_t cap = size_t(sm_count()) * per_sm;
    return int(blocks < cap ? (blocks ? blocks : 1) : cap);
}

// a1 at level 0: records of two switches per thread (16-byte load of four
// values of the caller's permutation) and Q[base + P[j]] = j - base.
template <bool PACKED>
__global__ void __launch_bounds__(kThreads)
k_inverse(const uint4 *__restrict__ P4, void *__restrict__ S, uint32_t *__restrict__ Q,
          size_t quads, int m) {
    const uint32_t mmask = (1u << m) - 1u;
    size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < quads; i += stride) {
        uint4 p = __ldcs(P4 + i);
        p.x = BENES_GUARD(p.x, mmask); p.y = BENES_GUARD(p.y, mmask); p.z = BENES_GUARD(p.z, mmask); p.w = BENES_GUARD(p.w, mmask);
        size_t j = i * 4;
        size_t base = j & ~size_t(mmask);
        uint32_t jl = uint32_t(j) & mmask;
        rec_write<PACKED>(S, 2 * i, m, p.x, p.y);
        rec_write<PACKED>(S, 2 * i + 1, m, p.z, p.w);
        Q[base + p.x] = jl;
        Q[base + p.y] = jl + 1;
        Q[base + p.z] = jl + 2;
        Q[base + p.w] = jl + 3;
    }
}

// a1 for large inputs, as two streaming passes instead of one pass of random
// 4-byte writes.  Q is cut into buckets of 2^blog consecutive entries.  Pass 1
// reads P in order, writes the switch records and appends (destination,
// source) pairs to the bucket of the destination: a CTA counts its 8192
// elements per bucket in shared memory (the count an element sees is its rank
// among the CTA's elements of that bucket), reserves room in every bucket with
// one global atomic per bucket, sorts its pairs by bucket in shared memory and
// writes them out in that order, so that the pairs of one bucket leave as one
// run of consecutive 8-byte entries (whole sectors instead of 32 scattered
// stores per warp).  A bucket of a permutation receives exactly as many pairs
// as it has entries; for other inputs positions wrap inside the bucket, so
// every access stays in bounds.  Pass 2 reads the pairs bucket by bucket and
// scatters inside the bucket's piece of Q: with buckets of 2^15 entries a CTA
// builds the piece in shared memory and writes it out in order; with buckets
// of 2^18 entries (inputs of more than 2^27 elements, whose 2^15-entry
// buckets would be too many for the counters) the piece stays in L2.
constexpr int kBucketSmemLog2 = 15;
constexpr int kBucketL2Log2 = 18;
constexpr int kPartChunk = 8192;
constexpr int kPartThreads = 1024;

inline int bucket_log2(size_t total) {
    return (total >> kBucketSmemLog2) <= size_t(kInverseMaxBuckets) ? kBucketSmemLog2 : kBucketL2Log2;
}
inline size_t partition_smem(uint32_t buckets) { return size_t(kPartChunk) * 8 + size_t(buckets) * 12; }

template <bool PACKED>
__global__ void __launch_bounds__(kPartThreads, 2)
k_inverse_partition(const uint32_t *__restrict__ P, void *__restrict__ S, uint2 *__restrict__ pairs,
                    uint32_t *__restrict__ fill, uint32_t buckets, int blog, int m, size_t j_first) {
    const uint32_t mmask = (1u << m) - 1u;
    extern __shared__ __align__(8) unsigned char part_smem[];
    uint2 *stage = reinterpret_cast<uint2 *>(part_smem);                  // the CTA's pairs, sorted by bucket
    uint32_t *count = reinterpret_cast<uint32_t *>(stage + kPartChunk);  // per bucket: elements of this CTA
    uint32_t *first = count + buckets;                                    // ... where they start in `stage`
    uint32_t *offset = first + buckets;                                   // ... and in the bucket
    __shared__ uint32_t warp_sum[kPartThreads / 32];
    const uint32_t tid = threadIdx.x, lane = tid & 31u, wid = tid >> 5;
    for (uint32_t b = tid; b < buckets; b += kPartThreads) count[b] = 0u;
    __syncthreads();
    const size_t j0 = j_first + size_t(blockIdx.x) * kPartChunk;
    constexpr int kPer = kPartChunk / kPartThreads;
    uint32_t dest[kPer], rank[kPer];
#pragma unroll
    for (int i = 0; i < kPer; i += 2) {
        // two values = one switch
        const size_t j = j0 + 2 * (size_t(i / 2) * kPartThreads + tid);
        const uint2 p = __ldcs(reinterpret_cast<const uint2 *>(P + j));
        const uint32_t px = BENES_GUARD(p.x, mmask), py = BENES_GUARD(p.y, mmask);
        rec_write<PACKED>(S, j >> 1, m, px, py);
        const uint32_t base = uint32_t(j) & ~mmask;
        dest[i] = base + px;
        dest[i + 1] = base + py;
        rank[i] = atomicAdd(count + (dest[i] >> blog), 1u);
        rank[i + 1] = atomicAdd(count + (dest[i + 1] >> blog), 1u);
    }
    __syncthreads();
    // exclusive prefix sum of the counts: a thread takes `per` consecutive buckets
    const uint32_t per = (buckets + kPartThreads - 1) / kPartThreads;
    const uint32_t b_lo = min(tid * per, buckets), b_hi = min(b_lo + per, buckets);
    uint32_t mine = 0;
    for (uint32_t b = b_lo; b < b_hi; ++b) mine += count[b];
    uint32_t incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= uint32_t(d)) incl += v;
    }
    if (lane == 31) warp_sum[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        const uint32_t w = warp_sum[lane];
        uint32_t wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, wi, d);
            if (lane >= uint32_t(d)) wi += v;
        }
        warp_sum[lane] = wi - w;
    }
    __syncthreads();
    uint32_t run = warp_sum[wid] + incl - mine;
    for (uint32_t b = b_lo; b < b_hi; ++b) {
        const uint32_t c = count[b];
        first[b] = run;
        run += c;
        offset[b] = c ? atomicAdd(fill + b, c) : 0u;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const size_t j = j0 + 2 * (size_t(i / 2) * kPartThreads + tid) + (i & 1);
        stage[first[dest[i] >> blog] + rank[i]] = make_uint2(dest[i], uint32_t(j) & mmask);
    }
    __syncthreads();
    const uint32_t in_bucket = (1u << blog) - 1u;
    for (uint32_t k = tid; k < uint32_t(kPartChunk); k += kPartThreads) {
        const uint2 pr = stage[k];
        const uint32_t b = pr.x >> blog;
        const uint32_t slot = (offset[b] + (k - first[b])) & in_bucket;
        pairs[(size_t(b) << blog) + slot] = pr;
    }
}

// Pass 2, buckets of 2^kBucketSmemLog2 entries: one CTA per bucket.
__global__ void __launch_bounds__(1024)
k_inverse_scatter_smem(const uint2 *__restrict__ pairs, uint32_t *__restrict__ Q, uint32_t mmask) {
    extern __shared__ __align__(16) uint32_t piece[];
    constexpr uint32_t kEntries = 1u << kBucketSmemLog2, kInBucket = kEntries - 1u;
    const size_t b0 = size_t(blockIdx.x) << kBucketSmemLog2;
    // entries no pair names (only possible if the input is not a permutation) read as 0
    for (uint32_t k = threadIdx.x; k < kEntries / 4; k += 1024)
        reinterpret_cast<uint4 *>(piece)[k] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    const uint4 *src = reinterpret_cast<const uint4 *>(pairs + b0);      // two pairs per load
    constexpr int kLoads = int(kEntries / 2 / 1024);                     // all of a thread's loads in flight
    uint4 two[kLoads];
#pragma unroll
    for (int i = 0; i < kLoads; ++i) two[i] = __ldcs(src + threadIdx.x + i * 1024);
#pragma unroll
    for (int i = 0; i < kLoads; ++i) {
        piece[two[i].x & kInBucket] = BENES_GUARD(two[i].y, mmask);
        piece[two[i].z & kInBucket] = BENES_GUARD(two[i].w, mmask);
    }
    // The finished piece leaves as ONE bulk asynchronous copy (shared -> global, 128 KiB, both
    // ends 16-byte aligned: the piece starts the dynamic shared memory, its place in Q is a
    // multiple of 128 KiB) issued by one thread: the copy engine streams it out while the
    // SM's load/store slots stay free for the next CTA's scatter.  The writes above went
    // through the generic proxy, hence the proxy fence before the barrier; the issuing
    // thread waits until the engine has read the piece, so the CTA's shared memory is not
    // handed to another CTA early (a hardware completion, not a flag to spin on).
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t src = uint32_t(__cvta_generic_to_shared(piece));
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                     :: "l"(Q + b0), "r"(src), "r"(uint32_t(kEntries * 4)) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
}

// Pass 2, buckets of 2^kBucketL2Log2 entries.
__global__ void __launch_bounds__(kThreads)
k_inverse_scatter(const uint2 *__restrict__ pairs, uint32_t *__restrict__ Q, size_t total, uint32_t mmask) {
    const size_t i = size_t(blockIdx.x) * kThreads + threadIdx.x;
    if (i >= total) return;
    const uint2 pr = __ldcs(pairs + i);
    // the destination is forced into the bucket this pair sits in
    constexpr uint32_t kInBucket = (1u << kBucketL2Log2) - 1u;
    const size_t d = (i & ~size_t(kInBucket)) | (pr.x & kInBucket);
    Q[d] = BENES_GUARD(pr.y, mmask);
}

__device__ __forceinline__ unsigned long long jump(unsigned long long w, unsigned long long t) {
    // new nxt = t.nxt, new mn = min(w.mn, t.mn): compare the high halves.
    unsigned long long hi = (w >> 32) < (t >> 32) ? (w >> 32) : (t >> 32);
    return (hi << 32) | (t & 0xFFFFFFFFull);
}

// a2 + a3 + a4 + output side of a5 over all outputs of the level, passes
// separated by grid-wide barriers (cooperative launch).
//   build : W[j] = (g(j), j), g(j) = base + Q[base + (P[j^1] ^ 1)]
//   passes: W[j] <- (W[nxt].nxt, min(mn, W[nxt].mn)), in place
//   last  : even outputs only; colour = leader & 1 -> output-side stage word
template <bool PACKED>
__global__ void __launch_bounds__(kThreads)
k_full_label(const void *__restrict__ S, const uint32_t *__restrict__ Q,
             unsigned long long *__restrict__ Wd, size_t total, int m, int passes,
             BitsLayout L, int out_stage, const uint32_t *__restrict__ gate) {
    if (gate && *gate == 0u) return;        // same value for every thread of the grid
    const uint32_t mmask = (1u << m) - 1u;
    cg::grid_group grid = cg::this_grid();
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    const size_t first = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
    ulonglong2 *W2 = reinterpret_cast<ulonglong2 *>(Wd);

    const size_t switches = total / 2;
    for (size_t t = first; t < switches; t += stride) {
        uint32_t p0, p1;
        rec_read<PACKED>(S, t, m, p0, p1);
        size_t j = 2 * t;
        size_t base = j & ~size_t(mmask);
        uint32_t b32 = uint32_t(base);
        uint32_t g0 = b32 + BENES_GUARD(__ldg(Q + base + (p1 ^ 1u)), mmask);
        uint32_t g1 = b32 + BENES_GUARD(__ldg(Q + base + (p0 ^ 1u)), mmask);
        ulonglong2 a;
        a.x = make_word(g0, uint32_t(j));
        a.y = make_word(g1, uint32_t(j) + 1u);
        W2[t] = a;
    }
    grid.sync();

    const size_t quads = total / 4;
    for (int r = 0; r < passes; ++r) {
        for (size_t i = first; i < quads; i += stride) {
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
        grid.sync();
    }

    for (size_t t = first; t < switches; t += stride) {
        unsigned long long w = __ldcg(Wd + 2 * t);
        unsigned long long v = __ldcg(Wd + uint32_t(w));
        uint32_t mn = uint32_t(jump(w, v) >> 32);
        uint32_t word = __ballot_sync(0xFFFFFFFFu, mn & 1u);
        if ((threadIdx.x & 31) == 0) L.bits[L.word(out_stage, t >> 5)] = word;
    }
}

// in-side half of a5 + a6: input-side stage word and Q'.  With `with_records`
// (no sampled labelling, or its gate raised) also the next level's records:
// position tl of the upper half-block takes P[2t or 2t+1] >> 1 of switch tl,
// so the thread that owns switches 2i and 2i+1 holds both values of one record
// of each half-block and stores whole records.
template <bool PACKED, bool NEXT_PACKED>
__global__ void __launch_bounds__(kThreads, 8)
k_split(const void *__restrict__ S, const uint4 *__restrict__ Q4, void *__restrict__ Sn,
        uint32_t *__restrict__ Qn, uint32_t pairs, int m, BitsLayout L, int in_stage,
        int out_stage, const uint32_t *__restrict__ gate, uint32_t rounds) {
    const bool with_records = !gate || *gate != 0u;
    const uint32_t mmask = (1u << m) - 1u;
    // a CTA takes `rounds` consecutive groups of blockDim.x pairs: the colour
    // words it gathers belong to one block of the level for a long time (L1 hits)
    const uint32_t stride = blockDim.x;
    const uint32_t last = min(pairs, (blockIdx.x + 1u) * rounds * stride);
    const uint32_t H = (mmask + 1) >> 1;
    // a thread owns the neighbouring switches t = 2i and t + 1 (inputs 2t .. 2t+3);
    // the inverses of the next round are on their way while this one is split
    // (pairs is a multiple of 32: a warp stays together)
    uint32_t i = blockIdx.x * rounds * stride + threadIdx.x;
    uint4 q = make_uint4(0, 0, 0, 0);
    if (i < last) q = __ldcs(Q4 + i);
    while (i < last) {
        const uint32_t inext = i + stride;
        uint4 qn = make_uint4(0, 0, 0, 0);
        if (inext < last) qn = __ldcs(Q4 + inext);
        const uint32_t t = 2u * i;
        const uint32_t base = (2u * t) & ~mmask;
        const uint32_t tl = t - (base >> 1);
        const uint32_t *colours = L.bits + L.word32(out_stage, (base >> 1) >> 5);   // the block's words of that stage
        if (with_records) {
            uint32_t px0, py0, px1, py1;
            rec_read<PACKED>(S, t, m, px0, py0);
            rec_read<PACKED>(S, t + 1, m, px1, py1);
            // colours of outputs 2t and 2t+2
            const uint32_t cwd = colours[tl >> 5];
            const uint32_t c0 = (cwd >> (tl & 31u)) & 1u, c1 = (cwd >> ((tl + 1u) & 31u)) & 1u;
            const uint32_t r = (base >> 1) + (tl >> 1);
            rec_write<NEXT_PACKED>(Sn, r, m - 1, (c0 ? py0 : px0) >> 1, (c1 ? py1 : px1) >> 1);
            rec_write<NEXT_PACKED>(Sn, r + (H >> 1), m - 1, (c0 ? px0 : py0) >> 1, (c1 ? px1 : py1) >> 1);
        }
        q.x = BENES_GUARD(q.x, mmask); q.y = BENES_GUARD(q.y, mmask); q.z = BENES_GUARD(q.z, mmask); q.w = BENES_GUARD(q.w, mmask);
        // colour of the output fed by input 2t (2t+2): that output's switch bit, flipped for an odd output
        const uint32_t cin0 = ((colours[q.x >> 6] >> ((q.x >> 1) & 31u)) ^ q.x) & 1u;
        const uint32_t cin1 = ((colours[q.z >> 6] >> ((q.z >> 1) & 31u)) ^ q.z) & 1u;
        store_stage_bits64(L.bits + L.word32(in_stage, (t - 2u * (threadIdx.x & 31u)) >> 5), cin0, cin1);
        // positions tl, tl+1 of the two half-blocks
        *reinterpret_cast<uint2 *>(Qn + base + tl) =
            make_uint2((cin0 ? q.y : q.x) >> 1, (cin1 ? q.w : q.z) >> 1);
        *reinterpret_cast<uint2 *>(Qn + base + H + tl) =
            make_uint2((cin0 ? q.x : q.y) >> 1, (cin1 ? q.z : q.w) >> 1);
        q = qn;
        i = inext;
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

// CTAs of k_full_label that are resident together on the current device.
int cooperative_grid(int *out) {
    constexpr int kMaxDev = 64;
    static int cached[kMaxDev] = {};
    int dev = 0;
    BENES_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDev) return BENES_ERR_CUDA;
    if (!cached[dev]) {
        int sms = 0, per_sm = 0, coop = 0;
        BENES_CUDA_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
        if (!coop) return BENES_ERR_CUDA;
        BENES_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        BENES_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_full_label<false>, kThreads, 0));
        int per_sm_packed = 0;
        BENES_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm_packed, k_full_label<true>, kThreads, 0));
        if (per_sm_packed < per_sm) per_sm = per_sm_packed;
        if (sms < 1 || per_sm < 1) return BENES_ERR_CUDA;
        cached[dev] = sms * per_sm;
    }
    *out = cached[dev];
    return BENES_OK;
}

}  // namespace

// Pass 1 over elements [j_first, j_first + count) (a multiple of 8192); `fill`
// must have been cleared before the first piece.  Pass 2 over everything.
int launch_inverse_clear(uint32_t *fill, size_t total, cudaStream_t s) {
    BENES_CUDA_TRY(cudaMemsetAsync(fill, 0, (total >> bucket_log2(total)) * 4, s));
    return BENES_OK;
}

int launch_inverse_partition_piece(const uint32_t *perm, void *S, bool packed, void *pairs, uint32_t *fill,
                                   size_t total, size_t j_first, size_t count, int log2m,
                                   cudaStream_t s) {
    const int blog = bucket_log2(total);
    const uint32_t buckets = uint32_t(total >> blog);
    const unsigned grid = unsigned(count / kPartChunk);
    const size_t smem = partition_smem(buckets);
    static OncePerDevice configured;
    {
        const int rc = configured.run([]() -> int {
            const int most = int(partition_smem(kInverseMaxBuckets));
            BENES_CUDA_TRY(cudaFuncSetAttribute(k_inverse_partition<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most));
            BENES_CUDA_TRY(cudaFuncSetAttribute(k_inverse_partition<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most));
            BENES_CUDA_TRY(cudaFuncSetAttribute(k_inverse_scatter_smem, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                4 << kBucketSmemLog2));
            return BENES_OK;
        });
        if (rc) return rc;
    }
    if (packed)
        k_inverse_partition<true><<<grid, kPartThreads, smem, s>>>(
            perm, S, static_cast<uint2 *>(pairs), fill, buckets, blog, log2m, j_first);
    else
        k_inverse_partition<false><<<grid, kPartThreads, smem, s>>>(
            perm, S, static_cast<uint2 *>(pairs), fill, buckets, blog, log2m, j_first);
    return launch_status();
}

int launch_inverse_scatter(const void *pairs, uint32_t *Q, size_t total, int log2m, cudaStream_t s) {
    if (bucket_log2(total) == kBucketSmemLog2)
        k_inverse_scatter_smem<<<unsigned(total >> kBucketSmemLog2), 1024, 4 << kBucketSmemLog2, s>>>(
            static_cast<const uint2 *>(pairs), Q, (1u << log2m) - 1u);
    else
        k_inverse_scatter<<<unsigned((total + kThreads - 1) / kThreads), kThreads, 0, s>>>(
            static_cast<const uint2 *>(pairs), Q, total, (1u << log2m) - 1u);
    return launch_status();
}

int launch_inverse_partitioned(const uint32_t *perm, void *S, bool packed, uint32_t *Q, void *pairs,
                               uint32_t *fill, size_t total, int log2m, cudaStream_t s) {
    int rc;
    if ((rc = launch_inverse_clear(fill, total, s))) return rc;
    if ((rc = launch_inverse_partition_piece(perm, S, packed, pairs, fill, total, 0, total, log2m, s)))
        return rc;
    return launch_inverse_scatter(pairs, Q, total, log2m, s);
}

int launch_inverse(const uint32_t *perm, void *S, bool packed, uint32_t *Q, size_t total, int log2m,
                   cudaStream_t s) {
    size_t quads = total / 4;
    const uint4 *P4 = reinterpret_cast<const uint4 *>(perm);
    if (packed) k_inverse<true><<<grid_for(quads), kThreads, 0, s>>>(P4, S, Q, quads, log2m);
    else k_inverse<false><<<grid_for(quads), kThreads, 0, s>>>(P4, S, Q, quads, log2m);
    return launch_status();
}

int launch_full_label(const void *S, bool packed, const uint32_t *Q, unsigned long long *Wd, size_t total,
                      int log2m, BitsLayout L, int out_stage, const uint32_t *gate,
                      cudaStream_t s) {
    int grid = 0;
    int rc = cooperative_grid(&grid);
    if (rc) return rc;
    size_t need = (total / 2 + kThreads - 1) / kThreads;
    if (size_t(grid) > need) grid = int(need);
    int passes = log2m - 2;
    void *args[] = {(void *)&S, (void *)&Q, (void *)&Wd, (void *)&total, (void *)&log2m,
                    (void *)&passes, (void *)&L, (void *)&out_stage, (void *)&gate};
    const void *kernel = packed ? (const void *)k_full_label<true> : (const void *)k_full_label<false>;
    if (cudaLaunchCooperativeKernel(kernel, dim3(grid), dim3(kThreads), args, 0, s) != cudaSuccess) {
        cudaGetLastError();
        return BENES_ERR_CUDA;
    }
    return launch_status();
}

int launch_split(const void *S, bool packed, const uint32_t *Q, void *Sn, bool next_packed, uint32_t *Qn,
                 size_t total, int log2m, BitsLayout L, int in_stage, int out_stage, const uint32_t *gate,
                 cudaStream_t s) {
    const uint32_t pairs = uint32_t(total / 4);                  // two switches per thread
    const uint4 *Q4 = reinterpret_cast<const uint4 *>(Q);
    // Colour words are gathered at random from the block's row of the output-side
    // stage (2^(m-1) bits).  Rows of 32 KiB and less stay in L1 whatever the CTAs
    // of an SM work on; for rows of 64 to 256 KiB the CTAs that are resident
    // together (8 per SM) should cover about one block, so that an SM sees one row.
    uint32_t rounds = stream_rounds(pairs, kThreads);
    if (log2m >= 20 && log2m <= 22 && rounds > (1u << (log2m - 20))) rounds = 1u << (log2m - 20);
    const unsigned grid = unsigned((size_t(pairs) + size_t(kThreads) * rounds - 1) / (size_t(kThreads) * rounds));
    if (packed)          // a packed level is followed by packed levels only
        k_split<true, true><<<grid, kThreads, 0, s>>>(S, Q4, Sn, Qn, pairs, log2m, L, in_stage,
                                                       out_stage, gate, rounds);
    else if (next_packed)
        k_split<false, true><<<grid, kThreads, 0, s>>>(S, Q4, Sn, Qn, pairs, log2m, L, in_stage,
                                                        out_stage, gate, rounds);
    else
        k_split<false, false><<<grid, kThreads, 0, s>>>(S, Q4, Sn, Qn, pairs, log2m, L, in_stage,
                                                         out_stage, gate, rounds);
    return launch_status();
}

int launch_validate(const uint32_t *perm, size_t total, int log2n, uint32_t *seen_words,
                    uint32_t *flag, cudaStream_t s) {
    k_validate<<<grid_for(total), kThreads, 0, s>>>(perm, total, (1u << log2n) - 1u, seen_words, flag);
    return launch_status();
}

}  // namespace benes
