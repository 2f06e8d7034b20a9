// extern "C" entry points (declared in include/benes.h), argument checks,
// workspace management and the host-side level loop.
#include "common.cuh"

#include <cstdio>
#include <mutex>
#include <new>
#include <vector>

namespace benes {

#ifdef BENES_DEBUG
namespace {
struct GuardEntry {
    GuardReader read;
    const char *file;
};
std::vector<GuardEntry> &guard_registry() {
    static std::vector<GuardEntry> entries;       // filled by static constructors of the kernel files
    return entries;
}
}  // namespace
void guard_register(GuardReader reader, const char *file) { guard_registry().push_back({reader, file}); }
#endif

namespace {

constexpr size_t kAlign = 256;

struct Workspace {
    void *own = nullptr;       // library-owned buffer
    size_t own_bytes = 0;
    bool pooled = false;       // `own` came from the device's stream-ordered pool
    void *user = nullptr;      // caller-owned buffer (takes precedence)
    size_t user_bytes = 0;
};

Workspace g_ws[kMaxDevices];
std::mutex g_mu;

// Tuning (benes_set_option), written and read under g_mu; an entry point works
// on the copy it took when it was called.
struct Options {
    int kappa = 4;                  // 0: pointer jumping over all outputs; 2..8: one ruler switch per 2^kappa
    int walk_cap = 1 << 14;
    int apply_fused = 1;
    int inverse_partitioned = 1;
    int chunk_log2 = 30;            // flat elements processed together by the per-level path (indices are 32 bit)
    int cluster = 0;                // 1: blocks of 2^16 are finished by clusters of two CTAs
    int walk_pairs = 1;             // two ruler walks per thread: 0 never, 1 where it pays, 2 wherever possible
};
Options g_opt;
constexpr int kMaxLevels = 32;

Options options() {
    std::lock_guard<std::mutex> lk(g_mu);
    return g_opt;
}

inline size_t align_up(size_t v) { return (v + kAlign - 1) & ~(kAlign - 1); }

bool pool_supported(int dev) {
    static int cached[kMaxDevices] = {};           // 0 unknown, 1 yes, 2 no
    if (!cached[dev]) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMemoryPoolsSupported, dev) != cudaSuccess) { cudaGetLastError(); v = 0; }
        cached[dev] = v ? 1 : 2;
    }
    return cached[dev] == 1;
}

// Frees the library-owned buffer of `w` (g_mu held).  Stream-ordered on `s` if it came from the
// pool and a stream is given; otherwise the device is synchronised first.
int drop_own(Workspace &w, int dev, bool have_stream, cudaStream_t s) {
    if (!w.own) return BENES_OK;
    if (w.pooled && have_stream) {
        BENES_CUDA_TRY(cudaFreeAsync(w.own, s));
    } else {
        BENES_CUDA_TRY(cudaDeviceSynchronize());
        if (w.pooled) {
            BENES_CUDA_TRY(cudaFreeAsync(w.own, nullptr));
            BENES_CUDA_TRY(cudaStreamSynchronize(nullptr));
            cudaMemPool_t pool = nullptr;
            if (cudaDeviceGetDefaultMemPool(&pool, dev) == cudaSuccess && pool) cudaMemPoolTrimTo(pool, 0);
            cudaGetLastError();
        } else {
            BENES_CUDA_TRY(cudaFree(w.own));
        }
    }
    w.own = nullptr;
    w.own_bytes = 0;
    w.pooled = false;
    return BENES_OK;
}

// Returns a device scratch buffer of at least `bytes` for work that is enqueued on `s`.  A
// library-owned buffer that is too small is replaced in stream order (cudaFreeAsync +
// cudaMallocAsync on `s`: no device-wide synchronisation; calls that share the workspace are
// ordered by contract, so everything that used the old buffer precedes the free), or, on a
// device without memory pools, after a device synchronisation.
int get_workspace(size_t bytes, void **out, cudaStream_t s) {
    int dev = 0;
    BENES_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BENES_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_mu);
    Workspace &w = g_ws[dev];
    if (w.user) {
        if (bytes > w.user_bytes) return BENES_ERR_NOMEM;
        *out = w.user;
        return BENES_OK;
    }
    if (bytes > w.own_bytes) {
        const bool pool = pool_supported(dev);
        int rc = drop_own(w, dev, pool, s);
        if (rc) return rc;
        const cudaError_t e = pool ? cudaMallocAsync(&w.own, bytes, s) : cudaMalloc(&w.own, bytes);
        if (e != cudaSuccess) {
            cudaGetLastError();
            w.own = nullptr;
            return BENES_ERR_NOMEM;
        }
        w.own_bytes = bytes;
        w.pooled = pool;
    }
    *out = w.own;
    return BENES_OK;
}

inline bool bad_shape(int log2n, int batch) {
    return log2n < 1 || log2n > BENES_MAX_LOG2N || batch < 1;
}

inline size_t stage_words(int log2n) { return log2n >= 6 ? (size_t(1) << (log2n - 6)) : 1; }

// permutations per chunk of the per-level path
inline size_t level_chunk(int log2n, size_t batch, int chunk_log2) {
    size_t per = (size_t(1) << chunk_log2) >> log2n;
    if (per < 1) per = 1;
    return batch < per ? batch : per;
}

// Scratch of the per-level path for T flat elements: two generations of switch
// records (16 B per switch) and of inverses, the 64-bit words of the full
// pointer jumping, the scratch of the sampled labelling, per-level gate flags.
constexpr int kMaxKappa = 8, kMinKappa = 2;
size_t route_ws_bytes(int log2n, size_t batch) {
    if (log2n <= kFusedLog2M) return 0;
    size_t T = level_chunk(log2n, batch, options().chunk_log2) << log2n;
    return 2 * align_up(T * 8) + 2 * align_up(T * 4) + align_up(T * 8) +
           align_up(sampled_scratch_bytes(T, kMinKappa)) + align_up(kMaxLevels * 4) +
           align_up(kInverseMaxBuckets * 4);
}

size_t apply_ws_bytes(int elem_bytes, int log2n, size_t batch) {
    if (log2n < 2) return 0;
    return align_up((batch << log2n) * size_t(elem_bytes));
}

// Host-buffer calls overlap their copies with the computation: the permutation
// arrives in pieces on a side stream (the bucketing pass of level 0 starts on a
// piece as soon as it is there), and the two stages a level has finished are
// copied to the host on the side stream while the next levels run.
constexpr int kMaxPieces = 8;
static_assert(kMaxPieces >= kApplyMaxParts, "the host pipe's events serve the apply parts too");
struct HostPipe {
    uint32_t *bits_host = nullptr;     // finished stages go here (same layout as `bits`)
    cudaStream_t side = nullptr;       // host -> device copies
    cudaStream_t back = nullptr;       // a second stream for device -> host copies (benes_route_apply_host)
    cudaStream_t d2h = nullptr;        // where this call's finished stages leave: `side` or `back`
    cudaEvent_t part_ready[kApplyMaxParts] = {};   // parts of a payload that have arrived
    int pieces = 0;                    // the permutation arrives in this many equal pieces
    cudaEvent_t piece_ready[kMaxPieces] = {};
    cudaEvent_t stage_ready[kMaxLevels] = {};
};

// rows `stage` of every permutation of the chunk, device -> host
int copy_stage_rows(const HostPipe &hp, const uint32_t *bits, int n, size_t batch, int stage, int rows,
                    cudaStream_t st) {
    const size_t w = stage_words(n) * 4, pitch = size_t(2 * n - 1) * w;
    BENES_CUDA_TRY(cudaMemcpy2DAsync(reinterpret_cast<char *>(hp.bits_host) + size_t(stage) * w, pitch,
                                     reinterpret_cast<const char *>(bits) + size_t(stage) * w, pitch,
                                     w * size_t(rows), batch, cudaMemcpyDeviceToHost, st));
    return BENES_OK;
}

// The levels whose blocks exceed the in-CTA size in HBM, then the fused tail.
int route_levels(const uint32_t *perm, int n, size_t batch, uint32_t *bits, char *ws, cudaStream_t s,
                 const Options &opt, const HostPipe *hp = nullptr) {
    const size_t T = batch << n;
    const size_t kFusedSplitWave = size_t(sm_count());   // CTAs of the fused kernel that run together (one per SM)
    void *Sbuf[2];                     // two generations of switch records (wide: 16 B per switch)
    uint32_t *Qbuf[2];
    size_t off = 0;
    Sbuf[0] = ws + off; off += align_up(T * 8);
    Sbuf[1] = ws + off; off += align_up(T * 8);
    Qbuf[0] = reinterpret_cast<uint32_t *>(ws + off); off += align_up(T * 4);
    Qbuf[1] = reinterpret_cast<uint32_t *>(ws + off); off += align_up(T * 4);
    unsigned long long *Wd = reinterpret_cast<unsigned long long *>(ws + off); off += align_up(T * 8);
    char *sampled = ws + off; off += align_up(sampled_scratch_bytes(T, kMinKappa));
    // per level: a gate, raised by a walk that gave up
    uint32_t *gates = reinterpret_cast<uint32_t *>(ws + off); off += align_up(kMaxLevels * 4);
    uint32_t *fill = reinterpret_cast<uint32_t *>(ws + off);
    // Small inputs are bound by the longest walk of a level, not by throughput:
    // closer rulers (shorter walks) pay there although the lists get longer.
    const int kappa = (opt.kappa > 3 && T <= (size_t(1) << 22)) ? 3 : opt.kappa;
    const uint32_t cap = uint32_t(opt.walk_cap);
    SampledScratch sc;
    int rc;
    if (kappa) {
        sampled_scratch_carve(sampled, T, kappa, &sc);
        BENES_CUDA_TRY(cudaMemsetAsync(gates, 0, kMaxLevels * 4, s));
        if ((rc = sampled_scratch_reset(sc, T, kappa, s))) return rc;
    }

    BitsLayout L{bits, n, n - 6};
    {
        ProfileScope ps(kInverse, s);
        // the 64-bit word array is free until the first level is labelled
        // (the bucketed form needs whole buckets, of 2^18 entries at most)
        const bool bucketed = opt.inverse_partitioned && T >= (size_t(1) << kInversePartitionMinLog2) &&
                              (T & ((size_t(1) << 18) - 1)) == 0;
        const int pieces = hp ? hp->pieces : 0;
        const bool pk = rec_is_packed(n, kappa);
        if (bucketed && pieces > 1) {
            if ((rc = launch_inverse_clear(fill, T, s))) return rc;
            const size_t per = T / size_t(pieces);
            for (int i = 0; i < pieces; ++i) {
                BENES_CUDA_TRY(cudaStreamWaitEvent(s, hp->piece_ready[i], 0));
                if ((rc = launch_inverse_partition_piece(perm, Sbuf[0], pk, Wd, fill, T, per * size_t(i),
                                                         per, n, s)))
                    return rc;
            }
            rc = launch_inverse_scatter(Wd, Qbuf[0], T, n, s);
        } else {
            for (int i = 0; i < pieces; ++i) BENES_CUDA_TRY(cudaStreamWaitEvent(s, hp->piece_ready[i], 0));
            rc = bucketed ? launch_inverse_partitioned(perm, Sbuf[0], pk, Qbuf[0], Wd, fill, T, n, s)
                          : launch_inverse(perm, Sbuf[0], pk, Qbuf[0], T, n, s);
        }
        if (rc) return rc;
    }
    // Blocks of 2^15 are finished by one CTA each.  Up to 64 of them would leave
    // more than half of the SMs idle during the longest kernel of the route: then
    // one more level runs in HBM and twice as many CTAs finish blocks of 2^14.
    const int fused_m = opt.cluster ? kFusedLog2M + 1 : (T >> kFusedLog2M) <= 64 ? kFusedLog2M - 1 : kFusedLog2M;
    int cur = 0;
    for (int level = 0; n - level > fused_m; ++level) {
        const int m = n - level;
        const int out_stage = 2 * n - 2 - level;
        void *S = Sbuf[cur];
        uint32_t *Q = Qbuf[cur];
        const bool pk = rec_is_packed(m, kappa), pk_next = rec_is_packed(m - 1, kappa);
        uint32_t *gate = nullptr;
        if (kappa) {
            // ruler-sampled labelling; raises `gate` if a walk had to give up
            gate = gates + level;
            if ((rc = sampled_label(S, pk, Q, Sbuf[cur ^ 1], pk_next, sc, T, m, kappa, uint32_t(level), cap,
                                    opt.walk_pairs, L, out_stage, gate, s)))
                return rc;
        }
        // pointer jumping over all outputs: the whole labelling when sampling is
        // off, otherwise gated (returns at once unless this level's walks gave up)
        {
            ProfileScope ps(kFullLabel, s);
            if ((rc = launch_full_label(S, pk, Q, Wd, T, m, L, out_stage, gate, s))) return rc;
        }
        {
            ProfileScope ps(kSplit, s);
            if ((rc = launch_split(S, pk, Q, Sbuf[cur ^ 1], pk_next, Qbuf[cur ^ 1], T, m, L, level, out_stage, gate, s)))
                return rc;
        }
        cur ^= 1;
        if (hp && hp->bits_host) {
            // stages `level` and `out_stage` are final: send them home behind the computation
            BENES_CUDA_TRY(cudaEventRecord(hp->stage_ready[level], s));
            BENES_CUDA_TRY(cudaStreamWaitEvent(hp->d2h, hp->stage_ready[level], 0));
            if ((rc = copy_stage_rows(*hp, bits, n, batch, level, 1, hp->d2h))) return rc;
            if ((rc = copy_stage_rows(*hp, bits, n, batch, out_stage, 1, hp->d2h))) return rc;
        }
    }
    const int records = rec_is_packed(fused_m, kappa) ? 2 : 1;
    const size_t blocks = T >> fused_m;
    // the stages of the in-CTA levels are one run of rows in the middle
    const int first = n - fused_m, rows = 2 * fused_m - 1;
    if (hp && hp->bits_host && batch == 1 && blocks >= 4 * kFusedSplitWave) {
        // Two launches of whole waves of CTAs (one CTA per SM): the columns the
        // first one has finished go to the host while the second one runs.
        const size_t waves = (blocks + kFusedSplitWave - 1) / kFusedSplitWave;
        const size_t b1 = ((waves + 1) / 2) * kFusedSplitWave;
        {
            ProfileScope ps(kFused, s);
            if ((rc = launch_fused(Sbuf[cur], records, T, fused_m, bits, n, s, 0, b1))) return rc;
        }
        BENES_CUDA_TRY(cudaEventRecord(hp->stage_ready[kMaxLevels - 2], s));
        {
            ProfileScope ps(kFused, s);
            if ((rc = launch_fused(Sbuf[cur], records, T, fused_m, bits, n, s, b1, blocks - b1))) return rc;
        }
        // a block of 2^m outputs owns 2^(m-6) words of every stage
        const size_t w = stage_words(n) * 4, col1 = (b1 << (fused_m - 6)) * 4;
        char *dst = reinterpret_cast<char *>(hp->bits_host) + size_t(first) * w;
        const char *src = reinterpret_cast<const char *>(bits) + size_t(first) * w;
        BENES_CUDA_TRY(cudaStreamWaitEvent(hp->d2h, hp->stage_ready[kMaxLevels - 2], 0));
        BENES_CUDA_TRY(cudaMemcpy2DAsync(dst, w, src, w, col1, size_t(rows), cudaMemcpyDeviceToHost, hp->d2h));
        BENES_CUDA_TRY(cudaEventRecord(hp->stage_ready[kMaxLevels - 3], s));
        BENES_CUDA_TRY(cudaStreamWaitEvent(hp->d2h, hp->stage_ready[kMaxLevels - 3], 0));
        BENES_CUDA_TRY(cudaMemcpy2DAsync(dst + col1, w, src + col1, w, w - col1, size_t(rows),
                                         cudaMemcpyDeviceToHost, hp->d2h));
        return BENES_OK;
    }
    {
        ProfileScope ps(kFused, s);
        if ((rc = launch_fused(Sbuf[cur], records, T, fused_m, bits, n, s))) return rc;
    }
    if (hp && hp->bits_host) {
        if ((rc = copy_stage_rows(*hp, bits, n, batch, first, rows, s))) return rc;
    }
    return BENES_OK;
}

// Side stream and events of the host-buffer calls, one set per device.
int host_pipe_for_current_device(HostPipe **out) {
    static HostPipe pipes[kMaxDevices];
    static bool ready[kMaxDevices] = {};
    int dev = 0;
    BENES_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BENES_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_mu);
    HostPipe &hp = pipes[dev];
    if (!ready[dev]) {
        BENES_CUDA_TRY(cudaStreamCreateWithFlags(&hp.side, cudaStreamNonBlocking));
        BENES_CUDA_TRY(cudaStreamCreateWithFlags(&hp.back, cudaStreamNonBlocking));
        for (cudaEvent_t &e : hp.part_ready) BENES_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        for (cudaEvent_t &e : hp.piece_ready) BENES_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        for (cudaEvent_t &e : hp.stage_ready) BENES_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        ready[dev] = true;
    }
    *out = &hp;
    return BENES_OK;
}

}  // namespace
}  // namespace benes

using namespace benes;

extern "C" {

size_t benes_switch_words(int log2n, int batch) {
    if (bad_shape(log2n, batch)) return 0;
    return size_t(batch) * size_t(2 * log2n - 1) * stage_words(log2n);
}

size_t benes_route_workspace_bytes(int log2n, int batch) {
    if (bad_shape(log2n, batch)) return 0;
    return route_ws_bytes(log2n, size_t(batch));
}

size_t benes_apply_workspace_bytes(int elem_bytes, int log2n, int batch) {
    if (bad_shape(log2n, batch) || (elem_bytes != 4 && elem_bytes != 8)) return 0;
    return apply_ws_bytes(elem_bytes, log2n, size_t(batch));
}

int benes_set_workspace(void *dev_ptr, size_t bytes) {
    if ((dev_ptr == nullptr) != (bytes == 0)) return BENES_ERR_BADARG;
    if (reinterpret_cast<uintptr_t>(dev_ptr) % kAlign) return BENES_ERR_BADARG;
    int dev = 0;
    BENES_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BENES_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_mu);
    g_ws[dev].user = dev_ptr;
    g_ws[dev].user_bytes = bytes;
    return BENES_OK;
}

int benes_release_workspace(void) {
    int dev = 0;
    BENES_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BENES_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_mu);
    return drop_own(g_ws[dev], dev, false, nullptr);
}

// benes_route on a given scratch buffer (`ws` may be null when route_ws_bytes is 0)
static int route_on(const uint32_t *perm, int n, int batch, uint32_t *switch_bits, char *ws, cudaStream_t s,
                    const Options &opt) {
    if (n <= kFusedLog2M) {
        // whole permutations fit one CTA each
        const size_t max_ctas = size_t(1) << 30;
        ProfileScope ps(kFused, s);
        for (size_t b0 = 0; b0 < size_t(batch); b0 += max_ctas) {
            size_t nb = size_t(batch) - b0 < max_ctas ? size_t(batch) - b0 : max_ctas;
            int rc = launch_fused(perm + (b0 << n), 0, nb << n, n,
                                  switch_bits + b0 * size_t(2 * n - 1) * stage_words(n), n, s);
            if (rc) return rc;
        }
        return BENES_OK;
    }
    if (n == kFusedLog2M + 1 && opt.cluster) {
        // whole permutations of 2^16, one cluster of two CTAs each
        ProfileScope ps(kFused, s);
        return launch_fused(perm, 0, size_t(batch) << n, n, switch_bits, n, s);
    }
    const size_t chunk = level_chunk(n, size_t(batch), opt.chunk_log2);
    for (size_t b0 = 0; b0 < size_t(batch); b0 += chunk) {
        size_t nb = size_t(batch) - b0 < chunk ? size_t(batch) - b0 : chunk;
        int rc = route_levels(perm + (b0 << n), n, nb, switch_bits + b0 * size_t(2 * n - 1) * stage_words(n), ws,
                              s, opt);
        if (rc) return rc;
    }
    return BENES_OK;
}

static bool route_needs_ws(int n, const Options &opt) {
    return n > kFusedLog2M && !(n == kFusedLog2M + 1 && opt.cluster);
}

// benes_apply_ex on a given scratch buffer of apply_ws_bytes
static int apply_on(const uint32_t *switch_bits, const void *in, void *out, int elem_bytes, int n, int batch,
                    void *ws, cudaStream_t s, const Options &opt) {
    const int stages = 2 * n - 1;
    if (opt.apply_fused) {
        ProfileScope ps(kApplyFused, s);
        return launch_apply_fused(switch_bits, in, out, ws, elem_bytes, n, size_t(batch), s);
    }
    // one stage per launch: ping-pong between `out` and the scratch buffer so
    // that the last stage lands in `out`
    const void *src = in;
    ProfileScope ps(kApply, s);
    for (int st = 0; st < stages; ++st) {
        void *dst = ((stages - 1 - st) % 2 == 0) ? out : ws;
        int rc = launch_apply_stage(switch_bits, src, dst, elem_bytes, st, n, size_t(batch), s);
        if (rc) return rc;
        src = dst;
    }
    return BENES_OK;
}

int benes_route(const uint32_t *perm, int log2n, int batch, uint32_t *switch_bits,
                benes_stream_t stream) {
    if (!perm || !switch_bits || bad_shape(log2n, batch)) return BENES_ERR_BADARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const Options opt = options();
    void *ws = nullptr;
    if (route_needs_ws(log2n, opt)) {
        int rc = get_workspace(route_ws_bytes(log2n, size_t(batch)), &ws, s);
        if (rc) return rc;
    }
    return route_on(perm, log2n, batch, switch_bits, static_cast<char *>(ws), s, opt);
}

int benes_apply_ex(const uint32_t *switch_bits, const void *in, void *out, int elem_bytes,
                   int log2n, int batch, benes_stream_t stream) {
    if (!switch_bits || !in || !out || in == out || bad_shape(log2n, batch)) return BENES_ERR_BADARG;
    if (elem_bytes != 4 && elem_bytes != 8) return BENES_ERR_BADARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    void *ws = nullptr;
    if (log2n >= 2) {
        int rc = get_workspace(apply_ws_bytes(elem_bytes, log2n, size_t(batch)), &ws, s);
        if (rc) return rc;
    }
    return apply_on(switch_bits, in, out, elem_bytes, log2n, batch, ws, s, options());
}

int benes_apply(const uint32_t *switch_bits, const void *in, void *out, int log2n, int batch,
                benes_stream_t stream) {
    return benes_apply_ex(switch_bits, in, out, 4, log2n, batch, stream);
}

int benes_export_butterfly(const uint32_t *switch_bits, uint32_t *butterfly_bits, int log2n, int batch,
                           benes_stream_t stream) {
    if (!switch_bits || !butterfly_bits || switch_bits == butterfly_bits || bad_shape(log2n, batch))
        return BENES_ERR_BADARG;
    return launch_export_butterfly(switch_bits, butterfly_bits, log2n, size_t(batch),
                                   reinterpret_cast<cudaStream_t>(stream));
}

int benes_padded_log2n(size_t n_elems) {
    if (n_elems < 1 || n_elems > (size_t(1) << BENES_MAX_LOG2N)) return 0;
    int n = 1;
    while ((size_t(1) << n) < n_elems) ++n;
    return n;
}

int benes_route_padded(const uint32_t *perm, size_t n_elems, int batch, uint32_t *switch_bits,
                       benes_stream_t stream) {
    const int n = benes_padded_log2n(n_elems);
    if (!perm || !switch_bits || n == 0 || batch < 1) return BENES_ERR_BADARG;
    if ((size_t(1) << n) == n_elems) return benes_route(perm, n, batch, switch_bits, stream);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t inner = align_up(route_ws_bytes(n, size_t(batch)));
    void *ws = nullptr;
    int rc = get_workspace(inner + align_up((size_t(batch) << n) * 4), &ws, s);
    if (rc) return rc;
    uint32_t *padded = reinterpret_cast<uint32_t *>(static_cast<char *>(ws) + inner);
    if ((rc = launch_pad_perm(perm, padded, n_elems, n, size_t(batch), s))) return rc;
    return benes_route(padded, n, batch, switch_bits, stream);
}

int benes_apply_padded(const uint32_t *switch_bits, const void *in, void *out, int elem_bytes,
                       size_t n_elems, int batch, benes_stream_t stream) {
    const int n = benes_padded_log2n(n_elems);
    if (!switch_bits || !in || !out || in == out || n == 0 || batch < 1) return BENES_ERR_BADARG;
    if (elem_bytes != 4 && elem_bytes != 8) return BENES_ERR_BADARG;
    if ((size_t(1) << n) == n_elems) return benes_apply_ex(switch_bits, in, out, elem_bytes, n, batch, stream);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t inner = align_up(apply_ws_bytes(elem_bytes, n, size_t(batch)));
    const size_t row_bytes = align_up((size_t(batch) << n) * size_t(elem_bytes));
    void *ws = nullptr;
    int rc = get_workspace(inner + 2 * row_bytes, &ws, s);
    if (rc) return rc;
    char *pin = static_cast<char *>(ws) + inner, *pout = pin + row_bytes;
    if ((rc = launch_pad_rows(in, pin, elem_bytes, true, n_elems, n, size_t(batch), s))) return rc;
    if ((rc = benes_apply_ex(switch_bits, pin, pout, elem_bytes, n, batch, stream))) return rc;
    return launch_pad_rows(pout, out, elem_bytes, false, n_elems, n, size_t(batch), s);
}

int benes_route_host(const uint32_t *perm_host, int log2n, int batch, uint32_t *switch_bits_host,
                     benes_stream_t stream) {
    if (!perm_host || !switch_bits_host || bad_shape(log2n, batch)) return BENES_ERR_BADARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t perm_bytes = (size_t(batch) << log2n) * 4;
    const size_t bits_bytes = benes_switch_words(log2n, batch) * 4;
    const size_t inner = route_ws_bytes(log2n, size_t(batch));
    void *ws = nullptr;
    int rc = get_workspace(align_up(inner) + align_up(perm_bytes) + align_up(bits_bytes), &ws, s);
    if (rc) return rc;
    char *base = static_cast<char *>(ws);
    uint32_t *d_perm = reinterpret_cast<uint32_t *>(base + align_up(inner));
    uint32_t *d_bits = reinterpret_cast<uint32_t *>(base + align_up(inner) + align_up(perm_bytes));
    const int n = log2n;
    const Options opt = options();
    if (n > kFusedLog2M && level_chunk(n, size_t(batch), opt.chunk_log2) == size_t(batch)) {
        // one chunk: copies overlapped with the levels (see HostPipe)
        HostPipe *hp = nullptr;
        if ((rc = host_pipe_for_current_device(&hp))) return rc;
        const size_t T = size_t(batch) << n;
        hp->bits_host = switch_bits_host;
        hp->d2h = hp->side;
        hp->pieces = (T >= (size_t(1) << 23)) ? kMaxPieces : 1;
        // the side stream must not touch the workspace before earlier work on `s` is done
        BENES_CUDA_TRY(cudaEventRecord(hp->stage_ready[kMaxLevels - 1], s));
        BENES_CUDA_TRY(cudaStreamWaitEvent(hp->side, hp->stage_ready[kMaxLevels - 1], 0));
        const size_t per = perm_bytes / size_t(hp->pieces);
        for (int i = 0; i < hp->pieces; ++i) {
            BENES_CUDA_TRY(cudaMemcpyAsync(reinterpret_cast<char *>(d_perm) + per * size_t(i),
                                           reinterpret_cast<const char *>(perm_host) + per * size_t(i), per,
                                           cudaMemcpyHostToDevice, hp->side));
            BENES_CUDA_TRY(cudaEventRecord(hp->piece_ready[i], hp->side));
        }
        rc = route_levels(d_perm, n, size_t(batch), d_bits, base, s, opt, hp);
        cudaError_t e1 = cudaStreamSynchronize(hp->side), e2 = cudaStreamSynchronize(s);
        if (rc) return rc;
        return (e1 == cudaSuccess && e2 == cudaSuccess) ? BENES_OK : BENES_ERR_CUDA;
    }
    BENES_CUDA_TRY(cudaMemcpyAsync(d_perm, perm_host, perm_bytes, cudaMemcpyHostToDevice, s));
    rc = benes_route(d_perm, log2n, batch, d_bits, stream);
    if (rc) return rc;
    BENES_CUDA_TRY(cudaMemcpyAsync(switch_bits_host, d_bits, bits_bytes, cudaMemcpyDeviceToHost, s));
    BENES_CUDA_TRY(cudaStreamSynchronize(s));
    return BENES_OK;
}

int benes_apply_host(const uint32_t *switch_bits_host, const void *in_host, void *out_host,
                     int elem_bytes, int log2n, int batch, benes_stream_t stream) {
    if (!switch_bits_host || !in_host || !out_host || bad_shape(log2n, batch)) return BENES_ERR_BADARG;
    if (elem_bytes != 4 && elem_bytes != 8) return BENES_ERR_BADARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t data_bytes = (size_t(batch) << log2n) * size_t(elem_bytes);
    const size_t bits_bytes = benes_switch_words(log2n, batch) * 4;
    const size_t inner = apply_ws_bytes(elem_bytes, log2n, size_t(batch));
    void *ws = nullptr;
    int rc = get_workspace(align_up(inner) + 2 * align_up(data_bytes) + align_up(bits_bytes), &ws, s);
    if (rc) return rc;
    char *base = static_cast<char *>(ws);
    char *d_in = base + align_up(inner);
    char *d_out = d_in + align_up(data_bytes);
    uint32_t *d_bits = reinterpret_cast<uint32_t *>(d_out + align_up(data_bytes));
    BENES_CUDA_TRY(cudaMemcpyAsync(d_bits, switch_bits_host, bits_bytes, cudaMemcpyHostToDevice, s));
    const size_t chunks = apply_fused_chunks(log2n, size_t(batch));
    if (options().apply_fused && data_bytes >= (size_t(1) << 26) && chunks % kApplyMaxParts == 0 && chunks > 0) {
        // The payload arrives in parts on the side stream, behind the switch words:
        // the first pass starts on a part as soon as it is there, and the parts the
        // last pass has finished leave on the side stream while it still runs.
        HostPipe *hp = nullptr;
        if ((rc = host_pipe_for_current_device(&hp))) return rc;
        ApplyHostPipe pipe;
        pipe.parts = kApplyMaxParts;
        pipe.side = hp->side;
        pipe.out_host = out_host;
        // the side stream must not touch the workspace before earlier work on `s` is done
        BENES_CUDA_TRY(cudaEventRecord(hp->stage_ready[kMaxLevels - 1], s));
        BENES_CUDA_TRY(cudaStreamWaitEvent(hp->side, hp->stage_ready[kMaxLevels - 1], 0));
        const size_t per = data_bytes / size_t(pipe.parts);
        for (int i = 0; i < pipe.parts; ++i) {
            pipe.in_ready[i] = hp->piece_ready[i];
            pipe.out_done[i] = hp->stage_ready[i];
            BENES_CUDA_TRY(cudaMemcpyAsync(d_in + per * size_t(i), static_cast<const char *>(in_host) + per * size_t(i),
                                           per, cudaMemcpyHostToDevice, hp->side));
            BENES_CUDA_TRY(cudaEventRecord(hp->piece_ready[i], hp->side));
        }
        {
            ProfileScope ps(kApplyFused, s);
            rc = launch_apply_fused(d_bits, d_in, d_out, base, elem_bytes, log2n, size_t(batch), s, &pipe);
        }
        cudaError_t e1 = cudaStreamSynchronize(s), e2 = cudaStreamSynchronize(hp->side);
        if (rc) return rc;
        return (e1 == cudaSuccess && e2 == cudaSuccess) ? BENES_OK : BENES_ERR_CUDA;
    }
    BENES_CUDA_TRY(cudaMemcpyAsync(d_in, in_host, data_bytes, cudaMemcpyHostToDevice, s));
    rc = benes_apply_ex(d_bits, d_in, d_out, elem_bytes, log2n, batch, stream);
    if (rc) return rc;
    BENES_CUDA_TRY(cudaMemcpyAsync(out_host, d_out, data_bytes, cudaMemcpyDeviceToHost, s));
    BENES_CUDA_TRY(cudaStreamSynchronize(s));
    return BENES_OK;
}

int benes_route_apply_host(const uint32_t *perm_host, const void *in_host, void *out_host, int elem_bytes,
                           int log2n, int batch, uint32_t *switch_bits_host, benes_stream_t stream) {
    if (!perm_host || !in_host || !out_host || bad_shape(log2n, batch)) return BENES_ERR_BADARG;
    if (elem_bytes != 4 && elem_bytes != 8) return BENES_ERR_BADARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int n = log2n;
    const Options opt = options();
    const size_t T = size_t(batch) << n;
    const size_t data_bytes = T * size_t(elem_bytes);
    const size_t chunks = apply_fused_chunks(n, size_t(batch));
    const bool piped = n > kFusedLog2M && level_chunk(n, size_t(batch), opt.chunk_log2) == size_t(batch) &&
                       opt.apply_fused && T >= (size_t(1) << 23) && chunks > 0 && chunks % kApplyMaxParts == 0;
    if (!piped) {
        // small or chunked inputs: one call after the other (the switch words stay on the host side
        // of the first call only if the caller wants them)
        const size_t words = benes_switch_words(n, batch);
        uint32_t *bits_tmp = switch_bits_host;
        if (!bits_tmp) {
            if (cudaMallocHost(&bits_tmp, words * 4) != cudaSuccess) { cudaGetLastError(); return BENES_ERR_NOMEM; }
        }
        int rc = benes_route_host(perm_host, n, batch, bits_tmp, stream);
        if (!rc) rc = benes_apply_host(bits_tmp, in_host, out_host, elem_bytes, n, batch, stream);
        if (!switch_bits_host) cudaFreeHost(bits_tmp);
        return rc;
    }
    const size_t perm_bytes = T * 4, bits_bytes = benes_switch_words(n, batch) * 4;
    const size_t route_ws = align_up(route_ws_bytes(n, size_t(batch)));
    const size_t apply_ws = align_up(apply_ws_bytes(elem_bytes, n, size_t(batch)));
    void *ws = nullptr;
    int rc = get_workspace(route_ws + apply_ws + align_up(perm_bytes) + align_up(bits_bytes) + 2 * align_up(data_bytes), &ws, s);
    if (rc) return rc;
    char *base = static_cast<char *>(ws);
    char *scratch = base + route_ws;
    uint32_t *d_perm = reinterpret_cast<uint32_t *>(scratch + apply_ws);
    uint32_t *d_bits = reinterpret_cast<uint32_t *>(reinterpret_cast<char *>(d_perm) + align_up(perm_bytes));
    char *d_in = reinterpret_cast<char *>(d_bits) + align_up(bits_bytes);
    char *d_out = d_in + align_up(data_bytes);
    HostPipe *hp = nullptr;
    if ((rc = host_pipe_for_current_device(&hp))) return rc;
    hp->bits_host = switch_bits_host;              // null: the switch words stay on the device
    hp->d2h = hp->back;
    hp->pieces = kMaxPieces;
    // the copy streams must not touch the workspace before earlier work on `s` is done
    BENES_CUDA_TRY(cudaEventRecord(hp->stage_ready[kMaxLevels - 1], s));
    BENES_CUDA_TRY(cudaStreamWaitEvent(hp->side, hp->stage_ready[kMaxLevels - 1], 0));
    BENES_CUDA_TRY(cudaStreamWaitEvent(hp->back, hp->stage_ready[kMaxLevels - 1], 0));
    // inbound: the permutation in pieces, then the payload in parts, behind one another on one
    // stream, while the levels run; outbound (second stream): finished stages, then finished parts
    const size_t per = perm_bytes / size_t(hp->pieces);
    for (int i = 0; i < hp->pieces; ++i) {
        BENES_CUDA_TRY(cudaMemcpyAsync(reinterpret_cast<char *>(d_perm) + per * size_t(i),
                                       reinterpret_cast<const char *>(perm_host) + per * size_t(i), per,
                                       cudaMemcpyHostToDevice, hp->side));
        BENES_CUDA_TRY(cudaEventRecord(hp->piece_ready[i], hp->side));
    }
    ApplyHostPipe pipe;
    pipe.parts = kApplyMaxParts;
    pipe.side = hp->back;
    pipe.out_host = out_host;
    const size_t part = data_bytes / size_t(pipe.parts);
    for (int i = 0; i < pipe.parts; ++i) {
        BENES_CUDA_TRY(cudaMemcpyAsync(d_in + part * size_t(i), static_cast<const char *>(in_host) + part * size_t(i),
                                       part, cudaMemcpyHostToDevice, hp->side));
        BENES_CUDA_TRY(cudaEventRecord(hp->part_ready[i], hp->side));
        pipe.in_ready[i] = hp->part_ready[i];
    }
    rc = route_levels(d_perm, n, size_t(batch), d_bits, base, s, opt, hp);
    if (!rc) {
        // the route no longer waits on these events; the apply's last pass reuses them
        for (int i = 0; i < pipe.parts; ++i) pipe.out_done[i] = hp->stage_ready[i];
        ProfileScope ps(kApplyFused, s);
        rc = launch_apply_fused(d_bits, d_in, d_out, scratch, elem_bytes, n, size_t(batch), s, &pipe);
    }
    cudaError_t e1 = cudaStreamSynchronize(s), e2 = cudaStreamSynchronize(hp->side), e3 = cudaStreamSynchronize(hp->back);
    if (rc) return rc;
    return (e1 == cudaSuccess && e2 == cudaSuccess && e3 == cudaSuccess) ? BENES_OK : BENES_ERR_CUDA;
}

struct benes_plan {
    int dev = 0;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    void *ws = nullptr;                   // the plan's own scratch: the captured launches point into it
    unsigned long long launches = 0;
};

int benes_plan_destroy(benes_plan_t *plan) {
    if (!plan) return BENES_OK;
    if (plan->exec) cudaGraphExecDestroy(plan->exec);
    if (plan->graph) cudaGraphDestroy(plan->graph);
    if (plan->ws) cudaFree(plan->ws);
    cudaGetLastError();
    delete plan;
    return BENES_OK;
}

int benes_plan_create(benes_plan_t **plan_out, const uint32_t *perm, int log2n, int batch, uint32_t *switch_bits,
                      const void *in, void *out, int elem_bytes) {
    if (!plan_out || !perm || !switch_bits || bad_shape(log2n, batch)) return BENES_ERR_BADARG;
    const bool with_apply = in != nullptr || out != nullptr;
    if (with_apply && (!in || !out || in == out || (elem_bytes != 4 && elem_bytes != 8))) return BENES_ERR_BADARG;
    if (benes_profile_enabled()) return BENES_ERR_BADARG;      // event brackets cannot live inside a graph
    *plan_out = nullptr;
    const Options opt = options();
    const int n = log2n;
    benes_plan *p = new (std::nothrow) benes_plan;
    if (!p) return BENES_ERR_NOMEM;
    cudaStream_t cap = nullptr;
    int rc = BENES_OK;
    auto fail = [&](int code) {
        if (cap) cudaStreamDestroy(cap);
        benes_plan_destroy(p);
        cudaGetLastError();
        return code;
    };
    if (cudaGetDevice(&p->dev) != cudaSuccess) return fail(BENES_ERR_CUDA);
    const size_t route_ws = route_needs_ws(n, opt) ? align_up(route_ws_bytes(n, size_t(batch))) : 0;
    const size_t apply_ws = with_apply ? align_up(apply_ws_bytes(elem_bytes, n, size_t(batch))) : 0;
    if (route_ws + apply_ws) {
        if (cudaMalloc(&p->ws, route_ws + apply_ws) != cudaSuccess) return fail(BENES_ERR_NOMEM);
    }
    char *ws = static_cast<char *>(p->ws);
    if (cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking) != cudaSuccess) return fail(BENES_ERR_CUDA);
    auto enqueue = [&]() -> int {
        int r = route_on(perm, n, batch, switch_bits, ws, cap, opt);
        if (!r && with_apply) r = apply_on(switch_bits, in, out, elem_bytes, n, batch, ws + route_ws, cap, opt);
        return r;
    };
    // once plainly (every kernel's attributes get set, and the buffers are checked by use), then captured
    if ((rc = enqueue())) return fail(rc);
    if (cudaStreamSynchronize(cap) != cudaSuccess) return fail(BENES_ERR_CUDA);
    const unsigned long long l0 = g_launches;
    if (cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return fail(BENES_ERR_CUDA);
    rc = enqueue();
    const cudaError_t e = cudaStreamEndCapture(cap, &p->graph);
    if (rc) return fail(rc);
    if (e != cudaSuccess || !p->graph) return fail(BENES_ERR_CUDA);
    p->launches = g_launches - l0;
    if (cudaGraphInstantiate(&p->exec, p->graph, 0) != cudaSuccess) return fail(BENES_ERR_CUDA);
    cudaStreamDestroy(cap);
    *plan_out = p;
    return BENES_OK;
}

int benes_plan_launch(const benes_plan_t *plan, benes_stream_t stream) {
    if (!plan || !plan->exec) return BENES_ERR_BADARG;
    BENES_CUDA_TRY(cudaGraphLaunch(plan->exec, reinterpret_cast<cudaStream_t>(stream)));
    g_launches += plan->launches;
    return BENES_OK;
}

int benes_validate_perm(const uint32_t *perm, int log2n, int batch, benes_stream_t stream) {
    if (!perm || bad_shape(log2n, batch)) return BENES_ERR_BADARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t total = size_t(batch) << log2n;
    const size_t seen_bytes = align_up(((total + 31) / 32) * 4);
    void *ws = nullptr;
    int rc = get_workspace(seen_bytes + kAlign, &ws, s);
    if (rc) return rc;
    uint32_t *seen = static_cast<uint32_t *>(ws);
    uint32_t *flag = reinterpret_cast<uint32_t *>(static_cast<char *>(ws) + seen_bytes);
    BENES_CUDA_TRY(cudaMemsetAsync(ws, 0, seen_bytes + kAlign, s));
    if ((rc = launch_validate(perm, total, log2n, seen, flag, s))) return rc;
    uint32_t h = 0;
    BENES_CUDA_TRY(cudaMemcpyAsync(&h, flag, 4, cudaMemcpyDeviceToHost, s));
    BENES_CUDA_TRY(cudaStreamSynchronize(s));
    return h ? BENES_ERR_NOT_PERMUTATION : BENES_OK;
}

unsigned long long benes_launch_count(void) { return g_launches; }

int benes_debug_build(void) {
#ifdef BENES_DEBUG
    return 1;
#else
    return 0;
#endif
}

int benes_debug_guard_hits(unsigned long long *hits, char *where, size_t where_bytes, int clear) {
    if (!hits) return BENES_ERR_BADARG;
    *hits = 0;
    if (where && where_bytes) where[0] = 0;
#ifdef BENES_DEBUG
    BENES_CUDA_TRY(cudaDeviceSynchronize());
    for (const GuardEntry &e : guard_registry()) {
        unsigned int w[2] = {0u, 0u};
        const int rc = e.read(w, clear);
        if (rc) return rc;
        if (w[0] && where && where_bytes) std::snprintf(where, where_bytes, "%s:%u", e.file, w[1]);
        *hits += w[0];
    }
#else
    (void)clear;
#endif
    return BENES_OK;
}

int benes_set_option(int key, int value) {
    std::lock_guard<std::mutex> lk(g_mu);
    switch (key) {
        case BENES_OPT_SAMPLE_LOG2K:
            if (value != 0 && (value < kMinKappa || value > kMaxKappa)) return BENES_ERR_BADARG;
            g_opt.kappa = value;
            return BENES_OK;
        case BENES_OPT_WALK_CAP:
            if (value < 1 || value > (1 << 24)) return BENES_ERR_BADARG;
            g_opt.walk_cap = value;
            return BENES_OK;
        case BENES_OPT_APPLY_FUSED:
            if (value != 0 && value != 1) return BENES_ERR_BADARG;
            g_opt.apply_fused = value;
            return BENES_OK;
        case BENES_OPT_INVERSE_PARTITIONED:
            if (value != 0 && value != 1) return BENES_ERR_BADARG;
            g_opt.inverse_partitioned = value;
            return BENES_OK;
        case BENES_OPT_CHUNK_LOG2:
            if (value < 16 || value > 30) return BENES_ERR_BADARG;
            g_opt.chunk_log2 = value;
            return BENES_OK;
        case BENES_OPT_CLUSTER:
            if (value != 0 && value != 1) return BENES_ERR_BADARG;
            g_opt.cluster = value;
            return BENES_OK;
        case BENES_OPT_WALK_PAIRS:
            if (value < 0 || value > 2) return BENES_ERR_BADARG;
            g_opt.walk_pairs = value;
            return BENES_OK;
        default: return BENES_ERR_BADARG;
    }
}

int benes_get_option(int key) {
    std::lock_guard<std::mutex> lk(g_mu);
    switch (key) {
        case BENES_OPT_SAMPLE_LOG2K: return g_opt.kappa;
        case BENES_OPT_WALK_CAP: return g_opt.walk_cap;
        case BENES_OPT_APPLY_FUSED: return g_opt.apply_fused;
        case BENES_OPT_INVERSE_PARTITIONED: return g_opt.inverse_partitioned;
        case BENES_OPT_CHUNK_LOG2: return g_opt.chunk_log2;
        case BENES_OPT_CLUSTER: return g_opt.cluster;
        case BENES_OPT_WALK_PAIRS: return g_opt.walk_pairs;
        default: return BENES_ERR_BADARG;
    }
}

int benes_fused_log2m(void) { return kFusedLog2M; }

const char *benes_status_string(int status) {
    switch (status) {
        case BENES_OK: return "ok";
        case BENES_ERR_BADARG: return "bad argument";
        case BENES_ERR_CUDA: return "CUDA runtime error";
        case BENES_ERR_NOMEM: return "workspace allocation failed or caller workspace too small";
        case BENES_ERR_NOT_PERMUTATION: return "input is not a permutation";
        case BENES_ERR_TOO_LARGE: return "payload larger than the built-in scratch of benes_apply_static";
        default: return "unknown status";
    }
}

}  // extern "C"
