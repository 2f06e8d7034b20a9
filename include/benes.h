/*
 * benes.h -- C ABI of the B200 (sm_100a) Benes-network routing library.
 *
 * Problem statement: a rearrangeable Benes network of N = 2^n inputs has 2n-1
 * stages of N/2 two-by-two switches.  benes_route computes the switch settings that make it
 * realise a permutation pi given in GATHER form, out[j] = in[pi[j]];
 * benes_apply pushes a payload through the stages.
 *
 * Canonical result.  Several settings realise the same pi; the library returns
 * the one in which, at every recursion level and in every sub-network, the
 * smallest output index of each constraint loop is served by the UPPER
 * half-size sub-network.  The result is therefore unique and is compared
 * bit for bit with the CPU oracle.
 *
 * Switch-bit layout (all entry points).  Stage-major.  A stage has
 * W = max(1, N/64) 32-bit words; switch w of a stage is bit (w & 31) of word
 * (w >> 5); 0 = straight, 1 = cross; unused bits are 0.  Recursion level l
 * (0 <= l <= n-1) consists of 2^l sub-networks ("blocks") of size M = N >> l,
 * block b owning flat positions [bM, (b+1)M) and, in every stage it owns,
 * switches [b*M/2, (b+1)*M/2).  Stage l <= n-2 is the input side of level l,
 * stage n-1 the middle, stage 2n-2-l the output side of level l.  Wiring: on
 * the input side, switch s of a block sends its upper output to position s of
 * the block's upper half and its lower output to position s of the lower
 * half; the output side is the mirror image.  A batch is `batch` such
 * records back to back: batch x (2n-1) x W words.
 *
 * Conventions.  Every pointer is a DEVICE pointer unless the name says
 * "_host".  The caller owns every buffer it passes; the library owns only its
 * internal workspace (one per device, or supplied by the caller).  A call that
 * needs more than the workspace holds replaces it in stream order on `stream`
 * (cudaFreeAsync + cudaMallocAsync from the device's default pool: no
 * device-wide synchronisation; only on a device without memory pools the old
 * cudaDeviceSynchronize + cudaFree + cudaMalloc).  Work is enqueued on
 * `stream` and the call returns without synchronising, except where stated.
 * Argument errors are detected on the host before anything is enqueued.
 * benes_route, benes_apply and benes_apply_ex do nothing but enqueue kernels and
 * memsets on `stream` once the workspace is large enough and every kernel has
 * run once on the device (i.e. after one ordinary call with the same sizes), so
 * they can be captured into a CUDA graph and replayed on new contents of the
 * same buffers; with the 2-50 small dependent launches of inputs up to about
 * 2^22 elements a replay is 10-40 % faster than the launches.
 * Nothing throws, aborts or traps.  The library is not re-entrant: calls that
 * share the workspace must be ordered (same stream, or externally
 * synchronised).
 */
#ifndef BENES_H_
#define BENES_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st *benes_stream_t; /* a cudaStream_t; NULL = default stream */

enum {
    BENES_OK = 0,
    BENES_ERR_BADARG = -1,          /* null pointer, log2n or batch out of range, bad elem_bytes */
    BENES_ERR_CUDA = -2,            /* a CUDA runtime call or launch failed */
    BENES_ERR_NOMEM = -3,           /* workspace could not be allocated / supplied one too small */
    BENES_ERR_NOT_PERMUTATION = -4, /* benes_validate_perm only */
    BENES_ERR_TOO_LARGE = -5        /* benes_apply_static only: payload exceeds the built-in scratch */
};
/* There is no time-out status: no kernel of the library waits on a flag, a peer
 * or another launch.  The only loops whose length depends on the data are the
 * walks, and those stop after BENES_OPT_WALK_CAP hops and hand the level to the
 * pointer-jumping kernel, whose pass count is fixed by the block size. */

#define BENES_MAX_LOG2N 30

/*
 * Switch settings (steps: inverse scatter, successor pairing, pointer-jumping
 * loop labelling to the minimum index, 2-colouring, first/last stage,
 * sub-permutation compaction; all n levels).
 *   perm        : batch x N uint32, each row a permutation of [0, N); read only.
 *   log2n       : 1 .. BENES_MAX_LOG2N.
 *   batch       : >= 1 independent permutations.
 *   switch_bits : batch x (2n-1) x W words (benes_switch_words), fully overwritten.
 * If a row is not a permutation the result is unspecified but every access
 * stays in bounds.  Returns BENES_OK or a negative status.
 */
int benes_route(const uint32_t *perm, int log2n, int batch, uint32_t *switch_bits,
                benes_stream_t stream);

/*
 * Route a payload of 4-byte elements through the 2n-1 stages of the network:
 * out[b][j] = in[b][pi_b[j]] when switch_bits came from benes_route(pi).
 *   in, out : batch x N elements; must not overlap; in is read only.
 */
int benes_apply(const uint32_t *switch_bits, const void *in, void *out, int log2n, int batch,
                benes_stream_t stream);

/* Same with an explicit element size: elem_bytes must be 4 or 8. */
int benes_apply_ex(const uint32_t *switch_bits, const void *in, void *out, int elem_bytes,
                   int log2n, int batch, benes_stream_t stream);

/*
 * Sizes that are not a power of two.  A permutation of [0, n_elems) is routed
 * through the network of N = 2^log2n inputs, log2n = benes_padded_log2n(n_elems)
 * (the smallest with N >= n_elems; 0 if n_elems is 0 or above 2^30), extended
 * by fixed points pi[j] = j for j >= n_elems.
 *   perm        : batch x n_elems uint32, each row a permutation of [0, n_elems).
 *   switch_bits : sized and laid out for (log2n, batch), see benes_switch_words.
 *   in, out     : batch x n_elems elements of elem_bytes (4 or 8); no overlap.
 * out[b][j] = in[b][pi_b[j]] for j < n_elems.  Padded copies live in the
 * library workspace.
 */
int benes_padded_log2n(size_t n_elems);
int benes_route_padded(const uint32_t *perm, size_t n_elems, int batch, uint32_t *switch_bits,
                       benes_stream_t stream);
int benes_apply_padded(const uint32_t *switch_bits, const void *in, void *out, int elem_bytes,
                       size_t n_elems, int batch, benes_stream_t stream);

/*
 * The same settings for the network drawn in place (no wiring between stages):
 * row r of butterfly_bits pairs positions u and u | 2^i that differ in bit i,
 * i = r for r <= n-1 and i = 2n-2-r after the middle; pair p of a row (u with
 * bit i taken out) is bit (p & 31) of word (p >> 5); a set bit swaps the two
 * positions.  Running the 2n-1 rows in order on a payload in place leaves
 * out[j] = in[pi[j]].  Same size as switch_bits (benes_switch_words); the two
 * buffers must be different.
 */
int benes_export_butterfly(const uint32_t *switch_bits, uint32_t *butterfly_bits, int log2n, int batch,
                           benes_stream_t stream);

/*
 * benes_apply_ex for callers that cannot allocate device memory.  (The paper
 * has no counterpart; this is a deployment convenience of this library.)
 *
 * Who needs it: a process that has given all device memory to another
 * allocator, where the cudaMalloc behind the library workspace would fail, and
 * a latency-critical loop that cannot take the device-wide stall of a
 * cudaMalloc / cudaFree.  This entry point never calls cudaMalloc, cudaFree or
 * any allocating routine: its one scratch buffer is a fixed array of
 * BENES_STATIC_SCRATCH_BYTES that is part of the library image (every GPU
 * that loads the library keeps it until the process exits).
 *
 * Same arguments, layout and result as benes_apply_ex, with one limit:
 * batch * N * elem_bytes must not exceed BENES_STATIC_SCRATCH_BYTES, otherwise
 * BENES_ERR_TOO_LARGE is returned and nothing is enqueued.
 *
 * The first call on each device looks up the array's device address with the
 * runtime.  That query allocates nothing by itself, but it can be the moment
 * the CUDA runtime loads the part of the library that holds the array and
 * reserves its 4 MiB on that device.  So make one call per device at start-up:
 * before the rest of the device memory is handed to another allocator (a
 * process that has already given everything away can see BENES_ERR_CUDA from
 * this first call), and outside any stream capture.  All calls share the one
 * array and it keeps the previous call's contents (nothing needs clearing:
 * each stage overwrites all it later reads).  Two calls whose kernels can
 * overlap on the GPU (different streams, no ordering) race on it: keep them on
 * one stream or order them yourself.
 */
#define BENES_STATIC_SCRATCH_BYTES (4u << 20)
int benes_apply_static(const uint32_t *switch_bits, const void *in, void *out, int elem_bytes,
                       int log2n, int batch, benes_stream_t stream);

/*
 * Host-buffer variants: copy the inputs to the device, run, copy the result
 * back and SYNCHRONISE `stream` before returning.  Buffers are ordinary or
 * pinned host memory (pinned memory lets the copies overlap the kernels).
 * Device staging lives in the library workspace.  Both calls overlap their
 * copies with the computation on a second stream the library owns (one per
 * device, created on the first call).  benes_route_host: the permutation
 * arrives in pieces, and the stages a level has finished go back while the next
 * levels run.  benes_apply_host (payloads of 64 MiB and more): the first pass
 * starts on each part of the payload as it arrives, and the parts the last
 * pass has finished go back while it still runs.
 */
int benes_route_host(const uint32_t *perm_host, int log2n, int batch, uint32_t *switch_bits_host,
                     benes_stream_t stream);
int benes_apply_host(const uint32_t *switch_bits_host, const void *in_host, void *out_host,
                     int elem_bytes, int log2n, int batch, benes_stream_t stream);

/*
 * Both steps for host buffers in one call: out_host[b][j] = in_host[b][pi_b[j]].
 * switch_bits_host may be NULL if the settings themselves are not wanted.  For
 * batch * N >= 2^23 the payload travels to the device while the levels run, the
 * finished stages and the finished parts of the routed payload travel back on a
 * second copy stream, and the switch words never make the round trip through
 * host memory that calling benes_route_host and benes_apply_host one after the
 * other costs.  Synchronises `stream` before returning.
 */
int benes_route_apply_host(const uint32_t *perm_host, const void *in_host, void *out_host, int elem_bytes,
                           int log2n, int batch, uint32_t *switch_bits_host, benes_stream_t stream);

/*
 * Plans: the same route (and, if `in` and `out` are given, the apply behind it)
 * on the same buffers, many times.  benes_plan_create runs the work once on a
 * stream of its own (synchronously), captures it into a CUDA graph and keeps a
 * scratch buffer of its own for it (cudaMalloc; freed by benes_plan_destroy), so
 * a plan is independent of the library workspace.  benes_plan_launch enqueues the
 * whole graph on `stream` with one call: for inputs of up to about 2^22 elements,
 * whose 2-50 dependent launches are short, that is 10-15 % faster than the
 * launches themselves.  The plan reads whatever `perm` (and `in`) hold at launch
 * time and is bound to the addresses, sizes and options it was created with; the
 * buffers must outlive it.  Launches of one plan are ordered one after another.
 * Not available while the per-kernel timing brackets are enabled.
 *   in, out, elem_bytes : NULL, NULL, 0 for a route-only plan.
 */
typedef struct benes_plan benes_plan_t;
int benes_plan_create(benes_plan_t **plan, const uint32_t *perm, int log2n, int batch, uint32_t *switch_bits,
                      const void *in, void *out, int elem_bytes);
int benes_plan_launch(const benes_plan_t *plan, benes_stream_t stream);
int benes_plan_destroy(benes_plan_t *plan);

/* Number of 32-bit words of switch_bits for (log2n, batch); 0 on bad arguments. */
size_t benes_switch_words(int log2n, int batch);

/* Scratch bytes benes_route / benes_apply_ex need for these arguments. */
size_t benes_route_workspace_bytes(int log2n, int batch);
size_t benes_apply_workspace_bytes(int elem_bytes, int log2n, int batch);

/*
 * Hand the library a caller-owned device scratch buffer (256-byte aligned) to
 * use instead of its own; pass (NULL, 0) to return to the internal one.  With
 * a caller buffer no entry point allocates; a call that needs more than
 * `bytes` fails with BENES_ERR_NOMEM.
 */
int benes_set_workspace(void *dev_ptr, size_t bytes);

/* Free the internal workspace of the current device (synchronises the device). */
int benes_release_workspace(void);

/*
 * Check that every row of perm is a permutation of [0, N).  Synchronises
 * `stream`.  Returns BENES_OK, BENES_ERR_NOT_PERMUTATION or another error.
 */
int benes_validate_perm(const uint32_t *perm, int log2n, int batch, benes_stream_t stream);

/*
 * Tuning of the loop labelling of benes_route (process-wide; set between calls).
 *   BENES_OPT_SAMPLE_LOG2K : 0 = label every loop by pointer jumping over all
 *       outputs; kappa in 2..8 (default 4) = label only one sampled "ruler"
 *       switch per 2^kappa switches by pointer jumping and reach the rest by
 *       sequential walks between rulers (for batch * N <= 2^22 at most 2^3: short
 *       walks matter more than short lists there).  The result is identical
 *       either way.
 *   BENES_OPT_WALK_CAP : hops (1 .. 2^24, default 2^14) after which a walk gives
 *       up; a level in which that happens is relabelled by full pointer jumping.
 *   BENES_OPT_APPLY_FUSED : 1 (default) = benes_apply / benes_apply_ex run up to
 *       25 stages per pass over the payload in shared memory; 0 = one stage per
 *       pass.  Same result.
 *   BENES_OPT_INVERSE_PARTITIONED : 1 (default) = for batch * N >= 2^22 the inverse
 *       permutation of level 0 is formed by bucketing (destination, source)
 *       pairs and scattering bucket by bucket; 0 = one pass of random writes.
 *   BENES_OPT_CHUNK_LOG2 : 16..30 (default 30): a batch whose levels do not fit one
 *       CTA is processed in chunks of at most 2^value elements (whole
 *       permutations, at least one); bounds the workspace of a large batch.
 *   BENES_OPT_CLUSTER : 1 = blocks of 2^16 outputs (whole permutations of N = 2^16,
 *       and the tail of larger ones) are finished by a thread-block cluster of two
 *       CTAs over distributed shared memory instead of one more level in global
 *       memory; 0 = blocks of 2^15 in one CTA.  Same result.
 *   BENES_OPT_WALK_PAIRS : at levels with packed 8-byte records a thread can advance the
 *       two walks that leave one ruler switch together (their chains of dependent
 *       accesses overlap).  0 = never, 1 (default) = where the halved number of
 *       threads still fills the GPU, 2 = at every such level.  Same result.
 * benes_set_option returns BENES_OK or BENES_ERR_BADARG; benes_get_option
 * returns the value, or BENES_ERR_BADARG for an unknown key.
 */
#define BENES_OPT_SAMPLE_LOG2K 0
#define BENES_OPT_WALK_CAP 1
#define BENES_OPT_APPLY_FUSED 2
#define BENES_OPT_INVERSE_PARTITIONED 3
#define BENES_OPT_CHUNK_LOG2 4
#define BENES_OPT_CLUSTER 5
#define BENES_OPT_WALK_PAIRS 6
int benes_set_option(int key, int value);
int benes_get_option(int key);

/* Kernels launched by this library in this process so far (host-side counter). */
unsigned long long benes_launch_count(void);

/*
 * Optional per-kernel timing.  While enabled, the library brackets each group
 * of consecutive launches of one kernel kind with a pair of CUDA events on the
 * caller's stream.  benes_profile_read synchronises those events and returns,
 * for one kind, the launches and the summed device time since the last reset.
 * Kinds: 0 inverse scatter, 1 pointer jumping over all outputs (one launch per
 * level), 2 input-side bits + compaction, 3 fused in-CTA levels, 4 payload-apply
 * stage, 5 ruler walk, 6 contracted-list assembly, 7 walk over a contracted
 * list, 8 in-CTA labelling of a contracted list, 9 labels back to a sampled
 * list, 10 colouring + output-side bits, 11 payload-apply over several stages.
 * BENES_PROFILE_KINDS = number of kinds.
 */
#define BENES_PROFILE_KINDS 12
int benes_profile_enable(int on);
int benes_profile_enabled(void);    /* 1 while the brackets are on */
int benes_profile_reset(void);
int benes_profile_read(int kind, unsigned long long *launches, double *milliseconds);
/* The index-th timed group since the last reset, in launch order (one group per
 * kind per recursion level): its kind, launches and device time.
 * BENES_ERR_BADARG once index is past the last group. */
int benes_profile_span(int index, int *kind, unsigned long long *launches, double *milliseconds);
const char *benes_profile_kind_name(int kind);

/*
 * Batch sharding over several GPUs.  The permutations of a batch are independent,
 * so G processes (one per GPU) each route a contiguous slice with no exchange
 * between them: rank r of `world` takes permutations [*first, *first + *count)
 * (slice sizes differ by at most one; *count may be 0 when world > batch) and
 * calls benes_route / benes_apply on perm + *first * N, switch_bits +
 * *first * (2n-1) * W and the matching payload rows.  Host-only arithmetic; no
 * CUDA call.  A single permutation does not shard: its top levels gather over
 * the whole array.
 */
int benes_shard_batch(int batch, int world, int rank, int *first, int *count);

/*
 * Measurement aid (no step of the method): `ops` (<= 2^32) random accesses to
 * table[0 .. 2^log2_records * record_bytes), each to a different pseudo-randomly
 * placed record when ops <= 2^log2_records, two in flight per thread, enqueued on
 * `stream`; the caller times it with events.  The ruler walks are chains of such
 * accesses, and these are the rates (and, under a profiler, the DRAM bytes per
 * access) they are compared with.  mode 0: 4-byte load; 1: 16-byte load; 2:
 * 16-byte load, then compare-and-swap on the record's third word; 3: 64-bit atomic
 * AND on the record's first 8 bytes; 4: 4-byte store to the third word.  Modes 2-4
 * overwrite the table.  record_bytes: a multiple of 4 / 16 / 16 / 8 / 16 for modes
 * 0..4.  `sink` is one device word; it is written only if the words a thread read
 * xor to one particular value (so that the reads cannot be dropped).
 */
int benes_probe_random_access(void *table, int log2_records, int record_bytes, int mode, size_t ops,
                              uint32_t *sink, benes_stream_t stream);

/*
 * Checked build.  Every index a kernel forms from data is forced into range (a
 * mask or a clamp), which is what keeps a non-permutation input memory-safe; on a
 * permutation no such guard ever changes its value.  The library built with
 * -DBENES_DEBUG (libbenes_debug.so, same ABI) counts, in device words, every guard
 * that did change a value, and remembers the source line of one of them.  Nothing
 * traps and nothing is printed.  benes_debug_build returns 1 for that build, 0
 * otherwise.  benes_debug_guard_hits synchronises the current device, stores the
 * number of such events since the last clearing in *hits (always 0 in the normal
 * build), writes "file:line" of one of them to `where` (may be NULL) and clears
 * the counters if `clear` is non-zero.
 */
int benes_debug_build(void);
int benes_debug_guard_hits(unsigned long long *hits, char *where, size_t where_bytes, int clear);

/* Largest block size (log2) finished inside one CTA by the fused kernel. */
int benes_fused_log2m(void);

const char *benes_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* BENES_H_ */
