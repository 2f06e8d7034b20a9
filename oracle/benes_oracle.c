/*
 * CPU oracle for Benes-network routing.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, sequential, obviously-correct statement of what the
 * CUDA library computes.  It shares no code, header, table or helper with the
 * CUDA path and must never be linked or imported by it.  Only tests, the smoke
 * check and the benchmark's CPU-baseline leg may call it.
 *
 * What it follows: the problem statement (a
 * rearrangeable Benes network of N = 2^n inputs must realise a permutation pi
 * in gather form, out[j] = in[pi[j]]) and the classical sequential "looping
 * algorithm": walk every constraint loop once, colour its elements
 * alternately, set the outermost two stages, recurse on the two half-size
 * sub-permutations.  The paper contains no statement of this method,
 * so every convention is written out here:
 *
 *   - A level l (0 <= l <= n-1) consists of 2^l independent sub-networks
 *     ("blocks") of size M = N >> l; block b owns flat indices [bM, (b+1)M).
 *   - Loops are indexed by OUTPUTS.  Output j and output j^1 share an output
 *     switch, so they must come from different halves; the two inputs of one
 *     input switch (i and i^1) must go to different halves.
 *   - Canonical rule: in each loop the smallest output index goes through the
 *     UPPER sub-network (colour 0).
 *   - Switch bit: 0 = straight, 1 = cross.
 *   - Stage l <= n-2 is the input side of level l, stage n-1 the middle,
 *     stage 2n-2-l the output side of level l.  Inside a stage, block b of
 *     level l owns switches [b*M/2, (b+1)*M/2).  Switch w is bit (w & 31) of
 *     32-bit word (w >> 5); every stage has max(1, N/64) words; unused bits
 *     are 0.
 *   - Wiring: on the input side the upper output of switch s goes to position
 *     s of the upper half-block, the lower output to position s of the lower
 *     half-block; the output side is the mirror image.
 *
 * Parity pins (tests/test_oracle_pins.py): exhaustive N = 2, 4, 8; a
 * recursive re-definition of the network; enumeration of all switch settings
 * at N = 4 and N = 8; closed forms (identity, cyclic shift); union-find
 * colouring; invariants at every level.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static size_t stage_words(int n) {
    size_t N = (size_t)1 << n;
    return N >= 64 ? N / 64 : 1;
}

static void set_bit(uint32_t *stage, size_t w, uint32_t v) {
    if (v) stage[w >> 5] |= (uint32_t)1 << (w & 31);
}

/*
 * One sub-network of size M (M >= 4) with block-local gather permutation p.
 * Fills colour[0..M) (0 = upper, 1 = lower), the block's input-side and
 * output-side switches, and the two half-size sub-permutations
 * (upper into pn[0..M/2), lower into pn[M/2..M)).
 */
static void route_block(const uint32_t *p, size_t M, uint32_t *inv, uint8_t *colour,
                        uint32_t *in_stage, uint32_t *out_stage, size_t first_switch,
                        uint32_t *pn) {
    size_t j, s;
    for (j = 0; j < M; ++j) inv[p[j]] = (uint32_t)j;
    memset(colour, 0xFF, M);
    for (size_t j0 = 0; j0 < M; ++j0) {
        if (colour[j0] != 0xFF) continue;
        /* j0 is the smallest output index of a loop not yet walked. */
        j = j0;
        for (;;) {
            colour[j] = 0;      /* this output is served by the upper half   */
            colour[j ^ 1] = 1;  /* its switch partner must use the lower half */
            /* The partner's source input p[j^1] sits on an input switch whose
             * other input, p[j^1]^1, must then go up; the output it feeds is
             * the next element of the loop. */
            size_t k = inv[p[j ^ 1] ^ 1];
            if (k == j0) break;
            j = k;
        }
    }
    for (s = 0; s < M / 2; ++s) {
        set_bit(in_stage, first_switch + s, colour[inv[2 * s]]);
        set_bit(out_stage, first_switch + s, colour[2 * s]);
    }
    for (j = 0; j < M; ++j)
        pn[(size_t)colour[j] * (M / 2) + (j >> 1)] = p[j] >> 1;
}

/*
 * Switch settings for one permutation.
 *   perm : N = 2^n values, a permutation of [0, N), gather form
 *   bits : (2n-1) * max(1, N/64) words, fully overwritten
 *   trace_p      : optional, n * N words; level l's block-local sub-permutations
 *   trace_colour : optional, n * N bytes; level l's colours (level n-1 unused)
 * Returns 0, or -1 on bad arguments / allocation failure.
 */
int oracle_route_trace(const uint32_t *perm, int n, uint32_t *bits,
                       uint32_t *trace_p, uint8_t *trace_colour) {
    if (!perm || !bits || n < 1 || n > 30) return -1;
    size_t N = (size_t)1 << n, W = stage_words(n);
    uint32_t *P = malloc(N * 4), *Pn = malloc(N * 4), *inv = malloc(N * 4);
    uint8_t *colour = malloc(N);
    if (!P || !Pn || !inv || !colour) { free(P); free(Pn); free(inv); free(colour); return -1; }
    memset(bits, 0, (size_t)(2 * n - 1) * W * 4);
    memcpy(P, perm, N * 4);
    for (int l = 0; l < n; ++l) {
        size_t M = N >> l;
        if (trace_p) memcpy(trace_p + (size_t)l * N, P, N * 4);
        if (M == 2) {
            /* middle stage: one switch per block, crossed iff output 0 takes input 1 */
            for (size_t b = 0; b < N / 2; ++b) set_bit(bits + (size_t)(n - 1) * W, b, P[2 * b]);
            break;
        }
        for (size_t base = 0; base < N; base += M)
            route_block(P + base, M, inv, colour + base, bits + (size_t)l * W,
                        bits + (size_t)(2 * n - 2 - l) * W, base / 2, Pn + base);
        if (trace_colour) memcpy(trace_colour + (size_t)l * N, colour, N);
        uint32_t *t = P; P = Pn; Pn = t;
    }
    free(P); free(Pn); free(inv); free(colour);
    return 0;
}

int oracle_route(const uint32_t *perm, int n, uint32_t *bits) {
    return oracle_route_trace(perm, n, bits, NULL, NULL);
}

/* batch independent permutations, packed back to back */
int oracle_route_batch(const uint32_t *perm, int n, int batch, uint32_t *bits) {
    if (batch < 1) return -1;
    size_t N = (size_t)1 << n, per = (size_t)(2 * n - 1) * stage_words(n);
    for (int b = 0; b < batch; ++b) {
        int rc = oracle_route(perm + (size_t)b * N, n, bits + (size_t)b * per);
        if (rc) return rc;
    }
    return 0;
}

static uint32_t get_bit(const uint32_t *stage, size_t w) {
    return (stage[w >> 5] >> (w & 31)) & 1u;
}

/*
 * Push a payload of N elements of elem_bytes bytes each through the 2n-1
 * stages, one stage at a time, one switch at a time.  in and out must not
 * overlap.  Returns 0 or -1.
 */
int oracle_apply(const uint32_t *bits, const void *in, void *out, int elem_bytes, int n) {
    if (!bits || !in || !out || n < 1 || n > 30 || elem_bytes < 1) return -1;
    size_t N = (size_t)1 << n, W = stage_words(n), e = (size_t)elem_bytes;
    unsigned char *x = malloc(N * e), *y = malloc(N * e);
    if (!x || !y) { free(x); free(y); return -1; }
    memcpy(x, in, N * e);
    for (int st = 0; st < 2 * n - 1; ++st) {
        const uint32_t *stage = bits + (size_t)st * W;
        int l = st <= n - 1 ? st : 2 * n - 2 - st;   /* recursion level of this stage */
        size_t M = N >> l, H = M / 2;
        for (size_t base = 0; base < N; base += M) {
            for (size_t s = 0; s < H; ++s) {
                uint32_t cross = get_bit(stage, base / 2 + s);
                size_t a, b, ya, yb;   /* source pair, destination pair */
                if (st < n - 1) {            /* input side: switch, then un-shuffle */
                    a = base + 2 * s; b = a + 1; ya = base + s; yb = base + H + s;
                } else if (st == n - 1) {    /* middle: a lone switch */
                    a = base; b = base + 1; ya = a; yb = b;
                } else {                     /* output side: shuffle, then switch */
                    a = base + s; b = base + H + s; ya = base + 2 * s; yb = ya + 1;
                }
                if (cross) { size_t t = a; a = b; b = t; }
                memcpy(y + ya * e, x + a * e, e);
                memcpy(y + yb * e, x + b * e, e);
            }
        }
        unsigned char *t = x; x = y; y = t;
    }
    memcpy(out, x, N * e);
    free(x); free(y);
    return 0;
}

int oracle_apply_batch(const uint32_t *bits, const void *in, void *out, int elem_bytes, int n, int batch) {
    if (batch < 1) return -1;
    size_t N = (size_t)1 << n, per = (size_t)(2 * n - 1) * stage_words(n);
    for (int b = 0; b < batch; ++b) {
        int rc = oracle_apply(bits + (size_t)b * per, (const char *)in + (size_t)b * N * elem_bytes,
                              (char *)out + (size_t)b * N * elem_bytes, elem_bytes, n);
        if (rc) return rc;
    }
    return 0;
}

/*
 * The two functions below run the SAME per-block routine and the SAME per-switch
 * loop as oracle_route_trace / oracle_apply, restricted to a range of the flat
 * array, so that a caller can hand independent sub-networks to several host
 * threads (the benchmark's all-core figure: top levels on one thread, the
 * sub-networks below them in parallel).  They add no arithmetic of their own;
 * tests/test_oracle_pins.py checks that any split into parts reproduces
 * oracle_route and oracle_apply word for word.
 */

/*
 * Levels first .. stop-1 (stop <= n) of the sub-networks that occupy the flat
 * range [lo, hi) at level `first` (lo and hi multiples of N >> first).
 *   P_first : the flat level-`first` array of block-local sub-permutations
 *             (N entries; only [lo, hi) is read)
 *   bits    : the permutation's whole (2n-1) x W array, NOT cleared here; only
 *             switches [lo/2, hi/2) of stages first..stop-1 and their mirror
 *             stages are set.  Concurrent callers need ranges whose switches do
 *             not share a 32-bit word: (hi - lo) a multiple of 64.
 *   P_stop  : if not NULL and stop < n, receives the level-`stop` array on [lo, hi)
 */
int oracle_route_part(const uint32_t *P_first, int n, int first, int stop, size_t lo, size_t hi,
                      uint32_t *bits, uint32_t *P_stop) {
    if (!P_first || !bits || n < 1 || n > 30 || first < 0 || stop > n || first > stop) return -1;
    size_t N = (size_t)1 << n, W = stage_words(n), M0 = N >> first, len = hi - lo;
    if (lo > hi || hi > N || lo % M0 || hi % M0) return -1;
    if (len == 0) return 0;
    uint32_t *P = malloc(len * 4), *Pn = malloc(len * 4), *inv = malloc(len * 4);
    uint8_t *colour = malloc(len);
    if (!P || !Pn || !inv || !colour) { free(P); free(Pn); free(inv); free(colour); return -1; }
    memcpy(P, P_first + lo, len * 4);
    for (int l = first; l < stop; ++l) {
        size_t M = N >> l;
        if (M == 2) {
            for (size_t b = 0; b < len / 2; ++b) set_bit(bits + (size_t)(n - 1) * W, lo / 2 + b, P[2 * b]);
            break;
        }
        for (size_t base = 0; base < len; base += M)
            route_block(P + base, M, inv, colour + base, bits + (size_t)l * W,
                        bits + (size_t)(2 * n - 2 - l) * W, (lo + base) / 2, Pn + base);
        uint32_t *t = P; P = Pn; Pn = t;
    }
    if (P_stop && stop < n) memcpy(P_stop + lo, P, len * 4);
    free(P); free(Pn); free(inv); free(colour);
    return 0;
}

/*
 * Stages st_first .. st_stop-1 of oracle_apply on the positions [lo, hi), which
 * must consist of whole blocks of every stage in that range.  x and tmp are
 * N-element buffers; the stages ping-pong between them inside [lo, hi) and the
 * result is left in x.
 */
int oracle_apply_part(const uint32_t *bits, void *xv, void *tmpv, int elem_bytes, int n,
                      int st_first, int st_stop, size_t lo, size_t hi) {
    if (!bits || !xv || !tmpv || n < 1 || n > 30 || elem_bytes < 1) return -1;
    if (st_first < 0 || st_stop > 2 * n - 1 || st_first > st_stop) return -1;
    size_t N = (size_t)1 << n, W = stage_words(n), e = (size_t)elem_bytes;
    if (lo > hi || hi > N) return -1;
    unsigned char *x = xv, *y = tmpv;
    for (int st = st_first; st < st_stop; ++st) {
        const uint32_t *stage = bits + (size_t)st * W;
        int l = st <= n - 1 ? st : 2 * n - 2 - st;
        size_t M = N >> l, H = M / 2;
        if (lo % M || hi % M) return -1;
        for (size_t base = lo; base < hi; base += M) {
            for (size_t s = 0; s < H; ++s) {
                uint32_t cross = get_bit(stage, base / 2 + s);
                size_t a, b, ya, yb;
                if (st < n - 1) {
                    a = base + 2 * s; b = a + 1; ya = base + s; yb = base + H + s;
                } else if (st == n - 1) {
                    a = base; b = base + 1; ya = a; yb = b;
                } else {
                    a = base + s; b = base + H + s; ya = base + 2 * s; yb = ya + 1;
                }
                if (cross) { size_t t = a; a = b; b = t; }
                memcpy(y + ya * e, x + a * e, e);
                memcpy(y + yb * e, x + b * e, e);
            }
        }
        unsigned char *t = x; x = y; y = t;
    }
    if (x != (unsigned char *)xv) memcpy((unsigned char *)xv + lo * e, x + lo * e, (hi - lo) * e);
    return 0;
}
