"""Pins for the CPU oracle (no GPU).

The oracle is an algorithm plus a canonical rule, so it is pinned against
things that do not come from it:
  * a recursive re-definition of the Benes network (input column, two
    half-size networks, output column) written here with numpy;
  * exhaustive checks at N = 2, 4, 8 (every permutation must be realised);
  * enumeration of ALL switch settings at N = 4 (2^6) and N = 8 (2^20): the
    network is rearrangeable, and among the settings that realise a given
    permutation exactly one obeys the canonical rule -- the oracle's;
  * closed forms that follow from the definition by induction (identity,
    cyclic shift by one);
  * hand-traced worked examples (tests/golden/worked_examples.txt);
  * an independent union-find 2-colouring of the constraint graph;
  * per-level invariants (sub-permutations are permutations, constraints hold).
"""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_1912_04050_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------
# helpers that do not use the oracle
# ----------------------------------------------------------------------------
def unpack(bits, n):
    """(2n-1, W) words -> (2n-1, N/2) array of 0/1, switch 0 first."""
    half = (1 << n) // 2
    b = np.asarray(bits, dtype=np.uint32).reshape(2 * n - 1, -1)
    sw = (b[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1
    sw = sw.reshape(2 * n - 1, -1)
    assert not sw[:, half:].any(), "padding bits must be zero"
    return sw[:, :half].astype(np.uint8)


def pack(sw, n):
    """inverse of unpack for arrays shaped (..., 2n-1, N/2)."""
    half = (1 << n) // 2
    W = max(1, (1 << n) // 64)
    pad = np.zeros(sw.shape[:-1] + (W * 32,), dtype=np.uint64)
    pad[..., :half] = sw
    words = (pad.reshape(sw.shape[:-1] + (W, 32)) << np.arange(32, dtype=np.uint64)).sum(-1)
    return words.astype(np.uint32)


def net(x, sw, n, level=0, first=0):
    """Recursive definition of the network, vectorised over a leading axis of
    settings.  x: (S, M) payload of one block; sw: (S, 2n-1, N/2) in {0,1};
    `first` is the block's first switch in every stage it owns."""
    M = x.shape[1]
    if M == 2:
        c = sw[:, n - 1, first].astype(bool)[:, None]
        return np.where(c, x[:, ::-1], x)
    H = M // 2
    cin = sw[:, level, first:first + H].astype(bool)
    a, b = x[:, 0::2], x[:, 1::2]
    upper = net(np.where(cin, b, a), sw, n, level + 1, first)
    lower = net(np.where(cin, a, b), sw, n, level + 1, first + H // 2)
    cout = sw[:, 2 * n - 2 - level, first:first + H].astype(bool)
    y = np.empty_like(x)
    y[:, 0::2] = np.where(cout, lower, upper)
    y[:, 1::2] = np.where(cout, upper, lower)
    return y


def realised_perm(sw, n):
    """Gather permutation realised by one setting sw (2n-1, N/2)."""
    x = np.arange(1 << n, dtype=np.int64)[None, :]
    return net(x, sw[None], n)[0]


class DSU:
    def __init__(self, m):
        self.p = list(range(m))

    def find(self, a):
        while self.p[a] != a:
            self.p[a] = self.p[self.p[a]]
            a = self.p[a]
        return a

    def union(self, a, b):
        a, b = self.find(a), self.find(b)
        if a != b:
            self.p[max(a, b)] = min(a, b)   # root = smallest index of the component


def loops_min_index(p):
    """For block-local gather permutation p: for each output j, the smallest
    output index of its constraint loop (edges: j~j^1 share an output switch;
    the outputs fed by inputs i and i^1 share an input switch)."""
    M = len(p)
    inv = [0] * M
    for j, v in enumerate(p):
        inv[int(v)] = j
    d = DSU(M)
    for j in range(0, M, 2):
        d.union(j, j + 1)
    for i in range(0, M, 2):
        d.union(inv[i], inv[i + 1])
    return [d.find(j) for j in range(M)], inv


def colouring_by_union_find(p):
    """Canonical 2-colouring without walking loops in order: breadth-first
    propagation of 'opposite colour' along both kinds of edges, seeded at each
    loop's smallest output with colour 0."""
    M = len(p)
    root, inv = loops_min_index(p)
    colour = [-1] * M
    for j0 in sorted(set(root)):
        colour[j0] = 0
        stack = [j0]
        while stack:
            j = stack.pop()
            for k in (j ^ 1, inv[int(p[j]) ^ 1]):
                if colour[k] < 0:
                    colour[k] = 1 - colour[j]
                    stack.append(k)
                else:
                    assert colour[k] == 1 - colour[j]
    return colour


def is_canonical(sw, n):
    """True iff, in every block of every level, the smallest output index of
    each constraint loop is served by the upper half.  Works from the setting
    alone: the block's realised permutation is rebuilt bottom-up."""
    def rec(level, first, M):
        if M == 2:
            c = int(sw[n - 1, first])
            return [c, 1 - c], True
        H = M // 2
        pu, ok_u = rec(level + 1, first, H)
        pl, ok_l = rec(level + 1, first + H // 2, H)
        p, half_of = [0] * M, [0] * M
        for j in range(M):
            t = j >> 1
            h = int(sw[2 * n - 2 - level, first + t]) ^ (j & 1)    # 0: from upper
            r = pu[t] if h == 0 else pl[t]                         # sub-network input
            cin = int(sw[level, first + r])
            p[j] = 2 * r + (cin ^ h)                               # upper gets 2r when straight
            half_of[j] = h
        root, _ = loops_min_index(p)
        ok = all(half_of[m] == 0 for m in set(root))
        return p, ok and ok_u and ok_l
    return rec(0, 0, 1 << n)[1]


def all_settings(n):
    """(2^S, 2n-1, N/2) array of every switch setting."""
    S = (2 * n - 1) * (1 << (n - 1))
    codes = np.arange(1 << S, dtype=np.uint32)
    sw = (codes[:, None] >> np.arange(S, dtype=np.uint32)[None, :]) & 1
    return sw.reshape(-1, 2 * n - 1, 1 << (n - 1)).astype(np.uint8)


def all_perms(N):
    return np.array(list(itertools.permutations(range(N))), dtype=np.uint32)


# ----------------------------------------------------------------------------
# apply: the oracle's flat stage loop equals the recursive definition
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 6, 7, 9])
def test_apply_matches_recursive_definition(n):
    rng = np.random.default_rng(100 + n)
    S, N = 16, 1 << n
    sw = rng.integers(0, 2, size=(S, 2 * n - 1, N // 2)).astype(np.uint8)
    x = rng.integers(0, 2 ** 32, size=(S, N), dtype=np.uint64).astype(np.uint32)
    want = net(x, sw, n)
    got = oracle.apply(pack(sw, n), x, n)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("dtype", [np.uint8, np.uint16, np.float32, np.uint64])
def test_apply_moves_whole_elements(dtype):
    n, rng = 6, np.random.default_rng(7)
    sw = rng.integers(0, 2, size=(1, 2 * n - 1, 32)).astype(np.uint8)
    x = rng.integers(0, 255, size=(1, 64)).astype(dtype)
    perm = realised_perm(sw[0], n)
    assert np.array_equal(oracle.apply(pack(sw, n), x, n)[0], x[0][perm])


# ----------------------------------------------------------------------------
# exhaustive: every permutation of N = 2, 4, 8 is routed exactly
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("n", [1, 2, 3])
def test_every_permutation_routes(n):
    N = 1 << n
    perms = all_perms(N)
    assert len(perms) == {2: 2, 4: 24, 8: 40320}[N]
    bits = oracle.route(perms, n)
    ident = np.tile(np.arange(N, dtype=np.uint32), (len(perms), 1))
    assert np.array_equal(oracle.apply(bits, ident, n), perms)
    # and through the recursive definition, which knows nothing of the oracle's apply
    sw = np.stack([unpack(b, n) for b in bits[:: max(1, len(perms) // 500)]])
    got = net(np.tile(np.arange(N), (len(sw), 1)), sw, n)
    assert np.array_equal(got, perms[:: max(1, len(perms) // 500)])


def test_n2_is_one_switch():
    assert oracle.route(np.array([0, 1], np.uint32), 1).tolist() == [[0]]
    assert oracle.route(np.array([1, 0], np.uint32), 1).tolist() == [[1]]


# ----------------------------------------------------------------------------
# all settings: rearrangeability and uniqueness of the canonical setting
# ----------------------------------------------------------------------------
def _group_settings(n):
    N = 1 << n
    sw = all_settings(n)
    out = net(np.tile(np.arange(N, dtype=np.int64), (len(sw), 1)), sw, n)
    key = (out * (N ** np.arange(N, dtype=np.int64))[None, :]).sum(1)
    return sw, out, key


def test_all_settings_n4_canonical_is_unique_and_is_the_oracle():
    n, N = 2, 4
    sw, out, key = _group_settings(n)
    assert len(np.unique(key)) == 24                      # rearrangeable
    counts = set()
    for perm in all_perms(N):
        k = int((perm.astype(np.int64) * (N ** np.arange(N))).sum())
        members = sw[key == k]
        counts.add(len(members))
        canon = [m for m in members if is_canonical(m, n)]
        assert len(canon) == 1
        assert np.array_equal(canon[0], unpack(oracle.route(perm, n), n))
    assert counts == {2, 4}                               # 2^(number of loops) settings each


def test_all_settings_n8_canonical_is_unique_and_is_the_oracle():
    n, N = 3, 8
    sw, out, key = _group_settings(n)
    uniq = np.unique(key)
    assert len(uniq) == 40320                             # rearrangeable: every permutation occurs
    order = np.argsort(key, kind="stable")
    skey = key[order]
    perms = all_perms(N)
    for perm in perms:                                    # every one of the 40320
        k = int((perm.astype(np.int64) * (N ** np.arange(N, dtype=np.int64))).sum())
        lo, hi = np.searchsorted(skey, k, "left"), np.searchsorted(skey, k, "right")
        members = sw[order[lo:hi]]
        assert len(members) >= 2
        canon = [m for m in members if is_canonical(m, n)]
        assert len(canon) == 1
        assert np.array_equal(canon[0], unpack(oracle.route(perm, n), n))


# ----------------------------------------------------------------------------
# closed forms
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("n", [1, 2, 3, 5, 8, 12, 16])
def test_identity_gives_all_straight(n):
    assert not oracle.route(inputs.identity_perm(n), n).any()


@pytest.mark.parametrize("n", [2, 3, 4, 7, 10, 13])
def test_cyclic_shift_closed_form(n):
    """pi[j] = j+1 mod N.  All even outputs are fed by odd inputs, so the single
    loop puts every even output up: output switches straight, every input
    switch crossed, upper sub-permutation = identity, lower = the same shift at
    half size.  By induction only the last block of each level is not the
    identity; the last middle switch is crossed."""
    N = 1 << n
    want = np.zeros((2 * n - 1, N // 2), dtype=np.uint8)
    for level in range(n - 1):
        M = N >> level
        want[level, N // 2 - M // 2:] = 1
    want[n - 1, N // 2 - 1] = 1
    assert np.array_equal(unpack(oracle.route(inputs.shift_perm(n, 1), n), n), want)


def test_worked_examples():
    with open(os.path.join(GOLDEN, "worked_examples.txt")) as f:
        lines = [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(lines) == 4
    for ln in lines:
        perm_s, stages_s = ln.split(";")
        perm = np.array(perm_s.split(), dtype=np.uint32)
        n = int(np.log2(len(perm)))
        want = np.array([st.split() for st in stages_s.split("|")], dtype=np.uint8)
        assert want.shape == (2 * n - 1, len(perm) // 2)
        assert np.array_equal(unpack(oracle.route(perm, n), n), want)


# ----------------------------------------------------------------------------
# independent colouring, invariants at every level
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("n,seed", [(2, 0), (3, 1), (4, 2), (6, 3), (8, 4), (10, 5)])
def test_colours_match_union_find_at_every_level(n, seed):
    N = 1 << n
    perm = inputs.random_perm(n, seed)
    _, tp, tc = oracle.route_trace(perm, n)
    for level in range(n - 1):
        M = N >> level
        for base in range(0, N, M):
            want = colouring_by_union_find(tp[level, base:base + M].tolist())
            assert tc[level, base:base + M].tolist() == want


@pytest.mark.parametrize("n,kind", [(5, "random"), (9, "random"), (12, "random"), (16, "random"),
                                    (12, "sattolo"), (12, "bitrev"), (12, "transpose"), (12, "shift1")])
def test_level_invariants(n, kind):
    N = 1 << n
    perm = inputs.random_perm(n, 40 + n) if kind == "random" else inputs.structured_perms(n)[kind]
    bits, tp, tc = oracle.route_trace(perm, n)
    sw = unpack(bits, n)
    assert np.array_equal(tp[0], perm)
    for level in range(n - 1):
        M, H = N >> level, (N >> level) // 2
        P = tp[level].reshape(-1, M).astype(np.int64)
        C = tc[level].reshape(-1, M).astype(np.int64)
        # every block-local sub-permutation is a permutation of [0, M)
        assert np.array_equal(np.sort(P, axis=1), np.tile(np.arange(M), (P.shape[0], 1)))
        # the two outputs of an output switch use different halves
        assert np.array_equal(C[:, 0::2] + C[:, 1::2], np.ones((P.shape[0], H), dtype=np.int64))
        # the two inputs of an input switch use different halves
        cin = np.empty_like(C)
        np.put_along_axis(cin, P, C, axis=1)           # cin[p[j]] = colour[j]
        assert np.array_equal(cin[:, 0::2] + cin[:, 1::2], np.ones((P.shape[0], H), dtype=np.int64))
        # canonical rule => output switch 0 of every block is straight
        assert not sw[2 * n - 2 - level].reshape(-1, H)[:, 0].any()
        # stage bits are the colours of the even outputs / of the outputs fed by even inputs
        assert np.array_equal(sw[2 * n - 2 - level].reshape(-1, H), C[:, 0::2])
        assert np.array_equal(sw[level].reshape(-1, H), cin[:, 0::2])
        # next level's sub-permutations: upper half then lower half, each in switch order
        nxt = tp[level + 1].reshape(-1, M)
        for h in (0, 1):
            sel = np.where(C == h)
            got = nxt[:, h * H:(h + 1) * H]
            want = (P[sel] >> 1).reshape(-1, H)      # row-major = ascending j within a block
            assert np.array_equal(got, want)
    # middle stage: crossed iff output 0 of the 2-block takes input 1
    assert np.array_equal(sw[n - 1], tp[n - 1].reshape(-1, 2)[:, 0])


@pytest.mark.parametrize("n,kind", [(14, "random"), (14, "sattolo"), (14, "bitrev"),
                                    (14, "transpose"), (14, "shift1"), (14, "identity"), (17, "random")])
def test_identity_payload_reproduces_pi(n, kind):
    perm = inputs.random_perm(n, n) if kind == "random" else inputs.structured_perms(n)[kind]
    bits = oracle.route(perm, n)
    assert np.array_equal(oracle.apply(bits, inputs.identity_perm(n), n), perm)
    # recursive definition agrees as well
    assert np.array_equal(realised_perm(unpack(bits, n), n), perm)


def test_bit_linear_permutations_have_short_loops():
    """Bit reversal and transposition are linear over GF(2): every constraint
    loop has at most 4 outputs.  A structural fact the pass-count logic relies on."""
    for kind in ("bitrev", "transpose"):
        p = inputs.structured_perms(10)[kind].tolist()
        root, _ = loops_min_index(p)
        assert max(np.bincount(root)) <= 4


# ---- the in-place ("butterfly") form of the settings -------------------------------------
def test_butterfly_form_routes_every_small_permutation():
    """The re-indexed settings, run as an in-place network (swap x[u], x[u | 2^i] where the
    bit is set; no movement between stages), realise the permutation: all of N = 2, 4, 8."""
    import itertools
    for n in (1, 2, 3):
        x = np.arange(1 << n) * 7 + 3
        for p in itertools.permutations(range(1 << n)):
            perm = np.array(p, dtype=np.uint32)
            bf = oracle.export_butterfly(oracle.route(perm, n), n)
            assert np.array_equal(oracle.apply_butterfly(bf, x, n), x[perm]), p


@pytest.mark.parametrize("n", [4, 5, 6, 7, 9, 12])
def test_butterfly_form_random(n):
    perm = inputs.random_perm(n, 50 + n)
    bits = oracle.route(perm, n)
    bf = oracle.export_butterfly(bits, n)
    x = np.arange(1 << n, dtype=np.uint64) * 11 + 1
    assert np.array_equal(oracle.apply_butterfly(bf, x, n), x[perm])
    # a re-indexing: every stage keeps its number of crossed switches
    for r in range(2 * n - 1):
        assert int(np.unpackbits(bf[r].view(np.uint8)).sum()) == int(np.unpackbits(bits[r].view(np.uint8)).sum())
    # identity: nothing crossed in either form
    ident = inputs.identity_perm(n)
    assert not oracle.export_butterfly(oracle.route(ident, n), n).any()


def _pack_rows(rows):
    """list of 0/1 lists (switch 0 first) -> (len, 1) uint32 words"""
    return np.array([[sum(b << i for i, b in enumerate(r))] for r in rows], dtype=np.uint32)


def test_butterfly_bit_order_hand_traced_rows():
    """tests/golden/butterfly_rows_n8.txt: the order of the bits inside a row, traced by hand."""
    n = 3
    with open(os.path.join(GOLDEN, "butterfly_rows_n8.txt")) as f:
        lines = [ln for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(lines) == 2
    for ln in lines:
        rec, inplace = ([[int(v) for v in row.split()] for row in side.split("|")] for side in ln.split(";"))
        assert np.array_equal(oracle.export_butterfly(_pack_rows(rec), n), _pack_rows(inplace))


def _bitrev(v, width):
    r = 0
    for i in range(width):
        r |= ((v >> i) & 1) << (width - 1 - i)
    return r


@pytest.mark.parametrize("n", [2, 3, 4, 6, 9, 11])
def test_butterfly_bit_order_closed_form(n):
    """Block b of level l (its bits are the up/down choices of levels 0..l-1, first choice on
    top) keeps choice k in bit k of the in-place position, and position r of the block sits
    above them: in-place position = r << l | reverse_l(b).  So recursive switch w = (b, s) of
    level l is in-place switch s << l | reverse_l(b), on both sides of the network."""
    rng = np.random.default_rng(n)
    N, W = 1 << n, max(1, (1 << n) // 64)
    bits = rng.integers(0, 2, size=(2 * n - 1, N // 2), dtype=np.uint8)
    want = np.zeros_like(bits)
    for r in range(2 * n - 1):
        l = r if r <= n - 1 else 2 * n - 2 - r
        per_block = 1 << (n - l - 1)
        for w in range(N // 2):
            b, s = w // per_block, w % per_block
            want[r, (s << l) | _bitrev(b, l)] = bits[r, w]

    def pack(a):
        full = np.zeros((2 * n - 1, W * 32), dtype=np.uint8)
        full[:, :N // 2] = a
        return np.packbits(full, axis=1, bitorder="little").view(np.uint32).reshape(2 * n - 1, W)

    assert np.array_equal(oracle.export_butterfly(pack(bits), n), pack(want))


# ---- range-restricted entry points (the benchmark's all-core leg) ------------------------
@pytest.mark.parametrize("n", [1, 2, 5, 6, 7, 8, 11, 15])
@pytest.mark.parametrize("threads", [1, 2, 3, 16])
def test_parts_reproduce_the_whole(n, threads):
    """Top levels on one thread, the sub-networks below on several: same words, same payload."""
    perm = inputs.random_perm(n, 300 + n)
    bits = oracle.route(perm, n)
    assert np.array_equal(oracle.route_parallel(perm, n, threads), bits)
    x = inputs.payload_u64(1 << n, n)
    out = oracle.apply_parallel(bits, x, n, threads)
    assert np.array_equal(out, oracle.apply(bits, x, n))
    assert np.array_equal(out, x[perm])


def test_parts_batched():
    perm = inputs.random_perm_batch(7, 21, seed0=3)
    bits = oracle.route(perm, 7)
    assert np.array_equal(oracle.route_parallel(perm, 7, 4), bits)
    x = np.arange(21 << 7, dtype=np.uint32).reshape(21, -1)
    assert np.array_equal(oracle.apply_parallel(bits, x, 7, 4), oracle.apply(bits, x, 7))
