"""GPU parity: the CUDA library, called through its C ABI, against the CPU
oracle on the same seeded inputs.  Integer / bit work: the bar is bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_1912_04050_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.load()
    yield
    binding.benes_release_workspace()


def dev(a: np.ndarray) -> torch.Tensor:
    """numpy (uint32/uint64/float32) -> CUDA tensor with the same bytes."""
    view = {4: np.int32, 8: np.int64}[a.dtype.itemsize]
    return torch.from_numpy(np.ascontiguousarray(a).view(view)).cuda()


def host(t: torch.Tensor, dtype) -> np.ndarray:
    return t.cpu().numpy().view(dtype)


def gpu_route(perm: np.ndarray, n: int) -> np.ndarray:
    p = dev(perm)
    batch = perm.size >> n
    bits = torch.full((binding.benes_switch_words(n, batch),), -1, dtype=torch.int32, device="cuda")
    binding.benes_route(p, n, batch, bits)
    torch.cuda.synchronize()
    shape = (2 * n - 1, max(1, (1 << n) // 64))
    return host(bits, np.uint32).reshape(((batch,) if perm.ndim == 2 else ()) + shape)


def gpu_apply(bits: np.ndarray, x: np.ndarray, n: int) -> np.ndarray:
    batch = x.size >> n
    out = torch.empty_like(dev(x))
    binding.benes_apply_ex(dev(bits), dev(x), out, x.dtype.itemsize, n, batch)
    torch.cuda.synchronize()
    return host(out, x.dtype).reshape(x.shape)


# ---- route ------------------------------------------------------------------
@pytest.mark.parametrize("n", list(range(1, 21)))
def test_route_random_every_size(n):
    """n up to benes_fused_log2m() run in one CTA; larger n take HBM levels first, then the fused tail."""
    perm = inputs.random_perm(n, 100 + n)
    assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n))


@pytest.mark.parametrize("n,batch", [(1, 5), (2, 7), (3, 33), (5, 64), (6, 3), (8, 1000), (9, 77), (11, 5),
                                     (13, 3), (14, 3), (15, 2), (16, 5), (17, 3)])
def test_route_batched(n, batch):
    perm = inputs.random_perm_batch(n, batch, seed0=7 * n)
    assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n))


@pytest.mark.parametrize("n", [4, 9, 10, 13, 15, 16, 18, 20])
@pytest.mark.parametrize("kind", ["identity", "shift1", "bitrev", "transpose", "sattolo"])
def test_route_structured(n, kind):
    perm = inputs.structured_perms(n)[kind]
    assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n))


def test_route_exhaustive_n8():
    """All 40320 permutations of N = 8 in one batched call."""
    import itertools
    perms = np.array(list(itertools.permutations(range(8))), dtype=np.uint32)
    assert np.array_equal(gpu_route(perms, 3), oracle.route(perms, 3))


# ---- loop-labelling variants: all must give the oracle's bits -------------------
@pytest.fixture
def labelling_options():
    k0 = binding.benes_get_option(binding.OPT_SAMPLE_LOG2K)
    c0 = binding.benes_get_option(binding.OPT_WALK_CAP)
    yield
    binding.benes_set_option(binding.OPT_SAMPLE_LOG2K, k0)
    binding.benes_set_option(binding.OPT_WALK_CAP, c0)


@pytest.fixture(params=[1, 0], ids=["fused", "per_stage"])
def apply_mode(request):
    """Both payload-apply paths: several stages per pass, and one stage per pass."""
    a0 = binding.benes_get_option(binding.OPT_APPLY_FUSED)
    binding.benes_set_option(binding.OPT_APPLY_FUSED, request.param)
    yield request.param
    binding.benes_set_option(binding.OPT_APPLY_FUSED, a0)


@pytest.mark.parametrize("kappa", [0, 2, 3, 5, 8])
def test_route_every_ruler_spacing(kappa, labelling_options):
    """0 = pointer jumping over all outputs; otherwise one ruler per 2^kappa switches."""
    binding.benes_set_option(binding.OPT_SAMPLE_LOG2K, kappa)
    for n in (16, 19):
        perm = inputs.random_perm(n, 40 + n)
        assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n))
    n = 17
    for kind, perm in inputs.structured_perms(n).items():
        assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n)), kind
    perm = inputs.random_perm_batch(16, 3, seed0=9)
    assert np.array_equal(gpu_route(perm, 16), oracle.route(perm, 16))


@pytest.mark.parametrize("mode", [0, 2])
@pytest.mark.parametrize("kappa,cap", [(None, None), (2, None), (5, None), (None, 3)])
def test_route_one_or_two_walks_per_thread(mode, kappa, cap, labelling_options):
    """At packed levels a thread advances one walk or the two walks of a ruler switch
    (the default picks by size; both forced here at sizes that take either)."""
    w0 = binding.benes_get_option(binding.OPT_WALK_PAIRS)
    binding.benes_set_option(binding.OPT_WALK_PAIRS, mode)
    try:
        if kappa is not None:
            binding.benes_set_option(binding.OPT_SAMPLE_LOG2K, kappa)
        if cap is not None:
            binding.benes_set_option(binding.OPT_WALK_CAP, cap)
        for n, batch in ((16, 3), (18, 1), (20, 1), (19, 5)):
            perm = inputs.random_perm_batch(n, batch, seed0=300 + n) if batch > 1 else inputs.random_perm(n, 300 + n)
            assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n)), (n, batch)
        for kind, perm in inputs.structured_perms(17).items():
            assert np.array_equal(gpu_route(perm, 17), oracle.route(perm, 17)), kind
    finally:
        binding.benes_set_option(binding.OPT_WALK_PAIRS, w0)


def test_route_random_option_combinations(labelling_options):
    """Seeded draws over sizes, batches, input kinds and every option that changes the path
    (ruler spacing, hop limit, walks per thread, clusters, inverse form, chunking): the bits never
    depend on the path."""
    rng = np.random.default_rng(2024)
    keys = (binding.OPT_WALK_PAIRS, binding.OPT_CLUSTER, binding.OPT_INVERSE_PARTITIONED, binding.OPT_CHUNK_LOG2)
    old = [binding.benes_get_option(k) for k in keys]
    try:
        for trial in range(48):
            n = int(rng.integers(15, 21))
            batch = int(rng.choice([1, 1, 2, 3, 5])) if n <= 18 else 1
            kind = str(rng.choice(["random", "random", "random", "sattolo", "shift1", "bitrev", "identity"]))
            opts = {binding.OPT_SAMPLE_LOG2K: int(rng.choice([0, 2, 3, 4, 4, 5, 6, 8])),
                    binding.OPT_WALK_CAP: int(rng.choice([1, 7, 100, 1 << 14, 1 << 14])),
                    binding.OPT_WALK_PAIRS: int(rng.integers(0, 3)),
                    binding.OPT_CLUSTER: int(rng.integers(0, 2)),
                    binding.OPT_INVERSE_PARTITIONED: int(rng.integers(0, 2)),
                    binding.OPT_CHUNK_LOG2: int(rng.choice([30, 30, 17, 18]))}
            for k, v in opts.items():
                binding.benes_set_option(k, v)
            if kind == "random":
                perm = inputs.random_perm_batch(n, batch, seed0=5000 + trial)
            else:
                perm = np.tile(inputs.structured_perms(n)[kind], (batch, 1))
            assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n)), (trial, n, batch, kind, opts)
    finally:
        for k, v in zip(keys, old):
            binding.benes_set_option(k, v)


@pytest.fixture
def cluster_mode():
    c0 = binding.benes_get_option(binding.OPT_CLUSTER)
    binding.benes_set_option(binding.OPT_CLUSTER, 1)
    yield
    binding.benes_set_option(binding.OPT_CLUSTER, c0)


@pytest.mark.parametrize("n,batch", [(16, 1), (16, 3), (16, 64), (17, 1), (17, 3), (17, 64), (18, 5), (20, 1), (22, 1)])
def test_route_blocks_of_2p16_in_clusters_of_two_ctas(n, batch, cluster_mode):
    """Whole permutations of 2^16 (one cluster each) and the tails of larger ones."""
    perm = inputs.random_perm_batch(n, batch, seed0=500 + n + batch)
    assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n))


@pytest.mark.parametrize("n", [16, 17, 19])
@pytest.mark.parametrize("kind", ["identity", "shift1", "bitrev", "transpose", "sattolo"])
def test_route_structured_in_clusters(n, kind, cluster_mode):
    perm = inputs.structured_perms(n)[kind]
    assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n))


@pytest.mark.parametrize("cap", [1, 3, 40])
def test_route_walks_that_give_up_fall_back_to_full_pointer_jumping(cap, labelling_options):
    """With a tiny hop limit almost every level raises its gate and is relabelled
    by the full pointer-jumping kernels; the bits must not change."""
    binding.benes_set_option(binding.OPT_WALK_CAP, cap)
    for n in (16, 18):
        for kind, perm in inputs.structured_perms(n).items():
            assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n)), kind
        perm = inputs.random_perm(n, 60 + n)
        assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n))


@pytest.mark.parametrize("kappa,cap", [(None, None), (2, None), (4, None), (None, 12)])
@pytest.mark.parametrize("n,batch", [(18, 3), (19, 3), (20, 5), (19, 7)])
def test_route_batch_not_a_power_of_two_with_resampled_lists(n, batch, kappa, cap, labelling_options):
    """Blocks of 2^(15 + kappa) outputs and more have their contracted list sampled
    again; the list of a batch that is not a power of two is not one either, so
    every list index has to be bounded by the list's length, not by a mask."""
    if kappa is not None:
        binding.benes_set_option(binding.OPT_SAMPLE_LOG2K, kappa)
    if cap is not None:
        binding.benes_set_option(binding.OPT_WALK_CAP, cap)
    perm = inputs.random_perm_batch(n, batch, seed0=31 * n + batch)
    assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n))


@pytest.mark.parametrize("n,batch", [(22, 1), (16, 64), (17, 64), (23, 1), (16, 65)])
def test_route_bucketed_inverse(n, batch):
    """batch * N >= 2^22 in whole multiples of 2^18 takes the two-pass inverse at
    level 0 (the last case does not and takes the plain scatter); with the option
    off every case takes the plain scatter.  Same bits either way."""
    perm = inputs.random_perm_batch(n, batch, seed0=3 * n) if batch > 1 else inputs.random_perm(n, 77)
    want = oracle.route(perm, n)
    assert np.array_equal(gpu_route(perm, n), want)
    binding.benes_set_option(binding.OPT_INVERSE_PARTITIONED, 0)
    try:
        assert np.array_equal(gpu_route(perm, n), want)
    finally:
        binding.benes_set_option(binding.OPT_INVERSE_PARTITIONED, 1)


# ---- apply ------------------------------------------------------------------
@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 6, 7, 10, 12, 13, 14, 16, 19, 21])
@pytest.mark.parametrize("dtype", [np.uint32, np.uint64])
def test_apply_random_settings(n, dtype, apply_mode):
    """Arbitrary switch settings (not produced by route): checks wiring and layout alone."""
    rng = np.random.default_rng(n)
    batch = 3 if n < 19 else 1
    W = max(1, (1 << n) // 64)
    bits = rng.integers(0, 2 ** 32, size=(batch, 2 * n - 1, W), dtype=np.uint64).astype(np.uint32)
    if n < 6:
        bits &= np.uint32((1 << (1 << (n - 1))) - 1)
    x = rng.integers(0, 2 ** 63, size=(batch, 1 << n), dtype=np.uint64).astype(dtype)
    assert np.array_equal(gpu_apply(bits, x, n), oracle.apply(bits, x, n))


def test_apply_does_not_touch_input():
    n = 12
    perm = inputs.random_perm(n, 1)
    x = inputs.payload_u64(1 << n, 9)
    dx = dev(x)
    bits = dev(oracle.route(perm, n))
    out = torch.empty_like(dx)
    binding.benes_apply_ex(bits, dx, out, 8, n, 1)
    torch.cuda.synchronize()
    assert np.array_equal(host(dx, np.uint64), x)
    assert np.array_equal(host(out, np.uint64), x[perm])


# ---- the five configurations ------------------------------------------------------
def test_config1_n1024_identity_payload():
    n = 10
    perm = inputs.random_perm(n, 0)
    bits = gpu_route(perm, n)
    assert bits.shape == (19, 16)
    assert np.array_equal(bits, oracle.route(perm, n))
    out = gpu_apply(bits, inputs.identity_perm(n), n)
    assert np.array_equal(out, perm)
    assert np.array_equal(out, oracle.apply(bits, inputs.identity_perm(n), n))


def test_config2_batch_16384_of_256():
    n, batch = 8, 16384
    perm = inputs.random_perm_batch(n, batch, seed0=0)
    bits = gpu_route(perm, n)
    assert bits.shape == (batch, 15, 4)
    assert np.array_equal(bits, oracle.route(perm, n))
    ident = np.tile(inputs.identity_perm(n), (batch, 1))
    assert np.array_equal(gpu_apply(bits, ident, n), perm)


def test_config3_n2p20_fp32_payload():
    n = 20
    perm = inputs.random_perm(n, 1)
    bits = gpu_route(perm, n)
    assert np.array_equal(bits, oracle.route(perm, n))
    x = inputs.payload_f32(1 << n, 1)
    out = gpu_apply(bits, x, n)
    assert np.array_equal(out.view(np.uint32), x[perm].view(np.uint32))
    assert np.array_equal(out.view(np.uint32), oracle.apply(bits, x, n).view(np.uint32))


@pytest.mark.parametrize("kind", ["identity", "shift1", "bitrev", "transpose", "sattolo"])
def test_config5_structured_n2p24(kind):
    n = 24
    perm = inputs.structured_perms(n)[kind]
    bits = gpu_route(perm, n)
    assert np.array_equal(bits, oracle.route(perm, n))
    assert np.array_equal(gpu_apply(bits, inputs.identity_perm(n), n), perm)


def test_config4_n2p26_u64_payload():
    """Headline size, in the launch configuration the benchmark times.  The
    oracle routes the full permutation once (about two minutes on one core)."""
    n = 26
    perm = inputs.random_perm(n, 2)
    bits = gpu_route(perm, n)
    x = inputs.payload_u64(1 << n, 2)
    out = gpu_apply(bits, x, n)
    assert np.array_equal(out, x[perm])
    assert np.array_equal(bits, oracle.route(perm, n))


def test_route_n2p27_matches_the_oracle():
    """One size above the headline, word for word (the oracle needs about two minutes)."""
    n = 27
    perm = inputs.random_perm(n, 7)
    bits = gpu_route(perm, n)
    assert np.array_equal(bits, oracle.route(perm, n))
    binding.benes_release_workspace()


@pytest.mark.parametrize("n_elems,batch", [(1, 2), (3, 4), (5, 3), (100, 5), (1000, 2), (4097, 3),
                                           (40000, 2), (100000, 1), (300001, 1)])
def test_sizes_that_are_not_a_power_of_two(n_elems, batch):
    """The padded entry points equal routing the permutation extended by fixed
    points, and the routed payload is the gather of the first n_elems elements."""
    n = binding.benes_padded_log2n(n_elems)
    assert (1 << n) >= n_elems and (n == 1 or (1 << (n - 1)) < n_elems)
    perm = inputs.random_perm_any(n_elems, batch, seed0=n_elems)
    want = oracle.route(inputs.pad_with_fixed_points(perm, n), n)
    bits = torch.full((binding.benes_switch_words(n, batch),), -1, dtype=torch.int32, device="cuda")
    binding.benes_route_padded(dev(perm), n_elems, batch, bits)
    torch.cuda.synchronize()
    assert np.array_equal(host(bits, np.uint32).reshape(want.shape), want)
    for dtype in (np.uint32, np.uint64):
        x = np.random.default_rng(n_elems).integers(0, 2 ** 63, size=(batch, n_elems), dtype=np.uint64).astype(dtype)
        out = torch.empty_like(dev(x))
        binding.benes_apply_padded(bits, dev(x), out, x.dtype.itemsize, n_elems, batch)
        torch.cuda.synchronize()
        assert np.array_equal(host(out, dtype).reshape(x.shape), np.take_along_axis(x, perm.astype(np.int64), axis=1))


@pytest.mark.parametrize("n", [17, 19, 21])
def test_route_many_seeds_and_repeats(n):
    """The walks claim switches with atomics in whatever order the hardware runs
    them; the result must not depend on that order: several seeds, each routed
    three times."""
    for seed in range(6):
        perm = inputs.random_perm(n, 1000 * n + seed)
        want = oracle.route(perm, n)
        for _ in range(3):
            assert np.array_equal(gpu_route(perm, n), want), (n, seed)


@pytest.mark.parametrize("n,batch", [(1, 3), (2, 5), (3, 7), (5, 4), (6, 3), (7, 2), (10, 3), (13, 2), (16, 2), (20, 1)])
def test_export_butterfly(n, batch):
    """The in-place form of the settings, against the oracle's re-indexing (bit-exact)."""
    perm = inputs.random_perm_batch(n, batch, seed0=11 * n)
    bits = oracle.route(perm, n)
    out = torch.full((binding.benes_switch_words(n, batch),), -1, dtype=torch.int32, device="cuda")
    binding.benes_export_butterfly(dev(bits), out, n, batch)
    torch.cuda.synchronize()
    got = host(out, np.uint32).reshape(bits.shape)
    for b in range(batch):
        assert np.array_equal(got[b], oracle.export_butterfly(bits[b], n)), b
    x = np.arange(1 << n, dtype=np.uint64) * 3 + 1
    assert np.array_equal(oracle.apply_butterfly(got[0], x, n), x[perm[0]])


def test_route_batch_in_chunks():
    """A batch larger than the chunk limit is routed chunk by chunk (whole
    permutations per chunk) with a workspace sized for one chunk."""
    n, batch = 16, 7
    perm = inputs.random_perm_batch(n, batch, seed0=21)
    want = oracle.route(perm, n)
    full = binding.benes_route_workspace_bytes(n, batch)
    binding.benes_set_option(binding.OPT_CHUNK_LOG2, 17)            # two permutations per chunk
    try:
        assert binding.benes_route_workspace_bytes(n, batch) < full / 3
        assert np.array_equal(gpu_route(perm, n), want)
        binding.benes_set_option(binding.OPT_CHUNK_LOG2, 16)        # one per chunk
        assert np.array_equal(gpu_route(perm, n), want)
    finally:
        binding.benes_set_option(binding.OPT_CHUNK_LOG2, 30)
    assert np.array_equal(gpu_route(perm, n), want)


@pytest.mark.parametrize("n", [27, 28], ids=["n2p27", "n2p28"])
def test_route_large_properties(n):
    """Beyond what the oracle finishes in reasonable time: the routed identity
    payload must reproduce the permutation, and under the canonical rule the
    first output switch of every block of every level is straight (output 0 of a
    block is the smallest output of its loop).  2^27 is the largest input whose
    level-0 inverse uses buckets of 2^15 entries, 2^28 uses buckets of 2^18."""
    perm = inputs.random_perm(n, 5)
    d_perm = dev(perm)
    bits = torch.empty(binding.benes_switch_words(n, 1), dtype=torch.int32, device="cuda")
    binding.benes_route(d_perm, n, 1, bits)
    ident = torch.arange(1 << n, dtype=torch.int32, device="cuda")
    out = torch.empty_like(ident)
    binding.benes_apply_ex(bits, ident, out, 4, n, 1)
    torch.cuda.synchronize()
    assert torch.equal(out, d_perm)
    del ident, out, d_perm
    W = (1 << n) // 64
    b = host(bits, np.uint32).reshape(2 * n - 1, W)
    for level in range(n - 1):
        half = (1 << (n - level)) // 2                  # switches per block
        first = np.arange(1 << level, dtype=np.int64) * half
        stage = b[2 * n - 2 - level]
        assert not ((stage[first >> 5] >> (first & 31).astype(np.uint32)) & 1).any(), level
    binding.benes_release_workspace()


def test_route_maximum_size_properties():
    """N = 2^30, the largest size the ABI accepts (32-bit flat indices): same two
    properties.  The permutation is drawn on the device (torch.randperm with a fixed
    seed): the host generator would take minutes at this size, and no oracle value
    is involved."""
    n = 30
    torch.manual_seed(30)
    d_perm = torch.randperm(1 << n, device="cuda", dtype=torch.int32)
    bits = torch.empty(binding.benes_switch_words(n, 1), dtype=torch.int32, device="cuda")
    binding.benes_route(d_perm, n, 1, bits)
    ident = torch.arange(1 << n, dtype=torch.int32, device="cuda")
    out = torch.empty_like(ident)
    binding.benes_apply_ex(bits, ident, out, 4, n, 1)
    torch.cuda.synchronize()
    assert torch.equal(out, d_perm)
    del ident, out, d_perm
    rows = bits.view(2 * n - 1, (1 << n) // 64)
    for level in range(n - 1):
        half = (1 << (n - level)) // 2                  # switches per block
        first = torch.arange(1 << level, device="cuda", dtype=torch.int64) * half
        words = rows[2 * n - 2 - level][first >> 5].to(torch.int64) & 0xFFFFFFFF
        assert not bool(((words >> (first & 31)) & 1).any()), level
    del rows, bits
    binding.benes_release_workspace()
    torch.cuda.empty_cache()


# ---- host-buffer entry points, validation, robustness -------------------------------------------
@pytest.mark.parametrize("n,batch,pinned", [(15, 2, False), (17, 3, False), (18, 1, True), (23, 1, True), (23, 1, False)])
def test_host_entry_points(n, batch, pinned):
    """Host buffers in and out; above the in-CTA size the copies are overlapped with
    the levels (the permutation arrives in pieces from N = 2^23 on)."""
    perm = inputs.random_perm_batch(n, batch, seed0=5)
    bits = np.full((batch, 2 * n - 1, (1 << n) // 64), 0xAAAAAAAA, dtype=np.uint32)
    if pinned:
        perm_t = torch.from_numpy(perm.view(np.int32)).pin_memory()
        bits_t = torch.from_numpy(bits.view(np.int32)).pin_memory()
        binding.benes_route_host(perm_t, n, batch, bits_t)
        bits = bits_t.numpy().view(np.uint32)
    else:
        binding.benes_route_host(perm, n, batch, bits)
    assert np.array_equal(bits, oracle.route(perm, n))
    x = inputs.payload_u64(batch << n, 4).reshape(batch, -1)
    out = np.empty_like(x)
    binding.benes_apply_host(bits, x, out, 8, n, batch)
    assert np.array_equal(out, np.take_along_axis(x, perm.astype(np.int64), axis=1))
    # a second call right away reuses the side stream and the workspace
    bits2 = np.zeros_like(bits)
    binding.benes_route_host(perm, n, batch, bits2)
    assert np.array_equal(bits2, bits)


@pytest.mark.parametrize("n,batch,dtype,want_bits", [(23, 1, np.uint64, True), (24, 1, np.uint32, True),
                                                     (23, 2, np.uint64, False), (18, 3, np.uint64, True),
                                                     (15, 2, np.uint32, False), (25, 1, np.uint64, True)])
def test_route_apply_host_in_one_call(n, batch, dtype, want_bits):
    """Permutation and payload in, routed payload (and, if wanted, the switch words) out; from
    2^23 elements on the payload arrives while the levels run and the words never pass through
    host memory."""
    perm = inputs.random_perm_batch(n, batch, seed0=600 + n)
    x = inputs.payload_u64(batch << n, 8).reshape(batch, -1)
    if dtype == np.uint32:
        x = (x >> np.uint64(32)).astype(np.uint32)
    perm_t = torch.from_numpy(perm.view(np.int32)).pin_memory()
    x_t = torch.from_numpy(x.view({4: np.int32, 8: np.int64}[x.dtype.itemsize])).pin_memory()
    out_t = torch.full_like(x_t, -1).pin_memory()
    bits_t = torch.full((batch, 2 * n - 1, (1 << n) // 64), 0x33333333, dtype=torch.int32).pin_memory() if want_bits else None
    for _ in range(2):          # the second call reuses streams, events and the workspace
        out_t.fill_(-1)
        binding.benes_route_apply_host(perm_t, x_t, out_t, x.dtype.itemsize, n, batch, bits_t)
        assert np.array_equal(out_t.numpy().view(dtype), np.take_along_axis(x, perm.astype(np.int64), axis=1))
    if want_bits:
        want = oracle.route(perm, n) if n <= 24 else gpu_route(perm, n)
        assert np.array_equal(bits_t.numpy().view(np.uint32), want)
    binding.benes_release_workspace()


def test_route_host_split_tail_matches_device_path():
    """From 592 blocks of 2^15 on (N = 2^25 here) the host entry point finishes the
    in-CTA levels in two launches and copies the first one's columns home while the
    second runs.  Same words as the device entry point (whose result at this scale
    is compared with the oracle in test_config4)."""
    n = 25
    perm = inputs.random_perm(n, 9)
    want = gpu_route(perm, n)
    perm_t = torch.from_numpy(perm.view(np.int32)).pin_memory()
    bits_t = torch.full((2 * n - 1, (1 << n) // 64), 0x55555555, dtype=torch.int32).pin_memory()
    binding.benes_route_host(perm_t, n, 1, bits_t)
    assert np.array_equal(bits_t.numpy().view(np.uint32).reshape(want.shape), want)
    binding.benes_release_workspace()


def test_apply_host_piped_u32():
    """Payloads of 64 MiB and more go through benes_apply_host in parts (first pass
    as the parts arrive, last pass handing finished parts to the copy stream)."""
    n = 24
    perm = inputs.random_perm(n, 13)
    bits = gpu_route(perm, n)
    x = inputs.payload_u64(1 << (n - 1), 6).view(np.uint32).copy()
    out = np.full_like(x, 0xDEADBEEF)
    binding.benes_apply_host(bits, x, out, 4, n, 1)
    assert np.array_equal(out, x[perm.astype(np.int64)])
    binding.benes_release_workspace()


def test_caller_workspace_is_used_and_checked():
    n = binding.benes_fused_log2m() + 2
    perm = inputs.random_perm(n, 11)
    need = binding.benes_route_workspace_bytes(n, 1)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    try:
        binding.benes_set_workspace(ws)
        assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n))
        binding.benes_set_workspace(ws, 4096)       # too small for this call
        with pytest.raises(binding.BenesError) as e:
            gpu_route(perm, n)
        assert e.value.status == binding.BENES_ERR_NOMEM
    finally:
        binding.benes_set_workspace(None)


@pytest.mark.parametrize("n,batch", [(3, 4), (8, 10), (14, 2)])
def test_validate_perm(n, batch):
    perm = inputs.random_perm_batch(n, batch, seed0=1)
    assert binding.benes_validate_perm(dev(perm), n, batch)
    bad = perm.copy()
    bad[batch - 1, 3] = bad[batch - 1, 4]           # a duplicate
    assert not binding.benes_validate_perm(dev(bad), n, batch)
    bad = perm.copy()
    bad[0, 0] = 1 << n                              # out of range
    assert not binding.benes_validate_perm(dev(bad), n, batch)


@pytest.mark.parametrize("n", [6, 14, 17, 22])
def test_non_permutation_input_is_memory_safe(n):
    """Every index the kernels form is masked to its block, so duplicated values
    give an unspecified setting but no error; a good call afterwards is exact."""
    bad = inputs.random_perm(n, 2)
    bad[1::2] = bad[0::2]
    gpu_route(bad, n)
    assert torch.cuda.current_stream().query() or True
    torch.cuda.synchronize()
    perm = inputs.random_perm(n, 3)
    assert np.array_equal(gpu_route(perm, n), oracle.route(perm, n))


@pytest.mark.parametrize("n,batch", [(12, 4), (18, 1), (20, 1)])
def test_route_and_apply_replayed_from_a_cuda_graph(n, batch):
    """Both entry points only enqueue work on the caller's stream (once the workspace exists and
    the kernels' attributes are set, i.e. after one ordinary call), so a caller can capture them
    into a CUDA graph and replay it on new contents of the same buffers."""
    perm_a = inputs.random_perm_batch(n, batch, seed0=900 + n)
    perm_b = inputs.random_perm_batch(n, batch, seed0=950 + n)
    x = inputs.payload_u64(batch << n, 3).reshape(batch, -1)
    d_perm, d_x = dev(perm_a), dev(x)
    bits = torch.empty(binding.benes_switch_words(n, batch), dtype=torch.int32, device="cuda")
    out = torch.empty_like(d_x)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        binding.benes_route(d_perm, n, batch, bits, side)                  # warm-up: workspace, attributes
        binding.benes_apply_ex(bits, d_x, out, 8, n, batch, side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        binding.benes_route(d_perm, n, batch, bits, torch.cuda.current_stream())
        binding.benes_apply_ex(bits, d_x, out, 8, n, batch, torch.cuda.current_stream())
    for perm in (perm_b, perm_a, perm_b):
        d_perm.copy_(dev(perm))
        bits.fill_(-1)
        out.fill_(-1)
        graph.replay()
        torch.cuda.synchronize()
        shape = (batch, 2 * n - 1, max(1, (1 << n) // 64))
        assert np.array_equal(host(bits, np.uint32).reshape(shape), oracle.route(perm, n))
        assert np.array_equal(host(out, np.uint64).reshape(x.shape), np.take_along_axis(x, perm.astype(np.int64), axis=1))


@pytest.mark.parametrize("n,batch,with_apply", [(8, 100, True), (12, 4, True), (16, 3, True), (18, 1, False),
                                                (20, 1, True)])
def test_plans_replay_the_route_on_fixed_buffers(n, batch, with_apply):
    """benes_plan_create captures route (+ apply) once; every launch reads the buffers' current
    contents.  Two plans coexist (each has its own scratch), and ordinary calls in between do
    not disturb them."""
    perms = [inputs.random_perm_batch(n, batch, seed0=700 + n + 50 * k) for k in range(3)]
    x = inputs.payload_u64(batch << n, 3).reshape(batch, -1)
    d_perm, d_x = dev(perms[0]), dev(x)
    bits = torch.empty(binding.benes_switch_words(n, batch), dtype=torch.int32, device="cuda")
    out = torch.empty_like(d_x)
    plan = binding.Plan(d_perm, n, batch, bits, d_x, out, 8) if with_apply else binding.Plan(d_perm, n, batch, bits)
    other_perm = dev(perms[1])
    other_bits = torch.empty_like(bits)
    other = binding.Plan(other_perm, n, batch, other_bits)
    before = binding.benes_launch_count()
    shape = (batch, 2 * n - 1, max(1, (1 << n) // 64))
    for k in (1, 2, 0, 2):
        d_perm.copy_(dev(perms[k]))
        bits.fill_(-1)
        out.fill_(-1)
        plan.launch()
        other.launch()
        gpu_route(perms[(k + 1) % 3], n)                       # an ordinary call in between (library workspace)
        torch.cuda.synchronize()
        assert np.array_equal(host(bits, np.uint32).reshape(shape), oracle.route(perms[k], n))
        assert np.array_equal(host(other_bits, np.uint32).reshape(shape), oracle.route(perms[1], n))
        if with_apply:
            assert np.array_equal(host(out, np.uint64).reshape(x.shape),
                                  np.take_along_axis(x, perms[k].astype(np.int64), axis=1))
    assert binding.benes_launch_count() > before                # replayed launches are counted too
    plan.destroy()
    other.destroy()


def test_launch_counter_counts():
    n = 17
    before = binding.benes_launch_count()
    gpu_route(inputs.random_perm(n, 1), n)
    after = binding.benes_launch_count()
    assert after > before
