"""The checked build (libbenes_debug.so: the same kernels compiled with -DBENES_DEBUG) stands in
for a memory checker.  Every index a kernel forms from data passes a guard (mask or clamp); the
checked build counts the guards that had to change a value.  On a permutation that count must
stay 0 whatever path the route takes, and the bits must still be the oracle's; on an input that is
not a permutation the guards are what keeps the accesses in bounds, so the count must move."""
import numpy as np
import pytest
import torch

import oracle
from paper_1912_04050_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def checked_library():
    path = build.build(debug=True)
    build.build()
    binding.use_library(path)
    assert binding.benes_debug_build()
    binding.benes_debug_guard_hits(clear=True)
    yield
    binding.benes_release_workspace()
    binding.use_library(None)


@pytest.fixture
def options():
    keys = (binding.OPT_SAMPLE_LOG2K, binding.OPT_WALK_CAP, binding.OPT_CLUSTER, binding.OPT_INVERSE_PARTITIONED,
            binding.OPT_WALK_PAIRS)
    old = [binding.benes_get_option(k) for k in keys]
    yield
    for k, v in zip(keys, old):
        binding.benes_set_option(k, v)


def route(perm, n):
    p = torch.from_numpy(np.ascontiguousarray(perm).view(np.int32)).cuda()
    batch = perm.size >> n
    bits = torch.full((binding.benes_switch_words(n, batch),), -1, dtype=torch.int32, device="cuda")
    binding.benes_route(p, n, batch, bits)
    torch.cuda.synchronize()
    shape = (2 * n - 1, max(1, (1 << n) // 64))
    return bits.cpu().numpy().view(np.uint32).reshape(((batch,) if perm.ndim == 2 else ()) + shape)


def assert_clean(what):
    hits, where = binding.benes_debug_guard_hits(clear=True)
    assert hits == 0, "%s: %d guarded indices were out of range, e.g. at %s" % (what, hits, where)


@pytest.mark.parametrize("n", [3, 6, 9, 12, 14, 15, 16, 17, 18])
def test_no_guard_fires_on_random_permutations(n):
    for batch in (1, 3):
        perm = inputs.random_perm_batch(n, batch, seed0=700 + n)
        assert np.array_equal(route(perm, n), oracle.route(perm, n))
        assert_clean("n=%d batch=%d" % (n, batch))


@pytest.mark.parametrize("n", [10, 16, 18])
def test_no_guard_fires_on_structured_permutations(n):
    for kind, perm in inputs.structured_perms(n).items():
        assert np.array_equal(route(perm, n), oracle.route(perm, n)), kind
        assert_clean("%s n=%d" % (kind, n))


@pytest.mark.parametrize("kappa", [0, 2, 3, 5, 8])
def test_no_guard_fires_for_any_ruler_spacing(kappa, options):
    binding.benes_set_option(binding.OPT_SAMPLE_LOG2K, kappa)
    for n, batch in ((16, 3), (18, 1)):
        perm = inputs.random_perm_batch(n, batch, seed0=800 + n)
        assert np.array_equal(route(perm, n), oracle.route(perm, n))
        assert_clean("kappa=%d n=%d" % (kappa, n))


@pytest.mark.parametrize("cap", [1, 3, 40])
def test_no_guard_fires_when_walks_give_up(cap, options):
    """Forced fallback: the walk records are then partly unused, the level is relabelled by
    pointer jumping over all outputs."""
    binding.benes_set_option(binding.OPT_WALK_CAP, cap)
    for n in (16, 18):
        perm = inputs.random_perm(n, 900 + n)
        assert np.array_equal(route(perm, n), oracle.route(perm, n))
        assert_clean("cap=%d n=%d" % (cap, n))
        perm = inputs.structured_perms(n)["shift1"]
        assert np.array_equal(route(perm, n), oracle.route(perm, n))
        assert_clean("cap=%d shift n=%d" % (cap, n))


def test_no_guard_fires_with_resampled_lists_bucketed_inverse_and_clusters(options):
    perm = inputs.random_perm_batch(18, 3, seed0=5)              # lists sampled again, batch not a power of two
    assert np.array_equal(route(perm, 18), oracle.route(perm, 18))
    assert_clean("18 x 3")
    perm = inputs.random_perm(22, 6)                             # bucketed inverse
    assert np.array_equal(route(perm, 22), oracle.route(perm, 22))
    assert_clean("2^22")
    binding.benes_set_option(binding.OPT_CLUSTER, 1)
    for n, batch in ((16, 3), (18, 1)):
        perm = inputs.random_perm_batch(n, batch, seed0=44)
        assert np.array_equal(route(perm, n), oracle.route(perm, n))
        assert_clean("clusters n=%d" % n)
    binding.benes_set_option(binding.OPT_CLUSTER, 0)
    binding.benes_set_option(binding.OPT_WALK_PAIRS, 2)
    for n, batch in ((17, 3), (19, 1)):
        perm = inputs.random_perm_batch(n, batch, seed0=45)
        assert np.array_equal(route(perm, n), oracle.route(perm, n))
        assert_clean("two walks per thread n=%d" % n)


@pytest.mark.parametrize("n", [6, 14, 17, 22])
def test_guards_fire_on_an_input_that_is_not_a_permutation(n):
    """Values out of range: the guards must catch them (and the call must stay in bounds:
    a good call afterwards is exact and clean)."""
    bad = inputs.random_perm(n, 2).copy()
    bad[::3] |= np.uint32(1 << n)                                # out of range
    route(bad, n)
    hits, where = binding.benes_debug_guard_hits(clear=True)
    assert hits > 0 and ":" in where
    perm = inputs.random_perm(n, 3)
    assert np.array_equal(route(perm, n), oracle.route(perm, n))
    assert_clean("after a bad input, n=%d" % n)


def test_the_normal_build_reports_no_checks():
    binding.use_library(None)
    try:
        assert not binding.benes_debug_build()
        assert binding.benes_debug_guard_hits() == (0, "")
    finally:
        binding.use_library(build.LIB_DEBUG)
