"""Seeded input generators: validity, structure and determinism (no GPU)."""
import numpy as np
import pytest

from paper_1912_04050_b200 import inputs


def _is_perm(p):
    return np.array_equal(np.sort(p), np.arange(len(p), dtype=p.dtype))


@pytest.mark.parametrize("n", [1, 2, 8, 10, 16])
def test_random_perm_is_a_permutation_and_seeded(n):
    a, b, c = inputs.random_perm(n, 5), inputs.random_perm(n, 5), inputs.random_perm(n, 6)
    assert _is_perm(a) and np.array_equal(a, b)
    if n >= 8:
        assert not np.array_equal(a, c)


def test_batch_uses_consecutive_seeds():
    p = inputs.random_perm_batch(8, 5, seed0=3)
    assert p.shape == (5, 256)
    for i in range(5):
        assert np.array_equal(p[i], inputs.random_perm(8, 3 + i))


def test_fisher_yates_is_uniform_on_n4():
    # 24 permutations, 24000 seeds: chi-square against uniform stays far below a 5-sigma bound
    p = inputs.random_perm_batch(2, 24000, seed0=1000).astype(np.int64)
    key = (p * np.array([1, 4, 16, 64])).sum(1)
    counts = np.unique(key, return_counts=True)[1]
    assert len(counts) == 24
    chi2 = ((counts - 1000.0) ** 2 / 1000.0).sum()
    assert chi2 < 23 + 5 * np.sqrt(2 * 23)


@pytest.mark.parametrize("n", [1, 4, 12])
def test_sattolo_is_one_cycle(n):
    p = inputs.sattolo_perm(n, 3)
    assert _is_perm(p)
    j, steps = 0, 0
    while True:
        j = int(p[j]); steps += 1
        if j == 0:
            break
    assert steps == 1 << n


def test_structured_perms():
    s = inputs.structured_perms(12)
    assert all(_is_perm(p) for p in s.values())
    assert s["shift1"][0] == 1 and s["shift1"][-1] == 0
    assert s["bitrev"][1] == 1 << 11 and s["bitrev"][3] == 3 << 10
    assert s["transpose"][1] == 64 and s["transpose"][64] == 1
    assert np.array_equal(s["bitrev"][s["bitrev"]], s["identity"])
    assert np.array_equal(s["transpose"][s["transpose"]], s["identity"])


def test_payloads():
    x = inputs.payload_f32(4096, 1)
    assert x.dtype == np.float32 and (x >= 0).all() and (x < 1).all() and len(np.unique(x)) > 4000
    y = inputs.payload_u64(4096, 2)
    assert np.array_equal(y & np.uint64(0xFFFFFFFF), np.arange(4096, dtype=np.uint64))
    assert len(np.unique(y >> np.uint64(32))) > 4000
