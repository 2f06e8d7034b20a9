"""benes_apply_static: the apply entry point for callers that cannot allocate
device memory (all of it belongs to another allocator, or a cudaMalloc stall is
unaffordable).  Its scratch is a fixed array inside the library, so this test
checks, through the C ABI, that it gives exactly what benes_apply_ex gives --
twice in a row, because the second call finds the first call's leftovers in
the shared array -- and that oversized payloads are refused.

Kept in a file that sorts last so that a run stopping at the first failure has
already been through every other test."""
import numpy as np
import pytest
import torch

from paper_1912_04050_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.load()


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a).view({4: np.int32, 8: np.int64}[a.dtype.itemsize])).cuda()


@pytest.mark.parametrize("n,batch,dtype", [(19, 1, np.uint64), (20, 1, np.uint32), (8, 1024, np.uint64),
                                           (1, 3, np.uint32), (5, 7, np.uint64)])
def test_static_apply_matches_regular_apply_twice(n, batch, dtype):
    perm = inputs.random_perm_batch(n, batch, seed0=31 * n)
    d_perm = _dev(perm)
    bits = binding.route(d_perm)
    outs = []
    for call in range(2):       # second call reuses the scratch the first one dirtied
        x = inputs.payload_u64(batch << n, 50 + call)
        if dtype == np.uint32:
            x = (x >> np.uint64(32)).astype(np.uint32)      # the seeded half of the 64-bit payload
        x = x.reshape(batch, -1)
        d_x = _dev(x)
        want = torch.empty_like(d_x)
        binding.benes_apply_ex(bits, d_x, want, x.dtype.itemsize, n, batch)
        got = torch.full_like(d_x, -1)
        binding.benes_apply_static(bits, d_x, got, x.dtype.itemsize, n, batch)
        torch.cuda.synchronize()
        assert torch.equal(got, want)                       # bit-exact, as everywhere in this suite
        assert np.array_equal(got.cpu().numpy().view(dtype),
                              np.take_along_axis(x, perm.astype(np.int64), axis=1))
        outs.append(got)
    assert not torch.equal(outs[0], outs[1])                # the two calls really had different payloads


def test_static_apply_refuses_what_does_not_fit():
    n = 20                                                   # 2^20 x 8 bytes = 8 MiB > 4 MiB
    dummy = torch.zeros(8, dtype=torch.int64, device="cuda")
    with pytest.raises(binding.BenesError) as e:
        binding.benes_apply_static(dummy, dummy, torch.zeros_like(dummy), 8, n, 1)
    assert e.value.status == binding.BENES_ERR_TOO_LARGE
    with pytest.raises(binding.BenesError) as e:
        binding.benes_apply_static(dummy, dummy, torch.zeros_like(dummy), 4, 10, 1 + (1 << 10))
    assert e.value.status == binding.BENES_ERR_TOO_LARGE
    assert "scratch" in binding.status_string(binding.BENES_ERR_TOO_LARGE)


def test_static_apply_needs_no_workspace_and_no_device_memory():
    """What the entry point is for: with a caller workspace of 256 bytes installed, any
    internal request for scratch fails (the regular entry point does, below), yet the
    allocation-free one still works, and the free device memory is the same before and
    after the call."""
    n, batch = 17, 2
    perm = inputs.random_perm_batch(n, batch, seed0=77)
    x = inputs.payload_u64(batch << n, 5).reshape(batch, -1)
    d_x = _dev(x)
    bits = binding.route(_dev(perm))
    got = torch.empty_like(d_x)
    binding.benes_apply_static(bits, d_x, got, 8, n, batch)          # first call on this device: address look-up
    torch.cuda.synchronize()
    tiny = torch.zeros(256, dtype=torch.uint8, device="cuda")
    binding.benes_set_workspace(tiny)
    try:
        with pytest.raises(binding.BenesError) as e:
            binding.benes_apply_ex(bits, d_x, torch.empty_like(d_x), 8, n, batch)
        assert e.value.status == binding.BENES_ERR_NOMEM
        got.fill_(-1)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        binding.benes_apply_static(bits, d_x, got, 8, n, batch)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0
    finally:
        binding.benes_set_workspace(None)
    assert np.array_equal(got.cpu().numpy().view(np.uint64), np.take_along_axis(x, perm.astype(np.int64), axis=1))
