"""The allocation-free Merkle entry point against the ordinary one and against the CPU oracle.

Some users of the library run where device allocation is off limits (a memory pool holds the whole
GPU, or the allocator may not be called from their loop).  `iv_merkle_root_noalloc` serves them from a
fixed scratch array inside the library.  Its root must equal `iv_merkle_root`'s bit for bit, also on a
second call that finds the first call's leftovers in the shared array; both are also held against the
oracle's root over the same leaves, so the two entry points cannot agree on a wrong answer.  This file sorts last on
purpose, so a run that stops at the first failure has already been through every other test.
"""
import pytest
import torch

import oracle
from paper_2510_23938_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def test_noalloc_root_equals_the_allocating_entry_point_on_consecutive_calls():
    assert torch.cuda.is_available(), "the gpu-marked tests need a CUDA device"
    out = torch.zeros(32, dtype=torch.uint8, device="cuda")
    with binding.Context(0) as ctx:
        # two calls in a row on different sizes, then the first size again (stale scratch from the second)
        for n in (28_672, 1_000, 28_672, 1, 2, 513, binding.NOALLOC_MAX_LEAVES):
            leaves = inputs.uniform_bytes(32 * n, seed=900 + n, device="cuda").view(n, 32)
            want = ctx.merkle_root(leaves)
            binding.merkle_root_noalloc(leaves, out)
            torch.cuda.synchronize()
            assert torch.equal(out, want), n
            assert out.cpu().numpy().tobytes() == oracle.merkle_root(leaves.cpu().numpy()), n
        # zero leaves: SHA-256 of the empty string, as the ordinary call gives
        empty = torch.empty((0, 32), dtype=torch.uint8, device="cuda")
        binding.merkle_root_noalloc(empty, out)
        assert torch.equal(out, ctx.merkle_root(empty))
        assert out.cpu().numpy().tobytes() == oracle.merkle_root(b"")


def test_noalloc_rejects_more_leaves_than_its_scratch_holds():
    out = torch.zeros(32, dtype=torch.uint8, device="cuda")
    leaves = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.IvError) as err:
        binding.merkle_root_noalloc(leaves, out, n_leaves=binding.NOALLOC_MAX_LEAVES + 1)
    assert err.value.code == binding.IV_ERR_TOO_LARGE
    assert not out.any()            # nothing was launched
