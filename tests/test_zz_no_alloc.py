"""The allocation-free partition entry point against the ordinary one.

``chicle_partition_noalloc`` is for callers that cannot allocate device memory at the moment they need a partition
map (a memory pool frozen at start-up, a serving loop with a fixed budget, a thread holding a lock the allocator
needs). It keeps its sort workspace in a fixed array inside the library, shared by all calls, so this test calls it
twice in a row with different arguments to show that leftovers of one call do not leak into the next, and compares
both results with ``chicle_partition`` bit for bit (integer work: no tolerance). This file is collected last on
purpose: a failure here cannot hide the other GPU tests from a run that stops at the first failure.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def reference_partition(n, K, seed):
    """owner and grouped members from the existing entry points (chicle_partition + chicle_get_partition)."""
    from paper_1909_04885_b200 import binding
    X = np.ones((n, 1), np.float32)
    y = np.ones(n, np.float32)
    glm = binding.Glm("hinge", "dense", n, 1, X, y, 0.1)
    try:
        glm.partition(K, seed)
        owner = glm.get_partition()
    finally:
        glm.close()
    members = np.argsort(owner, kind="stable").astype(np.int32)      # grouped by partition, ascending id inside
    return owner, members


def test_noalloc_partition_matches_the_allocating_one_twice_in_a_row():
    import torch
    assert torch.cuda.is_available()
    from paper_1909_04885_b200 import binding, build
    build.build()
    cases = [(100003, 300, 7), (5000, 16, 2**40 + 3)]                 # second call is smaller: stale tail in the workspace
    expected = [reference_partition(*c) for c in cases]
    nmax = max(c[0] for c in cases)
    owner = torch.full((nmax,), -1, dtype=torch.int32, device="cuda")
    members = torch.full((nmax,), -1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream().cuda_stream
    # One call at start-up, as the header asks of callers with a frozen budget: the runtime loads the library's kernels
    # and its workspace array lazily, which may take device memory once. From then on the device's free memory (the
    # driver's own count: it sees every allocation on the device, not only torch's) must not move.
    binding.partition_noalloc(1000, 3, 1, owner, members, device=0, stream=stream)
    torch.cuda.synchronize()
    for (n, K, seed), (want_owner, want_members) in zip(cases, expected):
        owner.fill_(-1)
        members.fill_(-1)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()   # (taken around the call alone: the checks below allocate with torch)
        binding.partition_noalloc(n, K, seed, owner, members, device=0, stream=stream)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        assert np.array_equal(owner[:n].cpu().numpy(), want_owner)
        assert np.array_equal(members[:n].cpu().numpy(), want_members)
        assert (owner[n:] == -1).all() and (members[n:] == -1).all()  # nothing written past n


def test_noalloc_partition_rejects_sizes_beyond_its_workspace():
    import torch
    from paper_1909_04885_b200 import binding
    o = torch.empty(8, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.ChicleError) as e:
        binding.partition_noalloc(131073, 4, 0, o, o)
    assert e.value.status == 5 and "131072" in str(e.value)
    with pytest.raises(binding.ChicleError) as e:
        binding.partition_noalloc(8, 9, 0, o, o)
    assert e.value.status == 1
