"""rtopk_sample_positions_static: the k-of-r positions for callers that must not allocate.

Some users of this library cannot call cudaMalloc while they run: their framework owns the device
memory through its own allocator, or they sit in a latency-critical loop where the device-wide stall
of an allocation is not acceptable.  A context allocates, so they get one entry point that keeps its
scratch in a fixed array inside the library.  This test calls it through the C ABI twice in a row
(the second call meets the first call's leftovers in the shared array) and compares the positions,
bit for bit, with the context-based entry point and with the CPU oracle's sequential Floyd loop;
positions are integers, so the tolerance is zero.
The file name makes pytest collect it after every other test.
"""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    import paper_2005_10761_b200 as pkg
    from paper_2005_10761_b200 import build
    build.build()
    return pkg


def _reference(lib, r, k, seed, step, worker, segment):
    ctx = lib.RTopK(d_max=r, W_max=1, r_max=r, k_max=k)
    pos = torch.zeros(k, dtype=torch.int32, device="cuda")
    ctx.sample_positions(r, k, seed, step, worker, segment, pos)
    torch.cuda.synchronize()
    ctx.close()
    return pos.cpu().numpy()


def test_static_scratch_call_matches_context_call_twice_in_a_row(lib):
    from paper_2005_10761_b200 import binding
    # a large set first, then a smaller one that must not see the first one's table or bitmap;
    # then k = r (no draws at all) and the largest supported r
    cases = [(200_003, 20_000, 0x1234567890ABCDEF, 7, 3, 1),
             (1_000, 999, 5, 0, 0, 0),
             (4_097, 4_097, 9, 2, 1, 0),
             (binding.STATIC_MAX_R, 1 << 16, 77, 1, 15, 2),
             (64, 1, 77, 1, 15, 2)]
    want = [_reference(lib, *c) for c in cases]
    free_before = None
    for c, w in zip(cases, want):
        r, k = c[0], c[1]
        pos = torch.full((k,), -1, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        if free_before is None:
            binding.sample_positions_static(*c, pos)        # first call on the device: does the set-up
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
        else:
            binding.sample_positions_static(*c, pos)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before      # the call took no device memory
        assert np.array_equal(pos.cpu().numpy(), w), f"r={r} k={k}"
        assert np.array_equal(pos.cpu().numpy().view(np.uint32), oracle.sample_positions(*c)), f"r={r} k={k} (oracle)"


def test_static_scratch_call_rejects_sizes_beyond_its_array(lib):
    from paper_2005_10761_b200 import binding
    pos = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(lib.RTopKError) as e:
        binding.sample_positions_static(binding.STATIC_MAX_R + 1, 8, 0, 0, 0, 0, pos)
    assert e.value.status == 4                                       # RTOPK_ERR_UNSUPPORTED
    with pytest.raises(lib.RTopKError) as e:
        binding.sample_positions_static(4, 8, 0, 0, 0, 0, pos)       # k > r
    assert e.value.status == 1
    torch.cuda.synchronize()
    assert bool((pos == 0).all())
