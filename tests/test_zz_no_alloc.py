"""mavg_batch_indices_noalloc, the entry point for hosts that cannot allocate device memory (all
of it already belongs to someone else's pool, or cudaMalloc's device-wide stall is not
acceptable where the call is made).  It must hand back exactly the indices that the handle-based
mavg_get_batch_indices produces, call after call, although every call reuses one fixed staging
array inside the library.  Collected last on purpose: a run that stops at the first failure has
then already seen every other test."""
import numpy as np
import pytest


def test_oversize_batch_is_refused_on_the_host():
    from paper_2110_00625_b200 import binding
    with pytest.raises(binding.MavgError, match="65536"):
        binding.batch_indices_noalloc(1, 1, 4, 0, 1, 1 << 20, 65537)
    with pytest.raises(binding.MavgError, match="MAVG_ERR_INVALID_ARG"):
        binding.batch_indices_noalloc(1, 1, 4, 4, 1, 4096, 32)      # learner out of range
    with pytest.raises(binding.MavgError, match="MAVG_ERR_INVALID_ARG"):
        binding.batch_indices_noalloc(1, 0, 4, 0, 1, 4096, 32)      # rounds start at 1


@pytest.mark.gpu
def test_matches_the_handle_based_entry_point_twice_in_a_row():
    import torch
    import paper_2110_00625_b200 as m
    from paper_2110_00625_b200 import binding
    seed, P, K, B, S = 0x211000625, 8, 8, 128, 50000
    dims = [32, 16, 10]
    x = np.zeros((S, dims[0]), dtype=np.float32)
    y = np.zeros(S, dtype=np.int32)
    w1 = m.workloads.mlp_init(dims)
    g = m.Mavg(w1, P=P, K=K, local_lr=0.05, mu=0.9, B=B, seed=seed, objective=m.OBJ_MLP,
               dims=dims, gemm_bf16=0, x=x, y=y)
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    # two calls in a row, the second must not see anything of the first
    for (rnd, learner, step) in [(1, 0, 1), (3, P - 1, K)]:
        got = binding.batch_indices_noalloc(seed, rnd, P, learner, step, S, B)
        want = g.get_batch_indices(rnd, learner, step)
        assert np.array_equal(got, want)       # integer work: bit-exact
    # a shorter batch after a longer one reads back only its own entries
    short = binding.batch_indices_noalloc(seed, 2, P, 3, 2, S, 16)
    assert np.array_equal(short, g.get_batch_indices(2, 3, 2)[:16])
    assert torch.cuda.memory_allocated() == before
    g.close()
