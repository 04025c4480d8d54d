"""The allocation-free linear entry point against the ordinary one.

Some users of this library run where device memory cannot be allocated once serving has started (the whole GPU
is handed to their own pool up front, or allocation calls are banned on the serving thread because they stall
the device).  For them the library carries its scratch in a fixed built-in array.  This file checks, through the
C ABI, that the built-in-scratch call returns what the caller-scratch call returns -- twice in a row with
different shapes, because the array keeps the previous call's contents -- and that oversize requests are refused.
It is named so that it is collected after every other test file.
"""
import numpy as np
import pytest
import torch

import workloads as W

pytestmark = pytest.mark.gpu


def case(rng, M, N, K, dtype):
    Wn = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    if dtype == "bf16":
        Wn = W.bf16_round(Wn)
    x = rng.standard_normal((M, K)).astype(np.float32)
    Wt = torch.from_numpy(Wn).cuda().to(torch.bfloat16 if dtype == "bf16" else torch.float32)
    return Wn, x, Wt, torch.from_numpy(x).cuda()


def test_static_scratch_linear_matches_the_regular_entry_point_twice_in_a_row():
    import paper_2609_17184_b200 as ls
    rng = np.random.default_rng(7)
    # two calls back to back; the second is smaller so stale bytes of the first stay behind it in the array
    for M, N, K, dtype in [(7, 2048, 1024, "bf16"), (3, 768, 256, "bf16"), (5, 256, 704, "fp32")]:
        Wn, x, Wt, xt = case(rng, M, N, K, dtype)
        want = ls.linear(Wt, xt).cpu().numpy()           # existing entry point, caller-provided scratch
        got = ls.linear_static(Wt, xt).cpu().numpy()     # new entry point, built-in scratch
        scale = np.abs(x).astype(np.float64) @ np.abs(Wn).astype(np.float64).T
        assert (np.abs(got.astype(np.float64) - want) <= 2e-6 * scale + 1e-30).all()
        ref = x.astype(np.float64) @ Wn.astype(np.float64).T
        assert (np.abs(got - ref) <= 2e-6 * scale + 1e-30).all()


def test_static_scratch_linear_refuses_what_does_not_fit():
    import paper_2609_17184_b200 as ls
    Wt = torch.zeros(8192, 2048, dtype=torch.bfloat16, device="cuda")      # 32 MiB of weights: beyond the 16 MiB array
    xt = torch.zeros(2, 2048, dtype=torch.float32, device="cuda")
    with pytest.raises(ls.LoopSpecError) as e:
        ls.linear_static(Wt, xt)
    assert e.value.status == "ECAPACITY"
    with pytest.raises(ls.LoopSpecError) as e:
        ls.linear_static(torch.zeros(250, 256, dtype=torch.bfloat16, device="cuda"), torch.zeros(2, 256, device="cuda"))
    assert e.value.status == "EINVAL"
    # the array is still usable afterwards
    Wn, x, Wt, xt = case(np.random.default_rng(1), 2, 128, 256, "bf16")
    assert np.array_equal(ls.linear_static(Wt, xt).cpu().numpy(), ls.linear(Wt, xt).cpu().numpy())
