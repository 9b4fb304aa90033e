"""The allocation-free index-set call against the context-based path and against the oracle.

A receiver of a random-k message needs the index set S_t but may hold no
context and may not allocate device memory (fixed memory pool; an allocation
in mid-step would synchronise or fail).  conef_randk_indices_noalloc serves
that caller out of a fixed scratch array inside the library.  Here its output
must equal, bit for bit, the indices that conef_step produces for the same
(seed, tensor, step), on two calls in a row (the scratch is shared between
calls and keeps the previous call's contents).

This file sorts last on purpose: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,cols,k_num,k_den", [(256, 512, 1, 100), (37, 53, 3, 100), (2048, 1024, 1, 100),
                                                   (1, 7, 1, 1)])
def test_noalloc_indices_equal_the_context_path_twice_in_a_row(rows, cols, k_num, k_den):
    from paper_2312_08538_b200 import binding as b
    from oracle import conef_oracle as orc
    seed = 231208551
    d = rows * cols
    q = dict(kind="randk", k_num=k_num, k_den=k_den, seed=seed)
    eng = b.ConEF([(rows, cols, 1)], 1, q, dict(kind="int8", block=256), 0.1)
    k = eng.message_elems(b.MSG_VALUES)
    assert k == max(1, d * k_num // k_den)
    g = [torch.randn(d, device="cuda")]
    out = torch.empty(k, dtype=torch.int32, device="cuda")
    for step in (3, 4):                      # two calls in a row on the shared scratch
        eng.step(step, g, 0)
        want = eng.indices(0).clone()
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        b.conef_randk_indices_noalloc(seed, 0, step, d, k, out)
        torch.cuda.synchronize()
        if step == 4:                        # (the first call may load the kernels' code onto the device)
            assert torch.cuda.mem_get_info()[0] >= free_before, "the call took device memory"
        assert torch.equal(out, want), f"step {step}: index sets differ"
        idx = out.cpu().numpy().view(np.uint32)
        assert np.array_equal(idx, orc.randk_indices(seed, 0, step, d, k)), f"step {step}: differs from the oracle"
        assert idx.size == k and np.all(np.diff(idx.astype(np.int64)) > 0) and idx.max() < d
    assert eng.last_status() == 0


def test_noalloc_rejects_what_its_fixed_scratch_cannot_hold():
    from paper_2312_08538_b200 import binding as b
    out = torch.empty(128, dtype=torch.int32, device="cuda")
    with pytest.raises(b.ConEFError) as e:
        b.conef_randk_indices_noalloc(1, 0, 0, b.NOALLOC_MAX_ELEMS + 1, 16, out)
    assert e.value.code == b.ERR_TOO_LARGE
    with pytest.raises(b.ConEFError) as e:
        b.conef_randk_indices_noalloc(1, 0, 0, 100, 101, out)      # k > d
    assert e.value.code == b.ERR_INVALID_ARG
    # the largest size it accepts still works
    d, k = b.NOALLOC_MAX_ELEMS, 16
    out.fill_(-1)
    b.conef_randk_indices_noalloc(7, 2, 5, d, k, out)
    torch.cuda.synchronize()
    idx = out[:k].cpu().numpy().view(np.uint32)
    from oracle import conef_oracle as orc
    assert np.array_equal(idx, orc.randk_indices(7, 2, 5, d, k))      # (the failure mark 0xFFFFFFFF would show here)
    assert int(out[k].item()) == -1, "nothing is written past the k entries"
