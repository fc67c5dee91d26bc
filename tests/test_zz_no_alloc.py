"""-m gpu: the allocation-free token permutation (cmoe_token_permute_static).

Some users of this library run where device memory cannot be allocated: a serving
process whose memory pool is fixed after start-up, or a plug-in that receives only
its input and output buffers.  For them the permutation's scratch matrix lives in a
1 MiB array inside the library.  This file checks, through the C-ABI, that the
variant returns exactly what cmoe_token_permute returns — on two calls in a row with
different inputs, because the array keeps the previous call's contents — and that it
refuses problems beyond its fixed capacity.  It is named to be collected last.
"""
import numpy as np
import pytest

from paper_2502_04416_b200 import binding

pytestmark = pytest.mark.gpu


def _selection(rng, n_rows, n_k, n_groups):
    return np.stack([rng.permutation(n_groups)[:n_k] for _ in range(n_rows)]).astype(np.int32)


@pytest.mark.parametrize("n_rows,n_k,n_groups", [(200, 2, 6), (5000, 2, 56), (16384, 4, 14),
                                                 (3000, 8, 1000)])
def test_static_permute_matches_scratch_permute_twice(n_rows, n_k, n_groups):
    import torch
    rng = np.random.default_rng(n_rows)
    out = (torch.empty(n_groups, dtype=torch.int32, device="cuda"),
           torch.empty(n_groups + 1, dtype=torch.int32, device="cuda"),
           torch.empty(n_rows * n_k, dtype=torch.int32, device="cuda"),
           torch.empty((n_rows, n_k), dtype=torch.int32, device="cuda"))
    for call in range(2):                       # second call: new input, stale scratch
        sel = torch.from_numpy(_selection(rng, n_rows, n_k, n_groups)).cuda()
        want = binding.token_permute(sel, n_groups)
        torch.cuda.synchronize()
        got = binding.token_permute_static(sel, n_groups, out=out)
        torch.cuda.synchronize()
        for g, w in zip(got, want):             # integer results: bit-exact
            assert torch.equal(g, w), f"call {call}: static-scratch permutation differs"


def test_static_permute_rejects_oversized_problems():
    import torch
    n_groups = 1024
    n_rows = (binding.STATIC_PERMUTE_MAX_CELLS // n_groups + 1) * 256     # one chunk too many
    sel = torch.zeros((n_rows, 1), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.CmoeError) as e:
        binding.token_permute_static(sel, n_groups)
    assert e.value.status == -4 and "262144" in str(e.value)
    ok_rows = binding.STATIC_PERMUTE_MAX_CELLS // n_groups * 256           # exactly at the limit
    sel = torch.zeros((ok_rows, 1), dtype=torch.int32, device="cuda")
    cnt, off, row_token, row_of = binding.token_permute_static(sel, n_groups)
    torch.cuda.synchronize()
    assert int(cnt[0]) == ok_rows and int(off[-1]) == ok_rows
    assert torch.equal(row_token, torch.arange(ok_rows, dtype=torch.int32, device="cuda"))
