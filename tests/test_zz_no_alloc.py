"""detox_vote_noalloc: the vote for callers that are not allowed to allocate device memory (allocator
callbacks, serving loops with a frozen memory plan).  Its scratch is a fixed array inside the library.

Checked against detox_vote, bit for bit, on two calls in a row: the second call sees the scratch
as the first one left it, so it only passes if each call clears what it uses.  Collected last, so a
failure here cannot hide one elsewhere in a run that stops at the first failure."""
import numpy as np
import pytest
import torch

import paper_1907_12205_b200 as dx

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def make(n, r, d, seed, spoil):
    """Groups of bitwise copies; in `spoil` groups one member differs (still an honest majority) and in
    the last group, when spoiled, nobody agrees."""
    rng = np.random.default_rng(seed)
    G = n // r
    members = rng.permutation(n).astype(np.int32)
    X = np.empty((n, d), np.float32)
    for j in range(G):
        grp = members[j * r:(j + 1) * r]
        X[grp] = rng.standard_normal(d).astype(np.float32)
        if j in spoil:
            X[grp[0], d // 2] += 1.0
            if j == G - 1:
                X[grp[1], 0] -= 1.0
    return torch.as_tensor(X).to(DEV), members


@pytest.mark.parametrize("r,G,d", [(3, 15, 40_003), (5, 4, 9_001)])
def test_noalloc_vote_equals_vote_on_two_calls_in_a_row(r, G, d):
    n = r * G
    # call 1: every group has a dissenting member (all scratch bits of the used pairs get set);
    # call 2: different data, only group 1 dissents -> stale bits from call 1 would give wrong winners.
    for seed, spoil in ((1, set(range(G))), (2, {1})):
        X, members = make(n, r, d, seed, spoil)
        Z_ref, w_ref = dx.detox_vote(X, r, members)
        Z = torch.full((G, d), float("nan"), dtype=torch.float32, device=DEV)
        w = torch.full((G,), -7, dtype=torch.int32, device=DEV)
        dx.detox_vote_noalloc(X, r, members, Z, w)
        torch.cuda.synchronize()
        assert torch.equal(w, w_ref)
        assert torch.equal(Z.view(torch.int32), Z_ref.contiguous().view(torch.int32))
    assert (w_ref.cpu().numpy() >= 0).all()


def test_noalloc_vote_rejects_more_groups_than_the_builtin_scratch():
    n = 3 * (dx.binding.NOALLOC_MAX_GROUPS + 1)
    X = torch.zeros((n, 8), dtype=torch.float32, device=DEV)
    w = torch.empty(n // 3, dtype=torch.int32, device=DEV)
    with pytest.raises(dx.DetoxError) as e:
        dx.detox_vote_noalloc(X, 3, np.arange(n), None, w)
    assert e.value.code == 2
