"""aa_shrink_compact_static: the shrink + compact entry point for callers that cannot allocate.

Some hosts of this library may not call cudaMalloc at all (a plug-in inside an application that owns
the device memory pool, a latency-critical loop that must stay out of the allocator), so they cannot
hand aa_create a workspace.  The static variant keeps its scan state in an array built into the
library.  It must give exactly the batch that aa_shrink_compact gives — on the first call on the
device and again on the next call, which finds the array as the first one left it.

This file sorts last so that a run stopping at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import aa_oracle as O
from paper_1905_03381_b200 import binding as B
from paper_1905_03381_b200 import build, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _with_context(score, mix, seed, step, id_base):
    n = score.numel()
    aa = B.AutoAssist(max_rows=n, max_d=8, device=DEV)
    idx = torch.full((n,), -7, dtype=torch.int32, device=DEV)
    cnt = torch.full((1,), -7, dtype=torch.int32, device=DEV)
    mask = torch.full((n,), 9, dtype=torch.uint8, device=DEV)
    aa.aa_shrink_compact(score, mix, seed, step, idx, cnt, mask, id_base=id_base)
    torch.cuda.synchronize()
    assert aa.aa_device_status() == B.AA_OK
    aa.close()
    return idx.cpu().numpy(), int(cnt.item()), mask.cpu().numpy()


def _static(score, mix, seed, step, id_base, capacity=None):
    n = score.numel()
    cap = n if capacity is None else capacity
    idx = torch.full((max(cap, 1),), -7, dtype=torch.int32, device=DEV)
    cnt = torch.full((1,), -7, dtype=torch.int32, device=DEV)
    mask = torch.full((max(n, 1),), 9, dtype=torch.uint8, device=DEV)
    status = torch.full((1,), -7, dtype=torch.int32, device=DEV)
    B.aa_shrink_compact_static(score, mix, seed, step, idx[:cap], cnt, mask, status, id_base=id_base, n=n)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), int(cnt.item()), mask.cpu().numpy()[:n], int(status.item())


def test_static_variant_matches_the_context_variant_on_two_calls_in_a_row():
    build.build()
    # two different pools back to back: several tiles with a ragged tail, then a larger pool
    calls = [(70001, 0.05, 77, 3, 12345), (1 << 20, 0.5, 5, 9, (1 << 32) - 100)]
    for n, mix, seed, step, id_base in calls:
        score = W.normal((n,), 2.0, 40 + n, torch.float32, DEV)
        ref_idx, ref_m, ref_mask = _with_context(score, mix, seed, step, id_base)
        idx, m, mask, status = _static(score, mix, seed, step, id_base)
        assert status == B.AA_OK
        assert m == ref_m and 0 < m < n
        assert np.array_equal(mask, ref_mask)          # integer work: bit-exact
        assert np.array_equal(idx[:m], ref_idx[:m])
        assert np.all(idx[m:] == -7)                   # nothing written past the count
    # the same call again: the array now holds the previous call's state and must be re-armed
    idx2, m2, mask2, status2 = _static(score, mix, seed, step, id_base)
    assert status2 == B.AA_OK and m2 == m and np.array_equal(idx2, idx) and np.array_equal(mask2, mask)


def test_static_variant_limits_and_latched_conditions():
    build.build()
    score = W.normal((5000,), 1.0, 1, torch.float32, DEV)
    full = _static(score, 0.5, 3, 3, 0)
    cut = _static(score, 0.5, 3, 3, 0, capacity=100)
    assert cut[1] == full[1] > 100 and np.array_equal(cut[0][:100], full[0][:100])
    assert cut[3] == B.AA_ERR_CAPACITY and full[3] == B.AA_OK
    # empty pool
    empty = torch.zeros(0, dtype=torch.float32, device=DEV)
    assert _static(empty, 0.1, 0, 0, 0)[1] == 0
    # beyond the built-in array: refused on the host, nothing enqueued
    cnt = torch.zeros(1, dtype=torch.int32, device=DEV)
    with pytest.raises(B.AutoAssistError) as err:
        B.aa_shrink_compact_static(score, 0.1, 0, 0, score.to(torch.int32), cnt, n=B.AA_STATIC_MAX_CANDIDATES + 1)
    assert err.value.status == B.AA_ERR_WORKSPACE


def _oracle_check(score, mix, seed, step, id_base, idx, m, mask):
    """The batch against the oracle's own shrink and compact (decisions bit-exact outside the tie band |p - c| < 1e-5,
    where fp32 and fp64 probabilities may fall on different sides; the list bit-exact given the mask)."""
    n = score.numel()
    g = O.sigmoid(score.double().cpu().numpy())
    keep = O.shrink(g, mix, seed, step, id_base=id_base)
    p = O.accept_prob(g, mix)
    c = O.uniform(seed, step, np.arange(n) + id_base)
    far = np.abs(p - c) >= 1e-5
    assert np.array_equal(mask[far], keep[far])
    assert m == int(mask.sum()) and np.array_equal(idx[:m], O.compact(mask))


def test_static_variant_against_the_oracle_and_at_the_edges_of_its_array():
    build.build()
    # directly against the oracle, not only against the context variant
    n, mix, seed, step, id_base = 70001, 0.2, 11, 4, 999
    score = W.normal((n,), 2.0, 40 + n, torch.float32, DEV)
    idx, m, mask, status = _static(score, mix, seed, step, id_base)
    assert status == B.AA_OK
    _oracle_check(score, mix, seed, step, id_base, idx, m, mask)

    # exactly the largest pool the array covers: every look-back word is in use, the last one included
    n_max = B.AA_STATIC_MAX_CANDIDATES
    big = W.normal((n_max,), 2.0, 41, torch.float32, DEV)
    ref_idx, ref_m, ref_mask = _with_context(big, 0.05, 3, 8, 0)
    idx_b, m_b, mask_b, status_b = _static(big, 0.05, 3, 8, 0)
    assert status_b == B.AA_OK and m_b == ref_m and np.array_equal(mask_b, ref_mask) and np.array_equal(idx_b[:m_b], ref_idx[:m_b])
    # the oracle on the pool's first and last tiles (their decisions do not depend on the rest of the pool)
    for lo, hi in ((0, 2048), (n_max - 2048, n_max)):
        g = O.sigmoid(big[lo:hi].double().cpu().numpy())
        keep = O.shrink(g, 0.05, 3, 8, id_base=lo)
        far = np.abs(O.accept_prob(g, 0.05) - O.uniform(3, 8, np.arange(lo, hi))) >= 1e-5
        assert np.array_equal(mask_b[lo:hi][far], keep[far])
    assert np.array_equal(idx_b[:m_b], np.nonzero(mask_b)[0])

    # a small pool right after the largest one: the words the big call left behind must not leak into this scan
    idx2, m2, mask2, status2 = _static(score, mix, seed, step, id_base)
    assert status2 == B.AA_OK and m2 == m and np.array_equal(idx2, idx) and np.array_equal(mask2, mask)

    # no mask, no status word, a stream of the caller's own
    side = torch.cuda.Stream(DEV)
    out_idx = torch.full((n,), -7, dtype=torch.int32, device=DEV)
    out_cnt = torch.full((1,), -7, dtype=torch.int32, device=DEV)
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        B.aa_shrink_compact_static(score, mix, seed, step, out_idx, out_cnt, None, None, id_base=id_base, stream=side)
    side.synchronize()
    assert int(out_cnt.item()) == m and np.array_equal(out_idx.cpu().numpy(), idx)
