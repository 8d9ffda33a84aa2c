"""Retrieval scoring on the device against the fp64 oracle.  Scores are compared by value; the
selection is compared exactly unless two fp64 scores (or a score and the threshold) are closer than
what fp32 accumulation over the embedding can resolve, where any consistent choice is accepted."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
import workloads as wl

EPS = 2e-6


def _check(E, q, k, thr, n_chunks=None):
    import paper_2502_20330_b200 as R
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    nc = None if n_chunks is None else torch.tensor(n_chunks, dtype=torch.int32, device="cuda")
    scores, sel, cnt = R.rapid_retrieval_select(E, q, k, status, threshold=thr, n_chunks=nc)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref_s, ref_sel = oracle.retrieval_select(E.cpu().numpy(), q.cpu().numpy(), k, thr, n_chunks)
    s = scores.cpu().numpy()
    np.testing.assert_allclose(s, ref_s, rtol=0, atol=EPS)
    sel, cnt = sel.cpu().numpy(), cnt.cpu().numpy()
    for b in range(E.shape[0]):
        n = E.shape[1] if n_chunks is None else n_chunks[b]
        got = sel[b, :cnt[b]].tolist()
        assert (sel[b, cnt[b]:] == -1).all() and len(set(got)) == len(got) and all(0 <= i < n for i in got)
        if got == ref_sel[b]:
            continue
        r = ref_s[b]
        assert all(r[i] >= thr - EPS for i in got)                                   # nothing clearly below the threshold
        assert all(r[got[j]] >= r[got[j + 1]] - EPS for j in range(len(got) - 1))    # best first
        clear = [i for i in range(n) if r[i] >= thr + EPS]
        if len(got) < k:
            assert set(clear) <= set(got)                                            # nothing clearly passing is left out
        else:
            worst = min(r[i] for i in got)
            assert all(r[i] <= worst + EPS for i in clear if i not in got)


@pytest.mark.parametrize("B,N,Dm,k", [(1, 256, 1024, 10), (4, 256, 1024, 8), (3, 64, 1024, 8), (2, 1000, 768, 21),
                                      (1, 4096, 128, 50), (5, 7, 1024, 10)])
def test_retrieval_against_oracle(B, N, Dm, k):
    E, q = wl.retrieval_inputs(B, N, Dm, seed=51, device="cuda")
    _check(E, q, k, 0.3)


def test_ragged_requests_ties_and_degenerate_vectors():
    E, q = wl.retrieval_inputs(3, 128, 1024, seed=52, device="cuda")
    E[0, 5] = E[0, 9]                       # an exact tie: the lower index goes first
    E[1, 3] = 0                             # a zero vector scores 0
    E[2, 100:] = float("nan")               # never read: request 2 has 100 chunks
    _check(E, q, 12, 0.3, n_chunks=[128, 128, 100])
    _check(E, q, 200, -1.0, n_chunks=[128, 50, 0])      # k above the count, a request without chunks


def test_argument_errors():
    import paper_2502_20330_b200 as R
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    E = torch.zeros(1, 5000, 64, device="cuda")
    with pytest.raises(R.RapidError) as e:
        R.rapid_retrieval_select(E, torch.zeros(1, 64, device="cuda"), 4, status)
    assert e.value.code == 2
    with pytest.raises(R.RapidError) as e:
        R.rapid_retrieval_select(torch.zeros(1, 8, 64, device="cuda"), torch.zeros(1, 64, device="cuda"), 0, status)
    assert e.value.code == 1
