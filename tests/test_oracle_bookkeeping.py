"""Pins for the oracle's step bookkeeping: invariants any correct append / commit must satisfy."""
import numpy as np

import oracle


def test_append_places_rows_and_touches_nothing_else():
    rng = np.random.default_rng(0)
    B, Hkv, Lmax, D, gamma = 3, 2, 20, 8, 2
    R = gamma + 1
    k = rng.integers(0, 60000, (B, Hkv, Lmax, D)).astype(np.uint16)
    v = rng.integers(0, 60000, (B, Hkv, Lmax, D)).astype(np.uint16)
    kn = rng.integers(0, 60000, (B, R, Hkv, D)).astype(np.uint16)
    vn = rng.integers(0, 60000, (B, R, Hkv, D)).astype(np.uint16)
    ctx = np.array([0, 7, 18], np.int32)          # the last one has no room for 3 rows
    k2, v2, ctx2, over = oracle.kv_append(k, v, kn, vn, ctx, gamma)
    assert over and ctx2.tolist() == [3, 10, 18]
    for b, L in ((0, 0), (1, 7)):
        for i in range(R):
            assert (k2[b, :, L + i] == kn[b, i]).all() and (v2[b, :, L + i] == vn[b, i]).all()
        mask = np.ones(Lmax, bool); mask[L:L + R] = False
        assert (k2[b][:, mask] == k[b][:, mask]).all() and (v2[b][:, mask] == v[b][:, mask]).all()
    assert (k2[2] == k[2]).all() and (v2[2] == v[2]).all()
    assert (k == k2).sum() < k.size and ctx.tolist() == [0, 7, 18]      # inputs were not modified


def test_commit_keeps_the_accepted_prefix():
    ctx = np.array([30, 30, 30, 30], np.int32)
    out = oracle.step_commit(ctx, np.array([0, 2, 5, 9]), gamma=5)      # 9 is clamped to gamma
    assert out.tolist() == [25, 27, 30, 30]
    # append then commit with n accepted leaves exactly 1 + n new rows
    for n in range(6):
        assert oracle.step_commit(np.array([100 + 6]), np.array([n]), 5)[0] == 100 + 1 + n
