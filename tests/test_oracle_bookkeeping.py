"""Pins for the oracle's step bookkeeping: invariants any correct append / commit must satisfy."""
import numpy as np
import pytest

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


def test_paged_gather_identity_table_is_a_reshape():
    """With block i of sequence 0 stored in physical block i, the gathered cache is the pool's
    blocks laid end to end."""
    rng = np.random.default_rng(3)
    nb, Hkv, bs, D = 5, 2, 4, 3
    pool = rng.integers(0, 65535, size=(nb, Hkv, bs, D), dtype=np.uint16)
    table = np.arange(nb, dtype=np.int32)[None, :]
    got = oracle.paged_gather(pool, table, [nb * bs])
    want = pool.transpose(1, 0, 2, 3).reshape(1, Hkv, nb * bs, D)
    np.testing.assert_array_equal(got, want)


def test_paged_gather_follows_the_table_and_stops_at_the_length():
    rng = np.random.default_rng(4)
    nb, Hkv, bs, D = 7, 1, 2, 2
    pool = rng.integers(1, 65535, size=(nb, Hkv, bs, D), dtype=np.uint16)
    table = np.array([[6, 0, 3], [2, 5, -1]], dtype=np.int32)
    got = oracle.paged_gather(pool, table, [5, 3])
    # sequence 0: keys 0,1 <- block 6; 2,3 <- block 0; 4 <- block 3 row 0; key 5 is past its length
    np.testing.assert_array_equal(got[0, 0, 0], pool[6, 0, 0])
    np.testing.assert_array_equal(got[0, 0, 3], pool[0, 0, 1])
    np.testing.assert_array_equal(got[0, 0, 4], pool[3, 0, 0])
    assert (got[0, 0, 5] == 0).all()
    # sequence 1: key 2 <- block 5 row 0; the -1 entry is never looked up
    np.testing.assert_array_equal(got[1, 0, 2], pool[5, 0, 0])
    assert (got[1, 0, 3:] == 0).all()
    with pytest.raises(ValueError):
        oracle.paged_gather(pool, np.array([[9]], dtype=np.int32), [1])


def test_paged_append_commutes_with_gather():
    """Appending to the paged cache and then writing it out contiguously gives what appending to the
    written-out cache gives."""
    rng = np.random.default_rng(5)
    B, Hkv, bs, D, gamma, mb = 3, 2, 4, 3, 2, 4
    R = gamma + 1
    nb = B * mb + 2
    perm = rng.permutation(nb)[:B * mb].reshape(B, mb).astype(np.int32)
    kp = rng.integers(1, 60000, (nb, Hkv, bs, D)).astype(np.uint16)
    vp = rng.integers(1, 60000, (nb, Hkv, bs, D)).astype(np.uint16)
    ctx = np.array([5, 0, 14], dtype=np.int32)          # the last one has no room for 3 more of 16
    kn = rng.integers(1, 60000, (B, R, Hkv, D)).astype(np.uint16)
    vn = rng.integers(1, 60000, (B, R, Hkv, D)).astype(np.uint16)
    kp2, vp2, ctx2, over, bad = oracle.kv_append_paged(kp, vp, perm, kn, vn, ctx, gamma)
    assert over and not bad
    kc, vc, ctx3, over3 = oracle.kv_append(oracle.paged_gather(kp, perm, [mb * bs] * B),
                                           oracle.paged_gather(vp, perm, [mb * bs] * B), kn, vn, ctx, gamma)
    np.testing.assert_array_equal(ctx2, ctx3)
    np.testing.assert_array_equal(ctx2, [8, 3, 14])
    np.testing.assert_array_equal(oracle.paged_gather(kp2, perm, [mb * bs] * B), kc)
    np.testing.assert_array_equal(oracle.paged_gather(vp2, perm, [mb * bs] * B), vc)
    # blocks no table entry names are untouched
    unused = sorted(set(range(nb)) - set(perm.ravel().tolist()))
    np.testing.assert_array_equal(kp2[unused], kp[unused])
