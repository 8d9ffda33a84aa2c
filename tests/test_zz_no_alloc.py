"""rapid_accept_static: the accept step for callers that may not allocate device memory.

Some users of the library run where obtaining device memory is off the table -- inside a host
process that owns the whole GPU memory pool, or in a decode loop that must not touch the
allocator once it is warm.  For them the library carries its own fixed scratch array.  This
test calls that entry point through the C ABI, twice in a row on different inputs, and
requires the same outputs as the ordinary rapid_accept with a caller workspace (same
kernels, so the comparison is exact); the second call also shows that nothing stale from the
first one (its status bit, its per-row statistics) leaks into the next.

The file name keeps this test last in collection order.
"""
import pytest
import torch

pytestmark = pytest.mark.gpu

import workloads as wl


def _reference(R, z, d, tok, u, eta, params):
    B, Rr, V = z.shape
    ws = R.new_workspace(R.accept_workspace_bytes(B, Rr - 1, V))
    alen = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    ntok = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    R.rapid_accept(z, d, tok, u, eta, alen, ntok, ws, params)
    torch.cuda.synchronize()
    return alen, ntok, R.workspace_status(ws)


def test_static_scratch_matches_workspace_version_on_two_calls():
    import paper_2502_20330_b200 as R
    cfg1 = wl.VerifyConfig("a", B=8, Hq=8, Hkv=2, D=64, gamma=4, V=32000, ctx_lens=(64,) * 8, target_sigma=1.0)
    cfg2 = wl.VerifyConfig("b", B=3, Hq=8, Hkv=2, D=64, gamma=7, V=128256, ctx_lens=(64,) * 3, target_sigma=1.0)
    calls = []
    for seed, cfg, eta, params in ((31, cfg1, 5.0, R.AcceptParams(temperature=1.0, tail_alpha=0.1)),
                                   (32, cfg2, 20.0, R.AcceptParams(temperature=0.5, tail_alpha=0.1, residual_mode=1))):
        z, d, tok, u = wl.accept_inputs(cfg, seed=seed, device="cuda")
        calls.append((z, d, tok, u, eta, params))
    # first call carries an out-of-range draft token so that it leaves a status bit behind
    calls[0][2][0, 0] = 10 ** 6

    for z, d, tok, u, eta, params in calls:
        alen = torch.full((z.shape[0],), -1, dtype=torch.int32, device="cuda")
        ntok = torch.full_like(alen, -1)
        status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        R.rapid_accept_static(z, d, tok, u, eta, alen, ntok, params, out_status=status)
        torch.cuda.synchronize()
        ref_alen, ref_ntok, ref_status = _reference(R, z, d, tok, u, eta, params)
        assert torch.equal(alen, ref_alen)
        assert torch.equal(ntok, ref_ntok)
        assert int(status.item()) == ref_status
    assert ref_status == 0          # the second call saw none of the first call's status bit


def test_static_scratch_rejects_shapes_beyond_its_size():
    import paper_2502_20330_b200 as R
    z = torch.zeros(103, 5, 64, device="cuda")       # 515 logit rows > 512
    d = torch.zeros(103, 4, 64, device="cuda")
    tok = torch.zeros(103, 4, dtype=torch.int32, device="cuda")
    u = torch.zeros(103, 5, device="cuda")
    o = torch.zeros(103, dtype=torch.int32, device="cuda")
    with pytest.raises(R.RapidError) as e:
        R.rapid_accept_static(z, d, tok, u, 0.5, o, o.clone())
    assert e.value.code == 2 and "512" in str(e.value)
