"""The chained verify step and its host-buffer form, against the oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from oracle import parity
import workloads as wl
from workloads import bf16_bits


def _inputs(cfg, seed, device):
    q, k, v, ctx = wl.attention_inputs(cfg, seed=seed, device=device)
    z, d, tok, u = wl.accept_inputs(cfg, seed=seed, device=device)
    return q, k, v, ctx, z, d, tok, u


def test_verify_step_chains_both_calls():
    import paper_2502_20330_b200 as R
    cfg = wl.CONFIGS["tiny"]
    q, k, v, ctx, z, d, tok, u = _inputs(cfg, 21, "cuda")
    aws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, k.shape[2], cfg.gamma))
    cws = R.new_workspace(R.accept_workspace_bytes(cfg.B, cfg.gamma, cfg.V))
    out = torch.empty_like(q)
    alen = torch.zeros(cfg.B, dtype=torch.int32, device="cuda"); ntok = torch.zeros_like(alen)
    R.kernel_launch_count_reset()
    R.rapid_verify_step(q, k, v, ctx, cfg.gamma, out, aws, z, d, tok, u, cfg.eta, alen, ntok, cws)
    torch.cuda.synchronize()
    assert R.kernel_launch_count() == 4  # plan, split, merge, accept
    ref, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx.cpu().numpy(), cfg.gamma)
    parity.check_attention(out.float().cpu().numpy(), ref)
    parity.check_accept(z.cpu().numpy(), d.cpu().numpy(), tok.cpu().numpy(), u.cpu().numpy(), cfg.eta, 1.0, 0.1, 0,
                        alen.cpu().numpy(), ntok.cpu().numpy())
    assert R.workspace_status(aws) == 0 and R.workspace_status(cws) == 0


def test_verify_step_host_buffers():
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("t", B=2, Hq=8, Hkv=2, D=128, gamma=3, V=4096, ctx_lens=(700, 300), Lmax=768)
    q, k, v, ctx, z, d, tok, u = [t.pin_memory() for t in _inputs(cfg, 22, "cpu")]
    arena = torch.empty(R.verify_step_host_arena_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, 768, cfg.gamma, cfg.V),
                        dtype=torch.uint8, device="cuda")
    out = torch.empty_like(q).pin_memory()
    alen = torch.zeros(cfg.B, dtype=torch.int32).pin_memory(); ntok = torch.zeros(cfg.B, dtype=torch.int32).pin_memory()
    for _ in range(2):
        status = R.rapid_verify_step_host(q, k, v, ctx, cfg.gamma, out, z, d, tok, u, 5.0, alen, ntok, arena)
        assert status == 0
        ref, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx.numpy(), cfg.gamma)
        parity.check_attention(out.float().numpy(), ref)
        parity.check_accept(z.numpy(), d.numpy(), tok.numpy(), u.numpy(), 5.0, 1.0, 0.1, 0, alen.numpy(), ntok.numpy())


def test_verify_step_replays_from_a_cuda_graph():
    """The chained step has no host synchronisation: it can be captured once and replayed."""
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("t", B=2, Hq=32, Hkv=8, D=128, gamma=8, V=32000, ctx_lens=(5000, 3000), target_sigma=1.0)
    q, k, v, ctx, z, d, tok, u = _inputs(cfg, 23, "cuda")
    aws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, k.shape[2], cfg.gamma))
    cws = R.new_workspace(R.accept_workspace_bytes(cfg.B, cfg.gamma, cfg.V))
    out = torch.zeros_like(q)
    alen = torch.zeros(cfg.B, dtype=torch.int32, device="cuda"); ntok = torch.zeros_like(alen)
    # eager reference
    R.rapid_verify_step(q, k, v, ctx, cfg.gamma, out, aws, z, d, tok, u, 5.0, alen, ntok, cws)
    torch.cuda.synchronize()
    ref_out, ref_alen, ref_ntok = out.clone(), alen.clone(), ntok.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            R.rapid_verify_step(q, k, v, ctx, cfg.gamma, out, aws, z, d, tok, u, 5.0, alen, ntok, cws, stream=side)
    for _ in range(3):
        out.zero_(); alen.zero_(); ntok.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, ref_out) and torch.equal(alen, ref_alen) and torch.equal(ntok, ref_ntok)
    # new inputs in the same buffers are picked up by the replay (pointers, not values, are captured)
    q2, k2, v2, _, z2, d2, tok2, u2 = _inputs(cfg, 24, "cuda")
    q.copy_(q2); k.copy_(k2); v.copy_(v2); z.copy_(z2); d.copy_(d2); tok.copy_(tok2); u.copy_(u2)
    g.replay()
    torch.cuda.synchronize()
    ref, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx.cpu().numpy(), cfg.gamma)
    parity.check_attention(out.float().cpu().numpy(), ref)
    parity.check_accept(z.cpu().numpy(), d.cpu().numpy(), tok.cpu().numpy(), u.cpu().numpy(), 5.0, 1.0, 0.1, 0,
                        alen.cpu().numpy(), ntok.cpu().numpy())
    assert R.workspace_status(aws) == 0 and R.workspace_status(cws) == 0


@pytest.mark.parametrize("name,nlayers", [("llama8b_32k", 4), ("drafter_8k", 6)])
def test_overlapping_layers_replay_bit_identically(name, nlayers):
    """A step's layers in one CUDA graph, every layer but the first with a settled plan and early copies of its
    old keys: the next layer's split kernel starts while this layer's still runs.  Forty replays must reproduce
    the first run bit for bit, and layer 0 must match the oracle."""
    import numpy as np
    import oracle
    from oracle import parity
    from workloads import bf16_bits
    import paper_2502_20330_b200 as R
    cfg = wl.CONFIGS[name]
    layers = [wl.attention_inputs(cfg, seed=9 + i, device="cuda", layer=i) for i in range(nlayers)]
    ctx, Lmax = layers[0][3], layers[0][1].shape[2]
    ws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lmax, cfg.gamma))
    outs = [torch.zeros_like(l[0]) for l in layers]

    def step():
        R.rapid_attention_plan(ctx, cfg.gamma, cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lmax, ws, R.AttnParams())
        for i, (q, k, v, _) in enumerate(layers):
            R.rapid_verify_attention(q, k, v, ctx, cfg.gamma, outs[i], ws,
                                     R.AttnParams(plan=R.PLAN_READY if i == 0 else R.PLAN_SETTLED, kv_settled=True))

    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        step()
        torch.cuda.synchronize()
        first = [o.clone() for o in outs]
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            step()
        for _ in range(40):
            for o in outs:
                o.zero_()
            g.replay()
            torch.cuda.synchronize()
            assert all(torch.equal(o, r) for o, r in zip(outs, first))
    assert R.workspace_status(ws) == 0
    q, k, v, _ = layers[0]
    ref, ref_lse = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx.cpu().numpy(), cfg.gamma)
    parity.check_attention(first[0].float().cpu().numpy(), ref, ~np.isnan(ref_lse))
