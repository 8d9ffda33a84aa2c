"""Seeded synthetic inputs for the RAPID verify step.

This module holds no arithmetic of the method: it only draws random tensors of
the shapes, sizes and value laws of the five named workloads (LLaMA-3.1-8B /
70B and Qwen2.5-7B shaped layers over 4K..128K-token caches, vocabularies of
4,096 / 128,256 / 152,064) and hands the same bits to whoever asks -- the CUDA
library and the CPU oracle both read inputs made here.

They stand in for the long-context benchmark prompts the paper evaluates on
(>100K-token documents): only shapes and lengths matter to this path.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional, Sequence

import torch


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    B: int
    Hq: int
    Hkv: int
    D: int
    gamma: int
    V: int
    ctx_lens: Optional[Sequence[int]] = None  # fixed lengths; None => drawn from ctx_range
    ctx_range: Optional[tuple] = None         # inclusive (lo, hi), uniform per sequence
    Lmax: Optional[int] = None                # cache capacity; None => max length
    draft_sigma: float = 2.0                  # draft logits ~ N(0, draft_sigma^2)
    target_sigma: float = 0.5                 # target = draft + N(0, target_sigma^2)
    eta: float = 0.5
    temperature: float = 1.0
    tail_alpha: float = 0.1
    layers: int = 1                           # independently seeded caches (seed + layer)
    q_scale: float = 1.0                      # multiplies the N(0,1) query rows

    @property
    def R(self) -> int:
        return self.gamma + 1

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv


CONFIGS = {
    "tiny": VerifyConfig("tiny", B=1, Hq=8, Hkv=2, D=64, gamma=4, V=4096, ctx_lens=(4096,)),
    "llama8b_32k": VerifyConfig("llama8b_32k", B=1, Hq=32, Hkv=8, D=128, gamma=8, V=128256,
                                ctx_lens=(32768,)),
    "llama8b_128k": VerifyConfig("llama8b_128k", B=1, Hq=32, Hkv=8, D=128, gamma=8, V=128256,
                                 ctx_lens=(131072,), layers=32),
    "llama70b_128k": VerifyConfig("llama70b_128k", B=1, Hq=64, Hkv=8, D=128, gamma=8, V=128256,
                                  ctx_lens=(131072,)),
    "drafter_8k": VerifyConfig("drafter_8k", B=1, Hq=32, Hkv=8, D=128, gamma=0, V=128256,
                               ctx_lens=(8192,)),
    "qwen7b_ragged": VerifyConfig("qwen7b_ragged", B=8, Hq=28, Hkv=4, D=128, gamma=4, V=152064,
                                  ctx_range=(16384, 65536), Lmax=65536, target_sigma=1.0),
}


def with_overrides(cfg: VerifyConfig, **kw) -> VerifyConfig:
    return replace(cfg, **kw)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def context_lengths(cfg: VerifyConfig, seed: int) -> torch.Tensor:
    """Per-sequence context lengths [B] int32 (CPU)."""
    if cfg.ctx_lens is not None:
        assert len(cfg.ctx_lens) == cfg.B
        return torch.tensor(list(cfg.ctx_lens), dtype=torch.int32)
    lo, hi = cfg.ctx_range
    g = _gen(seed * 7919 + 11, "cpu")
    return torch.randint(lo, hi + 1, (cfg.B,), generator=g, dtype=torch.int32)


def cache_capacity(cfg: VerifyConfig, ctx_lens: torch.Tensor) -> int:
    return int(cfg.Lmax) if cfg.Lmax is not None else int(ctx_lens.max())


def attention_inputs(cfg: VerifyConfig, seed: int, device="cpu", layer: int = 0,
                     poison_padding: bool = False):
    """Draw q [B,R,Hq,D], k, v [B,Hkv,Lmax,D] (bf16, ~N(0,1)) and ctx_lens [B] int32.

    ``poison_padding`` fills cache entries at positions >= ctx_lens[b] with NaN
    bit patterns: a correct implementation never lets them reach an output.
    """
    ctx = context_lengths(cfg, seed)
    Lmax = cache_capacity(cfg, ctx)
    g = _gen(seed * 1000003 + 17 * layer + 1, device)
    q = (torch.randn(cfg.B, cfg.R, cfg.Hq, cfg.D, generator=g, device=device,
                     dtype=torch.float32) * cfg.q_scale).to(torch.bfloat16)
    k = torch.empty(cfg.B, cfg.Hkv, Lmax, cfg.D, device=device, dtype=torch.bfloat16)
    v = torch.empty_like(k)
    # one (sequence, head) slab at a time keeps the fp32 staging buffer small at 128K
    for b in range(cfg.B):
        for h in range(cfg.Hkv):
            k[b, h] = torch.randn(Lmax, cfg.D, generator=g, device=device, dtype=torch.float32)
            v[b, h] = torch.randn(Lmax, cfg.D, generator=g, device=device, dtype=torch.float32)
    if poison_padding:
        for b in range(cfg.B):
            L = int(ctx[b])
            if L < Lmax:
                k[b, :, L:] = float("nan")
                v[b, :, L:] = float("nan")
    return q, k, v, ctx.to(device)


def paged_layout(k: torch.Tensor, v: torch.Tensor, ctx_lens: torch.Tensor, block_size: int, seed: int,
                 spare_blocks: int = 3, token_major: bool = False):
    """Scatter contiguous caches k, v [B,Hkv,Lmax,D] into a pool of ``block_size``-key blocks in a
    seeded random physical order, as a serving engine's allocator would leave them.

    Returns (k_pool, v_pool, block_table): pools [num_blocks, Hkv, block_size, D] (a strided view of
    [num_blocks, block_size, Hkv, D] storage when ``token_major``), block_table [B, max_blocks] int32.
    Blocks no sequence uses (``spare_blocks`` of them, and table entries past a sequence's length,
    which are -1) hold NaN: nothing may read them."""
    B, Hkv, Lmax, D = k.shape
    mb = (Lmax + block_size - 1) // block_size
    used = [(int(ctx_lens[b]) + block_size - 1) // block_size for b in range(B)]
    nb = sum(used) + spare_blocks
    g = _gen(seed * 3000017 + 23, "cpu")
    perm = torch.randperm(nb, generator=g)
    table = torch.full((B, mb), -1, dtype=torch.int32)
    if token_major:
        kp = torch.full((nb, block_size, Hkv, D), float("nan"), dtype=k.dtype, device=k.device).permute(0, 2, 1, 3)
        vp = torch.full((nb, block_size, Hkv, D), float("nan"), dtype=k.dtype, device=k.device).permute(0, 2, 1, 3)
    else:
        kp = torch.full((nb, Hkv, block_size, D), float("nan"), dtype=k.dtype, device=k.device)
        vp = torch.full((nb, Hkv, block_size, D), float("nan"), dtype=k.dtype, device=k.device)
    nxt = 0
    for b in range(B):
        for i in range(used[b]):
            blk = int(perm[nxt]); nxt += 1
            table[b, i] = blk
            lo, hi = i * block_size, min((i + 1) * block_size, Lmax)
            kp[blk, :, :hi - lo] = k[b, :, lo:hi]
            vp[blk, :, :hi - lo] = v[b, :, lo:hi]
    return kp, vp, table.to(k.device)


def retrieval_inputs(B: int, n_chunks: int, dim: int, seed: int, device="cpu", lo: float = 0.05, hi: float = 0.75):
    """Unit-norm chunk embeddings [B, n_chunks, dim] and query embeddings [B, dim] (float32) whose
    cosine similarities are spread over roughly [lo, hi], i.e. on both sides of the 0.3 threshold the
    paper filters at -- the shape of a 128K-token context cut into 512-token chunks (256 of them)
    embedded in 1024 dimensions.  Each chunk is a mix of the query direction and fresh noise."""
    g = _gen(seed * 4000037 + 29, device)
    q = torch.randn(B, dim, generator=g, device=device, dtype=torch.float32)
    q = q / q.norm(dim=-1, keepdim=True)
    a = lo + (hi - lo) * torch.rand(B, n_chunks, 1, generator=g, device=device, dtype=torch.float32)
    noise = torch.randn(B, n_chunks, dim, generator=g, device=device, dtype=torch.float32)
    noise = noise / noise.norm(dim=-1, keepdim=True)
    e = a * q[:, None, :] + (1 - a * a).sqrt() * noise
    e = e * (0.5 + torch.rand(B, n_chunks, 1, generator=g, device=device, dtype=torch.float32))  # norms vary
    return e.contiguous(), q.contiguous()


def accept_inputs(cfg: VerifyConfig, seed: int, device="cpu"):
    """Draw target_logits [B,R,V] f32, draft_logits [B,gamma,V] f32,
    draft_tokens [B,gamma] i32 (each ~ softmax of its draft row, by a library
    multinomial draw in fp64) and uniforms [B,R] f32 in [0,1)."""
    g = _gen(seed * 2000003 + 5, device)
    B, R, gamma, V = cfg.B, cfg.R, cfg.gamma, cfg.V
    draft = torch.randn(B, gamma, V, generator=g, device=device, dtype=torch.float32) * cfg.draft_sigma
    target = torch.randn(B, R, V, generator=g, device=device, dtype=torch.float32) * cfg.target_sigma
    if gamma > 0:
        target[:, :gamma] += draft
    # the bonus row has no draft row under it: give it the same marginal law
    target[:, gamma] += torch.randn(B, V, generator=g, device=device, dtype=torch.float32) * cfg.draft_sigma
    if gamma > 0:
        probs = torch.softmax(draft.double() / cfg.temperature, dim=-1).reshape(B * gamma, V)
        tokens = torch.multinomial(probs, 1, generator=g).reshape(B, gamma).to(torch.int32)
    else:
        tokens = torch.zeros(B, 0, dtype=torch.int32, device=device)
    uniforms = torch.rand(B, R, generator=g, device=device, dtype=torch.float32)
    return target, draft, tokens, uniforms


def bf16_bits(t: torch.Tensor):
    """Raw bits of a bf16 tensor as a numpy uint16 array on the host."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view("uint16")


def attention_inputs_fp8(cfg: VerifyConfig, seed: int, device="cpu", layer: int = 0, poison_padding: bool = False):
    """The same draws as ``attention_inputs`` with the cache stored as FP8 E4M3 codes: every (sequence,
    KV head) slab of K and of V ~ N(0,1) is divided by its own scale (largest magnitude / 448, the
    format's largest value) and rounded to E4M3 by the library's conversion.
    Returns q [B,R,Hq,D] bf16, k_codes, v_codes [B,Hkv,Lmax,D] uint8, k_scale, v_scale [B,Hkv] float32,
    ctx_lens [B] int32.  ``poison_padding`` fills positions >= ctx_lens[b] with the NaN code."""
    ctx = context_lengths(cfg, seed)
    Lmax = cache_capacity(cfg, ctx)
    g = _gen(seed * 1000003 + 17 * layer + 1, device)
    q = (torch.randn(cfg.B, cfg.R, cfg.Hq, cfg.D, generator=g, device=device,
                     dtype=torch.float32) * cfg.q_scale).to(torch.bfloat16)
    kc = torch.empty(cfg.B, cfg.Hkv, Lmax, cfg.D, device=device, dtype=torch.uint8)
    vc = torch.empty_like(kc)
    ks = torch.empty(cfg.B, cfg.Hkv, device=device, dtype=torch.float32)
    vs = torch.empty_like(ks)
    for b in range(cfg.B):
        for h in range(cfg.Hkv):
            for codes, scales in ((kc, ks), (vc, vs)):
                x = torch.randn(Lmax, cfg.D, generator=g, device=device, dtype=torch.float32)
                s = x.abs().max() / 448.0
                scales[b, h] = s
                codes[b, h] = (x / s).to(torch.float8_e4m3fn).view(torch.uint8)
    if poison_padding:
        for b in range(cfg.B):
            L = int(ctx[b])
            if L < Lmax:
                kc[b, :, L:] = 0x7F
                vc[b, :, L:] = 0xFF
    return q, kc, vc, ks, vs, ctx.to(device)
