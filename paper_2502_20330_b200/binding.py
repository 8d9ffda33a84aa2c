"""ctypes binding of include/rapid.h -- argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "librapid.so")

STATUS_BAD_CTX_LEN = 1
STATUS_BAD_DRAFT_TOKEN = 2
STATUS_RESIDUAL_FALLBACK = 4
STATUS_PIPELINE_TIMEOUT = 8
STATUS_BAD_BLOCK_TABLE = 16
STATUS_STALE_PLAN = 32
ATTN_KERNEL_AUTO, ATTN_KERNEL_ROWS_ON_M, ATTN_KERNEL_KEYS_ON_M, ATTN_KERNEL_CLUSTER_MERGE = 0, 1, 2, 3
PLAN_NONE, PLAN_READY, PLAN_SETTLED = 0, 1, 2
RESIDUAL_PAPER = 0
RESIDUAL_PHAT = 1

EXPORTS = [
    "rapid_attention_workspace_bytes", "rapid_accept_workspace_bytes", "rapid_workspace_init",
    "rapid_workspace_status", "rapid_verify_attention", "rapid_verify_attention_fp8", "rapid_attention_plan", "rapid_attention_describe", "rapid_verify_attention_paged", "rapid_merge_partials", "rapid_retrieval_select", "rapid_retrieval_budget_chunks", "rapid_draft_sample", "rapid_accept", "rapid_accept_static",
    "rapid_verify_step",
    "rapid_verify_step_host", "rapid_verify_step_host_arena_bytes", "rapid_kv_append", "rapid_kv_append_paged", "rapid_step_commit",
    "rapid_last_error",
    "rapid_version", "rapid_kernel_launch_count", "rapid_kernel_launch_count_reset",
]


class RapidError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"rapid error {code}: {message}")
        self.code = code


class _AttnShape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32),
                ("D", ctypes.c_int32), ("Lmax", ctypes.c_int64), ("kv_stride_b", ctypes.c_int64),
                ("kv_stride_h", ctypes.c_int64), ("kv_stride_l", ctypes.c_int64)]


class _PagedKv(ctypes.Structure):
    _fields_ = [("block_size", ctypes.c_int32), ("num_blocks", ctypes.c_int32),
                ("max_blocks_per_seq", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("stride_block", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_l", ctypes.c_int64)]


class _AttnParams(ctypes.Structure):
    _fields_ = [("scale", ctypes.c_float), ("num_ctas", ctypes.c_int32),
                ("lse_out", ctypes.c_void_p), ("out_f32", ctypes.c_void_p),
                ("split_done_event", ctypes.c_void_p), ("all_keys_visible", ctypes.c_int32),
                ("kernel", ctypes.c_int32), ("sink_keys", ctypes.c_int32), ("window_keys", ctypes.c_int32),
                ("plan", ctypes.c_int32), ("kv_fp8", ctypes.c_int32), ("wait_cycle_limit", ctypes.c_int64),
                ("kv_settled", ctypes.c_int32)]


class _LaunchInfo(ctypes.Structure):
    _fields_ = [("kernel", ctypes.c_int32), ("kernels_per_call", ctypes.c_int32), ("ctas", ctypes.c_int32),
                ("cluster_size", ctypes.c_int32), ("softmax_groups", ctypes.c_int32), ("columns", ctypes.c_int32),
                ("max_clusters", ctypes.c_int32 * 4)]


class _AcceptShape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("gamma", ctypes.c_int32), ("V", ctypes.c_int64),
                ("target_row_stride", ctypes.c_int64), ("draft_row_stride", ctypes.c_int64)]


class _AcceptParams(ctypes.Structure):
    _fields_ = [("temperature", ctypes.c_float), ("tail_alpha", ctypes.c_float),
                ("residual_mode", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("ratio_out", ctypes.c_void_p), ("draft_row_stats", ctypes.c_void_p), ("draft_logq", ctypes.c_void_p)]


@dataclass
class AttnParams:
    scale: float = 0.0
    num_ctas: int = 0
    lse_out: Optional[torch.Tensor] = None   # [B,R,Hq] float32
    out_f32: Optional[torch.Tensor] = None   # [B,R,Hq,D] float32
    split_done_event: Optional[int] = None   # cudaEvent_t handle recorded between split and merge
    all_keys_visible: bool = False           # no causal stair: a context shard without the rows' own keys
    kernel: int = 0                          # 0 automatic, 1 rows on the MMA's M axis, 2 keys on the M axis,
                                             # 3 keys on M with one cluster per (sequence, KV head), merged on chip
    sink_keys: int = 0                       # with window_keys: the first keys every row keeps seeing
    window_keys: int = 0                     # > 0: each row sees only that many newest keys up to its own
    plan: int = 0                            # PLAN_*: the workspace holds a plan made by rapid_attention_plan
    wait_cycle_limit: int = 0                # clock cycles an on-chip wait may take; 0 = the library's limit
    kv_fp8: bool = False                     # rapid_attention_plan / describe: the plan is for the FP8-cache call
    kv_settled: bool = False                 # with plan = PLAN_SETTLED: all but the newest R keys were final before
                                             # the preceding work was issued; their tiles may be copied early


@dataclass
class AcceptParams:
    temperature: float = 1.0
    tail_alpha: float = 0.1
    residual_mode: int = RESIDUAL_PAPER
    ratio_out: Optional[torch.Tensor] = None  # [B,gamma] float32
    draft_row_stats: Optional[torch.Tensor] = None  # [B,gamma,2] float32: rapid_draft_sample's out_row_stats
    draft_logq: Optional[torch.Tensor] = None       # [B,gamma] float32: rapid_draft_sample's out_logq


_lib = None


def lib_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads librapid.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            # build in-tree with nvcc if the toolchain is here; otherwise fail loudly
            try:
                from . import build as _build
                _build.build()
            except Exception as exc:
                raise RuntimeError(
                    f"{_LIB_PATH} is missing and could not be built ({exc}): run "
                    "`python -m paper_2502_20330_b200.build` (this package has no CPU or PyTorch fallback)")
        lib = ctypes.CDLL(_LIB_PATH)
        vp, i32, i64, sz, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t, ctypes.c_float
        lib.rapid_attention_workspace_bytes.restype = sz
        lib.rapid_attention_workspace_bytes.argtypes = [ctypes.POINTER(_AttnShape), i32]
        lib.rapid_accept_workspace_bytes.restype = sz
        lib.rapid_accept_workspace_bytes.argtypes = [ctypes.POINTER(_AcceptShape)]
        lib.rapid_workspace_init.restype = i32
        lib.rapid_workspace_init.argtypes = [vp, sz, vp]
        lib.rapid_workspace_status.restype = i32
        lib.rapid_workspace_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32)]
        attn_args = [vp, vp, vp, vp, i32, vp, ctypes.POINTER(_AttnShape), ctypes.POINTER(_AttnParams)]
        acc_args = [vp, vp, vp, vp, f32, vp, vp, ctypes.POINTER(_AcceptShape), ctypes.POINTER(_AcceptParams)]
        lib.rapid_verify_attention.restype = i32
        lib.rapid_verify_attention.argtypes = attn_args + [vp, sz, vp]
        lib.rapid_verify_attention_fp8.restype = i32
        lib.rapid_verify_attention_fp8.argtypes = [vp, vp, vp, vp, vp] + attn_args[3:] + [vp, sz, vp]
        lib.rapid_attention_plan.restype = i32
        lib.rapid_attention_plan.argtypes = [vp, i32, ctypes.POINTER(_AttnShape), ctypes.POINTER(_AttnParams), vp, sz, vp]
        lib.rapid_attention_describe.restype = i32
        lib.rapid_attention_describe.argtypes = [ctypes.POINTER(_AttnShape), i32, ctypes.POINTER(_AttnParams),
                                                 ctypes.POINTER(_LaunchInfo)]
        lib.rapid_verify_attention_paged.restype = i32
        lib.rapid_verify_attention_paged.argtypes = [vp, vp, vp, vp, ctypes.POINTER(_PagedKv)] + attn_args[3:] + [vp, sz, vp]
        lib.rapid_draft_sample.restype = i32
        lib.rapid_draft_sample.argtypes = [vp, vp, f32, vp, vp, vp, i32, i64, i64, vp, sz, vp]
        lib.rapid_retrieval_select.restype = i32
        lib.rapid_retrieval_select.argtypes = [vp, vp, vp, i32, i32, i32, f32, i32, vp, vp, vp, vp, vp]
        lib.rapid_retrieval_budget_chunks.restype = i64
        lib.rapid_retrieval_budget_chunks.argtypes = [i64, i32, i32, i32]
        lib.rapid_merge_partials.restype = i32
        lib.rapid_merge_partials.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp, vp]
        lib.rapid_accept.restype = i32
        lib.rapid_accept.argtypes = acc_args + [vp, sz, vp]
        lib.rapid_accept_static.restype = i32
        lib.rapid_accept_static.argtypes = acc_args + [vp, vp]
        lib.rapid_verify_step.restype = i32
        lib.rapid_verify_step.argtypes = attn_args + [vp, sz] + acc_args + [vp, sz, vp]
        lib.rapid_verify_step_host.restype = i32
        lib.rapid_verify_step_host.argtypes = attn_args + acc_args + [vp, sz, ctypes.POINTER(ctypes.c_int32), vp]
        lib.rapid_verify_step_host_arena_bytes.restype = sz
        lib.rapid_verify_step_host_arena_bytes.argtypes = [ctypes.POINTER(_AttnShape), i32, ctypes.POINTER(_AcceptShape)]
        lib.rapid_kv_append.restype = i32
        lib.rapid_kv_append.argtypes = [vp, vp, vp, vp, vp, i32, ctypes.POINTER(_AttnShape), vp, vp]
        lib.rapid_kv_append_paged.restype = i32
        lib.rapid_kv_append_paged.argtypes = [vp, vp, vp, vp, vp, ctypes.POINTER(_PagedKv), vp, i32, i32, i32, i32, vp, vp]
        lib.rapid_step_commit.restype = i32
        lib.rapid_step_commit.argtypes = [vp, vp, i32, i32, vp, vp]
        lib.rapid_last_error.restype = ctypes.c_char_p
        lib.rapid_version.restype = i32
        lib.rapid_kernel_launch_count.restype = i64
        lib.rapid_kernel_launch_count_reset.restype = None
        _lib = lib
    return _lib


def last_error() -> str:
    return load_library().rapid_last_error().decode()


def version() -> int:
    return int(load_library().rapid_version())


def kernel_launch_count() -> int:
    return int(load_library().rapid_kernel_launch_count())


def kernel_launch_count_reset() -> None:
    load_library().rapid_kernel_launch_count_reset()


def _check(rc: int):
    if rc != 0:
        raise RapidError(rc, last_error())


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _p(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _attn_shape(q: torch.Tensor, k: torch.Tensor) -> _AttnShape:
    B, R, Hq, D = q.shape
    Bk, Hkv, Lmax, Dk = k.shape
    if Bk != B or Dk != D:
        raise ValueError("q and k_cache disagree on batch or head_dim")
    if k.stride(3) != 1:
        raise ValueError("k_cache / v_cache must have a contiguous head_dim")
    return _AttnShape(B, Hq, Hkv, D, Lmax, k.stride(0), k.stride(1), k.stride(2))


def _attn_params(p: Optional[AttnParams]):
    if p is None:
        return None
    return ctypes.byref(_AttnParams(p.scale, p.num_ctas, p.lse_out.data_ptr() if p.lse_out is not None else None,
                                    p.out_f32.data_ptr() if p.out_f32 is not None else None,
                                    p.split_done_event, 1 if p.all_keys_visible else 0, int(p.kernel),
                                    int(p.sink_keys), int(p.window_keys), int(p.plan), 1 if p.kv_fp8 else 0,
                                    int(p.wait_cycle_limit), 1 if p.kv_settled else 0))


def _accept_shape(target_logits: torch.Tensor, draft_logits: torch.Tensor) -> _AcceptShape:
    B, R, V = target_logits.shape
    if target_logits.stride(2) != 1 or (draft_logits.numel() and draft_logits.stride(-1) != 1):
        raise ValueError("logits must be contiguous along the vocabulary")
    zs = target_logits.stride(1)
    ds = draft_logits.stride(1) if R > 1 else V
    if R > 1 and (target_logits.stride(0) != R * zs or draft_logits.stride(0) != (R - 1) * ds):
        raise ValueError("logit rows must be equally spaced")
    return _AcceptShape(B, R - 1, V, zs, ds)


def _accept_params(p: Optional[AcceptParams]):
    if p is None:
        return None
    for t in (p.draft_row_stats, p.draft_logq):
        if t is not None and (t.dtype != torch.float32 or not t.is_contiguous()):
            raise TypeError("draft_row_stats and draft_logq must be dense float32")
    return ctypes.byref(_AcceptParams(p.temperature, p.tail_alpha, p.residual_mode, 0,
                                      p.ratio_out.data_ptr() if p.ratio_out is not None else None,
                                      p.draft_row_stats.data_ptr() if p.draft_row_stats is not None else None,
                                      p.draft_logq.data_ptr() if p.draft_logq is not None else None))


def attention_workspace_bytes(B, Hq, Hkv, D, Lmax, gamma) -> int:
    s = _AttnShape(B, Hq, Hkv, D, Lmax, 0, 0, 0)
    return int(load_library().rapid_attention_workspace_bytes(ctypes.byref(s), gamma))


def accept_workspace_bytes(B, gamma, V) -> int:
    s = _AcceptShape(B, gamma, V, 0, 0)
    return int(load_library().rapid_accept_workspace_bytes(ctypes.byref(s)))


def verify_step_host_arena_bytes(B, Hq, Hkv, D, Lmax, gamma, V) -> int:
    a = _AttnShape(B, Hq, Hkv, D, Lmax, 0, 0, 0)
    c = _AcceptShape(B, gamma, V, 0, 0)
    return int(load_library().rapid_verify_step_host_arena_bytes(ctypes.byref(a), gamma, ctypes.byref(c)))


def workspace_init(workspace: torch.Tensor, stream=None) -> None:
    _check(load_library().rapid_workspace_init(_p(workspace), workspace.numel() * workspace.element_size(),
                                               _stream_ptr(stream)))


def new_workspace(nbytes: int, device="cuda", stream=None) -> torch.Tensor:
    """Allocates (with torch) and initialises a workspace of at least nbytes."""
    if nbytes <= 0:
        raise ValueError("workspace size query failed (invalid shape?)")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    workspace_init(ws, stream)
    return ws


def workspace_status(workspace: torch.Tensor, stream=None) -> int:
    out = ctypes.c_int32(0)
    _check(load_library().rapid_workspace_status(_p(workspace), _stream_ptr(stream), ctypes.byref(out)))
    return int(out.value)


def _nbytes(t: torch.Tensor) -> int:
    return t.numel() * t.element_size()


def rapid_verify_attention(q, k_cache, v_cache, ctx_lens, gamma, out, workspace, params: Optional[AttnParams] = None,
                           stream=None) -> None:
    """out[B,R,Hq,D] <- verify attention of q[B,R,Hq,D] over k_cache/v_cache[B,Hkv,Lmax,D] (bf16, CUDA)."""
    if q.dtype != torch.bfloat16 or k_cache.dtype != torch.bfloat16 or v_cache.dtype != torch.bfloat16 \
            or out.dtype != torch.bfloat16 or ctx_lens.dtype != torch.int32:
        raise TypeError("q/k/v/out must be bfloat16 and ctx_lens int32")
    if not (q.is_contiguous() and out.is_contiguous()) or q.shape[1] != gamma + 1 or out.shape != q.shape:
        raise ValueError("q and out must be dense [B, gamma+1, Hq, D]")
    if k_cache.stride() != v_cache.stride() or k_cache.shape != v_cache.shape:
        raise ValueError("k_cache and v_cache must share shape and strides")
    shape = _attn_shape(q, k_cache)
    _check(load_library().rapid_verify_attention(_p(q), _p(k_cache), _p(v_cache), _p(ctx_lens), gamma, _p(out),
                                                 ctypes.byref(shape), _attn_params(params), _p(workspace),
                                                 _nbytes(workspace), _stream_ptr(stream)))


def rapid_verify_attention_fp8(q, k_cache, v_cache, k_scale, v_scale, ctx_lens, gamma, out, workspace,
                               params: Optional[AttnParams] = None, stream=None) -> None:
    """Verify attention over an FP8 E4M3 cache: k_cache / v_cache [B,Hkv,Lmax,D] uint8 (or torch.float8_e4m3fn)
    codes, k_scale / v_scale [B,Hkv] float32; q and out bfloat16."""
    if q.dtype != torch.bfloat16 or out.dtype != torch.bfloat16 or ctx_lens.dtype != torch.int32:
        raise TypeError("q/out must be bfloat16 and ctx_lens int32")
    if k_cache.element_size() != 1 or v_cache.element_size() != 1:
        raise TypeError("k_cache / v_cache must hold one-byte E4M3 codes")
    if k_scale.dtype != torch.float32 or v_scale.dtype != torch.float32 or not (k_scale.is_contiguous() and v_scale.is_contiguous()):
        raise TypeError("k_scale / v_scale must be dense float32 [B, Hkv]")
    if not (q.is_contiguous() and out.is_contiguous()) or q.shape[1] != gamma + 1 or out.shape != q.shape:
        raise ValueError("q and out must be dense [B, gamma+1, Hq, D]")
    if k_cache.stride() != v_cache.stride() or k_cache.shape != v_cache.shape:
        raise ValueError("k_cache and v_cache must share shape and strides")
    if k_scale.shape != (q.shape[0], k_cache.shape[1]) or v_scale.shape != k_scale.shape:
        raise ValueError("k_scale / v_scale must be [B, Hkv]")
    shape = _attn_shape(q, k_cache)
    _check(load_library().rapid_verify_attention_fp8(_p(q), _p(k_cache), _p(v_cache), _p(k_scale), _p(v_scale),
                                                     _p(ctx_lens), gamma, _p(out), ctypes.byref(shape),
                                                     _attn_params(params), _p(workspace), _nbytes(workspace),
                                                     _stream_ptr(stream)))


def rapid_attention_plan(ctx_lens, gamma, B, Hq, Hkv, D, Lmax, workspace, params: Optional[AttnParams] = None,
                         stream=None) -> None:
    """Writes the work split of the attention calls over ``ctx_lens`` into ``workspace`` once; calls that
    name the same workspace with ``params.plan`` set read it instead of working it out again."""
    if ctx_lens.dtype != torch.int32 or ctx_lens.numel() != B:
        raise TypeError("ctx_lens must be int32 [B]")
    shape = _AttnShape(B, Hq, Hkv, D, Lmax, 0, 0, 0)
    _check(load_library().rapid_attention_plan(_p(ctx_lens), gamma, ctypes.byref(shape), _attn_params(params),
                                               _p(workspace), _nbytes(workspace), _stream_ptr(stream)))


def rapid_attention_describe(B, Hq, Hkv, D, Lmax, gamma, params: Optional[AttnParams] = None) -> dict:
    """What an attention call of this geometry would launch on the current device (see include/rapid.h)."""
    shape = _AttnShape(B, Hq, Hkv, D, Lmax, 0, 0, 0)
    info = _LaunchInfo()
    _check(load_library().rapid_attention_describe(ctypes.byref(shape), gamma, _attn_params(params), ctypes.byref(info)))
    return {"kernel": info.kernel, "kernels_per_call": info.kernels_per_call, "ctas": info.ctas,
            "cluster_size": info.cluster_size, "softmax_groups": info.softmax_groups, "columns": info.columns,
            "max_clusters": {16: info.max_clusters[0], 8: info.max_clusters[1], 4: info.max_clusters[2],
                             2: info.max_clusters[3]}}


def rapid_verify_attention_paged(q, k_pool, v_pool, block_table, ctx_lens, gamma, out, workspace,
                                 params: Optional[AttnParams] = None, stream=None) -> None:
    """Verify attention over a paged cache: k_pool/v_pool [num_blocks, Hkv, block_size, D] bf16 (any
    strides with a contiguous head_dim), block_table [B, max_blocks_per_seq] int32."""
    if q.dtype != torch.bfloat16 or k_pool.dtype != torch.bfloat16 or v_pool.dtype != torch.bfloat16 \
            or out.dtype != torch.bfloat16 or ctx_lens.dtype != torch.int32 or block_table.dtype != torch.int32:
        raise TypeError("q/k/v/out must be bfloat16, ctx_lens and block_table int32")
    if not (q.is_contiguous() and out.is_contiguous()) or q.shape[1] != gamma + 1 or out.shape != q.shape:
        raise ValueError("q and out must be dense [B, gamma+1, Hq, D]")
    if k_pool.stride() != v_pool.stride() or k_pool.shape != v_pool.shape or k_pool.stride(3) != 1:
        raise ValueError("k_pool and v_pool must share shape and strides, with a contiguous head_dim")
    if not block_table.is_contiguous() or block_table.shape[0] != q.shape[0]:
        raise ValueError("block_table must be dense [B, max_blocks_per_seq]")
    B, R, Hq, D = q.shape
    nb, Hkv, bs, Dk = k_pool.shape
    if Dk != D:
        raise ValueError("q and k_pool disagree on head_dim")
    mb = block_table.shape[1]
    shape = _AttnShape(B, Hq, Hkv, D, mb * bs, 0, 0, 0)
    paged = _PagedKv(bs, nb, mb, 0, k_pool.stride(0), k_pool.stride(1), k_pool.stride(2))
    _check(load_library().rapid_verify_attention_paged(_p(q), _p(k_pool), _p(v_pool), _p(block_table),
                                                       ctypes.byref(paged), _p(ctx_lens), gamma, _p(out),
                                                       ctypes.byref(shape), _attn_params(params), _p(workspace),
                                                       _nbytes(workspace), _stream_ptr(stream)))


def rapid_draft_sample(draft_logits, uniforms, temperature, out_token, out_logq, workspace, out_row_stats=None,
                       stream=None) -> None:
    """x' ~ softmax(draft_logits / T) by inverse CDF with the given uniforms; also log q(x') and, optionally,
    (max, log-sum-exp) of every row.  draft_logits [B, V] float32 (rows may be strided), uniforms [B]."""
    if draft_logits.dtype != torch.float32 or uniforms.dtype != torch.float32 or out_logq.dtype != torch.float32:
        raise TypeError("logits, uniforms and out_logq must be float32")
    if out_token.dtype != torch.int32 or (out_row_stats is not None and out_row_stats.dtype != torch.float32):
        raise TypeError("out_token must be int32 and out_row_stats float32")
    if draft_logits.dim() != 2 or draft_logits.stride(1) != 1:
        raise ValueError("draft_logits must be [B, V] with a contiguous vocabulary axis")
    B, V = draft_logits.shape
    if uniforms.numel() != B or out_token.numel() != B or out_logq.numel() != B or \
            (out_row_stats is not None and (out_row_stats.numel() != 2 * B or not out_row_stats.is_contiguous())):
        raise ValueError("uniforms, out_token, out_logq must hold B entries and out_row_stats [B, 2]")
    _check(load_library().rapid_draft_sample(_p(draft_logits), _p(uniforms), float(temperature), _p(out_token),
                                             _p(out_logq), _p(out_row_stats), B, V, draft_logits.stride(0),
                                             _p(workspace), _nbytes(workspace), _stream_ptr(stream)))


def rapid_retrieval_budget_chunks(context_tokens: int, chunk_tokens: int = 512, floor_tokens: int = 4096,
                                  divisor: int = 24) -> int:
    """Chunks the retrieved context may hold (the library's rapid_retrieval_budget_chunks)."""
    k = load_library().rapid_retrieval_budget_chunks(int(context_tokens), int(chunk_tokens), int(floor_tokens),
                                                     int(divisor))
    if k < 0:
        raise ValueError(load_library().rapid_last_error().decode())
    return int(k)


def rapid_retrieval_select(chunk_emb, query_emb, k, status_word, threshold=0.3, n_chunks=None, stream=None):
    """Cosine scores of chunk_emb [B, Nmax, Dm] against query_emb [B, Dm] (float32) and the k best chunks
    at or above ``threshold``.  Returns (scores [B, Nmax], sel_idx [B, k] padded with -1, sel_count [B])."""
    if chunk_emb.dtype != torch.float32 or query_emb.dtype != torch.float32:
        raise TypeError("embeddings must be float32")
    if chunk_emb.dim() != 3 or not chunk_emb.is_contiguous() or not query_emb.is_contiguous() \
            or query_emb.shape != (chunk_emb.shape[0], chunk_emb.shape[2]):
        raise ValueError("chunk_emb must be dense [B, Nmax, Dm] and query_emb dense [B, Dm]")
    if n_chunks is not None and (n_chunks.dtype != torch.int32 or n_chunks.numel() != chunk_emb.shape[0]):
        raise ValueError("n_chunks must be int32 [B]")
    B, Nmax, Dm = chunk_emb.shape
    scores = torch.empty(B, Nmax, dtype=torch.float32, device=chunk_emb.device)
    sel = torch.empty(B, k, dtype=torch.int32, device=chunk_emb.device)
    cnt = torch.empty(B, dtype=torch.int32, device=chunk_emb.device)
    _check(load_library().rapid_retrieval_select(_p(chunk_emb), _p(query_emb), _p(n_chunks), B, Nmax, Dm,
                                                 float(threshold), int(k), _p(scores), _p(sel), _p(cnt),
                                                 _p(status_word), _stream_ptr(stream)))
    return scores, sel, cnt


def rapid_merge_partials(o_parts, lse_parts, out=None, out_f32=None, lse_out=None, stream=None) -> None:
    """Log-sum-exp combination of P partial attention results: o_parts [P, ..., D] float32 (each normalised),
    lse_parts [P, ...] float32 -> out [..., D] bfloat16 and / or out_f32, lse_out [...]."""
    if o_parts.dtype != torch.float32 or lse_parts.dtype != torch.float32:
        raise TypeError("o_parts and lse_parts must be float32")
    if not (o_parts.is_contiguous() and lse_parts.is_contiguous()) or o_parts.shape[:-1] != lse_parts.shape:
        raise ValueError("o_parts must be dense [P, ..., D] and lse_parts dense [P, ...]")
    P, D = o_parts.shape[0], o_parts.shape[-1]
    rows = lse_parts[0].numel()
    for t, dt, n in ((out, torch.bfloat16, rows * D), (out_f32, torch.float32, rows * D), (lse_out, torch.float32, rows)):
        if t is not None and (t.dtype != dt or t.numel() != n or not t.is_contiguous()):
            raise ValueError("output tensors must be dense, of the rows' shape and of the documented dtype")
    _check(load_library().rapid_merge_partials(_p(o_parts), _p(lse_parts), P, rows, D, _p(out), _p(out_f32),
                                               _p(lse_out), _stream_ptr(stream)))


def rapid_accept(target_logits, draft_logits, draft_tokens, uniforms, eta, out_accept_len, out_next_token,
                 workspace, params: Optional[AcceptParams] = None, stream=None) -> None:
    """Algorithm 1's validation loop + residual draw on device tensors (see include/rapid.h)."""
    if target_logits.dtype != torch.float32 or draft_logits.dtype != torch.float32 or uniforms.dtype != torch.float32:
        raise TypeError("logits and uniforms must be float32")
    if draft_tokens.dtype != torch.int32 or out_accept_len.dtype != torch.int32 or out_next_token.dtype != torch.int32:
        raise TypeError("tokens and outputs must be int32")
    shape = _accept_shape(target_logits, draft_logits)
    _check(load_library().rapid_accept(_p(target_logits), _p(draft_logits), _p(draft_tokens), _p(uniforms),
                                       float(eta), _p(out_accept_len), _p(out_next_token), ctypes.byref(shape),
                                       _accept_params(params), _p(workspace), _nbytes(workspace),
                                       _stream_ptr(stream)))


def rapid_accept_static(target_logits, draft_logits, draft_tokens, uniforms, eta, out_accept_len, out_next_token,
                        params: Optional[AcceptParams] = None, out_status: Optional[torch.Tensor] = None,
                        stream=None) -> None:
    """rapid_accept for callers that cannot provide a workspace: the scratch is a fixed array inside
    the library (at most 512 logit rows, calls must not overlap on the GPU; see include/rapid.h).
    ``out_status`` is an optional int32 device tensor that receives this call's status word."""
    if target_logits.dtype != torch.float32 or draft_logits.dtype != torch.float32 or uniforms.dtype != torch.float32:
        raise TypeError("logits and uniforms must be float32")
    if draft_tokens.dtype != torch.int32 or out_accept_len.dtype != torch.int32 or out_next_token.dtype != torch.int32:
        raise TypeError("tokens and outputs must be int32")
    shape = _accept_shape(target_logits, draft_logits)
    _check(load_library().rapid_accept_static(_p(target_logits), _p(draft_logits), _p(draft_tokens), _p(uniforms),
                                              float(eta), _p(out_accept_len), _p(out_next_token),
                                              ctypes.byref(shape), _accept_params(params), _p(out_status),
                                              _stream_ptr(stream)))


def rapid_verify_step(q, k_cache, v_cache, ctx_lens, gamma, out, attn_workspace, target_logits, draft_logits,
                      draft_tokens, uniforms, eta, out_accept_len, out_next_token, accept_workspace,
                      attn_params: Optional[AttnParams] = None, accept_params: Optional[AcceptParams] = None,
                      stream=None) -> None:
    """Attention then accept on one stream, no host synchronisation."""
    ashape = _attn_shape(q, k_cache)
    cshape = _accept_shape(target_logits, draft_logits)
    _check(load_library().rapid_verify_step(
        _p(q), _p(k_cache), _p(v_cache), _p(ctx_lens), gamma, _p(out), ctypes.byref(ashape), _attn_params(attn_params),
        _p(attn_workspace), _nbytes(attn_workspace),
        _p(target_logits), _p(draft_logits), _p(draft_tokens), _p(uniforms), float(eta), _p(out_accept_len),
        _p(out_next_token), ctypes.byref(cshape), _accept_params(accept_params), _p(accept_workspace),
        _nbytes(accept_workspace), _stream_ptr(stream)))


def rapid_kv_append(k_new, v_new, k_cache, v_cache, ctx_lens, gamma, status_word, stream=None) -> None:
    """Appends k_new/v_new [B, gamma+1, Hkv, D] (bf16) at ctx_lens and adds gamma+1 to ctx_lens (in place)."""
    if k_new.dtype != torch.bfloat16 or v_new.dtype != torch.bfloat16 or ctx_lens.dtype != torch.int32:
        raise TypeError("k_new/v_new must be bfloat16 and ctx_lens int32")
    B, R, Hkv, D = k_new.shape
    if R != gamma + 1 or not (k_new.is_contiguous() and v_new.is_contiguous()) or k_new.shape != v_new.shape:
        raise ValueError("k_new and v_new must be dense [B, gamma+1, Hkv, D]")
    if k_cache.stride() != v_cache.stride() or k_cache.shape != v_cache.shape or k_cache.stride(3) != 1:
        raise ValueError("k_cache and v_cache must share shape and strides with a contiguous head_dim")
    shape = _AttnShape(B, Hkv, Hkv, D, k_cache.shape[2], k_cache.stride(0), k_cache.stride(1), k_cache.stride(2))
    _check(load_library().rapid_kv_append(_p(k_new), _p(v_new), _p(k_cache), _p(v_cache), _p(ctx_lens), gamma,
                                          ctypes.byref(shape), _p(status_word), _stream_ptr(stream)))


def rapid_kv_append_paged(k_new, v_new, k_pool, v_pool, block_table, ctx_lens, gamma, status_word, stream=None) -> None:
    """rapid_kv_append into pools [num_blocks, Hkv, block_size, D] through block_table [B, max_blocks] (int32)."""
    if k_new.dtype != torch.bfloat16 or v_new.dtype != torch.bfloat16 or ctx_lens.dtype != torch.int32 \
            or block_table.dtype != torch.int32 or k_pool.dtype != torch.bfloat16 or v_pool.dtype != torch.bfloat16:
        raise TypeError("k_new/v_new and the pools must be bfloat16, ctx_lens and block_table int32")
    B, R, Hkv, D = k_new.shape
    if R != gamma + 1 or not (k_new.is_contiguous() and v_new.is_contiguous()) or k_new.shape != v_new.shape:
        raise ValueError("k_new and v_new must be dense [B, gamma+1, Hkv, D]")
    if k_pool.stride() != v_pool.stride() or k_pool.shape != v_pool.shape or k_pool.stride(3) != 1 \
            or k_pool.shape[1] != Hkv or k_pool.shape[3] != D:
        raise ValueError("k_pool and v_pool must be [num_blocks, Hkv, block_size, D] with equal strides")
    if not block_table.is_contiguous() or block_table.shape[0] != B:
        raise ValueError("block_table must be dense [B, max_blocks_per_seq]")
    paged = _PagedKv(k_pool.shape[2], k_pool.shape[0], block_table.shape[1], 0, k_pool.stride(0), k_pool.stride(1),
                     k_pool.stride(2))
    _check(load_library().rapid_kv_append_paged(_p(k_new), _p(v_new), _p(k_pool), _p(v_pool), _p(block_table),
                                                ctypes.byref(paged), _p(ctx_lens), gamma, B, Hkv, D,
                                                _p(status_word), _stream_ptr(stream)))


def rapid_step_commit(ctx_lens, accept_len, gamma, status_word, stream=None) -> None:
    """ctx_lens[b] -= gamma - accept_len[b] (in place): drops the rejected drafts' rows from the cache."""
    if ctx_lens.dtype != torch.int32 or accept_len.dtype != torch.int32:
        raise TypeError("ctx_lens and accept_len must be int32")
    _check(load_library().rapid_step_commit(_p(ctx_lens), _p(accept_len), gamma, ctx_lens.numel(),
                                            _p(status_word), _stream_ptr(stream)))


def rapid_verify_step_host(q, k_cache, v_cache, ctx_lens, gamma, out, target_logits, draft_logits, draft_tokens,
                           uniforms, eta, out_accept_len, out_next_token, device_arena,
                           attn_params: Optional[AttnParams] = None, accept_params: Optional[AcceptParams] = None,
                           stream=None) -> int:
    """The step on HOST tensors (ideally pinned): copies in, runs, copies back, synchronises. Returns the status word."""
    for t in (q, k_cache, v_cache, ctx_lens, out, target_logits, draft_logits, draft_tokens, uniforms,
              out_accept_len, out_next_token):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("rapid_verify_step_host takes dense host tensors")
    B, R, Hq, D = q.shape
    _, Hkv, Lmax, _ = k_cache.shape
    ashape = _AttnShape(B, Hq, Hkv, D, Lmax, 0, 0, 0)
    cshape = _AcceptShape(B, gamma, target_logits.shape[2], 0, 0)
    status = ctypes.c_int32(0)
    _check(load_library().rapid_verify_step_host(
        _p(q), _p(k_cache), _p(v_cache), _p(ctx_lens), gamma, _p(out), ctypes.byref(ashape), _attn_params(attn_params),
        _p(target_logits), _p(draft_logits), _p(draft_tokens), _p(uniforms), float(eta), _p(out_accept_len),
        _p(out_next_token), ctypes.byref(cshape), _accept_params(accept_params), _p(device_arena),
        _nbytes(device_arena), ctypes.byref(status), _stream_ptr(stream)))
    return int(status.value)
