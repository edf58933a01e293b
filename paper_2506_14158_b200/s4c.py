"""ctypes binding of ``libs4c.so`` -- argument marshalling only; every step runs in the library's CUDA kernels.

The functions mirror the C ABI declared in ``include/s4c.h`` (same names, same argument meaning).  Tensors are
torch CUDA tensors used purely as device buffers: the binding checks dtype / contiguity / device, passes raw
pointers and the current CUDA stream, and raises :class:`S4CError` on a non-zero return code.  There is no
CPU fallback: importing this module fails if the library has not been built, and calls fail on CPU tensors.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

from ._build import lib_path

F32, BF16 = 0, 1
SEQ_OK, SEQ_BAD_PARENT, SEQ_TOKEN_RANGE, SEQ_CAPACITY, SEQ_DEPTH, SEQ_BAD_PATH, SEQ_TIMEOUT, SEQ_NONFINITE = 0, 1, 2, 4, 8, 16, 32, 64
SEQ_BAD_PAGE = 128
STATUS_NAMES = ["OK", "ERR_NULL", "ERR_SHAPE", "ERR_DTYPE", "ERR_ALIGN", "ERR_WORKSPACE", "ERR_UNSUPPORTED", "ERR_CUDA"]

EXPORTS = ["s4c_version", "s4c_status_string", "s4c_tree_attention_workspace_bytes", "s4c_tree_attention", "s4c_tree_attention_rows",
           "s4c_tree_accept_workspace_bytes", "s4c_tree_accept", "s4c_tree_accept_noalloc", "s4c_kv_compact",
           "s4c_launch_floor", "s4c_selftest_attention_timeout", "s4c_tree_build_workspace_bytes", "s4c_tree_build",
           "s4c_tree_attention_paged", "s4c_kv_compact_paged", "s4c_tree_accept_filtered_workspace_bytes",
           "s4c_tree_accept_filtered", "s4c_lm_head_greedy_workspace_bytes", "s4c_lm_head_greedy", "s4c_tree_accept_tokens",
           "s4c_qkv_rope_workspace_bytes", "s4c_qkv_rope", "s4c_qkv_rope_at", "s4c_qkv_rope_same_tree", "s4c_lm_head_topk_workspace_bytes", "s4c_lm_head_topk",
           "s4c_tree_build_topk", "s4c_lm_head_logits_workspace_bytes", "s4c_lm_head_logits", "s4c_linear_workspace_bytes", "s4c_linear", "s4c_linear_rmsnorm", "s4c_rmsnorm", "s4c_embed_gather"]
NOALLOC_SCRATCH_BYTES = 1 << 20


class S4CError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        msg = _lib.s4c_status_string(code).decode() if _lib is not None else ""
        name = STATUS_NAMES[code] if 0 <= code < len(STATUS_NAMES) else str(code)
        super().__init__(f"{fn} returned S4C_{name}: {msg}")


def _load() -> ctypes.CDLL:
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -c 'import __graft_entry__ as g; g.build()'` "
                          "(there is no CPU fallback)")
    lib = ctypes.CDLL(path)
    vp, i32p, i, f, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.s4c_version.restype = i
    lib.s4c_status_string.restype = ctypes.c_char_p
    lib.s4c_status_string.argtypes = [i]
    lib.s4c_tree_attention_workspace_bytes.restype = sz
    lib.s4c_tree_attention_workspace_bytes.argtypes = [i, i, i, i, i, i, i]
    lib.s4c_tree_attention.restype = i
    lib.s4c_tree_attention.argtypes = [vp, vp, vp, i32p, i32p, i32p, vp, i, i, i, i, i, i, i, i, f, i32p, vp, sz, vp]
    lib.s4c_tree_attention_rows.restype = i
    lib.s4c_tree_attention_rows.argtypes = [vp, vp, vp, i32p, i32p, i32p, vp, i, i, i, i, i, i, i, i, f, i32p, vp, sz, vp]
    lib.s4c_tree_accept_workspace_bytes.restype = sz
    lib.s4c_tree_accept_workspace_bytes.argtypes = [i, i, i]
    lib.s4c_tree_accept.restype = i
    lib.s4c_tree_accept.argtypes = [vp, vp, i32p, i32p, i32p, f, vp, i, i, i, i, i32p, i32p, i32p, vp, i32p, vp, sz, vp]
    lib.s4c_tree_accept_noalloc.restype = i
    lib.s4c_tree_accept_noalloc.argtypes = [vp, vp, i32p, i32p, i32p, f, vp, i, i, i, i, i32p, i32p, i32p, vp, i32p, vp]
    lib.s4c_kv_compact.restype = i
    lib.s4c_kv_compact.argtypes = [vp, vp, i, i32p, i32p, i32p, i, vp, vp, i, i, i, i, i, i, i, i32p, vp]
    lib.s4c_selftest_attention_timeout.restype = i
    lib.s4c_selftest_attention_timeout.argtypes = [vp, vp, vp, i32p, i32p, vp, i, i, i, i, i, i, i, i, i, i32p, vp]
    lib.s4c_tree_build_workspace_bytes.restype = sz
    lib.s4c_tree_build_workspace_bytes.argtypes = [i, i, i, i]
    lib.s4c_tree_build.restype = i
    lib.s4c_tree_build.argtypes = [vp, vp, i, i32p, i32p, i, i, i, i32p, i32p, i32p, i32p, vp, sz, vp]
    lib.s4c_tree_attention_paged.restype = i
    lib.s4c_tree_attention_paged.argtypes = [vp, vp, vp, i32p, i32p, i32p, i32p, vp, i, i, i, i, i, i, i, i, i, i, f, i32p, vp, sz, vp]
    lib.s4c_kv_compact_paged.restype = i
    lib.s4c_kv_compact_paged.argtypes = [vp, vp, i, i32p, i32p, i32p, i32p, i, vp, vp, i, i, i, i, i, i, i, i, i, i32p, vp]
    lib.s4c_tree_accept_filtered_workspace_bytes.restype = sz
    lib.s4c_tree_accept_filtered_workspace_bytes.argtypes = [i, i, i, i]
    lib.s4c_tree_accept_filtered.restype = i
    lib.s4c_tree_accept_filtered.argtypes = [vp, vp, i32p, i32p, i32p, f, i, f, vp, i, i, i, i, i32p, i32p, i32p, vp, i32p, vp, sz, vp]
    lib.s4c_lm_head_greedy_workspace_bytes.restype = sz
    lib.s4c_lm_head_greedy_workspace_bytes.argtypes = [i, i, i]
    lib.s4c_lm_head_greedy.restype = i
    lib.s4c_lm_head_greedy.argtypes = [vp, vp, i, i, i, i32p, vp, i32p, vp, sz, vp]
    lib.s4c_tree_accept_tokens.restype = i
    lib.s4c_tree_accept_tokens.argtypes = [i32p, i32p, i32p, i32p, i, i, i, i, i32p, i32p, i32p, i32p, vp]
    lib.s4c_qkv_rope_workspace_bytes.restype = sz
    lib.s4c_qkv_rope_workspace_bytes.argtypes = [i, i, i]
    lib.s4c_qkv_rope.restype = i
    lib.s4c_qkv_rope.argtypes = [vp, vp, i32p, i32p, i32p, vp, vp, vp, i, i, i, i, i, i, i, f, i32p, vp, sz, vp]
    lib.s4c_qkv_rope_at.restype = i
    lib.s4c_qkv_rope_at.argtypes = [vp, vp, i32p, i32p, i32p, i32p, vp, vp, vp, i, i, i, i, i, i, i, f, i32p, vp, sz, vp]
    lib.s4c_qkv_rope_same_tree.restype = i
    lib.s4c_qkv_rope_same_tree.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, i32p, vp, sz, vp]
    lib.s4c_lm_head_topk_workspace_bytes.restype = sz
    lib.s4c_lm_head_topk_workspace_bytes.argtypes = [i, i, i, i]
    lib.s4c_lm_head_topk.restype = i
    lib.s4c_lm_head_topk.argtypes = [vp, vp, i, i, i, i, i32p, vp, i32p, vp, sz, vp]
    lib.s4c_tree_build_topk.restype = i
    lib.s4c_tree_build_topk.argtypes = [i32p, i, vp, i, i32p, i32p, i, i, i32p, i32p, i32p, i32p, vp]
    lib.s4c_lm_head_logits_workspace_bytes.restype = sz
    lib.s4c_lm_head_logits_workspace_bytes.argtypes = [i, i, i]
    lib.s4c_lm_head_logits.restype = i
    lib.s4c_lm_head_logits.argtypes = [vp, vp, i, i, i, vp, i32p, vp, sz, vp]
    lib.s4c_linear_workspace_bytes.restype = sz
    lib.s4c_linear_workspace_bytes.argtypes = [i, i, i, i, i]
    lib.s4c_linear.restype = i
    lib.s4c_linear.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, i32p, vp, sz, vp]
    lib.s4c_linear_rmsnorm.restype = i
    lib.s4c_linear_rmsnorm.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, f, vp, i32p, vp, sz, vp]
    lib.s4c_rmsnorm.restype = i
    lib.s4c_rmsnorm.argtypes = [vp, vp, f, i, i, vp, vp]
    lib.s4c_embed_gather.restype = i
    lib.s4c_embed_gather.argtypes = [vp, i32p, i, i, i, vp, vp]
    lib.s4c_launch_floor.restype = i
    lib.s4c_launch_floor.argtypes = [i, i, i, i, i, i, i, i32p, i32p, vp]
    return lib


_lib = None
_lib = _load()


def version() -> int:
    return int(_lib.s4c_version())


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}: the library takes float32 or bfloat16")


def _dev(t: Optional[torch.Tensor], dtype=None, name="tensor") -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (the library has no CPU path)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


_ws_cache = {}


def _workspace(nbytes: int, device, tag: str) -> Optional[torch.Tensor]:
    """A cached scratch buffer per (device, call family); reused by calls ordered on one stream."""
    if nbytes == 0:
        return None
    key = (str(device), tag)
    buf = _ws_cache.get(key)
    if buf is None or buf.numel() < nbytes:
        buf = torch.empty(nbytes, dtype=torch.uint8, device=device)
        _ws_cache[key] = buf
    return buf


def tree_attention_workspace_bytes(B, T, Hq, Hkv, d, C, dtype) -> int:
    dt = F32 if dtype == torch.float32 else BF16
    return int(_lib.s4c_tree_attention_workspace_bytes(B, T, Hq, Hkv, d, C, dt))


def tree_attention(q, k_cache, v_cache, cache_len, parent, n_nodes=None, out=None, scale: float = 0.0, status=None,
                   workspace=None, stream=None, max_cache_len: int = 0, rows: bool = False):
    """s4c_tree_attention: q [B,Hq,T,d], k_cache/v_cache [B,Hkv,C,d] -> out [B,Hq,T,d] (same dtype).

    ``max_cache_len``: the host's upper bound on ``cache_len`` (0 = unknown); it shapes the launch, never the result.
    ``rows``: s4c_tree_attention_rows -- out is [B,T,Hq,d], the rows the output projection reads (bf16 only)."""
    B, Hq, T, d = q.shape
    _, Hkv, C, _ = k_cache.shape
    if k_cache.shape != (B, Hkv, C, d) or v_cache.shape != (B, Hkv, C, d):
        raise ValueError("k_cache / v_cache must be [B,Hkv,C,d]")
    if k_cache.dtype != q.dtype or v_cache.dtype != q.dtype:
        raise TypeError("q, k_cache and v_cache must share one dtype")
    if out is None:
        out = torch.empty(B, T, Hq, d, dtype=q.dtype, device=q.device) if rows else torch.empty_like(q)
    dt = _dt(q)
    need = int(_lib.s4c_tree_attention_workspace_bytes(B, T, Hq, Hkv, d, C, dt))
    if workspace is None:
        workspace = _workspace(need, q.device, "attn")
    rc = (_lib.s4c_tree_attention_rows if rows else _lib.s4c_tree_attention)(
        _dev(q, name="q"), _dev(k_cache, name="k_cache"), _dev(v_cache, name="v_cache"),
        _dev(cache_len, torch.int32, "cache_len"), _dev(parent, torch.int32, "parent"),
        _dev(n_nodes, torch.int32, "n_nodes"), _dev(out, q.dtype, "out"), B, T, Hq, Hkv, d, C, int(max_cache_len), dt,
        float(scale),
        _dev(status, torch.int32, "status"), _dev(workspace, name="workspace"),
        0 if workspace is None else workspace.numel() * workspace.element_size(), _stream(stream))
    if rc:
        raise S4CError("s4c_tree_attention_rows" if rows else "s4c_tree_attention", rc)
    return out


def tree_accept_workspace_bytes(B, T, V) -> int:
    return int(_lib.s4c_tree_accept_workspace_bytes(B, T, V))


def tree_accept(target_logits, draft_probs, tokens, parent, temperature: float, uniforms=None, n_nodes=None,
                max_depth: Optional[int] = None, accept_len=None, path=None, next_token=None, near_tie=None,
                status=None, workspace=None, stream=None):
    """s4c_tree_accept: returns dict(accept_len [B], path [B,max_depth+1], next_token [B], near_tie [B,T], status [B])."""
    B, T, V = target_logits.shape
    dev = target_logits.device
    if max_depth is None:
        max_depth = T - 1
    i32 = dict(dtype=torch.int32, device=dev)
    accept_len = torch.empty(B, **i32) if accept_len is None else accept_len
    path = torch.empty(B, max_depth + 1, **i32) if path is None else path
    next_token = torch.empty(B, **i32) if next_token is None else next_token
    near_tie = torch.empty(B, T, dtype=torch.uint8, device=dev) if near_tie is None else near_tie
    status = torch.empty(B, **i32) if status is None else status
    need = int(_lib.s4c_tree_accept_workspace_bytes(B, T, V))
    if workspace is None:
        workspace = _workspace(need, dev, "accept")
    rc = _lib.s4c_tree_accept(
        _dev(target_logits, torch.float32, "target_logits"), _dev(draft_probs, torch.float32, "draft_probs"),
        _dev(tokens, torch.int32, "tokens"), _dev(parent, torch.int32, "parent"), _dev(n_nodes, torch.int32, "n_nodes"),
        float(temperature), _dev(uniforms, torch.float32, "uniforms"), B, T, V, int(max_depth),
        _dev(accept_len, torch.int32, "accept_len"), _dev(path, torch.int32, "path"),
        _dev(next_token, torch.int32, "next_token"), _dev(near_tie, torch.uint8, "near_tie"),
        _dev(status, torch.int32, "status"), _dev(workspace, name="workspace"),
        0 if workspace is None else workspace.numel() * workspace.element_size(), _stream(stream))
    if rc:
        raise S4CError("s4c_tree_accept", rc)
    return dict(accept_len=accept_len, path=path, next_token=next_token, near_tie=near_tie, status=status)


def tree_accept_noalloc(target_logits, draft_probs, tokens, parent, temperature: float, uniforms=None, n_nodes=None,
                        max_depth: Optional[int] = None, out: Optional[dict] = None, stream=None):
    """s4c_tree_accept_noalloc: the acceptance step for callers that cannot allocate device memory.

    Same inputs and results as :func:`tree_accept`, but the library's built-in scratch array is used instead of a
    workspace, so the C call allocates nothing.  This wrapper allocates nothing either when ``out`` (a dict holding
    the five output tensors ``accept_len, path, next_token, near_tie, status``) is passed; it creates them only as a
    convenience when ``out`` is None.  Problems whose scratch need exceeds ``NOALLOC_SCRATCH_BYTES`` raise
    :class:`S4CError` (ERR_WORKSPACE).  Calls share the one array: keep them ordered on a stream.
    """
    B, T, V = target_logits.shape
    dev = target_logits.device
    if max_depth is None:
        max_depth = T - 1
    if out is None:
        i32 = dict(dtype=torch.int32, device=dev)
        out = dict(accept_len=torch.empty(B, **i32), path=torch.empty(B, max_depth + 1, **i32),
                   next_token=torch.empty(B, **i32), near_tie=torch.empty(B, T, dtype=torch.uint8, device=dev),
                   status=torch.empty(B, **i32))
    rc = _lib.s4c_tree_accept_noalloc(
        _dev(target_logits, torch.float32, "target_logits"), _dev(draft_probs, torch.float32, "draft_probs"),
        _dev(tokens, torch.int32, "tokens"), _dev(parent, torch.int32, "parent"), _dev(n_nodes, torch.int32, "n_nodes"),
        float(temperature), _dev(uniforms, torch.float32, "uniforms"), B, T, V, int(max_depth),
        _dev(out["accept_len"], torch.int32, "accept_len"), _dev(out["path"], torch.int32, "path"),
        _dev(out["next_token"], torch.int32, "next_token"), _dev(out["near_tie"], torch.uint8, "near_tie"),
        _dev(out["status"], torch.int32, "status"), _stream(stream))
    if rc:
        raise S4CError("s4c_tree_accept_noalloc", rc)
    return out


def cache_pointer_array(caches: Sequence[torch.Tensor]) -> torch.Tensor:
    """Device array of the layers' cache base pointers (int64), as s4c_kv_compact expects."""
    if not caches:
        return torch.zeros(1, dtype=torch.int64, device="cuda")
    for c in caches:
        _dev(c, caches[0].dtype, "cache")
        if c.shape != caches[0].shape:
            raise ValueError("all layer caches must share one shape")
    return torch.tensor([c.data_ptr() for c in caches], dtype=torch.int64, device=caches[0].device)


def kv_compact(k_ptrs, v_ptrs, n_layers: int, cache_shape, dtype, cache_len, path, accept_len, T: int,
               feat_in=None, feat_out=None, status=None, stream=None):
    """s4c_kv_compact.  k_ptrs / v_ptrs: device int64 arrays from :func:`cache_pointer_array`;
    cache_shape = (B,Hkv,C,d); cache_len is updated in place.  Returns status [B]."""
    B, Hkv, C, d = cache_shape
    max_depth = path.shape[1] - 1
    dt = F32 if dtype == torch.float32 else BF16
    if status is None:
        status = torch.empty(B, dtype=torch.int32, device=cache_len.device)
    hid = 0
    if feat_in is not None:
        if feat_in.dtype != dtype or feat_out is None or feat_out.dtype != dtype:
            raise TypeError("features must have the cache dtype")
        if feat_in.shape[:2] != (B, T) or feat_out.shape != (B, max_depth + 1, feat_in.shape[2]):
            raise ValueError("feat_in must be [B,T,hid] and feat_out [B,max_depth+1,hid]")
        hid = feat_in.shape[2]
    rc = _lib.s4c_kv_compact(
        _dev(k_ptrs, torch.int64, "k_ptrs") if n_layers else None, _dev(v_ptrs, torch.int64, "v_ptrs") if n_layers else None,
        int(n_layers), _dev(cache_len, torch.int32, "cache_len"), _dev(path, torch.int32, "path"),
        _dev(accept_len, torch.int32, "accept_len"), max_depth, _dev(feat_in, name="feat_in"),
        _dev(feat_out, name="feat_out"), B, T, Hkv, d, C, hid, dt, _dev(status, torch.int32, "status"), _stream(stream))
    if rc:
        raise S4CError("s4c_kv_compact", rc)
    return status


def launch_floor(ctas: int, cluster: int, threads: int, smem_bytes: int, tmem_cols: int, cluster_syncs: int,
                 dependent_launch: bool, word: Optional[torch.Tensor] = None, stream=None):
    """s4c_launch_floor: enqueue one empty kernel with the given launch shape (a measurement aid)."""
    rc = _lib.s4c_launch_floor(int(ctas), int(cluster), int(threads), int(smem_bytes), int(tmem_cols), int(cluster_syncs),
                               1 if dependent_launch else 0, _dev(word, torch.int32, "word"), None, _stream(stream))
    if rc:
        raise S4CError("s4c_launch_floor", rc)


def selftest_attention_timeout(q, k_cache, v_cache, cache_len, parent, out, status, withhold_tile: int, limit_us: int,
                               max_cache_len: int = 0, stream=None):
    """s4c_selftest_attention_timeout: the attention launch with one cache tile per CTA withheld and a short wait limit."""
    B, Hq, T, d = q.shape
    _, Hkv, C, _ = k_cache.shape
    rc = _lib.s4c_selftest_attention_timeout(
        _dev(q, torch.bfloat16, "q"), _dev(k_cache, torch.bfloat16, "k_cache"), _dev(v_cache, torch.bfloat16, "v_cache"),
        _dev(cache_len, torch.int32, "cache_len"), _dev(parent, torch.int32, "parent"), _dev(out, torch.bfloat16, "out"),
        B, T, Hq, Hkv, d, C, int(max_cache_len), int(withhold_tile), int(limit_us), _dev(status, torch.int32, "status"),
        _stream(stream))
    if rc:
        raise S4CError("s4c_selftest_attention_timeout", rc)


def tree_build_workspace_bytes(B, T, V, max_branch) -> int:
    return int(_lib.s4c_tree_build_workspace_bytes(B, T, V, max_branch))


def tree_build(draft_probs, branching: Sequence[int], root_token, cache_len=None, tokens=None, parent=None, position=None,
               n_nodes=None, workspace=None, stream=None):
    """s4c_tree_build: draft_probs [B,T,V] f32, branching (host ints), root_token [B] ->
    dict(tokens, parent, position [B,T], n_nodes [B]), all int32 on the device."""
    B, T, V = draft_probs.shape
    dev = draft_probs.device
    i32 = dict(dtype=torch.int32, device=dev)
    tokens = torch.empty(B, T, **i32) if tokens is None else tokens
    parent = torch.empty(B, T, **i32) if parent is None else parent
    position = torch.empty(B, T, **i32) if position is None else position
    n_nodes = torch.empty(B, **i32) if n_nodes is None else n_nodes
    br = (ctypes.c_int32 * max(1, len(branching)))(*[int(x) for x in branching])
    need = int(_lib.s4c_tree_build_workspace_bytes(B, T, V, max([1] + [int(x) for x in branching])))
    if workspace is None:
        workspace = _workspace(need, dev, "tree")
    rc = _lib.s4c_tree_build(
        _dev(draft_probs, torch.float32, "draft_probs"), ctypes.cast(br, ctypes.c_void_p), len(branching),
        _dev(root_token, torch.int32, "root_token"), _dev(cache_len, torch.int32, "cache_len"), B, T, V,
        _dev(tokens, torch.int32, "tokens"), _dev(parent, torch.int32, "parent"), _dev(position, torch.int32, "position"),
        _dev(n_nodes, torch.int32, "n_nodes"), _dev(workspace, name="workspace"),
        0 if workspace is None else workspace.numel() * workspace.element_size(), _stream(stream))
    if rc:
        raise S4CError("s4c_tree_build", rc)
    return dict(tokens=tokens, parent=parent, position=position, n_nodes=n_nodes)


def tree_attention_paged(q, k_pages, v_pages, block_table, cache_len, parent, n_nodes=None, out=None, scale: float = 0.0,
                         status=None, workspace=None, stream=None, max_cache_len: int = 0):
    """s4c_tree_attention_paged: q [B,Hq,T,d], k_pages / v_pages [n_pages,Hkv,page_size,d], block_table [B,max_blocks]."""
    B, Hq, T, d = q.shape
    n_pages, Hkv, page_size, _ = k_pages.shape
    max_blocks = block_table.shape[1]
    if v_pages.shape != k_pages.shape or k_pages.shape[3] != d or block_table.shape[0] != B:
        raise ValueError("k_pages / v_pages must be [n_pages,Hkv,page_size,d] and block_table [B,max_blocks]")
    if out is None:
        out = torch.empty_like(q)
    dt = _dt(q)
    need = int(_lib.s4c_tree_attention_workspace_bytes(B, T, Hq, Hkv, d, max_blocks * page_size, dt))
    if workspace is None:
        workspace = _workspace(need, q.device, "attn")
    rc = _lib.s4c_tree_attention_paged(
        _dev(q, name="q"), _dev(k_pages, q.dtype, "k_pages"), _dev(v_pages, q.dtype, "v_pages"),
        _dev(block_table, torch.int32, "block_table"), _dev(cache_len, torch.int32, "cache_len"),
        _dev(parent, torch.int32, "parent"), _dev(n_nodes, torch.int32, "n_nodes"), _dev(out, q.dtype, "out"), B, T, Hq, Hkv, d,
        n_pages, page_size, max_blocks, int(max_cache_len), dt, float(scale), _dev(status, torch.int32, "status"),
        _dev(workspace, name="workspace"), 0 if workspace is None else workspace.numel() * workspace.element_size(),
        _stream(stream))
    if rc:
        raise S4CError("s4c_tree_attention_paged", rc)
    return out


def kv_compact_paged(k_ptrs, v_ptrs, n_layers: int, pool_shape, dtype, block_table, cache_len, path, accept_len, T: int,
                     feat_in=None, feat_out=None, status=None, stream=None):
    """s4c_kv_compact_paged.  pool_shape = (n_pages,Hkv,page_size,d); k_ptrs / v_ptrs from :func:`cache_pointer_array`."""
    n_pages, Hkv, page_size, d = pool_shape
    B, max_blocks = block_table.shape
    max_depth = path.shape[1] - 1
    dt = F32 if dtype == torch.float32 else BF16
    if status is None:
        status = torch.empty(B, dtype=torch.int32, device=cache_len.device)
    hid = 0 if feat_in is None else feat_in.shape[2]
    rc = _lib.s4c_kv_compact_paged(
        _dev(k_ptrs, torch.int64, "k_ptrs") if n_layers else None, _dev(v_ptrs, torch.int64, "v_ptrs") if n_layers else None,
        int(n_layers), _dev(block_table, torch.int32, "block_table"), _dev(cache_len, torch.int32, "cache_len"),
        _dev(path, torch.int32, "path"), _dev(accept_len, torch.int32, "accept_len"), max_depth, _dev(feat_in, name="feat_in"),
        _dev(feat_out, name="feat_out"), B, T, Hkv, d, n_pages, page_size, max_blocks, hid, dt,
        _dev(status, torch.int32, "status"), _stream(stream))
    if rc:
        raise S4CError("s4c_kv_compact_paged", rc)
    return status


def tree_accept_filtered_workspace_bytes(B, T, V, top_k) -> int:
    return int(_lib.s4c_tree_accept_filtered_workspace_bytes(B, T, V, top_k))


def tree_accept_filtered(target_logits, draft_probs, tokens, parent, temperature: float, top_k: int, top_p: float, uniforms,
                         n_nodes=None, max_depth: Optional[int] = None, accept_len=None, path=None, next_token=None,
                         near_tie=None, status=None, workspace=None, stream=None):
    """s4c_tree_accept_filtered: the walk of :func:`tree_accept` against the top-k / nucleus filtered target distribution."""
    B, T, V = target_logits.shape
    dev = target_logits.device
    if max_depth is None:
        max_depth = T - 1
    i32 = dict(dtype=torch.int32, device=dev)
    accept_len = torch.empty(B, **i32) if accept_len is None else accept_len
    path = torch.empty(B, max_depth + 1, **i32) if path is None else path
    next_token = torch.empty(B, **i32) if next_token is None else next_token
    near_tie = torch.empty(B, T, dtype=torch.uint8, device=dev) if near_tie is None else near_tie
    status = torch.empty(B, **i32) if status is None else status
    need = int(_lib.s4c_tree_accept_filtered_workspace_bytes(B, T, V, int(top_k)))
    if workspace is None:
        workspace = _workspace(need, dev, "accept_filtered")
    rc = _lib.s4c_tree_accept_filtered(
        _dev(target_logits, torch.float32, "target_logits"), _dev(draft_probs, torch.float32, "draft_probs"),
        _dev(tokens, torch.int32, "tokens"), _dev(parent, torch.int32, "parent"), _dev(n_nodes, torch.int32, "n_nodes"),
        float(temperature), int(top_k), float(top_p), _dev(uniforms, torch.float32, "uniforms"), B, T, V, int(max_depth),
        _dev(accept_len, torch.int32, "accept_len"), _dev(path, torch.int32, "path"),
        _dev(next_token, torch.int32, "next_token"), _dev(near_tie, torch.uint8, "near_tie"),
        _dev(status, torch.int32, "status"), _dev(workspace, name="workspace"),
        0 if workspace is None else workspace.numel() * workspace.element_size(), _stream(stream))
    if rc:
        raise S4CError("s4c_tree_accept_filtered", rc)
    return dict(accept_len=accept_len, path=path, next_token=next_token, near_tie=near_tie, status=status)


def lm_head_greedy_workspace_bytes(R, V, H) -> int:
    return int(_lib.s4c_lm_head_greedy_workspace_bytes(R, V, H))


def lm_head_greedy(hidden, weight, token=None, max_logit=None, status=None, workspace=None, stream=None):
    """s4c_lm_head_greedy: token[r] = argmax_v sum_h hidden[r,h] * weight[v,h] (bf16 in, f32 accumulation), no logits in memory."""
    R, H = hidden.shape
    V = weight.shape[0]
    dev = hidden.device
    token = torch.empty(R, dtype=torch.int32, device=dev) if token is None else token
    max_logit = torch.empty(R, dtype=torch.float32, device=dev) if max_logit is None else max_logit
    status = torch.zeros(1, dtype=torch.int32, device=dev) if status is None else status
    if workspace is None:
        workspace = _workspace(int(_lib.s4c_lm_head_greedy_workspace_bytes(R, V, H)), dev, "lm_head")
    rc = _lib.s4c_lm_head_greedy(_dev(hidden, torch.bfloat16, "hidden"), _dev(weight, torch.bfloat16, "weight"), R, V, H,
                                 _dev(token, torch.int32, "token"), _dev(max_logit, torch.float32, "max_logit"),
                                 _dev(status, torch.int32, "status"), _dev(workspace, name="workspace"),
                                 workspace.numel() * workspace.element_size(), _stream(stream))
    if rc:
        raise S4CError("s4c_lm_head_greedy", rc)
    return dict(token=token, max_logit=max_logit, status=status)


def lm_head_logits_workspace_bytes(R, V, H) -> int:
    return int(_lib.s4c_lm_head_logits_workspace_bytes(R, V, H))


def lm_head_logits(hidden, weight, logits=None, status=None, workspace=None, stream=None):
    """s4c_lm_head_logits: logits [R,V] float32 = hidden @ weight^T (bf16 in, f32 sums), for stochastic verification."""
    R, H = hidden.shape
    V = weight.shape[0]
    logits = torch.empty(R, V, dtype=torch.float32, device=hidden.device) if logits is None else logits
    if workspace is None:
        workspace = _workspace(int(_lib.s4c_lm_head_logits_workspace_bytes(R, V, H)), hidden.device, "linear")
    rc = _lib.s4c_lm_head_logits(_dev(hidden, torch.bfloat16, "hidden"), _dev(weight, torch.bfloat16, "weight"), R, V, H,
                                 _dev(logits, torch.float32, "logits"), _dev(status, torch.int32, "status"),
                                 _dev(workspace, name="workspace"), 0 if workspace is None else workspace.numel() * workspace.element_size(),
                                 _stream(stream))
    if rc:
        raise S4CError("s4c_lm_head_logits", rc)
    return logits


def tree_accept_tokens(target_token, tokens, parent, V: int, n_nodes=None, max_depth: Optional[int] = None, accept_len=None,
                       path=None, next_token=None, status=None, stream=None):
    """s4c_tree_accept_tokens: greedy verification from the target's choice per node (target_token [B,T] int32)."""
    B, T = target_token.shape
    dev = target_token.device
    if max_depth is None:
        max_depth = T - 1
    i32 = dict(dtype=torch.int32, device=dev)
    accept_len = torch.empty(B, **i32) if accept_len is None else accept_len
    path = torch.empty(B, max_depth + 1, **i32) if path is None else path
    next_token = torch.empty(B, **i32) if next_token is None else next_token
    status = torch.empty(B, **i32) if status is None else status
    rc = _lib.s4c_tree_accept_tokens(_dev(target_token, torch.int32, "target_token"), _dev(tokens, torch.int32, "tokens"),
                                     _dev(parent, torch.int32, "parent"), _dev(n_nodes, torch.int32, "n_nodes"), B, T, int(V),
                                     int(max_depth), _dev(accept_len, torch.int32, "accept_len"), _dev(path, torch.int32, "path"),
                                     _dev(next_token, torch.int32, "next_token"), _dev(status, torch.int32, "status"),
                                     _stream(stream))
    if rc:
        raise S4CError("s4c_tree_accept_tokens", rc)
    return dict(accept_len=accept_len, path=path, next_token=next_token, status=status)


def qkv_rope_workspace_bytes(B, T, d) -> int:
    return int(_lib.s4c_qkv_rope_workspace_bytes(B, T, d))


def qkv_rope(x, w_qkv, cache_len, parent, q_out, k_cache, v_cache, n_nodes=None, rope_theta: float = 10000.0, status=None,
             workspace=None, stream=None, position_base=None):
    """s4c_qkv_rope: q/k/v projections of the tree tokens, rotary embedding at position cache_len + depth, q into
    ``q_out`` [B,Hq,T,d], k and v into the caches' tree slots (``k_cache``, ``v_cache`` [B,Hkv,C,d], written in place)."""
    B, T, H = x.shape
    _, Hq, _, d = q_out.shape
    _, Hkv, C, _ = k_cache.shape
    dev = x.device
    status = torch.empty(B, dtype=torch.int32, device=dev) if status is None else status
    if workspace is None:
        workspace = _workspace(int(_lib.s4c_qkv_rope_workspace_bytes(B, T, d)), dev, "qkv_rope")
    bf = torch.bfloat16
    tail = (_dev(q_out, bf, "q_out"), _dev(k_cache, bf, "k_cache"), _dev(v_cache, bf, "v_cache"), B, T, H, Hq, Hkv, d, C, float(rope_theta),
            _dev(status, torch.int32, "status"), _dev(workspace, name="workspace"), workspace.numel() * workspace.element_size(),
            _stream(stream))
    if position_base is None:
        rc = _lib.s4c_qkv_rope(_dev(x, bf, "x"), _dev(w_qkv, bf, "w_qkv"), _dev(cache_len, torch.int32, "cache_len"),
                               _dev(parent, torch.int32, "parent"), _dev(n_nodes, torch.int32, "n_nodes"), *tail)
    else:  # s4c_qkv_rope_at: positions count from position_base[b], slots from cache_len[b]
        rc = _lib.s4c_qkv_rope_at(_dev(x, bf, "x"), _dev(w_qkv, bf, "w_qkv"), _dev(cache_len, torch.int32, "cache_len"),
                                  _dev(position_base, torch.int32, "position_base"), _dev(parent, torch.int32, "parent"),
                                  _dev(n_nodes, torch.int32, "n_nodes"), *tail)
    if rc:
        raise S4CError("s4c_qkv_rope_at" if position_base is not None else "s4c_qkv_rope", rc)
    return dict(q=q_out, status=status)


def qkv_rope_same_tree(x, w_qkv, q_out, k_cache, v_cache, workspace, status=None, stream=None):
    """s4c_qkv_rope_same_tree: another layer's projections with the tree checks, positions and rotary table that the
    preceding :func:`qkv_rope` call left in ``workspace`` (``status``: that call's, kept and OR-ed with timeouts)."""
    B, T, H = x.shape
    _, Hq, _, d = q_out.shape
    _, Hkv, C, _ = k_cache.shape
    bf = torch.bfloat16
    rc = _lib.s4c_qkv_rope_same_tree(_dev(x, bf, "x"), _dev(w_qkv, bf, "w_qkv"), _dev(q_out, bf, "q_out"), _dev(k_cache, bf, "k_cache"),
                                     _dev(v_cache, bf, "v_cache"), B, T, H, Hq, Hkv, d, C, _dev(status, torch.int32, "status"),
                                     _dev(workspace, name="workspace"), workspace.numel() * workspace.element_size(),
                                     _stream(stream))
    if rc:
        raise S4CError("s4c_qkv_rope_same_tree", rc)
    return dict(q=q_out, status=status)


def lm_head_topk_workspace_bytes(R, V, H, k) -> int:
    return int(_lib.s4c_lm_head_topk_workspace_bytes(R, V, H, k))


def lm_head_topk(hidden, weight, k: int, token=None, logit=None, status=None, workspace=None, stream=None):
    """s4c_lm_head_topk: the k best tokens per row of hidden @ weight^T, best first (ties to the lower token)."""
    R, H = hidden.shape
    V = weight.shape[0]
    dev = hidden.device
    token = torch.empty(R, k, dtype=torch.int32, device=dev) if token is None else token
    logit = torch.empty(R, k, dtype=torch.float32, device=dev) if logit is None else logit
    status = torch.zeros(1, dtype=torch.int32, device=dev) if status is None else status
    if workspace is None:
        workspace = _workspace(int(_lib.s4c_lm_head_topk_workspace_bytes(R, V, H, int(k))), dev, "lm_head")
    rc = _lib.s4c_lm_head_topk(_dev(hidden, torch.bfloat16, "hidden"), _dev(weight, torch.bfloat16, "weight"), R, V, H, int(k),
                               _dev(token, torch.int32, "token"), _dev(logit, torch.float32, "logit"),
                               _dev(status, torch.int32, "status"), _dev(workspace, name="workspace"),
                               0 if workspace is None else workspace.numel() * workspace.element_size(), _stream(stream))
    if rc:
        raise S4CError("s4c_lm_head_topk", rc)
    return dict(token=token, logit=logit, status=status)


def tree_build_topk(topk, branching, root_token, cache_len=None, tokens=None, parent=None, position=None, n_nodes=None,
                    stream=None):
    """s4c_tree_build_topk: the verification tree from ranked choices topk [B,T,k] int32 (child j of node n = topk[b,n,j])."""
    B, T, k = topk.shape
    dev = topk.device
    i32 = dict(dtype=torch.int32, device=dev)
    tokens = torch.empty(B, T, **i32) if tokens is None else tokens
    parent = torch.empty(B, T, **i32) if parent is None else parent
    position = torch.empty(B, T, **i32) if position is None else position
    n_nodes = torch.empty(B, **i32) if n_nodes is None else n_nodes
    br = (ctypes.c_int32 * max(1, len(branching)))(*[int(x) for x in branching])
    rc = _lib.s4c_tree_build_topk(_dev(topk, torch.int32, "topk"), k, ctypes.cast(br, ctypes.c_void_p), len(branching),
                                  _dev(root_token, torch.int32, "root_token"), _dev(cache_len, torch.int32, "cache_len"), B, T,
                                  _dev(tokens, torch.int32, "tokens"), _dev(parent, torch.int32, "parent"),
                                  _dev(position, torch.int32, "position"), _dev(n_nodes, torch.int32, "n_nodes"), _stream(stream))
    if rc:
        raise S4CError("s4c_tree_build_topk", rc)
    return dict(tokens=tokens, parent=parent, position=position, n_nodes=n_nodes)


def linear_workspace_bytes(R, K1, K2, N, gate: bool = False) -> int:
    return int(_lib.s4c_linear_workspace_bytes(R, K1, K2, N, 1 if gate else 0))


def linear(x1, w, x2=None, bias=None, residual=None, gate: bool = False, out=None, status=None, workspace=None, stream=None):
    """s4c_linear: out = concat[x1, x2] @ w^T (+ bias) (gate: silu(gate rows) * up rows) (+ residual); bf16, f32 accumulation."""
    R, K1 = x1.shape
    K2 = 0 if x2 is None else x2.shape[1]
    N = w.shape[0] // 2 if gate else w.shape[0]
    bf = torch.bfloat16
    out = torch.empty(R, N, dtype=bf, device=x1.device) if out is None else out
    if workspace is None:
        workspace = _workspace(int(_lib.s4c_linear_workspace_bytes(R, K1, K2, N, 1 if gate else 0)), x1.device, "linear")
    rc = _lib.s4c_linear(_dev(x1, bf, "x1"), _dev(x2, bf, "x2"), _dev(w, bf, "w"), _dev(bias, bf, "bias"),
                         _dev(residual, bf, "residual"), _dev(out, bf, "out"), R, K1, K2, N, 1 if gate else 0,
                         _dev(status, torch.int32, "status"), _dev(workspace, name="workspace"),
                         0 if workspace is None else workspace.numel() * workspace.element_size(), _stream(stream))
    if rc:
        raise S4CError("s4c_linear", rc)
    return out


def linear_rmsnorm(x1, w, norm_weight, eps: float = 1e-6, x2=None, bias=None, residual=None, out=None, norm_out=None, status=None,
                   workspace=None, stream=None):
    """s4c_linear_rmsnorm: out as s4c_linear (ungated), norm_out = rmsnorm(out) with norm_weight; returns (out, norm_out)."""
    R, K1 = x1.shape
    K2 = 0 if x2 is None else x2.shape[1]
    N = w.shape[0]
    bf = torch.bfloat16
    out = torch.empty(R, N, dtype=bf, device=x1.device) if out is None else out
    norm_out = torch.empty(R, N, dtype=bf, device=x1.device) if norm_out is None else norm_out
    if workspace is None:
        workspace = _workspace(int(_lib.s4c_linear_workspace_bytes(R, K1, K2, N, 0)), x1.device, "linear")
    rc = _lib.s4c_linear_rmsnorm(_dev(x1, bf, "x1"), _dev(x2, bf, "x2"), _dev(w, bf, "w"), _dev(bias, bf, "bias"),
                                 _dev(residual, bf, "residual"), _dev(out, bf, "out"), R, K1, K2, N,
                                 _dev(norm_weight, bf, "norm_weight"), float(eps), _dev(norm_out, bf, "norm_out"),
                                 _dev(status, torch.int32, "status"), _dev(workspace, name="workspace"),
                                 0 if workspace is None else workspace.numel() * workspace.element_size(), _stream(stream))
    if rc:
        raise S4CError("s4c_linear_rmsnorm", rc)
    return out, norm_out


def rmsnorm(x, weight, eps: float = 1e-6, out=None, stream=None):
    """s4c_rmsnorm: x / sqrt(mean(x^2) + eps) * weight per row (bf16)."""
    R, H = x.shape
    out = torch.empty_like(x) if out is None else out
    rc = _lib.s4c_rmsnorm(_dev(x, torch.bfloat16, "x"), _dev(weight, torch.bfloat16, "weight"), float(eps), R, H,
                          _dev(out, torch.bfloat16, "out"), _stream(stream))
    if rc:
        raise S4CError("s4c_rmsnorm", rc)
    return out


def embed_gather(table, tokens, out=None, stream=None):
    """s4c_embed_gather: rows table[tokens] (bf16 table [V,H], int32 tokens [R])."""
    V, H = table.shape
    R = tokens.numel()
    out = torch.empty(R, H, dtype=table.dtype, device=table.device) if out is None else out
    rc = _lib.s4c_embed_gather(_dev(table, torch.bfloat16, "table"), _dev(tokens, torch.int32, "tokens"), R, V, H,
                               _dev(out, torch.bfloat16, "out"), _stream(stream))
    if rc:
        raise S4CError("s4c_embed_gather", rc)
    return out
