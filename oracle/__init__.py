"""Float64 CPU oracle for the S4C verify step (arXiv 2506.14158) -- TEST INFRASTRUCTURE ONLY.

This package wraps ``s4c_oracle.c`` (plain C, float64) with ctypes and numpy.  It is the
checker the CUDA library is compared against: it shares no code with the CUDA path and
does not import it.  Only the tests, the smoke check and the benchmark's CPU-baseline /
reference legs may import it; the product path never does.

Functions (array layouts are row-major numpy arrays):

* :func:`tree_attention`      -- Section 3.2 / Figure 3 tree mask: masked softmax attention by definition.
* :func:`accept_greedy`       -- Section 4.1.2 greedy decoding + Section 3.2 longest accepted path.
* :func:`accept_stochastic`   -- Section 2 speculative sampling, Eq. 11 / Eq. 12, step by step.
* :func:`accept_filtered`     -- the same against a top-k / nucleus filtered target (sampling regime of Section 4, RQ5).
* :func:`kv_compact`          -- Section 3.2 last paragraph: keep accepted tokens' K/V and features.
* :func:`build_tree`          -- Section 3.2 / Figure 3: the continuous verification tree (vertical top-1 chain, then
                                 horizontal top-k alternatives), breadth-first numbered.
* :func:`lm_head_greedy`      -- Eq. 6 / Section 3.2: the LM head over the tree nodes' hidden states and the greedy choice
                                 (numpy, float64; a library matrix product is the step).
* :func:`accept_greedy_tokens` -- the greedy walk when the target's choice per node is already known (plain Python).
* :func:`qkv_rope`, :func:`rope_rotate` -- the verify layer's input side: q/k/v projections of the tree tokens, rotary
                                 embedding at position cache_len + depth, k/v written into the caches' tree slots (numpy).
* :func:`linear`, :func:`rmsnorm`, :func:`embed_gather` -- Eq. 3 / Eq. 6 and the decoder layer's other pieces (numpy).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "s4c_oracle.c")
_LIB = os.path.join(_HERE, "libs4c_oracle.so")
_lock = threading.Lock()
_lib = None

SEQ_OK = 0
SEQ_BAD_PARENT = 1
SEQ_TOKEN_RANGE = 2
SEQ_CAPACITY = 4
SEQ_DEPTH = 8
SEQ_BAD_PATH = 16
SEQ_NONFINITE = 64


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP on the outer loops only) and return the library path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.s4c_oracle_max_threads.restype = ctypes.c_int
        lib.s4c_oracle_set_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().s4c_oracle_max_threads())


def set_threads(n: int) -> None:
    _load().s4c_oracle_set_threads(int(n))


def _ptr(a, ctype):
    if a is None:
        return None
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def tree_attention(q, k, v, cache_len, parent, n_nodes=None, scale=0.0):
    """q [B,Hq,T,d]; k, v [B,Hkv,C,d] (tree K/V at slots L_b..L_b+T-1); returns (out f64, status[B])."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = np.ascontiguousarray(k, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    B, Hq, T, d = q.shape
    _, Hkv, C, _ = k.shape
    assert k.shape == v.shape == (B, Hkv, C, d)
    cache_len = _i32(cache_len)
    parent = _i32(parent).reshape(B, T)
    n_nodes = _i32(n_nodes)
    out = np.full(q.shape, np.nan, dtype=np.float64)
    status = np.zeros(B, dtype=np.int32)
    dbl, i32 = ctypes.c_double, ctypes.c_int32
    rc = _load().s4c_oracle_tree_attention(
        _ptr(q, dbl), _ptr(k, dbl), _ptr(v, dbl), _ptr(cache_len, i32), _ptr(parent, i32),
        _ptr(n_nodes, i32), _ptr(out, dbl), _ptr(status, i32),
        B, T, Hq, Hkv, d, C, ctypes.c_double(scale))
    if rc:
        raise ValueError(f"oracle tree_attention rejected its arguments (code {rc})")
    return out, status


def _accept_outputs(B, max_depth):
    return (np.full(B, -7, dtype=np.int32), np.full((B, max_depth + 1), -7, dtype=np.int32),
            np.full(B, -7, dtype=np.int32), np.zeros(B, dtype=np.int32))


def accept_greedy(logits, tokens, parent, n_nodes=None, max_depth=None):
    """logits [B,T,V] f32 -> dict(accept_len[B], path[B,max_depth+1], next_token[B], status[B])."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    B, T, V = logits.shape
    tokens = _i32(tokens).reshape(B, T)
    parent = _i32(parent).reshape(B, T)
    n_nodes = _i32(n_nodes)
    if max_depth is None:
        max_depth = T - 1
    a, path, nxt, status = _accept_outputs(B, max_depth)
    f32, i32 = ctypes.c_float, ctypes.c_int32
    rc = _load().s4c_oracle_accept_greedy(
        _ptr(logits, f32), _ptr(tokens, i32), _ptr(parent, i32), _ptr(n_nodes, i32),
        B, T, V, max_depth, _ptr(a, i32), _ptr(path, i32), _ptr(nxt, i32), _ptr(status, i32))
    if rc:
        raise ValueError(f"oracle accept_greedy rejected its arguments (code {rc})")
    return dict(accept_len=a, path=path, next_token=nxt, status=status)


def accept_stochastic(logits, draft_probs, tokens, parent, temperature, uniforms, n_nodes=None,
                      max_depth=None):
    """Eq. 11 / Eq. 12 walk; returns dict(accept_len, path, next_token, near_tie[B,T], status)."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    draft_probs = np.ascontiguousarray(draft_probs, dtype=np.float32)
    B, T, V = logits.shape
    assert draft_probs.shape == (B, T, V)
    tokens = _i32(tokens).reshape(B, T)
    parent = _i32(parent).reshape(B, T)
    uniforms = np.ascontiguousarray(uniforms, dtype=np.float32).reshape(B, T)
    n_nodes = _i32(n_nodes)
    if max_depth is None:
        max_depth = T - 1
    a, path, nxt, status = _accept_outputs(B, max_depth)
    tie = np.zeros((B, T), dtype=np.uint8)
    f32, i32 = ctypes.c_float, ctypes.c_int32
    rc = _load().s4c_oracle_accept_stochastic(
        _ptr(logits, f32), _ptr(draft_probs, f32), _ptr(tokens, i32), _ptr(parent, i32),
        _ptr(n_nodes, i32), ctypes.c_double(float(temperature)), _ptr(uniforms, f32),
        B, T, V, max_depth, _ptr(a, i32), _ptr(path, i32), _ptr(nxt, i32),
        _ptr(tie, ctypes.c_uint8), _ptr(status, i32))
    if rc:
        raise ValueError(f"oracle accept_stochastic rejected its arguments (code {rc})")
    return dict(accept_len=a, path=path, next_token=nxt, near_tie=tie, status=status)


def accept_filtered(logits, draft_probs, tokens, parent, temperature, top_k, top_p, uniforms, n_nodes=None,
                    max_depth=None):
    """Speculative sampling against the top-k / nucleus filtered target distribution (steps F1-F3 of the C source)."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    draft_probs = np.ascontiguousarray(draft_probs, dtype=np.float32)
    B, T, V = logits.shape
    tokens = _i32(tokens).reshape(B, T)
    parent = _i32(parent).reshape(B, T)
    uniforms = np.ascontiguousarray(uniforms, dtype=np.float32).reshape(B, T)
    n_nodes = _i32(n_nodes)
    if max_depth is None:
        max_depth = T - 1
    a, path, nxt, status = _accept_outputs(B, max_depth)
    tie = np.zeros((B, T), dtype=np.uint8)
    f32, i32 = ctypes.c_float, ctypes.c_int32
    rc = _load().s4c_oracle_accept_filtered(
        _ptr(logits, f32), _ptr(draft_probs, f32), _ptr(tokens, i32), _ptr(parent, i32), _ptr(n_nodes, i32),
        ctypes.c_double(float(temperature)), int(top_k), ctypes.c_double(float(top_p)), _ptr(uniforms, f32),
        B, T, V, max_depth, _ptr(a, i32), _ptr(path, i32), _ptr(nxt, i32), _ptr(tie, ctypes.c_uint8), _ptr(status, i32))
    if rc:
        raise ValueError(f"oracle accept_filtered rejected its arguments (code {rc})")
    return dict(accept_len=a, path=path, next_token=nxt, near_tie=tie, status=status)


def kv_compact(k_caches, v_caches, cache_len, path, accept_len, T, feat_in=None, feat_out=None):
    """In place on lists of numpy caches [B,Hkv,C,d] (any fixed-size dtype); returns status[B].

    ``T`` is the number of tree slots per sequence.  ``cache_len`` (int32 array) is updated in
    place to L_b + a + 1; ``feat_out`` [B,max_depth+1,hid] receives rows 0..a of ``feat_in``
    [B,T,hid] gathered along the path.
    """
    n_layers = len(k_caches)
    assert len(v_caches) == n_layers
    assert cache_len.dtype == np.int32 and cache_len.flags.c_contiguous
    B = cache_len.shape[0]
    path = _i32(path).reshape(B, -1)
    max_depth = path.shape[1] - 1
    accept_len = _i32(accept_len)
    if n_layers:
        _, Hkv, C, d = k_caches[0].shape
        esz = k_caches[0].dtype.itemsize
    else:
        Hkv, C, d, esz = 1, 1, 1, (feat_in.dtype.itemsize if feat_in is not None else 1)
    for c in list(k_caches) + list(v_caches):
        assert c.flags.c_contiguous and c.shape == (B, Hkv, C, d) and c.dtype.itemsize == esz
    u8p = ctypes.POINTER(ctypes.c_uint8)
    karr = (u8p * max(n_layers, 1))(*[c.ctypes.data_as(u8p) for c in k_caches])
    varr = (u8p * max(n_layers, 1))(*[c.ctypes.data_as(u8p) for c in v_caches])
    hid = 0
    if feat_in is not None:
        assert feat_in.flags.c_contiguous and feat_out is not None and feat_out.flags.c_contiguous
        assert feat_in.shape[0] == B and feat_in.shape[1] == T and feat_in.dtype.itemsize == esz
        hid = feat_in.shape[2]
        assert feat_out.shape == (B, max_depth + 1, hid) and feat_out.dtype == feat_in.dtype
    status = np.zeros(B, dtype=np.int32)
    rc = _load().s4c_oracle_kv_compact(
        karr, varr, n_layers, _ptr(cache_len, ctypes.c_int32), _ptr(path, ctypes.c_int32),
        _ptr(accept_len, ctypes.c_int32), max_depth,
        None if feat_in is None else feat_in.ctypes.data_as(u8p),
        None if feat_out is None else feat_out.ctypes.data_as(u8p),
        B, T, Hkv, d, C, hid, esz, _ptr(status, ctypes.c_int32))
    if rc:
        raise ValueError(f"oracle kv_compact rejected its arguments (code {rc})")
    return status


def build_tree(draft_probs, branching, root_token, cache_len=None):
    """draft_probs [B,T,V] f32, branching (sequence of ints), root_token [B] -> dict(tokens, parent, position [B,T], n_nodes [B])."""
    draft_probs = np.ascontiguousarray(draft_probs, dtype=np.float32)
    B, T, V = draft_probs.shape
    br = np.ascontiguousarray(branching, dtype=np.int32)
    root_token = _i32(root_token).reshape(B)
    cache_len = _i32(cache_len)
    tokens = np.full((B, T), -7, dtype=np.int32)
    parent = np.full((B, T), -7, dtype=np.int32)
    position = np.full((B, T), -7, dtype=np.int32)
    n_nodes = np.full(B, -7, dtype=np.int32)
    f32, i32 = ctypes.c_float, ctypes.c_int32
    rc = _load().s4c_oracle_build_tree(_ptr(draft_probs, f32), _ptr(br, i32), int(len(br)), _ptr(root_token, i32),
                                       _ptr(cache_len, i32), B, T, V, _ptr(tokens, i32), _ptr(parent, i32),
                                       _ptr(position, i32), _ptr(n_nodes, i32))
    if rc:
        raise ValueError(f"oracle build_tree rejected its arguments (code {rc})")
    return dict(tokens=tokens, parent=parent, position=position, n_nodes=n_nodes)


# ------------------------------------------------------------------ paged caches (a layout, not a step of the method)
def pages_to_contiguous(pages, block_table):
    """The contiguous cache [B,Hkv,max_blocks*page_size,d] that a pool of pages [n_pages,Hkv,page_size,d] spells out under
    block_table [B,max_blocks] -- by definition of a paged cache: slot s of sequence b is slot s % page_size of page
    block_table[b, s // page_size].  (Entries outside the pool read as page 0 here; callers only list blocks in use.)"""
    pages = np.asarray(pages)
    bt = np.asarray(block_table, dtype=np.int64)
    n_pages, Hkv, ps, d = pages.shape
    B, nb = bt.shape
    safe = np.where((bt >= 0) & (bt < n_pages), bt, 0)
    g = pages[safe]                                  # [B, nb, Hkv, ps, d]
    return np.ascontiguousarray(g.transpose(0, 2, 1, 3, 4).reshape(B, Hkv, nb * ps, d))


def scatter_to_pages(pages, block_table, contiguous, blocks_in_use):
    """Writes the blocks in use (per sequence, a count) of a contiguous cache back into the pool, in place."""
    n_pages, Hkv, ps, d = pages.shape
    for b in range(contiguous.shape[0]):
        for i in range(int(blocks_in_use[b])):
            pages[int(block_table[b, i])] = contiguous[b, :, i * ps:(i + 1) * ps]
    return pages


def lm_head_greedy(hidden, weight):
    """The LM head of the verify pass followed by the greedy choice (Eq. 6: t = Argmax(LM_head(f)); Section 3.2: the
    target's logits at every tree node; Section 4.1: greedy decoding): logits[r, v] = sum_h hidden[r, h] * weight[v, h]
    in float64 (a library matrix product is the step), token[r] = the first maximum of row r.

    hidden [R, H], weight [V, H] (any float type: the values as given, e.g. already rounded to bf16).
    Returns dict(token [R] int32, max_logit [R] float64, logits [R, V] float64)."""
    h = np.asarray(hidden, dtype=np.float64)
    w = np.asarray(weight, dtype=np.float64)
    assert h.ndim == 2 and w.ndim == 2 and h.shape[1] == w.shape[1]
    logits = h @ w.T
    token = np.argmax(logits, axis=1).astype(np.int32)  # numpy returns the first of equal maxima
    return dict(token=token, max_logit=logits[np.arange(len(h)), token], logits=logits)


def accept_greedy_tokens(target_token, tokens, parent, n_nodes=None, max_depth=None, V=None):
    """Greedy verification (Section 4.1; longest accepted path, Section 3.2) when the target's greedy choice at every
    node is already known: a node is accepted when its parent is and its token is the target's choice at the parent; the
    path ends at the accepted node of greatest depth (lowest index among equals); the token emitted after the path is
    the target's choice at its end.

    target_token [B,T] int32 (row n: the choice after node n), tokens [B,T], parent [B,T]; V (optional): tokens outside
    [0, V) flag the sequence.  Returns dict(accept_len[B], path[B,max_depth+1] (-1 padded), next_token[B], status[B])
    like accept_greedy."""
    target_token = _i32(target_token)
    B, T = target_token.shape
    tokens = _i32(tokens).reshape(B, T)
    parent = _i32(parent).reshape(B, T)
    if max_depth is None:
        max_depth = T - 1
    a, path, nxt, status = _accept_outputs(B, max_depth)
    for b in range(B):
        n = T if n_nodes is None else int(n_nodes[b])
        flags = 0
        if n < 1 or n > T:
            flags |= SEQ_BAD_PARENT
        else:
            for i in range(n):
                p = int(parent[b, i])
                if (i == 0 and p != -1) or (i > 0 and not (0 <= p < i)):
                    flags |= SEQ_BAD_PARENT
        depth = [0] * T
        if not flags:
            for i in range(n):
                if i > 0:
                    depth[i] = depth[parent[b, i]] + 1
                if depth[i] > max_depth:
                    flags |= SEQ_DEPTH
                if V is not None and not (0 <= tokens[b, i] < V):
                    flags |= SEQ_TOKEN_RANGE
        status[b] = flags
        if flags:
            a[b], nxt[b], path[b, :] = -1, -1, -1
            continue
        ok = [False] * n
        ok[0], end = True, 0
        for i in range(1, n):
            p = int(parent[b, i])
            ok[i] = ok[p] and tokens[b, i] == target_token[b, p]
            if ok[i] and depth[i] > depth[end]:
                end = i
        walked = []
        i = end
        while i >= 0:
            walked.append(i)
            i = int(parent[b, i])
        walked.reverse()
        a[b] = len(walked) - 1
        path[b, :] = -1
        path[b, :len(walked)] = walked
        nxt[b] = target_token[b, end]
    return dict(accept_len=a, path=path, next_token=nxt, status=status)


def rope_rotate(x, pos, theta=10000.0):
    """Rotary position embedding in the rotate-half form used by the LLaMA / Vicuna family (the paper's target models): for
    a head vector x[0..d) at position pos, with x1 = x[:d/2], x2 = x[d/2:], angle_i = pos * theta**(-2i/d):
    out[:d/2] = x1*cos - x2*sin, out[d/2:] = x2*cos + x1*sin.  float64.  x [..., d], pos broadcastable to x[..., 0]."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    assert d % 2 == 0
    i = np.arange(d // 2, dtype=np.float64)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * theta ** (-2.0 * i / d)
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., : d // 2], x[..., d // 2:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def qkv_rope(x, w_qkv, cache_len, parent, Hq, Hkv, d, k_cache, v_cache, n_nodes=None, theta=10000.0, position_base=None):
    """The verify layer's input side (Section 3.2: the target's forward pass over the T tree tokens; a decoder layer of the
    LLaMA family): q, k, v = x W^T for every tree token (float64; a library matrix product is the step), rotary embedding of
    q and k at position cache_len[b] + depth(node), q into a [B,Hq,T,d] array, k and v into the caches' tree slots
    cache_len[b] + node (k_cache, v_cache [B,Hkv,C,d] float64 arrays, modified in place).

    x [B,T,H]; w_qkv [(Hq+2*Hkv)*d, H]: the q heads' rows, then the k heads', then the v heads'.
    position_base [B] (optional): the position of a sequence's root when it is not its cache length -- a drafter head whose own
    cache is shorter than the text (Section 3.1.1: every head keeps its own features): a node's position is then
    position_base[b] + depth(node); its slot stays cache_len[b] + node.  A negative base flags the sequence (SEQ_CAPACITY).

    Returns dict(q [B,Hq,T,d] float64 (rows of nodes >= n_nodes[b] and of flagged sequences are zero), status [B])."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w_qkv, dtype=np.float64)
    B, T, H = x.shape
    assert w.shape == ((Hq + 2 * Hkv) * d, H)
    parent = _i32(parent).reshape(B, T)
    cache_len = _i32(cache_len)
    C = k_cache.shape[2]
    q = np.zeros((B, Hq, T, d))
    status = np.zeros(B, dtype=np.int32)
    for b in range(B):
        n = T if n_nodes is None else int(n_nodes[b])
        flags = 0
        if n < 1 or n > T:
            flags |= SEQ_BAD_PARENT
        else:
            for i in range(n):
                p = int(parent[b, i])
                if (i == 0 and p != -1) or (i > 0 and not (0 <= p < i)):
                    flags |= SEQ_BAD_PARENT
        L = int(cache_len[b])
        if L < 0 or L + T > C:
            flags |= SEQ_CAPACITY
        P = L if position_base is None else int(position_base[b])
        if P < 0:
            flags |= SEQ_CAPACITY
        status[b] = flags
        if flags:
            continue
        depth = np.zeros(n, dtype=np.int64)
        for i in range(1, n):
            depth[i] = depth[parent[b, i]] + 1
        proj = x[b, :n] @ w.T                                   # [n, (Hq+2Hkv)*d]
        qh = proj[:, : Hq * d].reshape(n, Hq, d)
        kh = proj[:, Hq * d: (Hq + Hkv) * d].reshape(n, Hkv, d)
        vh = proj[:, (Hq + Hkv) * d:].reshape(n, Hkv, d)
        pos = (P + depth)[:, None]
        q[b, :, :n] = rope_rotate(qh, pos, theta).transpose(1, 0, 2)
        k_cache[b, :, L:L + n] = rope_rotate(kh, pos, theta).transpose(1, 0, 2)
        v_cache[b, :, L:L + n] = vh.transpose(1, 0, 2)
    return dict(q=q, status=status)


def lm_head_topk(hidden, weight, k):
    """The drafter's LM head followed by its top-k choice (Eq. 6 and Section 3.1: Argmax / top-2 of LM_head(f); Section 3.2:
    the top-k alternatives of the verification tree): float64 logits as in :func:`lm_head_greedy`, then per row the k tokens
    of greatest logit, greatest first, equal logits by lower token (a library sort, stable, is the step).

    Returns dict(token [R, k] int32 (-1 beyond the vocabulary when k > V), logit [R, k] float64, logits [R, V])."""
    h = np.asarray(hidden, dtype=np.float64)
    w = np.asarray(weight, dtype=np.float64)
    assert h.ndim == 2 and w.ndim == 2 and h.shape[1] == w.shape[1] and k >= 1
    logits = h @ w.T
    order = np.argsort(-logits, axis=1, kind="stable")[:, :k]
    R, V = logits.shape
    token = np.full((R, k), -1, dtype=np.int32)
    logit = np.full((R, k), -np.inf)
    token[:, : order.shape[1]] = order
    logit[:, : order.shape[1]] = np.take_along_axis(logits, order, axis=1)
    return dict(token=token, logit=logit, logits=logits)


def build_tree_from_topk(topk, branching, root_token, T, cache_len=None):
    """The continuous verification tree (Section 3.2 / Figure 3) from the drafter's ranked choices instead of its
    distributions: the same shape as :func:`build_tree` (vertical first, then horizontal, cut at T nodes, breadth-first
    numbering); child j of node n carries topk[b, n, j].  topk [B, T, k] int32 with k >= max(branching).
    Returns dict(tokens, parent, position, n_nodes) like build_tree."""
    topk = _i32(topk)
    B, T_, k = topk.shape
    assert T_ == T and k >= max(branching)
    # the shape, in creation order: the vertical chain of first choices, then, depth by depth, every node of the previous
    # depth is filled up to its branching factor, until T nodes exist
    cpar, cdep, nchild = [-1], [0], [0]
    tip = 0
    for l in range(len(branching)):
        if len(cpar) >= T:
            break
        cpar.append(tip), cdep.append(l + 1), nchild.append(0)
        nchild[tip] += 1
        tip = len(cpar) - 1
    for l in range(1, len(branching) + 1):
        for node in range(len(cpar)):
            if cdep[node] != l - 1:
                continue
            while nchild[node] < branching[l - 1] and len(cpar) < T:
                cpar.append(node), cdep.append(l), nchild.append(0)
                nchild[node] += 1
    # breadth-first numbering; a node's children keep their creation order (= rank order)
    order, head = [0], 0
    while head < len(order):
        u = order[head]
        head += 1
        order.extend(c for c in range(len(cpar)) if cpar[c] == u)
    newid = {c: i for i, c in enumerate(order)}
    parent = [-1 if c == 0 else newid[cpar[c]] for c in order]
    depth = [cdep[c] for c in order]
    n = len(parent)
    tokens = np.zeros((B, T), dtype=np.int32)
    par = np.full((B, T), -1, dtype=np.int32)
    pos = np.zeros((B, T), dtype=np.int32)
    base = np.zeros(B, dtype=np.int64) if cache_len is None else np.asarray(cache_len, dtype=np.int64)
    for b in range(B):
        tokens[b, 0] = root_token[b]
        rank = {}
        for i in range(1, n):
            j = rank.get(parent[i], 0)
            rank[parent[i]] = j + 1
            tokens[b, i] = topk[b, parent[i], j]
        par[b, :n] = parent
        pos[b, :n] = base[b] + np.asarray(depth)
    return dict(tokens=tokens, parent=par, position=pos, n_nodes=np.full(B, n, dtype=np.int32))


def linear(x, w, x2=None, bias=None, residual=None, gate=False):
    """A linear layer of the drafter / decoder layer in float64 (a library matrix product is the step).

    y = concat[x, x2] @ w^T (+ bias): with x2 this is Eq. 3, h = Linear(concat[e, f]) -- x the embeddings, x2 the features,
    w [N, K1 + K2].  gate=True: w holds 2N rows, the gate projection's N rows first, then the up projection's; the result is
    silu(gate) * up, the LLaMA-family MLP's inner product (silu(z) = z / (1 + exp(-z))).  residual [R, N] is added last."""
    xx = np.asarray(x, dtype=np.float64)
    if x2 is not None:
        xx = np.concatenate([xx, np.asarray(x2, dtype=np.float64)], axis=-1)
    ww = np.asarray(w, dtype=np.float64)
    y = xx @ ww.T
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)
    if gate:
        n = y.shape[-1] // 2
        g, u = y[..., :n], y[..., n:]
        y = g / (1.0 + np.exp(-g)) * u
    if residual is not None:
        y = y + np.asarray(residual, dtype=np.float64)
    return y


def rmsnorm(x, weight, eps=1e-6):
    """Root-mean-square layer normalisation of the LLaMA family: x / sqrt(mean(x^2) + eps) * weight, float64."""
    xx = np.asarray(x, dtype=np.float64)
    return xx / np.sqrt(np.mean(xx * xx, axis=-1, keepdims=True) + eps) * np.asarray(weight, dtype=np.float64)


def embed_gather(table, tokens):
    """Eq. 6: e = Embedding(t): rows of the embedding table."""
    return np.asarray(table)[np.asarray(tokens, dtype=np.int64)]
