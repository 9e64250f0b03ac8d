"""ctypes front-end of the CPU oracle (oracle/ss_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's cpu_baseline /
reference arm.  The CUDA package never imports this module and this module never imports the CUDA package.
All arrays are host numpy arrays; bf16 values travel as uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ss_oracle.cpp")
_LIB = os.path.join(_HERE, "libss_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ -O2 (no fast-math, so fp64 semantics are the plain IEEE ones)."""
    if force or (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-std=c++14", "-shared", "-fPIC", "-pthread", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.ss_oracle_dedup.restype = ctypes.c_int32
            lib.ss_oracle_tree_attention.restype = ctypes.c_int32
            lib.ss_oracle_topk.restype = None
            lib.ss_oracle_early_prune.restype = None
            lib.ss_oracle_branch_sample.restype = None
            _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dt):
    return None if a is None else np.ascontiguousarray(a, dtype=dt)


def _bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 bit patterns on the host."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


def dedup(tok_ids, tok_offsets, ctx_key=None, slot_in=None):
    """-> dict(canon, path_to_unique, unique_paths[U], multiplicity[U], slot_out or None, num_unique)."""
    lib = _load()
    tok_ids = _c(tok_ids, np.int32)
    tok_offsets = _c(tok_offsets, np.int64)
    n = int(tok_offsets.shape[0]) - 1
    ctx_key = _c(ctx_key, np.int64)
    slot_in = _c(slot_in, np.int32)
    canon = np.zeros(max(n, 1), np.int32)
    p2u = np.zeros(max(n, 1), np.int32)
    uniq = np.zeros(max(n, 1), np.int32)
    mult = np.zeros(max(n, 1), np.int32)
    slot_out = np.zeros(max(n, 1), np.int32) if slot_in is not None else None
    if tok_ids.size == 0:
        tok_ids = np.zeros(1, np.int32)
    u = lib.ss_oracle_dedup(_p(tok_ids), _p(tok_offsets), _p(ctx_key), _p(slot_in), ctypes.c_int32(n),
                            _p(canon), _p(p2u), _p(uniq), _p(mult), _p(slot_out))
    return dict(canon=canon[:n], path_to_unique=p2u[:n], unique_paths=uniq[:u].copy(),
                multiplicity=mult[:u].copy(), slot_out=None if slot_out is None else slot_out[:n],
                num_unique=int(u))


def tree_attention(num_q_heads, num_kv_heads, head_dim, page_size, sm_scale, k_pool_bits, v_pool_bits,
                   page_stride, head_stride, token_stride, node_parent, node_kv_len, node_page_offsets,
                   node_pages, path_leaf_node, path_q_len, q_offsets, q_bits, n_threads=None):
    """k_pool_bits / v_pool_bits: flat uint16 views whose element 0 is the K (resp. V) element of page 0,
    head 0, token 0, dim 0.  q_bits: uint16 [total_q][Hq][D].  -> (out f64 [total_q][Hq][D], lse f64)."""
    lib = _load()
    k_pool_bits = np.ascontiguousarray(k_pool_bits).reshape(-1)
    v_pool_bits = np.ascontiguousarray(v_pool_bits).reshape(-1)
    assert k_pool_bits.dtype == np.uint16 and v_pool_bits.dtype == np.uint16
    node_parent = _c(node_parent, np.int32)
    node_kv_len = _c(node_kv_len, np.int32)
    node_page_offsets = _c(node_page_offsets, np.int64)
    node_pages = _c(node_pages, np.int32)
    if node_pages.size == 0:
        node_pages = np.zeros(1, np.int32)
    path_leaf_node = _c(path_leaf_node, np.int32)
    path_q_len = _c(path_q_len, np.int32)
    q_offsets = _c(q_offsets, np.int64)
    n_paths = int(path_leaf_node.shape[0])
    total_q = int(q_offsets[n_paths]) if n_paths else 0
    q_bits = np.ascontiguousarray(q_bits).reshape(-1)
    assert q_bits.dtype == np.uint16
    if q_bits.size == 0:
        q_bits = np.zeros(1, np.uint16)
    out = np.zeros((max(total_q, 1), num_q_heads, head_dim), np.float64)
    lse = np.zeros((max(total_q, 1), num_q_heads), np.float64)
    if n_threads is None:
        n_threads = host_cores()
    rc = lib.ss_oracle_tree_attention(
        ctypes.c_int32(num_q_heads), ctypes.c_int32(num_kv_heads), ctypes.c_int32(head_dim),
        ctypes.c_int32(page_size), ctypes.c_double(sm_scale), _p(k_pool_bits), _p(v_pool_bits),
        ctypes.c_int64(page_stride), ctypes.c_int64(head_stride), ctypes.c_int64(token_stride),
        ctypes.c_int32(int(node_parent.shape[0])), _p(node_parent), _p(node_kv_len), _p(node_page_offsets),
        _p(node_pages), ctypes.c_int32(n_paths), _p(path_leaf_node), _p(path_q_len), _p(q_offsets),
        _p(q_bits), _p(out), _p(lse), ctypes.c_int32(int(n_threads)))
    if rc != 0:
        raise ValueError("oracle: malformed tree")
    return out[:total_q], lse[:total_q]


def tree_attention_workload(w, paths=None, sm_scale=None, n_threads=None):
    """Oracle attention on a synthetic workload object (host tensors), optionally restricted to `paths`
    (ascending logical indices; the outputs are then in the compacted query order)."""
    flat = _bits(w.kv_pool).reshape(-1)
    v_off = w.num_kv_heads * w.page_size * w.head_dim
    if paths is None:
        leaf, T, qoff = w.path_leaf_node, w.path_q_len, w.q_offsets
        qb = _bits(w.q)
    else:
        paths = np.asarray(paths, dtype=np.int64)
        leaf, T = w.path_leaf_node[paths], w.path_q_len[paths]
        qoff = np.zeros(len(paths) + 1, np.int64)
        np.cumsum(T.astype(np.int64), out=qoff[1:])
        rows = np.concatenate([np.arange(w.q_offsets[i], w.q_offsets[i + 1]) for i in paths]) if len(paths) \
            else np.zeros(0, np.int64)
        qb = _bits(w.q)[rows]
    if sm_scale is None:
        sm_scale = 1.0 / float(np.sqrt(w.head_dim))
    return tree_attention(w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_size, sm_scale, flat, flat[v_off:],
                          2 * v_off, w.page_size * w.head_dim, w.head_dim, w.node_parent, w.node_kv_len,
                          w.node_page_offsets, w.node_pages, leaf, T, qoff, qb, n_threads=n_threads)


def topk(scores, seg_offsets, k):
    """-> (survivors int32 [P][k] (-1 padded), keep uint8 [N])."""
    lib = _load()
    scores = _c(scores, np.float32)
    seg_offsets = _c(seg_offsets, np.int32)
    n_seg = int(seg_offsets.shape[0]) - 1
    n = int(scores.shape[0])
    surv = np.full((max(n_seg, 1), max(k, 1)), -1, np.int32)
    keep = np.zeros(max(n, 1), np.uint8)
    sc = scores if n else np.zeros(1, np.float32)
    lib.ss_oracle_topk(_p(sc), _p(seg_offsets), ctypes.c_int32(n_seg), ctypes.c_int32(k), _p(surv), _p(keep))
    return surv[:n_seg, :k].reshape(n_seg, k), keep[:n]


def early_prune(scores, verified, seg_offsets, k):
    """-> (pruned uint8 [N], selected int32 [P][k] (-1 padded), final uint8 [P])."""
    lib = _load()
    scores = _c(scores, np.float32)
    verified = _c(verified, np.uint8)
    seg_offsets = _c(seg_offsets, np.int32)
    n_seg = int(seg_offsets.shape[0]) - 1
    n = int(scores.shape[0])
    pruned = np.zeros(max(n, 1), np.uint8)
    sel = np.full((max(n_seg, 1), max(k, 1)), -1, np.int32)
    fin = np.zeros(max(n_seg, 1), np.uint8)
    sc = scores if n else np.zeros(1, np.float32)
    ve = verified if n else np.zeros(1, np.uint8)
    lib.ss_oracle_early_prune(_p(sc), _p(ve), _p(seg_offsets), ctypes.c_int32(n_seg), ctypes.c_int32(k), _p(pruned),
                              _p(sel), _p(fin))
    return pruned[:n], sel[:n_seg, :k].reshape(n_seg, k), fin[:n_seg]


def branch_sample(logits, draw_offsets, uniforms, temperature):
    """logits f32 [n_seq][vocab], draw_offsets int64 [n_seq+1], uniforms f32 [total draws] ->
    (tokens int32 [draws], seq int64 [draws], margin f64 [draws])."""
    lib = _load()
    logits = _c(logits, np.float32)
    draw_offsets = _c(draw_offsets, np.int64)
    uniforms = _c(uniforms, np.float32)
    n_seq, vocab = int(logits.shape[0]), int(logits.shape[1])
    n = int(draw_offsets[-1])
    tokens = np.zeros(max(n, 1), np.int32)
    seq = np.zeros(max(n, 1), np.int64)
    margin = np.zeros(max(n, 1), np.float64)
    un = uniforms if n else np.zeros(1, np.float32)
    lib.ss_oracle_branch_sample(_p(logits), _p(draw_offsets), _p(un), ctypes.c_int32(n_seq), ctypes.c_int32(vocab),
                                ctypes.c_double(float(temperature)), _p(tokens), _p(seq), _p(margin))
    return tokens[:n], seq[:n], margin[:n]


def gather_unique(unique_paths, num_unique, n_paths, path_leaf_node, path_q_len, q_offsets):
    """Per-path arguments of the single forward pass a group of equal candidates gets (paper, Section
    "Computation Deduplication"): the descriptor rows of the group representatives, in order, written as plain
    loops.  Entries past the number of unique paths are inert (-1 / 0 / 0, offsets stay at the total)."""
    U = max(0, min(int(num_unique), int(n_paths)))
    u_leaf = np.full(n_paths, -1, np.int32)
    u_q_len = np.zeros(n_paths, np.int32)
    u_q_src = np.zeros(n_paths, np.int64)
    u_q_offsets = np.zeros(n_paths + 1, np.int64)
    for p in range(n_paths):
        if p < U:
            s = int(unique_paths[p])
            u_leaf[p] = path_leaf_node[s]
            u_q_len[p] = path_q_len[s]
            u_q_src[p] = q_offsets[s]
        u_q_offsets[p + 1] = u_q_offsets[p] + int(u_q_len[p])
    return dict(u_leaf=u_leaf, u_q_len=u_q_len, u_q_offsets=u_q_offsets, u_q_src=u_q_src)


def build_prefix_tree(tok_ids, tok_offsets, page_size=16):
    """Radix tree of candidate paths over whole KV pages (paper, Section "Computation Deduplication": candidates share
    25-50 % of their tokens; Section "Experimental Setup": prefix caching and sharing of KV pages).

    Plain definition, written as a recursive partition: every path is cut into its full pages (tuples of `page_size`
    token ids) and a tail (the remaining tokens).  A group of at least two paths that share more full pages than the
    chain above them holds gets an inner node with exactly the pages ALL of them share; the group is then split
    wherever two neighbours (in sorted order) share no further page, and every part is treated the same way.  A
    single path gets a private leaf node with whatever the chain above it does not hold (pages + tail; possibly
    nothing).  So only whole pages are ever shared, and every inner node has at least two children.
    Order: paths sorted by token sequence (shorter first on a common prefix, then input index); nodes numbered in
    depth-first preorder along that order, so parents precede children and the paths below a node are contiguous.

    Returns order [n], path_leaf_node [n] (by rank), node_parent, node_kv_len, node_src_path (an input path that
    contains the node's tokens), node_src_offset (where they start in it)."""
    n = len(tok_offsets) - 1
    seqs = [tuple(int(t) for t in tok_ids[tok_offsets[i]:tok_offsets[i + 1]]) for i in range(n)]
    order = sorted(range(n), key=lambda i: (seqs[i], i))
    pages = [tuple(seqs[i][k * page_size:(k + 1) * page_size] for k in range(len(seqs[i]) // page_size)) for i in range(n)]
    node_parent, node_kv_len, node_src_path, node_src_offset = [], [], [], []
    path_leaf = [0] * n

    def shared_pages(a, b):                      # common full pages of two paths
        k = 0
        while k < len(pages[a]) and k < len(pages[b]) and pages[a][k] == pages[b][k]:
            k += 1
        return k

    def emit(lo, hi, depth, parent):
        """Paths order[lo:hi] all share `depth` pages, which the chain up to `parent` holds."""
        if hi - lo == 1:
            i = order[lo]
            node_parent.append(parent); node_kv_len.append(len(seqs[i]) - depth * page_size)
            node_src_path.append(i); node_src_offset.append(depth * page_size)
            path_leaf[lo] = len(node_parent) - 1
            return
        common = min(shared_pages(order[lo], order[r]) for r in range(lo + 1, hi))
        if common > depth:                        # an inner node with the pages every path of the group shares
            node_parent.append(parent); node_kv_len.append((common - depth) * page_size)
            node_src_path.append(order[lo]); node_src_offset.append(depth * page_size)
            parent = len(node_parent) - 1
            depth = common
        # split where neighbours share no more than `depth` pages
        start = lo
        for r in range(lo + 1, hi + 1):
            if r == hi or shared_pages(order[r - 1], order[r]) <= depth:
                emit(start, r, depth, parent)
                start = r

    if n:
        # top level: groups of neighbours that share at least one page; single paths otherwise
        start = 0
        for r in range(1, n + 1):
            if r == n or shared_pages(order[r - 1], order[r]) == 0:
                emit(start, r, 0, -1)
                start = r
    return dict(order=np.asarray(order, np.int32), path_leaf_node=np.asarray(path_leaf, np.int32),
                node_parent=np.asarray(node_parent, np.int32), node_kv_len=np.asarray(node_kv_len, np.int32),
                node_src_path=np.asarray(node_src_path, np.int32), node_src_offset=np.asarray(node_src_offset, np.int32))
