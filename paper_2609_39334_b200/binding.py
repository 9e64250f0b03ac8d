"""Thin ctypes binding of libspecscale.so - argument marshalling only.

The functions carry the names of the C ABI (include/specscale.h).  Tensors are torch tensors that already live on
the GPU; torch provides device memory and streams and nothing else.  There is no CPU fallback: if the CUDA
library is missing, loading fails with an error.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# SS_LIB_SUFFIX selects a build variant (build.build(defines=..., suffix=...)): "_checked" for the build with device-side
# range checks, or an instrumented build; the default is the production library.
LIB_PATH = os.path.join(_HERE, "libspecscale" + os.environ.get("SS_LIB_SUFFIX", "") + ".so")

SS_OK = 0
SS_ERR_INVALID_ARG = 1
SS_ERR_UNSUPPORTED = 2
SS_ERR_WORKSPACE_TOO_SMALL = 3
SS_ERR_CUDA = 4
SS_ERR_BAD_INPUT = 5
SS_ERR_TIMEOUT = 6
SS_FLAG_VALIDATE = 0x1
SS_FLAG_FORCE_GENERIC = 0x2
SS_FLAG_NO_TCGEN05 = 0x4
SS_FLAG_WEAK_HASH = 0x8
SS_FLAG_TILES_2CTA = 0x10
SS_MAX_DEPTH = 16
SS_STEP_COMPACT_TRANSFERS = 0x1
SS_DEDUP_STATIC_MAX_PATHS = 65536

EXPORTS = [
    "ss_status_string", "ss_last_device_status", "ss_dedup_workspace_bytes", "ss_dedup_paths",
    "ss_tree_attention_workspace_bytes", "ss_tree_attention", "ss_topk_workspace_bytes", "ss_topk_prune",
    "ss_launch_count", "ss_debug_umma_tile", "ss_debug_bounded_wait", "ss_profile_enable", "ss_profile_read",
    "ss_dedup_paths_static", "ss_debug_tile_kernel_occupancy", "ss_early_prune",
    "ss_branch_sample", "ss_gather_unique_paths", "ss_candidate_step_host_arena_bytes", "ss_candidate_step_host",
    "ss_prefix_tree_workspace_bytes", "ss_build_prefix_tree",
]
PHASES = ["plan", "tiles", "leaves", "generic", "merge"]


class SpecScaleError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class ss_attn_desc_t(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("flags", ctypes.c_uint32),
        ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("sm_scale", ctypes.c_float), ("max_sms", ctypes.c_int32),
        ("k_pool", ctypes.c_void_p), ("v_pool", ctypes.c_void_p),
        ("num_pages", ctypes.c_int64),
        ("kv_page_stride", ctypes.c_int64), ("kv_head_stride", ctypes.c_int64), ("kv_token_stride", ctypes.c_int64),
        ("num_nodes", ctypes.c_int32), ("reserved1", ctypes.c_int32),
        ("node_parent", ctypes.c_void_p), ("node_kv_len", ctypes.c_void_p),
        ("node_page_offsets", ctypes.c_void_p), ("node_pages", ctypes.c_void_p),
        ("total_node_pages", ctypes.c_int64),
        ("num_paths", ctypes.c_int32), ("reserved2", ctypes.c_int32),
        ("num_paths_dev", ctypes.c_void_p), ("path_leaf_node", ctypes.c_void_p), ("path_q_len", ctypes.c_void_p),
        ("q_offsets", ctypes.c_void_p), ("total_q", ctypes.c_int64),
        ("max_depth", ctypes.c_int32), ("max_decode_paths", ctypes.c_int32),
        ("q_src_offsets", ctypes.c_void_p), ("q_src_rows", ctypes.c_int64),
        ("q", ctypes.c_void_p), ("out", ctypes.c_void_p), ("lse", ctypes.c_void_p),
    ]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_39334_b200.build`; "
                               "there is no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        L.ss_status_string.restype = ctypes.c_char_p
        L.ss_status_string.argtypes = [ctypes.c_int32]
        L.ss_launch_count.restype = ctypes.c_int64
        for name in EXPORTS:
            if name not in ("ss_status_string", "ss_launch_count"):
                getattr(L, name).restype = ctypes.c_int32
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().ss_status_string(int(status)).decode()


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return ctypes.c_void_p(0)
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors only"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(rc: int, where: str):
    if rc != SS_OK:
        raise SpecScaleError(rc, where)


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    """Device scratch for one call (256-byte aligned: torch's allocator aligns to 512)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def ss_launch_count() -> int:
    return int(lib().ss_launch_count())


def ss_last_device_status(workspace: torch.Tensor, stream=None) -> int:
    out = ctypes.c_int32(-1)
    _check(lib().ss_last_device_status(_ptr(workspace), _stream(stream), ctypes.byref(out)), "ss_last_device_status")
    return int(out.value)


# ---------------------------------------------------------------------------------------------------------
def ss_dedup_workspace_bytes(n_paths: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().ss_dedup_workspace_bytes(ctypes.c_int32(n_paths), ctypes.byref(out)), "ss_dedup_workspace_bytes")
    return int(out.value)


def ss_dedup_paths(tok_ids, tok_offsets, ctx_key, slot_in, n_paths, flags, canon_out, path_to_unique_out,
                   unique_paths_out, multiplicity_out, slot_out, num_unique_out, workspace, stream=None,
                   check=True) -> int:
    rc = lib().ss_dedup_paths(_ptr(tok_ids), _ptr(tok_offsets), _ptr(ctx_key), _ptr(slot_in), ctypes.c_int32(n_paths),
                              ctypes.c_uint32(flags), _ptr(canon_out), _ptr(path_to_unique_out),
                              _ptr(unique_paths_out), _ptr(multiplicity_out), _ptr(slot_out), _ptr(num_unique_out),
                              _ptr(workspace), ctypes.c_size_t(workspace.numel() if workspace is not None else 0),
                              _stream(stream))
    if check:
        _check(rc, "ss_dedup_paths")
    return rc


def ss_dedup_paths_static(tok_ids, tok_offsets, ctx_key, slot_in, n_paths, flags, canon_out, path_to_unique_out,
                          unique_paths_out, multiplicity_out, slot_out, num_unique_out, stream=None, check=True) -> int:
    """ss_dedup_paths for callers that may not allocate: no workspace argument, the scratch is a fixed array inside
    the library (at most SS_DEDUP_STATIC_MAX_PATHS paths; calls must not overlap on the GPU)."""
    rc = lib().ss_dedup_paths_static(_ptr(tok_ids), _ptr(tok_offsets), _ptr(ctx_key), _ptr(slot_in),
                                     ctypes.c_int32(n_paths), ctypes.c_uint32(flags), _ptr(canon_out),
                                     _ptr(path_to_unique_out), _ptr(unique_paths_out), _ptr(multiplicity_out),
                                     _ptr(slot_out), _ptr(num_unique_out), _stream(stream))
    if check:
        _check(rc, "ss_dedup_paths_static")
    return rc


def ss_gather_unique_paths(unique_paths, num_unique, n_paths, path_leaf_node, path_q_len, q_offsets, u_leaf_out,
                           u_q_len_out, u_q_offsets_out, u_q_src_out, stream=None, check=True) -> int:
    """Descriptor rows of the unique paths (leaf node, query length, query offsets, source query row) gathered by
    `unique_paths`, ready to be passed to ss_tree_attention."""
    rc = lib().ss_gather_unique_paths(_ptr(unique_paths), _ptr(num_unique), ctypes.c_int32(n_paths),
                                      _ptr(path_leaf_node), _ptr(path_q_len), _ptr(q_offsets), _ptr(u_leaf_out),
                                      _ptr(u_q_len_out), _ptr(u_q_offsets_out), _ptr(u_q_src_out), _stream(stream))
    if check:
        _check(rc, "ss_gather_unique_paths")
    return rc


def ss_prefix_tree_workspace_bytes(n_paths: int, total_tok: int, page_size: int = 16) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().ss_prefix_tree_workspace_bytes(ctypes.c_int32(n_paths), ctypes.c_int64(total_tok),
                                                ctypes.c_int32(page_size), ctypes.byref(out)),
           "ss_prefix_tree_workspace_bytes")
    return int(out.value)


def ss_build_prefix_tree(tok_ids, tok_offsets, n_paths, total_tok, page_size, order_out, path_leaf_node_out,
                         node_parent_out, node_kv_len_out, node_src_path_out, node_src_offset_out, num_nodes_out,
                         workspace, stream=None, check=True) -> int:
    """Radix tree of the paths over whole pages (parents before children, paths in sorted order)."""
    rc = lib().ss_build_prefix_tree(_ptr(tok_ids), _ptr(tok_offsets), ctypes.c_int32(n_paths), ctypes.c_int64(total_tok),
                                    ctypes.c_int32(page_size), _ptr(order_out), _ptr(path_leaf_node_out),
                                    _ptr(node_parent_out), _ptr(node_kv_len_out), _ptr(node_src_path_out),
                                    _ptr(node_src_offset_out), _ptr(num_nodes_out), _ptr(workspace),
                                    ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream))
    if check:
        _check(rc, "ss_build_prefix_tree")
    return rc


class ss_host_step_t(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("dedup_flags", ctypes.c_uint32),
        ("attn", ctypes.c_void_p),
        ("n_paths", ctypes.c_int32), ("n_segments", ctypes.c_int32), ("top_k", ctypes.c_int32),
        ("flags", ctypes.c_uint32),
        ("total_tok", ctypes.c_int64), ("total_q", ctypes.c_int64),
    ] + [(n, ctypes.c_void_p) for n in (
        "tok_ids", "tok_offsets", "ctx_key", "slot_in", "path_leaf_node", "path_q_len", "q_offsets", "q", "scores",
        "seg_offsets", "canon", "path_to_unique", "unique_paths", "multiplicity", "slot_out", "num_unique",
        "u_q_offsets", "out", "lse", "survivors", "keep", "device_status")]


HOST_STEP_INPUTS = ("tok_ids", "tok_offsets", "ctx_key", "slot_in", "path_leaf_node", "path_q_len", "q_offsets", "q",
                    "scores", "seg_offsets")
HOST_STEP_RESULTS = ("canon", "path_to_unique", "unique_paths", "multiplicity", "slot_out", "num_unique",
                     "u_q_offsets", "out", "lse", "survivors", "keep", "device_status")


def make_host_step(attn_desc: "ss_attn_desc_t", *, n_paths, n_segments, top_k, total_tok, total_q, host_in: dict,
                   host_out: dict, dedup_flags=0, flags=0) -> ss_host_step_t:
    """Fills ss_host_step_t from dictionaries of HOST tensors (page-locked for asynchronous copies) keyed by the field
    names.  The returned object keeps references to the descriptor and the tensors."""
    s = ss_host_step_t()
    s.struct_size = ctypes.sizeof(ss_host_step_t)
    s.dedup_flags = dedup_flags
    s.flags = flags
    s.attn = ctypes.addressof(attn_desc)
    s.n_paths, s.n_segments, s.top_k = int(n_paths), int(n_segments), int(top_k)
    s.total_tok, s.total_q = int(total_tok), int(total_q)
    for name in HOST_STEP_INPUTS:
        t = host_in.get(name)
        assert t is None or (not t.is_cuda and t.is_contiguous()), name
        setattr(s, name, t.data_ptr() if t is not None and t.numel() else None)
    for name in HOST_STEP_RESULTS:
        t = host_out.get(name)
        assert t is None or (not t.is_cuda and t.is_contiguous()), name
        setattr(s, name, t.data_ptr() if t is not None and t.numel() else None)
    s._keep = (attn_desc, host_in, host_out)
    return s


def ss_candidate_step_host_arena_bytes(step: ss_host_step_t) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().ss_candidate_step_host_arena_bytes(ctypes.byref(step), ctypes.byref(out)),
           "ss_candidate_step_host_arena_bytes")
    return int(out.value)


def ss_candidate_step_host(step: ss_host_step_t, device_arena: torch.Tensor, stream=None, check=True) -> int:
    """The whole path for host-resident per-step data: copies in, dedup, gather, attention, top-k, copies out; all
    asynchronous on `stream`."""
    rc = lib().ss_candidate_step_host(ctypes.byref(step), _ptr(device_arena),
                                      ctypes.c_size_t(device_arena.numel() * device_arena.element_size()),
                                      _stream(stream))
    if check:
        _check(rc, "ss_candidate_step_host")
    return rc


# ---------------------------------------------------------------------------------------------------------
def make_attn_desc(*, num_q_heads, num_kv_heads, kv_pool=None, k_pool=None, v_pool=None, num_pages=None,
                   kv_page_stride=None, kv_head_stride=None, kv_token_stride=None, node_parent, node_kv_len,
                   node_page_offsets, node_pages, total_node_pages, path_leaf_node, path_q_len, q_offsets, total_q,
                   q, out, lse=None, num_paths=None, num_paths_dev=None, sm_scale=0.0, flags=0, max_depth=0,
                   max_decode_paths=0, head_dim=128, page_size=16, q_src_offsets=None, q_src_rows=0) -> ss_attn_desc_t:
    """Fills the descriptor.  `kv_pool` is the recommended single allocation [page][2][Hkv][16][128]; otherwise
    give k_pool / v_pool tensors and the element strides."""
    d = ss_attn_desc_t()
    d.struct_size = ctypes.sizeof(ss_attn_desc_t)
    d.flags = flags
    d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size = num_q_heads, num_kv_heads, head_dim, page_size
    d.sm_scale = float(sm_scale)
    if kv_pool is not None:
        assert kv_pool.dim() == 5 and kv_pool.is_contiguous() and kv_pool.dtype == torch.bfloat16
        blk = num_kv_heads * page_size * head_dim
        d.k_pool = kv_pool.data_ptr()
        d.v_pool = kv_pool.data_ptr() + blk * 2
        d.num_pages = kv_pool.shape[0]
        d.kv_page_stride, d.kv_head_stride, d.kv_token_stride = 2 * blk, page_size * head_dim, head_dim
    else:
        d.k_pool, d.v_pool = k_pool.data_ptr(), v_pool.data_ptr()
        d.num_pages = num_pages
        d.kv_page_stride, d.kv_head_stride, d.kv_token_stride = kv_page_stride, kv_head_stride, kv_token_stride
    d.num_nodes = int(node_parent.shape[0])
    d.node_parent, d.node_kv_len = node_parent.data_ptr(), node_kv_len.data_ptr()
    d.node_page_offsets, d.node_pages = node_page_offsets.data_ptr(), node_pages.data_ptr()
    d.total_node_pages = int(total_node_pages)
    d.num_paths = int(path_leaf_node.shape[0]) if num_paths is None else int(num_paths)
    d.num_paths_dev = num_paths_dev.data_ptr() if num_paths_dev is not None else None
    d.path_leaf_node, d.path_q_len, d.q_offsets = path_leaf_node.data_ptr(), path_q_len.data_ptr(), q_offsets.data_ptr()
    d.total_q = int(total_q)
    d.max_depth, d.max_decode_paths = int(max_depth), int(max_decode_paths)
    d.q_src_offsets = q_src_offsets.data_ptr() if q_src_offsets is not None else None
    d.q_src_rows = int(q_src_rows)
    d.q = q.data_ptr() if q is not None else None
    d.out = out.data_ptr() if out is not None else None
    d.lse = lse.data_ptr() if lse is not None else None
    return d


def ss_tree_attention_workspace_bytes(desc: ss_attn_desc_t) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().ss_tree_attention_workspace_bytes(ctypes.byref(desc), ctypes.byref(out)),
           "ss_tree_attention_workspace_bytes")
    return int(out.value)


def ss_tree_attention(desc: ss_attn_desc_t, workspace: torch.Tensor, stream=None, check=True) -> int:
    rc = lib().ss_tree_attention(ctypes.byref(desc), _ptr(workspace), ctypes.c_size_t(workspace.numel()),
                                 _stream(stream))
    if check:
        _check(rc, "ss_tree_attention")
    return rc


# ---------------------------------------------------------------------------------------------------------
def ss_topk_workspace_bytes(n_total: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().ss_topk_workspace_bytes(ctypes.c_int32(n_total), ctypes.byref(out)), "ss_topk_workspace_bytes")
    return int(out.value)


def ss_topk_prune(scores, seg_offsets, n_segments, n_total, k, survivors_out, keep_out, workspace, stream=None,
                  check=True) -> int:
    rc = lib().ss_topk_prune(_ptr(scores), _ptr(seg_offsets), ctypes.c_int32(n_segments), ctypes.c_int32(n_total),
                             ctypes.c_int32(k), _ptr(survivors_out), _ptr(keep_out), _ptr(workspace),
                             ctypes.c_size_t(workspace.numel() if workspace is not None else 0), _stream(stream))
    if check:
        _check(rc, "ss_topk_prune")
    return rc


def ss_early_prune(scores, verified, seg_offsets, n_segments, n_total, k, pruned_out, selected_out, final_out,
                   workspace, stream=None, check=True) -> int:
    rc = lib().ss_early_prune(_ptr(scores), _ptr(verified), _ptr(seg_offsets), ctypes.c_int32(n_segments),
                              ctypes.c_int32(n_total), ctypes.c_int32(k), _ptr(pruned_out), _ptr(selected_out),
                              _ptr(final_out), _ptr(workspace),
                              ctypes.c_size_t(workspace.numel() if workspace is not None else 0), _stream(stream))
    if check:
        _check(rc, "ss_early_prune")
    return rc


def ss_branch_sample(logits, draw_offsets, uniforms, n_seq, vocab, temperature, tokens_out, seq_out, stream=None,
                     check=True) -> int:
    rc = lib().ss_branch_sample(_ptr(logits), _ptr(draw_offsets), _ptr(uniforms), ctypes.c_int32(n_seq),
                                ctypes.c_int32(vocab), ctypes.c_float(temperature), _ptr(tokens_out), _ptr(seq_out),
                                _stream(stream))
    if check:
        _check(rc, "ss_branch_sample")
    return rc


def ss_debug_bounded_wait(status_out, stream=None) -> int:
    return lib().ss_debug_bounded_wait(_ptr(status_out), _stream(stream))


def ss_debug_umma_tile(a, b, c, n, k, b_is_mn_major, status_out, stream=None) -> int:
    return lib().ss_debug_umma_tile(_ptr(a), _ptr(b), _ptr(c), ctypes.c_int32(n), ctypes.c_int32(k),
                                    ctypes.c_int32(b_is_mn_major), _ptr(status_out), _stream(stream))


def ss_profile_enable(on: bool) -> None:
    _check(lib().ss_profile_enable(ctypes.c_int32(1 if on else 0)), "ss_profile_enable")


def ss_profile_read():
    """-> ({phase: total ms}, {phase: timed calls}) since the last read."""
    ms = (ctypes.c_float * len(PHASES))()
    calls = (ctypes.c_int64 * len(PHASES))()
    _check(lib().ss_profile_read(ms, calls), "ss_profile_read")
    return {p: float(ms[i]) for i, p in enumerate(PHASES)}, {p: int(calls[i]) for i, p in enumerate(PHASES)}
