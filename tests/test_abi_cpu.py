"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and its pure host entry points
(workspace queries, argument validation that happens before any CUDA call) behave."""
import ctypes
import os
import re

import pytest

from paper_2609_39334_b200 import binding as B
from paper_2609_39334_b200 import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    cuda_build.build()
    return B.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "specscale.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ss_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert "ss_dedup_paths" in names and "ss_tree_attention" in names and "ss_topk_prune" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == names


def test_status_strings(lib):
    seen = {B.status_string(i) for i in range(7)}
    assert len(seen) == 7 and B.status_string(0) == "ok"
    assert B.status_string(99) == "unknown status"


def test_workspace_queries(lib):
    assert B.ss_dedup_workspace_bytes(0) > 0
    a, b = B.ss_dedup_workspace_bytes(1000), B.ss_dedup_workspace_bytes(100000)
    assert a < b and a % 256 == 0
    assert B.ss_topk_workspace_bytes(16384) >= 2 * 16384 * 8
    out = ctypes.c_size_t(0)
    assert lib.ss_dedup_workspace_bytes(ctypes.c_int32(-1), ctypes.byref(out)) == B.SS_ERR_INVALID_ARG
    assert lib.ss_topk_workspace_bytes(ctypes.c_int32(5), None) == B.SS_ERR_INVALID_ARG


def _desc(**kw):
    d = B.ss_attn_desc_t()
    d.struct_size = ctypes.sizeof(B.ss_attn_desc_t)
    d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size = 12, 2, 128, 16
    d.kv_page_stride, d.kv_head_stride, d.kv_token_stride = 2 * 2 * 2048, 2048, 128
    d.num_nodes, d.num_paths, d.total_q, d.total_node_pages, d.num_pages = 10, 8, 8, 100, 100
    for k, v in kw.items():
        setattr(d, k, v)
    return d


def test_attention_descriptor_validation_on_host(lib):
    assert B.ss_tree_attention_workspace_bytes(_desc()) > 0
    small = B.ss_tree_attention_workspace_bytes(_desc(max_depth=2, max_decode_paths=8))
    assert small <= B.ss_tree_attention_workspace_bytes(_desc())
    out = ctypes.c_size_t(0)
    q = lambda d: lib.ss_tree_attention_workspace_bytes(ctypes.byref(d), ctypes.byref(out))
    assert q(_desc(struct_size=8)) == B.SS_ERR_INVALID_ARG
    assert q(_desc(head_dim=64)) == B.SS_ERR_UNSUPPORTED
    assert q(_desc(page_size=32)) == B.SS_ERR_UNSUPPORTED
    assert q(_desc(num_q_heads=13)) == B.SS_ERR_UNSUPPORTED
    assert q(_desc(kv_token_stride=256)) == B.SS_ERR_UNSUPPORTED
    assert q(_desc(max_depth=17)) == B.SS_ERR_UNSUPPORTED
    assert q(_desc(num_paths=-1)) == B.SS_ERR_INVALID_ARG
    assert q(_desc(flags=0x100)) == B.SS_ERR_INVALID_ARG
    # the call itself rejects a null workspace before touching CUDA
    assert lib.ss_tree_attention(ctypes.byref(_desc()), None, ctypes.c_size_t(0), None) == B.SS_ERR_INVALID_ARG


def test_attention_rejects_an_output_that_is_not_32_byte_aligned(lib):
    """The tile kernel writes whole 32-byte sectors of `out`; a pointer that is only 16-byte aligned is refused on the
    host, before anything is launched (the pointers below are never dereferenced)."""
    ok = 1 << 20
    d = _desc(k_pool=ok, v_pool=ok, node_parent=ok, node_kv_len=ok, node_page_offsets=ok, node_pages=ok,
              path_leaf_node=ok, path_q_len=ok, q_offsets=ok, q=ok, out=ok + 16)
    before = B.ss_launch_count()
    ws = ctypes.c_void_p(1 << 21)
    assert lib.ss_tree_attention(ctypes.byref(d), ws, ctypes.c_size_t(1 << 30), None) == B.SS_ERR_UNSUPPORTED
    assert B.ss_launch_count() == before


def test_dedup_and_topk_argument_validation_on_host(lib):
    null = ctypes.c_void_p(0)
    one = ctypes.c_void_p(256)     # never dereferenced: validation fails first
    rc = lib.ss_dedup_paths(null, null, null, null, ctypes.c_int32(-1), ctypes.c_uint32(0), null, null, null, null,
                            null, one, null, ctypes.c_size_t(0), null)
    assert rc == B.SS_ERR_INVALID_ARG
    rc = lib.ss_dedup_paths(one, one, null, one, ctypes.c_int32(4), ctypes.c_uint32(0), one, one, one, one,
                            null, one, one, ctypes.c_size_t(1 << 20), null)
    assert rc == B.SS_ERR_INVALID_ARG          # slot_in without slot_out
    rc = lib.ss_dedup_paths(one, one, null, null, ctypes.c_int32(4), ctypes.c_uint32(0), one, one, one, one,
                            null, one, one, ctypes.c_size_t(16), null)
    assert rc == B.SS_ERR_WORKSPACE_TOO_SMALL
    rc = lib.ss_topk_prune(one, one, ctypes.c_int32(2), ctypes.c_int32(10), ctypes.c_int32(0), one, one, one,
                           ctypes.c_size_t(1 << 20), null)
    assert rc == B.SS_ERR_INVALID_ARG          # k < 1
    rc = lib.ss_topk_prune(one, one, ctypes.c_int32(2), ctypes.c_int32(10), ctypes.c_int32(3), one, one, one,
                           ctypes.c_size_t(8), null)
    assert rc == B.SS_ERR_WORKSPACE_TOO_SMALL


def test_binding_fails_loudly_without_library(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/libspecscale.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.lib()


def test_every_kernel_waits_for_its_predecessor_first():
    """Kernels are launched with programmatic stream serialization; stream order then rests on every kernel calling
    grid_dependency_enter() before anything else (a kernel that skipped it could finish before its predecessor)."""
    import glob
    import re
    csrc = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2609_39334_b200", "csrc")
    n = 0
    for path in sorted(glob.glob(os.path.join(csrc, "*.cu"))):
        src = open(path).read()
        for m in re.finditer(r"__global__[^;{]*\{", src):
            n += 1
            rest = src[m.end():].lstrip()
            # (the leaf kernel that overlaps the tile kernel releases first and waits later, before it reads the tile
            #  kernel's results and before it ends: see grid_dependency_wait in common.cuh)
            ok = rest.startswith("ss::grid_dependency_enter();") or rest.startswith("ss::grid_dependency_enter_then_release();")
            if not ok and "leaf_stream_kernel" in m.group(0):
                body = rest[:rest.index("\n}\n")] if "\n}\n" in rest else rest
                ok = "ss::grid_dependency_release();" in rest[:600] and rest.count("ss::grid_dependency_wait();") >= 3
            if not ok and "tile_items_umma_split_kernel" in m.group(0):
                # block-local setup first (barriers, zeroed buffers, tensor memory), then the wait - before anything of
                # the plan is read
                body = rest[:rest.index("\n}\n")] if "\n}\n" in rest else rest
                at = body.find("ss::grid_dependency_enter_then_release();")
                first_plan_read = min(x for x in (body.find("P.hdr"), body.find("P.tile_items"), len(body)) if x >= 0)
                ok = 0 <= at < first_plan_read
            assert ok, (os.path.basename(path), m.group(0)[:80])
        assert "<<<" not in src, path            # every launch goes through the counting macro
    assert n >= 20
