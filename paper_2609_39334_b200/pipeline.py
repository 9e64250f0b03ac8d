"""Device-side plumbing around the three C-ABI calls: uploads a synthetic workload, owns the output and
workspace tensors, and runs   ss_dedup_paths -> ss_gather_unique_paths -> ss_tree_attention -> ss_topk_prune.

Only memory management and argument marshalling happen here: every step is a library call.  The query rows are not
moved by the gather: the attention call reads them in place through `q_src_offsets`.
"""
from __future__ import annotations

from typing import Dict

import numpy as np
import torch

from . import binding as B
from .synth import TreeWorkload


def _dev(a: np.ndarray, device, dtype=None) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.to(device)


class DevicePipeline:
    """Holds one workload on the GPU together with every buffer the three calls need (no allocation per step)."""

    def __init__(self, w: TreeWorkload, device="cuda:0", attn_flags: int = 0, dedup_flags: int = 0,
                 sm_scale: float = 0.0):
        self.w = w
        self.device = torch.device(device)
        dev = self.device
        self.attn_flags, self.dedup_flags, self.sm_scale = attn_flags, dedup_flags, sm_scale
        N = w.num_paths
        self.N = N
        # ---- resident state: tree + KV pool ------------------------------------------------------------------
        self.kv_pool = w.kv_pool.to(dev) if w.kv_pool.device != dev else w.kv_pool
        self.node_parent = _dev(w.node_parent, dev)
        self.node_kv_len = _dev(w.node_kv_len, dev)
        self.node_page_offsets = _dev(w.node_page_offsets, dev)
        self.node_pages = _dev(w.node_pages if w.node_pages.size else np.zeros(1, np.int32), dev)
        # ---- per-step inputs (logical candidates) ----------------------------------------------------------
        self.tok_ids = _dev(w.tok_ids if w.tok_ids.size else np.zeros(1, np.int32), dev)
        self.tok_offsets = _dev(w.tok_offsets, dev)
        self.ctx_key = _dev(w.ctx_key, dev)
        self.slot_in = _dev(w.slot_in, dev)
        self.path_leaf_node = _dev(w.path_leaf_node, dev)
        self.path_q_len = _dev(w.path_q_len, dev)
        self.q_offsets = _dev(w.q_offsets, dev)
        self.q = w.q.to(dev) if w.q.device != dev else w.q
        self.scores = _dev(w.scores, dev)
        self.seg_offsets = _dev(w.seg_offsets, dev)
        # ---- dedup outputs ----------------------------------------------------------------------------------------
        i32 = dict(dtype=torch.int32, device=dev)
        self.canon = torch.empty(max(N, 1), **i32)
        self.path_to_unique = torch.empty(max(N, 1), **i32)
        self.unique_paths = torch.empty(max(N, 1), **i32)
        self.multiplicity = torch.empty(max(N, 1), **i32)
        self.slot_out = torch.empty(max(N, 1), **i32)
        self.num_unique = torch.zeros(1, **i32)
        self.dedup_ws = B.alloc_workspace(B.ss_dedup_workspace_bytes(N), dev)
        # ---- compacted (unique-path) descriptor arrays; capacity N ---------------------------------------------
        self.u_leaf = torch.empty(max(N, 1), **i32)
        self.u_q_len = torch.empty(max(N, 1), **i32)
        self.u_q_offsets = torch.zeros(N + 1, dtype=torch.int64, device=dev)
        total_q = w.total_q
        self.u_q_src = torch.zeros(max(N, 1), dtype=torch.int64, device=dev)
        self.out = torch.empty((max(total_q, 1), w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
        self.lse = torch.empty((max(total_q, 1), w.num_q_heads), dtype=torch.float32, device=dev)
        depth = self._max_depth(w)
        self.desc = B.make_attn_desc(
            num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads, kv_pool=self.kv_pool,
            node_parent=self.node_parent, node_kv_len=self.node_kv_len, node_page_offsets=self.node_page_offsets,
            node_pages=self.node_pages, total_node_pages=int(w.node_page_offsets[-1]),
            path_leaf_node=self.u_leaf, path_q_len=self.u_q_len, q_offsets=self.u_q_offsets, total_q=total_q,
            q=self.q, q_src_offsets=self.u_q_src, q_src_rows=total_q, out=self.out, lse=self.lse, num_paths=N,
            num_paths_dev=self.num_unique,
            sm_scale=sm_scale, flags=attn_flags, max_depth=depth,
            max_decode_paths=int((w.path_q_len == 1).sum()))
        self.attn_ws = B.alloc_workspace(B.ss_tree_attention_workspace_bytes(self.desc), dev)
        # ---- top-k -----------------------------------------------------------------------------------------------
        self.P = int(w.seg_offsets.shape[0]) - 1
        self.survivors = torch.empty((max(self.P, 1), w.top_k), **i32)
        self.keep = torch.empty(max(N, 1), dtype=torch.uint8, device=dev)
        self.topk_ws = B.alloc_workspace(B.ss_topk_workspace_bytes(N), dev)

    @staticmethod
    def _max_depth(w: TreeWorkload) -> int:
        depth = np.zeros(w.num_nodes, np.int32)
        for n in range(w.num_nodes):          # parents come first
            p = int(w.node_parent[n])
            depth[n] = 1 if p < 0 else depth[p] + 1
        return int(depth.max()) if w.num_nodes else 1

    # ------------------------------------------------------------------------------------------------------------
    def dedup(self, stream=None):
        B.ss_dedup_paths(self.tok_ids, self.tok_offsets, self.ctx_key, self.slot_in, self.N, self.dedup_flags,
                         self.canon, self.path_to_unique, self.unique_paths, self.multiplicity, self.slot_out,
                         self.num_unique, self.dedup_ws, stream=stream)

    def compact_unique(self, stream=None):
        """Descriptor rows of the unique paths (ss_gather_unique_paths; device-side, no host sync: entries past the
        live count U are inert and ignored by the attention call).  Query rows stay where they are."""
        B.ss_gather_unique_paths(self.unique_paths, self.num_unique, self.N, self.path_leaf_node, self.path_q_len,
                                 self.q_offsets, self.u_leaf, self.u_q_len, self.u_q_offsets, self.u_q_src,
                                 stream=stream)

    def attention(self, stream=None):
        B.ss_tree_attention(self.desc, self.attn_ws, stream=stream)

    def topk(self, stream=None):
        B.ss_topk_prune(self.scores, self.seg_offsets, self.P, self.N, self.w.top_k, self.survivors, self.keep,
                        self.topk_ws, stream=stream)

    def step(self):
        """One pass of the whole hot path."""
        self.dedup()
        self.compact_unique()
        self.attention()
        self.topk()

    # ------------------------------------------------------------------------------------------------------------
    def results(self) -> Dict[str, np.ndarray]:
        torch.cuda.synchronize(self.device)
        st = B.ss_last_device_status(self.attn_ws)
        if st != B.SS_OK:
            raise B.SpecScaleError(st, "ss_tree_attention (device status)")
        U = int(self.num_unique.item())
        N = self.N
        tq = int(self.u_q_offsets[U].item()) if N else 0
        return dict(
            num_unique=U, canon=self.canon[:N].cpu().numpy(), path_to_unique=self.path_to_unique[:N].cpu().numpy(),
            unique_paths=self.unique_paths[:U].cpu().numpy(), multiplicity=self.multiplicity[:U].cpu().numpy(),
            slot_out=self.slot_out[:N].cpu().numpy(), total_q=tq,
            out=self.out[:tq].to(torch.float64).cpu().numpy(), lse=self.lse[:tq].to(torch.float64).cpu().numpy(),
            survivors=self.survivors[:self.P].cpu().numpy(), keep=self.keep[:N].cpu().numpy())


class HostStepPipeline:
    """`depth` independent (page-locked host buffers, device arena, stream) sets around ss_candidate_step_host, for a
    caller whose per-step data lives in host memory.  The tree and the KV pool are those of `resident` (they stay on
    the device).  submit(i) enqueues one whole step on set i and returns at once; alternating the sets overlaps the
    copies of one step with the kernels of another."""

    def __init__(self, resident: DevicePipeline, depth: int = 2, compact: bool = False):
        self.resident = resident
        self.compact = compact
        w, dev = resident.w, resident.device
        self.device = dev
        N, P, k = w.num_paths, resident.P, w.top_k
        Hq, D = w.num_q_heads, w.head_dim
        tq = w.total_q

        def pin(shape, dtype):
            return torch.empty(shape, dtype=dtype, pin_memory=True)

        def pin_like(a, dtype=None):
            t = a if isinstance(a, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(a))
            out = pin(tuple(t.shape), dtype or t.dtype)
            out.copy_(t)
            return out

        self.sets = []
        for _ in range(depth):
            h_in = dict(
                tok_ids=pin_like(w.tok_ids), tok_offsets=pin_like(w.tok_offsets, torch.int64),
                ctx_key=pin_like(w.ctx_key, torch.int64), slot_in=pin_like(w.slot_in, torch.int32),
                path_leaf_node=pin_like(w.path_leaf_node, torch.int32), path_q_len=pin_like(w.path_q_len, torch.int32),
                q_offsets=pin_like(w.q_offsets, torch.int64), q=pin_like(w.q),
                scores=pin_like(w.scores, torch.float32), seg_offsets=pin_like(w.seg_offsets, torch.int32))
            h_out = dict(
                canon=pin((max(N, 1),), torch.int32), path_to_unique=pin((max(N, 1),), torch.int32),
                unique_paths=pin((max(N, 1),), torch.int32), multiplicity=pin((max(N, 1),), torch.int32),
                slot_out=pin((max(N, 1),), torch.int32), num_unique=pin((1,), torch.int32),
                u_q_offsets=pin((N + 1,), torch.int64), out=pin((max(tq, 1), Hq, D), torch.bfloat16),
                lse=pin((max(tq, 1), Hq), torch.float32), survivors=pin((max(P, 1), k), torch.int32),
                keep=pin((max(N, 1),), torch.uint8), device_status=pin((1,), torch.int32))
            step = B.make_host_step(resident.desc, n_paths=N, n_segments=P, top_k=k,
                                    total_tok=int(w.tok_offsets[-1]), total_q=tq, host_in=h_in, host_out=h_out,
                                    dedup_flags=resident.dedup_flags,
                                    flags=B.SS_STEP_COMPACT_TRANSFERS if compact else 0)
            arena = B.alloc_workspace(B.ss_candidate_step_host_arena_bytes(step), dev)
            self.sets.append(dict(h_in=h_in, h_out=h_out, step=step, arena=arena, stream=torch.cuda.Stream(dev)))
        self.h2d_bytes = sum(t.numel() * t.element_size() for t in self.sets[0]["h_in"].values())
        self.d2h_bytes = sum(t.numel() * t.element_size() for t in self.sets[0]["h_out"].values())

    def measure_traffic(self):
        """Runs one step on set 0 and sets d2h_bytes to what that step moved back over the bus.  With
        SS_STEP_COMPACT_TRANSFERS (and page-locked, hence mapped, buffers) only the live rows of out / lse come back;
        that it happened is read off a sentinel row past the live ones (left untouched if so)."""
        s = self.sets[0]
        o, i = s["h_out"], s["h_in"]
        tq_all = o["out"].shape[0]
        o["out"][tq_all - 1].fill_(-7.0)
        self.submit(0)
        s["stream"].synchronize()
        U = int(o["num_unique"][0])
        tq_live = int(o["u_q_offsets"][U]) if self.resident.N else 0
        compact = tq_live < tq_all and bool((o["out"][tq_all - 1].float() == -7.0).all())
        if compact:
            row = o["out"].shape[1] * o["out"].shape[2] * 2
            small_out = sum(t.numel() * t.element_size() for k, t in o.items() if k not in ("out", "lse"))
            self.d2h_bytes = small_out + tq_live * (row + o["lse"].shape[1] * 4)
        return compact

    def submit(self, i: int):
        s = self.sets[i % len(self.sets)]
        B.ss_candidate_step_host(s["step"], s["arena"], stream=s["stream"])

    def synchronize(self):
        for s in self.sets:
            s["stream"].synchronize()

    def results(self, i: int) -> Dict[str, np.ndarray]:
        s = self.sets[i % len(self.sets)]
        s["stream"].synchronize()
        o = s["h_out"]
        st = int(o["device_status"][0])
        if st != B.SS_OK:
            raise B.SpecScaleError(st, "ss_candidate_step_host (device status)")
        N, P = self.resident.N, self.resident.P
        U = int(o["num_unique"][0])
        tq = int(o["u_q_offsets"][U]) if N else 0
        return dict(
            num_unique=U, canon=o["canon"][:N].numpy().copy(), path_to_unique=o["path_to_unique"][:N].numpy().copy(),
            unique_paths=o["unique_paths"][:U].numpy().copy(), multiplicity=o["multiplicity"][:U].numpy().copy(),
            slot_out=o["slot_out"][:N].numpy().copy(), total_q=tq,
            out=o["out"][:tq].to(torch.float64).numpy(), lse=o["lse"][:tq].to(torch.float64).numpy(),
            survivors=o["survivors"][:P].numpy().copy(), keep=o["keep"][:N].numpy().copy())
