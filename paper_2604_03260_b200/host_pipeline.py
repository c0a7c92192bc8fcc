"""The hot path fed from host memory, pipelined over KV-head groups.

A KV head together with the query heads that share it is an independent unit of the path (no step
exchanges anything between such groups), so a caller whose Q/K/V live in pinned host memory does not
have to copy the whole batch in, compute, and copy the result out in sequence: it can hand the
groups alternately to two CUDA streams, and the copies of one group (in and out) then overlap the
kernels of its neighbour.  This module is that orchestration, written against the same C-ABI calls
(through ``binding``) a C caller would use:

    per KV-head group g, on stream g % 2:
        H2D  Q[g*G:(g+1)*G], K[g], V[g], centroids[g]
        focus_assign (queries), focus_assign (keys), focus_build_tiles, focus_attn_fwd
        D2H  O[g*G:(g+1)*G], lse[g*G:(g+1)*G]

Every group is computed by exactly the kernels of the one-launch path on a shape with Hkv = 1, so
the result is bit-identical to a single call over all heads.  Nothing here does arithmetic.
"""
from __future__ import annotations

import torch

from . import binding as fb


class HostPipeline:
    """Device buffers, per-stream workspaces and the two streams for one workload shape.

    ``Hq, Hkv, n, D, K, topk, window, scale, softcap`` describe the whole layer; ``layout`` is the
    tiles layout to use (``binding.FOCUS_LAYOUT_AUTO`` lets the library choose from the per-group
    shape).  Device memory: one copy of Q, K, V, O, lse, the masks (unless ``allocate`` is False and the
    caller hands its own to ``adopt``) and two tiles workspaces of one KV-head group each."""

    def __init__(self, Hq, Hkv, n, D, K, topk, window, scale=0.0, softcap=0.0, layout=fb.FOCUS_LAYOUT_AUTO, device="cuda",
                 allocate=True):
        assert Hq % Hkv == 0
        self.Hq, self.Hkv, self.G, self.n, self.D = Hq, Hkv, Hq // Hkv, n, D
        self.shape_g = fb.make_shape(self.G, 1, n, D, K, topk, window, scale, softcap)
        self.layout = fb.focus_tiles_layout_of(self.shape_g, layout).layout
        bf, dev = torch.bfloat16, device
        self.streams = [torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)]
        self.ws = [fb.alloc_workspace(self.shape_g, self.layout, device=dev) for _ in self.streams]
        if not allocate:
            return
        self.Q = torch.empty((Hq, n, D), dtype=bf, device=dev)
        self.K = torch.empty((Hkv, n, D), dtype=bf, device=dev)
        self.V = torch.empty((Hkv, n, D), dtype=bf, device=dev)
        self.C = torch.empty((Hkv, K, D), dtype=torch.float32, device=dev)
        self.O = torch.empty((Hq, n, D), dtype=bf, device=dev)
        self.lse = torch.empty((Hq, n), dtype=torch.float32, device=dev)
        self.mq = torch.empty((Hq, n), dtype=torch.int32, device=dev)
        self.mk = torch.empty((Hkv, n), dtype=torch.int32, device=dev)
        self.near = torch.zeros(1, dtype=torch.int64, device=dev)
        self.status = torch.zeros(4, dtype=torch.int32, device=dev)

    def adopt(self, Q, K, V, C, O, lse, mq, mk, near, status):
        """Use the caller's device buffers instead of the ones allocated by the constructor."""
        self.Q, self.K, self.V, self.C, self.O, self.lse = Q, K, V, C, O, lse
        self.mq, self.mk, self.near, self.status = mq, mk, near, status
        return self

    def h2d_bytes(self):
        return sum(x.numel() * x.element_size() for x in (self.Q, self.K, self.V, self.C))

    def d2h_bytes(self):
        return sum(x.numel() * x.element_size() for x in (self.O, self.lse))

    def run(self, hQ, hK, hV, hC, hO, hL):
        """One pass: pinned host tensors in (Q [Hq,n,D], K/V [Hkv,n,D] bf16, centroids [Hkv,K,D] fp32), pinned host
        tensors out (O bf16 [Hq,n,D], lse fp32 [Hq,n]).  Enqueues everything and makes the current stream wait for
        both pipeline streams; it does not synchronise the host.  Afterwards ``status[0]`` must read 0 and ``near``
        (an int64 word: the near-tie count, bit 63 = fault flag of focus_assign) must not be negative."""
        G = self.G
        start = torch.cuda.Event()
        start.record()
        for st in self.streams:
            st.wait_event(start)
        for g in range(self.Hkv):
            st = self.streams[g % 2]
            qs, ks = slice(g * G, (g + 1) * G), slice(g, g + 1)
            with torch.cuda.stream(st):
                self.Q[qs].copy_(hQ[qs], non_blocking=True)
                self.K[ks].copy_(hK[ks], non_blocking=True)
                self.V[ks].copy_(hV[ks], non_blocking=True)
                self.C[ks].copy_(hC[ks], non_blocking=True)
                fb.focus_assign(self.shape_g, self.Q[qs], G, self.C[ks], self.mq[qs], self.near, stream=st)
                fb.focus_assign(self.shape_g, self.K[ks], 1, self.C[ks], self.mk[ks], self.near, stream=st)
                fb.focus_build_tiles(self.shape_g, self.mq[qs], self.mk[ks], self.layout, self.ws[g % 2], stream=st)
                fb.focus_attn_fwd(self.shape_g, self.Q[qs], self.K[ks], self.V[ks], self.mq[qs], self.mk[ks], self.ws[g % 2],
                                  self.layout, self.O[qs], self.lse[qs], self.status, stream=st)
                hO[qs].copy_(self.O[qs], non_blocking=True)
                hL[qs].copy_(self.lse[qs], non_blocking=True)
        for st in self.streams:
            done = torch.cuda.Event()
            done.record(st)
            torch.cuda.current_stream().wait_event(done)
