"""Transformer-block pipeline over the three C-ABI stages (Section 5, Setup: the linear layers of one block are
quantized from one pass of calibration inputs through that block).

Layers that read the same input share ONE Hessian and ONE factor U: q, k and v all read the block's normalised
hidden state, so a block of six linear layers needs four Hessians and four factorisations, not six.  The schedule
puts the Hessians back to back on one stream (most expensive first), each input group's stage 2 on that group's own
stream as soon as its Hessian is done, and every member layer's stage 3 on its own stream after that; the caller's
stream waits for all of them at the end.  Everything here is stream and buffer plumbing around the binding -- each
stage runs in the CUDA library.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Sequence

import torch

from . import binding as B


@dataclass
class Member:
    name: str
    W: torch.Tensor                      # [R, C] fp16, CUDA
    out: dict = field(default_factory=dict)


@dataclass
class InputGroup:
    name: str
    X: torch.Tensor                      # [tokens, C] bf16, CUDA: the input every member reads
    members: List[Member]


def group_by_shared_input(layers: Sequence, x_of, w_of) -> List[InputGroup]:
    """Groups workload layers (objects with .kind, .block_idx, .C, .name) by the input they read: k and v join the q
    layer of the same block when their input width matches; every other layer is a group of its own.
    x_of(layer) / w_of(layer) produce the device tensors."""
    groups: List[InputGroup] = []
    heads: Dict[tuple, InputGroup] = {}
    for L in layers:
        key = (L.block_idx, L.C)
        if L.kind in ("k", "v") and key in heads:
            heads[key].members.append(Member(L.name, w_of(L)))
            continue
        g = InputGroup(L.name, x_of(L), [Member(L.name, w_of(L))])
        groups.append(g)
        if L.kind == "q":
            heads[key] = g
    return groups


class BlockSolver:
    """Holds the buffers, workspaces and streams of one block and enqueues its solve."""

    def __init__(self, groups: Sequence[InputGroup], bits, group_size=0, sym=False, block=128, damp=0.01, scale_fp16=False,
                 factor=False):
        """factor=True: stages 2 and 3 in the factor form (gptq_prepare_factor / gptq_quantize_layer_factor: same results,
        the factor's inverse is never formed) for the input groups where that is supported and pays."""
        self.bits, self.group_size, self.sym, self.block, self.damp, self.scale_fp16 = bits, group_size, sym, block, damp, scale_fp16
        self.factor_form = factor
        dev = groups[0].X.device
        # most expensive Hessian first: the longest dependency chain starts earliest
        self.groups = sorted(groups, key=lambda g: -(g.X.shape[1] ** 2) * (g.X.shape[0] + g.X.shape[1]))
        self.state = []
        for g in self.groups:
            C, n = g.X.shape[1], g.X.shape[0]
            st = dict(g=g, H=torch.empty((C, C), dtype=torch.float32, device=dev),
                      U=torch.empty((C, C), dtype=torch.float32, device=dev),
                      info=torch.zeros(2, dtype=torch.int32, device=dev),
                      ws=torch.empty(max(256, B.gptq_hessian_workspace_bytes(C, n), B.gptq_prepare_hinv_workspace_bytes(C)),
                                     dtype=torch.uint8, device=dev),
                      stream=torch.cuda.Stream(device=dev), members=[],
                      # the factor form where it pays: the group's members all use the group's one factor
                      factor_form=bool(factor) and B.factor_form_supported(C, block, [group_size]) and
                      B.factor_form_pays(sum(m.W.shape[0] for m in g.members), C, 1))
            for m in g.members:
                R = m.W.shape[0]
                st["members"].append(dict(m=m, stream=torch.cuda.Stream(device=dev),
                                          ws=torch.empty(B.gptq_quantize_workspace_bytes(R, C, bits, group_size, block),
                                                         dtype=torch.uint8, device=dev)))
            self.state.append(st)
        self.main = torch.cuda.Stream(device=dev)

    # the three kinds of stage calls, separately, so that a caller can capture each into a CUDA graph
    def hessian(self, st):
        st["H"].zero_()
        B.gptq_hessian_accumulate(st["H"], st["g"].X, ws=st["ws"])

    def factor(self, st):
        B.gptq_prepare_hinv(st["H"], self.damp, U=st["U"], ws=st["ws"], dev_info=st["info"], factor=st["factor_form"])

    def quantize(self, st, ms):
        ms["m"].out = B.gptq_quantize_layer(ms["m"].W, st["U"], self.bits, self.group_size, self.sym, self.block, ws=ms["ws"],
                                            scale_fp16=self.scale_fp16, factor=st["factor_form"])

    def enqueue(self, run=None):
        """Enqueues the whole block.  `run(key, fn)` may replace the plain call of a stage (e.g. by a CUDA-graph
        replay); keys are ("H", gi), ("U", gi), ("Q", gi, mi).  Returns after making self.main wait for everything."""
        run = run or (lambda key, fn: fn())
        ends = []
        for gi, st in enumerate(self.state):
            with torch.cuda.stream(self.main):
                run(("H", gi), lambda st=st: self.hessian(st))
                h_done = torch.cuda.Event(); h_done.record(self.main)
            with torch.cuda.stream(st["stream"]):
                st["stream"].wait_event(h_done)
                run(("U", gi), lambda st=st: self.factor(st))
                u_done = torch.cuda.Event(); u_done.record(st["stream"])
            for mi, ms in enumerate(st["members"]):
                with torch.cuda.stream(ms["stream"]):
                    ms["stream"].wait_event(u_done)
                    run(("Q", gi, mi), lambda st=st, ms=ms: self.quantize(st, ms))
                    e = torch.cuda.Event(); e.record(ms["stream"]); ends.append(e)
        for e in ends:
            self.main.wait_event(e)

    def stage_calls(self):
        """(key, fn) of every stage call of the block, in enqueue order."""
        out = []
        for gi, st in enumerate(self.state):
            out.append((("H", gi), lambda st=st: self.hessian(st)))
            out.append((("U", gi), lambda st=st: self.factor(st)))
            for mi, ms in enumerate(st["members"]):
                out.append((("Q", gi, mi), lambda st=st, ms=ms: self.quantize(st, ms)))
        return out

    def results(self):
        return {ms["m"].name: ms["m"].out for st in self.state for ms in st["members"]}

    def check(self):
        for st in self.state:
            if st["info"].tolist()[0] != 0:
                raise B.GptqError(st["info"].tolist()[0], f"gptq_prepare_hinv ({st['g'].name})")
            for ms in st["members"]:
                if ms["m"].out and ms["m"].out["dev_info"].tolist()[0] != 0:
                    raise B.GptqError(ms["m"].out["dev_info"].tolist()[0], f"gptq_quantize_layer ({ms['m'].name})")


class HostLayerSolver:
    """Solves a set of independent layers whose weights and calibration activations sit in (pinned) HOST memory: every
    grid of `grids` for every layer, results back in pinned host memory.

    One copy stream carries all activations to the device, the most expensive layer first, in token chunks; on a second
    stream every layer's Hessian is accumulated chunk by chunk as its chunks land (H is a sum over tokens, Section 2), so
    the first Hessian starts after one chunk and the later layers' activations cross while the earlier layers are being
    solved; stages 2 and 3 of a layer run on that layer's own stream as soon as its Hessian is complete (every grid after the
    first on a stream and workspace of its own, beside the first: the grids are independent once the factor exists), and its packed
    codes, scales, zero-points and losses are copied back on that stream.  All layers' activations are resident at once
    (buffers are allocated once, for the shapes given, and reused by every solve()).
    """

    def __init__(self, shapes: Sequence[tuple], grids: Sequence[tuple], block=128, damp=0.01, chunk_bytes=4 << 30, device=None, graphs=True,
                 factor=False):
        """shapes: (R, C, n_tokens) per layer; grids: (bits, group_size, sym) per grid."""
        dev = torch.device("cuda", torch.cuda.current_device()) if device is None else device
        self.grids, self.block, self.damp, self.graphs = list(grids), block, damp, bool(graphs)
        # factor: stages 2 and 3 in the factor form (see BlockSolver) for the layers where it pays
        # graphs: after the first solve(), every layer's stages 2-3 are replayed from a CUDA graph
        # most expensive layer first (Hessian C^2 n, factor ~ C^3, stage 3 ~ 3 R C^2 executed per grid): the layers whose
        # activations cross last are then the cheapest ones, and the solve ends soon after the last copy
        self.order = sorted(range(len(shapes)), key=lambda i: -(shapes[i][1] ** 2) * (shapes[i][2] + shapes[i][1] +
                                                                                   3 * len(self.grids) * shapes[i][0]))
        self.copy_stream = torch.cuda.Stream(device=dev)
        self.main = torch.cuda.Stream(device=dev)
        self.state = []
        for li, (R, C, n) in enumerate(shapes):
            # token chunks of about chunk_bytes.  The layer whose activations cross first starts with short chunks that grow
            # by a quarter each: its Hessian is under way after a few milliseconds, and a chunk's copy never takes longer than
            # the accumulation of the chunk before it as long as accumulating is at least 1.25 x slower than copying (true of
            # the layers this order puts first), so the GPU does not wait for the next chunk
            sizes = []
            if li == self.order[0]:
                b = chunk_bytes / 16
                while b < chunk_bytes:
                    sizes.append(int(b)); b *= 1.25
            sizes.append(chunk_bytes)
            chunks, t0 = [], 0
            while t0 < n:
                cb = sizes[min(len(chunks), len(sizes) - 1)]
                ct = max(64, (cb // (2 * C)) // 64 * 64)
                chunks.append((t0, min(n, t0 + ct)))
                t0 += ct
            ws_bytes = max([256, B.gptq_hessian_workspace_bytes(C, n), B.gptq_prepare_hinv_workspace_bytes(C)] +
                           [B.gptq_quantize_workspace_bytes(R, C, b, g, block) for (b, g, _) in self.grids])
            outs = []
            for (b, g, _) in self.grids:
                G = C // g if g > 0 else 1
                outs.append(dict(qweight=torch.empty((R, C * B.field_bits(b) // 32), dtype=torch.int32).pin_memory(),
                                 scales=torch.empty((R, G), dtype=torch.float32).pin_memory(),
                                 zeros=torch.empty((R, G), dtype=torch.float32).pin_memory(),
                                 loss=torch.empty(1, dtype=torch.float64).pin_memory(),
                                 info=torch.empty(2, dtype=torch.int32).pin_memory()))
            self.state.append(dict(R=R, C=C, n=n, chunks=chunks,
                                   factor=bool(factor) and B.factor_form_pays(R, C, len(self.grids)) and
                                   B.factor_form_supported(C, block, [g for (_, g, _) in self.grids]),
                                   X=torch.empty((n, C), dtype=torch.bfloat16, device=dev),
                                   W=torch.empty((R, C), dtype=torch.float16, device=dev),
                                   H=torch.empty((C, C), dtype=torch.float32, device=dev),
                                   U=torch.empty((C, C), dtype=torch.float32, device=dev),
                                   info_h=torch.zeros((len(chunks), 2), dtype=torch.int32, device=dev),
                                   info_u=torch.zeros(2, dtype=torch.int32, device=dev),
                                   info_host=torch.empty((len(chunks) + 1, 2), dtype=torch.int32).pin_memory(),
                                   ws=torch.empty(ws_bytes, dtype=torch.uint8, device=dev),
                                   stream=torch.cuda.Stream(device=dev), outs=outs,
                                   # a layer's grids are independent once its factor exists: every grid after the first
                                   # has a stream and a stage-3 workspace of its own and runs beside the first
                                   grid_ws=[torch.empty(max(256, B.gptq_quantize_workspace_bytes(R, C, b, g, block)),
                                                        dtype=torch.uint8, device=dev) for (b, g, _) in self.grids[1:]],
                                   grid_streams=[torch.cuda.Stream(device=dev) for _ in self.grids[1:]]))

    def h2d_bytes(self):
        return sum(st["X"].numel() * 2 + st["W"].numel() * 2 for st in self.state)

    def d2h_bytes(self):
        return sum(t.numel() * t.element_size() for st in self.state for o in st["outs"] for t in o.values()) + \
            sum(st["info_host"].numel() * 4 for st in self.state)

    def solve(self, layers: Sequence[tuple]):
        """layers: (W_host [R, C] fp16, X_host [n_tokens, C] bf16) per layer, in the order of `shapes`.  Returns, per
        layer, one dict(qweight, scales, zeros, loss, info) of pinned CPU tensors per grid (reused by the next call).
        Returns when every result is on the host; raises GptqError on a device-side failure."""
        cur = torch.cuda.current_stream()
        start = torch.cuda.Event(); start.record(cur)
        self.copy_stream.wait_event(start); self.main.wait_event(start)
        landed = {}
        with torch.cuda.stream(self.copy_stream):
            for li in self.order:
                st, (Wh, Xh) = self.state[li], layers[li]
                for ci, (t0, t1) in enumerate(st["chunks"]):
                    st["X"][t0:t1].copy_(Xh[t0:t1], non_blocking=True)
                    e = torch.cuda.Event(); e.record(self.copy_stream); landed[(li, ci)] = e
                st["W"].copy_(Wh, non_blocking=True)
                e = torch.cuda.Event(); e.record(self.copy_stream); landed[(li, "W")] = e
        ends = []
        for li in self.order:
            st = self.state[li]
            with torch.cuda.stream(self.main):
                st["H"].zero_()
                for ci, (t0, t1) in enumerate(st["chunks"]):
                    self.main.wait_event(landed[(li, ci)])
                    B.gptq_hessian_accumulate(st["H"], st["X"][t0:t1], ws=st["ws"], dev_info=st["info_h"][ci],
                                              upper_only=ci + 1 < len(st["chunks"]))    # the last chunk mirrors H
                h_done = torch.cuda.Event(); h_done.record(self.main)
            s = st["stream"]
            with torch.cuda.stream(s):
                s.wait_event(h_done); s.wait_event(landed[(li, "W")])
                if st.get("graph") is not None:
                    st["graph"].replay()
                else:
                    self._chain(st, s)
                e = torch.cuda.Event(); e.record(s); ends.append(e)
        for e in ends:
            e.synchronize()
        for li, st in enumerate(self.state):
            for row in st["info_host"].tolist():
                if row[0] != 0:
                    raise B.GptqError(row[0], f"layer {li}: stage 1 / 2 (detail {row[1]})")
            for o in st["outs"]:
                if o["info"].tolist()[0] != 0:
                    raise B.GptqError(o["info"].tolist()[0], f"layer {li}: gptq_quantize_layer")
        if self.graphs and any(st.get("graph") is None for st in self.state):
            self._capture()
        return [st["outs"] for st in self.state]

    def _chain(self, st, s):
        """Stages 2 and 3 of one layer and their results' way back to the host, enqueued on s (the current stream)."""
        B.gptq_prepare_hinv(st["H"], self.damp, U=st["U"], ws=st["ws"], dev_info=st["info_u"], factor=st["factor"])
        st["info_host"][:-1].copy_(st["info_h"], non_blocking=True)
        st["info_host"][-1].copy_(st["info_u"], non_blocking=True)
        fac_done = torch.cuda.Event(); fac_done.record(s)

        def grid(gi, ws):                         # stage 3 for one grid and its results' way back, on the current stream
            (b, g, sym), o = self.grids[gi], st["outs"][gi]
            r = B.gptq_quantize_layer(st["W"], st["U"], b, g, sym, self.block, ws=ws, factor=st["factor"])
            for k, src in (("qweight", r["qweight"]), ("scales", r["scales"]), ("zeros", r["zeros"]), ("loss", r["loss"]),
                           ("info", r["dev_info"])):
                o[k].copy_(src, non_blocking=True)

        joins = []
        for gi, (gs, gws) in enumerate(zip(st["grid_streams"], st["grid_ws"]), start=1):
            with torch.cuda.stream(gs):
                gs.wait_event(fac_done)
                grid(gi, gws)
                joins.append(torch.cuda.Event()); joins[-1].record(gs)
        grid(0, st["ws"])
        for j in joins:
            s.wait_event(j)

    def _capture(self):
        """After the first solve() (which ran eagerly and was checked): every layer's stages 2-3 become one CUDA graph,
        the same kernels on the same buffers, so that later solves issue a few graph launches instead of thousands of
        kernel launches from the host."""
        torch.cuda.synchronize()
        for st in self.state:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st["stream"]):
                self._chain(st, st["stream"])
            st["graph"] = g
        torch.cuda.synchronize()
