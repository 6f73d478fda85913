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

    def __init__(self, groups: Sequence[InputGroup], bits, group_size=0, sym=False, block=128, damp=0.01, scale_fp16=False):
        self.bits, self.group_size, self.sym, self.block, self.damp, self.scale_fp16 = bits, group_size, sym, block, damp, scale_fp16
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
                      stream=torch.cuda.Stream(device=dev), members=[])
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
        B.gptq_prepare_hinv(st["H"], self.damp, U=st["U"], ws=st["ws"], dev_info=st["info"])

    def quantize(self, st, ms):
        ms["m"].out = B.gptq_quantize_layer(ms["m"].W, st["U"], self.bits, self.group_size, self.sym, self.block, ws=ms["ws"],
                                            scale_fp16=self.scale_fp16)

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
