"""Decoding rounds of several micro-batches on streams of their own.

One decoding round is draft -> build the tree -> verify -> walk, each step waiting for the one before it; the
conclusion of the paper names the idle time this leaves as future work.  Nothing in one sequence's round can
overlap, but the rounds of different sequences are independent, so the batch is split into micro-batches, each with
its own library context (scratch memory) and CUDA stream: while the target model verifies one micro-batch, the tree
builder of another runs, and the tree kernel, which keeps fewer CTAs than the GPU has SMs, shares the GPU with the
verifier's kernels.  This module only orders the calls; every step still runs in the library's kernels (the
verifier is the caller's).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Sequence

import torch

from .binding import Graft, TreeOut


@dataclass
class MicroBatch:
    """A context, its stream and the buffers one micro-batch's rounds write."""
    graft: Graft
    batch: int
    L: int
    stream: torch.cuda.Stream = None
    out: TreeOut = None
    accept_len: torch.Tensor = None
    accept_path: torch.Tensor = None
    bonus_token: torch.Tensor = None
    rounds_done: int = field(default=0)

    def __post_init__(self):
        dev = torch.device("cuda", torch.cuda.current_device())
        if self.stream is None:
            self.stream = torch.cuda.Stream(device=dev)
        if self.out is None:
            self.out = self.graft.alloc_out(self.batch)
        i32 = torch.int32
        if self.accept_len is None:
            self.accept_len = torch.empty(self.batch, dtype=i32, device=dev)
        if self.accept_path is None:
            self.accept_path = torch.empty((self.batch, self.L), dtype=i32, device=dev)
        if self.bonus_token is None:
            self.bonus_token = torch.empty(self.batch, dtype=i32, device=dev)


# draft(mb_index, round) -> dict(logits, hidden, root_token, hist, prefix_len, fixed_budget) of device tensors
DraftFn = Callable[[int, int], dict]
# verify(mb_index, round, tree_out) -> target_next [batch, n_max] int32 device tensor, enqueued on the current stream
VerifyFn = Callable[[int, int, TreeOut], torch.Tensor]


def run_rounds(micro: Sequence[MicroBatch], n_rounds: int, draft: DraftFn, verify: VerifyFn, overlap: bool = True,
               after_round: Callable[[int, int, MicroBatch], None] | None = None) -> None:
    """Enqueue `n_rounds` rounds of every micro-batch.

    overlap=True: micro-batch i runs on micro[i].stream, so its build overlaps the others' verification.
    overlap=False: the same calls in the same order on the current stream (the sequential schedule).
    `draft` and `verify` are called with the micro-batch's stream current and must enqueue their work there.
    `after_round` (optional) is called after a micro-batch's walk was enqueued, e.g. to copy results aside.
    The streams first wait for the work already enqueued on the current stream; the caller joins them with
    `join(micro)` (or synchronises) before it reads the results.
    """
    cur = torch.cuda.current_stream()
    if overlap:
        for mb in micro:
            mb.stream.wait_stream(cur)
    for r in range(n_rounds):
        for i, mb in enumerate(micro):
            with torch.cuda.stream(mb.stream if overlap else cur):
                x = draft(i, r)
                mb.graft.build_trees(x["logits"], x.get("hidden"), x["root_token"], x.get("hist"),
                                     x.get("prefix_len"), x.get("fixed_budget"), mb.out)
                tn = verify(i, r, mb.out)
                mb.graft.accept(mb.out, tn, mb.accept_len, mb.accept_path, mb.bonus_token)
                mb.rounds_done += 1
                if after_round is not None:
                    after_round(i, r, mb)


def join(micro: Sequence[MicroBatch]) -> None:
    """Make the current stream wait for every micro-batch's stream."""
    cur = torch.cuda.current_stream()
    for mb in micro:
        cur.wait_stream(mb.stream)
