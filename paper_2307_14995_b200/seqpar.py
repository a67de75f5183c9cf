"""Sequence parallelism: one long sequence cut into consecutive chunks, one chunk per GPU of a node.

Only the d x e state of the recurrence (Algorithm 2) crosses a cut, so a rank needs from the others nothing but their
[B,H,d,e] fp32 state contributions -- one all-gather per direction (a few MB over NVLink, bound by latency, not by
bandwidth), after which every rank chains the contributions of the ranks before it (forward) or after it (backward)
into the state at its own cut and runs the ordinary forward / backward pass on its chunk with that state.  The
results are those of the whole sequence on one device.

    forward, rank r:   S_r  = la_chunk_state(k, v)            own contribution, needs no one else
                       all-gather S
                       kv_in_r = la_chain_states(S, chunk=r)   lambda^(n_j)-weighted chain over j < r
                       o_r  = la_fwd(q, k, v, kv_in = kv_in_r)
    backward, rank r:  E_r  = la_chunk_state(q, dO, reverse)
                       all-gather E
                       g_r  = la_chain_states(E, chunk=r, reverse)   chain over j > r
                       dq, dk, dv = la_bwd(..., kv_in = kv_in_r, grad_kv_out = g_r)

Every arithmetic step runs in the library's kernels; this module only allocates, calls and gathers.  The gather goes
through torch.distributed (NCCL on GPUs): the contributions land in this rank's own memory first and the kernels
read only local memory.  The three phases of each direction are separate methods so that a single process can also
drive several emulated ranks one after the other (no kernel ever waits for another rank's kernel).
"""
from __future__ import annotations

from typing import Callable, Optional

import torch
import torch.distributed as dist

from . import binding as la


def dist_gather(group=None) -> Callable[[torch.Tensor, torch.Tensor], None]:
    """gather(dst[R, ...], src[...]) through torch.distributed."""

    def gather(dst: torch.Tensor, src: torch.Tensor) -> None:
        # views of dst, rank-major: the contributions land directly in the gathered tensor
        dist.all_gather(list(dst.unbind(0)), src, group=group)

    return gather


class SequenceParallel:
    """One rank's share of a sequence of `total_tokens` tokens cut into chunks of `chunk_tokens` (the last shorter)."""

    def __init__(self, rank: int, world: int, total_tokens: int, chunk_tokens: int, B: int, H: int, d: int, e: int,
                 lam, *, in_dtype=torch.bfloat16, out_dtype=torch.float32, layout=la.LA_LAYOUT_BHND, device=None,
                 gather: Optional[Callable] = None, api=la):
        if world < 1 or not (0 <= rank < world):
            raise ValueError("bad rank / world")
        if chunk_tokens < 1 or (total_tokens + chunk_tokens - 1) // chunk_tokens != world:
            raise ValueError("the chunks must cover the sequence with exactly one chunk per rank")
        self.rank, self.world = rank, world
        self.total, self.chunk = int(total_tokens), int(chunk_tokens)
        self.n_local = min(self.total, (rank + 1) * self.chunk) - rank * self.chunk
        self.lam = lam
        self.api = api
        self.device = device
        self.gather = gather if gather is not None else dist_gather()
        self.shape = api.make_shape(B, H, self.n_local, d, e, in_dtype, out_dtype, layout=layout)
        state = (B, H, d, e)
        new = lambda *s: torch.empty(s, dtype=torch.float32, device=device)
        self.local = new(*state)                 # this rank's contribution (either direction)
        self.gathered = new(world, *state)       # everybody's, rank-major
        self.kv_in = new(*state)                 # state entering this chunk (kept for the backward pass)
        self.gko = new(*state)                   # state gradient entering this chunk from the right
        nbytes = lambda n: torch.empty(max(int(n), 256), dtype=torch.uint8, device=device)
        self.ws_state = nbytes(api.chunk_state_workspace_bytes(self.shape))
        self.ws_fwd = nbytes(api.workspace_bytes(api.LA_OP_FWD, self.shape))
        self.ws_bwd = nbytes(api.workspace_bytes(api.LA_OP_BWD, self.shape))

    # ---- forward --------------------------------------------------------------------------------------------
    def fwd_local(self, k, v):
        self.api.la_chunk_state(self.shape, 0, k, v, self.lam, self.local, self.ws_state)

    def fwd_exchange(self):
        self.gather(self.gathered, self.local)

    def fwd_finish(self, q, k, v, o, kv_in=None, kv_out=None):
        """kv_in / kv_out: the state before the first and after the last token of the WHOLE sequence (any rank may ask)."""
        a = self.api
        a.la_chain_states(self.shape, self.total, self.chunk, 0, self.gathered, self.world, self.rank, kv_in, self.lam,
                          self.kv_in)
        a.la_fwd(self.shape, q, k, v, self.lam, o, self.kv_in, None, self.ws_fwd)
        if kv_out is not None:
            a.la_chain_states(self.shape, self.total, self.chunk, 0, self.gathered, self.world, self.world, kv_in,
                              self.lam, kv_out)

    def fwd(self, q, k, v, o, kv_in=None, kv_out=None):
        self.fwd_local(k, v)
        self.fwd_exchange()
        self.fwd_finish(q, k, v, o, kv_in, kv_out)

    # ---- backward (after fwd on the same inputs: it reuses the state entering the chunk) -----------------------
    def bwd_local(self, q, do):
        self.api.la_chunk_state(self.shape, 1, q, do, self.lam, self.local, self.ws_state)

    def bwd_exchange(self):
        self.gather(self.gathered, self.local)

    def bwd_finish(self, q, k, v, do, dq, dk, dv, grad_kv_out=None, grad_kv_in=None):
        a = self.api
        a.la_chain_states(self.shape, self.total, self.chunk, 1, self.gathered, self.world, self.rank, grad_kv_out,
                          self.lam, self.gko)
        a.la_bwd(self.shape, q, k, v, do, self.lam, dq, dk, dv, self.kv_in, self.gko, None, self.ws_bwd)
        if grad_kv_in is not None:
            a.la_chain_states(self.shape, self.total, self.chunk, 1, self.gathered, self.world, -1, grad_kv_out,
                              self.lam, grad_kv_in)

    def bwd(self, q, k, v, do, dq, dk, dv, grad_kv_out=None, grad_kv_in=None):
        self.bwd_local(q, do)
        self.bwd_exchange()
        self.bwd_finish(q, k, v, do, dq, dk, dv, grad_kv_out, grad_kv_in)
