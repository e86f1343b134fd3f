"""Expert-parallel exchange of the capacity-bounded buffers (the setting of the paper's efficiency
section: experts spread over ranks, token rows crossing in one All-to-All each way, whose size is
bounded by the expert capacity C, which is why a smaller C means less traffic).

Partition over W ranks of one process group: rank q owns the experts [q*E_local, (q+1)*E_local) with
their weights, and the tokens [q*T_local, (q+1)*T_local) of the batch (global token id = rank *
T_local + local id).  Expert choice is a selection over ALL tokens of the batch, so the path is

  1. affinities of the local tokens against all E experts                     (local, S1)
  2. `exchange_affinities`: every rank receives the columns of its experts for all T tokens
     (T_local * E_local floats per pair of ranks), and the batch maximum is all-reduced
  3. selection for the local experts over all T tokens                        (local, S3 with E = E_local)
  4. `build_plan`: the owners tell the token holders which rows they want (token ids and gates)
  5. `dispatch_rows`: token rows travel to the experts' buffers, at most E_local * C rows per rank
  6. expert FFN on the local experts                                          (local, S5)
  7. `return_rows` + `combine_local`: output rows travel back, each token sums its rows in ascending
     expert order, which is ascending (rank, row) order, so the result is deterministic       (S6)
The backward pass uses the same two row exchanges with the roles swapped (d O rows go out with
`dispatch_rows` semantics reversed, d Xp rows come back), plus gate gradients, one float per row.

Everything here is tensor plumbing on `torch.distributed` (gloo on CPU tensors in the tests, NCCL on
CUDA tensors in deployment); the arithmetic of each rank stays in the library's kernels.  No kernel
ever reads another GPU's memory: rows are copied into this rank's own buffers before any is used.
Covered by a two-rank CPU test of the exchanges against the oracle and by a GPU test in which two
ranks share one GPU (`ExpertParallelLayer`, exchanges over gloo); it has not run on several GPUs, so
it has no performance figure.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch
import torch.distributed as dist


def _a2a(out, inp, out_splits, in_splits, group):
    if inp.is_cuda and dist.get_backend(group) == "gloo":     # gloo moves host memory: stage through it
        o = torch.empty(out.shape, dtype=out.dtype)
        dist.all_to_all_single(o, inp.cpu(), list(out_splits), list(in_splits), group=group)
        out.copy_(o)
        return out
    dist.all_to_all_single(out, inp, list(out_splits), list(in_splits), group=group)
    return out


def _all_reduce(t, op, group):
    if t.is_cuda and dist.get_backend(group) == "gloo":
        h = t.cpu()
        dist.all_reduce(h, op=op, group=group)
        t.copy_(h)
    else:
        dist.all_reduce(t, op=op, group=group)
    return t


def exchange_affinities(delta_local: torch.Tensor, group=None):
    """delta_local [T_local, E] (this rank's tokens, all experts) -> delta_owner [T, E_local] (all tokens
    in global order, this rank's experts), and the batch maximum of delta over all ranks."""
    W = dist.get_world_size(group)
    T_local, E = delta_local.shape
    assert E % W == 0
    E_local = E // W
    send = delta_local.view(T_local, W, E_local).permute(1, 0, 2).contiguous()       # [dest, T_local, E_local]
    recv = torch.empty_like(send)                                                     # [source, T_local, E_local]
    n = T_local * E_local
    _a2a(recv.view(-1), send.view(-1), [n] * W, [n] * W, group)
    dmax = delta_local.max().reshape(1).clone()
    _all_reduce(dmax, dist.ReduceOp.MAX, group)
    return recv.view(W * T_local, E_local), dmax[0]


@dataclass
class ExchangePlan:
    """Who sends which token rows to whom.  Expert side: for every source rank the rows of the local
    expert buffers its tokens fill (`want_rows[s]`, ascending).  Token side: for every destination rank
    the local token ids it asked for, in the order it expects them, with their gates."""
    world: int
    rank: int
    T_local: int
    want_rows: list          # [W] int64 tensors: row ids in this rank's [E_local * C_stride] buffers
    send_tokens: list        # [W] int64 tensors: local token ids to send to each rank
    send_gates: list         # [W] float tensors: gate of each of those rows
    send_rows: list          # [W] int64 tensors: the row each of them fills in the destination's buffers
    rows_in: list            # splits of rows received by the expert side, per source rank
    rows_out: list           # splits of rows sent by the token side, per destination rank


def build_plan(slot_token: torch.Tensor, gate: torch.Tensor, T_local: int, group=None) -> ExchangePlan:
    """slot_token, gate: the routing maps of this rank's experts over the whole batch ([E_local *
    C_stride], global token ids, -1 for unused slots).  Two small exchanges: the row counts, then the
    token ids and gates every owner asks for."""
    W, rank = dist.get_world_size(group), dist.get_rank(group)
    rows = torch.nonzero(slot_token >= 0).flatten()
    src = torch.div(slot_token[rows], T_local, rounding_mode="floor")
    want_rows = [rows[src == s] for s in range(W)]                    # ascending row order inside a source
    rows_in = [int(r.numel()) for r in want_rows]
    counts_in = torch.tensor(rows_in, dtype=torch.int64, device=slot_token.device)
    counts_out = torch.empty_like(counts_in)
    _a2a(counts_out, counts_in, [1] * W, [1] * W, group)
    rows_out = [int(c) for c in counts_out]
    ask_tok = torch.cat([(slot_token[r] - s * T_local).to(torch.int64) for s, r in enumerate(want_rows)])
    ask_gate = torch.cat([gate[r] for r in want_rows])
    got_tok = torch.empty(sum(rows_out), dtype=torch.int64, device=slot_token.device)
    got_gate = torch.empty(sum(rows_out), dtype=gate.dtype, device=gate.device)
    got_row = torch.empty(sum(rows_out), dtype=torch.int64, device=slot_token.device)
    _a2a(got_tok, ask_tok, rows_out, rows_in, group)
    _a2a(got_gate, ask_gate, rows_out, rows_in, group)
    _a2a(got_row, torch.cat(want_rows), rows_out, rows_in, group)
    return ExchangePlan(W, rank, T_local, want_rows, list(got_tok.split(rows_out)),
                        list(got_gate.split(rows_out)), list(got_row.split(rows_out)), rows_in, rows_out)


def dispatch_rows(plan: ExchangePlan, X_local: torch.Tensor, n_buffer_rows: int, group=None) -> torch.Tensor:
    """Token rows to the experts' buffers: returns Xp [n_buffer_rows, d] of this rank's experts (rows not
    in use are zero).  One All-to-All of at most E_local * C rows of d elements per rank."""
    d = X_local.shape[1]
    send = X_local[torch.cat(plan.send_tokens)] if sum(plan.rows_out) else X_local[:0]
    recv = torch.empty(sum(plan.rows_in), d, dtype=X_local.dtype, device=X_local.device)
    _a2a(recv.view(-1), send.contiguous().view(-1), [r * d for r in plan.rows_in],
         [r * d for r in plan.rows_out], group)
    Xp = torch.zeros(n_buffer_rows, d, dtype=X_local.dtype, device=X_local.device)
    Xp[torch.cat(plan.want_rows)] = recv
    return Xp


def return_rows(plan: ExchangePlan, O: torch.Tensor, group=None) -> torch.Tensor:
    """The reverse exchange: the rows of O (or of d Xp in the backward pass) that belong to each rank's
    tokens travel back; returns them in the order of `plan.send_tokens` (destination rank major)."""
    d = O.shape[1]
    send = O[torch.cat(plan.want_rows)]
    recv = torch.empty(sum(plan.rows_out), d, dtype=O.dtype, device=O.device)
    _a2a(recv.view(-1), send.contiguous().view(-1), [r * d for r in plan.rows_out],
         [r * d for r in plan.rows_in], group)
    return recv


def scatter_rows_to_experts(plan: ExchangePlan, rows_by_token: torch.Tensor, n_buffer_rows: int, group=None):
    """Rows computed on the token side in the order of `plan.send_tokens` (d O = gate * dY in the backward
    pass) travel to the experts' buffers: the same traffic as dispatch_rows with rows given directly."""
    d = rows_by_token.shape[1]
    recv = torch.empty(sum(plan.rows_in), d, dtype=rows_by_token.dtype, device=rows_by_token.device)
    _a2a(recv.view(-1), rows_by_token.contiguous().view(-1), [r * d for r in plan.rows_in],
         [r * d for r in plan.rows_out], group)
    out = torch.zeros(n_buffer_rows, d, dtype=rows_by_token.dtype, device=rows_by_token.device)
    out[torch.cat(plan.want_rows)] = recv
    return out


def combine_local(plan: ExchangePlan, rows_back: torch.Tensor, accumulate_dtype=torch.float32) -> torch.Tensor:
    """Y[t] = sum over the token's rows of gate * O row, rows taken in ascending (rank, row) order, which
    is ascending expert order; tokens without a row get zeros.  Accumulates in `accumulate_dtype`."""
    d = rows_back.shape[1]
    Y = torch.zeros(plan.T_local, d, dtype=accumulate_dtype, device=rows_back.device)
    off = 0
    for q in range(plan.world):                       # ascending owner rank = ascending expert index
        n = plan.rows_out[q]
        if n == 0:
            continue
        tok, g = plan.send_tokens[q], plan.send_gates[q].to(accumulate_dtype)
        part = rows_back[off:off + n].to(accumulate_dtype) * g[:, None]
        # within one owner a token may hold several rows (one per expert of that owner), already in
        # ascending row order: add them one expert layer at a time to keep that order
        order = torch.argsort(tok, stable=True)
        tok_s, part_s = tok[order], part[order]
        first = torch.ones_like(tok_s, dtype=torch.bool)
        first[1:] = tok_s[1:] != tok_s[:-1]
        rank_in_tok = torch.arange(n, device=tok.device) - torch.cummax(
            torch.where(first, torch.arange(n, device=tok.device), torch.zeros_like(tok_s)), 0).values
        for layer in range(int(rank_in_tok.max()) + 1):
            sel = rank_in_tok == layer
            Y[tok_s[sel]] += part_s[sel]
        off += n
    return Y


def with_unit_gates(plan: ExchangePlan) -> ExchangePlan:
    """The same plan with every gate 1: `combine_local` then is the plain sum of a token's rows
    (the dispatch backward, d X[t] = sum of the token's rows of d Xp)."""
    return ExchangePlan(plan.world, plan.rank, plan.T_local, plan.want_rows, plan.send_tokens,
                        [torch.ones_like(g) for g in plan.send_gates], plan.send_rows, plan.rows_in,
                        plan.rows_out)


class ExpertParallelLayer:
    """Forward and backward of the layer with the experts spread over the ranks of `group`, expert
    choice, fixed capacity: the per-rank arithmetic runs in the library's kernels (affinity, selection,
    expert FFN and their backward forms through the C ABI), the exchanges in the functions above.

    Every rank passes its T_local tokens, the full expert embeddings R [E, m] and the weights of its
    own experts [E_local, ...].  The adaptive capacity bound needs the batch maximum of the affinities
    over all ranks, which `exchange_affinities` returns; here the capacity is the caller's number."""

    def __init__(self, *, T_local, d, D, E, h, capacity, group=None, device="cuda"):
        from . import etr
        self.etr, self.group = etr, group
        self.W, self.rank = dist.get_world_size(group), dist.get_rank(group)
        assert E % self.W == 0
        self.T_local, self.T, self.E, self.E_local, self.d, self.D, self.h = T_local, T_local * self.W, E, E // self.W, d, D, h
        # the local tokens against all experts (S1 and the dense router backward)
        self.cfg_tok = etr.make_config(T=T_local, d=d, D=D, E=E, k=1, h=h, capacity=capacity, dtype=etr.BF16,
                                       mode=etr.MODE_ECR, gate_mode=etr.GATE_SOFTMAX)
        # the local experts over all tokens (S3, S5 and their backward)
        self.cfg_own = etr.make_config(T=self.T, d=d, D=D, E=self.E_local, k=1, h=h, capacity=capacity,
                                       dtype=etr.BF16, mode=etr.MODE_ECR)
        self.own = etr.LayerBuffers(self.cfg_own, device=device)
        self.rows = self.E_local * etr.c_stride(self.cfg_own)
        f32 = dict(dtype=torch.float32, device=device)
        m = d // D
        self.delta = torch.empty(T_local, E, **f32)
        self.Z = torch.empty(T_local, m, **f32)
        self.xnorm, self.rnorm = torch.empty(T_local, **f32), torch.empty(E, **f32)
        self.stats_tok = torch.zeros(16, dtype=torch.int32, device=device)
        self.ws_tok = torch.empty(etr.workspace_bytes(self.cfg_tok), dtype=torch.uint8, device=device)
        self.ws_own = torch.empty(etr.workspace_bytes(self.cfg_own), dtype=torch.uint8, device=device)

    def forward(self, X, R, W1g, W1u, W2):
        etr, own = self.etr, self.own
        self.stats_tok.zero_()
        etr.affinity(self.cfg_tok, X, R, self.delta, self.Z, self.xnorm, self.rnorm, self.stats_tok)
        delta_own, self.delta_max = exchange_affinities(self.delta, self.group)
        own.delta.copy_(delta_own)
        own.stats.zero_()
        etr.select(self.cfg_own, own.delta, own.c.stats, own.route, self.ws_own)
        self.plan = build_plan(own.slot_token, own.gate, self.T_local, self.group)
        own.Xp.copy_(dispatch_rows(self.plan, X, self.rows, self.group))
        etr.expert_ffn(self.cfg_own, own.route, own.Xp, W1g, W1u, W2, own.G, own.U, own.H, own.O, own.c.stats,
                       self.ws_own)
        self.O_back = return_rows(self.plan, own.O, self.group)
        return combine_local(self.plan, self.O_back).to(X.dtype)

    def backward(self, X, R, W1g, W1u, W2, dY):
        """Returns dX [T_local, d], dR [E, m] (summed over the ranks) and the weight gradients of the local
        experts."""
        etr, own, plan = self.etr, self.own, self.plan
        send_tok = torch.cat(plan.send_tokens)
        gates = torch.cat(plan.send_gates)
        dY_rows = dY[send_tok].float()
        own.dO.copy_(scatter_rows_to_experts(plan, (dY_rows * gates[:, None]).to(dY.dtype), self.rows, self.group))
        dgate_rows = (dY_rows * self.O_back.float()).sum(1)
        dW1g, dW1u, dW2 = torch.empty_like(W1g), torch.empty_like(W1u), torch.empty_like(W2)
        etr.expert_ffn_bwd(self.cfg_own, own.route, own.dO, own.Xp, own.G, own.U, own.H, W1g, W1u, W2, own.dG,
                           own.dU, own.dXp, dW1g, dW1u, dW2, own.c.stats, self.ws_own)
        dX = combine_local(with_unit_gates(plan), return_rows(plan, own.dXp, self.group)).to(dY.dtype)
        # router gradient of the local tokens: d delta is non-zero on the token's selected pairs
        Cs = self.rows // self.E_local
        expert = torch.cat([q * self.E_local + torch.div(r, Cs, rounding_mode="floor")
                            for q, r in enumerate(plan.send_rows)])
        ddelta = torch.zeros_like(self.delta)
        ddelta[send_tok, expert] = dgate_rows
        n_rows = torch.zeros(self.T_local, dtype=torch.int32, device=dY.device)
        n_rows.index_add_(0, send_tok, torch.ones_like(send_tok, dtype=torch.int32))
        tok_ptr = torch.zeros(self.T_local + 1, dtype=torch.int32, device=dY.device)
        tok_ptr[1:] = torch.cumsum(n_rows, 0)
        spare = torch.zeros(max(int(tok_ptr[-1]), 4), dtype=torch.int32, device=dY.device)
        route = etr.Route(spare.data_ptr(), spare.data_ptr(), spare.data_ptr(), spare.data_ptr(),
                          tok_ptr.data_ptr(), spare.data_ptr())          # only tok_ptr is read: which tokens have rows
        dR = torch.empty_like(R)
        etr.affinity_bwd_dense(self.cfg_tok, X, R, self.delta, self.Z, self.xnorm, self.rnorm, route, ddelta, dX,
                               dR, self.ws_tok)
        _all_reduce(dR, dist.ReduceOp.SUM, self.group)
        st = etr.read_stats(own.c.stats)
        assert st.error_word == 0
        return dX, dR, dW1g, dW1u, dW2
