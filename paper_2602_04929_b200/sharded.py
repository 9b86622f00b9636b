"""One projection spread over several GPUs (one process per GPU, torch.distributed).

The path has two natural shard axes and one exchange on each side of the quantizer:

  tokens  every rank accumulates the un-normalised Hessian (and deviation correlation) of its own
          slice of the calibration tokens; ONE all-reduce (sum) of the d x d float matrices gives
          every rank the full H_in (and R).  Slices are multiples of 2048 tokens, the accumulation
          run of the Hessian kernel.
  heads   the heads of a projection are independent problems (the paper quantizes all heads at
          once for that reason), so rank r quantizes heads [h0, h1) only; the factors of H_in and
          the propagated-error operands are computed by every rank for itself from the all-reduced
          matrices (identical inputs, identical results, no broadcast); ONE all-gather per output
          returns the whole layer's codes, scales, zero-points, W_hat and per-head loss to all ranks.

torch.distributed only moves the tensors (NCCL over NVLink for CUDA tensors); every arithmetic step
is a call of the C-ABI library through `ops` (default: this package's binding, which raises without
the CUDA library).  With world size 1 no collective is issued and the result is that of the plain
calls.  After the all-reduce the float sums differ in the last bits from a single-GPU accumulation
over all tokens (another summation order), so codes can differ from a single-GPU run exactly as
they can between any two valid Hessians that agree to 1e-6; all ranks agree with one another bit
for bit.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

TOKEN_RUN = 2048


def shard_tokens(n_tok: int, world: int, rank: int) -> tuple[int, int]:
    """Token slice [t0, t1) of `rank`: runs of 2048 tokens dealt as evenly as possible, the ragged
    last run to the last rank that has any."""
    runs = -(-n_tok // TOKEN_RUN)
    per, extra = divmod(runs, world)
    r0 = rank * per + min(rank, extra)
    r1 = r0 + per + (1 if rank < extra else 0)
    return min(r0 * TOKEN_RUN, n_tok), min(r1 * TOKEN_RUN, n_tok)


def shard_heads(n_heads: int, world: int, rank: int) -> tuple[int, int]:
    """Head range [h0, h1) of `rank`: contiguous, sizes differing by at most one."""
    per, extra = divmod(n_heads, world)
    h0 = rank * per + min(rank, extra)
    return h0, h0 + per + (1 if rank < extra else 0)


@dataclass
class ShardedResult:
    codes: torch.Tensor
    scales: torch.Tensor
    zeros: torch.Tensor
    w_hat: torch.Tensor
    loss: torch.Tensor


class _LibraryOps:
    """The C-ABI calls the sharded path is made of (argument marshalling only)."""

    def __init__(self):
        from . import binding
        self.b = binding

    def accumulate(self, X, Xfp, alpha):
        d = X.shape[1]
        H = torch.zeros((d, d), dtype=torch.float32, device=X.device)
        R = None
        if X.shape[0]:
            self.b.tb_accumulate_hessian(H, X)
        if Xfp is not None:
            R = torch.zeros_like(H)
            if X.shape[0]:
                self.b.tb_accumulate_cross(R, X, Xfp, alpha)
        return H, R

    def finalize(self, H, R, n_total, damp):
        Hsum = torch.empty_like(H)
        self.b.tb_finalize_hessian(H, R, n_total, damp, Hsum_out=Hsum)
        return Hsum

    def factor(self, H):
        U, info = self.b.tb_factor(H)
        if int(info.max().item()) != 0:
            raise self.b.TurboBoAError(4, "tb_factor")
        return U

    def correction(self, R, U):
        return self.b.tb_prepare_correction(R, U)

    def build_hout(self, G, Hsum, n_heads, d_head, damp):
        return self.b.tb_build_hout(G, Hsum, n_heads, d_head, damp)

    def quantize(self, desc_kw, W, H, U, Hout, Uout, R, P, C):
        desc = self.b.layer_desc(**desc_kw)
        r = self.b.tb_quantize_layer(desc, W, H, U, Hout, Uout, R, P, C)
        return r.codes, r.scales, r.zeros, r.w_hat, r.loss


def _all_gather_rows(t: torch.Tensor, sizes: list[int], group) -> torch.Tensor:
    """Concatenation over ranks of tensors whose first dimension differs per rank."""
    import torch.distributed as dist
    biggest = max(sizes)
    pad = torch.zeros((biggest,) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
    pad[: t.shape[0]] = t
    parts = [torch.empty_like(pad) for _ in sizes]
    dist.all_gather(parts, pad, group=group)
    return torch.cat([p[:n] for p, n in zip(parts, sizes)], dim=0)


def quantize_projection_sharded(W, X_local, n_tok_total, n_heads, d_head, bits, quant_group, out_block, *, G=None,
                                g_heads=None, Xfp_local=None, alpha=0.25, damp=0.01, n_cand=16, cd_iters=1, flags=3,
                                group=None, ops=None) -> ShardedResult:
    """Quantizes W [n_heads * d_head, d] from this rank's token slice X_local (rows [t0, t1) of the
    calibration activations, see shard_tokens); every rank passes the same W and G and receives the
    whole result.  G: partner projection for H_out (None: H_out = identity, every row independent;
    the rows are then dealt like heads of d_head rows)."""
    import torch.distributed as dist
    ops = ops or _LibraryOps()
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    # 1. statistics of the local tokens, one all-reduce each
    H, R = ops.accumulate(X_local, Xfp_local, alpha)
    if world > 1:
        dist.all_reduce(H, op=dist.ReduceOp.SUM, group=group)
        if R is not None:
            dist.all_reduce(R, op=dist.ReduceOp.SUM, group=group)
    Hsum = ops.finalize(H, R, n_tok_total, damp)
    # 2. replicated prerequisites (identical on every rank)
    U = ops.factor(H)
    P = C = None
    if R is not None:
        P, C = ops.correction(R, U)
    # 3. this rank's heads
    h0, h1 = shard_heads(n_heads, world, rank)
    rows = slice(h0 * d_head, h1 * d_head)
    Hout = Uout = None
    if G is not None and h1 > h0:
        Hout_all = ops.build_hout(G, Hsum, n_heads, d_head, damp)
        Hout = Hout_all[h0:h1].contiguous()
        Uout = ops.factor(Hout)
    d = W.shape[1]
    ng = 1 if quant_group == 0 else d // quant_group
    if h1 > h0:
        desc_kw = dict(d_out=(h1 - h0) * d_head, d_in=d, n_heads=h1 - h0, d_head=d_head, bits=bits,
                       quant_group=quant_group, out_block=out_block if G is not None else d_head, n_cand=n_cand,
                       cd_iters=cd_iters, flags=flags)
        codes, scales, zeros, w_hat, loss = ops.quantize(desc_kw, W[rows].contiguous(), H, U, Hout, Uout, R, P, C)
    else:   # more ranks than heads: this rank holds nothing
        codes = torch.empty((0, d), dtype=torch.uint8, device=W.device)
        scales = torch.empty((0, ng), dtype=torch.float32, device=W.device)
        zeros = torch.empty((0, ng), dtype=torch.int32, device=W.device)
        w_hat = torch.empty((0, d), dtype=torch.float32, device=W.device)
        loss = torch.empty((0,), dtype=torch.float64, device=W.device)
    if world == 1:
        return ShardedResult(codes, scales, zeros, w_hat, loss)
    # 4. one all-gather per output
    heads_of = [shard_heads(n_heads, world, r) for r in range(world)]
    row_sizes = [(b - a) * d_head for a, b in heads_of]
    head_sizes = [b - a for a, b in heads_of]
    return ShardedResult(_all_gather_rows(codes, row_sizes, group), _all_gather_rows(scales, row_sizes, group),
                         _all_gather_rows(zeros, row_sizes, group), _all_gather_rows(w_hat, row_sizes, group),
                         _all_gather_rows(loss, head_sizes, group))
