"""Vocabulary-sharded speculation step: every rank holds a slice of the vocabulary axis of the logits
(a tensor-parallel output projection leaves them like that) and the full rows are never gathered.

Per step and rank: four library calls with two small all-gathers and one MAX all-reduce in between
(`step`); what crosses the ranks is 16 bytes per logit row plus 16 bytes per batch row, against
2·V bytes per logit row for gathering the logits.  The results are those of `speckv_step` on the
concatenated logits (paper Sec. 3.1, 4.1-4.3).

`step_emulated` runs the same calls for all shards on one device, the exchanges replaced by
stacking; it serves tests and machines with fewer devices than shards.  This module only marshals
arguments and moves the exchanged buffers: every arithmetic step is a kernel of the library.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Tuple

import torch

from . import binding as speckv


def shard_bounds(V: int, n_shards: int) -> Tuple[int, List[Tuple[int, int]]]:
    """Equal-width column slices, the last one possibly narrower: (width, [(begin, end), ...]).
    The width is rounded up to 8 columns so that bf16 and fp32 slices of a 16-byte aligned tensor stay
    16-byte aligned."""
    if n_shards < 1 or n_shards > 32:
        raise ValueError("1..32 shards")
    width = -(-V // n_shards)
    width = -(-width // 8) * 8
    if width * (n_shards - 1) >= V:
        raise ValueError(f"V = {V} is too small for {n_shards} shards of {width} columns")
    return width, [(r * width, min(V, (r + 1) * width)) for r in range(n_shards)]


@dataclass
class ShardBuffers:
    """Per-rank buffers of one step shape; reusable across steps."""
    state: torch.Tensor      # [B, 2G+1, 4] fp32
    tokl: torch.Tensor       # [B, G, 2] fp32
    all_state: torch.Tensor  # [n_shards, B, 2G+1, 4]
    all_tokl: torch.Tensor   # [n_shards, B, G, 2]
    weight: torch.Tensor     # [B, 2] fp64
    all_weight: torch.Tensor  # [n_shards, B, 2]
    row_info: torch.Tensor   # [B, 32] bytes
    workspace: torch.Tensor
    out: speckv.StepOutputs

    @staticmethod
    def allocate(local: speckv.Batch, n_shards: int, n_out: int = 4) -> "ShardBuffers":
        B, G, _ = local.shape()
        dev = local.draft_logits.device
        f = lambda *s: torch.zeros(*s, dtype=torch.float32, device=dev)
        out = speckv.StepOutputs(H=f(B, G), C=f(B, G), feat=f(B, 4), scores=f(B, n_out),
                                 gamma_next=torch.zeros(B, dtype=torch.int32, device=dev),
                                 n_accepted=torch.zeros(B, dtype=torch.int32, device=dev),
                                 out_tokens=torch.zeros(B, G + 1, dtype=torch.int32, device=dev),
                                 row_status=torch.zeros(B, dtype=torch.int32, device=dev),
                                 workspace=torch.empty(0, dtype=torch.uint8, device=dev))
        return ShardBuffers(state=f(B, 2 * G + 1, 4), tokl=f(B, G, 2), all_state=f(n_shards, B, 2 * G + 1, 4),
                            all_tokl=f(n_shards, B, G, 2),
                            weight=torch.zeros(B, 2, dtype=torch.float64, device=dev),
                            all_weight=torch.zeros(n_shards, B, 2, dtype=torch.float64, device=dev),
                            row_info=torch.zeros(B, speckv.ROW_INFO_BYTES, dtype=torch.uint8, device=dev),
                            workspace=speckv.shard_workspace(local), out=out)


def exchange_gather(dst: torch.Tensor, src: torch.Tensor, group=None) -> None:
    """dst[r] = rank r's src, in rank order."""
    import torch.distributed as dist
    # rank-major concatenation along the first axis (the form every backend accepts)
    dist.all_gather_into_tensor(dst.view(-1, *src.shape[1:]), src.contiguous(), group=group)


def exchange_max(t: torch.Tensor, group=None) -> None:
    import torch.distributed as dist
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)


def step(local: speckv.Batch, v_begin: int, shard_width: int, V_total: int, comp: Optional[torch.Tensor],
         mlp: Optional[speckv.Mlp], buf: Optional[ShardBuffers] = None, group=None) -> dict:
    """One step on this rank's slice; all ranks of `group` call it together and get the same result."""
    import torch.distributed as dist
    n_shards = dist.get_world_size(group)
    rank = dist.get_rank(group)
    buf = buf or ShardBuffers.allocate(local, n_shards, mlp.n_out if mlp is not None else 4)
    speckv.speckv_shard_sweep(local, v_begin, buf.state, buf.tokl, buf.workspace)
    exchange_gather(buf.all_state, buf.state, group)
    exchange_gather(buf.all_tokl, buf.tokl, group)
    speckv.speckv_shard_finish(local, n_shards, shard_width, V_total, buf.all_state, buf.all_tokl, comp, mlp,
                               buf.out, buf.row_info)
    speckv.speckv_shard_draw_sums(local, buf.row_info, buf.weight, buf.workspace)
    exchange_gather(buf.all_weight, buf.weight, group)
    speckv.speckv_shard_draw_pick(local, v_begin, rank, n_shards, buf.row_info, buf.all_weight, buf.out.out_tokens,
                                  buf.workspace)
    exchange_max(buf.out.out_tokens, group)
    return buf.out.as_dict()


def slice_batch(full: speckv.Batch, begin: int, end: int) -> speckv.Batch:
    """The columns [begin, end) of a full batch as a local batch (views, no copy)."""
    return speckv.Batch(draft_logits=full.draft_logits[:, :, begin:end], target_logits=full.target_logits[:, :, begin:end],
                        draft_tokens=full.draft_tokens, gamma=full.gamma, temperature=full.temperature,
                        uniforms=full.uniforms, temperature_scalar=full.temperature_scalar,
                        entropy_in_bits=full.entropy_in_bits)


def step_emulated(full: speckv.Batch, n_shards: int, comp: Optional[torch.Tensor], mlp: Optional[speckv.Mlp]) -> dict:
    """All shards' calls on one device, one shard after the other, the exchanges replaced by copies.
    Also checks that every shard's `finish` gives the same outputs.  Returns shard 0's outputs."""
    V = full.draft_logits.shape[2]
    width, bounds = shard_bounds(V, n_shards)
    locs = [slice_batch(full, a, e) for a, e in bounds]
    bufs = [ShardBuffers.allocate(l, n_shards, mlp.n_out if mlp is not None else 4) for l in locs]
    for r, (l, bf) in enumerate(zip(locs, bufs)):
        speckv.speckv_shard_sweep(l, bounds[r][0], bf.state, bf.tokl, bf.workspace)
    for bf in bufs:
        for r, src in enumerate(bufs):
            bf.all_state[r].copy_(src.state)
            bf.all_tokl[r].copy_(src.tokl)
    for l, bf in zip(locs, bufs):
        speckv.speckv_shard_finish(l, n_shards, width, V, bf.all_state, bf.all_tokl, comp, mlp, bf.out, bf.row_info)
        speckv.speckv_shard_draw_sums(l, bf.row_info, bf.weight, bf.workspace)
    for name in ("H", "C", "feat", "n_accepted", "out_tokens", "row_status", "gamma_next"):
        for bf in bufs[1:]:
            if not torch.equal(getattr(bf.out, name), getattr(bufs[0].out, name)):
                raise RuntimeError(f"shards disagree on {name}")
    for bf in bufs:
        for r, src in enumerate(bufs):
            bf.all_weight[r].copy_(src.weight)
    for r, (l, bf) in enumerate(zip(locs, bufs)):
        speckv.speckv_shard_draw_pick(l, bounds[r][0], r, n_shards, bf.row_info, bf.all_weight, bf.out.out_tokens,
                                      bf.workspace)
    toks = torch.stack([bf.out.out_tokens for bf in bufs]).max(dim=0).values
    bufs[0].out.out_tokens.copy_(toks)
    return bufs[0].out.as_dict()


def main():
    """Times one rank's four calls on its slice of a synthetic workload (one device; the exchanges
    are copies of this rank's own buffers, so only their sizes are reported)."""
    import argparse
    import json

    from . import synth

    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="b256")
    ap.add_argument("--shards", type=int, default=8)
    ap.add_argument("--rank", type=int, default=0)
    ap.add_argument("--rows", type=int, default=None)
    ap.add_argument("--iters", type=int, default=50)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: the library has no CPU path")
    dev = torch.device("cuda", 0)
    w = synth.WORKLOADS[args.workload]
    if args.rows:
        w = synth.scaled(w, B=args.rows)
    s = synth.make_step(w, 0, dev)
    width, bounds = shard_bounds(w.V, args.shards)
    a, e = bounds[args.rank]
    # a rank of a tensor-parallel projection holds its slice contiguously
    local = speckv.Batch(draft_logits=s["draft"][:, :, a:e].contiguous(), target_logits=s["target"][:, :, a:e].contiguous(),
                         draft_tokens=s["draft_tokens"], gamma=s["gamma"], temperature=s["temperature"],
                         uniforms=s["uniforms"])
    full = speckv.Batch(draft_logits=s["draft"], target_logits=s["target"], draft_tokens=s["draft_tokens"],
                        gamma=s["gamma"], temperature=s["temperature"], uniforms=s["uniforms"])
    mw = synth.make_mlp(w, dev)
    mlp = speckv.Mlp(mw["W1"], mw["b1"], mw["W2"], mw["b2"])
    # states of the other shards: computed once, from views of the full logits
    others = []
    for r, (ra, re) in enumerate(bounds):
        b = ShardBuffers.allocate(slice_batch(full, ra, re), args.shards, mlp.n_out)
        speckv.speckv_shard_sweep(slice_batch(full, ra, re), ra, b.state, b.tokl, b.workspace)
        others.append(b)
    buf = ShardBuffers.allocate(local, args.shards, mlp.n_out)
    for r, o in enumerate(others):
        buf.all_state[r].copy_(o.state)
        buf.all_tokl[r].copy_(o.tokl)
    speckv.speckv_shard_finish(local, args.shards, width, w.V, buf.all_state, buf.all_tokl, s["comp"], mlp, buf.out,
                               buf.row_info)
    for r, (o, (ra, re)) in enumerate(zip(others, bounds)):
        speckv.speckv_shard_draw_sums(slice_batch(full, ra, re), buf.row_info, o.weight, o.workspace)
        buf.all_weight[r].copy_(o.weight)
    torch.cuda.synchronize()

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.iters)]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    for it in range(args.iters + 3):
        flush.zero_()                                   # the slice is smaller than L2: evict it between iterations
        e5 = ev[max(it - 3, 0)]
        e5[0].record()
        speckv.speckv_shard_sweep(local, a, buf.state, buf.tokl, buf.workspace)
        e5[1].record()
        speckv.speckv_shard_finish(local, args.shards, width, w.V, buf.all_state, buf.all_tokl, s["comp"], mlp, buf.out,
                                   buf.row_info)
        e5[2].record()
        speckv.speckv_shard_draw_sums(local, buf.row_info, buf.weight, buf.workspace)
        e5[3].record()
        speckv.speckv_shard_draw_pick(local, a, args.rank, args.shards, buf.row_info, buf.all_weight, buf.out.out_tokens,
                                      buf.workspace)
        e5[4].record()
    torch.cuda.synchronize()
    us = [1e3 * sum(e5[k].elapsed_time(e5[k + 1]) for e5 in ev) / args.iters for k in range(4)]
    slice_bytes = int((2 * s["gamma"].long() + 1).sum()) * (e - a) * w.elem_bytes
    B, G = w.B, w.gamma_max
    print(json.dumps({
        "workload": w.name, "rows": B, "shards": args.shards, "rank": args.rank, "slice_columns": e - a,
        "us": {"sweep": us[0], "finish": us[1], "draw_sums": us[2], "draw_pick": us[3], "total": sum(us)},
        "slice_logit_bytes": slice_bytes, "sweep_GBps": slice_bytes / us[0] / 1e3,
        "exchanged_bytes_per_rank": {"states": B * (2 * G + 1) * 16, "token_logits": B * G * 8, "weights": B * 16,
                                     "tokens": B * (G + 1) * 4},
        "gathering_the_logits_instead_bytes_per_rank": slice_bytes,
        "l2": "a 256 MB buffer is overwritten before every iteration"}))


if __name__ == "__main__":
    main()
