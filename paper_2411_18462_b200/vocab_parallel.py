"""Vocabulary-parallel draft step: the exchange around svip_vp_partial / _combine / _locate.

Every rank holds V_shard columns of each logits row (a tensor-parallel LM head).  The three library
calls do the arithmetic on the GPU; this module only moves the 16-byte-per-row partials and the
4-byte tokens between the ranks with ``torch.distributed`` (NCCL on GPUs).  Two small collectives per
step: one all-gather of [B, 4] floats and one max-reduce of [B] int32.
"""
from __future__ import annotations


def shard_bounds(V: int, world: int, rank: int, align: int = 8):
    """Columns [lo, hi) of `rank`: contiguous, boundaries multiples of `align` elements (so that the
    shards of a 16-byte aligned row start 16-byte aligned for bf16 and fp32), sizes differing by at
    most `align` except for the ragged end of the last shard."""
    blocks = (V + align - 1) // align
    per, rem = divmod(blocks, world)
    lo_b = rank * per + min(rank, rem)
    hi_b = lo_b + per + (1 if rank < rem else 0)
    return min(lo_b * align, V), min(hi_b * align, V)


def gather_partials(partial, group=None):
    """[B, 4] per rank -> [G, B, 4], rank-major, identical on every rank."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return partial.unsqueeze(0).contiguous()
    parts = [torch.empty_like(partial) for _ in range(dist.get_world_size(group))]
    dist.all_gather(parts, partial.contiguous(), group=group)
    return torch.stack(parts).contiguous()


def share_tokens(token, group=None):
    """token[b] is -1 on every rank but the owner of row b: the max over ranks is the token."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(token, op=dist.ReduceOp.MAX, group=group)
    return token


def draft_step(ctx, shard_logits, dtype, B, V_shard, row_stride, T, thresh, uniforms, vocab_offset, rank=0,
               world=1, group=None, stream=None):
    """One draft token per row from vocabulary shards.  Returns (token int32 [B], entropy fp32 [B],
    stop uint8 [B]) as CUDA tensors, identical on every rank."""
    import torch
    dev = shard_logits.device
    partial = torch.empty((B, 4), dtype=torch.float32, device=dev)
    ctx.vp_partial(shard_logits, dtype, B, V_shard, row_stride, T, vocab_offset, partial, stream)
    partials = gather_partials(partial, group)
    entropy = torch.empty(B, dtype=torch.float32, device=dev)
    stop = torch.empty(B, dtype=torch.uint8, device=dev)
    token = torch.empty(B, dtype=torch.int32, device=dev)
    owner = torch.empty(B, dtype=torch.int32, device=dev)
    target = torch.empty(B, dtype=torch.float32, device=dev)
    active = torch.empty(B, dtype=torch.uint8, device=dev)
    ctx.vp_combine(partials, partials.shape[0], rank, B, T, thresh, uniforms, entropy, stop, token, owner, target,
                   active, stream)
    if T > 0:
        ctx.vp_locate(shard_logits, dtype, B, V_shard, row_stride, T, target, active, vocab_offset, token, stream)
        share_tokens(token, group)
    return token, entropy, stop
