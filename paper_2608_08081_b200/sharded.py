"""Context-sharded decode: every rank holds a slice of each sequence's rows in its own packed cache.

The attention path shards by sequence or KV head with no exchange at all; this is the other way to scale it, for a
context too long for one GPU. Each rank runs the fused decode kernel over its slice -- the split partials (m, l, acc)
of Appendix A's softmax are exactly what flash-decoding exchanges -- then ONE collective, an all-gather of those
partials ((head_dim + 2) * 4 bytes per head, split and rank, a few hundred KB over NVLink), and every rank merges
all of them with iq_combine_splits, which also applies the single inverse rotation. Nothing else crosses the ranks.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def gather_partials(part_acc, part_ml, part_argmax=None, row_offset=None, group=None):
    """All-gathers split partials over the ranks of `group`: part_acc [B][H][S][d], part_ml [B][H][S][2] and
    optionally part_argmax [B][H][S] (row indices local to the rank's slice; row_offset int32 [B] = the slice's first
    global row per sequence turns them into global rows). Returns the same tensors with world * S splits, rank r's
    splits at [r * S, (r + 1) * S). Works on any backend (the partials are ordinary tensors)."""
    world = dist.get_world_size(group)
    B, H, S, d = part_acc.shape

    def gather(t):
        t = t.contiguous()
        buf = [torch.empty_like(t) for _ in range(world)]
        dist.all_gather(buf, t, group=group)
        return torch.cat(buf, dim=2)        # [B][H][world * S][...]

    acc = gather(part_acc)
    ml = gather(part_ml)
    am = None
    if part_argmax is not None:
        am_local = part_argmax
        if row_offset is not None:          # empty splits keep their -1
            am_local = torch.where(part_argmax >= 0, part_argmax + row_offset.to(part_argmax.dtype)[:, None, None], part_argmax)
        am = gather(am_local)
    return acc, ml, am


def sharded_decode_step(iq, shape, rot_dev, codebook, q, cache_local, seq_lens_local, ws, row_offset=None, group=None, stream=None):
    """One decode step over a context that is sharded across the ranks of `group`: q [B][H_q][d] is the same on every
    rank, cache_local / seq_lens_local describe this rank's slice of every sequence, ws is a DecodeWorkspace for
    (shape, S). Returns (out, lse, argmax) -- identical on every rank -- in freshly allocated tensors."""
    iq.iq_decode_attention(shape, rot_dev, codebook, q, cache_local, seq_lens_local, ws.num_splits, ws.part_acc, ws.part_ml,
                           ws.part_argmax, ws.status, stream)
    acc, ml, am = gather_partials(ws.part_acc, ws.part_ml, ws.part_argmax, row_offset, group)
    out = torch.empty_like(ws.out)
    lse = torch.empty_like(ws.lse)
    argmax = torch.empty_like(ws.argmax) if am is not None else None
    iq.iq_combine_splits(shape, rot_dev, acc.shape[2], acc, ml, am, out, lse, argmax, stream)
    return out, lse, argmax
