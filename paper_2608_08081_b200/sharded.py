"""Context-sharded decode: every rank holds a slice of each sequence's rows in its own packed cache.

The attention path shards by sequence or KV head with no exchange at all; this is the other way to scale it, for a
context too long for one GPU. Each rank runs the fused decode kernel over its slice -- the split partials (m, l, acc)
of Appendix A's softmax are exactly what flash-decoding exchanges -- then ONE exchange, an all-gather of those
partials ((head_dim + 2) * 4 bytes per head, split and rank, a few hundred KB over NVLink) into a buffer that was
allocated once, and every rank merges all of them in place with iq_combine_splits_sharded, which also applies the
single inverse rotation. Nothing else crosses the ranks, no kernel of the library touches another GPU's memory, and a
step allocates nothing.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


class ShardedBuffers:
    """The gather buffers of a context-sharded decode, allocated once for (batch, heads, splits, head_dim, world):
    the ranks' partials rank after rank, as all_gather_into_tensor leaves them and iq_combine_splits_sharded reads them."""

    def __init__(self, batch: int, n_q_heads: int, num_splits: int, head_dim: int, world: int, want_argmax: bool, device):
        B, H, S, d = batch, n_q_heads, num_splits, head_dim
        self.world, self.num_splits = world, S
        self.acc = torch.empty((world, B, H, S, d), dtype=torch.float32, device=device)
        self.ml = torch.empty((world, B, H, S, 2), dtype=torch.float32, device=device)
        self.argmax = torch.empty((world, B, H, S), dtype=torch.int32, device=device) if want_argmax else None
        self.row_offsets = torch.zeros((world, B), dtype=torch.int32, device=device)   # first row of rank r's slice of sequence b

    def set_row_offsets(self, my_offsets, group=None) -> None:
        """Every rank contributes the first row of its slice of each sequence (int32 [B]); needed once, or whenever the
        slices move."""
        dist.all_gather_into_tensor(self.row_offsets.view(-1), my_offsets.to(self.row_offsets.dtype).contiguous(), group=group)

    def gather(self, part_acc, part_ml, part_argmax=None, group=None) -> None:
        """The one exchange of a step: this rank's partials ([B][H][S][..], contiguous) into every rank's buffers."""
        # (the output as the concatenation of the ranks' tensors along their first axis: every backend takes that form)
        dist.all_gather_into_tensor(self.acc.flatten(0, 1), part_acc, group=group)
        dist.all_gather_into_tensor(self.ml.flatten(0, 1), part_ml, group=group)
        if self.argmax is not None:
            dist.all_gather_into_tensor(self.argmax.flatten(0, 1), part_argmax, group=group)

    def slot_major(self):
        """The gathered partials viewed as [B][H][world * S][..] (rank r's slots at [r * S, (r + 1) * S)) with global
        argmax rows: for checking against a reference merge; the product path reads the buffers as they are."""
        W, B, H, S, d = self.acc.shape
        acc = self.acc.permute(1, 2, 0, 3, 4).reshape(B, H, W * S, d)
        ml = self.ml.permute(1, 2, 0, 3, 4).reshape(B, H, W * S, 2)
        am = None
        if self.argmax is not None:
            am = torch.where(self.argmax >= 0, self.argmax + self.row_offsets[:, :, None, None], self.argmax)
            am = am.permute(1, 2, 0, 3).reshape(B, H, W * S)
        return acc, ml, am


def sharded_decode_step(iq, shape, rot_dev, codebook, q, cache_local, seq_lens_local, ws, bufs: ShardedBuffers, group=None, stream=None):
    """One decode step over a context that is sharded across the ranks of `group`: q [B][H_q][d] is the same on every
    rank, cache_local / seq_lens_local describe this rank's slice of every sequence, ws is a DecodeWorkspace for
    (shape, S) and bufs the ShardedBuffers made for it (row offsets set). The result -- identical on every rank --
    lands in ws.out / ws.lse / ws.argmax; nothing is allocated."""
    iq.iq_decode_attention(shape, rot_dev, codebook, q, cache_local, seq_lens_local, ws.num_splits, ws.part_acc, ws.part_ml,
                           ws.part_argmax, ws.status, stream)
    bufs.gather(ws.part_acc, ws.part_ml, ws.part_argmax, group)
    iq.iq_combine_splits_sharded(shape, rot_dev, ws.num_splits, bufs.world, bufs.acc, bufs.ml, bufs.argmax,
                                 bufs.row_offsets if bufs.argmax is not None else None, ws.out, ws.lse, ws.argmax, stream)
    return ws.out, ws.lse, ws.argmax
