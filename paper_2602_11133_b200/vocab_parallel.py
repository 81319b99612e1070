"""Host side of a vocabulary-parallel LM head: which slice a rank owns, and the exchange of the per-row tuples.

Each rank runs the head over its slice of the vocabulary (jot_lm_head_stats_slice), the ranks all-gather the
16-byte tuples (top1, top2, sumexp, argmax) of every position, and every rank folds them with the device merge
(jot_merge_stats).  This module holds only the slice arithmetic and the collective: no statistic is computed
here.  Unmeasured on hardware: every call of this build has one GPU.
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def vocab_slice(rank: int, world: int, vocab: int, tile: int = 256) -> Tuple[int, int]:
    """[v_lo, v_hi) of `rank`: whole tiles of `tile` token ids spread as evenly as the tile count allows, the
    remainder on the lowest ranks; the last slice ends at the vocabulary.  A rank may come out empty (v_lo ==
    v_hi) when there are more ranks than tiles."""
    if not 0 <= rank < world or vocab <= 0 or tile <= 0:
        raise ValueError("bad slice request")
    n_tiles = (vocab + tile - 1) // tile
    base, rem = divmod(n_tiles, world)
    first = rank * base + min(rank, rem)
    count = base + (1 if rank < rem else 0)
    return min(first * tile, vocab), min((first + count) * tile, vocab)


def pack_tuples(top1: torch.Tensor, top2: torch.Tensor, sumexp: torch.Tensor, argmax: torch.Tensor) -> torch.Tensor:
    """[..., 4] float32 with the token id bit-cast into the fourth lane: one 16-byte tuple per position."""
    return torch.stack([top1, top2, sumexp, argmax.view(torch.float32)], dim=-1).contiguous()


def unpack_tuples(t: torch.Tensor):
    return t[..., 0].contiguous(), t[..., 1].contiguous(), t[..., 2].contiguous(), t[..., 3].contiguous().view(torch.int32)


def all_gather_tuples(packed: torch.Tensor, group=None) -> List[torch.Tensor]:
    """Every rank's packed tuples, in rank order (one all-gather of 16 bytes per position and rank)."""
    world = dist.get_world_size(group)
    out = [torch.empty_like(packed) for _ in range(world)]
    dist.all_gather(out, packed, group=group)
    return out
