"""Host side of the vocabulary-parallel LM head on CPU: slice arithmetic, and two gloo ranks that each take the
statistics of their slice (from the oracle: there is no device here), all-gather the 16-byte tuples through the
package's exchange and fold them; the result must be the oracle's statistics of the whole row."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_slices_tile_the_vocabulary():
    from paper_2602_11133_b200 import vocab_parallel as vp
    for vocab, tile in ((126464, 256), (152064, 128), (4096, 256), (1000, 256), (520, 128)):
        for world in (1, 2, 3, 4, 8):
            sl = [vp.vocab_slice(r, world, vocab, tile) for r in range(world)]
            assert sl[0][0] == 0 and sl[-1][1] == vocab
            for (a, b), (c, d) in zip(sl, sl[1:]):
                assert b == c and a <= b                                   # contiguous, in rank order
            assert all(a % tile == 0 for a, b in sl if b > a)              # whole tiles: a non-empty slice starts on one
            sizes = [(b - a + tile - 1) // tile for a, b in sl]
            assert max(sizes) - min(sizes) <= 1                            # as even as the tile count allows


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from oracle import jot_oracle as jo
    from paper_2602_11133_b200 import vocab_parallel as vp
    dist.init_process_group("gloo", rank=rank, world_size=world)
    V, R, mask_id = 1000, 24, 777
    rng = np.random.default_rng(5)                                          # the same logits on every rank
    logits = rng.normal(0, 2, size=(R, V)).round(1)                         # coarse values: exact ties occur
    logits[3, 10] = logits[3, 900] = 9.5                                    # a tie of the maxima across the two slices
    logits[4, mask_id] = 50.0                                               # the excluded token would win
    lo, hi = vp.vocab_slice(rank, world, V, 256)
    mine = [jo.row_stats_slice(logits[r], lo, hi, mask_id) for r in range(R)]
    f32 = lambda xs: torch.tensor(xs, dtype=torch.float32)
    packed = vp.pack_tuples(f32([s.m1 for s in mine]), f32([s.m2 for s in mine]), f32([s.S for s in mine]),
                            torch.tensor([s.i1 for s in mine], dtype=torch.int32))
    assert packed.shape == (R, 4) and packed.element_size() * 4 == 16
    parts = vp.all_gather_tuples(packed)
    assert len(parts) == world and torch.equal(parts[rank], packed)
    ok = True
    for r in range(R):
        acc = None
        for q in range(world):                                              # fold in rank order
            t1, t2, S, i1 = vp.unpack_tuples(parts[q])
            st = jo.RowStats(float(t1[r]), int(i1[r]), float(t2[r]), float(S[r]))
            acc = st if acc is None else jo.merge_row_stats(acc, st)
        want = jo.row_stats(logits[r], mask_id)
        ok &= (acc.i1 == want.i1 and abs(acc.m1 - want.m1) < 1e-6 and abs(acc.m2 - want.m2) < 1e-6
               and abs(acc.S - want.S) <= 1e-5 * want.S)
    with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
        f.write("1" if ok else "0")
    dist.destroy_process_group()


def test_two_gloo_ranks_exchange_and_merge_slice_tuples(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, free_port(), str(tmp_path)), nprocs=world, join=True)
    assert [open(tmp_path / f"ok{r}").read() for r in range(world)] == ["1", "1"]
