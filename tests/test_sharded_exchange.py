"""Workers spread over ranks: the exchange of upload messages and its bookkeeping, on CPU tensors with two gloo ranks.

The collective part of the multi-GPU path (paper_1909_07588_b200/sharded.py: exchange_uploads) moves, per iteration,
the radius and the code stream of every uploading worker from its owner to all other ranks.  Here two CPU processes
play the ranks; the code streams are fabricated, so the test covers who sends what to whom, the order of the merged
upload list, empty and one-sided iterations, and the byte counts against the paper's 32 + b p bits per upload.
"""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
M, WORDS, ITERS = 7, 33, 5          # 7 workers over 2 ranks (4 + 3), rows of 33 words


def _row(m, k):
    """The fabricated code stream of worker m at iteration k."""
    return torch.from_numpy(np.random.default_rng(1000 * k + m).integers(-2 ** 31, 2 ** 31, WORDS, dtype=np.int64)
                            .astype(np.int32))


def _uploaders(k):
    """Global uploader set of iteration k: everybody, nobody, one rank only, a mix."""
    return [list(range(M)), [], [0, 2, 4, 6], [1, 5], [0, 3, 6]][k]


def _radius(m, k):
    return np.float32(0.5 + m + 10 * k)


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    from paper_1909_07588_b200 import sharded
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local = list(range(rank, M, world))
    max_local = (M + world - 1) // world
    ok = True
    sent_bytes = 0
    for k in range(ITERS):
        rows = {m: _row(m, k) for m in local}                       # what the quantizer left in this rank's memory
        mailbox = {m: torch.zeros(WORDS, dtype=torch.int32) for m in range(M)}
        mine = [m for m in _uploaders(k) if m % world == rank]
        m_all, R_all, st = sharded.exchange_uploads(mine, [_radius(m, k) for m in mine], lambda m: rows[m],
                                                    lambda m: mailbox[m], max_local, world, rank)
        ok &= list(m_all) == _uploaders(k)                          # every rank sees all uploads, ascending
        ok &= all(R_all[i] == _radius(m, k) for i, m in enumerate(m_all))
        for m in _uploaders(k):
            if m % world != rank:
                ok &= bool(torch.equal(mailbox[m], _row(m, k)))     # the owner's stream arrived
        for m in range(M):
            if m not in _uploaders(k):
                ok &= not mailbox[m].any()                          # a skipping worker sent nothing
        ok &= st["messages"] == len(mine) and st["payload_bytes"] == len(mine) * WORDS * 4
        sent_bytes += st["payload_bytes"]
    with open(os.path.join(out_dir, "rank%d.txt" % rank), "w") as f:
        f.write("%d %d" % (int(ok), sent_bytes))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_exchange_only_the_uploaders_messages(tmp_path):
    world, port = 2, 31000 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    total = 0
    for rank in range(world):
        ok, sent = (int(v) for v in open(tmp_path / ("rank%d.txt" % rank)).read().split())
        assert ok == 1
        total += sent
    # payload = one code stream per upload (the radius travels in the header)
    assert total == sum(len(_uploaders(k)) for k in range(ITERS)) * WORDS * 4


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_1909_07588_b200 import sharded
    m_all, R_all, st = sharded.exchange_uploads([1, 4], [0.5, 2.0], lambda m: None, lambda m: None, 5, 1, 0)
    assert list(m_all) == [1, 4] and list(R_all) == [0.5, 2.0] and st["payload_bytes"] == 0


def test_message_size_is_the_papers():
    sys.path.insert(0, ROOT)
    from paper_1909_07588_b200 import sharded
    assert sharded.message_bits(4, 7840) == 32 + 4 * 7840           # text after Eq. (6)
    assert [sharded.owner_of(m, 4) for m in range(6)] == [0, 1, 2, 3, 0, 1]
