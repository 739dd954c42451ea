"""Workers spread over several GPUs: the upload of Algorithm 2 as a real exchange (Fig. 2 of the paper).

Rank r runs steps 1-4 for the workers r, r + W, r + 2W, ... on its own GPU and holds their Q_m.  Every rank holds
theta, the aggregated gradient and the stored differences, and applies every upload, so the server's side is
replicated and no parameter broadcast is needed.  What crosses the wire per iteration is exactly the paper's
message (text after Eq. (6)): for every UPLOADING worker its radius (32 bits) and its b p-bit code stream; a worker
that skips sends nothing but its place in a small header.

    exchange_uploads    the collective part, on plain torch tensors (CPU tensors with gloo, CUDA tensors with NCCL)
    ShardedLaq          one context per rank driven through laq_step_local / laq_local_uploads / laq_apply_uploads

The exchange uses torch.distributed only: an all-gather of the fixed-size header and one broadcast per uploader from
its owner into the other ranks' mailboxes (received rows land in this GPU's own memory before any kernel reads them).
"""
import numpy as np


def owner_of(m, world):
    """Rank that runs worker m."""
    return m % world


def message_bits(b, p):
    """Bits of one upload: the radius and p codes of b bits."""
    return 32 + b * p


def exchange_uploads(local_m, local_R, send_row, recv_row, max_local, world, rank, group=None, device="cpu"):
    """Make every rank know every upload of the iteration and hold every remote uploader's code stream.

    local_m, local_R   this rank's uploaders (global worker indices, ascending) and their radii
    send_row(m)        tensor holding local uploader m's code stream (int32 words)
    recv_row(m)        tensor that receives remote uploader m's code stream
    max_local          largest number of workers any rank owns (header slots per rank)
    Returns (m_all, R_all, stats): all uploaders in ascending order, their radii, and
    stats = dict(messages=..., header_bytes=..., payload_bytes=...) for this rank's SENT traffic.
    """
    import torch
    import torch.distributed as dist
    n = len(local_m)
    assert n <= max_local
    # header: per slot the global index (-1 = empty) and the radius' bit pattern, as int32 pairs
    head = torch.full((max_local, 2), -1, dtype=torch.int32)
    if n:
        head[:n, 0] = torch.from_numpy(np.asarray(local_m, np.int32))
        head[:n, 1] = torch.from_numpy(np.asarray(local_R, np.float32).view(np.int32))
    head = head.to(device)
    if world > 1:
        heads = torch.empty((world, max_local, 2), dtype=torch.int32, device=device)
        dist.all_gather_into_tensor(heads.view(-1), head.view(-1), group=group)
    else:
        heads = head[None]
    heads = heads.cpu().numpy()
    entries = []
    for r in range(world):
        for slot in range(max_local):
            m = int(heads[r, slot, 0])
            if m >= 0:
                assert owner_of(m, world) == r, "a rank announced a worker it does not own"
                entries.append((m, heads[r, slot, 1:2].view(np.float32)[0]))
    entries.sort(key=lambda e: e[0])
    m_all = np.array([e[0] for e in entries], np.int32)
    R_all = np.array([e[1] for e in entries], np.float32)
    sent = 0
    if world > 1:
        works = []
        for m in m_all:                                   # same order on every rank
            src = owner_of(int(m), world)
            t = send_row(int(m)) if src == rank else recv_row(int(m))
            if src == rank:
                sent += t.numel() * t.element_size()
            src_global = dist.get_global_rank(group, src) if group is not None else src
            works.append(dist.broadcast(t, src=src_global, group=group, async_op=True))
        for wk in works:
            wk.wait()
    stats = dict(messages=n, header_bytes=int(head.numel() * 4), payload_bytes=int(sent))
    return m_all, R_all, stats


class ShardedLaq:
    """One LAQ context per rank, workers spread round robin.  `make_ctx(world, rank)` builds the rank's context
    (e.g. ``lambda w, r: laq.from_workload(workload, world=w, rank=r)``)."""

    def __init__(self, make_ctx, world, rank, group=None):
        self.world, self.rank, self.group = world, rank, group
        self.ctx = make_ctx(world, rank)
        self.max_local = (self.ctx.M_total + world - 1) // world
        self.sent_payload_bytes = 0
        self.sent_messages = 0

    def step(self, n_iters=1):
        c = self.ctx
        for _ in range(n_iters):
            c.step_local()
            m_loc, R_loc = c.local_uploads()
            m_all, R_all, st = exchange_uploads(
                m_loc, R_loc,
                send_row=lambda m: c.code_row((m - self.rank) // self.world),
                recv_row=lambda m: c.mailbox_row(m),
                max_local=self.max_local, world=self.world, rank=self.rank, group=self.group,
                device=c.workspace.device)
            self.sent_payload_bytes += st["payload_bytes"]
            self.sent_messages += st["messages"]
            c.apply_uploads(m_all, R_all)

    def close(self):
        self.ctx.close()
