"""Message exchange for the data-parallel step of Algorithm 1 ("broadcast M^i to all peers"):
rank = worker, every rank contributes one encoded message and receives all K of them.

Only plumbing lives here (torch.distributed collectives and slot arithmetic); encoding and
decoding stay in the kernels. Fixed-width messages all have the same, statically known size, so
one all-gather into a K-slot buffer suffices. Elias messages differ in length: the ranks first
all-gather their four info words, then all-gather the messages padded to the longest one. The
gathered slots sit in this GPU's own memory before any decode kernel reads them.
"""
import torch
import torch.distributed as dist

SLOT_ALIGN = 256


def slot_bytes(max_message_bytes):
    """Slot pitch of the gathered buffer: the longest message rounded up to SLOT_ALIGN."""
    return (int(max_message_bytes) + SLOT_ALIGN - 1) // SLOT_ALIGN * SLOT_ALIGN


def gather_info(info, group=None):
    """All-gathers the per-rank info words (int64[4]: payload bits, table offset, message bytes,
    0). Returns an int64 tensor [K, 4] on the same device."""
    world = dist.get_world_size(group)
    out = torch.empty(world, 4, dtype=torch.int64, device=info.device)
    dist.all_gather_into_tensor(out.view(-1), info.contiguous().view(-1), group=group)
    return out


def gather_messages(msg, pitch, group=None, out=None):
    """All-gathers one message per rank into K slots of `pitch` bytes. `msg` is a uint8 tensor
    holding at least `pitch` bytes (bytes past the message length are transmitted but ignored)."""
    world = dist.get_world_size(group)
    if msg.numel() < pitch:
        raise ValueError("message buffer shorter than the slot pitch")
    if out is None:
        out = torch.empty(world * pitch, dtype=torch.uint8, device=msg.device)
    dist.all_gather_into_tensor(out, msg[:pitch].contiguous(), group=group)
    return out


def slots(gathered, pitch, infos, n, bucket, elias):
    """Per-rank views into the gathered buffer: (messages, tables). tables is None for the
    fixed-width code; for the Elias codes table k starts at byte infos[k][1] of slot k."""
    world = infos.shape[0]
    B = (n + bucket - 1) // bucket
    msgs, tables = [], []
    info_host = infos.cpu().tolist()
    for k in range(world):
        base = k * pitch
        total = int(info_host[k][2])
        msgs.append(gathered[base: base + total])
        if elias:
            off = base + int(info_host[k][1])
            tables.append(gathered[off: off + 8 * (B + 1)].view(torch.int64))
    return msgs, (tables if elias else None)


def exchange(msg, info, n, bucket, elias, fixed_bytes=None, group=None):
    """One exchange step. Returns (msgs, tables, infos) ready for the decode entry points."""
    if elias:
        infos = gather_info(info, group)
        pitch = slot_bytes(int(infos[:, 2].max().item()))
    else:
        world = dist.get_world_size(group)
        infos = info.view(1, 4).repeat(world, 1)          # same size on every rank
        pitch = slot_bytes(fixed_bytes)
    gathered = gather_messages(msg, pitch, group)
    msgs, tables = slots(gathered, pitch, infos, n, bucket, elias)
    return msgs, tables, infos
