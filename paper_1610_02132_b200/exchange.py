"""Message exchange for the data-parallel step of Algorithm 1 ("broadcast M^i to all peers",
"receive M^l"): every rank contributes the messages of the workers it plays and receives all K.

Only plumbing lives here (torch.distributed collectives and slot arithmetic); encoding and
decoding stay in the kernels. A rank encodes its W workers' messages into W slots of one buffer
(slot pitch = the message capacity rounded up to SLOT_ALIGN); one all-gather puts the K = world * W
slots, in worker order, into this GPU's own memory, and a second small all-gather does the same
for the four info words of each message. The decode entry points of the packed form
(qsgd_decode_*_packed) take exactly that: slot pointers, info-word pointers and the slot pitch as
the readable size; they find each offset table on the device, so the exchange needs no host
synchronisation at all.

Elias messages are shorter than their capacity. `exact=True` sends only as many bytes per slot
as the longest message of the step needs; that costs one host read-back of the gathered sizes
(32 bytes per message), which a sender of variable-length messages cannot avoid.
"""
import torch
import torch.distributed as dist

SLOT_ALIGN = 256


def slot_bytes(max_message_bytes):
    """Slot pitch of the gathered buffer: the longest message rounded up to SLOT_ALIGN."""
    return (int(max_message_bytes) + SLOT_ALIGN - 1) // SLOT_ALIGN * SLOT_ALIGN


class Exchange:
    """Buffers of one rank for a fixed message capacity: W local slots, K gathered slots, the info
    words of both. Allocated once; every step reuses them (slot and info addresses stay put, so a
    step's launches can be replayed)."""

    def __init__(self, capacity, workers_per_rank, device, group=None):
        self.group = group
        self.world = dist.get_world_size(group)
        self.W = int(workers_per_rank)
        self.K = self.world * self.W
        self.pitch = slot_bytes(capacity)
        self.local = torch.zeros(self.W * self.pitch, dtype=torch.uint8, device=device)
        self.local_info = torch.zeros(self.W, 4, dtype=torch.int64, device=device)
        self.gathered = torch.zeros(self.K * self.pitch, dtype=torch.uint8, device=device)
        self.infos = torch.zeros(self.K, 4, dtype=torch.int64, device=device)
        self._exact = None

    def local_slot(self, w):
        """Message buffer of local worker w (encode into this), and its info words."""
        return self.local[w * self.pitch: (w + 1) * self.pitch], self.local_info[w]

    def run(self, exact=False, with_info=True):
        """All-gathers the info words (Elias kinds need them; with_info=False skips it for the
        fixed-width code) and the slots. Returns (msgs, infos, msg_bytes): K slot views in worker
        order, K info-word views, and the readable bytes of each slot."""
        if with_info or exact:
            dist.all_gather_into_tensor(self.infos.view(-1), self.local_info.view(-1), group=self.group)
        pitch = self.pitch
        if exact:
            pitch = min(slot_bytes(int(self.infos[:, 2].max().item())), self.pitch)    # the one host read-back
        if pitch == self.pitch:
            gathered = self.gathered
            dist.all_gather_into_tensor(gathered, self.local, group=self.group)
        else:
            if self._exact is None or self._exact.numel() < self.K * pitch:
                self._exact = torch.empty(self.K * pitch, dtype=torch.uint8, device=self.local.device)
            gathered = self._exact[: self.K * pitch]
            send = self.local.view(self.W, self.pitch)[:, :pitch].contiguous().view(-1)
            dist.all_gather_into_tensor(gathered, send, group=self.group)
        msgs = [gathered[k * pitch: (k + 1) * pitch] for k in range(self.K)]
        infos = [self.infos[k] for k in range(self.K)]
        return msgs, infos, [pitch] * self.K
