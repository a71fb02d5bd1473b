"""Shared helpers of the GPU parity tests: host <-> device marshalling and the comparison rules."""
import numpy as np
import torch


def bf16_dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def bf16_bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def canon_fp4(packed):
    """Map the negative-zero nibble 0x8 to 0x0 (FP4 codes are compared by value)."""
    p = np.asarray(packed, dtype=np.uint8)
    lo, hi = p & 15, p >> 4
    lo = np.where(lo == 8, 0, lo)
    hi = np.where(hi == 8, 0, hi)
    return (lo | (hi << 4)).astype(np.uint8)


def rel_row_err(y, ref):
    """max_j |y - ref| / ||ref[i,:]||_2 per row (the parity metric: <= 1e-3)."""
    y = np.asarray(y, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    n = np.linalg.norm(ref, axis=-1)
    n = np.where(n == 0, 1.0, n)
    return np.abs(y - ref).max(axis=-1) / n


class GuardedAllocator:
    """Stand-in for the closed memory checker: every output tensor and workspace the binding creates sits between two
    bands of canary bytes; ``check()`` fails when a kernel wrote outside what it was given."""
    PAD = 4096            # bytes on either side (a multiple of every alignment the library asks for)
    CANARY = 0xA5

    def __init__(self):
        self.bufs = []

    def _carve(self, nbytes, device, fill=None):
        buf = torch.full((self.PAD + nbytes + self.PAD,), self.CANARY, dtype=torch.uint8, device=device)
        inner = buf[self.PAD:self.PAD + nbytes]
        if fill is not None:
            inner.fill_(fill)
        self.bufs.append((buf, nbytes))
        return inner

    def empty(self, shape, dtype, device):
        shape = tuple(shape) if isinstance(shape, (tuple, list, torch.Size)) else (int(shape),)
        n = 1
        for d in shape:
            n *= int(d)
        esz = torch.empty((), dtype=dtype).element_size()
        # outputs start as 0xA5 bytes too: an element the kernel forgot to write does not look like a result
        return self._carve(n * esz, device).view(dtype).view(shape)

    def workspace(self, nbytes, device="cuda"):
        return self._carve(max(int(nbytes), 1024) + 1024, device, fill=0)

    def check(self):
        torch.cuda.synchronize()
        for buf, n in self.bufs:
            head, tail = buf[:self.PAD], buf[self.PAD + n:]
            assert bool((head == self.CANARY).all()), "a kernel wrote BEFORE a buffer it was given"
            assert bool((tail == self.CANARY).all()), "a kernel wrote PAST a buffer it was given"
        self.bufs.clear()
