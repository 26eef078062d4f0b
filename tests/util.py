"""Test-side helpers: an independent numpy bit packer / unpacker and guard-region buffers.

None of this is shared with the CUDA library or with the oracle.
"""
import numpy as np
import torch


def words_per_row(K: int) -> int:
    return (K + 31) // 32


def pack_bits_ref(bits01: np.ndarray, ld_words: int = 0) -> np.ndarray:
    """uint8 0/1 [rows, K] -> uint32 [rows, ld_words]; element k -> bit k%32 of word k//32; pads zero."""
    rows, K = bits01.shape
    kw = words_per_row(K)
    ld = max(ld_words, kw)
    padded = np.zeros((rows, ld * 32), np.uint8)
    padded[:, :K] = bits01
    by = np.packbits(padded, axis=1, bitorder="little")            # [rows, ld*4] bytes, little-endian words
    return by.view("<u4").reshape(rows, ld).copy()


def unpack_words(words: np.ndarray, K: int) -> np.ndarray:
    """uint32 [rows, ld] -> uint8 0/1 [rows, K]; also asserts that pad bits of the used words are zero."""
    rows, ld = words.shape
    kw = words_per_row(K)
    by = np.ascontiguousarray(words[:, :kw].astype("<u4")).view(np.uint8).reshape(rows, kw * 4)
    bits = np.unpackbits(by, axis=1, bitorder="little")
    assert not bits[:, K:].any(), "pad bits must be zero"
    return bits[:, :K].copy()


GUARD = 0xA5


class Guarded:
    """A device buffer with 0xA5-filled guard zones before and after the payload."""

    def __init__(self, shape, dtype, device="cuda", guard_bytes=1024, fill=None):
        self.shape = tuple(shape)
        self.dtype = dtype
        n = int(np.prod(self.shape)) if len(self.shape) else 1
        self.nbytes = n * torch.empty(0, dtype=dtype).element_size()
        self.guard = guard_bytes
        self.raw = torch.full((self.nbytes + 2 * guard_bytes,), GUARD, dtype=torch.uint8, device=device)
        self.t = self.raw[guard_bytes:guard_bytes + self.nbytes].view(dtype).reshape(self.shape)
        if fill is not None:
            self.t.fill_(fill)

    def check(self):
        g = self.guard
        head = self.raw[:g].cpu().numpy()
        tail = self.raw[g + self.nbytes:].cpu().numpy()
        assert (head == GUARD).all(), "write before the start of an output buffer"
        assert (tail == GUARD).all(), "write past the end of an output buffer"


def dev(t, dtype=None):
    if isinstance(t, np.ndarray):
        t = torch.from_numpy(np.ascontiguousarray(t))
    if dtype is not None:
        t = t.to(dtype)
    return t.contiguous().cuda()


def as_i32_words(a: np.ndarray) -> torch.Tensor:
    """uint32 numpy words -> int32 torch tensor with the same bytes (torch has limited uint32 support)."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int32))


def words_np(t: torch.Tensor) -> np.ndarray:
    """int32 torch tensor (device or host) holding packed words -> uint32 numpy array."""
    return t.detach().cpu().numpy().view(np.uint32)
