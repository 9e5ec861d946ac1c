"""Helpers shared by the GPU parity tests (not a test module)."""
import numpy as np
import torch

from paper_2511_04214_b200 import synth


def gemm_scale_index(rows: int, K: int) -> np.ndarray:
    """Byte offset of every (row, group) in the tensor-core scale layout, as an int64 array
    [rows, K/32] (the documented formula, vectorised)."""
    r = np.arange(rows, dtype=np.int64)[:, None]
    g = np.arange(K // 32, dtype=np.int64)[None, :]
    kb = 2 * ((K + 255) // 256)
    return ((r // 128) * kb + g // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + (g % 4)


def to_canonical(scales_gemm: np.ndarray, rows: int, K: int) -> np.ndarray:
    return scales_gemm[gemm_scale_index(rows, K)]


def to_gemm_layout(scales_canon: np.ndarray, rows: int, K: int) -> np.ndarray:
    kb = 2 * ((K + 255) // 256)
    out = np.zeros(((rows + 127) // 128) * kb * 512, dtype=np.uint8)
    out[gemm_scale_index(rows, K)] = scales_canon
    return out


class Guarded:
    """A device byte buffer with poisoned guard bands before and after the payload."""
    PAD = 256

    def __init__(self, nbytes: int, fill: int = 0xA5):
        self.nbytes = nbytes
        self.fill = fill
        self.raw = torch.full((nbytes + 2 * self.PAD,), fill, dtype=torch.uint8, device="cuda")
        assert self.raw.data_ptr() % 256 == 0
        self.view = self.raw[self.PAD:self.PAD + nbytes]

    def check(self):
        head = self.raw[:self.PAD].cpu().numpy()
        tail = self.raw[self.PAD + self.nbytes:].cpu().numpy()
        assert (head == self.fill).all(), "write before the start of an output buffer"
        assert (tail == self.fill).all(), "write past the end of an output buffer"

    def numpy(self):
        return self.view.cpu().numpy()


def x_from_bits(bits: np.ndarray) -> torch.Tensor:
    return synth.bits_to_bf16(bits).cuda()
