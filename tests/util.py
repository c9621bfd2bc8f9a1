"""Helpers shared by the GPU parity tests: numpy bf16 bit patterns <-> torch device tensors."""
import numpy as np
import torch


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> bfloat16 CUDA tensor (bit-exact)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.cuda().view(torch.bfloat16)


def bits(t: torch.Tensor) -> np.ndarray:
    """Any 16-bit CUDA tensor -> numpy uint16 bit patterns."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def rel_fro(got: np.ndarray, ref: np.ndarray) -> float:
    g, r = got.astype(np.float64), ref.astype(np.float64)
    return float(np.linalg.norm(g - r) / max(np.linalg.norm(r), 1e-30))


def assert_close_elementwise(got: np.ndarray, ref: np.ndarray, K: int, what: str = "") -> None:
    """Element-wise bound for a bf16 output of a length-K float32-accumulated product against its
    float64 reference: half an output ulp is at most 2^-8 |ref| (2^-7 allows one flipped rounding),
    and K float32 additions of partial sums of size ~rms(ref) contribute at most K 2^-23 each with a
    small-integer factor for peaks, bounded here by K 2^-20 rms(ref). A wrong tile, chunk or row
    band produces errors of the order of rms(ref) itself and fails this where a norm over 10^7
    elements would not move."""
    g, r = got.astype(np.float64), ref.astype(np.float64)
    rms = float(np.sqrt(np.mean(r * r)))
    tol = 2.0 ** -7 * np.abs(r) + max(K, 64) * 2.0 ** -20 * rms
    bad = np.abs(g - r) > tol
    if bad.any():
        idx = np.argwhere(bad)
        i = tuple(idx[0])
        raise AssertionError(f"{what}: {int(bad.sum())} of {bad.size} elements outside the element-wise bound; "
                             f"first at {i}: got {g[i]!r}, ref {r[i]!r}, tol {tol[i]!r}; "
                             f"rows {idx[:, 0].min()}..{idx[:, 0].max()}, cols {idx[:, -1].min()}..{idx[:, -1].max()}")


CANARY_BYTES = 256
_CANARY = 0xA5


class Guarded:
    """A device buffer with 256 bytes of a known pattern on either side (the stand-in for a memory
    checker): ``t`` is the payload tensor handed to the library, ``check()`` asserts that no byte of
    the two guard zones changed."""

    def __init__(self, nbytes_or_shape, dtype=torch.uint8, zero: bool = False):
        shape = (nbytes_or_shape,) if isinstance(nbytes_or_shape, int) else tuple(nbytes_or_shape)
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        pad = (-n) % CANARY_BYTES
        self.raw = torch.full((CANARY_BYTES + n + pad + CANARY_BYTES,), _CANARY, dtype=torch.uint8, device="cuda")
        self.n, self.pad = n, pad
        self.t = self.raw[CANARY_BYTES:CANARY_BYTES + n].view(dtype).view(shape)
        if zero:
            self.t.zero_()

    def check(self, what: str = "") -> None:
        lo = self.raw[:CANARY_BYTES]
        hi = self.raw[CANARY_BYTES + self.n:]
        assert bool((lo == _CANARY).all()), f"{what}: bytes before the buffer were overwritten"
        assert bool((hi == _CANARY).all()), f"{what}: bytes after the buffer were overwritten"
